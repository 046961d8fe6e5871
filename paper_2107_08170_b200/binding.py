"""Thin ctypes binding over the C ABI in include/mv.h: argument marshalling only.

torch is used for device memory and streams; every step of the render path runs in the CUDA
library.  There is no fallback: if `libmv_b200.so` is missing or fails to load, calls raise.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libmv_b200.so"
_lib = None

MV_OK = 0
FLAG_MATERIAL_CLAMPED, FLAG_BOX_COUNT_CLAMPED, FLAG_BAD_CAMERA, FLAG_DEVICE_TIMEOUT = 1, 2, 4, 8
EXPORTS = ["mv_create_batch", "mv_upload_worlds", "mv_upload_worlds_at", "mv_set_cameras", "mv_render_batch", "mv_step_host",
           "mv_step_host_static", "mv_set_overlays", "mv_move_agents", "mv_merge_voxels", "mv_debug_staging", "mv_debug_occupancy_in_global", "mv_debug_agents_per_cta", "mv_query_status", "mv_launch_count", "mv_destroy", "mv_status_string"]


class BatchDesc(C.Structure):
    _fields_ = [("num_envs", C.c_int32), ("agents_per_env", C.c_int32),
                ("grid_x", C.c_int32), ("grid_y", C.c_int32), ("grid_z", C.c_int32),
                ("max_boxes", C.c_int32), ("width", C.c_int32), ("height", C.c_int32),
                ("palette_size", C.c_int32), ("hfov_rad", C.c_float), ("light_dir", C.c_float * 3),
                ("ambient", C.c_float), ("sky_rgb", C.c_uint8 * 3), ("pad", C.c_uint8),
                ("miss_depth", C.c_float), ("device", C.c_int32), ("max_overlay_rects", C.c_int32)]


class MvError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


def lib() -> C.CDLL:
    """Load the CUDA library (fails loudly when it has not been built)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: run `python -m paper_2107_08170_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(str(_LIB_PATH))
        vp, i = C.c_void_p, C.c_int
        L.mv_create_batch.argtypes = [C.POINTER(BatchDesc), C.POINTER(vp)]
        L.mv_upload_worlds.argtypes = [vp, i, i, vp, vp, vp, vp, vp]
        L.mv_upload_worlds_at.argtypes = [vp, i, vp, vp, vp, vp, vp, vp]
        L.mv_set_cameras.argtypes = [vp, vp, vp]
        L.mv_render_batch.argtypes = [vp, vp, vp, vp]
        L.mv_step_host.argtypes = [vp, vp, vp, vp, vp, vp, vp]
        L.mv_step_host_static.argtypes = [vp, vp, vp, vp, vp]
        L.mv_set_overlays.argtypes = [vp, vp, vp, vp]
        L.mv_move_agents.argtypes = [vp, vp, vp, vp, vp]
        L.mv_merge_voxels.argtypes = [vp, i, i, vp, vp, i, vp]
        L.mv_debug_staging.argtypes = [vp, i, i]
        L.mv_debug_occupancy_in_global.argtypes = [vp, i]
        L.mv_debug_agents_per_cta.argtypes = [vp, i]
        L.mv_query_status.argtypes = [vp, i, vp]
        L.mv_launch_count.argtypes = [vp]
        L.mv_launch_count.restype = C.c_int64
        L.mv_destroy.argtypes = [vp]
        L.mv_status_string.argtypes = [i]
        L.mv_status_string.restype = C.c_char_p
        for n in [e for e in EXPORTS if e not in ("mv_launch_count", "mv_status_string")]:
            getattr(L, n).restype = i
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().mv_status_string(int(code)).decode()


def _check(code: int, where: str):
    if code != MV_OK:
        raise MvError(code, where)


def make_desc(num_envs, agents_per_env, grid, max_boxes, width, height, palette_size, hfov_rad=None,
              light_dir=(0.36, 0.80, 0.48), ambient=0.3, sky_rgb=(127, 178, 229), miss_depth=0.0,
              device=0, max_overlay_rects=0) -> BatchDesc:
    import math
    d = BatchDesc()
    d.num_envs, d.agents_per_env = num_envs, agents_per_env
    d.grid_x, d.grid_y, d.grid_z = grid
    d.max_boxes, d.width, d.height, d.palette_size = max_boxes, width, height, palette_size
    d.hfov_rad = math.pi / 2 if hfov_rad is None else hfov_rad
    d.light_dir = (C.c_float * 3)(*light_dir)
    d.ambient = ambient
    d.sky_rgb = (C.c_uint8 * 3)(*sky_rgb)
    d.miss_depth = miss_depth
    d.device = device
    d.max_overlay_rects = max_overlay_rects
    return d


class BodyShape(C.Structure):
    _fields_ = [("half_width", C.c_float), ("below_eye", C.c_float), ("above_eye", C.c_float),
                ("max_pitch", C.c_float)]


def desc_from_config(cfg, device=0, max_overlay_rects=0) -> BatchDesc:
    return make_desc(cfg.num_envs, cfg.agents, cfg.grid, cfg.max_boxes, cfg.width, cfg.height,
                     cfg.palette_size, cfg.hfov_rad, cfg.light_dir, cfg.ambient, cfg.sky_rgb,
                     cfg.miss_depth, device, max_overlay_rects)


def _dptr(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _hptr(t, dtype=None):
    if t is None:
        return None
    if t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CPU tensor")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


class Batch:
    """Handle to one mv_batch.  Methods mirror the C entry points one to one."""

    def __init__(self, desc: BatchDesc):
        self.desc = desc
        self._h = C.c_void_p()
        _check(lib().mv_create_batch(C.byref(desc), C.byref(self._h)), "mv_create_batch")
        self.num_obs = desc.num_envs * desc.agents_per_env

    def upload_worlds(self, env_begin, env_count, grid=None, boxes=None, box_count=None, palette=None,
                      stream=None):
        _check(lib().mv_upload_worlds(self._h, env_begin, env_count, _dptr(grid, torch.uint8),
                                      _dptr(boxes, torch.int32), _dptr(box_count, torch.int32),
                                      _dptr(palette, torch.uint8), _stream(stream)), "mv_upload_worlds")

    def upload_worlds_at(self, env_index, grid=None, boxes=None, box_count=None, palette=None, stream=None):
        """env_index: strictly increasing env numbers (any int sequence or CPU tensor); the arrays hold
        one entry per listed env."""
        idx = torch.as_tensor(env_index, dtype=torch.int32, device="cpu").contiguous()
        _check(lib().mv_upload_worlds_at(self._h, idx.numel(), C.c_void_p(idx.data_ptr()), _dptr(grid, torch.uint8),
                                         _dptr(boxes, torch.int32), _dptr(box_count, torch.int32),
                                         _dptr(palette, torch.uint8), _stream(stream)), "mv_upload_worlds_at")

    def set_cameras(self, cams, stream=None):
        _check(lib().mv_set_cameras(self._h, _dptr(cams, torch.int32), _stream(stream)), "mv_set_cameras")

    def render_batch(self, rgb, depth, stream=None):
        _check(lib().mv_render_batch(self._h, _dptr(rgb, torch.uint8), _dptr(depth, torch.float32),
                                     _stream(stream)), "mv_render_batch")

    def step_host(self, cams, rgb, depth, boxes=None, box_count=None, stream=None):
        _check(lib().mv_step_host(self._h, _hptr(cams, torch.int32), _hptr(boxes, torch.int32),
                                  _hptr(box_count, torch.int32), _hptr(rgb, torch.uint8),
                                  _hptr(depth, torch.float32), _stream(stream)), "mv_step_host")

    def set_overlays(self, rects=None, count=None, stream=None):
        """rects: CUDA int32 [num_obs][max_overlay_rects][4] (the 16-byte records viewed as int32), or None."""
        _check(lib().mv_set_overlays(self._h, _dptr(rects, torch.int32), _dptr(count, torch.int32),
                                     _stream(stream)), "mv_set_overlays")

    def move_agents(self, cams, moves, shape=None, stream=None):
        """cams: CUDA int32 [num_obs][6], updated in place; moves: CUDA float32 [num_obs][4]."""
        sp = None
        if shape is not None:
            sp = C.byref(BodyShape(*shape))
        _check(lib().mv_move_agents(self._h, _dptr(cams, torch.int32), _dptr(moves, torch.float32), sp,
                                    _stream(stream)), "mv_move_agents")

    def merge_voxels(self, env_begin, env_count, max_out, stream=None):
        """Greedy voxel merge; returns (boxes int32 [env_count][max_out][8], counts int32 [env_count]) on the GPU."""
        dev = torch.device("cuda", self.desc.device)
        boxes = torch.zeros(env_count, max_out, 8, dtype=torch.int32, device=dev)
        counts = torch.zeros(env_count, dtype=torch.int32, device=dev)
        _check(lib().mv_merge_voxels(self._h, env_begin, env_count, _dptr(boxes), _dptr(counts), max_out,
                                     _stream(stream)), "mv_merge_voxels")
        return boxes, counts

    def step_host_static(self, cams, rgb, depth, stream=None):
        """The never-allocating host step (fixed 8 MiB device array inside the library): for callers
        that may not allocate GPU memory while running.  Raises MvError(-6) if the batch is too big."""
        _check(lib().mv_step_host_static(self._h, _hptr(cams, torch.int32), _hptr(rgb, torch.uint8),
                                         _hptr(depth, torch.float32), _stream(stream)), "mv_step_host_static")

    def debug_occupancy_in_global(self, on: bool):
        _check(lib().mv_debug_occupancy_in_global(self._h, int(on)), "mv_debug_occupancy_in_global")

    def debug_agents_per_cta(self, agents_per_cta: int):
        """1 = a CTA per observation, agents_per_env = a CTA per environment, 0 = the library's choice."""
        _check(lib().mv_debug_agents_per_cta(self._h, int(agents_per_cta)), "mv_debug_agents_per_cta")

    def debug_staging(self, skip_staging: bool, wait_polls: int = 1 << 18):
        _check(lib().mv_debug_staging(self._h, int(skip_staging), int(wait_polls)), "mv_debug_staging")

    def query_status(self, clear=False, stream=None) -> int:
        r = lib().mv_query_status(self._h, int(clear), _stream(stream))
        if r < 0:
            raise MvError(r, "mv_query_status")
        return r

    def launch_count(self) -> int:
        return int(lib().mv_launch_count(self._h))

    def alloc_outputs(self):
        dev = torch.device("cuda", self.desc.device)
        rgb = torch.empty(self.num_obs, self.desc.height, self.desc.width, 3, dtype=torch.uint8, device=dev)
        depth = torch.empty(self.num_obs, self.desc.height, self.desc.width, dtype=torch.float32, device=dev)
        return rgb, depth

    def destroy(self):
        if self._h:
            h, self._h = self._h, C.c_void_p()
            _check(lib().mv_destroy(h), "mv_destroy")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass
