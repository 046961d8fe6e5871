"""ctypes/numpy wrapper around the C oracle (oracle/mv_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the benchmark's
cpu-baseline leg.  The product path never imports this module, and this module never
imports the CUDA binding.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_LIB_PATH = _HERE / "libmv_oracle.so"
_lib = None


class Desc(C.Structure):
    _fields_ = [("gx", C.c_int32), ("gy", C.c_int32), ("gz", C.c_int32), ("max_boxes", C.c_int32),
                ("width", C.c_int32), ("height", C.c_int32), ("palette_size", C.c_int32),
                ("hfov", C.c_double), ("light_dir", C.c_double * 3), ("ambient", C.c_double),
                ("sky_rgb", C.c_uint8 * 3), ("pad", C.c_uint8), ("miss_depth", C.c_float)]


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (strict IEEE: no contraction, no fast-math)."""
    src = _HERE / "mv_oracle.c"
    if force or not _LIB_PATH.exists() or _LIB_PATH.stat().st_mtime < src.stat().st_mtime:
        tmp = _LIB_PATH.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp",
                               "-ffp-contract=off", "-fno-fast-math", "-o", str(tmp), str(src), "-lm"])
        os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(str(_LIB_PATH))
        _lib.mvo_render_obs.restype = C.c_int
        _lib.mvo_render_pixels.restype = C.c_int
    return _lib


def make_desc(grid_shape, max_boxes, width, height, palette_size, hfov=np.pi / 2,
              light_dir=(0.36, 0.80, 0.48), ambient=0.3, sky_rgb=(127, 178, 229), miss_depth=0.0):
    gy, gz, gx = grid_shape
    d = Desc()
    d.gx, d.gy, d.gz, d.max_boxes = gx, gy, gz, max_boxes
    d.width, d.height, d.palette_size = width, height, palette_size
    # the C ABI under test carries these four as float32, so the definition is evaluated (in
    # double) from the float32-rounded values
    d.hfov = float(np.float32(hfov))
    d.light_dir = (C.c_double * 3)(*[float(np.float32(x)) for x in light_dir])
    d.ambient = float(np.float32(ambient))
    d.sky_rgb = (C.c_uint8 * 3)(*[int(x) for x in sky_rgb])
    d.miss_depth = float(miss_depth)
    return d


def desc_from_config(cfg) -> Desc:
    gx, gy, gz = cfg.grid
    return make_desc((gy, gz, gx), cfg.max_boxes, cfg.width, cfg.height, cfg.palette_size,
                     cfg.hfov_rad, cfg.light_dir, cfg.ambient, cfg.sky_rgb, cfg.miss_depth)


def _ptr(a, t):
    return a.ctypes.data_as(C.POINTER(t)) if a is not None and a.size else None


def _unpack_cam(cam_row):
    """cam_row: int32[6] = float bits of (pos, yaw, pitch) + self_box."""
    cam_row = np.ascontiguousarray(cam_row, dtype=np.int32)
    f = cam_row[:5].view(np.float32)
    return np.ascontiguousarray(f[:3]), float(f[3]), float(f[4]), int(cam_row[5])


def render_obs(desc: Desc, grid, boxes, box_count, palette, cam_row):
    """One observation.  grid uint8[gy][gz][gx]; boxes int32[max_boxes][8] (or None);
    palette uint8[P][3]; cam_row int32[6].  Returns rgb[H][W][3], depth[H][W], id[H][W][3]."""
    W, H = desc.width, desc.height
    grid = np.ascontiguousarray(grid, dtype=np.uint8)
    palette = np.ascontiguousarray(palette, dtype=np.uint8)
    boxes = None if boxes is None else np.ascontiguousarray(boxes, dtype=np.int32)
    pos, yaw, pitch, self_box = _unpack_cam(cam_row)
    rgb = np.empty((H, W, 3), np.uint8)
    depth = np.empty((H, W), np.float32)
    ids = np.empty((H, W, 3), np.int32)
    r = lib().mvo_render_obs(C.byref(desc), _ptr(grid, C.c_uint8), _ptr(boxes, C.c_int32),
                             C.c_int(int(box_count)), _ptr(palette, C.c_uint8), _ptr(pos, C.c_float),
                             C.c_float(yaw), C.c_float(pitch), C.c_int(self_box),
                             _ptr(rgb, C.c_uint8), _ptr(depth, C.c_float), _ptr(ids, C.c_int32))
    if r < 0:
        raise RuntimeError(f"mvo_render_obs failed: {r}")
    return rgb, depth, ids


def render_pixels(desc: Desc, grid, boxes, box_count, palette, cam_row, pxy, oxy=None):
    """Selected pixels (pxy int32[n][2] = column,row) with optional sub-pixel offsets oxy[n][2]."""
    grid = np.ascontiguousarray(grid, dtype=np.uint8)
    palette = np.ascontiguousarray(palette, dtype=np.uint8)
    boxes = None if boxes is None else np.ascontiguousarray(boxes, dtype=np.int32)
    pxy = np.ascontiguousarray(pxy, dtype=np.int32).reshape(-1, 2)
    n = pxy.shape[0]
    oxy = None if oxy is None else np.ascontiguousarray(oxy, dtype=np.float64).reshape(n, 2)
    pos, yaw, pitch, self_box = _unpack_cam(cam_row)
    rgb = np.empty((n, 3), np.uint8)
    depth = np.empty((n,), np.float32)
    ids = np.empty((n, 3), np.int32)
    r = lib().mvo_render_pixels(C.byref(desc), _ptr(grid, C.c_uint8), _ptr(boxes, C.c_int32),
                                C.c_int(int(box_count)), _ptr(palette, C.c_uint8), _ptr(pos, C.c_float),
                                C.c_float(yaw), C.c_float(pitch), C.c_int(self_box), C.c_int(n),
                                _ptr(pxy, C.c_int32), _ptr(oxy, C.c_double),
                                _ptr(rgb, C.c_uint8), _ptr(depth, C.c_float), _ptr(ids, C.c_int32))
    if r < 0:
        raise RuntimeError(f"mvo_render_pixels failed: {r}")
    return rgb, depth, ids


def threads_used() -> int:
    """Threads the oracle's OpenMP loop runs on (what a render call returns)."""
    return int(os.environ.get("OMP_NUM_THREADS", 0)) or len(os.sched_getaffinity(0))


def render_scene(cfg, scene: dict, obs_indices=None):
    """Observations of a generated scene (arrays from paper_2107_08170_b200.scenes, as torch CPU
    tensors or numpy).  obs_indices index the scene's local observations.  Returns stacked
    rgb[n][H][W][3], depth[n][H][W], id[n][H][W][3]."""
    def np_(x):
        return x.cpu().numpy() if hasattr(x, "cpu") else np.asarray(x)
    grid, boxes, count = np_(scene["grid"]), np_(scene["boxes"]), np_(scene["box_count"])
    palette, cams = np_(scene["palette"]), np_(scene["cams"])
    desc = desc_from_config(cfg)
    A = cfg.agents
    idx = range(cams.shape[0]) if obs_indices is None else obs_indices
    out = []
    for o in idx:
        e = o // A
        b = boxes[e] if boxes.shape[1] > 0 else None
        out.append(render_obs(desc, grid[e], b, count[e], palette[e], cams[o]))
    rgb = np.stack([x[0] for x in out]); depth = np.stack([x[1] for x in out]); ids = np.stack([x[2] for x in out])
    return rgb, depth, ids


RECT_DTYPE = np.dtype([("x0", "<i2"), ("y0", "<i2"), ("x1", "<i2"), ("y1", "<i2"),
                       ("rgb", "u1", (3,)), ("pad0", "u1"), ("pad1", "<u4")])
assert RECT_DTYPE.itemsize == 16


def overlay(rgb, rects, count):
    """Paint `count` rectangles (RECT_DTYPE records) over one frame rgb[H][W][3], in place."""
    H, W, _ = rgb.shape
    rects = np.ascontiguousarray(rects, dtype=RECT_DTYPE)
    assert rgb.flags["C_CONTIGUOUS"] and rgb.dtype == np.uint8
    lib().mvo_overlay(C.c_int(W), C.c_int(H), rects.ctypes.data_as(C.c_void_p), C.c_int(int(count)),
                      rgb.ctypes.data_as(C.c_void_p))
    return rgb


def move_agent(grid, cam5, move4, shape3=(0.25, 0.75, 0.25), max_pitch=1.0):
    """One agent: cam5 = float32 (x,y,z,yaw,pitch) -> (new cam5, kept bits)."""
    grid = np.ascontiguousarray(grid, dtype=np.uint8)
    gy, gz, gx = grid.shape
    cam = np.array(cam5, dtype=np.float32).copy()
    move = np.array(move4, dtype=np.float32)
    shape = np.array(shape3, dtype=np.float32)
    L = lib()
    L.mvo_move_agent.restype = C.c_int
    kept = L.mvo_move_agent(_ptr(grid, C.c_uint8), C.c_int(gx), C.c_int(gy), C.c_int(gz), _ptr(cam, C.c_float),
                            _ptr(move, C.c_float), _ptr(shape, C.c_float), C.c_float(float(np.float32(max_pitch))))
    return cam, kept


def merge_voxels(grid, palette_size, max_out=4096):
    """Greedy voxel merging of one env: returns (boxes int32[count][8] in the C ABI's box layout,
    total count the pass produces)."""
    grid = np.ascontiguousarray(grid, dtype=np.uint8)
    gy, gz, gx = grid.shape
    out = np.zeros((max_out, 8), np.int32)
    L = lib()
    L.mvo_merge_voxels.restype = C.c_int
    n = L.mvo_merge_voxels(_ptr(grid, C.c_uint8), C.c_int(gx), C.c_int(gy), C.c_int(gz), C.c_int(palette_size),
                           out.ctypes.data_as(C.c_void_p), C.c_int(max_out))
    if n < 0:
        raise RuntimeError(f"mvo_merge_voxels failed: {n}")
    return out[:min(n, max_out)], n
