"""Seeded synthetic scene generators (inputs only; no rendering arithmetic lives here).

Both the CUDA library's tests/benchmark and the CPU oracle's tests draw their inputs from
this module, so the two sides always see byte-identical worlds, boxes and cameras.  The
scenes stand in for the paper's procedurally generated Megaverse-8 layouts (Section 4 and
Appendix B of the paper: voxel-grid rooms, obstacle courses, movable boxes, agent bodies),
whose generators are not published in the paper text.

Everything is derived from a counter-based integer hash (a splitmix64-style finaliser on
int64 tensors), so a generator gives the same arrays on the CPU and on a CUDA device and
any environment range can be generated on its own (chunked generation of large batches).

Array conventions (these are the C ABI's conventions, see include/mv.h):
  grid     uint8  [E][gy][gz][gx]   material id per voxel, 0 = empty, x fastest
  boxes    int32  [E][max_boxes][8] = {min xyz, max xyz} as float32 bit patterns, material, pad
  box_count int32 [E]
  palette  uint8  [E][P][3]
  cams     int32  [E*A][6] = {pos xyz, yaw, pitch} as float32 bit patterns, self_box
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import torch

_MASK64 = (1 << 64) - 1


def _i64(v: int) -> int:
    v &= _MASK64
    return v - (1 << 64) if v >= (1 << 63) else v


_C1 = _i64(0xBF58476D1CE4E5B9)
_C2 = _i64(0x94D049BB133111EB)
_GOLD = _i64(0x9E3779B97F4A7C15)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _C1
    x = (x ^ _lsr(x, 27)) * _C2
    return x ^ _lsr(x, 31)


class Rng:
    """Counter-based generator: value = hash(seed, stream, env, index)."""

    def __init__(self, seed: int, device="cpu"):
        self.seed = int(seed)
        self.device = torch.device(device)

    def _key(self, stream: int, env: torch.Tensor, idx: torch.Tensor) -> torch.Tensor:
        base = _i64((self.seed * 0x9E3779B97F4A7C15 + stream * 0xD1B54A32D192ED03) & _MASK64)
        k = _mix(env.to(torch.int64) * _GOLD + base)
        return _mix(k + idx.to(torch.int64) * _C2 + stream)

    def bits32(self, stream: int, env: torch.Tensor, idx: torch.Tensor) -> torch.Tensor:
        return _lsr(self._key(stream, env, idx), 32)

    def uniform(self, stream, env, idx) -> torch.Tensor:
        """float64 in [0, 1) with 32 random bits (exact on every device)."""
        return self.bits32(stream, env, idx).to(torch.float64) * (1.0 / 4294967296.0)

    def randint(self, stream, env, idx, lo: int, hi: int) -> torch.Tensor:
        """int64 in [lo, hi] inclusive."""
        n = hi - lo + 1
        return lo + ((self.bits32(stream, env, idx) * n) >> 32)

    def normal(self, stream, env, idx) -> torch.Tensor:
        """Approximately N(0,1): sum of 12 uniforms minus 6 (exact float64 arithmetic)."""
        acc = torch.zeros(torch.broadcast_shapes(env.shape, idx.shape), dtype=torch.float64,
                          device=self.device)
        for j in range(12):
            acc = acc + self.uniform(stream * 16 + j + 1000, env, idx)
        return acc - 6.0


@dataclass
class SceneConfig:
    name: str
    num_envs: int
    agents: int
    grid: tuple            # (gx, gy, gz)
    width: int
    height: int
    palette_size: int
    world: str             # "segments" | "rooms" | "columns"
    movable_boxes: int = 0
    body_boxes: bool = False
    cam_y_fixed: float | None = None
    seed: int = 0
    hfov_rad: float = math.pi / 2
    light_dir: tuple = (0.36, 0.80, 0.48)
    ambient: float = 0.3
    sky_rgb: tuple = (127, 178, 229)
    miss_depth: float = 0.0
    extra: dict = field(default_factory=dict)

    @property
    def max_boxes(self) -> int:
        return self.movable_boxes + (self.agents if self.body_boxes else 0)

    @property
    def num_obs(self) -> int:
        return self.num_envs * self.agents


def config(name: str, **over) -> SceneConfig:
    """The five workload shapes the benchmark definition lists, by short name."""
    table = {
        "tiny": dict(num_envs=4, agents=1, grid=(16, 8, 16), width=64, height=36, palette_size=16,
                     world="segments", cam_y_fixed=1.5, seed=1),
        "rooms": dict(num_envs=1024, agents=2, grid=(64, 16, 64), width=128, height=72,
                      palette_size=64, world="rooms", seed=2),
        "rooms_boxes": dict(num_envs=4096, agents=4, grid=(64, 16, 64), width=128, height=72,
                            palette_size=64, world="rooms", movable_boxes=32, body_boxes=True, seed=3),
        "headline": dict(num_envs=16384, agents=1, grid=(128, 32, 128), width=128, height=72,
                         palette_size=64, world="columns", movable_boxes=16, seed=4),
        "sweep": dict(num_envs=8192, agents=2, grid=(64, 16, 64), width=128, height=72,
                      palette_size=64, world="rooms", movable_boxes=32, seed=5),
    }
    kw = dict(table[name])
    kw.update(over)
    return SceneConfig(name=name, **kw)


# --------------------------------------------------------------------------- worlds

def _scatter_rects(rng: Rng, stream: int, env: torch.Tensor, n_rects: int, gx: int, gz: int,
                   wmax: int, dmax: int, hmin: int, hmax: int, P: int, thin: bool):
    """Heightmap + material map from n_rects random rectangles; the tallest rectangle wins a cell."""
    dev = rng.device
    E = env.numel()
    r = torch.arange(n_rects, device=dev)[None, :]
    e = env[:, None]
    x0 = rng.randint(stream + 0, e, r, 0, gx - 1)
    z0 = rng.randint(stream + 1, e, r, 0, gz - 1)
    w = rng.randint(stream + 2, e, r, 1, wmax)
    d = rng.randint(stream + 3, e, r, 1, dmax)
    if thin:  # wall segments: one voxel thick along a random axis
        along_x = rng.randint(stream + 6, e, r, 0, 1) == 1
        w = torch.where(along_x, w, torch.ones_like(w))
        d = torch.where(along_x, torch.ones_like(d), d)
    h = rng.randint(stream + 4, e, r, hmin, hmax)
    m = rng.randint(stream + 5, e, r, 1, P - 1)
    key = (h * 256 + m)[:, :, None, None]
    dz = torch.arange(dmax, device=dev)[None, None, :, None]
    dx = torch.arange(wmax, device=dev)[None, None, None, :]
    xx = x0[:, :, None, None] + dx
    zz = z0[:, :, None, None] + dz
    ok = (dx < w[:, :, None, None]) & (dz < d[:, :, None, None]) & (xx < gx) & (zz < gz)
    cell = torch.where(ok, zz * gx + xx, torch.zeros_like(xx)).reshape(E, -1)
    key = torch.where(ok, key.expand_as(ok), torch.zeros_like(xx)).reshape(E, -1)
    hm = torch.zeros(E, gz * gx, dtype=torch.int64, device=dev)
    hm.scatter_reduce_(1, cell, key, reduce="amax", include_self=True)
    hm = hm.reshape(E, gz, gx)
    return hm >> 8, hm & 255   # height above the floor layer, material


def _grid_from_heightmap(height, mat, floor_mat, gy):
    E, gz, gx = height.shape
    y = torch.arange(gy, device=height.device)[None, :, None, None]
    solid = (y >= 1) & (y <= height[:, None])
    g = torch.where(solid, mat[:, None].expand(E, gy, gz, gx), torch.zeros((), dtype=torch.int64, device=height.device))
    g[:, 0] = floor_mat[:, None, None]
    return g.to(torch.uint8)


def _world_rooms(rng: Rng, env, gx, gy, gz, P, n_lines=6, pitch=9, n_pillars=24):
    """Floor + border wall + jittered full-height wall lines with 2-wide doors + pillars."""
    dev = rng.device
    E = env.numel()
    e1 = env[:, None]
    li = torch.arange(n_lines, device=dev)[None, :]
    X = pitch * (li + 1) + rng.randint(20, e1, li, -2, 2)           # x of wall lines spanning z
    Z = pitch * (li + 1) + rng.randint(21, e1, li, -2, 2)           # z of wall lines spanning x
    X = X.clamp(2, gx - 3)
    Z = Z.clamp(2, gz - 3)
    matx = rng.randint(22, e1, li, 1, P - 1)
    matz = rng.randint(23, e1, li, 1, P - 1)
    matb = rng.randint(24, env, torch.zeros_like(env), 1, P - 1)
    floor = rng.randint(25, env, torch.zeros_like(env), 1, P - 1)

    mx = torch.zeros(E, gx, dtype=torch.int64, device=dev).scatter_(1, X, matx)
    mz = torch.zeros(E, gz, dtype=torch.int64, device=dev).scatter_(1, Z, matz)
    xs = torch.arange(gx, device=dev)
    zs = torch.arange(gz, device=dev)
    border = ((xs == 0) | (xs == gx - 1))[None, None, :] | ((zs == 0) | (zs == gz - 1))[None, :, None]
    M2 = torch.where(mx[:, None, :] > 0, mx[:, None, :].expand(E, gz, gx),
                     mz[:, :, None].expand(E, gz, gx))
    M2 = torch.where(border & (M2 == 0), matb[:, None, None].expand(E, gz, gx), M2)

    # doors: one per (line, segment between consecutive crossing lines / borders)
    seg = torch.arange(n_lines + 1, device=dev)[None, None, :]
    zero = torch.zeros(E, 1, dtype=torch.int64, device=dev)
    for axis in (0, 1):
        lines = X if axis == 0 else Z                # the wall lines that get doors
        cross, _ = torch.sort(Z if axis == 0 else X, dim=1)
        end = torch.full((E, 1), (gz if axis == 0 else gx) - 1, dtype=torch.int64, device=dev)
        lo = torch.cat([zero, cross], 1)[:, None, :]          # [E,1,S]
        hi = torch.cat([cross, end], 1)[:, None, :]
        room = (hi - lo - 1).clamp(min=0)                     # free cells between crossings
        idx = li[:, :, None] * 16 + seg
        u = rng.uniform(26 + axis, env[:, None, None], idx)
        off = (u * (room - 1).clamp(min=1).to(torch.float64)).to(torch.int64)
        d0 = lo + 1 + off                                     # first door cell, second is d0+1
        has = room >= 2
        for k in (0, 1):
            along = (d0 + k).clamp(max=(gz if axis == 0 else gx) - 2)
            fixed = lines[:, :, None].expand_as(along)
            cell = (along * gx + fixed) if axis == 0 else (fixed * gx + along)
            cell = torch.where(has.expand_as(cell), cell, torch.zeros_like(cell)).reshape(E, -1)
            M2 = M2.reshape(E, -1).scatter(1, cell, torch.zeros_like(cell)).reshape(E, gz, gx)
    M2[:, 0, 0] = matb                                        # cell 0 absorbed the masked scatters
    # pillars
    pi = torch.arange(n_pillars, device=dev)[None, :]
    px = rng.randint(28, e1, pi, 1, gx - 2)
    pz = rng.randint(29, e1, pi, 1, gz - 2)
    pm = rng.randint(30, e1, pi, 1, P - 1)
    # two pillars can fall on one cell: the one with the higher index wins (a maximum over keys, which has
    # one result on every device; a plain scatter with repeated indices does not)
    won = torch.zeros(E, gz * gx, dtype=torch.int64, device=dev)
    won.scatter_reduce_(1, pz * gx + px, pi * 256 + pm, reduce="amax", include_self=True)
    M2 = torch.where(won > 0, won & 255, M2.reshape(E, -1)).reshape(E, gz, gx)
    height = torch.where(M2 > 0, gy - 1, 0)
    return height, M2, floor


def make_worlds(cfg: SceneConfig, env_begin: int = 0, env_count: int | None = None, device="cpu", env_ids=None):
    """Grid, palette and the per-column stack height for envs [env_begin, env_begin+env_count), or for
    the seeded environment ids listed in `env_ids` (any order, any values)."""
    rng = Rng(cfg.seed, device)
    if env_ids is not None:
        env = torch.as_tensor(env_ids, dtype=torch.int64).to(rng.device)
        env_count = env.numel()
    else:
        env_count = cfg.num_envs - env_begin if env_count is None else env_count
        env = torch.arange(env_begin, env_begin + env_count, device=rng.device)
    gx, gy, gz = cfg.grid
    P = cfg.palette_size
    if cfg.world == "rooms":
        height, mat, floor = _world_rooms(rng, env, gx, gy, gz, P, **cfg.extra)
    elif cfg.world == "columns":
        n = cfg.extra.get("n_rects", 1050)
        height, mat = _scatter_rects(rng, 10, env, n, gx, gz, 6, 6, 1, 12, P, thin=False)
        floor = rng.randint(25, env, torch.zeros_like(env), 1, P - 1)
    elif cfg.world == "segments":
        n = cfg.extra.get("n_rects", 9)
        height, mat = _scatter_rects(rng, 10, env, n, gx, gz, 8, 8, 2, gy - 2, P, thin=True)
        floor = rng.randint(25, env, torch.zeros_like(env), 1, P - 1)
    else:
        raise ValueError(cfg.world)
    grid = _grid_from_heightmap(height, mat, floor, gy)
    pi = torch.arange(P * 3, device=rng.device)[None, :]
    palette = rng.randint(31, env[:, None], pi, 24, 255).to(torch.uint8).reshape(env_count, P, 3)
    return {"grid": grid, "palette": palette, "height": height, "env": env}


# --------------------------------------------------------------------------- boxes and cameras

def _f32_bits(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.float32).contiguous().view(torch.int32)


def make_boxes_and_cameras(cfg: SceneConfig, worlds: dict, step: int = 0):
    """Movable boxes resting on the surface under them, agent cameras standing on free
    cells (one body box per agent when cfg.body_boxes), all for the envs in `worlds`."""
    rng = Rng(cfg.seed, worlds["grid"].device)
    dev = rng.device
    env = worlds["env"]
    height = worlds["height"]                       # solid cells above the floor layer
    E = env.numel()
    gx, gy, gz = cfg.grid
    P = cfg.palette_size
    A = cfg.agents
    B = cfg.max_boxes
    surf = (height + 1)                             # y of the walkable surface per column
    e1 = env[:, None]

    boxes = torch.zeros(E, max(B, 1), 8, dtype=torch.int32, device=dev)
    count = torch.zeros(E, dtype=torch.int32, device=dev)
    nb = cfg.movable_boxes
    if nb > 0:
        bi = torch.arange(nb, device=dev)[None, :]
        size = [(0.3 + 0.7 * rng.uniform(40 + c, e1, bi)).to(torch.float32) for c in range(3)]
        cx = (0.5 + rng.uniform(43, e1, bi) * (gx - 1.0)).to(torch.float32)
        cz = (0.5 + rng.uniform(44, e1, bi) * (gz - 1.0)).to(torch.float32)
        lox, hix = cx - size[0] * 0.5, cx + size[0] * 0.5
        loz, hiz = cz - size[2] * 0.5, cz + size[2] * 0.5
        x0 = lox.floor().long().clamp(0, gx - 1); x1 = hix.floor().long().clamp(0, gx - 1)
        z0 = loz.floor().long().clamp(0, gz - 1); z1 = hiz.floor().long().clamp(0, gz - 1)
        flat = surf.reshape(E, -1)
        top = torch.stack([flat.gather(1, zz * gx + xx) for zz in (z0, z1) for xx in (x0, x1)], 0).amax(0)
        loy = top.to(torch.float32)
        hiy = loy + size[1]
        ok = (top < gy - 1) & (hiy <= gy)
        order = torch.argsort((~ok).to(torch.int64), dim=1, stable=True)   # accepted boxes first
        mat = rng.randint(45, e1, bi, 1, P - 1).to(torch.int32)
        rec = torch.stack([_f32_bits(lox), _f32_bits(loy), _f32_bits(loz), _f32_bits(hix),
                           _f32_bits(hiy), _f32_bits(hiz), mat, torch.zeros_like(mat)], -1)
        rec = rec.gather(1, order[:, :, None].expand(-1, -1, 8))
        n_ok = ok.sum(1)
        keep = torch.arange(nb, device=dev)[None, :] < n_ok[:, None]
        boxes[:, :nb] = torch.where(keep[:, :, None], rec, torch.zeros_like(rec))
        count = n_ok.to(torch.int32)

    # cameras: distinct standable columns per agent (top-A of random scores over non-wall columns)
    cells = torch.arange(gz * gx, device=dev)[None, :]
    score = rng.bits32(50 + 7 * step, e1, cells)
    walkable = (surf.reshape(E, -1) < gy - 1)
    interior = ((cells % gx) > 0) & ((cells % gx) < gx - 1) & ((cells // gx) > 0) & ((cells // gx) < gz - 1)
    score = torch.where(walkable & interior, score, torch.full_like(score, -1))
    pick = score.topk(A, dim=1).indices                          # [E, A]
    ai = torch.arange(A, device=dev)[None, :]
    cxi, czi = pick % gx, pick // gx
    cyi = surf.reshape(E, -1).gather(1, pick)
    off = [0.1 + 0.8 * rng.uniform(60 + c, e1, ai + 64 * step) for c in range(3)]
    px = (cxi + off[0]).to(torch.float32)
    pz = (czi + off[2]).to(torch.float32)
    if cfg.cam_y_fixed is not None:
        py = torch.full_like(px, cfg.cam_y_fixed) + (cyi - 1).to(torch.float32)
    else:
        py = (cyi + off[1]).to(torch.float32)
    yaw = (rng.uniform(63, e1, ai + 64 * step) * (2 * math.pi)).to(torch.float32)
    pitch = ((rng.uniform(64, e1, ai + 64 * step) - 0.5) * 0.6).to(torch.float32)
    self_box = torch.full((E, A), -1, dtype=torch.int32, device=dev)
    if cfg.body_boxes:
        slot = count[:, None].long() + ai                       # bodies follow the movable boxes
        bm = rng.randint(65, e1, ai, 1, P - 1).to(torch.int32)
        q = torch.float32
        body = torch.stack([_f32_bits(px - 0.25), _f32_bits(py - 0.75), _f32_bits(pz - 0.25),
                            _f32_bits(px + 0.25), _f32_bits(py + 0.25), _f32_bits(pz + 0.25),
                            bm, torch.zeros_like(bm)], -1)
        boxes.scatter_(1, slot[:, :, None].expand(-1, -1, 8), body)
        self_box = slot.to(torch.int32)
        count = count + A
    cams = torch.stack([_f32_bits(px), _f32_bits(py), _f32_bits(pz), _f32_bits(yaw), _f32_bits(pitch),
                        self_box], -1).reshape(E * A, 6).contiguous()
    return {"boxes": boxes[:, :max(B, 0)].contiguous() if B > 0 else boxes[:, :0].contiguous(),
            "box_count": count, "cams": cams}


def walk_cameras(cfg: SceneConfig, worlds: dict, cams: torch.Tensor, step: int):
    """The sweep workload's seeded camera update: yaw += N(0, 0.1), then 0.1 units along the
    horizontal forward direction; the old position is kept when the new cell is solid or
    outside the grid.  Pure input generation (no collision response beyond keep-or-move)."""
    rng = Rng(cfg.seed, cams.device)
    gx, gy, gz = cfg.grid
    O = cams.shape[0]
    A = cfg.agents
    o = torch.arange(O, device=cams.device)
    env = worlds["env"][o // A]
    f = cams[:, :5].contiguous().view(torch.float32)
    yaw = (f[:, 3].double() + 0.1 * rng.normal(70, env, (o % A) + 64 * step)).to(torch.float32)
    nx = (f[:, 0].double() + 0.1 * torch.sin(yaw.double())).to(torch.float32)
    nz = (f[:, 2].double() + 0.1 * torch.cos(yaw.double())).to(torch.float32)
    ix, iy, iz = nx.floor().long(), f[:, 1].floor().long(), nz.floor().long()
    inside = (ix >= 0) & (ix < gx) & (iz >= 0) & (iz < gz) & (iy >= 0) & (iy < gy)
    g = worlds["grid"]
    eidx = (o // A)
    solid = g[eidx, iy.clamp(0, gy - 1), iz.clamp(0, gz - 1), ix.clamp(0, gx - 1)] != 0
    move = inside & ~solid
    out = cams.clone()
    out[:, 0] = torch.where(move, _f32_bits(nx), cams[:, 0])
    out[:, 2] = torch.where(move, _f32_bits(nz), cams[:, 2])
    out[:, 3] = _f32_bits(yaw)
    return out


def make_scene(cfg: SceneConfig, env_begin: int = 0, env_count: int | None = None, device="cpu", env_ids=None):
    w = make_worlds(cfg, env_begin, env_count, device, env_ids)
    bc = make_boxes_and_cameras(cfg, w)
    return {**w, **bc}


def fill_fraction(grid: torch.Tensor) -> float:
    return float((grid != 0).double().mean())
