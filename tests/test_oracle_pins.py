"""Pins for the CPU oracle: closed forms, invariants, a hand-worked image and an independent
ray-marching check.  None of these tests re-types the oracle's own formula; each fixes the
output by something the geometry or the stated conventions determine on their own."""
import math
from pathlib import Path

import numpy as np
import pytest

from helpers import cam_row, box_rows, PALETTE_1, SKY, default_lut_intensities

GOLDEN = Path(__file__).resolve().parent / "golden"


def _desc(oracle, grid, W, H, P=2, max_boxes=0, **kw):
    return oracle.make_desc(grid.shape, max_boxes, W, H, P, **kw)


def test_empty_world_is_sky(oracle):
    grid = np.zeros((8, 8, 8), np.uint8)
    d = _desc(oracle, grid, 16, 8, miss_depth=-1.0)
    rgb, depth, ids = oracle.render_obs(d, grid, None, 0, PALETTE_1, cam_row(4.2, 3.1, 4.4, 0.7, 0.2))
    assert (rgb == np.array(SKY, np.uint8)).all()
    assert (depth == np.float32(-1.0)).all()
    assert (ids[..., 0] == -1).all()


def test_single_wall_planar_depth_and_floor_formula(oracle):
    """Wall plane z=k seen head-on has ONE depth k-cz on every wall pixel (planar depth), lit by
    ambient only on its -z face; floor pixels have depth 0.5/(-d_y) with d_y = b*ty/H."""
    gx, gy, gz, W, H = 32, 8, 16, 32, 18
    grid = np.zeros((gy, gz, gx), np.uint8)
    grid[0] = 1                # floor, top at y=1
    grid[:, 12, :] = 1         # wall filling the plane k=12
    cx, cz = 16.3, 2.6
    d = _desc(oracle, grid, W, H)
    rgb, depth, ids = oracle.render_obs(d, grid, None, 0, PALETTE_1, cam_row(cx, 1.5, cz, 0.0, 0.0))
    ty = math.tan(math.pi / 4) * H / W
    I = default_lut_intensities()
    for py in range(H):
        b = H - 1 - 2 * py
        dy = b * ty / H
        t_floor = (1.0 - 1.5) / dy if dy < 0 else math.inf
        t_wall = 12 - np.float32(cz)
        for px in range(W):
            if t_floor < t_wall:
                assert abs(depth[py, px] - t_floor) <= 1e-5 * t_floor
                assert ids[py, px, 2] == 3                       # +y face
                want = np.floor(np.array(PALETTE_1[1], float) * I["+y"] + 0.5)
            else:
                assert abs(depth[py, px] - t_wall) <= 1e-6
                assert ids[py, px, 2] == 4                       # -z face
                want = np.floor(np.array(PALETTE_1[1], float) * I["-z"] + 0.5)
            assert (rgb[py, px] == want).all()
    # the wall must cover the whole upper half, the floor part of the lower half
    assert (ids[: H // 2, :, 2] == 4).all() and (ids[H - 1, :, 2] == 3).all()


def test_handworked_4x4(oracle):
    rows = [l.split() for l in (GOLDEN / "handworked_4x4.txt").read_text().splitlines()
            if l and not l.startswith("#")]
    for variant in ("wall", "nowall"):
        grid = np.zeros((4, 4, 4), np.uint8)
        grid[0] = 1
        if variant == "wall":
            grid[:, 3, :] = 1
        d = _desc(oracle, grid, 4, 4)
        rgb, depth, _ = oracle.render_obs(d, grid, None, 0, PALETTE_1, cam_row(2.0, 1.5, 0.5, 0.0, 0.0))
        n = 0
        for v, py, px, r, g, b, dep in rows:
            if v != variant:
                continue
            py, px = int(py), int(px)
            assert tuple(rgb[py, px]) == (int(r), int(g), int(b)), (variant, py, px)
            assert abs(depth[py, px] - float(dep)) <= 1e-6, (variant, py, px)
            n += 1
        assert n == 16


def test_mirror_scene_gives_mirrored_frame(oracle):
    rng = np.random.default_rng(7)
    gx, gy, gz, W, H = 16, 8, 16, 48, 28
    half = rng.integers(0, 6, size=(gy, gz, gx // 2)).astype(np.uint8)
    half[half > 3] = 0
    half[:, :, -1] = 0                                  # keep the cells touching the plane free
    grid = np.concatenate([half, half[:, :, ::-1]], axis=2)
    grid[0] = 2
    pal = np.array([[0, 0, 0], [200, 100, 50], [30, 220, 90], [250, 250, 10]], np.uint8)
    d = _desc(oracle, grid, W, H, P=4, light_dir=(0.0, 0.8, 0.6))
    rgb, depth, ids = oracle.render_obs(d, grid, None, 0, pal, cam_row(gx / 2, 1.5, 1.5, 0.0, 0.1))
    assert (rgb == rgb[:, ::-1]).all()
    assert (depth == depth[:, ::-1]).all()
    assert (ids[..., 0] == 0).any()


def test_yaw_pitch_and_layout_conventions(oracle):
    """One voxel on each axis direction: yaw 0 sees +z, yaw pi/2 sees +x, positive pitch looks up,
    and grid[j][k][i] is indexed (y, z, x).  Depth to the facing side is the distance along the axis."""
    g = 24
    W, H = 32, 32
    c = 12.5

    def centre(grid, yaw, pitch):
        d = _desc(oracle, grid, W, H)
        rgb, depth, ids = oracle.render_obs(d, grid, None, 0, PALETTE_1, cam_row(c, c, c, yaw, pitch))
        return depth[H // 2 - 1: H // 2 + 1, W // 2 - 1: W // 2 + 1], ids[H // 2, W // 2]

    grid = np.zeros((g, g, g), np.uint8); grid[12, 20, 12] = 1          # (i=12, j=12, k=20): +z
    dep, idv = centre(grid, 0.0, 0.0)
    assert np.allclose(dep, 20 - c, atol=1e-5) and idv[2] == 4
    assert idv[1] == 12 + g * (20 + g * 12)
    dep, idv = centre(grid, math.pi, 0.0)
    assert (dep == 0).all() and idv[0] == -1                             # looking away: sky
    grid = np.zeros((g, g, g), np.uint8); grid[12, 12, 20] = 1          # i=20: +x
    dep, idv = centre(grid, math.pi / 2, 0.0)
    assert np.allclose(dep, 20 - c, atol=1e-4) and idv[2] == 0
    grid = np.zeros((g, g, g), np.uint8); grid[20, 12, 12] = 1          # j=20: up
    dep, idv = centre(grid, 0.3, math.pi / 2 - 1e-3)
    assert np.allclose(dep, 20 - c, atol=1e-3) and idv[2] == 2
    # row 0 is the top of the image: a voxel above the view axis shows in the upper rows only
    grid = np.zeros((g, g, g), np.uint8); grid[16, 20, 12] = 1
    d = _desc(oracle, grid, W, H)
    _, _, ids = oracle.render_obs(d, grid, None, 0, PALETTE_1, cam_row(c, c, c, 0.0, 0.0))
    hit_rows = np.where((ids[..., 0] == 0).any(axis=1))[0]
    assert hit_rows.size and hit_rows.max() < H // 2
    # yaw grows toward +x: a voxel at larger x shows right of centre
    grid = np.zeros((g, g, g), np.uint8); grid[12, 20, 16] = 1
    _, _, ids = oracle.render_obs(d, grid, None, 0, PALETTE_1, cam_row(c, c, c, 0.0, 0.0))
    hit_cols = np.where((ids[..., 0] == 0).any(axis=0))[0]
    assert hit_cols.size and hit_cols.min() >= W // 2


def test_field_of_view_edges(oracle):
    """hfov 90 deg: a wall filling the plane z=k is seen; the outermost pixel centres have
    |d_x| = (W-1)/W, so the hit on that wall is at x = cx +- (k-cz)(W-1)/W; check through voxel index."""
    gx, gy, gz, W, H = 64, 4, 16, 16, 2
    grid = np.zeros((gy, gz, gx), np.uint8); grid[:, 12, :] = 1
    cx, cz = 32.5, 2.0
    d = _desc(oracle, grid, W, H)
    _, depth, ids = oracle.render_obs(d, grid, None, 0, PALETTE_1, cam_row(cx, 1.5, cz, 0.0, 0.0))
    for px in range(W):
        x = cx + (12 - cz) * (2 * px + 1 - W) / W
        i = ids[0, px, 1] % gx
        assert i == math.floor(x)
        assert abs(depth[0, px] - 10.0) < 1e-6


def test_shade_lut_intensities(oracle):
    """Default light (0.36,0.80,0.48) is unit: lit faces get 0.3+0.7*component, the others 0.3."""
    g = 9
    pal = np.array([[0, 0, 0], [200, 100, 250]], np.uint8)
    want = {"+x": 0.552, "+y": 0.86, "+z": 0.636, "-x": 0.3, "-y": 0.3, "-z": 0.3}
    assert default_lut_intensities() == pytest.approx(want)
    looks = {"-z": (0.0, 0.0), "+z": (math.pi, 0.0), "-x": (math.pi / 2, 0.0), "+x": (-math.pi / 2, 0.0),
             "+y": (0.0, -math.pi / 2 + 1e-3), "-y": (0.0, math.pi / 2 - 1e-3)}
    for face, (yaw, pitch) in looks.items():
        grid = np.ones((g, g, g), np.uint8)
        grid[1:-1, 1:-1, 1:-1] = 0                      # hollow shell: every view hits one inner face
        d = _desc(oracle, grid, 8, 8)
        rgb, _, ids = oracle.render_obs(d, grid, None, 0, pal, cam_row(4.5, 4.5, 4.5, yaw, pitch))
        px = rgb[3, 3]
        expect = np.floor(pal[1].astype(float) * want[face] + 0.5)
        assert (px == expect).all(), face
    # inside a solid voxel: ambient only, depth 0
    grid = np.ones((g, g, g), np.uint8)
    d = _desc(oracle, grid, 8, 8)
    rgb, depth, ids = oracle.render_obs(d, grid, None, 0, pal, cam_row(4.5, 4.5, 4.5, 0.3, 0.1))
    assert (rgb == np.floor(pal[1] * 0.3 + 0.5).astype(np.uint8)).all() and (depth == 0).all()
    assert (ids[..., 2] == 6).all()


def test_box_equal_to_voxel_renders_the_same(oracle):
    rng = np.random.default_rng(3)
    gx = gy = gz = 8
    W, H = 40, 24
    pal = rng.integers(10, 255, size=(4, 3)).astype(np.uint8)
    cells = [(2, 3, 5), (5, 1, 6), (6, 4, 2), (3, 3, 3)]
    grid_v = np.zeros((gy, gz, gx), np.uint8)
    for n, (i, j, k) in enumerate(cells):
        grid_v[j, k, i] = 1 + n % 3
    boxes = box_rows([((i, j, k), (i + 1, j + 1, k + 1), 1 + n % 3) for n, (i, j, k) in enumerate(cells)])
    dv = _desc(oracle, grid_v, W, H, P=4)
    db = _desc(oracle, grid_v, W, H, P=4, max_boxes=4)
    cam = cam_row(0.7, 2.6, 0.4, 0.75, 0.05)
    rv, zv, iv = oracle.render_obs(dv, grid_v, None, 0, pal, cam)
    rb, zb, ib = oracle.render_obs(db, np.zeros_like(grid_v), boxes, 4, pal, cam)
    assert (iv[..., 0] == 0).sum() > 20
    assert (rv == rb).all() and (zv == zb).all()
    assert ((iv[..., 0] == 0) == (ib[..., 0] == 1)).all() and (iv[..., 2] == ib[..., 2]).all()


def test_translation_by_whole_voxels(oracle):
    rng = np.random.default_rng(5)
    W, H = 40, 24
    small = (rng.random((6, 6, 6)) < 0.15).astype(np.uint8) * rng.integers(1, 4, size=(6, 6, 6)).astype(np.uint8)
    pal = rng.integers(10, 255, size=(4, 3)).astype(np.uint8)
    a = np.zeros((16, 16, 16), np.uint8); a[1:7, 1:7, 1:7] = small
    b = np.zeros((16, 16, 16), np.uint8); b[5:11, 8:14, 3:9] = small      # shift (x+2, y+4, z+7)
    bx = [((2.25, 2.5, 1.75), (3.0, 3.25, 2.5), 2)]
    bx2 = [((4.25, 6.5, 8.75), (5.0, 7.25, 9.5), 2)]
    d = _desc(oracle, a, W, H, P=4, max_boxes=1)
    ra = oracle.render_obs(d, a, box_rows(bx), 1, pal, cam_row(0.5, 3.25, 0.75, 0.6, -0.1))
    rb = oracle.render_obs(d, b, box_rows(bx2), 1, pal, cam_row(2.5, 7.25, 7.75, 0.6, -0.1))
    assert (ra[0] == rb[0]).all() and (ra[1] == rb[1]).all()
    assert (ra[2][..., 0] == 0).any() and (ra[2][..., 0] == 1).any()


def test_occlusion_and_self_box(oracle):
    gx, gy, gz, W, H = 16, 8, 16, 32, 18
    grid = np.zeros((gy, gz, gx), np.uint8); grid[0] = 1; grid[:, 8, :] = 1
    pal = np.array([[0, 0, 0], [200, 100, 50], [10, 200, 30]], np.uint8)
    d = _desc(oracle, grid, W, H, P=3, max_boxes=2)
    cam = cam_row(8.5, 1.75, 2.5, 0.0, 0.0, self_box=-1)
    base = oracle.render_obs(d, grid, None, 0, pal, cam)
    behind = grid.copy(); behind[1:5, 10:14, 3:12] = 2
    hidden_box = box_rows([((4, 1, 10), (6, 3, 12), 2)])
    occ = oracle.render_obs(d, behind, hidden_box, 1, pal, cam)
    assert (base[0] == occ[0]).all() and (base[1] == occ[1]).all()
    # camera inside its own body box: skipping it leaves the frame unchanged, not skipping gives "inside"
    body = box_rows([((8.25, 1.0, 2.25), (8.75, 2.0, 2.75), 2)])
    own = oracle.render_obs(d, grid, body, 1, pal, cam_row(8.5, 1.75, 2.5, 0.0, 0.0, self_box=0))
    assert (own[0] == base[0]).all() and (own[1] == base[1]).all()
    other = oracle.render_obs(d, grid, body, 1, pal, cam_row(8.5, 1.75, 2.5, 0.0, 0.0, self_box=-1))
    assert (other[1] == 0).all() and (other[2][..., 2] == 6).all()
    # a second agent looking at that body sees it, at the distance of its near side
    seen = oracle.render_obs(d, grid, body, 1, pal, cam_row(8.5, 1.5, 0.5, 0.0, 0.0, self_box=-1))
    cy, cxp = H // 2, W // 2
    assert seen[2][cy, cxp, 0] == 1 and abs(seen[1][cy, cxp] - 1.75) < 1e-6


def _march(grid, boxes, P, d, step=2e-3, tmax=40.0):
    """First sample along P + t d that lies inside a filled voxel or a box (independent of slabs)."""
    gy, gz, gx = grid.shape
    t = np.arange(0.0, tmax, step)
    pts = P[None, :] + t[:, None] * d[None, :]
    ijk = np.floor(pts).astype(np.int64)
    inb = ((ijk >= 0) & (ijk < np.array([gx, gy, gz]))).all(axis=1)
    c = np.clip(ijk, 0, np.array([gx, gy, gz]) - 1)
    mat = np.where(inb, grid[c[:, 1], c[:, 2], c[:, 0]], 0)
    hit = mat != 0
    for lo, hi, m in boxes:
        hit |= ((pts >= np.array(lo)) & (pts <= np.array(hi))).all(axis=1)
    idx = np.argmax(hit)
    return (t[idx] if hit[idx] else None)


def test_depth_matches_ray_marching_on_tiny_scene(oracle):
    from paper_2107_08170_b200 import scenes
    cfg = scenes.config("tiny")
    sc = scenes.make_scene(cfg)
    desc = oracle.desc_from_config(cfg)
    grid = sc["grid"][2].numpy()
    cam = sc["cams"][2].numpy()
    f0 = cam[:5].view(np.float32)
    c1 = f0[:3].astype(float) + 1.5 * np.array([math.sin(f0[3]), 0.0, math.cos(f0[3])])
    c2 = f0[:3].astype(float) + 2.5 * np.array([math.sin(f0[3] + 0.4), 0.0, math.cos(f0[3] + 0.4)])
    boxes = [((c1[0] - 0.3, 1.0, c1[2] - 0.35), (c1[0] + 0.3, 1.8, c1[2] + 0.35), 3),
             ((c2[0] - 0.4, 1.2, c2[2] - 0.2), (c2[0] + 0.4, 2.3, c2[2] + 0.2), 5)]
    boxes = [(tuple(np.float32(lo).tolist()), tuple(np.float32(hi).tolist()), m) for lo, hi, m in boxes]
    desc.max_boxes = 2
    rgb, depth, ids = oracle.render_obs(desc, grid, box_rows(boxes), 2, sc["palette"][2].numpy(), cam)
    f = cam[:5].view(np.float32)
    P = f[:3].astype(np.float64)
    yaw, pitch = float(f[3]), float(f[4])
    F = np.array([math.cos(pitch) * math.sin(yaw), math.sin(pitch), math.cos(pitch) * math.cos(yaw)])
    R = np.array([math.cos(yaw), 0.0, -math.sin(yaw)])
    U = np.array([-math.sin(pitch) * math.sin(yaw), math.cos(pitch), -math.sin(pitch) * math.cos(yaw)])
    assert abs(np.dot(F, R)) < 1e-12 and abs(np.dot(F, U)) < 1e-12 and np.allclose(np.cross(R, F), -U)
    W, H = cfg.width, cfg.height
    tx = 1.0; ty = H / W
    rng = np.random.default_rng(0)
    checked = 0
    for py, px in zip(rng.integers(0, H, 150), rng.integers(0, W, 150)):
        d = F + (2 * px + 1 - W) / W * tx * R + (H - 1 - 2 * py) / H * ty * U
        tm = _march(grid, boxes, P, d)
        if tm is None:
            assert ids[py, px, 0] == -1
        else:
            assert ids[py, px, 0] != -1
            assert -1e-6 <= tm - depth[py, px] <= 2e-3 * 1.01 + 1e-5, (py, px, tm, depth[py, px])
        checked += 1
    assert checked == 150 and (ids[..., 0] == 1).any()


def test_batching_determinism_and_data_errors(oracle):
    from paper_2107_08170_b200 import scenes
    cfg = scenes.config("tiny")
    sc = scenes.make_scene(cfg)
    a = oracle.render_scene(cfg, sc)
    b = oracle.render_scene(cfg, sc, [2])
    assert (a[0][2] == b[0][0]).all() and (a[1][2] == b[1][0]).all()
    # non-finite camera: whole frame sky; out-of-range material id clamps to the last palette entry
    desc = oracle.desc_from_config(cfg)
    g = sc["grid"][0].numpy().copy()
    bad = oracle.render_obs(desc, g, None, 0, sc["palette"][0].numpy(), cam_row(float("nan"), 1.5, 2.0, 0.0, 0.0))
    assert (bad[2][..., 0] == -1).all()
    g2 = g.copy(); g2[g2 != 0] = 200
    g3 = g.copy(); g3[g3 != 0] = cfg.palette_size - 1
    r2 = oracle.render_obs(desc, g2, None, 0, sc["palette"][0].numpy(), sc["cams"][0].numpy())
    r3 = oracle.render_obs(desc, g3, None, 0, sc["palette"][0].numpy(), sc["cams"][0].numpy())
    assert (r2[0] == r3[0]).all()


def test_subpixel_offset_path_agrees_with_float_path(oracle):
    """The displaced-sample entry (edge rule) at zero displacement is the pixel-centre ray."""
    from paper_2107_08170_b200 import scenes
    cfg = scenes.config("tiny")
    sc = scenes.make_scene(cfg)
    desc = oracle.desc_from_config(cfg)
    full = oracle.render_obs(desc, sc["grid"][0].numpy(), None, 0, sc["palette"][0].numpy(), sc["cams"][0].numpy())
    pxy = np.array([[5, 7], [20, 30], [63, 35], [0, 0]], np.int32)
    tiny = np.full((4, 2), 1e-9)
    sub = oracle.render_pixels(desc, sc["grid"][0].numpy(), None, 0, sc["palette"][0].numpy(),
                               sc["cams"][0].numpy(), pxy, tiny)
    for q, (px, py) in enumerate(pxy):
        assert (sub[0][q] == full[0][py, px]).all()
        assert abs(sub[1][q] - full[1][py, px]) <= 1e-5 * max(full[1][py, px], 1e-3)


def test_vertical_field_of_view_and_square_pixels(oracle):
    """Square pixels: tan of the vertical half-angle is tan(hfov/2)*H/W, so on a wall at distance D the
    pixel row py meets height cy + D*(H-1-2py)/H * (H/W) = cy + D*(H-1-2py)/W."""
    gx, gy, gz, W, H = 8, 64, 16, 16, 8
    grid = np.zeros((gy, gz, gx), np.uint8); grid[:, 12, :] = 1
    cx, cy, cz = 4.5, 32.5, 2.0
    d = _desc(oracle, grid, W, H)
    _, depth, ids = oracle.render_obs(d, grid, None, 0, PALETTE_1, cam_row(cx, cy, cz, 0.0, 0.0))
    for py in range(H):
        y = cy + (12 - cz) * (H - 1 - 2 * py) / W
        j = ids[py, W // 2, 1] // (gx * gz)
        assert j == math.floor(y), (py, j, y)
    assert np.allclose(depth[:, W // 2], 10.0, atol=1e-6)


def test_tie_breaks_voxel_before_box_and_lower_box_first(oracle):
    gx = gy = gz = 8
    W, H = 16, 8
    pal = np.array([[0, 0, 0], [200, 0, 0], [0, 200, 0], [0, 0, 200]], np.uint8)
    grid = np.zeros((gy, gz, gx), np.uint8); grid[:, 6, :] = 1                      # wall face at z = 6
    # box 0 and box 1 identical, their front face coplanar with the wall face
    boxes = box_rows([((0, 0, 6), (8, 8, 7), 2), ((0, 0, 6), (8, 8, 7), 3)])
    d = _desc(oracle, grid, W, H, P=4, max_boxes=2)
    cam = cam_row(4.3, 4.2, 1.0, 0.0, 0.0)
    rgb, depth, ids = oracle.render_obs(d, grid, boxes, 2, pal, cam)
    c = slice(4, 12)                                                               # columns that see the wall
    assert (ids[:, c, 0] == 0).all() and np.allclose(depth[:, c], 5.0, atol=1e-6)   # voxel wins the tie
    rgb, depth, ids = oracle.render_obs(d, np.zeros_like(grid), boxes, 2, pal, cam)
    assert (ids[:, c, 0] == 1).all() and (ids[:, c, 1] == 0).all()                 # lower box index wins
    assert (rgb[:, c, 1] > 0).all() and (rgb[:, c, 2] == 0).all()                  # box 0's colour (green)


def test_axis_parallel_rays_zero_direction_component(oracle):
    """Rays with a direction component that is EXACTLY zero (an odd image size puts a pixel centre on
    the view axis: a = 2px+1-W = 0 in the centre column, b = H-1-2py = 0 in the centre row, and with
    yaw = pitch = 0 the basis has exact zeros).  Along such an axis the ray never moves, so a slab is
    crossed iff the eye lies within it, both ends included: geometry fixes every value below."""
    W = H = 5
    gx, gy, gz = 8, 16, 12
    grid = np.zeros((gy, gz, gx), np.uint8)
    grid[:, 9, :] = 1                                          # wall plane k = 9
    pal = PALETTE_1
    cx, cy, cz = 4.0, 7.5, 1.25                                # cx sits exactly on a cell face (x = 4)
    # boxes in front of the wall, all spanning y 7..8 unless said otherwise; material 1
    boxes = box_rows([
        ((3.5, 7.0, 4.0), (4.5, 8.0, 4.5), 1),                 # 0: x-range contains cx        -> centre column hits it
        ((4.0, 7.0, 5.0), (4.5, 8.0, 5.5), 1),                 # 1: cx exactly on lo.x         -> counts as inside
        ((3.5, 7.0, 6.0), (4.0, 8.0, 6.5), 1),                 # 2: cx exactly on hi.x         -> counts as inside
        ((4.25, 7.0, 3.0), (4.75, 8.0, 3.5), 1),               # 3: x-range excludes cx (nearest of all) -> missed
        ((3.0, 7.75, 2.0), (5.0, 8.0, 2.5), 1),                # 4: y-range excludes cy (nearer still)    -> missed by the centre row
    ])
    d = _desc(oracle, grid, W, H, max_boxes=8)
    cam = cam_row(cx, cy, cz, 0.0, 0.0)

    def centre(nboxes, which):
        rgb, depth, ids = oracle.render_obs(d, grid, boxes[which] if nboxes else None, nboxes, pal, cam)
        return rgb, depth, ids

    # no boxes: the centre pixel looks straight down +z (d = (0, 0, 1)) and meets the wall at k - cz
    rgb, depth, ids = centre(0, slice(0, 0))
    assert ids[2, 2].tolist()[0] == 0 and ids[2, 2, 2] == 4    # a voxel, its -z face
    assert abs(depth[2, 2] - (9 - cz)) <= 1e-6
    # cx = 4.0 lies on the shared face of x cells 3 and 4: both closed slabs contain it, the lowest index wins
    assert ids[2, 2, 1] == 3 + gx * (9 + gz * 7)
    # the whole centre column has d_x == 0 and the whole centre row d_y == 0: the wall voxels they meet
    # lie in the eye's own x column / y layer
    for py in range(H):
        assert ids[py, 2, 0] == 0 and ids[py, 2, 1] % gx in (3, 4)
    for px in (1, 2, 3):                                       # (the outermost two leave the 8-wide grid before the wall)
        assert ids[2, px, 0] == 0 and (ids[2, px, 1] // (gx * gz)) == 7

    want = {0: 4.0 - cz, 1: 5.0 - cz, 2: 6.0 - cz}
    for b, t in want.items():                                  # each containing box alone is hit head-on at its near z face
        rgb, depth, ids = centre(1, slice(b, b + 1))
        assert ids[2, 2].tolist() == [1, 0, 4], (b, ids[2, 2])
        assert abs(depth[2, 2] - t) <= 1e-6
    for b in (3, 4):                                           # boxes that exclude the eye's coordinate are missed
        rgb, depth, ids = centre(1, slice(b, b + 1))
        assert ids[2, 2, 0] == 0 and abs(depth[2, 2] - (9 - cz)) <= 1e-6, b
    # all together: box 4 and box 3 are nearer but missed; box 0 is the nearest that is hit
    rgb, depth, ids = centre(5, slice(0, 5))
    assert ids[2, 2].tolist() == [1, 0, 4] and abs(depth[2, 2] - (4.0 - cz)) <= 1e-6
    # box 4 is missed by the centre row only.  The row above looks up with d_y = b*ty/H = 2*1/5 = 0.4; at the
    # box's near z face (t = 2.0 - cz = 0.75) it is at y = 7.5 + 0.3 = 7.8, inside [7.75, 8]: a hit on the
    # -z face at depth 0.75
    assert ids[1, 2].tolist() == [1, 4, 4] and abs(depth[1, 2] - 0.75) <= 1e-6
    # colours: ambient-only (-z faces): floor(palette * 0.3 + 0.5)
    assert (rgb[2, 2] == np.floor(np.array(PALETTE_1[1], float) * 0.3 + 0.5)).all()
