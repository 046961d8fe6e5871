"""CUDA path (through the C ABI) against the CPU oracle, element by element."""
import math

import numpy as np
import pytest
import torch

from helpers import cam_row, box_rows
from paper_2107_08170_b200 import scenes
import parity

pytestmark = pytest.mark.gpu


def _binding():
    from paper_2107_08170_b200 import binding
    return binding


def _render_custom(oracle, grid, palette, cams, W, H, boxes=None, box_count=None, agents=1, max_boxes=0,
                   check=True, **desc_kw):
    """One env-batch of hand-made worlds: grid [E][gy][gz][gx], cams [E*agents][6]."""
    B = _binding()
    E, gy, gz, gx = grid.shape
    P = palette.shape[1]
    desc = B.make_desc(E, agents, (gx, gy, gz), max_boxes, W, H, P, **desc_kw)
    batch = B.Batch(desc)
    dev = torch.device("cuda", 0)
    t = lambda a, dt: torch.from_numpy(np.ascontiguousarray(a)).to(dt).to(dev)
    bt = ct = None
    if max_boxes > 0:
        bt, ct = t(boxes, torch.int32), t(box_count, torch.int32)
    batch.upload_worlds(0, E, t(grid, torch.uint8), bt, ct, t(palette, torch.uint8))
    batch.set_cameras(t(cams, torch.int32))
    rgb, depth = batch.alloc_outputs()
    batch.render_batch(rgb, depth)
    status = batch.query_status()
    g_rgb, g_depth = rgb.cpu().numpy(), depth.cpu().numpy()
    batch.destroy()
    if not check:
        return g_rgb, g_depth, status
    okw = dict(desc_kw)
    if "hfov_rad" in okw:
        okw["hfov"] = okw.pop("hfov_rad")                 # the two descriptors name the field differently
    od = oracle.make_desc((gy, gz, gx), max_boxes, W, H, P, **okw)
    total = None
    for o in range(E * agents):
        e = o // agents
        bx = boxes[e] if max_boxes > 0 else None
        bc = int(box_count[e]) if max_boxes > 0 else 0
        o_rgb, o_depth, o_ids = oracle.render_obs(od, grid[e], bx, bc, palette[e], cams[o])
        st = parity.compare_obs(oracle, od, grid[e], bx, bc, palette[e], cams[o], g_rgb[o], g_depth[o],
                                o_rgb, o_depth, o_ids)
        total = st if total is None else {k: total[k] + st[k] for k in st}
    return g_rgb, g_depth, status, total


def _pal(E, P, seed=0):
    return np.random.default_rng(seed).integers(20, 255, size=(E, P, 3)).astype(np.uint8)


def test_tiny_config_all_pixels(oracle):
    from gpu_util import render_scene, scene_to_numpy
    cfg = scenes.config("tiny")
    sc = scenes.make_scene(cfg)
    g_rgb, g_depth, status = render_scene(cfg, sc)
    assert status == 0
    st = parity.compare_scene(oracle, cfg, scene_to_numpy(sc), range(cfg.num_obs), g_rgb, g_depth)
    parity.assert_parity(st, "tiny")
    assert st["pixels"] == 4 * 64 * 36


def test_tiny_many_seeds_brute_force(oracle):
    from gpu_util import render_scene, scene_to_numpy
    tot = {"pixels": 0, "rgb_mismatch": 0, "mismatch": 0, "unexcused": 0}
    for seed in range(10, 16):
        cfg = scenes.config("tiny", seed=seed, num_envs=6)
        sc = scenes.make_scene(cfg)
        g_rgb, g_depth, status = render_scene(cfg, sc)
        st = parity.compare_scene(oracle, cfg, scene_to_numpy(sc), range(cfg.num_obs), g_rgb, g_depth)
        assert st["unexcused"] == 0, (seed, st)
        for k in tot:
            tot[k] += st[k]
    parity.assert_parity(tot, "tiny seeds")


def test_handmade_wall_floor_and_empty(oracle):
    gx, gy, gz, W, H = 32, 8, 16, 32, 20
    grid = np.zeros((3, gy, gz, gx), np.uint8)
    grid[0, 0] = 1; grid[0, :, 12, :] = 1            # floor + wall
    grid[2] = 1                                       # env 2 solid: camera inside
    pal = _pal(3, 4)
    cams = np.stack([cam_row(16.3, 1.5, 2.6, 0.0, 0.0), cam_row(5.2, 3.1, 4.4, 0.7, 0.2),
                     cam_row(7.5, 3.5, 8.5, 1.0, -0.2)])
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, pal, cams, W, H, miss_depth=-1.0)
    assert status == 0 and st["rgb_mismatch"] == 0 and st["depth_mismatch"] == 0
    assert np.allclose(g_depth[0, : H // 2], 12 - np.float32(2.6), atol=1e-6)      # planar wall depth
    assert (g_rgb[1] == np.array([127, 178, 229], np.uint8)).all() and (g_depth[1] == -1.0).all()
    assert (g_depth[2] == 0.0).all()
    assert (g_rgb[2] == np.floor(pal[2, 1] * np.float64(np.float32(0.3)) + 0.5).astype(np.uint8)).all()


def test_mirror_scene_bit_exact(oracle):
    rng = np.random.default_rng(7)
    gx, gy, gz, W, H = 16, 8, 16, 48, 28
    half = rng.integers(0, 6, size=(gy, gz, gx // 2)).astype(np.uint8)
    half[half > 3] = 0
    half[:, :, -1] = 0
    grid = np.concatenate([half, half[:, :, ::-1]], axis=2)[None].copy()
    grid[0, 0] = 2
    pal = _pal(1, 4)
    boxes = box_rows([((6.5, 1.0, 5.0), (7.25, 1.5, 5.5), 1), ((8.75, 1.0, 5.0), (9.5, 1.5, 5.5), 1)])[None]
    cams = cam_row(gx / 2, 1.5, 1.5, 0.0, 0.1)[None]
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, pal, cams, W, H, boxes=boxes,
                                                box_count=np.array([2]), max_boxes=2, light_dir=(0.0, 0.8, 0.6))
    assert st["unexcused"] == 0
    assert (g_rgb[0] == g_rgb[0][:, ::-1]).all() and (g_depth[0] == g_depth[0][:, ::-1]).all()


def test_camera_outside_grid_and_far_away(oracle):
    rng = np.random.default_rng(11)
    gx, gy, gz, W, H = 16, 8, 12, 64, 36
    grid = ((rng.random((1, gy, gz, gx)) < 0.2) * rng.integers(1, 4, size=(1, gy, gz, gx))).astype(np.uint8)
    grid = np.repeat(grid, 6, axis=0)
    pal = np.repeat(_pal(1, 4), 6, axis=0)
    look = lambda p, q: (math.atan2(q[0] - p[0], q[2] - p[2]),
                         math.atan2(q[1] - p[1], math.hypot(q[0] - p[0], q[2] - p[2])))
    c = (8.0, 4.0, 6.0)
    eyes = [(-6.3, 5.2, -4.1), (24.7, 3.3, 6.2), (8.2, 19.5, 6.4), (8.1, -7.5, 5.7), (16.0, 4.5, 6.5), (-40.0, 12.0, 30.0)]
    boxes = np.repeat(box_rows([((-3.0, 2.0, -2.0), (-1.5, 3.0, -1.0), 2), ((17.0, 1.0, 5.0), (19.0, 6.0, 7.5), 3)])[None], 6, 0)
    cams = np.stack([cam_row(*e, *look(e, c)) for e in eyes])
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, pal, cams, W, H, boxes=boxes,
                                                box_count=np.full(6, 2), max_boxes=2)
    parity.assert_parity(st, "outside")
    assert (g_depth > 0).mean() > 0.15


def test_boxes_selfbox_degenerate_and_many_boxes(oracle):
    rng = np.random.default_rng(21)
    gx, gy, gz, W, H = 24, 8, 24, 96, 56
    E, nb, A = 3, 70, 2
    grid = np.zeros((E, gy, gz, gx), np.uint8); grid[:, 0] = 1
    grid[:, 1:4, 20, :] = 2
    pal = _pal(E, 8)
    items = []
    for e in range(E):
        rows = []
        for b in range(nb):
            c = rng.uniform([2, 1, 2], [22, 3, 19]); s = rng.uniform(0.2, 1.2, 3)
            rows.append((c - s / 2, c + s / 2, int(rng.integers(1, 8))))
        rows[5] = ((3.0, 1.0, 3.0), (3.0, 2.0, 4.0), 1)            # zero width: ignored
        rows[6] = ((5.0, 2.0, 3.0), (4.0, 3.0, 4.0), 1)            # inverted: ignored
        items.append(box_rows(rows))
    boxes = np.stack(items)
    count = np.array([nb, nb - 7, 0])
    cams = []
    for e in range(E):
        for a in range(A):
            x, z = rng.uniform(4, 20), rng.uniform(3, 10)
            bid = 10 + a
            body = box_rows([((x - .25, 1.0, z - .25), (x + .25, 2.0, z + .25), 3)])[0]
            boxes[e, bid] = body
            cams.append(cam_row(x, 1.75, z, rng.uniform(-0.6, 0.6), rng.uniform(-0.3, 0.2), self_box=bid))
    cams = np.stack(cams)
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, pal, cams, W, H, boxes=boxes, box_count=count,
                                                agents=A, max_boxes=nb)
    parity.assert_parity(st, "boxes")
    assert status == 0


def test_voxel_as_box_and_axis_parallel_rays(oracle):
    """Boxes equal to voxel cells render like those voxels; yaw=pitch=0 gives rays with exact zeros
    in no component but exercises the aligned case; a camera on a voxel boundary plane too."""
    rng = np.random.default_rng(3)
    g = 8
    W, H = 40, 24
    cells = [(2, 3, 5), (5, 1, 6), (6, 4, 2), (3, 3, 3), (1, 1, 6)]
    grid = np.zeros((2, g, g, g), np.uint8)
    rows = []
    for n, (i, j, k) in enumerate(cells):
        grid[0, j, k, i] = 1 + n % 3
        rows.append(((i, j, k), (i + 1, j + 1, k + 1), 1 + n % 3))
    boxes = np.stack([box_rows(rows), box_rows(rows)])
    pal = np.repeat(_pal(1, 4), 2, axis=0)
    cams = np.stack([cam_row(0.7, 2.6, 0.4, 0.75, 0.05)] * 2)
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, pal, cams, W, H, boxes=boxes,
                                                box_count=np.array([0, 5]), max_boxes=5)
    parity.assert_parity(st, "voxel-as-box")
    same = (g_rgb[0] == g_rgb[1]).all(axis=-1) & parity.depth_close(g_depth[0], g_depth[1])
    assert same.mean() > 0.995
    # aligned camera on a boundary plane (x = 4.0), cells next to the plane empty
    grid2 = np.zeros((1, g, g, g), np.uint8); grid2[0, 0] = 1; grid2[0, :, 7, :] = 2; grid2[0, 1:3, 4, 1] = 3; grid2[0, 1:3, 4, 6] = 3
    cams2 = cam_row(4.0, 1.5, 0.5, 0.0, 0.0)[None]
    _, _, _, st2 = _render_custom(oracle, grid2, _pal(1, 4), cams2, W, H)
    parity.assert_parity(st2, "aligned")
    assert st2["rgb_mismatch"] == 0


def test_data_errors_set_flags_and_stay_in_bounds(oracle):
    B = _binding()
    gx, gy, gz, W, H = 8, 8, 8, 16, 8
    grid = np.zeros((2, gy, gz, gx), np.uint8); grid[:, 0] = 200; grid[:, :, 7, :] = 3
    pal = _pal(2, 4)
    boxes = np.stack([box_rows([((2, 1, 4), (3, 2, 5), 77), ((5, 1, 4), (6, 2, 5), 1)])] * 2)
    count = np.array([9, -3])
    cams = np.stack([cam_row(4.4, 2.45, 1.55, 0.1, 0.02), cam_row(float("nan"), 2.5, 1.5, 0.0, 0.0)])
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, pal, cams, W, H, boxes=boxes, box_count=count,
                                                max_boxes=2)
    assert status == (B.FLAG_MATERIAL_CLAMPED | B.FLAG_BOX_COUNT_CLAMPED | B.FLAG_BAD_CAMERA)
    assert st["unexcused"] == 0 and st["rgb_mismatch"] <= 1, st
    assert (g_rgb[1] == np.array([127, 178, 229], np.uint8)).all()


@pytest.mark.parametrize("name,envs", [("rooms", 6), ("rooms_boxes", 3), ("headline", 5), ("sweep", 3)])
def test_workload_shapes_small_batches(oracle, name, envs):
    from gpu_util import render_scene, scene_to_numpy
    cfg = scenes.config(name, num_envs=envs)
    sc = scenes.make_scene(cfg)
    g_rgb, g_depth, status = render_scene(cfg, sc)
    assert status == 0
    st = parity.compare_scene(oracle, cfg, scene_to_numpy(sc), range(cfg.num_obs), g_rgb, g_depth)
    parity.assert_parity(st, name)


@pytest.mark.parametrize("W,H", [(64, 36), (256, 144)])
def test_sweep_resolutions_with_camera_walk(oracle, W, H):
    from gpu_util import scene_to_numpy, upload_scene
    B = _binding()
    cfg = scenes.config("sweep", num_envs=2, width=W, height=H)
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    rgb, depth = batch.alloc_outputs()
    cams = sc["cams"]
    for step in (1, 2):
        cams = scenes.walk_cameras(cfg, sc, cams, step)
        batch.set_cameras(cams.cuda())
        batch.render_batch(rgb, depth)
    assert batch.query_status() == 0
    scn = scene_to_numpy(sc); scn["cams"] = cams.numpy()
    st = parity.compare_scene(oracle, cfg, scn, range(cfg.num_obs), rgb.cpu().numpy(), depth.cpu().numpy())
    parity.assert_parity(st, f"sweep {W}x{H}")
    batch.destroy()


def test_invariants_batching_permutation_determinism_translation():
    from gpu_util import render_scene
    cfg = scenes.config("rooms_boxes", num_envs=4)
    sc = scenes.make_scene(cfg)
    r1 = render_scene(cfg, sc)
    r2 = render_scene(cfg, sc)
    assert (r1[0] == r2[0]).all() and (r1[1] == r2[1]).all()                  # determinism
    perm = torch.tensor([2, 0, 3, 1])
    A = cfg.agents
    sp = {k: sc[k][perm] for k in ("grid", "palette", "boxes", "box_count")}
    sp["cams"] = sc["cams"].reshape(4, A, 6)[perm].reshape(-1, 6).contiguous()
    rp = render_scene(cfg, sp)
    want = r1[0].reshape(4, A, *r1[0].shape[1:])[perm.numpy()].reshape(r1[0].shape)
    assert (rp[0] == want).all()                                              # env permutation
    # one agent rendered alone equals the same camera inside the batch
    cfg1 = scenes.config("rooms_boxes", num_envs=1, agents=1, movable_boxes=cfg.max_boxes, body_boxes=False)
    e, a = 2, 3
    s1 = {"grid": sc["grid"][e:e + 1], "palette": sc["palette"][e:e + 1], "boxes": sc["boxes"][e:e + 1],
          "box_count": sc["box_count"][e:e + 1], "cams": sc["cams"][e * A + a: e * A + a + 1]}
    ra = render_scene(cfg1, s1)
    assert (ra[0][0] == r1[0][e * A + a]).all() and (ra[1][0] == r1[1][e * A + a]).all()


def test_step_host_matches_device_path():
    from gpu_util import upload_scene
    B = _binding()
    cfg = scenes.config("rooms_boxes", num_envs=12)
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    batch.set_cameras(sc["cams"].cuda())
    rgb, depth = batch.alloc_outputs()
    batch.render_batch(rgb, depth)
    h_rgb = torch.empty(rgb.shape, dtype=torch.uint8).pin_memory()
    h_depth = torch.empty(depth.shape, dtype=torch.float32).pin_memory()
    for _ in range(2):
        batch.step_host(sc["cams"].pin_memory(), h_rgb, h_depth, boxes=sc["boxes"].contiguous(),
                        box_count=sc["box_count"].contiguous())
        assert torch.equal(h_rgb, rgb.cpu()) and torch.equal(h_depth, depth.cpu())
    assert batch.query_status() == 0 and batch.launch_count() > 0
    batch.destroy()


def test_not_ready_and_argument_errors():
    B = _binding()
    cfg = scenes.config("tiny")
    batch = B.Batch(B.desc_from_config(cfg))
    rgb, depth = batch.alloc_outputs()
    with pytest.raises(B.MvError) as ei:
        batch.render_batch(rgb, depth)
    assert ei.value.code == -4
    sc = scenes.make_scene(cfg)
    with pytest.raises(B.MvError) as ei:
        batch.upload_worlds(2, 3, sc["grid"][:3].cuda(), None, None, sc["palette"][:3].cuda())
    assert ei.value.code == -1
    batch.upload_worlds(0, 2, sc["grid"][:2].cuda(), None, None, sc["palette"][:2].cuda())
    batch.set_cameras(sc["cams"].cuda())
    with pytest.raises(B.MvError) as ei:
        batch.render_batch(rgb, depth)                  # envs 2,3 still missing
    assert ei.value.code == -4
    batch.upload_worlds(2, 2, sc["grid"][2:].cuda(), None, None, sc["palette"][2:].cuda())
    batch.render_batch(rgb, depth)
    assert batch.query_status() == 0
    batch.destroy()


def test_scattered_upload_equals_env_by_env_upload():
    """mv_upload_worlds_at writes env i of its arrays to the listed env: the same bytes as one
    contiguous upload per listed env; readiness is tracked per listed env; bad lists are refused."""
    from gpu_util import upload_scene
    B = _binding()
    cfg = scenes.config("rooms_boxes", num_envs=12)
    old, new = scenes.make_scene(cfg), scenes.make_scene(scenes.config("rooms_boxes", num_envs=12, seed=91))
    where = [1, 4, 5, 9]
    dev = lambda t: t.cuda().contiguous()
    frames = []
    for scattered in (False, True):
        batch = B.Batch(B.desc_from_config(cfg))
        upload_scene(batch, old)
        if scattered:
            batch.upload_worlds_at(where, dev(new["grid"][:4]), dev(new["boxes"][:4]), dev(new["box_count"][:4]),
                                   dev(new["palette"][:4]))
        else:
            for i, e in enumerate(where):
                batch.upload_worlds(e, 1, dev(new["grid"][i:i + 1]), dev(new["boxes"][i:i + 1]),
                                    dev(new["box_count"][i:i + 1]), dev(new["palette"][i:i + 1]))
        batch.set_cameras(old["cams"].cuda())
        rgb, depth = batch.alloc_outputs()
        batch.render_batch(rgb, depth)
        assert batch.query_status() == 0
        frames.append((rgb.cpu(), depth.cpu()))
        batch.destroy()
    assert torch.equal(frames[0][0], frames[1][0]) and torch.equal(frames[0][1], frames[1][1])
    A = cfg.agents
    changed = [bool((frames[1][0][e * A:(e + 1) * A] != 0).any()) for e in range(12)]
    assert all(changed)
    # readiness: only the listed envs count as uploaded
    batch = B.Batch(B.desc_from_config(cfg))
    batch.upload_worlds_at([0, 2, 11], dev(new["grid"][:3]), None, None, dev(new["palette"][:3]))
    batch.set_cameras(old["cams"].cuda())
    rgb, depth = batch.alloc_outputs()
    with pytest.raises(B.MvError) as ei:
        batch.render_batch(rgb, depth)
    assert ei.value.code == -4
    rest = [e for e in range(12) if e not in (0, 2, 11)]
    batch.upload_worlds_at(rest, dev(old["grid"][:9]), None, None, dev(old["palette"][:9]))
    batch.render_batch(rgb, depth)
    for bad in ([3, 3], [5, 4], [-1, 2], [0, 12]):
        with pytest.raises(B.MvError) as ei:
            batch.upload_worlds_at(bad, dev(new["grid"][:2]), None, None, dev(new["palette"][:2]))
        assert ei.value.code == -1
    batch.upload_worlds_at([], None, None, None, None)          # nothing to do
    batch.destroy()


def test_limits_are_reported_not_faulted():
    B = _binding()
    import ctypes as C
    # per-observation tables (tile masks of a 4096 x 4096 image) beyond shared memory -> UNSUPPORTED, no launch
    d = B.make_desc(1, 1, (16, 8, 16), 32, 4096, 4096, 16)
    h = C.c_void_p()
    assert B.lib().mv_create_batch(C.byref(d), C.byref(h)) == -6 and not h.value


def test_occupancy_in_global_memory_matches_shared(oracle):
    """Grids too large for shared memory are walked in global memory; forcing that path on an
    ordinary workload gives the same bytes, and a grid that really is too large matches the oracle."""
    from gpu_util import upload_scene, scene_to_numpy
    B = _binding()
    cfg = scenes.config("rooms_boxes", num_envs=4)
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    batch.set_cameras(sc["cams"].cuda())
    rgb, depth = batch.alloc_outputs()
    batch.render_batch(rgb, depth)
    rgb2, depth2 = batch.alloc_outputs()
    batch.debug_occupancy_in_global(True)
    batch.render_batch(rgb2, depth2)
    assert torch.equal(rgb, rgb2) and torch.equal(depth, depth2) and batch.query_status() == 0
    batch.debug_occupancy_in_global(False)
    batch.destroy()
    # 256 x 32 x 256 voxels: 256 KiB of occupancy bits per env, more than an SM's shared memory
    big = scenes.config("headline", num_envs=2, grid=(256, 32, 256), width=64, height=36, extra={"n_rects": 4200})
    sb = scenes.make_scene(big)
    bb = B.Batch(B.desc_from_config(big))
    with pytest.raises(B.MvError):
        bb.debug_occupancy_in_global(False)              # cannot be staged
    upload_scene(bb, sb)
    bb.set_cameras(sb["cams"].cuda())
    r, d = bb.alloc_outputs()
    bb.render_batch(r, d)
    assert bb.query_status() == 0
    st = parity.compare_scene(oracle, big, scene_to_numpy(sb), range(big.num_obs), r.cpu().numpy(), d.cpu().numpy())
    parity.assert_parity(st, "large grid")
    bb.destroy()


def test_odd_grid_sizes_and_occupied_bounds(oracle):
    rng = np.random.default_rng(2)
    for gx in (20, 32, 44):
        grid = ((rng.random((2, 8, 12, gx)) < 0.1) * rng.integers(1, 4, size=(2, 8, 12, gx))).astype(np.uint8)
        grid[:, 5:] = 0                                  # nothing above y = 5
        grid[:, :, :, :3] = 0                            # nothing left of x = 3
        grid[1] = 0                                      # env 1 is empty
        cams = np.stack([cam_row(gx / 2 + 0.3, 6.5, 6.2, 0.4, -0.5), cam_row(2.2, 3.3, 4.4, 1.0, 0.1)])
        g_rgb, g_depth, status, st = _render_custom(oracle, grid, _pal(2, 4), cams, 64, 36)
        parity.assert_parity(st, f"gx={gx}")
        assert (g_depth[1] == 0).all() and (g_depth[0] > 0).mean() > 0.2


@pytest.mark.parametrize("case", [
    dict(W=8, H=4, grid=(12, 4, 28), P=1, kw=dict(hfov_rad=0.6, ambient=0.0, light_dir=(0.0, 1.0, 0.0))),
    dict(W=24, H=20, grid=(20, 8, 12), P=256, kw=dict(hfov_rad=2.6, ambient=1.0, miss_depth=-1.0, sky_rgb=(0, 255, 3))),
    dict(W=136, H=68, grid=(16, 32, 16), P=7, kw=dict(hfov_rad=1.2, light_dir=(-1.0, -0.2, 0.0), miss_depth=1000.0)),
    dict(W=64, H=36, grid=(36, 12, 8), P=16, kw=dict(light_dir=(0.0, 0.0, -3.0), ambient=0.5)),
    dict(W=512, H=288, grid=(16, 8, 16), P=16, kw=dict(hfov_rad=1.0)),       # 4608 tiles per observation
])
def test_descriptor_corners(oracle, case):
    """Descriptor fields away from the workloads' defaults: smallest image, image sizes that are no
    powers of two, narrow and very wide fields of view, one-entry and 256-entry palettes, lights along
    an axis and from below, ambient 0 and 1, other sky colours and miss depths, flat and full-height grids;
    boxes and cameras inside and outside the grid."""
    gx, gy, gz = case["grid"]
    W, H, P = case["W"], case["H"], case["P"]
    rng = np.random.default_rng(gx * 1000 + W)
    E, A, nb = 3, 2, 5
    if P > 1:
        grid = ((rng.random((E, gy, gz, gx)) < 0.12) * rng.integers(1, P, size=(E, gy, gz, gx))).astype(np.uint8)
        grid[:, 0] = 1                                   # a floor
    else:                                                # one palette entry: id 0 is "empty", so only boxes show
        grid = np.zeros((E, gy, gz, gx), np.uint8)
    boxes = np.zeros((E, nb, 8), np.int32)
    count = np.full(E, nb, np.int32)
    for e in range(E):
        items = []
        for _ in range(nb):
            c = rng.uniform([1, 1, 1], [gx - 1, gy - 1, gz - 1])
            h = rng.uniform(0.2, 1.2, 3)
            items.append((tuple(c - h), tuple(c + h), int(rng.integers(0, P))))
        boxes[e] = box_rows(items)
    cams = []
    for o in range(E * A):
        inside = o % 3 != 2
        pos = rng.uniform([1, 1.2, 1], [gx - 1, gy - 0.5, gz - 1]) if inside else \
            np.array([gx / 2, gy / 2, gz / 2]) + rng.normal(0, 1, 3) * np.array([gx, gy, gz])
        tgt = np.array([gx / 2, gy / 3, gz / 2]) + rng.normal(0, 2, 3)
        v = tgt - pos
        yaw = math.atan2(v[0], v[2]); pitch = math.atan2(v[1], math.hypot(v[0], v[2]))
        cams.append(cam_row(*pos, yaw, float(np.clip(pitch, -1.3, 1.3))))
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, _pal(E, P, seed=W), np.stack(cams), W, H, boxes=boxes,
                                                box_count=count, agents=A, max_boxes=nb, **case["kw"])
    assert status == 0
    parity.assert_parity(st, f"descriptor corner {W}x{H}")
    assert st["pixels"] == E * A * W * H
    miss = case["kw"].get("miss_depth", 0.0)
    assert (g_depth != miss).mean() > 0.05            # something was hit


def test_longest_grid_axis_thousand_steps(oracle):
    """The largest grid dimension the ABI takes (1024): rays that cross about a thousand cells before they
    hit a far wall.  Crossing times are accumulated in float, so this is where the depth error is largest
    (bounded by steps x 2^-24 relative, inside the 1e-4 bar) and where the walk's exit margin is widest."""
    gx, gy, gz = 1024, 4, 8
    grid = np.zeros((2, gy, gz, gx), np.uint8)
    grid[:, 0] = 1                                  # floor
    grid[0, :, :, 1020] = 2                         # a wall across the far end
    grid[1, :, :, 3] = 3                            # env 1: the wall at the near end, seen from the far end
    grid[:, 1, 4, 500] = 4                          # a lone voxel on the way, beside the view axis
    cams = np.stack([cam_row(0.5, 2.0, 3.6, math.pi / 2, 0.0),            # looks along +x
                     cam_row(1023.4, 2.1, 4.2, -math.pi / 2, 0.0002)])    # looks along -x
    # a field of view so narrow that the whole image stays inside the 8 x 4 cross-section for 1000 cells
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, _pal(2, 8), cams, 64, 36, hfov_rad=0.003)
    assert status == 0
    parity.assert_parity(st, "1024-long grid")
    assert (g_depth[0] > 1000).mean() > 0.3 and (g_depth[1] > 1000).mean() > 0.3     # the far walls are what is seen


def test_bounded_wait_runs_out_and_reports_a_status():
    """Failure detection without a fault: the staging copy is withheld, every CTA's bounded wait gives
    up, the host reads a timeout status, and the same batch renders normally afterwards."""
    from gpu_util import upload_scene
    B = _binding()
    cfg = scenes.config("tiny")
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    batch.set_cameras(sc["cams"].cuda())
    rgb, depth = batch.alloc_outputs()
    batch.render_batch(rgb, depth)
    good = rgb.clone()
    rgb.fill_(9)
    batch.debug_staging(True, 64)
    batch.render_batch(rgb, depth)
    with pytest.raises(B.MvError) as ei:
        batch.query_status(clear=True)
    assert ei.value.code == -5
    assert bool((rgb == 9).all())                       # the kernel left the outputs alone
    batch.debug_staging(False)
    batch.render_batch(rgb, depth)
    assert batch.query_status() == 0 and torch.equal(rgb, good)
    batch.destroy()


def test_translation_and_occlusion_invariants_on_gpu(oracle):
    """Shifting world, boxes and camera by whole voxels leaves the frames bit-identical; geometry added
    strictly behind a wall changes nothing."""
    rng = np.random.default_rng(5)
    W, H = 64, 36
    small = ((rng.random((6, 6, 6)) < 0.15) * rng.integers(1, 4, size=(6, 6, 6))).astype(np.uint8)
    a = np.zeros((1, 16, 16, 16), np.uint8); a[0, 1:7, 1:7, 1:7] = small
    b = np.zeros((1, 16, 16, 16), np.uint8); b[0, 5:11, 8:14, 3:9] = small            # shift (x+2, y+4, z+7)
    pal = _pal(1, 4)
    bx_a = box_rows([((2.25, 2.5, 1.75), (3.0, 3.25, 2.5), 2)])[None]
    bx_b = box_rows([((4.25, 6.5, 8.75), (5.0, 7.25, 9.5), 2)])[None]
    ra = _render_custom(oracle, a, pal, cam_row(0.5, 3.25, 0.75, 0.6, -0.1)[None], W, H, boxes=bx_a,
                        box_count=np.array([1]), max_boxes=1, check=False)
    rb = _render_custom(oracle, b, pal, cam_row(2.5, 7.25, 7.75, 0.6, -0.1)[None], W, H, boxes=bx_b,
                        box_count=np.array([1]), max_boxes=1, check=False)
    assert (ra[0] == rb[0]).all() and (ra[1] == rb[1]).all() and (ra[1] > 0).mean() > 0.05
    # occlusion
    g = np.zeros((1, 8, 16, 16), np.uint8); g[0, 0] = 1; g[0, :, 8, :] = 1
    g2 = g.copy(); g2[0, 1:5, 10:14, 3:12] = 2
    cam = cam_row(8.5, 1.75, 2.5, 0.0, 0.0)[None]
    pal3 = _pal(1, 3)
    hidden = box_rows([((4, 1, 10), (6, 3, 12), 2)])[None]
    r0 = _render_custom(oracle, g, pal3, cam, W, H, boxes=hidden, box_count=np.array([0]), max_boxes=1, check=False)
    r1 = _render_custom(oracle, g2, pal3, cam, W, H, boxes=hidden, box_count=np.array([1]), max_boxes=1, check=False)
    assert (r0[0] == r1[0]).all() and (r0[1] == r1[1]).all()


def test_fuzz_cameras_anywhere_with_boxes(oracle):
    """Random small worlds, cameras inside, outside, high above and inside solids, random boxes."""
    rng = np.random.default_rng(99)
    E, A, gx, gy, gz, W, H, nb = 24, 2, 16, 8, 12, 64, 36, 6
    grid = ((rng.random((E, gy, gz, gx)) < rng.uniform(0.02, 0.35, size=(E, 1, 1, 1))) *
            rng.integers(1, 8, size=(E, gy, gz, gx))).astype(np.uint8)
    grid[::3, 0] = 1
    grid[5] = 0                                                  # an empty world
    pal = _pal(E, 8, seed=4)
    boxes = np.zeros((E, nb, 8), np.int32)
    for e in range(E):
        rows = []
        for b in range(nb):
            c = rng.uniform([-3, -2, -3], [gx + 3, gy + 2, gz + 3]); s = rng.uniform(0.2, 3.0, 3)
            rows.append((c - s / 2, c + s / 2, int(rng.integers(0, 8))))
        boxes[e] = box_rows(rows)
    count = rng.integers(0, nb + 1, size=E)
    cams = []
    for o in range(E * A):
        pos = rng.uniform([-6, -4, -6], [gx + 6, gy + 6, gz + 6])
        if o % 4 == 0:
            pos = rng.uniform([0.5, 0.5, 0.5], [gx - 0.5, gy - 0.5, gz - 0.5])
        tgt = np.array([gx / 2, gy / 2, gz / 2]) + rng.normal(0, 3, 3)
        v = tgt - pos
        yaw = math.atan2(v[0], v[2]); pitch = math.atan2(v[1], math.hypot(v[0], v[2]))
        cams.append(cam_row(*pos, yaw, float(np.clip(pitch, -1.4, 1.4)), self_box=int(rng.integers(-1, nb))))
    g_rgb, g_depth, status, st = _render_custom(oracle, grid, pal, np.stack(cams), W, H, boxes=boxes,
                                                box_count=count, agents=A, max_boxes=nb)
    assert status == 0
    parity.assert_parity(st, "fuzz")
    assert st["pixels"] == E * A * W * H and (g_depth > 0).mean() > 0.2


def test_cta_per_environment_equals_cta_per_observation():
    """The render kernel may give one CTA a whole environment (block staged once for all its agents)
    or a single observation; both shapes must write the same bytes, overlay and bad cameras included."""
    from gpu_util import upload_scene
    B = _binding()
    cfg = scenes.config("rooms_boxes", num_envs=5)
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg, 0, max_overlay_rects=2))
    upload_scene(batch, sc)
    cams = sc["cams"].clone()
    cams[7, 3] = torch.tensor([float("nan")]).view(torch.int32)              # one bad camera in the middle of an env
    d_cams = cams.cuda().contiguous()
    rects = torch.zeros(cfg.num_obs, 2, 4, dtype=torch.int32)
    rects[:, 0, 0] = 4 | (2 << 16); rects[:, 0, 1] = 100 | (6 << 16); rects[:, 0, 2] = 0x20C0FF
    rects[:, 1, 0] = 60 | (40 << 16); rects[:, 1, 1] = 90 | (71 << 16); rects[:, 1, 2] = 0x00FF00
    count = (torch.arange(cfg.num_obs, dtype=torch.int32) % 3)
    batch.set_overlays(rects.cuda(), count.cuda())
    out = {}
    for apc in (1, cfg.agents):
        batch.debug_agents_per_cta(apc)
        batch.set_cameras(d_cams)                                            # (sets the bad-camera flag again)
        rgb, depth = batch.alloc_outputs()
        rgb.fill_(9); depth.fill_(-3.0)
        batch.render_batch(rgb, depth)
        assert batch.query_status(clear=True) == B.FLAG_BAD_CAMERA
        out[apc] = (rgb.cpu(), depth.cpu())
    assert torch.equal(out[1][0], out[cfg.agents][0]) and torch.equal(out[1][1], out[cfg.agents][1])
    assert (out[1][0][7] == torch.tensor([127, 178, 229], dtype=torch.uint8)).all()
    with pytest.raises(B.MvError):
        batch.debug_agents_per_cta(3)
    batch.debug_agents_per_cta(0)
    batch.destroy()


def test_twenty_agents_in_one_cta(oracle):
    """More agents per CTA than one pass of the CTA's threads over the per-agent set-up covers
    (20 x 24 table slots > 384 threads): every agent's frame must still equal the per-observation
    shape's, and the oracle's."""
    from gpu_util import upload_scene, scene_to_numpy
    B = _binding()
    cfg = scenes.config("tiny", num_envs=3, agents=20, seed=77)
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    batch.set_cameras(sc["cams"].cuda().contiguous())
    out = {}
    for apc in (1, cfg.agents):
        batch.debug_agents_per_cta(apc)
        rgb, depth = batch.alloc_outputs()
        rgb.fill_(9); depth.fill_(-3.0)
        batch.render_batch(rgb, depth)
        assert batch.query_status() == 0
        out[apc] = (rgb.cpu(), depth.cpu())
    assert torch.equal(out[1][0], out[20][0]) and torch.equal(out[1][1], out[20][1])
    st = parity.compare_scene(oracle, cfg, scene_to_numpy(sc), range(cfg.num_obs), out[20][0].numpy(), out[20][1].numpy())
    parity.assert_parity(st, "20 agents per CTA")
    batch.destroy()


def test_two_batches_of_different_shape_alive_together():
    """The kernel's shared-memory cap is per function and device, not per batch: a small batch created
    after a large one must not make the large one's launch fail."""
    from gpu_util import upload_scene
    B = _binding()
    big_cfg = scenes.config("headline", num_envs=3)
    small_cfg = scenes.config("tiny")
    big_sc, small_sc = scenes.make_scene(big_cfg), scenes.make_scene(small_cfg)
    big = B.Batch(B.desc_from_config(big_cfg))
    upload_scene(big, big_sc)
    big.set_cameras(big_sc["cams"].cuda())
    small = B.Batch(B.desc_from_config(small_cfg))
    upload_scene(small, small_sc)
    small.set_cameras(small_sc["cams"].cuda())
    frames = []
    for b in (big, small, big):
        rgb, depth = b.alloc_outputs()
        b.render_batch(rgb, depth)
        assert b.query_status() == 0
        frames.append((rgb.cpu(), depth.cpu()))
    assert torch.equal(frames[0][0], frames[2][0]) and torch.equal(frames[0][1], frames[2][1])
    assert (frames[0][1] > 0).any() and (frames[1][1] > 0).any()
    big.destroy(); small.destroy()


def _pitch_with_exact_zero_dy(W, hfov=np.float32(np.pi / 2)):
    """A float32 pitch for which the image row with b = H-1-2py = 1 has d_y = fma(1, Us_y, F_y) == 0
    exactly: F_y = float(sin p) and Us_y = float(cos p * ku), ku = tan(hfov/2)/W, must cancel.  Us_y is
    the same float over thousands of neighbouring pitches while float(sin p) steps through every float,
    so a short scan around -atan(ku) finds one.  Candidates whose double values sit close to a float
    rounding boundary are skipped, so that a last-place difference between two libm's cannot matter."""
    ku = math.tan(float(hfov) / 2.0) / W
    p0 = np.float32(-math.atan(ku))
    bits = p0.view(np.int32) + np.arange(-200000, 200000, dtype=np.int64)
    p = bits.astype(np.int32).view(np.float32)
    sp64, us64 = np.sin(p.astype(np.float64)), np.cos(p.astype(np.float64)) * ku
    sp, us = sp64.astype(np.float32), us64.astype(np.float32)
    ok = sp == -us
    ulp = np.spacing(np.abs(sp))
    safe = (np.abs(sp64 - sp) < 0.4 * ulp) & (np.abs(us64 - us) < 0.4 * np.spacing(us))
    idx = np.nonzero(ok & safe)[0]
    return (p[idx[len(idx) // 2]], len(idx)) if len(idx) else (None, 0)


def test_ray_direction_component_exactly_zero(oracle):
    """Even image sizes never put a pixel centre on the view axis, so an exactly zero direction component
    needs a pitch chosen for it: one whole image row then has d_y == 0 and travels at constant height.
    The library replaces the zero by 1e-30; away from the doubly degenerate case (eye exactly on a face
    AND component exactly zero) that must give the oracle's result: boxes whose height range contains the
    eye are hit, the others are missed, and the walk never changes layer."""
    W, H = 128, 72
    pitch, found = _pitch_with_exact_zero_dy(W)
    assert pitch is not None, "no float32 pitch with an exactly zero d_y in 400000 candidates"
    # the row with b = 1
    py0 = (H - 2) // 2
    gx, gy, gz = 32, 8, 32
    grid = np.zeros((1, gy, gz, gx), np.uint8)
    grid[0, 0] = 1
    grid[0, :, 0, :] = 2; grid[0, :, gz - 1, :] = 2; grid[0, :, :, 0] = 3; grid[0, :, :, gx - 1] = 3
    grid[0, 1:4, 20, 8:12] = 4                                   # a low wall the zero row passes over (eye above it)
    grid[0, 1:6, 24, 18:24] = 5                                  # a taller wall that it hits
    eye = (14.37, 4.41, 6.29)
    boxes = box_rows([((12.0, 4.0, 12.0), (13.0, 5.0, 13.0), 6),      # height range contains the eye: hit
                      ((15.0, 4.5, 12.0), (16.0, 5.5, 13.0), 7),      # starts above the eye: missed by the zero row
                      ((17.0, 3.0, 11.0), (18.0, 4.4, 12.0), 8)])[None]   # ends just below the eye: missed
    cams = np.stack([cam_row(*eye, 0.0, pitch), cam_row(*eye, 0.35, pitch)])
    grid2 = np.repeat(grid, 2, axis=0)
    g_rgb, g_depth, status, st = _render_custom(oracle, grid2, _pal(2, 10), cams, W, H, boxes=np.repeat(boxes, 2, axis=0),
                                                box_count=np.array([3, 3]), max_boxes=3)
    assert status == 0
    parity.assert_parity(st, "exact zero d_y")
    # the oracle confirms that the row really has d_y == 0: every hit in it keeps the eye's layer (voxels)
    od = oracle.make_desc((gy, gz, gx), 3, W, H, 10)
    for o in range(2):
        _, o_depth, ids = oracle.render_obs(od, grid2[o], boxes[0], 3, _pal(2, 10)[o], cams[o])
        row = ids[py0]
        vox = row[:, 0] == 0
        assert vox.any() and ((row[vox, 1] // (gx * gz)) == 4).all()          # voxel index -> layer 4 = floor(eye y)
        hit_boxes = set(row[row[:, 0] == 1, 1].tolist())
        assert hit_boxes <= {0} and (o == 1 or 0 in hit_boxes)
        # and the library's row agrees pixel for pixel
        assert parity.depth_close(g_depth[o, py0], o_depth[py0]).all()


def test_host_step_allocation_failure_is_reported_and_can_be_retried():
    """mv_step_host allocates its device-side frame buffers on first use.  When that cannot be satisfied
    (here: 100,000 observations of 640x480, over 200 GB of frames) the call reports OUT_OF_MEMORY, keeps
    nothing half-allocated, and a second call fails the same clean way instead of launching on null
    pointers.  No kernel runs in this test."""
    B = _binding()
    E = 100000
    desc = B.make_desc(E, 1, (4, 4, 4), 0, 640, 480, 2)
    batch = B.Batch(desc)
    dev = torch.device("cuda", 0)
    batch.upload_worlds(0, E, torch.zeros(E, 4, 4, 4, dtype=torch.uint8, device=dev), None, None,
                        torch.zeros(E, 2, 3, dtype=torch.uint8, device=dev))
    cams = torch.zeros(E, 6, dtype=torch.int32)
    rgb = torch.zeros(16, dtype=torch.uint8)          # never touched: the allocation fails before any copy
    depth = torch.zeros(16, dtype=torch.float32)
    for _ in range(2):
        with pytest.raises(B.MvError) as ei:
            batch.step_host(cams, rgb, depth)
        assert ei.value.code == -2
    assert batch.query_status() == 0
    batch.destroy()
    # the context is intact: an ordinary batch still renders
    from gpu_util import render_scene
    cfg = scenes.config("tiny")
    assert render_scene(cfg, scenes.make_scene(cfg))[2] == 0
