"""Pins for the oracle's overlay and agent-motion functions (closed forms and hand-made cases)."""
import math

import numpy as np


def test_overlay_rectangles_order_and_clipping(oracle):
    H, W = 8, 16
    rgb = np.full((H, W, 3), 9, np.uint8)
    rects = np.zeros(3, oracle.RECT_DTYPE)
    rects[0] = (0, 0, 10, 2, (255, 0, 0), 0, 0)            # time bar: rows 0-1, columns 0-9
    rects[1] = (8, 1, 40, 3, (0, 255, 0), 0, 0)            # overlaps the bar, runs off the right edge
    rects[2] = (5, 5, 5, 7, (1, 2, 3), 0, 0)               # empty (x1 == x0): paints nothing
    out = oracle.overlay(rgb.copy(), rects, 3)
    want = rgb.copy()
    want[0:2, 0:10] = (255, 0, 0)
    want[1:3, 8:16] = (0, 255, 0)                          # later rectangle on top, clipped at W
    assert (out == want).all()
    assert (oracle.overlay(rgb.copy(), rects, 1)[0:2, 0:10] == (255, 0, 0)).all()
    assert (oracle.overlay(rgb.copy(), rects, 0) == rgb).all()
    neg = np.zeros(1, oracle.RECT_DTYPE); neg[0] = (-5, -5, 2, 2, (7, 7, 7), 0, 0)
    o2 = oracle.overlay(rgb.copy(), neg, 1)
    assert (o2[0:2, 0:2] == 7).all() and (o2[2:, :] == 9).all() and (o2[:2, 2:] == 9).all()


def _room():
    g = np.zeros((8, 16, 16), np.uint8)
    g[0] = 1                      # floor
    g[:, 10, :] = 1               # wall plane z in [10, 11)
    g[1:, :, 12] = 1              # wall plane x in [12, 13)
    return g


def test_free_motion_follows_yaw_convention(oracle):
    g = _room()
    cam, kept = oracle.move_agent(g, (5.0, 1.75, 5.0, 0.0, 0.0), (0.5, 0.0, 0.0, 0.0))
    assert kept == 3 and np.allclose(cam[:3], (5.0, 1.75, 5.5)) and cam[3] == 0
    cam, kept = oracle.move_agent(g, (5.0, 1.75, 5.0, 0.0, 0.0), (0.0, 0.5, 0.0, 0.0))
    assert kept == 3 and np.allclose(cam[:3], (5.5, 1.75, 5.0))            # strafe right = +x at yaw 0
    cam, kept = oracle.move_agent(g, (5.0, 1.75, 5.0, 0.0, 0.0), (1.0, 0.0, math.pi / 2, 0.0))
    assert np.allclose(cam[:3], (6.0, 1.75, 5.0), atol=1e-6)               # turn first, then walk along +x
    assert abs(cam[3] - np.float32(math.pi / 2)) < 1e-7


def test_walls_block_and_allow_sliding(oracle):
    g = _room()
    # body half width 0.25: z + 0.25 must stay below 10 -> z = 9.6 + 0.2 would reach 10.05
    cam, kept = oracle.move_agent(g, (5.0, 1.75, 9.6, 0.0, 0.0), (0.2, 0.0, 0.0, 0.0))
    assert kept == 1 and cam[2] == np.float32(9.6)                         # z move rejected, x (no-op) kept
    cam, kept = oracle.move_agent(g, (5.0, 1.75, 9.6, 0.0, 0.0), (0.1, 0.0, 0.0, 0.0))
    assert kept == 3 and abs(cam[2] - 9.7) < 1e-6                          # 9.95 < 10: allowed
    # diagonal into the z-wall: the x component survives (sliding)
    cam, kept = oracle.move_agent(g, (5.0, 1.75, 9.6, math.pi / 4, 0.0), (0.4, 0.0, 0.0, 0.0))
    assert kept == 1 and abs(cam[0] - (5.0 + 0.4 * math.sin(math.pi / 4))) < 1e-6 and cam[2] == np.float32(9.6)
    # into the x-wall at x = 12
    cam, kept = oracle.move_agent(g, (11.6, 1.75, 5.0, math.pi / 2, 0.0), (0.3, 0.0, 0.0, 0.0))
    assert kept == 2 and cam[0] == np.float32(11.6)
    # leaving the grid is rejected; the floor under the feet (y - 0.75 = 1.0) does not block
    cam, kept = oracle.move_agent(g, (0.3, 1.75, 5.0, -math.pi / 2, 0.0), (0.2, 0.0, 0.0, 0.0))
    assert kept == 2 and cam[0] == np.float32(0.3)
    # a low ceiling voxel blocks: head at y + 0.25 = 2.0 touches cell j = 2
    g2 = _room(); g2[2, 6, 5] = 1
    cam, kept = oracle.move_agent(g2, (5.5, 1.75, 5.5, 0.0, 0.0), (0.5, 0.0, 0.0, 0.0))
    assert kept == 1 and cam[2] == np.float32(5.5)


def test_pitch_clamp_and_yaw_accumulation(oracle):
    g = _room()
    cam, _ = oracle.move_agent(g, (5.0, 1.75, 5.0, 1.0, 0.9), (0.0, 0.0, 0.25, 0.3), max_pitch=1.0)
    assert cam[3] == np.float32(1.25) and cam[4] == np.float32(1.0)
    cam, _ = oracle.move_agent(g, (5.0, 1.75, 5.0, 1.0, -0.9), (0.0, 0.0, 0.0, -0.3), max_pitch=1.0)
    assert cam[4] == np.float32(-1.0)


def test_many_random_moves_never_end_inside_a_voxel(oracle):
    from paper_2107_08170_b200 import scenes
    cfg = scenes.config("rooms_boxes", num_envs=2)
    sc = scenes.make_scene(cfg)
    g = sc["grid"][0].numpy()
    rng = np.random.default_rng(0)
    cam = np.ascontiguousarray(sc["cams"][0].numpy()[:5]).view(np.float32).copy()
    cam[1] = 1.75
    blocked = 0
    for _ in range(400):
        mv = (rng.uniform(-0.4, 0.4), rng.uniform(-0.2, 0.2), rng.normal(0, 0.3), rng.normal(0, 0.05))
        new, kept = oracle.move_agent(g, cam, mv)
        blocked += kept != 3
        lo = np.floor(new[:3] - np.float32([0.25, 0.75, 0.25])).astype(int)
        hi = np.floor(new[:3] + np.float32([0.25, 0.25, 0.25])).astype(int)
        if kept:                                           # a kept move leaves the body in free cells
            assert (g[lo[1]:hi[1] + 1, lo[2]:hi[2] + 1, lo[0]:hi[0] + 1] == 0).all()
        cam = new
    assert blocked > 0


def _paint(boxes, shape):
    gy, gz, gx = shape
    g = np.zeros(shape, np.int32)
    hits = np.zeros(shape, np.int32)
    for b in boxes:
        lo = b[:3].view(np.float32).astype(int); hi = b[3:6].view(np.float32).astype(int)
        g[lo[1]:hi[1], lo[2]:hi[2], lo[0]:hi[0]] = b[6]
        hits[lo[1]:hi[1], lo[2]:hi[2], lo[0]:hi[0]] += 1
    return g, hits


def test_merge_small_cases(oracle):
    g = np.zeros((4, 4, 4), np.uint8); g[1:3, 1:3, 1:3] = 2
    boxes, n = oracle.merge_voxels(g, 4)
    assert n == 1 and boxes[0, :6].view(np.float32).tolist() == [1, 1, 1, 3, 3, 3] and boxes[0, 6] == 2
    g[1:3, 1:3, 1] = 3                                   # a slab of another material splits it in two
    boxes, n = oracle.merge_voxels(g, 4)
    assert n == 2 and sorted(boxes[:, 6].tolist()) == [2, 3]
    # L shape in one layer: x-run first, so the long arm along x is one box and the rest another
    g = np.zeros((4, 4, 4), np.uint8); g[0, 0, 0:3] = 1; g[0, 1:3, 0] = 1
    boxes, n = oracle.merge_voxels(g, 2)
    assert n == 2
    assert boxes[0, :6].view(np.float32).tolist() == [0, 0, 0, 3, 1, 1]
    assert boxes[1, :6].view(np.float32).tolist() == [0, 0, 1, 1, 1, 3]
    assert oracle.merge_voxels(np.zeros((4, 4, 4), np.uint8), 2)[1] == 0


def test_merge_covers_exactly_and_is_compact(oracle):
    from paper_2107_08170_b200 import scenes
    for name, bound in (("rooms", 400), ("headline", 3000), ("tiny", 60)):
        cfg = scenes.config(name, num_envs=2)
        sc = scenes.make_scene(cfg)
        g = sc["grid"][1].numpy()
        boxes, n = oracle.merge_voxels(g, cfg.palette_size, 8192)
        assert n == len(boxes) and 0 < n <= bound, (name, n)
        painted, hits = _paint(boxes, g.shape)
        assert (painted == g).all()                      # union of the boxes is the grid, materials kept
        assert hits.max() == 1                           # and the boxes are disjoint
        assert n < int((g != 0).sum()) / 10


def test_merged_boxes_render_like_the_grid(oracle):
    from paper_2107_08170_b200 import scenes
    cfg = scenes.config("tiny")
    sc = scenes.make_scene(cfg)
    g = sc["grid"][2].numpy()
    boxes, n = oracle.merge_voxels(g, cfg.palette_size, 256)
    d_grid = oracle.desc_from_config(cfg)
    d_box = oracle.desc_from_config(cfg); d_box.max_boxes = n
    cam = sc["cams"][2].numpy()
    a = oracle.render_obs(d_grid, g, None, 0, sc["palette"][2].numpy(), cam)
    b = oracle.render_obs(d_box, np.zeros_like(g), boxes, n, sc["palette"][2].numpy(), cam)
    same = (a[0] == b[0]).all(axis=-1) & (np.abs(a[1] - b[1]) <= 1e-6 * np.maximum(a[1], 1e-3))
    assert same.mean() > 0.999
