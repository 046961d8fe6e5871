"""GUI overlay and agent motion on the GPU (through the C ABI) against the oracle."""
import numpy as np
import pytest
import torch

from paper_2107_08170_b200 import scenes
import parity

pytestmark = pytest.mark.gpu


def _random_rects(oracle, num_obs, max_rects, W, H, seed):
    rng = np.random.default_rng(seed)
    rects = np.zeros((num_obs, max_rects), oracle.RECT_DTYPE)
    count = rng.integers(0, max_rects + 2, size=num_obs).astype(np.int32)       # some beyond the limit
    for o in range(num_obs):
        for r in range(max_rects):
            x0, y0 = int(rng.integers(-8, W)), int(rng.integers(-4, H))
            rects[o, r] = (x0, y0, x0 + int(rng.integers(0, W // 2)), y0 + int(rng.integers(0, H // 3)),
                           tuple(int(v) for v in rng.integers(0, 256, 3)), 0, 0)
        rects[o, 0] = (0, 0, int(rng.integers(0, W + 1)), 2, (250, 240, 30), 0, 0)   # a time-left bar
    return rects, count


def test_overlay_matches_oracle_and_leaves_depth_alone(oracle):
    from paper_2107_08170_b200 import binding as B
    from gpu_util import upload_scene, scene_to_numpy
    cfg = scenes.config("rooms_boxes", num_envs=3)
    sc = scenes.make_scene(cfg)
    M = 4
    batch = B.Batch(B.desc_from_config(cfg, max_overlay_rects=M))
    upload_scene(batch, sc)
    batch.set_cameras(sc["cams"].cuda())
    rgb0, depth0 = batch.alloc_outputs()
    batch.render_batch(rgb0, depth0)                                          # no overlay yet
    rects, count = _random_rects(oracle, cfg.num_obs, M, cfg.width, cfg.height, 5)
    d_rects = torch.from_numpy(rects.view(np.int32).reshape(cfg.num_obs, M, 4)).cuda()
    batch.set_overlays(d_rects, torch.from_numpy(count).cuda())
    rgb1, depth1 = batch.alloc_outputs()
    batch.render_batch(rgb1, depth1)
    assert torch.equal(depth0, depth1)
    base = rgb0.cpu().numpy()
    got = rgb1.cpu().numpy()
    painted = 0
    for o in range(cfg.num_obs):
        want = oracle.overlay(base[o].copy(), rects[o], min(max(int(count[o]), 0), M))
        assert (got[o] == want).all(), o                                      # integer work: bit-exact
        painted += int((want != base[o]).any(axis=-1).sum())
    assert painted > 1000
    # the 3D part under the overlay is the ordinary render: check it against the oracle too
    st = parity.compare_scene(oracle, cfg, scene_to_numpy(sc), range(cfg.num_obs), base, depth0.cpu().numpy())
    parity.assert_parity(st, "overlay base")
    batch.set_overlays(None, None)
    rgb2, depth2 = batch.alloc_outputs()
    batch.render_batch(rgb2, depth2)
    assert torch.equal(rgb2, rgb0)
    batch.destroy()


def test_move_agents_matches_oracle_then_renders(oracle):
    from paper_2107_08170_b200 import binding as B
    from gpu_util import upload_scene, scene_to_numpy
    cfg = scenes.config("rooms_boxes", num_envs=6)
    sc = scenes.make_scene(cfg)
    scn = scene_to_numpy(sc)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    d_cams = sc["cams"].cuda().contiguous()
    cams = scn["cams"].copy()
    boxes = scn["boxes"].copy()
    rng = np.random.default_rng(1)
    shape = (0.25, 0.75, 0.25)
    mismatched = blocked = 0
    for step in range(12):
        moves = np.stack([rng.uniform(-0.45, 0.45, cfg.num_obs), rng.uniform(-0.2, 0.2, cfg.num_obs),
                          rng.normal(0, 0.3, cfg.num_obs), rng.normal(0, 0.1, cfg.num_obs)], 1).astype(np.float32)
        batch.move_agents(d_cams, torch.from_numpy(moves).cuda())
        for o in range(cfg.num_obs):
            e = o // cfg.agents
            f = cams[o, :5].view(np.float32)
            new, kept = oracle.move_agent(scn["grid"][e], f, moves[o], shape, 1.0)
            blocked += kept != 3
            cams[o, :5] = new.view(np.int32)
            sb = cams[o, 5]
            lo = np.float32(new[:3]) - np.float32([0.25, 0.75, 0.25])
            hi = np.float32(new[:3]) + np.float32([0.25, 0.25, 0.25])
            boxes[e, sb, :3] = lo.astype(np.float32).view(np.int32)
            boxes[e, sb, 3:6] = hi.astype(np.float32).view(np.int32)
        g = d_cams.cpu().numpy()
        diff = np.nonzero((g != cams).any(axis=1))[0]
        mismatched += len(diff)
        for o in diff:                           # a mismatching agent is off by one unit in the last place, in x or z only
            d = np.abs(g[o, :5].astype(np.int64) - cams[o, :5].astype(np.int64))
            assert d[1] == 0 and d[3] == 0 and d[4] == 0 and d[0] <= 1 and d[2] <= 1, (step, o, d)
        cams = g.copy()                          # a 1-ulp difference could flip a later collision: continue from the GPU's state
        for o in range(cfg.num_obs):             # and the boxes the GPU now holds for those agents
            e = o // cfg.agents
            f = cams[o, :5].view(np.float32)
            boxes[e, cams[o, 5], :3] = (f[:3] - np.float32([0.25, 0.75, 0.25])).view(np.int32)
            boxes[e, cams[o, 5], 3:6] = (f[:3] + np.float32([0.25, 0.25, 0.25])).view(np.int32)
    assert blocked > 10
    # double sin/cos differ by an ulp between libm and CUDA at most in rare roundings
    print(f"move_agents: {mismatched} of {12 * cfg.num_obs} agent-steps differ from the oracle (each by <= 1 ulp)")
    assert mismatched <= 1, mismatched
    rgb, depth = batch.alloc_outputs()
    batch.render_batch(rgb, depth)               # no mv_set_cameras: the move rebuilt the ray bases
    scn2 = dict(scn, cams=cams, boxes=boxes)
    st = parity.compare_scene(oracle, cfg, scn2, range(cfg.num_obs), rgb.cpu().numpy(), depth.cpu().numpy())
    parity.assert_parity(st, "after moves")
    assert batch.query_status() == 0
    batch.destroy()


def test_move_agents_headline_scale_properties(oracle):
    """At the headline size: agents never end inside a voxel; yaw/pitch follow the commands."""
    from paper_2107_08170_b200 import workload
    cfg = scenes.config("headline", num_envs=2048)
    batch, d_cams, kept = workload.build_batch(cfg, 0, keep_envs=[0, 1000, 2047])
    g = torch.Generator(device="cuda").manual_seed(0)
    # stand every agent with its feet on its surface (eye 0.75 above the cell floor)
    yf = d_cams[:, 1].contiguous().view(torch.float32)
    d_cams[:, 1] = (yf.floor() + 0.75).view(torch.int32)
    for e in kept:
        kept[e]["cams"][0, 1] = d_cams[e, 1].item()
    before = d_cams.clone()
    moves = (torch.rand(cfg.num_obs, 4, device="cuda", generator=g) - 0.5) * torch.tensor([1.0, 0.5, 0.6, 0.2], device="cuda")
    batch.move_agents(d_cams, moves.contiguous())
    after = d_cams.cpu().numpy()
    for e in kept:
        f0 = kept[e]["cams"][0, :5].view(np.float32)
        new, _ = oracle.move_agent(kept[e]["grid"], f0, moves[e].cpu().numpy(), (0.25, 0.75, 0.25), 1.0)
        assert (after[e, :5].view(np.float32) == new).all()
    fa = np.ascontiguousarray(after[:, :5]).view(np.float32)
    fb = np.ascontiguousarray(before.cpu().numpy()[:, :5]).view(np.float32)
    assert np.allclose(fa[:, 3], fb[:, 3] + moves[:, 2].cpu().numpy(), atol=1e-6)
    assert (np.abs(fa[:, 4]) <= 1.0).all() and (fa[:, 1] == fb[:, 1]).all()
    assert ((fa[:, 0] != fb[:, 0]) | (fa[:, 2] != fb[:, 2])).mean() > 0.2
    batch.destroy()


@pytest.mark.parametrize("name,envs,max_out", [("tiny", 4, 64), ("rooms", 5, 512), ("headline", 3, 4096)])
def test_merge_voxels_matches_oracle(oracle, name, envs, max_out):
    from paper_2107_08170_b200 import binding as B
    from gpu_util import upload_scene
    cfg = scenes.config(name, num_envs=envs)
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    boxes, counts = batch.merge_voxels(1, envs - 1, max_out)                 # a sub-range, on purpose
    torch.cuda.synchronize()
    boxes, counts = boxes.cpu().numpy(), counts.cpu().numpy()
    for n, e in enumerate(range(1, envs)):
        want, total = oracle.merge_voxels(sc["grid"][e].numpy(), cfg.palette_size, max_out)
        assert counts[n] == total, (e, counts[n], total)
        assert (boxes[n, :len(want)] == want).all()                            # same boxes, same order
    # too small an output array: the count still reports what the sweep produces
    b2, c2 = batch.merge_voxels(0, 1, 3)
    assert int(c2[0]) == oracle.merge_voxels(sc["grid"][0].numpy(), cfg.palette_size, 3)[1]
    batch.destroy()


def test_merged_boxes_render_like_the_grid_on_gpu(oracle):
    """Primitives versus grid steps: the merged boxes of a rooms world, rendered through the box path
    with an empty grid, give the frames of the grid path (off the box seams)."""
    from paper_2107_08170_b200 import binding as B
    from gpu_util import upload_scene
    cfg = scenes.config("rooms", num_envs=4)
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    batch.set_cameras(sc["cams"].cuda())
    rgb_g, depth_g = batch.alloc_outputs()
    batch.render_batch(rgb_g, depth_g)
    boxes, counts = batch.merge_voxels(0, cfg.num_envs, 256)
    assert int(counts.max()) <= 256
    cfg_b = scenes.config("rooms", num_envs=4, movable_boxes=256)
    bb = B.Batch(B.desc_from_config(cfg_b))
    empty = torch.zeros_like(sc["grid"]).cuda()
    bb.upload_worlds(0, cfg.num_envs, empty, boxes.contiguous(), counts.contiguous(), sc["palette"].cuda())
    bb.set_cameras(sc["cams"].cuda())
    rgb_b, depth_b = bb.alloc_outputs()
    bb.render_batch(rgb_b, depth_b)
    same = (rgb_g == rgb_b).all(dim=-1) & ((depth_g - depth_b).abs() <= 1e-4 * depth_g.clamp(min=1e-3))
    assert float(same.float().mean()) > 0.999
    batch.destroy(); bb.destroy()


def test_tall_grid_with_multi_word_columns(oracle):
    """Grids more than 32 voxels high keep several occupancy words per (x, z) column and take the indexed
    flavour of the walk; render, merge and agent motion all address voxels through the same index."""
    from paper_2107_08170_b200 import binding as B
    from gpu_util import upload_scene, scene_to_numpy
    from helpers import cam_row
    cfg = scenes.config("tiny", grid=(16, 40, 20), num_envs=3, seed=7, movable_boxes=3)
    sc = scenes.make_scene(cfg)
    rng = np.random.default_rng(5)
    grid = sc["grid"].numpy().copy()
    grid[:, 30:38, 3:9, 5:9] = rng.integers(0, 4, size=(3, 8, 6, 4)).astype(np.uint8)   # voxels above height 32
    sc["grid"] = torch.from_numpy(grid)
    cams = sc["cams"].numpy().copy()
    cams[1, :5] = np.array([8.3, 34.2, 12.7, 2.6, -0.4], np.float32).view(np.int32)      # an eye up there, looking down
    cams[2, :5] = np.array([-3.0, 45.0, 9.5, 1.2, -0.7], np.float32).view(np.int32)      # and one outside the grid
    sc["cams"] = torch.from_numpy(cams)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    batch.set_cameras(sc["cams"].cuda())
    rgb, depth = batch.alloc_outputs()
    batch.render_batch(rgb, depth)
    assert batch.query_status() == 0
    st = parity.compare_scene(oracle, cfg, scene_to_numpy(sc), range(cfg.num_obs), rgb.cpu().numpy(), depth.cpu().numpy())
    parity.assert_parity(st, "tall grid")
    assert (depth[1] > 0).float().mean() > 0.5
    # the same frames with the occupancy read from global memory
    rgb2, depth2 = batch.alloc_outputs()
    batch.debug_occupancy_in_global(True)
    batch.render_batch(rgb2, depth2)
    batch.debug_occupancy_in_global(False)
    assert torch.equal(rgb, rgb2) and torch.equal(depth, depth2)
    # merge: same boxes, same order as the serial sweep
    boxes, counts = batch.merge_voxels(0, 3, 512)
    for e in range(3):
        want, total = oracle.merge_voxels(grid[e], cfg.palette_size, 512)
        assert int(counts[e]) == total and (boxes[e, :len(want)].cpu().numpy() == want).all()
    # agent motion: collision against voxels above height 32
    d_cams = torch.from_numpy(np.stack([cam_row(7.0, 33.0, 2.0, 0.0, 0.0), cam_row(7.0, 20.0, 2.0, 0.0, 0.0),
                                        cam_row(7.0, 33.0, 2.0, 0.0, 0.0)])).cuda()
    solid = np.zeros_like(grid); solid[:, 30:38, 3:9, 5:9] = 1
    sc2 = dict(sc, grid=torch.from_numpy(np.where(solid > 0, 1, 0).astype(np.uint8)))
    upload_scene(batch, sc2)
    moves = torch.tensor([[2.0, 0, 0, 0]] * 3, dtype=torch.float32).cuda()
    batch.move_agents(d_cams, moves)
    after = d_cams.cpu().numpy()[:, :5].view(np.float32)
    for o in range(3):
        new, _ = oracle.move_agent(sc2["grid"][o].numpy(), np.array([7.0, 33.0 if o != 1 else 20.0, 2.0, 0.0, 0.0], np.float32),
                                   np.array([2.0, 0, 0, 0], np.float32), (0.25, 0.75, 0.25), 1.0)
        assert (after[o] == new).all(), (o, after[o], new)
    assert after[0, 2] == 2.0 and after[1, 2] == 4.0          # blocked by the block at z = 3 up there, free below it
    batch.destroy()


def test_scene_generators_give_the_same_arrays_on_cpu_and_gpu():
    """Seeded inputs must not depend on the device or on the order in which a device applies writes
    (two pillars of a rooms world can fall on the same cell): 1024 envs generated on the GPU twice and
    on the CPU once are the same arrays."""
    for name in ("rooms_boxes", "headline"):
        cfg = scenes.config(name, num_envs=1024 if name == "rooms_boxes" else 64)
        cpu = scenes.make_scene(cfg)
        for _ in range(2):
            gpu = scenes.make_scene(cfg, device=torch.device("cuda", 0))
            for k in ("grid", "palette", "boxes", "box_count", "cams"):
                assert torch.equal(cpu[k], gpu[k].cpu()), (name, k)
