"""The never-allocating host step (mv_step_host_static) against the ordinary host step.

Collected last on purpose: if it fails, a run that stops at the first failure has already run
every other test.  It must also pass when this file is run on its own in a fresh process.

Who needs that entry point: code that may not allocate GPU memory while it runs (a trainer
whose own pool already owns all free device memory, a latency-bound loop that cannot take the
implicit synchronisation of an allocation, a process that forbids allocation after start-up).
The frames are staged in a fixed 8 MiB device array inside the library instead of in buffers
allocated on first use, so its results must be the same bytes as mv_step_host's.
"""
import pytest
import torch

from paper_2107_08170_b200 import scenes

pytestmark = pytest.mark.gpu


def _setup(cfg):
    from paper_2107_08170_b200 import binding as B
    from gpu_util import upload_scene
    sc = scenes.make_scene(cfg)
    batch = B.Batch(B.desc_from_config(cfg))
    upload_scene(batch, sc)
    return B, sc, batch


def test_static_step_matches_host_step_on_two_calls_in_a_row():
    cfg = scenes.config("rooms_boxes", num_envs=12)            # 48 observations: fits the fixed array
    B, sc, batch = _setup(cfg)
    shape_rgb = (cfg.num_obs, cfg.height, cfg.width, 3)
    shape_d = (cfg.num_obs, cfg.height, cfg.width)
    cams_a = sc["cams"].contiguous().pin_memory()
    cams_b = scenes.walk_cameras(cfg, sc, sc["cams"], 1).contiguous().pin_memory()
    assert not torch.equal(cams_a, cams_b)
    want, got = [], []
    for cams in (cams_a, cams_b):                              # existing entry point
        rgb = torch.empty(shape_rgb, dtype=torch.uint8).pin_memory()
        dep = torch.empty(shape_d, dtype=torch.float32).pin_memory()
        batch.step_host(cams, rgb, dep)
        want.append((rgb.clone(), dep.clone()))
    for cams in (cams_a, cams_b):                              # new entry point, two calls in a row
        rgb = torch.full(shape_rgb, 7, dtype=torch.uint8).pin_memory()
        dep = torch.full(shape_d, -5.0, dtype=torch.float32).pin_memory()
        batch.step_host_static(cams, rgb, dep)
        got.append((rgb.clone(), dep.clone()))
    for (wr, wd), (gr, gd) in zip(want, got):
        assert torch.equal(wr, gr)                             # integer output: bit-exact
        assert torch.equal(wd, gd)                             # same kernel, same inputs: bit-exact
    assert not torch.equal(got[0][0], got[1][0])               # the second call really re-rendered
    assert batch.query_status() == 0
    batch.destroy()


def test_static_step_rejects_batches_beyond_the_fixed_array():
    cfg = scenes.config("rooms", num_envs=80)                  # 160 observations at 128x72 > 8 MiB
    B, sc, batch = _setup(cfg)
    rgb = torch.empty(cfg.num_obs, cfg.height, cfg.width, 3, dtype=torch.uint8)
    dep = torch.empty(cfg.num_obs, cfg.height, cfg.width, dtype=torch.float32)
    with pytest.raises(B.MvError) as ei:
        batch.step_host_static(sc["cams"].contiguous(), rgb, dep)
    assert ei.value.code == -6
    batch.destroy()


def test_static_step_allocates_nothing_on_a_fresh_batch():
    """The property the entry point exists for: on a batch that never went through mv_step_host (so no
    frame buffers exist yet), two static steps leave the amount of free device memory exactly as it was,
    and the frames equal those of the device-pointer path."""
    cfg = scenes.config("rooms_boxes", num_envs=10)            # 40 observations
    B, sc, batch = _setup(cfg)
    d_cams = sc["cams"].cuda().contiguous()
    want_rgb, want_depth = batch.alloc_outputs()
    batch.set_cameras(d_cams)
    batch.render_batch(want_rgb, want_depth)
    want_rgb, want_depth = want_rgb.cpu(), want_depth.cpu()
    cams = sc["cams"].contiguous().pin_memory()
    rgb = torch.empty(want_rgb.shape, dtype=torch.uint8).pin_memory()
    dep = torch.empty(want_depth.shape, dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for _ in range(2):
        rgb.fill_(3); dep.fill_(-1.0)
        batch.step_host_static(cams, rgb, dep)
        assert torch.equal(rgb, want_rgb) and torch.equal(dep, want_depth)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before
    assert batch.query_status() == 0
    batch.destroy()


def test_static_step_limit_is_exactly_the_documented_one():
    """129 observations at 128x72 fit the 8 MiB array, 130 do not."""
    for agents, ok in ((129, True), (130, False)):
        cfg = scenes.config("rooms", num_envs=1, agents=agents)
        B, sc, batch = _setup(cfg)
        cams = sc["cams"].contiguous()
        rgb = torch.empty(cfg.num_obs, cfg.height, cfg.width, 3, dtype=torch.uint8)
        dep = torch.empty(cfg.num_obs, cfg.height, cfg.width, dtype=torch.float32)
        if ok:
            batch.step_host_static(cams, rgb, dep)
            assert (dep > 0).any()
        else:
            with pytest.raises(B.MvError) as ei:
                batch.step_host_static(cams, rgb, dep)
            assert ei.value.code == -6
        batch.destroy()
