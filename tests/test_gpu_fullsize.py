"""Parity at the full workload sizes, in the launch configuration bench.py times: the whole batch is
built on the GPU through the C ABI, rendered in one launch, and sampled observations are compared
with the oracle pixel by pixel; properties that hold at any size are checked on the whole output."""
import numpy as np
import pytest
import torch

from paper_2107_08170_b200 import scenes
import parity

pytestmark = pytest.mark.gpu


def _run(oracle, name, sample_envs, **over):
    from paper_2107_08170_b200 import workload
    cfg = scenes.config(name, **over)
    keep = list(np.linspace(0, cfg.num_envs - 1, sample_envs).astype(int))
    batch, cams, kept = workload.build_batch(cfg, 0, keep_envs=keep)
    rgb, depth = batch.alloc_outputs()
    batch.set_cameras(cams)
    batch.render_batch(rgb, depth)
    assert batch.query_status() == 0
    A = cfg.agents
    total = None
    for e in keep:
        k = kept[e]
        sc = {"grid": k["grid"][None], "palette": k["palette"][None], "boxes": k["boxes"][None],
              "box_count": np.array([k["box_count"]]), "cams": k["cams"]}
        g_rgb = rgb[e * A:(e + 1) * A].cpu().numpy()
        g_depth = depth[e * A:(e + 1) * A].cpu().numpy()
        st = parity.compare_scene(oracle, cfg, sc, range(A), g_rgb, g_depth)
        total = st if total is None else {q: total[q] + st[q] for q in st}
    parity.assert_parity(total, name)
    # whole-output properties: determinism; depth 0 (= miss_depth) without the sky colour happens only
    # for the rare eye inside a box or solid
    rgb2, depth2 = batch.alloc_outputs()
    batch.render_batch(rgb2, depth2)
    assert torch.equal(rgb, rgb2) and torch.equal(depth, depth2)
    sky = torch.tensor(cfg.sky_rgb, dtype=torch.uint8, device=rgb.device)
    miss = depth == cfg.miss_depth
    assert float((miss & ~(rgb == sky).all(dim=-1)).float().mean()) < 2e-2
    assert bool((depth >= 0).all()) and bool(torch.isfinite(depth).all())
    frac_hit = 1.0 - float(miss.float().mean())
    batch.destroy()
    return total, frac_hit


def test_headline_full_size(oracle):
    st, frac_hit = _run(oracle, "headline", 8)
    assert st["pixels"] == 8 * 128 * 72 and frac_hit > 0.6


def test_rooms_full_size(oracle):
    st, frac_hit = _run(oracle, "rooms", 6)
    assert frac_hit > 0.9


def test_rooms_boxes_full_size(oracle):
    st, frac_hit = _run(oracle, "rooms_boxes", 3)
    assert frac_hit > 0.9


@pytest.mark.parametrize("W,H", [(64, 36), (128, 72), (256, 144)])
def test_sweep_full_size(oracle, W, H):
    st, frac_hit = _run(oracle, "sweep", 2 if W > 128 else 3, width=W, height=H)
    assert frac_hit > 0.9
