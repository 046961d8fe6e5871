"""The vectorised step() wrapper: bookkeeping on CPU, whole loop on the GPU against the oracle."""
import numpy as np
import pytest
import torch

from paper_2107_08170_b200 import scenes, vecenv


def test_time_bar_rects_layout():
    rec = vecenv.time_bar_rects([10, 5, 0], [10, 10, 4], 128, 2)
    assert rec.shape == (6, 1, 4) and rec.dtype == torch.int32
    raw = rec.numpy().view(np.int16).reshape(6, 8)
    assert raw[:, 0].tolist() == [0] * 6 and raw[:, 1].tolist() == [0] * 6          # x0, y0
    assert raw[:, 2].tolist() == [128, 128, 64, 64, 0, 0]                             # x1 = W * left / len
    assert (raw[:, 3] == vecenv.BAR_ROWS).all()                                       # y1
    assert (rec.numpy().view(np.uint8).reshape(6, 16)[:, 8:11] == np.array(vecenv.BAR_RGB, np.uint8)).all()


@pytest.mark.gpu
def test_step_loop_with_auto_reset_matches_oracle(oracle):
    import parity
    from gpu_util import scene_to_numpy
    cfg = scenes.config("rooms_boxes", num_envs=4)
    lens = [3, 4, 5, 50]
    env = vecenv.VecRenderEnv(cfg, lens)
    env.reset()
    A, E = cfg.agents, cfg.num_envs
    # CPU mirror of the state
    state = [scene_to_numpy(scenes.make_scene(cfg, e, 1)) for e in range(E)]
    t = np.zeros(E, int); ep = np.zeros(E, int)
    rng = np.random.default_rng(3)
    dones = []
    for step in range(7):
        moves = np.stack([rng.uniform(-0.4, 0.4, cfg.num_obs), rng.uniform(-0.2, 0.2, cfg.num_obs),
                          rng.normal(0, 0.3, cfg.num_obs), rng.normal(0, 0.05, cfg.num_obs)], 1).astype(np.float32)
        rgb, depth, done = env.step(torch.from_numpy(moves).cuda())
        dones.append(done.tolist())
        for e in range(E):
            s = state[e]
            for a in range(A):
                f = s["cams"][a, :5].view(np.float32)
                new, _ = oracle.move_agent(s["grid"][0], f, moves[e * A + a], (0.25, 0.75, 0.25), 1.0)
                s["cams"][a, :5] = new.view(np.int32)
                sb = s["cams"][a, 5]
                s["boxes"][0, sb, :3] = (new[:3] - np.float32([0.25, 0.75, 0.25])).view(np.int32)
                s["boxes"][0, sb, 3:6] = (new[:3] + np.float32([0.25, 0.25, 0.25])).view(np.int32)
            t[e] += 1
            if t[e] >= lens[e]:
                ep[e] += 1; t[e] = 0
                state[e] = scene_to_numpy(scenes.make_scene(cfg, e + ep[e] * E, 1))
    assert dones[2] == [True, False, False, False] and dones[3] == [False, True, False, False]
    assert dones[5] == [True, False, False, False] and not any(d[3] for d in dones)
    # final frames: 3D view per the oracle, then the time bar on top
    g_rgb, g_depth = rgb.cpu().numpy(), depth.cpu().numpy()
    bars = vecenv.time_bar_rects(np.array(lens) - t, lens, cfg.width, A).numpy()
    desc = oracle.desc_from_config(cfg)
    total = None
    for e in range(E):
        s = state[e]
        for a in range(A):
            o = e * A + a
            o_rgb, o_depth, o_ids = oracle.render_obs(desc, s["grid"][0], s["boxes"][0], s["box_count"][0],
                                                      s["palette"][0], s["cams"][a])
            rect = bars[o].view(oracle.RECT_DTYPE).reshape(-1)
            o_rgb = oracle.overlay(np.ascontiguousarray(o_rgb), rect, 1)
            # the bar hides the 3D pixels under it on both sides, so the parity rule applies as is
            st = parity.compare_obs(oracle, desc, s["grid"][0], s["boxes"][0], int(s["box_count"][0]),
                                    s["palette"][0], s["cams"][a], g_rgb[o], g_depth[o], o_rgb, o_depth, o_ids)
            total = st if total is None else {k: total[k] + st[k] for k in st}
    parity.assert_parity(total, "vecenv")
    bar_len = int(bars[0].view(np.int16).reshape(-1)[2])
    assert (g_rgb[0, :2, :bar_len] == np.array(vecenv.BAR_RGB, np.uint8)).all()
    env.close()
