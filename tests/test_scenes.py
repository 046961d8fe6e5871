"""The seeded input generators: shapes, fill levels, chunk consistency, free cameras and boxes."""
import numpy as np
import torch

from paper_2107_08170_b200 import scenes


def test_fill_levels_and_shapes():
    want = {"tiny": (0.15, 0.25), "rooms": (0.24, 0.26), "rooms_boxes": (0.24, 0.26),
            "headline": (0.14, 0.16), "sweep": (0.24, 0.26)}
    for name, (lo, hi) in want.items():
        cfg = scenes.config(name, num_envs=4 if name == "tiny" else 6)
        sc = scenes.make_scene(cfg)
        gx, gy, gz = cfg.grid
        assert sc["grid"].shape == (cfg.num_envs, gy, gz, gx) and sc["grid"].dtype == torch.uint8
        assert (sc["grid"][:, 0] != 0).all()                      # solid floor layer
        assert lo <= scenes.fill_fraction(sc["grid"]) <= hi, name
        assert int(sc["grid"].max()) < cfg.palette_size
        assert sc["boxes"].shape == (cfg.num_envs, cfg.max_boxes, 8)
        assert sc["cams"].shape == (cfg.num_obs, 6)
        assert int(sc["box_count"].max()) <= cfg.max_boxes


def test_chunks_equal_whole_batch():
    cfg = scenes.config("rooms_boxes", num_envs=8)
    whole = scenes.make_scene(cfg)
    part = scenes.make_scene(cfg, 5, 3)
    for k in ("grid", "palette", "boxes", "box_count"):
        assert torch.equal(whole[k][5:8], part[k]), k
    assert torch.equal(whole["cams"][5 * cfg.agents:], part["cams"])


def test_cameras_stand_in_free_cells_and_boxes_avoid_voxels():
    for name in ("rooms_boxes", "headline"):
        cfg = scenes.config(name, num_envs=5)
        sc = scenes.make_scene(cfg)
        g = sc["grid"].numpy()
        cams = sc["cams"].numpy()
        pos = np.ascontiguousarray(cams[:, :3]).view(np.float32)
        for o in range(cfg.num_obs):
            e = o // cfg.agents
            i, j, k = np.floor(pos[o]).astype(int)
            assert g[e, j, k, i] == 0 and g[e, j - 1, k, i] != 0
        b = sc["boxes"].numpy()
        for e in range(cfg.num_envs):
            n = int(sc["box_count"][e])
            assert n > 0
            for q in range(n):
                lo = b[e, q, :3].view(np.float32); hi = b[e, q, 3:6].view(np.float32)
                assert (lo < hi).all()
                is_body = cfg.body_boxes and q >= n - cfg.agents
                if is_body:
                    continue
                i0, j0, k0 = np.floor(lo).astype(int)
                i1, j1, k1 = np.floor(np.nextafter(hi, -np.inf)).astype(int)
                assert (g[e, j0:j1 + 1, k0:k1 + 1, i0:i1 + 1] == 0).all()
        if cfg.body_boxes:
            assert (cams[:, 5] >= 0).all()


def test_walk_cameras_moves_only_into_free_cells():
    cfg = scenes.config("sweep", num_envs=4)
    sc = scenes.make_scene(cfg)
    g = sc["grid"].numpy()
    cams = sc["cams"]
    for step in range(1, 4):
        cams = scenes.walk_cameras(cfg, sc, cams, step)
        pos = np.ascontiguousarray(cams.numpy()[:, :3]).view(np.float32)
        for o in range(cfg.num_obs):
            i, j, k = np.floor(pos[o]).astype(int)
            assert g[o // cfg.agents, j, k, i] == 0
    assert not torch.equal(cams, sc["cams"])
