"""Comparison of rendered frames with the oracle's, by the acceptance rule of the benchmark
definition: at least 99.95 % of RGB pixels bit-identical; every other pixel differs by at
most 1 LSB or lies on a silhouette edge; depth within 1e-4 relative on every non-edge pixel.
The 0.05 % budget covers every mismatching pixel, whether its colour or only its depth is off,
excused or not.

A mismatching pixel counts as a silhouette-edge pixel when (i) one of its 8 neighbours in
the oracle's id buffer shows a different surface (hit/miss, class, face or material), or
(ii) the oracle, re-run with the sample point moved by 1e-3 pixel in one of 8 directions,
reproduces the other side's colour and depth.
"""
from __future__ import annotations

import numpy as np

RGB_IDENTICAL_MIN = 0.9995
DEPTH_RTOL = 1e-4
DEPTH_FLOOR = 1e-3


def depth_close(g, o):
    return np.abs(g.astype(np.float64) - o.astype(np.float64)) <= DEPTH_RTOL * np.maximum(np.abs(o), DEPTH_FLOOR)


def surface_key(ids, grid, boxes, palette_size):
    """(class, face, material) folded into one integer per pixel; -1 for a miss."""
    cls, idx, face = ids[..., 0], ids[..., 1], ids[..., 2]
    mat = np.zeros_like(cls)
    vox = cls == 0
    mat[vox] = np.minimum(grid.reshape(-1)[idx[vox]], palette_size - 1)
    bx = cls == 1
    if bx.any():
        mat[bx] = np.minimum(boxes[idx[bx], 6].astype(np.int64) & 0xFFFFFFFF, palette_size - 1)
    key = (cls.astype(np.int64) * 8 + face) * 1024 + mat
    key[cls < 0] = -1
    return key


def neighbour_differs(key):
    H, W = key.shape
    pad = np.pad(key, 1, mode="edge")
    out = np.zeros((H, W), bool)
    for dy in (0, 1, 2):
        for dx in (0, 1, 2):
            if dy == 1 and dx == 1:
                continue
            out |= pad[dy:dy + H, dx:dx + W] != key
    return out


def compare_obs(oracle, desc, grid, boxes, box_count, palette, cam_row, g_rgb, g_depth, o_rgb, o_depth, o_ids):
    """Returns dict(pixels, rgb_mismatch, unexcused, worst_depth_rel)."""
    rgb_bad = (g_rgb != o_rgb).any(axis=-1)
    dep_bad = ~depth_close(g_depth, o_depth)
    bad = rgb_bad | dep_bad
    stats = {"pixels": int(bad.size), "rgb_mismatch": int(rgb_bad.sum()), "unexcused": 0,
             "depth_mismatch": int(dep_bad.sum()), "mismatch": int(bad.sum()), "edge_excused": 0, "lsb_only": 0,
             "details": []}
    if not bad.any():
        return stats
    key = surface_key(o_ids, grid, boxes if boxes is not None else np.zeros((0, 8), np.int32), desc.palette_size)
    edge = neighbour_differs(key)
    ys, xs = np.nonzero(bad)
    for py, px in zip(ys, xs):
        lsb = (np.abs(g_rgb[py, px].astype(int) - o_rgb[py, px].astype(int)).max() <= 1) and not dep_bad[py, px]
        if lsb:
            stats["lsb_only"] += 1
            continue
        if edge[py, px]:
            stats["edge_excused"] += 1
            continue
        offs = np.array([[dx, dy] for dx in (-1e-3, 0, 1e-3) for dy in (-1e-3, 0, 1e-3) if dx or dy])
        pxy = np.tile(np.array([[px, py]], np.int32), (8, 1))
        r, d, _ = oracle.render_pixels(desc, grid, boxes, box_count, palette, cam_row, pxy, offs)
        ok = ((r == g_rgb[py, px]).all(axis=1) & depth_close(np.full(8, g_depth[py, px], np.float32), d)).any()
        if ok:
            stats["edge_excused"] += 1
        else:
            stats["unexcused"] += 1
            if len(stats["details"]) < 10:
                stats["details"].append((int(py), int(px), g_rgb[py, px].tolist(), o_rgb[py, px].tolist(),
                                         float(g_depth[py, px]), float(o_depth[py, px]), o_ids[py, px].tolist()))
    return stats


def compare_scene(oracle, cfg, scene_np, obs_indices, g_rgb, g_depth):
    """scene_np: numpy arrays of a generated scene whose env 0 is scene-local; obs_indices
    index its observations; g_rgb/g_depth are the GPU frames of exactly those observations."""
    desc = oracle.desc_from_config(cfg)
    total = {"pixels": 0, "rgb_mismatch": 0, "unexcused": 0, "depth_mismatch": 0, "mismatch": 0, "edge_excused": 0,
             "lsb_only": 0, "details": []}
    A = cfg.agents
    for n, o in enumerate(obs_indices):
        e = o // A
        boxes = scene_np["boxes"][e] if scene_np["boxes"].shape[1] > 0 else None
        o_rgb, o_depth, o_ids = oracle.render_obs(desc, scene_np["grid"][e], boxes, scene_np["box_count"][e],
                                                  scene_np["palette"][e], scene_np["cams"][o])
        st = compare_obs(oracle, desc, scene_np["grid"][e], boxes, int(scene_np["box_count"][e]),
                         scene_np["palette"][e], scene_np["cams"][o], g_rgb[n], g_depth[n], o_rgb, o_depth, o_ids)
        for k in total:
            total[k] = total[k] + st[k] if k != "details" else total[k] + [(o,) + d for d in st[k]]
    return total


def assert_parity(stats, where=""):
    """No unexcused pixel, and the pixels whose colour OR depth mismatches (excused or not) within the budget."""
    frac_identical = 1.0 - stats["mismatch"] / max(stats["pixels"], 1)
    assert stats["unexcused"] == 0, (where, stats)
    assert frac_identical >= RGB_IDENTICAL_MIN, (where, frac_identical, stats)
