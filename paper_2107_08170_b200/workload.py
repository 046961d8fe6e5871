"""Build a whole benchmark workload on one GPU: generate the seeded scenes chunk by chunk on the
device, upload them through the C ABI, and keep CPU copies of a few sampled environments so a
checker can re-render them.  Argument marshalling and input generation only."""
from __future__ import annotations

import torch

from . import binding, scenes


def algorithmic_bytes(cfg) -> int:
    """Bytes one render step must move: every output byte once (3 B colour + 4 B depth per pixel),
    one camera record (64 B) per observation, one material byte per pixel, each environment's
    occupancy at 1 bit per voxel once per step, and its box list (32 B per box)."""
    gx, gy, gz = cfg.grid
    px = cfg.width * cfg.height
    return cfg.num_obs * (7 * px + 64 + px) + cfg.num_envs * (gx * gy * gz // 8 + 32 * cfg.max_boxes)


def build_batch(cfg, device: int = 0, env_offset: int = 0, keep_envs=(), chunk_envs: int = 512,
                max_overlay_rects: int = 0, camera_walk_steps: int = 0):
    """Returns (batch, cams_dev, kept) where kept[e] holds CPU arrays of env e (local index)
    for every e in keep_envs.  env_offset shifts the seeded env ids (one range per rank).
    With camera_walk_steps = K the second element is a list of K+1 camera tensors: the initial cameras
    followed by K seeded updates of the sweep workload (scenes.walk_cameras), pre-computed on the device."""
    dev = torch.device("cuda", device)
    batch = binding.Batch(binding.desc_from_config(cfg, device, max_overlay_rects))
    cams = torch.empty(cfg.num_obs, 6, dtype=torch.int32, device=dev)
    walk = [torch.empty_like(cams) for _ in range(camera_walk_steps)]
    kept = {}
    keep = set(int(e) for e in keep_envs)
    A = cfg.agents
    for e0 in range(0, cfg.num_envs, chunk_envs):
        n = min(chunk_envs, cfg.num_envs - e0)
        sc = scenes.make_scene(cfg, env_offset + e0, n, device=dev)
        boxes = count = None
        if cfg.max_boxes > 0:
            boxes, count = sc["boxes"].contiguous(), sc["box_count"].contiguous()
        batch.upload_worlds(e0, n, sc["grid"].contiguous(), boxes, count, sc["palette"].contiguous())
        cams[e0 * A:(e0 + n) * A] = sc["cams"]
        step_cams = sc["cams"]
        for k in range(camera_walk_steps):
            step_cams = scenes.walk_cameras(cfg, sc, step_cams, k + 1)
            walk[k][e0 * A:(e0 + n) * A] = step_cams
        for e in keep:
            if e0 <= e < e0 + n:
                i = e - e0
                kept[e] = {"grid": sc["grid"][i].cpu().numpy(), "palette": sc["palette"][i].cpu().numpy(),
                           "boxes": sc["boxes"][i].cpu().numpy(), "box_count": int(sc["box_count"][i]),
                           "cams": sc["cams"][i * A:(i + 1) * A].cpu().numpy()}
        torch.cuda.synchronize(dev)
        del sc
    return batch, ([cams] + walk if camera_walk_steps else cams), kept
