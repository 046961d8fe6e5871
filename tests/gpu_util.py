"""Run a generated scene through the CUDA library (C ABI via the binding) and fetch frames."""
import numpy as np
import torch

from paper_2107_08170_b200 import binding, scenes


def scene_to_numpy(scene):
    return {k: (v.cpu().numpy() if hasattr(v, "cpu") else v) for k, v in scene.items()}


def upload_scene(batch, scene, env_begin=0):
    dev = torch.device("cuda", batch.desc.device)
    n = scene["grid"].shape[0]
    grid = scene["grid"].to(dev).contiguous()
    pal = scene["palette"].to(dev).contiguous()
    boxes = count = None
    if scene["boxes"].shape[1] > 0:
        boxes = scene["boxes"].to(dev).contiguous()
        count = scene["box_count"].to(dev).contiguous()
    batch.upload_worlds(env_begin, n, grid, boxes, count, pal)


def render_scene(cfg, scene, device=0, return_batch=False):
    """Whole scene through create/upload/set_cameras/render; returns numpy rgb, depth (+ status)."""
    batch = binding.Batch(binding.desc_from_config(cfg, device))
    upload_scene(batch, scene)
    cams = scene["cams"].to(torch.device("cuda", device)).contiguous()
    batch.set_cameras(cams)
    rgb, depth = batch.alloc_outputs()
    batch.render_batch(rgb, depth)
    status = batch.query_status()
    out = rgb.cpu().numpy(), depth.cpu().numpy(), status
    if return_batch:
        return out + (batch,)
    batch.destroy()
    return out
