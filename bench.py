#!/usr/bin/env python
"""Benchmark of the batched render step (paper Section 3.2, Eq. 2) on the headline workload:
16384 environments x 1 agent, 128x32x128 voxel grid, 16 movable boxes, 128x72 RGB-D.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one pass of the whole per-step path: mv_set_cameras + mv_render_batch over the whole
batch, inputs resident in HBM.  `value` is observations per second over all ranks (device time,
CUDA events, max over ranks); `e2e` is the same metric through mv_step_host with page-locked host
buffers (cameras and boxes copied in, frames copied out, every step).  With --gpus N > 1 the script
starts N ranks itself (one per GPU, through torch.distributed.run) unless it already runs under
such a launcher; every rank renders its own 16384 seeded environments and nothing is exchanged on
the data path (weak scaling).  `--plan` prints which rank renders which environments and touches
no GPU.  `--impl reference` times the CPU oracle on a bounded sample of the same workload.
The sweep workload (`--workload sweep`) precedes every step by its seeded camera update, the
sequences pre-computed on the device.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

WORKLOAD = "headline"
# Profiler evidence that the bench line quotes next to its live timings.  Both figures come from one ncu
# capture of render_kernel on a 2048-environment slice of the headline workload (summary and command in
# profiles/render_kernel_headline_2048env_ncu_full.md); NCU_BUILD names the commit of the library they were
# taken on.  DRAM traffic grows in proportion to the environments, so a full launch is the slice x 8.
NCU_BUILD = "4762628"
NCU_SLICE_ENVS = 2048
NCU_SLICE_DRAM_BYTES = 147.42e6 + 85.17e6   # dram__bytes_read.sum + dram__bytes_write.sum of one launch on the slice
NCU_WARP_INSTRUCTIONS_PER_TILE = 233.9  # smsp__inst_executed.sum / (8x4-pixel tiles) on the slice


def measured_peak():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        try:
            return float(json.loads(p.read_text())["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """SM clock and throttle reasons sampled through NVML (read-only) in a thread while the
    timed region runs; falls back to one-shot nvidia-smi output if NVML is unavailable."""
    HW_SLOWDOWN, HW_THERMAL, SW_THERMAL, SW_POWER = 0x8, 0x40, 0x20, 0x4

    def __init__(self, torch_index: int):
        self.idx, self.samples, self.reasons, self.max_mhz = torch_index, [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(torch_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if isinstance(uuid, str) else uuid)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as e:          # noqa: BLE001
            self._err = repr(e)
            self._h = None

    def sample_now(self):
        """One sample from the calling thread (the timed loop calls it while its launches are still
        running on the GPU, so a short timed region has a sample under load even if the thread got no turn)."""
        if self._h is None:
            return
        nv = self._nv
        try:
            self.samples.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
            r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
            for bit, name in ((self.HW_SLOWDOWN, "hw_slowdown"), (self.HW_THERMAL, "hw_thermal_slowdown"),
                              (self.SW_THERMAL, "sw_thermal_slowdown"), (self.SW_POWER, "sw_power_cap")):
                if r & bit:
                    self.reasons.add(name)
        except Exception:               # noqa: BLE001
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample_now()
            self._stop.wait(0.002)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        if self.samples:
            return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                    "samples": len(self.samples), "reasons": sorted(self.reasons)}
        try:
            out = subprocess.run(["nvidia-smi", "--query-gpu=clocks.sm,clocks.max.sm", "--format=csv,noheader,nounits",
                                  "-i", str(self.idx)], capture_output=True, text=True, timeout=10).stdout
            a, b = [float(x) for x in out.strip().split(",")[:2]]
            return {"sm_mhz": a, "sm_max_mhz": b, "samples": 1, "reasons": ["sampled after the timed region (NVML unavailable)"]}
        except Exception:               # noqa: BLE001
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["clock sampling unavailable"]}


def cpu_affinity() -> str:
    """The cores this process may run on, as a compact range list."""
    cores = sorted(os.sched_getaffinity(0))
    out, i = [], 0
    while i < len(cores):
        j = i
        while j + 1 < len(cores) and cores[j + 1] == cores[j] + 1:
            j += 1
        out.append(str(cores[i]) if i == j else f"{cores[i]}-{cores[j]}")
        i = j + 1
    return ",".join(out)


def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


CPU_SAMPLE_OBS = 32      # observations the oracle renders for the cpu_baseline figure (about 10 s on 16 cores)


def cpu_oracle_rate(cfg, kept, max_seconds=25.0, max_obs=CPU_SAMPLE_OBS):
    """Observations per second of the oracle, as it stands, on this host's cores."""
    from oracle import mv_oracle
    mv_oracle.build()
    desc = mv_oracle.desc_from_config(cfg)
    done, t0 = 0, time.perf_counter()
    for e in sorted(kept)[:max_obs]:
        k = kept[e]
        boxes = k["boxes"] if cfg.max_boxes > 0 else None
        mv_oracle.render_obs(desc, k["grid"], boxes, k["box_count"], k["palette"], k["cams"][0])
        done += 1
        if time.perf_counter() - t0 > max_seconds:
            break
    dt = time.perf_counter() - t0
    return done / dt, done, dt, mv_oracle.threads_used()


def time_extras(batch, cfg, cams, rgb, depth, dev):
    """CUDA-event medians (ms) of the entry points beside the render step, on the benchmark's batch."""
    import torch
    from paper_2107_08170_b200 import vecenv

    def med(fn, n=15):
        for _ in range(3):
            fn()
        torch.cuda.synchronize(dev)
        ts = []
        for _ in range(n):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record(); torch.cuda.synchronize(dev)
            ts.append(e0.elapsed_time(e1))
        return statistics.median(ts)

    out = {"render_ms": med(lambda: batch.render_batch(rgb, depth))}
    E = cfg.num_envs
    rects = vecenv.time_bar_rects(torch.full((E,), 60), torch.full((E,), 100), cfg.width, cfg.agents).to(dev)
    count = torch.ones(cfg.num_obs, dtype=torch.int32, device=dev)
    out["set_overlays_ms"] = med(lambda: batch.set_overlays(rects, count))
    out["render_with_time_bar_ms"] = med(lambda: batch.render_batch(rgb, depth))
    batch.set_overlays(None, None)
    moved = cams.clone()
    yf = moved[:, 1].contiguous().view(torch.float32)
    moved[:, 1] = (yf.floor() + 0.75).view(torch.int32)             # feet on the surface
    moves = ((torch.rand(cfg.num_obs, 4, device=dev) - 0.5) * torch.tensor([0.4, 0.2, 0.3, 0.1], device=dev)).contiguous()
    out["move_agents_ms"] = med(lambda: batch.move_agents(moved, moves))
    out["set_cameras_ms"] = med(lambda: batch.set_cameras(cams))
    n = min(E, 8192)
    out["merge_voxels_ms_per_env"] = med(lambda: batch.merge_voxels(0, n, 2048), 3) / n
    out["merged_boxes_per_env"] = float(batch.merge_voxels(0, n, 2048)[1].float().mean())
    batch.debug_occupancy_in_global(True)
    out["render_occupancy_in_global_ms"] = med(lambda: batch.render_batch(rgb, depth))
    batch.debug_occupancy_in_global(False)
    # the vectorised step() wrapper at this size: move + collide, auto-reset of the ~1 % of environments whose
    # 100-step episode ends (new worlds generated and uploaded), time-left bar, render; wall clock over 20 steps
    env = vecenv.VecRenderEnv(cfg, 100, device=dev.index, phase=torch.arange(E) % 100)
    env.reset()
    for _ in range(2):
        env.step(moves)
    torch.cuda.synchronize(dev)
    t0 = time.perf_counter()
    n_steps, n_reset = 20, 0
    for _ in range(n_steps):
        _, _, done = env.step(moves)
        n_reset += int(done.sum())
    torch.cuda.synchronize(dev)
    dt = time.perf_counter() - t0
    out["vecenv_steps_per_s"] = n_steps / dt
    out["vecenv_obs_per_s"] = n_steps * cfg.num_obs / dt
    out["vecenv_envs_reset_per_step"] = n_reset / n_steps
    env.close()
    return out


def run_reference(args, rank):
    """The oracle timed on a bounded sample: each step renders `sample` observations."""
    if rank != 0:
        return
    import torch  # noqa: F401  (scenes use torch CPU tensors)
    from paper_2107_08170_b200 import scenes
    from oracle import mv_oracle
    mv_oracle.build()
    cfg = scenes.config(WORKLOAD)
    sample = 2
    n_env = sample * (args.steps + args.warmup)
    sc = scenes.make_scene(cfg, 0, n_env)
    desc = mv_oracle.desc_from_config(cfg)
    g, b, c, p, cams = (sc[k].numpy() for k in ("grid", "boxes", "box_count", "palette", "cams"))

    def step(i):
        for e in range(i * sample, (i + 1) * sample):
            mv_oracle.render_obs(desc, g[e], b[e], c[e], p[e], cams[e])

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.warmup, args.warmup + args.steps):
        step(i)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    cores = mv_oracle.threads_used()
    what = f"{sample} observations of the {WORKLOAD} workload per step, all {cfg.width}x{cfg.height} pixels"
    print(json.dumps({
        "impl": "reference", "metric": "observations/sec", "value": value, "unit": "obs/s",
        "grays_per_sec": value * cfg.width * cfg.height / 1e9, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg, args.gpus),
        "cpu_baseline": {"value": value, "unit": "obs/s", "cores": cores, "kind": "oracle", "cpu_model": cpu_model(),
                         "affinity": cpu_affinity(), "sample": what},
        "e2e": {"value": value, "unit": "obs/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def run_plan(args, rank, world):
    """Rank -> seeded environment range, gathered over the same launcher as the benchmark but on the
    CPU backend: every rank reports its own range, rank 0 prints them.  No CUDA call is made."""
    from paper_2107_08170_b200 import scenes, shard
    over = {"num_envs": args.envs} if args.envs is not None else {}
    cfg = scenes.config(WORKLOAD, **over)
    begin = shard.env_offset(rank, cfg.num_envs)
    mine = {"rank": rank, "env_begin": begin, "env_end": begin + cfg.num_envs, "observations": cfg.num_obs}
    plan = [mine]
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("gloo")
        plan = [None] * world
        dist.all_gather_object(plan, mine)
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps({"plan": plan, "n_gpus": world, "workload": WORKLOAD, "scaling": "weak",
                          "collectives_on_data_path": 0}))


def workload_config(cfg, n_gpus):
    gx, gy, gz = cfg.grid
    from paper_2107_08170_b200 import workload as wl
    big = wl.algorithmic_bytes(cfg) >= (512 << 20)
    return {"workload": f"{WORKLOAD}: {cfg.num_envs} envs x {cfg.agents} agent per GPU, grid {gx}x{gy}x{gz} uint8 "
                        f"({cfg.world}), {cfg.movable_boxes} movable boxes/env, {cfg.width}x{cfg.height} RGB u8 + depth f32",
            "envs_per_gpu": cfg.num_envs, "agents": cfg.agents, "grid": [gx, gy, gz], "boxes_per_env": cfg.max_boxes,
            "width": cfg.width, "height": cfg.height, "parallelism": f"env-sharded x{n_gpus}, no collective",
            "l2_policy": (f"inputs larger than L2 ({wl.algorithmic_bytes(cfg) / 1e9:.2f} GB of env blocks and frames per step "
                          "vs 126 MB L2)") if big else "L2 flushed (256 MB fill) between timed steps"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--envs", type=int, default=None, help="override envs per GPU (profiling small cases)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--workload", default="headline", choices=["tiny", "rooms", "rooms_boxes", "headline", "sweep"],
                    help="workload shape to time (the headline one is the benchmark; the others are for reference)")
    ap.add_argument("--width", type=int, default=None)
    ap.add_argument("--height", type=int, default=None)
    ap.add_argument("--extras", action="store_true",
                    help="also time the overlay, agent-motion and voxel-merge entry points (adds an \"extras\" object)")
    ap.add_argument("--plan", action="store_true",
                    help="print which rank renders which seeded environments and exit (no GPU is touched)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" and args.envs is None else args.warmup

    # --gpus N on its own starts the N ranks (one per GPU); under a launcher the ranks are already there
    if args.gpus > 1 and "RANK" not in os.environ and not (args.impl == "reference"):
        cmd = [sys.executable, "-m", "torch.distributed.run", "--standalone", "--local-addr", "127.0.0.1", "--nnodes=1",
               f"--nproc-per-node={args.gpus}", str(Path(__file__).resolve()), *sys.argv[1:]]
        raise SystemExit(subprocess.call(cmd))

    global WORKLOAD
    WORKLOAD = args.workload
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.plan:
        run_plan(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2107_08170_b200 import binding, scenes, shard, workload

    binding.lib()                                    # fails loudly if the CUDA library is missing
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    # under torchrun (RANK set) the process group is used even for one rank, so the single-GPU launch
    # exercises the same barrier and max-over-ranks code as the multi-GPU one
    use_dist = world > 1 or ("RANK" in os.environ and "MASTER_ADDR" in os.environ)
    if use_dist:
        dist.init_process_group("nccl", device_id=dev)

    over = {}
    if args.envs is not None:
        over["num_envs"] = args.envs
    if args.width is not None:
        over["width"], over["height"] = args.width, args.height or args.width * 9 // 16
    cfg = scenes.config(WORKLOAD, **over)
    # workloads whose per-step bytes do not dwarf the 126 MB L2 get an L2 flush between timed steps
    step_bytes = workload.algorithmic_bytes(cfg)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if step_bytes < (512 << 20) else None
    keep = list(range(0, cfg.num_envs, max(cfg.num_envs // CPU_SAMPLE_OBS, 1)))[:CPU_SAMPLE_OBS] if rank == 0 and not args.no_cpu else []
    # the sweep workload moves every camera before every step (seeded walk, pre-computed here)
    walk_steps = args.steps + args.warmup if WORKLOAD == "sweep" else 0
    batch, cams, kept = workload.build_batch(cfg, local, env_offset=shard.env_offset(rank, cfg.num_envs), keep_envs=keep,
                                             max_overlay_rects=1 if args.extras else 0, camera_walk_steps=walk_steps)
    cam_seq = cams[1:] if walk_steps else None
    if walk_steps:
        cams = cams[0]
    rgb, depth = batch.alloc_outputs()
    stream = torch.cuda.current_stream()

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def step(i):
        batch.set_cameras(cam_seq[i] if cam_seq is not None else cams)
        batch.render_batch(rgb, depth)

    for i in range(args.warmup):
        step(i)
    barrier()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    sampler.start()
    launches0 = batch.launch_count()
    barrier()
    t_begin.record(stream)
    for i, (e0, e1, e2) in enumerate(ev):
        if flush is not None:
            flush.fill_(1)
        e0.record(stream)
        batch.set_cameras(cam_seq[args.warmup + i] if cam_seq is not None else cams)
        e1.record(stream)
        batch.render_batch(rgb, depth)
        e2.record(stream)
    t_end.record(stream)
    sampler.sample_now()                       # the launches above are still running
    barrier()
    total_ms = t_begin.elapsed_time(t_end)
    if flush is not None:                      # the flushes sit between the steps: sum the steps alone
        total_ms = sum(e0.elapsed_time(e2) for e0, _, e2 in ev)
    launches = batch.launch_count() - launches0
    clocks = sampler.stop()
    render_ms = [e1.elapsed_time(e2) for _, e1, e2 in ev]
    status = batch.query_status()
    assert status == 0, f"device status word {status}"

    # end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        h_cams = cams.cpu().pin_memory()
        h_rgb = torch.empty(rgb.shape, dtype=torch.uint8).pin_memory()
        h_depth = torch.empty(depth.shape, dtype=torch.float32).pin_memory()
        sc_boxes = h_count = None
        if cfg.max_boxes > 0:
            # the boxes move every step in the simulator, so the end-to-end step re-sends them
            sc_boxes = torch.zeros(cfg.num_envs, cfg.max_boxes, 8, dtype=torch.int32)
            h_count = torch.zeros(cfg.num_envs, dtype=torch.int32)
            for e0 in range(0, cfg.num_envs, 512):
                n = min(512, cfg.num_envs - e0)
                sc = scenes.make_scene(cfg, rank * cfg.num_envs + e0, n, device=dev)
                sc_boxes[e0:e0 + n] = sc["boxes"].cpu(); h_count[e0:e0 + n] = sc["box_count"].cpu()
            sc_boxes, h_count = sc_boxes.pin_memory(), h_count.pin_memory()
        n_e2e = max(3, min(args.steps, 10))
        for _ in range(2):
            batch.step_host(h_cams, h_rgb, h_depth, boxes=sc_boxes, box_count=h_count)
        barrier()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        b0.record(stream)
        for _ in range(n_e2e):
            batch.step_host(h_cams, h_rgb, h_depth, boxes=sc_boxes, box_count=h_count)
        b1.record(stream)
        barrier()
        e2e_ms = b0.elapsed_time(b1) / n_e2e
        h2d = h_cams.numel() * 4 + (sc_boxes.numel() * 4 + h_count.numel() * 4 if sc_boxes is not None else 0)
        d2h = h_rgb.numel() + h_depth.numel() * 4
        e2e = (e2e_ms, h2d, d2h, n_e2e)

    # max over ranks
    mx = shard.max_over_ranks([total_ms, e2e[0] if e2e else 0.0], dev)
    total_ms = mx[0]
    if e2e:
        e2e = (mx[1],) + e2e[1:]

    if rank == 0:
        obs_total = cfg.num_obs * world
        ms_per_step = total_ms / args.steps
        value = obs_total / (ms_per_step * 1e-3)
        px = cfg.width * cfg.height
        peak, peak_kind = measured_peak()
        alg = workload.algorithmic_bytes(cfg)
        k_ms = statistics.mean(render_ms)
        achieved = alg / (k_ms * 1e-3) / 1e9
        traffic = None
        if WORKLOAD == "headline" and NCU_SLICE_DRAM_BYTES is not None:       # scaled from the profiled slice
            traffic = NCU_SLICE_DRAM_BYTES * cfg.num_envs / NCU_SLICE_ENVS
        out = {
            "metric": "observations/sec", "value": value, "unit": "obs/s",
            "grays_per_sec": value * px / 1e9,
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": workload_config(cfg, world),
            "clocks": clocks, "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "kernel": "render_kernel", "achieved": achieved, "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                         "traffic": traffic, "traffic_build": NCU_BUILD,
                         "traffic_how": f"ncu dram bytes of one launch on a {NCU_SLICE_ENVS}-env slice, scaled by envs",
                         "algorithmic_bytes_per_launch": alg,
                         "kernel_ms_mean": k_ms, "kernel_ms_min": min(render_ms), "kernel_ms_median": statistics.median(render_ms)},
            # the resource that actually binds: warp-instruction issue slots (one per scheduler per cycle)
            "issue_roofline": {"bound": "alu", "unit": "warp-instructions/s", "counter_build": NCU_BUILD,
                               "warp_instructions_per_tile": NCU_WARP_INSTRUCTIONS_PER_TILE,
                               "achieved": (NCU_WARP_INSTRUCTIONS_PER_TILE or 0) * (cfg.num_obs * px / 32) / (k_ms * 1e-3),
                               "peak": 148 * 4 * (clocks.get("sm_mhz") or 1965.0) * 1e6,
                               "peak_kind": "148 SMs x 4 schedulers x sampled SM clock"},
            "paper_context": "paper: 1.1e6 obs/s whole simulator on one 8x RTX 2080 Ti node (128x72 RGB, no depth)",
        }
        out["issue_roofline"]["frac"] = out["issue_roofline"]["achieved"] / out["issue_roofline"]["peak"]
        if WORKLOAD != "headline" or NCU_WARP_INSTRUCTIONS_PER_TILE is None:   # the figure belongs to the headline workload
            out.pop("issue_roofline")
        if e2e:
            out["e2e"] = {"value": obs_total / (e2e[0] * 1e-3), "unit": "obs/s", "ms_per_step": e2e[0],
                          "h2d_bytes_per_step": e2e[1], "d2h_bytes_per_step": e2e[2], "steps": e2e[3]}
        if not args.no_cpu and kept:
            rate, n, secs, cores = cpu_oracle_rate(cfg, kept)
            out["cpu_baseline"] = {"value": rate, "unit": "obs/s", "cores": cores, "kind": "oracle", "cpu_model": cpu_model(),
                                   "affinity": cpu_affinity(),
                                   "sample": f"{n} observations (every {max(cfg.num_envs // CPU_SAMPLE_OBS, 1)}th env) of this workload, all pixels, {secs:.1f} s"}
        print(json.dumps(out))
    if args.extras and rank == 0:
        print(json.dumps({"extras": time_extras(batch, cfg, cams, rgb, depth, dev)}), file=sys.stderr)
    batch.destroy()
    if use_dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
