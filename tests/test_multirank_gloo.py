"""World-size-2 checks of the multi-GPU plumbing on CPU (gloo): disjoint env ranges whose union
is the single-process batch, and the max-over-ranks reduction used for timing."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2107_08170_b200 import scenes, shard


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, envs_per_rank, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = scenes.config("rooms_boxes", num_envs=envs_per_rank)
        sc = scenes.make_scene(cfg, shard.env_offset(rank, envs_per_rank), envs_per_rank)
        digest = torch.stack([sc["grid"].long().sum(), sc["boxes"].long().sum(), sc["cams"].long().sum()])
        gathered = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(gathered, digest)
        mx = shard.max_over_ranks([1.0 + rank, 10.0 - rank], torch.device("cpu"))
        b, e = shard.split_envs(7, rank, world)
        q.put((rank, [g.tolist() for g in gathered], mx, (b, e)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_envs_without_overlap():
    world, envs = 2, 3
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, envs, q)) for r in range(world)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # the union of the two shards is the single-process batch of 6 envs, shard by shard
    cfg = scenes.config("rooms_boxes", num_envs=world * envs)
    whole = scenes.make_scene(cfg)
    A = cfg.agents
    for r in range(world):
        sl = slice(r * envs, (r + 1) * envs)
        want = [int(whole["grid"][sl].long().sum()), int(whole["boxes"][sl].long().sum()),
                int(whole["cams"][r * envs * A:(r + 1) * envs * A].long().sum())]
        assert out[0][1][r] == want and out[1][1][r] == want
    assert out[0][1][0] != out[0][1][1]
    assert out[0][2] == [2.0, 10.0] and out[1][2] == [2.0, 10.0]          # max over ranks
    assert out[0][3] == (0, 4) and out[1][3] == (4, 7)                    # strong-scaling split


def test_split_envs_covers_everything():
    for total in (1, 7, 16384):
        for world in (1, 2, 3, 8):
            ranges = [shard.split_envs(total, r, world) for r in range(world)]
            assert ranges[0][0] == 0 and ranges[-1][1] == total
            assert all(ranges[i][1] == ranges[i + 1][0] for i in range(world - 1))


def test_bench_starts_its_own_ranks_and_plans_disjoint_env_ranges():
    """`bench.py --gpus 2 --plan` launches two ranks by itself (no outer launcher), touches no GPU, and the
    two ranks take disjoint, adjacent ranges of seeded environments: scale-out is independent instances."""
    import json
    import subprocess
    import sys
    from pathlib import Path
    root = Path(__file__).resolve().parent.parent
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    env["CUDA_VISIBLE_DEVICES"] = ""
    out = subprocess.run([sys.executable, str(root / "bench.py"), "--gpus", "2", "--plan", "--envs", "96"],
                         capture_output=True, text=True, timeout=300, env=env, cwd=str(root))
    assert out.returncode == 0, out.stderr[-2000:]
    line = [l for l in out.stdout.splitlines() if l.startswith("{")][-1]
    plan = json.loads(line)
    assert plan["n_gpus"] == 2 and plan["collectives_on_data_path"] == 0
    r0, r1 = sorted(plan["plan"], key=lambda r: r["rank"])
    assert (r0["env_begin"], r0["env_end"]) == (0, 96) and (r1["env_begin"], r1["env_end"]) == (96, 192)
