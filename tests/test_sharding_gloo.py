"""The N > 1 path on CPU: two gloo ranks each own a contiguous env range (k2d.shard_envs) and pass
its offset as env_offset; no data-path collective is needed, and the union of their results equals
one process stepping all envs (level draws on auto-reset depend on the global env index only).
The CPU oracle stands in for the GPU engine here (no GPU in this test)."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2410_23208_b200 import k2d, scenes

N_ENVS, N_STEPS, SEED = 24, 30, 4242


def _levels():
    return scenes.make_levels("S", 8, 77, static_prob=0.1)


def _run(levels, offset, count, actions):
    from oracle import k2d_ref
    sim = k2d_ref.RefSim(levels, count, auto_reset=2, max_episode_steps=7, seed=SEED, env_offset=offset)
    sim.reset((np.arange(count) + offset) % levels["pos"].shape[0])
    r, d = sim.step(actions[:, offset:offset + count])
    return sim.pos.copy(), sim.level_id.copy(), r, d


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    levels = _levels()
    actions = scenes.make_actions(N_STEPS, N_ENVS, 2, 5)
    offset, count = k2d.shard_envs(N_ENVS, rank, world)
    pos, lvl, r, d = _run(levels, offset, count, actions)
    # the only cross-rank traffic of the benchmark: a barrier and a max over ranks of the local time
    t = torch.tensor([float(rank + 1)])
    dist.barrier()
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert t.item() == world
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), pos=pos, lvl=lvl, r=r, d=d, offset=offset, count=count)
    dist.destroy_process_group()


def test_two_ranks_reproduce_one_process(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    levels = _levels()
    actions = scenes.make_actions(N_STEPS, N_ENVS, 2, 5)
    pos, lvl, r, d = _run(levels, 0, N_ENVS, actions)
    parts = [np.load(tmp_path / f"rank{k}.npz") for k in range(2)]
    assert parts[0]["count"] + parts[1]["count"] == N_ENVS and parts[1]["offset"] == parts[0]["count"]
    assert np.array_equal(np.concatenate([p["pos"] for p in parts]), pos)
    assert np.array_equal(np.concatenate([p["lvl"] for p in parts]), lvl)
    assert np.array_equal(np.concatenate([p["r"] for p in parts], axis=1), r)
    assert np.array_equal(np.concatenate([p["d"] for p in parts], axis=1), d)
    assert d.sum() > N_ENVS            # resets happened, so the hash-based level draws were exercised


def test_bench_starts_its_own_ranks_with_disjoint_env_ranges():
    # `bench.py --gpus 2` outside torchrun starts two ranks itself; with --plan they do no GPU work, meet over gloo and rank 0
    # prints who would step what: every rank its own RANK / LOCAL_RANK and a range of envs that no other rank has
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--plan", "--envs", "96"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                   # rank 0 alone prints
    plan = json.loads(lines[0])
    assert plan["n_gpus"] == 2 and plan["total_envs"] == 192 and plan["scaling"] == "weak"
    assert [(p["rank"], p["local_rank"]) for p in plan["plan"]] == [(0, 0), (1, 1)]
    ranges = [range(p["env_offset"], p["env_offset"] + p["n_envs"]) for p in plan["plan"]]
    assert set(ranges[0]).isdisjoint(ranges[1]) and len(set(ranges[0]) | set(ranges[1])) == 192
    assert plan["shard_of_total"] == [[0, 96], [96, 96]]
