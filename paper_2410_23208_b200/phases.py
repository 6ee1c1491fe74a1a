"""Where a step's time goes: runs a benchmark workload on the build of the library whose step kernel counts SM cycles
per phase (-DK2D_PHASE_CLOCKS) and prints each phase's share.

    python -m paper_2410_23208_b200.phases [--workload 3] [--envs N] [--launches 4] [--fused 32]

The counting build is slower than the library proper (two clock reads and an atomic add per phase boundary), so the shares
are what to read, not the rate.
"""
from __future__ import annotations

import argparse
import json

from . import k2d, scenes


def phase_shares(workload: int = 3, n_envs: int = 0, launches: int = 4, fused: int = 32, lanes: int = 0) -> dict:
    import torch
    w = scenes.WORKLOADS[workload]
    n_envs = n_envs or w["n_envs"]
    seed = scenes.workload_seed(workload)
    levels = scenes.make_levels(w["size"], w["n_levels"], seed, static_prob=w["static_prob"])
    env = k2d.Env(levels, n_envs, phase_clocks=True, auto_reset=w["auto_reset"], max_episode_steps=w["max_episode_steps"], seed=seed,
                  max_fused_steps=fused, lanes_per_scene=lanes)
    actions = torch.from_numpy(scenes.make_actions(fused, n_envs, env.n_actions, seed)).cuda()
    env.step(actions)                       # warm-up launch, not counted
    env.phase_cycles()
    for _ in range(launches):
        env.step(actions)
    cycles = env.phase_cycles()
    total = float(sum(cycles.values())) or 1.0
    env_steps = launches * fused * n_envs
    return {"workload": workload, "size": w["size"], "n_envs": n_envs, "fused_steps": fused, "launches": launches,
            "cycles_per_env_step": total / env_steps,
            "share": {k: v / total for k, v in cycles.items()},
            "cycles_per_env_step_by_phase": {k: v / env_steps for k, v in cycles.items()}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", type=int, default=3, choices=sorted(scenes.WORKLOADS))
    ap.add_argument("--envs", type=int, default=0)
    ap.add_argument("--launches", type=int, default=4)
    ap.add_argument("--fused", type=int, default=32)
    ap.add_argument("--lanes", type=int, default=0)
    ap.add_argument("--json", action="store_true")
    args = ap.parse_args()
    out = phase_shares(args.workload, args.envs, args.launches, args.fused, args.lanes)
    if args.json:
        print(json.dumps(out))
        return
    print(f"workload {out['workload']} ({out['size']} scenes, {out['n_envs']} envs, {out['fused_steps']} steps per launch, {out['launches']} launches): "
          f"{out['cycles_per_env_step']:.0f} SM cycles per env-step of one scene group")
    for name in k2d.PHASES:
        print(f"  {name:20s} {100.0 * out['share'][name]:6.2f} %   {out['cycles_per_env_step_by_phase'][name]:9.1f} cycles per env-step")


if __name__ == "__main__":
    main()
