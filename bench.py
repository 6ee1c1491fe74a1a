#!/usr/bin/env python
"""Benchmark of the batched 2D rigid-body environment step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 3] [--impl reference]

With --gpus N > 1 and no torchrun environment the script starts the N ranks itself (one process per GPU,
rendezvous on 127.0.0.1); under torchrun it is one of the ranks.  Envs are sharded over the ranks with no
exchange of data; NCCL carries only the barrier and the maximum of the ranks' times.

One "step" of the benchmark is one pass of the whole hot path over one batch of synthetic input:
one k2d_step launch that advances every env by FUSED (32) engine steps (actions in, reward and done
out, auto-reset inside), followed by one k2d_obs launch (the symbolic per-entity observation).
Workload 3 is the configuration the headline metric is quoted on: L scenes, 16384 envs, auto-reset
from a pool of 1024 seeded levels, horizon 256.  Prints ONE JSON line.

`--impl reference` times the CPU oracle (a deliberately plain scalar program) on a bounded sample of
the same workload on the host cores; it uses no GPU.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2410_23208_b200 import scenes  # noqa: E402

FUSED = 32   # default number of engine steps fused per k2d_step launch (--fused)
METRIC = "env-steps/sec on 1 B200 (L scenes, 16384 envs); % of FP32 roofline"
UNIT = "env-steps/s"

# FP32 operations the method needs per unit of work, counted from the step's definition (an FMA
# counts 2, every other +,-,*,/,sqrt,compare 1; sincos = 30, tanh = 25).
FLOPS = dict(body=37, circle_box=4, polygon=84, box_test=8, cc=16, pc=94, pp=190,
             pair_prestep=5, man_prestep=54, man_warm=28, man_iter=57, man_pos=10,
             joint_fixed=48 + 33 + 18 + 8, joint_iter=38, thruster=27)


def kernel_source_sha256() -> str:
    import hashlib
    h = hashlib.sha256()
    for name in ("k2d_kernels.cuh", "k2d_api.cu"):
        with open(os.path.join(ROOT, "paper_2410_23208_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def ncu_dram_bytes_per_env_launch(size: str, fused: int, n_envs: int):
    """DRAM bytes (read + write) per env that an ncu capture of one k2d_step launch measured for this size class, number of
    fused steps and env count, from the tracked table of captures (JSON text).  None when no capture matches, and None
    when the kernel sources have changed since the capture (the table carries their hash)."""
    path = os.path.join(ROOT, "profiles", "k2d_step_kernel_dram_traffic.txt")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        table = json.load(f)
    if table.get("source_sha256") != kernel_source_sha256():
        return None
    return table.get("captures", {}).get(f"{size}/{fused}/{n_envs}")


def fp32_peak_tflops(sm_count: int = 148, sm_mhz: float = 1965.0) -> float:
    """148 SMs x 128 FP32 lanes x 2 (FMA) x max SM clock"""
    return sm_count * 128 * 2 * sm_mhz * 1e6 / 1e12


def measured_hbm_gbs() -> tuple:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def algorithmic_flops_per_env_step(dims, levels, counts, solver_iters: int) -> float:
    """Flop model: fixed per-scene work from the level pool's entity counts, the rest from the
    counters the step keeps (pairs past the box test by kind, active pairs, active manifolds)."""
    env_steps = max(1, int(counts[3]))
    n_shapes = float(np.mean(levels["active"].sum(1)))
    n_poly = float(np.mean(levels["active"][:, :dims.n_polygons].sum(1)))
    n_circ = n_shapes - n_poly
    n_joint = float(np.mean(levels["joint_active"].sum(1)))
    n_thr = float(np.mean(levels["thr_active"].sum(1)))
    n_box_tests = dims.n_pairs - n_joint  # unmasked pairs, to first order (joined pairs are masked)
    f = FLOPS
    fixed = (n_shapes * f["body"] + n_circ * f["circle_box"] + n_poly * f["polygon"] + n_box_tests * f["box_test"] +
             n_joint * (f["joint_fixed"] + solver_iters * f["joint_iter"]) + n_thr * f["thruster"])
    per = lambda k: float(counts[k]) / env_steps  # noqa: E731
    var = (per(4) * f["pp"] + per(5) * f["pc"] + per(6) * f["cc"] + per(7) * f["pair_prestep"] +
           per(2) * (f["man_prestep"] + f["man_warm"] + solver_iters * f["man_iter"] + f["man_pos"]))
    return fixed + var


def algorithmic_bytes_per_env_launch(dims, fused: int, mean_active_pairs: float, obs_floats: int) -> dict:
    """HBM bytes the method must move per env: dynamic state in and out once per launch, actions,
    reward, done per step, the observation once per launch.  Level constants come from the pool,
    which stays in L2."""
    n = dims.n_shapes
    state = 4 * (6 * n + 2 * dims.n_joints + 8 + 5 * mean_active_pairs)
    step_io = fused * (4 * dims.n_actions + 4 + 1)
    return dict(step=2 * state + step_io, obs=4 * obs_floats + state)


class ClockSampler:
    """nvidia-smi SM clock and throttle reasons while the timed region runs"""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.rows, self.proc, self.device_index = [], None, device_index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.device_index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def workload_levels(index: int):
    w = scenes.WORKLOADS[index]
    dims = scenes.SIZES[w["size"]]
    levels = scenes.make_levels(w["size"], w["n_levels"], scenes.workload_seed(index), static_prob=w["static_prob"])
    return w, dims, levels


def run_reference(args) -> dict:
    """The oracle as it stands on the host cores, on a bounded sample of the workload."""
    from oracle import k2d_ref
    w, dims, levels = workload_levels(args.workload)
    sample_envs = min(w["n_envs"], 2048)
    cores = os.cpu_count() or 1
    sim = k2d_ref.RefSim(levels, sample_envs, auto_reset=w["auto_reset"], max_episode_steps=w["max_episode_steps"],
                         seed=scenes.workload_seed(args.workload))
    FUSED = args.fused
    acts = scenes.make_actions(FUSED, sample_envs, dims.n_actions, 7)
    for _ in range(args.warmup):
        sim.step(acts, n_threads=cores)
        sim.obs()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        sim.step(acts, n_threads=cores)
        sim.obs()
    dt = time.perf_counter() - t0
    value = sample_envs * FUSED * args.steps / dt
    sample = f"first {sample_envs} envs of the workload, {FUSED} engine steps + 1 observation per bench step"
    return {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w['size']} scenes, {w['n_envs']} envs, {FUSED} fused steps + obs per bench step (config {args.workload})",
                   "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }


def cpu_baseline(args, w, dims, levels) -> dict:
    from oracle import k2d_ref
    cores = os.cpu_count() or 1
    sample_envs, sample_steps = min(w["n_envs"], 4096), 512      # about 20 core-seconds of oracle work for L scenes
    sim = k2d_ref.RefSim(levels, sample_envs, auto_reset=w["auto_reset"], max_episode_steps=w["max_episode_steps"],
                         seed=scenes.workload_seed(args.workload))
    acts = scenes.make_actions(sample_steps, sample_envs, dims.n_actions, 7)
    sim.step(acts[:4], n_threads=cores)
    t0 = time.perf_counter()
    sim.step(acts, n_threads=cores)
    dt = time.perf_counter() - t0
    n1 = min(256, sample_envs)
    one = k2d_ref.RefSim(levels, n1, auto_reset=w["auto_reset"], max_episode_steps=w["max_episode_steps"])
    t1 = time.perf_counter()
    one.step(acts[:32, :n1], n_threads=1)
    dt1 = time.perf_counter() - t1
    return {"value": sample_envs * sample_steps / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {sample_envs} envs x {sample_steps} engine steps of the workload, {cores} threads over envs",
            "one_core_value": n1 * 32 / dt1}


def run_gpu(args) -> dict:
    import torch
    from paper_2410_23208_b200 import k2d

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)

    FUSED = args.fused
    w, dims, levels = workload_levels(args.workload)
    n_envs = args.envs or w["n_envs"]
    # weak scaling: every rank steps its own n_envs; env_offset makes level draws global
    env = k2d.Env(levels, n_envs, device=local, auto_reset=w["auto_reset"], max_episode_steps=w["max_episode_steps"],
                  seed=scenes.workload_seed(args.workload), env_offset=rank * n_envs, max_fused_steps=FUSED,
                  lanes_per_scene=args.lanes, solver_batch=args.solver_batch)
    K, W = args.steps, args.warmup
    n_bufs = max(K, 1)
    host_actions = [torch.from_numpy(scenes.make_actions(FUSED, n_envs, dims.n_actions, 100 + rank * 1000 + i)).pin_memory()
                    for i in range(min(n_bufs, 4))]
    dev_actions = [host_actions[i % len(host_actions)].to(dev) for i in range(n_bufs)]   # K distinct buffers: inputs > L2
    reward = torch.empty((FUSED, n_envs), dtype=torch.float32, device=dev)
    done = torch.empty((FUSED, n_envs), dtype=torch.uint8, device=dev)
    obs = torch.empty((n_envs, env.obs_floats), dtype=torch.float32, device=dev)
    if args.pixels:
        obs = torch.empty((n_envs, 125, 125, 4), dtype=torch.uint8, device=dev)
        env.obs = env.render                      # same call shape: writes into the buffer it is given
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    host_reward = torch.empty((FUSED, n_envs), dtype=torch.float32).pin_memory()
    host_done = torch.empty((FUSED, n_envs), dtype=torch.uint8).pin_memory()
    stage = torch.empty_like(dev_actions[0])

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize(dev)

    clocks = ClockSampler(local)
    clocks.__enter__()
    for i in range(W):
        env.step(dev_actions[i % n_bufs], reward, done)
        env.obs(obs)
    barrier()
    counts0 = env.status().copy()

    launches_per_step = env.step_launches(FUSED) + 1      # the step kernel (with the two launches that sort the envs for its work queue, when it has one) and the observation kernel
    # ---- device-resident timing: events around each step (k2d_step, then k2d_obs); L2 flushed in between, untimed
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    barrier()
    t_wall = time.perf_counter()
    for i in range(K):
        flush.fill_(i & 0xFF)
        ev[i][0].record()
        env.step(dev_actions[i % n_bufs], reward, done)
        ev[i][1].record()
        env.obs(obs)
        ev[i][2].record()
    barrier()
    t_wall = time.perf_counter() - t_wall
    step_ms = [ev[i][0].elapsed_time(ev[i][1]) for i in range(K)]
    obs_ms = [ev[i][1].elapsed_time(ev[i][2]) for i in range(K)]
    total_ms = float(sum(step_ms) + sum(obs_ms))
    counts = env.status() - counts0

    # ---- end to end through the public API with host buffers: every step uploads its actions from pinned host
    # memory and reads reward + done back; a second stream carries the copies, so the upload of step i + 1 and
    # the read-back of step i - 1 overlap the launches of step i (two sets of device buffers)
    copy_stream = torch.cuda.Stream(dev)
    main_stream = torch.cuda.current_stream(dev)
    stages = [stage, torch.empty_like(stage)]
    rewards, dones = [reward, torch.empty_like(reward)], [done, torch.empty_like(done)]
    obses = [obs, torch.empty_like(obs)]
    host_obs = torch.empty(obs.shape, dtype=obs.dtype).pin_memory()

    def e2e_loop(n, with_obs):
        """n bench steps; with_obs: the observation of every step is copied to pinned host memory as well (two device
        observation buffers, so that the copy of step i overlaps the launches of step i + 1)"""
        ev_up = [torch.cuda.Event() for _ in range(n + 3)]
        ev_done = [torch.cuda.Event() for _ in range(n + 3)]
        ev_down = [torch.cuda.Event() for _ in range(n + 3)]

        def upload(i):
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(ev_done[i - 2])       # the launch that last read this staging buffer
                stages[i % 2].copy_(host_actions[i % len(host_actions)], non_blocking=True)
                ev_up[i].record(copy_stream)

        def run(i):
            main_stream.wait_event(ev_up[i])
            if i >= 2:
                main_stream.wait_event(ev_down[i - 2])           # its results have been read back
            env.step(stages[i % 2], rewards[i % 2], dones[i % 2])
            env.obs(obses[i % 2 if with_obs else 0])
            ev_done[i].record(main_stream)

        def download(i):
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(ev_done[i])
                host_reward.copy_(rewards[i % 2], non_blocking=True)
                host_done.copy_(dones[i % 2], non_blocking=True)
                if with_obs:
                    host_obs.copy_(obses[i % 2], non_blocking=True)
                ev_down[i].record(copy_stream)

        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        copy_stream.wait_event(e0)
        upload(0)
        for i in range(n):
            run(i)
            if i + 1 < n:
                upload(i + 1)
            download(i)
        main_stream.wait_event(ev_down[n - 1])
        e1.record()
        barrier()
        return e0.elapsed_time(e1)

    e2e_ms = e2e_loop(K, False)
    # ---- the same loop with the observation copied to the host as well (a learner on the host, or logging)
    K_OBS = min(K, 16)
    e2e_obs_ms = e2e_loop(K_OBS, True) * K / K_OBS

    # ---- how fast this GPU takes a stream of plain stores: the 256 MiB flush buffer filled five times (a yardstick for the
    # observation kernels, which write five to sixty times what they read; the copy figure in `peak` is half reads)
    fill_ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
    flush.fill_(1)
    for i in range(5):
        fill_ev[i].record()
        flush.fill_(i)
    fill_ev[5].record()
    barrier()
    write_only_gbs = flush.numel() / (min(fill_ev[i].elapsed_time(fill_ev[i + 1]) for i in range(5)) * 1e-3) / 1e9

    # ---- other ways to drive the same path (L2 not flushed; the state of 16384 envs stays in L2 between launches anyway):
    # one engine step and one observation per call, as a training loop does, with two launches and with the fused launch
    modes = {}
    if not args.pixels:
        one = [a[:1].contiguous() for a in dev_actions[:2]]
        r1, d1 = reward[:1], done[:1]
        n_it = 64
        for name in ("one_step_then_obs", "one_step_obs_fused"):
            for _ in range(4):
                env.step_obs(one[0], r1, d1, obs)
            barrier()
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0.record()
            for i in range(n_it):
                if name == "one_step_then_obs":
                    env.step(one[i & 1], r1, d1)
                    env.obs(obs)
                else:
                    env.step_obs(one[i & 1], r1, d1, obs)
            m1.record()
            barrier()
            modes[name] = m0.elapsed_time(m1) / n_it
    clocks.__exit__()
    clk = clocks.summary()   # sampled every 100 ms from the first warm-up step to the end of the end-to-end loop

    mode_names = sorted(modes)
    if world > 1:
        t = torch.tensor([total_ms, e2e_ms, float(np.mean(step_ms)), e2e_obs_ms] + [modes[k] for k in mode_names], device=dev, dtype=torch.float64)
        torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
        vals = [float(x) for x in t.tolist()]
        total_ms, e2e_ms, mean_step_ms, e2e_obs_ms = vals[:4]
        modes = dict(zip(mode_names, vals[4:]))
        torch.distributed.destroy_process_group()
    else:
        mean_step_ms = float(np.mean(step_ms))
    if rank != 0:
        return {}

    env_steps_per_launch = n_envs * FUSED
    value = world * env_steps_per_launch * K / (total_ms * 1e-3)
    e2e_value = world * env_steps_per_launch * K / (e2e_ms * 1e-3)
    flops_step = algorithmic_flops_per_env_step(dims, levels, counts, env.cfg.solver_iters)
    mean_pairs = float(counts[7]) / max(1, int(counts[3]))
    bytes_ = algorithmic_bytes_per_env_launch(dims, FUSED, mean_pairs, env.obs_floats)
    if args.pixels:
        bytes_["obs"] = 125 * 125 * 4 + 4 * 6 * dims.n_shapes      # the image out, the poses in
    achieved_tflops = flops_step * env_steps_per_launch / (mean_step_ms * 1e-3) / 1e12
    peak = fp32_peak_tflops()
    peak_measured = k2d.measure_fp32_peak(local)
    traffic_per_env = ncu_dram_bytes_per_env_launch(w["size"], FUSED, n_envs)
    hbm_peak, hbm_src = measured_hbm_gbs()
    hbm_gbs = bytes_["step"] * n_envs / (mean_step_ms * 1e-3) / 1e9
    obs_gbs = bytes_["obs"] * n_envs / (float(np.mean(obs_ms)) * 1e-3) / 1e9
    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w['size']} scenes, {n_envs} envs per GPU, {FUSED} fused engine steps + 1 observation per bench step "
                               f"(config {args.workload}: pool of {w['n_levels']} levels, horizon {w['max_episode_steps']})",
                   "lanes_per_scene": env.lanes_per_scene, "resident_scene_groups": env.resident_groups, "kernel_launches_per_bench_step": launches_per_step, "fused_steps": FUSED,
                   "observation": "pixels 125x125 RGBA (k2d_render)" if args.pixels else "symbolic entity rows (k2d_obs)",
                   "solver_batch": args.solver_batch,
                   "l2": "flushed between timed iterations (256 MiB write, untimed); K distinct action buffers"},
        "clocks": clk,
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": int(stage.numel() * 4), "d2h_bytes_per_step": int(host_reward.numel() * 4 + host_done.numel()),
                "note": "actions up, reward and done down every bench step; the observation stays on the device, where a policy network reads it"},
        "e2e_with_obs": {"value": world * env_steps_per_launch * K / (e2e_obs_ms * 1e-3), "unit": UNIT,
                         "h2d_bytes_per_step": int(stage.numel() * 4),
                         "d2h_bytes_per_step": int(host_reward.numel() * 4 + host_done.numel() + host_obs.numel() * host_obs.element_size()),
                         "note": "as e2e, and the observation is copied to pinned host memory every bench step (two device observation buffers; the copy overlaps the next step's launches)"},
        "modes": {k: {"ms_per_call": v, "value": world * n_envs / (v * 1e-3), "unit": UNIT,
                      "what": ("k2d_step(1 step) + k2d_obs: two launches per call" if k == "one_step_then_obs"
                               else "k2d_step_obs(1 step): one launch per call")} for k, v in modes.items()},
        "gpu_launches": launches_per_step * K,
        "roofline": {"bound": "alu", "kernel": "k2d_step_kernel", "achieved": achieved_tflops, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved_tflops / peak, "traffic": None if traffic_per_env is None else traffic_per_env * n_envs,
                     "peak_source": "derived: 148 SMs x 128 lanes x 2 x 1965 MHz",
                     "peak_measured": peak_measured, "frac_of_measured": achieved_tflops / peak_measured,
                     "peak_measured_source": "chains of fused multiply-adds on every SM, timed in this run (k2d_measure_fp32_peak)",
                     "flops_per_env_step": flops_step, "launch_ms": mean_step_ms,
                     "hbm": {"achieved": hbm_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": hbm_gbs / hbm_peak, "of": hbm_src,
                             "bytes_per_env_launch": bytes_["step"]},
                     "obs_kernel": {"achieved": obs_gbs, "peak": hbm_peak, "unit": "GB/s", "frac": obs_gbs / hbm_peak,
                                    "launch_ms": float(np.mean(obs_ms)), "bytes_per_env_launch": bytes_["obs"],
                                    "write_only_gbs": write_only_gbs, "frac_of_write_only": obs_gbs / write_only_gbs,
                                    "write_only_source": "a 256 MiB device buffer filled with torch's fill kernel, best of five, timed in this run"}},
        "work": {"manifolds_per_env_step": float(counts[2]) / max(1, int(counts[3])), "active_pairs_per_env_step": mean_pairs,
                 "resets": int(counts[1]), "nonfinite": int(counts[0]), "wall_s_timed_region": t_wall},
    }
    if world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(args, w, dims, levels)
    return out


def spawn_ranks(n: int) -> int:
    """--gpus N without a torchrun environment: start the N ranks (this script again, one process per GPU)."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    return max(p.wait() for p in procs)


def run_plan(args) -> dict:
    """--plan: no GPU work; every rank joins a gloo group and reports the env range it would step."""
    import torch
    import torch.distributed as dist
    from paper_2410_23208_b200 import k2d
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    n_envs = args.envs or scenes.WORKLOADS[args.workload]["n_envs"]
    mine = torch.tensor([rank, int(os.environ.get("LOCAL_RANK", "0")), rank * n_envs, n_envs], dtype=torch.int64)
    rows = [mine]
    if world > 1:
        dist.init_process_group("gloo")
        rows = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(rows, mine)
        dist.destroy_process_group()
    if rank != 0:
        return {}
    return {"plan": [dict(rank=int(r[0]), local_rank=int(r[1]), env_offset=int(r[2]), n_envs=int(r[3])) for r in rows],
            "n_gpus": world, "scaling": "weak", "total_envs": int(sum(int(r[3]) for r in rows)),
            "shard_of_total": [list(k2d.shard_envs(world * n_envs, k, world)) for k in range(world)]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=48)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="k2d", choices=["k2d", "reference"])
    ap.add_argument("--workload", type=int, default=3, choices=sorted(scenes.WORKLOADS))
    ap.add_argument("--envs", type=int, default=0, help="override the workload's env count (per GPU)")
    ap.add_argument("--lanes", type=int, default=0, help="lanes per scene (0 = library default)")
    ap.add_argument("--fused", type=int, default=FUSED, help="engine steps per k2d_step launch (1 = one launch and one observation per step)")
    ap.add_argument("--pixels", action="store_true", help="the observation of a bench step is the 125 x 125 pixel image (k2d_render) instead of the entity rows")
    ap.add_argument("--solver-batch", type=int, default=0, help="the paper's batched contact solve with batches of this many manifold slots (0 = sequential)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--plan", action="store_true", help="no GPU work: the ranks rendezvous over gloo and rank 0 prints which envs each would step")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and (args.impl == "k2d" or args.plan):
        sys.exit(spawn_ranks(args.gpus))
    if args.plan:
        out = run_plan(args)
        if out:
            print(json.dumps(out), flush=True)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "k2d" else args.warmup
    if args.impl == "reference":
        if int(os.environ.get("RANK", "0")) != 0:
            return
        print(json.dumps(run_reference(args)), flush=True)
        return
    out = run_gpu(args)
    if out:
        print(json.dumps(out), flush=True)


if __name__ == "__main__":
    main()
