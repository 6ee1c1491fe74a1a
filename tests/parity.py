"""Shared helpers of the GPU parity tests: run the CUDA library and the CPU oracle on the same
seeded inputs and compare the canonical state element by element."""
import numpy as np

from oracle import k2d_ref
from paper_2410_23208_b200 import k2d

# acceptance tolerances of the hot path (max abs error against the oracle)
POS_TOL_1, VEL_TOL_1, TOL_16 = 1e-4, 1e-3, 1e-2

STATE_KEYS = ("pos", "angle", "vel", "angvel", "acc", "jacc")
META_KEYS = ("step_count", "episode_count", "level_id", "status")

ORACLE_CFG = ("solver_iters", "warm_start", "auto_reset", "max_episode_steps", "dt", "gravity_y", "contact_alpha",
              "contact_beta", "slop", "restitution_threshold", "face_tol", "joint_alpha", "joint_beta", "joint_gamma", "motor_rho",
              "aabb_margin", "dense_kappa", "seed", "env_offset", "frame_skip", "n_actions", "solver_batch")


def make_pair(levels, n_envs, broadphase=0, **cfg):
    """(Env on cuda:0, RefSim) with the same configuration.  The oracle runs the narrowphase on every pair that
    may collide (``broadphase=0``): the library's bounding-box test in front of its narrowphase is thereby checked
    against a reference that has no such test.  ``broadphase=1`` gives the oracle the same test, which makes its
    counters of pairs past the test comparable too."""
    checked = cfg.pop("checked", False)
    phase_clocks = cfg.pop("phase_clocks", False)
    env = k2d.Env(levels, n_envs, checked=checked, phase_clocks=phase_clocks, **cfg)
    ocfg = {k: getattr(env.cfg, k) for k in ORACLE_CFG}
    ref = k2d_ref.RefSim(levels, n_envs, broadphase=broadphase, **ocfg)
    return env, ref


def counters_match(env, ref) -> bool:
    """k2d_status against the oracle's counters; the three counts of pairs past the bounding-box test only when the
    oracle runs that test"""
    got, want = env.status(), ref.counters
    keep = np.ones(8, bool)
    if not ref.cfg["broadphase"]:
        keep[4:7] = False
    return bool(np.array_equal(got[keep], want[keep]))


def errors(env, ref):
    """max abs difference per state array, and whether everything is bit-identical"""
    st = env.get_state()
    out, exact = {}, True
    for k in STATE_KEYS:
        a, b = st[k], getattr(ref, k)
        with np.errstate(invalid="ignore"):
            d = np.abs(a.astype(np.float64) - b.astype(np.float64))
        d = np.where(np.isnan(a) & np.isnan(b), 0.0, d)
        out[k] = float(np.nanmax(d)) if d.size else 0.0
        exact = exact and np.array_equal(a.view(np.uint32), b.view(np.uint32))
    for k in META_KEYS:
        same = np.array_equal(st[k], getattr(ref, k))
        out[k] = 0.0 if same else 1.0
        exact = exact and same
    return out, exact


def step_both(env, ref, actions_np, chunk=None, n_threads=1):
    """Steps both by all rows of actions_np; the GPU in launches of `chunk` fused steps."""
    import torch
    n = actions_np.shape[0]
    chunk = chunk or n
    r_ref, d_ref = ref.step(actions_np, n_threads=n_threads)
    rs, ds = [], []
    for s0 in range(0, n, chunk):
        a = torch.from_numpy(np.ascontiguousarray(actions_np[s0:s0 + chunk])).to(env.device)
        r, d = env.step(a)
        rs.append(r.cpu().numpy())
        ds.append(d.cpu().numpy())
    return (np.concatenate(rs), np.concatenate(ds)), (r_ref, d_ref)
