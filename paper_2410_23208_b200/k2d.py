"""Thin Python binding of the C ABI in include/k2d.h (argument marshalling only).

torch supplies device memory and the stream; every step of the path runs in the CUDA library.
There is no fallback: if the library cannot be loaded or no CUDA device is present, constructing
an :class:`Env` raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

from . import build as _build

MAX_POLYGONS, MAX_CIRCLES, MAX_SHAPES, MAX_JOINTS, MAX_THRUSTERS = 12, 4, 16, 6, 2
RESET_NONE, RESET_SAME_LEVEL, RESET_POOL = 0, 1, 2

EXPORTS = (
    "k2d_default_config", "k2d_state_bytes", "k2d_state_bytes_no_scratch", "k2d_level_pool_bytes", "k2d_create", "k2d_reset", "k2d_step",
    "k2d_step_discrete", "k2d_step_static_scratch", "k2d_step_obs", "k2d_obs", "k2d_render",
    "k2d_obs_floats", "k2d_canonical_words", "k2d_get_state", "k2d_set_state", "k2d_status", "k2d_level_info",
    "k2d_set_trace", "k2d_trace_slots", "k2d_is_checked_build", "k2d_phase_cycles", "k2d_resident_groups", "k2d_lanes_per_scene", "k2d_step_launches", "k2d_items_per_ticket", "k2d_set_wait_limit", "k2d_eval_sincos_tanh", "k2d_measure_fp32_peak", "k2d_error_string", "k2d_destroy",
)


class Config(C.Structure):
    _fields_ = (
        [(n, C.c_int32) for n in ("n_envs", "n_polygons", "n_circles", "n_joints", "n_thrusters", "n_actions", "n_levels",
                                  "solver_iters", "warm_start", "auto_reset", "max_episode_steps", "max_fused_steps", "frame_skip")] +
        [(n, C.c_float) for n in ("dt", "gravity_y", "contact_alpha", "contact_beta", "slop", "restitution_threshold",
                                  "face_tol", "joint_alpha", "joint_beta", "motor_rho", "aabb_margin", "joint_gamma", "dense_kappa")] +
        [("seed", C.c_uint64), ("env_offset", C.c_int64), ("device", C.c_int32), ("lanes_per_scene", C.c_int32),
         ("solver_batch", C.c_int32), ("reserved", C.c_int32), ("cuda_stream", C.c_void_p)])


LEVEL_DTYPE = np.dtype([
    ("poly_verts", np.float32, (MAX_POLYGONS, 4, 2)), ("poly_nverts", np.int32, (MAX_POLYGONS,)),
    ("circle_radius", np.float32, (MAX_CIRCLES,)),
    ("pos", np.float32, (MAX_SHAPES, 2)), ("angle", np.float32, (MAX_SHAPES,)),
    ("vel", np.float32, (MAX_SHAPES, 2)), ("angvel", np.float32, (MAX_SHAPES,)),
    ("density", np.float32, (MAX_SHAPES,)), ("friction", np.float32, (MAX_SHAPES,)), ("restitution", np.float32, (MAX_SHAPES,)),
    ("is_static", np.int32, (MAX_SHAPES,)), ("role", np.int32, (MAX_SHAPES,)), ("active", np.int32, (MAX_SHAPES,)),
    ("joint_a", np.int32, (MAX_JOINTS,)), ("joint_b", np.int32, (MAX_JOINTS,)),
    ("joint_anchor_a", np.float32, (MAX_JOINTS, 2)), ("joint_anchor_b", np.float32, (MAX_JOINTS, 2)),
    ("motor_speed", np.float32, (MAX_JOINTS,)), ("motor_power", np.float32, (MAX_JOINTS,)),
    ("motor_binding", np.int32, (MAX_JOINTS,)), ("joint_active", np.int32, (MAX_JOINTS,)),
    ("joint_fixed", np.int32, (MAX_JOINTS,)), ("joint_limited", np.int32, (MAX_JOINTS,)),
    ("joint_fixed_angle", np.float32, (MAX_JOINTS,)), ("joint_min", np.float32, (MAX_JOINTS,)), ("joint_max", np.float32, (MAX_JOINTS,)),
    ("thr_shape", np.int32, (MAX_THRUSTERS,)), ("thr_pos", np.float32, (MAX_THRUSTERS, 2)),
    ("thr_rot", np.float32, (MAX_THRUSTERS,)), ("thr_power", np.float32, (MAX_THRUSTERS,)),
    ("thr_binding", np.int32, (MAX_THRUSTERS,)), ("thr_active", np.int32, (MAX_THRUSTERS,)),
])

_libs = {}


PHASES = ("geometry", "actuators", "joint_prestep", "box_test", "narrowphase", "records", "levels", "warm_start", "iterations",
          "integrate_correct", "epilogue", "memory_record_solve", "load", "store")


def load_library(checked: bool = False, phase_clocks: bool = False):
    """Builds (if stale) and loads libk2d.so (checked=True: the build with index checks; phase_clocks=True: the build that
    counts cycles per phase of a step); raises if that is impossible."""
    key = "checked" if checked else ("phases" if phase_clocks else "")
    if key not in _libs:
        lib = C.CDLL(_build.build(checked=checked, phase_clocks=phase_clocks))
        vp, i32 = C.c_void_p, C.c_int32
        lib.k2d_default_config.argtypes = [C.POINTER(Config), i32, i32, i32, i32, i32]
        lib.k2d_state_bytes.argtypes = [C.POINTER(Config)]
        lib.k2d_state_bytes.restype = C.c_size_t
        lib.k2d_state_bytes_no_scratch.argtypes = [C.POINTER(Config)]
        lib.k2d_state_bytes_no_scratch.restype = C.c_size_t
        lib.k2d_level_pool_bytes.argtypes = [C.POINTER(Config)]
        lib.k2d_level_pool_bytes.restype = C.c_size_t
        lib.k2d_create.argtypes = [C.POINTER(Config), vp, vp, vp, C.POINTER(vp)]
        lib.k2d_reset.argtypes = [vp, vp]
        lib.k2d_step.argtypes = [vp, vp, i32, vp, vp]
        lib.k2d_step_static_scratch.argtypes = [vp, vp, i32, vp, vp]
        lib.k2d_step_discrete.argtypes = [vp, vp, i32, vp, vp]
        lib.k2d_step_obs.argtypes = [vp, vp, i32, vp, vp, vp]
        lib.k2d_obs.argtypes = [vp, vp]
        lib.k2d_render.argtypes = [vp, vp]
        lib.k2d_obs_floats.argtypes = [C.POINTER(Config)]
        lib.k2d_canonical_words.argtypes = [C.POINTER(Config)]
        lib.k2d_get_state.argtypes = [vp, vp]
        lib.k2d_set_state.argtypes = [vp, vp]
        lib.k2d_status.argtypes = [vp, vp]
        lib.k2d_level_info.argtypes = [C.POINTER(Config), vp, vp, vp, vp]
        lib.k2d_set_trace.argtypes = [vp, vp]
        lib.k2d_trace_slots.argtypes = [vp]
        lib.k2d_set_wait_limit.argtypes = [vp, C.c_uint32]
        lib.k2d_phase_cycles.argtypes = [vp, vp, i32]
        lib.k2d_resident_groups.argtypes = [vp]
        lib.k2d_lanes_per_scene.argtypes = [vp]
        lib.k2d_step_launches.argtypes = [vp, i32]
        lib.k2d_items_per_ticket.argtypes = [vp]
        lib.k2d_eval_sincos_tanh.argtypes = [vp, i32, vp, vp, vp, vp]
        lib.k2d_measure_fp32_peak.argtypes = [i32, vp, C.c_size_t, vp]
        lib.k2d_error_string.argtypes = [C.c_int]
        lib.k2d_error_string.restype = C.c_char_p
        lib.k2d_destroy.argtypes = [vp]
        _libs[key] = lib
    return _libs[key]


class K2DError(RuntimeError):
    pass


def _check(rc: int, what: str):
    if rc != 0:
        raise K2DError(f"{what}: {load_library().k2d_error_string(rc).decode()} ({rc})")


def pack_levels(levels: dict) -> np.ndarray:
    """Level dict (see scenes.make_levels) -> array of k2d_level structs."""
    n = levels["pos"].shape[0]
    out = np.zeros(n, LEVEL_DTYPE)
    for name in LEVEL_DTYPE.names:
        src = np.asarray(levels[name])
        dst = out[name]
        sl = (slice(None),) + tuple(slice(0, k) for k in src.shape[1:])
        dst[sl] = src
    return out


def make_config(levels: dict, n_envs: int, **kw) -> Config:
    """Default config for the dimensions of ``levels``, overridden by keyword arguments."""
    lib = load_library()
    P, Cn = levels["poly_nverts"].shape[1], levels["circle_radius"].shape[1]
    J, T = levels["joint_a"].shape[1], levels["thr_shape"].shape[1]
    cfg = Config()
    lib.k2d_default_config(C.byref(cfg), n_envs, P, Cn, J, T)
    cfg.n_levels = levels["pos"].shape[0]
    for k, v in kw.items():
        if not hasattr(cfg, k):
            raise TypeError(f"unknown config field {k}")
        setattr(cfg, k, v)
    return cfg


class Env:
    """n_envs scenes on one CUDA device, stepped by the library."""

    def __init__(self, levels: dict, n_envs: int, device: int = 0, stream=None, checked: bool = False, phase_clocks: bool = False, **cfg_kw):
        import torch
        if not torch.cuda.is_available():
            raise K2DError("no CUDA device: the k2d library has no CPU fallback")
        self.torch = torch
        self.lib = load_library(checked, phase_clocks)
        self.device = torch.device("cuda", device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self.cfg = make_config(levels, n_envs, device=device, **cfg_kw)
        self.cfg.cuda_stream = self.stream.cuda_stream
        self.n_envs, self.n_actions = n_envs, self.cfg.n_actions
        sb = self.lib.k2d_state_bytes(C.byref(self.cfg))
        lb = self.lib.k2d_level_pool_bytes(C.byref(self.cfg))
        if sb == 0 or lb == 0:
            raise K2DError("invalid config")
        with torch.cuda.device(self.device):
            self.state_buf = torch.empty(sb, dtype=torch.uint8, device=self.device)
            self.level_buf = torch.empty(lb, dtype=torch.uint8, device=self.device)
        packed = pack_levels(levels)
        h = C.c_void_p()
        _check(self.lib.k2d_create(C.byref(self.cfg), self.state_buf.data_ptr(), self.level_buf.data_ptr(),
                                   packed.ctypes.data, C.byref(h)), "k2d_create")
        self._h = h
        self.obs_floats = self.lib.k2d_obs_floats(C.byref(self.cfg))
        self.canonical_words = self.lib.k2d_canonical_words(C.byref(self.cfg))
        self._trace = None

    def close(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            self.lib.k2d_destroy(h)

    def __del__(self):
        self.close()

    def reset(self, level_ids=None):
        ids = None if level_ids is None else np.ascontiguousarray(level_ids, np.int32)
        _check(self.lib.k2d_reset(self._h, None if ids is None else ids.ctypes.data), "k2d_reset")

    def step(self, actions, reward=None, done=None, static_scratch=False, n_steps=None):
        """actions: CUDA float32 [n_steps, n_envs, n_actions]; returns (reward, done) CUDA tensors [n_steps, n_envs].

        ``static_scratch=True`` goes through k2d_step_static_scratch: same results, but the records of
        crowded scenes live in an array inside the library instead of the tail of the state buffer
        (for callers that cannot allocate that tail; at most 1024 envs)."""
        torch = self.torch
        assert actions.is_cuda and actions.dtype in (torch.float32, torch.int32) and actions.is_contiguous()
        discrete = actions.dtype == torch.int32        # multi-discrete codes go through k2d_step_discrete
        assert not (discrete and static_scratch)
        if actions.dim() == 2:
            actions = actions.unsqueeze(0)
        fs = max(1, int(self.cfg.frame_skip))
        n_steps = actions.shape[0] * fs if n_steps is None else int(n_steps)      # every action row is held for frame_skip steps
        assert tuple(actions.shape) == (-(-n_steps // fs), self.n_envs, self.n_actions), tuple(actions.shape)
        if reward is None:
            reward = torch.empty((n_steps, self.n_envs), dtype=torch.float32, device=self.device)
        if done is None:
            done = torch.empty((n_steps, self.n_envs), dtype=torch.uint8, device=self.device)
        fn, name = ((self.lib.k2d_step_static_scratch, "k2d_step_static_scratch") if static_scratch
                    else (self.lib.k2d_step_discrete, "k2d_step_discrete") if discrete else (self.lib.k2d_step, "k2d_step"))
        _check(fn(self._h, actions.data_ptr(), n_steps, reward.data_ptr(), done.data_ptr()), name)
        return reward, done

    def step_obs(self, actions, reward=None, done=None, obs=None, n_steps=None):
        """k2d_step_obs: the steps of ``step`` and the observation of the state they leave, in one launch;
        returns (reward, done, obs)"""
        torch = self.torch
        assert actions.is_cuda and actions.dtype == torch.float32 and actions.is_contiguous()
        if actions.dim() == 2:
            actions = actions.unsqueeze(0)
        fs = max(1, int(self.cfg.frame_skip))
        n_steps = actions.shape[0] * fs if n_steps is None else int(n_steps)
        assert tuple(actions.shape) == (-(-n_steps // fs), self.n_envs, self.n_actions), tuple(actions.shape)
        if reward is None:
            reward = torch.empty((n_steps, self.n_envs), dtype=torch.float32, device=self.device)
        if done is None:
            done = torch.empty((n_steps, self.n_envs), dtype=torch.uint8, device=self.device)
        if obs is None:
            obs = torch.empty((self.n_envs, self.obs_floats), dtype=torch.float32, device=self.device)
        _check(self.lib.k2d_step_obs(self._h, actions.data_ptr(), n_steps, reward.data_ptr(), done.data_ptr(), obs.data_ptr()), "k2d_step_obs")
        return reward, done, obs

    def obs(self, out=None):
        torch = self.torch
        if out is None:
            out = torch.empty((self.n_envs, self.obs_floats), dtype=torch.float32, device=self.device)
        _check(self.lib.k2d_obs(self._h, out.data_ptr()), "k2d_obs")
        return out

    def render(self, out=None):
        """RGBA byte images [n_envs, 125, 125, 4] of the scenes (the pixel observation)"""
        torch = self.torch
        if out is None:
            out = torch.empty((self.n_envs, 125, 125, 4), dtype=torch.uint8, device=self.device)
        _check(self.lib.k2d_render(self._h, out.data_ptr()), "k2d_render")
        return out

    # ---- canonical state
    def _split(self, raw: np.ndarray) -> dict:
        c = self.cfg
        N, J = c.n_polygons + c.n_circles, c.n_joints
        S = c.n_polygons * (c.n_polygons - 1) + c.n_polygons * c.n_circles + c.n_circles * (c.n_circles - 1) // 2
        f = raw.view(np.float32)
        o = 0
        out = {}
        for name, shape in (("pos", (N, 2)), ("angle", (N,)), ("vel", (N, 2)), ("angvel", (N,)), ("acc", (S, 2)), ("jacc", (J, 3))):
            n = int(np.prod(shape))
            out[name] = f[:, o:o + n].reshape((-1,) + shape).copy()
            o += n
        meta = raw[:, o:o + 4].view(np.int32)
        for k, name in enumerate(("step_count", "episode_count", "level_id", "status")):
            out[name] = meta[:, k].copy()
        return out

    def get_state(self) -> dict:
        raw = np.zeros((self.n_envs, self.canonical_words), np.uint32)
        _check(self.lib.k2d_get_state(self._h, raw.ctypes.data), "k2d_get_state")
        return self._split(raw)

    def set_state(self, st: dict):
        parts = [np.asarray(st[k], np.float32).reshape(self.n_envs, -1).view(np.uint32)
                 for k in ("pos", "angle", "vel", "angvel", "acc", "jacc")]
        parts += [np.asarray(st[k], np.int32).reshape(self.n_envs, 1).view(np.uint32)
                  for k in ("step_count", "episode_count", "level_id", "status")]
        raw = np.ascontiguousarray(np.concatenate(parts, axis=1))
        assert raw.shape == (self.n_envs, self.canonical_words)
        _check(self.lib.k2d_set_state(self._h, raw.ctypes.data), "k2d_set_state")

    def status(self) -> np.ndarray:
        out = np.zeros(8, np.int64)
        _check(self.lib.k2d_status(self._h, out.ctypes.data), "k2d_status")
        return out

    def set_wait_limit(self, polls: int):
        """test aid: polls a scene group waits for another group's part of the same env before it gives up"""
        _check(self.lib.k2d_set_wait_limit(self._h, int(polls)), "k2d_set_wait_limit")

    @property
    def resident_groups(self) -> int:
        """scenes the device steps at once for this handle"""
        return int(self.lib.k2d_resident_groups(self._h))

    @property
    def lanes_per_scene(self) -> int:
        return int(self.lib.k2d_lanes_per_scene(self._h))

    @property
    def items_per_ticket(self) -> int:
        """test aid: work items one ticket of the launch's work queue stands for"""
        return int(self.lib.k2d_items_per_ticket(self._h))

    def step_launches(self, n_steps: int) -> int:
        """kernel launches the next step call of n_steps steps makes (the step kernel, and the two that sort the envs when it does)"""
        return int(self.lib.k2d_step_launches(self._h, int(n_steps)))

    def phase_cycles(self) -> dict:
        """measurement aid (phase_clocks=True builds): SM cycles the scene groups spent in each phase of a step since the last
        call, by phase name; clears the sums"""
        out = (C.c_uint64 * len(PHASES))()
        _check(self.lib.k2d_phase_cycles(self._h, out, len(PHASES)), "k2d_phase_cycles")
        return {name: int(out[i]) for i, name in enumerate(PHASES)}

    def enable_trace(self):
        torch = self.torch
        slots = self.lib.k2d_trace_slots(self._h)
        self._trace = torch.zeros((self.n_envs, slots, 6), dtype=torch.float32, device=self.device)
        _check(self.lib.k2d_set_trace(self._h, self._trace.data_ptr()), "k2d_set_trace")
        return self._trace


def level_info(cfg: Config, packed_level: np.ndarray):
    """Host only: (inv_mass, inv_inertia, collide) the library derives for one packed level."""
    lib = load_library()
    N = cfg.n_polygons + cfg.n_circles
    im, ii = np.zeros(N, np.float32), np.zeros(N, np.float32)
    col = np.zeros(N * (N - 1) // 2, np.uint8)
    lvl = np.ascontiguousarray(packed_level)
    _check(lib.k2d_level_info(C.byref(cfg), lvl.ctypes.data, im.ctypes.data, ii.ctypes.data, col.ctypes.data), "k2d_level_info")
    return im, ii, col


def eval_sincos_tanh(x):
    """The library's own cos, sin and tanh of a CUDA float32 tensor."""
    import torch
    lib = load_library()
    x = x.contiguous()
    c, s, t = torch.empty_like(x), torch.empty_like(x), torch.empty_like(x)
    _check(lib.k2d_eval_sincos_tanh(x.data_ptr(), x.numel(), c.data_ptr(), s.data_ptr(), t.data_ptr(),
                                    torch.cuda.current_stream(x.device).cuda_stream), "k2d_eval_sincos_tanh")
    return c, s, t


def measure_fp32_peak(device: int = 0) -> float:
    """TFLOP/s the device's FP32 pipes reach on chains of fused multiply-adds (k2d_measure_fp32_peak)"""
    import torch
    lib = load_library()
    n = 2048 * torch.cuda.get_device_properties(device).multi_processor_count
    buf = torch.empty(n, dtype=torch.float32, device=torch.device("cuda", device))
    out = C.c_float()
    _check(lib.k2d_measure_fp32_peak(device, buf.data_ptr(), n, C.byref(out)), "k2d_measure_fp32_peak")
    return float(out.value)


def first_outcomes(reward: np.ndarray, done: np.ndarray) -> np.ndarray:
    """Per env, the reward at its first done step of a rollout without auto-reset ([n_steps][n_envs] arrays):
    +1 solved, -1 failed, 0 timed out or never done.  Host logic only."""
    reward, done = np.asarray(reward), np.asarray(done).astype(bool)
    first = np.argmax(done, axis=0)
    out = reward[first, np.arange(reward.shape[1])]
    return np.where(done.any(axis=0), np.sign(out), 0).astype(np.int8)


def noop_outcomes(levels: dict, n_steps: int, device: int = 0, chunk: int = 32, **cfg_kw) -> np.ndarray:
    """What doing nothing achieves on every level: one env per level, zero actions for ``n_steps`` steps, no
    auto-reset; returns +1 / -1 / 0 per level (see first_outcomes).  The paper's level generator rejects levels
    that the no-op policy solves ("trivially solvable"); this is that rollout, run by the CUDA library."""
    import torch
    n = levels["pos"].shape[0]
    env = Env(levels, n, device=device, auto_reset=RESET_NONE, max_fused_steps=chunk, **cfg_kw)
    zeros = torch.zeros((chunk, n, env.n_actions), dtype=torch.float32, device=env.device)
    rs, ds = [], []
    for s0 in range(0, n_steps, chunk):
        k = min(chunk, n_steps - s0)
        r, d = env.step(zeros[:k])
        rs.append(r.cpu().numpy())
        ds.append(d.cpu().numpy())
    env.close()
    return first_outcomes(np.concatenate(rs), np.concatenate(ds))


def shard_envs(n_envs_total: int, rank: int, world_size: int):
    """Contiguous env range of ``rank``: (offset, count).  Envs are independent, so ranks never
    exchange data; the offset goes into ``env_offset`` so that level draws on auto-reset do not
    depend on the number of ranks."""
    base, rem = divmod(n_envs_total, world_size)
    count = base + (1 if rank < rem else 0)
    offset = rank * base + min(rank, rem)
    return offset, count
