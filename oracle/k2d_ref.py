"""ctypes front end of the CPU oracle (TEST INFRASTRUCTURE, not the product).

Builds ``k2d_oracle.c`` with gcc (fp32 parity build and the fp64 build used by
closed-form pins) and wraps its calls.  Nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "k2d_oracle.c")
_LIBS = {}

DEFAULTS = dict(
    solver_iters=8, warm_start=1, auto_reset=0, max_episode_steps=0, broadphase=1, discrete_actions=0, frame_skip=1, solver_batch=0,
    dt=1.0 / 60.0, gravity_y=-9.81, contact_alpha=6.0, contact_beta=0.1, slop=0.005,
    restitution_threshold=1.0, face_tol=1e-3, joint_alpha=6.0, joint_beta=0.1, joint_gamma=6.0, dense_kappa=0.0, motor_rho=1.0,
    aabb_margin=0.01, seed=0, env_offset=0,
)

_REAL_FIELDS = ("dt", "gravity_y", "contact_alpha", "contact_beta", "slop", "restitution_threshold", "face_tol",
                "joint_alpha", "joint_beta", "motor_rho", "aabb_margin", "joint_gamma", "dense_kappa")
_INT_FIELDS = ("n_polygons", "n_circles", "n_joints", "n_thrusters", "n_actions", "n_levels", "n_envs",
               "solver_iters", "warm_start", "auto_reset", "max_episode_steps", "broadphase", "discrete_actions", "frame_skip", "solver_batch")

_LEVEL_REAL = ("poly_verts", "circle_radius", "pos", "angle", "vel", "angvel", "density", "friction", "restitution",
               "joint_anchor_a", "joint_anchor_b", "motor_speed", "motor_power", "joint_fixed_angle", "joint_min", "joint_max",
               "thr_pos", "thr_rot", "thr_power")
_LEVEL_ORDER = ("poly_verts", "poly_nverts", "circle_radius", "pos", "angle", "vel", "angvel", "density", "friction",
                "restitution", "is_static", "role", "active", "joint_a", "joint_b", "joint_anchor_a",
                "joint_anchor_b", "motor_speed", "motor_power", "motor_binding", "joint_active", "joint_fixed",
                "joint_limited", "joint_fixed_angle", "joint_min", "joint_max", "thr_shape",
                "thr_pos", "thr_rot", "thr_power", "thr_binding", "thr_active")


def build(force: bool = False) -> dict:
    """Compile both oracle libraries next to the source; returns their paths."""
    out = {}
    for tag, flags in (("f32", []), ("f64", ["-DK2D_ORACLE_F64"])):
        so = os.path.join(_HERE, f"libk2d_oracle_{tag}.so")
        if force or not os.path.exists(so) or os.path.getmtime(so) < os.path.getmtime(_SRC):
            cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared",
                   *flags, "-o", so, _SRC, "-lm", "-lpthread"]
            subprocess.check_call(cmd)
        out[tag] = so
    return out


def _lib(f64: bool):
    tag = "f64" if f64 else "f32"
    if tag not in _LIBS:
        lib = C.CDLL(build()[tag])
        real = C.c_double if f64 else C.c_float
        lib.k2d_ref_create.restype = C.c_void_p
        lib.k2d_ref_create.argtypes = [C.c_void_p, C.c_void_p]
        lib.k2d_ref_destroy.argtypes = [C.c_void_p]
        lib.k2d_ref_reset.argtypes = [C.c_void_p, C.c_void_p]
        lib.k2d_ref_views.argtypes = [C.c_void_p, C.c_void_p]
        lib.k2d_ref_step.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int]
        lib.k2d_ref_obs.argtypes = [C.c_void_p, C.c_void_p]
        lib.k2d_ref_render.argtypes = [C.c_void_p, C.c_void_p]
        lib.k2d_ref_obs_floats.argtypes = [C.c_void_p]
        lib.k2d_ref_obs_floats.restype = C.c_int
        lib.k2d_ref_sincos.argtypes = [real, C.c_void_p, C.c_void_p]
        lib.k2d_ref_tanh.argtypes = [real]
        lib.k2d_ref_tanh.restype = real
        lib.k2d_ref_mix64.argtypes = [C.c_uint64]
        lib.k2d_ref_mix64.restype = C.c_uint64
        lib.k2d_ref_manifold_cc.argtypes = [C.c_void_p, real, C.c_void_p, real, C.c_void_p]
        lib.k2d_ref_manifold_pc.argtypes = [C.c_void_p, C.c_int, C.c_void_p, real, C.c_void_p]
        lib.k2d_ref_manifold_pp.argtypes = [C.c_void_p, C.c_int, C.c_void_p, C.c_int, real, C.c_void_p]
        assert lib.k2d_ref_real_bytes() == (8 if f64 else 4)
        _LIBS[tag] = lib
    return _LIBS[tag]


def _config_struct(f64: bool):
    real = C.c_double if f64 else C.c_float

    class Config(C.Structure):
        _fields_ = ([(n, C.c_int32) for n in _INT_FIELDS] + [(n, real) for n in _REAL_FIELDS] +
                    [("seed", C.c_uint64), ("env_offset", C.c_int64)])
    return Config


class _Views(C.Structure):
    _fields_ = ([(n, C.c_void_p) for n in ("pos", "angle", "vel", "angvel", "acc", "jacc", "step_count",
                                            "episode_count", "level_id", "status", "manifold", "inv_mass",
                                            "inv_inertia", "pair_a", "pair_b", "pair_slot", "collide", "counters")] +
                [("n_pairs", C.c_int32), ("n_slots", C.c_int32)])


def _as(ptr, shape, dtype):
    n = int(np.prod(shape))
    if n == 0:
        return np.zeros(shape, dtype)
    buf = (C.c_char * (n * np.dtype(dtype).itemsize)).from_address(ptr)
    return np.frombuffer(buf, dtype=dtype).reshape(shape)


class RefSim:
    """The oracle for ``n_envs`` scenes drawn from a level dict (see scenes.make_levels)."""

    def __init__(self, levels: dict, n_envs: int, f64: bool = False, **cfg):
        self.f64 = f64
        self.real = np.float64 if f64 else np.float32
        self.lib = _lib(f64)
        P = levels["poly_nverts"].shape[1]
        Cn = levels["circle_radius"].shape[1]
        J = levels["joint_a"].shape[1]
        T = levels["thr_shape"].shape[1]
        L = levels["pos"].shape[0]
        full = dict(DEFAULTS)
        full.update(n_polygons=P, n_circles=Cn, n_joints=J, n_thrusters=T, n_actions=J + T, n_levels=L, n_envs=n_envs)
        full.update(cfg)
        self.cfg = full
        Config = _config_struct(f64)
        self._c = Config(**{k: (int(v) if k not in _REAL_FIELDS else float(v)) for k, v in full.items()})
        self._keep = []
        ptrs = []
        for name in _LEVEL_ORDER:
            dt = self.real if name in _LEVEL_REAL else np.int32
            a = np.ascontiguousarray(levels[name], dtype=dt)
            self._keep.append(a)
            ptrs.append(a.ctypes.data)
        arr = (C.c_void_p * len(ptrs))(*ptrs)
        self._h = self.lib.k2d_ref_create(C.byref(self._c), arr)
        v = _Views()
        self.lib.k2d_ref_views(self._h, C.byref(v))
        E, N = n_envs, P + Cn
        self.n_pairs, self.n_slots = v.n_pairs, v.n_slots
        r = self.real
        self.pos = _as(v.pos, (E, N, 2), r)
        self.angle = _as(v.angle, (E, N), r)
        self.vel = _as(v.vel, (E, N, 2), r)
        self.angvel = _as(v.angvel, (E, N), r)
        self.acc = _as(v.acc, (E, self.n_slots, 2), r)
        self.jacc = _as(v.jacc, (E, J, 3), r)
        self.step_count = _as(v.step_count, (E,), np.int32)
        self.episode_count = _as(v.episode_count, (E,), np.int32)
        self.level_id = _as(v.level_id, (E,), np.int32)
        self.status = _as(v.status, (E,), np.int32)
        self.manifold = _as(v.manifold, (E, self.n_slots, 6), r)
        self.inv_mass = _as(v.inv_mass, (L, N), r)
        self.inv_inertia = _as(v.inv_inertia, (L, N), r)
        self.pair_a = _as(v.pair_a, (self.n_pairs,), np.int32)
        self.pair_b = _as(v.pair_b, (self.n_pairs,), np.int32)
        self.pair_slot = _as(v.pair_slot, (self.n_pairs,), np.int32)
        self.collide = _as(v.collide, (L, self.n_pairs), np.uint8)
        self.counters = _as(v.counters, (8,), np.int64)
        self.n_envs, self.n_actions = E, int(full["n_actions"])
        self.obs_floats = self.lib.k2d_ref_obs_floats(C.byref(self._c))

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            self.lib.k2d_ref_destroy(h)

    def reset(self, level_ids=None):
        ids = None if level_ids is None else np.ascontiguousarray(level_ids, np.int32)
        self.lib.k2d_ref_reset(self._h, None if ids is None else ids.ctypes.data)

    def step(self, actions, n_threads: int = 1, n_steps=None):
        """actions [ceil(n_steps / frame_skip)][n_envs][n_actions] -> (reward [n_steps][n_envs], done uint8 [n_steps][n_envs])"""
        a = np.ascontiguousarray(actions, dtype=self.real)
        if a.ndim == 2:
            a = a[None]
        fs = max(1, int(self.cfg["frame_skip"]))
        n_steps = a.shape[0] * fs if n_steps is None else int(n_steps)
        assert a.shape == (-(-n_steps // fs), self.n_envs, self.n_actions), a.shape
        reward = np.zeros((n_steps, self.n_envs), self.real)
        done = np.zeros((n_steps, self.n_envs), np.uint8)
        self.lib.k2d_ref_step(self._h, a.ctypes.data, n_steps, reward.ctypes.data, done.ctypes.data, int(n_threads))
        return reward, done

    def obs(self):
        o = np.zeros((self.n_envs, self.obs_floats), self.real)
        self.lib.k2d_ref_obs(self._h, o.ctypes.data)
        return o

    def render(self):
        """RGBA byte images [n_envs][125][125][4] of the scenes (the pixel observation)"""
        img = np.zeros((self.n_envs, 125, 125, 4), np.uint8)
        self.lib.k2d_ref_render(self._h, img.ctypes.data)
        return img

    def snapshot(self) -> dict:
        return {k: getattr(self, k).copy() for k in ("pos", "angle", "vel", "angvel", "acc", "jacc", "step_count",
                                                     "episode_count", "level_id", "status")}


def sincos(theta, f64: bool = False):
    lib = _lib(f64)
    real = C.c_double if f64 else C.c_float
    th = np.atleast_1d(np.asarray(theta, np.float64 if f64 else np.float32))
    c = np.zeros_like(th)
    s = np.zeros_like(th)
    cc, ss = real(), real()
    for i, t in enumerate(th):
        lib.k2d_ref_sincos(real(t), C.byref(cc), C.byref(ss))
        c[i], s[i] = cc.value, ss.value
    return c, s


def tanh(x, f64: bool = False):
    lib = _lib(f64)
    real = C.c_double if f64 else C.c_float
    xs = np.atleast_1d(np.asarray(x, np.float64 if f64 else np.float32))
    return np.array([lib.k2d_ref_tanh(real(v)) for v in xs], xs.dtype)


def mix64(z: int) -> int:
    return int(_lib(False).k2d_ref_mix64(C.c_uint64(z & (2 ** 64 - 1))))


def _man(out):
    return dict(p=out[0:2].copy(), n=out[2:4].copy(), pen=float(out[4]), active=bool(out[5]))


def manifold_cc(pa, ra, pb, rb, f64: bool = False):
    lib, r = _lib(f64), (np.float64 if f64 else np.float32)
    a, b, out = np.asarray(pa, r), np.asarray(pb, r), np.zeros(6, r)
    lib.k2d_ref_manifold_cc(a.ctypes.data, float(ra), b.ctypes.data, float(rb), out.ctypes.data)
    return _man(out)


def manifold_pc(verts, c, radius, f64: bool = False):
    lib, r = _lib(f64), (np.float64 if f64 else np.float32)
    v = np.ascontiguousarray(verts, r)
    cc, out = np.asarray(c, r), np.zeros(6, r)
    lib.k2d_ref_manifold_pc(v.ctypes.data, len(v), cc.ctypes.data, float(radius), out.ctypes.data)
    return _man(out)


def manifold_pp(va, vb, face_tol=1e-3, f64: bool = False):
    lib, r = _lib(f64), (np.float64 if f64 else np.float32)
    a, b, out = np.ascontiguousarray(va, r), np.ascontiguousarray(vb, r), np.zeros(12, r)
    lib.k2d_ref_manifold_pp(a.ctypes.data, len(a), b.ctypes.data, len(b), float(face_tol), out.ctypes.data)
    return [_man(out[0:6]), _man(out[6:12])]
