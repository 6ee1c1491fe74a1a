"""Seeded synthetic scenes and actions for the batched 2D rigid-body step.

The paper's own workloads (its random level distribution and its 74 handmade
levels) are not available, so scenes with the paper's S / M / L entity counts
(table "The size of each environment class") are drawn here from stated
distributions.  This module only *describes* scenes (vertices, radii, poses,
material numbers, joints, thrusters, roles) and draws actions.  It contains
none of the engine's arithmetic: mass properties, collision geometry and the
step itself are computed separately by the CUDA library and by the CPU oracle,
which both take the arrays produced here as input.

Recipe per level (all draws from ``PCG64(SeedSequence([seed, level_index]))``):

* shape 0 is the fixated floor, a 10 m x 1 m box whose top face is y = 0;
* the other polygons are boxes with half-extents U[0.05, 1.0] (optionally
  triangles), circles have radius U[0.05, 0.5]; density U[0.5, 2], friction
  U[0, 1], restitution U[0, 0.5], angle U[-pi, pi), zero initial velocity;
* free shapes are placed by rejection in x U[-2.5, 2.5], y U[r + 0.02, 5] until
  their bounding circle clears every placed shape and the floor by 0.02 m; after
  200 failures the shape is dropped in just above the highest shape placed so
  far, so crowded (L) scenes start as a pile that falls and settles;
* ``n_joints`` shapes are attached to an earlier non-floor shape by a revolute
  joint with a motor (anchor within 0.8 of the partner's extent, at one end or
  the centre of the new shape), speed U[1, 4] rad/s, power scaled so one step
  changes the relative spin by at most U[0.1, 0.8] rad/s;
* thrusters sit on a random movable shape, power U[0.5, 2] x weight;
* one green and one blue shape (never joined to each other) in every level and
  a red one when ``with_red``; each non-floor shape is fixated with
  probability ``static_prob``.
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np

ROLE_NONE, ROLE_GREEN, ROLE_BLUE, ROLE_RED = 0, 1, 2, 3


@dataclass(frozen=True)
class SceneDims:
    n_polygons: int
    n_circles: int
    n_joints: int
    n_thrusters: int

    @property
    def n_shapes(self) -> int:
        return self.n_polygons + self.n_circles

    @property
    def n_actions(self) -> int:
        return self.n_joints + self.n_thrusters

    @property
    def n_pairs(self) -> int:
        n = self.n_shapes
        return n * (n - 1) // 2

    @property
    def n_slots(self) -> int:
        p, c = self.n_polygons, self.n_circles
        return p * (p - 1) + p * c + c * (c - 1) // 2


SIZES = {
    "S": SceneDims(5, 2, 1, 1),
    "M": SceneDims(6, 3, 2, 2),
    "L": SceneDims(12, 4, 6, 2),
}

LEVEL_FIELDS = (
    ("poly_verts", np.float32), ("poly_nverts", np.int32), ("circle_radius", np.float32),
    ("pos", np.float32), ("angle", np.float32), ("vel", np.float32), ("angvel", np.float32),
    ("density", np.float32), ("friction", np.float32), ("restitution", np.float32),
    ("is_static", np.int32), ("role", np.int32), ("active", np.int32),
    ("joint_a", np.int32), ("joint_b", np.int32), ("joint_anchor_a", np.float32), ("joint_anchor_b", np.float32),
    ("motor_speed", np.float32), ("motor_power", np.float32), ("motor_binding", np.int32), ("joint_active", np.int32),
    ("joint_fixed", np.int32), ("joint_limited", np.int32), ("joint_fixed_angle", np.float32),
    ("joint_min", np.float32), ("joint_max", np.float32),
    ("thr_shape", np.int32), ("thr_pos", np.float32), ("thr_rot", np.float32), ("thr_power", np.float32),
    ("thr_binding", np.int32), ("thr_active", np.int32),
)


def empty_levels(dims: SceneDims, n_levels: int) -> dict:
    """Zero-filled level arrays of the right shapes (all entities inactive)."""
    P, C, N, J, T = dims.n_polygons, dims.n_circles, dims.n_shapes, dims.n_joints, dims.n_thrusters
    shapes = {
        "poly_verts": (P, 4, 2), "poly_nverts": (P,), "circle_radius": (C,),
        "pos": (N, 2), "angle": (N,), "vel": (N, 2), "angvel": (N,),
        "density": (N,), "friction": (N,), "restitution": (N,),
        "is_static": (N,), "role": (N,), "active": (N,),
        "joint_a": (J,), "joint_b": (J,), "joint_anchor_a": (J, 2), "joint_anchor_b": (J, 2),
        "motor_speed": (J,), "motor_power": (J,), "motor_binding": (J,), "joint_active": (J,),
        "joint_fixed": (J,), "joint_limited": (J,), "joint_fixed_angle": (J,), "joint_min": (J,), "joint_max": (J,),
        "thr_shape": (T,), "thr_pos": (T, 2), "thr_rot": (T,), "thr_power": (T,),
        "thr_binding": (T,), "thr_active": (T,),
    }
    lv = {name: np.zeros((n_levels,) + shapes[name], dtype=dt) for name, dt in LEVEL_FIELDS}
    lv["poly_nverts"][:] = 4
    # a unit box keeps derived quantities finite for entities that stay inactive
    lv["poly_verts"][:] = np.array([[-0.5, -0.5], [0.5, -0.5], [0.5, 0.5], [-0.5, 0.5]], np.float32)
    lv["circle_radius"][:] = 0.5
    lv["density"][:] = 1.0
    return lv


class _Draws:
    """Sequential uniform draws from one level's stream, as Python floats."""

    def __init__(self, seed: int, index: int):
        self._rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(index)])))
        self._buf = []

    def u(self, lo: float = 0.0, hi: float = 1.0) -> float:
        if not self._buf:
            self._buf = self._rng.random(4096).tolist()[::-1]
        return lo + (hi - lo) * self._buf.pop()

    def integer(self, lo: int, hi: int) -> int:
        """uniform integer in [lo, hi)"""
        return min(hi - 1, lo + int(self.u() * (hi - lo)))


def _box(hx: float, hy: float):
    return [(-hx, -hy), (hx, -hy), (hx, hy), (-hx, hy)]


def _triangle(hx: float, hy: float):
    return [(-hx, -2.0 * hy / 3.0), (hx, -2.0 * hy / 3.0), (0.0, 4.0 * hy / 3.0), (0.0, 0.0)]


def _rot(c: float, s: float, v):
    return (c * v[0] - s * v[1], s * v[0] + c * v[1])


def _one_level(dims: SceneDims, seed: int, index: int, static_prob: float, with_red, triangle_prob: float, out: dict,
               fixed_prob: float = 0.0, limit_prob: float = 0.0):
    P, C, N, J, T = dims.n_polygons, dims.n_circles, dims.n_shapes, dims.n_joints, dims.n_thrusters
    d = _Draws(seed, index)
    verts = [None] * P
    nverts = [4] * P
    hx = [0.0] * N
    hy = [0.0] * N
    brad = [0.0] * N
    area = [0.0] * N
    inertia_per_density = [0.0] * N
    # --- shapes ---
    verts[0] = _box(5.0, 0.5)
    hx[0], hy[0] = 5.0, 0.5
    for i in range(1, P):
        hx[i], hy[i] = d.u(0.05, 1.0), d.u(0.05, 1.0)
        if d.u() < triangle_prob:
            verts[i] = _triangle(hx[i], hy[i])
            nverts[i] = 3
            brad[i] = max(math.hypot(v[0], v[1]) for v in verts[i][:3])
            area[i] = 2.0 * hx[i] * hy[i]
            inertia_per_density[i] = area[i] * (hx[i] ** 2 + hy[i] ** 2) / 4.5
        else:
            verts[i] = _box(hx[i], hy[i])
            brad[i] = math.hypot(hx[i], hy[i])
            area[i] = 4.0 * hx[i] * hy[i]
            inertia_per_density[i] = area[i] * (hx[i] ** 2 + hy[i] ** 2) / 3.0
    radius = [0.0] * C
    for c in range(C):
        r = d.u(0.05, 0.5)
        radius[c] = r
        i = P + c
        hx[i] = hy[i] = brad[i] = r
        area[i] = math.pi * r * r
        inertia_per_density[i] = area[i] * r * r / 2.0
    density = [1.0] + [d.u(0.5, 2.0) for _ in range(N - 1)]
    friction = [d.u(0.0, 1.0) for _ in range(N)]
    restitution = [d.u(0.0, 0.5) for _ in range(N)]
    static = [1] + [1 if d.u() < static_prob else 0 for _ in range(N - 1)]
    # --- joints: child shapes attached to an earlier non-floor shape ---
    children = []
    pool = list(range(2, N))
    for _ in range(min(J, len(pool))):
        children.append(pool.pop(d.integer(0, len(pool))))
    children.sort()
    partner = {}
    anchors = {}
    for ch in children:
        pa = d.integer(1, ch)
        partner[ch] = pa
        if static[ch] and static[pa]:
            static[ch] = 0
        if pa < P:
            anc_p = (d.u(-0.8, 0.8) * hx[pa], d.u(-0.8, 0.8) * hy[pa])
            if nverts[pa] == 3:
                anc_p = (anc_p[0] * 0.3, anc_p[1] * 0.3)
        else:
            rr, aa = 0.8 * radius[pa - P] * d.u(), d.u(-math.pi, math.pi)
            anc_p = (rr * math.cos(aa), rr * math.sin(aa))
        if ch < P:
            anc_c = ((0.8 if d.u() < 0.5 else -0.8) * hx[ch], 0.0)
            if nverts[ch] == 3:
                anc_c = (anc_c[0] * 0.3, 0.0)
        else:
            anc_c = (0.0, 0.0) if d.u() < 0.5 else (0.8 * radius[ch - P], 0.0)
        anchors[ch] = (anc_p, anc_c)
    # --- placement ---
    px = [0.0] * N
    py = [0.0] * N
    ang = [0.0] * N
    py[0] = -0.5
    placed = [0]

    def clear(i, x, y, skip):
        if y - brad[i] < 0.02:
            return False
        for k in placed:
            if k == 0 or k == skip:
                continue
            if math.hypot(x - px[k], y - py[k]) < brad[i] + brad[k] + 0.02:
                return False
        return True

    for i in range(1, N):
        ok = False
        if i in partner:
            pa = partner[i]
            anc_p, anc_c = anchors[i]
            cpa, spa = math.cos(ang[pa]), math.sin(ang[pa])
            wx, wy = _rot(cpa, spa, anc_p)
            wx += px[pa]
            wy += py[pa]
            for _ in range(200):
                a = d.u(-math.pi, math.pi)
                ox, oy = _rot(math.cos(a), math.sin(a), anc_c)
                x, y = wx - ox, wy - oy
                if clear(i, x, y, pa):
                    ok = True
                    break
            px[i], py[i], ang[i] = x, y, a
        else:
            for _ in range(200):
                x, y, a = d.u(-2.5, 2.5), d.u(brad[i] + 0.02, 5.0), d.u(-math.pi, math.pi)
                if clear(i, x, y, -1):
                    ok = True
                    break
            if not ok:
                top = max(py[k] + brad[k] for k in placed)
                x, y = d.u(-2.5, 2.5), top + brad[i] + 0.05
            px[i], py[i], ang[i] = x, y, a
        placed.append(i)
    # --- roles ---
    joined = {(min(c, p), max(c, p)) for c, p in partner.items()}
    role = [ROLE_NONE] * N
    cand = list(range(1, N))
    green = cand[d.integer(0, len(cand))]
    blues = [k for k in cand if k != green and (min(k, green), max(k, green)) not in joined]
    blue = blues[d.integer(0, len(blues))]
    role[green], role[blue] = ROLE_GREEN, ROLE_BLUE
    red_here = with_red if isinstance(with_red, bool) else (d.u() < float(with_red))
    if red_here:
        reds = [k for k in cand if k not in (green, blue)]
        role[reds[d.integer(0, len(reds))]] = ROLE_RED
    # --- write out ---
    o = out
    for i in range(P):
        o["poly_verts"][index, i] = np.asarray(verts[i], np.float32)
        o["poly_nverts"][index, i] = nverts[i]
    o["circle_radius"][index] = radius
    o["pos"][index, :, 0] = px
    o["pos"][index, :, 1] = py
    o["angle"][index] = ang
    o["density"][index] = density
    o["friction"][index] = friction
    o["restitution"][index] = restitution
    o["is_static"][index] = static
    o["role"][index] = role
    o["active"][index] = 1
    for j, ch in enumerate(children):
        pa = partner[ch]
        anc_p, anc_c = anchors[ch]
        o["joint_a"][index, j] = pa
        o["joint_b"][index, j] = ch
        o["joint_anchor_a"][index, j] = anc_p
        o["joint_anchor_b"][index, j] = anc_c
        o["motor_speed"][index, j] = d.u(1.0, 4.0)
        inv_i = 0.0
        for k in (pa, ch):
            if not static[k]:
                inv_i += 1.0 / (density[k] * inertia_per_density[k])
        o["motor_power"][index, j] = d.u(0.1, 0.8) / inv_i
        o["motor_binding"][index, j] = j
        o["joint_active"][index, j] = 1
    if fixed_prob > 0.0 or limit_prob > 0.0:
        # joint kinds come from a stream of their own, so that levels drawn without them do not change:
        # a fixed joint holds the relative rotation the level starts with, a limited one allows a
        # range of 0.2 .. 1 rad to either side of it
        dj = _Draws(seed ^ 0x51F1, index)
        for j, ch in enumerate(children):
            rel0 = ang[partner[ch]] - ang[ch]
            u = dj.u()
            lo, hi = dj.u(0.2, 1.0), dj.u(0.2, 1.0)
            if u < fixed_prob:
                o["joint_fixed"][index, j] = 1
                o["joint_fixed_angle"][index, j] = rel0
            elif u < fixed_prob + limit_prob:
                o["joint_limited"][index, j] = 1
                o["joint_min"][index, j] = rel0 - lo
                o["joint_max"][index, j] = rel0 + hi
    movable = [k for k in range(1, N) if not static[k]] or list(range(1, N))
    for t in range(T):
        k = movable[d.integer(0, len(movable))]
        scale = 0.3 if (k < P and nverts[k] == 3) else 0.8
        o["thr_shape"][index, t] = k
        o["thr_pos"][index, t] = (d.u(-scale, scale) * hx[k], d.u(-scale, scale) * hy[k])
        o["thr_rot"][index, t] = d.u(-math.pi, math.pi)
        o["thr_power"][index, t] = d.u(0.5, 2.0) * density[k] * area[k] * 9.81
        o["thr_binding"][index, t] = J + t
        o["thr_active"][index, t] = 1


def make_levels(size, n_levels: int, seed: int, static_prob: float = 0.0, with_red=None,
                triangle_prob: float = 0.0, fixed_prob: float = 0.0, limit_prob: float = 0.0) -> dict:
    """Draw ``n_levels`` scenes of size class ``size`` ("S", "M", "L" or a SceneDims).

    ``with_red``: True / False, or a probability; default is always for L and 1/2 otherwise.
    ``fixed_prob`` / ``limit_prob``: probability that a joint is a fixed joint / a revolute joint with
    rotation limits (the benchmark workloads use neither).
    Level ``k`` depends only on ``(seed, k)`` and the other arguments, not on ``n_levels``.
    """
    dims = SIZES[size] if isinstance(size, str) else size
    if with_red is None:
        with_red = True if dims == SIZES["L"] else 0.5
    out = empty_levels(dims, n_levels)
    for k in range(n_levels):
        _one_level(dims, seed, k, static_prob, with_red, triangle_prob, out, fixed_prob, limit_prob)
    return out


def make_actions(n_steps: int, n_envs: int, n_actions: int, seed: int) -> np.ndarray:
    """Uniform actions in [-1, 1), float32, laid out [n_steps][n_envs][n_actions]."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), 0xAC7])))
    a = rng.random((n_steps, n_envs, n_actions), dtype=np.float32)
    a *= 2.0
    a -= 1.0
    return a


def take_levels(levels: dict, idx) -> dict:
    """Sub-select levels (numpy fancy index) from a level dict."""
    return {k: np.ascontiguousarray(v[idx]) for k, v in levels.items()}


# the five benchmark workloads: size class, envs, steps, reset mode, level pool, horizon
WORKLOADS = {
    0: dict(size="S", n_envs=16, n_steps=100, auto_reset=0, n_levels=16, static_prob=0.0, max_episode_steps=0),
    1: dict(size="S", n_envs=4096, n_steps=256, auto_reset=1, n_levels=4096, static_prob=0.1, max_episode_steps=0),
    2: dict(size="M", n_envs=16384, n_steps=256, auto_reset=1, n_levels=4096, static_prob=0.1, max_episode_steps=0),
    3: dict(size="L", n_envs=16384, n_steps=512, auto_reset=2, n_levels=1024, static_prob=0.1, max_episode_steps=256),
    4: dict(size="L", n_envs=131072, n_steps=32, auto_reset=2, n_levels=1024, static_prob=0.1, max_episode_steps=256),
}


def workload_seed(config_index: int) -> int:
    return 1000 + int(config_index)


def custom_level(dims: SceneDims, polygons=(), circles=(), joints=(), thrusters=()) -> dict:
    """One hand-written level (leading dimension 1); entities not listed stay inactive.

    polygons: dicts with ``half=(hx, hy)`` or ``verts=[(x, y), ...]`` (3 or 4, CCW, centroid at the
    origin), plus optional pos, angle, vel, angvel, density, friction, restitution, static, role.
    circles: dicts with ``radius`` and the same optional keys.  Shape indices: polygons first, in the
    order given, then circles at ``dims.n_polygons + k``.
    joints: dicts with a, b, anchor_a, anchor_b and optional speed, power, binding, fixed (the relative
    rotation angle_a - angle_b a fixed joint holds), limits ((min, max) of that relative rotation).
    thrusters: dicts with shape and optional pos, rot, power, binding.
    """
    lv = empty_levels(dims, 1)
    P, J = dims.n_polygons, dims.n_joints

    def common(i, d):
        lv["pos"][0, i] = d.get("pos", (0.0, 0.0))
        lv["angle"][0, i] = d.get("angle", 0.0)
        lv["vel"][0, i] = d.get("vel", (0.0, 0.0))
        lv["angvel"][0, i] = d.get("angvel", 0.0)
        lv["density"][0, i] = d.get("density", 1.0)
        lv["friction"][0, i] = d.get("friction", 0.5)
        lv["restitution"][0, i] = d.get("restitution", 0.0)
        lv["is_static"][0, i] = int(d.get("static", 0))
        lv["role"][0, i] = int(d.get("role", ROLE_NONE))
        lv["active"][0, i] = 1

    assert len(polygons) <= P and len(circles) <= dims.n_circles
    assert len(joints) <= J and len(thrusters) <= dims.n_thrusters
    for i, d in enumerate(polygons):
        v = d["verts"] if "verts" in d else _box(*d["half"])
        lv["poly_nverts"][0, i] = len(v)
        lv["poly_verts"][0, i] = 0.0
        lv["poly_verts"][0, i, : len(v)] = np.asarray(v, np.float32)
        common(i, d)
    for k, d in enumerate(circles):
        lv["circle_radius"][0, k] = d["radius"]
        common(P + k, d)
    for j, d in enumerate(joints):
        lv["joint_a"][0, j], lv["joint_b"][0, j] = d["a"], d["b"]
        lv["joint_anchor_a"][0, j] = d.get("anchor_a", (0.0, 0.0))
        lv["joint_anchor_b"][0, j] = d.get("anchor_b", (0.0, 0.0))
        lv["motor_speed"][0, j] = d.get("speed", 0.0)
        lv["motor_power"][0, j] = d.get("power", 0.0)
        lv["motor_binding"][0, j] = d.get("binding", j)
        lv["joint_active"][0, j] = 1
        if "fixed" in d:
            lv["joint_fixed"][0, j] = 1
            lv["joint_fixed_angle"][0, j] = d["fixed"]
        if "limits" in d:
            lv["joint_limited"][0, j] = 1
            lv["joint_min"][0, j], lv["joint_max"][0, j] = d["limits"]
    for t, d in enumerate(thrusters):
        lv["thr_shape"][0, t] = d["shape"]
        lv["thr_pos"][0, t] = d.get("pos", (0.0, 0.0))
        lv["thr_rot"][0, t] = d.get("rot", 0.0)
        lv["thr_power"][0, t] = d.get("power", 0.0)
        lv["thr_binding"][0, t] = d.get("binding", J + t)
        lv["thr_active"][0, t] = 1
    return lv


def concat_levels(parts) -> dict:
    """Stack several level dicts of the same dims along the level axis."""
    parts = list(parts)
    return {k: np.concatenate([p[k] for p in parts], axis=0) for k in parts[0]}
