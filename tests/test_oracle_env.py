"""Pins for the oracle's environment layer: reward/done, auto-reset, hash, transcendental routines,
observation rows."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import k2d_ref
from paper_2410_23208_b200 import scenes
from paper_2410_23208_b200.scenes import ROLE_BLUE, ROLE_GREEN, ROLE_RED, SceneDims, custom_level

DIMS = SceneDims(3, 3, 1, 1)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def touching_level(gb, gr, joined=False):
    """green circle in the middle; the blue circle and/or the red box overlap it when asked to"""
    circles = [dict(radius=0.3, pos=(0.0, 5.0), role=ROLE_GREEN),
               dict(radius=0.3, pos=(0.55 if gb else 2.0, 5.0), role=ROLE_BLUE)]
    polys = [dict(half=(0.3, 0.3), pos=(-0.55 if gr else -2.0, 5.0), role=ROLE_RED)]
    joints = [dict(a=3, b=4, anchor_a=(0.275, 0.0), anchor_b=(-0.275, 0.0))] if joined else []
    return custom_level(DIMS, polygons=polys, circles=circles, joints=joints)


@pytest.mark.parametrize("gb,gr,timeout", list(itertools.product([0, 1], repeat=3)))
def test_reward_and_done_truth_table(gb, gr, timeout):
    sim = k2d_ref.RefSim(touching_level(gb, gr), 1, gravity_y=0.0, max_episode_steps=1 if timeout else 0)
    r, d = sim.step(np.zeros((1, 1, 2)))
    assert r[0, 0] == float(gb - gr)
    assert d[0, 0] == int(bool(gb or gr or timeout))


def test_touch_needs_a_colliding_pair():
    # green and blue overlap but are joined: the pair does not collide, so it never scores
    sim = k2d_ref.RefSim(touching_level(1, 0, joined=True), 1, gravity_y=0.0)
    r, d = sim.step(np.zeros((3, 1, 2)))
    assert np.all(r == 0) and np.all(d == 0)


def test_flags_repeat_without_auto_reset_and_physics_continues():
    sim = k2d_ref.RefSim(touching_level(1, 0), 1, gravity_y=0.0, auto_reset=0)
    x0 = sim.pos.copy()
    r, d = sim.step(np.zeros((2, 1, 2)))
    assert r[0, 0] == 1 and d[0, 0] == 1
    assert not np.array_equal(sim.pos, x0)            # the contact pushed the circles apart


def test_same_level_reset_restores_the_level_record():
    lv = scenes.make_levels("S", 4, 77, static_prob=0.1)
    sim = k2d_ref.RefSim(lv, 4, auto_reset=1, max_episode_steps=5)
    act = scenes.make_actions(5, 4, sim.n_actions, 1)
    r, d = sim.step(act)
    assert np.all(d[4] == 1)
    assert np.array_equal(sim.pos, lv["pos"]) and np.array_equal(sim.angle, lv["angle"])
    assert np.all(sim.vel == 0) and np.all(sim.angvel == 0) and np.all(sim.acc == 0) and np.all(sim.jacc == 0)
    assert np.all(sim.step_count == 0) and np.all(sim.episode_count >= 1)
    # determinism: the second episode replays the first when the actions repeat
    first = k2d_ref.RefSim(lv, 4, auto_reset=0)
    first.step(act[:3])
    sim.step(act[:3])
    keep = d[:4].sum(0) == 0                           # envs that did not reset earlier than the horizon
    assert keep.any() and np.array_equal(sim.pos[keep], first.pos[keep])


def test_mix64_published_vectors():
    want = [int(l, 16) for l in open(os.path.join(GOLDEN, "splitmix64_seed0.txt")) if l.startswith("0x")]
    got = [k2d_ref.mix64(k * 0x9E3779B97F4A7C15) for k in (1, 2, 3)]
    assert got == want


def test_pool_reset_draws_levels_by_hash():
    lv = scenes.make_levels("S", 16, 5)
    seed, off = 1234, 100
    sim = k2d_ref.RefSim(lv, 8, auto_reset=2, max_episode_steps=2, seed=seed, env_offset=off)
    sim.step(np.zeros((6, 8, sim.n_actions)))
    assert np.all(sim.episode_count == 3)
    M = 2 ** 64 - 1
    want = [k2d_ref.mix64((seed + (off + e + 1) * 0x9E3779B97F4A7C15 + 3 * 0xD1B54A32D192ED03) & M) % 16 for e in range(8)]
    assert list(sim.level_id) == want
    assert len(set(want)) > 2
    # independent of how the envs are sharded: env 5 of this sim is env 1 of a sim that starts at 104
    part = k2d_ref.RefSim(lv, 2, auto_reset=2, max_episode_steps=2, seed=seed, env_offset=off + 4)
    part.reset(np.array([4 % 16, 5 % 16]))
    part.step(np.zeros((6, 2, sim.n_actions)))
    assert list(part.level_id) == want[4:6]


def test_non_finite_state_ends_the_episode():
    lv = scenes.make_levels("S", 2, 9)
    sim = k2d_ref.RefSim(lv, 2, auto_reset=0)
    sim.vel[0, 2, 0] = np.inf
    r, d = sim.step(np.zeros((3, 2, sim.n_actions)))
    assert np.all(d[:, 0] == 1) and np.all(r[:, 0] == 0) and sim.status[0] == 1
    assert sim.status[1] == 0 and sim.counters[0] == 1
    again = k2d_ref.RefSim(lv, 2, auto_reset=1)
    again.vel[0, 2, 0] = np.nan
    r, d = again.step(np.zeros((2, 2, sim.n_actions)))
    assert d[0, 0] == 1 and r[0, 0] == 0 and again.status[0] == 0 and again.episode_count[0] == 1
    assert np.all(np.isfinite(again.pos[0])) and again.step_count[0] == 1


# ---------------------------------------------------------------- sincos / tanh
def test_sincos_accuracy_and_quadrants():
    rng = np.random.default_rng(0)
    th = np.concatenate([rng.uniform(-40, 40, 200000), rng.uniform(-1000, 1000, 20000),
                         np.arange(-16, 17) * (math.pi / 4), [0.0, -0.0, 1e-8, 1e5]]).astype(np.float32)
    c, s = k2d_ref.sincos(th)
    t64 = th.astype(np.float64)
    assert np.max(np.abs(c - np.cos(t64))) <= 4e-7
    assert np.max(np.abs(s - np.sin(t64))) <= 4e-7
    assert np.max(np.abs(c.astype(np.float64) ** 2 + s.astype(np.float64) ** 2 - 1)) < 1e-6
    c0, s0 = k2d_ref.sincos(np.float32(0.0))
    assert c0[0] == 1.0 and s0[0] == 0.0
    cn, sn = k2d_ref.sincos(np.float32(np.nan))
    assert np.isnan(cn[0]) and np.isnan(sn[0])
    cb, sb = k2d_ref.sincos(np.float32(3e7))
    assert np.isnan(cb[0])                                # outside the supported range: flagged, not wrong


def test_tanh_accuracy():
    rng = np.random.default_rng(1)
    x = np.concatenate([rng.uniform(-12, 12, 200000), rng.uniform(-0.01, 0.01, 20000),
                        [0.0, 1e-6, -1e-6, 9.99, 10.0, 50.0, -50.0, np.inf, -np.inf]]).astype(np.float32)
    y = k2d_ref.tanh(x)
    assert np.max(np.abs(y - np.tanh(x.astype(np.float64)))) <= 4e-7
    assert np.all(np.abs(y) <= 1.0) and np.all(np.sign(y) == np.sign(x))
    assert np.isnan(k2d_ref.tanh(np.float32(np.nan))[0])


# ---------------------------------------------------------------- observation
def test_observation_rows_against_a_direct_construction():
    lv = scenes.make_levels("M", 3, 31, static_prob=0.2, triangle_prob=0.3)
    lv["thr_active"][1, 1] = 0
    lv["joint_active"][2, 0] = 0
    sim = k2d_ref.RefSim(lv, 3, f64=True)
    act = scenes.make_actions(20, 3, sim.n_actions, 3)
    sim.step(act)
    o = sim.obs()
    d = scenes.SIZES["M"]
    N, P, J, T, A = d.n_shapes, d.n_polygons, d.n_joints, d.n_thrusters, d.n_actions
    assert o.shape == (3, N * 29 + 2 * J * (11 + A) + 6 * T) == (3, 333)
    for e in range(3):
        for i in range(N):
            row = o[e, i * 29:(i + 1) * 29]
            assert np.allclose(row[0:2], sim.pos[e, i]) and np.allclose(row[2:4], sim.vel[e, i])
            assert row[4] == sim.inv_mass[e, i] and row[5] == sim.inv_inertia[e, i]
            assert row[6] == lv["density"][e, i]
            assert row[7] == pytest.approx(math.tanh(sim.angvel[e, i] / 10), abs=1e-7)
            onehot = np.zeros(4)
            onehot[lv["role"][e, i]] = 1
            assert np.array_equal(row[8:12], onehot)
            assert row[12] == pytest.approx(math.sin(sim.angle[e, i]), abs=1e-12)
            assert row[13] == pytest.approx(math.cos(sim.angle[e, i]), abs=1e-12)
            assert row[14] == lv["friction"][e, i] and row[15] == lv["restitution"][e, i]
            if i < P:
                n = lv["poly_nverts"][e, i]
                assert tuple(row[16:19]) == (1, 0, 0)
                assert np.array_equal(row[19:19 + 2 * n], lv["poly_verts"][e, i, :n].ravel())
                assert np.all(row[19 + 2 * n:27] == 0)
                assert tuple(row[27:29]) == ((1, 0) if n == 3 else (0, 1))
            else:
                assert tuple(row[16:18]) == (0, 1) and row[18] == lv["circle_radius"][e, i - P]
                assert np.all(row[19:] == 0)
        jw = 11 + A
        for j in range(J):
            for dirn in range(2):
                row = o[e, N * 29 + (2 * j + dirn) * jw: N * 29 + (2 * j + dirn + 1) * jw]
                if not lv["joint_active"][e, j]:
                    assert np.all(row == 0)
                    continue
                a, b = lv["joint_a"][e, j], lv["joint_b"][e, j]
                frm, to = (b, a) if dirn else (a, b)
                af, at = (lv["joint_anchor_b"][e, j], lv["joint_anchor_a"][e, j]) if dirn else \
                         (lv["joint_anchor_a"][e, j], lv["joint_anchor_b"][e, j])
                assert tuple(row[0:2]) == (1, 0)
                assert np.array_equal(row[2:4], af) and np.array_equal(row[4:6], at)
                assert row[6] == lv["motor_power"][e, j] and row[7] == lv["motor_speed"][e, j] and row[8] == 0
                onehot = np.zeros(A)
                onehot[lv["motor_binding"][e, j]] = 1
                assert np.array_equal(row[9:9 + A], onehot)
                rel = sim.angle[e, to] - sim.angle[e, frm]
                assert row[9 + A] == pytest.approx(math.sin(rel), abs=1e-12)
                assert row[10 + A] == pytest.approx(math.cos(rel), abs=1e-12)
        for t in range(T):
            row = o[e, N * 29 + 2 * J * jw + 6 * t: N * 29 + 2 * J * jw + 6 * (t + 1)]
            if not lv["thr_active"][e, t]:
                assert np.all(row == 0)
                continue
            i = lv["thr_shape"][e, t]
            assert row[0] == 1 and np.array_equal(row[1:3], lv["thr_pos"][e, t]) and row[3] == lv["thr_power"][e, t]
            face = sim.angle[e, i] + float(lv["thr_rot"][e, t])
            assert row[4] == pytest.approx(math.sin(face), abs=1e-12)
            assert row[5] == pytest.approx(math.cos(face), abs=1e-12)


def test_f32_step_tracks_f64_step():
    # the parity build and the pin build run the same statements: over a short horizon they agree closely
    lv = scenes.make_levels("M", 16, 8)
    a32 = k2d_ref.RefSim(lv, 16)
    a64 = k2d_ref.RefSim(lv, 16, f64=True)
    act = scenes.make_actions(4, 16, a32.n_actions, 8)
    a32.step(act)
    a64.step(act)
    assert np.max(np.abs(a32.pos - a64.pos)) < 1e-4 and np.max(np.abs(a32.vel - a64.vel)) < 1e-2


def test_threads_do_not_change_results():
    lv = scenes.make_levels("S", 64, 12, static_prob=0.1)
    a = k2d_ref.RefSim(lv, 64, auto_reset=1, max_episode_steps=20)
    b = k2d_ref.RefSim(lv, 64, auto_reset=1, max_episode_steps=20)
    act = scenes.make_actions(50, 64, a.n_actions, 2)
    ra, da = a.step(act, n_threads=1)
    rb, db = b.step(act, n_threads=5)
    assert np.array_equal(a.pos, b.pos) and np.array_equal(ra, rb) and np.array_equal(da, db)
    assert np.array_equal(a.counters, b.counters)


# ---------------------------------------------------------------- multi-discrete actions, dense reward
def _motor_and_thruster_level():
    return custom_level(DIMS, polygons=[dict(half=(0.2, 0.2), pos=(0.0, 3.0), static=1),
                                        dict(half=(0.4, 0.1), pos=(0.0, 3.0), density=1.0),
                                        dict(half=(0.3, 0.3), pos=(2.0, 3.0), density=1.0)],
                        joints=[dict(a=0, b=1, speed=2.0, power=0.05)],
                        thrusters=[dict(shape=2, power=3.0, rot=0.5)])


@pytest.mark.parametrize("codes,continuous", [((0, 0), (0.0, 0.0)), ((1, 1), (1.0, 1.0)), ((2, 0), (-1.0, 0.0)), ((2, 1), (-1.0, 1.0))])
def test_multi_discrete_actions_are_off_or_full_power(codes, continuous):
    # paper, "Action Space": inactive, or at maximum power, motors forwards or backwards
    lv = _motor_and_thruster_level()
    d = k2d_ref.RefSim(lv, 1, discrete_actions=1)
    c = k2d_ref.RefSim(lv, 1)
    for _ in range(5):
        d.step(np.array(codes, np.float32).reshape(1, 1, 2))
        c.step(np.array(continuous, np.float32).reshape(1, 1, 2))
    for k in ("pos", "angle", "vel", "angvel"):
        assert np.array_equal(getattr(d, k), getattr(c, k)), k
    if codes != (0, 0):
        idle = k2d_ref.RefSim(lv, 1)
        for _ in range(5):
            idle.step(np.zeros((1, 1, 2), np.float32))
        assert not np.array_equal(idle.vel, d.vel) or not np.array_equal(idle.angvel, d.angvel)


def test_dense_reward_is_kappa_times_the_decrease_of_the_green_blue_distance():
    # a green circle flies at constant velocity towards a fixated blue one, no gravity: d_t - d_{t+1} = v dt
    kappa, v = 0.25, 1.5
    lv = custom_level(DIMS, circles=[dict(radius=0.25, pos=(-3.0, 2.0), vel=(v, 0.0), role=ROLE_GREEN),
                                     dict(radius=0.25, pos=(1.0, 2.0), static=1, role=ROLE_BLUE)])
    sim = k2d_ref.RefSim(lv, 1, f64=True, gravity_y=0.0, dense_kappa=kappa)
    r, d = sim.step(np.zeros((10, 1, sim.n_actions)))
    assert np.allclose(r[:, 0], kappa * v / 60.0, rtol=0, atol=1e-12) and not d.any()
    # moving away gives the negative; without kappa nothing
    lv["vel"][0, 3] = (-v, 0.0)
    sim = k2d_ref.RefSim(lv, 1, f64=True, gravity_y=0.0, dense_kappa=kappa)
    r, _ = sim.step(np.zeros((3, 1, sim.n_actions)))
    assert np.allclose(r[:, 0], -kappa * v / 60.0, rtol=0, atol=1e-12)
    sim = k2d_ref.RefSim(lv, 1, f64=True, gravity_y=0.0)
    r, _ = sim.step(np.zeros((3, 1, sim.n_actions)))
    assert np.all(r == 0.0)


def test_dense_reward_adds_to_the_touch_reward_and_needs_both_shapes():
    kappa = 0.5
    lv = touching_level(True, False)
    plain = k2d_ref.RefSim(lv, 1, f64=True)
    dense = k2d_ref.RefSim(lv, 1, f64=True, dense_kappa=kappa)
    g = int(np.argmax(lv["role"][0] == ROLE_GREEN)); b = int(np.argmax(lv["role"][0] == ROLE_BLUE))
    d0 = np.hypot(*(dense.pos[0, b] - dense.pos[0, g]))
    rp, _ = plain.step(np.zeros((1, 1, plain.n_actions)))
    rd, dd = dense.step(np.zeros((1, 1, dense.n_actions)))
    d1 = np.hypot(*(dense.pos[0, b] - dense.pos[0, g]))
    assert rp[0, 0] == 1.0 and dd[0, 0] == 1
    assert rd[0, 0] == pytest.approx(1.0 + kappa * (d0 - d1), abs=1e-12)
    lv["role"][0][lv["role"][0] == ROLE_BLUE] = 0
    sim = k2d_ref.RefSim(lv, 1, f64=True, dense_kappa=kappa)
    r, _ = sim.step(np.zeros((2, 1, sim.n_actions)))
    assert np.all(r == 0.0)


def test_oracle_trajectories_have_not_changed():
    # digests written by tests/golden/make_oracle_trajectories.py from the oracle alone
    import importlib.util
    here = os.path.dirname(os.path.abspath(__file__))
    spec = importlib.util.spec_from_file_location("make_oracle_trajectories", os.path.join(here, "golden", "make_oracle_trajectories.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = [ln.strip() for ln in open(os.path.join(here, "golden", "oracle_trajectories.txt")) if ln.strip() and not ln.startswith("#")]
    assert mod.lines() == stored


def test_frame_skip_holds_every_action_row():
    # paper, hyperparameter table: frame skip 2.  Holding a row for k steps equals repeating it k times.
    lv = _motor_and_thruster_level()
    rng = np.random.default_rng(3)
    rows = rng.uniform(-1, 1, (4, 1, 2)).astype(np.float32)
    held = k2d_ref.RefSim(lv, 1, frame_skip=3)
    rep = k2d_ref.RefSim(lv, 1)
    rh, dh = held.step(rows[:3], n_steps=8)               # 3 + 3 + 2 steps
    rr, dr = rep.step(np.repeat(rows[:3], 3, axis=0)[:8])
    assert np.array_equal(rh, rr) and np.array_equal(dh, dr) and rh.shape == (8, 1)
    for k in ("pos", "angle", "vel", "angvel"):
        assert np.array_equal(getattr(held, k), getattr(rep, k)), k
