"""Pins of the oracle's fixed joints and joint limits (paper, "Fixed Joints", "Joint Limits",
"Impulse Accumulation and Warm Starting") against closed forms and invariants.  CPU only."""
import math

import numpy as np
import pytest

from oracle import k2d_ref
from paper_2410_23208_b200.scenes import SceneDims, custom_level

DIMS = SceneDims(3, 2, 1, 1)
DT = 1.0 / 60.0
GAMMA = 6.0


def sim_of(level, **cfg):
    return k2d_ref.RefSim(level, 1, f64=True, **cfg)


def step(sim, n=1):
    for _ in range(n):
        sim.step(np.zeros((1, 1, sim.n_actions)))


def two_free_boxes(joint, wa=1.5, wb=-0.5, angle_a=0.0, angle_b=0.0):
    # joined at both centres, so the point constraint and the angular row do not interact
    return custom_level(DIMS, polygons=[dict(half=(0.3, 0.2), pos=(0.0, 2.0), angle=angle_a, angvel=wa, density=1.0),
                                        dict(half=(0.5, 0.1), pos=(0.0, 2.0), angle=angle_b, angvel=wb, density=2.0)],
                        joints=[dict(a=0, b=1, **joint)])


def test_fixed_joint_removes_the_relative_angular_velocity_and_keeps_angular_momentum():
    sim = sim_of(two_free_boxes(dict(fixed=0.0)), gravity_y=0.0)
    ia, ib = 1 / sim.inv_inertia[0, 0], 1 / sim.inv_inertia[0, 1]
    l0 = ia * 1.5 + ib * -0.5
    step(sim)
    wa, wb = sim.angvel[0, 0], sim.angvel[0, 1]
    # j_r = (w_a - w_b) / (1/I_a + 1/I_b): both end up with the common angular velocity L / (I_a + I_b)
    assert wa == pytest.approx(l0 / (ia + ib), abs=1e-12) and wb == pytest.approx(wa, abs=1e-12)
    assert ia * wa + ib * wb == pytest.approx(l0, abs=1e-12)
    # the accumulated angular impulse is the impulse that did it
    assert sim.jacc[0, 0, 2] == pytest.approx((1.5 - -0.5) / (1 / ia + 1 / ib), rel=1e-12)


def test_revolute_joint_leaves_the_relative_angular_velocity_alone():
    sim = sim_of(two_free_boxes(dict()), gravity_y=0.0)
    step(sim)
    assert sim.angvel[0, 0] == pytest.approx(1.5, abs=1e-12) and sim.angvel[0, 1] == pytest.approx(-0.5, abs=1e-12)
    assert sim.jacc[0, 0, 2] == 0.0


def test_fixed_joint_angle_error_decays_by_gamma_dt_per_step():
    c0 = 0.25                                                   # exact in float32, like every level value below
    sim = sim_of(two_free_boxes(dict(fixed=0.0), wa=0.0, wb=0.0, angle_a=c0), gravity_y=0.0)
    errs = []
    for _ in range(20):
        step(sim)
        errs.append(sim.angle[0, 0] - sim.angle[0, 1])
    # velocity correction: w_a - w_b = -gamma C each step, so C_n = C_0 (1 - gamma dt)^n
    want = c0 * (1 - GAMMA * DT) ** np.arange(1, 21)
    assert np.allclose(errs, want, rtol=0, atol=1e-12)
    # a different gamma is a different decay
    sim = sim_of(two_free_boxes(dict(fixed=0.0), wa=0.0, wb=0.0, angle_a=c0), gravity_y=0.0, joint_gamma=3.0)
    step(sim)
    assert sim.angle[0, 0] - sim.angle[0, 1] == pytest.approx(c0 * (1 - 3.0 * DT), abs=1e-12)


def test_fixed_joint_target_angle_is_relative_rotation_a_minus_b():
    sim = sim_of(two_free_boxes(dict(fixed=0.5), wa=0.0, wb=0.0, angle_a=0.75, angle_b=0.25), gravity_y=0.0)
    step(sim, 5)
    assert sim.angle[0, 0] - sim.angle[0, 1] == pytest.approx(0.5, abs=1e-12)       # already there: nothing happens
    assert abs(sim.angvel[0, 0]) < 1e-12 and abs(sim.angvel[0, 1]) < 1e-12


def welded_arm(**joint):
    # a bar held by its end on a fixated block, sticking out sideways under gravity
    return custom_level(DIMS, polygons=[dict(half=(0.1, 0.1), pos=(0.0, 4.0), static=1),
                                        dict(half=(0.5, 0.05), pos=(0.5, 4.0), density=1.0)],
                        joints=[dict(a=0, b=1, anchor_a=(0.0, 0.0), anchor_b=(-0.5, 0.0), **joint)])


def test_welded_arm_stays_up_and_its_accumulated_impulse_carries_the_torque():
    sim = sim_of(welded_arm(fixed=0.0))
    m = 1 / sim.inv_mass[0, 1]
    step(sim, 240)
    assert abs(sim.angle[0, 1]) < 2e-2 and abs(sim.angvel[0, 1]) < 1e-3           # a revolute joint would let it swing down
    assert np.hypot(*(sim.pos[0, 1] - (0.5, 4.0))) < 2e-2
    # at rest the joint's impulses per step balance gravity: force m g dt at the anchor, moment m g dt L/2 about it
    assert sim.jacc[0, 0, 1] == pytest.approx(m * 9.81 * DT, rel=2e-2)            # the point constraint pushes b (the bar) up with its weight
    assert abs(sim.jacc[0, 0, 2]) == pytest.approx(m * 9.81 * DT * 0.5, rel=5e-2)
    free = sim_of(welded_arm())
    step(free, 60)
    assert free.angle[0, 1] < -1.0


def test_fixed_joint_is_not_warm_started_when_warm_start_is_off():
    sim = sim_of(welded_arm(fixed=0.0), warm_start=0)
    step(sim, 3)
    # with warm starting off the accumulated impulses restart from zero every step, so they stay of the order of one step's load
    w = sim_of(welded_arm(fixed=0.0))
    step(w, 3)
    assert np.isfinite(sim.jacc).all() and abs(sim.angle[0, 1]) < 5e-2
    assert not np.allclose(sim.jacc, w.jacc)


def limited_pendulum(limits=None, theta0=0.0):
    L = 0.5
    piv = (0.0, 4.0)
    kw = dict(limits=limits) if limits is not None else {}
    # the rod starts horizontal-ish to the side and falls: relative rotation angle_a - angle_b = -angle_rod
    c = (piv[0] + L * math.cos(theta0), piv[1] + L * math.sin(theta0))
    return custom_level(DIMS, polygons=[dict(half=(0.1, 0.1), pos=piv, static=1),
                                        dict(half=(L, 0.05), pos=c, angle=theta0, density=1.0)],
                        joints=[dict(a=0, b=1, anchor_a=(0.0, 0.0), anchor_b=(-L, 0.0), **kw)])


def test_joint_limit_stops_the_swing_and_does_nothing_inside_the_range():
    lim = sim_of(limited_pendulum((-0.1, 0.6)))
    free = sim_of(limited_pendulum())
    rel_l, rel_f, same = [], [], 0
    for n in range(240):
        step(lim); step(free)
        rel_l.append(lim.angle[0, 0] - lim.angle[0, 1]); rel_f.append(free.angle[0, 0] - free.angle[0, 1])
        if same == n and np.array_equal(lim.angle, free.angle) and np.array_equal(lim.angvel, free.angvel):
            same = n + 1
    assert max(rel_f) > 2.0                                     # the free rod swings far past the limit
    assert max(rel_l) < 0.6 + 0.05 and min(rel_l) > -0.1 - 0.05
    # until the limit is first crossed the two runs are identical, bit for bit
    first_out = next(i for i, r in enumerate(rel_f) if r > 0.6)
    assert same >= first_out
    assert np.all(lim.jacc[0, :, 2] == 0.0)                     # limits are never accumulated


@pytest.mark.parametrize("side", [+1, -1])
def test_beyond_a_limit_returning_motion_is_left_alone_and_outward_motion_is_turned_back(side):
    c = 0.125                                                   # how far beyond the limit
    limits = (-0.5, 0.5)
    rel0 = side * (0.5 + c)
    # returning: nothing is applied (no correction, no impulse)
    sim = sim_of(two_free_boxes(dict(limits=limits), wa=-side * 0.75, wb=0.0, angle_a=rel0), gravity_y=0.0)
    step(sim)
    assert sim.angvel[0, 0] == pytest.approx(-side * 0.75, abs=1e-15) and sim.angvel[0, 1] == 0.0
    # moving further out: the relative angular velocity becomes the correction -gamma C, shared by inertia
    sim = sim_of(two_free_boxes(dict(limits=limits), wa=side * 0.75, wb=0.0, angle_a=rel0), gravity_y=0.0)
    ia, ib = 1 / sim.inv_inertia[0, 0], 1 / sim.inv_inertia[0, 1]
    step(sim)
    wrel = sim.angvel[0, 0] - sim.angvel[0, 1]
    assert wrel == pytest.approx(-GAMMA * side * c, abs=1e-12)
    assert ia * sim.angvel[0, 0] + ib * sim.angvel[0, 1] == pytest.approx(ia * side * 0.75, abs=1e-12)
    # at rest beyond the limit: pushed back at gamma C as well
    sim = sim_of(two_free_boxes(dict(limits=limits), wa=0.0, wb=0.0, angle_a=rel0), gravity_y=0.0)
    step(sim)
    assert sim.angvel[0, 0] - sim.angvel[0, 1] == pytest.approx(-GAMMA * side * c, abs=1e-12)


def test_inside_the_limits_a_limited_joint_is_a_revolute_joint():
    a = sim_of(two_free_boxes(dict(limits=(-1.0, 1.0))), gravity_y=0.0)
    b = sim_of(two_free_boxes(dict()), gravity_y=0.0)
    step(a, 10); step(b, 10)
    assert np.array_equal(a.angle, b.angle) and np.array_equal(a.angvel, b.angvel)


def test_observation_reports_fixed_joints():
    sim = sim_of(two_free_boxes(dict(fixed=0.0)))
    obs = sim.obs()[0]
    n_shapes, jw = DIMS.n_shapes, 11 + sim.n_actions
    row = obs[n_shapes * 29: n_shapes * 29 + jw]
    assert row[0] == 1.0 and row[1] == 1.0
    assert sim_of(two_free_boxes(dict())).obs()[0][n_shapes * 29 + 1] == 0.0
