"""Pins for parts of the oracle that the closed-form tests of single rows do not reach: the order in which
rows are visited inside a solver iteration, the positional correction of a joint, the reference-face
tolerance and the incident-face tie-break of the polygon-polygon manifold, the guards on motors and
thrusters whose shapes are absent, which green shape the dense reward measures from, and the reward of a
step that goes non-finite.  Every expected value comes from mechanics worked by hand in the test (momentum
sharing of point masses, distances), never from the oracle."""
import math

import numpy as np
import pytest

from oracle import k2d_ref
from paper_2410_23208_b200.scenes import ROLE_BLUE, ROLE_GREEN, ROLE_RED, SceneDims, custom_level

DT = 1.0 / 60.0


def sim_of(level, **cfg):
    return k2d_ref.RefSim(level, 1, f64=True, **cfg)


def merge(m1, v1, m2, v2):
    """two point masses leave a perfectly inelastic exchange with the velocity of their centre of mass"""
    return (m1 * v1 + m2 * v2) / (m1 + m2)


# ---------------------------------------------------------------- order of the rows inside one iteration
ROW = SceneDims(1, 4, 2, 1)


def test_one_iteration_visits_joints_in_index_order_then_contacts():
    # Four discs on a line.  Joints (c0, c1) and (c1, c2) are anchored at the disc centres, so each joint row is
    # the exchange of two point masses (the lever arms are zero); c3 touches c2 and runs into it.  With one
    # solver iteration the outcome depends on the order of the three rows; Algorithm 1 takes the joints first,
    # in index order, then the contacts.
    rho = (1.0, 2.5, 0.7, 1.8)
    v = [3.0, 0.0, -1.0, -4.0]
    r = 0.3
    xs = (0.0, 1.0, 2.0, 2.0 + 2 * r - 0.002)
    lv = custom_level(ROW, circles=[dict(radius=r, pos=(xs[k], 5.0), vel=(v[k], 0.0), density=rho[k], friction=0.0, restitution=0.0)
                                    for k in range(4)],
                      joints=[dict(a=1, b=2), dict(a=2, b=3)])
    sim = sim_of(lv, gravity_y=0.0, solver_iters=1, joint_alpha=0.0, joint_beta=0.0, contact_beta=0.0)
    m = [1.0 / sim.inv_mass[0, 1 + k] for k in range(4)]
    sim.step(np.zeros((1, 1, sim.n_actions)))
    v[0] = v[1] = merge(m[0], v[0], m[1], v[1])          # joint 0
    v[1] = v[2] = merge(m[1], v[1], m[2], v[2])          # joint 1
    assert v[3] < v[2]                                   # still approaching: the contact row acts
    v[2] = v[3] = merge(m[2], v[2], m[3], v[3])          # contact (c2, c3), no bounce
    assert np.allclose(sim.vel[0, 1:5, 0], v, rtol=0, atol=1e-12)
    assert np.all(sim.vel[0, 1:5, 1] == 0.0) and np.all(sim.angvel[0, 1:5] == 0.0)
    # the other orders give other numbers, so the comparison above really tells them apart
    w = [3.0, 0.0, -1.0, -4.0]
    w[1] = w[2] = merge(m[1], w[1], m[2], w[2])
    w[0] = w[1] = merge(m[0], w[0], m[1], w[1])
    assert abs(w[0] - v[0]) > 1e-3


def test_one_iteration_visits_contacts_in_pair_order():
    # three touching discs in a row, the outer two closing in: pair (c0, c1) is solved before pair (c1, c2)
    rho = (1.0, 0.6, 2.0)
    v = [2.0, 0.0, -3.0]
    r = 0.25
    d = 2 * r - 0.002
    lv = custom_level(ROW, circles=[dict(radius=r, pos=(k * d, 5.0), vel=(v[k], 0.0), density=rho[k], friction=0.0, restitution=0.0)
                                    for k in range(3)])
    sim = sim_of(lv, gravity_y=0.0, solver_iters=1, contact_beta=0.0)
    m = [1.0 / sim.inv_mass[0, 1 + k] for k in range(3)]
    sim.step(np.zeros((1, 1, sim.n_actions)))
    v[0] = v[1] = merge(m[0], v[0], m[1], v[1])
    v[1] = v[2] = merge(m[1], v[1], m[2], v[2])
    assert np.allclose(sim.vel[0, 1:4, 0], v, rtol=0, atol=1e-12)
    w = [2.0, 0.0, -3.0]
    w[1] = w[2] = merge(m[1], w[1], m[2], w[2])
    w[0] = w[1] = merge(m[0], w[0], m[1], w[1])
    assert abs(w[0] - v[0]) > 1e-3


# ---------------------------------------------------------------- joint positional correction
def test_joint_positional_correction_closes_beta_of_the_gap_split_by_inverse_mass():
    # paper, "Revolute Joints": velocity and positional corrections.  Two free discs at rest, joined at their
    # centres, which are 0.3 m apart: with the velocity correction off nothing moves but the positional
    # correction, which closes joint_beta of the gap, the lighter body moving more.
    dims = SceneDims(1, 2, 1, 1)
    gap = np.array([0.3, -0.4])
    lv = custom_level(dims, circles=[dict(radius=0.1, pos=(1.0, 5.0), density=1.0),
                                     dict(radius=0.1, pos=(1.0 + gap[0], 5.0 + gap[1]), density=3.0)],
                      joints=[dict(a=1, b=2)])
    beta = 0.25
    sim = sim_of(lv, gravity_y=0.0, joint_alpha=0.0, joint_beta=beta)
    ia, ib = sim.inv_mass[0, 1], sim.inv_mass[0, 2]
    xa0, xb0 = sim.pos[0, 1].copy(), sim.pos[0, 2].copy()
    gap = xb0 - xa0                                      # level data is stored in fp32
    sim.step(np.zeros((1, 1, sim.n_actions)))
    assert np.all(sim.vel[0] == 0.0)
    assert np.allclose(sim.pos[0, 1] - xa0, beta * gap * ia / (ia + ib), rtol=0, atol=1e-12)
    assert np.allclose(sim.pos[0, 2] - xb0, -beta * gap * ib / (ia + ib), rtol=0, atol=1e-12)
    assert np.allclose(sim.pos[0, 2] - sim.pos[0, 1], (1 - beta) * gap, rtol=0, atol=1e-12)
    # against a fixated partner the free body closes the whole share
    lv["is_static"][0, 1] = 1
    sim = sim_of(lv, gravity_y=0.0, joint_alpha=0.0, joint_beta=beta)
    sim.step(np.zeros((1, 1, sim.n_actions)))
    assert np.all(sim.pos[0, 1] == xa0) and np.allclose(sim.pos[0, 2] - xb0, -beta * gap, rtol=0, atol=1e-12)


# ---------------------------------------------------------------- polygon-polygon: reference face tolerance, incident tie
def _separations(a, b):
    """largest over a's faces of the smallest signed distance of b's corners to the face (brute force, double)"""
    a, b = np.asarray(a, float), np.asarray(b, float)
    best = -np.inf
    for k in range(len(a)):
        e = a[(k + 1) % len(a)] - a[k]
        n = np.array([e[1], -e[0]]) / np.hypot(*e)
        best = max(best, min((b - a[k]) @ n))
    return best


def _box(cx, cy, hx, hy, ang=0.0):
    c, s = math.cos(ang), math.sin(ang)
    return [(cx + c * x - s * y, cy + s * x + c * y) for x, y in ((-hx, -hy), (hx, -hy), (hx, hy), (-hx, hy))]


@pytest.mark.parametrize("phi,on_b", [(0.4e-3, False), (2.5e-3, True)])
def test_reference_face_stays_on_a_until_b_is_better_by_more_than_the_tolerance(phi, on_b):
    # a wide box b lies, turned by a tiny angle, on a narrower box a: b's lower face separates the two a little
    # better than a's upper face, by about (half width of b - half width of a) * phi.  Within face_tol the
    # reference face stays on a (normal exactly +y); beyond it moves to b (normal = minus b's lower face normal).
    tol = 1e-3
    a = _box(0.0, 0.0, 1.0, 1.0)
    b = _box(0.0, 1.0 + 0.5 - 0.01, 2.0, 0.5, phi)
    sa, sb = _separations(a, b), _separations(b, a)
    assert sa < 0 and sb < 0 and (sb - sa > tol) == on_b and sb > sa
    m = k2d_ref.manifold_pp(a, b, face_tol=tol, f64=True)
    assert m[0]["active"] or m[1]["active"]
    for k in range(2):
        if on_b:
            assert np.allclose(m[k]["n"], (-math.sin(phi), math.cos(phi)), rtol=0, atol=1e-12)
        else:
            assert m[k]["n"][0] == 0.0 and m[k]["n"][1] == 1.0
    # with a larger tolerance the second case stays on a as well
    m = k2d_ref.manifold_pp(a, b, face_tol=0.01, f64=True)
    assert m[0]["n"][0] == 0.0 and m[0]["n"][1] == 1.0


def test_incident_face_tie_goes_to_the_lower_index():
    # a square standing on its corner (first vertex = the lowest corner) dips into a box below it: its two lower
    # faces are equally anti-parallel to the reference normal; the first of them (corner 0 -> corner 1) is the
    # incident face, so slot 0 is the dipping corner and slot 1 the clipped far end
    h, depth = 0.5, 0.03
    tip = 1.0 - depth
    b = [(0.0, tip), (h, tip + h), (0.0, tip + 2 * h), (-h, tip + h)]
    a = _box(0.0, 0.0, 1.0, 1.0)
    m = k2d_ref.manifold_pp(a, b, f64=True)
    assert m[0]["active"] and not m[1]["active"]
    assert np.allclose(m[0]["p"], (0.0, tip), atol=1e-12) and m[0]["pen"] == pytest.approx(depth, abs=1e-12)
    assert np.allclose(m[1]["p"], (h, tip + h), atol=1e-12) and m[1]["pen"] == pytest.approx(depth - h, abs=1e-12)


# ---------------------------------------------------------------- guards on absent shapes
def test_motor_and_thruster_on_an_absent_shape_do_nothing():
    dims = SceneDims(2, 1, 1, 1)
    lv = custom_level(dims, polygons=[dict(half=(0.3, 0.2), pos=(0.0, 5.0))],
                      joints=[dict(a=0, b=1, anchor_a=(0.0, 0.0), anchor_b=(0.0, 0.0), speed=3.0, power=0.5)],
                      thrusters=[dict(shape=2, pos=(0.1, 0.0), rot=0.3, power=4.0)])
    assert lv["active"][0, 1] == 0 and lv["active"][0, 2] == 0           # polygon 1 and the circle are absent
    sim = sim_of(lv, gravity_y=0.0)
    sim.step(np.ones((3, 1, sim.n_actions)))
    assert np.all(sim.vel[0] == 0.0) and np.all(sim.angvel[0] == 0.0)
    assert np.array_equal(sim.pos[0], lv["pos"][0].astype(np.float64))
    # the same motor with its second shape present does act
    lv2 = custom_level(dims, polygons=[dict(half=(0.3, 0.2), pos=(0.0, 5.0)), dict(half=(0.2, 0.2), pos=(0.0, 5.0))],
                       joints=[dict(a=0, b=1, speed=3.0, power=0.5)])
    sim2 = sim_of(lv2, gravity_y=0.0)
    sim2.step(np.ones((1, 1, sim2.n_actions)))
    assert sim2.angvel[0, 0] > 0.0 > sim2.angvel[0, 1]


def test_motor_between_two_fixated_shapes_is_inert():
    dims = SceneDims(2, 1, 1, 1)
    lv = custom_level(dims, polygons=[dict(half=(0.3, 0.2), pos=(0.0, 5.0), static=1), dict(half=(0.2, 0.2), pos=(0.0, 5.0), static=1)],
                      joints=[dict(a=0, b=1, speed=3.0, power=0.5)])
    sim = sim_of(lv)
    sim.step(np.ones((2, 1, sim.n_actions)))
    assert np.all(sim.angvel[0] == 0.0) and np.all(sim.jacc[0] == 0.0)


# ---------------------------------------------------------------- dense reward: which green shape
def test_dense_reward_measures_from_the_first_green_and_the_first_blue_shape():
    dims = SceneDims(1, 4, 1, 1)
    kappa, v = 0.5, 1.25
    # greens at indices 1 and 3, blues at 2 and 4; only the first green moves (towards the first blue)
    lv = custom_level(dims, circles=[dict(radius=0.1, pos=(-2.0, 5.0), vel=(v, 0.0), role=ROLE_GREEN),
                                     dict(radius=0.1, pos=(2.0, 5.0), static=1, role=ROLE_BLUE),
                                     dict(radius=0.1, pos=(-2.0, 8.0), static=1, role=ROLE_GREEN),
                                     dict(radius=0.1, pos=(2.0, 9.0), vel=(0.0, 3.0), role=ROLE_BLUE)])
    sim = sim_of(lv, gravity_y=0.0, dense_kappa=kappa)
    r, d = sim.step(np.zeros((4, 1, sim.n_actions)))
    assert np.allclose(r[:, 0], kappa * v * DT, rtol=0, atol=1e-12) and not d.any()


# ---------------------------------------------------------------- a step that goes non-finite scores nothing
def test_a_non_finite_step_reports_zero_reward_even_when_green_touches_blue():
    dims = SceneDims(1, 3, 1, 1)
    lv = custom_level(dims, circles=[dict(radius=0.3, pos=(0.0, 5.0), role=ROLE_GREEN),
                                     dict(radius=0.3, pos=(0.55, 5.0), role=ROLE_BLUE),
                                     dict(radius=0.3, pos=(9.0, 9.0))])
    ok = k2d_ref.RefSim(lv, 1, gravity_y=0.0)
    r, d = ok.step(np.zeros((1, 1, ok.n_actions)))
    assert r[0, 0] == 1.0 and d[0, 0] == 1
    bad = k2d_ref.RefSim(lv, 1, gravity_y=0.0, dense_kappa=0.3)
    bad.vel[0, 3, 0] = np.inf                            # the bystander leaves the number range
    r, d = bad.step(np.zeros((1, 1, bad.n_actions)))
    assert r[0, 0] == 0.0 and d[0, 0] == 1 and bad.status[0] == 1
