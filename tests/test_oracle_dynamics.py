"""Pins for the oracle's dynamics: closed forms and invariants that do not come from the oracle."""
import math

import numpy as np
import pytest

from oracle import k2d_ref
from paper_2410_23208_b200 import scenes
from paper_2410_23208_b200.scenes import SceneDims, custom_level

DIMS = SceneDims(3, 2, 1, 1)
DT = 1.0 / 60.0
G = -9.81
FLOOR = dict(half=(5.0, 0.5), pos=(0.0, -0.5), static=1)


def sim_of(level, f64=True, **cfg):
    return k2d_ref.RefSim(level, 1, f64=f64, **cfg)


def zero_actions(sim, n):
    return np.zeros((n, 1, sim.n_actions))


# ---------------------------------------------------------------- gravity + Euler
@pytest.mark.parametrize("f64", [True, False])
def test_free_fall_closed_form(f64):
    v0, y0, n = 1.25, 50.0, 100
    lv = custom_level(DIMS, circles=[dict(radius=0.3, pos=(0.5, y0), vel=(0.75, v0))])
    sim = sim_of(lv, f64=f64)
    sim.step(zero_actions(sim, n))
    vy = v0 + n * G * DT
    y = y0 + n * v0 * DT + G * DT * DT * n * (n + 1) / 2
    tol = 1e-10 if f64 else 2e-4
    assert sim.vel[0, 3, 1] == pytest.approx(vy, abs=tol)
    assert sim.pos[0, 3, 1] == pytest.approx(y, abs=tol)
    assert sim.pos[0, 3, 0] == pytest.approx(0.5 + n * 0.75 * DT, abs=tol)
    assert sim.vel[0, 3, 0] == pytest.approx(0.75, abs=tol)


def test_static_shapes_do_not_fall():
    lv = custom_level(DIMS, polygons=[FLOOR], circles=[dict(radius=0.3, pos=(0.0, 9.0), static=1, vel=(1.0, 1.0))])
    sim = sim_of(lv)
    sim.step(zero_actions(sim, 10))
    assert np.all(sim.pos[0, 3] == (0.0, 9.0)) and np.all(sim.vel[0, 3] == 0.0)
    assert sim.inv_mass[0, 3] == 0.0 and sim.inv_inertia[0, 3] == 0.0


# ---------------------------------------------------------------- mass properties
def test_mass_properties_textbook():
    lv = custom_level(DIMS, polygons=[dict(half=(0.4, 0.7), density=1.5),
                                      dict(verts=[(-0.6, -0.2), (0.6, -0.2), (0.0, 0.4)], density=2.0)],
                      circles=[dict(radius=0.3, density=0.8)])
    sim = sim_of(lv)
    m = 1.5 * 4 * 0.4 * 0.7
    assert 1 / sim.inv_mass[0, 0] == pytest.approx(m, rel=1e-6)
    assert 1 / sim.inv_inertia[0, 0] == pytest.approx(m * (0.4 ** 2 + 0.7 ** 2) / 3, rel=1e-6)
    mc = 0.8 * math.pi * 0.09
    assert 1 / sim.inv_mass[0, 3] == pytest.approx(mc, rel=1e-6)
    assert 1 / sim.inv_inertia[0, 3] == pytest.approx(mc * 0.09 / 2, rel=1e-6)
    # isosceles triangle, base b = 1.2, height h = 0.6: I_centroid = m (b^2/24 + h^2/18)
    mt = 2.0 * 0.5 * 1.2 * 0.6
    assert 1 / sim.inv_mass[0, 1] == pytest.approx(mt, rel=1e-6)
    assert 1 / sim.inv_inertia[0, 1] == pytest.approx(mt * (1.2 ** 2 / 24 + 0.6 ** 2 / 18), rel=1e-6)


# ---------------------------------------------------------------- normal impulse, restitution
def two_circles(e_a, e_b, rho_a=1.0, rho_b=1.0, va=2.0, vb=-2.0, pen=0.004, r=0.5):
    d = 2 * r - pen
    return custom_level(DIMS, circles=[
        dict(radius=r, pos=(-d / 2, 3.0), vel=(va, 0.0), density=rho_a, restitution=e_a, friction=0.0),
        dict(radius=r, pos=(d / 2, 3.0), vel=(vb, 0.0), density=rho_b, restitution=e_b, friction=0.0)])


@pytest.mark.parametrize("e_a,e_b,rho_a,rho_b", [(0.8, 0.5, 1.0, 1.0), (0.3, 0.9, 2.0, 0.5), (0.0, 0.7, 1.0, 3.0)])
def test_two_circle_collision_restitution_and_momentum(e_a, e_b, rho_a, rho_b):
    sim = sim_of(two_circles(e_a, e_b, rho_a, rho_b), gravity_y=0.0)
    ma, mb = 1 / sim.inv_mass[0, 3], 1 / sim.inv_mass[0, 4]
    p0 = ma * 2.0 + mb * -2.0
    sim.step(zero_actions(sim, 1))
    va, vb = sim.vel[0, 3, 0], sim.vel[0, 4, 0]
    e = float(np.float32(min(e_a, e_b)))            # level data is stored in fp32
    # paper: the new relative velocity at the contact is -e times the old one (penetration below the
    # slop, so no velocity correction is added)
    assert vb - va == pytest.approx(-e * (-2.0 - 2.0), abs=1e-12)
    assert ma * va + mb * vb == pytest.approx(p0, abs=1e-12)
    assert sim.vel[0, 3, 1] == 0.0 and sim.angvel[0, 3] == 0.0


def test_elastic_equal_masses_swap_velocities():
    sim = sim_of(two_circles(1.0, 1.0, va=3.0, vb=-1.0), gravity_y=0.0)
    sim.step(zero_actions(sim, 1))
    assert sim.vel[0, 3, 0] == pytest.approx(-1.0, abs=1e-12) and sim.vel[0, 4, 0] == pytest.approx(3.0, abs=1e-12)


def test_inelastic_common_velocity():
    sim = sim_of(two_circles(0.0, 0.0, rho_a=1.0, rho_b=3.0, va=3.0, vb=-1.0), gravity_y=0.0)
    sim.step(zero_actions(sim, 1))
    assert sim.vel[0, 3, 0] == pytest.approx((1 * 3.0 + 3 * -1.0) / 4, abs=1e-12)
    assert sim.vel[0, 4, 0] == pytest.approx(sim.vel[0, 3, 0], abs=1e-12)


def test_velocity_correction_adds_alpha_times_penetration():
    # penetration 0.055 = slop + 0.05: the separating speed gains contact_alpha * 0.05
    sim = sim_of(two_circles(0.5, 0.5, pen=0.055), gravity_y=0.0)
    sim.step(zero_actions(sim, 1))
    assert sim.vel[0, 4, 0] - sim.vel[0, 3, 0] == pytest.approx(0.5 * 4.0 + 6.0 * 0.05, abs=1e-6)


def test_slow_approach_does_not_bounce():
    sim = sim_of(two_circles(0.5, 0.5, va=0.4, vb=-0.4), gravity_y=0.0)
    sim.step(zero_actions(sim, 1))
    assert sim.vel[0, 4, 0] - sim.vel[0, 3, 0] == pytest.approx(0.0, abs=1e-12)


def test_positional_correction_moves_apart_by_beta():
    # unequal masses: the split is by inverse mass, the total is beta * (pen - slop)
    lv = two_circles(0.0, 0.0, rho_a=1.0, rho_b=3.0, va=0.0, vb=0.0, pen=0.105)
    sim = sim_of(lv, gravity_y=0.0, contact_alpha=0.0)
    x0 = sim.pos[0, :, 0].copy()
    sim.step(zero_actions(sim, 1))
    da, db = x0[3] - sim.pos[0, 3, 0], sim.pos[0, 4, 0] - x0[4]
    assert da + db == pytest.approx(0.1 * 0.1, abs=1e-7)
    assert da / db == pytest.approx(3.0, rel=1e-9)


# ---------------------------------------------------------------- resting contact, warm start
def box_on_floor(**kw):
    d = dict(half=(0.5, 0.4), pos=(0.3, 0.4 - 0.002), friction=0.6, restitution=0.4, density=1.3)
    d.update(kw)
    return custom_level(DIMS, polygons=[dict(FLOOR, friction=0.3), d])


@pytest.mark.parametrize("f64", [True, False])
def test_box_rests_and_carries_its_weight(f64):
    sim = sim_of(box_on_floor(), f64=f64)
    sim.step(zero_actions(sim, 120))
    tol = 1e-9 if f64 else 2e-4
    assert np.abs(sim.vel[0, 1]).max() < tol and abs(sim.angvel[0, 1]) < tol
    slots = sim.manifold[0, 0:2]                     # pair (floor, box) owns slots 0 and 1
    assert np.all(slots[:, 5] == 1.0)
    assert np.all(slots[:, 4] > 0) and np.all(slots[:, 4] <= 0.005 + 1e-4)
    m = 1 / sim.inv_mass[0, 1]
    assert sim.acc[0, 0, 0] + sim.acc[0, 1, 0] == pytest.approx(m * -G * DT, rel=1e-6 if f64 else 1e-4)
    assert np.all(sim.acc[0, 0:2, 0] > 0)
    assert np.all(sim.acc[0, 2:] == 0)


def test_accumulators_are_wiped_when_contact_ends():
    sim = sim_of(box_on_floor())
    sim.step(zero_actions(sim, 30))
    assert sim.acc[0, 0, 0] > 0
    sim.pos[0, 1, 1] += 1.0                           # lift the box clear of the floor
    sim.step(zero_actions(sim, 1))
    assert np.all(sim.acc[0] == 0.0)


def test_without_restitution_threshold_a_resting_box_keeps_bouncing():
    # documents why the bounce needs a speed threshold: with the literal -e v_r target every solver
    # pass re-injects e times the gravity step, so the contact never settles as well
    lv = box_on_floor()
    lv["restitution"][0, 0] = 0.4                       # e = min(e_floor, e_box) = 0.4
    calm = sim_of(lv)
    jumpy = sim_of(lv, restitution_threshold=0.0)
    calm.step(zero_actions(calm, 120))
    jumpy.step(zero_actions(jumpy, 120))
    assert abs(calm.vel[0, 1, 1]) < 1e-9
    assert abs(jumpy.vel[0, 1, 1]) > 1e-3 or jumpy.pos[0, 1, 1] > calm.pos[0, 1, 1] + 1e-4


def test_stack_needs_warm_start_or_iterations():
    # three boxes stacked: with warm starting the stack carries its weight; the bottom contact holds 3 m g dt
    lv = custom_level(DIMS, polygons=[FLOOR, dict(half=(0.5, 0.25), pos=(0.0, 0.248)),
                                      dict(half=(0.45, 0.25), pos=(0.0, 0.746))])
    sim = sim_of(lv)
    sim.step(zero_actions(sim, 240))
    m1, m2 = 1 / sim.inv_mass[0, 1], 1 / sim.inv_mass[0, 2]
    bottom = sim.acc[0, 0, 0] + sim.acc[0, 1, 0]       # pair (0,1)
    top = sim.acc[0, 4, 0] + sim.acc[0, 5, 0]          # pair (1,2) is the third polygon pair
    assert bottom == pytest.approx((m1 + m2) * -G * DT, rel=1e-4)
    assert top == pytest.approx(m2 * -G * DT, rel=1e-4)
    assert np.abs(sim.vel[0, 1:3]).max() < 1e-6


# ---------------------------------------------------------------- friction
def test_sliding_block_coulomb_deceleration():
    mu_f, mu_b = 0.3, 0.4
    lv = box_on_floor(friction=mu_b, restitution=0.0, half=(1.0, 0.1), pos=(0.0, 0.1 - 0.002))
    lv["friction"][0, 0] = mu_f
    sim = sim_of(lv)
    sim.step(zero_actions(sim, 60))                    # settle
    v0 = 3.0
    sim.vel[0, 1, 0] = v0
    mu = math.sqrt(float(np.float32(mu_f)) ** 2 + float(np.float32(mu_b)) ** 2)
    n = 20
    sim.step(zero_actions(sim, n))
    assert sim.vel[0, 1, 0] == pytest.approx(v0 + n * mu * G * DT, rel=2e-3)
    # Coulomb bound on every slot
    assert np.all(np.abs(sim.acc[0, 0:2, 1]) <= mu * sim.acc[0, 0:2, 0] + 1e-9)
    sim.step(zero_actions(sim, 200))
    assert abs(sim.vel[0, 1, 0]) < 1e-6                # comes to rest, does not reverse


def test_circle_ends_up_rolling_without_slipping():
    lv = custom_level(DIMS, polygons=[dict(FLOOR, friction=0.9)],
                      circles=[dict(radius=0.3, pos=(-2.0, 0.298), vel=(2.0, 0.0), friction=0.9)])
    sim = sim_of(lv)
    sim.step(zero_actions(sim, 120))
    v, w = sim.vel[0, 3, 0], sim.angvel[0, 3]
    lever = sim.pos[0, 3, 1]                            # the contact point lies on the floor face, y = 0
    assert 0.29 < lever < 0.3
    assert v > 0.5 and v + w * lever == pytest.approx(0.0, abs=1e-6)
    # sliding friction on a disc: v_final = 2/3 v0 (angular momentum about the contact point)
    assert v == pytest.approx(2.0 * 2 / 3, rel=2e-2)


def test_frictionless_contact_transfers_no_tangential_momentum():
    lv = custom_level(DIMS, polygons=[dict(FLOOR, friction=0.0)],
                      circles=[dict(radius=0.3, pos=(-2.0, 0.298), vel=(2.0, 0.0), friction=0.0)])
    sim = sim_of(lv)
    sim.step(zero_actions(sim, 60))
    assert sim.vel[0, 3, 0] == pytest.approx(2.0, abs=1e-9) and abs(sim.angvel[0, 3]) < 1e-12


# ---------------------------------------------------------------- revolute joint
def pendulum(theta0):
    L = 0.5
    piv = (0.0, 4.0)
    rod_c = (piv[0] + L * math.sin(theta0), piv[1] - L * math.cos(theta0))
    return custom_level(DIMS, polygons=[dict(half=(0.1, 0.1), pos=piv, static=1),
                                        dict(half=(0.05, L), pos=rod_c, angle=theta0, density=1.0)],
                        joints=[dict(a=0, b=1, anchor_a=(0.0, 0.0), anchor_b=(0.0, L))])


def test_pendulum_period_and_energy():
    theta0, L = 0.15, 0.5
    sim = sim_of(pendulum(theta0))
    m, I = 1 / sim.inv_mass[0, 1], 1 / sim.inv_inertia[0, 1]
    period = 2 * math.pi * math.sqrt((I + m * L * L) / (m * -G * L))

    def energy():
        v, w, y = sim.vel[0, 1], sim.angvel[0, 1], sim.pos[0, 1, 1]
        return 0.5 * m * (v @ v) + 0.5 * I * w * w + m * -G * y
    e0 = energy()
    swing = m * -G * L * (1 - math.cos(theta0))
    angles, gaps, energies = [], [], []
    for _ in range(360):
        sim.step(zero_actions(sim, 1))
        th = sim.angle[0, 1]
        angles.append(th)
        tip = sim.pos[0, 1] + np.array([-math.sin(th) * L, math.cos(th) * L]) * 1.0
        gaps.append(np.hypot(*(tip - (0.0, 4.0))))
        energies.append(energy())
    assert max(gaps) < 1e-3                              # the joined points stay together
    assert max(abs(e - e0) for e in energies[:120]) < 0.05 * swing
    # period from downward zero crossings of the angle
    a = np.array(angles)
    idx = [i for i in range(1, len(a)) if a[i - 1] > 0 >= a[i]]
    times = [(i - 1 + a[i - 1] / (a[i - 1] - a[i])) * DT for i in idx]
    measured = np.mean(np.diff(times))
    assert measured == pytest.approx(period, rel=0.02)


def test_joint_disables_collision_of_the_joined_pair():
    lv = pendulum(0.0)
    sim = sim_of(lv)
    assert sim.collide[0, 0] == 0                       # pair (0, 1)
    lv2 = custom_level(DIMS, polygons=[dict(half=(0.1, 0.1), pos=(0.0, 4.0), static=1),
                                       dict(half=(0.05, 0.5), pos=(0.0, 3.5))])
    sim2 = sim_of(lv2)
    assert sim2.collide[0, 0] == 1


def test_joint_between_two_free_bodies_conserves_momentum():
    lv = custom_level(DIMS, polygons=[dict(half=(0.3, 0.1), pos=(0.0, 5.0), vel=(1.0, 0.5), angvel=2.0),
                                      dict(half=(0.3, 0.1), pos=(0.5, 5.0), vel=(-0.5, 0.2), angvel=-1.0, density=2.0)],
                      joints=[dict(a=0, b=1, anchor_a=(0.25, 0.0), anchor_b=(-0.25, 0.0))])
    sim = sim_of(lv, gravity_y=0.0, joint_beta=0.0)
    m = 1 / sim.inv_mass[0, :2]
    I = 1 / sim.inv_inertia[0, :2]

    def momenta():
        p = (m[:, None] * sim.vel[0, :2]).sum(0)
        x, v = sim.pos[0, :2], sim.vel[0, :2]
        ang = (I * sim.angvel[0, :2] + m * (x[:, 0] * v[:, 1] - x[:, 1] * v[:, 0])).sum()
        return p, ang
    p0, l0 = momenta()
    sim.step(zero_actions(sim, 50))
    p1, l1 = momenta()
    # linear momentum exactly; angular momentum up to (anchor gap) x (joint impulse)
    assert np.allclose(p0, p1, atol=1e-12) and l1 == pytest.approx(l0, abs=1e-5)
    # and the anchors have (nearly) the same velocity
    th = sim.angle[0, :2]
    ra = np.array([math.cos(th[0]) * 0.25, math.sin(th[0]) * 0.25])
    rb = -np.array([math.cos(th[1]) * 0.25, math.sin(th[1]) * 0.25])
    gap = (sim.pos[0, 1] + rb) - (sim.pos[0, 0] + ra)
    assert np.hypot(*gap) < 1e-3


# ---------------------------------------------------------------- motor, thruster
def test_motor_follows_the_tanh_recurrence():
    p, s, rho, A = float(np.float32(0.02)), 3.0, 1.0, 0.7
    lv = custom_level(DIMS, polygons=[dict(half=(0.1, 0.1), pos=(0.0, 4.0), static=1)],
                      circles=[dict(radius=0.4, pos=(0.0, 4.0))],
                      joints=[dict(a=0, b=3, speed=s, power=p)])
    sim = sim_of(lv, gravity_y=0.0, motor_rho=rho)
    inv_i = sim.inv_inertia[0, 3]
    act = np.zeros((1, 1, 2))
    act[0, 0, 0] = A
    w = 0.0
    for _ in range(200):
        sim.step(act)
        w = w + inv_i * p * math.tanh(((0.0 - w) - s * A) * rho)
        assert sim.angvel[0, 3] == pytest.approx(w, abs=1e-12)
    assert w == pytest.approx(-s * A, abs=1e-3)         # fixed point: w_a - w_b = s A
    assert np.all(sim.pos[0, 3] == (0.0, 4.0))
    # actions beyond [-1, 1] are clipped
    big = act * 10
    sim2 = sim_of(lv, gravity_y=0.0)
    sim3 = sim_of(lv, gravity_y=0.0)
    sim2.step(big)
    sim3.step(np.sign(big))
    assert sim2.angvel[0, 3] == sim3.angvel[0, 3]


def test_thruster_closed_form():
    power, A, phi = 2.0, 0.6, 0.4
    lv = custom_level(DIMS, polygons=[dict(half=(0.3, 0.2), pos=(0.0, 5.0), angle=0.3)],
                      thrusters=[dict(shape=0, pos=(0.0, 0.0), rot=phi, power=power)])
    sim = sim_of(lv, gravity_y=0.0)
    m = 1 / sim.inv_mass[0, 0]
    act = np.zeros((25, 1, 2))
    act[:, 0, 1] = A
    sim.step(act)
    d = np.array([math.cos(0.3 + phi), math.sin(0.3 + phi)])
    assert np.allclose(sim.vel[0, 0], 25 * power * A * DT / m * d, atol=1e-12)
    assert sim.angvel[0, 0] == 0.0


def test_thruster_off_centre_torque_and_clipping():
    power, r = 2.0, (0.25, -0.1)
    lv = custom_level(DIMS, polygons=[dict(half=(0.3, 0.2), pos=(0.0, 5.0))],
                      thrusters=[dict(shape=0, pos=r, rot=math.pi / 2, power=power)])
    sim = sim_of(lv, gravity_y=0.0)
    I = 1 / sim.inv_inertia[0, 0]
    act = np.zeros((1, 1, 2))
    act[0, 0, 1] = 2.5                                  # clipped to 1
    sim.step(act)
    assert sim.angvel[0, 0] == pytest.approx((r[0] * power - r[1] * 0.0) * DT / I, rel=1e-6)
    sim2 = sim_of(lv, gravity_y=0.0)
    act[0, 0, 1] = -0.8                                 # negative thrust is no thrust
    sim2.step(act)
    assert np.all(sim2.vel[0, 0] == 0.0) and sim2.angvel[0, 0] == 0.0


# ---------------------------------------------------------------- invariants on crowded scenes
def _free_soup(seed):
    """no floor, no gravity: a few overlapping movable shapes"""
    rng = np.random.default_rng(seed)
    polys = [dict(half=tuple(rng.uniform(0.2, 0.6, 2)), pos=tuple(rng.uniform(-1, 1, 2) + (0, 5)),
                  angle=rng.uniform(-3, 3), vel=tuple(rng.uniform(-2, 2, 2)), angvel=rng.uniform(-3, 3),
                  density=rng.uniform(0.5, 2), friction=rng.uniform(0, 1), restitution=rng.uniform(0, 0.5))
             for _ in range(3)]
    circs = [dict(radius=rng.uniform(0.2, 0.5), pos=tuple(rng.uniform(-1, 1, 2) + (0, 5)),
                  vel=tuple(rng.uniform(-2, 2, 2)), angvel=rng.uniform(-3, 3), density=rng.uniform(0.5, 2),
                  friction=rng.uniform(0, 1), restitution=rng.uniform(0, 0.5)) for _ in range(2)]
    return custom_level(DIMS, polygons=polys, circles=circs)


@pytest.mark.parametrize("seed", range(6))
def test_momentum_conserved_without_external_forces(seed):
    sim = sim_of(_free_soup(seed), gravity_y=0.0, contact_beta=0.0, joint_beta=0.0)
    m, I = 1 / sim.inv_mass[0], 1 / sim.inv_inertia[0]

    def momenta():
        x, v = sim.pos[0], sim.vel[0]
        return (m[:, None] * v).sum(0), (I * sim.angvel[0] + m * (x[:, 0] * v[:, 1] - x[:, 1] * v[:, 0])).sum()
    p0, l0 = momenta()
    act = np.random.default_rng(seed).uniform(-1, 1, (40, 1, 2))
    act[:, :, 1] = 0.0                                  # thruster is an external force: keep it off
    total = 0
    for s in range(40):
        sim.step(act[s:s + 1])
        total += int(sim.manifold[0, :, 5].sum())
        p1, l1 = momenta()
        assert np.allclose(p0, p1, atol=1e-11) and l1 == pytest.approx(l0, abs=1e-10)
    assert total > 10                                   # contacts did happen


@pytest.mark.parametrize("size,seed", [("S", 1), ("M", 2), ("L", 3)])
def test_accumulated_impulse_bounds_on_generated_scenes(size, seed):
    lv = scenes.make_levels(size, 8, seed, static_prob=0.1)
    sim = k2d_ref.RefSim(lv, 8, f64=True)
    act = scenes.make_actions(60, 8, sim.n_actions, seed)
    for s in range(60):
        sim.step(act[s:s + 1])
        fr = lv["friction"][sim.level_id].astype(np.float64)
        for p in range(sim.n_pairs):
            a, b, slot = sim.pair_a[p], sim.pair_b[p], sim.pair_slot[p]
            mu = np.sqrt(fr[:, a] ** 2 + fr[:, b] ** 2)
            for k in range(2 if b < lv["poly_nverts"].shape[1] else 1):
                an, at = sim.acc[:, slot + k, 0], sim.acc[:, slot + k, 1]
                assert np.all(an >= 0) and np.all(np.abs(at) <= mu * an + 1e-12)
                assert np.all((an == 0) | (sim.manifold[:, slot + k, 5] == 1))   # only active slots hold impulse
    assert sim.counters[2] > 0 and sim.status.sum() == 0


@pytest.mark.parametrize("size,seed", [("S", 4), ("M", 5), ("L", 6)])
def test_box_test_in_front_of_the_narrowphase_changes_nothing(size, seed):
    lv = scenes.make_levels(size, 32, seed, static_prob=0.1)
    a = k2d_ref.RefSim(lv, 32, broadphase=1)
    b = k2d_ref.RefSim(lv, 32, broadphase=0)
    act = scenes.make_actions(100, 32, a.n_actions, seed)
    ra, da = a.step(act)
    rb, db = b.step(act)
    for k in ("pos", "angle", "vel", "angvel", "acc", "jacc"):
        assert np.array_equal(getattr(a, k), getattr(b, k)), k
    assert np.array_equal(ra, rb) and np.array_equal(da, db)


def test_inactive_pairs_leave_the_state_untouched():
    # two shapes far apart, no gravity: one step changes nothing but position by v dt
    lv = custom_level(DIMS, polygons=[dict(half=(0.3, 0.3), pos=(-2.0, 5.0), vel=(0.1, 0.0))],
                      circles=[dict(radius=0.3, pos=(2.0, 5.0), vel=(-0.1, 0.0))])
    sim = sim_of(lv, gravity_y=0.0)
    sim.step(zero_actions(sim, 1))
    v = float(np.float32(0.1))
    assert sim.vel[0, 0, 0] == v and sim.vel[0, 3, 0] == -v and np.all(sim.acc == 0)
    assert sim.pos[0, 0, 0] == pytest.approx(-2.0 + v * DT, abs=1e-15)
