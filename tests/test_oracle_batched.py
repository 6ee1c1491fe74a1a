"""Pins for the oracle's batched contact solve (paper, "Parallelised Computation and Batched Impulse Resolution": the
manifold slots are solved in batches, side by side within a batch, batches one after the other, the active manifolds
spread over as many batches as possible).  Expected values are worked by hand from point-mass mechanics."""
import numpy as np
import pytest

from oracle import k2d_ref
from paper_2410_23208_b200 import scenes
from paper_2410_23208_b200.scenes import SceneDims, custom_level

ROW = SceneDims(1, 4, 1, 1)          # 4 polygon-circle + 6 circle-circle manifold slots = 10
SPEEDS = (2.0, 0.5, -1.0, -3.0)
RHO = (1.0, 0.6, 2.0, 1.5)


def four_discs():
    r = 0.25
    d = 2 * r - 0.002
    return custom_level(ROW, circles=[dict(radius=r, pos=(k * d, 5.0), vel=(SPEEDS[k], 0.0), density=RHO[k], friction=0.0, restitution=0.0)
                                      for k in range(4)])


def exchange(m, v, a, b, ref):
    """impulse that takes the approach speed of (a, b), measured in the velocities `ref`, to zero, applied to v"""
    lam = -(ref[b] - ref[a]) / (1.0 / m[a] + 1.0 / m[b])
    lam = max(lam, 0.0)
    v[a] -= lam / m[a]
    v[b] += lam / m[b]


@pytest.mark.parametrize("batch,order", [(0, "sequential"), (1, "sequential"), (3, "sequential"), (5, "two batches"), (10, "one batch"), (16, "one batch")])
def test_rows_of_a_batch_see_the_same_velocities_and_batches_follow_one_another(batch, order):
    # four touching discs in a row, all closing in: rows 0, 1, 2 = pairs (c0,c1), (c1,c2), (c2,c3); one iteration.
    # 10 slots: batches of 3 or fewer slots give 4 or more batches, one row each: the sequential sweep.  Batches of 5
    # give 2 batches: rows 0 and 2 together, then row 1.  Batches of 10 or more give one batch: all three rows side by side.
    sim = k2d_ref.RefSim(four_discs(), 1, f64=True, gravity_y=0.0, solver_iters=1, contact_beta=0.0, solver_batch=batch)
    m = [1.0 / sim.inv_mass[0, 1 + k] for k in range(4)]
    sim.step(np.zeros((1, 1, sim.n_actions)))
    v = list(SPEEDS)
    if order == "sequential":
        for a in (0, 1, 2):
            exchange(m, v, a, a + 1, v)
    elif order == "two batches":
        snap = list(v)
        exchange(m, v, 0, 1, snap); exchange(m, v, 2, 3, snap)
        exchange(m, v, 1, 2, list(v))
    else:
        snap = list(v)
        for a in (0, 1, 2):
            exchange(m, v, a, a + 1, snap)
    assert np.allclose(sim.vel[0, 1:5, 0], v, rtol=0, atol=1e-12), (sim.vel[0, 1:5, 0], v)
    # momentum is conserved whatever the batching
    assert sum(m[k] * sim.vel[0, 1 + k, 0] for k in range(4)) == pytest.approx(sum(m[k] * SPEEDS[k] for k in range(4)), abs=1e-12)


def test_the_three_orders_really_differ():
    out = []
    for batch in (0, 5, 10):
        sim = k2d_ref.RefSim(four_discs(), 1, f64=True, gravity_y=0.0, solver_iters=1, contact_beta=0.0, solver_batch=batch)
        sim.step(np.zeros((1, 1, sim.n_actions)))
        out.append(sim.vel[0, 1:5, 0].copy())
    assert np.abs(out[0] - out[1]).max() > 1e-3 and np.abs(out[0] - out[2]).max() > 1e-3 and np.abs(out[1] - out[2]).max() > 1e-3


@pytest.mark.parametrize("size,seed", [("S", 21), ("M", 22), ("L", 23)])
def test_batches_of_one_slot_are_the_sequential_sweep_bit_for_bit(size, seed):
    n = 24
    lv = scenes.make_levels(size, n, seed, static_prob=0.1, triangle_prob=0.2)
    lv["pos"][:4, 1:, 0] *= 0.2                          # a few crowded scenes too
    act = scenes.make_actions(60, n, lv["joint_a"].shape[1] + lv["thr_shape"].shape[1], seed)
    a = k2d_ref.RefSim(lv, n)
    b = k2d_ref.RefSim(lv, n, solver_batch=1)
    ra, da = a.step(act)
    rb, db = b.step(act)
    assert np.array_equal(ra, rb) and np.array_equal(da, db)
    for k in ("pos", "angle", "vel", "angvel", "acc", "jacc"):
        assert np.array_equal(getattr(a, k).view(np.uint32), getattr(b, k).view(np.uint32)), k


def test_default_batches_of_16_change_nothing_while_rows_are_no_more_than_batches():
    # L scenes have 186 manifold slots, 12 batches of 16: a scene with at most 12 active manifolds has one row per batch
    n = 32
    lv = scenes.make_levels("L", n, 31, static_prob=0.1)
    act = scenes.make_actions(1, n, 8, 31)
    a = k2d_ref.RefSim(lv, n)
    b = k2d_ref.RefSim(lv, n, solver_batch=16)
    few = np.ones(n, bool)
    for s in range(40):
        a.step(act); b.step(act)
        few &= ((a.manifold[:, :, 5] > 0).sum(1) <= 12) & ((b.manifold[:, :, 5] > 0).sum(1) <= 12)
    assert few.sum() >= 3 and (~few).sum() >= 3
    assert np.array_equal(a.pos[few].view(np.uint32), b.pos[few].view(np.uint32))
    assert not np.array_equal(a.pos[~few], b.pos[~few])


def test_resting_box_carries_its_weight_under_the_default_batches():
    dims = SceneDims(12, 4, 6, 2)
    lv = custom_level(dims, polygons=[dict(half=(5.0, 0.5), pos=(0.0, -0.5), static=1), dict(half=(0.4, 0.3), pos=(0.0, 0.3), density=1.5)])
    sim = k2d_ref.RefSim(lv, 1, f64=True, solver_batch=16)
    sim.step(np.zeros((120, 1, sim.n_actions)))
    m = 1.0 / sim.inv_mass[0, 1]
    assert np.abs(sim.vel[0, 1]).max() < 1e-6 and abs(sim.angvel[0, 1]) < 1e-6
    assert sim.acc[0, 0, 0] + sim.acc[0, 1, 0] == pytest.approx(m * 9.81 / 60.0, rel=1e-6)


def test_free_bodies_keep_their_momentum_when_all_rows_are_solved_side_by_side():
    dims = SceneDims(3, 3, 1, 1)
    rng = np.random.default_rng(5)
    polys = [dict(half=(0.3, 0.2), pos=(rng.uniform(-0.4, 0.4), 5.0 + 0.3 * k), vel=tuple(rng.uniform(-2, 2, 2)), angvel=rng.uniform(-2, 2), density=1.0 + k,
                  friction=0.4, restitution=0.2) for k in range(3)]
    circs = [dict(radius=0.25, pos=(rng.uniform(-0.4, 0.4), 4.8 - 0.3 * k), vel=tuple(rng.uniform(-2, 2, 2)), density=2.0, friction=0.4) for k in range(3)]
    lv = custom_level(dims, polygons=polys, circles=circs)
    sim = k2d_ref.RefSim(lv, 1, f64=True, gravity_y=0.0, contact_beta=0.0, solver_batch=10 ** 6)
    m, inertia = 1.0 / sim.inv_mass[0], 1.0 / sim.inv_inertia[0]

    def momenta():
        p = (m[:, None] * sim.vel[0]).sum(0)
        x, v = sim.pos[0], sim.vel[0]
        return p, (inertia * sim.angvel[0] + m * (x[:, 0] * v[:, 1] - x[:, 1] * v[:, 0])).sum()
    p0, l0 = momenta()
    sim.step(np.zeros((1, 1, sim.n_actions)))
    assert (sim.manifold[0, :, 5] > 0).sum() >= 4
    p1, l1 = momenta()
    assert np.allclose(p0, p1, atol=1e-10) and l1 == pytest.approx(l0, abs=1e-10)
