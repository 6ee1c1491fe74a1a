"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest

from oracle import k2d_ref
from paper_2410_23208_b200 import k2d, scenes
from tests import parity
from tests.parity import POS_TOL_1, TOL_16, VEL_TOL_1

pytestmark = pytest.mark.gpu


def _check_tolerances(err, after_steps):
    if after_steps <= 1:
        assert max(err["pos"], err["angle"]) <= POS_TOL_1 and max(err["vel"], err["angvel"]) <= VEL_TOL_1, err
    else:
        assert max(err["pos"], err["angle"], err["vel"], err["angvel"]) <= TOL_16, err
    for k in parity.META_KEYS:
        assert err[k] == 0.0, err


def test_sincos_tanh_bit_equal_to_the_oracle():
    import torch
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.uniform(-50, 50, 100000), rng.uniform(-0.01, 0.01, 5000), rng.uniform(-2000, 2000, 20000),
                        [0.0, -0.0, 10.0, -10.0, 1e5, np.inf, -np.inf, 3e7]]).astype(np.float32)
    c, s, t = k2d.eval_sincos_tanh(torch.from_numpy(x).cuda())
    rc, rs = k2d_ref.sincos(x)
    rt = k2d_ref.tanh(x)
    for got, want in ((c, rc), (s, rs), (t, rt)):
        assert np.array_equal(got.cpu().numpy().view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("size,n_envs,seed", [("S", 16, 1000), ("M", 48, 1002), ("L", 80, 1003)])
def test_step_parity_1_16_and_100_steps(size, n_envs, seed):
    lv = scenes.make_levels(size, n_envs, seed, static_prob=0.1)
    env, ref = parity.make_pair(lv, n_envs, max_fused_steps=128)
    act = scenes.make_actions(100, n_envs, env.n_actions, seed)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[:1])
    err, exact = parity.errors(env, ref)
    _check_tolerances(err, 1)
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[1:16])
    err, exact16 = parity.errors(env, ref)
    _check_tolerances(err, 16)
    assert np.array_equal(r, rr) and np.array_equal(d, dr)          # reward / done bit-exact over 16 steps
    (r, d), (rr, dr) = parity.step_both(env, ref, act[16:])
    err, exact100 = parity.errors(env, ref)
    _check_tolerances(err, 100)
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    # the arithmetic contract makes the two bit-identical, which is what keeps the flags exact
    assert exact and exact16 and exact100
    assert parity.counters_match(env, ref)


@pytest.mark.parametrize("size,n_envs,lanes", [("L", 72, 0), ("S", 40, 0), ("L", 24, 8)])
@pytest.mark.parametrize("warm_start,solver_iters", [(0, 8), (1, 0), (1, 1), (0, 4), (1, 16), (0, 0)])
def test_warm_start_off_and_other_iteration_counts(size, n_envs, lanes, warm_start, solver_iters):
    # paper, "Impulse Accumulation and Warm Starting" (on by default, can be off) and the number of solver steps
    # as a tunable trade-off; a third of the joints fixed or limited so that their rows take part
    lv = scenes.make_levels(size, n_envs, 11, static_prob=0.1, triangle_prob=0.2, fixed_prob=0.2, limit_prob=0.2)
    env, ref = parity.make_pair(lv, n_envs, warm_start=warm_start, solver_iters=solver_iters, lanes_per_scene=lanes,
                                auto_reset=2, max_episode_steps=25, seed=6)
    act = scenes.make_actions(45, n_envs, env.n_actions, 11)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[:1])
    err, exact = parity.errors(env, ref)
    _check_tolerances(err, 1)
    assert exact, err
    (r, d), (rr, dr) = parity.step_both(env, ref, act[1:], chunk=11)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    assert parity.counters_match(env, ref)


OTHER_CONSTANTS = (
    dict(dt=1.0 / 120.0, gravity_y=-5.0, contact_alpha=3.5, contact_beta=0.2, slop=0.01, restitution_threshold=0.5, face_tol=5e-3,
         aabb_margin=0.05, joint_alpha=4.0, joint_beta=0.2, joint_gamma=2.0, motor_rho=0.7),
    dict(dt=1.0 / 30.0, gravity_y=3.0, contact_alpha=0.0, contact_beta=0.0, slop=0.0, restitution_threshold=0.0, face_tol=0.0,
         aabb_margin=0.002, joint_alpha=0.0, joint_beta=0.0, joint_gamma=0.0, motor_rho=2.0),
)


@pytest.mark.parametrize("size,n_envs", [("L", 72), ("S", 40)])
@pytest.mark.parametrize("which", [0, 1])
def test_other_engine_constants(size, n_envs, which):
    # every constant the paper leaves open is a config field; none of them may be baked into the kernels.  The second
    # set switches all corrections, the slop, the restitution threshold and the face tolerance off (the literal text)
    # and turns gravity upside down
    lv = scenes.make_levels(size, n_envs, 12, static_prob=0.1, triangle_prob=0.2, fixed_prob=0.2, limit_prob=0.2)
    env, ref = parity.make_pair(lv, n_envs, **OTHER_CONSTANTS[which])
    act = scenes.make_actions(40, n_envs, env.n_actions, 12)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=20)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    assert parity.counters_match(env, ref)
    same = k2d_ref.RefSim(lv, n_envs)
    same.step(act)
    assert not np.array_equal(same.pos, ref.pos)                     # the constants did change the trajectories


@pytest.mark.parametrize("size,n_envs,lanes", [("L", 96, 16), ("M", 64, 32), ("S", 64, 8)])
def test_box_test_counters_match_an_oracle_that_runs_the_same_test(size, n_envs, lanes):
    # with the bounding-box test on in the oracle too, the counts of pairs that passed it (by kind) must agree
    lv = scenes.make_levels(size, n_envs, 13, static_prob=0.1, triangle_prob=0.2)
    env, ref = parity.make_pair(lv, n_envs, broadphase=1, lanes_per_scene=lanes)
    act = scenes.make_actions(50, n_envs, env.n_actions, 13)
    parity.step_both(env, ref, act, chunk=25)
    assert np.array_equal(env.status(), ref.counters) and ref.counters[4:7].min() > 0
    err, exact = parity.errors(env, ref)
    assert exact, err


def test_more_action_channels_than_lanes():
    # 16 action channels, 8 lanes per scene: the action row is loaded in two passes; bindings use the upper channels
    n_envs = 24
    lv = scenes.make_levels("L", n_envs, 14, static_prob=0.1)
    rng = np.random.default_rng(14)
    lv["motor_binding"][:] = rng.integers(0, 16, lv["motor_binding"].shape)
    lv["thr_binding"][:] = rng.integers(8, 16, lv["thr_binding"].shape)
    env, ref = parity.make_pair(lv, n_envs, lanes_per_scene=8, n_actions=16)
    assert env.n_actions == 16 and ref.n_actions == 16
    act = scenes.make_actions(30, n_envs, 16, 14)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=10)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    assert np.array_equal(env.obs().cpu().numpy().view(np.uint32), ref.obs().view(np.uint32))


@pytest.mark.parametrize("lanes", [8, 16, 32])
def test_lanes_per_scene_does_not_change_results(lanes):
    lv = scenes.make_levels("L", 40, 7, static_prob=0.1, triangle_prob=0.2)
    env, ref = parity.make_pair(lv, 40, lanes_per_scene=lanes)
    act = scenes.make_actions(48, 40, env.n_actions, 7)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=16)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)


def test_fusing_steps_does_not_change_results():
    import torch
    lv = scenes.make_levels("M", 32, 3, static_prob=0.1)
    a = k2d.Env(lv, 32)
    b = k2d.Env(lv, 32)
    act = torch.from_numpy(scenes.make_actions(32, 32, a.n_actions, 3)).cuda()
    ra, da = a.step(act)
    rb, db = zip(*[b.step(act[s:s + 1]) for s in range(32)])
    sa, sb = a.get_state(), b.get_state()
    for k in sa:
        assert np.array_equal(sa[k].view(np.uint32) if sa[k].dtype == np.float32 else sa[k],
                              sb[k].view(np.uint32) if sb[k].dtype == np.float32 else sb[k]), k
    assert torch.equal(ra, torch.cat(rb)) and torch.equal(da, torch.cat(db))


def test_checkpoint_resume_is_bit_identical():
    import torch
    lv = scenes.make_levels("L", 24, 5, static_prob=0.1)
    act = torch.from_numpy(scenes.make_actions(32, 24, 8, 5)).cuda()
    a = k2d.Env(lv, 24, auto_reset=1, max_episode_steps=20)
    a.step(act[:16])
    saved = a.get_state()
    a.step(act[16:])
    b = k2d.Env(lv, 24, auto_reset=1, max_episode_steps=20)
    b.set_state(saved)
    again = b.get_state()
    for k in saved:
        assert np.array_equal(saved[k], again[k], equal_nan=True), k
    b.step(act[16:])
    sa, sb = a.get_state(), b.get_state()
    for k in sa:
        assert np.array_equal(sa[k], sb[k], equal_nan=True), k


@pytest.mark.parametrize("mode,horizon", [(1, 12), (2, 9)])
def test_auto_reset_modes_match_the_oracle(mode, horizon):
    lv = scenes.make_levels("S", 32, 21, static_prob=0.1)
    env, ref = parity.make_pair(lv, 64, auto_reset=mode, max_episode_steps=horizon, seed=99, env_offset=1000)
    act = scenes.make_actions(60, 64, env.n_actions, 21)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=20)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr) and d.sum() >= 64 * (60 // horizon)
    assert parity.counters_match(env, ref)
    if mode == 2:
        assert len(set(ref.level_id.tolist())) > 8


def test_touch_rewards_match_on_crowded_scenes():
    # no horizon: every done comes from a green-blue or green-red touch
    lv = scenes.make_levels("L", 64, 33, static_prob=0.1)
    env, ref = parity.make_pair(lv, 256, auto_reset=2, seed=5)
    act = scenes.make_actions(64, 256, env.n_actions, 33)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=32)
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    assert (r > 0).sum() > 0 and (r < 0).sum() > 0
    err, exact = parity.errors(env, ref)
    assert exact, err


def test_custom_dimensions_and_inactive_entities():
    dims = scenes.SceneDims(3, 3, 1, 1)
    lv = scenes.make_levels(dims, 16, 41, static_prob=0.2, triangle_prob=0.4)
    lv["active"][2, 2] = 0
    lv["joint_active"][3, 0] = 0
    lv["thr_active"][4, 0] = 0
    env, ref = parity.make_pair(lv, 16)
    act = scenes.make_actions(40, 16, env.n_actions, 41)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=8)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)


@pytest.mark.parametrize("lanes", [8, 16, 32])
def test_more_active_pairs_than_lanes_and_than_shared_memory_records(lanes):
    # every shape of an L scene dropped on the same spot: far more touching pairs than twice the lanes
    # of a scene, so the step's contacts go through the global-memory scratch; as the pile spreads the
    # count falls through the range where lanes hold two records each, then one
    lv = scenes.make_levels("L", 6, 51)
    rng = np.random.default_rng(51)
    lv["pos"][:, 1:, 0] = rng.uniform(-0.3, 0.3, (6, 15)).astype(np.float32)
    lv["pos"][:, 1:, 1] = rng.uniform(0.8, 1.4, (6, 15)).astype(np.float32)
    lv["joint_active"][:] = 0
    env, ref = parity.make_pair(lv, 6, lanes_per_scene=lanes)
    trace = env.enable_trace()
    act = scenes.make_actions(12, 6, env.n_actions, 51)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[:1])
    on = ref.manifold[:, :, 5] > 0                   # 66 polygon pairs own two manifold slots each, the others one
    touching_pairs = (on[:, :132:2] | on[:, 1:132:2]).sum(1) + on[:, 132:].sum(1)
    assert touching_pairs.max() > lanes + lanes // 2        # more than the records a scene keeps on chip
    assert np.array_equal(trace.cpu().numpy()[:, :, 5], ref.manifold[:, :, 5])
    err, exact = parity.errors(env, ref)
    assert exact, err
    (r, d), (rr, dr) = parity.step_both(env, ref, act[1:], chunk=4)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)


def test_manifold_trace_matches_the_oracle():
    lv = scenes.make_levels("L", 32, 61, static_prob=0.1, triangle_prob=0.3)
    env, ref = parity.make_pair(lv, 32)
    trace = env.enable_trace()
    act = scenes.make_actions(30, 32, env.n_actions, 61)
    parity.step_both(env, ref, act)
    t = trace.cpu().numpy()
    m = ref.manifold
    assert np.array_equal(t[:, :, 5], m[:, :, 5]) and m[:, :, 5].sum() > 100
    on = m[:, :, 5] > 0
    assert np.array_equal(t[on].view(np.uint32), m[on].view(np.uint32))


@pytest.mark.parametrize("size", ["S", "M", "L"])
def test_observation_parity(size):
    lv = scenes.make_levels(size, 32, 71, static_prob=0.1, triangle_prob=0.3)
    lv["thr_active"][1, 0] = 0
    lv["joint_active"][2, 0] = 0
    env, ref = parity.make_pair(lv, 32)
    act = scenes.make_actions(10, 32, env.n_actions, 71)
    parity.step_both(env, ref, act)
    got = env.obs().cpu().numpy()
    want = ref.obs()
    assert got.shape == want.shape == (32, {"S": 235, "M": 333, "L": 704}[size])
    assert np.max(np.abs(got - want)) <= 1e-5
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


@pytest.mark.parametrize("size,n_envs,lanes,n_actions", [("S", 40, 0, 0), ("M", 40, 8, 0), ("L", 72, 16, 0), ("L", 24, 32, 16), ("L", 7000, 0, 0)])
def test_step_with_observation_in_one_launch(size, n_envs, lanes, n_actions):
    # k2d_step_obs = k2d_step then k2d_obs: one step at a time (the training loop's use), then launches of several steps,
    # with resets in between; 7000 envs are more than the device holds at once, so those launches are cut into runs and
    # the observation must come from the last run only
    import torch
    lv = scenes.make_levels(size, min(n_envs, 256), 15, static_prob=0.1, triangle_prob=0.2, fixed_prob=0.2)
    kw = dict(n_actions=n_actions) if n_actions else {}
    env, ref = parity.make_pair(lv, n_envs, auto_reset=2, max_episode_steps=7, seed=9, lanes_per_scene=lanes, max_fused_steps=20, **kw)
    act = scenes.make_actions(3 + 20 + 11, n_envs, env.n_actions, 15)
    for lo, hi in ((0, 1), (1, 2), (2, 3), (3, 23), (23, 34)):
        r, d, o = env.step_obs(torch.from_numpy(act[lo:hi]).cuda())
        rr, dr = ref.step(act[lo:hi], n_threads=8)
        assert np.array_equal(r.cpu().numpy(), rr) and np.array_equal(d.cpu().numpy(), dr)
        assert np.array_equal(o.cpu().numpy().view(np.uint32), ref.obs().view(np.uint32)), (lo, hi)
        assert torch.equal(o, env.obs())
    err, exact = parity.errors(env, ref)
    assert exact, err


@pytest.mark.parametrize("size,n_envs,lanes,batch", [("L", 72, 16, 16), ("L", 48, 32, 4), ("L", 24, 8, 1000), ("M", 48, 0, 16), ("S", 40, 0, 2), ("L", 40, 16, 1)])
def test_batched_contact_solve_matches_the_oracle(size, n_envs, lanes, batch):
    # the paper's batched impulse resolution (batches of `batch` manifold slots, rows of a batch solved side by side);
    # a quarter of the scenes crowded, so that batches really hold several rows; batches of one slot are the sequential solve
    lv = scenes.make_levels(size, n_envs, 16, static_prob=0.1, triangle_prob=0.2, fixed_prob=0.2)
    lv["pos"][: n_envs // 4, 1:, 0] *= 0.15
    env, ref = parity.make_pair(lv, n_envs, solver_batch=batch, lanes_per_scene=lanes, auto_reset=2, max_episode_steps=30, seed=8)
    act = scenes.make_actions(50, n_envs, env.n_actions, 16)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[:1])
    err, exact = parity.errors(env, ref)
    _check_tolerances(err, 1)
    assert exact, err
    (r, d), (rr, dr) = parity.step_both(env, ref, act[1:], chunk=7)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    assert parity.counters_match(env, ref)
    seq = k2d_ref.RefSim(lv, n_envs, auto_reset=2, max_episode_steps=30, seed=8)
    seq.step(act)
    if batch == 1:
        assert np.array_equal(seq.pos, ref.pos)          # batches of one slot: the sequential solve
    if batch >= 16:
        assert not np.array_equal(seq.pos, ref.pos)      # few batches: crowded scenes take another course


def test_non_finite_state_is_flagged_not_propagated():
    lv = scenes.make_levels("S", 8, 81)
    env, ref = parity.make_pair(lv, 8)
    st = env.get_state()
    st["vel"][3, 2, 0] = np.inf
    env.set_state(st)
    ref.vel[3, 2, 0] = np.inf
    act = scenes.make_actions(3, 8, env.n_actions, 81)
    (r, d), (rr, dr) = parity.step_both(env, ref, act)
    assert np.array_equal(r, rr) and np.array_equal(d, dr) and d[:, 3].all()
    assert env.get_state()["status"][3] == 1 and parity.counters_match(env, ref)


def test_step_rejects_too_many_fused_steps():
    import torch
    lv = scenes.make_levels("S", 4, 1)
    env = k2d.Env(lv, 4, max_fused_steps=4)
    act = torch.zeros((5, 4, env.n_actions), device="cuda")
    with pytest.raises(k2d.K2DError):
        env.step(act)


@pytest.mark.parametrize("size,lanes", [("L", 16), ("L", 32), ("M", 8), ("S", 16)])
def test_fixed_joints_and_joint_limits_match_the_oracle(size, lanes):
    # a third of the joints fixed, a third with rotation limits; motors push the limited ones against their stops
    n_envs = 96
    lv = scenes.make_levels(size, n_envs, 71, static_prob=0.1, triangle_prob=0.2, fixed_prob=0.34, limit_prob=0.33)
    assert lv["joint_fixed"].sum() > 0 and lv["joint_limited"].sum() > 0
    env, ref = parity.make_pair(lv, n_envs, lanes_per_scene=lanes, max_fused_steps=128)
    act = scenes.make_actions(120, n_envs, env.n_actions, 71)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[:1])
    err, exact = parity.errors(env, ref)
    _check_tolerances(err, 1)
    assert exact, err
    (r, d), (rr, dr) = parity.step_both(env, ref, act[1:], chunk=17)
    err, exact = parity.errors(env, ref)
    _check_tolerances(err, 120)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    assert np.abs(ref.jacc[:, :, 2]).max() > 0                    # fixed joints carry accumulated angular impulses
    assert np.array_equal(env.obs().cpu().numpy().view(np.uint32), ref.obs().view(np.uint32))


def test_joint_kinds_with_auto_reset_and_checkpoint():
    lv = scenes.make_levels("L", 32, 72, static_prob=0.1, fixed_prob=0.5, limit_prob=0.5)
    env, ref = parity.make_pair(lv, 64, auto_reset=2, max_episode_steps=7, seed=3, joint_gamma=3.0)
    act = scenes.make_actions(40, 64, env.n_actions, 72)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[:20], chunk=5)
    st = env.get_state()
    env2 = k2d.Env(lv, 64, auto_reset=2, max_episode_steps=7, seed=3, joint_gamma=3.0)
    env2.set_state(st)
    parity.step_both(env, ref, act[20:], chunk=20)
    import torch
    env2.step(torch.from_numpy(act[20:]).cuda())
    err, exact = parity.errors(env, ref)
    assert exact, err
    sa, sb = env.get_state(), env2.get_state()
    for k in sa:
        assert np.array_equal(sa[k], sb[k], equal_nan=True), k


def test_multi_discrete_actions_match_the_oracle():
    n_envs = 64
    lv = scenes.make_levels("L", n_envs, 81, static_prob=0.1)
    env = k2d.Env(lv, n_envs)
    ref = k2d_ref.RefSim(lv, n_envs, discrete_actions=1)
    codes = np.random.default_rng(81).integers(0, 3, (40, n_envs, env.n_actions)).astype(np.int32)
    (r, d), (rr, dr) = parity.step_both(env, ref, codes, chunk=10)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    # the same codes read as floats would be something else: the discrete entry point really decoded them
    env2 = k2d.Env(lv, n_envs)
    import torch
    env2.step(torch.from_numpy(codes.astype(np.float32)).cuda())
    assert not np.array_equal(env2.get_state()["angvel"], env.get_state()["angvel"])


@pytest.mark.parametrize("lanes", [16, 32])
def test_dense_reward_matches_the_oracle(lanes):
    n_envs = 128
    lv = scenes.make_levels("L", 64, 82, static_prob=0.1)
    env, ref = parity.make_pair(lv, n_envs, auto_reset=2, max_episode_steps=9, seed=4, dense_kappa=0.3, lanes_per_scene=lanes)
    act = scenes.make_actions(48, n_envs, env.n_actions, 82)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=16)
    assert np.array_equal(r.view(np.uint32), rr.view(np.uint32)) and np.array_equal(d, dr)
    assert np.count_nonzero((r != 0) & (np.abs(r) < 0.5)) > r.size // 2          # most steps carry a dense term
    err, exact = parity.errors(env, ref)
    assert exact, err


@pytest.mark.parametrize("size", ["S", "M", "L"])
def test_pixel_observation_matches_the_oracle(size):
    n_envs = 24
    lv = scenes.make_levels(size, n_envs, 91, static_prob=0.2, triangle_prob=0.3)
    lv["active"][3, 2] = 0
    env, ref = parity.make_pair(lv, n_envs)
    assert np.array_equal(env.render().cpu().numpy(), ref.render())       # the levels as placed
    act = scenes.make_actions(30, n_envs, env.n_actions, 91)
    parity.step_both(env, ref, act)
    img, want = env.render().cpu().numpy(), ref.render()
    assert np.array_equal(img, want)                                      # byte for byte after 30 steps
    assert (want[..., :3] != 255).any(-1).mean() > 0.05 and np.all(img[..., 3] == 255)


def test_degenerate_and_edge_cases_match_the_oracle():
    # hand-made scenes around the narrowphase's special cases, one env each: coincident circle centres, a circle
    # centre inside a polygon and exactly on a face, boxes resting with exactly parallel faces, a triangle tip in
    # a box, a lone floor (nothing to do), an all-fixated scene, and a single env on its own
    dims = scenes.SceneDims(4, 3, 1, 1)
    floor = dict(half=(5.0, 0.5), pos=(0.0, -0.5), static=1)
    cases = [
        scenes.custom_level(dims, polygons=[floor], circles=[dict(radius=0.3, pos=(0.0, 2.0)), dict(radius=0.2, pos=(0.0, 2.0))]),
        scenes.custom_level(dims, polygons=[floor, dict(half=(0.5, 0.5), pos=(0.0, 0.5))],
                            circles=[dict(radius=0.1, pos=(0.1, 0.6)), dict(radius=0.2, pos=(0.0, 1.0)), dict(radius=0.2, pos=(0.5, 0.5))]),
        scenes.custom_level(dims, polygons=[floor, dict(half=(0.5, 0.25), pos=(0.0, 0.25)), dict(half=(0.5, 0.25), pos=(0.0, 0.75)),
                                            dict(half=(0.25, 0.25), pos=(0.25, 1.25))]),
        scenes.custom_level(dims, polygons=[floor, dict(half=(0.6, 0.3), pos=(0.0, 0.3)),
                                            dict(verts=[(-0.3, 0.2), (0.0, -0.4), (0.3, 0.2)], pos=(0.1, 0.95))]),
        scenes.custom_level(dims, polygons=[floor]),
        scenes.custom_level(dims, polygons=[floor, dict(half=(0.3, 0.3), pos=(0.0, 0.2), static=1)],
                            circles=[dict(radius=0.2, pos=(0.1, 0.3), static=1)]),
    ]
    lv = scenes.concat_levels(cases)
    n = len(cases)
    env, ref = parity.make_pair(lv, n)
    act = scenes.make_actions(40, n, env.n_actions, 5)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[:1])
    err, exact = parity.errors(env, ref)
    _check_tolerances(err, 1)
    assert exact, err
    (r, d), (rr, dr) = parity.step_both(env, ref, act[1:], chunk=13)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    assert np.array_equal(env.obs().cpu().numpy().view(np.uint32), ref.obs().view(np.uint32))
    assert np.array_equal(env.render().cpu().numpy(), ref.render())
    # one env alone, one step at a time and the largest fused launch the handle allows
    one, one_ref = parity.make_pair(scenes.take_levels(lv, [2]), 1, max_fused_steps=64)
    a1 = scenes.make_actions(64 + 3, 1, one.n_actions, 6)
    parity.step_both(one, one_ref, a1[:3], chunk=1)
    parity.step_both(one, one_ref, a1[3:], chunk=64)
    err, exact = parity.errors(one, one_ref)
    assert exact, err


def test_noop_rollout_outcomes_match_the_oracle():
    lv = scenes.make_levels("M", 96, 95, static_prob=0.1)
    got = k2d.noop_outcomes(lv, 90, chunk=32)
    ref = k2d_ref.RefSim(lv, 96)
    r, d = ref.step(np.zeros((90, 96, ref.n_actions), np.float32))
    assert np.array_equal(got, k2d.first_outcomes(r, d))
    assert (got != 0).any()


def test_status_reports_a_wait_that_ran_out_and_reset_clears_it():
    # the kernel records a wait that ran out in a word of the control block; here the word is set from the host side
    # (nothing hangs, nothing waits) to check that k2d_status reports it and k2d_reset clears it
    import torch
    lv = scenes.make_levels("S", 4, 3)
    env = k2d.Env(lv, 4)
    env.status()
    env.state_buf[128:144].view(torch.int32)[2] = 1          # work-queue words follow the eight counters: ticket, left, error
    torch.cuda.synchronize()
    with pytest.raises(k2d.K2DError, match="waiting"):
        env.status()
    env.reset()
    assert env.status().sum() == 0


def test_a_wait_that_runs_out_ends_the_launch_and_is_reported():
    # With more envs than resident scene groups a launch of 16 steps is two runs of 8 steps per env, numbered in the order
    # (run, env) and handed out in batches: every scheduler group of warps starts with the batch of its own number, a ticket
    # counter hands out the rest.  Here the counter is moved on by one run's worth of batches from the host, so the first
    # runs of the last envs are skipped and only their second runs are handed out; each waits for a first run that nobody does.  The wait is bounded (64 polls of about 100 ns here): the first
    # group to run out records the error, every other wait ends at once, the kernel returns, k2d_status reports it and
    # k2d_reset clears it.  Nothing hangs and nothing faults.
    import torch
    n_envs = 6144
    lv = scenes.make_levels("L", 64, 5, static_prob=0.1)
    env = k2d.Env(lv, n_envs, max_fused_steps=16, lanes_per_scene=16)
    env.set_wait_limit(1)                                     # raised to the floor of 64 polls
    act = torch.zeros((16, n_envs, env.n_actions), device="cuda")
    before = env.get_state()
    # work-queue words follow the eight counters: ticket, left, error
    env.state_buf[128:144].view(torch.int32)[0] = -(-n_envs // env.items_per_ticket)
    torch.cuda.synchronize()
    env.step(act)
    torch.cuda.synchronize()
    with pytest.raises(k2d.K2DError, match="waiting"):
        env.status()
    after = env.get_state()
    # the envs beyond the device's scene groups (5920 on 148 SMs; which envs those are is the launch's business) were never
    # stepped, the others by 8 steps only
    idle = after["step_count"] == 0
    assert idle.sum() >= 200 and np.array_equal(before["pos"][idle], after["pos"][idle])
    assert after["step_count"].max() <= 8
    env.reset()
    assert env.status().sum() == 0
    env.set_wait_limit(1 << 24)
    r, d = env.step(act)                                       # the queue rewound itself: the next launch is an ordinary one
    torch.cuda.synchronize()
    assert np.all(env.get_state()["step_count"] == 16) and env.status()[3] == 16 * n_envs and d.shape == (16, n_envs)


def test_frame_skip_matches_the_oracle():
    n_envs = 64
    lv = scenes.make_levels("L", n_envs, 97, static_prob=0.1)
    env, ref = parity.make_pair(lv, n_envs, frame_skip=2, auto_reset=2, max_episode_steps=9, seed=2)
    import torch
    rows = scenes.make_actions(20, n_envs, env.n_actions, 97)
    r_ref, d_ref = ref.step(rows, n_steps=39)                         # the last row is held for one step only
    r, d = env.step(torch.from_numpy(rows).cuda(), n_steps=39)
    assert np.array_equal(r.cpu().numpy(), r_ref) and np.array_equal(d.cpu().numpy(), d_ref)
    err, exact = parity.errors(env, ref)
    assert exact, err
