"""GPU parity at the size and launch configuration the benchmark times: L scenes, 16384 envs, 32 fused
steps per launch, auto-reset from a pool of 1024 levels with horizon 256.  With more envs than scene
groups resident on the device, a launch is cut into chunks that the groups hand to one another, so this
is also the test of that hand-over.  The oracle steps every env (threads over envs)."""
import os

import numpy as np
import pytest

from paper_2410_23208_b200 import scenes
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("lanes,horizon", [(0, 256), (32, 12)])
def test_benchmark_configuration_matches_the_oracle_on_every_env(lanes, horizon):
    w = scenes.WORKLOADS[3]
    seed = scenes.workload_seed(3)
    lv = scenes.make_levels(w["size"], w["n_levels"], seed, static_prob=w["static_prob"])
    n_envs, fused = w["n_envs"], 32
    env, ref = parity.make_pair(lv, n_envs, auto_reset=w["auto_reset"], max_episode_steps=horizon, seed=seed,
                                max_fused_steps=fused, lanes_per_scene=lanes)
    act = scenes.make_actions(2 * fused + 5, n_envs, env.n_actions, seed)
    # two full launches and a short one; the library's default lanes with the benchmark's horizon, and one
    # warp per scene with a horizon of 12, under which every env resets several times
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=fused, n_threads=os.cpu_count() or 1)
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert parity.counters_match(env, ref)
    assert d.sum() >= (n_envs * 5 if horizon == 12 else 1)


@pytest.mark.parametrize("lanes,n_envs", [(0, 6000), (32, 3000)])
def test_a_few_more_envs_than_resident_groups(lanes, n_envs):
    # just above the number of scene groups a B200 holds at once (5920 half-warps, 2960 warps for L scenes):
    # the second chunk of the first envs is handed out while their first chunk may still be running on another
    # group, so groups really wait for one another here
    w = scenes.WORKLOADS[3]
    seed = 77
    lv = scenes.make_levels(w["size"], 256, seed, static_prob=w["static_prob"])
    env, ref = parity.make_pair(lv, n_envs, auto_reset=2, max_episode_steps=10, seed=seed, max_fused_steps=24, lanes_per_scene=lanes)
    act = scenes.make_actions(40, n_envs, env.n_actions, seed)
    # launches of 20 steps: work items of 8, 8 and 4 steps
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=20, n_threads=os.cpu_count() or 1)
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert parity.counters_match(env, ref)       # also says that no wait ran out


def test_a_thousand_steps_stay_bit_identical():
    # long horizon: 1024 L envs x 1024 steps with pool resets, fixed joints, limits and a dense reward
    seed = 123
    lv = scenes.make_levels("L", 128, seed, static_prob=0.1, triangle_prob=0.2, fixed_prob=0.15, limit_prob=0.25)
    n_envs = 1024
    env, ref = parity.make_pair(lv, n_envs, auto_reset=2, max_episode_steps=300, seed=seed, dense_kappa=0.1, max_fused_steps=64)
    act = scenes.make_actions(1024, n_envs, env.n_actions, seed)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=64, n_threads=os.cpu_count() or 1)
    assert np.array_equal(r.view(np.uint32), rr.view(np.uint32)) and np.array_equal(d, dr)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert parity.counters_match(env, ref) and ref.counters[0] == 0      # and nothing went non-finite


def _workload_pair(index, n_envs, fused, **over):
    w = scenes.WORKLOADS[index]
    seed = scenes.workload_seed(index)
    lv = scenes.make_levels(w["size"], w["n_levels"], seed, static_prob=w["static_prob"])
    cfg = dict(auto_reset=w["auto_reset"], max_episode_steps=w["max_episode_steps"], seed=seed, max_fused_steps=fused)
    cfg.update(over)
    env, ref = parity.make_pair(lv, n_envs, **cfg)
    return env, ref, seed


def _run_and_compare(env, ref, act, fused):
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=fused, n_threads=os.cpu_count() or 1)
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert parity.counters_match(env, ref)
    return d


def test_workload_1_small_scenes_4096_envs_256_steps_same_level_reset():
    # the second benchmark configuration in full: S scenes, 4096 envs, 256 steps in launches of 32, every env restarts
    # on its own level when it is done
    n_envs, fused = scenes.WORKLOADS[1]["n_envs"], 32
    env, ref, seed = _workload_pair(1, n_envs, fused)
    act = scenes.make_actions(scenes.WORKLOADS[1]["n_steps"], n_envs, env.n_actions, seed)
    d = _run_and_compare(env, ref, act, fused)
    assert d.sum() > 0 and ref.episode_count.max() >= 1
    got, want = env.obs().cpu().numpy(), ref.obs()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_workload_2_medium_scenes_16384_envs():
    # the third configuration: M scenes, 16384 envs (more than the device holds at once, so the launches go through the
    # work queue); two launches of 32 steps on every env, then all 256 steps on the first 1024 envs, which do not
    # depend on the others
    n_envs, fused = scenes.WORKLOADS[2]["n_envs"], 32
    env, ref, seed = _workload_pair(2, n_envs, fused)
    act = scenes.make_actions(scenes.WORKLOADS[2]["n_steps"], n_envs, env.n_actions, seed)
    _run_and_compare(env, ref, act[:2 * fused], fused)
    got, want = env.obs().cpu().numpy(), ref.obs()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    sub, sub_ref, _ = _workload_pair(2, 1024, fused)
    d = _run_and_compare(sub, sub_ref, np.ascontiguousarray(act[:, :1024]), fused)
    assert d.sum() > 0
    # the subset's first 64 steps are the big run's
    both = _workload_pair(2, 1024, fused)
    parity.step_both(both[0], both[1], np.ascontiguousarray(act[:2 * fused, :1024]), chunk=fused)
    assert np.array_equal(both[0].get_state()["pos"], env.get_state()["pos"][:1024])


@pytest.mark.parametrize("size,n_envs,lanes", [("S", 7000, 32), ("M", 9000, 16)])
def test_small_size_classes_through_the_work_queue(size, n_envs, lanes):
    # S and M scenes with more envs than resident scene groups and launches of several work items per env
    index = 1 if size == "S" else 2
    env, ref, seed = _workload_pair(index, n_envs, 24, lanes_per_scene=lanes, auto_reset=2, max_episode_steps=10)
    act = scenes.make_actions(44, n_envs, env.n_actions, seed)
    d = _run_and_compare(env, ref, act, 22)               # work items of 8, 8 and 6 steps
    assert d.sum() >= 4 * n_envs


def test_workload_4_large_scenes_131072_envs_fused_steps_and_observation():
    # the top of the fifth configuration's sweep: L scenes, 131072 envs, one launch of 32 fused steps, then the
    # symbolic observation; every env and every observation row against the oracle
    n_envs, fused = scenes.WORKLOADS[4]["n_envs"], 32
    env, ref, seed = _workload_pair(4, n_envs, fused)
    act = scenes.make_actions(fused, n_envs, env.n_actions, seed)
    _run_and_compare(env, ref, act, fused)
    got, want = env.obs().cpu().numpy(), ref.obs()
    assert got.shape == (n_envs, 704)
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # the horizon of 256 is not reached in 32 steps; resets here come from touches
    assert ref.counters[1] > 0


def test_short_launches_through_the_work_queue_reuse_and_renew_the_order_of_the_envs():
    # one and a half times as many envs as the device holds scene groups (so that launches sort them), one or two steps per launch: the launch hands the envs out in an order
    # sorted by cost that it keeps for 16 launches; a reset with level ids (which uses the same words) makes the next launch
    # sort again.  Whatever the order, every env is stepped once per step.
    n_envs = 9000
    lv = scenes.make_levels("L", 128, 91, static_prob=0.1)
    env, ref = parity.make_pair(lv, n_envs, auto_reset=2, max_episode_steps=12, seed=91, max_fused_steps=8, lanes_per_scene=16)
    act = scenes.make_actions(40, n_envs, env.n_actions, 91)
    n_threads = os.cpu_count() or 1
    (r, d), (rr, dr) = parity.step_both(env, ref, act[:20], chunk=1, n_threads=n_threads)      # 20 launches of one step
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    ids = (np.arange(n_envs)[::-1] % 128).astype(np.int32)
    env.reset(ids); ref.reset(ids)
    (r, d), (rr, dr) = parity.step_both(env, ref, act[20:], chunk=2, n_threads=n_threads)      # 10 launches of two steps
    assert np.array_equal(r, rr) and np.array_equal(d, dr) and d.sum() > 0
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert env.status()[3] == 20 * n_envs and parity.counters_match(env, ref)      # both count from the reset


def test_discrete_actions_and_the_fused_observation_through_the_sorted_work_queue():
    # the two other launching entry points with more envs than scene groups and launches long enough to sort the envs:
    # k2d_step_discrete (multi-discrete codes) and k2d_step_obs (observation written by the stepping groups)
    import torch
    from oracle import k2d_ref
    from paper_2410_23208_b200 import k2d
    n_envs = 9000
    lv = scenes.make_levels("L", 128, 93, static_prob=0.1)
    env = k2d.Env(lv, n_envs, auto_reset=2, max_episode_steps=11, seed=93, max_fused_steps=16, lanes_per_scene=16)
    ref = k2d_ref.RefSim(lv, n_envs, auto_reset=2, max_episode_steps=11, seed=93, broadphase=0, discrete_actions=1)
    codes = np.random.default_rng(93).integers(0, 3, (32, n_envs, env.n_actions)).astype(np.int32)
    (r, d), (rr, dr) = parity.step_both(env, ref, codes, chunk=16, n_threads=os.cpu_count() or 1)
    assert np.array_equal(r, rr) and np.array_equal(d, dr) and d.sum() > 0
    err, exact = parity.errors(env, ref)
    assert exact, err

    env, ref = parity.make_pair(lv, n_envs, auto_reset=2, max_episode_steps=11, seed=94, max_fused_steps=16, lanes_per_scene=16)
    act = scenes.make_actions(32, n_envs, env.n_actions, 94)
    for lo in (0, 16):
        r, d, o = env.step_obs(torch.from_numpy(act[lo:lo + 16]).cuda())
        rr, dr = ref.step(act[lo:lo + 16], n_threads=os.cpu_count() or 1)
        assert np.array_equal(r.cpu().numpy(), rr) and np.array_equal(d.cpu().numpy(), dr)
        assert np.array_equal(o.cpu().numpy().view(np.uint32), ref.obs().view(np.uint32))
    err, exact = parity.errors(env, ref)
    assert exact, err


@pytest.mark.parametrize("size,n_envs,lanes", [("L", 7200, 8), ("L", 3200, 32), ("M", 3200, 32)])
def test_one_block_per_sm_form_with_8_and_32_lanes_per_scene(size, n_envs, lanes):
    # enough envs to fill every scene group of the device at these lane counts, so the step kernel runs as one block per SM
    # whose warps step in lockstep per scheduler (three warps per scheduler for L scenes at 8 lanes, five otherwise)
    index = 3 if size == "L" else 2
    env, ref, seed = _workload_pair(index, n_envs, 24, lanes_per_scene=lanes, auto_reset=2, max_episode_steps=10)
    assert env.resident_groups <= n_envs and env.items_per_ticket > 32 // lanes      # several warps per ticket: the one-block form
    act = scenes.make_actions(40, n_envs, env.n_actions, seed)
    d = _run_and_compare(env, ref, act, 20)               # work items of 8, 8 and 4 steps
    assert d.sum() >= 2 * n_envs
