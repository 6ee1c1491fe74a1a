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
    assert np.array_equal(env.status(), ref.counters)
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
    assert np.array_equal(env.status(), ref.counters)       # also says that no wait ran out


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
    assert np.array_equal(env.status(), ref.counters) and ref.counters[0] == 0      # and nothing went non-finite
