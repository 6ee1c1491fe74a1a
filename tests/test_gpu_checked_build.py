"""The checked build of the library (-DK2D_CHECKED: every index the kernels unpack from packed words or read from tables is
compared with its limit, a violation sets a status bit and the access is redirected; nothing traps) run over the cases that
use the most index arithmetic: the three size classes, every lanes-per-scene setting, piles that overflow the on-chip
records, auto-reset from a pool, more envs than resident groups, the batched solve, the fused observation.  It stands in for
a memory checker: results must still equal the oracle's and no check may fire."""
import numpy as np
import pytest

from paper_2410_23208_b200 import k2d, scenes
from tests import parity


def test_checked_library_builds_and_says_so():
    lib = k2d.load_library(checked=True)
    assert lib.k2d_is_checked_build() == 1 and k2d.load_library().k2d_is_checked_build() == 0
    for name in k2d.EXPORTS:
        assert hasattr(lib, name), name


def _pair(lv, n_envs, **cfg):
    env, ref = parity.make_pair(lv, n_envs, checked=True, **cfg)
    assert env.lib.k2d_is_checked_build() == 1
    return env, ref


def _run(env, ref, act, chunk):
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=chunk, n_threads=8)
    assert np.array_equal(r, rr) and np.array_equal(d, dr)
    err, exact = parity.errors(env, ref)
    assert exact, err
    assert parity.counters_match(env, ref)          # k2d_status raises if an index check fired


@pytest.mark.gpu
@pytest.mark.parametrize("size,n_envs,lanes", [("S", 40, 8), ("S", 40, 0), ("M", 48, 16), ("M", 48, 32), ("L", 72, 8), ("L", 72, 16), ("L", 72, 32)])
def test_no_index_check_fires_on_generated_scenes(size, n_envs, lanes):
    lv = scenes.make_levels(size, n_envs, 17, static_prob=0.1, triangle_prob=0.2, fixed_prob=0.2, limit_prob=0.2)
    lv["pos"][: n_envs // 6, 1:, 0] *= 0.15            # some crowded scenes: second records and the memory-record path
    env, ref = _pair(lv, n_envs, lanes_per_scene=lanes, auto_reset=2, max_episode_steps=17, seed=4, dense_kappa=0.1)
    _run(env, ref, scenes.make_actions(60, n_envs, env.n_actions, 17), 13)
    import torch
    r, d, o = env.step_obs(torch.zeros((1, n_envs, env.n_actions), device="cuda"))
    ref.step(np.zeros((1, n_envs, env.n_actions), np.float32))
    assert np.array_equal(o.cpu().numpy().view(np.uint32), ref.obs().view(np.uint32))
    env.status()


@pytest.mark.gpu
@pytest.mark.parametrize("lanes", [8, 16, 32])
def test_no_index_check_fires_on_piles(lanes):
    lv = scenes.make_levels("L", 6, 51)
    rng = np.random.default_rng(51)
    lv["pos"][:, 1:, 0] = rng.uniform(-0.3, 0.3, (6, 15)).astype(np.float32)
    lv["pos"][:, 1:, 1] = rng.uniform(0.8, 1.4, (6, 15)).astype(np.float32)
    lv["joint_active"][:] = 0
    env, ref = _pair(lv, 6, lanes_per_scene=lanes)
    _run(env, ref, scenes.make_actions(16, 6, env.n_actions, 51), 4)


@pytest.mark.gpu
def test_no_index_check_fires_through_the_work_queue_and_in_the_batched_solve():
    lv = scenes.make_levels("L", 256, 77, static_prob=0.1)
    env, ref = _pair(lv, 6200, auto_reset=2, max_episode_steps=10, seed=77, max_fused_steps=24)
    _run(env, ref, scenes.make_actions(20, 6200, env.n_actions, 77), 20)
    lv = scenes.make_levels("M", 64, 78, static_prob=0.1)
    lv["pos"][:16, 1:, 0] *= 0.15
    env, ref = _pair(lv, 64, solver_batch=16)
    _run(env, ref, scenes.make_actions(30, 64, env.n_actions, 78), 10)


@pytest.mark.gpu
def test_a_bad_count_in_the_state_record_is_caught_and_redirected():
    # the number of warm entries of env 0 is overwritten with 1000 from the host (far beyond the 21 pairs of an S scene); the
    # checked build reports it through k2d_status and uses 0 instead, so nothing is read out of range; k2d_reset clears it
    import torch
    n_envs = 8
    lv = scenes.make_levels("S", n_envs, 3)
    env = k2d.Env(lv, n_envs, checked=True)
    act = torch.zeros((4, n_envs, env.n_actions), device="cuda")
    env.step(act)
    env.status()
    # state buffer: 4096-byte control block, then level ids and chunk counters (4 bytes per env each, 256-byte aligned), then
    # the env records; an S record has its meta words after 6 x 7 body words and 3 joint words, the count is meta word 4
    offset = 4096 + 512 + 4 * (6 * 7 + 3 + 4)
    assert int(env.state_buf[offset:offset + 4].view(torch.int32)[0]) <= 21
    env.state_buf[offset:offset + 4].view(torch.int32)[0] = 1000
    torch.cuda.synchronize()
    env.step(act)
    torch.cuda.synchronize()
    with pytest.raises(k2d.K2DError, match="index check"):
        env.status()
    env.reset()
    env.step(act)
    assert env.status()[3] == 4 * n_envs


# ---------------------------------------------------------------- the build that counts cycles per phase of a step
def test_phase_clock_library_builds_and_the_plain_library_refuses_the_call():
    from paper_2410_23208_b200 import build
    lib = k2d.load_library(phase_clocks=True)
    assert build.LIB_PHASES.endswith("libk2d_phases.so") and lib.k2d_is_checked_build() == 0
    assert len(k2d.PHASES) == 14


@pytest.mark.gpu
def test_phase_clocks_count_every_phase_and_change_no_result():
    n_envs = 96
    lv = scenes.make_levels("L", 48, 77, static_prob=0.1)
    lv["pos"][:8, 1:, 0] *= 0.2                          # some crowded scenes: the memory-record path is timed too
    env, ref = parity.make_pair(lv, n_envs, phase_clocks=True, lanes_per_scene=16, auto_reset=2, max_episode_steps=12, seed=5)
    act = scenes.make_actions(24, n_envs, env.n_actions, 77)
    (r, d), (rr, dr) = parity.step_both(env, ref, act, chunk=24)
    assert np.array_equal(r.view(np.uint32), rr.view(np.uint32)) and np.array_equal(d, dr)
    err, exact = parity.errors(env, ref)
    assert exact, err
    cycles = env.phase_cycles()
    assert set(cycles) == set(k2d.PHASES)
    for name in ("geometry", "box_test", "narrowphase", "records", "iterations", "integrate_correct", "epilogue", "load", "store"):
        assert cycles[name] > 0, name
    assert cycles["iterations"] > cycles["joint_prestep"]
    assert sum(env.phase_cycles().values()) == 0             # reading clears the sums
    # the library proper has no counters
    plain = k2d.Env(lv, 8)
    with pytest.raises(k2d.K2DError, match="build"):
        plain.phase_cycles()
