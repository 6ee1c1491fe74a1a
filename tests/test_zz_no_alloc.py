"""k2d_step_static_scratch against k2d_step, through the C ABI.

The variant is for callers that cannot allocate the scratch tail of the state buffer (a fixed
device arena, a plug-in with a pre-sized buffer, code that may not call cudaMalloc): it keeps the
contact records of crowded scenes in an array inside the library.  Results must not change, on a
first call and on a second one that finds the array as the first left it.  This file sorts after
the other test files, so a run that stops at the first failure has already run them.
"""
import numpy as np
import pytest

from paper_2410_23208_b200 import k2d, scenes
from tests import parity

pytestmark = pytest.mark.gpu


def _crowded_levels(n_levels, seed):
    # some scenes with every shape dropped on the same spot (far more than 32 touching pairs, so the
    # scratch really is used), the rest ordinary
    lv = scenes.make_levels("L", n_levels, seed)
    rng = np.random.default_rng(seed)
    k = n_levels // 2
    lv["pos"][:k, 1:, 0] = rng.uniform(-0.3, 0.3, (k, 15)).astype(np.float32)
    lv["pos"][:k, 1:, 1] = rng.uniform(0.8, 1.4, (k, 15)).astype(np.float32)
    lv["joint_active"][:k] = 0
    return lv


@pytest.mark.parametrize("lanes", [32, 16])
def test_static_scratch_step_equals_step_on_two_calls_in_a_row(lanes):
    import ctypes
    import torch
    n_envs = 24
    calls = ((0, 1), (1, 7))     # action rows of the first call (one step, the pile at its densest) and of the second
    lv = _crowded_levels(n_envs, 77)
    a = k2d.Env(lv, n_envs, lanes_per_scene=lanes)
    b = k2d.Env(lv, n_envs, lanes_per_scene=lanes)
    # the variant must leave the scratch tail of its state buffer alone: the tail is filled with a pattern here and
    # looked at again after every call
    tail = a.lib.k2d_state_bytes_no_scratch(ctypes.byref(b.cfg))
    assert 0 < tail < b.state_buf.numel()
    b.state_buf[tail:] = 0xA5
    trace = a.enable_trace()
    act = scenes.make_actions(calls[-1][1], n_envs, a.n_actions, 77)
    for call, (lo, hi) in enumerate(calls):
        x = torch.from_numpy(act[lo:hi]).cuda()
        ra, da = a.step(x)
        rb, db = b.step(x, static_scratch=True)
        torch.cuda.synchronize()
        # touching pairs in the latest step: 66 polygon pairs own two manifold slots each, the others one.  A scene keeps
        # the records of its first lanes + lanes / 2 touching pairs on chip; with more, all of the step's records go
        # through the scratch, which is what the first call must reach
        on = trace.cpu().numpy()[:, :, 5] > 0
        pairs = (on[:, :132:2] | on[:, 1:132:2]).sum(1) + on[:, 132:].sum(1)
        assert call > 0 or pairs.max() > lanes + lanes // 2, pairs
        assert torch.equal(ra, rb) and torch.equal(da, db)
        sa, sb = a.get_state(), b.get_state()
        for key in parity.STATE_KEYS:
            assert np.array_equal(sa[key].view(np.uint32), sb[key].view(np.uint32)), (call, key)
        for key in parity.META_KEYS:
            assert np.array_equal(sa[key], sb[key]), (call, key)
        assert np.array_equal(a.status(), b.status())
        assert bool((b.state_buf[tail:] == 0xA5).all())


def test_static_scratch_step_refuses_more_envs_than_its_array_holds():
    import torch
    n_envs = 1025
    lv = scenes.make_levels("L", 8, 78)
    env = k2d.Env(lv, n_envs)
    act = torch.zeros((1, n_envs, env.n_actions), dtype=torch.float32, device="cuda")
    with pytest.raises(k2d.K2DError, match="built-in limit"):
        env.step(act, static_scratch=True)
    env.step(act)      # the ordinary entry point takes the same handle
    torch.cuda.synchronize()
