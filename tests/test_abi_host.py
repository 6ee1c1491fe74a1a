"""CPU-side checks of the CUDA library: it loads, exports the declared symbols, and its host logic
(sizes, validation, level build) behaves as include/k2d.h says.  No kernel is launched."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import k2d_ref
from paper_2410_23208_b200 import k2d, scenes

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    lib = k2d.load_library()
    header = open(os.path.join(ROOT, "include", "k2d.h")).read()
    declared = set(re.findall(r"\b(k2d_[a-z0-9_]+)\s*\(", header))
    assert declared == set(k2d.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_struct_layouts_match_the_header():
    # sizes computed from the header's field lists
    assert C.sizeof(k2d.Config) == 13 * 4 + 13 * 4 + 8 + 8 + 4 + 4 + 4 + 4 + 8
    n_float = 12 * 4 * 2 + 4 + 16 * 2 + 16 + 16 * 2 + 16 + 3 * 16 + 6 * 2 * 2 + 6 * 2 + 6 * 3 + 2 * 2 + 2 + 2
    n_int = 12 + 3 * 16 + 2 * 6 + 2 * 6 + 2 * 6 + 2 + 2 * 2
    assert k2d.LEVEL_DTYPE.itemsize == 4 * (n_float + n_int)


def test_sizes_and_defaults():
    lib = k2d.load_library()
    cfg = k2d.Config()
    assert lib.k2d_default_config(C.byref(cfg), 16384, 12, 4, 6, 2) == 0
    assert (cfg.n_actions, cfg.solver_iters, cfg.warm_start) == (8, 8, 1)
    assert cfg.dt == pytest.approx(1 / 60) and cfg.gravity_y == pytest.approx(-9.81)
    assert lib.k2d_obs_floats(C.byref(cfg)) == 704
    assert lib.k2d_canonical_words(C.byref(cfg)) == 6 * 16 + 2 * 186 + 18 + 4
    sb = lib.k2d_state_bytes(C.byref(cfg))
    assert sb > 16384 * 6 * 16 * 4 and sb % 256 == 0
    # without the overflow-scratch tail: still the env states, and smaller by the tail (8192 slots of 120 pairs x 29 words)
    ns = lib.k2d_state_bytes_no_scratch(C.byref(cfg))
    assert 16384 * 6 * 16 * 4 < ns < sb and ns % 256 == 0 and sb - ns == 8192 * 120 * 29 * 4
    for dims, width in (((5, 2, 1, 1), 235), ((6, 3, 2, 2), 333)):
        lib.k2d_default_config(C.byref(cfg), 8, *dims)
        assert lib.k2d_obs_floats(C.byref(cfg)) == width
    bad = k2d.Config()
    assert lib.k2d_default_config(C.byref(bad), 8, 13, 4, 6, 2) == -2
    assert lib.k2d_state_bytes(C.byref(bad)) == 0


def _create(cfg, levels_packed, state=0x1000, pool=0x2000):
    lib = k2d.load_library()
    h = C.c_void_p()
    rc = lib.k2d_create(C.byref(cfg), state, pool, levels_packed.ctypes.data if levels_packed is not None else None, C.byref(h))
    return rc, h


def test_create_rejects_bad_arguments_before_touching_the_device():
    lv = scenes.make_levels("S", 2, 1)
    packed = k2d.pack_levels(lv)
    cfg = k2d.make_config(lv, 2)
    assert _create(cfg, None)[0] == -1                         # null levels
    assert _create(cfg, packed, state=0)[0] == -1              # null device buffer
    assert _create(cfg, packed, state=0x1004)[0] == -3         # misaligned
    cfg2 = k2d.make_config(lv, 2)
    cfg2.solver_iters = -1
    assert _create(cfg2, packed)[0] == -2
    cfg3 = k2d.make_config(lv, 2, lanes_per_scene=12)
    assert _create(cfg3, packed)[0] == -2
    for field, value in (("pos", np.nan), ("density", -1.0), ("poly_nverts", 5), ("joint_b", 99), ("motor_binding", 7),
                         ("role", 4), ("circle_radius", 0.0)):
        broken = packed.copy()
        broken[field][1].flat[1 if field in ("density", "poly_nverts", "role") else 0] = value
        assert _create(cfg, broken)[0] == -4, field
    # clockwise polygon
    broken = packed.copy()
    broken["poly_verts"][0, 1, :4] = broken["poly_verts"][0, 1, :4][::-1]
    assert _create(cfg, broken)[0] == -4
    # centroid not at the origin
    broken = packed.copy()
    broken["poly_verts"][0, 1, :, 0] += 0.2
    assert _create(cfg, broken)[0] == -4


def test_error_strings():
    lib = k2d.load_library()
    assert lib.k2d_error_string(0) == b"ok"
    assert len({lib.k2d_error_string(-k) for k in range(1, 8)}) == 7


@pytest.mark.parametrize("size,dims", [("S", None), ("M", None), ("L", None), (None, scenes.SceneDims(3, 3, 1, 1))])
def test_level_build_matches_the_oracle_bit_for_bit(size, dims):
    if size:
        lv = scenes.make_levels(size, 24, 17, static_prob=0.2, triangle_prob=0.3)
    else:
        lv = scenes.make_levels(dims, 24, 17, static_prob=0.2, triangle_prob=0.3)
        lv["active"][3, 2] = 0
        lv["joint_active"][5, 0] = 0
    n = lv["pos"].shape[0]
    cfg = k2d.make_config(lv, n)
    packed = k2d.pack_levels(lv)
    ref = k2d_ref.RefSim(lv, n)
    for l in range(n):
        im, ii, col = k2d.level_info(cfg, packed[l:l + 1])
        act = lv["active"][l] != 0
        assert np.array_equal(im[act], ref.inv_mass[l][act]) and np.array_equal(ii[act], ref.inv_inertia[l][act])
        assert np.array_equal(col, ref.collide[l])


def test_shard_envs_partitions_contiguously():
    for total, world in ((16384, 8), (10, 3), (7, 8)):
        spans = [k2d.shard_envs(total, r, world) for r in range(world)]
        assert spans[0][0] == 0 and sum(c for _, c in spans) == total
        for (o0, c0), (o1, _) in zip(spans, spans[1:]):
            assert o1 == o0 + c0


def test_first_outcomes_takes_the_reward_at_the_first_done_step():
    reward = np.array([[0, 0, 0, 0], [1, 0, -1, 0], [1, -1, 1, 0]], np.float32)
    done = np.array([[0, 0, 0, 0], [1, 0, 1, 0], [1, 1, 1, 0]], np.uint8)
    assert k2d.first_outcomes(reward, done).tolist() == [1, -1, -1, 0]
    # a done without reward (horizon) counts as neither
    assert k2d.first_outcomes(np.zeros((2, 1), np.float32), np.array([[0], [1]], np.uint8)).tolist() == [0]
