"""Writes tests/golden/oracle_trajectories.txt: digests of short oracle trajectories on the seeded workloads.

Only the oracle runs here.  The file guards the oracle's arithmetic against silent change (the pins in
tests/test_oracle_*.py say that it is right; this says that it is still the same): a deliberate change of
the oracle regenerates it, with the reason in the commit message.

    python tests/golden/make_oracle_trajectories.py
"""
import hashlib
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import k2d_ref  # noqa: E402
from paper_2410_23208_b200 import scenes  # noqa: E402

CASES = (
    # name, size, n_levels, n_envs, steps, level kwargs, sim kwargs
    ("S_plain", "S", 16, 16, 32, dict(), dict()),
    ("M_reset_same", "M", 32, 48, 32, dict(static_prob=0.1), dict(auto_reset=1, max_episode_steps=9)),
    ("L_reset_pool", "L", 32, 64, 32, dict(static_prob=0.1), dict(auto_reset=2, max_episode_steps=11, seed=1003)),
    ("L_joint_kinds_dense", "L", 32, 32, 32, dict(static_prob=0.1, triangle_prob=0.2, fixed_prob=0.34, limit_prob=0.33),
     dict(dense_kappa=0.3)),
)


def digest(name, size, n_levels, n_envs, steps, lkw, skw):
    lv = scenes.make_levels(size, n_levels, 4242, **lkw)
    sim = k2d_ref.RefSim(lv, n_envs, **skw)
    act = scenes.make_actions(steps, n_envs, sim.n_actions, 4242)
    r, d = sim.step(act)
    h = hashlib.sha256()
    for a in (sim.pos, sim.angle, sim.vel, sim.angvel, sim.acc, sim.jacc, r, d, sim.obs(), sim.render()):
        h.update(np.ascontiguousarray(a).tobytes())
    return h.hexdigest()


def lines():
    return ["%s %s" % (c[0], digest(*c)) for c in CASES]


if __name__ == "__main__":
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_trajectories.txt")
    with open(path, "w") as f:
        f.write("# sha256 of state, accumulated impulses, reward, done, observation and image after 32 oracle steps\n")
        f.write("# written by tests/golden/make_oracle_trajectories.py (oracle only)\n")
        f.write("\n".join(lines()) + "\n")
    print(open(path).read())
