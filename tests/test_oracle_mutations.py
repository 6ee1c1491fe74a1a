"""The pins must notice a wrong oracle: each case plants one plausible mistake in a scratch copy of oracle/k2d_oracle.c
(a dropped term, a flipped sign, a reversed order, a guard left out), builds that copy and runs the pins of
one test file (the one named with the case; test_oracle_order_and_guards.py if none is) against it in a child process; at least one pin has to fail.  The unchanged copy has to pass,
so a failure is the mistake's.  CPU only; nothing here touches the CUDA library."""
import os
import shutil
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
PINS = ["tests/test_oracle_order_and_guards.py"]
BATCHED_PINS = ["tests/test_oracle_batched.py"]
DYNAMICS_PINS = ["tests/test_oracle_dynamics.py"]
JOINT_PINS = ["tests/test_oracle_joint_kinds.py"]
ENV_PINS = ["tests/test_oracle_env.py"]

MISTAKES = {
    "unchanged": None,
    "joint positional correction dropped": (
        "real share = cf->joint_beta / msum;", "real share = RC(0) * cf->joint_beta / msum;"),
    "joint positional correction with the wrong sign on the second body": (
        "pos[2 * q->b] = R_FMA(-q->mb, q->corr_dir.x, pos[2 * q->b]);", "pos[2 * q->b] = R_FMA(q->mb, q->corr_dir.x, pos[2 * q->b]);"),
    "reference face chosen without the tolerance": (
        "int ref_on_b = sb > sa + face_tol;", "int ref_on_b = sb > sa;"),
    "incident face: the last of equal candidates": (
        "if (d < fd) { fd = d; f = k; }", "if (d <= fd) { fd = d; f = k; }"),
    "non-finite step keeps its reward": (
        "if (!finite) { reward = RC(0); done = 1;", "if (!finite) { done = 1;"),
    "motor applied to a joint whose shapes are absent or both fixated": (
        "if (!(S->lv_joint_active[l * J + j] && active[a] && active[b] && (inv_mass[a] + inv_mass[b] > RC(0)))) continue;",
        "if (!(S->lv_joint_active[l * J + j])) continue;"),
    "joints solved in reverse order": (
        "for (int j = 0; j < J; ++j) {\n            joint_row *q = &jr[j];\n            if (!q->on) continue;\n            real *va = vel + 2 * q->a, *vb = vel + 2 * q->b;\n            real wa",
        "for (int j = J - 1; j >= 0; --j) {\n            joint_row *q = &jr[j];\n            if (!q->on) continue;\n            real *va = vel + 2 * q->a, *vb = vel + 2 * q->b;\n            real wa"),
    "contacts solved in reverse order": (
        "for (int i = 0; i < n_rows; ++i) {\n            contact_row *r = &rows[i];\n            real *va = vel + 2 * r->a, *vb = vel + 2 * r->b;\n            real ma",
        "for (int i = n_rows - 1; i >= 0; --i) {\n            contact_row *r = &rows[i];\n            real *va = vel + 2 * r->a, *vb = vel + 2 * r->b;\n            real ma"),
    "dense reward measured from the last green shape": (
        "for (int i = N - 1; i >= 0; --i) if (active[i]) { if (role[i] == ROLE_GREEN) dense_g = i;",
        "for (int i = 0; i < N; ++i) if (active[i]) { if (role[i] == ROLE_GREEN) dense_g = i;"),
    "batched solve: a row's impulse taken as the whole accumulated one": (
        "dn[i] = nw - old;", "dn[i] = nw;", BATCHED_PINS),
    "batched solve: batches in reverse order": (
        "for (int b = 0; b < n_batches && b < n_rows; ++b) {", "for (int b = (n_batches < n_rows ? n_batches : n_rows) - 1; b >= 0; --b) {", BATCHED_PINS),
    "gravity on fixated shapes too": (
        "if (active[i] && inv_mass[i] > RC(0)) vel[2 * i + 1] = vel[2 * i + 1] + gdt;", "if (active[i]) vel[2 * i + 1] = vel[2 * i + 1] + gdt;", DYNAMICS_PINS),
    "restitution: the larger coefficient of the two": (
        "real er = rmin(rest[a], rest[b]);", "real er = rmax(rest[a], rest[b]);", DYNAMICS_PINS),
    "friction: coefficients added instead of combined by the root of the squares": (
        "r->mu = R_SQRT(R_FMA(fric[a], fric[a], fric[b] * fric[b]));", "r->mu = fric[a] + fric[b];", DYNAMICS_PINS),
    "penetration slop left out of the corrections": (
        "real depth = rmax(man[s].pen - cf->slop, RC(0));", "real depth = rmax(man[s].pen, RC(0));", DYNAMICS_PINS),
    "friction limited by the new impulse instead of the accumulated normal impulse": (
        "            real lim = r->mu * nw;\n            real oldt", "            real lim = r->mu * (nw - old);\n            real oldt", DYNAMICS_PINS),
    "joint limit pushes both ways": (
        "v = (wrel < RC(0)) ? wrel : wrel + q->bias_r;\n                    v = rmax(v, RC(0));", "v = (wrel < RC(0)) ? wrel : wrel + q->bias_r;", JOINT_PINS),
    "time-out one step late": (
        "S->step_count[e] >= cf->max_episode_steps;", "S->step_count[e] > cf->max_episode_steps;", ENV_PINS),
    "thruster on an absent shape fires": (
        "if (!active[i]) continue;\n        /* continuous in [0, 1]", "/* continuous in [0, 1]"),
}


@pytest.mark.parametrize("name", list(MISTAKES))
def test_pins_fail_on_a_planted_mistake(name, tmp_path):
    work = str(tmp_path / "copy")
    for sub in ("oracle", "tests", "paper_2410_23208_b200"):
        shutil.copytree(os.path.join(ROOT, sub), os.path.join(work, sub), ignore=shutil.ignore_patterns("__pycache__", "*.so", "csrc"))
    src = os.path.join(work, "oracle", "k2d_oracle.c")
    mistake = MISTAKES[name]
    if mistake is not None:
        with open(src) as f:
            text = f.read()
        assert text.count(mistake[0]) == 1, "the oracle no longer has the statement this case changes: update the case"
        with open(src, "w") as f:
            f.write(text.replace(mistake[0], mistake[1]))
    env = dict(os.environ, PYTHONPATH=work)
    pins = mistake[2] if mistake is not None and len(mistake) > 2 else PINS + (BATCHED_PINS if mistake is None else [])
    p = subprocess.run([sys.executable, "-m", "pytest", *pins, "-x", "-q", "-p", "no:cacheprovider", "--deselect", "tests/test_oracle_env.py::test_oracle_trajectories_have_not_changed"], cwd=work, env=env,
                       capture_output=True, text=True, timeout=600)
    if mistake is None:
        assert p.returncode == 0, p.stdout[-2000:]
    else:
        assert p.returncode == 1 and "failed" in p.stdout, f"no pin noticed: {name}\n{p.stdout[-1500:]}"
