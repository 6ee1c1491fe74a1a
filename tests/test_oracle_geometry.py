"""Pins for the oracle's collision manifolds against definitions that do not come from it:
closed forms, brute-force distances and polygon clipping."""
import math

import numpy as np
import pytest

from oracle import k2d_ref

FLOOR = [(-5.0, -1.0), (5.0, -1.0), (5.0, 0.0), (-5.0, 0.0)]


def box(cx, cy, hx, hy, ang=0.0):
    c, s = math.cos(ang), math.sin(ang)
    loc = [(-hx, -hy), (hx, -hy), (hx, hy), (-hx, hy)]
    return [(cx + c * x - s * y, cy + s * x + c * y) for x, y in loc]


# ---------------------------------------------------------------- circle-circle
def test_cc_closed_form():
    m = k2d_ref.manifold_cc((0.0, 0.0), 1.0, (1.5, 0.0), 0.75, f64=True)
    assert m["active"] and m["pen"] == pytest.approx(0.25, abs=1e-15)
    assert np.allclose(m["n"], (1.0, 0.0)) and np.allclose(m["p"], (1.0, 0.0))
    # 3-4-5 triangle, not touching: pen = ra + rb - 5
    m = k2d_ref.manifold_cc((1.0, 1.0), 2.0, (4.0, 5.0), 2.5, f64=True)
    assert not m["active"] and m["pen"] == pytest.approx(-0.5, abs=1e-14)
    assert np.allclose(m["n"], (0.6, 0.8)) and np.allclose(m["p"], (1.0 + 1.2, 1.0 + 1.6))
    # the normal points from a to b: swapping the circles flips it
    m2 = k2d_ref.manifold_cc((4.0, 5.0), 2.5, (1.0, 1.0), 2.0, f64=True)
    assert np.allclose(m2["n"], (-0.6, -0.8)) and m2["pen"] == pytest.approx(-0.5, abs=1e-14)


def test_cc_coincident_centres():
    m = k2d_ref.manifold_cc((1.0, 2.0), 0.5, (1.0, 2.0), 0.25)
    assert m["active"] and m["pen"] == pytest.approx(0.75) and tuple(m["n"]) == (0.0, 1.0)


# ---------------------------------------------------------------- polygon-circle
def test_pc_reduces_to_circle_plane():
    for x, y, r in [(0.3, 0.4, 0.5), (-2.0, 0.2, 0.25), (1.0, 0.6, 0.5), (4.0, 0.05, 0.1)]:
        m = k2d_ref.manifold_pc(FLOOR, (x, y), r, f64=True)
        assert m["pen"] == pytest.approx(r - y, abs=1e-13)
        assert m["active"] == (r - y > 0)
        assert np.allclose(m["n"], (0.0, 1.0), atol=1e-13) and np.allclose(m["p"], (x, 0.0), atol=1e-13)


def test_pc_corner_is_point_distance():
    # beyond the end of the top face the closest point is the corner (5, 0)
    a, b, r = 0.3, 0.4, 0.6
    m = k2d_ref.manifold_pc(FLOOR, (5.0 + a, b), r, f64=True)
    assert m["pen"] == pytest.approx(r - 0.5, abs=1e-13)
    assert np.allclose(m["n"], (0.6, 0.8), atol=1e-13) and np.allclose(m["p"], (5.0, 0.0), atol=1e-13)


def test_pc_centre_inside_polygon():
    # centre 0.2 below the top face of the floor: pushed out along that face
    m = k2d_ref.manifold_pc(FLOOR, (1.0, -0.2), 0.3, f64=True)
    assert m["active"] and m["pen"] == pytest.approx(0.5, abs=1e-13)
    assert np.allclose(m["n"], (0.0, 1.0), atol=1e-13) and np.allclose(m["p"], (1.0, 0.0), atol=1e-13)


def _boundary_samples(verts, n=4000):
    v = np.asarray(verts, np.float64)
    t = np.linspace(0.0, 1.0, n)[:, None]
    return np.concatenate([v[k] + t * (v[(k + 1) % len(v)] - v[k]) for k in range(len(v))])


def _inside(verts, c):
    v = np.asarray(verts, np.float64)
    for k in range(len(v)):
        e = v[(k + 1) % len(v)] - v[k]
        if e[0] * (c[1] - v[k][1]) - e[1] * (c[0] - v[k][0]) < 0:
            return False
    return True


def test_pc_brute_force_distance():
    rng = np.random.default_rng(11)
    checked_out = checked_in = 0
    for _ in range(300):
        n = 3 if rng.random() < 0.3 else 4
        ang = np.sort(rng.uniform(0, 2 * np.pi, n))
        if np.min(np.diff(np.concatenate([ang, [ang[0] + 2 * np.pi]]))) < 0.4:
            continue
        rad = rng.uniform(0.5, 1.0)
        verts = [(rad * math.cos(a) + 0.3, rad * math.sin(a) - 0.2) for a in ang]  # convex, CCW (on a circle)
        c = rng.uniform(-2, 2, 2) if rng.random() < 0.6 else rng.uniform(-0.5, 0.5, 2)
        r = rng.uniform(0.05, 0.6)
        m = k2d_ref.manifold_pc(verts, c, r, f64=True)
        samples = _boundary_samples(verts)
        dmin = np.min(np.hypot(samples[:, 0] - c[0], samples[:, 1] - c[1]))
        assert abs(m["n"] @ m["n"] - 1.0) < 1e-12
        if _inside(verts, c):
            # inside: pen = r + distance to the nearest edge line
            assert m["pen"] == pytest.approx(r + dmin, abs=2e-3)
            checked_in += 1
        else:
            assert m["pen"] == pytest.approx(r - dmin, abs=2e-3)
            q = c - (r - m["pen"]) * m["n"]          # the closest boundary point
            assert np.allclose(q, m["p"], atol=1e-9)
            assert np.min(np.hypot(samples[:, 0] - q[0], samples[:, 1] - q[1])) < 2e-3
            checked_out += 1
    assert checked_out > 100 and checked_in > 10


# ---------------------------------------------------------------- polygon-polygon
def _clip_area(subject, clip):
    """Area of subject ∩ clip by Sutherland-Hodgman (both convex, CCW)."""
    out = [tuple(p) for p in subject]
    cl = [tuple(p) for p in clip]
    for k in range(len(cl)):
        a, b = cl[k], cl[(k + 1) % len(cl)]
        inp, out = out, []
        if not inp:
            break

        def side(p):
            return (b[0] - a[0]) * (p[1] - a[1]) - (b[1] - a[1]) * (p[0] - a[0])
        for i in range(len(inp)):
            p, q = inp[i], inp[(i + 1) % len(inp)]
            sp, sq = side(p), side(q)
            if sp >= 0:
                out.append(p)
            if (sp >= 0) != (sq >= 0):
                t = sp / (sp - sq)
                out.append((p[0] + t * (q[0] - p[0]), p[1] + t * (q[1] - p[1])))
    if len(out) < 3:
        return 0.0
    a = 0.0
    for i in range(len(out)):
        p, q = out[i], out[(i + 1) % len(out)]
        a += p[0] * q[1] - p[1] * q[0]
    return 0.5 * a


def test_pp_box_on_floor_by_hand():
    m = k2d_ref.manifold_pp(FLOOR, box(1.0, 0.45, 0.5, 0.5), f64=True)
    assert m[0]["active"] and m[1]["active"]
    for k, x in ((0, 0.5), (1, 1.5)):     # end points of the box's bottom edge, in its vertex order
        assert m[k]["pen"] == pytest.approx(0.05, abs=1e-13)
        assert np.allclose(m[k]["n"], (0.0, 1.0), atol=1e-13)
        assert np.allclose(m[k]["p"], (x, -0.05), atol=1e-13)


def test_pp_overhang_is_clipped_to_the_reference_face():
    m = k2d_ref.manifold_pp(FLOOR, box(5.2, 0.45, 0.5, 0.5), f64=True)
    assert np.allclose(m[0]["p"], (4.7, -0.05), atol=1e-13)
    assert np.allclose(m[1]["p"], (5.0, -0.05), atol=1e-13)       # 5.7 clipped back to the floor's end
    assert m[0]["pen"] == pytest.approx(0.05, abs=1e-13) and m[1]["pen"] == pytest.approx(0.05, abs=1e-13)


def test_pp_reference_on_b_flips_the_normal():
    # a small box (a) pressed 0.1 into the side of a big one (b): b's face is the reference,
    # the manifold normal still points from a to b
    a = box(-0.45, 0.0, 0.25, 0.1)
    b = box(1.0, 0.0, 1.2, 1.5, 0.0)
    m = k2d_ref.manifold_pp(a, b, f64=True)
    # a's right face at x = -0.2, b's left face at x = -0.2 ... overlap 0 -> move a right by 0.1
    a = box(-0.35, 0.0, 0.25, 0.1)
    m = k2d_ref.manifold_pp(a, b, face_tol=0.0, f64=True)
    act = [k for k in m if k["active"]]
    assert len(act) == 2
    for k in act:
        assert np.allclose(k["n"], (1.0, 0.0), atol=1e-13) and k["pen"] == pytest.approx(0.1, abs=1e-13)


def test_pp_tilted_box_single_deep_corner():
    # box tilted by 0.3 rad with its lowest corner 0.02 below the floor's top face
    hx = hy = 0.5
    ang = 0.3
    low = min(y for _, y in box(0.0, 0.0, hx, hy, ang))
    b = box(0.0, -low - 0.02, hx, hy, ang)
    m = k2d_ref.manifold_pp(FLOOR, b, f64=True)
    pens = sorted(k["pen"] for k in m)
    assert pens[1] == pytest.approx(0.02, abs=1e-12) and pens[0] < 0  # other end of the incident edge is above
    deep = max(m, key=lambda k: k["pen"])
    assert np.allclose(deep["n"], (0.0, 1.0), atol=1e-12)
    assert deep["p"][1] == pytest.approx(-0.02, abs=1e-12)


def _random_quad(rng, centre, scale):
    ang = np.sort(rng.uniform(0, 2 * np.pi, 4))
    while np.min(np.diff(np.concatenate([ang, [ang[0] + 2 * np.pi]]))) < 0.5:
        ang = np.sort(rng.uniform(0, 2 * np.pi, 4))
    rad = rng.uniform(0.6, 1.0, 4) * scale
    # points on a slightly perturbed circle are convex when the perturbation is small
    pts = [(centre[0] + r * math.cos(a), centre[1] + r * math.sin(a)) for r, a in zip(np.full(4, rad.mean()), ang)]
    return pts


def test_pp_agrees_with_clipping_brute_force():
    rng = np.random.default_rng(5)
    n_overlap = n_apart = n_separated = n_missed = 0
    for _ in range(600):
        A = _random_quad(rng, (0.0, 0.0), 1.0)
        B = _random_quad(rng, rng.uniform(-1.6, 1.6, 2), rng.uniform(0.3, 1.0))
        area = _clip_area(A, B)
        m = k2d_ref.manifold_pp(A, B, face_tol=0.0, f64=True)
        any_active = m[0]["active"] or m[1]["active"]
        if area <= 0.0:
            assert not any_active           # disjoint polygons never give an active manifold
            n_apart += 1
            continue
        if not any_active:
            n_missed += 1                   # grazing corner overlaps may clip to nothing: must stay rare
            assert area < 0.02
            continue
        n_overlap += 1
        n = m[0]["n"]
        pen = max(k["pen"] for k in m if k["active"])
        # moving b along the manifold normal (a -> b) separates the polygons: the overlap shrinks,
        # and when the deepest vertex survived the clipping it vanishes after exactly `pen`
        moved = [(x + (pen + 1e-7) * n[0], y + (pen + 1e-7) * n[1]) for x, y in B]
        after = _clip_area(A, moved)
        assert after < area
        n_separated += after < 1e-9
    assert n_separated > 0.6 * n_overlap
    assert n_apart > 100 and n_overlap > 100 and n_missed < 0.05 * n_overlap


def test_pp_minimum_translation_face_contact():
    # boxes lying face-to-face on a wide box: the deepest vertex is inside the reference face, so the
    # largest penetration is exactly the minimum translation distance along the manifold normal
    rng = np.random.default_rng(9)
    for _ in range(100):
        ang = rng.uniform(-0.25, 0.25)
        hx, hy = rng.uniform(0.2, 0.8, 2)
        depth = rng.uniform(0.005, 0.05)
        low = min(y for _, y in box(0.0, 0.0, hx, hy, ang))
        B = box(rng.uniform(-2, 2), -low - depth, hx, hy, ang)
        m = k2d_ref.manifold_pp(FLOOR, B, face_tol=0.0, f64=True)
        pen = max(k["pen"] for k in m)
        n = m[0]["n"]
        assert pen == pytest.approx(depth, abs=1e-12)
        out = [(x + (pen + 1e-9) * n[0], y + (pen + 1e-9) * n[1]) for x, y in B]
        still = [(x + (pen - 1e-6) * n[0], y + (pen - 1e-6) * n[1]) for x, y in B]
        assert _clip_area(FLOOR, out) <= 1e-12 and _clip_area(FLOOR, still) > 0.0


def test_pp_rigid_transform_invariance():
    rng = np.random.default_rng(21)
    for _ in range(100):
        A = box(0.0, 0.0, rng.uniform(0.3, 1), rng.uniform(0.3, 1), rng.uniform(-3, 3))
        B = box(rng.uniform(-1, 1), rng.uniform(-1, 1), rng.uniform(0.3, 1), rng.uniform(0.3, 1), rng.uniform(-3, 3))
        m = k2d_ref.manifold_pp(A, B, f64=True)
        th, tx, ty = rng.uniform(-3, 3), rng.uniform(-4, 4), rng.uniform(-4, 4)
        c, s = math.cos(th), math.sin(th)

        def xf(P):
            return [(tx + c * x - s * y, ty + s * x + c * y) for x, y in P]
        m2 = k2d_ref.manifold_pp(xf(A), xf(B), f64=True)
        for k in range(2):
            assert m[k]["active"] == m2[k]["active"]
            if m[k]["active"]:
                assert m2[k]["pen"] == pytest.approx(m[k]["pen"], abs=1e-10)
                assert np.allclose(m2[k]["n"], (c * m[k]["n"][0] - s * m[k]["n"][1], s * m[k]["n"][0] + c * m[k]["n"][1]), atol=1e-10)
                assert np.allclose(m2[k]["p"], xf([m[k]["p"]])[0], atol=1e-10)


def test_pp_triangle_on_floor():
    tri = [(-0.5, -0.03), (0.5, -0.03), (0.0, 0.8)]
    m = k2d_ref.manifold_pp(FLOOR, tri, f64=True)
    assert m[0]["active"] and m[1]["active"]
    assert {round(float(k["p"][0]), 6) for k in m} == {-0.5, 0.5}
    assert all(k["pen"] == pytest.approx(0.03, abs=1e-13) for k in m)


def test_f32_manifolds_track_f64():
    rng = np.random.default_rng(3)
    for _ in range(200):
        A = box(0.0, 0.0, rng.uniform(0.3, 1), rng.uniform(0.3, 1), rng.uniform(-3, 3))
        B = box(rng.uniform(-1, 1), rng.uniform(-1, 1), rng.uniform(0.3, 1), rng.uniform(0.3, 1), rng.uniform(-3, 3))
        A32 = np.asarray(A, np.float32)
        B32 = np.asarray(B, np.float32)
        m64 = k2d_ref.manifold_pp(A32.astype(np.float64), B32.astype(np.float64), f64=True)
        m32 = k2d_ref.manifold_pp(A32, B32)
        for k in range(2):
            if abs(m64[k]["pen"]) > 1e-4 and m64[k]["pen"] > -0.5:
                assert m32[k]["active"] == m64[k]["active"]
            if m64[k]["active"] and m32[k]["active"]:
                assert m32[k]["pen"] == pytest.approx(m64[k]["pen"], abs=2e-5)
