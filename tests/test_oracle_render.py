"""Pins of the oracle's pixel observation (125 x 125, the paper's "Pixels" observation space) against
areas, known pixels and symmetries.  CPU only."""
import math

import numpy as np
import pytest

from oracle import k2d_ref
from paper_2410_23208_b200.scenes import ROLE_BLUE, ROLE_GREEN, ROLE_RED, SceneDims, custom_level

DIMS = SceneDims(3, 2, 1, 1)
S = 0.05                     # metres per pixel
X0, Y1 = -3.125, 5.75        # left and top edge of the window


def render(level, f64=True):
    return k2d_ref.RefSim(level, 1, f64=f64).render()[0]


def pixel_of(x, y):
    return int((Y1 - y) / S), int((x - X0) / S)


def drawn(img):
    return (img[..., :3] != 255).any(-1)


def test_empty_scene_is_white_and_opaque():
    img = render(custom_level(DIMS))
    assert img.shape == (125, 125, 4) and np.all(img == 255)


def test_box_covers_exactly_its_pixels():
    # pixel centres are at x = 0.05 k and y = 0.025 + 0.05 k; a 1.0 x 0.6 m box at (0.525, 2.0) has its edges
    # between them -> 20 x 12 pixel centres
    img = render(custom_level(DIMS, polygons=[dict(half=(0.5, 0.3), pos=(0.525, 2.0))]))
    m = drawn(img)
    assert m.sum() == 20 * 12
    rows, cols = np.nonzero(m)
    r0, c0 = pixel_of(0.05, 2.275)
    assert rows.min() == r0 and cols.min() == c0 and rows.max() == r0 + 11 and cols.max() == c0 + 19
    assert np.all(img[m][:, :3] == 128) and np.all(img[..., 3] == 255)


def test_circle_area_and_symmetry():
    r = 0.8
    img = render(custom_level(DIMS, circles=[dict(radius=r, pos=(0.0, 3.0))]))
    m = drawn(img)
    area_px = math.pi * r * r / (S * S)
    assert abs(m.sum() - area_px) < 0.02 * area_px
    # the centre (0, 3) lies on a pixel-centre column and between two rows: symmetric about both
    rc, cc = pixel_of(0.0, 3.0)
    sub = m[rc - 20:rc + 20, cc - 20:cc + 21]
    assert np.array_equal(sub, sub[::-1, :]) and np.array_equal(sub, sub[:, ::-1])


def test_rotation_by_a_quarter_turn_swaps_the_extents():
    a = drawn(render(custom_level(DIMS, polygons=[dict(half=(0.6, 0.2), pos=(0.025, 3.0), angle=math.pi / 2)])))
    b = drawn(render(custom_level(DIMS, polygons=[dict(half=(0.2, 0.6), pos=(0.025, 3.0))])))
    # the faces fall between pixel centres, so rounding in the rotation cannot move a pixel across them
    assert a.sum() == b.sum() == 8 * 24 and np.array_equal(a, b)


def test_triangle_area():
    verts = [(-0.6, -0.4), (0.6, -0.4), (0.0, 0.8)]
    img = render(custom_level(DIMS, polygons=[dict(verts=verts, pos=(0.3, 2.0), angle=0.3)]))
    area_px = 0.5 * 1.2 * 1.2 / (S * S)
    assert abs(drawn(img).sum() - area_px) < 0.04 * area_px


def test_roles_fixated_and_draw_order():
    lv = custom_level(DIMS, polygons=[dict(half=(1.0, 1.0), pos=(0.0, 3.0), static=1),
                                      dict(half=(0.5, 0.5), pos=(0.0, 3.0), role=ROLE_RED),
                                      dict(half=(0.25, 0.25), pos=(0.0, 3.0), role=ROLE_BLUE)],
                      circles=[dict(radius=0.1, pos=(0.0, 3.0), role=ROLE_GREEN),
                               dict(radius=0.2, pos=(2.0, 1.0))])
    img = render(lv)
    at = lambda x, y: tuple(int(v) for v in img[pixel_of(x, y)][:3])
    assert at(0.02, 3.02) == (0, 200, 0)            # the green circle is the highest index there
    assert at(0.2, 3.2) == (0, 0, 220)              # blue box over the red one
    assert at(0.4, 3.4) == (220, 0, 0)              # red box over the fixated grey one
    assert at(0.9, 3.9) == (64, 64, 64)             # fixated, no role
    assert at(2.02, 1.02) == (128, 128, 128)        # movable, no role
    assert at(-2.0, 5.0) == (255, 255, 255)
    # an inactive shape is not drawn
    lv["active"][0, 1] = 0
    assert tuple(int(v) for v in render(lv)[pixel_of(0.4, 3.4)][:3]) == (64, 64, 64)


def test_f32_and_f64_images_agree_on_a_generated_scene():
    from paper_2410_23208_b200 import scenes
    lv = scenes.make_levels("L", 1, 9)
    a, b = render(lv, f64=True), render(lv, f64=False)
    # pixel centres within rounding of a face may flip; everything else is identical
    assert (a != b).any(-1).sum() <= 8
