"""Pins of the oracle outputs that set the parity bars (no GPU): the per-primitive decision margin of the projection,
the per-pixel decision margin of the compositing, and the un-cancelled gradient sums `g2d_abs`.

The GPU tests use these three outputs to decide which pixels / primitives may legitimately differ and how large a
gradient difference may be, so each is fixed here by scenes whose margin is known in closed form and, for `g2d_abs`,
by its definition in terms of the (finite-difference pinned) gradient itself.  A margin that came out half as large,
or a `g2d_abs` twice as large, fails these tests.
"""
import numpy as np
import pytest

from paper_2607_19893_b200 import workloads as wl
from test_oracle_project_pins import cam_identity, one_splat
from test_oracle_render_pins import logit, stack_scenes

SQRT01 = np.sqrt(0.1)


def iso_scale_for_radius(rr, f=64.0, z=4.0):
    """Scale s of an isotropic on-axis splat whose 3-sigma extent is rr pixels: Sigma' = ((f s / z)^2 + 0.3) I, the
    radius formula adds sqrt(0.1) to the (double) eigenvalue."""
    lam = (rr / 3.0) ** 2
    return np.sqrt(lam - 0.3 - SQRT01) * z / f


# --------------------------------------------------------------------------------------------- project().margin
def test_project_margin_radius_rounding(oracle64):
    # 3 sigma = 7.9 px -> radius 8, 0.1 px below the integer; centre on a tile corner + 8: edges at 1.5 and 2.5 tiles
    s = one_splat((0, 0, 4.0), (np.log(iso_scale_for_radius(7.9)),) * 3, (1, 0, 0, 0))
    p = oracle64.project(s, cam_identity())
    assert p.radius[0] == 8 and tuple(p.rect[0]) == (1, 1, 3, 3)
    assert p.margin[0] == pytest.approx(0.1 / 7.9, rel=1e-9)
    # 3 sigma = 8.02 px -> radius 9, 0.02 above the integer below it
    s = one_splat((0, 0, 4.0), (np.log(iso_scale_for_radius(8.02)),) * 3, (1, 0, 0, 0))
    p = oracle64.project(s, cam_identity(w=66, h=66))  # cx = 33: edges (33 -+ 9) / 16 = 1.5, 2.625
    assert p.radius[0] == 9
    assert p.margin[0] == pytest.approx(0.02 / 8.02, rel=1e-9)


def test_project_margin_rectangle_edge(oracle64):
    # radius 8 from 7.5 (margin 0.0667); the principal point is shifted so that the left edge is 0.01 tile past a
    # tile boundary: (24.16 - 8) / 16 = 1.01, (24.16 + 8) / 16 = 2.01 -> min(0.01 / 1.01, 0.01 / 2.01)
    s = one_splat((0, 0, 4.0), (np.log(iso_scale_for_radius(7.5)),) * 3, (1, 0, 0, 0))
    cam = cam_identity()
    cam.cx = 24.16
    p = oracle64.project(s, cam)
    assert tuple(p.rect[0]) == (1, 1, 3, 3)
    assert p.margin[0] == pytest.approx(0.01 / 2.01, rel=1e-9)
    # the same distance on the other side of the boundary changes the rectangle and keeps the margin's size
    cam.cx = 23.84  # (23.84 - 8) / 16 = 0.99, (23.84 + 8) / 16 = 1.99
    p = oracle64.project(s, cam)
    assert tuple(p.rect[0]) == (0, 1, 2, 3)
    assert p.margin[0] == pytest.approx(0.01 / 1.99, rel=1e-9)


def test_project_margin_depth_plane_colour_and_jacobian_clamp(oracle64):
    ls = (np.log(iso_scale_for_radius(7.5, z=0.2 * 1.003)),) * 3
    cam = cam_identity()
    # just behind / just in front of the near plane (znear = 0.2)
    p = oracle64.project(one_splat((0, 0, 0.2 * 1.003), ls, (1, 0, 0, 0)), cam)
    assert p.tiles_touched[0] > 0 and p.margin[0] == pytest.approx(0.003, rel=1e-9)
    p = oracle64.project(one_splat((0, 0, 0.2 * 0.998), ls, (1, 0, 0, 0)), cam)
    assert p.tiles_touched[0] == 0 and p.margin[0] == pytest.approx(0.002, rel=1e-9)
    # a colour channel 0.004 above its clamp at 0
    s = one_splat((0, 0, 4.0), (np.log(iso_scale_for_radius(7.5)),) * 3, (1, 0, 0, 0), rgb=(0.6, 0.004, 0.5))
    assert oracle64.project(s, cam).margin[0] == pytest.approx(0.004, rel=1e-9)
    # t_x / t_z = 1.001 x the guard 1.3 * W / (2 fx); a wide image so the splat is still on screen
    cam = cam_identity(w=640, h=64, f=64.0)
    lim = 1.3 * 640 / (2 * 64.0)
    s = one_splat((lim * 1.001 * 4.0, 0, 4.0), (-1.0,) * 3, (1, 0, 0, 0))
    p = oracle64.project(s, cam)
    assert p.tiles_touched[0] > 0 and p.margin[0] == pytest.approx(0.001, rel=1e-9)


def test_project_margin_is_one_far_from_every_decision(oracle64):
    # culled far behind the camera: only the depth planes are looked at, both far away
    p = oracle64.project(one_splat((0, 0, -5.0), (-2,) * 3, (1, 0, 0, 0)), cam_identity())
    assert p.tiles_touched[0] == 0 and p.margin[0] == 1.0


# --------------------------------------------------------------------------------------------- render_fwd().pix_margin
def one_pixel_cam(bg=(0, 0, 0)):
    return wl._camera(1, 1, 64.0, np.concatenate([np.eye(3), np.zeros((3, 1))], axis=1), bg=bg)


def coaxial(opacities):
    """Splats centred on the single pixel's centre (dx = dy = 0, so G = 1 and alpha = min(0.99, opacity))."""
    return stack_scenes([one_splat((0, 0, 2.0 + 0.1 * i), (-2,) * 3, (1, 0, 0, 0), logit=logit(o))
                         for i, o in enumerate(opacities)])


@pytest.mark.parametrize("delta", [0.05, -0.05, 0.003])
def test_pix_margin_alpha_skip_threshold(oracle64, delta):
    f = oracle64.view_forward(coaxial([(1 + delta) / 255.0]), one_pixel_cam())
    assert f["pix_margin"][0, 0] == pytest.approx(abs(delta), rel=1e-7)
    assert f["n_contrib"][0, 0] == (1 if delta > 0 else 0)


@pytest.mark.parametrize("delta", [0.008, -0.04])
def test_pix_margin_alpha_clamp(oracle64, delta):
    # o * G = 0.99 (1 + delta); on the clamped side T' = 0.01 is far from 1e-4 and alpha far from 1/255
    o = 0.99 * (1 + delta)
    f = oracle64.view_forward(coaxial([o]), one_pixel_cam())
    assert f["pix_margin"][0, 0] == pytest.approx(abs(delta), rel=1e-7)
    assert f["final_T"][0, 0] == pytest.approx(1 - min(0.99, o), rel=1e-9)


@pytest.mark.parametrize("delta", [0.02, -0.02])
def test_pix_margin_termination_threshold(oracle64, delta):
    # twelve splats of alpha 0.5 leave T = 2^-12; the thirteenth would leave T' = 1e-4 (1 + delta)
    a_last = 1 - 1e-4 * (1 + delta) / 0.5 ** 12
    f = oracle64.view_forward(coaxial([0.5] * 12 + [a_last]), one_pixel_cam())
    assert f["pix_margin"][0, 0] == pytest.approx(abs(delta), rel=1e-6)
    assert f["n_contrib"][0, 0] == (13 if delta > 0 else 12)  # stop BEFORE the splat that would cross the threshold


def test_pix_margin_power_sign_and_untouched_pixels(oracle64):
    # an isotropic splat has B = 0: power = -(|q1| + |q2|) / 2 exactly, relative margin of the sign test 1; a pixel
    # far outside every rectangle traverses nothing and keeps margin 1
    s = one_splat((0, 0, 4.0), (np.log(iso_scale_for_radius(7.5)),) * 3, (1, 0, 0, 0), logit=logit(0.3))
    f = oracle64.view_forward(s, cam_identity())
    assert f["pix_margin"][0, 0] == 1.0 and f["n_contrib"][0, 0] == 0
    # along the row through the centre alpha = 0.3 exp(-dx^2 / (2 sigma'^2)); the margin of a pixel is its relative
    # distance to 1/255 (the clamp and the termination are farther away for alpha < 0.3)
    sig2 = (7.5 / 3.0) ** 2 - SQRT01
    for i in (26, 29, 31):
        dx = 32.0 - (i + 0.5)
        dy = 32.0 - 31.5
        alpha = 0.3 * np.exp(-(dx * dx + dy * dy) / (2 * sig2))
        want = min(abs(alpha - 1 / 255) * 255, abs(alpha - 0.99) / 0.99, abs((1 - alpha) - 1e-4) / 1e-4, 1.0)
        assert f["pix_margin"][31, i] == pytest.approx(want, rel=1e-9)


# --------------------------------------------------------------------------------------------- render_bwd_blend().g2d_abs
def blend_inputs(o, seed, n=8, sh_degree=0, size=16):
    s, cam = wl.tiny_scene(seed, n, sh_degree, width=size, height=size, f=20.0)
    f = o.view_forward(s, cam)
    return s, cam, f


def test_g2d_abs_is_the_sum_of_the_absolute_per_pixel_terms(oracle64):
    """With an incoming gradient on ONE pixel every gradient word is a single term per splat, so |g2d| of that run is
    the absolute term itself; g2d_abs of a full incoming gradient must equal the sum of those over the pixels."""
    s, cam, f = blend_inputs(oracle64, 41)
    rng = np.random.default_rng(5)
    dL = rng.uniform(-1, 1, (3, cam.height, cam.width))
    args = (f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"])
    g2d, g2d_abs = oracle64.render_bwd_blend(*args, dL, want_abs=True)
    acc_abs = np.zeros_like(g2d)
    acc = np.zeros_like(g2d)
    for j in range(cam.height):
        for i in range(cam.width):
            one = np.zeros_like(dL)
            one[:, j, i] = dL[:, j, i]
            g = oracle64.render_bwd_blend(*args, one)
            acc += g
            # the three colour words are one term per CHANNEL: split the pixel's gradient by channel for them
            acc_abs[:, :6] += np.abs(g[:, :6])
            for ch in range(3):
                one_ch = np.zeros_like(dL)
                one_ch[ch, j, i] = dL[ch, j, i]
                acc_abs[:, 6 + ch] += np.abs(oracle64.render_bwd_blend(*args, one_ch)[:, 6 + ch])
    assert np.abs(g2d).max() > 1e-3
    assert np.allclose(acc, g2d, rtol=1e-10, atol=1e-14)          # linearity (sanity of the decomposition)
    assert np.allclose(acc_abs, g2d_abs, rtol=1e-10, atol=1e-14)  # the pin
    assert (g2d_abs > 1.5 * np.abs(g2d)).any()                    # mixed signs really occur in this scene


def test_g2d_abs_single_sign_case_and_triangle_inequality(oracle64):
    # one splat, black background, positive incoming gradient: every per-pixel term of the colour and opacity words
    # is positive and every term of the A and C words negative, so the absolute sums are the sums themselves
    s = one_splat((0.05, -0.03, 4.0), (-1.9, -2.2, -2.0), (0.9, 0.2, -0.3, 0.1), logit=logit(0.6), rgb=(0.9, 0.4, 0.7))
    cam = cam_identity(w=32, h=32, f=48.0)
    f = oracle64.view_forward(s, cam)
    dL = np.random.default_rng(2).uniform(0.1, 1.0, (3, 32, 32))
    g2d, g2d_abs = oracle64.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], dL,
                                             want_abs=True)
    assert np.allclose(g2d_abs[0, 5:9], g2d[0, 5:9], rtol=1e-12) and np.all(g2d[0, 5:9] > 0)
    assert np.allclose(g2d_abs[0, [2, 4]], -g2d[0, [2, 4]], rtol=1e-12)
    # the centre words change sign across the splat: strictly larger than the cancelled sum
    assert np.all(g2d_abs[0, [0, 1, 3]] > 1.01 * np.abs(g2d[0, [0, 1, 3]]))
    # general scene: triangle inequality on every word, invariance under dL -> -dL, homogeneity
    s, cam, f = blend_inputs(oracle64, 43, n=12, sh_degree=1)
    dL = np.random.default_rng(3).uniform(-1, 1, (3, cam.height, cam.width))
    args = (f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"])
    g2d, g2d_abs = oracle64.render_bwd_blend(*args, dL, want_abs=True)
    assert np.all(np.abs(g2d) <= g2d_abs * (1 + 1e-12) + 1e-300)
    g2d_n, g2d_abs_n = oracle64.render_bwd_blend(*args, -dL, want_abs=True)
    assert np.array_equal(g2d_abs_n, g2d_abs) and np.array_equal(g2d_n, -g2d)
    _, g2d_abs_2 = oracle64.render_bwd_blend(*args, 2 * dL, want_abs=True)
    assert np.allclose(g2d_abs_2, 2 * g2d_abs, rtol=1e-13)


def test_g2d_abs_two_pixels_of_opposite_sign(oracle64):
    # isotropic splat centred between two horizontally adjacent pixels, incoming gradients +g and -g: the colour
    # words cancel exactly, their absolute sum is twice the single term alpha T g = o exp(-d^2 / 2 sigma'^2) g
    cam = cam_identity()
    s = one_splat((0, 0, 4.0), (np.log(iso_scale_for_radius(7.5)),) * 3, (1, 0, 0, 0), logit=logit(0.5))
    f = oracle64.view_forward(s, cam)
    dL = np.zeros((3, 64, 64))
    dL[:, 31, 31] = 0.25    # pixel centres (31.5, 31.5) and (32.5, 31.5): mirror images about u = 32
    dL[:, 31, 32] = -0.25
    g2d, g2d_abs = oracle64.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], dL,
                                             want_abs=True)
    sig2 = (7.5 / 3.0) ** 2 - SQRT01
    term = 0.5 * np.exp(-(0.25 + 0.25) / (2 * sig2)) * 0.25
    assert np.allclose(g2d[0, 6:9], 0.0, atol=1e-15)
    assert np.allclose(g2d_abs[0, 6:9], 2 * term, rtol=1e-9)
