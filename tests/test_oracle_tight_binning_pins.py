"""Pins of the oracle's tight-extent binning mode (an optimised-pipeline variant in the sense of Sec. 5: same
primitive-id namespace, same image): coverage by brute force, a closed form, identity of images and gradients with the
plain rectangle, and that it actually removes instances (no GPU)."""
import numpy as np

import oracle
from oracle.oracle import DEFAULT_CFG
from paper_2607_19893_b200 import workloads as wl
from test_oracle_project_pins import cam_identity, one_splat


def tight(dtype):
    cfg = DEFAULT_CFG.copy()
    cfg[7] = 1
    return oracle.Oracle(dtype, cfg=cfg)


def test_tight_rectangle_lies_inside_the_plain_one_and_covers_every_contributing_pixel(oracle64):
    w = wl.make_workload(2, n=4000)
    cam = w.cameras[1]
    p0, p1 = oracle64.project(w.scene, cam), tight(np.float64).project(w.scene, cam)
    vis0, vis1 = p0.tiles_touched > 0, p1.tiles_touched > 0
    assert not (vis1 & ~vis0).any()
    r0, r1 = p0.rect[vis1], p1.rect[vis1]
    assert np.all(r1[:, 0] >= r0[:, 0]) and np.all(r1[:, 1] >= r0[:, 1])
    assert np.all(r1[:, 2] <= r0[:, 2]) and np.all(r1[:, 3] <= r0[:, 3])
    # everything but the rectangle is untouched
    assert np.array_equal(p0.xy[vis1], p1.xy[vis1]) and np.array_equal(p0.conic_o[vis1], p1.conic_o[vis1])
    assert int(p1.tiles_touched.sum()) < 0.9 * int(p0.tiles_touched.sum())   # ~2 px splats: tile rounding dominates
    # brute force: every pixel of the plain rectangle whose alpha reaches 1/255 lies in a tile of the tight rectangle
    checked = 0
    for q in np.flatnonzero(vis0)[:600]:
        x0, y0, x1, y1 = p0.rect[q]
        xs = np.arange(16 * x0, min(16 * x1, cam.width)) + 0.5
        ys = np.arange(16 * y0, min(16 * y1, cam.height)) + 0.5
        dx, dy = p0.xy[q, 0] - xs[None, :], p0.xy[q, 1] - ys[:, None]
        A, B, C, o = p0.conic_o[q]
        power = -0.5 * (A * dx * dx + C * dy * dy) - B * dx * dy
        hit = (power <= 0) & (np.minimum(0.99, o * np.exp(power)) >= 1.0 / 255.0)
        jj, ii = np.nonzero(hit)
        if len(jj) == 0:
            continue
        tx, ty = (16 * x0 + ii) // 16, (16 * y0 + jj) // 16
        a0, b0, a1, b1 = p1.rect[q]
        assert p1.tiles_touched[q] > 0
        assert tx.min() >= a0 and tx.max() < a1 and ty.min() >= b0 and ty.max() < b1
        checked += 1
    assert checked > 300


def test_tight_extent_closed_form_for_an_isotropic_splat(oracle64):
    """Isotropic splat on the optical axis: Sigma' = (f s / z)^2 + 0.3 on the diagonal, so the extent is
    sqrt(2 ln(o 255) Sigma'_xx) pixels on either side of the centre."""
    f, z, s, lo = 64.0, 4.0, np.exp(0.3), -2.2
    cam = cam_identity(256, 256, f)
    sc = one_splat((0.0, 0.0, z), (np.log(s),) * 3, (1, 0, 0, 0), logit=lo)
    p = tight(np.float64).project(sc, cam)
    var = (f * s / z) ** 2 + 0.3
    ext = np.sqrt(2 * np.log(255 / (1 + np.exp(-lo))) * var)
    u = 128.0
    want_x0 = int(np.floor((u - ext - 0.5) / 16))
    want_x1 = int(np.floor((u + ext - 0.5) / 16)) + 1
    assert p.rect[0].tolist() == [want_x0, want_x0, want_x1, want_x1]
    # the plain rectangle of the same splat is wider: 3 sigma rounded up to whole pixels
    p0 = oracle64.project(sc, cam)
    assert p0.tiles_touched[0] > p.tiles_touched[0]
    # a splat whose opacity is below alpha_min can never contribute: no tiles at all
    faint = one_splat((0.0, 0.0, z), (np.log(s),) * 3, (1, 0, 0, 0), logit=np.log(0.003 / 0.997))
    assert tight(np.float64).project(faint, cam).tiles_touched[0] == 0 and oracle64.project(faint, cam).tiles_touched[0] > 0


def test_tight_binning_leaves_image_and_gradients_unchanged(oracle32):
    for cfg_id, n, view in ((1, None, 0), (2, 20_000, 5)):
        w = wl.make_workload(cfg_id, n=n)
        cam = w.cameras[view]
        t32 = tight(np.float32)
        f0, f1 = oracle32.view_forward(w.scene, cam), t32.view_forward(w.scene, cam)
        assert len(f1["vals"]) < len(f0["vals"])
        # the same pairs blend in the same order: bitwise the same image and transmittance
        assert np.array_equal(f0["out"], f1["out"]) and np.array_equal(f0["final_T"], f1["final_T"])
        dl = np.random.default_rng(3).uniform(-1, 1, f0["out"].shape).astype(np.float32)
        g0 = oracle32.render_bwd_blend(f0["proj"], f0["vals"], f0["ranges"], cam, f0["final_T"], f0["n_contrib"], dl)
        g1 = t32.render_bwd_blend(f1["proj"], f1["vals"], f1["ranges"], cam, f1["final_T"], f1["n_contrib"], dl)
        assert np.allclose(g0, g1, rtol=1e-11, atol=1e-14)  # same terms; the fp64 sums run in thread order
        # the realized active set does not depend on the binning either; primitives dropped from the candidate scope
        # were never active
        _, a0 = oracle32.realized_active(f0["proj"], f0["vals"], f0["ranges"], cam, f0["n_contrib"])
        _, a1 = t32.realized_active(f1["proj"], f1["vals"], f1["ranges"], cam, f1["n_contrib"])
        assert np.array_equal(a0, a1) and set(a1.tolist()) <= set(f1["idx"].tolist()) <= set(f0["idx"].tolist())
