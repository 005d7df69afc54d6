"""Pins of the oracle's exact binning mode (binning = 2; an optimised-pipeline variant in the sense of Sec. 5: same
primitive-id namespace, same image): a primitive keeps only the tiles of its rectangle that the region alpha >=
alpha_min reaches.  Pinned by brute force over pixels and over a dense sampling of the tile rectangle, by the closed form
for a circular footprint, by the kept tiles of a tile row being an interval, and by identity of image, gradients and
realized active set with the plain rectangle (no GPU)."""
import numpy as np

import oracle
from oracle.oracle import DEFAULT_CFG
from paper_2607_19893_b200 import workloads as wl
from test_oracle_project_pins import cam_identity, one_splat
from test_oracle_render_pins import logit


def exact(dtype):
    cfg = DEFAULT_CFG.copy()
    cfg[7] = 2
    return oracle.Oracle(dtype, cfg=cfg)


def kept_tiles(p, q):
    x0, y0, x1, y1 = p.rect[q]
    out = set()
    for j, ty in enumerate(range(y0, y1)):
        xa, xb = p.span_x[p.span_ptr[q] + j]
        out.update((tx, ty) for tx in range(xa, xb))
    return out


def test_kept_tiles_cover_every_contributing_pixel_and_lie_inside_the_rectangle(oracle64):
    w = wl.make_workload(3, n=6000, resolution=(400, 267))
    cam = w.cameras[1]
    p0, p2 = oracle64.project(w.scene, cam), exact(np.float64).project(w.scene, cam)
    vis0, vis2 = p0.tiles_touched > 0, p2.tiles_touched > 0
    assert not (vis2 & ~vis0).any()
    assert np.array_equal(p0.xy[vis2], p2.xy[vis2]) and np.array_equal(p0.conic_o[vis2], p2.conic_o[vis2])
    assert np.array_equal(p0.rect[vis2], p2.rect[vis2])            # the rectangle itself is the plain one
    assert int(p2.tiles_touched.sum()) < 0.75 * int(p0.tiles_touched.sum())
    checked = dropped_with_pixels = 0
    for q in np.flatnonzero(vis0)[:500]:
        x0, y0, x1, y1 = p0.rect[q]
        xs = np.arange(16 * x0, min(16 * x1, cam.width)) + 0.5
        ys = np.arange(16 * y0, min(16 * y1, cam.height)) + 0.5
        dx, dy = p0.xy[q, 0] - xs[None, :], p0.xy[q, 1] - ys[:, None]
        A, B, C, o = p0.conic_o[q]
        power = -0.5 * (A * dx * dx + C * dy * dy) - B * dx * dy
        hit = (power <= 0) & (np.minimum(0.99, o * np.exp(power)) >= 1.0 / 255.0)
        jj, ii = np.nonzero(hit)
        need = set(zip(((16 * x0 + ii) // 16).tolist(), ((16 * y0 + jj) // 16).tolist()))
        if not vis2[q]:
            assert not need  # a primitive that lost every tile contributes nowhere
            continue
        kept = kept_tiles(p2, q)
        assert need <= kept
        assert all(x0 <= tx < x1 and y0 <= ty < y1 for tx, ty in kept)
        assert len(kept) == p2.tiles_touched[q]
        checked += 1
    assert checked > 250


def test_tile_decision_against_a_dense_sampling_of_the_tile_rectangle(oracle64):
    """min of q over the rectangle of the tile's pixel centres, by brute force on a 151 x 151 grid (an upper bound of
    the true minimum, 1e-2 of a pixel apart): well below the threshold the tile must be kept, well above it dropped."""
    rng = np.random.default_rng(11)
    o = exact(np.float64)
    decided = [0, 0]
    for _ in range(4000):
        s1, s2 = rng.uniform(0.8, 30.0, 2)
        th = rng.uniform(0, np.pi)
        R = np.array([[np.cos(th), -np.sin(th)], [np.sin(th), np.cos(th)]])
        cov = R @ np.diag([s1 * s1, s2 * s2]) @ R.T
        con = np.linalg.inv(cov)
        A, B, C = con[0, 0], con[0, 1], con[1, 1]
        opac = rng.uniform(0.002, 0.99)
        u, v = rng.uniform(0, 160, 2)
        tx, ty = rng.integers(0, 10, 2)
        g = np.linspace(0, 15, 151)
        dx = (16 * tx + 0.5 + g)[None, :] - u
        dy = (16 * ty + 0.5 + g)[:, None] - v
        qmin = (A * dx * dx + 2 * B * dx * dy + C * dy * dy).min()
        got = o.tile_reached(u, v, (A, B, C, opac), int(tx), int(ty))
        if opac < 1 / 255:
            assert not got
            continue
        k = 2 * np.log(opac * 255)
        if qmin < 0.97 * k - 1e-2:
            assert got
            decided[0] += 1
        elif qmin > 1.03 * k + 0.1:
            assert not got
            decided[1] += 1
    assert decided[0] > 300 and decided[1] > 300


def test_circular_footprint_closed_form(oracle64):
    # isotropic splat on the axis: q = d^2 / var, so a tile is kept iff the distance from the centre to the rectangle of
    # its pixel centres is at most sqrt(bound * var), bound = k (1 + 1e-4) + 1e-3 + 2e-6 * (far-corner value of q)
    f, z, s, lo = 64.0, 4.0, np.exp(1.0), 0.4
    cam = cam_identity(512, 512, f)
    p = exact(np.float64).project(one_splat((0.0, 0.0, z), (np.log(s),) * 3, (1, 0, 0, 0), logit=lo), cam)
    var = (f * s / z) ** 2 + 0.3
    opac = 1 / (1 + np.exp(-lo))
    k = 2 * np.log(opac * 255)
    kept = kept_tiles(p, 0)
    x0, y0, x1, y1 = p.rect[0]
    n_border = 0
    for ty in range(y0, y1):
        for tx in range(x0, x1):
            xl, yl = 16 * tx + 0.5 - 256.0, 16 * ty + 0.5 - 256.0
            ddx = 0.0 if xl <= 0 <= xl + 15 else min(abs(xl), abs(xl + 15))
            ddy = 0.0 if yl <= 0 <= yl + 15 else min(abs(yl), abs(yl + 15))
            far = max(abs(xl), abs(xl + 15)) ** 2 + max(abs(yl), abs(yl + 15)) ** 2
            bound = k * 1.0001 + 1e-3 + 2e-6 * (far / var) * 1.0
            want = (ddx * ddx + ddy * ddy) / var <= bound
            # the oracle's `big` adds a cross term that is zero here (B = 0): the same expression
            assert ((tx, ty) in kept) == want, (tx, ty)
            n_border += want != ((ddx * ddx + ddy * ddy) / var <= 0.5 * k)
    assert len(kept) > 20 and n_border > 8 and len(kept) < (x1 - x0) * (y1 - y0)  # the corners of the rectangle go


def test_kept_tiles_of_a_tile_row_form_an_interval(oracle64):
    w = wl.make_workload(4, n=3000, resolution=(480, 270))
    cam = w.cameras[2]
    o = exact(np.float64)
    p = o.project(w.scene, cam)
    for q in np.flatnonzero(p.tiles_touched)[:150]:
        x0, y0, x1, y1 = p.rect[q]
        single = sum(o.tile_reached(p.xy[q, 0], p.xy[q, 1], p.conic_o[q], tx, ty) for ty in range(y0, y1)
                     for tx in range(x0, x1))
        assert single == p.tiles_touched[q]  # no gap inside any span


def test_image_gradients_and_active_set_equal_those_of_the_plain_rectangle(oracle64):
    w = wl.make_workload(2, n=3000)
    s, cam = w.scene.astype(np.float64), w.cameras[3]
    o0, o2 = oracle64, exact(np.float64)
    f0, f2 = o0.view_forward(s, cam), o2.view_forward(s, cam)
    assert len(f2["keys"]) < len(f0["keys"])
    assert np.array_equal(f0["out"], f2["out"]) and np.array_equal(f0["final_T"], f2["final_T"])
    dL = np.random.default_rng(4).uniform(-1, 1, f0["out"].shape)
    g0 = o0.render_bwd_blend(f0["proj"], f0["vals"], f0["ranges"], cam, f0["final_T"], f0["n_contrib"], dL)
    g2 = o2.render_bwd_blend(f2["proj"], f2["vals"], f2["ranges"], cam, f2["final_T"], f2["n_contrib"], dL)
    assert np.allclose(g0, g2, rtol=1e-11, atol=1e-15)  # the same terms; the OpenMP accumulation order is not fixed
    a0 = o0.realized_active(f0["proj"], f0["vals"], f0["ranges"], cam, f0["n_contrib"])[1]
    a2 = o2.realized_active(f2["proj"], f2["vals"], f2["ranges"], cam, f2["n_contrib"])[1]
    assert np.array_equal(a0, a2) and len(a0) > 100
    # the touched set shrinks to the primitives that keep a tile, and still contains every active one
    assert set(a2) <= set(f2["idx"]) <= set(f0["idx"])


def test_opacity_below_the_threshold_keeps_no_tile(oracle64):
    sc = one_splat((0.0, 0.0, 4.0), (-1.0,) * 3, (1, 0, 0, 0), logit=logit(0.0038))
    p = exact(np.float64).project(sc, cam_identity())
    assert p.tiles_touched[0] == 0
    sc = one_splat((0.0, 0.0, 4.0), (-1.0,) * 3, (1, 0, 0, 0), logit=logit(0.0040))
    assert exact(np.float64).project(sc, cam_identity()).tiles_touched[0] >= 1
