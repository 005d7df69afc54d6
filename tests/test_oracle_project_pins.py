"""Pins of the oracle's projection stage against closed forms and brute force (no GPU)."""
import numpy as np
import pytest

from paper_2607_19893_b200 import workloads as wl

SH_DC = 0.28209479177387814


def one_splat(mean, ls, q, logit=0.0, rgb=(0.6, 0.5, 0.4), sh_degree=0):
    k = (sh_degree + 1) ** 2
    sh = np.zeros((1, k, 3))
    sh[0, 0] = (np.asarray(rgb) - 0.5) / SH_DC
    return wl.Scene(sh_degree, np.array([mean], float), np.array([ls], float), np.array([q], float),
                    np.array([logit], float), sh)


def cam_identity(w=64, h=64, f=64.0, bg=(0, 0, 0)):
    return wl._camera(w, h, f, np.concatenate([np.eye(3), np.zeros((3, 1))], axis=1), bg=bg)


def test_sh_basis_is_orthonormal(oracle64):
    # Gauss-Legendre in cos(theta) x uniform in phi integrates degree<=6 polynomials exactly.
    xs, ws = np.polynomial.legendre.leggauss(12)
    nphi = 24
    gram = np.zeros((16, 16))
    for ct, w in zip(xs, ws):
        st = np.sqrt(1 - ct * ct)
        for j in range(nphi):
            phi = 2 * np.pi * (j + 0.5) / nphi
            y = oracle64.sh_basis(3, st * np.cos(phi), st * np.sin(phi), ct)
            gram += w * (2 * np.pi / nphi) * np.outer(y, y)
    assert np.allclose(gram, np.eye(16), atol=1e-12)


def test_sh_degree0_colour(oracle64):
    s = one_splat((0.1, -0.2, 4.0), (-2, -2, -2), (1, 0, 0, 0), rgb=(0.9, 0.25, 0.5))
    p = oracle64.project(s, cam_identity())
    assert np.allclose(p.rgb[0], SH_DC * s.sh[0, 0] + 0.5, atol=1e-14)
    assert np.allclose(p.rgb[0], (0.9, 0.25, 0.5), atol=1e-14)


def test_sh_colour_clamps_at_zero_and_flags(oracle64):
    s = one_splat((0.0, 0.0, 4.0), (-2, -2, -2), (1, 0, 0, 0), rgb=(-0.2, 0.5, 1.3))
    p = oracle64.project(s, cam_identity())
    assert p.rgb[0, 0] == 0.0 and p.clamp_flags[0] == 1
    assert np.allclose(p.rgb[0, 1:], (0.5, 1.3))


def test_sh_degree1_direction_dependence(oracle64):
    # Y_2 = sqrt(3/4pi) z: a coefficient on k=2 adds C1 * d_z to the colour
    s = one_splat((0.0, 0.0, 5.0), (-2, -2, -2), (1, 0, 0, 0), rgb=(0.5, 0.5, 0.5), sh_degree=1)
    s.sh[0, 2, :] = (0.1, 0.2, 0.3)
    p = oracle64.project(s, cam_identity())
    c1 = np.sqrt(3 / (4 * np.pi))
    assert np.allclose(p.rgb[0], 0.5 + c1 * 1.0 * np.array([0.1, 0.2, 0.3]), atol=1e-14)


@pytest.mark.parametrize("q", [(1, 0, 0, 0), (0.3, -0.5, 0.7, 0.2), (-0.3, 0.5, -0.7, -0.2), (2.0, 1.0, -4.0, 0.5)])
def test_isotropic_on_axis_closed_form(oracle64, q):
    s0, z, f = np.exp(-2.0), 4.0, 64.0
    s = one_splat((0.0, 0.0, z), (-2, -2, -2), q, logit=0.3)
    p = oracle64.project(s, cam_identity(f=f))
    var = (f * s0 / z) ** 2 + 0.3
    assert np.allclose(p.conic_o[0, :3], (1 / var, 0.0, 1 / var), atol=1e-12)
    assert np.isclose(p.conic_o[0, 3], 1 / (1 + np.exp(-0.3)))
    assert p.radius[0] == int(np.ceil(3 * np.sqrt(var)))
    assert np.allclose(p.xy[0], (32.0, 32.0)) and np.isclose(p.depth[0], z)


def test_isotropic_off_axis_closed_form(oracle64):
    # Sigma' = s^2 J J^T + 0.3 I with J the pinhole Jacobian at t
    s0, f = np.exp(-2.5), 80.0
    t = np.array([0.5, -0.3, 3.0])
    s = one_splat(t, (-2.5,) * 3, (0.9, 0.1, 0.2, -0.3))
    p = oracle64.project(s, cam_identity(f=f))
    J = np.array([[f / t[2], 0, -f * t[0] / t[2] ** 2], [0, f / t[2], -f * t[1] / t[2] ** 2]])
    cov = s0 ** 2 * J @ J.T + 0.3 * np.eye(2)
    inv = np.linalg.inv(cov)
    assert np.allclose(p.conic_o[0, :3], (inv[0, 0], inv[0, 1], inv[1, 1]), rtol=1e-12)
    assert np.allclose(p.xy[0], (f * t[0] / t[2] + 32, f * t[1] / t[2] + 32))


def test_axis_aligned_anisotropic_and_rotation(oracle64):
    f, z = 64.0, 4.0
    ls = np.array([-1.0, -2.0, -3.0])
    s = one_splat((0, 0, z), ls, (1, 0, 0, 0))
    p = oracle64.project(s, cam_identity(f=f))
    vx, vy = (f * np.exp(ls[0]) / z) ** 2 + 0.3, (f * np.exp(ls[1]) / z) ** 2 + 0.3
    assert np.allclose(p.conic_o[0, :3], (1 / vx, 0, 1 / vy), atol=1e-12)
    # 90 degrees about z swaps the x and y extents
    c = np.cos(np.pi / 4)
    p2 = oracle64.project(one_splat((0, 0, z), ls, (c, 0, 0, c)), cam_identity(f=f))
    assert np.allclose(p2.conic_o[0, :3], (1 / vy, 0, 1 / vx), atol=1e-12)
    # 90 degrees about y brings the z extent onto x
    p3 = oracle64.project(one_splat((0, 0, z), ls, (c, 0, c, 0)), cam_identity(f=f))
    vz = (f * np.exp(ls[2]) / z) ** 2 + 0.3
    assert np.allclose(p3.conic_o[0, :3], (1 / vz, 0, 1 / vy), atol=1e-12)


def test_general_covariance_against_numpy(oracle64):
    rng = np.random.default_rng(5)
    scene, cam = wl.tiny_scene(11, 40, 0)
    p = oracle64.project(scene, cam)
    R_c, t_c = cam.w2c[:, :3], cam.w2c[:, 3]
    for i in range(scene.n):
        if p.tiles_touched[i] == 0:
            continue
        w, x, y, z = scene.quats[i] / np.linalg.norm(scene.quats[i])
        # rotation by the textbook sandwich product q v q*, column by column
        def rot(v):
            qv = np.array([x, y, z])
            return v + 2 * np.cross(qv, np.cross(qv, v) + w * v)
        R = np.stack([rot(e) for e in np.eye(3)], axis=1)
        S = np.diag(np.exp(scene.log_scales[i]))
        Sig = R @ S @ S @ R.T
        t = R_c @ scene.means[i] + t_c
        J = np.array([[cam.fx / t[2], 0, -cam.fx * t[0] / t[2] ** 2], [0, cam.fy / t[2], -cam.fy * t[1] / t[2] ** 2]])
        cov = J @ R_c @ Sig @ R_c.T @ J.T + 0.3 * np.eye(2)
        inv = np.linalg.inv(cov)
        assert np.allclose(p.conic_o[i, :3], (inv[0, 0], inv[0, 1], inv[1, 1]), rtol=1e-10)
        lam = np.linalg.eigvalsh(cov)[-1]
        assert p.radius[i] == int(np.ceil(3 * np.sqrt(lam)))
    assert rng is not None


def test_jacobian_clamp_freezes_ratio(oracle64):
    # far off axis: t_x/t_z beyond 1.3 * (W/2)/fx = 0.65 is clamped inside J only
    f, t = 64.0, np.array([3.0, 0.0, 2.0])
    s0 = np.exp(-2.0)
    p = oracle64.project(one_splat(t, (-2,) * 3, (1, 0, 0, 0)), cam_identity(f=f))
    lim = 1.3 * 64 / (2 * f)
    J = np.array([[f / t[2], 0, -f * lim / t[2]], [0, f / t[2], 0.0]])
    inv = np.linalg.inv(s0 ** 2 * J @ J.T + 0.3 * np.eye(2))
    # the splat is off screen and may be culled by its rectangle; compare only if kept
    if p.tiles_touched[0]:
        assert np.allclose(p.conic_o[0, :3], (inv[0, 0], inv[0, 1], inv[1, 1]), rtol=1e-12)
    big = oracle64.project(one_splat(t, (0.5,) * 3, (1, 0, 0, 0)), cam_identity(f=f))
    assert big.tiles_touched[0] > 0
    inv = np.linalg.inv(np.exp(0.5) ** 2 * J @ J.T + 0.3 * np.eye(2))
    assert np.allclose(big.conic_o[0, :3], (inv[0, 0], inv[0, 1], inv[1, 1]), rtol=1e-12)
    assert np.isclose(big.xy[0, 0], f * 1.5 + 32)  # the pixel centre is not clamped


def test_depth_cull_and_lateral_cull(oracle64):
    cam = cam_identity()
    cam.znear, cam.zfar = 0.2, 50.0
    for z, vis in [(0.1, False), (0.2, False), (0.21, True), (49.0, True), (50.0, False), (-3.0, False)]:
        p = oracle64.project(one_splat((0, 0, z), (-3,) * 3, (1, 0, 0, 0)), cam)
        assert (p.tiles_touched[0] > 0) == vis
    p = oracle64.project(one_splat((40.0, 0, 4.0), (-3,) * 3, (1, 0, 0, 0)), cam)
    assert p.tiles_touched[0] == 0 and np.all(p.conic_o[0] == 0)


def test_rect_covers_every_pixel_within_radius(oracle32):
    w = wl.make_workload(2, n=4000)
    cam = w.cameras[3]
    p = oracle32.project(w.scene, cam)
    tx, ty = oracle32.grid(cam)
    vis = np.nonzero(p.tiles_touched)[0]
    assert len(vis) > 500
    px = np.arange(cam.width) + 0.5
    py = np.arange(cam.height) + 0.5
    for i in vis[:400]:
        x0, y0, x1, y1 = p.rect[i]
        assert 0 <= x0 < x1 <= tx and 0 <= y0 < y1 <= ty
        assert p.tiles_touched[i] == (x1 - x0) * (y1 - y0)
        inx = px[np.abs(px - p.xy[i, 0]) <= p.radius[i]]
        iny = py[np.abs(py - p.xy[i, 1]) <= p.radius[i]]
        if len(inx):
            assert x0 <= int(inx.min() // 16) and int(inx.max() // 16) < x1
        if len(iny):
            assert y0 <= int(iny.min() // 16) and int(iny.max() // 16) < y1
    # culled primitives carry zeros
    cul = p.tiles_touched == 0
    assert np.all(p.radius[cul] == 0) and np.all(p.rect[cul] == 0)


def test_radius_monotone_in_scale(oracle64):
    last = 0
    for ls in np.linspace(-4, 0, 9):
        p = oracle64.project(one_splat((0.2, 0.1, 4.0), (ls,) * 3, (1, 0, 0, 0)), cam_identity())
        assert p.radius[0] >= last
        last = p.radius[0]


def test_float_and_double_instantiations_agree(oracle32, oracle64):
    w = wl.make_workload(2, n=3000)
    a = oracle32.project(w.scene, w.cameras[1])
    b = oracle64.project(w.scene.astype(np.float64), w.cameras[1])
    safe = (a.margin > 1e-4) & (b.margin > 1e-4)
    assert safe.mean() > 0.95
    assert np.array_equal(a.tiles_touched[safe], b.tiles_touched[safe])
    assert np.array_equal(a.rect[safe], b.rect[safe])
    v = safe & (a.tiles_touched > 0)
    assert np.allclose(a.conic_o[v], b.conic_o[v], rtol=2e-4, atol=1e-6)
    assert np.allclose(a.xy[v], b.xy[v], atol=2e-3)
    assert np.allclose(a.rgb[v], b.rgb[v], atol=1e-5)
