"""Pins of the oracle's backward pass, Adam and set algebra (no GPU)."""
import os

import numpy as np
import pytest
import torch

from paper_2607_19893_b200 import workloads as wl
from test_oracle_project_pins import cam_identity, one_splat
from test_oracle_render_pins import logit

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def flat_params(s):
    return np.concatenate([s.means.ravel(), s.log_scales.ravel(), s.quats.ravel(), s.opacity_logit.ravel(), s.sh.ravel()])


def set_flat(s, x):
    o = 0
    for a in (s.means, s.log_scales, s.quats, s.opacity_logit, s.sh):
        a[...] = x[o:o + a.size].reshape(a.shape)
        o += a.size


def rows_to_flat(rows, idx, s):
    """Scatter compact gradient rows [V,F] into the flat parameter order of flat_params."""
    n, k = s.n, s.sh_k
    g = s.zeros_like()
    g.means[idx] = rows[:, 0:3]
    g.log_scales[idx] = rows[:, 3:6]
    g.quats[idx] = rows[:, 6:10]
    g.opacity_logit[idx] = rows[:, 10]
    g.sh[idx] = rows[:, 11:].reshape(-1, k, 3)
    assert g.means.shape[0] == n
    return flat_params(g)


def weighted_loss(o, s, cam, wgt):
    return float((o.view_forward(s, cam)["out"] * wgt).sum())


def analytic(o, s, cam, wgt):
    f = o.view_forward(s, cam)
    g2d = o.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], wgt)
    rows = o.render_bwd_project(s, cam, f["idx"], g2d, f["proj"].clamp_flags)
    return f, g2d, rows


@pytest.mark.parametrize("seed,sh_degree,n", [(21, 3, 6), (22, 0, 8), (23, 2, 5), (24, 1, 7)])
def test_gradients_match_central_differences(oracle64, seed, sh_degree, n):
    s, cam = wl.tiny_scene(seed, n, sh_degree)
    wgt = np.random.default_rng(seed).uniform(-1, 1, (3, cam.height, cam.width))
    f, g2d, rows = analytic(oracle64, s, cam, wgt)
    # the scene must sit away from every decision threshold, otherwise differences are meaningless
    assert f["pix_margin"].min() > 1e-6 and f["proj"].margin.min() > 1e-6
    assert len(f["idx"]) == n
    g = rows_to_flat(rows, f["idx"], s)
    x0 = flat_params(s)
    h = 1e-6
    fd = np.zeros_like(x0)
    for i in range(len(x0)):
        x = x0.copy()
        x[i] += h
        set_flat(s, x)
        lp = weighted_loss(oracle64, s, cam, wgt)
        x[i] -= 2 * h
        set_flat(s, x)
        lm = weighted_loss(oracle64, s, cam, wgt)
        fd[i] = (lp - lm) / (2 * h)
    set_flat(s, x0)
    scale = np.abs(fd).max()
    assert scale > 1e-3
    assert np.allclose(g, fd, rtol=2e-6, atol=2e-7 * scale), np.abs(g - fd).max()
    # every parameter group carries signal
    o = 0
    for a in (s.means, s.log_scales, s.quats, s.opacity_logit, s.sh):
        assert np.abs(fd[o:o + a.size]).max() > 0
        o += a.size


def test_gradients_with_jacobian_clamp_and_colour_clamp(oracle64):
    # wide field of view so some splats exceed the 1.3x guard; dark colours so some channels clamp
    s, cam = wl.tiny_scene(31, 8, 1, width=32, height=32, f=12.0, ls_mu=-0.6, depth=(1.5, 3.0), spread=2.2)
    s.sh[:4, 0, 0] = -0.6 / 0.28209479177387814
    # two big splats placed beyond the guard in camera space (x/z = 1.9 and y/z = -2.0 > 1.733)
    R_c, t_c = cam.w2c[:, :3], cam.w2c[:, 3]
    for i, tc in ((0, (3.8, 0.3, 2.0)), (5, (-0.4, -4.4, 2.2))):
        s.means[i] = R_c.T @ (np.array(tc) - t_c)
        s.log_scales[i] = (-0.2, -0.4, -0.3)
    wgt = np.random.default_rng(1).uniform(-1, 1, (3, 32, 32))
    f, g2d, rows = analytic(oracle64, s, cam, wgt)
    t = s.means @ R_c.T + t_c
    lim = 1.3 * 32 / (2 * 12.0)
    clamped = (np.abs(t[:, 0] / t[:, 2]) > lim) | (np.abs(t[:, 1] / t[:, 2]) > lim)
    assert clamped[f["idx"]].any() and f["proj"].clamp_flags.any()
    assert f["pix_margin"].min() > 1e-6 and f["proj"].margin.min() > 1e-6
    g = rows_to_flat(rows, f["idx"], s)
    x0 = flat_params(s)
    h = 1e-6
    fd = np.zeros_like(x0)
    for i in range(len(x0)):
        x = x0.copy(); x[i] += h; set_flat(s, x)
        lp = weighted_loss(oracle64, s, cam, wgt)
        x[i] -= 2 * h; set_flat(s, x)
        lm = weighted_loss(oracle64, s, cam, wgt)
        fd[i] = (lp - lm) / (2 * h)
    set_flat(s, x0)
    assert np.allclose(g, fd, rtol=2e-6, atol=2e-7 * np.abs(fd).max()), np.abs(g - fd).max()
    # clamped colour channels get exactly zero SH gradient
    for r, p in enumerate(f["idx"]):
        if f["proj"].clamp_flags[p] & 1:
            assert np.all(rows[r, 11::3] == 0)


def test_single_splat_opacity_gradient_closed_form(oracle64):
    # dL/do = sum_px G(px) * sum_ch (c - bg) g over pixels where alpha >= 1/255
    f_, z, o = 64.0, 4.0, 0.3
    c, bg = np.array([0.9, 0.4, 0.2]), np.array([0.1, 0.2, 0.3])
    cam = cam_identity(bg=bg)
    s = one_splat((0.03, -0.02, z), (-1.6,) * 3, (1, 0, 0, 0), logit(o), c)
    wgt = np.random.default_rng(0).uniform(-1, 1, (3, 64, 64))
    f, g2d, rows = analytic(oracle64, s, cam, wgt)
    A, B, C, _ = f["proj"].conic_o[0]
    u, v = f["proj"].xy[0]
    yy, xx = np.meshgrid(np.arange(64) + 0.5, np.arange(64) + 0.5, indexing="ij")
    G = np.exp(-0.5 * (A * (u - xx) ** 2 + C * (v - yy) ** 2) - B * (u - xx) * (v - yy))
    on = o * G >= 1 / 255
    want = (G * on * ((c - bg)[:, None, None] * wgt).sum(0)).sum()
    assert np.isclose(g2d[0, 5], want, rtol=1e-10)
    assert np.isclose(rows[0, 10], want * o * (1 - o), rtol=1e-10)
    # colour gradient: sum alpha * T(=1) * g
    assert np.allclose(g2d[0, 6:9], ((o * G * on)[None] * wgt).sum((1, 2)), rtol=1e-10)


def test_clamped_alpha_stops_the_chain(oracle64):
    cam = cam_identity()
    s = one_splat((0.5 * 4 / 64, 0.5 * 4 / 64, 4.0), (-9,) * 3, (1, 0, 0, 0), logit(0.9999), (1, 1, 1))
    wgt = np.ones((3, 64, 64))
    f, g2d, rows = analytic(oracle64, s, cam, wgt)
    # only the centre pixel has o*G > 0.99; the splat is sub-pixel so neighbours have alpha < 0.99
    assert f["n_contrib"][32, 32] == 1 and np.isclose(f["final_T"][32, 32], 0.01)
    G_nb = np.exp(-0.5 / ((64 * np.exp(-9) / 4) ** 2 + 0.3))
    # opacity gradient only from unclamped pixels: 4 edge neighbours (dx^2+dy^2=1) etc., none from the centre
    yy, xx = np.meshgrid(np.arange(64) - 32.0, np.arange(64) - 32.0, indexing="ij")
    var = (64 * np.exp(-9) / 4) ** 2 + 0.3
    G = np.exp(-0.5 * (xx ** 2 + yy ** 2) / var)
    a = 0.9999 * G
    on = (a >= 1 / 255) & (a <= 0.99)
    assert np.isclose(g2d[0, 5], 3 * (G * on).sum(), rtol=1e-9) and G_nb > 0


def test_culled_and_untouched_primitives_have_no_rows(oracle64):
    s, cam = wl.tiny_scene(5, 6, 0)
    s.means[2] = (0, 0, -5.0)  # behind the camera
    wgt = np.ones((3, cam.height, cam.width))
    f, g2d, rows = analytic(oracle64, s, cam, wgt)
    assert 2 not in f["idx"] and rows.shape[0] == len(f["idx"]) == 5
    assert np.all(g2d[2] == 0)


# ------------------------------------------------------------------------------- Adam
def make_state(n, k, rng, dt):
    def arrs():
        return wl.Scene(int(np.sqrt(k)) - 1, rng.standard_normal((n, 3)).astype(dt), rng.standard_normal((n, 3)).astype(dt),
                        rng.standard_normal((n, 4)).astype(dt), rng.standard_normal(n).astype(dt),
                        rng.standard_normal((n, k, 3)).astype(dt))
    return arrs()


def test_adam_hand_example(oracle64):
    # one scalar per group is enough: theta=1, g=0.5, t=1, lr=1e-3 -> m=0.05, v=2.5e-4, theta=0.999
    with open(os.path.join(GOLDEN, "adam_hand_example.txt")) as fh:
        vals = dict(line.split("=") for line in fh.read().split() if "=" in line)
    p = wl.Scene(0, np.ones((1, 3)), np.ones((1, 3)), np.ones((1, 4)), np.ones(1), np.ones((1, 1, 3)))
    m, v = p.zeros_like(), p.zeros_like()
    rows = np.full((1, 14), float(vals["g"]))
    oracle64.sparse_adam(p, m, v, rows, np.array([0]), np.full(6, float(vals["lr"])), 0.9, 0.999, 1e-15, 1)
    for a, b, c in zip((p.means, p.quats, p.sh), (m.means, m.quats, m.sh), (v.means, v.quats, v.sh)):
        assert np.allclose(a, float(vals["theta_after"]), atol=1e-12)
        assert np.allclose(b, float(vals["m_after"]), atol=1e-15) and np.allclose(c, float(vals["v_after"]), atol=1e-15)


@pytest.mark.parametrize("dt", [np.float64, np.float32])
def test_adam_all_rows_equals_torch_adam(dt):
    import oracle

    o = oracle.get(dt)
    rng = np.random.default_rng(7)
    n, k = 37, 16
    p = make_state(n, k, rng, dt)
    m, v = p.zeros_like(), p.zeros_like()
    tp = [torch.tensor(a.copy(), requires_grad=True) for a in (p.means, p.log_scales, p.quats, p.opacity_logit, p.sh)]
    lrs = np.array([1e-3, 2e-3, 5e-4, 1e-2, 3e-3, 1e-4])
    # sh is split in two torch groups (dc, rest) by giving it two optimisers over views of a copy
    opt = torch.optim.Adam([{"params": [tp[i]], "lr": float(lrs[i])} for i in range(4)], betas=(0.9, 0.999), eps=1e-8)
    sh_dc = torch.tensor(p.sh[:, :1].copy(), requires_grad=True)
    sh_rest = torch.tensor(p.sh[:, 1:].copy(), requires_grad=True)
    opt2 = torch.optim.Adam([{"params": [sh_dc], "lr": float(lrs[4])}, {"params": [sh_rest], "lr": float(lrs[5])}],
                            betas=(0.9, 0.999), eps=1e-8)
    idx = np.arange(n, dtype=np.uint32)
    for step in range(1, 6):
        rows = rng.standard_normal((n, 11 + 3 * k)).astype(dt)
        o.sparse_adam(p, m, v, rows, idx, lrs.astype(dt), 0.9, 0.999, 1e-8, step)
        tp[0].grad = torch.tensor(rows[:, 0:3]); tp[1].grad = torch.tensor(rows[:, 3:6])
        tp[2].grad = torch.tensor(rows[:, 6:10]); tp[3].grad = torch.tensor(rows[:, 10])
        gsh = rows[:, 11:].reshape(n, k, 3)
        sh_dc.grad = torch.tensor(gsh[:, :1].copy()); sh_rest.grad = torch.tensor(gsh[:, 1:].copy())
        opt.step(); opt2.step()
    tol = dict(rtol=1e-10, atol=1e-12) if dt == np.float64 else dict(rtol=2e-5, atol=2e-6)
    for a, b in zip((p.means, p.log_scales, p.quats, p.opacity_logit), tp):
        assert np.allclose(a, b.detach().numpy(), **tol)
    assert np.allclose(p.sh[:, :1], sh_dc.detach().numpy(), **tol)
    assert np.allclose(p.sh[:, 1:], sh_rest.detach().numpy(), **tol)


def test_adam_untouched_rows_are_bitwise_unchanged(oracle32):
    rng = np.random.default_rng(9)
    n, k = 200, 16
    p = make_state(n, k, rng, np.float32)
    m, v = make_state(n, k, rng, np.float32), make_state(n, k, rng, np.float32)
    for s in (v,):
        for a in (s.means, s.log_scales, s.quats, s.opacity_logit, s.sh):
            np.abs(a, out=a)
    before = [a.copy() for s in (p, m, v) for a in (s.means, s.log_scales, s.quats, s.opacity_logit, s.sh)]
    idx = np.sort(rng.choice(n, 60, replace=False)).astype(np.uint32)
    rows = rng.standard_normal((60, 59)).astype(np.float32)
    rows[5] = 0  # a touched row with zero gradient still decays its moments
    oracle32.sparse_adam(p, m, v, rows, idx, np.full(6, 1e-3, np.float32), 0.9, 0.999, 1e-15, 3)
    after = [a for s in (p, m, v) for a in (s.means, s.log_scales, s.quats, s.opacity_logit, s.sh)]
    un = np.setdiff1d(np.arange(n), idx)
    for b, a in zip(before, after):
        assert np.array_equal(b[un].view(np.uint32), a[un].view(np.uint32))
        assert not np.array_equal(b[idx], a[idx])
    assert np.allclose(m.means[idx[5]], 0.9 * before[5][idx[5]])
    # empty list: nothing moves
    snap = [a.copy() for a in after]
    oracle32.sparse_adam(p, m, v, np.zeros((0, 59), np.float32), np.zeros(0, np.uint32), np.full(6, 1e-3, np.float32),
                         0.9, 0.999, 1e-15, 4)
    for b, a in zip(snap, after):
        assert np.array_equal(b, a)


# ------------------------------------------------------------------------------- sets
def test_touched_set_bruteforce(oracle32):
    rng = np.random.default_rng(2)
    for n in (0, 1, 31, 32, 33, 1000, 4097):
        tt = (rng.random(n) < 0.3).astype(np.uint32) * rng.integers(1, 9, n).astype(np.uint32)
        mask, idx = oracle32.touched_set(tt)
        want = np.nonzero(tt)[0]
        assert np.array_equal(idx, want)
        bits = np.unpackbits(mask.view(np.uint8), bitorder="little")[:n]
        assert np.array_equal(np.nonzero(bits)[0], want)
        assert int(sum(bin(int(w)).count("1") for w in mask)) == len(idx)


def test_conflict_count_bruteforce_and_identities(oracle32):
    rng = np.random.default_rng(4)
    n = 5000
    sets = [np.sort(rng.choice(n, rng.integers(0, 3000), replace=False)).astype(np.uint32) for _ in range(5)]
    sets.append(np.zeros(0, np.uint32))
    for a in sets:
        assert oracle32.conflict_count(a, a) == len(a)
        assert oracle32.conflict_count(a, sets[-1]) == 0
        for b in sets:
            c = oracle32.conflict_count(a, b)
            assert c == len(set(a.tolist()) & set(b.tolist())) == oracle32.conflict_count(b, a)
            assert len(np.union1d(a, b)) == len(a) + len(b) - c  # inclusion-exclusion


def test_hazard_algebra_example(oracle32):
    """Sec. 4.3 hazard sets on a hand-written example: with R+ = W+ only WAW is non-empty."""
    sets = {}
    with open(os.path.join(GOLDEN, "hazard_sets_example.txt")) as fh:
        for line in fh:
            if line.startswith("#") or "=" not in line:
                continue
            k, v = line.split("=")
            sets[k.strip()] = np.array([int(x) for x in v.split()], np.uint32)
    waw = oracle32.conflict_count(sets["W_B"], sets["W_A"])
    assert waw == int(sets["n_WAW"][0])
    raw = np.intersect1d(np.setdiff1d(sets["R_B"], sets["W_B"]), sets["W_A"])
    war = np.intersect1d(sets["W_B"], np.setdiff1d(sets["R_A"], sets["W_A"]))
    assert len(raw) == int(sets["n_RAW"][0]) and len(war) == int(sets["n_WAR"][0])
    # in this build R+ = W+ = touched set, so RAW and WAR vanish identically
    assert len(np.setdiff1d(sets["W_B"], sets["W_B"])) == 0


def test_scope_nesting_on_a_rendered_view(oracle32):
    """Sec. 2.1: Theta >= G_i >= C_i.  Contributors of any pixel are inside the touched set."""
    w = wl.make_workload(1)
    f = oracle32.view_forward(w.scene, w.cameras[0])
    contributors = set()
    for t in range(len(f["ranges"])):
        s = f["ranges"][t, 0]
        nmax = f["n_contrib"].reshape(4, 16, 4, 16)[t // 4, :, t % 4, :].max()
        contributors |= set(f["vals"][s:s + nmax].tolist())
    assert contributors <= set(f["idx"].tolist()) <= set(range(w.scene.n))
