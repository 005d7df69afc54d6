"""Pins of the oracle's realized active set, gradient evidence, hazard sets and delayed-read gate (Sec. 2.1, Sec. 4.3)
against brute force, closed forms, invariants and a hand-worked example (no GPU)."""
import os

import numpy as np

from paper_2607_19893_b200 import workloads as wl
from test_oracle_project_pins import cam_identity, one_splat
from test_oracle_render_pins import stack_scenes

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def read_golden(name):
    sets = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            if line.startswith("#") or "=" not in line:
                continue
            k, v = line.split("=")
            sets[k.strip()] = v.split()
    return sets


# ------------------------------------------------------------------------------- realized active set
def brute_force_active(f, cam):
    """Independent restatement: walk every pixel's list front to back with the compositing rule and record who blends."""
    p = f["proj"]
    tx = (cam.width + 15) // 16
    alpha_min, alpha_max, t_min = 1.0 / 255.0, 0.99, 1e-4   # the method's constants
    active, fragile = set(), False
    for j in range(cam.height):
        for i in range(cam.width):
            s, e = f["ranges"][(j // 16) * tx + i // 16]
            T = 1.0
            for k in range(s, e):
                q = int(f["vals"][k])
                d = p.xy[q] - (i + 0.5, j + 0.5)
                A, B, Cc, o = p.conic_o[q]
                power = -0.5 * (A * d[0] * d[0] + Cc * d[1] * d[1]) - B * d[0] * d[1]
                if power > 0:
                    continue
                alpha = min(alpha_max, o * np.exp(power))
                if alpha < alpha_min:
                    continue
                if T * (1 - alpha) < t_min:
                    break
                active.add(q)
                T *= 1 - alpha
    return active


def test_realized_active_matches_bruteforce_and_is_nested(oracle64):
    w = wl.make_workload(1)
    cam = w.cameras[0]
    f = oracle64.view_forward(w.scene, cam)
    mask, idx = oracle64.realized_active(f["proj"], f["vals"], f["ranges"], cam, f["n_contrib"])
    want = brute_force_active(f, cam)
    assert set(idx.tolist()) == want
    # Theta >= G_i >= C_i (Sec. 2.1), ascending list, mask = the same set
    assert set(idx.tolist()) <= set(f["idx"].tolist()) <= set(range(w.scene.n))
    assert np.all(np.diff(idx.astype(np.int64)) > 0)
    bits = np.unpackbits(mask.view(np.uint8), bitorder="little")[: w.scene.n]
    assert np.array_equal(np.flatnonzero(bits), idx)
    # a primitive is active exactly when the colour gradient has a non-zero un-cancelled term sum for unit dL
    ones = np.ones_like(f["out"])
    _, g_abs = oracle64.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], ones,
                                         want_abs=True)
    assert np.array_equal(np.flatnonzero(g_abs[:, 6] > 0), idx)


def test_occluded_primitive_is_touched_but_not_active(oracle64):
    """Four wide, almost opaque splats in front of a tiny one on the same axis: after two of them the transmittance is
    1e-4 and the third would push it below the stop threshold, so every pixel the tiny splat could reach stops before
    it.  The tiny splat is in the candidate scope (it covers a tile) but not in the realized one.  Without the
    occluders it is active."""
    cam = cam_identity(64, 64, 64.0)
    fronts = [one_splat((0.0, 0.0, 2.0 + 0.1 * k), (0.0, 0.0, 0.0), (1, 0, 0, 0), logit=12.0) for k in range(4)]
    behind = one_splat((0.0, 0.0, 4.0), (-4.5, -4.5, -4.5), (1, 0, 0, 0), logit=2.0)
    scene = stack_scenes(fronts + [behind])
    f = oracle64.view_forward(scene, cam)
    assert 4 in f["idx"]                                        # touched: geometry locality sees it
    _, idx = oracle64.realized_active(f["proj"], f["vals"], f["ranges"], cam, f["n_contrib"])
    assert 4 not in idx and {0, 1} <= set(idx.tolist())
    assert f["n_contrib"][32, 32] == 2                          # the centre pixel stops at the third occluder
    f2 = oracle64.view_forward(behind, cam)
    _, idx2 = oracle64.realized_active(f2["proj"], f2["vals"], f2["ranges"], cam, f2["n_contrib"])
    assert idx2.tolist() == [0]


# ------------------------------------------------------------------------------- gradient evidence
def test_gradient_evidence_norms_mean_and_linearity(oracle64):
    g2d = np.zeros((6, 9))
    g2d[1, :2] = (3.0, 4.0)
    g2d[2, :2] = (-6.0, 8.0)
    g2d[4, :2] = (0.0, 0.0)
    g2d[:, 2:] = 7.0                                            # the other words do not enter the default evidence
    ev, mean = oracle64.gradient_evidence(g2d, [1, 2, 4])
    assert np.allclose(ev, (5.0, 10.0, 0.0)) and mean == 5.0
    ev2, mean2 = oracle64.gradient_evidence(-2.5 * g2d, [1, 2, 4])
    assert np.allclose(ev2, 2.5 * ev) and np.isclose(mean2, 2.5 * mean)
    ev0, mean0 = oracle64.gradient_evidence(g2d, [])
    assert len(ev0) == 0 and mean0 == 0.0
    # whole-row variant: rows of the touched primitives [2, 4, 5]; active [2, 5]
    rows = np.array([[1.0, 2.0, 2.0], [9.0, 9.0, 9.0], [0.0, 3.0, 4.0]])
    evr, meanr = oracle64.gradient_evidence(None, [2, 5], rows=rows, touched_idx=[2, 4, 5])
    assert np.allclose(evr, (3.0, 5.0)) and meanr == 4.0


def test_gradient_evidence_scales_with_the_loss_on_a_rendered_view(oracle64):
    w = wl.make_workload(1)
    cam = w.cameras[0]
    f = oracle64.view_forward(w.scene, cam)
    _, dl = oracle64.l1_loss(f["out"], w.target(0).astype(np.float64))
    g = oracle64.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], dl)
    g3 = oracle64.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], 3.0 * dl)
    _, idx = oracle64.realized_active(f["proj"], f["vals"], f["ranges"], cam, f["n_contrib"])
    ev, mean = oracle64.gradient_evidence(g, idx)
    ev3, mean3 = oracle64.gradient_evidence(g3, idx)
    assert np.allclose(ev3, 3 * ev, rtol=1e-12) and np.isclose(mean3, 3 * mean)
    # primitives outside the active set received no gradient at all
    inactive = np.setdiff1d(np.arange(w.scene.n), idx)
    assert not g[inactive].any()


# ------------------------------------------------------------------------------- hazards
def test_hazard_sets_hand_example_and_algebra(oracle64):
    s = {k: np.array([int(x) for x in v]) for k, v in read_golden("hazard_sets_example.txt").items()}
    waw, raw, war = oracle64.hazard_sets(s["R_A"], s["W_A"], s["R_B"], s["W_B"])
    assert waw.tolist() == [4, 6] and raw.tolist() == [8] and war.tolist() == [5]
    assert (len(waw), len(raw), len(war)) == (int(s["n_WAW"][0]), int(s["n_RAW"][0]), int(s["n_WAR"][0]))
    rng = np.random.default_rng(11)
    for _ in range(20):
        n = 400
        w_a = rng.choice(n, rng.integers(0, 200), replace=False)
        r_a = np.union1d(w_a, rng.choice(n, rng.integers(0, 100), replace=False))      # W+ is inside R+
        w_b = rng.choice(n, rng.integers(0, 200), replace=False)
        r_b = np.union1d(w_b, rng.choice(n, rng.integers(0, 100), replace=False))
        waw, raw, war = oracle64.hazard_sets(r_a, w_a, r_b, w_b)
        A_r, A_w, B_r, B_w = set(r_a.tolist()), set(w_a.tolist()), set(r_b.tolist()), set(w_b.tolist())
        assert set(waw.tolist()) == B_w & A_w
        assert set(raw.tolist()) == (B_r - B_w) & A_w
        assert set(war.tolist()) == B_w & (A_r - A_w)
        # RAW and WAW partition R+(B) & W+(A); the three sets are pairwise disjoint
        assert len(raw) + len(waw) == len(B_r & A_w)
        assert not (set(raw.tolist()) & set(waw.tolist())) and not (set(war.tolist()) & set(waw.tolist()))
        assert len(waw) == oracle64.conflict_count(np.sort(w_a).astype(np.uint32), np.sort(w_b).astype(np.uint32))
        # this build's pipeline declares R+ = W+: then only WAW can be non-empty
        _, raw0, war0 = oracle64.hazard_sets(w_a, w_a, w_b, w_b)
        assert len(raw0) == 0 and len(war0) == 0


def test_delayed_read_gate_hand_example(oracle64):
    g = read_golden("delayed_read_gate_example.txt")
    ints = lambda k: np.array([int(x) for x in g[k]])  # noqa: E731
    ev = np.array([float(x) for x in g["evidence_A"]])
    for case in ("1", "2", "3", "4"):
        out = oracle64.delayed_read_gate(ints("R_A"), ints("W_A"), ints("R_B" + case), ints("W_B" + case), ints("C_A"), ev,
                                         float(g["tau" + case][0]))
        assert out["n_delayed"] == int(g["n_delayed" + case][0])
        assert out["n_with_evidence"] == int(g["n_with_evidence" + case][0])
        assert out["n_pass"] == int(g["n_pass" + case][0])
        assert np.isclose(out["rho"], float(g["rho" + case][0]))
        assert out["admitted"] == (g["admitted" + case][0] == "yes")
    assert np.isclose(out["mean"], float(g["mean_A"][0]))
    # an empty consumer read scope has no delayed-read admission to perform
    out = oracle64.delayed_read_gate(ints("R_A"), ints("W_A"), [], [], ints("C_A"), ev, 1.0)
    assert out["rho"] is None and not out["admitted"] and out["n_delayed"] == 0


# ------------------------------------------------------------------------------- relative locality graph from counts
def dense_from_pairs(n, pairs, w):
    m = np.zeros((n, n), np.float32)
    for (a, b), x in zip(pairs, w):
        m[a, b] = m[b, a] = x
    return m


def test_rlg_weights_topk_and_sds_scores_hand_example(oracle64):
    g = read_golden("rlg_example.txt")
    sizes = np.array([int(x) for x in g["sizes"]])
    pairs = np.array([int(x) for x in g["pairs"]]).reshape(-1, 2)
    counts = np.array([int(x) for x in g["counts"]])
    w = oracle64.rlg_weights(sizes, pairs, counts)
    assert np.allclose(w, [float(x) for x in g["weights"]], rtol=1e-6)
    full = dense_from_pairs(4, pairs, w)
    top1 = oracle64.rlg_topk(full, 1)
    edges = {tuple(e) for e in np.array([int(x) for x in g["top1_edges"]]).reshape(-1, 2).tolist()}
    assert {(a, b) for a in range(4) for b in range(a + 1, 4) if top1[a, b] > 0} == edges
    assert np.array_equal(top1, top1.T) and not np.diag(top1).any()
    prev, cand = [int(x) for x in g["prev_unit"]], [int(x) for x in g["candidates"]]
    assert np.allclose(oracle64.sds_scores(full, prev, cand), [float(x) for x in g["scores_full"]], rtol=1e-6)
    assert np.allclose(oracle64.sds_scores(top1, prev, cand), [float(x) for x in g["scores_top1"]], rtol=1e-6)


def test_rlg_weights_are_jaccard_of_the_sets_and_topk_is_monotone(oracle64):
    rng = np.random.default_rng(21)
    n, views = 3000, 9
    sets = [set(rng.choice(n, rng.integers(0, 1500), replace=False).tolist()) for _ in range(views)]
    sets[4] = set()
    pairs = np.array([(a, b) for a in range(views) for b in range(a + 1, views)])
    counts = np.array([len(sets[a] & sets[b]) for a, b in pairs])
    sizes = np.array([len(s) for s in sets])
    w = oracle64.rlg_weights(sizes, pairs, counts)
    for (a, b), x in zip(pairs, w):
        u = len(sets[a] | sets[b])
        assert np.isclose(x, len(sets[a] & sets[b]) / u if u else 0.0, rtol=1e-6)
        assert 0.0 <= x <= 1.0
    full = dense_from_pairs(views, pairs, w)
    prev_edges = -1
    for k in range(0, views):
        g = oracle64.rlg_topk(full, k)
        assert np.array_equal(g, g.T)
        assert np.all((g == 0) | (g == full))                       # retention only removes edges
        deg_kept = [(np.argsort(-full[i], kind="stable")[:k]) for i in range(views)]
        for i in range(views):                                      # every item still sees its own k strongest
            for j in deg_kept[i]:
                if full[i, j] > 0:
                    assert g[i, j] == full[i, j]
        edges = int((g > 0).sum())
        assert edges >= prev_edges
        prev_edges = edges
    assert np.array_equal(oracle64.rlg_topk(full, views), full)     # k >= degree keeps everything
    # Eq. (2) is additive over the previous unit
    s01 = oracle64.sds_scores(full, [0, 1], [5, 6, 7])
    assert np.allclose(s01, oracle64.sds_scores(full, [0], [5, 6, 7]) + oracle64.sds_scores(full, [1], [5, 6, 7]))


# ------------------------------------------------------------------------------- task units of two views (Sec. 2.1, Sec. 6.1)
def test_accumulate_rows_hand_example(oracle64):
    idx_a, idx_b = [1, 4, 7], [0, 4, 9]
    rows_a = np.array([[1.0, 2.0], [3.0, 4.0], [5.0, 6.0]])
    rows_b = np.array([[10.0, 20.0], [30.0, 40.0], [50.0, 60.0]])
    union, rows = oracle64.accumulate_rows(idx_a, rows_a, idx_b, rows_b)
    assert union.tolist() == [0, 1, 4, 7, 9]
    assert rows.tolist() == [[10, 20], [1, 2], [33, 44], [5, 6], [50, 60]]
    u2, r2 = oracle64.accumulate_rows(idx_b, rows_b, idx_a, rows_a)            # symmetric
    assert np.array_equal(union, u2) and np.array_equal(rows, r2)
    u3, r3 = oracle64.accumulate_rows(idx_a, rows_a, [], np.zeros((0, 2)))    # an empty view adds nothing
    assert u3.tolist() == idx_a and np.array_equal(r3, rows_a)


def test_unit_step_equals_dense_adam_on_the_summed_gradients(oracle64):
    """Two views with the same parameters, gradients summed, one update: on the rows of the union this is textbook Adam
    fed with the sum of the two dense gradients (torch.optim.Adam as the library routine), and no other row moves."""
    import torch

    from paper_2607_19893_b200 import workloads as wl

    w = wl.make_workload(2, n=400)
    s = w.scene.astype(np.float64)
    m, v = s.zeros_like(), s.zeros_like()
    cams, tgts = [w.cameras[0], w.cameras[3]], [w.target(0).astype(np.float64), w.target(3).astype(np.float64)]
    before = s.copy()
    lr = w.lr.astype(np.float64)
    # dense reference: per-view gradients from the oracle's own backward (pinned by finite differences), summed
    dense = np.zeros((s.n, s.floats_per_primitive))
    for cam, tgt in zip(cams, tgts):
        f = oracle64.view_step(before.copy(), m.copy(), v.copy(), cam, tgt, lr, w.beta1, w.beta2, 1e-8, 1, update=False)
        dense[f["idx"].astype(np.int64)] += f["rows"]
    touched = np.flatnonzero(np.abs(dense).sum(axis=1) > 0)
    flat = lambda sc: np.concatenate([sc.means, sc.log_scales, sc.quats, sc.opacity_logit[:, None],  # noqa: E731
                                      sc.sh.reshape(sc.n, -1)], axis=1)
    out = oracle64.unit_step(s, m, v, cams, tgts, lr, w.beta1, w.beta2, 1e-8, 1)
    union = out["idx"].astype(np.int64)
    assert set(touched) <= set(union)
    p_t = torch.tensor(flat(before)[union], dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p_t], lr=float(lr[0]), betas=(w.beta1, w.beta2), eps=1e-8)
    p_t.grad = torch.tensor(dense[union], dtype=torch.float64)
    opt.step()
    assert np.allclose(flat(s)[union], p_t.detach().numpy(), rtol=1e-12, atol=1e-14)
    rest = np.setdiff1d(np.arange(s.n), union)
    assert np.array_equal(flat(s)[rest], flat(before)[rest]) and not flat(m)[rest].any()
    assert np.abs(flat(s)[union] - flat(before)[union]).max() > 1e-5
