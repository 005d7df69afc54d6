"""Parity of the realized active set, gradient evidence, unit unions, hazard counts and the delayed-read gate
(Sec. 2.1 Table 1, Sec. 4.3) through the C ABI against the oracle (needs a GPU)."""
import numpy as np
import pytest
import torch

from oracle import oracle as oracle_mod
from paper_2607_19893_b200 import binding as B
from paper_2607_19893_b200 import engine as E
from paper_2607_19893_b200 import workloads as wl

import gpu_util as G
from test_gpu_stages import load_sorted, oracle_view, faint_scene

pytestmark = pytest.mark.gpu


def mask_ids(words, n):
    return np.flatnonzero(np.unpackbits(np.ascontiguousarray(words).view(np.uint8), bitorder="little")[:n])


# ------------------------------------------------------------------------------------------------ active set
def check_active_set(oracle32, scene, cam, seed=0):
    n = scene.n
    f, inv = oracle_view(oracle32, scene, cam)
    rng = np.random.default_rng(seed)
    dl = rng.uniform(-1, 1, f["out"].shape).astype(np.float32)
    robust = f["pix_margin"] > 2e-5
    dl[:, ~robust] = 0  # see test_gpu_stages.check_backward
    g2d_o, g2d_abs = oracle32.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], dl,
                                               want_abs=True)
    rows_o = oracle32.render_bwd_project(scene, cam, f["idx"], g2d_o, f["proj"].clamp_flags).astype(np.float64)
    _, active_o = oracle32.realized_active(f["proj"], f["vals"], f["ranges"], cam, f["n_contrib"])
    # what is certain: activity through pixels whose decisions are all robust
    nc_sure = f["n_contrib"].copy()
    nc_sure[~robust] = 0
    _, active_sure = oracle32.realized_active(f["proj"], f["vals"], f["ranges"], cam, nc_sure)
    # what may differ: primitives inside the walked prefix of a fragile pixel
    tx = (cam.width + 15) // 16
    maybe = set()
    for j, i in np.argwhere(~robust):
        s = f["ranges"][(j // 16) * tx + i // 16, 0]
        maybe |= set(f["vals"][s:s + f["n_contrib"][j, i]].tolist())

    v = len(f["idx"])
    tr = G.trainer_for(scene, cam, row_capacity=max(v, 1), instance_capacity=len(f["vals"]) + 1)
    tr.track_active = True
    load_sorted(tr, f, inv)
    tr.render_fwd(B.make_camera(cam))  # the backward pass starts long lists from the states this leaves in the workspace
    tr.final_T.copy_(torch.from_numpy(f["final_T"]).to(tr.device))
    tr.n_contrib.copy_(torch.from_numpy(f["n_contrib"].view(np.int32)).to(tr.device))
    tr.dL.copy_(torch.from_numpy(dl).to(tr.device))
    for mode in (0, 1, 0):
        tr.render_bwd(B.make_camera(cam))
        tr.active_set(slot=0, evidence_mode=mode)
        G.poll_ok(tr)
        cnt = int(tr.active_count.item())
        idx = G.u32(tr.active_idx)[:cnt]
        # list, mask and flags describe the same set; ascending primitive ids
        assert np.all(np.diff(idx.astype(np.int64)) > 0)
        assert np.array_equal(mask_ids(G.u32(tr.active_masks[0]), n), idx)
        flags = tr.row_active.cpu().numpy()[:v].astype(bool)
        assert np.array_equal(f["idx"][flags], idx)
        # against the oracle: certain members present, nothing beyond what a fragile pixel can explain
        dev, want = set(idx.tolist()), set(active_o.tolist())
        assert set(active_sure.tolist()) <= dev
        assert (dev ^ want) <= maybe
        assert len(dev ^ want) <= max(2, int((~robust).sum()))
        assert dev <= set(f["idx"].tolist())  # C_i inside G_i
        # evidence of the primitives both sides call active
        both = np.array(sorted(dev & want), np.int64)
        ev_dev = tr.evidence.cpu().numpy()[:cnt].astype(np.float64)
        ev_dev_both = ev_dev[np.searchsorted(idx, both)]
        if mode == 0:
            ev_o, _ = oracle32.gradient_evidence(g2d_o, both)
            b = G.grad2d_bound(g2d_o[both, :2], g2d_abs[both, :2])
            tol = np.sqrt((b * b).sum(axis=1)) + 1e-6 * ev_o
        else:
            ev_o, _ = oracle32.gradient_evidence(None, both, rows=rows_o, touched_idx=f["idx"])
            bound = G.rows_bound(oracle32, scene, cam, f["idx"], f["proj"].clamp_flags, rows_o, g2d_o, g2d_abs)
            pos = np.searchsorted(f["idx"].astype(np.int64), both)
            tol = 10 * np.sqrt((bound[pos] ** 2).sum(axis=1)) + 1e-6 * ev_o
        assert np.all(np.abs(ev_dev_both - ev_o) <= tol), np.abs(ev_dev_both - ev_o).max()
        assert ev_o.max() > 1e-4
        # the sum is the sum of the listed evidence
        assert float(tr.evidence_sum.item()) == pytest.approx(float(ev_dev.sum()), rel=1e-12, abs=1e-30)
    tr.close()
    return len(active_o), v


def test_active_set_cfg1(oracle32):
    w = wl.make_workload(1)
    check_active_set(oracle32, w.scene, w.cameras[0])


def test_active_set_cfg2_many_occluded(oracle32):
    w = wl.make_workload(2, n=30_000)
    na, v = check_active_set(oracle32, w.scene, w.cameras[3], seed=2)
    assert na < v  # some touched primitives never blend: the realized scope is strictly inside the candidate scope


def test_active_set_long_lists_head_and_tail_kernels(oracle32):
    s, cam = faint_scene(n=12_000)
    check_active_set(oracle32, s, cam, seed=4)


def test_active_set_capacity_and_empty_view(oracle32):
    w = wl.make_workload(1)
    cam = w.cameras[0]
    f, inv = oracle_view(oracle32, w.scene, cam)
    v = len(f["idx"])
    tr = G.trainer_for(w.scene, cam, row_capacity=v, instance_capacity=len(f["vals"]) + 1)
    tr.track_active = True
    load_sorted(tr, f, inv)
    tr.render_fwd(B.make_camera(cam))  # the backward pass starts long lists from the states this leaves in the workspace
    tr.final_T.copy_(torch.from_numpy(f["final_T"]).to(tr.device))
    tr.n_contrib.copy_(torch.from_numpy(f["n_contrib"].view(np.int32)).to(tr.device))
    tr.render_bwd(B.make_camera(cam))
    # a list capacity smaller than the set: truncated list, deferred error, nothing written past the capacity
    small = torch.full((64,), -1, dtype=torch.int32, device=tr.device)
    ev = torch.full((64,), -1.0, dtype=torch.float32, device=tr.device)
    B.odin_active_set(tr.ctx, tr.proj.struct, tr.row_active, tr.grad2d, None, 0, tr.n, tr.active_masks[0], small, 50,
                      tr.active_count, ev, tr.evidence_sum, tr.ws)
    assert tr.poll() == B.ODIN_ERR_CAPACITY
    assert int(tr.active_count.item()) == 50
    got = small.cpu().numpy()
    assert np.all(got[50:] == -1) and np.all(np.diff(got[:50]) > 0) and np.all(ev.cpu().numpy()[50:] == -1.0)
    # no rows at all
    tr.proj.num_rows.zero_()
    tr.active_set()
    G.poll_ok(tr)
    assert int(tr.active_count.item()) == 0 and float(tr.evidence_sum.item()) == 0.0
    assert not G.u32(tr.active_masks[0]).any()
    tr.close()


def test_active_set_after_a_whole_view_step(oracle32):
    w = wl.make_workload(2, n=40_000)
    tr = G.trainer_for(w.scene, w.cameras[0], mask_slots=2)
    with pytest.raises(RuntimeError):
        tr.active_set()                                             # the flags have to be asked for first
    tr.track_active = True
    for s, view in enumerate((1, 5)):
        tr.target.copy_(torch.from_numpy(w.target(view)).to(tr.device))
        tr.view_step(B.make_camera(w.cameras[view]), s + 1, w.lr, w.beta1, w.beta2, w.eps, slot=s)
        tr.active_set(slot=s)
        G.poll_ok(tr)
        touched, active = G.u32(tr.masks[s]), G.u32(tr.active_masks[s])
        assert not (active & ~touched).any()                       # C_i inside G_i, word by word
        cnt = int(tr.active_count.item())
        assert 0 < cnt <= int(tr.count.item())
        assert cnt == int(np.unpackbits(active.view(np.uint8)).sum())
    tr.close()


# ------------------------------------------------------------------------------------------------ unions, hazards, gate
def random_scopes(rng, n, units):
    """Per unit: write scope inside read scope (Sec. 2.1: W+ inside R+)."""
    reads, writes = [], []
    for _ in range(units):
        w = np.sort(rng.choice(n, rng.integers(0, n // 2 + 1), replace=False))
        r = np.union1d(w, rng.choice(n, rng.integers(0, n // 3 + 1), replace=False))
        reads.append(r); writes.append(w)
    return reads, writes


def to_device_masks(id_lists, n, dev):
    from oracle.oracle import ids_to_mask
    words = (n + 31) // 32
    stride = (words + 3) // 4 * 4
    m = np.zeros((len(id_lists), stride), np.uint32)
    for k, ids in enumerate(id_lists):
        m[k, :words] = ids_to_mask(ids, n)
    return torch.from_numpy(m.view(np.int32)).to(dev), stride


@pytest.mark.parametrize("n", [1, 31, 4097, 250_003])
def test_hazard_counts_and_unions_match_the_set_algebra(oracle32, n):
    rng = np.random.default_rng(n)
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    units = 5
    reads, writes = random_scopes(rng, n, units)
    d_r, stride = to_device_masks(reads, n, dev)
    d_w, _ = to_device_masks(writes, n, dev)
    pairs = np.array([(a, b) for a in range(units) for b in range(units)], np.uint32)
    d_pairs = torch.from_numpy(pairs.view(np.int32)).to(dev)
    d_counts = torch.full((len(pairs), 4), -1, dtype=torch.int64, device=dev)
    B.odin_hazard_count(ctx, d_r, d_w, units, stride, n, d_pairs, len(pairs), d_counts)
    assert B.odin_poll(ctx) == B.ODIN_OK
    got = d_counts.cpu().numpy()
    for (a, b), g in zip(pairs, got):
        waw, raw, war = oracle32.hazard_sets(reads[a], writes[a], reads[b], writes[b])
        assert g.tolist() == [len(waw), len(raw), len(war), len(reads[b])]
    # the pipeline of this repository declares R+ = W+: RAW and WAR vanish, WAW is the conflict count
    B.odin_hazard_count(ctx, d_w, d_w, units, stride, n, d_pairs, len(pairs), d_counts)
    d_cc = torch.zeros(len(pairs), dtype=torch.int64, device=dev)
    B.odin_conflict_count(ctx, d_w, units, stride, n, d_pairs, len(pairs), d_cc)
    assert B.odin_poll(ctx) == B.ODIN_OK
    got = d_counts.cpu().numpy()
    assert not got[:, 1:3].any() and np.array_equal(got[:, 0], d_cc.cpu().numpy())
    # unit unions: R+(U) = union over the views of the unit
    members = np.array([0, 2, 3], np.uint32)
    d_out = torch.full((stride,), -1, dtype=torch.int32, device=dev)
    B.odin_mask_union(ctx, d_r, units, stride, n, torch.from_numpy(members.view(np.int32)).to(dev), 3, d_out)
    assert B.odin_poll(ctx) == B.ODIN_OK
    want = np.union1d(np.union1d(reads[0], reads[2]), reads[3])
    assert np.array_equal(mask_ids(G.u32(d_out), n), want)
    assert not G.u32(d_out)[(n + 31) // 32:].any()
    B.odin_mask_union(ctx, d_r, units, stride, n, None, 0, d_out)      # the union over no view is empty
    assert B.odin_poll(ctx) == B.ODIN_OK and not G.u32(d_out).any()
    # a pair naming a unit that does not exist is reported and counts nothing
    bad = torch.tensor([[0, units]], dtype=torch.int32, device=dev)
    B.odin_hazard_count(ctx, d_r, d_w, units, stride, n, bad, 1, d_counts)
    assert B.odin_poll(ctx) == B.ODIN_ERR_INVALID_ARG
    B.odin_destroy(ctx)


# ------------------------------------------------------------------------------------------------ locality graph
def test_locality_graph_from_the_masks_of_rendered_views(oracle32):
    """Eq. (1) on the touched sets of eight rendered views (sizes and intersections measured by the library), top-k
    retention, Eq. (2) scores: weights and retained edges bit exact, scores to fp32 summation order."""
    w = wl.make_workload(2, n=60_000)
    views = 8
    tr = G.trainer_for(w.scene, w.cameras[0], mask_slots=views)
    sizes = torch.zeros(views, dtype=torch.int32, device=tr.device)
    sets = []
    for v in range(views):
        tr.project(B.make_camera(w.cameras[v]))
        tr.touched_set(slot=v)
        sizes[v:v + 1].copy_(tr.count)
        G.poll_ok(tr)
        sets.append(G.u32(tr.idx)[: int(tr.count.item())].copy())
    pairs = np.array([(a, b) for a in range(views) for b in range(a + 1, views)], np.uint32)
    d_pairs = torch.from_numpy(pairs.view(np.int32)).to(tr.device)
    d_counts = torch.zeros(len(pairs), dtype=torch.int64, device=tr.device)
    tr.conflict_count(d_pairs, len(pairs), d_counts)
    d_w = torch.full((len(pairs),), -1.0, dtype=torch.float32, device=tr.device)
    B.odin_rlg_weights(tr.ctx, d_counts, sizes, d_pairs, len(pairs), views, d_w)
    G.poll_ok(tr)
    counts_o = np.array([oracle32.conflict_count(sets[a], sets[b]) for a, b in pairs])
    want_w = oracle32.rlg_weights([len(s) for s in sets], pairs, counts_o)
    assert np.array_equal(d_w.cpu().numpy(), want_w) and want_w.max() > 0.05
    full = np.zeros((views, views), np.float32)
    for (a, b), x in zip(pairs, want_w):
        full[a, b] = full[b, a] = x
    d_full = torch.from_numpy(full).to(tr.device)
    d_ret = torch.full((views, views), -1.0, dtype=torch.float32, device=tr.device)
    ws = torch.zeros(views * views, dtype=torch.uint8, device=tr.device)
    prev = torch.tensor([0, 3, 5], dtype=torch.int32, device=tr.device)
    cand = torch.tensor([1, 2, 4, 6, 7], dtype=torch.int32, device=tr.device)
    d_s = torch.zeros(5, dtype=torch.float32, device=tr.device)
    for k in (0, 1, 2, 3, 7, 100):
        B.odin_rlg_topk(tr.ctx, d_full, views, k, d_ret, ws)
        G.poll_ok(tr)
        want = oracle32.rlg_topk(full, k)
        assert np.array_equal(d_ret.cpu().numpy(), want)
        B.odin_sds_scores(tr.ctx, d_ret, views, prev, 3, cand, 5, d_s)
        G.poll_ok(tr)
        assert np.allclose(d_s.cpu().numpy(), oracle32.sds_scores(want, [0, 3, 5], [1, 2, 4, 6, 7]), rtol=1e-6, atol=1e-7)
    # equal weights: the lower index wins the last retained place
    tie = np.zeros((4, 4), np.float32)
    tie[0, 1] = tie[1, 0] = tie[0, 2] = tie[2, 0] = tie[0, 3] = tie[3, 0] = 0.25
    tie[2, 3] = tie[3, 2] = 0.5
    d_tie = torch.from_numpy(tie).to(tr.device)
    d_ret4 = torch.zeros((4, 4), dtype=torch.float32, device=tr.device)
    B.odin_rlg_topk(tr.ctx, d_tie, 4, 1, d_ret4, ws)
    G.poll_ok(tr)
    # item 0 keeps 1 (first of three equals), item 1 keeps 0, items 2 and 3 keep each other: {0,2} and {0,3} are dropped
    got = d_ret4.cpu().numpy()
    assert np.array_equal(got, oracle32.rlg_topk(tie, 1))
    assert got[0, 1] == 0.25 and got[0, 2] == 0 and got[0, 3] == 0 and got[2, 3] == 0.5
    # a pair that names a view that does not exist is reported
    bad = torch.tensor([[0, views]], dtype=torch.int32, device=tr.device)
    B.odin_rlg_weights(tr.ctx, d_counts, sizes, bad, 1, views, d_w)
    assert tr.poll() == B.ODIN_ERR_INVALID_ARG
    tr.close()


def admit_delayed_read(gate, active_count_a, tau):
    """The admission rule of Sec. 4.3 as the caller evaluates it from the four counts of odin_delayed_read_gate
    (#D+, #(D+ & C_A), #passing, #R+(B)): rho = #D+ / #R+(B) <= tau, C_A not empty, every delayed primitive has
    evidence and passes the gate."""
    n_delayed, n_with, n_pass, n_read_b = (int(x) for x in gate)
    return bool(n_read_b > 0 and n_delayed <= tau * n_read_b and active_count_a > 0 and n_with == n_delayed
                and n_pass == n_delayed)


def run_gate(ctx, dev, n, r_b, w_b, w_a, active_a, ev_a, tau, capacity=None):
    d_m, stride = to_device_masks([r_b, w_b, w_a], n, dev)
    cap = len(active_a) if capacity is None else capacity
    d_idx = torch.from_numpy(np.asarray(active_a, np.int32)).to(dev) if len(active_a) else torch.zeros(1, dtype=torch.int32, device=dev)
    d_ev = torch.from_numpy(np.asarray(ev_a, np.float32)).to(dev) if len(active_a) else torch.zeros(1, device=dev)
    d_cnt = torch.tensor([len(active_a)], dtype=torch.int32, device=dev)
    d_sum = torch.tensor([float(np.asarray(ev_a, np.float32).astype(np.float64).sum())], dtype=torch.float64, device=dev)
    d_gate = torch.full((4,), -1, dtype=torch.int64, device=dev)
    B.odin_delayed_read_gate(ctx, d_m[0], d_m[1], d_m[2], n, d_idx, d_ev, d_cnt, d_sum, cap, tau, d_gate)
    assert B.odin_poll(ctx) == B.ODIN_OK
    return d_gate.cpu().numpy()


def test_delayed_read_gate_hand_example(oracle32):
    from test_oracle_scope_pins import read_golden
    g = read_golden("delayed_read_gate_example.txt")
    ints = lambda k: np.array([int(x) for x in g[k]])  # noqa: E731
    ev = np.array([float(x) for x in g["evidence_A"]], np.float32)
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    for case in "1234":
        tau = float(g["tau" + case][0])
        gate = run_gate(ctx, dev, 32, ints("R_B" + case), ints("W_B" + case), ints("W_A"), ints("C_A"), ev, tau)
        assert gate.tolist() == [int(g["n_delayed" + case][0]), int(g["n_with_evidence" + case][0]),
                                 int(g["n_pass" + case][0]), len(ints("R_B" + case))]
        assert admit_delayed_read(gate, len(ints("C_A")), tau) == (g["admitted" + case][0] == "yes")
    B.odin_destroy(ctx)


@pytest.mark.parametrize("n", [33, 5000, 300_001])
def test_delayed_read_gate_random_scopes(oracle32, n):
    rng = np.random.default_rng(3 * n)
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    for trial in range(6):
        (r_a, r_b), (w_a, w_b) = random_scopes(rng, n, 2)
        # A's realized set: most of its write scope (so some delayed primitives lack evidence), heavy-tailed evidence
        active_a = np.sort(rng.choice(w_a, int(0.8 * len(w_a)), replace=False)) if len(w_a) else w_a
        ev_a = rng.lognormal(-2.0, 1.5, len(active_a)).astype(np.float32)
        tau = float(np.float32(rng.choice([0.05, 0.2, 0.5, 1.0])))
        want = oracle32.delayed_read_gate(r_a, w_a, r_b, w_b, active_a, ev_a, tau)
        gate = run_gate(ctx, dev, n, r_b, w_b, w_a, active_a, ev_a, tau)
        assert gate.tolist() == [want["n_delayed"], want["n_with_evidence"], want["n_pass"], want["n_read_b"]], trial
        assert admit_delayed_read(gate, len(active_a), tau) == want["admitted"]
    # with R+ = W+ nothing is ever delayed
    gate = run_gate(ctx, dev, n, w_b, w_b, w_a, active_a, ev_a, 0.2)
    assert gate[0] == 0 and gate[1] == 0
    B.odin_destroy(ctx)


# ------------------------------------------------------------------------------------------------ task unit of two views
def test_mask_to_list_and_accumulate_rows(oracle32):
    """The unit calls on their own: the list of a union mask against NumPy, the accumulated rows against the oracle's
    accumulate_rows (exact: one or two float additions per word), ragged sizes, a view with flagged zero rows."""
    rng = np.random.default_rng(17)
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    for n, da, db in ((70_001, 0.3, 0.2), (33, 0.5, 0.5), (3_000_000, 0.02, 0.05)):
        ia = np.flatnonzero(rng.random(n) < da).astype(np.uint32)
        ib = np.flatnonzero(rng.random(n) < db).astype(np.uint32)
        deg = 1
        f = 11 + 12
        ra, rb = rng.standard_normal((len(ia), f)).astype(np.float32), rng.standard_normal((len(ib), f)).astype(np.float32)
        za = (rng.random(len(ia)) < 0.3).astype(np.uint8)  # rows of view a that were flagged zero (their content is stale)
        ra_eff = ra.copy()
        ra_eff[za.astype(bool)] = 0
        union_o, rows_o = oracle32.accumulate_rows(ia, ra_eff, ib, rb)
        masks = torch.from_numpy(np.stack([oracle_mod.ids_to_mask(ia, n), oracle_mod.ids_to_mask(ib, n)]).view(np.int32)).to(dev)
        words = masks.shape[1]
        stride = (words + 3) // 4 * 4
        mpad = torch.zeros((2, stride), dtype=torch.int32, device=dev)
        mpad[:, :words] = masks
        umask = torch.zeros(stride, dtype=torch.int32, device=dev)
        members = torch.tensor([0, 1], dtype=torch.int32, device=dev)
        B.odin_mask_union(ctx, mpad, 2, stride, n, members, 2, umask)
        ws = torch.zeros(B.odin_workspace_bytes(ctx, n, 0), dtype=torch.uint8, device=dev)
        cap = len(union_o) + 3
        d_idx = torch.full((cap,), -1, dtype=torch.int32, device=dev)
        d_cnt = torch.zeros(1, dtype=torch.int32, device=dev)
        B.odin_mask_to_list(ctx, umask, n, d_idx, cap, d_cnt, ws)
        assert B.odin_poll(ctx) == B.ODIN_OK
        assert int(d_cnt.item()) == len(union_o)
        assert np.array_equal(d_idx.cpu().numpy().view(np.uint32)[: len(union_o)], union_o)

        def scene_of(rows, cap_rows):
            sc = E.DeviceScene(cap_rows, deg, dev)
            r = torch.from_numpy(rows).to(dev)
            k = len(rows)
            sc.means[:k] = r[:, 0:3]; sc.log_scales[:k] = r[:, 3:6]; sc.quats[:k] = r[:, 6:10]
            sc.opacity_logit[:k] = r[:, 10]; sc.sh[:k] = r[:, 11:].reshape(k, 4, 3)
            return sc

        sa, sb, su = scene_of(ra, len(ia) + 2), scene_of(rb, len(ib) + 1), E.DeviceScene(cap, deg, dev)
        t = lambda a, dt: torch.from_numpy(a.view(dt) if a.dtype != np.uint8 else a).to(dev)  # noqa: E731
        B.odin_accumulate_rows(ctx, sa.struct, t(za, np.uint8), t(ia, np.int32),
                               torch.tensor([len(ia)], dtype=torch.int32, device=dev), sb.struct, None, t(ib, np.int32),
                               torch.tensor([len(ib)], dtype=torch.int32, device=dev), d_idx, d_cnt, su.struct)
        assert B.odin_poll(ctx) == B.ODIN_OK
        assert np.array_equal(su.rows_as_matrix(len(union_o)), rows_o.astype(np.float32))
    B.odin_destroy(ctx)


def test_two_view_unit_step(oracle32):
    """Two views of preset 2 as one task unit against the oracle's unit_step: union list exact, accumulated rows inside
    the sum of the two views' gradient bars, Adam on every word of the union against the oracle's update of the
    device's own accumulated rows, untouched rows bitwise."""
    import gpu_util as G

    w = wl.make_workload(2, n=40_000)
    cams = [w.cameras[1], w.cameras[2]]
    tgts = [w.target(1), w.target(2)]
    tr = G.trainer_for(w.scene, cams[0], mask_slots=2)
    dev = tr.device
    p = w.scene.copy()
    m, v = p.zeros_like(), p.zeros_like()
    for step in (1, 2):  # the second unit runs on non-zero moments
        pre = [x.copy() for x in (p, m, v)]
        o = oracle32.unit_step(p, m, v, cams, tgts, w.lr, w.beta1, w.beta2, w.eps, step)
        tr.unit_step([B.make_camera(c) for c in cams], [torch.from_numpy(t).to(dev) for t in tgts], step, w.lr, w.beta1,
                     w.beta2, w.eps)
        G.poll_ok(tr)
        u = tr._unit
        nu = int(u["count_u"].item())
        idx_u = G.u32(u["idx_u"])[:nu]
        assert np.array_equal(idx_u, o["idx"])  # (no projection decision of these views sits on a threshold)
        rows_dev = u["grads_u"].rows_as_matrix(nu).astype(np.float64)
        # bar of a sum of two views = sum of the two bars
        bound = np.zeros_like(rows_dev)
        for view, cam in zip(o["views"], cams):
            _, g2d_abs = oracle32.render_bwd_blend(view["proj"], view["vals"], view["ranges"], cam, view["final_T"],
                                                   view["n_contrib"], view["dL_dout"], want_abs=True)
            b = G.rows_bound(oracle32, pre[0], cam, view["idx"], view["proj"].clamp_flags, view["rows"].astype(np.float64),
                             view["g2d"], g2d_abs)
            bound[np.searchsorted(idx_u, view["idx"])] += b
        err = np.abs(rows_dev - o["rows"])
        assert (err <= 8 * bound + 1e-30).mean() > 0.9995  # rows on fragile pixels are not singled out here
        # Adam on every word: the oracle's update applied to the device's accumulated rows
        names = ("means", "log_scales", "quats", "opacity_logit", "sh")
        q = [wl.Scene(p.sh_degree, *(np.ascontiguousarray(getattr(st, nm)[idx_u]) for nm in names)) for st in pre]
        oracle32.sparse_adam(q[0], q[1], q[2], rows_dev.astype(np.float32), np.arange(nu, dtype=np.uint32), w.lr, w.beta1,
                             w.beta2, w.eps, step)
        it = torch.from_numpy(idx_u.astype(np.int64)).to(dev)
        for st_dev, st_q, kind in ((tr.params, q[0], "p"), (tr.m, q[1], "m"), (tr.v, q[2], "v")):
            for t, nm in zip(st_dev.tensors(), names):
                got, want = t[it].cpu().numpy().astype(np.float64), getattr(st_q, nm).astype(np.float64)
                tol = 2e-5 * np.abs(want) + (2e-5 * float(w.lr.max()) if kind == "p" else 1e-30)
                if kind == "m":
                    tol = tol + 2e-5 * 1e-3  # first moments may be cancelled sums of terms up to ~1e-3
                assert np.all(np.abs(got - want) <= tol), (kind, nm)
        rest = np.setdiff1d(np.arange(p.n), idx_u)
        for t, h in zip(tr.params.tensors(), (p.means, p.log_scales, p.quats, p.opacity_logit, p.sh)):
            assert np.array_equal(t.cpu().numpy()[rest].view(np.uint32), h[rest].view(np.uint32))
        for st_dev, st_h in ((tr.params, p), (tr.m, m), (tr.v, v)):  # re-synchronise the oracle from the device
            for t, nm in zip(st_dev.tensors(), names):
                getattr(st_h, nm)[...] = t.cpu().numpy()
    tr.close()
