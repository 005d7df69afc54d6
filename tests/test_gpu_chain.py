"""End-to-end parity: whole training views through the C ABI against the oracle's view step (needs a GPU)."""
import numpy as np
import pytest
import torch

from paper_2607_19893_b200 import binding as B
from paper_2607_19893_b200 import workloads as wl

import gpu_util as G

pytestmark = pytest.mark.gpu


def run_chain(oracle32, w, steps, views, window=None, row_capacity=None, instance_capacity=None, cfg=None):
    """Runs `steps` views on both sides from the same start.  Both sides see the same parameters at every step
    because the oracle is re-synchronised from the device after each comparison (so one fragile decision cannot
    cascade); every step is compared on its own."""
    scene = w.scene
    n = scene.n
    cam0 = w.cameras[0]
    tr = G.trainer_for(scene, cam0, row_capacity=row_capacity, instance_capacity=instance_capacity,
                       mask_slots=max(len(views), 1), cfg=cfg)
    rng = np.random.default_rng(7)
    tr.keep_sorted_keys = True  # the sorted keys are compared below
    tr.track_active = True      # ... and the realized active set
    p = scene.copy()
    m, v = p.zeros_like(), p.zeros_like()
    masks_o = {}
    dev = tr.device
    n_fragile = 0
    for s in range(steps):
        view = views[s % len(views)]
        cam = w.cameras[view]
        tgt = w.target(view)
        pre = p.copy()  # parameters this view was rendered with
        o = oracle32.view_step(p, m, v, cam, tgt, w.lr, w.beta1, w.beta2, w.eps, s + 1)
        tr.target.copy_(torch.from_numpy(tgt).to(dev))
        slot = s % len(views)
        tr.view_step(B.make_camera(cam), s + 1, w.lr, w.beta1, w.beta2, w.eps, slot=slot)
        G.poll_ok(tr)
        # integer decisions of the projection may legitimately differ only on primitives that sit within a few
        # float ulps of a threshold; when none differs, every integer output of the chain must be bit exact
        fragile_prims = o["proj"].margin < 2e-6
        tt_dev = G.u32(tr.proj.tiles_touched)[:n]
        differs = tt_dev != o["proj"].tiles_touched
        assert not (differs & ~fragile_prims).any()
        n_fragile += int(differs.sum())
        vdev = int(tr.count.item())
        if not differs.any():
            # identical projected decisions: integer outputs are bit exact through the whole chain
            assert vdev == len(o["idx"])
            assert np.array_equal(G.u32(tr.idx)[:vdev], o["idx"])
            assert np.array_equal(G.u32(tr.masks[slot])[: len(o["mask"])], o["mask"])
            assert np.array_equal(G.u32(tr.proj.prim_id)[:vdev], o["idx"])
            mm = len(o["keys"])
            assert int(tr.proj.num_instances.item()) == mm
            rg = G.u32(tr.ranges)
            assert np.array_equal(rg[:, 1] - rg[:, 0], o["ranges"][:, 1] - o["ranges"][:, 0])
            # keys: tile ids are exact; depth bits come from the GPU projection (may differ in the last bit)
            assert np.array_equal(G.u64(tr.keys)[:mm] >> np.uint64(32), o["keys"] >> np.uint64(32))
        # realized active set of the view (row flags of the backward pass): inside the touched set; against the oracle
        # it may differ only by primitives whose activity hangs on a fragile pixel decision
        tr.active_set(slot=slot)
        G.poll_ok(tr)
        n_act = int(tr.active_count.item())
        act_dev = G.u32(tr.active_idx)[:n_act]
        assert not (G.u32(tr.active_masks[slot]) & ~G.u32(tr.masks[slot])).any()
        if not differs.any():
            _, act_o = oracle32.realized_active(o["proj"], o["vals"], o["ranges"], cam, o["n_contrib"])
            n_fragile_pix = int((o["pix_margin"] <= 2e-5).sum())
            assert len(np.setxor1d(act_dev, act_o)) <= max(4, n_fragile_pix)
            assert len(act_o) > 0
        robust = o["pix_margin"] > 1e-3
        out = tr.out.cpu().numpy()
        assert np.abs(out - o["out"])[:, robust].max() < 1e-4
        assert abs(float(tr.loss.item()) - o["loss"]) < 1e-5
        # updated state: compare the touched rows of params, m, v
        idx = o["idx"].astype(np.int64)
        host_state = [a for s_ in (p, m, v) for a in (s_.means, s_.log_scales, s_.quats, s_.opacity_logit, s_.sh)]
        dev_tensors = [t for s_ in (tr.params, tr.m, tr.v) for t in s_.tensors()]
        un = np.setdiff1d(np.arange(n), idx)
        if len(un) > 2_000_000:  # the largest scenes: a seeded sample of the untouched rows
            un = np.sort(rng.choice(un, 2_000_000, replace=False))
        un_dev, idx_dev = torch.from_numpy(un).to(dev), torch.from_numpy(idx).to(dev)
        for t, h in zip(dev_tensors, host_state):
            # untouched rows identical to the oracle's (which never changed them)
            assert np.array_equal(t[un_dev].cpu().numpy().view(np.uint32), h[un].view(np.uint32))
        dev_rows = [t[idx_dev].cpu().numpy() for t in dev_tensors]    # the touched rows, in row order
        host_rows = [h[idx] for h in host_state]
        # gradient rows: every word inside the bar derived from the un-cancelled term sums (see gpu_util)
        _, g2d_abs = oracle32.render_bwd_blend(o["proj"], o["vals"], o["ranges"], cam, o["final_T"], o["n_contrib"],
                                               o["dL_dout"], want_abs=True)
        rows = o["rows"].astype(np.float64)
        rows_dev = tr.gradient_rows(len(idx)).astype(np.float64)
        if not differs.any():
            bound = G.rows_bound(oracle32, pre, cam, o["idx"], o["proj"].clamp_flags, rows, o["g2d"], g2d_abs)
            # the chained run also carries the device's own projection and pixel rounding into the gradients
            assert (np.abs(rows_dev - rows) <= 4 * bound).mean() > 0.9999
        # Adam state and parameters.  With eps = 1e-15 a first Adam step is ~ lr * sign(g), so a gradient word that is
        # rounding noise (a cancelled sum) can legitimately move its parameter the other way: compare m, v and the
        # parameters wherever the two gradients agree to 1e-3 relative, and require that to be the bulk of the words.
        agree = np.abs(rows_dev - rows) <= 1e-3 * np.abs(rows)
        assert agree.mean() > 0.9, agree.mean()

        def as_rows(st):
            return np.concatenate([st[0], st[1], st[2], st[3][:, None], st[4].reshape(len(idx), -1)],
                                  axis=1).astype(np.float64)

        g_abs = np.abs(rows)
        dp, hp = as_rows(dev_rows[0:5]), as_rows(host_rows[0:5])
        dm, hm = as_rows(dev_rows[5:10]), as_rows(host_rows[5:10])
        dv, hv = as_rows(dev_rows[10:15]), as_rows(host_rows[10:15])
        assert np.all(np.abs(dm - hm)[agree] <= (1e-3 * (1 - w.beta1) * g_abs + 1e-6 * np.abs(hm) + 1e-30)[agree])
        assert np.all(np.abs(dv - hv)[agree] <= (2.1e-3 * (1 - w.beta2) * g_abs ** 2 + 1e-6 * np.abs(hv) + 1e-30)[agree])
        assert np.all(np.abs(dp - hp)[agree] <= 1e-3 * np.abs(hp)[agree] + 1e-5)
        masks_o[slot] = o["idx"]
        # re-synchronise the oracle's state from the device
        for s_dev, s_host in ((tr.params, p), (tr.m, m), (tr.v, v)):
            for t, a in zip(s_dev.tensors(), (s_host.means, s_host.log_scales, s_host.quats, s_host.opacity_logit, s_host.sh)):
                a[...] = t.cpu().numpy()
    # conflict counts over the latest mask of every view slot
    slots = sorted(masks_o)
    pairs = np.array([(a, b) for a in slots for b in slots if a < b], np.uint32).reshape(-1, 2)
    if len(pairs):
        d_pairs = torch.from_numpy(pairs.view(np.int32)).to(dev)
        d_counts = torch.zeros(len(pairs), dtype=torch.int64, device=dev)
        tr.conflict_count(d_pairs, len(pairs), d_counts)
        G.poll_ok(tr)
        want = np.array([oracle32.conflict_count(masks_o[a], masks_o[b]) for a, b in pairs], np.uint64)
        got = G.u64(d_counts)
        if n_fragile == 0:
            assert np.array_equal(got, want)
        else:
            assert np.all(np.abs(got.astype(np.int64) - want.astype(np.int64)) <= n_fragile)
    tr.close()


def test_chain_cfg1_one_step(oracle32):
    run_chain(oracle32, wl.make_workload(1), steps=1, views=[0])


def test_chain_cfg2_ten_steps_all_pairs(oracle32):
    # 100k splats, 8 orbit views, 10 steps cycling the views, then the 28 pairwise intersection counts
    run_chain(oracle32, wl.make_workload(2), steps=10, views=list(range(8)))


def test_chain_unbounded_scene_scaled(oracle32):
    w = wl.make_workload(3, n=100_000, n_cameras=4, resolution=(400, 267))
    run_chain(oracle32, w, steps=3, views=[0, 1, 2])


def test_chain_city_scaled(oracle32):
    w = wl.make_workload(5, n=300_000, n_cameras=4, resolution=(480, 270))
    run_chain(oracle32, w, steps=2, views=[0, 1])


def test_train_from_host_equals_the_plain_loop():
    """The double-buffered host-target loop is marshalling only: the same kernels on the same inputs, so losses, counts
    and the trained parameters are bitwise those of the plain loop (atomics aside: compared with a tolerance)."""
    w = wl.make_workload(2, n=30_000)
    steps = list(range(6))
    cams = [B.make_camera(c) for c in w.cameras]
    host_targets = [torch.from_numpy(w.target(v)).pin_memory() for v in range(len(w.cameras))]
    a = G.trainer_for(w.scene, w.cameras[0], mask_slots=3)
    b = G.trainer_for(w.scene, w.cameras[0], mask_slots=3)
    pairs = torch.tensor([[0, 1], [1, 2]], dtype=torch.int32, device=a.device)
    counts_a = torch.zeros(2, dtype=torch.int64, device=a.device)
    counts_b = torch.zeros(2, dtype=torch.int64, device=b.device)
    got = []
    a.train_from_host(steps, cam_of=lambda s: cams[s % 8], host_target_of=lambda s: host_targets[s % 8], lr=w.lr,
                      beta1=w.beta1, beta2=w.beta2, eps=w.eps, slot_of=lambda s: s % 3,
                      pairs_of=lambda s: (pairs, 2), d_counts=counts_a,
                      on_result=lambda s, loss, touched, counts: got.append((s, loss, touched, counts.tolist())))
    G.poll_ok(a)
    want = []
    for s in steps:
        b.target.copy_(host_targets[s % 8].to(b.device))
        b.view_step(cams[s % 8], s + 1, w.lr, w.beta1, w.beta2, w.eps, slot=s % 3, d_pairs=pairs, n_pairs=2,
                    d_counts=counts_b)
        G.poll_ok(b)
        want.append((s, float(b.loss.item()), int(b.count.item()), counts_b.cpu().tolist()))
    assert [g[0] for g in got] == steps
    for g, x in zip(got, want):
        assert g[2] == x[2] and g[3] == x[3] and abs(g[1] - x[1]) < 1e-6
    for ta, tb in zip(a.params.tensors(), b.params.tensors()):
        assert torch.allclose(ta, tb, rtol=1e-4, atol=1e-6)
    a.close(); b.close()


def test_chain_tight_extent_binning(oracle32):
    """The whole step with binning = 1 against the oracle in the same mode (every check of run_chain), and against
    the plain mode: fewer instances, the same image."""
    from test_gpu_stages import tight_oracle

    w = wl.make_workload(3, n=100_000, n_cameras=4, resolution=(400, 267))
    run_chain(tight_oracle(), w, steps=3, views=[0, 1, 2], cfg=B.default_config(binning=1))
    cam = w.cameras[1]
    outs, m = [], []
    for binning in (0, 1):
        tr = G.trainer_for(w.scene, cam, cfg=B.default_config(binning=binning))
        tr.target.copy_(torch.from_numpy(w.target(1)).to(tr.device))
        tr.view_step(B.make_camera(cam), 1, w.lr, w.beta1, w.beta2, w.eps, update=False)
        G.poll_ok(tr)
        outs.append(tr.out.cpu().numpy())
        m.append(int(tr.proj.num_instances.item()))
        tr.close()
    assert m[1] < 0.8 * m[0]
    assert np.array_equal(outs[0], outs[1])  # the same pairs blend in the same order: bitwise the same image


# ---------------------------------------------------------------------------------------------------------------
# The two workloads bench.py times, at full size and with the capacities it launches with.  Two consecutive steps, so
# the second one runs on non-zero Adam moments.  The oracle computes every output (a full view of these sizes takes
# it seconds); untouched rows of the 20 M scene are compared on a seeded sample of 2 M rows.
def test_chain_cfg3_full_size_as_benchmarked(oracle32):
    import bench

    w = wl.make_workload(3)
    run_chain(oracle32, w, steps=2, views=[0, 1], row_capacity=int(bench.ROW_CAP_FRAC[3] * w.scene.n),
              instance_capacity=bench.INSTANCE_CAP[3])


def test_chain_cfg5_full_size_as_benchmarked(oracle32):
    import bench

    w = wl.make_workload(5)
    row_cap = min(w.scene.n, max(int(bench.ROW_CAP_FRAC[5] * w.scene.n), 1_600_000))
    run_chain(oracle32, w, steps=2, views=[0, 1], row_capacity=row_cap, instance_capacity=bench.INSTANCE_CAP[5])
