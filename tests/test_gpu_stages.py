"""Stage-isolated parity of the CUDA library against the CPU oracle (needs a GPU).

Every stage is fed the ORACLE's outputs of the previous stages, so integer stages must agree bit for bit."""
import numpy as np
import pytest
import torch

from paper_2607_19893_b200 import binding as B
from paper_2607_19893_b200 import workloads as wl
from paper_2607_19893_b200.engine import DeviceScene

import gpu_util as G

pytestmark = pytest.mark.gpu

PIX_TOL = 1e-4          # absolute, rendered pixels


# ------------------------------------------------------------------------------------------------ touched set
@pytest.mark.parametrize("n", [1, 31, 32, 33, 2047, 2048, 2049, 100_003, 3_000_001])
def test_touched_set_bit_exact(oracle32, n):
    rng = np.random.default_rng(n)
    tt = ((rng.random(n) < 0.3) * rng.integers(1, 50, n)).astype(np.uint32)
    if n > 5000:
        tt[1000:4000] = 0          # a long empty run and a long full run
        tt[4000:9000] = 3
    mask_o, idx_o = oracle32.touched_set(tt)
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    d_tt = torch.from_numpy(tt.view(np.int32)).to(dev)
    words = (n + 31) // 32
    d_mask = torch.full((words,), -1, dtype=torch.int32, device=dev)
    d_idx = torch.full((n,), -1, dtype=torch.int32, device=dev)
    d_count = torch.zeros(1, dtype=torch.int32, device=dev)
    ws = torch.zeros(B.odin_workspace_bytes(ctx, n, 0), dtype=torch.uint8, device=dev)
    for _ in range(2):  # twice: the workspace is reused
        B.odin_touched_set(ctx, d_tt, n, d_mask, d_idx, n, d_count, ws)
        assert B.odin_poll(ctx) == B.ODIN_OK
        v = int(d_count.item())
        assert v == len(idx_o)
        assert np.array_equal(G.u32(d_mask), mask_o)
        assert np.array_equal(G.u32(d_idx[:v]), idx_o)
    # capacity smaller than V: truncated list, deferred error, nothing written past the capacity
    if len(idx_o) > 4:
        cap = len(idx_o) // 2
        d_idx.fill_(-1)
        B.odin_touched_set(ctx, d_tt, n, d_mask, d_idx, cap, d_count, ws)
        assert B.odin_poll(ctx) == B.ODIN_ERR_CAPACITY
        assert int(d_count.item()) == cap
        assert np.array_equal(G.u32(d_idx[:cap]), idx_o[:cap]) and bool((d_idx[cap:] == -1).all())
        assert B.odin_poll(ctx) == B.ODIN_OK  # cleared
    B.odin_destroy(ctx)


def test_touched_set_empty(oracle32):
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    d_count = torch.full((1,), 7, dtype=torch.int32, device=dev)
    B.odin_touched_set(ctx, None, 0, None, None, 0, d_count, None)
    assert B.odin_poll(ctx) == B.ODIN_OK and int(d_count.item()) == 0
    B.odin_destroy(ctx)


# ------------------------------------------------------------------------------------------------ conflict count
@pytest.mark.parametrize("n", [1, 127, 128, 129, 100_000, 5_000_001])
def test_conflict_count_bit_exact(oracle32, n):
    rng = np.random.default_rng(n + 1)
    views = 6
    dens = [0.0, 0.02, 0.3, 0.5, 0.97, 1.0]
    sets = [np.nonzero(rng.random(n) < d)[0].astype(np.uint32) for d in dens]
    words = (n + 31) // 32
    stride = (words + 3) // 4 * 4
    masks = np.zeros((views, stride), np.uint32)
    for i, s in enumerate(sets):
        np.bitwise_or.at(masks[i], s >> 5, np.uint32(1) << (s & 31))
    pairs = np.array([(a, b) for a in range(views) for b in range(views)], np.uint32)
    want = np.array([oracle32.conflict_count(sets[a], sets[b]) for a, b in pairs], np.uint64)
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    d_masks = torch.from_numpy(masks.view(np.int32)).to(dev)
    d_pairs = torch.from_numpy(pairs.view(np.int32)).to(dev)
    d_counts = torch.full((len(pairs),), -1, dtype=torch.int64, device=dev)
    B.odin_conflict_count(ctx, d_masks, views, stride, n, d_pairs, len(pairs), d_counts)
    assert B.odin_poll(ctx) == B.ODIN_OK
    assert np.array_equal(G.u64(d_counts), want)
    # a pair naming a missing view: deferred error, count 0
    bad = torch.tensor([[0, views]], dtype=torch.int32, device=dev)
    B.odin_conflict_count(ctx, d_masks, views, stride, n, bad, 1, d_counts)
    assert B.odin_poll(ctx) == B.ODIN_ERR_INVALID_ARG and int(d_counts[0].item()) == 0
    B.odin_destroy(ctx)


# ------------------------------------------------------------------------------------------------ Adam
@pytest.mark.parametrize("sh_degree,n,v", [(3, 5000, 1700), (0, 1024, 1024), (1, 999, 10), (2, 4001, 4001), (3, 300_000, 90_000)])
def test_sparse_adam_stage(oracle32, sh_degree, n, v):
    rng = np.random.default_rng(v)
    k = (sh_degree + 1) ** 2
    f = 11 + 3 * k

    def rand_scene(scale=1.0, positive=False):
        a = [rng.standard_normal(s).astype(np.float32) * np.float32(scale) for s in ((n, 3), (n, 3), (n, 4), (n,), (n, k, 3))]
        if positive:
            a = [np.abs(x) for x in a]
        return wl.Scene(sh_degree, *a)

    p, m, vv = rand_scene(), rand_scene(0.1), rand_scene(0.01, True)
    idx = np.sort(rng.choice(n, v, replace=False)).astype(np.uint32)
    rows = rng.standard_normal((v, f)).astype(np.float32)
    rows[rng.random((v, f)) < 0.1] = 0
    # a fifth of the rows have no gradient at all: on the device they are flagged, and what the gradient block holds
    # for them (here: NaN) must never be read
    zero_rows = rng.random(v) < 0.2
    rows[zero_rows] = 0
    rows_dev = rows.copy()
    rows_dev[zero_rows] = np.nan
    lr = np.array([1e-3, 2e-3, 5e-4, 1e-2, 3e-3, 1e-4], np.float32)
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    dp, dm, dv = (DeviceScene.from_host(s, dev) for s in (p, m, vv))
    g = wl.Scene(sh_degree, rows_dev[:, 0:3], rows_dev[:, 3:6], rows_dev[:, 6:10], rows_dev[:, 10],
                 rows_dev[:, 11:].reshape(v, k, 3))
    dg = DeviceScene.from_host(g, dev)
    d_zero = torch.from_numpy(zero_rows.astype(np.uint8)).to(dev)
    d_idx = torch.from_numpy(idx.view(np.int32)).to(dev)
    d_count = torch.tensor([v], dtype=torch.int32, device=dev)
    before = [t.clone() for s in (dp, dm, dv) for t in s.tensors()]
    for step in (1, 2, 7):
        oracle32.sparse_adam(p, m, vv, rows, idx, lr, 0.9, 0.999, 1e-15, step)
        B.odin_sparse_adam(ctx, dp.struct, dm.struct, dv.struct, dg.struct, d_zero, d_idx, d_count, lr, 0.9, 0.999, 1e-15,
                           step)
    assert B.odin_poll(ctx) == B.ODIN_OK
    after = [t for s in (dp, dm, dv) for t in s.tensors()]
    host = [a for s in (p, m, vv) for a in (s.means, s.log_scales, s.quats, s.opacity_logit, s.sh)]
    un = np.setdiff1d(np.arange(n), idx)
    for b, a, h in zip(before, after, host):
        a = a.cpu().numpy()
        assert np.allclose(a, h, rtol=2e-5, atol=1e-7)
        # untouched rows: bitwise identical
        assert np.array_equal(b.cpu().numpy()[un].view(np.uint32), a[un].view(np.uint32))
    # count = 0 on the device: nothing moves
    d_count.zero_()
    snap = [t.clone() for t in after]
    B.odin_sparse_adam(ctx, dp.struct, dm.struct, dv.struct, dg.struct, None, d_idx, d_count, lr, 0.9, 0.999, 1e-15, 8)
    assert B.odin_poll(ctx) == B.ODIN_OK
    for s, a in zip(snap, after):
        assert torch.equal(s, a)
    B.odin_destroy(ctx)


@pytest.mark.parametrize("sh_degree,eps", [(3, 1e-15), (0, 1e-8), (2, 0.0)])
def test_sparse_adam_live_flags(sh_degree, eps):
    """The update with per-primitive flags equals the update without them bit for bit, over several steps with changing
    row lists, zero rows (flagged and unflagged) and partially zero rows; the flags keep their promise (a clear flag
    means zero moments) and the refresh call gives exactly `any moment non-zero`."""
    rng = np.random.default_rng(11 + sh_degree)
    n, k = 20_000, (sh_degree + 1) ** 2
    f = 11 + 3 * k
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    p0 = wl.Scene(sh_degree, *[rng.standard_normal(s).astype(np.float32) for s in ((n, 3), (n, 3), (n, 4), (n,), (n, k, 3))])
    sides = []
    for _ in range(2):
        sides.append((DeviceScene.from_host(p0, dev), DeviceScene(n, sh_degree, dev), DeviceScene(n, sh_degree, dev)))
    live = torch.zeros(n, dtype=torch.uint8, device=dev)
    lr = np.array([1e-3, 2e-3, 5e-4, 1e-2, 3e-3, 1e-4], np.float32)

    def any_moment(m, v):
        return torch.stack([(t.reshape(n, -1) != 0).any(dim=1) for s in (m, v) for t in s.tensors()]).any(dim=0)

    for step in range(1, 7):
        v = int(rng.integers(2000, 9000))
        idx = np.sort(rng.choice(n, v, replace=False)).astype(np.uint32)
        rows = rng.standard_normal((v, f)).astype(np.float32)
        kind = rng.random(v)
        rows[kind < 0.5] = 0                         # no gradient at all ...
        flagged = kind < 0.3                         # ... most of them flagged, the gradient block then holds NaN
        part = (kind >= 0.5) & (kind < 0.7)          # gradient in a few words only
        rows[part] *= (rng.random((int(part.sum()), f)) < 0.05)
        rows_dev = rows.copy()
        rows_dev[flagged] = np.nan
        g = wl.Scene(sh_degree, rows_dev[:, 0:3], rows_dev[:, 3:6], rows_dev[:, 6:10], rows_dev[:, 10],
                     rows_dev[:, 11:].reshape(v, k, 3))
        dg = DeviceScene.from_host(g, dev)
        d_zero = torch.from_numpy(flagged.astype(np.uint8)).to(dev) if step % 3 else None
        if d_zero is None:                           # every third step without the row flags: zeros are read as zeros
            dg = DeviceScene.from_host(wl.Scene(sh_degree, rows[:, 0:3], rows[:, 3:6], rows[:, 6:10], rows[:, 10],
                                                rows[:, 11:].reshape(v, k, 3)), dev)
        d_idx = torch.from_numpy(idx.view(np.int32)).to(dev)
        d_count = torch.tensor([v], dtype=torch.int32, device=dev)
        (pa, ma, va), (pb, mb, vb) = sides
        B.odin_sparse_adam(ctx, pa.struct, ma.struct, va.struct, dg.struct, d_zero, d_idx, d_count, lr, 0.9, 0.999, eps, step)
        B.odin_sparse_adam_live(ctx, pb.struct, mb.struct, vb.struct, dg.struct, d_zero, d_idx, d_count, live, lr, 0.9,
                                0.999, eps, step)
        assert B.odin_poll(ctx) == B.ODIN_OK
        for sa, sb in zip(sides[0], sides[1]):
            for ta, tb in zip(sa.tensors(), sb.tensors()):
                assert torch.equal(ta.view(torch.int32), tb.view(torch.int32)), step
        truth = any_moment(mb, vb)
        assert not bool((truth & (live == 0)).any()), step        # a clear flag promises zero moments
        if eps > 0:
            assert int(live.sum().item()) < n                      # and the flags are not trivially all set
        fresh = torch.full((n,), 7, dtype=torch.uint8, device=dev)
        B.odin_adam_live_refresh(ctx, mb.struct, vb.struct, fresh)
        assert torch.equal(fresh.bool(), truth), step
    B.odin_destroy(ctx)


# ------------------------------------------------------------------------------------------------ projection
def check_projection(oracle32, scene, cam, row_capacity=None, cfg=None):
    tr = G.trainer_for(scene, cam, row_capacity=row_capacity, cfg=cfg)
    ccam = B.make_camera(cam)
    po = oracle32.project(scene, cam)
    for _ in range(2):
        tr.project(ccam)
        G.poll_ok(tr)
    tt = G.u32(tr.proj.tiles_touched)[: scene.n]
    # a primitive is "safe" when none of its integer decisions sits within ~30 float ulps of its threshold
    safe = po.margin > 2e-6
    assert safe.mean() > 0.995
    assert np.array_equal(tt[safe], po.tiles_touched[safe])
    v = int(tr.proj.num_rows.item())
    prim = G.u32(tr.proj.prim_id)[:v]
    assert np.array_equal(prim, np.nonzero(tt)[0])  # rows ascend with the primitive id and match tiles_touched
    assert int(tr.proj.num_instances.item()) == int(tt.astype(np.int64).sum())
    off = G.u32(tr.proj.tile_offset)[:v]
    assert np.array_equal(off, np.concatenate([[0], np.cumsum(tt[prim].astype(np.int64))[:-1]]).astype(np.uint32)[:v])
    ok = safe[prim] & (po.tiles_touched[prim] > 0)
    pp = prim[ok]
    rect = tr.proj.rect.cpu().numpy().view(np.uint16)[:v][ok]
    assert np.array_equal(rect.astype(np.int32), po.rect[pp])
    assert np.array_equal(tr.proj.radius.cpu().numpy()[:v][ok], po.radius[pp])
    assert np.array_equal(tr.proj.clamp_flags.cpu().numpy()[:v][ok], po.clamp_flags[pp])
    assert np.allclose(tr.proj.xy.cpu().numpy()[:v][ok], po.xy[pp], rtol=1e-5, atol=2e-3)
    assert np.allclose(tr.proj.depth.cpu().numpy()[:v][ok], po.depth[pp], rtol=1e-6)
    assert np.allclose(tr.proj.conic_opacity.cpu().numpy()[:v][ok], po.conic_o[pp], rtol=5e-4, atol=1e-7)
    assert np.allclose(tr.proj.rgb.cpu().numpy()[:v][ok], po.rgb[pp], rtol=1e-5, atol=2e-6)
    tr.close()
    return v


def test_project_cfg1(oracle32):
    w = wl.make_workload(1)
    assert check_projection(oracle32, w.scene, w.cameras[0]) == 1024


@pytest.mark.parametrize("view", [0, 5])
def test_project_cfg2(oracle32, view):
    w = wl.make_workload(2)
    check_projection(oracle32, w.scene, w.cameras[view])


def test_project_unbounded_ragged(oracle32):
    w = wl.make_workload(3, n=300_007, resolution=(800, 533))
    check_projection(oracle32, w.scene, w.cameras[3])


def test_project_city_low_visibility(oracle32):
    w = wl.make_workload(5, n=400_000, n_cameras=4)
    for c in (0, 1):
        v = check_projection(oracle32, w.scene, w.cameras[c])
        assert 0 < v < 0.1 * w.scene.n


@pytest.mark.parametrize("deg", [1, 2])
def test_project_other_sh_degrees(oracle32, deg):
    w = wl.make_workload(2, n=20_000)
    s = w.scene
    k = (deg + 1) ** 2
    s2 = wl.Scene(deg, s.means, s.log_scales, s.quats, s.opacity_logit, np.ascontiguousarray(s.sh[:, :k]))
    check_projection(oracle32, s2, w.cameras[1])


def tight_oracle():
    import oracle
    from oracle.oracle import DEFAULT_CFG
    cfg = DEFAULT_CFG.copy()
    cfg[7] = 1
    return oracle.Oracle(np.float32, cfg=cfg)


def test_project_tight_extent_binning(oracle32):
    """binning = 1: the rectangles (and with them tiles_touched, rows, offsets) are those of the oracle's tight rule."""
    ot = tight_oracle()
    w = wl.make_workload(3, n=200_000, resolution=(800, 533))
    v_tight = check_projection(ot, w.scene, w.cameras[2], cfg=B.default_config(binning=1))
    po, pt = oracle32.project(w.scene, w.cameras[2]), ot.project(w.scene, w.cameras[2])
    assert v_tight <= int((po.tiles_touched > 0).sum())
    assert int(pt.tiles_touched.sum()) < 0.8 * int(po.tiles_touched.sum())
    w2 = wl.make_workload(2, n=50_000)
    check_projection(ot, w2.scene, w2.cameras[6], cfg=B.default_config(binning=1))


def exact_oracle():
    import oracle
    from oracle.oracle import DEFAULT_CFG
    cfg = DEFAULT_CFG.copy()
    cfg[7] = 2
    return oracle.Oracle(np.float32, cfg=cfg)


def test_project_exact_binning(oracle32):
    """binning = 2: tiles_touched counts the tiles the region alpha >= alpha_min reaches, as the oracle's exact rule has
    it; primitives that keep no tile leave the touched set."""
    oe = exact_oracle()
    w = wl.make_workload(3, n=200_000, resolution=(800, 533))
    v_exact = check_projection(oe, w.scene, w.cameras[2], cfg=B.default_config(binning=2))
    po, pe = oracle32.project(w.scene, w.cameras[2]), oe.project(w.scene, w.cameras[2])
    assert v_exact <= int((po.tiles_touched > 0).sum())
    assert int(pe.tiles_touched.sum()) < 0.7 * int(po.tiles_touched.sum())
    w2 = wl.make_workload(4, n=60_000, n_cameras=4, resolution=(960, 540))  # large splats: long spans, the bisection
    check_projection(oe, w2.scene, w2.cameras[1], cfg=B.default_config(binning=2))


def test_bin_sort_exact_binning(oracle32):
    """binning = 2 through odin_bin_sort: the device recomputes the spans from the rows it is given (here the oracle's)
    and must produce the oracle's lists.  Its logarithm may differ from the host's in the last place, so a primitive
    with a tile decision within 1e-5 of the threshold is left out of the comparison on both sides."""
    oe = exact_oracle()
    for w, cam_i in ((wl.make_workload(3, n=120_000), 7), (wl.make_workload(4, n=40_000, n_cameras=4, resolution=(960, 540)), 1)):
        cam = w.cameras[cam_i]
        po = oe.project(w.scene, cam)
        mask, idx = oe.touched_set(po.tiles_touched)
        keys_o, vals_o, ranges_o = oe.bin_sort(po, cam)
        m = len(keys_o)
        tr = G.trainer_for(w.scene, cam, row_capacity=max(len(idx), 1), instance_capacity=m + 4096,
                           cfg=B.default_config(binning=2))
        G.load_oracle_projection(tr, po, idx)
        tr.keys.fill_(-1)
        tr.vals.fill_(-1)
        tr.bin_sort()
        G.poll_ok(tr)
        rg = G.u32(tr.ranges).astype(np.int64)
        m_dev = int(rg[-1, 1])
        keys_d, prims_d = G.u64(tr.keys)[:m_dev], idx[G.u32(tr.vals)[:m_dev]]
        assert np.all(keys_d[1:] >= keys_d[:-1])
        assert np.array_equal(np.repeat(np.arange(len(rg)), rg[:, 1] - rg[:, 0]), (keys_d >> np.uint64(32)).astype(np.int64))
        fragile = po.margin < 1e-5
        keep_d, keep_o = ~fragile[prims_d], ~fragile[vals_o]
        assert np.array_equal(keys_d[keep_d], keys_o[keep_o]) and np.array_equal(prims_d[keep_d], vals_o[keep_o])
        G.report("bin_sort exact", M=m, M_dev=m_dev, fragile_prims=int(fragile[idx].sum()), rows=len(idx))
        assert abs(m_dev - m) <= int(po.tiles_touched[fragile].sum()) and fragile[idx].mean() < 0.01
        tr.close()


def test_project_large_scene_two_kernels(oracle32):
    """Scenes of more than 2048 x 4 x 148 primitives do not take the fused kernel: a counting kernel (one thread per
    primitive, leaving packed totals per 256 primitives and exact totals per chunk) and a scan that starts from a sum
    over the chunks in front of it.  A ragged count just above the limit, both the rectangle rule and exact binning, the
    touched bitmask as a by-product, and truncation at the row capacity."""
    n = 2048 * 4 * 148 + 2048 * 3 + 77
    w = wl.make_workload(5, n=n, n_cameras=4)
    cam = w.cameras[1]
    v = check_projection(oracle32, w.scene, cam)
    assert 0 < v < 0.2 * n
    check_projection(exact_oracle(), w.scene, cam, cfg=B.default_config(binning=2))
    # the bitmask written by the scan, and row-capacity truncation, on this path
    tr = G.trainer_for(w.scene, cam, row_capacity=v // 2)
    words = (n + 31) // 32
    mask = torch.full((words + 8,), -1, dtype=torch.int32, device=tr.device)
    tr.proj.struct.touched_mask = mask[4:].data_ptr()
    tr.proj.prim_id.fill_(-1)
    tr.project(B.make_camera(cam))
    assert tr.poll() == B.ODIN_ERR_CAPACITY
    assert int(tr.proj.num_rows.item()) == v // 2
    tt = G.u32(tr.proj.tiles_touched)[:n]
    want = np.flatnonzero(tt)
    assert len(want) == v
    assert np.array_equal(G.u32(tr.proj.prim_id)[: v // 2], want[: v // 2])
    bits = np.unpackbits(G.u32(mask[4:4 + words]).view(np.uint8), bitorder="little")[:n]
    assert np.array_equal(bits, (tt > 0).astype(np.uint8))
    assert (mask[:4] == -1).all() and (mask[4 + words:] == -1).all()
    tr.proj.struct.touched_mask = None
    tr.close()


def test_project_row_capacity_overflow(oracle32):
    w = wl.make_workload(1)
    tr = G.trainer_for(w.scene, w.cameras[0], row_capacity=100)
    tr.proj.prim_id.fill_(-1)
    tr.project(B.make_camera(w.cameras[0]))
    assert tr.poll() == B.ODIN_ERR_CAPACITY
    assert int(tr.proj.num_rows.item()) == 100
    assert np.array_equal(G.u32(tr.proj.prim_id), np.arange(100))  # the first 100 rows, nothing beyond
    tr.close()


# ------------------------------------------------------------------------------------------------ bin / sort
# instance_sort 0: the counting scatter (radix passes only for images beyond its tile limits); 1: always the radix passes
SORT_PATHS = [0, 1]


def check_bin_sort(oracle32, scene, cam, instance_capacity=None, instance_sort=0):
    po = oracle32.project(scene, cam)
    mask, idx = oracle32.touched_set(po.tiles_touched)
    keys_o, vals_o, ranges_o = oracle32.bin_sort(po, cam)
    m = len(keys_o)
    tr = G.trainer_for(scene, cam, row_capacity=max(len(idx), 1),
                       instance_capacity=instance_capacity if instance_capacity is not None else m + 17,
                       cfg=B.default_config(instance_sort=instance_sort))
    G.load_oracle_projection(tr, po, idx)
    inv = np.full(scene.n, -1, np.int64)
    inv[idx] = np.arange(len(idx))
    for want_keys in (True, True, False):  # twice with the keys (workspace reuse), once without (values only)
        tr.keys.fill_(-1)
        tr.vals.fill_(-1)
        tr.bin_sort(want_keys=want_keys)
        G.poll_ok(tr)
        if want_keys:
            assert np.array_equal(G.u64(tr.keys)[:m], keys_o)
        else:
            assert bool((tr.keys == -1).all())
        assert np.array_equal(G.u32(tr.vals)[:m], G.rows_of(inv, vals_o).astype(np.uint32))
        rg = G.u32(tr.ranges)
        assert np.array_equal(rg[:, 1] - rg[:, 0], ranges_o[:, 1] - ranges_o[:, 0])
        ne = ranges_o[:, 1] > ranges_o[:, 0]
        assert np.array_equal(rg[ne], ranges_o[ne])
    tr.close()
    return m


@pytest.mark.parametrize("path", SORT_PATHS)
def test_bin_sort_cfg1(oracle32, path):
    w = wl.make_workload(1)
    check_bin_sort(oracle32, w.scene, w.cameras[0], instance_sort=path)


@pytest.mark.parametrize("path", SORT_PATHS)
def test_bin_sort_cfg2(oracle32, path):
    w = wl.make_workload(2)
    m = check_bin_sort(oracle32, w.scene, w.cameras[2], instance_sort=path)
    assert m > 3 * 4096  # several sort tiles / chunks of rows and a ragged tail


@pytest.mark.parametrize("path", SORT_PATHS)
def test_bin_sort_many_tiles_six_passes(oracle32, path):
    w = wl.make_workload(3, n=120_000)  # 6700 tiles -> 13 tile bits -> 6 digit passes, ~1.2M instances
    m = check_bin_sort(oracle32, w.scene, w.cameras[7], instance_sort=path)
    assert m > 500_000


def test_bin_sort_large_splats_many_rows_per_band(oracle32):
    """Preset 4's large splats at 960 x 540: a chunk of 2048 sorted rows puts hundreds of rows into every band of tile
    rows (several sub-batches of the scatter's bit matrix), and rectangles span many bands."""
    w = wl.make_workload(4, n=150_000, n_cameras=4, resolution=(960, 540))
    m = check_bin_sort(oracle32, w.scene, w.cameras[1])
    assert m > 1_500_000


def test_bin_sort_image_of_73728_tiles(oracle32):
    """8192 x 2304 pixels = 512 x 144 tiles: three passes over the tile-id digits, and more tiles than the
    shared-memory staging of the per-tile counts holds (the counts then go straight to global memory)."""
    w = wl.make_workload(3, n=20_000, resolution=(8192, 2304))
    cam = w.cameras[5]
    assert ((cam.width + 15) // 16) * ((cam.height + 15) // 16) == 73728
    m = check_bin_sort(oracle32, w.scene, cam)
    assert m > 1_000_000


@pytest.mark.parametrize("path", SORT_PATHS)
def test_bin_sort_image_of_one_tile(oracle32, path):
    w = wl.make_workload(1, resolution=(16, 16))
    check_bin_sort(oracle32, w.scene, w.cameras[0], instance_sort=path)


@pytest.mark.parametrize("path", SORT_PATHS)
def test_bin_sort_equal_depth_ties(oracle32, path):
    # many identical splats: identical keys, order decided by the row index alone
    w = wl.make_workload(1)
    s = w.scene
    rep = lambda a: np.ascontiguousarray(np.repeat(a[:3], 3000, axis=0))  # noqa: E731
    s2 = wl.Scene(0, rep(s.means), rep(s.log_scales), rep(s.quats), rep(s.opacity_logit), rep(s.sh))
    check_bin_sort(oracle32, s2, w.cameras[0], instance_sort=path)


@pytest.mark.parametrize("path", SORT_PATHS)
def test_bin_sort_empty_view(oracle32, path):
    w = wl.make_workload(1)
    s = w.scene.copy()
    s.means[:, 2] = -5.0  # everything behind the camera
    check_bin_sort(oracle32, s, w.cameras[0], instance_sort=path)


@pytest.mark.parametrize("path", SORT_PATHS)
def test_bin_sort_instance_capacity_overflow(oracle32, path):
    """More instances than the caller's capacity: the instances of the nearest rows are kept (the first `capacity` of
    the depth order, a row's rectangle in row-major order), sorted; nothing is written beyond the capacity."""
    w = wl.make_workload(1)
    cam = w.cameras[0]
    po = oracle32.project(w.scene, cam)
    mask, idx = oracle32.touched_set(po.tiles_touched)
    cap = 1000
    tr = G.trainer_for(w.scene, cam, instance_capacity=cap + 64, cfg=B.default_config(instance_sort=path))
    tr.instance_capacity = cap  # the buffers are 64 entries longer than the capacity the call is told
    G.load_oracle_projection(tr, po, idx)
    tr.keys.fill_(-1)
    tr.vals.fill_(-1)
    tr.bin_sort()
    assert tr.poll() == B.ODIN_ERR_CAPACITY
    assert bool((tr.keys[cap:] == -1).all()) and bool((tr.vals[cap:] == -1).all())
    # expected: emission order = rows by (depth bits, row), each rectangle row major; keep the first `cap`; stable sort
    bits = po.depth[idx].astype(np.float32).view(np.uint32)
    order = np.lexsort((np.arange(len(idx)), bits))
    tx = tr.tx
    tiles, rows = [], []
    for r in order:
        x0, y0, x1, y1 = po.rect[idx[r]]
        for yy in range(y0, y1):
            for xx in range(x0, x1):
                tiles.append(yy * tx + xx)
                rows.append(r)
    tiles, rows = np.array(tiles[:cap], np.int64), np.array(rows[:cap], np.int64)
    final = np.argsort(tiles, kind="stable")
    keys = G.u64(tr.keys)[:cap]
    assert np.array_equal(G.u32(tr.vals)[:cap], rows[final].astype(np.uint32))
    assert np.array_equal(keys, (tiles[final].astype(np.uint64) << np.uint64(32)) | bits[rows[final]].astype(np.uint64))
    rg = G.u32(tr.ranges).astype(np.int64)
    assert np.array_equal(rg[:, 1] - rg[:, 0], np.bincount(tiles, minlength=len(rg)))
    tr.close()


# ------------------------------------------------------------------------------------------------ forward
def oracle_view(oracle32, scene, cam):
    f = oracle32.view_forward(scene, cam)
    inv = np.full(scene.n, -1, np.int64)
    inv[f["idx"]] = np.arange(len(f["idx"]))
    return f, inv


def load_sorted(tr, f, inv):
    G.load_oracle_projection(tr, f["proj"], f["idx"])
    m = len(f["vals"])
    tr.vals[:m].copy_(torch.from_numpy(G.rows_of(inv, f["vals"]).astype(np.int32)).to(tr.device))
    tr.ranges.copy_(torch.from_numpy(f["ranges"].view(np.int32)).to(tr.device))


def check_forward(oracle32, scene, cam, min_robust=1 - 2e-3, extra_render_records=0, expect_status=B.ODIN_OK):
    f, inv = oracle_view(oracle32, scene, cam)
    tr = G.trainer_for(scene, cam, row_capacity=max(len(f["idx"]), 1), instance_capacity=len(f["vals"]) + 1,
                       extra_render_records=extra_render_records)
    load_sorted(tr, f, inv)
    tr.render_fwd(B.make_camera(cam))
    assert tr.poll() == expect_status
    out = tr.out.cpu().numpy()
    ft = tr.final_T.cpu().numpy()
    nc = G.u32(tr.n_contrib)
    # the device evaluates exp with ex2.approx (relative error ~1e-6): a threshold test within 2e-5 may flip
    robust = f["pix_margin"] > 2e-5
    assert robust.mean() > min_robust
    assert np.abs(out - f["out"])[:, robust].max() < PIX_TOL
    assert np.abs(ft - f["final_T"])[robust].max() < PIX_TOL
    assert np.array_equal(nc[robust], f["n_contrib"][robust])
    # fragile pixels (a decision within 1e-4 of its threshold) may flip one contribution: bounded by alpha * T <= 1/255
    # for the skip test and by 1e-4 for termination; they still have to stay close
    assert np.abs(out - f["out"]).max() < 5e-3
    tr.close()
    return f


def test_render_fwd_cfg1(oracle32):
    w = wl.make_workload(1)
    check_forward(oracle32, w.scene, w.cameras[0])


def test_render_fwd_cfg2(oracle32):
    w = wl.make_workload(2)
    cam = w.cameras[4]
    cam.bg = np.array([0.2, 0.5, 0.9])
    check_forward(oracle32, w.scene, cam)


def test_render_fwd_ragged_image_long_lists(oracle32):
    w = wl.make_workload(3, n=150_000, resolution=(410, 275))  # edge tiles, lists of several batches
    f = check_forward(oracle32, w.scene, w.cameras[1])
    assert (f["ranges"][:, 1] - f["ranges"][:, 0]).max() > 600


# ------------------------------------------------------------------------------------------------ loss
def test_l1_loss(oracle32):
    rng = np.random.default_rng(0)
    w_, h_ = 333, 77
    out = rng.random((3, h_, w_), dtype=np.float32)
    tgt = rng.random((3, h_, w_), dtype=np.float32)
    tgt[0, :5] = out[0, :5]  # exact zeros
    loss_o, g_o = oracle32.l1_loss(out, tgt)
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    d_out, d_tgt = torch.from_numpy(out).to(dev), torch.from_numpy(tgt).to(dev)
    d_loss = torch.zeros(1, device=dev)
    d_g = torch.zeros_like(d_out)
    B.odin_l1_loss(ctx, d_out, d_tgt, w_, h_, d_loss, d_g)
    assert B.odin_poll(ctx) == B.ODIN_OK
    assert abs(float(d_loss.item()) - loss_o) < 1e-6 * max(1.0, loss_o)
    assert np.array_equal(d_g.cpu().numpy(), g_o)
    # images that start 4 bytes into their allocations (no 16-byte alignment): the element-wise path
    count = out.size
    bufs = [torch.zeros(count + 1, device=dev) for _ in range(3)]
    m_out, m_tgt, m_g = (b[1:] for b in bufs)
    m_out.copy_(d_out.flatten())
    m_tgt.copy_(d_tgt.flatten())
    d_loss.zero_()
    B.odin_l1_loss(ctx, m_out, m_tgt, w_, h_, d_loss, m_g)
    assert B.odin_poll(ctx) == B.ODIN_OK
    assert abs(float(d_loss.item()) - loss_o) < 1e-6 * max(1.0, loss_o)
    assert np.array_equal(m_g.cpu().numpy().reshape(g_o.shape), g_o)
    B.odin_destroy(ctx)


# ------------------------------------------------------------------------------------------------ backward
def check_backward(oracle32, scene, cam, seed=0, min_robust=1 - 2e-3, extra_render_records=0):
    f, inv = oracle_view(oracle32, scene, cam)
    rng = np.random.default_rng(seed)
    dl = rng.uniform(-1, 1, f["out"].shape).astype(np.float32)
    # The backward pass re-takes the skip decisions of every (pixel, row) pair.  On a pixel where one of them sits
    # within float rounding of its threshold the two sides may replay a different set of rows, which is a different
    # (equally valid) function: such pixels (a fraction < 2e-3) get no incoming gradient here.
    robust = f["pix_margin"] > 2e-5
    assert robust.mean() > min_robust
    dl[:, ~robust] = 0
    g2d_o, g2d_abs = oracle32.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], dl,
                                               want_abs=True)
    rows_o = oracle32.render_bwd_project(scene, cam, f["idx"], g2d_o, f["proj"].clamp_flags).astype(np.float64)
    v = len(f["idx"])
    tr = G.trainer_for(scene, cam, row_capacity=max(v, 1), instance_capacity=len(f["vals"]) + 1,
                       extra_render_records=extra_render_records)
    load_sorted(tr, f, inv)
    # the backward pass starts the later segments of long lists from the per-pixel states the forward pass leaves in
    # the workspace; everything else it reads is the oracle's
    tr.render_fwd(B.make_camera(cam))
    tr.final_T.copy_(torch.from_numpy(f["final_T"]).to(tr.device))
    tr.n_contrib.copy_(torch.from_numpy(f["n_contrib"].view(np.int32)).to(tr.device))
    tr.dL.copy_(torch.from_numpy(dl).to(tr.device))
    for _ in range(2):  # twice: accumulators are re-zeroed, atomics order changes
        tr.render_bwd(B.make_camera(cam))
        G.poll_ok(tr)
        g2d = tr.grad2d.cpu().numpy()[:v].astype(np.float64)
        want2d, abs2d = g2d_o[f["idx"]], g2d_abs[f["idx"]]
        err = np.abs(g2d - want2d)
        bad = err > G.grad2d_bound(want2d, abs2d)
        assert not bad.any(), (int(bad.sum()), np.argwhere(bad)[:5], err[bad][:5], want2d[bad][:5], abs2d[bad][:5])
        assert np.abs(want2d).max() > 1e-3
        rows = tr.gradient_rows(v).astype(np.float64)
        bound = G.rows_bound(oracle32, scene, cam, f["idx"], f["proj"].clamp_flags, rows_o, g2d_o, g2d_abs)
        err = np.abs(rows - rows_o)
        bad = err > bound
        plain = err <= 1e-3 * np.abs(rows_o) + 1e-5
        G.report("bwd_stage rows", words=err.size, over_1x=float(bad.mean()), worst=float((err / bound).max()),
                 plain_bar=float(plain.mean()), rows_absmax=float(np.abs(rows_o).max()))
        # every word inside the bar (it includes a few ulp of the row's largest word for the cancellation inside a
        # Jacobian entry, e.g. the conic-to-covariance step of a nearly degenerate conic)
        assert not bad.any(), (int(bad.sum()), np.argwhere(bad)[:5], err[bad][:5], rows_o[bad][:5], bound[bad][:5])
        # with an incoming gradient of O(1) per pixel (not the 1/(3HW) of a real loss) the words are sums of hundreds
        # of O(1) terms; those that are not cancelled sums also meet the plain bar: 1e-3 relative, 1e-5 absolute floor
        assert plain.mean() > 0.999, plain.mean()
    tr.close()


def test_render_bwd_cfg1(oracle32):
    w = wl.make_workload(1)
    check_backward(oracle32, w.scene, w.cameras[0])


def test_render_bwd_cfg2(oracle32):
    w = wl.make_workload(2, n=30_000)
    cam = w.cameras[6]
    cam.bg = np.array([0.3, 0.1, 0.7])
    check_backward(oracle32, w.scene, cam, seed=3)


def test_render_bwd_ragged_image_other_degree(oracle32):
    w = wl.make_workload(3, n=60_000, resolution=(410, 275))
    s = w.scene
    s2 = wl.Scene(1, s.means, s.log_scales, s.quats, s.opacity_logit, np.ascontiguousarray(s.sh[:, :4]))
    check_backward(oracle32, s2, w.cameras[2], seed=5)


# ------------------------------------------------------------------------------------------------ long lists
def faint_scene(n=20_000, seed=9):
    """Many faint splats on a small image: no pixel saturates, so every tile walks thousands of list entries and
    both the one-warp head kernels and the eight-warp tail kernels are exercised."""
    w = wl.make_workload(1, n=n)
    s = w.scene.copy()
    rng = np.random.default_rng(seed)
    s.opacity_logit[:] = rng.uniform(-5.2, -3.5, n).astype(np.float32)
    s.log_scales[:] = (-2.6 + 0.3 * rng.standard_normal((n, 3))).astype(np.float32)
    cam = w.cameras[0]
    cam.bg = np.array([0.4, 0.2, 0.6])
    return s, cam


def test_render_fwd_lists_longer_than_the_head(oracle32):
    s, cam = faint_scene()
    # thousands of pairs per pixel: proportionally more pixels have one pair near a threshold
    f = check_forward(oracle32, s, cam, min_robust=0.98)
    assert f["n_contrib"].max() > 1500 and (f["ranges"][:, 1] - f["ranges"][:, 0]).min() > 512


def test_render_bwd_lists_longer_than_the_head(oracle32):
    s, cam = faint_scene(n=12_000, seed=10)
    check_backward(oracle32, s, cam, seed=11, min_robust=0.98)


def test_render_bwd_with_a_workspace_that_is_not_the_forward_pass_s(oracle32):
    """The backward pass reads segment records from the render workspace.  A workspace that holds something else
    (here: every byte 0xff, then every byte 0) must not lead it outside its buffers: every record is checked before
    use, the call completes, and what it computes without usable records is finite (exact wherever a list ends within
    its first 256 entries)."""
    s, cam = faint_scene(n=12_000, seed=10)
    f, inv = oracle_view(oracle32, s, cam)
    v = len(f["idx"])
    tr = G.trainer_for(s, cam, row_capacity=v, instance_capacity=len(f["vals"]) + 1)
    load_sorted(tr, f, inv)
    tr.render_fwd(B.make_camera(cam))
    G.poll_ok(tr)
    tr.dL.fill_(1.0 / 3.0)
    for byte in (0xFF, 0x00):
        tr.render_ws.fill_(byte)
        tr.render_bwd(B.make_camera(cam))
        G.poll_ok(tr)
        assert torch.isfinite(tr.grad2d[:v]).all()
        assert torch.isfinite(torch.from_numpy(tr.gradient_rows(v))).all()
    tr.close()


def test_render_fwd_mixed_short_and_long_lists(oracle32):
    # half of the image crowded with faint splats (tail kernel), the other half nearly empty (head kernel only)
    s, cam = faint_scene(n=16_000, seed=12)
    s.means[:, 0] = np.abs(s.means[:, 0])
    f = check_forward(oracle32, s, cam, min_robust=0.98)
    lens = f["ranges"][:, 1] - f["ranges"][:, 0]
    assert lens.min() < 512 < lens.max()
    check_backward(oracle32, s, cam, seed=13, min_robust=0.98)


def one_tile_scene_with_a_list_of_a_million(n_faint=1_060_000, n_solid=48, seed=21):
    """A 16x16 image (one tile) in front of which lie a million splats too faint to pass the alpha threshold, and a
    few ordinary ones behind them: the forward pass has to walk the whole list before anything blends, more than 4,100
    batches of 256 entries, each of which takes a segment record."""
    rng = np.random.default_rng(seed)
    n = n_faint + n_solid
    means = np.zeros((n, 3), np.float32)
    means[:, :2] = rng.uniform(-0.08, 0.08, (n, 2))
    means[:n_faint, 2] = rng.uniform(2.0, 4.0, n_faint)
    means[n_faint:, 2] = rng.uniform(5.0, 6.0, n_solid)
    log_scales = np.full((n, 3), np.log(0.05), np.float32) + 0.2 * rng.standard_normal((n, 3)).astype(np.float32)
    quats = rng.standard_normal((n, 4)).astype(np.float32)
    opacity_logit = np.full(n, np.log(0.003 / 0.997), np.float32)       # 0.003 < 1/255: never blends
    opacity_logit[n_faint:] = rng.uniform(-2.0, 0.0, n_solid).astype(np.float32)
    sh = rng.uniform(-1.0, 2.0, (n, 1, 3)).astype(np.float32)
    scene = wl.Scene(0, means, log_scales, quats, opacity_logit, sh)
    w2c = np.concatenate([np.eye(3), np.zeros((3, 1))], axis=1)
    cam = wl.Camera(16, 16, 64.0, 64.0, 8.0, 8.0, 0.2, 1.0e9, w2c, np.array([0.3, 0.1, 0.5]))
    return scene, cam


def test_render_more_segments_than_the_minimum_workspace_records(oracle32):
    s, cam = one_tile_scene_with_a_list_of_a_million()
    # the minimum render workspace of a one-tile image holds 2 + 4096 records: the image is still exact, the forward
    # call reports that the backward pass will lack records
    f = check_forward(oracle32, s, cam, expect_status=B.ODIN_ERR_CAPACITY)
    assert f["n_contrib"].max() > 1_050_000 and len(f["vals"]) > 1_050_000
    # with room for the ~4,140 records: no error, and the backward pass (one warp per segment, 4,140 of them for the one
    # tile, all but the last without a single contribution) meets the same bar as everywhere else
    check_forward(oracle32, s, cam, extra_render_records=256)
    check_backward(oracle32, s, cam, seed=22, extra_render_records=256)
