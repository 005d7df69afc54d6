"""Failure detection without a fault (needs a GPU): a bounded device-side wait that runs out, and checkpoint / resume.

The look-back of the prefix scans and of the radix sort waits for words that other thread blocks publish.  Every such
wait has a poll limit; when it runs out the kernel records ODIN_ERR_TIMEOUT, carries on with clamped addresses and
returns, so the context stays usable.  `odin_set_wait_limit(ctx, 0)` makes a wait give up the first time it finds its
predecessor unpublished, which with hundreds of concurrently running tiles happens at once: nothing hangs, nothing is
written out of bounds, the status says so, and the next call with the default limit is exact again.
"""
import io

import numpy as np
import pytest
import torch

from paper_2607_19893_b200 import binding as B
from paper_2607_19893_b200 import workloads as wl

import gpu_util as G

pytestmark = pytest.mark.gpu
SENTINEL = -7


def touched_call(ctx, ws, d_tt, n, cap):
    dev = d_tt.device
    words = (n + 31) // 32
    # guard words around every output: a write outside [0, size) of a buffer would land in them
    mask = torch.full((words + 64,), SENTINEL, dtype=torch.int32, device=dev)
    idx = torch.full((cap + 64,), SENTINEL, dtype=torch.int32, device=dev)
    count = torch.full((33,), SENTINEL, dtype=torch.int32, device=dev)
    B.odin_touched_set(ctx, d_tt, n, mask[32:32 + words], idx[32:32 + cap], cap, count[16:17], ws)
    return mask, idx, count


def test_a_wait_that_runs_out_reports_timeout_and_stays_in_bounds():
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    n = 1 << 24  # 8192 look-back tiles in 1024 blocks: several waves, every block waits for its predecessor
    rng = np.random.default_rng(5)
    tt = ((rng.random(n) < 0.3) * rng.integers(1, 50, n)).astype(np.uint32)
    d_tt = torch.from_numpy(tt.view(np.int32)).to(dev)
    ws = torch.zeros(B.odin_workspace_bytes(ctx, n, 0), dtype=torch.uint8, device=dev)
    want_idx = np.flatnonzero(tt).astype(np.uint32)
    cap = len(want_idx) + 5
    words = (n + 31) // 32
    B.odin_set_wait_limit(ctx, 0)
    seen = False
    for _ in range(5):  # one attempt is enough in practice; the loop only guards against a perfectly ordered launch
        mask, idx, count = touched_call(ctx, ws, d_tt, n, cap)
        status = B.odin_poll(ctx)  # returns: the kernel did not hang
        assert status in (B.ODIN_OK, B.ODIN_ERR_TIMEOUT)
        # nothing outside the buffers was written, whatever the status
        assert (mask[:32] == SENTINEL).all() and (mask[32 + words:] == SENTINEL).all()
        assert (idx[:32] == SENTINEL).all() and (idx[32 + cap:] == SENTINEL).all()
        assert (count[:16] == SENTINEL).all() and (count[17:] == SENTINEL).all()
        got_count = int(count[16].item())
        assert 0 <= got_count <= cap
        body = idx[32:32 + cap].cpu().numpy()
        written = body != SENTINEL
        assert np.all(body[written].view(np.uint32) < n)  # every index that was written names a primitive
        # the bitmask does not depend on the look-back: it is exact even when the list is not
        assert np.array_equal(np.unpackbits(G.u32(mask[32:32 + words]).view(np.uint8), bitorder="little")[:n],
                              (tt > 0).astype(np.uint8))
        if status == B.ODIN_ERR_TIMEOUT:
            seen = True
            break
    assert seen, "no wait ran out in five launches of 8192 tiles with a poll limit of 0"
    assert B.odin_poll(ctx) == B.ODIN_OK  # the status was cleared by the poll that returned it
    # the context is still usable: with the default limit the same call is exact
    B.odin_set_wait_limit(ctx, 1 << 22)
    mask, idx, count = touched_call(ctx, ws, d_tt, n, cap)
    assert B.odin_poll(ctx) == B.ODIN_OK
    assert int(count[16].item()) == len(want_idx)
    assert np.array_equal(G.u32(idx[32:32 + len(want_idx)]), want_idx)
    with pytest.raises(B.OdinError):
        B.odin_set_wait_limit(ctx, -1)
    B.odin_destroy(ctx)


def test_a_whole_view_with_a_zero_wait_limit_returns_and_recovers(oracle32):
    """Every look-back of a view step (projection scan, touched set, row sort, offsets, instance sort) with the poll
    limit at 0: the step returns, the deferred status is TIMEOUT (or OK), and the same trainer renders the view
    exactly once the limit is restored."""
    w = wl.make_workload(3, n=400_000, n_cameras=2, resolution=(800, 533))
    cam = w.cameras[0]
    tr = G.trainer_for(w.scene, cam)
    tr.target.copy_(torch.from_numpy(w.target(0)).to(tr.device))
    B.odin_set_wait_limit(tr.ctx, 0)
    tr.view_step(B.make_camera(cam), 1, w.lr, w.beta1, w.beta2, w.eps, update=False)
    assert tr.poll() in (B.ODIN_OK, B.ODIN_ERR_TIMEOUT)
    B.odin_set_wait_limit(tr.ctx, 1 << 22)
    tr.view_step(B.make_camera(cam), 1, w.lr, w.beta1, w.beta2, w.eps, update=False)
    G.poll_ok(tr)
    f = oracle32.view_forward(w.scene, cam)
    robust = f["pix_margin"] > 2e-5
    assert np.abs(tr.out.cpu().numpy() - f["out"])[:, robust].max() < 1e-4
    assert int(tr.count.item()) == len(f["idx"])
    tr.close()


def test_checkpoint_resume_equals_the_uninterrupted_run():
    """All training state is the caller's tensors (parameters, both Adam moments, the step counter), so a checkpoint
    is torch.save of them.  Ten views in one go against five views, save, a NEW trainer built from the file, five
    more: the touched sets and losses of every view agree, and so do the final parameters up to the order of the
    float atomics of the backward pass (the bar of the host-loop test)."""
    w = wl.make_workload(2, n=30_000)
    cams = [B.make_camera(c) for c in w.cameras]

    def run(tr, steps, log):
        for s in steps:
            tr.target.copy_(torch.from_numpy(w.target(s % 8)).to(tr.device))
            tr.view_step(cams[s % 8], s + 1, w.lr, w.beta1, w.beta2, w.eps)
            G.poll_ok(tr)
            log.append((s, float(tr.loss.item()), int(tr.count.item())))

    a = G.trainer_for(w.scene, w.cameras[0])
    log_a = []
    run(a, range(10), log_a)
    b = G.trainer_for(w.scene, w.cameras[0])
    log_b = []
    run(b, range(5), log_b)
    blob = io.BytesIO()
    torch.save({"step": 5, "params": [t.cpu() for t in b.params.tensors()], "m": [t.cpu() for t in b.m.tensors()],
                "v": [t.cpu() for t in b.v.tensors()]}, blob)
    b.close()
    blob.seek(0)
    ck = torch.load(blob)
    scene = wl.Scene(w.scene.sh_degree, *(t.numpy() for t in ck["params"]))
    c = G.trainer_for(scene, w.cameras[0])
    for dst, src in ((c.m, ck["m"]), (c.v, ck["v"])):
        for t, saved in zip(dst.tensors(), src):
            t.copy_(saved.to(c.device))
    c.moments_changed()  # the optimizer's per-primitive flags are derived from the restored moments
    run(c, range(ck["step"], 10), log_b)
    assert [x[0] for x in log_a] == [x[0] for x in log_b] == list(range(10))
    for x, y in zip(log_a, log_b):
        assert x[2] == y[2] and abs(x[1] - y[1]) < 1e-6
    for group in ("params", "m", "v"):
        G.assert_states_close(getattr(a, group).tensors(), getattr(c, group).tensors(), w.lr, 10)
    a.close(); c.close()
