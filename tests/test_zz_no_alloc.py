"""The allocation-free touched-set entry point (needs a GPU).

Some users of the library get their GPU memory handed out once and may not allocate afterwards (a component inside a
host application's memory pool, a real-time loop where an allocation may stall or fail).  They cannot create a
context or a workspace, so `odin_touched_set_static` keeps its scratch in a fixed array inside the library.  This
test calls it through the C ABI twice in a row and checks both results against `odin_touched_set`, bit for bit
(mask, index list and count are integer outputs).  It is collected last on purpose and must pass on its own as well.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2607_19893_b200 import binding as B

pytestmark = pytest.mark.gpu


def run_both(ctx, ws, tt, idx_capacity=None):
    """Runs the workspace entry point and the allocation-free one on the same input; returns both results."""
    dev = torch.device("cuda", 0)
    n = len(tt)
    cap = n if idx_capacity is None else idx_capacity
    d_tt = torch.from_numpy(tt.view(np.int32)).to(dev)
    words = (n + 31) // 32
    outs = []
    for static in (False, True):
        d_mask = torch.full((max(words, 1),), -1, dtype=torch.int32, device=dev)
        d_idx = torch.full((max(cap, 1),), -1, dtype=torch.int32, device=dev)
        d_count = torch.full((1,), -1, dtype=torch.int32, device=dev)
        d_status = torch.zeros(1, dtype=torch.int32, device=dev)
        if static:
            B.odin_touched_set_static(d_tt, n, d_mask, d_idx, cap, d_count, d_status)
            torch.cuda.synchronize()
            status = int(d_status.item())
        else:
            B.odin_touched_set(ctx, d_tt, n, d_mask, d_idx, cap, d_count, ws)
            status = B.odin_poll(ctx)
        outs.append((d_mask.cpu().numpy(), d_idx.cpu().numpy(), int(d_count.item()), status))
    return outs


def test_static_touched_set_matches_workspace_version_twice():
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    n_max = 2_500_003
    ws = torch.zeros(B.odin_workspace_bytes(ctx, n_max, 0), dtype=torch.uint8, device=dev)
    rng = np.random.default_rng(77)
    # two calls in a row with different sizes and densities: the second must not see anything left by the first
    for n, density in ((n_max, 0.31), (700_001, 0.04)):
        tt = ((rng.random(n) < density) * rng.integers(1, 400, n)).astype(np.uint32)
        (mask_a, idx_a, cnt_a, st_a), (mask_b, idx_b, cnt_b, st_b) = run_both(ctx, ws, tt)
        assert st_a == B.ODIN_OK and st_b == B.ODIN_OK
        assert cnt_a == cnt_b == int(np.count_nonzero(tt))
        assert np.array_equal(mask_a, mask_b)
        assert np.array_equal(idx_a, idx_b)
        assert np.array_equal(idx_b[:cnt_b].view(np.uint32), np.nonzero(tt)[0].astype(np.uint32))
    # a list capacity that is too small: same truncation and the same deferred status on both paths
    tt = np.ones(5000, np.uint32)
    (mask_a, idx_a, cnt_a, st_a), (mask_b, idx_b, cnt_b, st_b) = run_both(ctx, ws, tt, idx_capacity=1234)
    assert st_a == st_b == B.ODIN_ERR_CAPACITY and cnt_a == cnt_b == 1234
    assert np.array_equal(idx_a, idx_b) and np.array_equal(mask_a, mask_b)
    B.odin_destroy(ctx)


def test_static_touched_set_leaves_free_device_memory_unchanged():
    """The point of the entry point: after the warm-up call (which may make the runtime load the library's device code)
    a call allocates nothing, so the free device memory reported by the runtime is the same before and after it."""
    dev = torch.device("cuda", 0)
    n = 3_000_017
    rng = np.random.default_rng(78)
    tt = ((rng.random(n) < 0.2) * 3).astype(np.uint32)
    d_tt = torch.from_numpy(tt.view(np.int32)).to(dev)
    d_mask = torch.zeros((n + 31) // 32, dtype=torch.int32, device=dev)
    d_idx = torch.zeros(n, dtype=torch.int32, device=dev)
    d_count = torch.zeros(1, dtype=torch.int32, device=dev)
    B.odin_touched_set_static(d_tt, n, d_mask, d_idx, n, d_count, None)  # warm-up: first call on the device
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info(dev)
    for _ in range(3):
        B.odin_touched_set_static(d_tt, n, d_mask, d_idx, n, d_count, None)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info(dev)
    assert free_after == free_before
    assert int(d_count.item()) == int(np.count_nonzero(tt))


def test_static_touched_set_at_its_size_limit_and_without_a_status_word():
    dev = torch.device("cuda", 0)
    ctx = B.odin_create(0)
    n = 1 << 25  # the largest size: the whole fixed array is in use
    ws = torch.zeros(B.odin_workspace_bytes(ctx, n, 0), dtype=torch.uint8, device=dev)
    rng = np.random.default_rng(79)
    tt = (rng.random(n) < 0.03).astype(np.uint32)
    tt[-1] = 9  # the very last primitive
    (mask_a, idx_a, cnt_a, st_a), (mask_b, idx_b, cnt_b, st_b) = run_both(ctx, ws, tt, idx_capacity=1_200_000)
    assert st_a == st_b == B.ODIN_OK and cnt_a == cnt_b == int(np.count_nonzero(tt))
    assert np.array_equal(mask_a, mask_b) and np.array_equal(idx_a, idx_b)
    assert idx_b[cnt_b - 1] == n - 1
    B.odin_destroy(ctx)
    # no status word (NULL): an overflowing list is still cut at the capacity, the condition goes to the internal sink
    tt = np.ones(70_000, np.uint32)
    d_tt = torch.from_numpy(tt.view(np.int32)).to(dev)
    d_mask = torch.zeros((len(tt) + 31) // 32, dtype=torch.int32, device=dev)
    d_idx = torch.full((1000 + 64,), -1, dtype=torch.int32, device=dev)
    d_count = torch.zeros(1, dtype=torch.int32, device=dev)
    B.odin_touched_set_static(d_tt, len(tt), d_mask, d_idx[:1000], 1000, d_count, None)
    torch.cuda.synchronize()
    assert int(d_count.item()) == 1000
    assert np.array_equal(d_idx[:1000].cpu().numpy(), np.arange(1000)) and (d_idx[1000:] == -1).all()
    assert (d_mask.cpu().numpy().view(np.uint32)[: 70_000 // 32] == 0xFFFFFFFF).all()


def test_static_touched_set_limits_and_empty_input():
    dev = torch.device("cuda", 0)
    d_count = torch.full((1,), 9, dtype=torch.int32, device=dev)
    # larger than the fixed scratch: refused on the host, nothing launched, outputs untouched
    lib = B.lib()
    one = torch.zeros(4, dtype=torch.int32, device=dev)
    rc = lib.odin_touched_set_static(one.data_ptr(), (1 << 25) + 1, one.data_ptr(), one.data_ptr(), 4, d_count.data_ptr(),
                                     None, None)
    assert rc == B.ODIN_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert int(d_count.item()) == 9
    with pytest.raises(B.OdinError):
        B.odin_touched_set_static(one, (1 << 25) + 1, one, one, 4, d_count)
    # n = 0 is legal: the count becomes 0
    B.odin_touched_set_static(None, 0, None, None, 0, d_count)
    torch.cuda.synchronize()
    assert int(d_count.item()) == 0
    assert lib.odin_touched_set_static(None, 0, None, None, 0, None, None, None) == B.ODIN_ERR_NULL
    assert isinstance(C.c_void_p(one.data_ptr()).value, int)
