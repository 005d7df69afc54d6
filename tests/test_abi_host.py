"""Host-side checks of the C ABI that need no GPU: the library loads, exports every declared symbol, and rejects bad
arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2607_19893_b200 import binding as B
from paper_2607_19893_b200 import build as odin_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    odin_build.build()
    return B.lib()


def declared_functions():
    with open(os.path.join(ROOT, "include", "odin.h")) as fh:
        text = fh.read()
    names = re.findall(r"^(?:int|const char\*)\s+(odin_\w+)\s*\(", text, flags=re.M)
    assert len(names) >= 13
    return names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), name
    assert set(declared_functions()) == set(B.EXPORTS)


def test_status_strings(lib):
    seen = set()
    for code in range(0, -8, -1):
        s = B.status_string(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 8
    assert B.status_string(-99) == "unknown status"


def test_null_context_is_rejected_without_a_device(lib):
    null = C.c_void_p(None)
    assert lib.odin_destroy(null) == B.ODIN_ERR_NULL
    assert lib.odin_poll(null, None) == B.ODIN_ERR_NULL
    assert lib.odin_set_wait_limit(null, 0) == B.ODIN_ERR_NULL
    sz = C.c_size_t(0)
    assert lib.odin_workspace_bytes(null, 10, 10, C.byref(sz)) == B.ODIN_ERR_NULL
    assert lib.odin_project(null, None, None, None, None, 0, None) == B.ODIN_ERR_NULL
    assert lib.odin_touched_set(null, None, 0, None, None, 0, None, None, 0, None) == B.ODIN_ERR_NULL
    assert lib.odin_bin_sort(null, None, 16, 16, None, None, 0, None, None, 0, None) == B.ODIN_ERR_NULL
    assert lib.odin_render_workspace_bytes(null, 64, 64, C.byref(sz)) == B.ODIN_ERR_NULL
    assert lib.odin_render_fwd(null, None, None, None, None, None, None, None, None, 0, None) == B.ODIN_ERR_NULL
    assert lib.odin_l1_loss(null, None, None, 1, 1, None, None, None) == B.ODIN_ERR_NULL
    assert lib.odin_chain_begin(null) == B.ODIN_ERR_NULL and lib.odin_chain_end(null) == B.ODIN_ERR_NULL
    assert lib.odin_render_bwd(null, None, None, None, None, None, None, None, None, None, None, None, None, None, 0,
                               None) == B.ODIN_ERR_NULL
    assert lib.odin_active_set(null, None, None, None, None, 0, 0, None, None, 0, None, None, None, None, 0,
                               None) == B.ODIN_ERR_NULL
    assert lib.odin_mask_union(null, None, 0, 0, 0, None, 0, None, None) == B.ODIN_ERR_NULL
    assert lib.odin_hazard_count(null, None, None, 0, 0, 0, None, 0, None, None) == B.ODIN_ERR_NULL
    assert lib.odin_delayed_read_gate(null, None, None, None, 0, None, None, None, None, 0, 0.2, None,
                                      None) == B.ODIN_ERR_NULL
    assert lib.odin_rlg_weights(null, None, None, None, 0, 0, None, None) == B.ODIN_ERR_NULL
    assert lib.odin_rlg_topk(null, None, 0, 0, None, None, 0, None) == B.ODIN_ERR_NULL
    assert lib.odin_sds_scores(null, None, 0, None, 0, None, 0, None, None) == B.ODIN_ERR_NULL
    assert lib.odin_sparse_adam(null, None, None, None, None, None, None, None, None, 0.9, 0.999, 1e-8, 1,
                                None) == B.ODIN_ERR_NULL
    assert lib.odin_sparse_adam_live(null, None, None, None, None, None, None, None, None, None, 0.9, 0.999, 1e-8, 1,
                                     None) == B.ODIN_ERR_NULL
    assert lib.odin_adam_live_refresh(null, None, None, None, None) == B.ODIN_ERR_NULL
    assert lib.odin_conflict_count(null, None, 0, 0, 0, None, 0, None, None) == B.ODIN_ERR_NULL


def test_create_rejects_bad_configuration(lib):
    ctx = C.c_void_p()
    assert lib.odin_create(None, 0, None) == B.ODIN_ERR_NULL
    cfg = B.odin_config(1 / 255, 0.99, 1e-4, 0.3, 3.0, 1.3, 8)  # only 16-pixel tiles exist
    assert lib.odin_create(C.byref(ctx), 0, C.byref(cfg)) == B.ODIN_ERR_UNSUPPORTED
    cfg = B.odin_config(0.5, 0.4, 1e-4, 0.3, 3.0, 1.3, 16)  # alpha_max below alpha_min
    assert lib.odin_create(C.byref(ctx), 0, C.byref(cfg)) == B.ODIN_ERR_INVALID_ARG
    assert not ctx.value


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", str(tmp_path / "libodin.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        B.lib()
