"""Helpers shared by the GPU parity tests: build a trainer, feed oracle stage outputs to the device, read back."""
import numpy as np
import torch

from paper_2607_19893_b200 import binding as B
from paper_2607_19893_b200.engine import ViewTrainer


def trainer_for(scene, cam, row_capacity=None, instance_capacity=None, mask_slots=1, cfg=None, extra_render_records=0):
    n = scene.means.shape[0]
    return ViewTrainer(scene, cam.width, cam.height, row_capacity if row_capacity is not None else n,
                       instance_capacity if instance_capacity is not None else max(64 * n, 1 << 16), mask_slots, cfg=cfg,
                       extra_render_records=extra_render_records)


def compact_from_oracle(proj, idx):
    """Oracle's dense projection -> the compact arrays of odin_projected (row r <-> primitive idx[r])."""
    idx = idx.astype(np.int64)
    tt = proj.tiles_touched[idx].astype(np.uint64)
    off = np.concatenate([[0], np.cumsum(tt)[:-1]]).astype(np.uint32) if len(idx) else np.zeros(0, np.uint32)
    return dict(
        prim_id=idx.astype(np.uint32), xy=proj.xy[idx].astype(np.float32), depth=proj.depth[idx].astype(np.float32),
        conic_opacity=proj.conic_o[idx].astype(np.float32), rgb=proj.rgb[idx].astype(np.float32),
        radius=proj.radius[idx].astype(np.int32), rect=proj.rect[idx].astype(np.uint16), tile_offset=off,
        clamp_flags=proj.clamp_flags[idx].astype(np.uint8),
    )


def load_oracle_projection(tr, proj, idx):
    rows = compact_from_oracle(proj, idx)
    tr.proj.load_rows(**rows)
    tr.proj.tiles_touched[: len(proj.tiles_touched)].copy_(
        torch.from_numpy(proj.tiles_touched.view(np.int32)).to(tr.device))
    tr.proj.num_rows.fill_(len(idx))
    tr.proj.num_instances.fill_(int(proj.tiles_touched.astype(np.int64).sum()))
    return rows


def u32(t):
    return t.cpu().numpy().view(np.uint32)


def u64(t):
    return t.cpu().numpy().view(np.uint64)


def rows_of(inv_idx, vals):
    """Map oracle values (primitive ids) to compact row ids."""
    return inv_idx[vals.astype(np.int64)]


def poll_ok(tr):
    st = tr.poll()
    assert st == B.ODIN_OK, B.status_string(st)


# ---------------------------------------------------------------------------------------------------------------
# Gradient parity bar.  A gradient word is a sum over pixels of signed terms.  fp32 evaluation on the device
# (ex2.approx, transmittance recovered by division, atomic accumulation order) perturbs every TERM by a relative
# ~1e-6, so the error of the SUM scales with sum|term| (reported by the oracle), not with the possibly cancelled
# sum.  Bar for the nine compositing words:  |dev - oracle| <= 1e-3 |oracle| + 1e-5 sum|term|.
# The per-primitive chain rule is linear in those nine words, so the same absolute slack is pushed through the
# oracle's own Jacobian (nine evaluations on unit inputs) for the final gradient rows.
GRAD_RTOL = 1e-3
GRAD_FLOOR = 1e-5


def grad2d_bound(want2d, abs2d):
    return GRAD_RTOL * np.abs(want2d) + GRAD_FLOOR * abs2d + 1e-30


# The chain rule of a row runs in fp32 on both sides: every intermediate is rounded to 2^-24 relative, so a word that
# is a cancelled combination of intermediates carries an absolute error of a few ulp of the LARGEST quantities of the
# row, whatever its own size.  Eight ulp of the row's largest word are granted to every word of the row.
ROW_ULP_FLOOR = 8 * 2.0 ** -24


def rows_bound(oracle, scene, cam, idx, clamp_flags, rows_o, want2d_dense, abs2d_dense):
    n = want2d_dense.shape[0]
    # second term: rounding inside the fp32 chain rule itself (its own sums cancel too)
    slack2d = GRAD_FLOOR * abs2d_dense + GRAD_FLOOR * np.abs(want2d_dense)
    bound = GRAD_RTOL * np.abs(rows_o) + ROW_ULP_FLOOR * np.abs(rows_o).max(axis=1, keepdims=True) + 1e-30
    for c in range(9):
        unit = np.zeros((n, 9))
        unit[:, c] = 1.0
        jac_c = oracle.render_bwd_project(scene, cam, idx, unit, clamp_flags).astype(np.float64)
        bound = bound + np.abs(jac_c) * slack2d[idx.astype(np.int64), c][:, None]
    return bound


def assert_states_close(tensors_a, tensors_b, lr, steps, rtol=1e-4, atol=1e-6, max_fraction=1e-4):
    """Two runs of the same steps whose only difference is the order of the backward pass's atomic sums.  The optimizer
    normalises its step by the gradient's own magnitude, so an element whose gradient is a cancelled sum of the size of
    that rounding noise may move by learning rates in one run and not in the other.  Everything else must agree: at most
    `max_fraction` of the elements may lie outside rtol / atol, and none by more than the optimizer can move it in
    `steps` steps."""
    bad = total = 0
    worst = 0.0
    for ta, tb in zip(tensors_a, tensors_b):
        d = (ta - tb).abs()
        out = d > atol + rtol * tb.abs()
        bad += int(out.sum().item())
        total += d.numel()
        if bool(out.any()):
            worst = max(worst, float(d[out].max().item()))
    assert bad <= max_fraction * total, (bad, total)
    assert worst <= 10.0 * float(max(lr)) * steps, worst


# ---------------------------------------------------------------------------------------------------------------
# Measured distances to the bars are printed (pytest -rP or -s shows them) so that every slack factor in the chained
# tests can be read against what the device actually does.
def report(tag, **kv):
    print("PARITY " + tag + " " + " ".join(f"{k}={v:.4g}" if isinstance(v, float) else f"{k}={v}" for k, v in kv.items()),
          flush=True)


def blended_at_pixels(o, pixels_yx, upto, tx, alpha_min=1.0 / 255.0):
    """Primitive ids that blend (alpha within 1 % of the skip threshold or above) at the given pixels, looking at the
    first upto[k] entries of the pixel's tile list.  pixels_yx: [K,2] (row, column).  These are the primitives whose
    gradient changes when a decision of that pixel falls the other way."""
    out = []
    xy, co = o["proj"].xy.astype(np.float64), o["proj"].conic_o.astype(np.float64)
    for (y, x), n in zip(pixels_yx, upto):
        t = (y // 16) * tx + (x // 16)
        s, e = int(o["ranges"][t, 0]), int(o["ranges"][t, 1])
        prims = o["vals"][s:min(e, s + int(n))].astype(np.int64)
        dx, dy = xy[prims, 0] - (x + 0.5), xy[prims, 1] - (y + 0.5)
        power = -0.5 * (co[prims, 0] * dx * dx + co[prims, 2] * dy * dy) - co[prims, 1] * dx * dy
        alpha = co[prims, 3] * np.exp(np.minimum(power, 0.0))
        out.append(prims[(power <= 1e-6) & (alpha >= 0.99 * alpha_min)])
    return np.unique(np.concatenate(out)) if out else np.zeros(0, np.int64)
