"""NumPy/ctypes front end of the CPU oracle (test infrastructure; see odin_oracle.hpp)."""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB = os.path.join(_HERE, "liboracle.so")
_SRC = [os.path.join(_HERE, "oracle_capi.cpp"), os.path.join(_HERE, "odin_oracle.hpp")]

# alpha_min, alpha_max, t_min, dilation, radius_sigmas, jac_clamp, tile, binning (0 plain rectangle, 1 tight extent,
# 2 exact: only the tiles the region alpha >= alpha_min reaches)
DEFAULT_CFG = np.array([1.0 / 255.0, 0.99, 1e-4, 0.3, 3.0, 1.3, 16.0, 0.0], dtype=np.float64)


def build(force: bool = False) -> str:
    """Compile liboracle.so with g++ if it is missing or older than its sources."""
    if not force and os.path.exists(_LIB) and all(os.path.getmtime(_LIB) >= os.path.getmtime(s) for s in _SRC):
        return _LIB
    cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-o", _LIB, _SRC[0]]
    subprocess.run(cmd, check=True, cwd=_HERE)
    return _LIB


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def ids_to_mask(idx, n: int) -> np.ndarray:
    """Bitmask over primitive ids: bit (p & 31) of word (p >> 5)."""
    mask = np.zeros((n + 31) // 32, np.uint32)
    i = np.asarray(idx, np.int64)
    np.bitwise_or.at(mask, i >> 5, np.left_shift(np.uint32(1), (i & 31).astype(np.uint32)))
    return mask


def _cam(cam) -> np.ndarray:
    a = cam.as_f64() if hasattr(cam, "as_f64") else np.asarray(cam, dtype=np.float64)
    assert a.shape == (23,)
    return np.ascontiguousarray(a)


@dataclasses.dataclass
class Projected:
    """Dense (length N) projection outputs."""

    xy: np.ndarray  # [N,2]
    depth: np.ndarray  # [N]
    conic_o: np.ndarray  # [N,4] conic A,B,C and opacity
    rgb: np.ndarray  # [N,3]
    radius: np.ndarray  # [N] int32
    rect: np.ndarray  # [N,4] int32 x0,y0,x1,y1 (tile units, half open)
    tiles_touched: np.ndarray  # [N] uint32
    clamp_flags: np.ndarray  # [N] uint8, bit ch set when colour channel ch was clamped at 0
    margin: np.ndarray  # [N] relative distance to the nearest decision threshold
    span_ptr: Optional[np.ndarray] = None  # binning 2: [N+1] prefix of the rectangles' heights (tile rows)
    span_x: Optional[np.ndarray] = None  # binning 2: [span_ptr[N], 2] first / one-past-last kept tile of each tile row


class Oracle:
    def __init__(self, dtype=np.float32, cfg: Optional[np.ndarray] = None, tile: int = 16):
        self.dtype = np.dtype(dtype)
        assert self.dtype in (np.dtype(np.float32), np.dtype(np.float64))
        self.suf = "f32" if self.dtype == np.float32 else "f64"
        self.cfg = np.ascontiguousarray(DEFAULT_CFG.copy() if cfg is None else np.asarray(cfg, dtype=np.float64))
        self.cfg[6] = tile
        self.tile = tile
        self.lib = C.CDLL(build())
        self.lib.oracle_l1_loss_f32.restype = C.c_double
        self.lib.oracle_l1_loss_f64.restype = C.c_double
        self.lib.oracle_touched_set.restype = C.c_uint32
        self.lib.oracle_count_instances.restype = C.c_uint64
        self.lib.oracle_conflict_count.restype = C.c_uint64
        self.lib.oracle_num_threads.restype = C.c_int

    # ------------------------------------------------------------------ helpers
    def _f(self, name):
        return getattr(self.lib, f"{name}_{self.suf}")

    def _a(self, x):
        return np.ascontiguousarray(x, dtype=self.dtype)

    def num_threads(self) -> int:
        return int(self.lib.oracle_num_threads())

    def set_num_threads(self, t: int) -> None:
        self.lib.oracle_set_num_threads(C.c_int(t))

    def grid(self, cam):
        c = _cam(cam)
        w, h = int(c[0]), int(c[1])
        return (w + self.tile - 1) // self.tile, (h + self.tile - 1) // self.tile

    # ------------------------------------------------------------------ stages
    def project(self, scene, cam) -> Projected:
        n = scene.means.shape[0]
        dt = self.dtype
        out = Projected(
            np.zeros((n, 2), dt), np.zeros(n, dt), np.zeros((n, 4), dt), np.zeros((n, 3), dt),
            np.zeros(n, np.int32), np.zeros((n, 4), np.int32), np.zeros(n, np.uint32), np.zeros(n, np.uint8),
            np.zeros(n, dt),
        )
        means, ls, q, lo, sh = (self._a(scene.means), self._a(scene.log_scales), self._a(scene.quats),
                                self._a(scene.opacity_logit), self._a(scene.sh))
        c = _cam(cam)
        self._f("oracle_project")(
            C.c_int64(n), C.c_int(scene.sh_degree), _p(means), _p(ls), _p(q), _p(lo), _p(sh), _p(c), _p(self.cfg),
            _p(out.xy), _p(out.depth), _p(out.conic_o), _p(out.rgb), _p(out.radius), _p(out.rect),
            _p(out.tiles_touched), _p(out.clamp_flags), _p(out.margin),
        )
        if int(self.cfg[7]) == 2:
            # exact binning: of every rectangle only the tiles the region alpha >= alpha_min reaches; a primitive that
            # keeps no tile is not visible
            h = np.where(out.tiles_touched > 0, out.rect[:, 3] - out.rect[:, 1], 0).astype(np.int64)
            out.span_ptr = np.concatenate([[0], np.cumsum(h)]).astype(np.int64)
            out.span_x = np.zeros((int(out.span_ptr[-1]), 2), np.int32)
            self._f("oracle_tile_spans")(C.c_int64(n), _p(out.xy), _p(out.conic_o), _p(out.rect), _p(self.cfg),
                                         _p(out.span_ptr), _p(out.span_x), _p(out.tiles_touched), _p(out.margin))
            gone = out.tiles_touched == 0
            for a in (out.xy, out.depth, out.conic_o, out.rgb, out.radius, out.rect, out.clamp_flags):
                a[gone] = 0
        return out

    def tile_reached(self, u, v, conic_o, tx: int, ty: int) -> bool:
        """The exact-binning rule for one (primitive, tile) pair: can a pixel of the tile pass the skip test?"""
        ct = C.c_float if self.dtype == np.float32 else C.c_double
        a, b, c, o = (float(x) for x in conic_o)
        return bool(self._f("oracle_tile_reached")(ct(u), ct(v), ct(a), ct(b), ct(c), ct(o), _p(self.cfg), C.c_int(tx),
                                                   C.c_int(ty)))

    def touched_set(self, tiles_touched: np.ndarray):
        tt = np.ascontiguousarray(tiles_touched, dtype=np.uint32)
        n = tt.shape[0]
        mask = np.zeros((n + 31) // 32, np.uint32)
        idx = np.zeros(n, np.uint32)
        v = self.lib.oracle_touched_set(C.c_int64(n), _p(tt), _p(mask), _p(idx))
        return mask, idx[:v].copy()

    def bin_sort(self, proj: Projected, cam):
        tx, ty = self.grid(cam)
        n = proj.depth.shape[0]
        tt = np.ascontiguousarray(proj.tiles_touched, dtype=np.uint32)
        m = int(self.lib.oracle_count_instances(C.c_int64(n), _p(tt)))
        keys = np.zeros(m, np.uint64)
        vals = np.zeros(m, np.uint32)
        ranges = np.zeros((tx * ty, 2), np.uint32)
        d32 = np.ascontiguousarray(proj.depth, dtype=np.float32)
        rect = np.ascontiguousarray(proj.rect, dtype=np.int32)
        if proj.span_ptr is not None:
            self.lib.oracle_bin_sort_spans(C.c_int64(n), _p(d32), _p(rect), _p(tt), _p(proj.span_ptr),
                                           _p(np.ascontiguousarray(proj.span_x, np.int32)), C.c_int(tx), C.c_int(ty),
                                           _p(keys), _p(vals), _p(ranges))
            return keys, vals, ranges
        self.lib.oracle_bin_sort(C.c_int64(n), _p(d32), _p(rect), _p(tt), C.c_int(tx), C.c_int(ty), _p(keys), _p(vals),
                                 _p(ranges))
        return keys, vals, ranges

    def render_fwd(self, proj: Projected, vals, ranges, cam, want_margin: bool = True):
        c = _cam(cam)
        w, h = int(c[0]), int(c[1])
        dt = self.dtype
        out = np.zeros((3, h, w), dt)
        final_t = np.zeros((h, w), dt)
        ncon = np.zeros((h, w), np.uint32)
        margin = np.ones((h, w), dt) if want_margin else None
        counters = np.zeros(3, np.uint64)
        self._f("oracle_render_fwd")(
            _p(self._a(proj.xy)), _p(self._a(proj.conic_o)), _p(self._a(proj.rgb)),
            _p(np.ascontiguousarray(vals, np.uint32)), _p(np.ascontiguousarray(ranges, np.uint32)), _p(c), _p(self.cfg),
            _p(out), _p(final_t), _p(ncon), _p(margin), _p(counters),
        )
        return out, final_t, ncon, margin, counters

    def l1_loss(self, out: np.ndarray, target: np.ndarray):
        o, t = self._a(out), self._a(target)
        g = np.zeros_like(o)
        loss = self._f("oracle_l1_loss")(C.c_int64(o.size), _p(o), _p(t), _p(g))
        return float(loss), g

    def render_bwd_blend(self, proj: Projected, vals, ranges, cam, final_t, n_contrib, dl_dout, want_abs: bool = False):
        """Dense [N,9] gradient sums; with want_abs also the sums of the absolute per-pixel terms."""
        n = proj.depth.shape[0]
        g2d = np.zeros((n, 9), np.float64)
        g2d_abs = np.zeros((n, 9), np.float64) if want_abs else None
        self._f("oracle_render_bwd_blend")(
            _p(self._a(proj.xy)), _p(self._a(proj.conic_o)), _p(self._a(proj.rgb)),
            _p(np.ascontiguousarray(vals, np.uint32)), _p(np.ascontiguousarray(ranges, np.uint32)), _p(_cam(cam)),
            _p(self.cfg), _p(self._a(final_t)), _p(np.ascontiguousarray(n_contrib, np.uint32)), _p(self._a(dl_dout)),
            C.c_int64(n), _p(g2d), _p(g2d_abs),
        )
        return (g2d, g2d_abs) if want_abs else g2d

    def render_bwd_project(self, scene, cam, idx, g2d, clamp_flags) -> np.ndarray:
        idx = np.ascontiguousarray(idx, np.uint32)
        k = (scene.sh_degree + 1) ** 2
        rows = np.zeros((idx.shape[0], 11 + 3 * k), self.dtype)
        self._f("oracle_render_bwd_project")(
            C.c_int(scene.sh_degree), _p(self._a(scene.means)), _p(self._a(scene.log_scales)), _p(self._a(scene.quats)),
            _p(self._a(scene.opacity_logit)), _p(self._a(scene.sh)), _p(_cam(cam)), _p(self.cfg), _p(idx),
            C.c_uint32(idx.shape[0]), _p(np.ascontiguousarray(g2d, np.float64)),
            _p(np.ascontiguousarray(clamp_flags, np.uint8)), _p(rows),
        )
        return rows

    def sparse_adam(self, params, m, v, rows, idx, lr, beta1, beta2, eps, step) -> None:
        """In-place update of params / m / v (objects with means, log_scales, quats, opacity_logit, sh arrays
        of this oracle's dtype, C-contiguous)."""
        for s in (params, m, v):
            for a in (s.means, s.log_scales, s.quats, s.opacity_logit, s.sh):
                assert a.dtype == self.dtype and a.flags.c_contiguous
        idx = np.ascontiguousarray(idx, np.uint32)
        rows = self._a(rows)
        lr = self._a(lr)
        self._f("oracle_sparse_adam")(
            C.c_int(params.sh_degree),
            _p(params.means), _p(params.log_scales), _p(params.quats), _p(params.opacity_logit), _p(params.sh),
            _p(m.means), _p(m.log_scales), _p(m.quats), _p(m.opacity_logit), _p(m.sh),
            _p(v.means), _p(v.log_scales), _p(v.quats), _p(v.opacity_logit), _p(v.sh),
            _p(rows), _p(idx), C.c_uint32(idx.shape[0]), _p(lr), C.c_double(beta1), C.c_double(beta2), C.c_double(eps),
            C.c_uint32(step),
        )

    def conflict_count(self, idx_a, idx_b) -> int:
        a = np.ascontiguousarray(idx_a, np.uint32)
        b = np.ascontiguousarray(idx_b, np.uint32)
        return int(self.lib.oracle_conflict_count(_p(a), C.c_uint32(a.shape[0]), _p(b), C.c_uint32(b.shape[0])))

    # ------------------------------------------------------------------ realized scopes, evidence, hazards
    def realized_active(self, proj: Projected, vals, ranges, cam, n_contrib):
        """Realized active set C_i (Sec. 2.1): primitives blended into at least one pixel.  Returns (mask words,
        ascending primitive ids)."""
        n = proj.depth.shape[0]
        active = np.zeros(n, np.uint8)
        self._f("oracle_realized_active")(
            _p(self._a(proj.xy)), _p(self._a(proj.conic_o)), _p(np.ascontiguousarray(vals, np.uint32)),
            _p(np.ascontiguousarray(ranges, np.uint32)), _p(_cam(cam)), _p(self.cfg),
            _p(np.ascontiguousarray(n_contrib, np.uint32)), C.c_int64(n), _p(active))
        idx = np.flatnonzero(active).astype(np.uint32)
        return ids_to_mask(idx, n), idx

    @staticmethod
    def gradient_evidence(g2d_dense, active_idx, rows=None, touched_idx=None):
        """Gradient evidence g(p) of the active primitives (Sec. 2.1 g_U(p); Sec. 4.3 gradient gate) and its mean over
        the active set.  Default reading: Euclidean norm of the gradient with respect to the projected centre (u, v),
        the first two of the nine compositing words.  With `rows` ([V, F] final gradient rows of the touched primitives
        `touched_idx`): Euclidean norm of the whole parameter-gradient row instead."""
        a = np.asarray(active_idx, np.int64)
        if rows is None:
            g = np.asarray(g2d_dense, np.float64)[a, :2]
        else:
            pos = np.searchsorted(np.asarray(touched_idx, np.int64), a)
            g = np.asarray(rows, np.float64)[pos]
        ev = np.sqrt((g * g).sum(axis=1))
        return ev, (float(ev.sum() / len(a)) if len(a) else 0.0)

    @staticmethod
    def hazard_sets(r_a, w_a, r_b, w_b):
        """The three primitive-state hazards of Sec. 4.3 for producer A and consumer B, as ascending id arrays."""
        r_a, w_a, r_b, w_b = (np.unique(np.asarray(x, np.int64)) for x in (r_a, w_a, r_b, w_b))
        waw = np.intersect1d(w_b, w_a)
        raw = np.intersect1d(np.setdiff1d(r_b, w_b), w_a)
        war = np.intersect1d(w_b, np.setdiff1d(r_a, w_a))
        return waw, raw, war

    @classmethod
    def delayed_read_gate(cls, r_a, w_a, r_b, w_b, active_a, evidence_a, tau):
        """Throughput-first admission of Sec. 4.3: D+ = C_RAW+(A, B); rho = |D+| / |R+(B)|; every delayed primitive
        needs producer evidence (membership in C_A) no larger than tau times the mean evidence over C_A."""
        _, delayed, _ = cls.hazard_sets(r_a, w_a, r_b, w_b)
        n_rb = len(np.unique(np.asarray(r_b, np.int64)))
        active_a = np.asarray(active_a, np.int64)
        evidence_a = np.asarray(evidence_a, np.float64)
        mean = float(evidence_a.sum() / len(active_a)) if len(active_a) else 0.0
        pos = np.searchsorted(active_a, delayed)
        pos_ok = pos < len(active_a)
        has = np.zeros(len(delayed), bool)
        has[pos_ok] = active_a[pos[pos_ok]] == delayed[pos_ok]
        passes = np.zeros(len(delayed), bool)
        passes[has] = evidence_a[pos[has]] <= tau * mean
        out = dict(n_delayed=len(delayed), n_read_b=n_rb, n_with_evidence=int(has.sum()), n_pass=int(passes.sum()),
                   mean=mean)
        out["rho"] = len(delayed) / n_rb if n_rb else None
        out["admitted"] = bool(n_rb > 0 and len(delayed) / n_rb <= tau and len(active_a) > 0 and has.all()
                               and passes.all())
        return out

    # ------------------------------------------------------------------ task units of several views (Sec. 2.1, Sec. 6.1)
    @staticmethod
    def accumulate_rows(idx_a, rows_a, idx_b, rows_b):
        """Gradient rows of a task unit of two views (Sec. 2.1: the unit's scope is the union of its views' scopes;
        Sec. 6.1 runs two views per unit): the union of the two ascending index lists and, per member, the sum of the
        rows the views hold for it (a view that did not touch the primitive contributes nothing)."""
        idx_a, idx_b = np.asarray(idx_a, np.int64), np.asarray(idx_b, np.int64)
        union = np.union1d(idx_a, idx_b)
        out = np.zeros((len(union), np.asarray(rows_a).shape[1]), np.float64)
        out[np.searchsorted(union, idx_a)] += np.asarray(rows_a, np.float64)
        out[np.searchsorted(union, idx_b)] += np.asarray(rows_b, np.float64)
        return union.astype(np.uint32), out

    def unit_step(self, params, m, v, cams, targets, lr, beta1, beta2, eps, step):
        """One task unit of two views: both are rendered and differentiated with the SAME parameters, their gradient
        rows are accumulated over the union of their touched sets, and one sparse Adam update is applied to the union
        at the unit's step."""
        views = [self.view_step(params, m, v, cam, tgt, lr, beta1, beta2, eps, step, update=False)
                 for cam, tgt in zip(cams, targets)]
        union, rows = self.accumulate_rows(views[0]["idx"], views[0]["rows"], views[1]["idx"], views[1]["rows"])
        self.sparse_adam(params, m, v, rows.astype(self.dtype), union, lr, beta1, beta2, eps, step)
        return dict(views=views, idx=union, rows=rows)

    # ------------------------------------------------------------------ relative locality graph from counts (Sec. 4.1, 4.2)
    @staticmethod
    def rlg_weights(sizes, pairs, counts) -> np.ndarray:
        """Eq. (1) with the per-view primitive sets in the place of the track sets (the computation-based RLG of
        Sec. 4.1): w_ij = |P_i & P_j| / |P_i | P_j|, 0 when the union is empty.  One float32 division per pair."""
        sizes = np.asarray(sizes, np.int64)
        pairs = np.asarray(pairs, np.int64).reshape(-1, 2)
        inter = np.asarray(counts, np.int64)
        union = sizes[pairs[:, 0]] + sizes[pairs[:, 1]] - inter
        w = np.zeros(len(pairs), np.float32)
        nz = union > 0
        w[nz] = inter[nz].astype(np.float32) / union[nz].astype(np.float32)
        return w

    @staticmethod
    def rlg_topk(weights, k: int) -> np.ndarray:
        """Neighbour retention of Sec. 4.1: every item keeps its k strongest neighbours (larger weight first, lower
        index first among equals, zero weights are not edges); the graph is undirected, so an edge stays when either
        end keeps it.  Dropped edges read as w = 0."""
        w = np.array(weights, np.float32, copy=True)
        n = w.shape[0]
        np.fill_diagonal(w, 0)
        keep = np.zeros((n, n), bool)
        for i in range(n):
            order = sorted((j for j in range(n) if j != i and w[i, j] > 0), key=lambda j: (-w[i, j], j))
            keep[i, order[:k]] = True
        keep |= keep.T
        return np.where(keep, w, np.float32(0))

    @staticmethod
    def sds_scores(weights, prev_unit, candidates) -> np.ndarray:
        """Eq. (2): s(v | U_prev) = sum over u in U_prev of w_uv, for every candidate v."""
        w = np.asarray(weights, np.float64)
        prev_unit = np.asarray(prev_unit, np.int64)
        return np.array([w[prev_unit, v].sum() for v in np.asarray(candidates, np.int64)], np.float64)

    def sh_basis(self, degree: int, x: float, y: float, z: float) -> np.ndarray:
        out = np.zeros(16, self.dtype)
        ct = C.c_float if self.dtype == np.float32 else C.c_double
        self._f("oracle_sh_basis")(C.c_int(degree), ct(x), ct(y), ct(z), _p(out))
        return out[: (degree + 1) ** 2]

    # ------------------------------------------------------------------ whole view
    def view_forward(self, scene, cam):
        proj = self.project(scene, cam)
        mask, idx = self.touched_set(proj.tiles_touched)
        keys, vals, ranges = self.bin_sort(proj, cam)
        out, final_t, ncon, margin, counters = self.render_fwd(proj, vals, ranges, cam)
        return dict(proj=proj, mask=mask, idx=idx, keys=keys, vals=vals, ranges=ranges, out=out, final_T=final_t,
                    n_contrib=ncon, pix_margin=margin, counters=counters)

    def view_step(self, params, m, v, cam, target, lr, beta1, beta2, eps, step, update: bool = True):
        """One training view: project, touched set, bin/sort, composite, L1 loss, backward, sparse Adam."""
        f = self.view_forward(params, cam)
        loss, dl = self.l1_loss(f["out"], target)
        g2d = self.render_bwd_blend(f["proj"], f["vals"], f["ranges"], cam, f["final_T"], f["n_contrib"], dl)
        rows = self.render_bwd_project(params, cam, f["idx"], g2d, f["proj"].clamp_flags)
        if update:
            self.sparse_adam(params, m, v, rows, f["idx"], lr, beta1, beta2, eps, step)
        f.update(loss=loss, dL_dout=dl, g2d=g2d, rows=rows)
        return f


_CACHE = {}


def get(dtype=np.float32) -> Oracle:
    key = np.dtype(dtype).str
    if key not in _CACHE:
        _CACHE[key] = Oracle(dtype)
    return _CACHE[key]
