"""Device buffers (through PyTorch) and the call sequence of one training view.

This file only allocates memory and marshals arguments; all arithmetic happens inside libodin.so.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional

import numpy as np
import torch

from . import binding as B


def _dev(a: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


class DeviceScene:
    """Five aligned attribute tensors on the device + the odin_scene struct that points at them."""

    def __init__(self, n: int, sh_degree: int, device, tensors=None):
        k = (sh_degree + 1) ** 2
        self.n, self.sh_degree, self.k = int(n), int(sh_degree), k
        if tensors is None:
            z = lambda *s: torch.zeros(*s, dtype=torch.float32, device=device)  # noqa: E731
            tensors = (z(max(n, 1), 3), z(max(n, 1), 3), z(max(n, 1), 4), z(max(n, 1)), z(max(n, 1), k, 3))
        self.means, self.log_scales, self.quats, self.opacity_logit, self.sh = tensors
        self.struct = B.make_scene(n, sh_degree, self.means, self.log_scales, self.quats, self.opacity_logit, self.sh)

    @classmethod
    def from_host(cls, scene, device) -> "DeviceScene":
        t = tuple(_dev(np.asarray(a, dtype=np.float32), device)
                  for a in (scene.means, scene.log_scales, scene.quats, scene.opacity_logit, scene.sh))
        return cls(scene.means.shape[0], scene.sh_degree, device, t)

    def tensors(self):
        return (self.means, self.log_scales, self.quats, self.opacity_logit, self.sh)

    def to_host(self):
        return tuple(t[: self.n].cpu().numpy() for t in self.tensors())

    def rows_as_matrix(self, v: int) -> np.ndarray:
        """First v rows as one [v, 11+3K] matrix in the order mean, log scale, quaternion, opacity, SH."""
        m, ls, q, o, sh = (t[:v].cpu().numpy() for t in self.tensors())
        return np.concatenate([m, ls, q, o[:, None], sh.reshape(v, -1)], axis=1)


class ProjectedBuffers:
    def __init__(self, n: int, capacity: int, device):
        cap = max(int(capacity), 1)
        self.n, self.capacity = int(n), int(capacity)
        i32, u8, f32 = torch.int32, torch.uint8, torch.float32
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)  # noqa: E731
        self.tiles_touched = z(max(n, 1), i32)
        self.prim_id = z(cap, i32)
        self.xy = z((cap, 2), f32)
        self.depth = z(cap, f32)
        self.conic_opacity = z((cap, 4), f32)
        self.rgb = z((cap, 3), f32)
        self.radius = z(cap, i32)
        self.rect = z((cap, 4), torch.int16)
        self.tile_offset = z(cap, i32)
        self.clamp_flags = z(cap, u8)
        self.num_rows = z(1, i32)
        self.num_instances = z(1, torch.int64)
        self.struct = B.odin_projected(
            self.capacity, *(t.data_ptr() for t in (self.tiles_touched, self.prim_id, self.xy, self.depth,
                                                    self.conic_opacity, self.rgb, self.radius, self.rect, self.tile_offset,
                                                    self.clamp_flags, self.num_rows, self.num_instances)), None)

    def load_rows(self, **arrays) -> None:
        """Overwrite compact arrays from host data (used by stage-isolated tests)."""
        for name, a in arrays.items():
            t = getattr(self, name)
            src = torch.from_numpy(np.ascontiguousarray(a))
            if src.dtype == torch.uint32:
                src = src.view(torch.int32)
            if src.dtype == torch.uint16:
                src = src.view(torch.int16)
            if src.dtype == torch.uint64:
                src = src.view(torch.int64)
            t.view(-1)[: src.numel()].copy_(src.view(-1).to(t.device))


class ViewTrainer:
    """Owns every device buffer of the view step and enqueues the seven calls (plus the loss) on one stream."""

    def __init__(self, scene, width: int, height: int, row_capacity: int, instance_capacity: int, mask_slots: int = 1,
                 device: int = 0, cfg: Optional[B.odin_config] = None, extra_render_records: int = 0):
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.ctx = B.odin_create(device, cfg)
        self.n, self.sh_degree = scene.means.shape[0], scene.sh_degree
        self.width, self.height = int(width), int(height)
        self.tx, self.ty = (width + 15) // 16, (height + 15) // 16
        self.row_capacity, self.instance_capacity = int(row_capacity), int(instance_capacity)
        dev = self.device
        self.params = DeviceScene.from_host(scene, dev)
        self.m = DeviceScene(self.n, self.sh_degree, dev)
        self.v = DeviceScene(self.n, self.sh_degree, dev)
        # one byte per primitive beside the moments: 0 = every moment of the primitive is zero (odin_sparse_adam_live).
        # Whoever writes self.m / self.v by other means than the optimizer calls calls moments_changed() afterwards.
        self.live = torch.zeros(max(self.n, 1), dtype=torch.uint8, device=dev)
        self.grads = DeviceScene(self.row_capacity, self.sh_degree, dev)
        self.proj = ProjectedBuffers(self.n, self.row_capacity, dev)
        z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)  # noqa: E731
        self.keys = z(max(self.instance_capacity, 1), torch.int64)
        self.vals = z(max(self.instance_capacity, 1), torch.int32)
        self.ranges = z((self.tx * self.ty, 2), torch.int32)
        self.out = z((3, height, width), torch.float32)
        self.final_T = z((height, width), torch.float32)
        self.n_contrib = z((height, width), torch.int32)
        self.target = z((3, height, width), torch.float32)
        self.dL = z((3, height, width), torch.float32)
        self.loss = z(1, torch.float32)
        self.grad2d = z((max(self.row_capacity, 1), 9), torch.float32)
        self.mask_words = (self.n + 31) // 32
        self.mask_stride = (self.mask_words + 3) // 4 * 4
        self.mask_slots = int(mask_slots)
        self.masks = z((self.mask_slots, max(self.mask_stride, 4)), torch.int32)
        self.idx = z(max(self.row_capacity, 1), torch.int32)
        self.count = z(1, torch.int32)
        # realized active set of the last view (Sec. 2.1 C_i) and its gradient evidence
        self.row_active = z(max(self.row_capacity, 1), torch.uint8)
        self.active_masks = z((self.mask_slots, max(self.mask_stride, 4)), torch.int32)
        self.active_idx = z(max(self.row_capacity, 1), torch.int32)
        self.active_count = z(1, torch.int32)
        self.evidence = z(max(self.row_capacity, 1), torch.float32)
        self.evidence_sum = z(1, torch.float64)
        # one workspace for odin_project / odin_touched_set (sized by the pool) and odin_bin_sort (sized by the rows and,
        # if the image is too large for the counting scatter, by the instances)
        sort_ws = []
        for mode in (0, 1):  # sized for either way of ordering the instances (see choose_instance_sort)
            B.odin_set_instance_sort(self.ctx, mode)
            sort_ws.append(B.odin_bin_sort_workspace_bytes(self.ctx, self.row_capacity, self.instance_capacity, self.width,
                                                           self.height))
        B.odin_set_instance_sort(self.ctx, 0 if cfg is None else int(cfg.instance_sort))
        self.ws = z(max(B.odin_workspace_bytes(self.ctx, self.n, 0), *sort_ws), torch.uint8)
        # The render workspace is a buffer of its own: the forward pass leaves per-pixel records for long lists in it
        # that the backward pass of the same view reads, so nothing else may write there in between.  Every 8,208
        # bytes beyond the minimum hold one more record (a further 256 list entries of one tile).
        self.render_ws = z(B.odin_render_workspace_bytes(self.ctx, self.width, self.height)
                           + 8208 * int(extra_render_records), torch.uint8)
        self.kernel_launches_per_step = 0
        self.keep_sorted_keys = False  # view_step: also write the sorted 64-bit keys (only tests look at them)
        self.track_active = False      # render_bwd: also flag the rows that contributed (needed by active_set)
        self.skip_zero_rows = True     # render_bwd flags zero gradient rows instead of writing them; Adam takes the flags
        # the touched set as a by-product of the projection's scan (mask written by odin_project, list = its row map):
        # view_step then leaves the separate odin_touched_set call out.  self.idx / self.count name the buffers that
        # hold the list and its length of the last view either way.
        self.fused_touched = True
        self._own_idx, self._own_count = self.idx, self.count
        self.row_zero = z(max(self.row_capacity, 1), torch.uint8)
        self._row_zero_in_use = None   # the flags the last render_bwd wrote (None: every row was written)

    def close(self) -> None:
        if self.ctx is not None:
            B.odin_destroy(self.ctx)
            self.ctx = None

    # -------------------------------------------------------------------------------------------- stages
    def project(self, cam: B.odin_camera, stream=None) -> None:
        B.odin_project(self.ctx, self.params.struct, cam, self.proj.struct, self.ws, stream)

    def touched_set(self, slot: int = 0, stream=None) -> None:
        B.odin_touched_set(self.ctx, self.proj.tiles_touched, self.n, self.masks[slot], self.idx, self.row_capacity,
                           self.count, self.ws, stream)

    def bin_sort(self, stream=None, want_keys: bool = True) -> None:
        """Sorted values and tile ranges; the sorted 64-bit keys too unless want_keys is False (no later stage reads them)."""
        B.odin_bin_sort(self.ctx, self.proj.struct, self.width, self.height, self.keys if want_keys else None, self.vals,
                        self.instance_capacity, self.ranges, self.ws, stream)

    def choose_instance_sort(self, cam: B.odin_camera, reps: int = 3) -> int:
        """Warm-up calibration: times odin_bin_sort on the CURRENT projection both ways (CUDA events, a few repetitions)
        and keeps the faster for the later views.  Synchronises the device; call it outside any timed region, after at
        least one odin_project.  Returns the mode kept."""
        stream = torch.cuda.current_stream()
        best = None
        for mode in (0, 1):
            B.odin_set_instance_sort(self.ctx, mode)
            self.bin_sort(want_keys=False)  # warm
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            ev[0].record(stream)
            for _ in range(reps):
                self.bin_sort(want_keys=False)
            ev[1].record(stream)
            torch.cuda.synchronize()
            ms = ev[0].elapsed_time(ev[1]) / reps
            if best is None or ms < best[1]:
                best = (mode, ms)
        B.odin_set_instance_sort(self.ctx, best[0])
        self.instance_sort = best[0]
        return best[0]

    def render_fwd(self, cam: B.odin_camera, stream=None) -> None:
        B.odin_render_fwd(self.ctx, self.proj.struct, self.vals, self.ranges, cam, self.out, self.final_T, self.n_contrib,
                          self.render_ws, stream)

    def l1_loss(self, stream=None) -> None:
        B.odin_l1_loss(self.ctx, self.out, self.target, self.width, self.height, self.loss, self.dL, stream)

    def render_bwd(self, cam: B.odin_camera, stream=None) -> None:
        # rows whose gradient is zero (never blended: most touched rows) are flagged instead of written, unless the
        # realized active set is tracked (its evidence reads the gradient rows)
        self._row_zero_in_use = self.row_zero if (self.skip_zero_rows and not self.track_active) else None
        B.odin_render_bwd(self.ctx, self.params.struct, cam, self.proj.struct, self.vals, self.ranges, self.final_T,
                          self.n_contrib, self.dL, self.grad2d, self.grads.struct,
                          self.row_active if self.track_active else None, self._row_zero_in_use, self.render_ws, stream)

    def gradient_rows(self, v: int) -> np.ndarray:
        """The first v gradient rows as one matrix (see DeviceScene.rows_as_matrix), the rows that the backward pass
        flagged as zero instead of writing them filled in with zeros."""
        rows = self.grads.rows_as_matrix(v)
        if self._row_zero_in_use is not None:
            rows[self._row_zero_in_use[:v].cpu().numpy().astype(bool)] = 0
        return rows

    def active_set(self, slot: int = 0, evidence_mode: int = 0, stream=None) -> None:
        """Realized active set of the view whose backward pass ran last (with track_active set): mask (slot), list,
        count, evidence, sum."""
        if not self.track_active:
            raise RuntimeError("active_set needs the row flags of render_bwd: set track_active before the backward pass")
        B.odin_active_set(self.ctx, self.proj.struct, self.row_active, self.grad2d, self.grads.struct, evidence_mode,
                          self.n, self.active_masks[slot], self.active_idx, self.row_capacity, self.active_count,
                          self.evidence, self.evidence_sum, self.ws, stream)

    def sparse_adam(self, lr, beta1, beta2, eps, step: int, stream=None) -> None:
        B.odin_sparse_adam_live(self.ctx, self.params.struct, self.m.struct, self.v.struct, self.grads.struct,
                                self._row_zero_in_use, self.idx, self.count, self.live, lr, beta1, beta2, eps, step,
                                stream)

    def moments_changed(self, stream=None) -> None:
        """Recompute the per-primitive flags of the optimizer after self.m / self.v were written from outside."""
        B.odin_adam_live_refresh(self.ctx, self.m.struct, self.v.struct, self.live, stream)

    def conflict_count(self, d_pairs, n_pairs: int, d_counts, stream=None) -> None:
        B.odin_conflict_count(self.ctx, self.masks, self.mask_slots, self.masks.shape[1], self.n, d_pairs, n_pairs,
                              d_counts, stream)

    # -------------------------------------------------------------------------------------------- whole view
    def view_step(self, cam: B.odin_camera, step: int, lr, beta1: float, beta2: float, eps: float, slot: int = 0,
                  d_pairs=None, n_pairs: int = 0, d_counts=None, update: bool = True, stream=None,
                  fused_touched: Optional[bool] = None) -> None:
        """project -> touched set -> bin/sort -> composite -> L1 loss -> backward -> sparse Adam -> conflict counts.
        The target image must already be in self.target.  Nothing here synchronises the host."""
        fused = self.fused_touched if fused_touched is None else fused_touched
        # nothing but this library's calls is enqueued until the end of the step: the calls are chained (the first
        # kernel of each is launched behind the last kernel of the one before it without an idle seam)
        B.odin_chain_begin(self.ctx)
        try:
            if fused:
                self.proj.struct.touched_mask = self.masks[slot].data_ptr()
                self.project(cam, stream)
                self.idx, self.count = self.proj.prim_id, self.proj.num_rows
            else:
                self.proj.struct.touched_mask = None
                if self.idx is self.proj.prim_id:
                    self.idx, self.count = self._own_idx, self._own_count
                self.project(cam, stream)
                self.touched_set(slot, stream)
            self.bin_sort(stream, want_keys=self.keep_sorted_keys)
            self.render_fwd(cam, stream)
            self.l1_loss(stream)
            self.render_bwd(cam, stream)
            if update:
                self.sparse_adam(lr, beta1, beta2, eps, step, stream)
            if n_pairs:
                self.conflict_count(d_pairs, n_pairs, d_counts, stream)
        finally:
            B.odin_chain_end(self.ctx)

    # -------------------------------------------------------------------------------------------- task unit of two views
    def prepare_unit(self):
        """Second set of per-view outputs and the union buffers of unit_step (allocated once)."""
        u = getattr(self, "_unit", None)
        if u is None:
            dev, cap = self.device, max(self.row_capacity, 1)
            z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=dev)  # noqa: E731
            union_cap = min(self.n, 2 * self.row_capacity)
            u = {
                "grads_b": DeviceScene(self.row_capacity, self.sh_degree, dev), "idx_b": z(cap, torch.int32),
                "count_b": z(1, torch.int32), "row_zero_b": z(cap, torch.uint8),
                "mask": z(max(self.mask_stride, 4), torch.int32), "members": z(2, torch.int32),
                "union_cap": union_cap, "idx_u": z(max(union_cap, 1), torch.int32), "count_u": z(1, torch.int32),
                "grads_u": DeviceScene(union_cap, self.sh_degree, dev), "loss": z(2, torch.float32),
            }
            self._unit = u
        return u

    def unit_step(self, cams, targets, step: int, lr, beta1: float, beta2: float, eps: float, slots=(0, 1),
                  stream=None) -> None:
        """One task unit of two views (Sec. 2.1 unit scopes; Sec. 6.1): both views are projected, rendered and
        differentiated with the same parameters, their gradient rows are added up over the union of their touched sets
        and one sparse Adam update is applied to the union.  Afterwards the unit's losses are in self._unit["loss"],
        the union list / count in self._unit["idx_u"] / ["count_u"], the views' masks in self.masks[slots].
        Marshalling only: every kernel is the library's."""
        u = self.prepare_unit()
        if self.mask_slots < 2:
            raise RuntimeError("unit_step needs two mask slots")
        first = (self.grads, self.idx, self.count, self.row_zero, self.loss, self.target)
        per_view = [(self.grads, self._own_idx, self._own_count, self.row_zero),
                    (u["grads_b"], u["idx_b"], u["count_b"], u["row_zero_b"])]
        zero_flags = []
        try:
            for k in range(2):
                self.grads, self.idx, self.count, self.row_zero = per_view[k]
                self.loss, self.target = u["loss"][k:k + 1], targets[k]
                # (the two views need index lists of their own: the separate touched-set call writes them)
                self.view_step(cams[k], step, lr, beta1, beta2, eps, slot=slots[k], update=False, stream=stream,
                               fused_touched=False)
                zero_flags.append(self._row_zero_in_use)
        finally:
            self.grads, self.idx, self.count, self.row_zero, self.loss, self.target = first
        u["members"].copy_(torch.tensor(list(slots), dtype=torch.int32), non_blocking=True)
        B.odin_mask_union(self.ctx, self.masks, self.mask_slots, self.masks.shape[1], self.n, u["members"], 2, u["mask"],
                          stream)
        B.odin_mask_to_list(self.ctx, u["mask"], self.n, u["idx_u"], u["union_cap"], u["count_u"], self.ws, stream)
        (ga, ia, ca, _), (gb, ib, cb, _) = per_view
        B.odin_accumulate_rows(self.ctx, ga.struct, zero_flags[0], ia, ca, gb.struct, zero_flags[1], ib, cb, u["idx_u"],
                               u["count_u"], u["grads_u"].struct, stream)
        B.odin_sparse_adam_live(self.ctx, self.params.struct, self.m.struct, self.v.struct, u["grads_u"].struct, None,
                                u["idx_u"], u["count_u"], self.live, lr, beta1, beta2, eps, step, stream)

    def prepare_host_io(self, n_counts: int = 0):
        """Staging buffers, pinned result slots, copy stream and events of train_from_host (allocated once)."""
        io = getattr(self, "_host_io", None)
        if io is None or io["n_counts"] < n_counts:
            io = {
                "n_counts": n_counts,
                "copy_stream": torch.cuda.Stream(device=self.device),
                "staging": [torch.empty_like(self.target) for _ in range(2)],
                "h_loss": [torch.zeros(1, dtype=torch.float32).pin_memory() for _ in range(2)],
                "h_count": [torch.zeros(1, dtype=torch.int32).pin_memory() for _ in range(2)],
                "h_counts": [torch.zeros(max(n_counts, 1), dtype=torch.int64).pin_memory() for _ in range(2)],
                "copied": [torch.cuda.Event() for _ in range(2)],
                "consumed": [torch.cuda.Event() for _ in range(2)],
                "done": [torch.cuda.Event() for _ in range(2)],
                # the results of a step are read back on a stream of their own, from device slots of the step's parity,
                # so that the compute stream carries kernels only and the next step need not wait for the read
                "read_stream": torch.cuda.Stream(device=self.device),
                "d_loss": [torch.zeros_like(self.loss) for _ in range(2)],
                "d_count": [torch.zeros_like(self.count) for _ in range(2)],
                "d_counts": [torch.zeros(max(n_counts, 1), dtype=torch.int64, device=self.device) for _ in range(2)],
            }
            self._host_io = io
        return io

    def train_from_host(self, steps, cam_of, host_target_of, lr, beta1: float, beta2: float, eps: float,
                        slot_of=lambda s: 0, pairs_of=None, d_counts=None, on_result=None) -> None:
        """Training views whose targets live in pinned HOST memory.  For every step s in `steps`: the target
        host_target_of(s) is copied to the device, the view cam_of(s) is stepped, and the loss, the number of touched
        primitives and (if pairs_of is given) the conflict counts are read back into pinned memory and handed to
        on_result(s, loss, touched, counts).  Two staging buffers and a copy stream: the copy of the next target
        overlaps the current view's kernels, the results are read back on a third stream from device slots that
        alternate with the step, and the host waits for the results of the previous view while the current one runs.
        Afterwards self.loss, self.count and d_counts hold the last step's results.  Marshalling only: every kernel
        is the library's."""
        steps = list(steps)
        n_counts = 0 if d_counts is None else d_counts.numel()
        io = self.prepare_host_io(n_counts)
        if not steps:
            return
        stream = torch.cuda.current_stream()
        copy_stream, staging = io["copy_stream"], io["staging"]
        h_loss, h_count, h_counts = io["h_loss"], io["h_count"], io["h_counts"]
        copied, consumed, done = io["copied"], io["consumed"], io["done"]
        read_stream = io["read_stream"]
        saved_target, saved_loss, saved_count = self.target, self.loss, self.count

        def enqueue_copy(i):
            k = i & 1
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(consumed[k])  # the step that read this buffer last has finished
                staging[k].copy_(host_target_of(steps[i]), non_blocking=True)
                copied[k].record(copy_stream)

        def deliver(i):
            k = i & 1
            done[k].synchronize()
            if on_result is not None:
                on_result(steps[i], float(h_loss[k][0]), int(h_count[k][0]), h_counts[k][:n_counts].clone())

        for k in range(2):
            consumed[k].record(stream)
        enqueue_copy(0)
        for i, s in enumerate(steps):
            k = i & 1
            if i + 1 < len(steps):
                enqueue_copy(i + 1)
            stream.wait_event(copied[k])
            self.target, self.loss, self.count = staging[k], io["d_loss"][k], io["d_count"][k]
            step_counts = io["d_counts"][k][:n_counts] if n_counts else None
            pairs = pairs_of(s) if pairs_of is not None else None
            self.view_step(cam_of(s), s + 1, lr, beta1, beta2, eps, slot=slot_of(s), d_pairs=pairs[0] if pairs else None,
                           n_pairs=pairs[1] if pairs else 0, d_counts=step_counts, stream=stream)
            if self.count is not io["d_count"][k]:  # the count lives in the projection's buffers: keep this step's copy
                io["d_count"][k].copy_(self.count, non_blocking=True)
                self.count = io["d_count"][k]
            consumed[k].record(stream)
            with torch.cuda.stream(read_stream):
                read_stream.wait_event(consumed[k])
                h_loss[k].copy_(self.loss, non_blocking=True)
                h_count[k].copy_(self.count, non_blocking=True)
                if n_counts:
                    h_counts[k][:n_counts].copy_(step_counts, non_blocking=True)
                done[k].record(read_stream)
            if i > 0:
                deliver(i - 1)  # also: the slots of parity k ^ 1 are free again before step i + 1 writes them
        deliver(len(steps) - 1)
        # leave the trainer as the plain loop would: its own buffers hold the last step's results
        k = (len(steps) - 1) & 1
        saved_loss.copy_(io["d_loss"][k])
        saved_count.copy_(io["d_count"][k])
        if n_counts:
            d_counts.view(-1)[:n_counts].copy_(io["d_counts"][k][:n_counts])
        self.target, self.loss, self.count = saved_target, saved_loss, saved_count

    def poll(self, stream=None) -> int:
        return B.odin_poll(self.ctx, stream)
