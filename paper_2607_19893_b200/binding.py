"""ctypes binding of libodin.so: the same entry points as include/odin.h, argument marshalling only.

PyTorch is used for device memory and streams; every step of the path runs in the library's CUDA kernels.  There
is no CPU fallback: if libodin.so is missing or cannot be loaded, the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libodin.so")

ODIN_OK = 0
ODIN_ERR_NULL = -1
ODIN_ERR_INVALID_ARG = -2
ODIN_ERR_CAPACITY = -3
ODIN_ERR_WORKSPACE = -4
ODIN_ERR_CUDA = -5
ODIN_ERR_TIMEOUT = -6
ODIN_ERR_UNSUPPORTED = -7

EXPORTS = [
    "odin_create", "odin_destroy", "odin_status_string", "odin_poll", "odin_workspace_bytes", "odin_project",
    "odin_touched_set", "odin_bin_sort", "odin_render_fwd", "odin_l1_loss", "odin_chain_begin", "odin_chain_end", "odin_render_bwd", "odin_sparse_adam",
    "odin_conflict_count", "odin_kernel_count", "odin_kernel_name", "odin_profile_enable", "odin_profile_collect",
    "odin_touched_set_static", "odin_render_workspace_bytes", "odin_active_set", "odin_mask_union", "odin_hazard_count",
    "odin_delayed_read_gate", "odin_rlg_weights", "odin_rlg_topk", "odin_sds_scores", "odin_set_wait_limit",
    "odin_bin_sort_workspace_bytes", "odin_set_instance_sort", "odin_measure_fp32_peak", "odin_count_blend_pairs",
    "odin_mask_to_list", "odin_accumulate_rows", "odin_sparse_adam_live", "odin_adam_live_refresh",
]


class OdinError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


class odin_config(C.Structure):
    _fields_ = [("alpha_min", C.c_float), ("alpha_max", C.c_float), ("t_min", C.c_float), ("dilation", C.c_float),
                ("radius_sigmas", C.c_float), ("jac_clamp", C.c_float), ("tile", C.c_int), ("binning", C.c_int),
                ("instance_sort", C.c_int)]


def default_config(binning: int = 0, instance_sort: int = 0) -> odin_config:
    """The renderer constants of the method; binning 1 selects the tight-extent tile rectangles, instance_sort 1 the
    radix passes over the instances in place of the counting scatter."""
    return odin_config(1.0 / 255.0, 0.99, 1e-4, 0.3, 3.0, 1.3, 16, int(binning), int(instance_sort))


class odin_camera(C.Structure):
    _fields_ = [("width", C.c_int), ("height", C.c_int), ("fx", C.c_float), ("fy", C.c_float), ("cx", C.c_float),
                ("cy", C.c_float), ("znear", C.c_float), ("zfar", C.c_float), ("w2c", C.c_float * 12),
                ("bg", C.c_float * 3)]


class odin_scene(C.Structure):
    _fields_ = [("n", C.c_uint32), ("sh_degree", C.c_int), ("means", C.c_void_p), ("log_scales", C.c_void_p),
                ("quats", C.c_void_p), ("opacity_logit", C.c_void_p), ("sh", C.c_void_p)]


class odin_projected(C.Structure):
    _fields_ = [("capacity", C.c_uint32), ("tiles_touched", C.c_void_p), ("prim_id", C.c_void_p), ("xy", C.c_void_p),
                ("depth", C.c_void_p), ("conic_opacity", C.c_void_p), ("rgb", C.c_void_p), ("radius", C.c_void_p),
                ("rect", C.c_void_p), ("tile_offset", C.c_void_p), ("clamp_flags", C.c_void_p),
                ("num_rows", C.c_void_p), ("num_instances", C.c_void_p), ("touched_mask", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Loads libodin.so (once).  Raises if the CUDA library has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2607_19893_b200.build` "
                "(nvcc, sm_100a).  The CUDA library is the only implementation; there is no CPU fallback."
            )
        L = C.CDLL(LIB_PATH)
        L.odin_status_string.restype = C.c_char_p
        L.odin_status_string.argtypes = [C.c_int]
        vp, u32, u64, i32, f32 = C.c_void_p, C.c_uint32, C.c_uint64, C.c_int, C.c_float
        L.odin_create.argtypes = [C.POINTER(vp), i32, C.POINTER(odin_config)]
        L.odin_destroy.argtypes = [vp]
        L.odin_poll.argtypes = [vp, vp]
        L.odin_set_wait_limit.argtypes = [vp, i32]
        L.odin_set_instance_sort.argtypes = [vp, i32]
        L.odin_mask_to_list.argtypes = [vp, vp, u32, vp, u32, vp, vp, C.c_size_t, vp]
        L.odin_accumulate_rows.argtypes = [vp, C.POINTER(odin_scene), vp, vp, vp, C.POINTER(odin_scene), vp, vp, vp, vp, vp,
                                           C.POINTER(odin_scene), vp]
        L.odin_measure_fp32_peak.argtypes = [vp, vp, C.POINTER(C.c_float)]
        L.odin_count_blend_pairs.argtypes = [vp, C.POINTER(odin_projected), vp, vp, C.POINTER(odin_camera), vp, vp, vp]
        L.odin_workspace_bytes.argtypes = [vp, u32, u64, C.POINTER(C.c_size_t)]
        L.odin_bin_sort_workspace_bytes.argtypes = [vp, u32, u64, i32, i32, C.POINTER(C.c_size_t)]
        L.odin_project.argtypes = [vp, C.POINTER(odin_scene), C.POINTER(odin_camera), C.POINTER(odin_projected), vp,
                                   C.c_size_t, vp]
        L.odin_touched_set.argtypes = [vp, vp, u32, vp, vp, u32, vp, vp, C.c_size_t, vp]
        L.odin_bin_sort.argtypes = [vp, C.POINTER(odin_projected), i32, i32, vp, vp, u64, vp, vp, C.c_size_t, vp]
        L.odin_render_workspace_bytes.argtypes = [vp, i32, i32, C.POINTER(C.c_size_t)]
        L.odin_render_fwd.argtypes = [vp, C.POINTER(odin_projected), vp, vp, C.POINTER(odin_camera), vp, vp, vp, vp,
                                      C.c_size_t, vp]
        L.odin_l1_loss.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp]
        L.odin_chain_begin.argtypes = [vp]
        L.odin_chain_end.argtypes = [vp]
        L.odin_render_bwd.argtypes = [vp, C.POINTER(odin_scene), C.POINTER(odin_camera), C.POINTER(odin_projected), vp, vp,
                                      vp, vp, vp, vp, C.POINTER(odin_scene), vp, vp, vp, C.c_size_t, vp]
        L.odin_sparse_adam.argtypes = [vp, C.POINTER(odin_scene), C.POINTER(odin_scene), C.POINTER(odin_scene),
                                       C.POINTER(odin_scene), vp, vp, vp, C.POINTER(f32), f32, f32, f32, u32, vp]
        L.odin_sparse_adam_live.argtypes = [vp, C.POINTER(odin_scene), C.POINTER(odin_scene), C.POINTER(odin_scene),
                                            C.POINTER(odin_scene), vp, vp, vp, vp, C.POINTER(f32), f32, f32, f32, u32, vp]
        L.odin_adam_live_refresh.argtypes = [vp, C.POINTER(odin_scene), C.POINTER(odin_scene), vp, vp]
        L.odin_conflict_count.argtypes = [vp, vp, u32, u32, u32, vp, u32, vp, vp]
        L.odin_touched_set_static.argtypes = [vp, u32, vp, vp, u32, vp, vp, vp]
        L.odin_active_set.argtypes = [vp, C.POINTER(odin_projected), vp, vp, C.POINTER(odin_scene), i32, u32, vp, vp, u32,
                                      vp, vp, vp, vp, C.c_size_t, vp]
        L.odin_mask_union.argtypes = [vp, vp, u32, u32, u32, vp, u32, vp, vp]
        L.odin_hazard_count.argtypes = [vp, vp, vp, u32, u32, u32, vp, u32, vp, vp]
        L.odin_delayed_read_gate.argtypes = [vp, vp, vp, vp, u32, vp, vp, vp, vp, u32, f32, vp, vp]
        L.odin_rlg_weights.argtypes = [vp, vp, vp, vp, u32, u32, vp, vp]
        L.odin_rlg_topk.argtypes = [vp, vp, u32, u32, vp, vp, C.c_size_t, vp]
        L.odin_sds_scores.argtypes = [vp, vp, u32, vp, u32, vp, u32, vp, vp]
        L.odin_kernel_count.argtypes = []
        L.odin_kernel_name.argtypes = [i32]
        L.odin_profile_enable.argtypes = [vp, i32]
        L.odin_profile_collect.argtypes = [vp, vp, C.POINTER(f32), C.POINTER(u64)]
        for name in EXPORTS:
            if name not in ("odin_status_string", "odin_kernel_name"):
                getattr(L, name).restype = C.c_int
        L.odin_kernel_name.restype = C.c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().odin_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != ODIN_OK:
        raise OdinError(status, where)


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / raw integer / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch

        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def make_camera(cam) -> odin_camera:
    """From an object with width, height, fx, fy, cx, cy, znear, zfar, w2c[3][4], bg[3] attributes."""
    c = odin_camera()
    c.width, c.height = int(cam.width), int(cam.height)
    c.fx, c.fy, c.cx, c.cy = float(cam.fx), float(cam.fy), float(cam.cx), float(cam.cy)
    c.znear, c.zfar = float(cam.znear), float(min(cam.zfar, 3.0e38))
    w = np.asarray(cam.w2c, dtype=np.float32).reshape(12)
    for i in range(12):
        c.w2c[i] = float(w[i])
    for i in range(3):
        c.bg[i] = float(cam.bg[i])
    return c


def make_scene(n: int, sh_degree: int, means, log_scales, quats, opacity_logit, sh) -> odin_scene:
    return odin_scene(int(n), int(sh_degree), _ptr(means), _ptr(log_scales), _ptr(quats), _ptr(opacity_logit), _ptr(sh))


# ------------------------------------------------------------------------------------------------ entry points
def odin_create(device: int = 0, cfg: Optional[odin_config] = None) -> C.c_void_p:
    ctx = C.c_void_p()
    _check(lib().odin_create(C.byref(ctx), int(device), C.byref(cfg) if cfg is not None else None), "odin_create")
    return ctx


def odin_destroy(ctx) -> None:
    _check(lib().odin_destroy(ctx), "odin_destroy")


def odin_poll(ctx, stream=None) -> int:
    """Synchronises the stream and returns the deferred device-side status (0 = ok) without raising."""
    return int(lib().odin_poll(ctx, _stream(stream)))


def odin_bin_sort_workspace_bytes(ctx, row_capacity: int, max_instances: int, width: int, height: int) -> int:
    b = C.c_size_t(0)
    _check(lib().odin_bin_sort_workspace_bytes(ctx, int(row_capacity), int(max_instances), int(width), int(height),
                                               C.byref(b)), "odin_bin_sort_workspace_bytes")
    return int(b.value)


def odin_measure_fp32_peak(ctx, stream=None) -> float:
    """Sustained fp32 multiply-add rate of the device in TFLOP/s (synchronises)."""
    t = C.c_float(0.0)
    _check(lib().odin_measure_fp32_peak(ctx, _stream(stream), C.byref(t)), "odin_measure_fp32_peak")
    return float(t.value)


def odin_count_blend_pairs(ctx, proj: odin_projected, d_vals, d_tile_ranges, cam: odin_camera, d_n_contrib, d_counts,
                           stream=None) -> None:
    _check(lib().odin_count_blend_pairs(ctx, C.byref(proj), _ptr(d_vals), _ptr(d_tile_ranges), C.byref(cam),
                                        _ptr(d_n_contrib), _ptr(d_counts), _stream(stream)), "odin_count_blend_pairs")


def odin_mask_to_list(ctx, d_mask, n: int, d_idx, idx_capacity: int, d_count, ws, stream=None) -> None:
    _check(lib().odin_mask_to_list(ctx, _ptr(d_mask), int(n), _ptr(d_idx), int(idx_capacity), _ptr(d_count), _ptr(ws),
                                   0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "odin_mask_to_list")


def odin_accumulate_rows(ctx, rows_a: odin_scene, d_zero_a, d_idx_a, d_count_a, rows_b: odin_scene, d_zero_b, d_idx_b,
                         d_count_b, d_idx_u, d_count_u, rows_u: odin_scene, stream=None) -> None:
    _check(lib().odin_accumulate_rows(ctx, C.byref(rows_a), _ptr(d_zero_a), _ptr(d_idx_a), _ptr(d_count_a),
                                      C.byref(rows_b), _ptr(d_zero_b), _ptr(d_idx_b), _ptr(d_count_b), _ptr(d_idx_u),
                                      _ptr(d_count_u), C.byref(rows_u), _stream(stream)), "odin_accumulate_rows")


def odin_set_instance_sort(ctx, mode: int) -> None:
    _check(lib().odin_set_instance_sort(ctx, int(mode)), "odin_set_instance_sort")


def odin_set_wait_limit(ctx, polls: int) -> None:
    _check(lib().odin_set_wait_limit(ctx, int(polls)), "odin_set_wait_limit")


def odin_workspace_bytes(ctx, n: int, max_instances: int) -> int:
    b = C.c_size_t(0)
    _check(lib().odin_workspace_bytes(ctx, int(n), int(max_instances), C.byref(b)), "odin_workspace_bytes")
    return int(b.value)


def odin_project(ctx, scene: odin_scene, cam: odin_camera, out: odin_projected, ws, stream=None) -> None:
    _check(lib().odin_project(ctx, C.byref(scene), C.byref(cam), C.byref(out), _ptr(ws),
                              0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)), "odin_project")


def odin_touched_set(ctx, d_tiles_touched, n: int, d_mask, d_idx, idx_capacity: int, d_count, ws, stream=None) -> None:
    _check(lib().odin_touched_set(ctx, _ptr(d_tiles_touched), int(n), _ptr(d_mask), _ptr(d_idx), int(idx_capacity),
                                  _ptr(d_count), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                  _stream(stream)), "odin_touched_set")


def odin_touched_set_static(d_tiles_touched, n: int, d_mask, d_idx, idx_capacity: int, d_count, d_status=None,
                            stream=None) -> None:
    """Touched set for callers that are not allowed to allocate GPU memory (no context, no workspace): the scratch is
    a fixed array inside the library, n <= 2**25.  Calls on one device share that array: do not let two overlap."""
    _check(lib().odin_touched_set_static(_ptr(d_tiles_touched), int(n), _ptr(d_mask), _ptr(d_idx), int(idx_capacity),
                                         _ptr(d_count), _ptr(d_status), _stream(stream)), "odin_touched_set_static")


def odin_bin_sort(ctx, proj: odin_projected, width: int, height: int, d_keys, d_vals, capacity: int, d_tile_ranges, ws,
                  stream=None) -> None:
    _check(lib().odin_bin_sort(ctx, C.byref(proj), int(width), int(height), _ptr(d_keys), _ptr(d_vals), int(capacity),
                               _ptr(d_tile_ranges), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                               _stream(stream)), "odin_bin_sort")


def odin_render_fwd(ctx, proj: odin_projected, d_vals, d_tile_ranges, cam: odin_camera, d_rgb, d_final_T, d_n_contrib,
                    ws, stream=None) -> None:
    _check(lib().odin_render_fwd(ctx, C.byref(proj), _ptr(d_vals), _ptr(d_tile_ranges), C.byref(cam), _ptr(d_rgb),
                                 _ptr(d_final_T), _ptr(d_n_contrib), _ptr(ws),
                                 0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)), "odin_render_fwd")


def odin_chain_begin(ctx) -> None:
    _check(lib().odin_chain_begin(ctx), "odin_chain_begin")


def odin_chain_end(ctx) -> None:
    _check(lib().odin_chain_end(ctx), "odin_chain_end")


def odin_render_workspace_bytes(ctx, width: int, height: int) -> int:
    b = C.c_size_t(0)
    _check(lib().odin_render_workspace_bytes(ctx, int(width), int(height), C.byref(b)), "odin_render_workspace_bytes")
    return int(b.value)


def odin_l1_loss(ctx, d_rgb, d_target, width: int, height: int, d_loss, d_dL_drgb, stream=None) -> None:
    _check(lib().odin_l1_loss(ctx, _ptr(d_rgb), _ptr(d_target), int(width), int(height), _ptr(d_loss), _ptr(d_dL_drgb),
                              _stream(stream)), "odin_l1_loss")


def odin_render_bwd(ctx, scene: odin_scene, cam: odin_camera, proj: odin_projected, d_vals, d_tile_ranges, d_final_T,
                    d_n_contrib, d_dL_drgb, d_grad2d, grad_rows: odin_scene, d_row_active, d_row_zero, ws,
                    stream=None) -> None:
    _check(lib().odin_render_bwd(ctx, C.byref(scene), C.byref(cam), C.byref(proj), _ptr(d_vals), _ptr(d_tile_ranges),
                                 _ptr(d_final_T), _ptr(d_n_contrib), _ptr(d_dL_drgb), _ptr(d_grad2d), C.byref(grad_rows),
                                 _ptr(d_row_active), _ptr(d_row_zero), _ptr(ws),
                                 0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)),
           "odin_render_bwd")


def odin_sparse_adam(ctx, params: odin_scene, m: odin_scene, v: odin_scene, grad_rows: odin_scene, d_row_zero, d_idx,
                     d_count, lr: Sequence[float], beta1: float, beta2: float, eps: float, step: int, stream=None) -> None:
    lr_arr = (C.c_float * 6)(*[float(x) for x in lr])
    _check(lib().odin_sparse_adam(ctx, C.byref(params), C.byref(m), C.byref(v), C.byref(grad_rows), _ptr(d_row_zero),
                                  _ptr(d_idx), _ptr(d_count), lr_arr, float(beta1), float(beta2), float(eps), int(step),
                                  _stream(stream)), "odin_sparse_adam")


def odin_sparse_adam_live(ctx, params: odin_scene, m: odin_scene, v: odin_scene, grad_rows: odin_scene, d_row_zero, d_idx,
                          d_count, d_live, lr: Sequence[float], beta1: float, beta2: float, eps: float, step: int,
                          stream=None) -> None:
    lr_arr = (C.c_float * 6)(*[float(x) for x in lr])
    _check(lib().odin_sparse_adam_live(ctx, C.byref(params), C.byref(m), C.byref(v), C.byref(grad_rows), _ptr(d_row_zero),
                                       _ptr(d_idx), _ptr(d_count), _ptr(d_live), lr_arr, float(beta1), float(beta2),
                                       float(eps), int(step), _stream(stream)), "odin_sparse_adam_live")


def odin_adam_live_refresh(ctx, m: odin_scene, v: odin_scene, d_live, stream=None) -> None:
    _check(lib().odin_adam_live_refresh(ctx, C.byref(m), C.byref(v), _ptr(d_live), _stream(stream)),
           "odin_adam_live_refresh")


def odin_conflict_count(ctx, d_masks, n_masks: int, mask_stride_words: int, n_prims: int, d_pairs, n_pairs: int, d_counts,
                        stream=None) -> None:
    _check(lib().odin_conflict_count(ctx, _ptr(d_masks), int(n_masks), int(mask_stride_words), int(n_prims), _ptr(d_pairs),
                                     int(n_pairs), _ptr(d_counts), _stream(stream)), "odin_conflict_count")


def odin_active_set(ctx, proj: odin_projected, d_row_active, d_grad2d, grad_rows: Optional[odin_scene],
                    evidence_mode: int, n: int, d_mask, d_idx, idx_capacity: int, d_count, d_evidence, d_evidence_sum, ws,
                    stream=None) -> None:
    _check(lib().odin_active_set(ctx, C.byref(proj), _ptr(d_row_active), _ptr(d_grad2d),
                                 None if grad_rows is None else C.byref(grad_rows), int(evidence_mode), int(n),
                                 _ptr(d_mask), _ptr(d_idx), int(idx_capacity), _ptr(d_count), _ptr(d_evidence),
                                 _ptr(d_evidence_sum), _ptr(ws), 0 if ws is None else ws.numel() * ws.element_size(),
                                 _stream(stream)), "odin_active_set")


def odin_mask_union(ctx, d_masks, n_masks: int, mask_stride_words: int, n_prims: int, d_members, n_members: int, d_out,
                    stream=None) -> None:
    _check(lib().odin_mask_union(ctx, _ptr(d_masks), int(n_masks), int(mask_stride_words), int(n_prims), _ptr(d_members),
                                 int(n_members), _ptr(d_out), _stream(stream)), "odin_mask_union")


def odin_hazard_count(ctx, d_read_masks, d_write_masks, n_masks: int, mask_stride_words: int, n_prims: int, d_pairs,
                      n_pairs: int, d_counts, stream=None) -> None:
    _check(lib().odin_hazard_count(ctx, _ptr(d_read_masks), _ptr(d_write_masks), int(n_masks), int(mask_stride_words),
                                   int(n_prims), _ptr(d_pairs), int(n_pairs), _ptr(d_counts), _stream(stream)),
           "odin_hazard_count")


def odin_delayed_read_gate(ctx, d_read_b, d_write_b, d_write_a, n_prims: int, d_active_idx_a, d_evidence_a,
                           d_active_count_a, d_evidence_sum_a, active_capacity_a: int, tau: float, d_gate,
                           stream=None) -> None:
    _check(lib().odin_delayed_read_gate(ctx, _ptr(d_read_b), _ptr(d_write_b), _ptr(d_write_a), int(n_prims),
                                        _ptr(d_active_idx_a), _ptr(d_evidence_a), _ptr(d_active_count_a),
                                        _ptr(d_evidence_sum_a), int(active_capacity_a), float(tau), _ptr(d_gate),
                                        _stream(stream)), "odin_delayed_read_gate")


def odin_rlg_weights(ctx, d_counts, d_sizes, d_pairs, n_pairs: int, n_views: int, d_weights, stream=None) -> None:
    _check(lib().odin_rlg_weights(ctx, _ptr(d_counts), _ptr(d_sizes), _ptr(d_pairs), int(n_pairs), int(n_views),
                                  _ptr(d_weights), _stream(stream)), "odin_rlg_weights")


def odin_rlg_topk(ctx, d_weights, n_views: int, k: int, d_retained, ws, stream=None) -> None:
    _check(lib().odin_rlg_topk(ctx, _ptr(d_weights), int(n_views), int(k), _ptr(d_retained), _ptr(ws),
                               0 if ws is None else ws.numel() * ws.element_size(), _stream(stream)), "odin_rlg_topk")


def odin_sds_scores(ctx, d_weights, n_views: int, d_prev_unit, n_prev: int, d_candidates, n_candidates: int, d_scores,
                    stream=None) -> None:
    _check(lib().odin_sds_scores(ctx, _ptr(d_weights), int(n_views), _ptr(d_prev_unit), int(n_prev), _ptr(d_candidates),
                                 int(n_candidates), _ptr(d_scores), _stream(stream)), "odin_sds_scores")


def odin_kernel_count() -> int:
    return int(lib().odin_kernel_count())


def odin_kernel_name(kid: int) -> str:
    return lib().odin_kernel_name(int(kid)).decode()


def odin_profile_enable(ctx, on: bool) -> None:
    _check(lib().odin_profile_enable(ctx, 1 if on else 0), "odin_profile_enable")


def odin_profile_collect(ctx, stream=None):
    """Synchronises the stream; returns {kernel name: (milliseconds summed over its launches, launches)}."""
    k = odin_kernel_count()
    ms = (C.c_float * k)()
    cnt = (C.c_uint64 * k)()
    _check(lib().odin_profile_collect(ctx, _stream(stream), ms, cnt), "odin_profile_collect")
    return {odin_kernel_name(i): (float(ms[i]), int(cnt[i])) for i in range(k)}
