// Optimizer update restricted to the touched rows: bandwidth-bound gather / scatter Adam.
// The gradient side is read fully coalesced (consecutive threads, consecutive floats of the compact rows); the
// parameter side touches, per row, one contiguous span per attribute array (192 B for degree-3 SH = six full sectors).
#include "common.cuh"

namespace {

// A row whose gradient and both moments are zero is left alone: m' = v' = 0 and theta' = theta - step * 0 / (0 + eps) =
// theta bit for bit (eps > 0), so neither the parameter is read nor anything written.  Most touched rows of a view are
// occluded (zero gradient), and until a primitive has been active in some view its moments are zero too: for those
// rows the update costs the two moment reads only.  (skip_idle is off when eps == 0, where 0 / 0 would be the result.)
struct AdamK {
  int skip_idle;
  float beta1, beta2, omb1, omb2, eps;
  float step_size[6];  // lr_g / (1 - beta1^t)
  float inv_bc2s;      // 1 / sqrt(1 - beta2^t)
};

// The square root and the division are the hardware approximations (relative error ~1e-7 each, far inside the bar
// on the updated parameter): the correctly rounded forms are ~20 instructions per scalar, which made these kernels
// issue-bound next to their memory traffic.
__device__ __forceinline__ float adam_sqrt(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void adam_one(float& th, float& m, float& v, float g, float step_size, const AdamK& k) {
  m = k.beta1 * m + k.omb1 * g;
  v = k.beta2 * v + k.omb2 * g * g;
  th = th - __fdividef(step_size * m, adam_sqrt(v) * k.inv_bc2s + k.eps);
}

// Flags of the primitives whose moments may be non-zero (live[p] == 0: every moment of p, in every attribute, is zero).
// With them a row that has no gradient and no history costs its index and two bytes instead of a read of both moments.
__device__ __forceinline__ bool adam_cold(const uint8_t* live, size_t prim, const AdamK& k) {
  return live && k.skip_idle && live[prim] == 0;
}
// Called by a thread that is about to write moments that may be non-zero.
__device__ __forceinline__ void adam_mark_live(uint8_t* live, size_t prim, bool cold, const AdamK& k) {
  if (live && (cold || !k.skip_idle)) live[prim] = 1;
}

// Both kernels give a warp 32 consecutive rows of the list at a time.  The warp first looks at the rows themselves
// (index, row flag, primitive flag: three coalesced or nearly coalesced loads), drops the rows with nothing to do - no
// gradient and no history, or an index out of range - and leaves the others, in order, in shared memory; the elements
// of the remaining rows are then spread over the lanes.  Where most rows of a view are occluded a warp so works on full
// loads of the few rows that matter instead of running the whole chain of dependent loads for one live lane in eight.
constexpr int ADAM_WARPS = 8;

// returns the number of rows kept; s_prim[i] = primitive, s_info[i] = place in the group | zero << 8 | cold << 9
__device__ __forceinline__ uint32_t adam_stage_rows(uint32_t grp, uint32_t V, const uint32_t* __restrict__ idx,
                                                    const uint8_t* __restrict__ row_zero, const uint8_t* live,
                                                    uint32_t n_prims, const AdamK& k, uint32_t* s_prim, uint32_t* s_info,
                                                    unsigned lane) {
  const uint32_t r = grp * 32 + lane;
  uint32_t prim = 0;
  bool zero = false, cold = false, act = false;
  if (r < V) {
    prim = idx[r];
    if (prim < n_prims) {  // (an index list that is not a view's own, e.g. after a timed-out scan: no write)
      zero = row_zero && row_zero[r];  // the gradient row was not written: it is zero
      // cold: the primitive's flag says that all of its moments are zero, so they are not read.  (A thread of the
      // other kernel may raise the flag while this one reads it; either value is right here: the moments this kernel
      // owns are written by nobody else.)
      cold = adam_cold(live, prim, k);
      act = !(cold && zero);
    }
  }
  const uint32_t mask = __ballot_sync(0xffffffffu, act);
  __syncwarp();  // the previous group's entries have been read
  if (act) {
    const uint32_t pos = __popc(mask & ((1u << lane) - 1u));
    s_prim[pos] = prim;
    s_info[pos] = lane | (zero ? 256u : 0u) | (cold ? 512u : 0u);
  }
  __syncwarp();
  return (uint32_t)__popc(mask);
}

// SH block: ROWF floats per row (3, 12, 27 or 48), processed as VEC-wide elements.
template <int ROWF, int VEC>
__global__ void __launch_bounds__(ADAM_WARPS * 32)
adam_sh_kernel(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v, const float* __restrict__ g,
               const uint32_t* __restrict__ idx, const uint32_t* __restrict__ count, uint32_t cap, AdamK k,
               const uint8_t* __restrict__ row_zero, uint32_t n_prims, uint8_t* live) {
  odin_after_predecessor();
  constexpr int EPR = ROWF / VEC;  // elements per row
  __shared__ uint32_t s_prim[ADAM_WARPS][32], s_info[ADAM_WARPS][32];
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t V = min(*count, cap);
  const uint32_t groups = (V + 31) / 32;
  // with the primitive flags in use a row that gets this far nearly always has work: its parameters are then fetched
  // together with the moments instead of after the test on them
  const bool eager = live != nullptr;
  for (uint32_t grp = blockIdx.x * ADAM_WARPS + warp; grp < groups; grp += gridDim.x * ADAM_WARPS) {
    const uint32_t kept = adam_stage_rows(grp, V, idx, row_zero, live, n_prims, k, s_prim[warp], s_info[warp], lane);
    for (uint32_t q = lane; q < kept * EPR; q += 32) {
      const uint32_t slot = q / EPR, j = q - slot * EPR;
      const uint32_t prim = s_prim[warp][slot], info = s_info[warp][slot];
      const bool zero = info & 256u, cold = info & 512u;
      const size_t e = (size_t)(grp * 32 + (info & 255u)) * EPR + j;  // element of the compact gradient block
      const size_t dst = (size_t)prim * ROWF + (size_t)j * VEC;
      if (VEC == 4) {
        const float4 gg = zero ? make_float4(0.f, 0.f, 0.f, 0.f) : reinterpret_cast<const float4*>(g)[e];
        const bool gzero = gg.x == 0.f && gg.y == 0.f && gg.z == 0.f && gg.w == 0.f;
        if (cold && gzero) continue;
        float4 mm = make_float4(0.f, 0.f, 0.f, 0.f), vv = mm, pp = mm;
        if (!cold) { mm = *reinterpret_cast<float4*>(m + dst); vv = *reinterpret_cast<float4*>(v + dst); }
        if (eager) pp = *reinterpret_cast<float4*>(p + dst);
        if (k.skip_idle && gzero && mm.x == 0.f && mm.y == 0.f && mm.z == 0.f && mm.w == 0.f && vv.x == 0.f &&
            vv.y == 0.f && vv.z == 0.f && vv.w == 0.f)
          continue;
        adam_mark_live(live, prim, cold, k);
        if (!eager) pp = *reinterpret_cast<float4*>(p + dst);
        // floats 0..2 of a row are the degree-0 coefficients (group 4); the rest group 5
        const int f0 = j * 4;
        adam_one(pp.x, mm.x, vv.x, gg.x, k.step_size[f0 + 0 < 3 ? 4 : 5], k);
        adam_one(pp.y, mm.y, vv.y, gg.y, k.step_size[f0 + 1 < 3 ? 4 : 5], k);
        adam_one(pp.z, mm.z, vv.z, gg.z, k.step_size[f0 + 2 < 3 ? 4 : 5], k);
        adam_one(pp.w, mm.w, vv.w, gg.w, k.step_size[5], k);
        *reinterpret_cast<float4*>(p + dst) = pp;
        *reinterpret_cast<float4*>(m + dst) = mm;
        *reinterpret_cast<float4*>(v + dst) = vv;
      } else {
        const float gg = zero ? 0.f : g[e];
        if (cold && gg == 0.f) continue;
        float mm = 0.f, vv = 0.f, pp = 0.f;
        if (!cold) { mm = m[dst]; vv = v[dst]; }
        if (eager) pp = p[dst];
        if (k.skip_idle && gg == 0.f && mm == 0.f && vv == 0.f) continue;
        adam_mark_live(live, prim, cold, k);
        if (!eager) pp = p[dst];
        adam_one(pp, mm, vv, gg, k.step_size[j < 3 ? 4 : 5], k);
        p[dst] = pp; m[dst] = mm; v[dst] = vv;
      }
    }
  }
}

// Geometry block: four lanes per row - mean(3), log scale(3), quaternion(4), opacity(1) - on ONE code path (the part
// selects base pointers and a width), so that the loads of all four parts of eight rows are in flight together; with a
// branch per part the warp ran three chains of dependent loads one after the other.
__global__ void __launch_bounds__(ADAM_WARPS * 32)
adam_geom_kernel(float* __restrict__ p_mean, float* __restrict__ p_ls, float* __restrict__ p_q, float* __restrict__ p_o,
                 float* __restrict__ m_mean, float* __restrict__ m_ls, float* __restrict__ m_q, float* __restrict__ m_o,
                 float* __restrict__ v_mean, float* __restrict__ v_ls, float* __restrict__ v_q, float* __restrict__ v_o,
                 const float* __restrict__ g_mean, const float* __restrict__ g_ls, const float* __restrict__ g_q,
                 const float* __restrict__ g_o, const uint32_t* __restrict__ idx, const uint32_t* __restrict__ count,
                 uint32_t cap, AdamK k, const uint8_t* __restrict__ row_zero, uint32_t n_prims, uint8_t* live) {
  odin_after_predecessor();  // launched behind the SH kernel (which it does not depend on: the two overlap at the seam)
  __shared__ uint32_t s_prim[ADAM_WARPS][32], s_info[ADAM_WARPS][32];
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t V = min(*count, cap);
  const uint32_t groups = (V + 31) / 32;
  const bool eager = live != nullptr;  // (see the SH kernel)
  const int part = (int)(lane & 3);
  const int width = part < 2 ? 3 : (part == 2 ? 4 : 1);
  const float ss = k.step_size[part];
  for (uint32_t grp = blockIdx.x * ADAM_WARPS + warp; grp < groups; grp += gridDim.x * ADAM_WARPS) {
    const uint32_t kept = adam_stage_rows(grp, V, idx, row_zero, live, n_prims, k, s_prim[warp], s_info[warp], lane);
    for (uint32_t slot = lane >> 2; slot < kept; slot += 8) {
      const size_t d = s_prim[warp][slot];
      const uint32_t info = s_info[warp][slot];
      const bool zero = info & 256u, cold = info & 512u;
      const size_t r = (size_t)grp * 32 + (info & 255u);
      const size_t od = (size_t)width * d, og = (size_t)width * r;
      float* P = (part == 0 ? p_mean : part == 1 ? p_ls : part == 2 ? p_q : p_o) + od;
      float* M = (part == 0 ? m_mean : part == 1 ? m_ls : part == 2 ? m_q : m_o) + od;
      float* Vv = (part == 0 ? v_mean : part == 1 ? v_ls : part == 2 ? v_q : v_o) + od;
      const float* G = (part == 0 ? g_mean : part == 1 ? g_ls : part == 2 ? g_q : g_o) + og;
      float pp[4], mm[4], vv[4], gg[4];
      bool idle = true;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const bool on = i < width;
        mm[i] = (on && !cold) ? M[i] : 0.f;
        vv[i] = (on && !cold) ? Vv[i] : 0.f;
        gg[i] = (on && !zero) ? G[i] : 0.f;
        pp[i] = (on && eager) ? P[i] : 0.f;
        idle = idle && gg[i] == 0.f && mm[i] == 0.f && vv[i] == 0.f;
      }
      if (k.skip_idle && idle) continue;
      adam_mark_live(live, d, cold, k);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (i < width) {
          if (!eager) pp[i] = P[i];
          adam_one(pp[i], mm[i], vv[i], gg[i], ss, k);
          P[i] = pp[i]; M[i] = mm[i]; Vv[i] = vv[i];
        }
      }
    }
  }
}

// Gradient rows of a task unit: one warp per row of the union list looks the primitive up in the two views' ascending
// index lists (a 32-way search: three steps for a million rows) and adds the rows it finds.
struct RowsView {
  const float* means; const float* log_scales; const float* quats; const float* opacity_logit; const float* sh;
  const uint8_t* zero; const uint32_t* idx; const uint32_t* count; uint32_t cap;
};

__device__ __forceinline__ int warp_find(const uint32_t* __restrict__ idx, uint32_t n, uint32_t key, unsigned lane) {
  // position of key in the ascending idx[0..n), or -1; all lanes take part and receive the answer
  uint32_t lo = 0, hi = n;  // the key, if present, lies in [lo, hi)
  while (hi - lo > 32) {
    const uint32_t step = (hi - lo + 31) / 32;
    const uint32_t probe = lo + lane * step;
    const bool le = probe < hi && idx[probe] <= key;                // monotone: true for the first cnt lanes
    const uint32_t cnt = __popc(__ballot_sync(0xffffffffu, le));
    if (cnt == 0) return -1;                                        // idx[lo] > key (uniform over the warp)
    lo += (cnt - 1) * step;                                         // idx[lo] <= key < idx[lo + step]
    hi = min(hi, lo + step);
  }
  const uint32_t i = lo + lane;
  const uint32_t hit = __ballot_sync(0xffffffffu, i < hi && idx[i] == key);
  return hit ? (int)(lo + __ffs(hit) - 1) : -1;
}

__global__ void __launch_bounds__(256)
accumulate_rows_kernel(RowsView a, RowsView b, const uint32_t* __restrict__ idx_u, const uint32_t* __restrict__ count_u,
                       uint32_t cap_u, int sh_floats, float* __restrict__ o_means, float* __restrict__ o_ls,
                       float* __restrict__ o_q, float* __restrict__ o_op, float* __restrict__ o_sh) {
  const unsigned lane = threadIdx.x & 31;
  const uint32_t U = min(*count_u, cap_u);
  const uint32_t na = min(*a.count, a.cap), nb = min(*b.count, b.cap);
  for (uint32_t r = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); r < U; r += gridDim.x * (blockDim.x >> 5)) {
    const uint32_t p = idx_u[r];
    int ra = warp_find(a.idx, na, p, lane), rb = warp_find(b.idx, nb, p, lane);
    if (ra >= 0 && a.zero && a.zero[ra]) ra = -1;  // the view flagged the row as zero instead of writing it
    if (rb >= 0 && b.zero && b.zero[rb]) rb = -1;
    auto sum = [&](const float* xa, const float* xb, float* out, int width) {
      for (int i = lane; i < width; i += 32) {
        float s = 0.f;
        if (ra >= 0) s += xa[(size_t)ra * width + i];
        if (rb >= 0) s += xb[(size_t)rb * width + i];
        out[(size_t)r * width + i] = s;
      }
    };
    sum(a.means, b.means, o_means, 3);
    sum(a.log_scales, b.log_scales, o_ls, 3);
    sum(a.quats, b.quats, o_q, 4);
    sum(a.opacity_logit, b.opacity_logit, o_op, 1);
    sum(a.sh, b.sh, o_sh, sh_floats);
  }
}

// live[i / width] = 1 for every non-zero word a[i] (the flags are cleared first; one launch per attribute array)
__global__ void __launch_bounds__(256)
mark_nonzero_kernel(const float* __restrict__ a, size_t total, uint32_t width, uint8_t* __restrict__ live) {
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x)
    if (a[i] != 0.f) live[i / width] = 1;  // (a NaN counts as non-zero)
}

}  // namespace

extern "C" int odin_accumulate_rows(odin_ctx* ctx, const odin_scene* rows_a, const uint8_t* d_zero_a, const uint32_t* d_idx_a,
                                    const uint32_t* d_count_a, const odin_scene* rows_b, const uint8_t* d_zero_b,
                                    const uint32_t* d_idx_b, const uint32_t* d_count_b, const uint32_t* d_idx_u,
                                    const uint32_t* d_count_u, odin_scene* rows_u, void* stream) {
  if (!ctx || !d_count_a || !d_count_b || !d_count_u) return ODIN_ERR_NULL;
  int rc = odin_check_scene(rows_a);
  if (rc == ODIN_OK) rc = odin_check_scene(rows_b);
  if (rc == ODIN_OK) rc = odin_check_scene(rows_u);
  if (rc != ODIN_OK) return rc;
  if (rows_a->sh_degree != rows_u->sh_degree || rows_b->sh_degree != rows_u->sh_degree) return ODIN_ERR_INVALID_ARG;
  if (rows_u->n == 0) return ODIN_OK;
  if (!d_idx_u || (rows_a->n && !d_idx_a) || (rows_b->n && !d_idx_b)) return ODIN_ERR_NULL;
  const RowsView a = {rows_a->means, rows_a->log_scales, rows_a->quats, rows_a->opacity_logit, rows_a->sh, d_zero_a, d_idx_a,
                      d_count_a, rows_a->n};
  const RowsView b = {rows_b->means, rows_b->log_scales, rows_b->quats, rows_b->opacity_logit, rows_b->sh, d_zero_b, d_idx_b,
                      d_count_b, rows_b->n};
  const int K = (rows_u->sh_degree + 1) * (rows_u->sh_degree + 1);
  uint32_t grid = (rows_u->n + 7) / 8;
  if (grid > (uint32_t)ctx->sm_count * 16) grid = (uint32_t)ctx->sm_count * 16;
  OdinKernelScope ks(ctx, K_ACCUMULATE, (cudaStream_t)stream);
  accumulate_rows_kernel<<<grid, 256, 0, (cudaStream_t)stream>>>(a, b, d_idx_u, d_count_u, rows_u->n, 3 * K, rows_u->means,
                                                                rows_u->log_scales, rows_u->quats, rows_u->opacity_logit,
                                                                rows_u->sh);
  return odin_launch_status();
}

extern "C" int odin_adam_live_refresh(odin_ctx* ctx, const odin_scene* m, const odin_scene* v, uint8_t* d_live,
                                     void* stream) {
  if (!ctx || !d_live) return ODIN_ERR_NULL;
  int rc = odin_check_scene(m);
  if (rc == ODIN_OK) rc = odin_check_scene(v);
  if (rc != ODIN_OK) return rc;
  if (m->n != v->n || m->sh_degree != v->sh_degree) return ODIN_ERR_INVALID_ARG;
  if (m->n == 0) return ODIN_OK;
  cudaStream_t st = (cudaStream_t)stream;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(d_live, 0, m->n, st));
  const int K = (m->sh_degree + 1) * (m->sh_degree + 1);
  for (const odin_scene* s : {m, v}) {
    const float* arrays[5] = {s->means, s->log_scales, s->quats, s->opacity_logit, s->sh};
    const uint32_t widths[5] = {3, 3, 4, 1, (uint32_t)(3 * K)};
    for (int a = 0; a < 5; ++a) {
      const size_t total = (size_t)m->n * widths[a];
      size_t blocks = (total + 255) / 256;
      if (blocks > (size_t)ctx->sm_count * 16) blocks = (size_t)ctx->sm_count * 16;
      OdinKernelScope ks(ctx, K_ADAM_LIVE, st);
      mark_nonzero_kernel<<<(unsigned)blocks, 256, 0, st>>>(arrays[a], total, widths[a], d_live);
    }
  }
  return odin_launch_status();
}

extern "C" int odin_sparse_adam(odin_ctx* ctx, odin_scene* params, odin_scene* m, odin_scene* v,
                                const odin_scene* grad_rows, const uint8_t* d_row_zero, const uint32_t* d_idx,
                                const uint32_t* d_count, const float lr[6], float beta1, float beta2, float eps,
                                uint32_t step, void* stream) {
  return odin_sparse_adam_live(ctx, params, m, v, grad_rows, d_row_zero, d_idx, d_count, nullptr, lr, beta1, beta2, eps, step,
                               stream);
}

extern "C" int odin_sparse_adam_live(odin_ctx* ctx, odin_scene* params, odin_scene* m, odin_scene* v,
                                     const odin_scene* grad_rows, const uint8_t* d_row_zero, const uint32_t* d_idx,
                                     const uint32_t* d_count, uint8_t* d_live, const float lr[6], float beta1, float beta2,
                                     float eps, uint32_t step, void* stream) {
  if (!ctx || !lr || !d_count) return ODIN_ERR_NULL;
  int rc = odin_check_scene(params);
  if (rc == ODIN_OK) rc = odin_check_scene(m);
  if (rc == ODIN_OK) rc = odin_check_scene(v);
  if (rc == ODIN_OK) rc = odin_check_scene(grad_rows);
  if (rc != ODIN_OK) return rc;
  if (m->n != params->n || v->n != params->n || m->sh_degree != params->sh_degree || v->sh_degree != params->sh_degree ||
      grad_rows->sh_degree != params->sh_degree)
    return ODIN_ERR_INVALID_ARG;
  if (step == 0 || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps >= 0.f))
    return ODIN_ERR_INVALID_ARG;
  if (params->n == 0 || grad_rows->n == 0) return ODIN_OK;
  if (!d_idx) return ODIN_ERR_NULL;
  AdamK k;
  k.beta1 = beta1; k.beta2 = beta2; k.omb1 = 1.f - beta1; k.omb2 = 1.f - beta2; k.eps = eps;
  k.skip_idle = eps > 0.f ? 1 : 0;
  const float bc1 = 1.f - (float)pow((double)beta1, (double)step);
  const float bc2s = (float)sqrt(1.0 - pow((double)beta2, (double)step));
  for (int i = 0; i < 6; ++i) k.step_size[i] = lr[i] / bc1;
  k.inv_bc2s = 1.f / bc2s;
  cudaStream_t st = (cudaStream_t)stream;
  const uint32_t cap = grad_rows->n;
  const int K = (params->sh_degree + 1) * (params->sh_degree + 1);
  // a warp per 32 rows of the list
  size_t blocks = ((size_t)cap + 32 * ADAM_WARPS - 1) / (32 * ADAM_WARPS);
  if (blocks > (size_t)ctx->sm_count * 16) blocks = (size_t)ctx->sm_count * 16;
  const unsigned gsh = (unsigned)blocks;
  {
    OdinKernelScope ks(ctx, K_ADAM_SH, st);
    switch (params->sh_degree) {
    case 0: ODIN_CUDA(odin_launch(ctx, false, adam_sh_kernel<3, 1>, dim3(gsh), dim3(ADAM_WARPS * 32), 0, st, params->sh, m->sh, v->sh, grad_rows->sh, d_idx, d_count, cap, k, d_row_zero, params->n, d_live)); break;
    case 1: ODIN_CUDA(odin_launch(ctx, false, adam_sh_kernel<12, 4>, dim3(gsh), dim3(ADAM_WARPS * 32), 0, st, params->sh, m->sh, v->sh, grad_rows->sh, d_idx, d_count, cap, k, d_row_zero, params->n, d_live)); break;
    case 2: ODIN_CUDA(odin_launch(ctx, false, adam_sh_kernel<27, 1>, dim3(gsh), dim3(ADAM_WARPS * 32), 0, st, params->sh, m->sh, v->sh, grad_rows->sh, d_idx, d_count, cap, k, d_row_zero, params->n, d_live)); break;
    default: ODIN_CUDA(odin_launch(ctx, false, adam_sh_kernel<48, 4>, dim3(gsh), dim3(ADAM_WARPS * 32), 0, st, params->sh, m->sh, v->sh, grad_rows->sh, d_idx, d_count, cap, k, d_row_zero, params->n, d_live)); break;
    }
  }
  OdinKernelScope ks(ctx, K_ADAM_GEOM, st);
  ODIN_CUDA(odin_launch(ctx, true, adam_geom_kernel, dim3(gsh), dim3(ADAM_WARPS * 32), 0, st,
      params->means, params->log_scales, params->quats, params->opacity_logit, m->means, m->log_scales, m->quats,
      m->opacity_logit, v->means, v->log_scales, v->quats, v->opacity_logit, (const float*)grad_rows->means,
      (const float*)grad_rows->log_scales, (const float*)grad_rows->quats, (const float*)grad_rows->opacity_logit, d_idx,
      d_count, cap, k, d_row_zero, params->n, d_live));
  return odin_launch_status();
}
