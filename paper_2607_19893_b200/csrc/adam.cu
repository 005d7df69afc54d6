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

// SH block: ROWF floats per row (3, 12, 27 or 48), processed as VEC-wide elements; element e of the compact
// gradient block belongs to row e / (ROWF / VEC).
template <int ROWF, int VEC>
__global__ void __launch_bounds__(256)
adam_sh_kernel(float* __restrict__ p, float* __restrict__ m, float* __restrict__ v, const float* __restrict__ g,
               const uint32_t* __restrict__ idx, const uint32_t* __restrict__ count, uint32_t cap, AdamK k,
               const uint8_t* __restrict__ row_zero, uint32_t n_prims) {
  odin_after_predecessor();
  constexpr int EPR = ROWF / VEC;  // elements per row
  const uint32_t V = min(*count, cap);
  const size_t total = (size_t)V * EPR;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const uint32_t r = (uint32_t)(e / EPR);
    const uint32_t j = (uint32_t)(e - (size_t)r * EPR);
    const uint32_t prim = idx[r];
    if (prim >= n_prims) continue;  // an index list that is not a view's own (e.g. after a timed-out scan): no write
    const size_t dst = (size_t)prim * ROWF + (size_t)j * VEC;
    const bool zero = row_zero && row_zero[r];  // the gradient row was not written: it is zero
    if (VEC == 4) {
      const float4 gg = zero ? make_float4(0.f, 0.f, 0.f, 0.f) : reinterpret_cast<const float4*>(g)[e];
      float4 mm = *reinterpret_cast<float4*>(m + dst), vv = *reinterpret_cast<float4*>(v + dst);
      if (k.skip_idle && gg.x == 0.f && gg.y == 0.f && gg.z == 0.f && gg.w == 0.f && mm.x == 0.f && mm.y == 0.f &&
          mm.z == 0.f && mm.w == 0.f && vv.x == 0.f && vv.y == 0.f && vv.z == 0.f && vv.w == 0.f)
        continue;
      float4 pp = *reinterpret_cast<float4*>(p + dst);
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
      float mm = m[dst], vv = v[dst];
      const float gg = zero ? 0.f : g[e];
      if (k.skip_idle && gg == 0.f && mm == 0.f && vv == 0.f) continue;
      float pp = p[dst];
      adam_one(pp, mm, vv, gg, k.step_size[j < 3 ? 4 : 5], k);
      p[dst] = pp; m[dst] = mm; v[dst] = vv;
    }
  }
}

// Geometry block: four threads per row - mean(3), log scale(3), quaternion(4), opacity(1) - so that a row's twelve
// gathers are spread over four independent threads instead of queueing in one.
__global__ void __launch_bounds__(256)
adam_geom_kernel(float* __restrict__ p_mean, float* __restrict__ p_ls, float4* __restrict__ p_q, float* __restrict__ p_o,
                 float* __restrict__ m_mean, float* __restrict__ m_ls, float4* __restrict__ m_q, float* __restrict__ m_o,
                 float* __restrict__ v_mean, float* __restrict__ v_ls, float4* __restrict__ v_q, float* __restrict__ v_o,
                 const float* __restrict__ g_mean, const float* __restrict__ g_ls, const float4* __restrict__ g_q,
                 const float* __restrict__ g_o, const uint32_t* __restrict__ idx, const uint32_t* __restrict__ count,
                 uint32_t cap, AdamK k, const uint8_t* __restrict__ row_zero, uint32_t n_prims) {
  odin_after_predecessor();  // launched behind the SH kernel (which it does not depend on: the two overlap at the seam)
  const uint32_t V = min(*count, cap);
  const size_t total = (size_t)V * 4;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const uint32_t r = (uint32_t)(e >> 2);
    const int part = (int)(e & 3);
    const size_t d = idx[r];
    if (d >= n_prims) continue;
    const bool zero = row_zero && row_zero[r];  // the gradient row was not written: it is zero
    if (part < 2) {
      float* __restrict__ p = (part ? p_ls : p_mean) + 3 * d;
      float* __restrict__ m = (part ? m_ls : m_mean) + 3 * d;
      float* __restrict__ v = (part ? v_ls : v_mean) + 3 * d;
      const float* __restrict__ g = (part ? g_ls : g_mean) + 3 * (size_t)r;
      const float ss = k.step_size[part];
      float pp[3], mm[3], vv[3], gg[3];
#pragma unroll
      for (int i = 0; i < 3; ++i) { mm[i] = m[i]; vv[i] = v[i]; gg[i] = zero ? 0.f : g[i]; }
      if (k.skip_idle && gg[0] == 0.f && gg[1] == 0.f && gg[2] == 0.f && mm[0] == 0.f && mm[1] == 0.f && mm[2] == 0.f &&
          vv[0] == 0.f && vv[1] == 0.f && vv[2] == 0.f)
        continue;
#pragma unroll
      for (int i = 0; i < 3; ++i) pp[i] = p[i];
#pragma unroll
      for (int i = 0; i < 3; ++i) adam_one(pp[i], mm[i], vv[i], gg[i], ss, k);
#pragma unroll
      for (int i = 0; i < 3; ++i) { p[i] = pp[i]; m[i] = mm[i]; v[i] = vv[i]; }
    } else if (part == 2) {
      float4 mm = m_q[d], vv = v_q[d];
      const float4 gg = zero ? make_float4(0.f, 0.f, 0.f, 0.f) : g_q[r];
      if (k.skip_idle && gg.x == 0.f && gg.y == 0.f && gg.z == 0.f && gg.w == 0.f && mm.x == 0.f && mm.y == 0.f &&
          mm.z == 0.f && mm.w == 0.f && vv.x == 0.f && vv.y == 0.f && vv.z == 0.f && vv.w == 0.f)
        continue;
      float4 pp = p_q[d];
      adam_one(pp.x, mm.x, vv.x, gg.x, k.step_size[2], k);
      adam_one(pp.y, mm.y, vv.y, gg.y, k.step_size[2], k);
      adam_one(pp.z, mm.z, vv.z, gg.z, k.step_size[2], k);
      adam_one(pp.w, mm.w, vv.w, gg.w, k.step_size[2], k);
      p_q[d] = pp; m_q[d] = mm; v_q[d] = vv;
    } else {
      float mm = m_o[d], vv = v_o[d];
      const float gg = zero ? 0.f : g_o[r];
      if (k.skip_idle && gg == 0.f && mm == 0.f && vv == 0.f) continue;
      float pp = p_o[d];
      adam_one(pp, mm, vv, gg, k.step_size[3], k);
      p_o[d] = pp; m_o[d] = mm; v_o[d] = vv;
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

extern "C" int odin_sparse_adam(odin_ctx* ctx, odin_scene* params, odin_scene* m, odin_scene* v,
                                const odin_scene* grad_rows, const uint8_t* d_row_zero, const uint32_t* d_idx,
                                const uint32_t* d_count, const float lr[6], float beta1, float beta2, float eps,
                                uint32_t step, void* stream) {
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
  const size_t max_elems = (size_t)cap * (K == 9 ? 27 : (K == 1 ? 3 : 3 * K / 4));
  size_t blocks = (max_elems + 255) / 256;
  if (blocks > (size_t)ctx->sm_count * 16) blocks = (size_t)ctx->sm_count * 16;
  const unsigned gsh = (unsigned)blocks;
  {
    OdinKernelScope ks(ctx, K_ADAM_SH, st);
    switch (params->sh_degree) {
    case 0: ODIN_CUDA(odin_launch(ctx, false, adam_sh_kernel<3, 1>, dim3(gsh), dim3(256), 0, st, params->sh, m->sh, v->sh, grad_rows->sh, d_idx, d_count, cap, k, d_row_zero, params->n)); break;
    case 1: ODIN_CUDA(odin_launch(ctx, false, adam_sh_kernel<12, 4>, dim3(gsh), dim3(256), 0, st, params->sh, m->sh, v->sh, grad_rows->sh, d_idx, d_count, cap, k, d_row_zero, params->n)); break;
    case 2: ODIN_CUDA(odin_launch(ctx, false, adam_sh_kernel<27, 1>, dim3(gsh), dim3(256), 0, st, params->sh, m->sh, v->sh, grad_rows->sh, d_idx, d_count, cap, k, d_row_zero, params->n)); break;
    default: ODIN_CUDA(odin_launch(ctx, false, adam_sh_kernel<48, 4>, dim3(gsh), dim3(256), 0, st, params->sh, m->sh, v->sh, grad_rows->sh, d_idx, d_count, cap, k, d_row_zero, params->n)); break;
    }
  }
  size_t gb = ((size_t)cap * 4 + 255) / 256;
  if (gb > (size_t)ctx->sm_count * 16) gb = (size_t)ctx->sm_count * 16;
  OdinKernelScope ks(ctx, K_ADAM_GEOM, st);
  ODIN_CUDA(odin_launch(ctx, true, adam_geom_kernel, dim3((unsigned)gb), dim3(256), 0, st,
      params->means, params->log_scales, reinterpret_cast<float4*>(params->quats), params->opacity_logit, m->means,
      m->log_scales, reinterpret_cast<float4*>(m->quats), m->opacity_logit, v->means, v->log_scales,
      reinterpret_cast<float4*>(v->quats), v->opacity_logit, grad_rows->means, grad_rows->log_scales,
      reinterpret_cast<const float4*>(grad_rows->quats), grad_rows->opacity_logit, d_idx, d_count, cap, k, d_row_zero,
      params->n));
  return odin_launch_status();
}
