// Realized scope, gradient evidence and the admission arithmetic that the paper's runtime evaluates on primitive-index
// sets (Sec. 2.1 Table 1: C_i, g_U(p); Sec. 4.3: the three hazards, the delayed-read set and the gradient gate).
// Everything here streams over bitmasks or compact row lists; all of it is bandwidth-bound.
#include "common.cuh"
#include "layout.cuh"

namespace {

// ------------------------------------------------------------------------------------------------ active set
constexpr int AS_THREADS = 256;
constexpr int AS_ITEMS = 8;
constexpr uint32_t AS_TILE = AS_THREADS * AS_ITEMS;  // rows per look-back tile

struct GradRows {  // compact gradient rows in the layout of odin_scene
  const float* means;
  const float* log_scales;
  const float* quats;
  const float* opacity_logit;
  const float* sh;
  int sh_floats;  // 3 (sh_degree + 1)^2
};

// Compacts the rows flagged by the backward pass: ascending primitive ids, their evidence, the bitmask over primitive
// ids, the count and the evidence sum.  One tile of 2048 rows per block, blocks ordered by ticket, one decoupled
// look-back per block.
__global__ void __launch_bounds__(AS_THREADS)
active_set_kernel(const uint8_t* __restrict__ row_active, const uint32_t* __restrict__ prim_id,
                  const uint32_t* __restrict__ num_rows, uint32_t row_capacity, const float* __restrict__ grad2d,
                  GradRows rows, int evidence_mode, uint32_t* __restrict__ mask, uint32_t* __restrict__ idx,
                  uint32_t idx_capacity, uint32_t* __restrict__ count, float* __restrict__ evidence,
                  double* __restrict__ evidence_sum, uint32_t* ticket, uint64_t* state, int* status, int spin_limit,
                  uint32_t n_prims) {
  __shared__ uint32_t s_tile, s_base;
  __shared__ uint32_t s_warp[33];
  __shared__ double s_sum[AS_THREADS / 32];
  const uint32_t V = min(*num_rows, row_capacity);
  const uint32_t ntiles = (V + AS_TILE - 1) / AS_TILE;
  if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  if (tile >= ntiles) return;  // uniform over the block
  const uint32_t first = tile * AS_TILE + threadIdx.x * AS_ITEMS;
  uint32_t flags = 0, mine = 0;
#pragma unroll
  for (int k = 0; k < AS_ITEMS; ++k)
    if (first + k < V && row_active[first + k]) { flags |= 1u << k; ++mine; }
  uint32_t total;
  const uint32_t before = odin_block_exclusive_sum(mine, s_warp, &total);
  if (threadIdx.x < 32) {
    const uint64_t b = odin_lookback_u64(state, tile, (uint64_t)total, status, spin_limit);
    if (threadIdx.x == 0) {
      s_base = (uint32_t)b;
      if (tile == ntiles - 1) {  // last tile: totals
        const uint64_t all = b + total;
        *count = (uint32_t)(all < idx_capacity ? all : idx_capacity);
        if (all > idx_capacity) odin_set_error(status, ODIN_ERR_CAPACITY);
      }
    }
  }
  __syncthreads();
  uint32_t pos = s_base + before;
  double local = 0.0;
#pragma unroll
  for (int k = 0; k < AS_ITEMS; ++k) {
    if (!(flags >> k & 1u)) continue;
    const uint32_t r = first + k;
    const uint32_t p = prim_id[r];
    if (p >= n_prims) { ++pos; continue; }  // a row map that is not this view's own (e.g. after a timed-out scan)
    float ev;
    if (evidence_mode == 0) {
      const float gu = grad2d[(size_t)r * 9], gv = grad2d[(size_t)r * 9 + 1];
      ev = sqrtf(gu * gu + gv * gv);
    } else {
      float acc = 0.f;
      for (int c = 0; c < 3; ++c) {
        const float a = rows.means[(size_t)r * 3 + c], b = rows.log_scales[(size_t)r * 3 + c];
        acc = fmaf(a, a, acc); acc = fmaf(b, b, acc);
      }
      for (int c = 0; c < 4; ++c) { const float a = rows.quats[(size_t)r * 4 + c]; acc = fmaf(a, a, acc); }
      { const float a = rows.opacity_logit[r]; acc = fmaf(a, a, acc); }
      for (int c = 0; c < rows.sh_floats; ++c) {
        const float a = rows.sh[(size_t)r * rows.sh_floats + c];
        acc = fmaf(a, a, acc);
      }
      ev = sqrtf(acc);
    }
    atomicOr(&mask[p >> 5], 1u << (p & 31));
    if (pos < idx_capacity) {
      idx[pos] = p;
      evidence[pos] = ev;
      local += (double)ev;  // the sum covers exactly the listed primitives
    }
    ++pos;
  }
  for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
  if ((threadIdx.x & 31) == 0) s_sum[threadIdx.x >> 5] = local;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0.0;
    for (int i = 0; i < AS_THREADS / 32; ++i) t += s_sum[i];
    if (t != 0.0) atomicAdd(evidence_sum, t);
  }
}

// ------------------------------------------------------------------------------------------------ unions
__global__ void __launch_bounds__(256)
mask_union_kernel(const uint32_t* __restrict__ masks, uint32_t stride_words, uint32_t words, uint32_t n_masks,
                  const uint32_t* __restrict__ members, uint32_t n_members, uint32_t* __restrict__ out, int* status) {
  for (uint32_t w = blockIdx.x * blockDim.x + threadIdx.x; w < stride_words; w += gridDim.x * blockDim.x) {
    uint32_t acc = 0;
    if (w < words)
      for (uint32_t k = 0; k < n_members; ++k) {
        const uint32_t m = members[k];
        if (m < n_masks) acc |= masks[(size_t)m * stride_words + w];
        else if (w == 0) odin_set_error(status, ODIN_ERR_INVALID_ARG);
      }
    out[w] = acc;
  }
}

// ------------------------------------------------------------------------------------------------ hazards
constexpr int HZ_THREADS = 256;

__device__ __forceinline__ void block_add4(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                           unsigned long long* __restrict__ dst) {
  __shared__ uint32_t s[4][HZ_THREADS / 32];
  uint32_t c[4] = {c0, c1, c2, c3};
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    for (int o = 16; o > 0; o >>= 1) c[q] += __shfl_xor_sync(0xffffffffu, c[q], o);
    if ((threadIdx.x & 31) == 0) s[q][threadIdx.x >> 5] = c[q];
  }
  __syncthreads();
  if (threadIdx.x < 4) {
    uint32_t tot = 0;
    for (int i = 0; i < HZ_THREADS / 32; ++i) tot += s[threadIdx.x][i];
    if (tot) atomicAdd(&dst[threadIdx.x], (unsigned long long)tot);
  }
}

// One block column per pair (blockIdx.y); WAW, RAW, WAR and |R(B)| from one pass over the four masks of the pair.
__global__ void __launch_bounds__(HZ_THREADS)
hazard_count_kernel(const uint32_t* __restrict__ read_masks, const uint32_t* __restrict__ write_masks,
                    uint32_t stride_words, uint32_t words, const uint32_t* __restrict__ pairs, uint32_t n_masks,
                    unsigned long long* __restrict__ counts, int* status) {
  const uint32_t pair = blockIdx.y;
  const uint32_t ua = pairs[2 * pair], ub = pairs[2 * pair + 1];
  if (ua >= n_masks || ub >= n_masks) {  // uniform over the block: a pair naming a missing unit counts 0
    if (threadIdx.x == 0) odin_set_error(status, ODIN_ERR_INVALID_ARG);
    return;
  }
  const uint32_t* ra = read_masks + (size_t)ua * stride_words;
  const uint32_t* wa = write_masks + (size_t)ua * stride_words;
  const uint32_t* rb = read_masks + (size_t)ub * stride_words;
  const uint32_t* wb = write_masks + (size_t)ub * stride_words;
  uint32_t waw = 0, raw = 0, war = 0, nrb = 0;
  for (uint32_t i = blockIdx.x * HZ_THREADS + threadIdx.x; i < words; i += gridDim.x * HZ_THREADS) {
    const uint32_t a_r = ra[i], a_w = wa[i], b_r = rb[i], b_w = wb[i];
    waw += __popc(b_w & a_w);
    raw += __popc((b_r & ~b_w) & a_w);
    war += __popc(b_w & (a_r & ~a_w));
    nrb += __popc(b_r);
  }
  block_add4(waw, raw, war, nrb, counts + 4 * (size_t)pair);
}

// Delayed-read gate: #D+ and #R+(B) from the masks; #(D+ & C_A) and the number passing the gradient gate from A's
// active list (k -> primitive, evidence).
__global__ void __launch_bounds__(HZ_THREADS)
delayed_read_gate_kernel(const uint32_t* __restrict__ read_b, const uint32_t* __restrict__ write_b,
                         const uint32_t* __restrict__ write_a, uint32_t words, const uint32_t* __restrict__ active_idx,
                         const float* __restrict__ evidence, const uint32_t* __restrict__ active_count,
                         const double* __restrict__ evidence_sum, uint32_t active_capacity, uint32_t n_prims, float tau,
                         unsigned long long* __restrict__ gate) {
  uint32_t n_delayed = 0, n_with = 0, n_pass = 0, nrb = 0;
  const uint32_t stride = gridDim.x * HZ_THREADS, t0 = blockIdx.x * HZ_THREADS + threadIdx.x;
  for (uint32_t i = t0; i < words; i += stride) {
    const uint32_t b_r = read_b[i];
    n_delayed += __popc((b_r & ~write_b[i]) & write_a[i]);
    nrb += __popc(b_r);
  }
  const uint32_t ca = min(*active_count, active_capacity);
  const double threshold = ca ? (double)tau * (*evidence_sum / (double)ca) : 0.0;
  for (uint32_t k = t0; k < ca; k += stride) {
    const uint32_t p = active_idx[k];
    if (p >= n_prims) continue;
    const uint32_t w = p >> 5;
    if (((read_b[w] & ~write_b[w]) & write_a[w]) >> (p & 31) & 1u) {
      ++n_with;
      if ((double)evidence[k] <= threshold) ++n_pass;
    }
  }
  block_add4(n_delayed, n_with, n_pass, nrb, gate);
}

// ------------------------------------------------------------------------------------------------ locality graph
// Eq. (1) on per-view primitive sets: one float32 division per pair.
__global__ void rlg_weights_kernel(const unsigned long long* __restrict__ counts, const uint32_t* __restrict__ sizes,
                                   const uint32_t* __restrict__ pairs, uint32_t n_pairs, uint32_t n_views,
                                   float* __restrict__ weights, int* status) {
  for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n_pairs; i += gridDim.x * blockDim.x) {
    const uint32_t a = pairs[2 * i], b = pairs[2 * i + 1];
    float w = 0.f;
    if (a < n_views && b < n_views) {
      const unsigned long long inter = counts[i];
      const unsigned long long uni = (unsigned long long)sizes[a] + sizes[b] - inter;
      if (uni > 0) w = (float)inter / (float)uni;
    } else {
      odin_set_error(status, ODIN_ERR_INVALID_ARG);
    }
    weights[i] = w;
  }
}

// Neighbour retention.  keep[i][j] = 1 when j is among the k strongest neighbours of i (larger weight first, lower index
// first among equals, zero weights are not edges).  One block per item i, thread j ranks w_ij by counting who beats it.
__global__ void rlg_rank_kernel(const float* __restrict__ w, uint32_t n, uint32_t k, uint8_t* __restrict__ keep) {
  const uint32_t i = blockIdx.x;
  for (uint32_t j = threadIdx.x; j < n; j += blockDim.x) {
    const float x = (j == i) ? 0.f : w[(size_t)i * n + j];
    uint32_t rank = 0;
    if (x > 0.f)
      for (uint32_t q = 0; q < n; ++q) {
        if (q == i) continue;
        const float y = w[(size_t)i * n + q];
        rank += (y > x || (y == x && q < j)) ? 1u : 0u;
      }
    keep[(size_t)i * n + j] = (x > 0.f && rank < k) ? 1 : 0;
  }
}

// The graph is undirected: an edge stays when either end keeps it; dropped edges and the diagonal read as 0.
__global__ void rlg_retain_kernel(const float* __restrict__ w, const uint8_t* __restrict__ keep, uint32_t n,
                                  float* __restrict__ out) {
  const size_t total = (size_t)n * n;
  for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.x * blockDim.x) {
    const uint32_t i = (uint32_t)(e / n), j = (uint32_t)(e % n);
    out[e] = (i != j && (keep[e] || keep[(size_t)j * n + i])) ? w[e] : 0.f;
  }
}

// Eq. (2): one block per candidate v, threads stride over the previous unit.
__global__ void __launch_bounds__(128)
sds_scores_kernel(const float* __restrict__ w, uint32_t n, const uint32_t* __restrict__ prev, uint32_t n_prev,
                  const uint32_t* __restrict__ cand, float* __restrict__ scores, int* status) {
  __shared__ float s[4];
  const uint32_t v = cand[blockIdx.x];
  float acc = 0.f;
  if (v < n) {
    for (uint32_t q = threadIdx.x; q < n_prev; q += 128) {
      const uint32_t u = prev[q];
      if (u < n) acc += w[(size_t)u * n + v];
      else odin_set_error(status, ODIN_ERR_INVALID_ARG);
    }
  } else if (threadIdx.x == 0) {
    odin_set_error(status, ODIN_ERR_INVALID_ARG);
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) scores[blockIdx.x] = s[0] + s[1] + s[2] + s[3];
}

}  // namespace

extern "C" int odin_rlg_weights(odin_ctx* ctx, const uint64_t* d_counts, const uint32_t* d_sizes, const uint32_t* d_pairs,
                                uint32_t n_pairs, uint32_t n_views, float* d_weights, void* stream) {
  if (!ctx) return ODIN_ERR_NULL;
  if (n_pairs == 0) return ODIN_OK;
  if (!d_counts || !d_sizes || !d_pairs || !d_weights) return ODIN_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t grid = (n_pairs + 255) / 256;
  if (grid > (uint32_t)ctx->sm_count * 8) grid = (uint32_t)ctx->sm_count * 8;
  OdinKernelScope ks(ctx, K_RLG, st);
  rlg_weights_kernel<<<grid, 256, 0, st>>>(reinterpret_cast<const unsigned long long*>(d_counts), d_sizes, d_pairs,
                                          n_pairs, n_views, d_weights, ctx->d_status);
  return odin_launch_status();
}

extern "C" int odin_rlg_topk(odin_ctx* ctx, const float* d_weights, uint32_t n_views, uint32_t k, float* d_retained,
                             void* ws, size_t ws_bytes, void* stream) {
  if (!ctx) return ODIN_ERR_NULL;
  if (n_views == 0) return ODIN_OK;
  if (n_views > 32768) return ODIN_ERR_INVALID_ARG;
  if (!d_weights || !d_retained) return ODIN_ERR_NULL;
  if (d_weights == d_retained) return ODIN_ERR_INVALID_ARG;
  const size_t need = (size_t)n_views * n_views;
  if (!ws || ws_bytes < need) return ODIN_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  uint8_t* keep = reinterpret_cast<uint8_t*>(ws);
  {
    OdinKernelScope ks(ctx, K_RLG, st);
    rlg_rank_kernel<<<n_views, 128, 0, st>>>(d_weights, n_views, k, keep);
  }
  size_t grid = (need + 255) / 256;
  if (grid > (size_t)ctx->sm_count * 8) grid = (size_t)ctx->sm_count * 8;
  OdinKernelScope ks(ctx, K_RLG, st);
  rlg_retain_kernel<<<(unsigned)grid, 256, 0, st>>>(d_weights, keep, n_views, d_retained);
  return odin_launch_status();
}

extern "C" int odin_sds_scores(odin_ctx* ctx, const float* d_weights, uint32_t n_views, const uint32_t* d_prev_unit,
                               uint32_t n_prev, const uint32_t* d_candidates, uint32_t n_candidates, float* d_scores,
                               void* stream) {
  if (!ctx) return ODIN_ERR_NULL;
  if (n_candidates == 0) return ODIN_OK;
  if (!d_weights || !d_candidates || !d_scores || (n_prev > 0 && !d_prev_unit)) return ODIN_ERR_NULL;
  if (n_views == 0) return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  OdinKernelScope ks(ctx, K_RLG, st);
  sds_scores_kernel<<<n_candidates, 128, 0, st>>>(d_weights, n_views, d_prev_unit, n_prev, d_candidates, d_scores,
                                                 ctx->d_status);
  return odin_launch_status();
}

extern "C" int odin_active_set(odin_ctx* ctx, const odin_projected* proj, const uint8_t* d_row_active,
                               const float* d_grad2d, const odin_scene* grad_rows, int evidence_mode, uint32_t n,
                               uint32_t* d_mask, uint32_t* d_idx, uint32_t idx_capacity, uint32_t* d_count,
                               float* d_evidence, double* d_evidence_sum, void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || !proj || !d_count || !d_evidence_sum) return ODIN_ERR_NULL;
  if (evidence_mode != 0 && evidence_mode != 1) return ODIN_ERR_INVALID_ARG;
  if (n >= (1u << 28)) return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(d_count, 0, 4, st));
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(d_evidence_sum, 0, 8, st));
  const uint32_t words = (n + 31) / 32;
  if (words) {
    if (!d_mask) return ODIN_ERR_NULL;
    odin_chain_break(ctx);
    ODIN_CUDA(cudaMemsetAsync(d_mask, 0, (size_t)words * 4, st));
  }
  if (proj->capacity == 0 || n == 0) return ODIN_OK;
  if (!d_row_active || !proj->prim_id || !proj->num_rows || (idx_capacity > 0 && (!d_idx || !d_evidence)))
    return ODIN_ERR_NULL;
  GradRows rows = {};
  if (evidence_mode == 0) {
    if (!d_grad2d) return ODIN_ERR_NULL;
  } else {
    const int rc = odin_check_scene(grad_rows);
    if (rc != ODIN_OK) return rc;
    if (grad_rows->n < proj->capacity) return ODIN_ERR_INVALID_ARG;
    rows.means = grad_rows->means; rows.log_scales = grad_rows->log_scales; rows.quats = grad_rows->quats;
    rows.opacity_logit = grad_rows->opacity_logit; rows.sh = grad_rows->sh;
    rows.sh_floats = 3 * (grad_rows->sh_degree + 1) * (grad_rows->sh_degree + 1);
  }
  const uint32_t tiles = (proj->capacity + AS_TILE - 1) / AS_TILE;
  const size_t need = 256 + ws_align((size_t)tiles * 8);
  if (!ws || !odin_aligned(ws, 256) || ws_bytes < need) return ODIN_ERR_WORKSPACE;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(ws, 0, need, st));
  uint32_t* ticket = reinterpret_cast<uint32_t*>(ws);
  uint64_t* state = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(ws) + 256);
  OdinKernelScope ks(ctx, K_ACTIVE_SET, st);
  active_set_kernel<<<tiles, AS_THREADS, 0, st>>>(d_row_active, proj->prim_id, proj->num_rows, proj->capacity, d_grad2d,
                                                 rows, evidence_mode, d_mask, d_idx, idx_capacity, d_count, d_evidence,
                                                 d_evidence_sum, ticket, state, ctx->d_status, ctx->spin_limit, n);
  return odin_launch_status();
}

static int check_masks(const void* p, uint32_t n_masks, uint32_t stride_words, uint32_t words) {
  if (!p) return ODIN_ERR_NULL;
  if (n_masks == 0 || stride_words < words) return ODIN_ERR_INVALID_ARG;
  return ODIN_OK;
}

extern "C" int odin_mask_union(odin_ctx* ctx, const uint32_t* d_masks, uint32_t n_masks, uint32_t mask_stride_words,
                               uint32_t n_prims, const uint32_t* d_members, uint32_t n_members, uint32_t* d_out,
                               void* stream) {
  if (!ctx) return ODIN_ERR_NULL;
  const uint32_t words = (n_prims + 31) / 32;
  if (mask_stride_words == 0) return ODIN_OK;
  if (!d_out) return ODIN_ERR_NULL;
  if (n_members) {
    const int rc = check_masks(d_masks, n_masks, mask_stride_words, words);
    if (rc != ODIN_OK) return rc;
    if (!d_members) return ODIN_ERR_NULL;
  }
  cudaStream_t st = (cudaStream_t)stream;
  uint32_t grid = (mask_stride_words + 255) / 256;
  if (grid > (uint32_t)ctx->sm_count * 8) grid = (uint32_t)ctx->sm_count * 8;
  OdinKernelScope ks(ctx, K_MASK_UNION, st);
  mask_union_kernel<<<grid, 256, 0, st>>>(d_masks, mask_stride_words, words, n_masks, d_members, n_members, d_out,
                                         ctx->d_status);
  return odin_launch_status();
}

extern "C" int odin_hazard_count(odin_ctx* ctx, const uint32_t* d_read_masks, const uint32_t* d_write_masks,
                                 uint32_t n_masks, uint32_t mask_stride_words, uint32_t n_prims, const uint32_t* d_pairs,
                                 uint32_t n_pairs, uint64_t* d_counts, void* stream) {
  if (!ctx) return ODIN_ERR_NULL;
  if (n_pairs == 0) return ODIN_OK;
  if (!d_pairs || !d_counts) return ODIN_ERR_NULL;
  if (n_pairs > 65535) return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(d_counts, 0, (size_t)n_pairs * 32, st));
  const uint32_t words = (n_prims + 31) / 32;
  if (words == 0) return ODIN_OK;
  int rc = check_masks(d_read_masks, n_masks, mask_stride_words, words);
  if (rc == ODIN_OK) rc = check_masks(d_write_masks, n_masks, mask_stride_words, words);
  if (rc != ODIN_OK) return rc;
  uint32_t gx = (words + HZ_THREADS - 1) / HZ_THREADS;
  const uint32_t cap = (uint32_t)(ctx->sm_count * 8 + n_pairs - 1) / n_pairs;
  if (gx > cap) gx = cap;
  if (gx == 0) gx = 1;
  OdinKernelScope ks(ctx, K_HAZARD, st);
  hazard_count_kernel<<<dim3(gx, n_pairs), HZ_THREADS, 0, st>>>(d_read_masks, d_write_masks, mask_stride_words, words,
                                                               d_pairs, n_masks,
                                                               reinterpret_cast<unsigned long long*>(d_counts),
                                                               ctx->d_status);
  return odin_launch_status();
}

extern "C" int odin_delayed_read_gate(odin_ctx* ctx, const uint32_t* d_read_b, const uint32_t* d_write_b,
                                      const uint32_t* d_write_a, uint32_t n_prims, const uint32_t* d_active_idx_a,
                                      const float* d_evidence_a, const uint32_t* d_active_count_a,
                                      const double* d_evidence_sum_a, uint32_t active_capacity_a, float tau,
                                      uint64_t* d_gate, void* stream) {
  if (!ctx || !d_gate) return ODIN_ERR_NULL;
  if (!(tau >= 0.f && tau <= 1.f)) return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(d_gate, 0, 32, st));
  const uint32_t words = (n_prims + 31) / 32;
  if (words == 0) return ODIN_OK;
  if (!d_read_b || !d_write_b || !d_write_a || !d_active_count_a || !d_evidence_sum_a) return ODIN_ERR_NULL;
  if (active_capacity_a > 0 && (!d_active_idx_a || !d_evidence_a)) return ODIN_ERR_NULL;
  const uint32_t work = words > active_capacity_a ? words : active_capacity_a;
  uint32_t grid = (work + HZ_THREADS - 1) / HZ_THREADS;
  if (grid > (uint32_t)ctx->sm_count * 8) grid = (uint32_t)ctx->sm_count * 8;
  OdinKernelScope ks(ctx, K_GATE, st);
  delayed_read_gate_kernel<<<grid, HZ_THREADS, 0, st>>>(d_read_b, d_write_b, d_write_a, words, d_active_idx_a,
                                                       d_evidence_a, d_active_count_a, d_evidence_sum_a,
                                                       active_capacity_a, n_prims, tau,
                                                       reinterpret_cast<unsigned long long*>(d_gate));
  return odin_launch_status();
}
