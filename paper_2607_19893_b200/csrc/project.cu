// Preprocessing phase in three streaming kernels:
//   1. cull + count: every primitive -> number of tiles its rectangle covers (0 = culled); no synchronisation at all,
//      the attributes beyond the mean are only loaded for primitives that pass the depth test;
//   2. scan: single-pass decoupled look-back over the counts -> ascending list of visible primitives (the row map) and
//      the exclusive prefix of their tile counts (instance offsets), totals V and M;
//   3. rows: one thread per VISIBLE primitive recomputes the (deterministic) geometry and writes the compact record,
//      evaluates the SH colour and the opacity.
// At 2-30 % visibility recomputing the geometry of the visible rows is far cheaper than carrying per-primitive state
// through a block-wide scan in the first kernel.
#include "geom.cuh"
#include "layout.cuh"
#include "tilespan.cuh"

namespace {

struct Footprint {
  float u, v, depth, cA, cB, cC;
  int rad, x0, y0, x1, y1;
  uint32_t tiles;
};

// How the tile rectangle is chosen.  binning 0: the rectangle of the radius.  binning 1 (an optimised-pipeline variant
// in the sense of Sec. 5: same primitive ids, same image): additionally cut to the axis-aligned extent of the region in
// which alpha = opacity * exp(-q / 2) can reach alpha_min, q = d^T Sigma'^-1 d <= k = 2 ln(opacity / alpha_min), whose
// half extents are sqrt(k Sigma'_xx), sqrt(k Sigma'_yy) (widened by 1e-4 relative + 1e-3 pixels).  No pixel outside it
// passes the skip test of the blend kernels, so the instances that disappear never contributed.
struct BinRule {
  float dilation, radius_sigmas, alpha_min;
  int binning;
};

// Conic, radius and tile rectangle of one primitive.  Plain IEEE arithmetic (this file is compiled without fused
// multiply-add contraction): the integer results must not depend on which kernel evaluates them.
// PRETEST (the counting kernel, where most primitives end up with no tile): a primitive in front of the camera whose
// centre lies farther from the image than a bound on its radius cannot touch a tile, and the bound needs neither the
// quaternion nor the covariance.  With T = J W (W a rotation) the projected covariance satisfies
// lambda_max(T Sigma T^T) <= |J|_F^2 s_max^2, |J|_F^2 <= (fx/z)^2 (1 + limx^2) + (fy/z)^2 (1 + limy^2), and the radius
// formula adds at most sqrt(0.1) to the larger eigenvalue; the bound is then widened by 1 % + 2 pixels, far beyond
// rounding.  Only primitives for which the exact rectangle is certainly empty leave here, so the result is unchanged.
template <bool PRETEST = false>
__device__ __forceinline__ Footprint project_footprint(const CamParams& cam, const BinRule& rule,
                                                      const float* __restrict__ means,
                                                      const float* __restrict__ log_scales,
                                                      const float4* __restrict__ quats,
                                                      const float* __restrict__ opacity_logit, size_t p) {
  const float dilation = rule.dilation, radius_sigmas = rule.radius_sigmas;
  Footprint f;
  f.tiles = 0; f.u = f.v = f.depth = f.cA = f.cB = f.cC = 0.f; f.rad = f.x0 = f.y0 = f.x1 = f.y1 = 0;
  SplatGeom g;
  odin_camera_space(cam, means[3 * p], means[3 * p + 1], means[3 * p + 2], g.t);
  if (!(g.t[2] > cam.znear && g.t[2] < cam.zfar)) return f;
  const float ls[3] = {log_scales[3 * p], log_scales[3 * p + 1], log_scales[3 * p + 2]};
  if (PRETEST) {
    // hardware approximations (relative error ~1e-6) are enough here: the bound carries 1 % + 2 pixels of slack, and
    // most primitives of a large scene leave at this test
    const float iz = __fdividef(1.f, g.t[2]);
    const float uc = cam.fx * g.t[0] * iz + cam.cx, vc = cam.fy * g.t[1] * iz + cam.cy;
    const float smax = __expf(fmaxf(ls[0], fmaxf(ls[1], ls[2])));
    const float jx = cam.fx * iz, jy = cam.fy * iz;
    const float jn2 = jx * jx * (1.f + cam.limx * cam.limx) + jy * jy * (1.f + cam.limy * cam.limy);
    float root;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(root) : "f"(jn2 * smax * smax + dilation + 0.32f));
    const float rb = radius_sigmas * root * 1.01f + 2.f;
    if (uc + rb < 0.f || uc - rb > 16.f * (float)cam.TX || vc + rb < 0.f || vc - rb > 16.f * (float)cam.TY) return f;
  }
  odin_splat_geometry(cam, dilation, ls, quats[p], g);
  if (!(g.det > 0.f)) return f;
  f.cA = g.c / g.det; f.cB = -g.b / g.det; f.cC = g.a / g.det;
  const float mid = (g.a + g.c) / 2.f;
  const float lam = mid + sqrtf(fmaxf(0.1f, mid * mid - g.det));
  const float radf = ceilf(radius_sigmas * sqrtf(lam));
  f.u = cam.fx * g.t[0] / g.t[2] + cam.cx;
  f.v = cam.fy * g.t[1] / g.t[2] + cam.cy;
  f.depth = g.t[2];
  const float ftx = (float)cam.TX, fty = (float)cam.TY;
  f.x0 = (int)fminf(ftx, fmaxf(0.f, floorf((f.u - radf) / 16.f)));
  f.x1 = (int)fminf(ftx, fmaxf(0.f, ceilf((f.u + radf) / 16.f)));
  f.y0 = (int)fminf(fty, fmaxf(0.f, floorf((f.v - radf) / 16.f)));
  f.y1 = (int)fminf(fty, fmaxf(0.f, ceilf((f.v + radf) / 16.f)));
  if (rule.binning == 1) {
    const float opac = 1.f / (1.f + expf(-opacity_logit[p]));
    if (!(opac >= rule.alpha_min)) {
      f.x1 = f.x0;  // never reaches alpha_min anywhere
    } else {
      const float k = 2.f * logf(opac / rule.alpha_min);
      const float ex = sqrtf(k * g.a) * 1.0001f + 1e-3f, ey = sqrtf(k * g.c) * 1.0001f + 1e-3f;
      // tiles that hold a pixel centre (i + 0.5) within [u - ex, u + ex]
      const int tx0 = (int)fminf(ftx, fmaxf(0.f, floorf((f.u - ex - 0.5f) / 16.f)));
      const int tx1 = (int)fminf(ftx, fmaxf(0.f, floorf((f.u + ex - 0.5f) / 16.f) + 1.f));
      const int ty0 = (int)fminf(fty, fmaxf(0.f, floorf((f.v - ey - 0.5f) / 16.f)));
      const int ty1 = (int)fminf(fty, fmaxf(0.f, floorf((f.v + ey - 0.5f) / 16.f) + 1.f));
      f.x0 = max(f.x0, tx0); f.x1 = max(f.x0, min(f.x1, tx1));
      f.y0 = max(f.y0, ty0); f.y1 = max(f.y0, min(f.y1, ty1));
    }
  }
  f.tiles = (uint32_t)(f.x1 - f.x0) * (uint32_t)(f.y1 - f.y0);
  f.rad = (int)fminf(radf, 2.0e9f);
  return f;
}

template <bool EXACT>  // EXACT: binning 2 (a separate instantiation: the default path does not carry its registers)
__global__ void __launch_bounds__(256)
project_cull_kernel(const float* __restrict__ means, const float* __restrict__ log_scales, const float4* __restrict__ quats,
                    const float* __restrict__ opacity_logit, uint32_t n, CamParams cam, BinRule rule,
                    uint32_t* __restrict__ tiles_touched) {
  const uint32_t p = blockIdx.x * 256u + threadIdx.x;
  Footprint f = {};
  if (p < n) f = project_footprint<true>(cam, rule, means, log_scales, quats, opacity_logit, p);
  if (EXACT) {
    // exact binning: of the rectangle only the tiles the splat's alpha >= alpha_min region reaches (tilespan.cuh).  A
    // lane counts a rectangle of few tile rows by itself; the tall ones of the warp are counted by all 32 lanes together.
    SpanConic e;
    e.k = -1.f;
    if (f.tiles != 0) {
      const float opac = 1.f / (1.f + expf(-opacity_logit[p]));
      e = odin_span_conic(f.u, f.v, f.cA, f.cB, f.cC, opac, rule.alpha_min);
    }
    const bool tall = f.tiles != 0 && f.y1 - f.y0 > 4;
    if (f.tiles != 0 && !tall) {
      uint32_t kept = 0;
      for (int ty = f.y0; ty < f.y1; ++ty) {
        int xa, xb;
        odin_row_span(e, ty, f.x0, f.x1, xa, xb);
        kept += (uint32_t)(xb - xa);
      }
      f.tiles = kept;
    }
    uint32_t todo = __ballot_sync(0xffffffffu, tall);
    while (todo) {
      const int src = __ffs(todo) - 1;
      todo &= todo - 1;
      const SpanConic q = odin_span_conic_bcast(e, src);
      const uint32_t kept = odin_rect_kept_warp(q, __shfl_sync(0xffffffffu, f.x0, src), __shfl_sync(0xffffffffu, f.y0, src),
                                                __shfl_sync(0xffffffffu, f.x1, src), __shfl_sync(0xffffffffu, f.y1, src));
      if ((int)(threadIdx.x & 31) == src) f.tiles = kept;
    }
  }
  if (p < n) tiles_touched[p] = f.tiles;
}

// packed look-back value: rows in the upper 28 bits, tile instances in the lower 34 bits
constexpr int PACK_SHIFT = 34;
constexpr uint64_t PACK_LOW = (1ull << PACK_SHIFT) - 1;
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = PROJECT_TILE / SCAN_THREADS;

// Each warp owns 32 * SCAN_ITEMS consecutive primitives; load j of lane l is primitive warp_base + 32 j + l, so ranks
// inside the warp follow the primitive order.  Row index and instance offset come from one 64-bit look-back.
__global__ void __launch_bounds__(SCAN_THREADS)
project_scan_kernel(const uint32_t* __restrict__ tiles_touched, uint32_t n, uint32_t capacity,
                    uint32_t* __restrict__ prim_id, uint32_t* __restrict__ tile_offset, uint32_t* __restrict__ num_rows,
                    uint64_t* __restrict__ num_instances, uint32_t* ticket, uint64_t* state, int* status,
                    int scan_rounds, int spin_limit, uint32_t* __restrict__ touched_mask) {
  const uint32_t scan_chunk = PROJECT_TILE * (uint32_t)scan_rounds;
  __shared__ uint32_t s_tile;
  __shared__ uint64_t s_warp[SCAN_THREADS / 32 + 1];
  __shared__ uint64_t s_inst[SCAN_THREADS / 32];
  __shared__ uint64_t s_base;
  unsigned long long* exact_instances = reinterpret_cast<unsigned long long*>(ticket + 2);  // zeroed with the ticket
  if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t chunk_base = tile * scan_chunk;
  // pass A: packed (rows, instances) total of the chunk, then ONE look-back per scan_chunk primitives.  The instance
  // field holds 34 bits, a chunk can reach 2^14 primitives x 2^20 tiles and there are up to 2^14 chunks, so the packed
  // sums can carry into the row field when the view has 2^32 instances or more (an error by definition).  That case
  // is caught on a counter of its own: every chunk adds its exact instance count (kept apart in 64 bits, the packed
  // copy saturated) to a 64-bit total, and whoever sees that total reach 2^32 reports ODIN_ERR_CAPACITY.  The outputs
  // of such a view are meaningless but every write stays inside the caller's capacities (the row guard below).
  uint64_t mine = 0, mine_inst = 0;
#pragma unroll
  for (int rnd = 0; rnd < scan_rounds; ++rnd) {
    const uint32_t warp_base = chunk_base + rnd * PROJECT_TILE + warp * (32 * SCAN_ITEMS);
#pragma unroll
    for (int j = 0; j < SCAN_ITEMS; ++j) {
      const uint32_t p = warp_base + 32 * j + lane;
      const uint32_t t = (p < n) ? tiles_touched[p] : 0u;
      mine += t ? (1ull << PACK_SHIFT) : 0ull;
      mine_inst += t;
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    mine += __shfl_xor_sync(0xffffffffu, mine, o);
    mine_inst += __shfl_xor_sync(0xffffffffu, mine_inst, o);
  }
  if (lane == 0) { s_warp[warp] = mine; s_inst[warp] = mine_inst; }
  __syncthreads();
  if (threadIdx.x < 32) {
    uint64_t total = (lane < SCAN_THREADS / 32) ? s_warp[lane] : 0ull;
    uint64_t total_inst = (lane < SCAN_THREADS / 32) ? s_inst[lane] : 0ull;
    for (int o = 16; o > 0; o >>= 1) {
      total += __shfl_xor_sync(0xffffffffu, total, o);
      total_inst += __shfl_xor_sync(0xffffffffu, total_inst, o);
    }
    if (lane == 0 && total_inst != 0) {
      const unsigned long long before = atomicAdd(exact_instances, (unsigned long long)total_inst);
      if (before + total_inst >= (1ull << 32)) odin_set_error(status, ODIN_ERR_CAPACITY);
    }
    total |= total_inst < (1ull << 32) ? total_inst : ((1ull << 32) - 1);
    const uint64_t base = odin_lookback_u64(state, tile, total, status, spin_limit);
    if (lane == 0) {
      s_base = base;
      if (tile == (n + scan_chunk - 1) / scan_chunk - 1) {  // last chunk: totals
        const uint64_t all = base + total;
        const uint64_t rows = all >> PACK_SHIFT, inst = all & PACK_LOW;
        *num_rows = (uint32_t)(rows < capacity ? rows : capacity);
        *num_instances = inst;
        if (rows > capacity || inst >= (1ull << 32)) odin_set_error(status, ODIN_ERR_CAPACITY);
      }
    }
  }
  __syncthreads();
  uint64_t round_base = s_base;
  // pass B: re-read the chunk (from cache), 2048 primitives per round
  for (int rnd = 0; rnd < scan_rounds; ++rnd) {
    if (chunk_base + rnd * PROJECT_TILE >= n) break;  // uniform over the block
    const uint32_t warp_base = chunk_base + rnd * PROJECT_TILE + warp * (32 * SCAN_ITEMS);
    uint32_t t[SCAN_ITEMS];
#pragma unroll
    for (int j = 0; j < SCAN_ITEMS; ++j) {
      const uint32_t p = warp_base + 32 * j + lane;
      t[j] = (p < n) ? tiles_touched[p] : 0u;
    }
    // per item: packed (1 row, t tiles) exclusive prefix inside the warp, in primitive order
    uint64_t ex[SCAN_ITEMS];
    uint64_t run = 0;
#pragma unroll
    for (int j = 0; j < SCAN_ITEMS; ++j) {
      ex[j] = run;
      const uint32_t visible = __ballot_sync(0xffffffffu, t[j] != 0);
      // the 32 primitives of this load are one word of the touched bitmask
      if (touched_mask && lane == 0 && warp_base + 32 * j < n) touched_mask[(warp_base + 32 * j) >> 5] = visible;
      if (visible == 0) continue;  // 32 culled primitives in a row: nothing to scan
      const uint64_t v = t[j] ? ((1ull << PACK_SHIFT) | (uint64_t)t[j]) : 0ull;
      uint64_t inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint64_t y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= (unsigned)o) inc += y;
      }
      ex[j] = run + inc - v;
      run += __shfl_sync(0xffffffffu, inc, 31);
    }
    __syncthreads();  // previous round's readers of s_warp are done
    if (lane == 0) s_warp[warp] = run;
    __syncthreads();
    uint64_t before = 0, total = 0;
#pragma unroll
    for (int w = 0; w < SCAN_THREADS / 32; ++w) {
      const uint64_t x = s_warp[w];
      if (w < (int)warp) before += x;
      total += x;
    }
    const uint64_t base = round_base + before;
#pragma unroll
    for (int j = 0; j < SCAN_ITEMS; ++j) {
      if (t[j]) {
        const uint64_t e = base + ex[j];
        const uint64_t r = e >> PACK_SHIFT;
        if (r < capacity) {
          prim_id[r] = warp_base + 32 * j + lane;
          tile_offset[r] = (uint32_t)(e & PACK_LOW);
        }
      }
    }
    round_base += total;
  }
}

template <int DEG>
__global__ void __launch_bounds__(128)
project_rows_kernel(const float* __restrict__ means, const float* __restrict__ log_scales, const float4* __restrict__ quats,
                    const float* __restrict__ opacity_logit, const float* __restrict__ sh, CamParams cam, BinRule rule,
                    odin_projected out, uint32_t n) {
  constexpr int K = (DEG + 1) * (DEG + 1);
  const uint32_t V = min(*out.num_rows, out.capacity);
  for (uint32_t r = blockIdx.x * blockDim.x + threadIdx.x; r < V; r += gridDim.x * blockDim.x) {
    const size_t p = min(out.prim_id[r], n - 1);  // in range even if the scan gave up and left part of the map unwritten
    const Footprint f = project_footprint(cam, rule, means, log_scales, quats, opacity_logit, p);
    reinterpret_cast<float2*>(out.xy)[r] = make_float2(f.u, f.v);
    out.depth[r] = f.depth;
    const float o = 1.f / (1.f + expf(-opacity_logit[p]));
    reinterpret_cast<float4*>(out.conic_opacity)[r] = make_float4(f.cA, f.cB, f.cC, o);
    out.radius[r] = f.rad;
    reinterpret_cast<ushort4*>(out.rect)[r] =
        make_ushort4((unsigned short)f.x0, (unsigned short)f.y0, (unsigned short)f.x1, (unsigned short)f.y1);
    // colour
    float dx = means[3 * p] - cam.pos[0], dy = means[3 * p + 1] - cam.pos[1], dz = means[3 * p + 2] - cam.pos[2];
    const float len = sqrtf(dx * dx + dy * dy + dz * dz);
    dx /= len; dy /= len; dz /= len;
    float Y[16];
    odin_sh_basis<DEG>(dx, dy, dz, Y);
    float acc[3] = {0.f, 0.f, 0.f};
    const float* row = sh + p * (3 * K);
    if ((3 * K) % 4 == 0) {  // 12 or 48 floats: 16-byte loads
      const float4* row4 = reinterpret_cast<const float4*>(row);
#pragma unroll
      for (int i = 0; i < 3 * K / 4; ++i) {
        const float4 c = row4[i];
        const float e[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int w = 4 * i + j;
          acc[w % 3] += Y[w / 3] * e[j];
        }
      }
    } else {
#pragma unroll
      for (int w = 0; w < 3 * K; ++w) acc[w % 3] += Y[w / 3] * row[w];
    }
    uint8_t flags = 0;
#pragma unroll
    for (int ch = 0; ch < 3; ++ch) {
      acc[ch] += 0.5f;
      if (acc[ch] < 0.f) { acc[ch] = 0.f; flags |= (uint8_t)(1u << ch); }
    }
    out.rgb[3 * (size_t)r] = acc[0]; out.rgb[3 * (size_t)r + 1] = acc[1]; out.rgb[3 * (size_t)r + 2] = acc[2];
    out.clamp_flags[r] = flags;
  }
}

}  // namespace

extern "C" int odin_project(odin_ctx* ctx, const odin_scene* scene, const odin_camera* cam, odin_projected* out, void* ws,
                            size_t ws_bytes, void* stream) {
  if (!ctx || !out) return ODIN_ERR_NULL;
  int rc = odin_check_scene(scene);
  if (rc != ODIN_OK) return rc;
  rc = odin_check_camera(cam);
  if (rc != ODIN_OK) return rc;
  if (!out->num_rows || !out->num_instances) return ODIN_ERR_NULL;
  if (out->capacity > 0 && (!out->prim_id || !out->xy || !out->depth || !out->conic_opacity || !out->rgb || !out->radius ||
                            !out->rect || !out->tile_offset || !out->clamp_flags))
    return ODIN_ERR_NULL;
  if (!odin_aligned(out->xy, 8) || !odin_aligned(out->conic_opacity, 16) || !odin_aligned(out->rect, 8) ||
      !odin_aligned(out->num_instances, 8))
    return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const uint32_t n = scene->n;
  if (n == 0) {
    ODIN_CUDA(cudaMemsetAsync(out->num_rows, 0, 4, st));
    ODIN_CUDA(cudaMemsetAsync(out->num_instances, 0, 8, st));
    return ODIN_OK;
  }
  if (!out->tiles_touched) return ODIN_ERR_NULL;
  const size_t need = project_ws_bytes(n);
  if (!ws || !odin_aligned(ws, 256) || ws_bytes < need) return ODIN_ERR_WORKSPACE;
  ODIN_CUDA(cudaMemsetAsync(ws, 0, need, st));
  uint32_t* ticket = reinterpret_cast<uint32_t*>(ws);
  uint64_t* state = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(ws) + 256);
  const CamParams cp = odin_cam_params(cam, ctx->cfg);
  const float4* q4 = reinterpret_cast<const float4*>(scene->quats);
  const BinRule rule = {ctx->cfg.dilation, ctx->cfg.radius_sigmas, ctx->cfg.alpha_min, ctx->cfg.binning};
  {
    OdinKernelScope ks(ctx, K_PROJECT, st);
    if (rule.binning == 2)
      project_cull_kernel<true><<<(n + 255) / 256, 256, 0, st>>>(scene->means, scene->log_scales, q4, scene->opacity_logit,
                                                                 n, cp, rule, out->tiles_touched);
    else
      project_cull_kernel<false><<<(n + 255) / 256, 256, 0, st>>>(scene->means, scene->log_scales, q4,
                                                                  scene->opacity_logit, n, cp, rule, out->tiles_touched);
  }
  {
    OdinKernelScope ks(ctx, K_PROJECT_SCAN, st);
    const int scan_rounds = scan_rounds_for(n, ctx->sm_count);
    const uint32_t scan_chunk = PROJECT_TILE * (uint32_t)scan_rounds;
    project_scan_kernel<<<(n + scan_chunk - 1) / scan_chunk, SCAN_THREADS, 0, st>>>(
        out->tiles_touched, n, out->capacity, out->prim_id, out->tile_offset, out->num_rows, out->num_instances, ticket,
        state, ctx->d_status, scan_rounds, ctx->spin_limit, out->touched_mask);
  }
  if (out->capacity == 0) return odin_launch_status();
  const uint32_t blocks_cap = (out->capacity + 127) / 128;
  const uint32_t grid = blocks_cap < (uint32_t)ctx->sm_count * 16 ? blocks_cap : (uint32_t)ctx->sm_count * 16;
  OdinKernelScope ks(ctx, K_PROJECT_ROWS, st);
#define LAUNCH(D)                                                                                                      \
  project_rows_kernel<D><<<grid, 128, 0, st>>>(scene->means, scene->log_scales, q4, scene->opacity_logit, scene->sh, cp, \
                                               rule, *out, n)
  switch (scene->sh_degree) {
    case 0: LAUNCH(0); break;
    case 1: LAUNCH(1); break;
    case 2: LAUNCH(2); break;
    default: LAUNCH(3); break;
  }
#undef LAUNCH
  return odin_launch_status();
}
