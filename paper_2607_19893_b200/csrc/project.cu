// Preprocessing phase:
//   1. cull + count: every primitive -> number of tiles its rectangle covers (0 = culled): depth test on the mean, then
//      (attributes beyond the mean are only loaded for primitives in front of the camera) a lateral test from the scales
//      alone, and the covariance only for those that pass it;
//   2. scan of the counts (single-pass decoupled look-back) -> ascending list of visible primitives (the row map),
//      exclusive prefix of their tile counts (instance offsets), totals V and M, touched bitmask.  For scenes of up to
//      ~1.2 M primitives 1 and 2 are one kernel;
//   3. rows: one thread per VISIBLE primitive recomputes the (deterministic) geometry and writes the compact record,
//      evaluates the SH colour and the opacity.
// At 2-30 % visibility recomputing the geometry of the visible rows is far cheaper than carrying per-primitive state
// through the block-wide scan.
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

// packed look-back value: rows in the upper 28 bits, tile instances in the lower 34 bits
constexpr int PACK_SHIFT = 34;
constexpr uint64_t PACK_LOW = (1ull << PACK_SHIFT) - 1;
constexpr int SCAN_THREADS = 256;
constexpr int SCAN_ITEMS = PROJECT_TILE / SCAN_THREADS;
constexpr int SCAN_MAX_ROUNDS = 8;

// Cheap part of the footprint, for every primitive in front of the camera (t: camera-space mean, l: log scales): a
// lateral pre-test.  false = the exact rectangle is certainly empty.
// The lateral pre-test (most primitives of a large scene end up with no tile): a primitive in front of the camera whose
// centre lies farther from the image than a bound on its radius cannot touch a tile, and the bound needs neither the
// quaternion nor the covariance.  With T = J W (W a rotation) the projected covariance satisfies
// lambda_max(T Sigma T^T) <= |J|_F^2 s_max^2, |J|_F^2 <= (fx/z)^2 (1 + limx^2) + (fy/z)^2 (1 + limy^2), and the radius
// formula adds at most sqrt(0.1) to the larger eigenvalue; the bound is then widened by 1 % + 2 pixels, far beyond
// rounding.  Only primitives for which the exact rectangle is certainly empty leave here, so the result is unchanged.
__device__ __forceinline__ bool cull_survives(const CamParams& cam, const BinRule& rule, const float* t, float l0,
                                              float l1, float l2) {
  // hardware approximations (relative error ~1e-6) are enough here: the bound carries 1 % + 2 pixels of slack
  const float iz = __fdividef(1.f, t[2]);
  const float uc = cam.fx * t[0] * iz + cam.cx, vc = cam.fy * t[1] * iz + cam.cy;
  const float smax = __expf(fmaxf(l0, fmaxf(l1, l2)));
  const float jx = cam.fx * iz, jy = cam.fy * iz;
  const float jn2 = jx * jx * (1.f + cam.limx * cam.limx) + jy * jy * (1.f + cam.limy * cam.limy);
  float root;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(root) : "f"(jn2 * smax * smax + rule.dilation + 0.32f));
  const float rb = rule.radius_sigmas * root * 1.01f + 2.f;
  return !(uc + rb < 0.f || uc - rb > 16.f * (float)cam.TX || vc + rb < 0.f || vc - rb > 16.f * (float)cam.TY);
}

// Exact binning (binning 2): of the rectangle only the tiles the splat's alpha >= alpha_min region reaches
// (tilespan.cuh).  Called by all 32 lanes (f.tiles = 0 for lanes without a primitive): a lane counts a rectangle of few
// tile rows by itself; the tall ones of the warp are counted by all 32 lanes together.
__device__ __forceinline__ uint32_t exact_tiles_warp(const Footprint& f, const BinRule& rule,
                                                     const float* __restrict__ opacity_logit, size_t p) {
  const unsigned lane = threadIdx.x & 31;
  uint32_t tiles = f.tiles;
  SpanConic e;
  e.k = -1.f;
  if (tiles != 0) {
    const float opac = 1.f / (1.f + expf(-opacity_logit[p]));
    e = odin_span_conic(f.u, f.v, f.cA, f.cB, f.cC, opac, rule.alpha_min);
  }
  const bool tall = tiles != 0 && f.y1 - f.y0 > 4;
  if (tiles != 0 && !tall) {
    uint32_t kept = 0;
    for (int ty = f.y0; ty < f.y1; ++ty) {
      int xa, xb;
      odin_row_span(e, ty, f.x0, f.x1, xa, xb);
      kept += (uint32_t)(xb - xa);
    }
    tiles = kept;
  }
  uint32_t todo = __ballot_sync(0xffffffffu, tall);
  while (todo) {
    const int src = __ffs(todo) - 1;
    todo &= todo - 1;
    const SpanConic c = odin_span_conic_bcast(e, src);
    const uint32_t kept =
        odin_rect_kept_warp(c, __shfl_sync(0xffffffffu, f.x0, src), __shfl_sync(0xffffffffu, f.y0, src),
                            __shfl_sync(0xffffffffu, f.x1, src), __shfl_sync(0xffffffffu, f.y1, src));
    if ((int)lane == src) tiles = kept;
  }
  return tiles;
}

// Counting kernel for large scenes: one thread per primitive at full occupancy (64 warps per SM hide the covariance
// code of the few survivors behind the stream of means and scales; the kernel runs at ~80 % of the HBM bandwidth).
template <bool EXACT>
__global__ void __launch_bounds__(256)
project_cull_kernel(const float* __restrict__ means, const float* __restrict__ log_scales, const float4* __restrict__ quats,
                    const float* __restrict__ opacity_logit, uint32_t n, CamParams cam, BinRule rule,
                    uint32_t* __restrict__ tiles_touched, unsigned long long* __restrict__ group_total,
                    unsigned long long* __restrict__ chunk_total, uint32_t groups_per_chunk) {
  odin_after_predecessor();
  const uint32_t p = blockIdx.x * 256u + threadIdx.x;
  Footprint f = {};
  if (p < n) {
    float t[3];
    odin_camera_space(cam, means[3 * (size_t)p], means[3 * (size_t)p + 1], means[3 * (size_t)p + 2], t);
    if (t[2] > cam.znear && t[2] < cam.zfar &&
        cull_survives(cam, rule, t, log_scales[3 * (size_t)p], log_scales[3 * (size_t)p + 1], log_scales[3 * (size_t)p + 2]))
      f = project_footprint(cam, rule, means, log_scales, quats, opacity_logit, p);
  }
  if (EXACT) f.tiles = exact_tiles_warp(f, rule, opacity_logit, p);
  if (p < n) tiles_touched[p] = f.tiles;
  // what the scan needs to start anywhere without waiting: the packed (rows, instances) total of this block's 256
  // primitives and the exact totals of the chunk of blocks it belongs to, added up by the warps that have something to
  // add (both zeroed before the launch; no block barrier, so a warp with a long covariance path holds nobody up)
  const uint32_t rows_w = __popc(__ballot_sync(0xffffffffu, f.tiles != 0));
  if (rows_w == 0) return;
  uint32_t inst = f.tiles;  // at most 2^20 per primitive: 2^25 per warp
  for (int o = 16; o > 0; o >>= 1) inst += __shfl_xor_sync(0xffffffffu, inst, o);
  if ((threadIdx.x & 31) == 0) {
    atomicAdd(&group_total[blockIdx.x], ((unsigned long long)rows_w << PACK_SHIFT) | (unsigned long long)inst);
    const size_t c = blockIdx.x / groups_per_chunk;
    atomicAdd(&chunk_total[2 * c], (unsigned long long)rows_w);
    atomicAdd(&chunk_total[2 * c + 1], (unsigned long long)inst);
  }
}

// Scan of the tile counts, for small scenes fused with the counting.  A block takes `rounds` x 2048 consecutive
// primitives by ticket (more rounds = fewer look-backs, each of which walks back over the blocks in flight); in a round
// each of its eight warps owns 256 primitives, item j of lane l being primitive warp_base + 32 j + l, so that ranks
// inside the warp follow the primitive order and the 32 primitives of one item are one word of the touched bitmask.
//   A. per round, the tile counts of the warp's primitives.  FUSED (scenes whose blocks are all resident at once, where
//      a kernel launch and a pass over the counts are what there is to save): the cheap tests as three straight-line
//      sweeps, so that the loads of a sweep are all in flight together (means -> depth test -> log scales of those in
//      front of the camera -> lateral test); the survivors of the warp (2-30 % of a scene) are compacted into a list in
//      shared memory and taken 32 at a time: exact footprint -> number of tiles (a warp of survivors, not a warp with
//      one survivor and 31 idle lanes, runs the long covariance code); the dense counts are written.  Otherwise the
//      counts are read (project_cull_kernel wrote them).  Either way they are summed per (round, warp);
//   B. packed (rows, instances) total of the block, ONE decoupled look-back (the only two block barriers);
//   C. per round, every warp on its own: the counts again (from shared memory when fused, else from the cache), ranks by
//      population count and a 32-bit scan -> row map, instance offsets, touched bitmask.
template <bool EXACT, bool FUSED>  // EXACT: binning 2
__global__ void __launch_bounds__(SCAN_THREADS, EXACT && FUSED ? 3 : 4)
project_scan_kernel(const float* __restrict__ means, const float* __restrict__ log_scales,
                    const float4* __restrict__ quats, const float* __restrict__ opacity_logit, uint32_t n, CamParams cam,
                    BinRule rule, uint32_t* tiles_touched, uint32_t capacity, uint32_t* __restrict__ prim_id,
                    uint32_t* __restrict__ tile_offset, uint32_t* __restrict__ num_rows,
                    uint64_t* __restrict__ num_instances, uint32_t* ticket, uint64_t* state,
                    const uint64_t* __restrict__ group_total, const uint64_t* __restrict__ chunk_total, int* status,
                    int rounds, int spin_limit, uint32_t* __restrict__ touched_mask) {
  odin_after_predecessor();  // not fused: launched behind the counting kernel
  __shared__ uint32_t s_tile;
  __shared__ uint64_t s_warp[SCAN_THREADS / 32];
  __shared__ uint64_t s_inst[SCAN_THREADS / 32];
  __shared__ uint64_t s_base;
  __shared__ uint64_t s_tot[SCAN_MAX_ROUNDS][SCAN_THREADS / 32];  // packed total of (round, warp)
  __shared__ uint32_t s_t[FUSED ? SCAN_ITEMS : 1][SCAN_THREADS];  // fused (one round): tile count of item j of thread t
  __shared__ uint8_t s_list[FUSED ? SCAN_THREADS / 32 : 1][32 * SCAN_ITEMS];  // per warp: survivors as 32 j + lane
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t chunk = PROJECT_TILE * (uint32_t)rounds;
  int done = 0;  // rounds that hold primitives (uniform over the block)
  uint32_t tile, chunk_base;
  if (FUSED) {
    unsigned long long* exact_instances = reinterpret_cast<unsigned long long*>(ticket + 2);  // zeroed with the ticket
    if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
    __syncthreads();
    tile = s_tile;
    chunk_base = tile * chunk;
    // ---- A
    uint64_t rows_b = 0, inst_b = 0;  // the warp's rows and instances over all rounds (uniform over the warp)
    for (int rnd = 0; rnd < rounds; ++rnd) {
      if (chunk_base + rnd * PROJECT_TILE >= n) break;  // uniform over the block
      const uint32_t warp_base = chunk_base + rnd * PROJECT_TILE + warp * (32 * SCAN_ITEMS);
      uint32_t t[SCAN_ITEMS];
      {
        float ct[SCAN_ITEMS][3];  // mean, then camera-space mean
  #pragma unroll
        for (int j = 0; j < SCAN_ITEMS; ++j) {
          const uint32_t p = warp_base + 32 * j + lane;
          ct[j][0] = ct[j][1] = ct[j][2] = 0.f;
          if (p < n) {
            ct[j][0] = means[3 * (size_t)p]; ct[j][1] = means[3 * (size_t)p + 1]; ct[j][2] = means[3 * (size_t)p + 2];
          }
        }
        uint32_t front = 0;
  #pragma unroll
        for (int j = 0; j < SCAN_ITEMS; ++j) {
          const uint32_t p = warp_base + 32 * j + lane;
          const float mx = ct[j][0], my = ct[j][1], mz = ct[j][2];
          odin_camera_space(cam, mx, my, mz, ct[j]);
          if (p < n && ct[j][2] > cam.znear && ct[j][2] < cam.zfar) front |= 1u << j;
        }
        float ls[SCAN_ITEMS][3];
  #pragma unroll
        for (int j = 0; j < SCAN_ITEMS; ++j) {
          const uint32_t p = warp_base + 32 * j + lane;
          ls[j][0] = ls[j][1] = ls[j][2] = 0.f;
          if (front >> j & 1u) {
            ls[j][0] = log_scales[3 * (size_t)p]; ls[j][1] = log_scales[3 * (size_t)p + 1];
            ls[j][2] = log_scales[3 * (size_t)p + 2];
          }
        }
        uint32_t n_alive = 0;
  #pragma unroll
        for (int j = 0; j < SCAN_ITEMS; ++j) {
          const bool alive = (front >> j & 1u) && cull_survives(cam, rule, ct[j], ls[j][0], ls[j][1], ls[j][2]);
          const uint32_t b = __ballot_sync(0xffffffffu, alive);
          if (alive) s_list[warp][n_alive + __popc(b & ((1u << lane) - 1u))] = (uint8_t)(32 * j + lane);
          n_alive += __popc(b);
          s_t[j][threadIdx.x] = 0;
        }
        __syncwarp();
        // exact footprints of the survivors, a warp-load at a time
        for (uint32_t i0 = 0; i0 < n_alive; i0 += 32) {
          const bool have = i0 + lane < n_alive;
          const uint32_t q = have ? s_list[warp][i0 + lane] : 0u;
          const uint32_t p = warp_base + q;
          Footprint f = {};
          if (have) f = project_footprint(cam, rule, means, log_scales, quats, opacity_logit, p);
          if (EXACT) f.tiles = exact_tiles_warp(f, rule, opacity_logit, p);
          if (have) s_t[q >> 5][warp * 32 + (q & 31)] = f.tiles;
        }
        __syncwarp();
  #pragma unroll
        for (int j = 0; j < SCAN_ITEMS; ++j) {
          const uint32_t p = warp_base + 32 * j + lane;
          t[j] = s_t[j][threadIdx.x];
          if (p < n) tiles_touched[p] = t[j];
        }
      }
      // the warp's packed (rows, instances) total of this round
      uint32_t rows_w = 0;
      uint64_t inst_l = 0;
  #pragma unroll
      for (int j = 0; j < SCAN_ITEMS; ++j) {
        rows_w += __popc(__ballot_sync(0xffffffffu, t[j] != 0));
        inst_l += t[j];
      }
      for (int o = 16; o > 0; o >>= 1) inst_l += __shfl_xor_sync(0xffffffffu, inst_l, o);
      if (lane == 0) s_tot[rnd][warp] = ((uint64_t)rows_w << PACK_SHIFT) + inst_l;
      rows_b += rows_w;
      inst_b += inst_l;
      done = rnd + 1;
    }

    // ---- B.  The instance field of the packed value holds 34 bits and there are up to 2^21 blocks of up to 2^14 x 2^20
    // instances, so the packed sums can carry into the row field when the view has 2^32 instances or more (an error by
    // definition).  That case is caught on a counter of its own: every block adds its exact instance count (kept apart
    // in 64 bits, the packed copy saturated) to a 64-bit total, and whoever sees that total reach 2^32 reports
    // ODIN_ERR_CAPACITY.  The outputs of such a view are meaningless but every write stays inside the caller's
    // capacities (the row guard below).
    if (lane == 0) { s_warp[warp] = rows_b; s_inst[warp] = inst_b; }
    __syncthreads();
    if (threadIdx.x < 32) {
      uint64_t total = (lane < SCAN_THREADS / 32) ? s_warp[lane] : 0ull;
      uint64_t total_inst = (lane < SCAN_THREADS / 32) ? s_inst[lane] : 0ull;
      for (int o = 16; o > 0; o >>= 1) {
        total += __shfl_xor_sync(0xffffffffu, total, o);
        total_inst += __shfl_xor_sync(0xffffffffu, total_inst, o);
      }
      if (lane == 0 && total_inst != 0) {
        const unsigned long long seen = atomicAdd(exact_instances, (unsigned long long)total_inst);
        if (seen + total_inst >= (1ull << 32)) odin_set_error(status, ODIN_ERR_CAPACITY);
      }
      total = (total << PACK_SHIFT) | (total_inst < (1ull << 32) ? total_inst : ((1ull << 32) - 1));
      const uint64_t base = odin_lookback_u64(state, tile, total, status, spin_limit);
      if (lane == 0) {
        s_base = base;
        if (tile == (n + chunk - 1) / chunk - 1) {  // last block: totals
          const uint64_t all = base + total;
          const uint64_t rows = all >> PACK_SHIFT, inst = all & PACK_LOW;
          *num_rows = (uint32_t)(rows < capacity ? rows : capacity);
          *num_instances = inst;
          if (rows > capacity || inst >= (1ull << 32)) odin_set_error(status, ODIN_ERR_CAPACITY);
        }
      }
    }
    __syncthreads();

  } else {
    // The counting kernel left the packed total of every 256 primitives (one (round, warp) of this kernel) and the exact
    // totals of every chunk: the block's base is a sum over the chunks in front of it, nothing is waited for.
    tile = blockIdx.x;
    chunk_base = tile * chunk;
    const uint32_t groups = (n + 32 * SCAN_ITEMS - 1) / (32 * SCAN_ITEMS);
    if (threadIdx.x < (unsigned)rounds * (SCAN_THREADS / 32)) {
      const uint64_t g = (uint64_t)tile * rounds * (SCAN_THREADS / 32) + threadIdx.x;
      s_tot[threadIdx.x / (SCAN_THREADS / 32)][threadIdx.x % (SCAN_THREADS / 32)] = g < groups ? group_total[g] : 0ull;
    }
    if (warp == 0) {
      uint64_t rows = 0, inst = 0;
      for (uint32_t c = lane; c < tile; c += 32) { rows += chunk_total[2 * (size_t)c]; inst += chunk_total[2 * (size_t)c + 1]; }
      for (int o = 16; o > 0; o >>= 1) {
        rows += __shfl_xor_sync(0xffffffffu, rows, o);
        inst += __shfl_xor_sync(0xffffffffu, inst, o);
      }
      if (lane == 0) {
        // 2^32 instances or more are an error by definition: the packed base is saturated so that the row field stays
        // intact and every write stays inside the caller's capacities (the row guard below)
        s_base = (rows << PACK_SHIFT) | (inst < (1ull << 32) ? inst : ((1ull << 32) - 1));
        if (tile == (n + chunk - 1) / chunk - 1) {  // last block: totals
          rows += chunk_total[2 * (size_t)tile];
          inst += chunk_total[2 * (size_t)tile + 1];
          *num_rows = (uint32_t)(rows < capacity ? rows : capacity);
          *num_instances = inst;
          if (rows > capacity || inst >= (1ull << 32)) odin_set_error(status, ODIN_ERR_CAPACITY);
        }
      }
    }
    __syncthreads();
    const uint32_t left = n - chunk_base;  // the grid has no block behind the last primitive
    done = (int)min((uint32_t)rounds, (left + PROJECT_TILE - 1) / PROJECT_TILE);
  }

  // ---- C.  No barrier from here on: the packed prefix of (round, warp) follows from the per-warp totals of A.
  uint64_t base = s_base;
  for (int w = 0; w < (int)warp; ++w) base += s_tot[0][w];
  for (int rnd = 0; rnd < done; ++rnd) {
    const uint32_t warp_base = chunk_base + rnd * PROJECT_TILE + warp * (32 * SCAN_ITEMS);
    uint32_t t[SCAN_ITEMS];
#pragma unroll
    for (int j = 0; j < SCAN_ITEMS; ++j) {
      const uint32_t p = warp_base + 32 * j + lane;
      // fused: one round, the counts are still in shared memory; else from the cache (this thread read them in A)
      t[j] = FUSED ? s_t[j][threadIdx.x] : ((p < n) ? tiles_touched[p] : 0u);
    }
    uint64_t run = base;  // packed prefix in front of the warp's next item
#pragma unroll
    for (int j = 0; j < SCAN_ITEMS; ++j) {
      const uint32_t visible = __ballot_sync(0xffffffffu, t[j] != 0);
      // the 32 primitives of this load are one word of the touched bitmask
      if (touched_mask && lane == 0 && warp_base + 32 * j < n) touched_mask[(warp_base + 32 * j) >> 5] = visible;
      if (visible == 0) continue;  // 32 culled primitives in a row: nothing to scan
      // rows in front of the lane: a population count; instances: a 32-bit scan (32 x 2^20 fits)
      uint32_t inc = t[j];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= (unsigned)o) inc += y;
      }
      if (t[j]) {
        const uint64_t e = run + ((uint64_t)__popc(visible & ((1u << lane) - 1u)) << PACK_SHIFT) + (inc - t[j]);
        const uint64_t r = e >> PACK_SHIFT;
        if (r < capacity) {
          prim_id[r] = warp_base + 32 * j + lane;
          tile_offset[r] = (uint32_t)(e & PACK_LOW);
        }
      }
      run += ((uint64_t)__popc(visible) << PACK_SHIFT) + __shfl_sync(0xffffffffu, inc, 31);
    }
    // next round of this warp: behind the rest of this round and in front of the lower warps' share of the next one
    for (int w = (int)warp; w < SCAN_THREADS / 32; ++w) base += s_tot[rnd][w];
    if (rnd + 1 < done)
      for (int w = 0; w < (int)warp; ++w) base += s_tot[rnd + 1][w];
  }
}

template <int DEG>
__global__ void __launch_bounds__(128)
project_rows_kernel(const float* __restrict__ means, const float* __restrict__ log_scales, const float4* __restrict__ quats,
                    const float* __restrict__ opacity_logit, const float* __restrict__ sh, CamParams cam, BinRule rule,
                    odin_projected out, uint32_t n) {
  odin_after_predecessor();
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
    odin_chain_break(ctx);
    ODIN_CUDA(cudaMemsetAsync(out->num_rows, 0, 4, st));
    ODIN_CUDA(cudaMemsetAsync(out->num_instances, 0, 8, st));
    return ODIN_OK;
  }
  if (!out->tiles_touched) return ODIN_ERR_NULL;
  const size_t need = project_ws_bytes(n);
  if (!ws || !odin_aligned(ws, 256) || ws_bytes < need) return ODIN_ERR_WORKSPACE;
  ODIN_CUDA(odin_zero(ctx, ws, need, st));
  uint32_t* ticket = reinterpret_cast<uint32_t*>(ws);
  uint64_t* state = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(ws) + 256);
  const CamParams cp = odin_cam_params(cam, ctx->cfg);
  const float4* q4 = reinterpret_cast<const float4*>(scene->quats);
  const BinRule rule = {ctx->cfg.dilation, ctx->cfg.radius_sigmas, ctx->cfg.alpha_min, ctx->cfg.binning};
  // Scenes whose 2048-primitive blocks are all resident at once take the fused kernel; larger ones a counting kernel at
  // full occupancy and the scan with longer chunks (measured: 1 M primitives 0.031 ms fused against 0.044 ms; 20 M
  // primitives 0.19 ms fused against 0.16 ms).
  const bool fused = (n + PROJECT_TILE - 1) / PROJECT_TILE <= (uint32_t)ctx->sm_count * 4u;
  // not fused: up to 8 rounds per block (measured at 20 M primitives: 0.090 / 0.065 / 0.059 / 0.066 / 0.080 ms with
  // 2 / 4 / 8 / 17 / 24 rounds; 17 is the count at which all blocks are resident at once)
  const int rounds = fused ? 1 : scan_rounds_for(n, ctx->sm_count);
  const uint32_t chunk = PROJECT_TILE * (uint32_t)rounds;
  const uint32_t blocks = (n + chunk - 1) / chunk;
  uint64_t* group_total = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(ws) + project_ws_group_offset(n));
  uint64_t* chunk_total = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(ws) + project_ws_chunk_offset(n));
#define LAUNCH(E, F)                                                                                                   \
  ODIN_CUDA(odin_launch(ctx, !(F), project_scan_kernel<E, F>, dim3(blocks), dim3(SCAN_THREADS), 0, st, scene->means,   \
                        scene->log_scales, q4, scene->opacity_logit, n, cp, rule, out->tiles_touched, out->capacity,   \
                        out->prim_id, out->tile_offset, out->num_rows, out->num_instances, ticket, state, group_total, \
                        chunk_total, ctx->d_status, rounds, ctx->spin_limit, out->touched_mask))
  if (fused) {
    OdinKernelScope ks(ctx, K_PROJECT, st);
    if (rule.binning == 2) LAUNCH(true, true);
    else LAUNCH(false, true);
  } else {
    {
      OdinKernelScope ks(ctx, K_PROJECT, st);
      const uint32_t gpc = (uint32_t)rounds * (SCAN_THREADS / 32);  // counting blocks per chunk of the scan
      unsigned long long* ct = reinterpret_cast<unsigned long long*>(chunk_total);
      unsigned long long* gt = reinterpret_cast<unsigned long long*>(group_total);
      if (rule.binning == 2)
        ODIN_CUDA(odin_launch(ctx, false, project_cull_kernel<true>, dim3((n + 255) / 256), dim3(256), 0, st, scene->means,
                              scene->log_scales, q4, scene->opacity_logit,
                                                                   n, cp, rule, out->tiles_touched, gt, ct, gpc));
      else
        ODIN_CUDA(odin_launch(ctx, false, project_cull_kernel<false>, dim3((n + 255) / 256), dim3(256), 0, st, scene->means,
                              scene->log_scales, q4, scene->opacity_logit,
                                                                    n, cp, rule, out->tiles_touched, gt, ct, gpc));
    }
    OdinKernelScope ks(ctx, K_PROJECT_SCAN, st);
    LAUNCH(false, false);
  }
#undef LAUNCH
  if (out->capacity == 0) return odin_launch_status();
  const uint32_t blocks_cap = (out->capacity + 127) / 128;
  const uint32_t grid = blocks_cap < (uint32_t)ctx->sm_count * 16 ? blocks_cap : (uint32_t)ctx->sm_count * 16;
  OdinKernelScope ks(ctx, K_PROJECT_ROWS, st);
#define LAUNCH(D)                                                                                                      \
  ODIN_CUDA(odin_launch(ctx, true, project_rows_kernel<D>, dim3(grid), dim3(128), 0, st, scene->means,                 \
                        scene->log_scales, q4, scene->opacity_logit, scene->sh, cp, rule, *out, n))
  switch (scene->sh_degree) {
    case 0: LAUNCH(0); break;
    case 1: LAUNCH(1); break;
    case 2: LAUNCH(2); break;
    default: LAUNCH(3); break;
  }
#undef LAUNCH
  return odin_launch_status();
}
