// Rendering phase: front-to-back alpha compositing.  Head kernel: one WARP per 16x16 tile, eight pixels per lane (see
// blend.cuh), the tile's sorted rows staged 32 at a time through shared memory, warp-ballot early exit once every
// pixel of the tile has terminated; per row and lane the x-dependent terms are computed once, each pixel costs two
// fused multiply-adds, one ex2 (the exponent is kept in base 2 with the opacity folded in) and the blend.  Tiles still live after BLEND_HEAD entries are finished by the tail
// kernel (eight warps per tile, rows staged 256 at a time).  Also the L1 image loss.
#include "blend.cuh"

namespace {

__global__ void __launch_bounds__(BLEND_THREADS, 7)  // 7 blocks = 28 warps per SM: the kernel is latency-bound
render_fwd_kernel(const float2* __restrict__ xy, const float4* __restrict__ conic_o, const float* __restrict__ rgb,
                  const uint32_t* __restrict__ vals, const uint2* __restrict__ ranges, int W, int H, int TX, int n_tiles,
                  float bg0, float bg1, float bg2, float alpha_min, float alpha_max, float t_min, float* __restrict__ out,
                  float* __restrict__ final_T, uint32_t* __restrict__ n_contrib, uint32_t* __restrict__ tile_more,
                  uint32_t* __restrict__ ticket, uint32_t row_cap, uint32_t* __restrict__ tail_queue,
                  uint32_t* __restrict__ bwd_queue) {
  odin_after_predecessor();
  __shared__ BlendRow s_row[BLEND_WARPS][32];
  __shared__ float s_blue[BLEND_WARPS][32];
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const float l2amin = log2f(alpha_min);
  // Warps never synchronise with each other.  Each one keeps taking tiles from a ticket counter until none is left:
  // lists differ in length by orders of magnitude between tiles, and a fixed tile-to-warp map would leave most of the
  // GPU idle while the longest ones finish.
  while (true) {
  int tile = 0;
  if (lane == 0) tile = (int)atomicAdd(ticket, 1u);
  tile = __shfl_sync(0xffffffffu, tile, 0);
  if (tile >= n_tiles) return;
  const int tx = tile % TX, ty = tile / TX;
  const int px = tx * 16 + (int)(lane & 15);
  const int py0 = ty * 16 + (int)(lane >> 4);
  const float fx = (float)px + 0.5f, fy0 = (float)py0 + 0.5f;
  const float tile_x0 = (float)(tx * 16), tile_y0 = (float)(ty * 16);
  const uint2 rg = ranges[tile];
  const uint32_t start = rg.x;
  const uint32_t end = min(rg.y, rg.x + BLEND_HEAD);

  float T[BLEND_SLOTS], C0[BLEND_SLOTS], C1[BLEND_SLOTS], C2[BLEND_SLOTS];
  uint32_t last[BLEND_SLOTS];
  uint32_t live = 0;  // bit s: pixel of slot s still accumulating
#pragma unroll
  for (int s = 0; s < BLEND_SLOTS; ++s) {
    T[s] = 1.f; C0[s] = C1[s] = C2[s] = 0.f; last[s] = 0;
    if (px < W && py0 + 2 * s < H) live |= 1u << s;
  }
  const uint32_t inside = live;
  uint32_t n_eval = 0;  // rows evaluated for this tile: the class of its first segment in the backward pass

  for (uint32_t b = start; b < end; b += 32) {
    if (!__any_sync(0xffffffffu, live != 0)) break;
    const uint32_t i = b + lane;
    bool reach = false;
    if (i < end) {
      const uint32_t r = min(vals[i], row_cap - 1);  // in range whatever the list holds (e.g. after a timed-out sort)
      const float2 c = xy[r];
      BlendRow row;
      row.q0 = make_float4(c.x, c.y, rgb[3 * (size_t)r], rgb[3 * (size_t)r + 1]);
      const float4 co = conic_o[r];
      row.q1 = blend_stage_conic(co);
      s_row[warp][lane] = row;
      s_blue[warp][lane] = rgb[3 * (size_t)r + 2];
      reach = blend_reaches_tile(c.x, c.y, co.x, co.y, co.z, blend_power_cut(alpha_min, co.w), tile_x0 + 0.5f,
                                 tile_y0 + 0.5f);
    }
    // warp-uniform: only the rows whose ellipse reaches the tile are evaluated, in list order
    uint32_t rows = __ballot_sync(0xffffffffu, reach);
    n_eval += __popc(rows);
    __syncwarp();
    while (rows) {
      const int j = __ffs(rows) - 1;
      rows &= rows - 1;
      const float4 q0 = s_row[warp][j].q0, q1 = s_row[warp][j].q1;
      const float blue = s_blue[warp][j];
      float h0, h1, h2;
      blend_x_terms(q1, q0.x - fx, h0, h1, h2);
      const float dy0 = q0.y - fy0;
      const uint32_t ord = (b - start) + j + 1;
      // the eight exponents first (independent, they overlap in the pipeline), then test and blend slot by slot
      float power[BLEND_SLOTS];
#pragma unroll
      for (int s = 0; s < BLEND_SLOTS; ++s) power[s] = blend_power(h0, h1, h2, dy0 - (float)(2 * s));
#pragma unroll
      for (int s = 0; s < BLEND_SLOTS; ++s) {
        if (blend_passes(power[s], q1.w, l2amin) && (live >> s & 1u)) {
          const float alpha = fminf(alpha_max, blend_ex2(power[s]));
          const float w = alpha * T[s];
          const float Tn = T[s] - w;
          if (Tn < t_min) {
            live &= ~(1u << s);
          } else {
            C0[s] = fmaf(q0.z, w, C0[s]); C1[s] = fmaf(q0.w, w, C1[s]); C2[s] = fmaf(blue, w, C2[s]);
            T[s] = Tn;
            last[s] = ord;
          }
        }
      }
    }
    __syncwarp();
  }
  // the tail kernel takes over when entries remain and some pixel is still live
  const bool more = (rg.y > end) && __any_sync(0xffffffffu, live != 0);
  if (lane == 0) {
    const uint32_t bc = blend_bwd_class(n_eval);
    bwd_queue[bc * (uint32_t)n_tiles + atomicAdd(ticket + 8 + bc, 1u)] = (uint32_t)tile;
    tile_more[tile] = more ? 1u : 0u;
    if (more) {  // queue of the tail kernel, longest lists first (four classes)
      const uint32_t len = rg.y - rg.x;
      const uint32_t cls = len > 8 * BLEND_HEAD ? 0u : (len > 4 * BLEND_HEAD ? 1u : (len > 2 * BLEND_HEAD ? 2u : 3u));
      tail_queue[cls * (uint32_t)n_tiles + atomicAdd(ticket + 4 + cls, 1u)] = (uint32_t)tile;
    }
  }
  const size_t plane = (size_t)W * H;
#pragma unroll
  for (int s = 0; s < BLEND_SLOTS; ++s) {
    const int py = py0 + 2 * s;
    if (inside >> s & 1u) {
      const size_t pix = (size_t)py * W + px;
      const float tb = more ? 0.f : T[s];  // the background is added by whoever finishes the pixel
      out[pix] = C0[s] + tb * bg0;
      out[plane + pix] = C1[s] + tb * bg1;
      out[2 * plane + pix] = C2[s] + tb * bg2;
      final_T[pix] = T[s];
      n_contrib[pix] = last[s] | ((more && !(live >> s & 1u)) ? BLEND_DONE_BIT : 0u);
    }
  }
  __syncwarp();  // the staging arrays are reused by the next tile
  }
}

// Tail: one block of 256 threads per tile that the head kernel left unfinished, one pixel per thread, rows staged 256
// at a time.  Thread t handles column t % 16 and row t / 16 = 2 s + (row inside the slot pair), as in the head kernel.
// For every batch the block takes a segment slot and stores there, per pixel, the transmittance before the batch and
// the colour the batch added; when the tile is finished the stored colours are summed from the last record to the
// first into "colour still to come" (see blend.cuh): the backward pass starts its segments from these records.
__global__ void __launch_bounds__(BLEND_TAIL_THREADS, 3)
render_fwd_tail_kernel(const float2* __restrict__ xy, const float4* __restrict__ conic_o, const float* __restrict__ rgb,
                       const uint32_t* __restrict__ vals, const uint2* __restrict__ ranges, int W, int H, int TX,
                       float bg0, float bg1, float bg2, float alpha_min, float alpha_max, float t_min,
                       float* __restrict__ out, float* __restrict__ final_T, uint32_t* __restrict__ n_contrib,
                       uint32_t* __restrict__ tile_first, uint32_t* __restrict__ header,
                       const uint32_t* __restrict__ tail_queue, int n_tiles, uint2* __restrict__ seg_tile,
                       uint2* __restrict__ seg_link, BlendRecord* __restrict__ ckpt, uint32_t seg_cap, int* status,
                       uint32_t row_cap) {
  odin_after_predecessor();  // launched behind the head kernel
  __shared__ BlendRow s_row[BLEND_TAIL_THREADS];
  __shared__ uint32_t s_item;
  // The duration of this kernel is that of its longest list (a chain of batches), so the blocks take the tiles the head
  // kernel queued by ticket, the class of the longest lists first.
  const uint32_t c0 = header[4], c1 = header[5], c2 = header[6], c3 = header[7];
  while (true) {
  __syncthreads();  // the previous tile's readers of shared memory are done
  if (threadIdx.x == 0) s_item = atomicAdd(header + 3, 1u);
  __syncthreads();
  uint32_t item = s_item;
  if (item >= c0 + c1 + c2 + c3) return;
  uint32_t cls = 0;
  if (item >= c0) { item -= c0; cls = 1; if (item >= c1) { item -= c1; cls = 2; if (item >= c2) { item -= c2; cls = 3; } } }
  const int tile = (int)min(tail_queue[cls * (uint32_t)n_tiles + item], (uint32_t)n_tiles - 1);
  __shared__ float s_blue[BLEND_TAIL_THREADS];
  __shared__ uint32_t s_ord[BLEND_TAIL_THREADS];  // 1-based position of the row in the tile's list
  // the row's colour in double, converted once when the row is staged: the per-batch sums that feed the records are kept
  // in double, and a conversion per (pixel, row) pair made the conversion unit the limit of tiles with long dense lists
  __shared__ double s_cd[BLEND_TAIL_THREADS][3];
  __shared__ uint32_t s_wcnt[BLEND_TAIL_THREADS / 32];
  __shared__ uint32_t s_slot;
  const int tx = tile % TX, ty = tile / TX;
  const int lx = threadIdx.x & 15, ly = threadIdx.x >> 4;
  const int px = tx * 16 + lx, py = ty * 16 + ly;
  const bool inside = px < W && py < H;
  const float fx = (float)px + 0.5f;
  const float fy0 = (float)(ty * 16 + (ly & 1)) + 0.5f;
  const float slot2 = (float)(2 * (ly >> 1));
  const float l2amin = log2f(alpha_min);
  const uint2 rg = ranges[tile];
  const uint32_t start = rg.x, end = rg.y;
  const size_t pix = (size_t)py * W + px, plane = (size_t)W * H;
  float T = 1.f, C0 = 0.f, C1 = 0.f, C2 = 0.f;
  uint32_t last = 0;
  bool done = true;
  if (inside) {
    T = final_T[pix];
    C0 = out[pix]; C1 = out[plane + pix]; C2 = out[2 * plane + pix];
    const uint32_t nc = n_contrib[pix];
    last = nc & ~BLEND_DONE_BIT;
    done = (nc & BLEND_DONE_BIT) != 0;
  }
  const float tile_x0 = (float)(tx * 16) + 0.5f, tile_y0 = (float)(ty * 16) + 0.5f;
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t first_slot = 0, prev_slot = 0;  // 1 + slot; 0 = none
  uint32_t k = 1;                          // segment index: the batch starts at list entry k * BLEND_HEAD
  for (uint32_t b = start + BLEND_HEAD; b < end; b += BLEND_TAIL_THREADS, ++k) {
    if (__syncthreads_count(done) == BLEND_TAIL_THREADS) break;
    // stage 256 entries and keep, in list order, only the rows whose ellipse reaches the tile
    const uint32_t i = b + threadIdx.x;
    BlendRow row;
    float bp = 0.f;
    bool reach = false;
    if (i < end) {
      const uint32_t r = min(vals[i], row_cap - 1);
      const float2 c = xy[r];
      row.q0 = make_float4(c.x, c.y, rgb[3 * (size_t)r], rgb[3 * (size_t)r + 1]);
      const float4 co = conic_o[r];
      row.q1 = blend_stage_conic(co);
      bp = rgb[3 * (size_t)r + 2];
      reach = blend_reaches_tile(c.x, c.y, co.x, co.y, co.z, blend_power_cut(alpha_min, co.w), tile_x0, tile_y0);
    }
    const uint32_t wm = __ballot_sync(0xffffffffu, reach);
    if (lane == 0) s_wcnt[warp] = __popc(wm);
    if (threadIdx.x == 0) s_slot = atomicAdd(header + 2, 1u);
    __syncthreads();
    // the record of segment k: the transmittance before entry k * BLEND_HEAD (where the backward replay of segment
    // k - 1 begins) and, once the batch is done, the colour its entries added
    const uint32_t slot = s_slot;
    const bool have = slot < seg_cap;
    if (have) {
      if (threadIdx.x == 0) {
        seg_tile[slot] = make_uint2((uint32_t)tile, k);
        seg_link[slot] = make_uint2(0u, prev_slot);
        if (prev_slot) seg_link[prev_slot - 1].x = slot + 1;
      }
      if (!first_slot) first_slot = slot + 1;
      prev_slot = slot + 1;
    } else if (threadIdx.x == 0) {
      odin_set_error(status, ODIN_ERR_CAPACITY);  // the backward pass will miss this tile's later segments
    }
    const float T_start = T;
    double D0 = 0.0, D1 = 0.0, D2 = 0.0;
    int cnt = 0, pos = __popc(wm & ((1u << lane) - 1u));
#pragma unroll
    for (int w = 0; w < BLEND_TAIL_THREADS / 32; ++w) {
      const int c = (int)s_wcnt[w];
      if (w < (int)warp) pos += c;
      cnt += c;
    }
    if (reach) {
      s_row[pos] = row;
      s_blue[pos] = bp;
      s_ord[pos] = i - start + 1;
      s_cd[pos][0] = (double)row.q0.z; s_cd[pos][1] = (double)row.q0.w; s_cd[pos][2] = (double)bp;
    }
    __syncthreads();
    if (!done) {
      // four rows at a time: their exponents and skip tests are independent (a single pixel per thread has no other
      // source of instruction-level parallelism), the blends are then applied in order
      for (int j = 0; j < cnt && !done; j += 4) {
        float pw[4], cr[4], cg[4], cb[4];
        bool pass[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int ju = min(j + u, cnt - 1);
          const float4 q0 = s_row[ju].q0, q1 = s_row[ju].q1;
          float h0, h1, h2;
          blend_x_terms(q1, q0.x - fx, h0, h1, h2);
          pw[u] = blend_power(h0, h1, h2, (q0.y - fy0) - slot2);
          pass[u] = (j + u < cnt) && blend_passes(pw[u], q1.w, l2amin);
          cr[u] = q0.z; cg[u] = q0.w; cb[u] = s_blue[ju];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          if (pass[u] && !done) {
            const float alpha = fminf(alpha_max, blend_ex2(pw[u]));
            const float w = alpha * T;
            const float Tn = T - w;
            if (Tn < t_min) {
              done = true;
            } else {
              // the image keeps its one sequential sum per pixel (so it does not depend on where the batches fall);
              // the per-batch sums, in double, only feed the records
              C0 = fmaf(cr[u], w, C0); C1 = fmaf(cg[u], w, C1); C2 = fmaf(cb[u], w, C2);
              const double wd = (double)w;
              D0 = fma(s_cd[j + u][0], wd, D0); D1 = fma(s_cd[j + u][1], wd, D1); D2 = fma(s_cd[j + u][2], wd, D2);
              T = Tn;
              last = s_ord[j + u];
            }
          }
        }
      }
    }
    if (have) {
      BlendRecord rec;
      rec.T = T_start; rec.pad = 0.f; rec.S0 = D0; rec.S1 = D1; rec.S2 = D2;
      ckpt[(size_t)slot * BLEND_TAIL_THREADS + threadIdx.x] = rec;
    }
  }
  if (inside) {
    out[pix] = C0 + T * bg0;
    out[plane + pix] = C1 + T * bg1;
    out[2 * plane + pix] = C2 + T * bg2;
    final_T[pix] = T;
    n_contrib[pix] = last;
  }
  // colour added by a segment -> colour still to come at its start, summed from the tile's last record to its first
  // (each thread rewrites its own words; the links were written by thread 0 before barriers every thread has passed)
  __syncthreads();
  if (threadIdx.x == 0) tile_first[tile] = first_slot;
  double S0 = (double)T * (double)bg0, S1 = (double)T * (double)bg1, S2 = (double)T * (double)bg2;
  for (uint32_t s1 = prev_slot; s1 != 0;) {
    BlendRecord* c = ckpt + (size_t)(s1 - 1) * BLEND_TAIL_THREADS + threadIdx.x;
    S0 += c->S0; S1 += c->S1; S2 += c->S2;
    c->S0 = S0; c->S1 = S1; c->S2 = S2;
    s1 = seg_link[s1 - 1].y;
  }
  }
}

// Measurement aid (not part of the view step): how many (pixel, list entry) pairs the compositing of a view consists
// of.  One block per tile, one pixel per thread, the same tests as the forward kernels.  counts[0]: pairs inside the
// pixel's walked prefix (entries up to the last one that contributed to the pixel); counts[1]: those that blend (pass
// the skip tests): the pairs the backward pass differentiates.
__global__ void __launch_bounds__(256)
count_pairs_kernel(const float2* __restrict__ xy, const float4* __restrict__ conic_o, const uint32_t* __restrict__ vals,
                   const uint2* __restrict__ ranges, int W, int H, int TX, float alpha_min, float alpha_max,
                   const uint32_t* __restrict__ n_contrib, uint32_t row_cap, unsigned long long* __restrict__ counts) {
  const int tile = blockIdx.x;
  const int px = (tile % TX) * 16 + (int)(threadIdx.x & 15), py = (tile / TX) * 16 + (int)(threadIdx.x >> 4);
  unsigned long long walked = 0, blended = 0;
  if (px < W && py < H) {
    const uint32_t start = ranges[tile].x;
    const uint32_t n = min(n_contrib[(size_t)py * W + px], ranges[tile].y - start);
    const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
    walked = n;
    for (uint32_t k = 0; k < n; ++k) {
      const uint32_t r = min(vals[start + k], row_cap - 1);
      const float2 c = xy[r];
      const float4 q = conic_o[r];
      const float dx = c.x - fx, dy = c.y - fy;
      const float power = -0.5f * (q.x * dx * dx + q.z * dy * dy) - q.y * dx * dy;
      if (power > 0.f) continue;
      if (fminf(alpha_max, q.w * __expf(power)) < alpha_min) continue;
      ++blended;
    }
  }
  for (int o = 16; o > 0; o >>= 1) {
    walked += __shfl_xor_sync(0xffffffffu, walked, o);
    blended += __shfl_xor_sync(0xffffffffu, blended, o);
  }
  if ((threadIdx.x & 31) == 0 && walked) {
    atomicAdd(&counts[0], walked);
    atomicAdd(&counts[1], blended);
  }
}

constexpr int LB = 256;

__global__ void __launch_bounds__(LB)
l1_loss_kernel(const float* __restrict__ out, const float* __restrict__ target, size_t count, float inv, double* loss_acc,
               float* __restrict__ dL, double inv_count, float* __restrict__ loss, size_t vec4) {
  odin_after_predecessor();
  // vec4: number of leading float4 groups (0 when the three images are not 16-byte aligned); the rest one by one
  float acc = 0.f;
  const size_t tid = (size_t)blockIdx.x * LB + threadIdx.x, stride = (size_t)gridDim.x * LB;
  for (size_t i = tid; i < vec4; i += stride) {
    const float4 a = reinterpret_cast<const float4*>(out)[i], b = reinterpret_cast<const float4*>(target)[i];
    const float d0 = a.x - b.x, d1 = a.y - b.y, d2 = a.z - b.z, d3 = a.w - b.w;
    acc += (fabsf(d0) + fabsf(d1)) + (fabsf(d2) + fabsf(d3));
    reinterpret_cast<float4*>(dL)[i] = make_float4(d0 > 0.f ? inv : (d0 < 0.f ? -inv : 0.f), d1 > 0.f ? inv : (d1 < 0.f ? -inv : 0.f),
                                                   d2 > 0.f ? inv : (d2 < 0.f ? -inv : 0.f), d3 > 0.f ? inv : (d3 < 0.f ? -inv : 0.f));
  }
  for (size_t i = vec4 * 4 + tid; i < count; i += stride) {
    const float d = out[i] - target[i];
    acc += fabsf(d);
    dL[i] = d > 0.f ? inv : (d < 0.f ? -inv : 0.f);
  }
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  __shared__ float s[LB / 32];
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double t = 0;
    for (int i = 0; i < LB / 32; ++i) t += (double)s[i];
    atomicAdd(loss_acc, t);
    // the block that arrives last turns the sum into the mean (no second launch)
    __threadfence();
    uint32_t* arrivals = reinterpret_cast<uint32_t*>(loss_acc + 1);
    if (atomicAdd(arrivals, 1u) == gridDim.x - 1u) {
      __threadfence();
      *loss = (float)(atomicAdd(loss_acc, 0.0) * inv_count);
    }
  }
}

}  // namespace

extern "C" int odin_render_workspace_bytes(const odin_ctx* ctx, int width, int height, size_t* bytes) {
  if (!ctx || !bytes) return ODIN_ERR_NULL;
  if (width <= 0 || height <= 0 || width > 16384 || height > 16384) return ODIN_ERR_INVALID_ARG;
  *bytes = blend_ws_bytes(width, height);
  return ODIN_OK;
}

extern "C" int odin_render_fwd(odin_ctx* ctx, const odin_projected* proj, const uint32_t* d_vals,
                               const uint32_t* d_tile_ranges, const odin_camera* cam, float* d_rgb, float* d_final_T,
                               uint32_t* d_n_contrib, void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || !proj || !d_tile_ranges || !d_rgb || !d_final_T || !d_n_contrib) return ODIN_ERR_NULL;
  const int rc = odin_check_camera(cam);
  if (rc != ODIN_OK) return rc;
  if (proj->capacity > 0 && (!proj->xy || !proj->conic_opacity || !proj->rgb || !d_vals)) return ODIN_ERR_NULL;
  if (!odin_aligned(proj->xy, 8) || !odin_aligned(proj->conic_opacity, 16) || !odin_aligned(d_tile_ranges, 8))
    return ODIN_ERR_INVALID_ARG;
  const int TX = (cam->width + 15) / 16, TY = (cam->height + 15) / 16;
  const int n_tiles = TX * TY;
  if (!ws || !odin_aligned(ws, 256) || ws_bytes < blend_ws_bytes(cam->width, cam->height)) return ODIN_ERR_WORKSPACE;
  const BlendWs L = blend_ws_layout(n_tiles, blend_ws_segments(n_tiles, ws_bytes));
  char* base = reinterpret_cast<char*>(ws);
  uint32_t* header = reinterpret_cast<uint32_t*>(base);
  uint32_t* tile_first = reinterpret_cast<uint32_t*>(base + L.tile_first);
  uint32_t* tail_queue = reinterpret_cast<uint32_t*>(base + L.queue);
  cudaStream_t st = (cudaStream_t)stream;
  ODIN_CUDA(odin_zero(ctx, header, 96, st));  // tickets, segments taken, the class counts of the two queues
  {
    OdinKernelScope ks(ctx, K_FWD, st);
    const int blocks_all = (n_tiles + BLEND_WARPS - 1) / BLEND_WARPS;
    const int blocks = blocks_all < ctx->sm_count * 8 ? blocks_all : ctx->sm_count * 8;  // resident warps pull tiles
    ODIN_CUDA(odin_launch(ctx, false, render_fwd_kernel, dim3(blocks), dim3(BLEND_THREADS), 0, st,
        reinterpret_cast<const float2*>(proj->xy), reinterpret_cast<const float4*>(proj->conic_opacity), proj->rgb, d_vals,
        reinterpret_cast<const uint2*>(d_tile_ranges), cam->width, cam->height, TX, n_tiles, cam->bg[0], cam->bg[1],
        cam->bg[2], ctx->cfg.alpha_min, ctx->cfg.alpha_max, ctx->cfg.t_min, d_rgb, d_final_T, d_n_contrib, tile_first,
        header, proj->capacity, tail_queue, reinterpret_cast<uint32_t*>(base + L.bwd_queue)));
  }
  OdinKernelScope ks(ctx, K_FWD_TAIL, st);
  const int tail_blocks = n_tiles < ctx->sm_count * 3 ? n_tiles : ctx->sm_count * 3;  // resident blocks pull tiles
  ODIN_CUDA(odin_launch(ctx, true, render_fwd_tail_kernel, dim3(tail_blocks), dim3(BLEND_TAIL_THREADS), 0, st,
      reinterpret_cast<const float2*>(proj->xy), reinterpret_cast<const float4*>(proj->conic_opacity), proj->rgb, d_vals,
      reinterpret_cast<const uint2*>(d_tile_ranges), cam->width, cam->height, TX, cam->bg[0], cam->bg[1], cam->bg[2],
      ctx->cfg.alpha_min, ctx->cfg.alpha_max, ctx->cfg.t_min, d_rgb, d_final_T, d_n_contrib, tile_first, header,
      tail_queue, n_tiles, reinterpret_cast<uint2*>(base + L.seg_tile), reinterpret_cast<uint2*>(base + L.seg_link),
      reinterpret_cast<BlendRecord*>(base + L.ckpt), L.segments, ctx->d_status, proj->capacity));
  return odin_launch_status();
}

extern "C" int odin_count_blend_pairs(odin_ctx* ctx, const odin_projected* proj, const uint32_t* d_vals,
                                      const uint32_t* d_tile_ranges, const odin_camera* cam, const uint32_t* d_n_contrib,
                                      uint64_t* d_counts, void* stream) {
  if (!ctx || !proj || !d_tile_ranges || !d_n_contrib || !d_counts) return ODIN_ERR_NULL;
  const int rc = odin_check_camera(cam);
  if (rc != ODIN_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(d_counts, 0, 16, st));
  if (proj->capacity == 0) return ODIN_OK;
  if (!proj->xy || !proj->conic_opacity || !d_vals) return ODIN_ERR_NULL;
  const int TX = (cam->width + 15) / 16, TY = (cam->height + 15) / 16;
  count_pairs_kernel<<<TX * TY, 256, 0, st>>>(
      reinterpret_cast<const float2*>(proj->xy), reinterpret_cast<const float4*>(proj->conic_opacity), d_vals,
      reinterpret_cast<const uint2*>(d_tile_ranges), cam->width, cam->height, TX, ctx->cfg.alpha_min, ctx->cfg.alpha_max,
      d_n_contrib, proj->capacity, reinterpret_cast<unsigned long long*>(d_counts));
  return odin_launch_status();
}

extern "C" int odin_l1_loss(odin_ctx* ctx, const float* d_rgb, const float* d_target, int width, int height,
                            float* d_loss, float* d_dL_drgb, void* stream) {
  if (!ctx || !d_rgb || !d_target || !d_loss || !d_dL_drgb) return ODIN_ERR_NULL;
  if (width <= 0 || height <= 0) return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t count = (size_t)3 * width * height;
  // the accumulator (8 bytes) and the arrival counter of the blocks (4 bytes behind it) live behind the status word in
  // the context's device block
  double* acc = reinterpret_cast<double*>(reinterpret_cast<char*>(ctx->d_status) + 64);
  ODIN_CUDA(odin_zero(ctx, acc, 16, st));
  const bool aligned = odin_aligned(d_rgb, 16) && odin_aligned(d_target, 16) && odin_aligned(d_dL_drgb, 16);
  const size_t vec4 = aligned ? count / 4 : 0;
  size_t blocks = (count / 4 + LB - 1) / LB + 1;
  if (blocks > (size_t)ctx->sm_count * 8) blocks = (size_t)ctx->sm_count * 8;
  OdinKernelScope ks(ctx, K_L1, st);
  ODIN_CUDA(odin_launch(ctx, false, l1_loss_kernel, dim3((unsigned)blocks), dim3(LB), 0, st, d_rgb, d_target, count, (float)(1.0 / (double)count), acc, d_dL_drgb,
                                                  1.0 / (double)count, d_loss, vec4));
  return odin_launch_status();
}
