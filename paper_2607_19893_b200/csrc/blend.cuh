// Shared by the compositing kernel and its backward: pixel mapping of a warp over a 16x16 tile and the per-row
// quantities that both must evaluate with exactly the same arithmetic (so that skip / clamp decisions agree).
//
// One warp owns one tile.  Lane l handles column x = l % 16 and, for slot s = 0..7, row y = 2 s + l / 16: a slot is two
// adjacent pixel rows of the tile, so "does any lane of the warp touch this row in slot s" is spatially coherent and
// worth a warp-uniform branch.  Per row of the sorted list the lane computes once
//     dx = u - x,  h0 = sA dx^2 + lo,  h1 = sB dx,  h2 = sC          (see BlendRow)
// and per slot only  p = h0 + dy (h1 + h2 dy)  (two fused multiply-adds), alpha = min(alpha_max, 2^p).
#pragma once
#include "common.cuh"

// Long lists.  Forward: a tile whose pixels are still live after BLEND_HEAD list entries is finished by a second kernel
// that gives the tile eight warps (one pixel per thread): a single warp walking a list of thousands of entries would be
// the tail of the whole launch.  The per-pixel state travels through the output images.  Both kernels evaluate dy as
// (v - (y0 + 0.5)) - 2 s with y0 the first row of the lane's slot pair, so a pixel sees bit-identical power / alpha in
// either.
// Backward: the list of a tile is cut into SEGMENTS of BLEND_HEAD entries that are replayed independently, one warp
// each, all in one launch.  What a segment needs is the state of every pixel at its END: the transmittance and the
// colour still to come behind it.  The forward tail kernel leaves exactly that in the workspace: for every BLEND_HEAD
// entries it walks it takes a segment slot from a counter and stores, for its 256 pixels, the transmittance before
// those entries and the colour they added; when the tile is finished it walks its slots from the last to the first
// and replaces "colour added" by the running sum "colour still to come" (summed from the back, small terms first, as
// the sequential replay would: a difference final colour - colour so far would lose the small suffixes of nearly
// saturated pixels to rounding).  So the backward pass has no sequential tail at all, and the workspace of
// odin_render_bwd must be the one the odin_render_fwd of the same view used.
constexpr uint32_t BLEND_HEAD = 256;
constexpr uint32_t BLEND_DONE_BIT = 0x80000000u;  // in n_contrib while a tile is between the two forward kernels
constexpr int BLEND_TAIL_THREADS = 256;

// Workspace of the render calls (every region 256-byte aligned):
//   [256 B: u32 [0] tile ticket of the forward head kernel, [1] work ticket of the backward kernel, [2] segments taken,
//           [3] ticket of the forward tail kernel, [4..7] tiles queued for it in each of four classes of list length,
//           [8..23] tiles in each of the sixteen classes of the backward kernel's work order]
//   [tile_first: u32 x tiles   forward head: 1 = the tail kernel must continue; forward tail: 1 + slot of the tile's
//                              segment that starts at entry BLEND_HEAD (0 = none)]
//   [queue: u32 x 4 x tiles    tiles the forward tail kernel must finish, one region per class, longest lists first]
//   [bwd_queue: u32 x 16 x tiles  all tiles in sixteen classes of rows evaluated: work order of the backward kernel]
//   [seg_tile: uint2 x S       (tile, k): the slot holds the state before entry k * BLEND_HEAD of that tile]
//   [seg_link: uint2 x S       1 + slot of the same tile's segment k + 1, of segment k - 1 (0 = none)]
//   [ckpt: BlendRecord x 256 x S   per pixel (thread t = 16 * row + column of the tile): T, colour to come (3)]
// S, the number of segment slots, follows from the size of the workspace the caller passes; the minimum size holds
// 2 x tiles + 4096 of them.
// Work order of the backward kernel over the first segments of the tiles: sixteen classes by the number of rows the
// forward head kernel evaluated for the tile (those whose ellipse reaches it: the backward pass evaluates the same
// rows), most first; the head kernel files a tile when it finishes it.  The warps take items by ticket; in image order
// the expensive first segments of tiles late in the image were started last and the warps finished, on average, at
// 76 % of the kernel's duration.
constexpr int BLEND_BWD_CLASSES = 16;
__host__ __device__ inline uint32_t blend_bwd_class(uint32_t rows_evaluated) {
  const uint32_t c = rows_evaluated >> 4;  // at most BLEND_HEAD = 256 rows: 0 .. 16
  return c >= (uint32_t)BLEND_BWD_CLASSES ? 0u : (uint32_t)BLEND_BWD_CLASSES - 1u - c;
}

constexpr size_t BLEND_WS_HEADER = 256;
// The colour is kept in double: the backward pass needs its product with the pixel's incoming gradient, a sum over
// the three channels that cancels when the gradient's signs differ (an L1 loss: +-1/N), and a float colour would
// make that product wrong in its leading digits for every row of the segment at once.
struct BlendRecord {
  float T, pad;
  double S0, S1, S2;
};
static_assert(sizeof(BlendRecord) == 32, "record layout");
constexpr size_t BLEND_SEG_BYTES = 8 + 8 + 256 * sizeof(BlendRecord);
struct BlendWs {
  size_t tile_first, queue, bwd_queue, seg_tile, seg_link, ckpt, total;
  uint32_t segments;
};
static inline size_t blend_align(size_t x) { return (x + 255) / 256 * 256; }
static inline size_t blend_ws_flags_bytes(int n_tiles) { return BLEND_WS_HEADER + blend_align((size_t)n_tiles * 4); }
static inline BlendWs blend_ws_layout(int n_tiles, uint32_t segments) {
  BlendWs L;
  L.segments = segments;
  L.tile_first = BLEND_WS_HEADER;
  L.queue = L.tile_first + blend_align((size_t)n_tiles * 4);
  L.bwd_queue = L.queue + blend_align((size_t)n_tiles * 16);
  L.seg_tile = L.bwd_queue + blend_align((size_t)n_tiles * 4 * BLEND_BWD_CLASSES);
  L.seg_link = L.seg_tile + blend_align((size_t)segments * 8);
  L.ckpt = L.seg_link + blend_align((size_t)segments * 8);
  L.total = L.ckpt + (size_t)segments * 256 * sizeof(BlendRecord);
  return L;
}
static inline uint32_t blend_min_segments(int n_tiles) { return 2u * (uint32_t)n_tiles + 4096u; }
static inline size_t blend_ws_bytes(int width, int height) {
  const int n_tiles = ((width + 15) / 16) * ((height + 15) / 16);
  return blend_ws_layout(n_tiles, blend_min_segments(n_tiles)).total;
}
// the largest number of segment slots whose layout fits into ws_bytes (at least the minimum, which the caller checked)
static inline uint32_t blend_ws_segments(int n_tiles, size_t ws_bytes) {
  uint32_t s = blend_min_segments(n_tiles);
  const size_t fixed = blend_ws_layout(n_tiles, 0).total + 3 * 256;
  if (ws_bytes > fixed) {
    const size_t fit = (ws_bytes - fixed) / BLEND_SEG_BYTES;
    if (fit > s) s = (uint32_t)(fit < 0x7fffffffu ? fit : 0x7fffffffu);
  }
  while (blend_ws_layout(n_tiles, s).total > ws_bytes && s > blend_min_segments(n_tiles)) --s;
  return s;
}

constexpr int BLEND_SLOTS = 8;          // pixels per lane
constexpr int BLEND_WARPS = 4;          // tiles per block (warps do not synchronise with each other)
constexpr int BLEND_THREADS = 32 * BLEND_WARPS;

// One row of the tile's list as staged in shared memory.  The exponent is evaluated in base 2 with the opacity folded
// in: with sA = -A log2(e) / 2, sB = -B log2(e), sC = -C log2(e) / 2 and lo = log2(opacity),
//     p = sA dx^2 + sB dx dy + sC dy^2 + lo = log2(opacity * exp(power)),   alpha = min(alpha_max, 2^p),
// so a pixel costs two fused multiply-adds, the tests, one ex2 and one min.  The skip test "alpha < alpha_min" is
// p < log2(alpha_min), a constant of the launch, and "power > 0" is p > lo; a pixel that fails never reaches ex2.  All
// blend kernels stage rows through blend_stage_row and form p through blend_x_terms / blend_power, so they agree bit
// for bit on every (pixel, row) pair.  An opacity of 0 gives lo = -inf (nothing passes).
struct BlendRow {
  float4 q0;       // u, v, r, g
  float4 q1;       // sA, sB, sC, lo
};

constexpr float BLEND_LOG2E = 1.4426950408889634f;
constexpr float BLEND_LN2 = 0.6931471805599453f;

__device__ __forceinline__ float4 blend_stage_conic(float4 conic_o) {
  return make_float4(conic_o.x * (-0.5f * BLEND_LOG2E), conic_o.y * (-BLEND_LOG2E), conic_o.z * (-0.5f * BLEND_LOG2E),
                     log2f(conic_o.w));
}

// per row and lane: the terms of p that depend on the column only (dx = u - x)
__device__ __forceinline__ void blend_x_terms(const float4 q1, float dx, float& h0, float& h1, float& h2) {
  h0 = fmaf(q1.x * dx, dx, q1.w);
  h1 = q1.y * dx;
  h2 = q1.z;
}

__device__ __forceinline__ float blend_power(float h0, float h1, float h2, float dy) {
  return fmaf(dy, fmaf(h2, dy, h1), h0);
}

__device__ __forceinline__ bool blend_passes(float p, float lo, float l2amin) { return p <= lo && p >= l2amin; }

__device__ __forceinline__ float blend_ex2(float p) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(p));
  return y;
}

// Threshold of the natural exponent, power >= log(alpha_min / opacity), used by the tile test below when a row is
// staged.  An opacity of 0 gives +inf; an opacity below alpha_min gives a positive threshold (nothing passes).
__device__ __forceinline__ float blend_power_cut(float alpha_min, float opacity) { return logf(alpha_min / opacity); }

// Can the row pass the skip test at any pixel of the tile whose first pixel centre is (x_lo, y_lo)?  The set
// power >= cut is the ellipse q(dx, dy) = A dx^2 + 2 B dx dy + C dy^2 <= k, k = -2 cut, around the row's centre (u, v);
// the pixel centres of the tile lie in the rectangle [x_lo, x_lo + 15] x [y_lo, y_lo + 15].  q is convex, so its
// minimum over the rectangle is 0 if the centre lies inside and otherwise sits on one of the four edges, where it is
// the clamped one-dimensional minimiser.  The bound is widened by 1e-4 relative + 1e-3 + 2e-6 of the largest term any
// pixel of the tile can see (the rounding of this evaluation and of the per-pixel exponent is a few ulp of that term),
// so a row it rejects fails the per-pixel test everywhere in the tile and skipping it never changes a result.
// Evaluated once per (tile, row) by the thread that stages the row; anything that is not a proper ellipse is kept.
__device__ __forceinline__ bool blend_reaches_tile(float u, float v, float A, float B, float C, float cut, float x_lo,
                                                   float y_lo) {
  if (!(cut <= 0.f)) return false;  // opacity below alpha_min (cut > 0), zero (+inf) or not a number: nothing passes
  const float dxl = x_lo - u, dxh = dxl + 15.f, dyl = y_lo - v, dyh = dyl + 15.f;
  if (dxl <= 0.f && dxh >= 0.f && dyl <= 0.f && dyh >= 0.f) return true;
  if (!(A * C - B * B > 0.f) || !(A > 1e-30f) || !(C > 1e-30f) || !(A < 1e30f) || !(C < 1e30f)) return true;
  const float iA = __fdividef(1.f, A), iC = __fdividef(1.f, C);
  float qmin;
  {
    const float t0 = fminf(fmaxf(-B * dxl * iC, dyl), dyh), t1 = fminf(fmaxf(-B * dxh * iC, dyl), dyh);
    const float q0 = fmaf(t0, fmaf(C, t0, 2.f * B * dxl), A * dxl * dxl);
    const float q1 = fmaf(t1, fmaf(C, t1, 2.f * B * dxh), A * dxh * dxh);
    const float s0 = fminf(fmaxf(-B * dyl * iA, dxl), dxh), s1 = fminf(fmaxf(-B * dyh * iA, dxl), dxh);
    const float q2 = fmaf(s0, fmaf(A, s0, 2.f * B * dyl), C * dyl * dyl);
    const float q3 = fmaf(s1, fmaf(A, s1, 2.f * B * dyh), C * dyh * dyh);
    qmin = fminf(fminf(q0, q1), fminf(q2, q3));
  }
  const float mx = fmaxf(fabsf(dxl), fabsf(dxh)), my = fmaxf(fabsf(dyl), fabsf(dyh));
  const float big = A * mx * mx + 2.f * fabsf(B) * mx * my + C * my * my;
  const float bound = fmaf(-2.f * cut, 1.0001f, 1e-3f + 2e-6f * big);
  return !(qmin > bound);
}
