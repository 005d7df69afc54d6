// Shared by the compositing kernel and its backward: pixel mapping of a warp over a 16x16 tile and the per-row
// quantities that both must evaluate with exactly the same arithmetic (so that skip / clamp decisions agree).
//
// One warp owns one tile.  Lane l handles column x = l % 16 and, for slot s = 0..7, row y = 2 s + l / 16: a slot is two
// adjacent pixel rows of the tile, so "does any lane of the warp touch this row in slot s" is spatially coherent and
// worth a warp-uniform branch.  Per row of the sorted list the lane computes once
//     dx = u - x,  h0 = -A dx^2 / 2,  h1 = -B dx,  h2 = -C / 2
// and per slot only  power = h0 + dy (h1 + h2 dy)  (two fused multiply-adds), alpha = min(alpha_max, o * exp(power)).
#pragma once
#include "common.cuh"

// Long lists.  A tile whose pixels are still live after BLEND_HEAD list entries is finished by a second kernel that
// gives the tile eight warps (one pixel per thread): a single warp walking a list of thousands of entries would be the
// tail of the whole launch.  The per-pixel state travels through the output images (forward) or a workspace
// (backward).  Both kernels evaluate dy as (v - (y0 + 0.5)) - 2 s with y0 the first row of the lane's slot pair, so a
// pixel sees bit-identical power / alpha in either.
constexpr uint32_t BLEND_HEAD = 256;
constexpr uint32_t BLEND_DONE_BIT = 0x80000000u;  // in n_contrib while a tile is between the two kernels
constexpr int BLEND_TAIL_THREADS = 256;

// Workspace of the render calls:
//   [256 B: tile tickets of the forward ([0]) and backward ([1]) head kernels][tile flags u32 x tiles | 256-aligned]
//   [T, S0, S1, S2 planes, fp32 x pixels each]
constexpr size_t BLEND_WS_HEADER = 256;
static inline size_t blend_ws_flags_bytes(int n_tiles) { return BLEND_WS_HEADER + ((size_t)n_tiles * 4 + 255) / 256 * 256; }
static inline size_t blend_ws_bytes(int width, int height) {
  const int n_tiles = ((width + 15) / 16) * ((height + 15) / 16);
  return blend_ws_flags_bytes(n_tiles) + (size_t)16 * width * height;
}

constexpr int BLEND_SLOTS = 8;          // pixels per lane
constexpr int BLEND_WARPS = 4;          // tiles per block (warps do not synchronise with each other)
constexpr int BLEND_THREADS = 32 * BLEND_WARPS;

struct BlendRow {  // one row of the tile's list as staged in shared memory
  float4 q0;       // u, v, r, g
  float4 q1;       // conic A, B, C, opacity
};

__device__ __forceinline__ float blend_power(float h0, float h1, float h2, float dy) {
  return fmaf(dy, fmaf(h2, dy, h1), h0);
}

// The skip test "alpha = opacity * exp(power) < alpha_min" is taken on the exponent: power < log(alpha_min / opacity).
// The threshold is computed once per row when it is staged, so a pixel that fails costs two fused multiply-adds and
// two compares and never reaches ex2; all four blend kernels use this same form so that they agree on every pair.
// An opacity of 0 gives +inf (nothing passes); an opacity below alpha_min gives a positive threshold, which the
// additional test power <= 0 can never meet.
__device__ __forceinline__ float blend_power_cut(float alpha_min, float opacity) { return logf(alpha_min / opacity); }

// Box (x_lo, x_hi, y_lo, y_hi) in pixel-centre coordinates outside of which a row cannot pass the skip test.  The set
// power >= cut is the ellipse A dx^2 + 2 B dx dy + C dy^2 <= k with k = -2 cut; its half extents are
// sqrt(k C / det) in x and sqrt(k A / det) in y, det = A C - B^2.  The box is widened by 1e-4 relative + 1e-3 pixels,
// far more than the rounding of the per-pixel test, so skipping by it never changes a result.  Computed once per row
// by the lane that stages it; all lanes then take warp-uniform decisions from it (skip the row, restrict the slots).
__device__ __forceinline__ float4 blend_extent(float u, float v, float A, float B, float C, float cut) {
  const float k = fmaxf(-2.f * cut, 0.f);
  const float det = A * C - B * B;
  if (!(det > 0.f) || !(k < 3.0e38f)) {  // degenerate conic: no bound; cut = +inf (opacity 0) also lands here
    const float big = 3.0e38f;
    return (cut > 0.f) ? make_float4(big, -big, big, -big) : make_float4(-big, big, -big, big);
  }
  if (cut > 0.f) return make_float4(3.0e38f, -3.0e38f, 3.0e38f, -3.0e38f);  // opacity below alpha_min: never passes
  const float ex = sqrtf(k * C / det) * 1.0001f + 1e-3f;
  const float ey = sqrtf(k * A / det) * 1.0001f + 1e-3f;
  return make_float4(u - ex, u + ex, v - ey, v + ey);
}
