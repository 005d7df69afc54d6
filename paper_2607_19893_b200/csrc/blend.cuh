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
constexpr uint32_t BLEND_HEAD = 512;
constexpr uint32_t BLEND_DONE_BIT = 0x80000000u;  // in n_contrib while a tile is between the two kernels
constexpr int BLEND_TAIL_THREADS = 256;

// Workspace of the render calls: [tile flags u32 x tiles | 256-aligned][T, S0, S1, S2 planes, fp32 x pixels each]
static inline size_t blend_ws_flags_bytes(int n_tiles) { return ((size_t)n_tiles * 4 + 255) / 256 * 256; }
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
