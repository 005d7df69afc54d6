// Workspace layouts (host side).  Every region starts on a 256-byte boundary.
#pragma once
#include <stddef.h>
#include <stdint.h>

constexpr uint32_t PROJECT_TILE = 2048;   // primitives per look-back tile of the projection scan
constexpr uint32_t TOUCHED_TILE = 2048;   // primitives per look-back tile of the touched-set kernel
// The two scan kernels give every block `rounds` x 2048 primitives and one look-back (states are sized for
// 2048-primitive tiles, which is always enough).  More rounds = a shorter chain of dependent tiles; fewer = more
// blocks.  Aim at about four blocks per SM, at most 8 rounds.
static inline int scan_rounds_for(uint32_t n, int sm_count) {
  const uint64_t r = (uint64_t)n / ((uint64_t)2048 * (uint64_t)sm_count * 4);
  return r < 1 ? 1 : (r > 8 ? 8 : (int)r);
}
constexpr uint32_t SORT_TILE = 4096;      // keys per onesweep tile
// 8-bit digits.  (9-bit digits save one of six passes at 1080p but every pass costs ~30 % more: twice the histogram
// bins to zero, scan and look back over; measured 0.61 ms against 0.58 ms for 10.5 M keys.)
constexpr uint32_t SORT_RADIX_BITS = 8;
constexpr uint32_t SORT_RADIX = 1u << SORT_RADIX_BITS;
constexpr uint32_t SORT_MAX_PASSES = 7;                      // ceil((32 + 20 tile bits) / 8): images have <= 2^20 tiles
constexpr int SORT_DEPTH_DIGITS = 32 / SORT_RADIX_BITS;      // digits that contain depth bits only

static inline size_t ws_align(size_t x) { return (x + 255) / 256 * 256; }

// [ticket: 256 B][state: u64 per tile]
static inline size_t project_ws_bytes(uint32_t n) {
  return 256 + ws_align(((size_t)n + PROJECT_TILE - 1) / PROJECT_TILE * 8);
}
static inline size_t touched_ws_bytes(uint32_t n) {
  return 256 + ws_align(((size_t)n + TOUCHED_TILE - 1) / TOUCHED_TILE * 8);
}

struct BinSortLayout {
  size_t header;      // tickets: one u32 per pass (+ spare), 256 B
  size_t hist;        // [SORT_MAX_PASSES][SORT_RADIX] u32 global digit histograms
  size_t digit_base;  // [SORT_MAX_PASSES][SORT_RADIX] u32 exclusive scans of the histograms
  size_t states;      // [SORT_MAX_PASSES][tiles][SORT_RADIX] u32 look-back words
  size_t zero_bytes;  // header .. end of states must be zero before the launch sequence
  size_t alt_keys;    // u64[capacity]
  size_t alt_vals;    // u32[capacity]
  size_t chunk_row;   // u32[ceil(capacity / 2048)] first row of every 2048-slot emission chunk
  size_t total;
  uint32_t tiles;
};

static inline BinSortLayout binsort_layout(uint64_t capacity) {
  BinSortLayout L;
  L.tiles = (uint32_t)((capacity + SORT_TILE - 1) / SORT_TILE);
  if (L.tiles == 0) L.tiles = 1;
  size_t o = 0;
  L.header = o; o += 256;
  L.hist = o; o += ws_align((size_t)SORT_MAX_PASSES * SORT_RADIX * 4);
  L.digit_base = o; o += ws_align((size_t)SORT_MAX_PASSES * SORT_RADIX * 4);
  L.states = o; o += ws_align((size_t)SORT_MAX_PASSES * L.tiles * SORT_RADIX * 4);
  L.zero_bytes = o;
  L.alt_keys = o; o += ws_align((size_t)capacity * 8);
  L.alt_vals = o; o += ws_align((size_t)capacity * 4);
  L.chunk_row = o; o += ws_align(((size_t)capacity + 2047) / 2048 * 4 + 4);
  L.total = o;
  return L;
}
static inline size_t binsort_ws_bytes(uint64_t capacity) { return binsort_layout(capacity).total; }
