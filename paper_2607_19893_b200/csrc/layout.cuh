// Workspace layouts (host side).  Every region starts on a 256-byte boundary.
#pragma once
#include <stddef.h>
#include <stdint.h>

constexpr uint32_t PROJECT_TILE = 2048;   // primitives per look-back tile of the projection scan
constexpr uint32_t TOUCHED_TILE = 2048;   // primitives per look-back tile of the touched-set kernel
// The scan kernels (touched set; projection of scenes too large for its fused kernel) give every block `rounds` x 2048
// primitives (look-back states are sized for 2048-primitive tiles, which is always enough).  More rounds = fewer
// dependent tiles / chunk totals to sum; fewer = more blocks.  Aim at about four blocks per SM, at most 8 rounds.
static inline int scan_rounds_for(uint32_t n, int sm_count) {
  const uint64_t r = (uint64_t)n / ((uint64_t)2048 * (uint64_t)sm_count * 4);
  return r < 1 ? 1 : (r > 8 ? 8 : (int)r);
}
constexpr uint32_t SORT_TILE = 4096;     // keys per onesweep tile in the passes over the instances
constexpr uint32_t ROW_SORT_TILE = 2048;  // ... and in the passes over the rows
// 8-bit digits.  (9-bit digits save one of six passes at 1080p but every pass costs ~30 % more: twice the histogram
// bins to zero, scan and look back over; measured 0.61 ms against 0.58 ms for 10.5 M keys.)
constexpr uint32_t SORT_RADIX_BITS = 8;
constexpr uint32_t SORT_RADIX = 1u << SORT_RADIX_BITS;
constexpr int SORT_DEPTH_DIGITS = 32 / SORT_RADIX_BITS;      // passes over the rows (depth bits)
constexpr int SORT_MAX_TILE_DIGITS = 3;                      // passes over the instances: images have <= 2^20 tiles
constexpr uint32_t SORT_MAX_PASSES = SORT_DEPTH_DIGITS + SORT_MAX_TILE_DIGITS;
constexpr uint32_t OFFSET_TILE = 2048;                       // rows per look-back tile of the sorted-offset scan

static inline size_t ws_align(size_t x) { return (x + 255) / 256 * 256; }

// [ticket: 256 B][state: u64 per 2048 primitives][packed total per 256 primitives: u64][exact (rows, instances) per
// chunk of the scan, sized for chunks of 2048: 2 x u64]; the last two are used by scenes too large for the fused kernel
static inline size_t project_ws_group_offset(uint32_t n) {
  return 256 + ws_align(((size_t)n + PROJECT_TILE - 1) / PROJECT_TILE * 8);
}
static inline size_t project_ws_chunk_offset(uint32_t n) {
  return project_ws_group_offset(n) + ws_align(((size_t)n + 255) / 256 * 8);
}
static inline size_t project_ws_bytes(uint32_t n) {
  return project_ws_chunk_offset(n) + ws_align(((size_t)n + PROJECT_TILE - 1) / PROJECT_TILE * 16);
}
static inline size_t touched_ws_bytes(uint32_t n) {
  return 256 + ws_align(((size_t)n + TOUCHED_TILE - 1) / TOUCHED_TILE * 8);
}

// The sort runs in two stages: the rows are sorted by depth (SORT_DEPTH_DIGITS passes over `rows` 32-bit keys), then the
// instances are emitted in that order and sorted by tile id (1..SORT_MAX_TILE_DIGITS passes over `capacity` keys).
struct BinSortLayout {
  size_t header;       // tickets: u32 [0..3] row passes, [4..6] instance passes, [8] offset scan; 256 B
  size_t hist;         // [SORT_MAX_PASSES][SORT_RADIX] u32 global digit histograms (row digits first)
  size_t digit_base;   // [SORT_MAX_PASSES][SORT_RADIX] u32 exclusive scans of the histograms
  size_t tile_diff;    // u32[2^20 + 1] difference array of the instance counts over the tile ids (the first
                       // tiles + 1 words are used and must be zero)
  size_t scan_state;   // u64 per OFFSET_TILE rows: look-back words of the sorted-offset scan
  size_t row_states;   // [SORT_DEPTH_DIGITS][row_tiles][SORT_RADIX] u32 look-back words
  size_t inst_states;  // [SORT_MAX_TILE_DIGITS][tiles][SORT_RADIX] u32 look-back words
  // header .. the instance passes that run must be zero before the launch sequence
  size_t row_keys[2];  // u32[rows] depth bits, ping-pong
  size_t row_vals[2];  // u32[rows] row ids, ping-pong
  size_t sorted_off;   // u32[rows] exclusive prefix of the tile counts in depth order
  size_t inst_keys[2]; // u32[capacity] tile ids, ping-pong
  size_t alt_vals;     // u32[capacity]
  size_t chunk_row;    // u32[ceil(capacity / 2048)] first sorted row of every 2048-slot emission chunk
  size_t total;
  uint32_t tiles, row_tiles;
};

static inline BinSortLayout binsort_layout(uint64_t capacity, uint32_t rows) {
  BinSortLayout L;
  L.tiles = (uint32_t)((capacity + SORT_TILE - 1) / SORT_TILE);
  if (L.tiles == 0) L.tiles = 1;
  L.row_tiles = (rows + ROW_SORT_TILE - 1) / ROW_SORT_TILE;
  if (L.row_tiles == 0) L.row_tiles = 1;
  size_t o = 0;
  L.header = o; o += 256;
  L.hist = o; o += ws_align((size_t)SORT_MAX_PASSES * SORT_RADIX * 4);
  L.digit_base = o; o += ws_align((size_t)SORT_MAX_PASSES * SORT_RADIX * 4);
  L.tile_diff = o; o += ws_align((((size_t)1 << 20) + 1) * 4);
  L.scan_state = o; o += ws_align(((size_t)rows + OFFSET_TILE - 1) / OFFSET_TILE * 8 + 8);
  L.row_states = o; o += ws_align((size_t)SORT_DEPTH_DIGITS * L.row_tiles * SORT_RADIX * 4);
  L.inst_states = o; o += ws_align((size_t)SORT_MAX_TILE_DIGITS * L.tiles * SORT_RADIX * 4);
  for (int b = 0; b < 2; ++b) { L.row_keys[b] = o; o += ws_align((size_t)rows * 4); }
  for (int b = 0; b < 2; ++b) { L.row_vals[b] = o; o += ws_align((size_t)rows * 4); }
  L.sorted_off = o; o += ws_align((size_t)rows * 4 + 4);
  for (int b = 0; b < 2; ++b) { L.inst_keys[b] = o; o += ws_align((size_t)capacity * 4); }
  L.alt_vals = o; o += ws_align((size_t)capacity * 4);
  L.chunk_row = o; o += ws_align(((size_t)capacity + 2047) / 2048 * 4 + 4);
  L.total = o;
  return L;
}
static inline size_t binsort_ws_bytes(uint64_t capacity, uint32_t rows) { return binsort_layout(capacity, rows).total; }

// Counting scatter of the instances (the default for ordinary image sizes): the rows are sorted by depth as above, then
// every chunk of OFFSET_TILE sorted rows counts its instances per tile, a scan over the chunks turns the counts into the
// first position of every (chunk, tile) pair, and the instances are written straight to their final places: no pass
// over the instances at all.  Needs one counter per (chunk, tile): images of up to SCATTER_MAX_TILES tiles.
constexpr uint32_t SCATTER_MAX_TX = 768;        // tiles per image row the emission's shared-memory bit matrix can hold
constexpr uint32_t SCATTER_MAX_TILES = 40000;   // tiles whose difference array fits into one block's shared memory
struct ScatterLayout {
  size_t header;       // as in BinSortLayout; [10] arrival counter of the tile-base kernel
  size_t hist, digit_base;  // row digits only
  size_t scan_state, row_states;
  size_t row_keys[2], row_vals[2];
  size_t sorted_off;   // u32[rows + 1]
  size_t sorted_rect;  // ushort4[rows] rectangles in depth order
  size_t sorted_geo4;  // float4[rows] (u, v, conic A, B) in depth order   } exact binning only: what the span of a
  size_t sorted_geo2;  // float2[rows] (conic C, 2 ln(opacity / alpha_min)) } tile row is computed from
  size_t tile_total;   // u32[tiles]
  size_t counts;       // u32[chunks][tiles_pad]: instances of the tile in the chunk, then their exclusive prefix over the chunks
  size_t total;
  uint32_t row_tiles, chunks, tiles_pad;
};
static inline ScatterLayout scatter_layout(uint32_t rows, uint32_t n_tiles) {
  ScatterLayout L;
  L.row_tiles = (rows + ROW_SORT_TILE - 1) / ROW_SORT_TILE;
  if (L.row_tiles == 0) L.row_tiles = 1;
  L.chunks = (rows + OFFSET_TILE - 1) / OFFSET_TILE;
  if (L.chunks == 0) L.chunks = 1;
  L.tiles_pad = (n_tiles + 63) / 64 * 64;
  size_t o = 0;
  L.header = o; o += 256;
  L.hist = o; o += ws_align((size_t)SORT_DEPTH_DIGITS * SORT_RADIX * 4);
  L.digit_base = o; o += ws_align((size_t)SORT_DEPTH_DIGITS * SORT_RADIX * 4);
  L.scan_state = o; o += ws_align((size_t)L.chunks * 8 + 8);
  L.row_states = o; o += ws_align((size_t)SORT_DEPTH_DIGITS * L.row_tiles * SORT_RADIX * 4);
  for (int b = 0; b < 2; ++b) { L.row_keys[b] = o; o += ws_align((size_t)rows * 4); }
  for (int b = 0; b < 2; ++b) { L.row_vals[b] = o; o += ws_align((size_t)rows * 4); }
  L.sorted_off = o; o += ws_align((size_t)rows * 4 + 4);
  L.sorted_rect = o; o += ws_align((size_t)rows * 8);
  L.sorted_geo4 = o; o += ws_align((size_t)rows * 16);
  L.sorted_geo2 = o; o += ws_align((size_t)rows * 8);
  L.tile_total = o; o += ws_align((size_t)n_tiles * 4);
  L.counts = o; o += ws_align((size_t)L.chunks * L.tiles_pad * 4);
  L.total = o;
  return L;
}
static inline bool scatter_eligible(int TX, uint32_t n_tiles) {
  return (uint32_t)TX <= SCATTER_MAX_TX && n_tiles <= SCATTER_MAX_TILES;
}
