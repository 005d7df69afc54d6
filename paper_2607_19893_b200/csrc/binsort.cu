// Tile binning and sort.  The order asked for is that of a stable least-significant-digit radix sort of the instance
// keys tile_id << 32 | depth bits.  All instances of a row share the row's depth, so the passes over the depth digits are
// taken on the ROWS (several times fewer than the instances): rows are sorted by depth, the instances are emitted in
// that order (load balanced over instances), and only the passes over the tile-id digits run on the instances.  The
// result is the very sequence the full-width sort produces: after the depth passes an instance list is ordered by
// (depth, row, position in the row's rectangle) either way.  Every pass is a onesweep pass with decoupled look-back
// (no library sort).  The per-tile ranges and the digit histograms of the instance passes come from per-tile instance
// counts that are accumulated from the rectangles (a difference array over the tile ids), not from the instances.
#include "common.cuh"
#include "layout.cuh"
#include "tilespan.cuh"

namespace {

// Called by every thread of a block of 256 threads or more after the block's last update of the global histograms.  The block that
// arrives last of `expected` turns the `digits` 256-bin histograms into exclusive scans (the digit bases of the passes),
// which saves a launch per histogram kernel.  s_warp: 33 words, s_flag: 1 word of shared memory.
__device__ __forceinline__ void last_block_digit_bases(const uint32_t* hist, uint32_t* __restrict__ base, int digits,
                                                       uint32_t* arrivals, uint32_t expected, uint32_t* s_warp,
                                                       uint32_t* s_flag) {
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) *s_flag = (atomicAdd(arrivals, 1u) == expected - 1u) ? 1u : 0u;
  __syncthreads();
  if (!*s_flag) return;
  __threadfence();
  for (int d = 0; d < digits; ++d) {
    const bool owner = threadIdx.x < SORT_RADIX;  // thread d scans digit d; a larger block's other threads add nothing
    const uint32_t h = owner ? ld_volatile_u32(hist + d * SORT_RADIX + threadIdx.x) : 0u;
    uint32_t total;
    const uint32_t e = odin_block_exclusive_sum(h, s_warp, &total);
    if (owner) base[d * SORT_RADIX + threadIdx.x] = e;
  }
}

// ------------------------------------------------------------------------------------------------ row histograms
// Digit histograms of the depth bits of all rows, for the SORT_DEPTH_DIGITS row passes, and their exclusive scans.
// Plain shared atomics: aggregating the equal digits of a warp with match.any first (the high digits of a depth take
// few distinct values) was slower, 0.023 against 0.016 ms for 317 k rows - the match costs more than the conflicts.
constexpr int RH_THREADS = 1024;
__global__ void __launch_bounds__(RH_THREADS)
row_hist_kernel(const uint32_t* __restrict__ depth_bits, const uint32_t* __restrict__ num_rows, uint32_t* __restrict__ hist,
                uint32_t* __restrict__ base, uint32_t* arrivals) {
  odin_after_predecessor();
  __shared__ uint32_t s_hist[SORT_DEPTH_DIGITS][SORT_RADIX];
  __shared__ uint32_t s_warp[33], s_flag;
  for (int i = threadIdx.x; i < SORT_DEPTH_DIGITS * (int)SORT_RADIX; i += RH_THREADS) (&s_hist[0][0])[i] = 0;
  __syncthreads();
  const uint32_t V = *num_rows;
  const unsigned lane = threadIdx.x & 31;
  const uint32_t stride = gridDim.x * blockDim.x;
  for (uint32_t r0 = blockIdx.x * blockDim.x; r0 < V; r0 += stride) {  // uniform trip count inside a warp
    const uint32_t r = r0 + threadIdx.x;
    const bool valid = r < V;
    const uint32_t bits = valid ? depth_bits[r] : 0u;
#pragma unroll
    for (int d = 0; d < SORT_DEPTH_DIGITS; ++d) {
      const uint32_t digit = (bits >> (SORT_RADIX_BITS * d)) & (SORT_RADIX - 1);
      if (valid) atomicAdd(&s_hist[d][digit], 1u);
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < SORT_DEPTH_DIGITS * (int)SORT_RADIX; i += RH_THREADS) {
    const uint32_t c = (&s_hist[0][0])[i];
    if (c) atomicAdd(&hist[i], c);
  }
  last_block_digit_bases(hist, base, SORT_DEPTH_DIGITS, arrivals, gridDim.x, s_warp, &s_flag);
}

// Lanes of the warp that hold the same 8-bit digit: eight ballots, one per bit (match.any, the single instruction for
// this, occupies its pipe longer than these sixteen).
__device__ __forceinline__ uint32_t odin_match_digit(uint32_t d) {
  uint32_t peers = 0xffffffffu;
#pragma unroll
  for (int b = 0; b < (int)SORT_RADIX_BITS; ++b) {
    const uint32_t vote = __ballot_sync(0xffffffffu, (d >> b) & 1u);
    peers &= ((d >> b) & 1u) ? vote : ~vote;
  }
  return peers;
}

// ------------------------------------------------------------------------------------------------ onesweep pass
constexpr int OS_THREADS = 512;                           // threads per block in the passes over the instances
constexpr int OS_ROW_THREADS = 512;                       // ... and over the rows: one wave of tiles whose duration is the
                                                          // latency of a tile, so the tile is spread over more threads
static_assert(OS_THREADS >= (int)SORT_RADIX && OS_ROW_THREADS >= (int)SORT_RADIX, "thread d owns digit d");
constexpr int OS_INST_ITEMS = SORT_TILE / OS_THREADS;     // 8 keys per thread in the passes over the instances
constexpr int OS_ROW_ITEMS = ROW_SORT_TILE / OS_ROW_THREADS;  // 4 in the passes over the rows (tiles of 512 / 1024 / 2048 /
                                                          // 4096 keys on 256 threads: 0.074 / 0.070 / 0.064 / 0.065 ms for the four passes at 317 k rows)
constexpr int OS_INST_WINDOW = 2;                 // predecessors fetched per look-back step and digit (instances)
constexpr int OS_ROW_WINDOW = 8;                  // ... and in the passes over the rows
constexpr int OS_RESIDENT = 1024;               // resident threads per SM
constexpr uint32_t OS_FLAG_AGG = 1u << 30, OS_FLAG_INC = 2u << 30, OS_VALUE = (1u << 30) - 1;
constexpr size_t os_smem_bytes(int items, int threads) {
  return (size_t)items * threads * 8 + (size_t)(threads / 32) * SORT_RADIX * 4 + 2 * SORT_RADIX * 4 + 16;
}

// One pass over one 8-bit digit of 32-bit keys.  Persistent blocks take tiles of ITEMS * THREADS keys by ticket.  Per tile:
// warp-striped loads, per-warp digit ranking (stable; eight ballots per key), block
// digit counts published for look-back, exclusive global digit offsets by a per-digit look-back walk (thread d walks digit d), keys and values exchanged
// through shared memory so that the global scatter writes runs of consecutive addresses.
//   vals_in == nullptr: the values are the positions themselves (first pass over the rows)
//   keys_out == nullptr: the keys are not needed afterwards (last pass over the rows)
//   WIDE: the last pass over the instances may also write the full 64-bit key key << 32 | depth_bits[value]
//   the number of keys is *count32 if given, else min(*count64, capacity)
//   ITEMS keys per thread on THREADS threads: 8 x 512 for the instances, 4 x 512 for the rows, of which there are so few
//   that a pass is one wave of blocks and its duration is the latency of one tile (with 256 threads per tile the
//   ITEMS-long ranking chain and the write-out were twice as long: whole step 0.870 -> 0.855 ms at 317 k rows; the two
//   instance passes at 1.9 M instances 0.084 -> 0.075 ms)
template <bool WIDE, int ITEMS, int WINDOW, int THREADS>
__global__ void __launch_bounds__(THREADS, OS_RESIDENT / THREADS)
onesweep_kernel(const uint32_t* __restrict__ keys_in, const uint32_t* __restrict__ vals_in, uint32_t* __restrict__ keys_out,
                uint32_t* __restrict__ vals_out, uint64_t* __restrict__ keys64_out, const uint32_t* __restrict__ depth_bits,
                const uint32_t* __restrict__ count32, const uint64_t* __restrict__ count64, uint64_t capacity, int shift,
                const uint32_t* __restrict__ digit_base, uint32_t* states, uint32_t* ticket, int* status,
                int spin_limit, uint32_t depth_rows) {
  odin_after_predecessor();  // launched behind the histogram / the pass in front
  extern __shared__ __align__(16) unsigned char os_smem[];
  uint32_t* s_keys = reinterpret_cast<uint32_t*>(os_smem);
  constexpr uint32_t TILE = (uint32_t)ITEMS * THREADS;
  constexpr int OS_WARPS = THREADS / 32;
  constexpr int OS_DPT = 1;  // thread d owns digit d; the threads beyond the radix own none
  const bool owner = threadIdx.x < SORT_RADIX;
  uint32_t* s_vals = s_keys + TILE;
  uint32_t(*s_warp_hist)[SORT_RADIX] = reinterpret_cast<uint32_t(*)[SORT_RADIX]>(s_vals + TILE);
  uint32_t* s_digit_start = &s_warp_hist[0][0] + OS_WARPS * SORT_RADIX;
  uint32_t* s_global = s_digit_start + SORT_RADIX;
  uint32_t* s_misc = s_global + SORT_RADIX;  // [0] tile ticket
  __shared__ uint32_t s_scan[33];

  uint64_t M64;
  if (count32) {
    M64 = *count32;
  } else {
    const uint64_t M_all = *count64;
    M64 = M_all < capacity ? M_all : capacity;
  }
  const uint32_t M = (uint32_t)(M64 < (uint64_t)OS_VALUE ? M64 : (uint64_t)OS_VALUE);
  const uint32_t ntiles = (M + TILE - 1) / TILE;
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;

  // The keys and values of the NEXT tile are requested as soon as the registers of the current one are free (after
  // the exchange through shared memory), so that their latency overlaps the global scatter of the current tile.
  uint32_t key[ITEMS];
  uint32_t val[ITEMS];
  auto load_tile = [&](uint32_t t) {
    const uint32_t wb = t * TILE + warp * (32 * ITEMS);
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      const uint32_t i = wb + 32 * j + lane;
      const bool in = t < ntiles && i < M;
      key[j] = in ? keys_in[i] : ~0u;  // padding sorts to the end of the tile and is never written
      val[j] = in ? (vals_in ? vals_in[i] : i) : 0u;
    }
  };
  if (threadIdx.x == 0) s_misc[0] = atomicAdd(ticket, 1u);
  __syncthreads();
  uint32_t tile = s_misc[0];
  load_tile(tile);

  while (tile < ntiles) {
    for (int i = threadIdx.x; i < OS_WARPS * (int)SORT_RADIX; i += THREADS) (&s_warp_hist[0][0])[i] = 0;
    __syncthreads();
    const uint32_t tile_base = tile * TILE;
    const uint32_t tile_count = min(TILE, M - tile_base);

    uint32_t pos[ITEMS];
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      const uint32_t d = (key[j] >> shift) & (SORT_RADIX - 1);
      // (measured: ballots 0.060 against 0.064 ms with match.any for the four row passes at 317 k rows; no difference
      // in the passes over 1.9 M instances)
      const uint32_t peers = odin_match_digit(d);
      const int leader = __ffs(peers) - 1;
      uint32_t old = 0;
      if ((int)lane == leader) {
        old = s_warp_hist[warp][d];
        s_warp_hist[warp][d] = old + __popc(peers);
      }
      old = __shfl_sync(0xffffffffu, old, leader);
      pos[j] = old + __popc(peers & lt_mask);
      __syncwarp();
    }
    __syncthreads();

    // thread t owns digits t, t + 256, ...: exclusive offsets of the warps inside each digit, block totals published
    uint32_t cta_count[OS_DPT];
#pragma unroll
    for (int q = 0; q < OS_DPT; ++q) {
      const uint32_t d = threadIdx.x;
      uint32_t c = 0;
      if (owner) {
#pragma unroll
        for (int w = 0; w < OS_WARPS; ++w) {
          const uint32_t t = s_warp_hist[w][d];
          s_warp_hist[w][d] = c;
          c += t;
        }
        st_volatile_u32(states + (size_t)tile * SORT_RADIX + d, (tile == 0 ? OS_FLAG_INC : OS_FLAG_AGG) | c);
      }
      cta_count[q] = c;
    }
    uint32_t digit_start[OS_DPT];
    {
      uint32_t carry = 0;
#pragma unroll
      for (int q = 0; q < OS_DPT; ++q) {  // digits ascend with q first, so the scans chain
        uint32_t total;
        digit_start[q] = carry + odin_block_exclusive_sum(cta_count[q], s_scan, &total);
        if (owner) s_digit_start[threadIdx.x] = digit_start[q];
        carry += total;
      }
    }
    uint32_t exclusive[OS_DPT];
#pragma unroll
    for (int q = 0; q < OS_DPT; ++q) exclusive[q] = 0;
    if (tile > 0 && owner) {
      // walk back over the predecessors for all owned digits at once
      int64_t t[OS_DPT];
#pragma unroll
      for (int q = 0; q < OS_DPT; ++q) t[q] = (int64_t)tile - 1;
      int spins = 0;
      bool busy = true;
      while (busy) {
        busy = false;
        bool stalled = true;  // cleared as soon as any predecessor word is consumed
        // a window of WINDOW predecessors per digit is fetched at once: the walk is a chain of dependent L2 round
        // trips, and when a launch starts every resident tile has hundreds of aggregates in front of it
        uint32_t s[OS_DPT][WINDOW];
#pragma unroll
        for (int q = 0; q < OS_DPT; ++q)
#pragma unroll
          for (int k = 0; k < WINDOW; ++k)
            s[q][k] = (t[q] - k >= 0)
                          ? ld_volatile_u32(states + (size_t)(t[q] - k) * SORT_RADIX + threadIdx.x)
                          : 0u;
#pragma unroll
        for (int q = 0; q < OS_DPT; ++q) {
          if (t[q] < 0) continue;
#pragma unroll
          for (int k = 0; k < WINDOW; ++k) {
            if (t[q] < 0) break;
            const uint32_t flag = s[q][k] >> 30;
            if (flag == 0) break;  // not published yet: use what precedes it, come back
            exclusive[q] += s[q][k] & OS_VALUE;
            t[q] = (flag == 2) ? -1 : t[q] - 1;
            stalled = false;
          }
          if (t[q] >= 0) busy = true;
        }
        if (busy && stalled) {
          __nanosleep(32);
          if (++spins > spin_limit) { odin_set_error(status, ODIN_ERR_TIMEOUT); break; }
        }
      }
#pragma unroll
      for (int q = 0; q < OS_DPT; ++q)
        st_volatile_u32(states + (size_t)tile * SORT_RADIX + threadIdx.x,
                        OS_FLAG_INC | ((exclusive[q] + cta_count[q]) & OS_VALUE));
    }
#pragma unroll
    for (int q = 0; q < OS_DPT; ++q) {
      const uint32_t d = threadIdx.x;
      if (owner) s_global[d] = digit_base[d] + exclusive[q] - digit_start[q];  // + slot index inside the tile = address
    }
    __syncthreads();

#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      const uint32_t dg = (key[j] >> shift) & (SORT_RADIX - 1);
      const uint32_t slot = s_digit_start[dg] + s_warp_hist[warp][dg] + pos[j];
      s_keys[slot] = key[j];
      s_vals[slot] = val[j];
    }
    if (threadIdx.x == 0) s_misc[0] = atomicAdd(ticket, 1u);
    __syncthreads();
    const uint32_t next = s_misc[0];
    load_tile(next);  // in flight while the current tile is written out
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
      const uint32_t slot = j * THREADS + threadIdx.x;
      if (slot < tile_count) {
        const uint32_t k = s_keys[slot];
        const uint32_t dst = s_global[(k >> shift) & (SORT_RADIX - 1)] + slot;
        if (dst < M) {
          const uint32_t v = s_vals[slot];
          if (keys_out) keys_out[dst] = k;
          vals_out[dst] = v;
          if (WIDE) {
            // (depth_rows: length of depth_bits; the clamp only matters for a list that an earlier timed-out pass left
            // partly unwritten)
            if (keys64_out) keys64_out[dst] = ((uint64_t)k << 32) | (uint64_t)depth_bits[min(v, depth_rows - 1)];
          }
        }
      }
    }
    tile = next;
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------ sorted offsets
// sorted_off[i] = number of instances of the rows in front of position i of the depth order: an exclusive scan of the
// rectangles' tile counts gathered through sorted_row.  2048 positions per block, one decoupled look-back per block,
// blocks ordered by ticket.
constexpr int RO_THREADS = 1024;
constexpr int RO_ITEMS = OFFSET_TILE / RO_THREADS;
// the instances are emitted in chunks of DUP_CHUNK consecutive slots (emit_instances_kernel)
constexpr int DUP_THREADS = 256;
constexpr int DUP_ITEMS = 8;
constexpr int DUP_CHUNK = DUP_THREADS * DUP_ITEMS;  // a chunk spans at most DUP_CHUNK rows

//
// The same kernel counts the instances per tile without touching a single instance: one tile row of a rectangle is a
// run of consecutive tile ids [t0, t1), which adds 1 at t0 and subtracts 1 at t1 in a difference array over the tile
// ids; tile_scan_block integrates it.  Only the first `capacity` instances of the depth order count.
// It also fills chunk_row[c] = the position (in depth order) of the row whose slots contain slot c * DUP_CHUNK: a row
// writes an entry for every chunk boundary that falls inside its slot range (usually none or one).
__global__ void __launch_bounds__(RO_THREADS)
sorted_offsets_kernel(const uint32_t* __restrict__ sorted_row, const ushort4* __restrict__ rect,
                      const uint32_t* __restrict__ num_rows, uint32_t capacity, int TX, uint32_t* __restrict__ sorted_off,
                      uint32_t* __restrict__ chunk_row, uint32_t chunks_cap, uint32_t* __restrict__ tile_diff,
                      uint32_t diff_words, uint32_t* ticket, uint64_t* state, int* status, int spin_limit) {
  odin_after_predecessor();
  // diff_words != 0: the block first accumulates its part of the difference array in shared memory (`diff_words` =
  // tiles + 1 words of dynamic shared memory) and adds the non-zero words to the global one at the end: a tile on which
  // thousands of rectangles pile up would otherwise serialise that many global reductions on one address.
  extern __shared__ uint32_t s_tdiff[];
  __shared__ uint32_t s_tile, s_base;
  __shared__ uint32_t s_warp[33];
  const uint32_t V = *num_rows;
  const uint32_t ntiles = (V + OFFSET_TILE - 1) / OFFSET_TILE;
  if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  if (tile >= ntiles) return;  // uniform over the block; nobody waits for a tile past the end
  for (uint32_t i = threadIdx.x; i < diff_words; i += RO_THREADS) s_tdiff[i] = 0;  // (barriers of the scan follow)
  const uint32_t first = tile * OFFSET_TILE + threadIdx.x * RO_ITEMS;
  ushort4 rc[RO_ITEMS];
  uint32_t cnt[RO_ITEMS];
  uint32_t sum = 0;  // sums are taken modulo 2^32; the true totals fit (M >= 2^32 is an error raised by the projection)
#pragma unroll
  for (int k = 0; k < RO_ITEMS; ++k) {
    rc[k] = make_ushort4(0, 0, 0, 0);
    // (a row id is clamped to the rows of this view: it stays in range even if a pass of the row sort gave up and left
    // part of its output unwritten)
    if (first + k < V) rc[k] = rect[min(sorted_row[first + k], V - 1)];
    cnt[k] = ((uint32_t)rc[k].z - (uint32_t)rc[k].x) * ((uint32_t)rc[k].w - (uint32_t)rc[k].y);
    sum += cnt[k];
  }
  uint32_t total;
  const uint32_t before = odin_block_exclusive_sum(sum, s_warp, &total);
  if (threadIdx.x < 32) {
    const uint64_t b = odin_lookback_u64(state, tile, (uint64_t)total, status, spin_limit);
    if (threadIdx.x == 0) s_base = (uint32_t)b;
  }
  __syncthreads();
  uint32_t run = s_base + before;
#pragma unroll
  for (int k = 0; k < RO_ITEMS; ++k) {
    if (first + k < V) {
      sorted_off[first + k] = run;
      const uint64_t hi = (uint64_t)run + cnt[k];
      for (uint64_t c = ((uint64_t)run + DUP_CHUNK - 1) / DUP_CHUNK; c * DUP_CHUNK < hi && c < chunks_cap; ++c)
        chunk_row[c] = first + k;
    }
    // instances of this row that are emitted: those in front of the capacity
    uint32_t left = run < capacity ? min(cnt[k], capacity - run) : 0u;
    const uint32_t w = (uint32_t)rc[k].z - (uint32_t)rc[k].x;
    for (uint32_t y = rc[k].y; left != 0; ++y) {
      const uint32_t len = min(w, left);
      left -= len;
      const uint32_t t0 = y * (uint32_t)TX + (uint32_t)rc[k].x;
      uint32_t* diff = diff_words ? s_tdiff : tile_diff;
      atomicAdd(&diff[t0], 1u);
      atomicSub(&diff[t0 + len], 1u);
    }
    run += cnt[k];
  }
  if (diff_words) {
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < diff_words; i += RO_THREADS) {
      const uint32_t d = s_tdiff[i];
      if (d) atomicAdd(&tile_diff[i], d);
    }
  }
}

// Run by ONE block (all of its threads).  Integrates the difference array into the instance count of every tile (sums
// modulo 2^32; every prefix is a true count), writes the tile ranges [first, one past last) as the exclusive scan of
// the counts, and builds the digit histograms of the instances' tile ids and their exclusive scans (the digit bases of
// the instance passes).  Needs blockDim.x >= 256.
constexpr int TS_ITEMS = 4;

__device__ __forceinline__ void tile_scan_block(const uint32_t* __restrict__ tile_diff, uint32_t n_tiles, int tile_passes,
                                                uint32_t* __restrict__ ranges, uint32_t* __restrict__ base, uint32_t cap) {
  __shared__ uint32_t s_h[SORT_MAX_TILE_DIGITS][SORT_RADIX];
  __shared__ uint32_t s_warp[33];
  const unsigned lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < SORT_MAX_TILE_DIGITS * (int)SORT_RADIX; i += blockDim.x) (&s_h[0][0])[i] = 0;
  __syncthreads();
  uint32_t carry_count = 0, carry_off = 0;  // count of the tile in front of the batch; instances in front of the batch
  for (uint32_t b0 = 0; b0 < n_tiles; b0 += blockDim.x * TS_ITEMS) {
    const uint32_t t0 = b0 + threadIdx.x * TS_ITEMS;
    uint32_t c[TS_ITEMS];
    uint32_t run = 0;
#pragma unroll
    for (int k = 0; k < TS_ITEMS; ++k) {
      run += (t0 + k < n_tiles) ? tile_diff[t0 + k] : 0u;
      c[k] = run;  // inclusive prefix of the differences inside the thread
    }
    uint32_t total;
    const uint32_t before = carry_count + odin_block_exclusive_sum(run, s_warp, &total);
    uint32_t mine = 0;
#pragma unroll
    for (int k = 0; k < TS_ITEMS; ++k) {
      c[k] = (t0 + k < n_tiles) ? c[k] + before : 0u;  // instances of tile t0 + k
      mine += c[k];
    }
    carry_count += total;
    uint32_t total2;
    uint32_t off = carry_off + odin_block_exclusive_sum(mine, s_warp, &total2);
    carry_off += total2;
#pragma unroll
    for (int k = 0; k < TS_ITEMS; ++k) {
      const uint32_t t = t0 + k;
      if (t < n_tiles) {
        // never beyond the instance capacity (the counts already respect it unless a look-back gave up)
        reinterpret_cast<uint2*>(ranges)[t] = make_uint2(min(off, cap), min(off + c[k], cap));
        if (c[k]) atomicAdd(&s_h[0][t & (SORT_RADIX - 1)], c[k]);
        off += c[k];
      }
    }
    // higher digits: the 128 consecutive tiles of a warp share the digit unless they straddle a multiple of 256 (or
    // 65536), so the warp adds its sum once instead of 128 times to the same word
    for (int d = 1; d < tile_passes; ++d) {
      const int shift = (int)SORT_RADIX_BITS * d;
      const uint32_t first = __shfl_sync(0xffffffffu, t0, 0), last = __shfl_sync(0xffffffffu, t0 + TS_ITEMS - 1, 31);
      if ((first >> shift) == (last >> shift)) {
        const uint32_t sum = __reduce_add_sync(0xffffffffu, mine);
        if (lane == 0 && sum) atomicAdd(&s_h[d][(first >> shift) & (SORT_RADIX - 1)], sum);
      } else {
#pragma unroll
        for (int k = 0; k < TS_ITEMS; ++k)
          if (c[k]) atomicAdd(&s_h[d][((t0 + k) >> shift) & (SORT_RADIX - 1)], c[k]);
      }
    }
  }
  __syncthreads();
  for (int d = 0; d < tile_passes; ++d) {
    const uint32_t h = threadIdx.x < SORT_RADIX ? s_h[d][threadIdx.x] : 0u;
    uint32_t total;
    const uint32_t e = odin_block_exclusive_sum(h, s_warp, &total);
    if (threadIdx.x < SORT_RADIX) base[d * SORT_RADIX + threadIdx.x] = e;
  }
}

// ------------------------------------------------------------------------------------------------ emission

// Cooperative 256-ary upper bound: first r in [0, V) with off[r] > x (V if none).  All threads must call.
__device__ __forceinline__ uint32_t block_upper_bound(const uint32_t* __restrict__ off, uint32_t V, uint32_t x) {
  uint32_t lo = 0, hi = V;
  while (lo < hi) {
    const uint32_t span = hi - lo;
    const uint32_t step = (span + DUP_THREADS - 1) / DUP_THREADS;
    const uint32_t probe = lo + threadIdx.x * step;
    const int below = (probe < hi) && (off[probe] <= x);
    const uint32_t cnt = (uint32_t)__syncthreads_count(below);  // monotone predicate: the first cnt probes are <= x
    if (cnt == 0) { hi = lo; break; }
    const uint32_t new_lo = lo + (cnt - 1) * step + 1;
    const uint32_t new_hi = min(hi, lo + cnt * step);
    lo = new_lo; hi = new_hi;
  }
  return lo;
}

// Each chunk of DUP_CHUNK consecutive instance slots finds the positions of the depth order it overlaps, stages their
// offsets, row ids and rectangles in shared memory, and every thread expands its slots: slot i of a row is tile
// (y0 + k / w, x0 + k % w) with k = i - offset, w = x1 - x0.  Keys (tile ids) and values (row ids) are written fully
// coalesced.  The last block of the grid does something else at the same time: the scan over the tiles (ranges and
// digit bases), which is one block's work and would otherwise be a launch of its own on the critical path.
__global__ void __launch_bounds__(DUP_THREADS)
emit_instances_kernel(const uint32_t* __restrict__ sorted_off, const uint32_t* __restrict__ sorted_row,
                      const uint32_t* __restrict__ chunk_row, const ushort4* __restrict__ rect,
                      const uint32_t* __restrict__ num_rows, const uint64_t* __restrict__ num_instances, uint64_t capacity,
                      int TX, uint32_t* __restrict__ keys, uint32_t* __restrict__ vals, int* status,
                      const uint32_t* __restrict__ tile_diff, uint32_t n_tiles, int tile_passes,
                      uint32_t* __restrict__ ranges, uint32_t* __restrict__ tile_dbase) {
  odin_after_predecessor();
  if (blockIdx.x == 0) {  // block 0: it is scheduled first
    tile_scan_block(tile_diff, n_tiles, tile_passes, ranges, tile_dbase,
                    (uint32_t)(capacity < 0xffffffffull ? capacity : 0xffffffffull));
    return;
  }
  const uint32_t emit_blocks = gridDim.x - 1, emit_block = blockIdx.x - 1;
  __shared__ uint32_t s_off[DUP_CHUNK + 1];
  __shared__ ushort4 s_rect[DUP_CHUNK];
  __shared__ uint32_t s_row[DUP_CHUNK];
  __shared__ __align__(16) uint16_t s_map[DUP_CHUNK];  // slot of the chunk -> staged row of the chunk
  __shared__ uint32_t s_scan[DUP_THREADS / 32];
  const uint32_t V = *num_rows;
  const uint64_t M_all = *num_instances;
  const uint64_t M64 = M_all < capacity ? M_all : capacity;
  if (emit_block == 0 && threadIdx.x == 0 && M_all > capacity) odin_set_error(status, ODIN_ERR_CAPACITY);
  const uint32_t M = (uint32_t)(M64 < 0xffffffffull ? M64 : 0xffffffffull);
  const uint32_t chunks = V == 0 ? 0u : (M + DUP_CHUNK - 1) / DUP_CHUNK;
  const unsigned lane = threadIdx.x & 31;
  for (uint32_t chunk = emit_block; chunk < chunks; chunk += emit_blocks) {
    const uint32_t c0 = chunk * DUP_CHUNK;
    const uint32_t c1 = (M - c0 < (uint32_t)DUP_CHUNK) ? M : c0 + DUP_CHUNK;
    // first and last position of the chunk from the chunk table; only the last chunk has to search for its end
    // (every index taken from the tables is clamped: if a look-back gave up, parts of them were never written, and
    // the emission must still stay inside its buffers; with intact tables the clamps change nothing)
    const uint32_t row_lo = min(chunk_row[chunk], V - 1);
    uint32_t row_hi;
    if (chunk + 1 < chunks) {
      const uint32_t rn = min(chunk_row[chunk + 1], V - 1);  // position that holds slot c1
      row_hi = (sorted_off[rn] == c1 && rn > 0) ? rn - 1 : rn;
    } else {
      row_hi = max(block_upper_bound(sorted_off, V, c1 - 1), 1u) - 1;  // offset[0] = 0, so the bound is >= 1
    }
    row_hi = min(max(row_hi, row_lo), row_lo + (uint32_t)DUP_CHUNK - 1);
    const uint32_t nrows = row_hi - row_lo + 1;  // <= DUP_CHUNK: every row owns at least one slot
    for (uint32_t i = threadIdx.x; i < nrows; i += DUP_THREADS) {
      const uint32_t r = min(sorted_row[row_lo + i], V - 1);
      s_off[i] = sorted_off[row_lo + i];
      s_row[i] = r;
      s_rect[i] = rect[r];
    }
    if (threadIdx.x == 0) s_off[nrows] = (row_hi + 1 < V) ? sorted_off[row_hi + 1] : (uint32_t)M_all;
    for (int i = threadIdx.x; i < DUP_CHUNK; i += DUP_THREADS) s_map[i] = 0;
    __syncthreads();
    // slot -> staged row: every row marks its first slot, an inclusive max-scan fills the rest
    for (uint32_t i = threadIdx.x; i < nrows; i += DUP_THREADS)
      s_map[min(max(s_off[i], c0) - c0, (uint32_t)DUP_CHUNK - 1)] = (uint16_t)i;
    __syncthreads();
    {
      static_assert(DUP_ITEMS == 8, "a thread's slots are one 16-byte word of the map");
      uint4* map4 = reinterpret_cast<uint4*>(s_map) + threadIdx.x;
      const uint4 raw = *map4;
      const uint32_t rw[4] = {raw.x, raw.y, raw.z, raw.w};
      uint32_t m[DUP_ITEMS];
      uint32_t run = 0;
#pragma unroll
      for (int k = 0; k < DUP_ITEMS; ++k) {
        run = max(run, (rw[k >> 1] >> (16 * (k & 1))) & 0xffffu);
        m[k] = run;
      }
      uint32_t inc = run;  // inclusive max over the threads of the warp (values >= 0, so 0 is neutral)
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const uint32_t y = __shfl_up_sync(0xffffffffu, inc, o, 32);
        if (lane >= (unsigned)o) inc = max(inc, y);
      }
      if (lane == 31) s_scan[threadIdx.x >> 5] = inc;
      __syncthreads();
      uint32_t before = __shfl_up_sync(0xffffffffu, inc, 1);
      if (lane == 0) before = 0;
      for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) before = max(before, s_scan[w]);
#pragma unroll
      for (int k = 0; k < DUP_ITEMS; ++k) m[k] = max(m[k], before);
      *map4 = make_uint4(m[0] | (m[1] << 16), m[2] | (m[3] << 16), m[4] | (m[5] << 16), m[6] | (m[7] << 16));
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < DUP_ITEMS; ++k) {
      const uint32_t i = c0 + k * DUP_THREADS + threadIdx.x;
      if (i < c1) {
        const uint32_t lo = s_map[i - c0];  // staged row that owns this slot
        const ushort4 rc = s_rect[lo];
        const uint32_t local = i - s_off[lo];
        const uint32_t w = (uint32_t)rc.z - (uint32_t)rc.x;
        const uint32_t dy = local / w, dx = local - dy * w;
        keys[i] = ((uint32_t)rc.y + dy) * (uint32_t)TX + (uint32_t)rc.x + dx;
        vals[i] = s_row[lo];
      }
    }
    __syncthreads();
  }
}


// ------------------------------------------------------------------------------------------------ counting scatter
// The instances never need a sort of their own.  With the rows in depth order, the list of a tile is the subsequence of
// rows whose rectangle covers it, so the final position of an instance is
//     first position of the tile + instances of the tile in earlier chunks of rows + rank of the row inside its chunk,
// and all three are cheap: the rectangles give the per-(chunk, tile) counts through a difference array (one block per
// chunk of OFFSET_TILE sorted rows), a scan over the chunks and one over the tiles give the first positions, and the
// rank inside a chunk comes out of a bit matrix (tile x row) in shared memory in which set bits are read off in row
// order.  Three launches that together move 8V + 4M bytes plus the counters, against emission + two radix passes over
// 8-byte instances.

// One block per chunk, blocks ordered by ticket (one look-back for the running instance offset, which is only needed
// for the capacity rule: the instances in front of `capacity` in depth order are the ones that exist).  Writes the
// rectangles in depth order and the chunk's instance count for every tile.
// EXACT (binning 2): a row's instances are the kept spans of its rectangle's tile rows (tilespan.cuh), recomputed here
// from the row's centre, conic and opacity, which are also written out in depth order for the scatter kernel.
// THREADS x ITEMS = OFFSET_TILE rows per block: 256 x 8 for the plain rectangles, 1024 x 2 when the spans have to be
// computed (that is several hundred instructions per tile row of every rectangle: more warps per chunk)
template <bool EXACT, int THREADS, int ITEMS>
__global__ void __launch_bounds__(THREADS)
chunk_counts_kernel(const uint32_t* __restrict__ sorted_row, const ushort4* __restrict__ rect,
                    const float2* __restrict__ xy, const float4* __restrict__ conic_o, float alpha_min,
                    const uint32_t* __restrict__ num_rows, const uint64_t* __restrict__ num_instances, uint32_t capacity,
                    int TX, uint32_t n_tiles, uint32_t tiles_pad, uint32_t* __restrict__ sorted_off,
                    ushort4* __restrict__ sorted_rect, float4* __restrict__ sorted_geo4, float2* __restrict__ sorted_geo2,
                    uint32_t* __restrict__ counts, uint32_t* ticket, uint64_t* state, int* status, int spin_limit) {
  odin_after_predecessor();
  extern __shared__ __align__(16) uint32_t s_tdiff[];  // tiles_pad + 8 words
  __shared__ uint32_t s_tile, s_base;
  __shared__ uint32_t s_warp[33];
  const uint32_t V = *num_rows;
  const uint32_t ntiles = (V + OFFSET_TILE - 1) / OFFSET_TILE;
  if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  if (tile >= ntiles) return;  // uniform over the block; nobody waits for a chunk past the end
  for (uint32_t i = threadIdx.x; i < tiles_pad + 8; i += THREADS) s_tdiff[i] = 0;
  __syncthreads();
  // only when the view has more instances than the caller's capacity can a row be denied some of its instances (those
  // at or behind `capacity` in depth order); otherwise the counts do not depend on the running offset
  const bool cut = *num_instances > (uint64_t)capacity;
  const uint32_t first = tile * OFFSET_TILE + threadIdx.x * ITEMS;
  ushort4 rc[ITEMS];
  uint32_t cnt[ITEMS];
  uint32_t sum = 0;
  // adds the run of tiles [t0, t0 + len) to the difference array
  auto add_run = [&](uint32_t t0, uint32_t len) {
    t0 = min(t0, n_tiles);  // (clamps: see emit_instances_kernel)
    atomicAdd(&s_tdiff[t0], 1u);
    atomicSub(&s_tdiff[min(t0 + len, n_tiles)], 1u);
  };
#pragma unroll
  for (int k = 0; k < ITEMS; ++k) {
    rc[k] = make_ushort4(0, 0, 0, 0);
    cnt[k] = 0;
    SpanConic e;
    e.k = -1.f;
    if (first + k < V) {
      const uint32_t r = min(sorted_row[first + k], V - 1);
      rc[k] = rect[r];
      if (EXACT) {
        const float2 c = xy[r];
        const float4 q = conic_o[r];
        e = odin_span_conic(c.x, c.y, q.x, q.y, q.z, q.w, alpha_min);
        sorted_geo4[first + k] = make_float4(e.u, e.v, e.A, e.B);
        sorted_geo2[first + k] = make_float2(e.C, e.k);
      } else {
        cnt[k] = ((uint32_t)rc[k].z - (uint32_t)rc[k].x) * ((uint32_t)rc[k].w - (uint32_t)rc[k].y);
      }
    }
    if (EXACT) {
      // a lane walks the tile rows of a low rectangle by itself; the tall rectangles of the warp are walked by all 32
      // lanes together (one tile row per lane and step)
      const int h = (int)rc[k].w - (int)rc[k].y;
      const bool tall = h > 4;
      if (h > 0 && !tall)
        for (int y = rc[k].y; y < (int)rc[k].w; ++y) {
          int xa, xb;
          odin_row_span(e, y, rc[k].x, rc[k].z, xa, xb);
          if (xb > xa) {
            cnt[k] += (uint32_t)(xb - xa);
            if (!cut) add_run((uint32_t)y * (uint32_t)TX + (uint32_t)xa, (uint32_t)(xb - xa));
          }
        }
      uint32_t todo = __ballot_sync(0xffffffffu, tall);
      while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        const SpanConic q = odin_span_conic_bcast(e, src);
        const int qx0 = __shfl_sync(0xffffffffu, (int)rc[k].x, src), qy0 = __shfl_sync(0xffffffffu, (int)rc[k].y, src);
        const int qx1 = __shfl_sync(0xffffffffu, (int)rc[k].z, src), qy1 = __shfl_sync(0xffffffffu, (int)rc[k].w, src);
        uint32_t kept = 0;
        for (int y = qy0 + (int)(threadIdx.x & 31); y < qy1; y += 32) {
          int xa, xb;
          odin_row_span(q, y, qx0, qx1, xa, xb);
          if (xb > xa) {
            kept += (uint32_t)(xb - xa);
            if (!cut) add_run((uint32_t)y * (uint32_t)TX + (uint32_t)xa, (uint32_t)(xb - xa));
          }
        }
        kept = __reduce_add_sync(0xffffffffu, kept);
        if ((int)(threadIdx.x & 31) == src) cnt[k] = kept;
      }
    }
    sum += cnt[k];
  }
  uint32_t total;
  const uint32_t before = odin_block_exclusive_sum(sum, s_warp, &total);
  if (threadIdx.x < 32) {
    const uint64_t b = odin_lookback_u64(state, tile, (uint64_t)total, status, spin_limit);
    if (threadIdx.x == 0) s_base = (uint32_t)b;
  }
  __syncthreads();
  uint32_t run = s_base + before;
#pragma unroll
  for (int k = 0; k < ITEMS; ++k) {
    if (first + k < V) {
      sorted_off[first + k] = run;
      sorted_rect[first + k] = rc[k];
    }
    if (!EXACT || cut) {
      // the instances of the row that exist: those in front of `capacity`, its tiles taken in row-major order
      uint32_t left = run < capacity ? min(cnt[k], capacity - run) : 0u;
      const uint32_t w = (uint32_t)rc[k].z - (uint32_t)rc[k].x;
      SpanConic e;
      if (EXACT && left != 0) {
        const float4 g4 = sorted_geo4[first + k];  // written above by this thread
        const float2 g2 = sorted_geo2[first + k];
        e.u = g4.x; e.v = g4.y; e.A = g4.z; e.B = g4.w; e.C = g2.x; e.k = g2.y;
      }
      for (uint32_t y = rc[k].y; left != 0 && y < (uint32_t)rc[k].w; ++y) {
        uint32_t x0 = rc[k].x, len = w;
        if (EXACT) {
          int xa, xb;
          odin_row_span(e, (int)y, rc[k].x, rc[k].z, xa, xb);
          x0 = (uint32_t)xa; len = (uint32_t)(xb - xa);
          if (len == 0) continue;
        }
        len = min(len, left);
        left -= len;
        add_run(y * (uint32_t)TX + x0, len);
      }
    }
    run += cnt[k];
  }
  __syncthreads();
  // integrate the difference array: instances of every tile in this chunk
  uint32_t* __restrict__ out = counts + (size_t)tile * tiles_pad;
  uint32_t carry = 0;
  for (uint32_t b0 = 0; b0 < n_tiles; b0 += THREADS * 4) {
    const uint32_t t0 = b0 + threadIdx.x * 4;
    uint4 d = make_uint4(0, 0, 0, 0);
    if (t0 < n_tiles) d = *reinterpret_cast<const uint4*>(s_tdiff + t0);  // padded: words past n_tiles are zero or unused
    const uint32_t c0 = d.x, c1 = c0 + d.y, c2 = c1 + d.z, c3 = c2 + d.w;
    uint32_t tot;
    const uint32_t base = carry + odin_block_exclusive_sum(c3, s_warp, &tot);
    if (t0 + 3 < n_tiles) {
      *reinterpret_cast<uint4*>(out + t0) = make_uint4(c0 + base, c1 + base, c2 + base, c3 + base);
    } else {
      if (t0 < n_tiles) out[t0] = c0 + base;
      if (t0 + 1 < n_tiles) out[t0 + 1] = c1 + base;
      if (t0 + 2 < n_tiles) out[t0 + 2] = c2 + base;
    }
    carry += tot;
  }
}

// counts[c][t] -> exclusive prefix over the chunks c; tile totals; tile ranges.  A block owns 32 tiles; its eight warps
// split the chunks (each warp sums its share, the shares are combined in shared memory, then each warp rewrites its
// share), so the chains of dependent loads are an eighth as long.  The block that arrives last scans the tile totals
// into the ranges.
constexpr int TB_THREADS = 256;
constexpr int TB_PARTS = TB_THREADS / 32;

__global__ void __launch_bounds__(TB_THREADS)
tile_bases_kernel(uint32_t* __restrict__ counts, uint32_t tiles_pad, uint32_t n_tiles, const uint32_t* __restrict__ num_rows,
                  const uint64_t* __restrict__ num_instances, uint64_t capacity, uint32_t* tile_total,
                  uint32_t* __restrict__ ranges, uint32_t* arrivals, int* status) {
  odin_after_predecessor();
  __shared__ uint32_t s_part[TB_PARTS][32];
  __shared__ uint32_t s_warp[33];
  __shared__ uint32_t s_flag;
  const uint32_t V = *num_rows;
  const uint32_t nchunks = (V + OFFSET_TILE - 1) / OFFSET_TILE;
  const unsigned lane = threadIdx.x & 31, part = threadIdx.x >> 5;
  const uint32_t t = blockIdx.x * 32 + lane;
  const uint32_t per = (nchunks + TB_PARTS - 1) / TB_PARTS;
  const uint32_t c_lo = min(part * per, nchunks), c_hi = min(c_lo + per, nchunks);
  uint32_t* __restrict__ col = counts + t;
  uint32_t mine = 0;
  if (t < n_tiles) {
    uint32_t c = c_lo;
    for (; c + 8 <= c_hi; c += 8) {
      uint32_t v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = col[(size_t)(c + i) * tiles_pad];
#pragma unroll
      for (int i = 0; i < 8; ++i) mine += v[i];
    }
    for (; c < c_hi; ++c) mine += col[(size_t)c * tiles_pad];
  }
  s_part[part][lane] = mine;
  __syncthreads();
  uint32_t acc = 0, all = 0;
#pragma unroll
  for (int q = 0; q < TB_PARTS; ++q) {
    const uint32_t x = s_part[q][lane];
    if (q < (int)part) acc += x;
    all += x;
  }
  if (t < n_tiles) {
    if (part == 0) tile_total[t] = all;
    uint32_t c = c_lo;
    for (; c + 8 <= c_hi; c += 8) {
      uint32_t v[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = col[(size_t)(c + i) * tiles_pad];
#pragma unroll
      for (int i = 0; i < 8; ++i) { col[(size_t)(c + i) * tiles_pad] = acc; acc += v[i]; }
    }
    for (; c < c_hi; ++c) {
      const uint32_t v = col[(size_t)c * tiles_pad];
      col[(size_t)c * tiles_pad] = acc;
      acc += v;
    }
  }
  // the block that arrives last turns the tile totals into the tile ranges
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) s_flag = (atomicAdd(arrivals, 1u) == gridDim.x - 1u) ? 1u : 0u;
  __syncthreads();
  if (!s_flag) return;
  __threadfence();
  if (threadIdx.x == 0 && *num_instances > capacity) odin_set_error(status, ODIN_ERR_CAPACITY);
  const uint32_t cap = (uint32_t)(capacity < 0xffffffffull ? capacity : 0xffffffffull);
  uint32_t carry = 0;
  for (uint32_t b0 = 0; b0 < n_tiles; b0 += TB_THREADS * 4) {
    const uint32_t t0 = b0 + threadIdx.x * 4;
    uint32_t c[4], sum = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      c[k] = (t0 + k < n_tiles) ? ld_volatile_u32(tile_total + t0 + k) : 0u;
      sum += c[k];
    }
    uint32_t tot;
    uint32_t off = carry + odin_block_exclusive_sum(sum, s_warp, &tot);
    carry += tot;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      if (t0 + k < n_tiles) reinterpret_cast<uint2*>(ranges)[t0 + k] = make_uint2(min(off, cap), min(off + c[k], cap));
      off += c[k];
    }
  }
}

// Writes every instance to its final place.  A work item is (chunk of OFFSET_TILE sorted rows, band of `band_rows` tile
// rows); blocks loop over the items.  The rows of the chunk whose rectangle meets the band are compacted in order,
// then handled SC_SUB at a time: every such row sets its bit in the bit vector of each tile it covers inside the band
// (word-major bit matrix [SC_SUB / 32][tiles of the band]), and every tile reads its bits off in order, which is the
// depth order, and writes the row ids behind the position it has reached.
constexpr int SC_THREADS = 256;
constexpr int SC_ITEMS = OFFSET_TILE / SC_THREADS;
constexpr int SC_SUB = 256;
constexpr int SC_WORDS = SC_SUB / 32;
constexpr uint32_t SC_BAND_TILES = SCATTER_MAX_TX;  // tiles of a band: band_rows * TX <= this
// (the rows kept for a band are staged SC_SUB at a time, straight from the registers that hold the chunk's rectangles:
// 32 KB of shared memory per block instead of 64, seven resident blocks instead of three)
constexpr size_t SC_SMEM = (size_t)SC_SUB * (8 + 4 + 4 + 4) + (size_t)SC_WORDS * SC_BAND_TILES * 4 + SC_BAND_TILES * 4;

// EXACT (binning 2): the tiles of a row inside a tile row are the kept span (tilespan.cuh), recomputed from the row's
// centre, conic and threshold as chunk_counts_kernel left them in depth order.
template <bool WIDE, bool EXACT>
__global__ void __launch_bounds__(SC_THREADS)
scatter_instances_kernel(const ushort4* __restrict__ sorted_rect, const float4* __restrict__ sorted_geo4,
                         const float2* __restrict__ sorted_geo2, const uint32_t* __restrict__ sorted_row,
                         const uint32_t* __restrict__ sorted_off, const uint32_t* __restrict__ num_rows,
                         const uint64_t* __restrict__ num_instances, uint32_t capacity, int TX, int TY, int band_rows,
                         const uint32_t* __restrict__ counts, uint32_t tiles_pad, const uint2* __restrict__ ranges,
                         uint32_t* __restrict__ vals, uint64_t* __restrict__ keys64,
                         const uint32_t* __restrict__ depth_bits, uint32_t* __restrict__ item_ticket) {
  odin_after_predecessor();
  extern __shared__ __align__(16) unsigned char sc_smem[];
  ushort4* s_prect = reinterpret_cast<ushort4*>(sc_smem);                    // [SC_SUB] rectangles of the rows of the batch
  uint32_t* s_prow = reinterpret_cast<uint32_t*>(s_prect + SC_SUB);          // [SC_SUB] their row ids
  uint32_t* s_plim = s_prow + SC_SUB;                                        // [SC_SUB] instances they may emit
  uint32_t* s_pidx = s_plim + SC_SUB;                                        // [SC_SUB] place of the row in its chunk
  uint32_t* s_bits = s_pidx + SC_SUB;                                        // [SC_WORDS][band tiles]
  uint32_t* s_pos = s_bits + SC_WORDS * SC_BAND_TILES;                       // [band tiles] next position of the tile
  __shared__ uint32_t s_warp[33];
  const uint32_t V = *num_rows;
  const uint32_t nchunks = (V + OFFSET_TILE - 1) / OFFSET_TILE;
  const uint32_t nbands = ((uint32_t)TY + band_rows - 1) / band_rows;
  const uint32_t items = nchunks * nbands;
  const bool cut = *num_instances > (uint64_t)capacity;  // only then can a row be denied some of its instances
  __shared__ uint32_t s_item;
  while (true) {
    // items by ticket (they differ in cost by the number of rows of the chunk that meet the band)
    __syncthreads();
    if (threadIdx.x == 0) s_item = atomicAdd(item_ticket, 1u);
    __syncthreads();
    const uint32_t item = s_item;
    if (item >= items) break;
    const uint32_t chunk = item / nbands, band = item - chunk * nbands;  // neighbouring blocks share a chunk's rows
    const uint32_t by0 = band * band_rows, by1 = min((uint32_t)TY, by0 + band_rows);
    const uint32_t band_tiles = (by1 - by0) * (uint32_t)TX;
    const uint32_t first = chunk * OFFSET_TILE + threadIdx.x * SC_ITEMS;
    ushort4 rc[SC_ITEMS];
    uint32_t keep = 0;
#pragma unroll
    for (int k = 0; k < SC_ITEMS; ++k) {
      rc[k] = make_ushort4(0, 0, 0, 0);
      if (first + k < V) {
        rc[k] = sorted_rect[first + k];
        if ((uint32_t)rc[k].y < by1 && (uint32_t)rc[k].w > by0 && rc[k].z > rc[k].x) keep |= 1u << k;
      }
    }
    uint32_t npass;
    const uint32_t p0 = odin_block_exclusive_sum((uint32_t)__popc(keep), s_warp, &npass);  // (its barriers also fence
    if (npass == 0) continue;                                                             //  the reuse of s_pos; uniform)
    for (uint32_t t = threadIdx.x; t < band_tiles; t += SC_THREADS) {
      const uint32_t tile = by0 * (uint32_t)TX + t;
      s_pos[t] = ranges[tile].x + counts[(size_t)chunk * tiles_pad + tile];
    }
    __syncthreads();
    for (uint32_t sub = 0; sub < npass; sub += SC_SUB) {
      for (uint32_t i = threadIdx.x; i < SC_WORDS * band_tiles; i += SC_THREADS) s_bits[i] = 0;
      {
        // stage the rows of this batch: kept row number p0 + (kept rows of the thread in front of it)
        uint32_t p = p0;
#pragma unroll
        for (int k = 0; k < SC_ITEMS; ++k) {
          if (keep >> k & 1u) {
            if (p >= sub && p < sub + SC_SUB) {
              const uint32_t q = p - sub;
              s_prect[q] = rc[k];
              s_prow[q] = min(sorted_row[first + k], V - 1);
              uint32_t lim = 0xffffffffu;
              if (cut) {
                const uint32_t off = sorted_off[first + k];
                lim = off < capacity ? capacity - off : 0u;
              }
              s_plim[q] = lim;
              s_pidx[q] = threadIdx.x * SC_ITEMS + k;
            }
            ++p;
          }
        }
      }
      __syncthreads();
      {
        // Tile row by tile row of the band: the tiles of a row of the list inside one tile row are a run [xa, xa + len).
        // A lane sets the bits of a short run by itself; the long runs of a warp are then taken one at a time by all 32
        // lanes (one tile per lane and step), so that a splat as wide as the image costs the warp a few steps instead
        // of one lane a hundred.
        const uint32_t j = sub + threadIdx.x;
        const unsigned lane = threadIdx.x & 31;
        uint32_t* word = s_bits + (threadIdx.x >> 5) * band_tiles;  // the warp's 32 rows are the bits of these words
        uint32_t rx = 0, ry = 0, ry1 = 0, w = 1, lim = 0, x1 = 0;
        SpanConic e;
        e.k = -1.f;
        if (j < npass) {
          const ushort4 r = s_prect[threadIdx.x];
          rx = r.x; ry = r.y; ry1 = r.w; w = (uint32_t)r.z - (uint32_t)r.x; lim = s_plim[threadIdx.x];
          x1 = min((uint32_t)r.z, (uint32_t)TX);
          if (EXACT) {
            const uint32_t gi = chunk * OFFSET_TILE + s_pidx[threadIdx.x];
            const float4 g4 = sorted_geo4[gi];
            const float2 g2 = sorted_geo2[gi];
            e.u = g4.x; e.v = g4.y; e.A = g4.z; e.B = g4.w; e.C = g2.x; e.k = g2.y;
          }
        }
        for (uint32_t y = by0; y < by1; ++y) {
          uint32_t xa = 0, len = 0, k0 = 0;  // the lane's run in this tile row; k0: index of its first instance in the row
          if (j < npass && y >= ry && y < ry1) {
            if (EXACT) {
              int a, b;
              odin_row_span(e, (int)y, (int)rx, (int)x1, a, b);
              xa = (uint32_t)a; len = (uint32_t)(b - a);
              if (cut && len != 0)  // instances of the tile rows above (rare path: the view overflows the capacity)
                for (uint32_t yy = ry; yy < y; ++yy) {
                  odin_row_span(e, (int)yy, (int)rx, (int)x1, a, b);
                  k0 += (uint32_t)(b - a);
                }
            } else {
              xa = rx; len = x1 > rx ? x1 - rx : 0u; k0 = (y - ry) * w;
            }
          }
          uint32_t* line = word + (y - by0) * (uint32_t)TX;
          const bool large = len > 16;
          if (!large) {
            const uint32_t bit = 1u << lane;
            for (uint32_t i = 0; i < len; ++i)
              if (k0 + i < lim) atomicOr(line + xa + i, bit);  // other lanes of the warp may hold the same tile
          }
          uint32_t todo = __ballot_sync(0xffffffffu, large);
          __syncwarp();
          while (todo) {
            const int src = __ffs(todo) - 1;
            todo &= todo - 1;
            const uint32_t q_xa = __shfl_sync(0xffffffffu, xa, src), q_len = __shfl_sync(0xffffffffu, len, src);
            const uint32_t q_k0 = __shfl_sync(0xffffffffu, k0, src), q_lim = __shfl_sync(0xffffffffu, lim, src);
            const uint32_t bit = 1u << src;
            for (uint32_t c = lane; c < q_len; c += 32)  // distinct tiles per lane: no two lanes share a word here
              if (q_k0 + c < q_lim) line[q_xa + c] |= bit;
            __syncwarp();
          }
        }
      }
      __syncthreads();
      for (uint32_t t = threadIdx.x; t < band_tiles; t += SC_THREADS) {
        uint32_t pos = s_pos[t];
#pragma unroll
        for (int wd = 0; wd < SC_WORDS; ++wd) {
          uint32_t bits = s_bits[wd * band_tiles + t];
          while (bits) {
            const int b = __ffs(bits) - 1;
            bits &= bits - 1;
            const uint32_t row = s_prow[wd * 32 + b];
            if (pos < capacity) {
              vals[pos] = row;
              if (WIDE) keys64[pos] = ((uint64_t)(by0 * (uint32_t)TX + t) << 32) | (uint64_t)depth_bits[row];
            }
            ++pos;
          }
        }
        s_pos[t] = pos;
      }
      __syncthreads();
    }
  }
}

int tile_digit_passes(uint32_t n_tiles) {
  int tile_bits = 0;
  while ((1ull << tile_bits) < (unsigned long long)n_tiles) ++tile_bits;
  const int p = (tile_bits + (int)SORT_RADIX_BITS - 1) / (int)SORT_RADIX_BITS;
  return p < 1 ? 1 : p;  // a one-tile image still takes one pass, which moves the emission into the outputs
}

}  // namespace

extern "C" int odin_bin_sort_workspace_bytes(const odin_ctx* ctx, uint32_t row_capacity, uint64_t max_instances, int width,
                                            int height, size_t* bytes) {
  if (!ctx || !bytes) return ODIN_ERR_NULL;
  if (width <= 0 || height <= 0 || width > 16384 || height > 16384) return ODIN_ERR_INVALID_ARG;
  const int TX = (width + 15) / 16, TY = (height + 15) / 16;
  const uint32_t n_tiles = (uint32_t)TX * (uint32_t)TY;
  if (ctx->cfg.instance_sort != 1 && scatter_eligible(TX, n_tiles)) *bytes = scatter_layout(row_capacity, n_tiles).total;
  else *bytes = binsort_ws_bytes(max_instances, row_capacity);
  return ODIN_OK;
}

extern "C" int odin_bin_sort(odin_ctx* ctx, const odin_projected* proj, int width, int height, uint64_t* d_keys,
                             uint32_t* d_vals, uint64_t capacity, uint32_t* d_tile_ranges, void* ws, size_t ws_bytes,
                             void* stream) {
  if (!ctx || !proj || !d_tile_ranges) return ODIN_ERR_NULL;
  if (width <= 0 || height <= 0 || width > 16384 || height > 16384) return ODIN_ERR_INVALID_ARG;
  if (!proj->num_rows || !proj->num_instances) return ODIN_ERR_NULL;
  if (capacity >= (1ull << 30) || proj->capacity >= (1u << 30)) return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const int TX = (width + 15) / 16, TY = (height + 15) / 16;
  const uint32_t n_tiles = (uint32_t)TX * (uint32_t)TY;
  if (!odin_aligned(d_tile_ranges, 8)) return ODIN_ERR_INVALID_ARG;
  if (capacity == 0 || proj->capacity == 0) {
    odin_chain_break(ctx);
    ODIN_CUDA(cudaMemsetAsync(d_tile_ranges, 0, (size_t)n_tiles * 8, st));
    return ODIN_OK;
  }
  if (!d_vals || !proj->rect || !proj->depth) return ODIN_ERR_NULL;
  if ((d_keys && !odin_aligned(d_keys, 16)) || !odin_aligned(d_vals, 16) || !odin_aligned(proj->rect, 8))
    return ODIN_ERR_INVALID_ARG;
  const bool scatter = ctx->cfg.instance_sort != 1 && scatter_eligible(TX, n_tiles);
  const ScatterLayout F = scatter_layout(proj->capacity, n_tiles);
  const BinSortLayout L = binsort_layout(capacity, proj->capacity);
  const bool use_scatter = scatter && ws && ws_bytes >= F.total;
  const bool exact = ctx->cfg.binning == 2;
  if (exact && !use_scatter) return ODIN_ERR_UNSUPPORTED;  // the spans of exact binning exist in the scatter path only
  if (exact && (!proj->xy || !proj->conic_opacity)) return ODIN_ERR_NULL;
  if (!ws || !odin_aligned(ws, 256) || (!use_scatter && ws_bytes < L.total)) return ODIN_ERR_WORKSPACE;
  char* base = reinterpret_cast<char*>(ws);
  const int tile_passes = tile_digit_passes(n_tiles);
  // the regions both paths share (tickets, row histograms, look-back words of the row passes, ping-pong row buffers)
  const size_t o_hist = use_scatter ? F.hist : L.hist, o_dbase = use_scatter ? F.digit_base : L.digit_base;
  const size_t o_scan = use_scatter ? F.scan_state : L.scan_state, o_rstates = use_scatter ? F.row_states : L.row_states;
  const uint32_t row_tiles = use_scatter ? F.row_tiles : L.row_tiles;
  if (use_scatter) {
    // zero tickets, histograms and the look-back words of the offset scan and of the row passes
    ODIN_CUDA(odin_zero(ctx, base, F.row_keys[0], st));
  } else {
    // zero tickets, histograms, the used part of the difference array and the look-back words of the passes that run
    ODIN_CUDA(odin_zero(ctx, base, L.tile_diff + ((size_t)n_tiles + 1) * 4, st));
    ODIN_CUDA(odin_zero(ctx, base + L.scan_state,
                              L.inst_states + (size_t)tile_passes * L.tiles * SORT_RADIX * 4 - L.scan_state, st));
  }
  uint32_t* tickets = reinterpret_cast<uint32_t*>(base);
  uint32_t* hist = reinterpret_cast<uint32_t*>(base + o_hist);
  uint32_t* dbase = reinterpret_cast<uint32_t*>(base + o_dbase);
  uint64_t* scan_state = reinterpret_cast<uint64_t*>(base + o_scan);
  uint32_t* row_states = reinterpret_cast<uint32_t*>(base + o_rstates);
  uint32_t* row_keys[2], *row_vals[2];
  for (int b = 0; b < 2; ++b) {
    row_keys[b] = reinterpret_cast<uint32_t*>(base + (use_scatter ? F.row_keys[b] : L.row_keys[b]));
    row_vals[b] = reinterpret_cast<uint32_t*>(base + (use_scatter ? F.row_vals[b] : L.row_vals[b]));
  }
  uint32_t* sorted_off = reinterpret_cast<uint32_t*>(base + (use_scatter ? F.sorted_off : L.sorted_off));
  const uint32_t* depth_bits = reinterpret_cast<const uint32_t*>(proj->depth);
  const ushort4* rect = reinterpret_cast<const ushort4*>(proj->rect);
  const uint32_t sms = (uint32_t)ctx->sm_count;
  const uint32_t row_blocks = (proj->capacity + RH_THREADS - 1) / RH_THREADS;

  // ---- rows by depth
  {
    OdinKernelScope ks(ctx, K_ROW_HIST, st);
    // one block per SM at most: every block ends with 1024 global reductions onto the same 1024 words
    ODIN_CUDA(odin_launch(ctx, false, row_hist_kernel, dim3(row_blocks < sms ? row_blocks : sms), dim3(RH_THREADS), 0, st,
                          depth_bits, proj->num_rows, hist, dbase, tickets + 9));
  }
  constexpr size_t OS_SMEM = os_smem_bytes(OS_INST_ITEMS, OS_THREADS), OS_ROW_SMEM = os_smem_bytes(OS_ROW_ITEMS, OS_ROW_THREADS);
  const uint32_t* sorted_row = nullptr;
  {
    const uint32_t row_resident = sms * (OS_RESIDENT / OS_ROW_THREADS);
    const uint32_t grid = row_tiles < row_resident ? row_tiles : row_resident;
    const uint32_t* kin = depth_bits;
    const uint32_t* vin = nullptr;
    for (int p = 0; p < SORT_DEPTH_DIGITS; ++p) {
      OdinKernelScope ks(ctx, K_ROW_SORT, st);
      uint32_t* kout = (p + 1 < SORT_DEPTH_DIGITS) ? row_keys[p & 1] : nullptr;
      uint32_t* vout = row_vals[p & 1];
      ODIN_CUDA(odin_launch(ctx, true, onesweep_kernel<false, OS_ROW_ITEMS, OS_ROW_WINDOW, OS_ROW_THREADS>, dim3(grid), dim3(OS_ROW_THREADS),
                            OS_ROW_SMEM, st, kin, vin, kout, vout, nullptr, nullptr, proj->num_rows, nullptr, 0,
                            p * (int)SORT_RADIX_BITS, dbase + p * SORT_RADIX,
                            row_states + (size_t)p * row_tiles * SORT_RADIX, tickets + p, ctx->d_status, ctx->spin_limit,
                            proj->capacity));
      kin = kout;
      vin = vout;
    }
    sorted_row = vin;
  }
  if (use_scatter) {
    // ---- instances straight to their final places
    ushort4* sorted_rect = reinterpret_cast<ushort4*>(base + F.sorted_rect);
    uint32_t* tile_total = reinterpret_cast<uint32_t*>(base + F.tile_total);
    uint32_t* counts = reinterpret_cast<uint32_t*>(base + F.counts);
    float4* geo4 = reinterpret_cast<float4*>(base + F.sorted_geo4);
    float2* geo2 = reinterpret_cast<float2*>(base + F.sorted_geo2);
    const uint32_t cap32 = (uint32_t)capacity;
    {
      OdinKernelScope ks(ctx, K_ROW_OFFSETS, st);
      const size_t smem = ((size_t)F.tiles_pad + 8) * 4;
      const int max_smem = (int)(((size_t)SCATTER_MAX_TILES + 64 + 8) * 4);
      static_assert(RO_THREADS * RO_ITEMS == (int)OFFSET_TILE && 1024 * 2 == (int)OFFSET_TILE, "rows per chunk");
      ODIN_CUDA(cudaFuncSetAttribute(chunk_counts_kernel<false, 1024, 2>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
      ODIN_CUDA(cudaFuncSetAttribute(chunk_counts_kernel<true, 1024, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     max_smem));
#define LAUNCH_COUNTS(EXACT, THREADS, ITEMS)                                                                           \
  ODIN_CUDA(odin_launch(ctx, true, chunk_counts_kernel<EXACT, THREADS, ITEMS>, dim3(F.chunks), dim3(THREADS), smem, st, \
                        sorted_row, rect, reinterpret_cast<const float2*>(proj->xy),                                     \
                        reinterpret_cast<const float4*>(proj->conic_opacity), ctx->cfg.alpha_min, proj->num_rows,        \
                        proj->num_instances, cap32, TX, n_tiles, F.tiles_pad, sorted_off, sorted_rect, geo4, geo2,       \
                        counts, tickets + 8, scan_state, ctx->d_status, ctx->spin_limit))
      if (exact) LAUNCH_COUNTS(true, 1024, 2);
      else LAUNCH_COUNTS(false, 1024, 2);
#undef LAUNCH_COUNTS
    }
    {
      OdinKernelScope ks(ctx, K_TILE_BASES, st);
      ODIN_CUDA(odin_launch(ctx, true, tile_bases_kernel, dim3((n_tiles + 31) / 32), dim3(TB_THREADS), 0, st, counts,
                            F.tiles_pad, n_tiles, proj->num_rows, proj->num_instances, capacity, tile_total,
                            d_tile_ranges, tickets + 10, ctx->d_status));
    }
    {
      OdinKernelScope ks(ctx, K_EMIT, st);
      // two tile rows per band: the bit matrix of a band is mostly empty (a depth-ordered batch of rows is scattered
      // over the image), and the words to clear and to read off grow with the band while the instances do not
      // (measured at 1600 x 1066 and 1920 x 1080: 1 / 2 / 3 / 7 rows -> 0.170 / 0.145 / 0.160 / 0.183 ms)
      int band_rows = (int)(SC_BAND_TILES / (uint32_t)TX);
      if (band_rows > 2) band_rows = 2;
      if (band_rows > TY) band_rows = TY;
      const uint64_t items_cap = (uint64_t)F.chunks * (((uint32_t)TY + band_rows - 1) / band_rows);
      const uint32_t grid = (uint32_t)(items_cap < (uint64_t)sms * 6 ? items_cap : (uint64_t)sms * 6);
#define LAUNCH_SCATTER(WIDE, EXACT)                                                                                    \
  do {                                                                                                                 \
    ODIN_CUDA(cudaFuncSetAttribute(scatter_instances_kernel<WIDE, EXACT>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                                   (int)SC_SMEM));                                                                     \
    ODIN_CUDA(odin_launch(ctx, true, scatter_instances_kernel<WIDE, EXACT>, dim3(grid), dim3(SC_THREADS), SC_SMEM, st,  \
                          sorted_rect, geo4, geo2, sorted_row, sorted_off, proj->num_rows, proj->num_instances, cap32,  \
                          TX, TY, band_rows, counts, F.tiles_pad, reinterpret_cast<const uint2*>(d_tile_ranges), d_vals, \
                          d_keys, depth_bits, tickets + 11));                                                           \
  } while (0)
      if (d_keys) { if (exact) LAUNCH_SCATTER(true, true); else LAUNCH_SCATTER(true, false); }
      else { if (exact) LAUNCH_SCATTER(false, true); else LAUNCH_SCATTER(false, false); }
#undef LAUNCH_SCATTER
    }
    return odin_launch_status();
  }
  ODIN_CUDA(cudaFuncSetAttribute(onesweep_kernel<false, OS_INST_ITEMS, OS_INST_WINDOW, OS_THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)OS_SMEM));
  ODIN_CUDA(cudaFuncSetAttribute(onesweep_kernel<true, OS_INST_ITEMS, OS_INST_WINDOW, OS_THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)OS_SMEM));
  uint32_t* tile_diff = reinterpret_cast<uint32_t*>(base + L.tile_diff);
  uint32_t* inst_states = reinterpret_cast<uint32_t*>(base + L.inst_states);
  uint32_t* inst_keys[2] = {reinterpret_cast<uint32_t*>(base + L.inst_keys[0]), reinterpret_cast<uint32_t*>(base + L.inst_keys[1])};
  uint32_t* inst_vals[2] = {d_vals, reinterpret_cast<uint32_t*>(base + L.alt_vals)};
  uint32_t* chunk_row = reinterpret_cast<uint32_t*>(base + L.chunk_row);
  // ---- instances in depth order
  uint32_t* tile_dbase = dbase + SORT_DEPTH_DIGITS * SORT_RADIX;
  const uint64_t chunks_cap = (capacity + DUP_CHUNK - 1) / DUP_CHUNK;
  {
    OdinKernelScope ks(ctx, K_ROW_OFFSETS, st);
    // shared-memory staging of the difference array for images of up to 40,000 tiles (e.g. 4096 x 2304)
    const uint32_t diff_words = n_tiles + 1 <= 40001u ? n_tiles + 1 : 0u;
    const size_t diff_smem = (size_t)diff_words * 4;
    ODIN_CUDA(cudaFuncSetAttribute(sorted_offsets_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 40001 * 4));
    ODIN_CUDA(odin_launch(ctx, true, sorted_offsets_kernel, dim3((proj->capacity + OFFSET_TILE - 1) / OFFSET_TILE),
                          dim3(RO_THREADS), diff_smem, st, sorted_row, rect, proj->num_rows, (uint32_t)capacity, TX,
                          sorted_off, chunk_row, (uint32_t)chunks_cap, tile_diff, diff_words, tickets + 8, scan_state,
                          ctx->d_status, ctx->spin_limit));
  }
  // the emission goes to the buffers from which `tile_passes` ping-pong steps end in d_vals
  int cur = tile_passes & 1;
  {
    OdinKernelScope ks(ctx, K_EMIT, st);
    const uint32_t grid = (uint32_t)(chunks_cap < (uint64_t)sms * 5 - 1 ? chunks_cap : (uint64_t)sms * 5 - 1) + 1;
    ODIN_CUDA(odin_launch(ctx, true, emit_instances_kernel, dim3(grid), dim3(DUP_THREADS), 0, st, sorted_off, sorted_row,
                          chunk_row, rect, proj->num_rows, proj->num_instances, capacity, TX, inst_keys[cur], inst_vals[cur],
                          ctx->d_status, tile_diff, n_tiles, tile_passes, d_tile_ranges, tile_dbase));
  }
  // ---- instances by tile id
  const uint32_t os_grid = L.tiles < sms * (OS_RESIDENT / OS_THREADS) ? L.tiles : sms * (OS_RESIDENT / OS_THREADS);
  for (int p = 0; p < tile_passes; ++p) {
    OdinKernelScope ks(ctx, K_ONESWEEP, st);
    uint32_t* states = inst_states + (size_t)p * L.tiles * SORT_RADIX;
    if (p + 1 < tile_passes)
      ODIN_CUDA(odin_launch(ctx, true, onesweep_kernel<false, OS_INST_ITEMS, OS_INST_WINDOW, OS_THREADS>, dim3(os_grid),
                            dim3(OS_THREADS), OS_SMEM, st, inst_keys[cur], inst_vals[cur], inst_keys[cur ^ 1],
                            inst_vals[cur ^ 1], nullptr, nullptr, nullptr, proj->num_instances, capacity,
                            p * (int)SORT_RADIX_BITS, tile_dbase + p * SORT_RADIX, states,
                            tickets + SORT_DEPTH_DIGITS + p, ctx->d_status, ctx->spin_limit, proj->capacity));
    else  // the sorted tile ids themselves are not needed any more: the ranges came from the tile counts
      ODIN_CUDA(odin_launch(ctx, true, onesweep_kernel<true, OS_INST_ITEMS, OS_INST_WINDOW, OS_THREADS>, dim3(os_grid),
                            dim3(OS_THREADS), OS_SMEM, st, inst_keys[cur], inst_vals[cur], nullptr, inst_vals[cur ^ 1],
                            d_keys, depth_bits, nullptr, proj->num_instances, capacity, p * (int)SORT_RADIX_BITS,
                            tile_dbase + p * SORT_RADIX, states, tickets + SORT_DEPTH_DIGITS + p, ctx->d_status,
                            ctx->spin_limit, proj->capacity));
    cur ^= 1;
  }
  return odin_launch_status();
}
