// Touched-set bitmask + ascending index list (single pass, decoupled look-back) and pairwise intersection counts.
#include <atomic>

#include "common.cuh"
#include "layout.cuh"

namespace {

constexpr int TS_THREADS = 256;
constexpr int TS_ITEMS = TOUCHED_TILE / TS_THREADS;  // 8 words of 32 primitives per warp

// A block takes `scan_rounds` x 2048 consecutive primitives by ticket; each of its eight warps owns a contiguous eighth
// of them.  Load q of lane l is primitive span_base + 32 q + l, so one ballot is one mask word and ranks inside the
// warp follow the primitive order.  The ballots are kept (word q in lane q % 32), so the list is written after the
// look-back without reading the counts a second time.
constexpr int TS_MAX_ROUNDS = 8;

// FROM_MASK: the input is itself a bitmask over the primitives (`tiles_touched` then points at its words): the kernel
// only lists its members (the index list of a union of scopes, for example) and writes no mask.
template <bool FROM_MASK>
__global__ void __launch_bounds__(TS_THREADS)
touched_set_kernel(const uint32_t* __restrict__ tiles_touched, uint32_t n, uint32_t* __restrict__ mask,
                   uint32_t* __restrict__ idx, uint32_t idx_capacity, uint32_t* __restrict__ count, uint32_t* ticket,
                   uint64_t* state, int* status, int scan_rounds, int spin_limit) {
  const uint32_t scan_chunk = TOUCHED_TILE * (uint32_t)scan_rounds;
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_warp[33];
  __shared__ uint64_t s_base;
  if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int words = scan_rounds * TS_ITEMS;  // mask words (ballots) per warp: 8 .. 64
  const uint32_t span_base = tile * scan_chunk + warp * (uint32_t)words * 32u;
  const uint32_t n_words = (n + 31) / 32;
  // pass A: ballots of the warp's span; word q stays in lane q % 32 of keep[q / 32]
  uint32_t keep[TS_MAX_ROUNDS * TS_ITEMS / 32] = {0u, 0u};
  uint32_t warp_count = 0;
#pragma unroll 8
  for (int q = 0; q < words; ++q) {
    const uint32_t p = span_base + 32u * (uint32_t)q + lane;
    uint32_t bal;
    if (FROM_MASK) {
      const uint32_t word = span_base / 32 + (uint32_t)q;
      bal = word < n_words ? tiles_touched[word] : 0u;
      if (word == n_words - 1 && (n & 31u)) bal &= (1u << (n & 31u)) - 1u;  // bits past n do not name primitives
    } else {
      bal = __ballot_sync(0xffffffffu, p < n && tiles_touched[p] > 0);
    }
    warp_count += __popc(bal);
    if (lane == (unsigned)(q & 31)) keep[q >> 5] = bal;
  }
  // the mask words of the span: 32 consecutive words per store
  if (!FROM_MASK)
    for (int h = 0; h * 32 < words; ++h) {
      const uint32_t word = span_base / 32 + h * 32 + lane;
      if ((int)(h * 32 + lane) < words && word < n_words) mask[word] = keep[h];
    }
  uint32_t chunk_total;
  const uint32_t scan = odin_block_exclusive_sum(lane == 0 ? warp_count : 0u, s_warp, &chunk_total);
  const uint32_t warp_off = __shfl_sync(0xffffffffu, scan, 0);
  if (threadIdx.x < 32) {
    const uint64_t ex = odin_lookback_u64(state, tile, (uint64_t)chunk_total, status, spin_limit);
    if (threadIdx.x == 0) s_base = ex;
  }
  __syncthreads();
  const uint64_t base = s_base;
  if (tile == (n + scan_chunk - 1) / scan_chunk - 1 && threadIdx.x == 0) {
    const uint64_t v = base + chunk_total;
    *count = (uint32_t)(v < idx_capacity ? v : idx_capacity);
    if (v > idx_capacity) odin_set_error(status, ODIN_ERR_CAPACITY);
  }
  // pass B: the ascending list from the kept ballots
  uint64_t pos = base + warp_off;
  const uint32_t lt = (1u << lane) - 1u;
  for (int q = 0; q < words; ++q) {
    const uint32_t bal = __shfl_sync(0xffffffffu, keep[q >> 5], q & 31);
    if (bal >> lane & 1u) {
      const uint64_t dst = pos + __popc(bal & lt);
      if (dst < idx_capacity) idx[dst] = span_base + 32u * (uint32_t)q + lane;
    }
    pos += __popc(bal);
  }
}

constexpr int CC_THREADS = 256;

// One block column per pair (blockIdx.y); blocks of a column stride over the mask words four at a time.
__global__ void __launch_bounds__(CC_THREADS)
conflict_count_kernel(const uint32_t* __restrict__ masks, uint32_t stride_words, uint32_t words,
                      const uint32_t* __restrict__ pairs, uint32_t n_masks, unsigned long long* __restrict__ counts,
                      int* status) {
  odin_after_predecessor();
  const uint32_t pair = blockIdx.y;
  const uint32_t va = pairs[2 * pair], vb = pairs[2 * pair + 1];
  if (va >= n_masks || vb >= n_masks) {  // uniform over the block: a pair naming a missing view counts 0
    if (threadIdx.x == 0) odin_set_error(status, ODIN_ERR_INVALID_ARG);
    return;
  }
  const uint32_t* a = masks + (size_t)va * stride_words;
  const uint32_t* b = masks + (size_t)vb * stride_words;
  uint32_t c = 0;
  const uint32_t vec = words / 4;
  const uint4* a4 = reinterpret_cast<const uint4*>(a);
  const uint4* b4 = reinterpret_cast<const uint4*>(b);
  for (uint32_t i = blockIdx.x * CC_THREADS + threadIdx.x; i < vec; i += gridDim.x * CC_THREADS) {
    const uint4 x = a4[i], y = b4[i];
    c += __popc(x.x & y.x) + __popc(x.y & y.y) + __popc(x.z & y.z) + __popc(x.w & y.w);
  }
  if (blockIdx.x == 0)
    for (uint32_t i = vec * 4 + threadIdx.x; i < words; i += CC_THREADS) c += __popc(a[i] & b[i]);
  for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
  __shared__ uint32_t s[CC_THREADS / 32];
  if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t tot = 0;
    for (int i = 0; i < CC_THREADS / 32; ++i) tot += s[i];
    if (tot) atomicAdd(&counts[pair], (unsigned long long)tot);
  }
}

}  // namespace

extern "C" int odin_touched_set(odin_ctx* ctx, const uint32_t* d_tiles_touched, uint32_t n, uint32_t* d_mask,
                                uint32_t* d_idx, uint32_t idx_capacity, uint32_t* d_count, void* ws, size_t ws_bytes,
                                void* stream) {
  if (!ctx || !d_count) return ODIN_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  if (n >= (1u << 28)) return ODIN_ERR_INVALID_ARG;
  if (n == 0) {
    odin_chain_break(ctx);
    ODIN_CUDA(cudaMemsetAsync(d_count, 0, 4, st));
    return ODIN_OK;
  }
  if (!d_tiles_touched || !d_mask || (idx_capacity > 0 && !d_idx)) return ODIN_ERR_NULL;
  const size_t need = touched_ws_bytes(n);
  if (!ws || !odin_aligned(ws, 256) || ws_bytes < need) return ODIN_ERR_WORKSPACE;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(ws, 0, need, st));
  uint32_t* ticket = reinterpret_cast<uint32_t*>(ws);
  uint64_t* state = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(ws) + 256);
  const int scan_rounds = scan_rounds_for(n, ctx->sm_count);
  const uint32_t scan_chunk = TOUCHED_TILE * (uint32_t)scan_rounds;
  const uint32_t grid = (n + scan_chunk - 1) / scan_chunk;
  OdinKernelScope ks(ctx, K_TOUCHED, st);
  touched_set_kernel<false><<<grid, TS_THREADS, 0, st>>>(d_tiles_touched, n, d_mask, d_idx, idx_capacity, d_count, ticket,
                                                         state, ctx->d_status, scan_rounds, ctx->spin_limit);
  return odin_launch_status();
}

extern "C" int odin_mask_to_list(odin_ctx* ctx, const uint32_t* d_mask, uint32_t n, uint32_t* d_idx, uint32_t idx_capacity,
                                 uint32_t* d_count, void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || !d_count) return ODIN_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  if (n >= (1u << 28)) return ODIN_ERR_INVALID_ARG;
  if (n == 0) {
    odin_chain_break(ctx);
    ODIN_CUDA(cudaMemsetAsync(d_count, 0, 4, st));
    return ODIN_OK;
  }
  if (!d_mask || (idx_capacity > 0 && !d_idx)) return ODIN_ERR_NULL;
  const size_t need = touched_ws_bytes(n);
  if (!ws || !odin_aligned(ws, 256) || ws_bytes < need) return ODIN_ERR_WORKSPACE;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemsetAsync(ws, 0, need, st));
  uint32_t* ticket = reinterpret_cast<uint32_t*>(ws);
  uint64_t* state = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(ws) + 256);
  const int scan_rounds = scan_rounds_for(n, ctx->sm_count);
  const uint32_t scan_chunk = TOUCHED_TILE * (uint32_t)scan_rounds;
  OdinKernelScope ks(ctx, K_TOUCHED, st);
  touched_set_kernel<true><<<(n + scan_chunk - 1) / scan_chunk, TS_THREADS, 0, st>>>(
      d_mask, n, nullptr, d_idx, idx_capacity, d_count, ticket, state, ctx->d_status, scan_rounds, ctx->spin_limit);
  return odin_launch_status();
}

// ---------------------------------------------------------------------------------------------------------------
// Touched set without any allocation.  Some users of this library are handed all of their GPU memory up front and may
// never allocate again: a component embedded in a host application that owns the memory pool, or a real-time loop in
// which an allocation could stall or fail at a bad moment.  They cannot call odin_create (it allocates the status word)
// nor size and allocate a workspace.  For them this entry point runs the same kernel as odin_touched_set with its
// scratch (tile ticket, deferred-status sink, look-back words) in a fixed array that is part of the loaded library:
// every GPU that loads libodin.so holds these 128.3 KB until the process exits.
constexpr uint32_t TS_STATIC_MAX_N = 1u << 25;  // 33,554,432 primitives
constexpr size_t TS_STATIC_HEADER = 256;        // [0] ticket, [64] status sink
constexpr size_t TS_STATIC_BYTES = TS_STATIC_HEADER + (size_t)(TS_STATIC_MAX_N / TOUCHED_TILE) * 8;
static __device__ __align__(256) unsigned char g_touched_static_scratch[TS_STATIC_BYTES];

// In host code the array's name is only a handle for the runtime, not a device address, so the address is asked for
// once per device (with that device current) and cached.  The cache entries are atomics: two host threads that make
// the first call on a device at the same time both look the address up and store the same value.
constexpr int TS_STATIC_MAX_DEVICES = 64;
static std::atomic<unsigned char*> g_touched_static_ptr[TS_STATIC_MAX_DEVICES];

extern "C" int odin_touched_set_static(const uint32_t* d_tiles_touched, uint32_t n, uint32_t* d_mask, uint32_t* d_idx,
                                       uint32_t idx_capacity, uint32_t* d_count, int* d_status, void* stream) {
  if (!d_count) return ODIN_ERR_NULL;
  if (n > TS_STATIC_MAX_N) return ODIN_ERR_INVALID_ARG;  // beyond the fixed scratch: use odin_touched_set
  cudaStream_t st = (cudaStream_t)stream;
  if (n == 0) {
    ODIN_CUDA(cudaMemsetAsync(d_count, 0, 4, st));
    return ODIN_OK;
  }
  if (!d_tiles_touched || !d_mask || (idx_capacity > 0 && !d_idx)) return ODIN_ERR_NULL;
  int device = -1;
  ODIN_CUDA(cudaGetDevice(&device));
  if (device < 0 || device >= TS_STATIC_MAX_DEVICES) return ODIN_ERR_UNSUPPORTED;
  unsigned char* scratch = g_touched_static_ptr[device].load(std::memory_order_acquire);
  if (!scratch) {  // first call on this device: resolve the array's device address (this may load the module)
    void* p = nullptr;
    ODIN_CUDA(cudaGetSymbolAddress(&p, g_touched_static_scratch));
    if (!p) return ODIN_ERR_CUDA;
    scratch = static_cast<unsigned char*>(p);
    g_touched_static_ptr[device].store(scratch, std::memory_order_release);
  }
  const uint32_t tiles = (n + TOUCHED_TILE - 1) / TOUCHED_TILE;
  // the array keeps whatever the previous call left: the ticket, the sink and the look-back words must start at zero
  ODIN_CUDA(cudaMemsetAsync(scratch, 0, TS_STATIC_HEADER + (size_t)tiles * 8, st));
  uint32_t* ticket = reinterpret_cast<uint32_t*>(scratch);
  int* status = d_status ? d_status : reinterpret_cast<int*>(scratch + 64);
  uint64_t* state = reinterpret_cast<uint64_t*>(scratch + TS_STATIC_HEADER);
  // no context here, so the SM count is not looked up: the block size is chosen for the 148 SMs of a B200 (any other
  // count only changes how many blocks share the work, never the result)
  const int scan_rounds = scan_rounds_for(n, 148);
  const uint32_t scan_chunk = TOUCHED_TILE * (uint32_t)scan_rounds;
  touched_set_kernel<false><<<(n + scan_chunk - 1) / scan_chunk, TS_THREADS, 0, st>>>(
      d_tiles_touched, n, d_mask, d_idx, idx_capacity, d_count, ticket, state, status, scan_rounds,
      ODIN_DEFAULT_SPIN_LIMIT);
  return odin_launch_status();
}

extern "C" int odin_conflict_count(odin_ctx* ctx, const uint32_t* d_masks, uint32_t n_masks, uint32_t mask_stride_words,
                                   uint32_t n_prims, const uint32_t* d_pairs, uint32_t n_pairs, uint64_t* d_counts,
                                   void* stream) {
  if (!ctx) return ODIN_ERR_NULL;
  if (n_pairs == 0) return ODIN_OK;
  if (!d_pairs || !d_counts) return ODIN_ERR_NULL;
  if (n_pairs > 65535) return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  ODIN_CUDA(odin_zero(ctx, d_counts, (size_t)n_pairs * 8, st));
  const uint32_t words = (n_prims + 31) / 32;
  if (words == 0) return ODIN_OK;
  if (!d_masks) return ODIN_ERR_NULL;
  if (n_masks == 0 || mask_stride_words < words || (mask_stride_words % 4) != 0 || !odin_aligned(d_masks, 16))
    return ODIN_ERR_INVALID_ARG;
  uint32_t gx = (words / 4 + CC_THREADS - 1) / CC_THREADS;
  const uint32_t cap = (uint32_t)(ctx->sm_count * 8 + n_pairs - 1) / n_pairs;
  if (gx > cap) gx = cap;
  if (gx == 0) gx = 1;
  OdinKernelScope ks(ctx, K_CONFLICT, st);
  ODIN_CUDA(odin_launch(ctx, false, conflict_count_kernel, dim3(gx, n_pairs), dim3(CC_THREADS), 0, st, d_masks,
                        mask_stride_words, words, d_pairs, n_masks, reinterpret_cast<unsigned long long*>(d_counts),
                        ctx->d_status));
  return odin_launch_status();
}
