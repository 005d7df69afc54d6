// Shared internals of the CUDA library: context, argument checks, bounded decoupled look-back.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>
#include <vector>

#include "../../include/odin.h"

// Kernel ids for launch counting and optional per-kernel CUDA-event timing.
enum OdinKernelId {
  K_PROJECT = 0, K_TOUCHED, K_EMIT, K_ONESWEEP, K_FWD, K_L1, K_ZERO_ROWS,
  K_BWD_BLEND, K_BWD_PROJECT, K_ADAM_SH, K_ADAM_GEOM, K_CONFLICT, K_FWD_TAIL, K_PROJECT_SCAN,
  K_PROJECT_ROWS, K_ROW_HIST, K_ROW_SORT, K_ROW_OFFSETS, K_ACTIVE_SET, K_MASK_UNION, K_HAZARD,
  K_GATE, K_RLG, K_TILE_BASES, K_ACCUMULATE, K_ZERO, K_ADAM_LIVE, K_COUNT
};

struct OdinProf {
  bool enabled = false;
  std::vector<cudaEvent_t> events;  // start/stop pairs, reused between collections
  std::vector<int> ids;             // kernel id of pair i
  size_t used = 0;                  // pairs recorded since the last collection
  uint64_t launches[K_COUNT] = {};
};

struct odin_ctx {
  int device;
  int sm_count;
  odin_config cfg;
  int* d_status;  // first deferred device-side error (0 = none)
  int* h_status;  // pinned mirror read by odin_poll
  int spin_limit; // polls after which a device-side wait gives up (odin_set_wait_limit)
  int chain;      // odin_chain_begin: 0 = off, 1 = on and the next operation is the first (or follows a copy / memset),
                  // 2 = on and the last operation enqueued was a kernel of this library
  OdinProf prof;
};

// Brackets one kernel launch: counts it and, when profiling is on, records a CUDA event on the launch stream before
// and after it.
struct OdinKernelScope {
  odin_ctx* ctx;
  cudaStream_t st;
  bool rec = false;
  size_t slot = 0;
  OdinKernelScope(odin_ctx* c, int id, cudaStream_t s) : ctx(c), st(s) {
    OdinProf& p = c->prof;
    ++p.launches[id];
    if (!p.enabled || p.used >= (1u << 16)) return;
    slot = p.used++;
    if (p.events.size() < 2 * (slot + 1)) {
      cudaEvent_t a = nullptr, b = nullptr;
      if (cudaEventCreate(&a) != cudaSuccess || cudaEventCreate(&b) != cudaSuccess) { --p.used; return; }
      p.events.push_back(a); p.events.push_back(b); p.ids.push_back(id);
    } else {
      p.ids[slot] = id;
    }
    rec = true;
    cudaEventRecord(p.events[2 * slot], st);
  }
  ~OdinKernelScope() {
    if (rec) cudaEventRecord(ctx->prof.events[2 * slot + 1], st);
  }
};

// Programmatic dependent launch.  A kernel that calls odin_after_predecessor() as its first statement may be launched
// with odin_launch(dependent = true, ...) right behind another kernel of the same call on the same stream: its blocks
// are then scheduled while the kernel in front drains (once every block of that kernel has started) and wait here
// until it has completed and its writes are visible, so the ~3.5 us between two dependent launches are not spent idle.
// Nothing is read or written before the wait, so ordering is exactly that of a plain launch; without a programmatic
// predecessor both instructions do nothing.  `dependent` must be false unless the operation in front on the stream is
// a kernel launched by the same call (inside a chain, odin_chain_begin, the library keeps track across calls); it is
// also dropped while per-kernel events are recorded.  EVERY kernel launched through odin_launch calls
// odin_after_predecessor() first.
__device__ __forceinline__ void odin_after_predecessor() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
template <typename... KArgs, typename... Args>
static inline cudaError_t odin_launch(odin_ctx* ctx, bool dependent, void (*kernel)(KArgs...), dim3 grid, dim3 block,
                                      size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t lc = {};
  lc.gridDim = grid; lc.blockDim = block; lc.dynamicSmemBytes = smem; lc.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = at;
  // inside a chain (odin_chain_begin) the kernel in front may belong to the call before this one
  lc.numAttrs = ((dependent || ctx->chain == 2) && !ctx->prof.enabled) ? 1 : 0;
  if (ctx->chain) ctx->chain = 2;
  return cudaLaunchKernelEx(&lc, kernel, std::forward<Args>(args)...);
}

// Zeroing of scratch words at the start of a call.  Outside a chain a memset; inside a chain a small kernel, so that
// the kernels on both sides of it stay programmatic dependents (a memset between two kernels costs ~2.7 us by itself
// and the two launch seams around it).  bytes must be a multiple of 4, p 4-byte aligned.
static __global__ void odin_zero_words_kernel(uint32_t* __restrict__ p, size_t words) {
  odin_after_predecessor();
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < words; i += (size_t)gridDim.x * blockDim.x) p[i] = 0u;
}
static inline cudaError_t odin_zero(odin_ctx* ctx, void* p, size_t bytes, cudaStream_t st) {
  if (bytes == 0) return cudaSuccess;
  if (!ctx->chain || ctx->prof.enabled || (bytes & 3) || (reinterpret_cast<uintptr_t>(p) & 3)) {
    if (ctx->chain) ctx->chain = 1;
    return cudaMemsetAsync(p, 0, bytes, st);
  }
  OdinKernelScope ks(ctx, K_ZERO, st);
  const size_t words = bytes / 4;
  size_t blocks = (words + 1023) / 1024;
  if (blocks > 1184) blocks = 1184;
  return odin_launch(ctx, false, odin_zero_words_kernel, dim3((unsigned)blocks), dim3(256), 0, st,
                     reinterpret_cast<uint32_t*>(p), words);
}
// a copy or memset enqueued by a call inside a chain: the next kernel must not be a dependent of the kernel before it
static inline void odin_chain_break(odin_ctx* ctx) { if (ctx && ctx->chain) ctx->chain = 1; }

#define ODIN_CUDA(call)                          \
  do {                                           \
    cudaError_t e__ = (call);                    \
    if (e__ != cudaSuccess) return ODIN_ERR_CUDA; \
  } while (0)

static inline bool odin_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
static inline size_t odin_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int odin_launch_status() { return cudaGetLastError() == cudaSuccess ? ODIN_OK : ODIN_ERR_CUDA; }

__device__ __forceinline__ void odin_set_error(int* status, int code) { atomicCAS(status, 0, code); }

// ---------------------------------------------------------------------------------------------------------------
// Decoupled look-back for single-pass prefix sums.  A tile publishes first its own aggregate, then its inclusive
// prefix; a later tile walks backwards over its predecessors, adding aggregates until it meets an inclusive prefix.
// Tiles take their index from an atomic ticket, so every predecessor of a running tile has already started.
// Every wait is bounded: after `spin_limit` unsuccessful polls (a kernel argument; ODIN_DEFAULT_SPIN_LIMIT unless the
// context was told otherwise) the walker records ODIN_ERR_TIMEOUT and carries on with what it has (callers clamp every
// address they derive from the result).
constexpr int ODIN_DEFAULT_SPIN_LIMIT = 1 << 22;

constexpr uint64_t LB64_FLAG_SHIFT = 62;
constexpr uint64_t LB64_AGG = 1ull << LB64_FLAG_SHIFT;
constexpr uint64_t LB64_INC = 2ull << LB64_FLAG_SHIFT;
constexpr uint64_t LB64_VALUE = (1ull << LB64_FLAG_SHIFT) - 1;

__device__ __forceinline__ uint64_t ld_volatile_u64(const uint64_t* p) {
  uint64_t v;
  asm volatile("ld.volatile.global.u64 %0, [%1];" : "=l"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld_volatile_u32(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.volatile.global.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ void st_volatile_u64(uint64_t* p, uint64_t v) {
  asm volatile("st.volatile.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ void st_volatile_u32(uint32_t* p, uint32_t v) {
  asm volatile("st.volatile.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Called by ONE warp of the tile (all 32 lanes).  state[] has one 64-bit word per tile, zero before the launch.
// Returns the exclusive prefix (sum of the aggregates of tiles 0..tile-1) in every lane and publishes this tile's
// inclusive prefix.  `aggregate` must fit 62 bits; two packed counters are fine as long as neither overflows its field.
__device__ __forceinline__ uint64_t odin_lookback_u64(uint64_t* state, uint32_t tile, uint64_t aggregate, int* status,
                                                      int spin_limit) {
  const unsigned lane = threadIdx.x & 31;
  if (tile == 0) {
    if (lane == 0) st_volatile_u64(&state[0], LB64_INC | aggregate);
    return 0;
  }
  if (lane == 0) st_volatile_u64(&state[tile], LB64_AGG | aggregate);
  uint64_t exclusive = 0;
  int64_t look = (int64_t)tile - 1;  // lane l inspects tile look - l
  int spins = 0;
  while (true) {
    const int64_t t = look - lane;
    uint64_t s = (t >= 0) ? ld_volatile_u64(&state[t]) : LB64_INC;  // before tile 0: an inclusive prefix of 0
    const unsigned invalid = __ballot_sync(0xffffffffu, (s >> LB64_FLAG_SHIFT) == 0);
    const unsigned inc = __ballot_sync(0xffffffffu, (s >> LB64_FLAG_SHIFT) == 2);
    // usable lanes: those before the first invalid one; stop at the first inclusive prefix among them
    const unsigned first_invalid = invalid ? (__ffs(invalid) - 1) : 32;
    const unsigned first_inc = inc ? (__ffs(inc) - 1) : 32;
    if (first_inc < first_invalid) {
      uint64_t v = (lane <= first_inc) ? (s & LB64_VALUE) : 0;
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      exclusive += v;
      break;
    }
    if (first_invalid > 0) {  // consume the valid aggregates in front of the gap, then retry from the gap
      uint64_t v = (lane < first_invalid) ? (s & LB64_VALUE) : 0;
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      exclusive += v;
      look -= first_invalid;
    } else {
      __nanosleep(64);
      if (++spins > spin_limit) {
        if (lane == 0) odin_set_error(status, ODIN_ERR_TIMEOUT);
        break;
      }
    }
  }
  if (lane == 0) st_volatile_u64(&state[tile], LB64_INC | ((exclusive + aggregate) & LB64_VALUE));
  return exclusive;
}

// Block-wide exclusive sum of one uint32 per thread for blocks of up to 1024 threads.  `warp_sums` is shared memory
// for 33 uint32.  Returns the exclusive prefix; *total receives the block sum in every thread.
__device__ __forceinline__ uint32_t odin_block_exclusive_sum(uint32_t v, uint32_t* warp_sums, uint32_t* total) {
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    uint32_t y = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= (unsigned)o) inc += y;
  }
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = (lane < nwarps) ? warp_sums[lane] : 0;
    uint32_t winc = w;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      uint32_t y = __shfl_up_sync(0xffffffffu, winc, o);
      if (lane >= (unsigned)o) winc += y;
    }
    if (lane < nwarps) warp_sums[lane] = winc - w;
    if (lane == 31) warp_sums[32] = winc;
  }
  __syncthreads();
  *total = warp_sums[32];
  const uint32_t r = warp_sums[warp] + inc - v;
  __syncthreads();
  return r;
}

// Camera as kernel parameter (plain floats; derived quantities precomputed on the host).
struct CamParams {
  int W, H, TX, TY;
  float fx, fy, cx, cy, znear, zfar;
  float R[9], t[3], bg[3], pos[3];
  float limx, limy;
};

static inline CamParams odin_cam_params(const odin_camera* c, const odin_config& cfg) {
  CamParams k;
  k.W = c->width; k.H = c->height;
  k.TX = (c->width + 15) / 16; k.TY = (c->height + 15) / 16;
  k.fx = c->fx; k.fy = c->fy; k.cx = c->cx; k.cy = c->cy; k.znear = c->znear; k.zfar = c->zfar;
  for (int i = 0; i < 3; ++i) {
    for (int j = 0; j < 3; ++j) k.R[3 * i + j] = c->w2c[4 * i + j];
    k.t[i] = c->w2c[4 * i + 3];
    k.bg[i] = c->bg[i];
  }
  for (int j = 0; j < 3; ++j) k.pos[j] = -(k.R[j] * k.t[0] + k.R[3 + j] * k.t[1] + k.R[6 + j] * k.t[2]);
  k.limx = cfg.jac_clamp * (float)c->width / (2.0f * c->fx);
  k.limy = cfg.jac_clamp * (float)c->height / (2.0f * c->fy);
  return k;
}

static inline int odin_check_camera(const odin_camera* c) {
  if (!c) return ODIN_ERR_NULL;
  if (c->width <= 0 || c->height <= 0 || c->width > 16384 || c->height > 16384) return ODIN_ERR_INVALID_ARG;
  if (!(c->fx > 0) || !(c->fy > 0) || !(c->znear > 0) || !(c->zfar > c->znear)) return ODIN_ERR_INVALID_ARG;
  return ODIN_OK;
}

static inline int odin_check_scene(const odin_scene* s) {
  if (!s) return ODIN_ERR_NULL;
  if (s->sh_degree < 0 || s->sh_degree > 3) return ODIN_ERR_INVALID_ARG;
  if (s->n >= (1u << 28)) return ODIN_ERR_INVALID_ARG;
  if (s->n == 0) return ODIN_OK;
  if (!s->means || !s->log_scales || !s->quats || !s->opacity_logit || !s->sh) return ODIN_ERR_NULL;
  if (!odin_aligned(s->means, 16) || !odin_aligned(s->log_scales, 16) || !odin_aligned(s->quats, 16) ||
      !odin_aligned(s->opacity_logit, 16) || !odin_aligned(s->sh, 16))
    return ODIN_ERR_INVALID_ARG;
  return ODIN_OK;
}
