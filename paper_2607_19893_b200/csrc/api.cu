// Context management, deferred status and workspace sizing of the C ABI.
#include <new>

#include "common.cuh"
#include "layout.cuh"

extern "C" int odin_create(odin_ctx** out, int device, const odin_config* cfg) {
  if (!out) return ODIN_ERR_NULL;
  *out = nullptr;
  odin_config c = {1.0f / 255.0f, 0.99f, 1e-4f, 0.3f, 3.0f, 1.3f, 16, 0, 0};
  if (cfg) c = *cfg;
  if (c.tile != 16) return ODIN_ERR_UNSUPPORTED;
  if (c.binning < 0 || c.binning > 2) return ODIN_ERR_INVALID_ARG;
  if (c.instance_sort != 0 && c.instance_sort != 1) return ODIN_ERR_INVALID_ARG;
  if (!(c.alpha_min > 0) || !(c.alpha_max < 1) || !(c.alpha_max > c.alpha_min) || !(c.t_min > 0) || !(c.dilation >= 0) ||
      !(c.radius_sigmas > 0) || !(c.jac_clamp > 0))
    return ODIN_ERR_INVALID_ARG;
  ODIN_CUDA(cudaSetDevice(device));
  odin_ctx* ctx = new (std::nothrow) odin_ctx();
  if (!ctx) return ODIN_ERR_CUDA;
  ctx->device = device;
  ctx->cfg = c;
  ctx->d_status = nullptr;
  ctx->h_status = nullptr;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess || cudaMalloc(&ctx->d_status, 256) != cudaSuccess ||
      cudaMallocHost(&ctx->h_status, sizeof(int)) != cudaSuccess || cudaMemset(ctx->d_status, 0, 256) != cudaSuccess) {
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->h_status) cudaFreeHost(ctx->h_status);
    delete ctx;
    return ODIN_ERR_CUDA;
  }
  ctx->sm_count = prop.multiProcessorCount;
  ctx->spin_limit = ODIN_DEFAULT_SPIN_LIMIT;
  ctx->chain = 0;
  *ctx->h_status = 0;
  *out = ctx;
  return ODIN_OK;
}

extern "C" int odin_destroy(odin_ctx* ctx) {
  if (!ctx) return ODIN_ERR_NULL;
  cudaFree(ctx->d_status);
  cudaFreeHost(ctx->h_status);
  for (cudaEvent_t e : ctx->prof.events) cudaEventDestroy(e);
  delete ctx;
  return ODIN_OK;
}

extern "C" int odin_set_wait_limit(odin_ctx* ctx, int polls) {
  if (!ctx) return ODIN_ERR_NULL;
  if (polls < 0 || polls > (1 << 30)) return ODIN_ERR_INVALID_ARG;
  ctx->spin_limit = polls;
  return ODIN_OK;
}

extern "C" int odin_set_instance_sort(odin_ctx* ctx, int mode) {
  if (!ctx) return ODIN_ERR_NULL;
  if (mode != 0 && mode != 1) return ODIN_ERR_INVALID_ARG;
  ctx->cfg.instance_sort = mode;
  return ODIN_OK;
}

extern "C" const char* odin_status_string(int s) {
  switch (s) {
    case ODIN_OK: return "ok";
    case ODIN_ERR_NULL: return "null pointer";
    case ODIN_ERR_INVALID_ARG: return "invalid argument";
    case ODIN_ERR_CAPACITY: return "capacity exceeded (outputs truncated)";
    case ODIN_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case ODIN_ERR_CUDA: return "CUDA runtime error";
    case ODIN_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case ODIN_ERR_UNSUPPORTED: return "unsupported";
    default: return "unknown status";
  }
}

extern "C" int odin_poll(odin_ctx* ctx, void* stream) {
  if (!ctx) return ODIN_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  odin_chain_break(ctx);
  ODIN_CUDA(cudaMemcpyAsync(ctx->h_status, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  ODIN_CUDA(cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st));
  ODIN_CUDA(cudaStreamSynchronize(st));
  const int s = *ctx->h_status;
  *ctx->h_status = 0;
  return s;
}

static const char* const kKernelNames[K_COUNT] = {
    "project_cull", "touched_set", "emit_instances", "onesweep_pass", "render_fwd", "l1_loss",
    "zero_rows", "render_bwd_blend", "render_bwd_project", "adam_sh", "adam_geom", "conflict_count",
    "render_fwd_tail", "project_scan", "project_rows", "row_hist",
    "row_sort_pass", "row_offsets", "active_set", "mask_union", "hazard_count", "delayed_read_gate",
    "locality_graph", "tile_bases", "accumulate_rows", "zero_words", "adam_live_refresh"};

extern "C" int odin_chain_begin(odin_ctx* ctx) {
  if (!ctx) return ODIN_ERR_NULL;
  ctx->chain = 1;
  return ODIN_OK;
}

extern "C" int odin_chain_end(odin_ctx* ctx) {
  if (!ctx) return ODIN_ERR_NULL;
  ctx->chain = 0;
  return ODIN_OK;
}

extern "C" int odin_kernel_count(void) { return K_COUNT; }

extern "C" const char* odin_kernel_name(int id) { return (id >= 0 && id < K_COUNT) ? kKernelNames[id] : "unknown"; }

extern "C" int odin_profile_enable(odin_ctx* ctx, int on) {
  if (!ctx) return ODIN_ERR_NULL;
  ctx->prof.enabled = on != 0;
  return ODIN_OK;
}

extern "C" int odin_profile_collect(odin_ctx* ctx, void* stream, float* h_ms, uint64_t* h_launches) {
  if (!ctx) return ODIN_ERR_NULL;
  ODIN_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
  OdinProf& p = ctx->prof;
  for (int k = 0; k < K_COUNT; ++k) {
    if (h_ms) h_ms[k] = 0.f;
    if (h_launches) h_launches[k] = p.launches[k];
    p.launches[k] = 0;
  }
  for (size_t i = 0; i < p.used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, p.events[2 * i], p.events[2 * i + 1]) == cudaSuccess && h_ms) h_ms[p.ids[i]] += ms;
  }
  p.used = 0;
  return ODIN_OK;
}

// ---------------------------------------------------------------------------------------------------------------
// Measurement aid: the fp32 multiply-add rate this GPU sustains, the denominator for the kernels that are bound by
// plain ALU work (the two compositing kernels).  Every thread runs eight independent chains of fused multiply-adds.
namespace {
constexpr int FMA_CHAINS = 8;
__global__ void __launch_bounds__(256) fp32_peak_kernel(float* sink, int iters, float a, float b) {
  float x[FMA_CHAINS];
#pragma unroll
  for (int k = 0; k < FMA_CHAINS; ++k) x[k] = (float)(threadIdx.x + k) * 1e-3f;
  for (int i = 0; i < iters; ++i) {
#pragma unroll
    for (int k = 0; k < FMA_CHAINS; ++k) x[k] = fmaf(x[k], a, b);
  }
  float s = 0.f;
#pragma unroll
  for (int k = 0; k < FMA_CHAINS; ++k) s += x[k];
  if (s == 123.456f) sink[0] = s;  // keeps the chains alive; practically never true
}
}  // namespace

extern "C" int odin_measure_fp32_peak(odin_ctx* ctx, void* stream, float* h_tflops) {
  if (!ctx || !h_tflops) return ODIN_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  float* sink = reinterpret_cast<float*>(reinterpret_cast<char*>(ctx->d_status) + 128);
  const int iters = 1 << 14, blocks = ctx->sm_count * 8;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  ODIN_CUDA(cudaEventCreate(&e0));
  if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return ODIN_ERR_CUDA; }
  float best_ms = 0.f;
  for (int rep = 0; rep < 4; ++rep) {  // the first repetition warms up
    cudaEventRecord(e0, st);
    fp32_peak_kernel<<<blocks, 256, 0, st>>>(sink, iters, 0.999f, 1e-3f);
    cudaEventRecord(e1, st);
    if (cudaEventSynchronize(e1) != cudaSuccess) { cudaEventDestroy(e0); cudaEventDestroy(e1); return ODIN_ERR_CUDA; }
    float ms = 0.f;
    cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && (best_ms == 0.f || ms < best_ms)) best_ms = ms;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  const double flops = 2.0 * FMA_CHAINS * (double)iters * 256.0 * (double)blocks;
  *h_tflops = best_ms > 0.f ? (float)(flops / (best_ms * 1e-3) / 1e12) : 0.f;
  return odin_launch_status();
}

extern "C" int odin_workspace_bytes(const odin_ctx* ctx, uint32_t n, uint64_t max_instances, size_t* bytes) {
  if (!ctx || !bytes) return ODIN_ERR_NULL;
  size_t b = project_ws_bytes(n);
  const size_t t = touched_ws_bytes(n);
  const size_t s = binsort_ws_bytes(max_instances, n);  // a view has at most n rows
  if (t > b) b = t;
  if (s > b) b = s;
  *bytes = b;
  return ODIN_OK;
}
