// Rendering phase: front-to-back alpha compositing, one 16x16 block per tile, the tile's sorted rows staged through
// shared memory in batches of 256, early exit once every pixel of the tile has terminated.  Also the L1 image loss.
#include "common.cuh"

namespace {

constexpr int FB = 256;  // threads per block = pixels per tile = rows per batch

__global__ void __launch_bounds__(FB)
render_fwd_kernel(const float2* __restrict__ xy, const float4* __restrict__ conic_o, const float* __restrict__ rgb,
                  const uint32_t* __restrict__ vals, const uint2* __restrict__ ranges, int W, int H, int TX, float bg0,
                  float bg1, float bg2, float alpha_min, float alpha_max, float t_min, float* __restrict__ out,
                  float* __restrict__ final_T, uint32_t* __restrict__ n_contrib) {
  __shared__ float2 s_xy[FB];
  __shared__ float4 s_co[FB];
  __shared__ float s_rgb[FB][3];
  const int tile = blockIdx.x;
  const int tx = tile % TX, ty = tile / TX;
  const int lx = threadIdx.x & 15, ly = threadIdx.x >> 4;
  const int px = tx * 16 + lx, py = ty * 16 + ly;
  const bool inside = px < W && py < H;
  const float fx = (float)px + 0.5f, fy = (float)py + 0.5f;
  const uint2 rg = ranges[tile];
  const uint32_t start = rg.x, end = rg.y;
  float T = 1.f, C0 = 0.f, C1 = 0.f, C2 = 0.f;
  uint32_t last = 0;
  bool done = !inside;
  for (uint32_t b = start; b < end; b += FB) {
    if (__syncthreads_count(done) == FB) break;
    const uint32_t i = b + threadIdx.x;
    if (i < end) {
      const uint32_t r = vals[i];
      s_xy[threadIdx.x] = xy[r];
      s_co[threadIdx.x] = conic_o[r];
      s_rgb[threadIdx.x][0] = rgb[3 * (size_t)r];
      s_rgb[threadIdx.x][1] = rgb[3 * (size_t)r + 1];
      s_rgb[threadIdx.x][2] = rgb[3 * (size_t)r + 2];
    }
    __syncthreads();
    const int cnt = (int)min((uint32_t)FB, end - b);
    if (!done) {
      for (int j = 0; j < cnt; ++j) {
        const float2 c = s_xy[j];
        const float4 co = s_co[j];
        const float dx = c.x - fx, dy = c.y - fy;
        const float power = -0.5f * (co.x * dx * dx + co.z * dy * dy) - co.y * dx * dy;
        if (power > 0.f) continue;
        const float alpha = fminf(alpha_max, co.w * __expf(power));
        if (alpha < alpha_min) continue;
        const float Tn = T * (1.f - alpha);
        if (Tn < t_min) { done = true; break; }
        const float w = alpha * T;
        C0 += s_rgb[j][0] * w; C1 += s_rgb[j][1] * w; C2 += s_rgb[j][2] * w;
        T = Tn;
        last = (b - start) + j + 1;
      }
    }
  }
  if (inside) {
    const size_t pix = (size_t)py * W + px, plane = (size_t)W * H;
    out[pix] = C0 + T * bg0;
    out[plane + pix] = C1 + T * bg1;
    out[2 * plane + pix] = C2 + T * bg2;
    final_T[pix] = T;
    n_contrib[pix] = last;
  }
}

constexpr int LB = 256;

__global__ void __launch_bounds__(LB)
l1_loss_kernel(const float* __restrict__ out, const float* __restrict__ target, size_t count, float inv, double* loss_acc,
               float* __restrict__ dL) {
  float acc = 0.f;
  for (size_t i = (size_t)blockIdx.x * LB + threadIdx.x; i < count; i += (size_t)gridDim.x * LB) {
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
  }
}

__global__ void l1_finish_kernel(const double* acc, double inv, float* loss) { *loss = (float)(*acc * inv); }

}  // namespace

extern "C" int odin_render_fwd(odin_ctx* ctx, const odin_projected* proj, const uint32_t* d_vals,
                               const uint32_t* d_tile_ranges, const odin_camera* cam, float* d_rgb, float* d_final_T,
                               uint32_t* d_n_contrib, void* stream) {
  if (!ctx || !proj || !d_tile_ranges || !d_rgb || !d_final_T || !d_n_contrib) return ODIN_ERR_NULL;
  const int rc = odin_check_camera(cam);
  if (rc != ODIN_OK) return rc;
  if (proj->capacity > 0 && (!proj->xy || !proj->conic_opacity || !proj->rgb || !d_vals)) return ODIN_ERR_NULL;
  if (!odin_aligned(proj->xy, 8) || !odin_aligned(proj->conic_opacity, 16) || !odin_aligned(d_tile_ranges, 8))
    return ODIN_ERR_INVALID_ARG;
  const int TX = (cam->width + 15) / 16, TY = (cam->height + 15) / 16;
  OdinKernelScope ks(ctx, K_FWD, (cudaStream_t)stream);
  render_fwd_kernel<<<TX * TY, FB, 0, (cudaStream_t)stream>>>(
      reinterpret_cast<const float2*>(proj->xy), reinterpret_cast<const float4*>(proj->conic_opacity), proj->rgb, d_vals,
      reinterpret_cast<const uint2*>(d_tile_ranges), cam->width, cam->height, TX, cam->bg[0], cam->bg[1], cam->bg[2],
      ctx->cfg.alpha_min, ctx->cfg.alpha_max, ctx->cfg.t_min, d_rgb, d_final_T, d_n_contrib);
  return odin_launch_status();
}

extern "C" int odin_l1_loss(odin_ctx* ctx, const float* d_rgb, const float* d_target, int width, int height,
                            float* d_loss, float* d_dL_drgb, void* stream) {
  if (!ctx || !d_rgb || !d_target || !d_loss || !d_dL_drgb) return ODIN_ERR_NULL;
  if (width <= 0 || height <= 0) return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const size_t count = (size_t)3 * width * height;
  // the accumulator lives behind the status word in the context's device block
  double* acc = reinterpret_cast<double*>(reinterpret_cast<char*>(ctx->d_status) + 64);
  ODIN_CUDA(cudaMemsetAsync(acc, 0, 8, st));
  size_t blocks = (count + LB - 1) / LB;
  if (blocks > (size_t)ctx->sm_count * 8) blocks = (size_t)ctx->sm_count * 8;
  {
    OdinKernelScope ks(ctx, K_L1, st);
    l1_loss_kernel<<<(unsigned)blocks, LB, 0, st>>>(d_rgb, d_target, count, (float)(1.0 / (double)count), acc, d_dL_drgb);
  }
  OdinKernelScope ks(ctx, K_L1_FINISH, st);
  l1_finish_kernel<<<1, 1, 0, st>>>(acc, 1.0 / (double)count, d_loss);
  return odin_launch_status();
}
