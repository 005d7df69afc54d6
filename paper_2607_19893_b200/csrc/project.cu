// Preprocessing phase: cull, EWA projection, tile rectangle, SH colour; compaction of the visible rows and the
// exclusive scan of their tile counts in the same pass (decoupled look-back over 256-primitive tiles).
#include "geom.cuh"
#include "layout.cuh"

namespace {

// packed look-back value: rows in the upper 28 bits, tile instances in the lower 34 bits
constexpr int PACK_SHIFT = 34;
constexpr uint64_t PACK_LOW = (1ull << PACK_SHIFT) - 1;

template <int DEG>
__global__ void __launch_bounds__(PROJECT_TILE)
project_kernel(const float* __restrict__ means, const float* __restrict__ log_scales, const float4* __restrict__ quats,
               const float* __restrict__ opacity_logit, const float* __restrict__ sh, uint32_t n, CamParams cam,
               float dilation, float radius_sigmas, odin_projected out, uint32_t* ticket, uint64_t* state, int* status) {
  constexpr int K = (DEG + 1) * (DEG + 1);
  __shared__ uint32_t s_tile;
  __shared__ uint32_t s_warp[33];
  __shared__ uint32_t s_warp2[33];
  __shared__ uint64_t s_base;
  if (threadIdx.x == 0) s_tile = atomicAdd(ticket, 1u);
  __syncthreads();
  const uint32_t tile = s_tile;
  const uint32_t p = tile * PROJECT_TILE + threadIdx.x;

  uint32_t tiles = 0;
  float u = 0.f, v = 0.f, depth = 0.f, cA = 0.f, cB = 0.f, cC = 0.f;
  int rad = 0;
  int x0 = 0, y0 = 0, x1 = 0, y1 = 0;
  float mx = 0.f, my = 0.f, mz = 0.f;
  if (p < n) {
    mx = means[3 * (size_t)p]; my = means[3 * (size_t)p + 1]; mz = means[3 * (size_t)p + 2];
    SplatGeom g;
    odin_camera_space(cam, mx, my, mz, g.t);
    if (g.t[2] > cam.znear && g.t[2] < cam.zfar) {
      const float ls[3] = {log_scales[3 * (size_t)p], log_scales[3 * (size_t)p + 1], log_scales[3 * (size_t)p + 2]};
      odin_splat_geometry(cam, dilation, ls, quats[p], g);
      if (g.det > 0.f) {
        cA = g.c / g.det; cB = -g.b / g.det; cC = g.a / g.det;
        const float mid = (g.a + g.c) / 2.f;
        const float lam = mid + sqrtf(fmaxf(0.1f, mid * mid - g.det));
        const float radf = ceilf(radius_sigmas * sqrtf(lam));
        u = cam.fx * g.t[0] / g.t[2] + cam.cx;
        v = cam.fy * g.t[1] / g.t[2] + cam.cy;
        depth = g.t[2];
        const float ftx = (float)cam.TX, fty = (float)cam.TY;
        x0 = (int)fminf(ftx, fmaxf(0.f, floorf((u - radf) / 16.f)));
        x1 = (int)fminf(ftx, fmaxf(0.f, ceilf((u + radf) / 16.f)));
        y0 = (int)fminf(fty, fmaxf(0.f, floorf((v - radf) / 16.f)));
        y1 = (int)fminf(fty, fmaxf(0.f, ceilf((v + radf) / 16.f)));
        tiles = (uint32_t)(x1 - x0) * (uint32_t)(y1 - y0);
        rad = (int)fminf(radf, 2.0e9f);
      }
    }
    out.tiles_touched[p] = tiles;
  }

  // block scan of (visible, tiles) and look-back for the global row / instance offsets
  uint32_t total_rows, total_tiles;
  const uint32_t vis = tiles > 0 ? 1u : 0u;
  const uint32_t row_local = odin_block_exclusive_sum(vis, s_warp, &total_rows);
  // images are limited to 16384^2 pixels = 2^20 tiles, so 256 rectangles sum to < 2^32
  const uint32_t off_local = odin_block_exclusive_sum(tiles, s_warp2, &total_tiles);
  if (threadIdx.x < 32) {
    const uint64_t agg = ((uint64_t)total_rows << PACK_SHIFT) | (uint64_t)total_tiles;
    const uint64_t ex = odin_lookback_u64(state, tile, agg, status);
    if (threadIdx.x == 0) s_base = ex;
  }
  __syncthreads();
  const uint64_t base = s_base;
  const uint64_t row_base = base >> PACK_SHIFT, inst_base = base & PACK_LOW;

  if (tile == (n + PROJECT_TILE - 1) / PROJECT_TILE - 1 && threadIdx.x == 0) {  // last tile: totals
    const uint64_t rows = row_base + total_rows, inst = inst_base + total_tiles;
    *out.num_rows = (uint32_t)(rows < out.capacity ? rows : out.capacity);
    *out.num_instances = inst;
    if (rows > out.capacity || inst >= (1ull << 32)) odin_set_error(status, ODIN_ERR_CAPACITY);
  }
  if (!vis) return;
  const uint64_t r64 = row_base + row_local;
  if (r64 >= out.capacity) return;
  const size_t r = (size_t)r64;
  out.prim_id[r] = p;
  reinterpret_cast<float2*>(out.xy)[r] = make_float2(u, v);
  out.depth[r] = depth;
  const float o = 1.f / (1.f + expf(-opacity_logit[p]));
  reinterpret_cast<float4*>(out.conic_opacity)[r] = make_float4(cA, cB, cC, o);
  out.radius[r] = rad;
  reinterpret_cast<ushort4*>(out.rect)[r] = make_ushort4((unsigned short)x0, (unsigned short)y0, (unsigned short)x1,
                                                         (unsigned short)y1);
  out.tile_offset[r] = (uint32_t)(inst_base + off_local);

  // colour
  float dx = mx - cam.pos[0], dy = my - cam.pos[1], dz = mz - cam.pos[2];
  const float len = sqrtf(dx * dx + dy * dy + dz * dz);
  dx /= len; dy /= len; dz /= len;
  float Y[16];
  odin_sh_basis<DEG>(dx, dy, dz, Y);
  float acc[3] = {0.f, 0.f, 0.f};
  const float* row = sh + (size_t)p * (3 * K);
  if (K == 1) {
    acc[0] = Y[0] * row[0]; acc[1] = Y[0] * row[1]; acc[2] = Y[0] * row[2];
  } else {
    // 3K floats are a multiple of 4 for K = 4, 16 (and 27 = 3*9 for K = 9 is not): use scalar loads there
    if ((3 * K) % 4 == 0) {
      const float4* row4 = reinterpret_cast<const float4*>(row);
#pragma unroll
      for (int i = 0; i < 3 * K / 4; ++i) {
        const float4 c = row4[i];
        const float e[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int f = 4 * i + j;
          acc[f % 3] += Y[f / 3] * e[j];
        }
      }
    } else {
#pragma unroll
      for (int f = 0; f < 3 * K; ++f) acc[f % 3] += Y[f / 3] * row[f];
    }
  }
  uint8_t flags = 0;
#pragma unroll
  for (int ch = 0; ch < 3; ++ch) {
    acc[ch] += 0.5f;
    if (acc[ch] < 0.f) { acc[ch] = 0.f; flags |= (uint8_t)(1u << ch); }
  }
  out.rgb[3 * r] = acc[0]; out.rgb[3 * r + 1] = acc[1]; out.rgb[3 * r + 2] = acc[2];
  out.clamp_flags[r] = flags;
}

}  // namespace

extern "C" int odin_project(odin_ctx* ctx, const odin_scene* scene, const odin_camera* cam, odin_projected* out, void* ws,
                            size_t ws_bytes, void* stream) {
  if (!ctx || !out) return ODIN_ERR_NULL;
  int rc = odin_check_scene(scene);
  if (rc != ODIN_OK) return rc;
  rc = odin_check_camera(cam);
  if (rc != ODIN_OK) return rc;
  if (!out->num_rows || !out->num_instances) return ODIN_ERR_NULL;
  if (out->capacity > 0 && (!out->prim_id || !out->xy || !out->depth || !out->conic_opacity || !out->rgb || !out->radius ||
                            !out->rect || !out->tile_offset || !out->clamp_flags))
    return ODIN_ERR_NULL;
  if (!odin_aligned(out->xy, 8) || !odin_aligned(out->conic_opacity, 16) || !odin_aligned(out->rect, 8) ||
      !odin_aligned(out->num_instances, 8))
    return ODIN_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  const uint32_t n = scene->n;
  if (n == 0) {
    ODIN_CUDA(cudaMemsetAsync(out->num_rows, 0, 4, st));
    ODIN_CUDA(cudaMemsetAsync(out->num_instances, 0, 8, st));
    return ODIN_OK;
  }
  if (!out->tiles_touched) return ODIN_ERR_NULL;
  const size_t need = project_ws_bytes(n);
  if (!ws || !odin_aligned(ws, 256) || ws_bytes < need) return ODIN_ERR_WORKSPACE;
  ODIN_CUDA(cudaMemsetAsync(ws, 0, need, st));
  uint32_t* ticket = reinterpret_cast<uint32_t*>(ws);
  uint64_t* state = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(ws) + 256);
  const CamParams cp = odin_cam_params(cam, ctx->cfg);
  const uint32_t grid = (n + PROJECT_TILE - 1) / PROJECT_TILE;
  const float4* q4 = reinterpret_cast<const float4*>(scene->quats);
#define LAUNCH(D)                                                                                                    \
  project_kernel<D><<<grid, PROJECT_TILE, 0, st>>>(scene->means, scene->log_scales, q4, scene->opacity_logit, scene->sh, \
                                                   n, cp, ctx->cfg.dilation, ctx->cfg.radius_sigmas, *out, ticket, state, \
                                                   ctx->d_status)
  OdinKernelScope ks(ctx, K_PROJECT, st);
  switch (scene->sh_degree) {
    case 0: LAUNCH(0); break;
    case 1: LAUNCH(1); break;
    case 2: LAUNCH(2); break;
    default: LAUNCH(3); break;
  }
#undef LAUNCH
  return odin_launch_status();
}
