// Backward phase: (a) back-to-front replay of the compositing, one warp per segment of a tile's list, per-lane
// accumulation over eight pixels, one transposing warp reduction and one global atomic per (segment, row, word);
// (b) per-row chain rule through the projection into compact gradient rows.
#include "blend.cuh"
#include "geom.cuh"

namespace {

__global__ void zero_rows_kernel(float* __restrict__ g2d, uint8_t* __restrict__ row_active,
                                 const uint32_t* __restrict__ num_rows, uint32_t capacity) {
  odin_after_predecessor();
  const uint32_t V = min(*num_rows, capacity);
  const size_t count = (size_t)V * 9;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x) {
    g2d[i] = 0.f;
    if (row_active && i < V) row_active[i] = 0;
  }
}

// Sums eight values across the warp with 9 shuffles: at each of the first three steps a lane hands half of its
// values to its partner and keeps the other half, so after offsets 16, 8, 4 every lane holds one value summed over
// 8 lanes; offsets 2 and 1 finish it.  On return lane 4*v holds the warp total of value v.
__device__ __forceinline__ float warp_transpose_sum8(float a0, float a1, float a2, float a3, float a4, float a5, float a6,
                                                     float a7, unsigned lane) {
  const bool h16 = lane & 16, h8 = lane & 8, h4 = lane & 4;
  float b0 = (h16 ? a4 : a0) + __shfl_xor_sync(0xffffffffu, h16 ? a0 : a4, 16);
  float b1 = (h16 ? a5 : a1) + __shfl_xor_sync(0xffffffffu, h16 ? a1 : a5, 16);
  float b2 = (h16 ? a6 : a2) + __shfl_xor_sync(0xffffffffu, h16 ? a2 : a6, 16);
  float b3 = (h16 ? a7 : a3) + __shfl_xor_sync(0xffffffffu, h16 ? a3 : a7, 16);
  float c0 = (h8 ? b2 : b0) + __shfl_xor_sync(0xffffffffu, h8 ? b0 : b2, 8);
  float c1 = (h8 ? b3 : b1) + __shfl_xor_sync(0xffffffffu, h8 ? b1 : b3, 8);
  float d = (h4 ? c1 : c0) + __shfl_xor_sync(0xffffffffu, h4 ? c0 : c1, 4);
  d += __shfl_xor_sync(0xffffffffu, d, 2);
  d += __shfl_xor_sync(0xffffffffu, d, 1);
  return d;
}

// One warp per SEGMENT of a tile's list (BLEND_HEAD entries), eight pixels per lane (blend.cuh).  Segment 0 of every
// tile is a work item; the later segments are the ones the forward tail kernel recorded, together with the state of
// every pixel at the segment's start.  A segment is replayed back to front from the state at its END: that of the
// next segment's record, or the final state of the pixel when nothing behind the segment contributed.  For every row
// the lane accumulates, over its own pixels, the colour and opacity gradients and three moments of dL/dpower (sum,
// sum*dy, sum*dy^2); dx is constant per lane, so the conic / centre gradients follow from the moments with a handful
// of operations per row instead of per pixel.  One transposing warp reduction and nine global atomics per (segment,
// row) that contributed.
// TRACK: also flag the rows that contributed (realized active set).  A separate instantiation because this loop is
// sensitive to anything added to it: the flag store costs ~5 % of the kernel, and callers who do not ask for the flags
// do not pay for it.
template <bool TRACK>
__global__ void __launch_bounds__(BLEND_THREADS, 5)
render_bwd_blend_kernel(const float2* __restrict__ xy, const float4* __restrict__ conic_o, const float* __restrict__ rgb,
                        const uint32_t* __restrict__ vals, const uint2* __restrict__ ranges, int W, int H, int TX,
                        int n_tiles, float bg0, float bg1, float bg2, float alpha_min, float alpha_max,
                        const uint32_t* __restrict__ tile_first, const uint32_t* __restrict__ seg_count,
                        const uint2* __restrict__ seg_tile, const uint2* __restrict__ seg_link,
                        const BlendRecord* __restrict__ ckpt, uint32_t seg_cap,
                        const float* __restrict__ final_T, const uint32_t* __restrict__ n_contrib,
                        const float* __restrict__ dL, float* __restrict__ g2d, uint32_t* __restrict__ ticket,
                        uint8_t* __restrict__ row_active, uint32_t row_cap, const uint32_t* __restrict__ bwd_count,
                        const uint32_t* __restrict__ bwd_queue) {
  odin_after_predecessor();  // launched behind zero_rows_kernel
  __shared__ BlendRow s_rowdata[BLEND_WARPS][32];
  __shared__ float2 s_blue[BLEND_WARPS][32];  // blue, 1 / opacity
  __shared__ uint32_t s_rowid[BLEND_WARPS][32];
  const unsigned lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t n_seg = min(*seg_count, seg_cap);
  const float l2amin = log2f(alpha_min);
  // warps never synchronise with each other; each keeps taking work items from a ticket counter (see the forward
  // kernel).  The recorded segments come first: they are full-length, the segments 0 of most tiles are not.
  while (true) {
  uint32_t item = 0;
  if (lane == 0) item = atomicAdd(ticket, 1u);
  item = __shfl_sync(0xffffffffu, item, 0);
  int tile;
  uint32_t seg = 0, next;
  if (item < n_seg) {
    const uint2 st = seg_tile[item];
    tile = (int)st.x; seg = st.y; next = seg_link[item].x;
  } else {
    uint32_t pos = item - n_seg;
    if (pos >= (uint32_t)n_tiles) return;
    // the tiles in the order the forward pass filed them: classes of walked length, longest first (the class counts
    // add up to the number of tiles; whatever else the words hold, pos stays below it and the tile is clamped)
    uint32_t cls = 0;
    while (cls + 1 < (uint32_t)BLEND_BWD_CLASSES && pos >= bwd_count[cls]) { pos -= bwd_count[cls]; ++cls; }
    tile = (int)min(bwd_queue[cls * (uint32_t)n_tiles + min(pos, (uint32_t)n_tiles - 1)], (uint32_t)n_tiles - 1);
    next = tile_first[tile];
  }
  // a workspace that is not the forward call's own must not lead anywhere: records are checked before use
  if ((uint32_t)tile >= (uint32_t)n_tiles || seg >= (1u << 23)) continue;
  if (next > seg_cap) next = 0;
  const uint32_t seg_base = seg * BLEND_HEAD;
  const int tx = tile % TX, ty = tile / TX;
  const float tile_x0 = (float)(tx * 16), tile_y0 = (float)(ty * 16);
  const int px = tx * 16 + (int)(lane & 15);
  const int py0 = ty * 16 + (int)(lane >> 4);
  const float fx = (float)px + 0.5f, fy0 = (float)py0 + 0.5f;
  const uint32_t start = ranges[tile].x;
  const size_t plane = (size_t)W * H;

  float T[BLEND_SLOTS], SG[BLEND_SLOTS];  // SG: colour still to come times the pixel's incoming gradient
  float g0[BLEND_SLOTS], g1[BLEND_SLOTS], g2[BLEND_SLOTS];
  uint32_t last[BLEND_SLOTS];
  uint32_t total = 0;
#pragma unroll
  for (int s = 0; s < BLEND_SLOTS; ++s) {
    const int py = py0 + 2 * s;
    T[s] = 1.f; g0[s] = g1[s] = g2[s] = 0.f; last[s] = 0;
    if (px < W && py < H) {
      const size_t pix = (size_t)py * W + px;
      T[s] = final_T[pix];
      last[s] = n_contrib[pix];
      g0[s] = dL[pix]; g1[s] = dL[plane + pix]; g2[s] = dL[2 * plane + pix];
    }
    // Only the product of the colour to come with the pixel's incoming gradient is ever needed, so one scalar is
    // carried: SG = sum_ch S_ch g_ch with S = sum_{j>k} c_j alpha_j T_j + T_final bg.
    SG[s] = T[s] * (bg0 * g0[s] + bg1 * g1[s] + bg2 * g2[s]);
    total = max(total, last[s]);
  }
  for (int o = 16; o > 0; o >>= 1) total = max(total, __shfl_xor_sync(0xffffffffu, total, o));
  // `total` = list entries any pixel of the tile used
  if (total <= seg_base) continue;  // nothing in this segment contributed
  if (total > seg_base + BLEND_HEAD) {
    // rows behind this segment contributed: start from the state the forward pass recorded at the segment's end
    total = seg_base + BLEND_HEAD;
    // next == 0: the record is missing (the segment slots ran out, which the forward call reported, or n_contrib is
    // not the forward pass's own); the final state stands in, exact for the pixels that end inside this segment
    if (next != 0) {
      const BlendRecord* ck = ckpt + (size_t)(next - 1) * 256 + lane;
#pragma unroll
      for (int s = 0; s < BLEND_SLOTS; ++s) {
        const BlendRecord c = ck[32 * s];  // pixel (row 2 s + lane / 16, column lane % 16) = thread 32 s + lane of the tail
        T[s] = c.T;
        SG[s] = (float)fma(c.S2, (double)g2[s], fma(c.S1, (double)g1[s], c.S0 * (double)g0[s]));
      }
    }
  }
  total -= seg_base;  // entries of this segment to walk
  const uint32_t seg_start = start + seg_base;
  // walk the remaining entries back to front, 32 at a time
  const int nb = (int)((total + 31) / 32);
  for (int bi = nb - 1; bi >= 0; --bi) {
    const uint32_t b = (uint32_t)bi * 32;
    const int cnt = (int)min(32u, total - b);
    bool reach = false;
    if ((int)lane < cnt) {
      const uint32_t r = min(vals[seg_start + b + lane], row_cap - 1);  // in range whatever the list holds
      const float2 c = xy[r];
      BlendRow row;
      row.q0 = make_float4(c.x, c.y, rgb[3 * (size_t)r], rgb[3 * (size_t)r + 1]);
      const float4 co = conic_o[r];
      row.q1 = blend_stage_conic(co);
      s_rowdata[warp][lane] = row;
      s_blue[warp][lane] = make_float2(rgb[3 * (size_t)r + 2], 1.f / co.w);
      s_rowid[warp][lane] = r;
      reach = blend_reaches_tile(c.x, c.y, co.x, co.y, co.z, blend_power_cut(alpha_min, co.w), tile_x0 + 0.5f,
                                 tile_y0 + 0.5f);
    }
    // warp-uniform: only the rows whose ellipse reaches the tile are evaluated, back to front
    uint32_t rows = __ballot_sync(0xffffffffu, reach);
    __syncwarp();
    while (rows) {
      const int j = 31 - __clz(rows);
      rows ^= 1u << j;
      const float4 q0 = s_rowdata[warp][j].q0, q1 = s_rowdata[warp][j].q1;
      const float blue = s_blue[warp][j].x;
      const float dx = q0.x - fx;
      float h0, h1, h2;
      blend_x_terms(q1, dx, h0, h1, h2);
      const float dy0 = q0.y - fy0;
      const uint32_t k = seg_base + b + j;
      // the eight exponents first (independent, they overlap in the pipeline), then test and differentiate slot by slot;
      // per-lane sums over its eight pixels, the x-dependent factors are applied once at the end
      float pw[BLEND_SLOTS];
#pragma unroll
      for (int s = 0; s < BLEND_SLOTS; ++s) pw[s] = blend_power(h0, h1, h2, dy0 - (float)(2 * s));
      float ar = 0.f, ag = 0.f, ab = 0.f, gpsum = 0.f, m1y = 0.f, m2yy = 0.f;
      bool some = false;
#pragma unroll
      for (int s = 0; s < BLEND_SLOTS; ++s) {
        if (k < last[s] && blend_passes(pw[s], q1.w, l2amin)) {
          some = true;
          const float dy = dy0 - (float)(2 * s);
          const float og = blend_ex2(pw[s]);  // opacity * exp(power)
          const float alpha = fminf(alpha_max, og);
          const float inv = __fdividef(1.f, 1.f - alpha);
          const float Tb = T[s] * inv;  // transmittance in front of this row
          const float w = alpha * Tb;
          ar = fmaf(w, g0[s], ar); ag = fmaf(w, g1[s], ag); ab = fmaf(w, g2[s], ab);
          const float cg = fmaf(blue, g2[s], fmaf(q0.w, g1[s], q0.z * g0[s]));
          const float dLda = Tb * cg - SG[s] * inv;
          SG[s] = fmaf(w, cg, SG[s]);
          T[s] = Tb;
          if (og <= alpha_max) {  // a clamped alpha passes no gradient to opacity or geometry
            const float gp = og * dLda;  // dL/dpower; dL/dopacity is this over the opacity
            gpsum += gp;
            const float gy = gp * dy;
            m1y += gy;
            m2yy = fmaf(gy, dy, m2yy);
          }
        }
      }
      if (!__any_sync(0xffffffffu, some)) continue;  // the row blends nowhere in the tile
      const float gd = dx * gpsum;  // sum of dL/dpower * dx
      const float ao = gpsum * s_blue[warp][j].y;
      // the staged conic is (-A log2(e) / 2, -B log2(e), -C log2(e) / 2): -(A gd + B m1y) = ln 2 (2 sA gd + sB m1y)
      const float vu = BLEND_LN2 * fmaf(2.f * q1.x, gd, q1.y * m1y);
      const float vv = BLEND_LN2 * fmaf(2.f * q1.z, m1y, q1.y * gd);
      const float vA = -0.5f * dx * gd, vB = -dx * m1y, vC = -0.5f * m2yy;
      const float t8 = warp_transpose_sum8(vu, vv, vA, vB, vC, ao, ar, ag, lane);
      for (int o = 16; o > 0; o >>= 1) ab += __shfl_xor_sync(0xffffffffu, ab, o);
      const uint32_t rid = s_rowid[warp][j];
      float* dst = g2d + (size_t)rid * 9;
      if ((lane & 3) == 0) atomicAdd(dst + (lane >> 2), t8);
      if (lane == 1) atomicAdd(dst + 8, ab);
      if (TRACK) {
        if (lane == 2) row_active[rid] = 1;  // realized-active: blended into at least one pixel
      }
    }
    __syncwarp();
  }
  }
}

// ----------------------------------------------------------------------------------------------------------------
template <int DEG>
__global__ void __launch_bounds__(128)
render_bwd_project_kernel(const float* __restrict__ means, const float* __restrict__ log_scales,
                          const float4* __restrict__ quats, const float* __restrict__ opacity_logit,
                          const float* __restrict__ sh, CamParams cam, float dilation, const uint32_t* __restrict__ prim_id,
                          const uint8_t* __restrict__ clamp_flags, const uint32_t* __restrict__ num_rows, uint32_t capacity,
                          const float* __restrict__ g2d, float* __restrict__ g_means, float* __restrict__ g_ls,
                          float4* __restrict__ g_quats, float* __restrict__ g_opac, float* __restrict__ g_sh,
                          uint8_t* __restrict__ row_zero, uint32_t n) {
  odin_after_predecessor();
  constexpr int K = (DEG + 1) * (DEG + 1);
  const uint32_t V = min(*num_rows, capacity);
  for (uint32_t r = blockIdx.x * blockDim.x + threadIdx.x; r < V; r += gridDim.x * blockDim.x) {
    const size_t p = min(prim_id[r], n - 1);
    const float* gg = g2d + (size_t)r * 9;
    const float gu = gg[0], gv = gg[1], gA = gg[2], gB = gg[3], gC = gg[4], go = gg[5];
    const float grgb[3] = {gg[6], gg[7], gg[8]};
    // The chain rule is linear in these nine words.  Most touched rows never blend into a pixel (they are occluded)
    // and arrive with all nine at zero: their gradient row is zero and needs neither the scene nor any arithmetic.
    if (gu == 0.f && gv == 0.f && gA == 0.f && gB == 0.f && gC == 0.f && go == 0.f && grgb[0] == 0.f && grgb[1] == 0.f &&
        grgb[2] == 0.f) {
      if (row_zero) {  // the caller takes a flag instead of a row of zeros (the optimizer then reads no gradient for it)
        row_zero[r] = 1;
        continue;
      }
#pragma unroll
      for (int j = 0; j < 3; ++j) { g_means[3 * (size_t)r + j] = 0.f; g_ls[3 * (size_t)r + j] = 0.f; }
      g_quats[r] = make_float4(0.f, 0.f, 0.f, 0.f);
      g_opac[r] = 0.f;
      float* out = g_sh + (size_t)r * (3 * K);
      if ((3 * K) % 4 == 0) {
#pragma unroll
        for (int i = 0; i < 3 * K / 4; ++i) reinterpret_cast<float4*>(out)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      } else {
#pragma unroll
        for (int i = 0; i < 3 * K; ++i) out[i] = 0.f;
      }
      continue;
    }
    if (row_zero) row_zero[r] = 0;
    const float mx = means[3 * p], my = means[3 * p + 1], mz = means[3 * p + 2];
    SplatGeom g;
    odin_camera_space(cam, mx, my, mz, g.t);
    const float ls[3] = {log_scales[3 * p], log_scales[3 * p + 1], log_scales[3 * p + 2]};
    odin_splat_geometry(cam, dilation, ls, quats[p], g);
    // conic -> 2D covariance
    const float a = g.a, b = g.b, c = g.c, D = g.det * g.det;
    const float ga = (-c * c * gA + b * c * gB - b * b * gC) / D;
    const float gb = (2.f * b * c * gA - (a * c + b * b) * gB + 2.f * a * b * gC) / D;
    const float gc = (-b * b * gA + a * b * gB - a * a * gC) / D;
    const float Gs[4] = {ga, 0.5f * gb, 0.5f * gb, gc};
    float GT[6];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 3; ++j) GT[3 * i + j] = Gs[2 * i] * g.Tm[j] + Gs[2 * i + 1] * g.Tm[3 + j];
    const float S[9] = {g.Sig[0], g.Sig[1], g.Sig[2], g.Sig[1], g.Sig[3], g.Sig[4], g.Sig[2], g.Sig[4], g.Sig[5]};
    float gSig[9], gTm[6];
#pragma unroll
    for (int i = 0; i < 3; ++i)
#pragma unroll
      for (int j = 0; j < 3; ++j) gSig[3 * i + j] = g.Tm[i] * GT[j] + g.Tm[3 + i] * GT[3 + j];
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 3; ++j) gTm[3 * i + j] = 2.f * (GT[3 * i] * S[j] + GT[3 * i + 1] * S[3 + j] + GT[3 * i + 2] * S[6 + j]);
    // dL/dJ = dL/dTm R_c^T; only J00, J02, J11, J12 depend on t
    const float gJ00 = gTm[0] * cam.R[0] + gTm[1] * cam.R[1] + gTm[2] * cam.R[2];
    const float gJ02 = gTm[0] * cam.R[6] + gTm[1] * cam.R[7] + gTm[2] * cam.R[8];
    const float gJ11 = gTm[3] * cam.R[3] + gTm[4] * cam.R[4] + gTm[5] * cam.R[5];
    const float gJ12 = gTm[3] * cam.R[6] + gTm[4] * cam.R[7] + gTm[5] * cam.R[8];
    const float tx = g.t[0], ty = g.t[1], tz = g.t[2];
    const float iz = 1.f / tz, iz2 = iz * iz, iz3 = iz2 * iz;
    float gt0 = 0.f, gt1 = 0.f, gt2 = -(gJ00 * cam.fx + gJ11 * cam.fy) * iz2;
    if (g.clampx) gt2 += gJ02 * cam.fx * g.Lx * iz2;
    else { gt0 += -gJ02 * cam.fx * iz2; gt2 += 2.f * gJ02 * cam.fx * tx * iz3; }
    if (g.clampy) gt2 += gJ12 * cam.fy * g.Ly * iz2;
    else { gt1 += -gJ12 * cam.fy * iz2; gt2 += 2.f * gJ12 * cam.fy * ty * iz3; }
    gt0 += gu * cam.fx * iz; gt2 += -gu * cam.fx * tx * iz2;
    gt1 += gv * cam.fy * iz; gt2 += -gv * cam.fy * ty * iz2;
    float gmu[3];
#pragma unroll
    for (int j = 0; j < 3; ++j) gmu[j] = cam.R[j] * gt0 + cam.R[3 + j] * gt1 + cam.R[6 + j] * gt2;
    // Sigma = M M^T
    float gM[9], gR[9], gls[3];
#pragma unroll
    for (int i = 0; i < 3; ++i)
#pragma unroll
      for (int j = 0; j < 3; ++j)
        gM[3 * i + j] = 2.f * (gSig[3 * i] * g.M[j] + gSig[3 * i + 1] * g.M[3 + j] + gSig[3 * i + 2] * g.M[6 + j]);
#pragma unroll
    for (int j = 0; j < 3; ++j) {
      float gs = 0.f;
#pragma unroll
      for (int i = 0; i < 3; ++i) { gs += g.Rm[3 * i + j] * gM[3 * i + j]; gR[3 * i + j] = gM[3 * i + j] * g.s[j]; }
      gls[j] = g.s[j] * gs;
    }
    const float w = g.qn[0], x = g.qn[1], y = g.qn[2], z = g.qn[3];
    float gq[4];
    gq[0] = 2.f * (-z * gR[1] + y * gR[2] + z * gR[3] - x * gR[5] - y * gR[6] + x * gR[7]);
    gq[1] = 2.f * (y * gR[1] + z * gR[2] + y * gR[3] - 2.f * x * gR[4] - w * gR[5] + z * gR[6] + w * gR[7] - 2.f * x * gR[8]);
    gq[2] = 2.f * (-2.f * y * gR[0] + x * gR[1] + w * gR[2] + x * gR[3] + z * gR[5] - w * gR[6] + z * gR[7] - 2.f * y * gR[8]);
    gq[3] = 2.f * (-2.f * z * gR[0] - w * gR[1] + x * gR[2] + w * gR[3] - 2.f * z * gR[4] + y * gR[5] + x * gR[6] + y * gR[7]);
    const float qd = w * gq[0] + x * gq[1] + y * gq[2] + z * gq[3];
    const float iq = 1.f / g.qlen;
    // colour
    float dvx = mx - cam.pos[0], dvy = my - cam.pos[1], dvz = mz - cam.pos[2];
    const float len = sqrtf(dvx * dvx + dvy * dvy + dvz * dvz);
    const float d0 = dvx / len, d1 = dvy / len, d2 = dvz / len;
    float Y[16], dY[16][3];
    odin_sh_basis<DEG>(d0, d1, d2, Y);
    odin_sh_basis_grad<DEG>(d0, d1, d2, dY);
    const uint8_t flags = clamp_flags[r];
    float gch[3];
#pragma unroll
    for (int ch = 0; ch < 3; ++ch) gch[ch] = (flags & (1u << ch)) ? 0.f : grgb[ch];
    float gd[3] = {0.f, 0.f, 0.f};
    const float* shrow = sh + p * (3 * K);
    float* gshrow = g_sh + (size_t)r * (3 * K);
    if ((3 * K) % 4 == 0) {  // 12 or 48 floats per row: 16-byte loads and stores
      const float4* sh4 = reinterpret_cast<const float4*>(shrow);
      float4* gsh4 = reinterpret_cast<float4*>(gshrow);
#pragma unroll
      for (int i = 0; i < 3 * K / 4; ++i) {
        const float4 c = sh4[i];
        const float e[4] = {c.x, c.y, c.z, c.w};
        float o4[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int w = 4 * i + j, k = w / 3, ch = w % 3;
          o4[j] = Y[k] * gch[ch];
          if (k > 0) {
            const float wgt = e[j] * gch[ch];
            gd[0] += dY[k][0] * wgt; gd[1] += dY[k][1] * wgt; gd[2] += dY[k][2] * wgt;
          }
        }
        gsh4[i] = make_float4(o4[0], o4[1], o4[2], o4[3]);
      }
    } else {
#pragma unroll
      for (int k = 0; k < K; ++k) {
#pragma unroll
        for (int ch = 0; ch < 3; ++ch) {
          gshrow[3 * k + ch] = Y[k] * gch[ch];
          if (k > 0) {
            const float wgt = shrow[3 * k + ch] * gch[ch];
            gd[0] += dY[k][0] * wgt; gd[1] += dY[k][1] * wgt; gd[2] += dY[k][2] * wgt;
          }
        }
      }
    }
    const float dd = d0 * gd[0] + d1 * gd[1] + d2 * gd[2];
    gmu[0] += (gd[0] - d0 * dd) / len; gmu[1] += (gd[1] - d1 * dd) / len; gmu[2] += (gd[2] - d2 * dd) / len;
    g_means[3 * (size_t)r] = gmu[0]; g_means[3 * (size_t)r + 1] = gmu[1]; g_means[3 * (size_t)r + 2] = gmu[2];
    g_ls[3 * (size_t)r] = gls[0]; g_ls[3 * (size_t)r + 1] = gls[1]; g_ls[3 * (size_t)r + 2] = gls[2];
    g_quats[r] = make_float4((gq[0] - w * qd) * iq, (gq[1] - x * qd) * iq, (gq[2] - y * qd) * iq, (gq[3] - z * qd) * iq);
    const float o = 1.f / (1.f + expf(-opacity_logit[p]));
    g_opac[r] = o * (1.f - o) * go;
  }
}

}  // namespace

extern "C" int odin_render_bwd(odin_ctx* ctx, const odin_scene* scene, const odin_camera* cam, const odin_projected* proj,
                               const uint32_t* d_vals, const uint32_t* d_tile_ranges, const float* d_final_T,
                               const uint32_t* d_n_contrib, const float* d_dL_drgb, float* d_grad2d, odin_scene* grad_rows,
                               uint8_t* d_row_active, uint8_t* d_row_zero, void* ws, size_t ws_bytes, void* stream) {
  if (!ctx || !proj || !grad_rows) return ODIN_ERR_NULL;
  int rc = odin_check_scene(scene);
  if (rc != ODIN_OK) return rc;
  rc = odin_check_camera(cam);
  if (rc != ODIN_OK) return rc;
  rc = odin_check_scene(grad_rows);
  if (rc != ODIN_OK) return rc;
  if (grad_rows->sh_degree != scene->sh_degree) return ODIN_ERR_INVALID_ARG;
  if (proj->capacity == 0 || scene->n == 0) return ODIN_OK;
  if (grad_rows->n < proj->capacity) return ODIN_ERR_INVALID_ARG;
  if (!d_vals || !d_tile_ranges || !d_final_T || !d_n_contrib || !d_dL_drgb || !d_grad2d || !proj->xy ||
      !proj->conic_opacity || !proj->rgb || !proj->prim_id || !proj->clamp_flags || !proj->num_rows)
    return ODIN_ERR_NULL;
  cudaStream_t st = (cudaStream_t)stream;
  const int TX = (cam->width + 15) / 16, TY = (cam->height + 15) / 16;
  if (!ws || !odin_aligned(ws, 256) || ws_bytes < blend_ws_bytes(cam->width, cam->height)) return ODIN_ERR_WORKSPACE;
  const int n_tiles = TX * TY;
  const BlendWs L = blend_ws_layout(n_tiles, blend_ws_segments(n_tiles, ws_bytes));
  char* base = reinterpret_cast<char*>(ws);
  uint32_t* header = reinterpret_cast<uint32_t*>(base);
  uint32_t* ticket = header + 1;
  ODIN_CUDA(odin_zero(ctx, ticket, 4, st));  // in front of all three kernels: they are launched back to back
  const uint32_t zgrid = (uint32_t)ctx->sm_count * 8;
  {
    OdinKernelScope ks(ctx, K_ZERO_ROWS, st);
    ODIN_CUDA(odin_launch(ctx, false, zero_rows_kernel, dim3(zgrid), dim3(256), 0, st, d_grad2d, d_row_active, proj->num_rows,
                          proj->capacity));
  }
  {
    OdinKernelScope ks(ctx, K_BWD_BLEND, st);
    const size_t blocks_all = ((size_t)n_tiles + L.segments + BLEND_WARPS - 1) / BLEND_WARPS;
    const int blocks = blocks_all < (size_t)ctx->sm_count * 8 ? (int)blocks_all : ctx->sm_count * 8;  // resident warps pull work
#define LAUNCH_BLEND(TRACK)                                                                                             \
  ODIN_CUDA(odin_launch(ctx, true, render_bwd_blend_kernel<TRACK>, dim3(blocks), dim3(BLEND_THREADS), 0, st,            \
      reinterpret_cast<const float2*>(proj->xy), reinterpret_cast<const float4*>(proj->conic_opacity), proj->rgb,       \
      d_vals, reinterpret_cast<const uint2*>(d_tile_ranges), cam->width, cam->height, TX, n_tiles, cam->bg[0],          \
      cam->bg[1], cam->bg[2], ctx->cfg.alpha_min, ctx->cfg.alpha_max,                                                   \
      reinterpret_cast<const uint32_t*>(base + L.tile_first), header + 2,                                               \
      reinterpret_cast<const uint2*>(base + L.seg_tile), reinterpret_cast<const uint2*>(base + L.seg_link),             \
      reinterpret_cast<const BlendRecord*>(base + L.ckpt), L.segments, d_final_T, d_n_contrib, d_dL_drgb, d_grad2d, ticket,  \
      d_row_active, proj->capacity, header + 8, reinterpret_cast<const uint32_t*>(base + L.bwd_queue)))
    if (d_row_active) LAUNCH_BLEND(true);
    else LAUNCH_BLEND(false);
#undef LAUNCH_BLEND
  }
  const CamParams cp = odin_cam_params(cam, ctx->cfg);
  const uint32_t blocks_cap = (proj->capacity + 127) / 128;
  const uint32_t pgrid = blocks_cap < (uint32_t)ctx->sm_count * 16 ? blocks_cap : (uint32_t)ctx->sm_count * 16;
#define LAUNCH(D)                                                                                                       \
  ODIN_CUDA(odin_launch(ctx, true, render_bwd_project_kernel<D>, dim3(pgrid), dim3(128), 0, st,                         \
      scene->means, scene->log_scales, reinterpret_cast<const float4*>(scene->quats), scene->opacity_logit, scene->sh,  \
      cp, ctx->cfg.dilation, proj->prim_id, proj->clamp_flags, proj->num_rows, proj->capacity, d_grad2d,                \
      grad_rows->means, grad_rows->log_scales, reinterpret_cast<float4*>(grad_rows->quats), grad_rows->opacity_logit,    \
      grad_rows->sh, d_row_zero, scene->n))
  OdinKernelScope ks(ctx, K_BWD_PROJECT, st);
  switch (scene->sh_degree) {
    case 0: LAUNCH(0); break;
    case 1: LAUNCH(1); break;
    case 2: LAUNCH(2); break;
    default: LAUNCH(3); break;
  }
#undef LAUNCH
  return odin_launch_status();
}
