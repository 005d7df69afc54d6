// Exact binning (odin_config.binning = 2): which tiles of its rectangle a primitive keeps.  Shared by the projection
// (tile counts) and by the binning kernels (which recompute the spans instead of storing them), so every operation is
// an explicitly rounded intrinsic: the decisions must not depend on which translation unit, or which fused
// multiply-add contraction, evaluates them.
//
// Rule (Sec. 5 variant; the image is unchanged): a tile is kept iff the region alpha = opacity exp(-q/2) >= alpha_min,
// q(d) = A dx^2 + 2 B dx dy + C dy^2 <= k = 2 ln(opacity / alpha_min) around the centre, reaches the rectangle spanned
// by the tile's 16 x 16 pixel centres: the minimum of the convex q over that rectangle (0 if the centre is inside, else
// on one of the four edges at the clamped one-dimensional minimiser) is at most k (1 + 1e-4) + 1e-3 + 2e-6 x the
// largest term q can take on the rectangle.  The kept tiles of one tile row are an interval; it is reported as the
// span from the first to the last tile of the row that passes.
#pragma once
#include <cuda_runtime.h>

struct SpanConic {
  float u, v, A, B, C, k;  // centre, conic, threshold 2 ln(opacity / alpha_min); k < 0: nothing passes
};

__device__ __forceinline__ SpanConic odin_span_conic(float u, float v, float A, float B, float C, float opacity,
                                                     float alpha_min) {
  SpanConic e;
  e.u = u; e.v = v; e.A = A; e.B = B; e.C = C;
  e.k = (opacity >= alpha_min) ? __fmul_rn(2.f, logf(__fdiv_rn(opacity, alpha_min))) : -1.f;
  return e;
}

__device__ __forceinline__ float odin_span_q(const SpanConic& e, float dx, float dy) {
  const float a = __fmul_rn(__fmul_rn(e.A, dx), dx);
  const float b = __fmul_rn(__fmul_rn(__fmul_rn(2.f, e.B), dx), dy);
  const float c = __fmul_rn(__fmul_rn(e.C, dy), dy);
  return __fadd_rn(__fadd_rn(a, b), c);
}

__device__ __forceinline__ bool odin_tile_reached(const SpanConic& e, int tx, int ty) {
  if (e.k < 0.f) return false;
  const float xl = __fadd_rn(__fadd_rn(__fmul_rn((float)tx, 16.f), 0.5f), -e.u), xh = __fadd_rn(xl, 15.f);
  const float yl = __fadd_rn(__fadd_rn(__fmul_rn((float)ty, 16.f), 0.5f), -e.v), yh = __fadd_rn(yl, 15.f);
  float qmin = 0.f;
  if (!(xl <= 0.f && xh >= 0.f && yl <= 0.f && yh >= 0.f)) {
    const float t0 = fminf(fmaxf(__fdiv_rn(__fmul_rn(-e.B, xl), e.C), yl), yh);
    const float t1 = fminf(fmaxf(__fdiv_rn(__fmul_rn(-e.B, xh), e.C), yl), yh);
    const float s0 = fminf(fmaxf(__fdiv_rn(__fmul_rn(-e.B, yl), e.A), xl), xh);
    const float s1 = fminf(fmaxf(__fdiv_rn(__fmul_rn(-e.B, yh), e.A), xl), xh);
    qmin = fminf(fminf(odin_span_q(e, xl, t0), odin_span_q(e, xh, t1)), fminf(odin_span_q(e, s0, yl), odin_span_q(e, s1, yh)));
  }
  const float mx = fmaxf(fabsf(xl), fabsf(xh)), my = fmaxf(fabsf(yl), fabsf(yh));
  const float big = __fadd_rn(__fadd_rn(__fmul_rn(__fmul_rn(e.A, mx), mx),
                                        __fmul_rn(__fmul_rn(__fmul_rn(2.f, fabsf(e.B)), mx), my)),
                              __fmul_rn(__fmul_rn(e.C, my), my));
  const float bound = __fadd_rn(__fadd_rn(__fmul_rn(e.k, 1.0001f), 1e-3f), __fmul_rn(2e-6f, big));
  return qmin <= bound;
}

// Kept tiles [xa, xb) of tile row ty inside [x0, x1) (xa == xb: none).  Short rows are scanned.  For a long row the
// x extent of the ellipse inside the strip of the row's pixel centres is computed in closed form (with a bound that is
// at least the rule's for every tile of the row, so the estimate errs on the wide side by a tile at most), and both ends
// are then moved with the exact predicate until the end tiles pass and their outer neighbours do not.
__device__ __forceinline__ void odin_row_span(const SpanConic& e, int ty, int x0, int x1, int& xa, int& xb) {
  xa = xb = x0;
  if (e.k < 0.f || x1 <= x0) return;
  if (x1 - x0 <= 3) {
    int first = x1, last = x0 - 1;
    for (int tx = x0; tx < x1; ++tx)
      if (odin_tile_reached(e, tx, ty)) { first = min(first, tx); last = tx; }
    if (last >= first) { xa = first; xb = last + 1; }
    return;
  }
  const float yl = (float)ty * 16.f + 0.5f - e.v, yh = yl + 15.f;
  const float det = e.A * e.C - e.B * e.B;
  int a = x0, b = x1;  // estimate; the whole row if the conic is not a proper ellipse
  if (det > 0.f && e.A > 0.f && e.C > 0.f) {
    const float mx = fmaxf(fabsf((float)x0 * 16.f + 0.5f - e.u), fabsf((float)x1 * 16.f - 0.5f - e.u));
    const float my = fmaxf(fabsf(yl), fabsf(yh));
    const float kb = e.k * 1.0002f + 2e-3f + 4e-6f * (e.A * mx * mx + 2.f * fabsf(e.B) * mx * my + e.C * my * my);
    const float Y = sqrtf(kb * e.A / det);
    if (yl > Y || yh < -Y) return;              // the strip misses the ellipse
    const float X = sqrtf(kb * e.C / det);      // half extent in x, reached at dy = -+ B X / C
    const float dmax = -e.B * X / e.C, dmin = -dmax;
    float xmax = X, xmin = -X;
    if (dmax < yl || dmax > yh) {
      const float dyc = fminf(fmaxf(dmax, yl), yh);
      xmax = (-e.B * dyc + sqrtf(fmaxf(kb * e.A - det * dyc * dyc, 0.f))) / e.A;
    }
    if (dmin < yl || dmin > yh) {
      const float dyc = fminf(fmaxf(dmin, yl), yh);
      xmin = (-e.B * dyc - sqrtf(fmaxf(kb * e.A - det * dyc * dyc, 0.f))) / e.A;
    }
    // tile tx holds pixel centres 16 tx + 0.5 .. 16 tx + 15.5
    const float fa = ceilf((e.u + xmin - 15.5f) * 0.0625f) - 1.f, fb = floorf((e.u + xmax - 0.5f) * 0.0625f) + 2.f;
    a = (int)fminf(fmaxf(fa, (float)x0), (float)x1);
    b = (int)fminf(fmaxf(fb, (float)x0), (float)x1);
    if (b <= a) {  // a sliver between two tiles' pixel centres: look at the tiles around it
      a = max(x0, a - 1);
      b = min(x1, a + 2);
    }
  }
  while (a < b && !odin_tile_reached(e, a, ty)) ++a;
  if (a == b) return;
  while (b - 1 > a && !odin_tile_reached(e, b - 1, ty)) --b;
  while (a > x0 && odin_tile_reached(e, a - 1, ty)) --a;   // (only if the estimate was too narrow)
  while (b < x1 && odin_tile_reached(e, b, ty)) ++b;
  xa = a;
  xb = b;
}

// Kept tiles of a whole rectangle, the tile rows spread over the lanes of the warp (all 32 lanes must call with the
// same arguments).  For rectangles of many tile rows: one lane walking them would hold up its warp.
__device__ __forceinline__ uint32_t odin_rect_kept_warp(const SpanConic& e, int x0, int y0, int x1, int y1) {
  uint32_t kept = 0;
  for (int y = y0 + (int)(threadIdx.x & 31); y < y1; y += 32) {
    int xa, xb;
    odin_row_span(e, y, x0, x1, xa, xb);
    kept += (uint32_t)(xb - xa);
  }
  return __reduce_add_sync(0xffffffffu, kept);
}

__device__ __forceinline__ SpanConic odin_span_conic_bcast(const SpanConic& e, int src) {
  SpanConic q;
  q.u = __shfl_sync(0xffffffffu, e.u, src); q.v = __shfl_sync(0xffffffffu, e.v, src);
  q.A = __shfl_sync(0xffffffffu, e.A, src); q.B = __shfl_sync(0xffffffffu, e.B, src);
  q.C = __shfl_sync(0xffffffffu, e.C, src); q.k = __shfl_sync(0xffffffffu, e.k, src);
  return q;
}
