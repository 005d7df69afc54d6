// Device-side projection geometry shared by the preprocessing kernel and its backward.
#pragma once
#include "common.cuh"

struct SplatGeom {
  float t[3];          // camera-space mean
  float s[3];          // exp(log scale)
  float qn[4], qlen;   // normalised quaternion and |q|
  float Rm[9];         // rotation matrix
  float M[9];          // Rm diag(s)
  float Sig[6];        // symmetric 3x3: xx, xy, xz, yy, yz, zz
  float Tm[6];         // J R_c (2x3)
  float Lx, Ly;        // clamped ratios used inside J
  bool clampx, clampy;
  float a, b, c, det;  // 2D covariance (dilated) and its determinant
};

__device__ __forceinline__ void odin_camera_space(const CamParams& cam, float mx, float my, float mz, float* t) {
  t[0] = cam.R[0] * mx + cam.R[1] * my + cam.R[2] * mz + cam.t[0];
  t[1] = cam.R[3] * mx + cam.R[4] * my + cam.R[5] * mz + cam.t[1];
  t[2] = cam.R[6] * mx + cam.R[7] * my + cam.R[8] * mz + cam.t[2];
}

// Fills everything from g.t onwards (g.t must be set).  Plain IEEE operations only: integer decisions taken from
// these values (radius, rectangle) must not depend on approximate intrinsics.
__device__ __forceinline__ void odin_splat_geometry(const CamParams& cam, float dilation, const float* ls, const float4 q,
                                                    SplatGeom& g) {
  g.s[0] = expf(ls[0]); g.s[1] = expf(ls[1]); g.s[2] = expf(ls[2]);
  g.qlen = sqrtf(q.x * q.x + q.y * q.y + q.z * q.z + q.w * q.w);
  const float w = q.x / g.qlen, x = q.y / g.qlen, y = q.z / g.qlen, z = q.w / g.qlen;  // stored order is (w,x,y,z)
  g.qn[0] = w; g.qn[1] = x; g.qn[2] = y; g.qn[3] = z;
  g.Rm[0] = 1.f - 2.f * (y * y + z * z); g.Rm[1] = 2.f * (x * y - w * z); g.Rm[2] = 2.f * (x * z + w * y);
  g.Rm[3] = 2.f * (x * y + w * z); g.Rm[4] = 1.f - 2.f * (x * x + z * z); g.Rm[5] = 2.f * (y * z - w * x);
  g.Rm[6] = 2.f * (x * z - w * y); g.Rm[7] = 2.f * (y * z + w * x); g.Rm[8] = 1.f - 2.f * (x * x + y * y);
#pragma unroll
  for (int i = 0; i < 3; ++i)
#pragma unroll
    for (int j = 0; j < 3; ++j) g.M[3 * i + j] = g.Rm[3 * i + j] * g.s[j];
  g.Sig[0] = g.M[0] * g.M[0] + g.M[1] * g.M[1] + g.M[2] * g.M[2];
  g.Sig[1] = g.M[0] * g.M[3] + g.M[1] * g.M[4] + g.M[2] * g.M[5];
  g.Sig[2] = g.M[0] * g.M[6] + g.M[1] * g.M[7] + g.M[2] * g.M[8];
  g.Sig[3] = g.M[3] * g.M[3] + g.M[4] * g.M[4] + g.M[5] * g.M[5];
  g.Sig[4] = g.M[3] * g.M[6] + g.M[4] * g.M[7] + g.M[5] * g.M[8];
  g.Sig[5] = g.M[6] * g.M[6] + g.M[7] * g.M[7] + g.M[8] * g.M[8];
  const float tz = g.t[2];
  const float rx = g.t[0] / tz, ry = g.t[1] / tz;
  g.clampx = (rx < -cam.limx) || (rx > cam.limx);
  g.clampy = (ry < -cam.limy) || (ry > cam.limy);
  g.Lx = fminf(cam.limx, fmaxf(-cam.limx, rx));
  g.Ly = fminf(cam.limy, fmaxf(-cam.limy, ry));
  const float j00 = cam.fx / tz, j02 = -cam.fx * (g.Lx * tz) / (tz * tz);
  const float j11 = cam.fy / tz, j12 = -cam.fy * (g.Ly * tz) / (tz * tz);
#pragma unroll
  for (int j = 0; j < 3; ++j) {
    g.Tm[j] = j00 * cam.R[j] + j02 * cam.R[6 + j];
    g.Tm[3 + j] = j11 * cam.R[3 + j] + j12 * cam.R[6 + j];
  }
  // Sigma' = Tm Sigma Tm^T
  const float S[9] = {g.Sig[0], g.Sig[1], g.Sig[2], g.Sig[1], g.Sig[3], g.Sig[4], g.Sig[2], g.Sig[4], g.Sig[5]};
  float TS[6];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int j = 0; j < 3; ++j) TS[3 * i + j] = g.Tm[3 * i] * S[j] + g.Tm[3 * i + 1] * S[3 + j] + g.Tm[3 * i + 2] * S[6 + j];
  const float s00 = TS[0] * g.Tm[0] + TS[1] * g.Tm[1] + TS[2] * g.Tm[2];
  const float s01 = TS[0] * g.Tm[3] + TS[1] * g.Tm[4] + TS[2] * g.Tm[5];
  const float s11 = TS[3] * g.Tm[3] + TS[4] * g.Tm[4] + TS[5] * g.Tm[5];
  g.a = s00 + dilation; g.b = s01; g.c = s11 + dilation;
  g.det = g.a * g.c - g.b * g.b;
}

// Real spherical harmonics up to degree 3 as polynomials of the unit direction.
#define SH_C0 0.28209479177387814f
#define SH_C1 0.4886025119029199f
#define SH_C2A 1.0925484305920792f
#define SH_C2B 0.31539156525252005f
#define SH_C2C 0.5462742152960396f
#define SH_C3A 0.5900435899266435f
#define SH_C3B 2.890611442640554f
#define SH_C3C 0.4570457994644658f
#define SH_C3D 0.3731763325901154f
#define SH_C3E 1.445305721320277f

template <int DEG>
__device__ __forceinline__ void odin_sh_basis(float x, float y, float z, float* Y) {
  Y[0] = SH_C0;
  if (DEG >= 1) { Y[1] = -SH_C1 * y; Y[2] = SH_C1 * z; Y[3] = -SH_C1 * x; }
  if (DEG >= 2) {
    const float xx = x * x, yy = y * y, zz = z * z;
    Y[4] = SH_C2A * x * y; Y[5] = -SH_C2A * y * z; Y[6] = SH_C2B * (2.f * zz - xx - yy);
    Y[7] = -SH_C2A * x * z; Y[8] = SH_C2C * (xx - yy);
    if (DEG >= 3) {
      Y[9] = -SH_C3A * y * (3.f * xx - yy);
      Y[10] = SH_C3B * x * y * z;
      Y[11] = -SH_C3C * y * (4.f * zz - xx - yy);
      Y[12] = SH_C3D * z * (2.f * zz - 3.f * xx - 3.f * yy);
      Y[13] = -SH_C3C * x * (4.f * zz - xx - yy);
      Y[14] = SH_C3E * z * (xx - yy);
      Y[15] = -SH_C3A * x * (xx - 3.f * yy);
    }
  }
}

// d/d(x,y,z) of each basis polynomial (x, y, z treated as free variables).
template <int DEG>
__device__ __forceinline__ void odin_sh_basis_grad(float x, float y, float z, float (*dY)[3]) {
  dY[0][0] = dY[0][1] = dY[0][2] = 0.f;
  if (DEG >= 1) {
    dY[1][0] = 0.f; dY[1][1] = -SH_C1; dY[1][2] = 0.f;
    dY[2][0] = 0.f; dY[2][1] = 0.f; dY[2][2] = SH_C1;
    dY[3][0] = -SH_C1; dY[3][1] = 0.f; dY[3][2] = 0.f;
  }
  if (DEG >= 2) {
    const float xx = x * x, yy = y * y, zz = z * z;
    dY[4][0] = SH_C2A * y; dY[4][1] = SH_C2A * x; dY[4][2] = 0.f;
    dY[5][0] = 0.f; dY[5][1] = -SH_C2A * z; dY[5][2] = -SH_C2A * y;
    dY[6][0] = -2.f * SH_C2B * x; dY[6][1] = -2.f * SH_C2B * y; dY[6][2] = 4.f * SH_C2B * z;
    dY[7][0] = -SH_C2A * z; dY[7][1] = 0.f; dY[7][2] = -SH_C2A * x;
    dY[8][0] = 2.f * SH_C2C * x; dY[8][1] = -2.f * SH_C2C * y; dY[8][2] = 0.f;
    if (DEG >= 3) {
      dY[9][0] = -6.f * SH_C3A * x * y; dY[9][1] = -3.f * SH_C3A * (xx - yy); dY[9][2] = 0.f;
      dY[10][0] = SH_C3B * y * z; dY[10][1] = SH_C3B * x * z; dY[10][2] = SH_C3B * x * y;
      dY[11][0] = 2.f * SH_C3C * x * y; dY[11][1] = -SH_C3C * (4.f * zz - xx - 3.f * yy); dY[11][2] = -8.f * SH_C3C * y * z;
      dY[12][0] = -6.f * SH_C3D * x * z; dY[12][1] = -6.f * SH_C3D * y * z; dY[12][2] = 3.f * SH_C3D * (2.f * zz - xx - yy);
      dY[13][0] = -SH_C3C * (4.f * zz - 3.f * xx - yy); dY[13][1] = 2.f * SH_C3C * x * y; dY[13][2] = -8.f * SH_C3C * x * z;
      dY[14][0] = 2.f * SH_C3E * x * z; dY[14][1] = -2.f * SH_C3E * y * z; dY[14][2] = SH_C3E * (xx - yy);
      dY[15][0] = -3.f * SH_C3A * (xx - yy); dY[15][1] = 6.f * SH_C3A * x * y; dY[15][2] = 0.f;
    }
  }
}
