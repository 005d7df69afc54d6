// CPU oracle for the per-view training step of point-based (3D Gaussian) rendering.
//
// THIS IS TEST INFRASTRUCTURE.  It is the plain, slow, sequential-in-spirit statement of what the
// hot path computes; the product (the CUDA library) never calls it and shares no code, header,
// table or constant with it.  Only the tests, the smoke check and the benchmark's CPU-baseline leg
// may build or call it.
//
// What it follows.  The paper (Sec. 2.1) defines a training view as: render one camera, compute an
// image loss, update only the primitives that take part in that view; it defines the candidate
// scope G_i available before state observation, the conservative read/update scopes R_i^+, W_i^+
// (Sec. 2.1) and the hazard sets C_WAW^+, C_RAW^+, C_WAR^+ (Sec. 4.3, quality-first path).  The
// paper leaves the renderer itself to the 3D Gaussian Splatting pipeline it builds on (Sec. 1), so
// the renderer arithmetic below is the standard definition of that method, restated: EWA projection
// of an anisotropic 3D Gaussian to a 2D conic, 16x16 tile binning with keys (tile << 32 | depth
// bits), front-to-back alpha compositing with alpha clamp 0.99, skip below 1/255 and termination at
// transmittance 1e-4, its analytic backward pass, and Adam restricted to the touched rows.
//
// Precision.  Every function is templated on Real.  Real = float takes every integer decision
// (radius, tile rectangle, thresholds) in the precision the GPU uses; Real = double is used for the
// finite-difference pins.  All accumulations over many terms (pixel colour, per-primitive gradient
// sums, loss) are carried in double in both cases.
//
// Pins (tests/test_oracle_*.py): closed-form images of isotropic splats, transmittance products,
// partition of unity, SH orthonormality by quadrature, Sigma = s^2 I for isotropic scales, the EWA
// closed form J J^T s^2 + 0.3 I, brute-force binning and sorting, central finite differences of the
// double instantiation for every gradient word, textbook Adam via torch.optim.Adam, brute-force set
// intersection.  "Parity unpinned" remains for one thing only: agreement with the *trained* scenes
// and images of the paper's pipelines, which do not exist here.
#pragma once
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

namespace odin_oracle {

struct Config {
  double alpha_min = 1.0 / 255.0;  // contributions with alpha below this are skipped
  double alpha_max = 0.99;         // alpha clamp
  double t_min = 1e-4;             // stop before the splat that would push transmittance below this
  double dilation = 0.3;           // low-pass term added to the 2D covariance diagonal
  double radius_sigmas = 3.0;      // screen-space extent in standard deviations
  double jac_clamp = 1.3;          // guard on t_x/t_z, t_y/t_z inside the projection Jacobian
  int tile = 16;
  int binning = 0;                 // 0: rectangle of the radius; 1: additionally cut to the extent of alpha >= alpha_min;
                                   // 2: only the tiles of that rectangle which the region alpha >= alpha_min reaches
};

struct CameraD {
  int W, H;
  double fx, fy, cx, cy, znear, zfar;
  double w2c[12];  // row-major [R|t]
  double bg[3];
};

template <class Real>
struct Cam {
  int W, H, TX, TY;
  Real fx, fy, cx, cy, znear, zfar;
  Real R[9], t[3], bg[3], pos[3];
};

template <class Real>
Cam<Real> make_cam(const CameraD& c, int tile) {
  Cam<Real> k;
  k.W = c.W; k.H = c.H;
  k.TX = (c.W + tile - 1) / tile; k.TY = (c.H + tile - 1) / tile;
  k.fx = (Real)c.fx; k.fy = (Real)c.fy; k.cx = (Real)c.cx; k.cy = (Real)c.cy;
  k.znear = (Real)c.znear; k.zfar = (Real)c.zfar;
  for (int i = 0; i < 3; ++i) {
    for (int j = 0; j < 3; ++j) k.R[3 * i + j] = (Real)c.w2c[4 * i + j];
    k.t[i] = (Real)c.w2c[4 * i + 3];
    k.bg[i] = (Real)c.bg[i];
  }
  // camera centre in world coordinates: -R^T t
  for (int j = 0; j < 3; ++j) k.pos[j] = -(k.R[0 + j] * k.t[0] + k.R[3 + j] * k.t[1] + k.R[6 + j] * k.t[2]);
  return k;
}

// ---------------------------------------------------------------------------------------------
// Real spherical harmonics up to degree 3, evaluated as polynomials in the unit direction (x,y,z).
// Constants are computed from their closed forms sqrt(a / (b*pi)).
template <class Real>
struct SHConst {
  Real C0, C1, C2a, C2b, C2c, C3a, C3b, C3c, C3d, C3e;
  SHConst() {
    const double pi = 3.14159265358979323846;
    C0 = (Real)std::sqrt(1.0 / (4 * pi));   C1 = (Real)std::sqrt(3.0 / (4 * pi));
    C2a = (Real)std::sqrt(15.0 / (4 * pi)); C2b = (Real)std::sqrt(5.0 / (16 * pi));
    C2c = (Real)std::sqrt(15.0 / (16 * pi)); C3a = (Real)std::sqrt(35.0 / (32 * pi));
    C3b = (Real)std::sqrt(105.0 / (4 * pi)); C3c = (Real)std::sqrt(21.0 / (32 * pi));
    C3d = (Real)std::sqrt(7.0 / (16 * pi)); C3e = (Real)std::sqrt(105.0 / (16 * pi));
  }
};

template <class Real>
void sh_basis(int degree, Real x, Real y, Real z, Real* Y) {
  static const SHConst<Real> k;
  Y[0] = k.C0;
  if (degree < 1) return;
  Y[1] = -k.C1 * y; Y[2] = k.C1 * z; Y[3] = -k.C1 * x;
  if (degree < 2) return;
  Real xx = x * x, yy = y * y, zz = z * z;
  Y[4] = k.C2a * x * y; Y[5] = -k.C2a * y * z; Y[6] = k.C2b * (2 * zz - xx - yy);
  Y[7] = -k.C2a * x * z; Y[8] = k.C2c * (xx - yy);
  if (degree < 3) return;
  Y[9] = -k.C3a * y * (3 * xx - yy);
  Y[10] = k.C3b * x * y * z;
  Y[11] = -k.C3c * y * (4 * zz - xx - yy);
  Y[12] = k.C3d * z * (2 * zz - 3 * xx - 3 * yy);
  Y[13] = -k.C3c * x * (4 * zz - xx - yy);
  Y[14] = k.C3e * z * (xx - yy);
  Y[15] = -k.C3a * x * (xx - 3 * yy);
}

// Gradient of each basis polynomial with respect to (x,y,z), treated as free variables.
template <class Real>
void sh_basis_grad(int degree, Real x, Real y, Real z, Real (*dY)[3]) {
  static const SHConst<Real> k;
  dY[0][0] = dY[0][1] = dY[0][2] = 0;
  if (degree < 1) return;
  dY[1][0] = 0; dY[1][1] = -k.C1; dY[1][2] = 0;
  dY[2][0] = 0; dY[2][1] = 0; dY[2][2] = k.C1;
  dY[3][0] = -k.C1; dY[3][1] = 0; dY[3][2] = 0;
  if (degree < 2) return;
  Real xx = x * x, yy = y * y, zz = z * z;
  dY[4][0] = k.C2a * y; dY[4][1] = k.C2a * x; dY[4][2] = 0;
  dY[5][0] = 0; dY[5][1] = -k.C2a * z; dY[5][2] = -k.C2a * y;
  dY[6][0] = -2 * k.C2b * x; dY[6][1] = -2 * k.C2b * y; dY[6][2] = 4 * k.C2b * z;
  dY[7][0] = -k.C2a * z; dY[7][1] = 0; dY[7][2] = -k.C2a * x;
  dY[8][0] = 2 * k.C2c * x; dY[8][1] = -2 * k.C2c * y; dY[8][2] = 0;
  if (degree < 3) return;
  dY[9][0] = -k.C3a * 6 * x * y; dY[9][1] = -k.C3a * (3 * xx - 3 * yy); dY[9][2] = 0;
  dY[10][0] = k.C3b * y * z; dY[10][1] = k.C3b * x * z; dY[10][2] = k.C3b * x * y;
  dY[11][0] = k.C3c * 2 * x * y; dY[11][1] = -k.C3c * (4 * zz - xx - 3 * yy); dY[11][2] = -k.C3c * 8 * y * z;
  dY[12][0] = -k.C3d * 6 * x * z; dY[12][1] = -k.C3d * 6 * y * z; dY[12][2] = k.C3d * (6 * zz - 3 * xx - 3 * yy);
  dY[13][0] = -k.C3c * (4 * zz - 3 * xx - yy); dY[13][1] = k.C3c * 2 * x * y; dY[13][2] = -k.C3c * 8 * x * z;
  dY[14][0] = k.C3e * 2 * x * z; dY[14][1] = -k.C3e * 2 * y * z; dY[14][2] = k.C3e * (xx - yy);
  dY[15][0] = -k.C3a * (3 * xx - 3 * yy); dY[15][1] = k.C3a * 6 * x * y; dY[15][2] = 0;
}

// ---------------------------------------------------------------------------------------------
// Small geometry helpers shared by projection forward and backward.
template <class Real>
struct Geo {      // everything projection computes for one primitive on the way to the conic
  Real t[3];      // camera-space mean
  Real s[3];      // exp(log scale)
  Real qn[4];     // normalised quaternion (w,x,y,z)
  Real qlen;      // |q|
  Real Rm[9];     // rotation matrix of qn
  Real M[9];      // Rm * diag(s)
  Real Sig[9];    // M M^T
  Real J[6];      // 2x3 projection Jacobian (J[0]=J00, J[2]=J02, J[4]=J11, J[5]=J12)
  bool clampx, clampy;
  Real Lx, Ly;    // clamped ratio t~_x/t_z, t~_y/t_z
  Real Tm[6];     // J * R_c (2x3)
  Real a, b, c, det;
};

template <class Real>
void quat_to_rot(const Real* q, Real* R) {
  Real w = q[0], x = q[1], y = q[2], z = q[3];
  R[0] = 1 - 2 * (y * y + z * z); R[1] = 2 * (x * y - w * z); R[2] = 2 * (x * z + w * y);
  R[3] = 2 * (x * y + w * z); R[4] = 1 - 2 * (x * x + z * z); R[5] = 2 * (y * z - w * x);
  R[6] = 2 * (x * z - w * y); R[7] = 2 * (y * z + w * x); R[8] = 1 - 2 * (x * x + y * y);
}

// Covariance of the 3D Gaussian and its EWA projection.  Returns false if culled by depth.
template <class Real>
bool geometry(const Cam<Real>& cam, const Config& cfg, const Real* mu, const Real* ls, const Real* q, Geo<Real>& g) {
  for (int i = 0; i < 3; ++i)
    g.t[i] = cam.R[3 * i] * mu[0] + cam.R[3 * i + 1] * mu[1] + cam.R[3 * i + 2] * mu[2] + cam.t[i];
  if (!(g.t[2] > cam.znear) || !(g.t[2] < cam.zfar)) return false;
  for (int i = 0; i < 3; ++i) g.s[i] = std::exp(ls[i]);
  g.qlen = std::sqrt(q[0] * q[0] + q[1] * q[1] + q[2] * q[2] + q[3] * q[3]);
  for (int i = 0; i < 4; ++i) g.qn[i] = q[i] / g.qlen;
  quat_to_rot(g.qn, g.Rm);
  for (int i = 0; i < 3; ++i)
    for (int j = 0; j < 3; ++j) g.M[3 * i + j] = g.Rm[3 * i + j] * g.s[j];
  for (int i = 0; i < 3; ++i)
    for (int j = 0; j < 3; ++j)
      g.Sig[3 * i + j] = g.M[3 * i] * g.M[3 * j] + g.M[3 * i + 1] * g.M[3 * j + 1] + g.M[3 * i + 2] * g.M[3 * j + 2];
  Real tz = g.t[2];
  Real limx = (Real)cfg.jac_clamp * (Real)cam.W / (2 * cam.fx);
  Real limy = (Real)cfg.jac_clamp * (Real)cam.H / (2 * cam.fy);
  Real rx = g.t[0] / tz, ry = g.t[1] / tz;
  g.clampx = (rx < -limx) || (rx > limx);
  g.clampy = (ry < -limy) || (ry > limy);
  g.Lx = std::min(limx, std::max(-limx, rx));
  g.Ly = std::min(limy, std::max(-limy, ry));
  Real txc = g.Lx * tz, tyc = g.Ly * tz;
  g.J[0] = cam.fx / tz; g.J[1] = 0; g.J[2] = -cam.fx * txc / (tz * tz);
  g.J[3] = 0; g.J[4] = cam.fy / tz; g.J[5] = -cam.fy * tyc / (tz * tz);
  for (int i = 0; i < 2; ++i)
    for (int j = 0; j < 3; ++j)
      g.Tm[3 * i + j] = g.J[3 * i] * cam.R[j] + g.J[3 * i + 1] * cam.R[3 + j] + g.J[3 * i + 2] * cam.R[6 + j];
  // Sigma' = Tm Sigma Tm^T
  Real TS[6];
  for (int i = 0; i < 2; ++i)
    for (int j = 0; j < 3; ++j)
      TS[3 * i + j] = g.Tm[3 * i] * g.Sig[j] + g.Tm[3 * i + 1] * g.Sig[3 + j] + g.Tm[3 * i + 2] * g.Sig[6 + j];
  Real s00 = TS[0] * g.Tm[0] + TS[1] * g.Tm[1] + TS[2] * g.Tm[2];
  Real s01 = TS[0] * g.Tm[3] + TS[1] * g.Tm[4] + TS[2] * g.Tm[5];
  Real s11 = TS[3] * g.Tm[3] + TS[4] * g.Tm[4] + TS[5] * g.Tm[5];
  g.a = s00 + (Real)cfg.dilation; g.b = s01; g.c = s11 + (Real)cfg.dilation;
  g.det = g.a * g.c - g.b * g.b;
  return true;
}

// ---------------------------------------------------------------------------------------------
// Projection (preprocessing phase): cull, conic, radius, tile rectangle, colour, opacity.
// Outputs are dense over the N primitives; a culled primitive has tiles_touched = 0 and zeros.
// margin[p] = smallest relative distance of any integer/branch decision of p to its threshold
// (radius rounding, rectangle edges, depth planes, Jacobian clamp, colour clamp); parity tests use
// it to recognise primitives for which a last-bit difference may legitimately flip a decision.
template <class Real>
void project(int64_t n, int sh_degree, const Real* means, const Real* log_scales, const Real* quats,
             const Real* opacity_logit, const Real* sh, const CameraD& camd, const Config& cfg,
             Real* xy, Real* depth, Real* conic_o, Real* rgb, int32_t* radius, int32_t* rect,
             uint32_t* tiles_touched, uint8_t* clamp_flags, Real* margin) {
  const Cam<Real> cam = make_cam<Real>(camd, cfg.tile);
  const int K = (sh_degree + 1) * (sh_degree + 1);
  const Real tile = (Real)cfg.tile;
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < n; ++p) {
    xy[2 * p] = xy[2 * p + 1] = 0; depth[p] = 0;
    for (int i = 0; i < 4; ++i) { conic_o[4 * p + i] = 0; rect[4 * p + i] = 0; }
    for (int i = 0; i < 3; ++i) rgb[3 * p + i] = 0;
    radius[p] = 0; tiles_touched[p] = 0; clamp_flags[p] = 0; margin[p] = 1;
    Geo<Real> g;
    if (!geometry(cam, cfg, means + 3 * p, log_scales + 3 * p, quats + 4 * p, g)) {
      // depth-plane margin of a culled primitive
      Real tz = g.t[2];
      Real m = std::min(std::abs(tz - cam.znear) / cam.znear, std::abs(tz - cam.zfar) / cam.zfar);
      margin[p] = std::min<Real>(1, m);
      continue;
    }
    Real mg = std::min<Real>(1, std::min(std::abs(g.t[2] - cam.znear) / cam.znear, std::abs(g.t[2] - cam.zfar) / cam.zfar));
    if (!(g.det > 0)) continue;
    Real A = g.c / g.det, B = -g.b / g.det, C = g.a / g.det;
    Real mid = (g.a + g.c) / 2;
    Real lam = mid + std::sqrt(std::max<Real>((Real)0.1, mid * mid - g.det));
    Real rr = (Real)cfg.radius_sigmas * std::sqrt(lam);
    Real rad = std::ceil(rr);
    Real u = cam.fx * g.t[0] / g.t[2] + cam.cx;
    Real v = cam.fy * g.t[1] / g.t[2] + cam.cy;
    Real fx0 = std::floor((u - rad) / tile), fx1 = std::ceil((u + rad) / tile);
    Real fy0 = std::floor((v - rad) / tile), fy1 = std::ceil((v + rad) / tile);
    int x0 = (int)std::min<Real>((Real)cam.TX, std::max<Real>(0, fx0));
    int x1 = (int)std::min<Real>((Real)cam.TX, std::max<Real>(0, fx1));
    int y0 = (int)std::min<Real>((Real)cam.TY, std::max<Real>(0, fy0));
    int y1 = (int)std::min<Real>((Real)cam.TY, std::max<Real>(0, fy1));
    const Real opac = 1 / (1 + std::exp(-opacity_logit[p]));
    if (cfg.binning == 1) {
      // Optimised-pipeline variant (Sec. 5: pipelines with tighter kernels keep the same primitive-id namespace): the
      // rectangle is cut to the axis-aligned extent of the region where alpha = opac * exp(-q/2) can reach alpha_min,
      // q = d^T Sigma'^-1 d <= k = 2 ln(opac / alpha_min), whose half extents are sqrt(k Sigma'_xx), sqrt(k Sigma'_yy).
      // No pixel outside it passes the skip test, so images and gradients are those of the plain rectangle.  The
      // extent is widened by 1e-4 relative + 1e-3 pixels against rounding of the per-pixel test.
      const Real amin = (Real)cfg.alpha_min;
      mg = std::min(mg, std::abs(opac - amin) / amin);
      if (!(opac >= amin)) {
        x1 = x0;  // never reaches alpha_min anywhere
      } else {
        const Real k = 2 * std::log(opac / amin);
        const Real ex = std::sqrt(k * g.a) * (Real)1.0001 + (Real)1e-3, ey = std::sqrt(k * g.c) * (Real)1.0001 + (Real)1e-3;
        // tiles that hold a pixel centre (i + 0.5) within [u - ex, u + ex]
        const Real e[4] = {(u - ex - (Real)0.5) / tile, (u + ex - (Real)0.5) / tile, (v - ey - (Real)0.5) / tile,
                           (v + ey - (Real)0.5) / tile};
        const int tx0 = (int)std::min<Real>((Real)cam.TX, std::max<Real>(0, std::floor(e[0])));
        const int tx1 = (int)std::min<Real>((Real)cam.TX, std::max<Real>(0, std::floor(e[1]) + 1));
        const int ty0 = (int)std::min<Real>((Real)cam.TY, std::max<Real>(0, std::floor(e[2])));
        const int ty1 = (int)std::min<Real>((Real)cam.TY, std::max<Real>(0, std::floor(e[3]) + 1));
        x0 = std::max(x0, tx0); x1 = std::max(x0, std::min(x1, tx1));
        y0 = std::max(y0, ty0); y1 = std::max(y0, std::min(y1, ty1));
        for (int i = 0; i < 4; ++i) {
          Real f = e[i] - std::floor(e[i]);
          mg = std::min(mg, std::min(f, 1 - f) / std::max<Real>(1, std::abs(e[i])));
        }
      }
    }
    // decision margins: radius rounding and the four rectangle edges (in units of one tile)
    {
      Real fr = rr - std::floor(rr);
      mg = std::min(mg, std::min(fr, 1 - fr) / std::max<Real>(1, rr));
      const Real e[4] = {(u - rad) / tile, (u + rad) / tile, (v - rad) / tile, (v + rad) / tile};
      for (int i = 0; i < 4; ++i) {
        Real f = e[i] - std::floor(e[i]);
        mg = std::min(mg, std::min(f, 1 - f) / std::max<Real>(1, std::abs(e[i])));
      }
      Real limx = (Real)cfg.jac_clamp * (Real)cam.W / (2 * cam.fx), limy = (Real)cfg.jac_clamp * (Real)cam.H / (2 * cam.fy);
      mg = std::min(mg, std::abs(std::abs(g.t[0] / g.t[2]) - limx) / limx);
      mg = std::min(mg, std::abs(std::abs(g.t[1] / g.t[2]) - limy) / limy);
    }
    margin[p] = mg;
    uint32_t tt = (uint32_t)(x1 - x0) * (uint32_t)(y1 - y0);
    if (tt == 0) continue;
    tiles_touched[p] = tt;
    radius[p] = (int32_t)rad;
    rect[4 * p] = x0; rect[4 * p + 1] = y0; rect[4 * p + 2] = x1; rect[4 * p + 3] = y1;
    xy[2 * p] = u; xy[2 * p + 1] = v; depth[p] = g.t[2];
    conic_o[4 * p] = A; conic_o[4 * p + 1] = B; conic_o[4 * p + 2] = C;
    conic_o[4 * p + 3] = opac;
    // view-dependent colour
    Real d[3] = {means[3 * p] - cam.pos[0], means[3 * p + 1] - cam.pos[1], means[3 * p + 2] - cam.pos[2]};
    Real len = std::sqrt(d[0] * d[0] + d[1] * d[1] + d[2] * d[2]);
    for (int i = 0; i < 3; ++i) d[i] /= len;
    Real Y[16];
    sh_basis(sh_degree, d[0], d[1], d[2], Y);
    uint8_t flags = 0;
    for (int ch = 0; ch < 3; ++ch) {
      Real acc = 0;
      for (int k = 0; k < K; ++k) acc += Y[k] * sh[(p * K + k) * 3 + ch];
      acc += (Real)0.5;
      margin[p] = std::min(margin[p], std::abs(acc));
      if (acc < 0) { acc = 0; flags |= (uint8_t)(1u << ch); }
      rgb[3 * p + ch] = acc;
    }
    clamp_flags[p] = flags;
  }
}

// ---------------------------------------------------------------------------------------------
// Exact binning (binning = 2; an optimised-pipeline variant in the sense of Sec. 5: same primitive ids, same image).
// A primitive keeps a tile of its rectangle only if some pixel of the tile can pass the skip test, i.e. if the region
// alpha = opac * exp(-q/2) >= alpha_min, the ellipse q(d) = A dx^2 + 2 B dx dy + C dy^2 <= k with k = 2 ln(opac /
// alpha_min) around the centre, reaches the rectangle spanned by the tile's 16 x 16 pixel centres.  q is convex, so
// its minimum over that rectangle is 0 when the centre lies inside and otherwise sits on one of the four edges, at the
// clamped minimiser of the one-dimensional restriction.  The tile is kept iff  min q <= k (1 + 1e-4) + 1e-3 +
// 2e-6 * (largest value q takes on the rectangle's corners, by absolute terms): the slack covers the rounding of this
// evaluation and of the per-pixel test, so a dropped tile holds no pixel that passes.  The tiles a primitive keeps in
// one tile row are reported as the span from the first to the last tile of the row that passes (the set is an
// interval, the ellipse being convex).  *margin receives the relative distance of the decision to its threshold.
template <class Real>
bool tile_reached(Real u, Real v, Real A, Real B, Real C, Real opac, const Config& cfg, int tx, int ty, Real* margin) {
  const Real amin = (Real)cfg.alpha_min;
  if (!(opac >= amin)) { if (margin) *margin = std::abs(opac - amin) / amin; return false; }
  const Real k = 2 * std::log(opac / amin);
  const Real T = (Real)cfg.tile;
  const Real xl = (Real)tx * T + (Real)0.5 - u, xh = xl + (T - 1);
  const Real yl = (Real)ty * T + (Real)0.5 - v, yh = yl + (T - 1);
  auto q = [&](Real dx, Real dy) { return A * dx * dx + 2 * B * dx * dy + C * dy * dy; };
  auto clampv = [](Real x, Real lo, Real hi) { return std::min(std::max(x, lo), hi); };
  Real qmin;
  if (xl <= 0 && xh >= 0 && yl <= 0 && yh >= 0) {
    qmin = 0;
  } else {
    // edges x = xl, x = xh: minimise over dy; edges y = yl, y = yh: minimise over dx
    const Real q0 = q(xl, clampv(-B * xl / C, yl, yh)), q1 = q(xh, clampv(-B * xh / C, yl, yh));
    const Real q2 = q(clampv(-B * yl / A, xl, xh), yl), q3 = q(clampv(-B * yh / A, xl, xh), yh);
    qmin = std::min(std::min(q0, q1), std::min(q2, q3));
  }
  const Real mx = std::max(std::abs(xl), std::abs(xh)), my = std::max(std::abs(yl), std::abs(yh));
  const Real big = A * mx * mx + 2 * std::abs(B) * mx * my + C * my * my;
  const Real bound = k * (Real)1.0001 + (Real)1e-3 + (Real)2e-6 * big;
  if (margin) *margin = std::abs(qmin - bound) / std::max<Real>(bound, 1);
  return qmin <= bound;
}

// Spans of the kept tiles for every (primitive, tile row of its rectangle).  span_ptr [n + 1]: prefix of the
// rectangles' heights; span_x [2 * span_ptr[n]]: first and one-past-last kept tile of each tile row (equal = none).
// tiles_touched is replaced by the number of kept tiles; margin is lowered to the closest tile decision.
template <class Real>
void tile_spans(int64_t n, const Real* xy, const Real* conic_o, const int32_t* rect, const Config& cfg,
                const int64_t* span_ptr, int32_t* span_x, uint32_t* tiles_touched, Real* margin) {
#pragma omp parallel for schedule(dynamic, 256)
  for (int64_t p = 0; p < n; ++p) {
    if (tiles_touched[p] == 0) continue;
    const int x0 = rect[4 * p], y0 = rect[4 * p + 1], x1 = rect[4 * p + 2], y1 = rect[4 * p + 3];
    uint32_t kept = 0;
    Real mg = margin[p];
    for (int ty = y0; ty < y1; ++ty) {
      int first = x1, last = x0 - 1;
      for (int tx = x0; tx < x1; ++tx) {
        Real m1;
        if (tile_reached(xy[2 * p], xy[2 * p + 1], conic_o[4 * p], conic_o[4 * p + 1], conic_o[4 * p + 2],
                         conic_o[4 * p + 3], cfg, tx, ty, &m1)) {
          first = std::min(first, tx);
          last = std::max(last, tx);
        }
        mg = std::min(mg, m1);
      }
      int32_t* sp = span_x + 2 * (span_ptr[p] + (ty - y0));
      if (last >= first) { sp[0] = first; sp[1] = last + 1; kept += (uint32_t)(last + 1 - first); }
      else { sp[0] = x0; sp[1] = x0; }
    }
    tiles_touched[p] = kept;
    margin[p] = mg;
  }
}

// Binning and sort from spans: as bin_sort, the instances of a primitive being the kept tiles of its rectangle in
// row-major order.
inline void bin_sort_spans(int64_t n, const float* depth32, const int32_t* rect, const uint32_t* tiles_touched,
                           const int64_t* span_ptr, const int32_t* span_x, int TX, int TY, uint64_t* keys, uint32_t* vals,
                           uint32_t* ranges) {
  std::vector<std::pair<uint64_t, uint32_t>> kv;
  uint64_t M = 0;
  for (int64_t p = 0; p < n; ++p) M += tiles_touched[p];
  kv.reserve(M);
  for (int64_t p = 0; p < n; ++p) {
    if (tiles_touched[p] == 0) continue;
    uint32_t bits;
    std::memcpy(&bits, &depth32[p], 4);
    for (int ty = rect[4 * p + 1]; ty < rect[4 * p + 3]; ++ty) {
      const int32_t* sp = span_x + 2 * (span_ptr[p] + (ty - rect[4 * p + 1]));
      for (int tx = sp[0]; tx < sp[1]; ++tx) kv.emplace_back(((uint64_t)(uint32_t)(ty * TX + tx) << 32) | bits, (uint32_t)p);
    }
  }
  std::stable_sort(kv.begin(), kv.end(), [](const auto& a, const auto& b) { return a.first < b.first; });
  for (uint64_t i = 0; i < M; ++i) { keys[i] = kv[i].first; vals[i] = kv[i].second; }
  uint64_t pos = 0;
  for (int t = 0; t < TX * TY; ++t) {
    ranges[2 * t] = (uint32_t)pos;
    while (pos < M && (uint32_t)(keys[pos] >> 32) == (uint32_t)t) ++pos;
    ranges[2 * t + 1] = (uint32_t)pos;
  }
}

// ---------------------------------------------------------------------------------------------
// Touched set (Sec. 2.1: the candidate scope G_i = R_i^+ = W_i^+ of the view): every primitive
// that projects onto at least one tile.  Bit (p & 31) of word (p >> 5); ascending index list.
inline uint32_t touched_set(int64_t n, const uint32_t* tiles_touched, uint32_t* mask, uint32_t* idx) {
  const int64_t words = (n + 31) / 32;
  for (int64_t w = 0; w < words; ++w) mask[w] = 0;
  uint32_t V = 0;
  for (int64_t p = 0; p < n; ++p)
    if (tiles_touched[p] > 0) {
      mask[p >> 5] |= 1u << (p & 31);
      idx[V++] = (uint32_t)p;
    }
  return V;
}

// ---------------------------------------------------------------------------------------------
// Binning and sort.  One (key, value) per (tile, primitive) pair: key = tile_id << 32 | bits of the
// float32 depth, value = primitive index.  Stable sort by key; equal keys keep ascending primitive
// order.  ranges[t] = [first, one past last) position whose key names tile t (empty: first == last).
inline uint64_t count_instances(int64_t n, const uint32_t* tiles_touched) {
  uint64_t M = 0;
  for (int64_t p = 0; p < n; ++p) M += tiles_touched[p];
  return M;
}

inline void bin_sort(int64_t n, const float* depth32, const int32_t* rect, const uint32_t* tiles_touched, int TX, int TY,
                     uint64_t* keys, uint32_t* vals, uint32_t* ranges) {
  std::vector<std::pair<uint64_t, uint32_t>> kv;
  kv.reserve(count_instances(n, tiles_touched));
  for (int64_t p = 0; p < n; ++p) {
    if (tiles_touched[p] == 0) continue;
    uint32_t bits;
    std::memcpy(&bits, &depth32[p], 4);
    for (int ty = rect[4 * p + 1]; ty < rect[4 * p + 3]; ++ty)
      for (int tx = rect[4 * p]; tx < rect[4 * p + 2]; ++tx)
        kv.emplace_back(((uint64_t)(uint32_t)(ty * TX + tx) << 32) | bits, (uint32_t)p);
  }
  std::stable_sort(kv.begin(), kv.end(), [](const auto& a, const auto& b) { return a.first < b.first; });
  const uint64_t M = kv.size();
  for (uint64_t i = 0; i < M; ++i) { keys[i] = kv[i].first; vals[i] = kv[i].second; }
  uint64_t pos = 0;
  for (int t = 0; t < TX * TY; ++t) {
    ranges[2 * t] = (uint32_t)pos;
    while (pos < M && (uint32_t)(keys[pos] >> 32) == (uint32_t)t) ++pos;
    ranges[2 * t + 1] = (uint32_t)pos;
  }
}

// ---------------------------------------------------------------------------------------------
// Forward compositing (rendering phase).  Per pixel, front to back over the tile's sorted list.
// Counters (optional, may be null): [0] list entries traversed summed over tiles (an entry counts
// while any pixel of the tile is still live), [1] pixel-splat pairs evaluated, [2] pairs contributing.
template <class Real>
void render_fwd(const Real* xy, const Real* conic_o, const Real* rgb, const uint32_t* vals, const uint32_t* ranges,
                const CameraD& camd, const Config& cfg, Real* out_rgb, Real* final_T, uint32_t* n_contrib,
                Real* pix_margin, uint64_t* counters) {
  const Cam<Real> cam = make_cam<Real>(camd, cfg.tile);
  const int W = cam.W, H = cam.H;
  const Real amin = (Real)cfg.alpha_min, amax = (Real)cfg.alpha_max, tmin = (Real)cfg.t_min;
  uint64_t c_trav = 0, c_pairs = 0, c_contrib = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : c_trav, c_pairs, c_contrib)
  for (int t = 0; t < cam.TX * cam.TY; ++t) {
    const int tx = t % cam.TX, ty = t / cam.TX;
    const uint32_t start = ranges[2 * t], end = ranges[2 * t + 1];
    uint32_t tile_max_trav = 0;
    for (int j = ty * cfg.tile; j < std::min(H, (ty + 1) * cfg.tile); ++j)
      for (int i = tx * cfg.tile; i < std::min(W, (tx + 1) * cfg.tile); ++i) {
        const Real px = (Real)i + (Real)0.5, py = (Real)j + (Real)0.5;
        Real T = 1;
        double C[3] = {0, 0, 0};
        uint32_t last = 0, trav = 0;
        Real mg = 1;
        for (uint32_t k = start; k < end; ++k) {
          ++trav;
          const uint32_t p = vals[k];
          const Real dx = xy[2 * p] - px, dy = xy[2 * p + 1] - py;
          const Real A = conic_o[4 * p], B = conic_o[4 * p + 1], Cc = conic_o[4 * p + 2], o = conic_o[4 * p + 3];
          const Real q1 = A * dx * dx, q2 = Cc * dy * dy, q3 = B * dx * dy;
          const Real power = -(Real)0.5 * (q1 + q2) - q3;
          ++c_pairs;
          {  // how close the sign test is, relative to the size of the cancelling terms
            Real sc = (Real)0.5 * (std::abs(q1) + std::abs(q2)) + std::abs(q3);
            if (sc > 0) mg = std::min(mg, std::abs(power) / sc + ((dx == 0 && dy == 0) ? 1 : 0));
          }
          if (power > 0) continue;
          const Real G = std::exp(power);
          const Real og = o * G;
          const Real alpha = std::min(amax, og);
          mg = std::min(mg, std::abs(alpha - amin) / amin);
          if (alpha < amin) continue;
          mg = std::min(mg, std::abs(og - amax) / amax);
          const Real Tn = T * (1 - alpha);
          mg = std::min(mg, std::abs(Tn - tmin) / tmin);
          if (Tn < tmin) break;
          for (int ch = 0; ch < 3; ++ch) C[ch] += (double)(rgb[3 * p + ch] * alpha * T);
          T = Tn;
          last = (k - start) + 1;
          ++c_contrib;
        }
        tile_max_trav = std::max(tile_max_trav, trav);
        for (int ch = 0; ch < 3; ++ch) out_rgb[((size_t)ch * H + j) * W + i] = (Real)(C[ch] + (double)(T * cam.bg[ch]));
        final_T[(size_t)j * W + i] = T;
        n_contrib[(size_t)j * W + i] = last;
        if (pix_margin) pix_margin[(size_t)j * W + i] = mg;
      }
    c_trav += tile_max_trav;
  }
  if (counters) { counters[0] = c_trav; counters[1] = c_pairs; counters[2] = c_contrib; }
}

// ---------------------------------------------------------------------------------------------
// Image loss (Sec. 2.1: "computes an image loss"): mean absolute error over 3*H*W values and its
// gradient sign(out - target) / (3HW), sign(0) = 0.
template <class Real>
double l1_loss(int64_t count, const Real* out, const Real* target, Real* dL_dout) {
  double acc = 0;
  const Real inv = (Real)(1.0 / (double)count);
  for (int64_t i = 0; i < count; ++i) {
    const Real d = out[i] - target[i];
    acc += std::abs((double)d);
    dL_dout[i] = d > 0 ? inv : (d < 0 ? -inv : (Real)0);
  }
  return acc / (double)count;
}

// ---------------------------------------------------------------------------------------------
// Backward of the compositing.  For every pixel the contributing splats are replayed front to
// back (same skip tests; the list stops at n_contrib), then visited in reverse with the suffix sum
// S_k = sum_{j>k} c_j alpha_j T_j + T_final * bg.  Output: dense [N,9] double gradient sums with
// columns (u, v, conicA, conicB, conicC, opacity, r, g, b).  g2d_abs (optional, same shape) receives the sum of the
// absolute values of the same per-pixel terms: the size against which a cancelled sum has to be judged.
template <class Real>
void render_bwd_blend(const Real* xy, const Real* conic_o, const Real* rgb, const uint32_t* vals, const uint32_t* ranges,
                      const CameraD& camd, const Config& cfg, const Real* final_T, const uint32_t* n_contrib,
                      const Real* dL_dout, int64_t n, double* g2d, double* g2d_abs) {
  const Cam<Real> cam = make_cam<Real>(camd, cfg.tile);
  const int W = cam.W, H = cam.H;
  const Real amin = (Real)cfg.alpha_min, amax = (Real)cfg.alpha_max;
  for (int64_t i = 0; i < 9 * n; ++i) g2d[i] = 0;
  if (g2d_abs)
    for (int64_t i = 0; i < 9 * n; ++i) g2d_abs[i] = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int t = 0; t < cam.TX * cam.TY; ++t) {
    const int tx = t % cam.TX, ty = t / cam.TX;
    const uint32_t start = ranges[2 * t];
    struct Hit { uint32_t p; Real alpha, T, G, dx, dy; bool clamped; };
    std::vector<Hit> hits;
    for (int j = ty * cfg.tile; j < std::min(H, (ty + 1) * cfg.tile); ++j)
      for (int i = tx * cfg.tile; i < std::min(W, (tx + 1) * cfg.tile); ++i) {
        const size_t pix = (size_t)j * W + i;
        const Real px = (Real)i + (Real)0.5, py = (Real)j + (Real)0.5;
        hits.clear();
        Real T = 1;
        for (uint32_t k = start; k < start + n_contrib[pix]; ++k) {
          const uint32_t p = vals[k];
          const Real dx = xy[2 * p] - px, dy = xy[2 * p + 1] - py;
          const Real A = conic_o[4 * p], B = conic_o[4 * p + 1], Cc = conic_o[4 * p + 2], o = conic_o[4 * p + 3];
          const Real power = -(Real)0.5 * (A * dx * dx + Cc * dy * dy) - B * dx * dy;
          if (power > 0) continue;
          const Real G = std::exp(power);
          const Real og = o * G;
          const Real alpha = std::min(amax, og);
          if (alpha < amin) continue;
          hits.push_back({p, alpha, T, G, dx, dy, og > amax});
          T = T * (1 - alpha);
        }
        const Real g[3] = {dL_dout[((size_t)0 * H + j) * W + i], dL_dout[((size_t)1 * H + j) * W + i],
                           dL_dout[((size_t)2 * H + j) * W + i]};
        double S[3];
        for (int ch = 0; ch < 3; ++ch) S[ch] = (double)final_T[pix] * (double)cam.bg[ch];
        for (size_t h = hits.size(); h-- > 0;) {
          const Hit& e = hits[h];
          const uint32_t p = e.p;
          double dL_dalpha = 0;
          for (int ch = 0; ch < 3; ++ch) {
            const double c = (double)rgb[3 * p + ch];
            dL_dalpha += (c * (double)e.T - S[ch] / (1.0 - (double)e.alpha)) * (double)g[ch];
            const double dc = (double)e.alpha * (double)e.T * (double)g[ch];
#pragma omp atomic
            g2d[9 * (size_t)p + 6 + ch] += dc;
            if (g2d_abs) {
#pragma omp atomic
              g2d_abs[9 * (size_t)p + 6 + ch] += std::abs(dc);
            }
            S[ch] += c * (double)e.alpha * (double)e.T;
          }
          if (e.clamped) continue;  // alpha = 0.99 is constant there
          const double o = (double)conic_o[4 * p + 3], A = (double)conic_o[4 * p], B = (double)conic_o[4 * p + 1],
                       Cc = (double)conic_o[4 * p + 2];
          const double G = (double)e.G, dx = (double)e.dx, dy = (double)e.dy;
          const double dL_dG = o * dL_dalpha;
          const double gp = G * dL_dG;  // dL/dpower
          const double add[6] = {(-A * dx - B * dy) * gp, (-Cc * dy - B * dx) * gp, -0.5 * dx * dx * gp,
                                 -dx * dy * gp,           -0.5 * dy * dy * gp,      G * dL_dalpha};
          for (int w = 0; w < 6; ++w) {
#pragma omp atomic
            g2d[9 * (size_t)p + w] += add[w];
            if (g2d_abs) {
#pragma omp atomic
              g2d_abs[9 * (size_t)p + w] += std::abs(add[w]);
            }
          }
        }
      }
  }
}

// ---------------------------------------------------------------------------------------------
// Realized active set C_i (Sec. 2.1, Table 1: the primitives that actually take part in the view's
// computation, known only after it has executed; Theta >= G_i >= C_i).  Reading: a primitive is
// realized-active when it is blended into at least one pixel, i.e. it passes the skip tests inside
// that pixel's n_contrib prefix - exactly the (pixel, primitive) pairs the backward differentiates.
// active [n] receives 0 / 1.
template <class Real>
void realized_active(const Real* xy, const Real* conic_o, const uint32_t* vals, const uint32_t* ranges,
                     const CameraD& camd, const Config& cfg, const uint32_t* n_contrib, int64_t n, uint8_t* active) {
  const Cam<Real> cam = make_cam<Real>(camd, cfg.tile);
  const int W = cam.W, H = cam.H;
  const Real amin = (Real)cfg.alpha_min, amax = (Real)cfg.alpha_max;
  for (int64_t i = 0; i < n; ++i) active[i] = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (int t = 0; t < cam.TX * cam.TY; ++t) {
    const int tx = t % cam.TX, ty = t / cam.TX;
    const uint32_t start = ranges[2 * t];
    for (int j = ty * cfg.tile; j < std::min(H, (ty + 1) * cfg.tile); ++j)
      for (int i = tx * cfg.tile; i < std::min(W, (tx + 1) * cfg.tile); ++i) {
        const size_t pix = (size_t)j * W + i;
        const Real px = (Real)i + (Real)0.5, py = (Real)j + (Real)0.5;
        for (uint32_t k = start; k < start + n_contrib[pix]; ++k) {
          const uint32_t p = vals[k];
          const Real dx = xy[2 * p] - px, dy = xy[2 * p + 1] - py;
          const Real A = conic_o[4 * p], B = conic_o[4 * p + 1], Cc = conic_o[4 * p + 2], o = conic_o[4 * p + 3];
          const Real power = -(Real)0.5 * (A * dx * dx + Cc * dy * dy) - B * dx * dy;
          if (power > 0) continue;
          const Real alpha = std::min(amax, o * std::exp(power));
          if (alpha < amin) continue;
#pragma omp atomic write
          active[p] = 1;
        }
      }
  }
}

// ---------------------------------------------------------------------------------------------
// Backward of the projection, per touched primitive (row r <-> primitive idx[r]).  Branch decisions
// (Jacobian clamp, colour clamp) are frozen at their forward values.  Output rows [V, F] with
// F = 11 + 3K ordered mean(3), log_scale(3), quat(4), opacity logit(1), sh[K][3].
template <class Real>
void render_bwd_project(int sh_degree, const Real* means, const Real* log_scales, const Real* quats,
                        const Real* opacity_logit, const Real* sh, const CameraD& camd, const Config& cfg,
                        const uint32_t* idx, uint32_t V, const double* g2d, const uint8_t* clamp_flags, Real* rows) {
  const Cam<Real> cam = make_cam<Real>(camd, cfg.tile);
  const int K = (sh_degree + 1) * (sh_degree + 1);
  const int F = 11 + 3 * K;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < (int64_t)V; ++r) {
    const size_t p = idx[r];
    Real* row = rows + (size_t)r * F;
    for (int i = 0; i < F; ++i) row[i] = 0;
    Geo<Real> g;
    if (!geometry(cam, cfg, means + 3 * p, log_scales + 3 * p, quats + 4 * p, g)) continue;
    const Real gu = (Real)g2d[9 * p], gv = (Real)g2d[9 * p + 1];
    const Real gA = (Real)g2d[9 * p + 2], gB = (Real)g2d[9 * p + 3], gC = (Real)g2d[9 * p + 4];
    const Real go = (Real)g2d[9 * p + 5];
    const Real grgb[3] = {(Real)g2d[9 * p + 6], (Real)g2d[9 * p + 7], (Real)g2d[9 * p + 8]};
    // conic -> 2D covariance entries
    const Real a = g.a, b = g.b, c = g.c, D = g.det * g.det;
    const Real ga = (-c * c * gA + b * c * gB - b * b * gC) / D;
    const Real gb = (2 * b * c * gA - (a * c + b * b) * gB + 2 * a * b * gC) / D;
    const Real gc = (-b * b * gA + a * b * gB - a * a * gC) / D;
    const Real Gs[4] = {ga, gb / 2, gb / 2, gc};
    // dL/dSigma = Tm^T Gs Tm ; dL/dTm = 2 Gs Tm Sigma
    Real GT[6];  // Gs * Tm (2x3)
    for (int i = 0; i < 2; ++i)
      for (int j = 0; j < 3; ++j) GT[3 * i + j] = Gs[2 * i] * g.Tm[j] + Gs[2 * i + 1] * g.Tm[3 + j];
    Real gSig[9];
    for (int i = 0; i < 3; ++i)
      for (int j = 0; j < 3; ++j) gSig[3 * i + j] = g.Tm[i] * GT[j] + g.Tm[3 + i] * GT[3 + j];
    Real gTm[6];
    for (int i = 0; i < 2; ++i)
      for (int j = 0; j < 3; ++j)
        gTm[3 * i + j] = 2 * (GT[3 * i] * g.Sig[j] + GT[3 * i + 1] * g.Sig[3 + j] + GT[3 * i + 2] * g.Sig[6 + j]);
    // Tm = J R_c  ->  dL/dJ = dL/dTm R_c^T
    Real gJ[6];
    for (int i = 0; i < 2; ++i)
      for (int j = 0; j < 3; ++j)
        gJ[3 * i + j] = gTm[3 * i] * cam.R[3 * j] + gTm[3 * i + 1] * cam.R[3 * j + 1] + gTm[3 * i + 2] * cam.R[3 * j + 2];
    const Real tx = g.t[0], ty = g.t[1], tz = g.t[2];
    Real gt[3] = {0, 0, 0};
    // J00 = fx/tz, J11 = fy/tz
    gt[2] += -gJ[0] * cam.fx / (tz * tz) - gJ[4] * cam.fy / (tz * tz);
    // J02 = -fx * (Lx tz) / tz^2 with Lx = tx/tz (free) or +-lim (frozen)
    if (g.clampx) gt[2] += gJ[2] * cam.fx * g.Lx / (tz * tz);
    else { gt[0] += -gJ[2] * cam.fx / (tz * tz); gt[2] += gJ[2] * 2 * cam.fx * tx / (tz * tz * tz); }
    if (g.clampy) gt[2] += gJ[5] * cam.fy * g.Ly / (tz * tz);
    else { gt[1] += -gJ[5] * cam.fy / (tz * tz); gt[2] += gJ[5] * 2 * cam.fy * ty / (tz * tz * tz); }
    // pixel centre u = fx tx/tz + cx, v likewise
    gt[0] += gu * cam.fx / tz; gt[2] += -gu * cam.fx * tx / (tz * tz);
    gt[1] += gv * cam.fy / tz; gt[2] += -gv * cam.fy * ty / (tz * tz);
    Real gmu[3];
    for (int j = 0; j < 3; ++j) gmu[j] = cam.R[j] * gt[0] + cam.R[3 + j] * gt[1] + cam.R[6 + j] * gt[2];
    // Sigma = M M^T -> dL/dM = 2 gSig M
    Real gM[9];
    for (int i = 0; i < 3; ++i)
      for (int j = 0; j < 3; ++j)
        gM[3 * i + j] = 2 * (gSig[3 * i] * g.M[j] + gSig[3 * i + 1] * g.M[3 + j] + gSig[3 * i + 2] * g.M[6 + j]);
    Real gR[9];
    for (int j = 0; j < 3; ++j) {
      Real gs = 0;
      for (int i = 0; i < 3; ++i) { gs += g.Rm[3 * i + j] * gM[3 * i + j]; gR[3 * i + j] = gM[3 * i + j] * g.s[j]; }
      row[3 + j] = g.s[j] * gs;
    }
    {
      const Real w = g.qn[0], x = g.qn[1], y = g.qn[2], z = g.qn[3];
      Real gq[4];
      gq[0] = 2 * (-z * gR[1] + y * gR[2] + z * gR[3] - x * gR[5] - y * gR[6] + x * gR[7]);
      gq[1] = 2 * (y * gR[1] + z * gR[2] + y * gR[3] - 2 * x * gR[4] - w * gR[5] + z * gR[6] + w * gR[7] - 2 * x * gR[8]);
      gq[2] = 2 * (-2 * y * gR[0] + x * gR[1] + w * gR[2] + x * gR[3] + z * gR[5] - w * gR[6] + z * gR[7] - 2 * y * gR[8]);
      gq[3] = 2 * (-2 * z * gR[0] - w * gR[1] + x * gR[2] + w * gR[3] - 2 * z * gR[4] + y * gR[5] + x * gR[6] + y * gR[7]);
      Real dot = 0;
      for (int i = 0; i < 4; ++i) dot += g.qn[i] * gq[i];
      for (int i = 0; i < 4; ++i) row[6 + i] = (gq[i] - g.qn[i] * dot) / g.qlen;
    }
    // opacity = sigmoid(logit)
    {
      const Real o = 1 / (1 + std::exp(-opacity_logit[p]));
      row[10] = o * (1 - o) * go;
    }
    // colour: rgb_ch = max(0, 0.5 + sum_k Y_k(d) sh[k][ch])
    {
      Real dv[3] = {means[3 * p] - cam.pos[0], means[3 * p + 1] - cam.pos[1], means[3 * p + 2] - cam.pos[2]};
      const Real len = std::sqrt(dv[0] * dv[0] + dv[1] * dv[1] + dv[2] * dv[2]);
      Real d[3] = {dv[0] / len, dv[1] / len, dv[2] / len};
      Real Y[16], dY[16][3];
      sh_basis(sh_degree, d[0], d[1], d[2], Y);
      sh_basis_grad(sh_degree, d[0], d[1], d[2], dY);
      Real gd[3] = {0, 0, 0};
      for (int ch = 0; ch < 3; ++ch) {
        if (clamp_flags[p] & (1u << ch)) continue;
        for (int k = 0; k < K; ++k) {
          row[11 + 3 * k + ch] = Y[k] * grgb[ch];
          const Real w = sh[(p * K + k) * 3 + ch] * grgb[ch];
          for (int i = 0; i < 3; ++i) gd[i] += dY[k][i] * w;
        }
      }
      Real dot = d[0] * gd[0] + d[1] * gd[1] + d[2] * gd[2];
      for (int i = 0; i < 3; ++i) gmu[i] += (gd[i] - d[i] * dot) / len;
    }
    for (int i = 0; i < 3; ++i) row[i] = gmu[i];
  }
}

// ---------------------------------------------------------------------------------------------
// Sparse Adam (update phase; Sec. 2.1: only the primitives that take part in the view change).
// Global 1-based step t for the bias correction; rows not listed in idx are not read or written.
// lr: mean, scale, quat, opacity, sh_dc, sh_rest.  grads are compact rows [V, F].
template <class Real>
void sparse_adam(int sh_degree, Real* means, Real* log_scales, Real* quats, Real* opacity_logit, Real* sh,
                 Real* m_means, Real* m_ls, Real* m_q, Real* m_o, Real* m_sh,
                 Real* v_means, Real* v_ls, Real* v_q, Real* v_o, Real* v_sh,
                 const Real* rows, const uint32_t* idx, uint32_t V, const Real* lr, Real beta1, Real beta2, Real eps,
                 uint32_t step) {
  const int K = (sh_degree + 1) * (sh_degree + 1);
  const int F = 11 + 3 * K;
  const Real bc1 = 1 - (Real)std::pow((double)beta1, (double)step);
  const Real bc2s = (Real)std::sqrt(1 - std::pow((double)beta2, (double)step));
  auto upd = [&](Real& th, Real& m, Real& v, Real g, Real lrg) {
    m = beta1 * m + (1 - beta1) * g;
    v = beta2 * v + (1 - beta2) * g * g;
    th = th - (lrg / bc1) * m / (std::sqrt(v) / bc2s + eps);
  };
  for (uint32_t r = 0; r < V; ++r) {
    const size_t p = idx[r];
    const Real* g = rows + (size_t)r * F;
    for (int i = 0; i < 3; ++i) upd(means[3 * p + i], m_means[3 * p + i], v_means[3 * p + i], g[i], lr[0]);
    for (int i = 0; i < 3; ++i) upd(log_scales[3 * p + i], m_ls[3 * p + i], v_ls[3 * p + i], g[3 + i], lr[1]);
    for (int i = 0; i < 4; ++i) upd(quats[4 * p + i], m_q[4 * p + i], v_q[4 * p + i], g[6 + i], lr[2]);
    upd(opacity_logit[p], m_o[p], v_o[p], g[10], lr[3]);
    for (int k = 0; k < K; ++k)
      for (int ch = 0; ch < 3; ++ch) {
        const size_t e = (p * K + k) * 3 + ch;
        upd(sh[e], m_sh[e], v_sh[e], g[11 + 3 * k + ch], k == 0 ? lr[4] : lr[5]);
      }
  }
}

// ---------------------------------------------------------------------------------------------
// Conflict count (Sec. 4.3): |W^+(A) ∩ W^+(B)| = size of C_WAW^+; with R^+ = W^+ the RAW and WAR
// sets are empty.  Computed as a plain merge of the two ascending index lists.
inline uint64_t conflict_count(const uint32_t* idx_a, uint32_t na, const uint32_t* idx_b, uint32_t nb) {
  uint64_t c = 0;
  uint32_t i = 0, j = 0;
  while (i < na && j < nb) {
    if (idx_a[i] < idx_b[j]) ++i;
    else if (idx_b[j] < idx_a[i]) ++j;
    else { ++c; ++i; ++j; }
  }
  return c;
}

}  // namespace odin_oracle
