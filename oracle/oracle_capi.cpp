// C entry points of the CPU oracle (test infrastructure; see odin_oracle.hpp).
// Suffix _f32 / _f64 selects the precision of the per-element arithmetic.
#include <omp.h>

#include "odin_oracle.hpp"

using namespace odin_oracle;

namespace {
CameraD cam_from(const double* c) {
  CameraD k;
  k.W = (int)c[0]; k.H = (int)c[1];
  k.fx = c[2]; k.fy = c[3]; k.cx = c[4]; k.cy = c[5]; k.znear = c[6]; k.zfar = c[7];
  for (int i = 0; i < 12; ++i) k.w2c[i] = c[8 + i];
  for (int i = 0; i < 3; ++i) k.bg[i] = c[20 + i];
  return k;
}
Config cfg_from(const double* c) {
  Config k;
  if (c) {
    k.alpha_min = c[0]; k.alpha_max = c[1]; k.t_min = c[2]; k.dilation = c[3];
    k.radius_sigmas = c[4]; k.jac_clamp = c[5]; k.tile = (int)c[6]; k.binning = (int)c[7];
  }
  return k;
}
}  // namespace

#define ORACLE_DEFINE(SUF, Real)                                                                                       \
  extern "C" void oracle_project_##SUF(int64_t n, int sh_degree, const Real* means, const Real* log_scales,           \
                                       const Real* quats, const Real* opacity_logit, const Real* sh,                   \
                                       const double* cam, const double* cfg, Real* xy, Real* depth, Real* conic_o,     \
                                       Real* rgb, int32_t* radius, int32_t* rect, uint32_t* tiles_touched,             \
                                       uint8_t* clamp_flags, Real* margin) {                                           \
    project<Real>(n, sh_degree, means, log_scales, quats, opacity_logit, sh, cam_from(cam), cfg_from(cfg), xy, depth,  \
                  conic_o, rgb, radius, rect, tiles_touched, clamp_flags, margin);                                     \
  }                                                                                                                    \
  extern "C" void oracle_render_fwd_##SUF(const Real* xy, const Real* conic_o, const Real* rgb, const uint32_t* vals, \
                                          const uint32_t* ranges, const double* cam, const double* cfg, Real* out_rgb, \
                                          Real* final_T, uint32_t* n_contrib, Real* pix_margin, uint64_t* counters) {  \
    render_fwd<Real>(xy, conic_o, rgb, vals, ranges, cam_from(cam), cfg_from(cfg), out_rgb, final_T, n_contrib,        \
                     pix_margin, counters);                                                                            \
  }                                                                                                                    \
  extern "C" double oracle_l1_loss_##SUF(int64_t count, const Real* out, const Real* target, Real* dL_dout) {         \
    return l1_loss<Real>(count, out, target, dL_dout);                                                                 \
  }                                                                                                                    \
  extern "C" void oracle_render_bwd_blend_##SUF(const Real* xy, const Real* conic_o, const Real* rgb,                 \
                                                const uint32_t* vals, const uint32_t* ranges, const double* cam,       \
                                                const double* cfg, const Real* final_T, const uint32_t* n_contrib,     \
                                                const Real* dL_dout, int64_t n, double* g2d,           \
                                                double* g2d_abs) {                                                     \
    render_bwd_blend<Real>(xy, conic_o, rgb, vals, ranges, cam_from(cam), cfg_from(cfg), final_T, n_contrib, dL_dout,  \
                           n, g2d, g2d_abs);                                                                           \
  }                                                                                                                    \
  extern "C" void oracle_realized_active_##SUF(const Real* xy, const Real* conic_o, const uint32_t* vals,              \
                                               const uint32_t* ranges, const double* cam, const double* cfg,           \
                                               const uint32_t* n_contrib, int64_t n, uint8_t* active) {                \
    realized_active<Real>(xy, conic_o, vals, ranges, cam_from(cam), cfg_from(cfg), n_contrib, n, active);              \
  }                                                                                                                    \
  extern "C" void oracle_render_bwd_project_##SUF(int sh_degree, const Real* means, const Real* log_scales,           \
                                                  const Real* quats, const Real* opacity_logit, const Real* sh,        \
                                                  const double* cam, const double* cfg, const uint32_t* idx,           \
                                                  uint32_t V, const double* g2d, const uint8_t* clamp_flags,           \
                                                  Real* rows) {                                                        \
    render_bwd_project<Real>(sh_degree, means, log_scales, quats, opacity_logit, sh, cam_from(cam), cfg_from(cfg),     \
                             idx, V, g2d, clamp_flags, rows);                                                          \
  }                                                                                                                    \
  extern "C" void oracle_sparse_adam_##SUF(int sh_degree, Real* means, Real* log_scales, Real* quats,                 \
                                           Real* opacity_logit, Real* sh, Real* m_means, Real* m_ls, Real* m_q,        \
                                           Real* m_o, Real* m_sh, Real* v_means, Real* v_ls, Real* v_q, Real* v_o,     \
                                           Real* v_sh, const Real* rows, const uint32_t* idx, uint32_t V,              \
                                           const Real* lr, double beta1, double beta2, double eps, uint32_t step) {    \
    sparse_adam<Real>(sh_degree, means, log_scales, quats, opacity_logit, sh, m_means, m_ls, m_q, m_o, m_sh, v_means,  \
                      v_ls, v_q, v_o, v_sh, rows, idx, V, lr, (Real)beta1, (Real)beta2, (Real)eps, step);              \
  }                                                                                                                    \
  extern "C" void oracle_sh_basis_##SUF(int degree, Real x, Real y, Real z, Real* Y) {                                \
    sh_basis<Real>(degree, x, y, z, Y);                                                                                \
  }                                                                                                                    \
  extern "C" void oracle_tile_spans_##SUF(int64_t n, const Real* xy, const Real* conic_o, const int32_t* rect,        \
                                          const double* cfg, const int64_t* span_ptr, int32_t* span_x,                 \
                                          uint32_t* tiles_touched, Real* margin) {                                     \
    tile_spans<Real>(n, xy, conic_o, rect, cfg_from(cfg), span_ptr, span_x, tiles_touched, margin);                    \
  }                                                                                                                    \
  extern "C" int oracle_tile_reached_##SUF(Real u, Real v, Real A, Real B, Real C, Real opac, const double* cfg,      \
                                           int tx, int ty) {                                                           \
    return tile_reached<Real>(u, v, A, B, C, opac, cfg_from(cfg), tx, ty, (Real*)nullptr) ? 1 : 0;                     \
  }

ORACLE_DEFINE(f32, float)
ORACLE_DEFINE(f64, double)

extern "C" uint32_t oracle_touched_set(int64_t n, const uint32_t* tiles_touched, uint32_t* mask, uint32_t* idx) {
  return touched_set(n, tiles_touched, mask, idx);
}
extern "C" uint64_t oracle_count_instances(int64_t n, const uint32_t* tiles_touched) {
  return count_instances(n, tiles_touched);
}
extern "C" void oracle_bin_sort(int64_t n, const float* depth32, const int32_t* rect, const uint32_t* tiles_touched,
                                int TX, int TY, uint64_t* keys, uint32_t* vals, uint32_t* ranges) {
  bin_sort(n, depth32, rect, tiles_touched, TX, TY, keys, vals, ranges);
}
extern "C" void oracle_bin_sort_spans(int64_t n, const float* depth32, const int32_t* rect, const uint32_t* tiles_touched,
                                      const int64_t* span_ptr, const int32_t* span_x, int TX, int TY, uint64_t* keys,
                                      uint32_t* vals, uint32_t* ranges) {
  bin_sort_spans(n, depth32, rect, tiles_touched, span_ptr, span_x, TX, TY, keys, vals, ranges);
}
extern "C" uint64_t oracle_conflict_count(const uint32_t* idx_a, uint32_t na, const uint32_t* idx_b, uint32_t nb) {
  return conflict_count(idx_a, na, idx_b, nb);
}
extern "C" int oracle_num_threads() { return omp_get_max_threads(); }
extern "C" void oracle_set_num_threads(int t) { omp_set_num_threads(t); }
