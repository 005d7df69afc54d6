/* odin.h -- C ABI of the per-view training step of point-based (3D Gaussian) neural rendering on one B200.
 *
 * The paper schedules "training views": render one camera, compute an image loss, back-propagate, and update only the
 * primitives that take part in the view (Sec. 2.1), in the phase order preprocessing / rendering / backward / optimizer
 * update (Sec. 4.1 phase task graph, Fig. 7 labels P/R/B/U).  Its runtime publishes and checks, per view, the
 * primitive-index scope the view may read and update (Sec. 2.1 scopes G_i, R_i^+, W_i^+; Sec. 4.3 hazard sets).  This
 * library is that view step and that scope state as CUDA kernels for sm_100a; the paper leaves the renderer arithmetic to
 * the 3D Gaussian Splatting method it builds on (Sec. 1), which is restated beside each call below.
 *
 * Conventions
 *  - Pointers named d_* and every pointer inside odin_scene / odin_projected are DEVICE pointers owned by the caller.
 *    Structs themselves (odin_scene, odin_projected, odin_camera, odin_config) are HOST structs read at call time.
 *  - Every call enqueues its kernels on `stream` (a cudaStream_t passed as void*, NULL = default stream) and returns
 *    without synchronising the host, except odin_create / odin_destroy / odin_poll.
 *  - The library allocates device memory only inside odin_create (a few hundred bytes).  Scratch comes from the
 *    caller's workspace `ws` (>= odin_workspace_bytes(), 256-byte aligned).  Calls on one context must not overlap on
 *    the GPU when they share a workspace.
 *  - Return value: ODIN_OK (0) or a negative odin_status.  Arguments are validated on the host before any launch.
 *    Data-dependent failures (more rows or instances than the caller's capacity, a bounded device-side wait that ran
 *    out) are recorded on the device, never write out of bounds, and are returned by the next odin_poll.
 *  - Counts that are only known on the device (number of touched primitives V, number of (tile, primitive) instances
 *    M) stay on the device: later calls take the device pointers and size their work from them.
 *  - Row-major arrays; "row r" of a compact array belongs to primitive prim_id[r]; rows ascend with the primitive id.
 *  - No call spins without a bound, traps, or aborts.
 */
#ifndef ODIN_H_
#define ODIN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  ODIN_OK = 0,
  ODIN_ERR_NULL = -1,        /* a required pointer is NULL */
  ODIN_ERR_INVALID_ARG = -2, /* bad size, degree, alignment, tile size ... */
  ODIN_ERR_CAPACITY = -3,    /* deferred: V > row capacity or M > instance capacity; outputs are truncated */
  ODIN_ERR_WORKSPACE = -4,   /* workspace missing, misaligned or too small */
  ODIN_ERR_CUDA = -5,        /* a CUDA runtime call failed */
  ODIN_ERR_TIMEOUT = -6,     /* deferred: a bounded device-side wait gave up; outputs of that call are invalid */
  ODIN_ERR_UNSUPPORTED = -7
} odin_status;

typedef struct odin_ctx odin_ctx; /* opaque: device ordinal, configuration, deferred-status word */

/* Renderer constants.  Defaults (pass NULL to odin_create): 1/255, 0.99, 1e-4, 0.3, 3, 1.3, 16, 0, 0. */
typedef struct {
  float alpha_min;     /* a contribution with alpha below this is skipped */
  float alpha_max;     /* alpha clamp */
  float t_min;         /* a pixel stops before the splat that would push its transmittance below this */
  float dilation;      /* low-pass term added to both diagonal entries of the 2D covariance */
  float radius_sigmas; /* screen extent in standard deviations of the major axis */
  float jac_clamp;     /* t_x/t_z and t_y/t_z are clamped to +-jac_clamp * (half image / focal) inside the Jacobian */
  int tile;            /* tile edge in pixels; only 16 is supported */
  int binning;         /* 0: tile rectangle of the radius (the method as published).  1: the rectangle is additionally cut
                          to the axis-aligned extent of the region where opacity * exp(-q/2) can reach alpha_min
                          (half extents sqrt(2 ln(opacity/alpha_min) * Sigma'_xx), ..._yy; a primitive whose opacity is
                          below alpha_min gets no tile).  An optimised-pipeline variant in the sense of Sec. 5: the
                          primitive ids, the image and the gradients are unchanged, the instance lists are shorter.
                          2: exact binning.  The rectangle stays that of the radius, but a primitive keeps only those of
                          its tiles that the region opacity * exp(-q/2) >= alpha_min reaches: the minimum of the conic's
                          quadratic form q over the rectangle of the tile's 16 x 16 pixel centres is at most
                          2 ln(opacity / alpha_min) (widened for rounding: a dropped tile holds no pixel that passes the
                          skip test).  The kept tiles of a tile row are one span; tiles_touched counts the kept tiles, a
                          primitive that keeps none is not visible, and odin_bin_sort recomputes the spans from the
                          rows (xy, conic_opacity, rect).  Same image, gradients and realized active set; about half
                          the instances on scenes of large splats.  Needs the counting scatter (instance_sort 0 on an
                          image within its limits); otherwise odin_bin_sort returns ODIN_ERR_UNSUPPORTED. */
  int instance_sort;   /* how odin_bin_sort orders the (tile, row) instances; the result is the same either way.
                          0: counting scatter (per-chunk tile counts from the rectangles, every instance written once, to
                          its final place) for images of up to 768 x 40,000 tiles (per row / in all), radix passes beyond;
                          1: always radix passes over the instances (tile-id digits, onesweep). */
} odin_config;

/* Pinhole camera (host struct).  w2c is the row-major 3x4 world-to-camera matrix [R|t]; camera axes are x right,
 * y down, z forward; pixel (i,j) is sampled at (i+0.5, j+0.5).  bg is the colour behind everything. */
typedef struct {
  int width, height;
  float fx, fy, cx, cy, znear, zfar;
  float w2c[12];
  float bg[3];
} odin_camera;

/* The primitive pool as aligned per-attribute tensors indexed by primitive id (Sec. 2.1, Fig. 4).  The same struct
 * shape holds the parameters, the two Adam moments, and a compact block of gradient rows (n = row capacity).
 *   means [n][3], log_scales [n][3], quats [n][4] (w,x,y,z; normalised inside the step), opacity_logit [n],
 *   sh [n][(sh_degree+1)^2][3].  All float32, each array 16-byte aligned. */
typedef struct {
  uint32_t n;
  int sh_degree; /* 0..3 */
  float* means;
  float* log_scales;
  float* quats;
  float* opacity_logit;
  float* sh;
} odin_scene;

/* Output of the preprocessing phase.  tiles_touched is dense (one entry per primitive, 0 = culled); everything else
 * is compact: one row per visible primitive, rows in ascending primitive order, at most `capacity` rows. */
typedef struct {
  uint32_t capacity;        /* rows the compact arrays can hold */
  uint32_t* tiles_touched;  /* [n]       number of 16x16 tiles the splat's rectangle covers (0 = not visible) */
  uint32_t* prim_id;        /* [capacity] primitive id of the row */
  float* xy;                /* [capacity][2] pixel-space centre (u, v) */
  float* depth;             /* [capacity] camera-space z */
  float* conic_opacity;     /* [capacity][4] inverse 2D covariance (A, B, C) and opacity */
  float* rgb;               /* [capacity][3] view-dependent colour, clamped at 0 */
  int32_t* radius;          /* [capacity] screen radius in pixels */
  uint16_t* rect;           /* [capacity][4] tile rectangle x0,y0,x1,y1 (half open, tile units) */
  uint32_t* tile_offset;    /* [capacity] exclusive prefix sum of tiles_touched over the rows */
  uint8_t* clamp_flags;     /* [capacity] bit c set when colour channel c was clamped at 0 */
  uint32_t* num_rows;       /* [1] V: number of rows written (device) */
  uint64_t* num_instances;  /* [1] M: sum of tiles_touched (device) */
  uint32_t* touched_mask;   /* [ceil(n/32)] optional (NULL: not wanted).  odin_project then also writes the view's touched
                               bitmask (bit p & 31 of word p >> 5), exactly what odin_touched_set derives from
                               tiles_touched; with prim_id (the ascending list) and num_rows (its length) the whole
                               touched set of Sec. 2.1 is then an output of the projection's own scan and the separate
                               call (one more pass over tiles_touched) can be left out. */
} odin_projected;

/* ---- context ------------------------------------------------------------------------------------------------- */

/* Creates a context on CUDA device `device` (made current for the call).  cfg == NULL selects the defaults. */
int odin_create(odin_ctx** ctx, int device, const odin_config* cfg);
int odin_destroy(odin_ctx* ctx);
const char* odin_status_string(int status);

/* Synchronises `stream`, returns the first deferred device-side status since the last poll (ODIN_OK if none) and
 * clears it. */
int odin_poll(odin_ctx* ctx, void* stream);

/* Chained calls.  Between odin_chain_begin and odin_chain_end the caller promises to enqueue NOTHING but calls of this
 * library with this context on one stream (no copies, memsets, event waits or kernels of its own in between).  The
 * library then launches the first kernel of a call as a programmatic dependent of the last kernel of the call before it
 * (it is scheduled while that one drains and starts with griddepcontrol.wait, so the order of all memory operations is
 * unchanged) and zeroes its scratch words with a small kernel of the same kind instead of a memset.  Results are those
 * of unchained calls; only the idle time at the seams between calls goes (about 3 us each).  Calls that enqueue a copy
 * or memset themselves (odin_poll, the scope calls) are allowed inside a chain and simply interrupt it.  Host-side
 * state of the context: not thread safe. */
int odin_chain_begin(odin_ctx* ctx);
int odin_chain_end(odin_ctx* ctx);

/* Number of unsuccessful polls after which a device-side wait of this context's later calls gives up (the look-back of
 * the prefix scans and of the radix sort waits for a word another thread block publishes).  Default 2^22, far beyond
 * anything a healthy launch needs.  A wait that gives up defers ODIN_ERR_TIMEOUT, the kernel carries on with clamped
 * addresses and returns; the outputs of that call are then invalid but nothing is written outside the caller's
 * buffers.  0 makes a wait give up the first time it finds its predecessor unpublished: for diagnostics and tests of
 * the timeout path.  polls in [0, 2^30]. */
int odin_set_wait_limit(odin_ctx* ctx, int polls);

/* Workspace size sufficient for odin_project, odin_touched_set and odin_bin_sort with at most n primitives and
 * `max_instances` instance capacity. */
int odin_workspace_bytes(const odin_ctx* ctx, uint32_t n, uint64_t max_instances, size_t* bytes);

/* Workspace size sufficient for odin_bin_sort on a width x height image with at most `row_capacity` visible rows
 * (odin_projected.capacity) and `max_instances` instance capacity: the counting scatter needs one counter per (2048
 * sorted rows, tile) and no instance buffers; the radix passes need three instance-sized buffers.  odin_bin_sort takes
 * the counting scatter whenever the image qualifies and the workspace it is given is at least this large. */
int odin_bin_sort_workspace_bytes(const odin_ctx* ctx, uint32_t row_capacity, uint64_t max_instances, int width, int height,
                                  size_t* bytes);

/* Changes odin_config.instance_sort for the later odin_bin_sort calls of this context (0 or 1, see odin_config).  The
 * counting scatter wins when rectangles cover many tiles (it never moves an instance twice), the radix passes when they
 * cover a handful (their cost per instance does not depend on how the instances are spread over the image); a caller
 * can time one view either way during warm-up and keep the faster.  A workspace sized by odin_bin_sort_workspace_bytes
 * under one mode may be too small for the other: size it for both if the mode is going to change. */
int odin_set_instance_sort(odin_ctx* ctx, int mode);

/* Minimum workspace size for odin_render_fwd / odin_render_bwd on a width x height image.  The forward call leaves in
 * it, for every tile whose list is longer than 256 entries, one record (8 KB: transmittance and colour still to come of
 * the tile's 256 pixels) per further 256 entries that it walks; the backward call of the same view replays the
 * segments of such lists independently from these records, so it must be given the SAME workspace, unmodified in
 * between.  The minimum size holds 2 x tiles + 4096 records; a larger workspace is used in full.  If a view needs more
 * records than fit, the image is still complete, ODIN_ERR_CAPACITY is deferred by the forward call and the gradients
 * of the affected tiles are approximate.  The same workspace may serve all five calls if it is at least as large as
 * both sizes (odin_project / odin_touched_set / odin_bin_sort of the NEXT view may overwrite it). */
int odin_render_workspace_bytes(const odin_ctx* ctx, int width, int height, size_t* bytes);

/* Launch accounting and optional per-kernel timing (the coarse phase profile the paper's scheduler consumes, Sec. 4.2,
 * is built from numbers like these).  Every kernel launch of the library is counted per kernel id.  After
 * odin_profile_enable(ctx, 1) each launch is also bracketed by two CUDA events on its stream (at most 65536 launches
 * between collections).  odin_profile_collect synchronises `stream`, writes per kernel id the summed event time in
 * milliseconds (h_ms, may be NULL) and the launch count since the last collection (h_launches, may be NULL) into HOST
 * arrays of odin_kernel_count() entries, and resets both. */
int odin_kernel_count(void);
const char* odin_kernel_name(int id);
int odin_profile_enable(odin_ctx* ctx, int on);
int odin_profile_collect(odin_ctx* ctx, void* stream, float* h_ms, uint64_t* h_launches);

/* Measurement aids (not part of the view step; bench.py uses them for its roofline figures).
 * odin_measure_fp32_peak: runs a kernel of independent fp32 fused multiply-add chains on every SM, synchronises, and
 * writes the sustained rate in TFLOP/s (2 flop per multiply-add) to the HOST float *h_tflops: the denominator for the
 * compositing kernels, which are bound by plain ALU work.
 * odin_count_blend_pairs: d_counts [2] (device, overwritten) = number of (pixel, list entry) pairs inside the pixels'
 * walked prefixes (d_n_contrib of odin_render_fwd), and how many of them blend (pass the skip tests): the work the
 * method itself defines for the two compositing passes of the view. */
int odin_measure_fp32_peak(odin_ctx* ctx, void* stream, float* h_tflops);
int odin_count_blend_pairs(odin_ctx* ctx, const odin_projected* proj, const uint32_t* d_vals,
                           const uint32_t* d_tile_ranges, const odin_camera* cam, const uint32_t* d_n_contrib,
                           uint64_t* d_counts, void* stream);

/* ---- the seven calls of the view step ------------------------------------------------------------------------ */

/* Preprocessing (phase P).  For every primitive: camera-space mean t = R mu + t_c; cull unless znear < t_z < zfar;
 * Sigma = R(q) diag(exp(ls))^2 R(q)^T; Sigma' = J R_c Sigma R_c^T J^T + dilation I with the pinhole Jacobian J
 * (ratio t_x/t_z, t_y/t_z clamped inside J only); conic = inverse of Sigma'; radius = ceil(radius_sigmas *
 * sqrt(larger eigenvalue)); tile rectangle = floor/ceil of (centre -+ radius)/16 clamped to the grid, cull if empty;
 * opacity = sigmoid(logit); colour = max(0, 0.5 + sum_k Y_k(dir) sh[k]) with the real SH basis up to degree 3 and
 * dir the unit vector from the camera centre to the mean.  Writes `out` as described at odin_projected.  Rows beyond
 * out->capacity are dropped and ODIN_ERR_CAPACITY is deferred; so is M >= 2^32. */
int odin_project(odin_ctx* ctx, const odin_scene* scene, const odin_camera* cam, odin_projected* out, void* ws,
                 size_t ws_bytes, void* stream);

/* Touched set: the view's candidate scope G_i = R_i^+ = W_i^+ (Sec. 2.1), i.e. every primitive with tiles_touched > 0.
 * d_mask [ceil(n/32)]: bit (p & 31) of word (p >> 5); d_idx: the ascending list of those primitive ids (first
 * idx_capacity of them; more defers ODIN_ERR_CAPACITY); d_count [1]: their number V. */
int odin_touched_set(odin_ctx* ctx, const uint32_t* d_tiles_touched, uint32_t n, uint32_t* d_mask, uint32_t* d_idx,
                     uint32_t idx_capacity, uint32_t* d_count, void* ws, size_t ws_bytes, void* stream);

/* Touched set for callers that may not allocate.  (The paper has no counterpart; this is a packaging variant of
 * odin_touched_set.)  Some users get all of their GPU memory handed out up front and are never allowed to allocate
 * again - a component living inside a host application's memory pool, a real-time loop where an allocation may stall or
 * fail - so they can neither create a context nor allocate a workspace.  This call needs neither: it runs the same
 * kernel with its scratch in a fixed device array that is part of the library image (128.3 KB on every GPU that loads
 * the library, held until the process exits).  It calls no cudaMalloc / cudaFree and no allocating library routine.
 *  - Inputs and outputs are the caller's device buffers, exactly as for odin_touched_set; the work runs on the device
 *    that is current when the call is made.
 *  - n may be at most 33,554,432 (2^25) primitives; a larger n returns ODIN_ERR_INVALID_ARG and nothing is launched.
 *  - d_status (device int, may be NULL) is where a deferred ODIN_ERR_CAPACITY / ODIN_ERR_TIMEOUT is written (only if it
 *    holds 0, so clear it beforehand); with NULL those conditions are dropped (outputs are still truncated safely).
 *  - The first call on each device also looks up the array's device address, which may make the CUDA runtime load the
 *    library's device code onto that GPU (that is when the array itself comes into being, and the runtime may
 *    synchronise the device while it does so).  Treat the first call per device as a warm-up: make it during
 *    start-up, before the phase in which nothing may allocate begins and before any stream capture.
 *  - The block size is chosen for the 148 SMs of a B200 (there is no context to ask); on another GPU the result is the
 *    same, only the split of the work differs.
 *  - Every call on a device shares the one array.  The call clears the part it uses, but two calls whose kernels
 *    overlap on the GPU (different streams, different host threads) race on it: serialise them. */
int odin_touched_set_static(const uint32_t* d_tiles_touched, uint32_t n, uint32_t* d_mask, uint32_t* d_idx,
                            uint32_t idx_capacity, uint32_t* d_count, int* d_status, void* stream);

/* Binning and sort.  Emits one (key, value) per (tile, row) pair of the rectangles: key = tile_id << 32 | bit pattern
 * of the float32 depth, tile_id = ty * ceil(width/16) + tx; value = ROW index r (the primitive is proj->prim_id[r]).
 * The result is the order of a stable least-significant-digit radix sort by key (equal keys keep ascending row order):
 * d_vals [capacity] the sorted values, d_keys [capacity] the sorted keys (may be NULL when only the values are wanted:
 * the later calls read d_vals and d_tile_ranges only), d_tile_ranges [tiles][2] = [first, one past last) position of
 * each tile (an empty tile has first == last).
 * When M > capacity only the `capacity` instances of the nearest rows are produced (ODIN_ERR_CAPACITY deferred). */
int odin_bin_sort(odin_ctx* ctx, const odin_projected* proj, int width, int height, uint64_t* d_keys, uint32_t* d_vals,
                  uint64_t capacity, uint32_t* d_tile_ranges, void* ws, size_t ws_bytes, void* stream);

/* Rendering (phase R).  Per pixel, front to back over its tile's sorted rows: dx = u - x, dy = v - y,
 * power = -(A dx^2 + C dy^2)/2 - B dx dy; skip if power > 0; alpha = min(alpha_max, opacity * exp(power)); skip if
 * alpha < alpha_min; stop if T (1 - alpha) < t_min; colour += rgb * alpha * T; T *= 1 - alpha.
 * d_rgb [3][H][W] = colour + T * bg (planar, not clamped); d_final_T [H][W]; d_n_contrib [H][W] = 1 + list offset of the
 * last row that contributed (0 if none).
 * ws (at least odin_render_workspace_bytes, 256-byte aligned): scratch, and the records that odin_render_bwd of the
 * same view reads (see odin_render_workspace_bytes); ODIN_ERR_CAPACITY is deferred when they do not all fit (the
 * outputs of this call are complete in any case). */
int odin_render_fwd(odin_ctx* ctx, const odin_projected* proj, const uint32_t* d_vals, const uint32_t* d_tile_ranges,
                    const odin_camera* cam, float* d_rgb, float* d_final_T, uint32_t* d_n_contrib, void* ws, size_t ws_bytes,
                    void* stream);

/* Image loss of the view (Sec. 2.1): d_loss [1] = mean |rgb - target| over 3*H*W values;
 * d_dL_drgb [3][H][W] = sign(rgb - target) / (3 H W). */
int odin_l1_loss(odin_ctx* ctx, const float* d_rgb, const float* d_target, int width, int height, float* d_loss,
                 float* d_dL_drgb, void* stream);

/* Backward (phase B).  (a) Per pixel, back to front over the rows that contributed: gradients of the loss with
 * respect to each row's colour, opacity, conic and centre (a clamped alpha passes no gradient), summed over pixels
 * into d_grad2d [capacity][9] = (u, v, A, B, C, opacity, r, g, b).  (b) Per row: chain rule through the conic
 * inverse, the EWA projection, the Jacobian (clamp frozen), Sigma = M M^T, scale = exp(log scale), the rotation and
 * the quaternion normalisation, the pixel centre, the SH colour (clamped channels pass nothing; the direction term
 * reaches the mean) and the sigmoid.  grad_rows: compact rows (row r <-> proj->prim_id[r]) in the layout of
 * odin_scene with n >= V.
 * d_row_active [capacity] (bytes, may be NULL): 1 for every row that was blended into at least one pixel - the
 * realized active set C_i of Sec. 2.1, observed where the paper observes it, after the backward pass - else 0.
 * d_row_zero [capacity] (bytes, may be NULL): if given, a row whose nine words of d_grad2d are all zero (it never
 * blended: most touched rows are occluded) is NOT written to grad_rows; d_row_zero[r] = 1 says so instead, 0 marks the
 * rows that were written.  odin_sparse_adam takes the same flags and reads no gradient for the flagged rows.
 * ws: the workspace the odin_render_fwd call of this view used, unmodified since (see odin_render_workspace_bytes). */
int odin_render_bwd(odin_ctx* ctx, const odin_scene* scene, const odin_camera* cam, const odin_projected* proj,
                    const uint32_t* d_vals, const uint32_t* d_tile_ranges, const float* d_final_T,
                    const uint32_t* d_n_contrib, const float* d_dL_drgb, float* d_grad2d, odin_scene* grad_rows,
                    uint8_t* d_row_active, uint8_t* d_row_zero, void* ws, size_t ws_bytes, void* stream);

/* Optimizer update (phase U) restricted to the touched rows: for every r < *d_count and every scalar theta of
 * primitive d_idx[r] with gradient g: m = b1 m + (1-b1) g; v = b2 v + (1-b2) g^2;
 * theta -= lr_group / (1 - b1^step) * m / (sqrt(v) / sqrt(1 - b2^step) + eps).  step is the global 1-based step.
 * lr: mean, log scale, quaternion, opacity, SH degree 0, SH degrees >= 1.  Rows that are not listed are neither read
 * nor written.  d_idx must be strictly ascending (as produced by odin_touched_set / odin_project).
 * d_row_zero [rows] (bytes, may be NULL): the flags of odin_render_bwd; a flagged row's gradient is taken as zero
 * without reading grad_rows (its moments still decay and its parameters still move, exactly as with a row of zeros). */
int odin_sparse_adam(odin_ctx* ctx, odin_scene* params, odin_scene* m, odin_scene* v, const odin_scene* grad_rows,
                     const uint8_t* d_row_zero, const uint32_t* d_idx, const uint32_t* d_count, const float lr[6],
                     float beta1, float beta2, float eps, uint32_t step, void* stream);

/* The same update with one byte of optimizer state per primitive that lets it leave untouched history unread (phase U
 * of Sec. 4.1; most rows a view touches are occluded, receive no gradient and have never received one).
 * d_live [params->n] (bytes, device, caller-owned, may be NULL = odin_sparse_adam): d_live[p] == 0 promises that
 * EVERY moment of primitive p, in m and in v, is zero.  A listed row with a zero gradient and d_live == 0 is then
 * skipped without reading its moments (the result is what the full update gives bit for bit: zero moments stay zero
 * and theta - step * 0 / (0 + eps) = theta; with eps == 0 nothing is skipped); the call sets d_live[p] = 1 for every
 * primitive to which it writes moments that may be non-zero, so the promise holds again on return.  The array belongs
 * with m and v: zero it when they are zeroed, store and restore it with them, and after writing m or v by any other
 * means call odin_adam_live_refresh (or set every byte to 1, which is always valid).  Not to be shared between two
 * calls that overlap in time. */
int odin_sparse_adam_live(odin_ctx* ctx, odin_scene* params, odin_scene* m, odin_scene* v, const odin_scene* grad_rows,
                          const uint8_t* d_row_zero, const uint32_t* d_idx, const uint32_t* d_count, uint8_t* d_live,
                          const float lr[6], float beta1, float beta2, float eps, uint32_t step, void* stream);

/* d_live[p] = 1 if any moment of primitive p (any word of its rows in m or v) is non-zero, else 0, for all p < m->n:
 * the tightest flags that keep the promise of odin_sparse_adam_live.  One pass over both moment pools. */
int odin_adam_live_refresh(odin_ctx* ctx, const odin_scene* m, const odin_scene* v, uint8_t* d_live, void* stream);

/* Conflict counts (Sec. 4.3): for each listed pair (a, b) of views, |W^+(a) & W^+(b)| = popcount of the AND of their
 * touched bitmasks, the size of C_WAW^+ (C_RAW^+ and C_WAR^+ are empty because R^+ = W^+ here).
 * d_masks [n_masks][mask_stride_words]; d_pairs [n_pairs][2] view slots; d_counts [n_pairs] (overwritten). */
int odin_conflict_count(odin_ctx* ctx, const uint32_t* d_masks, uint32_t n_masks, uint32_t mask_stride_words,
                        uint32_t n_prims, const uint32_t* d_pairs, uint32_t n_pairs, uint64_t* d_counts, void* stream);

/* ---- realized scope, gradient evidence and admission arithmetic (Sec. 2.1 Table 1, Sec. 4.3) -------------------- */

/* Realized active set C_i and gradient evidence g(p) of a view (Sec. 2.1: Theta >= G_i >= C_i; g_U(p) = per-primitive
 * gradient magnitude of the active primitives).  From the row flags of odin_render_bwd:
 * d_mask [ceil(n/32)] bit per primitive id (overwritten); d_idx: ascending primitive ids of the active rows (first
 * idx_capacity; more defers ODIN_ERR_CAPACITY); d_count [1]; d_evidence [idx_capacity] parallel to d_idx;
 * d_evidence_sum [1] (double) = sum of the evidence over C_i (mean = sum / count).
 * evidence_mode 0: Euclidean norm of the gradient with respect to the projected centre, sqrt(g_u^2 + g_v^2) of
 * d_grad2d (the quantity point-based pipelines accumulate per primitive); 1: Euclidean norm of the whole gradient row
 * (grad_rows, required in this mode).  Sec. 2.1 / Sec. 4.3 leave the norm of g(p) open, so both readings are
 * offered.  n = number of primitives of the pool. */
int odin_active_set(odin_ctx* ctx, const odin_projected* proj, const uint8_t* d_row_active, const float* d_grad2d,
                    const odin_scene* grad_rows, int evidence_mode, uint32_t n, uint32_t* d_mask, uint32_t* d_idx,
                    uint32_t idx_capacity, uint32_t* d_count, float* d_evidence, double* d_evidence_sum, void* ws,
                    size_t ws_bytes, void* stream);

/* Unit unions (Sec. 2.1: R^+(U), W^+(U), C_U are unions over the views of a task unit): d_out [stride_words] = OR of
 * the masks d_masks[d_members[k]], k < n_members (zero words for n_members = 0). */
int odin_mask_union(odin_ctx* ctx, const uint32_t* d_masks, uint32_t n_masks, uint32_t mask_stride_words,
                    uint32_t n_prims, const uint32_t* d_members, uint32_t n_members, uint32_t* d_out, void* stream);

/* Task units of several views (Sec. 2.1: the scope of a unit is the union of its views' scopes; Sec. 6.1 runs two views
 * per unit): the views of a unit are rendered and differentiated with the same parameters, their gradient rows are
 * added up over the union of their touched sets, and ONE optimizer update is applied to the union.
 * odin_mask_to_list: the ascending list of the members of a bitmask over the primitives (for example the OR of two
 * views' touched masks from odin_mask_union): d_idx (first idx_capacity members; more defers ODIN_ERR_CAPACITY),
 * d_count [1].  Bits at or beyond n are ignored.  ws: at least odin_workspace_bytes(n, 0).
 * odin_accumulate_rows: rows_u[r] = (row of primitive d_idx_u[r] in view a, if a lists it) + (the same for view b),
 * for r < *d_count_u.  rows_a / rows_b: the compact gradient rows of the two views (row i <-> d_idx_a[i], i <
 * *d_count_a; d_zero_a: the row_zero flags of odin_render_bwd, may be NULL); rows_u: n >= union size, same SH degree.
 * odin_sparse_adam(params, m, v, rows_u, NULL, d_idx_u, d_count_u, ...) then updates the unit. */
int odin_mask_to_list(odin_ctx* ctx, const uint32_t* d_mask, uint32_t n, uint32_t* d_idx, uint32_t idx_capacity,
                      uint32_t* d_count, void* ws, size_t ws_bytes, void* stream);
int odin_accumulate_rows(odin_ctx* ctx, const odin_scene* rows_a, const uint8_t* d_zero_a, const uint32_t* d_idx_a,
                         const uint32_t* d_count_a, const odin_scene* rows_b, const uint8_t* d_zero_b,
                         const uint32_t* d_idx_b, const uint32_t* d_count_b, const uint32_t* d_idx_u,
                         const uint32_t* d_count_u, odin_scene* rows_u, void* stream);

/* The three primitive-state hazards of the quality-first path (Sec. 4.3) for pairs (A, B) = (producer, consumer):
 *   WAW = W(B) & W(A);  RAW = (R(B) \ W(B)) & W(A);  WAR = W(B) & (R(A) \ W(A)).
 * d_read_masks, d_write_masks [n_masks][mask_stride_words]: the conservative scopes R^+, W^+ of each unit;
 * d_pairs [n_pairs][2] = (A, B); d_counts [n_pairs][4] (overwritten) = (#WAW, #RAW, #WAR, #R^+(B)). */
int odin_hazard_count(odin_ctx* ctx, const uint32_t* d_read_masks, const uint32_t* d_write_masks, uint32_t n_masks,
                      uint32_t mask_stride_words, uint32_t n_prims, const uint32_t* d_pairs, uint32_t n_pairs,
                      uint64_t* d_counts, void* stream);

/* Evidence for the throughput-first admission (Sec. 4.3).  Delayed-read set D^+ = C_RAW^+(A, B) =
 * (R(B) \ W(B)) & W(A).  A delayed primitive has producer evidence when it is in C_A; it passes the gradient gate
 * when g_A(p) <= tau * mean of g_A over C_A.  Inputs: the three masks [ceil(n_prims/32)], A's active list, evidence,
 * count and evidence sum as written by odin_active_set.  d_gate [4] (overwritten) = (#D^+, #(D^+ & C_A), #passing the
 * gate, #R^+(B)).  The caller admits the delayed read iff #R^+(B) > 0, #D^+ / #R^+(B) <= tau, C_A is not empty and
 * all three first counts are equal. */
int odin_delayed_read_gate(odin_ctx* ctx, const uint32_t* d_read_b, const uint32_t* d_write_b, const uint32_t* d_write_a,
                           uint32_t n_prims, const uint32_t* d_active_idx_a, const float* d_evidence_a,
                           const uint32_t* d_active_count_a, const double* d_evidence_sum_a, uint32_t active_capacity_a,
                           float tau, uint64_t* d_gate, void* stream);

/* ---- relative locality graph from the measured scopes (Sec. 4.1 Eq. (1), Sec. 4.2 Eq. (2)) ------------------------
 * The paper builds its ahead-of-time graph from SfM tracks and says that realized activity can refresh the scores
 * later; these calls evaluate the same formulas on the per-view primitive sets this library produces (the
 * computation-based graph of Sec. 4.1): set sizes from odin_touched_set / odin_active_set, intersections from
 * odin_conflict_count / odin_hazard_count. */

/* Eq. (1): d_weights [n_pairs] = d_counts[i] / (d_sizes[a] + d_sizes[b] - d_counts[i]) for pair i = (a, b), 0 when the
 * union is empty (one float32 division).  d_counts [n_pairs] u64 intersection sizes, d_sizes [n_views] set sizes. */
int odin_rlg_weights(odin_ctx* ctx, const uint64_t* d_counts, const uint32_t* d_sizes, const uint32_t* d_pairs,
                     uint32_t n_pairs, uint32_t n_views, float* d_weights, void* stream);

/* Neighbour retention: every item keeps its k strongest neighbours (larger weight first, lower index first among equal
 * weights; zero weights are not edges); the graph is undirected, so an edge stays when either end keeps it.
 * d_weights, d_retained [n_views][n_views] row major (distinct buffers; d_weights symmetric); dropped edges and the
 * diagonal are written as 0.  ws: n_views^2 bytes.  n_views <= 32768. */
int odin_rlg_topk(odin_ctx* ctx, const float* d_weights, uint32_t n_views, uint32_t k, float* d_retained, void* ws,
                  size_t ws_bytes, void* stream);

/* Eq. (2): d_scores[c] = sum over u in the previous unit of w[u][v], v = d_candidates[c] (fp32 accumulation). */
int odin_sds_scores(odin_ctx* ctx, const float* d_weights, uint32_t n_views, const uint32_t* d_prev_unit, uint32_t n_prev,
                    const uint32_t* d_candidates, uint32_t n_candidates, float* d_scores, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* ODIN_H_ */
