/*
 * zgr.h - C ABI of the ZGR hot path: the zeroth-order (ZOO) step with cloud-guided gradient
 * rectification of CooperLLM, as hand-written CUDA for NVIDIA B200 (sm_100a).
 *
 * What one step does (Sec. 3.2, Eq. (perturbation), Eq. (grad), Algorithm 1).  For every weight
 * tensor theta_l (rows x cols, row-major) the hybrid perturbation
 *
 *      z_l = a * Z_l  +  b * U_l * G_l
 *
 * is regenerated on the fly from a 64-bit seed: Z_l is isotropic Gaussian noise, U_l (rows x r,
 * orthonormal columns) is the cloud-supplied gradient subspace of that tensor and G_l (r x cols)
 * holds the guided coefficients, either drawn from the seed or delivered compressed (Sec. 3.4,
 * DTC).  A step is three in-place sweeps over the weights and never stores z:
 *
 *      zgr_perturb(seed, +eps)            theta <- rnd(theta + eps z)       forward pass -> L+
 *      zgr_perturb(seed, -2 eps)          theta <- rnd(theta - 2 eps z)     forward pass -> L-
 *      zgr_restore_update(seed, L+, L-, lr)
 *                                         theta <- rnd(theta + (eps - lr (L+ - L-)/(2 eps)) z)
 *
 * Conventions.
 *   - Every `void* stream` is a cudaStream_t (NULL = the legacy default stream).  Sweeps are
 *     enqueued on it and return without synchronising.  The sweeps of one context must be ordered
 *     with respect to each other (one stream, or streams that the caller orders): they write the
 *     same weights and share the library's work-item counters.
 *   - "device" pointers are CUDA device addresses on the current device; the library never
 *     dereferences them on the host and never frees them.  They are borrowed for the life of the
 *     context.
 *   - All functions return 0 on success or a negative ZGR_E* code.  Arguments are validated before
 *     anything is launched: a call that fails validation leaves the weights untouched.
 *   - A context is bound to the device that is current when zgr_init is called and is not
 *     thread-safe; use one per thread or serialise calls.  Every call that enqueues work checks that
 *     this device is still the current one and returns ZGR_EINVAL otherwise, before anything is launched.
 */
#ifndef ZGR_H_
#define ZGR_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ZGR_MAX_RANK 64 /* largest subspace rank r per tensor */
#define ZGR_MAX_SEEDS 8 /* most (seed, coefficient) terms one sweep can apply */

enum { ZGR_OK = 0, ZGR_EINVAL = -1, ZGR_ESTATE = -2, ZGR_ECUDA = -3, ZGR_ENOMEM = -4, ZGR_ETOOBIG = -5 };

/* storage type of a weight tensor; arithmetic is fp32, one round-to-nearest-even per sweep */
enum { ZGR_F32 = 0, ZGR_F16 = 1, ZGR_BF16 = 2 };

/* Normalisation of Eq. (perturbation), with n := d = total parameters and m := K = total guided
 * coefficients (sum of rank * cols over tensors that have a subspace):
 *   ZGR_SCALE_PAPER  a = sqrt(alpha/d),  b = sqrt((1-alpha)/K)          (E|z|^2 = 1)
 *   ZGR_SCALE_UNIT   a = sqrt(alpha),    b = sqrt((1-alpha) d/K)        (E|z|^2 = d; alpha = 1 is
 *                                                                       exactly the z of Eq. (ZOO)) */
enum { ZGR_SCALE_PAPER = 0, ZGR_SCALE_UNIT = 1 };

/* Stream tags of the counter-based generator (fourth counter word). */
enum { ZGR_TAG_ISO = 0, ZGR_TAG_COEFF = 1 };

typedef struct zgr_ctx zgr_ctx; /* opaque; created by zgr_init, released by zgr_destroy */

/* One weight tensor.  1-D tensors are given as rows = 1, cols = length, U = NULL, rank = 0. */
typedef struct {
  void* data;       /* device; rows*cols elements of `dtype`, row-major, contiguous, updated in place.
                       Must be aligned to the element size; 16-byte alignment and cols a multiple of
                       16 bytes' worth of elements select the vectorised kernels.  fp32 storage with
                       rank > 8 is served by the one-element-per-thread fallback kernel (exact fp32
                       contraction; none of the paper-shaped configurations needs it) */
  int64_t rows;     /* m_l >= 1 */
  int64_t cols;     /* n_l >= 1 */
  int32_t dtype;    /* ZGR_F32 | ZGR_F16 | ZGR_BF16 */
  int32_t rank;     /* r_l in [0, ZGR_MAX_RANK]; 0 = isotropic noise only */
  const float* U;   /* device; rows x rank fp32 row-major, orthonormal columns (not checked, not
                       re-orthonormalised); NULL iff rank == 0 */
} zgr_tensor;

typedef struct {
  double alpha;            /* mixing ratio of Eq. (perturbation), in [0, 1] */
  double eps;              /* perturbation scale epsilon > 0 of Eq. (ZOO) */
  int32_t scale_mode;      /* ZGR_SCALE_PAPER | ZGR_SCALE_UNIT */
  int32_t bits_per_normal; /* 32: one generator block per 4 elements; 16: one per 8 elements */
  int32_t stats;           /* != 0: the first perturbation under every seed also keeps the norm bookkeeping
                              (see zgr_get_stats); it can be switched later with zgr_enable_stats */
} zgr_config;

/* Build a context over `n` tensors (Algorithm 1, "Require": model, epsilon, alpha, subspace).
 * `tensors` and `cfg` are host pointers, copied.  Tensor l gets generator tensor-id l.
 * Allocates only the library's own descriptor and work tables on the current device.
 * ZGR_EINVAL: null argument, n <= 0, bad dtype/rank/shape, misaligned data, alpha outside [0,1],
 * eps <= 0 or not finite, unknown scale_mode or bits_per_normal.  ZGR_ECUDA / ZGR_ENOMEM: no usable
 * device or allocation failure (also the answer on a machine without a GPU). */
int zgr_init(zgr_ctx** out, const zgr_tensor* tensors, int32_t n, const zgr_config* cfg);

/* theta_l <- rnd(theta_l + scale * z_l(seed)) for every tensor (Algorithm 1, "Compute loss
 * difference": W + eps z_h, then W - eps z_h, reached by scale = +eps followed by scale = -2 eps).
 * The context remembers `seed` and the sum of the scales applied under it.
 * ZGR_EINVAL: scale not finite.  ZGR_ESTATE: a different seed is still active (its
 * restore_update has not been called); zgr_sweep_multi is the call that may overlap seeds. */
int zgr_perturb(zgr_ctx* ctx, uint64_t seed, double scale, void* stream);

/* Undo the net perturbation of `seed` and take the projected-gradient step in the same sweep
 * (Eq. (grad); Algorithm 1 "Recover gradient", "Update"):
 *     g = (loss_plus - loss_minus) / (2 eps),   theta_l <- rnd(theta_l + (-net - lr g) z_l(seed)).
 * lr = 0 is a pure restore.  Scalars are combined in double on the host and passed to the kernel
 * as fp32.  ZGR_EINVAL: a loss or lr is not finite.  ZGR_ESTATE: `seed` is not the active seed. */
int zgr_restore_update(zgr_ctx* ctx, uint64_t seed, double loss_plus, double loss_minus, double lr, void* stream);

/* Several seeds in one sweep:  theta_l <- rnd(theta_l + sum_i coeffs[i] * z_l(seeds[i]))  for every tensor,
 * one rounding.  This is the sum over seeds of Algorithm 1 ("Recover gradient": sum_t g_t z_t, applied
 * by "Update") as one pass over the weights instead of one pass per seed: the edge server's
 * aggregation of its clients' projected gradients, a step that averages several perturbation queries,
 * or the fusion of one query's restore with the next query's perturbation
 * (seeds = {s_q, s_q+1}, coeffs = {+eps, +eps} after perturb(s_q, +eps), perturb(s_q, -2 eps)).
 * seeds, coeffs: HOST arrays of n entries, 1 <= n <= ZGR_MAX_SEEDS, seeds pairwise different.
 * The context adds coeffs[i] to the net coefficient it keeps for seeds[i]; a seed whose net
 * coefficient returns to exactly 0 is idle again.  Unlike zgr_perturb it may be called while other
 * seeds are active.  ZGR_EINVAL: null pointer, n out of range, repeated seed, coefficient not finite. */
int zgr_sweep_multi(zgr_ctx* ctx, int32_t n, const uint64_t* seeds, const double* coeffs, void* stream);

/* zgr_restore_update for n seeds in one sweep (Eq. (grad) per seed; Algorithm 1 "Recover gradient" and
 * "Update" with the sum over seeds):
 *     g_i = (loss_plus[i] - loss_minus[i]) / (2 eps),
 *     theta_l <- rnd(theta_l + sum_i (-net_i - lr g_i) z_l(seeds[i])),
 * net_i being the net coefficient still applied under seeds[i] (0 for a seed that is not active, which
 * is the server-side case: nothing to undo, only the update).  `lr` is the step applied per seed: pass
 * lr/n to average n queries.  The listed seeds are idle afterwards; other active seeds stay active.
 * All arrays are HOST arrays of n entries, 1 <= n <= ZGR_MAX_SEEDS, seeds pairwise different.
 * ZGR_EINVAL: null pointer, n out of range, repeated seed, a loss or lr not finite. */
int zgr_restore_update_multi(zgr_ctx* ctx, int32_t n, const uint64_t* seeds, const double* loss_plus, const double* loss_minus, double lr,
                             void* stream);

/* Change the mixing ratio alpha of Eq. (perturbation) between steps; a and b are recomputed as in
 * zgr_init.  This is the hook for the adaptive choice of the mixing ratio announced in Sec. 1, which is to
 * follow the sizes of the guided and the isotropic part; the paper gives no rule, so the caller applies its
 * own to the norms of zgr_get_stats (or uses zgr_adapt_alpha below) and sets the result here.
 * ZGR_EINVAL: alpha outside [0, 1].  ZGR_ESTATE: a perturbation is active, or the context was built with
 * alpha = 1 (its sweep plan carries no subspace operands) and alpha < 1 is asked for. */
int zgr_set_alpha(zgr_ctx* ctx, double alpha);

/* One candidate for that adaptive choice, off unless the caller invokes it: balance the energies of the two
 * parts of Eq. (perturbation).  `stats` (HOST, 3 doubles per tensor, as written by zgr_get_stats under the
 * context's current alpha) gives sum (a Z)^2 and sum (b U G)^2; divided by a^2 d and b^2 K they are the energy
 * of each part per unit of its mixing weight, e_iso and e_g, and the two parts carry the same energy at
 *     alpha* = e_g / (e_iso + e_g).
 * The context moves to  alpha = clamp((1 - eta) alpha_old + eta alpha*, alpha_min, alpha_max)  (a, b recomputed
 * as in zgr_set_alpha) and *alpha_out receives it.  With seed-drawn unit coefficients and an orthonormal U the
 * balance sits at 1/2; compressed coefficients whose scale is not that of a unit Gaussian, or a subspace that
 * is not orthonormal, move it.  If one of the parts is switched off (alpha = 0 or 1, or no tensor has a
 * subspace) alpha is left as it is.  The rule is this library's: Sec. 1 announces an adaptive ratio that
 * follows the relative sizes of the two parts and states none.
 * ZGR_EINVAL: null pointer, bounds not 0 <= alpha_min <= alpha_max <= 1, eta outside [0, 1], a norm that is
 * negative or not finite.  ZGR_ESTATE: a perturbation is active. */
int zgr_adapt_alpha(zgr_ctx* ctx, const double* stats, double alpha_min, double alpha_max, double eta, double* alpha_out);

/* Deliver the guided coefficients of one tensor compressed (Sec. 3.4, DTC): from now on
 *     G_l[k][c] = scale[k] * (q[k][c] - zero[k])       (x = lambda (x_quant - delta))
 * replaces the seed-drawn G_l.  scale: device, rank fp32; zero: device, rank fp32, or NULL for delta = 0.
 *   bits = 8: q is device, rank x cols int8 (signed codes) row-major.
 *   bits = 4: the paper's INT4 payload.  q is device, rank rows of (cols + 1)/2 bytes; each byte holds two
 *             unsigned codes in [0, 15], the even column in the low nibble (the last byte of a row with an
 *             odd number of columns has its high nibble ignored).  The zero point carries the offset.
 * Pointers are borrowed, not copied.
 * ZGR_EINVAL: bad tensor index, tensor without subspace, null q/scale, bits not 8 or 4.
 * ZGR_ESTATE: a perturbation is active (the coefficients must not change between a perturb and
 * its restore_update). */
int zgr_set_coeffs_dtc(zgr_ctx* ctx, int32_t tensor, const int8_t* q, const float* scale, const float* zero, int32_t bits);

/* The same with only a proportion of the payload compressed (Sec. 3.4, the adaptive proportion omega): the
 * first n_rows rows of G_l come from the codes (q: n_rows rows in the layout of `bits`; scale, zero: n_rows
 * entries), rows n_rows .. rank-1 are drawn from the seed as if nothing had been delivered for them.
 * 1 <= n_rows <= rank; n_rows = rank is zgr_set_coeffs_dtc.  Errors as there, plus ZGR_EINVAL for n_rows out of range. */
int zgr_set_coeffs_dtc_rows(zgr_ctx* ctx, int32_t tensor, const int8_t* q, const float* scale, const float* zero, int32_t bits, int32_t n_rows);

/* zgr_perturb, layer by layer, with the guided payload of each layer arriving from the host while earlier
 * layers are swept (Sec. 3.3, the layer-wise sample -> transmit -> apply pipeline; Sec. 3.4, the transmission
 * of a layer is to fit under the compute of another).  layer_end: HOST array of n_layers strictly increasing
 * tensor indices, layer L being the tensors [layer_end[L-1], layer_end[L]) and layer_end[n_layers-1] the number
 * of tensors.  deliveries: HOST array; entry i names a tensor and gives HOST sources (pinned memory, or the
 * copies do not overlap anything) for its compressed coefficients (q, scale, zero: the tensor's coefficients
 * must have been set with zgr_set_coeffs_dtc(_rows); same sizes and layout, copied into those device buffers)
 * and/or for its subspace (U: rows x rank fp32, copied into the subspace buffer given to zgr_init; the
 * tensor-core operand copies are rebuilt before the layer is swept).  All copies are enqueued at once on
 * `copy_stream`, in layer order, behind the work already on `stream`; the sweep of a layer waits for that
 * layer's copies only, so later layers travel while earlier ones are swept.  Consecutive layers are swept on two
 * streams in turn (`stream` and one of the library's), which lets a layer start on the SMs that the previous
 * one has already left; `stream` waits for all of it at the end.  n_deliveries = 0 gives the same sweep as
 * zgr_perturb, issued as one launch per kernel family and layer.
 * The result is identical to copying everything first and calling zgr_perturb.
 * ZGR_EINVAL: scale not finite, bad layer table, a delivery naming a bad or repeated tensor or carrying
 * nothing, coefficients for a tensor without compressed coefficients, a zero point given for a tensor
 * registered without one (or the reverse), a subspace for a tensor without one.
 * ZGR_ESTATE: as zgr_perturb; with deliveries, also if any seed is active (the payload may not change between
 * a perturbation and its restore). */
typedef struct {
  int32_t tensor;
  const void* q;       /* HOST: codes of the delivered rows, or NULL if only a subspace is delivered */
  const float* scale;  /* HOST: one per delivered row (NULL iff q is NULL) */
  const float* zero;   /* HOST: one per delivered row, or NULL if the tensor was registered without zero points */
  const float* U;      /* HOST: rows x rank fp32 subspace, or NULL */
} zgr_coeff_delivery;
int zgr_perturb_layers(zgr_ctx* ctx, uint64_t seed, double scale, int32_t n_layers, const int32_t* layer_end, int32_t n_deliveries,
                       const zgr_coeff_delivery* deliveries, void* stream, void* copy_stream);

/* Back to seed-drawn coefficients for `tensor` (Algorithm 1, "Sample z_g").  Errors as above. */
int zgr_clear_coeffs(zgr_ctx* ctx, int32_t tensor);

/* A guided round delivers a new subspace for `tensor` (Algorithm 1, "Collect gradients to build basis
 * V_r", transmitted layer by layer as in Sec. 3.3).  U_src: rows x rank fp32 row-major, on the host
 * (src_is_host != 0; pinned memory makes the copy asynchronous) or on the device, or NULL if the caller
 * has already rewritten the device buffer given to zgr_init in place.  The values are copied into that
 * device buffer (it is overwritten) on `stream`, and the library's own operand copy of U for the
 * tensor-core kernels is rebuilt.  ZGR_EINVAL: bad index or tensor without subspace.
 * ZGR_ESTATE: a perturbation is active. */
int zgr_update_subspace(zgr_ctx* ctx, int32_t tensor, const float* U_src, int32_t src_is_host, void* stream);

/* zgr_update_subspace for n tensors in one call (tensors[i] gets U_src[i]; U_src may be NULL, or hold NULL
 * entries, for buffers already rewritten in place; all sources on the host or all on the device).  The copies are
 * enqueued one by one; when the list names every tensor that the tensor-core path serves, their operand copies
 * are rebuilt by a single launch instead of one per tensor, which is what a guided round that refreshes the
 * whole model wants.  tensors: HOST array of pairwise different indices.  Errors as zgr_update_subspace, plus
 * ZGR_EINVAL for n < 1 or a repeated index. */
int zgr_update_subspaces(zgr_ctx* ctx, int32_t n, const int32_t* tensors, const float* const* U_src, int32_t src_is_host, void* stream);

/* Build the subspace of `tensor` on the device from collected gradient directions (Algorithm 1, "Collect
 * gradients to build basis V_r"; Sec. 3.2, cloud side).  grads: rows x rank fp32 row-major whose column j is the
 * j-th direction collected in the row space of the tensor (the paper does not say how a gradient of a matrix
 * becomes a direction of its row space; that reduction is the caller's), on the host (src_is_host != 0) or on
 * the device, or NULL if the directions were written into the subspace buffer given to zgr_init.  The result is
 * the orthonormal basis of their span that a QR factorisation with a positive diagonal of R gives, column k
 * spanning, with the columns before it, the first k + 1 directions.  It overwrites that subspace buffer, and the
 * library's operand copies are rebuilt as by zgr_update_subspace.  Cholesky QR applied twice, carried in double:
 * orthonormal to about 1e-7 for inputs whose condition number is below about 1e6.  Allocates scratch on
 * first use (and when a larger tensor comes); synchronises `stream`.
 * ZGR_EINVAL: bad index, tensor without subspace, fewer rows than rank, misaligned pointer, or directions that
 * are linearly dependent to working precision (nothing is written then).  ZGR_ESTATE: a perturbation is active. */
int zgr_build_subspace(zgr_ctx* ctx, int32_t tensor, const float* grads, int32_t src_is_host, void* stream);

/* Norm bookkeeping for the adaptive choice of alpha mentioned in Sec. 1: for each tensor l,
 * out[3l+0] = sum (a Z_l)^2, out[3l+1] = sum (b U_l G_l)^2, out[3l+2] = sum z_l^2 for `seed`.
 * `out` is a HOST array of 3*n doubles; the call synchronises `stream`.
 * With the bookkeeping switched on (zgr_config.stats, zgr_enable_stats) the first zgr_perturb or
 * zgr_perturb_layers under a seed accumulates these sums inside its sweep (per work item and warp; that sweep
 * costs about a quarter more), and zgr_get_stats for that seed only adds the partial sums up and reads them
 * back, as long as alpha, the subspaces and the coefficients have not changed since.  Otherwise the call makes
 * a pass of its own that regenerates Z and U G for `seed` and reads no weights.  Either way the partial sums
 * are added in a fixed order: repeated calls give identical bits.  (The two routes agree to about 1e-6
 * relative, not bit for bit: the sweep takes the guided part as accumulator minus weight.) */
int zgr_get_stats(zgr_ctx* ctx, uint64_t seed, double* out, void* stream);
int zgr_enable_stats(zgr_ctx* ctx, int32_t enable);

/* The norms of ONE tensor, computed without allocating anything.  (The paper has no counterpart; this
 * entry point exists for callers that cannot allocate device memory while they run: loops in which the
 * device-wide synchronisation implied by cudaMalloc/cudaFree would stall other streams, and processes
 * whose framework has already claimed all free device memory for its own pool.)
 * Same three sums as zgr_get_stats for `tensor`, written to dev_out3 (DEVICE, 3 doubles, 8-byte
 * aligned) by work enqueued on `stream`; the call does not synchronise.  All intermediate storage is a
 * fixed array inside the library image: 3 * ZGR_NOALLOC_MAX_TILES doubles (192 KiB), resident on every
 * GPU that loads the library until the process exits.  A tile is 1024 rows x 64 columns, so tensors
 * up to ZGR_NOALLOC_MAX_TILES tiles (e.g. 32000 x 16384) fit; larger ones are refused with ZGR_ETOOBIG.
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress); make that
 * first call outside any stream capture.  Every call uses the same array: two calls whose kernels can
 * overlap on the GPU (different streams, different contexts of this library) race on it, so issue
 * them on one stream or order them yourself.  Nothing has to be cleared between calls (each call
 * writes every slot it later reads); after a call the array holds that call's partial sums.  The
 * summation order is fixed, so repeated calls give identical bits.  Calls no cudaMalloc / cudaFree.
 * ZGR_EINVAL: null or misaligned dev_out3, bad tensor index. */
#define ZGR_NOALLOC_MAX_TILES 8192
int zgr_tensor_norms_noalloc(zgr_ctx* ctx, uint64_t seed, int32_t tensor, double* dev_out3, void* stream);

/* Test hooks.  zgr_debug_philox writes n_blocks raw generator blocks (4 uint32 each) of stream
 * (seed, tensor, tag) starting at first_block to dev_out (device).  zgr_debug_z writes z_l(seed) as
 * fp32 (rows*cols, device): it sweeps a zeroed fp32 scratch image of the tensor with scale 1 through the
 * kernel family of the tensor's storage type, except that tensors which the sweeps serve with the tcgen05
 * kernel (16-bit storage, rank > 8) go through the legacy mma.sync kernel here, because the tcgen05 kernel
 * reads and writes 16-bit tiles only.  zgr_debug_z_tcgen05 is the hook for that kernel.
 * zgr_debug_check_device is the host-only comparison behind the "current device" check of every
 * launching call: ZGR_OK if ctx_device is a valid ordinal equal to current_device, else ZGR_EINVAL. */
int zgr_debug_philox(zgr_ctx* ctx, uint64_t seed, int32_t tensor, int32_t tag, uint64_t first_block, int64_t n_blocks,
                     uint32_t* dev_out, void* stream);
int zgr_debug_z(zgr_ctx* ctx, uint64_t seed, int32_t tensor, float* dev_out, void* stream);
int zgr_debug_check_device(int32_t ctx_device, int32_t current_device);

/* z_l(seed) as the tcgen05 sweep kernel computes it: that kernel itself (same TMA loads, tensor-core
 * products, tensor-memory reads and epilogue arithmetic as in zgr_perturb) sweeps a zeroed 16-bit image
 * of the tensor with coefficient 1, and its fp32 result for every element, taken just before the rounding
 * to the storage type, is written to dev_out (device, rows*cols fp32, 16-byte aligned).  The weights are
 * not touched.  Allocates and frees the image; synchronises `stream`.
 * ZGR_ESTATE: the sweeps do not serve this tensor with the tcgen05 kernel (fp32 storage, rank <= 8,
 * unaligned data, alpha = 1 at zgr_init, or the legacy tensor-core path was selected). */
int zgr_debug_z_tcgen05(zgr_ctx* ctx, uint64_t seed, int32_t tensor, float* dev_out, void* stream);

/* The work plan of a sweep, computed on the host alone (no device is needed or touched): which kernel
 * family serves which part of which tensor.  Test hook for the planner: the items of a plan must cover
 * every element of every tensor exactly once.  path: 0 isotropic (elements [row0_or_e0, +nrows_or_count) of
 * the tensor), otherwise rows [row0_or_e0, +nrows_or_count) x columns [col0, +ncols): 1 CUDA-core rank <= 8,
 * 2 legacy tensor-core, 3 fallback, 4 tcgen05.  `tensors[].data / U` are only inspected for alignment and
 * null-ness.  tcgen05 != 0 plans as on a device where tensor maps can be made; multi != 0 gives the plan of
 * the multi-seed sweeps.  Up to max_items items are written to out; *n_items receives the full count.
 * Errors as zgr_init (ZGR_EINVAL), plus sm_count < 1 or a null n_items. */
typedef struct {
  int32_t path, kpad, tensor, ncols;
  int64_t row0_or_e0, nrows_or_count, col0;
} zgr_plan_item;
int zgr_debug_plan(const zgr_tensor* tensors, int32_t n, const zgr_config* cfg, int32_t sm_count, int32_t tcgen05, int32_t multi,
                   zgr_plan_item* out, int64_t max_items, int64_t* n_items);

/* Per-kernel timing.  While enabled, every sweep launch is bracketed by CUDA events on its stream.
 * zgr_profile_read synchronises the device, writes one entry per kernel family that ran since the
 * last read (up to max_entries) and clears the record.  path: 0 isotropic, 1 CUDA-core rank<=8,
 * 2 tensor-core, 3 fallback; elements = weights covered by one launch. */
typedef struct {
  int32_t path, dtype, kpad, launches;
  int64_t elements;
  double ms_total;
} zgr_kernel_time;
int zgr_profile(zgr_ctx* ctx, int32_t enable);
int zgr_profile_read(zgr_ctx* ctx, zgr_kernel_time* out, int32_t max_entries, int32_t* n_entries);

/* Device-side health.  The tensor-core sweep waits on hardware barriers (TMA, tensor memory) with a
 * time limit; a wait that gives up records a non-zero code, abandons the sweep and lets the kernel
 * exit cleanly instead of hanging the GPU.  This call synchronises the device and returns that code
 * in *code (0 = healthy).  A non-zero code makes the context unusable (every later call returns
 * ZGR_ECUDA): the interrupted sweep left the weights partly updated. */
int zgr_device_status(zgr_ctx* ctx, int32_t* code);

/* Introspection: mixing scalars a, b in double; number of active seeds (0 when idle), the seed most
 * recently swept and the net coefficient still applied under it; number of kernel launches issued by
 * this context so far. */
int zgr_get_scalars(const zgr_ctx* ctx, double* a, double* b);
int zgr_get_state(const zgr_ctx* ctx, int32_t* active, uint64_t* seed, double* net_scale);
int64_t zgr_launch_count(const zgr_ctx* ctx);

void zgr_destroy(zgr_ctx* ctx);
const char* zgr_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* ZGR_H_ */
