// Host side of the ZGR library: context, validation, work planning and the C entry points
// declared in include/zgr.h.  Everything numerical happens in the kernels; the host only
// combines the step scalars in double (Eq. (grad), Eq. (perturbation)) and hands them over as fp32.
#include <cuda_runtime.h>

#include <algorithm>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <map>
#include <new>
#include <vector>

#include "zgr.h"
#include "zgr_internal.h"
#include "zgr_host_internal.h"
#include "zgr_kernels.h"
#include "zgr_subspace.h"

using namespace zgr;

namespace {

struct Group {
  KernelChoice kc;
  std::vector<WorkItem> items;
  WorkItem* d_items = nullptr;
  int grid = 0;
  int64_t elements = 0;                                   // weights covered by one launch
  double* d_item_stats = nullptr;                         // kStatSlots x 3 doubles per item (norm bookkeeping), allocated on first use
  int32_t* d_sched = nullptr;                             // CUDA-core contraction kernel: two item counters (caller's stream, library's second stream)
  std::vector<int32_t> first_item;                        // per tensor l: index of its first item in `items` (size n + 1; items are in tensor order)
  std::vector<std::pair<cudaEvent_t, cudaEvent_t>> timed;  // per-launch events while profiling is on
};

int dtype_bytes(int dt) { return dt == ZGR_F32 ? 4 : 2; }

}  // namespace

struct zgr_ctx {
  int device = 0;
  int sm_count = 0;
  zgr_config cfg{};
  double a = 0, b = 0;
  int64_t d = 0, K = 0;
  std::vector<TensorDesc> descs;      // host mirror of the device table
  TensorDesc* d_descs = nullptr;
  bool descs_dirty = false;
  std::vector<void*> owned;           // device allocations made by the library
  std::vector<Group> groups;          // sweep plan
  std::vector<WorkItem> stats_items;  // plan of the norm kernel (tensors not served by the tcgen05 kernel)
  bool stats_planned = false;
  WorkItem* d_stats_items = nullptr;
  double* d_stats_slots = nullptr;    // slots of the separate norm pass over stats_items
  std::vector<int32_t> stats_first;   // per tensor: first item in stats_items (size n + 1)
  StatRange* d_ranges_pass = nullptr; // per tensor: where the separate pass leaves its partial sums
  StatRange* d_ranges_sweep = nullptr;  // per tensor: where a sweep with bookkeeping leaves them
  bool sweep_stats_ready = false;     // slots and ranges of the sweep plan exist
  bool stats_on = false;              // zgr_config.stats / zgr_enable_stats
  bool held_valid = false;            // the slots of the sweep plan hold the norms of held_seed, scaled by held_c^2
  uint64_t held_seed = 0;
  double held_c = 0.0;
  double* d_stats = nullptr;
  std::map<uint64_t, double> ledger;  // seeds whose perturbation is applied to the weights -> sum of the coefficients applied
  uint64_t last_seed = 0;             // most recently swept seed (introspection)
  bool guided_at_init = false;        // b != 0 when the sweep plan was made
  SplitJob* d_split_jobs = nullptr;   // one job per tensor served by the tcgen05 kernel: rebuild of its operand copy of U
  int n_split_jobs = 0;
  std::vector<char> frag_stale;       // per tensor: the fragment-order copy of U (legacy tensor-core kernel) lags behind U
  std::vector<Group> groups_multi;    // plan of multi-seed sweeps when it differs from `groups` (legacy tensor-core path only)
  bool multi_planned = false;
  int sticky = 0;                     // first CUDA failure, returned by every later call
  int64_t launches = 0;
  bool profiling = false;
  CUtensorMap* d_tmaps = nullptr;     // three per tensor (theta, U hi, U lo); tcgen05 path only
  std::vector<CUtensorMap> tmaps;     // host mirror
  int* d_err = nullptr;               // set by a kernel whose bounded wait gave up
  std::vector<cudaEvent_t> layer_events;  // zgr_perturb_layers: one per layer plus two, created on first use
  cudaStream_t aux_stream = nullptr;      // zgr_perturb_layers: odd layers run here, so that one layer's tail overlaps the next one's start
  void* d_qr = nullptr;               // scratch of zgr_build_subspace (grown on demand)
  size_t qr_bytes = 0;
};

namespace {

PhiloxKeys make_keys(uint64_t seed) {
  PhiloxKeys k;
  uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    k.k0[r] = k0;
    k.k1[r] = k1;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return k;
}

NormalScale make_scale(double s, int bits) {
  const double kTwoPi = 6.283185307179586476925286766559;
  const int nb = bits == 32 ? 23 : 16;
  const double off = std::ldexp(1.0, -(nb + 1)) - 1.0;
  NormalScale ns;
  ns.kr = static_cast<float>(-2.0 * std::log(2.0) * s * s);
  ns.s = static_cast<float>(s);
  ns.phase = static_cast<float>(kTwoPi * off + (s >= 0 ? -kTwoPi : -0.5 * kTwoPi));
  ns.u1_off = static_cast<float>(off);
  return ns;
}

// Power of two that brings the coefficient strips of the tcgen05 kernel near 1: the smallest k with
// cb 2^k >= 1/2, cb = sum_q |c_q| b (0 if there is no guided part in this call).
int kshift_for(double cb) {
  if (!(cb > 0.0) || !std::isfinite(cb)) return 0;
  const int k = static_cast<int>(std::ceil(-std::log2(cb))) - 1;
  return std::min(std::max(k, -24), 40);
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                   const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// cuTensorMapEncodeTiled through the runtime (the library does not link against libcuda).
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// 2-D map over a row-major 16-bit matrix (rows x cols, row pitch = cols), box = box_cols x 128 rows,
// swizzle matching the box's row length in bytes (32, 64 or 128).
bool make_map_16bit(CUtensorMap* out, const void* base, int64_t rows, int64_t cols, int box_cols) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(box_cols), 128};
  const cuuint32_t estr[2] = {1, 1};
  const int row_bytes = box_cols * 2;
  const CUtensorMapSwizzle sw = row_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : (row_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
  return fn(out, CU_TENSOR_MAP_DATA_TYPE_UINT16, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool umma_wanted() {
  const char* e = std::getenv("ZGR_TENSOR_PATH");
  return !(e && std::strcmp(e, "legacy") == 0);
}

int blocks_per_sm(int path) {
  switch (path) {
    case PATH_ISO: return 6;
    case PATH_GENERIC: return 4;
    case PATH_UMMA: return 1;
    default: return 2;
  }
}

// Split the tensors listed in `which` into work items, grouped by the kernel that serves them.
// The kernel family follows the tensor's own storage type (fp32 tensors take the accurate transform and
// an exact fp32 contraction); `kernel_dtype` >= 0 overrides only the type the kernel reads and writes,
// which lets the test hook run a 16-bit tensor's kernel family on an fp32 image.
void plan(const std::vector<TensorDesc>& descs, const std::vector<int>& which, bool guided_on, int bits, int sm_count,
          std::vector<Group>& out, int kernel_dtype = -1, bool multi = false) {
  int64_t total = 0;
  for (int l : which) total += descs[l].rows * descs[l].cols;
  // elements per item: enough items for ~16 rounds over the resident CTAs, but large enough that the
  // coefficient strip of an item is a small fraction of its work
  int64_t target = total / (static_cast<int64_t>(sm_count) * 2 * 16);
  target = std::min<int64_t>(std::max<int64_t>(target, 16384), 524288);

  std::map<std::tuple<int, int, int, int>, size_t> index;  // (path, dtype, kpad, precise) -> group
  auto group_for = [&](int path, int real_dtype, int kpad) -> Group& {
    const int precise = real_dtype == ZGR_F32 ? 1 : 0;
    const int dtype = kernel_dtype >= 0 ? kernel_dtype : real_dtype;
    auto key = std::make_tuple(path, dtype, kpad, precise);
    auto it = index.find(key);
    if (it == index.end()) {
      index[key] = out.size();
      Group g;
      g.kc = KernelChoice{path, dtype, kpad, bits, precise};
      out.push_back(std::move(g));
      return out.back();
    }
    return out[it->second];
  };

  for (int l : which) {
    const TensorDesc& t = descs[l];
    const bool aligned = (reinterpret_cast<uintptr_t>(t.data) & 15) == 0;
    const bool guided = guided_on && t.rank > 0;
    if (!guided) {
      Group& g = group_for(PATH_ISO, t.dtype, 0);
      const int64_t n = t.rows * t.cols;
      const int64_t chunk = std::max<int64_t>(8, (target / 8) * 8);
      for (int64_t e0 = 0; e0 < n; e0 += chunk)
        g.items.push_back(WorkItem{l, aligned ? 1 : 0, e0, std::min(chunk, n - e0), 0});
      continue;
    }
    const bool vec = aligned && (t.cols % 8 == 0);
    int path, kpad, strip, row_step;
    const bool umma_ok = t.umma && kernel_dtype < 0;
    if (!vec || (t.rank > 8 && t.Ufrag == nullptr) || (multi && t.rank > 8 && !umma_ok)) {
      // (the legacy tensor-core kernel applies one term per sweep; several terms take the fallback)
      path = PATH_GENERIC; kpad = 0; strip = 64; row_step = 1;
    } else if (t.rank <= 8) {
      path = PATH_FMA; kpad = t.rank <= 4 ? 4 : 8; strip = 256; row_step = 1;
    } else if (umma_ok) {
      path = PATH_UMMA; kpad = t.kpad; strip = umma_strip_cols(kpad); row_step = 128;
    } else {
      path = PATH_MMA; kpad = t.rank <= 16 ? 16 : (t.rank <= 32 ? 32 : 64);
      strip = mma_strip_cols(kpad); row_step = mma_rows_per_iter(kpad);
    }
    Group& g = group_for(path, t.dtype, kpad);
    for (int64_t c0 = 0; c0 < t.cols; c0 += strip) {
      const int ncols = static_cast<int>(std::min<int64_t>(strip, t.cols - c0));
      // (the CUDA-core contraction kernel hands its items out dynamically and regenerates its coefficient strip per item:
      //  larger items there; the tcgen05 kernel's items are two tiles wide)
      int64_t nrows = std::max<int64_t>(1, (path == PATH_UMMA || path == PATH_FMA ? 2 * target : target) / ncols);
      nrows = ((nrows + row_step - 1) / row_step) * row_step;
      // even out the chunks of this strip
      const int64_t n_chunks = (t.rows + nrows - 1) / nrows;
      nrows = (t.rows + n_chunks - 1) / n_chunks;
      nrows = ((nrows + row_step - 1) / row_step) * row_step;
      for (int64_t r0 = 0; r0 < t.rows; r0 += nrows)
        g.items.push_back(WorkItem{l, ncols, r0, std::min(nrows, t.rows - r0), c0});
    }
  }
  for (Group& g : out) {
    g.elements = 0;
    for (const WorkItem& w : g.items) g.elements += g.kc.path == PATH_ISO ? w.nrows_or_count : w.nrows_or_count * w.ncols;
  }
  for (Group& g : out) g.grid = static_cast<int>(std::min<int64_t>(static_cast<int64_t>(g.items.size()), static_cast<int64_t>(sm_count) * blocks_per_sm(g.kc.path)));
  // tensors were visited in ascending order, so each tensor's items are contiguous within its group
  for (Group& g : out) {
    g.first_item.assign(descs.size() + 1, static_cast<int32_t>(g.items.size()));
    for (size_t i = g.items.size(); i-- > 0;) g.first_item[static_cast<size_t>(g.items[i].tensor)] = static_cast<int32_t>(i);
    for (size_t l = descs.size(); l-- > 0;)
      if (g.first_item[l] > g.first_item[l + 1]) g.first_item[l] = g.first_item[l + 1];   // tensors without items in this group
    // (after the two passes first_item is non-decreasing and [first_item[l], first_item[l+1]) are the items of tensor l)
  }
}

int check(zgr_ctx* ctx, cudaError_t e) {
  if (e == cudaSuccess) return ZGR_OK;
  const int code = (e == cudaErrorMemoryAllocation) ? ZGR_ENOMEM : ZGR_ECUDA;
  if (ctx && ctx->sticky == 0) ctx->sticky = code;
  return code;
}

template <typename T>
int dev_alloc(zgr_ctx* ctx, T** p, size_t count) {
  void* q = nullptr;
  const int rc = check(ctx, cudaMalloc(&q, std::max<size_t>(count, 1) * sizeof(T)));
  if (rc != ZGR_OK) return rc;
  ctx->owned.push_back(q);
  *p = static_cast<T*>(q);
  return ZGR_OK;
}

int upload_groups(zgr_ctx* ctx, std::vector<Group>& groups) {
  for (Group& g : groups) {
    if (g.items.empty()) continue;
    int rc = dev_alloc(ctx, &g.d_items, g.items.size());
    if (rc != ZGR_OK) return rc;
    rc = check(ctx, cudaMemcpy(g.d_items, g.items.data(), g.items.size() * sizeof(WorkItem), cudaMemcpyHostToDevice));
    if (rc != ZGR_OK) return rc;
    if (g.kc.path == PATH_FMA) {
      rc = dev_alloc(ctx, &g.d_sched, 2);
      if (rc != ZGR_OK) return rc;
      rc = check(ctx, cudaMemset(g.d_sched, 0, 2 * sizeof(int32_t)));
      if (rc != ZGR_OK) return rc;
    }
  }
  // the copies and the zeroing above are not ordered with launches on the caller's (possibly non-blocking) streams
  return check(ctx, cudaDeviceSynchronize());
}

// One sweep  theta <- rnd(theta + sum_q c_q z(seed_q))  over the planned groups (n terms, 1 <= n <= kMaxTerms).
// t0 <= t1 restricts the sweep to the tensors [t0, t1) (layer-wise sweeps); t1 < 0 means all of them.
int sweep(zgr_ctx* ctx, std::vector<Group>& groups, const TensorDesc* d_descs, int n, const uint64_t* seeds, const double* c, cudaStream_t st,
          int32_t t0 = 0, int32_t t1 = -1, bool keep_stats = false) {
  SweepParams p;
  std::memset(&p, 0, sizeof(p));
  for (int q = 0; q < n; ++q) {
    p.term[q].keys = make_keys(seeds[q]);
    p.term[q].iso = make_scale(c[q] * ctx->a, ctx->cfg.bits_per_normal);
    p.term[q].cb = static_cast<float>(c[q] * ctx->b);
  }
  p.n_terms = n;
  p.unit = make_scale(1.0, ctx->cfg.bits_per_normal);
  p.tensors = d_descs;
  double cb_total = 0.0;
  for (int q = 0; q < n; ++q) cb_total += std::fabs(c[q] * ctx->b);
  p.kshift = kshift_for(cb_total);
  for (Group& g : groups) {
    if (g.items.empty()) continue;
    p.items = g.d_items;
    p.n_items = static_cast<int32_t>(g.items.size());
    p.item_stats = keep_stats ? g.d_item_stats : nullptr;
    p.item_base = 0;
    p.sched = g.d_sched ? g.d_sched + (ctx->aux_stream != nullptr && st == ctx->aux_stream ? 1 : 0) : nullptr;
    int grid = g.grid;
    if (t1 >= 0) {
      const int32_t b0 = g.first_item[static_cast<size_t>(t0)], b1 = g.first_item[static_cast<size_t>(t1)];
      if (b1 <= b0) continue;
      p.items = g.d_items + b0;
      p.n_items = b1 - b0;
      p.item_base = b0;
      grid = static_cast<int>(std::min<int64_t>(p.n_items, static_cast<int64_t>(ctx->sm_count) * blocks_per_sm(g.kc.path)));
    }
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (ctx->profiling && t1 < 0) {
      if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) {
        if (e0) cudaEventDestroy(e0);
        return check(ctx, cudaErrorUnknown);
      }
      cudaEventRecord(e0, st);
    }
    const int rc = check(ctx, g.kc.path == PATH_UMMA ? launch_sweep_umma(g.kc, p, ctx->d_tmaps, ctx->d_err, grid, st)
                                                     : launch_sweep(g.kc, p, grid, st));
    if (rc != ZGR_OK) {
      if (e0) cudaEventDestroy(e0);
      if (e1) cudaEventDestroy(e1);
      return rc;
    }
    if (e0) {
      cudaEventRecord(e1, st);
      g.timed.emplace_back(e0, e1);
    }
    ctx->launches++;
  }
  return ZGR_OK;
}

int flush_descs(zgr_ctx* ctx, cudaStream_t st) {
  if (!ctx->descs_dirty) return ZGR_OK;
  const int rc = check(ctx, cudaMemcpyAsync(ctx->d_descs, ctx->descs.data(), ctx->descs.size() * sizeof(TensorDesc), cudaMemcpyHostToDevice, st));
  if (rc == ZGR_OK) ctx->descs_dirty = false;
  return rc;
}

bool is_finite(double x) { return std::isfinite(x); }

// Rebuild the library's operand copies of U for one tensor from the subspace buffer (enqueued on st).
int refresh_operands(zgr_ctx* ctx, int32_t tensor, cudaStream_t st) {
  TensorDesc& td = ctx->descs[static_cast<size_t>(tensor)];
  int rc = ZGR_OK;
  if (td.Ufrag != nullptr) {
    if (td.umma) {
      // the sweeps of this tensor read the row-major copy below; the fragment-order copy is only needed by
      // zgr_debug_z and is rebuilt there on demand
      ctx->frag_stale[static_cast<size_t>(tensor)] = 1;
    } else {
      rc = check(ctx, launch_split_subspace(td.U, td.rows, td.rank, td.kpad, const_cast<uint4*>(td.Ufrag), st));
      if (rc == ZGR_OK) ctx->launches++;
    }
  }
  if (rc == ZGR_OK && td.umma) {
    const int64_t rows_pad = ((td.rows + 127) / 128) * 128;
    rc = check(ctx, launch_split_subspace_rowmajor(td.U, td.rows, td.rank, td.kpad, rows_pad, td.ushift, td.Uhi, td.Ulo, st));
    if (rc == ZGR_OK) ctx->launches++;
  }
  return rc;
}

// Bookkeeping slots of a plan: kStatSlots x 3 doubles per work item, zeroed once (slots that no warp owns stay
// zero; the others are rewritten by every launch that keeps the bookkeeping).
int alloc_slots(zgr_ctx* ctx, double** out, size_t n_items) {
  const size_t count = std::max<size_t>(n_items, 1) * kStatSlots * 3;
  int rc = dev_alloc(ctx, out, count);
  if (rc == ZGR_OK) rc = check(ctx, cudaMemset(*out, 0, count * sizeof(double)));
  return rc;
}

// In-sweep bookkeeping needs every group of the sweep plan to be a kernel family that keeps it.
bool sweep_stats_possible(const zgr_ctx* ctx) {
  for (const Group& g : ctx->groups)
    if (!g.items.empty() && g.kc.path == PATH_MMA) return false;
  return true;
}

int prepare_sweep_stats(zgr_ctx* ctx) {
  if (ctx->sweep_stats_ready) return ZGR_OK;
  const size_t n = ctx->descs.size();
  std::vector<StatRange> ranges(n, StatRange{nullptr, 0, 0});
  for (Group& g : ctx->groups) {
    if (g.items.empty()) continue;
    const int rc = alloc_slots(ctx, &g.d_item_stats, g.items.size());
    if (rc != ZGR_OK) return rc;
    for (size_t l = 0; l < n; ++l)
      if (g.first_item[l + 1] > g.first_item[l]) ranges[l] = StatRange{g.d_item_stats, g.first_item[l], g.first_item[l + 1] - g.first_item[l]};
  }
  int rc = dev_alloc(ctx, &ctx->d_ranges_sweep, n);
  if (rc == ZGR_OK) rc = check(ctx, cudaMemcpy(ctx->d_ranges_sweep, ranges.data(), n * sizeof(StatRange), cudaMemcpyHostToDevice));
  if (rc == ZGR_OK) ctx->sweep_stats_ready = true;
  return rc;
}

// A context's tables, tensor maps and borrowed pointers live on the device that was current at zgr_init.
// Launching from another current device would hand its kernels foreign addresses, so every entry point
// that enqueues work checks this first and refuses before anything is launched.
bool on_ctx_device(const zgr_ctx* ctx) {
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess) return false;
  return zgr_debug_check_device(ctx->device, cur) == ZGR_OK;
}

// Mixing scalars of Eq. (perturbation) with n := d and m := K
void set_mixing(zgr_ctx* ctx, double alpha) {
  const double d = static_cast<double>(ctx->d), K = static_cast<double>(ctx->K);
  ctx->cfg.alpha = alpha;
  ctx->a = std::sqrt(alpha / d);
  ctx->b = ctx->K > 0 ? std::sqrt((1.0 - alpha) / K) : 0.0;
  if (ctx->cfg.scale_mode == ZGR_SCALE_UNIT) {
    ctx->a *= std::sqrt(d);
    ctx->b *= std::sqrt(d);
  }
}

// Argument checks shared by zgr_init and zgr_debug_plan; d = parameters, K = guided coefficients.
int validate_model(const zgr_tensor* tensors, int32_t n, const zgr_config* cfg, int64_t* d_out, int64_t* K_out) {
  if (!tensors || !cfg || n <= 0) return ZGR_EINVAL;
  if (!(cfg->alpha >= 0.0 && cfg->alpha <= 1.0) || !is_finite(cfg->eps) || !(cfg->eps > 0.0)) return ZGR_EINVAL;
  if (cfg->scale_mode != ZGR_SCALE_PAPER && cfg->scale_mode != ZGR_SCALE_UNIT) return ZGR_EINVAL;
  if (cfg->bits_per_normal != 32 && cfg->bits_per_normal != 16) return ZGR_EINVAL;
  int64_t d = 0, K = 0;
  for (int32_t l = 0; l < n; ++l) {
    const zgr_tensor& t = tensors[l];
    if (!t.data || t.rows < 1 || t.cols < 1) return ZGR_EINVAL;
    if (t.dtype != ZGR_F32 && t.dtype != ZGR_F16 && t.dtype != ZGR_BF16) return ZGR_EINVAL;
    if (t.rank < 0 || t.rank > ZGR_MAX_RANK) return ZGR_EINVAL;
    if ((t.rank == 0) != (t.U == nullptr)) return ZGR_EINVAL;
    if (reinterpret_cast<uintptr_t>(t.data) % dtype_bytes(t.dtype) != 0) return ZGR_EINVAL;
    if (t.U && reinterpret_cast<uintptr_t>(t.U) % 4 != 0) return ZGR_EINVAL;
    if (t.rows > (INT64_MAX / t.cols)) return ZGR_EINVAL;
    d += t.rows * t.cols;
    K += static_cast<int64_t>(t.rank) * t.cols;
  }
  *d_out = d;
  *K_out = K;
  return ZGR_OK;
}

// Book-keeping of the coefficients applied under each seed; a seed whose coefficients cancel is idle again.
void ledger_add(zgr_ctx* ctx, uint64_t seed, double c) {
  double& net = ctx->ledger[seed];
  net += c;
  if (net == 0.0) ctx->ledger.erase(seed);
  ctx->last_seed = seed;
}

// Plan used by sweeps with several terms: the sweep plan itself unless it contains the legacy
// tensor-core kernel, which applies one term per sweep; those tensors are re-planned onto the fallback.
std::vector<Group>& multi_groups(zgr_ctx* ctx, int* rc) {
  *rc = ZGR_OK;
  bool legacy = false;
  for (const Group& g : ctx->groups) legacy = legacy || (g.kc.path == PATH_MMA && !g.items.empty());
  if (!legacy) return ctx->groups;
  if (!ctx->multi_planned) {
    std::vector<int> all(ctx->descs.size());
    for (size_t l = 0; l < all.size(); ++l) all[l] = static_cast<int>(l);
    plan(ctx->descs, all, ctx->guided_at_init, ctx->cfg.bits_per_normal, ctx->sm_count, ctx->groups_multi, -1, true);
    *rc = upload_groups(ctx, ctx->groups_multi);
    ctx->multi_planned = true;
  }
  return ctx->groups_multi;
}

}  // namespace

namespace zgr {
PhiloxKeys host_make_keys(uint64_t seed) { return make_keys(seed); }
NormalScale host_make_scale(double s, int bits) { return make_scale(s, bits); }
bool host_ctx_view(const zgr_ctx* ctx, int32_t l, TensorDesc* desc, double* a, double* b, int* bits, int* sticky, int* device) {
  if (!ctx || l < 0 || l >= static_cast<int32_t>(ctx->descs.size())) return false;
  *desc = ctx->descs[static_cast<size_t>(l)];
  *a = ctx->a;
  *b = ctx->b;
  *bits = ctx->cfg.bits_per_normal;
  *sticky = ctx->sticky;
  *device = ctx->device;
  return true;
}
}  // namespace zgr

// ------------------------------------------------------------------------------------------------
extern "C" {

int zgr_init(zgr_ctx** out, const zgr_tensor* tensors, int32_t n, const zgr_config* cfg) {
  if (!out) return ZGR_EINVAL;
  *out = nullptr;
  int64_t d = 0, K = 0;
  const int valid = validate_model(tensors, n, cfg, &d, &K);
  if (valid != ZGR_OK) return valid;

  zgr_ctx* ctx = new (std::nothrow) zgr_ctx();
  if (!ctx) return ZGR_ENOMEM;
  ctx->cfg = *cfg;
  ctx->stats_on = cfg->stats != 0;
  ctx->d = d;
  ctx->K = K;
  set_mixing(ctx, cfg->alpha);

  int rc = check(ctx, cudaGetDevice(&ctx->device));
  if (rc == ZGR_OK) rc = check(ctx, cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device));
  if (rc != ZGR_OK) {
    delete ctx;
    return rc;
  }

  ctx->descs.resize(static_cast<size_t>(n));
  ctx->frag_stale.assign(static_cast<size_t>(n), 0);
  ctx->tmaps.resize(static_cast<size_t>(3 * n));
  std::memset(ctx->tmaps.data(), 0, ctx->tmaps.size() * sizeof(CUtensorMap));
  const bool guided_on = ctx->b != 0.0;
  ctx->guided_at_init = guided_on;
  for (int32_t l = 0; l < n && rc == ZGR_OK; ++l) {
    const zgr_tensor& t = tensors[l];
    TensorDesc& td = ctx->descs[static_cast<size_t>(l)];
    td.data = t.data;
    td.U = t.U;
    td.Ufrag = nullptr;
    td.q = nullptr;
    td.qscale = nullptr;
    td.qzero = nullptr;
    td.qbits = 8;
    td.qrows = 0;
    td.rows = t.rows;
    td.cols = t.cols;
    td.rank = t.rank;
    td.kpad = 0;
    td.id = l;
    td.dtype = t.dtype;
    td.umma = 0;
    td.ushift = 0;
    td.Uhi = nullptr;
    td.Ulo = nullptr;
    const bool vec = (reinterpret_cast<uintptr_t>(t.data) & 15) == 0 && (t.cols % 8 == 0);
    if (guided_on && t.rank > 8 && vec && t.dtype != ZGR_F32) {
      // tensor-core path: library-owned copy of U in A-fragment order
      td.kpad = t.rank <= 16 ? 16 : (t.rank <= 32 ? 32 : 64);
      const int64_t tiles = (t.rows + 15) / 16;
      const size_t n_frag = static_cast<size_t>(tiles) * (td.kpad / 16) * 2 * 32;
      uint4* frag = nullptr;
      rc = dev_alloc(ctx, &frag, n_frag);
      if (rc == ZGR_OK) rc = check(ctx, launch_split_subspace(t.U, t.rows, t.rank, td.kpad, frag, nullptr));
      if (rc == ZGR_OK) ctx->launches++;
      td.Ufrag = frag;
      // tcgen05 + TMA path: row-major hi/lo copies of U and three tensor maps
      if (rc == ZGR_OK && umma_wanted() && encode_tiled_fn() != nullptr && t.rows < (int64_t{1} << 31) - 256 && t.cols < (int64_t{1} << 31) - 256) {
        const int64_t rows_pad = ((t.rows + 127) / 128) * 128;
        // entries of an orthonormal U are about 1/sqrt(rows): scaled by 2^ushift they sit between 1 and 2 in size
        // (capped at 2^12, which leaves fp16 room for entries up to 16 in size)
        td.ushift = std::min<int32_t>(12, static_cast<int32_t>(std::ceil(0.5 * std::log2(static_cast<double>(t.rows)))));
        uint16_t *hi = nullptr, *lo = nullptr;
        rc = dev_alloc(ctx, &hi, static_cast<size_t>(rows_pad) * td.kpad);
        if (rc == ZGR_OK) rc = dev_alloc(ctx, &lo, static_cast<size_t>(rows_pad) * td.kpad);
        if (rc == ZGR_OK) rc = check(ctx, launch_split_subspace_rowmajor(t.U, t.rows, t.rank, td.kpad, rows_pad, td.ushift, hi, lo, nullptr));
        if (rc == ZGR_OK) {
          ctx->launches++;
          CUtensorMap* m = &ctx->tmaps[static_cast<size_t>(3 * l)];
          if (make_map_16bit(m, t.data, t.rows, t.cols, 64) && make_map_16bit(m + 1, hi, rows_pad, td.kpad, td.kpad) &&
              make_map_16bit(m + 2, lo, rows_pad, td.kpad, td.kpad)) {
            td.umma = 1;
            td.Uhi = hi;
            td.Ulo = lo;
          }
        }
      }
    }
  }
  if (rc == ZGR_OK) {
    std::vector<SplitJob> jobs;
    for (const TensorDesc& td : ctx->descs)
      if (td.umma) jobs.push_back(SplitJob{td.U, td.Uhi, td.Ulo, td.rows, ((td.rows + 127) / 128) * 128, td.rank, td.kpad, td.ushift});
    ctx->n_split_jobs = static_cast<int>(jobs.size());
    if (!jobs.empty()) {
      rc = dev_alloc(ctx, &ctx->d_split_jobs, jobs.size());
      if (rc == ZGR_OK) rc = check(ctx, cudaMemcpy(ctx->d_split_jobs, jobs.data(), jobs.size() * sizeof(SplitJob), cudaMemcpyHostToDevice));
    }
  }
  if (rc == ZGR_OK) rc = dev_alloc(ctx, &ctx->d_tmaps, ctx->tmaps.size());
  if (rc == ZGR_OK) rc = check(ctx, cudaMemcpy(ctx->d_tmaps, ctx->tmaps.data(), ctx->tmaps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice));
  if (rc == ZGR_OK) rc = dev_alloc(ctx, &ctx->d_err, 1);
  if (rc == ZGR_OK) rc = check(ctx, cudaMemset(ctx->d_err, 0, sizeof(int)));
  if (rc == ZGR_OK) rc = dev_alloc(ctx, &ctx->d_descs, ctx->descs.size());
  if (rc == ZGR_OK) rc = check(ctx, cudaMemcpy(ctx->d_descs, ctx->descs.data(), ctx->descs.size() * sizeof(TensorDesc), cudaMemcpyHostToDevice));
  if (rc == ZGR_OK) {
    std::vector<int> all(static_cast<size_t>(n));
    for (int32_t l = 0; l < n; ++l) all[static_cast<size_t>(l)] = l;
    plan(ctx->descs, all, guided_on, cfg->bits_per_normal, ctx->sm_count, ctx->groups);
    rc = upload_groups(ctx, ctx->groups);
  }
  if (rc == ZGR_OK) rc = dev_alloc(ctx, &ctx->d_stats, static_cast<size_t>(3 * n));
  if (rc == ZGR_OK) rc = check(ctx, cudaDeviceSynchronize());  // the subspace copies are complete
  if (rc != ZGR_OK) {
    zgr_destroy(ctx);
    return rc;
  }
  ctx->sticky = 0;
  *out = ctx;
  return ZGR_OK;
}

int zgr_perturb(zgr_ctx* ctx, uint64_t seed, double scale, void* stream) {
  if (!ctx || !is_finite(scale)) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  if (!ctx->ledger.empty() && !(ctx->ledger.size() == 1 && ctx->ledger.count(seed) == 1)) return ZGR_ESTATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = flush_descs(ctx, st);
  if (rc != ZGR_OK) return rc;
  // the first perturbation under a seed also keeps the norm bookkeeping when that is switched on
  const bool keep = ctx->stats_on && ctx->ledger.empty() && scale != 0.0 && sweep_stats_possible(ctx);
  if (keep) {
    rc = prepare_sweep_stats(ctx);
    if (rc != ZGR_OK) return rc;
    ctx->held_valid = false;
  }
  rc = sweep(ctx, ctx->groups, ctx->d_descs, 1, &seed, &scale, st, 0, -1, keep);
  if (rc != ZGR_OK) return rc;
  if (keep) {
    ctx->held_valid = true;
    ctx->held_seed = seed;
    ctx->held_c = scale;
  }
  ledger_add(ctx, seed, scale);
  return ZGR_OK;
}

int zgr_restore_update(zgr_ctx* ctx, uint64_t seed, double loss_plus, double loss_minus, double lr, void* stream) {
  if (!ctx || !is_finite(loss_plus) || !is_finite(loss_minus) || !is_finite(lr)) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  const auto active = ctx->ledger.find(seed);
  if (active == ctx->ledger.end()) return ZGR_ESTATE;
  // Eq. (grad): projected gradient; Algorithm 1 "Update": W <- W - eta g z, fused with the restore
  const double g = (loss_plus - loss_minus) / (2.0 * ctx->cfg.eps);
  const double c = -active->second - lr * g;
  if (!is_finite(c)) return ZGR_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = flush_descs(ctx, st);
  if (rc != ZGR_OK) return rc;
  rc = sweep(ctx, ctx->groups, ctx->d_descs, 1, &seed, &c, st);
  if (rc != ZGR_OK) return rc;
  ctx->ledger.erase(seed);
  ctx->last_seed = seed;
  return ZGR_OK;
}

int zgr_sweep_multi(zgr_ctx* ctx, int32_t n, const uint64_t* seeds, const double* coeffs, void* stream) {
  if (!ctx || !seeds || !coeffs || n < 1 || n > ZGR_MAX_SEEDS) return ZGR_EINVAL;
  for (int32_t i = 0; i < n; ++i) {
    if (!is_finite(coeffs[i])) return ZGR_EINVAL;
    for (int32_t j = 0; j < i; ++j)
      if (seeds[j] == seeds[i]) return ZGR_EINVAL;
  }
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = flush_descs(ctx, st);
  if (rc != ZGR_OK) return rc;
  std::vector<Group>& groups = n > 1 ? multi_groups(ctx, &rc) : ctx->groups;
  if (rc != ZGR_OK) return rc;
  rc = sweep(ctx, groups, ctx->d_descs, n, seeds, coeffs, st);
  if (rc != ZGR_OK) return rc;
  for (int32_t i = 0; i < n; ++i) ledger_add(ctx, seeds[i], coeffs[i]);
  return ZGR_OK;
}

int zgr_restore_update_multi(zgr_ctx* ctx, int32_t n, const uint64_t* seeds, const double* loss_plus, const double* loss_minus, double lr,
                             void* stream) {
  if (!ctx || !seeds || !loss_plus || !loss_minus || n < 1 || n > ZGR_MAX_SEEDS || !is_finite(lr)) return ZGR_EINVAL;
  double c[ZGR_MAX_SEEDS];
  for (int32_t i = 0; i < n; ++i) {
    if (!is_finite(loss_plus[i]) || !is_finite(loss_minus[i])) return ZGR_EINVAL;
    for (int32_t j = 0; j < i; ++j)
      if (seeds[j] == seeds[i]) return ZGR_EINVAL;
    // Eq. (grad) per seed; Algorithm 1 "Recover gradient" sums g_t z_t over the seeds, "Update" applies it
    const double g = (loss_plus[i] - loss_minus[i]) / (2.0 * ctx->cfg.eps);
    const auto it = ctx->ledger.find(seeds[i]);
    c[i] = -(it == ctx->ledger.end() ? 0.0 : it->second) - lr * g;
    if (!is_finite(c[i])) return ZGR_EINVAL;
  }
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = flush_descs(ctx, st);
  if (rc != ZGR_OK) return rc;
  std::vector<Group>& groups = n > 1 ? multi_groups(ctx, &rc) : ctx->groups;
  if (rc != ZGR_OK) return rc;
  rc = sweep(ctx, groups, ctx->d_descs, n, seeds, c, st);
  if (rc != ZGR_OK) return rc;
  for (int32_t i = 0; i < n; ++i) ctx->ledger.erase(seeds[i]);
  ctx->last_seed = seeds[n - 1];
  return ZGR_OK;
}

int zgr_set_alpha(zgr_ctx* ctx, double alpha) {
  if (!ctx || !(alpha >= 0.0 && alpha <= 1.0)) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!ctx->ledger.empty()) return ZGR_ESTATE;
  // The kernels serving each tensor were chosen at zgr_init; a context built with alpha = 1 (no guided
  // part at all) has no tensor-core operands and keeps serving every tensor without its subspace.
  if (ctx->guided_at_init == false && alpha < 1.0 && ctx->K > 0) return ZGR_ESTATE;
  set_mixing(ctx, alpha);
  ctx->held_valid = false;
  return ZGR_OK;
}

int zgr_adapt_alpha(zgr_ctx* ctx, const double* stats, double alpha_min, double alpha_max, double eta, double* alpha_out) {
  if (!ctx || !stats || !alpha_out) return ZGR_EINVAL;
  if (!(alpha_min >= 0.0 && alpha_min <= alpha_max && alpha_max <= 1.0) || !(eta >= 0.0 && eta <= 1.0)) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!ctx->ledger.empty()) return ZGR_ESTATE;
  const double alpha_old = ctx->cfg.alpha;
  *alpha_out = alpha_old;
  // Energy of each part per unit of its mixing weight, from the norms measured under the current (a, b):
  // sum (a Z)^2 / a^2 per parameter and sum (b U G)^2 / b^2 per guided coefficient.  Eq. (perturbation) gives
  // the parts the weights alpha/d and (1 - alpha)/K (times d in the unit normalisation), so their energies
  // are equal where alpha / (1 - alpha) = e_g / e_iso.  A part that is switched off cannot be measured:
  // the ratio then stays as it is.
  if (ctx->a == 0.0 || ctx->b == 0.0 || ctx->K == 0) return ZGR_OK;
  double iso = 0.0, guided = 0.0;
  for (size_t l = 0; l < ctx->descs.size(); ++l) {
    if (!is_finite(stats[3 * l]) || !is_finite(stats[3 * l + 1]) || stats[3 * l] < 0.0 || stats[3 * l + 1] < 0.0) return ZGR_EINVAL;
    iso += stats[3 * l];
    guided += stats[3 * l + 1];
  }
  const double e_iso = iso / (ctx->a * ctx->a) / static_cast<double>(ctx->d);
  const double e_g = guided / (ctx->b * ctx->b) / static_cast<double>(ctx->K);
  if (!(e_iso + e_g > 0.0)) return ZGR_OK;
  double alpha = (1.0 - eta) * alpha_old + eta * (e_g / (e_iso + e_g));
  alpha = std::min(std::max(alpha, alpha_min), alpha_max);
  set_mixing(ctx, alpha);
  ctx->held_valid = false;
  *alpha_out = alpha;
  return ZGR_OK;
}

int zgr_set_coeffs_dtc_rows(zgr_ctx* ctx, int32_t tensor, const int8_t* q, const float* scale, const float* zero, int32_t bits, int32_t n_rows) {
  if (!ctx || tensor < 0 || tensor >= static_cast<int32_t>(ctx->descs.size())) return ZGR_EINVAL;
  if (!q || !scale || (bits != 8 && bits != 4)) return ZGR_EINVAL;
  TensorDesc& td = ctx->descs[static_cast<size_t>(tensor)];
  if (td.rank == 0 || n_rows < 1 || n_rows > td.rank) return ZGR_EINVAL;
  if (!ctx->ledger.empty()) return ZGR_ESTATE;
  td.q = q;
  td.qscale = scale;
  td.qzero = zero;
  td.qbits = bits;
  td.qrows = n_rows;
  ctx->descs_dirty = true;
  ctx->held_valid = false;
  return ZGR_OK;
}

int zgr_set_coeffs_dtc(zgr_ctx* ctx, int32_t tensor, const int8_t* q, const float* scale, const float* zero, int32_t bits) {
  if (!ctx || tensor < 0 || tensor >= static_cast<int32_t>(ctx->descs.size())) return ZGR_EINVAL;
  return zgr_set_coeffs_dtc_rows(ctx, tensor, q, scale, zero, bits, ctx->descs[static_cast<size_t>(tensor)].rank);
}

int zgr_perturb_layers(zgr_ctx* ctx, uint64_t seed, double scale, int32_t n_layers, const int32_t* layer_end, int32_t n_deliveries,
                       const zgr_coeff_delivery* deliveries, void* stream, void* copy_stream) {
  if (!ctx || !is_finite(scale) || n_layers < 1 || !layer_end || n_deliveries < 0 || (n_deliveries > 0 && !deliveries)) return ZGR_EINVAL;
  const int32_t n = static_cast<int32_t>(ctx->descs.size());
  for (int32_t L = 0; L < n_layers; ++L)
    if (layer_end[L] <= (L ? layer_end[L - 1] : 0) || layer_end[L] > n) return ZGR_EINVAL;
  if (layer_end[n_layers - 1] != n) return ZGR_EINVAL;
  // which layer each delivery belongs to; every delivery must name a tensor whose compressed coefficients are set
  std::vector<std::vector<int32_t>> by_layer(static_cast<size_t>(n_layers));
  std::vector<char> seen(static_cast<size_t>(n), 0);
  for (int32_t i = 0; i < n_deliveries; ++i) {
    const zgr_coeff_delivery& d = deliveries[i];
    if (d.tensor < 0 || d.tensor >= n || seen[static_cast<size_t>(d.tensor)] || (!d.q && !d.U)) return ZGR_EINVAL;
    seen[static_cast<size_t>(d.tensor)] = 1;
    const TensorDesc& td = ctx->descs[static_cast<size_t>(d.tensor)];
    if (d.q && (!d.scale || td.q == nullptr || (d.zero != nullptr) != (td.qzero != nullptr))) return ZGR_EINVAL;
    if (!d.q && (d.scale || d.zero)) return ZGR_EINVAL;
    if (d.U && td.rank == 0) return ZGR_EINVAL;
    const int32_t L = static_cast<int32_t>(std::upper_bound(layer_end, layer_end + n_layers, d.tensor) - layer_end);
    by_layer[static_cast<size_t>(L)].push_back(i);
  }
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  if (!ctx->ledger.empty() && (n_deliveries > 0 || !(ctx->ledger.size() == 1 && ctx->ledger.count(seed) == 1))) return ZGR_ESTATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream), cs = static_cast<cudaStream_t>(copy_stream);
  int rc = flush_descs(ctx, st);
  if (rc != ZGR_OK) return rc;
  if (!ctx->aux_stream) {
    rc = check(ctx, cudaStreamCreateWithFlags(&ctx->aux_stream, cudaStreamNonBlocking));
    if (rc != ZGR_OK) return rc;
  }
  while (ctx->layer_events.size() < static_cast<size_t>(n_layers) + 2) {
    cudaEvent_t e = nullptr;
    rc = check(ctx, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    if (rc != ZGR_OK) return rc;
    ctx->layer_events.push_back(e);
  }
  if (n_deliveries > 0) {
    // The copies may not overtake work already enqueued on `stream` that still reads the destination buffers.
    rc = check(ctx, cudaEventRecord(ctx->layer_events[static_cast<size_t>(n_layers)], st));
    if (rc == ZGR_OK) rc = check(ctx, cudaStreamWaitEvent(cs, ctx->layer_events[static_cast<size_t>(n_layers)], 0));
    if (rc != ZGR_OK) return rc;
    // All copies are enqueued up front, layer by layer: the copy engine runs ahead of the sweeps as far as it can,
    // so layer l + 1 (and later ones) travel while layer l is swept (Sec. 3.3).
    for (int32_t L = 0; L < n_layers; ++L) {
      if (by_layer[static_cast<size_t>(L)].empty()) continue;
      for (int32_t i : by_layer[static_cast<size_t>(L)]) {
        const zgr_coeff_delivery& d = deliveries[i];
        const TensorDesc& td = ctx->descs[static_cast<size_t>(d.tensor)];
        const size_t row_bytes = td.qbits == 4 ? static_cast<size_t>((td.cols + 1) / 2) : static_cast<size_t>(td.cols);
        if (d.q) {
          rc = check(ctx, cudaMemcpyAsync(const_cast<int8_t*>(td.q), d.q, row_bytes * static_cast<size_t>(td.qrows), cudaMemcpyHostToDevice, cs));
          if (rc == ZGR_OK)
            rc = check(ctx, cudaMemcpyAsync(const_cast<float*>(td.qscale), d.scale, sizeof(float) * static_cast<size_t>(td.qrows), cudaMemcpyHostToDevice, cs));
          if (rc == ZGR_OK && d.zero)
            rc = check(ctx, cudaMemcpyAsync(const_cast<float*>(td.qzero), d.zero, sizeof(float) * static_cast<size_t>(td.qrows), cudaMemcpyHostToDevice, cs));
        }
        if (rc == ZGR_OK && d.U)
          rc = check(ctx, cudaMemcpyAsync(const_cast<float*>(td.U), d.U, sizeof(float) * static_cast<size_t>(td.rows) * td.rank, cudaMemcpyHostToDevice, cs));
        if (rc != ZGR_OK) return rc;
      }
      rc = check(ctx, cudaEventRecord(ctx->layer_events[static_cast<size_t>(L)], cs));
      if (rc != ZGR_OK) return rc;
    }
  }
  const bool keep = ctx->stats_on && ctx->ledger.empty() && scale != 0.0 && sweep_stats_possible(ctx);
  if (keep) {
    rc = prepare_sweep_stats(ctx);
    if (rc != ZGR_OK) return rc;
  }
  ctx->held_valid = false;     // (a delivery changes the coefficients that earlier norms were taken with)
  // Layers touch disjoint tensors, so consecutive layers need no ordering between them: even layers run on the
  // caller's stream, odd ones on a stream of the library's, and the blocks of one layer's kernels start on the
  // SMs that the previous layer's last blocks have not reached any more.  The library's stream starts behind the
  // work already on the caller's stream, and the caller's stream ends by waiting for it.
  cudaEvent_t ev_begin = ctx->layer_events[static_cast<size_t>(n_layers) + 1];
  rc = check(ctx, cudaEventRecord(ev_begin, st));
  if (rc == ZGR_OK) rc = check(ctx, cudaStreamWaitEvent(ctx->aux_stream, ev_begin, 0));
  if (rc != ZGR_OK) return rc;
  for (int32_t L = 0; L < n_layers; ++L) {
    cudaStream_t ls = (L & 1) ? ctx->aux_stream : st;
    if (n_deliveries > 0 && !by_layer[static_cast<size_t>(L)].empty()) {
      rc = check(ctx, cudaStreamWaitEvent(ls, ctx->layer_events[static_cast<size_t>(L)], 0));
      if (rc != ZGR_OK) return rc;
      for (int32_t i : by_layer[static_cast<size_t>(L)])
        if (deliveries[i].U) {
          rc = refresh_operands(ctx, deliveries[i].tensor, ls);   // the delivered subspace, split for the tensor cores
          if (rc != ZGR_OK) return rc;
        }
    }
    rc = sweep(ctx, ctx->groups, ctx->d_descs, 1, &seed, &scale, ls, L ? layer_end[L - 1] : 0, layer_end[L], keep);
    if (rc != ZGR_OK) return rc;   // (a failure here leaves the earlier layers swept: the context is sticky-failed by check())
  }
  if (n_layers > 1) {
    rc = check(ctx, cudaEventRecord(ev_begin, ctx->aux_stream));
    if (rc == ZGR_OK) rc = check(ctx, cudaStreamWaitEvent(st, ev_begin, 0));
    if (rc != ZGR_OK) return rc;
  }
  if (keep) {
    ctx->held_valid = true;
    ctx->held_seed = seed;
    ctx->held_c = scale;
  }
  ledger_add(ctx, seed, scale);
  return ZGR_OK;
}

int zgr_clear_coeffs(zgr_ctx* ctx, int32_t tensor) {
  if (!ctx || tensor < 0 || tensor >= static_cast<int32_t>(ctx->descs.size())) return ZGR_EINVAL;
  TensorDesc& td = ctx->descs[static_cast<size_t>(tensor)];
  if (td.rank == 0) return ZGR_EINVAL;
  if (!ctx->ledger.empty()) return ZGR_ESTATE;
  td.q = nullptr;
  td.qscale = nullptr;
  td.qzero = nullptr;
  td.qrows = 0;
  ctx->descs_dirty = true;
  ctx->held_valid = false;
  return ZGR_OK;
}

int zgr_get_stats(zgr_ctx* ctx, uint64_t seed, double* out, void* stream) {
  if (!ctx || !out) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = flush_descs(ctx, st);
  if (rc != ZGR_OK) return rc;
  const size_t n = ctx->descs.size();
  if (ctx->held_valid && ctx->held_seed == seed) {
    // The first perturbation under this seed kept the bookkeeping: add up its partial sums (fixed order) and
    // read them back; they are the norms of c z, c being that perturbation's coefficient.
    rc = check(ctx, launch_stats_finish(ctx->d_ranges_sweep, static_cast<int>(n), ctx->d_stats, st));
    if (rc == ZGR_OK) ctx->launches++;
    if (rc == ZGR_OK) rc = check(ctx, cudaMemcpyAsync(out, ctx->d_stats, 3 * n * sizeof(double), cudaMemcpyDeviceToHost, st));
    if (rc == ZGR_OK) rc = check(ctx, cudaStreamSynchronize(st));
    if (rc != ZGR_OK) return rc;
    const double inv = 1.0 / (ctx->held_c * ctx->held_c);
    for (size_t i = 0; i < 3 * n; ++i) out[i] *= inv;
    return ZGR_OK;
  }
  // A pass of its own: regenerate Z and U G for `seed` without touching the weights.
  rc = prepare_sweep_stats(ctx);      // (the tcgen05 groups leave their partial sums in the slots of the sweep plan)
  if (rc != ZGR_OK) return rc;
  ctx->held_valid = false;
  if (!ctx->stats_planned) {
    // tensors served by the tcgen05 kernel reuse its work items; all others get a generic tiling (strips of 64 columns)
    int64_t total = ctx->d;
    int64_t target = std::min<int64_t>(std::max<int64_t>(total / (static_cast<int64_t>(ctx->sm_count) * 64), 4096), 131072);
    ctx->stats_first.assign(n + 1, 0);
    for (size_t l = 0; l < n; ++l) {
      const TensorDesc& t = ctx->descs[l];
      ctx->stats_first[l] = static_cast<int32_t>(ctx->stats_items.size());
      if (t.umma && ctx->guided_at_init) continue;
      for (int64_t c0 = 0; c0 < t.cols; c0 += 64) {
        const int ncols = static_cast<int>(std::min<int64_t>(64, t.cols - c0));
        const int64_t nrows = std::max<int64_t>(1, target / ncols);
        for (int64_t r0 = 0; r0 < t.rows; r0 += nrows)
          ctx->stats_items.push_back(WorkItem{static_cast<int32_t>(l), ncols, r0, std::min(nrows, t.rows - r0), c0});
      }
    }
    ctx->stats_first[n] = static_cast<int32_t>(ctx->stats_items.size());
    if (!ctx->stats_items.empty()) {
      rc = dev_alloc(ctx, &ctx->d_stats_items, ctx->stats_items.size());
      if (rc == ZGR_OK)
        rc = check(ctx, cudaMemcpy(ctx->d_stats_items, ctx->stats_items.data(), ctx->stats_items.size() * sizeof(WorkItem), cudaMemcpyHostToDevice));
      if (rc != ZGR_OK) return rc;
    }
    rc = alloc_slots(ctx, &ctx->d_stats_slots, ctx->stats_items.size());
    if (rc != ZGR_OK) return rc;
    std::vector<StatRange> ranges(n);
    for (size_t l = 0; l < n; ++l) {
      ranges[l] = StatRange{ctx->d_stats_slots, ctx->stats_first[l], ctx->stats_first[l + 1] - ctx->stats_first[l]};
      if (ctx->descs[l].umma && ctx->guided_at_init)
        for (const Group& g : ctx->groups)
          if (g.kc.path == PATH_UMMA && g.first_item[l + 1] > g.first_item[l])
            ranges[l] = StatRange{g.d_item_stats, g.first_item[l], g.first_item[l + 1] - g.first_item[l]};
    }
    rc = dev_alloc(ctx, &ctx->d_ranges_pass, n);
    if (rc == ZGR_OK) rc = check(ctx, cudaMemcpy(ctx->d_ranges_pass, ranges.data(), n * sizeof(StatRange), cudaMemcpyHostToDevice));
    if (rc != ZGR_OK) return rc;
    ctx->stats_planned = true;
  }
  SweepParams p;
  std::memset(&p, 0, sizeof(p));
  p.n_terms = 1;
  p.term[0].keys = make_keys(seed);
  p.term[0].iso = make_scale(ctx->a, ctx->cfg.bits_per_normal);
  p.unit = make_scale(1.0, ctx->cfg.bits_per_normal);
  p.tensors = ctx->d_descs;
  p.items = ctx->d_stats_items;
  p.n_items = static_cast<int32_t>(ctx->stats_items.size());
  p.term[0].cb = static_cast<float>(ctx->b);
  p.kshift = kshift_for(std::fabs(ctx->b));
  p.item_stats = ctx->d_stats_slots;
  p.item_base = 0;
  if (p.n_items > 0) {
    const int grid = static_cast<int>(std::min<int64_t>(p.n_items, static_cast<int64_t>(ctx->sm_count) * 4));
    rc = check(ctx, launch_stats(ctx->cfg.bits_per_normal, p, grid, st));
    if (rc != ZGR_OK) return rc;
    ctx->launches++;
  }
  for (const Group& g : ctx->groups) {
    if (g.kc.path != PATH_UMMA || g.items.empty()) continue;
    p.items = g.d_items;
    p.n_items = static_cast<int32_t>(g.items.size());
    p.item_stats = g.d_item_stats;
    rc = check(ctx, launch_stats_umma(g.kc, p, ctx->d_tmaps, ctx->d_err, g.grid, st));
    if (rc != ZGR_OK) return rc;
    ctx->launches++;
  }
  rc = check(ctx, launch_stats_finish(ctx->d_ranges_pass, static_cast<int>(n), ctx->d_stats, st));
  if (rc != ZGR_OK) return rc;
  ctx->launches++;
  rc = check(ctx, cudaMemcpyAsync(out, ctx->d_stats, 3 * n * sizeof(double), cudaMemcpyDeviceToHost, st));
  if (rc != ZGR_OK) return rc;
  return check(ctx, cudaStreamSynchronize(st));
}

int zgr_enable_stats(zgr_ctx* ctx, int32_t enable) {
  if (!ctx) return ZGR_EINVAL;
  ctx->stats_on = enable != 0;     // norms already held stay available until something they depend on changes
  return ZGR_OK;
}

int zgr_debug_philox(zgr_ctx* ctx, uint64_t seed, int32_t tensor, int32_t tag, uint64_t first_block, int64_t n_blocks, uint32_t* dev_out,
                     void* stream) {
  if (!ctx || !dev_out || n_blocks < 0 || tensor < 0 || tag < 0) return ZGR_EINVAL;
  if (reinterpret_cast<uintptr_t>(dev_out) % 16 != 0) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  if (n_blocks == 0) return ZGR_OK;
  const int rc = check(ctx, launch_philox_blocks(make_keys(seed), static_cast<uint32_t>(tensor), static_cast<uint32_t>(tag), first_block, n_blocks,
                                                 dev_out, static_cast<cudaStream_t>(stream)));
  if (rc == ZGR_OK) ctx->launches++;
  return rc;
}

int zgr_debug_z(zgr_ctx* ctx, uint64_t seed, int32_t tensor, float* dev_out, void* stream) {
  if (!ctx || !dev_out || tensor < 0 || tensor >= static_cast<int32_t>(ctx->descs.size())) return ZGR_EINVAL;
  if (reinterpret_cast<uintptr_t>(dev_out) % 4 != 0) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (ctx->frag_stale[static_cast<size_t>(tensor)]) {
    const TensorDesc& cur = ctx->descs[static_cast<size_t>(tensor)];
    const int rcf = check(ctx, launch_split_subspace(cur.U, cur.rows, cur.rank, cur.kpad, const_cast<uint4*>(cur.Ufrag), st));
    if (rcf != ZGR_OK) return rcf;
    ctx->launches++;
    ctx->frag_stale[static_cast<size_t>(tensor)] = 0;
  }
  // a one-tensor model whose weights are the zeroed output buffer, swept once with scale 1
  std::vector<TensorDesc> one(1, ctx->descs[static_cast<size_t>(tensor)]);
  one[0].data = dev_out;
  std::vector<Group> groups;
  const bool guided_on = ctx->guided_at_init;
  plan(one, std::vector<int>(1, 0), guided_on, ctx->cfg.bits_per_normal, ctx->sm_count, groups, ZGR_F32);
  const size_t owned_before = ctx->owned.size();
  TensorDesc* d_one = nullptr;
  int rc = dev_alloc(ctx, &d_one, 1);
  if (rc == ZGR_OK) rc = check(ctx, cudaMemcpy(d_one, one.data(), sizeof(TensorDesc), cudaMemcpyHostToDevice));
  if (rc == ZGR_OK) rc = upload_groups(ctx, groups);
  if (rc == ZGR_OK) rc = check(ctx, cudaMemsetAsync(dev_out, 0, static_cast<size_t>(one[0].rows * one[0].cols) * sizeof(float), st));
  const double one_scale = 1.0;
  if (rc == ZGR_OK) rc = sweep(ctx, groups, d_one, 1, &seed, &one_scale, st);
  if (rc == ZGR_OK) rc = check(ctx, cudaStreamSynchronize(st));
  for (size_t i = owned_before; i < ctx->owned.size(); ++i) cudaFree(ctx->owned[i]);
  ctx->owned.resize(owned_before);
  return rc;
}

int zgr_debug_z_tcgen05(zgr_ctx* ctx, uint64_t seed, int32_t tensor, float* dev_out, void* stream) {
  if (!ctx || !dev_out || tensor < 0 || tensor >= static_cast<int32_t>(ctx->descs.size())) return ZGR_EINVAL;
  if (reinterpret_cast<uintptr_t>(dev_out) % 16 != 0) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  const TensorDesc& cur = ctx->descs[static_cast<size_t>(tensor)];
  if (!cur.umma || !ctx->guided_at_init) return ZGR_ESTATE;   // the sweeps do not serve this tensor with the tcgen05 kernel
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = flush_descs(ctx, st);
  if (rc != ZGR_OK) return rc;
  // A one-tensor model whose weights are a zeroed 16-bit image, swept once with coefficient 1 by the tcgen05
  // kernel itself; its fp32 results go to dev_out instead of being rounded into the image.
  const size_t owned_before = ctx->owned.size();
  const size_t numel = static_cast<size_t>(cur.rows * cur.cols);
  uint16_t* image = nullptr;
  CUtensorMap* d_maps = nullptr;
  TensorDesc* d_one = nullptr;
  std::vector<Group> groups;
  rc = dev_alloc(ctx, &image, numel);
  if (rc == ZGR_OK) rc = check(ctx, cudaMemsetAsync(image, 0, numel * sizeof(uint16_t), st));
  CUtensorMap maps[3];
  if (rc == ZGR_OK) {
    maps[1] = ctx->tmaps[static_cast<size_t>(3 * tensor + 1)];
    maps[2] = ctx->tmaps[static_cast<size_t>(3 * tensor + 2)];
    if (!make_map_16bit(&maps[0], image, cur.rows, cur.cols, 64)) rc = check(ctx, cudaErrorUnknown);
  }
  if (rc == ZGR_OK) rc = dev_alloc(ctx, &d_maps, 3);
  if (rc == ZGR_OK) rc = check(ctx, cudaMemcpyAsync(d_maps, maps, sizeof(maps), cudaMemcpyHostToDevice, st));
  std::vector<TensorDesc> one(1, cur);
  one[0].data = image;
  if (rc == ZGR_OK) rc = dev_alloc(ctx, &d_one, 1);
  if (rc == ZGR_OK) rc = check(ctx, cudaMemcpyAsync(d_one, one.data(), sizeof(TensorDesc), cudaMemcpyHostToDevice, st));
  if (rc == ZGR_OK) {
    plan(one, std::vector<int>(1, 0), true, ctx->cfg.bits_per_normal, ctx->sm_count, groups);
    rc = upload_groups(ctx, groups);
  }
  if (rc == ZGR_OK) {
    SweepParams p;
    std::memset(&p, 0, sizeof(p));
    p.term[0].keys = make_keys(seed);
    p.term[0].iso = make_scale(ctx->a, ctx->cfg.bits_per_normal);
    p.term[0].cb = static_cast<float>(ctx->b);
    p.n_terms = 1;
    p.unit = make_scale(1.0, ctx->cfg.bits_per_normal);
    p.tensors = d_one;
    p.zout = dev_out;
    p.kshift = kshift_for(std::fabs(ctx->b));
    for (Group& g : groups) {
      if (g.items.empty()) continue;
      if (g.kc.path != PATH_UMMA) { rc = ZGR_ESTATE; break; }
      p.items = g.d_items;
      p.n_items = static_cast<int32_t>(g.items.size());
      rc = check(ctx, launch_debug_z_umma(g.kc, p, d_maps, ctx->d_err, g.grid, st));
      if (rc != ZGR_OK) break;
      ctx->launches++;
    }
  }
  const int rc_sync = check(ctx, cudaStreamSynchronize(st));
  if (rc == ZGR_OK) rc = rc_sync;
  for (size_t i = owned_before; i < ctx->owned.size(); ++i) cudaFree(ctx->owned[i]);
  ctx->owned.resize(owned_before);
  return rc;
}

int zgr_update_subspace(zgr_ctx* ctx, int32_t tensor, const float* U_src, int32_t src_is_host, void* stream) {
  if (!ctx || tensor < 0 || tensor >= static_cast<int32_t>(ctx->descs.size())) return ZGR_EINVAL;
  TensorDesc& td = ctx->descs[static_cast<size_t>(tensor)];
  if (td.rank == 0) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  if (!ctx->ledger.empty()) return ZGR_ESTATE;
  ctx->held_valid = false;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int rc = ZGR_OK;
  if (U_src != nullptr && U_src != td.U) {
    const size_t bytes = static_cast<size_t>(td.rows) * td.rank * sizeof(float);
    rc = check(ctx, cudaMemcpyAsync(const_cast<float*>(td.U), U_src, bytes, src_is_host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice, st));
    if (rc != ZGR_OK) return rc;
  }
  return refresh_operands(ctx, tensor, st);
}

int zgr_build_subspace(zgr_ctx* ctx, int32_t tensor, const float* grads, int32_t src_is_host, void* stream) {
  if (!ctx || tensor < 0 || tensor >= static_cast<int32_t>(ctx->descs.size())) return ZGR_EINVAL;
  TensorDesc& td = ctx->descs[static_cast<size_t>(tensor)];
  if (td.rank == 0 || td.rows < td.rank) return ZGR_EINVAL;
  if (grads && reinterpret_cast<uintptr_t>(grads) % 4 != 0) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  if (!ctx->ledger.empty()) return ZGR_ESTATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t need = subspace_scratch_bytes(td.rows, td.rank);
  if (need > ctx->qr_bytes) {
    void* q = nullptr;
    const int rc = check(ctx, cudaMalloc(&q, need));
    if (rc != ZGR_OK) return rc;
    ctx->owned.push_back(q);          // an outgrown scratch buffer stays owned until zgr_destroy; work enqueued on it may still run
    ctx->d_qr = q;
    ctx->qr_bytes = need;
  }
  float* U = const_cast<float*>(td.U);
  const float* A = U;                  // NULL source: the gradient directions were written into the subspace buffer itself
  if (grads != nullptr && grads != td.U) {
    if (src_is_host) {
      const size_t bytes = static_cast<size_t>(td.rows) * td.rank * sizeof(float);
      const int rc = check(ctx, cudaMemcpyAsync(U, grads, bytes, cudaMemcpyHostToDevice, st));
      if (rc != ZGR_OK) return rc;
    } else {
      A = grads;
    }
  }
  int* d_status = nullptr;
  int rc = check(ctx, launch_build_subspace(A, td.rows, td.rank, U, ctx->d_qr, &d_status, nullptr, st));
  if (rc != ZGR_OK) return rc;
  ctx->launches += 6;
  int status = 0;
  rc = check(ctx, cudaMemcpyAsync(&status, d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  if (rc == ZGR_OK) rc = check(ctx, cudaStreamSynchronize(st));
  if (rc != ZGR_OK) return rc;
  if (status != 0) return ZGR_EINVAL;  // linearly dependent directions: nothing was written
  // the new basis is in place: refresh the tensor-core operand copies exactly as for a delivered subspace
  return zgr_update_subspace(ctx, tensor, nullptr, 0, stream);
}

int zgr_debug_plan(const zgr_tensor* tensors, int32_t n, const zgr_config* cfg, int32_t sm_count, int32_t tcgen05, int32_t multi,
                   zgr_plan_item* out, int64_t max_items, int64_t* n_items) {
  if (!n_items || sm_count < 1 || max_items < 0 || (max_items > 0 && !out)) return ZGR_EINVAL;
  int64_t d = 0, K = 0;
  const int valid = validate_model(tensors, n, cfg, &d, &K);
  if (valid != ZGR_OK) return valid;
  const bool guided_on = K > 0 && cfg->alpha < 1.0;
  std::vector<TensorDesc> descs(static_cast<size_t>(n));
  std::vector<int> all(static_cast<size_t>(n));
  for (int32_t l = 0; l < n; ++l) {
    const zgr_tensor& t = tensors[l];
    TensorDesc& td = descs[static_cast<size_t>(l)];
    std::memset(&td, 0, sizeof(td));
    td.data = t.data; td.U = t.U; td.rows = t.rows; td.cols = t.cols; td.rank = t.rank; td.id = l; td.dtype = t.dtype; td.qbits = 8;
    const bool vec = (reinterpret_cast<uintptr_t>(t.data) & 15) == 0 && (t.cols % 8 == 0);
    if (guided_on && t.rank > 8 && vec && t.dtype != ZGR_F32) {
      // what zgr_init would have built for this tensor: operand copies for the tensor-core kernels
      td.kpad = t.rank <= 16 ? 16 : (t.rank <= 32 ? 32 : 64);
      td.Ufrag = reinterpret_cast<const uint4*>(uintptr_t{16});   // marker only: never dereferenced by the planner
      td.umma = (tcgen05 && t.rows < (int64_t{1} << 31) - 256 && t.cols < (int64_t{1} << 31) - 256) ? 1 : 0;
    }
    all[static_cast<size_t>(l)] = l;
  }
  std::vector<Group> groups;
  plan(descs, all, guided_on, cfg->bits_per_normal, sm_count, groups, -1, multi != 0);
  int64_t count = 0;
  for (const Group& g : groups)
    for (const WorkItem& w : g.items) {
      if (count < max_items)
        out[count] = zgr_plan_item{g.kc.path, g.kc.kpad, w.tensor, w.ncols, w.row0_or_e0, w.nrows_or_count, w.col0};
      ++count;
    }
  *n_items = count;
  return ZGR_OK;
}

int zgr_update_subspaces(zgr_ctx* ctx, int32_t n, const int32_t* tensors, const float* const* U_src, int32_t src_is_host, void* stream) {
  if (!ctx || !tensors || n < 1) return ZGR_EINVAL;
  std::vector<char> seen(ctx->descs.size(), 0);
  int n_umma = 0;
  for (int32_t i = 0; i < n; ++i) {
    const int32_t l = tensors[i];
    if (l < 0 || l >= static_cast<int32_t>(ctx->descs.size()) || seen[static_cast<size_t>(l)]) return ZGR_EINVAL;
    seen[static_cast<size_t>(l)] = 1;
    if (ctx->descs[static_cast<size_t>(l)].rank == 0) return ZGR_EINVAL;
    n_umma += ctx->descs[static_cast<size_t>(l)].umma ? 1 : 0;
  }
  if (ctx->sticky) return ctx->sticky;
  if (!on_ctx_device(ctx)) return ZGR_EINVAL;
  if (!ctx->ledger.empty()) return ZGR_ESTATE;
  ctx->held_valid = false;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // every tensor of the tcgen05 path is listed: their operand copies are rebuilt by one launch after the copies
  const bool fused = n_umma > 0 && n_umma == ctx->n_split_jobs;
  for (int32_t i = 0; i < n; ++i) {
    const int32_t l = tensors[i];
    TensorDesc& td = ctx->descs[static_cast<size_t>(l)];
    const float* src = U_src ? U_src[i] : nullptr;
    if (src != nullptr && src != td.U) {
      const size_t bytes = static_cast<size_t>(td.rows) * td.rank * sizeof(float);
      const int rc = check(ctx, cudaMemcpyAsync(const_cast<float*>(td.U), src, bytes, src_is_host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice, st));
      if (rc != ZGR_OK) return rc;
    }
    if (td.Ufrag != nullptr) {
      if (td.umma) {
        ctx->frag_stale[static_cast<size_t>(l)] = 1;
      } else {
        const int rc = check(ctx, launch_split_subspace(td.U, td.rows, td.rank, td.kpad, const_cast<uint4*>(td.Ufrag), st));
        if (rc != ZGR_OK) return rc;
        ctx->launches++;
      }
    }
    if (td.umma && !fused) {
      const int64_t rows_pad = ((td.rows + 127) / 128) * 128;
      const int rc = check(ctx, launch_split_subspace_rowmajor(td.U, td.rows, td.rank, td.kpad, rows_pad, td.ushift, td.Uhi, td.Ulo, st));
      if (rc != ZGR_OK) return rc;
      ctx->launches++;
    }
  }
  if (fused) {
    const int rc = check(ctx, launch_split_subspace_rowmajor_all(ctx->d_split_jobs, ctx->n_split_jobs, st));
    if (rc != ZGR_OK) return rc;
    ctx->launches++;
  }
  return ZGR_OK;
}

int zgr_profile(zgr_ctx* ctx, int32_t enable) {
  if (!ctx) return ZGR_EINVAL;
  ctx->profiling = enable != 0;
  return ZGR_OK;
}

int zgr_profile_read(zgr_ctx* ctx, zgr_kernel_time* out, int32_t max_entries, int32_t* n_entries) {
  if (!ctx || !out || !n_entries || max_entries < 0) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  const int rc = check(ctx, cudaDeviceSynchronize());
  if (rc != ZGR_OK) return rc;
  int32_t n = 0;
  for (std::vector<Group>* gs : {&ctx->groups, &ctx->groups_multi})
  for (Group& g : *gs) {
    if (g.timed.empty()) continue;
    double total = 0.0;
    for (auto& ev : g.timed) {
      float ms = 0.0f;
      if (cudaEventElapsedTime(&ms, ev.first, ev.second) == cudaSuccess) total += ms;
      cudaEventDestroy(ev.first);
      cudaEventDestroy(ev.second);
    }
    if (n < max_entries) {
      zgr_kernel_time& o = out[n];
      o.path = g.kc.path;
      o.dtype = g.kc.dtype;
      o.kpad = g.kc.kpad;
      o.launches = static_cast<int32_t>(g.timed.size());
      o.elements = g.elements;
      o.ms_total = total;
      ++n;
    }
    g.timed.clear();
  }
  *n_entries = n;
  return ZGR_OK;
}

int zgr_device_status(zgr_ctx* ctx, int32_t* code) {
  if (!ctx || !code) return ZGR_EINVAL;
  if (ctx->sticky) return ctx->sticky;
  int rc = check(ctx, cudaDeviceSynchronize());
  if (rc != ZGR_OK) return rc;
  int v = 0;
  rc = check(ctx, cudaMemcpy(&v, ctx->d_err, sizeof(int), cudaMemcpyDeviceToHost));
  if (rc != ZGR_OK) return rc;
  *code = v;
  if (v != 0) ctx->sticky = ZGR_ECUDA;   // a kernel gave up on a wait: its sweep is incomplete, the weights are not trustworthy
  return ZGR_OK;
}

int zgr_get_scalars(const zgr_ctx* ctx, double* a, double* b) {
  if (!ctx || !a || !b) return ZGR_EINVAL;
  *a = ctx->a;
  *b = ctx->b;
  return ZGR_OK;
}

int zgr_get_state(const zgr_ctx* ctx, int32_t* active, uint64_t* seed, double* net_scale) {
  if (!ctx || !active || !seed || !net_scale) return ZGR_EINVAL;
  *active = static_cast<int32_t>(ctx->ledger.size());
  const auto it = ctx->ledger.find(ctx->last_seed);
  *seed = ctx->last_seed;
  *net_scale = it == ctx->ledger.end() ? 0.0 : it->second;
  return ZGR_OK;
}

int zgr_debug_check_device(int32_t ctx_device, int32_t current_device) {
  return (ctx_device >= 0 && ctx_device == current_device) ? ZGR_OK : ZGR_EINVAL;
}

int64_t zgr_launch_count(const zgr_ctx* ctx) { return ctx ? ctx->launches : -1; }

void zgr_destroy(zgr_ctx* ctx) {
  if (!ctx) return;
  for (std::vector<Group>* gs : {&ctx->groups, &ctx->groups_multi})
    for (Group& g : *gs)
      for (auto& ev : g.timed) {
        cudaEventDestroy(ev.first);
        cudaEventDestroy(ev.second);
      }
  for (cudaEvent_t e : ctx->layer_events) cudaEventDestroy(e);
  if (ctx->aux_stream) cudaStreamDestroy(ctx->aux_stream);
  for (void* p : ctx->owned) cudaFree(p);
  delete ctx;
}

const char* zgr_strerror(int code) {
  switch (code) {
    case ZGR_OK: return "ok";
    case ZGR_EINVAL: return "invalid argument";
    case ZGR_ESTATE: return "call out of sequence (perturb / restore_update seeds do not match)";
    case ZGR_ECUDA: return "CUDA runtime error (no device, launch failure); the context is unusable";
    case ZGR_ENOMEM: return "out of device or host memory";
    case ZGR_ETOOBIG: return "tensor larger than the fixed scratch of the allocation-free entry point (ZGR_NOALLOC_MAX_TILES tiles of 1024 x 64)";
    default: return "unknown error code";
  }
}

}  // extern "C"
