// Structures shared by the host side of the library and its kernels.
#ifndef ZGR_INTERNAL_H_
#define ZGR_INTERNAL_H_

#include <stdint.h>

namespace zgr {

// Device-side description of one weight tensor.
struct TensorDesc {
  void* data;            // weights, rows x cols, row-major
  const float* U;        // rows x rank fp32 (caller's), or null
  const uint4* Ufrag;    // library-owned copy of U, split into bf16 hi/lo and laid out in the
                         // register order of the m16n8k16 A operand (tensor-core path only)
  const int8_t* q;       // DTC codes qrows x cols (int8), or qrows rows of (cols+1)/2 bytes holding two unsigned
                         // 4-bit codes each, even column in the low nibble; null -> coefficients drawn from the seed
  const float* qscale;   // rank
  const float* qzero;    // rank or null
  int64_t rows, cols;
  int32_t rank;          // r
  int32_t kpad;          // r rounded up to the contraction width of the path in use
  int32_t id;            // generator tensor id (third counter word)
  int32_t dtype;
  int32_t qbits;         // 8 or 4: width of the codes behind q
  int32_t qrows;         // rows of G taken from the codes (Sec. 3.4, proportion omega); rows beyond it are drawn from the seed
  int32_t umma;          // 1: served by the tcgen05 + TMA kernel (tensor maps and row-major hi/lo copies of U exist)
  int32_t ushift;        // the hi/lo copies hold U * 2^ushift (brings a typical entry of an orthonormal U near 1)
  void* Uhi;             // library-owned, rows_pad x kpad fp16 row-major (TMA source), or null
  void* Ulo;
};

// One unit of work of a sweep kernel.
//   flat items (isotropic kernel): elements [e0, e0 + count) of the tensor, e0 a multiple of 8
//   tile items (guided kernels):   rows [row0, row0 + nrows) x columns [col0, col0 + ncols)
struct WorkItem {
  int32_t tensor;        // index into the descriptor table
  int32_t ncols;
  int64_t row0_or_e0;
  int64_t nrows_or_count;
  int64_t col0;
};

// Round keys of Philox4x32-10 for one seed: the key bumped by the Weyl constants once per round.
struct PhiloxKeys {
  uint32_t k0[10];
  uint32_t k1[10];
};

// Constants of the Gaussian transform with an output scale s folded in (see box_muller()).
struct NormalScale {
  float kr;       // -2 ln(2) s^2      : rho'^2 = kr * log2(u1)
  float s;        // the scale itself (accurate transform)
  float phase;    // 2 pi (2^-(nb+1) - 1) - 2 pi   (s >= 0)   or   ... - pi   (s < 0)
  float u1_off;   // 2^-(nb+1) - 1
};

// One (seed, coefficient) term of a sweep  theta <- rnd(theta + sum_q c_q z(seed_q)).
struct SeedTerm {
  PhiloxKeys keys;       // round keys of seed_q
  NormalScale iso;       // isotropic normals of this seed, scaled by c_q * a
  float cb;              // c_q * b : coefficient of U G(seed_q)
};

constexpr int kMaxTerms = 8;   // ZGR_MAX_SEEDS of the C ABI
constexpr int kStatSlots = 16; // partial sums kept per work item (one per warp that works on it; unused slots stay zero)

// Per-launch constants (passed by value in the kernel parameter space).  A single-seed sweep uses
// term[0] only, addressed with a compile-time index so that its round keys stay constant-bank
// operands; multi-seed instantiations loop over term[0 .. n_terms).
struct SweepParams {
  SeedTerm term[kMaxTerms];
  int32_t n_terms;
  NormalScale unit;      // coefficient normals, unscaled
  const TensorDesc* tensors;
  const WorkItem* items;
  int32_t n_items;
  float* zout;           // rows x cols fp32 image of the one tensor swept (test hook of the tcgen05 kernel only)
  double* item_stats;    // norm bookkeeping: kStatSlots x 3 doubles per work item of the group (partial sums per warp), or null
  int32_t item_base;     // index of items[0] in the group's full item list (layer-wise launches start in the middle)
  int32_t* sched;        // CUDA-core contraction kernel: this launch's item counter (zero between launches), see sweep_fma_kernel
  int32_t kshift;        // tcgen05 kernel: the coefficient strips are scaled by a power of two so that sum_q |c_q| b 2^kshift
                         // is near 1 (see the operand precision note in zgr_umma.cu)
};

}  // namespace zgr
#endif  // ZGR_INTERNAL_H_
