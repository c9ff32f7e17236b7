// Host-visible launchers of the sweep kernels.
#ifndef ZGR_KERNELS_H_
#define ZGR_KERNELS_H_

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>

#include "zgr_internal.h"

namespace zgr {

enum Path { PATH_ISO = 0, PATH_FMA = 1, PATH_MMA = 2, PATH_GENERIC = 3, PATH_UMMA = 4, PATH_COUNT = 5 };

// Which kernel instantiation a group of work items runs on.
struct KernelChoice {
  int path;   // Path
  int dtype;  // ZGR_F32 | ZGR_F16 | ZGR_BF16
  int kpad;   // FMA: 4 or 8;  MMA: 16, 32 or 64;  otherwise 0
  int bits;   // 32 or 16 random bits per normal
  int precise;  // accurate Gaussian transform (tensors stored in fp32)
};

int mma_strip_cols(int kpad);     // columns of a CTA strip on the tensor-core path
int mma_rows_per_iter(int kpad);  // rows a CTA advances per iteration there
size_t mma_smem_bytes(int kpad);

cudaError_t launch_sweep(const KernelChoice& kc, const SweepParams& p, int grid, cudaStream_t st);
// tcgen05 + TMA sweep (16-bit weights, rank > 8).  tmaps: three tensor maps per tensor (theta, U hi, U lo).
int umma_strip_cols(int kpad);
size_t umma_smem_bytes(int kpad);
cudaError_t launch_sweep_umma(const KernelChoice& kc, const SweepParams& p, const CUtensorMap* tmaps, int* error, int grid, cudaStream_t st);
// Test hook: the sweep kernel with its fp32 results diverted to p.zout (see the ZOUT parameter of the kernel).
cudaError_t launch_debug_z_umma(const KernelChoice& kc, const SweepParams& p, const CUtensorMap* tmaps, int* error, int grid, cudaStream_t st);
cudaError_t launch_stats_umma(const KernelChoice& kc, const SweepParams& p, const CUtensorMap* tmaps, int* error, int grid, cudaStream_t st);
cudaError_t launch_split_subspace_rowmajor(const float* U, int64_t rows, int r, int kp, int64_t rows_pad, int shift, void* hi, void* lo, cudaStream_t st);
// The same for a device-resident list of tensors in one launch (grid.y = job).
struct SplitJob {
  const float* U;
  void* hi;
  void* lo;
  int64_t rows, rows_pad;
  int32_t r, kp;
  int32_t shift;   // the copies hold U * 2^shift
};
cudaError_t launch_split_subspace_rowmajor_all(const SplitJob* d_jobs, int n_jobs, cudaStream_t st);

cudaError_t launch_stats(int bits, const SweepParams& p, int grid, cudaStream_t st);
// Norm bookkeeping, second stage: tensor l owns the work items [first, first + count) of the slot array `slots`
// (kStatSlots x 3 doubles per item); out[3 l + j] receives their sum, added in a fixed order.
struct StatRange {
  const double* slots;
  int32_t first, count;
};
cudaError_t launch_stats_finish(const StatRange* d_ranges, int n_tensors, double* d_out, cudaStream_t st);
cudaError_t launch_split_subspace(const float* U, int64_t rows, int r, int kp, uint4* out, cudaStream_t st);
cudaError_t launch_philox_blocks(const PhiloxKeys& keys, uint32_t tensor, uint32_t tag, uint64_t first_block, int64_t n_blocks,
                                 uint32_t* out, cudaStream_t st);

}  // namespace zgr
#endif  // ZGR_KERNELS_H_
