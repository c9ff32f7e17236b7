// Subspace construction on the device (Algorithm 1, "Collect gradients to build basis V_r"; Sec. 3.2
// "Guided Perturbation Sampling on Cloud"): an orthonormal basis U (rows x r, r <= 64) of the span of the r
// gradient directions collected for one tensor, given as the columns of A (rows x r fp32, row-major).
//
// Method: Cholesky QR, applied twice.  One pass forms the Gram matrix  S = A^T A  (r x r), factors it
// S = R^T R  (R upper triangular with a positive diagonal) and returns  Q = A R^-1.  In exact arithmetic that is
// the thin Q of the QR factorisation with R_kk > 0, i.e. the same basis, column for column, as a Householder QR
// with that sign convention.  In floating point the first pass loses orthogonality in proportion to the
// square of the condition number of A; the second pass, applied to the nearly orthonormal Q of the first,
// restores it to working precision.  Everything between the fp32 input and the fp32 output is carried in
// double: the Gram matrices (rows x r^2 multiply-adds, a few hundred MFLOP at most for the largest tensor of
// the paper-shaped models), the r x r factorisations and the products A R^-1.  Tall-skinny and tiny in
// arithmetic, the job is bound by reading A twice and writing U once; tensor cores would add nothing but
// rounding (their split-bf16 product is good to 2^-16, an orthogonality of 1e-6 needs more).
//
// Three kernels per pass:
//   gram_partial   one block per chunk of 128 rows: partial Gram matrix of the chunk, written to scratch
//   factor         one block: sums the partials in a fixed order, Cholesky factor, inverse of R, status
//   apply          one block per chunk of 128 rows: Q = A R^-1
// The summation order is fixed, so the result does not depend on the launch history.
#include <cuda_runtime.h>

#include "zgr_subspace.h"

namespace zgr {
namespace {

constexpr int kChunkRows = 128;
constexpr int kLd = 65;               // leading dimension of the shared-memory matrices (64 + 1: no bank conflicts down a column)
constexpr int kQrThreads = 256;
constexpr int kMaxR = 64;

// Partial Gram matrix of rows [chunk*128, +128) of X (rows x r).  X is fp32 (SRC_DOUBLE = false) or double.
template <bool SRC_DOUBLE>
__global__ void __launch_bounds__(kQrThreads) gram_partial_kernel(const void* __restrict__ Xv, int64_t rows, int r, double* __restrict__ partials) {
  extern __shared__ double dyn_smem[];
  double (*Xs)[kLd] = reinterpret_cast<double (*)[kLd]>(dyn_smem);          // [kChunkRows][kLd]
  const int64_t row0 = static_cast<int64_t>(blockIdx.x) * kChunkRows;
  const int nrows = static_cast<int>(min(static_cast<int64_t>(kChunkRows), rows - row0));
  for (int idx = threadIdx.x; idx < kChunkRows * r; idx += kQrThreads) {
    const int i = idx / r, k = idx % r;
    double v = 0.0;
    if (i < nrows) {
      const int64_t e = (row0 + i) * r + k;
      v = SRC_DOUBLE ? static_cast<const double*>(Xv)[e] : static_cast<double>(static_cast<const float*>(Xv)[e]);
    }
    Xs[i][k] = v;
  }
  __syncthreads();
  double* out = partials + static_cast<int64_t>(blockIdx.x) * r * r;
  for (int idx = threadIdx.x; idx < r * r; idx += kQrThreads) {
    const int a = idx / r, b = idx % r;
    double s = 0.0;
    if (b >= a) {                       // upper triangle; the factorisation reads nothing else
      for (int i = 0; i < kChunkRows; ++i) s = fma(Xs[i][a], Xs[i][b], s);
    }
    out[idx] = s;
  }
}

// S = sum of the partials (fixed order), S = R^T R, W = R^-1 (upper triangular, double, r x r row-major).
// status[0] = 0, or 1 + k if the k-th pivot is not positive (the columns of A are linearly dependent to
// working precision); W is then left unset.  If Racc is not null it is multiplied from the left by this pass's R
// (Racc <- R Racc), which after two passes is the triangular factor of A itself.
__global__ void __launch_bounds__(kQrThreads) factor_kernel(const double* __restrict__ partials, int n_chunks, int r, double* __restrict__ W,
                                                            double* __restrict__ Racc, int first_pass, int* __restrict__ status) {
  extern __shared__ double dyn_smem[];
  double (*S)[kLd] = reinterpret_cast<double (*)[kLd]>(dyn_smem);                       // [kMaxR][kLd]
  double (*Winv)[kLd] = reinterpret_cast<double (*)[kLd]>(dyn_smem + kMaxR * kLd);
  double (*Old)[kLd] = reinterpret_cast<double (*)[kLd]>(dyn_smem + 2 * kMaxR * kLd);
  __shared__ int bad;
  if (threadIdx.x == 0) bad = 0;
  for (int idx = threadIdx.x; idx < r * r; idx += kQrThreads) {
    double s = 0.0;
    for (int c = 0; c < n_chunks; ++c) s += partials[static_cast<int64_t>(c) * r * r + idx];
    S[idx / r][idx % r] = s;
  }
  __syncthreads();
  // Cholesky, column by column (right-looking), upper triangular factor kept in the upper triangle of S
  for (int k = 0; k < r; ++k) {
    if (threadIdx.x == 0) {
      const double p = S[k][k];
      if (!(p > 0.0) && bad == 0) bad = 1 + k;
      S[k][k] = p > 0.0 ? sqrt(p) : 1.0;
    }
    __syncthreads();
    const double d = S[k][k];
    for (int j = k + 1 + threadIdx.x; j < r; j += kQrThreads) S[k][j] /= d;
    __syncthreads();
    for (int idx = threadIdx.x; idx < (r - k - 1) * (r - k - 1); idx += kQrThreads) {
      const int i = k + 1 + idx / (r - k - 1), j = k + 1 + idx % (r - k - 1);
      if (j >= i) S[i][j] -= S[k][i] * S[k][j];
    }
    __syncthreads();
  }
  // inverse of the upper triangular R by back substitution, one column per thread
  for (int j = threadIdx.x; j < r; j += kQrThreads) {
    for (int i = r - 1; i >= 0; --i) {
      double v = (i == j) ? 1.0 : 0.0;
      for (int k = i + 1; k <= j; ++k) v -= S[i][k] * Winv[k][j];
      Winv[i][j] = (i <= j) ? v / S[i][i] : 0.0;
    }
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < r * r; idx += kQrThreads) W[idx] = Winv[idx / r][idx % r];
  if (Racc != nullptr) {
    // Racc <- R Racc  (first pass: Racc = R)
    for (int idx = threadIdx.x; idx < r * r; idx += kQrThreads) Old[idx / r][idx % r] = first_pass ? ((idx / r == idx % r) ? 1.0 : 0.0) : Racc[idx];
    __syncthreads();
    for (int idx = threadIdx.x; idx < r * r; idx += kQrThreads) {
      const int i = idx / r, j = idx % r;
      double v = 0.0;
      for (int k = i; k <= j; ++k) v += S[i][k] * Old[k][j];
      Racc[idx] = (j >= i) ? v : 0.0;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0 && bad != 0 && status[0] == 0) status[0] = bad;
}

// Y = X W for rows [chunk*128, +128): X fp32 or double (rows x r), W double upper triangular, Y double or fp32.
template <bool SRC_DOUBLE, bool DST_DOUBLE>
__global__ void __launch_bounds__(kQrThreads) apply_kernel(const void* __restrict__ Xv, int64_t rows, int r, const double* __restrict__ W,
                                                           void* __restrict__ Yv, const int* __restrict__ status) {
  if (status[0] != 0) return;          // the factorisation failed: leave the destination alone
  extern __shared__ double dyn_smem[];
  double (*Xs)[kLd] = reinterpret_cast<double (*)[kLd]>(dyn_smem);                      // [kChunkRows][kLd]
  double (*Ws)[kLd] = reinterpret_cast<double (*)[kLd]>(dyn_smem + kChunkRows * kLd);   // [kMaxR][kLd]
  const int64_t row0 = static_cast<int64_t>(blockIdx.x) * kChunkRows;
  const int nrows = static_cast<int>(min(static_cast<int64_t>(kChunkRows), rows - row0));
  for (int idx = threadIdx.x; idx < r * r; idx += kQrThreads) Ws[idx / r][idx % r] = W[idx];
  for (int idx = threadIdx.x; idx < nrows * r; idx += kQrThreads) {
    const int i = idx / r, k = idx % r;
    const int64_t e = (row0 + i) * r + k;
    Xs[i][k] = SRC_DOUBLE ? static_cast<const double*>(Xv)[e] : static_cast<double>(static_cast<const float*>(Xv)[e]);
  }
  __syncthreads();
  for (int idx = threadIdx.x; idx < nrows * r; idx += kQrThreads) {
    const int i = idx / r, j = idx % r;
    double v = 0.0;
    for (int k = 0; k <= j; ++k) v = fma(Xs[i][k], Ws[k][j], v);
    const int64_t e = (row0 + i) * r + j;
    if (DST_DOUBLE) static_cast<double*>(Yv)[e] = v;
    else static_cast<float*>(Yv)[e] = static_cast<float>(v);
  }
}

}  // namespace

size_t subspace_scratch_bytes(int64_t rows, int r) {
  const int64_t n_chunks = (rows + kChunkRows - 1) / kChunkRows;
  // partial Gram matrices, R^-1, accumulated R, the double image of the first pass's Q, status word
  return static_cast<size_t>(n_chunks) * r * r * sizeof(double) + 2 * static_cast<size_t>(r) * r * sizeof(double) +
         static_cast<size_t>(rows) * r * sizeof(double) + 256;
}

cudaError_t launch_build_subspace(const float* A, int64_t rows, int r, float* U_out, void* scratch, int** status_out, double** r_out, cudaStream_t st) {
  if (r < 1 || r > kMaxR || rows < r) return cudaErrorInvalidValue;
  const int n_chunks = static_cast<int>((rows + kChunkRows - 1) / kChunkRows);
  uint8_t* base = static_cast<uint8_t*>(scratch);
  int* status = reinterpret_cast<int*>(base);
  double* partials = reinterpret_cast<double*>(base + 256);
  double* W = partials + static_cast<size_t>(n_chunks) * r * r;
  double* Racc = W + static_cast<size_t>(r) * r;
  double* Q1 = Racc + static_cast<size_t>(r) * r;
  constexpr int kGramSmem = kChunkRows * kLd * sizeof(double);
  constexpr int kFactorSmem = 3 * kMaxR * kLd * sizeof(double);
  constexpr int kApplySmem = (kChunkRows + kMaxR) * kLd * sizeof(double);
  static bool attributes_set = false;   // per process; setting them again is harmless
  if (!attributes_set) {
    cudaError_t a = cudaFuncSetAttribute(gram_partial_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGramSmem);
    if (a == cudaSuccess) a = cudaFuncSetAttribute(gram_partial_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kGramSmem);
    if (a == cudaSuccess) a = cudaFuncSetAttribute(factor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFactorSmem);
    if (a == cudaSuccess) a = cudaFuncSetAttribute(apply_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kApplySmem);
    if (a == cudaSuccess) a = cudaFuncSetAttribute(apply_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kApplySmem);
    if (a != cudaSuccess) return a;
    attributes_set = true;
  }
  cudaError_t e = cudaMemsetAsync(status, 0, sizeof(int), st);
  if (e != cudaSuccess) return e;
  // pass 1: A (fp32) -> Q1 (double)
  gram_partial_kernel<false><<<n_chunks, kQrThreads, kGramSmem, st>>>(A, rows, r, partials);
  factor_kernel<<<1, kQrThreads, kFactorSmem, st>>>(partials, n_chunks, r, W, Racc, 1, status);
  apply_kernel<false, true><<<n_chunks, kQrThreads, kApplySmem, st>>>(A, rows, r, W, Q1, status);
  // pass 2: Q1 (double) -> U (fp32)
  gram_partial_kernel<true><<<n_chunks, kQrThreads, kGramSmem, st>>>(Q1, rows, r, partials);
  factor_kernel<<<1, kQrThreads, kFactorSmem, st>>>(partials, n_chunks, r, W, Racc, 0, status);
  apply_kernel<true, false><<<n_chunks, kQrThreads, kApplySmem, st>>>(Q1, rows, r, W, U_out, status);
  if (status_out) *status_out = status;
  if (r_out) *r_out = Racc;
  return cudaGetLastError();
}

}  // namespace zgr
