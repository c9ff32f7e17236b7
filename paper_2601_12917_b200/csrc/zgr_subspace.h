// Launcher of the subspace construction kernels (Cholesky QR applied twice, carried in double).
#ifndef ZGR_SUBSPACE_H_
#define ZGR_SUBSPACE_H_

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace zgr {

// Bytes of device scratch that launch_build_subspace needs for a rows x r input.
size_t subspace_scratch_bytes(int64_t rows, int r);

// Orthonormal basis of the span of the columns of A (device, rows x r fp32 row-major, r <= 64, rows >= r) into
// U_out (device, rows x r fp32 row-major; may be A itself).  Work is enqueued on `st`.  *status_out (if not null)
// receives the device address of an int that is 0 afterwards, or 1 + k if the k-th column of A depends linearly
// on the earlier ones to working precision (U_out is then left untouched).  *r_out (if not null) receives the
// device address of the triangular factor R (r x r doubles, row-major, A = U R, positive diagonal).
cudaError_t launch_build_subspace(const float* A, int64_t rows, int r, float* U_out, void* scratch, int** status_out, double** r_out, cudaStream_t st);

}  // namespace zgr
#endif  // ZGR_SUBSPACE_H_
