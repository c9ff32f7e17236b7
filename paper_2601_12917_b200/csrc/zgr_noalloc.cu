// Per-tensor perturbation norms without any device allocation.
//
// zgr_get_stats keeps its accumulators and its work table in memory that it obtains from cudaMalloc.
// Some users of this library must not allocate while they run: a serving or training loop in which
// an implicit device-wide synchronisation (cudaMalloc and cudaFree both cause one) would stall every
// other stream, or a process whose framework has already handed all free device memory to its own
// caching pool, so that a driver-level allocation can simply fail.  For them this file offers the same
// three sums for one tensor with all intermediate storage in a fixed array that is part of the
// library image.  The price: a size limit, one shared scratch area (calls that overlap on the GPU
// race on it), and 192 KiB of device memory held by every GPU that loads the library, until exit.
#include <cuda_runtime.h>

#include "zgr.h"
#include "zgr_device.cuh"
#include "zgr_host_internal.h"

namespace zgr {
namespace {

constexpr int kTileCols = 64;     // columns per tile (one thread column each)
constexpr int kTileRows = 1024;   // rows per tile
constexpr int kNormThreads = 256;

// One partial triple per tile.  Every slot that a call reads is written by that same call first, so
// nothing needs clearing between calls; the contents after a call are that call's partial sums.
static __device__ __align__(256) double g_norm_partials[3 * ZGR_NOALLOC_MAX_TILES];

// Device address of g_norm_partials per device ordinal; looked up on the first call on that device.
// The table is filled without a lock: two host threads that make their first call on the same device at
// the same time both look the address up and both store the same value.
constexpr int kMaxDevices = 64;
double* g_partials_addr[kMaxDevices] = {};

template <int BITS>
__global__ void __launch_bounds__(kNormThreads) norms_tile_kernel(const TensorDesc td, const PhiloxKeys keys, const NormalScale iso,
                                                                  const NormalScale unit, const float cb, const int row_tiles,
                                                                  double* __restrict__ partials) {
  __shared__ float Gs[64][kTileCols + 1];
  __shared__ double red[kNormThreads / 32][3];
  const int tile = blockIdx.x;
  const int strip = tile / row_tiles, rt = tile % row_tiles;
  const int64_t col0 = static_cast<int64_t>(strip) * kTileCols;
  const int ncols = static_cast<int>(min(static_cast<int64_t>(kTileCols), td.cols - col0));
  const int64_t row0 = static_cast<int64_t>(rt) * kTileRows;
  const int64_t row_end = min(row0 + kTileRows, td.rows);
  const int cl = threadIdx.x & 63, rg = threadIdx.x >> 6, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t tid = static_cast<uint32_t>(td.id);
  const int r = cb != 0.0f ? td.rank : 0;
  for (int idx = threadIdx.x; idx < r * 64; idx += kNormThreads) {
    const int k = idx >> 6, c = idx & 63;
    if (c < ncols) Gs[k][c] = coeff1<BITS, true>(td, keys, unit, cb, k, col0 + c);
  }
  __syncthreads();
  double s0 = 0.0, s1 = 0.0, s2 = 0.0;
  if (cl < ncols) {
    for (int64_t row = row0 + rg; row < row_end; row += kNormThreads / 64) {
      const int64_t e = row * td.cols + col0 + cl;
      const float zi = normal1<BITS, true>(keys, tid, 0u, static_cast<uint64_t>(e), iso);
      float gd = 0.0f;
      for (int k = 0; k < r; ++k) gd = fmaf(__ldg(td.U + row * td.rank + k), Gs[k][cl], gd);
      s0 += static_cast<double>(zi) * zi;
      s1 += static_cast<double>(gd) * gd;
      s2 += static_cast<double>(zi + gd) * (zi + gd);
    }
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    s0 += __shfl_xor_sync(0xFFFFFFFFu, s0, off);
    s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, off);
    s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, off);
  }
  if (lane == 0) {
    red[warp][0] = s0; red[warp][1] = s1; red[warp][2] = s2;
  }
  __syncthreads();
  if (threadIdx.x < 3) {
    double t = 0.0;
    for (int w = 0; w < kNormThreads / 32; ++w) t += red[w][threadIdx.x];   // fixed order
    partials[3 * tile + threadIdx.x] = t;
  }
}

// Sum the tile partials in a fixed order (same bits on every run) into the caller's three doubles.
__global__ void __launch_bounds__(kNormThreads) norms_finish_kernel(const double* __restrict__ partials, int n_tiles, double* __restrict__ out3) {
  __shared__ double red[kNormThreads][3];
  double t[3] = {0.0, 0.0, 0.0};
  for (int i = threadIdx.x; i < n_tiles; i += kNormThreads)
    for (int j = 0; j < 3; ++j) t[j] += partials[3 * i + j];
  for (int j = 0; j < 3; ++j) red[threadIdx.x][j] = t[j];
  __syncthreads();
  for (int half = kNormThreads / 2; half > 0; half >>= 1) {
    if (threadIdx.x < half)
      for (int j = 0; j < 3; ++j) red[threadIdx.x][j] += red[threadIdx.x + half][j];
    __syncthreads();
  }
  if (threadIdx.x < 3) out3[threadIdx.x] = red[0][threadIdx.x];
}

}  // namespace
}  // namespace zgr

using namespace zgr;

extern "C" int zgr_tensor_norms_noalloc(zgr_ctx* ctx, uint64_t seed, int32_t tensor, double* dev_out3, void* stream) {
  TensorDesc td;
  double a, b;
  int bits, sticky, ctx_device;
  if (!dev_out3 || (reinterpret_cast<uintptr_t>(dev_out3) & 7) != 0) return ZGR_EINVAL;
  if (!host_ctx_view(ctx, tensor, &td, &a, &b, &bits, &sticky, &ctx_device)) return ZGR_EINVAL;
  if (sticky) return sticky;
  const int64_t strips = (td.cols + kTileCols - 1) / kTileCols;
  const int64_t row_tiles = (td.rows + kTileRows - 1) / kTileRows;
  if (strips * row_tiles > ZGR_NOALLOC_MAX_TILES) return ZGR_ETOOBIG;   // the fixed scratch cannot hold this tensor's partial sums

  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ZGR_ECUDA;
  // The tensor's subspace and coefficient pointers belong to the context's device; the scratch address
  // below belongs to the current one.  They must be the same device.
  if (zgr_debug_check_device(ctx_device, dev) != ZGR_OK) return ZGR_EINVAL;
  if (g_partials_addr[dev] == nullptr) {
    // One-time set-up on this device: translate the symbol into a device address.  (The symbol's
    // name is only a host-side handle; passing it to a kernel directly would hand the GPU a host address.)
    double* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_norm_partials) != cudaSuccess || p == nullptr) return ZGR_ECUDA;
    g_partials_addr[dev] = p;
  }
  double* partials = g_partials_addr[dev];

  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const PhiloxKeys keys = host_make_keys(seed);
  const NormalScale iso = host_make_scale(a, bits);
  const NormalScale unit = host_make_scale(1.0, bits);
  const float cb = static_cast<float>(b);
  const int n_tiles = static_cast<int>(strips * row_tiles);
  if (bits == 32) norms_tile_kernel<32><<<n_tiles, kNormThreads, 0, st>>>(td, keys, iso, unit, cb, static_cast<int>(row_tiles), partials);
  else norms_tile_kernel<16><<<n_tiles, kNormThreads, 0, st>>>(td, keys, iso, unit, cb, static_cast<int>(row_tiles), partials);
  if (cudaGetLastError() != cudaSuccess) return ZGR_ECUDA;
  norms_finish_kernel<<<1, kNormThreads, 0, st>>>(partials, n_tiles, dev_out3);
  if (cudaGetLastError() != cudaSuccess) return ZGR_ECUDA;
  return ZGR_OK;
}
