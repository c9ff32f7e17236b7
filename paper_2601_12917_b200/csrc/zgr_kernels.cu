// Sweep kernels of the ZGR step for sm_100a:   theta <- rnd(theta + c * (a Z + b U G)).
//
// Eq. (perturbation) builds the perturbation, Algorithm 1 applies it three times per step with
// c = +eps, -2 eps and (eps - lr (L+ - L-)/(2 eps)); every application is one of the kernels below.
// The weights are read once and written once per sweep (HBM-bound); Z, G and U G are regenerated
// in registers / shared memory and never stored.
//
//   sweep_iso      tensors without a subspace (1-D tensors, rank 0) or with b = 0
//   sweep_fma      rank <= 8: U G on CUDA-core FMAs in fp32, G strip in shared memory and registers
//   sweep_mma      rank  > 8: U G on tensor cores, bf16 hi/lo split operands (three products per
//                  tile, fp32 accumulate), accumulators initialised with theta so the tensor-core
//                  result is already theta + c b U G in the register layout of the 128-bit stores
//   sweep_generic  any shape or alignment, one element per thread (correctness fallback)
//
// All kernels are persistent over a device-resident list of work items (static round-robin), so a
// sweep over a model with hundreds of tensors is a handful of launches.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cmath>

#include "zgr_device.cuh"
#include "zgr_kernels.h"

namespace zgr {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

// Rows ahead that the CUDA-core kernel prefetches into L2 (0 = off).
#ifndef ZGR_FMA_PREFETCH
#define ZGR_FMA_PREFETCH 2
#endif

// ---------------------------------------------------------------------------------------------
// isotropic sweep
// ---------------------------------------------------------------------------------------------
// SSTATS = true (single-term sweeps only) also accumulates the norm bookkeeping of the sweep: per work item and
// warp the sums of (c a Z)^2, (c b U G)^2 and (c z)^2 over its elements, stored in the item's slots (the
// finishing kernel adds them up per tensor in a fixed order; the host divides by c^2).
template <typename T, int BITS, bool PRECISE, bool MULTI, bool SSTATS = false>
__global__ void __launch_bounds__(kThreads) sweep_iso_kernel(const __grid_constant__ SweepParams p) {
  for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
    const WorkItem w = p.items[it];
    const TensorDesc& td = p.tensors[w.tensor];
    T* base = static_cast<T*>(td.data);
    const uint32_t tid = static_cast<uint32_t>(td.id);
    const int64_t e0 = w.row0_or_e0, count = w.nrows_or_count;
    const int64_t n_oct = w.ncols ? count / 8 : 0;  // ncols != 0: 128-bit access is legal for this tensor
    double s_iso = 0.0;
#pragma unroll 2
    for (int64_t v = threadIdx.x; v < n_oct; v += kThreads) {
      const int64_t e = e0 + 8 * v;
      float th[8], z[8];
      Storage<T>::load8(base + e, th);
      iso8<BITS, PRECISE, MULTI>(p, tid, static_cast<uint64_t>(e), z);
      if (SSTATS) {
        float f = 0.0f;
#pragma unroll
        for (int i = 0; i < 8; ++i) f = fmaf(z[i], z[i], f);
        s_iso += static_cast<double>(f);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) th[i] += z[i];
      Storage<T>::store8(base + e, th);
    }
    for (int64_t e = e0 + 8 * n_oct + threadIdx.x; e < e0 + count; e += kThreads) {
      const float z = iso1<BITS, PRECISE, MULTI>(p, tid, static_cast<uint64_t>(e));
      if (SSTATS) s_iso += static_cast<double>(z) * z;
      Storage<T>::store1(base + e, Storage<T>::load1(base + e) + z);
    }
    if (SSTATS) store_item_stats(p, it, threadIdx.x >> 5, s_iso, 0.0, s_iso);
  }
}

// ---------------------------------------------------------------------------------------------
// rank <= R (R = 4 or 8): CUDA-core contraction.
// A CTA owns a strip of up to 256 columns; lane l of every warp owns the octet of columns
// [8l, 8l+8) of the strip and keeps its R x 8 coefficients in registers; the eight warps walk
// the rows of the item in an interleaved fashion, each row being one 128-bit access per lane.
// ---------------------------------------------------------------------------------------------
template <typename T, int BITS, bool PRECISE, int R, bool MULTI, bool SSTATS = false>
__global__ void __launch_bounds__(kThreads, 2) sweep_fma_kernel(const __grid_constant__ SweepParams p) {
  __shared__ float Gs[R][256 + 8];
  __shared__ int next_item;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (;;) {
    // Items are handed out in order by a counter in global memory: the models this kernel serves have few items per
    // CTA (about 18 for a RoBERTa-large-sized set), so a fixed assignment leaves the SMs that drew one item fewer
    // idle for 3-5 % of the sweep.  Every CTA makes exactly one fetch beyond the end; the last of those puts the
    // counter back to zero for the next launch (launches that share a counter are ordered by their stream).
    __syncthreads();  // readers of the previous strip and of next_item are done
    if (threadIdx.x == 0) {
      const int t = atomicAdd(p.sched, 1);
      if (t == p.n_items + static_cast<int>(gridDim.x) - 1) *p.sched = 0;
      next_item = t;
    }
    __syncthreads();
    const int it = next_item;
    if (it >= p.n_items) break;
    const WorkItem w = p.items[it];
    const TensorDesc& td = p.tensors[w.tensor];
    T* base = static_cast<T*>(td.data);
    const uint32_t tid = static_cast<uint32_t>(td.id);
    const int r = td.rank;
    const int64_t cols = td.cols;
    for (int idx = threadIdx.x; idx < R * 32; idx += kThreads) {
      const int k = idx >> 5, o = idx & 31;
      if (8 * o < w.ncols) {
        float g[8];
        if (k < r) {
          guided8<BITS, PRECISE, MULTI>(td, p, k, w.col0 + 8 * o, g);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) g[i] = 0.0f;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) Gs[k][8 * o + i] = g[i];
      }
    }
    __syncthreads();
    const bool active = 8 * lane < w.ncols;
    float g[R][8];
#pragma unroll
    for (int k = 0; k < R; ++k)
#pragma unroll
      for (int i = 0; i < 8; ++i) g[k][i] = active ? Gs[k][8 * lane + i] : 0.0f;
    const bool u_vec = (r == R) && ((reinterpret_cast<uintptr_t>(td.U) & 15) == 0);
    const int64_t row_end = w.row0_or_e0 + w.nrows_or_count;
    double s_iso = 0.0, s_gd = 0.0, s_z = 0.0;   // SSTATS only
    for (int64_t row = w.row0_or_e0 + warp; row < row_end; row += kWarps) {
#if ZGR_FMA_PREFETCH
      // this warp's row after next: start it on its way from HBM to L2 now (each lane asks for its own 8 elements);
      // with four warps per scheduler there is not enough other work to cover a full DRAM round trip otherwise
      if (active && row + ZGR_FMA_PREFETCH * kWarps < row_end) {
        const T* nxt = base + (row + ZGR_FMA_PREFETCH * kWarps) * cols + w.col0 + 8 * lane;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(nxt));
      }
#endif
      float u[R];
      if (u_vec) {
#pragma unroll
        for (int k4 = 0; k4 < R / 4; ++k4) {
          const float4 q = __ldg(reinterpret_cast<const float4*>(td.U + row * R) + k4);
          u[4 * k4] = q.x; u[4 * k4 + 1] = q.y; u[4 * k4 + 2] = q.z; u[4 * k4 + 3] = q.w;
        }
      } else {
#pragma unroll
        for (int k = 0; k < R; ++k) u[k] = k < r ? __ldg(td.U + row * r + k) : 0.0f;
      }
      if (active) {
        const int64_t e = row * cols + w.col0 + 8 * lane;
        float th[8], z[8];
        Storage<T>::load8(base + e, th);
        iso8<BITS, PRECISE, MULTI>(p, tid, static_cast<uint64_t>(e), z);
        float f_iso = 0.0f, f_gd = 0.0f, f_z = 0.0f;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          float acc = z[i];  // the perturbation is summed on its own scale, then added to theta once
#pragma unroll
          for (int k = 0; k < R; ++k) acc = fmaf(u[k], g[k][i], acc);
          if (SSTATS) {
            const float gd = acc - z[i];
            f_iso = fmaf(z[i], z[i], f_iso);
            f_gd = fmaf(gd, gd, f_gd);
            f_z = fmaf(acc, acc, f_z);
          }
          th[i] += acc;
        }
        if (SSTATS) {
          s_iso += static_cast<double>(f_iso);
          s_gd += static_cast<double>(f_gd);
          s_z += static_cast<double>(f_z);
        }
        Storage<T>::store8(base + e, th);
      }
    }
    if (SSTATS) store_item_stats(p, it, warp, s_iso, s_gd, s_z);
  }
}

// ---------------------------------------------------------------------------------------------
// any shape: one element per thread, strip of 64 columns, rank <= 64.
// ---------------------------------------------------------------------------------------------
template <typename T, int BITS, bool PRECISE, bool MULTI, bool SSTATS = false>
__global__ void __launch_bounds__(kThreads) sweep_generic_kernel(const __grid_constant__ SweepParams p) {
  __shared__ float Gs[64][64 + 1];
  const int cl = threadIdx.x & 63, rg = threadIdx.x >> 6;
  for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
    const WorkItem w = p.items[it];
    const TensorDesc& td = p.tensors[w.tensor];
    T* base = static_cast<T*>(td.data);
    const uint32_t tid = static_cast<uint32_t>(td.id);
    const int r = td.rank;
    __syncthreads();
    for (int idx = threadIdx.x; idx < r * 64; idx += kThreads) {
      const int k = idx >> 6, c = idx & 63;
      if (c < w.ncols) Gs[k][c] = guided1<BITS, PRECISE, MULTI>(td, p, k, w.col0 + c);
    }
    __syncthreads();
    double s_iso = 0.0, s_gd = 0.0, s_z = 0.0;   // SSTATS only
    if (cl < w.ncols) {
      const int64_t row_end = w.row0_or_e0 + w.nrows_or_count;
      for (int64_t row = w.row0_or_e0 + rg; row < row_end; row += kThreads / 64) {
        const int64_t e = row * td.cols + w.col0 + cl;
        const float iso = iso1<BITS, PRECISE, MULTI>(p, tid, static_cast<uint64_t>(e));
        float acc = iso;
        for (int k = 0; k < r; ++k) acc = fmaf(__ldg(td.U + row * r + k), Gs[k][cl], acc);
        if (SSTATS) {
          const float gd = acc - iso;
          s_iso += static_cast<double>(iso) * iso;
          s_gd += static_cast<double>(gd) * gd;
          s_z += static_cast<double>(acc) * acc;
        }
        Storage<T>::store1(base + e, Storage<T>::load1(base + e) + acc);
      }
    }
    if (SSTATS) store_item_stats(p, it, threadIdx.x >> 5, s_iso, s_gd, s_z);
  }
}

// ---------------------------------------------------------------------------------------------
// rank > 8: tensor-core contraction (mma.sync m16n8k16, bf16 operands, fp32 accumulate).
//
// Operand precision.  U and c b G are each split into bf16 hi + bf16 lo; the tile product is
// Uhi Ghi + Ulo Ghi + Uhi Glo, i.e. about 2^-16 relative error per term, accumulated in fp32.
//
// Register layout.  A warp owns 16 rows x 64 columns.  In the m16n8k16 accumulator a thread
// (g = lane/4, t = lane%4) holds rows g and g+8, columns 2t, 2t+1 of every 8-wide tile.  The "n"
// index of the contraction is only a label for a column, so tile j and slot p are assigned the
// real column  32 (j/4) + 8 (p/2) + 2 (j%4) + (p%2):  thread t then owns the 8 contiguous columns
// [8t, 8t+8) (tiles 0-3) and [32+8t, 32+8t+8) (tiles 4-7) of each of its two rows, which is exactly
// one 128-bit access per (row, half) for 16-bit weights.  The coefficient strip is written to
// shared memory in that same tile order, so ldmatrix returns B fragments for it directly.
//
// U arrives pre-split and pre-ordered (TensorDesc::Ufrag): for row tile m, k-step s, part
// (hi|lo), lane: one uint4 holding the four A registers, so an A fragment is one coalesced 128-bit
// load, served from L1/L2 for all warps of the CTA that share the rows.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(smem_addr));
}

// bf16 hi/lo split of a pair of floats, packed as bf16x2 (first value in the low half).
__device__ __forceinline__ void split2(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  const float r0 = x0 - __uint_as_float(hi << 16);
  const float r1 = x1 - __uint_as_float(hi & 0xFFFF0000u);
  const __nv_bfloat162 l = __floats2bfloat162_rn(r0, r1);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// Storage row (tile order) of real column c64 in [0, 64) of a warp's column group.
__device__ __forceinline__ int tile_row_of_column(int c64) {
  const int hf = c64 >> 5, c32 = c64 & 31, t = c32 >> 3, o = c32 & 7;
  const int j = 4 * hf + (o >> 1), pp = 2 * t + (o & 1);
  return 8 * j + pp;
}

// XOR swizzle of the 16-byte chunk index inside a coefficient row of KP bf16 (KP/8 chunks), chosen
// so that the eight rows read by one ldmatrix phase fall into eight different bank groups.
template <int KP>
__device__ __forceinline__ int chunk_swizzle(int row) {
  const int pp = row & 7;
  return KP == 16 ? ((pp >> 2) & 1) : (KP == 32 ? ((pp >> 1) & 3) : pp);
}

template <typename T, int BITS, bool PRECISE, int KP, int WM>
__global__ void __launch_bounds__(kThreads, 2) sweep_mma_kernel(const __grid_constant__ SweepParams p) {
  constexpr int WN = kWarps / WM;          // warps side by side along the columns
  constexpr int STRIP = WN * 64;           // columns per CTA strip
  constexpr int KS = KP / 16;              // k-steps
  constexpr int CH = KP / 8;               // 16-byte chunks per coefficient row
  extern __shared__ __align__(16) uint32_t smem[];
  uint32_t* Ghi = smem;                    // [STRIP][KP/2] words, swizzled chunks
  uint32_t* Glo = smem + STRIP * (KP / 2);

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wm = warp / WN, wn = warp % WN;
  const int g = lane >> 2, t = lane & 3;

  for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
    const WorkItem w = p.items[it];
    const TensorDesc& td = p.tensors[w.tensor];
    T* base = static_cast<T*>(td.data);
    const uint32_t tid = static_cast<uint32_t>(td.id);
    const int r = td.rank;
    const int64_t cols = td.cols;

    // ---- coefficient strip: (k pair, column octet) -> hi/lo words in tile order ----
    __syncthreads();
    for (int idx = threadIdx.x; idx < (KP / 2) * (STRIP / 8); idx += kThreads) {
      const int kp = idx / (STRIP / 8), o = idx % (STRIP / 8);
      const int c = 8 * o;
      float g0[8], g1[8];
      if (c < w.ncols && 2 * kp < r) {
        guided8<BITS, PRECISE, false>(td, p, 2 * kp, w.col0 + c, g0);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) g0[i] = 0.0f;
      }
      if (c < w.ncols && 2 * kp + 1 < r) {
        guided8<BITS, PRECISE, false>(td, p, 2 * kp + 1, w.col0 + c, g1);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) g1[i] = 0.0f;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int cc = c + i;
        const int row = (cc & ~63) + tile_row_of_column(cc & 63);
        const int word = (row * CH + ((kp >> 2) ^ chunk_swizzle<KP>(row))) * 4 + (kp & 3);
        uint32_t hi, lo;
        split2(g0[i], g1[i], hi, lo);
        Ghi[word] = hi;
        Glo[word] = lo;
      }
    }
    __syncthreads();

    // ---- rows ----
    const int64_t row_end = w.row0_or_e0 + w.nrows_or_count;
    const int64_t colw = w.col0 + 64 * wn;                     // first column of this warp's group
    const bool act0 = 64 * wn + 8 * t < w.ncols;               // columns [8t, 8t+8) of the group
    const bool act1 = 64 * wn + 32 + 8 * t < w.ncols;          // columns [32+8t, 32+8t+8)
    if (!act0 && !act1 && 64 * wn >= w.ncols) continue;        // whole warp outside the strip
    const uint32_t sm_base = static_cast<uint32_t>(__cvta_generic_to_shared(lane < 16 ? Ghi : Glo));
    for (int64_t row0 = w.row0_or_e0 + 16 * wm; row0 < row_end; row0 += 16 * WM) {
      const int64_t rows2[2] = {row0 + g, row0 + g + 8};
      float acc[8][4];
      // accumulators start as theta
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const bool rok = rows2[h] < row_end;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          float th[8];
          if (rok && (hf ? act1 : act0)) {
            Storage<T>::load8(base + rows2[h] * cols + colw + 32 * hf + 8 * t, th);
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) th[i] = 0.0f;
          }
#pragma unroll
          for (int i = 0; i < 8; ++i) acc[4 * hf + (i >> 1)][2 * h + (i & 1)] = th[i];
        }
      }
      // A fragments of this row tile
      const uint4* uf = td.Ufrag + (static_cast<int64_t>(row0 >> 4) * KS * 2) * 32 + lane;
      uint4 ahi[KS], alo[KS];
#pragma unroll
      for (int s = 0; s < KS; ++s) {
        ahi[s] = __ldg(uf + (2 * s) * 32);
        alo[s] = __ldg(uf + (2 * s + 1) * 32);
      }
      // tensor-core contraction
#pragma unroll
      for (int j = 0; j < 8; ++j) {
#pragma unroll
        for (int s = 0; s < KS; ++s) {
          const int row = 64 * wn + 8 * j + (lane & 7);
          const int chunk = (2 * s + ((lane >> 3) & 1)) ^ chunk_swizzle<KP>(row);
          uint32_t b[4];
          ldmatrix_x4(b, sm_base + static_cast<uint32_t>((row * CH + chunk) * 16));
          mma_bf16(acc[j], alo[s], b[0], b[1]);
          mma_bf16(acc[j], ahi[s], b[2], b[3]);
          mma_bf16(acc[j], ahi[s], b[0], b[1]);
        }
      }
      // isotropic part, rounding, store
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const bool rok = rows2[h] < row_end;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          if (rok && (hf ? act1 : act0)) {
            const int64_t e = rows2[h] * cols + colw + 32 * hf + 8 * t;
            float z[8], th[8];
            iso8<BITS, PRECISE, false>(p, tid, static_cast<uint64_t>(e), z);
#pragma unroll
            for (int i = 0; i < 8; ++i) th[i] = acc[4 * hf + (i >> 1)][2 * h + (i & 1)] + z[i];
            Storage<T>::store8(base + e, th);
          }
        }
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Norm bookkeeping: per tensor sum (a Z)^2, sum (b U G)^2, sum z^2 (no weights are read).
// Same tiling as the generic kernel; fp32 per element, double partial sums, one slot per warp and work item
// (summed per tensor in a fixed order by stats_finish_kernel, so repeated calls give identical bits).
// ---------------------------------------------------------------------------------------------
template <int BITS>
__global__ void __launch_bounds__(kThreads) stats_kernel(const __grid_constant__ SweepParams p) {
  __shared__ float Gs[64][64 + 1];
  const int cl = threadIdx.x & 63, rg = threadIdx.x >> 6;
  for (int it = blockIdx.x; it < p.n_items; it += gridDim.x) {
    const WorkItem w = p.items[it];
    const TensorDesc& td = p.tensors[w.tensor];
    const uint32_t tid = static_cast<uint32_t>(td.id);
    const int r = p.term[0].cb != 0.0f ? td.rank : 0;
    __syncthreads();
    for (int idx = threadIdx.x; idx < r * 64; idx += kThreads) {
      const int k = idx >> 6, c = idx & 63;
      if (c < w.ncols) Gs[k][c] = guided1<BITS, true, false>(td, p, k, w.col0 + c);
    }
    __syncthreads();
    double s0 = 0.0, s1 = 0.0, s2 = 0.0;
    if (cl < w.ncols) {
      const int64_t row_end = w.row0_or_e0 + w.nrows_or_count;
      for (int64_t row = w.row0_or_e0 + rg; row < row_end; row += kThreads / 64) {
        const int64_t e = row * td.cols + w.col0 + cl;
        const float iso = iso1<BITS, true, false>(p, tid, static_cast<uint64_t>(e));
        float gd = 0.0f;
        for (int k = 0; k < r; ++k) gd = fmaf(__ldg(td.U + row * td.rank + k), Gs[k][cl], gd);
        s0 += static_cast<double>(iso) * iso;
        s1 += static_cast<double>(gd) * gd;
        s2 += static_cast<double>(iso + gd) * (iso + gd);
      }
    }
    store_item_stats(p, it, threadIdx.x >> 5, s0, s1, s2);
  }
}

// out[3 l + j] = sum over the work items of tensor l and their slots, in a fixed order.
__global__ void __launch_bounds__(kThreads) stats_finish_kernel(const StatRange* __restrict__ ranges, double* __restrict__ out) {
  __shared__ double red[kThreads][3];
  const StatRange r = ranges[blockIdx.x];
  double t[3] = {0.0, 0.0, 0.0};
  for (int i = threadIdx.x; i < r.count; i += kThreads) {
    const double* src = r.slots + static_cast<int64_t>(r.first + i) * kStatSlots * 3;
    for (int sl = 0; sl < kStatSlots; ++sl)
      for (int j = 0; j < 3; ++j) t[j] += src[3 * sl + j];
  }
  for (int j = 0; j < 3; ++j) red[threadIdx.x][j] = t[j];
  __syncthreads();
  for (int half = kThreads / 2; half > 0; half >>= 1) {
    if (threadIdx.x < half)
      for (int j = 0; j < 3; ++j) red[threadIdx.x][j] += red[threadIdx.x + half][j];
    __syncthreads();
  }
  if (threadIdx.x < 3) out[3 * blockIdx.x + threadIdx.x] = red[0][threadIdx.x];
}

// U (rows x r fp32) -> A-operand fragments, bf16 hi/lo, zero padded to whole 16-row tiles and to KP.
__global__ void split_subspace_kernel(const float* __restrict__ U, int64_t rows, int r, int kp, uint4* __restrict__ out, int64_t n_out) {
  const int64_t idx = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;  // ((tile*KS + s)*2 + part)*32 + lane
  if (idx >= n_out) return;
  const int lane = static_cast<int>(idx & 31);
  const int part = static_cast<int>((idx >> 5) & 1);
  const int64_t ts = idx >> 6;
  const int ks = kp / 16;
  const int s = static_cast<int>(ts % ks);
  const int64_t tile = ts / ks;
  const int g = lane >> 2, t = lane & 3;
  uint32_t regs[4];
#pragma unroll
  for (int q = 0; q < 4; ++q) {
    const int64_t row = tile * 16 + g + ((q & 1) ? 8 : 0);
    const int k = 16 * s + 2 * t + ((q & 2) ? 8 : 0);
    const float x0 = (row < rows && k < r) ? U[row * r + k] : 0.0f;
    const float x1 = (row < rows && k + 1 < r) ? U[row * r + k + 1] : 0.0f;
    uint32_t hi, lo;
    split2(x0, x1, hi, lo);
    regs[q] = part ? lo : hi;
  }
  out[idx] = make_uint4(regs[0], regs[1], regs[2], regs[3]);
}

// U (rows x r fp32) -> two row-major fp16 matrices (hi, lo) holding U * 2^shift, rows padded to a multiple of
// 128 and columns to KP with zeros: the TMA source of the A operand of the tcgen05 kernel.  hi + lo carries
// 22 significant bits as long as the scaled entry is not far below 1 (lo must stay a normal fp16 number).
__device__ __forceinline__ void split_f16_scaled(float x, float scale, __half& hi, __half& lo) {
  const float y = x * scale;                       // power of two: exact
  hi = __float2half_rn(y);
  lo = __float2half_rn(y - __half2float(hi));
}

__global__ void split_subspace_rowmajor_kernel(const float* __restrict__ U, int64_t rows, int r, int kp, int64_t rows_pad, float scale,
                                               __half* __restrict__ hi, __half* __restrict__ lo) {
  const int64_t idx = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
  if (idx >= rows_pad * kp) return;
  const int64_t row = idx / kp;
  const int k = static_cast<int>(idx % kp);
  const float x = (row < rows && k < r) ? U[row * r + k] : 0.0f;
  split_f16_scaled(x, scale, hi[idx], lo[idx]);
}

__global__ void split_subspace_rowmajor_all_kernel(const SplitJob* __restrict__ jobs) {
  const SplitJob j = jobs[blockIdx.y];
  const int64_t n = j.rows_pad * j.kp;
  __half* hi = static_cast<__half*>(j.hi);
  __half* lo = static_cast<__half*>(j.lo);
  const float scale = __int_as_float((127 + j.shift) << 23);
  for (int64_t idx = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; idx < n; idx += static_cast<int64_t>(gridDim.x) * blockDim.x) {
    const int64_t row = idx / j.kp;
    const int k = static_cast<int>(idx % j.kp);
    const float x = (row < j.rows && k < j.r) ? j.U[row * j.r + k] : 0.0f;
    split_f16_scaled(x, scale, hi[idx], lo[idx]);
  }
}

// Raw generator blocks (test hook).
__global__ void philox_blocks_kernel(PhiloxKeys keys, uint32_t tensor, uint32_t tag, uint64_t first_block, int64_t n_blocks,
                                     uint32_t* __restrict__ out) {
  const int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x;
  if (i >= n_blocks) return;
  uint32_t x[4];
  philox_block(first_block + static_cast<uint64_t>(i), tensor, tag, keys, x);
  reinterpret_cast<uint4*>(out)[i] = make_uint4(x[0], x[1], x[2], x[3]);
}

// ---------------------------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------------------------
namespace {

template <typename T, int BITS, bool PRECISE, bool MULTI>
cudaError_t launch_typed(const KernelChoice& kc, const SweepParams& p, int grid, cudaStream_t st) {
  if constexpr (!MULTI) {
    if (p.item_stats != nullptr) {      // the sweep also accumulates the norm bookkeeping
      switch (kc.path) {
        case PATH_ISO:
          sweep_iso_kernel<T, BITS, PRECISE, false, true><<<grid, kThreads, 0, st>>>(p);
          return cudaGetLastError();
        case PATH_FMA:
          if (kc.kpad == 4) sweep_fma_kernel<T, BITS, PRECISE, 4, false, true><<<grid, kThreads, 0, st>>>(p);
          else sweep_fma_kernel<T, BITS, PRECISE, 8, false, true><<<grid, kThreads, 0, st>>>(p);
          return cudaGetLastError();
        case PATH_GENERIC:
          sweep_generic_kernel<T, BITS, PRECISE, false, true><<<grid, kThreads, 0, st>>>(p);
          return cudaGetLastError();
        default:
          return cudaErrorInvalidValue;  // the legacy tensor-core kernel keeps no bookkeeping; the host does not ask it to
      }
    }
  }
  switch (kc.path) {
    case PATH_ISO:
      sweep_iso_kernel<T, BITS, PRECISE, MULTI><<<grid, kThreads, 0, st>>>(p);
      break;
    case PATH_FMA:
      if (kc.kpad == 4) sweep_fma_kernel<T, BITS, PRECISE, 4, MULTI><<<grid, kThreads, 0, st>>>(p);
      else sweep_fma_kernel<T, BITS, PRECISE, 8, MULTI><<<grid, kThreads, 0, st>>>(p);
      break;
    case PATH_GENERIC:
      sweep_generic_kernel<T, BITS, PRECISE, MULTI><<<grid, kThreads, 0, st>>>(p);
      break;
    case PATH_MMA: {
      if constexpr (PRECISE || MULTI) {
        return cudaErrorInvalidValue;  // the split-bf16 contraction cannot meet the fp32 tolerance; several terms go through the tcgen05 or the fallback kernel
      } else {
        const size_t smem = mma_smem_bytes(kc.kpad);
        if (kc.kpad == 16) {
          auto k = sweep_mma_kernel<T, BITS, false, 16, 1>;
          cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
          k<<<grid, kThreads, smem, st>>>(p);
        } else if (kc.kpad == 32) {
          auto k = sweep_mma_kernel<T, BITS, false, 32, 1>;
          cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
          k<<<grid, kThreads, smem, st>>>(p);
        } else {
          auto k = sweep_mma_kernel<T, BITS, false, 64, 2>;
          cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
          k<<<grid, kThreads, smem, st>>>(p);
        }
      }
      break;
    }
    default:
      return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

template <typename T, bool MULTI>
cudaError_t launch_dtype(const KernelChoice& kc, const SweepParams& p, int grid, cudaStream_t st) {
  if (kc.precise) {
    if constexpr (sizeof(T) == 4) {
      if (kc.bits == 32) return launch_typed<T, 32, true, MULTI>(kc, p, grid, st);
      return launch_typed<T, 16, true, MULTI>(kc, p, grid, st);
    } else {
      return cudaErrorInvalidValue;  // 16-bit storage never needs the accurate transform
    }
  }
  if (kc.bits == 32) return launch_typed<T, 32, false, MULTI>(kc, p, grid, st);
  return launch_typed<T, 16, false, MULTI>(kc, p, grid, st);
}

}  // namespace

int mma_strip_cols(int kpad) { return kpad == 64 ? 256 : 512; }
int mma_rows_per_iter(int kpad) { return kpad == 64 ? 32 : 16; }
size_t mma_smem_bytes(int kpad) { return static_cast<size_t>(mma_strip_cols(kpad)) * kpad * 2 * 2; }

cudaError_t launch_sweep(const KernelChoice& kc, const SweepParams& p, int grid, cudaStream_t st) {
  if (p.n_terms > 1) {
    switch (kc.dtype) {
      case 0: return launch_dtype<float, true>(kc, p, grid, st);
      case 1: return launch_dtype<__half, true>(kc, p, grid, st);
      case 2: return launch_dtype<__nv_bfloat16, true>(kc, p, grid, st);
      default: return cudaErrorInvalidValue;
    }
  }
  switch (kc.dtype) {
    case 0: return launch_dtype<float, false>(kc, p, grid, st);
    case 1: return launch_dtype<__half, false>(kc, p, grid, st);
    case 2: return launch_dtype<__nv_bfloat16, false>(kc, p, grid, st);
    default: return cudaErrorInvalidValue;
  }
}

cudaError_t launch_stats(int bits, const SweepParams& p, int grid, cudaStream_t st) {
  if (bits == 32) stats_kernel<32><<<grid, kThreads, 0, st>>>(p);
  else stats_kernel<16><<<grid, kThreads, 0, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_stats_finish(const StatRange* d_ranges, int n_tensors, double* d_out, cudaStream_t st) {
  if (n_tensors <= 0) return cudaSuccess;
  stats_finish_kernel<<<n_tensors, kThreads, 0, st>>>(d_ranges, d_out);
  return cudaGetLastError();
}

cudaError_t launch_split_subspace(const float* U, int64_t rows, int r, int kp, uint4* out, cudaStream_t st) {
  const int64_t tiles = (rows + 15) / 16;
  const int64_t n_out = tiles * (kp / 16) * 2 * 32;
  const int block = 256;
  const int64_t grid = (n_out + block - 1) / block;
  split_subspace_kernel<<<static_cast<unsigned>(grid), block, 0, st>>>(U, rows, r, kp, out, n_out);
  return cudaGetLastError();
}

cudaError_t launch_split_subspace_rowmajor_all(const SplitJob* d_jobs, int n_jobs, cudaStream_t st) {
  if (n_jobs <= 0) return cudaSuccess;
  split_subspace_rowmajor_all_kernel<<<dim3(64, static_cast<unsigned>(n_jobs)), 256, 0, st>>>(d_jobs);
  return cudaGetLastError();
}

cudaError_t launch_split_subspace_rowmajor(const float* U, int64_t rows, int r, int kp, int64_t rows_pad, int shift, void* hi, void* lo, cudaStream_t st) {
  const int64_t n = rows_pad * kp;
  const int block = 256;
  split_subspace_rowmajor_kernel<<<static_cast<unsigned>((n + block - 1) / block), block, 0, st>>>(
      U, rows, r, kp, rows_pad, std::ldexp(1.0f, shift), static_cast<__half*>(hi), static_cast<__half*>(lo));
  return cudaGetLastError();
}

cudaError_t launch_philox_blocks(const PhiloxKeys& keys, uint32_t tensor, uint32_t tag, uint64_t first_block, int64_t n_blocks,
                                 uint32_t* out, cudaStream_t st) {
  const int block = 256;
  const int64_t grid = (n_blocks + block - 1) / block;
  philox_blocks_kernel<<<static_cast<unsigned>(grid), block, 0, st>>>(keys, tensor, tag, first_block, n_blocks, out);
  return cudaGetLastError();
}

}  // namespace zgr
