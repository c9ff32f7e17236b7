// Device-side building blocks of the ZGR sweeps: the counter-based generator, the Gaussian
// transform, and 8-element ("octet") access to the three storage types.
#ifndef ZGR_DEVICE_CUH_
#define ZGR_DEVICE_CUH_

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "zgr_internal.h"

#ifndef ZGR_DTC_VECTOR
#define ZGR_DTC_VECTOR 1
#endif

namespace zgr {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11).  The paper asks only that client and edge server
// regenerate the same perturbation from a shared seed (Algorithm 1); a counter-based generator
// makes every element a pure function of (seed, tensor, stream tag, element index), so any tiling
// of the sweep produces the same bits.  Round keys arrive precomputed in the kernel parameters and
// become constant-bank operands of the xors.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKeys& k,
                                              uint32_t (&x)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = static_cast<uint64_t>(0xD2511F53u) * c0;
    const uint64_t p1 = static_cast<uint64_t>(0xCD9E8D57u) * c2;
    const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ k.k0[r];
    const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ k.k1[r];
    c1 = static_cast<uint32_t>(p1);
    c3 = static_cast<uint32_t>(p0);
    c0 = n0;
    c2 = n2;
  }
  x[0] = c0; x[1] = c1; x[2] = c2; x[3] = c3;
}

__device__ __forceinline__ void philox_block(uint64_t j, uint32_t tensor, uint32_t tag, const PhiloxKeys& k, uint32_t (&x)[4]) {
  philox4x32_10(static_cast<uint32_t>(j), static_cast<uint32_t>(j >> 32), tensor, tag, k, x);
}

// ---------------------------------------------------------------------------------------------
// Box-Muller on odd-numerator uniforms  u = (2k+1) / 2^(nb+1),  k an nb-bit field (nb = 23 or 16):
//     n0 = s rho cos(phi),  n1 = s rho sin(phi),   rho = sqrt(-2 ln u1),  phi = 2 pi u2,
// with the output scale s folded in: |s| goes under the square root, the sign of s becomes a half
// turn of the angle.  The field k sits in the mantissa of 1.0f, so t = 1 + k 2^-23 costs no
// conversion instruction, and u1 = t + (2^-(nb+1) - 1) is exact in fp32.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float lg2_approx(float x) {
  float r;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float sqrt_approx(float x) {
  float r;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float sin_approx(float x) {
  float r;
  asm("sin.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ float cos_approx(float x) {
  float r;
  asm("cos.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x));
  return r;
}

// sin and cos of (pi/2) y for y in [0, 4] (y = 4 u2, exact in fp32).  y = q + r with q the nearest integer and
// r in [-1/2, 1/2]; sin((pi/2) r) and cos((pi/2) r) come from odd / even polynomials in r fitted on that
// interval (least squares reweighted towards the minimax solution; maximum absolute error 8.6e-8 and 5.8e-8
// in fp32 arithmetic, about one fp32 ulp of the result), the quadrant q swaps and negates them.  The argument
// range is known, so none of the range checks of a general-purpose routine are needed.
__device__ __forceinline__ void sincos_quarter_turns(float y, float& sn, float& cs) {
  const float biased = __fadd_rn(y, 12582912.0f);          // 1.5 * 2^23: the sum's low mantissa bits hold rint(y)
  const int q = __float_as_int(biased);
  const float r = y - __fsub_rn(biased, 12582912.0f);      // exact
  const float u = r * r;
  float S = fmaf(u, -0.004602177068591118f, 0.07968022674322128f);
  S = fmaf(S, u, -0.6459634900093079f);
  S = fmaf(S, u, 1.5707963705062866f);
  S *= r;
  float C = fmaf(u, 0.0009036316769197583f, -0.02086007222533226f);
  C = fmaf(C, u, 0.25366920232772827f);
  C = fmaf(C, u, -1.2337005138397217f);
  C = fmaf(C, u, 1.0f);
  const bool swap = (q & 1) != 0;
  const float s0 = swap ? C : S, c0 = swap ? S : C;
  sn = __int_as_float(__float_as_int(s0) ^ ((q & 2) << 30));
  cs = __int_as_float(__float_as_int(c0) ^ (((q + 1) & 2) << 30));
}

// -2 ln(u1) for the accurate transform, written for the argument that occurs here: u1 is a multiple of
// 2^-(nb+1) in (0, 1), so v = 1 - u1 is exact in fp32.
//   v <= 1/16:  -2 ln(1 - v) = 2 v (1 + v/2 + v^2/3 + ... + v^6/7), truncation below 3e-11, a few fp32 ulp in all.
//               This is the range where the hardware log2 fails the tolerance: its absolute error of 2^-22 is
//               a relative error of 1/|log2 u1| 2^-22, unbounded as u1 -> 1, and the square root passes half of it on.
//   otherwise:  -2 ln 2 * lg2.approx(u1): relative error at most 2.6e-6 (at u1 = 15/16), 2^-22 below 1/2,
//               i.e. at most 5e-7 absolute on the radius.
// Both are computed and one is selected (no divergence).  The square root that follows is the hardware one
// (relative error 2^-23).  Replaces logf and sqrtf, which cost about three times as many instructions.
__device__ __forceinline__ float neg2_log(float u1) {
  const float v = 1.0f - u1;                                   // exact
  float q = fmaf(v, 0.2857142857f, 0.3333333333f);             // 2/7, 2/6
  q = fmaf(q, v, 0.4f);                                        // 2/5
  q = fmaf(q, v, 0.5f);                                        // 2/4
  q = fmaf(q, v, 0.6666666667f);                               // 2/3
  q = fmaf(q, v, 1.0f);                                        // 2/2
  q = fmaf(q, v, 2.0f);                                        // 2/1
  const float near_one = q * v;
  const float general = -1.3862943611f * lg2_approx(u1);       // -2 ln 2
  return v <= 0.0625f ? near_one : general;
}

// m1, m2: the two uniform fields in mantissa position (bits 0..22) under the exponent of 1.0f (field23 / field16a / field16b).
//
// PRECISE = false (16-bit weights): hardware log2 / sqrt / sin / cos approximations; absolute error of
// a unit normal about 4e-6, far below one ulp of the storage type times any step coefficient.
// PRECISE = true (fp32 weights, tolerance 1e-6 max|theta|): neg2_log, the hardware square root (2^-23) and
// sincos_quarter_turns on the exactly representable angle 4 u2 (in quarter turns): below 1e-6 absolute on a
// unit normal.
// The fast form cannot serve fp32: besides the sin/cos error, the hardware log2 has an absolute
// error near 2^-22 for u1 close to 1, which the square root amplifies for the smallest radii.
template <bool PRECISE>
__device__ __forceinline__ void box_muller(uint32_t m1, uint32_t m2, const NormalScale& ns, float& n0, float& n1) {
  const float u1 = __uint_as_float(m1) + ns.u1_off;
  const float t2 = __uint_as_float(m2);
  if (PRECISE) {
    float sn, cs;
    sincos_quarter_turns(fmaf(4.0f, t2, 4.0f * ns.u1_off), sn, cs);   // 4 u2 in (0, 4), exact
    const float rho = ns.s * sqrt_approx(neg2_log(u1));
    n0 = rho * cs;
    n1 = rho * sn;
  } else {
    const float rho = sqrt_approx(fabsf(ns.kr * lg2_approx(u1)));
    const float phi = fmaf(t2, 6.28318530717958647692f, ns.phase);
    n0 = rho * cos_approx(phi);
    n1 = rho * sin_approx(phi);
  }
}

// (x & mask) | bits as ONE logic instruction.  Written with two constants in C++ it becomes two instructions
// (the three-input logic instruction takes a single immediate); with both constants as register operands it
// is one, which saves 8 of the ~106 instructions that eight normals cost (measured: 3 % of a sweep).
__device__ __forceinline__ uint32_t and_or(uint32_t x, uint32_t mask, uint32_t bits) {
  uint32_t r;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(r) : "r"(x), "r"(mask), "r"(bits));
  return r;
}

// Uniform fields of a generator word, in mantissa position and already carrying the exponent of 1.0f
// (see box_muller): one logic operation each, plus the rotation for the second 16-bit field.
//   32-bit mode: the low 23 bits of the word.
//   16-bit mode: bits 7..22 of the word (radius) and bits 7..22 of the word rotated by 16 (angle).
__device__ __forceinline__ uint32_t field23(uint32_t x) { return and_or(x, 0x7FFFFFu, 0x3F800000u); }
__device__ __forceinline__ uint32_t field16a(uint32_t x) { return and_or(x, 0x7FFF80u, 0x3F800000u); }
__device__ __forceinline__ uint32_t field16b(uint32_t x) { return and_or(__funnelshift_l(x, x, 16), 0x7FFF80u, 0x3F800000u); }

// Eight consecutive normals of stream (tensor, tag) starting at element e (a multiple of 8), each
// already multiplied by the scale folded into `ns`.
//   BITS == 32: blocks e/4 and e/4+1; words (x0,x1) -> normals 0,1 and (x2,x3) -> normals 2,3.
//   BITS == 16: block e/8; word w -> normals 2w, 2w+1.
template <int BITS, bool PRECISE>
__device__ __forceinline__ void normals8(const PhiloxKeys& keys, uint32_t tensor, uint32_t tag, uint64_t e, const NormalScale& ns,
                                         float (&z)[8]) {
  uint32_t x[4];
  if (BITS == 32) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      philox_block((e >> 2) + h, tensor, tag, keys, x);
      box_muller<PRECISE>(field23(x[0]), field23(x[1]), ns, z[4 * h + 0], z[4 * h + 1]);
      box_muller<PRECISE>(field23(x[2]), field23(x[3]), ns, z[4 * h + 2], z[4 * h + 3]);
    }
  } else {
    philox_block(e >> 3, tensor, tag, keys, x);
#pragma unroll
    for (int w = 0; w < 4; ++w) box_muller<PRECISE>(field16a(x[w]), field16b(x[w]), ns, z[2 * w], z[2 * w + 1]);
  }
}

// Fast transform fused with its consumer: acc0 += s rho cos(phi), acc1 += s rho sin(phi).
__device__ __forceinline__ void box_muller_acc(uint32_t m1, uint32_t m2, const NormalScale& ns, float& acc0, float& acc1) {
  const float u1 = __uint_as_float(m1) + ns.u1_off;
  const float t2 = __uint_as_float(m2);
  const float rho = sqrt_approx(fabsf(ns.kr * lg2_approx(u1)));
  const float phi = fmaf(t2, 6.28318530717958647692f, ns.phase);
  acc0 = fmaf(rho, cos_approx(phi), acc0);
  acc1 = fmaf(rho, sin_approx(phi), acc1);
}

// The same, also adding the squared radius of the pair to rsum: (s rho cos)^2 + (s rho sin)^2 = s^2 rho^2 is the
// argument of the square root, so the energy of the two normals costs one addition.
__device__ __forceinline__ void box_muller_acc_rsum(uint32_t m1, uint32_t m2, const NormalScale& ns, float& acc0, float& acc1, float& rsum) {
  const float u1 = __uint_as_float(m1) + ns.u1_off;
  const float t2 = __uint_as_float(m2);
  const float x = fabsf(ns.kr * lg2_approx(u1));
  rsum += x;
  const float rho = sqrt_approx(x);
  const float phi = fmaf(t2, 6.28318530717958647692f, ns.phase);
  acc0 = fmaf(rho, cos_approx(phi), acc0);
  acc1 = fmaf(rho, sin_approx(phi), acc1);
}

// acc[0..7] += the eight scaled normals of octet number `oct` (= element index / 8, as two 32-bit
// halves) of stream (tensor, tag 0).  Hardware-approximation transform only.
template <int BITS>
__device__ __forceinline__ void normals8_acc(const PhiloxKeys& keys, uint32_t tensor, uint32_t oct_lo, uint32_t oct_hi, const NormalScale& ns,
                                             float (&acc)[8]) {
  uint32_t x[4];
  if (BITS == 32) {
    const uint32_t b_lo = oct_lo << 1, b_hi = (oct_hi << 1) | (oct_lo >> 31);   // block 2*oct; 2*oct + 1 cannot carry
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      philox4x32_10(b_lo + h, b_hi, tensor, 0u, keys, x);
      box_muller_acc(field23(x[0]), field23(x[1]), ns, acc[4 * h + 0], acc[4 * h + 1]);
      box_muller_acc(field23(x[2]), field23(x[3]), ns, acc[4 * h + 2], acc[4 * h + 3]);
    }
  } else {
    philox4x32_10(oct_lo, oct_hi, tensor, 0u, keys, x);
#pragma unroll
    for (int w = 0; w < 4; ++w) box_muller_acc(field16a(x[w]), field16b(x[w]), ns, acc[2 * w], acc[2 * w + 1]);
  }
}

// normals8_acc that also returns the energy of its eight normals (sum of their squares) in rsum.
template <int BITS>
__device__ __forceinline__ void normals8_acc_rsum(const PhiloxKeys& keys, uint32_t tensor, uint32_t oct_lo, uint32_t oct_hi, const NormalScale& ns,
                                                  float (&acc)[8], float& rsum) {
  uint32_t x[4];
  if (BITS == 32) {
    const uint32_t b_lo = oct_lo << 1, b_hi = (oct_hi << 1) | (oct_lo >> 31);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      philox4x32_10(b_lo + h, b_hi, tensor, 0u, keys, x);
      box_muller_acc_rsum(field23(x[0]), field23(x[1]), ns, acc[4 * h + 0], acc[4 * h + 1], rsum);
      box_muller_acc_rsum(field23(x[2]), field23(x[3]), ns, acc[4 * h + 2], acc[4 * h + 3], rsum);
    }
  } else {
    philox4x32_10(oct_lo, oct_hi, tensor, 0u, keys, x);
#pragma unroll
    for (int w = 0; w < 4; ++w) box_muller_acc_rsum(field16a(x[w]), field16b(x[w]), ns, acc[2 * w], acc[2 * w + 1], rsum);
  }
}

// Partial sums of the norm bookkeeping of one warp for one work item: reduce over the lanes in a fixed order and
// store them in the item's slot.  Every slot that the finishing kernel reads is written by each launch first.
__device__ __forceinline__ void store_item_stats(const SweepParams& p, int item, int slot, double s0, double s1, double s2) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    s0 += __shfl_xor_sync(0xFFFFFFFFu, s0, off);
    s1 += __shfl_xor_sync(0xFFFFFFFFu, s1, off);
    s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, off);
  }
  if ((threadIdx.x & 31) == 0) {
    double* dst = p.item_stats + (static_cast<int64_t>(p.item_base + item) * kStatSlots + slot) * 3;
    dst[0] = s0; dst[1] = s1; dst[2] = s2;
  }
}

// One normal at an arbitrary element index (ragged tails and the unaligned fallback kernels).
template <int BITS, bool PRECISE>
__device__ __forceinline__ float normal1(const PhiloxKeys& keys, uint32_t tensor, uint32_t tag, uint64_t e, const NormalScale& ns) {
  uint32_t x[4];
  float n0, n1;
  if (BITS == 32) {
    philox_block(e >> 2, tensor, tag, keys, x);
    const int pair = static_cast<int>(e & 3) >> 1;
    box_muller<PRECISE>(field23(pair ? x[2] : x[0]), field23(pair ? x[3] : x[1]), ns, n0, n1);
  } else {
    philox_block(e >> 3, tensor, tag, keys, x);
    const int w = static_cast<int>(e & 7) >> 1;
    const uint32_t word = w == 0 ? x[0] : (w == 1 ? x[1] : (w == 2 ? x[2] : x[3]));
    box_muller<PRECISE>(field16a(word), field16b(word), ns, n0, n1);
  }
  return (e & 1) ? n1 : n0;
}

// ---------------------------------------------------------------------------------------------
// Storage access: eight contiguous elements as fp32, 128-bit transactions, streaming cache hints
// (every weight is touched exactly once per sweep).  Stores round to nearest even.
// ---------------------------------------------------------------------------------------------
template <typename T>
struct Storage;

template <>
struct Storage<float> {
  static __device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
    const float4 b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
  static __device__ __forceinline__ void store8(float* p, const float (&v)[8]) {
    __stcs(reinterpret_cast<float4*>(p), make_float4(v[0], v[1], v[2], v[3]));
    __stcs(reinterpret_cast<float4*>(p) + 1, make_float4(v[4], v[5], v[6], v[7]));
  }
  static __device__ __forceinline__ float load1(const float* p) { return *p; }
  static __device__ __forceinline__ void store1(float* p, float v) { *p = v; }
};

template <>
struct Storage<__half> {
  static __device__ __forceinline__ void load8(const __half* p, float (&v)[8]) {
    const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
      v[2 * i] = f.x;
      v[2 * i + 1] = f.y;
    }
  }
  static __device__ __forceinline__ void store8(__half* p, const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __half2 h = __floats2half2_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
  }
  static __device__ __forceinline__ float load1(const __half* p) { return __half2float(*p); }
  static __device__ __forceinline__ void store1(__half* p, float v) { *p = __float2half_rn(v); }
};

template <>
struct Storage<__nv_bfloat16> {
  static __device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  static __device__ __forceinline__ void store8(__nv_bfloat16* p, const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    __stcs(reinterpret_cast<uint4*>(p), make_uint4(w[0], w[1], w[2], w[3]));
  }
  static __device__ __forceinline__ float load1(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  static __device__ __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// ---------------------------------------------------------------------------------------------
// Guided coefficients G_l[k][c .. c+7], multiplied by `cb`  (Algorithm 1 "Sample z_g"; Sec. 3.4 for
// the compressed form  x = lambda (x_quant - delta)).
// ---------------------------------------------------------------------------------------------
template <int BITS, bool PRECISE>
__device__ __forceinline__ void coeffs8(const TensorDesc& td, const PhiloxKeys& keys, const NormalScale& unit, float cb, int k,
                                        int64_t c, float (&g)[8]) {
  if (td.q != nullptr && k < td.qrows) {
    const float lambda = td.qscale[k] * cb;
    const float delta = td.qzero ? td.qzero[k] : 0.0f;
    if (td.qbits == 4) {
      // two unsigned 4-bit codes per byte, even column in the low nibble (c is a multiple of 8)
      const uint8_t* src = reinterpret_cast<const uint8_t*>(td.q) + static_cast<int64_t>(k) * ((td.cols + 1) >> 1) + (c >> 1);
      uint32_t word;
      if ((reinterpret_cast<uintptr_t>(src) & 3) == 0) {
        word = __ldg(reinterpret_cast<const uint32_t*>(src));          // eight 4-bit codes in one load
      } else {
        word = static_cast<uint32_t>(src[0]) | (static_cast<uint32_t>(src[1]) << 8) | (static_cast<uint32_t>(src[2]) << 16) |
               (static_cast<uint32_t>(src[3]) << 24);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) g[i] = lambda * (static_cast<float>((word >> (4 * i)) & 15u) - delta);
    } else {
      const int8_t* src = td.q + static_cast<int64_t>(k) * td.cols + c;
      if (ZGR_DTC_VECTOR && (reinterpret_cast<uintptr_t>(src) & 7) == 0) {
        // eight signed codes in one 64-bit load (the strips are rebuilt once per work item and wait for these
        // loads with nothing else to do: eight single-byte loads made that 5 % of a rank-64 sweep)
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(src));
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          g[i] = lambda * (static_cast<float>(static_cast<int>(static_cast<int8_t>(raw.x >> (8 * i)))) - delta);
          g[4 + i] = lambda * (static_cast<float>(static_cast<int>(static_cast<int8_t>(raw.y >> (8 * i)))) - delta);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) g[i] = lambda * (static_cast<float>(src[i]) - delta);
      }
    }
  } else {
    normals8<BITS, PRECISE>(keys, static_cast<uint32_t>(td.id), 1u, static_cast<uint64_t>(k) * static_cast<uint64_t>(td.cols) + static_cast<uint64_t>(c),
                            unit, g);
#pragma unroll
    for (int i = 0; i < 8; ++i) g[i] *= cb;
  }
}

template <int BITS, bool PRECISE>
__device__ __forceinline__ float coeff1(const TensorDesc& td, const PhiloxKeys& keys, const NormalScale& unit, float cb, int k, int64_t c) {
  if (td.q != nullptr && k < td.qrows) {
    const float delta = td.qzero ? td.qzero[k] : 0.0f;
    float code;
    if (td.qbits == 4) {
      const uint32_t byte = reinterpret_cast<const uint8_t*>(td.q)[static_cast<int64_t>(k) * ((td.cols + 1) >> 1) + (c >> 1)];
      code = static_cast<float>((c & 1) ? (byte >> 4) : (byte & 15u));
    } else {
      code = static_cast<float>(td.q[static_cast<int64_t>(k) * td.cols + c]);
    }
    return td.qscale[k] * cb * (code - delta);
  }
  return cb * normal1<BITS, PRECISE>(keys, static_cast<uint32_t>(td.id), 1u,
                                     static_cast<uint64_t>(k) * static_cast<uint64_t>(td.cols) + static_cast<uint64_t>(c), unit);
}

// ---------------------------------------------------------------------------------------------
// The terms of a sweep.  A sweep applies  sum_q c_q z(seed_q)  with  z = a Z + b U G  (Algorithm 1:
// one term for a perturbation or a single restore+update; several when the projected gradients of
// several seeds are applied together, the sum over t in "Recover gradient" / "Update").  MULTI = false
// reads term[0] with constant addressing, which is the single-seed hot path unchanged.
// ---------------------------------------------------------------------------------------------
// sum_q c_q a Z_q  for eight consecutive elements starting at e (a multiple of 8)
template <int BITS, bool PRECISE, bool MULTI>
__device__ __forceinline__ void iso8(const SweepParams& p, uint32_t tensor, uint64_t e, float (&z)[8]) {
  normals8<BITS, PRECISE>(p.term[0].keys, tensor, 0u, e, p.term[0].iso, z);
  if (MULTI) {
#pragma unroll 1
    for (int q = 1; q < p.n_terms; ++q) {
      float y[8];
      normals8<BITS, PRECISE>(p.term[q].keys, tensor, 0u, e, p.term[q].iso, y);
#pragma unroll
      for (int i = 0; i < 8; ++i) z[i] += y[i];
    }
  }
}

template <int BITS, bool PRECISE, bool MULTI>
__device__ __forceinline__ float iso1(const SweepParams& p, uint32_t tensor, uint64_t e) {
  float z = normal1<BITS, PRECISE>(p.term[0].keys, tensor, 0u, e, p.term[0].iso);
  if (MULTI) {
#pragma unroll 1
    for (int q = 1; q < p.n_terms; ++q) z += normal1<BITS, PRECISE>(p.term[q].keys, tensor, 0u, e, p.term[q].iso);
  }
  return z;
}

// sum_q c_q b G_q[k][c .. c+7].  Compressed coefficients (rows below td.qrows) do not depend on the seed: they
// are scaled by the sum of the terms' factors.
template <int BITS, bool PRECISE, bool MULTI>
__device__ __forceinline__ void guided8(const TensorDesc& td, const SweepParams& p, int k, int64_t c, float (&g)[8]) {
  if (!MULTI) {
    coeffs8<BITS, PRECISE>(td, p.term[0].keys, p.unit, p.term[0].cb, k, c, g);
  } else if (td.q != nullptr && k < td.qrows) {
    float cb = 0.0f;
    for (int q = 0; q < p.n_terms; ++q) cb += p.term[q].cb;
    coeffs8<BITS, PRECISE>(td, p.term[0].keys, p.unit, cb, k, c, g);
  } else {
    coeffs8<BITS, PRECISE>(td, p.term[0].keys, p.unit, p.term[0].cb, k, c, g);
#pragma unroll 1
    for (int q = 1; q < p.n_terms; ++q) {
      float y[8];
      coeffs8<BITS, PRECISE>(td, p.term[q].keys, p.unit, p.term[q].cb, k, c, y);
#pragma unroll
      for (int i = 0; i < 8; ++i) g[i] += y[i];
    }
  }
}

template <int BITS, bool PRECISE, bool MULTI>
__device__ __forceinline__ float guided1(const TensorDesc& td, const SweepParams& p, int k, int64_t c) {
  if (!MULTI) return coeff1<BITS, PRECISE>(td, p.term[0].keys, p.unit, p.term[0].cb, k, c);
  if (td.q != nullptr && k < td.qrows) {
    float cb = 0.0f;
    for (int q = 0; q < p.n_terms; ++q) cb += p.term[q].cb;
    return coeff1<BITS, PRECISE>(td, p.term[0].keys, p.unit, cb, k, c);
  }
  float g = 0.0f;
#pragma unroll 1
  for (int q = 0; q < p.n_terms; ++q) g += coeff1<BITS, PRECISE>(td, p.term[q].keys, p.unit, p.term[q].cb, k, c);
  return g;
}

}  // namespace zgr
#endif  // ZGR_DEVICE_CUH_
