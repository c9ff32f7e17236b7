// Blackwell-native sweep for 16-bit weights with a rank > 8 subspace:
//     theta <- rnd(theta + c (a Z + b U G))            (Eq. (perturbation) applied as in Algorithm 1)
//
// The generator and the Gaussian transform alone fill about 80 % of an SM's issue slots at the rate
// HBM can feed the weights, so everything else is taken out of the SM's instruction stream:
//
//   * TMA brings a 128-row x NS-column tile of theta (and the matching 128 x KP tiles of U, pre-split
//     into fp16 hi/lo) into shared memory, and writes the finished tile back; no thread issues a
//     global load or store for the weights.
//   * tcgen05.mma builds   D = theta + c b U G   in tensor memory (fp32):
//       - "theta" enters through identity products  D[:, 16j:16j+16] = theta[:, 16j:16j+16] * I16
//         with theta's own 16-bit tile as the A operand, which unpacks it to fp32 exactly, for free;
//       - U G is formed first, as  Ulo Ghi + Uhi Glo + Uhi Ghi  with fp16 split operands (hi + lo carries 22
//         significant bits, against 16 for a bf16 split, whose representation error of 4.5e-6 relative was the
//         whole error of z on this path).  fp16 has a narrow exponent range, so both operands are kept near 1
//         by powers of two: the library's copy of U holds U 2^j (j from the tensor's row count), the strips hold
//         c b G 2^(s-j), and the accumulator therefore holds 2^s c b U G.  The identity products that bring
//         theta in come last and use the instruction's accumulator scaling,  D <- theta I + 2^-s D
//         (s <= 15 is an immediate of the instruction), which removes the factor exactly and for free.
//         The strips of c b G live in shared memory as the K-major B operand for all row tiles of a work item.
//   * The epilogue warps, in two groups that take alternate tiles (32 rows x 64 columns per warp, 32 columns
//     at a time), read D with tcgen05.ld (one row per thread), add the isotropic
//     normals (Philox4x32-10 + Box-Muller in registers), round to the storage type and write the
//     tile into the shared-memory buffer the TMA store reads.
//
// Warp roles: warp 0 = TMA producer (loads and stores), warp 1 = MMA issuer and owner of the tensor
// memory allocation, warps 2.. = epilogue.  The two single-thread roles run in the lane picked by
// elect.sync, which lets their loop state and descriptors live in uniform registers.  One CTA per SM
// (the shared-memory footprint enforces it), persistent over a static round-robin list of work items.
//
// Every wait on an mbarrier is bounded: when a wait gives up it records where in *p.error, raises a
// CTA-wide abort flag, and all roles fall through to the common exit, where the producer drains its
// outstanding copies and warp 1 returns the tensor memory.
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include "zgr_device.cuh"
#include "zgr_kernels.h"

namespace zgr {
namespace {

constexpr unsigned kStaggerNs = 800;
// Sleep between two polls of a barrier: the single-thread roles (which run ahead of the epilogue and share
// their schedulers with epilogue warps) and the epilogue warps themselves.
#ifndef ZGR_ROLE_SLEEP_NS
#define ZGR_ROLE_SLEEP_NS 64
#endif
#ifndef ZGR_EPI_SLEEP_NS
#define ZGR_EPI_SLEEP_NS 0
#endif
constexpr unsigned long long kWaitLimitCycles = 4000000000ull;  // ~2 s at 2 GHz

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(2000u) /* suspend-time hint in ns: waiting warps sleep instead of spinning */
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if it gave up or the CTA is already aborting.  The abort flag and
// the clock are looked at only every 256 polls, so a waiting warp costs few issue slots;
// BACKOFF adds a short sleep between polls for the two single-thread roles, which run ahead of the
// epilogue and must not steal issue slots from the warps that share their scheduler.
template <bool BACKOFF>
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* error, int where) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = clock64();
  uint32_t polls = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if (BACKOFF) __nanosleep(ZGR_ROLE_SLEEP_NS);
    else if (ZGR_EPI_SLEEP_NS > 0) __nanosleep(ZGR_EPI_SLEEP_NS);
    if ((++polls & 255u) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > kWaitLimitCycles) {
        *abort_flag = 1;
        atomicCAS(error, 0, where);
        return false;
      }
    }
  }
}

// True in exactly one lane of a converged warp.  Unlike a test of the lane index, this tells the
// compiler that the guarded region runs in a single thread, so loop counters, addresses and
// descriptors in it can live in uniform registers, which is where TMA and tcgen05.mma take them from.
__device__ __forceinline__ bool elect_one() {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "elect.sync _|p, 0xFFFFFFFF;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok));
  return ok != 0;
}

__device__ __forceinline__ void sts128(uint32_t saddr, const uint4& v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(saddr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void sts32(uint32_t saddr, uint32_t v) { asm volatile("st.shared.b32 [%0], %1;" ::"r"(saddr), "r"(v) : "memory"); }

__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const void* tmap, int x, int y, uint32_t bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(dst),
               "l"(tmap), "r"(bar), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_store_2d(const void* tmap, int x, int y, uint32_t src) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tmap), "r"(src), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void tma_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tma_wait_all0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() { asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D <- A B + 2^-SC D  (the accumulator-scaling form of the instruction; SC in [0, 15] is an immediate)
template <int SC>
__device__ __forceinline__ void umma_scaled_d(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, 1, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p, %4;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "n"(SC)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]),
                 "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
               : "r"(taddr)
               : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand whose rows are `row_bytes` (32, 64 or 128)
// long and swizzled with the matching mode: eight rows form one swizzle atom, atoms follow each
// other every 8*row_bytes (the stride byte offset); the leading byte offset is not used by
// swizzled K-major layouts and is set to 1 (16 bytes).  Bits 46-47 = 1: Blackwell descriptor.
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, int row_bytes) {
  const uint64_t layout = row_bytes == 128 ? 2ull : (row_bytes == 64 ? 4ull : 6ull);
  uint64_t d = 0;
  d |= static_cast<uint64_t>((saddr >> 4) & 0x3FFF);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(((8 * row_bytes) >> 4) & 0x3FFF) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= layout << 61;
  return d;
}
// Instruction descriptor, kind::f16: fp32 accumulate, A and B both `fmt` (0 = f16, 1 = bf16), both
// K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t make_idesc(int fmt, int n) {
  return (1u << 4) | (static_cast<uint32_t>(fmt) << 7) | (static_cast<uint32_t>(fmt) << 10) | (static_cast<uint32_t>(n >> 3) << 17) |
         (static_cast<uint32_t>(128 >> 4) << 24);
}
// XOR swizzle of a byte offset inside a buffer aligned to 1024 bytes (rows of row_bytes bytes).
__device__ __forceinline__ uint32_t swizzle(uint32_t off, int row_bytes) {
  const uint32_t mask = row_bytes == 128 ? 7u : (row_bytes == 64 ? 3u : 1u);
  return off ^ (((off >> 7) & mask) << 4);
}

template <typename T>
struct Pack16;
template <>
struct Pack16<__nv_bfloat16> {
  static constexpr int kFmt = 1;
  static constexpr uint16_t kOne = 0x3F80;
  static __device__ __forceinline__ uint32_t pack(float a, float b) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
  }
};
template <>
struct Pack16<__half> {
  static constexpr int kFmt = 0;
  static constexpr uint16_t kOne = 0x3C00;
  static __device__ __forceinline__ uint32_t pack(float a, float b) {
    const __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<const uint32_t*>(&h);
  }
};

// the eight 16-bit values of a 16-byte chunk as floats
template <typename T>
__device__ __forceinline__ void unpack8(const uint4& raw, float (&v)[8]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if constexpr (sizeof(T) == 2 && Pack16<T>::kFmt == 1) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    } else {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[i]));
      v[2 * i] = f.x;
      v[2 * i + 1] = f.y;
    }
  }
}
__device__ __forceinline__ uint4 lds128(uint32_t saddr) {
  uint4 v;
  asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(saddr) : "memory");
  return v;
}

// fp16 hi/lo split of a pair of floats, packed as f16x2 (first value in the low half)
__device__ __forceinline__ void split_f16(float x0, float x1, uint32_t& hi, uint32_t& lo) {
  const __half2 h = __floats2half2_rn(x0, x1);
  hi = *reinterpret_cast<const uint32_t*>(&h);
  const float2 hf = __half22float2(h);
  const __half2 l = __floats2half2_rn(x0 - hf.x, x1 - hf.y);
  lo = *reinterpret_cast<const uint32_t*>(&l);
}

// Accumulator scale of a tensor in this call: s = clamp(ushift + kshift, 0, 15) (see the operand precision note above)
__device__ __forceinline__ int acc_shift(const TensorDesc& td, const SweepParams& p) { return min(max(td.ushift + p.kshift, 0), 15); }

// Tile configuration per contraction width: compile-time parameters (-D...) whose defaults are the measured
// optimum on B200.  TILE_N = 192 runs 24 epilogue warps on 128 x 192 tiles (three 64-column boxes);
// TILE_N = 128 runs 16 on 128 x 128 tiles.  S = theta stages, N = adjacent tiles per strip.
#ifndef ZGR_TILE_N16
#define ZGR_TILE_N16 128
#endif
#ifndef ZGR_TILE_N32
#define ZGR_TILE_N32 128
#endif
#ifndef ZGR_S16
#define ZGR_S16 6
#endif
#ifndef ZGR_S32
#define ZGR_S32 5
#endif
#ifndef ZGR_S64
#define ZGR_S64 4
#endif
#ifndef ZGR_N16
#define ZGR_N16 2
#endif
#ifndef ZGR_N32
#define ZGR_N32 2
#endif
#ifndef ZGR_N64
#define ZGR_N64 1
#endif
// Epilogue groups: 1 = every epilogue warp works on every tile (32 rows x 32 columns each); 2 (4) = two (four)
// groups of warps take tiles in turn (32 rows x 64 (128) columns each, in two (four) passes), so that one group's
// per-tile waits fall under the other groups' arithmetic.
#ifndef ZGR_GROUPS
#define ZGR_GROUPS 2
#endif
template <int KP>
struct UmmaCfg {
  static constexpr int NS = KP == 64 ? 128 : (KP == 32 ? ZGR_TILE_N32 : ZGR_TILE_N16);   // columns per tile / per accumulator buffer
  static constexpr bool WIDE = NS > 128;
  static constexpr int EPI_WARPS = NS / 8;                 // one epilogue warp per 32 rows x 32 columns of a tile
  static constexpr int THREADS = 32 * (2 + EPI_WARPS);
  static constexpr int GROUPS = NS == 128 ? ZGR_GROUPS : 1;   // epilogue groups on alternate tiles (1, 2 or 4; see ZGR_GROUPS)
  static constexpr int NSUB = KP == 64 ? ZGR_N64 : (KP == 32 ? ZGR_N32 : ZGR_N16);   // adjacent tiles per row block that share one U tile
  static constexpr int STAGES = KP == 64 ? ZGR_S64 : (KP == 32 ? ZGR_S32 : ZGR_S16);  // theta tiles in flight (loaded, transformed in place, stored)
  static constexpr int USTAGES = 2;                        // U tiles in flight
  static constexpr int NACC = WIDE ? 2 : 4;                // accumulator buffers in tensor memory
  static constexpr int ROWB = KP * 2;                      // bytes per row of the U and G operands
  static constexpr int THETA_BYTES = 128 * NS * 2;         // NS/64 boxes of 128 rows x 128 B
  static constexpr int U_BYTES = 128 * ROWB;               // one of hi / lo
  static constexpr int G_BYTES = NS * ROWB;                // one of hi / lo, one tile's strip
  static constexpr int ID_BYTES = 1024;                    // 16 x 16 identity (512 B), padded to the swizzle alignment
  static constexpr int BAR_BYTES = 1024;
  static constexpr int SMEM_BYTES =
      STAGES * THETA_BYTES + USTAGES * 2 * U_BYTES + NSUB * 2 * G_BYTES + ID_BYTES + BAR_BYTES + 1024 /* alignment slack */;
  static constexpr int TMEM_COLS = NACC * NS <= 256 ? 256 : 512;   // allocations are powers of two
  static_assert(SMEM_BYTES <= 232448, "shared-memory budget of one CTA");
};

struct TileCoord {
  int32_t tensor;
  int32_t col0;
  int32_t row0;
  int32_t ncols;   // columns of this tile that exist in the tensor (<= 128)
};

}  // namespace

// Work item = NSUB adjacent column tiles (a strip of up to 128*NSUB columns) x a range of rows.
// Tiles are visited row block by row block, the NSUB tiles of a row block one after the other, so
// that a CTA touches up to 256*NSUB contiguous bytes of every row and loads each U tile once.
// STATS = true turns the same pipeline into the norm bookkeeping: no weights are loaded or stored,
// D = b U G only, and the epilogue accumulates sum (a Z)^2, sum (b U G)^2 and sum z^2 per tensor
// (term[0].iso carries the scale a, term[0].cb = b; the sums go to the work item's bookkeeping slots).
// MULTI = true applies several (seed, coefficient) terms in the one pass: the coefficient strips of
// the terms are summed before the split (U (sum_q c_q b G_q) is one product), the isotropic normals
// are added term by term in the epilogue.
// ZOUT = true is the test hook of this kernel: the same loads, products and epilogue arithmetic, but the fp32
// result of every element (accumulator plus normals, before the rounding to the storage type) goes to
// p.zout[row * cols + col] by plain stores and nothing is written back to the weights.  On a zeroed
// weight image with coefficient 1 that is z itself as this kernel computes it.
// SSTATS = true (single-term sweeps) is the sweep itself with the norm bookkeeping folded in: before a thread
// overwrites its 16 bytes of the staged tile it reads theta back from them, so that the guided part (accumulator
// minus theta) and the whole step (result minus theta) can be squared and summed; the isotropic part costs one
// addition per pair of normals (the squared radius is the argument of the square root).  The sums are of
// (c a Z)^2, (c b U G)^2 and (c z)^2; the host divides by c^2.
template <typename T, int BITS, int KP, bool STATS = false, bool MULTI = false, bool ZOUT = false, bool SSTATS = false>
__global__ void __launch_bounds__(UmmaCfg<KP>::THREADS, 1) sweep_umma_kernel(const __grid_constant__ SweepParams p, const CUtensorMap* __restrict__ tmaps,
                                                                     int* __restrict__ error) {
  using Cfg = UmmaCfg<KP>;
  constexpr int NS = Cfg::NS, S = Cfg::STAGES, US = Cfg::USTAGES, ROWB = Cfg::ROWB, NACC = Cfg::NACC, NSUB = Cfg::NSUB;
  constexpr int kEpiWarps = Cfg::EPI_WARPS, kUmmaThreads = Cfg::THREADS;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
  uint8_t* theta_base = smem;                                           // S tiles
  uint8_t* u_base = theta_base + S * Cfg::THETA_BYTES;                  // US x (hi, lo)
  uint8_t* g_base = u_base + US * 2 * Cfg::U_BYTES;                     // NSUB x (hi, lo)
  uint8_t* ident = g_base + NSUB * 2 * Cfg::G_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(ident + Cfg::ID_BYTES);
  const uint32_t bar0 = smem_u32(bars);
  auto BAR_FULL = [&](int s) { return bar0 + 8u * static_cast<uint32_t>(s); };                          // theta tile landed
  auto BAR_OUT = [&](int s) { return bar0 + 8u * static_cast<uint32_t>(S + s); };                       // result written into the stage
  auto BAR_ACC_FULL = [&](int b) { return bar0 + 8u * static_cast<uint32_t>(2 * S + b); };              // accumulator complete
  auto BAR_ACC_EMPTY = [&](int b) { return bar0 + 8u * static_cast<uint32_t>(2 * S + NACC + b); };      // accumulator read out
  auto BAR_U_FULL = [&](int u) { return bar0 + 8u * static_cast<uint32_t>(2 * S + 2 * NACC + u); };     // U tile landed
  auto BAR_U_FREE = [&](int u) { return bar0 + 8u * static_cast<uint32_t>(2 * S + 2 * NACC + US + u); };  // U tile consumed
  const uint32_t BAR_G = bar0 + 8u * static_cast<uint32_t>(2 * S + 2 * NACC + 2 * US);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * S + 2 * NACC + 2 * US + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    constexpr int kWarpsPerTile = kEpiWarps / Cfg::GROUPS;   // epilogue warps that work on one tile
    for (int s = 0; s < S; ++s) {
      mbar_init(BAR_FULL(s), 1);
      mbar_init(BAR_OUT(s), kWarpsPerTile);
    }
    for (int b = 0; b < NACC; ++b) {
      mbar_init(BAR_ACC_FULL(b), 1);
      mbar_init(BAR_ACC_EMPTY(b), kWarpsPerTile);
    }
    for (int u = 0; u < US; ++u) {
      mbar_init(BAR_U_FULL(u), 1);
      mbar_init(BAR_U_FREE(u), 1);
    }
    mbar_init(BAR_G, kEpiWarps);
    *abort_flag = 0;
    fence_mbar_init();
  }
  // 16 x 16 identity in the storage type, K-major rows of 32 bytes, 32-byte swizzle
  for (int i = threadIdx.x; i < 256; i += kUmmaThreads) {
    const int n = i >> 4, k = i & 15;
    *reinterpret_cast<uint16_t*>(ident + swizzle(static_cast<uint32_t>(n * 32 + k * 2), 32)) = (n == k) ? Pack16<T>::kOne : uint16_t(0);
  }
  fence_proxy_async();
  __syncthreads();
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), Cfg::TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // The three roles walk the same sequence of (item, row block, tile) triples; t counts tiles and
  // rb counts row blocks over the whole life of the CTA, which fixes every ring slot and phase.
  if (warp == 0) {
    // ===================================== TMA producer =====================================
    if (elect_one()) {
      TileCoord ring[S];
      int t = 0, rb = 0;
      bool ok = true;
      auto store_tile = [&](int s) {
        const TileCoord& o = ring[s];
        const CUtensorMap* tm = tmaps + 3 * o.tensor;
        const uint32_t src = smem_u32(theta_base + s * Cfg::THETA_BYTES);
        for (int c = 0; c * 64 < o.ncols; ++c) tma_store_2d(tm, o.col0 + 64 * c, o.row0, src + c * 16384);
        tma_commit();
      };
      for (int it = blockIdx.x; it < p.n_items && ok; it += gridDim.x) {
        const WorkItem w = p.items[it];
        const CUtensorMap* tm = tmaps + 3 * w.tensor;
        const int row_end = static_cast<int>(w.row0_or_e0 + w.nrows_or_count);
        const int nsub = (w.ncols + NS - 1) / NS;
        for (int row0 = static_cast<int>(w.row0_or_e0); row0 < row_end && ok; row0 += 128, ++rb) {
          const int u = rb % US;
          if (rb >= US && !mbar_wait<true>(BAR_U_FREE(u), ((rb / US) - 1) & 1, abort_flag, error, 8)) { ok = false; break; }
          const uint32_t udst = smem_u32(u_base + u * 2 * Cfg::U_BYTES);
          mbar_arrive_expect_tx(BAR_U_FULL(u), static_cast<uint32_t>(2 * Cfg::U_BYTES));
          tma_load_2d(udst, tm + 1, 0, row0, BAR_U_FULL(u));
          tma_load_2d(udst + Cfg::U_BYTES, tm + 2, 0, row0, BAR_U_FULL(u));
          for (int sub = 0; sub < nsub && !STATS; ++sub, ++t) {
            const int s = t % S;
            if (t >= S) {
              // the epilogue has written tile t-S into this stage: store it, then the stage is free
              if (!mbar_wait<true>(BAR_OUT(s), ((t / S) - 1) & 1, abort_flag, error, 1)) { ok = false; break; }
              if (!ZOUT) {
                store_tile(s);
                tma_wait_read0();
              }
            }
            const int col0 = static_cast<int>(w.col0) + NS * sub;
            const int ncols = min(NS, w.ncols - NS * sub);
            ring[s] = TileCoord{w.tensor, col0, row0, ncols};
            const int nbox = (ncols + 63) / 64;
            const uint32_t dst = smem_u32(theta_base + s * Cfg::THETA_BYTES);
            mbar_arrive_expect_tx(BAR_FULL(s), static_cast<uint32_t>(nbox * 16384));
            for (int c = 0; c < nbox; ++c) tma_load_2d(dst + c * 16384, tm, col0 + 64 * c, row0, BAR_FULL(s));
          }
        }
      }
      // drain: store the last tiles
      const int total = t;
      for (int v = (total > S ? total - S : 0); v < total && ok && !STATS; ++v) {
        if (!mbar_wait<true>(BAR_OUT(v % S), (v / S) & 1, abort_flag, error, 2)) { ok = false; break; }
        if (!ZOUT) store_tile(v % S);
      }
      if (!ok) {
        // aborting: let the loads already issued land before the CTA gives up its shared memory
        for (int v = (total > S ? total - S : 0); v < total; ++v) {
          const unsigned long long t0 = clock64();
          while (!mbar_try_wait(BAR_FULL(v % S), (v / S) & 1) && clock64() - t0 < kWaitLimitCycles) {
          }
        }
        for (int v = (rb > US ? rb - US : 0); v < rb; ++v) {
          const unsigned long long t0 = clock64();
          while (!mbar_try_wait(BAR_U_FULL(v % US), (v / US) & 1) && clock64() - t0 < kWaitLimitCycles) {
          }
        }
      }
      tma_wait_all0();
    }
  } else if (warp == 1) {
    // ===================================== MMA issuer =====================================
    if (elect_one()) {
      const uint32_t idesc_id = make_idesc(Pack16<T>::kFmt, 16);
      const uint32_t idesc_ug = make_idesc(0, NS);          // fp16 operands
      const uint64_t desc_id = make_desc(smem_u32(ident), 32);
      // Descriptors differ only in their start-address field (bits 0-13, address >> 4), so every
      // operand below is one of these bases plus a small constant.
      const uint64_t desc_theta0 = make_desc(smem_u32(theta_base), 128);
      const uint64_t desc_u0 = make_desc(smem_u32(u_base), ROWB);
      const uint64_t desc_g0 = make_desc(smem_u32(g_base), ROWB);
      int t = 0, rb = 0, item_no = 0;
      bool ok = true;
      for (int it = blockIdx.x; it < p.n_items && ok; it += gridDim.x, ++item_no) {
        const WorkItem w = p.items[it];
        const int sh = acc_shift(p.tensors[w.tensor], p);
        if (!mbar_wait<true>(BAR_G, item_no & 1, abort_flag, error, 3)) break;
        tc_fence_after();
        const int row_end = static_cast<int>(w.row0_or_e0 + w.nrows_or_count);
        const int nsub = (w.ncols + NS - 1) / NS;
        for (int row0 = static_cast<int>(w.row0_or_e0); row0 < row_end && ok; row0 += 128, ++rb) {
          const int u = rb % US;
          if (!mbar_wait<true>(BAR_U_FULL(u), (rb / US) & 1, abort_flag, error, 9)) { ok = false; break; }
          const uint64_t desc_uhi = desc_u0 + static_cast<uint64_t>((u * 2 * Cfg::U_BYTES) >> 4);
          const uint64_t desc_ulo = desc_uhi + static_cast<uint64_t>(Cfg::U_BYTES >> 4);
          for (int sub = 0; sub < nsub; ++sub, ++t) {
            const int s = t % S, b = t % NACC;
            if (t >= NACC && !mbar_wait<true>(BAR_ACC_EMPTY(b), ((t / NACC) - 1) & 1, abort_flag, error, 5)) { ok = false; break; }
            tc_fence_after();
            const uint64_t desc_theta = desc_theta0 + static_cast<uint64_t>((s * Cfg::THETA_BYTES) >> 4);
            const uint32_t d = tmem_base + static_cast<uint32_t>(b * NS);
            const int nbox = (min(NS, w.ncols - NS * sub) + 63) / 64;
            // 2^s c b U G, split operands
            const uint64_t desc_ghi = desc_g0 + static_cast<uint64_t>((sub * 2 * Cfg::G_BYTES) >> 4);
            const uint64_t desc_glo = desc_ghi + static_cast<uint64_t>(Cfg::G_BYTES >> 4);
#pragma unroll
            for (int k = 0; k < KP / 16; ++k)
              umma(d, desc_ulo + static_cast<uint64_t>(2 * k), desc_ghi + static_cast<uint64_t>(2 * k), idesc_ug, k == 0 ? 0u : 1u);
#pragma unroll
            for (int k = 0; k < KP / 16; ++k) umma(d, desc_uhi + static_cast<uint64_t>(2 * k), desc_glo + static_cast<uint64_t>(2 * k), idesc_ug, 1u);
#pragma unroll
            for (int k = 0; k < KP / 16; ++k) umma(d, desc_uhi + static_cast<uint64_t>(2 * k), desc_ghi + static_cast<uint64_t>(2 * k), idesc_ug, 1u);
            // theta last, 16 columns at a time:  D <- theta I + 2^-s D
            if (!STATS) {
              if (!mbar_wait<true>(BAR_FULL(s), (t / S) & 1, abort_flag, error, 4)) { ok = false; break; }
              tc_fence_after();
#define ZGR_THETA_IN(SC)                                                                                                   \
  _Pragma("unroll") for (int c = 0; c < NS / 64; ++c) {                                                                    \
    if (c < nbox) {                                                                                                        \
      _Pragma("unroll") for (int k = 0; k < 4; ++k)                                                                        \
          umma_scaled_d<SC>(d + static_cast<uint32_t>(64 * c + 16 * k), desc_theta + static_cast<uint64_t>((c * 16384 + 32 * k) >> 4), \
                            desc_id, idesc_id);                                                                            \
    }                                                                                                                      \
  }
              switch (sh) {
                case 0: ZGR_THETA_IN(0) break;
                case 1: ZGR_THETA_IN(1) break;
                case 2: ZGR_THETA_IN(2) break;
                case 3: ZGR_THETA_IN(3) break;
                case 4: ZGR_THETA_IN(4) break;
                case 5: ZGR_THETA_IN(5) break;
                case 6: ZGR_THETA_IN(6) break;
                case 7: ZGR_THETA_IN(7) break;
                case 8: ZGR_THETA_IN(8) break;
                case 9: ZGR_THETA_IN(9) break;
                case 10: ZGR_THETA_IN(10) break;
                case 11: ZGR_THETA_IN(11) break;
                case 12: ZGR_THETA_IN(12) break;
                case 13: ZGR_THETA_IN(13) break;
                case 14: ZGR_THETA_IN(14) break;
                default: ZGR_THETA_IN(15) break;
              }
#undef ZGR_THETA_IN
            }
            umma_commit(BAR_ACC_FULL(b));
          }
          if (ok) umma_commit(BAR_U_FREE(u));   // arrives once every product that reads this U tile has completed
        }
      }
    }
  } else {
    // ===================================== epilogue warps =====================================
    // Warp (quad, cgrp) owns rows 32 quad .. 32 quad + 31 and columns 32 cgrp .. 32 cgrp + 31 of every tile.
    const int e = warp - 2;                 // 0..15
    const int quad = warp & 3;              // tensor-memory lane quadrant this warp may read
    constexpr int GROUPS = Cfg::GROUPS;                                      // each warp covers GROUPS column groups of its tiles
    const int grp = e / (kEpiWarps / GROUPS);                                // which tiles: t % GROUPS == grp
    const int cg_first = ((e >> 2) % (kEpiWarps / 4 / GROUPS)) * GROUPS;     // first 32-column group of this warp
    const int et = e * 32 + lane;
    const uint32_t tmem_row = tmem_base + (static_cast<uint32_t>(32 * quad) << 16);
    const int row_in_tile = 32 * quad + lane;
    const uint32_t row_xor16 = static_cast<uint32_t>(row_in_tile & 7) << 4;   // 128-byte swizzle: the 16-byte chunk index is xor-ed with the row
    const uint32_t theta_s32 = smem_u32(theta_base);
    const uint32_t g_s32 = smem_u32(g_base);
    int t = 0, item_no = 0;
    bool ok = true;
    for (int it = blockIdx.x; it < p.n_items && ok; it += gridDim.x, ++item_no) {
      const WorkItem w = p.items[it];
      const TensorDesc& td = p.tensors[w.tensor];
      const uint32_t tid = static_cast<uint32_t>(td.id);
      const int r = td.rank;
      const uint64_t tcols = static_cast<uint64_t>(td.cols);   // kept in a register: the barriers below force reloads of anything read through td
      const int sh = acc_shift(td, p);
      const float gscale = __int_as_float((127 + sh - td.ushift) << 23);   // 2^(s - j): the strips hold c b G 2^(s - j)
      if (GROUPS > 1 && t > 0) {
        // The strips are about to be overwritten.  With two groups this warp may be one tile ahead of the
        // other group, whose last tile of the previous item can still have products in flight that read the
        // old strips: wait until that tile's accumulator is complete (no later product exists before BAR_G).
        const int tp = t - 1;
        if (!mbar_wait<false>(BAR_ACC_FULL(tp % NACC), (tp / NACC) & 1, abort_flag, error, 11)) break;
      }
      // ---- coefficient strips c b G -> K-major hi/lo operands, one per tile of a row block ----
      for (int idx = et; idx < (KP / 2) * (NSUB * NS / 8); idx += kEpiWarps * 32) {
        // consecutive lanes take consecutive pairs of rows k of the same columns: their 32-bit stores below then
        // fall into KP/2 consecutive words of one operand row (with the octet index fastest they would all hit
        // one bank: 27 wavefronts per store instead of 2)
        const int kp = idx % (KP / 2), o = idx / (KP / 2);
        const int cc = 8 * o;                       // column within the item's strip
        if (cc >= ((w.ncols + NS - 1) / NS) * NS) continue;   // tiles of this item that do not exist
        float g0[8], g1[8];
        if (cc < w.ncols && 2 * kp < r) {
          guided8<BITS, false, MULTI>(td, p, 2 * kp, w.col0 + cc, g0);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) g0[i] = 0.0f;
        }
        if (cc < w.ncols && 2 * kp + 1 < r) {
          guided8<BITS, false, MULTI>(td, p, 2 * kp + 1, w.col0 + cc, g1);
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) g1[i] = 0.0f;
        }
        const uint32_t g_hi = g_s32 + static_cast<uint32_t>((cc / NS) * 2 * Cfg::G_BYTES);
        const uint32_t g_lo = g_hi + static_cast<uint32_t>(Cfg::G_BYTES);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          uint32_t hi, lo;
          split_f16(g0[i] * gscale, g1[i] * gscale, hi, lo);
          const uint32_t off = swizzle(static_cast<uint32_t>(((cc % NS) + i) * ROWB + 4 * kp), ROWB);
          sts32(g_hi + off, hi);
          sts32(g_lo + off, lo);
        }
      }
      fence_proxy_async();
      __syncwarp();
      if (lane == 0) mbar_arrive(BAR_G);
      // The epilogue warps of a scheduler run the same instruction stream from the same starting
      // point: first the integer rounds of the generator, then the special-function half of the
      // transform.  Holding every other column group back once per item puts half of each scheduler's
      // warps in the other phase, so the two pipes overlap (measured with one group: 6.5 -> 6.15 ms per 7B sweep;
      // with two groups the groups are out of step by construction).
      if (GROUPS == 1 && (cg_first & 1)) __nanosleep(kStaggerNs);

      const int row_end = static_cast<int>(w.row0_or_e0 + w.nrows_or_count);
      const int nsub = (w.ncols + NS - 1) / NS;
      double sum_iso = 0.0, sum_gd = 0.0, sum_z = 0.0;   // STATS / SSTATS only
      for (int row0 = static_cast<int>(w.row0_or_e0); row0 < row_end && ok; row0 += 128) {
        const int64_t row = static_cast<int64_t>(row0) + row_in_tile;
        const uint64_t row_oct0 = (static_cast<uint64_t>(row) * tcols + static_cast<uint64_t>(w.col0)) >> 3;   // octet index of the strip's first column in this row
        for (int sub = 0; sub < nsub; ++sub, ++t) {
          if (GROUPS > 1 && (t % GROUPS) != grp) continue;     // another group's tile
          const int s = t % S, b = t % NACC;
          if (!mbar_wait<false>(BAR_ACC_FULL(b), (t / NACC) & 1, abort_flag, error, 6)) { ok = false; break; }
          tc_fence_after();
#pragma unroll
          for (int pass = 0; pass < GROUPS; ++pass) {
          const int cgrp = cg_first + pass;                // which 32 columns of the tile
          const uint32_t tmem_warp = tmem_row + static_cast<uint32_t>(32 * cgrp);
          const uint32_t chunk0 = static_cast<uint32_t>(((32 * cgrp) & 63) >> 3);
          const uint32_t out_off = static_cast<uint32_t>(((32 * cgrp) >> 6) * 16384 + row_in_tile * 128);
          if (NS * sub + 32 * cgrp < w.ncols) {
            const uint64_t oct0 = row_oct0 + static_cast<uint64_t>((NS * sub + 32 * cgrp) >> 3);
            const uint32_t oct0_lo = static_cast<uint32_t>(oct0), oct0_hi = static_cast<uint32_t>(oct0 >> 32);
            // the row's 128 bytes in the staged tile start on a 128-byte boundary, so the swizzled chunk offset
            // (bits 4..6) can be xor-ed in rather than added: one logic instruction per chunk
            const uint32_t out_box = (theta_s32 + static_cast<uint32_t>(s * Cfg::THETA_BYTES) + out_off) ^ row_xor16;
            uint32_t h0[16], h1[16];
            tmem_ld16(tmem_warp + static_cast<uint32_t>(b * NS), h0);
            tmem_ld16(tmem_warp + static_cast<uint32_t>(b * NS + 16), h1);
            tmem_ld_wait();
            if constexpr (STATS) {
              const float descale = __int_as_float((127 - sh) << 23);
              float f_iso = 0.0f, f_gd = 0.0f, f_z = 0.0f;
#pragma unroll
              for (int o = 0; o < 4; ++o) {
                float zi[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) zi[i] = 0.0f;
                const uint32_t lo = oct0_lo + static_cast<uint32_t>(o);
                normals8_acc<BITS>(p.term[0].keys, tid, lo, oct0_hi + (lo < oct0_lo ? 1u : 0u), p.term[0].iso, zi);
                const bool live = row < row_end && NS * sub + 32 * cgrp + 8 * o < w.ncols;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const float gd = __uint_as_float(o < 2 ? h0[8 * (o & 1) + i] : h1[8 * (o & 1) + i]) * descale;   // no identity product here: undo 2^s
                  if (live) {
                    f_iso = fmaf(zi[i], zi[i], f_iso);
                    f_gd = fmaf(gd, gd, f_gd);
                    f_z = fmaf(zi[i] + gd, zi[i] + gd, f_z);
                  }
                }
              }
              sum_iso += static_cast<double>(f_iso);
              sum_gd += static_cast<double>(f_gd);
              sum_z += static_cast<double>(f_z);
            } else {
            // four octets per thread, kept independent so that their generator chains interleave
#pragma unroll
            for (int o = 0; o < 4; ++o) {
              float acc[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) acc[i] = __uint_as_float(o < 2 ? h0[8 * (o & 1) + i] : h1[8 * (o & 1) + i]);
              const uint32_t lo = oct0_lo + static_cast<uint32_t>(o);
              if constexpr (SSTATS) {
                const uint32_t chunk_addr = out_box ^ ((chunk0 + static_cast<uint32_t>(o)) << 4);
                float th[8];
                unpack8<T>(lds128(chunk_addr), th);                      // theta, before this thread overwrites it
                float f_iso = 0.0f, f_gd = 0.0f, f_z = 0.0f;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const float gd = acc[i] - th[i];
                  f_gd = fmaf(gd, gd, f_gd);
                }
                normals8_acc_rsum<BITS>(p.term[0].keys, tid, lo, oct0_hi + (lo < oct0_lo ? 1u : 0u), p.term[0].iso, acc, f_iso);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                  const float zc = acc[i] - th[i];
                  f_z = fmaf(zc, zc, f_z);
                }
                if (row < row_end && NS * sub + 32 * cgrp + 8 * o < w.ncols) {
                  sum_iso += static_cast<double>(f_iso);
                  sum_gd += static_cast<double>(f_gd);
                  sum_z += static_cast<double>(f_z);
                }
              } else
              normals8_acc<BITS>(p.term[0].keys, tid, lo, oct0_hi + (lo < oct0_lo ? 1u : 0u), p.term[0].iso, acc);
              if (MULTI) {
#pragma unroll 1
                for (int q = 1; q < p.n_terms; ++q)
                  normals8_acc<BITS>(p.term[q].keys, tid, lo, oct0_hi + (lo < oct0_lo ? 1u : 0u), p.term[q].iso, acc);
              }
              if constexpr (ZOUT) {
                const int col = NS * sub + 32 * cgrp + 8 * o;          // within the item's strip
                if (row < row_end && col < w.ncols) {
                  float4* dst = reinterpret_cast<float4*>(p.zout + static_cast<uint64_t>(row) * tcols + static_cast<uint64_t>(w.col0 + col));
                  dst[0] = make_float4(acc[0], acc[1], acc[2], acc[3]);
                  dst[1] = make_float4(acc[4], acc[5], acc[6], acc[7]);
                }
              } else {
                const uint4 q = make_uint4(Pack16<T>::pack(acc[0], acc[1]), Pack16<T>::pack(acc[2], acc[3]), Pack16<T>::pack(acc[4], acc[5]),
                                           Pack16<T>::pack(acc[6], acc[7]));
                sts128(out_box ^ ((chunk0 + static_cast<uint32_t>(o)) << 4), q);
              }
            }
            }
          }
          }
          tc_fence_before();
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(BAR_ACC_EMPTY(b));
            if (!STATS) mbar_arrive(BAR_OUT(s));
          }
        }
      }
      if constexpr (STATS || SSTATS) {
        if (ok) store_item_stats(p, it, e, sum_iso, sum_gd, sum_z);   // one slot per epilogue warp (at most kStatSlots of them)
      }
    }
  }

  // ---- common exit ----
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, Cfg::TMEM_COLS);
  }
}

size_t umma_smem_bytes(int kpad) {
  return kpad == 16 ? UmmaCfg<16>::SMEM_BYTES : (kpad == 32 ? UmmaCfg<32>::SMEM_BYTES : UmmaCfg<64>::SMEM_BYTES);
}
int umma_strip_cols(int kpad) { return kpad == 64 ? UmmaCfg<64>::NS * UmmaCfg<64>::NSUB : (kpad == 32 ? UmmaCfg<32>::NS * UmmaCfg<32>::NSUB : UmmaCfg<16>::NS * UmmaCfg<16>::NSUB); }

namespace {
template <typename T, int BITS, bool STATS = false, bool MULTI = false, bool ZOUT = false, bool SSTATS = false>
cudaError_t launch_umma_kp(int kpad, const SweepParams& p, const CUtensorMap* tmaps, int* error, int grid, cudaStream_t st) {
  static_assert(UmmaCfg<16>::EPI_WARPS <= kStatSlots && UmmaCfg<32>::EPI_WARPS <= kStatSlots && UmmaCfg<64>::EPI_WARPS <= kStatSlots,
                "one bookkeeping slot per epilogue warp");
#define ZGR_LAUNCH_UMMA(KPV)                                                                                       \
  {                                                                                                                \
    auto k = sweep_umma_kernel<T, BITS, KPV, STATS, MULTI, ZOUT, SSTATS>;                                                 \
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, UmmaCfg<KPV>::SMEM_BYTES); \
    if (e != cudaSuccess) return e;                                                                                \
    k<<<grid, UmmaCfg<KPV>::THREADS, UmmaCfg<KPV>::SMEM_BYTES, st>>>(p, tmaps, error);                                      \
  }
  if (kpad == 16) ZGR_LAUNCH_UMMA(16)
  else if (kpad == 32) ZGR_LAUNCH_UMMA(32)
  else ZGR_LAUNCH_UMMA(64)
#undef ZGR_LAUNCH_UMMA
  return cudaGetLastError();
}
}  // namespace

namespace {
template <typename T>
cudaError_t launch_umma_typed(const KernelChoice& kc, const SweepParams& p, const CUtensorMap* tmaps, int* error, int grid, cudaStream_t st) {
  if (p.n_terms > 1) {
    return kc.bits == 32 ? launch_umma_kp<T, 32, false, true>(kc.kpad, p, tmaps, error, grid, st)
                         : launch_umma_kp<T, 16, false, true>(kc.kpad, p, tmaps, error, grid, st);
  }
  if (p.item_stats != nullptr) {   // the sweep also accumulates the norm bookkeeping
    return kc.bits == 32 ? launch_umma_kp<T, 32, false, false, false, true>(kc.kpad, p, tmaps, error, grid, st)
                         : launch_umma_kp<T, 16, false, false, false, true>(kc.kpad, p, tmaps, error, grid, st);
  }
  return kc.bits == 32 ? launch_umma_kp<T, 32>(kc.kpad, p, tmaps, error, grid, st) : launch_umma_kp<T, 16>(kc.kpad, p, tmaps, error, grid, st);
}
}  // namespace

cudaError_t launch_sweep_umma(const KernelChoice& kc, const SweepParams& p, const CUtensorMap* tmaps, int* error, int grid, cudaStream_t st) {
  if (kc.dtype == 2) return launch_umma_typed<__nv_bfloat16>(kc, p, tmaps, error, grid, st);
  if (kc.dtype == 1) return launch_umma_typed<__half>(kc, p, tmaps, error, grid, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_debug_z_umma(const KernelChoice& kc, const SweepParams& p, const CUtensorMap* tmaps, int* error, int grid, cudaStream_t st) {
  if (p.zout == nullptr || p.n_terms != 1) return cudaErrorInvalidValue;
  if (kc.dtype == 2)
    return kc.bits == 32 ? launch_umma_kp<__nv_bfloat16, 32, false, false, true>(kc.kpad, p, tmaps, error, grid, st)
                         : launch_umma_kp<__nv_bfloat16, 16, false, false, true>(kc.kpad, p, tmaps, error, grid, st);
  if (kc.dtype == 1)
    return kc.bits == 32 ? launch_umma_kp<__half, 32, false, false, true>(kc.kpad, p, tmaps, error, grid, st)
                         : launch_umma_kp<__half, 16, false, false, true>(kc.kpad, p, tmaps, error, grid, st);
  return cudaErrorInvalidValue;
}

cudaError_t launch_stats_umma(const KernelChoice& kc, const SweepParams& p, const CUtensorMap* tmaps, int* error, int grid, cudaStream_t st) {
  // the storage type plays no role when no weights are touched: one instantiation serves all
  return kc.bits == 32 ? launch_umma_kp<__nv_bfloat16, 32, true>(kc.kpad, p, tmaps, error, grid, st)
                       : launch_umma_kp<__nv_bfloat16, 16, true>(kc.kpad, p, tmaps, error, grid, st);
}

}  // namespace zgr
