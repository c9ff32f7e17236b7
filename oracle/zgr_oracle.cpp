// CPU oracle for the ZGR step (zeroth-order step with cloud-guided gradient rectification).
//
// TEST INFRASTRUCTURE ONLY.  This file is the slow, plain, double-precision statement of what the
// hot path computes.  It shares no code with the CUDA library, is never called by it, and is used
// only by the tests, by the smoke check and by the benchmark's CPU-baseline leg.
//
// Every function below cites the passage of the paper it follows:
//   Eq. (ZOO)           two-point antithetic estimator          g = (L+ - L-)/(2 eps) * z
//   Eq. (perturbation)  hybrid perturbation                     z_h = sqrt(alpha/n) z + sqrt((1-alpha)/m) V z_g
//   Eq. (grad)          gradient recovery with z_h, regenerated from the shared seed
//   Algorithm 1         client / edge-server procedure, update  W <- W - eta * g
//   Sec. 3.4 (DTC)      x_quant = round(x/lambda + delta),  x = lambda (x_quant - delta)
//
// Where the paper is silent the reading is fixed here once (and listed in the design notes):
//   * "the seed" -> Philox4x32-10 (Salmon et al., SC'11), key = (seed lo, seed hi),
//     counter = (block lo, block hi, tensor id, stream tag).
//   * uniforms -> normals by Box-Muller on exactly representable odd-numerator uniforms.
//   * V = blockdiag_l(U_l (x) I_{n_l}) with U_l (m_l x r) orthonormal columns, z_g = vec(G_l),
//     so n := d = sum m_l n_l and m := K = sum r_l n_l in Eq. (perturbation).
//
// Parity pins (tests/test_oracle_*.py): Philox against two independent library implementations,
// moments/KS of the normal stream, brute-force dense construction of Eq. (perturbation),
// span and covariance properties, exactness of the central difference on a quadratic, restore at
// lr = 0 with double storage, DTC error bound, rounding against brute-force nearest search;
// multi-seed sweeps against single sweeps, linearity and a dense construction; the Householder basis
// against a library QR, its defining properties and a hand-worked 3 x 2 case; the adaptive mixing ratio
// against the balance it is defined by, recomputed from the norms after the change.
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10.  One round multiplies counter words 0 and 2 by fixed odd constants, keeps the low
// halves, and xors the high halves with the other two words and the round key; the key is bumped
// by the Weyl constants between rounds.
// ---------------------------------------------------------------------------------------------
constexpr uint32_t kMul0 = 0xD2511F53u;
constexpr uint32_t kMul1 = 0xCD9E8D57u;
constexpr uint32_t kWeyl0 = 0x9E3779B9u;  // floor(2^32 * (golden ratio - 1))
constexpr uint32_t kWeyl1 = 0xBB67AE85u;  // floor(2^32 * (sqrt(3) - 1))

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) {
      k0 += kWeyl0;
      k1 += kWeyl1;
    }
    const uint64_t p0 = static_cast<uint64_t>(kMul0) * c0;
    const uint64_t p1 = static_cast<uint64_t>(kMul1) * c2;
    const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
    const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n1 = lo1;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    const uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// Block j of stream (seed, tensor, tag).
void stream_block(uint64_t seed, uint64_t j, uint32_t tensor, uint32_t tag, uint32_t out[4]) {
  const uint32_t ctr[4] = {static_cast<uint32_t>(j), static_cast<uint32_t>(j >> 32), tensor, tag};
  const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
  philox4x32_10(ctr, key, out);
}

constexpr double kTwoPi = 6.283185307179586476925286766559;

// Uniform in (0,1) from the top `nbits` bits k of a field: u = (2k+1) / 2^(nbits+1).
inline double odd_uniform(uint32_t k, int nbits) {
  return (2.0 * static_cast<double>(k) + 1.0) * std::ldexp(1.0, -(nbits + 1));
}

// Box-Muller: (u1,u2) -> (rho cos phi, rho sin phi), rho = sqrt(-2 ln u1), phi = 2 pi u2.
inline double box_muller(double u1, double u2, int which) {
  const double rho = std::sqrt(-2.0 * std::log(u1));
  const double phi = kTwoPi * u2;
  return which == 0 ? rho * std::cos(phi) : rho * std::sin(phi);
}

// Standard normal attached to element index e of stream (seed, tensor, tag)  [z ~ N(0, I_d), Eq. (ZOO)].
//   bits == 32: block j = e/4 serves elements 4j..4j+3; words (x0,x1) -> normals 0,1 and (x2,x3) ->
//               normals 2,3; the uniform field of a word is its low 23 bits: k = x & 0x7FFFFF.
//   bits == 16: block j = e/8 serves elements 8j..8j+7; word x_w -> normals 2w, 2w+1 with
//               k1 = bits 7..22 of x (radius) and k2 = bits 7..22 of x rotated by 16, i.e. the
//               remaining bits 23..31 (low part of k2) and 0..6 (high part of k2) (angle).
double normal_at(uint64_t seed, uint32_t tensor, uint32_t tag, int bits, uint64_t e) {
  uint32_t x[4];
  if (bits == 32) {
    stream_block(seed, e / 4, tensor, tag, x);
    const int w = static_cast<int>(e % 4);
    const int pair = w / 2;
    const double u1 = odd_uniform(x[2 * pair] & 0x7FFFFFu, 23);
    const double u2 = odd_uniform(x[2 * pair + 1] & 0x7FFFFFu, 23);
    return box_muller(u1, u2, w % 2);
  }
  stream_block(seed, e / 8, tensor, tag, x);
  const int w = static_cast<int>(e % 8);
  const uint32_t word = x[w / 2];
  const uint32_t rot = (word << 16) | (word >> 16);
  const double u1 = odd_uniform((word >> 7) & 0xFFFFu, 16);
  const double u2 = odd_uniform((rot >> 7) & 0xFFFFu, 16);
  return box_muller(u1, u2, w % 2);
}

// ---------------------------------------------------------------------------------------------
// Storage types and round-to-nearest-even from double, done directly (no detour through float).
// ---------------------------------------------------------------------------------------------
enum { DT_F32 = 0, DT_F16 = 1, DT_BF16 = 2, DT_F64 = 3 };

// Round x to a binary format with `p` significand bits (incl. the hidden one), minimum normal
// exponent emin (value of the smallest normal = 2^emin) and largest finite value maxfinite.
double round_to_format(double x, int p, int emin, double maxfinite) {
  if (std::isnan(x) || std::isinf(x) || x == 0.0) return x;
  int e;
  std::frexp(x, &e);              // |x| = f * 2^e with f in [0.5, 1)
  int ex = e - 1;                 // |x| in [2^ex, 2^(ex+1))
  if (ex < emin) ex = emin;       // subnormal range shares the quantum of the smallest normal
  const double quantum = std::ldexp(1.0, ex - (p - 1));
  const double q = std::nearbyint(x / quantum);   // default rounding mode: ties to even
  const double r = q * quantum;
  // Overflow threshold of round-to-nearest: halfway between maxfinite and the next power of two.
  const double ulp_top = std::ldexp(1.0, static_cast<int>(std::floor(std::log2(maxfinite))) - (p - 1));
  if (std::fabs(r) > maxfinite) {
    if (std::fabs(x) >= maxfinite + 0.5 * ulp_top) return std::copysign(std::numeric_limits<double>::infinity(), x);
    return std::copysign(maxfinite, x);
  }
  return r;
}

double round_to(double x, int dtype) {
  switch (dtype) {
    case DT_F32: return static_cast<double>(static_cast<float>(x));  // IEEE conversion, RNE
    case DT_F16: return round_to_format(x, 11, -14, 65504.0);
    case DT_BF16: return round_to_format(x, 8, -126, 3.3895313892515355e38);
    default: return x;
  }
}

// Bit-level encode/decode of the 16-bit types (values are already representable when encoding).
double decode_f16(uint16_t h) {
  const int sign = h >> 15, ex = (h >> 10) & 0x1F, man = h & 0x3FF;
  double v;
  if (ex == 0) v = std::ldexp(static_cast<double>(man), -24);
  else if (ex == 31) v = man ? std::numeric_limits<double>::quiet_NaN() : std::numeric_limits<double>::infinity();
  else v = std::ldexp(1.0 + man / 1024.0, ex - 15);
  return sign ? -v : v;
}
uint16_t encode_f16(double v) {
  uint16_t sign = std::signbit(v) ? 0x8000u : 0u;
  double a = std::fabs(v);
  if (std::isnan(v)) return 0x7E00u;
  if (std::isinf(v)) return sign | 0x7C00u;
  if (a == 0.0) return sign;
  if (a < std::ldexp(1.0, -14)) return sign | static_cast<uint16_t>(std::ldexp(a, 24));
  int e;
  const double f = std::frexp(a, &e);  // a = f 2^e, f in [0.5,1)
  const int ex = e - 1 + 15;
  const int man = static_cast<int>((f * 2.0 - 1.0) * 1024.0);
  return sign | static_cast<uint16_t>(ex << 10) | static_cast<uint16_t>(man);
}
double decode_bf16(uint16_t h) {
  const uint32_t w = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &w, 4);
  return static_cast<double>(f);
}
uint16_t encode_bf16(double v) {
  const float f = static_cast<float>(v);  // exact: v is a bf16 value
  uint32_t w;
  std::memcpy(&w, &f, 4);
  return static_cast<uint16_t>(w >> 16);
}

double load_elem(const void* base, int dtype, int64_t i) {
  switch (dtype) {
    case DT_F32: return static_cast<double>(static_cast<const float*>(base)[i]);
    case DT_F16: return decode_f16(static_cast<const uint16_t*>(base)[i]);
    case DT_BF16: return decode_bf16(static_cast<const uint16_t*>(base)[i]);
    default: return static_cast<const double*>(base)[i];
  }
}
void store_elem(void* base, int dtype, int64_t i, double v) {
  switch (dtype) {
    case DT_F32: static_cast<float*>(base)[i] = static_cast<float>(v); break;
    case DT_F16: static_cast<uint16_t*>(base)[i] = encode_f16(v); break;
    case DT_BF16: static_cast<uint16_t*>(base)[i] = encode_bf16(v); break;
    default: static_cast<double*>(base)[i] = v; break;
  }
}

// Coefficient G_l[k,c]  [z_g ~ N(0, I_m), Algorithm 1 "Sample z_g"]: either the tag-1 normal at
// element k*cols + c, or the DTC-dequantised value lambda_k (q[k,c] - delta_k)  [Sec. 3.4].
// A proportion of the payload may arrive compressed (Sec. 3.4, the adaptive proportion omega): here the first
// qrows rows of G_l come from the codes and the remaining rows are drawn from the seed.
struct CoeffSource {
  const int8_t* q;      // qrows x cols, or null -> seed-generated
  const float* scale;   // qrows
  const float* zero;    // qrows or null (delta = 0)
  int64_t qrows;        // rows of G_l taken from the codes (= rank when everything arrives compressed)
};
double coeff_at(const CoeffSource& cs, uint64_t seed, uint32_t tensor, int bits, int64_t cols, int64_t k, int64_t c) {
  if (cs.q && k < cs.qrows) {
    const double lambda = static_cast<double>(cs.scale[k]);
    const double delta = cs.zero ? static_cast<double>(cs.zero[k]) : 0.0;
    return lambda * (static_cast<double>(cs.q[k * cols + c]) - delta);
  }
  return normal_at(seed, tensor, /*tag=*/1u, bits, static_cast<uint64_t>(k) * static_cast<uint64_t>(cols) + static_cast<uint64_t>(c));
}

}  // namespace

extern "C" {

// --- generator ------------------------------------------------------------------------------
void zgro_philox4x32_10(const uint32_t* ctr, const uint32_t* key, uint32_t* out) { philox4x32_10(ctr, key, out); }

void zgro_blocks(uint64_t seed, uint32_t tensor, uint32_t tag, uint64_t first_block, int64_t n_blocks, uint32_t* out) {
  for (int64_t b = 0; b < n_blocks; ++b) stream_block(seed, first_block + static_cast<uint64_t>(b), tensor, tag, out + 4 * b);
}

// Normals for elements e0 .. e0+count-1 of stream (seed, tensor, tag).
void zgro_normals(uint64_t seed, uint32_t tensor, uint32_t tag, int bits, uint64_t e0, int64_t count, double* out) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) out[i] = normal_at(seed, tensor, tag, bits, e0 + static_cast<uint64_t>(i));
}

// --- scalars --------------------------------------------------------------------------------
// Mixing scalars of Eq. (perturbation) with n := d (all parameters), m := K (all guided coefficients).
//   scale_mode 0: a = sqrt(alpha/d),  b = sqrt((1-alpha)/K)             (the equation to the letter)
//   scale_mode 1: both multiplied by sqrt(d): a = sqrt(alpha), b = sqrt((1-alpha) d / K)
//                 (unit per-element variance; alpha = 1 gives exactly the z of Eq. (ZOO))
// K == 0 (no guided tensor) gives b = 0.
void zgro_mix_scalars(double alpha, int64_t d, int64_t K, int scale_mode, double* a, double* b) {
  const double dd = static_cast<double>(d), kk = static_cast<double>(K);
  double aa = std::sqrt(alpha / dd);
  double bb = K > 0 ? std::sqrt((1.0 - alpha) / kk) : 0.0;
  if (scale_mode == 1) {
    aa *= std::sqrt(dd);
    bb *= std::sqrt(dd);
  }
  *a = aa;
  *b = bb;
}

// Projected-gradient scalar of Eq. (grad): g = (L+ - L-) / (2 eps).
double zgro_projected_grad(double loss_plus, double loss_minus, double eps) { return (loss_plus - loss_minus) / (2.0 * eps); }

// --- rounding -------------------------------------------------------------------------------
void zgro_round(const double* x, int64_t n, int dtype, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = round_to(x[i], dtype);
}
void zgro_decode(const void* src, int dtype, int64_t n, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = load_elem(src, dtype, i);
}
void zgro_encode(const double* src, int dtype, int64_t n, void* out) {
  for (int64_t i = 0; i < n; ++i) store_elem(out, dtype, i, round_to(src[i], dtype));
}

// --- coefficients and perturbation ------------------------------------------------------------
// G_l (rank x cols) as doubles.
void zgro_coeffs(uint64_t seed, uint32_t tensor, int bits, int64_t rank, int64_t cols, const int8_t* q, const float* scale,
                 const float* zero, int64_t qrows, double* out) {
  const CoeffSource cs{q, scale, zero, qrows};
#pragma omp parallel for schedule(static)
  for (int64_t k = 0; k < rank; ++k)
    for (int64_t c = 0; c < cols; ++c) out[k * cols + c] = coeff_at(cs, seed, tensor, bits, cols, k, c);
}

// Hybrid perturbation of one tensor  [Eq. (perturbation); Algorithm 1 "Form hybrid perturbation"]:
//   z[i,c] = a * z_iso[i,c] + b * sum_k U[i,k] G[k,c],     z_iso[i,c] = tag-0 normal at i*cols + c.
// U is rows x rank row-major (fp32 values); rank == 0 or U == null -> isotropic part only.
// Any of z_out / iso_out / guided_out may be null.  iso_out receives a*z_iso, guided_out b*U G.
void zgro_z_tensor(uint64_t seed, uint32_t tensor, int bits, int64_t rows, int64_t cols, const float* U, int64_t rank,
                   const int8_t* q, const float* scale, const float* zero, int64_t qrows, double a, double b, double* z_out,
                   double* iso_out, double* guided_out) {
  const bool guided = (U != nullptr && rank > 0);
  std::vector<double> G;
  if (guided) {
    G.resize(static_cast<size_t>(rank * cols));
    zgro_coeffs(seed, tensor, bits, rank, cols, q, scale, zero, qrows, G.data());
  }
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < rows; ++i) {
    for (int64_t c = 0; c < cols; ++c) {
      const uint64_t e = static_cast<uint64_t>(i) * static_cast<uint64_t>(cols) + static_cast<uint64_t>(c);
      const double iso = a * normal_at(seed, tensor, 0u, bits, e);
      double p = 0.0;
      if (guided)
        for (int64_t k = 0; k < rank; ++k) p += static_cast<double>(U[i * rank + k]) * G[static_cast<size_t>(k * cols + c)];
      const double g = b * p;
      if (z_out) z_out[e] = iso + g;
      if (iso_out) iso_out[e] = iso;
      if (guided_out) guided_out[e] = g;
    }
  }
}

// The same perturbation at selected elements (random access): idx are linear indices i*cols + c.
void zgro_z_elements(uint64_t seed, uint32_t tensor, int bits, int64_t rows, int64_t cols, const float* U, int64_t rank,
                     const int8_t* q, const float* scale, const float* zero, int64_t qrows, double a, double b, int64_t n_idx,
                     const int64_t* idx, double* z_out) {
  (void)rows;
  const bool guided = (U != nullptr && rank > 0);
  const CoeffSource cs{q, scale, zero, qrows};
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < n_idx; ++t) {
    const int64_t e = idx[t];
    const int64_t i = e / cols, c = e % cols;
    double z = a * normal_at(seed, tensor, 0u, bits, static_cast<uint64_t>(e));
    if (guided) {
      double p = 0.0;
      for (int64_t k = 0; k < rank; ++k) p += static_cast<double>(U[i * rank + k]) * coeff_at(cs, seed, tensor, bits, cols, k, c);
      z += b * p;
    }
    z_out[t] = z;
  }
}

// --- sweeps ---------------------------------------------------------------------------------
// One sweep over a whole tensor, in place:  theta <- rnd_dtype(theta + c * z)
//   perturbation:    c = +eps, then c = -2 eps            [Algorithm 1 "Compute loss difference"]
//   restore+update:  c = -net - lr * g                    [Eq. (grad); Algorithm 1 "Update"]
// One rounding to the storage type per sweep.
void zgro_sweep_tensor(void* theta, int dtype, uint64_t seed, uint32_t tensor, int bits, int64_t rows, int64_t cols,
                       const float* U, int64_t rank, const int8_t* q, const float* scale, const float* zero, int64_t qrows, double a,
                       double b, double c) {
  const bool guided = (U != nullptr && rank > 0);
  std::vector<double> G;
  if (guided) {
    G.resize(static_cast<size_t>(rank * cols));
    zgro_coeffs(seed, tensor, bits, rank, cols, q, scale, zero, qrows, G.data());
  }
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < rows; ++i) {
    for (int64_t col = 0; col < cols; ++col) {
      const int64_t e = i * cols + col;
      double z = a * normal_at(seed, tensor, 0u, bits, static_cast<uint64_t>(e));
      if (guided) {
        double p = 0.0;
        for (int64_t k = 0; k < rank; ++k) p += static_cast<double>(U[i * rank + k]) * G[static_cast<size_t>(k * cols + col)];
        z += b * p;
      }
      const double th = load_elem(theta, dtype, e);
      store_elem(theta, dtype, e, round_to(th + c * z, dtype));
    }
  }
}

// The same sweep at selected elements: theta_in[t] is the current stored value of element idx[t]
// (already exact in the storage type); theta_out[t] receives the rounded result.
void zgro_sweep_elements(const double* theta_in, int dtype, uint64_t seed, uint32_t tensor, int bits, int64_t rows,
                         int64_t cols, const float* U, int64_t rank, const int8_t* q, const float* scale,
                         const float* zero, int64_t qrows, double a, double b, double c, int64_t n_idx, const int64_t* idx,
                         double* theta_out) {
  std::vector<double> z(static_cast<size_t>(n_idx));
  zgro_z_elements(seed, tensor, bits, rows, cols, U, rank, q, scale, zero, qrows, a, b, n_idx, idx, z.data());
  for (int64_t t = 0; t < n_idx; ++t) theta_out[t] = round_to(theta_in[t] + c * z[static_cast<size_t>(t)], dtype);
}

// Per-tensor energies of the two parts and of their sum: out = { sum (a z_iso)^2, sum (b U G)^2, sum z^2 }.
void zgro_stats_tensor(uint64_t seed, uint32_t tensor, int bits, int64_t rows, int64_t cols, const float* U, int64_t rank,
                       const int8_t* q, const float* scale, const float* zero, int64_t qrows, double a, double b, double* out3) {
  const int64_t n = rows * cols;
  std::vector<double> iso(static_cast<size_t>(n)), gd(static_cast<size_t>(n));
  zgro_z_tensor(seed, tensor, bits, rows, cols, U, rank, q, scale, zero, qrows, a, b, nullptr, iso.data(), gd.data());
  double s0 = 0, s1 = 0, s2 = 0;
  for (int64_t i = 0; i < n; ++i) {
    const double x = iso[static_cast<size_t>(i)], y = gd[static_cast<size_t>(i)];
    s0 += x * x;
    s1 += y * y;
    s2 += (x + y) * (x + y);
  }
  out3[0] = s0; out3[1] = s1; out3[2] = s2;
}

// --- several seeds in one sweep -----------------------------------------------------------------
// theta <- rnd_dtype(theta + sum_q c_q z(seed_q)), in place  [Algorithm 1: "Recover gradient" sums g_t z_t over
// the seeds (and, on the edge server, over the clients), "Update" applies the sum].  One rounding to the
// storage type for the whole sum; the terms are added in the order given.
void zgro_sweep_multi_tensor(void* theta, int dtype, int n_terms, const uint64_t* seeds, const double* coeffs, uint32_t tensor, int bits,
                             int64_t rows, int64_t cols, const float* U, int64_t rank, const int8_t* q, const float* scale, const float* zero,
                             int64_t qrows, double a, double b) {
  const bool guided = (U != nullptr && rank > 0);
  std::vector<std::vector<double>> G(static_cast<size_t>(n_terms));
  if (guided)
    for (int t = 0; t < n_terms; ++t) {
      G[static_cast<size_t>(t)].resize(static_cast<size_t>(rank * cols));
      zgro_coeffs(seeds[t], tensor, bits, rank, cols, q, scale, zero, qrows, G[static_cast<size_t>(t)].data());
    }
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < rows; ++i) {
    for (int64_t col = 0; col < cols; ++col) {
      const int64_t e = i * cols + col;
      double acc = load_elem(theta, dtype, e);
      for (int t = 0; t < n_terms; ++t) {
        const double iso = a * normal_at(seeds[t], tensor, 0u, bits, static_cast<uint64_t>(e));
        double p = 0.0;
        if (guided)
          for (int64_t k = 0; k < rank; ++k)
            p += static_cast<double>(U[i * rank + k]) * G[static_cast<size_t>(t)][static_cast<size_t>(k * cols + col)];
        const double z = iso + b * p;
        acc += coeffs[t] * z;
      }
      store_elem(theta, dtype, e, round_to(acc, dtype));
    }
  }
}

// The same at selected elements (theta_in: their current stored values; theta_out: the rounded results).
void zgro_sweep_multi_elements(const double* theta_in, int dtype, int n_terms, const uint64_t* seeds, const double* coeffs, uint32_t tensor,
                               int bits, int64_t rows, int64_t cols, const float* U, int64_t rank, const int8_t* q, const float* scale,
                               const float* zero, int64_t qrows, double a, double b, int64_t n_idx, const int64_t* idx, double* theta_out) {
  std::vector<double> acc(theta_in, theta_in + n_idx), z(static_cast<size_t>(n_idx));
  for (int t = 0; t < n_terms; ++t) {
    zgro_z_elements(seeds[t], tensor, bits, rows, cols, U, rank, q, scale, zero, qrows, a, b, n_idx, idx, z.data());
    for (int64_t j = 0; j < n_idx; ++j) acc[static_cast<size_t>(j)] += coeffs[t] * z[static_cast<size_t>(j)];
  }
  for (int64_t j = 0; j < n_idx; ++j) theta_out[j] = round_to(acc[static_cast<size_t>(j)], dtype);
}

// Coefficient of the fused restore + update sweep  [Eq. (grad); Algorithm 1 "Update": W <- W - eta g z]:
// the perturbation still applied under the seed (net) is taken back and the projected-gradient step added.
double zgro_update_coefficient(double net, double loss_plus, double loss_minus, double eps, double lr) {
  const double g = zgro_projected_grad(loss_plus, loss_minus, eps);
  return -net - lr * g;
}

// --- adaptive mixing ratio ------------------------------------------------------------------------
// Sec. 1 announces that the ZGR parameter follows the relative sizes of the guided (back-propagation
// based) and the isotropic (zeroth-order) part of the perturbation, and gives no rule.  The candidate
// taken: balance their energies.  With the per-tensor norms  S_iso = sum (a0 Z)^2,  S_g = sum (b0 U G)^2
// measured under the current scalars (a0, b0), the energies per unit of mixing weight are
//   rho_iso = (S_iso / a0^2) / d    and    rho_g = (S_g / b0^2) / K        (d, K as in zgro_mix_scalars),
// and Eq. (perturbation) with ratio alpha gives the parts the energies  alpha * s * rho_iso  and
// (1 - alpha) * s * rho_g  (s = 1 or d by scale mode).  They are equal at
//   alpha* = rho_g / (rho_iso + rho_g).
// The result is damped towards the old value and clamped:  alpha = clamp((1 - eta) alpha_old + eta alpha*).
// A part that is absent (a0 = 0, b0 = 0 or K = 0) leaves alpha unchanged.
double zgro_adapt_alpha(const double* stats3, int64_t n_tensors, double a0, double b0, int64_t d, int64_t K, double alpha_old,
                        double alpha_min, double alpha_max, double eta) {
  if (a0 == 0.0 || b0 == 0.0 || K <= 0) return alpha_old;
  double s_iso = 0.0, s_g = 0.0;
  for (int64_t l = 0; l < n_tensors; ++l) {
    s_iso += stats3[3 * l + 0];
    s_g += stats3[3 * l + 1];
  }
  const double rho_iso = s_iso / (a0 * a0) / static_cast<double>(d);
  const double rho_g = s_g / (b0 * b0) / static_cast<double>(K);
  if (!(rho_iso + rho_g > 0.0)) return alpha_old;
  const double target = rho_g / (rho_iso + rho_g);
  const double mixed = (1.0 - eta) * alpha_old + eta * target;
  return std::fmin(std::fmax(mixed, alpha_min), alpha_max);
}

// --- subspace construction ------------------------------------------------------------------------
// Algorithm 1 "Collect gradients to build basis V_r" (Sec. 3.2): an orthonormal basis of the span of the
// last r gradients of a tensor.  A is rows x r (column j = gradient j, row-major storage); Householder QR in
// double, A = Q R with R upper triangular; the thin Q (rows x r) is returned with the sign convention
// R_kk > 0, which makes it unique for a full-rank A.  R (r x r, row-major) is returned if R_out is not null.
void zgro_householder_qr(const double* A, int64_t rows, int64_t r, double* Q_out, double* R_out) {
  std::vector<double> W(A, A + rows * r);                       // working copy, becomes R in its upper triangle
  std::vector<double> V(static_cast<size_t>(rows * r), 0.0);    // Householder vectors, column k in V[:, k]
  std::vector<double> beta(static_cast<size_t>(r), 0.0);
  for (int64_t k = 0; k < r; ++k) {
    double norm2 = 0.0;
    for (int64_t i = k; i < rows; ++i) norm2 += W[static_cast<size_t>(i * r + k)] * W[static_cast<size_t>(i * r + k)];
    const double norm = std::sqrt(norm2);
    if (norm == 0.0) continue;
    const double x0 = W[static_cast<size_t>(k * r + k)];
    const double alpha = x0 >= 0.0 ? -norm : norm;            // reflect x onto alpha e_k, away from x0 (no cancellation)
    double vnorm2 = 0.0;
    for (int64_t i = k; i < rows; ++i) {
      double v = W[static_cast<size_t>(i * r + k)];
      if (i == k) v -= alpha;
      V[static_cast<size_t>(i * r + k)] = v;
      vnorm2 += v * v;
    }
    beta[static_cast<size_t>(k)] = vnorm2 > 0.0 ? 2.0 / vnorm2 : 0.0;
    for (int64_t j = k; j < r; ++j) {                          // W <- (I - beta v v^T) W on the trailing columns
      double dot = 0.0;
      for (int64_t i = k; i < rows; ++i) dot += V[static_cast<size_t>(i * r + k)] * W[static_cast<size_t>(i * r + j)];
      const double f = beta[static_cast<size_t>(k)] * dot;
      for (int64_t i = k; i < rows; ++i) W[static_cast<size_t>(i * r + j)] -= f * V[static_cast<size_t>(i * r + k)];
    }
  }
  // Q = H_0 H_1 ... H_{r-1} applied to the first r columns of the identity
  std::vector<double> Q(static_cast<size_t>(rows * r), 0.0);
  for (int64_t j = 0; j < r && j < rows; ++j) Q[static_cast<size_t>(j * r + j)] = 1.0;
  for (int64_t k = r - 1; k >= 0; --k) {
    for (int64_t j = 0; j < r; ++j) {
      double dot = 0.0;
      for (int64_t i = k; i < rows; ++i) dot += V[static_cast<size_t>(i * r + k)] * Q[static_cast<size_t>(i * r + j)];
      const double f = beta[static_cast<size_t>(k)] * dot;
      for (int64_t i = k; i < rows; ++i) Q[static_cast<size_t>(i * r + j)] -= f * V[static_cast<size_t>(i * r + k)];
    }
  }
  // sign convention: R_kk > 0
  for (int64_t k = 0; k < r; ++k) {
    const double sgn = W[static_cast<size_t>(k * r + k)] < 0.0 ? -1.0 : 1.0;
    for (int64_t i = 0; i < rows; ++i) Q_out[i * r + k] = sgn * Q[static_cast<size_t>(i * r + k)];
    if (R_out)
      for (int64_t j = 0; j < r; ++j) R_out[k * r + j] = j >= k ? sgn * W[static_cast<size_t>(k * r + j)] : 0.0;
  }
}

// --- DTC (Sec. 3.4) ---------------------------------------------------------------------------
// Affine b-bit quantiser of one row:  lambda = (max - min)/(2^b - 1),  x_q = round(x/lambda + delta),
// x = lambda (x_q - delta).  The zero point printed in the paper is garbled; the reading taken is the
// one that makes the codes span the signed b-bit range: delta = round(-min/lambda) - 2^(b-1).
// symmetric != 0 selects the zero-point-free form used for int8 coefficients:
//   lambda = max|x| / (2^(b-1) - 1),  delta = 0,  codes clamped to +-(2^(b-1) - 1).
void zgro_dtc_quantise_row(const double* x, int64_t n, int bits, int symmetric, int8_t* q_out, float* scale_out, float* zero_out) {
  double lo = x[0], hi = x[0], amax = std::fabs(x[0]);
  for (int64_t i = 1; i < n; ++i) {
    lo = std::fmin(lo, x[i]);
    hi = std::fmax(hi, x[i]);
    amax = std::fmax(amax, std::fabs(x[i]));
  }
  const double qmax = std::ldexp(1.0, bits - 1) - 1.0, qmin = symmetric ? -qmax : -std::ldexp(1.0, bits - 1);
  double lambda, delta;
  if (symmetric) {
    lambda = amax > 0 ? amax / qmax : 1.0;
    delta = 0.0;
  } else {
    lambda = hi > lo ? (hi - lo) / (std::ldexp(1.0, bits) - 1.0) : 1.0;
    delta = std::nearbyint(-lo / lambda) - std::ldexp(1.0, bits - 1);
  }
  const float lambda_f = static_cast<float>(lambda);   // the scale travels as fp32
  const double lam = static_cast<double>(lambda_f);
  for (int64_t i = 0; i < n; ++i) {
    double code = std::nearbyint(x[i] / lam + delta);
    code = std::fmin(std::fmax(code, qmin), qmax);
    q_out[i] = static_cast<int8_t>(code);
  }
  *scale_out = lambda_f;
  *zero_out = static_cast<float>(delta);
}

void zgro_dtc_dequantise_row(const int8_t* q, int64_t n, float scale, float zero, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = static_cast<double>(scale) * (static_cast<double>(q[i]) - static_cast<double>(zero));
}

// The paper's INT4 payload of Sec. 3.4: unsigned codes x_q in [0, 15], lambda = (max - min)/15 and a zero point
// per row, x = lambda (x_q - delta).  It is the affine 4-bit quantiser above with codes and zero point moved by
// 8 from the signed range [-8, 7] to the unsigned one (the dequantised values are unchanged).
void zgro_dtc_quantise_row_int4(const double* x, int64_t n, int8_t* q_out, float* scale_out, float* zero_out) {
  zgro_dtc_quantise_row(x, n, 4, 0, q_out, scale_out, zero_out);
  for (int64_t i = 0; i < n; ++i) q_out[i] = static_cast<int8_t>(q_out[i] + 8);
  *zero_out = *zero_out + 8.0f;
}

// Transmission layout of 4-bit codes: a row of `cols` codes becomes (cols + 1)/2 bytes, column 2j in the low
// nibble of byte j and column 2j + 1 in its high nibble; a missing last column is stored as 0.
void zgro_dtc_pack4(const int8_t* codes, int64_t rows, int64_t cols, uint8_t* out) {
  const int64_t nb = (cols + 1) / 2;
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t j = 0; j < nb; ++j) {
      const unsigned lo = static_cast<unsigned>(codes[r * cols + 2 * j]) & 15u;
      const unsigned hi = (2 * j + 1 < cols) ? (static_cast<unsigned>(codes[r * cols + 2 * j + 1]) & 15u) : 0u;
      out[r * nb + j] = static_cast<uint8_t>(lo | (hi << 4));
    }
}
void zgro_dtc_unpack4(const uint8_t* packed, int64_t rows, int64_t cols, int8_t* out) {
  const int64_t nb = (cols + 1) / 2;
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t c = 0; c < cols; ++c) {
      const unsigned byte = packed[r * nb + c / 2];
      out[r * cols + c] = static_cast<int8_t>((c & 1) ? (byte >> 4) : (byte & 15u));
    }
}

int zgro_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
