// Scalar building blocks of the race: Philox4x32-10, the Exp(1) transform and
// the two evaluations of a race key.  Plain C++ when compiled without nvcc so
// that a host harness can check the error bounds that the kernels rely on.
#pragma once
#include <math.h>
#include <stdint.h>
#include <string.h>

#if defined(__CUDACC__)
#define ERSD_HD __host__ __device__ __forceinline__
#else
#define ERSD_HD inline
#endif

namespace ersd {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

ERSD_HD void mulhilo(uint32_t a, uint32_t b, uint32_t& hi, uint32_t& lo) {
  const uint64_t p = (uint64_t)a * (uint64_t)b;
  hi = (uint32_t)(p >> 32);
  lo = (uint32_t)p;
}

// Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11): ten rounds of two
// 32x32->64 products and a word shuffle, the key advancing by the Weyl
// constants between rounds.
ERSD_HD void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                           uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t hi0, lo0, hi1, lo1;
    mulhilo(kPhiloxM0, c0, hi0, lo0);
    mulhilo(kPhiloxM1, c2, hi1, lo1);
    c0 = hi1 ^ c1 ^ k0;
    c1 = lo1;
    c2 = hi0 ^ c3 ^ k1;
    c3 = lo0;
    k0 += kPhiloxW0;
    k1 += kPhiloxW1;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

// Philox4x32-10 for one race: the counter is (c0, position, sequence id, 0) with only c0
// varying along a row, so everything that does not depend on c0 is folded once per row:
// round 1 needs one product (the other multiplies the sequence id), round 2 one product
// (its c0 is a row constant), and three of the key/word xors collapse into constants.
// 18 wide multiplies and 19 xors per call instead of 20 and 20.
struct PhiloxRow {
  uint32_t r1_k1;        // round 1: c2' = hi(M0*c0) ^ r1_k1            (c3 = 0)
  uint32_t r2_a;         // round 2: c0' = hi(M1*c2) ^ r2_a             (r2_a = lo(M1*seq) ^ k0[1])
  uint32_t r2_b;         // round 2: c2' = c3 ^ r2_b                    (r2_b = hi(M0*A0) ^ k1[1])
  uint32_t r3_b;         // round 3: c2' = hi(M0*c0) ^ r3_b             (r3_b = lo(M0*A0) ^ k1[2])
  uint32_t k0[10], k1[10];  // round keys (entries 2.. / 3.. are used)

  ERSD_HD void init(uint64_t seed, uint32_t seq_id, uint32_t position) {
    uint32_t a = (uint32_t)seed, b = (uint32_t)(seed >> 32);
#pragma unroll
    for (int r = 0; r < 10; ++r) {
      k0[r] = a;
      k1[r] = b;
      a += kPhiloxW0;
      b += kPhiloxW1;
    }
    uint32_t hi1, lo1, H0, L0;
    mulhilo(kPhiloxM1, seq_id, hi1, lo1);
    const uint32_t A0 = hi1 ^ position ^ k0[0];  // c0 after round 1
    mulhilo(kPhiloxM0, A0, H0, L0);
    r1_k1 = k1[0];
    r2_a = lo1 ^ k0[1];
    r2_b = H0 ^ k1[1];
    r3_b = L0 ^ k1[2];
  }

  ERSD_HD void words(uint32_t c0, uint32_t out[4]) const {
    uint32_t hi0, lo0, hi1, lo1;
    mulhilo(kPhiloxM0, c0, hi0, lo0);  // round 1
    uint32_t c2 = hi0 ^ r1_k1, c3 = lo0;
    mulhilo(kPhiloxM1, c2, hi1, lo1);  // round 2
    uint32_t n0 = hi1 ^ r2_a, n1 = lo1, n2 = c3 ^ r2_b;
    mulhilo(kPhiloxM0, n0, hi0, lo0);  // round 3
    mulhilo(kPhiloxM1, n2, hi1, lo1);
    uint32_t c0v = hi1 ^ n1 ^ k0[2], c1 = lo1;
    c2 = hi0 ^ r3_b;
    c3 = lo0;
#pragma unroll
    for (int r = 3; r < 10; ++r) {
      mulhilo(kPhiloxM0, c0v, hi0, lo0);
      mulhilo(kPhiloxM1, c2, hi1, lo1);
      c0v = hi1 ^ c1 ^ k0[r];
      c1 = lo1;
      c2 = hi0 ^ c3 ^ k1[r];
      c3 = lo0;
    }
    out[0] = c0v;
    out[1] = c1;
    out[2] = c2;
    out[3] = c3;
  }
};

// The 32-bit word of token i in the race keyed by (seed, seq_id, position).
ERSD_HD uint32_t token_word(uint64_t seed, uint32_t seq_id, uint32_t position, uint32_t i) {
  uint32_t o[4];
  philox4x32_10(i >> 2, position, seq_id, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), o);
  return o[i & 3u];
}

ERSD_HD float lg2_fast(float a) {
#if defined(__CUDA_ARCH__)
  float r;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(a));
  return r;
#else
  return log2f(a);
#endif
}

// 1 / d for d in [1, 4], to double precision: hardware seed and three Newton steps on the
// device (each squares the relative error), a plain division on the host.
ERSD_HD double recip_1_4(double d) {
#if defined(__CUDA_ARCH__)
  double r;
  asm("rcp.approx.ftz.f64 %0, %1;" : "=d"(r) : "d"(d));
  double e = fma(-d, r, 1.0);
  r = fma(r, e, r);
  e = fma(-d, r, 1.0);
  r = fma(r, e, r);
  e = fma(-d, r, 1.0);
  r = fma(r, e, r);
  return r;
#else
  return 1.0 / d;
#endif
}

ERSD_HD double bits_to_double(uint64_t b) {
#if defined(__CUDA_ARCH__)
  return __longlong_as_double((long long)b);
#else
  double d;
  memcpy(&d, &b, sizeof d);
  return d;
#endif
}
ERSD_HD uint64_t double_to_bits(double d) {
#if defined(__CUDA_ARCH__)
  return (uint64_t)__double_as_longlong(d);
#else
  uint64_t b;
  memcpy(&b, &d, sizeof b);
  return b;
#endif
}

// atanh(s) / s - 1 = s^2/3 + s^4/5 + ... truncated after s^(2 N); for |s| <= 1/3 and N = 16
// (resp. |s| <= 0.1716 and N = 10) the truncation is below 2^-56 of the sum.
template <int N>
ERSD_HD double atanh_tail(double s2) {
  double p = 1.0 / (2 * N + 1);
#pragma unroll
  for (int n = N - 1; n >= 1; --n) p = fma(p, s2, 1.0 / (2 * n + 1));
  return p * s2;
}

// ln(u) for a positive normal double, straight-line: u = m 2^k with m in [sqrt(1/2), sqrt(2)),
// ln m = 2 atanh((m - 1) / (m + 1)).  A few ulp; no special cases (callers keep u in range).
ERSD_HD double ln_pos(double u) {
  uint64_t b = double_to_bits(u);
  const int32_t hi = (int32_t)(b >> 32);
  const int32_t k = (hi - 0x3FE6A09E) >> 20;  // high word of sqrt(1/2); arithmetic shift = floor
  b -= (uint64_t)((int64_t)k << 52);
  const double m = bits_to_double(b);
  const double s = (m - 1.0) * recip_1_4(m + 1.0);
  const double lnm = 2.0 * fma(s, atanh_tail<10>(s * s), s);
  return fma((double)k, 0.6931471805599453, lnm);
}

// ln(e) for e = -log1p(-w), w = (x + 1/2) 2^-32, in double precision (a few 1e-16 relative in
// e, below 1e-14 absolute in ln e).  This is the value that decides winners.
//   x <  2^31:  -log1p(-w) = 2 atanh(w / (2 - w)),   w / (2 - w) <= 1/3
//   x >= 2^31:  1 - w = (~x + 1/2) 2^-32 exactly,    e = -ln(1 - w)
ERSD_HD double exact_ln_e(uint32_t x) {
  double e;
  if ((int32_t)x >= 0) {
    const double w = ((double)x + 0.5) * (1.0 / 4294967296.0);
    const double s = w * recip_1_4(2.0 - w);
    e = 2.0 * fma(s, atanh_tail<16>(s * s), s);
  } else {
    const double v = ((double)(~x) + 0.5) * (1.0 / 4294967296.0);
    e = -ln_pos(v);
  }
  return ln_pos(e);
}

// Exact race key in natural-log units, inv_T = 1 / T in double; greedy rows use -z.
ERSD_HD double exact_key(uint32_t x, float z, double inv_T, bool greedy) {
  if (z != z) return (double)INFINITY;  // NaN logit counts as -inf
  if (greedy) return -(double)z;
  if (z == INFINITY) return -(double)INFINITY;
  if (z == -INFINITY) return (double)INFINITY;
  return fma(-(double)z, inv_T, exact_ln_e(x));
}
ERSD_HD double exact_key(uint32_t x, float z, float T) {
  return exact_key(x, z, T == 0.0f ? 0.0 : 1.0 / (double)T, T == 0.0f);
}

// Screening value: log2(e) in single precision from one int->float conversion
// and two lg2.approx.  x < 2^31: w = v below; else 1 - w = v.
//   w < 2^-6        e = w (1 + w/2)          (series; relative error < w^2/3)
//   2^-6 <= w < 1/2 e = -ln(1 - w)
//   w >= 1/2        e = -ln(1 - w), with 1 - w = (~x + 1/2) 2^-32 formed exactly
// The result is within kScreenCore of log2(e) for every x (host harness and a
// device test check this over all regimes).
constexpr float kScreenCore = 1.0f / 2048.0f;
ERSD_HD float screen_lg2_e(uint32_t x) {
  const uint32_t t = x ^ (uint32_t)((int32_t)x >> 31);  // x < 2^31 ? x : ~x
  const float v = fmaf((float)t, 2.3283064365386963e-10f, 1.1641532182693481e-10f);
  const bool low = (int32_t)x >= 0;
  const float a = low ? (1.0f - v) : v;
  const float el = -lg2_fast(a);                           // e / ln 2 (both upper regimes)
  const float es = v * fmaf(v, 0.5f, 1.0f) * 1.4426950408889634f;  // series, also / ln 2
  const float e_over_ln2 = (low && v < 0.015625f) ? es : el;
  return lg2_fast(e_over_ln2) - 0.5287663729448977f;       // + log2(ln 2)
}

// Slack (log2 units) that makes a comparison of a screening key against a
// threshold tau safe: |screen key - true key| <= slack(tau) whenever the true
// key is within a few units of tau.  Covers the core error above, the
// rounding of log2(e)/T, of the fused multiply-add and of unit conversions.
ERSD_HD float screen_slack(float tau) { return 0.001953125f + 9.5367431640625e-7f * fabsf(tau); }

}  // namespace ersd
