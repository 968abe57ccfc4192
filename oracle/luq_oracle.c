/*
 * CPU oracle for the 4-bit training hot path (LUQ paper).  TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, scalar C.  It shares no code, table or constant with the CUDA
 * library; only tests, the smoke check and the benchmark's cpu_baseline leg may
 * call it.  Every function names the passage of the paper it follows.
 *
 * Conventions (row-major everywhere):
 *   activations A[M x K], weights W[N x K], pre-activation gradient G[M x N]
 *   forward  Z  = A . W^T   [M x N]      (Eq. "Forward")
 *   backward dA = G . W     [M x K]      (Eq. "Backward")
 *   update   dW = G^T . A   [N x K]      (Eq. "Update")
 *   packed codes: two 4-bit codes per byte along the contiguous dimension,
 *   element 2j in the low nibble and element 2j+1 in the high nibble.
 *
 * Parity pins (see tests marked "not gpu"): grid membership, fixed points,
 * exact expectation, the literal two-draw transcription of T_alpha / Q_alpha,
 * the paper's worked values, Table 1 closed forms, brute force GEMMs, and the
 * Philox constants and stream (cuRAND's header constants and cuRAND's own block
 * function compiled for the host).  On a machine without the CUDA toolkit the
 * raw Philox stream is "parity unpinned": any fixed bijective stream satisfies
 * the paper, which names no generator.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_FLAG_NONFINITE 1
#define ORACLE_FLAG_RANGE 2

static uint32_t bits_of(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float float_of(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* ------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon et al., SC'11).  The paper is silent on the random  */
/* source (Sec. 4, Appendix A.5); the build's reading fixes this generator.  */
/* ------------------------------------------------------------------------ */
static const uint32_t PHILOX_MUL_A = 0xD2511F53u;  /* multiplies counter word 0 */
static const uint32_t PHILOX_MUL_B = 0xCD9E8D57u;  /* multiplies counter word 2 */
static const uint32_t PHILOX_WEYL_0 = 0x9E3779B9u; /* floor(2^32 (golden ratio - 1)) */
static const uint32_t PHILOX_WEYL_1 = 0xBB67AE85u; /* floor(2^32 (sqrt 3 - 1)) */

void oracle_philox_constants(uint32_t out[4]) {
  out[0] = PHILOX_MUL_A; out[1] = PHILOX_MUL_B; out[2] = PHILOX_WEYL_0; out[3] = PHILOX_WEYL_1;
}

void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    uint64_t p0 = (uint64_t)PHILOX_MUL_A * c0;
    uint64_t p1 = (uint64_t)PHILOX_MUL_B * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += PHILOX_WEYL_0; k1 += PHILOX_WEYL_1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 32-bit word that decides element `index` of sample `sample`:
 * key = seed + sample (64 bit, wrapping), counter = index / 4, word index % 4. */
uint32_t oracle_random_word(uint64_t seed, uint32_t sample, uint64_t index) {
  uint64_t s = seed + (uint64_t)sample;
  uint64_t block = index >> 2;
  uint32_t ctr[4] = {(uint32_t)block, (uint32_t)(block >> 32), 0u, 0u};
  uint32_t key[2] = {(uint32_t)s, (uint32_t)(s >> 32)};
  uint32_t w[4];
  oracle_philox4x32_10(ctr, key, w);
  return w[index & 3];
}

/* ------------------------------------------------------------------------ */
/* max|x| of a tensor (Sec. 4 "Above FP maximum", Eq. alpha: max(|x|)).       */
/* flags gets ORACLE_FLAG_NONFINITE if any element is NaN or Inf.            */
/* ------------------------------------------------------------------------ */
float oracle_amax(const float* x, size_t n, int* flags) {
  float m = 0.0f;
  int bad = 0;
  for (size_t i = 0; i < n; ++i) {
    float a = fabsf(x[i]);
    if (!(a <= 3.402823466e38f)) bad = 1; /* NaN or Inf */
    else if (a > m) m = a;
  }
  if (flags) *flags = bad ? ORACLE_FLAG_NONFINITE : 0;
  return m;
}

static int scale_usable(float c, int* flags) {
  /* A clip / max that is zero, non-finite or outside [2^-100, 2^100] produces
   * all-zero codes and a zero scale (build's convention; the paper is silent). */
  if (flags) *flags = 0;
  if (c == 0.0f) return 0;
  if (!(c <= 3.402823466e38f) || c < 0.0f) { if (flags) *flags = ORACLE_FLAG_NONFINITE; return 0; }
  if (c < 0x1p-100f || c > 0x1p100f) { if (flags) *flags = ORACLE_FLAG_RANGE; return 0; }
  return 1;
}

/* ------------------------------------------------------------------------ */
/* Q_INT: INT4 round-to-nearest (Sec. 3.3: RDN for weights and activations;  */
/* Appendix A.1: one high-precision scale per tensor).  Signed symmetric      */
/* grid -7..7, step s = clip/7, ties to even, two's-complement nibble.        */
/* ------------------------------------------------------------------------ */
float oracle_quant_int4(const float* x, size_t n, float clip, uint8_t* codes, int* flags) {
  if (!scale_usable(clip, flags)) { memset(codes, 0, (n + 1) / 2); return 0.0f; }
  float s = clip / 7.0f;
  float inv = 7.0f / clip;
  memset(codes, 0, (n + 1) / 2);
  for (size_t i = 0; i < n; ++i) {
    float y = x[i] * inv;
    float r = rintf(y); /* default rounding mode: nearest, ties to even */
    if (r > 7.0f) r = 7.0f;
    if (r < -7.0f) r = -7.0f;
    if (r != r) r = 0.0f; /* NaN element (only with a caller-supplied clip) -> 0 */
    int q = (int)r;
    uint8_t nib = (uint8_t)(q & 0xF);
    codes[i >> 1] |= (uint8_t)(nib << ((i & 1) * 4));
  }
  return s;
}

/* ------------------------------------------------------------------------ */
/* Unsigned INT4 for tensors that cannot be negative (post-ReLU activations).  */
/* Appendix "Quantization formats": scale = Delta / (2^b - 1), Delta the        */
/* quantized range: for the range [0, clip] and b = 4, s = clip/15 and the      */
/* codes are the integers 0..15 (all sixteen levels on one side of zero).       */
/* Round to nearest, ties to even; negative inputs clamp to 0.                  */
/* ------------------------------------------------------------------------ */
float oracle_quant_uint4(const float* x, size_t n, float clip, uint8_t* codes, int* flags) {
  if (!scale_usable(clip, flags)) { memset(codes, 0, (n + 1) / 2); return 0.0f; }
  float s = clip / 15.0f;
  float inv = 15.0f / clip;
  memset(codes, 0, (n + 1) / 2);
  for (size_t i = 0; i < n; ++i) {
    float y = x[i] * inv;
    float r = rintf(y);
    if (r > 15.0f) r = 15.0f;
    if (r < 0.0f) r = 0.0f;
    if (r != r) r = 0.0f; /* NaN element -> 0 */
    uint8_t nib = (uint8_t)((int)r & 0xF);
    codes[i >> 1] |= (uint8_t)(nib << ((i & 1) * 4));
  }
  return s;
}

int oracle_int4_value(uint8_t nibble) { /* two's complement 4 bit */
  int v = nibble & 0xF;
  return v >= 8 ? v - 16 : v;
}

/* ------------------------------------------------------------------------ */
/* LUQ = Q_alpha(T_alpha(x)) (Sec. 4).                                        */
/*   alpha = max|x| / 2^kmax            (Eq. alpha; the paper prints 2^(2^(b-1)) */
/*                                       with b = 3, i.e. kmax = 4)           */
/*   |x| <  alpha : sign*alpha w.p. |x|/alpha, else 0   (Eq. StochasticPruning) */
/*   2^(n-1) alpha <= |x| < 2^n alpha : up w.p. (|x| - 2^(n-1) alpha)/(2^(n-1) alpha) */
/*                                                      (Eq. unbiasedFpQ)     */
/* One random word decides both stages: T_alpha outputs 0, +-alpha or an     */
/* untouched in-range value and Q_alpha is deterministic on 0 and +-alpha.   */
/* t = |x|/alpha in IEEE binary32.  For t >= 1 the mantissa field of t is the */
/* up-probability times 2^23 and its exponent is the lower level's index.    */
/* Code c: 0 -> 0, c >= 1 -> alpha * 2^(c-1); nibble = sign<<3 | c, zero is 0x0. */
/* ------------------------------------------------------------------------ */
typedef struct { uint32_t lo_code; uint32_t threshold; } luq_bin;

static luq_bin luq_bin_of(float a, float alpha, int kmax) {
  luq_bin b;
  float t = a / alpha; /* IEEE-754 binary32 division, round to nearest even */
  if (t < 1.0f) {
    b.lo_code = 0;
    b.threshold = (uint32_t)(t * 4294967296.0f); /* exact scaling, truncation */
  } else {
    uint32_t u = bits_of(t);
    int e = (int)((u >> 23) & 0xFF) - 127;
    if (e >= kmax) { /* at or above the top level (or NaN/Inf): top code, no draw */
      b.lo_code = (uint32_t)(kmax + 1);
      b.threshold = 0;
    } else {
      b.lo_code = (uint32_t)(1 + e);
      b.threshold = (u & 0x7FFFFFu) << 9;
    }
  }
  return b;
}

float oracle_luq_alpha(float mx, int kmax) { return ldexpf(mx, -kmax); }

/* codes: n_samples planes of (n+1)/2 bytes each, sample-major. Returns alpha.
 * x[0] is element `first_index` (even) of the full tensor: the random word of an
 * element depends on its index in the whole tensor, so a window can be checked
 * without quantizing everything before it. */
float oracle_quant_luq_window(const float* x, size_t n, uint64_t first_index, float mx, int kmax,
                              uint64_t seed, int n_samples, uint8_t* codes, int* flags);

float oracle_quant_luq(const float* x, size_t n, float mx, int kmax, uint64_t seed,
                       int n_samples, uint8_t* codes, int* flags) {
  return oracle_quant_luq_window(x, n, 0, mx, kmax, seed, n_samples, codes, flags);
}

float oracle_quant_luq_window(const float* x, size_t n, uint64_t first_index, float mx, int kmax,
                              uint64_t seed, int n_samples, uint8_t* codes, int* flags) {
  size_t plane = (n + 1) / 2;
  memset(codes, 0, plane * (size_t)n_samples);
  if (!scale_usable(mx, flags)) return 0.0f;
  float alpha = oracle_luq_alpha(mx, kmax);
  for (int s = 0; s < n_samples; ++s) {
    uint8_t* out = codes + plane * (size_t)s;
    for (size_t i = 0; i < n; ++i) {
      float a = fabsf(x[i]);
      uint32_t sign = bits_of(x[i]) >> 31;
      luq_bin b = luq_bin_of(a, alpha, kmax);
      uint32_t r = oracle_random_word(seed, (uint32_t)s, first_index + (uint64_t)i);
      uint32_t c = b.lo_code + (r < b.threshold ? 1u : 0u);
      uint8_t nib = c ? (uint8_t)((sign << 3) | c) : 0;
      out[i >> 1] |= (uint8_t)(nib << ((i & 1) * 4));
    }
  }
  return alpha;
}

/* ------------------------------------------------------------------------ */
/* Biased logarithmic quantization: the "FP4" baseline of the ablation         */
/* (Sec. 4, Eq. RC).  Same grid, scale and code layout as LUQ, no randomness.  */
/*   in range  : RDNP(2^x) = 2^floor(log2(4/3 * 2^x)): the level nearest in     */
/*               linear distance; the midpoint of [2^n, 2^(n+1)] is 3/2 * 2^n   */
/*               and goes up (the floor of an exact integer).                   */
/*   below alpha (reading: the paper only draws it): the nearer of 0 and alpha, */
/*               |x| = alpha/2 goes up like the other midpoints.                */
/*   above max : the top level (cannot happen with mx = the tensor maximum).    */
/* Written on t = fl32(|x|/alpha), the quantity the LUQ decisions use too.      */
/* ------------------------------------------------------------------------ */
float oracle_quant_fp_nearest(const float* x, size_t n, float mx, int kmax, uint8_t* codes, int* flags) {
  size_t plane = (n + 1) / 2;
  memset(codes, 0, plane);
  if (!scale_usable(mx, flags)) return 0.0f;
  float alpha = oracle_luq_alpha(mx, kmax);
  for (size_t i = 0; i < n; ++i) {
    float t = fabsf(x[i]) / alpha;
    uint32_t sign = bits_of(x[i]) >> 31;
    uint32_t c;
    if (!(t < ldexpf(1.0f, kmax))) {      /* at or above the top level, Inf, NaN */
      c = (uint32_t)kmax + 1u;
    } else if (t < 1.0f) {
      c = (t >= 0.5f) ? 1u : 0u;
    } else {
      /* floor(log2(4/3 t)): the largest m with 2^m <= 4t/3, i.e. 3 * 2^m <= 4t (exact in double) */
      int m = 0;
      while (3.0 * ldexp(1.0, m + 1) <= 4.0 * (double)t) ++m;
      c = (uint32_t)m + 1u;                /* level alpha * 2^m has code m + 1 */
    }
    uint8_t nib = c ? (uint8_t)((sign << 3) | c) : 0;
    codes[i >> 1] |= (uint8_t)(nib << ((i & 1) * 4));
  }
  return alpha;
}

/* ------------------------------------------------------------------------ */
/* Partially unbiased arms of the ablation (Sec. 4, ablation figure and its    */
/* caption): "SR" makes the quantizer unbiased inside the range, "SU" below     */
/* it.  The grid, the scale alpha = max/2^kmax and the code layout are LUQ's;   */
/* each region follows either the stochastic rule or the deterministic one:    */
/*   |x| <  alpha : su ? sign*alpha w.p. |x|/alpha (Eq. StochasticPruning)      */
/*                     : the nearer of 0 and alpha, alpha/2 up                   */
/*   in range     : sr ? up w.p. (|x| - lo)/lo (Eq. unbiasedFpQ)                 */
/*                     : nearest power, midpoint 3/2 * 2^n up (Eq. RC)           */
/* sr and su both set is LUQ, both clear is the biased "FP4" baseline.          */
/* Reading: the paper names the arms and draws them, it does not print them.    */
/* ------------------------------------------------------------------------ */
float oracle_quant_fp_ablation(const float* x, size_t n, float mx, int kmax, uint64_t seed, int n_samples,
                               int sr, int su, uint8_t* codes, int* flags) {
  size_t plane = (n + 1) / 2;
  memset(codes, 0, plane * (size_t)n_samples);
  if (!scale_usable(mx, flags)) return 0.0f;
  float alpha = oracle_luq_alpha(mx, kmax);
  float top = ldexpf(1.0f, kmax);
  for (int s = 0; s < n_samples; ++s) {
    uint8_t* out = codes + plane * (size_t)s;
    for (size_t i = 0; i < n; ++i) {
      float t = fabsf(x[i]) / alpha; /* IEEE binary32 quotient, as in LUQ */
      uint32_t sign = bits_of(x[i]) >> 31;
      uint32_t r = oracle_random_word(seed, (uint32_t)s, (uint64_t)i);
      uint32_t c;
      if (!(t < top)) {                /* top level, Inf, NaN: nothing to decide */
        c = (uint32_t)kmax + 1u;
      } else if (t < 1.0f) {           /* below the range */
        if (su) c = (r < (uint32_t)(t * 4294967296.0f)) ? 1u : 0u;
        else c = (t >= 0.5f) ? 1u : 0u;
      } else {                         /* 2^e <= t < 2^(e+1), level codes e+1 and e+2 */
        int e = 0;
        while (ldexpf(1.0f, e + 1) <= t) ++e;
        float lo = ldexpf(1.0f, e);
        int up;
        if (sr) {
          /* (t - lo)/lo is exact in binary32: t - lo is exact and lo a power of two */
          float p = (t - lo) / lo;
          up = r < (uint32_t)(p * 4294967296.0f);
        } else {
          up = t >= 1.5f * lo;
        }
        c = (uint32_t)(e + 1 + up);
      }
      uint8_t nib = c ? (uint8_t)((sign << 3) | c) : 0;
      out[i >> 1] |= (uint8_t)(nib << ((i & 1) * 4));
    }
  }
  return alpha;
}

/* ------------------------------------------------------------------------ */
/* "INT4 unbiased" arm of the ablation: the uniform signed grid -7..7 with     */
/* stochastic rounding (Sec. 3.1, Eq. SR: up w.p. (x - l)/(u - l)).  The top    */
/* level is the tensor maximum, so nothing clips: s = max/7.  Taken on the     */
/* magnitude (the rule is symmetric): y = fl32(|x| * fl32(7/max)), clamped to   */
/* 7; l = floor(y); up w.p. y - l, decided as r < trunc((y - l) * 2^32);        */
/* the sign is applied afterwards, the code is the two's-complement nibble.    */
/* The random word of element i, sample s is the one LUQ would use.            */
/* ------------------------------------------------------------------------ */
float oracle_quant_int4_sr(const float* x, size_t n, float mx, uint64_t seed, int n_samples,
                           uint8_t* codes, int* flags) {
  size_t plane = (n + 1) / 2;
  memset(codes, 0, plane * (size_t)n_samples);
  if (!scale_usable(mx, flags)) return 0.0f;
  float s7 = mx / 7.0f;
  float inv = 7.0f / mx;
  for (int s = 0; s < n_samples; ++s) {
    uint8_t* out = codes + plane * (size_t)s;
    for (size_t i = 0; i < n; ++i) {
      float y = fabsf(x[i]) * inv;
      if (y != y) y = 0.0f;          /* NaN element -> 0 */
      if (y > 7.0f) y = 7.0f;
      float l = floorf(y);
      float frac = y - l;            /* exact: same binade or below, l <= y */
      uint32_t r = oracle_random_word(seed, (uint32_t)s, (uint64_t)i);
      int m = (int)l + (r < (uint32_t)(frac * 4294967296.0f) ? 1 : 0);
      int q = (bits_of(x[i]) >> 31) ? -m : m;
      out[i >> 1] |= (uint8_t)((q & 0xF) << ((i & 1) * 4));
    }
  }
  return s7;
}

/* ------------------------------------------------------------------------ */
/* Power-of-two LUQ (Appendix A.7): alpha_PW2 = 2^ceil(log2 max|x|) / 2^kmax. */
/* The maximum is rounded UP to a power of two (so nothing is clipped), the   */
/* quantizer itself is unchanged; every level is then a power of two.         */
/* ------------------------------------------------------------------------ */
float oracle_pw2_ceil(float mx) {
  if (!(mx > 0.0f) || !(mx <= 3.402823466e38f)) return mx; /* 0, NaN, Inf pass through */
  int e;
  float m = frexpf(mx, &e); /* mx = m * 2^e, m in [0.5, 1) */
  return (m == 0.5f) ? mx : ldexpf(1.0f, e);
}

/* ------------------------------------------------------------------------ */
/* In-hindsight maximum (Sec. 7 "Reducing the data movement", Appendix A.5.4): */
/*   m_hat^t = (1 - eta) * max|x^(t-1)| + eta * m_hat^(t-1),  eta = 0.1 in the */
/* paper's runs.  Tensor t is quantized with m_hat^t (values above it clip to  */
/* the top level) while its own maximum is measured for step t+1.  Evaluated   */
/* in binary32, each operation rounded once.                                   */
/* Reading where the paper is silent (it assumes finite tensors and a running  */
/* estimate that already exists): a measurement that is not finite (an Inf or  */
/* NaN element) carries no information about the range and leaves the estimate */
/* as it was, otherwise one overflowed element would make every later estimate */
/* Inf; an estimate that is itself not a positive finite number (0 before the  */
/* first step, or Inf/NaN handed in) has no history to blend with and is       */
/* replaced by the measurement.                                                */
/* ------------------------------------------------------------------------ */
float oracle_hindsight_next(float measured_max, float m_hat, float eta) {
  if (!(measured_max <= 3.402823466e38f)) return m_hat;              /* NaN or Inf measured */
  if (!(m_hat > 0.0f) || !(m_hat <= 3.402823466e38f)) return measured_max; /* no usable history */
  float keep = 1.0f - eta;
  float a = keep * measured_max;
  float b = eta * m_hat;
  return a + b;
}

/* Exact-expectation helper (test only): per element the two candidate levels
 * (as multiples of alpha: 0, 1, 2, 4, ...) and the 32-bit threshold, so that
 * E[Q(x)] = alpha*(lo + (hi-lo)*thr/2^32) can be evaluated without sampling. */
void oracle_luq_bins(const float* x, size_t n, float mx, int kmax,
                     double* lo, double* hi, uint32_t* thr) {
  float alpha = oracle_luq_alpha(mx, kmax);
  for (size_t i = 0; i < n; ++i) {
    luq_bin b = luq_bin_of(fabsf(x[i]), alpha, kmax);
    uint32_t c = b.lo_code;
    lo[i] = c ? ldexp(1.0, (int)c - 1) : 0.0;
    hi[i] = ((int)c >= kmax + 1) ? lo[i] : ldexp(1.0, (int)c);
    thr[i] = b.threshold;
  }
}

double oracle_luq_value(uint8_t nibble) { /* in units of alpha */
  int c = nibble & 7;
  if (c == 0) return 0.0;
  double v = ldexp(1.0, c - 1);
  return (nibble & 8) ? -v : v;
}

/* ------------------------------------------------------------------------ */
/* Dequantise and multiply (Eqs. Forward / Backward / Update on quantized     */
/* tensors).  Appendix A.1: a quantized tensor is ONE high-precision scale    */
/* times low-precision values, and "all MACs act on the low-precision values": */
/*   out = (s_x * s_y) * sum_k v_x[k] * v_y[k]                                 */
/* with v the integer-valued codes (INT4: q; LUQ: +-2^(c-1); unsigned: nibble). */
/* The sum is formed in double over those integers - exact below 2^53, so an   */
/* output whose products cancel is exactly 0 - and the scale product is        */
/* applied once.  SMP (Sec. 5.1) averages the RESULTS of the n_s samples: the   */
/* samples' products are added and the sum is divided by n_s at the end.        */
/* kind: 0 = INT4 codes (value q*scale), 1 = LUQ codes (value +-scale*2^(c-1)),  */
/*       2 = unsigned INT4 codes (value nibble*scale)                            */
/* ------------------------------------------------------------------------ */
static double code_value(const uint8_t* codes, size_t idx, int kind) {
  uint8_t nib = (codes[idx >> 1] >> ((idx & 1) * 4)) & 0xF;
  if (kind == 2) return (double)nib;
  return kind ? oracle_luq_value(nib) : (double)oracle_int4_value(nib);
}

void oracle_dequant(const uint8_t* codes, size_t n, double scale, int kind, double* out) {
  for (size_t i = 0; i < n; ++i) out[i] = scale * code_value(codes, i, kind);
}

/* the low-precision values of a packed tensor, as doubles (unit scale) */
static double* code_values(const uint8_t* codes, size_t n, int kind) {
  double* v = (double*)malloc(sizeof(double) * (n ? n : 1));
  for (size_t i = 0; i < n; ++i) v[i] = code_value(codes, i, kind);
  return v;
}

/* Z[M x N] = (sa*sw) * A_v . W_v^T, A_v / W_v the values of the A codes [M x K] / W codes [N x K] */
void oracle_gemm_fwd(const uint8_t* a_codes, double sa, const uint8_t* w_codes, double sw,
                     int64_t M, int64_t N, int64_t K, double* Z) {
  double* Av = code_values(a_codes, (size_t)(M * K), 0);
  double* Wv = code_values(w_codes, (size_t)(N * K), 0);
  const double scale = sa * sw;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      double acc = 0.0;
      for (int64_t k = 0; k < K; ++k) acc += Av[m * K + k] * Wv[n * K + k];
      Z[m * N + n] = scale * acc;
    }
  free(Av); free(Wv);
}

/* dA[M x K] = (alpha*sw) * (sum_s G_v,s . W_v) / n_s */
void oracle_gemm_bwd(const uint8_t* g_codes, double alpha, int n_samples,
                     const uint8_t* w_codes, double sw,
                     int64_t M, int64_t N, int64_t K, double* dA) {
  size_t gn = (size_t)(M * N), plane = (gn + 1) / 2;
  double** Gv = (double**)malloc(sizeof(double*) * (size_t)n_samples);
  for (int s = 0; s < n_samples; ++s) Gv[s] = code_values(g_codes + plane * (size_t)s, gn, 1);
  double* Wv = code_values(w_codes, (size_t)(N * K), 0);
  const double scale = alpha * sw;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t k = 0; k < K; ++k) {
      double acc = 0.0;
      for (int s = 0; s < n_samples; ++s)
        for (int64_t n = 0; n < N; ++n) acc += Gv[s][m * N + n] * Wv[n * K + k];
      dA[m * K + k] = scale * acc / (double)n_samples;
    }
  for (int s = 0; s < n_samples; ++s) free(Gv[s]);
  free(Gv); free(Wv);
}

/* dW[N x K] = (alpha*sa) * (sum_s G_v,s^T . A_v) / n_s  (Sec. 5.1: the average of the samples' weight gradients) */
void oracle_gemm_wgrad(const uint8_t* g_codes, double alpha, int n_samples,
                       const uint8_t* a_codes, double sa,
                       int64_t M, int64_t N, int64_t K, double* dW) {
  size_t gn = (size_t)(M * N), plane = (gn + 1) / 2;
  double** Gv = (double**)malloc(sizeof(double*) * (size_t)n_samples);
  for (int s = 0; s < n_samples; ++s) Gv[s] = code_values(g_codes + plane * (size_t)s, gn, 1);
  double* Av = code_values(a_codes, (size_t)(M * K), 0);
  const double scale = alpha * sa;
#pragma omp parallel for schedule(static)
  for (int64_t n = 0; n < N; ++n)
    for (int64_t k = 0; k < K; ++k) {
      double acc = 0.0;
      for (int s = 0; s < n_samples; ++s)
        for (int64_t m = 0; m < M; ++m) acc += Gv[s][m * N + n] * Av[m * K + k];
      dW[n * K + k] = scale * acc / (double)n_samples;
    }
  for (int s = 0; s < n_samples; ++s) free(Gv[s]);
  free(Gv); free(Av);
}

/* The same three products for operands of any code kind (the unsigned INT4 activations of
 * Appendix "Quantization formats", the INT4 gradient codes of the ablation's uniform arm):
 * which 0 fwd  out[M x N] = (sx*sy)   sum_k   x[m,k] y[n,k]        x = activations, y = weights
 *       1 bwd  out[M x K] = (sx*sy)/ns sum_s,n x_s[m,n] y[n,k]     x = gradient planes, y = weights
 *       2 wgrad out[N x K] = (sx*sy)/ns sum_s,m x_s[m,n] y[m,k]    x = gradient planes, y = activations */
void oracle_gemm_general(int which, const uint8_t* x_codes, int x_kind, double sx, int n_samples,
                         const uint8_t* y_codes, int y_kind, double sy,
                         int64_t M, int64_t N, int64_t K, double* out) {
  const double scale = sx * sy;
  if (which == 0) {
    double* Xv = code_values(x_codes, (size_t)(M * K), x_kind);
    double* Yv = code_values(y_codes, (size_t)(N * K), y_kind);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
      for (int64_t n = 0; n < N; ++n) {
        double acc = 0.0;
        for (int64_t k = 0; k < K; ++k) acc += Xv[m * K + k] * Yv[n * K + k];
        out[m * N + n] = scale * acc;
      }
    free(Xv); free(Yv);
    return;
  }
  size_t gn = (size_t)(M * N), plane = (gn + 1) / 2;
  double** Gv = (double**)malloc(sizeof(double*) * (size_t)n_samples);
  for (int s = 0; s < n_samples; ++s) Gv[s] = code_values(x_codes + plane * (size_t)s, gn, x_kind);
  if (which == 1) {
    double* Wv = code_values(y_codes, (size_t)(N * K), y_kind);
#pragma omp parallel for schedule(static)
    for (int64_t m = 0; m < M; ++m)
      for (int64_t k = 0; k < K; ++k) {
        double acc = 0.0;
        for (int s = 0; s < n_samples; ++s)
          for (int64_t n = 0; n < N; ++n) acc += Gv[s][m * N + n] * Wv[n * K + k];
        out[m * K + k] = scale * acc / (double)n_samples;
      }
    free(Wv);
  } else {
    double* Av = code_values(y_codes, (size_t)(M * K), y_kind);
#pragma omp parallel for schedule(static)
    for (int64_t n = 0; n < N; ++n)
      for (int64_t k = 0; k < K; ++k) {
        double acc = 0.0;
        for (int s = 0; s < n_samples; ++s)
          for (int64_t m = 0; m < M; ++m) acc += Gv[s][m * N + n] * Av[m * K + k];
        out[n * K + k] = scale * acc / (double)n_samples;
      }
    free(Av);
  }
  for (int s = 0; s < n_samples; ++s) free(Gv[s]);
  free(Gv);
}

/* The same sums in integer arithmetic (a cross-check of the double sums above):
 * the values are multiplied and summed in int64.
 * which: 0 fwd, 1 bwd, 2 wgrad.  out gets the integer sums (not yet scaled,
 * summed over the n_samples planes). */
void oracle_gemm_int64(int which, const uint8_t* x_codes, int n_samples, const uint8_t* y_codes,
                       int64_t M, int64_t N, int64_t K, int64_t* out) {
  if (which == 0) {
    for (int64_t m = 0; m < M; ++m)
      for (int64_t n = 0; n < N; ++n) {
        int64_t acc = 0;
        for (int64_t k = 0; k < K; ++k)
          acc += (int64_t)code_value(x_codes, (size_t)(m * K + k), 0) *
                 (int64_t)code_value(y_codes, (size_t)(n * K + k), 0);
        out[m * N + n] = acc;
      }
    return;
  }
  size_t plane = ((size_t)(M * N) + 1) / 2;
  if (which == 1) {
    for (int64_t m = 0; m < M; ++m)
      for (int64_t k = 0; k < K; ++k) {
        int64_t acc = 0;
        for (int s = 0; s < n_samples; ++s)
          for (int64_t n = 0; n < N; ++n)
            acc += (int64_t)code_value(x_codes + plane * (size_t)s, (size_t)(m * N + n), 1) *
                   (int64_t)code_value(y_codes, (size_t)(n * K + k), 0);
        out[m * K + k] = acc;
      }
  } else {
    for (int64_t n = 0; n < N; ++n)
      for (int64_t k = 0; k < K; ++k) {
        int64_t acc = 0;
        for (int s = 0; s < n_samples; ++s)
          for (int64_t m = 0; m < M; ++m)
            acc += (int64_t)code_value(x_codes + plane * (size_t)s, (size_t)(m * N + n), 1) *
                   (int64_t)code_value(y_codes, (size_t)(m * K + k), 0);
        out[n * K + k] = acc;
      }
  }
}

/* Selected output entries of the three products at any size, computed one by
 * one from the codes (same definition as above: the values' products added in
 * double, one scale product, the samples' sum divided by n_s at the end).  which: 0 fwd (r=m, c=n), 1 bwd (r=m, c=k), 2 wgrad (r=n, c=k). */
void oracle_gemm_entries(int which, const uint8_t* x_codes, double sx, int n_samples,
                         const uint8_t* y_codes, double sy,
                         int64_t M, int64_t N, int64_t K,
                         const int64_t* rows, const int64_t* cols, size_t count, double* out) {
  size_t plane = ((size_t)(M * N) + 1) / 2;
#pragma omp parallel for schedule(dynamic, 4)
  for (size_t e = 0; e < count; ++e) {
    int64_t r = rows[e], c = cols[e];
    double acc = 0.0;
    if (which == 0) {
      for (int64_t k = 0; k < K; ++k)
        acc += code_value(x_codes, (size_t)(r * K + k), 0) * code_value(y_codes, (size_t)(c * K + k), 0);
    } else if (which == 1) {
      for (int s = 0; s < n_samples; ++s)
        for (int64_t n = 0; n < N; ++n)
          acc += code_value(x_codes + plane * (size_t)s, (size_t)(r * N + n), 1) *
                 code_value(y_codes, (size_t)(n * K + c), 0);
    } else {
      for (int s = 0; s < n_samples; ++s)
        for (int64_t m = 0; m < M; ++m)
          acc += code_value(x_codes + plane * (size_t)s, (size_t)(m * N + r), 1) *
                 code_value(y_codes, (size_t)(m * K + c), 0);
    }
    acc = (sx * sy) * acc / (double)n_samples;
    out[e] = acc;
  }
}

/* ------------------------------------------------------------------------ */
/* Deterministic rounding rules used as pins (Table 1, Sec. 3.1).            */
/* ------------------------------------------------------------------------ */
double oracle_round_nearest_in_bin(double x, double l, double u) { return (x - l <= u - x) ? l : u; }

/* exported for the bit-level tests */
uint32_t oracle_float_bits(float f) { return bits_of(f); }
float oracle_bits_float(uint32_t u) { return float_of(u); }
