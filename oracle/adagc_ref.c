/*
 * CPU oracle for AdamW with AdaGC (Algorithm 1 of the paper; Eq. 2, Eq. 3), in plain C.
 *
 * TEST INFRASTRUCTURE ONLY: a slow, float64, per-tensor restatement of the paper's
 * algorithm for checking the CUDA library at sizes where the numpy oracle is too slow.
 * It shares no code, header or table with the CUDA path and is never a fallback for it.
 *
 * Arithmetic: every per-element and per-tensor quantity is float64; the sum of squares of a
 * tensor is accumulated sequentially, in element order, in long double.  Stored state
 * (theta, m, v, gamma) is fp32 and is rounded once per step on store.  OpenMP, if enabled,
 * only distributes whole tensors (norms) or independent elements (update) over threads; it
 * never changes the order of a reduction.
 *
 * Readings of the paper (same as the numpy oracle): 1-based step; warm-up = steps
 * 1..T_start with global-norm clipping (Eq. 2) and min-seeding of gamma from the clipped
 * per-tensor norms; at step 1 the incoming gamma is ignored; strict ">" activates the clip and
 * the clipped norm is then lambda_rel * gamma itself (Section 4.2).
 *
 * Parity pins: tests/test_oracle_pins.py runs the same pins against this file and the numpy oracle.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC adagc_ref.c -o libadagc_ref.so -lm
 */
#include <math.h>
#include <stdint.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static inline double bf16_to_double(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* Round a double to the nearest bfloat16 (ties to even), from the format's definition:
 * 8 exponent bits with bias 127, 7 stored mantissa bits, subnormals below 2^-126. */
static uint16_t double_to_bf16(double x) {
  float f;
  uint32_t u;
  if (isnan(x)) return 0x7fc0;
  if (isinf(x) || x == 0.0) {
    f = (float)x;
    memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
  }
  int e;
  (void)frexp(x, &e); /* |x| = frac * 2^e, frac in [0.5, 1)  ->  floor(log2|x|) = e - 1 */
  int p = e - 1;
  if (p < -126) p = -126;
  double q = ldexp(x, 7 - p);  /* exact power-of-two scaling; |q| < 2^8 */
  double r = nearbyint(q);     /* round to nearest, ties to even (default rounding mode) */
  double y = ldexp(r, p - 7);  /* representable in bf16 unless it overflows */
  f = (float)y;                /* exact, or +-inf on overflow beyond the fp32 range */
  memcpy(&u, &f, 4);
  if ((u & 0x7f800000u) == 0x7f800000u) return (uint16_t)((u >> 16) & 0xff80);
  return (uint16_t)(u >> 16);
}

int adagc_ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

uint16_t adagc_ref_double_to_bf16(double x) { return double_to_bf16(x); }

/* sum_j g_j^2 of one tensor (the square of the norm in Eq. 3). */
double adagc_ref_sumsq(const void* g, int is_bf16, int64_t n) {
  long double acc = 0.0L;
  if (is_bf16) {
    const uint16_t* p = (const uint16_t*)g;
    for (int64_t j = 0; j < n; ++j) {
      double x = bf16_to_double(p[j]);
      acc += (long double)(x * x);
    }
  } else {
    const float* p = (const float*)g;
    for (int64_t j = 0; j < n; ++j) {
      double x = (double)p[j];
      acc += (long double)(x * x);
    }
  }
  return (double)acc;
}

/* Sums of squares of T tensors that live at element offsets off[i] of one arena. */
void adagc_ref_sumsq_tensors(const void* arena, int is_bf16, int32_t T, const int64_t* off,
                             const int64_t* numel, double* s_out) {
  const char* base = (const char*)arena;
  const int64_t esz = is_bf16 ? 2 : 4;
#pragma omp parallel for schedule(dynamic, 1)
  for (int32_t i = 0; i < T; ++i) s_out[i] = adagc_ref_sumsq(base + off[i] * esz, is_bf16, numel[i]);
}

/*
 * Clip factors, flags and the EMA update of one step (Algorithm 1: the warm-up branch with
 * Eq. 2, or the AdaGC branch with Eq. 3).  gamma is fp32 state, updated in place.
 * Outputs per tensor: norm, h, flag, clipped norm, decision margin |norm - thr| / thr.
 */
void adagc_ref_clip_decisions_ex(int32_t T, const double* s, float* gamma, int64_t step,
                                 double lambda_rel, double beta, double lambda_abs, int64_t warmup,
                                 int variant, double* norm, double* h, uint8_t* flag, double* clipped,
                                 double* margin, double* global_norm);

void adagc_ref_clip_decisions(int32_t T, const double* s, float* gamma, int64_t step,
                              double lambda_rel, double beta, double lambda_abs, int64_t warmup,
                              double* norm, double* h, uint8_t* flag, double* clipped,
                              double* margin, double* global_norm) {
  adagc_ref_clip_decisions_ex(T, s, gamma, step, lambda_rel, beta, lambda_abs, warmup, 0, norm, h, flag,
                              clipped, margin, global_norm);
}

/* The same with the ablation variants of the paper's Section 5 (bits of `variant`):
 *   1  keep the caller's gamma_0: no seeding at t = 1 ("constant initialization");
 *   2  "Global AdaGC": one adaptive threshold for the whole model = this algorithm on the single tensor
 *      that all gradients form together; every tensor gets that clip factor, flag and gamma;
 * and, with gamma_cap > 0, "thresholded initialization" (EMA Initialization Strategy, variant 3): wherever the
 * default seeds gamma or takes the running minimum, gamma_t,i = min(||hat(g)_t,i||, gamma_cap) instead -- the
 * constant takes the place of gamma_t-1,i, so nothing is carried from one warm-up step to the next. */
void adagc_ref_clip_decisions_cap(int32_t T, const double* s, float* gamma, int64_t step,
                                  double lambda_rel, double beta, double lambda_abs, int64_t warmup,
                                  int variant, double gamma_cap, double* norm, double* h, uint8_t* flag,
                                  double* clipped, double* margin, double* global_norm) {
  const int seed = (step == 1) && !(variant & 1);
  const int capped = gamma_cap > 0.0;
  long double tot = 0.0L;
  for (int32_t i = 0; i < T; ++i) {
    norm[i] = sqrt(s[i]);
    tot += (long double)s[i];
  }
  const double G = sqrt((double)tot); /* ||g_t|| */
  *global_norm = G;
  if (variant & 2) {
    double s1 = (double)tot, n1, h1, c1, m1, G1;
    uint8_t f1;
    float g1 = gamma[0];
    adagc_ref_clip_decisions_cap(1, &s1, &g1, step, lambda_rel, beta, lambda_abs, warmup, variant & 1, gamma_cap,
                                 &n1, &h1, &f1, &c1, &m1, &G1);
    for (int32_t i = 0; i < T; ++i) {
      h[i] = h1;
      flag[i] = f1;
      clipped[i] = h1 * norm[i];
      margin[i] = m1;
      gamma[i] = g1;
    }
    return;
  }
  if (step <= warmup) {
    const int clip_all = G > lambda_abs;
    const double h_t = clip_all ? lambda_abs / G : 1.0; /* min{lambda_abs/||g_t||, 1} */
    for (int32_t i = 0; i < T; ++i) {
      h[i] = h_t;
      flag[i] = (uint8_t)clip_all;
      clipped[i] = h_t * norm[i]; /* ||hat(g)_t,i|| */
      margin[i] = lambda_abs > 0 ? fabs(G - lambda_abs) / lambda_abs : INFINITY;
      double gprev = (double)gamma[i];
      double gnew;
      if (capped) gnew = clipped[i] < gamma_cap ? clipped[i] : gamma_cap;
      else gnew = seed ? clipped[i] : (clipped[i] < gprev ? clipped[i] : gprev);
      gamma[i] = (float)gnew;
    }
  } else {
    for (int32_t i = 0; i < T; ++i) {
      double gprev = seed ? (double)(float)norm[i] : (double)gamma[i];
      if (seed && capped && !(gprev < gamma_cap)) gprev = gamma_cap;
      const double thr = lambda_rel * gprev;
      margin[i] = thr > 0 ? fabs(norm[i] - thr) / thr : INFINITY;
      if (norm[i] > thr) {
        flag[i] = 1;
        h[i] = thr / norm[i];
        clipped[i] = thr;
      } else {
        flag[i] = 0;
        h[i] = 1.0;
        clipped[i] = norm[i];
      }
      gamma[i] = (float)(beta * gprev + (1.0 - beta) * clipped[i]);
    }
  }
}

void adagc_ref_clip_decisions_ex(int32_t T, const double* s, float* gamma, int64_t step,
                                 double lambda_rel, double beta, double lambda_abs, int64_t warmup,
                                 int variant, double* norm, double* h, uint8_t* flag, double* clipped,
                                 double* margin, double* global_norm) {
  adagc_ref_clip_decisions_cap(T, s, gamma, step, lambda_rel, beta, lambda_abs, warmup, variant, 0.0, norm, h,
                               flag, clipped, margin, global_norm);
}

/* The four AdamW lines of Algorithm 1 on hat(g) = h * g for n elements, in place. */
void adagc_ref_adamw(float* theta, const void* g, int g_is_bf16, float* m, float* v, int64_t n,
                     double h, int64_t step, double lr, double beta1, double beta2, double eps,
                     double wd) {
  const double bc1 = 1.0 - pow(beta1, (double)step);
  const double bc2 = 1.0 - pow(beta2, (double)step);
  const uint16_t* gb = (const uint16_t*)g;
  const float* gf = (const float*)g;
#pragma omp parallel for schedule(static) if (n > 65536)
  for (int64_t j = 0; j < n; ++j) {
    const double gj = g_is_bf16 ? bf16_to_double(gb[j]) : (double)gf[j];
    const double gh = h * gj;
    const double m1 = beta1 * (double)m[j] + (1.0 - beta1) * gh;
    const double v1 = beta2 * (double)v[j] + (1.0 - beta2) * gh * gh;
    const double mh = m1 / bc1;
    const double vh = v1 / bc2;
    const double th = (double)theta[j];
    theta[j] = (float)(th - lr * wd * th - lr * mh / (sqrt(vh) + eps));
    m[j] = (float)m1;
    v[j] = (float)v1;
  }
}

/* Lion on hat(g) = h * g for n elements, in place (Section 4.2: AdaGC with other optimizers; Lion's
 * published rule: c = beta1 m + (1-beta1) g;  theta -= lr (sign(c) + wd theta);  m = beta2 m + (1-beta2) g).
 * sign(c) is a discrete decision: where the two terms of c nearly cancel, an implementation that rounds
 * differently may legitimately take the other sign.  If near_tie is not NULL, near_tie[j] is incremented
 * (saturating at 255) when |c| < tie_tol * (|beta1 m| + |(1-beta1) hat(g)|), so that a comparison can
 * tell such elements from real errors. */
void adagc_ref_lion(float* theta, const void* g, int g_is_bf16, float* m, int64_t n, double h, double lr,
                    double beta1, double beta2, double wd, uint8_t* near_tie, double tie_tol) {
  const uint16_t* gb = (const uint16_t*)g;
  const float* gf = (const float*)g;
#pragma omp parallel for schedule(static) if (n > 65536)
  for (int64_t j = 0; j < n; ++j) {
    const double gj = g_is_bf16 ? bf16_to_double(gb[j]) : (double)gf[j];
    const double gh = h * gj;
    const double mj = (double)m[j];
    const double a = beta1 * mj, b = (1.0 - beta1) * gh;
    const double c = a + b;
    const double sgn = (c > 0.0) - (c < 0.0);
    if (near_tie && fabs(c) < tie_tol * (fabs(a) + fabs(b)) && near_tie[j] < 255) near_tie[j] += 1;
    const double th = (double)theta[j];
    theta[j] = (float)(th - lr * (sgn + wd * th));
    m[j] = (float)(beta2 * mj + (1.0 - beta2) * gh);
  }
}

/* SGD with momentum on hat(g) = h * g, in place (Section 4.2: AdaGC with other optimizers): heavy-ball form
 * with L2 weight decay folded into the gradient: d = hat(g) + wd theta;  m = momentum m + d;  theta -= lr m. */
void adagc_ref_sgdm(float* theta, const void* g, int g_is_bf16, float* m, int64_t n, double h, double lr,
                    double momentum, double wd) {
  const uint16_t* gb = (const uint16_t*)g;
  const float* gf = (const float*)g;
#pragma omp parallel for schedule(static) if (n > 65536)
  for (int64_t j = 0; j < n; ++j) {
    const double gj = g_is_bf16 ? bf16_to_double(gb[j]) : (double)gf[j];
    const double th = (double)theta[j];
    const double d = h * gj + wd * th;
    const double m1 = momentum * (double)m[j] + d;
    theta[j] = (float)(th - lr * m1);
    m[j] = (float)m1;
  }
}

/*
 * Stochastic rounding of stored bfloat16 moments.  Random numbers: the counter-based generator Philox4x32-10 (Salmon,
 * Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3", SC 2011), from its definition: ten rounds, each
 * replacing the counter (c0, c1, c2, c3) by (hi(M1 c2) ^ c1 ^ k0, lo(M1 c2), hi(M0 c0) ^ c3 ^ k1, lo(M0 c0)); the key
 * is bumped by (W0, W1) between rounds.
 */
void adagc_ref_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1, n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1,
                   n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    if (r < 9) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The 16-bit random numbers of the element at arena position `index` at step `step`: elements 4q..4q+3 share the call
 * with counter (lo q, hi q, lo step, hi step) and key (lo seed, hi seed); element 4q + l takes output word l, the low
 * half for m (which = 0), the high half for v (which = 1). */
static uint32_t rounding_random(int64_t index, int64_t step, uint64_t seed, int which) {
  const uint64_t q = (uint64_t)index >> 2;
  const uint32_t ctr[4] = {(uint32_t)q, (uint32_t)(q >> 32), (uint32_t)step, (uint32_t)((uint64_t)step >> 32)};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t out[4];
  adagc_ref_philox4x32_10(ctr, key, out);
  const uint32_t w = out[index & 3];
  return which ? (w >> 16) : (w & 0xFFFFu);
}

/* Stochastic rounding of a float to bfloat16 with the 16-bit random integer r: the neighbour of larger magnitude is taken
 * with probability (distance to the smaller neighbour) / spacing -- add r to the low half of the bit pattern, drop that
 * half.  Infinities and NaN are rounded to nearest. */
static uint16_t float_to_bf16_stochastic(float x, uint32_t r) {
  if (isnan(x) || isinf(x)) return double_to_bf16((double)x);
  uint32_t u;
  memcpy(&u, &x, 4);
  return (uint16_t)((u + r) >> 16);
}

uint16_t adagc_ref_float_to_bf16_stochastic(float x, uint32_t r) { return float_to_bf16_stochastic(x, r); }

/* Distance from x to the nearest point where rounding to bfloat16 flips (the midpoint between two
 * neighbouring bfloat16 values): an implementation whose x differs by less than this rounds alike. */
static double bf16_flip_distance(double x) {
  if (!isfinite(x) || x == 0.0) return INFINITY;
  int e;
  (void)frexp(x, &e);
  int p = e - 1;
  if (p < -126) p = -126;
  double q = fabs(ldexp(x, 7 - p));
  double frac = q - floor(q);
  double dist = fabs(frac - 0.5); /* in units of the spacing 2^(p-7) */
  /* just above a power of two the values below are twice as dense: the flip below 2^p is a quarter spacing under it */
  if (floor(q) == 128.0 && p > -126 && frac + 0.25 < dist) dist = frac + 0.25;
  return dist * ldexp(1.0, p - 7);
}

static inline void count_near_tie(uint8_t* near_tie, int64_t j, double x, double scale, double tie_tol) {
  if (near_tie && bf16_flip_distance(x) < tie_tol * scale && near_tie[j] < 255) near_tie[j] += 1;
}

/*
 * The AdamW lines of Algorithm 1 with the moments STORED as bfloat16 (the paper trains in bfloat16 / float8
 * precision and does not say how optimizer state is rounded; reading taken: fp32 master theta, m and v read
 * exactly from their stored bfloat16, theta updated from the UNROUNDED new moments, the moments rounded to the
 * nearest bfloat16, ties to even, when stored).  In place.
 *
 * Rounding to bfloat16 is a discrete decision.  fp32_decision = 0: everything in float64 (the plain definition;
 * if near_tie is not NULL, near_tie[j] is incremented, saturating, whenever the new m or v lies within tie_tol,
 * relative to the terms it is summed from, of a point where the rounding flips).  fp32_decision = 1: the value
 * that is rounded to bfloat16 is evaluated in the precision the stored format is defined for, single precision,
 * in this order, every operation rounded once (fl = round to float, coefficients rounded to float first):
 *     gh = fl(h * g);   m' = fl(beta1 * m + fl((1 - beta1) * gh));   v' = fl(beta2 * v + fl((1 - beta2) * fl(gh * gh)))
 * (the sum and its first product are one fused multiply-add).  With bfloat16 m, bfloat16 g and beta1 = 0.9 the
 * float64 value of m' is an exact decimal tie (x.5 spacings) for about one element in twenty, so which neighbour is
 * stored depends on how the coefficients themselves are rounded: the decision has to name its precision.
 * theta is always computed in float64 from the float64 moments.
 * stochastic = 1 (with fp32_decision): the single-precision m' and v' are rounded stochastically instead, with the random
 * numbers of the element's arena position (index[j] if index is given, else index0 + j), `step` and `seed`.
 */
void adagc_ref_adamw_bf16state(float* theta, const void* g, int g_is_bf16, uint16_t* m, uint16_t* v, int64_t n,
                               double h, int64_t step, double lr, double beta1, double beta2, double eps,
                               double wd, uint8_t* near_tie, double tie_tol, int fp32_decision, int stochastic,
                               uint64_t seed, int64_t index0, const int64_t* index) {
  const double bc1 = 1.0 - pow(beta1, (double)step);
  const double bc2 = 1.0 - pow(beta2, (double)step);
  const uint16_t* gb = (const uint16_t*)g;
  const float* gf = (const float*)g;
  const float hf = (float)h, b1f = (float)beta1, omb1f = (float)(1.0 - beta1), b2f = (float)beta2,
              omb2f = (float)(1.0 - beta2);
#pragma omp parallel for schedule(static) if (n > 65536)
  for (int64_t j = 0; j < n; ++j) {
    const double gj = g_is_bf16 ? bf16_to_double(gb[j]) : (double)gf[j];
    const double gh = h * gj;
    const double a = beta1 * bf16_to_double(m[j]), b = (1.0 - beta1) * gh;
    const double m1 = a + b;
    const double v1 = beta2 * bf16_to_double(v[j]) + (1.0 - beta2) * gh * gh;
    const double mh = m1 / bc1;
    const double vh = v1 / bc2;
    const double th = (double)theta[j];
    theta[j] = (float)(th - lr * wd * th - lr * mh / (sqrt(vh) + eps));
    count_near_tie(near_tie, j, m1, fabs(a) + fabs(b), tie_tol);
    count_near_tie(near_tie, j, v1, v1, tie_tol);
    if (fp32_decision) {
      const float ghf = hf * (float)gj; /* g is exactly a float */
      const float m1f = fmaf(b1f, (float)bf16_to_double(m[j]), omb1f * ghf);
      const float v1f = fmaf(b2f, (float)bf16_to_double(v[j]), omb2f * (ghf * ghf));
      if (stochastic) { /* (only with fp32_decision: the rounding acts on the bits of the single-precision value) */
        const int64_t at = index ? index[j] : index0 + j; /* position of the element in the arenas */
        m[j] = float_to_bf16_stochastic(m1f, rounding_random(at, step, seed, 0));
        v[j] = float_to_bf16_stochastic(v1f, rounding_random(at, step, seed, 1));
      } else {
        m[j] = double_to_bf16((double)m1f);
        v[j] = double_to_bf16((double)v1f);
      }
    } else {
      m[j] = double_to_bf16(m1);
      v[j] = double_to_bf16(v1);
    }
  }
}

/* Lion (see adagc_ref_lion) with the momentum stored as bfloat16, rounded to nearest even on store.
 * near_tie counts both kinds of discrete decision: sign(c) and the rounding of m.  fp32_decision = 1: the stored
 * value is the rounding of  fl(beta2 * m + fl((1 - beta2) * fl(h * g)))  evaluated in single precision (see above);
 * sign(c) stays a float64 decision.  stochastic = 1: that value is rounded stochastically (random numbers of arena
 * position index0 + j, `step`, `seed`; the half of the word that AdamW uses for m). */
void adagc_ref_lion_bf16state(float* theta, const void* g, int g_is_bf16, uint16_t* m, int64_t n, double h,
                              double lr, double beta1, double beta2, double wd, uint8_t* near_tie,
                              double tie_tol, int fp32_decision, int stochastic, uint64_t seed, int64_t step,
                              int64_t index0) {
  const uint16_t* gb = (const uint16_t*)g;
  const float* gf = (const float*)g;
  const float hf = (float)h, b2f = (float)beta2, omb2f = (float)(1.0 - beta2);
#pragma omp parallel for schedule(static) if (n > 65536)
  for (int64_t j = 0; j < n; ++j) {
    const double gj = g_is_bf16 ? bf16_to_double(gb[j]) : (double)gf[j];
    const double gh = h * gj;
    const double mj = bf16_to_double(m[j]);
    const double a = beta1 * mj, b = (1.0 - beta1) * gh;
    const double c = a + b;
    const double sgn = (c > 0.0) - (c < 0.0);
    if (near_tie && fabs(c) < tie_tol * (fabs(a) + fabs(b)) && near_tie[j] < 255) near_tie[j] += 1;
    const double th = (double)theta[j];
    theta[j] = (float)(th - lr * (sgn + wd * th));
    const double a2 = beta2 * mj, b2 = (1.0 - beta2) * gh;
    if (fp32_decision) {
      const float m1f = fmaf(b2f, (float)mj, omb2f * (hf * (float)gj));
      m[j] = stochastic ? float_to_bf16_stochastic(m1f, rounding_random(index0 + j, step, seed, 0))
                        : double_to_bf16((double)m1f);
    } else {
      count_near_tie(near_tie, j, a2 + b2, fabs(a2) + fabs(b2), tie_tol);
      m[j] = double_to_bf16(a2 + b2);
    }
  }
}

/* Momentum SGD (see adagc_ref_sgdm) with the momentum stored as bfloat16; theta sees the unrounded momentum.
 * fp32_decision = 1: the stored value is the rounding of  fl(momentum * m + fl(wd * theta + fl(h * g)))  evaluated in
 * single precision (both sums fused multiply-adds). */
void adagc_ref_sgdm_bf16state(float* theta, const void* g, int g_is_bf16, uint16_t* m, int64_t n, double h,
                              double lr, double momentum, double wd, uint8_t* near_tie, double tie_tol,
                              int fp32_decision, int stochastic, uint64_t seed, int64_t step, int64_t index0) {
  const uint16_t* gb = (const uint16_t*)g;
  const float* gf = (const float*)g;
  const float hf = (float)h, muf = (float)momentum, wdf = (float)wd;
#pragma omp parallel for schedule(static) if (n > 65536)
  for (int64_t j = 0; j < n; ++j) {
    const double gj = g_is_bf16 ? bf16_to_double(gb[j]) : (double)gf[j];
    const double th = (double)theta[j];
    const double d = h * gj + wd * th;
    const double a = momentum * bf16_to_double(m[j]);
    const double m1 = a + d;
    const float m1f = fmaf(muf, (float)bf16_to_double(m[j]), fmaf(wdf, theta[j], hf * (float)gj));
    theta[j] = (float)(th - lr * m1);
    if (fp32_decision) {
      m[j] = stochastic ? float_to_bf16_stochastic(m1f, rounding_random(index0 + j, step, seed, 0))
                        : double_to_bf16((double)m1f);
    } else {
      count_near_tie(near_tie, j, m1, fabs(a) + fabs(h * gj) + fabs(wd * th), tie_tol);
      m[j] = double_to_bf16(m1);
    }
  }
}

/* hat(g) = h * g written in the gradient's dtype (clip-only use with other optimizers). */
void adagc_ref_scale(void* out, const void* g, int is_bf16, int64_t n, double h) {
  if (is_bf16) {
    const uint16_t* p = (const uint16_t*)g;
    uint16_t* o = (uint16_t*)out;
#pragma omp parallel for schedule(static) if (n > 65536)
    for (int64_t j = 0; j < n; ++j) o[j] = double_to_bf16(h * bf16_to_double(p[j]));
  } else {
    const float* p = (const float*)g;
    float* o = (float*)out;
#pragma omp parallel for schedule(static) if (n > 65536)
    for (int64_t j = 0; j < n; ++j) o[j] = (float)(h * (double)p[j]);
  }
}

/* One whole step of Algorithm 1 over T tensors laid out in shared arenas.
 * Stats outputs may be NULL.  Returns the number of tensors clipped. */
int32_t adagc_ref_step(int32_t T, const int64_t* off, const int64_t* numel, float* theta,
                       const void* grads, int g_is_bf16, float* m, float* v, float* gamma,
                       int64_t step, double lr, double beta1, double beta2, double eps, double wd,
                       double lambda_rel, double beta, double lambda_abs, int64_t warmup,
                       double* s_ws /* T */, double* norm, double* h, uint8_t* flag,
                       double* clipped, double* margin, double* global_norm) {
  adagc_ref_sumsq_tensors(grads, g_is_bf16, T, off, numel, s_ws);
  adagc_ref_clip_decisions(T, s_ws, gamma, step, lambda_rel, beta, lambda_abs, warmup, norm, h,
                           flag, clipped, margin, global_norm);
  const int64_t esz = g_is_bf16 ? 2 : 4;
  int32_t n_clipped = 0;
  for (int32_t i = 0; i < T; ++i) n_clipped += flag[i];
  /* large tensors one after another (threads split their elements) ... */
  for (int32_t i = 0; i < T; ++i) {
    if (numel[i] <= 65536) continue;
    adagc_ref_adamw(theta + off[i], (const char*)grads + off[i] * esz, g_is_bf16, m + off[i],
                    v + off[i], numel[i], h[i], step, lr, beta1, beta2, eps, wd);
  }
  /* ... small tensors distributed whole over the threads. */
#pragma omp parallel for schedule(dynamic, 16)
  for (int32_t i = 0; i < T; ++i) {
    if (numel[i] > 65536) continue;
    adagc_ref_adamw(theta + off[i], (const char*)grads + off[i] * esz, g_is_bf16, m + off[i],
                    v + off[i], numel[i], h[i], step, lr, beta1, beta2, eps, wd);
  }
  return n_clipped;
}
