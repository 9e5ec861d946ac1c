/*
 * bro_ref.c — CPU oracle (test infrastructure only; see bro_ref.h).
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 * -ffp-contract=off matters: every fp32 add/sub/mul below must be one IEEE round-to-nearest
 * operation, never fused.
 */
#include "bro_ref.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define MX_GROUP 32 /* Sec. 4.1: fixed group size of 32 */

/* E2M1 magnitudes for mag = 0..7: exponent field e = mag>>1 (bias 1), mantissa bit m = mag&1.
 * e == 0 is the subnormal binade (value m * 0.5); otherwise (1 + m/2) * 2^(e-1).  (Sec. 4.1) */
static const double E2M1_GRID[8] = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0};

int bro_ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void bro_ref_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

static inline float bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

static inline uint32_t f32_bits(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  return u;
}

static int is_pow2(int64_t v) { return v > 0 && (v & (v - 1)) == 0; }

float bro_ref_hadamard_norm(int64_t block) {
  /* 1/sqrt(B) for B = 2^p is 2^(-p/2): a power of two when p is even, sqrt(2) * 2^(-(p+1)/2)
   * when p is odd.  Rounding sqrt(2) to fp32 and scaling by a power of two is exact, so this
   * is the fp32 value nearest to 1/sqrt(B). */
  int p = 0;
  while (((int64_t)1 << p) < block) ++p;
  if ((p & 1) == 0) return ldexpf(1.0f, -p / 2);
  return ldexpf((float)sqrt(2.0), -(p + 1) / 2);
}

/* One block: v <- H_B v (Sylvester / natural order) by the fast transform, ascending stride.
 * Every a+b and a-b is a single fp32 round-to-nearest operation. */
static void fwht_block(float* v, int64_t B) {
  for (int64_t h = 1; h < B; h <<= 1) {
    for (int64_t i = 0; i < B; ++i) {
      if ((i & h) == 0) {
        float a = v[i];
        float b = v[i + h];
        v[i] = a + b;
        v[i + h] = a - b;
      }
    }
  }
}

int bro_ref_rotate_rs(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, int block,
                      const uint16_t* signs, float* y) {
  if (!x || !y) return 1;
  if (M < 0 || K <= 0 || ldx < K) return 2;
  int64_t B = block == 0 ? K : block;
  if (!is_pow2(B) || K % B != 0) return 2;
  const float c = bro_ref_hadamard_norm(B);
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m) {
    float* row = y + m * K;
    for (int64_t k = 0; k < K; ++k) {
      float v = bf16_to_f32(x[m * ldx + k]);
      /* x diag(s): channel k is negated where s_k = -1 (exact) */
      if (signs && (signs[k] & 0x8000u)) v = -v;
      row[k] = v;
    }
    for (int64_t b0 = 0; b0 < K; b0 += B) {
      fwht_block(row + b0, B);
      for (int64_t i = 0; i < B; ++i) row[b0 + i] = row[b0 + i] * c; /* one multiply, at the end */
    }
  }
  return 0;
}

int bro_ref_rotate(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, int block, float* y) {
  return bro_ref_rotate_rs(x, M, K, ldx, block, NULL, y);
}

/* Round a non-negative scaled magnitude r onto the E2M1 grid, nearest, ties to the even code,
 * saturating at 6 (mag 7). */
static inline unsigned e2m1_round(float r) {
  if (r <= 0.25f) return 0; /* tie .25 -> 0   (even) */
  if (r < 0.75f) return 1;
  if (r <= 1.25f) return 2; /* ties .75, 1.25 -> 1.0 (even) */
  if (r < 1.75f) return 3;
  if (r <= 2.5f) return 4; /* ties 1.75, 2.5 -> 2.0 (even) */
  if (r < 3.5f) return 5;
  if (r <= 5.0f) return 6; /* ties 3.5, 5 -> 4.0 (even) */
  return 7;                /* (5, inf): 6.0, saturating */
}

static void quantize_group(const float* y, uint8_t* codes16, uint8_t* scale) {
  float amax = 0.0f;
  for (int i = 0; i < MX_GROUP; ++i) {
    float a = fabsf(y[i]);
    if (a > amax) amax = a;
  }
  /* floor(log2(amax)) for a normal fp32 is its biased exponent field minus 127.  The shared
   * exponent is that minus emax_elem (= 2 for E2M1), clamped below at the smallest E8M0 value. */
  int ef = (int)((f32_bits(amax) >> 23) & 0xFF);
  int s = ef - 2;
  if (s < 0) s = 0;
  int E = s - 127;
  *scale = (uint8_t)s;
  for (int i = 0; i < MX_GROUP; i += 2) {
    unsigned c[2];
    for (int j = 0; j < 2; ++j) {
      float v = y[i + j];
      float r = ldexpf(fabsf(v), -E); /* exact power-of-two scaling */
      unsigned mag = e2m1_round(r);
      unsigned sign = (f32_bits(v) >> 31) & 1u;
      c[j] = (sign << 3) | mag;
    }
    codes16[i / 2] = (uint8_t)(c[0] | (c[1] << 4));
  }
}

int bro_ref_quantize(const float* y, int64_t rows, int64_t K, uint8_t* codes, uint8_t* scales) {
  if (!y || !codes || !scales) return 1;
  if (rows < 0 || K <= 0 || K % MX_GROUP != 0) return 2;
  const int64_t ng = K / MX_GROUP;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t g = 0; g < ng; ++g)
      quantize_group(y + r * K + g * MX_GROUP, codes + r * (K / 2) + g * (MX_GROUP / 2),
                     scales + r * ng + g);
  return 0;
}

static inline double decode_one(unsigned code, int E) {
  double v = ldexp(E2M1_GRID[code & 7u], E);
  return (code & 8u) ? -v : v;
}

int bro_ref_decode(const uint8_t* codes, const uint8_t* scales, int64_t rows, int64_t K,
                   double* out) {
  if (!codes || !scales || !out) return 1;
  if (rows < 0 || K <= 0 || K % MX_GROUP != 0) return 2;
  const int64_t ng = K / MX_GROUP;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t k = 0; k < K; ++k) {
      uint8_t byte = codes[r * (K / 2) + k / 2];
      unsigned code = (k & 1) ? (byte >> 4) : (byte & 0xF);
      int E = (int)scales[r * ng + k / MX_GROUP] - 127;
      out[r * K + k] = decode_one(code, E);
    }
  return 0;
}

int bro_ref_rotate_quantize_mxfp4_rs(const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                                     int block, const uint16_t* signs, uint8_t* codes,
                                     uint8_t* scales) {
  if (!x || !codes || !scales) return 1;
  if (M < 0 || K <= 0 || K % MX_GROUP != 0) return 2;
  if (M == 0) return 0;
  float* y = (float*)malloc((size_t)M * (size_t)K * sizeof(float));
  if (!y) return 3;
  int rc = bro_ref_rotate_rs(x, M, K, ldx, block, signs, y);
  if (rc == 0) rc = bro_ref_quantize(y, M, K, codes, scales);
  free(y);
  return rc;
}

int bro_ref_rotate_quantize_mxfp4(const uint16_t* x, int64_t M, int64_t K, int64_t ldx,
                                  int block, uint8_t* codes, uint8_t* scales) {
  return bro_ref_rotate_quantize_mxfp4_rs(x, M, K, ldx, block, NULL, codes, scales);
}

int bro_ref_pack_weights(const uint16_t* w, int64_t N, int64_t K, int64_t ldw, int block,
                         uint8_t* wcodes, uint8_t* wscales) {
  /* "Weights are rotated and quantised the same way": rows of W are output channels, the
   * rotation acts on the K axis exactly as for activations (R_block R_block^T = I, Eq. 1). */
  return bro_ref_rotate_quantize_mxfp4(w, N, K, ldw, block, wcodes, wscales);
}

int bro_ref_gemm_mxfp4(const uint8_t* acodes, const uint8_t* ascales, const uint8_t* wcodes,
                       const uint8_t* wscales, int64_t M, int64_t N, int64_t K, double* y,
                       double* S) {
  if (!acodes || !ascales || !wcodes || !wscales || !y) return 1;
  if (M < 0 || N < 0 || K <= 0 || K % MX_GROUP != 0) return 2;
  if (M == 0 || N == 0) return 0;
  double* A = (double*)malloc((size_t)M * (size_t)K * sizeof(double));
  double* W = (double*)malloc((size_t)N * (size_t)K * sizeof(double));
  if (!A || !W) {
    free(A);
    free(W);
    return 3;
  }
  bro_ref_decode(acodes, ascales, M, K, A);
  bro_ref_decode(wcodes, wscales, N, K, W);
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t n = 0; n < N; ++n) {
      double acc = 0.0, sabs = 0.0;
      for (int64_t k = 0; k < K; ++k) {
        double p = A[m * K + k] * W[n * K + k]; /* exact in fp64 */
        acc += p;
        sabs += fabs(p);
      }
      y[m * N + n] = acc;
      if (S) S[m * N + n] = sabs;
    }
  free(A);
  free(W);
  return 0;
}

int bro_ref_gemm_mxfp4_points(const uint8_t* acodes, const uint8_t* ascales,
                              const uint8_t* wcodes, const uint8_t* wscales, int64_t M,
                              int64_t N, int64_t K, const int64_t* pm, const int64_t* pn,
                              int64_t npoints, double* y, double* S) {
  if (!acodes || !ascales || !wcodes || !wscales || !pm || !pn || !y) return 1;
  if (M <= 0 || N <= 0 || K <= 0 || K % MX_GROUP != 0 || npoints < 0) return 2;
  const int64_t ng = K / MX_GROUP;
  for (int64_t p = 0; p < npoints; ++p)
    if (pm[p] < 0 || pm[p] >= M || pn[p] < 0 || pn[p] >= N) return 2;
#pragma omp parallel for schedule(static)
  for (int64_t p = 0; p < npoints; ++p) {
    const int64_t m = pm[p], n = pn[p];
    double acc = 0.0, sabs = 0.0;
    for (int64_t k = 0; k < K; ++k) {
      uint8_t ab = acodes[m * (K / 2) + k / 2];
      uint8_t wb = wcodes[n * (K / 2) + k / 2];
      unsigned ac = (k & 1) ? (ab >> 4) : (ab & 0xF);
      unsigned wc = (k & 1) ? (wb >> 4) : (wb & 0xF);
      double a = decode_one(ac, (int)ascales[m * ng + k / MX_GROUP] - 127);
      double w = decode_one(wc, (int)wscales[n * ng + k / MX_GROUP] - 127);
      double prod = a * w;
      acc += prod;
      sabs += fabs(prod);
    }
    y[p] = acc;
    if (S) S[p] = sabs;
  }
  return 0;
}

int bro_ref_linear(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, int block,
                   const uint8_t* wcodes, const uint8_t* wscales, int64_t N, double* y,
                   double* S) {
  if (!x || !wcodes || !wscales || !y) return 1;
  if (M < 0 || N < 0 || K <= 0 || K % MX_GROUP != 0) return 2;
  if (M == 0 || N == 0) return 0;
  uint8_t* ac = (uint8_t*)malloc((size_t)M * (size_t)(K / 2));
  uint8_t* as = (uint8_t*)malloc((size_t)M * (size_t)(K / MX_GROUP));
  if (!ac || !as) {
    free(ac);
    free(as);
    return 3;
  }
  int rc = bro_ref_rotate_quantize_mxfp4(x, M, K, ldx, block, ac, as);
  if (rc == 0) rc = bro_ref_gemm_mxfp4(ac, as, wcodes, wscales, M, N, K, y, S);
  free(ac);
  free(as);
  return rc;
}

int bro_ref_group_mse(const float* y, const uint8_t* codes, const uint8_t* scales,
                      int64_t rows, int64_t K, double* mse) {
  if (!y || !codes || !scales || !mse) return 1;
  if (rows < 0 || K <= 0 || K % MX_GROUP != 0) return 2;
  const int64_t ng = K / MX_GROUP;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t g = 0; g < ng; ++g) {
      int E = (int)scales[r * ng + g] - 127;
      double acc = 0.0;
      for (int i = 0; i < MX_GROUP; ++i) {
        int64_t k = g * MX_GROUP + i;
        uint8_t byte = codes[r * (K / 2) + k / 2];
        unsigned code = (k & 1) ? (byte >> 4) : (byte & 0xF);
        double d = (double)y[r * K + k] - decode_one(code, E);
        acc += d * d;
      }
      mse[r * ng + g] = acc / MX_GROUP;
    }
  return 0;
}

/* ---- comparison formats (analysis only) -------------------------------------------------------- */

/* fp32 -> nearest-even fp16 value, returned as a float; clamped to the largest finite fp16. */
static float round_to_fp16(float f) {
  if (!(f == f)) return f;
  float a = fabsf(f);
  if (a >= 65520.0f) a = 65504.0f; /* would round to infinity: saturate */
  else if (a < 6.103515625e-05f) { /* below 2^-14: fp16 subnormals, spacing 2^-24 */
    a = (float)(rint((double)a * 16777216.0) / 16777216.0);
  } else {
    int e;
    (void)frexpf(a, &e); /* a = m * 2^e, m in [0.5, 1): 11 significant bits -> spacing 2^(e-11) */
    double q = ldexp(1.0, e - 11);
    a = (float)(rint((double)a / q) * q);
  }
  return f < 0 ? -a : a;
}

/* INT4 with one scale per ROW (Sec. 3.2 / Fig. 2: "INT4 — weight per-channel symmetric quantization with
 * per-token asymmetric activation quantization"): format 4 is the symmetric form (a row of W is an output
 * channel), format 5 the asymmetric form (a row of X is a token). */
static void int4_row(const float* v, int64_t K, int asym, double* out) {
  if (!asym) {
    float amax = 0.0f;
    for (int64_t i = 0; i < K; ++i)
      if (fabsf(v[i]) > amax) amax = fabsf(v[i]);
    const float sc = round_to_fp16(amax / 7.0f);
    for (int64_t i = 0; i < K; ++i) {
      if (sc == 0.0f) { out[i] = 0.0; continue; }
      double q = rint((double)(fabsf(v[i]) / sc)); /* fp32 division, ties to even */
      if (q > 7.0) q = 7.0;
      q *= (double)sc;
      out[i] = (f32_bits(v[i]) >> 31) ? -q : q;
    }
    return;
  }
  /* the range always contains zero, so that zero stays exactly representable */
  float lo = 0.0f, hi = 0.0f;
  for (int64_t i = 0; i < K; ++i) {
    if (v[i] < lo) lo = v[i];
    if (v[i] > hi) hi = v[i];
  }
  const float sc = round_to_fp16((hi - lo) / 15.0f); /* fp32 subtraction and division, then fp16 */
  if (sc == 0.0f) {
    for (int64_t i = 0; i < K; ++i) out[i] = 0.0;
    return;
  }
  double z = rint((double)(-lo / sc)); /* zero point: the code of 0.0 */
  if (z > 15.0) z = 15.0;
  for (int64_t i = 0; i < K; ++i) {
    double q = rint((double)(v[i] / sc));
    if (q > 31.0) q = 31.0;
    if (q < -16.0) q = -16.0;
    q += z;
    if (q > 15.0) q = 15.0;
    if (q < 0.0) q = 0.0;
    out[i] = (q - z) * (double)sc;
  }
}

int bro_ref_fake_quantize(const float* y, int64_t rows, int64_t K, int format, double* deq) {
  if (!y || !deq) return 1;
  if (rows < 0 || K <= 0 || K % MX_GROUP != 0 || format < 0 || format > 5) return 2;
  if (format >= 4) {
#pragma omp parallel for schedule(static)
    for (int64_t r = 0; r < rows; ++r) int4_row(y + r * K, K, format == 5, deq + r * K);
    return 0;
  }
  const int64_t ng = K / MX_GROUP;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < rows; ++r)
    for (int64_t g = 0; g < ng; ++g) {
      const float* v = y + r * K + g * MX_GROUP;
      double* out = deq + r * K + g * MX_GROUP;
      float amax = 0.0f;
      for (int i = 0; i < MX_GROUP; ++i)
        if (fabsf(v[i]) > amax) amax = fabsf(v[i]);
      const int ef = (int)((f32_bits(amax) >> 23) & 0xFF);
      if (format == 0 || format == 2) {
        /* power-of-two scale: MXFP4 keeps 2 integer bits above the scale, MXINT4 none */
        int s = format == 0 ? ef - 2 : ef;
        if (s < 0) s = 0;
        const int E = s - 127;
        for (int i = 0; i < MX_GROUP; ++i) {
          const float rr = ldexpf(fabsf(v[i]), -E);
          double q;
          if (format == 0) q = E2M1_GRID[e2m1_round(rr)];
          else {
            double k = rint((double)rr * 4.0); /* exact product, ties to even */
            if (k > 7.0) k = 7.0;
            q = k / 4.0;
          }
          q = ldexp(q, E);
          out[i] = (f32_bits(v[i]) >> 31) ? -q : q;
        }
      } else {
        const float qmax = format == 1 ? 6.0f : 7.0f;
        const float sc = round_to_fp16(amax / qmax); /* fp32 division, then fp16 rounding */
        for (int i = 0; i < MX_GROUP; ++i) {
          if (sc == 0.0f) { out[i] = 0.0; continue; }
          const float rr = fabsf(v[i]) / sc; /* fp32 division */
          double q;
          if (format == 1) q = E2M1_GRID[e2m1_round(rr)];
          else {
            q = rint((double)rr);
            if (q > 7.0) q = 7.0;
          }
          q *= (double)sc;
          out[i] = (f32_bits(v[i]) >> 31) ? -q : q;
        }
      }
    }
  return 0;
}

/* ---- scale statistics (Sec. 4.1 regular / outlier blocks; Sec. 4.2 Fig. 6; App. A.3) ---------------- */
static int cmp_u16_desc(const void* a, const void* b) {
  uint16_t x = *(const uint16_t*)a, y = *(const uint16_t*)b;
  return (x < y) - (x > y);
}

int bro_ref_outlier_groups(const uint16_t* x, int64_t M, int64_t K, int64_t ldx, int64_t top_ppm,
                           uint8_t* mask, uint16_t* threshold_bits) {
  if (!x || !mask) return 1;
  if (M <= 0 || K <= 0 || K % MX_GROUP != 0 || ldx < K || top_ppm <= 0 || top_ppm > 1000000) return 2;
  const int64_t n = M * K;
  /* |x| of a finite bf16 is ordered like its low 15 bits read as an integer */
  uint16_t* mag = (uint16_t*)malloc((size_t)n * sizeof(uint16_t));
  if (!mag) return 3;
  for (int64_t m = 0; m < M; ++m)
    for (int64_t k = 0; k < K; ++k) mag[m * K + k] = (uint16_t)(x[m * ldx + k] & 0x7FFFu);
  qsort(mag, (size_t)n, sizeof(uint16_t), cmp_u16_desc);
  int64_t k = (n * top_ppm + 999999) / 1000000; /* ceil */
  if (k < 1) k = 1;
  const uint16_t t = mag[k - 1];
  free(mag);
  if (threshold_bits) *threshold_bits = t;
  const int64_t ng = K / MX_GROUP;
  for (int64_t m = 0; m < M; ++m)
    for (int64_t g = 0; g < ng; ++g) {
      uint8_t any = 0;
      for (int i = 0; i < MX_GROUP; ++i)
        if ((uint16_t)(x[m * ldx + g * MX_GROUP + i] & 0x7FFFu) >= t) any = 1;
      mask[m * ng + g] = any;
    }
  return 0;
}

int bro_ref_scale_histogram(const uint8_t* scales, const uint8_t* mask, int64_t n, uint64_t* hist) {
  if (!scales || !mask || !hist) return 1;
  if (n < 0) return 2;
  memset(hist, 0, 2 * 256 * sizeof(uint64_t));
  for (int64_t i = 0; i < n; ++i) hist[(mask[i] ? 256 : 0) + scales[i]] += 1;
  return 0;
}

int bro_ref_scale_inflation(const uint8_t* before, const uint8_t* after, const uint8_t* mask, int64_t n,
                            uint64_t* counts) {
  if (!before || !after || !mask || !counts) return 1;
  if (n < 0) return 2;
  memset(counts, 0, 6 * sizeof(uint64_t));
  for (int64_t i = 0; i < n; ++i) {
    const int j = after[i] < before[i] ? 0 : (after[i] == before[i] ? 1 : 2);
    counts[(mask[i] ? 3 : 0) + j] += 1;
  }
  return 0;
}

/* ---- gated MLP activation feeding the online rotation (Sec. 4.3, the R_4 site before down_proj) ------- */
static inline float f32_from_bits(uint32_t u) {
  float f;
  memcpy(&f, &u, 4);
  return f;
}

static inline float silu_mul_f32(float g, float u) {
  const float LOG2E = f32_from_bits(0x3FB8AA3Bu);  /* fp32(log2 e) */
  const float LN2_HI = f32_from_bits(0x3F317218u); /* fp32(ln 2) */
  const float LN2_LO = f32_from_bits(0xB102E308u); /* fp32(ln 2 - LN2_HI) = -1.9046543e-9 */
  const float t = -fabsf(g);
  float e = 0.0f;
  if (t >= -86.0f) {
    const float n = rintf(t * LOG2E); /* round to nearest, ties to even */
    float r = fmaf(n, -LN2_HI, t);
    r = fmaf(n, -LN2_LO, r);
    float p = f32_from_bits(0x3AB60B61u);        /* 1/720 */
    p = fmaf(p, r, f32_from_bits(0x3C088889u));  /* 1/120 */
    p = fmaf(p, r, f32_from_bits(0x3D2AAAABu));  /* 1/24 */
    p = fmaf(p, r, f32_from_bits(0x3E2AAAABu));  /* 1/6 */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    /* p in [0.70, 1.42], n in [-124, 0]: scaling by 2^n is an exponent-field addition, exact */
    e = f32_from_bits(f32_bits(p) + ((uint32_t)(int32_t)n << 23));
  }
  const float d = 1.0f + e;
  const float num = (g >= 0.0f) ? 1.0f : e;
  const float s = num / d;
  const float a = g * s;
  return a * u;
}

static inline uint16_t f32_to_bf16_rne(float f) {
  uint32_t u = f32_bits(f);
  /* finite inputs: add half an ulp of bf16 minus one, plus the lowest kept bit (ties to even) */
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

int bro_ref_swiglu_f32(const uint16_t* gate, const uint16_t* up, int64_t n, float* h32) {
  if (!gate || !up || !h32) return 1;
  if (n < 0) return 2;
  for (int64_t i = 0; i < n; ++i) h32[i] = silu_mul_f32(bf16_to_f32(gate[i]), bf16_to_f32(up[i]));
  return 0;
}

int bro_ref_swiglu(const uint16_t* gate, const uint16_t* up, int64_t M, int64_t K, int64_t ldg, int64_t ldu,
                   uint16_t* h) {
  if (!gate || !up || !h) return 1;
  if (M < 0 || K <= 0 || ldg < K || ldu < K) return 2;
#pragma omp parallel for schedule(static)
  for (int64_t m = 0; m < M; ++m)
    for (int64_t k = 0; k < K; ++k)
      h[m * K + k] = f32_to_bf16_rne(silu_mul_f32(bf16_to_f32(gate[m * ldg + k]), bf16_to_f32(up[m * ldu + k])));
  return 0;
}

int bro_ref_swiglu_rotate_quantize_mxfp4(const uint16_t* gate, const uint16_t* up, int64_t M, int64_t K,
                                         int64_t ldg, int64_t ldu, int block, const uint16_t* signs,
                                         uint8_t* codes, uint8_t* scales) {
  if (M < 0 || K <= 0) return 2;
  uint16_t* h = (uint16_t*)malloc((size_t)(M > 0 ? M : 1) * (size_t)K * sizeof(uint16_t));
  if (!h) return 3;
  int rc = bro_ref_swiglu(gate, up, M, K, ldg, ldu, h);
  if (rc == 0) rc = bro_ref_rotate_quantize_mxfp4_rs(h, M, K, K, block, signs, codes, scales);
  free(h);
  return rc;
}
