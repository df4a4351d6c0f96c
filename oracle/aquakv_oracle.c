/*
 * aquakv_oracle.c -- plain, slow CPU statement of the AQUA-KV per-token KV-cache codec.
 *
 * TEST INFRASTRUCTURE ONLY.  This file defines what the CUDA library must compute; it shares no
 * code, header, table or helper with that library, and the library never calls it.  Only the
 * tests, the smoke check and the benchmark's CPU-baseline leg build and run it.
 *
 * Written from the paper ("Cache Me If You Must: Adaptive Key-Value Quantization for Large
 * Language Models"), following its steps in its order:
 *   - Algorithm 2 (encode):  K_pred = f_key(K^_prev);  K_q = Q(K - K_pred);
 *                            K^ = Q^-1(K_q) + K_pred;  V_pred = f_value([V^_prev ; K^]);
 *                            V_q = Q(V - V_pred)
 *   - Algorithm 3 (decode):  K^ = Q^-1(K_q) + f_key(K^_prev);
 *                            V^ = Q^-1(V_q) + f_value([V^_prev ; K^])
 *   - Section 3.2: f_key, f_value are linear regressors (a matrix, optionally a bias).
 *   - Section 2 "Vector Quantization" and Section 4.1 "Alternative quantizers": Q is group-wise
 *     vector quantization after a randomized Hadamard transform: scale each group, rotate, round
 *     every p=2 consecutive rotated values to the nearest of n fixed grid points; one 16-bit scale
 *     per group (2 + 16/1024 = 2.02 bits per value at n=16, group 1024).
 *   - Algorithm 4, the attention read: a new query attends over the decoded cache.
 *
 * All arithmetic is double precision.  Roundings happen only where a stored format forces them:
 * the scale is stored as fp16, reconstructed keys/values as fp16 or bf16 (round to nearest even).
 *
 * Readings taken where the paper is silent (each is a parameter or stated here):
 *   - group scale = root mean square of the group's residual, rounded to fp16; the rotated
 *     values are normalised with the ROUNDED scale so encoder and decoder agree;
 *   - Hadamard matrix in Sylvester (natural) order H[i][j] = (-1)^popcount(i&j), orthonormal
 *     factor 1/sqrt(h); signs multiply before H on encode and after H on decode;
 *   - nearest point by squared Euclidean distance, lowest index wins ties;
 *   - codes packed LSB-first: pair j occupies bits [j*b, (j+1)*b) of the row's byte stream;
 *   - the value predictor reads the 16-bit-rounded K^ (the only value a decoder has);
 *   - adapter matrices are stored [out_features][in_features].
 *
 * Parity pins live in tests/test_oracle_*.py (Hadamard against a library Hadamard matrix,
 * search against a library nearest-neighbour routine, float formats against numpy/torch,
 * closed-form special cases, the paper's bits-per-value figures).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define AQO_F16 0
#define AQO_BF16 1

typedef struct {
  int32_t d_kv;        /* values per token row */
  int32_t had_block;   /* h: Hadamard block (power of two), divides d_kv */
  int32_t scale_group; /* g: values per fp16 scale, multiple of h, divides d_kv */
  int32_t grid_size;   /* n: number of 2-D grid points (power of two) */
  int32_t dtype;       /* AQO_F16 or AQO_BF16: storage of K, V, K^, V^, adapters */
} aqo_params;

/* ------------------------------------------------------------------------------------------ */
/* Small binary floating-point formats (fp16: 5 exponent / 10 mantissa bits; bf16: 8 / 7)      */
/* ------------------------------------------------------------------------------------------ */

static double small_to_double(uint16_t bits, int ebits, int mbits) {
  int sign = (bits >> 15) & 1;
  int e = (bits >> mbits) & ((1 << ebits) - 1);
  int m = bits & ((1 << mbits) - 1);
  int bias = (1 << (ebits - 1)) - 1;
  double v;
  if (e == (1 << ebits) - 1) {
    v = m ? NAN : INFINITY;
  } else if (e == 0) {
    v = ldexp((double)m, 1 - bias - mbits);
  } else {
    v = ldexp((double)(m + (1 << mbits)), e - bias - mbits);
  }
  return sign ? -v : v;
}

/* Round to nearest, ties to even (nearbyint under the default rounding mode). */
static uint16_t double_to_small(double x, int ebits, int mbits) {
  int bias = (1 << (ebits - 1)) - 1;
  int emax = bias;          /* largest unbiased exponent of a finite number */
  int emin = 1 - bias;      /* unbiased exponent of the smallest normal */
  uint16_t sign = signbit(x) ? 0x8000u : 0u;
  uint16_t inf = (uint16_t)(((1 << ebits) - 1) << mbits);
  double a = fabs(x);
  if (isnan(x)) return (uint16_t)(sign | inf | 1u);
  if (a == 0.0) return sign;
  if (isinf(a)) return (uint16_t)(sign | inf);
  int e2;
  (void)frexp(a, &e2);      /* a = f * 2^e2, f in [0.5, 1)  =>  a in [2^(e2-1), 2^e2) */
  int E = e2 - 1;
  if (E < emin) {
    double q = nearbyint(ldexp(a, -(emin - mbits)));   /* multiples of the subnormal step */
    return (uint16_t)(sign | (uint16_t)q);              /* q == 2^mbits lands on the min normal */
  }
  double q = nearbyint(ldexp(a, mbits - E));            /* in [2^mbits, 2^(mbits+1)] */
  if (q >= (double)(2 << mbits)) { q = (double)(1 << mbits); E += 1; }
  if (E > emax) return (uint16_t)(sign | inf);
  return (uint16_t)(sign | (uint16_t)((E + bias) << mbits) | (uint16_t)((int)q - (1 << mbits)));
}

double aqo_f16_to_double(uint16_t b) { return small_to_double(b, 5, 10); }
double aqo_bf16_to_double(uint16_t b) { return small_to_double(b, 8, 7); }
uint16_t aqo_double_to_f16(double x) { return double_to_small(x, 5, 10); }
uint16_t aqo_double_to_bf16(double x) { return double_to_small(x, 8, 7); }

static double load16(uint16_t b, int dtype) {
  return dtype == AQO_F16 ? aqo_f16_to_double(b) : aqo_bf16_to_double(b);
}
static uint16_t store16(double x, int dtype) {
  return dtype == AQO_F16 ? aqo_double_to_f16(x) : aqo_double_to_bf16(x);
}

/* ------------------------------------------------------------------------------------------ */
/* Hadamard transform                                                                          */
/* ------------------------------------------------------------------------------------------ */

static int popcount32(uint32_t v) { int c = 0; while (v) { c += (int)(v & 1u); v >>= 1; } return c; }

/* The definition: y[i] = sum_j (-1)^popcount(i&j) x[j], unnormalised, O(h^2). */
void aqo_hadamard_definition(const double* x, double* y, int h) {
  for (int i = 0; i < h; ++i) {
    double acc = 0.0;
    for (int j = 0; j < h; ++j) acc += (popcount32((uint32_t)(i & j)) & 1) ? -x[j] : x[j];
    y[i] = acc;
  }
}

/* The same transform by butterflies, in place, unnormalised, O(h log h). */
void aqo_hadamard_butterfly(double* x, int h) {
  for (int len = 1; len < h; len <<= 1)
    for (int i = 0; i < h; i += 2 * len)
      for (int j = i; j < i + len; ++j) {
        double a = x[j], b = x[j + len];
        x[j] = a + b;
        x[j + len] = a - b;
      }
}

/* ------------------------------------------------------------------------------------------ */
/* Q and Q^-1 on one row                                                                       */
/* ------------------------------------------------------------------------------------------ */

static int log2i(int n) { int b = 0; while ((1 << b) < n) ++b; return b; }

int aqo_code_bytes(const aqo_params* p) { return p->d_kv / 2 * log2i(p->grid_size) / 8; }

static int params_ok(const aqo_params* p) {
  if (!p || p->d_kv <= 0 || p->had_block <= 1 || p->scale_group <= 0 || p->grid_size < 2) return 0;
  if (p->had_block & (p->had_block - 1)) return 0;
  if (p->grid_size & (p->grid_size - 1)) return 0;
  if (p->d_kv % p->scale_group || p->scale_group % p->had_block) return 0;
  if ((p->d_kv / 2 * log2i(p->grid_size)) % 8) return 0;
  if (p->dtype != AQO_F16 && p->dtype != AQO_BF16) return 0;
  return 1;
}

/* Q^-1 of one row: xhat = s16 * xi (.) (H G[c]) / sqrt(h), per Hadamard block, per scale group. */
static void dequantize_row(const aqo_params* p, const double* grid, const int8_t* signs,
                           const uint8_t* codes, const uint16_t* scales, double* xhat) {
  const int d = p->d_kv, h = p->had_block, g = p->scale_group, b = log2i(p->grid_size);
  const double rs = 1.0 / sqrt((double)h);
  for (int j = 0; j < d / 2; ++j) {
    int bit = j * b, c = 0;
    for (int k = 0; k < b; ++k, ++bit) c |= ((codes[bit >> 3] >> (bit & 7)) & 1) << k;
    xhat[2 * j] = grid[2 * c];
    xhat[2 * j + 1] = grid[2 * c + 1];
  }
  for (int o = 0; o < d; o += h) aqo_hadamard_butterfly(xhat + o, h);
  for (int i = 0; i < d; ++i) {
    double s16 = aqo_f16_to_double(scales[i / g]);
    xhat[i] = s16 * (double)signs[i] * (xhat[i] * rs);
  }
}

/* Q of one row (residual r, double).  Outputs: codes, scales (fp16 bits), and optionally the
 * nearest-point margins, the unrounded scales and the rotated normalised values y. */
static void quantize_row(const aqo_params* p, const double* grid, const int8_t* signs,
                         const double* r, uint8_t* codes, uint16_t* scales, double* margins,
                         double* scales_exact, double* y_out, double* y /* scratch [d] */) {
  const int d = p->d_kv, h = p->had_block, g = p->scale_group, n = p->grid_size, b = log2i(n);
  const double rs = 1.0 / sqrt((double)h);
  /* group scale: root mean square, stored as fp16 (clamped to the largest finite fp16) */
  for (int k = 0; k < d / g; ++k) {
    double ss = 0.0;
    for (int i = k * g; i < (k + 1) * g; ++i) ss += r[i] * r[i];
    double s = sqrt(ss / (double)g);
    if (scales_exact) scales_exact[k] = s;
    if (s > 65504.0) s = 65504.0;
    scales[k] = aqo_double_to_f16(s);
  }
  /* normalise with the rounded scale, apply signs, rotate */
  for (int i = 0; i < d; ++i) {
    double s16 = aqo_f16_to_double(scales[i / g]);
    double inv = s16 > 0.0 ? 1.0 / s16 : 0.0;
    y[i] = (double)signs[i] * r[i] * inv;
  }
  for (int o = 0; o < d; o += h) aqo_hadamard_butterfly(y + o, h);
  for (int i = 0; i < d; ++i) y[i] *= rs;
  if (y_out) memcpy(y_out, y, sizeof(double) * (size_t)d);
  /* nearest grid point for every consecutive pair; lowest index wins ties */
  memset(codes, 0, (size_t)aqo_code_bytes(p));
  for (int j = 0; j < d / 2; ++j) {
    double best = INFINITY, second = INFINITY;
    int arg = 0;
    for (int c = 0; c < n; ++c) {
      double d0 = y[2 * j] - grid[2 * c], d1 = y[2 * j + 1] - grid[2 * c + 1];
      double dist = d0 * d0 + d1 * d1;
      if (dist < best) { second = best; best = dist; arg = c; }
      else if (dist < second) { second = dist; }
    }
    if (margins) margins[j] = (second - best) / (second + best + 1e-30);
    int bit = j * b;
    for (int k = 0; k < b; ++k, ++bit) codes[bit >> 3] |= (uint8_t)(((arg >> k) & 1) << (bit & 7));
  }
}

/* Row-batched Q on double residuals (exposed for the pins). */
int aqo_quantize(const aqo_params* p, const float* grid_f, const int8_t* signs, int64_t T,
                 const double* R, uint8_t* codes, uint16_t* scales, double* margins,
                 double* scales_exact, double* Y) {
  if (!params_ok(p)) return -1;
  const int d = p->d_kv, cb = aqo_code_bytes(p), ng = d / p->scale_group;
  double* grid = (double*)malloc(sizeof(double) * 2 * (size_t)p->grid_size);
  for (int i = 0; i < 2 * p->grid_size; ++i) grid[i] = (double)grid_f[i];
#pragma omp parallel
  {
    double* y = (double*)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(static)
    for (int64_t t = 0; t < T; ++t)
      quantize_row(p, grid, signs, R + t * d, codes + t * cb, scales + t * ng,
                   margins ? margins + t * (d / 2) : NULL,
                   scales_exact ? scales_exact + t * ng : NULL, Y ? Y + t * d : NULL, y);
    free(y);
  }
  free(grid);
  return 0;
}

/* Row-batched Q^-1 to double (exposed for the pins). */
int aqo_dequantize(const aqo_params* p, const float* grid_f, const int8_t* signs, int64_t T,
                   const uint8_t* codes, const uint16_t* scales, double* Xhat) {
  if (!params_ok(p)) return -1;
  const int d = p->d_kv, cb = aqo_code_bytes(p), ng = d / p->scale_group;
  double* grid = (double*)malloc(sizeof(double) * 2 * (size_t)p->grid_size);
  for (int i = 0; i < 2 * p->grid_size; ++i) grid[i] = (double)grid_f[i];
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < T; ++t)
    dequantize_row(p, grid, signs, codes + t * cb, scales + t * ng, Xhat + t * d);
  free(grid);
  return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Linear predictor: pred[c] = sum_r x[r] * W[c][r] (+ bias[c]), x = concatenation of n_in rows */
/* ------------------------------------------------------------------------------------------ */

static void predict_row(const aqo_params* p, int n_in, const uint16_t* const* in_rows,
                        const uint16_t* W, const float* bias, double* pred, double* x /*[n_in*d]*/) {
  const int d = p->d_kv;
  if (!W) { for (int c = 0; c < d; ++c) pred[c] = 0.0; return; }   /* layer 0: no predictor */
  for (int s = 0; s < n_in; ++s)
    for (int r = 0; r < d; ++r) x[s * d + r] = load16(in_rows[s][r], p->dtype);
  const int kin = n_in * d;
  for (int c = 0; c < d; ++c) {
    double acc = 0.0;
    const uint16_t* w = W + (size_t)c * (size_t)kin;
    for (int r = 0; r < kin; ++r) acc += x[r] * load16(w[r], p->dtype);
    pred[c] = acc + (bias ? (double)bias[c] : 0.0);
  }
}

int aqo_predict(const aqo_params* p, int64_t T, int n_in, const uint16_t* in0, const uint16_t* in1,
                const uint16_t* W, const float* bias, double* P) {
  if (!params_ok(p) || n_in < 1 || n_in > 2) return -1;
  const int d = p->d_kv;
#pragma omp parallel
  {
    double* x = (double*)malloc(sizeof(double) * 2 * (size_t)d);
#pragma omp for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
      const uint16_t* rows[2] = {in0 + t * d, in1 ? in1 + t * d : NULL};
      predict_row(p, n_in, rows, W, bias, P + t * d, x);
    }
    free(x);
  }
  return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* One phase of Algorithm 2 (predict, quantize the residual, reconstruct: keys or values)     */
/*   pred = f(inputs);  q = Q(X - pred);  hat = round16(Q^-1(q) + pred)                        */
/* ------------------------------------------------------------------------------------------ */

int aqo_encode_phase(const aqo_params* p, const float* grid_f, const int8_t* signs, int64_t T,
                     const uint16_t* X, int n_in, const uint16_t* in0, const uint16_t* in1,
                     const uint16_t* W, const float* bias,
                     uint8_t* codes, uint16_t* scales, uint16_t* hat,
                     double* margins, double* scales_exact, double* hat_exact, double* pred_out) {
  if (!params_ok(p)) return -1;
  if (W && (n_in < 1 || n_in > 2 || !in0 || (n_in == 2 && !in1))) return -1;
  const int d = p->d_kv, cb = aqo_code_bytes(p), ng = d / p->scale_group;
  double* grid = (double*)malloc(sizeof(double) * 2 * (size_t)p->grid_size);
  for (int i = 0; i < 2 * p->grid_size; ++i) grid[i] = (double)grid_f[i];
#pragma omp parallel
  {
    double* buf = (double*)malloc(sizeof(double) * 6 * (size_t)d);
    double *pred = buf, *r = buf + d, *y = buf + 2 * d, *xh = buf + 3 * d, *x = buf + 4 * d;
#pragma omp for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
      const uint16_t* rows[2] = {in0 ? in0 + t * d : NULL, in1 ? in1 + t * d : NULL};
      predict_row(p, n_in, rows, W, bias, pred, x);                      /* predict           */
      for (int i = 0; i < d; ++i) r[i] = load16(X[t * d + i], p->dtype) - pred[i];
      quantize_row(p, grid, signs, r, codes + t * cb, scales + t * ng,    /* quantize    */
                   margins ? margins + t * (d / 2) : NULL,
                   scales_exact ? scales_exact + t * ng : NULL, NULL, y);
      dequantize_row(p, grid, signs, codes + t * cb, scales + t * ng, xh); /* rebuild */
      for (int i = 0; i < d; ++i) {
        double v = pred[i] + xh[i];
        if (hat_exact) hat_exact[t * d + i] = v;
        if (hat) hat[t * d + i] = store16(v, p->dtype);
        if (pred_out) pred_out[t * d + i] = pred[i];
      }
    }
    free(buf);
  }
  free(grid);
  return 0;
}

/* One phase of Algorithm 3 (keys or values): hat = round16(Q^-1(q) + f(in)). */
int aqo_decode_phase(const aqo_params* p, const float* grid_f, const int8_t* signs, int64_t T,
                     const uint8_t* codes, const uint16_t* scales,
                     int n_in, const uint16_t* in0, const uint16_t* in1,
                     const uint16_t* W, const float* bias, uint16_t* hat, double* hat_exact) {
  if (!params_ok(p)) return -1;
  if (W && (n_in < 1 || n_in > 2 || !in0 || (n_in == 2 && !in1))) return -1;
  const int d = p->d_kv, cb = aqo_code_bytes(p), ng = d / p->scale_group;
  double* grid = (double*)malloc(sizeof(double) * 2 * (size_t)p->grid_size);
  for (int i = 0; i < 2 * p->grid_size; ++i) grid[i] = (double)grid_f[i];
#pragma omp parallel
  {
    double* buf = (double*)malloc(sizeof(double) * 4 * (size_t)d);
    double *pred = buf, *xh = buf + d, *x = buf + 2 * d;
#pragma omp for schedule(static)
    for (int64_t t = 0; t < T; ++t) {
      const uint16_t* rows[2] = {in0 ? in0 + t * d : NULL, in1 ? in1 + t * d : NULL};
      predict_row(p, n_in, rows, W, bias, pred, x);
      dequantize_row(p, grid, signs, codes + t * cb, scales + t * ng, xh);
      for (int i = 0; i < d; ++i) {
        double v = pred[i] + xh[i];
        if (hat_exact) hat_exact[t * d + i] = v;
        if (hat) hat[t * d + i] = store16(v, p->dtype);
      }
    }
    free(buf);
  }
  free(grid);
  return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Algorithm 2 / Algorithm 3 for one layer (keys first, then values reading the rounded K^)    */
/* ------------------------------------------------------------------------------------------ */

int aqo_encode_layer(const aqo_params* p, const float* grid, const int8_t* signs_k,
                     const int8_t* signs_v, int64_t T, const uint16_t* K, const uint16_t* V,
                     const uint16_t* Khat_prev, const uint16_t* Vhat_prev,
                     const uint16_t* Wk, const uint16_t* Wv, const float* bk, const float* bv,
                     uint8_t* Kcodes, uint16_t* Kscales, uint8_t* Vcodes, uint16_t* Vscales,
                     uint16_t* Khat, uint16_t* Vhat, double* Kmargins, double* Vmargins) {
  int rc = aqo_encode_phase(p, grid, signs_k, T, K, 1, Khat_prev, NULL, Wk, bk,
                            Kcodes, Kscales, Khat, Kmargins, NULL, NULL, NULL);
  if (rc) return rc;
  return aqo_encode_phase(p, grid, signs_v, T, V, 2, Vhat_prev, Khat, Wv, bv,
                          Vcodes, Vscales, Vhat, Vmargins, NULL, NULL, NULL);
}

int aqo_decode_layer(const aqo_params* p, const float* grid, const int8_t* signs_k,
                     const int8_t* signs_v, int64_t T,
                     const uint8_t* Kcodes, const uint16_t* Kscales,
                     const uint8_t* Vcodes, const uint16_t* Vscales,
                     const uint16_t* Khat_prev, const uint16_t* Vhat_prev,
                     const uint16_t* Wk, const uint16_t* Wv, const float* bk, const float* bv,
                     uint16_t* Khat, uint16_t* Vhat) {
  int rc = aqo_decode_phase(p, grid, signs_k, T, Kcodes, Kscales, 1, Khat_prev, NULL, Wk, bk,
                            Khat, NULL);
  if (rc) return rc;
  return aqo_decode_phase(p, grid, signs_v, T, Vcodes, Vscales, 2, Vhat_prev, Khat, Wv, bv,
                          Vhat, NULL);
}

/* ------------------------------------------------------------------------------------------ */
/* Single-query attention over the decoded cache (Algorithm 4's attention read), grouped-query heads  */
/*   token index of (sequence b, position t) is b*ctx + t; kv head of query head qh is          */
/*   qh / (n_q_heads / n_kv_heads); out = softmax_t(scale * q . K^_t) . V^_t                     */
/* ------------------------------------------------------------------------------------------ */

int aqo_attention(int dtype, int32_t batch, int64_t ctx, int32_t n_q_heads, int32_t n_kv_heads,
                  int32_t head_dim, double softmax_scale, const uint16_t* q,
                  const uint16_t* Khat, const uint16_t* Vhat, double* out, double* lse) {
  if (batch < 0 || ctx <= 0 || n_kv_heads <= 0 || n_q_heads % n_kv_heads) return -1;
  const int d = n_kv_heads * head_dim, rep = n_q_heads / n_kv_heads;
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < batch; ++b)
    for (int qh = 0; qh < n_q_heads; ++qh) {
      const int kvh = qh / rep;
      const uint16_t* qv = q + ((size_t)b * n_q_heads + qh) * head_dim;
      double* s = (double*)malloc(sizeof(double) * (size_t)ctx);
      double m = -INFINITY;
      for (int64_t t = 0; t < ctx; ++t) {
        const uint16_t* kr = Khat + ((size_t)b * ctx + t) * d + kvh * head_dim;
        double acc = 0.0;
        for (int i = 0; i < head_dim; ++i) acc += load16(qv[i], dtype) * load16(kr[i], dtype);
        s[t] = softmax_scale * acc;
        if (s[t] > m) m = s[t];
      }
      double z = 0.0;
      for (int64_t t = 0; t < ctx; ++t) { s[t] = exp(s[t] - m); z += s[t]; }
      double* o = out + ((size_t)b * n_q_heads + qh) * head_dim;
      for (int i = 0; i < head_dim; ++i) o[i] = 0.0;
      for (int64_t t = 0; t < ctx; ++t) {
        const uint16_t* vr = Vhat + ((size_t)b * ctx + t) * d + kvh * head_dim;
        double w = s[t] / z;
        for (int i = 0; i < head_dim; ++i) o[i] += w * load16(vr[i], dtype);
      }
      if (lse) lse[(size_t)b * n_q_heads + qh] = m + log(z);
      free(s);
    }
  return 0;
}

int aqo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

void aqo_set_num_threads(int n) {
#ifdef _OPENMP
  if (n > 0) omp_set_num_threads(n);
#else
  (void)n;
#endif
}
