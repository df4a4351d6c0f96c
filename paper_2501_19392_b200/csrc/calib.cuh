// Predictor calibration (Algorithm 1, its two least-squares fits; Section 3.2: linear regressors that are
// trained in closed form; Appendix A: the regularizer rate is 1e-3):
//
//   W = argmin_W || X W^T (+ b) - Y ||^2 + rate * trace(X^T X) / n_in * ||W||^2
//
// over the calibration tokens, X = [in0 ; in1] (16-bit rows), Y the layer's keys or values.
//
// Device pipeline (every step a kernel of this library):
//   1. X and Y are transposed into token-contiguous 16-bit matrices (zero-padded to a multiple of 64
//      tokens), so that the normal equations G = X^T X and C = X^T Y are K-major products for the
//      tcgen05 GEMM of gemm_pred.cuh (16-bit products are exact, accumulation is fp32).
//   2. Column sums (only with an intercept), the trace and the ridge term; G and C go to double
//      precision with the centring correction  - s_i s_j / T  and the ridge on the diagonal.
//   3. Blocked Cholesky factorisation G = L L^T and the two triangular solves in double precision
//      (panels of 32; the rank-32 updates are one generic kernel).
//   4. W^T is rounded to the cache's 16-bit type as [d_kv][n_in] (a linear layer's weight); the
//      intercept is b = mean(Y) - mean(X) W^T.
#pragma once

#include "common.cuh"

namespace aquakv {

constexpr int kFitNB = 32;          // panel width of the factorisation and the solves

// out[c][t] = in[t][c] for t < T, 0 for T <= t < Tp.  Grid (Tp/32, ncols/32), block (32, 8).
__global__ void fit_transpose_kernel(const uint16_t* __restrict__ in, long long ld_in, long long T, long long Tp,
                                     uint16_t* __restrict__ out) {
  __shared__ uint16_t tile[32][33];
  const long long t0 = (long long)blockIdx.x * 32;
  const int c0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += 8) {
    const long long t = t0 + r;
    tile[r][threadIdx.x] = t < T ? in[t * ld_in + c0 + threadIdx.x] : uint16_t(0);
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += 8) out[(long long)(c0 + r) * Tp + t0 + threadIdx.x] = tile[threadIdx.x][r];
}

template <bool kBf16>
__device__ __forceinline__ float fit_to_float(uint16_t b) {
  if constexpr (kBf16) return __uint_as_float(uint32_t(b) << 16);
  else return __half2float(__ushort_as_half(b));
}

// sums[c] += sum over this block's tokens of in[t][c].  Grid (ceil(T / 256), ncols/32), block (32, 8).
template <bool kBf16>
__global__ void fit_colsum_kernel(const uint16_t* __restrict__ in, long long ld_in, long long T,
                                  double* __restrict__ sums) {
  __shared__ double part[8][32];
  const int c = blockIdx.y * 32 + threadIdx.x;
  const long long t0 = (long long)blockIdx.x * 256;
  double s = 0.0;
  for (int r = threadIdx.y; r < 256; r += 8) {
    const long long t = t0 + r;
    if (t < T) s += double(fit_to_float<kBf16>(in[t * ld_in + c]));
  }
  part[threadIdx.y][threadIdx.x] = s;
  __syncthreads();
  if (threadIdx.y == 0) {
    for (int r = 1; r < 8; ++r) s += part[r][threadIdx.x];
    atomicAdd(&sums[c], s);
  }
}

// ridge = rate * trace(centred G) / n.  One block of 256 threads.  sx == nullptr: no centring.
__global__ void fit_ridge_kernel(const float* __restrict__ G, int n, double T, const double* __restrict__ sx,
                                 double rate, double* __restrict__ ridge) {
  __shared__ double part[256];
  double s = 0.0;
  for (int i = threadIdx.x; i < n; i += 256) {
    double g = double(G[size_t(i) * n + i]);
    if (sx != nullptr) g -= sx[i] * sx[i] / T;
    s += g;
  }
  part[threadIdx.x] = s;
  __syncthreads();
  for (int w = 128; w > 0; w >>= 1) {
    if (threadIdx.x < w) part[threadIdx.x] += part[threadIdx.x + w];
    __syncthreads();
  }
  if (threadIdx.x == 0) *ridge = rate * part[0] / double(n);
}

// Gd = G - sx sx^T / T + ridge I   (n x n),   Cd = C - sx sy^T / T   (n x d).  One thread per element
// of the wider of the two; sx == nullptr: no centring.
__global__ void fit_prepare_kernel(const float* __restrict__ G, const float* __restrict__ C, int n, int d, double T,
                                   const double* __restrict__ sx, const double* __restrict__ sy,
                                   const double* __restrict__ ridge, double* __restrict__ Gd,
                                   double* __restrict__ Cd) {
  const int i = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < n) {
    double g = double(G[size_t(i) * n + j]);
    if (sx != nullptr) g -= sx[i] * sx[j] / T;
    if (i == j) g += *ridge;
    Gd[size_t(i) * n + j] = g;
  }
  if (j < d) {
    double c = double(C[size_t(i) * d + j]);
    if (sx != nullptr) c -= sx[i] * sy[j] / T;
    Cd[size_t(i) * d + j] = c;
  }
}

// Cholesky of the 32 x 32 diagonal block at (k, k), in place (lower triangle).  One block of 32 x 32
// threads.  A pivot that is not positive sets *status (the matrix was not positive definite) and is
// replaced by 1 so that the remaining kernels stay finite.
__global__ void fit_chol_diag_kernel(double* __restrict__ A, int n, int k, int* __restrict__ status) {
  __shared__ double a[kFitNB][kFitNB + 1];
  const int r = threadIdx.y, c = threadIdx.x;
  a[r][c] = A[size_t(k + r) * n + k + c];
  __syncthreads();
  for (int j = 0; j < kFitNB; ++j) {
    if (r == j && c == j) {
      double p = a[j][j];
      if (!(p > 0.0)) {
        atomicExch(status, kStatusNumeric);
        p = 1.0;
      }
      a[j][j] = sqrt(p);
    }
    __syncthreads();
    if (c == j && r > j) a[r][j] /= a[j][j];
    __syncthreads();
    if (c > j && r >= c) a[r][c] -= a[r][j] * a[c][j];
    __syncthreads();
  }
  if (c <= r) A[size_t(k + r) * n + k + c] = a[r][c];
}

// Panel below the diagonal block: L21 = A21 L11^-T for 32 rows per block.  Block of 32 threads (one per
// row); grid = (n - k - 32) / 32.
__global__ void fit_chol_panel_kernel(double* __restrict__ A, int n, int k) {
  __shared__ double l[kFitNB][kFitNB + 1];
  const int t = threadIdx.x;
  for (int r = 0; r < kFitNB; ++r) l[r][t] = A[size_t(k + r) * n + k + t];
  __syncthreads();
  const size_t row = size_t(k + kFitNB + blockIdx.x * kFitNB + t);
  double x[kFitNB];
#pragma unroll
  for (int j = 0; j < kFitNB; ++j) x[j] = A[row * n + k + j];
#pragma unroll
  for (int j = 0; j < kFitNB; ++j) {
    double s = x[j];
#pragma unroll
    for (int p = 0; p < j; ++p) s -= x[p] * l[j][p];
    x[j] = s / l[j][j];
  }
#pragma unroll
  for (int j = 0; j < kFitNB; ++j) A[row * n + k + j] = x[j];
}

// C[M x N] -= op(A)[M x 32] op(B)[32 x N]   (row-major, double).
//   op(A)(i, p) = transA ? A[p * lda + i] : A[i * lda + p]
//   op(B)(p, j) = transB ? B[j * ldb + p] : B[p * ldb + j]
// lower_only skips the 64 x 64 tiles strictly above the diagonal (symmetric update of a lower
// triangle).  Block of 16 x 16 threads, 4 x 4 results each; grid (ceil(N/64), ceil(M/64)).
__global__ void fit_update_kernel(double* __restrict__ C, long long ldc, const double* __restrict__ A, long long lda,
                                  int transA, const double* __restrict__ B, long long ldb, int transB, int M, int N,
                                  int lower_only) {
  if (lower_only && blockIdx.x > blockIdx.y) return;
  __shared__ double As[kFitNB][64 + 1];   // [p][i]
  __shared__ double Bs[kFitNB][64 + 1];   // [p][j]
  const int i0 = blockIdx.y * 64, j0 = blockIdx.x * 64;
  const int tid = threadIdx.y * 16 + threadIdx.x;
  for (int e = tid; e < 64 * kFitNB; e += 256) {
    int i, p;
    if (transA) { i = e % 64; p = e / 64; } else { p = e % kFitNB; i = e / kFitNB; }
    const int gi = i0 + i;
    As[p][i] = gi < M ? (transA ? A[(long long)p * lda + gi] : A[(long long)gi * lda + p]) : 0.0;
    int j, q;
    if (transB) { q = e % kFitNB; j = e / kFitNB; } else { j = e % 64; q = e / 64; }
    const int gj = j0 + j;
    Bs[q][j] = gj < N ? (transB ? B[(long long)gj * ldb + q] : B[(long long)q * ldb + gj]) : 0.0;
  }
  __syncthreads();
  double acc[4][4];
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int v = 0; v < 4; ++v) acc[u][v] = 0.0;
#pragma unroll 8
  for (int p = 0; p < kFitNB; ++p) {
    double av[4], bv[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) av[u] = As[p][threadIdx.y + 16 * u];
#pragma unroll
    for (int v = 0; v < 4; ++v) bv[v] = Bs[p][threadIdx.x + 16 * v];
#pragma unroll
    for (int u = 0; u < 4; ++u)
#pragma unroll
      for (int v = 0; v < 4; ++v) acc[u][v] += av[u] * bv[v];
  }
#pragma unroll
  for (int u = 0; u < 4; ++u) {
    const int gi = i0 + threadIdx.y + 16 * u;
    if (gi >= M) continue;
#pragma unroll
    for (int v = 0; v < 4; ++v) {
      const int gj = j0 + threadIdx.x + 16 * v;
      if (gj < N) C[(long long)gi * ldc + gj] -= acc[u][v];
    }
  }
}

// Z_k <- L_kk^-1 Z_k (forward) or L_kk^-T Z_k (backward) for the 32 rows at k of Z [n x d]; one thread
// per column.  Block of 128 threads; grid = ceil(d / 128).
__global__ void fit_solve_diag_kernel(const double* __restrict__ L, int n, int k, double* __restrict__ Z, int d,
                                      int backward) {
  __shared__ double l[kFitNB][kFitNB + 1];
  for (int e = threadIdx.x; e < kFitNB * kFitNB; e += blockDim.x)
    l[e / kFitNB][e % kFitNB] = L[size_t(k + e / kFitNB) * n + k + e % kFitNB];
  __syncthreads();
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= d) return;
  double x[kFitNB];
#pragma unroll
  for (int r = 0; r < kFitNB; ++r) x[r] = Z[size_t(k + r) * d + c];
  if (!backward) {
#pragma unroll
    for (int r = 0; r < kFitNB; ++r) {
      double s = x[r];
#pragma unroll
      for (int p = 0; p < r; ++p) s -= l[r][p] * x[p];
      x[r] = s / l[r][r];
    }
  } else {
#pragma unroll
    for (int r = kFitNB - 1; r >= 0; --r) {
      double s = x[r];
#pragma unroll
      for (int p = r + 1; p < kFitNB; ++p) s -= l[p][r] * x[p];
      x[r] = s / l[r][r];
    }
  }
#pragma unroll
  for (int r = 0; r < kFitNB; ++r) Z[size_t(k + r) * d + c] = x[r];
}

// W16[c][r] = round16(Wt[r][c]), W32[c][r] = float(Wt[r][c]) (optional); Wt is [n][d].
// Grid (n/32, d/32), block (32, 8).
template <bool kBf16>
__global__ void fit_store_kernel(const double* __restrict__ Wt, int n, int d, uint16_t* __restrict__ W16,
                                 float* __restrict__ W32) {
  __shared__ double tile[32][33];
  const int r0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += 8) tile[r][threadIdx.x] = Wt[size_t(r0 + r) * d + c0 + threadIdx.x];
  __syncthreads();
  for (int c = threadIdx.y; c < 32; c += 8) {
    const double v = tile[threadIdx.x][c];
    const size_t o = size_t(c0 + c) * n + r0 + threadIdx.x;
    // one rounding, from the double
    uint16_t b;
    if constexpr (kBf16) {
      // round the double's mantissa to bf16's 8 significant bits, ties to even, on its bit pattern
      unsigned long long u = (unsigned long long)__double_as_longlong(v);
      const unsigned long long lsb = (u >> 45) & 1ull;
      u = (u + ((1ull << 44) - 1ull) + lsb) & ~((1ull << 45) - 1ull);
      b = uint16_t(__float_as_uint(float(__longlong_as_double((long long)u))) >> 16);
    } else {
      b = __half_as_ushort(__double2half(v));
    }
    W16[o] = b;
    if (W32 != nullptr) W32[o] = float(v);
  }
}

// bias[c] = (sy[c] - sum_r sx[r] Wt[r][c]) / T.  Grid = ceil(d / 128), block of 128 threads.
__global__ void fit_bias_kernel(const double* __restrict__ Wt, int n, int d, const double* __restrict__ sx,
                                const double* __restrict__ sy, double T, float* __restrict__ bias) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= d) return;
  double s = sy[c];
  for (int r = 0; r < n; ++r) s -= sx[r] * Wt[size_t(r) * d + c];
  bias[c] = float(s / T);
}

}  // namespace aquakv
