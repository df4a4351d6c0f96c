// Backbone vector quantizer with the four-dimensional grid (Section 4.1 "Alternative quantizers": besides
// the p = 2 grids the paper runs one 2-bit grid with d = 4, n = 256, for which it had no fast GPU kernel;
// its d is the grid dimension).  The steps are those of the p = 2 quantizer (Section 2; the residual / add-back
// steps of Algorithm 2 and Algorithm 3) with consecutive 4-tuples in place of pairs: root-mean-square
// group scale stored as fp16, normalisation with the rounded scale, random signs, Hadamard rotation in
// blocks of h values, nearest of the 256 grid points (lowest index on a tie), one byte per tuple.
//
// One warp per row, the whole row in registers as in the rotated kernels of uniform.cuh: v[c][i] is value
// 256 c + 8 lane + i, so a lane holds the tuples 64 c + 2 lane and 64 c + 2 lane + 1 of every chunk and
// writes their codes as one 16-bit store.  The points sit in shared memory with half their squared norm,
// so a candidate costs four FMAs and a compare: argmin |y - g|^2 = argmin (|g|^2 / 2 - y . g).
//
// Search.  The hypercube [-4, 4)^4 is cut into 32^4 cells of side 1/4.  A table built on the device when
// the context is created (grid4_table_kernel) lists, for every cell, every point that can be the nearest
// one somewhere in the cell: with dmin(g) / dmax(g) the smallest / largest squared distance from the
// (slightly inflated) cell to g and U = min_g dmax(g), the nearest point of any y in the cell has
// dmin <= U, so the list {g : dmin(g) <= U (1 + 1e-4) + 1e-6} in ascending index order contains every
// winner and every point tied with it; evaluating it with a strict "<" gives the result of the
// exhaustive search.  An entry is 16 bytes: up to 15 indices, the last one repeated as padding, and their
// count (4.8 on average for a Gaussian-optimal grid, where the exhaustive loop visits 256); 255 as the
// count marks a cell with more candidates.  Tuples in such a cell or outside the hypercube (6e-5 of the
// coordinates of a normalised row; also every non-finite value) take the exhaustive loop.
#pragma once

#include "uniform.cuh"

namespace aquakv {

struct Grid4Args {
  UniformArgs u;              // X, P, codes, scales, hat, T, d, log_g as for the uniform backbone
  const float4* grid;         // [256] grid points
  const uint4* table;         // [32^4] candidate lists of the cells (grid4_table_kernel); encode only
  const uint32_t* signmask;   // [32]: lane's word, bit 8 c + i set where the sign of value 256 c + 8 lane + i is -1
  int log_h;                  // 6 .. 10
};

struct Grid4Smem {
  float4 g[256];
};

constexpr int kGrid4Cells = 32;             // per dimension
constexpr float kGrid4Lo = -4.0f;           // the table covers [-4, 4)^4
constexpr float kGrid4InvW = 4.0f;          // 1 / cell width
constexpr unsigned kGrid4Overflow = 255u;   // count byte of a cell with more than 15 candidates

__device__ __forceinline__ void grid4_load(Grid4Smem& sm, const float4* grid) {
  for (int k = threadIdx.x; k < 256; k += blockDim.x) sm.g[k] = grid[k];
  __syncthreads();
}

// |g_k|^2 / 2 - y . g_k: the same instruction sequence wherever a candidate is evaluated.  The half norm
// is recomputed from the point (five fp32 operations on an idle pipe) rather than looked up: a second
// shared-memory access at a random index would cost more than it saves.
__device__ __forceinline__ float grid4_score(const Grid4Smem& sm, int k, float y0, float y1, float y2, float y3) {
  const float4 g = sm.g[k];
  const float half_norm = 0.5f * fmaf(g.w, g.w, fmaf(g.z, g.z, fmaf(g.y, g.y, g.x * g.x)));
  float s = fmaf(-y0, g.x, half_norm);
  s = fmaf(-y1, g.y, s);
  s = fmaf(-y2, g.z, s);
  return fmaf(-y3, g.w, s);
}

// Candidate lists of all cells: one thread per cell, distances in double.
__global__ void __launch_bounds__(256) grid4_table_kernel(const float4* __restrict__ grid, uint4* __restrict__ table) {
  __shared__ float4 g[256];
  for (int k = threadIdx.x; k < 256; k += blockDim.x) g[k] = grid[k];
  __syncthreads();
  constexpr int C = kGrid4Cells;
  const long long n_cells = (long long)C * C * C * C;
  for (long long cell = (long long)blockIdx.x * blockDim.x + threadIdx.x; cell < n_cells;
       cell += (long long)gridDim.x * blockDim.x) {
    int idx[4] = {int(cell / (C * C * C)), int(cell / (C * C) % C), int(cell / C % C), int(cell % C)};
    double lo[4], hi[4];
    for (int k = 0; k < 4; ++k) {
      // inflated by 1e-5: the kernel finds the cell of a value with one fp32 rounding
      lo[k] = double(kGrid4Lo) + double(idx[k]) / double(kGrid4InvW) - 1e-5;
      hi[k] = double(kGrid4Lo) + double(idx[k] + 1) / double(kGrid4InvW) + 1e-5;
    }
    auto bounds = [&](int p, double& dmin, double& dmax) {
      const double c[4] = {double(g[p].x), double(g[p].y), double(g[p].z), double(g[p].w)};
      dmin = dmax = 0.0;
      for (int k = 0; k < 4; ++k) {
        const double below = lo[k] - c[k], above = c[k] - hi[k];
        const double out = below > 0.0 ? below : (above > 0.0 ? above : 0.0);
        const double far = fmax(fabs(c[k] - lo[k]), fabs(c[k] - hi[k]));
        dmin += out * out;
        dmax += far * far;
      }
    };
    double U = 1.0e300;
    for (int p = 0; p < 256; ++p) {
      double dmin, dmax;
      bounds(p, dmin, dmax);
      U = fmin(U, dmax);
    }
    const double limit = U * (1.0 + 1e-4) + 1e-6;
    unsigned w[4] = {0u, 0u, 0u, 0u};
    int n = 0, last = 0;
    for (int p = 0; p < 256; ++p) {
      double dmin, dmax;
      bounds(p, dmin, dmax);
      if (dmin <= limit) {
        if (n < 15) w[n >> 2] |= unsigned(p) << (8 * (n & 3));
        last = p;
        ++n;
      }
    }
    if (n > 15) {
      w[3] = (w[3] & 0x00ffffffu) | (kGrid4Overflow << 24);
    } else {
      for (int i = n; i < 15; ++i) w[i >> 2] |= unsigned(last) << (8 * (i & 3));
      w[3] |= unsigned(n) << 24;
    }
    table[cell] = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

// hat = round16(pred + s16 * signs . H(y) / sqrt(h)) for the row's grid points y; sf[c] is the scale of chunk c's group.
template <bool kBf16, int NCH>
__device__ __forceinline__ void grid4_finish(const Grid4Args& ga, long long t, int lane, uint32_t sbits,
                                             float (&y)[NCH][8], const float (&sf)[NCH], const float (&pred)[NCH][8]) {
  uniform_hadamard<NCH>(y, ga.log_h, lane);
  uniform_scale_all<NCH>(y, rsqrtf(float(1 << ga.log_h)));
  uniform_apply_signs<NCH>(y, sbits);
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    float h[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) h[i] = fmaf(y[c][i], sf[c], pred[c][i]);
    uniform_store8<kBf16>(ga.u.hat + t * ga.u.ldHat + 256 * c + 8 * lane, h);
  }
}

template <bool kBf16, int NCH>
__global__ void __launch_bounds__(kUniformWarps * 32)
grid4_encode_rows_kernel(const Grid4Args ga) {
  __shared__ Grid4Smem sm;
  grid4_load(sm, ga.grid);
  const UniformArgs& a = ga.u;
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * kUniformWarps + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * kUniformWarps;
  const int lanes_per_group = a.log_g >= 8 ? 32 : 1 << (a.log_g - 3);
  const int chunks_per_group = a.log_g > 8 ? 1 << (a.log_g - 8) : 1;
  const int n_groups = a.d >> a.log_g;
  const uint32_t sbits = ga.signmask[lane];
  const float rs = rsqrtf(float(1 << ga.log_h));
  const float inv_g = 1.0f / float(1 << a.log_g);
  for (long long t = warp; t < a.T; t += n_warps) {
    float v[NCH][8];
    {
      // the prediction is read again for the reconstruction: holding it through the search would cost 32 registers
      float pred[NCH][8];
      uniform_load_pred_row<NCH, false>(a, t, lane, pred);
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(a.X + t * a.ldX + 256 * c + 8 * lane));
        float lo, hi;
        unpack2(load16x2<kBf16>(raw.x), lo, hi); v[c][0] = lo - pred[c][0]; v[c][1] = hi - pred[c][1];
        unpack2(load16x2<kBf16>(raw.y), lo, hi); v[c][2] = lo - pred[c][2]; v[c][3] = hi - pred[c][3];
        unpack2(load16x2<kBf16>(raw.z), lo, hi); v[c][4] = lo - pred[c][4]; v[c][5] = hi - pred[c][5];
        unpack2(load16x2<kBf16>(raw.w), lo, hi); v[c][6] = lo - pred[c][6]; v[c][7] = hi - pred[c][7];
      }
    }
    // group scale: root mean square of the residual, rounded to fp16; the rounded value normalises
    float ss[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      ss[c] = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) ss[c] = fmaf(v[c][i], v[c][i], ss[c]);
      for (int off = 1; off < lanes_per_group; off <<= 1) ss[c] += __shfl_xor_sync(0xffffffffu, ss[c], off);
    }
    float sf[NCH];
#pragma unroll
    for (int c0 = 0; c0 < NCH; ++c0) {
      float sum = 0.0f;                  // a group of several chunks: the sum over its chunks
#pragma unroll
      for (int c = 0; c < NCH; ++c)
        if ((c & ~(chunks_per_group - 1)) == (c0 & ~(chunks_per_group - 1))) sum += ss[c];
      const __half s16 = __float2half_rn(fminf(sqrtf(sum * inv_g), 65504.0f));
      sf[c0] = __half2float(s16);
      if ((lane & (lanes_per_group - 1)) == 0 && (c0 & (chunks_per_group - 1)) == 0)
        a.scales[t * n_groups + ((256 * c0 + 8 * lane) >> a.log_g)] = __half_as_ushort(s16);
    }
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const float inv = sf[c] > 0.0f ? __fdiv_rn(1.0f, sf[c]) : 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) v[c][i] *= inv;
    }
    uniform_apply_signs<NCH>(v, sbits);
    uniform_hadamard<NCH>(v, ga.log_h, lane);
    uniform_scale_all<NCH>(v, rs);
    // nearest grid point of every 4-tuple: the candidates of the tuple's cell in ascending order, strict "<"
    // keeps the lowest index; the exhaustive loop for what the table does not cover
    uint4 entry[NCH][2];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        int cell = 0;
        bool inside = true;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float f = floorf((v[c][4 * u + k] - kGrid4Lo) * kGrid4InvW);
          inside = inside && f >= 0.0f && f < float(kGrid4Cells);     // false for NaN
          cell = cell * kGrid4Cells + int(fminf(fmaxf(f, 0.0f), float(kGrid4Cells - 1)));
        }
        entry[c][u] = inside ? __ldg(ga.table + cell) : make_uint4(0u, 0u, 0u, kGrid4Overflow << 24);
      }
    }
    int arg[NCH][2];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const float y0 = v[c][4 * u], y1 = v[c][4 * u + 1], y2 = v[c][4 * u + 2], y3 = v[c][4 * u + 3];
        const unsigned n = entry[c][u].w >> 24;
        const bool listed = n != kGrid4Overflow;
        const unsigned n_max = __reduce_max_sync(0xffffffffu, listed ? n : 0u);
        const unsigned words[4] = {entry[c][u].x, entry[c][u].y, entry[c][u].z, entry[c][u].w};
        float best = 3.0e38f;
        int best_k = 0;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
          if (unsigned(4 * w) < n_max) {         // the same for the whole warp; shorter lists repeat their last index
            // the four candidates of a word are scored side by side (independent look-ups), then compared in order
            int k[4];
            float sc[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              k[j] = int((words[w] >> (8 * j)) & 0xffu);
              if (4 * w + j < 15) sc[j] = grid4_score(sm, k[j], y0, y1, y2, y3);
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (4 * w + j < 15 && sc[j] < best) {
                best = sc[j];
                best_k = k[j];
              }
            }
          }
        }
        if (!listed) {
          best = 3.0e38f;
          best_k = 0;
          for (int k = 0; k < 256; ++k) {
            const float sc = grid4_score(sm, k, y0, y1, y2, y3);
            if (sc < best) {
              best = sc;
              best_k = k;
            }
          }
        }
        arg[c][u] = best_k;
      }
    }
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      *reinterpret_cast<uint16_t*>(a.codes + t * (long long)(a.d / 4) + 64 * c + 2 * lane) =
          uint16_t(arg[c][0] | (arg[c][1] << 8));
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const float4 g = sm.g[arg[c][u]];
        v[c][4 * u] = g.x;
        v[c][4 * u + 1] = g.y;
        v[c][4 * u + 2] = g.z;
        v[c][4 * u + 3] = g.w;
      }
    }
    if (a.hat != nullptr) {
      float pred[NCH][8];
      uniform_load_pred_row<NCH>(a, t, lane, pred);
      grid4_finish<kBf16, NCH>(ga, t, lane, sbits, v, sf, pred);
    }
  }
}

template <bool kBf16, int NCH>
__global__ void __launch_bounds__(kUniformWarps * 32)
grid4_decode_rows_kernel(const Grid4Args ga) {
  __shared__ Grid4Smem sm;
  grid4_load(sm, ga.grid);
  const UniformArgs& a = ga.u;
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * kUniformWarps + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * kUniformWarps;
  const int n_groups = a.d >> a.log_g;
  const uint32_t sbits = ga.signmask[lane];
  for (long long t = warp; t < a.T; t += n_warps) {
    float y[NCH][8], pred[NCH][8], sf[NCH];
    uniform_load_pred_row<NCH>(a, t, lane, pred);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const uint32_t two = *reinterpret_cast<const uint16_t*>(a.codes + t * (long long)(a.d / 4) + 64 * c + 2 * lane);
      sf[c] = __half2float(__ushort_as_half(a.scales[t * n_groups + ((256 * c + 8 * lane) >> a.log_g)]));
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const float4 g = sm.g[(two >> (8 * u)) & 0xffu];
        y[c][4 * u] = g.x;
        y[c][4 * u + 1] = g.y;
        y[c][4 * u + 2] = g.z;
        y[c][4 * u + 3] = g.w;
      }
    }
    grid4_finish<kBf16, NCH>(ga, t, lane, sbits, y, sf, pred);
  }
}

}  // namespace aquakv
