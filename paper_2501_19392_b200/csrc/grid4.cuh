// Backbone vector quantizer with the four-dimensional grid (Section 4.1 "Alternative quantizers": besides
// the p = 2 grids the paper runs "one grid without fast GPU support (2-bit precision, d = 4, n = 256)";
// its d is the grid dimension).  The steps are those of the p = 2 quantizer (Section 2; Algorithm 2
// lines 6-7, 9 and Algorithm 3 lines 5, 7) with consecutive 4-tuples in place of pairs: root-mean-square
// group scale stored as fp16, normalisation with the rounded scale, random signs, Hadamard rotation in
// blocks of h values, nearest of the 256 grid points (lowest index on a tie), one byte per tuple.
//
// One warp per row, the whole row in registers as in the rotated kernels of uniform.cuh: v[c][i] is value
// 256 c + 8 lane + i, so a lane holds the tuples 64 c + 2 lane and 64 c + 2 lane + 1 of every chunk and
// writes their codes as one 16-bit store.  The search is exhaustive: a 256-point grid in four dimensions
// has no cheap cell structure like the planar grids' table, and this grid is the paper's slow one.  The
// points sit in shared memory with half their squared norm, so a candidate costs four FMAs and a
// compare: argmin |y - g|^2 = argmin (|g|^2 / 2 - y . g).  A lane's two tuples of a chunk go through the
// packed two-lane fp32 FMA together (each lane rounds like the scalar instruction), which is why the
// encoder's copy of the grid holds every coordinate twice.
#pragma once

#include "uniform.cuh"

namespace aquakv {

struct Grid4Args {
  UniformArgs u;              // X, P, codes, scales, hat, T, d, log_g as for the uniform backbone
  const float4* grid;         // [256] grid points
  const uint32_t* signmask;   // [32]: lane's word, bit 8 c + i set where the sign of value 256 c + 8 lane + i is -1
  int log_h;                  // 6 .. 10
};

struct Grid4Smem {
  float4 g[256];
};

// The encoder's search copy: (x, x, y, y), (z, z, w, w) and (|g|^2 / 2, |g|^2 / 2) per point.
struct Grid4SearchSmem {
  float4 xy[256];
  float4 zw[256];
  float2 half_norm[256];
};

__device__ __forceinline__ void grid4_load(Grid4Smem& sm, const float4* grid) {
  for (int k = threadIdx.x; k < 256; k += blockDim.x) sm.g[k] = grid[k];
  __syncthreads();
}

__device__ __forceinline__ void grid4_load_search(Grid4SearchSmem& ss, const float4* grid) {
  for (int k = threadIdx.x; k < 256; k += blockDim.x) {
    const float4 p = grid[k];
    ss.xy[k] = make_float4(p.x, p.x, p.y, p.y);
    ss.zw[k] = make_float4(p.z, p.z, p.w, p.w);
    const float hn = 0.5f * (p.x * p.x + p.y * p.y + p.z * p.z + p.w * p.w);
    ss.half_norm[k] = make_float2(hn, hn);
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
  __shared__ Grid4SearchSmem ss_grid;
  grid4_load_search(ss_grid, ga.grid);
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
    // nearest grid point of every 4-tuple: exhaustive, candidates in ascending order, strict "<" keeps the lowest index
    float best[NCH][2];
    int arg[NCH][2];
    f32x2_t ny[NCH][4];                  // (-y_j of the first tuple, -y_j of the second) for j = 0 .. 3
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      best[c][0] = best[c][1] = 3.0e38f;
      arg[c][0] = arg[c][1] = 0;
#pragma unroll
      for (int j = 0; j < 4; ++j) ny[c][j] = pack2(-v[c][j], -v[c][4 + j]);
    }
#pragma unroll 2
    for (int k = 0; k < 256; ++k) {
      const float4 gxy = ss_grid.xy[k], gzw = ss_grid.zw[k];
      const float2 hn = ss_grid.half_norm[k];
      const f32x2_t gx = pack2(gxy.x, gxy.y), gy = pack2(gxy.z, gxy.w), gz = pack2(gzw.x, gzw.y), gw = pack2(gzw.z, gzw.w);
      const f32x2_t h2 = pack2(hn.x, hn.y);
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        f32x2_t s2 = fma2(ny[c][0], gx, h2);
        s2 = fma2(ny[c][1], gy, s2);
        s2 = fma2(ny[c][2], gz, s2);
        s2 = fma2(ny[c][3], gw, s2);
        float s0, s1;
        unpack2(s2, s0, s1);
        if (s0 < best[c][0]) {
          best[c][0] = s0;
          arg[c][0] = k;
        }
        if (s1 < best[c][1]) {
          best[c][1] = s1;
          arg[c][1] = k;
        }
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
