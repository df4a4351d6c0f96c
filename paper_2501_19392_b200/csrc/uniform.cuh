// Alternative backbone quantizer (Section 4.1 "Alternative quantizers": the Quanto-style
// one, plain rounding to the nearest level after dividing by the group's largest magnitude, groups of 64
// values inside a token; Section 3.2: any quantizer Q can sit under the predictors) for the residual / add-back steps of
// Algorithm 2 and Algorithm 3.
//
// For b bits per value the levels are the 2^b signed integers -2^(b-1) .. 2^(b-1)-1 times the group
// scale; scale = absmax / 2^(b-1), stored as fp16 (clamped to 65504), and the ROUNDED scale normalises;
// a value goes to the nearest level, the lower one on an exact tie, saturating at the ends; a group of
// zeros has scale 0 and level 0.  The code of a value is level + 2^(b-1); codes are packed LSB-first in
// value order.  No rotation, no sign flips.
//
// Rotated variant (the appendix' additional results for Section 4.1: a backbone that puts a randomized
// Hadamard transform in front of ordinary scalar quantization, one group per row): had_block = h > 1
// multiplies the residual by the role's random signs, rotates every block of h values by the orthonormal
// Hadamard matrix, quantizes the ROTATED values as above (absmax after the rotation), and the inverse
// rotates level * scale back and applies the signs again (kernels uniform_rot_*).
//
// One warp per row.  Lane L holds the 8 consecutive values 256 c + 8 L .. + 7 of every 256-value chunk c
// (16-byte accesses); a group of g <= 256 values is g/8 neighbouring lanes, so its absmax is log2(g/8)
// shuffle steps; a larger group (512 or 1024 values: whole chunks) takes a first pass over its chunks for
// the absmax and reads them again to quantize.  The lane's 8 codes are b contiguous bytes of the row's
// code stream.
#pragma once

#include "codec.cuh"

namespace aquakv {

struct UniformArgs {
  const uint16_t* X;        // encode: target rows (16-bit) [T, ldX]
  long long ldX;
  const float* P;           // prediction rows (fp32) or nullptr [T, ldP]
  long long ldP;
  uint8_t* codes;           // [T, d * b / 8]
  uint16_t* scales;         // [T, d / g] fp16 bits
  uint16_t* hat;            // reconstruction rows or nullptr (encode) [T, ldHat]
  long long ldHat;
  int T;
  int d;                    // 256, 512 or 1024
  int log_g;                // 5 .. 10
};

// |x - pred| maximum of this lane's 8 values of chunk c of row t.
template <bool kBf16>
__device__ __forceinline__ float uniform_chunk_absmax(const UniformArgs& a, long long t, int c, int lane) {
  const int e0 = 256 * c + 8 * lane;
  const uint4 raw = __ldg(reinterpret_cast<const uint4*>(a.X + t * a.ldX + e0));
  float r[8], lo, hi;
  unpack2(load16x2<kBf16>(raw.x), lo, hi); r[0] = lo; r[1] = hi;
  unpack2(load16x2<kBf16>(raw.y), lo, hi); r[2] = lo; r[3] = hi;
  unpack2(load16x2<kBf16>(raw.z), lo, hi); r[4] = lo; r[5] = hi;
  unpack2(load16x2<kBf16>(raw.w), lo, hi); r[6] = lo; r[7] = hi;
  if (a.P != nullptr) {
    const float4 p0 = *reinterpret_cast<const float4*>(a.P + t * a.ldP + e0);
    const float4 p1 = *(reinterpret_cast<const float4*>(a.P + t * a.ldP + e0) + 1);
    r[0] -= p0.x; r[1] -= p0.y; r[2] -= p0.z; r[3] -= p0.w;
    r[4] -= p1.x; r[5] -= p1.y; r[6] -= p1.z; r[7] -= p1.w;
  }
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(r[i]));
  return m;
}

constexpr int kUniformWarps = 4;

template <bool kBf16>
__device__ __forceinline__ void uniform_store8(uint16_t* dst, const float (&v)[8]) {
  uint4 out;
  out.x = store16x2p<kBf16>(pack2(v[0], v[1]));
  out.y = store16x2p<kBf16>(pack2(v[2], v[3]));
  out.z = store16x2p<kBf16>(pack2(v[4], v[5]));
  out.w = store16x2p<kBf16>(pack2(v[6], v[7]));
  __stcs(reinterpret_cast<uint4*>(dst), out);
}

__device__ __forceinline__ void uniform_load_pred8(const float* p, float (&v)[8]) {
  const float4 a = __ldcs(reinterpret_cast<const float4*>(p));
  const float4 b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// codes, scales = Q(x - pred);  hat = round16(pred + Q^-1(codes, scales)).
template <int BITS, bool kBf16>
__global__ void __launch_bounds__(kUniformWarps * 32)
uniform_encode_rows_kernel(const UniformArgs a) {
  constexpr int HALF = 1 << (BITS - 1);
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * kUniformWarps + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * kUniformWarps;
  const int lanes_per_group = a.log_g >= 8 ? 32 : 1 << (a.log_g - 3);
  const int chunks_per_group = a.log_g > 8 ? 1 << (a.log_g - 8) : 1;
  const int n_groups = a.d >> a.log_g;
  for (long long t = warp; t < a.T; t += n_warps) {
    float m_group = 0.0f;      // groups of several chunks: their absmax, found before the first chunk is quantized
    for (int c = 0; c < a.d / 256; ++c) {
      if (chunks_per_group > 1 && (c & (chunks_per_group - 1)) == 0) {
        m_group = 0.0f;
        for (int cc = c; cc < c + chunks_per_group; ++cc) m_group = fmaxf(m_group, uniform_chunk_absmax<kBf16>(a, t, cc, lane));
      }
      const int e0 = 256 * c + 8 * lane;
      float r[8], pred[8];
      {
        const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(a.X + t * a.ldX + e0));
        float lo, hi;
        unpack2(load16x2<kBf16>(raw.x), lo, hi); r[0] = lo; r[1] = hi;
        unpack2(load16x2<kBf16>(raw.y), lo, hi); r[2] = lo; r[3] = hi;
        unpack2(load16x2<kBf16>(raw.z), lo, hi); r[4] = lo; r[5] = hi;
        unpack2(load16x2<kBf16>(raw.w), lo, hi); r[6] = lo; r[7] = hi;
      }
      if (a.P != nullptr) {
        uniform_load_pred8(a.P + t * a.ldP + e0, pred);
#pragma unroll
        for (int i = 0; i < 8; ++i) r[i] -= pred[i];
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) pred[i] = 0.0f;
      }
      float m = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) m = fmaxf(m, fabsf(r[i]));
      if (chunks_per_group > 1) m = m_group;
      for (int off = 1; off < lanes_per_group; off <<= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, off));
      const __half s16 = __float2half_rn(fminf(m * (1.0f / HALF), 65504.0f));
      const float sf = __half2float(s16);
      if ((lane & (lanes_per_group - 1)) == 0 && (c & (chunks_per_group - 1)) == 0)
        a.scales[t * n_groups + ((e0) >> a.log_g)] = __half_as_ushort(s16);
      uint32_t word = 0;
      float q[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        // nearest level, the lower one on a tie: ceil(x - 0.5); the division is IEEE
        const float x = sf > 0.0f ? __fdiv_rn(r[i], sf) : 0.0f;
        float lv = ceilf(x - 0.5f);
        lv = fminf(fmaxf(lv, float(-HALF)), float(HALF - 1));
        q[i] = lv;
        word |= uint32_t(int(lv) + HALF) << (BITS * i);
      }
      uint8_t* cdst = a.codes + t * (long long)(a.d * BITS / 8) + (32 * c + lane) * BITS;
      if constexpr (BITS == 2) {
        *reinterpret_cast<uint16_t*>(cdst) = uint16_t(word);
      } else if constexpr (BITS == 4) {
        *reinterpret_cast<uint32_t*>(cdst) = word;
      } else {
        cdst[0] = uint8_t(word);
        cdst[1] = uint8_t(word >> 8);
        cdst[2] = uint8_t(word >> 16);
      }
      if (a.hat != nullptr) {
        float h[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) h[i] = fmaf(q[i], sf, pred[i]);
        uniform_store8<kBf16>(a.hat + t * a.ldHat + e0, h);
      }
    }
  }
}

// hat = round16(pred + Q^-1(codes, scales)).
template <int BITS, bool kBf16>
__global__ void __launch_bounds__(kUniformWarps * 32)
uniform_decode_rows_kernel(const UniformArgs a) {
  constexpr int HALF = 1 << (BITS - 1);
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * kUniformWarps + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * kUniformWarps;
  const int n_groups = a.d >> a.log_g;
  for (long long t = warp; t < a.T; t += n_warps) {
    for (int c = 0; c < a.d / 256; ++c) {
      const int e0 = 256 * c + 8 * lane;
      const uint8_t* csrc = a.codes + t * (long long)(a.d * BITS / 8) + (32 * c + lane) * BITS;
      uint32_t word;
      if constexpr (BITS == 2) word = *reinterpret_cast<const uint16_t*>(csrc);
      else if constexpr (BITS == 4) word = *reinterpret_cast<const uint32_t*>(csrc);
      else word = uint32_t(csrc[0]) | (uint32_t(csrc[1]) << 8) | (uint32_t(csrc[2]) << 16);
      const float sf = __half2float(__ushort_as_half(a.scales[t * n_groups + (e0 >> a.log_g)]));
      float pred[8], h[8];
      if (a.P != nullptr) {
        uniform_load_pred8(a.P + t * a.ldP + e0, pred);
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) pred[i] = 0.0f;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float lv = float(int((word >> (BITS * i)) & uint32_t((1 << BITS) - 1)) - HALF);
        h[i] = fmaf(lv, sf, pred[i]);
      }
      uniform_store8<kBf16>(a.hat + t * a.ldHat + e0, h);
    }
  }
}

// ---- rotated variant ------------------------------------------------------------------------------
//
// The whole row sits in the warp's registers: v[c][i] is value 256 c + 8 lane + i, so index bits 0-2 are
// register bits, bits 3-7 the lane's bits and bits 8-9 register bits again; a Hadamard block of h = 2^k
// values is one butterfly per index bit below k.

struct UniformRotArgs {
  UniformArgs u;
  const uint32_t* signmask;   // [32]: lane's word, bit 8 c + i set where the sign of value 256 c + 8 lane + i is -1
  int log_h;                  // 6 .. 10
};

template <int NCH>
__device__ __forceinline__ void uniform_hadamard(float (&v)[NCH][8], int log_h, int lane) {
#pragma unroll
  for (int k = 0; k < 3; ++k) {
#pragma unroll
    for (int c = 0; c < NCH; ++c)
#pragma unroll
      for (int i = 0; i < 8; ++i)
        if ((i & (1 << k)) == 0) {
          const float a = v[c][i], b = v[c][i | (1 << k)];
          v[c][i] = a + b;
          v[c][i | (1 << k)] = a - b;
        }
  }
#pragma unroll
  for (int k = 3; k < 8; ++k) {
    if (k < log_h) {
      const int mask = 1 << (k - 3);
      const bool upper = (lane & mask) != 0;
#pragma unroll
      for (int c = 0; c < NCH; ++c)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float other = __shfl_xor_sync(0xffffffffu, v[c][i], mask);
          v[c][i] = upper ? other - v[c][i] : v[c][i] + other;
        }
    }
  }
#pragma unroll
  for (int k = 8; k < 10; ++k) {
    if ((1 << (k - 8)) < NCH && k < log_h) {
#pragma unroll
      for (int c = 0; c < NCH; ++c)
        if ((c & (1 << (k - 8))) == 0) {
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float a = v[c][i], b = v[c | (1 << (k - 8))][i];
            v[c][i] = a + b;
            v[c | (1 << (k - 8))][i] = a - b;
          }
        }
    }
  }
}

// Negates the values whose sign bit is set.
template <int NCH>
__device__ __forceinline__ void uniform_apply_signs(float (&v)[NCH][8], uint32_t bits) {
#pragma unroll
  for (int c = 0; c < NCH; ++c)
#pragma unroll
    for (int i = 0; i < 8; ++i)
      if ((bits >> (8 * c + i)) & 1u) v[c][i] = -v[c][i];
}

template <int NCH>
__device__ __forceinline__ void uniform_scale_all(float (&v)[NCH][8], float f) {
#pragma unroll
  for (int c = 0; c < NCH; ++c)
#pragma unroll
    for (int i = 0; i < 8; ++i) v[c][i] *= f;
}

// kStream: the last read of the prediction (evict-first); otherwise it stays cached for a second read.
template <int NCH, bool kStream = true>
__device__ __forceinline__ void uniform_load_pred_row(const UniformArgs& a, long long t, int lane, float (&pred)[NCH][8]) {
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    if (a.P != nullptr) {
      if constexpr (kStream) {
        uniform_load_pred8(a.P + t * a.ldP + 256 * c + 8 * lane, pred[c]);
      } else {
        const float4* p = reinterpret_cast<const float4*>(a.P + t * a.ldP + 256 * c + 8 * lane);
        const float4 lo = p[0], hi = p[1];
        pred[c][0] = lo.x; pred[c][1] = lo.y; pred[c][2] = lo.z; pred[c][3] = lo.w;
        pred[c][4] = hi.x; pred[c][5] = hi.y; pred[c][6] = hi.z; pred[c][7] = hi.w;
      }
    } else {
#pragma unroll
      for (int i = 0; i < 8; ++i) pred[c][i] = 0.0f;
    }
  }
}

// hat = round16(pred + signs . H(y) / sqrt(h)) for the row's level * scale values y.
template <bool kBf16, int NCH>
__device__ __forceinline__ void uniform_rot_finish(const UniformRotArgs& ra, long long t, int lane, uint32_t sbits,
                                                   float (&y)[NCH][8], const float (&pred)[NCH][8]) {
  uniform_hadamard<NCH>(y, ra.log_h, lane);
  uniform_scale_all<NCH>(y, rsqrtf(float(1 << ra.log_h)));
  uniform_apply_signs<NCH>(y, sbits);
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    float h[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) h[i] = y[c][i] + pred[c][i];
    uniform_store8<kBf16>(ra.u.hat + t * ra.u.ldHat + 256 * c + 8 * lane, h);
  }
}

template <int BITS, bool kBf16, int NCH>
__global__ void __launch_bounds__(kUniformWarps * 32)
uniform_rot_encode_rows_kernel(const UniformRotArgs ra) {
  constexpr int HALF = 1 << (BITS - 1);
  const UniformArgs& a = ra.u;
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * kUniformWarps + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * kUniformWarps;
  const int lanes_per_group = a.log_g >= 8 ? 32 : 1 << (a.log_g - 3);
  const int chunks_per_group = a.log_g > 8 ? 1 << (a.log_g - 8) : 1;
  const int n_groups = a.d >> a.log_g;
  const uint32_t sbits = ra.signmask[lane];
  const float rs = rsqrtf(float(1 << ra.log_h));
  for (long long t = warp; t < a.T; t += n_warps) {
    float v[NCH][8], pred[NCH][8];
    uniform_load_pred_row<NCH>(a, t, lane, pred);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(a.X + t * a.ldX + 256 * c + 8 * lane));
      float lo, hi;
      unpack2(load16x2<kBf16>(raw.x), lo, hi); v[c][0] = lo - pred[c][0]; v[c][1] = hi - pred[c][1];
      unpack2(load16x2<kBf16>(raw.y), lo, hi); v[c][2] = lo - pred[c][2]; v[c][3] = hi - pred[c][3];
      unpack2(load16x2<kBf16>(raw.z), lo, hi); v[c][4] = lo - pred[c][4]; v[c][5] = hi - pred[c][5];
      unpack2(load16x2<kBf16>(raw.w), lo, hi); v[c][6] = lo - pred[c][6]; v[c][7] = hi - pred[c][7];
    }
    uniform_apply_signs<NCH>(v, sbits);
    uniform_hadamard<NCH>(v, ra.log_h, lane);
    uniform_scale_all<NCH>(v, rs);
    // group absmax of the rotated values
    float m[NCH];
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      m[c] = 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) m[c] = fmaxf(m[c], fabsf(v[c][i]));
      for (int off = 1; off < lanes_per_group; off <<= 1) m[c] = fmaxf(m[c], __shfl_xor_sync(0xffffffffu, m[c], off));
    }
    // a group of several chunks: the maximum over its chunks (mg is a second array: m is read in full)
    float mg[NCH];
#pragma unroll
    for (int c0 = 0; c0 < NCH; ++c0) {
      mg[c0] = 0.0f;
#pragma unroll
      for (int c = 0; c < NCH; ++c)
        if ((c & ~(chunks_per_group - 1)) == (c0 & ~(chunks_per_group - 1))) mg[c0] = fmaxf(mg[c0], m[c]);
    }
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int e0 = 256 * c + 8 * lane;
      const __half s16 = __float2half_rn(fminf(mg[c] * (1.0f / HALF), 65504.0f));
      const float sf = __half2float(s16);
      if ((lane & (lanes_per_group - 1)) == 0 && (c & (chunks_per_group - 1)) == 0)
        a.scales[t * n_groups + (e0 >> a.log_g)] = __half_as_ushort(s16);
      uint32_t word = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float x = sf > 0.0f ? __fdiv_rn(v[c][i], sf) : 0.0f;
        float lv = ceilf(x - 0.5f);
        lv = fminf(fmaxf(lv, float(-HALF)), float(HALF - 1));
        v[c][i] = lv * sf;
        word |= uint32_t(int(lv) + HALF) << (BITS * i);
      }
      uint8_t* cdst = a.codes + t * (long long)(a.d * BITS / 8) + (32 * c + lane) * BITS;
      if constexpr (BITS == 2) {
        *reinterpret_cast<uint16_t*>(cdst) = uint16_t(word);
      } else if constexpr (BITS == 4) {
        *reinterpret_cast<uint32_t*>(cdst) = word;
      } else {
        cdst[0] = uint8_t(word);
        cdst[1] = uint8_t(word >> 8);
        cdst[2] = uint8_t(word >> 16);
      }
    }
    if (a.hat != nullptr) uniform_rot_finish<kBf16, NCH>(ra, t, lane, sbits, v, pred);
  }
}

template <int BITS, bool kBf16, int NCH>
__global__ void __launch_bounds__(kUniformWarps * 32)
uniform_rot_decode_rows_kernel(const UniformRotArgs ra) {
  constexpr int HALF = 1 << (BITS - 1);
  const UniformArgs& a = ra.u;
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * kUniformWarps + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * kUniformWarps;
  const int n_groups = a.d >> a.log_g;
  const uint32_t sbits = ra.signmask[lane];
  for (long long t = warp; t < a.T; t += n_warps) {
    float y[NCH][8], pred[NCH][8];
    uniform_load_pred_row<NCH>(a, t, lane, pred);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const int e0 = 256 * c + 8 * lane;
      const uint8_t* csrc = a.codes + t * (long long)(a.d * BITS / 8) + (32 * c + lane) * BITS;
      uint32_t word;
      if constexpr (BITS == 2) word = *reinterpret_cast<const uint16_t*>(csrc);
      else if constexpr (BITS == 4) word = *reinterpret_cast<const uint32_t*>(csrc);
      else word = uint32_t(csrc[0]) | (uint32_t(csrc[1]) << 8) | (uint32_t(csrc[2]) << 16);
      const float sf = __half2float(__ushort_as_half(a.scales[t * n_groups + (e0 >> a.log_g)]));
#pragma unroll
      for (int i = 0; i < 8; ++i)
        y[c][i] = float(int((word >> (BITS * i)) & uint32_t((1 << BITS) - 1)) - HALF) * sf;
    }
    uniform_rot_finish<kBf16, NCH>(ra, t, lane, sbits, y, pred);
  }
}

}  // namespace aquakv
