// Row kernels of the backbone quantizer Q / Q^-1 (Section 2 "Vector Quantization", Section 4.1
// "Alternative quantizers": group scale, randomized Hadamard transform, nearest point of a fixed
// 2-D grid, packed codes) and of the residual / add-back steps of Algorithm 2 (lines 6-7, 9) and
// Algorithm 3 (lines 5, 7).
//
// One warp owns one token row.  Element e of the row lives in lane (e/8)%32, register
// (e/256)*8 + e%8, so every global access is a 16-byte (16-bit data) or 2x16-byte (fp32) vector
// per lane and a warp touches whole 128-byte lines.  The Hadamard butterflies over index bits
// 0-2 and 8-9 are register-local, bits 3-7 are warp shuffles.  The value pair (2j, 2j+1) that
// shares one code always sits in one lane.
#pragma once

#include "common.cuh"

namespace aquakv {

constexpr int kCodecWarps = 8;
constexpr int kCodecThreads = kCodecWarps * 32;

// Grid in kernel-parameter (constant) space for the unrolled nearest-point search:
// score_i(y) = hn[i] + nx[i]*y0 + ny[i]*y1 with nx = -g_x, ny = -g_y, hn = |g|^2 / 2, whose
// argmin over i is the nearest grid point.
template <int N>
struct GridConst {
  float nx[N];
  float ny[N];
  float hn[N];
};

struct CodecArgs {
  const uint16_t* X;        // encode: target rows (16-bit)              [T, ldX]
  long long ldX;
  const float* P;           // prediction rows (fp32) or nullptr          [T, ldP]
  long long ldP;
  const uint32_t* signmask; // [32]: bit (c*8+i) of entry `lane` set <=> sign of element
                            //       c*256 + lane*8 + i is -1
  const float4* grid4;      // [n]: (g_x, g_y, |g|^2/2, 0)
  uint8_t* codes;           // [T, code_bytes]
  uint16_t* scales;         // [T, D/G] fp16 bits
  uint16_t* hat;            // reconstruction rows (16-bit) or nullptr    [T, ldHat]
  long long ldHat;
  int T;
  int log_h;                // log2 of the Hadamard block
  int log_g;                // log2 of the scale group
};

template <int NV>
__device__ __forceinline__ void fwht_regs_and_lanes(float (&v)[NV], int log_h, int lane) {
  // index bits 0..2: inside each 8-element register chunk (h >= 64, so always applied)
#pragma unroll
  for (int b = 0; b < 3; ++b) {
#pragma unroll
    for (int i = 0; i < NV; ++i) {
      if ((i & (1 << b)) == 0) {
        const float a = v[i], c = v[i | (1 << b)];
        v[i] = a + c;
        v[i | (1 << b)] = a - c;
      }
    }
  }
  // index bits 3..7: lane bits 0..4
#pragma unroll
  for (int b = 3; b < 8; ++b) {
    if (b < log_h) {
      const int m = 1 << (b - 3);
      const float sg = (lane & m) ? -1.0f : 1.0f;
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        const float o = __shfl_xor_sync(0xffffffffu, v[i], m);
        v[i] = fmaf(sg, v[i], o);   // lower partner: v + o; upper partner: o - v (both exact adds)
      }
    }
  }
  // index bits 8..9: register chunk index
#pragma unroll
  for (int b = 8; b < 10; ++b) {
    if ((NV >> 3) > (1 << (b - 8)) && b < log_h) {
      const int cm = 1 << (b - 8);
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        if (((i >> 3) & cm) == 0) {
          const int j = i + (cm << 3);
          if (j < NV) {
            const float a = v[i], c = v[j];
            v[i] = a + c;
            v[j] = a - c;
          }
        }
      }
    }
  }
}

__device__ __forceinline__ float apply_sign(float x, uint32_t mask, int i) {
  // flips the sign bit of x when bit i of mask is set
  return __uint_as_float(__float_as_uint(x) ^ ((mask << (31 - i)) & 0x80000000u));
}

// Q^-1 without the prediction: grid points of this lane's codes -> inverse rotation -> scale.
// `w` enters holding the gathered grid coordinates and leaves holding xhat.  The exact operation
// order (multiply by 1/sqrt(h), then by the scale, sign flip) is shared by encode and decode so
// that both produce bit-identical reconstructions.
template <int NV>
__device__ __forceinline__ void rotate_back_and_scale(float (&w)[NV], const float (&sf)[NV / 8],
                                                      uint32_t signmask, int log_h, int lane) {
  fwht_regs_and_lanes<NV>(w, log_h, lane);
  const float rs = exp2f(-0.5f * static_cast<float>(log_h));   // exact for even log_h
#pragma unroll
  for (int i = 0; i < NV; ++i)
    w[i] = apply_sign(__fmul_rn(__fmul_rn(w[i], rs), sf[i >> 3]), signmask, i);
}

template <int BITS>
__device__ __forceinline__ uint32_t load_code_word(const uint8_t* row_codes, int chunk, int lane) {
  const int idx = chunk * 32 + lane;   // 8 values = 4 codes = 4*BITS bits per (chunk, lane)
  if constexpr (BITS == 4) {
    return *reinterpret_cast<const uint16_t*>(row_codes + idx * 2);
  } else if constexpr (BITS == 8) {
    return *reinterpret_cast<const uint32_t*>(row_codes + idx * 4);
  } else {
    const uint8_t* p = row_codes + idx * 3;
    return uint32_t(p[0]) | (uint32_t(p[1]) << 8) | (uint32_t(p[2]) << 16);
  }
}

template <int BITS>
__device__ __forceinline__ void store_code_word(uint8_t* row_codes, int chunk, int lane, uint32_t w) {
  const int idx = chunk * 32 + lane;
  if constexpr (BITS == 4) {
    *reinterpret_cast<uint16_t*>(row_codes + idx * 2) = static_cast<uint16_t>(w);
  } else if constexpr (BITS == 8) {
    *reinterpret_cast<uint32_t*>(row_codes + idx * 4) = w;
  } else {
    uint8_t* p = row_codes + idx * 3;
    p[0] = static_cast<uint8_t>(w);
    p[1] = static_cast<uint8_t>(w >> 8);
    p[2] = static_cast<uint8_t>(w >> 16);
  }
}

// Sum of squares of each scale group, delivered to every lane for each of its register chunks.
template <int NC>
__device__ __forceinline__ void group_sums(const float (&v)[NC * 8], float (&ss)[NC], int log_g) {
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    float s = 0.0f;
#pragma unroll
    for (int i = 0; i < 8; ++i) s = fmaf(v[c * 8 + i], v[c * 8 + i], s);
#pragma unroll
    for (int b = 3; b < 8; ++b)
      if (b < log_g) s += __shfl_xor_sync(0xffffffffu, s, 1 << (b - 3));
    ss[c] = s;
  }
  if (log_g > 8) {
    const int cpg = 1 << (log_g - 8);   // register chunks per group
    float tot[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      float s = 0.0f;
#pragma unroll
      for (int c2 = 0; c2 < NC; ++c2)
        if ((c2 / cpg) == (c / cpg)) s += ss[c2];
      tot[c] = s;
    }
#pragma unroll
    for (int c = 0; c < NC; ++c) ss[c] = tot[c];
  }
}

template <int D, int NPTS, bool kBf16>
__global__ void __launch_bounds__(kCodecThreads)
encode_rows_kernel(const __grid_constant__ GridConst<(NPTS <= 64 ? NPTS : 1)> gc, const CodecArgs a) {
  constexpr int NC = D / 256, NV = NC * 8;
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = D / 2 * BITS / 8;
  __shared__ float4 grid_s[NPTS];
  for (int i = threadIdx.x; i < NPTS; i += blockDim.x) grid_s[i] = a.grid4[i];
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t signmask = a.signmask[lane];
  const int n_groups = D >> a.log_g;
  const float inv_g = exp2f(-static_cast<float>(a.log_g));
  const float rs = exp2f(-0.5f * static_cast<float>(a.log_h));

  for (long long row = (long long)blockIdx.x * kCodecWarps + warp; row < a.T;
       row += (long long)gridDim.x * kCodecWarps) {
    float v[NV], p[NV];
    // ---- residual r = x - pred (Algorithm 2 line 6 / 9) -------------------------------------
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const int e0 = c * 256 + lane * 8;
      const uint4 raw = *reinterpret_cast<const uint4*>(a.X + row * a.ldX + e0);
      const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
      if (a.P != nullptr) {
        const float4 p0 = *reinterpret_cast<const float4*>(a.P + row * a.ldP + e0);
        const float4 p1 = *reinterpret_cast<const float4*>(a.P + row * a.ldP + e0 + 4);
        p[c * 8 + 0] = p0.x; p[c * 8 + 1] = p0.y; p[c * 8 + 2] = p0.z; p[c * 8 + 3] = p0.w;
        p[c * 8 + 4] = p1.x; p[c * 8 + 5] = p1.y; p[c * 8 + 6] = p1.z; p[c * 8 + 7] = p1.w;
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) p[c * 8 + i] = 0.0f;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[c * 8 + 2 * i] = __fsub_rn(load16<kBf16>(uint16_t(w[i] & 0xffffu)), p[c * 8 + 2 * i]);
        v[c * 8 + 2 * i + 1] = __fsub_rn(load16<kBf16>(uint16_t(w[i] >> 16)), p[c * 8 + 2 * i + 1]);
      }
    }
    // ---- group scale: root mean square, stored as fp16; normalise with the rounded value ----
    float ss[NC], sf[NC];
    group_sums<NC>(v, ss, a.log_g);
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const float s = fminf(sqrtf(ss[c] * inv_g), 65504.0f);
      const __half s16 = __float2half_rn(s);
      sf[c] = __half2float(s16);
      // one lane per group writes the scale
      if (a.log_g >= 8) {
        const int cpg = 1 << (a.log_g - 8);
        if (lane == 0 && (c % cpg) == 0) a.scales[row * n_groups + c / cpg] = __half_as_ushort(s16);
      } else {
        const int lpg = 1 << (a.log_g - 3);   // lanes per group
        if ((lane % lpg) == 0)
          a.scales[row * n_groups + c * (256 >> a.log_g) + lane / lpg] = __half_as_ushort(s16);
      }
      const float inv = sf[c] > 0.0f ? 1.0f / sf[c] : 0.0f;
#pragma unroll
      for (int i = 0; i < 8; ++i) v[c * 8 + i] = apply_sign(v[c * 8 + i] * inv, signmask, c * 8 + i);
    }
    // ---- rotate -------------------------------------------------------------------------------
    fwht_regs_and_lanes<NV>(v, a.log_h, lane);
    // ---- nearest grid point per pair, pack, gather the chosen points --------------------------
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      uint32_t word = 0;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float y0 = v[c * 8 + 2 * k] * rs, y1 = v[c * 8 + 2 * k + 1] * rs;
        int idx = 0;
        if constexpr (NPTS <= 64) {
          float best = fmaf(gc.ny[0], y1, fmaf(gc.nx[0], y0, gc.hn[0]));
#pragma unroll
          for (int i = 1; i < NPTS; ++i) {
            const float t = fmaf(gc.ny[i], y1, fmaf(gc.nx[i], y0, gc.hn[i]));
            if (t < best) { best = t; idx = i; }     // strict: lowest index wins ties
          }
        } else {
          float best = 3.0e38f;
          for (int i = 0; i < NPTS; ++i) {
            const float4 g = grid_s[i];
            const float t = fmaf(-g.y, y1, fmaf(-g.x, y0, g.z));
            if (t < best) { best = t; idx = i; }
          }
        }
        word |= uint32_t(idx) << (k * BITS);
        const float4 g = grid_s[idx];
        v[c * 8 + 2 * k] = g.x;
        v[c * 8 + 2 * k + 1] = g.y;
      }
      store_code_word<BITS>(a.codes + row * CODE_BYTES, c, lane, word);
    }
    // ---- reconstruction (Algorithm 2 line 7): hat = round16(pred + Q^-1(codes)) ---------------
    if (a.hat != nullptr) {
      rotate_back_and_scale<NV>(v, sf, signmask, a.log_h, lane);
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const uint32_t lo = store16<kBf16>(__fadd_rn(p[c * 8 + 2 * i], v[c * 8 + 2 * i]));
          const uint32_t hi = store16<kBf16>(__fadd_rn(p[c * 8 + 2 * i + 1], v[c * 8 + 2 * i + 1]));
          o[i] = lo | (hi << 16);
        }
        *reinterpret_cast<uint4*>(a.hat + row * a.ldHat + c * 256 + lane * 8) =
            make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  }
}

// Algorithm 3 line 5 / 7 given the prediction: hat = round16(pred + Q^-1(codes, scales)).
template <int D, int NPTS, bool kBf16>
__global__ void __launch_bounds__(kCodecThreads) decode_rows_kernel(const CodecArgs a) {
  constexpr int NC = D / 256, NV = NC * 8;
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = D / 2 * BITS / 8;
  __shared__ float2 grid_s[NPTS];
  for (int i = threadIdx.x; i < NPTS; i += blockDim.x) {
    const float4 g = a.grid4[i];
    grid_s[i] = make_float2(g.x, g.y);
  }
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t signmask = a.signmask[lane];
  const int n_groups = D >> a.log_g;

  for (long long row = (long long)blockIdx.x * kCodecWarps + warp; row < a.T;
       row += (long long)gridDim.x * kCodecWarps) {
    float w[NV], sf[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const uint32_t word = load_code_word<BITS>(a.codes + row * CODE_BYTES, c, lane);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const float2 g = grid_s[(word >> (k * BITS)) & (NPTS - 1)];
        w[c * 8 + 2 * k] = g.x;
        w[c * 8 + 2 * k + 1] = g.y;
      }
      const int e0 = c * 256 + lane * 8;
      sf[c] = __half2float(__ushort_as_half(a.scales[row * n_groups + (e0 >> a.log_g)]));
    }
    rotate_back_and_scale<NV>(w, sf, signmask, a.log_h, lane);
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const int e0 = c * 256 + lane * 8;
      float p[8];
      if (a.P != nullptr) {
        const float4 p0 = *reinterpret_cast<const float4*>(a.P + row * a.ldP + e0);
        const float4 p1 = *reinterpret_cast<const float4*>(a.P + row * a.ldP + e0 + 4);
        p[0] = p0.x; p[1] = p0.y; p[2] = p0.z; p[3] = p0.w;
        p[4] = p1.x; p[5] = p1.y; p[6] = p1.z; p[7] = p1.w;
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i) p[i] = 0.0f;
      }
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t lo = store16<kBf16>(__fadd_rn(p[2 * i], w[c * 8 + 2 * i]));
        const uint32_t hi = store16<kBf16>(__fadd_rn(p[2 * i + 1], w[c * 8 + 2 * i + 1]));
        o[i] = lo | (hi << 16);
      }
      *reinterpret_cast<uint4*>(a.hat + row * a.ldHat + e0) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

}  // namespace aquakv
