// Single-query grouped-query attention over freshly decoded keys/values (Algorithm 4 lines 5-9:
// the block attends to the recovered cache).  Split-KV: one CTA reduces a block of consecutive
// tokens of one sequence to per-query-head partials (running max, sum, unnormalised output), a
// second kernel merges the partials of a sequence by log-sum-exp.  All accumulation is fp32.
//
// One CTA owns (token block, KV head) and up to four of that KV head's query heads at once, so
// K/V bytes are read once per KV head.  Inside a warp, 8 lanes share one token (each lane owns
// HD/8 head dimensions as 16-byte pieces) and the 4 lane groups take consecutive tokens; the 8
// warps interleave over the block's tokens and merge through shared memory.
#pragma once

#include "common.cuh"

namespace aquakv {

constexpr int kAttnWarps = 8;
constexpr int kAttnThreads = kAttnWarps * 32;
constexpr int kAttnMaxGq = 4;       // query heads per KV head processed by one pass
constexpr float kNegBig = -1.0e30f;

struct AttnArgs {
  const uint16_t* q;      // [batch][n_q_heads][HD]
  const uint16_t* Kh;     // decoded keys, row r = global token (tok_base + r)   [*, ld]
  const uint16_t* Vh;
  long long ld;
  long long tok_base;
  long long blk_begin;    // first global block (sequence * n_splits + split) of this launch
  int ctx;                // tokens per sequence
  int n_q_heads;
  int n_kv_heads;
  int n_splits;           // blocks per sequence
  int block_tokens;       // tokens per block
  float scale_log2;       // softmax_scale * log2(e)
  float* part_ml;         // [batch][n_splits][n_q_heads][2]  (max in log2 units, sum)
  float* part_o;          // [batch][n_splits][n_q_heads][HD]
};

template <bool kBf16>
__device__ __forceinline__ void unpack8(const uint4& raw, float (&f)[8]) {
  const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    f[2 * i] = load16<kBf16>(uint16_t(w[i] & 0xffffu));
    f[2 * i + 1] = load16<kBf16>(uint16_t(w[i] >> 16));
  }
}

template <int HD, int GQ, bool kBf16>
__global__ void __launch_bounds__(kAttnThreads, 2) attn_partial_kernel(const AttnArgs a) {
  constexpr int NP = HD / 64;          // 16-byte pieces per lane per row (8 dims each)
  constexpr int DPL = NP * 8;          // dims per lane
  __shared__ float sm_m[kAttnWarps][GQ];
  __shared__ float sm_l[kAttnWarps][GQ];
  __shared__ float sm_o[kAttnWarps][GQ][HD];
  __shared__ float sm_q[GQ][HD];       // queries, pre-multiplied by softmax_scale * log2(e)
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int tg = lane >> 3, dl = lane & 7;
  const long long gb = a.blk_begin + blockIdx.x;
  const int b = int(gb / a.n_splits), split = int(gb % a.n_splits);
  const int t_begin = split * a.block_tokens;
  const int t_end = min(a.ctx, t_begin + a.block_tokens);
  const int rep = a.n_q_heads / a.n_kv_heads;
  const int kvh = blockIdx.y;
  const int g0 = blockIdx.z * GQ;      // first query head (within the KV group) of this pass

  for (int idx = threadIdx.x; idx < GQ * HD; idx += kAttnThreads) {
    const int g = idx / HD, i = idx % HD;
    const uint16_t qb = a.q[((long long)b * a.n_q_heads + kvh * rep + g0 + g) * HD + i];
    sm_q[g][i] = load16<kBf16>(qb) * a.scale_log2;
  }
  __syncthreads();

  float m[GQ], l[GQ], acc[GQ][DPL];
#pragma unroll
  for (int g = 0; g < GQ; ++g) {
    m[g] = kNegBig;
    l[g] = 0.0f;
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[g][i] = 0.0f;
  }
  const long long row0 = (long long)b * a.ctx - a.tok_base;
  // warp w takes tokens t_begin + 4*(w + 8*j) + {0,1,2,3}; its four lane groups take one each.
  // The next iteration's key/value pieces are fetched before the current ones are used.
  uint4 kraw[NP], vraw[NP], kraw_n[NP], vraw_n[NP];
  auto fetch = [&](int tb, uint4 (&kr)[NP], uint4 (&vr)[NP]) {
    const int t = tb + tg;
    const long long row = row0 + (t < t_end ? t : t_begin);
    const uint16_t* kp = a.Kh + row * a.ld + kvh * HD + dl * 8;
    const uint16_t* vp = a.Vh + row * a.ld + kvh * HD + dl * 8;
#pragma unroll
    for (int pc = 0; pc < NP; ++pc) {
      kr[pc] = __ldcs(reinterpret_cast<const uint4*>(kp + pc * 64));
      vr[pc] = __ldcs(reinterpret_cast<const uint4*>(vp + pc * 64));
    }
  };
  int tb = t_begin + warp * 4;
  if (tb < t_end) fetch(tb, kraw, vraw);
  for (; tb < t_end; tb += 4 * kAttnWarps) {
    const int tbn = tb + 4 * kAttnWarps;
    if (tbn < t_end) fetch(tbn, kraw_n, vraw_n);
    const bool valid = tb + tg < t_end;
    float kf[DPL], vf[DPL];
#pragma unroll
    for (int pc = 0; pc < NP; ++pc) {
      float f[8];
      unpack8<kBf16>(kraw[pc], f);
#pragma unroll
      for (int i = 0; i < 8; ++i) kf[pc * 8 + i] = f[i];
      unpack8<kBf16>(vraw[pc], f);
#pragma unroll
      for (int i = 0; i < 8; ++i) vf[pc * 8 + i] = f[i];
    }
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
      float s = 0.0f;
#pragma unroll
      for (int pc = 0; pc < NP; ++pc) {
        const float4 q0 = *reinterpret_cast<const float4*>(&sm_q[g][pc * 64 + dl * 8]);
        const float4 q1 = *reinterpret_cast<const float4*>(&sm_q[g][pc * 64 + dl * 8 + 4]);
        s = fmaf(q0.x, kf[pc * 8 + 0], s); s = fmaf(q0.y, kf[pc * 8 + 1], s);
        s = fmaf(q0.z, kf[pc * 8 + 2], s); s = fmaf(q0.w, kf[pc * 8 + 3], s);
        s = fmaf(q1.x, kf[pc * 8 + 4], s); s = fmaf(q1.y, kf[pc * 8 + 5], s);
        s = fmaf(q1.z, kf[pc * 8 + 6], s); s = fmaf(q1.w, kf[pc * 8 + 7], s);
      }
      s += __shfl_xor_sync(0xffffffffu, s, 1);
      s += __shfl_xor_sync(0xffffffffu, s, 2);
      s += __shfl_xor_sync(0xffffffffu, s, 4);
      if (valid) {
        const float m_new = fmaxf(m[g], s);
        const float corr = exp2f(m[g] - m_new);
        const float pr = exp2f(s - m_new);
        m[g] = m_new;
        l[g] = fmaf(l[g], corr, pr);
#pragma unroll
        for (int i = 0; i < DPL; ++i) acc[g][i] = fmaf(acc[g][i], corr, pr * vf[i]);
      }
    }
#pragma unroll
    for (int pc = 0; pc < NP; ++pc) {
      kraw[pc] = kraw_n[pc];
      vraw[pc] = vraw_n[pc];
    }
  }
  // merge the four token groups of the warp
#pragma unroll
  for (int mask = 8; mask <= 16; mask <<= 1) {
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
      const float m_o = __shfl_xor_sync(0xffffffffu, m[g], mask);
      const float l_o = __shfl_xor_sync(0xffffffffu, l[g], mask);
      const float m_new = fmaxf(m[g], m_o);
      const float c_s = exp2f(m[g] - m_new), c_o = exp2f(m_o - m_new);
      l[g] = l[g] * c_s + l_o * c_o;
#pragma unroll
      for (int i = 0; i < DPL; ++i) {
        const float a_o = __shfl_xor_sync(0xffffffffu, acc[g][i], mask);
        acc[g][i] = acc[g][i] * c_s + a_o * c_o;
      }
      m[g] = m_new;
    }
  }
  if (tg == 0) {
#pragma unroll
    for (int g = 0; g < GQ; ++g) {
      if (dl == 0) {
        sm_m[warp][g] = m[g];
        sm_l[warp][g] = l[g];
      }
#pragma unroll
      for (int pc = 0; pc < NP; ++pc)
#pragma unroll
        for (int i = 0; i < 8; ++i) sm_o[warp][g][pc * 64 + dl * 8 + i] = acc[g][pc * 8 + i];
    }
  }
  __syncthreads();
  // merge the warps; thread -> (query head g, dimension i)
  for (int idx = threadIdx.x; idx < GQ * HD; idx += kAttnThreads) {
    const int g = idx / HD, i = idx % HD;
    float M = kNegBig;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) M = fmaxf(M, sm_m[w][g]);
    float o = 0.0f, L = 0.0f;
#pragma unroll
    for (int w = 0; w < kAttnWarps; ++w) {
      const float sc = exp2f(sm_m[w][g] - M);
      o = fmaf(sm_o[w][g][i], sc, o);
      L = fmaf(sm_l[w][g], sc, L);
    }
    const int qh = kvh * rep + g0 + g;
    const long long pidx = ((long long)b * a.n_splits + split) * a.n_q_heads + qh;
    a.part_o[pidx * HD + i] = o;
    if (i == 0) {
      a.part_ml[pidx * 2] = M;
      a.part_ml[pidx * 2 + 1] = L;
    }
  }
}

struct AttnCombineArgs {
  const float* part_ml;
  const float* part_o;
  uint16_t* out;      // [batch][n_q_heads][HD] 16-bit
  float* lse;         // [batch][n_q_heads] natural-log sum-exp, or nullptr
  int n_q_heads;
  int n_splits;
};

// One CTA per (sequence, query head); thread i owns output dimension i.
template <int HD, bool kBf16>
__global__ void __launch_bounds__(HD) attn_combine_kernel(const AttnCombineArgs a) {
  const int b = blockIdx.x / a.n_q_heads, qh = blockIdx.x % a.n_q_heads;
  const int i = threadIdx.x;
  float M = kNegBig;
  for (int s = 0; s < a.n_splits; ++s)
    M = fmaxf(M, a.part_ml[(((long long)b * a.n_splits + s) * a.n_q_heads + qh) * 2]);
  float L = 0.0f, o = 0.0f;
  for (int s = 0; s < a.n_splits; ++s) {
    const long long pidx = ((long long)b * a.n_splits + s) * a.n_q_heads + qh;
    const float w = exp2f(a.part_ml[pidx * 2] - M);
    L = fmaf(a.part_ml[pidx * 2 + 1], w, L);
    o = fmaf(a.part_o[pidx * HD + i], w, o);
  }
  a.out[((long long)b * a.n_q_heads + qh) * HD + i] = store16<kBf16>(o / L);
  if (a.lse != nullptr && i == 0)
    a.lse[(long long)b * a.n_q_heads + qh] = (M + log2f(L)) * 0.6931471805599453f;
}

}  // namespace aquakv
