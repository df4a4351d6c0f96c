// Single-query grouped-query attention over freshly decoded keys/values (the attention read of Algorithm 4:
// the block attends to the recovered cache).  Split-KV: one CTA reduces a block of consecutive
// tokens of one sequence to per-query-head partials (running max, sum, unnormalised output), a
// second kernel merges the partials of a sequence by log-sum-exp.  All accumulation is fp32.
//
// One CTA owns (token block, KV head) and up to eight of that KV head's query heads at once, so
// K/V bytes are read once per KV head.
#pragma once

#include "common.cuh"

namespace aquakv {

constexpr float kNegBig = -1.0e30f;

struct AttnArgs {
  const uint16_t* q;      // [batch][n_q_heads][HD]
  const uint16_t* Kh;     // decoded keys, row r = global token (tok_base + r)   [*, ld]
  const uint16_t* Vh;     // decoded values                                      [*, ld_v]
  long long ld;
  long long ld_v;
  long long tok_base;
  long long blk_begin;    // first global block (sequence * n_splits + split) of this launch
  int ctx;                // tokens per sequence
  int n_q_heads;
  int n_kv_heads;
  int n_splits;           // blocks per sequence
  int block_tokens;       // tokens per block
  int gq;                 // query heads of a KV group handled by one pass (grid z = passes), <= 8
  float scale_log2;       // softmax_scale * log2(e)
  float* part_ml;         // [batch][n_splits][n_q_heads][2]  (max in log2 units, sum)
  float* part_o;          // [batch][n_splits][n_q_heads][HD]
};

// D += A * B for one m16n8k16 tile (fp32 accumulate), A and B in the cache's 16-bit type.
template <bool kBf16>
__device__ __forceinline__ void mma_16x8x16(float& d0, float& d1, float& d2, float& d3, uint32_t a0,
                                            uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
  if constexpr (kBf16) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3)
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  } else {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3)
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
  }
}

// The kernel is bound by reading K^ and V^ once (HD * 4 bytes per token and KV head), so it is built
// to issue few instructions per byte: both contractions run as warp-level 16x8x16 matrix products
// with the query heads of the KV group on the M side (up to 8 rows used, the other 8 are zero) and
// every operand fragment filled straight from 16-byte global loads.
//   scores: A = queries, B = keys.  The product sums over head dimensions, so their order inside a
//           32-dimension chunk is free: lane (n, j) loads dimensions [32c + 8j, 32c + 8j + 8) of
//           token n as one 16-byte piece and uses it as the B fragments of two k-steps; the query
//           fragments use the same order.
//   output: A = probabilities (the score accumulators, rounded to the 16-bit type, already have the
//           A-fragment layout), B = values.  A B register pairs two consecutive tokens at one
//           dimension; it is made from the 16-byte pieces of those two token rows with one byte
//           permute.  Column n of output tile u stands for head dimension 8n + u (u < 8) or
//           64 + 8n + (u - 8), so lane group n reads contiguous 16-byte pieces.
// A warp takes 32 tokens at a time (four 8-token score tiles, two 16-token k-steps of the output
// product) with an online softmax across its groups; the warps of a CTA merge through shared memory.
constexpr int kAttnMmaWarps = 4;
constexpr int kAttnMmaThreads = kAttnMmaWarps * 32;
constexpr int kAttnMmaMaxGq = 8;    // query heads per KV head in one pass (rows of the M = 16 tile in use)

template <int HD, bool kBf16>
__global__ void __launch_bounds__(kAttnMmaThreads, 2) attn_partial_kernel(const AttnArgs a) {
  constexpr int NCH = HD / 32;         // 32-dimension chunks of the score product
  constexpr int NVH = HD / 64;         // 64-dimension halves of a value row (one 16-byte piece per lane each)
  constexpr int NOT = HD / 8;          // output tiles of 8 dimensions
  __shared__ float sm_m[kAttnMmaWarps][kAttnMmaMaxGq];
  __shared__ float sm_l[kAttnMmaWarps][kAttnMmaMaxGq];
  __shared__ float sm_o[kAttnMmaWarps][kAttnMmaMaxGq][HD];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int g = lane >> 2, j = lane & 3;
  const long long gb = a.blk_begin + blockIdx.x;
  const int b = int(gb / a.n_splits), split = int(gb % a.n_splits);
  const int t_begin = split * a.block_tokens;
  const int t_end = min(a.ctx, t_begin + a.block_tokens);
  const int rep = a.n_q_heads / a.n_kv_heads;
  const int kvh = blockIdx.y;
  const int g0 = blockIdx.z * a.gq;    // first query head (within the KV group) of this pass
  const int gq = min(a.gq, rep - g0);  // query heads of this pass

  // query fragments: row g = query head g0 + g of the KV group (rows >= gq and rows 8..15 are zero)
  uint32_t qa[NCH][2][2];
  {
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
        a.q + ((long long)b * a.n_q_heads + kvh * rep + g0 + (g < gq ? g : 0)) * HD);
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
      const uint4 w = *reinterpret_cast<const uint4*>(qrow + (c * 32 + j * 8) / 2);
      const bool on = g < gq;
      qa[c][0][0] = on ? w.x : 0u;
      qa[c][0][1] = on ? w.y : 0u;
      qa[c][1][0] = on ? w.z : 0u;
      qa[c][1][1] = on ? w.w : 0u;
    }
  }
  float m_run = kNegBig, l_run = 0.0f;     // row g's running maximum (log2 units) and this lane's part of its sum
  float o[NOT][2];
#pragma unroll
  for (int u = 0; u < NOT; ++u) o[u][0] = o[u][1] = 0.0f;
  float dz0 = 0.0f, dz1 = 0.0f;            // rows 8..15 of every product: stay zero

  const long long row0 = (long long)b * a.ctx - a.tok_base;
  const uint16_t* kbase = a.Kh + kvh * HD;
  const uint16_t* vbase = a.Vh + kvh * HD;
  // keys of a group: score tile t, token g of it, 16-byte piece j of every 32-dimension chunk
  uint4 kq[4][NCH];
  auto load_keys = [&](int tb) {
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int tok = tb + 8 * t + g;
      const uint16_t* kp = kbase + (row0 + (tok < t_end ? tok : t_begin)) * a.ld + j * 8;
#pragma unroll
      for (int c = 0; c < NCH; ++c) kq[t][c] = __ldcs(reinterpret_cast<const uint4*>(kp + c * 32));
    }
  };
  if (t_begin + warp * 32 < t_end) load_keys(t_begin + warp * 32);
  for (int tb = t_begin + warp * 32; tb < t_end; tb += 32 * kAttnMmaWarps) {
    // ---- values of this group (k-step ks, tokens 2j.. of it); its keys were fetched one group ahead ----
    uint4 vq[2][4][NVH];
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const int tok = tb + 16 * ks + (r >> 1) * 8 + 2 * j + (r & 1);
        const uint16_t* vp = vbase + (row0 + (tok < t_end ? tok : t_begin)) * a.ld_v + g * 8;
#pragma unroll
        for (int h = 0; h < NVH; ++h) vq[ks][r][h] = __ldcs(reinterpret_cast<const uint4*>(vp + h * 64));
      }
    }
    // ---- scores ---------------------------------------------------------------------------------
    float sc[4][2];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        mma_16x8x16<kBf16>(s0, s1, dz0, dz1, qa[c][0][0], 0u, qa[c][0][1], 0u, kq[t][c].x, kq[t][c].y);
        mma_16x8x16<kBf16>(s0, s1, dz0, dz1, qa[c][1][0], 0u, qa[c][1][1], 0u, kq[t][c].z, kq[t][c].w);
      }
      const int tok = tb + 8 * t + 2 * j;
      sc[t][0] = tok < t_end ? s0 * a.scale_log2 : kNegBig;
      sc[t][1] = tok + 1 < t_end ? s1 * a.scale_log2 : kNegBig;
    }
    if (tb + 32 * kAttnMmaWarps < t_end) load_keys(tb + 32 * kAttnMmaWarps);   // in flight during the rest
    // ---- online softmax of row g over the group's 32 tokens (8 per lane, 4 lanes per row) ------
    float mx = fmaxf(fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1])),
                     fmaxf(fmaxf(sc[2][0], sc[2][1]), fmaxf(sc[3][0], sc[3][1])));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m_run, mx);
    const float corr = exp2f(m_run - m_new);
    m_run = m_new;
    // probabilities as 16-bit A fragments.  bf16 keeps 8 bits, too few for the output's tolerance, so
    // a probability goes in as two terms (rounded value + rounded remainder, together good to 2^-17).
    uint32_t pa[4], pb[4];
    float lsum = 0.0f;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      // masked tokens get probability 0 even when the whole group is masked (sc == m_new == kNegBig)
      const float p0 = sc[t][0] > 0.5f * kNegBig ? exp2f(sc[t][0] - m_new) : 0.0f;
      const float p1 = sc[t][1] > 0.5f * kNegBig ? exp2f(sc[t][1] - m_new) : 0.0f;
      pa[t] = store16x2<kBf16>(p0, p1);
      if constexpr (kBf16) {
        pb[t] = store16x2<kBf16>(p0 - load16<kBf16>(uint16_t(pa[t] & 0xffffu)),
                                 p1 - load16<kBf16>(uint16_t(pa[t] >> 16)));
        lsum += p0 + p1;
      } else {
        pb[t] = 0u;
        // the row sum uses the rounded probabilities, the ones the output product multiplies by
        lsum += load16<kBf16>(uint16_t(pa[t] & 0xffffu)) + load16<kBf16>(uint16_t(pa[t] >> 16));
      }
    }
    l_run = fmaf(l_run, corr, lsum);
#pragma unroll
    for (int u = 0; u < NOT; ++u) {
      o[u][0] *= corr;
      o[u][1] *= corr;
    }
    // ---- output: O[g][:] += P[g][tokens] * V[tokens][:] ---------------------------------------------
#pragma unroll
    for (int ks = 0; ks < 2; ++ks) {
#pragma unroll
      for (int h = 0; h < NVH; ++h) {
        const uint32_t w0[4] = {vq[ks][0][h].x, vq[ks][0][h].y, vq[ks][0][h].z, vq[ks][0][h].w};
        const uint32_t w1[4] = {vq[ks][1][h].x, vq[ks][1][h].y, vq[ks][1][h].z, vq[ks][1][h].w};
        const uint32_t w2[4] = {vq[ks][2][h].x, vq[ks][2][h].y, vq[ks][2][h].z, vq[ks][2][h].w};
        const uint32_t w3[4] = {vq[ks][3][h].x, vq[ks][3][h].y, vq[ks][3][h].z, vq[ks][3][h].w};
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
          const uint32_t b0 = __byte_perm(w0[e >> 1], w1[e >> 1], sel);
          const uint32_t b1 = __byte_perm(w2[e >> 1], w3[e >> 1], sel);
          mma_16x8x16<kBf16>(o[h * 8 + e][0], o[h * 8 + e][1], dz0, dz1, pa[2 * ks], 0u, pa[2 * ks + 1], 0u, b0, b1);
          if constexpr (kBf16)
            mma_16x8x16<kBf16>(o[h * 8 + e][0], o[h * 8 + e][1], dz0, dz1, pb[2 * ks], 0u, pb[2 * ks + 1], 0u, b0, b1);
        }
      }
    }
  }
  // ---- merge the warps of the CTA -----------------------------------------------------------------
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  if (g < gq) {
    if (j == 0) {
      sm_m[warp][g] = m_run;
      sm_l[warp][g] = l_run;
    }
#pragma unroll
    for (int u = 0; u < NOT; ++u) {
      const int base = (u < 8 ? 0 : 64) + (u & 7);
      sm_o[warp][g][base + (2 * j) * 8] = o[u][0];
      sm_o[warp][g][base + (2 * j + 1) * 8] = o[u][1];
    }
  }
  __syncthreads();
  // thread -> (query head q, dimension i)
  for (int idx = threadIdx.x; idx < gq * HD; idx += kAttnMmaThreads) {
    const int qi = idx / HD, i = idx % HD;
    float M = kNegBig;
#pragma unroll
    for (int w = 0; w < kAttnMmaWarps; ++w) M = fmaxf(M, sm_m[w][qi]);
    float ov = 0.0f, L = 0.0f;
#pragma unroll
    for (int w = 0; w < kAttnMmaWarps; ++w) {
      const float scl = exp2f(sm_m[w][qi] - M);
      ov = fmaf(sm_o[w][qi][i], scl, ov);
      L = fmaf(sm_l[w][qi], scl, L);
    }
    const int qh = kvh * rep + g0 + qi;
    const long long pidx = ((long long)b * a.n_splits + split) * a.n_q_heads + qh;
    a.part_o[pidx * HD + i] = ov;
    if (i == 0) {
      a.part_ml[pidx * 2] = M;
      a.part_ml[pidx * 2 + 1] = L;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// The same product for ONE warp, at most 128 consecutive tokens of one sequence, one KV head and 64 of
// its output dimensions: the attention role of the fused decode kernel (layer_kernel.cuh) calls it
// on every token block as soon as the block's reconstructed rows exist, so the rows are read from L2
// and never need to come back from DRAM.  With head_dim 128 two warps share a head: both form the
// scores (the keys are read twice, from L2), each accumulates one half of the output dimensions, so a
// warp holds 16 accumulator registers and can keep its loads one phase ahead within the fused
// kernel's register budget: the values of a step are requested before its scores are formed, the
// keys of the next step right after them.  16 tokens per step (two 8-token score tiles, one
// 16-token k-step of the output product).  Rows are read with ld.global.cg: other SMs of the same
// kernel have just written them.
//   Krows: row r = token r of the segment, offset to the KV head's first dimension.
//   Vrows: the same, offset to the first of this warp's 64 output dimensions.
//   qrows: query head 0 of the KV group (gq heads, HD values each), re-read every step (L1 hits).
//   ml_out[q][2] = (running maximum in log2 units, sum) or nullptr (the head's other warp writes it);
//   o_out[q][HD]: unnormalised output, offset to this warp's first dimension.
// ---------------------------------------------------------------------------------------------
template <int HD, bool kBf16>
__device__ __forceinline__ void attn_segment_warp(const uint16_t* __restrict__ Krows, const uint16_t* __restrict__ Vrows,
                                                  long long ldK, long long ldV, int n_tok,
                                                  const uint16_t* __restrict__ qrows, int gq, float scale_log2,
                                                  float* __restrict__ ml_out, float* __restrict__ o_out, int lane) {
  constexpr int NCH = HD / 32;
  const int g = lane >> 2, j = lane & 3;
  float m_run = kNegBig, l_run = 0.0f;
  float o[8][2];
#pragma unroll
  for (int u = 0; u < 8; ++u) o[u][0] = o[u][1] = 0.0f;
  float dz0 = 0.0f, dz1 = 0.0f;            // rows 8..15 of every product: stay zero
  const uint32_t* qrow = reinterpret_cast<const uint32_t*>(qrows + (g < gq ? g : 0) * HD);
  const bool q_on = g < gq;
  uint4 kq[2][NCH];
  auto load_keys = [&](int tb) {
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const int tok = tb + 8 * t + g;
      const uint16_t* kp = Krows + (long long)(tok < n_tok ? tok : 0) * ldK + j * 8;
#pragma unroll
      for (int c = 0; c < NCH; ++c) kq[t][c] = __ldcg(reinterpret_cast<const uint4*>(kp + c * 32));
    }
  };
  load_keys(0);
#pragma unroll 1
  for (int tb = 0; tb < n_tok; tb += 16) {
    // ---- this step's values: requested now, used after the softmax -----------------------------------
    uint4 w[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      const int tok = tb + (r >> 1) * 8 + 2 * j + (r & 1);
      w[r] = __ldcg(reinterpret_cast<const uint4*>(Vrows + (long long)(tok < n_tok ? tok : 0) * ldV + g * 8));
    }
    // ---- scores of 16 tokens ------------------------------------------------------------------------
    float sc[2][2];
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      float s0 = 0.0f, s1 = 0.0f;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const uint4 qw = __ldg(reinterpret_cast<const uint4*>(qrow + (c * 32 + j * 8) / 2));
        mma_16x8x16<kBf16>(s0, s1, dz0, dz1, q_on ? qw.x : 0u, 0u, q_on ? qw.y : 0u, 0u, kq[t][c].x, kq[t][c].y);
        mma_16x8x16<kBf16>(s0, s1, dz0, dz1, q_on ? qw.z : 0u, 0u, q_on ? qw.w : 0u, 0u, kq[t][c].z, kq[t][c].w);
      }
      const int tok = tb + 8 * t + 2 * j;
      sc[t][0] = tok < n_tok ? s0 * scale_log2 : kNegBig;
      sc[t][1] = tok + 1 < n_tok ? s1 * scale_log2 : kNegBig;
    }
    if (tb + 16 < n_tok) load_keys(tb + 16);     // in flight during the softmax and the output product
    // ---- online softmax of row g (4 tokens per lane, 4 lanes per row) -------------------------------
    float mx = fmaxf(fmaxf(sc[0][0], sc[0][1]), fmaxf(sc[1][0], sc[1][1]));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    const float m_new = fmaxf(m_run, mx);
    const float corr = exp2f(m_run - m_new);
    m_run = m_new;
    uint32_t pa[2], pb[2];
    float lsum = 0.0f;
#pragma unroll
    for (int t = 0; t < 2; ++t) {
      const float p0 = sc[t][0] > 0.5f * kNegBig ? exp2f(sc[t][0] - m_new) : 0.0f;
      const float p1 = sc[t][1] > 0.5f * kNegBig ? exp2f(sc[t][1] - m_new) : 0.0f;
      pa[t] = store16x2<kBf16>(p0, p1);
      if constexpr (kBf16) {     // two terms: 8 bits are too few for the output's tolerance
        pb[t] = store16x2<kBf16>(p0 - load16<kBf16>(uint16_t(pa[t] & 0xffffu)),
                                 p1 - load16<kBf16>(uint16_t(pa[t] >> 16)));
        lsum += p0 + p1;
      } else {
        pb[t] = 0u;
        lsum += load16<kBf16>(uint16_t(pa[t] & 0xffffu)) + load16<kBf16>(uint16_t(pa[t] >> 16));
      }
    }
    l_run = fmaf(l_run, corr, lsum);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      o[u][0] *= corr;
      o[u][1] *= corr;
    }
    // ---- output: O[g][dims] += P[g][tokens] * V[tokens][dims] ------------------------------------------
    {
      const uint32_t w0[4] = {w[0].x, w[0].y, w[0].z, w[0].w};
      const uint32_t w1[4] = {w[1].x, w[1].y, w[1].z, w[1].w};
      const uint32_t w2[4] = {w[2].x, w[2].y, w[2].z, w[2].w};
      const uint32_t w3[4] = {w[3].x, w[3].y, w[3].z, w[3].w};
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
        const uint32_t b0 = __byte_perm(w0[e >> 1], w1[e >> 1], sel);
        const uint32_t b1 = __byte_perm(w2[e >> 1], w3[e >> 1], sel);
        mma_16x8x16<kBf16>(o[e][0], o[e][1], dz0, dz1, pa[0], 0u, pa[1], 0u, b0, b1);
        if constexpr (kBf16)
          mma_16x8x16<kBf16>(o[e][0], o[e][1], dz0, dz1, pb[0], 0u, pb[1], 0u, b0, b1);
      }
    }
  }
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  if (g < gq) {
    if (j == 0 && ml_out != nullptr) {
      ml_out[g * 2] = m_run;
      ml_out[g * 2 + 1] = l_run;
    }
    // column n of output tile u stands for dimension 8n + u of the warp's 64
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      o_out[g * HD + u + (2 * j) * 8] = o[u][0];
      o_out[g * HD + u + (2 * j + 1) * 8] = o[u][1];
    }
  }
}

struct AttnCombineArgs {
  const float* part_ml;
  const float* part_o;
  uint16_t* out;      // [batch][n_q_heads][HD] 16-bit
  float* lse;         // [batch][n_q_heads] natural-log sum-exp, or nullptr
  int n_q_heads;
  int n_splits;       // slots per sequence in the partial arrays
  int ctx;            // tokens per sequence
  int block_tokens;   // > 0: partials per block of that many tokens of the FLATTENED token index (a sequence
                      // uses as many slots as blocks overlap it); 0: every sequence uses all n_splits slots
  // a second set of partials per sequence, merged after the first (the uncompressed rows a cache policy keeps
  // beside the compressed ones: attention sinks and the recent-token buffer, Section 3.3); 0 slots = none
  const float* extra_ml;   // [batch][extra_splits][n_q_heads][2]
  const float* extra_o;    // [batch][extra_splits][n_q_heads][HD]
  int extra_splits;
};

// One CTA per (sequence, query head); thread i owns output dimension i.
template <int HD, bool kBf16>
__global__ void __launch_bounds__(HD) attn_combine_kernel(const AttnCombineArgs a) {
  const int b = blockIdx.x / a.n_q_heads, qh = blockIdx.x % a.n_q_heads;
  const int i = threadIdx.x;
  int n_s = a.n_splits;
  if (a.ctx == 0) {
    n_s = 0;
  } else if (a.block_tokens > 0) {
    const long long t0 = (long long)b * a.ctx, t1 = t0 + a.ctx - 1;
    n_s = int(t1 / a.block_tokens - t0 / a.block_tokens) + 1;
  }
  const float* xml = a.extra_ml + ((long long)b * a.extra_splits * a.n_q_heads + qh) * 2;
  const float* xpo = a.extra_o + ((long long)b * a.extra_splits * a.n_q_heads + qh) * HD + i;
  // Both passes keep several independent loads in flight: with many slots per sequence the kernel is
  // bound by the latency of its loads, not by their number.
  const float* ml = a.part_ml + ((long long)b * a.n_splits * a.n_q_heads + qh) * 2;
  const float* po = a.part_o + ((long long)b * a.n_splits * a.n_q_heads + qh) * HD + i;
  const long long ml_step = (long long)a.n_q_heads * 2, o_step = (long long)a.n_q_heads * HD;
  float M = kNegBig;
  {
    float m4[4] = {kNegBig, kNegBig, kNegBig, kNegBig};
    int s = 0;
    for (; s + 4 <= n_s; s += 4) {
#pragma unroll
      for (int u = 0; u < 4; ++u) m4[u] = fmaxf(m4[u], ml[(s + u) * ml_step]);
    }
    for (; s < n_s; ++s) m4[0] = fmaxf(m4[0], ml[s * ml_step]);
    for (int x = 0; x < a.extra_splits; ++x) m4[1] = fmaxf(m4[1], xml[x * ml_step]);
    M = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
  }
  float L = 0.0f, o = 0.0f;
  {
    int s = 0;
    for (; s + 4 <= n_s; s += 4) {
      float mv[4], lv[4], ov[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        mv[u] = ml[(s + u) * ml_step];
        lv[u] = ml[(s + u) * ml_step + 1];
        ov[u] = po[(s + u) * o_step];
      }
#pragma unroll
      for (int u = 0; u < 4; ++u) {          // accumulated in slot order
        const float w = exp2f(mv[u] - M);
        L = fmaf(lv[u], w, L);
        o = fmaf(ov[u], w, o);
      }
    }
    for (; s < n_s; ++s) {
      const float w = exp2f(ml[s * ml_step] - M);
      L = fmaf(ml[s * ml_step + 1], w, L);
      o = fmaf(po[s * o_step], w, o);
    }
    for (int x = 0; x < a.extra_splits; ++x) {
      const float w = exp2f(xml[x * ml_step] - M);
      L = fmaf(xml[x * ml_step + 1], w, L);
      o = fmaf(xpo[x * o_step], w, o);
    }
  }
  a.out[((long long)b * a.n_q_heads + qh) * HD + i] = store16<kBf16>(o / L);
  if (a.lse != nullptr && i == 0)
    a.lse[(long long)b * a.n_q_heads + qh] = (M + log2f(L)) * 0.6931471805599453f;
}

}  // namespace aquakv
