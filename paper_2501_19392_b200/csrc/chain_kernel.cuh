// Algorithm 4's loop over layers for SMALL calls (a decode step of a batch of sequences, a short
// prompt): Algorithm 2 (encode) or Algorithm 3 (decode) for every layer in ONE persistent launch.
//
// Why a second kernel.  The per-layer kernel (layer_kernel.cuh) is built for tens of thousands of
// tokens: a 128 x 256 tcgen05 tile per CTA pair, a wave of token blocks per job.  With 64 tokens one
// layer is a chain of four dependent steps (key prediction -> key rows -> value prediction -> value
// rows) in which four CTA pairs stream 6 MB of adapter weights while 140 SMs wait, and every layer
// pays a launch, a prologue and six tensor-map encodings.  The bound of such a call is the weight
// stream (6 d^2 bytes per layer) and the latency of the hand-offs, not arithmetic.  So here
//   - the predictor products are cut into units of 16 tokens x 64 features x 128 input features, one
//     warp each, so that EVERY SM streams a share of the weights; a unit is a handful of warp-level
//     m16n8k16 tensor-core products whose operand fragments come straight from 16-byte global loads
//     (the order of the summation index inside a 32-element chunk is free as long as both operands
//     use the same one).  The tcgen05 path needs M >= 64 rows per instruction and an operand round
//     trip through shared memory, which a 16-row unit bound by its load latency does not repay;
//   - the units of one output tile (its 8 or 16 slices of input features) run on the warps of one CTA
//     at the same time and are added through shared memory in ascending slice order (then the bias),
//     so the result does not depend on timing and the fp32 prediction is written once;
//   - the key chain (K^_l needs only K^_{l-1}) runs on one team of CTAs, the value chain
//     (V^_l needs V^_{l-1} and K^_l) on another, one layer behind where it must be, so a layer costs
//     the key chain's two hand-offs, not four;
//   - completion is counted per 16-token tile and stage in global memory (release/acquire), every
//     wait is bounded, all CTAs are resident (at most one per SM), and a stage only waits on
//     earlier stages, so the schedule cannot dead-lock;
//   - while a warp waits it asks L2 for the weight slice of its next unit.
// The row work itself is that of codec.cuh / rowwarp.cuh, unchanged.
//
// The partial sums are added in a different order than the per-layer kernel's single accumulation,
// so reconstructions can differ from that kernel's in the last bit of the 16-bit type; a cache
// written by the chain encoder is reproduced bit for bit by the chain decoder.
#pragma once

#include "attn.cuh"
#include "codec.cuh"
#include "common.cuh"
#include "layer_kernel.cuh"
#include "rowwarp.cuh"

namespace aquakv {

constexpr int kChainMaxLayers = 128;
constexpr int kChainWarps = 16;
constexpr int kChainThreads = kChainWarps * 32;
constexpr int kChainMT = 16;       // tokens of a unit (MMA M)
constexpr int kChainNT = 64;       // output features of a unit
constexpr int kChainKS = 128;      // input features of a unit

struct ChainLayer {
  const uint16_t* K;       // encode targets [T, ldX] (encode only)
  const uint16_t* V;
  const uint16_t* Wk;      // [d][d]; nullptr: the layer has no predictor
  const uint16_t* Wv;      // [d][2d]
  const float* bk;         // optional biases
  const float* bv;
  uint8_t* Kcodes;         // written by encode, read by decode
  uint16_t* Kscales;
  uint8_t* Vcodes;
  uint16_t* Vscales;
  uint16_t* Khat;          // this layer's reconstruction [T, ldHat] (caller's or workspace)
  uint16_t* Vhat;
  long long ldHat;
};

struct ChainArgs {
  int T, L;
  long long ldX;
  const uint16_t* Khat_init;   // reconstruction of the layer before the first one (needed iff layer 0 has a predictor)
  const uint16_t* Vhat_init;
  long long ldInit;
  float* Pk;                   // key predictions   [T][d] fp32
  float* Pv;                   // value predictions [T][d] fp32
  int* counters;               // [4][L][n_mt], zero at launch: feature tiles / rows done per stage, layer and 16-token tile
  int n_ctas_k;                // CTAs of the key team (the rest run the value chain)
  const uint32_t* signmask_k;
  const uint32_t* signmask_v;
  const float4* grid4;
  SearchDev search;
  int log_h, log_g;
  int* status;
  ChainLayer layer[kChainMaxLayers];
};

// One unit: the 16 x 64 fp32 partial product  A[row0 .. row0+15][k-slice] . W[n0 .. n0+63][k-slice]^T,
// left in `red` (row-major [16][64], shared memory) for the CTA's reduction over the slices.
template <bool kBf16>
__device__ __forceinline__ void chain_gemm_unit(const uint16_t* __restrict__ A, long long ldA, int ka,
                                                const uint16_t* __restrict__ W, long long ldW, int kw,
                                                int row0, int T, int n0, float* __restrict__ red, int lane) {
  const int g = lane >> 2, j = lane & 3;
  float acc[8][4];
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.0f;
  const int ra = row0 + g < T ? row0 + g : T - 1, rb = row0 + g + 8 < T ? row0 + g + 8 : T - 1;
  const uint16_t* pa = A + (long long)ra * ldA + ka + j * 8;      // written by other SMs of this kernel: read through L2
  const uint16_t* pb = A + (long long)rb * ldA + ka + j * 8;
  const uint16_t* pw = W + (long long)(n0 + g) * ldW + kw + j * 8;
#pragma unroll
  for (int half = 0; half < kChainKS / 64; ++half) {
    uint4 alo[2], ahi[2], b[2][8];
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      const int kk = (2 * half + c) * 32;
      alo[c] = __ldcg(reinterpret_cast<const uint4*>(pa + kk));
      ahi[c] = __ldcg(reinterpret_cast<const uint4*>(pb + kk));
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) b[c][nt] = __ldg(reinterpret_cast<const uint4*>(pw + (long long)nt * 8 * ldW + kk));
    }
#pragma unroll
    for (int c = 0; c < 2; ++c) {
#pragma unroll
      for (int nt = 0; nt < 8; ++nt) {
        mma_16x8x16<kBf16>(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3], alo[c].x, ahi[c].x, alo[c].y, ahi[c].y,
                           b[c][nt].x, b[c][nt].y);
        mma_16x8x16<kBf16>(acc[nt][0], acc[nt][1], acc[nt][2], acc[nt][3], alo[c].z, ahi[c].z, alo[c].w, ahi[c].w,
                           b[c][nt].z, b[c][nt].w);
      }
    }
  }
#pragma unroll
  for (int nt = 0; nt < 8; ++nt) {
    *reinterpret_cast<float2*>(red + g * kChainNT + nt * 8 + 2 * j) = make_float2(acc[nt][0], acc[nt][1]);
    *reinterpret_cast<float2*>(red + (g + 8) * kChainNT + nt * 8 + 2 * j) = make_float2(acc[nt][2], acc[nt][3]);
  }
}

// Polls *ctr until it reaches target, like counter_wait_bounded but with short pauses: in this kernel a
// wait is on the critical path of the whole call and few warps poll one counter.
__device__ __forceinline__ bool chain_wait(const int* ctr, int target, volatile int* abort_flag, int* status) {
  if (ld_acquire(ctr) >= target) return true;
  const unsigned long long t0 = global_timer_ns();
  uint32_t spins = 0;
  while (ld_acquire(ctr) < target) {
    __nanosleep(40);
    if ((++spins & 0xFFu) == 0) {
      if (*abort_flag) return false;
      if (global_timer_ns() - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, kStatusTimeout);
        return false;
      }
    }
  }
  return true;
}

template <int D, int NPTS, bool kEncode, bool kWarpRows>
struct ChainSmem {
  typename LayerTables<kEncode, NPTS>::type tables;
  LayerRowScratch<D, kChainWarps, kWarpRows> scratch;
  float red[kChainWarps][kChainMT * kChainNT];     // one unit's partial product per warp
  int abort_flag;
};

// kWarpRows (D = 1024 with Hadamard block = scale group = 1024 only, checked on the host): the
// one-warp-per-row routines, which keep more rows in flight; otherwise the team routines (D / 256 warps per
// row, any supported block / group), whose rows finish sooner.  A layer of a small call is a chain of
// dependent steps, so the host picks the team routines while every row still gets a team at once
// (64 tokens x 32 layers: 11.5 against 13.9 us per layer) and the warp routines beyond.
template <bool kEncode, int D, int NPTS, bool kBf16, bool kWarpRows>
__global__ void __launch_bounds__(kChainThreads, 1) chain_kernel(const __grid_constant__ ChainArgs a) {
  static_assert(!kWarpRows || D == 1024, "one warp per row needs d_kv = 1024");
  constexpr bool WR = kWarpRows;
  constexpr int TEAM = WR ? 1 : RowTeam<D>::TEAM;
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = D / 2 * BITS / 8;
  constexpr int NTILES = D / kChainNT;               // feature tiles of a row
  extern __shared__ __align__(16) uint8_t chain_smem_raw[];
  ChainSmem<D, NPTS, kEncode, kWarpRows>* sm = reinterpret_cast<ChainSmem<D, NPTS, kEncode, kWarpRows>*>(chain_smem_raw);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if constexpr (kEncode) {
    row_smem_fill<NPTS>(&sm->tables, a.search.table, a.grid4);
  } else {
    for (int i = threadIdx.x; i < NPTS; i += blockDim.x) {
      const float4 g = a.grid4[i];
      sm->tables.grid[i] = pack2(g.x, g.y);
    }
  }
  if (threadIdx.x == 0) sm->abort_flag = 0;
  __syncthreads();
  volatile int* abort_flag = &sm->abort_flag;

  const bool is_v = int(blockIdx.x) >= a.n_ctas_k;
  const int team_ctas = is_v ? int(gridDim.x) - a.n_ctas_k : a.n_ctas_k;
  const int n_warps = team_ctas * kChainWarps;
  const int n_mt = (a.T + kChainMT - 1) / kChainMT;
  int* g_done = a.counters + (is_v ? 2 : 0) * a.L * n_mt;      // units done  [L][n_mt]
  int* r_done = a.counters + (is_v ? 3 : 1) * a.L * n_mt;      // rows done   [L][n_mt]
  const int* kr_done = a.counters + 1 * a.L * n_mt;            // key rows done (the value predictor reads K^)
  const int n_in = is_v ? 2 : 1;
  const int n_slices = n_in * D / kChainKS;
  float* P = is_v ? a.Pv : a.Pk;
  const int log_h = WR ? 10 : a.log_h, log_g = WR ? 10 : a.log_g;
  const int n_groups = D >> log_g;

  // row contexts
  RowCtx rck;
  WarpRowCtx wrc;
  if constexpr (WR) {
    wrc.lane = lane;
    wrc.inv_w = a.search.inv_w;
    wrc.signs = (is_v ? a.signmask_v : a.signmask_k)[lane];
    rck.member = 0;
    rck.barrier = 0;
  } else {
    row_ctx_init(rck, is_v ? a.signmask_v : a.signmask_k, a.search.inv_w, log_h, log_g, lane, warp % TEAM,
                 RowTeam<D>::NV, 1 + warp / TEAM);
  }

  const int cta = int(blockIdx.x) - (is_v ? a.n_ctas_k : 0);
  for (int l = 0; l < a.L; ++l) {
    // the warps of a CTA enter a layer together (its prediction stage uses CTA-wide barriers), and a
    // wait that expired anywhere in the CTA ends the kernel for all of them here
    __syncthreads();
    if (*abort_flag) break;
    const ChainLayer& ly = a.layer[l];
    const bool has_pred = ly.Wk != nullptr;
    // ------------------------------------------------------------------------------------------
    // predictions of this layer: the n_slices units of an output tile (16 tokens x 64 features) run on
    // n_slices warps of ONE CTA and are added through shared memory in ascending slice order
    // ------------------------------------------------------------------------------------------
    if (has_pred) {
      const uint16_t* W = is_v ? ly.Wv : ly.Wk;
      const float* bias = is_v ? ly.bv : ly.bk;
      const long long ldW = (long long)n_in * D;
      const uint16_t* prev = is_v ? (l == 0 ? a.Vhat_init : a.layer[l - 1].Vhat) : (l == 0 ? a.Khat_init : a.layer[l - 1].Khat);
      const long long ld_prev = l == 0 ? a.ldInit : a.layer[l - 1].ldHat;
      const int tiles_per_round = kChainWarps / n_slices;          // 1 .. 8
      const int n_tiles = n_mt * NTILES;
      const int n_rounds = (n_tiles + tiles_per_round - 1) / tiles_per_round;
      bool stop = false;
      for (int q = cta; !stop && q < n_rounds; q += team_ctas) {
        const int tile = q * tiles_per_round + warp / n_slices, ks = warp % n_slices;
        if (tile < n_tiles) {
          const int mt = tile / NTILES, nt = tile % NTILES;
          const bool from_k = is_v && ks * kChainKS >= D;           // this slice reads the layer's fresh K^
          const uint16_t* A = from_k ? ly.Khat : prev;
          const long long ldA = from_k ? ly.ldHat : ld_prev;
          const int ka = from_k ? ks * kChainKS - D : ks * kChainKS;
          // the weight slice does not depend on anything: ask L2 for it before waiting
          {
            const uint16_t* pw = W + (long long)(nt * kChainNT + lane * 2) * ldW + ks * kChainKS;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(pw));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(pw + 64));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(pw + ldW));
            asm volatile("prefetch.global.L2 [%0];" ::"l"(pw + ldW + 64));
          }
          const int rows_mt = a.T - mt * kChainMT < kChainMT ? a.T - mt * kChainMT : kChainMT;
          bool ok = true;
          if (lane == 0) {
            // the previous layer's rows of this tile: they produced the input of the slices that read the
            // previous reconstruction, and they were the last readers of the prediction tile that this
            // round overwrites
            if (l > 0) ok = chain_wait(r_done + (l - 1) * n_mt + mt, rows_mt, abort_flag, a.status);
            if (ok && from_k) ok = chain_wait(kr_done + l * n_mt + mt, rows_mt, abort_flag, a.status);
          }
          ok = __shfl_sync(0xffffffffu, ok, 0);
          if (ok)
            chain_gemm_unit<kBf16>(A, ldA, ka, W, ldW, ks * kChainKS, mt * kChainMT, a.T, nt * kChainNT, sm->red[warp], lane);
        }
        __syncthreads();
        if (*abort_flag) { stop = true; break; }
        for (int o = threadIdx.x; o < tiles_per_round * kChainMT * kChainNT; o += kChainThreads) {
          const int ti = o / (kChainMT * kChainNT), idx = o % (kChainMT * kChainNT);
          const int tile2 = q * tiles_per_round + ti;
          if (tile2 >= n_tiles) break;
          float sum = sm->red[ti * n_slices][idx];
          for (int sl = 1; sl < n_slices; ++sl) sum += sm->red[ti * n_slices + sl][idx];
          const int row = (tile2 / NTILES) * kChainMT + idx / kChainNT, col = (tile2 % NTILES) * kChainNT + idx % kChainNT;
          if (row < a.T) P[(long long)row * D + col] = bias != nullptr ? sum + __ldg(bias + col) : sum;
        }
        __syncthreads();
        if (int(threadIdx.x) < tiles_per_round) {      // one releasing thread per tile, after the barrier
          const int tile2 = q * tiles_per_round + int(threadIdx.x);
          if (tile2 < n_tiles) {
            asm volatile("fence.acq_rel.gpu;" ::: "memory");     // release: the barrier above ordered the CTA's stores before it
            atomicAdd(g_done + l * n_mt + tile2 / NTILES, 1);
          }
        }
      }
      if (stop) break;
    }
    // ------------------------------------------------------------------------------------------
    // rows of this layer (TEAM warps per row)
    // ------------------------------------------------------------------------------------------
    // consecutive rows go to different CTAs, so that a stage of few rows has an SM per row
    const int team = (warp / TEAM) * team_ctas + cta, n_teams = n_warps / TEAM;
    for (int r = team; r < a.T; r += n_teams) {
      const int mt = r / kChainMT;
      float* pred_row = has_pred ? P + (long long)r * D : nullptr;
      uint8_t* codes_row = (is_v ? ly.Vcodes : ly.Kcodes) + (long long)r * CODE_BYTES;
      // the row's own input does not depend on the prediction: pull it towards L2 before waiting
      if constexpr (kEncode) {
        const uint16_t* x_row = (is_v ? ly.V : ly.K) + (long long)r * a.ldX;
        if (lane * 64 < D / TEAM) asm volatile("prefetch.global.L2 [%0];" ::"l"(x_row + rck.member * (D / TEAM) + lane * 64));
      } else {
        if (lane * 128 < CODE_BYTES / TEAM)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(codes_row + rck.member * (CODE_BYTES / TEAM) + lane * 128));
      }
      bool ok = true;
      if (has_pred) {
        if (TEAM > 1) {
          if (rck.member == 0 && lane == 0)
            chain_wait(g_done + l * n_mt + mt, NTILES, abort_flag, a.status);
          team_barrier<D>(rck.barrier);
          ok = *abort_flag == 0;
          team_barrier<D>(rck.barrier);
        } else {
          if (lane == 0) ok = chain_wait(g_done + l * n_mt + mt, NTILES, abort_flag, a.status);
          ok = __shfl_sync(0xffffffffu, ok, 0);
        }
        if (!ok) break;          // the abort flag is set: the CTA leaves at the next layer's barrier
      }
      uint16_t* hat_row = (is_v ? ly.Vhat : ly.Khat) + (long long)r * ly.ldHat;
      uint16_t* scales_row = (is_v ? ly.Vscales : ly.Kscales) + (long long)r * n_groups;
      if constexpr (WR) {
        unsigned long long* xbuf = sm->scratch.xbuf[warp];
        if constexpr (kEncode) {
          wr_encode_row<NPTS, kBf16>(wrc, &sm->tables, xbuf, (is_v ? ly.V : ly.K) + (long long)r * a.ldX, pred_row, codes_row,
                                     scales_row, hat_row);
        } else {
          wr_decode_row<NPTS, kBf16>(wrc, sm->tables.grid, xbuf, codes_row, scales_row, pred_row, hat_row);
        }
      } else {
        TeamSmem<D>* ts = &sm->scratch.team[warp / TEAM];
        if constexpr (kEncode) {
          encode_row<D, NPTS, kBf16>(rck, &sm->tables, ts, (is_v ? ly.V : ly.K) + (long long)r * a.ldX, pred_row, codes_row,
                                     scales_row, hat_row);
        } else {
          decode_row<D, NPTS, kBf16>(rck, sm->tables.grid, ts, codes_row, scales_row, pred_row, hat_row);
        }
      }
      if (TEAM > 1) team_barrier<D>(rck.barrier); else __syncwarp();
      if (rck.member == 0 && lane == 0) {
        asm volatile("fence.acq_rel.gpu;" ::: "memory");
        atomicAdd(r_done + l * n_mt + mt, 1);
      }
    }
  }
}

}  // namespace aquakv
