// One persistent kernel per layer call for Algorithm 2 (encode) and Algorithm 3 (decode) with
// predictors: the predictor GEMMs (the two predictions of Algorithm 2 / Algorithm 3) run on
// the tensor cores while, on the same SMs, other warps run the row work of the quantizer
// (Section 2 "Vector Quantization") and of the reconstruction on tokens whose prediction is
// already complete.  The fp32 prediction is handed from the GEMM warps to the row warps through a
// small ring of buffers that stays resident in L2; completion is tracked with counters in global
// memory.
//
// Work layout.  A token block is 128 tokens; a GEMM tile is one token block x 256 output features,
// so NTN = d_kv/256 CTAs share a token block.  CTAs run as pairs (clusters of two): pair p owns
// feature tile n = p % NTN and the two token-block slots ml = 2 * (p / NTN) + rank, and computes
// both tiles with one tcgen05.mma.cta_group::2 of M = 256: each CTA loads its own 128 token rows
// and HALF of the 256 weight rows, so a k-block costs 32 KB of L2 traffic per CTA instead of 48 KB
// (the GEMM is bound by L2 bandwidth, not by the tensor pipe).  Every "wave" covers
// gridDim.x / NTN token blocks.  For each wave a CTA computes
// its key-phase tile and its value-phase tile, and runs the row work of 128/NTN rows of its token
// block for both phases.  Jobs are ordered  K0, K1, V0, K2, V1, ..., so that the value-phase GEMM of
// a wave (which reads the reconstructed keys of that wave) is issued one job after its key rows.
//
// Dependencies (all counted per job j and token-block slot ml, targets NTN):
//   gemm_done[j][ml]  -- feature tiles of job j written to the ring        (row warps wait)
//   rows_done[j][ml]  -- row teams that finished job j on token block ml (target: CTAs per block
//                        x teams per CTA)                                    (the value-phase TMA
//                        producer waits for the key rows of its wave; the GEMM epilogue waits for
//                        job j - ring size before it overwrites that ring slot)
// Every job waits only on jobs with a smaller index (or the same index of the other role), so the
// schedule cannot dead-lock as long as all CTAs are resident, which the launch guarantees by using at
// most one CTA per SM.  Every wait is bounded; on expiry the CTA records AQUAKV_ERR_TIMEOUT and
// all its roles leave their loops.
//
// Warp roles: warp 0 = TMA producer, warp 1 = tensor-memory owner + MMA issuer, warps 2..5 =
// GEMM epilogue (tensor memory -> fp32 rows in the ring), then the row warps and, in the decoder
// instantiation that also attends (the attention read of Algorithm 4), four attention warps: as soon as the value
// rows of the CTA's token block are reconstructed they read the block's keys and values back from
// L2, form the single-query attention partials of the CTA's share of the KV heads for every sequence
// the block overlaps, and release the block's rows (attn_done), so that decoded rows which the
// caller does not ask for live only in a ring of three waves that never needs to reach DRAM.
#pragma once

#include "attn.cuh"
#include "codec.cuh"
#include "common.cuh"
#include "gemm_pred.cuh"
#include "rowwarp.cuh"

namespace aquakv {

// Operand stages of 32 KB per CTA: four, except three for the encoder with one warp per row (kWarpRows),
// whose row work is the longer side and whose shared memory is better spent on more row warps
// (measured: 3 and 4 stages alike).
constexpr int kLayerStagesMax = 4;
template <bool kEncode, bool kWarpRows> constexpr int kLayerStagesT = (kEncode && kWarpRows) ? 3 : 4;
constexpr int kPairBBytes = (kBN / 2) * kBK * 2;        // this CTA's half of a weight tile k-block
constexpr int kPairStageBytes = kABytes + kPairBBytes;   // 32 KB

// Row warps of a CTA.  With d_kv = 1024 and the Hadamard block and scale group spanning the whole row
// (kFull) a single warp owns a row (rowwarp.cuh); otherwise teams of d_kv/256 warps share a row
// (codec.cuh): 24 warps at 64 registers.  The register file is split over the SM's four schedulers, so
// the budget per thread follows from the warps per scheduler: 4 -> 128, 5 -> 96, 6 -> 80 registers.
//   encoder: its row work is the longer side of the kernel and gains from every resident warp, even at
//            80 registers (12 / 14 / 16 / 18-20 row warps measured: 1.51 / 1.48 / 1.38 / 1.46-1.48 ms per
//            131072 tokens);
//   decoder: the GEMM is the longer side; 10 row warps keep the CTA at 16 warps and 128 registers, which
//            lets a row issue its prediction loads before the look-ups and the rotation (8 / 10 / 12 row
//            warps: 0.836 / 0.801-0.809 / 0.835 ms per 131072 tokens).
constexpr int kWrEncodeWarps = 16;
constexpr int kWrDecodeWarps = 10;
constexpr int kWrAttnDecodeWarps = 6;  // beside four attention warps: again 16 warps and 128 registers, which the
                                       // attention warps need as much as the row warps (4 / 5 / 6 / 7 / 10 row warps:
                                       // 2.19 / 2.07 / 2.07 / 2.35 / 2.22 ms per 8 x 32768 tokens)
static_assert(kWrAttnDecodeWarps <= kWrDecodeWarps, "the decoder's shared memory is sized for kWrDecodeWarps row warps");
template <bool kEncode, int D, bool kFull, int kAttnHD = 0>
struct LayerGeom {
  static constexpr bool WR = D == 1024 && kFull;
  static constexpr int ROW_WARPS =
      WR ? (kEncode ? kWrEncodeWarps : (kAttnHD > 0 ? kWrAttnDecodeWarps : kWrDecodeWarps)) : 24;
  static constexpr int TEAM = WR ? 1 : RowTeam<D>::TEAM;
  static constexpr int TEAMS = ROW_WARPS / TEAM;          // rows a CTA works on at a time
  static constexpr int THREADS = 32 * (6 + ROW_WARPS);
  // With at most 16 warps per CTA (four per scheduler) a thread may use 128 registers: the row
  // routines then load ahead (next row's input, the prediction before the rotation).
  static constexpr bool AHEAD = WR && 6 + ROW_WARPS + (kAttnHD > 0 ? 4 : 0) <= 16;
};
constexpr int kAttnWarps = 4;
constexpr int kAttnSubTokens = 128;  // tokens of a token block that one attention warp covers (one partial slot each)
template <bool kEncode, int D, bool kFull, int kAttnHD>
constexpr int layer_threads() {
  return LayerGeom<kEncode, D, kFull, kAttnHD>::THREADS + (kAttnHD > 0 ? 32 * kAttnWarps : 0);
}

struct LayerSmemTail {
  uint64_t full[kLayerStagesMax];
  uint64_t empty[kLayerStagesMax];
  uint64_t acc_full[kAccStages];
  uint64_t acc_empty[kAccStages];
  uint32_t tmem_base;
  int abort_flag;
};

// Grid only (decode needs no search table).
template <int NPTS>
struct GridSmem {
  f32x2_t grid[NPTS];
};
template <bool kEncode, int NPTS> struct LayerTables { typedef RowSmem<NPTS> type; };
template <int NPTS> struct LayerTables<false, NPTS> { typedef GridSmem<NPTS> type; };

template <int D, int ROW_WARPS, bool WR> struct LayerRowScratch { TeamSmem<D> team[ROW_WARPS / RowTeam<D>::TEAM]; };
template <int D, int ROW_WARPS> struct LayerRowScratch<D, ROW_WARPS, true> { unsigned long long xbuf[ROW_WARPS][kWrItems]; };

template <bool kEncode, int D, int NPTS, bool kFull>
struct LayerRowSmem {
  typename LayerTables<kEncode, NPTS>::type tables;
  LayerRowScratch<D, LayerGeom<kEncode, D, kFull>::ROW_WARPS, LayerGeom<kEncode, D, kFull>::WR> scratch;
};

// The GEMM epilogue stages each 32-row x 32-column fp32 piece of a tile in shared memory (128-byte
// swizzle) and hands it to a TMA store.  With one warp per row: one 4 KB buffer per epilogue warp
// (two measured 2-3 % slower in the decoder and no faster in the encoder, where the space goes to
// the row warps).  With row teams: two, which the short calls of that path gain from, or one for the
// encoder with the 256-point grid, whose 2 KB grid would otherwise not fit.
constexpr int kEpiPieceBytes = 32 * 32 * 4;
template <bool kEncode, int NPTS, bool kWarpRows>
constexpr int kEpiBufs = (kWarpRows || (kEncode && NPTS > 64)) ? 1 : 2;
template <bool kEncode, int NPTS, bool kWarpRows>
constexpr int kEpiBytes = 4 * kEpiBufs<kEncode, NPTS, kWarpRows> * kEpiPieceBytes;

template <bool kEncode, int D, int NPTS, bool kFull>
constexpr size_t layer_smem_bytes() {
  constexpr bool WR = LayerGeom<kEncode, D, kFull>::WR;
  return 1024 + size_t(kLayerStagesT<kEncode, WR>) * kPairStageBytes + kEpiBytes<kEncode, NPTS, WR> + sizeof(LayerSmemTail) + 16 +
         sizeof(LayerRowSmem<kEncode, D, NPTS, kFull>);
}

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* smem_src, int32_t x, int32_t y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(
                   reinterpret_cast<uint64_t>(map)),
               "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void tma_store_2d_hint(const CUtensorMap* map, const void* smem_src, int32_t x, int32_t y,
                                                  uint64_t policy) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group.L2::cache_hint [%0, {%2, %3}], [%1], %4;" ::"l"(
                   reinterpret_cast<uint64_t>(map)),
               "r"(smem_u32(smem_src)), "r"(x), "r"(y), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

struct LayerArgs {
  int T;                  // tokens
  int n_mblocks;          // ceil(T / 128)
  int mw;                 // token blocks per wave (gridDim.x / NTN)
  int n_waves;
  int nb;                 // prediction buffers in the ring
  const float* bk;        // optional biases [d_kv]
  const float* bv;
  float* P;               // ring: [nb][mw * 128][d_kv] fp32
  int* gemm_done;         // [2 * n_waves][mw], zero at launch
  int* rows_done;         // [2 * n_waves][mw], zero at launch
  int khat_ring;          // 0: K^ rows are indexed by token; r > 0: ring of r waves (rows of mw*128)
  // encode inputs
  const uint16_t* K;
  const uint16_t* V;
  long long ldX;
  // compressed cache (written by encode, read by decode)
  uint8_t* Kcodes;
  uint16_t* Kscales;
  uint8_t* Vcodes;
  uint16_t* Vscales;
  // reconstructions
  uint16_t* Khat;         // output rows (khat_ring == 0) or the ring
  long long ldKhat;
  uint16_t* Vhat;         // output rows or nullptr (encode only)
  long long ldVhat;
  const uint32_t* signmask_k;
  const uint32_t* signmask_v;
  const float4* grid4;
  SearchDev search;
  int log_h, log_g;
  int* status;
  // single-query attention over the decoded rows (decoder instantiations with kAttnHD > 0)
  int vhat_ring;            // like khat_ring, for V^ (both rings or neither)
  const uint16_t* q;        // [batch][n_q_heads][head_dim]
  int ctx;                  // tokens per sequence: token t belongs to sequence t / ctx
  int n_q_heads, n_kv_heads;
  int n_splits;             // partial slots per sequence: slot s of sequence b = sub-block (of kAttnSubTokens tokens) b*ctx/kAttnSubTokens + s
  float scale_log2;         // softmax scale * log2(e)
  float* part_ml;           // [batch][n_splits][n_q_heads][2]
  float* part_o;            // [batch][n_splits][n_q_heads][head_dim]
  int* attn_done;           // [n_waves][mw], zero at launch: attention warps that are done with the block
};

// The layers of one launch.  A launch of several layers (Algorithm 2 / 3 inside Algorithm 4's loop over
// layers) runs them back to back without a barrier in between: every role walks the layers on its own,
// the prediction ring and its counters continue across the layer boundary, and a layer's first jobs start
// while the previous layer's last wave is still being finished (a layer's wave w needs only wave w of the
// layer before it).  All layers share T, the wave geometry and the ring.
struct LayerMaps {
  CUtensorMap kprev, vprev, khat, wk, wv, p;
};
constexpr int kLayerBatchMax = 24;      // 24 x (arguments + six tensor maps) stays inside the 32 KB of kernel parameters
template <int kBatch>
struct LayerBatch {
  int n_layers;
  LayerArgs layer[kBatch];
  LayerMaps maps[kBatch];
};
static_assert(sizeof(LayerBatch<kLayerBatchMax>) <= 32764, "kernel parameters are limited to 32764 bytes");

__device__ __forceinline__ void layer_job(int j, int n_waves, int& phase, int& wave) {
  if (j == 0) { phase = 0; wave = 0; }
  else if (j == 2 * n_waves - 1) { phase = 1; wave = n_waves - 1; }
  else if (j & 1) { phase = 0; wave = (j + 1) >> 1; }
  else { phase = 1; wave = (j >> 1) - 1; }
}
__device__ __forceinline__ int layer_key_job(int wave) { return wave == 0 ? 0 : 2 * wave - 1; }
__device__ __forceinline__ int layer_value_job(int wave, int n_waves) {
  return wave == n_waves - 1 ? 2 * n_waves - 1 : 2 * wave + 2;
}

// Row work of a wave is spread evenly over ALL CTAs: CTA slot s takes rows [s*rpc, (s+1)*rpc) of
// the wave, rpc = the power of two >= rows / CTAs.  For a full wave this is rpc = 128 / NTN rows of
// the CTA's own token block; in the short last wave it keeps every SM busy instead of a few.
struct WaveRows {
  int tokens;      // rows of the wave
  int blocks;      // token blocks of the wave
  int rpc;         // rows per CTA slot (power of two, <= 128 / NTN)
};
__device__ __forceinline__ WaveRows wave_rows(int wave, int T, int mw, int n_ctas) {
  WaveRows w;
  const long long left = (long long)T - (long long)wave * mw * kBM;
  w.tokens = left < (long long)mw * kBM ? int(left) : mw * kBM;
  w.blocks = (w.tokens + kBM - 1) / kBM;
  const int need = (w.tokens + n_ctas - 1) / n_ctas;
  int rpc = 1;
  while (rpc < need) rpc <<= 1;
  w.rpc = rpc;
  return w;
}

// Number of row teams that report on token block `block` of that wave (CTA slots on the block x teams).
__device__ __forceinline__ int wave_block_teams(const WaveRows& w, int block, int n_ctas, int teams) {
  const int per_block = kBM / w.rpc;
  const int hi = (block + 1) * per_block < n_ctas ? (block + 1) * per_block : n_ctas;
  const int n = hi - block * per_block;
  return (n > 0 ? n : 0) * teams;
}

__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// Spins until *ctr >= target.  Returns false after kWaitLimitNs or if the CTA already aborted.
__device__ __forceinline__ bool counter_wait_bounded(const int* ctr, int target, volatile int* abort_flag,
                                                     int* status) {
  if (ld_acquire(ctr) >= target) return true;
  const unsigned long long t0 = global_timer_ns();
  uint32_t spins = 0;
  uint32_t pause = 64;          // polls cost issue slots the row warps need: back off up to 2 us
  while (ld_acquire(ctr) < target) {
    __nanosleep(pause);
    if (pause < 2048) pause <<= 1;
    if ((++spins & 0x3Fu) == 0) {
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

__device__ __forceinline__ void named_barrier(int id, int threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(threads) : "memory");
}
__device__ __forceinline__ void fence_acq_rel_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async_all() {
  asm volatile("fence.proxy.async;" ::: "memory");
}

// kFull: the Hadamard block and the scale group both span the whole row (the paper's setting for
// d_kv = 1024, Section 4.1); their logarithms are then compile-time constants of the row code.
// kAttnHD: 0, or the head dimension (64 / 128) of the attention the decoder also computes.
template <bool kEncode, int D, int NPTS, bool kBf16, bool kFull, int kAttnHD = 0, int kBatch = 1>
__global__ void __launch_bounds__((layer_threads<kEncode, D, kFull, kAttnHD>()), 1)
layer_kernel(const __grid_constant__ LayerBatch<kBatch> B) {
  using G = LayerGeom<kEncode, D, kFull, kAttnHD>;
  const LayerArgs& a = B.layer[0];         // what all layers of the launch share: geometry, tables, status word
  const int n_layers = kBatch == 1 ? 1 : B.n_layers;
  constexpr int NTN = D / kBN;             // feature tiles per token block = CTAs per token block
  constexpr int NKD = D / kBK;             // k-blocks per d_kv input features
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = D / 2 * BITS / 8;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  uint8_t* epi_smem = smem + size_t(kLayerStagesT<kEncode, G::WR>) * kPairStageBytes;      // 1024-byte aligned
  LayerSmemTail* tail = reinterpret_cast<LayerSmemTail*>(epi_smem + kEpiBytes<kEncode, NPTS, G::WR>);
  LayerRowSmem<kEncode, D, NPTS, kFull>* rsm = reinterpret_cast<LayerRowSmem<kEncode, D, NPTS, kFull>*>(
      (reinterpret_cast<uintptr_t>(tail) + sizeof(LayerSmemTail) + 15) & ~uintptr_t(15));

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();          // 0 = leader of the pair (issues the MMAs)
  const int pair = blockIdx.x >> 1;
  const int ml = 2 * (pair / NTN) + int(rank);
  const int ml0 = 2 * (pair / NTN);                 // the pair is active in a wave iff its first block exists
  const int n_blk = pair % NTN;
  const int n_jobs = 2 * a.n_waves;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kLayerStagesT<kEncode, G::WR>; ++s) {
      mbar_init(&tail->full[s], 1);
      mbar_init(&tail->empty[s], 1);
    }
    for (int s = 0; s < kAccStages; ++s) {
      mbar_init(&tail->acc_full[s], 1);
      mbar_init(&tail->acc_empty[s], 8);     // 4 epilogue warps of each CTA (used in the leader only)
    }
    tail->abort_flag = 0;
    mbar_fence_init();
  }
  if constexpr (kEncode) {
    row_smem_fill<NPTS>(&rsm->tables, a.search.table, a.grid4);
  } else {
    for (int i = threadIdx.x; i < NPTS; i += blockDim.x) {
      const float4 g = a.grid4[i];
      rsm->tables.grid[i] = pack2(g.x, g.y);
    }
  }
  if (warp == 1) {
    tmem_alloc_pair(&tail->tmem_base, kTmemCols);
    tmem_relinquish_pair();
  }
  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();          // the peer's barriers are initialised before anything signals them
  tc_fence_after_sync();
  const uint32_t tmem_base = tail->tmem_base;
  volatile int* abort_flag = &tail->abort_flag;

  if (warp == 0) {
    // ------------------------------- TMA producer --------------------------------------------
    if (lane == 0) {
      const uint64_t pol_stream = l2_policy_evict_first(), pol_keep = l2_policy_evict_last();
      int stage = 0;
      uint32_t phase_bit = 0;
      bool ok = true;
      int issued = 0;
      for (int l = 0; ok && l < n_layers; ++l) {
      const LayerArgs& a = B.layer[l];
      const LayerMaps& tm = B.maps[l];
      tma_prefetch_desc(&tm.kprev);
      tma_prefetch_desc(&tm.vprev);
      tma_prefetch_desc(&tm.khat);
      tma_prefetch_desc(&tm.wk);
      tma_prefetch_desc(&tm.wv);
      for (int j = 0; ok && j < n_jobs; ++j) {
        int ph, wave;
        layer_job(j, a.n_waves, ph, wave);
        const int m = wave * a.mw + ml;
        if (wave * a.mw + ml0 >= a.n_mblocks) continue;
        const int nk = ph == 0 ? NKD : 2 * NKD;
        const int khat_row = a.khat_ring ? ((wave % a.khat_ring) * a.mw + ml) * kBM : m * kBM;
        for (int kb = 0; kb < nk; ++kb) {
          if (l > 0 && kb == 0 && m < a.n_mblocks) {
            // the previous layer of this launch wrote this job's first input (its reconstructed keys for
            // the key phase, values for the value phase): its row warps must be done with this token block
            const LayerArgs& pa = B.layer[l - 1];
            const int pj = ph == 0 ? layer_key_job(wave) : layer_value_job(wave, a.n_waves);
            const int target = wave_block_teams(wave_rows(wave, a.T, a.mw, gridDim.x), ml, gridDim.x, G::TEAMS);
            if (!counter_wait_bounded(pa.rows_done + pj * a.mw + ml, target, abort_flag, a.status)) {
              ok = false;
              break;
            }
            fence_proxy_async_all();
          }
          if (ph == 1 && kb == NKD && m < a.n_mblocks) {
            // the remaining k-blocks read this wave's reconstructed keys, written by row warps
            const int target = wave_block_teams(wave_rows(wave, a.T, a.mw, gridDim.x), ml, gridDim.x, G::TEAMS);
            if (!counter_wait_bounded(a.rows_done + layer_key_job(wave) * a.mw + ml, target, abort_flag,
                                      a.status)) {
              ok = false;
              break;
            }
            fence_proxy_async_all();
          }
          if (!mbar_wait_bounded(&tail->empty[stage], phase_bit ^ 1u, abort_flag, a.status)) {
            ok = false;
            break;
          }
          uint8_t* a_dst = smem + size_t(stage) * kPairStageBytes;
          uint8_t* b_dst = a_dst + kABytes;
          // the leader's barrier collects the bytes of both CTAs
          if (rank == 0) mbar_arrive_expect_tx(&tail->full[stage], 2 * kPairStageBytes);
          const int w_row = n_blk * kBN + int(rank) * (kBN / 2);     // this CTA's half of the weight rows
          // token rows stream through L2 once; the adapter tiles are read again by every wave
          if (ph == 0) {
            tma_load_2d_pair_hint(a_dst, &tm.kprev, &tail->full[stage], kb * kBK, m * kBM, pol_stream);
            tma_load_2d_pair_hint(b_dst, &tm.wk, &tail->full[stage], kb * kBK, w_row, pol_keep);
          } else {
            if (kb < NKD) {
              tma_load_2d_pair_hint(a_dst, &tm.vprev, &tail->full[stage], kb * kBK, m * kBM, pol_stream);
            } else {
              tma_load_2d_pair_hint(a_dst, &tm.khat, &tail->full[stage], (kb - NKD) * kBK, khat_row, pol_stream);
            }
            tma_load_2d_pair_hint(b_dst, &tm.wv, &tail->full[stage], kb * kBK, w_row, pol_keep);
          }
          ++issued;
          if (++stage == kLayerStagesT<kEncode, G::WR>) { stage = 0; phase_bit ^= 1u; }
        }
      }
      }   // layers
      if (!ok && rank == 0) {
        // let the copies in flight land before the shared memory is released
        int s = stage;
        uint32_t pb = phase_bit;
        const int pending = issued < kLayerStagesT<kEncode, G::WR> ? issued : kLayerStagesT<kEncode, G::WR>;
        for (int i = 0; i < pending; ++i) {
          if (s == 0) { s = kLayerStagesT<kEncode, G::WR>; pb ^= 1u; }
          --s;
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(&tail->full[s], pb) && global_timer_ns() - t0 < kWaitLimitNs) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer ----------------------------------------------
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = umma_idesc_f16(2 * kBM, kBN, kBf16);
      int stage = 0;
      uint32_t phase_bit = 0;
      bool ok = true;
      int it = 0;
      for (int l = 0; ok && l < n_layers; ++l)
      for (int j = 0; ok && j < n_jobs; ++j) {
        int ph, wave;
        layer_job(j, a.n_waves, ph, wave);
        if (wave * a.mw + ml0 >= a.n_mblocks) continue;
        const int nk = ph == 0 ? NKD : 2 * NKD;
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1u;
        ++it;
        if (!mbar_wait_bounded(&tail->acc_empty[acc], acc_phase ^ 1u, abort_flag, a.status)) { ok = false; break; }
        tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + uint32_t(acc * kBN);
        for (int kb = 0; kb < nk; ++kb) {
          if (!mbar_wait_bounded(&tail->full[stage], phase_bit, abort_flag, a.status)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(smem + size_t(stage) * kPairStageBytes);
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            const uint64_t da = umma_smem_desc_k128(a_addr + k * kUmmaK * 2);
            const uint64_t db = umma_smem_desc_k128(b_addr + k * kUmmaK * 2);
            umma_f16_pair(tmem_d, da, db, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          umma_commit_pair(&tail->empty[stage]);   // frees the stage in both CTAs
          if (++stage == kLayerStagesT<kEncode, G::WR>) { stage = 0; phase_bit ^= 1u; }
        }
        if (ok) umma_commit_pair(&tail->acc_full[acc]);
      }
    }
  } else if (warp < 6) {
    // ------------------------------- GEMM epilogue (4 warps) ---------------------------------
    const int quarter = warp & 3;   // tensor-memory lanes [32*quarter, 32*quarter+32)
    int it = 0;
    bool stop = false;
    for (int l = 0; !stop && l < n_layers; ++l) {
    const LayerArgs& a = B.layer[l];
    const LayerMaps& tm = B.maps[l];
    for (int j = 0; j < n_jobs; ++j) {
      int ph, wave;
      layer_job(j, a.n_waves, ph, wave);
      if (wave * a.mw + ml0 >= a.n_mblocks) continue;
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1u;
      ++it;
      bool ok = true;
      // the ring slot of this job was last used nb jobs earlier (counted through the layers of the launch):
      // that job's row work must be over
      const int gj = l * n_jobs + j;
      // ... the latest such job in whose wave this token block exists (the short last wave may not have it:
      // nobody then read or reports on this block's part of the slot)
      int go = gj - a.nb, ph_old = 0, wave_old = 0;
      while (go >= 0) {
        layer_job(go % n_jobs, a.n_waves, ph_old, wave_old);
        if (ml < wave_rows(wave_old, a.T, a.mw, gridDim.x).blocks) break;
        go -= a.nb;
      }
      if (go >= 0) {
        const int lo = go / n_jobs, jo = go % n_jobs;
        const int target = wave_block_teams(wave_rows(wave_old, a.T, a.mw, gridDim.x), ml, gridDim.x, G::TEAMS);
        // one thread polls for the four warps; a failed wait has set the abort flag
        if (warp == 2 && lane == 0)
          counter_wait_bounded(B.layer[lo].rows_done + jo * a.mw + ml, target, abort_flag, a.status);
        named_barrier(1, 128);
        ok = *abort_flag == 0;
      }
      if (ok) ok = mbar_wait_bounded(&tail->acc_full[acc], acc_phase, abort_flag, a.status);
      if (ok) {
        tc_fence_after_sync();
        const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(acc * kBN);
        // ring row of this warp's 32 tokens; rows past the last token are written too (never read)
        const int ring_row = (gj % a.nb) * a.mw * kBM + ml * kBM + quarter * 32;
        const float* bias = ph == 0 ? a.bk : a.bv;
        constexpr int EB = kEpiBufs<kEncode, NPTS, G::WR>;
        const uint64_t pol_keep = l2_policy_evict_last();
        uint8_t* my_epi = epi_smem + (warp - 2) * EB * kEpiPieceBytes;
#pragma unroll 1
        for (int c = 0; c < kBN / 32; ++c) {
          float v[32];
          tmem_ld_32x32b_x32(taddr + uint32_t(c * 32), v);
          if (bias != nullptr) {
            const float* b = bias + n_blk * kBN + c * 32;
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __fadd_rn(v[i], __ldg(b + i));
          }
          uint8_t* buf = my_epi + (c & (EB - 1)) * kEpiPieceBytes;
          if (c >= EB) {                 // the store that last read this buffer must be done with it
            if (lane == 0) {
              if constexpr (EB == 2) bulk_wait_read_1(); else bulk_wait_read_0();
            }
            __syncwarp();
          }
          // lane = row of the piece; 16-byte chunk q of row r sits at chunk position q ^ (r % 8)
#pragma unroll
          for (int q = 0; q < 8; ++q)
            *reinterpret_cast<float4*>(buf + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) {
            tma_store_2d_hint(&tm.p, buf, n_blk * kBN + c * 32, ring_row, pol_keep);   // read back soon by the row warps
            bulk_commit();
          }
        }
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_leader(&tail->acc_empty[acc]);   // the leader's MMA issuer waits for both CTAs
          bulk_wait_all();               // the tile's rows are written
          fence_proxy_async_all();
        }
        __syncwarp();
      }
      // release by one thread after the barrier: its fence also covers the stores of the threads it
      // has synchronised with, and only that thread waits for them to become visible
      named_barrier(1, 128);
      if (*abort_flag) { stop = true; break; }
      if (warp == 2 && lane == 0) {
        __threadfence();
        atomicAdd(a.gemm_done + j * a.mw + ml, 1);
      }
    }
    }   // layers
  } else if (warp < 6 + G::ROW_WARPS) {
    // ------------------------------- row warps (TEAM warps per row; TEAMS rows at a time) ------
    constexpr int TEAM = G::TEAM, TEAMS = G::TEAMS;
    const int rw = warp - 6;
    const int team = rw / TEAM;
    constexpr int LOG_D = D == 1024 ? 10 : (D == 512 ? 9 : 8);
    const int log_h = kFull ? LOG_D : a.log_h, log_g = kFull ? LOG_D : a.log_g;
    // one context per warp; the sign bits are switched between key and value jobs
    RowCtx rck;
    WarpRowCtx wrc;
    uint32_t signs_k, signs_v;
    if constexpr (G::WR) {
      wrc.lane = lane;
      wrc.inv_w = a.search.inv_w;
      wrc.signs = 0u;
      signs_k = a.signmask_k[lane];
      signs_v = a.signmask_v[lane];
      rck.member = 0;
      rck.barrier = 0;
    } else {
      row_ctx_init(rck, a.signmask_k, a.search.inv_w, log_h, log_g, lane, rw % TEAM, RowTeam<D>::NV, 3 + team);
      signs_k = a.signmask_k[lane] >> (rck.member * RowTeam<D>::NV);
      signs_v = a.signmask_v[lane] >> (rck.member * RowTeam<D>::NV);
    }
    const int n_groups = D >> log_g;
    bool stop = false;
    for (int l = 0; !stop && l < n_layers; ++l) {
    const LayerArgs& a = B.layer[l];
    for (int j = 0; j < n_jobs; ++j) {
      int ph, wave;
      layer_job(j, a.n_waves, ph, wave);
      const int gj = l * n_jobs + j;
      const WaveRows wr = wave_rows(wave, a.T, a.mw, gridDim.x);
      if (wr.tokens <= 0) continue;
      if constexpr (G::WR) wrc.signs = ph == 0 ? signs_k : signs_v;
      else row_ctx_set_signs(rck, ph == 0 ? signs_k : signs_v);
      const int slot_row = (ml * NTN + n_blk) * wr.rpc;      // first row (within the wave) of this CTA's slice
      const int rb = slot_row / kBM;                         // token block (within the wave) the slice lies in
      if (rb >= wr.blocks) continue;                         // nothing assigned, nobody waits for this CTA
      const int r_begin = slot_row % kBM;
      const int m = wave * a.mw + rb;
      const long long rows_left = (long long)a.T - (long long)m * kBM;
      const int r_end = rows_left < r_begin + wr.rpc ? int(rows_left) : r_begin + wr.rpc;
      if constexpr (kEncode) {
        // pull this job's input rows towards L2 while the prediction is still being produced
        const uint16_t* xin = ph == 0 ? a.K : a.V;
        for (int r = r_begin + (team + j) % TEAMS; r < r_end; r += TEAMS) {
          const long long g = (long long)m * kBM + r;
          if (lane < D / 256 / TEAM * 4)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(xin + g * a.ldX + rck.member * (D / TEAM) + lane * 64));
        }
      }
      bool ok = true;
      if constexpr (kAttnHD > 0) {
        // this layer's rows overwrite the reconstructions of two layers earlier (the caller alternates
        // two buffer pairs), which that layer's attention warps may, in principle, still be reading
        if (l >= 2) {
          if (lane == 0)
            ok = counter_wait_bounded(B.layer[l - 2].attn_done + wave * a.mw + rb, NTN * kAttnWarps, abort_flag, a.status);
          ok = __shfl_sync(0xffffffffu, ok, 0);
        }
        // the key rows of this wave reuse the ring rows of wave - ring depth: the attention warps must
        // be done with them (they trail the rows by about one job, so this rarely waits)
        if (ok && ph == 0 && a.khat_ring > 0 && wave >= a.khat_ring) {
          if (lane == 0)
            ok = counter_wait_bounded(a.attn_done + (wave - a.khat_ring) * a.mw + rb, NTN * kAttnWarps, abort_flag,
                                      a.status);
          ok = __shfl_sync(0xffffffffu, ok, 0);
        }
      }
      if (!ok) {
        // fall through to the report below with the abort flag set
      } else if (TEAM > 1) {
        // one thread polls for the team; all its warps must take the same path, so they agree
        // through the abort flag (set by a failed wait) between two barriers
        if (rck.member == 0 && lane == 0)
          counter_wait_bounded(a.gemm_done + j * a.mw + rb, NTN, abort_flag, a.status);
        team_barrier<D>(rck.barrier);
        ok = *abort_flag == 0;
        team_barrier<D>(rck.barrier);
      } else {
        if (lane == 0) ok = counter_wait_bounded(a.gemm_done + j * a.mw + rb, NTN, abort_flag, a.status);
        ok = __shfl_sync(0xffffffffu, ok, 0);
      }
      if (ok) {
        const float* pbuf = a.P + (size_t(gj % a.nb) * a.mw * kBM + size_t(rb) * kBM) * D;
        const size_t khat_base = a.khat_ring ? size_t((wave % a.khat_ring) * a.mw + rb) * kBM
                                             : size_t(m) * kBM;
        [[maybe_unused]] uint4 xraw[4];
        [[maybe_unused]] bool first_row = true;
        for (int r = r_begin + (team + j) % TEAMS; r < r_end; r += TEAMS) {   // rotated per job for balance
          const long long g = (long long)m * kBM + r;
          const float* pred_row = pbuf + size_t(r) * D;
          uint16_t* hat_row;
          if (ph == 0) hat_row = a.Khat + (khat_base + r) * a.ldKhat;
          else if (a.vhat_ring) hat_row = a.Vhat + (khat_base + r) * a.ldVhat;     // same ring geometry as K^
          else hat_row = a.Vhat != nullptr ? a.Vhat + g * a.ldVhat : nullptr;
          uint8_t* codes_row = (ph == 0 ? a.Kcodes : a.Vcodes) + g * CODE_BYTES;
          uint16_t* scales_row = (ph == 0 ? a.Kscales : a.Vscales) + g * n_groups;
          if constexpr (G::WR) {
            unsigned long long* xbuf = rsm->scratch.xbuf[rw];
            if constexpr (kEncode) {
              const uint16_t* x_row = (ph == 0 ? a.K : a.V) + g * a.ldX;
              if constexpr (G::AHEAD) {
                if (first_row) wr_load_x_row(x_row, lane, xraw);
                first_row = false;
                const uint16_t* x_next = r + TEAMS < r_end ? x_row + TEAMS * a.ldX : nullptr;
                wr_encode_row_x<NPTS, kBf16, true>(wrc, &rsm->tables, xbuf, xraw, x_next, pred_row, codes_row, scales_row,
                                                   hat_row);
              } else {
                wr_encode_row<NPTS, kBf16>(wrc, &rsm->tables, xbuf, x_row, pred_row, codes_row, scales_row, hat_row);
              }
            } else {
              wr_decode_row<NPTS, kBf16, false, G::AHEAD>(wrc, rsm->tables.grid, xbuf, codes_row, scales_row, pred_row,
                                                          hat_row);
            }
          } else {
            TeamSmem<D>* ts = &rsm->scratch.team[team];
            if constexpr (kEncode) {
              const uint16_t* x_row = (ph == 0 ? a.K : a.V) + g * a.ldX;
              encode_row<D, NPTS, kBf16>(rck, &rsm->tables, ts, x_row, pred_row, codes_row,
                                         scales_row, hat_row);
            } else {
              decode_row<D, NPTS, kBf16>(rck, rsm->tables.grid, ts, codes_row, scales_row,
                                         pred_row, hat_row);
            }
          }
          // The row's prediction has been read for the last time: drop its lines from L2 without
          // writing them back (the ring is scratch; only whole, 128-byte aligned lines are dropped).
          if (hat_row != nullptr || !kEncode) {
            __syncwarp();
            if constexpr (G::WR) {
              const float* mine = pred_row + lane * 32;             // the row's 32 lines, one per lane
              if ((reinterpret_cast<uintptr_t>(mine) & 127) == 0)
                asm volatile("discard.global.L2 [%0], 128;" ::"l"(mine) : "memory");
            } else {
              const float* mine = pred_row + rck.member * 256 + lane * 8;
              if ((lane & 3) == 0 && (reinterpret_cast<uintptr_t>(mine) & 127) == 0)
                asm volatile("discard.global.L2 [%0], 128;" ::"l"(mine) : "memory");
            }
          }
        }
      }
      // each team reports on its own, so a slow team never holds the others back
      if (TEAM > 1) team_barrier<D>(rck.barrier); else __syncwarp();
      if (*abort_flag) { stop = true; break; }
      if (rck.member == 0 && lane == 0) {   // one releasing thread per team (see the epilogue)
        // Key rows are read back by other CTAs' TMA loads (value-phase GEMM) and, like the value rows,
        // by other CTAs' attention warps: those need the stores released, the TMA also across the
        // proxies.  Value rows without attention are read by nobody in this launch; the counter then
        // only tells the epilogue that the ring slot's prediction has been read (the row's stores
        // depend on those loads, so they have completed).  With a further layer in the launch the value
        // rows are read by its TMA loads like the key rows.
        if (ph == 0 || l + 1 < n_layers) {
          fence_acq_rel_gpu();
          fence_proxy_async_all();
        } else if (kAttnHD > 0) {
          fence_acq_rel_gpu();
        }
        atomicAdd(a.rows_done + j * a.mw + rb, 1);
      }
    }
    }   // layers
  } else {
    // ------------------------------- attention warps ------------------------------------------------
    if constexpr (kAttnHD > 0) {
      // A warp takes one KV head, 64 of its output dimensions (with head_dim 128 two warps share a head)
      // and one sub-block of kAttnSubTokens tokens of the token block; every (sub-block, sequence) has
      // its own partial slot.  (Eight warps on 64-token sub-blocks measured slower than four on whole
      // blocks: the kernel then runs at 80 registers and the row warps spill.)
      constexpr int WPH = kAttnHD / 64;                // warps per head and sub-block
      constexpr int NSUB = kBM / kAttnSubTokens;       // sub-blocks of a token block
      constexpr int HPAR = kAttnWarps / (WPH * NSUB);  // heads in flight per CTA
      const int aw = warp - 6 - G::ROW_WARPS;
      const int half = aw % WPH;
      const int sub = (aw / WPH) % NSUB;
      const int hpc = a.n_kv_heads / NTN;              // KV heads of a token block that this CTA attends over
      const int rep = a.n_q_heads / a.n_kv_heads;
      bool stop = false;
      for (int l = 0; !stop && l < n_layers; ++l) {
      const LayerArgs& a = B.layer[l];
      for (int wave = 0; wave < a.n_waves; ++wave) {
        const WaveRows wr = wave_rows(wave, a.T, a.mw, gridDim.x);
        if (ml >= wr.blocks) continue;                  // this CTA's block does not exist in the (last) wave
        bool ok = true;
        if (lane == 0)
          ok = counter_wait_bounded(a.rows_done + layer_value_job(wave, a.n_waves) * a.mw + ml,
                                    wave_block_teams(wr, ml, gridDim.x, G::TEAMS), abort_flag, a.status);
        ok = __shfl_sync(0xffffffffu, ok, 0);
        if (!ok) { stop = true; break; }
        const long long blk = (long long)wave * a.mw + ml;       // token block of the call
        const long long sblk = blk * NSUB + sub;                 // this warp's sub-block of the call
        const long long tok0 = sblk * kAttnSubTokens;
        const long long tok1 = tok0 + kAttnSubTokens < a.T ? tok0 + kAttnSubTokens : a.T;
        const long long ring_row0 =
            a.khat_ring ? ((long long)(wave % a.khat_ring) * a.mw + ml) * kBM + sub * kAttnSubTokens : tok0;
        for (int h = n_blk * hpc + aw / (WPH * NSUB); h < (n_blk + 1) * hpc; h += HPAR) {
          long long t = tok0;
          while (t < tok1) {                            // one segment per sequence the sub-block overlaps
            const long long b = t / a.ctx;
            const long long seg_end = (b + 1) * a.ctx < tok1 ? (b + 1) * a.ctx : tok1;
            const long long row = ring_row0 + (t - tok0);
            const long long split = sblk - (b * a.ctx) / kAttnSubTokens;
            const long long pidx = (b * a.n_splits + split) * a.n_q_heads + (long long)h * rep;
            attn_segment_warp<kAttnHD, kBf16>(a.Khat + row * a.ldKhat + h * kAttnHD,
                                              a.Vhat + row * a.ldVhat + h * kAttnHD + half * 64, a.ldKhat, a.ldVhat,
                                              int(seg_end - t), a.q + (b * a.n_q_heads + (long long)h * rep) * kAttnHD,
                                              rep, a.scale_log2, half == 0 ? a.part_ml + pidx * 2 : nullptr,
                                              a.part_o + pidx * kAttnHD + half * 64, lane);
            t = seg_end;
          }
        }
        __syncwarp();
        if (lane == 0) {
          __threadfence();
          atomicAdd(a.attn_done + wave * a.mw + ml, 1);
        }
      }
      }   // layers
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  cluster_sync_all();          // neither CTA leaves while its peer may still signal its barriers
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

}  // namespace aquakv
