// Predictor GEMM (the predictions of Algorithm 2 and Algorithm 3; Section 3.2: the
// predictors are linear):  P[t][c] = sum_r X[t][r] * W[c][r] (+ bias[c]),  fp32 accumulate.
//
// X is the row-wise concatenation of up to two token-major 16-bit tensors (the value predictor
// reads [Vhat_prev ; Khat]); W is [d_kv][n_in*d_kv] row-major, so both operands are K-major for
// the tensor core.  One persistent CTA per SM walks 128x256 output tiles; operands arrive by TMA
// (128-byte swizzle, 4-stage ring), tcgen05.mma accumulates in tensor memory (two 256-column
// accumulators so a tile's epilogue overlaps the next tile's MMAs), and four epilogue warps read
// the accumulator back with tcgen05.ld and write fp32 rows.
//
// Warp roles: warp 0 = TMA producer, warp 1 = TMEM owner + MMA issuer, warps 2..5 = epilogue.
// Every wait is bounded (see mbar_wait_bounded); on expiry the CTA records AQUAKV_ERR_TIMEOUT,
// drains its outstanding copies, frees its tensor memory and returns.
#pragma once

#include "common.cuh"

namespace aquakv {

constexpr int kBM = 128;            // tokens per tile (MMA M)
constexpr int kBN = 256;            // output features per tile (MMA N)
constexpr int kBK = 64;             // 16-bit elements per k-block = one 128-byte swizzle row
constexpr int kStages = 4;
constexpr int kAccStages = 2;
constexpr int kUmmaK = 16;
constexpr int kABytes = kBM * kBK * 2;
constexpr int kBBytes = kBN * kBK * 2;
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kGemmThreads = 192;
constexpr int kTmemCols = kAccStages * kBN;   // 512: the whole tensor memory of the SM

struct GemmSmemTail {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t acc_full[kAccStages];
  uint64_t acc_empty[kAccStages];
  uint32_t tmem_base;
  int abort_flag;
};

constexpr size_t kGemmSmemBytes = 1024 /*alignment slack*/ + size_t(kStages) * kStageBytes +
                                  sizeof(GemmSmemTail);

struct GemmArgs {
  int M;              // tokens
  int N;              // output features (d_kv), multiple of kBN
  int nk0;            // k-blocks taken from the first input tensor
  int nk1;            // k-blocks taken from the second input tensor (0 = single input)
  float* P;           // [M, ldP] fp32 out
  long long ldP;
  const float* bias;  // [N] or nullptr
  int* status;
};

template <bool kBf16>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_pred_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
                 const __grid_constant__ CUtensorMap tmB, const GemmArgs args) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) &
                                             ~uintptr_t(1023));
  GemmSmemTail* tail = reinterpret_cast<GemmSmemTail*>(smem + size_t(kStages) * kStageBytes);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int n_tiles_n = args.N / kBN;
  const int n_tiles_m = (args.M + kBM - 1) / kBM;
  const int n_tiles = n_tiles_m * n_tiles_n;
  const int nk = args.nk0 + args.nk1;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&tail->full[s], 1);
      mbar_init(&tail->empty[s], 1);
    }
    for (int a = 0; a < kAccStages; ++a) {
      mbar_init(&tail->acc_full[a], 1);
      mbar_init(&tail->acc_empty[a], 4);
    }
    tail->abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(&tail->tmem_base, kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = tail->tmem_base;
  volatile int* abort_flag = &tail->abort_flag;

  if (warp == 0) {
    // ------------------------------- TMA producer --------------------------------------------
    if (lane == 0) {
      tma_prefetch_desc(&tmA0);
      tma_prefetch_desc(&tmA1);
      tma_prefetch_desc(&tmB);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int issued = 0;   // k-blocks issued in total (to drain on abort)
      for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x) {
        const int m_blk = tile / n_tiles_n, n_blk = tile % n_tiles_n;
        for (int kb = 0; kb < nk; ++kb) {
          if (!mbar_wait_bounded(&tail->empty[stage], phase ^ 1u, abort_flag, args.status)) {
            ok = false;
            break;
          }
          uint8_t* a_dst = smem + size_t(stage) * kStageBytes;
          uint8_t* b_dst = a_dst + kABytes;
          mbar_arrive_expect_tx(&tail->full[stage], kStageBytes);
          if (kb < args.nk0) {
            tma_load_2d(a_dst, &tmA0, &tail->full[stage], kb * kBK, m_blk * kBM);
          } else {
            tma_load_2d(a_dst, &tmA1, &tail->full[stage], (kb - args.nk0) * kBK, m_blk * kBM);
          }
          tma_load_2d(b_dst, &tmB, &tail->full[stage], kb * kBK, n_blk * kBN);
          ++issued;
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        // Let this CTA's copies in flight land before its shared memory is released: wait
        // (bounded, ignoring the abort flag) for the most recently armed phase of each stage.
        int s = stage;
        uint32_t ph = phase;
        const int pending = issued < kStages ? issued : kStages;
        for (int i = 0; i < pending; ++i) {
          if (s == 0) { s = kStages; ph ^= 1u; }
          --s;
          const unsigned long long t0 = global_timer_ns();
          while (!mbar_try_wait(&tail->full[s], ph) && global_timer_ns() - t0 < kWaitLimitNs) {
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------- MMA issuer ----------------------------------------------
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_f16(kBM, kBN, kBf16);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      int it = 0;
      for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++it) {
        const int acc = it & 1;
        const uint32_t acc_phase = (it >> 1) & 1u;
        if (!mbar_wait_bounded(&tail->acc_empty[acc], acc_phase ^ 1u, abort_flag, args.status)) {
          ok = false;
          break;
        }
        tc_fence_after_sync();
        const uint32_t tmem_d = tmem_base + uint32_t(acc * kBN);
        for (int kb = 0; kb < nk; ++kb) {
          if (!mbar_wait_bounded(&tail->full[stage], phase, abort_flag, args.status)) {
            ok = false;
            break;
          }
          tc_fence_after_sync();
          const uint32_t a_addr = smem_u32(smem + size_t(stage) * kStageBytes);
          const uint32_t b_addr = a_addr + kABytes;
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            const uint64_t da = umma_smem_desc_k128(a_addr + k * kUmmaK * 2);
            const uint64_t db = umma_smem_desc_k128(b_addr + k * kUmmaK * 2);
            umma_f16(tmem_d, da, db, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          umma_commit(&tail->empty[stage]);   // frees the smem slot once these MMAs have read it
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (ok) umma_commit(&tail->acc_full[acc]);
      }
    }
  } else {
    // ------------------------------- epilogue (4 warps) --------------------------------------
    const int quarter = warp & 3;   // TMEM lanes [32*quarter, 32*quarter+32) belong to this warp
    bool ok = true;
    int it = 0;
    for (int tile = blockIdx.x; ok && tile < n_tiles; tile += gridDim.x, ++it) {
      const int m_blk = tile / n_tiles_n, n_blk = tile % n_tiles_n;
      const int acc = it & 1;
      const uint32_t acc_phase = (it >> 1) & 1u;
      if (!mbar_wait_bounded(&tail->acc_full[acc], acc_phase, abort_flag, args.status)) {
        ok = false;
        break;
      }
      tc_fence_after_sync();
      const int row = m_blk * kBM + quarter * 32 + lane;
      const uint32_t taddr = tmem_base + (uint32_t(quarter * 32) << 16) + uint32_t(acc * kBN);
      float* out = args.P + (long long)row * args.ldP + n_blk * kBN;
#pragma unroll 1
      for (int c = 0; c < kBN / 32; ++c) {
        float v[32];
        tmem_ld_32x32b_x32(taddr + uint32_t(c * 32), v);
        if (row < args.M) {
          if (args.bias != nullptr) {
            const float* b = args.bias + n_blk * kBN + c * 32;
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = __fadd_rn(v[i], __ldg(b + i));
          }
#pragma unroll
          for (int i = 0; i < 32; i += 4)
            *reinterpret_cast<float4*>(out + c * 32 + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
        }
      }
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&tail->acc_empty[acc]);
    }
  }

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
}

}  // namespace aquakv
