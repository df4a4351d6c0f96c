// Row routines of the backbone quantizer Q / Q^-1 (Section 2 "Vector Quantization", Section 4.1
// "Alternative quantizers") and of the residual / add-back steps of Algorithm 2 and
// Algorithm 3 for the paper's main setting: d_kv = 1024 with the Hadamard block and the
// scale group spanning the whole token row.
//
// ONE warp owns a token row; each lane holds 32 of its 1024 values as 16 packed fp32 pairs.  The
// ten butterfly stages of the 1024-point Hadamard transform are split so that nine of them are
// register-local:
//   load layout     lane L, pair k = 4c + r/2 holds elements e = 256c + 8L + r, r = 2(k%4), +1
//                   (16-byte global accesses, whole 128-byte lines per warp);
//                   element index bits 0, 1, 2, 8, 9 select a register  -> five stages in registers
//   transposition   through a 4 KB shared-memory buffer of the warp: within each half-warp the
//                   pair index k (bits 1, 2, 8, 9) trades places with the lane index (bits 3..6)
//   search layout   lane L', pair m holds elements with bits 3..6 = m, bits (1, 2, 8, 9) = L' % 16,
//                   bit 7 = L' / 16                                        -> four stages in registers
//   bit 7           one shuffle stage between the two half-warps.
// The two values that share a code (2j, 2j+1) stay in one register pair throughout.  Compared with
// a row spread over four warps (codec.cuh) this removes four of five shuffle stages and all
// cross-warp barriers: the row work is bound by the SM's load/store and shuffle pipe, which the
// tensor-core GEMM beside it also needs for its operand reads.
//
// In the search layout lane L' holds the codes of pairs j = (L' % 4) + 4m + 64q, m = 0..15, with
// q = L'/16 + 2 * ((L'/4) % 2) + 4 * ((L'/8) % 2): four neighbouring lanes together hold one chunk of
// 64 consecutive codes (8 * BITS bytes of the row's bit stream) and merge or split it with shuffles.
#pragma once

#include "codec.cuh"

namespace aquakv {

constexpr int kWrItems = 2 * 16 * 16;      // 64-bit items of a warp's transposition buffer (4 KB)

struct WarpRowCtx {
  uint32_t signs;    // bit i set <=> value i (pair i/2, half i%2) of this lane in the load layout is multiplied by -1
  float inv_w;       // SearchDev::inv_w
  int lane;
};

// This lane's eight fp32 prediction values of one 256-element chunk as four packed pairs, in ONE
// 32-byte load: a warp's request then covers 1 KB of whole 32-byte sectors.  (Two 16-byte loads per
// lane would each touch all 32 sectors of that kilobyte and use half of every one; the loads bypass
// L1, because another SM wrote the prediction just before, so each would fetch them from L2 again.)
// p must be 32-byte aligned.
__device__ __forceinline__ void wr_load_pred8(const float* p, f32x2_t (&out)[4]) {
  asm volatile("ld.global.cg.v4.b64 {%0, %1, %2, %3}, [%4];"
               : "=l"(out[0]), "=l"(out[1]), "=l"(out[2]), "=l"(out[3])
               : "l"(p)
               : "memory");
}

// Butterfly over element index bit 0: inside each packed pair.
__device__ __forceinline__ void wr_stage_pair(f32x2_t (&vp)[16]) {
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    float a, b;
    unpack2(vp[k], a, b);
    vp[k] = pack2(a + b, a - b);
  }
}

// Butterflies over the four index bits that select one of the lane's 16 pairs, ascending.
__device__ __forceinline__ void wr_stage_regs(f32x2_t (&vp)[16]) {
#pragma unroll
  for (int s = 0; s < 4; ++s) {
    const int m = 1 << s;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      if ((k & m) == 0) {
        const f32x2_t x = vp[k], y = vp[k | m];
        vp[k] = add2(x, y);
        vp[k | m] = sub2(x, y);
      }
    }
  }
}

// Butterfly between the two half-warps (element index bit 7 in the search layout).
__device__ __forceinline__ void wr_stage_halves(f32x2_t (&vp)[16], int lane) {
  const float sg = (lane & 16) ? -1.0f : 1.0f;
  const f32x2_t sg2 = pack2(sg, sg);
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    float a, c;
    unpack2(vp[k], a, c);
    const float oa = __shfl_xor_sync(0xffffffffu, a, 16);
    const float oc = __shfl_xor_sync(0xffffffffu, c, 16);
    vp[k] = fma2(sg2, vp[k], pack2(oa, oc));   // lower half: v + o; upper half: o - v
  }
}

// Trades the pair index for the low four lane bits inside each half-warp: afterwards pair m of lane
// l holds what pair l of lane m held.  Item (k, l) sits at column l ^ k of row k, so the 16 lanes of
// a half-warp touch 16 different 8-byte columns both when they write (fixed k) and when they read
// (row = lane): no bank conflicts.  The same call converts in both directions.
__device__ __forceinline__ void wr_transpose(f32x2_t (&vp)[16], unsigned long long* xbuf, int lane) {
  unsigned long long* half = xbuf + (lane >> 4) * 256;
  const int l = lane & 15;
#pragma unroll
  for (int k = 0; k < 16; ++k) half[k * 16 + (l ^ k)] = vp[k];
  __syncwarp();
#pragma unroll
  for (int m = 0; m < 16; ++m) vp[m] = half[l * 16 + (m ^ l)];
  __syncwarp();
}

// H_1024 (unnormalised) from the load layout to the search layout.
__device__ __forceinline__ void wr_rotate_forward(f32x2_t (&vp)[16], unsigned long long* xbuf, int lane) {
  wr_stage_pair(vp);
  wr_stage_regs(vp);
  wr_transpose(vp, xbuf, lane);
  wr_stage_regs(vp);
  wr_stage_halves(vp, lane);
}

// H_1024 (unnormalised) from the search layout back to the load layout.  Encode and decode both
// reconstruct through this one routine, so their results agree bit for bit.
__device__ __forceinline__ void wr_rotate_back(f32x2_t (&wp)[16], unsigned long long* xbuf, int lane) {
  wr_stage_halves(wp, lane);
  wr_stage_regs(wp);
  wr_transpose(wp, xbuf, lane);
  wr_stage_regs(wp);
  wr_stage_pair(wp);
}

// Multiplies value i of the lane by -1 where bit i of `signs` is set (load layout).
__device__ __forceinline__ void wr_apply_signs(f32x2_t (&vp)[16], uint32_t signs) {
#pragma unroll
  for (int k = 0; k < 16; ++k) {
    float a, b;
    unpack2(vp[k], a, b);
    a = __uint_as_float(__float_as_uint(a) ^ ((signs << (31 - 2 * k)) & 0x80000000u));
    b = __uint_as_float(__float_as_uint(b) ^ ((signs << (30 - 2 * k)) & 0x80000000u));
    vp[k] = pack2(a, b);
  }
}

// The chunk of the row's code stream that this lane's group of four lanes covers.
__device__ __forceinline__ int wr_code_chunk(int lane) {
  return (lane >> 4) + 2 * ((lane >> 2) & 1) + 4 * ((lane >> 3) & 1);
}

// The lane's 32 fp32 prediction values in the load layout (pair 4c + i = elements 256c + 8 lane + 2i, +1).
// The loads are issued here and their values first used by wr_finish_row, so that the trip to L2
// overlaps the rotation in between (32 registers: only where the register budget allows it).
__device__ __forceinline__ void wr_load_pred_row(const float* __restrict__ pred_row, int lane, f32x2_t (&pr)[16]) {
#pragma unroll
  for (int ch = 0; ch < 4; ++ch) {
    f32x2_t p[4];
    wr_load_pred8(pred_row + ch * 256 + lane * 8, p);
#pragma unroll
    for (int i = 0; i < 4; ++i) pr[4 * ch + i] = p[i];
  }
}

// hat = round16(pred + c * sign * wp) for the lane's 32 values in the load layout; `wp` holds the
// rotated-back grid points, c = scale / sqrt(1024).  kEarly: the prediction was loaded into `pr`
// before the rotation; otherwise it is read here, chunk by chunk.
// kKeep stores the rows with the default policy instead of as streaming data (measured 2-4 % slower
// even when the attention warps of the same kernel read them back, so nothing selects it).
template <bool kBf16, bool kKeep = false, bool kEarly = false>
__device__ __forceinline__ void wr_finish_row(const WarpRowCtx& rc, f32x2_t (&wp)[16], float c,
                                              const float* __restrict__ pred_row, const f32x2_t (&pr)[16],
                                              uint16_t* __restrict__ hat_row) {
  const int lane = rc.lane;
  const f32x2_t c2 = pack2(c, c);
#pragma unroll
  for (int k = 0; k < 16; ++k) wp[k] = mul2(wp[k], c2);
  wr_apply_signs(wp, rc.signs);
#pragma unroll
  for (int ch = 0; ch < 4; ++ch) {
    if (pred_row != nullptr) {
      if constexpr (kEarly) {
#pragma unroll
        for (int i = 0; i < 4; ++i) wp[4 * ch + i] = add2(pr[4 * ch + i], wp[4 * ch + i]);
      } else {
        f32x2_t p[4];
        wr_load_pred8(pred_row + ch * 256 + lane * 8, p);
#pragma unroll
        for (int i = 0; i < 4; ++i) wp[4 * ch + i] = add2(p[i], wp[4 * ch + i]);
      }
    } else {
      // adding the zero prediction turns a -0 (a zero value whose sign was flipped) into +0
#pragma unroll
      for (int i = 0; i < 4; ++i) wp[4 * ch + i] = add2(pack2(0.0f, 0.0f), wp[4 * ch + i]);
    }
    const uint4 out = make_uint4(store16x2p<kBf16>(wp[4 * ch + 0]), store16x2p<kBf16>(wp[4 * ch + 1]),
                                 store16x2p<kBf16>(wp[4 * ch + 2]), store16x2p<kBf16>(wp[4 * ch + 3]));
    // otherwise a streaming store: the reconstruction is read at most once more before it leaves L2
    if constexpr (kKeep) *reinterpret_cast<uint4*>(hat_row + ch * 256 + lane * 8) = out;
    else __stcs(reinterpret_cast<uint4*>(hat_row + ch * 256 + lane * 8), out);
  }
}

// The lane's 32 input values of a row (16-bit, load layout) as loaded.
__device__ __forceinline__ void wr_load_x_row(const uint16_t* __restrict__ x_row, int lane, uint4 (&xraw)[4]) {
#pragma unroll
  for (int ch = 0; ch < 4; ++ch) xraw[ch] = __ldcs(reinterpret_cast<const uint4*>(x_row + ch * 256 + lane * 8));   // read once
}

// One token row of Q and of the reconstruction (Algorithm 2, keys or values):
//   codes, scale = Q(x - pred);  hat = round16(pred + Q^-1(codes, scale)).
// Row pointers address the start of the row.  pred_row == nullptr: no predictor.  hat_row == nullptr:
// reconstruction not wanted.  The prediction is read twice (for the residual and again for the
// reconstruction) instead of being held in 32 registers across the rotation and the search (a copy in
// the warp's shared memory measured 4 % slower than the second read: that pipe is the scarcer one); both
// reads bypass L1 because another SM of the same kernel may have written it just before.  The
// prediction rows must be 32-byte aligned.
// kAhead (for callers with registers to spare): `xraw` holds this row's input on entry and, if x_next
// is not null, the next row's on return (its loads are issued before the reconstruction so that they
// overlap it), and the second prediction read is issued before the rotation back.
template <int NPTS, bool kBf16, bool kAhead>
__device__ __forceinline__ void wr_encode_row_x(const WarpRowCtx& rc, const RowSmem<NPTS>* __restrict__ rsm,
                                                unsigned long long* xbuf, uint4 (&xraw)[4],
                                                const uint16_t* __restrict__ x_next,
                                                const float* __restrict__ pred_row,
                                                uint8_t* __restrict__ codes_row,
                                                uint16_t* __restrict__ scales_row,
                                                uint16_t* __restrict__ hat_row) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int NW = 2 * BITS;               // 32-bit words of a 64-code chunk
  const int lane = rc.lane;
  // ---- residual r = x - pred -------------------------------------------------------------------
  f32x2_t vp[16];
#pragma unroll
  for (int ch = 0; ch < 4; ++ch) {
    const uint4 raw = xraw[ch];
    vp[4 * ch + 0] = load16x2<kBf16>(raw.x);
    vp[4 * ch + 1] = load16x2<kBf16>(raw.y);
    vp[4 * ch + 2] = load16x2<kBf16>(raw.z);
    vp[4 * ch + 3] = load16x2<kBf16>(raw.w);
  }
  if (pred_row != nullptr) {
#pragma unroll
    for (int ch = 0; ch < 4; ++ch) {
      f32x2_t p[4];
      wr_load_pred8(pred_row + ch * 256 + lane * 8, p);
#pragma unroll
      for (int i = 0; i < 4; ++i) vp[4 * ch + i] = sub2(vp[4 * ch + i], p[i]);
    }
  }
  // ---- sum of squares of the row (four partial sums per lane, then the lanes) ---------------------
  float ss;
  {
    f32x2_t acc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) acc[u] = mul2(vp[u], vp[u]);
#pragma unroll
    for (int k = 4; k < 16; ++k) acc[k & 3] = fma2(vp[k], vp[k], acc[k & 3]);
    float lo, hi;
    unpack2(add2(add2(acc[0], acc[1]), add2(acc[2], acc[3])), lo, hi);
    ss = lo + hi;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
  }
  // ---- sign flip and rotation (the division by the scale comes afterwards: the rotation is linear) --
  wr_apply_signs(vp, rc.signs);
  wr_rotate_forward(vp, xbuf, lane);
  // ---- scale: root mean square, stored as fp16; normalise with the rounded value -------------------
  const float sc = fminf(sqrtf(ss * (1.0f / 1024.0f)), 65504.0f);
  const __half s16 = __float2half_rn(sc);
  const float sf = __half2float(s16);
  if (lane == 0) scales_row[0] = __half_as_ushort(s16);
  {
    const float inv = (sf > 0.0f ? __frcp_rn(sf) : 0.0f) * (1.0f / 32.0f);
    const f32x2_t inv2 = pack2(inv, inv);
#pragma unroll
    for (int k = 0; k < 16; ++k) vp[k] = mul2(vp[k], inv2);
  }
  // ---- nearest grid point per pair, four pairs at a time; code m goes to bit 4 * BITS * m of the
  //      lane's copy of the chunk, the pair itself is replaced by its grid point --------------------
  uint32_t W[NW];
#pragma unroll
  for (int w = 0; w < NW; ++w) W[w] = 0u;
#pragma unroll
  for (int g = 0; g < 4; ++g) {
    uint32_t entry[4];
    uint32_t emax = 0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      float y0, y1;
      unpack2(vp[4 * g + t], y0, y1);
      entry[t] = search_entry(y0, y1, rc.inv_w, rsm->table);
      emax = max(emax, entry[t]);
    }
    int idx[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) idx[t] = nearest_of_candidates<NPTS>(vp[4 * g + t], entry[t], rsm->grid);
    if (__any_sync(0xffffffffu, emax >= kCellSpecialDev)) {   // a pair in a cell with more candidates (rare for n <= 64)
#pragma unroll
      for (int t = 0; t < 4; ++t)
        if (entry[t] >= kCellSpecialDev) idx[t] = nearest_special<NPTS>(vp[4 * g + t], entry[t], rsm);
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      constexpr int kStep = 4 * BITS;
      const int pos = kStep * (4 * g + t);
      W[pos >> 5] |= uint32_t(idx[t]) << (pos & 31);
      vp[4 * g + t] = rsm->grid[idx[t]];
    }
  }
  // ---- pack: shift the lane's codes to their place inside each group of four, merge the four lanes
  //      of the chunk so that each ends up with a quarter of its words, store ---------------------------
  {
    const uint32_t sh = uint32_t(BITS * (lane & 3));
#pragma unroll
    for (int w = NW - 1; w > 0; --w) W[w] = __funnelshift_l(W[w - 1], W[w], sh);
    W[0] <<= sh;
    const bool b0 = (lane & 1) != 0, b1 = (lane & 2) != 0;
    uint32_t H[BITS];
#pragma unroll
    for (int i = 0; i < BITS; ++i) {
      const uint32_t send = b0 ? W[i] : W[i + BITS];
      const uint32_t keep = b0 ? W[i + BITS] : W[i];
      H[i] = keep | __shfl_xor_sync(0xffffffffu, send, 1);
    }
    uint32_t F[BITS / 2];
#pragma unroll
    for (int i = 0; i < BITS / 2; ++i) {
      const uint32_t send = b1 ? H[i] : H[i + BITS / 2];
      const uint32_t keep = b1 ? H[i + BITS / 2] : H[i];
      F[i] = keep | __shfl_xor_sync(0xffffffffu, send, 2);
    }
    uint32_t* dst = reinterpret_cast<uint32_t*>(codes_row + wr_code_chunk(lane) * (8 * BITS)) +
                    (b0 ? BITS : 0) + (b1 ? BITS / 2 : 0);
    if constexpr (BITS == 4) {
      *reinterpret_cast<uint2*>(dst) = make_uint2(F[0], F[1]);
    } else if constexpr (BITS == 8) {
      *reinterpret_cast<uint4*>(dst) = make_uint4(F[0], F[1], F[2], F[3]);
    } else {
#pragma unroll
      for (int i = 0; i < BITS / 2; ++i) dst[i] = F[i];
    }
  }
  // ---- reconstruction: hat = round16(pred + Q^-1(codes)) ---------------------------------------
  if constexpr (kAhead) {
    if (x_next != nullptr) wr_load_x_row(x_next, lane, xraw);
  }
  if (hat_row != nullptr) {      // uniform over the warp
    f32x2_t pr[16];
    if constexpr (kAhead) {
      if (pred_row != nullptr) wr_load_pred_row(pred_row, lane, pr);
    }
    wr_rotate_back(vp, xbuf, lane);
    wr_finish_row<kBf16, false, kAhead>(rc, vp, sf * (1.0f / 32.0f), pred_row, pr, hat_row);
  }
}

template <int NPTS, bool kBf16>
__device__ __forceinline__ void wr_encode_row(const WarpRowCtx& rc, const RowSmem<NPTS>* __restrict__ rsm,
                                              unsigned long long* xbuf, const uint16_t* __restrict__ x_row,
                                              const float* __restrict__ pred_row,
                                              uint8_t* __restrict__ codes_row,
                                              uint16_t* __restrict__ scales_row,
                                              uint16_t* __restrict__ hat_row) {
  uint4 xraw[4];
  wr_load_x_row(x_row, rc.lane, xraw);
  wr_encode_row_x<NPTS, kBf16, false>(rc, rsm, xbuf, xraw, nullptr, pred_row, codes_row, scales_row, hat_row);
}

// One token row of Algorithm 3 (keys or values) given the prediction:
//   hat = round16(pred + Q^-1(codes, scale)).
template <int NPTS, bool kBf16, bool kKeep = false, bool kEarly = false>
__device__ __forceinline__ void wr_decode_row(const WarpRowCtx& rc, const f32x2_t* __restrict__ grid_s,
                                              unsigned long long* xbuf,
                                              const uint8_t* __restrict__ codes_row,
                                              const uint16_t* __restrict__ scales_row,
                                              const float* __restrict__ pred_row,
                                              uint16_t* __restrict__ hat_row) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int NW = 2 * BITS;
  const int lane = rc.lane;
  f32x2_t pr[16];
  if constexpr (kEarly) {
    if (pred_row != nullptr) wr_load_pred_row(pred_row, lane, pr);   // in flight during the look-ups and the rotation
  }
  // the chunk of 64 codes this lane's group of four covers (each of the four lanes reads all of it)
  uint32_t W[NW];
  {
    const uint4* src = reinterpret_cast<const uint4*>(codes_row + wr_code_chunk(lane) * (8 * BITS));
#pragma unroll
    for (int i = 0; i < NW / 4; ++i) {
      const uint4 t = __ldcs(src + i);
      W[4 * i + 0] = t.x;
      W[4 * i + 1] = t.y;
      W[4 * i + 2] = t.z;
      W[4 * i + 3] = t.w;
    }
  }
  const float sf = __half2float(__ushort_as_half(scales_row[0]));
  const uint32_t sh = uint32_t(BITS * (lane & 3));
#pragma unroll
  for (int w = 0; w < NW - 1; ++w) W[w] = __funnelshift_r(W[w], W[w + 1], sh);
  W[NW - 1] >>= sh;
  f32x2_t wp[16];
#pragma unroll
  for (int m = 0; m < 16; ++m) {
    constexpr int kStep = 4 * BITS;
    const int pos = kStep * m;
    wp[m] = grid_s[(W[pos >> 5] >> (pos & 31)) & uint32_t(NPTS - 1)];
  }
  wr_rotate_back(wp, xbuf, lane);
  wr_finish_row<kBf16, kKeep, kEarly>(rc, wp, sf * (1.0f / 32.0f), pred_row, pr, hat_row);
}

// ---------------------------------------------------------------------------------------------
// Stand-alone row kernels for this setting (layer 0 and the single-phase entry points): four row
// warps per CTA, several CTAs per SM.
// ---------------------------------------------------------------------------------------------
constexpr int kWrKernelWarps = 4;

__device__ __forceinline__ WarpRowCtx wr_make_ctx(const uint32_t* signmask, float inv_w) {
  WarpRowCtx rc;
  rc.lane = threadIdx.x & 31;
  rc.signs = signmask[rc.lane];
  rc.inv_w = inv_w;
  return rc;
}

template <int NPTS, bool kBf16>
__global__ void __launch_bounds__(kWrKernelWarps * 32, 4) encode_rows_warp_kernel(const CodecArgs a) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = 1024 / 2 * BITS / 8;
  __shared__ RowSmem<NPTS> tables;
  __shared__ __align__(16) unsigned long long xbuf[kWrKernelWarps][kWrItems];
  row_smem_fill<NPTS>(&tables, a.search.table, a.grid4);
  __syncthreads();
  const WarpRowCtx rc = wr_make_ctx(a.signmask, a.search.inv_w);
  const int warp = threadIdx.x >> 5;
  for (long long row = (long long)blockIdx.x * kWrKernelWarps + warp; row < a.T;
       row += (long long)gridDim.x * kWrKernelWarps) {
    wr_encode_row<NPTS, kBf16>(rc, &tables, xbuf[warp], a.X + row * a.ldX,
                               a.P != nullptr ? a.P + row * a.ldP : nullptr, a.codes + row * CODE_BYTES,
                               a.scales + row, a.hat != nullptr ? a.hat + row * a.ldHat : nullptr);
  }
}

template <int NPTS, bool kBf16>
__global__ void __launch_bounds__(kWrKernelWarps * 32, 4) decode_rows_warp_kernel(const CodecArgs a) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = 1024 / 2 * BITS / 8;
  __shared__ f32x2_t grid_s[NPTS];
  __shared__ __align__(16) unsigned long long xbuf[kWrKernelWarps][kWrItems];
  for (int i = threadIdx.x; i < NPTS; i += blockDim.x) {
    const float4 g = a.grid4[i];
    grid_s[i] = pack2(g.x, g.y);
  }
  __syncthreads();
  const WarpRowCtx rc = wr_make_ctx(a.signmask, a.search.inv_w);
  const int warp = threadIdx.x >> 5;
  for (long long row = (long long)blockIdx.x * kWrKernelWarps + warp; row < a.T;
       row += (long long)gridDim.x * kWrKernelWarps) {
    wr_decode_row<NPTS, kBf16>(rc, grid_s, xbuf[warp], a.codes + row * CODE_BYTES, a.scales + row,
                               a.P != nullptr ? a.P + row * a.ldP : nullptr, a.hat + row * a.ldHat);
  }
}

}  // namespace aquakv
