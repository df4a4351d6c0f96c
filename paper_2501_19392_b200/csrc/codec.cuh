// Row kernels of the backbone quantizer Q / Q^-1 (Section 2 "Vector Quantization", Section 4.1
// "Alternative quantizers": group scale, randomized Hadamard transform, nearest point of a fixed
// 2-D grid, packed codes) and of the residual / add-back steps of Algorithm 2 and
// Algorithm 3.
//
// A team of d_kv/256 warps (1, 2 or 4) owns one token row; each warp holds one 256-element chunk.
// Element e of the row lives in warp e/256, lane (e/8)%32, register e%8, so every global access is
// a 16-byte (16-bit data) or 2x16-byte (fp32) vector per lane and a warp touches whole 128-byte
// lines.  The Hadamard butterflies over index bits 0-2 are register-local, bits 3-7 are warp
// shuffles, bits 8-9 cross the warps of the team through shared memory.  The row code is a long
// chain of dependent shuffles and shared-memory gathers whose throughput grows with the number of
// resident warps; eight values per lane keep it near 64 registers per thread, which lets 24 row
// warps sit beside the GEMM warps of the fused kernel.  The value pair (2j, 2j+1) that shares one
// code always sits in one lane.
#pragma once

#include "common.cuh"

namespace aquakv {

// Packed pairs of fp32 values: sm_100 executes add/sub/fma on two fp32 lanes of a 64-bit register
// pair in one instruction (add.f32x2 / fma.rn.f32x2), each lane rounded exactly like the scalar
// operation.  The rotation keeps (v[2k], v[2k+1]) packed, which halves its arithmetic instructions.
typedef unsigned long long f32x2_t;
__device__ __forceinline__ f32x2_t pack2(float lo, float hi) {
  f32x2_t r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f32x2_t p, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(p));
}
__device__ __forceinline__ f32x2_t add2(f32x2_t a, f32x2_t b) {
  f32x2_t r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2_t sub2(f32x2_t a, f32x2_t b) {
  f32x2_t r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ f32x2_t fma2(f32x2_t a, f32x2_t b, f32x2_t c) {
  f32x2_t r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}
__device__ __forceinline__ f32x2_t mul2(f32x2_t a, f32x2_t b) {
  f32x2_t r;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}

constexpr int kCodecWarps = 8;
constexpr int kCodecThreads = kCodecWarps * 32;

// Nearest-point search.  dist_i(y) = (y0 - g_i.x)^2 + (y1 - g_i.y)^2; the lowest index wins ties.
// A cell table built on the host (search_table.h) lists, for the cell that holds y, every point
// that can win there, so only three (n = 16) or four distances are evaluated; cells with more candidates and
// values outside the table's square fall back to the exhaustive loop.  Both paths evaluate the same
// fp32 expression, so the result is the exhaustive arg-min bit for bit.  The table (64 x 64
// entries) and the grid live in shared memory: the row kernels are bound by the load/store and
// shuffle pipe, and shared-memory gathers of 4 and 8 bytes cost far fewer cycles there than
// global gathers or 16-byte records.
constexpr int kSearchCells = 64;          // cells per side of the table (see search_table.h)
constexpr int kSearchLogCells = 6;
constexpr uint32_t kCellBruteDev = 0xFFFFFFFFu;   // "search all points" (the largest entry value)
constexpr uint32_t kCellSpecialDev = 0xFF000000u; // entries from here up: second-level list (low 24 bits) or kCellBruteDev

struct SearchDev {
  const uint32_t* table;   // global copy [64*64] of the candidate lists, then the second-level lists (two words each)
  float inv_w;             // cells / (2 * half extent)
};

// Shared-memory tables of the row routines.
template <int NPTS>
struct RowSmem {
  uint32_t table[kSearchCells * kSearchCells];
  f32x2_t grid[NPTS];      // (g.x, g.y) as packed fp32 pairs
  const uint2* lists;      // second-level candidate lists (global memory: only the rare path reads them)
};

template <int NPTS>
__device__ __forceinline__ void row_smem_fill(RowSmem<NPTS>* rs, const uint32_t* table, const float4* grid4) {
  for (int i = threadIdx.x; i < kSearchCells * kSearchCells; i += blockDim.x) rs->table[i] = table[i];
  if (threadIdx.x == 0) rs->lists = reinterpret_cast<const uint2*>(table + kSearchCells * kSearchCells);
  for (int i = threadIdx.x; i < NPTS; i += blockDim.x) {
    const float4 g = grid4[i];
    rs->grid[i] = pack2(g.x, g.y);
  }
}

struct CodecArgs {
  const uint16_t* X;        // encode: target rows (16-bit)              [T, ldX]
  long long ldX;
  const float* P;           // prediction rows (fp32) or nullptr          [T, ldP]
  long long ldP;
  const uint32_t* signmask; // [32]: bit (c*8+i) of entry `lane` set <=> sign of element
                            //       c*256 + lane*8 + i is -1
  const float4* grid4;      // [n]: (g_x, g_y, 0, 0)
  SearchDev search;
  uint8_t* codes;           // [T, code_bytes]
  uint16_t* scales;         // [T, D/G] fp16 bits
  uint16_t* hat;            // reconstruction rows (16-bit) or nullptr    [T, ldHat]
  long long ldHat;
  int T;
  int log_h;                // log2 of the Hadamard block
  int log_g;                // log2 of the scale group
};

// Hadamard butterflies of one warp's NV values per lane (element index bits 0-2 in registers,
// 3-7 across lanes, the next bit between the warp's two chunks when NV == 16), by ascending bit.
// vp[k] holds (v[2k], v[2k+1]).
template <int NV>
__device__ __forceinline__ void fwht_packed(f32x2_t (&vp)[NV / 2], int log_h, int lane) {
  // bit 0: inside each packed pair
#pragma unroll
  for (int k = 0; k < NV / 2; ++k) {
    float a, b;
    unpack2(vp[k], a, b);
    vp[k] = pack2(a + b, a - b);
  }
  // bits 1, 2: between packed pairs k and k ^ 1, k ^ 2
#pragma unroll
  for (int b = 1; b < 3; ++b) {
    const int m = 1 << (b - 1);
#pragma unroll
    for (int k = 0; k < NV / 2; ++k) {
      if ((k & m) == 0) {
        const f32x2_t x = vp[k], y = vp[k | m];
        vp[k] = add2(x, y);
        vp[k | m] = sub2(x, y);
      }
    }
  }
  // bits 3..7: lane bits 0..4
#pragma unroll
  for (int b = 3; b < 8; ++b) {
    if (b < log_h) {
      const int m = 1 << (b - 3);
      const float sg = (lane & m) ? -1.0f : 1.0f;
      const f32x2_t sg2 = pack2(sg, sg);
#pragma unroll
      for (int k = 0; k < NV / 2; ++k) {
        float a, c;
        unpack2(vp[k], a, c);
        const float oa = __shfl_xor_sync(0xffffffffu, a, m);
        const float oc = __shfl_xor_sync(0xffffffffu, c, m);
        vp[k] = fma2(sg2, vp[k], pack2(oa, oc));   // lower partner: v + o; upper partner: o - v
      }
    }
  }
  // bit 8: between the two chunks of a 16-value warp
  if constexpr (NV == 16) {
    if (8 < log_h) {
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const f32x2_t x = vp[k], y = vp[k + 4];
        vp[k] = add2(x, y);
        vp[k + 4] = sub2(x, y);
      }
    }
  }
}

__device__ __forceinline__ float apply_sign(float x, uint32_t mask, int i) {
  // flips the sign bit of x when bit i of mask is set
  return __uint_as_float(__float_as_uint(x) ^ ((mask << (31 - i)) & 0x80000000u));
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

// Cell-table entry of one value pair.  The cell coordinates saturate at the table's border cells,
// which the host marks "search all points", so values outside the square need no separate test.
__device__ __forceinline__ uint32_t search_entry(float y0, float y1, float inv_w,
                                                 const uint32_t* __restrict__ table_s) {
  const unsigned ix = min(__float2uint_rd(fmaf(y0, inv_w, 0.5f * kSearchCells)), unsigned(kSearchCells - 1));
  const unsigned iy = min(__float2uint_rd(fmaf(y1, inv_w, 0.5f * kSearchCells)), unsigned(kSearchCells - 1));
  return table_s[(iy << kSearchLogCells) + ix];
}

// Squared distance of the packed pair y to the grid point g (both as packed fp32 pairs).
__device__ __forceinline__ float pair_dist(f32x2_t y, f32x2_t g) {
  const f32x2_t d = sub2(y, g);
  float qx, qy;
  unpack2(mul2(d, d), qx, qy);
  return __fadd_rn(qx, qy);
}

// Arg-min over the ascending candidates of a table entry (bytes 3, 2, 1 and, for n > 16, 0).  Indices
// are masked to the grid so that special entries, whose result is replaced afterwards, stay in range.
template <int NPTS>
__device__ __forceinline__ int nearest_of_candidates(f32x2_t y, uint32_t e, const f32x2_t* __restrict__ grid_s) {
  const int c0 = (e >> 24) & (NPTS - 1), c1 = (e >> 16) & (NPTS - 1), c2 = (e >> 8) & (NPTS - 1);
  const float t0 = pair_dist(y, grid_s[c0]);
  const float t1 = pair_dist(y, grid_s[c1]);
  const float t2 = pair_dist(y, grid_s[c2]);
  int idx = c0;
  float best = t0;
  if (t1 < best) { best = t1; idx = c1; }
  if (t2 < best) { best = t2; idx = c2; }
  if constexpr (NPTS > 16) {
    const int c3 = e & (NPTS - 1);
    const float t3 = pair_dist(y, grid_s[c3]);
    if (t3 < best) { idx = c3; }
  }
  return idx;
}

// The pair's nearest point for a special table entry: arg-min over all points or, for the large grid
// (the host builds second-level lists only for n > 64: smaller grids practically never need them),
// over the entry's list of eight ascending candidates (repeats at the end change nothing).  One
// rolled loop, so that this rarely taken path adds little code and no registers to the row loop.
template <int NPTS>
__device__ __forceinline__ int nearest_special(f32x2_t y, uint32_t e, const RowSmem<NPTS>* rsm) {
  float best = 3.0e38f;
  int idx = 0;
  if constexpr (NPTS > 64) {
    const bool all = e == kCellBruteDev;
    uint2 lst = make_uint2(0u, 0u);
    if (!all) lst = __ldg(rsm->lists + (e & 0x00FFFFFFu));
    const int count = all ? NPTS : 8;
#pragma unroll 1
    for (int i = 0; i < count; ++i) {
      const int c = all ? i : int((((i & 4) ? lst.y : lst.x) >> (8 * (i & 3))) & (NPTS - 1));
      const float t = pair_dist(y, rsm->grid[c]);
      if (t < best) { best = t; idx = c; }             // strict: lowest index wins ties
    }
  } else {
#pragma unroll 1
    for (int i = 0; i < NPTS; ++i) {
      const float t = pair_dist(y, rsm->grid[i]);
      if (t < best) { best = t; idx = i; }
    }
  }
  return idx;
}

// Geometry of a row team: one warp per 256-element chunk of the row.
template <int D>
struct RowTeam {
  static constexpr int NC = D / 256;                 // 256-element chunks per row
  static constexpr int TEAM = NC;                    // warps per row (1, 2 or 4)
  static constexpr int LOG_TEAM = NC == 4 ? 2 : (NC == 2 ? 1 : 0);
  static constexpr int CPM = 1;                      // chunks per warp
  static constexpr int NV = 8;                       // values per lane
};

// Exchange buffers of one team (only used when TEAM > 1).  Two copies used alternately: a warp
// writes copy n % 2 in its n-th exchange after passing the barrier of exchange n - 1, which every
// warp reaches only after it has read copy n % 2 in exchange n - 2, so one barrier per exchange
// is enough.
template <int D>
struct TeamSmem {
  ulonglong2 x[2][RowTeam<D>::TEAM][RowTeam<D>::NV / 4][32];   // [copy][member][16-byte piece][lane]
  float ss[2][RowTeam<D>::TEAM];                               // [copy][member] sum of squares of its chunk
};

// Per-warp constants of the row routines.
struct RowCtx {
  f32x2_t sgn2[4];         // this lane's Hadamard signs as packed (+-1, +-1) multipliers, pair k = values 2k, 2k+1
  float inv_w;             // SearchDev::inv_w
  float inv_g;             // 1 / scale group
  float rs;                // 1 / sqrt(Hadamard block)
  int log_h, log_g;
  int lane;
  int member;              // which chunk of the row this warp holds
  int barrier;             // named barrier shared by the warps of the team
  mutable int xcopy;       // exchange-buffer copy the next exchange uses (same in all warps of a team)
};

// bits: bit i set <=> value i of this lane is multiplied by -1.
__device__ __forceinline__ void row_ctx_set_signs(RowCtx& rc, uint32_t bits) {
#pragma unroll
  for (int k = 0; k < 4; ++k)
    rc.sgn2[k] = pack2((bits >> (2 * k)) & 1u ? -1.0f : 1.0f, (bits >> (2 * k + 1)) & 1u ? -1.0f : 1.0f);
}

// Fills the fields that depend only on the parameters and on the warp's place in its team.
__device__ __forceinline__ void row_ctx_init(RowCtx& rc, const uint32_t* signmask, float inv_w, int log_h,
                                             int log_g, int lane, int member, int values_per_warp,
                                             int barrier) {
  rc.lane = lane;
  rc.member = member;
  rc.barrier = barrier;
  rc.xcopy = 0;
  row_ctx_set_signs(rc, signmask[lane] >> (member * values_per_warp));
  rc.inv_w = inv_w;
  rc.log_h = log_h;
  rc.log_g = log_g;
  rc.inv_g = __int_as_float((127 - log_g) << 23);                       // 2^-log_g, exact
  rc.rs = __int_as_float((127 - (log_h >> 1)) << 23) * ((log_h & 1) ? 0.70710678118654752f : 1.0f);
}

template <int D>
__device__ __forceinline__ void team_barrier(int id) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(RowTeam<D>::TEAM * 32) : "memory");
}

// Publishes this warp's values (and optionally its sum of squares) and reads those of `partner`.
// Returns the buffer copy that was used (the sums of all members can be read from it).
template <int D, bool kWithSum>
__device__ __forceinline__ int team_exchange(const RowCtx& rc, TeamSmem<D>* ts, int partner,
                                             const f32x2_t (&vp)[RowTeam<D>::NV / 2],
                                             f32x2_t (&op)[RowTeam<D>::NV / 2], float ss) {
  constexpr int NV = RowTeam<D>::NV;
  const int cp = rc.xcopy;
  rc.xcopy ^= 1;
#pragma unroll
  for (int q = 0; q < NV / 4; ++q)
    ts->x[cp][rc.member][q][rc.lane] = make_ulonglong2(vp[2 * q], vp[2 * q + 1]);
  if (kWithSum && rc.lane == 0) ts->ss[cp][rc.member] = ss;
  team_barrier<D>(rc.barrier);
#pragma unroll
  for (int q = 0; q < NV / 4; ++q) {
    const ulonglong2 t = ts->x[cp][partner][q][rc.lane];
    op[2 * q] = t.x;
    op[2 * q + 1] = t.y;
  }
  return cp;
}

// Publishes only the sums of squares (scale groups that span warps while Hadamard blocks do not).
template <int D>
__device__ __forceinline__ int team_exchange_sums(const RowCtx& rc, TeamSmem<D>* ts, float ss) {
  const int cp = rc.xcopy;
  rc.xcopy ^= 1;
  if (rc.lane == 0) ts->ss[cp][rc.member] = ss;
  team_barrier<D>(rc.barrier);
  return cp;
}

// Butterfly over an index bit that separates warps: the lower warp keeps a + b, the upper one a - b
// (a = lower warp's value, b = upper warp's).
template <int NP>
__device__ __forceinline__ void cross_butterfly(f32x2_t (&vp)[NP], const f32x2_t (&op)[NP], bool upper) {
  const float sg = upper ? -1.0f : 1.0f;
  const f32x2_t sg2 = pack2(sg, sg);
#pragma unroll
  for (int k = 0; k < NP; ++k) vp[k] = fma2(sg2, vp[k], op[k]);
}

// The Hadamard stages over the index bits that separate the warps of a team (bits 8, 9), ascending.
// kWithSum: the first exchange also publishes this warp's sum of squares; returns the buffer copy
// holding the sums, or -1 if no exchange published them.
template <int D, bool kWithSum>
__device__ __forceinline__ int team_cross_stages(const RowCtx& rc, TeamSmem<D>* ts,
                                                 f32x2_t (&vp)[RowTeam<D>::NV / 2], float ss) {
  using RT = RowTeam<D>;
  int sums_copy = -1;
#pragma unroll
  for (int k = 0; k < RT::LOG_TEAM; ++k) {
    if (8 + k < rc.log_h) {
      f32x2_t op[RT::NV / 2];
      if (kWithSum && k == 0) {
        sums_copy = team_exchange<D, true>(rc, ts, rc.member ^ (1 << k), vp, op, ss);
      } else {
        team_exchange<D, false>(rc, ts, rc.member ^ (1 << k), vp, op, 0.0f);
      }
      cross_butterfly<RT::NV / 2>(vp, op, (rc.member >> k) & 1);
    }
  }
  return sums_copy;
}

// Q^-1 without the prediction for this warp's chunk of the row: `wp` enters holding the gathered grid
// points (packed pairs) and leaves holding xhat.  The operation order (rotation stages by ascending
// index bit, multiply by 1/sqrt(h), then by the signed scale) is shared by encode and decode so that
// both produce bit-identical reconstructions.
template <int D>
__device__ __forceinline__ void team_rotate_back_and_scale(const RowCtx& rc, TeamSmem<D>* ts,
                                                           f32x2_t (&wp)[4], float scale) {
  fwht_packed<8>(wp, rc.log_h, rc.lane);
  team_cross_stages<D, false>(rc, ts, wp, 0.0f);
  const f32x2_t rs2 = pack2(rc.rs, rc.rs), s2 = pack2(scale, scale);
#pragma unroll
  for (int k = 0; k < 4; ++k) wp[k] = mul2(mul2(wp[k], rs2), mul2(s2, rc.sgn2[k]));
}

// (lo, hi) 16-bit values of a 32-bit word as a packed fp32 pair.
template <bool kBf16>
__device__ __forceinline__ f32x2_t load16x2(uint32_t w) {
  if constexpr (kBf16) {
    return pack2(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
  } else {
    const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w));
    return pack2(f.x, f.y);
  }
}
template <bool kBf16>
__device__ __forceinline__ uint32_t store16x2p(f32x2_t v) {
  float lo, hi;
  unpack2(v, lo, hi);
  return store16x2<kBf16>(lo, hi);
}

// This warp's part of one token row of Q and of the reconstruction (Algorithm 2, keys or values):
//   codes, scales = Q(x - pred);  hat = round16(pred + Q^-1(codes, scales)).
// All row pointers address the start of the row.  pred_row == nullptr: no predictor.
// hat_row == nullptr: reconstruction not wanted.  The prediction is read twice (for the residual and
// again for the reconstruction) instead of being held in registers across the rotation and the
// search; both reads bypass L1 (ld.global.cg) because the prediction may have been written by
// another SM of the same kernel just before.  Both warps of a team must call this together.
template <int D, int NPTS, bool kBf16, typename AfterLoad>
__device__ __forceinline__ void encode_row_core(const RowCtx& rc, const RowSmem<NPTS>* __restrict__ rsm,
                                                TeamSmem<D>* ts, const uint4 (&raw)[1],
                                                const float4 (&pq0)[1][2],
                                                const float* __restrict__ pred_row,
                                                uint8_t* __restrict__ codes_row,
                                                uint16_t* __restrict__ scales_row,
                                                uint16_t* __restrict__ hat_row, AfterLoad after_load) {
  using RT = RowTeam<D>;
  constexpr int NC = RT::NC;
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  const int lane = rc.lane;
  const int cg = rc.member;                          // this warp's chunk
  // ---- residual r = x - pred (raw = this lane's 16-bit inputs, pq0 = its prediction values) -----
  f32x2_t vp[4];
  {
    const uint32_t w[4] = {raw[0].x, raw[0].y, raw[0].z, raw[0].w};
#pragma unroll
    for (int k = 0; k < 4; ++k) vp[k] = load16x2<kBf16>(w[k]);
    if (pred_row != nullptr) {
      vp[0] = sub2(vp[0], pack2(pq0[0][0].x, pq0[0][0].y));
      vp[1] = sub2(vp[1], pack2(pq0[0][0].z, pq0[0][0].w));
      vp[2] = sub2(vp[2], pack2(pq0[0][1].x, pq0[0][1].y));
      vp[3] = sub2(vp[3], pack2(pq0[0][1].z, pq0[0][1].w));
    }
  }
  after_load();   // raw and pq0 are consumed: the caller may start fetching the next row's inputs
  // ---- sum of squares of the chunk (lane bits reduced by shuffles), sign flip --------------------
  float ss;
  {
    f32x2_t acc = mul2(vp[0], vp[0]);
#pragma unroll
    for (int k = 1; k < 4; ++k) acc = fma2(vp[k], vp[k], acc);
    float lo, hi;
    unpack2(acc, lo, hi);
    ss = lo + hi;
#pragma unroll
    for (int b = 3; b < 8; ++b)
      if (b < rc.log_g) ss += __shfl_xor_sync(0xffffffffu, ss, 1 << (b - 3));
#pragma unroll
    for (int k = 0; k < 4; ++k) vp[k] = mul2(vp[k], rc.sgn2[k]);
  }
  // ---- rotate (the division by the scale is applied afterwards: the rotation is linear) ---------
  fwht_packed<8>(vp, rc.log_h, lane);
  int sums_copy = 0;
  {
    // stages across warps; the sums of squares travel with the first exchange when groups span warps
    const bool need_sums = RT::TEAM > 1 && rc.log_g > 8;
    if (need_sums) {
      sums_copy = team_cross_stages<D, true>(rc, ts, vp, ss);
      if (sums_copy < 0) sums_copy = team_exchange_sums<D>(rc, ts, ss);
    } else {
      team_cross_stages<D, false>(rc, ts, vp, 0.0f);
    }
  }
  // ---- group scale: root mean square, stored as fp16; normalise with the rounded value ----------
  float sf;
  {
    float tot = ss;
    if (RT::TEAM > 1 && rc.log_g > 8) {      // groups of several chunks: add them in ascending order
      const int cpg = 1 << (rc.log_g - 8);
      tot = 0.0f;
#pragma unroll
      for (int c2 = 0; c2 < NC; ++c2)
        if ((c2 / cpg) == (cg / cpg)) tot += ts->ss[sums_copy][c2];
    }
    const float sc = fminf(sqrtf(tot * rc.inv_g), 65504.0f);
    const __half s16 = __float2half_rn(sc);
    sf = __half2float(s16);
    if (rc.log_g >= 8) {                     // one lane per group writes the scale
      const int cpg = 1 << (rc.log_g - 8);
      if (lane == 0 && (cg % cpg) == 0) scales_row[cg / cpg] = __half_as_ushort(s16);
    } else {
      const int lpg = 1 << (rc.log_g - 3);   // lanes per group
      if ((lane % lpg) == 0) scales_row[cg * (256 >> rc.log_g) + lane / lpg] = __half_as_ushort(s16);
    }
    const float inv = (sf > 0.0f ? __frcp_rn(sf) : 0.0f) * rc.rs;
    const f32x2_t inv2 = pack2(inv, inv);
#pragma unroll
    for (int k = 0; k < 4; ++k) vp[k] = mul2(vp[k], inv2);
  }
  // the prediction is needed again for the reconstruction: start reading it now, the search hides it
  float4 pq[2];
  if (hat_row != nullptr && pred_row != nullptr) {
    pq[0] = __ldcg(reinterpret_cast<const float4*>(pred_row + cg * 256 + lane * 8));
    pq[1] = __ldcg(reinterpret_cast<const float4*>(pred_row + cg * 256 + lane * 8 + 4));
  } else {
    pq[0] = pq[1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  }
  // ---- nearest grid point per pair: all table entries first, then the candidates ----------------
  uint32_t entry[4];
  uint32_t emax = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    float y0, y1;
    unpack2(vp[k], y0, y1);
    entry[k] = search_entry(y0, y1, rc.inv_w, rsm->table);
    emax = max(emax, entry[k]);
  }
  const bool slow = __any_sync(0xffffffffu, emax >= kCellSpecialDev);
  int idx[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) idx[k] = nearest_of_candidates<NPTS>(vp[k], entry[k], rsm->grid);
  if (slow) {     // some lane of the warp has a pair in a cell with more candidates (rare for n <= 64)
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (entry[k] >= kCellSpecialDev) idx[k] = nearest_special<NPTS>(vp[k], entry[k], rsm);
  }
  uint32_t word = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    word |= uint32_t(idx[k]) << (k * BITS);
    vp[k] = rsm->grid[idx[k]];
  }
  store_code_word<BITS>(codes_row, cg, lane, word);
  // ---- reconstruction: hat = round16(pred + Q^-1(codes)) ---------------------------------------
  if (hat_row != nullptr) {      // uniform over the team
    team_rotate_back_and_scale<D>(rc, ts, vp, sf);
    uint32_t o[4];
    o[0] = store16x2p<kBf16>(add2(pack2(pq[0].x, pq[0].y), vp[0]));
    o[1] = store16x2p<kBf16>(add2(pack2(pq[0].z, pq[0].w), vp[1]));
    o[2] = store16x2p<kBf16>(add2(pack2(pq[1].x, pq[1].y), vp[2]));
    o[3] = store16x2p<kBf16>(add2(pack2(pq[1].z, pq[1].w), vp[3]));
    // streaming store: the reconstruction is read at most once more (by the value-phase GEMM) before it
    // leaves L2
    __stcs(reinterpret_cast<uint4*>(hat_row + cg * 256 + lane * 8), make_uint4(o[0], o[1], o[2], o[3]));
  }
}

// encode_row_core with the row's inputs read straight from global memory.
template <int D, int NPTS, bool kBf16>
__device__ __forceinline__ void encode_row(const RowCtx& rc, const RowSmem<NPTS>* __restrict__ rsm,
                                           TeamSmem<D>* ts, const uint16_t* __restrict__ x_row,
                                           const float* __restrict__ pred_row,
                                           uint8_t* __restrict__ codes_row,
                                           uint16_t* __restrict__ scales_row,
                                           uint16_t* __restrict__ hat_row) {
  constexpr int CPM = RowTeam<D>::CPM;
  const int c0 = rc.member * CPM;
  uint4 raw[CPM];
  float4 pq[CPM][2];
#pragma unroll
  for (int c = 0; c < CPM; ++c) {
    raw[c] = __ldcs(reinterpret_cast<const uint4*>(x_row + (c0 + c) * 256 + rc.lane * 8));   // read once
    if (pred_row != nullptr) {
      pq[c][0] = __ldcg(reinterpret_cast<const float4*>(pred_row + (c0 + c) * 256 + rc.lane * 8));
      pq[c][1] = __ldcg(reinterpret_cast<const float4*>(pred_row + (c0 + c) * 256 + rc.lane * 8 + 4));
    } else {
      pq[c][0] = pq[c][1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }
  }
  encode_row_core<D, NPTS, kBf16>(rc, rsm, ts, raw, pq, pred_row, codes_row, scales_row, hat_row, [] {});
}

// Shared memory of the stand-alone row kernels: search tables plus one exchange buffer per team.
template <int D, int NPTS>
struct RowKernelSmem {
  RowSmem<NPTS> tables;
  TeamSmem<D> team[kCodecWarps / RowTeam<D>::TEAM];
};

__device__ __forceinline__ RowCtx make_row_ctx(const CodecArgs& a, int team_size, int values_per_warp,
                                               int first_barrier) {
  RowCtx rc;
  const int warp = threadIdx.x >> 5;
  row_ctx_init(rc, a.signmask, a.search.inv_w, a.log_h, a.log_g, threadIdx.x & 31, warp % team_size,
               values_per_warp, first_barrier + warp / team_size);
  return rc;
}

template <int D, int NPTS, bool kBf16>
__global__ void __launch_bounds__(kCodecThreads, 4) encode_rows_kernel(const CodecArgs a) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = D / 2 * BITS / 8;
  constexpr int TEAM = RowTeam<D>::TEAM, TEAMS = kCodecWarps / TEAM;
  __shared__ RowKernelSmem<D, NPTS> sm;
  row_smem_fill<NPTS>(&sm.tables, a.search.table, a.grid4);
  __syncthreads();
  const RowCtx rc = make_row_ctx(a, TEAM, RowTeam<D>::NV, 1);
  const int team = (threadIdx.x >> 5) / TEAM;
  const int n_groups = D >> a.log_g;
  for (long long row = (long long)blockIdx.x * TEAMS + team; row < a.T; row += (long long)gridDim.x * TEAMS) {
    encode_row<D, NPTS, kBf16>(rc, &sm.tables, &sm.team[team], a.X + row * a.ldX,
                               a.P != nullptr ? a.P + row * a.ldP : nullptr,
                               a.codes + row * CODE_BYTES, a.scales + row * n_groups,
                               a.hat != nullptr ? a.hat + row * a.ldHat : nullptr);
  }
}

// This warp's part of one token row of Algorithm 3 (keys or values) given the prediction:
//   hat = round16(pred + Q^-1(codes, scales)).  words = this lane's packed codes per chunk, sf = the
// scale of each chunk; get_pred(pq) delivers the prediction values of this lane just before they are
// added, so a caller can fetch them while the rotation runs.
template <int D, int NPTS, bool kBf16, typename GetPred>
__device__ __forceinline__ void decode_row_core(const RowCtx& rc, const f32x2_t* __restrict__ grid_s,
                                                TeamSmem<D>* ts, const uint32_t (&words)[1],
                                                const float (&sf)[1], GetPred get_pred,
                                                uint16_t* __restrict__ hat_row) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  f32x2_t wp[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) wp[k] = grid_s[(words[0] >> (k * BITS)) & (NPTS - 1)];
  team_rotate_back_and_scale<D>(rc, ts, wp, sf[0]);
  float4 pq[1][2];
  get_pred(pq);     // the prediction values of this lane (zeros without a predictor)
  uint32_t o[4];
  o[0] = store16x2p<kBf16>(add2(pack2(pq[0][0].x, pq[0][0].y), wp[0]));
  o[1] = store16x2p<kBf16>(add2(pack2(pq[0][0].z, pq[0][0].w), wp[1]));
  o[2] = store16x2p<kBf16>(add2(pack2(pq[0][1].x, pq[0][1].y), wp[2]));
  o[3] = store16x2p<kBf16>(add2(pack2(pq[0][1].z, pq[0][1].w), wp[3]));
  __stcs(reinterpret_cast<uint4*>(hat_row + rc.member * 256 + rc.lane * 8), make_uint4(o[0], o[1], o[2], o[3]));
}

// This lane's codes and scales of one row (the small inputs of decode_row_core).
template <int D, int NPTS>
__device__ __forceinline__ void decode_row_load_codes(const RowCtx& rc, const uint8_t* __restrict__ codes_row,
                                                      const uint16_t* __restrict__ scales_row,
                                                      uint32_t (&words)[RowTeam<D>::CPM],
                                                      float (&sf)[RowTeam<D>::CPM]) {
  constexpr int CPM = RowTeam<D>::CPM;
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  const int c0 = rc.member * CPM;
#pragma unroll
  for (int c = 0; c < CPM; ++c) {
    words[c] = load_code_word<BITS>(codes_row, c0 + c, rc.lane);
    const int e0 = (c0 + c) * 256 + rc.lane * 8;
    sf[c] = __half2float(__ushort_as_half(scales_row[e0 >> rc.log_g]));
  }
}

// decode_row_core with the row's inputs read straight from global memory.
template <int D, int NPTS, bool kBf16>
__device__ __forceinline__ void decode_row(const RowCtx& rc, const f32x2_t* __restrict__ grid_s,
                                           TeamSmem<D>* ts, const uint8_t* __restrict__ codes_row,
                                           const uint16_t* __restrict__ scales_row,
                                           const float* __restrict__ pred_row,
                                           uint16_t* __restrict__ hat_row) {
  constexpr int CPM = RowTeam<D>::CPM;
  const int c0 = rc.member * CPM;
  float4 pq[CPM][2];
#pragma unroll
  for (int c = 0; c < CPM; ++c) {
    if (pred_row != nullptr) {
      pq[c][0] = __ldcg(reinterpret_cast<const float4*>(pred_row + (c0 + c) * 256 + rc.lane * 8));
      pq[c][1] = __ldcg(reinterpret_cast<const float4*>(pred_row + (c0 + c) * 256 + rc.lane * 8 + 4));
    } else {
      pq[c][0] = pq[c][1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }
  }
  uint32_t words[CPM];
  float sf[CPM];
  decode_row_load_codes<D, NPTS>(rc, codes_row, scales_row, words, sf);
  decode_row_core<D, NPTS, kBf16>(rc, grid_s, ts, words, sf,
                                  [&](float4 (&out)[CPM][2]) {
#pragma unroll
                                    for (int c = 0; c < CPM; ++c) { out[c][0] = pq[c][0]; out[c][1] = pq[c][1]; }
                                  },
                                  hat_row);
}

template <int D, int NPTS, bool kBf16>
__global__ void __launch_bounds__(kCodecThreads, 4) decode_rows_kernel(const CodecArgs a) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = D / 2 * BITS / 8;
  constexpr int TEAM = RowTeam<D>::TEAM, TEAMS = kCodecWarps / TEAM;
  __shared__ f32x2_t grid_s[NPTS];
  __shared__ TeamSmem<D> team_s[TEAMS];
  for (int i = threadIdx.x; i < NPTS; i += blockDim.x) {
    const float4 g = a.grid4[i];
    grid_s[i] = pack2(g.x, g.y);
  }
  __syncthreads();
  const RowCtx rc = make_row_ctx(a, TEAM, RowTeam<D>::NV, 1);
  const int team = (threadIdx.x >> 5) / TEAM;
  const int n_groups = D >> a.log_g;
  for (long long row = (long long)blockIdx.x * TEAMS + team; row < a.T; row += (long long)gridDim.x * TEAMS) {
    decode_row<D, NPTS, kBf16>(rc, grid_s, &team_s[team], a.codes + row * CODE_BYTES,
                               a.scales + row * n_groups,
                               a.P != nullptr ? a.P + row * a.ldP : nullptr, a.hat + row * a.ldHat);
  }
}

// ---------------------------------------------------------------------------------------------
// Row gather (Section 4.3 "Compatibility with Pruning": a token-pruning policy picks the tokens to
// keep and only those are compressed).  dst[i][0..d) = src[idx[i]][0..d) for 16-bit rows; idx ==
// nullptr copies row i (used to carry an unquantised first layer into the chain's buffers).  One warp
// per row, 16-byte accesses.  An index outside [0, n_src_rows) zero-fills the row and records
// kStatusBadIndex.
// ---------------------------------------------------------------------------------------------
constexpr int kStatusBadIndex = -1;     // AQUAKV_ERR_INVALID_ARG
__global__ void gather_rows_kernel(const uint16_t* __restrict__ src, long long ld_src, const long long* __restrict__ idx,
                                   long long n_rows, long long n_src_rows, int d, uint16_t* __restrict__ dst,
                                   long long ld_dst, int* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long i = warp; i < n_rows; i += n_warps) {
    const long long r = idx != nullptr ? idx[i] : i;
    const bool ok = r >= 0 && r < n_src_rows;
    if (!ok && lane == 0) atomicExch(status, kStatusBadIndex);
    uint4* out = reinterpret_cast<uint4*>(dst + i * ld_dst);
    const uint4* in = reinterpret_cast<const uint4*>(src + (ok ? r : 0) * ld_src);
    for (int c = lane; c < d / 8; c += 32) out[c] = ok ? __ldcs(in + c) : make_uint4(0u, 0u, 0u, 0u);
  }
}

}  // namespace aquakv
