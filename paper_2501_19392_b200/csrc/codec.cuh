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
constexpr uint32_t kCellBruteDev = 1u;    // the one non-ascending entry: search all points

struct SearchDev {
  const uint32_t* table;   // global copy [64*64] of the candidate lists
  float inv_w;             // cells / (2 * half extent)
};

// Shared-memory tables of the row routines.
template <int NPTS>
struct RowSmem {
  uint32_t table[kSearchCells * kSearchCells];
  float2 grid[NPTS];
};

template <int NPTS>
__device__ __forceinline__ void row_smem_fill(RowSmem<NPTS>* rs, const uint32_t* table, const float4* grid4) {
  for (int i = threadIdx.x; i < kSearchCells * kSearchCells; i += blockDim.x) rs->table[i] = table[i];
  for (int i = threadIdx.x; i < NPTS; i += blockDim.x) {
    const float4 g = grid4[i];
    rs->grid[i] = make_float2(g.x, g.y);
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

// Cell-table entry of one value pair (marked exhaustive outside the square).
__device__ __forceinline__ uint32_t search_entry(float y0, float y1, float inv_w,
                                                 const uint32_t* __restrict__ table_s) {
  const int ix = __float2int_rd(fmaf(y0, inv_w, 0.5f * kSearchCells));
  const int iy = __float2int_rd(fmaf(y1, inv_w, 0.5f * kSearchCells));
  const bool inside = static_cast<unsigned>(ix | iy) < unsigned(kSearchCells);
  const uint32_t e = table_s[inside ? ((iy << kSearchLogCells) + ix) : 0];
  return inside ? e : kCellBruteDev;
}

__device__ __forceinline__ float pair_dist(float y0, float y1, float2 g) {
  const float dx = __fsub_rn(y0, g.x), dy = __fsub_rn(y1, g.y);
  return fmaf(dy, dy, __fmul_rn(dx, dx));
}

// Arg-min over the ascending candidates of a table entry (three for n = 16, else four).
template <int NPTS>
__device__ __forceinline__ int nearest_of_candidates(float y0, float y1, uint32_t e,
                                                     const float2* __restrict__ grid_s) {
  const int c0 = e & 0xffu, c1 = (e >> 8) & 0xffu, c2 = (e >> 16) & 0xffu;
  const float t0 = pair_dist(y0, y1, grid_s[c0]);
  const float t1 = pair_dist(y0, y1, grid_s[c1]);
  const float t2 = pair_dist(y0, y1, grid_s[c2]);
  int idx = c0;
  float best = t0;
  if (t1 < best) { best = t1; idx = c1; }
  if (t2 < best) { best = t2; idx = c2; }
  if constexpr (NPTS > 16) {
    const int c3 = e >> 24;
    const float t3 = pair_dist(y0, y1, grid_s[c3]);
    if (t3 < best) { idx = c3; }
  }
  return idx;
}

template <int NPTS>
__device__ __noinline__ int nearest_exhaustive(float y0, float y1, const float2* __restrict__ grid_s) {
  float best = 3.0e38f;
  int idx = 0;
  for (int i = 0; i < NPTS; ++i) {
    const float t = pair_dist(y0, y1, grid_s[i]);
    if (t < best) { best = t; idx = i; }             // strict: lowest index wins ties
  }
  return idx;
}

// Per-warp constants of the row routines.
struct RowCtx {
  uint32_t signmask;       // this lane's entry of CodecArgs::signmask
  float inv_w;             // SearchDev::inv_w
  int log_h, log_g;
  int lane;
};

// One token row of Q and of the reconstruction (Algorithm 2 lines 6-7 / 9):
//   codes, scales = Q(x - pred);  hat = round16(pred + Q^-1(codes, scales)).
// pred_row == nullptr: no predictor.  hat_row == nullptr: reconstruction not wanted.  The prediction
// is read twice (for the residual and again for the reconstruction) instead of being held in 32
// registers across the rotation and the search; both reads bypass L1 (ld.global.cg) because the
// prediction may have been written by another SM of the same kernel just before.
template <int D, int NPTS, bool kBf16>
__device__ __forceinline__ void encode_row(const RowCtx& rc, const RowSmem<NPTS>* __restrict__ rsm,
                                           const uint16_t* __restrict__ x_row,
                                           const float* __restrict__ pred_row,
                                           uint8_t* __restrict__ codes_row,
                                           uint16_t* __restrict__ scales_row,
                                           uint16_t* __restrict__ hat_row) {
  constexpr int NC = D / 256, NV = NC * 8;
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  const int lane = rc.lane;
  const float inv_g = exp2f(-static_cast<float>(rc.log_g));
  const float rs = exp2f(-0.5f * static_cast<float>(rc.log_h));
  float v[NV];
  // ---- residual r = x - pred -------------------------------------------------------------------
  {
    uint4 raw[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c)
      raw[c] = *reinterpret_cast<const uint4*>(x_row + c * 256 + lane * 8);
    if (pred_row != nullptr) {
      float4 pq[NC][2];
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        pq[c][0] = __ldcg(reinterpret_cast<const float4*>(pred_row + c * 256 + lane * 8));
        pq[c][1] = __ldcg(reinterpret_cast<const float4*>(pred_row + c * 256 + lane * 8 + 4));
      }
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
        const float pp[8] = {pq[c][0].x, pq[c][0].y, pq[c][0].z, pq[c][0].w,
                             pq[c][1].x, pq[c][1].y, pq[c][1].z, pq[c][1].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          v[c * 8 + 2 * i] = __fsub_rn(load16<kBf16>(uint16_t(w[i] & 0xffffu)), pp[2 * i]);
          v[c * 8 + 2 * i + 1] = __fsub_rn(load16<kBf16>(uint16_t(w[i] >> 16)), pp[2 * i + 1]);
        }
      }
    } else {
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        const uint32_t w[4] = {raw[c].x, raw[c].y, raw[c].z, raw[c].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          v[c * 8 + 2 * i] = load16<kBf16>(uint16_t(w[i] & 0xffffu));
          v[c * 8 + 2 * i + 1] = load16<kBf16>(uint16_t(w[i] >> 16));
        }
      }
    }
  }
  // ---- group scale: root mean square, stored as fp16; normalise with the rounded value --------
  float ss[NC], sf[NC], inv[NC];
  group_sums<NC>(v, ss, rc.log_g);
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    const float s = fminf(sqrtf(ss[c] * inv_g), 65504.0f);
    const __half s16 = __float2half_rn(s);
    sf[c] = __half2float(s16);
    if (rc.log_g >= 8) {                 // one lane per group writes the scale
      const int cpg = 1 << (rc.log_g - 8);
      if (lane == 0 && (c % cpg) == 0) scales_row[c / cpg] = __half_as_ushort(s16);
    } else {
      const int lpg = 1 << (rc.log_g - 3);   // lanes per group
      if ((lane % lpg) == 0) scales_row[c * (256 >> rc.log_g) + lane / lpg] = __half_as_ushort(s16);
    }
    // the rotation is linear: the division by the scale is applied after it, merged with 1/sqrt(h)
    inv[c] = (sf[c] > 0.0f ? 1.0f / sf[c] : 0.0f) * rs;
#pragma unroll
    for (int i = 0; i < 8; ++i) v[c * 8 + i] = apply_sign(v[c * 8 + i], rc.signmask, c * 8 + i);
  }
  // ---- rotate ------------------------------------------------------------------------------------
  fwht_regs_and_lanes<NV>(v, rc.log_h, lane);
#pragma unroll
  for (int c = 0; c < NC; ++c)
#pragma unroll
    for (int i = 0; i < 8; ++i) v[c * 8 + i] *= inv[c];
  // ---- nearest grid point per pair: all table entries first, then the candidates ----------------
  uint32_t entry[NV / 2];
  uint32_t any_brute = 0;
#pragma unroll
  for (int j = 0; j < NV / 2; ++j) {
    entry[j] = search_entry(v[2 * j], v[2 * j + 1], rc.inv_w, rsm->table);
    any_brute |= uint32_t(entry[j] == kCellBruteDev);
  }
  const bool slow = __any_sync(0xffffffffu, any_brute != 0);
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    uint32_t word = 0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int j = c * 4 + k;
      int idx;
      if (!slow) {
        idx = nearest_of_candidates<NPTS>(v[2 * j], v[2 * j + 1], entry[j], rsm->grid);
      } else {
        idx = entry[j] == kCellBruteDev
                  ? nearest_exhaustive<NPTS>(v[2 * j], v[2 * j + 1], rsm->grid)
                  : nearest_of_candidates<NPTS>(v[2 * j], v[2 * j + 1], entry[j], rsm->grid);
      }
      word |= uint32_t(idx) << (k * BITS);
      const float2 g = rsm->grid[idx];
      v[2 * j] = g.x;
      v[2 * j + 1] = g.y;
    }
    store_code_word<BITS>(codes_row, c, lane, word);
  }
  // ---- reconstruction: hat = round16(pred + Q^-1(codes)) ---------------------------------------
  if (hat_row != nullptr) {
    float4 pq[NC][2];
    if (pred_row != nullptr) {
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        pq[c][0] = __ldcg(reinterpret_cast<const float4*>(pred_row + c * 256 + lane * 8));
        pq[c][1] = __ldcg(reinterpret_cast<const float4*>(pred_row + c * 256 + lane * 8 + 4));
      }
    } else {
#pragma unroll
      for (int c = 0; c < NC; ++c) pq[c][0] = pq[c][1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    }
    rotate_back_and_scale<NV>(v, sf, rc.signmask, rc.log_h, lane);
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const float pp[8] = {pq[c][0].x, pq[c][0].y, pq[c][0].z, pq[c][0].w,
                           pq[c][1].x, pq[c][1].y, pq[c][1].z, pq[c][1].w};
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const uint32_t lo = store16<kBf16>(__fadd_rn(pp[2 * i], v[c * 8 + 2 * i]));
        const uint32_t hi = store16<kBf16>(__fadd_rn(pp[2 * i + 1], v[c * 8 + 2 * i + 1]));
        o[i] = lo | (hi << 16);
      }
      *reinterpret_cast<uint4*>(hat_row + c * 256 + lane * 8) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
}

template <int D, int NPTS, bool kBf16>
__global__ void __launch_bounds__(kCodecThreads, 2) encode_rows_kernel(const CodecArgs a) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = D / 2 * BITS / 8;
  __shared__ RowSmem<NPTS> rsm;
  row_smem_fill<NPTS>(&rsm, a.search.table, a.grid4);
  __syncthreads();
  RowCtx rc;
  rc.lane = threadIdx.x & 31;
  rc.signmask = a.signmask[rc.lane];
  rc.inv_w = a.search.inv_w;
  rc.log_h = a.log_h;
  rc.log_g = a.log_g;
  const int warp = threadIdx.x >> 5;
  const int n_groups = D >> a.log_g;
  for (long long row = (long long)blockIdx.x * kCodecWarps + warp; row < a.T;
       row += (long long)gridDim.x * kCodecWarps) {
    encode_row<D, NPTS, kBf16>(rc, &rsm, a.X + row * a.ldX,
                               a.P != nullptr ? a.P + row * a.ldP : nullptr,
                               a.codes + row * CODE_BYTES, a.scales + row * n_groups,
                               a.hat != nullptr ? a.hat + row * a.ldHat : nullptr);
  }
}

// One token row of Algorithm 3 line 5 / 7 given the prediction:
//   hat = round16(pred + Q^-1(codes, scales)).  pred_row == nullptr: no predictor.
template <int D, int NPTS, bool kBf16, typename GridT>
__device__ __forceinline__ void decode_row(const RowCtx& rc, const GridT* __restrict__ grid_s,
                                           const uint8_t* __restrict__ codes_row,
                                           const uint16_t* __restrict__ scales_row,
                                           const float* __restrict__ pred_row,
                                           uint16_t* __restrict__ hat_row) {
  constexpr int NC = D / 256, NV = NC * 8;
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  const int lane = rc.lane;
  float w[NV], sf[NC];
  float4 pq[NC][2];
  if (pred_row != nullptr) {
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      pq[c][0] = __ldcg(reinterpret_cast<const float4*>(pred_row + c * 256 + lane * 8));
      pq[c][1] = __ldcg(reinterpret_cast<const float4*>(pred_row + c * 256 + lane * 8 + 4));
    }
  } else {
#pragma unroll
    for (int c = 0; c < NC; ++c) pq[c][0] = pq[c][1] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  }
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    const uint32_t word = load_code_word<BITS>(codes_row, c, lane);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const GridT g = grid_s[(word >> (k * BITS)) & (NPTS - 1)];
      w[c * 8 + 2 * k] = g.x;
      w[c * 8 + 2 * k + 1] = g.y;
    }
    const int e0 = c * 256 + lane * 8;
    sf[c] = __half2float(__ushort_as_half(scales_row[e0 >> rc.log_g]));
  }
  rotate_back_and_scale<NV>(w, sf, rc.signmask, rc.log_h, lane);
#pragma unroll
  for (int c = 0; c < NC; ++c) {
    const float pp[8] = {pq[c][0].x, pq[c][0].y, pq[c][0].z, pq[c][0].w,
                         pq[c][1].x, pq[c][1].y, pq[c][1].z, pq[c][1].w};
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t lo = store16<kBf16>(__fadd_rn(pp[2 * i], w[c * 8 + 2 * i]));
      const uint32_t hi = store16<kBf16>(__fadd_rn(pp[2 * i + 1], w[c * 8 + 2 * i + 1]));
      o[i] = lo | (hi << 16);
    }
    *reinterpret_cast<uint4*>(hat_row + c * 256 + lane * 8) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

template <int D, int NPTS, bool kBf16>
__global__ void __launch_bounds__(kCodecThreads) decode_rows_kernel(const CodecArgs a) {
  constexpr int BITS = NPTS == 16 ? 4 : (NPTS == 64 ? 6 : 8);
  constexpr int CODE_BYTES = D / 2 * BITS / 8;
  __shared__ float2 grid_s[NPTS];
  for (int i = threadIdx.x; i < NPTS; i += blockDim.x) {
    const float4 g = a.grid4[i];
    grid_s[i] = make_float2(g.x, g.y);
  }
  __syncthreads();
  RowCtx rc;
  rc.lane = threadIdx.x & 31;
  rc.signmask = a.signmask[rc.lane];
  rc.inv_w = a.search.inv_w;
  rc.log_h = a.log_h;
  rc.log_g = a.log_g;
  const int warp = threadIdx.x >> 5;
  const int n_groups = D >> a.log_g;
  for (long long row = (long long)blockIdx.x * kCodecWarps + warp; row < a.T;
       row += (long long)gridDim.x * kCodecWarps) {
    decode_row<D, NPTS, kBf16>(rc, grid_s, a.codes + row * CODE_BYTES, a.scales + row * n_groups,
                               a.P != nullptr ? a.P + row * a.ldP : nullptr, a.hat + row * a.ldHat);
  }
}

}  // namespace aquakv
