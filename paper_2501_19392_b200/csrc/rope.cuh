// Rotary position encoding of cached PRE-RoPE keys at attention time (Section 3.3 "Positional
// embeddings": predictors and quantizers work on the keys before RoPE, so the reconstructed keys are
// rotated when the block attends to them in Algorithm 4).
//
// For a head of HD values and a token at position pos, frequency i < HD/2 has the angle
// pos * theta_base^(-2 i / HD) and rotates the pair (x[i], x[i + HD/2]) (half-split pairing):
//   y[i] = x[i] cos - x[i + HD/2] sin,   y[i + HD/2] = x[i + HD/2] cos + x[i] sin,
// computed in fp32 from a table of (cos, sin) pairs that rope_table_kernel fills in double precision,
// and rounded once to the cache's 16-bit type.  Values are not rotated; the query arrives rotated.
#pragma once

#include "codec.cuh"

namespace aquakv {

// table[pos * half + i] = (cos, sin)(pos * theta_base^(-2 i / head_dim)), pos < n_pos, i < half = head_dim / 2.
__global__ void rope_table_kernel(float2* __restrict__ table, long long n_pos, int half, double theta_base) {
  const long long n = n_pos * half;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < n;
       idx += (long long)gridDim.x * blockDim.x) {
    const long long pos = idx / half;
    const int i = int(idx % half);
    const double freq = pow(theta_base, -double(i) / double(half));
    double s, c;
    sincos(double(pos) * freq, &s, &c);
    table[idx] = make_float2(float(c), float(s));
  }
}

struct RopeArgs {
  const uint16_t* in;      // key rows [rows, ld_in]
  long long ld_in;
  uint16_t* out;           // rotated rows [rows, ld_out]
  long long ld_out;
  long long rows;
  int n_kv_heads;
  int head_dim;            // 64 or 128
  const float2* table;     // [n_pos][head_dim / 2]
  long long n_pos;
  // position of row r: pos_list != nullptr ? pos_list[r % period] : pos0 + (row_base + r) % period
  const int* pos_list;
  long long period;
  long long row_base;
  long long pos0;
  int* status;             // kStatusBadIndex when a position falls outside the table (the row is zero-filled)
};

// One thread per 8 + 8 values: dimensions [8 p, 8 p + 8) of a head and their partners HD/2 further on.
template <bool kBf16>
__global__ void __launch_bounds__(256) rope_rows_kernel(const RopeArgs a) {
  const int half = a.head_dim / 2;
  const int pieces = half / 8;                       // per head
  const long long units_per_row = (long long)a.n_kv_heads * pieces;
  const long long n_units = a.rows * units_per_row;
  for (long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x; u < n_units;
       u += (long long)gridDim.x * blockDim.x) {
    const long long r = u / units_per_row;
    const int w = int(u % units_per_row);
    const int head = w / pieces, piece = w % pieces;
    const long long pos = a.pos_list != nullptr ? (long long)a.pos_list[r % a.period]
                                                : a.pos0 + (a.row_base + r) % a.period;
    const bool ok = pos >= 0 && pos < a.n_pos;
    uint16_t* dst = a.out + r * a.ld_out + head * a.head_dim + piece * 8;
    if (!ok) {
      atomicExch(a.status, kStatusBadIndex);
      *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
      *reinterpret_cast<uint4*>(dst + half) = make_uint4(0u, 0u, 0u, 0u);
      continue;
    }
    const uint16_t* src = a.in + r * a.ld_in + head * a.head_dim + piece * 8;
    const uint4 lo_raw = __ldcs(reinterpret_cast<const uint4*>(src));
    const uint4 hi_raw = __ldcs(reinterpret_cast<const uint4*>(src + half));
    const float4* tab = reinterpret_cast<const float4*>(a.table + pos * half + piece * 8);
    float lo[8], hi[8], ylo[8], yhi[8];
    unpack2(load16x2<kBf16>(lo_raw.x), lo[0], lo[1]);
    unpack2(load16x2<kBf16>(lo_raw.y), lo[2], lo[3]);
    unpack2(load16x2<kBf16>(lo_raw.z), lo[4], lo[5]);
    unpack2(load16x2<kBf16>(lo_raw.w), lo[6], lo[7]);
    unpack2(load16x2<kBf16>(hi_raw.x), hi[0], hi[1]);
    unpack2(load16x2<kBf16>(hi_raw.y), hi[2], hi[3]);
    unpack2(load16x2<kBf16>(hi_raw.z), hi[4], hi[5]);
    unpack2(load16x2<kBf16>(hi_raw.w), hi[6], hi[7]);
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const float4 cs = __ldg(tab + k);              // (cos, sin) of dimensions 2k and 2k + 1
      ylo[2 * k] = fmaf(lo[2 * k], cs.x, -hi[2 * k] * cs.y);
      yhi[2 * k] = fmaf(hi[2 * k], cs.x, lo[2 * k] * cs.y);
      ylo[2 * k + 1] = fmaf(lo[2 * k + 1], cs.z, -hi[2 * k + 1] * cs.w);
      yhi[2 * k + 1] = fmaf(hi[2 * k + 1], cs.z, lo[2 * k + 1] * cs.w);
    }
    uint4 o_lo, o_hi;
    o_lo.x = store16x2p<kBf16>(pack2(ylo[0], ylo[1]));
    o_lo.y = store16x2p<kBf16>(pack2(ylo[2], ylo[3]));
    o_lo.z = store16x2p<kBf16>(pack2(ylo[4], ylo[5]));
    o_lo.w = store16x2p<kBf16>(pack2(ylo[6], ylo[7]));
    o_hi.x = store16x2p<kBf16>(pack2(yhi[0], yhi[1]));
    o_hi.y = store16x2p<kBf16>(pack2(yhi[2], yhi[3]));
    o_hi.z = store16x2p<kBf16>(pack2(yhi[4], yhi[5]));
    o_hi.w = store16x2p<kBf16>(pack2(yhi[6], yhi[7]));
    *reinterpret_cast<uint4*>(dst) = o_lo;
    *reinterpret_cast<uint4*>(dst + half) = o_hi;
  }
}

}  // namespace aquakv
