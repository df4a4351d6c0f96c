// Host side of the AQUA-KV codec library: the C ABI declared in include/aquakv.h, argument
// validation, workspace carving, tensor-map construction and kernel launches.  Every step of
// Algorithm 2 / Algorithm 3 / the attention read of Algorithm 4 runs in the kernels of
// layer_kernel.cuh, gemm_pred.cuh, codec.cuh and attn.cuh; nothing is computed on the host and
// there is no fallback path.
//
// The single-phase entry points cut large calls into token chunks sized so that one chunk's fp32
// prediction stays resident in the 126 MB L2 between the GEMM that writes it and the row kernel
// that reads it; the fused attention entry point works on chunks of about 32 waves of the layer
// kernel.
#include <cuda.h>
#include <cuda_runtime.h>

#include <atomic>

#include <cmath>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "aquakv.h"
#include "attn.cuh"
#include "calib.cuh"
#include "chain_kernel.cuh"
#include "codec.cuh"
#include "gemm_pred.cuh"
#include "grid4.cuh"
#include "layer_kernel.cuh"
#include "rope.cuh"
#include "search_table.h"
#include "uniform.cuh"

using namespace aquakv;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct aquakv_ctx {
  aquakv_params p;
  int log_h, log_g, bits, code_bytes, n_groups;
  bool bf16;
  int device;
  int sm_count;
  int chunk_tokens;        // tokens per L2-resident chunk
  int attn_block_tokens;   // tokens per split-KV block
  int attn_mode;           // AQUAKV_ATTN_SPLIT or AQUAKV_ATTN_FUSED (aquakv_set_attn_mode)
  float4* d_grid4;
  uint4* d_grid4_table;    // candidate lists of the four-dimensional grid's cells (grid_dim 4 only)
  uint32_t* d_signmask[2]; // [0] keys, [1] values
  int* d_status;
  uint32_t* d_search_table;
  SearchTableSpec search_spec;
  EncodeTiledFn encode_tiled;
  int64_t launches;
  // optional per-kernel-class timing (aquakv_profile_*): event pairs recorded around launches
  bool prof_on;
  int prof_n;                       // pairs recorded since the last read
  cudaEvent_t* prof_ev;             // 2 * kProfMaxPairs events, created when profiling is enabled
  uint8_t* prof_class;              // kernel class of each pair
};

namespace {

constexpr int kRoleK = 0, kRoleV = 1;
constexpr int kProfMaxPairs = 8192;

// Brackets one kernel launch with a pair of events when profiling is enabled.
struct ProfScope {
  aquakv_ctx* c;
  cudaStream_t st;
  int slot;
  ProfScope(aquakv_ctx* ctx, cudaStream_t s, int kernel_class) : c(ctx), st(s), slot(-1) {
    if (c->prof_on && c->prof_n < kProfMaxPairs) {
      slot = c->prof_n++;
      c->prof_class[slot] = uint8_t(kernel_class);
      cudaEventRecord(c->prof_ev[2 * slot], st);
    }
  }
  ~ProfScope() {
    if (slot >= 0) cudaEventRecord(c->prof_ev[2 * slot + 1], st);
  }
};

inline int ilog2(int v) {
  int b = 0;
  while ((1 << b) < v) ++b;
  return b;
}
inline bool is_pow2(int v) { return v > 0 && (v & (v - 1)) == 0; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t round_up(size_t v, size_t m) { return (v + m - 1) / m * m; }
// The kernels want their scratch on 128-byte lines (32-byte vector loads, whole-line L2 discards); the
// caller's workspace need only be 16-byte aligned, so every workspace size includes this slack.
constexpr size_t kWsSlack = 128;
inline uint8_t* ws_base(void* workspace) {
  return reinterpret_cast<uint8_t*>(round_up(reinterpret_cast<uintptr_t>(workspace), kWsSlack));
}

int check_params(const aquakv_params* p) {
  if (p == nullptr) return AQUAKV_ERR_INVALID_ARG;
  if (p->d_kv <= 0 || p->had_block <= 0 || p->scale_group <= 0 || p->grid_size <= 0)
    return AQUAKV_ERR_INVALID_ARG;
  if (p->dtype != AQUAKV_F16 && p->dtype != AQUAKV_BF16) return AQUAKV_ERR_INVALID_ARG;
  if (p->grid_dim == 1) {
    // uniform round-to-nearest backbone with absmax normalisation: grid_size = 2^b levels per value,
    // groups of 32 .. d_kv values; had_block 1: no rotation, 64 .. d_kv: random signs and a Hadamard
    // rotation of that block size before the levels
    if (p->d_kv != 256 && p->d_kv != 512 && p->d_kv != 1024) return AQUAKV_ERR_UNSUPPORTED;
    if (p->grid_size != 4 && p->grid_size != 8 && p->grid_size != 16) return AQUAKV_ERR_UNSUPPORTED;
    if (p->had_block != 1 && (!is_pow2(p->had_block) || p->had_block < 64 || p->had_block > p->d_kv))
      return AQUAKV_ERR_UNSUPPORTED;
    if (!is_pow2(p->scale_group) || p->scale_group < 32 || p->scale_group > p->d_kv) return AQUAKV_ERR_UNSUPPORTED;
    return AQUAKV_OK;
  }
  if (p->grid_dim != 2 && p->grid_dim != 4) return AQUAKV_ERR_UNSUPPORTED;
  if (p->d_kv != 256 && p->d_kv != 512 && p->d_kv != 1024) return AQUAKV_ERR_UNSUPPORTED;
  if (p->grid_dim == 4) {
    // the four-dimensional grid: 256 points, one byte per four values
    if (p->grid_size != 256) return AQUAKV_ERR_UNSUPPORTED;
  } else if (p->grid_size != 16 && p->grid_size != 64 && p->grid_size != 256) {
    return AQUAKV_ERR_UNSUPPORTED;
  }
  if (!is_pow2(p->had_block) || p->had_block < 64 || p->had_block > p->d_kv)
    return AQUAKV_ERR_UNSUPPORTED;
  if (!is_pow2(p->scale_group) || p->scale_group < p->had_block || p->scale_group > p->d_kv)
    return AQUAKV_ERR_UNSUPPORTED;
  return AQUAKV_OK;
}

// ---------------------------------------------------------------------------------------------
// launches
// ---------------------------------------------------------------------------------------------
int make_tmap(const aquakv_ctx* c, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols,
              uint64_t ld_elems, uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {ld_elems * 2};
  const cuuint32_t box[2] = {uint32_t(kBK), box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = c->encode_tiled(
      m, c->bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2,
      const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
      CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

// P[M, d] = [in0 ; in1] W^T + bias for M rows starting at the given pointers.
int launch_predict(aquakv_ctx* c, cudaStream_t st, int M, const void* in0, const void* in1,
                   int64_t ld_in0, int64_t ld_in1, const void* W, const float* bias, float* P,
                   int64_t ldP) {
  const int d = c->p.d_kv;
  const int n_in = in1 != nullptr ? 2 : 1;
  CUtensorMap tA0, tA1, tB;
  int rc = make_tmap(c, &tA0, in0, uint64_t(M), uint64_t(d), uint64_t(ld_in0), kBM);
  if (rc) return rc;
  if (in1 != nullptr) {
    rc = make_tmap(c, &tA1, in1, uint64_t(M), uint64_t(d), uint64_t(ld_in1), kBM);
    if (rc) return rc;
  } else {
    tA1 = tA0;
  }
  rc = make_tmap(c, &tB, W, uint64_t(d), uint64_t(n_in) * d, uint64_t(n_in) * d, kBN);
  if (rc) return rc;
  GemmArgs g;
  g.M = M;
  g.N = d;
  g.nk0 = d / kBK;
  g.nk1 = in1 != nullptr ? d / kBK : 0;
  g.P = P;
  g.ldP = ldP;
  g.bias = bias;
  g.status = c->d_status;
  const int tiles = ((M + kBM - 1) / kBM) * (d / kBN);
  const int grid = tiles < c->sm_count ? tiles : c->sm_count;
  ProfScope prof(c, st, AQUAKV_KERNEL_PREDICT);
  if (c->bf16) {
    gemm_pred_kernel<true><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tA0, tA1, tB, g);
  } else {
    gemm_pred_kernel<false><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tA0, tA1, tB, g);
  }
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

// d_kv = 1024 with the Hadamard block and the scale group spanning the row: one warp per row.
inline bool warp_rows(const CodecArgs& a, int d) { return d == 1024 && a.log_h == 10 && a.log_g == 10; }

template <int D, int NPTS, bool BF>
void launch_encode_rows_t(aquakv_ctx*, cudaStream_t st, const CodecArgs& a, int grid) {
  if constexpr (D == 1024) {
    if (warp_rows(a, D)) {
      encode_rows_warp_kernel<NPTS, BF><<<grid, kWrKernelWarps * 32, 0, st>>>(a);
      return;
    }
  }
  encode_rows_kernel<D, NPTS, BF><<<grid, kCodecThreads, 0, st>>>(a);
}

template <int D, int NPTS, bool BF>
void launch_decode_rows_t(aquakv_ctx*, cudaStream_t st, const CodecArgs& a, int grid) {
  if constexpr (D == 1024) {
    if (warp_rows(a, D)) {
      decode_rows_warp_kernel<NPTS, BF><<<grid, kWrKernelWarps * 32, 0, st>>>(a);
      return;
    }
  }
  decode_rows_kernel<D, NPTS, BF><<<grid, kCodecThreads, 0, st>>>(a);
}

#define AQ_DISPATCH_DNB(FN, ...)                                                     \
  do {                                                                               \
    const int d_ = c->p.d_kv, n_ = c->p.grid_size;                                   \
    const bool b_ = c->bf16;                                                         \
    if (d_ == 256 && n_ == 16 && b_) FN<256, 16, true>(__VA_ARGS__);                 \
    else if (d_ == 256 && n_ == 16) FN<256, 16, false>(__VA_ARGS__);                 \
    else if (d_ == 256 && n_ == 64 && b_) FN<256, 64, true>(__VA_ARGS__);            \
    else if (d_ == 256 && n_ == 64) FN<256, 64, false>(__VA_ARGS__);                 \
    else if (d_ == 256 && b_) FN<256, 256, true>(__VA_ARGS__);                       \
    else if (d_ == 256) FN<256, 256, false>(__VA_ARGS__);                            \
    else if (d_ == 512 && n_ == 16 && b_) FN<512, 16, true>(__VA_ARGS__);            \
    else if (d_ == 512 && n_ == 16) FN<512, 16, false>(__VA_ARGS__);                 \
    else if (d_ == 512 && n_ == 64 && b_) FN<512, 64, true>(__VA_ARGS__);            \
    else if (d_ == 512 && n_ == 64) FN<512, 64, false>(__VA_ARGS__);                 \
    else if (d_ == 512 && b_) FN<512, 256, true>(__VA_ARGS__);                       \
    else if (d_ == 512) FN<512, 256, false>(__VA_ARGS__);                            \
    else if (n_ == 16 && b_) FN<1024, 16, true>(__VA_ARGS__);                        \
    else if (n_ == 16) FN<1024, 16, false>(__VA_ARGS__);                             \
    else if (n_ == 64 && b_) FN<1024, 64, true>(__VA_ARGS__);                        \
    else if (n_ == 64) FN<1024, 64, false>(__VA_ARGS__);                             \
    else if (b_) FN<1024, 256, true>(__VA_ARGS__);                                   \
    else FN<1024, 256, false>(__VA_ARGS__);                                          \
  } while (0)

int codec_grid(const aquakv_ctx* c, int rows) {
  const bool wr = c->p.d_kv == 1024 && c->log_h == 10 && c->log_g == 10;   // one warp per row, four per CTA
  const int rows_per_block = wr ? kWrKernelWarps : kCodecWarps / (c->p.d_kv / 256);   // else one warp per 256-element chunk
  const int blocks = (rows + rows_per_block - 1) / rows_per_block;
  const int cap = c->sm_count * 8;
  return blocks < cap ? blocks : cap;
}

CodecArgs codec_args(const aquakv_ctx* c, int role, int rows) {
  CodecArgs a;
  std::memset(&a, 0, sizeof(a));
  a.signmask = c->d_signmask[role];
  a.grid4 = c->d_grid4;
  a.search.table = c->d_search_table;
  a.search.inv_w = c->search_spec.inv_w;
  a.T = rows;
  a.log_h = c->log_h;
  a.log_g = c->log_g;
  return a;
}

// One phase of Algorithm 2 on `rows` rows: codes/scales = Q(X - P), hat = round16(P + Q^-1(..)).
// Backbones without a fused layer kernel (the uniform levels, grid_dim 1, and the four-dimensional grid,
// grid_dim 4): predictor GEMM and a stand-alone row kernel per phase, per-layer entry points only.
inline bool uniform_backbone(const aquakv_ctx* c) { return c->p.grid_dim != 2; }

// Row kernels of the four-dimensional grid (grid4.cuh): X == nullptr decodes.
int launch_grid4_rows(aquakv_ctx* c, cudaStream_t st, int role, int rows, const void* X, int64_t ldX, const float* P,
                      int64_t ldP, uint8_t* codes, uint16_t* scales, void* hat, int64_t ldHat) {
  Grid4Args ga;
  UniformArgs& a = ga.u;
  ga.grid = c->d_grid4;
  ga.table = c->d_grid4_table;
  ga.signmask = c->d_signmask[role];
  ga.log_h = c->log_h;
  a.X = static_cast<const uint16_t*>(X);
  a.ldX = ldX;
  a.P = P;
  a.ldP = ldP;
  a.codes = codes;
  a.scales = scales;
  a.hat = static_cast<uint16_t*>(hat);
  a.ldHat = ldHat;
  a.T = rows;
  a.d = c->p.d_kv;
  a.log_g = c->log_g;
  int64_t blocks = (int64_t(rows) + kUniformWarps - 1) / kUniformWarps;
  const int64_t cap = int64_t(c->sm_count) * 8;
  if (blocks > cap) blocks = cap;
  const int grid = int(blocks), threads = kUniformWarps * 32;
  const bool enc = X != nullptr;
  ProfScope prof(c, st, enc ? AQUAKV_KERNEL_ENCODE_ROWS : AQUAKV_KERNEL_DECODE_ROWS);
#define AQ_GRID4(NCH)                                                                                 \
  do {                                                                                                \
    if (enc) {                                                                                        \
      if (c->bf16) grid4_encode_rows_kernel<true, NCH><<<grid, threads, 0, st>>>(ga);                 \
      else grid4_encode_rows_kernel<false, NCH><<<grid, threads, 0, st>>>(ga);                        \
    } else {                                                                                          \
      if (c->bf16) grid4_decode_rows_kernel<true, NCH><<<grid, threads, 0, st>>>(ga);                 \
      else grid4_decode_rows_kernel<false, NCH><<<grid, threads, 0, st>>>(ga);                        \
    }                                                                                                 \
  } while (0)
  if (a.d == 256) AQ_GRID4(1);
  else if (a.d == 512) AQ_GRID4(2);
  else AQ_GRID4(4);
#undef AQ_GRID4
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

// Row kernels of the uniform backbone (uniform.cuh): X == nullptr decodes.
int launch_uniform_rows(aquakv_ctx* c, cudaStream_t st, int role, int rows, const void* X, int64_t ldX, const float* P,
                        int64_t ldP, uint8_t* codes, uint16_t* scales, void* hat, int64_t ldHat) {
  if (c->p.grid_dim == 4) return launch_grid4_rows(c, st, role, rows, X, ldX, P, ldP, codes, scales, hat, ldHat);
  UniformRotArgs ra;
  UniformArgs& a = ra.u;
  ra.signmask = c->d_signmask[role];
  ra.log_h = c->log_h;
  a.X = static_cast<const uint16_t*>(X);
  a.ldX = ldX;
  a.P = P;
  a.ldP = ldP;
  a.codes = codes;
  a.scales = scales;
  a.hat = static_cast<uint16_t*>(hat);
  a.ldHat = ldHat;
  a.T = rows;
  a.d = c->p.d_kv;
  a.log_g = c->log_g;
  int64_t blocks = (int64_t(rows) + kUniformWarps - 1) / kUniformWarps;
  const int64_t cap = int64_t(c->sm_count) * 16;
  if (blocks > cap) blocks = cap;
  const int grid = int(blocks), threads = kUniformWarps * 32;
  const bool enc = X != nullptr;
  ProfScope prof(c, st, enc ? AQUAKV_KERNEL_ENCODE_ROWS : AQUAKV_KERNEL_DECODE_ROWS);
#define AQ_UNIFORM(BITS)                                                                              \
  do {                                                                                                \
    if (enc) {                                                                                        \
      if (c->bf16) uniform_encode_rows_kernel<BITS, true><<<grid, threads, 0, st>>>(a);               \
      else uniform_encode_rows_kernel<BITS, false><<<grid, threads, 0, st>>>(a);                      \
    } else {                                                                                          \
      if (c->bf16) uniform_decode_rows_kernel<BITS, true><<<grid, threads, 0, st>>>(a);               \
      else uniform_decode_rows_kernel<BITS, false><<<grid, threads, 0, st>>>(a);                      \
    }                                                                                                 \
  } while (0)
#define AQ_UNIFORM_ROT2(BITS, NCH)                                                                    \
  do {                                                                                                \
    if (enc) {                                                                                        \
      if (c->bf16) uniform_rot_encode_rows_kernel<BITS, true, NCH><<<grid, threads, 0, st>>>(ra);     \
      else uniform_rot_encode_rows_kernel<BITS, false, NCH><<<grid, threads, 0, st>>>(ra);            \
    } else {                                                                                          \
      if (c->bf16) uniform_rot_decode_rows_kernel<BITS, true, NCH><<<grid, threads, 0, st>>>(ra);     \
      else uniform_rot_decode_rows_kernel<BITS, false, NCH><<<grid, threads, 0, st>>>(ra);            \
    }                                                                                                 \
  } while (0)
#define AQ_UNIFORM_ROT(BITS)                                                                          \
  do {                                                                                                \
    if (a.d == 256) AQ_UNIFORM_ROT2(BITS, 1);                                                         \
    else if (a.d == 512) AQ_UNIFORM_ROT2(BITS, 2);                                                    \
    else AQ_UNIFORM_ROT2(BITS, 4);                                                                    \
  } while (0)
  if (c->log_h > 0) {
    if (c->bits == 2) AQ_UNIFORM_ROT(2);
    else if (c->bits == 3) AQ_UNIFORM_ROT(3);
    else AQ_UNIFORM_ROT(4);
  } else if (c->bits == 2) AQ_UNIFORM(2);
  else if (c->bits == 3) AQ_UNIFORM(3);
  else AQ_UNIFORM(4);
#undef AQ_UNIFORM_ROT
#undef AQ_UNIFORM_ROT2
#undef AQ_UNIFORM
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

int launch_encode_rows(aquakv_ctx* c, cudaStream_t st, int role, int rows, const void* X,
                       int64_t ldX, const float* P, int64_t ldP, uint8_t* codes, uint16_t* scales,
                       void* hat, int64_t ldHat) {
  if (uniform_backbone(c)) return launch_uniform_rows(c, st, role, rows, X, ldX, P, ldP, codes, scales, hat, ldHat);
  CodecArgs a = codec_args(c, role, rows);
  a.X = static_cast<const uint16_t*>(X);
  a.ldX = ldX;
  a.P = P;
  a.ldP = ldP;
  a.codes = codes;
  a.scales = scales;
  a.hat = static_cast<uint16_t*>(hat);
  a.ldHat = ldHat;
  const int grid = codec_grid(c, rows);
  ProfScope prof(c, st, AQUAKV_KERNEL_ENCODE_ROWS);
  AQ_DISPATCH_DNB(launch_encode_rows_t, c, st, a, grid);
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

// One phase of Algorithm 3 on `rows` rows: hat = round16(P + Q^-1(codes, scales)).
int launch_decode_rows(aquakv_ctx* c, cudaStream_t st, int role, int rows, const uint8_t* codes,
                       const uint16_t* scales, const float* P, int64_t ldP, void* hat,
                       int64_t ldHat) {
  if (uniform_backbone(c))
    return launch_uniform_rows(c, st, role, rows, nullptr, 0, P, ldP, const_cast<uint8_t*>(codes),
                               const_cast<uint16_t*>(scales), hat, ldHat);
  CodecArgs a = codec_args(c, role, rows);
  a.P = P;
  a.ldP = ldP;
  a.codes = const_cast<uint8_t*>(codes);
  a.scales = const_cast<uint16_t*>(scales);
  a.hat = static_cast<uint16_t*>(hat);
  a.ldHat = ldHat;
  const int grid = codec_grid(c, rows);
  ProfScope prof(c, st, AQUAKV_KERNEL_DECODE_ROWS);
  AQ_DISPATCH_DNB(launch_decode_rows_t, c, st, a, grid);
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

int launch_attn_partial(aquakv_ctx* c, cudaStream_t st, AttnArgs a, int head_dim, int n_blocks) {
  const int rep = a.n_q_heads / a.n_kv_heads;
  const int passes = (rep + kAttnMmaMaxGq - 1) / kAttnMmaMaxGq;
  a.gq = (rep + passes - 1) / passes;
  const dim3 grid(n_blocks, a.n_kv_heads, passes);
  ProfScope prof(c, st, AQUAKV_KERNEL_ATTN);
  if (head_dim == 64) {
    if (c->bf16) attn_partial_kernel<64, true><<<grid, kAttnMmaThreads, 0, st>>>(a);
    else attn_partial_kernel<64, false><<<grid, kAttnMmaThreads, 0, st>>>(a);
  } else {
    if (c->bf16) attn_partial_kernel<128, true><<<grid, kAttnMmaThreads, 0, st>>>(a);
    else attn_partial_kernel<128, false><<<grid, kAttnMmaThreads, 0, st>>>(a);
  }
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

int launch_attn_combine(aquakv_ctx* c, cudaStream_t st, const AttnCombineArgs& a, int head_dim,
                        int batch) {
  const int grid = batch * a.n_q_heads;
  ProfScope prof(c, st, AQUAKV_KERNEL_ATTN);
  if (head_dim == 64) {
    if (c->bf16) attn_combine_kernel<64, true><<<grid, 64, 0, st>>>(a);
    else attn_combine_kernel<64, false><<<grid, 64, 0, st>>>(a);
  } else {
    if (c->bf16) attn_combine_kernel<128, true><<<grid, 128, 0, st>>>(a);
    else attn_combine_kernel<128, false><<<grid, 128, 0, st>>>(a);
  }
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// argument checks shared by the entry points
// ---------------------------------------------------------------------------------------------
int check_adapters(const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev, const void* Wk,
                   const void* Wv, const float* bk, const float* bv, int d, bool* has_pred) {
  const int n_set = (Khat_prev != nullptr) + (Vhat_prev != nullptr) + (Wk != nullptr) + (Wv != nullptr);
  if (n_set != 0 && n_set != 4) return AQUAKV_ERR_INVALID_ARG;
  *has_pred = n_set == 4;
  if (!*has_pred) {
    if (bk != nullptr || bv != nullptr) return AQUAKV_ERR_INVALID_ARG;
    return AQUAKV_OK;
  }
  if (ld_prev < d) return AQUAKV_ERR_INVALID_ARG;
  if (ld_prev % 8) return AQUAKV_ERR_ALIGNMENT;
  if (!aligned16(Khat_prev) || !aligned16(Vhat_prev) || !aligned16(Wk) || !aligned16(Wv))
    return AQUAKV_ERR_ALIGNMENT;
  if ((bk != nullptr && !aligned16(bk)) || (bv != nullptr && !aligned16(bv)))
    return AQUAKV_ERR_ALIGNMENT;
  return AQUAKV_OK;
}

int check_rows(const void* p, int64_t ld, int d, bool required) {
  if (p == nullptr) return required ? AQUAKV_ERR_INVALID_ARG : AQUAKV_OK;
  if (ld < d) return AQUAKV_ERR_INVALID_ARG;
  if (ld % 8 || !aligned16(p)) return AQUAKV_ERR_ALIGNMENT;
  return AQUAKV_OK;
}

// Packed codes are read and written as 16-byte vectors (every token's codes are a multiple of 16
// bytes), scales as 16-bit words.
int check_cache(const void* Kcodes, const void* Kscales, const void* Vcodes, const void* Vscales) {
  if (Kcodes == nullptr || Kscales == nullptr || Vcodes == nullptr || Vscales == nullptr)
    return AQUAKV_ERR_INVALID_ARG;
  if (!aligned16(Kcodes) || !aligned16(Vcodes)) return AQUAKV_ERR_ALIGNMENT;
  if ((reinterpret_cast<uintptr_t>(Kscales) & 1u) || (reinterpret_cast<uintptr_t>(Vscales) & 1u))
    return AQUAKV_ERR_ALIGNMENT;
  return AQUAKV_OK;
}

struct EncodeWs {
  size_t p_off, khat_off, total;
  int chunk;
};

EncodeWs encode_ws(const aquakv_ctx* c, int64_t T) {
  EncodeWs w;
  const int64_t t128 = int64_t(round_up(size_t(T), 128));
  w.chunk = int(t128 < c->chunk_tokens ? t128 : c->chunk_tokens);
  w.p_off = 0;
  w.khat_off = round_up(size_t(w.chunk) * c->p.d_kv * sizeof(float), 256);
  w.total = w.khat_off + round_up(size_t(w.chunk) * c->p.d_kv * 2, 256) + kWsSlack;
  return w;
}

// ---------------------------------------------------------------------------------------------
// calibration of one predictor (calib.cuh)
// ---------------------------------------------------------------------------------------------
struct FitWs {
  size_t xt_off, yt_off, g_off, c_off, gd_off, cd_off, sums_off, ridge_off, total;
  int64_t Tp;
  int n;           // input features
};

FitWs fit_ws(const aquakv_ctx* c, int64_t T, int n_inputs) {
  FitWs w;
  const size_t d = size_t(c->p.d_kv);
  w.n = int(d) * n_inputs;
  w.Tp = (T + 63) / 64 * 64;
  const size_t n = size_t(w.n);
  size_t off = 0;
  auto take = [&](size_t bytes) { const size_t o = off; off += round_up(bytes, 256); return o; };
  w.xt_off = take(n * size_t(w.Tp) * 2);
  w.yt_off = take(d * size_t(w.Tp) * 2);
  w.g_off = take(n * n * sizeof(float));
  w.c_off = take(n * d * sizeof(float));
  w.gd_off = take(n * n * sizeof(double));
  w.cd_off = take(n * d * sizeof(double));
  w.sums_off = take((n + d) * sizeof(double));
  w.ridge_off = take(sizeof(double));
  w.total = off + kWsSlack;
  return w;
}

// out[M][N] (fp32) = A B^T for token-contiguous 16-bit A [M][Tp], B [N][Tp] on the tensor cores.
int launch_gram(aquakv_ctx* c, cudaStream_t st, const void* A, int M, const void* B, int N, int64_t Tp, float* out) {
  CUtensorMap tA, tB;
  int rc = make_tmap(c, &tA, A, uint64_t(M), uint64_t(Tp), uint64_t(Tp), kBM);
  if (rc) return rc;
  if ((rc = make_tmap(c, &tB, B, uint64_t(N), uint64_t(Tp), uint64_t(Tp), kBN))) return rc;
  GemmArgs g;
  g.M = M;
  g.N = N;
  g.nk0 = int(Tp / kBK);
  g.nk1 = 0;
  g.P = out;
  g.ldP = N;
  g.bias = nullptr;
  g.status = c->d_status;
  const int tiles = (M / kBM) * (N / kBN);
  const int grid = tiles < c->sm_count ? tiles : c->sm_count;
  if (c->bf16) gemm_pred_kernel<true><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tA, tA, tB, g);
  else gemm_pred_kernel<false><<<grid, kGemmThreads, kGemmSmemBytes, st>>>(tA, tA, tB, g);
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

void launch_fit_update(aquakv_ctx* c, cudaStream_t st, double* C, long long ldc, const double* A, long long lda,
                       int transA, const double* B, long long ldb, int transB, int M, int N, int lower_only) {
  if (M <= 0 || N <= 0) return;
  const dim3 grid((N + 63) / 64, (M + 63) / 64), block(16, 16);
  fit_update_kernel<<<grid, block, 0, st>>>(C, ldc, A, lda, transA, B, ldb, transB, M, N, lower_only);
  ++c->launches;
}

// ---------------------------------------------------------------------------------------------
// fused layer kernel (predictor GEMMs + row work in one persistent launch)
// ---------------------------------------------------------------------------------------------
constexpr int kLayerRing = 3;       // prediction buffers
constexpr int kKhatRing = 3;        // waves of reconstructed keys kept when the caller wants none

struct LayerWs {
  size_t p_off, khat_off, vhat_off, flags_off, flags_bytes, total;
  int mw, n_waves, n_mblocks;
  int grid_mw;     // token-block slots the launched grid covers (>= mw)
};

LayerWs layer_ws(const aquakv_ctx* c, int64_t T, bool with_attn = false) {
  LayerWs w;
  const int d = c->p.d_kv, ntn = d / kBN;
  w.n_mblocks = int((T + kBM - 1) / kBM);
  int mw = (c->sm_count / ntn) & ~1;          // CTAs work in pairs on two token blocks
  if (mw < 2) mw = 2;
  // A call with fewer token blocks than a wave keeps its buffers small (mw shrinks) but still
  // launches the whole grid: the CTAs without a GEMM tile take their share of the row work, which is
  // what the latency of a small call consists of.
  w.grid_mw = mw;
  if (mw > w.n_mblocks) mw = (w.n_mblocks + 1) & ~1;
  w.mw = mw;
  w.n_waves = (w.n_mblocks + mw - 1) / mw;
  w.p_off = 0;
  w.khat_off = round_up(size_t(kLayerRing) * mw * kBM * d * sizeof(float), 256);
  w.vhat_off = w.khat_off + round_up(size_t(kKhatRing) * mw * kBM * d * 2, 256);
  w.flags_off = with_attn ? w.vhat_off + round_up(size_t(kKhatRing) * mw * kBM * d * 2, 256) : w.vhat_off;
  w.flags_bytes = size_t(with_attn ? 5 : 4) * w.n_waves * mw * sizeof(int);   // gemm_done, rows_done (two jobs per wave each), attn_done
  w.total = w.flags_off + round_up(w.flags_bytes, 256) + kWsSlack;
  return w;
}

struct AttnWs {
  size_t layer_off, khat_off, vhat_off, ml_off, o_off, total;
  int chunk_blocks;     // split-KV blocks per chunk (two-kernel path)
  int n_splits;         // partial slots per sequence
  bool fused;           // decode and attention in one launch of the layer kernel
};

bool fused_attn_supported(const aquakv_ctx* c);

// Workspace of aquakv_decode_attn.  In the fused mode (aquakv_set_attn_mode), with predictors at
// d_kv = 1024 (Hadamard block = scale group = the row), decode and attention are ONE launch of the
// layer kernel: the workspace holds that kernel's buffers (prediction ring, rings of three waves of
// decoded keys / values, counters) and the attention partials, one slot per 128-token block that
// overlaps a sequence.  Otherwise the cache is decoded chunk by chunk, about 32 waves each, into the
// workspace (or the caller's Khat/Vhat) and a separate kernel attends over each chunk in blocks of
// 1024 tokens.
AttnWs attn_ws(const aquakv_ctx* c, int32_t batch, int64_t ctx_len, int32_t n_q_heads,
               int32_t head_dim, bool want_fused) {
  AttnWs w;
  const size_t d = size_t(c->p.d_kv);
  w.fused = want_fused && fused_attn_supported(c);
  if (w.fused) {
    w.n_splits = int((ctx_len + kAttnSubTokens - 2) / kAttnSubTokens) + 1;   // sub-blocks of the flattened token
                                                                             // index a sequence can overlap
    w.chunk_blocks = 0;
    const int64_t slots = int64_t(batch) * w.n_splits;
    w.layer_off = 0;
    w.khat_off = w.vhat_off = 0;
    w.ml_off = round_up(layer_ws(c, int64_t(batch) * ctx_len, true).total, 256);
    w.o_off = w.ml_off + round_up(size_t(slots) * n_q_heads * 2 * sizeof(float), 256);
    w.total = w.o_off + round_up(size_t(slots) * n_q_heads * head_dim * sizeof(float), 256) + kWsSlack;
    return w;
  }
  const int tb = c->attn_block_tokens;
  w.n_splits = int((ctx_len + tb - 1) / tb);
  const int wave_tokens = (c->sm_count / int(d / kBN) > 0 ? c->sm_count / int(d / kBN) : 1) * kBM;
  int cb = 32 * wave_tokens / tb;
  if (cb < 1) cb = 1;
  const int64_t total_blocks = int64_t(batch) * w.n_splits;
  if (cb > total_blocks) cb = int(total_blocks);
  w.chunk_blocks = cb;
  const size_t chunk_rows = size_t(cb) * tb;
  const size_t phase_bytes = round_up(chunk_rows * d * sizeof(float), 256);   // separate-kernel path
  const size_t layer_bytes = layer_ws(c, int64_t(chunk_rows)).total;
  w.layer_off = 0;
  w.khat_off = phase_bytes > layer_bytes ? phase_bytes : layer_bytes;
  w.vhat_off = w.khat_off + round_up(chunk_rows * d * 2, 256);
  w.ml_off = w.vhat_off + round_up(chunk_rows * d * 2, 256);
  w.o_off = w.ml_off + round_up(size_t(total_blocks) * n_q_heads * 2 * sizeof(float), 256);
  w.total = w.o_off + round_up(size_t(total_blocks) * n_q_heads * head_dim * sizeof(float), 256) + kWsSlack;
  return w;
}

template <bool ENC, int D, int NPTS, bool BF, bool FULL, int AHD, int NB>
int launch_layer_t(int device, cudaStream_t st, int grid, const LayerBatch<NB>& B) {
  // the shared-memory opt-in is a per-device attribute of the function: one bit per device and
  // instantiation (setting it twice from two threads is harmless)
  static std::atomic<unsigned long long> attr_devices{0};
  constexpr size_t smem = layer_smem_bytes<ENC, D, NPTS, FULL>();
  const unsigned long long bit = 1ull << (device & 63);
  if (device >= 64 || !(attr_devices.load(std::memory_order_acquire) & bit)) {
    if (cudaFuncSetAttribute(layer_kernel<ENC, D, NPTS, BF, FULL, AHD, NB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             int(smem)) != cudaSuccess)
      return AQUAKV_ERR_CUDA;
    if (device < 64) attr_devices.fetch_or(bit, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(unsigned(grid));
  cfg.blockDim = dim3(unsigned(layer_threads<ENC, D, FULL, AHD>()));
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  // The CTAs of this kernel wait for one another, so all CTA pairs of the grid must fit the device at
  // once (asked once per device and instantiation; an idle device is assumed, see the header).
  static std::atomic<unsigned long long> fits_devices{0};
  if (device >= 64 || !(fits_devices.load(std::memory_order_acquire) & bit)) {
    int max_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&max_clusters, layer_kernel<ENC, D, NPTS, BF, FULL, AHD, NB>, &cfg) != cudaSuccess)
      return AQUAKV_ERR_CUDA;
    if (max_clusters * 2 < grid) return AQUAKV_ERR_UNSUPPORTED;
    if (device < 64) fits_devices.fetch_or(bit, std::memory_order_release);
  }
  return cudaLaunchKernelEx(&cfg, layer_kernel<ENC, D, NPTS, BF, FULL, AHD, NB>, B) == cudaSuccess ? AQUAKV_OK
                                                                                                      : AQUAKV_ERR_CUDA;
}
// Launches of several layers exist for the paper's main setting only (d_kv = 1024, Hadamard block = scale
// group = the row); everything else runs layer by layer.
template <int D, int NPTS, bool BF, int NB>
void launch_layer_enc_t(int* rc, int device, cudaStream_t st, int grid, const LayerBatch<NB>& B) {
  // Hadamard block = scale group = the whole row: the encoder has an instantiation with those sizes
  // fixed at compile time (measured 8-10 % faster; the decoder measured no gain and has none)
  const LayerArgs& a = B.layer[0];
  const bool full = a.log_h == a.log_g && (1 << a.log_h) == D;
  if constexpr (NB > 1) {
    if constexpr (D == 1024) {
      *rc = full ? launch_layer_t<true, D, NPTS, BF, true, 0, NB>(device, st, grid, B) : AQUAKV_ERR_UNSUPPORTED;
    } else {
      *rc = AQUAKV_ERR_UNSUPPORTED;
    }
  } else {
    *rc = full ? launch_layer_t<true, D, NPTS, BF, true, 0, NB>(device, st, grid, B)
               : launch_layer_t<true, D, NPTS, BF, false, 0, NB>(device, st, grid, B);
  }
}
template <int D, int NPTS, bool BF, int NB>
void launch_layer_dec_t(int* rc, int device, cudaStream_t st, int grid, const LayerBatch<NB>& B) {
  // the decoder has the fixed-size instantiation only where it selects the one-warp-per-row routines
  const LayerArgs& a = B.layer[0];
  if constexpr (D == 1024) {
    if (a.log_h == 10 && a.log_g == 10) {
      if (a.q != nullptr) {       // decode + single-query attention in one kernel
        *rc = a.n_kv_heads * 128 == D ? launch_layer_t<false, D, NPTS, BF, true, 128, NB>(device, st, grid, B)
                                      : launch_layer_t<false, D, NPTS, BF, true, 64, NB>(device, st, grid, B);
        return;
      }
      *rc = launch_layer_t<false, D, NPTS, BF, true, 0, NB>(device, st, grid, B);
      return;
    }
  }
  if constexpr (NB > 1) {
    *rc = AQUAKV_ERR_UNSUPPORTED;
  } else {
    *rc = a.q != nullptr ? AQUAKV_ERR_UNSUPPORTED : launch_layer_t<false, D, NPTS, BF, false, 0, NB>(device, st, grid, B);
  }
}

// The attention a decode launch also computes (the attention read of Algorithm 4); q == nullptr: none.
struct LayerAttnArgs {
  const void* q;
  int ctx, n_q_heads, n_kv_heads, n_splits;
  float scale_log2;
  float* part_ml;
  float* part_o;
};

// True if decode + attention runs as one launch of the layer kernel for this context.
bool fused_attn_supported(const aquakv_ctx* c) { return c->p.d_kv == 1024 && c->log_h == 10 && c->log_g == 10; }

// Arguments and tensor maps of one layer of a launch.  `flags` is the layer's counter block (gemm_done,
// rows_done and, with attention, attn_done; zero at launch), `P` the prediction ring.
int fill_layer(aquakv_ctx* c, const LayerWs& ws, uint8_t* wsb, int* flags, int64_t T, const void* K, const void* V,
               int64_t ld_kv, const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev, const void* Wk,
               const void* Wv, const float* bk, const float* bv, uint8_t* Kcodes, uint16_t* Kscales, uint8_t* Vcodes,
               uint16_t* Vscales, void* Khat, void* Vhat, int64_t ld_hat, const LayerAttnArgs* attn, LayerArgs* out,
               LayerMaps* maps) {
  const int d = c->p.d_kv;
  LayerArgs& a = *out;
  std::memset(&a, 0, sizeof(a));
  a.T = int(T);
  a.n_mblocks = ws.n_mblocks;
  a.mw = ws.mw;
  a.n_waves = ws.n_waves;
  a.nb = kLayerRing;
  a.bk = bk;
  a.bv = bv;
  a.P = reinterpret_cast<float*>(wsb + ws.p_off);
  a.gemm_done = flags;
  a.rows_done = a.gemm_done + size_t(2) * ws.n_waves * ws.mw;
  a.K = static_cast<const uint16_t*>(K);
  a.V = static_cast<const uint16_t*>(V);
  a.ldX = ld_kv;
  a.Kcodes = Kcodes;
  a.Kscales = Kscales;
  a.Vcodes = Vcodes;
  a.Vscales = Vscales;
  if (Khat != nullptr) {
    a.khat_ring = 0;
    a.Khat = static_cast<uint16_t*>(Khat);
    a.ldKhat = ld_hat;
  } else {
    a.khat_ring = kKhatRing;
    a.Khat = reinterpret_cast<uint16_t*>(wsb + ws.khat_off);
    a.ldKhat = d;
  }
  a.Vhat = static_cast<uint16_t*>(Vhat);
  a.ldVhat = ld_hat;
  if (attn != nullptr) {
    if (Vhat == nullptr) {       // decoded values the caller does not want: a ring like the keys'
      a.vhat_ring = kKhatRing;
      a.Vhat = reinterpret_cast<uint16_t*>(wsb + ws.vhat_off);
      a.ldVhat = d;
    }
    a.q = static_cast<const uint16_t*>(attn->q);
    a.ctx = attn->ctx;
    a.n_q_heads = attn->n_q_heads;
    a.n_kv_heads = attn->n_kv_heads;
    a.n_splits = attn->n_splits;
    a.scale_log2 = attn->scale_log2;
    a.part_ml = attn->part_ml;
    a.part_o = attn->part_o;
    a.attn_done = a.rows_done + size_t(2) * ws.n_waves * ws.mw;
  }
  a.signmask_k = c->d_signmask[kRoleK];
  a.signmask_v = c->d_signmask[kRoleV];
  const CodecArgs ca = codec_args(c, kRoleK, 0);
  a.grid4 = ca.grid4;
  a.search = ca.search;
  a.log_h = c->log_h;
  a.log_g = c->log_g;
  a.status = c->d_status;
  {
    // the prediction ring as a 2-D fp32 tensor for the epilogue's TMA stores (32 x 32 boxes)
    const cuuint64_t dims[2] = {cuuint64_t(d), cuuint64_t(kLayerRing) * ws.mw * kBM};
    const cuuint64_t strides[1] = {cuuint64_t(d) * sizeof(float)};
    const cuuint32_t box[2] = {32, 32};
    const cuuint32_t estr[2] = {1, 1};
    if (c->encode_tiled(&maps->p, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, a.P, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return AQUAKV_ERR_CUDA;
  }
  int rc = make_tmap(c, &maps->kprev, Khat_prev, uint64_t(T), uint64_t(d), uint64_t(ld_prev), kBM);
  if (rc) return rc;
  if ((rc = make_tmap(c, &maps->vprev, Vhat_prev, uint64_t(T), uint64_t(d), uint64_t(ld_prev), kBM))) return rc;
  const uint64_t khat_rows = a.khat_ring ? uint64_t(kKhatRing) * ws.mw * kBM : uint64_t(T);
  if ((rc = make_tmap(c, &maps->khat, a.Khat, khat_rows, uint64_t(d), uint64_t(a.ldKhat), kBM))) return rc;
  // weight tiles are fetched half (128 rows) per CTA of a pair
  if ((rc = make_tmap(c, &maps->wk, Wk, uint64_t(d), uint64_t(d), uint64_t(d), kBN / 2))) return rc;
  return make_tmap(c, &maps->wv, Wv, uint64_t(d), uint64_t(2) * d, uint64_t(2) * d, kBN / 2);
}

// Algorithm 2 (encode = true) or Algorithm 3 for one layer with predictors, all tokens, one launch.
int launch_layer(aquakv_ctx* c, cudaStream_t st, bool encode, int64_t T, const void* K, const void* V,
                 int64_t ld_kv, const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev,
                 const void* Wk, const void* Wv, const float* bk, const float* bv, uint8_t* Kcodes,
                 uint16_t* Kscales, uint8_t* Vcodes, uint16_t* Vscales, void* Khat, void* Vhat,
                 int64_t ld_hat, void* workspace, const LayerAttnArgs* attn = nullptr) {
  const int d = c->p.d_kv;
  const LayerWs ws = layer_ws(c, T, attn != nullptr);
  uint8_t* wsb = ws_base(workspace);
  LayerBatch<1> B;
  B.n_layers = 1;
  int rc = fill_layer(c, ws, wsb, reinterpret_cast<int*>(wsb + ws.flags_off), T, K, V, ld_kv, Khat_prev, Vhat_prev,
                      ld_prev, Wk, Wv, bk, bv, Kcodes, Kscales, Vcodes, Vscales, Khat, Vhat, ld_hat, attn, &B.layer[0],
                      &B.maps[0]);
  if (rc) return rc;
  if (cudaMemsetAsync(B.layer[0].gemm_done, 0, ws.flags_bytes, st) != cudaSuccess) return AQUAKV_ERR_CUDA;
  const int grid = ws.grid_mw * (d / kBN);
  ProfScope prof(c, st, AQUAKV_KERNEL_LAYER);
  if (encode) {
    AQ_DISPATCH_DNB(launch_layer_enc_t, &rc, c->device, st, grid, B);
  } else {
    AQ_DISPATCH_DNB(launch_layer_dec_t, &rc, c->device, st, grid, B);
  }
  if (rc) return rc;
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// chain kernel (all layers of a small call in one persistent launch)
// ---------------------------------------------------------------------------------------------
constexpr int64_t kChainMaxTokens = 2048;

struct ChainWs {
  size_t pk_off, pv_off, cnt_off, cnt_bytes, hat_off, hat_bytes, total;
};

ChainWs chain_ws(const aquakv_ctx* c, int64_t T, int L) {
  ChainWs w;
  const size_t d = size_t(c->p.d_kv);
  const size_t n_mt = size_t((T + kChainMT - 1) / kChainMT);
  w.pk_off = 0;
  w.pv_off = round_up(size_t(T) * d * sizeof(float), 256);
  w.cnt_off = w.pv_off + round_up(size_t(T) * d * sizeof(float), 256);
  w.cnt_bytes = size_t(4) * L * n_mt * sizeof(int);
  w.hat_off = w.cnt_off + round_up(w.cnt_bytes, 256);
  w.hat_bytes = round_up(size_t(T) * d * 2, 256);           // one layer's K^ or V^
  w.total = w.hat_off + size_t(2) * L * w.hat_bytes + kWsSlack;
  return w;
}

template <bool ENC, int D, int NPTS, bool BF, bool WROWS>
int launch_chain_t(int device, cudaStream_t st, int grid, const ChainArgs& a) {
  static std::atomic<unsigned long long> attr_devices{0};
  constexpr size_t smem = sizeof(ChainSmem<D, NPTS, ENC, WROWS>);
  const unsigned long long bit = 1ull << (device & 63);
  if (device >= 64 || !(attr_devices.load(std::memory_order_acquire) & bit)) {
    if (cudaFuncSetAttribute(chain_kernel<ENC, D, NPTS, BF, WROWS>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) !=
        cudaSuccess)
      return AQUAKV_ERR_CUDA;
    if (device < 64) attr_devices.fetch_or(bit, std::memory_order_release);
  }
  // all CTAs wait for one another: one per SM must fit (asked once per device and instantiation)
  static std::atomic<unsigned long long> fits_devices{0};
  if (device >= 64 || !(fits_devices.load(std::memory_order_acquire) & bit)) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, chain_kernel<ENC, D, NPTS, BF, WROWS>, kChainThreads, smem) !=
        cudaSuccess)
      return AQUAKV_ERR_CUDA;
    if (per_sm < 1) return AQUAKV_ERR_UNSUPPORTED;
    if (device < 64) fits_devices.fetch_or(bit, std::memory_order_release);
  }
  chain_kernel<ENC, D, NPTS, BF, WROWS><<<grid, kChainThreads, smem, st>>>(a);
  return AQUAKV_OK;
}
template <int D, int NPTS, bool BF>
void launch_chain_dnb(int* rc, bool encode, int device, cudaStream_t st, int grid, const ChainArgs& a) {
  // one warp per row once the teams of four warps no longer cover every row of a layer at once
  if constexpr (D == 1024) {
    const bool warp_rows = 2 * a.T > grid * (kChainWarps / RowTeam<D>::TEAM);
    if (warp_rows) {
      *rc = encode ? launch_chain_t<true, D, NPTS, BF, true>(device, st, grid, a)
                   : launch_chain_t<false, D, NPTS, BF, true>(device, st, grid, a);
      return;
    }
  }
  *rc = encode ? launch_chain_t<true, D, NPTS, BF, false>(device, st, grid, a)
               : launch_chain_t<false, D, NPTS, BF, false>(device, st, grid, a);
}

// ---------------------------------------------------------------------------------------------
// Several layers of a LARGE call per launch of the layer kernel (the chain entry points beyond the
// chain kernel's token limit): layers without predictors run through the per-layer row kernels, runs
// of predicted layers go to the layer kernel kLayerBatchMax at a time.
// ---------------------------------------------------------------------------------------------
struct LayersWs {
  LayerWs layer;
  size_t flags_off, flags_stride, total;
};
LayersWs layers_ws(const aquakv_ctx* c, int64_t T, int L) {
  LayersWs w;
  w.layer = layer_ws(c, T);
  const int nb = L < kLayerBatchMax ? (L > 0 ? L : 1) : kLayerBatchMax;
  w.flags_stride = round_up(w.layer.flags_bytes, 256);
  w.flags_off = round_up(w.layer.total, 256);
  w.total = w.flags_off + size_t(nb) * w.flags_stride + kWsSlack;
  return w;
}

bool layers_supported(const aquakv_ctx* c) { return c->p.d_kv == 1024 && c->log_h == 10 && c->log_g == 10 && !uniform_backbone(c); }

int run_layers(aquakv_ctx* c, bool encode, int64_t T, int32_t L, const void* const* K, const void* const* V,
               int64_t ld_kv, const void* Khat_init, const void* Vhat_init, int64_t ld_init, const void* const* Wk,
               const void* const* Wv, const float* const* bk, const float* const* bv, uint8_t* const* Kcodes,
               uint16_t* const* Kscales, uint8_t* const* Vcodes, uint16_t* const* Vscales, void* const* Khat,
               void* const* Vhat, int64_t ld_hat, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!layers_supported(c)) return AQUAKV_ERR_TOO_LARGE;
  if (T > (int64_t(1) << 30)) return AQUAKV_ERR_UNSUPPORTED;
  const int d = c->p.d_kv;
  if (Wk == nullptr || Wv == nullptr || Kcodes == nullptr || Kscales == nullptr || Vcodes == nullptr || Vscales == nullptr ||
      Khat == nullptr || Vhat == nullptr)
    return AQUAKV_ERR_INVALID_ARG;
  if (encode && (K == nullptr || V == nullptr)) return AQUAKV_ERR_INVALID_ARG;
  int rc;
  for (int l = 0; l < L; ++l) {
    if ((rc = check_cache(Kcodes[l], Kscales[l], Vcodes[l], Vscales[l]))) return rc;
    if (encode) {
      if ((rc = check_rows(K[l], ld_kv, d, true))) return rc;
      if ((rc = check_rows(V[l], ld_kv, d, true))) return rc;
    }
    if ((Wk[l] == nullptr) != (Wv[l] == nullptr)) return AQUAKV_ERR_INVALID_ARG;
    if (Wk[l] != nullptr && (!aligned16(Wk[l]) || !aligned16(Wv[l]))) return AQUAKV_ERR_ALIGNMENT;
    const float* b0 = bk ? bk[l] : nullptr;
    const float* b1 = bv ? bv[l] : nullptr;
    if (Wk[l] == nullptr && (b0 != nullptr || b1 != nullptr)) return AQUAKV_ERR_INVALID_ARG;
    if ((b0 != nullptr && !aligned16(b0)) || (b1 != nullptr && !aligned16(b1))) return AQUAKV_ERR_ALIGNMENT;
    if ((rc = check_rows(Khat[l], ld_hat, d, true))) return rc;
    if ((rc = check_rows(Vhat[l], ld_hat, d, true))) return rc;
    if (Khat[l] == Vhat[l] || (encode && (Khat[l] == K[l] || Khat[l] == V[l] || Vhat[l] == K[l] || Vhat[l] == V[l])))
      return AQUAKV_ERR_INVALID_ARG;
    // a layer reads the reconstructions of the layer before it while it writes its own
    const void* pk = l == 0 ? Khat_init : Khat[l - 1];
    const void* pv = l == 0 ? Vhat_init : Vhat[l - 1];
    if (Wk[l] != nullptr) {
      if (pk == nullptr || pv == nullptr) return AQUAKV_ERR_INVALID_ARG;
      if (Khat[l] == pk || Khat[l] == pv || Vhat[l] == pk || Vhat[l] == pv) return AQUAKV_ERR_INVALID_ARG;
    }
  }
  if (Wk[0] != nullptr) {
    if ((rc = check_rows(Khat_init, ld_init, d, true))) return rc;
    if ((rc = check_rows(Vhat_init, ld_init, d, true))) return rc;
  } else if (Khat_init != nullptr || Vhat_init != nullptr) {
    return AQUAKV_ERR_INVALID_ARG;
  }
  const LayersWs ws = layers_ws(c, T, L);
  if (workspace == nullptr || workspace_bytes < ws.total) return AQUAKV_ERR_WORKSPACE;
  if (!aligned16(workspace)) return AQUAKV_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* wsb = ws_base(workspace);
  const int grid = ws.layer.grid_mw * (d / kBN);
  int l = 0;
  while (l < L) {
    if (Wk[l] == nullptr) {
      // no predictor: the row kernels alone
      const int cb = c->code_bytes, ng = c->n_groups;
      const int64_t chunk = int64_t(1) << 30;
      for (int64_t t0 = 0; t0 < T; t0 += chunk) {
        const int rows = int(T - t0 < chunk ? T - t0 : chunk);
        uint16_t* kh = static_cast<uint16_t*>(Khat[l]) + t0 * ld_hat;
        uint16_t* vh = static_cast<uint16_t*>(Vhat[l]) + t0 * ld_hat;
        if (encode) {
          rc = launch_encode_rows(c, st, kRoleK, rows, static_cast<const uint16_t*>(K[l]) + t0 * ld_kv, ld_kv, nullptr, d,
                                  Kcodes[l] + t0 * cb, Kscales[l] + t0 * ng, kh, ld_hat);
          if (rc) return rc;
          rc = launch_encode_rows(c, st, kRoleV, rows, static_cast<const uint16_t*>(V[l]) + t0 * ld_kv, ld_kv, nullptr, d,
                                  Vcodes[l] + t0 * cb, Vscales[l] + t0 * ng, vh, ld_hat);
        } else {
          rc = launch_decode_rows(c, st, kRoleK, rows, Kcodes[l] + t0 * cb, Kscales[l] + t0 * ng, nullptr, d, kh, ld_hat);
          if (rc) return rc;
          rc = launch_decode_rows(c, st, kRoleV, rows, Vcodes[l] + t0 * cb, Vscales[l] + t0 * ng, nullptr, d, vh, ld_hat);
        }
        if (rc) return rc;
      }
      ++l;
      continue;
    }
    // a run of predicted layers, at most kLayerBatchMax per launch
    int n = 0;
    while (l + n < L && n < kLayerBatchMax && Wk[l + n] != nullptr) ++n;
    static thread_local LayerBatch<kLayerBatchMax> B;      // 26 KB: not on the stack of a caller's thread
    B.n_layers = n;
    for (int i = 0; i < n; ++i) {
      const int li = l + i;
      const void* pk = li == 0 ? Khat_init : Khat[li - 1];
      const void* pv = li == 0 ? Vhat_init : Vhat[li - 1];
      const int64_t ldp = li == 0 ? ld_init : ld_hat;
      rc = fill_layer(c, ws.layer, wsb, reinterpret_cast<int*>(wsb + ws.flags_off + size_t(i) * ws.flags_stride), T,
                      encode ? K[li] : nullptr, encode ? V[li] : nullptr, ld_kv, pk, pv, ldp, Wk[li], Wv[li],
                      bk ? bk[li] : nullptr, bv ? bv[li] : nullptr, Kcodes[li], Kscales[li], Vcodes[li], Vscales[li],
                      Khat[li], Vhat[li], ld_hat, nullptr, &B.layer[i], &B.maps[i]);
      if (rc) return rc;
    }
    if (cudaMemsetAsync(wsb + ws.flags_off, 0, size_t(n) * ws.flags_stride, st) != cudaSuccess) return AQUAKV_ERR_CUDA;
    {
      ProfScope prof(c, st, AQUAKV_KERNEL_LAYER);
      if (encode) {
        AQ_DISPATCH_DNB(launch_layer_enc_t, &rc, c->device, st, grid, B);
      } else {
        AQ_DISPATCH_DNB(launch_layer_dec_t, &rc, c->device, st, grid, B);
      }
    }
    if (rc) return rc;
    ++c->launches;
    if (cudaGetLastError() != cudaSuccess) return AQUAKV_ERR_CUDA;
    l += n;
  }
  return AQUAKV_OK;
}

// Algorithm 2 (encode) or Algorithm 3 for n_layers layers in one launch; argument checks included.
int run_chain(aquakv_ctx* c, bool encode, int64_t T, int32_t L, const void* const* K, const void* const* V,
              int64_t ld_kv, const void* Khat_init, const void* Vhat_init, int64_t ld_init, const void* const* Wk,
              const void* const* Wv, const float* const* bk, const float* const* bv, uint8_t* const* Kcodes,
              uint16_t* const* Kscales, uint8_t* const* Vcodes, uint16_t* const* Vscales, void* const* Khat,
              void* const* Vhat, int64_t ld_hat, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (c != nullptr && uniform_backbone(c)) return AQUAKV_ERR_UNSUPPORTED;   // per-layer entry points only
  if (c == nullptr || T < 0 || L < 0) return AQUAKV_ERR_INVALID_ARG;
  if (T == 0 || L == 0) return AQUAKV_OK;
  if (L > kChainMaxLayers) return AQUAKV_ERR_TOO_LARGE;
  if (T > kChainMaxTokens)      // beyond the chain kernel: launches of the layer kernel that take several layers each
    return run_layers(c, encode, T, L, K, V, ld_kv, Khat_init, Vhat_init, ld_init, Wk, Wv, bk, bv, Kcodes, Kscales, Vcodes,
                      Vscales, Khat, Vhat, ld_hat, workspace, workspace_bytes, cuda_stream);
  const int d = c->p.d_kv;
  if (d == 1024 && !(c->log_h == 10 && c->log_g == 10)) return AQUAKV_ERR_UNSUPPORTED;
  if (Wk == nullptr || Wv == nullptr || Kcodes == nullptr || Kscales == nullptr || Vcodes == nullptr || Vscales == nullptr)
    return AQUAKV_ERR_INVALID_ARG;
  if (encode && (K == nullptr || V == nullptr)) return AQUAKV_ERR_INVALID_ARG;
  int rc;
  const ChainWs ws = chain_ws(c, T, L);
  bool any_hat = false;
  for (int l = 0; l < L; ++l) {
    if ((rc = check_cache(Kcodes[l], Kscales[l], Vcodes[l], Vscales[l]))) return rc;
    if (encode) {
      if ((rc = check_rows(K[l], ld_kv, d, true))) return rc;
      if ((rc = check_rows(V[l], ld_kv, d, true))) return rc;
    }
    if ((Wk[l] == nullptr) != (Wv[l] == nullptr)) return AQUAKV_ERR_INVALID_ARG;
    if (Wk[l] != nullptr && (!aligned16(Wk[l]) || !aligned16(Wv[l]))) return AQUAKV_ERR_ALIGNMENT;
    const float* b0 = bk ? bk[l] : nullptr;
    const float* b1 = bv ? bv[l] : nullptr;
    if (Wk[l] == nullptr && (b0 != nullptr || b1 != nullptr)) return AQUAKV_ERR_INVALID_ARG;
    if ((b0 != nullptr && !aligned16(b0)) || (b1 != nullptr && !aligned16(b1))) return AQUAKV_ERR_ALIGNMENT;
    const void* kh = Khat ? Khat[l] : nullptr;
    const void* vh = Vhat ? Vhat[l] : nullptr;
    if ((rc = check_rows(kh, ld_hat, d, false))) return rc;
    if ((rc = check_rows(vh, ld_hat, d, false))) return rc;
    if (kh != nullptr && (kh == vh || (encode && (kh == K[l] || kh == V[l])))) return AQUAKV_ERR_INVALID_ARG;
    any_hat = any_hat || kh != nullptr || vh != nullptr;
  }
  if (Wk[0] != nullptr) {
    if ((rc = check_rows(Khat_init, ld_init, d, true))) return rc;
    if ((rc = check_rows(Vhat_init, ld_init, d, true))) return rc;
  } else if (Khat_init != nullptr || Vhat_init != nullptr) {
    return AQUAKV_ERR_INVALID_ARG;
  }
  if (workspace == nullptr || workspace_bytes < ws.total) return AQUAKV_ERR_WORKSPACE;
  if (!aligned16(workspace)) return AQUAKV_ERR_ALIGNMENT;
  (void)any_hat;

  uint8_t* wsb = ws_base(workspace);
  ChainArgs a;
  std::memset(&a, 0, sizeof(a));
  a.T = int(T);
  a.L = L;
  a.ldX = ld_kv;
  a.Khat_init = static_cast<const uint16_t*>(Khat_init);
  a.Vhat_init = static_cast<const uint16_t*>(Vhat_init);
  a.ldInit = ld_init;
  a.Pk = reinterpret_cast<float*>(wsb + ws.pk_off);
  a.Pv = reinterpret_cast<float*>(wsb + ws.pv_off);
  a.counters = reinterpret_cast<int*>(wsb + ws.cnt_off);
  a.signmask_k = c->d_signmask[kRoleK];
  a.signmask_v = c->d_signmask[kRoleV];
  const CodecArgs ca = codec_args(c, kRoleK, 0);
  a.grid4 = ca.grid4;
  a.search = ca.search;
  a.log_h = c->log_h;
  a.log_g = c->log_g;
  a.status = c->d_status;
  for (int l = 0; l < L; ++l) {
    ChainLayer& y = a.layer[l];
    y.K = encode ? static_cast<const uint16_t*>(K[l]) : nullptr;
    y.V = encode ? static_cast<const uint16_t*>(V[l]) : nullptr;
    y.Wk = static_cast<const uint16_t*>(Wk[l]);
    y.Wv = static_cast<const uint16_t*>(Wv[l]);
    y.bk = bk ? bk[l] : nullptr;
    y.bv = bv ? bv[l] : nullptr;
    y.Kcodes = Kcodes[l];
    y.Kscales = Kscales[l];
    y.Vcodes = Vcodes[l];
    y.Vscales = Vscales[l];
    void* kh = Khat ? Khat[l] : nullptr;
    void* vh = Vhat ? Vhat[l] : nullptr;
    // the K and V reconstructions of a layer share ld: both the caller's or both the workspace's
    if ((kh == nullptr) != (vh == nullptr)) return AQUAKV_ERR_INVALID_ARG;
    if (kh != nullptr) {
      y.Khat = static_cast<uint16_t*>(kh);
      y.Vhat = static_cast<uint16_t*>(vh);
      y.ldHat = ld_hat;
    } else {
      y.Khat = reinterpret_cast<uint16_t*>(wsb + ws.hat_off + size_t(2 * l) * ws.hat_bytes);
      y.Vhat = reinterpret_cast<uint16_t*>(wsb + ws.hat_off + size_t(2 * l + 1) * ws.hat_bytes);
      y.ldHat = d;
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(a.counters, 0, ws.cnt_bytes, st) != cudaSuccess) return AQUAKV_ERR_CUDA;
  const int grid = c->sm_count;
  a.n_ctas_k = grid * 2 / 5 > 0 ? grid * 2 / 5 : 1;
  if (grid < 2) return AQUAKV_ERR_UNSUPPORTED;
  ProfScope prof(c, st, AQUAKV_KERNEL_CHAIN);
  AQ_DISPATCH_DNB(launch_chain_dnb, &rc, encode, c->device, st, grid, a);
  if (rc) return rc;
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

}  // namespace

// =============================================================================================
// C ABI
// =============================================================================================
extern "C" {

int aquakv_code_bytes(const aquakv_params* params) {
  const int rc = check_params(params);
  if (rc) return rc;
  return params->d_kv / params->grid_dim * ilog2(params->grid_size) / 8;
}

const char* aquakv_status_string(int status) {
  switch (status) {
    case AQUAKV_OK: return "ok";
    case AQUAKV_ERR_INVALID_ARG: return "invalid argument";
    case AQUAKV_ERR_UNSUPPORTED: return "unsupported parameter combination";
    case AQUAKV_ERR_ALIGNMENT: return "misaligned pointer or leading dimension";
    case AQUAKV_ERR_WORKSPACE: return "workspace missing or too small";
    case AQUAKV_ERR_CUDA: return "CUDA call failed";
    case AQUAKV_ERR_TIMEOUT: return "bounded device-side wait expired";
    case AQUAKV_ERR_TOO_LARGE: return "more tokens than the fixed scratch of the no-allocation call holds";
    case AQUAKV_ERR_NUMERIC: return "normal equations of a fit not positive definite";
    default: return "unknown status";
  }
}

int aquakv_search_table_host(const float* grid_host, int32_t grid_size, int32_t* cells_per_side,
                             float* half_extent, uint32_t* table, size_t table_capacity,
                             int32_t* second_level_lists) {
  if (grid_host == nullptr || cells_per_side == nullptr || half_extent == nullptr)
    return AQUAKV_ERR_INVALID_ARG;
  if (grid_size != 16 && grid_size != 64 && grid_size != 256) return AQUAKV_ERR_UNSUPPORTED;
  for (int i = 0; i < 2 * grid_size; ++i)
    if (!std::isfinite(grid_host[i])) return AQUAKV_ERR_INVALID_ARG;
  const SearchTableSpec spec = search_table_spec(grid_host, grid_size);
  *cells_per_side = spec.cells;
  *half_extent = spec.half;
  if (table == nullptr) return AQUAKV_OK;
  if (table_capacity < search_table_words(spec)) return AQUAKV_ERR_INVALID_ARG;
  const int n_lists = build_search_table(grid_host, grid_size, spec, table);
  if (second_level_lists != nullptr) *second_level_lists = n_lists;
  return AQUAKV_OK;
}

int aquakv_create(const aquakv_params* params, const float* grid_host, const int8_t* signs_k_host,
                  const int8_t* signs_v_host, aquakv_ctx** out) {
  if (out == nullptr) return AQUAKV_ERR_INVALID_ARG;
  *out = nullptr;
  int rc = check_params(params);
  if (rc) return rc;
  const bool uniform = params->grid_dim == 1;      // its levels are implied: the grid is not read
  const bool rotated = !uniform || params->had_block > 1;   // the signs are read
  if (!uniform && grid_host == nullptr) return AQUAKV_ERR_INVALID_ARG;
  if (rotated && (signs_k_host == nullptr || signs_v_host == nullptr)) return AQUAKV_ERR_INVALID_ARG;
  const int d = params->d_kv, n = params->grid_size, gdim = params->grid_dim;
  if (!uniform)
    for (int i = 0; i < gdim * n; ++i)
      if (!std::isfinite(grid_host[i])) return AQUAKV_ERR_INVALID_ARG;
  if (rotated) {
    for (int i = 0; i < d; ++i) {
      if (signs_k_host[i] != 1 && signs_k_host[i] != -1) return AQUAKV_ERR_INVALID_ARG;
      if (signs_v_host[i] != 1 && signs_v_host[i] != -1) return AQUAKV_ERR_INVALID_ARG;
    }
  }
  aquakv_ctx* c = new (std::nothrow) aquakv_ctx();
  if (c == nullptr) return AQUAKV_ERR_CUDA;
  std::memset(c, 0, sizeof(*c));
  c->p = *params;
  c->log_h = ilog2(params->had_block);
  c->log_g = ilog2(params->scale_group);
  c->bits = ilog2(n);
  c->code_bytes = d / gdim * c->bits / 8;
  c->n_groups = d / params->scale_group;
  c->bf16 = params->dtype == AQUAKV_BF16;
  c->attn_block_tokens = 1024;

  float4 g4[256];
  std::memset(g4, 0, sizeof(g4));
  std::vector<uint32_t> table(4, 0u);
  if (gdim == 4) {
    for (int i = 0; i < n; ++i)
      g4[i] = make_float4(grid_host[4 * i], grid_host[4 * i + 1], grid_host[4 * i + 2], grid_host[4 * i + 3]);
  } else if (!uniform) {
    for (int i = 0; i < n; ++i) {
      const float gx = grid_host[2 * i], gy = grid_host[2 * i + 1];
      g4[i] = make_float4(gx, gy, 0.0f, 0.0f);
    }
    c->search_spec = search_table_spec(grid_host, n);
    table.assign(search_table_words(c->search_spec), 0u);
    build_search_table(grid_host, n, c->search_spec, table.data());
  }
  uint32_t masks[2][32];
  std::memset(masks, 0, sizeof(masks));
  for (int role = 0; role < 2 && rotated; ++role) {
    const int8_t* s = role == kRoleK ? signs_k_host : signs_v_host;
    for (int e = 0; e < d; ++e)
      if (s[e] < 0) masks[role][(e >> 3) & 31] |= 1u << (((e >> 8) << 3) | (e & 7));
  }

  bool ok = cudaGetDevice(&c->device) == cudaSuccess;
  ok = ok && cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device) == cudaSuccess;
  if (ok) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    ok = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
         q == cudaDriverEntryPointSuccess && fn != nullptr;
    c->encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
  }
  ok = ok && cudaMalloc(&c->d_grid4, sizeof(float4) * 256) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_signmask[0], sizeof(uint32_t) * 32) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_signmask[1], sizeof(uint32_t) * 32) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_status, sizeof(int)) == cudaSuccess;
  ok = ok && cudaMalloc(&c->d_search_table, table.size() * sizeof(uint32_t)) == cudaSuccess;
  ok = ok && cudaMemcpy(c->d_search_table, table.data(), table.size() * sizeof(uint32_t),
                        cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->d_grid4, g4, sizeof(float4) * n, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->d_signmask[0], masks[0], sizeof(masks[0]), cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(c->d_signmask[1], masks[1], sizeof(masks[1]), cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemset(c->d_status, 0, sizeof(int)) == cudaSuccess;
  if (ok && gdim == 4) {
    // the search table of the four-dimensional grid (16 MB) is computed on the device
    const size_t n_cells = size_t(kGrid4Cells) * kGrid4Cells * kGrid4Cells * kGrid4Cells;
    ok = cudaMalloc(&c->d_grid4_table, n_cells * sizeof(uint4)) == cudaSuccess;
    if (ok) {
      grid4_table_kernel<<<c->sm_count * 8, 256>>>(c->d_grid4, c->d_grid4_table);
      ok = cudaGetLastError() == cudaSuccess;
    }
  }
  ok = ok && cudaFuncSetAttribute(gemm_pred_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  int(kGemmSmemBytes)) == cudaSuccess;
  ok = ok && cudaFuncSetAttribute(gemm_pred_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                  int(kGemmSmemBytes)) == cudaSuccess;
  ok = ok && cudaDeviceSynchronize() == cudaSuccess;
  if (!ok) {
    (void)cudaGetLastError();
    aquakv_destroy(c);
    return AQUAKV_ERR_CUDA;
  }
  // Two full waves of 128x256 GEMM tiles per chunk: 2 * SMs * 128 * 256 fp32 = 38.8 MB of
  // prediction, well inside L2 next to the chunk's 16-bit rows.
  c->chunk_tokens = 2 * c->sm_count * kBM / (d / kBN);
  *out = c;
  return AQUAKV_OK;
}

int aquakv_destroy(aquakv_ctx* c) {
  if (c == nullptr) return AQUAKV_OK;
  bool ok = true;
  if (c->d_grid4) ok = cudaFree(c->d_grid4) == cudaSuccess && ok;
  if (c->d_grid4_table) ok = cudaFree(c->d_grid4_table) == cudaSuccess && ok;
  if (c->d_signmask[0]) ok = cudaFree(c->d_signmask[0]) == cudaSuccess && ok;
  if (c->d_signmask[1]) ok = cudaFree(c->d_signmask[1]) == cudaSuccess && ok;
  if (c->d_status) ok = cudaFree(c->d_status) == cudaSuccess && ok;
  if (c->d_search_table) ok = cudaFree(c->d_search_table) == cudaSuccess && ok;
  if (c->prof_ev) {
    for (int i = 0; i < 2 * kProfMaxPairs; ++i)
      if (c->prof_ev[i]) cudaEventDestroy(c->prof_ev[i]);
    delete[] c->prof_ev;
    delete[] c->prof_class;
  }
  delete c;
  return ok ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

size_t aquakv_workspace_bytes(const aquakv_ctx* c, int64_t n_tokens, int op) {
  if (c == nullptr || n_tokens <= 0) return 0;
  if (op == AQUAKV_OP_ENCODE || op == AQUAKV_OP_DECODE) {
    const size_t phase_bytes = encode_ws(c, n_tokens).total;
    if (uniform_backbone(c)) return phase_bytes;
    const size_t layer_bytes = layer_ws(c, n_tokens).total;
    return phase_bytes > layer_bytes ? phase_bytes : layer_bytes;
  }
  return 0;
}

size_t aquakv_decode_attn_workspace_bytes(const aquakv_ctx* c, int32_t batch, int64_t ctx_len,
                                          int32_t n_q_heads, int32_t head_dim) {
  if (c != nullptr && uniform_backbone(c)) return 0;
  if (c == nullptr || batch <= 0 || ctx_len <= 0 || n_q_heads <= 0 || head_dim <= 0) return 0;
  // the caller may or may not pass predictors and may switch the mode: the larger of the two layouts
  const size_t a = attn_ws(c, batch, ctx_len, n_q_heads, head_dim, true).total;
  const size_t b = attn_ws(c, batch, ctx_len, n_q_heads, head_dim, false).total;
  return a > b ? a : b;
}

int64_t aquakv_launch_count(const aquakv_ctx* c) { return c ? c->launches : 0; }

int aquakv_profile_enable(aquakv_ctx* c, int enable) {
  if (c == nullptr) return AQUAKV_ERR_INVALID_ARG;
  if (enable && c->prof_ev == nullptr) {
    c->prof_ev = new (std::nothrow) cudaEvent_t[2 * kProfMaxPairs]();
    c->prof_class = new (std::nothrow) uint8_t[kProfMaxPairs]();
    if (c->prof_ev == nullptr || c->prof_class == nullptr) return AQUAKV_ERR_CUDA;
    for (int i = 0; i < 2 * kProfMaxPairs; ++i)
      if (cudaEventCreate(&c->prof_ev[i]) != cudaSuccess) return AQUAKV_ERR_CUDA;
  }
  c->prof_on = enable != 0;
  c->prof_n = 0;
  return AQUAKV_OK;
}

int aquakv_profile_read(aquakv_ctx* c, int kernel_class, int64_t* launches, double* total_ms) {
  if (c == nullptr || launches == nullptr || total_ms == nullptr) return AQUAKV_ERR_INVALID_ARG;
  *launches = 0;
  *total_ms = 0.0;
  for (int i = 0; i < c->prof_n; ++i) {
    if (c->prof_class[i] != kernel_class) continue;
    if (cudaEventSynchronize(c->prof_ev[2 * i + 1]) != cudaSuccess) return AQUAKV_ERR_CUDA;
    float ms = 0.0f;
    if (cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]) != cudaSuccess)
      return AQUAKV_ERR_CUDA;
    *total_ms += ms;
    ++*launches;
  }
  return AQUAKV_OK;
}

int aquakv_gather_rows(aquakv_ctx* c, int64_t n_rows, const int64_t* idx, int64_t n_src_rows, const void* src,
                       int64_t ld_src, void* dst, int64_t ld_dst, void* cuda_stream) {
  if (c == nullptr || n_rows < 0 || n_src_rows < 0) return AQUAKV_ERR_INVALID_ARG;
  if (n_rows == 0) return AQUAKV_OK;
  const int d = c->p.d_kv;
  int rc;
  if ((rc = check_rows(src, ld_src, d, true))) return rc;
  if ((rc = check_rows(dst, ld_dst, d, true))) return rc;
  if (src == dst || (idx == nullptr && n_rows > n_src_rows)) return AQUAKV_ERR_INVALID_ARG;
  if (idx != nullptr && (reinterpret_cast<uintptr_t>(idx) & 7u)) return AQUAKV_ERR_ALIGNMENT;
  const int warps_per_block = 8;
  int64_t blocks = (n_rows + warps_per_block - 1) / warps_per_block;
  const int64_t cap = int64_t(c->sm_count) * 16;
  if (blocks > cap) blocks = cap;
  gather_rows_kernel<<<int(blocks), warps_per_block * 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      static_cast<const uint16_t*>(src), ld_src, reinterpret_cast<const long long*>(idx), n_rows, n_src_rows, d,
      static_cast<uint16_t*>(dst), ld_dst, c->d_status);
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

size_t aquakv_fit_workspace_bytes(const aquakv_ctx* c, int64_t n_tokens, int32_t n_inputs) {
  if (c == nullptr || n_tokens <= 0 || n_inputs < 1 || n_inputs > 2) return 0;
  return fit_ws(c, n_tokens, n_inputs).total;
}

int aquakv_fit_predictor(aquakv_ctx* c, int64_t n_tokens, const void* in0, const void* in1, int64_t ld_in,
                         const void* target, int64_t ld_target, double rate, int fit_bias, void* W_out,
                         float* W32_out, float* bias_out, void* workspace, size_t workspace_bytes,
                         void* cuda_stream) {
  if (c == nullptr || n_tokens <= 0 || !(rate >= 0.0) || W_out == nullptr) return AQUAKV_ERR_INVALID_ARG;
  const int d = c->p.d_kv;
  if (d % kBN) return AQUAKV_ERR_UNSUPPORTED;
  if (n_tokens > (int64_t(1) << 30)) return AQUAKV_ERR_TOO_LARGE;
  int rc;
  if ((rc = check_rows(in0, ld_in, d, true))) return rc;
  if ((rc = check_rows(in1, ld_in, d, false))) return rc;
  if ((rc = check_rows(target, ld_target, d, true))) return rc;
  if (fit_bias && bias_out == nullptr) return AQUAKV_ERR_INVALID_ARG;
  if (!aligned16(W_out) || !aligned16(W32_out) || (fit_bias && !aligned16(bias_out))) return AQUAKV_ERR_ALIGNMENT;
  const int n_inputs = in1 != nullptr ? 2 : 1;
  const FitWs w = fit_ws(c, n_tokens, n_inputs);
  if (workspace == nullptr || !aligned16(workspace) || workspace_bytes < w.total) return AQUAKV_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = ws_base(workspace);
  uint16_t* Xt = reinterpret_cast<uint16_t*>(ws + w.xt_off);
  uint16_t* Yt = reinterpret_cast<uint16_t*>(ws + w.yt_off);
  float* G = reinterpret_cast<float*>(ws + w.g_off);
  float* C = reinterpret_cast<float*>(ws + w.c_off);
  double* Gd = reinterpret_cast<double*>(ws + w.gd_off);
  double* Cd = reinterpret_cast<double*>(ws + w.cd_off);
  double* sx = reinterpret_cast<double*>(ws + w.sums_off);
  double* sy = sx + w.n;
  double* ridge = reinterpret_cast<double*>(ws + w.ridge_off);
  const int n = w.n;
  const long long T = n_tokens, Tp = w.Tp;
  ProfScope prof(c, st, AQUAKV_KERNEL_FIT);

  // 1. token-contiguous copies
  {
    const dim3 block(32, 8);
    const dim3 grid_x((unsigned)(Tp / 32), (unsigned)(d / 32));
    fit_transpose_kernel<<<grid_x, block, 0, st>>>(static_cast<const uint16_t*>(in0), ld_in, T, Tp, Xt);
    if (in1 != nullptr)
      fit_transpose_kernel<<<grid_x, block, 0, st>>>(static_cast<const uint16_t*>(in1), ld_in, T, Tp,
                                                     Xt + size_t(d) * size_t(Tp));
    fit_transpose_kernel<<<grid_x, block, 0, st>>>(static_cast<const uint16_t*>(target), ld_target, T, Tp, Yt);
    c->launches += in1 != nullptr ? 3 : 2;
  }
  // 2. normal equations on the tensor cores
  if ((rc = launch_gram(c, st, Xt, n, Xt, n, Tp, G))) return rc;
  if ((rc = launch_gram(c, st, Xt, n, Yt, d, Tp, C))) return rc;
  // column sums for the intercept
  if (fit_bias) {
    if (cudaMemsetAsync(sx, 0, size_t(n + d) * sizeof(double), st) != cudaSuccess) return AQUAKV_ERR_CUDA;
    const dim3 block(32, 8);
    const dim3 grid_s((unsigned)((T + 255) / 256), (unsigned)(d / 32));
    if (c->bf16) {
      fit_colsum_kernel<true><<<grid_s, block, 0, st>>>(static_cast<const uint16_t*>(in0), ld_in, T, sx);
      if (in1) fit_colsum_kernel<true><<<grid_s, block, 0, st>>>(static_cast<const uint16_t*>(in1), ld_in, T, sx + d);
      fit_colsum_kernel<true><<<grid_s, block, 0, st>>>(static_cast<const uint16_t*>(target), ld_target, T, sy);
    } else {
      fit_colsum_kernel<false><<<grid_s, block, 0, st>>>(static_cast<const uint16_t*>(in0), ld_in, T, sx);
      if (in1) fit_colsum_kernel<false><<<grid_s, block, 0, st>>>(static_cast<const uint16_t*>(in1), ld_in, T, sx + d);
      fit_colsum_kernel<false><<<grid_s, block, 0, st>>>(static_cast<const uint16_t*>(target), ld_target, T, sy);
    }
    c->launches += in1 != nullptr ? 3 : 2;
  }
  const double* sxp = fit_bias ? sx : nullptr;
  const double* syp = fit_bias ? sy : nullptr;
  fit_ridge_kernel<<<1, 256, 0, st>>>(G, n, double(T), sxp, rate, ridge);
  {
    const int wide = n > d ? n : d;
    const dim3 grid_p((wide + 255) / 256, n);
    fit_prepare_kernel<<<grid_p, 256, 0, st>>>(G, C, n, d, double(T), sxp, syp, ridge, Gd, Cd);
  }
  c->launches += 2;
  // 3. Cholesky factorisation, panel by panel
  for (int k = 0; k < n; k += kFitNB) {
    fit_chol_diag_kernel<<<1, dim3(kFitNB, kFitNB), 0, st>>>(Gd, n, k, c->d_status);
    ++c->launches;
    const int below = n - k - kFitNB;
    if (below > 0) {
      fit_chol_panel_kernel<<<below / kFitNB, kFitNB, 0, st>>>(Gd, n, k);
      ++c->launches;
      double* A22 = Gd + size_t(k + kFitNB) * n + (k + kFitNB);
      const double* L21 = Gd + size_t(k + kFitNB) * n + k;
      launch_fit_update(c, st, A22, n, L21, n, 0, L21, n, 1, below, below, 1);
    }
  }
  // forward solve L Z = Cd, then backward solve L^T Wt = Z (both in place in Cd)
  const int solve_grid = (d + 127) / 128;
  for (int k = 0; k < n; k += kFitNB) {
    fit_solve_diag_kernel<<<solve_grid, 128, 0, st>>>(Gd, n, k, Cd, d, 0);
    ++c->launches;
    const int below = n - k - kFitNB;
    launch_fit_update(c, st, Cd + size_t(k + kFitNB) * d, d, Gd + size_t(k + kFitNB) * n + k, n, 0,
                      Cd + size_t(k) * d, d, 0, below, d, 0);
  }
  for (int k = n - kFitNB; k >= 0; k -= kFitNB) {
    fit_solve_diag_kernel<<<solve_grid, 128, 0, st>>>(Gd, n, k, Cd, d, 1);
    ++c->launches;
    launch_fit_update(c, st, Cd, d, Gd + size_t(k) * n, n, 1, Cd + size_t(k) * d, d, 0, k, d, 0);
  }
  // 4. the adapter in its storage layout, and the intercept
  {
    const dim3 block(32, 8), grid_o(n / 32, d / 32);
    if (c->bf16) fit_store_kernel<true><<<grid_o, block, 0, st>>>(Cd, n, d, static_cast<uint16_t*>(W_out), W32_out);
    else fit_store_kernel<false><<<grid_o, block, 0, st>>>(Cd, n, d, static_cast<uint16_t*>(W_out), W32_out);
    ++c->launches;
    if (fit_bias) {
      fit_bias_kernel<<<(d + 127) / 128, 128, 0, st>>>(Cd, n, d, sx, sy, double(T), bias_out);
      ++c->launches;
    }
  }
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

int aquakv_poll_status(aquakv_ctx* c, void* cuda_stream) {
  if (c == nullptr) return AQUAKV_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaStreamSynchronize(st) != cudaSuccess) return AQUAKV_ERR_CUDA;
  int h = 0;
  if (cudaMemcpy(&h, c->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return AQUAKV_ERR_CUDA;
  if (h != 0 && cudaMemset(c->d_status, 0, sizeof(int)) != cudaSuccess) return AQUAKV_ERR_CUDA;
  return h;
}

int aquakv_selftest_bounded_wait(aquakv_ctx* c, int64_t limit_ns, void* cuda_stream) {
  if (c == nullptr || limit_ns <= 0 || limit_ns > int64_t(kWaitLimitNs)) return AQUAKV_ERR_INVALID_ARG;
  bounded_wait_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      c->d_status, static_cast<unsigned long long>(limit_ns));
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

int aquakv_predict(aquakv_ctx* c, int64_t n_tokens, const void* in0, const void* in1, int64_t ld_in,
                   const void* W, const float* bias, float* P, int64_t ldP, void* cuda_stream) {
  if (c == nullptr || n_tokens < 0) return AQUAKV_ERR_INVALID_ARG;
  if (n_tokens == 0) return AQUAKV_OK;
  const int d = c->p.d_kv;
  if (in0 == nullptr || W == nullptr || P == nullptr || ld_in < d || ldP < d)
    return AQUAKV_ERR_INVALID_ARG;
  if (ld_in % 8 || ldP % 4 || !aligned16(in0) || !aligned16(in1) || !aligned16(W) || !aligned16(P) ||
      (bias != nullptr && !aligned16(bias)))
    return AQUAKV_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t step = int64_t(1) << 20;   // rows per launch (keeps per-launch row counts in int)
  for (int64_t t0 = 0; t0 < n_tokens; t0 += step) {
    const int rows = int(n_tokens - t0 < step ? n_tokens - t0 : step);
    const uint16_t* a0 = static_cast<const uint16_t*>(in0) + t0 * ld_in;
    const uint16_t* a1 = in1 ? static_cast<const uint16_t*>(in1) + t0 * ld_in : nullptr;
    const int rc = launch_predict(c, st, rows, a0, a1, ld_in, ld_in, W, bias, P + t0 * ldP, ldP);
    if (rc) return rc;
  }
  return AQUAKV_OK;
}

int aquakv_encode_phase(aquakv_ctx* c, int role, int64_t n_tokens, const void* X, int64_t ld_x,
                        const void* in0, const void* in1, int64_t ld_in, const void* W,
                        const float* bias, uint8_t* codes, uint16_t* scales, void* hat,
                        int64_t ld_hat, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (c == nullptr || n_tokens < 0 || (role != kRoleK && role != kRoleV)) return AQUAKV_ERR_INVALID_ARG;
  if (n_tokens == 0) return AQUAKV_OK;
  const int d = c->p.d_kv;
  int rc;
  if ((rc = check_rows(X, ld_x, d, true))) return rc;
  if ((rc = check_rows(hat, ld_hat, d, false))) return rc;
  if ((rc = check_cache(codes, scales, codes, scales))) return rc;
  const bool has_pred = W != nullptr;
  if (has_pred) {
    if ((rc = check_rows(in0, ld_in, d, true))) return rc;
    if ((rc = check_rows(in1, ld_in, d, false))) return rc;
    if (!aligned16(W) || (bias != nullptr && !aligned16(bias))) return AQUAKV_ERR_ALIGNMENT;
  } else if (in0 != nullptr || in1 != nullptr || bias != nullptr) {
    return AQUAKV_ERR_INVALID_ARG;
  }
  if (hat != nullptr && (hat == X || hat == in0 || hat == in1)) return AQUAKV_ERR_INVALID_ARG;
  const EncodeWs ws = encode_ws(c, n_tokens);
  if (has_pred) {
    if (workspace == nullptr || workspace_bytes < ws.total) return AQUAKV_ERR_WORKSPACE;
    if (!aligned16(workspace)) return AQUAKV_ERR_ALIGNMENT;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  float* P = has_pred ? reinterpret_cast<float*>(ws_base(workspace) + ws.p_off) : nullptr;
  const int cb = c->code_bytes, ng = c->n_groups;
  const uint16_t* Xp = static_cast<const uint16_t*>(X);
  const uint16_t* a0 = static_cast<const uint16_t*>(in0);
  const uint16_t* a1 = static_cast<const uint16_t*>(in1);
  for (int64_t t0 = 0; t0 < n_tokens; t0 += ws.chunk) {
    const int rows = int(n_tokens - t0 < ws.chunk ? n_tokens - t0 : ws.chunk);
    if (has_pred) {
      rc = launch_predict(c, st, rows, a0 + t0 * ld_in, a1 ? a1 + t0 * ld_in : nullptr, ld_in, ld_in,
                          W, bias, P, d);
      if (rc) return rc;
    }
    rc = launch_encode_rows(c, st, role, rows, Xp + t0 * ld_x, ld_x, P, d, codes + t0 * cb,
                            scales + t0 * ng,
                            hat != nullptr ? static_cast<uint16_t*>(hat) + t0 * ld_hat : nullptr, ld_hat);
    if (rc) return rc;
  }
  return AQUAKV_OK;
}

int aquakv_decode_phase(aquakv_ctx* c, int role, int64_t n_tokens, const uint8_t* codes,
                        const uint16_t* scales, const void* in0, const void* in1, int64_t ld_in,
                        const void* W, const float* bias, void* hat, int64_t ld_hat,
                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (c == nullptr || n_tokens < 0 || (role != kRoleK && role != kRoleV)) return AQUAKV_ERR_INVALID_ARG;
  if (n_tokens == 0) return AQUAKV_OK;
  const int d = c->p.d_kv;
  int rc;
  if ((rc = check_rows(hat, ld_hat, d, true))) return rc;
  if ((rc = check_cache(codes, scales, codes, scales))) return rc;
  const bool has_pred = W != nullptr;
  if (has_pred) {
    if ((rc = check_rows(in0, ld_in, d, true))) return rc;
    if ((rc = check_rows(in1, ld_in, d, false))) return rc;
    if (!aligned16(W) || (bias != nullptr && !aligned16(bias))) return AQUAKV_ERR_ALIGNMENT;
  } else if (in0 != nullptr || in1 != nullptr || bias != nullptr) {
    return AQUAKV_ERR_INVALID_ARG;
  }
  if (hat == in0 || hat == in1) return AQUAKV_ERR_INVALID_ARG;
  const EncodeWs ws = encode_ws(c, n_tokens);
  if (has_pred) {
    if (workspace == nullptr || workspace_bytes < ws.total) return AQUAKV_ERR_WORKSPACE;
    if (!aligned16(workspace)) return AQUAKV_ERR_ALIGNMENT;
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  float* P = has_pred ? reinterpret_cast<float*>(ws_base(workspace) + ws.p_off) : nullptr;
  const int cb = c->code_bytes, ng = c->n_groups;
  const uint16_t* a0 = static_cast<const uint16_t*>(in0);
  const uint16_t* a1 = static_cast<const uint16_t*>(in1);
  for (int64_t t0 = 0; t0 < n_tokens; t0 += ws.chunk) {
    const int rows = int(n_tokens - t0 < ws.chunk ? n_tokens - t0 : ws.chunk);
    if (has_pred) {
      rc = launch_predict(c, st, rows, a0 + t0 * ld_in, a1 ? a1 + t0 * ld_in : nullptr, ld_in, ld_in,
                          W, bias, P, d);
      if (rc) return rc;
    }
    rc = launch_decode_rows(c, st, role, rows, codes + t0 * cb, scales + t0 * ng, P, d,
                            static_cast<uint16_t*>(hat) + t0 * ld_hat, ld_hat);
    if (rc) return rc;
  }
  return AQUAKV_OK;
}

int aquakv_encode(aquakv_ctx* c, int64_t n_tokens, const void* K, const void* V, int64_t ld_kv,
                  const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev, const void* Wk,
                  const void* Wv, const float* bk, const float* bv, uint8_t* Kcodes,
                  uint16_t* Kscales, uint8_t* Vcodes, uint16_t* Vscales, void* Khat, void* Vhat,
                  int64_t ld_hat, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (c == nullptr || n_tokens < 0) return AQUAKV_ERR_INVALID_ARG;
  if (n_tokens == 0) return AQUAKV_OK;
  const int d = c->p.d_kv;
  int rc;
  if ((rc = check_rows(K, ld_kv, d, true))) return rc;
  if ((rc = check_rows(V, ld_kv, d, true))) return rc;
  if ((rc = check_rows(Khat, ld_hat, d, false))) return rc;
  if ((rc = check_rows(Vhat, ld_hat, d, false))) return rc;
  if ((rc = check_cache(Kcodes, Kscales, Vcodes, Vscales))) return rc;
  bool has_pred = false;
  if ((rc = check_adapters(Khat_prev, Vhat_prev, ld_prev, Wk, Wv, bk, bv, d, &has_pred))) return rc;
  if ((Khat != nullptr && (Khat == Khat_prev || Khat == K || Khat == Vhat_prev)) ||
      (Vhat != nullptr && (Vhat == Vhat_prev || Vhat == V || Vhat == Khat_prev || Vhat == Khat)))
    return AQUAKV_ERR_INVALID_ARG;
  if (has_pred) {
    if (workspace == nullptr || workspace_bytes < aquakv_workspace_bytes(c, n_tokens, AQUAKV_OP_ENCODE))
      return AQUAKV_ERR_WORKSPACE;
    if (!aligned16(workspace)) return AQUAKV_ERR_ALIGNMENT;
  }
  if (has_pred && uniform_backbone(c)) {
    // no fused kernel for this backbone: the key phase, then the value phase on the reconstructed keys
    if (Khat == nullptr) return AQUAKV_ERR_INVALID_ARG;
    if (ld_prev != ld_hat) return AQUAKV_ERR_UNSUPPORTED;   // the value phase reads both inputs with one stride
    if ((rc = aquakv_encode_phase(c, AQUAKV_ROLE_KEY, n_tokens, K, ld_kv, Khat_prev, nullptr, ld_prev, Wk, bk, Kcodes,
                                  Kscales, Khat, ld_hat, workspace, workspace_bytes, cuda_stream)))
      return rc;
    return aquakv_encode_phase(c, AQUAKV_ROLE_VALUE, n_tokens, V, ld_kv, Vhat_prev, Khat, ld_prev, Wv, bv, Vcodes,
                               Vscales, Vhat, ld_hat, workspace, workspace_bytes, cuda_stream);
  }
  if (has_pred) {
    if (n_tokens > (int64_t(1) << 30)) return AQUAKV_ERR_UNSUPPORTED;
    return launch_layer(c, static_cast<cudaStream_t>(cuda_stream), true, n_tokens, K, V, ld_kv, Khat_prev,
                        Vhat_prev, ld_prev, Wk, Wv, bk, bv, Kcodes, Kscales, Vcodes, Vscales, Khat, Vhat,
                        ld_hat, workspace);
  }
  // no predictor (layer 0): the row kernels alone, in launches of up to 2^30 rows (no prediction
  // buffer bounds them)
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int cb = c->code_bytes, ng = c->n_groups;
  const uint16_t* Kp = static_cast<const uint16_t*>(K);
  const uint16_t* Vp = static_cast<const uint16_t*>(V);
  const int64_t chunk = int64_t(1) << 30;
  for (int64_t t0 = 0; t0 < n_tokens; t0 += chunk) {
    const int rows = int(n_tokens - t0 < chunk ? n_tokens - t0 : chunk);
    rc = launch_encode_rows(c, st, kRoleK, rows, Kp + t0 * ld_kv, ld_kv, nullptr, d, Kcodes + t0 * cb,
                            Kscales + t0 * ng,
                            Khat != nullptr ? static_cast<uint16_t*>(Khat) + t0 * ld_hat : nullptr, ld_hat);
    if (rc) return rc;
    rc = launch_encode_rows(c, st, kRoleV, rows, Vp + t0 * ld_kv, ld_kv, nullptr, d, Vcodes + t0 * cb,
                            Vscales + t0 * ng,
                            Vhat != nullptr ? static_cast<uint16_t*>(Vhat) + t0 * ld_hat : nullptr, ld_hat);
    if (rc) return rc;
  }
  return AQUAKV_OK;
}

int aquakv_decode(aquakv_ctx* c, int64_t n_tokens, const uint8_t* Kcodes, const uint16_t* Kscales,
                  const uint8_t* Vcodes, const uint16_t* Vscales, const void* Khat_prev,
                  const void* Vhat_prev, int64_t ld_prev, const void* Wk, const void* Wv,
                  const float* bk, const float* bv, void* Khat, void* Vhat, int64_t ld_hat,
                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (c == nullptr || n_tokens < 0) return AQUAKV_ERR_INVALID_ARG;
  if (n_tokens == 0) return AQUAKV_OK;
  const int d = c->p.d_kv;
  int rc;
  if ((rc = check_rows(Khat, ld_hat, d, true))) return rc;
  if ((rc = check_rows(Vhat, ld_hat, d, true))) return rc;
  if ((rc = check_cache(Kcodes, Kscales, Vcodes, Vscales))) return rc;
  bool has_pred = false;
  if ((rc = check_adapters(Khat_prev, Vhat_prev, ld_prev, Wk, Wv, bk, bv, d, &has_pred))) return rc;
  if (Khat == Khat_prev || Khat == Vhat_prev || Vhat == Vhat_prev || Vhat == Khat_prev || Vhat == Khat)
    return AQUAKV_ERR_INVALID_ARG;
  if (has_pred) {
    if (workspace == nullptr || workspace_bytes < aquakv_workspace_bytes(c, n_tokens, AQUAKV_OP_DECODE))
      return AQUAKV_ERR_WORKSPACE;
    if (!aligned16(workspace)) return AQUAKV_ERR_ALIGNMENT;
    if (uniform_backbone(c)) {
      if (ld_prev != ld_hat) return AQUAKV_ERR_UNSUPPORTED;
      if ((rc = aquakv_decode_phase(c, AQUAKV_ROLE_KEY, n_tokens, Kcodes, Kscales, Khat_prev, nullptr, ld_prev, Wk, bk,
                                    Khat, ld_hat, workspace, workspace_bytes, cuda_stream)))
        return rc;
      return aquakv_decode_phase(c, AQUAKV_ROLE_VALUE, n_tokens, Vcodes, Vscales, Vhat_prev, Khat, ld_prev, Wv, bv,
                                 Vhat, ld_hat, workspace, workspace_bytes, cuda_stream);
    }
    if (n_tokens > (int64_t(1) << 30)) return AQUAKV_ERR_UNSUPPORTED;
    return launch_layer(c, static_cast<cudaStream_t>(cuda_stream), false, n_tokens, nullptr, nullptr, 0,
                        Khat_prev, Vhat_prev, ld_prev, Wk, Wv, bk, bv, const_cast<uint8_t*>(Kcodes),
                        const_cast<uint16_t*>(Kscales), const_cast<uint8_t*>(Vcodes),
                        const_cast<uint16_t*>(Vscales), Khat, Vhat, ld_hat, workspace);
  }
  // no predictor (layer 0): the row kernels alone, in launches of up to 2^30 rows
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int cb = c->code_bytes, ng = c->n_groups;
  uint16_t* Kh = static_cast<uint16_t*>(Khat);
  uint16_t* Vh = static_cast<uint16_t*>(Vhat);
  const int64_t chunk = int64_t(1) << 30;
  for (int64_t t0 = 0; t0 < n_tokens; t0 += chunk) {
    const int rows = int(n_tokens - t0 < chunk ? n_tokens - t0 : chunk);
    rc = launch_decode_rows(c, st, kRoleK, rows, Kcodes + t0 * cb, Kscales + t0 * ng, nullptr, d,
                            Kh + t0 * ld_hat, ld_hat);
    if (rc) return rc;
    rc = launch_decode_rows(c, st, kRoleV, rows, Vcodes + t0 * cb, Vscales + t0 * ng, nullptr, d,
                            Vh + t0 * ld_hat, ld_hat);
    if (rc) return rc;
  }
  return AQUAKV_OK;
}

size_t aquakv_chain_workspace_bytes(const aquakv_ctx* c, int64_t n_tokens, int32_t n_layers) {
  if (c != nullptr && uniform_backbone(c)) return 0;
  if (c == nullptr || n_tokens <= 0 || n_layers <= 0 || n_layers > kChainMaxLayers) return 0;
  if (n_tokens > kChainMaxTokens) return layers_supported(c) ? layers_ws(c, n_tokens, n_layers).total : 0;
  return chain_ws(c, n_tokens, n_layers).total;
}

int aquakv_encode_chain(aquakv_ctx* c, int64_t n_tokens, int32_t n_layers, const void* const* K, const void* const* V,
                        int64_t ld_kv, const void* Khat_init, const void* Vhat_init, int64_t ld_init,
                        const void* const* Wk, const void* const* Wv, const float* const* bk, const float* const* bv,
                        uint8_t* const* Kcodes, uint16_t* const* Kscales, uint8_t* const* Vcodes,
                        uint16_t* const* Vscales, void* const* Khat, void* const* Vhat, int64_t ld_hat, void* workspace,
                        size_t workspace_bytes, void* cuda_stream) {
  return run_chain(c, true, n_tokens, n_layers, K, V, ld_kv, Khat_init, Vhat_init, ld_init, Wk, Wv, bk, bv, Kcodes, Kscales,
                   Vcodes, Vscales, Khat, Vhat, ld_hat, workspace, workspace_bytes, cuda_stream);
}

int aquakv_decode_chain(aquakv_ctx* c, int64_t n_tokens, int32_t n_layers, const uint8_t* const* Kcodes,
                        const uint16_t* const* Kscales, const uint8_t* const* Vcodes, const uint16_t* const* Vscales,
                        const void* Khat_init, const void* Vhat_init, int64_t ld_init, const void* const* Wk,
                        const void* const* Wv, const float* const* bk, const float* const* bv, void* const* Khat,
                        void* const* Vhat, int64_t ld_hat, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return run_chain(c, false, n_tokens, n_layers, nullptr, nullptr, 0, Khat_init, Vhat_init, ld_init, Wk, Wv, bk, bv,
                   const_cast<uint8_t* const*>(Kcodes), const_cast<uint16_t* const*>(Kscales),
                   const_cast<uint8_t* const*>(Vcodes), const_cast<uint16_t* const*>(Vscales), Khat, Vhat, ld_hat, workspace,
                   workspace_bytes, cuda_stream);
}

// ---------------------------------------------------------------------------------------------
// aquakv_decode without a caller workspace: the prediction goes through a fixed array that is part
// of the library image.  In host code the symbol below is only a handle; the device address the
// kernels need comes from cudaGetSymbolAddress, looked up once per device.
// ---------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char
    g_noalloc_scratch[size_t(AQUAKV_NOALLOC_MAX_TOKENS) * 1024 * sizeof(float)];

namespace {
constexpr int kNoallocMaxDevices = 64;
std::mutex g_noalloc_mu;
float* g_noalloc_ptr[kNoallocMaxDevices] = {};

// Device address of the scratch array on `device`, which must be the current device.
int noalloc_scratch(int device, float** out) {
  if (device < 0 || device >= kNoallocMaxDevices) return AQUAKV_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  if (g_noalloc_ptr[device] == nullptr) {
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess) return AQUAKV_ERR_CUDA;
    if (cur != device) return AQUAKV_ERR_INVALID_ARG;
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return AQUAKV_ERR_CUDA;
    }
    g_noalloc_ptr[device] = static_cast<float*>(p);
  }
  *out = g_noalloc_ptr[device];
  return AQUAKV_OK;
}
}  // namespace

int aquakv_decode_noalloc(aquakv_ctx* c, int64_t n_tokens, const uint8_t* Kcodes,
                          const uint16_t* Kscales, const uint8_t* Vcodes, const uint16_t* Vscales,
                          const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev,
                          const void* Wk, const void* Wv, const float* bk, const float* bv,
                          void* Khat, void* Vhat, int64_t ld_hat, void* cuda_stream) {
  if (c != nullptr && uniform_backbone(c)) return AQUAKV_ERR_UNSUPPORTED;
  if (c == nullptr || n_tokens < 0) return AQUAKV_ERR_INVALID_ARG;
  if (n_tokens > AQUAKV_NOALLOC_MAX_TOKENS) return AQUAKV_ERR_TOO_LARGE;
  if (n_tokens == 0) return AQUAKV_OK;
  const int d = c->p.d_kv;   // <= 1024, so n_tokens * d floats fit the array
  int rc;
  if ((rc = check_rows(Khat, ld_hat, d, true))) return rc;
  if ((rc = check_rows(Vhat, ld_hat, d, true))) return rc;
  if ((rc = check_cache(Kcodes, Kscales, Vcodes, Vscales))) return rc;
  bool has_pred = false;
  if ((rc = check_adapters(Khat_prev, Vhat_prev, ld_prev, Wk, Wv, bk, bv, d, &has_pred))) return rc;
  if (Khat == Khat_prev || Khat == Vhat_prev || Vhat == Vhat_prev || Vhat == Khat_prev || Vhat == Khat)
    return AQUAKV_ERR_INVALID_ARG;
  float* P = nullptr;
  if (has_pred && (rc = noalloc_scratch(c->device, &P))) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int rows = int(n_tokens);
  const uint16_t* Kpv = static_cast<const uint16_t*>(Khat_prev);
  const uint16_t* Vpv = static_cast<const uint16_t*>(Vhat_prev);
  uint16_t* Kh = static_cast<uint16_t*>(Khat);
  uint16_t* Vh = static_cast<uint16_t*>(Vhat);
  if (has_pred && (rc = launch_predict(c, st, rows, Kpv, nullptr, ld_prev, 0, Wk, bk, P, d))) return rc;
  if ((rc = launch_decode_rows(c, st, kRoleK, rows, Kcodes, Kscales, P, d, Kh, ld_hat))) return rc;
  if (has_pred && (rc = launch_predict(c, st, rows, Vpv, Kh, ld_prev, ld_hat, Wv, bv, P, d))) return rc;
  return launch_decode_rows(c, st, kRoleV, rows, Vcodes, Vscales, P, d, Vh, ld_hat);
}

// Rotary position encoding of the keys the attention reads (rope.cuh).
struct RopeSpec {
  const float* table;     // device, [n_pos][head_dim / 2][2]
  int64_t n_pos;
  int64_t pos0;           // position of compressed token 0 of every sequence
  const int32_t* pos16;   // device, positions of the uncompressed rows [n16], or nullptr when there are none
};

static int launch_rope_rows(aquakv_ctx* c, cudaStream_t st, const RopeSpec& rope, const uint16_t* in, int64_t ld_in,
                            uint16_t* out, int64_t ld_out, int64_t rows, int n_kv_heads, int head_dim,
                            const int32_t* pos_list, int64_t period, int64_t row_base) {
  if (rows <= 0) return AQUAKV_OK;
  RopeArgs a;
  a.in = in;
  a.ld_in = ld_in;
  a.out = out;
  a.ld_out = ld_out;
  a.rows = rows;
  a.n_kv_heads = n_kv_heads;
  a.head_dim = head_dim;
  a.table = reinterpret_cast<const float2*>(rope.table);
  a.n_pos = rope.n_pos;
  a.pos_list = pos_list;
  a.period = period;
  a.row_base = row_base;
  a.pos0 = rope.pos0;
  a.status = c->d_status;
  const int64_t units = rows * (c->p.d_kv / 16);
  int64_t blocks = (units + 255) / 256;
  const int64_t cap = int64_t(c->sm_count) * 16;
  if (blocks > cap) blocks = cap;
  ProfScope prof(c, st, AQUAKV_KERNEL_ATTN);
  if (c->bf16) rope_rows_kernel<true><<<int(blocks), 256, 0, st>>>(a);
  else rope_rows_kernel<false><<<int(blocks), 256, 0, st>>>(a);
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

// Rotated copies of the keys: one chunk of decoded rows and the uncompressed rows.
struct RopeWs {
  size_t krot_off, k16_off, total;
};
static RopeWs rope_ws(const aquakv_ctx* c, size_t base_total, size_t chunk_rows, int32_t batch, int64_t n16) {
  RopeWs w;
  const size_t d = size_t(c->p.d_kv);
  w.krot_off = round_up(base_total, 256);
  w.k16_off = w.krot_off + round_up(chunk_rows * d * 2, 256);
  w.total = w.k16_off + round_up(size_t(batch) * size_t(n16) * d * 2, 256) + kWsSlack;
  return w;
}

// Partial-result arrays of the uncompressed rows that are attended to beside the compressed cache.
struct AttnExtWs {
  size_t ml_off, o_off, total;
  int splits;
};
static AttnExtWs attn_ext_ws(const aquakv_ctx* c, size_t base_total, int32_t batch, int64_t n16, int32_t n_q_heads,
                             int32_t head_dim) {
  AttnExtWs w;
  const int tb = c->attn_block_tokens;
  w.splits = n16 > 0 ? int((n16 + tb - 1) / tb) : 0;
  const size_t slots = size_t(batch) * size_t(w.splits);
  w.ml_off = round_up(base_total, 256);
  w.o_off = w.ml_off + round_up(slots * n_q_heads * 2 * sizeof(float), 256);
  w.total = w.o_off + round_up(slots * n_q_heads * head_dim * sizeof(float), 256) + kWsSlack;
  return w;
}

static int decode_attn_impl(aquakv_ctx* c, int32_t batch, int64_t ctx_len, int32_t n_q_heads,
                            int32_t n_kv_heads, int32_t head_dim, float softmax_scale, const void* q,
                            const uint8_t* Kcodes, const uint16_t* Kscales, const uint8_t* Vcodes,
                            const uint16_t* Vscales, const void* Khat_prev, const void* Vhat_prev,
                            int64_t ld_prev, const void* Wk, const void* Wv, const float* bk,
                            const float* bv, void* out, float* lse, void* Khat, void* Vhat,
                            int64_t ld_hat, const void* K16, const void* V16, int64_t n16, int64_t ld16,
                            const RopeSpec* rope, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (c != nullptr && uniform_backbone(c)) return AQUAKV_ERR_UNSUPPORTED;
  if (c == nullptr || batch < 0 || ctx_len < 0 || n16 < 0) return AQUAKV_ERR_INVALID_ARG;
  if (batch == 0 || (ctx_len == 0 && n16 == 0)) return AQUAKV_OK;
  const int d = c->p.d_kv;
  if (rope != nullptr) {
    if (rope->table == nullptr || rope->n_pos <= 0 || rope->pos0 < 0) return AQUAKV_ERR_INVALID_ARG;
    if (n16 > 0 && rope->pos16 == nullptr) return AQUAKV_ERR_INVALID_ARG;
    if (!aligned16(rope->table)) return AQUAKV_ERR_ALIGNMENT;
    if (rope->pos0 + ctx_len > rope->n_pos) return AQUAKV_ERR_INVALID_ARG;
  }
  if (n16 > 0) {
    int rc16;
    if ((rc16 = check_rows(K16, ld16, d, true))) return rc16;
    if ((rc16 = check_rows(V16, ld16, d, true))) return rc16;
    if (n16 > (int64_t(1) << 24)) return AQUAKV_ERR_UNSUPPORTED;
  }
  if (ctx_len == 0) {
    // nothing compressed yet: the uncompressed rows alone
    if (n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0) return AQUAKV_ERR_INVALID_ARG;
    if (n_kv_heads * head_dim != d || n_q_heads % n_kv_heads) return AQUAKV_ERR_INVALID_ARG;
    if ((head_dim != 64 && head_dim != 128) || n_q_heads / n_kv_heads > kAttnMmaMaxGq) return AQUAKV_ERR_UNSUPPORTED;
    if (q == nullptr || out == nullptr) return AQUAKV_ERR_INVALID_ARG;
    if (!aligned16(q) || !aligned16(out)) return AQUAKV_ERR_ALIGNMENT;
    if (!(softmax_scale == softmax_scale)) return AQUAKV_ERR_INVALID_ARG;
    const AttnExtWs xw = attn_ext_ws(c, 0, batch, n16, n_q_heads, head_dim);
    const RopeWs rw0 = rope_ws(c, xw.total, 0, batch, n16);
    if (workspace == nullptr || workspace_bytes < (rope != nullptr ? rw0.total : xw.total)) return AQUAKV_ERR_WORKSPACE;
    if (!aligned16(workspace)) return AQUAKV_ERR_ALIGNMENT;
    cudaStream_t st0 = static_cast<cudaStream_t>(cuda_stream);
    uint8_t* wsb0 = ws_base(workspace);
    AttnArgs a;
    a.q = static_cast<const uint16_t*>(q);
    a.Kh = static_cast<const uint16_t*>(K16);
    a.Vh = static_cast<const uint16_t*>(V16);
    a.ld = ld16;
    a.ld_v = ld16;
    if (rope != nullptr) {
      uint16_t* k16rot = reinterpret_cast<uint16_t*>(wsb0 + rw0.k16_off);
      int rcr = launch_rope_rows(c, st0, *rope, a.Kh, ld16, k16rot, d, int64_t(batch) * n16, n_kv_heads, head_dim,
                                 rope->pos16, n16, 0);
      if (rcr) return rcr;
      a.Kh = k16rot;
      a.ld = d;
    }
    a.tok_base = 0;
    a.blk_begin = 0;
    a.ctx = int(n16);
    a.n_q_heads = n_q_heads;
    a.n_kv_heads = n_kv_heads;
    a.n_splits = xw.splits;
    a.block_tokens = c->attn_block_tokens;
    a.scale_log2 = softmax_scale * 1.4426950408889634f;
    a.part_ml = reinterpret_cast<float*>(wsb0 + xw.ml_off);
    a.part_o = reinterpret_cast<float*>(wsb0 + xw.o_off);
    int rc0 = launch_attn_partial(c, st0, a, head_dim, batch * xw.splits);
    if (rc0) return rc0;
    AttnCombineArgs ca;
    ca.part_ml = a.part_ml;
    ca.part_o = a.part_o;
    ca.out = static_cast<uint16_t*>(out);
    ca.lse = lse;
    ca.n_q_heads = n_q_heads;
    ca.n_splits = xw.splits;
    ca.ctx = int(n16);
    ca.block_tokens = 0;
    ca.extra_ml = nullptr;
    ca.extra_o = nullptr;
    ca.extra_splits = 0;
    return launch_attn_combine(c, st0, ca, head_dim, batch);
  }
  if (n_q_heads <= 0 || n_kv_heads <= 0 || head_dim <= 0) return AQUAKV_ERR_INVALID_ARG;
  if (n_kv_heads * head_dim != d || n_q_heads % n_kv_heads) return AQUAKV_ERR_INVALID_ARG;
  if ((head_dim != 64 && head_dim != 128) || n_q_heads / n_kv_heads > kAttnMmaMaxGq)
    return AQUAKV_ERR_UNSUPPORTED;
  if (ctx_len > (int64_t(1) << 30)) return AQUAKV_ERR_UNSUPPORTED;
  if (q == nullptr || out == nullptr || Kcodes == nullptr || Kscales == nullptr ||
      Vcodes == nullptr || Vscales == nullptr)
    return AQUAKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out)) return AQUAKV_ERR_ALIGNMENT;
  if (!(softmax_scale == softmax_scale)) return AQUAKV_ERR_INVALID_ARG;
  int rc;
  if ((rc = check_cache(Kcodes, Kscales, Vcodes, Vscales))) return rc;
  if ((Khat == nullptr) != (Vhat == nullptr)) return AQUAKV_ERR_INVALID_ARG;
  if ((rc = check_rows(Khat, ld_hat, d, false))) return rc;
  if ((rc = check_rows(Vhat, ld_hat, d, false))) return rc;
  bool has_pred = false;
  if ((rc = check_adapters(Khat_prev, Vhat_prev, ld_prev, Wk, Wv, bk, bv, d, &has_pred))) return rc;
  if (Khat != nullptr && (Khat == Khat_prev || Khat == Vhat_prev || Vhat == Vhat_prev ||
                          Vhat == Khat_prev || Vhat == Khat))
    return AQUAKV_ERR_INVALID_ARG;
  // with rotary keys the attention reads a rotated copy of the decoded rows: the two-kernel layout
  const AttnWs ws = attn_ws(c, batch, ctx_len, n_q_heads, head_dim,
                            has_pred && rope == nullptr && c->attn_mode == AQUAKV_ATTN_FUSED);
  const AttnExtWs xw = attn_ext_ws(c, ws.total, batch, n16, n_q_heads, head_dim);
  const RopeWs rw = rope_ws(c, n16 > 0 ? xw.total : ws.total,
                            rope != nullptr ? size_t(ws.chunk_blocks) * size_t(c->attn_block_tokens) : 0, batch, n16);
  if (workspace == nullptr ||
      workspace_bytes < (rope != nullptr ? rw.total : (n16 > 0 ? xw.total : ws.total)))
    return AQUAKV_ERR_WORKSPACE;
  if (!aligned16(workspace)) return AQUAKV_ERR_ALIGNMENT;
  // partials of the uncompressed rows (attention sinks, recent-token buffer), merged by the combine kernel
  const float* extra_ml = nullptr;
  const float* extra_o = nullptr;
  if (n16 > 0) {
    uint8_t* wsx = ws_base(workspace);
    AttnArgs a;
    a.q = static_cast<const uint16_t*>(q);
    a.Kh = static_cast<const uint16_t*>(K16);
    a.Vh = static_cast<const uint16_t*>(V16);
    a.ld = ld16;
    a.ld_v = ld16;
    a.tok_base = 0;
    a.blk_begin = 0;
    a.ctx = int(n16);
    a.n_q_heads = n_q_heads;
    a.n_kv_heads = n_kv_heads;
    a.n_splits = xw.splits;
    a.block_tokens = c->attn_block_tokens;
    a.scale_log2 = softmax_scale * 1.4426950408889634f;
    a.part_ml = reinterpret_cast<float*>(wsx + xw.ml_off);
    a.part_o = reinterpret_cast<float*>(wsx + xw.o_off);
    if (rope != nullptr) {
      uint16_t* k16rot = reinterpret_cast<uint16_t*>(wsx + rw.k16_off);
      if ((rc = launch_rope_rows(c, static_cast<cudaStream_t>(cuda_stream), *rope, a.Kh, ld16, k16rot, d,
                                 int64_t(batch) * n16, n_kv_heads, head_dim, rope->pos16, n16, 0)))
        return rc;
      a.Kh = k16rot;
      a.ld = d;
    }
    if ((rc = launch_attn_partial(c, static_cast<cudaStream_t>(cuda_stream), a, head_dim, batch * xw.splits))) return rc;
    extra_ml = a.part_ml;
    extra_o = a.part_o;
  }
  const int extra_splits = n16 > 0 ? xw.splits : 0;
  if (ws.fused) {
    // Algorithm 3 and the attention read of Algorithm 4 in ONE launch: the attention warps of the layer
    // kernel consume every token block's decoded rows from L2 as soon as they exist
    if (int64_t(batch) * ctx_len > (int64_t(1) << 30)) return AQUAKV_ERR_UNSUPPORTED;
    uint8_t* wsb = ws_base(workspace);
    LayerAttnArgs at;
    at.q = q;
    at.ctx = int(ctx_len);
    at.n_q_heads = n_q_heads;
    at.n_kv_heads = n_kv_heads;
    at.n_splits = ws.n_splits;
    at.scale_log2 = softmax_scale * 1.4426950408889634f;
    at.part_ml = reinterpret_cast<float*>(wsb + ws.ml_off);
    at.part_o = reinterpret_cast<float*>(wsb + ws.o_off);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    rc = launch_layer(c, st, false, int64_t(batch) * ctx_len, nullptr, nullptr, 0, Khat_prev, Vhat_prev, ld_prev, Wk, Wv,
                      bk, bv, const_cast<uint8_t*>(Kcodes), const_cast<uint16_t*>(Kscales),
                      const_cast<uint8_t*>(Vcodes), const_cast<uint16_t*>(Vscales), Khat, Vhat, ld_hat,
                      wsb + ws.layer_off, &at);
    if (rc) return rc;
    AttnCombineArgs ca;
    ca.part_ml = at.part_ml;
    ca.part_o = at.part_o;
    ca.out = static_cast<uint16_t*>(out);
    ca.lse = lse;
    ca.n_q_heads = n_q_heads;
    ca.n_splits = ws.n_splits;
    ca.ctx = int(ctx_len);
    ca.block_tokens = kAttnSubTokens;
    ca.extra_ml = extra_ml;
    ca.extra_o = extra_o;
    ca.extra_splits = extra_splits;
    return launch_attn_combine(c, st, ca, head_dim, batch);
  }

  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  uint8_t* wsb = ws_base(workspace);
  float* part_ml = reinterpret_cast<float*>(wsb + ws.ml_off);
  float* part_o = reinterpret_cast<float*>(wsb + ws.o_off);
  const int cb = c->code_bytes, ng = c->n_groups, tb = c->attn_block_tokens;
  const uint16_t* Kpv = static_cast<const uint16_t*>(Khat_prev);
  const uint16_t* Vpv = static_cast<const uint16_t*>(Vhat_prev);
  const int64_t total_blocks = int64_t(batch) * ws.n_splits;
  auto block_token = [&](int64_t gb) -> int64_t {   // first global token of global block gb
    if (gb >= total_blocks) return int64_t(batch) * ctx_len;
    return (gb / ws.n_splits) * ctx_len + (gb % ws.n_splits) * int64_t(tb);
  };
  for (int64_t gb0 = 0; gb0 < total_blocks; gb0 += ws.chunk_blocks) {
    const int64_t gb1 = gb0 + ws.chunk_blocks < total_blocks ? gb0 + ws.chunk_blocks : total_blocks;
    const int64_t t0 = block_token(gb0), t1 = block_token(gb1);
    const int rows = int(t1 - t0);
    uint16_t* kh = Khat != nullptr ? static_cast<uint16_t*>(Khat) + t0 * ld_hat
                                   : reinterpret_cast<uint16_t*>(wsb + ws.khat_off);
    uint16_t* vh = Vhat != nullptr ? static_cast<uint16_t*>(Vhat) + t0 * ld_hat
                                   : reinterpret_cast<uint16_t*>(wsb + ws.vhat_off);
    const int64_t ldh = Khat != nullptr ? ld_hat : d;
    if (has_pred) {
      // Algorithm 3 for the chunk in one fused launch (predictor GEMMs + row work)
      rc = launch_layer(c, st, false, rows, nullptr, nullptr, 0, Kpv + t0 * ld_prev, Vpv + t0 * ld_prev,
                        ld_prev, Wk, Wv, bk, bv, const_cast<uint8_t*>(Kcodes) + t0 * cb,
                        const_cast<uint16_t*>(Kscales) + t0 * ng, const_cast<uint8_t*>(Vcodes) + t0 * cb,
                        const_cast<uint16_t*>(Vscales) + t0 * ng, kh, vh, ldh, wsb + ws.layer_off);
      if (rc) return rc;
    } else {
      rc = launch_decode_rows(c, st, kRoleK, rows, Kcodes + t0 * cb, Kscales + t0 * ng, nullptr, d, kh, ldh);
      if (rc) return rc;
      rc = launch_decode_rows(c, st, kRoleV, rows, Vcodes + t0 * cb, Vscales + t0 * ng, nullptr, d, vh, ldh);
      if (rc) return rc;
    }
    AttnArgs a;
    a.q = static_cast<const uint16_t*>(q);
    a.Kh = kh;
    a.Vh = vh;
    a.ld = ldh;
    a.ld_v = ldh;
    if (rope != nullptr) {
      // global row t0 + r is token (t0 + r) mod ctx_len of its sequence
      uint16_t* krot = reinterpret_cast<uint16_t*>(wsb + rw.krot_off);
      if ((rc = launch_rope_rows(c, st, *rope, kh, ldh, krot, d, rows, n_kv_heads, head_dim, nullptr, ctx_len, t0)))
        return rc;
      a.Kh = krot;
      a.ld = d;
    }
    a.tok_base = t0;
    a.blk_begin = gb0;
    a.ctx = int(ctx_len);
    a.n_q_heads = n_q_heads;
    a.n_kv_heads = n_kv_heads;
    a.n_splits = ws.n_splits;
    a.block_tokens = tb;
    a.scale_log2 = softmax_scale * 1.4426950408889634f;
    a.part_ml = part_ml;
    a.part_o = part_o;
    rc = launch_attn_partial(c, st, a, head_dim, int(gb1 - gb0));
    if (rc) return rc;
  }
  AttnCombineArgs ca;
  ca.part_ml = part_ml;
  ca.part_o = part_o;
  ca.out = static_cast<uint16_t*>(out);
  ca.lse = lse;
  ca.n_q_heads = n_q_heads;
  ca.n_splits = ws.n_splits;
  ca.ctx = int(ctx_len);
  ca.block_tokens = 0;
  ca.extra_ml = extra_ml;
  ca.extra_o = extra_o;
  ca.extra_splits = extra_splits;
  return launch_attn_combine(c, st, ca, head_dim, batch);
}

int aquakv_decode_attn(aquakv_ctx* c, int32_t batch, int64_t ctx_len, int32_t n_q_heads,
                       int32_t n_kv_heads, int32_t head_dim, float softmax_scale, const void* q,
                       const uint8_t* Kcodes, const uint16_t* Kscales, const uint8_t* Vcodes,
                       const uint16_t* Vscales, const void* Khat_prev, const void* Vhat_prev,
                       int64_t ld_prev, const void* Wk, const void* Wv, const float* bk,
                       const float* bv, void* out, float* lse, void* Khat, void* Vhat,
                       int64_t ld_hat, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return decode_attn_impl(c, batch, ctx_len, n_q_heads, n_kv_heads, head_dim, softmax_scale, q, Kcodes, Kscales, Vcodes,
                          Vscales, Khat_prev, Vhat_prev, ld_prev, Wk, Wv, bk, bv, out, lse, Khat, Vhat, ld_hat, nullptr,
                          nullptr, 0, 0, nullptr, workspace, workspace_bytes, cuda_stream);
}

size_t aquakv_decode_attn_buffered_workspace_bytes(const aquakv_ctx* c, int32_t batch, int64_t ctx_len,
                                                   int64_t n_uncompressed, int32_t n_q_heads, int32_t head_dim) {
  if (c == nullptr || batch <= 0 || ctx_len < 0 || n_uncompressed < 0 || n_q_heads <= 0 || head_dim <= 0) return 0;
  if (uniform_backbone(c)) return 0;
  const size_t base = ctx_len > 0 ? aquakv_decode_attn_workspace_bytes(c, batch, ctx_len, n_q_heads, head_dim) : 0;
  return attn_ext_ws(c, base, batch, n_uncompressed, n_q_heads, head_dim).total;
}

int aquakv_decode_attn_buffered(aquakv_ctx* c, int32_t batch, int64_t ctx_len, int32_t n_q_heads,
                                int32_t n_kv_heads, int32_t head_dim, float softmax_scale, const void* q,
                                const uint8_t* Kcodes, const uint16_t* Kscales, const uint8_t* Vcodes,
                                const uint16_t* Vscales, const void* Khat_prev, const void* Vhat_prev,
                                int64_t ld_prev, const void* Wk, const void* Wv, const float* bk,
                                const float* bv, const void* K16, const void* V16, int64_t n_uncompressed,
                                int64_t ld16, void* out, float* lse, void* Khat, void* Vhat, int64_t ld_hat,
                                void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return decode_attn_impl(c, batch, ctx_len, n_q_heads, n_kv_heads, head_dim, softmax_scale, q, Kcodes, Kscales, Vcodes,
                          Vscales, Khat_prev, Vhat_prev, ld_prev, Wk, Wv, bk, bv, out, lse, Khat, Vhat, ld_hat, K16, V16,
                          n_uncompressed, ld16, nullptr, workspace, workspace_bytes, cuda_stream);
}

int aquakv_set_attn_mode(aquakv_ctx* c, int mode) {
  if (c == nullptr || (mode != AQUAKV_ATTN_SPLIT && mode != AQUAKV_ATTN_FUSED)) return AQUAKV_ERR_INVALID_ARG;
  c->attn_mode = mode;
  return AQUAKV_OK;
}

int aquakv_rope_table(aquakv_ctx* c, int32_t head_dim, double theta_base, int64_t n_positions, float* table,
                      void* cuda_stream) {
  if (c == nullptr || table == nullptr || n_positions < 0) return AQUAKV_ERR_INVALID_ARG;
  if (head_dim != 64 && head_dim != 128) return AQUAKV_ERR_UNSUPPORTED;
  if (!(theta_base > 1.0) || !std::isfinite(theta_base)) return AQUAKV_ERR_INVALID_ARG;
  if (!aligned16(table)) return AQUAKV_ERR_ALIGNMENT;
  if (n_positions == 0) return AQUAKV_OK;
  if (n_positions > (int64_t(1) << 31)) return AQUAKV_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int half = head_dim / 2;
  int64_t blocks = (n_positions * half + 255) / 256;
  const int64_t cap = int64_t(c->sm_count) * 16;
  if (blocks > cap) blocks = cap;
  ProfScope prof(c, st, AQUAKV_KERNEL_ATTN);
  rope_table_kernel<<<int(blocks), 256, 0, st>>>(reinterpret_cast<float2*>(table), n_positions, half, theta_base);
  ++c->launches;
  return cudaGetLastError() == cudaSuccess ? AQUAKV_OK : AQUAKV_ERR_CUDA;
}

size_t aquakv_decode_attn_rope_workspace_bytes(const aquakv_ctx* c, int32_t batch, int64_t ctx_len,
                                               int64_t n_uncompressed, int32_t n_q_heads, int32_t head_dim) {
  if (c == nullptr || batch <= 0 || ctx_len < 0 || n_uncompressed < 0 || n_q_heads <= 0 || head_dim <= 0) return 0;
  if (uniform_backbone(c)) return 0;
  size_t base = 0, chunk_rows = 0;
  if (ctx_len > 0) {
    const AttnWs ws = attn_ws(c, batch, ctx_len, n_q_heads, head_dim, false);
    base = ws.total;
    chunk_rows = size_t(ws.chunk_blocks) * size_t(c->attn_block_tokens);
  }
  if (n_uncompressed > 0 || ctx_len == 0) base = attn_ext_ws(c, base, batch, n_uncompressed, n_q_heads, head_dim).total;
  return rope_ws(c, base, chunk_rows, batch, n_uncompressed).total;
}

int aquakv_decode_attn_rope(aquakv_ctx* c, int32_t batch, int64_t ctx_len, int32_t n_q_heads,
                            int32_t n_kv_heads, int32_t head_dim, float softmax_scale, const void* q,
                            const uint8_t* Kcodes, const uint16_t* Kscales, const uint8_t* Vcodes,
                            const uint16_t* Vscales, const void* Khat_prev, const void* Vhat_prev,
                            int64_t ld_prev, const void* Wk, const void* Wv, const float* bk,
                            const float* bv, const void* K16, const void* V16, int64_t n_uncompressed,
                            int64_t ld16, const float* rope_table, int64_t rope_positions, int64_t pos0,
                            const int32_t* pos16, void* out, float* lse, void* Khat, void* Vhat, int64_t ld_hat,
                            void* workspace, size_t workspace_bytes, void* cuda_stream) {
  RopeSpec rope;
  rope.table = rope_table;
  rope.n_pos = rope_positions;
  rope.pos0 = pos0;
  rope.pos16 = pos16;
  return decode_attn_impl(c, batch, ctx_len, n_q_heads, n_kv_heads, head_dim, softmax_scale, q, Kcodes, Kscales, Vcodes,
                          Vscales, Khat_prev, Vhat_prev, ld_prev, Wk, Wv, bk, bv, out, lse, Khat, Vhat, ld_hat, K16, V16,
                          n_uncompressed, ld16, &rope, workspace, workspace_bytes, cuda_stream);
}

}  // extern "C"
