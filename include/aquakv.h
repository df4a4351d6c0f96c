/*
 * aquakv.h -- C ABI of the B200 (sm_100a) AQUA-KV per-token KV-cache codec.
 *
 * The operations are those of the paper "Cache Me If You Must: Adaptive Key-Value Quantization
 * for Large Language Models": Algorithm 2 (encode), Algorithm 3 (decode) and the attention read
 * of Algorithm 4, with the backbone quantizer Q of Section 2 ("Vector Quantization")
 * and Section 4.1 ("Alternative quantizers"): group-wise vector quantization after a randomized
 * Hadamard transform, p = 2 values per code, n in {16, 64, 256} grid points, one fp16 scale per
 * group.
 *
 * Conventions shared by every entry point
 *   - Every data pointer is a DEVICE pointer owned by the caller unless its name ends in _host.
 *     The library allocates nothing per call; it uses only the caller's workspace.
 *   - 16-bit tensors (K, V, reconstructions, adapter matrices, queries, attention output) are
 *     fp16 or bf16 as chosen in aquakv_params.dtype; all of them share that type.
 *   - Token-major layout: row t holds the d_kv = n_kv_heads * head_dim values of token t,
 *     consecutive in memory; rows are `ld` ELEMENTS apart (ld >= d_kv, ld % 8 == 0).  Base
 *     pointers of 16-bit tensors and of the workspace are 16-byte aligned.
 *   - Adapter (predictor) matrices are row-major [out_features][in_features] like a linear
 *     layer's weight: pred[c] = sum_r x[r] * W[c][r] (+ bias[c]).  Wk is [d_kv][d_kv]; Wv is
 *     [d_kv][2*d_kv] and its input is the concatenation [Vhat_prev ; Khat] (columns 0..d_kv-1
 *     act on Vhat_prev, columns d_kv..2*d_kv-1 on the freshly reconstructed Khat).  Biases are
 *     optional fp32 [d_kv] (NULL = none).  Wk == NULL (then Wv, Khat_prev, Vhat_prev must be NULL
 *     too) selects the predictor-free path of layer 0 (the first layer of Algorithm 2).
 *   - Compressed cache, per tensor (keys and values are separate arrays), per token t:
 *       codes[t]  : d_kv/2 * log2(n) / 8 bytes; the code of value pair j (values 2j, 2j+1 of the
 *                   rotated row) occupies bits [j*log2(n), (j+1)*log2(n)) of the row's bit
 *                   stream, least significant bit first (n = 16: two codes per byte, low nibble
 *                   = even pair; n = 64: four codes per three bytes; n = 256: one byte each);
 *       scales[t] : d_kv/scale_group IEEE fp16 bit patterns, the group's root-mean-square
 *                   residual rounded to nearest even.
 *     Code arrays are 16-byte aligned (a token's codes are a multiple of 16 bytes, and the kernels
 *     move them as 16-byte vectors), scale arrays 2-byte aligned; AQUAKV_ERR_ALIGNMENT otherwise.
 *     Bits per value = log2(n)/2 + 16/scale_group (2.02 at n = 16, group 1024).
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream).  They never synchronise, print, abort or throw.  Every function
 *     returning int returns AQUAKV_OK or a negative AQUAKV_ERR_* code; argument errors are
 *     detected on the host before anything is launched.  n_tokens == 0 is AQUAKV_OK, no launch.
 *   - Non-finite inputs are memory-safe; the resulting codes/scales are unspecified.
 *   - A context may be used from one host thread at a time, on the device that was current
 *     when it was created.
 *   - The layer calls with predictors (encode, decode, decode_attn) and the chain calls run
 *     persistent kernels whose CTAs wait for one another and therefore must all be resident: do
 *     not let them overlap other kernels on the same device (other streams, other contexts).  If
 *     the grid cannot fit an idle device the call returns AQUAKV_ERR_UNSUPPORTED; if it is
 *     crowded out at run time, its waits expire after two seconds and the call's outputs are
 *     invalid, which only aquakv_poll_status reports (AQUAKV_ERR_TIMEOUT).
 */
#ifndef AQUAKV_H_
#define AQUAKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AQUAKV_F16 0
#define AQUAKV_BF16 1

#define AQUAKV_OK 0
#define AQUAKV_ERR_INVALID_ARG (-1) /* NULL where data is required, negative size, aliasing */
#define AQUAKV_ERR_UNSUPPORTED (-2) /* a parameter combination the kernels do not cover      */
#define AQUAKV_ERR_ALIGNMENT (-3)   /* pointer not 16-byte aligned or ld not a multiple of 8 */
#define AQUAKV_ERR_WORKSPACE (-4)   /* workspace NULL or smaller than aquakv_workspace_bytes */
#define AQUAKV_ERR_CUDA (-5)        /* a CUDA runtime/driver call failed                     */
#define AQUAKV_ERR_TIMEOUT (-6)     /* a bounded device-side wait expired (see poll_status)  */
#define AQUAKV_ERR_TOO_LARGE (-7)   /* more tokens than the fixed scratch of a *_noalloc call  */
#define AQUAKV_ERR_NUMERIC (-8)     /* a fit's normal equations were not positive definite (poll_status) */

#define AQUAKV_OP_ENCODE 0
#define AQUAKV_OP_DECODE 1
#define AQUAKV_OP_DECODE_ATTN 2

/* How aquakv_decode_attn and its variants run (aquakv_set_attn_mode). */
#define AQUAKV_ATTN_SPLIT 0 /* decode kernel, then a split-KV attention kernel over the fresh rows (default) */
#define AQUAKV_ATTN_FUSED 1 /* attention warps inside the decode kernel where the shape allows it          */

/* Parameters of the quantizer Q (Section 4.1: group size, p, n) and of the tensors. */
typedef struct aquakv_params {
  int32_t d_kv;        /* values per token row; supported: 256, 512, 1024                       */
  int32_t had_block;   /* h: Hadamard block, power of two, 64 <= h <= d_kv, divides d_kv        */
  int32_t scale_group; /* g: values per fp16 scale; multiple of h that divides d_kv             */
  int32_t grid_dim;    /* p: values per code; 2 (1: uniform backbone, 4: see aquakv_create)     */
  int32_t grid_size;   /* n: 16, 64 or 256 grid points (2, 3, 4 bits per value)                 */
  int32_t dtype;       /* AQUAKV_F16 or AQUAKV_BF16                                             */
} aquakv_params;

typedef struct aquakv_ctx aquakv_ctx; /* opaque; owns the device copies of grid, signs, status */

/* Bytes of one token's codes for these parameters: d_kv / grid_dim * log2(grid_size) / 8 (d_kv/2 * log2(n) / 8
 * for the planar grids; grid_dim 1 and 4: see aquakv_create), or a negative error. */
int aquakv_code_bytes(const aquakv_params* params);

/*
 * Creates a context on the current device.  grid_host: n x 2 floats, the fixed grid of Section 2
 * (a point set tuned for normally distributed vectors), index = code.  signs_k_host /
 * signs_v_host: d_kv values in {+1,-1}, the random diagonal of the randomized Hadamard transform
 * for keys and for values.  All three are copied; the caller may free them after the call.
 * This is the only entry point that allocates device memory (a few KB) and it synchronises the
 * device once.  Errors: INVALID_ARG (NULL, sign not +-1, non-finite grid), UNSUPPORTED, CUDA.
 *
 * Alternative backbone (Section 4.1 "Alternative quantizers": the Quanto-style one, rounding to the nearest
 * level after dividing by the group's largest magnitude, groups of 64 values inside a token; Section 3.2: any Q fits):
 * grid_dim = 1 selects it.  grid_size = 2^b in {4, 8, 16} is then the number of levels PER VALUE (b bits
 * per value): the signed integers -2^(b-1) .. 2^(b-1)-1 times the group scale, scale = absmax / 2^(b-1)
 * stored as fp16, nearest level with the lower one on a tie, saturation at the ends, code = level +
 * 2^(b-1), codes packed LSB-first in value order (d_kv * b / 8 bytes per token); scale_group a power of
 * two from 32 to d_kv; grid_host is not read and may be NULL.  had_block = 1: no rotation, the sign arrays
 * are not read and may be NULL.  had_block = h, a power of two from 64 to d_kv (the appendix' additional
 * results for Section 4.1: a backbone that puts a randomized Hadamard transform in front of ordinary
 * scalar quantization): the residual times the role's signs is rotated by the orthonormal Hadamard
 * matrix in blocks of h values, the ROTATED values are quantized as above (absmax after the rotation;
 * scale_group is independent of h), and the inverse rotates level * scale back and applies the signs again;
 * the sign arrays are then required.
 *
 * Four-dimensional grid (Section 4.1: the 2-bit grid with d = 4, n = 256, for which the paper had no fast GPU
 * kernel, its d being the grid dimension): grid_dim = 4 with grid_size = 256.  grid_host is then 256 x 4
 * floats; every consecutive 4-tuple of rotated normalised values goes to the nearest of the 256 points
 * (lowest index on a tie; a table of candidate lists per cell of [-4, 4)^4, 16 MB, computed on the device
 * by this call, with an exhaustive search for what it does not cover) and takes one byte (d_kv / 4 bytes
 * per token); scale,
 * signs, rotation and reconstruction are those of the planar grids, with the same rules for had_block and
 * scale_group.  It is served like the uniform backbone.
 *
 * A ctx with grid_dim 1 or 4 serves aquakv_encode / aquakv_decode (with predictors: two launches per phase, and
 * Khat is required because the value phase reads it), the *_phase entry points, aquakv_predict,
 * aquakv_fit_predictor and aquakv_gather_rows; the chain, no-allocation and attention entry points return
 * AQUAKV_ERR_UNSUPPORTED.
 */
int aquakv_create(const aquakv_params* params, const float* grid_host, const int8_t* signs_k_host,
                  const int8_t* signs_v_host, aquakv_ctx** out);

/*
 * The host-built cell table that prunes the nearest-point search of Q (Section 2: each pair of
 * rotated values goes to the nearest grid point).  The square [-half_extent, half_extent)^2 is cut
 * into cells_per_side^2 cells; entry [iy*cells_per_side + ix] holds, in bytes 3, 2, 1, 0, the
 * ascending indices of every grid point that is nearest somewhere in that cell (byte 3 the lowest;
 * short lists repeat the last index; at most three distinct ones for grid_size 16, four otherwise).
 * For grid_size 256 a cell with more candidates, up to eight, holds 0xFF000000 + i, a reference to
 * second-level list i (the smaller grids practically never need one and have none):
 * words [cells^2 + 2i, cells^2 + 2i + 1] of the same buffer hold its eight ascending candidates, one
 * per byte, byte 0 of the first word the lowest.  0xFFFFFFFF means "search all points" (cells with
 * still more candidates, and the border cells, which also stand for everything outside the square).
 * The kernels use the same table, so a host test can check that it never excludes the true nearest
 * point.  HOST memory only, no GPU needed.  table == NULL: only report the dimensions; otherwise
 * table_capacity (in words) must be at least cells^2 + AQUAKV_SEARCH_TABLE_LIST_WORDS.
 * second_level_lists (may be NULL) receives the number of second-level lists in use.
 */
#define AQUAKV_SEARCH_TABLE_LIST_WORDS 4096
int aquakv_search_table_host(const float* grid_host, int32_t grid_size, int32_t* cells_per_side,
                             float* half_extent, uint32_t* table, size_t table_capacity,
                             int32_t* second_level_lists);

/* Frees the context's device tables.  NULL is accepted.  Pending work must have completed. */
int aquakv_destroy(aquakv_ctx* ctx);

/*
 * Workspace the caller must provide to the given operation for n_tokens tokens (bytes, 16-byte
 * aligned base).  It is bounded: large calls are processed in token chunks sized so that the
 * intermediate prediction stays resident in the B200's L2 cache.  Returns 0 for n_tokens <= 0,
 * for an unknown op and for AQUAKV_OP_DECODE_ATTN (use aquakv_decode_attn_workspace_bytes).
 */
size_t aquakv_workspace_bytes(const aquakv_ctx* ctx, int64_t n_tokens, int op);

/*
 * Workspace of aquakv_decode_attn for this problem shape (its attention partials depend on the
 * batch and head counts, which aquakv_workspace_bytes does not see).  0 on invalid arguments.
 * The cache is decoded in chunks of up to about 147 K tokens into the workspace (4 * d_kv bytes per
 * token of a chunk; nothing when Khat/Vhat are given) and a second kernel attends over each chunk.  In
 * the fused mode (aquakv_set_attn_mode), with predictors at d_kv = 1024 (Hadamard block = scale group =
 * d_kv), decode and attention run as one kernel: the workspace then holds that kernel's buffers (the
 * prediction ring and, when Khat/Vhat are not requested, rings of three waves of decoded keys and
 * values: about 0.1 GB in all) and one attention partial per 128-token block and query head (about 130
 * bytes per token at 32 query heads).  The returned size covers either mode.
 */
size_t aquakv_decode_attn_workspace_bytes(const aquakv_ctx* ctx, int32_t batch, int64_t ctx_len,
                                          int32_t n_q_heads, int32_t head_dim);

/*
 * The predictor alone (Section 3.2: f_key, f_value are linear regressors; the two predictions
 * of Algorithm 2):  P[t][c] = sum_r x_t[r] * W[c][r] + bias[c]  with x_t = in0[t] (in1 == NULL, W is
 * [d_kv][d_kv]) or the concatenation [in0[t] ; in1[t]] (W is [d_kv][2*d_kv]).  P is fp32
 * [n_tokens, ldP] (ldP % 4 == 0, 16-byte aligned); accumulation is fp32 on the tensor cores.
 * Needs no workspace.
 */
int aquakv_predict(aquakv_ctx* ctx, int64_t n_tokens, const void* in0, const void* in1,
                   int64_t ld_in, const void* W, const float* bias, float* P, int64_t ldP,
                   void* cuda_stream);

#define AQUAKV_ROLE_KEY 0
#define AQUAKV_ROLE_VALUE 1

/*
 * One phase of Algorithm 2 on its own (predict, quantize the residual, reconstruct: for keys or for
 * values), for callers that supply the predictor inputs themselves (e.g. teacher-forced checks):
 *   pred = [in0 ; in1] W^T + bias;  codes,scales = Q(X - pred);  hat = round16(Q^-1(..) + pred).
 * role selects the Hadamard signs (AQUAKV_ROLE_KEY / AQUAKV_ROLE_VALUE).  in1 == NULL: single
 * input, W is [d_kv][d_kv]; otherwise W is [d_kv][2*d_kv].  W == NULL (then in0, in1, bias NULL):
 * no predictor.  hat may be NULL.  Workspace as for AQUAKV_OP_ENCODE (needed only with W).
 */
int aquakv_encode_phase(aquakv_ctx* ctx, int role, int64_t n_tokens, const void* X, int64_t ld_x,
                        const void* in0, const void* in1, int64_t ld_in, const void* W,
                        const float* bias, uint8_t* codes, uint16_t* scales, void* hat,
                        int64_t ld_hat, void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * One phase of Algorithm 3 on its own (for keys or for values):
 *   hat = round16(Q^-1(codes, scales) + [in0 ; in1] W^T + bias).  Arguments as above.
 */
int aquakv_decode_phase(aquakv_ctx* ctx, int role, int64_t n_tokens, const uint8_t* codes,
                        const uint16_t* scales, const void* in0, const void* in1, int64_t ld_in,
                        const void* W, const float* bias, void* hat, int64_t ld_hat,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Algorithm 2 (encode) for one layer and n_tokens tokens:
 *   K_pred = Khat_prev Wk^T + bk;  Kcodes,Kscales = Q(K - K_pred);  Khat = Q^-1(..) + K_pred;
 *   V_pred = [Vhat_prev ; Khat] Wv^T + bv;  Vcodes,Vscales = Q(V - V_pred);  Vhat = Q^-1(..) + V_pred.
 * The reconstructions Khat/Vhat (rounded once to the 16-bit type) are what Algorithm 4's cache update
 * obtains by decoding the fresh codes again; here they are by-products.  Khat, Vhat may be NULL
 * (not written; Khat is then kept in the workspace for the value predictor).  Outputs must not
 * alias inputs.  K,V: [n_tokens, ld_kv]; *_prev: [n_tokens, ld_prev]; Khat,Vhat: [n_tokens, ld_hat].
 */
int aquakv_encode(aquakv_ctx* ctx, int64_t n_tokens,
                  const void* K, const void* V, int64_t ld_kv,
                  const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev,
                  const void* Wk, const void* Wv, const float* bk, const float* bv,
                  uint8_t* Kcodes, uint16_t* Kscales, uint8_t* Vcodes, uint16_t* Vscales,
                  void* Khat, void* Vhat, int64_t ld_hat,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Algorithm 3 (decode) for one layer:
 *   Khat = Q^-1(Kcodes,Kscales) + Khat_prev Wk^T + bk;
 *   Vhat = Q^-1(Vcodes,Vscales) + [Vhat_prev ; Khat] Wv^T + bv,
 * each rounded once to the 16-bit type.  On the same device, with the same arguments, Khat/Vhat
 * are bit-identical to those aquakv_encode produced (the reconstruction of Algorithm 2 and the decode of Algorithm 3
 * are the same expression).  Khat and Vhat are required.
 */
int aquakv_decode(aquakv_ctx* ctx, int64_t n_tokens,
                  const uint8_t* Kcodes, const uint16_t* Kscales,
                  const uint8_t* Vcodes, const uint16_t* Vscales,
                  const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev,
                  const void* Wk, const void* Wv, const float* bk, const float* bv,
                  void* Khat, void* Vhat, int64_t ld_hat,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Algorithm 4's loop over layers for SMALL calls -- a decode step of a batch of sequences, a short
 * prompt -- in ONE launch: Algorithm 2 (encode_chain) or Algorithm 3 (decode_chain) for n_layers
 * consecutive layers, each layer's predictors reading the previous layer's reconstruction (the layer loop of
 * Algorithm 4; Section 3.3).  A per-layer call of a few tokens is bound by launch and hand-off
 * latency and by a handful of SMs streaming the adapter weights; here every SM streams a share of
 * the weights, the key chain runs ahead of the value chain, and the layers hand over through
 * counters in device memory.
 *
 * Per-layer arguments are HOST arrays of n_layers DEVICE pointers (read during the call only):
 * K[l], V[l] (encode), Wk[l], Wv[l] (both NULL: layer l has no predictor, e.g. the model's first
 * layer), bk[l], bv[l] (the arrays or single entries may be NULL), codes and scales, and the optional
 * outputs Khat[l], Vhat[l] ([n_tokens, ld_hat]; arrays or entries NULL: that layer's reconstruction
 * stays in the workspace; give both or neither of a layer).  If layer 0 has a predictor, Khat_init /
 * Vhat_init ([n_tokens, ld_init]) are the reconstruction of the layer before it; otherwise they must
 * be NULL.  n_layers <= 128 (AQUAKV_ERR_TOO_LARGE beyond).  Up to 2048 tokens the call is one launch of
 * the chain kernel; d_kv = 1024 then requires Hadamard block = scale group = 1024 (AQUAKV_ERR_UNSUPPORTED
 * otherwise).  Workspace: aquakv_chain_workspace_bytes.
 *
 * LARGE calls (n_tokens > 2048; d_kv = 1024 with Hadamard block = scale group = 1024 only,
 * AQUAKV_ERR_TOO_LARGE otherwise: use the per-layer calls) run the persistent layer kernel of
 * aquakv_encode / aquakv_decode on up to 24 consecutive predicted layers per launch: no barrier between
 * the layers, a layer's first token blocks start while the previous layer's last ones are being
 * finished, which removes the pipeline fill and drain that every per-layer launch pays (about 60 us of
 * an encode and 20 us of a decode launch).  Every layer then needs its Khat[l] / Vhat[l] from the
 * caller (AQUAKV_ERR_INVALID_ARG otherwise); a layer may reuse the buffers of the layer TWO before it
 * (two alternating pairs suffice), not those of the layer before it, which it reads.  Results are
 * bit-identical to the per-layer calls.
 *
 * Results satisfy the same bounds against the definition as the per-layer calls; the fp32 prediction
 * is summed in a different order, so a reconstruction can differ from aquakv_encode / aquakv_decode in
 * the last bit of the 16-bit type.  decode_chain reproduces encode_chain's reconstructions bit for bit.
 * Calls on one context must not overlap on the device, and no other kernel may occupy the device's
 * SMs while a chain call runs (its CTAs wait for one another; a wait that finds no partner expires
 * after two seconds with AQUAKV_ERR_TIMEOUT in the status word).
 */
size_t aquakv_chain_workspace_bytes(const aquakv_ctx* ctx, int64_t n_tokens, int32_t n_layers);
int aquakv_encode_chain(aquakv_ctx* ctx, int64_t n_tokens, int32_t n_layers,
                        const void* const* K, const void* const* V, int64_t ld_kv,
                        const void* Khat_init, const void* Vhat_init, int64_t ld_init,
                        const void* const* Wk, const void* const* Wv,
                        const float* const* bk, const float* const* bv,
                        uint8_t* const* Kcodes, uint16_t* const* Kscales,
                        uint8_t* const* Vcodes, uint16_t* const* Vscales,
                        void* const* Khat, void* const* Vhat, int64_t ld_hat,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);
int aquakv_decode_chain(aquakv_ctx* ctx, int64_t n_tokens, int32_t n_layers,
                        const uint8_t* const* Kcodes, const uint16_t* const* Kscales,
                        const uint8_t* const* Vcodes, const uint16_t* const* Vscales,
                        const void* Khat_init, const void* Vhat_init, int64_t ld_init,
                        const void* const* Wk, const void* const* Wv,
                        const float* const* bk, const float* const* bv,
                        void* const* Khat, void* const* Vhat, int64_t ld_hat,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * aquakv_decode for callers that cannot allocate device memory and therefore have no workspace to
 * hand over.  (The paper has no counterpart: this is a packaging variant of aquakv_decode, same
 * arithmetic, same kernels.)  Who needs it: a decode step running inside a region where
 * cudaMalloc is off limits -- a plugin that is given device buffers for its inputs and outputs only,
 * an inference server whose memory pool is frozen after start-up, a real-time loop that must not
 * take the allocator's locks or its implicit device synchronisation.
 *
 * The fp32 prediction that aquakv_decode keeps in the caller's workspace lives here in a fixed
 * array inside the library image: AQUAKV_NOALLOC_MAX_TOKENS * 1024 * 4 bytes = 4 MiB of device
 * memory, reserved on every GPU that loads the library for as long as the process lives.  The
 * call itself performs no cudaMalloc / cudaFree and calls no routine that allocates.
 *
 *   - n_tokens > AQUAKV_NOALLOC_MAX_TOKENS returns AQUAKV_ERR_TOO_LARGE and launches nothing;
 *     split larger batches into several calls on the same stream.
 *   - The first call on a device looks up the array's device address (once per device, with that
 *     device current, which must be the context's device).  Make that first call during start-up,
 *     before any stream capture; later calls only launch kernels.
 *   - Every call on a device uses the same array.  Calls issued to one stream are ordered and
 *     safe; calls that can overlap on the GPU (different streams, different contexts or threads)
 *     race on it and produce garbage.  The array keeps whatever the last call left there; nothing
 *     in it needs to start at zero because each call overwrites every row it later reads.
 *   - All other arguments, results (bit-identical to aquakv_decode) and errors are those of
 *     aquakv_decode.
 */
#define AQUAKV_NOALLOC_MAX_TOKENS 1024
int aquakv_decode_noalloc(aquakv_ctx* ctx, int64_t n_tokens,
                          const uint8_t* Kcodes, const uint16_t* Kscales,
                          const uint8_t* Vcodes, const uint16_t* Vscales,
                          const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev,
                          const void* Wk, const void* Wv, const float* bk, const float* bv,
                          void* Khat, void* Vhat, int64_t ld_hat, void* cuda_stream);

/*
 * Algorithm 3 fused with the attention read of Algorithm 4 for single-token queries:
 * decodes `batch` sequences of `ctx_len` cached tokens each (token index = b*ctx_len + t,
 * n_tokens = batch*ctx_len) and computes, per sequence b and query head qh,
 *   out[b][qh] = softmax_t(softmax_scale * q[b][qh] . Khat[b,t][kvh]) . Vhat[b,t][kvh],
 * kvh = qh / (n_q_heads / n_kv_heads) (grouped-query attention), accumulating in fp32.
 * n_kv_heads * head_dim must equal d_kv; head_dim must be 64 or 128; n_q_heads a multiple of
 * n_kv_heads with n_q_heads/n_kv_heads <= 8.  q, out: [batch][n_q_heads][head_dim] 16-bit,
 * contiguous.  lse: optional fp32 [batch][n_q_heads] log-sum-exp of the scaled scores (NULL =
 * not written).  Khat, Vhat: optional outputs [n_tokens, ld_hat] for the next layer's decode.
 *
 * Two ways to run it (aquakv_set_attn_mode; the results agree to the rounding of the fp32 partial sums):
 *   AQUAKV_ATTN_SPLIT (default): the layer kernel decodes a chunk of tokens (predictions on the tensor
 *     cores, row warps reconstruct the rows into Khat/Vhat or the workspace), a split-KV kernel attends
 *     over the chunk's rows right behind it and a small third kernel merges the partials of each sequence.
 *   AQUAKV_ATTN_FUSED: with predictors at d_kv = 1024 and Hadamard block = scale group = d_kv (the paper's
 *     setting) ONE kernel: while the tensor cores form the predictions and the row warps reconstruct
 *     token rows, attention warps of the same kernel take every 128-token block as soon as its keys and
 *     values exist and reduce it to per-block softmax partials; the merge kernel follows.  Without
 *     Khat/Vhat the decoded rows then live only in a ring of three waves of tokens in the workspace and
 *     never reach HBM.  Other shapes and layer 0 fall back to the split form.
 * The split form is the default because it is the faster one on B200: the row warps are what bounds the
 * layer kernel, and the fused kernel has to give four of its ten row-warp slots per CTA to the attention
 * warps (0.325 ms against 0.251 ms for 32768 tokens, 8.6 ms against 7.6 ms for 32 x 32768 with Khat/Vhat
 * written in both).
 */
int aquakv_set_attn_mode(aquakv_ctx* ctx, int mode); /* INVALID_ARG for an unknown mode; takes effect on the next call */
int aquakv_decode_attn(aquakv_ctx* ctx, int32_t batch, int64_t ctx_len,
                       int32_t n_q_heads, int32_t n_kv_heads, int32_t head_dim, float softmax_scale,
                       const void* q,
                       const uint8_t* Kcodes, const uint16_t* Kscales,
                       const uint8_t* Vcodes, const uint16_t* Vscales,
                       const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev,
                       const void* Wk, const void* Wv, const float* bk, const float* bv,
                       void* out, float* lse,
                       void* Khat, void* Vhat, int64_t ld_hat,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * The same with the cache policy of Section 3.3 / Section 4.1 around it: the first four tokens (the attention
 * sinks) and a buffer of the 128 newest tokens stay uncompressed, and every query attends to both
 * the compressed cache and those rows.  K16 / V16: [batch][n_uncompressed][ld16] 16-bit rows of the
 * ctx's type (device, 16-byte aligned, ld16 >= d_kv and a multiple of 8), each sequence's uncompressed
 * rows in any order (attention does not depend on it; position encoding is the caller's business, as in
 * aquakv_decode_attn).  Their split-KV partials are formed by the library's attention kernel and merged
 * with the partials of the compressed cache in fp32 before the single rounding of `out`, so the result
 * is the attention over the concatenation [compressed ; uncompressed] (the attention read of Algorithm 4 with
 * the buffered rows appended to the decoded ones).  ctx_len may be 0 (nothing compressed yet: the cache
 * pointers are then ignored), n_uncompressed may be 0 (identical to aquakv_decode_attn); both 0 does
 * nothing.  Workspace: aquakv_decode_attn_buffered_workspace_bytes.  Everything else as aquakv_decode_attn.
 */
size_t aquakv_decode_attn_buffered_workspace_bytes(const aquakv_ctx* ctx, int32_t batch, int64_t ctx_len,
                                                   int64_t n_uncompressed, int32_t n_q_heads, int32_t head_dim);
int aquakv_decode_attn_buffered(aquakv_ctx* ctx, int32_t batch, int64_t ctx_len, int32_t n_q_heads,
                                int32_t n_kv_heads, int32_t head_dim, float softmax_scale, const void* q,
                                const uint8_t* Kcodes, const uint16_t* Kscales, const uint8_t* Vcodes,
                                const uint16_t* Vscales, const void* Khat_prev, const void* Vhat_prev,
                                int64_t ld_prev, const void* Wk, const void* Wv, const float* bk,
                                const float* bv, const void* K16, const void* V16, int64_t n_uncompressed,
                                int64_t ld16, void* out, float* lse, void* Khat, void* Vhat, int64_t ld_hat,
                                void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Rotary position encoding on the fly (Section 3.3 "Positional embeddings": keys are compressed BEFORE
 * RoPE, where the predictors work better, so the reconstructed keys are rotated when the block attends to
 * them).  For a head of head_dim values and a token at position pos, frequency i < head_dim/2 has the
 * angle pos * theta_base^(-2 i / head_dim) and rotates the pair (x[i], x[i + head_dim/2]):
 *   y[i] = x[i] cos - x[i + head_dim/2] sin,   y[i + head_dim/2] = x[i + head_dim/2] cos + x[i] sin
 * (the half-split pairing of the Llama-family models the paper evaluates), computed in fp32 and rounded
 * once to the ctx's 16-bit type; values are not rotated and q must arrive rotated by its own position.
 *
 * aquakv_rope_table fills table[pos][i] = (cos, sin) of that angle as fp32 pairs, evaluated in double
 * precision, for pos < n_positions (device, 16-byte aligned, n_positions * head_dim/2 * 2 floats; owned by
 * the caller, reusable by every layer and call with the same head_dim and theta_base).  head_dim 64 or 128,
 * theta_base > 1 (10000 in the original formulation, 500000 for Llama 3).  Errors: INVALID_ARG,
 * UNSUPPORTED, ALIGNMENT, CUDA.
 *
 * aquakv_decode_attn_rope is aquakv_decode_attn_buffered with the keys rotated: compressed token t of
 * every sequence sits at position pos0 + t, uncompressed row r of every sequence at pos16[r] (device,
 * n_uncompressed entries, shared by the sequences of the batch; may be NULL when n_uncompressed is 0).
 * The decoded rows returned in Khat stay un-rotated (they feed the next layer's predictor); the attention
 * reads rotated copies that live in the workspace, so decode, rotation and attention are separate
 * kernels here for every shape.  pos0 + ctx_len must not exceed rope_positions (INVALID_ARG); an entry of
 * pos16 outside the table sets the status word to AQUAKV_ERR_INVALID_ARG and that key row counts as zero.
 * Workspace: aquakv_decode_attn_rope_workspace_bytes.  Everything else as aquakv_decode_attn_buffered.
 */
int aquakv_rope_table(aquakv_ctx* ctx, int32_t head_dim, double theta_base, int64_t n_positions, float* table,
                      void* cuda_stream);
size_t aquakv_decode_attn_rope_workspace_bytes(const aquakv_ctx* ctx, int32_t batch, int64_t ctx_len,
                                               int64_t n_uncompressed, int32_t n_q_heads, int32_t head_dim);
int aquakv_decode_attn_rope(aquakv_ctx* ctx, int32_t batch, int64_t ctx_len, int32_t n_q_heads,
                            int32_t n_kv_heads, int32_t head_dim, float softmax_scale, const void* q,
                            const uint8_t* Kcodes, const uint16_t* Kscales,
                            const uint8_t* Vcodes, const uint16_t* Vscales,
                            const void* Khat_prev, const void* Vhat_prev, int64_t ld_prev,
                            const void* Wk, const void* Wv, const float* bk, const float* bv,
                            const void* K16, const void* V16, int64_t n_uncompressed, int64_t ld16,
                            const float* rope_table, int64_t rope_positions, int64_t pos0, const int32_t* pos16,
                            void* out, float* lse,
                            void* Khat, void* Vhat, int64_t ld_hat,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Row gather for compressing a subset of the tokens (Section 4.3: a pruning policy such as H2O
 * selects the tokens to keep, "and [we] apply AQUA-KV compression [to] those tokens"): dst row i =
 * src row idx[i], 16-bit rows of d_kv values; the compact rows then go through aquakv_encode like any
 * other batch (their previous-layer reconstructions are compact in the same order).  idx is a device
 * array of n_rows int64 values in [0, n_src_rows), or NULL for the identity (a plain row copy, which is
 * how an unquantised first layer - the Qwen-2.5 setting of the appendix tables - enters the chain's
 * buffers).  src / dst: device, 16-byte aligned, ld multiples of 8 and >= d_kv, no overlap.
 * Asynchronous on cuda_stream.  An index out of range zero-fills its row and is reported by
 * aquakv_poll_status as AQUAKV_ERR_INVALID_ARG.                                                       */
int aquakv_gather_rows(aquakv_ctx* ctx, int64_t n_rows, const int64_t* idx, int64_t n_src_rows, const void* src,
                       int64_t ld_src, void* dst, int64_t ld_dst, void* cuda_stream);

/* ---------------------------------------------------------------------------------------------
 * Calibration of one predictor (Algorithm 1, its two least-squares fits; Section 3.2: linear regressors
 * trained in closed form; Appendix A: the regularizer rate is 1e-3):
 *
 *   W = argmin_W || [in0 ; in1] W^T (+ b) - target ||^2 + rate * trace(X^T X) / n_in * ||W||^2
 *
 * over n_tokens calibration tokens.  in0 / in1 (in1 may be NULL: one input tensor, the key predictor;
 * two: the value predictor on [V_old ; K_rec]) and target are 16-bit device rows [n_tokens][ld],
 * ld_in / ld_target >= d_kv and multiples of 8, pointers 16-byte aligned.  rate >= 0.  fit_bias != 0
 * fits an intercept (inputs and targets centred; b = mean(target) - mean(X) W^T) into bias_out
 * (fp32 [d_kv], device); otherwise bias_out is not touched and may be NULL.  W_out receives the
 * matrix rounded once to the ctx's 16-bit type, laid out [d_kv][n_in * d_kv] like every adapter of this
 * library; W32_out (may be NULL) the same matrix in fp32.  The normal equations are formed on the
 * tensor cores with fp32 accumulation and solved by a Cholesky factorisation in double precision,
 * all inside this library's kernels.  Algorithm 1's loop over layers (fit the key predictor, encode
 * the keys, fit the value predictor on the reconstructed keys, encode the values, hand the
 * reconstructions to the next layer) is made of this call and aquakv_encode_phase.
 * Workspace: aquakv_fit_workspace_bytes(ctx, n_tokens, n_inputs) bytes of device memory, owned by the
 * caller, not read after the call's kernels finish.  Asynchronous on cuda_stream.  Errors: the usual
 * argument codes and nothing launched; a matrix that is not positive definite (possible only with
 * rate == 0 and dependent inputs) is reported by aquakv_poll_status as AQUAKV_ERR_NUMERIC.
 * d_kv must be a multiple of 256 (AQUAKV_ERR_UNSUPPORTED otherwise).                                */
size_t aquakv_fit_workspace_bytes(const aquakv_ctx* ctx, int64_t n_tokens, int32_t n_inputs);
int aquakv_fit_predictor(aquakv_ctx* ctx, int64_t n_tokens, const void* in0, const void* in1, int64_t ld_in,
                         const void* target, int64_t ld_target, double rate, int fit_bias, void* W_out,
                         float* W32_out, float* bias_out, void* workspace, size_t workspace_bytes,
                         void* cuda_stream);

/*
 * Synchronises `cuda_stream` and returns the context's device status word: AQUAKV_OK, or
 * AQUAKV_ERR_TIMEOUT if a bounded wait inside a kernel (on a TMA or tensor-core completion
 * barrier) expired since the last poll, in which case that call's outputs are invalid.  The word
 * is cleared by the poll.  AQUAKV_ERR_CUDA if the stream reports an error.
 */
int aquakv_poll_status(aquakv_ctx* ctx, void* cuda_stream);

/*
 * Failure-path check of the device-side waits.  Every wait inside the kernels (on a TMA or
 * tensor-core completion barrier, on another CTA's progress counter) gives up after a time limit,
 * records AQUAKV_ERR_TIMEOUT in the context's status word and lets the kernel return.  This call
 * launches one warp that waits, with a limit of limit_ns nanoseconds (0 < limit_ns <= 2e9), on a
 * barrier that nothing arrives on, so the next aquakv_poll_status returns AQUAKV_ERR_TIMEOUT (and
 * clears it) while the context stays usable.  Diagnostic only; not part of the paper's method.
 */
int aquakv_selftest_bounded_wait(aquakv_ctx* ctx, int64_t limit_ns, void* cuda_stream);

/* Number of kernels this context has launched since creation (for benchmarks' bookkeeping). */
int64_t aquakv_launch_count(const aquakv_ctx* ctx);

/*
 * Optional per-kernel timing for benchmarks.  While enabled, every kernel launch of this context
 * is bracketed by a pair of CUDA events on the launching stream (up to 8192 launches; later ones
 * are not recorded).  aquakv_profile_enable(ctx, 1) creates the events on first use (do this
 * outside stream capture) and clears the record; (ctx, 0) stops recording.
 * aquakv_profile_read waits for the recorded launches of one kernel class and returns their
 * number and summed device time.  Not part of the paper's method: measurement support only.
 */
#define AQUAKV_KERNEL_PREDICT 0     /* tcgen05 predictor GEMM                    */
#define AQUAKV_KERNEL_ENCODE_ROWS 1 /* residual, scale, rotation, search, pack   */
#define AQUAKV_KERNEL_DECODE_ROWS 2 /* unpack, gather, inverse rotation, add-back */
#define AQUAKV_KERNEL_ATTN 3        /* split-KV attention partials and combine   */
#define AQUAKV_KERNEL_LAYER 4       /* fused layer kernel: predictor GEMMs + row work */
#define AQUAKV_KERNEL_CHAIN 5       /* all layers of a small call in one launch       */
#define AQUAKV_KERNEL_FIT 6         /* calibration: transposes, normal equations, solve */
int aquakv_profile_enable(aquakv_ctx* ctx, int enable);
int aquakv_profile_read(aquakv_ctx* ctx, int kernel_class, int64_t* launches, double* total_ms);

/* Static, human-readable name of a status code. */
const char* aquakv_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* AQUAKV_H_ */
