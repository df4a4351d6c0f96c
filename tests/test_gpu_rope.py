"""Rotary position encoding applied on the fly to cached pre-RoPE keys (Section 3.3 "Positional
embeddings"): the table kernel against the oracle's double-precision angles, the rotated attention
against the oracle's (rotation in double, one rounding to the cache type, attention in double) over
the SAME un-rotated rows the kernel decoded (teacher-forced like the other attention tests: 2e-3 of
the head's largest output or a one-ulp flip of the 16-bit output), and the error paths."""
import dataclasses
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import rope as orope
from paper_2501_19392_b200 import synth
from parity import gpu_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make(shape, n=16):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(n, seed=7, n_samples=1 << 14, iters=25)
    return api.Codec(shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype,
                     synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12))


@pytest.mark.parametrize("hd,base,n_pos", [(128, 500000.0, 5000), (64, 10000.0, 70000)])
def test_table_is_the_double_precision_cos_sin_rounded_to_fp32(hd, base, n_pos):
    codec = make(synth.CONFIGS[1])
    table = codec.rope_table(hd, base, n_pos, DEV)
    torch.cuda.synchronize()
    a = orope.angles(np.arange(n_pos), hd, base)
    got = table.cpu().numpy().astype(np.float64)
    assert got.shape == (n_pos, hd // 2, 2)
    # fp32 rounding of a value in [-1, 1] is within 2^-24; the device's double sincos / pow add ~1e-11 at angle 7e4
    assert np.abs(got[:, :, 0] - np.cos(a)).max() <= 2.0 ** -24 + 1e-10
    assert np.abs(got[:, :, 1] - np.sin(a)).max() <= 2.0 ** -24 + 1e-10
    assert np.array_equal(got[0, :, 0], np.ones(hd // 2)) and not got[0, :, 1].any()


def rope_attn_check(out, lse, q, rows_k, rows_v, positions, shape, scale, base, batch=1):
    n = rows_k.shape[0] // batch
    ref, ref_lse = orope.attention_rope(shape.dtype, batch, n, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                                        scale, synth.to_bits(q.cpu()), rows_k, rows_v, positions, base)
    o = out.to(torch.float64).cpu().numpy()
    ref_bits = synth.to_bits(torch.from_numpy(ref).to(out.dtype)).astype(np.int64)
    adjacent = np.abs(gpu_bits(out).astype(np.int64) - ref_bits) <= 1
    denom = np.abs(ref).max(axis=-1, keepdims=True)
    assert np.all((np.abs(o - ref) <= 2e-3 * denom) | adjacent)
    if lse is not None:
        assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 2e-4
    return ref


CASES = [  # config, ctx, n16, with_pred, pos0, dtype, theta
    (5, 300, 132, True, 4, oracle.BF16, 500000.0),       # d_kv 1024: the fused shape takes the two-kernel path here
    (5, 2500, 0, True, 0, oracle.BF16, 500000.0),        # several attention blocks, a ragged tail
    (5, 0, 77, False, 0, oracle.BF16, 10000.0),          # nothing compressed yet
    (5, 384, 4, False, 4, oracle.F16, 10000.0),          # layer 0 (no predictor), fp16 cache
    (7, 1000, 1500, True, 100, oracle.BF16, 1000000.0),  # d_kv 512, more uncompressed rows than one split
]


@pytest.mark.parametrize("cfg,ctx,n16,with_pred,pos0,dtype,base", CASES)
def test_rotated_attention_matches_the_oracle(cfg, ctx, n16, with_pred, pos0, dtype, base):
    from paper_2501_19392_b200 import api
    shape = dataclasses.replace(synth.CONFIGS[cfg], n_tokens=max(ctx, 1), n_layers=2, batch=1, dtype=dtype)
    codec = make(shape)
    d, hd = shape.d_kv, shape.head_dim
    scale = 1.0 / math.sqrt(hd)
    q = synth.random_16bit((1, shape.n_q_heads, hd), dtype, 1, device=DEV)
    K16 = synth.random_16bit((1, max(n16, 1), d), dtype, 2, device=DEV)[:, :n16] if n16 else None
    V16 = synth.random_16bit((1, max(n16, 1), d), dtype, 3, device=DEV)[:, :n16] if n16 else None
    # uncompressed rows: a few sinks at positions 0.., the rest after the compressed tokens, in a shuffled order
    rng = np.random.default_rng(ctx + n16)
    pos16_np = np.concatenate([np.arange(min(4, n16)), pos0 + ctx + np.arange(max(n16 - 4, 0))])[:n16]
    pos16_np = rng.permutation(pos16_np).astype(np.int32)
    pos16 = torch.from_numpy(pos16_np).to(DEV) if n16 else None
    n_pos = int(max(pos0 + ctx, pos16_np.max() + 1 if n16 else 0)) + 3
    table = codec.rope_table(hd, base, n_pos, DEV)
    if ctx:
        rc = synth.random_cache(dataclasses.replace(shape, n_tokens=ctx), seed=4, device=DEV, n_layers=1)
        ad = synth.random_adapters(shape, seed=5, device=DEV)
        Kp = synth.random_16bit((ctx, d), dtype, 6, device=DEV) if with_pred else None
        Vp = synth.random_16bit((ctx, d), dtype, 7, device=DEV) if with_pred else None
        Wk, Wv = (ad.Wk[1], ad.Wv[1]) if with_pred else (None, None)
        Kh = torch.empty((ctx, d), dtype=codec.torch_dtype, device=DEV)
        Vh = torch.empty_like(Kh)
        out, lse = codec.decode_attn_rope(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx,
                                          shape.n_kv_heads, scale, table, pos0, K16, V16, pos16, Kp, Vp, Wk, Wv,
                                          Khat=Kh, Vhat=Vh, want_lse=True)
        # the returned rows are the un-rotated reconstructions: those of the plain entry point
        Kh2, Vh2 = torch.empty_like(Kh), torch.empty_like(Vh)
        codec.decode_attn(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx, shape.n_kv_heads, scale,
                          Kp, Vp, Wk, Wv, Khat=Kh2, Vhat=Vh2)
        assert torch.equal(Kh, Kh2) and torch.equal(Vh, Vh2)
        # without the caller's row buffers the result is the same
        out3, _ = codec.decode_attn_rope(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx,
                                         shape.n_kv_heads, scale, table, pos0, K16, V16, pos16, Kp, Vp, Wk, Wv)
        assert torch.equal(out, out3)
        rows_k = np.concatenate([gpu_bits(Kh)] + ([gpu_bits(K16[0])] if n16 else []), axis=0)
        rows_v = np.concatenate([gpu_bits(Vh)] + ([gpu_bits(V16[0])] if n16 else []), axis=0)
    else:
        empty_c = torch.empty((0, codec.code_bytes), dtype=torch.uint8, device=DEV)
        empty_s = torch.empty((0, codec.n_groups), dtype=torch.float16, device=DEV)
        out, lse = codec.decode_attn_rope(q, empty_c, empty_s, empty_c, empty_s, 0, shape.n_kv_heads, scale, table,
                                          pos0, K16, V16, pos16, want_lse=True)
        rows_k, rows_v = gpu_bits(K16[0]), gpu_bits(V16[0])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    positions = np.concatenate([pos0 + np.arange(ctx), pos16_np.astype(np.int64)])
    ref = rope_attn_check(out, lse, q, rows_k, rows_v, positions, shape, scale, base)
    # the rotation matters: the oracle without it is far away
    plain, _ = oracle.attention(dtype, 1, rows_k.shape[0], shape.n_q_heads, shape.n_kv_heads, hd, scale,
                                synth.to_bits(q.cpu()), rows_k, rows_v)
    assert np.abs(plain - ref).max() > 20 * 2e-3 * np.abs(ref).max()


def test_batch_of_sequences_shares_the_positions():
    from paper_2501_19392_b200 import api
    B, ctx, n16, pos0, base = 3, 700, 9, 4, 500000.0
    shape = dataclasses.replace(synth.CONFIGS[5], n_tokens=B * ctx, n_layers=2, batch=B)
    codec = make(shape)
    d, hd, dt = shape.d_kv, shape.head_dim, shape.dtype
    scale = 1.0 / math.sqrt(hd)
    q = synth.random_16bit((B, shape.n_q_heads, hd), dt, 1, device=DEV)
    K16 = synth.random_16bit((B, n16, d), dt, 2, device=DEV)
    V16 = synth.random_16bit((B, n16, d), dt, 3, device=DEV)
    pos16_np = np.concatenate([np.arange(4), pos0 + ctx + np.arange(n16 - 4)]).astype(np.int32)
    table = codec.rope_table(hd, base, pos0 + ctx + n16, DEV)
    rc = synth.random_cache(shape, seed=4, device=DEV, n_layers=1)
    ad = synth.random_adapters(shape, seed=5, device=DEV)
    Kp = synth.random_16bit((B * ctx, d), dt, 6, device=DEV)
    Vp = synth.random_16bit((B * ctx, d), dt, 7, device=DEV)
    Kh = torch.empty((B * ctx, d), dtype=codec.torch_dtype, device=DEV)
    Vh = torch.empty_like(Kh)
    out, lse = codec.decode_attn_rope(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx, shape.n_kv_heads,
                                      scale, table, pos0, K16, V16, torch.from_numpy(pos16_np).to(DEV), Kp, Vp,
                                      ad.Wk[1], ad.Wv[1], Khat=Kh, Vhat=Vh, want_lse=True)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    positions = np.concatenate([pos0 + np.arange(ctx), pos16_np.astype(np.int64)])
    for b in range(B):
        rows_k = np.concatenate([gpu_bits(Kh[b * ctx:(b + 1) * ctx]), gpu_bits(K16[b])], axis=0)
        rows_v = np.concatenate([gpu_bits(Vh[b * ctx:(b + 1) * ctx]), gpu_bits(V16[b])], axis=0)
        rope_attn_check(out[b:b + 1], lse[b:b + 1], q[b:b + 1], rows_k, rows_v, positions, shape, scale, base)


def test_full_context_across_a_chunk_border():
    """6 sequences x 32768 tokens (196608 cached tokens: two decode chunks, the border inside the fifth
    sequence), 32 query heads / 8 KV heads x 128, predictors: the oracle attends over the decoded rows of the
    sequence that straddles the border and of the last one."""
    from paper_2501_19392_b200 import api
    B, ctx, pos0, base = 6, 32768, 4, 500000.0
    shape = dataclasses.replace(synth.CONFIGS[5], n_tokens=B * ctx, n_layers=2, batch=B)
    codec = make(shape)
    d, hd, dt = shape.d_kv, shape.head_dim, shape.dtype
    scale = 1.0 / math.sqrt(hd)
    q = synth.random_16bit((B, shape.n_q_heads, hd), dt, 1, device=DEV)
    table = codec.rope_table(hd, base, pos0 + ctx, DEV)
    rc = synth.random_cache(shape, seed=4, device=DEV, n_layers=1)
    ad = synth.random_adapters(shape, seed=5, device=DEV)
    Kp = synth.random_16bit((B * ctx, d), dt, 6, device=DEV)
    Vp = synth.random_16bit((B * ctx, d), dt, 7, device=DEV)
    Kh = torch.empty((B * ctx, d), dtype=codec.torch_dtype, device=DEV)
    Vh = torch.empty_like(Kh)
    out, lse = codec.decode_attn_rope(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx, shape.n_kv_heads,
                                      scale, table, pos0, None, None, None, Kp, Vp, ad.Wk[1], ad.Wv[1], Khat=Kh, Vhat=Vh,
                                      want_lse=True)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    positions = pos0 + np.arange(ctx)
    for b in (4, B - 1):
        sl = slice(b * ctx, (b + 1) * ctx)
        rope_attn_check(out[b:b + 1], lse[b:b + 1], q[b:b + 1], gpu_bits(Kh[sl]), gpu_bits(Vh[sl]), positions, shape,
                        scale, base)


def test_error_paths():
    from paper_2501_19392_b200 import api
    shape = dataclasses.replace(synth.CONFIGS[5], n_tokens=256, n_layers=2, batch=1)
    codec = make(shape)
    d, hd, dt = shape.d_kv, shape.head_dim, shape.dtype
    for bad in (dict(hd=96), dict(base=1.0), dict(base=float("nan"))):
        with pytest.raises(api.AquaKVError) as e:
            codec.rope_table(bad.get("hd", 128), bad.get("base", 1e4), 16, DEV)
        assert e.value.status == (-2 if "hd" in bad else -1)
    table = codec.rope_table(hd, 1e4, 300, DEV)
    q = synth.random_16bit((1, shape.n_q_heads, hd), dt, 1, device=DEV)
    rc = synth.random_cache(shape, seed=4, device=DEV, n_layers=1)
    args = (q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], 256, shape.n_kv_heads, 0.1, table)
    with pytest.raises(api.AquaKVError) as e:          # compressed positions run past the table
        codec.decode_attn_rope(*args, pos0=45)
    assert e.value.status == -1
    K16 = synth.random_16bit((1, 5, d), dt, 2, device=DEV)
    with pytest.raises(api.AquaKVError) as e:          # uncompressed rows without positions
        codec.decode_attn_rope(*args, pos0=0, K16=K16, V16=K16)
    assert e.value.status == -1
    with pytest.raises(api.AquaKVError) as e:          # workspace too small: nothing is launched
        codec.decode_attn_rope(*args, pos0=0, workspace=torch.empty(1024, dtype=torch.uint8, device=DEV))
    assert e.value.status == -4
    assert codec.poll_status() == 0
    # a position of an uncompressed row outside the table: flagged by the kernel, the context stays usable
    pos16 = torch.tensor([0, 1, 2, 3, 300], dtype=torch.int32, device=DEV)
    codec.decode_attn_rope(*args, pos0=0, K16=K16, V16=K16, pos16=pos16)
    torch.cuda.synchronize()
    assert codec.poll_status() == -1
    assert codec.poll_status() == 0
    codec.decode_attn_rope(*args, pos0=0, K16=K16, V16=K16, pos16=pos16 - 1 + (pos16 == 0).int())
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
