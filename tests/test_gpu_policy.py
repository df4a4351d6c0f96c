"""Cache policy around the codec (Section 3.3 / Section 4.1: attention sinks and a recent-token buffer in
16 bits, a 4-bit first layer, chunks compressed when the buffer overflows) and the attention over
[compressed | sinks | recent] (aquakv_decode_attn_buffered).

The attention arithmetic is checked teacher-forced, like the other attention tests: the oracle attends
over the SAME rows the kernel attended over (the decoded compressed rows it returns, then the
uncompressed rows), bar 2e-3 of the head's largest output or a one-ulp flip of the 16-bit output.  The
policy itself is plumbing: the cache it builds must equal encoding the same chunks directly."""
import dataclasses
import math

import numpy as np
import pytest
import torch

import oracle
from paper_2501_19392_b200 import synth
from parity import gpu_bits

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make(shape, n):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(n, seed=7, n_samples=1 << 14, iters=25)
    return api.Codec(shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype,
                     synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12))


def attn_check(out, q, rows_k, rows_v, shape, scale):
    """out [1, n_q, hd] against the oracle's attention over the given 16-bit rows (numpy bits [n, d])."""
    n = rows_k.shape[0]
    ref, _ = oracle.attention(shape.dtype, 1, n, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, scale,
                              synth.to_bits(q.cpu()), rows_k, rows_v)
    o = out.to(torch.float64).cpu().numpy()
    ref_bits = synth.to_bits(torch.from_numpy(ref).to(out.dtype)).astype(np.int64)
    adjacent = np.abs(gpu_bits(out).astype(np.int64) - ref_bits) <= 1
    denom = np.abs(ref).max(axis=-1, keepdims=True)
    assert np.all((np.abs(o - ref) <= 2e-3 * denom) | adjacent)


@pytest.mark.parametrize("ctx,n16,with_pred", [(300, 132, True), (0, 77, False), (1000, 1500, True), (256, 0, True),
                                               (384, 4, False)])
def test_buffered_attention_is_attention_over_the_concatenation(ctx, n16, with_pred):
    from paper_2501_19392_b200 import api
    shape = dataclasses.replace(synth.CONFIGS[5], n_tokens=max(ctx, 1), n_layers=2, batch=1)
    codec = make(shape, 16)
    d, dt = shape.d_kv, shape.dtype
    scale = 1.0 / math.sqrt(shape.head_dim)
    q = synth.random_16bit((1, shape.n_q_heads, shape.head_dim), dt, 1, device=DEV)
    K16 = synth.random_16bit((1, max(n16, 1), d), dt, 2, device=DEV)[:, :n16] if n16 else None
    V16 = synth.random_16bit((1, max(n16, 1), d), dt, 3, device=DEV)[:, :n16] if n16 else None
    if ctx:
        rc = synth.random_cache(dataclasses.replace(shape, n_tokens=ctx), seed=4, device=DEV, n_layers=1)
        ad = synth.random_adapters(shape, seed=5, device=DEV)
        Kp = synth.random_16bit((ctx, d), dt, 6, device=DEV) if with_pred else None
        Vp = synth.random_16bit((ctx, d), dt, 7, device=DEV) if with_pred else None
        Kh = torch.empty((ctx, d), dtype=codec.torch_dtype, device=DEV)
        Vh = torch.empty_like(Kh)
        out, lse = codec.decode_attn_buffered(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx,
                                              shape.n_kv_heads, scale, K16, V16, Kp, Vp,
                                              ad.Wk[1] if with_pred else None, ad.Wv[1] if with_pred else None,
                                              Khat=Kh, Vhat=Vh, want_lse=True)
        rows_k = np.concatenate([gpu_bits(Kh)] + ([gpu_bits(K16[0])] if n16 else []), axis=0)
        rows_v = np.concatenate([gpu_bits(Vh)] + ([gpu_bits(V16[0])] if n16 else []), axis=0)
        if n16 == 0:      # identical to the plain entry point
            out2, _ = codec.decode_attn(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx,
                                        shape.n_kv_heads, scale, Kp, Vp, ad.Wk[1] if with_pred else None,
                                        ad.Wv[1] if with_pred else None)
            assert torch.equal(out, out2)
    else:
        empty_c = torch.empty((0, codec.code_bytes), dtype=torch.uint8, device=DEV)
        empty_s = torch.empty((0, codec.n_groups), dtype=torch.float16, device=DEV)
        out, lse = codec.decode_attn_buffered(q, empty_c, empty_s, empty_c, empty_s, 0, shape.n_kv_heads, scale,
                                              K16, V16, want_lse=True)
        rows_k, rows_v = gpu_bits(K16[0]), gpu_bits(V16[0])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    attn_check(out, q, rows_k, rows_v, shape, scale)
    ref, ref_lse = oracle.attention(dt, 1, rows_k.shape[0], shape.n_q_heads, shape.n_kv_heads, shape.head_dim, scale,
                                    synth.to_bits(q.cpu()), rows_k, rows_v)
    assert np.abs(lse.cpu().numpy() - ref_lse).max() <= 1e-4


def test_policy_keeps_sinks_and_recent_tokens_and_compresses_the_rest():
    from paper_2501_19392_b200 import api, policy
    B, L, total = 2, 3, 4 + 128 + 128 + 45          # sinks + one flushed chunk + a partly filled buffer
    shape = dataclasses.replace(synth.CONFIGS[5], n_tokens=B * total, n_layers=L, batch=B)
    codec, codec0 = make(shape, 16), make(shape, 256)          # 2-bit layers, 4-bit first layer
    d, dt = shape.d_kv, shape.dtype
    kv = synth.kv_chain(shape, seed=21, device=DEV)
    ad = synth.random_adapters(shape, seed=22, device=DEV)
    K = [k.view(B, total, d) for k in kv.K]
    V = [v.view(B, total, d) for v in kv.V]
    cache = policy.BufferedKVCache(codec, ad, L, B, max_tokens=512, device=DEV, first_layer_codec=codec0)
    # a prefill of 200 tokens, then single-token steps
    cache.append([k[:, :200] for k in K], [v[:, :200] for v in V])
    assert (cache.ctx, cache.fill, cache.n_sinks_held) == (0, 196, 4)
    for t in range(200, total):
        cache.append([k[:, t:t + 1] for k in K], [v[:, t:t + 1] for v in V])
    assert (cache.ctx, cache.n_uncompressed) == (128, 4 + 128 + 45)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0 and codec0.poll_status() == 0
    for b in range(B):
        for l in range(L):
            # uncompressed rows: the sinks, then tokens 132 .. total-1 in order
            exp = torch.cat([K[l][b, :4], K[l][b, 132:total]], dim=0)
            assert torch.equal(cache.K16[l][b, :cache.n_uncompressed], exp)
        # the compressed chunk is tokens 4 .. 131 encoded through the layers, first layer at 4 bits
        Kc0, Ks0, Vc0, Vs0, Kh, Vh = codec0.encode(K[0][b, 4:132].contiguous(), V[0][b, 4:132].contiguous())
        assert torch.equal(cache.Kcodes[0][b, :128], Kc0) and torch.equal(cache.Vscales[0][b, :128], Vs0)
        assert cache.Kcodes[0].shape[2] == 2 * cache.Kcodes[1].shape[2]
        for l in range(1, L):
            Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(K[l][b, 4:132].contiguous(), V[l][b, 4:132].contiguous(), Kh, Vh,
                                                  ad.Wk[l], ad.Wv[l])
            assert torch.equal(cache.Kcodes[l][b, :128], Kc) and torch.equal(cache.Vcodes[l][b, :128], Vc)
            assert torch.equal(cache.Kscales[l][b, :128], Ks) and torch.equal(cache.Vscales[l][b, :128], Vs)
    # attention of every layer over [compressed | sinks | recent], teacher-forced on the decoded rows
    scale = 1.0 / math.sqrt(shape.head_dim)
    q = [synth.random_16bit((B, shape.n_q_heads, shape.head_dim), dt, 30 + l, device=DEV) for l in range(L)]
    outs = cache.attend(q, shape.n_kv_heads, scale)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0 and codec0.poll_status() == 0
    for b in range(B):
        Kh = Vh = None
        for l in range(L):
            cdc = codec0 if l == 0 else codec
            args = (cache.Kcodes[l][b, :128], cache.Kscales[l][b, :128], cache.Vcodes[l][b, :128], cache.Vscales[l][b, :128])
            Kh, Vh = cdc.decode(*args, Kh, Vh, ad.Wk[l] if l else None, ad.Wv[l] if l else None)
            n16 = cache.n_uncompressed
            rows_k = np.concatenate([gpu_bits(Kh), gpu_bits(cache.K16[l][b, :n16])], axis=0)
            rows_v = np.concatenate([gpu_bits(Vh), gpu_bits(cache.V16[l][b, :n16])], axis=0)
            attn_check(outs[l][b:b + 1], q[l][b:b + 1], rows_k, rows_v, shape, scale)
    # the same with the cached keys taken as pre-RoPE keys of tokens 0 .. total-1 (Section 3.3): sinks at
    # 0 .. 3, compressed tokens at 4 .. 131, recent rows at 132 ..
    from oracle import rope as orope
    base = 500000.0
    table = codec.rope_table(shape.head_dim, base, total, DEV)
    outs_r = cache.attend(q, shape.n_kv_heads, scale, rope_table=table)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0 and codec0.poll_status() == 0
    positions = np.concatenate([4 + np.arange(128), np.arange(4), np.arange(132, total)])
    for b in range(B):
        Kh = Vh = None
        for l in range(L):
            cdc = codec0 if l == 0 else codec
            args = (cache.Kcodes[l][b, :128], cache.Kscales[l][b, :128], cache.Vcodes[l][b, :128], cache.Vscales[l][b, :128])
            Kh, Vh = cdc.decode(*args, Kh, Vh, ad.Wk[l] if l else None, ad.Wv[l] if l else None)
            n16 = cache.n_uncompressed
            rows_k = np.concatenate([gpu_bits(Kh), gpu_bits(cache.K16[l][b, :n16])], axis=0)
            rows_v = np.concatenate([gpu_bits(Vh), gpu_bits(cache.V16[l][b, :n16])], axis=0)
            ref, _ = orope.attention_rope(dt, 1, rows_k.shape[0], shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                                          scale, synth.to_bits(q[l][b:b + 1].cpu()), rows_k, rows_v, positions, base)
            o = outs_r[l][b:b + 1]
            ref_bits = synth.to_bits(torch.from_numpy(ref).to(o.dtype)).astype(np.int64)
            adjacent = np.abs(gpu_bits(o).astype(np.int64) - ref_bits) <= 1
            assert np.all((np.abs(o.to(torch.float64).cpu().numpy() - ref) <= 2e-3 * np.abs(ref).max(axis=-1, keepdims=True))
                          | adjacent)
            assert not torch.equal(o, outs[l][b:b + 1])
