"""Pins for the oracle's single-query attention over the decoded cache (the attention read of Algorithm 4):
scipy's softmax / logsumexp as library references and closed-form special cases."""
import numpy as np
import pytest
from scipy.special import logsumexp, softmax

import oracle
from paper_2501_19392_b200 import synth
from util import bits_to_f64


def rand(shape, seed, dtype=oracle.BF16):
    return synth.to_bits(synth.random_16bit(shape, dtype, seed))


@pytest.mark.parametrize("dtype", [oracle.F16, oracle.BF16])
def test_matches_library_softmax(dtype):
    B, ctx, Hq, Hkv, hd = 2, 37, 8, 2, 16
    q = rand((B, Hq, hd), 1, dtype)
    K = rand((B * ctx, Hkv * hd), 2, dtype)
    V = rand((B * ctx, Hkv * hd), 3, dtype)
    scale = 1.0 / np.sqrt(hd)
    out, lse = oracle.attention(dtype, B, ctx, Hq, Hkv, hd, scale, q, K, V)
    qf = bits_to_f64(q, dtype)
    Kf = bits_to_f64(K, dtype).reshape(B, ctx, Hkv, hd)
    Vf = bits_to_f64(V, dtype).reshape(B, ctx, Hkv, hd)
    for b in range(B):
        for h in range(Hq):
            g = h // (Hq // Hkv)
            s = scale * Kf[b, :, g, :] @ qf[b, h]
            ref = softmax(s) @ Vf[b, :, g, :]
            assert np.abs(out[b, h] - ref).max() <= 1e-12
            assert abs(lse[b, h] - logsumexp(s)) <= 1e-12


def test_single_token_context_returns_its_value():
    B, Hq, Hkv, hd = 3, 4, 2, 8
    q, K, V = rand((B, Hq, hd), 4), rand((B, Hkv * hd), 5), rand((B, Hkv * hd), 6)
    out, lse = oracle.attention(oracle.BF16, B, 1, Hq, Hkv, hd, 0.3, q, K, V)
    Vf = bits_to_f64(V, oracle.BF16).reshape(B, Hkv, hd)
    for h in range(Hq):
        assert np.array_equal(out[:, h], Vf[:, h // 2])


def test_identical_keys_average_the_values():
    B, ctx, Hq, Hkv, hd = 1, 12, 2, 1, 8
    q = rand((B, Hq, hd), 7)
    K = np.repeat(rand((1, hd), 8), ctx, axis=0)
    V = rand((ctx, hd), 9)
    out, lse = oracle.attention(oracle.BF16, B, ctx, Hq, Hkv, hd, 1.0, q, K, V)
    mean = bits_to_f64(V, oracle.BF16).mean(0)
    assert np.abs(out[0] - mean[None, :]).max() <= 1e-13
    s = bits_to_f64(q, oracle.BF16)[0] @ bits_to_f64(K, oracle.BF16)[0]
    assert np.abs(lse[0] - (s + np.log(ctx))).max() <= 1e-12


def test_split_context_merges_by_log_sum_exp():
    B, ctx, Hq, Hkv, hd = 1, 40, 4, 2, 8
    q, K, V = rand((B, Hq, hd), 10), rand((ctx, Hkv * hd), 11), rand((ctx, Hkv * hd), 12)
    full, lse = oracle.attention(oracle.BF16, B, ctx, Hq, Hkv, hd, 0.35, q, K, V)
    o1, l1 = oracle.attention(oracle.BF16, B, 15, Hq, Hkv, hd, 0.35, q, K[:15], V[:15])
    o2, l2 = oracle.attention(oracle.BF16, B, 25, Hq, Hkv, hd, 0.35, q, K[15:], V[15:])
    w1 = np.exp(l1 - lse)[..., None]
    w2 = np.exp(l2 - lse)[..., None]
    assert np.abs(w1 * o1 + w2 * o2 - full).max() <= 1e-12
