"""Pins for the oracle of rotary position encoding on cached pre-RoPE keys (Section 3.3 "Positional
embeddings").  Independent references: complex multiplication, a hand-worked row, the defining
properties of the rotary embedding (position 0 is the identity, rotations compose, scores depend on
the position difference only, norms are kept), and the plain attention oracle on pre-rotated rows."""
import math

import numpy as np
import pytest

import oracle
from oracle import rope
from oracle.calibration import bits_to_double, double_to_bits
from paper_2501_19392_b200 import synth


def test_hand_worked_row():
    # head_dim 4, base 10000: frequencies 1 and 0.01; pairs (x0, x2) and (x1, x3)
    K = np.array([[1.0, 0.0, 0.0, 1.0], [2.0, 3.0, 0.0, 0.0]])
    Y = rope.rotate_rows(K, np.array([1, 2]), 1, 4, 10000.0)
    want0 = [math.cos(1.0), -math.sin(0.01), math.sin(1.0), math.cos(0.01)]
    want1 = [2 * math.cos(2.0), 3 * math.cos(0.02), 2 * math.sin(2.0), 3 * math.sin(0.02)]
    np.testing.assert_allclose(Y, [want0, want1], rtol=0, atol=1e-15)
    np.testing.assert_allclose(rope.angles(np.array([3]), 8, 16.0), [[3.0, 1.5, 0.75, 0.375]], rtol=1e-15)


@pytest.mark.parametrize("heads,hd,base", [(8, 128, 500000.0), (2, 64, 10000.0)])
def test_equals_complex_multiplication_and_keeps_pair_norms(heads, hd, base):
    rng = np.random.default_rng(hd)
    n = 40
    K = rng.standard_normal((n, heads * hd))
    pos = rng.integers(0, 100000, size=n)
    Y = rope.rotate_rows(K, pos, heads, hd, base)
    X = K.reshape(n, heads, hd)
    z = X[:, :, :hd // 2] + 1j * X[:, :, hd // 2:]
    w = np.exp(1j * pos[:, None].astype(np.float64) * base ** (-np.arange(hd // 2) * 2.0 / hd))[:, None, :]
    zz = z * w
    want = np.concatenate([zz.real, zz.imag], axis=2).reshape(n, heads * hd)
    np.testing.assert_allclose(Y, want, rtol=0, atol=1e-12)
    Yr = Y.reshape(n, heads, hd)
    np.testing.assert_allclose(Yr[:, :, :hd // 2] ** 2 + Yr[:, :, hd // 2:] ** 2, np.abs(z) ** 2, rtol=1e-12)


def test_identity_at_position_zero_composition_and_relative_scores():
    rng = np.random.default_rng(1)
    heads, hd, base = 2, 64, 10000.0
    K = rng.standard_normal((6, heads * hd))
    Q = rng.standard_normal((6, heads * hd))
    assert np.array_equal(rope.rotate_rows(K, np.zeros(6, np.int64), heads, hd, base), K)
    a, b = np.array([3, 10, 0, 7, 100, 1]), np.array([5, 1, 9, 7, 23, 0])
    twice = rope.rotate_rows(rope.rotate_rows(K, a, heads, hd, base), b, heads, hd, base)
    np.testing.assert_allclose(twice, rope.rotate_rows(K, a + b, heads, hd, base), rtol=0, atol=1e-12)
    # <R(p) q, R(t) k> per head depends on p - t only
    p, t, shift = np.array([50, 7, 7, 12, 3, 9]), np.array([20, 7, 1, 30, 0, 8]), 1234
    def scores(pp, tt):
        q = rope.rotate_rows(Q, pp, heads, hd, base).reshape(6, heads, hd)
        k = rope.rotate_rows(K, tt, heads, hd, base).reshape(6, heads, hd)
        return (q * k).sum(axis=2)
    np.testing.assert_allclose(scores(p, t), scores(p + shift, t + shift), rtol=0, atol=1e-9)
    assert np.abs(scores(p, t) - scores(p, t + 1)).max() > 1e-3


def test_sixteen_bit_rounding_and_attention_over_rotated_rows():
    batch, ctx, hq, hkv, hd, base = 2, 37, 6, 2, 64, 10000.0
    d = hkv * hd
    dtype = oracle.BF16
    K = synth.to_bits(synth.random_16bit((batch * ctx, d), dtype, 11))
    V = synth.to_bits(synth.random_16bit((batch * ctx, d), dtype, 12))
    q = synth.to_bits(synth.random_16bit((batch, hq, hd), dtype, 13))
    pos = np.arange(ctx) + 4
    rot_bits, exact = rope.rotate_rows_16bit(K, np.tile(pos, batch), hkv, hd, base, dtype)
    # one rounding: the 16-bit rows are the nearest representable values of the exact rotation
    np.testing.assert_array_equal(rot_bits, double_to_bits(exact, dtype))
    err = np.abs(bits_to_double(rot_bits, dtype) - exact)
    assert (err <= np.abs(exact) * 2.0 ** -8 + 1e-40).all()
    out, lse = rope.attention_rope(dtype, batch, ctx, hq, hkv, hd, 0.125, q, K, V, pos, base)
    # brute force over the rotated rows
    Kr = bits_to_double(rot_bits, dtype).reshape(batch, ctx, hkv, hd)
    Vd = bits_to_double(V, dtype).reshape(batch, ctx, hkv, hd)
    qd = bits_to_double(q, dtype)
    for b in range(batch):
        for h in range(hq):
            s = 0.125 * Kr[b, :, h // (hq // hkv), :] @ qd[b, h]
            w = np.exp(s - s.max())
            np.testing.assert_allclose(out[b, h], (w / w.sum()) @ Vd[b, :, h // (hq // hkv), :], rtol=1e-10, atol=1e-12)
            np.testing.assert_allclose(lse[b, h], s.max() + np.log(w.sum()), rtol=1e-12)
    # positions matter: other positions give another result; equal shifts of keys alone do too
    out2, _ = rope.attention_rope(dtype, batch, ctx, hq, hkv, hd, 0.125, q, K, V, pos + 1, base)
    assert np.abs(out - out2).max() > 1e-4
