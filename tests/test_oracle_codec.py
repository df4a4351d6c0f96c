"""Pins for the oracle's Algorithm 2 / Algorithm 3 (predict, quantize the residual, add back).
Independent references: numpy float64 matmul for the predictor, closed-form special cases
(zero adapters, identity adapter), the paper's predictor sizes, encode/decode consistency."""
import dataclasses
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2501_19392_b200 import synth
from util import bits_to_f64, f64_to_bits, read_golden

GOLD = read_golden(os.path.join(os.path.dirname(__file__), "golden", "paper_figures.txt"))


def setup(cfg=1, T=24, L=3, seed=0, bias=False):
    shape = dataclasses.replace(synth.CONFIGS[cfg], n_tokens=T, n_layers=L)
    grid = synth.lloyd_grid(shape.grid_size, seed=7, n_samples=1 << 14, iters=25)
    o = oracle.Oracle(shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype,
                      synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12))
    kv = synth.kv_chain(shape, seed=1000 * cfg + seed)
    ad = synth.random_adapters(shape, seed=1000 * cfg + 500 + seed, bias=bias)
    return shape, o, kv, ad


@pytest.mark.parametrize("cfg", [1, 2])
def test_predictor_is_a_plain_matmul(cfg):
    shape, o, kv, ad = setup(cfg, T=9, bias=True)
    x0, x1 = synth.to_bits(kv.K[0]), synth.to_bits(kv.V[0])
    Wk, Wv = synth.to_bits(ad.Wk[1]), synth.to_bits(ad.Wv[1])
    bk, bv = ad.bk[1].numpy(), ad.bv[1].numpy()
    P = o.predict([x0], Wk, bk)
    ref = bits_to_f64(x0, shape.dtype) @ bits_to_f64(Wk, shape.dtype).T + bk.astype(np.float64)
    assert np.abs(P - ref).max() <= 1e-12 * np.abs(ref).max()
    # concatenation order [V_prev ; K_hat]: first d input columns act on the first input
    P2 = o.predict([x1, x0], Wv, bv)
    cat = np.concatenate([bits_to_f64(x1, shape.dtype), bits_to_f64(x0, shape.dtype)], axis=1)
    ref2 = cat @ bits_to_f64(Wv, shape.dtype).T + bv.astype(np.float64)
    assert np.abs(P2 - ref2).max() <= 1e-12 * np.abs(ref2).max()
    swapped = o.predict([x0, x1], Wv, bv)
    assert np.abs(swapped - ref2).max() > 1e-3


def test_predictor_sizes_match_paper():
    d = 1024
    for L, key in ((28, "predictor_mib_28_layers"), (80, "predictor_mib_80_layers")):
        shape = dataclasses.replace(synth.CONFIGS[2], n_layers=L, n_tokens=1)
        per_layer = (d * d + d * 2 * d) * 2            # W_k [d,d] + W_v [d,2d], 16-bit
        assert round((L - 1) * per_layer / 2 ** 20) == GOLD[key]
    ad = synth.random_adapters(dataclasses.replace(synth.CONFIGS[1], n_layers=2), seed=1)
    assert ad.Wk[0] is None and tuple(ad.Wk[1].shape) == (512, 512) and tuple(ad.Wv[1].shape) == (512, 1024)


@pytest.mark.parametrize("cfg", [1, 2])
def test_zero_adapters_reduce_to_plain_rotated_vq(cfg):
    # Algorithm 2, first layer: layer 0 has no predictor; a zero matrix must give the same bits
    shape, o, kv, ad = setup(cfg)
    K, V = synth.to_bits(kv.K[1]), synth.to_bits(kv.V[1])
    prevK, prevV = synth.to_bits(kv.K[0]), synth.to_bits(kv.V[0])
    d = shape.d_kv
    k0, v0 = o.encode_layer(K, V)
    kz, vz = o.encode_layer(K, V, prevK, prevV, np.zeros((d, d), np.uint16), np.zeros((d, 2 * d), np.uint16))
    for a, b in ((k0, kz), (v0, vz)):
        for key in ("codes", "scales", "hat"):
            assert np.array_equal(a[key], b[key])
    # and the plain path equals Q / Q^-1 applied to the stored values themselves
    q = o.quantize(bits_to_f64(K, shape.dtype), "k")
    assert np.array_equal(q["codes"], k0["codes"]) and np.array_equal(q["scales"], k0["scales"])
    X = o.dequantize(q["codes"], q["scales"], "k")
    assert np.array_equal(k0["hat_exact"], X)
    # rounding to the 16-bit type: torch's conversion (through fp32) may differ only by rare double rounding
    assert np.mean(k0["hat"] != f64_to_bits(X, shape.dtype)) < 1e-3


def test_identity_adapter_predicts_exactly():
    # K == K_hat_prev and W_k = I  =>  residual 0, scales 0, K_hat = K_hat_prev
    shape, o, kv, ad = setup(1)
    d = shape.d_kv
    prevK = synth.to_bits(kv.K[0])
    eye = synth.to_bits(torch.eye(d, dtype=synth.torch_dtype(shape.dtype)))
    k = o.encode_phase(prevK, [prevK], eye, None, "k")
    assert np.all(k["scales"] == 0)
    assert np.array_equal(k["hat"], prevK)
    assert np.all(k["pred"] == bits_to_f64(prevK, shape.dtype))


@pytest.mark.parametrize("cfg", [1, 2])
def test_residual_is_target_minus_prediction(cfg):
    # sign/ordering of Algorithm 2's residual: Q acts on K - K_pred (not K_pred - K, not K)
    shape, o, kv, ad = setup(cfg, bias=True)
    K, prevK = synth.to_bits(kv.K[1]), synth.to_bits(kv.K[0])
    Wk, bk = synth.to_bits(ad.Wk[1]), ad.bk[1].numpy()
    k = o.encode_phase(K, [prevK], Wk, bk, "k")
    P = bits_to_f64(prevK, shape.dtype) @ bits_to_f64(Wk, shape.dtype).T + bk
    q = o.quantize(bits_to_f64(K, shape.dtype) - P, "k")
    assert np.mean(q["codes"] == k["codes"]) > 0.999        # identical up to summation-order ties
    assert np.array_equal(q["scales"], k["scales"])
    X = o.dequantize(k["codes"], k["scales"], "k")
    assert np.abs(k["hat_exact"] - (P + X)).max() <= 1e-10
    # the reconstruction really is closer to K than the prediction alone
    Kf = bits_to_f64(K, shape.dtype)
    assert ((k["hat_exact"] - Kf) ** 2).sum() < 0.2 * ((P - Kf) ** 2).sum()


@pytest.mark.parametrize("cfg", [1, 2])
def test_encode_then_decode_reproduces_encoders_reconstruction(cfg):
    # Algorithm 2's reconstruction and Algorithm 3's decode are the same expression
    shape, o, kv, ad = setup(cfg, L=3)
    prevK = prevV = None
    for l in range(shape.n_layers):
        K, V = synth.to_bits(kv.K[l]), synth.to_bits(kv.V[l])
        Wk = synth.to_bits(ad.Wk[l]) if l else None
        Wv = synth.to_bits(ad.Wv[l]) if l else None
        ek, ev = o.encode_layer(K, V, prevK, prevV, Wk, Wv)
        dk, dv = o.decode_layer(ek["codes"], ek["scales"], ev["codes"], ev["scales"], prevK, prevV, Wk, Wv)
        assert np.array_equal(ek["hat"], dk["hat"]) and np.array_equal(ev["hat"], dv["hat"])
        prevK, prevV = ek["hat"], ev["hat"]
        err = bits_to_f64(prevK, shape.dtype) - bits_to_f64(K, shape.dtype)
        assert (err ** 2).sum() < 0.5 * (bits_to_f64(K, shape.dtype) ** 2).sum()


def test_value_predictor_reads_the_rounded_key_reconstruction():
    shape, o, kv, ad = setup(2, T=8)
    K, V = synth.to_bits(kv.K[1]), synth.to_bits(kv.V[1])
    prevK, prevV = synth.to_bits(kv.K[0]), synth.to_bits(kv.V[0])
    Wk, Wv = synth.to_bits(ad.Wk[1]), synth.to_bits(ad.Wv[1])
    ek, ev = o.encode_layer(K, V, prevK, prevV, Wk, Wv)
    cat = np.concatenate([bits_to_f64(prevV, shape.dtype), bits_to_f64(ek["hat"], shape.dtype)], axis=1)
    ref = cat @ bits_to_f64(Wv, shape.dtype).T
    assert np.abs(ev["pred"] - ref).max() <= 1e-12 * np.abs(ref).max()
    # the C one-call layer function takes the same route
    import ctypes
    T, d = K.shape
    outs = dict(kc=np.zeros_like(ek["codes"]), ks=np.zeros_like(ek["scales"]), vc=np.zeros_like(ev["codes"]),
                vs=np.zeros_like(ev["scales"]), kh=np.zeros_like(K), vh=np.zeros_like(V))
    P = lambda a: ctypes.c_void_p(a.ctypes.data)
    rc = oracle.lib().aqo_encode_layer(ctypes.byref(o.params), P(o.grid), P(o.signs["k"]), P(o.signs["v"]),
                                       ctypes.c_int64(T), P(K), P(V), P(prevK), P(prevV), P(Wk), P(Wv), None, None,
                                       P(outs["kc"]), P(outs["ks"]), P(outs["vc"]), P(outs["vs"]),
                                       P(outs["kh"]), P(outs["vh"]), None, None)
    assert rc == 0
    assert np.array_equal(outs["kc"], ek["codes"]) and np.array_equal(outs["vc"], ev["codes"])
    assert np.array_equal(outs["kh"], ek["hat"]) and np.array_equal(outs["vh"], ev["hat"])
    assert np.array_equal(outs["vs"], ev["scales"])


def test_rows_are_independent_through_layers():
    shape, o, kv, ad = setup(1, T=16)
    rows = [2, 5, 13]
    K, V = synth.to_bits(kv.K[1]), synth.to_bits(kv.V[1])
    prevK, prevV = synth.to_bits(kv.K[0]), synth.to_bits(kv.V[0])
    Wk, Wv = synth.to_bits(ad.Wk[1]), synth.to_bits(ad.Wv[1])
    fk, fv = o.encode_layer(K, V, prevK, prevV, Wk, Wv)
    sk, sv = o.encode_layer(K[rows], V[rows], prevK[rows], prevV[rows], Wk, Wv)
    assert np.array_equal(fk["codes"][rows], sk["codes"]) and np.array_equal(fv["codes"][rows], sv["codes"])
    assert np.array_equal(fv["hat"][rows], sv["hat"])
