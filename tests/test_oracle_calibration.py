"""Pins for the calibration oracle (Algorithm 1; Section 3.2; Appendix A: closed form, regularizer
rate).  Independent references: closed forms of ridge regression (one feature, orthonormal design),
the normal equations as an identity, numpy's SVD-based least squares on the augmented system, a
planted noiseless map, and the scalar 16-bit converters of the C oracle."""
import dataclasses

import numpy as np
import pytest

import oracle
from oracle import calibration as cal
from paper_2501_19392_b200 import synth


def test_array_conversions_match_the_scalar_converters():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(5000) * 10.0 ** rng.integers(-6, 6, 5000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.001953125, 1.005859375, -1.001953125, 255.5,
                         1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -8 + 2.0 ** -40]])
    b = cal.double_to_bits(x, oracle.BF16)
    assert np.array_equal(b, np.array([oracle.double_to_bf16(float(v)) for v in x], dtype=np.uint16))
    xs = x[np.abs(x) < 6e4]
    h = cal.double_to_bits(xs, oracle.F16)
    assert np.array_equal(h, np.array([oracle.double_to_f16(float(v)) for v in xs], dtype=np.uint16))
    assert np.array_equal(cal.bits_to_double(b, oracle.BF16),
                          np.array([oracle.bf16_to_double(int(v)) for v in b]))
    assert np.array_equal(cal.bits_to_double(h, oracle.F16),
                          np.array([oracle.f16_to_double(int(v)) for v in h]))


def test_one_feature_closed_form():
    # trace(X^T X)/n_in = sum x^2, so w = sum(xy) / ((1 + rate) sum x^2)
    rng = np.random.default_rng(1)
    x = rng.standard_normal((500, 1))
    y = 0.7 * x + 0.1 * rng.standard_normal((500, 1))
    for rate in (0.0, 1e-3, 0.5):
        W, b = cal.ridge_fit(x, y, rate)
        assert b is None
        assert W.shape == (1, 1)
        np.testing.assert_allclose(W[0, 0], (x * y).sum() / ((1 + rate) * (x * x).sum()), rtol=1e-12)


def test_orthonormal_design_shrinks_by_one_over_one_plus_rate():
    # X = s * Q with orthonormal columns: X^T X = s^2 I, trace/n_in = s^2, W = Y^T X / (s^2 (1 + rate))
    rng = np.random.default_rng(2)
    Q, _ = np.linalg.qr(rng.standard_normal((200, 6)))
    s = 3.5
    X = s * Q
    Y = rng.standard_normal((200, 4))
    W, _ = cal.ridge_fit(X, Y, 0.25)
    np.testing.assert_allclose(W, Y.T @ X / (s * s * 1.25), rtol=1e-11, atol=1e-13)


def test_planted_map_is_recovered_and_not_transposed():
    rng = np.random.default_rng(3)
    A = rng.standard_normal((5, 3))            # y = x A: 5 inputs, 3 outputs, not square
    X = rng.standard_normal((400, 5))
    Y = X @ A
    W, _ = cal.ridge_fit(X, Y, 0.0)
    assert W.shape == (3, 5)                   # [d_out][n_in], a linear layer's weight
    np.testing.assert_allclose(W, A.T, atol=1e-10)
    np.testing.assert_allclose(X @ W.T, Y, atol=1e-9)


def test_normal_equations_and_augmented_least_squares():
    rng = np.random.default_rng(4)
    X = rng.standard_normal((300, 12)) * np.exp(rng.standard_normal(12))       # unequal feature scales
    Y = X @ rng.standard_normal((12, 7)) + 0.3 * rng.standard_normal((300, 7))
    rate = 1e-3
    W, _ = cal.ridge_fit(X, Y, rate)
    ridge = rate * (X * X).sum() / 12
    # stationarity: X^T (Y - X W^T) = ridge * W^T
    np.testing.assert_allclose(X.T @ (Y - X @ W.T), ridge * W.T, rtol=1e-8, atol=1e-8)
    # ridge as plain least squares on [X ; sqrt(ridge) I] W^T = [Y ; 0] (SVD-based routine)
    Xa = np.concatenate([X, np.sqrt(ridge) * np.eye(12)], axis=0)
    Ya = np.concatenate([Y, np.zeros((12, 7))], axis=0)
    Wl = np.linalg.lstsq(Xa, Ya, rcond=None)[0].T
    np.testing.assert_allclose(W, Wl, rtol=1e-9, atol=1e-10)
    # any other matrix has a larger penalised loss
    loss = lambda M: ((X @ M.T - Y) ** 2).sum() + ridge * (M ** 2).sum()
    for _ in range(5):
        assert loss(W + 1e-3 * rng.standard_normal(W.shape)) > loss(W)


def test_scale_invariance_of_the_relative_rate():
    rng = np.random.default_rng(5)
    X = rng.standard_normal((200, 8))
    Y = X @ rng.standard_normal((8, 8)) + 0.5 * rng.standard_normal((200, 8))
    W1, _ = cal.ridge_fit(X, Y, 1e-2)
    W2, _ = cal.ridge_fit(16.0 * X, 16.0 * Y, 1e-2)
    np.testing.assert_allclose(W1, W2, rtol=1e-10)


def test_intercept():
    rng = np.random.default_rng(6)
    A = rng.standard_normal((4, 3))
    c = np.array([2.0, -1.0, 0.5])
    X = rng.standard_normal((500, 4)) + np.array([5.0, -3.0, 0.0, 1.0])
    Y = X @ A + c
    W, b = cal.ridge_fit(X, Y, 0.0, fit_bias=True)
    np.testing.assert_allclose(W, A.T, atol=1e-10)
    np.testing.assert_allclose(b, c, atol=1e-9)
    # with a rate: the same as an unpenalised constant column beside penalised centred features
    rate = 1e-2
    Yn = Y + 0.2 * rng.standard_normal(Y.shape)
    W, b = cal.ridge_fit(X, Yn, rate, fit_bias=True)
    Xc = X - X.mean(0)
    ridge = rate * (Xc * Xc).sum() / 4
    Xa = np.concatenate([np.concatenate([Xc, np.ones((500, 1))], 1),
                         np.concatenate([np.sqrt(ridge) * np.eye(4), np.zeros((4, 1))], 1)], 0)
    Ya = np.concatenate([Yn, np.zeros((4, 3))], 0)
    sol = np.linalg.lstsq(Xa, Ya, rcond=None)[0]
    np.testing.assert_allclose(W, sol[:4].T, rtol=1e-9, atol=1e-10)
    np.testing.assert_allclose(b, sol[4] - X.mean(0) @ sol[:4], rtol=1e-9, atol=1e-9)


def _small_setup(T=1536, L=3, n=16, seed=0):
    shape = dataclasses.replace(synth.CONFIGS[1], n_tokens=T, n_layers=L, grid_size=n, dtype=oracle.BF16,
                                n_kv_heads=2, head_dim=64, had_block=64, scale_group=64)
    d = shape.d_kv
    kv = synth.kv_chain(shape, seed=seed + 1)
    K = [synth.to_bits(k) for k in kv.K]
    V = [synth.to_bits(v) for v in kv.V]
    grid = synth.lloyd_grid(n, seed=7, n_samples=1 << 14, iters=25)
    o = oracle.Oracle(d, 64, 64, grid, oracle.BF16, synth.hadamard_signs(d, 11), synth.hadamard_signs(d, 12))
    return o, K, V


def test_algorithm_1_trains_on_reconstructions_layer_after_layer():
    o, K, V = _small_setup()
    res = cal.calibrate(o, K, V, rate=1e-3)
    assert len(res) == 2
    # layer 1's inputs are the quantised layer 0 (Q alone), not the exact one
    k0 = o.encode_phase(K[0], [], None, None, "k")["hat"]
    v0 = o.encode_phase(V[0], [], None, None, "v")["hat"]
    W_rec, _ = cal.ridge_fit(cal.bits_to_double(k0, o.dtype), cal.bits_to_double(K[1], o.dtype), 1e-3)
    W_exact_in, _ = cal.ridge_fit(cal.bits_to_double(K[0], o.dtype), cal.bits_to_double(K[1], o.dtype), 1e-3)
    np.testing.assert_allclose(res[0]["Wk_exact"], W_rec, rtol=1e-12, atol=1e-14)
    assert np.abs(res[0]["Wk_exact"] - W_exact_in).max() > 1e-4
    # the value predictor reads [V_old ; K_rec] with K_rec the layer's own reconstructed keys
    X = np.concatenate([cal.bits_to_double(v0, o.dtype), cal.bits_to_double(res[0]["Khat"], o.dtype)], 1)
    Wv, _ = cal.ridge_fit(X, cal.bits_to_double(V[1], o.dtype), 1e-3)
    np.testing.assert_allclose(res[0]["Wv_exact"], Wv, rtol=1e-12, atol=1e-14)
    assert res[0]["Wv"].shape == (o.d, 2 * o.d) and res[0]["Wk"].shape == (o.d, o.d)
    # K_rec is Algorithm 2's reconstruction with the ROUNDED predictor
    k1 = o.encode_phase(K[1], [k0], res[0]["Wk"], None, "k")["hat"]
    assert np.array_equal(k1, res[0]["Khat"])
    # layer 2 trains on layer 1's reconstructions
    W2, _ = cal.ridge_fit(cal.bits_to_double(res[0]["Khat"], o.dtype), cal.bits_to_double(K[2], o.dtype), 1e-3)
    np.testing.assert_allclose(res[1]["Wk_exact"], W2, rtol=1e-12, atol=1e-14)
    # the printed listing's variant (exact first layer) is a different fit
    res_x = cal.calibrate(o, K[:2], V[:2], rate=1e-3, first_layer_exact=True)
    np.testing.assert_allclose(res_x[0]["Wk_exact"], W_exact_in, rtol=1e-12, atol=1e-14)


def test_fitted_predictors_buy_accuracy_at_equal_bits():
    # Section 3.1: a predictor that explains as much variance as a b-bit quantizer saves about b bits.
    # The synthetic keys are 0.92 explained by the previous layer, so 2-bit residual coding must beat
    # 2-bit direct coding by a wide margin, and come close to or beat 3-bit direct coding.
    o, K, V = _small_setup(T=2048, L=3, n=16)
    res = cal.calibrate(o, K, V, rate=1e-3)
    direct2 = o.encode_phase(K[2], [], None, None, "k")["hat"]
    err_fit = cal.relative_error(K[2], res[1]["Khat"], o.dtype)
    err_direct = cal.relative_error(K[2], direct2, o.dtype)
    assert err_fit < 0.35 * err_direct
    o3, _, _ = _small_setup(T=2048, L=3, n=64)
    direct3 = o3.encode_phase(K[2], [], None, None, "k")["hat"]
    assert err_fit < 1.2 * cal.relative_error(K[2], direct3, o.dtype)
    # values: the previous layer and the keys explain less of them (the synthetic recurrence adds 0.7 noise)
    verr_fit = cal.relative_error(V[2], res[1]["Vhat"], o.dtype)
    verr_direct = cal.relative_error(V[2], o.encode_phase(V[2], [], None, None, "v")["hat"], o.dtype)
    assert verr_fit < 0.8 * verr_direct
