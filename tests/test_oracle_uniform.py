"""Pins for the oracle of the uniform round-to-nearest backbone with absmax normalisation (Section 4.1
"Alternative quantizers").  Independent references: brute-force nearest level, numpy's float16, hand-made
ties and saturation cases, bit packing re-derived with Python integers."""
import numpy as np
import pytest

import oracle
from oracle import uniform as uq
from oracle.calibration import bits_to_double
from paper_2501_19392_b200 import synth


@pytest.mark.parametrize("b,g", [(2, 64), (3, 64), (4, 32), (4, 256)])
def test_nearest_level_by_brute_force_scale_and_error_bound(b, g):
    rng = np.random.default_rng(b * 100 + g)
    T, d = 64, 512
    R = rng.standard_normal((T, d)) * np.exp(rng.standard_normal((T, 1)))
    out = uq.quantize(R, b, g)
    half = 1 << (b - 1)
    absmax = np.abs(R.reshape(T, d // g, g)).max(axis=2)
    s16 = (absmax / half).astype(np.float16)
    assert np.array_equal(out["scales"], s16.view(np.uint16))
    np.testing.assert_allclose(out["scales_exact"], absmax / half, rtol=1e-15)
    levels = np.arange(-half, half)[None, None, None, :] * s16.astype(np.float64)[:, :, None, None]
    dist = np.abs(R.reshape(T, d // g, g)[..., None] - levels)
    brute = dist.argmin(axis=3)                       # numpy's argmin returns the lowest index on ties
    got = uq._unpack(out["codes"], b, d).reshape(T, d // g, g)
    assert np.array_equal(got, brute)
    xhat = uq.dequantize(out["codes"], out["scales"], b, g, d)
    err = np.abs(R - xhat).reshape(T, d // g, g)
    s = s16.astype(np.float64)[:, :, None]
    # half a spacing everywhere, except above the top level (the positive maximum saturates): one spacing
    top = R.reshape(T, d // g, g) > (half - 1) * s
    assert (err[~top] <= 0.5 * s.repeat(g, 2)[~top] * (1 + 1e-12)).all()
    # (the fp16 rounding of the scale moves the top of the range by up to half * 2^-11 spacings)
    assert (err[top] <= s.repeat(g, 2)[top] * (1 + half * 2.0 ** -10)).all()
    # margins: distance to the nearest boundary, never more than half a spacing inside the range
    x = R.reshape(T, d // g, g) / s
    inside = (x > -half) & (x < half - 1)
    assert (out["margins"].reshape(T, d // g, g)[inside] <= 0.5 + 1e-12).all()


def test_ties_saturation_and_zero_groups():
    b, g = 2, 64
    R = np.zeros((3, 64))
    # row 0: scale exactly 1 (absmax 2): values on every boundary go to the lower level
    R[0, :7] = [2.0, -1.5, -0.5, 0.5, 1.5, -2.0, 0.49999]
    # row 1: all zero; row 2: a single negative maximum
    R[2, 5] = -3.0
    out = uq.quantize(R, b, g)
    lv = uq._unpack(out["codes"], b, 64) - 2
    assert list(lv[0, :7]) == [1, -2, -1, 0, 1, -2, 0]            # 2.0 saturates at +1; x.5 goes down
    assert out["scales"][0, 0] == np.float16(1.0).view(np.uint16)
    assert out["scales"][1, 0] == 0 and (lv[1] == 0).all()
    xh = uq.dequantize(out["codes"], out["scales"], b, g, 64)
    assert (xh[1] == 0).all()
    assert xh[2, 5] == -3.0 and lv[2, 5] == -2 and (np.delete(lv[2], 5) == 0).all()   # the negative maximum is exact
    assert out["margins"][0, 1] == 0.0 and out["margins"][0, 3] == 0.0


def test_packing_is_lsb_first_in_value_order():
    assert uq._pack(np.array([[0, 1, 2, 3]]), 2).tolist() == [[0xE4]]
    for b in (2, 3, 4):
        rng = np.random.default_rng(b)
        v = rng.integers(0, 1 << b, size=(5, 64))
        packed = uq._pack(v, b)
        for t in range(5):
            big = sum(int(x) << (b * i) for i, x in enumerate(v[t]))
            assert bytes(packed[t]) == big.to_bytes(64 * b // 8, "little")
        assert np.array_equal(uq._unpack(packed, b, 64), v)


def test_codes_do_not_depend_on_the_scale_of_the_input():
    rng = np.random.default_rng(9)
    R = rng.standard_normal((16, 256))
    a = uq.quantize(R, 3, 64)
    c = uq.quantize(R * 2.0 ** -7, 3, 64)
    assert np.array_equal(a["codes"], c["codes"])


def test_phases_round_trip_and_reduce_to_the_plain_quantizer():
    d, T = 256, 96
    grid = synth.lloyd_grid(16, seed=7, n_samples=1 << 12, iters=10)
    lin = oracle.Oracle(d, 64, 64, grid, oracle.BF16, synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2))
    o = uq.UniformOracle(lin, 2, 64)
    X = synth.to_bits(synth.random_16bit((T, d), oracle.BF16, 3))
    prev = synth.to_bits(synth.random_16bit((T, d), oracle.BF16, 4))
    W = synth.to_bits(synth.random_16bit((d, d), oracle.BF16, 5, std=1.0 / 16))
    e = o.encode_phase(X, [prev], W)
    np.testing.assert_allclose(e["pred"], bits_to_double(prev, oracle.BF16) @ bits_to_double(W, oracle.BF16).T,
                               rtol=1e-12, atol=1e-12)
    dcd = o.decode_phase(e["codes"], e["scales"], [prev], W)
    assert np.array_equal(dcd["hat"], e["hat"])
    # zero adapter == no predictor
    e0 = o.encode_phase(X, [prev], np.zeros((d, d), np.uint16))
    e1 = o.encode_phase(X, [], None)
    assert np.array_equal(e0["codes"], e1["codes"]) and np.array_equal(e0["hat"], e1["hat"])
    # error of the reconstruction: half a spacing of the group (+ one 16-bit rounding of the output)
    x = bits_to_double(X, oracle.BF16)
    s = bits_to_double(e1["scales"], oracle.F16).repeat(64, axis=1)
    err = np.abs(x - bits_to_double(e1["hat"], oracle.BF16))
    assert (err <= s * (1 + 2.0 ** -9) + np.abs(x) * 2.0 ** -8).all()


# ---- rotated variant (random signs + Hadamard rotation before the uniform levels) -------------------

def _sylvester(h):
    """Orthonormal Hadamard matrix by Kronecker products (independent of the oracle's butterflies)."""
    H = np.ones((1, 1))
    while H.shape[0] < h:
        H = np.kron(H, np.array([[1.0, 1.0], [1.0, -1.0]]))
    return H / np.sqrt(float(h))


@pytest.mark.parametrize("d,h", [(256, 64), (512, 512), (1024, 256)])
def test_rotation_is_the_signed_blockwise_hadamard_matrix_and_its_own_inverse(d, h):
    rng = np.random.default_rng(d + h)
    R = rng.standard_normal((5, d))
    s = synth.hadamard_signs(d, 11)
    Y = uq.rotate(R, s, h)
    H = _sylvester(h)
    want = np.concatenate([(R * s)[:, o:o + h] @ H.T for o in range(0, d, h)], axis=1)
    np.testing.assert_allclose(Y, want, rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.linalg.norm(Y, axis=1), np.linalg.norm(R, axis=1), rtol=1e-13)
    np.testing.assert_allclose(uq.rotate_back(Y, s, h), R, rtol=0, atol=1e-12)


def _rotated_oracle(d, h, b, g, dtype=oracle.BF16):
    grid = synth.lloyd_grid(16, seed=7, n_samples=1 << 12, iters=10)
    sk, sv = synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2)
    lin = oracle.Oracle(d, 64, 64, grid, dtype, sk, sv)
    return uq.UniformOracle(lin, b, g, had_block=h, signs_k=sk, signs_v=sv), sk, sv


def test_rotated_quantizer_on_a_single_hadamard_column_has_a_closed_form():
    # r = a * s . c with c the j-th +-1 Hadamard column: s . r = a * sqrt(h) * (orthonormal column j), which the
    # orthonormal transform maps to the spike a * sqrt(h) * e_j.
    d, h, b, g, j, a = 256, 256, 2, 256, 37, 0.75
    o, sk, sv = _rotated_oracle(d, h, b, g)
    col = _sylvester(h)[:, j] * np.sqrt(float(h))          # +-1 entries
    R = (a * sk * col)[None, :]
    q = o.quantize(R, "k")
    spike = a * np.sqrt(float(h))                          # 12.0: exactly representable, scale 6.0 exact in fp16
    assert np.allclose(q["Y"][0, j], spike, atol=1e-12) and np.abs(np.delete(q["Y"][0], j)).max() < 1e-12
    lv = uq._unpack(q["codes"], b, d)[0] - 2
    assert lv[j] == 1 and (np.delete(lv, j) == 0).all()     # the positive maximum saturates at the top level
    assert q["scales"][0, 0] == np.float16(spike / 2).view(np.uint16)
    back = o.dequantize(q["codes"], q["scales"], "k")
    np.testing.assert_allclose(back[0], 0.5 * R[0], rtol=0, atol=1e-12)   # level 1 of 2: half the spike
    # the value signs give another row
    assert not np.array_equal(o.quantize(R, "v")["codes"], q["codes"])


def test_rotated_quantizer_error_is_the_rotated_domain_error_and_had_block_one_is_the_plain_one():
    d, h, b, g = 512, 128, 4, 64
    o, sk, sv = _rotated_oracle(d, h, b, g)
    rng = np.random.default_rng(3)
    R = rng.standard_normal((32, d))
    q = o.quantize(R, "v")
    Yhat = uq.dequantize(q["codes"], q["scales"], b, g, d)
    back = o.dequantize(q["codes"], q["scales"], "v")
    np.testing.assert_allclose(np.linalg.norm(R - back, axis=1), np.linalg.norm(q["Y"] - Yhat, axis=1), rtol=1e-12)
    # levels are those of the plain quantizer applied to the rotated rows
    assert np.array_equal(q["codes"], uq.quantize(uq.rotate(R, sv, h), b, g)["codes"])
    plain = uq.UniformOracle(o.linear, b, g)
    p = plain.quantize(R)
    assert np.array_equal(p["codes"], uq.quantize(R, b, g)["codes"])
    assert np.array_equal(plain.dequantize(p["codes"], p["scales"]), uq.dequantize(p["codes"], p["scales"], b, g, d))


def test_rotation_spreads_an_outlier_so_that_the_other_values_survive():
    # Why the appendix' rotated backbone works with one group per row where the plain one collapses:
    # one outlier sets the plain scale and flattens everything else to level 0 (or -1 .. 0).
    d, h, b, g = 1024, 1024, 2, 1024
    o, sk, sv = _rotated_oracle(d, h, b, g)
    rng = np.random.default_rng(5)
    R = rng.standard_normal((16, d))
    R[:, 17] = 60.0
    plain = uq.UniformOracle(o.linear, b, g)
    qp = plain.quantize(R)
    err_plain = np.linalg.norm(np.delete(R - plain.dequantize(qp["codes"], qp["scales"]), 17, axis=1), axis=1)
    qr = o.quantize(R, "k")
    err_rot = np.linalg.norm(R - o.dequantize(qr["codes"], qr["scales"], "k"), axis=1)
    base = np.linalg.norm(np.delete(R, 17, axis=1), axis=1)
    assert (err_plain > 0.95 * base).all()          # nothing but the outlier is kept
    assert (err_rot < 0.8 * np.linalg.norm(R, axis=1)).all()


def test_rotated_phases_round_trip():
    d, T = 256, 64
    o, sk, sv = _rotated_oracle(d, 256, 2, 256)
    X = synth.to_bits(synth.random_16bit((T, d), oracle.BF16, 3))
    prev = synth.to_bits(synth.random_16bit((T, d), oracle.BF16, 4))
    W = synth.to_bits(synth.random_16bit((d, d), oracle.BF16, 5, std=1.0 / 16))
    for role in ("k", "v"):
        e = o.encode_phase(X, [prev], W, role=role)
        dcd = o.decode_phase(e["codes"], e["scales"], [prev], W, role=role)
        assert np.array_equal(dcd["hat"], e["hat"])
        x = bits_to_double(X, oracle.BF16)
        want = e["pred"] + o.dequantize(e["codes"], e["scales"], role)
        np.testing.assert_allclose(e["hat_exact"], want, rtol=0, atol=0)
        assert np.array_equal(e["codes"], o.quantize(x - e["pred"], role)["codes"])
