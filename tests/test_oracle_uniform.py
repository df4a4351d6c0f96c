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
