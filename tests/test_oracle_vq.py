"""Pins for the oracle of the backbone vector quantizer with a grid of any dimension (Section 4.1: the
2-bit grid with p = 4, n = 256).  Independent references: the p = 2 oracle written in C, a library
nearest-neighbour routine, a hand-made row that lands exactly on grid points, the bit layout re-derived
with Python integers, the orthogonality of the rotation."""
import numpy as np
import pytest
from scipy.spatial import cKDTree

import oracle
from oracle import vq
from oracle.calibration import bits_to_double
from paper_2501_19392_b200 import synth


def _linear(d, dtype=oracle.BF16):
    grid2 = synth.lloyd_grid(16, seed=7, n_samples=1 << 12, iters=10)
    return oracle.Oracle(d, 64, 64, grid2, dtype, synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2))


@pytest.mark.parametrize("d,h,g,n", [(256, 64, 64, 16), (512, 256, 512, 64), (1024, 1024, 1024, 256)])
def test_dimension_two_is_the_c_oracle_bit_for_bit(d, h, g, n):
    grid = synth.lloyd_grid(n, seed=3, n_samples=1 << 13, iters=10)
    sk, sv = synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2)
    c = oracle.Oracle(d, h, g, grid, oracle.BF16, sk, sv)
    o = vq.VectorOracle(_linear(d), grid, h, g, sk, sv)
    assert o.code_bytes == c.code_bytes
    rng = np.random.default_rng(d)
    R = rng.standard_normal((24, d)) * np.exp(rng.standard_normal((24, 1)))
    R[5] = 0.0
    for role in ("k", "v"):
        a, b = c.quantize(R, role), o.quantize(R, role)
        assert np.array_equal(a["codes"], b["codes"]) and np.array_equal(a["scales"], b["scales"])
        np.testing.assert_allclose(b["Y"], a["Y"], rtol=0, atol=1e-12)
        np.testing.assert_allclose(b["margins"], a["margins"], rtol=0, atol=1e-9)
        np.testing.assert_allclose(o.dequantize(a["codes"], a["scales"], role), c.dequantize(a["codes"], a["scales"], role),
                                   rtol=0, atol=1e-12)


def test_four_dimensional_search_against_a_library_nearest_neighbour_routine():
    d, h, g = 1024, 1024, 1024
    grid = synth.lloyd_grid(256, seed=9, n_samples=1 << 14, iters=8, dim=4)
    sk, sv = synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2)
    o = vq.VectorOracle(_linear(d), grid, h, g, sk, sv)
    assert (o.p, o.n, o.b, o.code_bytes) == (4, 256, 8, d // 4)          # 2 bits per value
    rng = np.random.default_rng(4)
    R = rng.standard_normal((16, d)) * 3.0
    q = o.quantize(R, "v")
    _, nn = cKDTree(grid.astype(np.float64)).query(q["Y"].reshape(-1, 4), k=1)
    clear = q["margins"].reshape(-1) > 1e-9
    assert clear.mean() > 0.999
    assert np.array_equal(q["codes"].reshape(-1)[clear], nn[clear].astype(np.uint8))      # one byte per 4 values
    # rotated normalised values have unit root mean square per group (the scale is the RMS, fp16-rounded)
    np.testing.assert_allclose(np.sqrt((q["Y"] ** 2).mean(axis=1)), 1.0, rtol=1e-3)
    # orthogonality: the reconstruction error is the grid error times the scale
    back = o.dequantize(q["codes"], q["scales"], "v")
    s = bits_to_double(q["scales"], oracle.F16)[:, 0]
    Yhat = grid.astype(np.float64)[q["codes"].astype(np.int64)].reshape(16, d)
    np.testing.assert_allclose(np.linalg.norm(R - back, axis=1), s * np.linalg.norm(q["Y"] - Yhat, axis=1), rtol=1e-10)
    # and it is small: a 256-point grid in four dimensions keeps most of a Gaussian row
    assert (np.linalg.norm(R - back, axis=1) < 0.45 * np.linalg.norm(R, axis=1)).all()


def test_a_row_that_lands_on_grid_points_ties_zero_rows_and_the_bit_layout():
    d, h, g, p = 256, 64, 128, 4
    # 16 sign patterns (+-1)^4 first (unit root mean square), then the origin, then far-away filler
    pts = [[(1.0 if (i >> k) & 1 else -1.0) for k in range(4)] for i in range(16)]
    pts.append([0.0, 0.0, 0.0, 0.0])
    pts.append([0.0, 0.0, 0.0, 0.0])                      # a duplicate of the origin: the lower index must win
    while len(pts) < 64:
        pts.append([9.0 + len(pts), 0.0, 0.0, 0.0])
    grid = np.array(pts, dtype=np.float32)                # n = 64: 6 bits per 4 values
    sk, sv = synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2)
    o = vq.VectorOracle(_linear(d), grid, h, g, sk, sv)
    assert (o.b, o.code_bytes) == (6, d // 4 * 6 // 8)
    rng = np.random.default_rng(0)
    want = rng.integers(0, 16, size=d // p)
    Y = grid.astype(np.float64)[want].reshape(1, d)
    R = 0.5 * vq.rotate_back(Y, sk, h)                    # scale 0.5 (exact in fp16): normalised rotation gives Y back
    R = np.concatenate([R, np.zeros((1, d))], axis=0)
    q = o.quantize(R, "k")
    assert list(q["scales"][0]) == [int(np.float16(0.5).view(np.uint16))] * 2 and not q["scales"][1].any()
    got = vq._unpack(q["codes"], 6, d // p)
    assert np.array_equal(got[0], want)
    assert (got[1] == 16).all()                           # zero row: the point at the origin, the lower of the two
    back = o.dequantize(q["codes"], q["scales"], "k")
    np.testing.assert_allclose(back[0], R[0], rtol=0, atol=1e-12)
    assert not back[1].any()
    # tuple j occupies bits [6 j, 6 j + 6) of the row's byte stream, LSB first
    big = sum(int(c) << (6 * j) for j, c in enumerate(want))
    assert bytes(q["codes"][0]) == big.to_bytes(o.code_bytes, "little")


def test_phases_round_trip():
    d, T = 256, 48
    grid = synth.lloyd_grid(256, seed=9, n_samples=1 << 13, iters=6, dim=4)
    sk, sv = synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2)
    o = vq.VectorOracle(_linear(d), grid, 256, 256, sk, sv)
    X = synth.to_bits(synth.random_16bit((T, d), oracle.BF16, 3))
    prev = synth.to_bits(synth.random_16bit((T, d), oracle.BF16, 4))
    W = synth.to_bits(synth.random_16bit((d, d), oracle.BF16, 5, std=1.0 / 16))
    for role in ("k", "v"):
        e = o.encode_phase(X, [prev], W, role=role)
        np.testing.assert_allclose(e["pred"], bits_to_double(prev, oracle.BF16) @ bits_to_double(W, oracle.BF16).T,
                                   rtol=1e-12, atol=1e-12)
        dcd = o.decode_phase(e["codes"], e["scales"], [prev], W, role=role)
        assert np.array_equal(dcd["hat"], e["hat"])
        x = bits_to_double(X, oracle.BF16)
        assert np.array_equal(e["codes"], o.quantize(x - e["pred"], role)["codes"])
