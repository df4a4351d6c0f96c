"""Pins for the oracle's backbone quantizer Q / Q^-1 (rotated vector quantization with group
scales).  Independent references: scipy's Hadamard matrix and k-d tree, numpy's float16, and the
figures the paper prints (tests/golden/paper_figures.txt)."""
import os

import numpy as np
import pytest
from scipy.linalg import hadamard
from scipy.spatial import cKDTree

import oracle
from paper_2501_19392_b200 import synth
from util import pack_codes, read_golden, unpack_codes

GOLD = read_golden(os.path.join(os.path.dirname(__file__), "golden", "paper_figures.txt"))


def make(d, h, g, n, dtype=oracle.BF16, seed=0):
    grid = synth.lloyd_grid(n, seed=7, n_samples=1 << 14, iters=25)
    return oracle.Oracle(d, h, g, grid, dtype, synth.hadamard_signs(d, seed + 1),
                         synth.hadamard_signs(d, seed + 2))


def rotated_reference(o, R, role="k"):
    """Y = H_h (xi * R / s16) / sqrt(h) built from library pieces only."""
    T, d = R.shape
    h, g = o.params.had_block, o.params.scale_group
    s = np.sqrt((R.reshape(T, d // g, g) ** 2).mean(-1))
    s16 = np.minimum(s, 65504.0).astype(np.float16)
    inv = np.where(s16 > 0, 1.0 / np.maximum(s16.astype(np.float64), 1e-300), 0.0)
    u = o.signs[role][None, :] * R * np.repeat(inv, g, axis=1)
    H = hadamard(h).astype(np.float64)
    Y = (u.reshape(T, d // h, h) @ H.T).reshape(T, d) / np.sqrt(h)
    return Y, s, s16


@pytest.mark.parametrize("d,h,g,n", [(512, 64, 64, 16), (1024, 1024, 1024, 16),
                                      (1024, 1024, 1024, 64), (1024, 256, 512, 256)])
def test_scale_rotation_and_search_against_library_routines(d, h, g, n):
    o = make(d, h, g, n)
    rng = np.random.default_rng(5)
    R = rng.standard_normal((6, d)) * np.exp(rng.standard_normal((1, d)))
    q = o.quantize(R)
    Y, s, s16 = rotated_reference(o, R)
    assert np.allclose(q["scales_exact"], s, rtol=1e-13, atol=0)
    assert np.array_equal(q["scales"], s16.view(np.uint16))
    assert np.abs(q["Y"] - Y).max() <= 1e-11 * max(1.0, np.abs(Y).max())
    # nearest grid point: k-d tree on the same rotated values
    bits = int(np.log2(n))
    idx = unpack_codes(q["codes"], bits)
    _, nn = cKDTree(o.grid.astype(np.float64)).query(Y.reshape(-1, 2))
    nn = nn.reshape(idx.shape)
    clear = q["margins"] > 1e-9
    assert clear.mean() > 0.999
    assert np.array_equal(idx[clear], nn[clear])


def test_search_is_brute_force_on_tiny_input():
    o = make(64, 64, 64, 16)
    rng = np.random.default_rng(11)
    R = rng.standard_normal((4, 64))
    q = o.quantize(R)
    idx = unpack_codes(q["codes"], 4)
    G = o.grid.astype(np.float64)
    for t in range(4):
        for j in range(32):
            y = q["Y"][t, 2 * j:2 * j + 2]
            dist = sorted((float(((y - G[c]) ** 2).sum()), c) for c in range(16))
            assert idx[t, j] == dist[0][1]
            m = (dist[1][0] - dist[0][0]) / (dist[1][0] + dist[0][0] + 1e-30)
            assert abs(q["margins"][t, j] - m) <= 1e-12


def test_ties_go_to_the_lowest_index():
    # h = g = 2, signs +1: every block (1, 0) rotates to (y, y), equidistant from (1,0) and (0,1)
    ones = np.ones(8, dtype=np.int8)
    for grid in ([[0, 1], [1, 0], [-1, 0], [0, -1]], [[-1, 0], [1, 0], [0, 1], [0, -1]]):
        o = oracle.Oracle(8, 2, 2, np.array(grid, np.float32), oracle.BF16, ones, ones)
        q = o.quantize(np.array([[1.0, 0.0] * 4]))
        assert abs(q["Y"][0, 0] - q["Y"][0, 1]) == 0.0
        tied = [i for i, gp in enumerate(grid) if gp in ([0, 1], [1, 0])]
        assert np.all(unpack_codes(q["codes"], 2)[0] == min(tied))
        assert np.all(q["margins"][0] == 0.0)


@pytest.mark.parametrize("n", [16, 64, 256])
def test_code_byte_layout_lsb_first(n):
    bits = int(np.log2(n))
    d = 512
    o = make(d, 64, 64, n)
    rng = np.random.default_rng(2)
    idx = rng.integers(0, n, size=(3, d // 2))
    codes = pack_codes(idx, bits)
    assert codes.shape == (3, o.code_bytes)
    if n == 16:      # two codes per byte, low nibble = even pair
        assert np.array_equal(codes, (idx[:, 0::2] | (idx[:, 1::2] << 4)).astype(np.uint8))
    if n == 256:
        assert np.array_equal(codes, idx.astype(np.uint8))
    one = np.full((3, d // 64), np.float16(1.0).view(np.uint16), np.uint16)
    X = o.dequantize(codes, one)
    H = hadamard(64).astype(np.float64)
    pts = o.grid.astype(np.float64)[idx].reshape(3, d)
    ref = (pts.reshape(3, d // 64, 64) @ H.T).reshape(3, d) / 8.0 * o.signs["k"][None, :]
    assert np.abs(X - ref).max() <= 1e-12


@pytest.mark.parametrize("k", [-6, 3, 9])
def test_scale_independence_for_powers_of_two(k):
    # footnote of Section 3.1: ||Q^-1 Q(aX) - aX|| = a ||Q^-1 Q(X) - X||; exact for a = 2^k
    o = make(1024, 1024, 1024, 16)
    rng = np.random.default_rng(8)
    R = rng.standard_normal((5, 1024))
    a = 2.0 ** k
    q1, q2 = o.quantize(R), o.quantize(a * R)
    assert np.array_equal(q1["codes"], q2["codes"])
    assert np.array_equal(q1["scales"].view(np.float16).astype(np.float64) * a,
                          q2["scales"].view(np.float16).astype(np.float64))
    x1 = o.dequantize(q1["codes"], q1["scales"])
    x2 = o.dequantize(q2["codes"], q2["scales"])
    assert np.array_equal(x1 * a, x2)


def test_relative_error_bands_on_gaussian_input():
    # Section 3.1: a 2-bit quantizer explains about 0.89 of the variance; finer grids do better
    rng = np.random.default_rng(21)
    R = rng.standard_normal((64, 1024))
    rel = {}
    for n in (16, 64, 256):
        grid = synth.lloyd_grid(n, seed=7, n_samples=1 << 15, iters=40)
        o = oracle.Oracle(1024, 1024, 1024, grid, oracle.BF16, synth.hadamard_signs(1024, 1),
                          synth.hadamard_signs(1024, 2))
        q = o.quantize(R)
        X = o.dequantize(q["codes"], q["scales"])
        rel[n] = ((X - R) ** 2).sum() / (R ** 2).sum()
    assert 0.08 < rel[16] < 0.13, rel
    assert 0.02 < rel[64] < 0.045, rel
    assert 0.004 < rel[256] < 0.015, rel
    assert rel[256] < rel[64] < rel[16]


def test_rotation_is_what_makes_outliers_cheap():
    # one huge channel: after the rotation its energy is spread, so the error stays in band
    o = make(1024, 1024, 1024, 16)
    rng = np.random.default_rng(4)
    R = rng.standard_normal((8, 1024))
    R[:, 17] *= 100.0
    q = o.quantize(R)
    X = o.dequantize(q["codes"], q["scales"])
    assert ((X - R) ** 2).sum() / (R ** 2).sum() < 0.2


@pytest.mark.parametrize("d,g,n,key", [(1024, 1024, 16, "bits_per_value_n16_g1024"),
                                       (1024, 1024, 64, "bits_per_value_n64_g1024"),
                                       (1024, 1024, 256, "bits_per_value_n256_g1024"),
                                       (256, 256, 16, "bits_per_value_n16_g256"),
                                       (512, 512, 16, "bits_per_value_n16_g512")])
def test_bits_per_value_accounting_matches_paper(d, g, n, key):
    o = make(d, g if g <= 1024 else 1024, g, n)
    bits = 8.0 * (o.code_bytes + 2 * o.n_groups) / d
    assert bits == np.log2(n) / 2 + 16.0 / g
    assert round(bits, 2) == GOLD[key]


def test_layer_averaged_bits_match_paper():
    b2, b3, b4 = 2 + 16 / 1024, 3 + 16 / 1024, 4 + 16 / 1024
    for L, key, b in ((28, "avg_bits_28_layers_2bit", b2), (32, "avg_bits_32_layers_2bit", b2),
                      (80, "avg_bits_80_layers_2bit", b2), (28, "avg_bits_28_layers_3bit", b3),
                      (80, "avg_bits_80_layers_3bit", b3)):
        assert round((b4 + (L - 1) * b) / L, 2) == GOLD[key]
    cache16 = 80 * 2 * 1024 * (1 << 17) * 2 / 2 ** 30
    assert round(cache16) == GOLD["cache_gib_70b_16bit"]


def test_zero_group_gives_zero_scale_and_origin_code():
    o = make(512, 64, 64, 16)
    R = np.random.default_rng(1).standard_normal((2, 512))
    R[0, 64:128] = 0.0
    q = o.quantize(R)
    assert q["scales"][0, 1] == 0
    origin = int(np.argmin((o.grid.astype(np.float64) ** 2).sum(1)))
    assert np.all(unpack_codes(q["codes"], 4)[0, 32:64] == origin)
    X = o.dequantize(q["codes"], q["scales"])
    assert np.all(X[0, 64:128] == 0.0)


def test_rows_are_independent():
    o = make(1024, 1024, 1024, 16)
    R = np.random.default_rng(9).standard_normal((12, 1024))
    full = o.quantize(R)
    sub = o.quantize(R[[3, 7, 11]])
    assert np.array_equal(full["codes"][[3, 7, 11]], sub["codes"])
    assert np.array_equal(full["scales"][[3, 7, 11]], sub["scales"])


def test_key_and_value_roles_use_their_own_signs():
    o = make(512, 64, 64, 16)
    R = np.random.default_rng(10).standard_normal((2, 512))
    qk, qv = o.quantize(R, "k"), o.quantize(R, "v")
    assert not np.array_equal(qk["codes"], qv["codes"])
    Yv, _, _ = rotated_reference(o, R, "v")
    assert np.abs(qv["Y"] - Yv).max() <= 1e-11
