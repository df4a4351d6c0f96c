"""Pins for the oracle's 16-bit float conversions: numpy's float16 and torch's bfloat16 are the
independent references (IEEE round-to-nearest-even)."""
import numpy as np
import torch

import oracle


def test_f16_decode_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ref = bits.view(np.float16).astype(np.float64)
    got = np.array([oracle.f16_to_double(int(b)) for b in bits])
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    m = ~np.isnan(ref)
    assert np.array_equal(ref[m], got[m])
    assert np.array_equal(np.signbit(ref[m]), np.signbit(got[m]))


def test_bf16_decode_all_bit_patterns():
    bits = np.arange(65536, dtype=np.uint16)
    ref = torch.from_numpy(bits.copy()).view(torch.bfloat16).to(torch.float64).numpy()
    got = np.array([oracle.bf16_to_double(int(b)) for b in bits])
    m = ~np.isnan(ref)
    assert np.array_equal(np.isnan(ref), np.isnan(got))
    assert np.array_equal(ref[m], got[m])


def _cases(rng):
    x = np.concatenate([
        rng.standard_normal(4000),
        rng.standard_normal(2000) * 1e-5,      # fp16 subnormal range
        rng.standard_normal(2000) * 1e-8,      # below the smallest fp16 subnormal
        rng.standard_normal(1000) * 3e4,       # near fp16 overflow
        np.array([0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e6, -1e6, 2.0 ** -24, 2.0 ** -25,
                  1.5 * 2.0 ** -25, 6.103515625e-05, 1.0, 1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11]),
    ])
    return x


def test_f16_encode_matches_numpy_rne():
    x = _cases(np.random.default_rng(0))
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    got = np.array([oracle.double_to_f16(v) for v in x], dtype=np.uint16)
    assert np.array_equal(ref, got)


def test_f16_encode_exact_ties_go_to_even():
    # midpoints between consecutive fp16 numbers, normal and subnormal
    for lo_bits in (0x3C00, 0x3C01, 0x0001, 0x0002, 0x03FF, 0x7BFE):
        lo = oracle.f16_to_double(lo_bits)
        hi = oracle.f16_to_double(lo_bits + 1)
        mid = 0.5 * (lo + hi)
        want = lo_bits if lo_bits % 2 == 0 else lo_bits + 1
        assert oracle.double_to_f16(mid) == want
        assert oracle.double_to_f16(-mid) == (want | 0x8000)


def test_bf16_encode_matches_torch_rne():
    # float32-representable inputs so torch's float32 -> bfloat16 path is a single rounding
    x = _cases(np.random.default_rng(1)).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.uint16).numpy()
    got = np.array([oracle.double_to_bf16(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(ref, got)


def test_bf16_encode_exact_ties_go_to_even():
    for lo_bits in (0x3F80, 0x3F81, 0x4000, 0x4001, 0x0080, 0x0081):
        lo = oracle.bf16_to_double(lo_bits)
        hi = oracle.bf16_to_double(lo_bits + 1)
        mid = 0.5 * (lo + hi)
        want = lo_bits if lo_bits % 2 == 0 else lo_bits + 1
        assert oracle.double_to_bf16(mid) == want


def test_roundtrip_all_finite_values():
    for enc, dec in ((oracle.double_to_f16, oracle.f16_to_double),
                     (oracle.double_to_bf16, oracle.bf16_to_double)):
        for b in range(0, 65536, 7):
            v = dec(b)
            if v == v:
                assert enc(v) == b
