"""Shared helpers for the tests (no codec arithmetic beyond bit unpacking of the documented layout)."""
import numpy as np
import torch

from paper_2501_19392_b200 import synth


def read_golden(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


def unpack_codes(codes: np.ndarray, bits: int) -> np.ndarray:
    """Documented layout: pair j's code occupies bits [j*bits, (j+1)*bits) of the row, LSB first."""
    T = codes.shape[0]
    b = np.unpackbits(codes, axis=1, bitorder="little").reshape(T, -1, bits)
    w = (1 << np.arange(bits)).astype(np.int64)
    return (b.astype(np.int64) * w).sum(-1)


def pack_codes(idx: np.ndarray, bits: int) -> np.ndarray:
    T, n = idx.shape
    b = ((idx[:, :, None] >> np.arange(bits)[None, None, :]) & 1).astype(np.uint8).reshape(T, n * bits)
    return np.packbits(b, axis=1, bitorder="little")


def bits_to_f64(a: np.ndarray, dtype: int) -> np.ndarray:
    return synth.from_bits(a, dtype).to(torch.float64).numpy()


def f64_to_bits(a: np.ndarray, dtype: int) -> np.ndarray:
    """Round float64 -> 16-bit through float32 (callers pass values exactly representable in fp32)."""
    t = torch.from_numpy(np.ascontiguousarray(a)).to(torch.float32).to(synth.torch_dtype(dtype))
    return synth.to_bits(t)
