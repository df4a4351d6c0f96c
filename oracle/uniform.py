"""CPU oracle of the alternative backbone quantizer: round-to-nearest on a uniform grid with absmax
normalisation per group, applied per token (Section 4.1 "Alternative quantizers": the Quanto-style
backbone, plain rounding to the nearest level after dividing by the group's largest magnitude, groups of
64 values inside a token; Section 3.2: any quantizer Q can sit under the predictors).

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain numpy in double precision.

Reading (the paper names the scheme, not its arithmetic).  For b bits per value the levels are the
2^b signed integers -2^(b-1) .. 2^(b-1)-1 times the group scale; the scale is absmax / 2^(b-1), stored
as fp16 (clamped to the largest finite fp16) and it is the ROUNDED scale that normalises, so encoder
and decoder agree; a value goes to the nearest level, the lower one on an exact tie (the codec's rule
"lowest index wins"), and saturates at the ends (the group's positive maximum maps to 2^(b-1)-1); a
group of zeros has scale 0 and level 0.  The code of a value is its level + 2^(b-1) as an unsigned
b-bit number; codes are packed LSB-first in value order; no rotation, no sign flips.  Predictors,
residual and add-back are those of Algorithms 2 and 3: codes = Q(x - pred), hat = round16(pred + Q^-1).

Rotated variant (the appendix' additional results for Section 4.1: a backbone that puts a randomized
Hadamard transform in front of ordinary scalar quantization, group size 1024).  Reading: the
residual is multiplied by the role's random signs and rotated by the orthonormal Hadamard matrix in
blocks of `had_block` values (the transform of Section 3.1's vector quantizer), the ROTATED values are
quantized as above (the group's absmax is taken after the rotation), and Q^-1 rotates the levels times
scale back and multiplies by the signs again: Q(r) = U(H (s . r) / sqrt(h)), Q^-1 = s . H(U^-1) / sqrt(h).
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np

from . import F16, Oracle, hadamard_butterfly
from .calibration import bits_to_double, double_to_bits


def _pack(levels_unsigned: np.ndarray, b: int) -> np.ndarray:
    """[T, d] unsigned b-bit numbers -> [T, d*b/8] bytes, LSB-first in value order."""
    T, d = levels_unsigned.shape
    bits = ((levels_unsigned[:, :, None] >> np.arange(b)[None, None, :]) & 1).astype(np.uint8).reshape(T, d * b)
    return np.packbits(bits, axis=1, bitorder="little")


def _unpack(codes: np.ndarray, b: int, d: int) -> np.ndarray:
    T = codes.shape[0]
    bits = np.unpackbits(np.ascontiguousarray(codes, dtype=np.uint8), axis=1, bitorder="little")[:, :d * b]
    return (bits.reshape(T, d, b).astype(np.int64) << np.arange(b)[None, None, :]).sum(axis=2)


def quantize(R: np.ndarray, b: int, g: int):
    """Q on double residuals R [T, d].  Returns codes, scales (fp16 bits), margins (distance of every
    normalised value from the nearest decision boundary, in level spacings) and the unrounded scales."""
    R = np.asarray(R, dtype=np.float64)
    T, d = R.shape
    half = 1 << (b - 1)
    G = R.reshape(T, d // g, g)
    s_exact = np.abs(G).max(axis=2) / half
    s16_bits = double_to_bits(np.minimum(s_exact, 65504.0), F16)
    s16 = bits_to_double(s16_bits, F16)
    with np.errstate(divide="ignore", invalid="ignore"):
        x = np.where(s16[:, :, None] > 0, G / np.where(s16 > 0, s16, 1.0)[:, :, None], 0.0)
    q = np.ceil(x - 0.5)                                   # nearest integer, the lower one on a tie
    q = np.clip(q, -half, half - 1)
    # decision boundaries are the half-integers between neighbouring levels: -half + 0.5 .. half - 1.5
    boundary = np.clip(np.floor(x) + 0.5, -half + 0.5, half - 1.5)
    margins = np.abs(x - boundary)
    codes = _pack((q + half).astype(np.int64).reshape(T, d), b)
    return dict(codes=codes, scales=s16_bits, margins=margins.reshape(T, d), scales_exact=s_exact)


def dequantize(codes: np.ndarray, scales: np.ndarray, b: int, g: int, d: int) -> np.ndarray:
    """Q^-1 to double: level * scale."""
    T = codes.shape[0]
    q = _unpack(codes, b, d) - (1 << (b - 1))
    s16 = bits_to_double(np.ascontiguousarray(scales, dtype=np.uint16).reshape(T, d // g), F16)
    return (q.reshape(T, d // g, g) * s16[:, :, None]).reshape(T, d)


def rotate(R: np.ndarray, signs: np.ndarray, h: int) -> np.ndarray:
    """Rows of R times the signs, then the orthonormal Hadamard transform of every block of h values."""
    R = np.asarray(R, dtype=np.float64) * np.asarray(signs, dtype=np.float64)[None, :]
    Y = np.empty_like(R)
    for t in range(R.shape[0]):
        for o in range(0, R.shape[1], h):
            Y[t, o:o + h] = hadamard_butterfly(R[t, o:o + h]) / np.sqrt(float(h))
    return Y


def rotate_back(Y: np.ndarray, signs: np.ndarray, h: int) -> np.ndarray:
    """Inverse of `rotate`: the Hadamard matrix is symmetric and orthonormal, the signs are +-1."""
    Y = np.asarray(Y, dtype=np.float64)
    R = np.empty_like(Y)
    for t in range(Y.shape[0]):
        for o in range(0, Y.shape[1], h):
            R[t, o:o + h] = hadamard_butterfly(Y[t, o:o + h]) / np.sqrt(float(h))
    return R * np.asarray(signs, dtype=np.float64)[None, :]


class UniformOracle:
    """Algorithm 2 / 3 phases with the uniform backbone.  `linear` is a codec oracle of the same width
    and 16-bit type, used for the predictor product only."""

    def __init__(self, linear: Oracle, bits: int, group: int, had_block: int = 1,
                 signs_k: Optional[np.ndarray] = None, signs_v: Optional[np.ndarray] = None):
        self.linear, self.b, self.g, self.h = linear, bits, group, had_block
        self.d, self.dtype = linear.d, linear.dtype
        self.code_bytes = self.d * bits // 8
        self.n_groups = self.d // group
        self.signs = {"k": signs_k, "v": signs_v}
        assert had_block == 1 or (signs_k is not None and signs_v is not None)

    def quantize(self, R: np.ndarray, role: str = "k"):
        """Q on double residuals (rotated first when had_block > 1); `Y` is what the levels were chosen for."""
        Y = rotate(R, self.signs[role], self.h) if self.h > 1 else np.asarray(R, dtype=np.float64)
        out = quantize(Y, self.b, self.g)
        out["Y"] = Y
        return out

    def dequantize(self, codes, scales, role: str = "k") -> np.ndarray:
        Yhat = dequantize(codes, scales, self.b, self.g, self.d)
        return rotate_back(Yhat, self.signs[role], self.h) if self.h > 1 else Yhat

    def _pred(self, T, inputs, W, bias):
        if W is None:
            return np.zeros((T, self.d), np.float64)
        return self.linear.predict(list(inputs), W, bias)

    def encode_phase(self, X: np.ndarray, inputs: Sequence[np.ndarray], W: Optional[np.ndarray],
                     bias: Optional[np.ndarray] = None, role: str = "k"):
        x = bits_to_double(X, self.dtype)
        pred = self._pred(x.shape[0], inputs, W, bias)
        out = self.quantize(x - pred, role)                                        # Algorithm 2: quantize the residual
        hat_exact = pred + self.dequantize(out["codes"], out["scales"], role)      # ... and reconstruct
        out.update(hat=double_to_bits(hat_exact, self.dtype), hat_exact=hat_exact, pred=pred)
        return out

    def decode_phase(self, codes, scales, inputs, W, bias=None, role: str = "k"):
        T = codes.shape[0]
        hat_exact = self._pred(T, inputs, W, bias) + self.dequantize(codes, scales, role)   # Algorithm 3: add the prediction back
        return dict(hat=double_to_bits(hat_exact, self.dtype), hat_exact=hat_exact)
