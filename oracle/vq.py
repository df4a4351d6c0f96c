"""CPU oracle of the backbone vector quantizer for a grid of ANY dimension p (Section 2 "Vector
Quantization" and Section 4.1 "Alternative quantizers": besides the p = 2 grids with n = 16 / 64 / 256
points the paper runs one 2-bit grid with d = 4, n = 256, for which it had no fast GPU kernel -- its d is
the grid dimension, written p here).

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain numpy in double precision.

The steps are those of the p = 2 quantizer in aquakv_oracle.c, with consecutive p-tuples in place of
pairs: the group scale is the root mean square of the group's residual, stored as fp16 (clamped to the
largest finite fp16); the residual is normalised with the ROUNDED scale, multiplied by the role's signs
and rotated by the orthonormal Hadamard matrix in blocks of h values; every consecutive p-tuple of
rotated values goes to the nearest grid point (squared Euclidean distance, lowest index on a tie); the
code of tuple j occupies bits [j b, (j + 1) b) of the row's byte stream, b = log2 n, LSB first.
Q^-1 looks the points up, rotates back, applies the signs and multiplies by the scale.
"""
from __future__ import annotations

from typing import Optional, Sequence

import numpy as np

from . import F16, Oracle
from .calibration import bits_to_double, double_to_bits
from .uniform import _pack, _unpack, rotate, rotate_back


class VectorOracle:
    """`linear` is a codec oracle of the same width and 16-bit type, used for the predictor product only."""

    def __init__(self, linear: Oracle, grid: np.ndarray, had_block: int, scale_group: int,
                 signs_k: np.ndarray, signs_v: np.ndarray):
        self.grid = np.ascontiguousarray(grid, dtype=np.float32).astype(np.float64)
        self.n, self.p = self.grid.shape
        self.b = int(round(np.log2(self.n)))
        assert 1 << self.b == self.n
        self.linear, self.h, self.g = linear, had_block, scale_group
        self.d, self.dtype = linear.d, linear.dtype
        assert self.d % self.p == 0 and (self.d // self.p * self.b) % 8 == 0
        self.code_bytes = self.d // self.p * self.b // 8
        self.n_groups = self.d // scale_group
        self.signs = {"k": np.asarray(signs_k), "v": np.asarray(signs_v)}

    def quantize(self, R: np.ndarray, role: str = "k"):
        """Q on double residuals R [T, d]: codes, scales (fp16 bits), margins per tuple
        ((second - best) / (second + best) of the two smallest squared distances), unrounded scales, and Y,
        the rotated normalised values the points were chosen for."""
        R = np.asarray(R, dtype=np.float64)
        T, d = R.shape
        G = R.reshape(T, d // self.g, self.g)
        s_exact = np.sqrt((G * G).sum(axis=2) / float(self.g))
        s16_bits = double_to_bits(np.minimum(s_exact, 65504.0), F16)
        s16 = bits_to_double(s16_bits, F16)
        inv = np.where(s16 > 0, 1.0 / np.where(s16 > 0, s16, 1.0), 0.0)
        Y = rotate((G * inv[:, :, None]).reshape(T, d), self.signs[role], self.h)
        idx = np.empty((T, d // self.p), dtype=np.int64)
        margins = np.empty((T, d // self.p), dtype=np.float64)
        for t in range(T):                                   # one row at a time: [d/p, n] distances
            v = Y[t].reshape(d // self.p, self.p)
            dist = ((v[:, None, :] - self.grid[None, :, :]) ** 2).sum(axis=2)
            idx[t] = dist.argmin(axis=1)                     # numpy's argmin: the lowest index on a tie
            two = np.partition(dist, 1, axis=1)[:, :2]
            margins[t] = (two[:, 1] - two[:, 0]) / (two[:, 1] + two[:, 0] + 1e-30)
        return dict(codes=_pack(idx, self.b), scales=s16_bits, margins=margins, scales_exact=s_exact, Y=Y)

    def dequantize(self, codes: np.ndarray, scales: np.ndarray, role: str = "k") -> np.ndarray:
        T = codes.shape[0]
        idx = _unpack(codes, self.b, self.d // self.p)
        Yhat = self.grid[idx].reshape(T, self.d)
        s16 = bits_to_double(np.ascontiguousarray(scales, dtype=np.uint16).reshape(T, self.n_groups), F16)
        X = rotate_back(Yhat, self.signs[role], self.h)
        return (X.reshape(T, self.n_groups, self.g) * s16[:, :, None]).reshape(T, self.d)

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
