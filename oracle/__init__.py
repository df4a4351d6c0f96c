"""Python face of the CPU oracle (oracle/aquakv_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's
CPU-baseline leg.  The CUDA library and its Python binding never import this package, and this
package imports nothing from them.

16-bit tensors (fp16 / bf16) travel as numpy uint16 arrays of raw bits; everything the oracle
computes internally is double precision.  See the C file's header for the paper passages each
step follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

F16 = 0
BF16 = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aquakv_oracle.c")
_LIB = os.path.join(_HERE, "libaquakv_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp, no BLAS, no intrinsics)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Params(ctypes.Structure):
    _fields_ = [("d_kv", ctypes.c_int32), ("had_block", ctypes.c_int32),
                ("scale_group", ctypes.c_int32), ("grid_size", ctypes.c_int32),
                ("dtype", ctypes.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.aqo_f16_to_double.restype = ctypes.c_double
        L.aqo_f16_to_double.argtypes = [ctypes.c_uint16]
        L.aqo_bf16_to_double.restype = ctypes.c_double
        L.aqo_bf16_to_double.argtypes = [ctypes.c_uint16]
        L.aqo_double_to_f16.restype = ctypes.c_uint16
        L.aqo_double_to_f16.argtypes = [ctypes.c_double]
        L.aqo_double_to_bf16.restype = ctypes.c_uint16
        L.aqo_double_to_bf16.argtypes = [ctypes.c_double]
        L.aqo_num_threads.restype = ctypes.c_int
        L.aqo_set_num_threads.argtypes = [ctypes.c_int]
        L.aqo_code_bytes.restype = ctypes.c_int
        _lib = L
    return _lib


def _p(a: Optional[np.ndarray]):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


def _u16(a, shape=None) -> Optional[np.ndarray]:
    if a is None:
        return None
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    if shape is not None:
        assert tuple(a.shape) == tuple(shape), (a.shape, shape)
    return a


def num_threads() -> int:
    return int(lib().aqo_num_threads())


def set_num_threads(n: int) -> None:
    lib().aqo_set_num_threads(int(n))


def hadamard_definition(x: np.ndarray) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty_like(x)
    lib().aqo_hadamard_definition(_p(x), _p(y), ctypes.c_int(x.shape[0]))
    return y


def hadamard_butterfly(x: np.ndarray) -> np.ndarray:
    y = np.array(x, dtype=np.float64, order="C", copy=True)
    lib().aqo_hadamard_butterfly(_p(y), ctypes.c_int(y.shape[0]))
    return y


def f16_to_double(bits: int) -> float:
    return float(lib().aqo_f16_to_double(int(bits)))


def bf16_to_double(bits: int) -> float:
    return float(lib().aqo_bf16_to_double(int(bits)))


def double_to_f16(x: float) -> int:
    return int(lib().aqo_double_to_f16(float(x)))


def double_to_bf16(x: float) -> int:
    return int(lib().aqo_double_to_bf16(float(x)))


def attention(dtype: int, batch: int, ctx: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
              softmax_scale: float, q: np.ndarray, Khat: np.ndarray, Vhat: np.ndarray):
    """softmax(scale * q K^T) V per (sequence, query head) over the decoded cache, in double.
    q uint16 [batch, n_q_heads, head_dim]; Khat/Vhat uint16 [batch*ctx, n_kv_heads*head_dim].
    Returns (out float64 [batch, n_q_heads, head_dim], lse float64 [batch, n_q_heads])."""
    d = n_kv_heads * head_dim
    q = _u16(q, (batch, n_q_heads, head_dim))
    Khat = _u16(Khat, (batch * ctx, d))
    Vhat = _u16(Vhat, (batch * ctx, d))
    out = np.empty((batch, n_q_heads, head_dim), dtype=np.float64)
    lse = np.empty((batch, n_q_heads), dtype=np.float64)
    rc = lib().aqo_attention(ctypes.c_int(dtype), ctypes.c_int32(batch), ctypes.c_int64(ctx),
                             ctypes.c_int32(n_q_heads), ctypes.c_int32(n_kv_heads),
                             ctypes.c_int32(head_dim), ctypes.c_double(softmax_scale),
                             _p(q), _p(Khat), _p(Vhat), _p(out), _p(lse))
    if rc:
        raise ValueError("aqo_attention: bad arguments")
    return out, lse


class Oracle:
    """The codec for one parameter set: grid float32 [n,2], signs int8 [d_kv] per tensor role."""

    def __init__(self, d_kv: int, had_block: int, scale_group: int, grid: np.ndarray, dtype: int,
                 signs_k: np.ndarray, signs_v: np.ndarray):
        self.grid = np.ascontiguousarray(grid, dtype=np.float32)
        assert self.grid.ndim == 2 and self.grid.shape[1] == 2
        self.params = _Params(d_kv, had_block, scale_group, self.grid.shape[0], dtype)
        self.signs = {"k": np.ascontiguousarray(signs_k, dtype=np.int8),
                      "v": np.ascontiguousarray(signs_v, dtype=np.int8)}
        assert self.signs["k"].shape == (d_kv,) and self.signs["v"].shape == (d_kv,)
        self.d = d_kv
        self.dtype = dtype
        self.code_bytes = int(lib().aqo_code_bytes(ctypes.byref(self.params)))
        self.n_groups = d_kv // scale_group

    # -- Q / Q^-1 on double residuals ---------------------------------------------------------
    def quantize(self, R: np.ndarray, role: str = "k"):
        R = np.ascontiguousarray(R, dtype=np.float64)
        T = R.shape[0]
        assert R.shape == (T, self.d)
        out = dict(codes=np.zeros((T, self.code_bytes), np.uint8),
                   scales=np.zeros((T, self.n_groups), np.uint16),
                   margins=np.zeros((T, self.d // 2), np.float64),
                   scales_exact=np.zeros((T, self.n_groups), np.float64),
                   Y=np.zeros((T, self.d), np.float64))
        rc = lib().aqo_quantize(ctypes.byref(self.params), _p(self.grid), _p(self.signs[role]),
                                ctypes.c_int64(T), _p(R), _p(out["codes"]), _p(out["scales"]),
                                _p(out["margins"]), _p(out["scales_exact"]), _p(out["Y"]))
        if rc:
            raise ValueError("aqo_quantize: bad parameters")
        return out

    def dequantize(self, codes: np.ndarray, scales: np.ndarray, role: str = "k") -> np.ndarray:
        codes = np.ascontiguousarray(codes, dtype=np.uint8)
        T = codes.shape[0]
        assert codes.shape == (T, self.code_bytes)
        scales = _u16(scales, (T, self.n_groups))
        X = np.zeros((T, self.d), np.float64)
        rc = lib().aqo_dequantize(ctypes.byref(self.params), _p(self.grid), _p(self.signs[role]),
                                  ctypes.c_int64(T), _p(codes), _p(scales), _p(X))
        if rc:
            raise ValueError("aqo_dequantize: bad parameters")
        return X

    # -- predictor ----------------------------------------------------------------------------
    def predict(self, inputs: Sequence[np.ndarray], W: Optional[np.ndarray],
                bias: Optional[np.ndarray] = None) -> np.ndarray:
        n_in = len(inputs)
        T = inputs[0].shape[0]
        ins = [_u16(a, (T, self.d)) for a in inputs]
        W = _u16(W, (self.d, n_in * self.d)) if W is not None else None
        bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
        P = np.zeros((T, self.d), np.float64)
        rc = lib().aqo_predict(ctypes.byref(self.params), ctypes.c_int64(T), ctypes.c_int(n_in),
                               _p(ins[0]), _p(ins[1]) if n_in > 1 else None, _p(W), _p(bias), _p(P))
        if rc:
            raise ValueError("aqo_predict: bad arguments")
        return P

    # -- one phase of Algorithm 2 / 3 -----------------------------------------------------------
    def encode_phase(self, X: np.ndarray, inputs: Sequence[np.ndarray], W: Optional[np.ndarray],
                     bias: Optional[np.ndarray] = None, role: str = "k"):
        T = X.shape[0]
        X = _u16(X, (T, self.d))
        n_in = len(inputs) if W is not None else 0
        ins = [_u16(a, (T, self.d)) for a in inputs] if W is not None else []
        W = _u16(W, (self.d, n_in * self.d)) if W is not None else None
        bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
        out = dict(codes=np.zeros((T, self.code_bytes), np.uint8),
                   scales=np.zeros((T, self.n_groups), np.uint16),
                   hat=np.zeros((T, self.d), np.uint16),
                   margins=np.zeros((T, self.d // 2), np.float64),
                   scales_exact=np.zeros((T, self.n_groups), np.float64),
                   hat_exact=np.zeros((T, self.d), np.float64),
                   pred=np.zeros((T, self.d), np.float64))
        rc = lib().aqo_encode_phase(
            ctypes.byref(self.params), _p(self.grid), _p(self.signs[role]), ctypes.c_int64(T),
            _p(X), ctypes.c_int(n_in), _p(ins[0]) if n_in > 0 else None,
            _p(ins[1]) if n_in > 1 else None, _p(W), _p(bias),
            _p(out["codes"]), _p(out["scales"]), _p(out["hat"]), _p(out["margins"]),
            _p(out["scales_exact"]), _p(out["hat_exact"]), _p(out["pred"]))
        if rc:
            raise ValueError("aqo_encode_phase: bad arguments")
        return out

    def decode_phase(self, codes: np.ndarray, scales: np.ndarray, inputs: Sequence[np.ndarray],
                     W: Optional[np.ndarray], bias: Optional[np.ndarray] = None, role: str = "k"):
        codes = np.ascontiguousarray(codes, dtype=np.uint8)
        T = codes.shape[0]
        scales = _u16(scales, (T, self.n_groups))
        n_in = len(inputs) if W is not None else 0
        ins = [_u16(a, (T, self.d)) for a in inputs] if W is not None else []
        W = _u16(W, (self.d, n_in * self.d)) if W is not None else None
        bias = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
        hat = np.zeros((T, self.d), np.uint16)
        hat_exact = np.zeros((T, self.d), np.float64)
        rc = lib().aqo_decode_phase(
            ctypes.byref(self.params), _p(self.grid), _p(self.signs[role]), ctypes.c_int64(T),
            _p(codes), _p(scales), ctypes.c_int(n_in), _p(ins[0]) if n_in > 0 else None,
            _p(ins[1]) if n_in > 1 else None, _p(W), _p(bias), _p(hat), _p(hat_exact))
        if rc:
            raise ValueError("aqo_decode_phase: bad arguments")
        return dict(hat=hat, hat_exact=hat_exact)

    # -- Algorithm 2 / Algorithm 3 for one layer -------------------------------------------------
    def encode_layer(self, K, V, Khat_prev=None, Vhat_prev=None, Wk=None, Wv=None, bk=None, bv=None):
        k = self.encode_phase(K, [Khat_prev], Wk, bk, "k")
        v = self.encode_phase(V, [Vhat_prev, k["hat"]], Wv, bv, "v")
        return k, v

    def decode_layer(self, Kcodes, Kscales, Vcodes, Vscales, Khat_prev=None, Vhat_prev=None,
                     Wk=None, Wv=None, bk=None, bv=None):
        k = self.decode_phase(Kcodes, Kscales, [Khat_prev], Wk, bk, "k")
        v = self.decode_phase(Vcodes, Vscales, [Vhat_prev, k["hat"]], Wv, bv, "v")
        return k, v
