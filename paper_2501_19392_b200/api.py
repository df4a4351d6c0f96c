"""Thin Python binding of libaquakv.so (the C ABI in include/aquakv.h).

Argument marshalling only: torch supplies device memory and the current stream; every step of
encode / decode / decode-attention runs in the library's CUDA kernels.  There is no CPU or
PyTorch fallback: importing this module without the built library raises, and every call
raises `AquaKVError` on a non-zero status.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np
import torch

F16 = 0
BF16 = 1
OP_ENCODE = 0
OP_DECODE = 1
OP_DECODE_ATTN = 2
ROLE_KEY = 0
ROLE_VALUE = 1
NOALLOC_MAX_TOKENS = 1024
KERNEL_PREDICT, KERNEL_ENCODE_ROWS, KERNEL_DECODE_ROWS, KERNEL_ATTN, KERNEL_LAYER, KERNEL_CHAIN = 0, 1, 2, 3, 4, 5
KERNEL_FIT = 6
ERR_NUMERIC = -8
ATTN_SPLIT, ATTN_FUSED = 0, 1
CHAIN_MAX_TOKENS, CHAIN_MAX_LAYERS = 2048, 128

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaquakv.so")

SYMBOLS = [
    "aquakv_code_bytes", "aquakv_search_table_host", "aquakv_create", "aquakv_destroy", "aquakv_workspace_bytes",
    "aquakv_decode_attn_workspace_bytes", "aquakv_predict", "aquakv_encode", "aquakv_decode",
    "aquakv_decode_attn", "aquakv_decode_noalloc", "aquakv_encode_phase", "aquakv_decode_phase", "aquakv_poll_status", "aquakv_launch_count", "aquakv_status_string",
    "aquakv_profile_enable", "aquakv_profile_read", "aquakv_selftest_bounded_wait",
    "aquakv_chain_workspace_bytes", "aquakv_encode_chain", "aquakv_decode_chain",
    "aquakv_fit_workspace_bytes", "aquakv_fit_predictor", "aquakv_gather_rows",
    "aquakv_decode_attn_buffered_workspace_bytes", "aquakv_decode_attn_buffered",
    "aquakv_rope_table", "aquakv_decode_attn_rope_workspace_bytes", "aquakv_decode_attn_rope",
    "aquakv_set_attn_mode",
]


class AquaKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s failed: %d (%s)" % (where, status, status_string(status)))


class Params(ctypes.Structure):
    _fields_ = [("d_kv", ctypes.c_int32), ("had_block", ctypes.c_int32),
                ("scale_group", ctypes.c_int32), ("grid_dim", ctypes.c_int32),
                ("grid_size", ctypes.c_int32), ("dtype", ctypes.c_int32)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError("libaquakv.so is not built (run `python -m paper_2501_19392_b200.build` "
                          "or __graft_entry__.build()); there is no fallback path")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    L.aquakv_code_bytes.restype = ctypes.c_int
    L.aquakv_code_bytes.argtypes = [ctypes.POINTER(Params)]
    L.aquakv_search_table_host.restype = ctypes.c_int
    L.aquakv_search_table_host.argtypes = [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(f32), vp, sz,
                                           ctypes.POINTER(i32)]
    L.aquakv_create.restype = ctypes.c_int
    L.aquakv_create.argtypes = [ctypes.POINTER(Params), vp, vp, vp, ctypes.POINTER(vp)]
    L.aquakv_destroy.restype = ctypes.c_int
    L.aquakv_destroy.argtypes = [vp]
    L.aquakv_workspace_bytes.restype = sz
    L.aquakv_workspace_bytes.argtypes = [vp, i64, ctypes.c_int]
    L.aquakv_decode_attn_workspace_bytes.restype = sz
    L.aquakv_decode_attn_workspace_bytes.argtypes = [vp, i32, i64, i32, i32]
    L.aquakv_predict.restype = ctypes.c_int
    L.aquakv_predict.argtypes = [vp, i64, vp, vp, i64, vp, vp, vp, i64, vp]
    L.aquakv_encode.restype = ctypes.c_int
    L.aquakv_encode.argtypes = [vp, i64, vp, vp, i64, vp, vp, i64, vp, vp, vp, vp,
                                vp, vp, vp, vp, vp, vp, i64, vp, sz, vp]
    L.aquakv_decode.restype = ctypes.c_int
    L.aquakv_decode.argtypes = [vp, i64, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp,
                                vp, vp, i64, vp, sz, vp]
    L.aquakv_decode_noalloc.restype = ctypes.c_int
    L.aquakv_decode_noalloc.argtypes = [vp, i64, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp,
                                        vp, vp, i64, vp]
    L.aquakv_decode_attn.restype = ctypes.c_int
    L.aquakv_decode_attn.argtypes = [vp, i32, i64, i32, i32, i32, f32, vp, vp, vp, vp, vp,
                                     vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, sz, vp]
    L.aquakv_encode_phase.restype = ctypes.c_int
    L.aquakv_encode_phase.argtypes = [vp, ctypes.c_int, i64, vp, i64, vp, vp, i64, vp, vp, vp, vp, vp, i64,
                                      vp, sz, vp]
    L.aquakv_decode_phase.restype = ctypes.c_int
    L.aquakv_decode_phase.argtypes = [vp, ctypes.c_int, i64, vp, vp, vp, vp, i64, vp, vp, vp, i64, vp, sz, vp]
    L.aquakv_poll_status.restype = ctypes.c_int
    L.aquakv_poll_status.argtypes = [vp, vp]
    L.aquakv_launch_count.restype = i64
    L.aquakv_launch_count.argtypes = [vp]
    L.aquakv_profile_enable.restype = ctypes.c_int
    L.aquakv_profile_enable.argtypes = [vp, ctypes.c_int]
    L.aquakv_profile_read.restype = ctypes.c_int
    L.aquakv_profile_read.argtypes = [vp, ctypes.c_int, ctypes.POINTER(i64), ctypes.POINTER(ctypes.c_double)]
    L.aquakv_decode_attn_buffered_workspace_bytes.restype = sz
    L.aquakv_decode_attn_buffered_workspace_bytes.argtypes = [vp, i32, i64, i64, i32, i32]
    L.aquakv_decode_attn_buffered.restype = ctypes.c_int
    L.aquakv_decode_attn_buffered.argtypes = [vp, i32, i64, i32, i32, i32, f32, vp, vp, vp, vp, vp,
                                              vp, vp, i64, vp, vp, vp, vp, vp, vp, i64, i64, vp, vp, vp, vp, i64,
                                              vp, sz, vp]
    L.aquakv_set_attn_mode.restype = ctypes.c_int
    L.aquakv_set_attn_mode.argtypes = [vp, ctypes.c_int]
    L.aquakv_rope_table.restype = ctypes.c_int
    L.aquakv_rope_table.argtypes = [vp, i32, ctypes.c_double, i64, vp, vp]
    L.aquakv_decode_attn_rope_workspace_bytes.restype = sz
    L.aquakv_decode_attn_rope_workspace_bytes.argtypes = [vp, i32, i64, i64, i32, i32]
    L.aquakv_decode_attn_rope.restype = ctypes.c_int
    L.aquakv_decode_attn_rope.argtypes = [vp, i32, i64, i32, i32, i32, f32, vp, vp, vp, vp, vp,
                                          vp, vp, i64, vp, vp, vp, vp, vp, vp, i64, i64, vp, i64, i64, vp,
                                          vp, vp, vp, vp, i64, vp, sz, vp]
    L.aquakv_gather_rows.restype = ctypes.c_int
    L.aquakv_gather_rows.argtypes = [vp, i64, vp, i64, vp, i64, vp, i64, vp]
    L.aquakv_fit_workspace_bytes.restype = sz
    L.aquakv_fit_workspace_bytes.argtypes = [vp, i64, i32]
    L.aquakv_fit_predictor.restype = ctypes.c_int
    L.aquakv_fit_predictor.argtypes = [vp, i64, vp, vp, i64, vp, i64, ctypes.c_double, ctypes.c_int, vp, vp, vp,
                                       vp, sz, vp]
    L.aquakv_chain_workspace_bytes.restype = sz
    L.aquakv_chain_workspace_bytes.argtypes = [vp, i64, i32]
    L.aquakv_encode_chain.restype = ctypes.c_int
    L.aquakv_encode_chain.argtypes = [vp, i64, i32, vp, vp, i64, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64,
                                      vp, sz, vp]
    L.aquakv_decode_chain.restype = ctypes.c_int
    L.aquakv_decode_chain.argtypes = [vp, i64, i32, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, vp, i64, vp, sz, vp]
    L.aquakv_selftest_bounded_wait.restype = ctypes.c_int
    L.aquakv_selftest_bounded_wait.argtypes = [vp, i64, vp]
    L.aquakv_status_string.restype = ctypes.c_char_p
    L.aquakv_status_string.argtypes = [ctypes.c_int]
    return L


lib = _load()


def status_string(status: int) -> str:
    return lib.aquakv_status_string(int(status)).decode()


def code_bytes(d_kv: int, grid_size: int, had_block: int = 64, scale_group: int = 64, dtype: int = BF16) -> int:
    p = Params(d_kv, had_block, scale_group, 2, grid_size, dtype)
    return int(lib.aquakv_code_bytes(ctypes.byref(p)))


SEARCH_TABLE_LIST_WORDS = 4096


def search_table(grid: np.ndarray):
    """(cells_per_side, half_extent, table uint32 [cells, cells], lists uint8 [n_lists, 8]) of
    aquakv_search_table_host: the cell entries and the second-level candidate lists they refer to."""
    g = np.ascontiguousarray(grid, dtype=np.float32)
    cells, half, n_lists = ctypes.c_int32(0), ctypes.c_float(0.0), ctypes.c_int32(0)
    rc = lib.aquakv_search_table_host(g.ctypes.data, g.shape[0], ctypes.byref(cells), ctypes.byref(half), None, 0,
                                      None)
    if rc:
        raise AquaKVError(rc, "aquakv_search_table_host")
    c = cells.value
    buf = np.zeros(c * c + SEARCH_TABLE_LIST_WORDS, dtype=np.uint32)
    rc = lib.aquakv_search_table_host(g.ctypes.data, g.shape[0], ctypes.byref(cells), ctypes.byref(half),
                                      buf.ctypes.data, buf.size, ctypes.byref(n_lists))
    if rc:
        raise AquaKVError(rc, "aquakv_search_table_host")
    lists = buf[c * c:c * c + 2 * n_lists.value].view(np.uint8).reshape(n_lists.value, 8)
    return int(c), float(half.value), buf[:c * c].reshape(c, c).copy(), lists.copy()


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    return int(t)


def _ld(t: Optional[torch.Tensor], default: int) -> int:
    return default if t is None else int(t.stride(0))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


class Codec:
    """One aquakv_ctx.  Tensors are torch CUDA tensors: 16-bit rows [T, d_kv] (stride(1) == 1),
    codes uint8 [T, code_bytes], scales float16 [T, d_kv/scale_group] (both contiguous)."""

    def __init__(self, d_kv: int, had_block: int, scale_group: int, grid: Optional[np.ndarray], dtype: int,
                 signs_k: Optional[np.ndarray] = None, signs_v: Optional[np.ndarray] = None, levels: int = 0):
        """grid [n, 2] (or [256, 4]) with sign vectors: the rotated vector quantizer.  grid None with `levels` = 2^b: the
        uniform round-to-nearest backbone with absmax normalisation; had_block 1 leaves the residual as it is,
        had_block >= 64 (with sign vectors) rotates it first."""
        h = ctypes.c_void_p()
        if grid is None:
            self.params = Params(d_kv, had_block, scale_group, 1, int(levels), dtype)
            sk = None if signs_k is None else np.ascontiguousarray(signs_k, dtype=np.int8)
            sv = None if signs_v is None else np.ascontiguousarray(signs_v, dtype=np.int8)
            rc = lib.aquakv_create(ctypes.byref(self.params), None, None if sk is None else sk.ctypes.data,
                                   None if sv is None else sv.ctypes.data, ctypes.byref(h))
        else:
            # grid [n, 2], or [256, 4]: the four-dimensional grid (per-layer entry points only)
            self.params = Params(d_kv, had_block, scale_group, int(np.asarray(grid).shape[1]),
                                 int(np.asarray(grid).shape[0]), dtype)
            g = np.ascontiguousarray(grid, dtype=np.float32)
            sk = np.ascontiguousarray(signs_k, dtype=np.int8)
            sv = np.ascontiguousarray(signs_v, dtype=np.int8)
            rc = lib.aquakv_create(ctypes.byref(self.params), g.ctypes.data, sk.ctypes.data, sv.ctypes.data,
                                   ctypes.byref(h))
        if rc:
            raise AquaKVError(rc, "aquakv_create")
        self.h = h
        self.d = d_kv
        self.dtype = dtype
        self.torch_dtype = torch.float16 if dtype == F16 else torch.bfloat16
        self.code_bytes = int(lib.aquakv_code_bytes(ctypes.byref(self.params)))
        self.n_groups = d_kv // scale_group
        self._ws = None

    def close(self):
        if getattr(self, "h", None):
            lib.aquakv_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- workspace ----------------------------------------------------------------------------
    def workspace_bytes(self, n_tokens: int, op: int) -> int:
        return int(lib.aquakv_workspace_bytes(self.h, n_tokens, op))

    def decode_attn_workspace_bytes(self, batch: int, ctx_len: int, n_q_heads: int, head_dim: int) -> int:
        return int(lib.aquakv_decode_attn_workspace_bytes(self.h, batch, ctx_len, n_q_heads, head_dim))

    def _workspace(self, nbytes: int, device) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes or self._ws.device != device:
            self._ws = torch.empty(max(nbytes, 256), dtype=torch.uint8, device=device)
        return self._ws

    # -- entry points -----------------------------------------------------------------------------
    def predict(self, in0, in1, W, bias=None, out=None):
        T = in0.shape[0]
        if out is None:
            out = torch.empty((T, self.d), dtype=torch.float32, device=in0.device)
        rc = lib.aquakv_predict(self.h, T, _ptr(in0), _ptr(in1), _ld(in0, self.d), _ptr(W), _ptr(bias),
                                _ptr(out), _ld(out, self.d), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_predict")
        return out

    def encode(self, K, V, Khat_prev=None, Vhat_prev=None, Wk=None, Wv=None, bk=None, bv=None,
               Kcodes=None, Kscales=None, Vcodes=None, Vscales=None, Khat=None, Vhat=None,
               want_hat: bool = True, workspace=None):
        T, dev = K.shape[0], K.device
        if Kcodes is None:
            Kcodes = torch.empty((T, self.code_bytes), dtype=torch.uint8, device=dev)
            Vcodes = torch.empty((T, self.code_bytes), dtype=torch.uint8, device=dev)
            Kscales = torch.empty((T, self.n_groups), dtype=torch.float16, device=dev)
            Vscales = torch.empty((T, self.n_groups), dtype=torch.float16, device=dev)
        if want_hat and Khat is None:
            Khat = torch.empty((T, self.d), dtype=self.torch_dtype, device=dev)
            Vhat = torch.empty((T, self.d), dtype=self.torch_dtype, device=dev)
        ws = workspace if workspace is not None else self._workspace(self.workspace_bytes(T, OP_ENCODE), dev)
        rc = lib.aquakv_encode(self.h, T, _ptr(K), _ptr(V), _ld(K, self.d), _ptr(Khat_prev), _ptr(Vhat_prev),
                               _ld(Khat_prev, self.d), _ptr(Wk), _ptr(Wv), _ptr(bk), _ptr(bv),
                               _ptr(Kcodes), _ptr(Kscales), _ptr(Vcodes), _ptr(Vscales),
                               _ptr(Khat), _ptr(Vhat), _ld(Khat, self.d), _ptr(ws), ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_encode")
        return Kcodes, Kscales, Vcodes, Vscales, Khat, Vhat

    def decode(self, Kcodes, Kscales, Vcodes, Vscales, Khat_prev=None, Vhat_prev=None, Wk=None, Wv=None,
               bk=None, bv=None, Khat=None, Vhat=None, workspace=None):
        T, dev = Kcodes.shape[0], Kcodes.device
        if Khat is None:
            Khat = torch.empty((T, self.d), dtype=self.torch_dtype, device=dev)
            Vhat = torch.empty((T, self.d), dtype=self.torch_dtype, device=dev)
        ws = workspace if workspace is not None else self._workspace(self.workspace_bytes(T, OP_DECODE), dev)
        rc = lib.aquakv_decode(self.h, T, _ptr(Kcodes), _ptr(Kscales), _ptr(Vcodes), _ptr(Vscales),
                               _ptr(Khat_prev), _ptr(Vhat_prev), _ld(Khat_prev, self.d), _ptr(Wk), _ptr(Wv),
                               _ptr(bk), _ptr(bv), _ptr(Khat), _ptr(Vhat), _ld(Khat, self.d),
                               _ptr(ws), ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_decode")
        return Khat, Vhat

    def decode_noalloc(self, Kcodes, Kscales, Vcodes, Vscales, Khat_prev=None, Vhat_prev=None, Wk=None,
                       Wv=None, bk=None, bv=None, Khat=None, Vhat=None):
        """aquakv_decode_noalloc: decode without a workspace, for callers that may not allocate
        device memory; at most NOALLOC_MAX_TOKENS tokens per call.  Khat/Vhat should be passed in by
        such callers (this wrapper creates them with torch only when they are omitted)."""
        T, dev = Kcodes.shape[0], Kcodes.device
        if Khat is None:
            Khat = torch.empty((T, self.d), dtype=self.torch_dtype, device=dev)
            Vhat = torch.empty((T, self.d), dtype=self.torch_dtype, device=dev)
        rc = lib.aquakv_decode_noalloc(self.h, T, _ptr(Kcodes), _ptr(Kscales), _ptr(Vcodes), _ptr(Vscales),
                                       _ptr(Khat_prev), _ptr(Vhat_prev), _ld(Khat_prev, self.d), _ptr(Wk),
                                       _ptr(Wv), _ptr(bk), _ptr(bv), _ptr(Khat), _ptr(Vhat),
                                       _ld(Khat, self.d), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_decode_noalloc")
        return Khat, Vhat

    def decode_attn(self, q, Kcodes, Kscales, Vcodes, Vscales, ctx_len: int, n_kv_heads: int,
                    softmax_scale: float, Khat_prev=None, Vhat_prev=None, Wk=None, Wv=None, bk=None, bv=None,
                    out=None, lse=None, Khat=None, Vhat=None, want_lse: bool = False, workspace=None):
        batch, n_q_heads, head_dim = q.shape
        dev = q.device
        if out is None:
            out = torch.empty_like(q)
        if want_lse and lse is None:
            lse = torch.empty((batch, n_q_heads), dtype=torch.float32, device=dev)
        ws = workspace if workspace is not None else self._workspace(
            self.decode_attn_workspace_bytes(batch, ctx_len, n_q_heads, head_dim), dev)
        rc = lib.aquakv_decode_attn(self.h, batch, ctx_len, n_q_heads, n_kv_heads, head_dim, softmax_scale,
                                    _ptr(q), _ptr(Kcodes), _ptr(Kscales), _ptr(Vcodes), _ptr(Vscales),
                                    _ptr(Khat_prev), _ptr(Vhat_prev), _ld(Khat_prev, self.d), _ptr(Wk), _ptr(Wv),
                                    _ptr(bk), _ptr(bv), _ptr(out), _ptr(lse), _ptr(Khat), _ptr(Vhat),
                                    _ld(Khat, self.d), _ptr(ws), ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_decode_attn")
        return out, lse

    def gather_rows(self, src, idx=None, out=None):
        """Rows idx (int64 device tensor; None = all rows in order) of a 16-bit [T, d] tensor, compact."""
        n = src.shape[0] if idx is None else idx.shape[0]
        if out is None:
            out = torch.empty((n, self.d), dtype=src.dtype, device=src.device)
        rc = lib.aquakv_gather_rows(self.h, n, _ptr(idx), src.shape[0], _ptr(src), _ld(src, self.d), _ptr(out),
                                    _ld(out, self.d), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_gather_rows")
        return out

    def fit_workspace_bytes(self, n_tokens: int, n_inputs: int) -> int:
        return int(lib.aquakv_fit_workspace_bytes(self.h, n_tokens, n_inputs))

    def fit_predictor(self, target, in0, in1=None, rate: float = 1e-3, fit_bias: bool = False,
                      want_fp32: bool = False, workspace=None):
        """One predictor of Algorithm 1 (aquakv_fit_predictor): returns (W [d, n_in*d] 16-bit, bias or None,
        W in fp32 or None)."""
        T, dev = target.shape[0], target.device
        n_in = 2 if in1 is not None else 1
        W = torch.empty((self.d, n_in * self.d), dtype=self.torch_dtype, device=dev)
        W32 = torch.empty((self.d, n_in * self.d), dtype=torch.float32, device=dev) if want_fp32 else None
        bias = torch.empty((self.d,), dtype=torch.float32, device=dev) if fit_bias else None
        ws = workspace if workspace is not None else self._workspace(self.fit_workspace_bytes(T, n_in), dev)
        rc = lib.aquakv_fit_predictor(self.h, T, _ptr(in0), _ptr(in1), _ld(in0, self.d), _ptr(target),
                                      _ld(target, self.d), float(rate), int(bool(fit_bias)), _ptr(W), _ptr(W32),
                                      _ptr(bias), _ptr(ws), ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_fit_predictor")
        return W, bias, W32

    def decode_attn_buffered(self, q, Kcodes, Kscales, Vcodes, Vscales, ctx_len: int, n_kv_heads: int,
                             softmax_scale: float, K16, V16, Khat_prev=None, Vhat_prev=None, Wk=None, Wv=None,
                             bk=None, bv=None, out=None, lse=None, Khat=None, Vhat=None, want_lse: bool = False,
                             workspace=None):
        """decode_attn over the compressed cache plus uncompressed rows K16 / V16 [batch, n, d] (sinks, recent
        tokens); ctx_len may be 0."""
        batch, n_q_heads, head_dim = q.shape
        dev = q.device
        n16 = 0 if K16 is None else K16.shape[1]
        if out is None:
            out = torch.empty_like(q)
        if want_lse and lse is None:
            lse = torch.empty((batch, n_q_heads), dtype=torch.float32, device=dev)
        ws = workspace if workspace is not None else self._workspace(int(
            lib.aquakv_decode_attn_buffered_workspace_bytes(self.h, batch, ctx_len, n16, n_q_heads, head_dim)), dev)
        ld16 = self.d if K16 is None else int(K16.stride(1))
        rc = lib.aquakv_decode_attn_buffered(self.h, batch, ctx_len, n_q_heads, n_kv_heads, head_dim, softmax_scale,
                                             _ptr(q), _ptr(Kcodes), _ptr(Kscales), _ptr(Vcodes), _ptr(Vscales),
                                             _ptr(Khat_prev), _ptr(Vhat_prev), _ld(Khat_prev, self.d), _ptr(Wk),
                                             _ptr(Wv), _ptr(bk), _ptr(bv), _ptr(K16), _ptr(V16), n16, ld16, _ptr(out),
                                             _ptr(lse), _ptr(Khat), _ptr(Vhat), _ld(Khat, self.d), _ptr(ws),
                                             ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_decode_attn_buffered")
        return out, lse

    def set_attn_mode(self, mode: int) -> None:
        """ATTN_SPLIT (default: decode kernel, then attention over the fresh rows) or ATTN_FUSED (attention
        warps inside the decode kernel where the shape allows it)."""
        rc = lib.aquakv_set_attn_mode(self.h, int(mode))
        if rc:
            raise AquaKVError(rc, "aquakv_set_attn_mode")

    def rope_table(self, head_dim: int, theta_base: float, n_positions: int, device=None):
        """fp32 (cos, sin) pairs [n_positions, head_dim/2, 2] of the rotary angles, evaluated in double."""
        dev = device if device is not None else torch.device("cuda", torch.cuda.current_device())
        table = torch.empty((n_positions, head_dim // 2, 2), dtype=torch.float32, device=dev)
        rc = lib.aquakv_rope_table(self.h, head_dim, float(theta_base), n_positions, _ptr(table), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_rope_table")
        return table

    def decode_attn_rope(self, q, Kcodes, Kscales, Vcodes, Vscales, ctx_len: int, n_kv_heads: int,
                         softmax_scale: float, rope_table, pos0: int = 0, K16=None, V16=None, pos16=None,
                         Khat_prev=None, Vhat_prev=None, Wk=None, Wv=None, bk=None, bv=None, out=None, lse=None,
                         Khat=None, Vhat=None, want_lse: bool = False, workspace=None):
        """decode_attn_buffered over pre-RoPE keys: compressed token t sits at position pos0 + t, uncompressed
        row r at pos16[r] (int32, device); q is rotated by the caller."""
        batch, n_q_heads, head_dim = q.shape
        dev = q.device
        n16 = 0 if K16 is None else K16.shape[1]
        if out is None:
            out = torch.empty_like(q)
        if want_lse and lse is None:
            lse = torch.empty((batch, n_q_heads), dtype=torch.float32, device=dev)
        ws = workspace if workspace is not None else self._workspace(int(
            lib.aquakv_decode_attn_rope_workspace_bytes(self.h, batch, ctx_len, n16, n_q_heads, head_dim)), dev)
        ld16 = self.d if K16 is None else int(K16.stride(1))
        rc = lib.aquakv_decode_attn_rope(self.h, batch, ctx_len, n_q_heads, n_kv_heads, head_dim, softmax_scale,
                                         _ptr(q), _ptr(Kcodes), _ptr(Kscales), _ptr(Vcodes), _ptr(Vscales),
                                         _ptr(Khat_prev), _ptr(Vhat_prev), _ld(Khat_prev, self.d), _ptr(Wk),
                                         _ptr(Wv), _ptr(bk), _ptr(bv), _ptr(K16), _ptr(V16), n16, ld16,
                                         _ptr(rope_table), int(rope_table.shape[0]), int(pos0), _ptr(pos16),
                                         _ptr(out), _ptr(lse), _ptr(Khat), _ptr(Vhat), _ld(Khat, self.d), _ptr(ws),
                                         ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_decode_attn_rope")
        return out, lse

    def encode_phase(self, role: int, X, in0=None, in1=None, W=None, bias=None, want_hat: bool = True):
        T, dev = X.shape[0], X.device
        codes = torch.empty((T, self.code_bytes), dtype=torch.uint8, device=dev)
        scales = torch.empty((T, self.n_groups), dtype=torch.float16, device=dev)
        hat = torch.empty((T, self.d), dtype=self.torch_dtype, device=dev) if want_hat else None
        ws = self._workspace(self.workspace_bytes(T, OP_ENCODE), dev)
        rc = lib.aquakv_encode_phase(self.h, role, T, _ptr(X), _ld(X, self.d), _ptr(in0), _ptr(in1),
                                     _ld(in0, self.d), _ptr(W), _ptr(bias), _ptr(codes), _ptr(scales),
                                     _ptr(hat), _ld(hat, self.d), _ptr(ws), ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_encode_phase")
        return codes, scales, hat

    def decode_phase(self, role: int, codes, scales, in0=None, in1=None, W=None, bias=None):
        T, dev = codes.shape[0], codes.device
        hat = torch.empty((T, self.d), dtype=self.torch_dtype, device=dev)
        ws = self._workspace(self.workspace_bytes(T, OP_DECODE), dev)
        rc = lib.aquakv_decode_phase(self.h, role, T, _ptr(codes), _ptr(scales), _ptr(in0), _ptr(in1),
                                     _ld(in0, self.d), _ptr(W), _ptr(bias), _ptr(hat), _ld(hat, self.d),
                                     _ptr(ws), ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_decode_phase")
        return hat

    # -- all layers of a small call in one launch ---------------------------------------------------
    @staticmethod
    def _ptr_array(tensors, n):
        """Host array of n device pointers (None entries and a None list give NULL)."""
        if tensors is None:
            return None
        assert len(tensors) == n
        return (ctypes.c_void_p * n)(*[_ptr(t) for t in tensors])

    def chain_workspace_bytes(self, n_tokens: int, n_layers: int) -> int:
        return int(lib.aquakv_chain_workspace_bytes(self.h, n_tokens, n_layers))

    def encode_chain(self, K, V, Wk, Wv, Kcodes, Kscales, Vcodes, Vscales, bk=None, bv=None, Khat=None, Vhat=None,
                     Khat_init=None, Vhat_init=None, workspace=None):
        """Lists with one entry per layer (Wk[l] = Wv[l] = None: no predictor for layer l)."""
        L, T = len(K), int(K[0].shape[0])
        ws = workspace if workspace is not None else self._workspace(self.chain_workspace_bytes(T, L), K[0].device)
        arr = lambda ts: self._ptr_array(ts, L)
        hats = [t for t in (Khat or []) if t is not None]
        rc = lib.aquakv_encode_chain(self.h, T, L, arr(K), arr(V), _ld(K[0], self.d), _ptr(Khat_init), _ptr(Vhat_init),
                                     _ld(Khat_init, self.d), arr(Wk), arr(Wv), arr(bk), arr(bv), arr(Kcodes),
                                     arr(Kscales), arr(Vcodes), arr(Vscales), arr(Khat), arr(Vhat),
                                     _ld(hats[0] if hats else None, self.d), _ptr(ws), ws.numel(), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_encode_chain")

    def decode_chain(self, Kcodes, Kscales, Vcodes, Vscales, Wk, Wv, bk=None, bv=None, Khat=None, Vhat=None,
                     Khat_init=None, Vhat_init=None, workspace=None):
        L, T = len(Kcodes), int(Kcodes[0].shape[0])
        ws = workspace if workspace is not None else self._workspace(self.chain_workspace_bytes(T, L), Kcodes[0].device)
        arr = lambda ts: self._ptr_array(ts, L)
        hats = [t for t in (Khat or []) if t is not None]
        rc = lib.aquakv_decode_chain(self.h, T, L, arr(Kcodes), arr(Kscales), arr(Vcodes), arr(Vscales), _ptr(Khat_init),
                                     _ptr(Vhat_init), _ld(Khat_init, self.d), arr(Wk), arr(Wv), arr(bk), arr(bv),
                                     arr(Khat), arr(Vhat), _ld(hats[0] if hats else None, self.d), _ptr(ws), ws.numel(),
                                     _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_decode_chain")

    def poll_status(self) -> int:
        return int(lib.aquakv_poll_status(self.h, _stream()))

    def launch_count(self) -> int:
        return int(lib.aquakv_launch_count(self.h))

    def selftest_bounded_wait(self, limit_ns: int) -> None:
        rc = lib.aquakv_selftest_bounded_wait(self.h, int(limit_ns), _stream())
        if rc:
            raise AquaKVError(rc, "aquakv_selftest_bounded_wait")

    def profile_enable(self, enable: bool) -> None:
        rc = lib.aquakv_profile_enable(self.h, 1 if enable else 0)
        if rc:
            raise AquaKVError(rc, "aquakv_profile_enable")

    def profile_read(self, kernel_class: int):
        n, ms = ctypes.c_int64(0), ctypes.c_double(0.0)
        rc = lib.aquakv_profile_read(self.h, kernel_class, ctypes.byref(n), ctypes.byref(ms))
        if rc:
            raise AquaKVError(rc, "aquakv_profile_read")
        return int(n.value), float(ms.value)
