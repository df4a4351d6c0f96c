"""Seeded synthetic inputs for the AQUA-KV codec: shapes, grids, signs, adapters, caches.

This module serves BOTH the CPU oracle and the CUDA library, so it holds none of the codec's
arithmetic (no prediction, no rotation, no nearest-point search, no packing).  It only draws
numbers: Llama-3.x-shaped key/value tensors with the cross-layer "linear map plus noise"
structure the paper measures with its probes (Section 3.1, Figure 2), random linear adapters,
random +-1 Hadamard signs, a Gaussian-optimal 2-D grid (Section 2, "Vector Quantization": a
lattice optimised for normally distributed vectors; built here by Lloyd iterations), and random
packed caches for the bulk-decode workloads.

Every tensor is a torch tensor so the same stored values can be handed to the oracle (through
`to_bits(...)` -> numpy) and to the CUDA library (through `.data_ptr()`).
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional

import numpy as np
import torch

F16 = 0
BF16 = 1

_TORCH_DTYPE = {F16: torch.float16, BF16: torch.bfloat16}


def torch_dtype(dtype: int) -> torch.dtype:
    return _TORCH_DTYPE[dtype]


def to_bits(t: torch.Tensor) -> np.ndarray:
    """Raw 16-bit storage of an fp16/bf16 tensor as a C-contiguous numpy uint16 array."""
    assert t.dtype in (torch.float16, torch.bfloat16)
    return t.detach().contiguous().cpu().view(torch.uint16).numpy()


def from_bits(a: np.ndarray, dtype: int, device="cpu") -> torch.Tensor:
    """Inverse of `to_bits`."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint16)).view(torch_dtype(dtype))
    return t.to(device)


@dataclasses.dataclass(frozen=True)
class Shape:
    """One workload shape.  d_kv = n_kv_heads * head_dim."""

    name: str
    n_kv_heads: int
    head_dim: int
    n_q_heads: int
    n_layers: int
    n_tokens: int
    dtype: int
    had_block: int
    scale_group: int
    grid_size: int
    channel_scales: bool = False   # heavy-tailed per-channel scales (log-normal)
    batch: int = 1                 # sequences (decode-attention: n_tokens = batch * ctx)

    @property
    def d_kv(self) -> int:
        return self.n_kv_heads * self.head_dim

    @property
    def code_bits(self) -> int:
        return int(round(math.log2(self.grid_size)))

    @property
    def code_bytes(self) -> int:
        return self.d_kv // 2 * self.code_bits // 8

    @property
    def n_groups(self) -> int:
        return self.d_kv // self.scale_group


# The five benchmark workloads (Llama-3.x-shaped, synthetic).  `n_layers`/`n_tokens` are the full
# sizes; tests shrink them with dataclasses.replace.
CONFIGS = {
    1: Shape("llama3.2-1b-2layer-roundtrip", 8, 64, 32, 2, 1024, F16, 64, 64, 16),
    2: Shape("llama3.2-3b-prefill-encode", 8, 128, 24, 28, 32768, BF16, 1024, 1024, 16,
             channel_scales=True),
    3: Shape("llama3.1-8b-decode-step-encode", 8, 128, 32, 32, 64, BF16, 1024, 1024, 16),
    4: Shape("llama3.3-70b-bulk-decode", 8, 128, 64, 80, 131072, BF16, 1024, 1024, 16),
    5: Shape("llama3.1-8b-decode-attn", 8, 128, 32, 1, 32 * 32768, BF16, 1024, 1024, 16,
             batch=32),
    # second workload: Qwen-2.5-shaped caches (2 and 4 KV heads of 128: d_kv 256 / 512, group = d_kv, first
    # layer left in 16 bits), compressed for the 20 % of a 131072-token context that a pruning policy keeps
    6: Shape("qwen2.5-3b-kept-token-encode", 2, 128, 16, 36, 131072, BF16, 256, 256, 16),
    7: Shape("qwen2.5-7b-kept-token-encode", 4, 128, 28, 28, 131072, BF16, 512, 512, 16),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn(shape, g: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


# --------------------------------------------------------------------------------------------
# Grid and signs
# --------------------------------------------------------------------------------------------

def lloyd_grid(n: int, seed: int = 7, n_samples: int = 1 << 18, iters: int = 60, dim: int = 2) -> np.ndarray:
    """A dim-dimensional, n-point codebook fitted to N(0, I) samples by Lloyd's algorithm.

    Stands in for the fixed Gaussian-optimal grid of the paper's backbone quantizer (Section 4.1
    "Alternative quantizers": p = 2, n in {16, 64, 256}, and the slower p = 4, n = 256 grid).
    Deterministic for a given seed; rows are sorted lexicographically so that code indices are
    canonical.  Returned as float32 [n, dim] (the storage type of the library's grid argument).
    """
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n_samples, dim))
    c = x[rng.choice(n_samples, size=n, replace=False)].copy()
    for _ in range(iters):
        # squared distances up to the sample's own norm, by blocks of samples (memory)
        a = np.empty(n_samples, dtype=np.int64)
        for lo in range(0, n_samples, 1 << 16):
            blk = x[lo:lo + (1 << 16)]
            a[lo:lo + (1 << 16)] = ((c * c).sum(1)[None, :] - 2.0 * blk @ c.T).argmin(1) if dim > 2 else \
                ((blk[:, None, :] - c[None, :, :]) ** 2).sum(-1).argmin(1)
        for i in range(n):
            m = a == i
            if m.any():
                c[i] = x[m].mean(0)
    order = np.lexsort(tuple(c[:, k] for k in range(dim - 1, -1, -1)))
    return np.ascontiguousarray(c[order], dtype=np.float32)


def hadamard_signs(d_kv: int, seed: int) -> np.ndarray:
    """Random +-1 diagonal of the randomized Hadamard transform, int8 [d_kv]."""
    rng = np.random.default_rng(seed)
    return (rng.integers(0, 2, size=d_kv, dtype=np.int8) * 2 - 1).astype(np.int8)


# --------------------------------------------------------------------------------------------
# Adapters (linear predictors), stored [out_features, in_features] like a linear layer's weight
# --------------------------------------------------------------------------------------------

@dataclasses.dataclass
class Adapters:
    Wk: List[Optional[torch.Tensor]]   # per layer: [d, d]   (None for layer 0)
    Wv: List[Optional[torch.Tensor]]   # per layer: [d, 2d]  columns 0..d-1 act on V_prev, d..2d-1 on K_hat
    bk: List[Optional[torch.Tensor]]   # per layer: [d] fp32 or None
    bv: List[Optional[torch.Tensor]]


def random_adapters(shape: Shape, seed: int, device="cpu", bias: bool = False) -> Adapters:
    """Seeded random adapters with entries N(0, 1/d_kv) (random, not fitted)."""
    d = shape.d_kv
    dt = torch_dtype(shape.dtype)
    g = _gen(seed, device)
    Wk, Wv, bk, bv = [None], [None], [None], [None]
    for _ in range(1, shape.n_layers):
        Wk.append((_randn((d, d), g, device) / math.sqrt(d)).to(dt))
        Wv.append((_randn((d, 2 * d), g, device) / math.sqrt(d)).to(dt))
        if bias:
            bk.append(0.1 * _randn((d,), g, device))
            bv.append(0.1 * _randn((d,), g, device))
        else:
            bk.append(None)
            bv.append(None)
    return Adapters(Wk, Wv, bk, bv)


# --------------------------------------------------------------------------------------------
# Key/value chains with cross-layer structure
# --------------------------------------------------------------------------------------------

@dataclasses.dataclass
class KVChain:
    K: List[torch.Tensor]   # per layer [T, d] 16-bit
    V: List[torch.Tensor]


def kv_chain(shape: Shape, seed: int, device="cpu", token_chunk: int = 8192) -> KVChain:
    """Keys/values for all layers: K_0 ~ N(0,1); K_l = K_{l-1} A_l + 0.3 N(0,1) with
    A_l ~ N(0, 1/d); V_0 = (N(0,1) + K_0)/sqrt(2); V_l = [V_{l-1}; K_l] B_l + 0.7 N(0,1) with
    B_l ~ N(0, 1/(2d)).  With `channel_scales` every channel of every layer is multiplied by
    exp(N(0,1)) (heavy-tailed outlier channels).  Values are rounded once to the 16-bit type.
    The recurrence runs in fp32 on the unscaled, unrounded values, chunked over tokens.
    """
    d, T, L = shape.d_kv, shape.n_tokens, shape.n_layers
    dt = torch_dtype(shape.dtype)
    g = _gen(seed, device)
    A = [None] + [_randn((d, d), g, device) / math.sqrt(d) for _ in range(1, L)]
    B = [None] + [_randn((2 * d, d), g, device) / math.sqrt(2 * d) for _ in range(1, L)]
    if shape.channel_scales:
        sk = [torch.exp(_randn((d,), g, device)) for _ in range(L)]
        sv = [torch.exp(_randn((d,), g, device)) for _ in range(L)]
    else:
        sk = sv = None
    K = [torch.empty((T, d), dtype=dt, device=device) for _ in range(L)]
    V = [torch.empty((T, d), dtype=dt, device=device) for _ in range(L)]
    for t0 in range(0, T, token_chunk):
        t1 = min(T, t0 + token_chunk)
        n = t1 - t0
        k = _randn((n, d), g, device)
        v = (_randn((n, d), g, device) + k) / math.sqrt(2.0)
        for l in range(L):
            if l > 0:
                k = k @ A[l] + 0.3 * _randn((n, d), g, device)
                v = torch.cat([v, k], dim=1) @ B[l] + 0.7 * _randn((n, d), g, device)
            K[l][t0:t1] = (k * sk[l] if sk is not None else k).to(dt)
            V[l][t0:t1] = (v * sv[l] if sv is not None else v).to(dt)
    return KVChain(K, V)


# --------------------------------------------------------------------------------------------
# Random packed caches (bulk decode / decode-attention workloads)
# --------------------------------------------------------------------------------------------

@dataclasses.dataclass
class PackedCache:
    Kcodes: List[torch.Tensor]    # per layer uint8 [T, code_bytes]
    Kscales: List[torch.Tensor]   # per layer fp16 [T, n_groups]
    Vcodes: List[torch.Tensor]
    Vscales: List[torch.Tensor]


def random_cache(shape: Shape, seed: int, device="cpu", n_layers: Optional[int] = None) -> PackedCache:
    """Uniform random code bytes and fp16 scales 0.3 * exp(0.25 N(0,1))."""
    T, L = shape.n_tokens, (n_layers or shape.n_layers)
    g = _gen(seed, device)
    out = PackedCache([], [], [], [])
    for _ in range(L):
        for codes, scales in ((out.Kcodes, out.Kscales), (out.Vcodes, out.Vscales)):
            codes.append(torch.randint(0, 256, (T, shape.code_bytes), generator=g, device=device,
                                       dtype=torch.uint8))
            s = 0.3 * torch.exp(0.25 * _randn((T, shape.n_groups), g, device))
            scales.append(s.to(torch.float16))
    return out


def random_16bit(shape_, dtype: int, seed: int, device="cpu", std: float = 1.0) -> torch.Tensor:
    """N(0, std^2) rounded once to the 16-bit type (queries, previous-layer reconstructions)."""
    g = _gen(seed, device)
    return (std * _randn(tuple(shape_), g, device)).to(torch_dtype(dtype))


# --------------------------------------------------------------------------------------------
# Token sharding for multi-GPU runs (tokens are independent through all layers, so ranks take
# disjoint token ranges and exchange nothing)
# --------------------------------------------------------------------------------------------

def kept_tokens(n_tokens: int, fraction: float, seed: int) -> np.ndarray:
    """Sorted indices of the tokens a pruning policy keeps: a seeded random subset of round(fraction *
    n_tokens) tokens (stand-in for a heavy-hitter selection, which depends on attention scores the
    harness does not have)."""
    rng = np.random.default_rng(seed)
    n_keep = int(round(fraction * n_tokens))
    return np.sort(rng.choice(n_tokens, size=n_keep, replace=False)).astype(np.int64)


def shard_range(n: int, rank: int, world: int, multiple: int = 1):
    """Contiguous [begin, end) of rank's share of n items, every share but the last a multiple
    of `multiple`."""
    units = (n + multiple - 1) // multiple
    lo = (units * rank) // world * multiple
    hi = (units * (rank + 1)) // world * multiple
    return min(lo, n), min(hi, n)
