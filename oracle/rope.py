"""CPU oracle of rotary position encoding applied to cached PRE-RoPE keys at attention time
(Section 3.3 "Positional embeddings": predictors and quantizers work on the keys before RoPE, so the
reconstructed keys are rotated when the block attends to them in Algorithm 4; RoPE is the
rotary embedding of Su et al. that the paper cites).

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain numpy in double precision.

Reading (the paper names RoPE, not its layout).  For a head of `head_dim` values and a token at
position pos, frequency i < head_dim/2 has the angle pos * theta_base^(-2 i / head_dim) and rotates
the PAIR (x[i], x[i + head_dim/2]) -- the half-split pairing of the Llama-family models the paper
evaluates -- by that angle:
    y[i]              = x[i] cos - x[i + head_dim/2] sin
    y[i + head_dim/2] = x[i + head_dim/2] cos + x[i] sin.
The rotated key is rounded ONCE to the cache's 16-bit type (it stands for the key tensor a model would
hand to its attention) and the attention of Algorithm 4 runs over the rotated rows.  The query comes
rotated by its own position already; values are not rotated.
"""
from __future__ import annotations

import numpy as np

from . import attention
from .calibration import bits_to_double, double_to_bits


def angles(positions: np.ndarray, head_dim: int, theta_base: float) -> np.ndarray:
    """[n, head_dim/2] angles pos * theta_base^(-2 i / head_dim) in double."""
    i = np.arange(head_dim // 2, dtype=np.float64)
    freq = np.power(float(theta_base), -2.0 * i / float(head_dim))
    return np.asarray(positions, dtype=np.float64)[:, None] * freq[None, :]


def rotate_rows(K: np.ndarray, positions: np.ndarray, n_kv_heads: int, head_dim: int, theta_base: float) -> np.ndarray:
    """Rows K [n, n_kv_heads*head_dim] (double) rotated head by head, row r by positions[r]."""
    n = K.shape[0]
    half = head_dim // 2
    a = angles(positions, head_dim, theta_base)
    cos, sin = np.cos(a)[:, None, :], np.sin(a)[:, None, :]
    X = np.asarray(K, dtype=np.float64).reshape(n, n_kv_heads, head_dim)
    lo, hi = X[:, :, :half], X[:, :, half:]
    Y = np.empty_like(X)
    Y[:, :, :half] = lo * cos - hi * sin
    Y[:, :, half:] = hi * cos + lo * sin
    return Y.reshape(n, n_kv_heads * head_dim)


def rotate_rows_16bit(K_bits: np.ndarray, positions: np.ndarray, n_kv_heads: int, head_dim: int,
                      theta_base: float, dtype: int):
    """16-bit rows in, (rotated rows rounded once to the 16-bit type, the unrounded doubles) out."""
    exact = rotate_rows(bits_to_double(K_bits, dtype), positions, n_kv_heads, head_dim, theta_base)
    return double_to_bits(exact, dtype), exact


def attention_rope(dtype: int, batch: int, ctx: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                   softmax_scale: float, q: np.ndarray, K_bits: np.ndarray, V_bits: np.ndarray,
                   positions: np.ndarray, theta_base: float):
    """The attention read of Algorithm 4 over pre-RoPE key rows [batch*ctx, d]: row r of every sequence sits at
    positions[r] ([ctx] entries, the same for every sequence)."""
    pos = np.tile(np.asarray(positions, dtype=np.int64), batch)
    K_rot, _ = rotate_rows_16bit(K_bits, pos, n_kv_heads, head_dim, theta_base, dtype)
    return attention(dtype, batch, ctx, n_q_heads, n_kv_heads, head_dim, softmax_scale, q, K_rot, V_bits)
