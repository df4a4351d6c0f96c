"""Layer-chain driver (Algorithm 4: layer i's reconstruction feeds layer i+1's predictors).

Host loops only: each layer is one call into the C library; the reconstructed keys/values live in
two ping-pong buffer pairs so that only the previous layer is ever materialised (Section 3.3:
one reconstructed layer at a time is enough).  Nothing is computed here.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional

import torch

from . import api


@dataclasses.dataclass
class CompressedCache:
    """Per-layer packed codes and fp16 scales for keys and values."""
    Kcodes: List[torch.Tensor]
    Kscales: List[torch.Tensor]
    Vcodes: List[torch.Tensor]
    Vscales: List[torch.Tensor]

    @staticmethod
    def empty(codec: api.Codec, n_layers: int, n_tokens: int, device) -> "CompressedCache":
        mk = lambda shape, dt: [torch.empty(shape, dtype=dt, device=device) for _ in range(n_layers)]
        return CompressedCache(mk((n_tokens, codec.code_bytes), torch.uint8),
                               mk((n_tokens, codec.n_groups), torch.float16),
                               mk((n_tokens, codec.code_bytes), torch.uint8),
                               mk((n_tokens, codec.n_groups), torch.float16))

    def nbytes(self) -> int:
        return sum(t.numel() * t.element_size() for lst in
                   (self.Kcodes, self.Kscales, self.Vcodes, self.Vscales) for t in lst)


class PingPong:
    """Two (K_hat, V_hat) buffer pairs [n_tokens, d_kv]; layer l writes pair l % 2."""

    def __init__(self, codec: api.Codec, n_tokens: int, device):
        mk = lambda: torch.empty((n_tokens, codec.d), dtype=codec.torch_dtype, device=device)
        self.K = [mk(), mk()]
        self.V = [mk(), mk()]


def encode_chain(codec: api.Codec, K: List[torch.Tensor], V: List[torch.Tensor], adapters,
                 cache: CompressedCache, bufs: PingPong) -> None:
    """Algorithm 2 for every layer in order; layer 0 has no predictor."""
    for l in range(len(K)):
        cur, prv = l % 2, (l + 1) % 2
        has = l > 0
        codec.encode(K[l], V[l],
                     bufs.K[prv] if has else None, bufs.V[prv] if has else None,
                     adapters.Wk[l] if has else None, adapters.Wv[l] if has else None,
                     adapters.bk[l] if has else None, adapters.bv[l] if has else None,
                     cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                     bufs.K[cur], bufs.V[cur])


def encode_layers(codec: api.Codec, K: List[torch.Tensor], V: List[torch.Tensor], adapters,
                  cache: CompressedCache, bufs: PingPong) -> None:
    """encode_chain through aquakv_encode_chain: for large token counts several layers per launch of the
    layer kernel (no pipeline fill and drain between layers), layer l writing buffer pair l % 2."""
    L = len(K)
    codec.encode_chain(K, V, adapters.Wk, adapters.Wv, cache.Kcodes, cache.Kscales, cache.Vcodes, cache.Vscales,
                       adapters.bk, adapters.bv, [bufs.K[l % 2] for l in range(L)], [bufs.V[l % 2] for l in range(L)])


def decode_layers(codec: api.Codec, cache: CompressedCache, adapters, bufs: PingPong,
                  n_layers: Optional[int] = None) -> int:
    """decode_chain through aquakv_decode_chain (see encode_layers); returns the buffer pair of the last layer."""
    L = n_layers or len(cache.Kcodes)
    codec.decode_chain(cache.Kcodes[:L], cache.Kscales[:L], cache.Vcodes[:L], cache.Vscales[:L], adapters.Wk[:L],
                       adapters.Wv[:L], adapters.bk[:L], adapters.bv[:L], [bufs.K[l % 2] for l in range(L)],
                       [bufs.V[l % 2] for l in range(L)])
    return (L - 1) % 2


def encode_chain_kept(codec: api.Codec, K: List[torch.Tensor], V: List[torch.Tensor], idx: torch.Tensor,
                      adapters, cache: CompressedCache, bufs: PingPong, stage_k: torch.Tensor,
                      stage_v: torch.Tensor, first_layer_16bit: bool = False) -> None:
    """Algorithm 2 over the tokens a pruning policy keeps (Section 4.3): each layer's kept rows are
    gathered into the compact staging tensors and encoded like any batch; cache and buffers hold
    len(idx) tokens.  first_layer_16bit leaves the first layer unquantised (the Qwen-2.5 setting of the
    appendix tables): its kept rows are carried into the buffers as they are and nothing is stored for it."""
    for l in range(len(K)):
        cur, prv = l % 2, (l + 1) % 2
        has = l > 0
        if l == 0 and first_layer_16bit:
            codec.gather_rows(K[0], idx, bufs.K[cur])
            codec.gather_rows(V[0], idx, bufs.V[cur])
            continue
        codec.gather_rows(K[l], idx, stage_k)
        codec.gather_rows(V[l], idx, stage_v)
        codec.encode(stage_k, stage_v,
                     bufs.K[prv] if has else None, bufs.V[prv] if has else None,
                     adapters.Wk[l] if has else None, adapters.Wv[l] if has else None,
                     adapters.bk[l] if has else None, adapters.bv[l] if has else None,
                     cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                     bufs.K[cur], bufs.V[cur])


def decode_chain(codec: api.Codec, cache: CompressedCache, adapters, bufs: PingPong,
                 n_layers: Optional[int] = None) -> int:
    """Algorithm 3 for every layer in order; returns the index of the buffer pair holding the last
    layer's reconstruction."""
    L = n_layers or len(cache.Kcodes)
    for l in range(L):
        cur, prv = l % 2, (l + 1) % 2
        has = l > 0
        codec.decode(cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                     bufs.K[prv] if has else None, bufs.V[prv] if has else None,
                     adapters.Wk[l] if has else None, adapters.Wv[l] if has else None,
                     adapters.bk[l] if has else None, adapters.bv[l] if has else None,
                     bufs.K[cur], bufs.V[cur])
    return (L - 1) % 2


def decode_attn_chain(codec: api.Codec, cache: CompressedCache, adapters, bufs: PingPong,
                      q: List[torch.Tensor], out: List[torch.Tensor], ctx_len: int, n_kv_heads: int,
                      softmax_scale: float) -> None:
    """The decode-and-attend loop of Algorithm 4 for every layer: decode the layer's cache (feeding the next layer's
    predictors through the ping-pong buffers) and attend to it with that layer's queries."""
    for l in range(len(q)):
        cur, prv = l % 2, (l + 1) % 2
        has = l > 0
        codec.decode_attn(q[l], cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                          ctx_len, n_kv_heads, softmax_scale,
                          bufs.K[prv] if has else None, bufs.V[prv] if has else None,
                          adapters.Wk[l] if has else None, adapters.Wv[l] if has else None,
                          adapters.bk[l] if has else None, adapters.bv[l] if has else None,
                          out=out[l], Khat=bufs.K[cur], Vhat=bufs.V[cur])
