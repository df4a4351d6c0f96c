"""Cache policy around the codec (Section 3.3; Section 4.1 "Evaluation setup": the first four
tokens, the attention sinks, and a buffer of the 128 newest tokens are left uncompressed, and the first layer
gets 4 bits per value): the first `n_sink` tokens and the most recent tokens stay in
16 bits, older tokens are compressed in chunks of `chunk` tokens whenever the recent buffer holds
`recent + chunk` of them, and every query attends to [compressed | sinks | recent] in one call.

Host policy only: bookkeeping of which rows are where.  Compression is chain.encode_chain on the
flushed chunk (all layers, the chunk's own reconstructions feeding the next layer), row movement is
aquakv_gather_rows, attention is aquakv_decode_attn_buffered.  Sequences of a batch advance in lockstep
(the same number of tokens each); every sequence has its own cache arrays and is served by its own
calls.  Keys are cached as given; with a rotary table (`attend(..., rope_table=...)`, Section 3.3
"Positional embeddings": keys are compressed before RoPE) they are taken as pre-RoPE keys of tokens 0, 1, ...
and rotated by their positions when attended to (aquakv_decode_attn_rope): sinks at 0 .. n_sink-1, compressed
token t at n_sink + t, the recent rows after them.
"""
from __future__ import annotations

from typing import List, Optional

import torch

from . import api, chain


class BufferedKVCache:
    def __init__(self, codec: api.Codec, adapters, n_layers: int, batch: int, max_tokens: int, device,
                 n_sink: int = 4, recent: int = 128, chunk: int = 128, first_layer_codec: Optional[api.Codec] = None):
        """first_layer_codec: a codec with a finer grid for layer 0 (the paper's 4-bit first layer); layer 0 has
        no predictor, so only its code size differs."""
        self.codec, self.codec0 = codec, first_layer_codec or codec
        self.ad, self.L, self.B, self.dev = adapters, n_layers, batch, device
        self.n_sink, self.recent, self.chunk = n_sink, recent, chunk
        self.cap = recent + chunk                      # rows of the recent buffer
        self.max_ctx = max_tokens
        d, dt = codec.d, codec.torch_dtype
        mk = lambda *shape, dtype=dt: torch.zeros(shape, dtype=dtype, device=device)
        # uncompressed rows per layer and sequence: [sinks | recent buffer], valid rows are a prefix
        self.K16 = [mk(batch, n_sink + self.cap, d) for _ in range(n_layers)]
        self.V16 = [mk(batch, n_sink + self.cap, d) for _ in range(n_layers)]
        cb = lambda l: (self.codec0 if l == 0 else codec).code_bytes
        self.Kcodes = [mk(batch, max_tokens, cb(l), dtype=torch.uint8) for l in range(n_layers)]
        self.Vcodes = [mk(batch, max_tokens, cb(l), dtype=torch.uint8) for l in range(n_layers)]
        self.Kscales = [mk(batch, max_tokens, codec.n_groups, dtype=torch.float16) for _ in range(n_layers)]
        self.Vscales = [mk(batch, max_tokens, codec.n_groups, dtype=torch.float16) for _ in range(n_layers)]
        self.n_sinks_held = 0       # sink rows filled so far
        self.fill = 0               # valid rows of the recent buffer
        self.ctx = 0                # compressed tokens per sequence
        self._bufs = chain.PingPong(codec, chunk, device)
        self._dec = None            # ping-pong buffers of the attention pass, sized on demand

    # -- appending ------------------------------------------------------------------------------
    def append(self, K: List[torch.Tensor], V: List[torch.Tensor]) -> None:
        """K[l], V[l]: [batch, n_new, d_kv] 16-bit, the new tokens' keys / values of every layer."""
        n_new = K[0].shape[1]
        t = 0
        while t < n_new:
            if self.n_sinks_held < self.n_sink:
                n = min(self.n_sink - self.n_sinks_held, n_new - t)
                self._store(K, V, t, n, self.n_sinks_held)
                self.n_sinks_held += n
            else:
                n = min(self.cap - self.fill, n_new - t)
                self._store(K, V, t, n, self.n_sink + self.fill)
                self.fill += n
                if self.fill == self.cap:
                    self._flush()
            t += n

    def _store(self, K, V, t, n, row):
        for l in range(self.L):
            for b in range(self.B):
                self.codec.gather_rows(K[l][b, t:t + n], None, self.K16[l][b, row:row + n])
                self.codec.gather_rows(V[l][b, t:t + n], None, self.V16[l][b, row:row + n])

    def _flush(self):
        """Compresses the oldest `chunk` rows of the recent buffer (all layers) and closes the gap."""
        assert self.ctx + self.chunk <= self.max_ctx, "compressed cache is full"
        s0, c, r = self.n_sink, self.chunk, self.recent
        for b in range(self.B):
            Kc = [self.K16[l][b, s0:s0 + c] for l in range(self.L)]
            Vc = [self.V16[l][b, s0:s0 + c] for l in range(self.L)]
            sl = slice(self.ctx, self.ctx + c)
            view = chain.CompressedCache([x[b, sl] for x in self.Kcodes], [x[b, sl] for x in self.Kscales],
                                         [x[b, sl] for x in self.Vcodes], [x[b, sl] for x in self.Vscales])
            self._encode_chunk(Kc, Vc, view)
        # the remaining `recent` rows move to the front of the buffer (through the chunk-sized scratch rows:
        # source and destination may overlap when recent > chunk)
        tmpK, tmpV = self._bufs.K[0], self._bufs.V[0]
        for l in range(self.L):
            for b in range(self.B):
                for o in range(0, r, c):
                    n = min(c, r - o)
                    self.codec.gather_rows(self.K16[l][b, s0 + c + o:s0 + c + o + n], None, tmpK[:n])
                    self.codec.gather_rows(tmpK[:n], None, self.K16[l][b, s0 + o:s0 + o + n])
                    self.codec.gather_rows(self.V16[l][b, s0 + c + o:s0 + c + o + n], None, tmpV[:n])
                    self.codec.gather_rows(tmpV[:n], None, self.V16[l][b, s0 + o:s0 + o + n])
        self.fill -= c
        self.ctx += c

    def _encode_chunk(self, Kc, Vc, view):
        """Algorithm 2 over the layers for one chunk of one sequence; layer 0 through the first-layer codec."""
        bufs, ad = self._bufs, self.ad
        for l in range(self.L):
            cur, prv = l % 2, (l + 1) % 2
            if l == 0:
                self.codec0.encode(Kc[0], Vc[0], None, None, None, None, None, None, view.Kcodes[0], view.Kscales[0],
                                   view.Vcodes[0], view.Vscales[0], bufs.K[cur], bufs.V[cur])
            else:
                self.codec.encode(Kc[l], Vc[l], bufs.K[prv], bufs.V[prv], ad.Wk[l], ad.Wv[l], ad.bk[l], ad.bv[l],
                                  view.Kcodes[l], view.Kscales[l], view.Vcodes[l], view.Vscales[l], bufs.K[cur],
                                  bufs.V[cur])

    # -- attention ------------------------------------------------------------------------------
    @property
    def n_uncompressed(self) -> int:
        return self.n_sinks_held + self.fill

    def attend(self, q: List[torch.Tensor], n_kv_heads: int, softmax_scale: float,
               rope_table: Optional[torch.Tensor] = None) -> List[torch.Tensor]:
        """The decode-and-attend loop of Algorithm 4 for every layer: q[l] [batch, n_q_heads, head_dim] -> outputs of the same shape.
        The decoded compressed rows of layer l feed layer l + 1's predictors and are dropped afterwards.
        rope_table (Codec.rope_table): the cached keys are pre-RoPE and are rotated by their positions; q[l] must
        be rotated by the caller."""
        out = [torch.empty_like(x) for x in q]
        n16 = self.n_uncompressed
        pos16 = None
        if rope_table is not None and n16:
            first_recent = self.n_sinks_held + self.ctx
            pos16 = torch.cat([torch.arange(self.n_sinks_held, dtype=torch.int32, device=self.dev),
                               torch.arange(first_recent, first_recent + self.fill, dtype=torch.int32, device=self.dev)])
        if self.ctx > 0 and (self._dec is None or self._dec.K[0].shape[0] < self.ctx):
            self._dec = chain.PingPong(self.codec, self.max_ctx, self.dev)
        for b in range(self.B):
            for l in range(self.L):
                cur, prv = l % 2, (l + 1) % 2
                cdc = self.codec0 if l == 0 else self.codec
                has = l > 0 and self.ctx > 0
                kh = self._dec.K[cur][:self.ctx] if self.ctx > 0 else None
                vh = self._dec.V[cur][:self.ctx] if self.ctx > 0 else None
                cache = (q[l][b:b + 1], self.Kcodes[l][b, :self.ctx], self.Kscales[l][b, :self.ctx],
                         self.Vcodes[l][b, :self.ctx], self.Vscales[l][b, :self.ctx], self.ctx, n_kv_heads, softmax_scale)
                rows16 = (self.K16[l][b:b + 1, :n16] if n16 else None, self.V16[l][b:b + 1, :n16] if n16 else None)
                pred = (self._dec.K[prv][:self.ctx] if has else None, self._dec.V[prv][:self.ctx] if has else None,
                        self.ad.Wk[l] if has else None, self.ad.Wv[l] if has else None,
                        self.ad.bk[l] if has else None, self.ad.bv[l] if has else None)
                if rope_table is None:
                    cdc.decode_attn_buffered(*cache, *rows16, *pred, out=out[l][b:b + 1], Khat=kh, Vhat=vh)
                else:
                    cdc.decode_attn_rope(*cache, rope_table, self.n_sinks_held, *rows16, pos16, *pred,
                                         out=out[l][b:b + 1], Khat=kh, Vhat=vh)
        return out
