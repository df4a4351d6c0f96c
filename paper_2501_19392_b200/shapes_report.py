"""Times the library on all five workload shapes of `synth.CONFIGS` and prints one JSON line each.

    python -m paper_2501_19392_b200.shapes_report [--configs 1,3,4,5] [--layers-cap 8]

Each line gives the time per layer call (CUDA events, after warm-up, inputs resident in HBM and
larger than L2 for the big shapes), tokens/s per layer, and the fraction of that shape's roofline
max(6 d^2 T / tensor peak, algorithmic bytes / HBM bandwidth) with the peaks of MEASURED_PEAKS.json
at the repository root when present.  Shapes with many layers are timed on `--layers-cap` layers:
the metric is per layer and every layer after the first costs the same.  The default benchmark
(`bench.py`) covers shape 2 in full; this script is the measured record for the others.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
import os

import torch

from . import api, chain, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p["hbm_gbs"] * 1e9, p["bf16_tflops"] * 1e12, "measured (burst)"
    return 6650e9, 1590e12, "fallback"


def _bytes_per_token(shape: synth.Shape, tokens: int, encode: bool, write_hat: bool = True) -> float:
    d = shape.d_kv
    codes = 2 * shape.code_bytes + 2 * 2 * shape.n_groups
    weights = 6.0 * d * d / tokens
    by = codes + 4 * d + weights + (4 * d if write_hat else 0)   # codes, prev in, (hats out), weights
    if encode:
        by += 4 * d                                              # K, V in
    return by


def _time(fn, reps: int, warm: int = 3) -> float:
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps


def _line(shape, op, tokens, layers_timed, ms_per_layer, by_per_token, extra=None):
    hbm, tf, src = _peaks()
    d = shape.d_kv
    t_tensor = 6.0 * d * d / tf
    t_hbm = by_per_token / hbm
    t_roof = max(t_tensor, t_hbm)
    tps = tokens / (ms_per_layer * 1e-3)
    out = {"workload": shape.name, "op": op, "tokens": tokens, "layers_timed": layers_timed, "d_kv": d,
           "grid_points": shape.grid_size, "ms_per_layer": ms_per_layer, "token_layers_per_s": tps,
           "bound": "tensor" if t_tensor >= t_hbm else "hbm", "roofline_token_layers_per_s": 1.0 / t_roof,
           "frac_of_roofline": tps * t_roof, "peaks": src}
    if extra:
        out.update(extra)
    print(json.dumps(out), flush=True)


def _codec(shape, dev):
    grid = synth.lloyd_grid(shape.grid_size, seed=7, n_samples=1 << 14, iters=25)
    return api.Codec(shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype,
                     synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12))


def encode_shape(cfg: int, shape: synth.Shape, dev, cap: int, reps: int):
    """Encode chain (layer 0 without predictor, then predicted layers); time per predicted layer."""
    L = min(shape.n_layers, cap)
    shape = dataclasses.replace(shape, n_layers=L)
    T = shape.n_tokens
    codec = _codec(shape, dev)
    kv = synth.kv_chain(shape, seed=1000 * cfg + 1, device=dev)
    ad = synth.random_adapters(shape, seed=1000 * cfg + 2, device=dev)
    cache = chain.CompressedCache.empty(codec, L, T, dev)
    bufs = chain.PingPong(codec, T, dev)
    chain.encode_chain(codec, kv.K, kv.V, ad, cache, bufs)          # fills bufs for the timed layer
    ms_chain = _time(lambda: chain.encode_chain(codec, kv.K, kv.V, ad, cache, bufs), reps)
    l = L - 1
    prv, cur = (l + 1) % 2, l % 2
    one = lambda: codec.encode(kv.K[l], kv.V[l], bufs.K[prv], bufs.V[prv], ad.Wk[l], ad.Wv[l], None, None,
                               cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                               bufs.K[cur], bufs.V[cur])
    ms_one = _time(one, reps * 4)
    assert codec.poll_status() == 0
    _line(shape, "encode", T, L, ms_one, _bytes_per_token(shape, T, True),
          {"ms_chain": ms_chain, "chain_layers": L})
    return codec, cache, ad, bufs, shape


def decode_shape(cfg: int, shape: synth.Shape, dev, cap: int, reps: int, from_encode=None):
    """Decode chain over a random packed cache (or the cache an encode just wrote)."""
    if from_encode is None:
        L = min(shape.n_layers, cap)
        shape = dataclasses.replace(shape, n_layers=L)
        codec = _codec(shape, dev)
        rc = synth.random_cache(shape, seed=1000 * cfg + 3, device=dev)
        cache = chain.CompressedCache(rc.Kcodes, rc.Kscales, rc.Vcodes, rc.Vscales)
        ad = synth.random_adapters(shape, seed=1000 * cfg + 2, device=dev)
        bufs = chain.PingPong(codec, shape.n_tokens, dev)
    else:
        codec, cache, ad, bufs, shape = from_encode
        L = shape.n_layers
    T = shape.n_tokens
    chain.decode_chain(codec, cache, ad, bufs)
    ms_chain = _time(lambda: chain.decode_chain(codec, cache, ad, bufs), reps)
    l = L - 1
    prv, cur = (l + 1) % 2, l % 2
    one = lambda: codec.decode(cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                               bufs.K[prv], bufs.V[prv], ad.Wk[l], ad.Wv[l], None, None, bufs.K[cur], bufs.V[cur])
    ms_one = _time(one, reps * 4)
    assert codec.poll_status() == 0
    _line(shape, "decode", T, L, ms_one, _bytes_per_token(shape, T, False),
          {"ms_chain": ms_chain, "chain_layers": L})


def decode_attn_shape(cfg: int, shape: synth.Shape, dev, reps: int):
    """One fused decode + single-query attention layer call at the shape's batch and context."""
    shape = dataclasses.replace(shape, n_layers=2)       # a predicted layer: adapters of layer 1
    T, d = shape.n_tokens, shape.d_kv
    codec = _codec(shape, dev)
    rc = synth.random_cache(shape, seed=1000 * cfg + 3, device=dev, n_layers=1)
    ad = synth.random_adapters(shape, seed=1000 * cfg + 2, device=dev)
    Kp = synth.random_16bit((T, d), shape.dtype, 1000 * cfg + 4, device=dev)
    Vp = synth.random_16bit((T, d), shape.dtype, 1000 * cfg + 5, device=dev)
    q = synth.random_16bit((shape.batch, shape.n_q_heads, shape.head_dim), shape.dtype, 1000 * cfg + 6, device=dev)
    out = torch.empty_like(q)
    ctx = T // shape.batch
    scale = 1.0 / math.sqrt(shape.head_dim)
    one = lambda: codec.decode_attn(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx,
                                    shape.n_kv_heads, scale, Kp, Vp, ad.Wk[1], ad.Wv[1], None, None, out=out)
    ms = _time(one, reps)
    assert codec.poll_status() == 0
    _line(shape, "decode_attn", T, 1, ms, _bytes_per_token(shape, T, False, write_hat=False),
          {"batch": shape.batch, "ctx": ctx, "n_q_heads": shape.n_q_heads})


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--configs", default="1,2,3,4,5")
    ap.add_argument("--layers-cap", type=int, default=8)
    ap.add_argument("--reps", type=int, default=5)
    args = ap.parse_args()
    # importing `api` above already failed loudly if the CUDA library is not built
    dev = torch.device("cuda", 0)
    for cfg in [int(c) for c in args.configs.split(",")]:
        shape = synth.CONFIGS[cfg]
        if cfg in (1, 2):
            enc = encode_shape(cfg, shape, dev, args.layers_cap, args.reps)
            decode_shape(cfg, shape, dev, args.layers_cap, args.reps, from_encode=enc)
        elif cfg == 3:
            for n in (16, 64):
                encode_shape(cfg, dataclasses.replace(shape, grid_size=n), dev, shape.n_layers, args.reps)
        elif cfg == 4:
            decode_shape(cfg, shape, dev, args.layers_cap, args.reps)
        elif cfg == 5:
            decode_attn_shape(cfg, shape, dev, args.reps)
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
