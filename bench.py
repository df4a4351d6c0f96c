#!/usr/bin/env python
"""Benchmark of the AQUA-KV codec hot path on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input: the encode chain
(Algorithm 2 for every layer, each layer's predictors reading the previous layer's
reconstruction) followed by the decode + attention chain (Algorithm 3 and the attention read of
Algorithm 4 for every layer).  The workload is the Llama-3.2-3B-shaped prefill configuration:
28 layers x 32768 tokens, 8 KV heads x 128 (d_kv = 1024), bf16, 2 bits per value (16-point 2-D
grid, Hadamard block = scale group = 1024).

Metric: KV tokens/s per layer = tokens x layers carried through the step / step time.  The
headline `value` counts a token-layer once per round trip (encode + decode-attention); the per-op
rates (encode, decode-attention, plain decode) are under `ops`.

After the timed step the other four workload shapes are timed as well (one predicted-layer call
each, inputs resident in HBM) and reported under `ops_by_config` with their fraction of the roofline
max(6 d^2 T / tensor peak, algorithmic bytes / HBM bandwidth) against both the burst and the
sustained measured tensor peak.

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle on a bounded sample of the
same workload instead (the reference arm).
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2501_19392_b200 import synth  # noqa: E402

# dram__bytes_read.sum + dram__bytes_write.sum per layer_kernel launch (32768 tokens, d_kv 1024, n 16):
# mean of the encode (526 MB) and decode (258 MB) launches of profiles/layer_kernel_3layer_32768tok.md
LAYER_KERNEL_DRAM_BYTES_PER_LAUNCH = 392.0e6

METRIC = "KV tokens/s per layer (encode + decode-attention round trip) at 2 bits/value"
UNIT = "token-layers/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tf_burst=p["bf16_tflops"], tf_sustained=p["bf16_tflops_sustained"],
                    sm_max_mhz=p.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, tf_burst=1590.0, tf_sustained=1400.0, sm_max_mhz=1965.0, source="fallback")


def workload(args):
    base = synth.CONFIGS[2]
    shape = dataclasses.replace(base, n_tokens=args.tokens or base.n_tokens, n_layers=args.layers or base.n_layers)
    batch = 4 if shape.n_tokens % 4 == 0 and shape.n_tokens >= 4 * 256 else 1
    return shape, batch


def algorithmic_bytes(shape, n_rows_per_call):
    """Bytes the method itself must move per token-layer: inputs, outputs, codes, scales and the
    adapters once per call; re-reads and the fp32 prediction scratch are implementation traffic."""
    d, g = shape.d_kv, shape.scale_group
    codes = 2 * (d // 2 * shape.code_bits // 8) + 2 * 2 * (d // g)
    weights = 6 * d * d / n_rows_per_call
    enc = 4 * d + 4 * d + 4 * d + codes + weights          # K,V in; prev in; hats out; codes; weights
    dec = codes + 4 * d + 4 * d + weights                  # codes; prev in; hats out; weights
    return enc, dec


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                power.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                    power_w_max=float(max(power)), samples=len(sm))


# ------------------------------------------------------------------------------------------------
# CPU oracle arm (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------

def oracle_sample_run(shape, rows, layers, n_q_heads, seed):
    """One encode chain + decode chain + attention over `rows` tokens x `layers` layers on the CPU
    oracle.  Returns seconds."""
    import oracle
    small = dataclasses.replace(shape, n_tokens=rows, n_layers=layers)
    kv = synth.kv_chain(small, seed=seed)
    ad = synth.random_adapters(small, seed=seed + 1)
    grid = synth.lloyd_grid(shape.grid_size, seed=7, n_samples=1 << 14, iters=25)
    o = oracle.Oracle(shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype,
                      synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12))
    q = synth.to_bits(synth.random_16bit((1, n_q_heads, shape.head_dim), shape.dtype, seed + 2))
    Kb = [synth.to_bits(t) for t in kv.K]
    Vb = [synth.to_bits(t) for t in kv.V]
    Wk = [None] + [synth.to_bits(w) for w in ad.Wk[1:]]
    Wv = [None] + [synth.to_bits(w) for w in ad.Wv[1:]]
    t0 = time.perf_counter()
    pk = pv = None
    codes = []
    for l in range(layers):
        ek, ev = o.encode_layer(Kb[l], Vb[l], pk, pv, Wk[l], Wv[l])
        codes.append((ek["codes"], ek["scales"], ev["codes"], ev["scales"]))
        pk, pv = ek["hat"], ev["hat"]
    pk = pv = None
    for l in range(layers):
        dk, dv = o.decode_layer(*codes[l], pk, pv, Wk[l], Wv[l])
        pk, pv = dk["hat"], dv["hat"]
        oracle.attention(shape.dtype, 1, rows, n_q_heads, shape.n_kv_heads, shape.head_dim,
                         1.0 / math.sqrt(shape.head_dim), q, pk, pv)
    return time.perf_counter() - t0


def oracle_baseline(shape, n_q_heads, target_s=12.0):
    import oracle
    probe_rows, layers = 64, 2
    t = oracle_sample_run(shape, probe_rows, layers, n_q_heads, seed=2000)
    per_unit = t / (probe_rows * layers)
    rows = int(min(8192, max(64, target_s / (per_unit * 4))))
    rows = rows // 64 * 64
    layers = 4
    t = oracle_sample_run(shape, rows, layers, n_q_heads, seed=2001)
    cores = oracle.num_threads()
    # the same oracle on one thread, on a sample sized for a few seconds
    rows1 = max(64, int(rows / max(1, cores) / 2) // 64 * 64)
    oracle.set_num_threads(1)
    try:
        t1 = oracle_sample_run(shape, rows1, layers, n_q_heads, seed=2002)
    finally:
        oracle.set_num_threads(cores)
    return dict(value=rows * layers / t, unit=UNIT, cores=cores, kind="oracle",
                sample="%d tokens x %d layers of the workload (encode chain + decode chain + attention), %.1f s"
                       % (rows, layers, t),
                value_1thread=rows1 * layers / t1,
                sample_1thread="%d tokens x %d layers, %.1f s" % (rows1, layers, t1))


def run_reference(args):
    """Reference arm: the CPU oracle as it stands, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    shape, _ = workload(args)
    n_q = shape.n_q_heads
    rows, layers = 256, 4
    for _ in range(args.warmup):
        oracle_sample_run(shape, 64, 2, n_q, seed=2100)
    t0 = time.perf_counter()
    for s in range(args.steps):
        oracle_sample_run(shape, rows, layers, n_q, seed=2200 + s)
    dt = (time.perf_counter() - t0) / args.steps
    val = rows * layers / dt
    sample = "%d tokens x %d layers per step" % (rows, layers)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": shape.name, "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ------------------------------------------------------------------------------------------------
# The other workload shapes (one predicted-layer call each)
# ------------------------------------------------------------------------------------------------

def _time_calls(fn, reps, warm=3):
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


def _shape_bytes(shape, tokens, encode, write_hat=True):
    """Algorithmic bytes per token-layer of one predicted-layer call over `tokens` tokens."""
    d = shape.d_kv
    codes = 2 * shape.code_bytes + 2 * 2 * shape.n_groups
    by = codes + 4 * d + 6.0 * d * d / tokens + (4 * d if write_hat else 0)   # codes, prev in, weights, hats out
    return by + (4 * d if encode else 0)                                          # K, V in


def _shape_entry(peaks, shape, op, tokens, ms, by_per_token, **extra):
    d = shape.d_kv
    t_hbm = by_per_token / (peaks["hbm_gbs"] * 1e9)
    tps = tokens / (ms * 1e-3)
    out = {"workload": shape.name, "op": op, "tokens_per_call": tokens, "d_kv": d, "grid_points": shape.grid_size,
           "ms_per_layer_call": ms, "token_layers_per_s": tps}
    for key, tf in (("burst", peaks["tf_burst"]), ("sustained", peaks["tf_sustained"])):
        t_tensor = 6.0 * d * d / (tf * 1e12)
        t_roof = max(t_tensor, t_hbm)
        out["frac_of_roofline_" + key] = tps * t_roof
        if key == "burst":
            out["bound"] = "tensor" if t_tensor >= t_hbm else "hbm"
            out["roofline_token_layers_per_s"] = 1.0 / t_roof
    out.update(extra)
    return out


def _shape_codec(api, shape):
    grid = synth.lloyd_grid(shape.grid_size, seed=7, n_samples=1 << 14, iters=25)
    return api.Codec(shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype,
                     synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12))


def ops_by_config(api, chain, peaks, dev, reps=5):
    """Times configs 1, 3, 4 and 5 (config 2 is the timed step itself): per predicted-layer call, with
    the previous layer's reconstruction already in the ping-pong buffers."""
    out = []

    def encode_case(cfg, shape, layers, want_decode):
        shape = dataclasses.replace(shape, n_layers=layers)
        T = shape.n_tokens
        codec = _shape_codec(api, shape)
        kv = synth.kv_chain(shape, seed=1000 * cfg + 1, device=dev)
        ad = synth.random_adapters(shape, seed=1000 * cfg + 2, device=dev)
        cache = chain.CompressedCache.empty(codec, layers, T, dev)
        bufs = chain.PingPong(codec, T, dev)
        chain.encode_chain(codec, kv.K, kv.V, ad, cache, bufs)
        ms_chain = _time_calls(lambda: chain.encode_chain(codec, kv.K, kv.V, ad, cache, bufs), reps)
        l = layers - 1
        prv, cur = (l + 1) % 2, l % 2
        one = lambda: codec.encode(kv.K[l], kv.V[l], bufs.K[prv], bufs.V[prv], ad.Wk[l], ad.Wv[l], None, None,
                                   cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                                   bufs.K[cur], bufs.V[cur])
        ms = _time_calls(one, reps * 4)
        out.append(_shape_entry(peaks, shape, "encode", T, ms, _shape_bytes(shape, T, True),
                                config=cfg, ms_chain=ms_chain, chain_layers=layers))
        if want_decode:
            chain.decode_chain(codec, cache, ad, bufs)
            one = lambda: codec.decode(cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                                       bufs.K[prv], bufs.V[prv], ad.Wk[l], ad.Wv[l], None, None,
                                       bufs.K[cur], bufs.V[cur])
            ms = _time_calls(one, reps * 4)
            out.append(_shape_entry(peaks, shape, "decode", T, ms, _shape_bytes(shape, T, False), config=cfg))
        # the same layers through the chain entry points (all layers in one launch)
        mk = lambda cols, dt: [torch.empty((T, cols), dtype=dt, device=dev) for _ in range(layers)]
        Kc, Ks = mk(codec.code_bytes, torch.uint8), mk(codec.n_groups, torch.float16)
        Vc, Vs = mk(codec.code_bytes, torch.uint8), mk(codec.n_groups, torch.float16)
        Kh, Vh = mk(shape.d_kv, codec.torch_dtype), mk(shape.d_kv, codec.torch_dtype)
        ms = _time_calls(lambda: codec.encode_chain(kv.K, kv.V, ad.Wk, ad.Wv, Kc, Ks, Vc, Vs), reps * 4)
        out.append(_shape_entry(peaks, shape, "encode_chain", T, ms / layers, _shape_bytes(shape, T, True),
                                config=cfg, ms_chain=ms, chain_layers=layers,
                                note="aquakv_encode_chain: all layers in one launch; per layer = launch time / layers"))
        if want_decode:
            ms = _time_calls(lambda: codec.decode_chain(Kc, Ks, Vc, Vs, ad.Wk, ad.Wv, Khat=Kh, Vhat=Vh), reps * 4)
            out.append(_shape_entry(peaks, shape, "decode_chain", T, ms / layers, _shape_bytes(shape, T, False),
                                    config=cfg, ms_chain=ms, chain_layers=layers,
                                    note="aquakv_decode_chain: all layers in one launch; per layer = launch time / layers"))
        assert codec.poll_status() == 0

    # config 1: two layers, encode + decode round trip
    encode_case(1, synth.CONFIGS[1], 2, True)
    # config 3: decode-step encode, 2 and 3 bits per value
    for n in (16, 64):
        encode_case(3, dataclasses.replace(synth.CONFIGS[3], grid_size=n), synth.CONFIGS[3].n_layers, False)
    torch.cuda.empty_cache()
    # config 4: bulk decode over a random packed cache, 8 of its 80 layers (every layer after the
    # first costs the same; the metric is per layer)
    shape = dataclasses.replace(synth.CONFIGS[4], n_layers=8)
    codec = _shape_codec(api, shape)
    rc = synth.random_cache(shape, seed=4003, device=dev)
    cache = chain.CompressedCache(rc.Kcodes, rc.Kscales, rc.Vcodes, rc.Vscales)
    ad = synth.random_adapters(shape, seed=4002, device=dev)
    bufs = chain.PingPong(codec, shape.n_tokens, dev)
    chain.decode_chain(codec, cache, ad, bufs)
    ms_chain = _time_calls(lambda: chain.decode_chain(codec, cache, ad, bufs), max(2, reps // 2))
    ms = (ms_chain - _time_calls(lambda: chain.decode_chain(codec, cache, ad, bufs, n_layers=1), reps)) / 7
    out.append(_shape_entry(peaks, shape, "decode", shape.n_tokens, ms, _shape_bytes(shape, shape.n_tokens, False),
                            config=4, ms_chain=ms_chain, chain_layers=8, layers_of_the_full_shape=80))
    assert codec.poll_status() == 0
    del cache, rc, bufs
    torch.cuda.empty_cache()
    # config 5: decode + single-query attention, batch 32 x context 32768, one layer call
    shape = dataclasses.replace(synth.CONFIGS[5], n_layers=2)
    T, d = shape.n_tokens, shape.d_kv
    codec = _shape_codec(api, shape)
    rc = synth.random_cache(shape, seed=5003, device=dev, n_layers=1)
    ad = synth.random_adapters(shape, seed=5002, device=dev)
    Kp = synth.random_16bit((T, d), shape.dtype, 5004, device=dev)
    Vp = synth.random_16bit((T, d), shape.dtype, 5005, device=dev)
    q = synth.random_16bit((shape.batch, shape.n_q_heads, shape.head_dim), shape.dtype, 5006, device=dev)
    o = torch.empty_like(q)
    ctx_len = T // shape.batch
    one = lambda: codec.decode_attn(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx_len,
                                    shape.n_kv_heads, 1.0 / math.sqrt(shape.head_dim), Kp, Vp, ad.Wk[1], ad.Wv[1],
                                    None, None, out=o)
    ms = _time_calls(one, max(2, reps // 2), warm=2)
    out.append(_shape_entry(peaks, shape, "decode_attn", T, ms, _shape_bytes(shape, T, False, write_hat=False),
                            config=5, batch=shape.batch, ctx=ctx_len, n_q_heads=shape.n_q_heads))
    # the fused form: attention warps inside the decode kernel, decoded rows only in a ring in L2
    codec.set_attn_mode(api.ATTN_FUSED)
    ms_f = _time_calls(one, max(2, reps // 2), warm=2)
    codec.set_attn_mode(api.ATTN_SPLIT)
    out.append(_shape_entry(peaks, shape, "decode_attn_fused", T, ms_f, _shape_bytes(shape, T, False, write_hat=False),
                            config=5, batch=shape.batch, ctx=ctx_len, n_q_heads=shape.n_q_heads,
                            note="aquakv_set_attn_mode(AQUAKV_ATTN_FUSED): one launch of the layer kernel with attention "
                                 "warps + the merge kernel; the default form is decode kernel, split-KV attention, merge"))
    # the same with the cache policy's uncompressed rows beside the compressed cache: 4 attention sinks and 128
    # recent tokens per sequence (Section 4.1), merged in the same combine kernel
    n16 = 132
    K16 = synth.random_16bit((shape.batch, n16, d), shape.dtype, 5007, device=dev)
    V16 = synth.random_16bit((shape.batch, n16, d), shape.dtype, 5008, device=dev)
    buf = lambda: codec.decode_attn_buffered(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx_len,
                                             shape.n_kv_heads, 1.0 / math.sqrt(shape.head_dim), K16, V16, Kp, Vp,
                                             ad.Wk[1], ad.Wv[1], None, None, out=o)
    ms_b = _time_calls(buf, max(2, reps // 2), warm=2)
    out.append(_shape_entry(peaks, shape, "decode_attn_buffered", T, ms_b,
                            _shape_bytes(shape, T, False, write_hat=False), config=5, batch=shape.batch, ctx=ctx_len,
                            n_q_heads=shape.n_q_heads, uncompressed_rows_per_sequence=n16,
                            note="compressed cache + 4 sink and 128 recent tokens per sequence in 16 bits"))
    # and with the cached keys taken as pre-RoPE keys, rotated on the fly (Section 3.3): sinks at positions 0 .. 3,
    # compressed tokens from 4, recent rows after them; decode, rotation and attention are separate kernels here
    table = codec.rope_table(shape.head_dim, 500000.0, 4 + ctx_len + 128, dev)
    pos16 = torch.cat([torch.arange(4, dtype=torch.int32), torch.arange(4 + ctx_len, 4 + ctx_len + 128, dtype=torch.int32)]).to(dev)
    rot = lambda: codec.decode_attn_rope(q, rc.Kcodes[0], rc.Kscales[0], rc.Vcodes[0], rc.Vscales[0], ctx_len,
                                         shape.n_kv_heads, 1.0 / math.sqrt(shape.head_dim), table, 4, K16, V16, pos16,
                                         Kp, Vp, ad.Wk[1], ad.Wv[1], None, None, out=o)
    ms_r = _time_calls(rot, max(2, reps // 2), warm=2)
    out.append(_shape_entry(peaks, shape, "decode_attn_rope", T, ms_r,
                            _shape_bytes(shape, T, False, write_hat=False), config=5, batch=shape.batch, ctx=ctx_len,
                            n_q_heads=shape.n_q_heads, uncompressed_rows_per_sequence=n16,
                            note="as decode_attn_buffered with rotary position encoding applied to the decoded keys; "
                                 "three kernels per chunk (layer kernel, rotation, split-KV attention)"))
    assert codec.poll_status() == 0
    del rc, Kp, Vp, table
    torch.cuda.empty_cache()

    # configs 6 / 7 (second workload): Qwen-2.5-shaped caches, only the 20 % of a 131072-token context that a
    # pruning policy keeps are compressed, first layer left in 16 bits; time of one predicted layer
    # (gather of the kept keys and values + encode of the compact rows)
    for cfg in (6, 7):
        shape = dataclasses.replace(synth.CONFIGS[cfg], n_layers=3)
        codec = _shape_codec(api, shape)
        kv = synth.kv_chain(shape, seed=1000 * cfg + 1, device=dev)
        ad = synth.random_adapters(shape, seed=1000 * cfg + 2, device=dev)
        idx = torch.from_numpy(synth.kept_tokens(shape.n_tokens, 0.2, seed=1000 * cfg + 3)).to(dev)
        n_keep = int(idx.shape[0])
        cache = chain.CompressedCache.empty(codec, shape.n_layers, n_keep, dev)
        bufs = chain.PingPong(codec, n_keep, dev)
        sk, sv = torch.empty_like(bufs.K[0]), torch.empty_like(bufs.V[0])
        run = lambda: chain.encode_chain_kept(codec, kv.K, kv.V, idx, ad, cache, bufs, sk, sv, first_layer_16bit=True)
        run()
        ms_chain = _time_calls(run, reps)
        first = lambda: (codec.gather_rows(kv.K[0], idx, bufs.K[0]), codec.gather_rows(kv.V[0], idx, bufs.V[0]))
        ms = (ms_chain - _time_calls(first, reps)) / (shape.n_layers - 1)
        out.append(_shape_entry(peaks, shape, "encode_kept_tokens", n_keep, ms, _shape_bytes(shape, n_keep, True),
                                config=cfg, context_tokens=shape.n_tokens, kept_fraction=0.2, ms_chain=ms_chain,
                                chain_layers=shape.n_layers,
                                note="per predicted layer: gather of the kept K and V rows + encode; first layer in 16 bits"))
        assert codec.poll_status() == 0
        del kv, cache, bufs, sk, sv
        torch.cuda.empty_cache()
    return out


def calibration_entry(api, peaks, dev, reps=3):
    """Algorithm 1 on the prefill-shaped workload: three layers of 32768 calibration tokens (two fitted
    layers), d_kv 1024, 2 bits.  Time per fitted layer (key fit, key reconstruction, value fit, value
    reconstruction), against the time the normal equations need on the tensor cores plus the time the
    solve needs on the fp64 units; and what the fitted predictors buy: relative reconstruction error
    of the last layer with fitted predictors, with the seeded random adapters, and without predictors
    at 2 and at 3 bits per value."""
    from paper_2501_19392_b200 import calibrate as gcal
    shape = dataclasses.replace(synth.CONFIGS[2], n_layers=3)
    T, d, L = shape.n_tokens, shape.d_kv, shape.n_layers
    codec = _shape_codec(api, shape)
    kv = synth.kv_chain(shape, seed=6001, device=dev)
    run = lambda: gcal.calibrate(codec, kv.K, kv.V, rate=1e-3, keep_reconstructions=True)
    preds, recs = run()
    ms_all = _time_calls(run, reps, warm=1)
    ms_layer0 = _time_calls(lambda: (codec.encode_phase(api.ROLE_KEY, kv.K[0]), codec.encode_phase(api.ROLE_VALUE, kv.V[0])),
                            reps, warm=1)
    ms_layer = (ms_all - ms_layer0) / (L - 1)
    ms_fit_k = _time_calls(lambda: codec.fit_predictor(kv.K[1], recs[0][0], None, 1e-3), reps, warm=1)
    ms_fit_v = _time_calls(lambda: codec.fit_predictor(kv.V[1], recs[0][1], recs[1][0], 1e-3), reps, warm=1)
    assert codec.poll_status() == 0
    gram_flops = 2.0 * T * (d * (d + d) + 2 * d * (2 * d + d))            # X^T X and X^T Y of both fits
    solve_flops = sum(n ** 3 / 3.0 + 2.0 * n * n * d for n in (d, 2 * d)) * 2.0   # Cholesky + two triangular solves, multiply-adds x 2
    fp64_peak = 148 * 64 * 2 * 1.965e9                                      # 64 fp64 FMA lanes per SM at the maximum clock
    t_roof_ms = (gram_flops / (peaks["tf_burst"] * 1e12) + solve_flops / fp64_peak) * 1e3

    def rel_err(X, Xh):
        X, Xh = X.float(), Xh.float()
        return float(((X - Xh) ** 2).sum() / ((X - X.mean(dim=0)) ** 2).sum())

    last = L - 1
    quality = {"fitted_2bit": {"K": rel_err(kv.K[last], recs[last][0]), "V": rel_err(kv.V[last], recs[last][1])}}
    # the same chain with the seeded random adapters of the throughput runs
    ad = synth.random_adapters(shape, seed=6002, device=dev)
    _, _, Kh = codec.encode_phase(api.ROLE_KEY, kv.K[0])
    _, _, Vh = codec.encode_phase(api.ROLE_VALUE, kv.V[0])
    for l in range(1, L):
        _, _, Kn = codec.encode_phase(api.ROLE_KEY, kv.K[l], Kh, None, ad.Wk[l])
        _, _, Vh = codec.encode_phase(api.ROLE_VALUE, kv.V[l], Vh, Kn, ad.Wv[l])
        Kh = Kn
    quality["random_adapters_2bit"] = {"K": rel_err(kv.K[last], Kh), "V": rel_err(kv.V[last], Vh)}
    for n, name in ((16, "no_predictor_2bit"), (64, "no_predictor_3bit")):
        c = _shape_codec(api, dataclasses.replace(shape, grid_size=n))
        _, _, Kd = c.encode_phase(api.ROLE_KEY, kv.K[last])
        _, _, Vd = c.encode_phase(api.ROLE_VALUE, kv.V[last])
        quality[name] = {"K": rel_err(kv.K[last], Kd), "V": rel_err(kv.V[last], Vd)}
    torch.cuda.empty_cache()
    return {"config": "calibration", "workload": shape.name + " (3 layers of calibration tokens)", "op": "calibrate",
            "tokens_per_call": T, "d_kv": d, "grid_points": shape.grid_size, "regularizer_rate": 1e-3,
            "ms_per_fitted_layer": ms_layer, "ms_fit_key_predictor": ms_fit_k, "ms_fit_value_predictor": ms_fit_v,
            "token_layers_per_s": T / (ms_layer * 1e-3), "gram_tflop_per_layer": gram_flops / 1e12,
            "solve_fp64_gflop_per_layer": solve_flops / 1e9, "roofline_ms_per_layer": t_roof_ms,
            "frac_of_roofline_burst": t_roof_ms / (ms_fit_k + ms_fit_v), "bound": "tensor + fp64 alu",
            "fp64_peak_tflops": fp64_peak / 1e12,
            "note": "roofline = normal equations at the tensor peak + solve at 148 SMs x 64 fp64 lanes x 2 x 1.965 GHz; "
                    "fraction taken over the two fits (the reconstructions between them are encode calls)",
            "relative_error_last_layer": quality}


def uniform_backbone_entries(api, chain, peaks, dev, reps=5):
    """The alternative backbones, 2 bits per value, on the prefill-shaped workload: uniform round-to-nearest
    levels with absmax normalisation, plain with groups of 64 (2.25 bits with the scales) and rotated with one
    group per row (random signs + Hadamard rotation first; 2.02 bits), and the vector quantizer with the
    256-point grid in four dimensions (2.02 bits; the grid for which the paper had no fast GPU kernel).  Time of
    one predicted layer through the per-layer entry points (two launches per phase: predictor GEMM, row
    kernel), and what fitted predictors buy each backbone (Section 4.1 evaluates each backbone with and
    without them)."""
    from paper_2501_19392_b200 import calibrate as gcal

    def rel_err(X, Xh):
        X, Xh = X.float(), Xh.float()
        return float(((X - Xh) ** 2).sum() / ((X - X.mean(dim=0)) ** 2).sum())

    out = []
    for tag, h, g in (("uniform-backbone", 1, 64), ("rotated-uniform-backbone", 1024, 1024),
                      ("four-dimensional-grid-backbone", 1024, 1024)):
        shape = dataclasses.replace(synth.CONFIGS[2], n_layers=3, had_block=h, scale_group=g, grid_size=4)
        T, d, L = shape.n_tokens, shape.d_kv, shape.n_layers
        signs = (synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2)) if h > 1 else (None, None)
        grid4 = tag.startswith("four")     # the 256-point grid in four dimensions (2 bits per value, exhaustive search)
        if grid4:
            codec = api.Codec(d, h, g, synth.lloyd_grid(256, seed=9, n_samples=1 << 16, iters=20, dim=4), shape.dtype,
                              signs[0], signs[1])
        else:
            codec = api.Codec(d, h, g, None, shape.dtype, levels=4, signs_k=signs[0], signs_v=signs[1])
        kv = synth.kv_chain(shape, seed=7001, device=dev)
        preds, recs = gcal.calibrate(codec, kv.K, kv.V, rate=1e-3, keep_reconstructions=True)
        l = L - 1
        mk = lambda cols, dt: torch.empty((T, cols), dtype=dt, device=dev)
        Kc, Ks, Vc, Vs = mk(codec.code_bytes, torch.uint8), mk(codec.n_groups, torch.float16), \
            mk(codec.code_bytes, torch.uint8), mk(codec.n_groups, torch.float16)
        Kh, Vh = mk(d, codec.torch_dtype), mk(d, codec.torch_dtype)
        enc = lambda: codec.encode(kv.K[l], kv.V[l], recs[l - 1][0], recs[l - 1][1], preds.Wk[l], preds.Wv[l], None,
                                   None, Kc, Ks, Vc, Vs, Kh, Vh)
        ms_enc = _time_calls(enc, reps)
        dec = lambda: codec.decode(Kc, Ks, Vc, Vs, recs[l - 1][0], recs[l - 1][1], preds.Wk[l], preds.Wv[l], None,
                                   None, Kh, Vh)
        ms_dec = _time_calls(dec, reps)
        assert codec.poll_status() == 0
        _, _, Kd = codec.encode_phase(api.ROLE_KEY, kv.K[l])
        _, _, Vd = codec.encode_phase(api.ROLE_VALUE, kv.V[l])
        quality = {"fitted_predictors": {"K": rel_err(kv.K[l], recs[l][0]), "V": rel_err(kv.V[l], recs[l][1])},
                   "no_predictor": {"K": rel_err(kv.K[l], Kd), "V": rel_err(kv.V[l], Vd)}}
        if h > 1 and not grid4:      # the same group size without the rotation (the appendix' row with the larger group)
            plain = api.Codec(d, 1, g, None, shape.dtype, levels=4)
            _, _, Kp = plain.encode_phase(api.ROLE_KEY, kv.K[l])
            _, _, Vp = plain.encode_phase(api.ROLE_VALUE, kv.V[l])
            quality["no_predictor_no_rotation_same_group"] = {"K": rel_err(kv.K[l], Kp), "V": rel_err(kv.V[l], Vp)}
            assert plain.poll_status() == 0
            plain.close()
        code_bytes = 2 * codec.code_bytes + 2 * 2 * codec.n_groups
        by_enc = 4 * d * 2 + 4 * d + code_bytes + 6.0 * d * d * 2 / T       # K,V in; prev in; K^,V^ out; codes; adapters
        by_dec = 4 * d + 4 * d + code_bytes + 6.0 * d * d * 2 / T
        for op, ms, by in (("encode_" + tag.replace("-", "_"), ms_enc, by_enc),
                           ("decode_" + tag.replace("-", "_"), ms_dec, by_dec)):
            out.append(_shape_entry(peaks, shape, op, T, ms, by, config=tag, bits_per_value=2.0 + 16.0 / g,
                                    scale_group=g, had_block=h, relative_error_last_layer=quality,
                                    note="per predicted layer; two launches per phase (tcgen05 predictor GEMM, row kernel)"))
        del kv, recs, preds, Kd, Vd
        codec.close()
        torch.cuda.empty_cache()
    return out


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--tokens", type=int, default=0, help="override tokens per GPU (testing only)")
    ap.add_argument("--layers", type=int, default=0, help="override layer count (testing only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the per-call timing of configs 1, 3, 4, 5")
    ap.add_argument("--only-calibration", action="store_true",
                    help="run only the calibration entry of ops_by_config and print it (profiling aid)")
    ap.add_argument("--only-uniform-backbone", action="store_true",
                    help="run only the uniform-backbone entries of ops_by_config and print them (profiling aid)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    from paper_2501_19392_b200 import api, chain    # raises if the CUDA library is missing

    peaks = load_peaks()
    if args.only_calibration:
        if rank == 0:
            print(json.dumps(calibration_entry(api, peaks, dev, reps=1)))
        return
    if args.only_uniform_backbone:
        if rank == 0:
            print(json.dumps(uniform_backbone_entries(api, chain, peaks, dev, reps=2)))
        return
    shape, batch = workload(args)
    T, L, d = shape.n_tokens, shape.n_layers, shape.d_kv
    ctx_len = T // batch
    n_q = shape.n_q_heads
    scale = 1.0 / math.sqrt(shape.head_dim)

    # ---- synthetic inputs, resident in HBM (each rank draws its own tokens: weak scaling) ----------
    seed = 2000 + 17 * rank
    kv = synth.kv_chain(shape, seed=seed, device=dev)
    ad = synth.random_adapters(shape, seed=2500, device=dev)
    grid = synth.lloyd_grid(shape.grid_size, seed=7, n_samples=1 << 14, iters=25)
    codec = api.Codec(d, shape.had_block, shape.scale_group, grid, shape.dtype,
                      synth.hadamard_signs(d, 11), synth.hadamard_signs(d, 12))
    cache = chain.CompressedCache.empty(codec, L, T, dev)
    bufs = chain.PingPong(codec, T, dev)
    q = [synth.random_16bit((batch, n_q, shape.head_dim), shape.dtype, 2600 + l, device=dev) for l in range(L)]
    out = [torch.empty_like(q[0]) for _ in range(L)]

    def step(ev_mid=None):
        chain.encode_chain(codec, kv.K, kv.V, ad, cache, bufs)
        if ev_mid is not None:
            ev_mid.record()
        chain.decode_attn_chain(codec, cache, ad, bufs, q, out, ctx_len, shape.n_kv_heads, scale)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert codec.poll_status() == 0, "device status word reports a timed-out wait"

    # ---- timed region --------------------------------------------------------------------------
    sampler = ClockSampler(local)
    codec.profile_enable(True)
    launches0 = codec.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    mids = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True),
             torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    barrier()
    sampler.start()
    ev0.record()
    for s in range(args.steps):
        mids[s][0].record()
        step(mids[s][1])
        mids[s][2].record()
    ev1.record()
    barrier()
    clocks = sampler.stop()
    ms_total = ev0.elapsed_time(ev1)
    launches = codec.launch_count() - launches0
    enc_ms = sum(a.elapsed_time(b) for a, b, _ in mids) / args.steps
    dec_ms = sum(b.elapsed_time(c) for _, b, c in mids) / args.steps
    prof = {name: codec.profile_read(k) for name, k in
            (("layer_fused", api.KERNEL_LAYER), ("chain", api.KERNEL_CHAIN), ("predict_gemm", api.KERNEL_PREDICT),
             ("encode_rows", api.KERNEL_ENCODE_ROWS), ("decode_rows", api.KERNEL_DECODE_ROWS),
             ("attention", api.KERNEL_ATTN))}
    codec.profile_enable(False)
    assert codec.poll_status() == 0

    ms_step = ms_total / args.steps
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms_step], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_step = float(t.item())
    value = world * T * L / (ms_step * 1e-3)

    # ---- plain decode chain (Algorithm 3 alone), reported beside the step ----------------------------
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    chain.decode_chain(codec, cache, ad, bufs)
    torch.cuda.synchronize()
    e0.record()
    chain.decode_chain(codec, cache, ad, bufs)
    e1.record()
    torch.cuda.synchronize()
    plain_dec_ms = e0.elapsed_time(e1)

    # ---- rooflines --------------------------------------------------------------------------------
    rows_per_call = min(T, 2 * 148 * 128 * 256 // d)
    enc_bytes, dec_bytes = algorithmic_bytes(shape, T)
    flops_tl = 6.0 * d * d * (L - 1) / L                    # layer 0 has no predictor
    t_tensor = flops_tl / (peaks["tf_burst"] * 1e12)
    roof = {}
    t_tensor_sus = flops_tl / (peaks["tf_sustained"] * 1e12)
    for name, ms, by in (("encode", enc_ms, enc_bytes), ("decode_attn", dec_ms, dec_bytes),
                         ("decode", plain_dec_ms, dec_bytes)):
        t_hbm = by / (peaks["hbm_gbs"] * 1e9)
        t_roof = max(t_tensor, t_hbm)
        tps = T * L / (ms * 1e-3)
        roof[name] = {"token_layers_per_s": tps, "ms": ms, "roofline_token_layers_per_s": 1.0 / t_roof,
                      "frac_of_roofline": tps * t_roof, "frac_of_roofline_sustained": tps * max(t_tensor_sus, t_hbm),
                      "bound": "tensor" if t_tensor >= t_hbm else "hbm",
                      "achieved_tflops": tps * flops_tl / 1e12, "achieved_gbs": tps * by / 1e9}

    gemm_flops_total = args.steps * 2 * (L - 1) * 6.0 * d * d * T      # encode + decode-attn chains
    kernels = {}
    for name, (n, ms) in prof.items():
        kernels[name] = {"launches": n, "total_ms": ms, "share": ms / max(1e-9, sum(v[1] for v in prof.values()))}
    # Dominant kernel by time share: the fused layer kernel (predictor GEMMs on the tensor cores with
    # the quantizer's row work overlapped on the same SMs).  By the benchmark's roofline definition
    # (adapter FLOPs at tensor peak vs algorithmic bytes at HBM bandwidth) it is tensor-bound, so it
    # is reported as achieved predictor TFLOP/s against the measured sustained bf16 peak.
    dominant = max(prof.items(), key=lambda kv_: kv_[1][1])[0]
    n_l, ms_l = prof["layer_fused"]
    achieved = gemm_flops_total / max(1e-9, ms_l * 1e-3) / 1e12
    roofline = {"kernel": "layer_kernel", "bound": "tensor", "achieved": achieved,
                "peak": peaks["tf_sustained"], "unit": "TFLOP/s", "frac": achieved / peaks["tf_sustained"],
                "frac_burst": achieved / peaks["tf_burst"], "peak_burst": peaks["tf_burst"],
                "traffic": LAYER_KERNEL_DRAM_BYTES_PER_LAUNCH if (T, d, shape.grid_size) == (32768, 1024, 16) else None,
                "traffic_unit": "bytes per launch (ncu dram read+write, mean of the encode and decode launches)",
                "algorithmic_bytes_per_launch": 0.5 * (enc_bytes + dec_bytes) * T,
                "peak_source": peaks["source"] + " (sustained)", "dominant_by_time": dominant,
                "launches": n_l, "avg_launch_ms": ms_l / max(1, n_l)}

    # ---- end to end through the C ABI with host buffers ------------------------------------------
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, codec, chain, shape, kv, ad, cache, bufs, q, out, ctx_len, scale, dev, world)

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": shape.name, "tokens_per_gpu": T, "layers": L, "d_kv": d, "bits_per_value": 2,
                   "grid_points": shape.grid_size, "hadamard_block": shape.had_block, "attn_batch": batch,
                   "attn_ctx": ctx_len, "n_q_heads": n_q, "l2": "inputs (%.1f GB of K/V per step) exceed L2" %
                   (2 * L * T * d * 2 / 1e9), "rows_per_chunk": rows_per_call},
        "ops": roof, "kernels": kernels, "roofline": roofline, "clocks": clocks, "gpu_launches": launches,
        "e2e": e2e,
    }
    if world == 1 and not args.no_other_configs and not (args.tokens or args.layers):
        # the same encode and plain-decode chains through aquakv_encode_chain / aquakv_decode_chain, which run up
        # to 24 layers per launch of the layer kernel at this size (no pipeline fill and drain between layers)
        multi = []
        for name, fn, enc in (("encode_layers", lambda: chain.encode_layers(codec, kv.K, kv.V, ad, cache, bufs), True),
                              ("decode_layers", lambda: chain.decode_layers(codec, cache, ad, bufs), False)):
            ms_chain = _time_calls(fn, 5, warm=2)
            multi.append(_shape_entry(peaks, shape, name, T, ms_chain / L, _shape_bytes(shape, T, enc), config=2,
                                      ms_chain=ms_chain, chain_layers=L,
                                      note="all layers through the chain entry point (24 layers per launch); per layer = "
                                           "chain time / layers, the unpredicted first layer included"))
        assert codec.poll_status() == 0
        del kv, cache, bufs, q, out
        torch.cuda.empty_cache()
        result["ops_by_config"] = ([dict(config=2, workload=shape.name, op=name, tokens_per_call=T, **v)
                                    for name, v in roof.items()] + multi + ops_by_config(api, chain, peaks, dev) +
                                   [calibration_entry(api, peaks, dev)] + uniform_backbone_entries(api, chain, peaks, dev))
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        result["cpu_baseline"] = oracle_baseline(shape, n_q)
    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def run_e2e(args, codec, chain, shape, kv, ad, cache, bufs, q, out, ctx_len, scale, dev, world):
    """Same step, but every input starts in pinned host memory and every product ends there:
    per layer H2D(K, V) -> encode -> D2H(codes, scales); then H2D(codes, scales, q) -> decode +
    attention -> D2H(attention output).  Copies are inside the timed region (on copy streams that
    the timed stream waits for)."""
    T, L, d = shape.n_tokens, shape.n_layers, shape.d_kv
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype, device="cpu", pin_memory=True).copy_(t)
    hK = [pin(t) for t in kv.K]
    hV = [pin(t) for t in kv.V]
    hq = [pin(t) for t in q]
    hc = [[torch.empty(t.shape, dtype=t.dtype, device="cpu", pin_memory=True) for t in lst]
          for lst in (cache.Kcodes, cache.Kscales, cache.Vcodes, cache.Vscales)]
    ho = [torch.empty(t.shape, dtype=t.dtype, device="cpu", pin_memory=True) for t in out]
    # Copies run on their own streams (PCIe is full duplex) and overlap the kernels of other layers:
    # inputs are double-buffered on the device, events order copy -> kernel -> copy per layer.
    dK = [torch.empty_like(kv.K[0]) for _ in range(2)]
    dV = [torch.empty_like(kv.V[0]) for _ in range(2)]
    dq = [torch.empty_like(q[0]) for _ in range(2)]
    dlists = (cache.Kcodes, cache.Kscales, cache.Vcodes, cache.Vscales)
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    ev = lambda: torch.cuda.Event()

    def e2e_step():
        start = ev()
        start.record(main)
        s_in.wait_event(start)
        s_out.wait_event(start)
        used = [None, None]            # event: the kernel that last read input buffer b has been issued
        d2h_done = []
        for l in range(L):
            b = l % 2
            with torch.cuda.stream(s_in):
                if used[b] is not None:
                    s_in.wait_event(used[b])
                dK[b].copy_(hK[l], non_blocking=True)
                dV[b].copy_(hV[l], non_blocking=True)
                arrived = ev()
                arrived.record(s_in)
            main.wait_event(arrived)
            cur, prv = l % 2, (l + 1) % 2
            has = l > 0
            codec.encode(dK[b], dV[b], bufs.K[prv] if has else None, bufs.V[prv] if has else None,
                         ad.Wk[l] if has else None, ad.Wv[l] if has else None, None, None,
                         cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                         bufs.K[cur], bufs.V[cur])
            used[b] = ev()
            used[b].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(used[b])
                for h, dl in zip(hc, dlists):
                    h[l].copy_(dl[l], non_blocking=True)
                done = ev()
                done.record(s_out)
                d2h_done.append(done)
        usedq = [None, None]
        for l in range(L):
            b = l % 2
            with torch.cuda.stream(s_in):
                s_in.wait_event(d2h_done[l])          # the codes of this layer have reached the host
                if usedq[b] is not None:
                    s_in.wait_event(usedq[b])
                for h, dl in zip(hc, dlists):
                    dl[l].copy_(h[l], non_blocking=True)
                dq[b].copy_(hq[l], non_blocking=True)
                arrived = ev()
                arrived.record(s_in)
            main.wait_event(arrived)
            cur, prv = l % 2, (l + 1) % 2
            has = l > 0
            codec.decode_attn(dq[b], cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l],
                              ctx_len, shape.n_kv_heads, scale,
                              bufs.K[prv] if has else None, bufs.V[prv] if has else None,
                              ad.Wk[l] if has else None, ad.Wv[l] if has else None, None, None,
                              out=out[l], Khat=bufs.K[cur], Vhat=bufs.V[cur])
            usedq[b] = ev()
            usedq[b].record(main)
            with torch.cuda.stream(s_out):
                s_out.wait_event(usedq[b])
                ho[l].copy_(out[l], non_blocking=True)
        end_out = ev()
        end_out.record(s_out)
        main.wait_event(end_out)              # the step ends when its last result is on the host

    nbytes = lambda ts: sum(t.numel() * t.element_size() for t in ts)
    code_bytes = sum(nbytes(lst) for lst in hc)
    h2d = nbytes(hK) + nbytes(hV) + code_bytes + nbytes(hq)
    d2h = code_bytes + nbytes(ho)
    e2e_step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = max(1, min(args.steps, 2))
    e0.record()
    for _ in range(steps):
        e2e_step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    if world > 1:
        import torch.distributed as dist
        t = torch.tensor([ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return {"value": world * T * L / (ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "ms_per_step": ms}


if __name__ == "__main__":
    main()
