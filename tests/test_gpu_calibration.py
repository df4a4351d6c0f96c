"""aquakv_fit_predictor and the calibration loop (Algorithm 1; Section 3.2; Appendix A) against the
calibration oracle.

What is compared.  A fit solves (G + ridge I) W^T = C with G = X^T X, C = X^T Y.  The GPU forms G and C
on the tensor cores (exact 16-bit products, fp32 accumulation) and solves in double; the oracle does
everything in double.  The accumulation error of G and C is the only difference: relative to the
diagonal of G about 2^-24 times the square root of the number of accumulation steps, a few 1e-6,
amplified in the directions that the data determines poorly.  Measured on the cases below: the two
solutions differ by 6e-6 ... 9.5e-5 of the matrix in Frobenius norm and their predictions X W^T by
5.6e-6 ... 3.5e-5; the bounds are ten times the largest measured value (1e-3 and 3e-4).  The 16-bit
adapter is the double solution rounded once.  Against the oracle's rounded matrix an element may
differ by one 16-bit spacing where the two double values straddle a rounding boundary, or, for
elements far below the matrix' scale, by their absolute error (bound: 1e-3 of the matrix' rms);
the share of elements that differ at all is about (relative difference of the solutions) / (relative
16-bit spacing): measured 0.3 % to 1.2 % for bf16 (spacing 2^-8) and 20 % for the fp16 case (spacing
2^-11, solutions 9.5e-5 apart); bound: three times that ratio plus 1 %.
"""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from oracle import calibration as cal
from paper_2501_19392_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make(shape):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(shape.grid_size, seed=7, n_samples=1 << 14, iters=25)
    sk, sv = synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12)
    args = (shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype, sk, sv)
    return api.Codec(*args), oracle.Oracle(*args)


def small_shape(d_heads, T, L, dtype, channel_scales=False, n=16):
    return dataclasses.replace(synth.CONFIGS[2], n_kv_heads=d_heads, head_dim=128, n_tokens=T, n_layers=L,
                               dtype=dtype, had_block=128 * d_heads, scale_group=128 * d_heads, grid_size=n,
                               channel_scales=channel_scales)


def compare_fit(o, W16, W32, bias, ref, X64, want_bias):
    W32 = W32.cpu().numpy().astype(np.float64)
    Wr = ref["W_exact"]
    fro = np.linalg.norm(W32 - Wr) / np.linalg.norm(Wr)
    pred = np.linalg.norm(X64 @ (W32 - Wr).T) / np.linalg.norm(X64 @ Wr.T)
    assert fro < 1e-3, fro
    assert pred < 3e-4, pred
    got_bits, exp_bits = synth.to_bits(W16.cpu()), ref["W"]
    dt = oracle.F16 if W16.dtype == torch.float16 else oracle.BF16
    got, exp = cal.bits_to_double(got_bits, dt), cal.bits_to_double(exp_bits, dt)
    # an element may land on the neighbouring 16-bit value when the two double solutions straddle a
    # rounding boundary; elements far below the matrix' scale may move by their (tiny) absolute error
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(exp), 1e-30))) - (10 if dt == oracle.F16 else 7))
    rms = np.sqrt((Wr ** 2).mean())
    mism = (got_bits != exp_bits).mean()
    assert (np.abs(got - exp) <= np.maximum(ulp, 1e-3 * rms)).all()
    assert mism < 3.0 * fro / (2.0 ** -11 if dt == oracle.F16 else 2.0 ** -8) + 1e-2, (mism, fro)
    if want_bias:
        b = bias.cpu().numpy().astype(np.float64)
        scale = np.abs(ref["bias"]).max() + 1e-3
        assert np.abs(b - ref["bias"]).max() < 1e-4 * scale + 1e-5
    return fro, pred


@pytest.mark.parametrize("heads,T,dtype,two_inputs,bias,scales", [
    (2, 3000, oracle.BF16, False, False, False),     # d_kv 256, ragged token count
    (2, 4096, oracle.F16, True, True, False),        # value predictor with intercept, fp16
    (4, 2048, oracle.BF16, True, False, True),       # d_kv 512, fewer tokens than 2 x features, outlier channels
    (8, 6144, oracle.BF16, False, False, True),      # d_kv 1024 (the benchmark's width), outlier channels
])
def test_fit_matches_the_oracle(heads, T, dtype, two_inputs, bias, scales):
    shape = small_shape(heads, T, 2, dtype, scales)
    codec, ora = make(shape)
    kv = synth.kv_chain(shape, seed=9100 + heads)
    if bias:
        off = torch.linspace(-3.0, 3.0, shape.d_kv)
        kv.K[0] = (kv.K[0].float() + off).to(kv.K[0].dtype)
        kv.V[1] = (kv.V[1].float() - 0.5 * off).to(kv.V[1].dtype)
    if two_inputs:
        ins, tgt = [kv.V[0], kv.K[1]], kv.V[1]
    else:
        ins, tgt = [kv.K[0]], kv.K[1]
    W16, b, W32 = codec.fit_predictor(tgt.to(DEV), ins[0].to(DEV), ins[1].to(DEV) if two_inputs else None,
                                      rate=1e-3, fit_bias=bias, want_fp32=True)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    ref = cal.fit_predictor([synth.to_bits(t) for t in ins], synth.to_bits(tgt), dtype, 1e-3, bias)
    X64 = np.concatenate([cal.bits_to_double(synth.to_bits(t), dtype) for t in ins], axis=1)
    if bias:
        X64 = X64 - X64.mean(axis=0)
    compare_fit(ora, W16, W32, b, ref, X64, bias)


def test_fit_at_the_benchmark_size():
    # the key fit bench.py times: 32768 calibration tokens, d_kv 1024, outlier channels
    shape = small_shape(8, 32768, 2, oracle.BF16, channel_scales=True)
    codec, ora = make(shape)
    kv = synth.kv_chain(shape, seed=6001)
    W16, _, W32 = codec.fit_predictor(kv.K[1].to(DEV), kv.K[0].to(DEV), None, rate=1e-3, want_fp32=True)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    ref = cal.fit_predictor([synth.to_bits(kv.K[0])], synth.to_bits(kv.K[1]), shape.dtype, 1e-3)
    compare_fit(ora, W16, W32, None, ref, cal.bits_to_double(synth.to_bits(kv.K[0]), shape.dtype), False)


def test_rows_with_padding_and_rate_zero_on_a_planted_map():
    # strided inputs (ld > d_kv) and an exactly linear target: W is the planted matrix up to 16-bit rounding
    shape = small_shape(2, 2048, 2, oracle.BF16)
    codec, ora = make(shape)
    d = shape.d_kv
    g = torch.Generator().manual_seed(5)
    Xbig = torch.randn((2048, d + 64), generator=g).bfloat16()
    X = Xbig[:, :d]
    A = (torch.randn((d, d), generator=g) / 16.0)
    Ybig = torch.zeros((2048, d + 8), dtype=torch.bfloat16)
    Ybig[:, :d] = (X.float() @ A.T).bfloat16()
    Xd, Yd = Xbig.to(DEV)[:, :d], Ybig.to(DEV)[:, :d]
    assert Xd.stride(0) == d + 64 and Yd.stride(0) == d + 8
    W16, _, W32 = codec.fit_predictor(Yd, Xd, None, rate=0.0, want_fp32=True)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    ref = cal.fit_predictor([synth.to_bits(X.contiguous())], synth.to_bits(Ybig[:, :d].contiguous()), oracle.BF16, 0.0)
    W = W32.cpu().numpy().astype(np.float64)
    assert np.linalg.norm(W - ref["W_exact"]) / np.linalg.norm(ref["W_exact"]) < 1e-3
    # the target was rounded to bf16 (relative 2^-9 per element), so A is recovered to about that
    assert np.linalg.norm(W - A.numpy()) / np.linalg.norm(A.numpy()) < 1e-2


def test_calibration_loop_teacher_forced_and_free_running():
    shape = small_shape(2, 4096, 4, oracle.BF16, channel_scales=True)
    codec, ora = make(shape)
    from paper_2501_19392_b200 import calibrate as gcal
    kv = synth.kv_chain(shape, seed=9300)
    K = [synth.to_bits(t) for t in kv.K]
    V = [synth.to_bits(t) for t in kv.V]
    ref = cal.calibrate(ora, K, V, rate=1e-3)
    dt = shape.dtype
    # teacher-forced: every GPU fit sees the oracle's reconstructions of the previous layer
    k_old = ora.encode_phase(K[0], [], None, None, "k")["hat"]
    v_old = ora.encode_phase(V[0], [], None, None, "v")["hat"]
    up = lambda bits: synth.from_bits(bits, dt, DEV)
    for l in range(1, shape.n_layers):
        r = ref[l - 1]
        Wk16, _, Wk32 = codec.fit_predictor(up(K[l]), up(k_old), None, 1e-3, want_fp32=True)
        Xk = cal.bits_to_double(k_old, dt)
        compare_fit(ora, Wk16, Wk32, None, dict(W=r["Wk"], W_exact=r["Wk_exact"]), Xk, False)
        Wv16, _, Wv32 = codec.fit_predictor(up(V[l]), up(v_old), up(r["Khat"]), 1e-3, want_fp32=True)
        Xv = np.concatenate([cal.bits_to_double(v_old, dt), cal.bits_to_double(r["Khat"], dt)], axis=1)
        compare_fit(ora, Wv16, Wv32, None, dict(W=r["Wv"], W_exact=r["Wv_exact"]), Xv, False)
        k_old, v_old = r["Khat"], r["Vhat"]
    assert codec.poll_status() == 0
    # free-running: the whole of Algorithm 1 on the GPU; the two chains differ by near-tie code flips and
    # 16-bit roundings, so compare what the calibration is for: the reconstruction error it reaches
    preds, recs = gcal.calibrate(codec, [t.to(DEV) for t in kv.K], [t.to(DEV) for t in kv.V], rate=1e-3,
                                 keep_reconstructions=True)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    for l in range(1, shape.n_layers):
        ek = cal.relative_error(K[l], synth.to_bits(recs[l][0].cpu()), dt)
        ev = cal.relative_error(V[l], synth.to_bits(recs[l][1].cpu()), dt)
        rk = cal.relative_error(K[l], ref[l - 1]["Khat"], dt)
        rv = cal.relative_error(V[l], ref[l - 1]["Vhat"], dt)
        assert abs(ek - rk) <= 0.01 * rk and abs(ev - rv) <= 0.01 * rv, (l, ek, rk, ev, rv)
        # and the fitted predictors do their job: far below coding the layer directly at the same bits
        dk = cal.relative_error(K[l], ora.encode_phase(K[l], [], None, None, "k")["hat"], dt)
        assert ek < 0.5 * dk
        assert preds.Wk[l].shape == (shape.d_kv, shape.d_kv) and preds.Wv[l].shape == (shape.d_kv, 2 * shape.d_kv)


def test_argument_errors_and_a_matrix_that_is_not_positive_definite():
    from paper_2501_19392_b200 import api
    shape = small_shape(2, 256, 2, oracle.BF16)
    codec, _ = make(shape)
    d = shape.d_kv
    X = torch.randn((256, d), device=DEV).bfloat16()
    Y = torch.randn((256, d), device=DEV).bfloat16()
    small = torch.empty(1024, dtype=torch.uint8, device=DEV)
    with pytest.raises(api.AquaKVError) as e:
        codec.fit_predictor(Y, X, None, workspace=small)
    assert e.value.status == -4
    with pytest.raises(api.AquaKVError) as e:
        codec.fit_predictor(Y, X, None, rate=-1.0)
    assert e.value.status == -1
    with pytest.raises(api.AquaKVError) as e:
        codec.fit_predictor(Y, X[:, 1:], None)          # misaligned rows
    assert e.value.status in (-1, -3)
    # all-zero inputs without a ridge term: the first pivot is zero -> reported, nothing faults, ctx usable
    Z = torch.zeros((256, d), device=DEV, dtype=torch.bfloat16)
    codec.fit_predictor(Y, Z, None, rate=0.0)
    assert codec.poll_status() == api.ERR_NUMERIC
    assert codec.poll_status() == 0
    W16, _, _ = codec.fit_predictor(Y, X, None, rate=1e-3)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0 and torch.isfinite(W16.float()).all()
