"""The uniform round-to-nearest backbone with absmax normalisation (Section 4.1 "Alternative quantizers")
against its oracle: layer 0 (Q alone), teacher-forced key and value phases with predictors, decode on
the oracle's codes, and the one-call entry points against the phases.  Levels must equal the oracle's
wherever its normalised value is more than 1e-4 of a level spacing away from a decision boundary (the
kernel divides in fp32, the oracle in double); reconstructions follow the rule of the other parity
tests (2e-3 of the row's scale or one 16-bit spacing) on rows whose levels and scales all agree."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from oracle import uniform as uq
from oracle import calibration as cal
from paper_2501_19392_b200 import synth
from parity import check_recon, gpu_bits, scale_rows_ok

pytestmark = pytest.mark.gpu
DEV = "cuda"
MARGIN = 1e-4
# The scale is ONE element's |x - pred| (the group's maximum), so it carries that element's fp32
# prediction error in full: about 1e-6 of the prediction's magnitude, which is a few times the
# residual's.  A scale may therefore differ from the oracle's by one fp16 step when the oracle's
# unrounded value is within 1e-5 of a rounding boundary (2e-6 for the root-mean-square scale of the
# rotated quantizer, which averages the errors of a whole group).
SCALE_TOL = 1e-5


def make(d, b, g, dtype, h=1):
    """h > 1: the rotated variant (random signs + Hadamard blocks of h values before the levels)."""
    from paper_2501_19392_b200 import api
    sk, sv = synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2)
    codec = api.Codec(d, h, g, None, dtype, levels=1 << b, signs_k=sk if h > 1 else None,
                      signs_v=sv if h > 1 else None)
    grid = synth.lloyd_grid(16, seed=7, n_samples=1 << 12, iters=10)
    lin = oracle.Oracle(d, 64, 64, grid, dtype, sk, sv)
    return codec, uq.UniformOracle(lin, b, g, had_block=h, signs_k=sk, signs_v=sv)


def check_levels(gpu_codes, ora, b, d, rows_ok):
    got = uq._unpack(gpu_codes, b, d)
    exp = uq._unpack(ora["codes"], b, d)
    clear = ora["margins"] > MARGIN
    rows = rows_ok[:, None] & np.ones_like(clear)
    assert np.array_equal(got[clear & rows], exp[clear & rows])
    # what is left over differs by at most one level
    assert (np.abs(got - exp)[rows] <= 1).all()
    # (16-bit inputs over a 16-bit-derived scale land exactly on boundaries quite often; exact ties are
    # decided alike by both sides, so what is bounded is the share of levels that actually differ)
    assert (got != exp)[rows].mean() < 1e-3
    return rows_ok & (got == exp).all(axis=1)


CASES = [(256, 2, 64, oracle.BF16, 700, 1), (512, 3, 64, oracle.F16, 513, 1), (1024, 4, 32, oracle.BF16, 300, 1),
         (1024, 2, 256, oracle.BF16, 1000, 1), (1024, 2, 1024, oracle.BF16, 600, 1), (512, 4, 512, oracle.F16, 257, 1),
         # rotated variant: one group per row (the appendix' setting), and blocks / groups of other sizes
         (1024, 2, 1024, oracle.BF16, 700, 1024), (512, 3, 64, oracle.F16, 513, 128), (256, 4, 256, oracle.BF16, 300, 64),
         (1024, 2, 128, oracle.BF16, 400, 512), (512, 2, 512, oracle.BF16, 257, 512)]


@pytest.mark.parametrize("d,b,g,dtype,T,h", CASES)
def test_layer0_and_predicted_phases_match_the_oracle(d, b, g, dtype, T, h):
    from paper_2501_19392_b200 import api
    codec, ora = make(d, b, g, dtype, h)
    assert codec.code_bytes == d * b // 8 and codec.n_groups == d // g
    shape = dataclasses.replace(synth.CONFIGS[2], n_kv_heads=d // 128, head_dim=128, n_tokens=T, n_layers=2,
                                dtype=dtype, channel_scales=True)
    kv = synth.kv_chain(shape, seed=4000 + d + b)
    ad = synth.random_adapters(shape, seed=4100 + d + b)
    bits = synth.to_bits
    up = lambda a: None if a is None else (a.to(DEV) if isinstance(a, torch.Tensor) else synth.from_bits(a, dtype, DEV))
    # ---- layer 0: Q alone
    o0 = ora.encode_phase(bits(kv.K[0]), [], None)
    Kc, Ks, Kh = codec.encode_phase(api.ROLE_KEY, up(kv.K[0]))
    assert codec.poll_status() == 0
    rows_ok, _ = scale_rows_ok(gpu_bits(Ks.view(torch.float16)), o0["scales"], o0["scales_exact"], SCALE_TOL)
    same = check_levels(Kc.cpu().numpy(), o0, b, d, rows_ok)
    assert same.mean() > 0.9
    check_recon(gpu_bits(Kh), o0["hat_exact"], o0["hat"], dtype, same)
    Khd = codec.decode_phase(api.ROLE_KEY, torch.from_numpy(o0["codes"]).to(DEV),
                             torch.from_numpy(o0["scales"]).view(torch.float16).to(DEV))
    if h == 1:
        assert np.array_equal(gpu_bits(Khd), o0["hat"])      # level * scale rounded once: exact
    else:
        check_recon(gpu_bits(Khd), o0["hat_exact"], o0["hat"], dtype)
    # ---- layer 1, teacher-forced on the oracle's reconstructions
    ov0 = ora.encode_phase(bits(kv.V[0]), [], None, role="v")
    ok1 = ora.encode_phase(bits(kv.K[1]), [o0["hat"]], bits(ad.Wk[1]))
    Kc1, Ks1, Kh1 = codec.encode_phase(api.ROLE_KEY, up(kv.K[1]), up(o0["hat"]), None, up(ad.Wk[1]))
    rows_ok, _ = scale_rows_ok(gpu_bits(Ks1.view(torch.float16)), ok1["scales"], ok1["scales_exact"], SCALE_TOL)
    same = check_levels(Kc1.cpu().numpy(), ok1, b, d, rows_ok)
    check_recon(gpu_bits(Kh1), ok1["hat_exact"], ok1["hat"], dtype, same)
    ov1 = ora.encode_phase(bits(kv.V[1]), [ov0["hat"], ok1["hat"]], bits(ad.Wv[1]), role="v")
    Vc1, Vs1, Vh1 = codec.encode_phase(api.ROLE_VALUE, up(kv.V[1]), up(ov0["hat"]), up(ok1["hat"]), up(ad.Wv[1]))
    rows_ok, _ = scale_rows_ok(gpu_bits(Vs1.view(torch.float16)), ov1["scales"], ov1["scales_exact"], SCALE_TOL)
    same_v = check_levels(Vc1.cpu().numpy(), ov1, b, d, rows_ok)
    check_recon(gpu_bits(Vh1), ov1["hat_exact"], ov1["hat"], dtype, same_v)
    # decode on the oracle's codes
    oc = lambda o: (torch.from_numpy(o["codes"]).to(DEV), torch.from_numpy(o["scales"]).view(torch.float16).to(DEV))
    Vhd = codec.decode_phase(api.ROLE_VALUE, *oc(ov1), up(ov0["hat"]), up(ok1["hat"]), up(ad.Wv[1]))
    check_recon(gpu_bits(Vhd), ov1["hat_exact"], ov1["hat"], dtype)
    # ---- the one-call entry points are the two phases; decode reproduces encode bit for bit
    Kc2, Ks2, Vc2, Vs2, Kh2, Vh2 = codec.encode(up(kv.K[1]), up(kv.V[1]), up(o0["hat"]), up(ov0["hat"]),
                                                up(ad.Wk[1]), up(ad.Wv[1]))
    assert torch.equal(Kc2, Kc1) and torch.equal(Ks2, Ks1) and torch.equal(Kh2, Kh1)
    Vc3, Vs3, Vh3 = codec.encode_phase(api.ROLE_VALUE, up(kv.V[1]), up(ov0["hat"]), Kh2, up(ad.Wv[1]))
    assert torch.equal(Vc2, Vc3) and torch.equal(Vs2, Vs3) and torch.equal(Vh2, Vh3)
    Kh4, Vh4 = codec.decode(Kc2, Ks2, Vc2, Vs2, up(o0["hat"]), up(ov0["hat"]), up(ad.Wk[1]), up(ad.Wv[1]))
    assert torch.equal(Kh4, Kh2) and torch.equal(Vh4, Vh2)
    assert codec.poll_status() == 0


def test_zero_rows_ties_and_saturation_on_the_gpu():
    from paper_2501_19392_b200 import api
    d, b, g = 256, 2, 64
    codec, ora = make(d, b, g, oracle.BF16)
    X = torch.zeros((4, d), dtype=torch.bfloat16)
    X[0, :7] = torch.tensor([2.0, -1.5, -0.5, 0.5, 1.5, -2.0, 0.4375])     # scale exactly 1: every boundary is hit
    X[2, 70] = -3.0                                                          # a lone negative maximum is exact
    X[3, :] = 1.0e38                                                         # scale clamps at the largest fp16
    o = ora.encode_phase(synth.to_bits(X), [], None)
    Kc, Ks, Kh = codec.encode_phase(api.ROLE_KEY, X.to(DEV))
    assert np.array_equal(Kc.cpu().numpy(), o["codes"])
    assert np.array_equal(gpu_bits(Ks.view(torch.float16)), o["scales"])
    assert np.array_equal(gpu_bits(Kh), o["hat"])
    lv = uq._unpack(Kc.cpu().numpy(), b, d) - 2
    assert list(lv[0, :7]) == [1, -2, -1, 0, 1, -2, 0] and (lv[1] == 0).all() and lv[2, 70] == -2
    assert not Kh[1].any() and float(Kh[2, 70]) == -3.0
    assert codec.poll_status() == 0


def test_parameter_checks_and_unsupported_entry_points():
    from paper_2501_19392_b200 import api
    for bad in (dict(had_block=32), dict(had_block=512), dict(had_block=96), dict(levels=32), dict(scale_group=16), dict(scale_group=512), dict(scale_group=96)):
        kw = dict(had_block=1, scale_group=64, levels=4)
        kw.update(bad)
        with pytest.raises(api.AquaKVError) as e:
            api.Codec(256, kw["had_block"], kw["scale_group"], None, api.BF16, levels=kw["levels"])
        assert e.value.status == -2
    with pytest.raises(api.AquaKVError) as e:          # a rotation needs its signs
        api.Codec(256, 64, 64, None, api.BF16, levels=4)
    assert e.value.status == -1
    codec, _ = make(256, 2, 64, oracle.BF16)
    T = 64
    c = torch.zeros((T, codec.code_bytes), dtype=torch.uint8, device=DEV)
    s = torch.ones((T, codec.n_groups), dtype=torch.float16, device=DEV)
    q = torch.zeros((1, 8, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(api.AquaKVError) as e:
        codec.decode_attn(q, c, s, c, s, T, 2, 0.1, workspace=torch.empty(1 << 20, dtype=torch.uint8, device=DEV))
    assert e.value.status == -2
    with pytest.raises(api.AquaKVError) as e:
        codec.decode_noalloc(c, s, c, s)
    assert e.value.status == -2
    assert codec.chain_workspace_bytes(T, 2) == 0


def test_rotated_variant_spike_row_zero_row_and_clamp_on_the_gpu():
    from paper_2501_19392_b200 import api
    d, b, g, h = 256, 2, 256, 256
    codec, ora = make(d, b, g, oracle.BF16, h)
    sk = synth.hadamard_signs(d, 1).astype(np.float64)
    j = 37
    col = np.array([(-1.0) ** bin(i & j).count("1") for i in range(d)])
    X = torch.zeros((3, d), dtype=torch.bfloat16)
    X[0] = torch.from_numpy(0.75 * sk * col).to(torch.bfloat16)          # rotates to the spike 12 e_j: scale 6
    X[2] = torch.from_numpy(1.0e30 * sk * col).to(torch.bfloat16)        # spike far beyond fp16: the scale clamps
    o = ora.encode_phase(synth.to_bits(X), [], None)
    Kc, Ks, Kh = codec.encode_phase(api.ROLE_KEY, X.to(DEV))
    assert np.array_equal(Kc.cpu().numpy(), o["codes"])
    assert np.array_equal(gpu_bits(Ks.view(torch.float16)), o["scales"])
    lv = uq._unpack(Kc.cpu().numpy(), b, d) - 2
    assert lv[0, j] == 1 and (np.delete(lv[0], j) == 0).all() and (lv[1] == 0).all()
    assert float(Ks.view(torch.float16)[0, 0]) == 6.0 and float(Ks.view(torch.float16)[2, 0]) == 65504.0
    assert np.array_equal(gpu_bits(Kh[:2]), o["hat"][:2])                 # 0.375 * (+-1) and zeros: exact
    assert torch.equal(Kh[0].float().cpu(), 0.5 * X[0].float()) and not Kh[1].any()
    check_recon(gpu_bits(Kh)[[0, 2]], o["hat_exact"][[0, 2]], o["hat"][[0, 2]], oracle.BF16)
    assert codec.poll_status() == 0


@pytest.mark.parametrize("b,g,h", [(2, 64, 1), (2, 1024, 1024)])
def test_full_size_call_on_sampled_rows(b, g, h):
    """The benchmark's launch configuration (32768 tokens x d_kv 1024 in one call: four chunks of predictor
    GEMM + row kernel per phase, the last one short) against the oracle on sampled rows, chunk borders
    included; rows are independent, so the oracle's result for a row does not depend on the others."""
    from paper_2501_19392_b200 import api
    d, T, dtype = 1024, 32768, oracle.BF16
    codec, ora = make(d, b, g, dtype, h)
    shape = dataclasses.replace(synth.CONFIGS[2], n_tokens=T, n_layers=2)
    kv = synth.kv_chain(shape, seed=4700 + h, device=DEV)
    ad = synth.random_adapters(shape, seed=4701 + h, device=DEV)
    prevK, prevV = kv.K[0], kv.V[0]          # any 16-bit rows serve as the previous layer's reconstruction
    Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(kv.K[1], kv.V[1], prevK, prevV, ad.Wk[1], ad.Wv[1])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    rng = np.random.default_rng(47)
    rows = np.unique(np.concatenate([[0, 1, 9471, 9472, 18943, 18944, 28415, 28416, T - 2, T - 1],
                                     rng.integers(0, T, 120)]))
    idx = torch.from_numpy(rows).to(DEV)
    bits = synth.to_bits
    sel = lambda t: bits(t[idx])
    ok_ = ora.encode_phase(sel(kv.K[1]), [sel(prevK)], bits(ad.Wk[1]), role="k")
    rows_ok, _ = scale_rows_ok(gpu_bits(Ks[idx].view(torch.float16)), ok_["scales"], ok_["scales_exact"], SCALE_TOL)
    same = check_levels(Kc[idx].cpu().numpy(), ok_, b, d, rows_ok)
    check_recon(gpu_bits(Kh[idx]), ok_["hat_exact"], ok_["hat"], dtype, same)
    ov_ = ora.encode_phase(sel(kv.V[1]), [sel(prevV), gpu_bits(Kh[idx])], bits(ad.Wv[1]), role="v")
    rows_ok, _ = scale_rows_ok(gpu_bits(Vs[idx].view(torch.float16)), ov_["scales"], ov_["scales_exact"], SCALE_TOL)
    same_v = check_levels(Vc[idx].cpu().numpy(), ov_, b, d, rows_ok)
    check_recon(gpu_bits(Vh[idx]), ov_["hat_exact"], ov_["hat"], dtype, same_v)
    assert same.mean() > 0.8 and same_v.mean() > 0.8
    # decode of the library's own codes reproduces the encoder's reconstruction bit for bit, all rows
    Kh2, Vh2 = codec.decode(Kc, Ks, Vc, Vs, prevK, prevV, ad.Wk[1], ad.Wv[1])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    assert torch.equal(Kh2, Kh) and torch.equal(Vh2, Vh)


def test_fitted_predictors_help_this_backbone_too():
    # Section 4.1 evaluates each backbone both with the learned predictors and without them
    from paper_2501_19392_b200 import api, calibrate as gcal
    d, b, g = 256, 2, 64
    codec, ora = make(d, b, g, oracle.BF16)
    shape = dataclasses.replace(synth.CONFIGS[2], n_kv_heads=2, head_dim=128, n_tokens=4096, n_layers=3,
                                channel_scales=False)
    kv = synth.kv_chain(shape, seed=4500)
    K, V = [t.to(DEV) for t in kv.K], [t.to(DEV) for t in kv.V]
    preds, recs = gcal.calibrate(codec, K, V, rate=1e-3, keep_reconstructions=True)
    _, _, direct = codec.encode_phase(api.ROLE_KEY, K[2])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    e_fit = cal.relative_error(synth.to_bits(kv.K[2]), gpu_bits(recs[2][0]), shape.dtype)
    e_dir = cal.relative_error(synth.to_bits(kv.K[2]), gpu_bits(direct), shape.dtype)
    assert e_fit < 0.5 * e_dir, (e_fit, e_dir)
