"""The backbone quantizer with the four-dimensional 256-point grid (Section 4.1: the 2-bit grid with
d = 4, n = 256, for which the paper had no fast GPU kernel) against its oracle: layer 0 (Q alone), teacher-forced key
and value phases with predictors, decode on the oracle's codes, the one-call entry points against the
phases, edge rows.  Codes (one byte per 4 values) must equal the oracle's for every tuple whose margin
(relative gap between the two smallest squared distances) exceeds 1e-4; scales and reconstructions follow
the rules of the planar grids."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from oracle import vq
from paper_2501_19392_b200 import synth
from parity import MARGIN, check_recon, gpu_bits, scale_rows_ok

pytestmark = pytest.mark.gpu
DEV = "cuda"
# Share of 4-tuples whose oracle margin is not above 1e-4, measured with the oracle on 2000 Gaussian rows
# of 1024 values: 3.1e-4 (a point of this grid has more near neighbours than one of a planar grid: 1.2e-4 there).
UNCLEAR_RATE = 4.0e-4


def make(d, h, g, dtype):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(256, seed=9, n_samples=1 << 15, iters=12, dim=4)
    sk, sv = synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2)
    codec = api.Codec(d, h, g, grid, dtype, sk, sv)
    grid2 = synth.lloyd_grid(16, seed=7, n_samples=1 << 12, iters=10)
    lin = oracle.Oracle(d, 64, 64, grid2, dtype, sk, sv)
    return codec, vq.VectorOracle(lin, grid, h, g, sk, sv)


def check_tuples(gpu_codes, ora, rows_ok):
    got, exp = gpu_codes.astype(np.int64), ora["codes"].astype(np.int64)       # one byte per tuple
    clear = ora["margins"] > MARGIN
    rows = rows_ok[:, None] & np.ones_like(clear)
    n = int(rows.sum())
    n_unclear = int((~clear & rows).sum())
    assert n_unclear <= UNCLEAR_RATE * n + 4.0 * np.sqrt(UNCLEAR_RATE * n) + 2.0
    assert np.array_equal(got[clear & rows], exp[clear & rows])
    same = rows_ok & (got == exp).all(axis=1)
    # a row can differ only where one of its tuples is under the margin
    p = min(1.0, got.shape[1] * UNCLEAR_RATE)
    assert same.sum() >= rows_ok.sum() - (rows_ok.sum() * p + 3.0 * np.sqrt(rows_ok.sum() * p * (1 - p)) + 1.0)
    return same


CASES = [(1024, 1024, 1024, oracle.BF16, 700), (512, 128, 256, oracle.F16, 513), (256, 64, 64, oracle.BF16, 300),
         (1024, 256, 512, oracle.BF16, 257)]


@pytest.mark.parametrize("d,h,g,dtype,T", CASES)
def test_layer0_and_predicted_phases_match_the_oracle(d, h, g, dtype, T):
    from paper_2501_19392_b200 import api
    codec, ora = make(d, h, g, dtype)
    assert codec.code_bytes == d // 4 and codec.n_groups == d // g
    shape = dataclasses.replace(synth.CONFIGS[2], n_kv_heads=d // 128, head_dim=128, n_tokens=T, n_layers=2,
                                dtype=dtype, channel_scales=True)
    kv = synth.kv_chain(shape, seed=6000 + d)
    ad = synth.random_adapters(shape, seed=6100 + d)
    bits = synth.to_bits
    up = lambda a: None if a is None else (a.to(DEV) if isinstance(a, torch.Tensor) else synth.from_bits(a, dtype, DEV))
    sc = lambda t: gpu_bits(t.view(torch.float16))
    # ---- layer 0: Q alone
    o0 = ora.encode_phase(bits(kv.K[0]), [], None, role="k")
    Kc, Ks, Kh = codec.encode_phase(api.ROLE_KEY, up(kv.K[0]))
    assert codec.poll_status() == 0
    rows_ok, _ = scale_rows_ok(sc(Ks), o0["scales"], o0["scales_exact"])
    same = check_tuples(Kc.cpu().numpy(), o0, rows_ok)
    check_recon(gpu_bits(Kh), o0["hat_exact"], o0["hat"], dtype, same)
    oc = lambda o: (torch.from_numpy(o["codes"]).to(DEV), torch.from_numpy(o["scales"]).view(torch.float16).to(DEV))
    Khd = codec.decode_phase(api.ROLE_KEY, *oc(o0))
    check_recon(gpu_bits(Khd), o0["hat_exact"], o0["hat"], dtype)
    # ---- layer 1, teacher-forced on the oracle's reconstructions
    ov0 = ora.encode_phase(bits(kv.V[0]), [], None, role="v")
    ok1 = ora.encode_phase(bits(kv.K[1]), [o0["hat"]], bits(ad.Wk[1]), role="k")
    Kc1, Ks1, Kh1 = codec.encode_phase(api.ROLE_KEY, up(kv.K[1]), up(o0["hat"]), None, up(ad.Wk[1]))
    rows_ok, _ = scale_rows_ok(sc(Ks1), ok1["scales"], ok1["scales_exact"])
    same = check_tuples(Kc1.cpu().numpy(), ok1, rows_ok)
    check_recon(gpu_bits(Kh1), ok1["hat_exact"], ok1["hat"], dtype, same)
    ov1 = ora.encode_phase(bits(kv.V[1]), [ov0["hat"], ok1["hat"]], bits(ad.Wv[1]), role="v")
    Vc1, Vs1, Vh1 = codec.encode_phase(api.ROLE_VALUE, up(kv.V[1]), up(ov0["hat"]), up(ok1["hat"]), up(ad.Wv[1]))
    rows_ok, _ = scale_rows_ok(sc(Vs1), ov1["scales"], ov1["scales_exact"])
    same_v = check_tuples(Vc1.cpu().numpy(), ov1, rows_ok)
    check_recon(gpu_bits(Vh1), ov1["hat_exact"], ov1["hat"], dtype, same_v)
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


def test_full_size_call_on_sampled_rows():
    """The benchmark's launch configuration (32768 tokens x d_kv 1024 in one call: four chunks of predictor
    GEMM + row kernel per phase, the last one short) against the oracle on sampled rows, chunk borders
    included; rows are independent, so the oracle's result for a row does not depend on the others."""
    from paper_2501_19392_b200 import api
    d, T, dtype = 1024, 32768, oracle.BF16
    codec, ora = make(d, d, d, dtype)
    shape = dataclasses.replace(synth.CONFIGS[2], n_tokens=T, n_layers=2)
    kv = synth.kv_chain(shape, seed=6700, device=DEV)
    ad = synth.random_adapters(shape, seed=6701, device=DEV)
    prevK, prevV = kv.K[0], kv.V[0]          # any 16-bit rows serve as the previous layer's reconstruction
    Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(kv.K[1], kv.V[1], prevK, prevV, ad.Wk[1], ad.Wv[1])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    rng = np.random.default_rng(67)
    rows = np.unique(np.concatenate([[0, 1, 9471, 9472, 18943, 18944, 28415, 28416, T - 2, T - 1],
                                     rng.integers(0, T, 120)]))
    idx = torch.from_numpy(rows).to(DEV)
    bits = synth.to_bits
    sel = lambda t: bits(t[idx])
    sc = lambda t: gpu_bits(t.view(torch.float16))
    ok_ = ora.encode_phase(sel(kv.K[1]), [sel(prevK)], bits(ad.Wk[1]), role="k")
    rows_ok, _ = scale_rows_ok(sc(Ks[idx]), ok_["scales"], ok_["scales_exact"])
    same = check_tuples(Kc[idx].cpu().numpy(), ok_, rows_ok)
    check_recon(gpu_bits(Kh[idx]), ok_["hat_exact"], ok_["hat"], dtype, same)
    ov_ = ora.encode_phase(sel(kv.V[1]), [sel(prevV), gpu_bits(Kh[idx])], bits(ad.Wv[1]), role="v")
    rows_ok, _ = scale_rows_ok(sc(Vs[idx]), ov_["scales"], ov_["scales_exact"])
    same_v = check_tuples(Vc[idx].cpu().numpy(), ov_, rows_ok)
    check_recon(gpu_bits(Vh[idx]), ov_["hat_exact"], ov_["hat"], dtype, same_v)
    # decode of the library's own codes reproduces the encoder's reconstruction bit for bit, all rows
    Kh2, Vh2 = codec.decode(Kc, Ks, Vc, Vs, prevK, prevV, ad.Wk[1], ad.Wv[1])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    assert torch.equal(Kh2, Kh) and torch.equal(Vh2, Vh)


def test_tuples_outside_the_search_table_and_many_plain_rows():
    """The encoder finds a tuple's candidates in a table over [-4, 4)^4 and searches all 256 points for
    tuples outside it and for cells with more than 15 candidates.  Rows built so that a few percent of their
    rotated, normalised tuples lie outside the table (coordinates up to +-5), and 2000 plain Gaussian rows (about 40 of
    their half a million tuples fall into crowded cells, about 80 outside the table), must give the oracle's
    codes wherever its margin is clear."""
    from paper_2501_19392_b200 import api
    from oracle.uniform import rotate_back
    d, h, g = 1024, 256, 1024
    codec, ora = make(d, h, g, oracle.BF16)
    rng = np.random.default_rng(11)
    Y = rng.standard_normal((64, d))
    far = rng.random((64, d // 4)) < 0.1
    Y = Y.reshape(64, d // 4, 4)
    Y[far] = rng.choice([-1.0, 1.0], size=(int(far.sum()), 4)) * rng.uniform(4.2, 7.0, size=(int(far.sum()), 4)) \
        * (rng.random((int(far.sum()), 4)) < 0.5) + Y[far] * 0.3
    Y = Y.reshape(64, d)
    Y /= np.sqrt((Y ** 2).mean(axis=1, keepdims=True))             # unit root mean square: the scale is then s
    R = 0.37 * rotate_back(Y, synth.hadamard_signs(d, 1), h)
    X = torch.from_numpy(R).to(torch.bfloat16)
    o = ora.encode_phase(synth.to_bits(X), [], None, role="k")
    outside = (np.abs(o["Y"].reshape(64, d // 4, 4)) >= 4.0).any(axis=2)
    assert outside.mean() > 0.02                                   # the rows do reach beyond the table
    Kc, Ks, Kh = codec.encode_phase(api.ROLE_KEY, X.to(DEV))
    rows_ok, _ = scale_rows_ok(gpu_bits(Ks.view(torch.float16)), o["scales"], o["scales_exact"])
    clear = (o["margins"] > MARGIN) & rows_ok[:, None]
    got = Kc.cpu().numpy()
    assert np.array_equal(got[clear], o["codes"][clear])
    assert clear[outside].mean() > 0.9 and np.array_equal(got[clear & outside], o["codes"][clear & outside])
    same = rows_ok & (got == o["codes"]).all(axis=1)
    check_recon(gpu_bits(Kh), o["hat_exact"], o["hat"], oracle.BF16, same)
    # many plain rows
    Xg = synth.random_16bit((2000, d), oracle.BF16, 12)
    og = ora.encode_phase(synth.to_bits(Xg), [], None, role="v")
    Vc, Vs, Vh = codec.encode_phase(api.ROLE_VALUE, Xg.to(DEV))
    rows_ok, _ = scale_rows_ok(gpu_bits(Vs.view(torch.float16)), og["scales"], og["scales_exact"])
    same = check_tuples(Vc.cpu().numpy(), og, rows_ok)
    check_recon(gpu_bits(Vh), og["hat_exact"], og["hat"], oracle.BF16, same)
    assert codec.poll_status() == 0


def test_zero_rows_clamped_scale_and_rows_on_grid_points():
    from paper_2501_19392_b200 import api
    d, h, g = 256, 256, 256
    codec, ora = make(d, h, g, oracle.BF16)
    grid = ora.grid
    nearest_origin = int((grid ** 2).sum(axis=1).argmin())
    X = torch.zeros((4, d), dtype=torch.bfloat16)
    X[2] = 3.0e38                                    # root mean square far beyond fp16: the scale clamps at 65504
    X[3, 5] = 1.0                                    # a single spike: every rotated value has the same magnitude
    o = ora.encode_phase(synth.to_bits(X), [], None, role="k")
    Kc, Ks, Kh = codec.encode_phase(api.ROLE_KEY, X.to(DEV))
    assert (Kc[:2].cpu().numpy() == nearest_origin).all() and not Ks[:2].view(torch.int16).any() and not Kh[:2].any()
    assert np.array_equal(gpu_bits(Ks.view(torch.float16)), o["scales"])
    assert float(Ks.view(torch.float16)[2, 0]) == 65504.0
    clear = o["margins"] > MARGIN
    assert np.array_equal(Kc.cpu().numpy()[clear], o["codes"][clear])
    same = (Kc.cpu().numpy() == o["codes"]).all(axis=1)
    assert same[:2].all()
    check_recon(gpu_bits(Kh)[same & (np.arange(4) >= 2)], o["hat_exact"][same & (np.arange(4) >= 2)],
                o["hat"][same & (np.arange(4) >= 2)], oracle.BF16)
    assert codec.poll_status() == 0


def test_parameter_checks_and_unsupported_entry_points():
    from paper_2501_19392_b200 import api
    sk, sv = synth.hadamard_signs(256, 1), synth.hadamard_signs(256, 2)
    g4 = synth.lloyd_grid(64, seed=9, n_samples=1 << 12, iters=4, dim=4)
    with pytest.raises(api.AquaKVError) as e:          # only the 256-point grid
        api.Codec(256, 64, 64, g4, api.BF16, sk, sv)
    assert e.value.status == -2
    g3 = np.zeros((256, 3), dtype=np.float32)
    with pytest.raises(api.AquaKVError) as e:
        api.Codec(256, 64, 64, g3, api.BF16, sk, sv)
    assert e.value.status == -2
    codec, _ = make(256, 64, 64, oracle.BF16)
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


def test_two_bits_on_this_grid_beat_two_bits_on_the_planar_grid():
    # Section 4.1 runs the slower grid at the same 2 bits per value: a 256-point grid in four dimensions
    # packs a Gaussian better than a 16-point grid in two
    from paper_2501_19392_b200 import api
    d = 1024
    codec4, _ = make(d, d, d, oracle.BF16)
    grid2 = synth.lloyd_grid(16, seed=7, n_samples=1 << 14, iters=25)
    codec2 = api.Codec(d, d, d, grid2, api.BF16, synth.hadamard_signs(d, 1), synth.hadamard_signs(d, 2))
    assert codec4.code_bytes == codec2.code_bytes
    X = synth.random_16bit((2048, d), oracle.BF16, 5, device=DEV)
    _, _, H4 = codec4.encode_phase(api.ROLE_KEY, X)
    _, _, H2 = codec2.encode_phase(api.ROLE_KEY, X)
    e4 = float(((X.float() - H4.float()) ** 2).sum() / (X.float() ** 2).sum())
    e2 = float(((X.float() - H2.float()) ** 2).sum() / (X.float() ** 2).sum())
    assert e4 < 0.95 * e2, (e4, e2)
    assert codec4.poll_status() == 0 and codec2.poll_status() == 0
