"""Parity of the CUDA library (through its C ABI) against the CPU oracle, element by element, on
seeded inputs small enough for the oracle but spanning several 128-row GEMM tiles, several
8-row codec blocks and ragged tails."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2501_19392_b200 import synth
from parity import check_codes, check_recon, check_same_rows, gpu_bits, scale_rows_ok
from util import bits_to_f64

pytestmark = pytest.mark.gpu

DEV = "cuda"


def make(d, h, g, n, dtype):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(n, seed=7, n_samples=1 << 14, iters=25)
    sk, sv = synth.hadamard_signs(d, 11), synth.hadamard_signs(d, 12)
    return api.Codec(d, h, g, grid, dtype, sk, sv), oracle.Oracle(d, h, g, grid, dtype, sk, sv)


def chain(cfg, T, L, seed=0, **kw):
    shape = dataclasses.replace(synth.CONFIGS[cfg], n_tokens=T, n_layers=L, **kw)
    kv = synth.kv_chain(shape, seed=1000 * cfg + seed)
    ad = synth.random_adapters(shape, seed=1000 * cfg + 500 + seed, bias=False)
    return shape, kv, ad


LAYER0_CASES = [
    (512, 64, 64, 16, synth.F16), (1024, 1024, 1024, 16, synth.BF16), (1024, 1024, 1024, 64, synth.BF16),
    (1024, 1024, 1024, 256, synth.BF16), (1024, 256, 512, 16, synth.F16), (512, 512, 512, 64, synth.BF16),
    (256, 256, 256, 16, synth.BF16), (256, 64, 128, 256, synth.F16), (512, 128, 512, 16, synth.BF16),
]


@pytest.mark.parametrize("d,h,g,n,dtype", LAYER0_CASES)
@pytest.mark.parametrize("T", [1, 37, 300])
def test_layer0_encode_and_decode_match_oracle(d, h, g, n, dtype, T):
    codec, ora = make(d, h, g, n, dtype)
    bits = int(np.log2(n))
    X = synth.random_16bit((T, d), dtype, seed=d + n + T, std=1.7)
    Xv = synth.random_16bit((T, d), dtype, seed=d + n + T + 1, std=0.02)
    ok_, ov_ = ora.encode_layer(synth.to_bits(X), synth.to_bits(Xv))
    Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(X.to(DEV), Xv.to(DEV))
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    for o, c, s, hhat in ((ok_, Kc, Ks, Kh), (ov_, Vc, Vs, Vh)):
        rows_ok, n_bad = scale_rows_ok(gpu_bits(s.view(torch.float16)), o["scales"], o["scales_exact"])
        assert n_bad <= max(1, T // 50)
        check_codes(c.cpu().numpy(), o, bits, rows_ok)
    # decode of the ORACLE's codes against the oracle's reconstruction
    Kh2, Vh2 = codec.decode(torch.from_numpy(ok_["codes"]).to(DEV),
                            torch.from_numpy(ok_["scales"]).view(torch.float16).to(DEV),
                            torch.from_numpy(ov_["codes"]).to(DEV),
                            torch.from_numpy(ov_["scales"]).view(torch.float16).to(DEV))
    check_recon(gpu_bits(Kh2), ok_["hat_exact"], ok_["hat"], dtype)
    check_recon(gpu_bits(Vh2), ov_["hat_exact"], ov_["hat"], dtype)
    # the library's decode of its OWN codes reproduces its encoder's reconstruction bit for bit
    Kh3, Vh3 = codec.decode(Kc, Ks, Vc, Vs)
    assert torch.equal(Kh3, Kh) and torch.equal(Vh3, Vh)


@pytest.mark.parametrize("cfg,T", [(1, 300), (2, 300), (2, 129), (1, 5)])
def test_predictor_matches_oracle(cfg, T):
    shape, kv, ad = chain(cfg, T, 2)
    codec, ora = make(shape.d_kv, shape.had_block, shape.scale_group, shape.grid_size, shape.dtype)
    K0, V0 = kv.K[0], kv.V[0]
    for ins, W in (([K0], ad.Wk[1]), ([V0, K0], ad.Wv[1])):
        P = codec.predict(ins[0].to(DEV), ins[1].to(DEV) if len(ins) > 1 else None, W.to(DEV))
        ref = ora.predict([synth.to_bits(t) for t in ins], synth.to_bits(W))
        err = np.abs(P.cpu().numpy().astype(np.float64) - ref)
        assert err.max() <= 2e-5 * np.sqrt((ref ** 2).mean()) + 1e-6, err.max()
    assert codec.poll_status() == 0


@pytest.mark.parametrize("cfg,T,n", [(1, 300, 16), (2, 300, 16), (2, 131, 64), (3, 64, 16), (3, 64, 64)])
def test_encode_with_adapters_teacher_forced(cfg, T, n):
    shape, kv, ad = chain(cfg, T, 3, grid_size=n)
    codec, ora = make(shape.d_kv, shape.had_block, shape.scale_group, n, shape.dtype)
    bits = shape.code_bits
    prevK = prevV = None            # the oracle's reconstructions feed both sides (teacher forcing)
    for l in range(shape.n_layers):
        K, V = kv.K[l], kv.V[l]
        Wk, Wv = (ad.Wk[l], ad.Wv[l]) if l else (None, None)
        ok_, ov_ = ora.encode_layer(synth.to_bits(K), synth.to_bits(V), prevK, prevV,
                                    synth.to_bits(Wk) if l else None, synth.to_bits(Wv) if l else None)
        dev = lambda a: None if a is None else (a.to(DEV) if isinstance(a, torch.Tensor)
                                                 else synth.from_bits(a, shape.dtype, DEV))
        Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(dev(K), dev(V), dev(prevK), dev(prevV), dev(Wk), dev(Wv))
        assert codec.poll_status() == 0
        rows_ok, _ = scale_rows_ok(gpu_bits(Ks.view(torch.float16)), ok_["scales"], ok_["scales_exact"])
        check_codes(Kc.cpu().numpy(), ok_, bits, rows_ok)
        # reconstruction: rows whose codes agree (a near-tie flip legitimately moves its whole Hadamard block)
        same_codes = rows_ok & (Kc.cpu().numpy() == ok_["codes"]).all(axis=1)
        check_same_rows(same_codes, shape.d_kv, int((~rows_ok).sum()))
        check_recon(gpu_bits(Kh), ok_["hat_exact"], ok_["hat"], shape.dtype, same_codes)
        # values, teacher-forced inside the layer too: the value phase is given the ORACLE's K_hat
        from paper_2501_19392_b200 import api
        okh = dev(ok_["hat"])
        if l:
            Vc2, Vs2, Vh2 = codec.encode_phase(api.ROLE_VALUE, dev(V), dev(prevV), okh, dev(Wv))
        else:
            Vc2, Vs2, Vh2 = codec.encode_phase(api.ROLE_VALUE, dev(V))
        rows_ok_v, _ = scale_rows_ok(gpu_bits(Vs2.view(torch.float16)), ov_["scales"], ov_["scales_exact"])
        check_codes(Vc2.cpu().numpy(), ov_, bits, rows_ok_v)
        same_codes_v = rows_ok_v & (Vc2.cpu().numpy() == ov_["codes"]).all(axis=1)
        check_same_rows(same_codes_v, shape.d_kv, int((~rows_ok_v).sum()))
        check_recon(gpu_bits(Vh2), ov_["hat_exact"], ov_["hat"], shape.dtype, same_codes_v)
        # the one-call encode agrees with its own phases wherever its K_hat equals the oracle's
        same_k = (gpu_bits(Kh) == ok_["hat"]).all(axis=1)
        if same_k.any():
            assert np.array_equal(Vc.cpu().numpy()[same_k], Vc2.cpu().numpy()[same_k])
            assert np.array_equal(gpu_bits(Vh)[same_k], gpu_bits(Vh2)[same_k])
        # decode on the oracle's codes
        oc = lambda o: (torch.from_numpy(o["codes"]).to(DEV), torch.from_numpy(o["scales"]).view(torch.float16).to(DEV))
        Khd = codec.decode_phase(api.ROLE_KEY, *oc(ok_), dev(prevK) if l else None, None, dev(Wk))
        check_recon(gpu_bits(Khd), ok_["hat_exact"], ok_["hat"], shape.dtype)
        Vhd = codec.decode_phase(api.ROLE_VALUE, *oc(ov_), dev(prevV) if l else None, okh if l else None, dev(Wv))
        check_recon(gpu_bits(Vhd), ov_["hat_exact"], ov_["hat"], shape.dtype)
        # self-consistency: decode(own codes) == encoder's reconstruction, bit for bit
        Kh3, Vh3 = codec.decode(Kc, Ks, Vc, Vs, dev(prevK), dev(prevV), dev(Wk), dev(Wv))
        assert torch.equal(Kh3, Kh) and torch.equal(Vh3, Vh)
        prevK, prevV = ok_["hat"], ov_["hat"]


def _sample_rows(T, seed):
    rng = np.random.default_rng(seed)
    edges = [0, 1, 31, 32, 127, 128, 129, 4735, 4736, 4737, 9471, 9472, T - 129, T - 128, T - 2, T - 1]
    rows = sorted({r for r in edges if 0 <= r < T} | set(rng.integers(0, T, 160).tolist()))
    return np.array(rows, dtype=np.int64)


@pytest.mark.parametrize("T,n", [(32768, 16), (9549, 16), (4737, 64), (2500, 16), (2500, 256)])
def test_full_size_layer_on_sampled_rows(T, n):
    """One layer of the benchmark's launch configuration (all tokens in one call: several waves of
    token blocks through the fused layer kernel, ragged last block) against the oracle on sampled
    rows; rows are independent, so the oracle's result for a row does not depend on the others.
    2500 tokens are less than one wave: most CTAs of the grid have no GEMM tile and only share the
    row work; with 256 grid points the search goes through the second-level lists."""
    shape, kv, ad = chain(2, T, 2, grid_size=n)
    d, dtype, bits = shape.d_kv, shape.dtype, shape.code_bits
    codec, ora = make(d, shape.had_block, shape.scale_group, n, dtype)
    prevK, prevV = kv.K[0], kv.V[0]          # any 16-bit rows serve as the previous layer's reconstruction
    K, V, Wk, Wv = kv.K[1], kv.V[1], ad.Wk[1], ad.Wv[1]
    g = lambda t: t.to(DEV)
    Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(g(K), g(V), g(prevK), g(prevV), g(Wk), g(Wv))
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    rows = _sample_rows(T, seed=T + n)
    b = synth.to_bits
    sel = lambda t: b(t)[rows]
    ok_ = ora.encode_phase(sel(K), [sel(prevK)], b(Wk), None, "k")
    rows_ok, n_bad = scale_rows_ok(gpu_bits(Ks.view(torch.float16))[rows], ok_["scales"], ok_["scales_exact"])
    assert n_bad <= 2
    check_codes(Kc.cpu().numpy()[rows], ok_, bits, rows_ok)
    same = rows_ok & (Kc.cpu().numpy()[rows] == ok_["codes"]).all(axis=1)
    check_same_rows(same, d, int((~rows_ok).sum()))
    check_recon(gpu_bits(Kh)[rows], ok_["hat_exact"], ok_["hat"], dtype, same)
    # values: the oracle is given the library's reconstructed keys of those rows (teacher forcing)
    ov_ = ora.encode_phase(sel(V), [sel(prevV), gpu_bits(Kh)[rows]], b(Wv), None, "v")
    rows_ok_v, n_bad = scale_rows_ok(gpu_bits(Vs.view(torch.float16))[rows], ov_["scales"], ov_["scales_exact"])
    assert n_bad <= 2
    check_codes(Vc.cpu().numpy()[rows], ov_, bits, rows_ok_v)
    same_v = rows_ok_v & (Vc.cpu().numpy()[rows] == ov_["codes"]).all(axis=1)
    check_same_rows(same_v, d, int((~rows_ok_v).sum()))
    check_recon(gpu_bits(Vh)[rows], ov_["hat_exact"], ov_["hat"], dtype, same_v)
    # decode of the library's own codes reproduces the encoder's reconstruction bit for bit, all rows
    Kh2, Vh2 = codec.decode(Kc, Ks, Vc, Vs, g(prevK), g(prevV), g(Wk), g(Wv))
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    assert torch.equal(Kh2, Kh) and torch.equal(Vh2, Vh)
    # the single-phase entry points (separate GEMM and row kernels) agree with the fused kernel, all rows
    from paper_2501_19392_b200 import api
    Kc3, Ks3, Kh3 = codec.encode_phase(api.ROLE_KEY, g(K), g(prevK), None, g(Wk))
    assert torch.equal(Kc3, Kc) and torch.equal(Ks3, Ks) and torch.equal(Kh3, Kh)
    Vc3, Vs3, Vh3 = codec.encode_phase(api.ROLE_VALUE, g(V), g(prevV), Kh, g(Wv))
    assert torch.equal(Vc3, Vc) and torch.equal(Vs3, Vs) and torch.equal(Vh3, Vh)
    # encode without the optional reconstructions (keys kept in the workspace ring) gives the same codes
    Kc4, Ks4, Vc4, Vs4, _, _ = codec.encode(g(K), g(V), g(prevK), g(prevV), g(Wk), g(Wv), want_hat=False)
    torch.cuda.synchronize()
    assert torch.equal(Kc4, Kc) and torch.equal(Vc4, Vc) and torch.equal(Ks4, Ks) and torch.equal(Vs4, Vs)


@pytest.mark.parametrize("d,hd,h,g,n,dtype,T", [
    (256, 64, 256, 256, 16, synth.BF16, 131),     # one 256-wide feature tile per token block, one-warp teams
    (512, 64, 64, 64, 16, synth.F16, 1),          # a single token
    (512, 64, 128, 256, 64, synth.BF16, 259),     # Hadamard block < scale group < row, four candidates per cell
    (1024, 128, 1024, 1024, 256, synth.BF16, 200),  # 256-point grid: second-level search lists, single-buffered GEMM epilogue
    (1024, 128, 512, 1024, 16, synth.F16, 385),   # Hadamard block = one warp's half row, group = whole row
])
def test_fused_layer_shapes_strides_and_bias(d, hd, h, g, n, dtype, T):
    """The fused layer kernel on the other supported shapes, with
    predictor biases and row strides larger than d_kv, against the oracle (teacher-forced)."""
    from paper_2501_19392_b200 import api
    shape = dataclasses.replace(synth.CONFIGS[2], n_kv_heads=d // hd, head_dim=hd, n_tokens=T, n_layers=2,
                                dtype=dtype, had_block=h, scale_group=g, grid_size=n, channel_scales=False)
    kv = synth.kv_chain(shape, seed=77 + d + T)
    ad = synth.random_adapters(shape, seed=78 + d + T, bias=True)
    codec, ora = make(d, h, g, n, dtype)
    bits = shape.code_bits
    b = synth.to_bits
    ld = d + 64                                     # padded rows: ld % 8 == 0, ld > d_kv
    def padded(t):
        buf = torch.zeros((T, ld), dtype=t.dtype, device=DEV)
        buf[:, :d] = t.to(DEV)
        return buf[:, :d]
    K, V, pK, pV = padded(kv.K[1]), padded(kv.V[1]), padded(kv.K[0]), padded(kv.V[0])
    Kh = torch.zeros((T, ld), dtype=codec.torch_dtype, device=DEV)[:, :d]
    Vh = torch.zeros((T, ld), dtype=codec.torch_dtype, device=DEV)[:, :d]
    Wk, Wv, bk, bv = ad.Wk[1].to(DEV), ad.Wv[1].to(DEV), ad.bk[1].to(DEV), ad.bv[1].to(DEV)
    Kc, Ks, Vc, Vs, _, _ = codec.encode(K, V, pK, pV, Wk, Wv, bk, bv, Khat=Kh, Vhat=Vh)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    ok_ = ora.encode_phase(b(kv.K[1]), [b(kv.K[0])], b(ad.Wk[1]), ad.bk[1].numpy(), "k")
    rows_ok, n_bad = scale_rows_ok(gpu_bits(Ks.view(torch.float16)), ok_["scales"], ok_["scales_exact"])
    assert n_bad <= 2
    check_codes(Kc.cpu().numpy(), ok_, bits, rows_ok)
    same = rows_ok & (Kc.cpu().numpy() == ok_["codes"]).all(axis=1)
    check_same_rows(same, d, int((~rows_ok).sum()))
    check_recon(gpu_bits(Kh), ok_["hat_exact"], ok_["hat"], dtype, same)
    ov_ = ora.encode_phase(b(kv.V[1]), [b(kv.V[0]), gpu_bits(Kh)], b(ad.Wv[1]), ad.bv[1].numpy(), "v")
    rows_ok_v, n_bad = scale_rows_ok(gpu_bits(Vs.view(torch.float16)), ov_["scales"], ov_["scales_exact"])
    assert n_bad <= 2
    check_codes(Vc.cpu().numpy(), ov_, bits, rows_ok_v)
    same_v = rows_ok_v & (Vc.cpu().numpy() == ov_["codes"]).all(axis=1)
    check_same_rows(same_v, d, int((~rows_ok_v).sum()))
    check_recon(gpu_bits(Vh), ov_["hat_exact"], ov_["hat"], dtype, same_v)
    # decode of the oracle's codes (fused kernel) against the oracle's reconstruction
    oc = lambda o: (torch.from_numpy(o["codes"]).to(DEV), torch.from_numpy(o["scales"]).view(torch.float16).to(DEV))
    Kd = torch.zeros((T, ld), dtype=codec.torch_dtype, device=DEV)[:, :d]
    Vd = torch.zeros((T, ld), dtype=codec.torch_dtype, device=DEV)[:, :d]
    codec.decode(*oc(ok_), *oc(ov_), pK, pV, Wk, Wv, bk, bv, Khat=Kd, Vhat=Vd)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    check_recon(gpu_bits(Kd), ok_["hat_exact"], ok_["hat"], dtype)
    same_k = (gpu_bits(Kd) == gpu_bits(Kh)).all(axis=1)       # rows whose value predictor saw the same keys
    check_recon(gpu_bits(Vd)[same_k], ov_["hat_exact"][same_k], ov_["hat"][same_k], dtype)
    # own codes decode to the encoder's reconstruction bit for bit; the row padding is untouched
    Kd2, Vd2 = codec.decode(Kc, Ks, Vc, Vs, pK, pV, Wk, Wv, bk, bv)
    assert torch.equal(Kd2, Kh) and torch.equal(Vd2, Vh)
    assert not Kh._base[:, d:].any() and not Vh._base[:, d:].any()


def test_empty_and_argument_errors_on_device():
    from paper_2501_19392_b200 import api
    codec, _ = make(1024, 1024, 1024, 16, synth.BF16)
    e = torch.empty((0, 1024), dtype=torch.bfloat16, device=DEV)
    out = codec.encode(e, e)                       # zero tokens: no launch, no error
    assert out[0].shape[0] == 0 and codec.launch_count() == 0
    x = synth.random_16bit((8, 1024), synth.BF16, 1).to(DEV)
    w = synth.random_16bit((1024, 1024), synth.BF16, 2).to(DEV)
    with pytest.raises(api.AquaKVError) as err:    # adapters must come as a full set
        codec.encode(x, x, x, None, w, None)
    assert err.value.status == -1
    with pytest.raises(api.AquaKVError) as err:    # misaligned row stride
        codec.encode(x[:, :1024], x, Khat=torch.empty((8, 1028), dtype=torch.bfloat16, device=DEV)[:, :1024],
                     Vhat=torch.empty((8, 1028), dtype=torch.bfloat16, device=DEV)[:, :1024])
    assert err.value.status == -3
    wv = synth.random_16bit((1024, 2048), synth.BF16, 3).to(DEV)
    small = torch.empty(1024, dtype=torch.uint8, device=DEV)
    with pytest.raises(api.AquaKVError) as err:    # workspace too small
        codec.encode(x, x, x, x, w, wv, workspace=small)
    assert err.value.status == -4
    assert codec.poll_status() == 0


def test_bulk_decode_shape_on_sampled_rows():
    """Llama-3.3-70B-shaped bulk decode (131072 cached tokens, d_kv 1024, 2-bit codes and fp16 scales
    drawn from seed, adapters on the previous layer's reconstruction), one layer in the launch
    configuration of a real call (all tokens in one fused launch), against the oracle on sampled rows."""
    T = 131072
    shape = dataclasses.replace(synth.CONFIGS[4], n_tokens=T, n_layers=2)
    d, dtype = shape.d_kv, shape.dtype
    codec, ora = make(d, shape.had_block, shape.scale_group, shape.grid_size, dtype)
    cache = synth.random_cache(shape, seed=4001, device=DEV, n_layers=1)
    ad = synth.random_adapters(shape, seed=4002, device=DEV)
    pK = synth.random_16bit((T, d), dtype, 4003, device=DEV)
    pV = synth.random_16bit((T, d), dtype, 4004, device=DEV)
    Kh, Vh = codec.decode(cache.Kcodes[0], cache.Kscales[0], cache.Vcodes[0], cache.Vscales[0], pK, pV,
                          ad.Wk[1], ad.Wv[1])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    rows = _sample_rows(T, seed=4005)
    idx = torch.from_numpy(rows).to(DEV)
    b = synth.to_bits
    kd = ora.decode_phase(cache.Kcodes[0][idx].cpu().numpy(), b(cache.Kscales[0][idx]), [b(pK[idx])],
                          b(ad.Wk[1]), None, "k")
    check_recon(gpu_bits(Kh[idx]), kd["hat_exact"], kd["hat"], dtype)
    vd = ora.decode_phase(cache.Vcodes[0][idx].cpu().numpy(), b(cache.Vscales[0][idx]),
                          [b(pV[idx]), gpu_bits(Kh[idx])], b(ad.Wv[1]), None, "v")
    check_recon(gpu_bits(Vh[idx]), vd["hat_exact"], vd["hat"], dtype)


@pytest.mark.parametrize("T,L", [(512, 6), (512, 28)])
def test_free_running_chain_tracks_the_oracle_chain(T, L):
    """Each side feeds itself through all layers (no teacher forcing; 28 layers is the depth the
    benchmark's chain runs): codes may drift apart after near-ties, so the chains are compared
    statistically: per layer, the library's relative reconstruction error stays within 1 % (relative)
    of the oracle's, and in the first layers most codes still agree."""
    from paper_2501_19392_b200 import chain as chain_mod
    shape, kv, ad = chain(2, T, L)
    d, dtype, bits = shape.d_kv, shape.dtype, shape.code_bits
    codec, ora = make(d, shape.had_block, shape.scale_group, shape.grid_size, dtype)
    g = lambda t: None if t is None else t.to(DEV)
    adg = dataclasses.replace(ad, Wk=[g(w) for w in ad.Wk], Wv=[g(w) for w in ad.Wv])
    cache = chain_mod.CompressedCache.empty(codec, L, T, DEV)
    bufs = chain_mod.PingPong(codec, T, DEV)
    Kg, Vg = [g(t) for t in kv.K], [g(t) for t in kv.V]
    b = synth.to_bits
    pk = pv = None
    worst, least = 0.0, 1.0
    for l in range(L):
        has = l > 0
        cur, prv = l % 2, (l + 1) % 2
        codec.encode(Kg[l], Vg[l], bufs.K[prv] if has else None, bufs.V[prv] if has else None,
                     adg.Wk[l] if has else None, adg.Wv[l] if has else None, None, None,
                     cache.Kcodes[l], cache.Kscales[l], cache.Vcodes[l], cache.Vscales[l], bufs.K[cur], bufs.V[cur])
        ok_, ov_ = ora.encode_layer(b(kv.K[l]), b(kv.V[l]), pk, pv, b(ad.Wk[l]) if has else None,
                                    b(ad.Wv[l]) if has else None)
        pk, pv = ok_["hat"], ov_["hat"]
        for x, hat_gpu, o in ((kv.K[l], bufs.K[cur], ok_), (kv.V[l], bufs.V[cur], ov_)):
            x64 = x.to(torch.float64).numpy()
            err_gpu = ((hat_gpu.to(torch.float64).cpu().numpy() - x64) ** 2).sum() / (x64 ** 2).sum()
            err_ora = ((bits_to_f64(o["hat"], dtype) - x64) ** 2).sum() / (x64 ** 2).sum()
            worst = max(worst, abs(err_gpu - err_ora) / err_ora)
            assert abs(err_gpu - err_ora) <= 0.01 * err_ora, (l, err_gpu, err_ora)
        # a row whose codes differ once keeps drifting (its residuals differ from then on), so the share
        # of equal code bytes falls with depth; it is a requirement only for the first layers
        agree = (cache.Kcodes[l].cpu().numpy() == ok_["codes"]).mean()
        least = min(least, agree)
        if l < 4:
            assert agree > 0.9, (l, agree)
    print("free-running chain, %d layers: largest relative gap of the reconstruction error %.2e, "
          "smallest share of equal key code bytes %.3f" % (L, worst, least))
    assert codec.poll_status() == 0


# ---------------------------------------------------------------------------------------------------
# Degenerate cases of the quantizer (Section 2 "Vector Quantization": group-wise scales, round to the
# nearest grid point), each against the oracle
# ---------------------------------------------------------------------------------------------------

@pytest.mark.parametrize("d,h,g,dtype", [(1024, 1024, 1024, synth.BF16), (512, 64, 64, synth.F16), (512, 128, 256, synth.BF16)])
def test_zero_rows_and_zero_groups(d, h, g, dtype):
    """Rows and scale groups that are exactly zero (what padded batches look like): scale 0, every
    pair takes the code of the grid point nearest the origin, the reconstruction is the prediction.
    Checked without a predictor and with one (zero previous-layer rows give a zero prediction)."""
    n, T = 16, 70
    codec, ora = make(d, h, g, n, dtype)
    X = synth.random_16bit((T, d), dtype, seed=31, std=1.3)
    X[3] = 0                                 # a whole row
    X[T - 1] = 0                             # the last row of the call
    X[10, :g] = 0                            # the first group of a row
    X[11, d - g:] = 0                        # the last group of a row
    Xv = synth.random_16bit((T, d), dtype, seed=32)
    Xv[0] = 0
    b = synth.to_bits
    ok_, ov_ = ora.encode_layer(b(X), b(Xv))
    Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(X.to(DEV), Xv.to(DEV))
    assert codec.poll_status() == 0
    origin = int(np.argmin((codec_grid(n) ** 2).sum(axis=1)))
    for o, c, sc, hat in ((ok_, Kc, Ks, Kh), (ov_, Vc, Vs, Vh)):
        rows_ok, n_bad = scale_rows_ok(gpu_bits(sc.view(torch.float16)), o["scales"], o["scales_exact"])
        assert n_bad <= 1
        check_codes(c.cpu().numpy(), o, 4, rows_ok)
    ks = gpu_bits(Ks.view(torch.float16))
    assert (ks[3] == 0).all() and (ks[T - 1] == 0).all() and ks[10, 0] == 0 and ks[11, -1] == 0
    from util import unpack_codes
    ki = unpack_codes(Kc.cpu().numpy(), 4)
    assert (ki[3] == origin).all() and (ki[T - 1] == origin).all()
    assert (ki[10, :g // 2] == origin).all() and (ki[11, -(g // 2):] == origin).all()
    assert np.array_equal(ki[3], unpack_codes(ok_["codes"], 4)[3])
    for rows_hat, o, r in ((Kh, ok_, 3), (Kh, ok_, T - 1), (Vh, ov_, 0)):       # zero, as the oracle's (+0)
        assert not gpu_bits(rows_hat)[r].any() and np.array_equal(gpu_bits(rows_hat)[r], o["hat"][r])
    # with a predictor: previous-layer rows of zeros predict zero, so zero targets leave a zero residual
    shape = dataclasses.replace(synth.CONFIGS[2], n_kv_heads=d // 64, head_dim=64, n_tokens=T, n_layers=2, dtype=dtype,
                                had_block=h, scale_group=g, grid_size=n, channel_scales=False)
    ad = synth.random_adapters(shape, seed=33)
    pK = synth.random_16bit((T, d), dtype, seed=34)
    pV = synth.random_16bit((T, d), dtype, seed=35)
    pK[3] = 0
    pV[3] = 0
    Xv[3] = 0
    dev = lambda t: t.to(DEV)
    ok2, ov2 = ora.encode_layer(b(X), b(Xv), b(pK), b(pV), b(ad.Wk[1]), b(ad.Wv[1]))
    Kc2, Ks2, Vc2, Vs2, Kh2, Vh2 = codec.encode(dev(X), dev(Xv), dev(pK), dev(pV), dev(ad.Wk[1]), dev(ad.Wv[1]))
    assert codec.poll_status() == 0
    assert (gpu_bits(Ks2.view(torch.float16))[3] == 0).all() and (gpu_bits(Vs2.view(torch.float16))[3] == 0).all()
    assert (unpack_codes(Kc2.cpu().numpy(), 4)[3] == origin).all() and (unpack_codes(Vc2.cpu().numpy(), 4)[3] == origin).all()
    assert np.array_equal(Kc2.cpu().numpy()[3], ok2["codes"][3]) and np.array_equal(Vc2.cpu().numpy()[3], ov2["codes"][3])
    assert not gpu_bits(Kh2)[3].any() and not gpu_bits(Vh2)[3].any()
    Kd, Vd = codec.decode(Kc2, Ks2, Vc2, Vs2, dev(pK), dev(pV), dev(ad.Wk[1]), dev(ad.Wv[1]))
    assert torch.equal(Kd, Kh2) and torch.equal(Vd, Vh2)


def codec_grid(n):
    return synth.lloyd_grid(n, seed=7, n_samples=1 << 14, iters=25).astype(np.float64)


@pytest.mark.parametrize("d,h", [(1024, 1024), (512, 64)])
def test_scale_is_clamped_to_the_largest_fp16(d, h):
    """A bf16 row whose residual RMS exceeds 65504 (finite values only): the stored scale is the
    largest finite fp16 and the codes follow from dividing by it, as in the oracle."""
    n, T, dtype = 16, 40, synth.BF16
    codec, ora = make(d, h, h, n, dtype)
    X = synth.random_16bit((T, d), dtype, seed=41, std=1.5e5)        # RMS about 1.5e5 in every group
    X[1] = synth.random_16bit((d,), dtype, seed=42, std=4.0e4)       # below the clamp
    X[2] = synth.random_16bit((d,), dtype, seed=43, std=3.0e6)       # far above: rotated values of about 45 grid units
    Xv = synth.random_16bit((T, d), dtype, seed=44)
    b = synth.to_bits
    ok_, ov_ = ora.encode_layer(b(X), b(Xv))
    Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(X.to(DEV), Xv.to(DEV))
    assert codec.poll_status() == 0
    ks = gpu_bits(Ks.view(torch.float16))
    assert (ks[0] == 0x7BFF).all() and (ks[2] == 0x7BFF).all() and (ks[1] < 0x7BFF).all()
    rows_ok, n_bad = scale_rows_ok(ks, ok_["scales"], ok_["scales_exact"])
    assert n_bad <= 1
    check_codes(Kc.cpu().numpy(), ok_, 4, rows_ok)
    Kd, Vd = codec.decode(torch.from_numpy(ok_["codes"]).to(DEV), torch.from_numpy(ok_["scales"]).view(torch.float16).to(DEV),
                          torch.from_numpy(ov_["codes"]).to(DEV), torch.from_numpy(ov_["scales"]).view(torch.float16).to(DEV))
    check_recon(gpu_bits(Kd), ok_["hat_exact"], ok_["hat"], dtype)


@pytest.mark.parametrize("d,h,dtype", [(512, 64, synth.F16), (1024, 1024, synth.BF16)])
def test_exact_ties_go_to_the_lowest_index(d, h, dtype):
    """Inputs built so that the rotated, normalised values are small dyadic numbers that land exactly
    on Voronoi boundaries of a symmetric 4 x 4 grid (margin 0): both sides must pick the lowest index,
    so every code is compared with the oracle's, ties included."""
    from paper_2501_19392_b200 import api
    from util import unpack_codes
    side = np.array([-1.5, -0.5, 0.5, 1.5])
    grid = np.array([[x, y] for x in side for y in side], dtype=np.float32)       # sorted lexicographically
    sk, sv = synth.hadamard_signs(d, 11), synth.hadamard_signs(d, 12)
    codec, ora = api.Codec(d, h, h, grid, dtype, sk, sv), oracle.Oracle(d, h, h, grid, dtype, sk, sv)
    rng = np.random.default_rng(51)
    T = 64
    H = np.array([[1.0]])
    while H.shape[0] < h:
        H = np.block([[H, H], [H, -H]])
    X = np.zeros((T, d))
    for t in range(T):
        for blk in range(d // h):
            # rotated target with mean square exactly 1: a quarter zeros, half +-1, an eighth +-2, an eighth zeros
            y = np.concatenate([np.zeros(h // 4), rng.choice([-1.0, 1.0], h // 2), rng.choice([-2.0, 2.0], h // 8),
                                np.zeros(h // 8)])
            y = y[rng.permutation(h)]
            s = 2.0 ** rng.integers(-3, 3)                       # the group's scale: a power of two
            u = s * (H @ y) / np.sqrt(h)                         # H / sqrt(h) is orthonormal and symmetric
            X[t, blk * h:(blk + 1) * h] = u * sk[blk * h:(blk + 1) * h]
    Xt = torch.from_numpy(X).to(synth.torch_dtype(dtype))
    assert np.array_equal(Xt.to(torch.float64).numpy(), X), "the construction must be exact in the 16-bit type"
    Xv = synth.random_16bit((T, d), dtype, seed=52)
    b = synth.to_bits
    ok_, ov_ = ora.encode_layer(b(Xt), b(Xv))
    assert (ok_["margins"] == 0).mean() > 0.3, "the construction must produce exact ties"
    Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(Xt.to(DEV), Xv.to(DEV))
    assert codec.poll_status() == 0
    assert np.array_equal(gpu_bits(Ks.view(torch.float16)), ok_["scales"])
    assert np.array_equal(unpack_codes(Kc.cpu().numpy(), 4), unpack_codes(ok_["codes"], 4))
    assert np.array_equal(gpu_bits(Kh), ok_["hat"])              # every step of this case is exact


def test_a_bounded_wait_that_runs_out_is_reported_and_leaves_the_context_usable():
    """One warp waits 1 ms on a barrier that nothing arrives on: the kernel returns, the status word
    reads AQUAKV_ERR_TIMEOUT once, and an ordinary decode on the same context then succeeds."""
    codec, ora = make(1024, 1024, 1024, 16, synth.BF16)
    assert codec.poll_status() == 0
    codec.selftest_bounded_wait(1_000_000)
    assert codec.poll_status() == -6              # AQUAKV_ERR_TIMEOUT
    assert codec.poll_status() == 0               # cleared by the poll
    shape = dataclasses.replace(synth.CONFIGS[4], n_tokens=200, n_layers=2)
    cache = synth.random_cache(shape, seed=61, n_layers=1)
    ad = synth.random_adapters(shape, seed=62)
    pK = synth.random_16bit((200, 1024), synth.BF16, seed=63)
    pV = synth.random_16bit((200, 1024), synth.BF16, seed=64)
    g = lambda t: t.to(DEV)
    Kh, Vh = codec.decode(g(cache.Kcodes[0]), g(cache.Kscales[0]), g(cache.Vcodes[0]), g(cache.Vscales[0]),
                          g(pK), g(pV), g(ad.Wk[1]), g(ad.Wv[1]))
    assert codec.poll_status() == 0
    b = synth.to_bits
    kd = ora.decode_phase(cache.Kcodes[0].numpy(), b(cache.Kscales[0]), [b(pK)], b(ad.Wk[1]), None, "k")
    check_recon(gpu_bits(Kh), kd["hat_exact"], kd["hat"], synth.BF16)
