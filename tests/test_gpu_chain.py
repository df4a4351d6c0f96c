"""aquakv_encode_chain / aquakv_decode_chain (all layers of a small call in one launch; Algorithm 4's
loop over layers around Algorithm 2 / Algorithm 3) against the CPU oracle: teacher-forced layer by
layer (the chain is given the oracle's reconstruction of the previous layer), free-running over the
whole depth (statistically, since the two chains drift apart after near-ties), and the chain decoder
against the chain encoder bit for bit."""
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


def make(shape):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(shape.grid_size, seed=7, n_samples=1 << 14, iters=25)
    sk, sv = synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12)
    args = (shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype, sk, sv)
    return api.Codec(*args), oracle.Oracle(*args)


def buffers(codec, L, T):
    mk = lambda cols, dt: [torch.empty((T, cols), dtype=dt, device=DEV) for _ in range(L)]
    return (mk(codec.code_bytes, torch.uint8), mk(codec.n_groups, torch.float16),
            mk(codec.code_bytes, torch.uint8), mk(codec.n_groups, torch.float16),
            mk(codec.d, codec.torch_dtype), mk(codec.d, codec.torch_dtype))


CASES = [
    # config, tokens, layers, grid points
    (3, 64, 32, 16),      # Llama-3.1-8B-shaped decode step, 2 bits per value
    (3, 64, 32, 64),      # the same at 3 bits per value
    (1, 1024, 2, 16),     # Llama-3.2-1B-shaped round trip: d_kv 512, fp16, Hadamard block 64
    (3, 37, 3, 256),      # ragged 16-token tiles, 4 bits
    (1, 1, 3, 16),        # a single token
    (3, 600, 3, 16),      # d_kv 1024 with more rows than four-warp teams at once: one warp per row
]


@pytest.mark.parametrize("cfg,T,L,n", CASES)
def test_chain_free_running_and_decode_reproduces_encode(cfg, T, L, n):
    shape = dataclasses.replace(synth.CONFIGS[cfg], n_tokens=T, n_layers=L, grid_size=n)
    codec, ora = make(shape)
    kv = synth.kv_chain(shape, seed=7000 + cfg)
    ad = synth.random_adapters(shape, seed=7100 + cfg)
    g = lambda t: None if t is None else t.to(DEV)
    K, V = [g(t) for t in kv.K], [g(t) for t in kv.V]
    Wk, Wv = [g(w) for w in ad.Wk], [g(w) for w in ad.Wv]
    Kc, Ks, Vc, Vs, Kh, Vh = buffers(codec, L, T)
    codec.encode_chain(K, V, Wk, Wv, Kc, Ks, Vc, Vs, Khat=Kh, Vhat=Vh)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    # layer 0 has no predictor: codes against the oracle exactly as for the per-layer call
    b = synth.to_bits
    pk = pv = None
    worst = 0.0
    for l in range(L):
        ok_, ov_ = ora.encode_layer(b(kv.K[l]), b(kv.V[l]), pk, pv, b(ad.Wk[l]) if l else None, b(ad.Wv[l]) if l else None)
        pk, pv = ok_["hat"], ov_["hat"]
        if l == 0:
            rows_ok, _ = scale_rows_ok(gpu_bits(Ks[0].view(torch.float16)), ok_["scales"], ok_["scales_exact"])
            check_codes(Kc[0].cpu().numpy(), ok_, shape.code_bits, rows_ok)
        if T >= 64:    # a statistical statement needs enough values
            for x, hat_gpu, o in ((kv.K[l], Kh[l], ok_), (kv.V[l], Vh[l], ov_)):
                x64 = x.to(torch.float64).numpy()
                err_gpu = ((hat_gpu.to(torch.float64).cpu().numpy() - x64) ** 2).sum() / (x64 ** 2).sum()
                err_ora = ((bits_to_f64(o["hat"], shape.dtype) - x64) ** 2).sum() / (x64 ** 2).sum()
                # 64 tokens x 1024 values: the sampling noise of the ratio is a few per cent by itself
                band = 0.01 if T >= 512 else 0.05
                worst = max(worst, abs(err_gpu - err_ora) / err_ora)
                assert abs(err_gpu - err_ora) <= band * err_ora, (l, err_gpu, err_ora)
    print("chain of %d layers x %d tokens: largest relative gap of the reconstruction error %.2e" % (L, T, worst))
    # the chain decoder reproduces the chain encoder's reconstructions bit for bit, from the codes alone
    _, _, _, _, Kd, Vd = buffers(codec, L, T)
    codec.decode_chain(Kc, Ks, Vc, Vs, Wk, Wv, Khat=Kd, Vhat=Vd)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    for l in range(L):
        assert torch.equal(Kd[l], Kh[l]) and torch.equal(Vd[l], Vh[l]), l
    # without the optional outputs (reconstructions kept in the workspace) the codes are the same
    Kc2, Ks2, Vc2, Vs2, _, _ = buffers(codec, L, T)
    codec.encode_chain(K, V, Wk, Wv, Kc2, Ks2, Vc2, Vs2)
    torch.cuda.synchronize()
    for l in range(L):
        assert torch.equal(Kc2[l], Kc[l]) and torch.equal(Vc2[l], Vc[l]) and torch.equal(Ks2[l], Ks[l]) and torch.equal(Vs2[l], Vs[l])


@pytest.mark.parametrize("cfg,T,n,bias", [(3, 64, 16, False), (3, 64, 64, True), (1, 300, 16, False), (2, 200, 16, True),
                                          (2, 700, 16, False)])     # the last: d_kv 1024 on the one-warp-per-row routines
def test_chain_teacher_forced_layers(cfg, T, n, bias):
    """A chain of ONE predicted layer started from the oracle's reconstruction of the layer before it:
    codes, scales and reconstructions against the oracle under the rules of the per-layer tests; then
    the value phase is checked with the oracle given the library's own reconstructed keys."""
    L = 3
    shape = dataclasses.replace(synth.CONFIGS[cfg], n_tokens=T, n_layers=L, grid_size=n, channel_scales=False)
    codec, ora = make(shape)
    d, dtype, bits = shape.d_kv, shape.dtype, shape.code_bits
    kv = synth.kv_chain(shape, seed=7200 + cfg)
    ad = synth.random_adapters(shape, seed=7300 + cfg, bias=bias)
    b = synth.to_bits
    dev = lambda a: synth.from_bits(a, dtype, DEV) if isinstance(a, np.ndarray) else a.to(DEV)
    pk = pv = None
    for l in range(L):
        has = l > 0
        bk = ad.bk[l].numpy() if has and bias else None
        bv = ad.bv[l].numpy() if has and bias else None
        ok_ = ora.encode_phase(b(kv.K[l]), [pk], b(ad.Wk[l]) if has else None, bk, "k")
        Kc, Ks, Vc, Vs, Kh, Vh = buffers(codec, 1, T)
        codec.encode_chain([dev(kv.K[l])], [dev(kv.V[l])], [dev(ad.Wk[l]) if has else None], [dev(ad.Wv[l]) if has else None],
                           Kc, Ks, Vc, Vs, bk=[dev(ad.bk[l])] if has and bias else None,
                           bv=[dev(ad.bv[l])] if has and bias else None, Khat=Kh, Vhat=Vh,
                           Khat_init=dev(pk) if has else None, Vhat_init=dev(pv) if has else None)
        torch.cuda.synchronize()
        assert codec.poll_status() == 0
        rows_ok, n_bad = scale_rows_ok(gpu_bits(Ks[0].view(torch.float16)), ok_["scales"], ok_["scales_exact"])
        assert n_bad <= 2
        check_codes(Kc[0].cpu().numpy(), ok_, bits, rows_ok)
        same = rows_ok & (Kc[0].cpu().numpy() == ok_["codes"]).all(axis=1)
        check_same_rows(same, d, int((~rows_ok).sum()))
        check_recon(gpu_bits(Kh[0]), ok_["hat_exact"], ok_["hat"], dtype, same)
        # values: the oracle is given the library's reconstructed keys (teacher forcing inside the layer)
        ov_ = ora.encode_phase(b(kv.V[l]), [pv, gpu_bits(Kh[0])], b(ad.Wv[l]) if has else None, bv, "v")
        rows_ok_v, n_bad = scale_rows_ok(gpu_bits(Vs[0].view(torch.float16)), ov_["scales"], ov_["scales_exact"])
        assert n_bad <= 2
        check_codes(Vc[0].cpu().numpy(), ov_, bits, rows_ok_v)
        same_v = rows_ok_v & (Vc[0].cpu().numpy() == ov_["codes"]).all(axis=1)
        check_same_rows(same_v, d, int((~rows_ok_v).sum()))
        check_recon(gpu_bits(Vh[0]), ov_["hat_exact"], ov_["hat"], dtype, same_v)
        # decode chain of the ORACLE's codes for this layer against the oracle's reconstruction
        ovo = ora.encode_phase(b(kv.V[l]), [pv, ok_["hat"]], b(ad.Wv[l]) if has else None, bv, "v")
        t = lambda o: ([torch.from_numpy(o["codes"]).to(DEV)], [torch.from_numpy(o["scales"]).view(torch.float16).to(DEV)])
        _, _, _, _, Kd, Vd = buffers(codec, 1, T)
        codec.decode_chain(*t(ok_), *t(ovo), [dev(ad.Wk[l]) if has else None], [dev(ad.Wv[l]) if has else None],
                           bk=[dev(ad.bk[l])] if has and bias else None, bv=[dev(ad.bv[l])] if has and bias else None,
                           Khat=Kd, Vhat=Vd, Khat_init=dev(pk) if has else None, Vhat_init=dev(pv) if has else None)
        torch.cuda.synchronize()
        assert codec.poll_status() == 0
        check_recon(gpu_bits(Kd[0]), ok_["hat_exact"], ok_["hat"], dtype)
        same_k = (gpu_bits(Kd[0]) == ok_["hat"]).all(axis=1)     # rows whose value predictor saw the oracle's keys
        check_recon(gpu_bits(Vd[0])[same_k], ovo["hat_exact"][same_k], ovo["hat"][same_k], dtype)
        pk, pv = ok_["hat"], ovo["hat"]


def test_chain_argument_errors():
    from paper_2501_19392_b200 import api
    shape = dataclasses.replace(synth.CONFIGS[3], n_tokens=8, n_layers=2)
    codec, _ = make(shape)
    T, d = 8, 1024
    x = synth.random_16bit((T, d), synth.BF16, 1).to(DEV)
    w = synth.random_16bit((d, d), synth.BF16, 2).to(DEV)
    wv = synth.random_16bit((d, 2 * d), synth.BF16, 3).to(DEV)
    Kc, Ks, Vc, Vs, Kh, Vh = buffers(codec, 2, T)
    with pytest.raises(api.AquaKVError) as e:       # a predictor on layer 0 needs the reconstruction before it
        codec.encode_chain([x, x], [x, x], [w, w], [wv, wv], Kc, Ks, Vc, Vs)
    assert e.value.status == -1
    with pytest.raises(api.AquaKVError) as e:       # adapters come in pairs
        codec.encode_chain([x, x], [x, x], [None, w], [None, None], Kc, Ks, Vc, Vs)
    assert e.value.status == -1
    with pytest.raises(api.AquaKVError) as e:       # workspace too small
        codec.encode_chain([x, x], [x, x], [None, w], [None, wv], Kc, Ks, Vc, Vs,
                           workspace=torch.empty(1024, dtype=torch.uint8, device=DEV))
    assert e.value.status == -4
    big = torch.empty((api.CHAIN_MAX_TOKENS + 1, d), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(api.AquaKVError) as e:       # a large call needs every layer's output buffers
        codec.encode_chain([big], [big], [None], [None], *[[t] for t in (Kc[0], Ks[0], Vc[0], Vs[0])],
                           workspace=torch.empty(1024, dtype=torch.uint8, device=DEV))
    assert e.value.status == (-1 if d == 1024 else -7)
    assert codec.launch_count() == 0 and codec.poll_status() == 0


@pytest.mark.parametrize("T,L,n,first_pred", [(5000, 5, 16, False), (2304, 27, 16, True), (9549, 3, 64, False)])
def test_large_calls_run_several_layers_per_launch_and_equal_the_per_layer_calls(T, L, n, first_pred):
    """Beyond 2048 tokens the chain entry points run the layer kernel on up to 24 layers per launch; the result
    must be the per-layer calls' bit for bit (27 layers: two launches; first_pred: layer 0 has a predictor and
    reads Khat_init / Vhat_init)."""
    from paper_2501_19392_b200 import api, chain
    shape = dataclasses.replace(synth.CONFIGS[2], n_tokens=T, n_layers=L, grid_size=n)
    codec, _ = make(shape)
    kv = synth.kv_chain(shape, seed=8800 + L, device=DEV)
    ad = synth.random_adapters(shape, seed=8900 + L, device=DEV)
    Wk, Wv = list(ad.Wk), list(ad.Wv)
    init_k = init_v = None
    if first_pred:
        Wk[0], Wv[0] = ad.Wk[1], ad.Wv[1]
        init_k = synth.random_16bit((T, shape.d_kv), shape.dtype, 1, device=DEV)
        init_v = synth.random_16bit((T, shape.d_kv), shape.dtype, 2, device=DEV)
    ad = dataclasses.replace(ad, Wk=Wk, Wv=Wv)
    # per-layer reference
    ref = chain.CompressedCache.empty(codec, L, T, DEV)
    bufs = chain.PingPong(codec, T, DEV)
    hats = []
    for l in range(L):
        cur, prv = l % 2, (l + 1) % 2
        has = Wk[l] is not None
        pk = (init_k if l == 0 else bufs.K[prv]) if has else None
        pv = (init_v if l == 0 else bufs.V[prv]) if has else None
        codec.encode(kv.K[l], kv.V[l], pk, pv, Wk[l], Wv[l], None, None, ref.Kcodes[l], ref.Kscales[l], ref.Vcodes[l],
                     ref.Vscales[l], bufs.K[cur], bufs.V[cur])
        hats.append((bufs.K[cur].clone(), bufs.V[cur].clone()))
    before = codec.launch_count()
    got = chain.CompressedCache.empty(codec, L, T, DEV)
    bufs2 = chain.PingPong(codec, T, DEV)
    codec.encode_chain(kv.K, kv.V, Wk, Wv, got.Kcodes, got.Kscales, got.Vcodes, got.Vscales, None, None,
                       [bufs2.K[l % 2] for l in range(L)], [bufs2.V[l % 2] for l in range(L)], init_k, init_v)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    n_pred = sum(w is not None for w in Wk)
    assert codec.launch_count() - before == 2 * (L - n_pred) + (n_pred + 23) // 24       # row kernels of layer 0 + batches
    for l in range(L):
        assert torch.equal(got.Kcodes[l], ref.Kcodes[l]) and torch.equal(got.Vcodes[l], ref.Vcodes[l]), l
        assert torch.equal(got.Kscales[l], ref.Kscales[l]) and torch.equal(got.Vscales[l], ref.Vscales[l]), l
    assert torch.equal(bufs2.K[(L - 1) % 2], hats[-1][0]) and torch.equal(bufs2.V[(L - 1) % 2], hats[-1][1])
    assert torch.equal(bufs2.K[(L - 2) % 2], hats[-2][0]) and torch.equal(bufs2.V[(L - 2) % 2], hats[-2][1])
    # decode through the same entry point reproduces the reconstructions
    bufs3 = chain.PingPong(codec, T, DEV)
    codec.decode_chain(got.Kcodes, got.Kscales, got.Vcodes, got.Vscales, Wk, Wv, None, None,
                       [bufs3.K[l % 2] for l in range(L)], [bufs3.V[l % 2] for l in range(L)], init_k, init_v)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    assert torch.equal(bufs3.K[(L - 1) % 2], hats[-1][0]) and torch.equal(bufs3.V[(L - 1) % 2], hats[-1][1])
    assert torch.equal(bufs3.K[(L - 2) % 2], hats[-2][0]) and torch.equal(bufs3.V[(L - 2) % 2], hats[-2][1])
