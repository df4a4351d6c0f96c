"""Second workload: Qwen-2.5-shaped caches (d_kv 256 / 512, scale group = Hadamard block = d_kv, first
layer left in 16 bits: the setting of the paper's appendix tables) compressed only for the tokens a
pruning policy keeps (Section 4.3, "Compatibility with Pruning").

The oracle side is the codec oracle applied to the selected rows (selection is indexing, nothing of
the method's arithmetic); the GPU side gathers with aquakv_gather_rows and encodes the compact rows.
Teacher-forced per layer like every encode parity test: both sides are given the oracle's
reconstruction of the previous layer."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2501_19392_b200 import synth
from parity import check_codes, check_recon, check_same_rows, gpu_bits, scale_rows_ok

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make(shape):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(shape.grid_size, seed=7, n_samples=1 << 14, iters=25)
    sk, sv = synth.hadamard_signs(shape.d_kv, 11), synth.hadamard_signs(shape.d_kv, 12)
    args = (shape.d_kv, shape.had_block, shape.scale_group, grid, shape.dtype, sk, sv)
    return api.Codec(*args), oracle.Oracle(*args)


def test_gather_rows_is_an_exact_row_copy_and_reports_bad_indices():
    from paper_2501_19392_b200 import api
    shape = dataclasses.replace(synth.CONFIGS[6], n_tokens=1000, n_layers=1)
    codec, _ = make(shape)
    d = shape.d_kv
    src = synth.random_16bit((1000, d + 8), shape.dtype, 1, device=DEV)[:, :d]       # rows with padding
    idx = torch.from_numpy(synth.kept_tokens(1000, 0.2, seed=3)).to(DEV)
    out = codec.gather_rows(src, idx)
    assert out.shape == (200, d) and torch.equal(out, src[idx])
    # identity copy into a strided destination, empty selection, repeated and unsorted indices
    dst = torch.zeros((1000, d + 16), dtype=src.dtype, device=DEV)
    codec.gather_rows(src, None, dst[:, :d])
    assert torch.equal(dst[:, :d], src) and not dst[:, d:].any()
    assert codec.gather_rows(src, idx[:0]).shape == (0, d)
    odd = torch.tensor([999, 0, 0, 512, 7], dtype=torch.int64, device=DEV)
    assert torch.equal(codec.gather_rows(src, odd), src[odd])
    assert codec.poll_status() == 0
    bad = torch.tensor([3, 1000, -1, 5], dtype=torch.int64, device=DEV)
    got = codec.gather_rows(src, bad)
    assert codec.poll_status() == -1 and codec.poll_status() == 0
    assert torch.equal(got[0], src[3]) and torch.equal(got[3], src[5]) and not got[1].any() and not got[2].any()
    with pytest.raises(api.AquaKVError):
        codec.gather_rows(src[:, 1:], idx)                 # misaligned rows


@pytest.mark.parametrize("cfg,T,L,n", [(6, 4000, 3, 16), (7, 3000, 3, 64)])
def test_kept_token_encode_matches_the_oracle_on_the_kept_rows(cfg, T, L, n):
    from paper_2501_19392_b200 import api, chain
    shape = dataclasses.replace(synth.CONFIGS[cfg], n_tokens=T, n_layers=L, grid_size=n)
    codec, ora = make(shape)
    kv = synth.kv_chain(shape, seed=8000 + cfg)
    ad = synth.random_adapters(shape, seed=8100 + cfg)
    keep = synth.kept_tokens(T, 0.2, seed=8200 + cfg)
    n_keep = len(keep)
    idx = torch.from_numpy(keep).to(DEV)
    bits = shape.code_bits
    up = lambda a: None if a is None else (a.to(DEV) if isinstance(a, torch.Tensor)
                                           else synth.from_bits(a, shape.dtype, DEV))
    # first layer in 16 bits: the kept rows themselves are the next layer's predictor inputs
    prevK, prevV = synth.to_bits(kv.K[0])[keep], synth.to_bits(kv.V[0])[keep]
    gK0 = codec.gather_rows(up(kv.K[0]), idx)
    assert np.array_equal(gpu_bits(gK0), prevK)
    for l in range(1, L):
        Kb, Vb = synth.to_bits(kv.K[l])[keep], synth.to_bits(kv.V[l])[keep]
        ok_, ov_ = ora.encode_layer(Kb, Vb, prevK, prevV, synth.to_bits(ad.Wk[l]), synth.to_bits(ad.Wv[l]))
        Kg, Vg = codec.gather_rows(up(kv.K[l]), idx), codec.gather_rows(up(kv.V[l]), idx)
        Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(Kg, Vg, up(prevK), up(prevV), up(ad.Wk[l]), up(ad.Wv[l]))
        assert codec.poll_status() == 0
        rows_ok, _ = scale_rows_ok(gpu_bits(Ks.view(torch.float16)), ok_["scales"], ok_["scales_exact"])
        check_codes(Kc.cpu().numpy(), ok_, bits, rows_ok)
        same = rows_ok & (Kc.cpu().numpy() == ok_["codes"]).all(axis=1)
        check_same_rows(same, shape.d_kv, int((~rows_ok).sum()))
        check_recon(gpu_bits(Kh), ok_["hat_exact"], ok_["hat"], shape.dtype, same)
        # values with the oracle's reconstructed keys
        Vc2, Vs2, Vh2 = codec.encode_phase(api.ROLE_VALUE, Vg, up(prevV), up(ok_["hat"]), up(ad.Wv[l]))
        rows_ok_v, _ = scale_rows_ok(gpu_bits(Vs2.view(torch.float16)), ov_["scales"], ov_["scales_exact"])
        check_codes(Vc2.cpu().numpy(), ov_, bits, rows_ok_v)
        same_v = rows_ok_v & (Vc2.cpu().numpy() == ov_["codes"]).all(axis=1)
        check_same_rows(same_v, shape.d_kv, int((~rows_ok_v).sum()))
        check_recon(gpu_bits(Vh2), ov_["hat_exact"], ov_["hat"], shape.dtype, same_v)
        prevK, prevV = ok_["hat"], ov_["hat"]
    # the chain helper does the same gathers and calls: its cache equals per-layer calls on its own buffers
    cache = chain.CompressedCache.empty(codec, L, n_keep, DEV)
    bufs = chain.PingPong(codec, n_keep, DEV)
    sk, sv = torch.empty_like(bufs.K[0]), torch.empty_like(bufs.V[0])
    chain.encode_chain_kept(codec, [up(t) for t in kv.K], [up(t) for t in kv.V], idx,
                            dataclasses.replace(ad, Wk=[up(w) for w in ad.Wk], Wv=[up(w) for w in ad.Wv]),
                            cache, bufs, sk, sv, first_layer_16bit=True)
    Kh_prev, Vh_prev = codec.gather_rows(up(kv.K[0]), idx), codec.gather_rows(up(kv.V[0]), idx)
    for l in range(1, L):
        Kg, Vg = codec.gather_rows(up(kv.K[l]), idx), codec.gather_rows(up(kv.V[l]), idx)
        Kc, Ks, Vc, Vs, Kh_prev, Vh_prev = codec.encode(Kg, Vg, Kh_prev, Vh_prev, up(ad.Wk[l]), up(ad.Wv[l]))
        assert torch.equal(Kc, cache.Kcodes[l]) and torch.equal(Vc, cache.Vcodes[l])
        assert torch.equal(Ks, cache.Kscales[l]) and torch.equal(Vs, cache.Vscales[l])
    assert torch.equal(Kh_prev, bufs.K[(L - 1) % 2]) and torch.equal(Vh_prev, bufs.V[(L - 1) % 2])
    assert codec.poll_status() == 0


def test_kept_token_encode_at_the_benchmark_size_on_sampled_rows():
    # the launch configuration bench.py times for config 6: 26214 kept tokens of a 131072-token context, d_kv 256;
    # rows are independent, so the oracle checks a sample of them
    from paper_2501_19392_b200 import api
    shape = dataclasses.replace(synth.CONFIGS[6], n_layers=2)
    codec, ora = make(shape)
    kv = synth.kv_chain(shape, seed=6001, device=DEV)
    ad = synth.random_adapters(shape, seed=6002, device=DEV)
    keep = synth.kept_tokens(shape.n_tokens, 0.2, seed=6003)
    idx = torch.from_numpy(keep).to(DEV)
    K0, V0 = codec.gather_rows(kv.K[0], idx), codec.gather_rows(kv.V[0], idx)          # first layer in 16 bits
    K1, V1 = codec.gather_rows(kv.K[1], idx), codec.gather_rows(kv.V[1], idx)
    Kc, Ks, Vc, Vs, Kh, Vh = codec.encode(K1, V1, K0, V0, ad.Wk[1], ad.Wv[1])
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    assert Kc.shape[0] == len(keep) == 26214
    rng = np.random.default_rng(5)
    sample = np.sort(np.concatenate([rng.choice(len(keep), 1500, replace=False), [0, len(keep) - 1]]))
    sel = torch.from_numpy(sample).to(DEV)
    b = lambda t: synth.to_bits(t[sel].cpu())
    src = lambda t: synth.to_bits(t[idx[sel]].cpu())
    assert np.array_equal(b(K1), src(kv.K[1])) and np.array_equal(b(V0), src(kv.V[0]))
    ok_ = ora.encode_phase(src(kv.K[1]), [src(kv.K[0])], synth.to_bits(ad.Wk[1].cpu()), None, "k")
    rows_ok, _ = scale_rows_ok(gpu_bits(Ks[sel].view(torch.float16)), ok_["scales"], ok_["scales_exact"])
    check_codes(Kc[sel].cpu().numpy(), ok_, shape.code_bits, rows_ok)
    same = rows_ok & (Kc[sel].cpu().numpy() == ok_["codes"]).all(axis=1)
    check_same_rows(same, shape.d_kv, int((~rows_ok).sum()))
    check_recon(b(Kh), ok_["hat_exact"], ok_["hat"], shape.dtype, same)
    # values: the oracle is given the GPU's reconstructed keys of the sampled rows (teacher forcing inside the layer)
    ov_ = ora.encode_phase(src(kv.V[1]), [src(kv.V[0]), b(Kh)], synth.to_bits(ad.Wv[1].cpu()), None, "v")
    rows_ok_v, _ = scale_rows_ok(gpu_bits(Vs[sel].view(torch.float16)), ov_["scales"], ov_["scales_exact"])
    check_codes(Vc[sel].cpu().numpy(), ov_, shape.code_bits, rows_ok_v)
    same_v = rows_ok_v & (Vc[sel].cpu().numpy() == ov_["codes"]).all(axis=1)
    check_same_rows(same_v, shape.d_kv, int((~rows_ok_v).sum()))
    check_recon(b(Vh), ov_["hat_exact"], ov_["hat"], shape.dtype, same_v)
