"""aquakv_decode_noalloc, the decode entry point for callers that are not allowed to allocate device
memory (plugins handed only their input/output buffers, servers with a frozen memory pool,
real-time loops that must stay clear of the allocator).  It keeps the fp32 prediction in a fixed
4 MiB array inside the library instead of a caller workspace, so its results must be those of
aquakv_decode bit for bit -- also on a second call, which finds the first call's leftovers in the
shared array -- and it must refuse more tokens than the array holds.

Collected last on purpose: a failure here cannot hide a failure of any other test under `-x`.
"""
import dataclasses

import pytest
import torch

from paper_2501_19392_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _case(codec_mod, d, hd, dtype, n, T, seed):
    shape = dataclasses.replace(synth.CONFIGS[4], n_kv_heads=d // hd, head_dim=hd, n_tokens=T, n_layers=2,
                                dtype=dtype, had_block=d, scale_group=d, grid_size=n)
    cache = synth.random_cache(shape, seed=seed, n_layers=1)
    ad = synth.random_adapters(shape, seed=seed + 1)
    prevK = synth.random_16bit((T, d), dtype, seed=seed + 2)
    prevV = synth.random_16bit((T, d), dtype, seed=seed + 3)
    g = lambda t: t.to(DEV)
    return (g(cache.Kcodes[0]), g(cache.Kscales[0]), g(cache.Vcodes[0]), g(cache.Vscales[0]),
            g(prevK), g(prevV), g(ad.Wk[1]), g(ad.Wv[1]))


@pytest.mark.parametrize("d,hd,dtype,n", [(1024, 128, synth.BF16, 16), (512, 64, synth.F16, 64)])
def test_noalloc_decode_equals_decode_on_two_calls_in_a_row(d, hd, dtype, n):
    from paper_2501_19392_b200 import api
    grid = synth.lloyd_grid(n, seed=7, n_samples=1 << 14, iters=25)
    codec = api.Codec(d, d, d, grid, dtype, synth.hadamard_signs(d, 11), synth.hadamard_signs(d, 12))
    # first call: the maximum size, so the whole shared array is written
    a1 = _case(api, d, hd, dtype, n, api.NOALLOC_MAX_TOKENS, seed=9100)
    ref_k1, ref_v1 = codec.decode(*a1)
    k1 = torch.empty_like(ref_k1)
    v1 = torch.empty_like(ref_v1)
    codec.decode_noalloc(*a1, Khat=k1, Vhat=v1)
    # second call straight after it, other inputs, ragged size: must not see the first call's rows
    a2 = _case(api, d, hd, dtype, n, 333, seed=9200)
    k2 = torch.empty((333, d), dtype=codec.torch_dtype, device=DEV)
    v2 = torch.empty_like(k2)
    codec.decode_noalloc(*a2, Khat=k2, Vhat=v2)
    torch.cuda.synchronize()
    assert codec.poll_status() == 0
    ref_k2, ref_v2 = codec.decode(*a2)
    torch.cuda.synchronize()
    assert torch.equal(k1, ref_k1) and torch.equal(v1, ref_v1)
    assert torch.equal(k2, ref_k2) and torch.equal(v2, ref_v2)
    # layer-0 form (no predictor, the array is not touched at all)
    k0, v0 = codec.decode_noalloc(*a2[:4])
    r0k, r0v = codec.decode(*a2[:4])
    assert torch.equal(k0, r0k) and torch.equal(v0, r0v)


def test_noalloc_decode_rejects_more_tokens_than_its_array_holds():
    from paper_2501_19392_b200 import api
    d = 1024
    grid = synth.lloyd_grid(16, seed=7, n_samples=1 << 14, iters=25)
    codec = api.Codec(d, d, d, grid, synth.BF16, synth.hadamard_signs(d, 11), synth.hadamard_signs(d, 12))
    a = _case(api, d, 128, synth.BF16, 16, api.NOALLOC_MAX_TOKENS + 1, seed=9300)
    with pytest.raises(api.AquaKVError) as e:
        codec.decode_noalloc(*a)
    assert e.value.status == -7 and "scratch" in api.status_string(-7)
