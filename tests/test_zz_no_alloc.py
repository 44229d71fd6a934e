"""freqkv_compress_noalloc, the entry point for callers that cannot allocate device memory
(code under a lock an allocation could deadlock against, frozen memory budgets, frameworks that
own all device memory): its result must equal that of freqkv_compress on the same input, call
after call, although every call reuses the same fixed work arrays inside the library; it must
match the CPU oracle like every other path; and it must leave the amount of free device memory
exactly as it found it.  Collected last on purpose, so that a run that
stops at the first failure has already run every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2505_00570_b200 import binding as fk
from paper_2505_00570_b200 import synth

pytestmark = pytest.mark.gpu


def make(cap, dtype, seed, B=2, Ly=2, H=3, hd=128):
    w = synth.Workload("na", B, Ly, H, hd, cap, dtype, 4, 0.9, 2, synth.BASE_SEED + seed)
    return synth.make_cache(w, "cuda")


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_noalloc_matches_compress_on_two_calls_in_a_row(dtype):
    ctx = fk.Context(0)
    try:
        ctx.set_variant(fk.SIMT)
        # first a larger shape, then a smaller one whose basis occupies only part of what the
        # first call left behind in the shared arrays, then the first shape again
        for seed, (cache_len, kept) in enumerate([(600, 298), (104, 37), (600, 298)]):
            k, v = make(cache_len + 6, dtype, 40 + seed)
            k_ref, v_ref = k.clone(), v.clone()
            ctx.compress(k_ref, v_ref, cache_len, kept, 4)
            new_len = fk.compress_noalloc(k, v, cache_len, kept, 4)
            torch.cuda.synchronize()
            assert new_len == 4 + kept
            tol = 1e-2 if dtype == torch.bfloat16 else 1e-5
            for got, want in ((k, k_ref), (v, v_ref)):
                g, r = got.double(), want.double()
                assert (g - r).norm() <= tol * r.norm()
                assert torch.equal(got, want)  # same kernels, same arithmetic: identical bits
    finally:
        ctx.close()


def test_noalloc_many_matrices_use_the_staging_area_in_groups():
    # 2 * 1 * 8 * 40 = 640 matrices of 500 x 128 bf16 = 80 MB of compressed rows >> 4 MiB staging
    k, v = make(1010, torch.bfloat16, 50, B=1, Ly=8, H=40)
    ctx = fk.Context(0)
    try:
        ctx.set_variant(fk.SIMT)
        k_ref, v_ref = k.clone(), v.clone()
        ctx.compress(k_ref, v_ref, 1004, 500, 4)
        fk.compress_noalloc(k, v, 1004, 500, 4)
        torch.cuda.synchronize()
        assert torch.equal(k, k_ref) and torch.equal(v, v_ref)
    finally:
        ctx.close()


def test_noalloc_rejects_sizes_beyond_its_arrays():
    k, v = make(4096, torch.bfloat16, 60, B=1, Ly=1, H=1)
    before = k.clone()
    with pytest.raises(fk.FreqKVError) as e:
        fk.compress_noalloc(k, v, 4096, 2046, 4)   # 4096 x 2048 basis entries > 1 Mi
    assert e.value.status == fk.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert torch.equal(k, before)
    with pytest.raises(fk.FreqKVError) as e:
        fk.compress_noalloc(k, v, 100, 97, 4)      # kept_len > cache_len - sink
    assert e.value.status == fk.ERR_INVALID_ARG
    assert fk.compress_noalloc(k, v, 100, 96, 4) == 100   # identity: nothing to do


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_noalloc_matches_the_oracle_and_allocates_nothing(dtype):
    """Against oracle.compress_matrix on the same bits (relative L2 <= 1e-2 bf16 / 1e-5 fp32, every
    matrix), sink rows and rows past the new length bit-exact; and the property the entry point
    exists for: free device memory is unchanged across calls made after the first one."""
    cache_len, kept, sink = 517, 256, 4
    k, v = make(cache_len + 3, dtype, 70, B=1, Ly=2, H=2)
    k_in, v_in = k.clone(), v.clone()
    spare_k, spare_v = k.clone(), v.clone()
    fk.compress_noalloc(spare_k, spare_v, cache_len, kept, sink)   # first call on this device: address look-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    assert fk.compress_noalloc(k, v, cache_len, kept, sink) == sink + kept
    fk.compress_noalloc(spare_k, spare_v, sink + kept, 100, sink)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before, "freqkv_compress_noalloc changed the amount of free device memory"
    tol = 1e-2 if dtype == torch.bfloat16 else 1e-5
    for t_in, t_out in ((k_in, k), (v_in, v)):
        assert torch.equal(t_out[..., :sink, :], t_in[..., :sink, :])
        assert torch.equal(t_out[..., sink + kept:, :], t_in[..., sink + kept:, :])
        for l in range(2):
            for h in range(2):
                want = oracle.compress_matrix(t_in[0, l, h, sink:cache_len].double().cpu().numpy(), kept)
                got = t_out[0, l, h, sink:sink + kept].double().cpu().numpy()
                assert np.linalg.norm(got - want) <= tol * np.linalg.norm(want)


def test_noalloc_rejects_host_memory():
    k, v = make(128, torch.bfloat16, 80, B=1, Ly=1, H=1)
    host = v.cpu().pin_memory()
    with pytest.raises(fk.FreqKVError) as e:
        fk.compress_noalloc(k, host, 100, 40, 4)   # V is not device memory
    assert e.value.status == fk.ERR_INVALID_ARG
