"""freqkv_compress_noalloc, the entry point for callers that cannot allocate device memory
(stream capture, frozen memory budgets, frameworks that own all device memory): its result must
equal that of freqkv_compress on the same input, call after call, although every call reuses
the same fixed work arrays inside the library.  Collected last on purpose, so that a run that
stops at the first failure has already run every other test."""
import pytest
import torch

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
