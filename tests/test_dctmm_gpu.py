"""GPU parity of the fast transform on the tensor cores (variant FDCT for bf16 caches) against the
fp64 oracle, through the C ABI: relative L2 <= 1e-2 per matrix, the per-row bound, and every byte
outside the rewritten rows bit-exact (in place, no scratch)."""
import dataclasses

import pytest
import torch

from paper_2505_00570_b200 import binding as fk
from paper_2505_00570_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = fk.Context(0)
    yield c
    c.close()


def wl(cap, sink, B=1, Ly=1, H=2, hd=128, rho=0.9, seed=21):
    return synth.Workload("fast", B, Ly, H, hd, cap, torch.bfloat16, sink, rho, 2, synth.BASE_SEED + seed)


@pytest.mark.parametrize("family", [fk.PRIME_FACTOR, fk.COOLEY_TUKEY])
@pytest.mark.parametrize("n_in,kept,sink", [(1024, 512, 0), (4096, 2048, 0), (4092, 2046, 4), (4092, 1023, 4), (4092, 3069, 4), (2046, 1534, 4),
                                            (1000, 333, 3), (2046, 1023, 2), (3000, 1500, 4), (300, 150, 4), (4094, 2047, 0),
                                            (4092, 40, 4), (4400, 2200, 4), (4340, 2170, 0)])
def test_fast_transform_lengths(ctx, n_in, kept, sink, family):
    """Both families of factorisation (coprime factors without twiddles; any factors with twiddles),
    each on every pair of lengths it can factor."""
    w = wl(n_in + sink + 5, sink)
    ctx.set_variant(fk.FDCT)
    ctx.set_fast_family(family)
    try:
        lay = fk.layout_of(torch.empty(1, 1, 2, n_in + sink + 5, 128, dtype=torch.bfloat16))
        if ctx.resolve_variant(lay, n_in, kept) != fk.FDCT:
            pytest.skip("no factorisation of this family fits the kernel for these lengths")
        parity.check_compress(ctx, w, n_in + sink, kept, sink, fk.FDCT)
    finally:
        ctx.set_fast_family(0)


def test_fast_family_switch(ctx):
    """The default takes the prime-factor stages where the lengths have coprime factors; each family can be
    forced; a family that cannot factor a shape leaves it to another kernel; other values are refused."""
    lay = fk.layout_of(torch.empty(1, 1, 2, 4100, 64, dtype=torch.bfloat16))   # head_dim 64: no tensor-core projection
    w = wl(4100, 4, hd=64)
    outs = []
    try:
        for family in (0, fk.PRIME_FACTOR, fk.COOLEY_TUKEY):
            ctx.set_fast_family(family)
            ctx.set_variant(fk.AUTO)
            assert ctx.resolve_variant(lay, 4092, 2046) == fk.FDCT
            k, v = synth.make_cache(w, "cuda")
            ctx.compress(k, v, 4096, 2046, 4)
            outs.append(k[..., 4:2050, :].clone())
        assert ctx.last_device_status() == fk.OK
        assert torch.equal(outs[0], outs[1])              # the default is the prime-factor family here
        assert not torch.equal(outs[1], outs[2])          # another chain of roundings ...
        a, b = outs[1].double(), outs[2].double()
        assert ((a - b).norm() / a.norm()).item() < 1e-2  # ... of the same result
        ctx.set_fast_family(fk.PRIME_FACTOR)              # 4400 = 2^4 x 5^2 x 11 has no coprime factors within the limits
        ctx.set_variant(fk.AUTO)
        big = fk.layout_of(torch.empty(1, 1, 2, 4500, 64, dtype=torch.bfloat16))
        assert ctx.resolve_variant(big, 4400, 2200) == fk.SIMT
        ctx.set_fast_family(fk.COOLEY_TUKEY)
        assert ctx.resolve_variant(big, 4400, 2200) == fk.FDCT
        with pytest.raises(fk.FreqKVError) as e:
            ctx.set_fast_family(3)
        assert e.value.status == fk.ERR_INVALID_ARG
    finally:
        ctx.set_fast_family(0)


def test_fast_transform_white_noise(ctx):
    """Half of the energy is discarded: still the plain metric."""
    parity.check_compress(ctx, wl(4096, 4, rho=0.0), 4096, 2046, 4, fk.FDCT)


def test_fast_transform_input_without_energy_in_the_kept_band(ctx):
    """rho = -0.9 puts 97 % of the energy into the discarded half; the roundings of the chain scale
    with the whole signal, so the error is measured against the evenly-spread output norm."""
    parity.check_compress(ctx, wl(4096, 4, rho=-0.9), 4096, 2046, 4, fk.FDCT, energy_scaled=True)


def test_fast_transform_many_slabs_padding_and_batches(ctx):
    """More slabs than SMs (persistent loop), padded rows, several sequences / layers / heads."""
    parity.check_compress(ctx, wl(1030, 4, B=2, Ly=3, H=5), 1028, 512, 4, fk.FDCT, row_pad=8)


@pytest.mark.parametrize("hd", [64, 8, 256])
def test_fast_transform_other_head_dims(ctx, hd):
    parity.check_compress(ctx, wl(1100, 4, hd=hd, H=3), 1028, 512, 4, fk.FDCT)


def test_fast_transform_is_deterministic_and_repeatable(ctx):
    w = wl(4096, 4, Ly=2, H=4)
    k, v = synth.make_cache(w, "cuda")
    k2, v2 = k.clone(), v.clone()
    ctx.set_variant(fk.FDCT)
    ctx.compress(k, v, 4096, 2046, 4)
    ctx.compress(k2, v2, 4096, 2046, 4)
    ctx.set_variant(fk.AUTO)
    assert ctx.last_device_status() == fk.OK
    assert torch.equal(k, k2) and torch.equal(v, v2)


def test_fast_transform_7b_shape_sample(ctx):
    w = dataclasses.replace(synth.WORKLOADS["llama2_7b"], layers=2, kv_heads=8)
    parity.check_compress(ctx, w, 4096, 2046, 4, fk.FDCT, sample=8)
