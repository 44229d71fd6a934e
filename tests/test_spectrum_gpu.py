"""GPU parity of freqkv_power_spectrum (average DCT power spectrum of the cached states,
Section 3.1) against the fp64 oracle on the same seeded caches.

Tolerance: relative L2 of each (layer, head) spectrum <= 1e-2.  The components are computed with
bf16 operands (the folded inputs and the DCT matrix are rounded to bf16: about 2e-3 relative each)
and fp32 accumulation; a squared component carries twice the relative error of the component,
and averaging over channels and sequences does not reduce the part of it that is common to them
(the rounding of the DCT matrix)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2505_00570_b200 import binding as fk
from paper_2505_00570_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu
TOL = 1e-2


@pytest.fixture(scope="module")
def ctx():
    c = fk.Context(0)
    yield c
    c.close()


def check(ctx, w, cache_len, sink, heads=None):
    k, v = synth.make_cache(w, "cuda")
    k0, v0 = k.clone(), v.clone()
    sk, sv = ctx.power_spectrum(k, v, cache_len, sink)
    assert ctx.last_device_status() == fk.OK
    assert torch.equal(k, k0) and torch.equal(v, v0)
    pick = heads if heads is not None else [(l, h) for l in range(w.layers) for h in range(w.kv_heads)]
    worst = 0.0
    for l, h in pick:
        for t, s in ((k, sk), (v, sv)):
            x = parity.to_f64(t[:, l, h, sink:cache_len])
            want = oracle.power_spectrum(x)
            got = s[l, h].double().cpu().numpy()
            worst = max(worst, parity.rel_l2(got, want))
            # orthonormal transform: the spectrum sums to the mean energy per channel
            assert abs(got.sum() / np.mean(np.sum(x * x, axis=1)) - 1) < TOL
    assert worst <= TOL, f"relative L2 {worst:.3e}"
    return worst


@pytest.mark.parametrize("n_in,sink,B", [(296, 4, 2), (297, 3, 1), (64, 0, 3), (1, 2, 1), (700, 4, 2)])
def test_spectrum_small_all_heads(ctx, n_in, sink, B):
    w = synth.Workload("spec", B, 2, 3, 128, n_in + sink + 5, torch.bfloat16, sink, 0.9, 2, synth.BASE_SEED + 31)
    check(ctx, w, n_in + sink, sink)


def test_spectrum_is_low_frequency_dominated_like_the_paper_figure(ctx):
    """The synthetic caches stand in for states whose energy sits at low frequencies: the lowest
    eighth of the components must hold most of the energy (AR(1), rho = 0.9: about 80 %)."""
    w = synth.Workload("spec", 4, 1, 2, 128, 1024, torch.bfloat16, 0, 0.9, 0, synth.BASE_SEED + 32)
    k, v = synth.make_cache(w, "cuda")
    sk, _ = ctx.power_spectrum(k, v, 1024, 0)
    frac = (sk[0, 0, :128].sum() / sk[0, 0].sum()).item()
    assert 0.7 < frac < 0.9


def test_spectrum_7b_shape_sampled_heads(ctx):
    w = dataclasses.replace(synth.WORKLOADS["llama2_7b"], layers=4, kv_heads=32)
    check(ctx, w, 4096, 4, heads=[(0, 0), (3, 31), (2, 17)])


def test_spectrum_unsupported_and_invalid(ctx):
    k = torch.zeros(1, 1, 1, 64, 128, device="cuda", dtype=torch.float32)
    with pytest.raises(fk.FreqKVError) as e:
        ctx.power_spectrum(k, torch.zeros_like(k), 64, 0)
    assert e.value.status == fk.ERR_UNSUPPORTED
    kb = torch.zeros(1, 1, 1, 64, 128, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(fk.FreqKVError) as e:
        ctx.power_spectrum(kb, torch.zeros_like(kb), 4, 4)
    assert e.value.status == fk.ERR_INVALID_ARG
