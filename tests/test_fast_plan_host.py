"""The plan of the fast-transform variant, checked on the CPU: the factored chain (four dense
stages, two twiddle passes, the index maps between them) that the FDCT kernel runs, applied in
fp64 on the host by ``freqkv_fast_plan_apply_host``, must reproduce the CPU oracle's defining sums
(Section 3.3, Eq. 2-3; Appendix A) to rounding error for every pair of lengths it accepts."""
import numpy as np
import pytest

import oracle
from paper_2505_00570_b200 import binding as fk

SHAPES = [(4096, 2048), (4092, 2046), (4092, 1023), (4092, 3069), (4092, 40), (2046, 1023), (1000, 333), (1024, 512),
          (4094, 2047), (3000, 1500), (2050, 1025), (256, 128), (300, 150), (4608, 2304), (64, 32), (96, 90)]


@pytest.mark.parametrize("n_in,n_keep", SHAPES)
def test_factored_chain_equals_the_definition(n_in, n_keep):
    rng = np.random.default_rng(n_in * 7 + n_keep)
    x = rng.standard_normal((n_in, 3))
    x[:, 1] = np.cos(np.pi * 5 * (2 * np.arange(n_in) + 1) / (2 * n_in))   # one low-frequency component: resampled exactly
    try:
        y, (n1, n2, l1, l2) = fk.fast_plan_apply_host(x, n_keep)
    except fk.FreqKVError as e:
        assert e.status == fk.ERR_UNSUPPORTED
        pytest.skip("no factorisation of these lengths fits the kernel")
    assert n1 * n2 == n_in and l1 * l2 == n_keep
    want = oracle.compress_matrix(x, n_keep)
    assert np.abs(y - want).max() <= 1e-11 * max(1.0, np.abs(want).max())
    if n_keep > 5:
        closed = np.cos(np.pi * 5 * (2 * np.arange(n_keep) + 1) / (2 * n_keep))
        assert np.abs(y[:, 1] - closed).max() <= 1e-11


def test_the_benchmark_shapes_are_accepted():
    for n_in, n_keep in [(4096, 2048), (4092, 2046)]:
        fk.fast_plan_apply_host(np.zeros((n_in, 1)), n_keep)


def test_lengths_without_a_fitting_factorisation_are_refused():
    for n_in, n_keep in [(4099, 2049), (8188, 4094), (600, 298)]:   # a prime; too long for shared memory; 298 = 2 x 149
        with pytest.raises(fk.FreqKVError) as e:
            fk.fast_plan_apply_host(np.zeros((n_in, 1)), n_keep)
        assert e.value.status == fk.ERR_UNSUPPORTED
    with pytest.raises(fk.FreqKVError) as e:
        fk.fast_plan_apply_host(np.zeros((64, 1)), 64)
    assert e.value.status == fk.ERR_INVALID_ARG
