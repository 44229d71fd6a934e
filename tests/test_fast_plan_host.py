"""The plan of the fast-transform variant, checked on the CPU: the factored chain (four dense
stages and the passes between them: index maps, twiddles or the signed placement table) that the
FDCT kernel runs, applied in fp64 on the host by ``freqkv_fast_plan_apply_host``, must reproduce
the CPU oracle's defining sums (Section 3.3, Eq. 2-3; Appendix A) to rounding error for every pair
of lengths it accepts, in both families of factorisation (prime-factor: coprime factors, real
arithmetic; Cooley-Tukey: any factors, complex arithmetic with twiddles)."""
import numpy as np
import pytest

import oracle
from paper_2505_00570_b200 import binding as fk

SHAPES = [(4096, 2048), (4092, 2046), (4092, 1023), (4092, 3069), (4092, 40), (2046, 1023), (1000, 333), (1024, 512),
          (4094, 2047), (3000, 1500), (2050, 1025), (256, 128), (300, 150), (4400, 2200), (64, 32), (96, 90)]


@pytest.mark.parametrize("family", [0, fk.COOLEY_TUKEY, fk.PRIME_FACTOR])
@pytest.mark.parametrize("n_in,n_keep", SHAPES)
def test_factored_chain_equals_the_definition(n_in, n_keep, family):
    rng = np.random.default_rng(n_in * 7 + n_keep)
    x = rng.standard_normal((n_in, 3))
    x[:, 1] = np.cos(np.pi * 5 * (2 * np.arange(n_in) + 1) / (2 * n_in))   # one low-frequency component: resampled exactly
    try:
        y, (n1, n2, l1, l2, used) = fk.fast_plan_apply_host(x, n_keep, family)
    except fk.FreqKVError as e:
        assert e.status == fk.ERR_UNSUPPORTED
        pytest.skip("no factorisation of this family fits the kernel for these lengths")
    assert n1 * n2 == n_in and l1 * l2 == n_keep
    assert used == family or (family == 0 and used in (fk.COOLEY_TUKEY, fk.PRIME_FACTOR))
    if used == fk.PRIME_FACTOR:   # coprime factors, the transform-like ones odd
        assert np.gcd(4 * n1, n2) == 1 and np.gcd(4 * l1, l2) == 1
    want = oracle.compress_matrix(x, n_keep)
    assert np.abs(y - want).max() <= 1e-11 * max(1.0, np.abs(want).max())
    if n_keep > 5:
        closed = np.cos(np.pi * 5 * (2 * np.arange(n_keep) + 1) / (2 * n_keep))
        assert np.abs(y[:, 1] - closed).max() <= 1e-11


def test_the_benchmark_shapes_are_accepted():
    for n_in, n_keep in [(4096, 2048), (4092, 2046)]:
        fk.fast_plan_apply_host(np.zeros((n_in, 1)), n_keep)
    # the paper's lengths split into coprime factors (44 x 93 -> 22 x 93): no twiddles; a power of two has no such split
    assert fk.fast_plan_apply_host(np.zeros((4092, 1)), 2046)[1] == (44, 93, 22, 93, fk.PRIME_FACTOR)
    assert fk.fast_plan_apply_host(np.zeros((4096, 1)), 2048)[1][4] == fk.COOLEY_TUKEY
    with pytest.raises(fk.FreqKVError) as e:
        fk.fast_plan_apply_host(np.zeros((4096, 1)), 2048, fk.PRIME_FACTOR)
    assert e.value.status == fk.ERR_UNSUPPORTED
    with pytest.raises(fk.FreqKVError) as e:
        fk.fast_plan_apply_host(np.zeros((4096, 1)), 2048, 7)
    assert e.value.status == fk.ERR_INVALID_ARG


def test_lengths_without_a_fitting_factorisation_are_refused():
    for n_in, n_keep in [(4099, 2049), (8188, 4094), (600, 298)]:   # a prime; too long for shared memory; 298 = 2 x 149
        with pytest.raises(fk.FreqKVError) as e:
            fk.fast_plan_apply_host(np.zeros((n_in, 1)), n_keep)
        assert e.value.status == fk.ERR_UNSUPPORTED
    with pytest.raises(fk.FreqKVError) as e:
        fk.fast_plan_apply_host(np.zeros((64, 1)), 64)
    assert e.value.status == fk.ERR_INVALID_ARG
