"""Pins for the CPU oracle: it is checked against what the paper and the mathematics fix,
never against the CUDA path.  Each pin is chosen so that a plausible slip in the oracle (a
dropped rescale, a wrong alpha_0, a wrong phase, a transposed operand, an N-point instead
of an L-point inverse) fails at least one of them."""
import math
import os

import numpy as np
import pytest
import scipy.fft

import oracle
from paper_2505_00570_b200 import synth

TOL = 1e-11
SIZES = [(1, 1), (2, 1), (3, 2), (5, 5), (8, 4), (12, 6), (31, 15), (64, 64), (128, 64), (257, 100), (1023, 511)]


def rng(seed):
    return np.random.default_rng(seed)


def rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


# ---- the transform pair against a library routine (textbook orthonormal DCT-II / DCT-III)
@pytest.mark.parametrize("N", [1, 2, 3, 7, 16, 62, 129, 512, 1000])
def test_dct2_matches_library(N):
    x = rng(N).standard_normal((N, 5))
    assert rel(oracle.dct2(x), scipy.fft.dct(x, type=2, norm="ortho", axis=0)) < TOL
    n_out = max(1, N // 3)
    assert rel(oracle.dct2(x, n_out), scipy.fft.dct(x, type=2, norm="ortho", axis=0)[:n_out]) < TOL


@pytest.mark.parametrize("L", [1, 2, 3, 7, 16, 62, 129, 511])
def test_idct_matches_library(L):
    z = rng(L + 1).standard_normal((L, 4))
    assert rel(oracle.idct(z), scipy.fft.idct(z, type=2, norm="ortho", axis=0)) < TOL


@pytest.mark.parametrize("N,L", SIZES)
def test_compress_matches_library_pipeline(N, L):
    x = rng(N * 1000 + L).standard_normal((N, 3))
    z = scipy.fft.dct(x, type=2, norm="ortho", axis=0)[:L]
    want = math.sqrt(L / N) * scipy.fft.idct(z, type=2, norm="ortho", axis=0)
    assert rel(oracle.compress_matrix(x, L), want) < TOL


# ---- closed forms and invariants
@pytest.mark.parametrize("N", [1, 4, 33, 512])
def test_identity_at_retention_one(N):
    x = rng(N).standard_normal((N, 6))
    assert rel(oracle.compress_matrix(x, N), x) < TOL
    assert rel(oracle.idct(oracle.dct2(x)), x) < TOL


@pytest.mark.parametrize("N,L", SIZES)
def test_constant_sequence_keeps_only_dc_and_is_reproduced(N, L):
    c = np.array([[3.25, -1.5, 0.0]])
    x = np.repeat(c, N, axis=0)
    z = oracle.dct2(x)
    assert np.allclose(z[0], c[0] * math.sqrt(N), atol=1e-11)
    assert np.abs(z[1:]).max(initial=0.0) < 1e-11
    y = oracle.compress_matrix(x, L)
    assert y.shape == (L, 3)
    assert np.abs(y - c).max() < 1e-11  # this is what the sqrt(L/N) rescale is for


@pytest.mark.parametrize("N,L", SIZES)
def test_parseval(N, L):
    x = rng(7 * N + L).standard_normal((N, 4))
    z = oracle.dct2(x)
    assert np.allclose((z ** 2).sum(0), (x ** 2).sum(0), rtol=1e-11)  # orthonormal DCT
    y = oracle.compress_matrix(x, L)
    assert np.allclose((y ** 2).sum(0), (L / N) * (z[:L] ** 2).sum(0), rtol=1e-11)


@pytest.mark.parametrize("N,L", [(12, 6), (31, 15), (64, 17), (512, 256), (1023, 511)])
def test_single_cosine_is_resampled_exactly(N, L):
    """x_n = cos(pi k (2n+1)/(2N)) -> y_m = cos(pi k (2m+1)/(2L)) for k < L, and 0 for
    L <= k < N (direct substitution in the two Appendix A sums and Eq. 3)."""
    n = np.arange(N)[:, None]
    m = np.arange(L)[:, None]
    ks = sorted({0, 1, 2, L // 2, L - 1, L, min(N - 1, L + 3), N - 1})
    for k in ks:
        x = np.cos(np.pi * k * (2 * n + 1) / (2 * N))
        y = oracle.compress_matrix(x, L)
        want = np.cos(np.pi * k * (2 * m + 1) / (2 * L)) if k < L else np.zeros((L, 1))
        assert np.abs(y - want).max() < 1e-11, (N, L, k)


def test_band_limited_signal_survives_repeated_compression():
    N, L1, L2 = 96, 48, 24
    n = np.arange(N)[:, None]
    x = sum(a * np.cos(np.pi * k * (2 * n + 1) / (2 * N)) for k, a in [(0, 0.5), (3, -2.0), (11, 1.25)])
    y2 = oracle.compress_matrix(oracle.compress_matrix(x, L1), L2)
    m = np.arange(L2)[:, None]
    want = sum(a * np.cos(np.pi * k * (2 * m + 1) / (2 * L2)) for k, a in [(0, 0.5), (3, -2.0), (11, 1.25)])
    assert np.abs(y2 - want).max() < 1e-11


@pytest.mark.parametrize("N,L", [(1, 1), (2, 1), (3, 2), (5, 3), (8, 4), (12, 6), (16, 16), (16, 5)])
def test_brute_force_matrices_tiny(N, L):
    """Explicit orthonormal DCT matrices built entry by entry with math.cos and multiplied
    naively: Y = sqrt(L/N) * C_L^T * C_N[0:L, :] * X."""

    def dct_matrix(n):
        return [[(math.sqrt(1.0 / n) if t == 0 else math.sqrt(2.0 / n))
                 * math.cos(math.pi * t * (2 * j + 1) / (2 * n)) for j in range(n)] for t in range(n)]

    CN, CL = dct_matrix(N), dct_matrix(L)
    x = rng(N + 31 * L).standard_normal((N, 2))
    want = np.zeros((L, 2))
    for c in range(2):
        z = [sum(CN[t][n] * x[n, c] for n in range(N)) for t in range(L)]
        for m in range(L):
            want[m, c] = math.sqrt(L / N) * sum(CL[t][m] * z[t] for t in range(L))
    assert np.abs(oracle.compress_matrix(x, L) - want).max() < 1e-12


def test_projection_invariants():
    """The map x -> y is Y = P X with P P^T = (L/N) I, rows of P summing to 1 and columns
    to L/N (consequences of orthonormality and of the rescale)."""
    for N, L in [(12, 6), (31, 15), (100, 37)]:
        P = oracle.compress_matrix(np.eye(N), L)
        assert np.abs(P @ P.T - (L / N) * np.eye(L)).max() < 1e-12
        assert np.abs(P.sum(1) - 1.0).max() < 1e-12
        assert np.abs(P.sum(0) - L / N).max() < 1e-12


def test_linearity():
    N, L = 77, 30
    r = rng(5)
    x1, x2 = r.standard_normal((N, 3)), r.standard_normal((N, 3))
    lhs = oracle.compress_matrix(2.5 * x1 - 0.75 * x2, L)
    rhs = 2.5 * oracle.compress_matrix(x1, L) - 0.75 * oracle.compress_matrix(x2, L)
    assert np.abs(lhs - rhs).max() < 1e-11


def test_inverse_is_l_point_not_subsampled_n_point():
    """A ramp distinguishes the L-point inverse from an N-point inverse of a zero-padded
    spectrum that is then subsampled (the reading this build does not take)."""
    N, L = 32, 16
    x = np.arange(N, dtype=np.float64)[:, None]
    z = scipy.fft.dct(x, type=2, norm="ortho", axis=0)
    zp = np.zeros_like(z)
    zp[:L] = z[:L]
    other = scipy.fft.idct(zp, type=2, norm="ortho", axis=0)[::2]
    y = oracle.compress_matrix(x, L)
    assert np.abs(y - other).max() > 1e-3
    # the mean survives exactly, as the constant pin demands
    assert abs(y.mean() - x.mean()) < 1e-11


# ---- cache-level bookkeeping: sinks, untouched rows, length
def test_cache_sinks_and_untouched_rows():
    r = rng(11)
    cache = r.standard_normal((2, 3, 40, 8))
    new, length = oracle.compress_cache(cache, cache_len=36, kept_len=16, sink=4)
    assert length == 20
    assert np.array_equal(new[..., :4, :], cache[..., :4, :])      # sink tokens
    assert np.array_equal(new[..., 20:, :], cache[..., 20:, :])    # stale rows and free rows
    for i in range(2):
        for j in range(3):
            assert rel(new[i, j, 4:20], oracle.compress_matrix(cache[i, j, 4:36], 16)) < TOL


def test_cache_degenerate_sizes():
    cache = rng(3).standard_normal((1, 10, 4))
    same, n = oracle.compress_cache(cache, 10, 6, 4)   # L == N': identity
    assert n == 10 and rel(same, cache) < TOL
    none, n = oracle.compress_cache(cache, 10, 0, 4)   # L == 0: only the sinks remain
    assert n == 4 and np.array_equal(none, cache)
    empty, n = oracle.compress_cache(cache, 4, 0, 4)   # N' == 0
    assert n == 4 and np.array_equal(empty, cache)
    with pytest.raises(ValueError):
        oracle.compress_cache(cache, 10, 7, 4)
    with pytest.raises(ValueError):
        oracle.compress_cache(cache, 11, 2, 4)


def test_append_and_overflow():
    cache = np.zeros((2, 6, 3))
    rows = rng(1).standard_normal((2, 2, 3))
    new, n = oracle.append(cache, rows, 3)
    assert n == 5 and np.array_equal(new[:, 3:5], rows) and np.array_equal(new[:, :3], cache[:, :3])
    with pytest.raises(OverflowError):
        oracle.append(cache, rows, 5)


# ---- the trigger rule against the counts the paper prints
def test_compression_counts_match_paper_tables(golden_dir):
    rows = []
    with open(os.path.join(golden_dir, "compression_counts.txt")) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                t, c, _ = line.split()
                rows.append((int(t), int(c)))
    assert len(rows) == 11
    for total, count in rows:
        assert oracle.compression_count(total, capacity=4096, sink=4, kept_len=2046) == count, total


def test_stream_agrees_with_count_and_one_shot():
    """Small stream: the count follows the same rule and the first compression equals a
    one-shot compression of the first `capacity` rows."""
    cap, S, T, d = 32, 4, 74, 3
    toks = rng(9).standard_normal((T, d))
    cache, length, count = oracle.stream(toks, cap, S, 0.5)
    L = (cap - S) // 2
    assert count == oracle.compression_count(T, cap, S, L) == 3
    assert length == T - count * (cap - S - L)
    assert np.array_equal(cache[:S], toks[:S])
    first = oracle.compress_matrix(toks[S:cap], L)
    second = oracle.compress_matrix(np.concatenate([first, toks[cap:cap + cap - S - L]]), L)
    third = oracle.compress_matrix(np.concatenate([second, toks[2 * cap - S - L:3 * cap - 2 * (S + L)]]), L)
    assert rel(cache[S:S + L], third) < TOL


# ---- the synthetic generator has the spectrum it is meant to have (sanity, loose)
def test_ar1_energy_is_low_frequency():
    w = synth.WORKLOADS["tiny"]
    k, _ = synth.make_cache(w, "cpu")
    x = k[0, 0, 0].double().numpy()
    scale = np.sqrt((x ** 2).mean(0, keepdims=True))
    y = oracle.compress_matrix(x / scale, 256)
    frac = (y ** 2).mean() / 1.0
    expected = (2 / math.pi) * math.atan((1 + w.rho) / (1 - w.rho))  # AR(1) low-half energy
    assert abs(frac - expected) < 0.05


# ---- retaining another band of components (the high/low-frequency ablation)
@pytest.mark.parametrize("N,L", [(8, 4), (31, 15), (128, 64), (257, 100)])
def test_band_zero_offset_is_the_low_pass_compression(N, L):
    x = rng(N + L).standard_normal((N, 3))
    assert rel(oracle.compress_band_matrix(x, L, 0), oracle.compress_matrix(x, L)) < TOL


@pytest.mark.parametrize("N,L,t0", [(12, 6, 6), (12, 5, 3), (64, 32, 32), (100, 25, 60), (31, 15, 16)])
def test_band_single_cosine_is_shifted_down_and_resampled(N, L, t0):
    """x_n = cos(pi k (2n+1)/(2N)) has the single DCT component k; retained in the band it becomes
    component k - t0 of the L-point inverse: y_m = cos(pi (k - t0)(2m+1)/(2L)) (times 1/sqrt 2 when it
    lands on component 0, whose weight differs); outside the band the output is zero."""
    n, m = np.arange(N), np.arange(L)
    for k in {t0, t0 + 1, t0 + L - 1, max(0, t0 - 1), min(N - 1, t0 + L)} - {0}:
        x = np.cos(np.pi * k * (2 * n + 1) / (2 * N))[:, None]
        y = oracle.compress_band_matrix(x, L, t0)[:, 0]
        if t0 <= k < t0 + L:
            want = np.cos(np.pi * (k - t0) * (2 * m + 1) / (2 * L)) * (1 / math.sqrt(2) if k == t0 else 1.0)
        else:
            want = np.zeros(L)
        assert np.max(np.abs(y - want)) < 1e-11


@pytest.mark.parametrize("N,L,t0", [(64, 32, 32), (100, 30, 11), (257, 100, 157)])
def test_band_parseval_and_linearity(N, L, t0):
    r = rng(N * 7 + t0)
    x, x2 = r.standard_normal((N, 4)), r.standard_normal((N, 4))
    z = scipy.fft.dct(x, type=2, norm="ortho", axis=0)
    y = oracle.compress_band_matrix(x, L, t0)
    assert abs(np.sum(y * y) - (L / N) * np.sum(z[t0:t0 + L] ** 2)) < 1e-10 * np.sum(x * x)
    want = math.sqrt(L / N) * scipy.fft.idct(z[t0:t0 + L], type=2, norm="ortho", axis=0)   # library pipeline
    assert rel(y, want) < TOL
    assert rel(oracle.compress_band_matrix(2 * x - 3 * x2, L, t0), 2 * y - 3 * oracle.compress_band_matrix(x2, L, t0)) < TOL


def test_band_low_plus_high_halves_carry_all_the_energy():
    N = 64
    x = rng(5).standard_normal((N, 2))
    lo, hi = oracle.compress_band_matrix(x, 32, 0), oracle.compress_band_matrix(x, 32, 32)
    assert abs(np.sum(lo * lo) + np.sum(hi * hi) - 0.5 * np.sum(x * x)) < 1e-10


# ---- average power spectrum (Section 3.1)
def test_power_spectrum_parseval_constant_and_single_cosine():
    N, d = 96, 5
    x = rng(21).standard_normal((3, N, d))
    p = oracle.power_spectrum(x)
    assert abs(p.sum() - np.mean(np.sum(x * x, axis=1))) < 1e-10            # orthonormal transform: energy is kept
    c = np.full((N, 2), 1.5)
    pc = oracle.power_spectrum(c)
    assert abs(pc[0] - N * 1.5 ** 2) < 1e-10 and np.max(np.abs(pc[1:])) < 1e-20   # a constant has its DC term only
    n = np.arange(N)
    k = 7
    pk = oracle.power_spectrum(np.cos(np.pi * k * (2 * n + 1) / (2 * N))[:, None] * 2.0)
    want = np.zeros(N)
    want[k] = 4.0 * N / 2                                                     # alpha_k^2 (sum cos^2)^2 = (2/N)(N/2)^2
    assert np.max(np.abs(pk - want)) < 1e-10


def test_power_spectrum_of_ar1_follows_the_textbook_spectrum():
    """Many AR(1) channels: the averaged DCT power at component t approaches the AR(1) spectral
    density (1 - rho^2) / (1 - 2 rho cos w + rho^2) at w = pi t / N (away from the edges)."""
    N, rho = 256, 0.9
    e = rng(22).standard_normal((40, N + 200, 16))
    x = np.zeros_like(e)
    for i in range(1, N + 200):
        x[:, i] = rho * x[:, i - 1] + math.sqrt(1 - rho * rho) * e[:, i]
    p = oracle.power_spectrum(x[:, 200:])
    w = np.pi * np.arange(N) / N
    want = (1 - rho * rho) / (1 - 2 * rho * np.cos(w) + rho * rho)
    band = slice(8, N - 8)
    assert np.max(np.abs(p[band] / want[band] - 1)) < 0.25                    # 640 channels: ~6 % noise per component
    assert abs(np.mean(p[band] / want[band]) - 1) < 0.03
