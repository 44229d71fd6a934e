"""FreqKV compression oracle -- TEST INFRASTRUCTURE, not part of the product.

Plain fp64 CPU statement of the hot path (append, lazy trigger, compress), written from
the paper's definitions.  The transform sums live in ``freqkv_oracle.c`` (plain C, the
defining cosine sums of Appendix A); this module loads that file through ``ctypes`` and
adds the cache-level bookkeeping of Sections 3.3-3.4 in numpy.

Only ``tests/``, ``__graft_entry__.smoke()`` and ``bench.py``'s cpu_baseline / reference
leg may import this package.  It imports nothing from the CUDA package.

Pins: see ``tests/test_oracle_pins.py`` (library DCT cross-check, identity at retention 1,
constant sequence, Parseval, single-cosine resampling, brute-force matrices on tiny
lengths, linearity, and the paper's compression-count tables for the trigger rule).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "freqkv_oracle.c")
_LIB = os.path.join(_HERE, "libfreqkv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``freqkv_oracle.c`` into a shared object beside it (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", _SRC, "-o", tmp, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        p = ctypes.POINTER(ctypes.c_double)
        i64 = ctypes.c_int64
        lib.freqkv_oracle_dct2.argtypes = [p, i64, i64, i64, p]
        lib.freqkv_oracle_idct.argtypes = [p, i64, i64, p]
        lib.freqkv_oracle_compress.argtypes = [p, i64, i64, i64, p]
        for f in (lib.freqkv_oracle_dct2, lib.freqkv_oracle_idct, lib.freqkv_oracle_compress):
            f.restype = ctypes.c_int
        lib.freqkv_oracle_threads.restype = ctypes.c_int
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _as_matrix(x) -> np.ndarray:
    x = np.ascontiguousarray(np.asarray(x, dtype=np.float64))
    if x.ndim == 1:
        x = x[:, None]
    if x.ndim != 2:
        raise ValueError("expected a [tokens, channels] matrix")
    return x


def threads() -> int:
    """Threads the C loops use."""
    return int(_load().freqkv_oracle_threads())


def dct2(x, n_out: int | None = None) -> np.ndarray:
    """Orthonormal DCT-II along axis 0 (Appendix A); first ``n_out`` components."""
    x = _as_matrix(x)
    N, d = x.shape
    n_out = N if n_out is None else int(n_out)
    z = np.empty((n_out, d), dtype=np.float64)
    if _load().freqkv_oracle_dct2(_ptr(x), N, d, n_out, _ptr(z)) != 0:
        raise ValueError("freqkv_oracle_dct2: bad sizes")
    return z


def idct(z) -> np.ndarray:
    """Orthonormal inverse DCT along axis 0, of the length of ``z`` (Appendix A)."""
    z = _as_matrix(z)
    L, d = z.shape
    y = np.empty((L, d), dtype=np.float64)
    if _load().freqkv_oracle_idct(_ptr(z), L, d, _ptr(y)) != 0:
        raise ValueError("freqkv_oracle_idct: bad sizes")
    return y


def compress_matrix(x, kept_len: int) -> np.ndarray:
    """sqrt(L/N) * IDCT_L(DCT_N(x)[0:L]) for one [N, d] matrix (Section 3.3, Eq. 2-3)."""
    x = _as_matrix(x)
    N, d = x.shape
    L = int(kept_len)
    if L < 0 or L > N:
        raise ValueError("kept_len must lie in [0, N]")
    y = np.empty((L, d), dtype=np.float64)
    if L and _load().freqkv_oracle_compress(_ptr(x), N, L, d, _ptr(y)) != 0:
        raise ValueError("freqkv_oracle_compress: bad sizes")
    return y


def compress_band_matrix(x, kept_len: int, first: int) -> np.ndarray:
    """The ablation of Appendix "Retaining High/Low-Frequency Components": keep the ``kept_len``
    DCT components ``first .. first + kept_len - 1`` instead of the lowest ones, then the same
    L-point inverse and rescale:  sqrt(L/N) * IDCT_L(DCT_N(x)[first : first + L]).
    ``first = 0`` is ``compress_matrix``; ``first = N - L`` retains the highest frequencies.
    (The paper does not say where the retained components go in the inverse transform; they
    take positions 0 .. L-1 here, the only choice that keeps the output length L.)"""
    x = _as_matrix(x)
    N, d = x.shape
    L, t0 = int(kept_len), int(first)
    if L < 0 or t0 < 0 or t0 + L > N:
        raise ValueError("need 0 <= first and first + kept_len <= N")
    if L == 0:
        return np.empty((0, d))
    z = dct2(x)                      # all N components (Appendix A, DCT-II)
    kept = np.ascontiguousarray(z[t0:t0 + L])
    return np.sqrt(L / N) * idct(kept)


def power_spectrum(states) -> np.ndarray:
    """Average power spectrum along the token axis (Section 3.1, the analysis behind the
    paper's power-spectrum figures): every channel of every ``[N, d]`` matrix in ``states``
    (``[..., N, d]``; the leading axes are samples) is transformed with the orthonormal DCT-II
    of Appendix A and the squared components are averaged over samples and channels.
    Returns ``[N]``.  ("Power" is read as the squared amplitude of a component.)"""
    a = np.asarray(states, dtype=np.float64)
    N, d = a.shape[-2], a.shape[-1]
    flat = a.reshape(-1, N, d)
    total = np.zeros(N)
    for x in flat:
        z = dct2(x)
        total += np.sum(z * z, axis=1)
    return total / (flat.shape[0] * d)


def compress_cache(cache, cache_len: int, kept_len: int, sink: int) -> tuple[np.ndarray, int]:
    """One compression of every matrix of a cache (Sections 3.3-3.4).

    ``cache`` is ``[..., capacity, head_dim]`` (any leading axes: batch, layer, kv_head).
    Rows ``[sink, cache_len)`` of each matrix are the signal; rows ``[sink, sink+kept_len)``
    of the result hold the compressed signal, every other row is returned as it was (sink
    tokens stay uncompressed, Section 3.4; stale rows past the new length are not cleared).
    Returns ``(new cache in fp64, new length sink + kept_len)``.
    """
    a = np.array(cache, dtype=np.float64)  # exact for bf16/fp32 inputs; a copy
    cap, d = a.shape[-2], a.shape[-1]
    S, N, L = int(sink), int(cache_len) - int(sink), int(kept_len)
    if not (0 <= S <= cache_len <= cap) or L < 0 or L > N:
        raise ValueError("need 0 <= sink <= cache_len <= capacity and 0 <= kept_len <= cache_len - sink")
    flat = a.reshape(-1, cap, d)
    if N > 0 and L > 0:
        for i in range(flat.shape[0]):
            flat[i, S:S + L, :] = compress_matrix(flat[i, S:S + N, :], L)
    return a, S + L


def append(cache, new_rows, cache_len: int) -> tuple[np.ndarray, int]:
    """Rows ``[cache_len, cache_len + n_new)`` <- ``new_rows`` (Section 3.4: incoming
    tokens are appended to the compressed cache).  Raises when the cache has no room:
    that is the caller's cue to compress first (the lazy trigger below)."""
    a = np.array(cache, dtype=np.float64)
    new = np.asarray(new_rows, dtype=np.float64)
    n_new = new.shape[-2]
    if cache_len + n_new > a.shape[-2]:
        raise OverflowError("cache full")
    a[..., cache_len:cache_len + n_new, :] = new
    return a, cache_len + n_new


def compression_count(total_tokens: int, capacity: int, sink: int, kept_len: int) -> int:
    """How many compressions a stream of ``total_tokens`` tokens causes (Section 3.4).

    Tokens enter one at a time; a compression happens when a token must enter a cache
    that already holds ``capacity`` tokens (reading pinned by the paper's two
    compression-count tables: a 4K input causes none).  After it the cache holds
    ``sink + kept_len`` tokens.
    """
    length, count = 0, 0
    for _ in range(int(total_tokens)):
        if length == capacity:
            length = sink + kept_len
            count += 1
        length += 1
    return count


def stream(tokens, capacity: int, sink: int, retain: float = 0.5) -> tuple[np.ndarray, int, int]:
    """Iterative compression of a token stream for one matrix (Section 3.4, Figure 3b).

    ``tokens``: ``[T, d]``.  Rows are appended one at a time; when a row must enter a full
    cache, the non-sink part is compressed to ``floor(retain * (capacity - sink))`` rows
    first.  Returns ``(cache [capacity, d] fp64, final length, compression count)``.
    """
    tokens = _as_matrix(tokens)
    d = tokens.shape[1]
    cache = np.zeros((capacity, d), dtype=np.float64)
    length, count = 0, 0
    L = int(np.floor(retain * (capacity - sink)))
    for row in tokens:
        if length == capacity:
            # same steps as compress_cache / append above, written on the one array in place
            # (a stream of 10^5 tokens would otherwise copy the whole cache once per token)
            cache[sink:sink + L, :] = compress_matrix(cache[sink:length, :], L)
            length = sink + L
            count += 1
        cache[length, :] = row
        length += 1
    return cache, length, count
