"""Thin ctypes binding of ``libfreqkv.so`` (declared in ``include/freqkv.h``).

Argument marshalling only: tensors are passed as ``data_ptr()``, the stream as
``torch.cuda.current_stream().cuda_stream``; every step of the path runs in the library's
kernels.  There is no fallback: if the library is not built, or a call fails, an exception is
raised.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_int, c_int32, c_int64, c_void_p

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfreqkv.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CAPACITY, ERR_ALLOC, ERR_CUDA, ERR_TIMEOUT = range(7)
BF16, F32 = 0, 1
AUTO, GEMM, FDCT, SIMT = 0, 1, 2, 3
COOLEY_TUKEY, PRIME_FACTOR = 1, 2   # families of the bf16 fast transform (freqkv_set_fast_family)
VARIANT_NAMES = {AUTO: "auto", GEMM: "gemm", FDCT: "fdct", SIMT: "simt"}

EXPORTS = [
    "freqkv_layout_contiguous", "freqkv_create", "freqkv_destroy", "freqkv_set_variant",
    "freqkv_resolve_variant", "freqkv_plan", "freqkv_compress", "freqkv_compress_ragged",
    "freqkv_append", "freqkv_last_device_status", "freqkv_check_compress", "freqkv_check_append",
    "freqkv_last_error", "freqkv_status_string", "freqkv_version", "freqkv_compress_host",
    "freqkv_set_timing", "freqkv_get_timing", "freqkv_compress_noalloc", "freqkv_attend_decode",
    "freqkv_check_attend", "freqkv_compress_band", "freqkv_power_spectrum",
    "freqkv_attend_prefill", "freqkv_check_attend_prefill",
    "freqkv_decode_graph_create", "freqkv_decode_graph_launch", "freqkv_decode_graph_destroy",
    "freqkv_set_wait_limit", "freqkv_selftest_bounded_wait", "freqkv_fast_plan_apply_host", "freqkv_set_fast_family", "freqkv_gemm_fold_levels",
]
NOALLOC_MAX_BASIS_ELEMS = 1 << 20
NOALLOC_STAGING_BYTES = 4 << 20


class Layout(ctypes.Structure):
    """Mirror of ``freqkv_layout``."""

    _fields_ = [
        ("dtype", c_int32), ("batch", c_int32), ("layers", c_int32), ("kv_heads", c_int32),
        ("capacity", c_int32), ("head_dim", c_int32),
        ("stride_batch", c_int64), ("stride_layer", c_int64), ("stride_head", c_int64), ("stride_token", c_int64),
    ]


class FreqKVError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(what)


_lib = None


def lib() -> ctypes.CDLL:
    """Load the library on first use; raise loudly if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FreqKVError(ERR_CUDA, f"{LIB_PATH} is missing: build it with "
                                        "`python -m paper_2505_00570_b200.build` (there is no fallback path)")
        L = ctypes.CDLL(LIB_PATH)
        LP = POINTER(Layout)
        I32P = POINTER(c_int32)
        L.freqkv_layout_contiguous.argtypes = [LP, c_int, c_int32, c_int32, c_int32, c_int32, c_int32]
        L.freqkv_create.argtypes = [POINTER(c_void_p), c_int]
        L.freqkv_destroy.argtypes = [c_void_p]
        L.freqkv_set_variant.argtypes = [c_void_p, c_int]
        L.freqkv_resolve_variant.argtypes = [c_void_p, LP, c_int32, c_int32, I32P]
        L.freqkv_plan.argtypes = [c_void_p, c_int32, c_int32, c_int, c_int, c_void_p]
        L.freqkv_compress.argtypes = [c_void_p, LP, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p]
        L.freqkv_compress_band.argtypes = [c_void_p, LP, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_int32, c_void_p]
        L.freqkv_power_spectrum.argtypes = [c_void_p, LP, c_void_p, c_void_p, c_int32, c_int32, c_void_p, c_void_p, c_void_p]
        L.freqkv_decode_graph_create.argtypes = [c_void_p, LP, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_int32,
                                                 c_int32, POINTER(c_void_p)]
        L.freqkv_decode_graph_launch.argtypes = [c_void_p, c_void_p]
        L.freqkv_decode_graph_destroy.argtypes = [c_void_p]
        L.freqkv_compress_ragged.argtypes = [c_void_p, LP, c_void_p, c_void_p, I32P, I32P, c_int32, c_void_p]
        L.freqkv_append.argtypes = [c_void_p, LP, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, I32P, c_void_p]
        L.freqkv_last_device_status.argtypes = [c_void_p, c_void_p]
        L.freqkv_check_compress.argtypes = [LP, c_void_p, c_void_p, c_int32, c_int32, c_int32]
        L.freqkv_check_append.argtypes = [LP, c_void_p, c_void_p, c_void_p, c_void_p, c_int32, I32P]
        L.freqkv_compress_host.argtypes = [c_void_p, LP, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p,
                                           POINTER(c_int64), POINTER(c_int64)]
        L.freqkv_set_timing.argtypes = [c_void_p, c_int32]
        L.freqkv_get_timing.argtypes = [c_void_p, POINTER(c_int64), POINTER(ctypes.c_double), POINTER(c_int64)]
        L.freqkv_compress_noalloc.argtypes = [LP, c_void_p, c_void_p, c_int32, c_int32, c_int32, c_void_p]
        L.freqkv_attend_decode.argtypes = [c_void_p, LP, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_int32, I32P,
                                           ctypes.c_float, ctypes.c_float, c_void_p]
        L.freqkv_check_attend.argtypes = [LP, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_int32, I32P]
        L.freqkv_attend_prefill.argtypes = [c_void_p, LP, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_int32, c_int32,
                                            I32P, ctypes.c_float, ctypes.c_float, c_void_p]
        L.freqkv_check_attend_prefill.argtypes = [LP, c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_int32, c_int32, I32P]
        L.freqkv_set_wait_limit.argtypes = [c_void_p, c_int64]
        L.freqkv_selftest_bounded_wait.argtypes = [c_void_p, c_int64, c_void_p]
        L.freqkv_fast_plan_apply_host.argtypes = [c_int32, c_int32, c_int32, c_void_p, c_int32, c_void_p, I32P]
        L.freqkv_set_fast_family.argtypes = [c_void_p, c_int32]
        L.freqkv_gemm_fold_levels.argtypes = [c_int32, c_int32, c_int32]
        L.freqkv_gemm_fold_levels.restype = c_int32
        L.freqkv_last_error.argtypes = [c_void_p]
        L.freqkv_last_error.restype = c_char_p
        L.freqkv_status_string.argtypes = [c_int]
        L.freqkv_status_string.restype = c_char_p
        L.freqkv_version.restype = c_int32
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().freqkv_status_string(status).decode()


def dtype_code(dtype: torch.dtype) -> int:
    if dtype == torch.bfloat16:
        return BF16
    if dtype == torch.float32:
        return F32
    raise FreqKVError(ERR_UNSUPPORTED, f"unsupported cache dtype {dtype}")


_layout_cache: dict = {}


def layout_of(t: torch.Tensor) -> Layout:
    """``freqkv_layout`` of a ``[batch, layers, kv_heads, capacity, head_dim]`` tensor (a view
    with arbitrary strides is fine as long as head_dim is contiguous).  Structs are cached by
    (dtype, shape, strides): a decode loop asks for the same one every step."""
    key = (t.dtype, tuple(t.shape), t.stride())
    lay = _layout_cache.get(key)
    if lay is None:
        if t.dim() != 5 or t.stride(4) != 1:
            raise FreqKVError(ERR_UNSUPPORTED, "cache must be [batch, layers, kv_heads, capacity, head_dim] with contiguous head_dim")
        lay = Layout(dtype_code(t.dtype), t.shape[0], t.shape[1], t.shape[2], t.shape[3], t.shape[4],
                     t.stride(0), t.stride(1), t.stride(2), t.stride(3))
        if len(_layout_cache) > 256:
            _layout_cache.clear()
        _layout_cache[key] = lay
    return lay


def layout_contiguous(dtype: int, batch: int, layers: int, kv_heads: int, capacity: int, head_dim: int):
    """(status, Layout) from ``freqkv_layout_contiguous``."""
    out = Layout()
    st = lib().freqkv_layout_contiguous(ctypes.byref(out), dtype, batch, layers, kv_heads, capacity, head_dim)
    return st, out


def check_compress(layout: Layout, k_ptr: int, v_ptr: int, cache_len: int, kept_len: int, sink: int) -> int:
    return lib().freqkv_check_compress(ctypes.byref(layout), k_ptr, v_ptr, cache_len, kept_len, sink)


def check_append(layout: Layout, k_ptr: int, v_ptr: int, nk_ptr: int, nv_ptr: int, n_new: int, lens) -> int:
    arr = (c_int32 * len(lens))(*lens)
    return lib().freqkv_check_append(ctypes.byref(layout), k_ptr, v_ptr, nk_ptr, nv_ptr, n_new, arr)


def check_attend(layout: Layout, k_ptr: int, v_ptr: int, layer: int, q_ptr: int, out_ptr: int, group: int, lens) -> int:
    arr = (c_int32 * len(lens))(*lens)
    return lib().freqkv_check_attend(ctypes.byref(layout), k_ptr, v_ptr, layer, q_ptr, out_ptr, group, arr)


def check_attend_prefill(layout: Layout, k_ptr: int, v_ptr: int, layer: int, q_ptr: int, out_ptr: int, group: int,
                         n_new: int, lens) -> int:
    arr = (c_int32 * len(lens))(*lens)
    return lib().freqkv_check_attend_prefill(ctypes.byref(layout), k_ptr, v_ptr, layer, q_ptr, out_ptr, group, n_new, arr)


def gemm_fold_levels(n_in: int, kept_len: int, first_component: int = 0) -> int:
    """``freqkv_gemm_fold_levels``: 0, 1 or 2 levels of the symmetry fold for these lengths (host only)."""
    return lib().freqkv_gemm_fold_levels(n_in, kept_len, first_component)


def fast_plan_apply_host(x, n_keep: int, family: int = 0):
    """``freqkv_fast_plan_apply_host``: the FDCT variant's factored chain applied in fp64 on the
    host to a float64 numpy array ``x`` [n_in, channels] (a plan diagnostic, not a compute path).
    ``family``: 0 = the kernel's own choice, ``COOLEY_TUKEY`` or ``PRIME_FACTOR``.
    Returns (y [n_keep, channels], (N1, N2, L1, L2, family used)); raises
    FreqKVError(ERR_UNSUPPORTED) when the lengths do not factor within the kernel's limits."""
    import numpy as np

    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty((n_keep, x.shape[1]), dtype=np.float64)
    fac = (c_int32 * 5)()
    st = lib().freqkv_fast_plan_apply_host(x.shape[0], n_keep, family, x.ctypes.data, x.shape[1], y.ctypes.data, fac)
    if st != OK:
        raise FreqKVError(st, f"freqkv_fast_plan_apply_host: {status_string(st)}")
    return y, tuple(fac)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def compress_noalloc(k: torch.Tensor, v: torch.Tensor, cache_len: int, kept_len: int, sink: int, stream=None) -> int:
    """``freqkv_compress_noalloc``: in-place compression without a context and without any
    device allocation, for callers that cannot call cudaMalloc (frozen memory budgets,
    frameworks that own all device memory).  Small shapes only: see the limits in ``include/freqkv.h``.  Returns the new
    cache length; raises FreqKVError (ERR_UNSUPPORTED beyond the size limits)."""
    lay = layout_of(k)
    if tuple(v.shape) != tuple(k.shape) or v.stride() != k.stride() or v.dtype != k.dtype:
        raise FreqKVError(ERR_INVALID_ARG, "K and V must share shape, strides and dtype")
    st = lib().freqkv_compress_noalloc(ctypes.byref(lay), k.data_ptr(), v.data_ptr(), cache_len, kept_len, sink,
                                       _stream_ptr(stream))
    if st != OK:
        raise FreqKVError(st, f"freqkv_compress_noalloc: {status_string(st)}")
    return sink + kept_len


class DecodeGraph:
    """``freqkv_decode_graph``: one decode step (device-side trigger, compression when the cache is
    full, append of the staged row) replayed as a CUDA graph.  ``lens`` is an int32 device tensor
    the graph updates; ``new_k`` / ``new_v`` are the staging rows the caller refills before ``launch``."""

    def __init__(self, ctx: "Context", k: torch.Tensor, v: torch.Tensor, new_k: torch.Tensor, new_v: torch.Tensor,
                 lens: torch.Tensor, kept_len: int, sink: int):
        lay = layout_of(k)
        if lens.dtype != torch.int32 or not lens.is_cuda or lens.numel() != lay.batch or not lens.is_contiguous():
            raise FreqKVError(ERR_INVALID_ARG, "lens must be a dense int32 device tensor with one entry per sequence")
        want = (k.shape[0], k.shape[1], k.shape[2], 1, k.shape[4])
        if tuple(new_k.shape) != want or tuple(new_v.shape) != want or not (new_k.is_contiguous() and new_v.is_contiguous()) \
                or new_k.dtype != k.dtype or new_v.dtype != k.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "staging rows must be dense [batch, layers, kv_heads, 1, head_dim] in the cache dtype")
        self._keep = (ctx, k, v, new_k, new_v, lens)   # the graph holds raw pointers into these
        self._h = c_void_p()
        st = lib().freqkv_decode_graph_create(ctx._h, ctypes.byref(lay), k.data_ptr(), v.data_ptr(), new_k.data_ptr(),
                                              new_v.data_ptr(), lens.data_ptr(), kept_len, sink, ctypes.byref(self._h))
        if st != OK:
            self._h = c_void_p()
            ctx._check(st, "freqkv_decode_graph_create")

    def launch(self, stream=None):
        st = lib().freqkv_decode_graph_launch(self._h, _stream_ptr(stream))
        if st != OK:
            raise FreqKVError(st, f"freqkv_decode_graph_launch: {status_string(st)}")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib().freqkv_decode_graph_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Context:
    """Owns one ``freqkv_ctx`` (plan cache, scratch, status word) on one device."""

    def __init__(self, device: int | None = None):
        if device is None:
            device = torch.cuda.current_device()
        self.device = int(device)
        self._h = c_void_p()
        st = lib().freqkv_create(ctypes.byref(self._h), self.device)
        if st != OK:
            self._h = c_void_p()
            raise FreqKVError(st, f"freqkv_create: {status_string(st)} (a B200 and the built library are required)")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            lib().freqkv_destroy(self._h)
            self._h = c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int, what: str):
        if st != OK:
            detail = lib().freqkv_last_error(self._h).decode() if st in (ERR_CUDA, ERR_ALLOC, ERR_TIMEOUT) else ""
            raise FreqKVError(st, f"{what}: {status_string(st)} {detail}".strip())

    def set_variant(self, variant: int):
        self._check(lib().freqkv_set_variant(self._h, variant), "freqkv_set_variant")

    def set_fast_family(self, family: int):
        self._check(lib().freqkv_set_fast_family(self._h, family), "freqkv_set_fast_family")

    def resolve_variant(self, layout: Layout, n_in: int, n_keep: int) -> int:
        out = c_int32(-1)
        st = lib().freqkv_resolve_variant(self._h, ctypes.byref(layout), n_in, n_keep, ctypes.byref(out))
        if st == ERR_UNSUPPORTED:
            return -1
        self._check(st, "freqkv_resolve_variant")
        return out.value

    def plan(self, n_in: int, n_keep: int, dtype: int, variant: int = AUTO, stream=None):
        self._check(lib().freqkv_plan(self._h, n_in, n_keep, dtype, variant, _stream_ptr(stream)), "freqkv_plan")

    def compress(self, k: torch.Tensor, v: torch.Tensor, cache_len: int, kept_len: int, sink: int, stream=None) -> int:
        """In-place compression of rows [sink, cache_len) of every matrix to kept_len rows.
        Returns the new cache length."""
        lay = layout_of(k)
        if tuple(v.shape) != tuple(k.shape) or v.stride() != k.stride() or v.dtype != k.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "K and V must share shape, strides and dtype")
        st = lib().freqkv_compress(self._h, ctypes.byref(lay), k.data_ptr(), v.data_ptr(), cache_len, kept_len, sink,
                                   _stream_ptr(stream))
        self._check(st, "freqkv_compress")
        return sink + kept_len

    def compress_band(self, k: torch.Tensor, v: torch.Tensor, cache_len: int, kept_len: int, sink: int,
                      first_component: int, stream=None) -> int:
        """Like ``compress`` but keeping DCT components ``first_component .. first_component +
        kept_len - 1`` (the high/low-frequency ablation).  Returns the new cache length."""
        lay = layout_of(k)
        if tuple(v.shape) != tuple(k.shape) or v.stride() != k.stride() or v.dtype != k.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "K and V must share shape, strides and dtype")
        st = lib().freqkv_compress_band(self._h, ctypes.byref(lay), k.data_ptr(), v.data_ptr(), cache_len, kept_len, sink,
                                        first_component, _stream_ptr(stream))
        self._check(st, "freqkv_compress_band")
        return sink + kept_len

    def power_spectrum(self, k: torch.Tensor, v: torch.Tensor, cache_len: int, sink: int, stream=None):
        """Average DCT power spectrum of rows [sink, cache_len) over batch and channels:
        (spectrum_k, spectrum_v), each fp32 ``[layers, kv_heads, cache_len - sink]`` on the cache's device."""
        lay = layout_of(k)
        if tuple(v.shape) != tuple(k.shape) or v.stride() != k.stride() or v.dtype != k.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "K and V must share shape, strides and dtype")
        n = max(cache_len - sink, 0)
        sk = torch.empty(lay.layers, lay.kv_heads, n, dtype=torch.float32, device=k.device)
        sv = torch.empty_like(sk)
        st = lib().freqkv_power_spectrum(self._h, ctypes.byref(lay), k.data_ptr(), v.data_ptr(), cache_len, sink,
                                         sk.data_ptr(), sv.data_ptr(), _stream_ptr(stream))
        self._check(st, "freqkv_power_spectrum")
        return sk, sv

    def compress_ragged(self, k: torch.Tensor, v: torch.Tensor, lens: list[int], kept_len: list[int], sink: int,
                        stream=None) -> list[int]:
        lay = layout_of(k)
        if tuple(v.shape) != tuple(k.shape) or v.stride() != k.stride() or v.dtype != k.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "K and V must share shape, strides and dtype")
        if len(lens) != lay.batch or len(kept_len) != lay.batch:
            raise FreqKVError(ERR_INVALID_ARG, "lens and kept_len need one entry per sequence")
        c_lens = (c_int32 * lay.batch)(*lens)
        c_keep = (c_int32 * lay.batch)(*kept_len)
        st = lib().freqkv_compress_ragged(self._h, ctypes.byref(lay), k.data_ptr(), v.data_ptr(), c_lens, c_keep, sink,
                                          _stream_ptr(stream))
        self._check(st, "freqkv_compress_ragged")
        return list(c_lens)

    def append(self, k: torch.Tensor, v: torch.Tensor, new_k: torch.Tensor, new_v: torch.Tensor, lens: list[int],
               stream=None) -> list[int]:
        """Append new_k / new_v ``[batch, layers, kv_heads, n_new, head_dim]`` (dense) at each
        sequence's length; returns the new lengths.  Raises FreqKVError(ERR_CAPACITY) when a
        sequence has no room: compress and retry."""
        lay = layout_of(k)
        if not (new_k.is_contiguous() and new_v.is_contiguous()) or new_k.shape != new_v.shape:
            raise FreqKVError(ERR_INVALID_ARG, "new_k / new_v must be dense and of equal shape")
        if tuple(new_k.shape[:3]) != tuple(k.shape[:3]) or new_k.shape[4] != k.shape[4] or new_k.dtype != k.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "new rows do not match the cache")
        n_new = new_k.shape[3]
        c_lens = (c_int32 * lay.batch)(*lens)
        st = lib().freqkv_append(self._h, ctypes.byref(lay), k.data_ptr(), v.data_ptr(), new_k.data_ptr(),
                                 new_v.data_ptr(), n_new, c_lens, _stream_ptr(stream))
        self._check(st, "freqkv_append")
        return list(c_lens)

    def attend_decode(self, k: torch.Tensor, v: torch.Tensor, layer: int, q: torch.Tensor, lens: list[int],
                      rope_base: float = 10000.0, scale: float = 0.0, out: torch.Tensor | None = None,
                      stream=None) -> torch.Tensor:
        """Attention of one new token per sequence over cache rows [0, lens[b]) of `layer`
        (keys rotated to their in-cache positions).  ``q``: dense [batch, q_heads, head_dim], cache
        dtype, before RoPE; q_heads must be a multiple of the cache's kv_heads.  Returns ``out``."""
        lay = layout_of(k)
        if tuple(v.shape) != tuple(k.shape) or v.stride() != k.stride() or v.dtype != k.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "K and V must share shape, strides and dtype")
        if q.dim() != 3 or not q.is_contiguous() or q.dtype != k.dtype or q.shape[0] != lay.batch or \
                q.shape[2] != lay.head_dim or q.shape[1] % lay.kv_heads != 0:
            raise FreqKVError(ERR_INVALID_ARG, "q must be dense [batch, q_heads, head_dim] in the cache dtype")
        if out is None:
            out = torch.empty_like(q)
        c_lens = (c_int32 * lay.batch)(*lens)
        st = lib().freqkv_attend_decode(self._h, ctypes.byref(lay), k.data_ptr(), v.data_ptr(), layer, q.data_ptr(),
                                        out.data_ptr(), q.shape[1] // lay.kv_heads, c_lens, rope_base, scale,
                                        _stream_ptr(stream))
        self._check(st, "freqkv_attend_decode")
        return out

    def attend_prefill(self, k: torch.Tensor, v: torch.Tensor, layer: int, q: torch.Tensor, lens: list[int],
                       rope_base: float = 10000.0, scale: float = 0.0, out: torch.Tensor | None = None,
                       stream=None) -> torch.Tensor:
        """Causal attention of a chunk of tokens, already appended as cache rows [lens[b] - n_new, lens[b])
        of `layer`, over rows [0, lens[b]) (keys and queries rotated to their in-cache positions).
        ``q``: dense [batch, q_heads, n_new, head_dim], bf16, before RoPE.  Returns ``out``."""
        lay = layout_of(k)
        if tuple(v.shape) != tuple(k.shape) or v.stride() != k.stride() or v.dtype != k.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "K and V must share shape, strides and dtype")
        if q.dim() != 4 or not q.is_contiguous() or q.dtype != k.dtype or q.shape[0] != lay.batch or \
                q.shape[3] != lay.head_dim or q.shape[1] % lay.kv_heads != 0:
            raise FreqKVError(ERR_INVALID_ARG, "q must be dense [batch, q_heads, n_new, head_dim] in the cache dtype")
        if out is None:
            out = torch.empty_like(q)
        c_lens = (c_int32 * lay.batch)(*lens)
        st = lib().freqkv_attend_prefill(self._h, ctypes.byref(lay), k.data_ptr(), v.data_ptr(), layer, q.data_ptr(),
                                         out.data_ptr(), q.shape[1] // lay.kv_heads, q.shape[2], c_lens, rope_base, scale,
                                         _stream_ptr(stream))
        self._check(st, "freqkv_attend_prefill")
        return out

    def compress_host(self, k_host: torch.Tensor, v_host: torch.Tensor, cache_len: int, kept_len: int, sink: int,
                      stream=None) -> tuple[int, int, int]:
        """Host-buffer form: K and V live in (pinned) host memory; the library copies the
        non-sink rows in, compresses on the device and copies the kept rows back, all enqueued
        on the stream.  Returns (new length, bytes host->device, bytes device->host)."""
        if k_host.is_cuda or v_host.is_cuda:
            raise FreqKVError(ERR_INVALID_ARG, "compress_host takes host tensors")
        lay = layout_of(k_host)
        if tuple(v_host.shape) != tuple(k_host.shape) or v_host.stride() != k_host.stride() or v_host.dtype != k_host.dtype:
            raise FreqKVError(ERR_INVALID_ARG, "K and V must share shape, strides and dtype")
        h2d, d2h = c_int64(0), c_int64(0)
        st = lib().freqkv_compress_host(self._h, ctypes.byref(lay), k_host.data_ptr(), v_host.data_ptr(), cache_len,
                                        kept_len, sink, _stream_ptr(stream), ctypes.byref(h2d), ctypes.byref(d2h))
        self._check(st, "freqkv_compress_host")
        return sink + kept_len, h2d.value, d2h.value

    def set_timing(self, enabled: bool):
        self._check(lib().freqkv_set_timing(self._h, 1 if enabled else 0), "freqkv_set_timing")

    def get_timing(self) -> tuple[int, float, int]:
        """(timed transform launches, their summed device ms, kernels launched since creation)."""
        n, ms, k = c_int64(0), ctypes.c_double(0.0), c_int64(0)
        self._check(lib().freqkv_get_timing(self._h, ctypes.byref(n), ctypes.byref(ms), ctypes.byref(k)), "freqkv_get_timing")
        return n.value, ms.value, k.value

    def set_wait_limit(self, nanoseconds: int):
        self._check(lib().freqkv_set_wait_limit(self._h, nanoseconds), "freqkv_set_wait_limit")

    def selftest_bounded_wait(self, nanoseconds: int, stream=None):
        """Enqueue the one-thread kernel whose bounded barrier wait runs out after `nanoseconds`."""
        self._check(lib().freqkv_selftest_bounded_wait(self._h, nanoseconds, _stream_ptr(stream)), "freqkv_selftest_bounded_wait")

    def last_error(self) -> str:
        return lib().freqkv_last_error(self._h).decode()

    def last_device_status(self, stream=None) -> int:
        return lib().freqkv_last_device_status(self._h, _stream_ptr(stream))
