"""Helpers shared by the GPU parity tests: run the CUDA path through the C ABI on a seeded
cache surrounded by canaries and compare it with the CPU oracle on the same bits."""
from __future__ import annotations

import numpy as np
import torch

import oracle
from paper_2505_00570_b200 import binding as fk
from paper_2505_00570_b200 import synth

TOL = {torch.float32: 1e-5, torch.bfloat16: 1e-2}  # max per-matrix relative L2 (the stated tolerances)
# A matrix norm over a few hundred thousand values cannot see one bad row or one bad 16-byte
# vector, so every row is bounded too: |got_row - want_row| <= ROW_TOL * max(|want_row|, rms row
# norm of the matrix).  Three times the matrix bar: a row's error is a sum over the same number of
# rounded terms as any other, and single rows scatter around the matrix average.
ROW_TOL = {torch.float32: 3e-5, torch.bfloat16: 3e-2}
GUARD = 4096  # canary elements before and after each tensor


def guarded_cache(w: synth.Workload, device, fill_len=None, row_pad: int = 0, batch=None):
    """K and V as views into larger buffers: canaries before and after, and (row_pad > 0)
    padding elements after every row, all of which must survive a call bit for bit."""
    k0, v0 = synth.make_cache(w, device, fill_len=fill_len, batch=batch)
    out = []
    for t in (k0, v0):
        B, Ly, H, cap, hd = t.shape
        st = hd + row_pad
        n = B * Ly * H * cap * st
        buf = torch.empty(n + 2 * GUARD, dtype=t.dtype, device=device)
        buf.fill_(-7.0)  # canary value
        view = buf[GUARD:GUARD + n].view(B, Ly, H, cap, st)[..., :hd]
        view.copy_(t)
        out.append((buf, view))
    return out[0], out[1]


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def rel_l2(got: np.ndarray, want: np.ndarray) -> float:
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


def row_error(got: np.ndarray, want: np.ndarray) -> float:
    """Worst row of a matrix: |got_row - want_row| / max(|want_row|, rms row norm of `want`)."""
    if want.size == 0:
        return 0.0
    rows = np.linalg.norm(want, axis=1)
    floor = max(float(np.sqrt(np.mean(rows * rows))), 1e-300)
    return float(np.max(np.linalg.norm(got - want, axis=1) / np.maximum(rows, floor)))


def channel_error(got: np.ndarray, want: np.ndarray) -> float:
    """Worst channel (column) of a matrix, relative L2 against the channel's own norm (reported,
    not gated: a channel that holds almost no energy in the kept band has no meaningful ratio)."""
    if want.size == 0:
        return 0.0
    cols = np.linalg.norm(want, axis=0)
    floor = max(float(np.sqrt(np.mean(cols * cols))), 1e-300)
    return float(np.max(np.linalg.norm(got - want, axis=0) / np.maximum(cols, 1e-3 * floor)))


def check_matrix(got: np.ndarray, want: np.ndarray, dtype, what: str = "") -> tuple[float, float, float]:
    """Gate one output matrix: relative L2 over the matrix and the per-row bound.  Returns
    (matrix error, worst row, worst channel)."""
    m, r, c = rel_l2(got, want), row_error(got, want), channel_error(got, want)
    assert m <= TOL[dtype], f"{what}: relative L2 {m:.3e} exceeds {TOL[dtype]:.0e}"
    assert r <= ROW_TOL[dtype], f"{what}: worst row {r:.3e} exceeds {ROW_TOL[dtype]:.0e} (matrix {m:.3e})"
    return m, r, c


def check_compress(ctx: fk.Context, w: synth.Workload, cache_len: int, kept_len: int, sink: int, variant: int,
                   row_pad: int = 0, sample: int | None = None, batch=None, first: int = 0, band_plain: bool = False,
                   energy_scaled: bool = False):
    """Compress on the GPU, then check (1) every byte outside rows [sink, sink+kept_len) is
    unchanged, canaries and padding included, (2) the rewritten rows match the oracle matrix by
    matrix within the tolerance of the dtype.  Returns the worst relative L2."""
    dev = torch.device("cuda", ctx.device)
    (kbuf, k), (vbuf, v) = guarded_cache(w, dev, fill_len=cache_len, row_pad=row_pad, batch=batch)
    kbuf0, vbuf0 = kbuf.clone(), vbuf.clone()
    k_in, v_in = k.clone(), v.clone()
    ctx.set_variant(variant)
    if first:
        new_len = ctx.compress_band(k, v, cache_len, kept_len, sink, first)  # components first .. first+kept_len-1
    else:
        new_len = ctx.compress(k, v, cache_len, kept_len, sink)
    assert ctx.last_device_status() == fk.OK
    assert new_len == sink + kept_len

    # (1) bit-exact outside the rewritten rows
    for buf, buf0, t in ((kbuf, kbuf0, k), (vbuf, vbuf0, v)):
        mask_src = torch.zeros_like(t, dtype=torch.bool)
        mask_src[..., sink:sink + kept_len, :] = True
        B, Ly, H, cap, hd = t.shape
        st = hd + row_pad
        full = torch.zeros(buf.numel(), dtype=torch.bool, device=dev)
        full[GUARD:GUARD + B * Ly * H * cap * st].view(B, Ly, H, cap, st)[..., :hd].copy_(mask_src)
        raw, raw0 = buf.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32), \
            buf0.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32)
        assert torch.equal(raw[~full], raw0[~full]), "bytes outside rows [sink, sink+kept_len) changed"

    # (2) oracle parity on all (or a seeded sample of) matrices
    n_mat = 2 * k.shape[0] * k.shape[1] * k.shape[2]
    ids = range(n_mat) if sample is None else synth.sample_matrix_ids(n_mat, sample, w.seed + 5)
    worst = worst_row = worst_channel = plain_band = 0.0
    n_in = cache_len - sink
    per = n_mat // 2
    for i in ids:
        t_in, t_out = (k_in, k) if i < per else (v_in, v)
        j = i % per
        b, l, h = j // (k.shape[1] * k.shape[2]), (j // k.shape[2]) % k.shape[1], j % k.shape[2]
        x = to_f64(t_in[b, l, h, sink:sink + n_in])
        want = oracle.compress_band_matrix(x, kept_len, first) if first else oracle.compress_matrix(x, kept_len)
        got = to_f64(t_out[b, l, h, sink:sink + kept_len])
        if kept_len == n_in:
            assert np.array_equal(got, x)  # identity must be bit-exact
        if first:
            # a band away from the low frequencies holds little of an AR(1) signal's energy, while the
            # rounding errors of the inputs scale with the whole signal: the error is measured against
            # the norm the output would have if the energy were spread evenly over the spectrum
            scale = max(np.linalg.norm(want), np.sqrt(kept_len / n_in) * np.linalg.norm(x))
            worst = max(worst, float(np.linalg.norm(got - want) / scale))
            plain_band = max(plain_band, rel_l2(got, want))
            if band_plain:  # the input has energy in the retained band: the plain metric itself
                worst = max(worst, rel_l2(got, want))
        elif energy_scaled:
            # an input with almost no energy in the kept band (the opposite of the paper's workloads):
            # same scaled metric as for a band away from the signal's energy
            scale = max(np.linalg.norm(want), np.sqrt(kept_len / n_in) * np.linalg.norm(x))
            worst = max(worst, float(np.linalg.norm(got - want) / scale))
            plain_band = max(plain_band, rel_l2(got, want))
        else:
            worst = max(worst, rel_l2(got, want))
            worst_row = max(worst_row, row_error(got, want))
            worst_channel = max(worst_channel, channel_error(got, want))
    if first or energy_scaled:
        print(f"band {first}..{first + kept_len - 1} of {n_in}: scaled metric {worst:.3e}, plain relative L2 {plain_band:.3e}")
    else:
        print(f"{n_in}->{kept_len}: matrix {worst:.3e}, worst row {worst_row:.3e}, worst channel {worst_channel:.3e}")
    assert worst <= TOL[w.dtype], f"relative L2 {worst:.3e} exceeds {TOL[w.dtype]:.0e}"
    assert worst_row <= ROW_TOL[w.dtype], f"worst row {worst_row:.3e} exceeds {ROW_TOL[w.dtype]:.0e}"
    return worst
