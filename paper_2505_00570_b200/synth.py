"""Seeded synthetic KV caches shaped like the paper's workloads.

The paper's inputs are key/value states of LLaMA-2/3 on text corpora; neither weights nor
data are available, so caches are drawn from a generator with the property the paper's
power-spectrum figures show: energy concentrated at low frequencies along the token axis.
Every channel is an AR(1) Gaussian sequence along tokens,

    x_0 = e_0,   x_n = rho * x_{n-1} + sqrt(1 - rho^2) * e_n,   e_n ~ N(0, 1) i.i.d.,

(unit stationary variance), multiplied by a per-channel scale drawn from U[0.5, 2]; a few
channels per (layer, kv_head) are outliers with their scale multiplied by 8.

This module holds input generation only -- none of the method's arithmetic -- and serves
both the CUDA path's tests/bench and the CPU oracle's tests.  It does not load the CUDA
library.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

BASE_SEED = 20250500


@dataclass(frozen=True)
class Workload:
    """One of the benchmark/test configurations."""

    name: str
    batch: int
    layers: int
    kv_heads: int
    head_dim: int
    capacity: int
    dtype: torch.dtype
    sink: int
    rho: float
    outliers: int  # outlier channels per (layer, kv_head)
    seed: int

    @property
    def n_matrices(self) -> int:
        """Independent [tokens, head_dim] matrices per call (K and V counted)."""
        return 2 * self.batch * self.layers * self.kv_heads

    def kept_len(self, cache_len: int, retain: float = 0.5) -> int:
        """L = floor(retain * (cache_len - sink))."""
        return int((cache_len - self.sink) * retain)


WORKLOADS = {
    # config 1: tiny single-head fp32, 512 -> 256, no sinks, no outliers
    "tiny": Workload("tiny", 1, 1, 1, 128, 512, torch.float32, 0, 0.9, 0, BASE_SEED + 1),
    # config 2: LLaMA-2-7B-shaped, cap 4096, 4 sinks, 4092 -> 2046 (the headline)
    "llama2_7b": Workload("llama2_7b", 1, 32, 32, 128, 4096, torch.bfloat16, 4, 0.9, 2, BASE_SEED + 2),
    # config 2': the literal power-of-two shape 4096 -> 2048, no sinks
    "llama2_7b_pow2": Workload("llama2_7b_pow2", 1, 32, 32, 128, 4096, torch.bfloat16, 0, 0.9, 2, BASE_SEED + 2),
    # config 3: LLaMA-3-8B-shaped GQA, batch 8, cap 8192, 8188 -> 4094
    "llama3_8b": Workload("llama3_8b", 8, 32, 8, 128, 8192, torch.bfloat16, 4, 0.95, 2, BASE_SEED + 3),
    # config 4: decode stream, LLaMA-2-7B shapes, batch 16
    "stream_7b": Workload("stream_7b", 16, 32, 32, 128, 4096, torch.bfloat16, 4, 0.9, 2, BASE_SEED + 4),
    # config 5a: chunked prefill, LLaMA-2-7B shapes, batch 1
    "prefill_7b": Workload("prefill_7b", 1, 32, 32, 128, 4096, torch.bfloat16, 4, 0.9, 2, BASE_SEED + 5),
    # config 5b: ragged batch 32, 32 layers x 8 KV heads, lengths U{1024..8192}
    "ragged_8b": Workload("ragged_8b", 32, 32, 8, 128, 8192, torch.bfloat16, 4, 0.9, 2, BASE_SEED + 6),
}


def channel_scales(w: Workload, gen: torch.Generator, device) -> torch.Tensor:
    """Per-channel scales [layers, kv_heads, head_dim]: U[0.5, 2], outliers x8."""
    s = 0.5 + 1.5 * torch.rand(w.layers, w.kv_heads, w.head_dim, generator=gen, device=device)
    if w.outliers > 0:
        pick = torch.rand(w.layers, w.kv_heads, w.head_dim, generator=gen, device=device)
        idx = pick.topk(w.outliers, dim=-1).indices
        s.scatter_(-1, idx, s.gather(-1, idx) * 8.0)
    return s


def ar1_rows(
    w: Workload,
    n_tokens: int,
    gen: torch.Generator,
    device,
    scales: torch.Tensor,
    state: torch.Tensor | None = None,
    batch: int | None = None,
) -> tuple[torch.Tensor, torch.Tensor]:
    """Next ``n_tokens`` rows of the AR(1) process for every (batch, layer, kv_head).

    Returns ``(rows [batch, layers, kv_heads, n_tokens, head_dim] in w.dtype, state)``;
    pass ``state`` back in to continue the same sequences (None starts them).
    """
    b = w.batch if batch is None else batch
    cols = b * w.layers * w.kv_heads * w.head_dim
    out = torch.empty((b, w.layers, w.kv_heads, n_tokens, w.head_dim), dtype=w.dtype, device=device)
    innov = (1.0 - w.rho * w.rho) ** 0.5
    # The recursion runs a block of tokens at a time as one matrix product: inside a block
    #   x_j = rho^(j+1) * x_prev + innov * sum_{i <= j} rho^(j-i) * e_i
    # (a lower-triangular Toeplitz matrix applied to the block's innovations), so a block costs
    # a handful of launches instead of a few per token.  Block size bounded by memory.
    block = max(16, min(1024, (1 << 28) // max(cols, 1)))
    steps = torch.arange(block, device=device, dtype=torch.float64)
    lag = steps[:, None] - steps[None, :]
    toeplitz = torch.where(lag >= 0, innov * torch.pow(torch.tensor(w.rho, dtype=torch.float64, device=device), lag.clamp(min=0)),
                           torch.zeros((), dtype=torch.float64, device=device)).to(torch.float32)
    carry = torch.pow(torch.tensor(w.rho, dtype=torch.float64, device=device), steps + 1).to(torch.float32)
    n0 = 0
    while n0 < n_tokens:
        nb = min(block, n_tokens - n0)
        eps = torch.randn((nb, cols), generator=gen, device=device, dtype=torch.float32)
        if state is None:
            # the very first token is the stationary draw itself: x_0 = e_0
            state = eps[0].clone()
            x = torch.empty_like(eps)
            x[0] = state
            if nb > 1:
                x[1:] = toeplitz[:nb - 1, :nb - 1] @ eps[1:] + carry[:nb - 1, None] * state[None, :]
        else:
            x = toeplitz[:nb, :nb] @ eps + carry[:nb, None] * state.reshape(-1)[None, :]
        state = x[nb - 1].clone()
        scaled = x.view(nb, b, w.layers, w.kv_heads, w.head_dim) * scales
        out[:, :, :, n0:n0 + nb, :] = scaled.permute(1, 2, 3, 0, 4).to(w.dtype)
        n0 += nb
    if state is not None:
        state = state.view(b, w.layers, w.kv_heads, w.head_dim)
    return out, state


def make_cache(
    w: Workload,
    device="cpu",
    fill_len: int | None = None,
    seed_offset: int = 0,
    batch: int | None = None,
) -> tuple[torch.Tensor, torch.Tensor]:
    """K and V caches ``[batch, layers, kv_heads, capacity, head_dim]`` with the first
    ``fill_len`` (default: capacity) rows drawn from the generator and the rest zero."""
    b = w.batch if batch is None else batch
    n = w.capacity if fill_len is None else fill_len
    caches = []
    for which in range(2):  # 0 = K, 1 = V: independent draws
        gen = torch.Generator(device=device)
        gen.manual_seed(w.seed + 1000 * which + seed_offset)
        scales = channel_scales(w, gen, device)
        cache = torch.zeros((b, w.layers, w.kv_heads, w.capacity, w.head_dim), dtype=w.dtype, device=device)
        rows, _ = ar1_rows(w, n, gen, device, scales, batch=b)
        cache[:, :, :, :n, :] = rows
        caches.append(cache)
    return caches[0], caches[1]


def ragged_lengths(w: Workload, lo: int = 1024, hi: int = 8192) -> list[int]:
    """Seeded per-sequence cache lengths, uniform on [lo, hi]."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(w.seed + 77)
    return torch.randint(lo, hi + 1, (w.batch,), generator=gen).tolist()


def sample_matrix_ids(n_matrices: int, count: int, seed: int) -> list[int]:
    """Seeded sample of matrix indices, always holding the first and the last."""
    gen = torch.Generator(device="cpu")
    gen.manual_seed(seed)
    ids = {0, n_matrices - 1}
    if n_matrices > 2:
        perm = torch.randperm(n_matrices, generator=gen).tolist()
        for i in perm:
            if len(ids) >= min(count, n_matrices):
                break
            ids.add(i)
    return sorted(ids)
