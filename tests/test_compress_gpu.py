"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the
same seeded inputs.  Tolerances: relative L2 <= 1e-5 (fp32 caches), <= 1e-2 (bf16 caches),
worst matrix; every byte outside the rewritten rows bit-exact."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2505_00570_b200 import binding as fk
from paper_2505_00570_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = fk.Context(0)
    yield c
    c.close()


def small(name="t", B=1, Ly=2, H=2, hd=128, cap=512, dtype=torch.float32, sink=0, rho=0.9, outliers=0, seed=7):
    return synth.Workload(name, B, Ly, H, hd, cap, dtype, sink, rho, outliers, synth.BASE_SEED + seed)


# ---- config 1: tiny single-head fp32, 512 -> 256, no sinks
def test_config1_tiny_fp32(ctx):
    w = synth.WORKLOADS["tiny"]
    worst = parity.check_compress(ctx, w, 512, 256, 0, fk.AUTO)
    assert worst < 1e-5


@pytest.mark.parametrize("variant", [fk.SIMT])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n_in,kept", [(1, 1), (2, 1), (3, 2), (5, 2), (8, 4), (31, 15), (62, 31), (127, 63),
                                        (128, 64), (129, 64), (300, 150), (500, 125), (508, 381)])
def test_small_lengths(ctx, variant, dtype, n_in, kept):
    sink = 4
    w = small(cap=n_in + sink + 3, dtype=dtype, sink=sink, outliers=2 if dtype == torch.bfloat16 else 0)
    parity.check_compress(ctx, w, n_in + sink, kept, sink, variant)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_row_padding_and_canaries(ctx, dtype):
    w = small(cap=200, dtype=dtype, sink=4, B=2)
    parity.check_compress(ctx, w, 197, 96, 4, fk.SIMT, row_pad=8)


@pytest.mark.parametrize("hd", [64, 96, 256])
def test_other_head_dims(ctx, hd):
    w = small(cap=160, hd=hd, dtype=torch.bfloat16, sink=2)
    parity.check_compress(ctx, w, 150, 74, 2, fk.SIMT)


def test_degenerate_cases_write_nothing(ctx):
    w = small(cap=64, dtype=torch.bfloat16, sink=4)
    parity.check_compress(ctx, w, 64, 60, 4, fk.AUTO)   # identity
    parity.check_compress(ctx, w, 64, 0, 4, fk.AUTO)    # keep nothing
    parity.check_compress(ctx, w, 4, 0, 4, fk.AUTO)     # only sinks in the cache


def test_invalid_arguments_raise(ctx):
    k = torch.zeros(1, 1, 1, 64, 128, device="cuda", dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    with pytest.raises(fk.FreqKVError) as e:
        ctx.compress(k, v, 64, 61, 4)
    assert e.value.status == fk.ERR_INVALID_ARG
    with pytest.raises(fk.FreqKVError):
        ctx.compress(k, k, 64, 30, 4)
    with pytest.raises(fk.FreqKVError):
        ctx.compress(k, v.float(), 64, 30, 4)


# ---- config 2 shapes (LLaMA-2-7B: 4092 -> 2046, 4 sinks), a few heads, sampled matrices
def test_config2_shape_simt(ctx):
    w = dataclasses.replace(synth.WORKLOADS["llama2_7b"], layers=1, kv_heads=4)
    parity.check_compress(ctx, w, 4096, 2046, 4, fk.SIMT, sample=4)


# ---- append, the lazy trigger and a short iterative stream against the oracle
def test_append_rows_and_capacity(ctx):
    w = small(cap=40, dtype=torch.bfloat16, B=3, sink=4)
    k, v = synth.make_cache(w, "cuda", fill_len=0)
    k.fill_(1.5), v.fill_(-2.5)
    k0, v0 = k.clone(), v.clone()
    nk = torch.randn(3, 2, 2, 5, 128, device="cuda").to(torch.bfloat16)
    nv = torch.randn(3, 2, 2, 5, 128, device="cuda").to(torch.bfloat16)
    lens = ctx.append(k, v, nk, nv, [0, 7, 35])
    assert lens == [5, 12, 40]
    for b, start in enumerate([0, 7, 35]):
        assert torch.equal(k[b, :, :, start:start + 5], nk[b]) and torch.equal(v[b, :, :, start:start + 5], nv[b])
        keep = torch.ones(40, dtype=torch.bool)
        keep[start:start + 5] = False
        assert torch.equal(k[b][:, :, keep], k0[b][:, :, keep]) and torch.equal(v[b][:, :, keep], v0[b][:, :, keep])
    with pytest.raises(fk.FreqKVError) as e:
        ctx.append(k, v, nk, nv, [5, 12, 36])
    assert e.value.status == fk.ERR_CAPACITY
    assert torch.equal(k[2, :, :, 35:40], nk[2])  # a refused append wrote nothing


@pytest.mark.parametrize("dtype,row_pad", [(torch.bfloat16, 0), (torch.bfloat16, 8), (torch.float32, 0)])
def test_append_large_chunk(ctx, dtype, row_pad):
    """A prefill-sized chunk (hundreds of rows per matrix) takes the per-matrix copy kernel:
    rows land at each sequence's own length, every other byte (padding and canaries included)
    keeps its value."""
    w = small(cap=700, dtype=dtype, B=2, Ly=2, H=3, sink=4)
    (kbuf, k), (vbuf, v) = parity.guarded_cache(w, torch.device("cuda"), fill_len=700, row_pad=row_pad)
    kbuf0, vbuf0 = kbuf.clone(), vbuf.clone()
    n_new = 333
    nk = torch.randn(2, 2, 3, n_new, 128, device="cuda").to(dtype)
    nv = torch.randn(2, 2, 3, n_new, 128, device="cuda").to(dtype)
    starts = [0, 367]
    lens = ctx.append(k, v, nk, nv, starts)
    assert lens == [n_new, 700]
    for b, start in enumerate(starts):
        assert torch.equal(k[b, :, :, start:start + n_new], nk[b]) and torch.equal(v[b, :, :, start:start + n_new], nv[b])
    # restore the appended rows: the buffers must then equal their pre-call copies bit for bit
    k0 = kbuf0[parity.GUARD:parity.GUARD + k.shape[0] * k.shape[1] * k.shape[2] * 700 * (128 + row_pad)].view(2, 2, 3, 700, 128 + row_pad)[..., :128]
    v0 = vbuf0[parity.GUARD:parity.GUARD + k.shape[0] * k.shape[1] * k.shape[2] * 700 * (128 + row_pad)].view(2, 2, 3, 700, 128 + row_pad)[..., :128]
    for b, start in enumerate(starts):
        k[b, :, :, start:start + n_new] = k0[b, :, :, start:start + n_new]
        v[b, :, :, start:start + n_new] = v0[b, :, :, start:start + n_new]
    assert torch.equal(kbuf.view(torch.int16 if dtype == torch.bfloat16 else torch.int32),
                       kbuf0.view(torch.int16 if dtype == torch.bfloat16 else torch.int32))
    assert torch.equal(vbuf.view(torch.int16 if dtype == torch.bfloat16 else torch.int32),
                       vbuf0.view(torch.int16 if dtype == torch.bfloat16 else torch.int32))


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_iterative_stream_matches_oracle(ctx, dtype):
    """Tokens enter one at a time; a full cache is compressed to half its non-sink length
    before the next token goes in (Section 3.4).  The GPU cache is compared with the oracle's
    replay of the same stream after every compression."""
    cap, S, T, hd = 48, 4, 200, 64
    w = small(cap=cap, hd=hd, dtype=dtype, sink=S, Ly=1, H=2, B=2)
    ctx.set_variant(fk.AUTO)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed)
    scales = synth.channel_scales(w, gen, "cuda")
    k, v = synth.make_cache(w, "cuda", fill_len=0)
    toks_k, state_k = synth.ar1_rows(w, T, gen, "cuda", scales)
    toks_v, state_v = synth.ar1_rows(w, T, gen, "cuda", scales)
    lens = [0, 0]
    L = (cap - S) // 2
    count = 0
    for t in range(T):
        try:
            lens = ctx.append(k, v, toks_k[:, :, :, t:t + 1].contiguous(), toks_v[:, :, :, t:t + 1].contiguous(), lens)
        except fk.FreqKVError as e:
            assert e.status == fk.ERR_CAPACITY
            new_len = ctx.compress(k, v, cap, L, S)
            lens = [new_len, new_len]
            count += 1
            lens = ctx.append(k, v, toks_k[:, :, :, t:t + 1].contiguous(), toks_v[:, :, :, t:t + 1].contiguous(), lens)
    assert count == oracle.compression_count(T, cap, S, L)
    # oracle replay: it compresses its own fp64 state, so the gap grows with the number of
    # compressions by at most one rounding of the cache dtype each time
    tol = {torch.float32: 1e-5, torch.bfloat16: 1e-2}[dtype] * max(1, count) ** 0.5
    for b in range(2):
        for h in range(2):
            for cache_t, toks in ((k, toks_k), (v, toks_v)):
                want, n, c = oracle.stream(parity.to_f64(toks[b, 0, h]), cap, S, 0.5)
                assert n == lens[b] and c == count
                got = parity.to_f64(cache_t[b, 0, h, :n])
                assert np.array_equal(got[:S], want[:S])
                assert parity.rel_l2(got, want[:n]) < tol


def test_ragged_batch_small(ctx):
    """Sequences of different lengths, each compressed to half its own non-sink length."""
    w = small(cap=300, dtype=torch.bfloat16, sink=4, B=4, Ly=1, H=2, outliers=2)
    k, v = synth.make_cache(w, "cuda")
    k_in, v_in = k.clone(), v.clone()
    lens = [300, 41, 177, 177]
    kept = [(n - 4) // 2 for n in lens]
    ctx.set_variant(fk.AUTO)
    new_lens = ctx.compress_ragged(k, v, lens, kept, 4)
    assert new_lens == [4 + x for x in kept]
    for b in range(4):
        for h in range(2):
            for t_in, t_out in ((k_in, k), (v_in, v)):
                want = oracle.compress_matrix(parity.to_f64(t_in[b, 0, h, 4:lens[b]]), kept[b])
                got = parity.to_f64(t_out[b, 0, h, 4:4 + kept[b]])
                assert parity.rel_l2(got, want) < 1e-2
                assert torch.equal(t_out[b, 0, h, :4], t_in[b, 0, h, :4])
                assert torch.equal(t_out[b, 0, h, 4 + kept[b]:], t_in[b, 0, h, 4 + kept[b]:])


def test_ragged_batch_in_two_launches(ctx):
    """A ragged batch whose sequences all take the folded tensor-core form runs as ONE fold launch
    and ONE tensor-core launch (the kernel counter says so); odd and even lengths, one sequence
    left alone (kept == length), one with more than one tile of rows.  Against the oracle, against
    the bytes outside the rewritten rows, and against compressing each sequence on its own: bit
    for bit where that call runs the same arithmetic (one level of the symmetry fold), and to well
    inside the tolerance where the lengths halve twice and the single call folds twice."""
    w = small(cap=1400, dtype=torch.bfloat16, sink=4, B=6, Ly=2, H=3, outliers=2)
    k, v = synth.make_cache(w, "cuda")
    k_in, v_in = k.clone(), v.clone()
    lens = [1400, 523, 1101, 523, 700, 1337]
    kept = [(n - 4) // 2 for n in lens]
    kept[4] = 700 - 4          # identity: nothing to do for this sequence
    ctx.set_variant(fk.AUTO)
    before = ctx.get_timing()[2]
    new_lens = ctx.compress_ragged(k, v, lens, kept, 4)
    assert ctx.last_device_status() == fk.OK
    launched = ctx.get_timing()[2] - before
    assert new_lens == [4 + x for x in kept]
    plans = len({(n, kp) for n, kp in zip(lens, kept) if kp != n - 4})
    assert launched <= 2 + 2 * plans, f"{launched} kernels for the batch (2 + at most {2 * plans} plan builders expected)"
    before = ctx.get_timing()[2]
    k2, v2 = k_in.clone(), v_in.clone()
    assert ctx.compress_ragged(k2, v2, lens, kept, 4) == new_lens
    assert ctx.get_timing()[2] - before == 2          # plans cached: exactly the two launches
    assert torch.equal(k2, k) and torch.equal(v2, v)
    for b in range(6):
        one_k, one_v = k_in[b:b + 1].clone(), v_in[b:b + 1].clone()
        ctx.compress(one_k, one_v, lens[b], kept[b], 4)
        if (lens[b] - 4) % 4 == 0 and kept[b] % 2 == 0 and kept[b] > 256:   # the single call folds twice
            for one, both in ((one_k, k), (one_v, v)):
                a, c = one[0, :, :, 4:4 + kept[b]].double(), both[b, :, :, 4:4 + kept[b]].double()
                assert ((a - c).norm() / c.norm()).item() < 5e-3
                assert torch.equal(one[0, :, :, :4], both[b, :, :, :4]) and torch.equal(one[0, :, :, 4 + kept[b]:], both[b, :, :, 4 + kept[b]:])
        else:
            assert torch.equal(one_k[0], k[b]) and torch.equal(one_v[0], v[b]), f"sequence {b} differs from its own compression"
        for t_in, t_out in ((k_in, k), (v_in, v)):
            assert torch.equal(t_out[b, :, :, :4], t_in[b, :, :, :4])
            assert torch.equal(t_out[b, :, :, 4 + kept[b]:], t_in[b, :, :, 4 + kept[b]:])
            for (l, h) in ((0, 0), (1, 2)):
                want = oracle.compress_matrix(parity.to_f64(t_in[b, l, h, 4:lens[b]]), kept[b])
                parity.check_matrix(parity.to_f64(t_out[b, l, h, 4:4 + kept[b]]), want, torch.bfloat16, f"sequence {b}")


# ---- tensor-core projection (tcgen05 / TMEM / TMA), bf16 caches with head_dim 128
@pytest.mark.parametrize("n_in,kept,sink", [(128, 64, 0), (256, 128, 4), (300, 150, 4), (700, 350, 4), (1000, 999, 1),
                                            (1023, 511, 0), (1500, 100, 4), (64, 32, 2), (17, 5, 0)])
def test_gemm_lengths(ctx, n_in, kept, sink):
    w = small(cap=n_in + sink + 5, dtype=torch.bfloat16, sink=sink, outliers=2, Ly=1, H=2)
    parity.check_compress(ctx, w, n_in + sink, kept, sink, fk.GEMM)


@pytest.mark.parametrize("n_in,kept,sink", [(2048, 1024, 0), (4092, 2728, 4), (1396, 698, 4), (4092, 2046, 4), (2732, 1366, 0)])
def test_gemm_two_fold_levels(ctx, n_in, kept, sink):
    """Lengths that halve twice (n_in a multiple of 4, kept even) run the symmetry fold at two levels: a whole
    number of 256-row tiles (2048 -> 1024), a ragged last tile (2728 kept rows: 682 twice-folded ones), an odd
    kept / 2 whose middle row is its own mirror (698, 2046, 1366), several sequences, layers and heads, padded rows."""
    w = small(cap=n_in + sink + 3, dtype=torch.bfloat16, sink=sink, outliers=2, B=2, Ly=2, H=3)
    parity.check_compress(ctx, w, n_in + sink, kept, sink, fk.GEMM)
    parity.check_compress(ctx, w, n_in + sink, kept, sink, fk.GEMM, row_pad=8)


def test_gemm_batch_layers_heads_and_padding(ctx):
    w = small(cap=333, dtype=torch.bfloat16, sink=4, outliers=2, B=2, Ly=3, H=2)
    parity.check_compress(ctx, w, 330, 163, 4, fk.GEMM)
    parity.check_compress(ctx, w, 333, 164, 4, fk.GEMM, row_pad=8)


def test_gemm_many_tiles_more_than_sms(ctx):
    """More output tiles than SMs, so every CTA runs several tiles through its pipeline."""
    w = small(cap=600, dtype=torch.bfloat16, sink=4, outliers=2, B=1, Ly=8, H=16)
    parity.check_compress(ctx, w, 600, 298, 4, fk.GEMM, sample=24)


def test_config2_shape_gemm(ctx):
    w = dataclasses.replace(synth.WORKLOADS["llama2_7b"], layers=2, kv_heads=8)
    parity.check_compress(ctx, w, 4096, 2046, 4, fk.GEMM, sample=8)


def test_config3_shape_gemm(ctx):
    w = dataclasses.replace(synth.WORKLOADS["llama3_8b"], batch=2, layers=1, kv_heads=2)
    parity.check_compress(ctx, w, 8192, 4094, 4, fk.GEMM, sample=4)


def test_gemm_in_place_equals_fresh_copy(ctx):
    """Running on a cache and on a clone of it gives bit-identical results (no dependence on
    scheduling or on what the tiles of other matrices do)."""
    w = small(cap=520, dtype=torch.bfloat16, sink=4, outliers=2, B=1, Ly=4, H=4)
    k, v = synth.make_cache(w, "cuda")
    k2, v2 = k.clone(), v.clone()
    ctx.set_variant(fk.GEMM)
    ctx.compress(k, v, 520, 258, 4)
    ctx.compress(k2, v2, 520, 258, 4)
    assert ctx.last_device_status() == fk.OK
    assert torch.equal(k, k2) and torch.equal(v, v2)


def test_calls_on_two_streams_share_one_context_safely(ctx):
    """The context's scratch is shared: calls enqueued on different streams without any host
    synchronisation must still give the results of running them one after the other."""
    w = small(cap=1100, dtype=torch.bfloat16, sink=4, outliers=2, B=1, Ly=4, H=8)
    caches = [synth.make_cache(dataclasses.replace(w, seed=w.seed + i), "cuda") for i in range(4)]
    want = []
    ctx.set_variant(fk.GEMM)
    for k, v in caches:
        k2, v2 = k.clone(), v.clone()
        ctx.compress(k2, v2, 1100, 548, 4)
        want.append((k2, v2))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for i, (k, v) in enumerate(caches):
        with torch.cuda.stream(streams[i % 2]):
            ctx.compress(k, v, 1100, 548, 4, stream=streams[i % 2])
    torch.cuda.synchronize()
    ctx.set_variant(fk.AUTO)
    assert ctx.last_device_status() == fk.OK
    for (k, v), (k2, v2) in zip(caches, want):
        assert torch.equal(k, k2) and torch.equal(v, v2)


def test_permuted_strides_layer_outermost(ctx):
    """A cache stored layer-major ([layers, batch, heads, tokens, dim] in memory, presented as
    [batch, layers, ...]): compression, append and decode attention must follow the strides."""
    B, Ly, H, cap = 3, 2, 2, 300
    w = small(cap=cap, dtype=torch.bfloat16, sink=4, outliers=2, B=B, Ly=Ly, H=H)
    k0, v0 = synth.make_cache(w, "cuda")
    k = k0.permute(1, 0, 2, 3, 4).contiguous().permute(1, 0, 2, 3, 4)   # same values, layer-major storage
    v = v0.permute(1, 0, 2, 3, 4).contiguous().permute(1, 0, 2, 3, 4)
    assert k.stride(1) > k.stride(0) and torch.equal(k, k0)
    for variant in (fk.GEMM, fk.SIMT):
        ka, va, kb, vb = k.clone(memory_format=torch.preserve_format), v.clone(memory_format=torch.preserve_format), k0.clone(), v0.clone()
        assert ka.stride() == k.stride()
        ctx.set_variant(variant)
        ctx.compress(ka, va, cap, 148, 4)
        ctx.compress(kb, vb, cap, 148, 4)
        assert torch.equal(ka, kb) and torch.equal(va, vb)
    ctx.set_variant(fk.AUTO)
    nk = torch.randn(B, Ly, H, 7, 128, device="cuda").to(torch.bfloat16)
    ka, kb = k.clone(memory_format=torch.preserve_format), k0.clone()
    va, vb = v.clone(memory_format=torch.preserve_format), v0.clone()
    assert ctx.append(ka, va, nk, nk, [10, 200, 293]) == ctx.append(kb, vb, nk, nk, [10, 200, 293])
    assert torch.equal(ka, kb) and torch.equal(va, vb)
    q = torch.randn(B, H, 128, device="cuda").to(torch.bfloat16)
    assert torch.equal(ctx.attend_decode(ka, va, 1, q, [17, 207, 300]), ctx.attend_decode(kb, vb, 1, q, [17, 207, 300]))


# ---- other retention patterns: retaining ratios 0.25 / 0.75 / 1 %, and another band of components
@pytest.mark.parametrize("n_in,kept", [(4092, 1023), (4092, 3069), (4092, 40), (1000, 10)])
def test_other_retaining_ratios_gemm(ctx, n_in, kept):
    w = small(cap=n_in + 4, dtype=torch.bfloat16, sink=4, outliers=2, Ly=1, H=2)
    parity.check_compress(ctx, w, n_in + 4, kept, 4, fk.GEMM)


@pytest.mark.parametrize("variant,dtype", [(fk.GEMM, torch.bfloat16), (fk.SIMT, torch.float32), (fk.SIMT, torch.bfloat16)])
@pytest.mark.parametrize("n_in,kept,first", [(300, 150, 150), (300, 150, 75), (301, 150, 151), (257, 101, 33),
                                             (1024, 512, 512), (64, 63, 1), (700, 350, 0)])
def test_band_retention(ctx, variant, dtype, n_in, kept, first):
    """Components first .. first+kept-1 retained (first = n_in - kept: the highest frequencies);
    even and odd `first` take different signs in the tensor-core epilogue."""
    w = small(cap=n_in + 7, dtype=dtype, sink=4, outliers=2 if dtype == torch.bfloat16 else 0, Ly=2, H=2)
    if first == 0:
        parity.check_compress(ctx, w, n_in + 4, kept, 4, variant)
    else:
        parity.check_compress(ctx, w, n_in + 4, kept, 4, variant, first=first)


def test_band_config2_shape_high_frequencies(ctx):
    w = dataclasses.replace(synth.WORKLOADS["llama2_7b"], layers=1, kv_heads=4)
    parity.check_compress(ctx, w, 4096, 2046, 4, fk.AUTO, sample=4, first=2046)


@pytest.mark.parametrize("variant,dtype", [(fk.GEMM, torch.bfloat16), (fk.SIMT, torch.bfloat16), (fk.SIMT, torch.float32)])
@pytest.mark.parametrize("rho", [-0.9, 0.0])
@pytest.mark.parametrize("n_in,kept,first", [(300, 150, 150), (301, 150, 151), (1024, 512, 512), (1000, 333, 667), (700, 300, 201)])
def test_band_with_energy_in_the_band_plain_metric(ctx, variant, dtype, rho, n_in, kept, first):
    """Retaining High/Low-Frequency Components (the paper's ablation) on inputs that HAVE energy in
    the retained band -- an AR(1) process with rho = -0.9 (energy at the high frequencies) and white
    noise (rho = 0) -- held to the plain metric |Y_gpu - Y_oracle| / |Y_oracle| <= 1e-2 (bf16),
    1e-5 (fp32); even and odd first components (opposite signs in the tensor-core epilogue)."""
    w = small(cap=n_in + 7, dtype=dtype, sink=4, rho=rho, outliers=2 if dtype == torch.bfloat16 else 0, Ly=2, H=2)
    parity.check_compress(ctx, w, n_in + 4, kept, 4, variant, first=first, band_plain=True)


@pytest.mark.parametrize("rho", [-0.9, 0.0])
def test_band_config2_shape_high_frequencies_plain_metric(ctx, rho):
    """The highest 2046 of 4092 components on the 7B shape, input energy in that band, plain metric."""
    w = dataclasses.replace(synth.WORKLOADS["llama2_7b"], layers=1, kv_heads=4, rho=rho)
    parity.check_compress(ctx, w, 4096, 2046, 4, fk.AUTO, sample=8, first=2046, band_plain=True)


def test_band_invalid_and_fast_transform(ctx):
    k = torch.zeros(1, 1, 1, 600, 128, device="cuda", dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    ctx.set_variant(fk.AUTO)
    for first in (-1, 257):
        with pytest.raises(fk.FreqKVError) as e:
            ctx.compress_band(k, v, 516, 256, 4, first)
        assert e.value.status == fk.ERR_INVALID_ARG
    ctx.set_variant(fk.FDCT)
    with pytest.raises(fk.FreqKVError) as e:
        ctx.compress_band(k, v, 516, 256, 4, 256)
    assert e.value.status == fk.ERR_UNSUPPORTED
    ctx.set_variant(fk.AUTO)


# ---- host-buffer entry point: cache in host memory, copies pipelined with the compression
@pytest.mark.parametrize("layers,pinned", [(3, True), (20, True), (5, False)])
def test_compress_host_matches_device_path(ctx, layers, pinned):
    """Same bits as freqkv_compress on a device copy; rows outside [sink, sink+kept) of the host
    cache untouched; byte counts are those of the rows moved."""
    w = small(cap=300, dtype=torch.bfloat16, sink=4, outliers=2, B=2, Ly=layers, H=2)
    k, v = synth.make_cache(w, "cuda")
    kh, vh = k.cpu(), v.cpu()
    if pinned:
        kh, vh = kh.pin_memory(), vh.pin_memory()
    kh0, vh0 = kh.clone(), vh.clone()
    ctx.set_variant(fk.AUTO)
    new_len, h2d, d2h = ctx.compress_host(kh, vh, 300, 148, 4)
    torch.cuda.synchronize()
    assert ctx.last_device_status() == fk.OK and new_len == 152
    rows = 2 * 2 * layers * 2  # tensors x batch x layers x heads
    assert h2d == rows * 296 * 128 * 2 and d2h == rows * 148 * 128 * 2
    ctx.compress(k, v, 300, 148, 4)
    assert torch.equal(kh, k.cpu()) and torch.equal(vh, v.cpu())
    for t, t0 in ((kh, kh0), (vh, vh0)):
        assert torch.equal(t[..., :4, :], t0[..., :4, :]) and torch.equal(t[..., 152:, :], t0[..., 152:, :])
    want = oracle.compress_matrix(parity.to_f64(kh0[1, layers - 1, 1, 4:300]), 148)
    assert parity.rel_l2(parity.to_f64(kh[1, layers - 1, 1, 4:152]), want) < 1e-2


# ---- fast-transform variant (power-of-two lengths), in place without scratch
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("n_in,kept,sink", [(128, 64, 0), (256, 128, 4), (512, 256, 0), (1024, 128, 4), (2048, 16, 1),
                                            (2048, 1024, 4), (4096, 2048, 0), (4096, 512, 4), (8192, 4096, 4)])
def test_fdct_lengths(ctx, dtype, n_in, kept, sink):
    w = small(cap=n_in + sink + 3, dtype=dtype, sink=sink, outliers=2 if dtype == torch.bfloat16 else 0, Ly=1, H=2)
    parity.check_compress(ctx, w, n_in + sink, kept, sink, fk.FDCT)


def test_fdct_row_padding_batch_and_head_dim(ctx):
    w = small(cap=520, dtype=torch.bfloat16, sink=4, outliers=2, B=2, Ly=2, H=2)
    parity.check_compress(ctx, w, 516, 256, 4, fk.FDCT, row_pad=8)
    w64 = small(cap=256, hd=64, dtype=torch.float32, sink=0, B=1, Ly=1, H=3)
    parity.check_compress(ctx, w64, 256, 128, 0, fk.FDCT)


def test_fdct_refuses_other_lengths(ctx):
    k = torch.zeros(1, 1, 1, 600, 128, device="cuda", dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    ctx.set_variant(fk.FDCT)
    with pytest.raises(fk.FreqKVError) as e:
        ctx.compress(k, v, 591, 250, 4)      # 587 rows: a prime has no factorisation for the tensor-core stages
    assert e.value.status == fk.ERR_UNSUPPORTED
    kf, vf = k.float(), v.float()
    with pytest.raises(fk.FreqKVError) as e:
        ctx.compress(kf, vf, 504, 250, 4)    # fp32: the radix-16 kernel takes powers of two only
    assert e.value.status == fk.ERR_UNSUPPORTED
    ctx.set_variant(fk.AUTO)


def test_config2_pow2_shape_fdct(ctx):
    w = dataclasses.replace(synth.WORKLOADS["llama2_7b_pow2"], layers=2, kv_heads=8)
    parity.check_compress(ctx, w, 4096, 2048, 0, fk.FDCT, sample=8)


def test_auto_picks_documented_variants(ctx):
    ctx.set_variant(fk.AUTO)
    bf = fk.layout_contiguous(fk.BF16, 1, 1, 1, 8192, 128)[1]
    f32 = fk.layout_contiguous(fk.F32, 1, 1, 1, 8192, 128)[1]
    assert ctx.resolve_variant(bf, 4096, 2048) == fk.GEMM
    assert ctx.resolve_variant(fk.layout_contiguous(fk.BF16, 1, 1, 1, 8192, 64)[1], 4096, 2048) == fk.FDCT
    assert ctx.resolve_variant(bf, 4092, 2046) == fk.GEMM
    assert ctx.resolve_variant(fk.layout_contiguous(fk.BF16, 1, 1, 1, 8192, 64)[1], 4092, 2046) == fk.FDCT    # tensor-core stages
    assert ctx.resolve_variant(fk.layout_contiguous(fk.BF16, 1, 1, 1, 8192, 256)[1], 4099, 2049) == fk.SIMT   # a prime length
    assert ctx.resolve_variant(bf, 8188, 4094) == fk.GEMM
    assert ctx.resolve_variant(f32, 512, 256) == fk.FDCT
    assert ctx.resolve_variant(f32, 500, 250) == fk.SIMT
    assert ctx.resolve_variant(bf, 100, 50) == fk.SIMT
