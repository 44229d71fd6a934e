"""GPU parity of freqkv_attend_prefill (causal attention of a chunk of incoming tokens over the
bounded cache, RoPE at in-cache positions; Section 3.3, chunk-wise prefilling) against the fp64
oracle of oracle/attention.py on the same seeded inputs.

Tolerance, per query head and query token, relative L2 of the 128 output channels: 1e-2.  The
output is rounded once to bf16 (2^-9); the rotated keys and the scaled queries are rounded to fp16
(2^-12 each, score errors of a few 1e-3 at most for scores of magnitude 10-20), the softmax weights
to bf16 before the second product (2^-9 each, averaged over the attended rows)."""
import numpy as np
import pytest
import torch

import oracle
from oracle import attention as oa
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


def workload(B, Ly, H, cap, seed=21):
    return synth.Workload("prefill_attn", B, Ly, H, 128, cap, torch.bfloat16, 4, 0.9, 2, synth.BASE_SEED + seed)


def queries(B, heads, n, seed):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    return torch.randn(B, heads, n, 128, generator=gen, device="cuda").to(torch.bfloat16)


def check(ctx, k, v, layer, q, lens, base, scale=0.0, heads=None, tokens=None):
    """Compare sampled (sequence, KV head) groups and chunk tokens with the oracle; token i of the
    chunk is the decoding step of the cache of length lens[b] - n + i + 1."""
    out = ctx.attend_prefill(k, v, layer, q, lens, rope_base=base, scale=scale)
    assert ctx.last_device_status() == fk.OK
    B, Hq, n = q.shape[0], q.shape[1], q.shape[2]
    G = Hq // k.shape[2]
    pick = heads if heads is not None else [(b, h) for b in range(B) for h in range(k.shape[2])]
    worst = 0.0
    for b, h in pick:
        K, V = parity.to_f64(k[b, layer, h]), parity.to_f64(v[b, layer, h])
        Q, got = parity.to_f64(q[b, h * G:(h + 1) * G]), parity.to_f64(out[b, h * G:(h + 1) * G])
        rows = range(n) if tokens is None else sorted({i for i in tokens if 0 <= i < n})
        for i in rows:
            want = oa.attend_decode(Q[:, i], K, V, lens[b] - n + i + 1, base, None if scale <= 0 else scale)
            for g in range(G):
                worst = max(worst, parity.rel_l2(got[g, i], want[g]))
    assert np.isfinite(parity.to_f64(out)).all()
    assert worst <= TOL, f"relative L2 {worst:.3e}"
    return worst


SPOTS = (0, 1, 30, 31, 32, 63, 64, 99, 126, 127, 128, 129, 199, 255, 256, 257)


@pytest.mark.parametrize("G", [1, 4])
def test_prefill_small_every_head_two_query_tiles_three_key_tiles(ctx, G):
    w = workload(2, 2, 2, 384)
    k, v = synth.make_cache(w, "cuda")
    k0, v0 = k.clone(), v.clone()
    q = queries(2, 2 * G, 200, 40 + G)
    check(ctx, k, v, 1, q, [300, 237], 10000.0, tokens=SPOTS + (150, 198))
    assert torch.equal(k, k0) and torch.equal(v, v0)  # the cache is only read


def test_prefill_whole_oracle_function_on_a_tiny_chunk(ctx):
    w = workload(1, 1, 1, 128, seed=22)
    k, v = synth.make_cache(w, "cuda")
    q = queries(1, 2, 9, 5)
    out = ctx.attend_prefill(k, v, 0, q, [50], rope_base=10000.0)
    want = oa.attend_prefill(parity.to_f64(q[0]), parity.to_f64(k[0, 0, 0]), parity.to_f64(v[0, 0, 0]), 50, 10000.0)
    got = parity.to_f64(out[0])
    assert max(parity.rel_l2(got[g, i], want[g, i]) for g in range(2) for i in range(9)) <= TOL


def test_prefill_chunk_is_the_whole_cache(ctx):
    """No history: token 0 sees only itself, so its output is its own value row."""
    w = workload(1, 1, 2, 256, seed=23)
    k, v = synth.make_cache(w, "cuda")
    q = queries(1, 2, 256, 6)
    out = ctx.attend_prefill(k, v, 0, q, [256], rope_base=10000.0)
    assert torch.equal(out[0, :, 0], v[0, 0, :, 0])
    check(ctx, k, v, 0, q, [256], 10000.0, tokens=SPOTS)


def test_prefill_one_token_is_the_decoding_step(ctx):
    w = workload(2, 1, 2, 300, seed=24)
    k, v = synth.make_cache(w, "cuda")
    q = queries(2, 4, 1, 7)
    lens = [300, 129]
    out = ctx.attend_prefill(k, v, 0, q, lens, rope_base=10000.0)
    dec = ctx.attend_decode(k, v, 0, q[:, :, 0].contiguous(), lens, rope_base=10000.0)
    assert parity.rel_l2(parity.to_f64(out[:, :, 0]), parity.to_f64(dec)) < 5e-3
    check(ctx, k, v, 0, q, lens, 10000.0)


@pytest.mark.parametrize("base,scale", [(0.0, 0.0), (500000.0, 0.05), (10000.0, 0.2)])
def test_prefill_rope_off_other_base_and_scale(ctx, base, scale):
    w = workload(1, 2, 3, 200, seed=25)
    k, v = synth.make_cache(w, "cuda")
    check(ctx, k, v, 1, queries(1, 6, 70, 3), [199], base, scale=scale, tokens=(0, 1, 35, 68, 69))


def test_prefill_stale_rows_past_the_length_may_hold_anything(ctx):
    """Rows at and after the length are never attended; NaN there must not reach any output.
    The cache rows carry padding and canaries, which must survive the call."""
    w = workload(1, 1, 2, 512, seed=26)
    (kbuf, k), (vbuf, v) = parity.guarded_cache(w, torch.device("cuda"), fill_len=512, row_pad=8)
    q = queries(1, 4, 131, 8)
    for n_len in (131, 200, 256, 257, 385, 511):
        k[:, :, :, n_len:] = float("nan")
        v[:, :, :, n_len:] = float("nan")
        kb, vb = kbuf.clone(), vbuf.clone()
        check(ctx, k, v, 0, q, [n_len], 10000.0, tokens=(0, 1, 64, 127, 128, 129, 130))
        assert torch.equal(kbuf.view(torch.int16), kb.view(torch.int16)) and torch.equal(vbuf.view(torch.int16), vb.view(torch.int16))
        k2, v2 = synth.make_cache(w, "cuda")
        k.copy_(k2)
        v.copy_(v2)


def test_prefill_known_answers_on_the_gpu_result(ctx):
    """All keys equal: token i returns the mean of value rows 0 .. pos0 + i.  One huge key: its value."""
    k = torch.zeros(1, 1, 1, 256, 128, device="cuda", dtype=torch.bfloat16)
    v = torch.randn(1, 1, 1, 256, 128, device="cuda").to(torch.bfloat16)
    q = torch.zeros(1, 1, 140, 128, device="cuda", dtype=torch.bfloat16)
    q[..., 0] = 1.0
    out = ctx.attend_prefill(k, v, 0, q, [200], rope_base=0.0)      # pos0 = 60
    for i in (0, 1, 77, 139):
        want = v[0, 0, 0, :60 + i + 1].float().mean(dim=0)
        assert torch.allclose(out[0, 0, i].float(), want, atol=2e-2, rtol=2e-2)
    k[0, 0, 0, 100, 0] = 3000.0                                        # visible from token 40 on
    out = ctx.attend_prefill(k, v, 0, q, [200], rope_base=0.0)
    assert torch.equal(out[0, 0, 40], v[0, 0, 0, 100]) and torch.equal(out[0, 0, 139], v[0, 0, 0, 100])
    assert torch.allclose(out[0, 0, 39].float(), v[0, 0, 0, :100].float().mean(dim=0), atol=2e-2, rtol=2e-2)


def test_prefill_7b_chunk_after_a_compression_sampled(ctx):
    """One 7B-shaped layer (32 heads, 4096 rows): the 2046 tokens that refill the cache after a
    compression attend to 4 sinks + 2046 compressed rows + the chunk; sampled heads and tokens."""
    w = workload(1, 2, 32, 4096, seed=27)
    k, v = synth.make_cache(w, "cuda")
    q = queries(1, 32, 2046, 9)
    check(ctx, k, v, 1, q, [4096], 10000.0, heads=[(0, 0), (0, 31), (0, 17)], tokens=(0, 127, 128, 1000, 2045))


def test_prefill_gqa_8b_shape_ragged_lengths_sampled(ctx):
    w = workload(2, 1, 8, 8192, seed=28)
    k, v = synth.make_cache(w, "cuda")
    q = queries(2, 32, 1000, 10)
    check(ctx, k, v, 0, q, [8192, 4099], 500000.0, heads=[(0, 0), (1, 7)], tokens=(0, 500, 999))


def test_prefill_invalid_arguments(ctx):
    k = torch.zeros(1, 2, 2, 64, 128, device="cuda", dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    q = torch.zeros(1, 2, 10, 128, device="cuda", dtype=torch.bfloat16)
    for bad in ([9], [65]):
        with pytest.raises(fk.FreqKVError) as e:
            ctx.attend_prefill(k, v, 0, q, bad)
        assert e.value.status == fk.ERR_INVALID_ARG
    with pytest.raises(fk.FreqKVError) as e:
        ctx.attend_prefill(k, v, 2, q, [10])
    assert e.value.status == fk.ERR_INVALID_ARG
    kf = torch.zeros(1, 1, 1, 64, 128, device="cuda")
    with pytest.raises(fk.FreqKVError) as e:
        ctx.attend_prefill(kf, torch.zeros_like(kf), 0, torch.zeros(1, 1, 10, 128, device="cuda"), [10])
    assert e.value.status == fk.ERR_UNSUPPORTED


def test_chunkwise_prefill_interleaves_attention_and_compression(ctx):
    """The loop of Section 3.3 on a small cache (256 rows, 4 sinks, 252 -> 126): every chunk is
    appended, attended, and the full cache compressed before the next chunk goes in.  The oracle
    runs its own fp64 pipeline (its own compressed caches, never the GPU's), so the comparison
    covers the interplay of freqkv_append, freqkv_attend_prefill and freqkv_compress; the
    tolerance grows with the number of compressions as in the stream tests."""
    cap, sink, kept, total, H, G = 256, 4, 126, 900, 2, 2
    rng = np.random.default_rng(20250500 + 31)
    def ar1(n, d):  # low-frequency dominated rows, as the cache generator's channels
        x = np.empty((n, d))
        x[0] = rng.standard_normal(d)
        for i in range(1, n):
            x[i] = 0.9 * x[i - 1] + np.sqrt(1 - 0.81) * rng.standard_normal(d)
        return x
    toks_k = torch.tensor(np.stack([ar1(total, 128) for _ in range(H)])).to(torch.bfloat16)   # [H, T, d]
    toks_v = torch.tensor(np.stack([ar1(total, 128) for _ in range(H)])).to(torch.bfloat16)
    toks_q = torch.tensor(rng.standard_normal((H * G, total, 128))).to(torch.bfloat16)
    k = torch.zeros(1, 1, H, cap, 128, device="cuda", dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    ok = [np.zeros((cap, 128)) for _ in range(H)]   # the oracle's caches
    ov = [np.zeros((cap, 128)) for _ in range(H)]
    length, count, t0, worst = 0, 0, 0, 0.0
    while t0 < total:
        if length == cap:
            length = ctx.compress(k, v, cap, kept, sink)
            for h in range(H):
                ok[h][sink:sink + kept] = oracle.compress_matrix(ok[h][sink:cap], kept)
                ov[h][sink:sink + kept] = oracle.compress_matrix(ov[h][sink:cap], kept)
            count += 1
        n = min(total - t0, cap - length)
        nk = toks_k[:, t0:t0 + n].reshape(1, 1, H, n, 128).contiguous().cuda()
        nv = toks_v[:, t0:t0 + n].reshape(1, 1, H, n, 128).contiguous().cuda()
        for h in range(H):
            ok[h][length:length + n] = parity.to_f64(toks_k[h, t0:t0 + n])
            ov[h][length:length + n] = parity.to_f64(toks_v[h, t0:t0 + n])
        length = ctx.append(k, v, nk, nv, [length])[0]
        q = toks_q[:, t0:t0 + n].reshape(1, H * G, n, 128).contiguous().cuda()
        out = ctx.attend_prefill(k, v, 0, q, [length], rope_base=10000.0)
        tol = TOL * (1 + count) ** 0.5
        for i in sorted({0, n // 2, n - 1}):
            for h in range(H):
                want = oa.attend_decode(parity.to_f64(q[0, h * G:(h + 1) * G, i]), ok[h], ov[h], length - n + i + 1, 10000.0)
                got = parity.to_f64(out[0, h * G:(h + 1) * G, i])
                for g in range(G):
                    err = parity.rel_l2(got[g], want[g])
                    assert err <= tol, f"chunk at token {t0}, row {i}: relative L2 {err:.3e} after {count} compressions"
                    worst = max(worst, err)
        t0 += n
    assert ctx.last_device_status() == fk.OK
    assert count == oracle.compression_count(total, cap, sink, kept) and count >= 5


def test_prefill_more_sequences_than_one_launch_takes(ctx):
    """130 short sequences: the lengths travel as kernel arguments, 128 per launch."""
    w = workload(130, 1, 1, 96, seed=29)
    k, v = synth.make_cache(w, "cuda")
    lens = [96 - (b % 50) for b in range(130)]
    q = queries(130, 2, 7, 11)
    check(ctx, k, v, 0, q, lens, 10000.0, heads=[(0, 0), (127, 0), (128, 0), (129, 0)])


@pytest.mark.parametrize("G", [3, 8])
def test_prefill_other_group_sizes(ctx, G):
    """Any number of query heads per KV head: each query head is its own CTA column."""
    w = workload(1, 1, 2, 192, seed=30)
    k, v = synth.make_cache(w, "cuda")
    check(ctx, k, v, 0, queries(1, 2 * G, 40, 12 + G), [150], 10000.0, tokens=(0, 17, 39))


def test_prefill_smallest_caches(ctx):
    """One token in a cache of one row; a chunk that is a whole cache whose length is no multiple of the tile sizes."""
    w = workload(1, 1, 1, 128, seed=31)
    k, v = synth.make_cache(w, "cuda")
    q1 = queries(1, 1, 1, 13)
    out = ctx.attend_prefill(k, v, 0, q1, [1], rope_base=10000.0)
    assert torch.equal(out[0, 0, 0], v[0, 0, 0, 0])
    check(ctx, k, v, 0, queries(1, 1, 100, 14), [100], 10000.0, tokens=(0, 1, 63, 64, 65, 99))
