"""GPU parity of freqkv_attend_decode (decode attention over the bounded cache, RoPE at in-cache
positions) against the fp64 oracle of oracle/attention.py on the same seeded inputs.

Tolerances, per query head, relative L2 of the 128 output channels: bf16 caches 1e-2 (the output
is rounded once to bf16: 2^-9); fp32 caches 2e-4 -- the scores carry the error of an fp32 rotation
whose cos/sin are stepped row to row for up to 32 rows (about 3e-6 relative per score term, times
scores of magnitude 10-20 in these inputs), which the softmax turns into the same relative error
of the weights."""
import numpy as np
import pytest
import torch

from oracle import attention as oa
from paper_2505_00570_b200 import binding as fk
from paper_2505_00570_b200 import synth
from tests import parity

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 2e-4, torch.bfloat16: 1e-2}


@pytest.fixture(scope="module")
def ctx():
    c = fk.Context(0)
    yield c
    c.close()


def workload(B, Ly, H, cap, dtype, seed=11):
    return synth.Workload("attn", B, Ly, H, 128, cap, dtype, 4, 0.9, 2, synth.BASE_SEED + seed)


def queries(B, heads, dtype, seed):
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    return torch.randn(B, heads, 128, generator=gen, device="cuda").to(dtype)


def check(ctx, k, v, layer, q, lens, base, heads=None, scale=0.0):
    out = ctx.attend_decode(k, v, layer, q, lens, rope_base=base, scale=scale)
    assert ctx.last_device_status() == fk.OK
    B, Hq = q.shape[0], q.shape[1]
    G = Hq // k.shape[2]
    worst = 0.0
    pick = heads if heads is not None else [(b, h) for b in range(B) for h in range(k.shape[2])]
    for b, h in pick:
        want = oa.attend_decode(parity.to_f64(q[b, h * G:(h + 1) * G]), parity.to_f64(k[b, layer, h]),
                                parity.to_f64(v[b, layer, h]), lens[b], base, None if scale <= 0 else scale)
        got = parity.to_f64(out[b, h * G:(h + 1) * G])
        for g in range(G):
            worst = max(worst, parity.rel_l2(got[g], want[g]))
    assert worst <= TOL[q.dtype], f"relative L2 {worst:.3e}"
    return worst


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
@pytest.mark.parametrize("G", [1, 2, 4, 8])
def test_attend_small_all_heads(ctx, dtype, G):
    w = workload(3, 3, 2, 300, dtype)
    k, v = synth.make_cache(w, "cuda")
    k0, v0 = k.clone(), v.clone()
    q = queries(3, 2 * G, dtype, 5 + G)
    check(ctx, k, v, 1, q, [300, 37, 1], 10000.0)
    assert torch.equal(k, k0) and torch.equal(v, v0)  # the cache is only read


@pytest.mark.parametrize("base,scale", [(0.0, 0.0), (500000.0, 0.05), (10000.0, 0.2)])
def test_attend_rope_off_other_base_and_scale(ctx, base, scale):
    w = workload(2, 2, 3, 200, torch.bfloat16, seed=12)
    k, v = synth.make_cache(w, "cuda")
    check(ctx, k, v, 0, queries(2, 6, torch.bfloat16, 3), [199, 64], base, scale=scale)
    check(ctx, k, v, 1, queries(2, 6, torch.bfloat16, 4), [2, 200], base, scale=scale)


def test_attend_row_padding_and_lengths_around_the_split_sizes(ctx):
    w = workload(1, 1, 2, 1100, torch.bfloat16, seed=13)
    (_, k), (_, v) = parity.guarded_cache(w, torch.device("cuda"), fill_len=1100, row_pad=8)
    q = queries(1, 4, torch.bfloat16, 6)
    for n in (15, 16, 17, 63, 64, 65, 255, 256, 257, 1023, 1024, 1025, 1100):
        check(ctx, k, v, 0, q, [n], 10000.0)


def test_attend_dominant_key_and_uniform_keys(ctx):
    """Special cases with known answers, straight on the GPU result."""
    k = torch.zeros(1, 1, 1, 128, 128, device="cuda", dtype=torch.float32)
    v = torch.randn(1, 1, 1, 128, 128, device="cuda")
    q = torch.zeros(1, 1, 128, device="cuda")
    q[0, 0, 0] = 1.0
    out = ctx.attend_decode(k, v, 0, q, [100], rope_base=0.0)          # all scores equal: the mean
    assert torch.allclose(out[0, 0], v[0, 0, 0, :100].mean(dim=0), atol=1e-5)
    k[0, 0, 0, 41, 0] = 2000.0                                          # one key wins
    out = ctx.attend_decode(k, v, 0, q, [100], rope_base=0.0)
    assert torch.allclose(out[0, 0], v[0, 0, 0, 41], atol=1e-5)


def test_attend_7b_shape_one_layer_sampled(ctx):
    """Batch 16 of 7B-shaped caches (32 KV heads, 4096 rows), two layers resident, the second one
    attended: 512 heads x 2.1 MB in one call; sampled heads against the oracle."""
    w = workload(16, 2, 32, 4096, torch.bfloat16, seed=14)
    k, v = synth.make_cache(w, "cuda")
    lens = [4096 - 37 * b for b in range(16)]
    q = queries(16, 32, torch.bfloat16, 8)
    check(ctx, k, v, 1, q, lens, 10000.0, heads=[(0, 0), (15, 31), (7, 13)])


def test_attend_gqa_8b_shape_sampled(ctx):
    w = workload(2, 1, 8, 8192, torch.bfloat16, seed=15)
    k, v = synth.make_cache(w, "cuda")
    check(ctx, k, v, 0, queries(2, 32, torch.bfloat16, 9), [8192, 4098], 500000.0, heads=[(0, 0), (1, 7)])


def test_attend_invalid_arguments(ctx):
    k = torch.zeros(1, 2, 2, 64, 128, device="cuda", dtype=torch.bfloat16)
    v = torch.zeros_like(k)
    q = torch.zeros(1, 2, 128, device="cuda", dtype=torch.bfloat16)
    for bad in ([0], [65]):
        with pytest.raises(fk.FreqKVError) as e:
            ctx.attend_decode(k, v, 0, q, bad)
        assert e.value.status == fk.ERR_INVALID_ARG
    with pytest.raises(fk.FreqKVError) as e:
        ctx.attend_decode(k, v, 2, q, [10])
    assert e.value.status == fk.ERR_INVALID_ARG
    with pytest.raises(fk.FreqKVError) as e:
        ctx.attend_decode(k, v, 0, torch.zeros(1, 6, 128, device="cuda", dtype=torch.bfloat16), [10])  # 3 query heads per KV head
    assert e.value.status == fk.ERR_UNSUPPORTED
    k64 = torch.zeros(1, 1, 1, 64, 64, device="cuda", dtype=torch.bfloat16)
    with pytest.raises(fk.FreqKVError) as e:
        ctx.attend_decode(k64, torch.zeros_like(k64), 0, torch.zeros(1, 1, 64, device="cuda", dtype=torch.bfloat16), [10])
    assert e.value.status == fk.ERR_UNSUPPORTED


@pytest.mark.parametrize("G", [1, 4])
def test_attend_more_sequences_than_one_launch_takes(ctx, G):
    """131 short sequences: the lengths travel as kernel arguments, 128 per launch, and one merge
    launch follows the last of them."""
    w = workload(131, 1, 1, 96, torch.bfloat16, seed=16)
    k, v = synth.make_cache(w, "cuda")
    lens = [96 - (b % 60) for b in range(131)]
    check(ctx, k, v, 0, queries(131, G, torch.bfloat16, 17 + G), lens, 10000.0, heads=[(0, 0), (1, 0), (127, 0), (128, 0), (130, 0)])
