"""The decode step as a CUDA graph with device-resident lengths (device-side trigger, conditional
compression, append) against the host-driven path: the same token stream must leave bit-identical
caches and lengths, with the compression count the trigger rule gives."""
import pytest
import torch

import oracle
from paper_2505_00570_b200 import binding as fk
from paper_2505_00570_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = fk.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("cap,sink,kept,T", [(300, 4, 148, 1000), (132, 0, 33, 500)])
def test_decode_graph_equals_host_driven_stream(ctx, cap, sink, kept, T):
    w = synth.Workload("dg", 2, 2, 2, 128, cap, torch.bfloat16, sink, 0.9, 2, synth.BASE_SEED + 41)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed)
    scales = synth.channel_scales(w, gen, "cuda")
    toks_k, _ = synth.ar1_rows(w, T, gen, "cuda", scales)
    toks_v, _ = synth.ar1_rows(w, T, gen, "cuda", scales)

    # host-driven reference run (tensor-core variant, like the graph)
    ctx.set_variant(fk.GEMM)
    k1, v1 = synth.make_cache(w, "cuda", fill_len=0)
    lens, count = [0, 0], 0
    for t in range(T):
        nk, nv = toks_k[:, :, :, t:t + 1].contiguous(), toks_v[:, :, :, t:t + 1].contiguous()
        try:
            lens = ctx.append(k1, v1, nk, nv, lens)
        except fk.FreqKVError as e:
            assert e.status == fk.ERR_CAPACITY
            n = ctx.compress(k1, v1, cap, kept, sink)
            count += 1
            lens = ctx.append(k1, v1, nk, nv, [n, n])
    ctx.set_variant(fk.AUTO)
    assert count == oracle.compression_count(T, cap, sink, kept) and count >= 3

    # graph run: lengths live on the device, nothing is read back between steps
    k2, v2 = synth.make_cache(w, "cuda", fill_len=0)
    lens_dev = torch.zeros(2, dtype=torch.int32, device="cuda")
    stage_k, stage_v = torch.empty_like(toks_k[:, :, :, :1]).contiguous(), torch.empty_like(toks_v[:, :, :, :1]).contiguous()
    graph = fk.DecodeGraph(ctx, k2, v2, stage_k, stage_v, lens_dev, kept, sink)
    try:
        for t in range(T):
            stage_k.copy_(toks_k[:, :, :, t:t + 1])
            stage_v.copy_(toks_v[:, :, :, t:t + 1])
            graph.launch()
        torch.cuda.synchronize()
        assert ctx.last_device_status() == fk.OK
        assert lens_dev.tolist() == lens
        n = lens[0]
        assert torch.equal(k2[:, :, :, :n], k1[:, :, :, :n]) and torch.equal(v2[:, :, :, :n], v1[:, :, :, :n])
    finally:
        graph.close()


def test_decode_graph_survives_larger_calls_on_its_context(ctx):
    """The graph's kernels have the addresses of the fold scratch and of the basis baked in.  Other
    calls on the same context that need a larger scratch (a bigger cache) or rebuild plans must not
    move or free what a live graph replays from: the graph owns its own.  The stream through the
    graph, with such calls in between, must still be bit-identical to the host-driven one."""
    cap, sink, kept, T = 300, 4, 148, 700
    w = synth.Workload("dg", 2, 2, 2, 128, cap, torch.bfloat16, sink, 0.9, 2, synth.BASE_SEED + 43)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(w.seed)
    scales = synth.channel_scales(w, gen, "cuda")
    toks, _ = synth.ar1_rows(w, T, gen, "cuda", scales)
    big = synth.Workload("dg_big", 3, 4, 4, 128, 1500, torch.bfloat16, sink, 0.9, 2, synth.BASE_SEED + 44)
    ctx.set_variant(fk.GEMM)
    k1, v1 = synth.make_cache(w, "cuda", fill_len=0)
    lens = [0, 0]
    for t in range(T):
        nk = toks[:, :, :, t:t + 1].contiguous()
        try:
            lens = ctx.append(k1, v1, nk, nk, lens)
        except fk.FreqKVError as e:
            assert e.status == fk.ERR_CAPACITY
            n = ctx.compress(k1, v1, cap, kept, sink)
            lens = ctx.append(k1, v1, nk, nk, [n, n])
    k2, v2 = synth.make_cache(w, "cuda", fill_len=0)
    lens_dev = torch.zeros(2, dtype=torch.int32, device="cuda")
    stage_k = torch.empty_like(toks[:, :, :, :1]).contiguous()
    stage_v = torch.empty_like(stage_k)
    graph = fk.DecodeGraph(ctx, k2, v2, stage_k, stage_v, lens_dev, kept, sink)
    try:
        for t in range(T):
            if t in (10, 350):   # a call that needs a much larger fold scratch, and the graph's own shape again
                kb, vb = synth.make_cache(big, "cuda")
                ctx.compress(kb, vb, 1500, 748, sink)
                ks, vs = synth.make_cache(w, "cuda")
                ctx.compress(ks, vs, cap, kept, sink)
                del kb, vb, ks, vs
            stage_k.copy_(toks[:, :, :, t:t + 1])
            stage_v.copy_(toks[:, :, :, t:t + 1])
            graph.launch()
        torch.cuda.synchronize()
        assert ctx.last_device_status() == fk.OK
        assert lens_dev.tolist() == lens
        n = lens[0]
        assert torch.equal(k2[:, :, :, :n], k1[:, :, :, :n]) and torch.equal(v2[:, :, :, :n], v1[:, :, :, :n])
    finally:
        graph.close()
        ctx.set_variant(fk.AUTO)


def test_decode_graph_reports_a_batch_that_is_not_uniform(ctx):
    w = synth.Workload("dg", 2, 1, 1, 128, 200, torch.bfloat16, 4, 0.9, 0, synth.BASE_SEED + 42)
    k, v = synth.make_cache(w, "cuda")
    k0 = k.clone()
    lens_dev = torch.tensor([200, 10], dtype=torch.int32, device="cuda")
    stage = torch.ones(2, 1, 1, 1, 128, device="cuda", dtype=torch.bfloat16)
    graph = fk.DecodeGraph(ctx, k, v, stage, stage.clone(), lens_dev, 98, 4)
    try:
        graph.launch()
        torch.cuda.synchronize()
        assert ctx.last_device_status() == fk.ERR_CAPACITY
        assert lens_dev.tolist() == [200, 11]                      # the full sequence was skipped, the other appended
        assert torch.equal(k[0], k0[0]) and torch.equal(k[1, 0, 0, 10], stage[1, 0, 0, 0])
        assert ctx.last_device_status() == fk.OK                   # the report clears the word
    finally:
        graph.close()


def test_decode_graph_argument_checks(ctx):
    k = torch.zeros(1, 1, 1, 64, 128, device="cuda", dtype=torch.float32)
    lens_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    stage = torch.zeros(1, 1, 1, 1, 128, device="cuda", dtype=torch.float32)
    with pytest.raises(fk.FreqKVError) as e:
        fk.DecodeGraph(ctx, k, torch.zeros_like(k), stage, stage.clone(), lens_dev, 30, 4)   # fp32: no tensor-core variant
    assert e.value.status == fk.ERR_UNSUPPORTED
    kb = k.to(torch.bfloat16)
    sb = stage.to(torch.bfloat16)
    with pytest.raises(fk.FreqKVError) as e:
        fk.DecodeGraph(ctx, kb, torch.zeros_like(kb), sb, sb.clone(), lens_dev, 60, 4)       # kept_len leaves no room
    assert e.value.status == fk.ERR_INVALID_ARG
