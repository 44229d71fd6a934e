#!/usr/bin/env python
"""Benchmark of the FreqKV hot path on B200: KV-compress GB/s of cache in.

One *step* is one pass of the whole hot path over one batch of synthetic input, as in the
chunk-wise loop of Section 3.4: the cache is full, so the incoming chunk is refused
(``FREQKV_ERR_CAPACITY``, the lazy trigger), every K and V matrix is compressed in place
(DCT-II -> keep L -> L-point IDCT -> rescale, sinks untouched), and the chunk of
``capacity - sink - L`` new rows is appended, which fills the cache again for the next step.

``value`` = (bytes of cache in per step) / (device time per step), inputs resident in HBM.
``e2e``   = the same metric through ``freqkv_compress_host`` with the cache in pinned host
            memory (host->device and device->host copies inside the timed region).
``roofline`` describes the dominant kernel (the transform), timed with CUDA events recorded by
the library around that launch on the launching stream.

Launch: ``python bench.py --gpus N --steps K --warmup W``; for N > 1 under
``python -m torch.distributed.run --nproc-per-node N``: the path has no exchange step, so N
ranks are N independent replicas (weak scaling, no collective on the data path).
``--impl reference`` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "KV-compress GB/s of cache in (7B shape, 4096->2048) and % of roofline"
UNIT = "GB/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        p["source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["source"] = "fallback"
    return p


def load_traffic(workload: str, variant: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, if any."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    if not os.path.exists(path):
        return None
    with open(path) as f:
        table = json.load(f)
    return table.get(f"{workload}:{variant}")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, device_index: int, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._period = period_s
        try:
            import pynvml

            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self._nv = pynvml
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # NVML missing: report that, do not fail the bench
            self._nv = None
            self.error = repr(e)

    def _run(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        get_reasons = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or getattr(
            nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                mask = get_reasons(self._h)
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self._period)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
               "samples": len(self.samples)}
        if self.samples:
            s = sorted(self.samples)
            out["sm_mhz"] = s[len(s) // 2]
        if self._nv is None:
            out["error"] = getattr(self, "error", "nvml unavailable")
        return out


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(ms: float, device) -> float:
    """Slowest rank's time (replicas run side by side; the job is as slow as its slowest)."""
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier():
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def workload_numbers(w, cache_len, kept, sink, first=0):
    e = 2 if w.dtype == torch.bfloat16 else 4
    m = w.n_matrices
    n_in = cache_len - sink
    # Multiply-adds the tensor-core variant executes.  One level of the symmetry fold: even and odd parts,
    # ceil(L/2) x ceil(N/2) each.  Where the lengths halve twice (N a multiple of 4, L even, the lowest
    # components kept) the even part is folded again: ceil(L/4) rows x (N/4 + N/4 + N/2 + N/2) columns.
    from paper_2505_00570_b200 import binding as _fk
    fold_levels = _fk.gemm_fold_levels(n_in, kept, first)   # the library's own rule (0 = no fold pass: few kept rows)
    if fold_levels == 2:
        folded = 2.0 * ((kept // 2 + 1) // 2) * 3 * (n_in // 2) * w.head_dim * m
    else:
        folded = 2.0 * 2 * ((kept + 1) // 2) * ((n_in + 1) // 2) * w.head_dim * m
    return {
        "fold_levels": fold_levels,
        "matrices": m,
        "cache_in_bytes": m * cache_len * w.head_dim * e,
        "algorithmic_bytes": m * (n_in + kept) * w.head_dim * e,   # read N' rows, write L rows
        "projection_flops": 2.0 * kept * n_in * w.head_dim * m,    # the dense L x N projection (CUDA-core variant)
        "folded_flops": folded,
        "append_bytes": 2 * m * (cache_len - sink - kept) * w.head_dim * e,
    }


def run_reference(args, rank):
    """CPU oracle arm: each step compresses a bounded sample (one matrix) of the workload."""
    if rank != 0:
        return
    import oracle
    from paper_2505_00570_b200 import synth
    import dataclasses

    w = synth.WORKLOADS[args.workload]
    cache_len, sink = w.capacity, w.sink
    kept = w.kept_len(cache_len)
    one = dataclasses.replace(w, batch=1, layers=1, kv_heads=1)
    k, _ = synth.make_cache(one, "cpu")
    x = k[0, 0, 0, sink:cache_len].to(torch.float64).numpy()
    e = 2 if w.dtype == torch.bfloat16 else 4
    bytes_in = cache_len * w.head_dim * e
    for _ in range(args.warmup):
        oracle.compress_matrix(x, kept)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.compress_matrix(x, kept)
    dt = time.perf_counter() - t0
    val = bytes_in * args.steps / dt / 1e9
    cores = oracle.threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "cache_len": cache_len, "kept_len": kept, "sink": sink,
                   "sample": "1 of %d matrices per step" % w.n_matrices},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": "one %dx%d matrix per step, %d steps" % (cache_len - sink, w.head_dim, args.steps)},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def cpu_baseline(w, k, v, cache_len, kept, sink, budget_s=12.0):
    """The oracle, as it stands, on a bounded sample of this workload's matrices."""
    import oracle

    e = 2 if w.dtype == torch.bfloat16 else 4
    flat = k.view(-1, k.shape[-2], k.shape[-1])
    x0 = flat[0, sink:cache_len].to("cpu").to(torch.float64).numpy()
    t0 = time.perf_counter()
    oracle.compress_matrix(x0, kept)
    one = time.perf_counter() - t0
    count = int(max(2, min(256, budget_s / max(one, 1e-3))))
    ids = torch.linspace(0, flat.shape[0] - 1, count).long().tolist()
    xs = [flat[i, sink:cache_len].to("cpu").to(torch.float64).numpy() for i in ids]
    t0 = time.perf_counter()
    for x in xs:
        oracle.compress_matrix(x, kept)
    dt = time.perf_counter() - t0
    return {"value": count * cache_len * w.head_dim * e / dt / 1e9, "unit": UNIT, "cores": oracle.threads(),
            "kind": "oracle", "sample": "%d of %d matrices (%dx%d -> %d rows), %.1f s" %
            (count, w.n_matrices, cache_len - sink, w.head_dim, kept, dt)}


def run_ragged(args, ctx, fk, synth, w, dev, peaks):
    """Config 5b: one freqkv_compress_ragged call over a batch of caches of different lengths."""
    sink = w.sink
    lens = synth.ragged_lengths(w)
    kept = [(n - sink) // 2 for n in lens]
    k, v = synth.make_cache(w, dev)
    e = 2
    m_per_seq = 2 * w.layers * w.kv_heads
    cache_in = sum(lens) * w.head_dim * e * m_per_seq
    moved = sum((n - sink) + kp for n, kp in zip(lens, kept)) * w.head_dim * e * m_per_seq
    flops = sum(4.0 * ((kp + 1) // 2) * ((n - sink + 1) // 2) for n, kp in zip(lens, kept)) * w.head_dim * m_per_seq
    for _ in range(args.warmup):
        ctx.compress_ragged(k, v, lens, kept, sink)
    torch.cuda.synchronize()
    _, _, launched0 = ctx.get_timing()
    ctx.set_timing(True)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        ctx.compress_ragged(k, v, lens, kept, sink)
    b.record()
    torch.cuda.synchronize()
    n_launch, t_ms, launched1 = ctx.get_timing()
    ctx.set_timing(False)
    ms = a.elapsed_time(b) / args.steps
    gemm_ms = t_ms / args.steps
    return {"metric": METRIC, "value": cache_in / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "batch": w.batch, "layers": w.layers, "kv_heads": w.kv_heads, "head_dim": w.head_dim,
                       "capacity": w.capacity, "sink": sink, "lens": lens, "step": "one freqkv_compress_ragged call",
                       "l2": "inputs larger than L2 (%.1f GB of cache per step)" % (cache_in / 1e9)},
            "compress_only": {"ms": ms, "cache_in_GBps": cache_in / (ms * 1e-3) / 1e9, "moved_GBps": moved / (ms * 1e-3) / 1e9,
                              "hbm_floor_ms": moved / (peaks["hbm_gbs"] * 1e9) * 1e3},
            "roofline": {"bound": "tensor", "achieved": flops / (gemm_ms * 1e-3) / 1e12, "peak": peaks["bf16_tflops_sustained"],
                         "unit": "TFLOP/s", "frac": flops / (gemm_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"],
                         "peak_kind": "sustained, of " + peaks["source"], "kernel": "gemm", "kernel_ms": gemm_ms / (n_launch / args.steps),
                         "frac_of_burst_peak": flops / (gemm_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                         "launches_per_call": n_launch / args.steps, "traffic": None},
            "kernels_per_call": (launched1 - launched0) / args.steps,
            "cpu_baseline": None, "e2e": None, "gpu_launches": launched1 - launched0}


def run_stream_graph(args, ctx, fk, synth, w, dev, peaks, total_tokens=32768):
    """Config 4 through the decode graph: lengths on the device, the trigger and the compression
    inside the graph; per step the host only refills the staging rows and launches the graph."""
    cap, sink = w.capacity, w.sink
    kept = w.kept_len(cap)
    k, v = synth.make_cache(w, dev, fill_len=0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed)
    scales = synth.channel_scales(w, gen, dev)
    ring, _ = synth.ar1_rows(w, 64, gen, dev, scales)
    toks = [ring[:, :, :, j:j + 1].contiguous() for j in range(64)]
    lens = torch.zeros(w.batch, dtype=torch.int32, device=dev)
    stage_k, stage_v = torch.empty_like(toks[0]), torch.empty_like(toks[0])
    graph = fk.DecodeGraph(ctx, k, v, stage_k, stage_v, lens, kept, sink)
    for t in range(8):   # warm-up launches on a scratch run, then reset
        stage_k.copy_(toks[t]); stage_v.copy_(toks[t]); graph.launch()
    lens.zero_()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    a.record()
    for t in range(total_tokens):
        nk = toks[t & 63]
        stage_k.copy_(nk)
        stage_v.copy_(nk)
        graph.launch()
    b.record()
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    final = lens.tolist()
    graph.close()
    count = 0 if total_tokens <= cap else 1 + (total_tokens - cap - 1) // (cap - sink - kept)  # fills after the first one
    per_tok_us = wall / total_tokens * 1e6
    e = 2
    cache_in = w.n_matrices * cap * w.head_dim * e
    return {"metric": METRIC, "value": cache_in * count / wall / 1e9, "unit": UNIT, "n_gpus": 1, "steps": total_tokens,
            "warmup": 8, "ms_per_step": wall / total_tokens * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name + "_graph", "batch": w.batch, "layers": w.layers, "kv_heads": w.kv_heads,
                       "head_dim": w.head_dim, "capacity": cap, "sink": sink, "kept_len": kept, "tokens": total_tokens,
                       "step": "staging rows refilled + one freqkv_decode_graph_launch (device-side trigger)"},
            "stream": {"compressions": count, "final_lens": final[:2], "wall_s": wall, "device_ms": a.elapsed_time(b),
                       "amortised_us_per_token_step": per_tok_us, "amortised_us_per_token_per_sequence": per_tok_us / w.batch},
            "roofline": None, "cpu_baseline": None, "e2e": None, "gpu_launches": None}


def run_stream(args, ctx, fk, synth, w, dev, peaks, total_tokens=32768):
    """Config 4: tokens appended one per step from empty caches; a full cache is compressed to
    half its non-sink length before the next token goes in.  Reports the amortised time per
    generated token (wall clock of the whole loop: host launch cost included)."""
    cap, sink = w.capacity, w.sink
    kept = w.kept_len(cap)
    k, v = synth.make_cache(w, dev, fill_len=0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed)
    scales = synth.channel_scales(w, gen, dev)
    ring, _ = synth.ar1_rows(w, 64, gen, dev, scales)   # 64 seeded token rows, reused cyclically
    toks = [ring[:, :, :, j:j + 1].contiguous() for j in range(64)]
    ctx.plan(cap - sink, kept, fk.BF16, fk.AUTO)
    lens, count = [0] * w.batch, 0
    comp_ev = []
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for t in range(total_tokens):
        nk = toks[t & 63]
        try:
            lens = ctx.append(k, v, nk, nk, lens)
        except fk.FreqKVError as err:
            if err.status != fk.ERR_CAPACITY:
                raise
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            new_len = ctx.compress(k, v, cap, kept, sink)
            b.record()
            comp_ev.append((a, b))
            count += 1
            lens = ctx.append(k, v, nk, nk, [new_len] * w.batch)
    torch.cuda.synchronize()
    wall = time.perf_counter() - t0
    comp_ms = sum(a.elapsed_time(b) for a, b in comp_ev)
    e = 2
    cache_in = w.n_matrices * cap * w.head_dim * e
    per_tok_us = wall / total_tokens * 1e6
    return {"metric": METRIC, "value": cache_in * count / (comp_ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1,
            "steps": total_tokens, "warmup": 0, "ms_per_step": wall / total_tokens * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "batch": w.batch, "layers": w.layers, "kv_heads": w.kv_heads, "head_dim": w.head_dim,
                       "capacity": cap, "sink": sink, "kept_len": kept, "tokens": total_tokens,
                       "step": "one token appended to every sequence (+ compression when the cache is full)"},
            "stream": {"compressions": count, "compress_ms_each": comp_ms / max(count, 1),
                       "compress_ms_total": comp_ms, "wall_s": wall, "amortised_us_per_token_step": per_tok_us,
                       "amortised_us_per_token_per_sequence": per_tok_us / w.batch,
                       "compress_share": comp_ms * 1e-3 / wall},
            "roofline": None, "cpu_baseline": None, "e2e": None, "gpu_launches": None}


def run_attend(args, ctx, fk, synth, name, dev, peaks):
    """Decode attention of one new token per sequence over full caches (the step after the
    compression path): one freqkv_attend_decode call per step, layers alternating so that no
    call finds its rows in L2."""
    import dataclasses

    B, H, G, cap, base, rho = {"attend_7b": (16, 32, 1, 4096, 10000.0, 0.9), "attend_8b": (8, 8, 4, 8192, 500000.0, 0.95)}[name]
    layers = args.layers if args.layers > 0 else 4   # one layer (1.07 GB on 7B) is already far larger than L2: enough for a profiler capture
    w = synth.Workload(name, B, layers, H, 128, cap, torch.bfloat16, 4, rho, 2, synth.BASE_SEED + 7)
    k, v = synth.make_cache(w, dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed + 1)
    q = torch.randn(B, H * G, 128, generator=gen, device=dev).to(torch.bfloat16)
    out = torch.empty_like(q)
    lens = [cap] * B
    bytes_per_call = 2 * B * H * cap * 128 * 2  # every K and V row of the layer once
    for i in range(max(args.warmup, 3)):
        ctx.attend_decode(k, v, i % layers, q, lens, rope_base=base, out=out)
    torch.cuda.synchronize()
    ctx.get_timing()
    ctx.set_timing(True)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(args.steps):
        ctx.attend_decode(k, v, i % layers, q, lens, rope_base=base, out=out)
    b.record()
    torch.cuda.synchronize()
    n, t_ms, _ = ctx.get_timing()
    ctx.set_timing(False)
    ms = a.elapsed_time(b) / args.steps
    kernel_ms = t_ms / max(n, 1)
    achieved = bytes_per_call / (kernel_ms * 1e-3) / 1e9
    return {"metric": "decode attention GB/s of cache read", "value": bytes_per_call / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": name, "batch": B, "kv_heads": H, "q_heads_per_kv": G, "head_dim": 128, "cache_len": cap,
                       "rope_base": base, "step": "one freqkv_attend_decode call over one layer",
                       "l2": "%d layers alternate, %.2f GB read per call" % (layers, bytes_per_call / 1e9)},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": achieved / peaks["hbm_gbs"], "peak_kind": "copy, of " + peaks["source"],
                         "kernel": ("attend_mma_kernel" if G >= 2 else "attend_partial_kernel") + " + attend_merge_kernel",
                         "kernel_ms": kernel_ms,
                         "traffic": load_traffic(name, "attend")},
            "cpu_baseline": None, "e2e": None, "gpu_launches": 2 * args.steps}


def run_prefill_attend(args, ctx, fk, synth, name, dev, peaks):
    """Chunk-wise prefilling attention (Section 3.3) of one layer: the tokens that refill the cache
    after a compression (2046 on the 7B shape, 4094 on the 8B shape) attend causally to 4 sinks +
    the compressed rows + the chunk.  One freqkv_attend_prefill call per step, layers alternating."""
    B, H, G, cap, base = {"prefill_attend_7b": (1, 32, 1, 4096, 10000.0), "prefill_attend_8b": (1, 8, 4, 8192, 500000.0)}[name]
    n_new = cap - 4 - (cap - 4) // 2
    layers = 4
    w = synth.Workload(name, B, layers, H, 128, cap, torch.bfloat16, 4, 0.9, 2, synth.BASE_SEED + 8)
    k, v = synth.make_cache(w, dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(w.seed + 1)
    q = torch.randn(B, H * G, n_new, 128, generator=gen, device=dev).to(torch.bfloat16)
    out = torch.empty_like(q)
    lens = [cap] * B
    pos0 = cap - n_new
    attended = n_new * pos0 + n_new * (n_new + 1) // 2          # (query, key) pairs under the causal mask, per head
    flops_per_call = 4 * 128 * attended * B * H * G             # two products, 2 flop per multiply-add
    for i in range(max(args.warmup, 3)):
        ctx.attend_prefill(k, v, i % layers, q, lens, rope_base=base, out=out)
    torch.cuda.synchronize()
    ctx.get_timing()
    ctx.set_timing(True)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for i in range(args.steps):
        ctx.attend_prefill(k, v, i % layers, q, lens, rope_base=base, out=out)
    b.record()
    torch.cuda.synchronize()
    n, t_ms, _ = ctx.get_timing()
    ctx.set_timing(False)
    ms = a.elapsed_time(b) / args.steps
    kernel_ms = t_ms / max(n, 1)
    achieved = flops_per_call / (kernel_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]
    return {"metric": "prefill attention TFLOP/s (causal pairs only)", "value": flops_per_call / (ms * 1e-3) / 1e12, "unit": "TFLOP/s",
            "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": name, "batch": B, "kv_heads": H, "q_heads_per_kv": G, "head_dim": 128,
                       "cache_len": cap, "chunk": n_new, "rope_base": base,
                       "step": "one freqkv_attend_prefill call over one layer", "l2": "%d layers alternate" % layers},
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                         "peak_kind": "cuBLAS bf16 burst, of " + peaks["source"],
                         "kernel": "prefill_rope_kernel + prefill_attend_kernel", "kernel_ms": kernel_ms, "traffic": load_traffic(name, "attend")},
            "cpu_baseline": None, "e2e": None, "gpu_launches": 2 * args.steps}


def run_spectrum(args, ctx, fk, synth, dev, peaks):
    """Average DCT power spectrum of a 7B-shaped cache (Section 3.1): one freqkv_power_spectrum call per step."""
    w = synth.WORKLOADS["llama2_7b"]
    cache_len, sink = w.capacity, w.sink
    n_in = cache_len - sink
    k, v = synth.make_cache(w, dev)
    for _ in range(max(args.warmup, 3)):
        ctx.power_spectrum(k, v, cache_len, sink)
    torch.cuda.synchronize()
    ctx.get_timing()
    ctx.set_timing(True)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        ctx.power_spectrum(k, v, cache_len, sink)
    b.record()
    torch.cuda.synchronize()
    n, t_ms, _ = ctx.get_timing()
    ctx.set_timing(False)
    ms = a.elapsed_time(b) / args.steps
    kernel_ms = t_ms / max(n, 1)
    nh = (n_in + 1) // 2
    flops = 2.0 * 2 * nh * nh * w.head_dim * w.n_matrices      # even rows on u, odd rows on v
    cache_in = w.n_matrices * cache_len * w.head_dim * 2
    achieved = flops / (kernel_ms * 1e-3) / 1e12
    return {"metric": "power-spectrum GB/s of cache in", "value": cache_in / (ms * 1e-3) / 1e9, "unit": UNIT, "n_gpus": 1,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "spectrum_7b", "batch": w.batch, "layers": w.layers, "kv_heads": w.kv_heads,
                       "head_dim": w.head_dim, "cache_len": cache_len, "sink": sink,
                       "step": "one freqkv_power_spectrum call (fold + all N DCT components + squared sums)",
                       "l2": "inputs larger than L2 (%.2f GB of cache per step)" % (cache_in / 1e9)},
            "roofline": {"bound": "tensor", "achieved": achieved, "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                         "frac": achieved / peaks["bf16_tflops_sustained"], "peak_kind": "sustained, of " + peaks["source"],
                         "frac_of_burst_peak": achieved / peaks["bf16_tflops"], "kernel": "freqkv_gemm_kernel<spectrum>",
                         "kernel_ms": kernel_ms, "flops_per_launch": flops, "traffic": None},
            "cpu_baseline": None, "e2e": None, "gpu_launches": 2 * args.steps}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b")
    ap.add_argument("--variant", default="auto", choices=["auto", "gemm", "fdct", "simt"])
    ap.add_argument("--fast-family", default="auto", choices=["auto", "cooley-tukey", "prime-factor"],
                    help="factorisation used by the bf16 fast transform (variant fdct)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--retain", type=float, default=0.5, help="retaining ratio gamma: kept_len = floor(gamma * (cache_len - sink))")
    ap.add_argument("--high-frequencies", action="store_true",
                    help="retain the highest kept_len DCT components instead of the lowest (the paper's ablation)")
    ap.add_argument("--layers", type=int, default=0, help="shrink the workload to this many layers (profiling only)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    rank, local_rank, world = dist_env()

    if args.impl == "reference":
        run_reference(args, rank)
        return

    from paper_2505_00570_b200 import binding as fk
    from paper_2505_00570_b200 import synth

    if args.workload == "spectrum_7b":
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
        if rank == 0:
            torch.cuda.set_device(local_rank)
            ctx = fk.Context(local_rank)
            print(json.dumps(run_spectrum(args, ctx, fk, synth, torch.device("cuda", local_rank), load_peaks())), flush=True)
            ctx.close()
        return
    if args.workload in ("prefill_attend_7b", "prefill_attend_8b"):  # side workload: chunk-wise prefilling attention
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
        if rank == 0:
            torch.cuda.set_device(local_rank)
            ctx = fk.Context(local_rank)
            print(json.dumps(run_prefill_attend(args, ctx, fk, synth, args.workload, torch.device("cuda", local_rank), load_peaks())), flush=True)
            ctx.close()
        return
    if args.workload in ("attend_7b", "attend_8b"):   # side workload: the step after the compression path
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
        if rank == 0:
            torch.cuda.set_device(local_rank)
            ctx = fk.Context(local_rank)
            print(json.dumps(run_attend(args, ctx, fk, synth, args.workload, torch.device("cuda", local_rank), load_peaks())), flush=True)
            ctx.close()
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    n_gpus = world

    w = synth.WORKLOADS["stream_7b" if args.workload == "stream_7b_graph" else args.workload]
    if args.layers > 0:
        import dataclasses

        w = dataclasses.replace(w, layers=args.layers)
    cache_len, sink = w.capacity, w.sink
    kept = w.kept_len(cache_len, args.retain)
    first = cache_len - sink - kept if args.high_frequencies else 0
    n_new = cache_len - sink - kept
    nums = workload_numbers(w, cache_len, kept, sink, first)

    ctx = fk.Context(local_rank)
    variant = {"auto": fk.AUTO, "gemm": fk.GEMM, "fdct": fk.FDCT, "simt": fk.SIMT}[args.variant]
    ctx.set_variant(variant)
    ctx.set_fast_family({"auto": 0, "cooley-tukey": fk.COOLEY_TUKEY, "prime-factor": fk.PRIME_FACTOR}[args.fast_family])
    if args.workload in ("ragged_8b", "stream_7b", "stream_7b_graph"):   # side workloads: one line each, single GPU
        if rank == 0:
            fn = {"ragged_8b": run_ragged, "stream_7b": run_stream, "stream_7b_graph": run_stream_graph}[args.workload]
            print(json.dumps(fn(args, ctx, fk, synth, w, dev, load_peaks())), flush=True)
        ctx.close()
        return
    k, v = synth.make_cache(w, dev, seed_offset=rank)
    lay = fk.layout_of(k)
    chosen = ctx.resolve_variant(lay, cache_len - sink, kept)
    if chosen < 0:
        raise SystemExit(f"variant {args.variant} cannot run {args.workload}")
    chosen_name = fk.VARIANT_NAMES[chosen]
    base = cpu_baseline(w, k, v, cache_len, kept, sink) if (rank == 0 and n_gpus == 1 and not args.no_cpu_baseline) else None

    # the incoming chunk: the first n_new rows of a second seeded draw, resident in HBM
    nk = k[:, :, :, :n_new].flip(3).contiguous()
    nv = v[:, :, :, :n_new].flip(3).contiguous()
    lens = [cache_len] * w.batch

    def step(lens):
        try:
            return ctx.append(k, v, nk, nv, lens)        # refused while the cache is full
        except fk.FreqKVError as err:
            if err.status != fk.ERR_CAPACITY:
                raise
        new_len = ctx.compress_band(k, v, cache_len, kept, sink, first) if first else ctx.compress(k, v, cache_len, kept, sink)
        return ctx.append(k, v, nk, nv, [new_len] * w.batch)

    for _ in range(args.warmup):
        lens = step(lens)
    torch.cuda.synchronize()
    if ctx.last_device_status() != fk.OK:
        raise SystemExit("device status reported an error during warm-up")
    ctx.get_timing()
    _, _, launches0 = ctx.get_timing()
    ctx.set_timing(True)

    sampler = ClockSampler(local_rank)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    torch.cuda.synchronize()
    sampler.start()
    start.record()
    for _ in range(args.steps):
        lens = step(lens)
    stop.record()
    torch.cuda.synchronize()
    barrier()
    clocks = sampler.stop()
    ms_total = max_over_ranks(start.elapsed_time(stop), dev)
    t_launches, t_ms, launches1 = ctx.get_timing()
    ctx.set_timing(False)
    status = ctx.last_device_status()
    if status != fk.OK:
        raise SystemExit("device status reported an error in the timed region")
    ms_step = ms_total / args.steps
    value = n_gpus * nums["cache_in_bytes"] / (ms_step * 1e-3) / 1e9

    # ---- the two calls of a step timed on their own (same buffers, same launch configuration)
    def timed(fn, reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    reps = max(3, min(args.steps, 20))
    compress_ms = timed(lambda: ctx.compress_band(k, v, cache_len, kept, sink, first) if first
                        else ctx.compress(k, v, cache_len, kept, sink), reps)
    append_ms = timed(lambda: ctx.append(k, v, nk, nv, [sink + kept] * w.batch), reps)

    # ---- roofline of the dominant kernel (the transform launch)
    peaks = load_peaks()
    kernel_ms = t_ms / max(t_launches, 1)                  # average duration of one launch of the dominant kernel
    per_call = max(t_launches, 1) / args.steps             # launches per compression (large caches take several passes)
    for key in ("folded_flops", "projection_flops", "algorithmic_bytes"):
        nums[key + "_per_launch"] = nums[key] / per_call
    if chosen == fk.GEMM and kept <= 256:
        # few kept rows: the tensor-core variant reads the cache directly (no fold pass, one tile per
        # matrix pair) and is bound by that one read of the cache
        achieved = nums["algorithmic_bytes_per_launch"] / (kernel_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_kind": "copy, of " + peaks["source"]}
    elif chosen == fk.GEMM:
        achieved = nums["folded_flops_per_launch"] / (kernel_ms * 1e-3) / 1e12
        # the burst figure is the denominator for a timed region of under a second, the sustained
        # one (power cap reached) for longer loops; both fractions are printed
        burst = ms_total < 1000.0
        peak = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
        fold_ms = max(compress_ms - kernel_ms * per_call, 0.0)
        roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak, "peak_kind": ("burst" if burst else "sustained") + ", of " + peaks["source"],
                "frac_of_burst_peak": achieved / peaks["bf16_tflops"],
                "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
                "flops_per_launch": nums["folded_flops_per_launch"], "fold_levels": nums["fold_levels"],
                "dense_equivalent_flops_per_launch": nums["projection_flops_per_launch"],
                # the fold pass the kernel cannot run without: its time (compress call minus the
                # timed kernel) and the bytes it moves (every non-sink row read once, written once)
                "fold_ms": fold_ms, "fold_bytes": 2 * nums["matrices"] * (cache_len - sink) * w.head_dim * 2,
                "frac_of_burst_peak_whole_call": nums["folded_flops"] / (compress_ms * 1e-3) / 1e12 / peaks["bf16_tflops"]}
    elif chosen == fk.FDCT:
        achieved = nums["algorithmic_bytes_per_launch"] / (kernel_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "peak_kind": "copy, of " + peaks["source"]}
    else:
        # fp32 FFMA: 148 SMs x 128 lanes x 2 flop x 1.965 GHz
        peak = 148 * 128 * 2 * 1.965e9 / 1e12
        achieved = nums["projection_flops_per_launch"] / (kernel_ms * 1e-3) / 1e12
        roof = {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_kind": "fp32 FFMA, derived from unit counts and max clock"}
    roof["kernel"] = chosen_name
    roof["kernel_ms"] = kernel_ms
    roof["launches_per_step"] = per_call
    roof["traffic"] = load_traffic(args.workload, chosen_name) if (args.retain == 0.5 and not first) else None

    # ---- end to end through the host-buffer entry point (rank-local pinned host cache)
    e2e = None
    if args.e2e_steps > 0:
        kh = torch.empty(k.shape, dtype=k.dtype, pin_memory=True)
        vh = torch.empty(v.shape, dtype=v.dtype, pin_memory=True)
        kh.copy_(k), vh.copy_(v)
        torch.cuda.synchronize()
        h2d = d2h = 0
        for i in range(1 + args.e2e_steps):
            if i == 1:
                barrier()
                torch.cuda.synchronize()
                t0 = time.perf_counter()
            _, h2d, d2h = ctx.compress_host(kh, vh, cache_len, kept, sink)
            torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt_ms = max_over_ranks(dt * 1e3 / args.e2e_steps, dev)
        e2e = {"value": n_gpus * nums["cache_in_bytes"] / (dt_ms * 1e-3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": dt_ms, "steps": args.e2e_steps,
               "call": "freqkv_compress_host, cache in pinned host memory"}
        del kh, vh

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": n_gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if w.dtype == torch.bfloat16 else "f32", "data": "synthetic",
            "config": {"workload": args.workload, "batch": w.batch, "layers": w.layers, "kv_heads": w.kv_heads,
                       "head_dim": w.head_dim, "capacity": w.capacity, "cache_len": cache_len, "sink": sink,
                       "kept_len": kept, "first_component": first, "appended_rows_per_step": n_new, "variant": chosen_name,
                       "l2": "inputs larger than L2 (%.2f GB of cache per step)" % (nums["cache_in_bytes"] / 1e9),
                       "parallelism": "replicas only" if n_gpus > 1 else "single GPU",
                       "step": "refused append (lazy trigger) + compress K,V in place + append chunk"},
            "compress_only": {"ms": compress_ms, "cache_in_GBps": nums["cache_in_bytes"] / (compress_ms * 1e-3) / 1e9,
                              "moved_GBps": nums["algorithmic_bytes"] / (compress_ms * 1e-3) / 1e9,
                              "hbm_floor_ms": nums["algorithmic_bytes"] / (peaks["hbm_gbs"] * 1e9) * 1e3},
            "append_only": {"ms": append_ms, "GBps": nums["append_bytes"] / (append_ms * 1e-3) / 1e9},
            "roofline": roof, "cpu_baseline": base, "e2e": e2e, "clocks": clocks,
            "gpu_launches": launches1 - launches0,
        }
        print(json.dumps(line), flush=True)
    ctx.close()
    if world > 1:
        import torch.distributed as dist

        dist.destroy_process_group()


if __name__ == "__main__":
    main()
