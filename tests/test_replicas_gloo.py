"""The N > 1 path of bench.py is "replicas only": no exchange on the data path, only a barrier
and a max-over-ranks of the timing.  World-size-2 gloo run on CPU of exactly those helpers, and
of the reference arm's rule that rank 0 alone works and prints."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    sys.path.insert(0, ROOT)
    import bench

    dist.init_process_group("gloo", rank=rank, world_size=world)
    bench.barrier()
    slowest = bench.max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))
    assert bench.dist_env() == (rank, rank, world)
    out[rank] = slowest
    dist.destroy_process_group()


def test_max_over_ranks_and_barrier_world2():
    port = free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
        assert dict(out) == {0: 15.0, 1: 15.0}  # every rank sees the slowest rank's time


def test_single_process_helpers_are_no_ops():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(3.5, torch.device("cpu")) == 3.5
    bench.barrier()
    n = bench.workload_numbers(__import__("paper_2505_00570_b200.synth", fromlist=["x"]).WORKLOADS["llama2_7b"], 4096, 2046, 4)
    assert n["matrices"] == 2048
    assert n["cache_in_bytes"] == 2048 * 4096 * 128 * 2
    assert n["algorithmic_bytes"] == 2048 * (4092 + 2046) * 128 * 2
    assert n["projection_flops"] == 2.0 * 2046 * 4092 * 128 * 2048
    # 4092 -> 2046 halves twice: 512 twice-folded rows x (1023 + 1023 + 2046 + 2046) columns, three quarters of one level
    assert n["fold_levels"] == 2 and n["folded_flops"] == 2.0 * 512 * 3 * 2046 * 128 * 2048
    one = bench.workload_numbers(__import__("paper_2505_00570_b200.synth", fromlist=["x"]).WORKLOADS["llama2_7b"], 4096, 2045, 4)
    assert one["fold_levels"] == 1 and one["folded_flops"] == 2.0 * 2 * 1023 * 2046 * 128 * 2048


def test_reference_arm_rank0_only_prints():
    env = dict(os.environ, OMP_NUM_THREADS="2")
    outs = []
    for rank in (0, 1):
        e = dict(env, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2")
        r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                            "--steps", "1", "--warmup", "0", "--workload", "tiny"],
                           capture_output=True, text=True, env=e, timeout=300)
        assert r.returncode == 0, r.stderr
        outs.append(r.stdout.strip())
    line = json.loads(outs[0])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0
    assert outs[1] == ""
