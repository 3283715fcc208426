"""The benchmark's N > 1 bookkeeping on CPU ranks (gloo, world size 2): every rank runs one replica of the workload,
the slowest rank's time decides, and the reported value is the work of all ranks over that time."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 0 is fast, rank 1 slow: per-phase times in ms over 10 steps
    mine = [10.0, 30.0, 41.0] if rank == 0 else [12.5, 28.0, 43.0]
    got = bench.max_over_ranks(mine, dist, "cpu")
    dist.barrier()
    if rank == 0:
        out.put(got)
    dist.destroy_process_group()


def test_two_cpu_ranks_take_the_slowest_time_and_sum_the_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert got == [12.5, 30.0, 43.0]
    sys.path.insert(0, ROOT)
    import bench
    # 2 replicas x 100 units x 10 steps over 12.5 ms
    assert bench.throughput(2, 100.0, 10, got[0]) == pytest.approx(2 * 100.0 * 10 / 12.5e-3)
    assert bench.max_over_ranks([1.0, 2.0], None, "cpu") == [1.0, 2.0]


def test_workload_constants_match_the_llama2_7b_shapes():
    sys.path.insert(0, ROOT)
    import bench
    import sasq_workloads as W
    elems = 2048 * (6 * 4096 + 11008)
    assert bench.quantizer_bytes(2048) == 8 * elems == 583_008_256
    assert bench.linear_ops(2048) == 2 * 2048 * sum(K * N for _, K, N in W.LLAMA2_7B_LINEARS) == 828_928_688_128
    # the full stack: 32 layers over 8 x 2048 tokens, 224 quantizers
    assert bench.quantizer_bytes(16384, 32) == 32 * 8 * 16384 * (6 * 4096 + 11008)
    assert bench.linear_ops(16384, 32) == 32 * 8 * bench.linear_ops(2048)
    assert "T16384" in bench.workload_name(32, 16384) and "32_layers" in bench.workload_name(32, 16384)


def test_tensor_peak_follows_the_length_of_the_timed_region():
    sys.path.insert(0, ROOT)
    import bench
    peaks = {"bf16_tflops": 1600.0, "bf16_tflops_sustained": 1400.0}
    assert bench.tensor_peak_for(0.0075, peaks, "measured")[0] == 3200.0        # a burst of a few ms
    assert bench.tensor_peak_for(2.5, peaks, "measured")[0] == 2800.0           # seconds under the power cap
    assert "burst" in bench.tensor_peak_for(0.0075, peaks, "measured")[1]
    assert "sustained" in bench.tensor_peak_for(2.5, peaks, "measured")[1]
