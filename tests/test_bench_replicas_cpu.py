"""The multi-GPU path of bench.py is N independent replicas (the layer has no exchange step): the only
cross-rank logic is "time = slowest rank, throughput = N x bytes / time".  Exercised here with two gloo ranks
on the CPU, and the rank/world parsing of the launcher environment."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    assert bench.dist_env() == (rank, world, rank)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
        ms = bench.max_over_ranks(local_ms, world)
        dist.barrier()
        out[rank] = (ms, bench.job_throughput_gbs(ms / 100.0, world))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_the_summed_throughput():
    import bench
    world = 2
    port = 29500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, gbs = res[0]
    assert ms == 15.0
    assert gbs == pytest.approx(2 * bench.STEP_BYTES / (15.0 / 100.0 * 1e-3) / 1e9)
    # one rank: no process group needed
    assert bench.max_over_ranks(7.5, 1) == 7.5
    assert bench.job_throughput_gbs(0.05, 1) == pytest.approx(bench.STEP_BYTES / 0.05e-3 / 1e9)


def test_step_bytes_match_the_storage_model():
    import bench
    # 7 matrices of a LLaMA-3-8B layer: 2-bit planes + fp16 scale pairs + x + y
    total = 0
    for n, k in ((4096, 4096), (1024, 4096), (1024, 4096), (4096, 4096), (14336, 4096), (14336, 4096), (4096, 14336)):
        total += n * k // 2 + 4 * n * k // 128 + 2 * k + 2 * n
    assert bench.STEP_BYTES == total == 116031488
