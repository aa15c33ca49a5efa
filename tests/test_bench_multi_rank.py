"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own replica time; rank 0 must
report the aggregate over both replicas at the slowest rank's time."""
import os
import sys

import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 2.0 if rank == 0 else 3.5                # rank 1 is the slow replica
    ms = bench.max_over_ranks(local_ms, world, device="cpu")
    val = bench.aggregate_value(1_000_000_000, world, ms * 1e-3)
    dist.barrier()
    out.put((rank, ms, val))
    dist.destroy_process_group()


def test_two_rank_aggregation_on_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, val in res:
        assert ms == pytest.approx(3.5)                                  # max over ranks on every rank
        assert val == pytest.approx(2 * 1.0 / 3.5e-3)                    # 2 GB over 3.5 ms, in GB/s


def test_byte_accounting_of_the_algorithmic_bytes():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.linear_bytes(16, 2560, 9728, 128) == 13_331_456
    assert bench.linear_bytes(16, 9728, 2560, 128) == 13_331_456
    assert bench.linear_bytes(16, 2560, 6144, 128) == 8_450_048
    assert bench.linear_bytes(16, 4096, 2560, 128) == 5_660_672
    total, per_layer = bench.step_bytes(16, 128, 36, lm_head=False)
    assert per_layer == 54_105_088 and total == 1_947_783_168
