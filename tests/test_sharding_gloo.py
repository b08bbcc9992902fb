"""The N > 1 host logic on CPU: two gloo ranks, sequences partitioned with no data-path exchange."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2502_19078_b200 import sharding


def test_shard_range_partitions_exactly():
    for n in (0, 1, 7, 16, 17, 256):
        for world in (1, 2, 3, 8):
            covered = []
            for r in range(world):
                lo, hi = sharding.shard_range(n, r, world)
                assert 0 <= lo <= hi <= n
                covered += list(range(lo, hi))
            assert covered == list(range(n))
            sizes = sharding.shard_sizes(n, world)
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.shard_range(4, 2, 2)


def test_single_process_is_identity():
    assert sharding.max_over_ranks(3.5) == 3.5
    rate, ms = sharding.whole_job_rate(100, 50.0)
    assert ms == 50.0 and abs(rate - 2000.0) < 1e-9


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = sharding.shard_range(5, rank, world)          # 5 sequences over 2 ranks: 2 + 3
        units = (hi - lo) * 128                                 # decode tokens this rank processed
        elapsed = 10.0 if rank == 0 else 25.0                   # rank 1 is the slow one
        dist.barrier()
        rate, ms = sharding.whole_job_rate(units, elapsed)
        out[rank] = (lo, hi, rate, ms)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_report_the_whole_job():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(2, port, out), nprocs=2, join=True)
    assert out[0][:2] == (0, 2) and out[1][:2] == (2, 5)
    for r in (0, 1):
        _, _, rate, ms = out[r]
        assert ms == 25.0                                        # max over ranks
        assert abs(rate - 5 * 128 / 25e-3) < 1e-6                # all ranks' tokens / slowest time
