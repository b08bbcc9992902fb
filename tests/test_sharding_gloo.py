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


_RANK_SCRIPT = r"""
import json, os, sys
import torch.distributed as dist
sys.path.insert(0, os.environ["CLADA_ROOT"])
from paper_2502_19078_b200 import sharding
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert int(os.environ["LOCAL_RANK"]) == rank and os.environ["MASTER_ADDR"] == "127.0.0.1"
dist.init_process_group("gloo", rank=rank, world_size=world)
rate, ms = sharding.whole_job_rate(100.0 * (rank + 1), 10.0 * (rank + 1))
dist.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": world, "rate": rate, "ms": ms}), flush=True)
dist.destroy_process_group()
"""


def test_launch_ranks_starts_one_process_per_rank(tmp_path, capfd):
    """The launcher behind `bench.py --gpus N`: N children, each with its rank and the world size, rendezvous on
    127.0.0.1, rank 0's line reports the whole job."""
    import json
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    rc = sharding.launch_ranks(2, [str(script)], devices_available=2, timeout_s=120, extra_env={"CLADA_ROOT": root})
    assert rc == 0
    out = capfd.readouterr().out
    rec = json.loads([l for l in out.splitlines() if l.startswith("{")][0])
    assert rec["n_gpus"] == 2 and rec["ms"] == 20.0 and abs(rec["rate"] - 300.0 / 20e-3) < 1e-6


def test_launch_ranks_refuses_more_ranks_than_devices(tmp_path):
    with pytest.raises(ValueError, match="more devices"):
        sharding.launch_ranks(4, ["-c", "pass"], devices_available=1)


def test_launch_ranks_reports_a_failed_rank(tmp_path):
    script = tmp_path / "fail.py"
    script.write_text("import os, sys, time\nif os.environ['RANK'] == '1':\n    sys.exit(3)\ntime.sleep(30)\n")
    rc = sharding.launch_ranks(2, [str(script)], devices_available=2, timeout_s=60)
    assert rc != 0


def test_bench_gpus_flag_refuses_without_devices():
    """`python bench.py --gpus 2` started by hand becomes the launcher; on a box with fewer devices it says so."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    if torch.cuda.device_count() >= 2:
        pytest.skip("this box has the devices")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "1"],
                         capture_output=True, text=True, timeout=300, env=env, cwd=root)
    assert out.returncode != 0 and "more devices" in out.stderr
