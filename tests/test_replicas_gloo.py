"""The N > 1 path is replicas with no data-path collective; what crosses ranks is the measurement.  Two gloo
ranks on CPU check the host logic: image shards are disjoint and cover the batch, seeds differ per rank, the
reported time is the slowest rank's and the throughput counts every rank's tokens."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2503_23367_b200 import replicas as R


def test_image_shards_partition_the_batch():
    for n in (0, 1, 2, 7, 8, 13):
        for w in (1, 2, 3, 8):
            shards = [R.image_shard(n, r, w) for r in range(w)]
            assert sorted(i for s in shards for i in s) == list(range(n))
            assert max(len(s) for s in shards) - min(len(s) for s in shards) <= 1
    with pytest.raises(ValueError):
        R.image_shard(4, 2, 2)
    assert R.world() == (0, 1) and R.max_over_ranks(3.5) == 3.5 and R.aggregate_throughput(10, 2) == 5.0
    assert len({R.rank_seed(40, r) for r in range(8)}) == 8


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world_size: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world_size))
    dist.init_process_group("gloo", rank=rank, world_size=world_size)
    try:
        assert R.world() == (rank, world_size)
        shard = R.image_shard(5, rank, world_size)
        # every rank "processes" its images; rank 1 is the slow one
        seconds = 0.25 * (rank + 1)
        tokens = 820.0 * len(shard)
        R.barrier()
        slowest = R.max_over_ranks(seconds)
        rate = R.aggregate_throughput(tokens, seconds)
        owned = torch.zeros(5, dtype=torch.int64)
        owned[list(shard)] = 1
        dist.all_reduce(owned)
        out.put((rank, slowest, rate, owned.tolist(), R.rank_seed(1000, rank)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_time_and_all_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, rate, owned, seed in got:
        assert slowest == 0.5                                   # max over ranks, on every rank
        assert abs(rate - 820.0 * 5 / 0.5) < 1e-9               # all ranks' tokens over the slowest time
        assert owned == [1, 1, 1, 1, 1]                         # each image owned exactly once
    assert got[0][4] != got[1][4]


def test_bench_started_plainly_with_gpus_n_launches_n_ranks(monkeypatch):
    """`python bench.py --gpus N` (no launcher around it) must itself start N ranks, one per GPU, on 127.0.0.1 and
    hand them its own arguments; under a launcher (WORLD_SIZE set) it must not."""
    import importlib
    import subprocess
    import sys

    bench = importlib.import_module("bench")
    seen = {}

    def fake_call(cmd, *a, **k):
        seen["cmd"] = cmd
        return 0

    monkeypatch.setattr(subprocess, "call", fake_call)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "4", "--steps", "2", "--warmup", "3"])
    with pytest.raises(SystemExit) as e:
        bench.main()
    assert e.value.code == 0
    cmd = seen["cmd"]
    assert "torch.distributed.run" in cmd and "--nproc-per-node=4" in cmd and "127.0.0.1" in cmd
    assert cmd[-6:] == ["--gpus", "4", "--steps", "2", "--warmup", "3"] and cmd[-7].endswith("bench.py")
