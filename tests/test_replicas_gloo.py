"""The multi-GPU path is "replicas only": this covers its host-side plumbing with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_03586_b200 import replicas


def test_shard_sequences_partitions_exactly():
    for n, world in ((32, 8), (32, 3), (5, 8), (0, 2), (7, 7)):
        got = [i for r in range(world) for i in replicas.shard_sequences(n, r, world)]
        assert got == list(range(n))
        sizes = [len(replicas.shard_sequences(n, r, world)) for r in range(world)]
        assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        replicas.shard_sequences(4, 2, 2)


def test_single_process_is_identity():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    r = replicas.whole_job_rate(10.0, 2.0)
    assert r == {"world": 1, "ms_per_step": 2.0, "units_per_s": 5000.0}


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms_local = 2.0 + rank          # rank 1 is the slow one
        r = replicas.whole_job_rate(100.0, ms_local)
        mx = replicas.max_over_ranks([float(rank), 7.0 - rank])
        out.put((rank, r, mx, list(replicas.shard_sequences(5, rank, world))))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_rank_and_sum_the_work():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, r, mx, shard in results:
        assert r["world"] == 2 and r["ms_per_step"] == 3.0
        assert abs(r["units_per_s"] - 2 * 100.0 / 3e-3) < 1e-6
        assert mx == [1.0, 7.0]
    assert results[0][3] + results[1][3] == [0, 1, 2, 3, 4]
