"""world_size-2 gloo tests (CPU) of the host logic bench.py uses when it runs on more than one GPU."""
import os
import socket

import pytest

from paper_2609_14339_b200 import multi
from synth.generator import config_shapes


def test_shard_matrices_partition_is_disjoint_complete_and_balanced():
    shapes = config_shapes("llama8b")
    for world in (1, 2, 4, 8):
        parts = multi.shard_matrices(shapes, world)
        flat = sorted(i for p in parts for i in p)
        assert flat == list(range(len(shapes)))
        loads = [sum(shapes[i][0] * shapes[i][1] for i in p) for p in parts]
        assert max(loads) - min(loads) <= max(m * n for m, n in shapes)
        assert parts == multi.shard_matrices(shapes, world)          # deterministic
    with pytest.raises(ValueError):
        multi.shard_matrices(shapes, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = multi.max_over_ranks(10.0 + 5.0 * rank)                 # rank 1 is slower
        sq = multi.global_sqnorm(float((rank + 1) ** 2))            # 1 + 4
        parts = multi.shard_matrices([(4, 4), (8, 8), (2, 2), (8, 4)], world)
        dist.barrier()
        q.put((rank, ms, sq, parts[rank], multi.whole_job_throughput(100.0, world, ms)))
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo_max_time_and_norm():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]                       # both ranks report the slowest rank's time
    assert [g[2] for g in got] == [5.0, 5.0]
    assert sorted(got[0][3] + got[1][3]) == [0, 1, 2, 3] and not set(got[0][3]) & set(got[1][3])
    assert abs(got[0][4] - 2 * 100.0 / 15e-3) < 1e-6


def test_helpers_are_identity_without_a_process_group():
    assert multi.max_over_ranks(3.5) == 3.5
    assert multi.global_sqnorm(2.0) == 2.0
