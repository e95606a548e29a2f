"""The N-GPU path is batch sharding with no data-path collective: test the host logic with two
gloo ranks on CPU (ranges partition the batch; the timing reduction takes the slowest rank)."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2511_15898_b200 import sharding as S


def test_shard_ranges_partition_the_batch():
    for batch in (0, 1, 7, 1024, 4097):
        for world in (1, 2, 3, 8):
            got = [S.shard_range(batch, world, r) for r in range(world)]
            assert got[0][0] == 0 and got[-1][1] == batch
            for a, b in zip(got, got[1:]):
                assert a[1] == b[0]
            sizes = [hi - lo for lo, hi in got]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        S.shard_range(10, 2, 2)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    lo, hi = S.shard_range(1001, world, rank)
    # every rank "processes" its slice; rank 1 is slower
    secs = 0.5 + rank
    dist.barrier()
    slowest = S.max_over_ranks(secs)
    thr = S.aggregate_throughput(500, secs)
    rows = torch.tensor([hi - lo], dtype=torch.int64)
    dist.all_reduce(rows)             # test-only check that the slices cover the batch
    out.put((rank, lo, hi, slowest, thr, int(rows.item())))
    dist.destroy_process_group()


def test_two_gloo_ranks_share_a_batch_and_report_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, lo0, hi0, s0, t0, n0), (r1, lo1, hi1, s1, t1, n1) = res
    assert (lo0, hi0, lo1, hi1) == (0, 501, 501, 1001)
    assert s0 == s1 == 1.5 and n0 == n1 == 1001
    assert abs(t0 - 2 * 500 / 1.5) < 1e-9 and t0 == t1
