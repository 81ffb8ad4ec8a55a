"""The N > 1 host logic on CPU: two gloo ranks shard the batch rows, take the maximum of their
timings and the sum of their unit counts, exactly as the benchmark does around its timed region."""
import os
import socket

import pytest
import torch.multiprocessing as mp

from paper_2608_15533_b200 import launch


def test_shard_rows_covers_every_row_once():
    for rows in (1, 7, 128, 513):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                first, n = launch.shard_rows(rows, world, r)
                seen += list(range(first, first + n))
            assert seen == list(range(rows))
            sizes = [launch.shard_rows(rows, world, r)[1] for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    assert launch.init("gloo") == (rank, world, rank)
    first, n = launch.shard_rows(129, world, rank)
    launch.barrier()
    ms = launch.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slow one
    units = launch.sum_over_ranks(n * 32)
    q.put((rank, first, n, ms, units))
    launch.finalize()


def test_two_gloo_ranks_max_time_and_total_units():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1:3] for r in res] == [(0, 65), (65, 64)]
    assert all(r[3] == 15.0 for r in res)                   # both ranks report the maximum
    assert all(r[4] == 129 * 32 for r in res)               # whole-job units


def test_single_process_is_a_no_op():
    assert launch.max_over_ranks(3.5) == 3.5 and launch.sum_over_ranks(7) == 7.0
    launch.barrier()
