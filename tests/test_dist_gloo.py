"""The N>1 plumbing on CPU: two gloo ranks shard a batch and reduce their timings."""
import os
import socket

import torch.multiprocessing as mp

from paper_1611_07151_b200 import dist as D


def test_shard_covers_the_batch_without_overlap():
    for total in (1, 7, 256, 257):
        for world in (1, 2, 3, 8):
            parts = [D.shard(total, r, world) for r in range(world)]
            assert parts[0][0] == 0 and parts[-1][1] == total
            assert all(parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in parts]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    assert D.init("gloo") == world
    lo, hi = D.shard(10, rank, world)
    D.barrier()
    value, ms = D.job_throughput(units_local=(hi - lo) * 4, ms_local=100.0 * (rank + 1))
    out.put((rank, lo, hi, value, ms))
    D.barrier()


def test_two_gloo_ranks_take_max_time_and_sum_units():
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
    assert [(r[1], r[2]) for r in res] == [(0, 5), (5, 10)]
    for r in res:
        assert r[4] == 200.0                       # slowest rank
        assert abs(r[3] - 40 / 0.2) < 1e-9         # all units / slowest time
