"""The N > 1 plumbing on CPU: two gloo ranks shard independent units and agree on the max time."""
import os
import socket

import torch.multiprocessing as mp

from paper_2604_09244_b200 import dist as D


def test_shard_covers_all_units_once():
    for n in (1, 7, 16, 33):
        for world in (1, 2, 3, 8):
            got = [u for r in range(world) for u in D.shard(n, r, world)]
            assert got == list(range(n))
            sizes = [len(D.shard(n, r, world)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, _, w = D.init("gloo")
    units = D.shard(5, r, w)
    D.barrier(w)
    slowest = D.max_over_ranks(1.0 + r, w)
    total = D.sum_over_ranks(len(units), w)
    q.put((r, units, slowest, total))


def test_two_gloo_ranks_agree_on_max_time_and_total_units():
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
    assert res[0][1] == [0, 1, 2] and res[1][1] == [3, 4]
    assert all(r[2] == 2.0 and r[3] == 5.0 for r in res)
