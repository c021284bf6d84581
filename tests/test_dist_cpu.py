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


# ---------------------------------------------------------------- head-sharded scores
def _tp_worker(rank, world, port, q):
    import numpy as np
    import torch
    import oracle
    from paper_2604_09244_b200 import tensor_parallel as TP
    from paper_2604_09244_b200 import workloads as W
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    D.init("gloo")
    wl = W.small_workload(71, batch=1, D=64, H=4, d=16, dtype="fp32", n_txt=(5,), n_2d=(23,), n_3d=(31,))
    t, s = wl.steps[0], wl.samples[0]
    ql = TP.head_shard(torch.from_numpy(t.q), rank, world).numpy()
    kl = TP.head_shard(torch.from_numpy(t.k), rank, world).numpy()
    local = torch.from_numpy(oracle.salience(ql, kl, 4 // world, 16, s))      # mean over this rank's heads
    TP.average_over_ranks_(local)
    full = oracle.salience(t.q, t.k, 4, 16, s)
    q.put((rank, float(np.abs(local.numpy() - full).max() / full.max()), local.numpy().tobytes()))


def test_head_sharded_scores_average_to_the_full_scores():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_tp_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(r[1] < 1e-13 for r in res)              # the mean of the ranks' means is the mean over all heads
    assert res[0][2] == res[1][2]                      # and every rank holds the same bits: same decisions downstream
