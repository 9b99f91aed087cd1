"""The multi-rank path on CPU: two gloo ranks split the chains of one job, each runs its range (here with the
oracle standing in for the GPU, which this container lacks) and the ranks agree on the winner. The result must
equal a single-process run over all chains."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2508_13231_b200 import sharding, workloads as wl

GB = 10 ** 9
TOTAL, MOVES = 11, 1500          # odd chain count: the two ranges differ in length


def _problem():
    from oracle import kvpo
    U, S, cap = 48, 24, 12
    A = wl.random_access(U, S, 0.3, seed=31)
    return kvpo.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)


def _rank(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    o = _problem()
    first, count = sharding.chain_range(rank, world, TOTAL)
    res = o.anneal(o.make_params(chains=count, moves=MOVES, seed=7, levels=8, first_chain=first))
    ticks, chain = sharding.combine_best(dist, res["best_ticks"], res["best_chain"])
    out.put((rank, first, count, res["best_ticks"], res["best_chain"], ticks, chain))
    dist.barrier()
    dist.destroy_process_group()


def test_chain_range_is_a_partition():
    for total in (1, 7, 1024, 1025):
        for world in (1, 2, 3, 8):
            parts = [sharding.chain_range(r, world, total) for r in range(world)]
            assert parts[0][0] == 0 and sum(c for _, c in parts) == total
            assert all(parts[i][0] + parts[i][1] == parts[i + 1][0] for i in range(world - 1))
            assert max(c for _, c in parts) - min(c for _, c in parts) <= 1


def test_two_ranks_agree_with_one_process():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    o = _problem()
    ref = o.anneal(o.make_params(chains=TOTAL, moves=MOVES, seed=7, levels=8))
    assert [(g[1], g[2]) for g in got] == [(0, 6), (6, 5)]
    for g in got:
        assert (g[5], g[6]) == (ref["best_ticks"], ref["best_chain"])       # both ranks hold the global winner
    assert min(g[3] for g in got) == ref["best_ticks"]
    assert np.all([g[0] in (0, 1) for g in got])
