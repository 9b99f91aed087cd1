"""The multi-rank path on CPU: two or three gloo ranks split the chains of one job, each runs its range (here with
the oracle standing in for the GPU, which this container lacks) and the ranks agree on the winner. The result must
equal a single-process run over all chains, also when the winner belongs to the last rank."""
import os
import socket

import numpy as np
import torch.multiprocessing as mp

from paper_2508_13231_b200 import sharding, workloads as wl

GB = 10 ** 9
TOTAL, MOVES = 11, 1500          # odd chain count: the two ranges differ in length


# a small instance on which every chain finds the optimum (the winner is a tie, resolved to chain 0), and a larger
# one with a short, cold search on which the chains end apart and chain 9 of 11 wins (the last rank's range)
CASES = {"small": dict(shape=(48, 24, 12), access_seed=31, kw=dict(moves=MOVES, seed=7, levels=8)),
         "apart": dict(shape=(200, 60, 50), access_seed=32, kw=dict(moves=600, seed=11, levels=8, p0=0.01))}


def _problem(case="small"):
    from oracle import kvpo
    U, S, cap = CASES[case]["shape"]
    A = wl.random_access(U, S, 0.3, seed=CASES[case]["access_seed"])
    return kvpo.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)


def _rank(rank, world, port, out, case="small"):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    o = _problem(case)
    first, count = sharding.chain_range(rank, world, TOTAL)
    res = o.anneal(o.make_params(chains=count, first_chain=first, **CASES[case]["kw"]))
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


def test_three_ranks_winner_on_the_last_rank():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, 3, port, q, "apart")) for r in range(3)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    o = _problem("apart")
    ref = o.anneal(o.make_params(chains=TOTAL, **CASES["apart"]["kw"]))
    assert [(g[1], g[2]) for g in got] == [(0, 4), (4, 4), (8, 3)]
    assert ref["best_chain"] >= 8                                            # the last rank's range holds the winner
    ticks = [r.best_ticks for r in ref["per_chain"]]
    assert ticks.count(min(ticks)) == 1 and len(set(ticks)) >= 3             # the chains really ended apart
    for g in got:
        assert (g[5], g[6]) == (ref["best_ticks"], ref["best_chain"])
    assert got[2][3] == ref["best_ticks"] and got[0][3] > ref["best_ticks"] and got[1][3] > ref["best_ticks"]


def _xrank(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    o = _problem("apart")
    first, count = sharding.ladder_range(rank, world, 20, 4)
    res = o.anneal_exchange(o.make_params(chains=count, first_chain=first, **XKW), 4, 25)
    ticks, chain = sharding.combine_best(dist, res["best_ticks"], res["best_chain"])
    out.put((rank, first, count, [r.astuple() for r in res["per_chain"]], res["final_rung"].tolist(), ticks, chain))
    dist.barrier()
    dist.destroy_process_group()


XKW = dict(moves=1500, levels=4, p0=0.4, alpha=0.5, seed=13)


def test_ladder_range_keeps_ladders_whole():
    for total, rungs in ((20, 4), (8, 8), (36, 3)):
        for world in (1, 2, 3, 5):
            parts = [sharding.ladder_range(r, world, total, rungs) for r in range(world)]
            assert parts[0][0] == 0 and sum(c for _, c in parts) == total
            assert all(f % rungs == 0 and c % rungs == 0 for f, c in parts)
            assert all(parts[i][0] + parts[i][1] == parts[i + 1][0] for i in range(world - 1))


def test_replica_exchange_split_by_ladders_over_two_ranks():
    """Five ladders of four replicas over two ranks (three and two ladders): every chain, the rungs held at the end
    and the agreed winner equal those of one process running all twenty chains."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_xrank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    o = _problem("apart")
    ref = o.anneal_exchange(o.make_params(chains=20, **XKW), 4, 25)
    assert [(g[1], g[2]) for g in got] == [(0, 12), (12, 8)]
    assert got[0][3] + got[1][3] == [r.astuple() for r in ref["per_chain"]]
    assert got[0][4] + got[1][4] == ref["final_rung"].tolist()
    assert ref["n_exchanged"].sum() > 0
    for g in got:
        assert (g[5], g[6]) == (ref["best_ticks"], ref["best_chain"])
