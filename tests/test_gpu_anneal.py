"""Annealing kernels vs oracle: per-chain trajectories, bound and winner schedule, all bit-exact."""
import os

import numpy as np
import pytest
import torch

from paper_2508_13231_b200 import workloads as wl
from gpu_util import both_problems, named_problem, to_dev, to_np, trace_on_gpu
from oracle_pool import oracle_chains_parallel

pytestmark = pytest.mark.gpu
GB = 10 ** 9
NEVER = 2 ** 64 - 1


@pytest.fixture(scope="module")
def kvp():
    from paper_2508_13231_b200 import kvp
    return kvp


@pytest.fixture(params=[3, 1, 2], ids=["wide", "narrow1", "narrow2"])
def warps_per_chain(request, hooks):
    """The wide chain kernel (one warp per chain, four proposals per lane; the library's choice for jobs of many
    chains) and both forms of the narrow one (one proposal per lane; one warp per chain, or two warps that take a
    chain's batches in turn; the choice for few chains)."""
    hooks(warps_per_chain=request.param)
    return request.param


def _params(g, o, **kw):
    return g.make_params(**kw), o.make_params(**kw)


def _check_against_oracle(g, o, gp, op, chains_to_check=None, check_schedule=True):
    out = g.anneal(gp, want_per_chain=True)
    stats = out["stats"]
    temps, mean = o.temps(op)
    assert stats.calib_mean_delta == mean and stats.temp0 == temps[0]
    chains = range(gp.chains) if chains_to_check is None else chains_to_check
    for c in chains:
        want, _, _ = o.anneal_chains(op, c, 1)
        assert out["per_chain"][c].astuple() == want[0].astuple(), c
    if check_schedule and chains_to_check is None:
        ref = o.anneal(op)
        assert out["best_ticks"] == ref["best_ticks"] and stats.best_chain == ref["best_chain"]
        assert np.array_equal(to_np(out["best_schedule"]), ref["best_schedule"])
        assert out["best_seconds"] == pytest.approx(ref["best_seconds"], rel=1e-9)
    assert stats.moves_total == sum(r.moves_done for r in out["per_chain"])
    assert stats.best_ticks == min(r.best_ticks for r in out["per_chain"])
    return out


def test_anneal_tiny_all_chains(kvp, oracle, warps_per_chain):
    g, o, cfg, A = named_problem(kvp, oracle, "tiny")
    for p0 in (0.8, 1e-3):
        gp, op = _params(g, o, chains=cfg["chains"], moves=cfg["moves"], seed=0, p0=p0)
        out = _check_against_oracle(g, o, gp, op)
        assert out["stats"].init_ticks == o.eval(o.init_placement(1))["total_ticks"]


@pytest.mark.parametrize("U,S,cap,bw,flags", [
    (45, 40, 12, (4900, 900, 500), 3),      # odd sizes, ragged words both ways, Table I weights
    (33, 1, 5, (8000, 900, 900), 3),        # a single step: no migration can ever be charged
    (1, 7, 1, (8000, 900, 900), 3),         # a single unit
    (64, 95, 0, (8000, 900, 900), 3),       # nothing fits in HBM: every flip-in is infeasible
    (64, 64, 64, (8000, 900, 900), 3),      # everything fits
    (200, 130, 37, (4900, 500, 900), 2),    # link slower than DRAM, migrations free on the HBM side
    (90, 33, 20, (3, 1, 1), 0),             # free migration
])
def test_anneal_small_shapes(kvp, oracle, U, S, cap, bw, flags, warps_per_chain):
    A = wl.random_access(U, S, 0.3, seed=U + S)
    hw = (np.arange(S) % 2).astype(np.uint32)
    ew = (np.arange(S) % 3).astype(np.uint32)
    g, o = both_problems(kvp, oracle, U, 8192, S, A, cap, tuple(b * GB for b in bw), mig_flags=flags, hw=hw, ew=ew)
    for init in (kvp.INIT_STATIC_FIRST, kvp.INIT_STATIC_FREQ):
        gp, op = _params(g, o, chains=9, moves=3001, seed=12345678901234, levels=7, init_mode=init, p_swap_256=100,
                         max_len_log2=4)
        _check_against_oracle(g, o, gp, op)


def test_anneal_options(kvp, oracle, warps_per_chain):
    U, S, cap = 120, 70, 30
    A = wl.random_access(U, S, 0.25, seed=3)
    g, o = both_problems(kvp, oracle, U, 8192, S, A, cap, (8000 * GB, 900 * GB, 900 * GB))
    # caller-supplied temperature ladder, only flips / only swaps, a single level, fewer moves than levels
    for kw in (dict(chains=5, moves=2000, levels=4, temps=[900.0, 90.0, 9.0, 0.5]),
               dict(chains=5, moves=2000, levels=3, p_swap_256=0), dict(chains=5, moves=2000, levels=3, p_swap_256=256),
               dict(chains=3, moves=500, levels=1), dict(chains=3, moves=5, levels=16), dict(chains=1, moves=1),
               dict(chains=4, moves=64000, levels=64, early_stop_permille=1),
               dict(chains=4, moves=64000, levels=64, early_stop_permille=5, early_stop_from_level=30, p0=0.01),
               dict(chains=40, moves=777, levels=5, max_len_log2=0, seed=2 ** 63 + 5)):
        gp, op = _params(g, o, **kw)
        _check_against_oracle(g, o, gp, op)
    # a slice of a larger job: chains 5..9 behave exactly as in a run of chains 0..15
    gp16, op16 = _params(g, o, chains=16, moves=1500, levels=5)
    gp5, _ = _params(g, o, chains=5, moves=1500, levels=5, first_chain=5)
    whole, part = g.anneal(gp16, want_per_chain=True), g.anneal(gp5, want_per_chain=True)
    assert [r.astuple() for r in part["per_chain"]] == [r.astuple() for r in whole["per_chain"][5:10]]
    assert 5 <= part["stats"].best_chain < 10
    ref = o.anneal(o.make_params(chains=5, moves=1500, levels=5, first_chain=5))
    assert (part["best_ticks"], part["stats"].best_chain) == (ref["best_ticks"], ref["best_chain"])
    assert np.array_equal(to_np(part["best_schedule"]), ref["best_schedule"])
    # user-supplied initial schedule
    init = wl.random_schedules(U, S, cap, 1, seed=4, churn=0.1)[0]
    gp = g.make_params(chains=6, moves=1500, levels=5, init_mode=kvp.INIT_USER, init_schedule=to_dev(init))
    op = o.make_params(chains=6, moves=1500, levels=5, init_mode=oracle.INIT_USER, init_schedule=init)
    _check_against_oracle(g, o, gp, op)
    # an infeasible initial schedule is refused (Eq. 5)
    bits = wl.unpack_bits(init, U); bits[10, :cap + 1] = 1
    gp = g.make_params(chains=2, moves=10, init_mode=kvp.INIT_USER, init_schedule=to_dev(wl.pack_bits(bits)))
    with pytest.raises(kvp.KvpError) as e:
        g.anneal(gp)
    assert e.value.code == kvp.ERR_CAPACITY
    for bad in (dict(chains=0, moves=10), dict(chains=1, moves=0), dict(chains=1, moves=1, max_len_log2=6),
                dict(chains=1, moves=1, p0=1.5), dict(chains=1, moves=1, levels=0)):
        with pytest.raises(kvp.KvpError) as e:
            g.anneal(g.make_params(**bad))
        assert e.value.code == kvp.ERR_ARG


def test_chain_state_replay(kvp, oracle):
    U, S, cap = 150, 100, 40
    A = wl.random_access(U, S, 0.25, seed=8)
    g, o = both_problems(kvp, oracle, U, 8192, S, A, cap, (4900 * GB, 900 * GB, 500 * GB))
    gp, op = _params(g, o, chains=4, moves=5000, levels=10, seed=99)
    for chain, upto in [(0, 0), (1, 1), (2, 31), (3, 33), (2, 1234), (3, 5000), (0, 99999)]:
        sched, res = g.chain_state(gp, chain, upto)
        want, fin, _ = o.anneal_chains(op, chain, 1, upto_moves=min(upto, 5000), want_final=True)
        assert np.array_equal(to_np(sched), fin[0]), (chain, upto)
        assert res.astuple() == want[0].astuple()
        assert int(g.eval(sched)["total_ticks"][0]) == want[0].final_ticks


def test_anneal_single_head_benchmark_configuration(kvp, oracle):
    # the configuration the benchmark times: 1024 chains x 100k moves, schedule resident in shared memory.
    # The oracle replays chains on the host cores (as many as the time allows) plus the winner.
    g, o, cfg, A = named_problem(kvp, oracle, "single_head")
    kw = dict(chains=cfg["chains"], moves=cfg["moves"], seed=0, p0=cfg.get("p0", 0.8))
    gp, op = _params(g, o, **kw)
    out = g.anneal(gp, want_per_chain=True)
    cores = os.cpu_count() or 1
    n_check = 1024 if cores >= 32 else (256 if cores >= 8 else 64)
    want = oracle_chains_parallel("single_head", kw, n_check)
    got = [r.astuple() for r in out["per_chain"][:n_check]]
    assert got == want
    st = out["stats"]
    w = st.best_chain
    ref, _, bst = o.anneal_chains(op, w, 1, want_best=True)
    assert ref[0].astuple() == out["per_chain"][w].astuple()
    assert np.array_equal(to_np(out["best_schedule"]), bst[0])
    assert out["best_ticks"] == ref[0].best_ticks == min(r.best_ticks for r in out["per_chain"])
    assert o.eval(bst[0])["total_ticks"] == out["best_ticks"] and o.eval(bst[0])["bad_step"] == -1
    assert st.moves_total == 1024 * 100_000


def test_anneal_layer_8b_global_state(kvp, oracle):
    # schedule too large for shared memory: chain state lives in global scratch
    g, o, cfg, A = named_problem(kvp, oracle, "layer_8b")
    kw = dict(chains=64, moves=20_000, seed=0, p0=1e-3)
    gp, op = _params(g, o, **kw)
    out = _check_against_oracle(g, o, gp, op, chains_to_check=[0, 1, 31, 63], check_schedule=False)
    w = out["stats"].best_chain
    ref, _, bst = o.anneal_chains(op, w, 1, want_best=True)
    assert np.array_equal(to_np(out["best_schedule"]), bst[0]) and out["best_ticks"] == ref[0].best_ticks


def _spread(chains):
    """Chain indices that fall into every wave of a job however it is cut: both ends, both sides of every 1/8th
    boundary (waves are equal parts of the job), and a few in between."""
    picks = {0, 1, chains - 2, chains - 1}
    for k in range(1, 8):
        picks |= {k * chains // 8 - 1, k * chains // 8}
    picks |= {(k * 2654435761) % chains for k in range(1, 5)}
    return sorted(picks)


@pytest.mark.parametrize("name,moves,p0", [("full_8b", 6000, 1e-6), ("full_8b", 6000, 0.3), ("long_70b", 6000, 1e-6),
                                            ("long_70b", 6000, 0.3)])
def test_anneal_full_shape_all_waves(kvp, oracle, name, moves, p0):
    """The two large configurations at their real shape and chain count (4096 and 8192 chains, which come in several
    waves of resident chains; later waves take over the scratch of earlier ones), with a reduced move budget so that
    the oracle can follow: the access bitmap is the oracle's own (and the trace kernel's full-size output is compared
    with it), about twenty chains spread over every wave plus the winner are recomputed by the oracle on the host
    cores, all eight per-chain outputs and the winner's schedule bit for bit. Near-greedy and hot start."""
    from oracle_pool import oracle_chains_sampled, oracle_trace_parallel
    cfg = wl.CONFIGS[name]
    U, S, cap, chains = wl.units(cfg), cfg["steps"], cfg["cap"], cfg["chains"]
    A, path = oracle_trace_parallel(name, 0)
    assert np.array_equal(to_np(trace_on_gpu(kvp, wl.trace_params(name, seed=0))), A)
    g = kvp.Problem(U, cfg["bytes_per_unit"], S, to_dev(A), cap, *cfg["bw"])
    kw = dict(chains=chains, moves=moves, seed=0, p0=p0, levels=8)
    out = g.anneal(g.make_params(**kw), want_per_chain=True)
    st = out["stats"]
    w = st.best_chain
    assert w == min(range(chains), key=lambda c: (out["per_chain"][c].best_ticks, c))
    mean, want, best = oracle_chains_sampled(name, path, kw, _spread(chains), want_best=[w])
    assert st.calib_mean_delta == mean
    for c, tup in want.items():
        assert out["per_chain"][c].astuple() == tup, c
    assert np.array_equal(to_np(out["best_schedule"]), best[w])
    assert out["best_ticks"] == want[w][0] <= st.init_ticks
    assert st.moves_total == sum(r.moves_done for r in out["per_chain"])
    ev = g.eval(out["best_schedule"])
    assert int(ev["total_ticks"][0]) == out["best_ticks"] and int(ev["bad_step"][0]) == -1
    if p0 > 0.1:
        assert min(r.n_changed for r in out["per_chain"]) > 100       # the hot start rewrites hundreds of units
    if name == "full_8b":
        # the same job on the narrow kernel, one and two warps per chain: slices of this size are copy-on-write overlays
        # of the initial schedule there too, the chains come in more waves, and the winner is walked back in its overlay
        for warps in (1, 2):
            kvp.set_test_hooks(warps_per_chain=warps)
            try:
                again = g.anneal(g.make_params(**kw), want_per_chain=True)
            finally:
                kvp.set_test_hooks()
            assert not again["stats"].wide_kernel and again["stats"].chain_launches >= (2, 4)[warps - 1]
            assert [r.astuple() for r in again["per_chain"]] == [r.astuple() for r in out["per_chain"]]
            assert again["stats"].best_chain == w and again["best_ticks"] == out["best_ticks"]
            assert np.array_equal(to_np(again["best_schedule"]), best[w])


def test_anneal_layer_8b_stated_budget(kvp, oracle):
    """layer_8b at its stated 1024 chains x 200,000 moves; the oracle recomputes a spread of the chains and the winner."""
    from oracle_pool import oracle_chains_sampled, oracle_trace_parallel
    name = "layer_8b"
    cfg = wl.CONFIGS[name]
    A, path = oracle_trace_parallel(name, 0)
    g = kvp.Problem(wl.units(cfg), cfg["bytes_per_unit"], cfg["steps"], to_dev(A), cfg["cap"], *cfg["bw"])
    kw = dict(chains=cfg["chains"], moves=cfg["moves"], seed=0, p0=cfg["p0"])
    out = g.anneal(g.make_params(**kw), want_per_chain=True)
    w = out["stats"].best_chain
    mean, want, best = oracle_chains_sampled(name, path, kw, _spread(cfg["chains"]), want_best=[w])
    assert out["stats"].calib_mean_delta == mean
    for c, tup in want.items():
        assert out["per_chain"][c].astuple() == tup, c
    assert np.array_equal(to_np(out["best_schedule"]), best[w]) and out["best_ticks"] == want[w][0]
    assert out["stats"].moves_total == cfg["chains"] * cfg["moves"]


def test_global_state_winner_paths(kvp, oracle, warps_per_chain):
    # chains in global scratch rebuild the winner by walking its logged moves back; check the three ways this can go:
    # a short log, a log that overflows (hot start: thousands of applied moves after the best; falls back to a replay),
    # and a winner from an earlier wave of a run with more chains than are resident at once
    g, o, cfg, A = named_problem(kvp, oracle, "layer_8b")
    for kw in (dict(chains=8, moves=30_000, seed=3, p0=1e-3), dict(chains=8, moves=40_000, seed=3, p0=0.8, levels=4),
               dict(chains=2500, moves=600, seed=5, p0=1e-3, levels=4)):
        gp, op = _params(g, o, **kw)
        out = g.anneal(gp, want_per_chain=True)
        w = out["stats"].best_chain
        assert w == min(range(kw["chains"]), key=lambda c: (out["per_chain"][c].best_ticks, c))
        ref, _, bst = o.anneal_chains(op, w, 1, want_best=True)
        assert ref[0].astuple() == out["per_chain"][w].astuple()
        assert np.array_equal(to_np(out["best_schedule"]), bst[0]) and out["best_ticks"] == ref[0].best_ticks


@pytest.mark.parametrize("overlay", [1, 2], ids=["overlay", "plain"])
def test_later_waves_start_afresh(kvp, oracle, hooks, warps_per_chain, overlay):
    """More chains than are resident at once: a chain of a later wave takes over a slice of global scratch that holds
    the final state of an earlier chain. With copy-on-write slices it starts from an empty overlay of the initial
    schedule, with plain slices from a fresh copy (the narrow kernel has both forms, test hook; the wide kernel always
    the first). Chains of every wave against the oracle, after a warm start with few rewritten units and after a hot
    one that rewrites most of them."""
    hooks(overlay=overlay)
    g, o, cfg, A = named_problem(kvp, oracle, "layer_8b")
    for kw, hot in ((dict(chains=5000, moves=2000, seed=7, p0=0.3, levels=4), False),
                    (dict(chains=2600, moves=160_000, seed=7, p0=0.8, levels=4), True)):
        gp, op = _params(g, o, **kw)
        out = g.anneal(gp, want_per_chain=True)
        n = kw["chains"]
        changed = [r.n_changed for r in out["per_chain"]]
        assert min(changed) > (16384 if hot else 0)     # hot: more applied moves than the problem has units
        assert out["stats"].chain_launches >= 2
        for c in (0, 1, n // 2, n // 2 + 1, n - 2, n - 1):
            want, _, _ = o.anneal_chains(op, c, 1)
            assert out["per_chain"][c].astuple() == want[0].astuple(), c
        w = out["stats"].best_chain
        ref, _, bst = o.anneal_chains(op, w, 1, want_best=True)
        assert np.array_equal(to_np(out["best_schedule"]), bst[0]) and out["best_ticks"] == ref[0].best_ticks


@pytest.mark.parametrize("overlay", [1, 2], ids=["overlay", "plain"])
@pytest.mark.parametrize("resident", [1, 3, 4])
def test_small_job_in_several_waves(kvp, oracle, hooks, resident, warps_per_chain, overlay):
    """Schedules in global memory, at most `resident` chains at a time (test hook): every chain but the first ones
    starts in a slice that an earlier chain left behind, as a copy-on-write overlay of the initial schedule or as a
    plain copy of it (test hook; the narrow kernel has both forms). All chains, the bound and the winner's schedule
    (walked back in its slice) against the oracle, at a hot and a cold start, with the stop rule, and with a winner
    that an early wave produced."""
    hooks(resident=resident, overlay=overlay)
    U, S, cap = 3000, 300, 700
    A = wl.random_access(U, S, 0.2, seed=21)
    g, o = both_problems(kvp, oracle, U, 8192, S, A, cap, (8000 * GB, 900 * GB, 900 * GB))
    for kw in (dict(chains=10, moves=3000, levels=6, p0=0.5, seed=1), dict(chains=7, moves=4000, levels=5, p0=1e-3, seed=2),
               dict(chains=9, moves=6400, levels=64, p0=0.3, seed=3, early_stop_permille=20)):
        gp, op = _params(g, o, **kw)
        _check_against_oracle(g, o, gp, op)


def test_turn_wait_is_bounded(kvp, oracle, hooks):
    """A hand-over that never comes: the waiting warp gives up after its poll limit (about a second), kvp_anneal
    returns KVP_ERR_TIMEOUT instead of holding the GPU, and the next call on the same problem is exact again."""
    g, o, cfg, A = named_problem(kvp, oracle, "tiny")
    hooks(warps_per_chain=2, drop_turn=1)
    with pytest.raises(kvp.KvpError) as e:
        g.anneal(g.make_params(chains=4, moves=1000, seed=0))
    assert e.value.code == kvp.ERR_TIMEOUT
    hooks(drop_turn=0)
    gp, op = _params(g, o, chains=4, moves=1000, seed=0)
    _check_against_oracle(g, o, gp, op)


@pytest.mark.parametrize("name,p0", [("single_head", 1e-6), ("single_head", 0.3), ("layer_8b", 1e-6)])
def test_two_warp_chains_repeat_exactly(kvp, oracle, hooks, name, p0):
    """Two warps per chain evaluate ahead of each other's commits, so their timing varies from run to run; the
    results may not. All chains of the configuration, twenty runs, against one run with one warp per chain (which the
    other tests compare with the oracle), at a cold and at a hot start (many applied moves, many re-evaluations)."""
    g, o, cfg, A = named_problem(kvp, oracle, name)
    moves = min(cfg["moves"], 50_000)
    gp = g.make_params(chains=cfg["chains"], moves=moves, seed=3, p0=p0)
    hooks(warps_per_chain=1)
    ref = g.anneal(gp, want_per_chain=True)
    want = [r.astuple() for r in ref["per_chain"]]
    hooks(warps_per_chain=2)
    for _ in range(20):
        out = g.anneal(gp, want_per_chain=True)
        assert [r.astuple() for r in out["per_chain"]] == want
        assert out["best_ticks"] == ref["best_ticks"]
        assert torch.equal(out["best_schedule"], ref["best_schedule"])


@pytest.mark.parametrize("split", [0, 20, 64])
def test_work_queue_in_two_halves(kvp, oracle, hooks, split, warps_per_chain):
    """Chains in shared memory with the access bitmap staged beside them keep half a work queue and work a batch
    with more items than it holds off in two halves. Ordinary inputs never fill it, so the hook lowers the limit:
    dense accesses, a churning initial schedule and a hot start give batches of a few hundred items."""
    hooks(split_queue=split)
    U, S, cap = 64, 200, 32
    A = wl.random_access(U, S, 0.5, seed=9)
    g, o = both_problems(kvp, oracle, U, 8192, S, A, cap, (8000 * GB, 900 * GB, 900 * GB))
    init = wl.random_schedules(U, S, cap, 1, seed=4, churn=0.5)[0]
    kw = dict(chains=6, moves=2500, levels=5, p0=0.5, p_swap_256=200)
    gp = g.make_params(init_mode=kvp.INIT_USER, init_schedule=to_dev(init), **kw)
    op = o.make_params(init_mode=oracle.INIT_USER, init_schedule=init, **kw)
    _check_against_oracle(g, o, gp, op)
    gp, op = _params(g, o, chains=6, moves=2500, levels=5, p0=1e-3)
    _check_against_oracle(g, o, gp, op)
