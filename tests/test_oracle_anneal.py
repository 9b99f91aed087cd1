"""Pins of the oracle's annealer: exact optima by exhaustive search on tiny instances,
invariants of the incremental bookkeeping, and the meaning of the acceptance table."""
import itertools
import math

import numpy as np
import pytest

from paper_2508_13231_b200 import workloads as wl

GB = 10 ** 9


def _exact_dynamic_optimum(prob, U, S, cap):
    """Shortest path over placement subsets: the cost of step s depends only on (P[s-1], P[s]).
    Step costs are obtained from the oracle's eval on two-row probes, the search itself is independent."""
    rows = [r for r in itertools.product([0, 1], repeat=U) if sum(r) <= cap]
    packed = [wl.pack_bits(np.array(r, np.uint8)) for r in rows]
    n = len(rows)

    def step_cost(s, i_prev, i_cur):
        P = np.zeros((S, (U + 31) // 32), np.uint32)
        if s > 0:
            P[s - 1] = packed[i_prev]
        P[s] = packed[i_cur]
        return int(prob.eval(P)["step_ticks"][s])

    dist = [step_cost(0, i, i) for i in range(n)]            # P[-1] := P[0]
    for s in range(1, S):
        dist = [min(dist[i] + step_cost(s, i, j) for i in range(n)) for j in range(n)]
    return min(dist)


def test_sa_reaches_exact_dynamic_optimum_small(oracle):
    U, S, cap = 5, 4, 2
    A = wl.random_access(U, S, 0.5, seed=21)
    prob = oracle.Problem(U, 8192, S, A, cap, 3 * GB, 1 * GB, 1 * GB)
    opt = _exact_dynamic_optimum(prob, U, S, cap)
    ap = prob.make_params(chains=16, moves=4000, seed=3, levels=32, max_len_log2=2)
    out = prob.anneal(ap)
    assert out["best_ticks"] >= opt                          # nothing beats the exhaustive optimum
    assert out["best_ticks"] == opt                          # and 16 short chains find it
    assert prob.eval(out["best_schedule"])["total_ticks"] == out["best_ticks"]
    assert prob.eval(out["best_schedule"])["bad_step"] == -1


def test_full_enumeration_u4_s3(oracle):
    # every schedule of 4 units x 3 steps with at most 2 resident units: 11^3 schedules
    U, S, cap = 4, 3, 2
    A = wl.pack_bits(np.array([[1, 1, 0, 0], [0, 1, 1, 0], [0, 0, 1, 1]], np.uint8))
    prob = oracle.Problem(U, 8192, S, A, cap, 4 * GB, 1 * GB, 2 * GB)
    rows = [r for r in itertools.product([0, 1], repeat=U) if sum(r) <= cap]
    assert len(rows) == 11
    best = min(prob.eval(wl.pack_bits(np.array(c, np.uint8)))["total_ticks"]
               for c in itertools.product(rows, repeat=S))
    assert best == _exact_dynamic_optimum(prob, U, S, cap)
    out = prob.anneal(prob.make_params(chains=8, moves=3000, seed=1, levels=16, max_len_log2=1))
    assert out["best_ticks"] == best


def test_best_static_placement_brute_force_tiny(oracle):
    # all C(16, <=6) = 14,893 static placements of the tiny configuration; the annealer starts from a
    # static placement and may migrate, so its bound can only be at or below the best static one
    cfg = wl.CONFIGS["tiny"]
    tp = wl.trace_params("tiny", seed=0)
    A = oracle.trace_generate(**tp)
    U, S, cap = 16, 32, cfg["cap"]
    prob = oracle.Problem(U, cfg["bytes_per_unit"], S, A, cap, *cfg["bw"])
    bits = wl.unpack_bits(A, U).astype(np.int64)
    a = bits.sum(axis=1)
    kh, ke = prob.weights["kh"], prob.weights["ke"]
    # a static schedule has no migrations, so its step cost needs only hr: an independent restatement
    best, best_row, count = None, None, 0
    for k in range(cap + 1):
        for comb in itertools.combinations(range(U), k):
            count += 1
            hr = bits[:, list(comb)].sum(axis=1) if k else np.zeros(S, np.int64)
            T = int(np.maximum(kh * hr, ke * (a - hr)).sum())
            if best is None or T < best:
                best, best_row = T, comb
    assert count == 14893
    row = np.zeros(U, np.uint8); row[list(best_row)] = 1
    assert prob.eval(wl.pack_bits(np.tile(row, (S, 1))))["total_ticks"] == best
    ap = prob.make_params(chains=cfg["chains"], moves=cfg["moves"], seed=0)
    out = prob.anneal(ap)
    assert out["best_ticks"] <= best
    init = prob.eval(prob.init_placement(oracle.INIT_STATIC_FREQ))["total_ticks"]
    assert best <= init
    lower = sum(-(-kh * ke * int(x) // (kh + ke)) for x in a)     # aggregate-bandwidth bound, rounded up
    assert out["best_ticks"] >= lower


def test_incremental_bookkeeping_matches_full_evaluation(oracle):
    U, S, cap = 45, 40, 12
    A = wl.random_access(U, S, 0.3, seed=22)
    for bw, flags in [((8000, 900, 900), 3), ((4900, 900, 500), 3), ((4900, 500, 900), 2), ((3, 1, 1), 0)]:
        prob = oracle.Problem(U, 8192, S, A, cap, bw[0] * GB, bw[1] * GB, bw[2] * GB, mig_flags=flags,
                              hw=np.arange(S) % 3, ew=np.arange(S) % 2)
        ap = prob.make_params(chains=6, moves=3000, seed=5, levels=16)
        for upto in (1, 17, 500, 3000):
            res, fin, bst = prob.anneal_chains(ap, 0, 6, upto_moves=upto, want_final=True, want_best=True)
            for r, f, b in zip(res, fin, bst):
                assert r.moves_done == upto
                assert prob.check_total(f, r.final_ticks)       # running total == Eq. 1 recomputed
                assert prob.check_total(b, r.best_ticks)
                assert r.best_ticks <= r.final_ticks
                occ = wl.unpack_bits(f, U).sum(axis=1)
                assert occ.max() <= cap                          # Eq. 5 after every prefix of moves
                assert r.n_changed <= r.n_accepted <= upto - r.n_infeasible


def test_chains_are_reproducible_and_independent(oracle):
    U, S, cap = 33, 20, 9
    A = wl.random_access(U, S, 0.3, seed=23)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    ap = prob.make_params(chains=8, moves=2000, seed=9, levels=8)
    all_, _, _ = prob.anneal_chains(ap, 0, 8)
    some, _, _ = prob.anneal_chains(ap, 3, 2)
    assert [r.astuple() for r in some] == [r.astuple() for r in all_[3:5]]
    assert len({r.traj_hash for r in all_}) == 8                # different chains take different paths
    # replaying a chain up to its best move reproduces its best state
    r3 = all_[3]
    if r3.best_move != 2 ** 64 - 1:
        rep, fin, _ = prob.anneal_chains(ap, 3, 1, upto_moves=r3.best_move + 1, want_final=True)
        assert rep[0].final_ticks == r3.best_ticks and prob.check_total(fin[0], r3.best_ticks)


def test_zero_temperature_never_goes_uphill(oracle):
    U, S, cap = 40, 16, 10
    A = wl.random_access(U, S, 0.3, seed=24)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    levels = 4
    cold = np.full(levels, 1.0)                                   # 1 tick: exp(-delta/1) ~ 0 for real deltas
    ap = prob.make_params(chains=4, moves=5000, seed=2, levels=levels, temps=cold)
    res, _, _ = prob.anneal_chains(ap, 0, 4)
    for r in res:
        assert r.final_ticks == r.best_ticks                     # greedy descent: the last state is the best
    hot = np.full(levels, 1e12)                # (nearly) everything feasible is accepted: the first bin of
                                               # the table holds exp(-(half a bin)/C) >= exp(-23/2048)
    ap = prob.make_params(chains=2, moves=2000, seed=2, levels=levels, temps=hot)
    res, _, _ = prob.anneal_chains(ap, 0, 2)
    for r in res:
        assert r.n_accepted >= 0.97 * (r.moves_done - r.n_infeasible)


def test_early_stop_rule(oracle):
    U, S, cap = 40, 16, 10
    A = wl.random_access(U, S, 0.3, seed=25)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    ap = prob.make_params(chains=8, moves=64000, seed=4, levels=64, early_stop_permille=1)
    res, _, _ = prob.anneal_chains(ap, 0, 8)
    full, _, _ = prob.anneal_chains(prob.make_params(chains=8, moves=64000, seed=4, levels=64), 0, 8)
    for r, f in zip(res, full):
        assert r.moves_done % 1000 == 0 and 1000 <= r.moves_done <= 64000   # stops only on level boundaries
        assert r.best_ticks >= f.best_ticks or r.moves_done == 64000
    assert any(r.moves_done < 64000 for r in res)
    late = prob.make_params(chains=8, moves=64000, seed=4, levels=64, early_stop_permille=1, early_stop_from_level=40)
    res2, _, _ = prob.anneal_chains(late, 0, 8)
    assert all(r.moves_done >= 40000 for r in res2)


def test_accept_table_is_metropolis(oracle):
    temps = np.array([5000.0, 123.4, 1.0, 0.01, 3.0e7])
    table, shifts = oracle.accept_table(temps)
    for j, C in enumerate(temps):
        C = max(C, 1.0)
        sh = int(shifts[j])
        assert 1024 * 2 ** sh >= 23 * C and (sh == 0 or 1024 * 2 ** (sh - 1) < 23 * C)
        t = table[j].astype(np.float64) / 2 ** 32
        assert np.all(np.diff(table[j].astype(np.int64)) <= 0)          # colder with growing delta
        # every delta of a bin is accepted with exp(-delta/C) up to the half-bin quantisation
        rel = math.exp(2 ** sh / (2 * C)) - 1
        for q in (0, 1, 7, 100, 1023):
            for delta in (q * 2 ** sh, q * 2 ** sh + 2 ** sh - 1):
                if delta == 0:
                    continue
                exact = math.exp(-delta / C)
                assert abs(t[q] - exact) <= exact * rel + 2.0 ** -32
        assert table[j][1023] <= 2 ** 32 * math.exp(-22.4) + 1           # beyond the table: never accepted


def test_default_temperature_ladder(oracle):
    U, S, cap = 64, 32, 16
    A = wl.random_access(U, S, 0.25, seed=26)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    ap = prob.make_params(chains=1, moves=1000, seed=7, levels=10, p0=0.8, alpha=0.9)
    temps, mean = prob.temps(ap)
    assert mean > 0
    assert math.exp(-mean / temps[0]) == pytest.approx(0.8, rel=1e-12)    # p0 at the mean uphill step
    assert np.allclose(temps[1:] / temps[:-1], 0.9, rtol=1e-12)           # geometric cooling
    # first level: measured acceptance of uphill proposals is near p0 (loose: few hundred samples)
    table, shifts = oracle.accept_table(temps)
    q = mean >> int(shifts[0])
    assert abs(table[0][q] / 2 ** 32 - 0.8) < 0.03
