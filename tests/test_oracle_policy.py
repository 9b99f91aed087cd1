"""Pins of the oracle's placement policies and of the paper-literal (W, R) annealer."""
import os

import numpy as np
import pytest

from paper_2508_13231_b200 import workloads as wl

GB = 10 ** 9
GOLD = os.path.join(os.path.dirname(__file__), "golden", "policies_worked.txt")


def _rows(text):
    return [[int(x) for x in r.split(",")] if r else [] for r in text.split("|")]


def _bits(rows, U):
    b = np.zeros((len(rows), U), np.uint8)
    for s, r in enumerate(rows):
        b[s, r] = 1
    return b


def test_hand_worked_policies(oracle):
    A_look = wl.pack_bits(_bits([[1], [1, 2], [2]], 4))
    look = oracle.Problem(4, 8192, 3, A_look, 1, 8000 * GB, 900 * GB, 900 * GB)
    A_re = wl.pack_bits(_bits([[2], [0], [3], []], 4))
    react = oracle.Problem(4, 8192, 4, A_re, 2, 8000 * GB, 900 * GB, 900 * GB)
    n = 0
    for line in open(GOLD):
        f = line.split()
        if not f or f[0].startswith("#"):
            continue
        if f[0] == "lookahead":
            W, R = int(f[1][2:]), int(f[2][2:])
            got = wl.unpack_bits(oracle.policy_lookahead(look, W, R), 4)
            assert np.array_equal(got, _bits(_rows(f[4]), 4)), line
        elif f[0] == "reactive":
            got = wl.unpack_bits(oracle.policy_reactive(react), 4)
            assert np.array_equal(got, _bits(_rows(f[2]), 4)), line
        else:
            A_pg = wl.pack_bits(_bits([[2, 3, 5], [4, 5, 6]], 8))
            pg = oracle.Problem(8, 8192, 2, A_pg, 2, 8000 * GB, 900 * GB, 900 * GB)
            got = wl.unpack_bits(oracle.policy_page(pg, 2), 8)
            assert np.array_equal(got, _bits(_rows(f[2]), 8)), line
        n += 1
    assert n == 6


def test_lookahead_invariants(oracle):
    U, S, cap = 70, 40, 15
    A = wl.random_access(U, S, 0.2, seed=41)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    static = prob.init_placement(oracle.INIT_STATIC_FIRST)
    a = wl.unpack_bits(A, U)
    for W in (1, 3, 17, 64):
        assert np.array_equal(oracle.policy_lookahead(prob, W, 0), static)          # R = 0: Static Placement
        for R in (100, 500, 1000):
            P = oracle.policy_lookahead(prob, W, R)
            ev = prob.eval(P)
            assert ev["bad_step"] == -1                                             # Eq. 5 at every step
            bits = wl.unpack_bits(P, U)
            # a unit only enters HBM if it is accessed within the window
            entered = np.argwhere((bits[1:] == 1) & (bits[:-1] == 0))
            for s, u in entered:
                assert a[s + 1:s + 1 + W, u].any()
    # with room for every step's accessed set, W = 1 and R = 1 put all of it in HBM: nothing is read off-package
    roomy = oracle.Problem(U, 8192, S, A, int(a.sum(axis=1).max()), 8000 * GB, 900 * GB, 900 * GB)
    ev = roomy.eval(oracle.policy_lookahead(roomy, 1, 1000))
    assert np.array_equal(ev["counts"][:, 0], a.sum(axis=1))


def test_reactive_invariants(oracle):
    U, S, cap = 60, 50, 12
    A = wl.random_access(U, S, 0.15, seed=42)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    P = oracle.policy_reactive(prob)
    bits, a = wl.unpack_bits(P, U), wl.unpack_bits(A, U)
    assert prob.eval(P)["bad_step"] == -1
    for s in range(S - 1):
        missed = np.flatnonzero((a[s] == 1) & (bits[s] == 0))[:cap]
        assert np.all(bits[s + 1, missed] == 1)                  # promoted after the miss
        hit = (a[s] == 1) & (bits[s] == 1)
        if missed.size <= cap - hit.sum():
            assert np.all(bits[s + 1, hit] == 1)                 # what was just used is not the LRU victim
        if missed.size == 0:
            assert np.array_equal(bits[s + 1], bits[s])          # no miss, no migration


def test_page_invariants(oracle):
    U, S, cap, page = 128, 30, 40, 8
    A = wl.random_access(U, S, 0.1, seed=43)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    bits = wl.unpack_bits(oracle.policy_page(prob, page), U).reshape(S, U // page, page)
    assert np.all((bits.sum(axis=2) == 0) | (bits.sum(axis=2) == page))          # whole pages only
    assert np.all((bits.sum(axis=2) > 0).sum(axis=1) <= cap // page)              # capacity in pages
    a = wl.unpack_bits(A, U).reshape(S, U // page, page).sum(axis=2)
    res = bits[:, :, 0].astype(bool)
    for s in range(S):                                                            # no resident page scores less than
        if (~res[s]).any() and res[s].any() and (a[s][~res[s]] > 0).any():        # a page left outside
            assert a[s][res[s]].min() >= a[s][~res[s]].max()


def test_policies_reproduce_the_papers_ordering_on_a_synthetic_trace(oracle):
    # Section IV-B, qualitatively: first-come Static << Reactive < best look-ahead < Unlimited HBM (in speed)
    cfg = wl.CONFIGS["single_head"]
    A = oracle.trace_generate(**wl.trace_params("single_head", 0))
    U, S = 256, 512
    prob = oracle.Problem(U, cfg["bytes_per_unit"], S, A, cfg["cap"], *cfg["bw"])
    static = prob.eval(prob.init_placement(oracle.INIT_STATIC_FIRST))["total_ticks"]
    reactive = prob.eval(oracle.policy_reactive(prob))["total_ticks"]
    look = min(prob.eval(oracle.policy_lookahead(prob, W, R))["total_ticks"] for W in (8, 16) for R in (100, 300))
    unlimited = 9 * int(wl.unpack_bits(A, U).sum())
    assert unlimited < look < reactive < static
    assert 4.0 < static / look < 8.0                             # the paper reports up to 5.87x over Static


def test_wr_annealer(oracle):
    # a bowl with its minimum at (W, r) = (6, 3)
    w_max, n_ratio = 12, 11
    T = np.array([[1000 + 40 * (w - 6) ** 2 + 25 * (r - 3) ** 2 for r in range(n_ratio)] for w in range(1, w_max + 1)],
                 np.uint64)
    wp = oracle.wr_params(chains=8, iters=4000, seed=3, levels=16)
    temps, mean = oracle.wr_temps(T, wp)
    assert mean > 0 and np.exp(-mean / temps[0]) == pytest.approx(0.8, rel=1e-12)
    res = oracle.wr_anneal(T, wp)
    for r in res:
        assert (r.best_ticks, r.best_w, r.best_r) == (1000, 6, 3)
        assert r.final_ticks == int(T[r.final_w - 1, r.final_r]) and r.iters_done == 4000
    assert len({r.n_accepted for r in res}) > 1                  # chains differ
    # a flat table accepts every proposal that stays on the grid; a 1 x 2 grid only has ratio moves that stay
    flat = np.full((1, 2), 7, np.uint64)
    r = oracle.wr_anneal(flat, oracle.wr_params(chains=1, iters=20000, seed=1, levels=4))[0]
    assert 0.18 * 20000 < r.n_accepted < 0.22 * 20000            # P(ratio move) * P(direction stays) = 0.4 * 0.5
    # the stop rule ends a chain that no longer improves
    r = oracle.wr_anneal(T, oracle.wr_params(chains=4, iters=64000, seed=2, levels=64, early_stop_permille=1))
    assert all(x.iters_done % 1000 == 0 and x.iters_done < 64000 for x in r)
