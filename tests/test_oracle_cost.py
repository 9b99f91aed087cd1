"""Pins of the oracle's cost model (Eq. 1-5) against what the paper and arithmetic fix.

None of these tests re-types the oracle's formula: expected values are hand-worked
numbers from tests/golden/, closed forms, bounds, monotonicity and brute force.
"""
import itertools
import os

import numpy as np
import pytest

from paper_2508_13231_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")
GB = 10 ** 9


def _rows(name):
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield line.split()


def test_philox_known_answers(oracle):
    n = 0
    for r in _rows("philox4x32_10_kat.txt"):
        v = [int(x, 16) for x in r]
        assert oracle.philox(v[0:4], v[4:6]) == tuple(v[6:10])
        n += 1
    assert n == 3


def test_tick_weights_examples(oracle):
    # Table I: 4.9 TB/s, 900 GB/s, 500 GB/s -> 49:9:5 -> lcm 2205
    w = oracle.tick_weights(4900 * GB, 900 * GB, 500 * GB)
    assert (w["kh"], w["kk"], w["kd"], w["ke"], w["lcm"]) == (45, 245, 441, 441, 2205)
    w = oracle.tick_weights(8000 * GB, 900 * GB, 900 * GB)
    assert (w["kh"], w["kk"], w["kd"], w["ke"]) == (9, 80, 80, 80)
    w = oracle.tick_weights(8, 1, 1)
    assert (w["kh"], w["ke"]) == (1, 8)
    # weights are exactly inversely proportional to the bandwidths
    for bw in [(7, 3, 2), (4900, 900, 500), (123456, 7890, 4321)]:
        w = oracle.tick_weights(*bw)
        assert w["kh"] * bw[0] == w["kk"] * bw[1] == w["kd"] * bw[2] == w["lcm"] * w["gcd"]


def _instance_with_counts(oracle, bw, hr, er, mi, mo, hw, ew, extra=3):
    """Two-step instance whose step 1 has exactly the given cardinalities."""
    U = hr + er + mi + mo + extra
    ids = iter(range(U))
    A = np.zeros((2, U), np.uint8)
    P = np.zeros((2, U), np.uint8)
    for _ in range(hr):
        u = next(ids); A[1, u] = 1; P[0, u] = 1; P[1, u] = 1
    for _ in range(er):
        u = next(ids); A[1, u] = 1
    for _ in range(mi):
        u = next(ids); P[1, u] = 1
    for _ in range(mo):
        u = next(ids); P[0, u] = 1
    prob = oracle.Problem(U, 4096, 2, wl.pack_bits(A), U, bw[0] * GB, bw[1] * GB, bw[2] * GB,
                          hw=[0, hw], ew=[0, ew])
    return prob, wl.pack_bits(P)


def test_eq34_hand_worked(oracle):
    n = 0
    for r in _rows("eq34_worked.txt"):
        v = [int(x) for x in r]
        bw, (hr, er, mi, mo, hw, ew), (th, te, f) = v[0:3], v[3:9], v[9:12]
        prob, P = _instance_with_counts(oracle, bw, hr, er, mi, mo, hw, ew)
        out = prob.eval(P)
        assert list(out["counts"][1]) == [hr, mi, mo, hr + mi], r
        assert int(out["step_ticks"][1]) == f == max(th, te), r
        # step 0 reads nothing and, because P[-1] := P[0], migrates nothing
        assert int(out["step_ticks"][0]) == 0
        assert out["total_ticks"] == f
        n += 1
    assert n == 6


def test_seconds_scale(oracle):
    # one unit of 8 KB read from HBM at 8 TB/s takes 8192 / 8e12 s
    U = 8
    A = np.zeros((1, U), np.uint8); A[0, 0] = 1
    prob = oracle.Problem(U, 8192, 1, wl.pack_bits(A), U, 8000 * GB, 900 * GB, 900 * GB)
    out = prob.eval(wl.pack_bits(np.ones((1, U), np.uint8)))
    assert out["total_seconds"] == pytest.approx(8192 / 8e12, rel=1e-12)
    # the same unit read from off-package DRAM at 0.9 TB/s
    out = prob.eval(wl.pack_bits(np.zeros((1, U), np.uint8)))
    assert out["total_seconds"] == pytest.approx(8192 / 0.9e12, rel=1e-12)


def test_unlimited_hbm_closed_form(oracle):
    # everything resident, nothing migrates: T = sum_s |A[s]| * bytes / B_h  (Unlimited HBM, Section IV-A)
    U, S = 70, 9
    A = wl.random_access(U, S, 0.3, seed=1)
    prob = oracle.Problem(U, 8192, S, A, U, 4900 * GB, 900 * GB, 500 * GB)
    P = wl.pack_bits(np.ones((S, U), np.uint8))
    out = prob.eval(P)
    a = wl.unpack_bits(A, U).sum(axis=1)
    assert out["total_ticks"] == 45 * int(a.sum())
    assert out["total_seconds"] == pytest.approx(int(a.sum()) * 8192 / 4.9e12, rel=1e-12)
    assert out["bad_step"] == -1
    assert np.all(out["counts"][:, 1:3] == 0)


def test_static_schedule_has_no_migration_and_capacity_flag(oracle):
    U, S, cap = 40, 6, 10
    A = wl.random_access(U, S, 0.4, seed=2)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    row = np.zeros(U, np.uint8); row[:cap] = 1
    out = prob.eval(wl.pack_bits(np.tile(row, (S, 1))))
    assert np.all(out["counts"][:, 1:3] == 0) and out["bad_step"] == -1
    # exceed capacity from step 3 on: Eq. 5 violated, first offending step reported
    P = np.tile(row, (S, 1)); P[3:, cap] = 1
    assert prob.eval(wl.pack_bits(P))["bad_step"] == 3


def test_aggregate_bandwidth_lower_bound(oracle):
    # no step can be faster than its accessed bytes over B_h + min(B_k, B_d):
    # f_s * (kh + ke) >= kh * ke * a_s, for any schedule
    U, S, cap = 90, 12, 30
    A = wl.random_access(U, S, 0.35, seed=3)
    a = wl.unpack_bits(A, U).sum(axis=1).astype(np.int64)
    for bw in [(8000, 900, 900), (4900, 900, 500), (4900, 500, 900)]:
        prob = oracle.Problem(U, 8192, S, A, cap, bw[0] * GB, bw[1] * GB, bw[2] * GB)
        kh, ke = prob.weights["kh"], prob.weights["ke"]
        for P in wl.random_schedules(U, S, cap, 6, seed=4, churn=0.2):
            f = prob.eval(P)["step_ticks"].astype(np.int64)
            assert np.all(f * (kh + ke) >= kh * ke * a)


def test_free_migration_optimum_by_enumeration(oracle):
    # with migration free each step is independent; its best split puts h of the a_s accessed
    # units in HBM with h <= min(cap, a_s) minimising max(kh*h, ke*(a_s-h)); enumerate all placements
    U, S, cap = 7, 3, 3
    A = wl.random_access(U, S, 0.6, seed=5)
    prob = oracle.Problem(U, 8192, S, A, cap, 3 * GB, 1 * GB, 1 * GB, mig_flags=0)
    kh, ke = prob.weights["kh"], prob.weights["ke"]
    a = wl.unpack_bits(A, U).sum(axis=1)
    rows = [r for r in itertools.product([0, 1], repeat=U) if sum(r) <= cap]
    for s in range(S):
        best = None
        for r in rows:
            P = np.zeros((S, U), np.uint8); P[s] = r
            f = int(prob.eval(wl.pack_bits(P))["step_ticks"][s])
            best = f if best is None else min(best, f)
        closed = min(max(kh * h, ke * (int(a[s]) - h)) for h in range(min(cap, int(a[s])) + 1))
        assert best == closed


def test_cost_monotone_in_access_and_bandwidth(oracle):
    U, S, cap = 50, 8, 15
    A = wl.random_access(U, S, 0.3, seed=6)
    scheds = wl.random_schedules(U, S, cap, 4, seed=7, churn=0.3)
    prob = oracle.Problem(U, 8192, S, A, cap, 4900 * GB, 900 * GB, 500 * GB)
    bits = wl.unpack_bits(A, U)
    rng = np.random.default_rng(8)
    for P in scheds:
        base = prob.eval(P)
        for _ in range(10):
            s, u = int(rng.integers(S)), int(rng.integers(U))
            if bits[s, u]:
                continue
            b2 = bits.copy(); b2[s, u] = 1
            p2 = oracle.Problem(U, 8192, S, wl.pack_bits(b2), cap, 4900 * GB, 900 * GB, 500 * GB)
            o2 = p2.eval(P)
            assert o2["total_ticks"] >= base["total_ticks"]           # one more access never helps
            assert np.all(o2["step_ticks"] >= base["step_ticks"])
        for bw in [(9800, 900, 500), (4900, 1800, 500), (4900, 900, 1000)]:
            p3 = oracle.Problem(U, 8192, S, A, cap, bw[0] * GB, bw[1] * GB, bw[2] * GB)
            assert p3.eval(P)["total_seconds"] <= base["total_seconds"] * (1 + 1e-12)  # faster memory never hurts


def test_migration_direction_matters(oracle):
    # with a slow link and fast DRAM (B_k < B_d) the outbound and inbound link terms differ:
    # moving 3 units out and 1 in costs kappa_k*3 on the link, the mirror image costs the same,
    # but moving 3 out with ew = 2 writes sharing the outbound link costs kappa_k*5.
    prob, P = _instance_with_counts(oracle, (4900, 500, 900), 0, 0, 1, 3, 0, 2)
    assert int(prob.eval(P)["step_ticks"][1]) == max(45 * 4, max(441 * 5, 441 * 1, 245 * 6))
    prob, P = _instance_with_counts(oracle, (4900, 500, 900), 0, 0, 3, 1, 0, 2)
    assert int(prob.eval(P)["step_ticks"][1]) == max(45 * 4, max(441 * 3, 441 * 3, 245 * 6))


def test_pad_bits_ignored(oracle):
    U, S = 37, 4                     # 27 pad bits in the second word
    A = wl.random_access(U, S, 0.5, seed=9)
    prob = oracle.Problem(U, 8192, S, A, 12, 8000 * GB, 900 * GB, 900 * GB)
    P = wl.random_schedules(U, S, 12, 1, seed=10)[0]
    dirty_A = A.copy(); dirty_A[:, -1] |= np.uint32(0xFFFFFFE0)
    dirty_P = P.copy(); dirty_P[:, -1] |= np.uint32(0xFFFFFFE0)
    prob2 = oracle.Problem(U, 8192, S, dirty_A, 12, 8000 * GB, 900 * GB, 900 * GB)
    assert prob2.eval(dirty_P)["total_ticks"] == prob.eval(P)["total_ticks"]


def test_init_placements(oracle):
    U, S, cap = 60, 10, 17
    A = wl.random_access(U, S, 0.25, seed=11)
    prob = oracle.Problem(U, 8192, S, A, cap, 8000 * GB, 900 * GB, 900 * GB)
    first = wl.unpack_bits(prob.init_placement(oracle.INIT_STATIC_FIRST), U)
    assert np.all(first[:, :cap] == 1) and np.all(first[:, cap:] == 0)
    freq = wl.unpack_bits(prob.init_placement(oracle.INIT_STATIC_FREQ), U)
    cnt = wl.unpack_bits(A, U).sum(axis=0).astype(np.int64)
    order = np.lexsort((np.arange(U), -cnt))[:cap]      # count descending, index ascending
    want = np.zeros(U, np.uint8); want[order] = 1
    assert np.all(freq == want[None, :])
