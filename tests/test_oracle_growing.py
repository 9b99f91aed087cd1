"""Pins of the oracle's growing-cache form (newly written entries H^w / E^w as decisions, (n, l) steps).

Expected values come from a hand-worked fixture, closed forms, and exact reductions to the fixed-population model,
which tests/test_oracle_cost.py pins on its own; the annealer is checked against exhaustive search.
"""
import itertools
import os

import numpy as np
import pytest

from paper_2508_13231_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")
GB = 10 ** 9
TABLE1 = (4900 * GB, 900 * GB, 500 * GB)


def _pack(bits):
    return wl.pack_bits(np.asarray(bits, np.uint8))


def _random_growing(rng, U, S, cap_frac=0.4, p_old=0.4, density=0.3):
    """Random births, an access pattern that respects them, a capacity."""
    birth = np.where(rng.random(U) < p_old, 0, rng.integers(1, S, U)).astype(np.uint32)
    alive = birth[None, :] <= np.arange(S)[:, None]
    A = ((rng.random((S, U)) < density) & alive).astype(np.uint8)
    return birth, alive, A, max(1, int(cap_frac * U))


def test_worked_example(oracle):
    birth = [0, 1, 2]
    A = _pack([[1, 0, 0], [1, 1, 0], [0, 1, 1]])
    prob = oracle.Problem(3, 1, 3, A, 2, *TABLE1, birth=birth)
    n = 0
    with open(os.path.join(GOLD, "growing_worked.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            r = line.split()
            P = _pack([[int(c) for c in row] for row in r[0:3]])
            e = prob.eval(P)
            assert [int(x) for x in e["step_ticks"]] == [int(x) for x in r[3:6]], line
            assert e["total_ticks"] == int(r[6])
            n += 1
    assert n == 3


def test_no_births_is_the_fixed_model(oracle):
    rng = np.random.default_rng(11)
    for _ in range(5):
        U, S = int(rng.integers(5, 70)), int(rng.integers(2, 40))
        A = _pack(rng.random((S, U)) < 0.3)
        P = _pack(rng.random((S, U)) < 0.3)
        hw, ew = rng.integers(0, 4, S), rng.integers(0, 4, S)
        a = oracle.Problem(U, 64, S, A, U, *TABLE1, hw=hw, ew=ew)
        b = oracle.Problem(U, 64, S, A, U, *TABLE1, hw=hw, ew=ew, birth=np.zeros(U, np.uint32))
        ea, eb = a.eval(P), b.eval(P)
        assert np.array_equal(ea["step_ticks"], eb["step_ticks"]) and np.array_equal(ea["counts"], eb["counts"])
        assert not eb["hb"].any()


def test_reduces_to_fixed_model_with_adjusted_writes(oracle):
    """T_growing(P) = T_fixed(P', hw + hb, ew + nb - hb): P' repeats a unit's bit of its birth step at all earlier
    steps, which removes the edge at birth from the fixed model's migration counts, and the written entries are
    handed to the fixed model as its per-step constants."""
    rng = np.random.default_rng(5)
    for case in range(8):
        U, S = int(rng.integers(4, 80)), int(rng.integers(3, 50))
        birth, alive, A, cap = _random_growing(rng, U, S)
        Pb = (rng.random((S, U)) < 0.35) & alive
        hw, ew = rng.integers(0, 3, S).astype(np.uint32), rng.integers(0, 3, S).astype(np.uint32)
        g = oracle.Problem(U, 4096, S, _pack(A), U, *TABLE1, hw=hw, ew=ew, birth=birth)
        eg = g.eval(_pack(Pb))
        nb = np.bincount(birth[birth > 0], minlength=S).astype(np.uint32)
        hb = np.array([int(Pb[s, birth == s].sum()) if s else 0 for s in range(S)], np.uint32)
        assert np.array_equal(eg["hb"], hb)
        Pext = Pb.copy()
        for u in range(U):
            Pext[:birth[u], u] = Pb[birth[u], u]
        f = oracle.Problem(U, 4096, S, _pack(A), U, *TABLE1, hw=hw + hb, ew=ew + nb - hb)
        ef = f.eval(_pack(Pext))
        assert np.array_equal(eg["step_ticks"], ef["step_ticks"]), case
        # bits of units that do not exist yet are ignored
        noisy = Pb | (~alive & (rng.random((S, U)) < 0.5))
        en = g.eval(_pack(noisy))
        assert np.array_equal(en["step_ticks"], eg["step_ticks"]) and np.array_equal(en["counts"], eg["counts"])


def test_closed_forms(oracle):
    rng = np.random.default_rng(2)
    U, S = 40, 25
    birth, alive, A, _ = _random_growing(rng, U, S)
    g = oracle.Problem(U, 1, S, _pack(A), U, *TABLE1, birth=birth)
    w = g.weights
    a = A.sum(1)
    nb = np.bincount(birth[birth > 0], minlength=S)
    # everything in HBM from the moment it exists: reads and writes at HBM speed, nothing else moves
    e = g.eval(_pack(alive))
    assert [int(x) for x in e["step_ticks"]] == [int(w["kh"] * (a[s] + nb[s])) for s in range(S)]
    # nothing ever in HBM: reads over min(B_k, B_d), writes over the slower of link and DRAM channels
    e = g.eval(_pack(np.zeros((S, U))))
    assert [int(x) for x in e["step_ticks"]] == [int(w["ke"] * a[s] + max(w["kk"], w["kd"]) * nb[s]) for s in range(S)]


def test_set_births_rejects_bad_input(oracle):
    A = _pack([[1, 1], [1, 1]])
    with pytest.raises(Exception):
        oracle.Problem(2, 1, 2, A, 2, *TABLE1, birth=[0, 1])       # unit 1 is read at step 0, before it exists
    with pytest.raises(Exception):
        oracle.Problem(2, 1, 2, _pack([[1, 0], [1, 1]]), 2, *TABLE1, birth=[0, 2])     # birth beyond the horizon


def test_static_init_follows_births(oracle):
    rng = np.random.default_rng(8)
    U, S = 30, 20
    birth, alive, A, cap = _random_growing(rng, U, S)
    g = oracle.Problem(U, 1, S, _pack(A), cap, *TABLE1, birth=birth)
    f = oracle.Problem(U, 1, S, _pack(A), cap, *TABLE1)
    for mode in (0, 1):
        Pg = wl.unpack_bits(g.init_placement(mode), U)
        Pf = wl.unpack_bits(f.init_placement(mode), U)
        assert np.array_equal(Pg, Pf & alive)


def _all_clean_schedules(alive):
    S, U = alive.shape
    cells = [(s, u) for s in range(S) for u in range(U) if alive[s, u]]
    for bits in itertools.product((0, 1), repeat=len(cells)):
        P = np.zeros((S, U), np.uint8)
        for (s, u), b in zip(cells, bits):
            P[s, u] = b
        yield P


def test_annealer_reaches_the_exhaustive_optimum(oracle):
    """Tiny growing instances: every schedule is enumerated; the annealed bound is never below the optimum and,
    with a generous budget, reaches it."""
    rng = np.random.default_rng(3)
    for case in range(3):
        U, S, cap = 3, 4, 2
        birth = np.array([0, 1, 2], np.uint32) if case else np.array([0, 0, 2], np.uint32)
        alive = birth[None, :] <= np.arange(S)[:, None]
        A = ((rng.random((S, U)) < 0.7) & alive).astype(np.uint8)
        g = oracle.Problem(U, 1, S, _pack(A), cap, *TABLE1, birth=birth)
        best = None
        for P in _all_clean_schedules(alive):
            if (P.sum(1) > cap).any():
                continue
            t = g.eval(_pack(P))["total_ticks"]
            best = t if best is None else min(best, t)
        ap = g.make_params(chains=8, moves=4000, seed=case, levels=16, p0=0.5)
        out = g.anneal(ap)
        assert out["best_ticks"] >= best
        assert out["best_ticks"] == best
        assert g.check_total(out["best_schedule"], out["best_ticks"])


def test_incremental_cost_and_clean_state(oracle):
    rng = np.random.default_rng(21)
    U, S = 48, 40
    birth, alive, A, cap = _random_growing(rng, U, S, cap_frac=0.3)
    g = oracle.Problem(U, 1, S, _pack(A), cap, *TABLE1, birth=birth)
    for p0 in (0.8, 1e-3):
        ap = g.make_params(chains=3, moves=3000, seed=4, levels=8, p0=p0)
        res, fin, best = g.anneal_chains(ap, 0, 3, want_final=True, want_best=True)
        for r, F, B in zip(res, fin, best):
            assert g.check_total(F, r.final_ticks) and g.check_total(B, r.best_ticks)
            assert not (wl.unpack_bits(F, U) & ~alive).any()           # nothing placed before it exists
            assert r.n_changed > 0


def test_trace_layers(oracle):
    """With L layers a group reads only at the steps of its layer, and there its picks are those of the single-layer
    generator run over the tokens (the importance of a unit advances once per token)."""
    L, heads, n, N, k = 3, 2, 24, 7, 5
    tp = wl.custom_trace_params(L * heads, n, N * L, k, rho=0.9, seed=6)
    base = tp.pop("base")
    accL = wl.unpack_bits(oracle.trace_generate(**tp, base=base, layers=L), L * heads * n)
    tp1 = dict(tp, steps=N)
    acc1 = wl.unpack_bits(oracle.trace_generate(**tp1, base=base), L * heads * n)
    for s in range(N * L):
        tok, layer = divmod(s, L)
        for g in range(L * heads):
            row = accL[s, g * n:(g + 1) * n]
            if g // heads == layer:
                assert np.array_equal(row, acc1[tok, g * n:(g + 1) * n])
            else:
                assert not row.any()


def test_trace_births(oracle):
    L, heads, n, N, k = 2, 2, 16, 10, 4
    U = L * heads * n
    prompt = 3
    birth = np.zeros(U, np.uint32)
    for g in range(L * heads):
        for i in range(prompt, n):
            birth[g * n + i] = min((i - prompt) * L + g // heads + 1, N * L - 1)
    tp = wl.custom_trace_params(L * heads, n, N * L, k, rho=0.9, seed=9)
    base = tp.pop("base")
    acc = wl.unpack_bits(oracle.trace_generate(**tp, base=base, layers=L, birth=birth), U)
    alive = birth[None, :] <= np.arange(N * L)[:, None]
    assert not (acc & ~alive).any()
    for s in range(N * L):
        for g in range(L * heads):
            sl = slice(g * n, (g + 1) * n)
            want = min(k, int(alive[s, sl].sum())) if g // heads == s % L else 0
            assert int(acc[s, sl].sum()) == want
    # once every unit exists the picks are those of the trace without births
    full = wl.unpack_bits(oracle.trace_generate(**tp, base=base, layers=L), U)
    late = [s for s in range(N * L) if alive[s].all()]
    assert late and all(np.array_equal(acc[s], full[s]) for s in late)
