"""Pins of the oracle's replica exchange (parallel tempering over the temperature ladder).

What the mathematics fixes: on an instance small enough to enumerate (3 units x 2 steps, 49 feasible schedules) a
replica that holds rung j visits the schedules with their Boltzmann weights exp(-T/C_j) / Z_j, with or without
exchanges (moves are their own inverses and proposed independently of the state, so Metropolis acceptance keeps those
weights; a correct exchange rule keeps them too, a wrong one mixes the rungs); an exchange is certain when the colder
rung holds the worse schedule and has probability exp(-d / C_pair) otherwise; a ladder of equal temperatures
exchanges always and changes nothing; one rung alone is the plain annealer at one level; ladders are independent.
"""
import itertools
import math

import numpy as np
import pytest

from paper_2508_13231_b200 import workloads as wl

GB = 10 ** 9
U, S, CAP = 3, 2, 2
TEMPS = [400.0, 200.0, 100.0, 50.0]


@pytest.fixture(scope="module")
def small(oracle):
    A = wl.pack_bits(np.array([[1, 1, 0], [0, 1, 1]], np.uint8))
    prob = oracle.Problem(U, 8192, S, A, CAP, 8000 * GB, 900 * GB, 900 * GB)
    rows = [r for r in itertools.product([0, 1], repeat=U) if sum(r) <= CAP]
    energy = {}
    for a in rows:
        for b in rows:
            code = sum(x << i for i, x in enumerate(a)) | (sum(x << i for i, x in enumerate(b)) << 32)
            energy[code] = prob.eval(wl.pack_bits(np.array([a, b], np.uint8)))["total_ticks"]
    assert len(energy) == 49 and len(set(energy.values())) >= 8
    return prob, energy


def _boltzmann(energy, C):
    w = {c: math.exp(-e / C) for c, e in energy.items()}
    Z = sum(w.values())
    return {c: x / Z for c, x in w.items()}


def _tv(emp, ref):
    return 0.5 * sum(abs(emp.get(c, 0.0) - p) for c, p in ref.items()) + 0.5 * sum(v for c, v in emp.items() if c not in ref)


def _occupancy(samples, rung):
    codes = samples[..., 1][samples[..., 0] == rung]
    vals, cnt = np.unique(codes, return_counts=True)
    return dict(zip(vals.tolist(), (cnt / cnt.sum()).tolist())), len(codes)


def test_every_rung_keeps_its_boltzmann_weights(small):
    prob, energy = small
    rungs = len(TEMPS)
    # An exchange after every second move: the chains have no time to settle again between exchanges, so that a wrong
    # exchange rule shows in the occupancies (accepting every exchange puts them 0.05 to 0.33 off in total variation;
    # the correct rule stays below 0.01 at this sample size).
    ap = prob.make_params(chains=rungs * 8, moves=80_000, levels=rungs, temps=TEMPS, seed=5, max_len_log2=1)
    out = prob.anneal_exchange(ap, rungs, every=2, want_log=True, want_samples=True)
    ref = [_boltzmann(energy, C) for C in TEMPS]
    assert _tv(ref[0], ref[-1]) > 0.15 and _tv(ref[1], ref[2]) > 0.05      # the rungs are far enough apart to tell
    for j in range(rungs):
        emp, n = _occupancy(out["samples"], j)
        assert n == 8 * 40_000
        assert set(emp) <= set(energy)                                      # only feasible schedules are visited
        assert _tv(emp, ref[j]) < 0.02, j
    # exchanges did happen, in both directions, and moved every chain through the ladder
    lg = out["xlog"]
    tried = lg[..., 2] < 2
    assert tried.sum() > 50_000 and 0.3 < (lg[..., 2] == 1).sum() / tried.sum() < 0.95
    assert out["n_exchanged"].min() > 1000
    visited = {(c, int(r)) for c in range(rungs * 8) for r in np.unique(out["samples"][:, c, 0])}
    assert len(visited) == rungs * rungs * 8


def test_exchange_rule(small):
    prob, energy = small
    rungs = len(TEMPS)
    ap = prob.make_params(chains=rungs * 16, moves=100_000, levels=rungs, temps=TEMPS, seed=9, max_len_log2=1)
    out = prob.anneal_exchange(ap, rungs, every=10, want_log=True)
    lg, tb = out["xlog"], out["tables"]
    # round t tries the pairs (j, j+1) with j = t (mod 2) and no others; the last round tries none
    rounds = lg.shape[0]
    for t in (0, 1, 2, 3, rounds - 2):
        for j in range(rungs - 1):
            assert np.all((lg[t, :, j, 2] < 2) == (j % 2 == t % 2)), (t, j)
    assert np.all(lg[rounds - 1, :, :, 2] == 2)
    tried = lg[..., 2] < 2
    hot, cold, acc = lg[..., 0].astype(np.int64), lg[..., 1].astype(np.int64), lg[..., 2]
    # certain when the colder rung holds the worse schedule (or an equal one)
    sure = tried & (hot <= cold)
    assert sure.sum() > 1000 and np.all(acc[sure] == 1)
    # otherwise exp(-d / C_pair) with 1/C_pair = 1/C_cold - 1/C_hot: observed acceptances against the expectation
    for j in range(rungs - 1):
        c_pair = 1.0 / (1.0 / TEMPS[j + 1] - 1.0 / TEMPS[j])
        assert tb["pair_temps"][j] == pytest.approx(c_pair, rel=1e-12) and tb["xalways"][j] == 0
        open_ = tried[:, :, j] & (hot[:, :, j] > cold[:, :, j])
        d = (hot[:, :, j] - cold[:, :, j])[open_]
        prob_acc = np.exp(-d / c_pair)
        got = (acc[:, :, j][open_] == 1).sum()
        sigma = math.sqrt(float((prob_acc * (1 - prob_acc)).sum()))
        assert open_.sum() > 2000 and 0 < got < open_.sum()
        # the table takes exp at the middle of a bin of 2^shift ticks: at most half a bin off, relative e^(bin/2C) - 1
        slack = float(prob_acc.sum()) * (math.exp(0.5 * (1 << int(tb["xshifts"][j])) / c_pair) - 1.0)
        assert abs(got - float(prob_acc.sum())) < 5 * sigma + slack, j
    # bookkeeping: the rungs of a ladder stay a permutation, and the exchange counts are those of the log
    fr = out["final_rung"].reshape(-1, rungs)
    assert np.all(np.sort(fr, axis=1) == np.arange(rungs))
    assert out["n_exchanged"].sum() == 2 * int((acc == 1).sum())


def test_equal_temperatures_exchange_always_and_change_nothing(small):
    prob, energy = small
    rungs, C = 3, 150.0
    ap = prob.make_params(chains=rungs * 8, moves=120_000, levels=rungs, temps=[C] * rungs, seed=2, max_len_log2=1)
    out = prob.anneal_exchange(ap, rungs, every=15, want_log=True, want_samples=True)
    assert list(out["tables"]["xalways"][:rungs - 1]) == [1, 1]
    lg = out["xlog"]
    assert np.all(lg[..., 2][lg[..., 2] < 2] == 1)
    ref = _boltzmann(energy, C)
    for j in range(rungs):
        emp, _ = _occupancy(out["samples"], j)
        assert _tv(emp, ref) < 0.02


def test_one_rung_is_the_plain_annealer_at_one_level(small, oracle):
    prob, _ = small
    for every in (1, 7, 1000, 10 ** 9):
        ap = prob.make_params(chains=6, moves=5000, levels=1, temps=[120.0], seed=11, max_len_log2=1)
        out = prob.anneal_exchange(ap, 1, every=every)
        ref = prob.anneal(ap)
        assert [r.astuple() for r in out["per_chain"]] == [r.astuple() for r in ref["per_chain"]]
        assert list(out["final_rung"]) == [0] * 6 and out["n_exchanged"].sum() == 0
    # and on a larger instance with every option of the move set
    Ux, Sx, capx = 60, 40, 15
    A = wl.random_access(Ux, Sx, 0.3, seed=4)
    big = oracle.Problem(Ux, 8192, Sx, A, capx, 4900 * GB, 900 * GB, 500 * GB)
    ap = big.make_params(chains=3, moves=3000, levels=1, p0=0.3, seed=3)
    assert ([r.astuple() for r in big.anneal_exchange(ap, 1, every=64)["per_chain"]] ==
            [r.astuple() for r in big.anneal(ap)["per_chain"]])


def test_ladders_are_independent(oracle):
    """A job split by ladders (what a multi-GPU run does) gives the results of the whole job."""
    Ux, Sx, capx = 40, 30, 10
    A = wl.random_access(Ux, Sx, 0.3, seed=8)
    prob = oracle.Problem(Ux, 8192, Sx, A, capx, 8000 * GB, 900 * GB, 900 * GB)
    rungs, kw = 4, dict(moves=4000, levels=4, p0=0.5, alpha=0.6, seed=21)
    whole = prob.anneal_exchange(prob.make_params(chains=12, **kw), rungs, every=50)
    assert whole["n_exchanged"].sum() > 0
    for first in (0, 4, 8):
        part = prob.anneal_exchange(prob.make_params(chains=4, first_chain=first, **kw), rungs, every=50)
        assert [r.astuple() for r in part["per_chain"]] == [r.astuple() for r in whole["per_chain"][first:first + 4]]
        assert np.array_equal(part["final_rung"], whole["final_rung"][first:first + 4])
        assert np.array_equal(part["n_exchanged"], whole["n_exchanged"][first:first + 4])


def test_a_colder_ladder_finds_better_schedules_than_its_hot_end(oracle):
    """Sanity of the whole scheme on a non-trivial instance: the best schedule comes from the cold end of the ladder,
    and exchanging helps the cold rungs against the same ladder without exchanges (every > moves)."""
    Ux, Sx, capx = 64, 48, 16
    A = wl.random_access(Ux, Sx, 0.25, seed=5)
    prob = oracle.Problem(Ux, 8192, Sx, A, capx, 8000 * GB, 900 * GB, 900 * GB)
    rungs = 8
    kw = dict(chains=rungs * 4, moves=20_000, levels=rungs, p0=0.5, alpha=0.5, seed=1)
    on = prob.anneal_exchange(prob.make_params(**kw), rungs, every=100)
    off = prob.anneal_exchange(prob.make_params(**kw), rungs, every=10 ** 9)
    init = prob.eval(prob.init_placement(1))["total_ticks"]
    assert on["best_ticks"] < init and off["best_ticks"] < init
    assert off["n_exchanged"].sum() == 0 and list(off["final_rung"][:rungs]) == list(range(rungs))
    finals_off = np.array([r.final_ticks for r in off["per_chain"]]).reshape(-1, rungs).mean(axis=0)
    assert finals_off[-1] < finals_off[0]                         # cold rungs sit lower than hot ones
    assert on["best_ticks"] <= off["best_ticks"] * 1.02           # exchanging does not hurt the bound


def test_argument_errors(small):
    prob, _ = small
    with pytest.raises(RuntimeError):
        prob.anneal_exchange(prob.make_params(chains=5, moves=10, levels=2, temps=[9.0, 3.0]), 2, every=5)   # 5 % 2
    with pytest.raises(RuntimeError):
        prob.anneal_exchange(prob.make_params(chains=4, moves=10, levels=2, temps=[3.0, 9.0]), 2, every=5)   # rising
    with pytest.raises(RuntimeError):
        prob.anneal_exchange(prob.make_params(chains=4, moves=10, levels=2, temps=[9.0, 3.0], first_chain=1), 2, every=5)
