"""Replica exchange on the GPU vs the oracle: every chain's results, the rungs held at the end, the exchange counts,
the bound and the winner's schedule, all bit-exact."""
import numpy as np
import pytest
import torch

from paper_2508_13231_b200 import workloads as wl
from gpu_util import both_problems, named_problem, to_dev, to_np

pytestmark = pytest.mark.gpu
GB = 10 ** 9


@pytest.fixture(scope="module")
def kvp():
    from paper_2508_13231_b200 import kvp
    return kvp


def _check(g, o, rungs, every, **kw):
    gp, op = g.make_params(**kw), o.make_params(**kw)
    out = g.anneal_exchange(gp, rungs, every)
    ref = o.anneal_exchange(op, rungs, every, want_best=True)
    assert [r.astuple() for r in out["per_chain"]] == [r.astuple() for r in ref["per_chain"]]
    assert out["final_rung"] == ref["final_rung"].tolist()
    assert out["n_exchanged"] == ref["n_exchanged"].tolist()
    st = out["stats"]
    assert (out["best_ticks"], st.best_chain) == (ref["best_ticks"], ref["best_chain"])
    assert np.array_equal(to_np(out["best_schedule"]), ref["best_schedule"])
    assert out["best_seconds"] == pytest.approx(ref["best_ticks"] * o.seconds_per_tick, rel=1e-9)
    assert st.exchanges_accepted * 2 == sum(out["n_exchanged"])
    rounds = (kw["moves"] + every - 1) // every
    assert st.exchange_rounds == rounds and st.moves_total == kw["chains"] * kw["moves"]
    ev = g.eval(out["best_schedule"])
    assert int(ev["total_ticks"][0]) == out["best_ticks"] and int(ev["bad_step"][0]) == -1
    return out


def test_exchange_tables_match_the_oracle(kvp, oracle):
    import ctypes as C
    temps = np.array([900.0, 333.3, 333.3, 40.0, 3.0, 0.5, 0.2], np.float64)
    pair = np.zeros(6, np.float64)
    always = np.zeros(6, np.uint32)
    assert kvp._lib().kvp_exchange_temps(C.c_void_p(temps.ctypes.data), C.c_uint32(7), C.c_void_p(pair.ctypes.data),
                                         C.c_void_p(always.ctypes.data)) == 0
    opair = np.ones(6, np.float64)
    oalways = np.zeros(6, np.uint32)
    assert oracle.lib().kvpo_exchange_temps(temps.ctypes.data_as(C.POINTER(C.c_double)), C.c_uint32(7),
                                            opair.ctypes.data_as(C.POINTER(C.c_double)),
                                            oalways.ctypes.data_as(C.POINTER(C.c_uint32))) == 0
    assert np.array_equal(pair, opair) and np.array_equal(always, oalways)
    assert list(always) == [0, 1, 0, 0, 0, 1]                # equal temperatures, and two below one tick


@pytest.mark.parametrize("U,S,cap", [(120, 70, 30),          # schedules in shared memory
                                     (3, 2, 2),              # the enumerable instance of the oracle's pins
                                     (3000, 300, 700)])      # schedules in global scratch (copy-on-write slices)
def test_exchange_parity_shapes(kvp, oracle, U, S, cap):
    A = wl.random_access(U, S, 0.25, seed=U + S)
    g, o = both_problems(kvp, oracle, U, 8192, S, A, cap, (8000 * GB, 900 * GB, 900 * GB))
    # ladders of 4 with a given ladder; of 8 with the default ladder; one rung; exchanges after every move; a round
    # length that does not divide the budget; more rounds than moves allow
    _check(g, o, 4, 50, chains=12, moves=3000, levels=4, temps=[900.0, 300.0, 100.0, 30.0], seed=3)
    _check(g, o, 8, 64, chains=16, moves=2500, levels=8, p0=0.6, alpha=0.6, seed=4)
    _check(g, o, 1, 100, chains=5, moves=1000, levels=1, temps=[200.0], seed=5)
    _check(g, o, 2, 1, chains=6, moves=300, levels=2, temps=[500.0, 100.0], seed=6)
    _check(g, o, 3, 777, chains=9, moves=2000, levels=3, temps=[400.0, 400.0, 60.0], seed=7, p_swap_256=200, max_len_log2=3)
    _check(g, o, 4, 10 ** 6, chains=8, moves=500, levels=4, p0=0.5, alpha=0.5, seed=8)


def test_exchange_split_by_ladders(kvp, oracle):
    U, S, cap = 200, 90, 50
    A = wl.random_access(U, S, 0.3, seed=12)
    g, o = both_problems(kvp, oracle, U, 8192, S, A, cap, (4900 * GB, 900 * GB, 500 * GB))
    kw = dict(moves=3000, levels=4, p0=0.5, alpha=0.55, seed=9)
    whole = g.anneal_exchange(g.make_params(chains=16, **kw), 4, 40)
    for first in (0, 8, 12):
        part = _check(g, o, 4, 40, chains=4, first_chain=first, **kw)
        assert [r.astuple() for r in part["per_chain"]] == [r.astuple() for r in whole["per_chain"][first:first + 4]]
        assert part["final_rung"] == whole["final_rung"][first:first + 4]


def test_exchange_single_head_many_ladders(kvp, oracle):
    # a GPU-filling job: 128 ladders of 8 on the single_head problem; the oracle follows four of the ladders
    g, o, cfg, A = named_problem(kvp, oracle, "single_head")
    kw = dict(moves=20_000, levels=8, p0=0.3, alpha=0.5, seed=2)
    out = g.anneal_exchange(g.make_params(chains=1024, **kw), 8, 250)
    assert out["stats"].exchanges_tried > 0 and 0 < out["stats"].exchanges_accepted < out["stats"].exchanges_tried
    for first in (0, 8, 504, 1016):
        ref = o.anneal_exchange(o.make_params(chains=8, first_chain=first, **kw), 8, 250)
        assert [r.astuple() for r in out["per_chain"][first:first + 8]] == [r.astuple() for r in ref["per_chain"]]
        assert out["final_rung"][first:first + 8] == ref["final_rung"].tolist()
    w = out["stats"].best_chain
    assert w == min(range(1024), key=lambda c: (out["per_chain"][c].best_ticks, c))
    lad = w // 8 * 8
    ref = o.anneal_exchange(o.make_params(chains=8, first_chain=lad, **kw), 8, 250, want_best=True)
    assert ref["best_chain"] == w and ref["best_ticks"] == out["best_ticks"]
    assert np.array_equal(to_np(out["best_schedule"]), ref["best_schedule"])


def test_exchange_layer_8b_global_slices(kvp, oracle):
    # schedules of 512 KB in global scratch, winner rebuilt by replaying the chain through the rungs it held
    g, o, cfg, A = named_problem(kvp, oracle, "layer_8b")
    kw = dict(moves=6000, levels=4, p0=0.05, alpha=0.3, seed=6)
    out = g.anneal_exchange(g.make_params(chains=64, **kw), 4, 200)
    for first in (0, 28, 60):
        ref = o.anneal_exchange(o.make_params(chains=4, first_chain=first, **kw), 4, 200)
        assert [r.astuple() for r in out["per_chain"][first:first + 4]] == [r.astuple() for r in ref["per_chain"]]
        assert out["final_rung"][first:first + 4] == ref["final_rung"].tolist()
        assert out["n_exchanged"][first:first + 4] == ref["n_exchanged"].tolist()
    w = out["stats"].best_chain
    lad = w // 4 * 4
    ref = o.anneal_exchange(o.make_params(chains=4, first_chain=lad, **kw), 4, 200, want_best=True)
    assert ref["best_chain"] == w and np.array_equal(to_np(out["best_schedule"]), ref["best_schedule"])


def test_exchange_argument_errors(kvp, oracle):
    A = wl.random_access(64, 20, 0.3, seed=1)
    g, _ = both_problems(kvp, oracle, 64, 8192, 20, A, 16, (8000 * GB, 900 * GB, 900 * GB))
    for rungs, every, kw in ((2, 5, dict(chains=5, moves=10, levels=2)),              # chains not a multiple of rungs
                             (2, 5, dict(chains=4, moves=10, levels=3)),              # levels != rungs
                             (2, 0, dict(chains=4, moves=10, levels=2)),              # no round length
                             (2, 5, dict(chains=4, moves=10, levels=2, first_chain=1)),
                             (2, 5, dict(chains=4, moves=10, levels=2, temps=[3.0, 9.0])),   # a rising ladder
                             (2, 5, dict(chains=4, moves=10, levels=2, early_stop_permille=1))):
        with pytest.raises(kvp.KvpError) as e:
            g.anneal_exchange(g.make_params(**kw), rungs, every)
        assert e.value.code == kvp.ERR_ARG
