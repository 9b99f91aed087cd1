"""Growing cache and (token, layer) steps on the GPU vs the oracle: trace, cost and annealing, all bit-exact."""
import numpy as np
import pytest
import torch

from paper_2508_13231_b200 import workloads as wl
from gpu_util import to_dev, to_np, u64
from oracle_pool import oracle_chains_parallel

pytestmark = pytest.mark.gpu
GB = 10 ** 9


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


def _birth_dev(birth):
    return torch.from_numpy(np.ascontiguousarray(birth, np.uint32).view(np.int32)).cuda()


def _shape(layers, heads, n, prompt):
    cfg = dict(layers=layers, heads=heads, units_per_group=n, prompt=prompt)
    groups, U, S = wl.growing_shape(cfg)
    return cfg, groups, U, S, wl.growing_births(cfg)


def _trace_both(kvp, oracle, tp, layers, birth):
    base = tp["base"]
    args = {k: v for k, v in tp.items() if k != "base"}
    ref = oracle.trace_generate(**args, base=base, layers=layers, birth=birth)
    got = kvp.trace_generate(**args, base=None if base is None else torch.from_numpy(base).cuda(), layers=layers,
                             birth=None if birth is None else _birth_dev(birth))
    return got, ref


def _problems(kvp, oracle, U, bpu, S, A, cap, bw, birth, hw=None, ew=None, mig_flags=3):
    g = kvp.Problem(U, bpu, S, to_dev(A), cap, *bw, mig_flags=mig_flags, hw=hw, ew=ew, birth=_birth_dev(birth))
    o = oracle.Problem(U, bpu, S, A, cap, *bw, mig_flags=mig_flags, hw=hw, ew=ew, birth=birth)
    return g, o


def _named(kvp, oracle, name, seed=0):
    cfg = wl.GROWING[name]
    groups, U, S = wl.growing_shape(cfg)
    birth = wl.growing_births(cfg)
    tp = wl.growing_trace_params(name, seed)
    got, A = _trace_both(kvp, oracle, tp, cfg["layers"], birth)
    assert np.array_equal(to_np(got), A)
    return _problems(kvp, oracle, U, cfg["bytes_per_unit"], S, A, cfg["cap"], cfg["bw"], birth) + (cfg, A, birth)


@pytest.mark.parametrize("layers,heads,n,prompt,k", [
    (2, 1, 12, 4, 3), (4, 2, 64, 32, 8), (3, 1, 45, 20, 7), (3, 2, 235, 100, 40), (1, 2, 96, 90, 95), (5, 1, 33, 0, 4),
    (2, 2, 2500, 2400, 100),
])
def test_trace_layers_and_births(kvp, oracle, layers, heads, n, prompt, k):
    cfg, groups, U, S, birth = _shape(layers, heads, n, prompt)
    tp = wl.custom_trace_params(groups, n, S, k, rho=0.9, zipf=(0.8, 1.2), seed=layers + n)
    got, ref = _trace_both(kvp, oracle, tp, layers, birth)
    assert np.array_equal(to_np(got), ref)
    got, ref = _trace_both(kvp, oracle, tp, layers, None)         # layers alone
    assert np.array_equal(to_np(got), ref)


def test_trace_growing_8b_sampled_groups(kvp, oracle):
    cfg = wl.GROWING["growing_8b"]
    groups, U, S = wl.growing_shape(cfg)
    birth = wl.growing_births(cfg)
    tp = wl.growing_trace_params("growing_8b", seed=0)
    base = tp["base"]
    args = {k: v for k, v in tp.items() if k != "base"}
    got = to_np(kvp.trace_generate(**args, base=torch.from_numpy(base).cuda(), layers=cfg["layers"], birth=_birth_dev(birth)))
    n = cfg["units_per_group"]
    for g in (0, 7, 100, 255):
        ref = oracle.trace_generate(**args, base=base, layers=cfg["layers"], birth=birth, group_begin=g, group_count=1)
        w0, w1 = g * n // 32, (g + 1) * n // 32
        assert np.array_equal(got[:, w0:w1], ref[:, w0:w1]), g


@pytest.mark.parametrize("layers,heads,n,prompt", [
    (2, 1, 12, 4),          # one word per row
    (3, 1, 45, 20),         # 5 words: narrow rows, scalar loads
    (4, 2, 64, 32),         # 16 words: narrow rows, vector loads
    (3, 1, 235, 100),       # 23 words: wide rows, scalar loads
    (4, 4, 256, 200),       # 128 words: wide rows, vector loads
])
def test_eval_growing(kvp, oracle, layers, heads, n, prompt):
    cfg, groups, U, S, birth = _shape(layers, heads, n, prompt)
    rng = np.random.default_rng(U + S)
    alive = birth[None, :] <= np.arange(S)[:, None]
    A = wl.pack_bits(((rng.random((S, U)) < 0.2) & alive).astype(np.uint8))
    hw, ew = (np.arange(S) % 3).astype(np.uint32), (np.arange(S) % 2).astype(np.uint32)
    cap = max(1, U // 3)
    for flags, bw in ((3, (4900 * GB, 900 * GB, 500 * GB)), (0, (8000 * GB, 900 * GB, 900 * GB))):
        g, o = _problems(kvp, oracle, U, 512, S, A, cap, bw, birth, hw=hw, ew=ew, mig_flags=flags)
        scheds = []
        for i in range(4):
            P = (rng.random((S, U)) < (0.1 + 0.2 * i))
            if i % 2 == 0:
                P &= alive                                    # a clean schedule; the others carry bits of unborn units
            scheds.append(wl.pack_bits(P.astype(np.uint8)))
        out = g.eval(to_dev(np.stack(scheds)))
        for i, P in enumerate(scheds):
            ref = o.eval(P)
            assert np.array_equal(u64(out["step_ticks"])[i], ref["step_ticks"]), (flags, i)
            assert int(u64(out["total_ticks"])[i]) == ref["total_ticks"]
            assert int(out["bad_step"][i]) == ref["bad_step"]
        g.close()


def test_eval_growing_8b(kvp, oracle):
    g, o, cfg, A, birth = _named(kvp, oracle, "growing_8b")
    groups, U, S = wl.growing_shape(cfg)
    P0 = o.init_placement(1)
    rng = np.random.default_rng(1)
    noisy = P0 ^ wl.pack_bits((rng.random((S, U)) < 0.01).astype(np.uint8))
    out = g.eval(to_dev(np.stack([P0, noisy])))
    for i, P in enumerate((P0, noisy)):
        ref = o.eval(P)
        assert np.array_equal(u64(out["step_ticks"])[i], ref["step_ticks"])
        assert int(out["bad_step"][i]) == ref["bad_step"]


def test_set_births_errors(kvp, oracle):
    S, U = 6, 40
    A = np.zeros((S, 2), np.uint32); A[0, 0] = 0b11
    ok = np.zeros(U, np.uint32)
    def make(birth):
        return kvp.Problem(U, 512, S, to_dev(A), 10, 8000 * GB, 900 * GB, 900 * GB, birth=_birth_dev(birth))
    bad = ok.copy(); bad[1] = 2                                   # unit 1 is read at step 0
    with pytest.raises(kvp.KvpError) as e:
        make(bad)
    assert e.value.code == kvp.ERR_ARG
    bad = ok.copy(); bad[5] = S                                   # beyond the horizon
    with pytest.raises(kvp.KvpError):
        make(bad)
    good = ok.copy(); good[5] = S - 1
    g = make(good)
    P = to_dev(np.zeros((1, S, 2), np.uint32))
    with pytest.raises(kvp.KvpError):
        g.policy_reactive()
    with pytest.raises(kvp.KvpError):
        g.eval_counts(P)
    tt = torch.empty(1, dtype=torch.int64, device="cuda")
    with pytest.raises(kvp.KvpError):
        g.eval_noalloc(P, None, tt, None, None, None)
    assert int(u64(g.eval(P)["total_ticks"])[0]) > 0


def _check_chains(g, o, gp, op, chains=None):
    out = g.anneal(gp, want_per_chain=True)
    temps, mean = o.temps(op)
    assert out["stats"].calib_mean_delta == mean and out["stats"].temp0 == temps[0]
    for c in (range(gp.chains) if chains is None else chains):
        want, _, _ = o.anneal_chains(op, c, 1)
        assert out["per_chain"][c].astuple() == want[0].astuple(), c
    if chains is None:
        ref = o.anneal(op)
        assert out["best_ticks"] == ref["best_ticks"] and out["stats"].best_chain == ref["best_chain"]
        assert np.array_equal(to_np(out["best_schedule"]), ref["best_schedule"])
    return out


@pytest.mark.parametrize("name", ["growing_tiny", "growing_small"])
def test_anneal_growing_named(kvp, oracle, name):
    g, o, cfg, A, birth = _named(kvp, oracle, name)
    for p0, init in ((0.8, kvp.INIT_STATIC_FREQ), (1e-3, kvp.INIT_STATIC_FIRST)):
        kw = dict(chains=min(cfg["chains"], 24), moves=min(cfg["moves"], 6000), seed=3, p0=p0, init_mode=init, levels=8)
        out = _check_chains(g, o, g.make_params(**kw), o.make_params(**kw))
        assert sum(r.n_changed for r in out["per_chain"]) > 0
        assert out["stats"].init_ticks == o.eval(o.init_placement(init))["total_ticks"]


def test_anneal_growing_odd_shapes_and_options(kvp, oracle, warps_per_chain):
    cfg, groups, U, S, birth = _shape(3, 1, 45, 20)
    rng = np.random.default_rng(4)
    alive = birth[None, :] <= np.arange(S)[:, None]
    A = wl.pack_bits(((rng.random((S, U)) < 0.3) & alive).astype(np.uint8))
    hw, ew = (np.arange(S) % 2).astype(np.uint32), (np.arange(S) % 3).astype(np.uint32)
    g, o = _problems(kvp, oracle, U, 512, S, A, 30, (4900 * GB, 900 * GB, 500 * GB), birth, hw=hw, ew=ew)
    user = wl.pack_bits((rng.random((S, U)) < 0.15).astype(np.uint8))      # carries bits of unborn units on purpose
    for kw in (dict(chains=7, moves=3001, seed=99, levels=5, p_swap_256=100, max_len_log2=4),
               dict(chains=5, moves=2000, levels=3, p_swap_256=0), dict(chains=5, moves=2000, levels=3, p_swap_256=256),
               dict(chains=4, moves=2500, levels=6, early_stop_permille=1)):
        _check_chains(g, o, g.make_params(**kw), o.make_params(**kw))
    gp = g.make_params(chains=4, moves=1500, levels=3, init_mode=kvp.INIT_USER, init_schedule=to_dev(user))
    op = o.make_params(chains=4, moves=1500, levels=3, init_mode=2, init_schedule=user)
    _check_chains(g, o, gp, op)
    # replay of one chain to an intermediate point
    gp, op = g.make_params(chains=3, moves=2000, seed=5, levels=4), o.make_params(chains=3, moves=2000, seed=5, levels=4)
    sched, res = g.chain_state(gp, 2, 777)
    want, fin, _ = o.anneal_chains(op, 2, 1, upto_moves=777, want_final=True)
    assert res.astuple() == want[0].astuple() and np.array_equal(to_np(sched), fin[0])


def test_anneal_growing_global_state(kvp, oracle, warps_per_chain):
    """A schedule too large for shared memory: chains in global scratch, the winner walked back through its undo log."""
    cfg, groups, U, S, birth = _shape(4, 4, 256, 200)
    tp = wl.custom_trace_params(groups, 256, S, 24, rho=0.95, zipf=(0.8, 1.4), seed=2)
    got, A = _trace_both(kvp, oracle, tp, 4, birth)
    assert np.array_equal(to_np(got), A)
    g, o = _problems(kvp, oracle, U, 512, S, A, 800, (8000 * GB, 900 * GB, 900 * GB), birth)
    for p0 in (0.5, 1e-6):
        kw = dict(chains=6, moves=20000, seed=8, p0=p0, levels=8)
        out = _check_chains(g, o, g.make_params(**kw), o.make_params(**kw))
        if p0 < 0.1:                                          # the near-greedy run improves on its start: the winner
            assert out["stats"].best_move != 2 ** 64 - 1      # is a walked-back state, not the initial schedule


def test_anneal_growing_8b_sampled_chains(kvp, oracle):
    g, o, cfg, A, birth = _named(kvp, oracle, "growing_8b")
    kw = dict(chains=16, moves=20000, seed=0, p0=cfg["p0"])
    out = g.anneal(g.make_params(**kw), want_per_chain=True)
    op = o.make_params(**kw)
    temps, mean = o.temps(op)
    assert out["stats"].calib_mean_delta == mean
    for c in (0, 9, out["stats"].best_chain):
        want, _, best = o.anneal_chains(op, c, 1, want_best=True)
        assert out["per_chain"][c].astuple() == want[0].astuple(), c
        if c == out["stats"].best_chain:
            assert np.array_equal(to_np(out["best_schedule"]), best[0])
