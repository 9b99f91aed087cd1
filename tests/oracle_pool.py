"""Runs oracle chains of a named configuration on several host cores (separate processes, started with spawn
so that no child inherits a CUDA context). Imports nothing but the oracle and the workload definitions."""
import multiprocessing as mp
import os


def _chunk(args):
    name, kw, lo, hi = args
    from oracle import kvpo
    from paper_2508_13231_b200 import workloads as wl
    cfg = wl.CONFIGS[name]
    A = kvpo.trace_generate(**wl.trace_params(name, 0))
    o = kvpo.Problem(wl.units(cfg), cfg["bytes_per_unit"], cfg["steps"], A, cfg["cap"], *cfg["bw"])
    res, _, _ = o.anneal_chains(o.make_params(**kw), lo, hi - lo)
    return [r.astuple() for r in res]


def oracle_chains_parallel(name, kw, n_chains, max_procs=32):
    """Per-chain result tuples of chains 0..n_chains-1, computed by the oracle."""
    procs = max(1, min(os.cpu_count() or 1, max_procs, n_chains))
    step = (n_chains + procs - 1) // procs
    jobs = [(name, kw, lo, min(lo + step, n_chains)) for lo in range(0, n_chains, step)]
    with mp.get_context("spawn").Pool(procs) as pool:
        chunks = pool.map(_chunk, jobs)
    return [t for ch in chunks for t in ch]
