"""Runs the oracle on several host cores (separate processes, started with spawn so that no child inherits a
CUDA context). Imports nothing but the oracle and the workload definitions.

Chains are independent and so are the (layer, head) groups of a trace, so both are farmed out in contiguous pieces.
For the large configurations the access bitmap is generated once (in parallel, by the oracle), kept in a file of the
system's temporary folder for the rest of the test session and mapped by the workers that run chains on it."""
import atexit
import multiprocessing as mp
import os
import tempfile

import numpy as np

_trace_files = {}


def _procs(limit, jobs):
    return max(1, min(os.cpu_count() or 1, limit, jobs))


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
    procs = _procs(max_procs, n_chains)
    step = (n_chains + procs - 1) // procs
    jobs = [(name, kw, lo, min(lo + step, n_chains)) for lo in range(0, n_chains, step)]
    with mp.get_context("spawn").Pool(procs) as pool:
        chunks = pool.map(_chunk, jobs)
    return [t for ch in chunks for t in ch]


def _groups(args):
    name, seed, lo, n = args
    from oracle import kvpo
    from paper_2508_13231_b200 import workloads as wl
    return kvpo.trace_generate(**wl.trace_params(name, seed), group_begin=lo, group_count=n)


def oracle_trace_parallel(name, seed=0, max_procs=32):
    """The oracle's access bitmap of a named configuration, its groups spread over the host cores.
    -> (uint32 [S][W32], path of a .npy copy that worker processes map)."""
    key = (name, seed)
    if key in _trace_files:
        return np.load(_trace_files[key]), _trace_files[key]
    from paper_2508_13231_b200 import workloads as wl
    G = wl.CONFIGS[name]["groups"]
    procs = _procs(max_procs, G)
    step = max(1, (G + 4 * procs - 1) // (4 * procs))
    jobs = [(name, seed, lo, min(step, G - lo)) for lo in range(0, G, step)]
    with mp.get_context("spawn").Pool(procs) as pool:
        parts = pool.map(_groups, jobs)
    A = parts[0]
    for part in parts[1:]:
        A |= part                                  # a piece holds the bits of its own groups only
    fd, path = tempfile.mkstemp(prefix=f"kvpo_trace_{name}_{seed}_", suffix=".npy")
    os.close(fd)
    np.save(path, A)
    _trace_files[key] = path
    atexit.register(lambda p=path: os.path.exists(p) and os.remove(p))
    return A, path


def _sampled(args):
    name, path, kw, chains, want_best = args
    from oracle import kvpo
    from paper_2508_13231_b200 import workloads as wl
    cfg = wl.CONFIGS[name]
    A = np.load(path, mmap_mode="r")
    o = kvpo.Problem(wl.units(cfg), cfg["bytes_per_unit"], cfg["steps"], np.ascontiguousarray(A), cfg["cap"], *cfg["bw"])
    ap = o.make_params(**kw)
    temps, mean = o.temps(ap)
    table, shifts = kvpo.accept_table(temps)
    out = []
    for c in chains:
        res, _, bst = o.anneal_chains(ap, c, 1, want_best=want_best, table=table, shifts=shifts)
        out.append((c, res[0].astuple(), bst[0] if want_best else None))
    return mean, out


def oracle_chains_sampled(name, trace_path, kw, chains, want_best=(), max_procs=32):
    """The oracle's results of the listed chains of a named configuration on the bitmap stored at trace_path.
    -> (calibration mean delta, {chain: result tuple}, {chain: best schedule} for the chains in want_best)."""
    chains = sorted(set(chains) | set(want_best))
    procs = _procs(max_procs, len(chains))
    plain = [c for c in chains if c not in set(want_best)]
    jobs = [(name, trace_path, kw, plain[i::procs], False) for i in range(procs) if plain[i::procs]]
    jobs += [(name, trace_path, kw, [c], True) for c in want_best]
    with mp.get_context("spawn").Pool(_procs(max_procs, len(jobs))) as pool:
        parts = pool.map(_sampled, jobs)
    results, best = {}, {}
    for mean, out in parts:
        for c, tup, bst in out:
            results[c] = tup
            if bst is not None:
                best[c] = bst
    return parts[0][0], results, best
