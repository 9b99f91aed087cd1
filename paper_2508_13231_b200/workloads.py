"""Seeded synthetic workloads: sizes, parameters and random inputs only.

This module holds none of the method's arithmetic. It names the benchmark
configurations (shapes of LLaMA-class KV caches under block-sparse attention,
standing in for the recorded LongBench/NarrativeQA attention traces of the
paper's Section IV-A, which are not reproduced), turns their real-valued
parameters into the integer parameters the trace generator takes, draws the
static per-unit log-importance `base` with numpy, and draws random feasible
schedules for cost-model tests. It is the only module used by both the CUDA
path's callers and the CPU oracle's callers; it imports neither.
"""
import math

import numpy as np

TB = 10 ** 12
Q16 = 65536

# name -> shape and recipe. p0: initial acceptance ratio used by the benchmarks (a near-greedy start: with the paper's 0.8
# the walk randomises a schedule of 10^5..10^8 bits that these move budgets cannot re-anneal).
#  bw = (B_h, B_k, B_d) bytes/s. importance:
#   zipf: base[u] = -s_g * ln(rank+1), rank = random permutation inside the group
#   recency_blocks/recency_boost: the last blocks of each group get a static boost
CONFIGS = {
    "tiny": dict(groups=1, units_per_group=16, steps=32, topk=4, bytes_per_unit=8192, cap=6,
                 bw=(8 * TB, 1 * TB, 1 * TB), rho=0.9, sigma=1.0, zipf=None,
                 recency_blocks=2, recency_boost=2.0, burst_p=0.0, burst_jump=0.0,
                 chains=64, moves=10_000, p0=1e-6),
    "single_head": dict(groups=1, units_per_group=256, steps=512, topk=26, bytes_per_unit=8192, cap=64,
                        bw=(8 * TB, 9 * TB // 10, 9 * TB // 10), rho=0.95, sigma=1.0, zipf=(1.1, 1.1),
                        recency_blocks=0, recency_boost=0.0, burst_p=0.0, burst_jump=0.0,
                        chains=1024, moves=100_000, p0=1e-6),
    "layer_8b": dict(groups=8, units_per_group=2048, steps=256, topk=256, bytes_per_unit=8192, cap=4915,
                     bw=(8 * TB, 9 * TB // 10, 9 * TB // 10), rho=0.98, sigma=1.0, zipf=(0.8, 1.4),
                     recency_blocks=0, recency_boost=0.0, burst_p=0.0, burst_jump=0.0,
                     chains=1024, moves=200_000, p0=1e-6),
    "full_8b": dict(groups=256, units_per_group=2048, steps=128, topk=205, bytes_per_unit=8192, cap=104857,
                    bw=(8 * TB, 9 * TB // 10, 9 * TB // 10), rho=0.97, sigma=1.0, zipf=None,
                    recency_blocks=16, recency_boost=16.0, burst_p=0.0, burst_jump=0.0,
                    chains=4096, moves=250_000, p0=1e-6),
    "long_70b": dict(groups=640, units_per_group=4096, steps=64, topk=205, bytes_per_unit=16384, cap=262144,
                     bw=(8 * TB, 45 * TB // 100, 45 * TB // 100), rho=0.95, sigma=1.0, zipf=None,
                     recency_blocks=0, recency_boost=0.0, burst_p=0.01, burst_jump=4.0,
                     chains=8192, moves=1_000_000, p0=1e-6),
    # Table I bandwidths (4.9 TB/s HBM, 900 GB/s link, 500 GB/s DRAM) on the layer_8b shape
    "gh200": dict(groups=8, units_per_group=2048, steps=256, topk=256, bytes_per_unit=8192, cap=4915,
                  bw=(49 * TB // 10, 9 * TB // 10, 5 * TB // 10), rho=0.98, sigma=1.0, zipf=(0.8, 1.4),
                  recency_blocks=0, recency_boost=0.0, burst_p=0.0, burst_jump=0.0,
                  chains=1024, moves=200_000, p0=1e-6),
    # long_70b cut down to 8 of its 640 groups (same steps, top-k, bursts, capacity share, bandwidths): the chains run the
    # same kernel instantiation as long_70b (two-word columns in global scratch) on 256 KB of schedule each, small enough
    # for a profiler to hold a GPU-filling job of thousands of chains in a few hundred MB
    "profile_70b": dict(groups=8, units_per_group=4096, steps=64, topk=205, bytes_per_unit=16384, cap=3276,
                        bw=(8 * TB, 45 * TB // 100, 45 * TB // 100), rho=0.95, sigma=1.0, zipf=None,
                        recency_blocks=0, recency_boost=0.0, burst_p=0.01, burst_jump=4.0,
                        chains=2368, moves=100_000, p0=1e-6),
}
ORDER = ["tiny", "single_head", "layer_8b", "full_8b", "long_70b"]

# Growing caches with (token, layer) steps: `layers` x `heads` groups of `units_per_group` units (one unit = the KV
# entry of one token in one (layer, kv-head)); the first `prompt` units of every group exist from the start, unit
# prompt + j is written by decoded token j + 1 at the step of its layer. steps = layers * (units_per_group - prompt + 1).
GROWING = {
    "growing_tiny": dict(layers=2, heads=1, units_per_group=12, prompt=4, topk=3, bytes_per_unit=512, cap=6,
                         bw=(49 * TB // 10, 9 * TB // 10, 5 * TB // 10), rho=0.9, zipf=None,
                         chains=32, moves=4_000, p0=1e-6),
    "growing_small": dict(layers=4, heads=2, units_per_group=64, prompt=32, topk=8, bytes_per_unit=512, cap=96,
                          bw=(8 * TB, 9 * TB // 10, 9 * TB // 10), rho=0.95, zipf=(0.8, 1.4),
                          chains=256, moves=20_000, p0=1e-6),
    # the shape of LLaMA-3.1-8B (32 layers, 8 KV heads): 480 prompt tokens, 32 decoded ones
    "growing_8b": dict(layers=32, heads=8, units_per_group=512, prompt=480, topk=51, bytes_per_unit=512, cap=26214,
                       bw=(8 * TB, 9 * TB // 10, 9 * TB // 10), rho=0.97, zipf=(0.8, 1.4),
                       chains=1024, moves=100_000, p0=1e-6),
}


def growing_shape(cfg):
    """-> (groups, units, steps) of a GROWING configuration."""
    groups = cfg["layers"] * cfg["heads"]
    tokens = cfg["units_per_group"] - cfg["prompt"] + 1
    return groups, groups * cfg["units_per_group"], cfg["layers"] * tokens


def growing_births(cfg):
    """uint32 [U]: 0 for the prompt's units, else the step (token * layers + layer) at which the unit is written."""
    groups, _, _ = growing_shape(cfg)
    n, L = cfg["units_per_group"], cfg["layers"]
    birth = np.zeros((groups, n), np.uint32)
    for g in range(groups):
        layer = g // cfg["heads"]
        j = np.arange(n - cfg["prompt"])
        birth[g, cfg["prompt"]:] = (j + 1) * L + layer
    return birth.reshape(-1)


def growing_trace_params(name, seed=0):
    """Trace parameters of a GROWING configuration (pass layers=cfg['layers'] and the births to the generator too)."""
    cfg = GROWING[name]
    groups, _, steps = growing_shape(cfg)
    return custom_trace_params(groups, cfg["units_per_group"], steps, cfg["topk"], cfg["rho"], zipf=cfg["zipf"], seed=seed)


def units(cfg):
    return cfg["groups"] * cfg["units_per_group"]


def words_per_row(cfg):
    return (units(cfg) + 31) // 32


def trace_params(name, seed=0):
    """Integer parameters of the trace generator for a named configuration.

    -> dict(groups, units_per_group, steps, topk, seed, rho_q, c_q, sigma_q,
            burst_jump, burst_thr, base (int32 [U] or None))
    """
    cfg = CONFIGS[name]
    G, n = cfg["groups"], cfg["units_per_group"]
    rng = np.random.Generator(np.random.PCG64([seed, 0x6B7670]))
    base = None
    if cfg["zipf"] is not None or cfg["recency_blocks"]:
        base = np.zeros((G, n), np.int64)
        if cfg["zipf"] is not None:
            lo, hi = cfg["zipf"]
            for g in range(G):
                s_g = lo if lo == hi else rng.uniform(lo, hi)
                rank = rng.permutation(n)
                base[g] -= np.rint(s_g * np.log(rank + 1.0) * Q16).astype(np.int64)
        if cfg["recency_blocks"]:
            base[:, n - cfg["recency_blocks"]:] += int(round(cfg["recency_boost"] * Q16))
        base = base.reshape(-1).astype(np.int32)
    rho, sigma = cfg["rho"], cfg["sigma"]
    return dict(
        groups=G, units_per_group=n, steps=cfg["steps"], topk=cfg["topk"], seed=seed,
        rho_q=int(round(rho * Q16)), c_q=int(round(sigma * math.sqrt(1.0 - rho * rho) * Q16)),
        sigma_q=int(round(sigma * Q16)), burst_jump=int(round(cfg["burst_jump"] * Q16)),
        burst_thr=int(cfg["burst_p"] * 2 ** 32), base=base)


def custom_trace_params(groups, units_per_group, steps, topk, rho, sigma=1.0, zipf=None, seed=0):
    """Trace parameters for an ad-hoc shape (same recipe as the named configurations, no recency, no bursts)."""
    rng = np.random.Generator(np.random.PCG64([seed, 0x637573]))
    base = None
    if zipf is not None:
        lo, hi = zipf
        base = np.zeros((groups, units_per_group), np.int64)
        for g in range(groups):
            s_g = lo if lo == hi else rng.uniform(lo, hi)
            base[g] = -np.rint(s_g * np.log(rng.permutation(units_per_group) + 1.0) * Q16).astype(np.int64)
        base = base.reshape(-1).astype(np.int32)
    return dict(groups=groups, units_per_group=units_per_group, steps=steps, topk=topk, seed=seed,
                rho_q=int(round(rho * Q16)), c_q=int(round(sigma * math.sqrt(1.0 - rho * rho) * Q16)),
                sigma_q=int(round(sigma * Q16)), burst_jump=0, burst_thr=0, base=base)


def random_schedules(num_units, steps, cap, count, seed, churn=0.02):
    """`count` random feasible schedules, uint32 [count][steps][ceil(U/32)].

    Row 0 holds a random subset of at most `cap` units; each later row evicts and
    admits a few random units (about `churn` of the capacity) so that migration
    terms are exercised. Pad bits are 0.
    """
    rng = np.random.Generator(np.random.PCG64([seed, 0x736368]))
    w32 = (num_units + 31) // 32
    out = np.zeros((count, steps, w32), np.uint32)
    for i in range(count):
        fill = int(rng.integers(0, cap + 1)) if cap else 0
        res = np.zeros(num_units, bool)
        if fill:
            res[rng.choice(num_units, size=fill, replace=False)] = True
        for s in range(steps):
            if s:
                k = int(rng.integers(0, max(2, int(churn * max(cap, 1)) + 1)))
                inside = np.flatnonzero(res)
                if inside.size and k:
                    res[rng.choice(inside, size=min(k, inside.size), replace=False)] = False
                room = cap - int(res.sum())
                outside = np.flatnonzero(~res)
                k2 = int(rng.integers(0, max(1, min(room, k + 1)) + 1)) if room > 0 else 0
                if outside.size and k2:
                    res[rng.choice(outside, size=min(k2, outside.size, room), replace=False)] = True
            bits = np.zeros(w32 * 32, np.uint8)
            bits[:num_units] = res
            out[i, s] = np.packbits(bits.reshape(w32, 32), axis=1, bitorder="little").view(np.uint32).reshape(w32)
    return out


def random_access(num_units, steps, density, seed):
    """Unstructured random access bitmap (each bit set with probability `density`)."""
    rng = np.random.Generator(np.random.PCG64([seed, 0x616363]))
    w32 = (num_units + 31) // 32
    bits = np.zeros((steps, w32 * 32), np.uint8)
    bits[:, :num_units] = rng.random((steps, num_units)) < density
    return np.packbits(bits.reshape(steps, w32, 32), axis=2, bitorder="little").view(np.uint32).reshape(steps, w32)


def unpack_bits(bitmap, num_units):
    """uint32 [..., W32] -> uint8 [..., num_units] of 0/1."""
    b = np.ascontiguousarray(bitmap, dtype=np.uint32)
    bits = np.unpackbits(b.view(np.uint8).reshape(*b.shape, 4), axis=-1, bitorder="little")
    return bits.reshape(*b.shape[:-1], b.shape[-1] * 32)[..., :num_units]


def pack_bits(bits):
    """uint8/bool [..., U] -> uint32 [..., ceil(U/32)]."""
    bits = np.asarray(bits).astype(np.uint8)
    U = bits.shape[-1]
    w32 = (U + 31) // 32
    pad = np.zeros(bits.shape[:-1] + (w32 * 32,), np.uint8)
    pad[..., :U] = bits
    return np.packbits(pad.reshape(*pad.shape[:-1], w32, 32), axis=-1, bitorder="little").view(np.uint32).reshape(
        *pad.shape[:-1], w32)
