"""Benchmark of the whole hot path on the `single_head` configuration.

One step = trace kernel -> kvp_create (layout kernels) -> cost kernel on a small batch of schedules ->
kvp_anneal (initial cost, calibration, all chains, cross-chain reduction, winner replay and re-score).
Metric: simulated-annealing move evaluations per second (chains x moves / step time), whole job.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

N > 1 is launched with torch.distributed.run, one rank per GPU; the chains of an N x 1024-chain job are
split over the ranks (chains are independent; the only exchange is a final 8-byte MIN on the host side).
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "single_head"
METRIC = "sa_move_evals_per_sec"
UNIT = "move-evals/s"
# Issue-slot roofline of the chain kernel: 148 SMs x 4 warp schedulers x 1.965 GHz, one warp instruction per
# scheduler and cycle. Algorithmic work per move evaluation with one proposal per lane: 16 warp instructions
# (per 32 moves: Philox and decode ~105, window extraction and word-parallel bit logic ~100, work-queue scan
# and push ~100, about 35 (lane, step) cost evaluations of ~70 thread instructions each in two warp rounds
# ~150, Metropolis and in-order commit ~50).
ISSUE_PEAK_GWIPS = 148 * 4 * 1.965
# dram__bytes_read.sum + dram__bytes_write.sum of one chain-kernel launch on this workload (ncu capture summarised in
# profiles/chain_kernel_single_head.md; set to None whenever the kernel changes until it is captured again)
CHAIN_KERNEL_DRAM_BYTES = 390144
# what that capture shows of the integer datapath (fractions of peak over the launch; context beside the timed figure)
CHAIN_KERNEL_NCU = {"issue_active": 0.665, "alu_pipe": 0.574, "imad_pipe": 0.365, "warp_inst_per_move": 30.4}
ALG_WARP_INSTR_PER_MOVE = 16.0


def _clock_sampler(stop, samples):
    """SM clock and throttle reasons of this rank's GPU through NVML, every 20 ms while the timed region runs."""
    try:
        import pynvml
        pynvml.nvmlInit()
        visible = os.environ.get("CUDA_VISIBLE_DEVICES")
        idx = int(os.environ.get("LOCAL_RANK", "0"))
        if visible:
            idx = int(visible.split(",")[idx])
        h = pynvml.nvmlDeviceGetHandleByIndex(idx)
        smax = pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)
    except Exception:
        return
    bits = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}
    while not stop.is_set():
        try:
            sm = pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)
            try:
                r = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
            except Exception:
                r = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
            samples.append((float(sm), float(smax), [n for b, n in bits.items() if r & b]))
        except Exception:
            pass
        stop.wait(0.02)


def _clock_summary(samples):
    if not samples:
        return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unsampled"]}
    sm = sorted(s[0] for s in samples)
    return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": samples[0][1], "samples": len(samples),
            "reasons": sorted({n for s in samples for n in s[2]})}


def run_reference(args):
    """The oracle as it stands, on host cores, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from oracle import kvpo
    from paper_2508_13231_b200 import workloads as wl
    kvpo.build()
    cfg = wl.CONFIGS[WORKLOAD]
    tp = wl.trace_params(WORKLOAD, seed=0)
    sample_chains = 8
    U = wl.units(cfg)

    def step(seed):
        A = kvpo.trace_generate(**dict(tp, seed=seed))
        o = kvpo.Problem(U, cfg["bytes_per_unit"], cfg["steps"], A, cfg["cap"], *cfg["bw"])
        for P in wl.random_schedules(U, cfg["steps"], cfg["cap"], 2, seed=seed):
            o.eval(P)
        ap = o.make_params(chains=sample_chains, moves=cfg["moves"], seed=seed, p0=cfg["p0"])
        res, _, _ = o.anneal_chains(ap, 0, sample_chains)
        return sum(r.moves_done for r in res)

    for w in range(args.warmup):
        step(1000 + w)
    t0 = time.perf_counter()
    moves = 0
    for k in range(args.steps):
        moves += step(k)
    dt = time.perf_counter() - t0
    value = moves / dt
    sample = (f"{sample_chains} of {cfg['chains']} chains x {cfg['moves']} moves per step (plus the full trace, "
              f"problem set-up and 2 schedule evaluations), single thread")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1000 * dt / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int32/uint64 ticks", "data": "synthetic",
        "config": {"workload": WORKLOAD, "chains": sample_chains, "moves": cfg["moves"]},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(cfg, tp):
    """Oracle timed on this machine's host: a bounded sample of the benchmark workload, one thread."""
    from oracle import kvpo
    from paper_2508_13231_b200 import workloads as wl
    kvpo.build()
    sample_chains = 768
    t0 = time.perf_counter()
    A = kvpo.trace_generate(**tp)
    o = kvpo.Problem(wl.units(cfg), cfg["bytes_per_unit"], cfg["steps"], A, cfg["cap"], *cfg["bw"])
    ap = o.make_params(chains=sample_chains, moves=cfg["moves"], seed=0, p0=cfg["p0"])
    res, _, _ = o.anneal_chains(ap, 0, sample_chains)
    dt = time.perf_counter() - t0
    return {"value": sum(r.moves_done for r in res) / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"chains 0..{sample_chains - 1} of {cfg['chains']}, all {cfg['moves']} moves each, plus trace "
                      f"and set-up; {dt:.1f} s on one thread"}


def run_cost_kernel(args):
    """The cost kernel alone (Eq. 1-5 over a batch of schedules) on the rows of the largest configuration: HBM roofline.

    A batch of schedules of long_70b (81,920 words per row, 64 rows, 20 MB each) is scored by kvp_eval; the
    batch plus the access bitmap is larger than L2. Algorithmic bytes: every placement word once and the access
    bitmap once per batch (it stays in L2 across the batch), (n + 1) * S * W32 * 4.
    """
    import numpy as np
    import torch
    from paper_2508_13231_b200 import kvp, workloads as wl
    torch.cuda.set_device(0)
    name, n = "long_70b", 96
    cfg = wl.CONFIGS[name]
    tp = wl.trace_params(name, seed=0)
    U, S, W32 = wl.units(cfg), cfg["steps"], wl.words_per_row(cfg)
    A = kvp.trace_generate(**{k: v for k, v in tp.items() if k != "base"}, base=None)
    prob = kvp.Problem(U, cfg["bytes_per_unit"], S, A, cfg["cap"], *cfg["bw"])
    g = torch.Generator(device="cuda"); g.manual_seed(1)
    # random words thinned to ~6% density (three ANDed draws halve it each time; 1/8 would exceed the capacity check,
    # which only sets a flag and costs nothing)
    sched = torch.randint(-2 ** 31, 2 ** 31 - 1, (n, S, W32), dtype=torch.int32, device="cuda", generator=g)
    for _ in range(3):
        sched &= torch.randint(-2 ** 31, 2 ** 31 - 1, (n, S, W32), dtype=torch.int32, device="cuda", generator=g)
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    for _ in range(max(3, args.warmup)):
        prob.eval(sched, want_steps=False, want_seconds=False)
    torch.cuda.synchronize()
    total_ms = 0.0
    for k in range(args.steps):
        flush.fill_(k & 255)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        prob.eval(sched, want_steps=False, want_seconds=False)
        e1.record(stream)
        torch.cuda.synchronize()
        total_ms += e0.elapsed_time(e1)
    ms = total_ms / args.steps
    alg_bytes = (n + 1) * S * W32 * 4
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak, src = (peaks["hbm_gbs"], "measured copy bandwidth (MEASURED_PEAKS.json)") if "hbm_gbs" in peaks else \
        (6650.0, "fallback 6.65 TB/s")
    achieved = alg_bytes / (ms * 1e-3) / 1e9
    print(json.dumps({
        "kernel": "count_wide_kernel+finish_kernel (kvp_eval)", "metric": "schedules_scored_per_sec",
        "value": n / (ms * 1e-3), "unit": "schedules/s", "ms_per_call": ms, "steps": args.steps,
        "config": {"workload": name, "batch": n, "words_per_row": W32, "rows": S,
                   "l2": "flushed with a 256 MB write between timed iterations"},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "algorithmic_bytes": alg_bytes, "peak_source": src}}))


# Algorithmic thread instructions of the trace kernels per (unit, step): one Philox4x32-10 for the noise (10 rounds
# of two wide multiplies, four xors and two key additions: 60 with 3-input logic ops), the 8-term Irwin-Hall sum
# and the AR(1) update 22, a second Philox and a compare for the burst draw 62 when bursts are on, and the top-k
# search: the range reduction (2), three histogram passes of a prefix compare, a digit and a shared-memory add per
# unit (12) and the selection compares (4): 18.
# Multiplier pipe: 148 SMs x 4 schedulers x 1.965 GHz, a warp-wide 32 x 32 -> 64 bit multiply every four cycles
# (measured: ncu's pipe-busy cycles of the score pass divided by its multiply instructions) = 9.3e12 multiplies/s.
WIDE_MUL_PEAK_T = 148 * 4 * 1.965e9 / 4 * 32 / 1e12


def trace_alg_thread_instr(bursts):
    return 60 + 22 + (62 if bursts else 0) + 18


def run_trace_kernel(args):
    """The trace kernel alone (synthetic access sets) on the largest configuration: plain-ALU (issue-slot) roofline.

    long_70b: 640 groups of 4096 units, 64 steps, k = 205, bursts on; two passes (scores by a thread per unit, then one
    selection per group and step). Besides the issue-slot roofline the line gives the rate of 32 x 32 -> 64 bit
    multiplies (20 per Philox block, 2 in the AR(1) update) against the multiplier pipe: the score pass keeps that
    pipe 90% busy, a wide multiply occupying a scheduler's pipe for four cycles per warp (both from ncu). Memory traffic: the int32 score matrix written once and read once (2 * U * S * 4 = 1.3 GB) and
    the output (S * W32 * 4 = 21 MB), reported as GB/s beside the instruction rate.
    """
    import torch
    from paper_2508_13231_b200 import kvp, workloads as wl
    torch.cuda.set_device(0)
    name = "long_70b"
    cfg = wl.CONFIGS[name]
    tp = wl.trace_params(name, seed=0)
    U, S, W32 = wl.units(cfg), cfg["steps"], wl.words_per_row(cfg)
    base = torch.from_numpy(tp["base"]).cuda() if tp["base"] is not None else None
    targs = {k: v for k, v in tp.items() if k not in ("base", "seed")}
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    for w in range(max(3, args.warmup)):
        kvp.trace_generate(**targs, seed=100 + w, base=base)
    torch.cuda.synchronize()
    total_ms = 0.0
    for k in range(args.steps):
        flush.fill_(k & 255)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        kvp.trace_generate(**targs, seed=k, base=base)
        e1.record(stream)
        torch.cuda.synchronize()
        total_ms += e0.elapsed_time(e1)
    ms = total_ms / args.steps
    alg = trace_alg_thread_instr(bool(tp.get("burst_thr"))) / 32.0 * U * S           # warp instructions
    wide = 42 if tp.get("burst_thr") else 22                                         # 32 x 32 -> 64 bit multiplies per (unit, step)
    achieved = alg / (ms * 1e-3) / 1e9
    print(json.dumps({
        "kernel": "trace_scores_unit_kernel + trace_select_kernel (kvp_trace_generate)", "metric": "unit_steps_per_sec", "value": U * S / (ms * 1e-3),
        "unit": "unit-steps/s", "ms_per_call": ms, "steps": args.steps,
        "config": {"workload": name, "groups": cfg["groups"], "units_per_group": cfg["units_per_group"], "rows": S,
                   "topk": cfg["topk"], "l2": "flushed with a 256 MB write between timed iterations"},
        "roofline": {"bound": "alu", "achieved": achieved, "peak": ISSUE_PEAK_GWIPS, "unit": "Gwarp-inst/s",
                     "frac": achieved / ISSUE_PEAK_GWIPS, "traffic": None,
                     "peak_source": "148 SMs x 4 issue slots x 1.965 GHz (unit counts and clocks)",
                     "wide_multiplies": {"achieved": wide * U * S / (ms * 1e-3) / 1e12, "peak": WIDE_MUL_PEAK_T,
                                         "unit": "T multiplies/s", "frac": wide * U * S / (ms * 1e-3) / 1e12 / WIDE_MUL_PEAK_T,
                                         "per_unit_step": wide},
                     "memory_gbs": (2 * U * S * 4 + S * W32 * 4 + (U * 4 if base is not None else 0)) / (ms * 1e-3) / 1e9}}))


def run_growing(args):
    """The whole path on a growing cache with (token, layer) steps (Section III-A), configuration growing_8b:
    layered trace with births -> kvp_create + kvp_set_births -> kvp_eval of 4 schedules -> kvp_anneal.

    The chains' schedules (17 MB each) live in global memory; the oracle is timed on a few chains beside it.
    """
    import numpy as np
    import torch
    from paper_2508_13231_b200 import kvp, workloads as wl
    torch.cuda.set_device(0)
    name = "growing_8b"
    cfg = wl.GROWING[name]
    groups, U, S = wl.growing_shape(cfg)
    birth_np = wl.growing_births(cfg)
    birth = torch.from_numpy(birth_np.view(np.int32)).cuda()
    tp = wl.growing_trace_params(name, seed=0)
    base = torch.from_numpy(tp["base"]).cuda()
    targs = {k: v for k, v in tp.items() if k not in ("base", "seed")}
    chains, moves = cfg["chains"], cfg["moves"]
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    g = torch.Generator(device="cuda"); g.manual_seed(3)
    w32 = (U + 31) // 32
    scheds = torch.randint(-2 ** 31, 2 ** 31 - 1, (4, S, w32), dtype=torch.int32, device="cuda", generator=g)
    for _ in range(3):                                        # ~6% density, below the capacity
        scheds &= torch.randint(-2 ** 31, 2 ** 31 - 1, (4, S, w32), dtype=torch.int32, device="cuda", generator=g)

    def step(seed):
        A = kvp.trace_generate(**targs, seed=seed, base=base, layers=cfg["layers"], birth=birth)
        prob = kvp.Problem(U, cfg["bytes_per_unit"], S, A, cfg["cap"], *cfg["bw"], birth=birth)
        prob.eval(scheds, want_steps=False)
        out = prob.anneal(prob.make_params(chains=chains, moves=moves, seed=seed, p0=cfg["p0"]), want_schedule=False)
        prob.close()
        return out

    for w in range(max(3, args.warmup)):
        step(1000 + w)
    torch.cuda.synchronize()
    total_ms = chain_ms = 0.0
    for k in range(args.steps):
        flush.fill_(k & 255)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        out = step(k)
        e1.record(stream)
        torch.cuda.synchronize()
        total_ms += e0.elapsed_time(e1)
        chain_ms += out["stats"].ms_chains
    ms, cms = total_ms / args.steps, chain_ms / args.steps
    achieved = ALG_WARP_INSTR_PER_MOVE * chains * moves / (cms * 1e-3) / 1e9
    line = {"metric": METRIC, "value": chains * moves / (ms * 1e-3), "unit": UNIT, "ms_per_step": ms, "steps": args.steps,
            "config": {"workload": name, "units": U, "steps": S, "layers": cfg["layers"], "chains": chains, "moves": moves,
                       "p0": cfg["p0"], "l2": "flushed with a 256 MB write between timed iterations"},
            "roofline": {"bound": "alu", "kernel": "chain_kernel<global, growing>", "achieved": achieved,
                         "peak": ISSUE_PEAK_GWIPS, "unit": "Gwarp-inst/s", "frac": achieved / ISSUE_PEAK_GWIPS,
                         "traffic": None, "ms_per_launch": cms,
                         "peak_source": "148 SMs x 4 issue slots x 1.965 GHz (unit counts and clocks)"},
            "anneal_ms": {"init": out["stats"].ms_init, "chains": out["stats"].ms_chains, "finish": out["stats"].ms_finish},
            "bound_ticks": out["best_ticks"], "init_ticks": out["stats"].init_ticks}
    if not args.no_cpu_baseline:
        from oracle import kvpo
        t0 = time.perf_counter()
        A = kvpo.trace_generate(**targs, seed=0, base=tp["base"], layers=cfg["layers"], birth=birth_np)
        o = kvpo.Problem(U, cfg["bytes_per_unit"], S, A, cfg["cap"], *cfg["bw"], birth=birth_np)
        n = 2
        res, _, _ = o.anneal_chains(o.make_params(chains=chains, moves=moves, seed=0, p0=cfg["p0"]), 0, n)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": sum(r.moves_done for r in res) / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": f"chains 0..{n - 1} of {chains}, all {moves} moves each, plus trace and "
                                          f"set-up; {dt:.1f} s on one thread"}
    print(json.dumps(line))


def time_to_bound(kvp, cfg, targs, base_dev, U, S):
    """Outside the timed region: wall time of kvp_anneal (all of its kernels, warm) to reach the bound.

    full: the whole budget, the stop rule off. early_stop: the same call with the paper's rule on (a chain stops at
    a level boundary when its best improved by less than 0.1% since the previous one). smallest_budget: the smallest
    of moves/16, /8, /4, /2, moves whose bound is within 0.1% of the full-budget bound, and its wall time.
    """
    import torch
    A = kvp.trace_generate(**targs, seed=0, base=base_dev)
    prob = kvp.Problem(U, cfg["bytes_per_unit"], S, A, cfg["cap"], *cfg["bw"])

    def run(moves, permille=0):
        prm = prob.make_params(chains=cfg["chains"], moves=moves, seed=0, p0=cfg["p0"], early_stop_permille=permille)
        prob.anneal(prm, want_schedule=False)                       # warm
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        out = prob.anneal(prm, want_schedule=False)
        torch.cuda.synchronize()
        return out["best_ticks"], 1e3 * (time.perf_counter() - t0), out["stats"].moves_total

    full_ticks, full_ms, _ = run(cfg["moves"])
    es_ticks, es_ms, es_moves = run(cfg["moves"], permille=1)
    res = {"full_budget": {"moves_per_chain": cfg["moves"], "bound_ticks": full_ticks, "ms": full_ms},
           "early_stop_0.1pct": {"bound_ticks": es_ticks, "ms": es_ms, "moves_executed": es_moves}}
    for div in (16, 8, 4, 2, 1):
        ticks, ms, _ = run(cfg["moves"] // div)
        if (ticks - full_ticks) * 1000 <= full_ticks:
            res["smallest_budget_within_0.1pct"] = {"moves_per_chain": cfg["moves"] // div, "bound_ticks": ticks, "ms": ms}
            break
    prob.close()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="kvp", choices=["kvp", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel", default="path", choices=["path", "cost", "trace", "growing"],
                    help="path: the whole hot path (the benchmark line); cost / trace: that kernel alone on full-size rows; "
                         "growing: the whole path on a growing cache with (token, layer) steps")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.kernel == "cost":
        return run_cost_kernel(args)
    if args.kernel == "trace":
        return run_trace_kernel(args)
    if args.kernel == "growing":
        return run_growing(args)

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2508_13231_b200 import kvp, sharding, workloads as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    cfg = wl.CONFIGS[WORKLOAD]
    tp = wl.trace_params(WORKLOAD, seed=0)
    U, S = wl.units(cfg), cfg["steps"]
    chains, moves = cfg["chains"], cfg["moves"]
    n_eval = 8
    scheds_host = torch.from_numpy(wl.random_schedules(U, S, cfg["cap"], n_eval, seed=5).view(np.int32)).pin_memory()
    base_host = torch.from_numpy(tp["base"]).pin_memory()
    targs = {k: v for k, v in tp.items() if k not in ("base", "seed")}
    stream = torch.cuda.current_stream()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")     # > 126 MB L2
    launches = [0]

    def step(seed, base_dev, scheds_dev):
        """One pass of the hot path. Returns (best_ticks, stats, best_schedule)."""
        A = kvp.trace_generate(**targs, seed=seed, base=base_dev)
        prob = kvp.Problem(U, cfg["bytes_per_unit"], S, A, cfg["cap"], *cfg["bw"])
        prob.eval(scheds_dev, want_steps=False)
        first, count = sharding.chain_range(rank, world, world * chains)
        prm = prob.make_params(chains=count, moves=moves, seed=seed, p0=cfg["p0"], first_chain=first)
        out = prob.anneal(prm)
        # kernels: 2 trace (scores, select) + 6 create (clean, popcount, transpose, unit counts, histogram,
        #          static row) + 2 eval (count, finish) + those kvp_anneal reports
        launches[0] = 2 + 6 + 2 + out["stats"].kernel_launches
        prob.close()
        return out

    def timed(n_steps, e2e):
        total_ms, chain_ms, last = 0.0, 0.0, None
        for k in range(n_steps):
            flush.fill_(k & 255)                                   # evict L2 between timed iterations
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            if e2e:
                b = base_host.to("cuda", non_blocking=True)
                sc = scheds_host.to("cuda", non_blocking=True)
                out = step(k, b, sc)
                sched_host = out["best_schedule"].to("cpu")         # device -> host read of the result
                last = (out, sched_host)
            else:
                out = step(k, base_dev, scheds_dev)
                last = (out, None)
            e1.record(stream)
            torch.cuda.synchronize()
            total_ms += e0.elapsed_time(e1)
            chain_ms += out["stats"].ms_chains
        return total_ms, chain_ms, last

    base_dev = base_host.to("cuda")
    scheds_dev = scheds_host.to("cuda")
    for w in range(max(3, args.warmup)):
        step(1000 + w, base_dev, scheds_dev)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x):
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    samples, stop = [], threading.Event()
    th = threading.Thread(target=_clock_sampler, args=(stop, samples), daemon=True)
    th.start()
    barrier()
    total_ms, chain_ms, (out, _) = timed(args.steps, e2e=False)
    barrier()
    stop.set(); th.join()
    total_ms = max_over_ranks(total_ms)
    # the cross-rank part of the reduction: two 8-byte MIN reductions over (ticks, chain)
    if world > 1:
        sharding.combine_best(dist, out["best_ticks"], out["stats"].best_chain, device="cuda")
    barrier()
    e2e_ms, _, (out2, sched_host) = timed(args.steps, e2e=True)
    barrier()
    e2e_ms = max_over_ranks(e2e_ms)

    if rank == 0:
        work = float(world) * chains * moves * args.steps
        value = work / (total_ms * 1e-3)
        per_launch_ms = chain_ms / args.steps
        achieved = ALG_WARP_INSTR_PER_MOVE * chains * moves / (per_launch_ms * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int32/uint64 ticks", "data": "synthetic",
            "config": {"workload": WORKLOAD, "units": U, "steps": S, "chains_per_gpu": chains, "moves": moves,
                       "p0": cfg["p0"], "l2": "flushed with a 256 MB write between timed iterations",
                       "eval_batch": n_eval},
            "clocks": _clock_summary(samples),
            "e2e": {"value": work / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": base_host.numel() * 4 + scheds_host.numel() * 4,
                    "d2h_bytes_per_step": sched_host.numel() * 4 + 16},
            "gpu_launches": launches[0] * args.steps,
            "roofline": {"bound": "alu", "kernel": "chain_kernel<smem>", "achieved": achieved,
                         "peak": ISSUE_PEAK_GWIPS, "unit": "Gwarp-inst/s", "frac": achieved / ISSUE_PEAK_GWIPS,
                         "traffic": CHAIN_KERNEL_DRAM_BYTES, "ncu": CHAIN_KERNEL_NCU, "ms_per_launch": per_launch_ms,
                         "peak_source": "148 SMs x 4 issue slots x 1.965 GHz (unit counts and clocks)"},
            "bound_ticks": out["best_ticks"], "init_ticks": out["stats"].init_ticks,
        }
        if world == 1:
            line["time_to_bound"] = time_to_bound(kvp, cfg, targs, base_dev, U, S)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(cfg, tp)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
