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
    sample_chains = 256
    t0 = time.perf_counter()
    A = kvpo.trace_generate(**tp)
    o = kvpo.Problem(wl.units(cfg), cfg["bytes_per_unit"], cfg["steps"], A, cfg["cap"], *cfg["bw"])
    ap = o.make_params(chains=sample_chains, moves=cfg["moves"], seed=0, p0=cfg["p0"])
    res, _, _ = o.anneal_chains(ap, 0, sample_chains)
    dt = time.perf_counter() - t0
    return {"value": sum(r.moves_done for r in res) / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"chains 0..{sample_chains - 1} of {cfg['chains']}, all {cfg['moves']} moves each, plus trace "
                      f"and set-up; {dt:.1f} s on one thread"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="kvp", choices=["kvp", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2508_13231_b200 import kvp, workloads as wl

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
        prm = prob.make_params(chains=chains, moves=moves, seed=seed, p0=cfg["p0"], first_chain=rank * chains)
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
    # the cross-rank part of the reduction: minimum of (ticks, chain) keys, 8 bytes per rank
    if world > 1:
        key = torch.tensor([(out["best_ticks"] << 21) | out["stats"].best_chain], dtype=torch.int64, device="cuda")
        dist.all_reduce(key, op=dist.ReduceOp.MIN)
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
                         "traffic": None, "ms_per_launch": per_launch_ms,
                         "peak_source": "148 SMs x 4 issue slots x 1.965 GHz (unit counts and clocks)"},
            "bound_ticks": out["best_ticks"], "init_ticks": out["stats"].init_ticks,
        }
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(cfg, tp)
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
