"""Synthetic reruns of the paper's sensitivity study (Section IV-B, Fig. 3-5) on one B200.

    python -m paper_2508_13231_b200.figures [--quick]

One attention head at token granularity: 4096 tokens (512 B of K+V each), 512 decode steps, HBM room for 25% of
them, 8 TB/s HBM against 0.9 TB/s off-package, Zipf(1.1) importance with AR(1) drift. The recorded LLaMA-3.1-8B /
LongBench traces of the paper are not available; these traces are synthetic, so the numbers show the same trends,
not the paper's values. Strategies (Section IV-A): Unlimited HBM, Static Placement (first come), Reactive (LRU),
Page granularity (16 tokens), SA-guided = the paper's annealer over the look-ahead policy's (W, R), followed by
direct annealing of the schedule it found. Everything runs in the library's kernels; this file only calls them.
"""
import argparse

import numpy as np
import torch

from . import kvp, workloads as wl

TOKENS, STEPS, CAP, BPU = 4096, 512, 1024, 512
BW = (8 * wl.TB, 9 * wl.TB // 10, 9 * wl.TB // 10)


def strategies(topk, rho, quick=False, seed=0):
    """-> dict name -> (total ticks, HBM hit rate)."""
    tp = wl.custom_trace_params(1, TOKENS, STEPS, topk, rho, zipf=(1.1, 1.1), seed=seed)
    base = torch.from_numpy(tp["base"]).cuda()
    A = kvp.trace_generate(**{k: v for k, v in tp.items() if k != "base"}, base=base)
    prob = kvp.Problem(TOKENS, BPU, STEPS, A, CAP, *BW)
    unlimited = kvp.Problem(TOKENS, BPU, STEPS, A, TOKENS, *BW)
    accessed = STEPS * topk

    def score(p, sched):
        ticks = int(p.eval(sched, want_steps=False, want_seconds=False)["total_ticks"][0])
        hits = int(p.eval_counts(sched)[0, :, 0].sum())
        return ticks, hits / accessed

    out = {}
    ones = torch.full((STEPS, TOKENS // 32), -1, dtype=torch.int32, device="cuda")
    out["unlimited"] = score(unlimited, ones)
    static = prob.policy_lookahead([1], [0])[0].contiguous()              # R = 0: first-come placement, no migration
    out["static"] = score(prob, static)
    out["reactive"] = score(prob, prob.policy_reactive())
    out["page16"] = score(prob, prob.policy_page(16))
    w_max = 16 if quick else 64
    table = prob.wr_grid(w_max, 11)
    _, best = kvp.wr_anneal(table, kvp.wr_params(chains=64, iters=2000, seed=seed, levels=32, early_stop_permille=1))
    look = prob.policy_lookahead([best.best_w], [100 * best.best_r])[0].contiguous()
    out["lookahead_sa"] = score(prob, look) + ((best.best_w, best.best_r / 10),)
    prm = prob.make_params(chains=64 if quick else 256, moves=50_000 if quick else 400_000, seed=seed, p0=1e-3,
                           init_mode=kvp.INIT_USER, init_schedule=look)
    res = prob.anneal(prm)
    out["sa_guided"] = score(prob, res["best_schedule"])
    prob.close(); unlimited.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true")
    args = ap.parse_args()
    names = ["unlimited", "static", "reactive", "page16", "lookahead_sa", "sa_guided"]
    print("Fig. 3 analogue: tokens/s normalised to Static Placement (rho = 0.95)\n")
    print("| sparsity | " + " | ".join(names) + " | best (W, R) |")
    print("|---|" + "---|" * (len(names) + 1))
    keep = {}
    for sparsity in (50, 60, 70, 80, 90, 95):
        topk = TOKENS * (100 - sparsity) // 100
        r = strategies(topk, 0.95, args.quick)
        keep[sparsity] = r
        print(f"| {sparsity}% | " + " | ".join(f"{r['static'][0] / r[n][0]:.2f}" for n in names) +
              f" | {r['lookahead_sa'][2]} |")
    print("\nFig. 4 analogue: tokens/s normalised to Unlimited HBM at 60% sparsity\n")
    print("| variation | " + " | ".join(names[1:]) + " |")
    print("|---|" + "---|" * (len(names) - 1))
    for label, rho in (("low (rho 0.99)", 0.99), ("high (rho 0.5)", 0.5)):
        r = strategies(TOKENS * 40 // 100, rho, args.quick)
        print(f"| {label} | " + " | ".join(f"{r['unlimited'][0] / r[n][0]:.2f}" for n in names[1:]) + " |")
    print("\nFig. 5 analogue: HBM hit rate at 60% sparsity (rho = 0.95)\n")
    r = keep[60]
    print("| " + " | ".join(names[1:]) + " |")
    print("|" + "---|" * (len(names) - 1))
    print("| " + " | ".join(f"{r[n][1]:.3f}" for n in names[1:]) + " |")


if __name__ == "__main__":
    main()
