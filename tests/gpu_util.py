"""Helpers shared by the GPU parity tests: numpy <-> torch bitmaps and problem construction on both sides."""
import numpy as np
import torch

from paper_2508_13231_b200 import workloads as wl


def to_dev(a):
    """uint32 numpy bitmap -> int32 CUDA tensor with the same bits."""
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.uint32).view(np.int32)).cuda()


def to_np(t):
    """int32 tensor with uint32 bit patterns -> uint32 numpy array."""
    return t.detach().cpu().numpy().view(np.uint32)


def u64(t):
    return t.detach().cpu().numpy().view(np.uint64)


def both_problems(kvp, oracle, U, bpu, S, A, cap, bw, mig_flags=3, hw=None, ew=None):
    """The same instance on the CUDA library and on the oracle."""
    g = kvp.Problem(U, bpu, S, to_dev(A), cap, bw[0], bw[1], bw[2], mig_flags=mig_flags, hw=hw, ew=ew)
    o = oracle.Problem(U, bpu, S, A, cap, bw[0], bw[1], bw[2], mig_flags=mig_flags, hw=hw, ew=ew)
    return g, o


def trace_on_gpu(kvp, tp, flags=0):
    base = None if tp["base"] is None else torch.from_numpy(tp["base"]).cuda()
    args = {k: v for k, v in tp.items() if k != "base"}
    return kvp.trace_generate(**args, base=base, flags=flags)


def named_problem(kvp, oracle, name, A=None, seed=0):
    """Named configuration on both sides; A defaults to the oracle's trace."""
    cfg = wl.CONFIGS[name]
    if A is None:
        A = oracle.trace_generate(**wl.trace_params(name, seed))
    U = wl.units(cfg)
    return both_problems(kvp, oracle, U, cfg["bytes_per_unit"], cfg["steps"], A, cfg["cap"], cfg["bw"]) + (cfg, A)
