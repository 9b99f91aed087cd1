"""Splitting a job over ranks: chains are independent, so each rank runs a contiguous range of chain
indices (`first_chain`, `chains` of the anneal parameters) and the ranks agree on the winner with two
8-byte MIN reductions. No other data crosses ranks. Works on any torch.distributed backend.
A replica-exchange job is split by whole ladders: the exchange step stays inside a ladder, hence inside a rank."""
import torch


def chain_range(rank, world, total_chains):
    """Contiguous, balanced split of chain indices 0..total_chains-1 -> (first_chain, count) of `rank`."""
    base, extra = divmod(total_chains, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def ladder_range(rank, world, total_chains, rungs):
    """Split of a replica-exchange job: whole ladders of `rungs` chains per rank (ladders exchange only among their own
    chains, so they are independent units) -> (first_chain, count) of `rank`, both multiples of `rungs`."""
    if total_chains % rungs:
        raise ValueError("the chains of a replica-exchange job come in whole ladders")
    first, count = chain_range(rank, world, total_chains // rungs)
    return first * rungs, count * rungs


def combine_best(dist, best_ticks, best_chain, device="cpu"):
    """Global (lowest ticks, lowest chain index among those) over all ranks -> (ticks, chain)."""
    t = torch.tensor([best_ticks], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MIN)
    gt = int(t.item())
    c = torch.tensor([best_chain if best_ticks == gt else 2 ** 62], dtype=torch.int64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.MIN)
    return gt, int(c.item())
