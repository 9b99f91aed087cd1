"""Splitting a job over ranks: chains are independent, so each rank runs a contiguous range of chain
indices (`first_chain`, `chains` of the anneal parameters) and the ranks agree on the winner with two
8-byte MIN reductions. No other data crosses ranks. Works on any torch.distributed backend."""
import torch


def chain_range(rank, world, total_chains):
    """Contiguous, balanced split of chain indices 0..total_chains-1 -> (first_chain, count) of `rank`."""
    base, extra = divmod(total_chains, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def combine_best(dist, best_ticks, best_chain, device="cpu"):
    """Global (lowest ticks, lowest chain index among those) over all ranks -> (ticks, chain)."""
    t = torch.tensor([best_ticks], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MIN)
    gt = int(t.item())
    c = torch.tensor([best_chain if best_ticks == gt else 2 ** 62], dtype=torch.int64, device=device)
    dist.all_reduce(c, op=dist.ReduceOp.MIN)
    return gt, int(c.item())
