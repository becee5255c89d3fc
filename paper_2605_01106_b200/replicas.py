"""Host-side logic of running the decode path on several GPUs: independent replicas, no collective on the data path.

Sequences are independent, so N GPUs run N replicas of the library, each with its own weights copy and its own
share of the sequences.  The only communication is for reporting: the slowest rank's device time and the total
number of tokens.  Works with any torch.distributed backend (nccl on GPUs, gloo in the CPU tests)."""
from __future__ import annotations


def shard_range(n_items: int, rank: int, world: int) -> range:
    """Contiguous share of n_items for this rank; shares differ by at most one item and cover 0..n_items-1."""
    if world < 1 or not (0 <= rank < world) or n_items < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(n_items, world)
    start = rank * base + min(rank, extra)
    return range(start, start + base + (1 if rank < extra else 0))


def reduce_max_sum(local_ms: float, local_tokens: float, world: int, device=None):
    """(max over ranks of local_ms, sum over ranks of local_tokens).  world == 1: no communication."""
    if world == 1:
        return float(local_ms), float(local_tokens)
    import torch
    import torch.distributed as dist
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    n = torch.tensor([local_tokens], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


def job_throughput(local_ms: float, local_tokens: float, world: int, device=None) -> float:
    """Whole-job tokens/s: all ranks' tokens over the slowest rank's device time."""
    ms, tokens = reduce_max_sum(local_ms, local_tokens, world, device)
    return tokens / (ms * 1e-3)
