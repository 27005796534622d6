"""Data-parallel plumbing: which batch a rank works on and how per-rank timings are combined.

The path shards by batch (every rank runs the whole step on its own prompts; nothing is exchanged
on the data path), so the only communication is the reduction of timings and token counts for
reporting.  Works with any torch.distributed backend (NCCL on GPUs, gloo in the CPU tests).
"""
import torch
import torch.distributed as dist


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch that `rank` processes: ranks draw disjoint batches."""
    return int(base_seed) + int(rank)


def combine_over_ranks(times_ms, tokens, device="cpu"):
    """times_ms: this rank's timings (list of floats); tokens: valid tokens this rank processed per step.
    Returns (max over ranks of each timing, sum over ranks of tokens).  A single process needs no group."""
    t = torch.tensor([float(x) for x in times_ms], dtype=torch.float64, device=device)
    n = torch.tensor([float(tokens)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], float(n.item())


def throughput(tokens_all_ranks: float, ms_per_step: float) -> float:
    """Whole-job valid tokens per second."""
    return tokens_all_ranks / (ms_per_step / 1e3)
