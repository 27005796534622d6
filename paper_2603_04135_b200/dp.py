"""Data-parallel plumbing: which part of the work a rank takes and how per-rank results are combined.

The path shards in two ways, neither of which exchanges anything while the kernels run:

* by batch (the benchmark): every rank runs the whole step on its own prompts;
* by packed row: the small steps (advantages, pruning, rescaling, packing) are repeated on every rank from the
  same seed, the packed rows of the batch are dealt out in contiguous ranges, and every rank sweeps the logits of
  its own rows.  The loss is a sum over tokens, so the per-rank results combine with one all-reduce of the five
  loss scalars; the fused LM-head adds one all-reduce of dW.

Both collectives are plain torch.distributed calls (NCCL on GPUs, gloo in the CPU tests); nothing here touches
another rank's memory.
"""
import torch
import torch.distributed as dist


def _group_size(group=None):
    if dist.is_available() and dist.is_initialized():
        return dist.get_world_size(group)
    return 1


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the batch that `rank` processes: ranks draw disjoint batches."""
    return int(base_seed) + int(rank)


def combine_over_ranks(times_ms, tokens, device="cpu"):
    """times_ms: this rank's timings (list of floats); tokens: valid tokens this rank processed per step.
    Returns (max over ranks of each timing, sum over ranks of tokens).  A single process needs no group."""
    t = torch.tensor([float(x) for x in times_ms], dtype=torch.float64, device=device)
    n = torch.tensor([float(tokens)], dtype=torch.float64, device=device)
    if _group_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], float(n.item())


def throughput(tokens_all_ranks: float, ms_per_step: float) -> float:
    """Whole-job valid tokens per second."""
    return tokens_all_ranks / (ms_per_step / 1e3)


def shard_rows(row_of_placed, cu_seqlens, n_units, world, rank):
    """Contiguous range of packed rows for `rank`, balanced by loss tokens.

    row_of_placed[p] is the row of the unit placed p-th and cu_seqlens the packer's scan of loss tokens in
    placement order (rows are filled one after the other, so a range of rows is a range of placements and a
    range of tokens).  Rows are dealt out greedily: rank r's range ends at the first row boundary at or past
    (r + 1)/world of the tokens.  Returns a dict with the rank's placements [seq_lo, seq_hi), tokens
    [tok_lo, tok_hi) and rows [row_lo, row_hi); a rank can come out empty when there are fewer rows than ranks.
    """
    rows = [int(x) for x in row_of_placed[:n_units]]
    cu = [int(x) for x in cu_seqlens[:n_units + 1]]
    total = cu[n_units] if n_units > 0 else 0
    bounds = [0]                                                   # placement index where each rank's range starts
    p = 0
    for r in range(1, world):
        want = total * r / world
        while p < n_units and (cu[p] < want or (p > 0 and rows[p] == rows[p - 1])):
            p += 1
        bounds.append(max(p, bounds[-1]))
    bounds.append(n_units)
    lo, hi = bounds[rank], bounds[rank + 1]
    row_lo = rows[lo] if lo < n_units else (rows[-1] + 1 if rows else 0)
    row_hi = rows[hi] if hi < n_units else (rows[-1] + 1 if rows else 0)
    return dict(seq_lo=lo, seq_hi=hi, tok_lo=cu[lo] if n_units else 0, tok_hi=cu[hi] if n_units else 0,
                row_lo=row_lo, row_hi=row_hi)


def all_reduce_loss(loss_out, group=None, average=False):
    """Combines the five loss scalars {loss, policy-gradient part, KL part, clipped fraction, T} of all ranks,
    in place, and returns the tensor: the first three are summed, the clipped fraction is weighted by each rank's
    token count, T is summed.

    With the sequence weights of the whole batch on every rank (rows sharded, the small steps repeated from one
    seed) the sum IS the loss of the batch.  With one batch per rank, each normalised by its own prompt count,
    pass average=True: loss, policy-gradient and KL parts are divided by the number of ranks, which is the loss of
    the union of the batches."""
    world = _group_size(group)
    if world == 1:
        return loss_out
    v = loss_out.detach().to(torch.float64).clone()
    v[3] = v[3] * v[4]                                             # clipped tokens
    dist.all_reduce(v, op=dist.ReduceOp.SUM, group=group)
    v[3] = v[3] / v[4] if float(v[4]) > 0 else 0.0
    if average:
        v[:3] /= world
    loss_out.copy_(v.to(loss_out.dtype))
    return loss_out


def reduce_dW(dW, group=None, average=False):
    """Sum (or mean) over ranks of the LM-head weight gradient, in place: the one collective the fused LM-head
    path needs when tokens are sharded (dhidden stays local to the rank that owns the tokens)."""
    world = _group_size(group)
    if world > 1:
        dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=group)
        if average:
            dW /= world
    return dW
