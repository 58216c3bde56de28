"""Host logic for running the path on several GPUs (one process per GPU).

EGAE and the token filter are independent per sequence and the two losses per token, so a batch is
split by sequence and every rank runs the same four calls on its own packed slice.  The only
coupling is the token-level mean of Eq. 1 and of the value loss (Section 4.1.1 of the paper trains
on a token-level loss): every rank must divide by the number of selected tokens of the WHOLE batch.
That takes one all-reduce of two integers before the loss calls (the result is passed as `denom`)
and one all-reduce of the scalar losses after them; the gradients need no exchange here because
they are per token.

The LM-head variant can instead be split by vocabulary (every rank holds a column shard of the
weight and all rows): `combine_row_stats` is the exchange between its two calls.  No arithmetic of
the method lives in this file; the one arithmetic step of that exchange is passed in as a callable.
"""
from __future__ import annotations

import numpy as np
import torch

PER_SEQUENCE = ("prompt_len", "prev_len", "new_len", "truncated", "bootstrap")
PER_TOKEN = ("rewards", "values", "old_values", "targets", "old_logp_noise", "extra_policy_mask",
             "extra_value_mask", "logits")


def partition_sequences(tokens_per_sequence, world: int):
    """Contiguous ranges [lo, hi) of sequence indices, one per rank, balanced by token count.

    Contiguous so that a rank's slice of the packed arrays is one interval.  Every sequence lands on
    exactly one rank; ranks may get an empty range when there are fewer sequences than ranks."""
    t = np.asarray(tokens_per_sequence, np.int64)
    B = len(t)
    csum = np.concatenate([[0], np.cumsum(t)])
    total = int(csum[-1])
    cuts = [0]
    for r in range(1, world):
        target = total * r / world
        k = int(np.searchsorted(csum, target, side="left"))       # first boundary at or past the target
        if k > 0 and abs(csum[k - 1] - target) <= abs(csum[min(k, B)] - target):
            k -= 1
        cuts.append(min(max(k, cuts[-1]), B))
    cuts.append(B)
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def shard_batch(c: dict, lo: int, hi: int) -> dict:
    """The packed batch `c` (as made by `synth`) restricted to sequences lo..hi-1, offsets re-based."""
    sb = np.asarray(c["seq_begin"], np.int64)
    p0, p1 = int(sb[lo]), int(sb[hi])
    out = {k: v for k, v in c.items() if k not in PER_SEQUENCE + PER_TOKEN
           and k not in ("seq_begin", "seg_begin", "seg_end", "B", "N")}
    out["B"], out["N"] = hi - lo, p1 - p0
    out["token_offset"] = p0
    out["seq_begin"] = (sb[lo:hi + 1] - p0).astype(np.int32)
    out["seg_begin"] = (np.asarray(c["seg_begin"], np.int64)[lo:hi] - p0).astype(np.int32)
    out["seg_end"] = (np.asarray(c["seg_end"], np.int64)[lo:hi] - p0).astype(np.int32)
    for k in PER_SEQUENCE:
        if k in c:
            out[k] = None if c[k] is None else c[k][lo:hi]
    for k in PER_TOKEN:
        if k in c:
            out[k] = None if c[k] is None else c[k][p0:p1]
    return out


def global_token_counts(n_policy: int, n_value: int, group=None, device="cpu"):
    """Sum of the ranks' selected-token counts: the `denom` every rank passes to the two loss calls."""
    import torch.distributed as dist
    t = torch.tensor([int(n_policy), int(n_value)], dtype=torch.int64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return int(t[0]), int(t[1])


def reduce_losses(policy_loss: float, value_loss: float, group=None, device="cpu"):
    """Whole-batch losses from the ranks' partial ones (each already divided by the global count)."""
    import torch.distributed as dist
    t = torch.tensor([float(policy_loss), float(value_loss)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return float(t[0]), float(t[1])


def combine_row_stats(row_max, row_sumexp, row_target_logit, rescale, group=None):
    """Whole-vocabulary row statistics from each rank's shard statistics, in place.

    row_max, row_sumexp, row_target_logit: this rank's [M] float32 tensors (maximum logit, sum of
    exponentials relative to it, target logit or 0) over its vocabulary shard.  `rescale(row_max,
    row_max_all, row_sumexp)` multiplies row_sumexp by exp(row_max - row_max_all) in place (on a GPU:
    `binding.tppo_lmhead_shard_rescale`).  Afterwards all three hold the whole-vocabulary values on
    every rank.  Two all-reduces' worth of traffic: 4 bytes x M for the maximum, 8 bytes x M for the sums.
    """
    import torch.distributed as dist
    multi = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1
    if not multi:
        return row_max, row_sumexp, row_target_logit
    row_max_all = row_max.clone()
    dist.all_reduce(row_max_all, op=dist.ReduceOp.MAX, group=group)
    rescale(row_max, row_max_all, row_sumexp)
    sums = torch.stack([row_sumexp, row_target_logit])
    dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)
    row_max.copy_(row_max_all)
    row_sumexp.copy_(sums[0])
    row_target_logit.copy_(sums[1])
    return row_max, row_sumexp, row_target_logit


def vocab_shard_bounds(V: int, world: int, align: int = 8):
    """Column ranges [lo, hi) of the LM-head weight, one per rank: equal widths rounded up to
    `align` columns (the GEMM kernels want multiples of 8), the last rank taking what is left."""
    width = (-(-V // world) + align - 1) // align * align
    cuts = [min(r * width, V) for r in range(world)] + [V]
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def vocab_parallel_step(stats_fn, rescale_fn, grads_fn, group=None):
    """One step of the vocabulary-parallel LM-head on this rank; every collective it needs is here.

    stats_fn() -> (row_max, row_sumexp, row_target_logit): this rank's [M] float32 statistics over its
        column shard (on a GPU: `binding.tppo_lmhead_shard_stats`).
    rescale_fn(row_max, row_max_all, row_sumexp): see `combine_row_stats`.
    grads_fn(row_max, row_sumexp, row_target_logit) -> dhidden_partial or None: loss and gradients
        from the whole-vocabulary statistics (`binding.tppo_lmhead_shard_fwd_bwd`); the [M, K] tensor
        it returns holds this shard's term of dX * W^T.
    The returned tensor is the complete dhidden (the partial terms summed over the ranks, in place).
    Traffic per rank: 12 bytes x M for the statistics and one all-reduce of M x K gradient elements.
    No rank reads another rank's memory; the collectives are torch.distributed's (NCCL on GPUs).
    """
    import torch.distributed as dist
    row_max, row_sumexp, row_target_logit = stats_fn()
    combine_row_stats(row_max, row_sumexp, row_target_logit, rescale_fn, group=group)
    dhidden = grads_fn(row_max, row_sumexp, row_target_logit)
    multi = dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1
    if dhidden is not None and multi:
        dist.all_reduce(dhidden, op=dist.ReduceOp.SUM, group=group)
    return dhidden
