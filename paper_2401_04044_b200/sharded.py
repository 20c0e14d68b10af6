"""Calibration over a token set that is spread over batches, layers and ranks (Section 4.2: the scores
come from a pass over a small calibration set; Eq. 3 is a sum over tokens, so it can be taken in pieces).

Host-side control flow only -- every number is produced by the callables handed in (in production the
library's entry points: ffsplit_score with scores = NULL to accumulate, ffsplit_forward to produce the next
layer's input, ffsplit_score_finalize to form the scores), which is also what lets the flow be exercised
on CPU ranks with any other scorer.

  * token sharding: every rank accumulates the energy e_j = sum_t sigma(x_t U_j)^2 of its own tokens; ONE
    all-reduce (sum) of the float32 vector e [m] per layer then gives every rank the same total, and every
    rank forms the same scores and runs the same deterministic top-k -- no index exchange is needed;
  * streaming over layers: a calibration batch is pushed through the stack once, layer l scoring the
    activations that layer l - 1 produced for that batch, so that no layer's inputs are ever stored.
"""
from __future__ import annotations

from typing import Callable, Iterable, List, Optional, Sequence

import torch
import torch.distributed as dist


def shard_bounds(n_tokens: int, world: int, rank: int):
    """Contiguous, near-equal shares: rank r takes tokens [lo, hi)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    return n_tokens * rank // world, n_tokens * (rank + 1) // world


def batches(lo: int, hi: int, batch: int):
    """[lo, hi) cut into pieces of at most `batch` tokens."""
    if batch < 1:
        raise ValueError("batch must be >= 1")
    return [(a, min(a + batch, hi)) for a in range(lo, hi, batch)]


def all_reduce_energy(energy: torch.Tensor, group=None):
    """Sum of the per-rank energy vectors, in place, the same bits on every rank afterwards.  One collective of
    m float32 values (80 KB at m = 20480): latency-bound, so it is issued once per layer, after the last batch."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(energy, op=dist.ReduceOp.SUM, group=group)
    return energy


def score_token_sharded(score_batch: Callable[[int, int, bool], None], finalize: Callable[[], None],
                        energy: torch.Tensor, n_tokens: int, batch: int, group=None,
                        rank: Optional[int] = None, world: Optional[int] = None):
    """Scores of one layer from a calibration set of `n_tokens` tokens spread over the ranks of `group`.

    score_batch(lo, hi, accumulate) adds the energy of tokens [lo, hi) (global token numbers) to `energy`
    (overwrites it when accumulate is False); finalize() forms the scores from `energy`.  A rank whose share
    is empty contributes zeros.  Returns the number of tokens this rank scored."""
    if world is None:
        world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1
    if rank is None:
        rank = dist.get_rank(group) if dist.is_available() and dist.is_initialized() else 0
    lo, hi = shard_bounds(n_tokens, world, rank)
    pieces = batches(lo, hi, batch)
    if not pieces:
        energy.zero_()
    for i, (a, b) in enumerate(pieces):
        score_batch(a, b, i > 0)
    all_reduce_energy(energy, group)
    finalize()
    return hi - lo


def calibrate_stack_streaming(n_layers: int, token_batches: Iterable, score_layer: Callable[[int, object, bool], None],
                              forward_layer: Callable[[int, object], object], energies: Sequence[torch.Tensor],
                              finalize_layer: Callable[[int], None], group=None):
    """One pass of the calibration set through a stack, batch by batch.

    For every batch x (this rank's share of it): layer l adds the energy of its input to energies[l]
    (score_layer(l, x, accumulate)), then x = forward_layer(l, x) is what layer l + 1 sees (the dense layer: the
    heavy set is not known yet).  After the last batch the energies are summed over the ranks, one all-reduce per
    layer, and finalize_layer(l) forms each layer's scores.  Returns the number of batches seen."""
    seen = 0
    for x in token_batches:
        for l in range(n_layers):
            score_layer(l, x, seen > 0)
            if l + 1 < n_layers:
                x = forward_layer(l, x)
        seen += 1
    for l in range(n_layers):
        if seen == 0:
            energies[l].zero_()
        all_reduce_energy(energies[l], group)
        finalize_layer(l)
    return seen


# ------------------------------------------------------------------------------------------------
# The same flows bound to a library context (device tensors; NCCL does the all-reduce).
def ctx_score_token_sharded(ctx, shape, W1, b1, W2, X_local: torch.Tensor, energy, scores, mode=0, W1u=None,
                            batch: int = 8192, group=None):
    """X_local holds THIS rank's calibration tokens (already sharded by the caller, e.g. by shard_bounds)."""
    n = X_local.shape[0]

    def score_batch(a, b, acc):
        ctx.score(shape, W1, b1, W2, X_local[a:b], energy, None, mode=mode, accumulate=acc, W1u=W1u)

    pieces = batches(0, n, batch)
    if not pieces:
        energy.zero_()
    for i, (a, b) in enumerate(pieces):
        score_batch(a, b, i > 0)
    all_reduce_energy(energy, group)
    ctx.score_finalize(shape, W2, energy, scores, mode=mode)
    return n
