"""Data-parallel plumbing for more than one GPU (one process per GPU, torch.distributed).

Algorithm 1 runs the per-batch body on every worker and then averages the gradients; here each rank
holds a full replica of the graph and takes every world-th batch of positives.  The only collective on
the path is that gradient average (one all-reduce of the flat gradient vector, at most ~1.3 MB).
"""
from __future__ import annotations


def batch_for(step: int, rank: int, world: int, n_batches: int) -> int:
    """Index of the batch that `rank` processes at global step `step`: ranks take consecutive batches
    of the epoch, wrapping around, so one step consumes `world` distinct batches."""
    return (step * world + rank) % n_batches


def sync_gradients(grads, world: int, dist=None) -> float:
    """Sum the ranks' gradients in place (all-reduce) and return the factor 1 / world that the
    optimiser applies (lp_adam_step's grad_scale), i.e. the average of Algorithm 1's synchronise step."""
    if world > 1:
        dist.all_reduce(grads)
    return 1.0 / world
