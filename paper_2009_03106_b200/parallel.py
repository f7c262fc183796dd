"""Batch-sharded step over several GPUs (one process per GPU).

The path shards by example: norms, factors and each example's term of the
clipped sum touch only that example's rows.  Every rank runs the kernels on
its own examples, the partial clipped sums are combined by ONE all-reduce of
the flat gradient buffer (NCCL over NVLink on GPUs), and the noise is added
after the reduction, once, with the same (seed, stream) on every rank so that
all ranks hold the same released gradient.

`ops` is the set of entry points to call; it defaults to the CUDA binding
(whose whole-step call covers everything before the reduction).  Tests on CPU
ranks (gloo) pass their own object with the four per-stage methods.
"""
from __future__ import annotations

import torch.distributed as dist


def sharded_step(plan, C: float, sigma: float, seed: int, stream_id0: int = 0, group=None, ops=None) -> None:
    if ops is None:
        from . import binding as ops
    whole = getattr(ops, "dpclip_step", None)
    mixed = any(getattr(y, "kind", 0) != 0 for y in plan.layers)      # LayerNorm / feature-map convolution layers
    if whole is not None:
        # norms -> factors -> clipped sums of this rank's examples in one library call (sigma = 0: the noise
        # belongs after the reduction); all-T=1 models take the one-launch fused kernel this way
        (ops.dpclip_model_step if mixed else whole)(plan, C, 0.0, seed, stream_id0)
    else:
        for l, y in enumerate(plan.layers):
            ops.dpclip_layer_sqnorms(y.A, y.Zbar, y.has_bias, plan.sq_layers[l], plan.workspace, y.method)
        ops.dpclip_factors(plan.sq_layers, C, plan.clip, plan.norms)
        for l, y in enumerate(plan.layers):
            ops.dpclip_clipped_grad(y.A, y.Zbar, plan.clip, plan.gW[l], plan.gb[l], plan.workspace)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(plan.flat, op=dist.ReduceOp.SUM, group=group)
    all_noise = getattr(ops, "dpclip_step_noise", None)
    if all_noise is not None and not mixed:
        all_noise(plan, C, sigma, seed, stream_id0)               # every tensor's noise in one launch
        return
    for l in range(len(plan.layers)):
        ops.dpclip_add_noise(plan.gW[l].view(-1), sigma, C, seed, stream_id0 + 2 * l)
        if plan.gb[l] is not None:
            ops.dpclip_add_noise(plan.gb[l], sigma, C, seed, stream_id0 + 2 * l + 1)


def shard_examples(B: int, rank: int, world: int):
    """Contiguous, balanced slice [lo, hi) of a global batch of B examples."""
    base, rem = divmod(B, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
