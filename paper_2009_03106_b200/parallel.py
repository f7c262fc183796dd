"""Batch-sharded step over several GPUs (one process per GPU).

The path shards by example: norms, factors and each example's term of the
clipped sum touch only that example's rows.  Every rank runs the kernels on
its own examples, the partial clipped sums are combined by an all-reduce of
the flat gradient buffer (NCCL over NVLink on GPUs), and the noise is added
after the reduction, once, with the same (seed, stream) on every rank so that
all ranks hold the same released gradient.

`ops` is the set of entry points to call; it defaults to the CUDA binding
(whose whole-step call covers everything before the reduction).  Tests on CPU
ranks (gloo) pass their own object: one with the four per-stage methods, or
one that also has the whole-step call, which is the branch GPUs take.
"""
from __future__ import annotations

from typing import List, Tuple

import torch.distributed as dist


def _local_step(plan, C: float, seed: int, stream_id0: int, ops) -> None:
    """Norms -> factors -> clipped sums of this rank's examples, sigma = 0 (the noise belongs after the reduction)."""
    whole = getattr(ops, "dpclip_step", None)
    mixed = any(getattr(y, "kind", 0) != 0 for y in plan.layers)      # LayerNorm / feature-map convolution layers
    if whole is not None:
        # one library call; all-T=1 models take the one-launch fused kernel this way
        (ops.dpclip_model_step if mixed else whole)(plan, C, 0.0, seed, stream_id0)
        return
    for l, y in enumerate(plan.layers):
        ops.dpclip_layer_sqnorms(y.A, y.Zbar, y.has_bias, plan.sq_layers[l], plan.workspace, y.method)
    ops.dpclip_factors(plan.sq_layers, C, plan.clip, plan.norms)
    for l, y in enumerate(plan.layers):
        ops.dpclip_clipped_grad(y.A, y.Zbar, plan.clip, plan.gW[l], plan.gb[l], plan.workspace)


def _noise_once(plan, C: float, sigma: float, seed: int, stream_id0: int, ops) -> None:
    mixed = any(getattr(y, "kind", 0) != 0 for y in plan.layers)
    all_noise = getattr(ops, "dpclip_step_noise", None)
    if all_noise is not None and not mixed:
        all_noise(plan, C, sigma, seed, stream_id0)               # every tensor's noise in one launch
        return
    for l in range(len(plan.layers)):
        ops.dpclip_add_noise(plan.gW[l].view(-1), sigma, C, seed, stream_id0 + 2 * l)
        if plan.gb[l] is not None:
            ops.dpclip_add_noise(plan.gb[l], sigma, C, seed, stream_id0 + 2 * l + 1)


def buckets(n_elements: int, bucket_elements: int) -> List[Tuple[int, int]]:
    """Contiguous [lo, hi) slices of the flat gradient buffer, one all-reduce each.  NVSwitch gives every GPU
    full bandwidth to every peer, so a bucket is sized for launch latency and pipelining (a few MB), not for a
    link count; the last bucket takes the remainder."""
    if n_elements <= 0:
        return []
    bucket_elements = max(1, int(bucket_elements))
    cuts = list(range(0, n_elements, bucket_elements)) + [n_elements]
    if len(cuts) > 2 and cuts[-1] - cuts[-2] < bucket_elements // 4:
        del cuts[-2]                                              # no tiny tail bucket
    return list(zip(cuts[:-1], cuts[1:]))


def sharded_step(plan, C: float, sigma: float, seed: int, stream_id0: int = 0, group=None, ops=None,
                 bucket_elements: int = 0) -> None:
    """One step on this rank's shard + the reduction over ranks + the noise (added once, after the last bucket).
    bucket_elements = 0: ONE all-reduce of the flat buffer; > 0: one asynchronous all-reduce per bucket, all
    waited for before the noise."""
    if ops is None:
        from . import binding as ops
    _local_step(plan, C, seed, stream_id0, ops)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        if bucket_elements <= 0:
            dist.all_reduce(plan.flat, op=dist.ReduceOp.SUM, group=group)
        else:
            pending = [dist.all_reduce(plan.flat[lo:hi], op=dist.ReduceOp.SUM, group=group, async_op=True)
                       for lo, hi in buckets(plan.flat.numel(), bucket_elements)]
            for h in pending:
                h.wait()
    _noise_once(plan, C, sigma, seed, stream_id0, ops)


class ShardedStep:
    """The sharded step of one rank with its launches recorded once: the local step (ONE dpclip_step_streams
    call; dpclip_step for all-T=1 models) as a CUDA graph, then the bucketed all-reduce, then the noise.  NCCL
    stays outside the graph (its launches are few and large), so a rank that fails between steps leaves no
    captured collective behind."""

    def __init__(self, plan, C: float, sigma: float, seed: int, stream_id0: int = 0, group=None,
                 bucket_bytes: int = 4 << 20, branches: int = 4):
        from . import binding as ops
        self.plan, self.C, self.sigma, self.seed, self.sid0, self.group, self.ops = plan, C, sigma, seed, stream_id0, group, ops
        all_t1 = all(y.A.dim() == 2 or y.A.shape[1] == 1 for y in plan.layers)
        self.branches = 1 if all_t1 else branches
        self.graph = plan.capture(C, 0.0, seed, stream_id0, branches=self.branches)
        self.buckets = buckets(plan.flat.numel(), bucket_bytes // 4)
        self.world = dist.get_world_size(group) if dist.is_available() and dist.is_initialized() else 1

    def run(self) -> None:
        self.graph.replay()
        if self.world > 1:
            pending = [dist.all_reduce(self.plan.flat[lo:hi], op=dist.ReduceOp.SUM, group=self.group, async_op=True)
                       for lo, hi in self.buckets]
            for h in pending:
                h.wait()
        _noise_once(self.plan, self.C, self.sigma, self.seed, self.sid0, self.ops)

    def describe(self) -> str:
        return (f"per rank: CUDA graph of one dpclip_step{'_streams' if self.branches > 1 else ''} call on the rank's "
                f"examples (sigma = 0), {len(self.buckets)} asynchronous NCCL all-reduce(s) over the flat gradient buffer, "
                "one noise launch after the last bucket; events around every step, max over ranks")


def shard_examples(B: int, rank: int, world: int):
    """Contiguous, balanced slice [lo, hi) of a global batch of B examples."""
    base, rem = divmod(B, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)
