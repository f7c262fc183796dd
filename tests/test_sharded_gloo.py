"""world_size-2 test of the batch-sharded step's host logic on CPU ranks (gloo).

No GPU here, so the four entry points are replaced by an oracle-backed stand-in
(test infrastructure); what is under test is the sharding, the single
all-reduce of the flat gradient buffer and the add-noise-once rule."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class OracleOps:
    """The binding's call signatures, computed by the CPU oracle."""

    def __init__(self):
        import oracle
        self.o = oracle

    def dpclip_layer_sqnorms(self, A, Z, has_bias, sq_row, workspace, method=0):
        sq_row.copy_(torch.from_numpy(self.o.layer_sqnorms(A.numpy(), Z.numpy(), has_bias)).float())

    def dpclip_factors(self, sq_layers, C, clip, norms=None):
        n, c = self.o.factors(sq_layers.numpy(), C)
        clip.copy_(torch.from_numpy(c).float())
        if norms is not None:
            norms.copy_(torch.from_numpy(n).float())

    def dpclip_clipped_grad(self, A, Z, clip, gW, gb, workspace):
        w, b = self.o.clipped_grad(A.numpy(), Z.numpy(), clip.numpy())
        gW.copy_(torch.from_numpy(w).float())
        if gb is not None:
            gb.copy_(torch.from_numpy(b).float())

    def dpclip_add_noise(self, g, sigma, C, seed, stream_id):
        g.copy_(torch.from_numpy(self.o.add_noise(g.numpy(), sigma, C, seed, stream_id)).float())


class OracleWholeStepOps(OracleOps):
    """The same with the whole-step call and the all-tensors noise call of the CUDA binding: drives the branch
    of the sharded step that GPUs take (one library call before the reduction, one noise call after it)."""

    def dpclip_step(self, plan, C, sigma, seed, stream_id0=0):
        assert sigma == 0.0                                   # the noise belongs after the reduction
        layers = [(y.A.numpy(), y.Zbar.numpy()) for y in plan.layers]
        r = self.o.step(layers, [y.has_bias for y in plan.layers], C, 0.0, seed, stream_id0)
        plan.clip.copy_(torch.from_numpy(r["clip"]).float()); plan.norms.copy_(torch.from_numpy(r["norms"]).float())
        for l in range(len(layers)):
            plan.gW[l].copy_(torch.from_numpy(r["gW"][l]).float())
            if plan.gb[l] is not None:
                plan.gb[l].copy_(torch.from_numpy(r["gb"][l]).float())
        self.whole_calls = getattr(self, "whole_calls", 0) + 1

    def dpclip_step_noise(self, plan, C, sigma, seed, stream_id0=0):
        for l in range(len(plan.layers)):
            self.dpclip_add_noise(plan.gW[l].view(-1), sigma, C, seed, stream_id0 + 2 * l)
            if plan.gb[l] is not None:
                self.dpclip_add_noise(plan.gb[l], sigma, C, seed, stream_id0 + 2 * l + 1)


class CpuPlan:
    def __init__(self, layers, has_bias):
        from types import SimpleNamespace
        self.layers = [SimpleNamespace(A=torch.from_numpy(A), Zbar=torch.from_numpy(Z), has_bias=hb, method=0)
                       for (A, Z), hb in zip(layers, has_bias)]
        B = layers[0][0].shape[0]
        sizes = []
        for (A, Z), hb in zip(layers, has_bias):
            sizes += [Z.shape[2] * A.shape[2], Z.shape[2] if hb else 0]
        self.flat = torch.zeros(sum(sizes))
        self.gW, self.gb, off = [], [], 0
        for i, ((A, Z), hb) in enumerate(zip(layers, has_bias)):
            n = sizes[2 * i]; self.gW.append(self.flat[off:off + n].view(Z.shape[2], A.shape[2])); off += n
            n = sizes[2 * i + 1]; self.gb.append(self.flat[off:off + n] if hb else None); off += n
        self.sq_layers = torch.zeros(len(layers), B)
        self.clip = torch.zeros(B); self.norms = torch.zeros(B)
        self.workspace = None


def _worker(rank, world, port, q, whole=False, bucket_elements=0):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"; os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import workloads
    from paper_2009_03106_b200 import parallel
    w = workloads.mlp_small()
    full = workloads.generate(w, seed=0)
    lo, hi = parallel.shard_examples(w.B, rank, world)
    mine = [(A[lo:hi], Z[lo:hi]) for A, Z in full]
    hb = [s.has_bias for s in w.layers]
    plan = CpuPlan(mine, hb)
    ops = OracleWholeStepOps() if whole else OracleOps()
    parallel.sharded_step(plan, 78.0, w.sigma, seed=5, stream_id0=0, ops=ops, bucket_elements=bucket_elements)
    if whole:
        assert ops.whole_calls == 1
    q.put((rank, lo, hi, plan.flat.numpy().copy(), plan.clip.numpy().copy()))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,whole,bucket_elements", [(2, False, 0), (2, True, 0), (3, True, 50000)])
def test_sharded_step_equals_single_process_step(world, whole, bucket_elements):
    """Per-stage ops and one all-reduce; the whole-step branch GPUs take; and three ranks with an uneven split
    (11 + 11 + 10 examples) whose reduction goes out in several asynchronous buckets."""
    import oracle
    import workloads
    from paper_2009_03106_b200 import parallel
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q, whole, bucket_elements)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted([q.get(timeout=180) for _ in procs], key=lambda t: t[0])
    for p in procs:
        p.join(60); assert p.exitcode == 0
    w = workloads.mlp_small()
    full = workloads.generate(w, seed=0)
    hb = [s.has_bias for s in w.layers]
    ref = oracle.step(full, hb, 78.0, w.sigma, seed=5)
    want = np.concatenate([np.concatenate([ref["outW"][l].ravel(), ref["outb"][l]]) for l in range(2)])
    assert 0 < (ref["clip"] < 1).sum() < w.B
    # ranks cover the batch once, agree with each other, and match the unsharded result
    assert [(g[1], g[2]) for g in got] == [parallel.shard_examples(w.B, r, world) for r in range(world)]
    if world == 3:
        assert [g[2] - g[1] for g in got] == [11, 11, 10]
    for g in got[1:]:
        np.testing.assert_array_equal(got[0][3], g[3])
    np.testing.assert_allclose(got[0][3], want, rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(np.concatenate([g[4] for g in got]), ref["clip"], rtol=1e-6)


def test_buckets_cover_the_buffer_once():
    from paper_2009_03106_b200 import parallel
    for n, b in [(10, 3), (1 << 20, 1 << 18), (1000, 1 << 20), (1025, 256), (7, 1)]:
        cuts = parallel.buckets(n, b)
        assert cuts[0][0] == 0 and cuts[-1][1] == n
        assert all(cuts[i][1] == cuts[i + 1][0] for i in range(len(cuts) - 1))
        assert all(hi > lo for lo, hi in cuts)
    assert parallel.buckets(0, 4) == []


def test_shard_examples_partitions_the_batch():
    from paper_2009_03106_b200 import parallel
    for B, world in [(128, 8), (10, 3), (2, 4)]:
        cuts = [parallel.shard_examples(B, r, world) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == B
        assert all(cuts[r][1] == cuts[r + 1][0] for r in range(world - 1))
