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


def _worker(rank, world, port, q):
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
    parallel.sharded_step(plan, 78.0, w.sigma, seed=5, stream_id0=0, ops=OracleOps())
    q.put((rank, lo, hi, plan.flat.numpy().copy(), plan.clip.numpy().copy()))
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_step_equals_single_process_step():
    import oracle
    import workloads
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0)); port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
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
    assert (got[0][1], got[0][2], got[1][1], got[1][2]) == (0, 16, 16, 32)
    np.testing.assert_array_equal(got[0][3], got[1][3])
    np.testing.assert_allclose(got[0][3], want, rtol=1e-5, atol=1e-5)
    np.testing.assert_allclose(np.concatenate([got[0][4], got[1][4]]), ref["clip"], rtol=1e-6)


def test_shard_examples_partitions_the_batch():
    from paper_2009_03106_b200 import parallel
    for B, world in [(128, 8), (10, 3), (2, 4)]:
        cuts = [parallel.shard_examples(B, r, world) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == B
        assert all(cuts[r][1] == cuts[r + 1][0] for r in range(world - 1))
