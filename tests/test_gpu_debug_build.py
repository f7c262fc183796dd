"""The range-checked build (-DDPCLIP_DEBUG) stands in for a memory checker, which is closed on this machine: every
checked index that leaves its buffer sets DPCLIP_ERR_RANGE in the workspace's status word and the access is
skipped.  A child process loads that build instead of the normal one, runs the clipped-sum kernels that carry
the checks (CTA-pair kernel: exact, ragged, short-example and multi-layer launches) and whole steps, and must
find the status word clean and the results equal to the oracle's."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
import numpy as np, torch
sys.path.insert(0, ROOT); sys.path.insert(0, ROOT + "/tests")
import oracle, workloads
import paper_2009_03106_b200 as dp
from util import TOL, Guarded, rel_fro, to_device
dp.load_library()
assert dp.dpclip_debug_build()
for seed, (B, T, d_in, d_out) in enumerate([(4, 256, 512, 512), (3, 100, 264, 500), (40, 33, 72, 512), (1, 16, 64, 512),
                                            (24, 128, 128, 1024)]):
    A, Z = workloads.random_layer(seed, B, T, d_in, d_out, "bf16", scale_z=0.05)
    clip = np.random.default_rng(seed).uniform(0.05, 1.0, B).astype(np.float32)
    gW, gb = Guarded(d_out, d_in), Guarded(d_out)
    ws = torch.empty(dp.dpclip_workspace_bytes(B, T, d_in, d_out, dp.DPCLIP_BF16), dtype=torch.uint8, device="cuda")
    dp.dpclip_workspace_init(ws)
    dp.dpclip_clipped_grad(to_device(A, "bf16"), to_device(Z, "bf16"), torch.from_numpy(clip).cuda(), gW.t, gb.t, ws)
    assert dp.dpclip_read_status(ws) == 0, (B, T, d_in, d_out)
    gW.check(); gb.check()
    refW, refb = oracle.clipped_grad(A, Z, clip)
    assert rel_fro(gW.t.cpu().numpy(), refW) <= TOL["bf16"]["grad"] and rel_fro(gb.t.cpu().numpy(), refb) <= TOL["bf16"]["grad"]
# whole steps: several layers in one pair launch (d = 512 projections + wide layers), and the small MLP
for w in (workloads.seq("bf16", B=3, T=128, d=512, d_ff=1024), workloads.mlp_small()):
    layers = workloads.generate(w, seed=0)
    hb = [s.has_bias for s in w.layers]
    plan = dp.StepPlan([dp.Layer(to_device(A, w.dtype), to_device(Z, w.dtype), b) for (A, Z), b in zip(layers, hb)])
    plan.run(w.C, 0.0, seed=1)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    ref = oracle.step(layers, hb, w.C, 0.0, seed=1)
    for l in range(len(layers)):
        assert rel_fro(plan.gW[l].cpu().numpy(), ref["gW"][l]) <= TOL[w.dtype]["grad"], (w.name, l)
print("debug build ok")
"""


def test_range_checked_build_reports_no_violation():
    from paper_2009_03106_b200 import build as b
    lib = b.build(debug=True)                       # normally already built in-tree (build entry point)
    env = dict(os.environ, DPCLIP_LIBRARY=lib)
    out = subprocess.run([sys.executable, "-c", "ROOT = %r\n" % ROOT + CHILD], env=env, capture_output=True, text=True,
                         timeout=600)
    assert out.returncode == 0, out.stdout[-2000:] + out.stderr[-4000:]
    assert "debug build ok" in out.stdout
