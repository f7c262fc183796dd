"""The workspace-free clipped sum (for callers that cannot give the library device memory) must
return what dpclip_clipped_grad returns, and what the oracle returns.  Collected last on purpose: a run that stops at the first
failure has then already run every other test."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from util import TOL, rel_fro, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dp():
    import paper_2009_03106_b200 as pkg
    pkg.load_library()
    return pkg


def _both(dp, B, T, d_in, d_out, dtype, seed, with_bias=True):
    A, Z = workloads.random_layer(seed, B, T, d_in, d_out, dtype, scale_z=0.05)
    clip = np.random.default_rng(seed).uniform(0.1, 1.0, B).astype(np.float32)
    dA, dZ, dc = to_device(A, dtype), to_device(Z, dtype), torch.from_numpy(clip).cuda()
    ws = torch.empty(dp.dpclip_workspace_bytes(B, T, d_in, d_out, dp.DPCLIP_BF16), dtype=torch.uint8, device="cuda")
    dp.dpclip_workspace_init(ws)
    ref_W = torch.empty((d_out, d_in), device="cuda"); ref_b = torch.empty(d_out, device="cuda") if with_bias else None
    dp.dpclip_clipped_grad(dA, dZ, dc, ref_W, ref_b, ws)
    got_W = torch.full((d_out, d_in), 7.0, device="cuda"); got_b = torch.full((d_out,), 7.0, device="cuda") if with_bias else None
    dp.dpclip_clipped_grad_noalloc(dA, dZ, dc, got_W, got_b)
    torch.cuda.synchronize()
    # the oracle's clipped sum of the same inputs: the new entry point is held to the path's own tolerance
    want_W, want_b = oracle.clipped_grad(A, Z, clip)
    assert rel_fro(got_W.cpu().numpy(), want_W) <= TOL[dtype]["grad"]
    if with_bias:
        assert rel_fro(got_b.cpu().numpy(), want_b) <= TOL[dtype]["grad"]
    return ref_W.cpu().numpy(), got_W.cpu().numpy(), (ref_b.cpu().numpy() if with_bias else None), \
        (got_b.cpu().numpy() if with_bias else None)


def test_no_alloc_entry_matches_workspace_entry_twice_in_a_row(dp):
    # two calls back to back on different data and shapes: the shared scratch keeps the first call's
    # contents, which must not leak into the second result
    for seed, shape in ((1, (32, 256, 512, 512)), (2, (16, 128, 264, 136))):
        ref_W, got_W, ref_b, got_b = _both(dp, *shape, "bf16", seed)
        # same kernels, only the row split differs: agreement far inside the bf16 tolerance
        assert rel_fro(got_W, ref_W) <= 1e-5 and rel_fro(got_W, ref_W) <= TOL["bf16"]["grad"]
        assert rel_fro(got_b, ref_b) <= 1e-5


def test_no_alloc_entry_at_the_size_limit_with_a_bias(dp):
    # the largest output the entry point accepts (8 MB padded), with a bias: the fixed array holds 31 partial
    # tiles of 512 x 256 for the 16 output tiles, so the row split is clamped far below the usual one
    ref_W, got_W, ref_b, got_b = _both(dp, 3, 96, 2048, 1024, "bf16", 5)
    assert rel_fro(got_W, ref_W) <= 1e-5 and rel_fro(got_b, ref_b) <= 1e-5
    # and twice in a row on the same shape with other data
    ref_W, got_W, ref_b, got_b = _both(dp, 3, 96, 2048, 1024, "bf16", 6)
    assert rel_fro(got_W, ref_W) <= 1e-5 and rel_fro(got_b, ref_b) <= 1e-5


def test_no_alloc_entry_on_the_fp32_path_and_limits(dp):
    ref_W, got_W, ref_b, got_b = _both(dp, 8, 17, 27, 33, "f32", 3)
    assert rel_fro(got_W, ref_W) <= TOL["f32"]["grad"] and rel_fro(got_b, ref_b) <= TOL["f32"]["grad"]
    # a layer whose padded output exceeds the stated maximum is refused before anything is launched
    assert dp.dpclip_noalloc_max_output_bytes() == 8 << 20
    A = torch.zeros((2, 1, 4096), device="cuda", dtype=torch.bfloat16)
    Z = torch.zeros((2, 1, 1024), device="cuda", dtype=torch.bfloat16)
    gW = torch.empty((1024, 4096), device="cuda")
    with pytest.raises(dp.DpclipError) as err:
        dp.dpclip_clipped_grad_noalloc(A, Z, None, gW, None)
    assert err.value.status == -4
