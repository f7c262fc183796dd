"""Parity of the CUDA path (through the C ABI) with the fp64 oracle, element by
element on the same seeded inputs.  Sizes span several tiles and ragged tails."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from util import SAT_BAND, TOL, Guarded, check_saturation, max_rel, rel_fro, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dp():
    import paper_2009_03106_b200 as pkg
    pkg.load_library()          # fails loudly if the CUDA library is missing
    return pkg


def _ws(dp, nbytes=None):
    if nbytes is None:          # enough for any layer of either dtype
        nbytes = max(dp.dpclip_workspace_bytes(1, 1, 1, 1, dp.DPCLIP_BF16), 1 << 20)
    ws = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    dp.dpclip_workspace_init(ws)
    return ws


def _sqnorms(dp, A, Z, dtype, has_bias, method=0):
    dA, dZ = to_device(A, dtype), to_device(Z, dtype)
    guard = Guarded(A.shape[0], fill=-1.0)              # every norm test writes between guard bands
    sq = guard.t
    ws = _ws(dp, max(1 << 20, dp.dpclip_workspace_bytes(A.shape[0], A.shape[1], A.shape[2], Z.shape[2],
                                                       0 if dtype == "f32" else 1, method)))
    dp.dpclip_layer_sqnorms(dA, dZ, has_bias, sq, ws, method)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(ws) == 0
    guard.check()
    return sq.cpu().numpy()


# ---------------------------------------------------------------------------
# (a) T = 1 norms
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,d_in,d_out", [(1, 1, 1), (3, 10, 27), (3, 33, 1), (32, 784, 256), (32, 256, 10),
                                          (128, 1000, 1000), (128, 8192, 256), (5, 4099, 13)])
@pytest.mark.parametrize("has_bias", [True, False])
def test_t1_norms(dp, dtype, B, d_in, d_out, has_bias):
    A, Z = workloads.random_layer(1, B, 1, d_in, d_out, dtype, scale_z=0.1)
    ref = oracle.layer_sqnorms(A, Z, has_bias)
    got = _sqnorms(dp, A, Z, dtype, has_bias)
    # squared norms: twice the relative tolerance of the norm
    assert max_rel(np.sqrt(got), np.sqrt(ref)) <= TOL["f32"]["norm"]     # inputs identical, fp32 accumulate


def test_t1_norms_strided_rows_and_zero_example(dp):
    B, d_in, d_out = 6, 50, 20
    A, Z = workloads.random_layer(2, B, 1, d_in, d_out)
    A[2] = 0.0                                           # an all-zero example has norm 0
    bigA = torch.zeros((B, 1, 64), device="cuda"); bigA[:, :, :d_in] = torch.from_numpy(A).cuda()
    bigZ = torch.zeros((B, 1, 24), device="cuda"); bigZ[:, :, :d_out] = torch.from_numpy(Z).cuda()
    bigA[:, :, d_in:] = 7.0; bigZ[:, :, d_out:] = 7.0    # padding must not be read
    sq = torch.empty(B, device="cuda")
    dp.dpclip_layer_sqnorms(bigA[:, :, :d_in], bigZ[:, :, :d_out], False, sq, _ws(dp))
    ref = oracle.layer_sqnorms(A, Z, False)
    got = sq.cpu().numpy()
    assert got[2] == 0.0
    assert max_rel(got, ref) <= 2e-5


# ---------------------------------------------------------------------------
# (b) T > 1 norms, fp32-ALU tile kernel
# ---------------------------------------------------------------------------
SIMT_SHAPES = [(5, 2, 1, 1), (3, 17, 27, 33), (2, 64, 70, 65), (4, 130, 64, 64), (3, 33, 129, 10),
               (2, 256, 288, 64)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,T,d_in,d_out", SIMT_SHAPES)
@pytest.mark.parametrize("has_bias", [True, False])
def test_simt_norms(dp, dtype, B, T, d_in, d_out, has_bias):
    A, Z = workloads.random_layer(3, B, T, d_in, d_out, dtype, scale_z=0.05)
    ref = oracle.layer_sqnorms(A, Z, has_bias)
    got = _sqnorms(dp, A, Z, dtype, has_bias, method=dp.DPCLIP_SIMT)
    assert max_rel(np.sqrt(got), np.sqrt(ref)) <= TOL["f32"]["norm"]


# ---------------------------------------------------------------------------
# (b) T > 1 norms on the tensor cores (bf16): Gram form and materialised tiles
# ---------------------------------------------------------------------------
TC_SHAPES = [(3, 256, 64, 128), (4, 128, 72, 64), (5, 64, 64, 64), (7, 40, 64, 32), (3, 200, 128, 64),
             (2, 384, 64, 64), (3, 40, 320, 136), (2, 130, 8, 8), (9, 16, 264, 64), (1, 2, 64, 64)]


@pytest.mark.parametrize("method", ["gram", "materialize"])
@pytest.mark.parametrize("B,T,d_in,d_out", TC_SHAPES)
@pytest.mark.parametrize("has_bias", [True, False])
def test_tensor_core_norms(dp, method, B, T, d_in, d_out, has_bias):
    A, Z = workloads.random_layer(5, B, T, d_in, d_out, "bf16", scale_z=0.05)
    ref = oracle.layer_sqnorms(A, Z, has_bias)
    m = dp.DPCLIP_GRAM if method == "gram" else dp.DPCLIP_MATERIALIZE
    got = _sqnorms(dp, A, Z, "bf16", has_bias, method=m)
    # bf16 products are exact in fp32; only the accumulation order differs from the oracle
    assert max_rel(np.sqrt(got), np.sqrt(ref)) <= 2e-5, (got, ref)


def test_tensor_core_norms_run_twice_identically_shaped(dp):
    """Back-to-back launches reuse tensor memory and barriers cleanly."""
    A, Z = workloads.random_layer(6, 20, 256, 192, 128, "bf16", scale_z=0.05)
    ref = oracle.layer_sqnorms(A, Z, True)
    for m in (dp.DPCLIP_GRAM, dp.DPCLIP_MATERIALIZE, dp.DPCLIP_GRAM):
        got = _sqnorms(dp, A, Z, "bf16", True, method=m)
        assert max_rel(np.sqrt(got), np.sqrt(ref)) <= 2e-5


# the shapes with d_out = 500 ... 1024 take the CTA-pair kernel (512 x 256 tiles): exact and ragged tiles, short
# examples (a factor per row), a single stage (one item per tile: direct stores), several row slices
@pytest.mark.parametrize("B,T,d_in,d_out", [(128, 1, 512, 256), (4, 256, 512, 256), (3, 100, 264, 136),
                                            (2, 2048, 64, 64), (16, 64, 576, 128), (4, 256, 512, 512),
                                            (3, 100, 264, 500), (2, 300, 200, 1000), (40, 33, 72, 512),
                                            (1, 16, 64, 512), (24, 128, 128, 1024)])
def test_tensor_core_clipped_grad(dp, B, T, d_in, d_out):
    A, Z = workloads.random_layer(8, B, T, d_in, d_out, "bf16", scale_z=0.05)
    clip = np.random.default_rng(B).uniform(0.05, 1.0, B).astype(np.float32)
    clip[::2] = 1.0
    refW, refb = oracle.clipped_grad(A, Z, clip)
    dA, dZ = to_device(A, "bf16"), to_device(Z, "bf16")
    guard_W, guard_b = Guarded(d_out, d_in), Guarded(d_out)       # outputs between guard bands
    gW, gb = guard_W.t, guard_b.t
    ws = _ws(dp)
    dp.dpclip_clipped_grad(dA, dZ, torch.from_numpy(clip).cuda(), gW, gb, ws)
    assert dp.dpclip_read_status(ws) == 0
    guard_W.check(); guard_b.check()
    assert rel_fro(gW.cpu().numpy(), refW) <= TOL["bf16"]["grad"]
    assert rel_fro(gb.cpu().numpy(), refb) <= 2e-3          # fp32 sums of the bf16-rounded clip*zbar values
    refW1, refb1 = oracle.clipped_grad(A, Z, None)
    dp.dpclip_clipped_grad(dA, dZ, None, gW, gb, ws)
    assert rel_fro(gW.cpu().numpy(), refW1) <= 2e-5
    assert rel_fro(gb.cpu().numpy(), refb1) <= 1e-5


# ---------------------------------------------------------------------------
# fp32 layers on the tensor cores (error-compensated tf32): still inside the fp32 tolerance
# ---------------------------------------------------------------------------
# (1, 16384, ...) is one long accumulation: 512 stages, drained to registers every few stages
TF32_SHAPES = [(8, 256, 288, 64), (6, 200, 264, 136), (2, 2048, 128, 128), (16, 64, 576, 128), (40, 33, 100, 260),
               (1, 16384, 128, 128)]


@pytest.mark.parametrize("B,T,d_in,d_out", TF32_SHAPES)
@pytest.mark.parametrize("has_bias", [True, False])
def test_tf32_norms(dp, B, T, d_in, d_out, has_bias):
    A, Z = workloads.random_layer(11, B, T, d_in, d_out, "f32", scale_z=0.05)
    ref = oracle.layer_sqnorms(A, Z, has_bias)
    got = _sqnorms(dp, A, Z, "f32", has_bias, method=dp.DPCLIP_MATERIALIZE)
    assert max_rel(np.sqrt(got), np.sqrt(ref)) <= TOL["f32"]["norm"], max_rel(np.sqrt(got), np.sqrt(ref))
    assert dp.dpclip_pick_method(B, T, d_in, d_out, d_in, d_out, dp.DPCLIP_F32) == dp.DPCLIP_MATERIALIZE


@pytest.mark.parametrize("B,T,d_in,d_out", TF32_SHAPES + [(128, 1, 8192, 256)])
def test_tf32_clipped_grad(dp, B, T, d_in, d_out):
    A, Z = workloads.random_layer(12, B, T, d_in, d_out, "f32", scale_z=0.05)
    clip = np.random.default_rng(B).uniform(0.05, 1.0, B).astype(np.float32)
    clip[::2] = 1.0
    refW, refb = oracle.clipped_grad(A, Z, clip)
    dA, dZ = to_device(A, "f32"), to_device(Z, "f32")
    gW = torch.full((d_out, d_in), 9.0, device="cuda"); gb = torch.full((d_out,), 9.0, device="cuda")
    ws = _ws(dp)
    dp.dpclip_clipped_grad(dA, dZ, torch.from_numpy(clip).cuda(), gW, gb, ws)
    assert dp.dpclip_read_status(ws) == 0
    e = rel_fro(gW.cpu().numpy(), refW)
    assert e <= TOL["f32"]["grad"], e
    assert rel_fro(gb.cpu().numpy(), refb) <= TOL["f32"]["grad"]


# ---------------------------------------------------------------------------
# element-wise parameter layers (LayerNorm gain / shift)
# ---------------------------------------------------------------------------
EW_SHAPES = [(1, 1, 1), (3, 1, 10), (5, 7, 33), (4, 40, 64), (6, 37, 260), (128, 1, 1000), (16, 256, 512), (3, 300, 1028)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,T,d", EW_SHAPES)
def test_elementwise_norms_and_clipped_sums(dp, B, T, d, dtype):
    H, Z = workloads.layernorm_pair(31, B, T, d, dtype, var_z=0.01)
    tol = TOL[dtype]
    dH, dZ = to_device(H, dtype), to_device(Z, dtype)
    for has_shift in (True, False):
        ref = oracle.elementwise_sqnorms(H, Z, has_shift)
        sq = torch.full((B,), -1.0, device="cuda")
        dp.dpclip_elementwise_sqnorms(dH, dZ, has_shift, sq)
        got = sq.cpu().numpy()
        assert max_rel(np.sqrt(got), np.sqrt(ref)) <= tol["norm"], max_rel(np.sqrt(got), np.sqrt(ref))
    clip = np.random.default_rng(B + d).uniform(0.05, 1.0, B).astype(np.float32)
    clip[::2] = 1.0
    for c in (clip, None):
        ref_g, ref_s = oracle.elementwise_clipped_grad(H, Z, c)
        g_scale = torch.full((d,), 7.0, device="cuda"); g_shift = torch.full((d,), 7.0, device="cuda")
        dp.dpclip_elementwise_clipped_grad(dH, dZ, None if c is None else torch.from_numpy(c).cuda(), g_scale, g_shift)
        assert rel_fro(g_scale.cpu().numpy(), ref_g) <= tol["grad"], rel_fro(g_scale.cpu().numpy(), ref_g)
        assert rel_fro(g_shift.cpu().numpy(), ref_s) <= tol["grad"]
    only = torch.full((d,), 7.0, device="cuda")
    dp.dpclip_elementwise_clipped_grad(dH, dZ, torch.from_numpy(clip).cuda(), only, None)     # no shift parameter
    assert rel_fro(only.cpu().numpy(), oracle.elementwise_clipped_grad(H, Z, clip)[0]) <= tol["grad"]


def test_elementwise_padded_rows(dp):
    """Row stride larger than the width, and a width that is not a multiple of 4 (scalar path)."""
    B, T, d, ld = 5, 9, 30, 32
    H, Z = workloads.layernorm_pair(32, B, T, d, "f32", var_z=0.01)
    Hp = torch.full((B, T, ld), float("nan"), device="cuda"); Zp = torch.full((B, T, ld), float("nan"), device="cuda")
    Hp[:, :, :d] = torch.from_numpy(H).cuda(); Zp[:, :, :d] = torch.from_numpy(Z).cuda()
    sq = torch.empty(B, device="cuda")
    dp.dpclip_elementwise_sqnorms(Hp[:, :, :d], Zp[:, :, :d], True, sq)
    assert max_rel(np.sqrt(sq.cpu().numpy()), np.sqrt(oracle.elementwise_sqnorms(H, Z, True))) <= TOL["f32"]["norm"]
    g = torch.empty(d, device="cuda"); s = torch.empty(d, device="cuda")
    dp.dpclip_elementwise_clipped_grad(Hp[:, :, :d], Zp[:, :, :d], None, g, s)
    rg, rs = oracle.elementwise_clipped_grad(H, Z, None)
    assert rel_fro(g.cpu().numpy(), rg) <= TOL["f32"]["grad"] and rel_fro(s.cpu().numpy(), rs) <= TOL["f32"]["grad"]


def test_transformer_block_with_layernorms(dp):
    """Dense layers and LayerNorm parameters of one block clipped together: per-layer norm rows from both
    kinds of entry points, one factor computation, clipped sums and noise per tensor."""
    B, T, d, dff, C, sigma, seed = 6, 24, 64, 136, 1.0, 0.7, 9
    w = workloads.seq("bf16", B=B, T=T, d=d, d_ff=dff)
    dense = workloads.generate(w, 3)
    lns = [workloads.layernorm_pair(40 + k, B, T, d, "bf16", var_z=1.0 / (B * T)) for k in range(2)]
    hb = [s.has_bias for s in w.layers]
    sq_ref = [oracle.layer_sqnorms(A, Z, b) for (A, Z), b in zip(dense, hb)] + [oracle.elementwise_sqnorms(H, Z, True) for H, Z in lns]
    # spread the norms around C as the calibrated workloads do
    n0, _ = oracle.factors(np.stack(sq_ref), C)
    r = workloads.spread_factors(B, 1) * C / n0
    scale = lambda Z: workloads.round_to_bf16((Z.astype(np.float64) * r[:, None, None]).astype(np.float32))   # noqa: E731
    dense = [(A, scale(Z)) for A, Z in dense]
    lns = [(H, scale(Z)) for H, Z in lns]
    sq_ref = np.stack([oracle.layer_sqnorms(A, Z, b) for (A, Z), b in zip(dense, hb)] +
                      [oracle.elementwise_sqnorms(H, Z, True) for H, Z in lns])
    norms_ref, clip_ref = oracle.factors(sq_ref, C)
    L = len(dense) + len(lns)
    sq = torch.empty(L, B, device="cuda"); ws = _ws(dp)
    dd = [(to_device(A, "bf16"), to_device(Z, "bf16")) for A, Z in dense]
    dl = [(to_device(H, "bf16"), to_device(Z, "bf16")) for H, Z in lns]
    for l, ((A, Z), b) in enumerate(zip(dd, hb)):
        dp.dpclip_layer_sqnorms(A, Z, b, sq[l], ws)
    for k, (H, Z) in enumerate(dl):
        dp.dpclip_elementwise_sqnorms(H, Z, True, sq[len(dd) + k])
    clip = torch.empty(B, device="cuda"); norms = torch.empty(B, device="cuda")
    dp.dpclip_factors(sq, C, clip, norms)
    assert max_rel(norms.cpu().numpy(), norms_ref) <= TOL["bf16"]["norm"]
    check_saturation(clip.cpu().numpy(), norms_ref, clip_ref, C)
    assert 0 < int((clip < 1).sum()) < B
    for k, ((H, Z), (Hn, Zn)) in enumerate(zip(dl, lns)):
        g = torch.empty(d, device="cuda"); s = torch.empty(d, device="cuda")
        dp.dpclip_elementwise_clipped_grad(H, Z, clip, g, s)
        rg, rs = oracle.elementwise_clipped_grad(Hn, Zn, clip_ref)
        assert rel_fro(g.cpu().numpy(), rg) <= TOL["bf16"]["grad"] and rel_fro(s.cpu().numpy(), rs) <= TOL["bf16"]["grad"]
        pre = g.clone()
        sid = 2 * (len(dd) + k)
        dp.dpclip_add_noise(g, sigma, C, seed, sid)
        xi = oracle.normals(d, seed, sid)
        assert np.max(np.abs((g - pre).cpu().numpy() - sigma * C * xi)) <= 1e-5 * sigma * C + 1e-6
    assert dp.dpclip_read_status(ws) == 0


# ---------------------------------------------------------------------------
# convolution layers given by their input feature map (implicit im2col)
# ---------------------------------------------------------------------------
CONV_CASES = [  # B, C, H, W, k, pad, stride, d_out
    (3, 3, 8, 8, 3, 1, 1, 5), (2, 4, 9, 7, (3, 2), 1, 2, 70), (4, 32, 16, 16, 3, 1, 1, 64), (2, 5, 6, 6, 1, 0, 1, 3),
    (2, 2, 11, 10, 5, 2, 3, 9), (3, 8, 4, 4, 4, 0, 1, 6),
    # large enough for the tensor-core form (fp32, dL/dZ row-major): ragged tiles, stride, rectangular kernel
    (8, 32, 16, 16, 3, 1, 1, 64), (64, 16, 20, 18, (3, 2), 1, 2, 72), (3, 40, 30, 30, 3, 0, 1, 132),
    # shapes the bf16 tensor-core form takes (stride 1, output width 8 .. 64, T % 64 == 0, d_out % 8 == 0, <= 128): three
    # blocks of patch columns with both Zb chunks, more examples than SMs, a rectangular kernel without padding, a 5 x 5
    # kernel with a ragged d_out, a 32 x 32 map
    (5, 64, 8, 8, 3, 1, 1, 128), (160, 4, 8, 8, 3, 1, 1, 16), (3, 6, 10, 8, (3, 1), 0, 1, 24), (2, 8, 16, 16, 5, 2, 1, 40),
    (2, 3, 32, 32, 3, 1, 1, 32),
    # a first layer (27 patch columns, 32 outputs) large enough for the explicit-patch-matrix route in fp32
    (40, 3, 32, 32, 3, 1, 1, 32),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", CONV_CASES)
def test_conv_implicit_im2col(dp, case, dtype):
    """Norms and clipped sums straight from the feature map equal the oracle's on the unfolded patch matrix,
    with dL/dZ in either layout."""
    B, C, H, W, k, pad, stride, d_out = case
    kh, kw = (k, k) if isinstance(k, int) else k
    X, Z = workloads.conv_inputs(17, B, C, H, W, k, pad, stride, d_out, dtype, var_z=0.01)
    A = workloads.im2col(X, k, pad, stride)                      # what Algorithm 3 would build
    tol = TOL[dtype]
    dX, dZ = to_device(X, dtype), to_device(Z, dtype)
    dZcm = dZ.transpose(1, 2).contiguous()                        # [B][d_out][T], the layout of dL/dZ itself
    clip = np.random.default_rng(B).uniform(0.1, 1.0, B).astype(np.float32)
    refW, refb = oracle.clipped_grad(A, Z, clip)
    ws = _ws(dp)
    # with a workspace the library may take the tensor-core form; without one it stays on the fp32-ALU tiles
    # channel-major fp32 layers reach the tensor cores through a row-major copy of dL/dZ in the workspace when it
    # has the room the conv query asks for
    ws_cm = torch.empty(dp.dpclip_conv_workspace_bytes(dX, dZcm, kh, kw, stride, pad, True), dtype=torch.uint8, device="cuda")
    dp.dpclip_workspace_init(ws_cm)
    variants = [(False, dZ, ws), (False, dZ, None), (True, dZcm, ws)]
    if ws_cm.numel() > ws.numel():
        variants.append((True, dZcm, ws_cm))
    for cm, z, w in variants:
        for has_bias in (True, False):
            ref = oracle.layer_sqnorms(A, Z, has_bias)
            sq = torch.full((B,), -1.0, device="cuda")
            dp.dpclip_conv_sqnorms(dX, z, kh, kw, stride, pad, has_bias, sq, z_channel_major=cm, workspace=w)
            assert max_rel(np.sqrt(sq.cpu().numpy()), np.sqrt(ref)) <= tol["norm"], (cm, w is None, has_bias)
        gW = torch.full((d_out, C * kh * kw), 3.0, device="cuda"); gb = torch.full((d_out,), 3.0, device="cuda")
        dp.dpclip_conv_clipped_grad(dX, z, kh, kw, stride, pad, torch.from_numpy(clip).cuda(), gW, gb,
                                    z_channel_major=cm, workspace=w)
        assert rel_fro(gW.cpu().numpy(), refW) <= tol["grad"] and rel_fro(gb.cpu().numpy(), refb) <= tol["grad"]
        gW.fill_(3.0)
        dp.dpclip_conv_clipped_grad(dX, z, kh, kw, stride, pad, None, gW, None, z_channel_major=cm, workspace=w)
        assert rel_fro(gW.cpu().numpy(), oracle.clipped_grad(A, Z, None)[0]) <= tol["grad"]
    assert dp.dpclip_read_status(ws) == 0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_model_step_mixed_layer_kinds(dp, dtype):
    """One dpclip_model_step call over a convolution given by its feature map (channel-major dL/dZ), a
    LayerNorm's gain and shift, a sequence layer and a T = 1 head: row l of the norms, the factors over all
    layers, clipped sums and the noise streams 2l / 2l + 1 equal the oracle's, layer kind by layer kind."""
    B, C, sigma, seed, sid0 = 7, 1.0, 0.6, 21, 4
    cin, H, W, k, pad, stride, cout = 3, 8, 8, 3, 1, 1, 16
    X, Zc = workloads.conv_inputs(5, B, cin, H, W, k, pad, stride, cout, dtype, var_z=0.02)
    Ac = workloads.im2col(X, k, pad, stride)
    Hn, Zn = workloads.layernorm_pair(6, B, 12, 48, dtype, var_z=0.01)
    rng = np.random.default_rng(8)
    rnd = (lambda a: workloads.round_to_bf16(a.astype(np.float32))) if dtype == "bf16" else (lambda a: a.astype(np.float32))
    As, Zs = rnd(rng.standard_normal((B, 12, 48))), rnd(rng.standard_normal((B, 12, 40)) * 0.1)
    A1, Z1 = rnd(rng.standard_normal((B, 1, 40))), rnd(rng.standard_normal((B, 1, 10)) * 0.5)
    sq_ref = np.stack([oracle.layer_sqnorms(Ac, Zc, True), oracle.elementwise_sqnorms(Hn, Zn, True),
                       oracle.layer_sqnorms(As, Zs, True), oracle.layer_sqnorms(A1, Z1, False)])
    # rescale dL/dZ per example so that the norms straddle C (both sides of the threshold occur)
    n0, _ = oracle.factors(sq_ref, C)
    r = (workloads.spread_factors(B, 1) * C / n0)
    sc = lambda Z: rnd(Z.astype(np.float64) * r.reshape((B,) + (1,) * (Z.ndim - 1)))          # noqa: E731
    Zc, Zn, Zs, Z1 = sc(Zc), sc(Zn), sc(Zs), sc(Z1)
    sq_ref = np.stack([oracle.layer_sqnorms(Ac, Zc, True), oracle.elementwise_sqnorms(Hn, Zn, True),
                       oracle.layer_sqnorms(As, Zs, True), oracle.layer_sqnorms(A1, Z1, False)])
    norms_ref, clip_ref = oracle.factors(sq_ref, C)
    assert 0 < (clip_ref < 1).sum() < B
    ref = [oracle.clipped_grad(Ac, Zc, clip_ref), oracle.elementwise_clipped_grad(Hn, Zn, clip_ref),
           oracle.clipped_grad(As, Zs, clip_ref), (oracle.clipped_grad(A1, Z1, clip_ref)[0], None)]
    dZc = to_device(Zc, dtype).transpose(1, 2).contiguous()          # [B][d_out][T]
    plan = dp.ModelPlan([
        dp.ModelLayer(dp.DPCLIP_KIND_CONV, to_device(X, dtype), dZc, True, conv=(k, k, stride, pad), z_channel_major=True),
        dp.ModelLayer(dp.DPCLIP_KIND_ELEMENTWISE, to_device(Hn, dtype), to_device(Zn, dtype), True),
        dp.ModelLayer(dp.DPCLIP_KIND_DENSE, to_device(As, dtype), to_device(Zs, dtype), True),
        dp.ModelLayer(dp.DPCLIP_KIND_DENSE, to_device(A1, dtype), to_device(Z1, dtype), False)])
    tol = TOL[dtype]
    for sg in (0.0, sigma):
        plan.flat.fill_(float("nan"))
        plan.run(C, sg, seed, sid0)
        torch.cuda.synchronize()
        assert dp.dpclip_read_status(plan.workspace) == 0
        assert max_rel(np.sqrt(plan.sq_layers.cpu().numpy()), np.sqrt(sq_ref)) <= tol["norm"]
        assert max_rel(plan.norms.cpu().numpy(), norms_ref) <= tol["norm"]
        check_saturation(plan.clip.cpu().numpy(), norms_ref, clip_ref, C)
        for l, (rW, rb) in enumerate(ref):
            eW = oracle.add_noise(rW.reshape(-1), sg, C, seed, sid0 + 2 * l).reshape(rW.shape)
            assert plan.gW[l].shape == rW.shape
            assert rel_fro(plan.gW[l].cpu().numpy(), eW) <= tol["grad"], (sg, l)
            if rb is not None:
                eb = oracle.add_noise(rb, sg, C, seed, sid0 + 2 * l + 1)
                assert rel_fro(plan.gb[l].cpu().numpy(), eb) <= tol["grad"], (sg, l)
            else:
                assert plan.gb[l] is None
    # the same path recorded as per-layer calls on three streams
    eager = [t.clone() for t in plan.gW] + [plan.clip.clone()]
    graph = plan.capture(C, sigma, seed, sid0, branches=3)
    plan.flat.fill_(float("nan")); plan.clip.fill_(float("nan"))
    graph.replay(); graph.replay()
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    assert np.allclose(plan.clip.cpu().numpy(), eager[-1].cpu().numpy(), rtol=2e-6, atol=0)
    for l in range(plan.L):
        assert rel_fro(plan.gW[l].cpu().numpy(), eager[l].cpu().numpy()) <= 2e-6, l
    # the data-parallel wrapper on one rank: the model step without noise, then the noise per tensor
    from paper_2009_03106_b200 import parallel
    plan.flat.fill_(float("nan"))
    parallel.sharded_step(plan, C, sigma, seed, sid0)
    torch.cuda.synchronize()
    for l in range(plan.L):
        assert rel_fro(plan.gW[l].cpu().numpy(), eager[l].cpu().numpy()) <= 2e-6, l
    # a model of dense layers only is dpclip_step
    dense = [dp.ModelLayer(dp.DPCLIP_KIND_DENSE, to_device(As, dtype), to_device(Zs, dtype), True),
             dp.ModelLayer(dp.DPCLIP_KIND_DENSE, to_device(A1, dtype), to_device(Z1, dtype), False)]
    mp = dp.ModelPlan(dense); mp.run(C, sigma, seed, sid0)
    sp = dp.StepPlan([dp.Layer(y.A, y.Zbar, y.has_bias) for y in dense]); sp.run(C, sigma, seed, sid0)
    torch.cuda.synchronize()
    assert torch.equal(mp.clip, sp.clip)
    for l in range(2):
        assert torch.equal(mp.gW[l], sp.gW[l])


# ---------------------------------------------------------------------------
# (c) factors
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("B,L", [(1, 1), (32, 2), (128, 3), (1024, 7), (1500, 2)])
def test_factors(dp, B, L):
    rng = np.random.default_rng(B + L)
    sq = (rng.uniform(0.0, 2.0, (L, B)) ** 2).astype(np.float32)
    sq[:, 0] = 0.0
    C = 1.5
    if B > 4:
        sq[:, 1] = 0.0; sq[0, 1] = np.float32(C * C)                  # exactly on the threshold: not clipped
        sq[:, 2] = 0.0; sq[0, 2] = np.float32(C * C * (1 + 3e-5))     # inside the band
    norms_ref, clip_ref = oracle.factors(sq, C)
    d_sq = torch.from_numpy(sq).cuda()
    clip = torch.empty(B, device="cuda"); norms = torch.empty(B, device="cuda")
    cnt = torch.full((1,), -5, dtype=torch.int32, device="cuda")
    dp.dpclip_factors(d_sq, C, clip, norms, cnt)
    clip, norms = clip.cpu().numpy(), norms.cpu().numpy()
    assert max_rel(norms, norms_ref) <= 1e-6
    assert np.max(np.abs(clip - clip_ref)) <= 1e-6
    check_saturation(clip, norms_ref, clip_ref, C)
    assert clip[0] == 1.0
    if B > 4:
        assert clip[1] == 1.0
    assert int(cnt.item()) == int((clip < 1.0).sum())
    assert np.all(clip.astype(np.float64) * norms_ref <= C * (1 + 1e-6))
    # optional outputs may be omitted
    clip2 = torch.empty(B, device="cuda")
    dp.dpclip_factors(d_sq, C, clip2)
    assert np.array_equal(clip2.cpu().numpy(), clip)


# ---------------------------------------------------------------------------
# (d) clipped sum
# ---------------------------------------------------------------------------
GRAD_SHAPES = [(1, 1, 1, 1), (32, 1, 784, 256), (128, 1, 1000, 10), (7, 1, 129, 65)] + SIMT_SHAPES


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,T,d_in,d_out", GRAD_SHAPES)
def test_clipped_grad(dp, dtype, B, T, d_in, d_out):
    A, Z = workloads.random_layer(4, B, T, d_in, d_out, dtype, scale_z=0.05)
    clip = np.random.default_rng(B).uniform(0.05, 1.0, B).astype(np.float32)
    clip[::3] = 1.0
    refW, refb = oracle.clipped_grad(A, Z, clip)
    dA, dZ = to_device(A, dtype), to_device(Z, dtype)
    guard_W, guard_b = Guarded(d_out, d_in), Guarded(d_out)
    gW, gb = guard_W.t, guard_b.t
    ws = _ws(dp)
    dp.dpclip_clipped_grad(dA, dZ, torch.from_numpy(clip).cuda(), gW, gb, ws)
    guard_W.check(); guard_b.check()
    # identical inputs and fp32 accumulation: the fp32 bound applies, except on the tensor-core path,
    # which rounds clip*zbar to bf16 in shared memory (bf16 rows that are 16-byte multiples take it)
    narrow = T > 1 and d_in + 1 <= 32 and d_out <= 64
    on_tc = dtype == "bf16" and ((d_in % 8 == 0 and d_out % 8 == 0) or narrow)
    tol = TOL["bf16"]["grad"] if on_tc else TOL["f32"]["grad"]
    assert rel_fro(gW.cpu().numpy(), refW) <= tol
    assert rel_fro(gb.cpu().numpy(), refb) <= tol
    # clip = NULL: plain batch gradient; gb = NULL: weights only; padded output rows stay untouched
    refW1, _ = oracle.clipped_grad(A, Z, None)
    wide = torch.full((d_out, d_in + 3), 9.0, device="cuda")
    dp.dpclip_clipped_grad(dA, dZ, None, wide[:, :d_in], None, ws)
    assert rel_fro(wide[:, :d_in].cpu().numpy(), refW1) <= 2e-5       # no factor, no rounding: exact products
    assert torch.all(wide[:, d_in:] == 9.0)
    assert dp.dpclip_read_status(ws) == 0


@pytest.mark.parametrize("dtype,B,T,d_in,d_out", [("bf16", 8, 256, 512, 256), ("f32", 6, 17, 27, 33),
                                                  ("bf16", 128, 1, 512, 256)])
def test_clipped_grad_noise_equals_separate_calls(dp, dtype, B, T, d_in, d_out):
    A, Z = workloads.random_layer(9, B, T, d_in, d_out, dtype, scale_z=0.05)
    clip = torch.from_numpy(np.random.default_rng(1).uniform(0.2, 1.0, B).astype(np.float32)).cuda()
    dA, dZ = to_device(A, dtype), to_device(Z, dtype)
    ws = _ws(dp)
    W1 = torch.empty((d_out, d_in), device="cuda"); b1 = torch.empty(d_out, device="cuda")
    dp.dpclip_clipped_grad(dA, dZ, clip, W1, b1, ws)
    dp.dpclip_add_noise(W1.view(-1), 0.9, 1.3, 77, 4)
    dp.dpclip_add_noise(b1, 0.9, 1.3, 77, 5)
    W2 = torch.empty((d_out, d_in), device="cuda"); b2 = torch.empty(d_out, device="cuda")
    dp.dpclip_clipped_grad_noise(dA, dZ, clip, W2, b2, 0.9, 1.3, 77, 4, 5, ws)
    if dtype == "bf16":       # deterministic tensor-core path: identical bits
        assert torch.equal(W1, W2) and torch.equal(b1, b2)
    else:                     # fp32-ALU path combines row slices with atomics
        assert rel_fro(W2.cpu().numpy(), W1.cpu().numpy()) <= 1e-6


# ---------------------------------------------------------------------------
# (e) noise
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("n", [1, 3, 4, 5, 1023, 4096, 100003])
def test_noise_matches_oracle(dp, n):
    sigma, C, seed, sid = 1.1, 0.7, 0x123456789ABCDEF, (1 << 40) + 5
    base = np.random.default_rng(n).standard_normal(n).astype(np.float32)
    guard = Guarded(n)
    g = guard.t
    g.copy_(torch.from_numpy(base))
    dp.dpclip_add_noise(g, sigma, C, seed, sid)
    guard.check()
    ref = oracle.add_noise(base, sigma, C, seed, sid)
    assert np.max(np.abs(g.cpu().numpy() - ref)) <= 1e-5 * sigma * C + 1e-6 * np.max(np.abs(ref))
    # noise-only tensor, and an output that does not start on a 16-byte boundary
    buf = torch.zeros(n + 1, device="cuda")
    dp.dpclip_add_noise(buf[1:], 1.0, 1.0, seed, sid)
    xi = oracle.normals(n, seed, sid)
    assert np.max(np.abs(buf[1:].cpu().numpy() - xi)) <= 1e-5
    assert buf[0].item() == 0.0


def test_step_noise_equals_per_tensor_noise(dp):
    """One launch for all tensors of a model gives bit for bit what one dpclip_add_noise call per tensor gives."""
    w = workloads.cnn("f32")
    layers = workloads.generate(w, 0, examples=2)
    mk = lambda: dp.StepPlan([dp.Layer(to_device(A, "f32"), to_device(Z, "f32"), s.has_bias)     # noqa: E731
                              for (A, Z), s in zip(layers, w.layers)])
    a, b = mk(), mk()
    dp.dpclip_step_noise(a, 0.7, 1.3, 99, 6)
    for l in range(len(layers)):
        dp.dpclip_add_noise(b.gW[l].view(-1), 1.3, 0.7, 99, 6 + 2 * l)
        dp.dpclip_add_noise(b.gb[l], 1.3, 0.7, 99, 6 + 2 * l + 1)
    torch.cuda.synchronize()
    for l in range(len(layers)):
        assert torch.equal(a.gW[l], b.gW[l]) and torch.equal(a.gb[l], b.gb[l])
        assert float(a.gW[l].abs().max()) > 0


@pytest.mark.parametrize("n", [1, 5, 4096, 100003])
def test_dp_sgd_and_adam_steps(dp, n):
    """Parameter updates with the noise folded in (Algorithm 1's last line; the private Adam of the
    experiments) against the oracle, over several steps so that the moments carry over."""
    rng = np.random.default_rng(n)
    # both sides start from the same (fp32-representable) hyper-parameters: 1 - 0.999 differs by 1.3e-5 between
    # the fp32 and the fp64 reading of 0.999
    tau, C, sigma, lr, b1, b2, eps = (128, 1.0, float(np.float32(1.1)), float(np.float32(1e-3)), float(np.float32(0.9)),
                                      float(np.float32(0.999)), float(np.float32(1e-8)))
    th0 = rng.standard_normal(n).astype(np.float32)
    # SGD
    gsum = (rng.standard_normal(n) * 5).astype(np.float32)
    th = torch.from_numpy(th0.copy()).cuda()
    dp.dpclip_dp_sgd_step(th, torch.from_numpy(gsum).cuda(), 1.0 / tau, C, sigma, 7, 11, 0.05)
    ref = oracle.dp_sgd_step(th0, gsum, 1.0 / tau, C, sigma, 7, 11, 0.05)
    assert np.max(np.abs(th.cpu().numpy() - ref)) <= 1e-5 * 0.05 + 2e-7 * np.max(np.abs(ref))
    # Adam, 3 steps
    th = torch.from_numpy(th0.copy()).cuda(); m = torch.zeros(n, device="cuda"); v = torch.zeros(n, device="cuda")
    rth, rm, rv = th0.astype(np.float64), np.zeros(n), np.zeros(n)
    for t in range(1, 4):
        gsum = (rng.standard_normal(n) * 5).astype(np.float32)
        dp.dpclip_dp_adam_step(th, m, v, torch.from_numpy(gsum).cuda(), 1.0 / tau, C, sigma, 7, 20 + t, lr, b1, b2, eps, t)
        rth, rm, rv = oracle.dp_adam_step(rth, rm, rv, gsum, 1.0 / tau, C, sigma, 7, 20 + t, lr, b1, b2, eps, t)
        # the moments are sums of terms of either sign: the error scales with the terms (|g| ~ 5 / tau), not with
        # what is left of them
        gs = 5.0 / tau
        assert np.max(np.abs(m.cpu().numpy() - rm)) <= 1e-5 * np.max(np.abs(rm)) + 1e-6 * gs
        assert np.max(np.abs(v.cpu().numpy() - rv)) <= 1e-5 * np.max(np.abs(rv)) + 1e-6 * gs * gs
        assert np.max(np.abs(th.cpu().numpy() - rth)) <= 1e-4 * lr + 2e-7 * np.max(np.abs(rth))
    # sigma = 0 draws nothing: plain optimiser
    th = torch.ones(n, device="cuda"); g = torch.full((n,), 2.0, device="cuda")
    dp.dpclip_dp_sgd_step(th, g, 0.5, 1.0, 0.0, 1, 1, 0.1)
    assert torch.allclose(th, torch.full((n,), 0.9, device="cuda"), rtol=1e-6)


def test_noise_is_stateless_and_stream_dependent(dp):
    n = 10007
    a = torch.zeros(n, device="cuda"); b = torch.zeros(n, device="cuda"); c = torch.zeros(n, device="cuda")
    dp.dpclip_add_noise(a, 1.0, 1.0, 7, 0)
    dp.dpclip_add_noise(b, 1.0, 1.0, 7, 0)
    dp.dpclip_add_noise(c, 1.0, 1.0, 7, 1)
    assert torch.equal(a, b)
    assert abs(np.corrcoef(a.cpu().numpy(), c.cpu().numpy())[0, 1]) < 0.05
    z = torch.ones(n, device="cuda")
    dp.dpclip_add_noise(z, 0.0, 1.0, 7, 0)
    assert torch.all(z == 1.0)


# ---------------------------------------------------------------------------
# whole step on the paper-shaped workloads
# ---------------------------------------------------------------------------
def _calibrate(w, layers, seed, C):
    """Spread per-example norms around C (the stated distributions put every
    norm far above it): scale example i's Zbar rows, in every layer, by
    r_i * C / median norm, r_i log-uniform on [1/8, 8]; a few examples are put
    within 1e-3 of the threshold."""
    hb = [l.has_bias for l in w.layers]
    sq = np.stack([oracle.layer_sqnorms(A, Z, b) for (A, Z), b in zip(layers, hb)])
    n, _ = oracle.factors(sq, C)
    r = workloads.spread_factors(len(n), seed)
    r[:3] = [1.0005, 0.9995, 1.0]
    s = r * C / n
    out = []
    for (A, Z) in layers:
        Zs = (Z.astype(np.float64) * s[:, None, None]).astype(np.float32)
        if w.dtype == "bf16":
            Zs = workloads.round_to_bf16(Zs)
        out.append((A, Zs))
    return out


def _run_step(dp, w, layers, C, sigma, seed, methods=None):
    dls = [dp.Layer(to_device(A, w.dtype), to_device(Z, w.dtype), spec.has_bias,
                    methods[i] if methods else dp.DPCLIP_AUTO)
           for i, ((A, Z), spec) in enumerate(zip(layers, w.layers))]
    plan = dp.StepPlan(dls)
    plan.run(C, sigma, seed, 0)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    return plan


def _check_step(dp, w, layers, C, sigma, seed):
    hb = [l.has_bias for l in w.layers]
    tol = TOL[w.dtype]
    ref = oracle.step(layers, hb, C, sigma, seed, 0)
    pre = _run_step(dp, w, layers, C, 0.0, seed)            # sigma = 0: the pre-noise gradient
    assert max_rel(np.sqrt(pre.sq_layers.cpu().numpy()), np.sqrt(ref["sq_layers"])) <= tol["norm"]
    assert max_rel(pre.norms.cpu().numpy(), ref["norms"]) <= tol["norm"]
    clip = pre.clip.cpu().numpy()
    check_saturation(clip, ref["norms"], ref["clip"], C)
    assert np.max(np.abs(clip - ref["clip"]) / ref["clip"]) <= max(tol["norm"], 2 * SAT_BAND)
    got_all, ref_all = [], []
    for l in range(len(layers)):
        gw = pre.gW[l].cpu().numpy()
        assert rel_fro(gw, ref["gW"][l]) <= tol["grad"], (l, rel_fro(gw, ref["gW"][l]))
        got_all.append(gw.ravel()); ref_all.append(ref["gW"][l].ravel())
        if hb[l]:
            gb = pre.gb[l].cpu().numpy()
            assert rel_fro(gb, ref["gb"][l]) <= tol["grad"]
            got_all.append(gb); ref_all.append(ref["gb"][l])
    assert rel_fro(np.concatenate(got_all), np.concatenate(ref_all)) <= tol["grad"]
    # every clipped per-example contribution is within C
    assert np.all(clip.astype(np.float64) * ref["norms"] <= C * (1 + 1e-4))
    # with noise: final output = pre-noise + sigma*C*xi, checked against the oracle's noised tensors
    post = _run_step(dp, w, layers, C, sigma, seed)
    for l in range(len(layers)):
        d = post.gW[l].cpu().numpy().astype(np.float64) - pre.gW[l].cpu().numpy()
        xi = (ref["outW"][l] - ref["gW"][l])
        assert np.max(np.abs(d - xi)) <= 1e-5 * sigma * C + 4e-7 * np.max(np.abs(ref["outW"][l]))
        if hb[l]:
            d = post.gb[l].cpu().numpy().astype(np.float64) - pre.gb[l].cpu().numpy()
            xi = (ref["outb"][l] - ref["gb"][l])
            assert np.max(np.abs(d - xi)) <= 1e-5 * sigma * C + 4e-7 * np.max(np.abs(ref["outb"][l]))
    return ref, pre


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_step_mlp_small(dp, seed):
    w = workloads.mlp_small()
    layers = workloads.generate(w, seed)
    _check_step(dp, w, layers, w.C, w.sigma, seed)
    ref, _ = _check_step(dp, w, _calibrate(w, layers, seed, w.C), w.C, w.sigma, seed)
    assert 0 < (ref["clip"] < 1).sum() < w.B


@pytest.mark.parametrize("C", [0.1, 1.0, 10.0])
def test_step_mlp_large(dp, C):
    w = workloads.mlp_large(C=C)
    layers = workloads.generate(w, 0)
    _check_step(dp, w, layers, C, w.sigma, 0)
    # calibrated at C = 1: about all / half / none of the examples are clipped at 0.1 / 1 / 10
    cal = _calibrate(w, layers, 0, 1.0)
    ref, _ = _check_step(dp, w, cal, C, w.sigma, 0)
    frac = (ref["clip"] < 1).mean()
    assert {0.1: frac > 0.9, 1.0: 0.3 < frac < 0.7, 10.0: frac < 0.1}[C]


def test_step_mlp_per_layer_path(dp, path_switch):
    """The general per-layer path on an all-T=1 model (the fused two-launch path is switched off)."""
    path_switch("DPCLIP_NO_FUSED_T1", "1")
    w = workloads.mlp_large(C=1.0)
    layers = workloads.generate(w, 1)
    _check_step(dp, w, _calibrate(w, layers, 1, 1.0), 1.0, w.sigma, 1)


def test_step_mlp_bf16_and_odd_widths(dp):
    """Fused T=1 step with bf16 inputs, and with widths that are not multiples of 4 (scalar paths)."""
    w = workloads.mlp_small("bf16")
    layers = workloads.generate(w, 0)
    _check_step(dp, w, _calibrate(w, layers, 0, w.C), w.C, w.sigma, 0)
    odd = workloads.Workload("mlp_odd", 9, "f32",
                             (workloads.LayerSpec("fc1", 1, 131, 67, True, "normal"),
                              workloads.LayerSpec("fc2", 1, 67, 5, False, "relu"),
                              workloads.LayerSpec("fc3", 1, 5, 1, True, "relu")), 1.0, 0.7, 1.0 / 9)
    layers = workloads.generate(odd, 3)
    _check_step(dp, odd, _calibrate(odd, layers, 3, odd.C), odd.C, odd.sigma, 3)


def test_step_mlp_tensor_core_edges(dp):
    """Fused T=1 step on the tensor cores (fp32, rows TMA can address): a batch that is not a multiple of
    the 32-row stage and spans two accumulation windows, ragged tiles, a layer without bias, a thin head."""
    w = workloads.Workload("mlp_tc_edges", 200, "f32",
                           (workloads.LayerSpec("fc1", 1, 132, 260, True, "normal"),
                            workloads.LayerSpec("fc2", 1, 260, 36, False, "relu"),
                            workloads.LayerSpec("fc3", 1, 36, 16, True, "relu"),
                            workloads.LayerSpec("fc4", 1, 16, 3, True, "relu")), 1.0, 0.9, 1.0 / 200)
    layers = workloads.generate(w, 5)
    _check_step(dp, w, _calibrate(w, layers, 5, w.C), w.C, w.sigma, 5)
    # more output tiles (13 x 12 + 1 x 13 = 169) than SMs: every CTA of the one-launch kernel walks several
    # items, so the stage ring, the two accumulator buffers and the noise drawing carry over between items
    big = workloads.Workload("mlp_tc_many_tiles", 48, "f32",
                             (workloads.LayerSpec("fc1", 1, 1536, 1664, True, "normal"),
                              workloads.LayerSpec("fc2", 1, 1664, 12, True, "relu")), 1.0, 0.9, 1.0 / 48)
    layers = workloads.generate(big, 6)
    _check_step(dp, big, _calibrate(big, layers, 6, big.C), big.C, big.sigma, 6)


def test_step_mlp_bf16_tensor_core(dp, path_switch):
    """Fused T=1 step on the tensor cores with bf16 inputs (one kind::f16 instruction per 16 rows, no low
    planes): the paper-shaped MLPs, ragged tiles with a bias-free layer and a thin head, more tiles than SMs,
    and the two-launch form."""
    for w, seed in ((workloads.mlp_small("bf16"), 2), (workloads.mlp_large("bf16", C=1.0), 3)):
        layers = workloads.generate(w, seed)
        _check_step(dp, w, _calibrate(w, layers, seed, w.C), w.C, w.sigma, seed)
    edges = workloads.Workload("mlp_tc_edges_bf16", 200, "bf16",
                               (workloads.LayerSpec("fc1", 1, 136, 264, True, "normal"),
                                workloads.LayerSpec("fc2", 1, 264, 40, False, "relu"),
                                workloads.LayerSpec("fc3", 1, 40, 16, True, "relu"),
                                workloads.LayerSpec("fc4", 1, 16, 3, True, "relu")), 1.0, 0.9, 1.0 / 200)
    layers = workloads.generate(edges, 5)
    _check_step(dp, edges, _calibrate(edges, layers, 5, edges.C), edges.C, edges.sigma, 5)
    big = workloads.Workload("mlp_tc_many_tiles_bf16", 48, "bf16",
                             (workloads.LayerSpec("fc1", 1, 1536, 1664, True, "normal"),
                              workloads.LayerSpec("fc2", 1, 1664, 12, True, "relu")), 1.0, 0.9, 1.0 / 48)
    layers = workloads.generate(big, 6)
    _check_step(dp, big, _calibrate(big, layers, 6, big.C), big.C, big.sigma, 6)
    path_switch("DPCLIP_T1_ONE_LAUNCH", "0")
    layers = workloads.generate(edges, 7)
    _check_step(dp, edges, _calibrate(edges, layers, 7, edges.C), edges.C, edges.sigma, 7)


NARROW_TC_SHAPES = [(128, 1024, 27, 32),      # the first convolution of the CNN: aligned 32-row blocks, vector loads
                    (3, 100, 27, 32),         # item starts off the 16-byte grid: element-wise loads
                    (5, 72, 27, 32),          # aligned, a ragged last block (72 = 2 * 32 + 8)
                    (300, 64, 24, 64),        # more examples than SMs (several items per CTA), both lane quarters
                    (4, 40, 31, 40), (2, 33, 5, 3), (7, 2, 1, 1)]


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("B,T,d_in,d_out", NARROW_TC_SHAPES)
@pytest.mark.parametrize("has_bias", [True, False])
def test_narrow_layers_tensor_core(dp, B, T, d_in, d_out, has_bias, dtype):
    """Narrow layers on the tensor cores: raw chunks re-arranged into operand tiles in shared memory, four 16-row
    groups per instruction for d_out <= 32 (bf16 and fp32 as error-compensated tf32), one group for bf16 up to 64
    outputs.  Norms see exact products; the bf16 clipped sum rounds c * zb once to bf16."""
    A, Z = workloads.random_layer(60, B, T, d_in, d_out, dtype, scale_z=0.05)
    n = min(B, 12)                                            # the oracle materialises every example: sample
    idx = np.unique(np.concatenate([np.arange(min(n, B)), np.arange(max(0, B - 3), B), [B // 2]]))
    ref = oracle.layer_sqnorms(A[idx], Z[idx], has_bias)
    got = _sqnorms(dp, A, Z, dtype, has_bias)
    assert max_rel(np.sqrt(got[idx]), np.sqrt(ref)) <= TOL["f32"]["norm"]
    clip = np.random.default_rng(B).uniform(0.05, 1.0, B).astype(np.float32)
    clip[::3] = 1.0
    refW, refb = oracle.clipped_grad(A, Z, clip)
    gW = torch.full((d_out, d_in), 9.0, device="cuda")
    gb = torch.full((d_out,), 9.0, device="cuda") if has_bias else None
    ws = _ws(dp)
    dp.dpclip_clipped_grad(to_device(A, dtype), to_device(Z, dtype), torch.from_numpy(clip).cuda(), gW, gb, ws)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(ws) == 0
    assert rel_fro(gW.cpu().numpy(), refW) <= TOL[dtype]["grad"]
    if has_bias:
        assert rel_fro(gb.cpu().numpy(), refb) <= TOL[dtype]["grad"]
    # no factors: exact products, fp32 accumulation
    refW1, _ = oracle.clipped_grad(A, Z, None)
    dp.dpclip_clipped_grad(to_device(A, dtype), to_device(Z, dtype), None, gW, gb, ws)
    assert rel_fro(gW.cpu().numpy(), refW1) <= 2e-5


def test_narrow_packed_kernel_bf16(dp, path_switch):
    """The four-groups-per-instruction kernel with bf16 operands (fp32 layers take it by default, bf16 layers
    only on request)."""
    path_switch("DPCLIP_NARROW_PACK_BF16", "1")
    B, T, d_in, d_out = 150, 136, 27, 32
    A, Z = workloads.random_layer(61, B, T, d_in, d_out, "bf16", scale_z=0.05)
    idx = np.array([0, 1, 74, 149])
    got = _sqnorms(dp, A, Z, "bf16", True)
    assert max_rel(np.sqrt(got[idx]), np.sqrt(oracle.layer_sqnorms(A[idx], Z[idx], True))) <= TOL["f32"]["norm"]
    clip = np.random.default_rng(3).uniform(0.05, 1.0, B).astype(np.float32)
    refW, refb = oracle.clipped_grad(A, Z, clip)
    gW = torch.empty(d_out, d_in, device="cuda"); gb = torch.empty(d_out, device="cuda")
    dp.dpclip_clipped_grad(to_device(A, "bf16"), to_device(Z, "bf16"), torch.from_numpy(clip).cuda(), gW, gb, _ws(dp))
    assert rel_fro(gW.cpu().numpy(), refW) <= TOL["bf16"]["grad"] and rel_fro(gb.cpu().numpy(), refb) <= TOL["bf16"]["grad"]


def test_narrow_layer_register_staged_form(dp, path_switch):
    """fp32 narrow layers normally take the cp.async ring kernel; the register-staged kernel (what bf16 and
    unaligned layers use) must give the same norms and clipped sums on the same fp32 input."""
    path_switch("DPCLIP_NO_NARROW_RING", "1")
    B, T, d_in, d_out = 5, 200, 27, 32
    A, Z = workloads.random_layer(33, B, T, d_in, d_out, "f32", scale_z=0.05)
    ref = oracle.layer_sqnorms(A, Z, True)
    got = _sqnorms(dp, A, Z, "f32", True)
    assert max_rel(np.sqrt(got), np.sqrt(ref)) <= TOL["f32"]["norm"]
    clip = np.random.default_rng(1).uniform(0.1, 1.0, B).astype(np.float32)
    refW, refb = oracle.clipped_grad(A, Z, clip)
    gW = torch.empty(d_out, d_in, device="cuda"); gb = torch.empty(d_out, device="cuda")
    dp.dpclip_clipped_grad(to_device(A, "f32"), to_device(Z, "f32"), torch.from_numpy(clip).cuda(), gW, gb, _ws(dp))
    assert rel_fro(gW.cpu().numpy(), refW) <= TOL["f32"]["grad"] and rel_fro(gb.cpu().numpy(), refb) <= TOL["f32"]["grad"]


def test_step_mlp_fp32_alu_kernel(dp, path_switch):
    """The fp32-ALU second launch of the fused step (what models the tensor-core launch rejects fall back to)."""
    path_switch("DPCLIP_NO_T1_TF32", "1")
    w = workloads.mlp_small()
    layers = workloads.generate(w, 4)
    _check_step(dp, w, _calibrate(w, layers, 4, w.C), w.C, w.sigma, 4)


def test_step_mlp_padded_rows(dp):
    """Input rows padded to a 16-byte stride with a width that is not a multiple of 4: tensor-core launch,
    element-wise noise and store paths."""
    B, d_in, d_out, C, sigma, seed = 70, 130, 72, 1.0, 0.8, 11
    A, Z = workloads.random_layer(21, B, 1, d_in, d_out, "f32", scale_z=0.05)
    hb = [True]
    ref = oracle.step([(A, Z)], hb, C, sigma, seed, 0)
    Ap = torch.zeros(B, 1, 132, device="cuda"); Ap[:, :, :d_in] = torch.from_numpy(A).cuda()
    plan = dp.StepPlan([dp.Layer(Ap[:, :, :d_in], to_device(Z, "f32"), True)])
    plan.run(C, sigma, seed, 0)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    assert max_rel(plan.norms.cpu().numpy(), ref["norms"]) <= TOL["f32"]["norm"]
    assert rel_fro(plan.gW[0].cpu().numpy(), ref["outW"][0]) <= TOL["f32"]["grad"]
    assert rel_fro(plan.gb[0].cpu().numpy(), ref["outb"][0]) <= TOL["f32"]["grad"]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_step_cnn(dp, dtype):
    w = workloads.cnn(dtype)
    layers = workloads.generate(w, 0)
    _check_step(dp, w, layers, w.C, w.sigma, 0)
    _check_step(dp, w, _calibrate(w, layers, 1, w.C), w.C, w.sigma, 1)


def test_step_seq_small(dp):
    """The sequence-model layer mix at a size the oracle finishes in seconds."""
    w = workloads.seq("bf16", B=6, T=40, d=64, d_ff=136)
    layers = workloads.generate(w, 0)
    _check_step(dp, w, layers, w.C, w.sigma, 0)
    _check_step(dp, w, _calibrate(w, layers, 2, w.C), w.C, w.sigma, 2)


def test_gram_layers_in_one_launch(dp):
    """Gram-identity norms of several layers in one launch: examples of one, two and three 128-row blocks,
    examples that share a block, ragged lengths, with and without bias, more layers than one launch takes;
    every row of sq equals the oracle's, layers the entry point does not take are reported as such."""
    B = 3
    shapes = [(256, 64, 136, True), (128, 72, 64, False), (64, 64, 64, True), (256, 136, 64, False),   # two-block and shorter examples
              (100, 64, 72, True), (384, 64, 64, False), (40, 136, 64, True)]                            # the rest
    shapes += [(64, 64, 8 * k, bool(k & 1)) for k in range(1, 9)]          # 10 layers of one-or-two-block examples: two launches
    data = [workloads.random_layer(50 + i, B, T, d_in, d_out, "bf16", scale_z=0.05) for i, (T, d_in, d_out, _) in enumerate(shapes)]
    layers = [dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), hb, dp.DPCLIP_GRAM) for (A, Z), (_, _, _, hb) in zip(data, shapes)]
    # a T = 1 layer, an fp32-ALU layer (rows TMA cannot address) and a lone layer of its class are left alone
    A1, Z1 = workloads.random_layer(90, B, 1, 64, 64, "bf16", scale_z=0.05)
    A2, Z2 = workloads.random_layer(91, B, 24, 27, 64, "bf16", scale_z=0.05)
    layers += [dp.Layer(to_device(A1, "bf16"), to_device(Z1, "bf16"), True),
               dp.Layer(to_device(A2, "bf16"), to_device(Z2, "bf16"), True, dp.DPCLIP_GRAM)]
    plan = dp.StepPlan(layers)
    plan.sq_layers.fill_(float("nan"))
    taken = dp.dpclip_gram_layers_sqnorms(plan)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    assert taken == [True] * len(shapes) + [False, False]
    sq = plan.sq_layers.cpu().numpy()
    for l, ((A, Z), (_, _, _, hb)) in enumerate(zip(data, shapes)):
        ref = oracle.layer_sqnorms(A, Z, hb)
        assert max_rel(np.sqrt(sq[l]), np.sqrt(ref)) <= TOL["bf16"]["norm"], (l, shapes[l])
    assert np.isnan(sq[len(shapes):]).all()
    # one candidate only: nothing is taken
    lone = dp.StepPlan(layers[:1])
    assert dp.dpclip_gram_layers_sqnorms(lone) == [False]


def test_step_factors_in_the_tail_of_the_gram_launch(dp, path_switch):
    """When one Gram launch takes every layer of the model, its last CTA computes the clip factors (no factors
    launch): same bits as the factors kernel (the path with the shared launch switched off), equal to the oracle,
    and repeatable (the CTA counter in the workspace header returns to zero)."""
    w = workloads.seq("bf16", B=40, T=256, d=64, d_ff=136)
    data = workloads.generate(w, 5)
    cal = _calibrate(w, data, 5, w.C)
    mk = lambda: dp.StepPlan([dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), s.has_bias, dp.DPCLIP_GRAM)   # noqa: E731
                              for (A, Z), s in zip(cal, w.layers)])
    plan = mk()
    n0 = dp.dpclip_launch_count()
    plan.run(w.C, 0.0, 3)
    launches_with_tail = dp.dpclip_launch_count() - n0
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    hb = [s.has_bias for s in w.layers]
    sq = np.stack([oracle.layer_sqnorms(A, Z, b) for (A, Z), b in zip(cal, hb)])
    n_ref, c_ref = oracle.factors(sq, w.C)
    assert max_rel(plan.norms.cpu().numpy(), n_ref) <= TOL["bf16"]["norm"]
    check_saturation(plan.clip.cpu().numpy(), n_ref, c_ref, w.C)
    assert 0 < (c_ref < 1).sum() < w.B
    first_clip, first_flat = plan.clip.clone(), plan.flat.clone()
    for _ in range(50):
        plan.clip.fill_(float("nan"))
        plan.run(w.C, 0.0, 3)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    # examples of two row blocks: every norm is stored by its CTA as a fixed-order sum, so repeats give the same bits
    assert torch.equal(plan.clip, first_clip) and torch.equal(plan.flat, first_flat)
    path_switch("DPCLIP_NO_GRAM_GROUP", "1")
    other = mk()
    n0 = dp.dpclip_launch_count()
    other.run(w.C, 0.0, 3)
    assert dp.dpclip_launch_count() - n0 > launches_with_tail          # per-layer norms + a factors launch
    torch.cuda.synchronize()
    assert np.allclose(other.clip.cpu().numpy(), first_clip.cpu().numpy(), rtol=2e-6, atol=0)


@pytest.mark.parametrize("shapes", [
    # three 512 -> 512 layers (2 tiles each) and a 256 -> 1024 layer (2 tiles): gangs of 8, one super-layer
    [(512, 512, False), (512, 512, True), (512, 512, False), (256, 1024, True)],
    # 2 + 2 + 8 tiles: the narrow layers share a super-layer that stays half empty (pairs without a tile)
    [(512, 512, True), (512, 504, False), (512, 2048, True)],
    # 3 + 2 tiles: five tiles side by side in gangs of 5
    [(768, 512, True), (512, 512, False)],
    # 8 + 7 tiles: gangs of 8, the second super-layer has a position without a tile (that pair idles there)
    [(512, 2048, True), (256, 3584, False)],
    # 17 tiles: no gang width divides it -> tile-major runs (W = 1)
    [(256, 8704, True)],
])
def test_wide_layers_of_any_shape_share_one_pair_launch(dp, shapes):
    """Layers wide enough for the CTA-pair kernel share ONE clipped-sum launch whatever their shapes (same T):
    packed into super-layers, runs cut per gang, segments reduced per tile.  Every output against the oracle;
    with noise, the difference to the sigma = 0 result is each layer's own noise stream."""
    B, T = 3, 192                                   # 9 stages per tile: runs of 8 stages cross tile boundaries
    L = workloads.LayerSpec
    specs = tuple(L(f"l{i}", T, d_in, d_out, hb, "normal") for i, (d_in, d_out, hb) in enumerate(shapes))
    w = workloads.Workload("wide_mixed", B, "bf16", specs, 1.0, 0.7, 1.0 / (B * T))
    data = workloads.generate(w, 11)
    plan = dp.StepPlan([dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), s.has_bias) for (A, Z), s in zip(data, specs)])
    clip = np.array([1.0, 0.37, 0.052], np.float32)
    plan.clip.copy_(torch.from_numpy(clip))
    plan.flat.fill_(float("nan"))
    taken = dp.dpclip_same_shape_layers_clipped_grad_noise(plan, 1.0, 0.0, seed=0)
    torch.cuda.synchronize()
    assert (all(taken) or len(shapes) == 1) and dp.dpclip_read_status(plan.workspace) == 0
    if len(shapes) == 1:            # a single layer takes the same kernel through its own entry point
        dp.dpclip_clipped_grad(plan.layers[0].A, plan.layers[0].Zbar, plan.clip, plan.gW[0], plan.gb[0], plan.workspace)
        torch.cuda.synchronize()
    for l, ((A, Z), s) in enumerate(zip(data, specs)):
        refW, refb = oracle.clipped_grad(A, Z, clip)
        assert rel_fro(plan.gW[l].cpu().numpy(), refW) <= TOL["bf16"]["grad"], l
        if s.has_bias:
            assert rel_fro(plan.gb[l].cpu().numpy(), refb) <= 1e-5, l        # bias sums are taken in fp32
    if len(shapes) == 1:
        return
    pre = plan.flat.clone()
    dp.dpclip_same_shape_layers_clipped_grad_noise(plan, 1.3, 0.7, seed=5, stream_id0=40)
    torch.cuda.synchronize()
    for l, s in enumerate(specs):
        xi = oracle.normals(s.d_out * s.d_in, 5, 40 + 2 * l).reshape(s.d_out, s.d_in)
        off = plan.gW[l].data_ptr() - plan.flat.data_ptr()
        base = pre[off // 4: off // 4 + s.d_out * s.d_in].view(s.d_out, s.d_in)
        assert np.max(np.abs((plan.gW[l] - base).cpu().numpy() - 0.7 * 1.3 * xi)) <= 1e-5 * 0.91 + 1e-6 * float(base.abs().max()), l
        if s.has_bias:
            xb = oracle.normals(s.d_out, 5, 40 + 2 * l + 1)
            offb = (plan.gb[l].data_ptr() - plan.flat.data_ptr()) // 4
            assert np.max(np.abs((plan.gb[l] - pre[offb:offb + s.d_out]).cpu().numpy() - 0.91 * xb)) <= 1e-5, l


def test_step_clipped_sum_launch_overlaps_the_gram_tail(dp, path_switch):
    """A model whose layers all share one Gram launch (factors in its tail) and one CTA-pair clipped-sum launch:
    the second launch asks for programmatic serialization, so its CTAs may load inputs while the Gram launch
    drains, but read the factors only after it has completed.  Whole step against the oracle, repeated calls give
    the same bits (norms are stored in a fixed order, segments added in a fixed order), and the path with the
    overlap switched off gives those bits too."""
    B, T = 7, 256
    L = workloads.LayerSpec
    specs = (L("q", T, 512, 512, True, "normal"), L("k", T, 512, 512, False, "normal"), L("up", T, 256, 1024, True, "relu"))
    w = workloads.Workload("wide_overlap", B, "bf16", specs, 1.0, 0.6, 1.0 / (B * T))
    data = workloads.generate(w, 21)
    cal = _calibrate(w, data, 21, w.C)
    _check_step(dp, w, cal, w.C, w.sigma, 9)
    mk = lambda: dp.StepPlan([dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), s.has_bias) for (A, Z), s in zip(cal, specs)])  # noqa: E731
    plan = mk()
    n0 = dp.dpclip_launch_count()
    plan.run(w.C, w.sigma, 9)
    assert dp.dpclip_launch_count() - n0 == 3                # Gram + factors tail, CTA pairs, segment reduce + noise
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    first_flat, first_clip = plan.flat.clone(), plan.clip.clone()
    assert 0 < int((first_clip < 1).sum()) < B
    for _ in range(20):
        plan.flat.fill_(float("nan")); plan.clip.fill_(float("nan"))
        plan.run(w.C, w.sigma, 9)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    assert torch.equal(plan.clip, first_clip) and torch.equal(plan.flat, first_flat)
    path_switch("DPCLIP_NO_OVERLAP", "1")
    other = mk()
    other.run(w.C, w.sigma, 9)
    torch.cuda.synchronize()
    assert torch.equal(other.clip, first_clip) and torch.equal(other.flat, first_flat)


def test_step_same_shape_layers_share_launches(dp, path_switch):
    """Layers of one shape go through one clipped-sum launch (stacked d_out tiles, one set of partial tiles,
    one reduce with every layer's own noise streams): 256-row and 128-row tile forms, ragged d_out, layers
    with and without bias in one group, a group next to single layers; and the same model layer by layer."""
    L = workloads.LayerSpec
    w = workloads.Workload("same_shape_groups", 5, "bf16",
                           (L("a1", 48, 72, 136, True, "normal"), L("b1", 48, 136, 72, False, "normal"),
                            L("a2", 48, 72, 136, False, "normal"), L("c", 48, 64, 64, True, "normal"),
                            L("a3", 48, 72, 136, True, "relu"), L("b2", 48, 136, 72, False, "relu"),
                            L("head", 1, 136, 24, True, "relu")), 1.0, 0.8, 1.0 / (5 * 48))
    layers = workloads.generate(w, 3)
    cal = _calibrate(w, layers, 3, w.C)
    _check_step(dp, w, cal, w.C, w.sigma, 3)
    plan = _run_step(dp, w, cal, w.C, w.sigma, 3)
    taken = dp.dpclip_same_shape_layers_clipped_grad_noise(plan, w.C, w.sigma, 3, 0)
    torch.cuda.synchronize()
    assert taken == [True, True, True, False, True, True, False]
    path_switch("DPCLIP_NO_GRAD_GROUP", "1")
    path_switch("DPCLIP_NO_GRAM_GROUP", "1")
    single = _run_step(dp, w, cal, w.C, w.sigma, 3)
    for l in range(len(layers)):
        a, b = plan.gW[l].cpu().numpy(), single.gW[l].cpu().numpy()
        assert rel_fro(a, b) <= 1e-5            # same products, another summation order
    _check_step(dp, w, cal, w.C, w.sigma, 3)


def test_per_layer_clipping_through_the_same_entry_points(dp):
    """Per-layer clipping (each layer's gradient clipped to C / sqrt(L) on its own, the variant the paper's
    per-layer norms make possible): the rows of sq stay separate, so it is dpclip_factors on one row at a
    time and a clipped sum per layer with that layer's factors."""
    w = workloads.seq("bf16", B=6, T=24, d=64, d_ff=136)
    layers = workloads.generate(w, 8)
    L, C = len(layers), 0.05
    Cl = C / np.sqrt(L)
    ws = _ws(dp)
    total_sq = np.zeros(w.B)
    for (A, Z), spec in zip(layers, w.layers):
        sq_ref = oracle.layer_sqnorms(A, Z, spec.has_bias)
        n_ref, c_ref = oracle.factors(sq_ref[None, :], Cl)
        gW_ref, gb_ref = oracle.clipped_grad(A, Z, c_ref)
        dA, dZ = to_device(A, "bf16"), to_device(Z, "bf16")
        sq = torch.empty(1, w.B, device="cuda"); clip = torch.empty(w.B, device="cuda")
        dp.dpclip_layer_sqnorms(dA, dZ, spec.has_bias, sq[0], ws)
        dp.dpclip_factors(sq, Cl, clip)
        check_saturation(clip.cpu().numpy(), n_ref, c_ref, Cl)
        gW = torch.empty(spec.d_out, spec.d_in, device="cuda")
        gb = torch.empty(spec.d_out, device="cuda") if spec.has_bias else None
        dp.dpclip_clipped_grad(dA, dZ, clip, gW, gb, ws)
        assert rel_fro(gW.cpu().numpy(), gW_ref) <= TOL["bf16"]["grad"]
        total_sq += (c_ref ** 2) * sq_ref
    # every example's clipped gradient over all layers is then within C
    assert np.all(np.sqrt(total_sq) <= C * (1 + 1e-6))
    assert dp.dpclip_read_status(ws) == 0


@pytest.mark.parametrize("which", ["seq_bf16", "mlp_f32"])
def test_step_per_layer_clipping(dp, which):
    """dpclip_step_per_layer: every layer clipped to its own threshold in one call; factors, clipped sums and
    the noise N(0, sigma^2 sum_l C_l^2) equal the oracle's layer by layer."""
    w = workloads.seq("bf16", B=6, T=24, d=64, d_ff=136) if which == "seq_bf16" else workloads.mlp_small()
    layers = workloads.generate(w, 8)
    L, sigma, seed, sid0 = len(layers), 0.9, 13, 2
    sq_ref = [oracle.layer_sqnorms(A, Z, s.has_bias) for (A, Z), s in zip(layers, w.layers)]
    # thresholds near each layer's median norm, so that both sides of every threshold occur
    Cl = [float(np.median(np.sqrt(q))) for q in sq_ref]
    C_total = float(np.sqrt(np.sum(np.square(np.array(Cl, np.float32).astype(np.float64)))))
    plan = dp.StepPlan([dp.Layer(to_device(A, w.dtype), to_device(Z, w.dtype), s.has_bias)
                        for (A, Z), s in zip(layers, w.layers)])
    norms = torch.empty(L, w.B, device="cuda")
    plan.flat.fill_(float("nan"))
    clip = dp.dpclip_step_per_layer(plan, Cl, sigma, seed, sid0, norms_layers=norms)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    tol = TOL[w.dtype]
    for l, ((A, Z), s) in enumerate(zip(layers, w.layers)):
        n_ref, c_ref = oracle.factors(sq_ref[l][None, :], np.float32(Cl[l]))
        assert 0 < (c_ref < 1).sum() < w.B
        assert max_rel(norms[l].cpu().numpy(), n_ref) <= tol["norm"]
        check_saturation(clip[l].cpu().numpy(), n_ref, c_ref, Cl[l])
        gW_ref, gb_ref = oracle.clipped_grad(A, Z, c_ref)
        eW = oracle.add_noise(gW_ref.reshape(-1), sigma, C_total, seed, sid0 + 2 * l).reshape(gW_ref.shape)
        assert rel_fro(plan.gW[l].cpu().numpy(), eW) <= tol["grad"], l
        if s.has_bias:
            eb = oracle.add_noise(gb_ref, sigma, C_total, seed, sid0 + 2 * l + 1)
            assert rel_fro(plan.gb[l].cpu().numpy(), eb) <= tol["grad"], l


def test_sharded_step_single_rank_equals_step(dp):
    """The data-parallel wrapper on one rank (no process group): whole-step call without noise, then the
    noise launches, must give what one dpclip_step call gives."""
    from paper_2009_03106_b200 import parallel
    for w, seed in ((workloads.mlp_small(), 3), (workloads.seq("bf16", B=5, T=40, d=64, d_ff=136), 4)):
        layers = workloads.generate(w, seed)
        ref = _run_step(dp, w, layers, w.C, w.sigma, seed)
        dls = [dp.Layer(to_device(A, w.dtype), to_device(Z, w.dtype), spec.has_bias)
               for (A, Z), spec in zip(layers, w.layers)]
        plan = dp.StepPlan(dls)
        parallel.sharded_step(plan, w.C, w.sigma, seed, 0)
        torch.cuda.synchronize()
        assert dp.dpclip_read_status(plan.workspace) == 0
        assert torch.equal(plan.clip, ref.clip)
        assert rel_fro(plan.flat.cpu().numpy(), ref.flat.cpu().numpy()) <= 1e-6
        # the recorded form the multi-GPU benchmark replays (graph of the local step, bucketed reduction, noise once)
        plan2 = dp.StepPlan(dls)
        step = parallel.ShardedStep(plan2, w.C, w.sigma, seed, 0, bucket_bytes=1 << 12)
        step.run(); step.run()
        torch.cuda.synchronize()
        assert all(dp.dpclip_read_status(x) == 0 for x in plan2.workspaces())
        assert np.allclose(plan2.clip.cpu().numpy(), ref.clip.cpu().numpy(), rtol=2e-6, atol=0)
        assert rel_fro(plan2.flat.cpu().numpy(), ref.flat.cpu().numpy()) <= 2e-6


def test_step_host_matches_device_step(dp):
    w = workloads.mlp_small()
    layers = workloads.generate(w, 0)
    dev = _run_step(dp, w, layers, w.C, w.sigma, 3)
    host_layers = [dp.Layer(torch.from_numpy(A).pin_memory(), torch.from_numpy(Z).pin_memory(), s.has_bias)
                   for (A, Z), s in zip(layers, w.layers)]
    hs = dp.HostStep(host_layers)
    hs.run(w.C, w.sigma, 3, 0)
    torch.cuda.synchronize()
    assert np.allclose(hs.clip.numpy(), dev.clip.cpu().numpy(), rtol=1e-6)
    for l in range(len(layers)):
        assert rel_fro(hs.gW[l].numpy(), dev.gW[l].cpu().numpy()) <= 1e-6
    # inputs packed into one pinned buffer (one copy per direction): same results
    hp = dp.HostStep(host_layers, pack_inputs=True)
    hp.run(w.C, w.sigma, 3, 0)
    torch.cuda.synchronize()
    assert np.array_equal(hp.clip.numpy(), hs.clip.numpy()) and np.array_equal(hp.norms.numpy(), hs.norms.numpy())
    # the merged copies stop at the last tensor's real end (B = 32: norms take 128 of their 256-byte slot):
    # the guard band behind the results keeps its pattern
    for h in (hs, hp):
        assert h._out_end % 256 != 0 and bool((h._out_flat[h._out_end:] == 0xA5).all())
    for l in range(len(layers)):
        assert np.array_equal(hp.gW[l].numpy(), hs.gW[l].numpy())
        assert np.array_equal(hp.gb[l].numpy(), hs.gb[l].numpy())
        assert rel_fro(hs.gb[l].numpy(), dev.gb[l].cpu().numpy()) <= 1e-6
