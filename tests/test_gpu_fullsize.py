"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot finish these workloads whole, so it is run on sampled
examples (norms, factors, and the clipped sum restricted to those examples via
a clip vector that is zero elsewhere -- same shapes, same grid), and the whole
clipped sum is checked with random bilinear probes u^T G v, which the
definition gives in O(B T (d_in + d_out)) in fp64."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from util import TOL, check_saturation, max_rel, rel_fro, to_device

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dp():
    import paper_2009_03106_b200 as pkg
    pkg.load_library()
    return pkg


def _probe(A, Z, clip, u, v):
    """u^T (sum_i c_i Zb_i^T A_i) v from the definition, fp64, chunked over examples."""
    tot = 0.0
    for i in range(A.shape[0]):
        tot += clip[i] * float((Z[i].astype(np.float64) @ u) @ (A[i].astype(np.float64) @ v))
    return tot


def _check_layer_full(dp, A, Z, spec, dtype, sample, ws, probes=4):
    B = A.shape[0]
    dA, dZ = to_device(A, dtype), to_device(Z, dtype)
    tol = TOL[dtype]
    # norms of sampled examples, every method that applies
    ref_sq = oracle.layer_sqnorms(A[sample], Z[sample], spec.has_bias)
    methods = [dp.DPCLIP_AUTO]
    if dtype == "bf16" and spec.T > 1 and spec.d_in % 8 == 0 and spec.d_out % 8 == 0:
        methods += [dp.DPCLIP_GRAM, dp.DPCLIP_MATERIALIZE]
    for m in methods:
        sq = torch.empty(B, device="cuda")
        dp.dpclip_layer_sqnorms(dA, dZ, spec.has_bias, sq, ws, m)
        got = sq.cpu().numpy()
        assert max_rel(np.sqrt(got[sample]), np.sqrt(ref_sq)) <= tol["norm"], (spec.name, m)
        assert np.all(np.isfinite(got)) and np.all(got > 0)
    # clipped sum restricted to the sampled examples: exact comparison with the oracle
    rng = np.random.default_rng(7)
    clip = np.zeros(B, np.float32)
    clip[sample] = rng.uniform(0.2, 1.0, len(sample)).astype(np.float32)
    clip[sample[0]] = 1.0
    gW = torch.empty((spec.d_out, spec.d_in), device="cuda")
    gb = torch.empty((spec.d_out,), device="cuda") if spec.has_bias else None
    dp.dpclip_clipped_grad(dA, dZ, torch.from_numpy(clip).cuda(), gW, gb, ws)
    refW, refb = oracle.clipped_grad(A[sample], Z[sample], clip[sample])
    assert rel_fro(gW.cpu().numpy(), refW) <= tol["grad"], spec.name
    if gb is not None:
        assert rel_fro(gb.cpu().numpy(), refb) <= tol["grad"]
    # whole clipped sum, random probes (E[(u^T E v)^2] = |E|_F^2 for unit Gaussian u, v)
    full_clip = rng.uniform(0.05, 1.0, B).astype(np.float32)
    dp.dpclip_clipped_grad(dA, dZ, torch.from_numpy(full_clip).cuda(), gW, gb, ws)
    G = gW.cpu().numpy().astype(np.float64)
    errs, mags = [], []
    for _ in range(probes):
        u = rng.standard_normal(spec.d_out); v = rng.standard_normal(spec.d_in)
        want = _probe(A, Z, full_clip.astype(np.float64), u, v)
        errs.append(u @ G @ v - want); mags.append(want)
    scale = np.linalg.norm(G)        # |u^T G v| ~ |G|_F for unit Gaussian probes
    assert np.sqrt(np.mean(np.square(errs))) <= 3 * tol["grad"] * scale, (spec.name, errs, scale)
    assert dp.dpclip_read_status(ws) == 0


def test_sequence_workload_full_size(dp):
    w = workloads.seq("bf16")
    layers = workloads.generate(w, seed=0)
    sample = np.array([0, 17, 63, 64, 127])
    ws = torch.empty(dp.dpclip_workspace_bytes(w.B, 256, 512, 512, dp.DPCLIP_BF16), dtype=torch.uint8, device="cuda")
    dp.dpclip_workspace_init(ws)
    for (A, Z), spec in zip(layers, w.layers):
        if spec.name in ("attn_k", "attn_v"):          # same shape as attn_q
            continue
        _check_layer_full(dp, A, Z, spec, "bf16", sample, ws)


def test_sequence_workload_full_step_factors(dp):
    """Whole dpclip_step at full size: norms and factors of sampled examples."""
    w = workloads.seq("bf16")
    layers = workloads.generate(w, seed=1)
    sample = np.array([3, 40, 101])
    hb = [s.has_bias for s in w.layers]
    plan = dp.StepPlan([dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), b) for (A, Z), b in zip(layers, hb)])
    C = 170.0                                           # the stated distributions give norms around 170
    plan.run(C, 0.0, seed=0)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    sq = np.stack([oracle.layer_sqnorms(A[sample], Z[sample], b) for (A, Z), b in zip(layers, hb)])
    n_ref, c_ref = oracle.factors(sq, C)
    assert max_rel(plan.norms.cpu().numpy()[sample], n_ref) <= TOL["bf16"]["norm"]
    clip = plan.clip.cpu().numpy()
    assert np.max(np.abs(clip[sample] - c_ref)) <= 5e-3
    assert 0 < (clip < 1).sum() < w.B                   # both sides of the threshold occur


@pytest.mark.parametrize("B,T,d_in,d_out", [(256, 16, 1024, 1024), (256, 128, 1024, 4096), (64, 2048, 1024, 1024),
                                            (256, 512, 1024, 4096), (1024, 16, 4096, 1024), (1024, 512, 1024, 1024),
                                            (256, 2048, 1024, 1024)])
def test_sweep_points(dp, B, T, d_in, d_out):
    """Points of the Gram-vs-materialise sweep (both norm forms must agree with the oracle)."""
    spec = workloads.LayerSpec("dense", T, d_in, d_out, True, "normal")
    g = torch.Generator(device="cuda").manual_seed(B + T)
    dA = torch.randn((B, T, d_in), generator=g, device="cuda").to(torch.bfloat16)
    dZ = (torch.randn((B, T, d_out), generator=g, device="cuda") / (B * T) ** 0.5).to(torch.bfloat16)
    sample = np.array([0, B // 2, B - 1])
    A_s = dA[sample].float().cpu().numpy(); Z_s = dZ[sample].float().cpu().numpy()
    ref_sq = oracle.layer_sqnorms(A_s, Z_s, True)
    ws = torch.empty(dp.dpclip_workspace_bytes(B, T, d_in, d_out, dp.DPCLIP_BF16), dtype=torch.uint8, device="cuda")
    dp.dpclip_workspace_init(ws)
    for m in (dp.DPCLIP_GRAM, dp.DPCLIP_MATERIALIZE):
        sq = torch.empty(B, device="cuda")
        dp.dpclip_layer_sqnorms(dA, dZ, True, sq, ws, m)
        assert max_rel(np.sqrt(sq.cpu().numpy()[sample]), np.sqrt(ref_sq)) <= 2e-5, m
    clip = np.zeros(B, np.float32); clip[sample] = [1.0, 0.5, 0.25]
    gW = torch.empty((d_out, d_in), device="cuda"); gb = torch.empty((d_out,), device="cuda")
    dp.dpclip_clipped_grad(dA, dZ, torch.from_numpy(clip).cuda(), gW, gb, ws)
    refW, refb = oracle.clipped_grad(A_s, Z_s, clip[sample])
    assert rel_fro(gW.cpu().numpy(), refW) <= TOL["bf16"]["grad"]
    assert rel_fro(gb.cpu().numpy(), refb) <= TOL["bf16"]["grad"]
    assert dp.dpclip_read_status(ws) == 0
    # The last point has 64 output tiles and long row ranges: with the queried workspace it is cut into several
    # waves of row slices; the smallest workspace the entry point accepts makes it run as one wave.  Same sums.
    floor = dp.dpclip_workspace_bytes(1, 1, 1, 1, dp.DPCLIP_BF16)
    if ws.numel() > floor:
        ws2 = torch.empty(floor, dtype=torch.uint8, device="cuda")
        dp.dpclip_workspace_init(ws2)
        gW2 = torch.empty_like(gW); gb2 = torch.empty_like(gb)
        dp.dpclip_clipped_grad(dA, dZ, torch.from_numpy(clip).cuda(), gW2, gb2, ws2)
        assert rel_fro(gW2.cpu().numpy(), gW.cpu().numpy()) <= 1e-6
        assert rel_fro(gb2.cpu().numpy(), gb.cpu().numpy()) <= 1e-6
        assert dp.dpclip_read_status(ws2) == 0


def _probe_whole_gradient(A, Z, clip, G, rng, tol, probes=4):
    """Random bilinear probes u^T G v of a whole clipped sum against the definition (fp64).  For unit Gaussian
    u, v: E[(u^T E v)^2] = |E|_F^2, so the root mean square over the probes estimates the Frobenius error."""
    G = G.astype(np.float64)
    errs = []
    for _ in range(probes):
        u = rng.standard_normal(G.shape[0]); v = rng.standard_normal(G.shape[1])
        errs.append(u @ G @ v - _probe(A, Z, clip, u, v))
    return float(np.sqrt(np.mean(np.square(errs)))), 3 * tol * float(np.linalg.norm(G))


def _bias_definition(Z, clip):
    """sum_i c_i sum_t zb_{i,t} from the definition, fp64."""
    return np.einsum("i,itd->d", clip.astype(np.float64), Z.astype(np.float64))


@pytest.mark.parametrize("form", ["one_call", "graph_of_one_call", "graph_four_streams"])
def test_sequence_workload_full_step_gradients(dp, form):
    """The whole step at B=128, T=256 in the launch configurations the benchmark times (the seven layers' norms
    in one Gram launch, the four 512->512 clipped sums stacked in one launch, one reduce with per-layer noise
    streams): EVERY released tensor is checked, weights by random bilinear probes with the step's own factors,
    biases element by element.  sigma = 0, so the released tensors are the clipped sums themselves."""
    w = workloads.seq("bf16")
    layers = workloads.generate(w, seed=2)
    hb = [s.has_bias for s in w.layers]
    plan = dp.StepPlan([dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), b) for (A, Z), b in zip(layers, hb)])
    C = 170.0                                           # norms are around 170: both sides of the threshold occur
    if form == "one_call":
        plan.flat.fill_(float("nan"))
        plan.run(C, 0.0, seed=0)
    else:
        graph = plan.capture(C, 0.0, seed=0, branches=1 if form == "graph_of_one_call" else 4)
        plan.flat.fill_(float("nan")); plan.clip.fill_(float("nan"))
        graph.replay()
    torch.cuda.synchronize()
    assert all(dp.dpclip_read_status(x) == 0 for x in plan.workspaces())
    clip = plan.clip.cpu().numpy()
    assert 0 < (clip < 1).sum() < w.B
    sample = np.array([5, 77, 126])
    sq = np.stack([oracle.layer_sqnorms(A[sample], Z[sample], b) for (A, Z), b in zip(layers, hb)])
    n_ref, c_ref = oracle.factors(sq, C)
    assert max_rel(plan.norms.cpu().numpy()[sample], n_ref) <= TOL["bf16"]["norm"]
    assert np.max(np.abs(clip[sample] - c_ref)) <= 5e-3
    rng = np.random.default_rng(11)
    for l, ((A, Z), spec) in enumerate(zip(layers, w.layers)):
        G = plan.gW[l].cpu().numpy()
        assert np.all(np.isfinite(G)), spec.name
        err, bound = _probe_whole_gradient(A, Z, clip.astype(np.float64), G, rng, TOL["bf16"]["grad"])
        assert err <= bound, (form, spec.name, err, bound)
        if spec.has_bias:
            assert rel_fro(plan.gb[l].cpu().numpy(), _bias_definition(Z, clip)) <= TOL["bf16"]["grad"], spec.name


def test_sequence_workload_full_step_per_layer_clipping(dp):
    """Per-layer clipping at B=128, T=256 (every layer against its own threshold, Sec. "Related Work"): one Gram launch
    for the norms, one launch for all rows of factors, one CTA-pair launch in which every layer carries its own
    factor vector.  Factors of sampled examples against the oracle; every released tensor by probes with that
    layer's own factor row."""
    w = workloads.seq("bf16")
    layers = workloads.generate(w, seed=3)
    hb = [s.has_bias for s in w.layers]
    plan = dp.StepPlan([dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), b) for (A, Z), b in zip(layers, hb)])
    sample = np.array([1, 66, 120])
    sq = np.stack([oracle.layer_sqnorms(A[sample], Z[sample], b) for (A, Z), b in zip(layers, hb)])
    # thresholds near each layer's own typical norm, so that both sides of every threshold occur
    Cl = [float(np.sqrt(np.median(sq[l]))) for l in range(plan.L)]
    plan.flat.fill_(float("nan"))
    clip_layers = dp.dpclip_step_per_layer(plan, Cl, 0.0, seed=0)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    clips = clip_layers.cpu().numpy()
    rng = np.random.default_rng(13)
    for l, ((A, Z), spec) in enumerate(zip(layers, w.layers)):
        n_ref, c_ref = oracle.factors(sq[l:l + 1], Cl[l])
        assert np.max(np.abs(clips[l][sample] - c_ref)) <= 5e-3, spec.name
        assert 0 < (clips[l] < 1).sum() < w.B, spec.name
        G = plan.gW[l].cpu().numpy()
        assert np.all(np.isfinite(G)), spec.name
        err, bound = _probe_whole_gradient(A, Z, clips[l].astype(np.float64), G, rng, TOL["bf16"]["grad"])
        assert err <= bound, (spec.name, err, bound)
        if spec.has_bias:
            assert rel_fro(plan.gb[l].cpu().numpy(), _bias_definition(Z, clips[l])) <= TOL["bf16"]["grad"], spec.name


def test_same_shape_layers_launch_full_size_against_the_oracle(dp):
    """The launch that carries the four 512->512 projections at B=128, T=256 (their d_out tiles stacked, 14 stages
    per CTA, one reduce over all four with per-layer outputs), called directly with factors that are zero outside
    five examples, so that the oracle can give every output element: tensor-by-tensor comparison."""
    w = workloads.seq("bf16")
    data = workloads.generate(w, seed=4)[:4]
    specs = w.layers[:4]
    plan = dp.StepPlan([dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), s.has_bias) for (A, Z), s in zip(data, specs)])
    sample = np.array([0, 31, 64, 99, 127])
    clip = np.zeros(w.B, np.float32)
    clip[sample] = [1.0, 0.75, 0.3, 0.011, 0.6]
    plan.clip.copy_(torch.from_numpy(clip))
    plan.flat.fill_(float("nan"))
    taken = dp.dpclip_same_shape_layers_clipped_grad_noise(plan, 1.0, 0.0, seed=0)
    torch.cuda.synchronize()
    assert all(taken)
    assert dp.dpclip_read_status(plan.workspace) == 0
    for l, (A, Z) in enumerate(data):
        refW, _ = oracle.clipped_grad(A[sample], Z[sample], clip[sample])
        assert rel_fro(plan.gW[l].cpu().numpy(), refW) <= TOL["bf16"]["grad"], l
    # with noise: the difference to the sigma = 0 result is the oracle's noise tensor of that layer's stream
    pre = [g.clone() for g in plan.gW]
    dp.dpclip_same_shape_layers_clipped_grad_noise(plan, 1.0, 0.8, seed=9, stream_id0=100)
    torch.cuda.synchronize()
    for l in range(4):
        xi = oracle.normals(512 * 512, 9, 100 + 2 * l).reshape(512, 512)
        got = (plan.gW[l] - pre[l]).cpu().numpy()
        assert np.max(np.abs(got - 0.8 * xi)) <= 1e-5 * 0.8 + 1e-6 * float(pre[l].abs().max()), l


def test_mlp_large_graph_replay_full_size(dp):
    """The headline workload at full size in the launch configuration the benchmark times: one dpclip_step
    call recorded into a CUDA graph and replayed (the one-launch fused kernel), checked against the oracle on
    every output."""
    w = workloads.mlp_large()
    layers = workloads.generate(w, 0)
    hb = [l.has_bias for l in w.layers]
    ref = oracle.step(layers, hb, w.C, w.sigma, 1, 0)
    plan = dp.StepPlan([dp.Layer(to_device(A, w.dtype), to_device(Z, w.dtype), s.has_bias)
                        for (A, Z), s in zip(layers, w.layers)])
    graph = plan.capture(w.C, w.sigma, 1, branches=1)
    for _ in range(3):                       # replays must not depend on what the previous one left behind
        plan.flat.fill_(float("nan")); plan.clip.fill_(float("nan"))
        graph.replay()
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    assert max_rel(plan.norms.cpu().numpy(), ref["norms"]) <= TOL["f32"]["norm"]
    check_saturation(plan.clip.cpu().numpy(), ref["norms"], ref["clip"], w.C)
    for l in range(len(layers)):
        assert rel_fro(plan.gW[l].cpu().numpy(), ref["outW"][l]) <= TOL["f32"]["grad"]
        assert rel_fro(plan.gb[l].cpu().numpy(), ref["outb"][l]) <= TOL["f32"]["grad"]
        # noise dominates the released tensor, so also compare element by element
        assert np.max(np.abs(plan.gW[l].cpu().numpy() - ref["outW"][l])) <= 2e-5 * max(1.0, np.max(np.abs(ref["outW"][l])))


def test_multi_branch_graph_matches_eager_step(dp):
    """Models with T > 1 layers are timed as a graph that holds ONE dpclip_step_streams call (the library forks
    over four streams and joins): it must give what the single-stream dpclip_step call gives."""
    for w in (workloads.seq("bf16", B=6, T=40, d=64, d_ff=136), workloads.cnn("f32")):
        layers = workloads.generate(w, 2)
        mk = lambda: dp.StepPlan([dp.Layer(to_device(A, w.dtype), to_device(Z, w.dtype), s.has_bias)   # noqa: E731
                                  for (A, Z), s in zip(layers, w.layers)])
        eager = mk(); eager.run(w.C, w.sigma, 7)
        # the same call outside a graph, eager on four streams
        direct = mk(); direct.run_streams(w.C, w.sigma, 7, branches=4)
        torch.cuda.synchronize()
        assert all(dp.dpclip_read_status(x) == 0 for x in direct.workspaces())
        assert np.allclose(direct.clip.cpu().numpy(), eager.clip.cpu().numpy(), rtol=2e-6, atol=0)
        for l in range(len(layers)):
            assert rel_fro(direct.gW[l].cpu().numpy(), eager.gW[l].cpu().numpy()) <= 2e-6
        plan = mk()
        graph = plan.capture(w.C, w.sigma, 7, branches=4)
        plan.flat.fill_(float("nan"))
        graph.replay(); graph.replay()
        torch.cuda.synchronize()
        assert len(plan.workspaces()) == 4 and all(dp.dpclip_read_status(x) == 0 for x in plan.workspaces())
        assert np.allclose(plan.clip.cpu().numpy(), eager.clip.cpu().numpy(), rtol=2e-6, atol=0)
        for l in range(len(layers)):             # (the flat buffer has alignment gaps nobody writes)
            assert rel_fro(plan.gW[l].cpu().numpy(), eager.gW[l].cpu().numpy()) <= 2e-6
            if plan.gb[l] is not None:
                assert rel_fro(plan.gb[l].cpu().numpy(), eager.gb[l].cpu().numpy()) <= 2e-6


def test_one_launch_step_repeats_bit_for_bit(dp):
    """The one-launch step crosses a grid-wide barrier whose counter lives in the workspace and resets itself:
    thousands of back-to-back launches, and launches from two streams at once (own workspaces), must keep
    giving the same bits and leave the status word clean."""
    w = workloads.mlp_large()
    layers = workloads.generate(w, 0)
    mk = lambda: dp.StepPlan([dp.Layer(to_device(A, w.dtype), to_device(Z, w.dtype), s.has_bias)     # noqa: E731
                              for (A, Z), s in zip(layers, w.layers)])
    a, b = mk(), mk()
    a.run(w.C, w.sigma, 1)
    torch.cuda.synchronize()
    ref, ref_clip = a.flat.clone(), a.clip.clone()
    for it in range(3000):
        a.run(w.C, w.sigma, 1)
        if it % 500 == 0:
            assert torch.equal(a.flat, ref) and torch.equal(a.clip, ref_clip)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for it in range(500):
        with torch.cuda.stream(s1):
            a.run(w.C, w.sigma, 1)
        with torch.cuda.stream(s2):
            b.run(w.C, w.sigma, 1)
    torch.cuda.synchronize()
    assert torch.equal(a.flat, ref) and torch.equal(b.flat, ref)
    assert dp.dpclip_read_status(a.workspace) == 0 and dp.dpclip_read_status(b.workspace) == 0


def test_grid_barrier_timeout_is_reported_and_recoverable(dp):
    """A grid barrier that cannot complete (its counter in the workspace header is corrupted before the launch,
    so one arrival is lost) must run into its bounded wait: the kernel returns, the status word says TIMEOUT,
    the context stays usable, and after dpclip_workspace_init the same plan gives the right answer again."""
    w = workloads.mlp_small()
    layers = workloads.generate(w, 0)
    plan = dp.StepPlan([dp.Layer(to_device(A, w.dtype), to_device(Z, w.dtype), s.has_bias)
                        for (A, Z), s in zip(layers, w.layers)])
    plan.run(w.C, w.sigma, 1)
    torch.cuda.synchronize()
    good = plan.flat.clone()
    plan.workspace[64:68].view(torch.int32).fill_(0x7FFFFFFF)      # the barrier counter: the first arrival wraps it to 0
    plan.run(w.C, w.sigma, 1)
    torch.cuda.synchronize()                                         # returns after the two-second wait limit
    assert dp.dpclip_read_status(plan.workspace) == -6               # DPCLIP_ERR_TIMEOUT
    dp.dpclip_workspace_init(plan.workspace)
    plan.flat.zero_()
    plan.run(w.C, w.sigma, 1)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    assert torch.equal(plan.flat, good)


def test_grouped_launches_repeat_over_thousands_of_calls(dp):
    """The Gram kernel for two-block examples draws its items from a counter in the workspace header that must be
    back at zero after every launch (it wraps after total + grid draws), and the narrow tensor-core kernel
    re-arms its rings per launch: two thousand back-to-back launches of each give the first launch's result every
    time (the sums are combined by atomics, so equal up to fp32 rounding order), and the status word stays clear."""
    w = workloads.seq("bf16", B=40, T=256, d=64, d_ff=136)
    data = workloads.generate(w, 3)
    layers = [dp.Layer(to_device(A, "bf16"), to_device(Z, "bf16"), s.has_bias, dp.DPCLIP_GRAM)
              for (A, Z), s in zip(data, w.layers)]
    plan = dp.StepPlan(layers)
    taken = dp.dpclip_gram_layers_sqnorms(plan)
    assert all(taken)
    torch.cuda.synchronize()
    first = plan.sq_layers.clone()
    sample = [0, 17, 39]
    for l, ((A, Z), s) in enumerate(zip(data, w.layers)):
        ref = oracle.layer_sqnorms(A[sample], Z[sample], s.has_bias)
        assert max_rel(np.sqrt(first[l].cpu().numpy()[sample]), np.sqrt(ref)) <= TOL["bf16"]["norm"]
    worst = torch.zeros((), device="cuda")
    for it in range(2000):
        dp.dpclip_gram_layers_sqnorms(plan)
        if it % 100 == 99:
            worst = torch.maximum(worst, ((plan.sq_layers - first).abs() / first).max())
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(plan.workspace) == 0
    assert float(worst) <= 1e-5
    # narrow tensor-core kernel: norms (several items per CTA) and clipped sum, 2000 launches each
    B, T, d_in, d_out = 200, 128, 27, 32
    A, Z = workloads.random_layer(71, B, T, d_in, d_out, "bf16", scale_z=0.05)
    dA, dZ = to_device(A, "bf16"), to_device(Z, "bf16")
    ws = torch.empty(max(1 << 20, dp.dpclip_workspace_bytes(B, T, d_in, d_out, 1, 0)), dtype=torch.uint8, device="cuda")
    dp.dpclip_workspace_init(ws)
    sq = torch.empty(B, device="cuda"); gW = torch.empty(d_out, d_in, device="cuda"); gb = torch.empty(d_out, device="cuda")
    clip = torch.rand(B, device="cuda") * 0.9 + 0.1
    dp.dpclip_layer_sqnorms(dA, dZ, True, sq, ws); dp.dpclip_clipped_grad(dA, dZ, clip, gW, gb, ws)
    torch.cuda.synchronize()
    sq0, gW0, gb0 = sq.clone(), gW.clone(), gb.clone()
    ref = oracle.layer_sqnorms(A[:4], Z[:4], True)
    assert max_rel(np.sqrt(sq0.cpu().numpy()[:4]), np.sqrt(ref)) <= TOL["bf16"]["norm"]
    same = torch.ones((), dtype=torch.bool, device="cuda")
    for it in range(2000):
        dp.dpclip_layer_sqnorms(dA, dZ, True, sq, ws)
        dp.dpclip_clipped_grad(dA, dZ, clip, gW, gb, ws)
        if it % 100 == 99:
            same &= torch.equal(sq, sq0) & torch.equal(gW, gW0) & torch.equal(gb, gb0)
    torch.cuda.synchronize()
    assert dp.dpclip_read_status(ws) == 0
    assert bool(same)                       # no atomics on this path: bit for bit
