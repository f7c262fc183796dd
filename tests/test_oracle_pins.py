"""Pins for the fp64 CPU oracle (no GPU needed).

The oracle is checked against things other than itself: per-example
gradients from an automatic differentiator and from finite differences on
tiny networks, closed forms, invariants and library routines.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
import workloads



@pytest.fixture(autouse=True)
def _fp64_default():
    """The tiny reference networks are built in fp64; restore the default afterwards."""
    old = torch.get_default_dtype()
    torch.set_default_dtype(torch.float64)
    yield
    torch.set_default_dtype(old)


# ---------------------------------------------------------------------------
# brute-force per-example backprop on tiny networks
# ---------------------------------------------------------------------------
def _per_example_autograd(loss_fn, params, B):
    """Gradient of each example's own loss w.r.t. every parameter, one
    backward pass per example (the naive loop the method replaces)."""
    out = []
    for i in range(B):
        gs = torch.autograd.grad(loss_fn(i), params, retain_graph=True)
        out.append([g.detach().numpy().copy() for g in gs])
    return out


def _mlp_case(seed=0, B=5, d0=7, d1=6, d2=4):
    g = torch.Generator().manual_seed(seed)
    X = torch.randn(B, d0, generator=g)
    W1 = torch.randn(d1, d0, generator=g, requires_grad=True)
    b1 = torch.randn(d1, generator=g, requires_grad=True)
    W2 = torch.randn(d2, d1, generator=g, requires_grad=True)
    b2 = torch.randn(d2, generator=g, requires_grad=True)
    y = torch.randint(0, d2, (B,), generator=g)
    Z1 = X @ W1.T + b1
    H1 = torch.tanh(Z1)
    Z2 = H1 @ W2.T + b2
    losses = F.cross_entropy(Z2, y, reduction="none")
    return X, (W1, b1, W2, b2), (Z1, Z2), (X, H1), losses


def test_dense_per_example_gradient_matches_autograd():
    X, params, Zs, As, losses = _mlp_case()
    B = X.shape[0]
    ref = _per_example_autograd(lambda i: losses[i], params, B)
    # backprop signal of example i = d loss_i / d Z (row i); other rows are zero
    for i in range(B):
        zbars = torch.autograd.grad(losses[i], Zs, retain_graph=True)
        for l in range(2):
            G, gb = oracle.example_grad(As[l][i:i + 1].detach().numpy(), zbars[l][i:i + 1].numpy())
            np.testing.assert_allclose(G, ref[i][2 * l], rtol=1e-12, atol=1e-14)
            np.testing.assert_allclose(gb, ref[i][2 * l + 1], rtol=1e-12, atol=1e-14)


def test_dense_per_example_gradient_matches_finite_differences():
    B, d0, d1 = 3, 4, 3
    rng = np.random.default_rng(5)
    X = rng.standard_normal((B, d0)); W = rng.standard_normal((d1, d0)); b = rng.standard_normal(d1)
    tgt = rng.standard_normal((B, d1))

    def loss_i(W_, b_, i):
        z = W_ @ X[i] + b_
        return float(np.sum(np.cosh(z - tgt[i])))

    h = 1e-6
    for i in range(B):
        z = W @ X[i] + b
        zbar = np.sinh(z - tgt[i])            # d loss_i / d z, by hand
        G, gb = oracle.example_grad(X[i:i + 1], zbar[None, :])
        fdW = np.zeros_like(W); fdb = np.zeros_like(b)
        for o in range(d1):
            for k in range(d0):
                E = np.zeros_like(W); E[o, k] = h
                fdW[o, k] = (loss_i(W + E, b, i) - loss_i(W - E, b, i)) / (2 * h)
            e = np.zeros_like(b); e[o] = h
            fdb[o] = (loss_i(W, b + e, i) - loss_i(W, b - e, i)) / (2 * h)
        np.testing.assert_allclose(G, fdW, rtol=1e-6, atol=1e-8)
        np.testing.assert_allclose(gb, fdb, rtol=1e-6, atol=1e-8)


@pytest.mark.parametrize("k,stride,pad", [(3, 1, 1), (2, 1, 0), (3, 2, 1)])
def test_conv_per_example_gradient_matches_autograd(k, stride, pad):
    B, cin, cout, H, W = 3, 2, 4, 6, 5
    g = torch.Generator().manual_seed(k * 10 + stride)
    X = torch.randn(B, cin, H, W, generator=g)
    Wt = torch.randn(cout, cin, k, k, generator=g, requires_grad=True)
    b = torch.randn(cout, generator=g, requires_grad=True)
    Z = F.conv2d(X, Wt, b, stride=stride, padding=pad)
    Z.retain_grad()
    losses = (torch.sigmoid(Z) ** 2).sum(dim=(1, 2, 3))
    P = F.unfold(X, k, padding=pad, stride=stride).transpose(1, 2)      # (B, T, cin*k*k), order (c,ky,kx)
    T = P.shape[1]
    assert T == Z.shape[2] * Z.shape[3]
    for i in range(B):
        gW, gbias, zbar = torch.autograd.grad(losses[i], (Wt, b, Z), retain_graph=True)
        zb = zbar[i].reshape(cout, T).T                                  # (T, cout)
        G, gb = oracle.example_grad(P[i].numpy(), zb.numpy())
        np.testing.assert_allclose(G.reshape(cout, cin, k, k), gW.numpy(), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(gb, gbias.numpy(), rtol=1e-12, atol=1e-14)


def test_im2col_generator_matches_library_unfold():
    rng = np.random.default_rng(0)
    fmap = rng.standard_normal((2, 3, 6, 5)).astype(np.float32)
    ours = workloads.im2col(fmap, 3, 1)
    ref = F.unfold(torch.from_numpy(fmap).double(), 3, padding=1).transpose(1, 2).numpy()
    np.testing.assert_array_equal(ours.astype(np.float64), ref)
    # strides, rectangular kernels, no padding
    for k, pad, stride in ((2, 0, 2), ((3, 2), 1, 1), ((1, 3), 2, 2), (5, 2, 3)):
        ours = workloads.im2col(fmap, k, pad, stride)
        ref = F.unfold(torch.from_numpy(fmap).double(), k, padding=pad, stride=stride).transpose(1, 2).numpy()
        np.testing.assert_array_equal(ours.astype(np.float64), ref)


def test_recurrent_per_example_gradient_matches_autograd():
    """Weights shared over time: the per-example gradient is the SUM over
    steps of the outer products (and of the signals, for the bias)."""
    B, T, n, m = 3, 4, 3, 5
    g = torch.Generator().manual_seed(3)
    X = torch.randn(B, T, n, generator=g)
    Wh = (0.5 * torch.randn(m, m, generator=g)).requires_grad_()
    V = torch.randn(m, n, generator=g).requires_grad_()
    b = torch.randn(m, generator=g).requires_grad_()
    h = torch.zeros(B, m)
    Hprev, Zs = [], []
    for t in range(T):
        Hprev.append(h)
        z = h @ Wh.T + X[:, t] @ V.T + b
        Zs.append(z)
        h = torch.tanh(z)
    losses = (h ** 2).sum(dim=1) + sum((zz ** 3).sum(dim=1) for zz in Zs) * 0.01
    for i in range(B):
        gWh, gV, gb_ref = torch.autograd.grad(losses[i], (Wh, V, b), retain_graph=True)
        zbars = torch.autograd.grad(losses[i], Zs, retain_graph=True)
        zb = torch.stack([z_[i] for z_ in zbars]).numpy()               # (T, m)
        hp = torch.stack([h_[i] for h_ in Hprev]).detach().numpy()      # (T, m)
        G, gb = oracle.example_grad(hp, zb)
        np.testing.assert_allclose(G, gWh.numpy(), rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(gb, gb_ref.numpy(), rtol=1e-11, atol=1e-13)
        G, _ = oracle.example_grad(X[i].numpy(), zb)
        np.testing.assert_allclose(G, gV.numpy(), rtol=1e-11, atol=1e-13)


def test_attention_projection_gradient_matches_autograd():
    B, S, d = 2, 5, 4
    g = torch.Generator().manual_seed(11)
    X = torch.randn(B, S, d, generator=g)
    Wq = torch.randn(d, d, generator=g, requires_grad=True)
    Wk = torch.randn(d, d, generator=g, requires_grad=True)
    Wv = torch.randn(d, d, generator=g, requires_grad=True)
    Q = X @ Wq.T; K = X @ Wk.T; Vv = X @ Wv.T
    att = torch.softmax(Q @ K.transpose(1, 2) / d ** 0.5, dim=-1) @ Vv
    losses = (att ** 2).sum(dim=(1, 2))
    for i in range(B):
        gq, gk, gv = torch.autograd.grad(losses[i], (Wq, Wk, Wv), retain_graph=True)
        zq, zk, zv = torch.autograd.grad(losses[i], (Q, K, Vv), retain_graph=True)
        for zbar, ref in ((zq, gq), (zk, gk), (zv, gv)):
            G, _ = oracle.example_grad(X[i].numpy(), zbar[i].numpy())
            np.testing.assert_allclose(G, ref.numpy(), rtol=1e-11, atol=1e-13)


def test_whole_step_matches_naive_clip_of_autograd_gradients():
    """Norms, factors and the clipped sum against the naive loop: flatten each
    example's autograd gradient, clip it with z / max(1, |z|/c), sum."""
    X, params, Zs, As, losses = _mlp_case(seed=4, B=6)
    B = X.shape[0]
    ref = _per_example_autograd(lambda i: losses[i], params, B)
    flat = [np.concatenate([g.ravel() for g in ref[i]]) for i in range(B)]
    ref_norms = np.array([np.linalg.norm(f) for f in flat])
    C = float(np.median(ref_norms))                     # half clipped, half not
    clipped_sum = sum(f / max(1.0, np.linalg.norm(f) / C) for f in flat)

    layers = []
    for l in range(2):
        zb = np.stack([torch.autograd.grad(losses[i], Zs[l], retain_graph=True)[0][i].numpy()
                       for i in range(B)])
        layers.append((As[l].detach().numpy()[:, None, :], zb[:, None, :]))
    res = oracle.step(layers, [True, True], C, sigma=0.0, seed=0)
    np.testing.assert_allclose(res["norms"], ref_norms, rtol=1e-12)
    assert 0 < int((res["clip"] < 1).sum()) < B
    got = np.concatenate([res["gW"][0].ravel(), res["gb"][0], res["gW"][1].ravel(), res["gb"][1]])
    np.testing.assert_allclose(got, clipped_sum, rtol=1e-11, atol=1e-13)
    # sigma = 0: the noised outputs equal the clipped sums
    np.testing.assert_array_equal(res["outW"][0], res["gW"][0])


# ---------------------------------------------------------------------------
# closed forms and invariants
# ---------------------------------------------------------------------------
def test_t1_closed_form():
    A, Z = workloads.random_layer(1, 9, 1, 13, 7)
    a2 = (A.astype(np.float64) ** 2).sum(axis=(1, 2))
    z2 = (Z.astype(np.float64) ** 2).sum(axis=(1, 2))
    np.testing.assert_allclose(oracle.layer_sqnorms(A, Z, False), a2 * z2, rtol=1e-13)
    np.testing.assert_allclose(oracle.layer_sqnorms(A, Z, True), (a2 + 1.0) * z2, rtol=1e-13)


@pytest.mark.parametrize("T,d_in,d_out", [(2, 3, 4), (5, 2, 2), (7, 6, 3)])
def test_gram_identity_and_library_matmul(T, d_in, d_out):
    A, Z = workloads.random_layer(2, 4, T, d_in, d_out)
    A64, Z64 = A.astype(np.float64), Z.astype(np.float64)
    sq = oracle.layer_sqnorms(A, Z, True)
    for i in range(4):
        gram = ((A64[i] @ A64[i].T) * (Z64[i] @ Z64[i].T)).sum() + (Z64[i] @ Z64[i].T).sum()
        mat = np.linalg.norm(Z64[i].T @ A64[i]) ** 2 + np.linalg.norm(Z64[i].sum(0)) ** 2
        np.testing.assert_allclose(sq[i], gram, rtol=1e-12)
        np.testing.assert_allclose(sq[i], mat, rtol=1e-12)


def test_norm_invariances():
    B, T, d_in, d_out = 3, 6, 5, 4
    A, Z = workloads.random_layer(3, B, T, d_in, d_out)
    base = oracle.layer_sqnorms(A, Z, True)
    rng = np.random.default_rng(0)
    pt = rng.permutation(T)
    np.testing.assert_allclose(oracle.layer_sqnorms(A[:, pt], Z[:, pt], True), base, rtol=1e-12)
    np.testing.assert_allclose(
        oracle.layer_sqnorms(A[:, :, rng.permutation(d_in)], Z[:, :, rng.permutation(d_out)], True),
        base, rtol=1e-12)
    np.testing.assert_allclose(oracle.layer_sqnorms(A, 3.0 * Z.astype(np.float64), True), 9.0 * base, rtol=1e-12)
    # zero rows (e.g. convolution padding) contribute nothing
    A2 = np.concatenate([A, np.zeros((B, 2, d_in), np.float32)], axis=1)
    Z2 = np.concatenate([Z, np.ones((B, 2, d_out), np.float32)], axis=1)
    np.testing.assert_allclose(oracle.layer_sqnorms(A2, Z2, False), oracle.layer_sqnorms(A, Z, False), rtol=1e-12)
    # weight sharing: the sum over t is taken BEFORE the norm
    per_t = sum(oracle.layer_sqnorms(A[:, t:t + 1], Z[:, t:t + 1], False) for t in range(T))
    assert not np.allclose(per_t, oracle.layer_sqnorms(A, Z, False), rtol=1e-3)


def test_clip_factor_properties():
    sq = np.array([[0.0, 0.25, 1.0, 4.0, 1e6], [0.0, 0.0, 0.0, 5.0, 0.0]])
    norms, clip = oracle.factors(sq, 1.0)
    np.testing.assert_allclose(norms, [0.0, 0.5, 1.0, 3.0, 1000.0])
    assert clip[0] == 1.0 and clip[1] == 1.0 and clip[2] == 1.0     # zero norm, below, tie
    np.testing.assert_allclose(clip[3:], [1 / 3.0, 1e-3], rtol=1e-15)
    for C in (0.1, 1.0, 10.0):
        n, c = oracle.factors(sq, C)
        assert np.all(c * n <= C * (1 + 1e-6))
        assert np.all(c[n <= C] == 1.0)
        np.testing.assert_allclose(c, np.minimum(1.0, C / np.maximum(n, 1e-300)), rtol=1e-15)


def test_clipped_sum_limits_and_linearity():
    B, T, d_in, d_out = 5, 3, 6, 4
    A, Z = workloads.random_layer(7, B, T, d_in, d_out)
    A64, Z64 = A.astype(np.float64), Z.astype(np.float64)
    # no clipping (C -> infinity): the plain batch gradient Zbar^T A
    sq = oracle.layer_sqnorms(A, Z, True)[None]
    _, clip = oracle.factors(sq, 1e30)
    assert np.all(clip == 1.0)
    gW, gb = oracle.clipped_grad(A, Z, clip)
    np.testing.assert_allclose(gW, np.einsum("bto,btk->ok", Z64, A64), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(gb, Z64.sum(axis=(0, 1)), rtol=1e-12, atol=1e-13)
    gW1, _ = oracle.clipped_grad(A, Z, None)
    np.testing.assert_array_equal(gW, gW1)
    # linear in the factors
    c = np.random.default_rng(1).uniform(0.1, 1.0, B)
    gWc, gbc = oracle.clipped_grad(A, Z, c)
    acc = np.zeros_like(gWc); accb = np.zeros_like(gbc)
    for i in range(B):
        e = np.zeros(B); e[i] = 1.0
        w, b_ = oracle.clipped_grad(A, Z, e)
        acc += c[i] * w; accb += c[i] * b_
    np.testing.assert_allclose(gWc, acc, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(gbc, accb, rtol=1e-12, atol=1e-13)
    # and equal to the library contraction with diag(c)
    np.testing.assert_allclose(gWc, np.einsum("b,bto,btk->ok", c, Z64, A64), rtol=1e-12, atol=1e-13)


def test_single_example_output_norm_is_min_of_norm_and_C():
    A, Z = workloads.random_layer(9, 1, 4, 5, 3)
    for C in (0.01, 1e3):
        res = oracle.step([(A, Z)], [True], C, sigma=0.0, seed=0)
        out = np.sqrt((res["gW"][0] ** 2).sum() + (res["gb"][0] ** 2).sum())
        np.testing.assert_allclose(out, min(res["norms"][0], C), rtol=1e-12)
    # direction only: scaling an already-clipped example's signal changes nothing
    r1 = oracle.step([(A, Z)], [True], 0.01, 0.0, 0)
    r2 = oracle.step([(A, 5.0 * Z.astype(np.float64))], [True], 0.01, 0.0, 0)
    np.testing.assert_allclose(r1["gW"][0], r2["gW"][0], rtol=1e-12)


def test_every_clipped_example_is_within_C_on_a_workload():
    w = workloads.mlp_small()
    layers = workloads.generate(w, seed=0)
    res = oracle.step(layers, [l.has_bias for l in w.layers], w.C, 0.0, 0)
    assert np.all(res["clip"] * res["norms"] <= w.C * (1 + 1e-6))
    # the stated distributions put every norm far above C = 1
    assert np.all(res["clip"] < 1.0)
    # clipped sum of B examples has norm at most B*C
    tot = np.sqrt(sum((g ** 2).sum() for g in res["gW"]) + sum((g ** 2).sum() for g in res["gb"]))
    assert tot <= w.B * w.C * (1 + 1e-9)


# ---------------------------------------------------------------------------
# element-wise parameter layers (LayerNorm gain and shift)
# ---------------------------------------------------------------------------
def test_layernorm_per_example_gradient_matches_autograd():
    """A LayerNorm inside a small sequence network: the per-example gradients of its gain and shift,
    taken by one backward pass per example, equal sum_t zbar (.) hbar and sum_t zbar."""
    B, S, d = 3, 5, 6
    g = torch.Generator().manual_seed(21)
    X = torch.randn(B, S, d, generator=g)
    W = torch.randn(d, d, generator=g)
    gamma = torch.randn(d, generator=g, requires_grad=True)
    beta = torch.randn(d, generator=g, requires_grad=True)
    U = torch.tanh(X @ W.T)
    mu = U.mean(dim=-1, keepdim=True)
    var = ((U - mu) ** 2).mean(dim=-1, keepdim=True)
    Hbar = (U - mu) / torch.sqrt(var + 1e-5)                   # normalised input: what the caller supplies
    Hout = gamma * Hbar + beta
    # the library routine must agree with this hand-written forward pass
    np.testing.assert_allclose(Hout.detach().numpy(),
                               F.layer_norm(U, (d,), gamma, beta, 1e-5).detach().numpy(), rtol=1e-12, atol=1e-12)
    losses = (torch.sin(Hout) * torch.arange(1, S + 1).view(1, S, 1)).sum(dim=(1, 2))
    for i in range(B):
        gg_ref, gs_ref = torch.autograd.grad(losses[i], (gamma, beta), retain_graph=True)
        (zbar,) = torch.autograd.grad(losses[i], (Hout,), retain_graph=True)
        gg, gs = oracle.elementwise_example_grad(Hbar[i].detach().numpy(), zbar[i].numpy())
        np.testing.assert_allclose(gg, gg_ref.numpy(), rtol=1e-11, atol=1e-13)
        np.testing.assert_allclose(gs, gs_ref.numpy(), rtol=1e-11, atol=1e-13)


def test_elementwise_layer_is_the_diagonal_of_the_dense_layer():
    """h = gamma (.) hbar is a dense layer whose weight is diag(gamma): its gradient is the diagonal of
    the dense per-example gradient, which the autograd pins above already fix."""
    rng = np.random.default_rng(5)
    B, T, d = 4, 7, 9
    H = rng.standard_normal((B, T, d)); Z = rng.standard_normal((B, T, d))
    sq = oracle.elementwise_sqnorms(H, Z, True)
    sq_noshift = oracle.elementwise_sqnorms(H, Z, False)
    for i in range(B):
        G, gb = oracle.example_grad(H[i], Z[i])
        gg, gs = oracle.elementwise_example_grad(H[i], Z[i])
        np.testing.assert_allclose(gg, np.diag(G), rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(gs, gb, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(sq[i], (np.diag(G) ** 2).sum() + (gb ** 2).sum(), rtol=1e-13)
        np.testing.assert_allclose(sq_noshift[i], (np.diag(G) ** 2).sum(), rtol=1e-13)
    # T = 1: the section's Algorithm, G = Z (.) H row by row
    H1, Z1 = H[:, :1], Z[:, :1]
    np.testing.assert_allclose(oracle.elementwise_sqnorms(H1, Z1, False), ((Z1 * H1) ** 2).sum(axis=(1, 2)), rtol=1e-13)


def test_elementwise_clipped_sum_limits_and_linearity():
    rng = np.random.default_rng(6)
    B, T, d = 5, 3, 8
    H = rng.standard_normal((B, T, d)); Z = rng.standard_normal((B, T, d))
    g1, s1 = oracle.elementwise_clipped_grad(H, Z, None)                    # all factors one
    np.testing.assert_allclose(g1, np.einsum("btj,btj->j", Z, H), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(s1, Z.sum(axis=(0, 1)), rtol=1e-12, atol=1e-13)
    c = rng.uniform(0.1, 1.0, B)
    gc, sc = oracle.elementwise_clipped_grad(H, Z, c)
    np.testing.assert_allclose(gc, np.einsum("i,itj,itj->j", c, Z, H), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(sc, np.einsum("i,itj->j", c, Z), rtol=1e-12, atol=1e-13)
    acc_g = np.zeros(d)
    for i in range(B):                                                      # linear in the factors
        e = np.zeros(B); e[i] = 1.0
        acc_g += c[i] * oracle.elementwise_clipped_grad(H, Z, e)[0]
    np.testing.assert_allclose(acc_g, gc, rtol=1e-12, atol=1e-13)
    # permuting the positions of an example (jointly in H and Z) changes nothing
    perm = rng.permutation(T)
    np.testing.assert_allclose(oracle.elementwise_sqnorms(H[:, perm], Z[:, perm], True),
                               oracle.elementwise_sqnorms(H, Z, True), rtol=1e-12)


# ---------------------------------------------------------------------------
# parameter updates (Algorithm 1's last line; the private Adam of the experiments)
# ---------------------------------------------------------------------------
def test_dp_updates_match_library_optimizers():
    """Fed with the same noisy mean gradient, the oracle's SGD and Adam steps must be the library's."""
    rng = np.random.default_rng(9)
    n, tau, C, sigma, lr = 37, 16, 1.3, 0.7, 1e-3
    theta0 = rng.standard_normal(n)
    for opt_name in ("sgd", "adam"):
        p = torch.tensor(theta0.copy(), requires_grad=True)
        opt = torch.optim.SGD([p], lr=lr) if opt_name == "sgd" else torch.optim.Adam([p], lr=lr, betas=(0.9, 0.999), eps=1e-8)
        th = theta0.copy(); m = np.zeros(n); v = np.zeros(n)
        for t in range(1, 5):
            gsum = rng.standard_normal(n) * 3.0
            g = (gsum + sigma * C * oracle.normals(n, 5, 100 + t)) / tau        # the noisy mean gradient
            p.grad = torch.tensor(g)
            opt.step()
            if opt_name == "sgd":
                th = oracle.dp_sgd_step(th, gsum, 1.0 / tau, C, sigma, 5, 100 + t, lr)
            else:
                th, m, v = oracle.dp_adam_step(th, m, v, gsum, 1.0 / tau, C, sigma, 5, 100 + t, lr, 0.9, 0.999, 1e-8, t)
                st = opt.state[p]
                np.testing.assert_allclose(m, st["exp_avg"].numpy(), rtol=1e-12, atol=1e-15)
                np.testing.assert_allclose(v, st["exp_avg_sq"].numpy(), rtol=1e-12, atol=1e-18)
            np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-11, atol=1e-14)


def test_dp_sgd_step_without_noise_is_plain_descent():
    th = oracle.dp_sgd_step(np.ones(5), np.arange(5.0), 0.25, 1.0, 0.0, 1, 2, 0.1)
    np.testing.assert_allclose(th, 1.0 - 0.1 * 0.25 * np.arange(5.0), rtol=1e-15)
