"""Pins of the CPU oracle against things other than itself (no GPU needed).

Each test names the passage of the paper (or the published definition) that fixes the expected value.
"""
import os

import numpy as np
import pytest
import torch

import oracle as O
from paper_2509_03110_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
M64 = (1 << 64) - 1


# ------------------------------------------------------------------------------------------- schedule
def test_mix64_matches_published_splitmix64_vector():
    want = [int(l) for l in open(os.path.join(GOLD, "splitmix64_seed1234567.txt")) if l.strip() and not l.startswith("#")]
    s = 1234567
    got = []
    for _ in range(5):
        s = (s + 0x9E3779B97F4A7C15) & M64
        got.append(O.mix64(s))
    assert got == want


def test_hash_chain_structure():
    # H(seed, tag, t, k, j) = mix(mix(mix(seed ^ tag) + t) + (k * 2^20 + j)): composition checked through the
    # pinned mixer itself, for a few arguments including wrap-around.
    for seed, tag, t, k, j in [(0, O.lib().oracle_tag_idx(), 0, 0, 0), (M64, 12345, 7, 3, 99), (42, O.lib().oracle_tag_stale(), 10**6, 31, 255)]:
        inner = (O.mix64((O.mix64(seed ^ tag) + t) & M64) + ((k << 20) + j)) & M64
        assert O.hash5(seed, tag, t, k, j) == O.mix64(inner)
    assert O.lib().oracle_tag_idx() != O.lib().oracle_tag_stale()


def _flat_oracle(K=3, d=5, **kw):
    cfg = O.make_config(O.MODEL_FLAT, K=K, flat_d=d, **kw)
    x0, y0, g1, g2 = synth.flat_problem(K, d, seed=3)
    o = O.Oracle(cfg, None, None, x0, y0)
    o.set_external_grads(g1, g2)
    return o, x0, y0, g1, g2


def test_schedule_indices_in_range_and_spread():
    cfg = O.make_config(O.MODEL_LSQ, widths=(4,), K=4, batch=64, n_samples=10, seed=5)
    X = np.zeros((10, 4), np.float32)
    y = np.zeros(10, np.float32)
    o = O.Oracle(cfg, X, y, np.zeros((4, 4)), np.zeros(4))
    counts = np.zeros(10)
    for t in range(50):
        idx, stale, _ = o.read_schedule(t)
        assert idx.min() >= 0 and idx.max() < 10
        assert (stale == 0).all()
        counts += np.bincount(idx.ravel(), minlength=10)
    # 12800 i.i.d. draws over 10 cells: chi-square with 9 dof, 99.99 % quantile is 33.7
    e = counts.sum() / 10
    assert ((counts - e) ** 2 / e).sum() < 33.7
    # different replicas and different steps draw different minibatches
    a, _, _ = o.read_schedule(0)
    b, _, _ = o.read_schedule(1)
    assert not (a[0] == a[1]).all() and not (a[0] == b[0]).all()


def test_staleness_uniform_and_version_lookup():
    K, tau, smax = 4, 2, 3
    o, *_ = _flat_oracle(K=K, d=3, tau=tau, stale_max=smax, seed=11, lam=0.1)
    ver_at_step = []
    t_y = 0
    hist = np.zeros(smax + 1)
    for t in range(200):
        ver_at_step.append(t_y)
        o.step(0.01, 0.05)
        _, stale, ver = o.read_schedule(t)
        assert stale.min() >= 0 and stale.max() <= smax
        hist += np.bincount(stale, minlength=smax + 1)
        want = [ver_at_step[max(0, t - int(s))] for s in stale]
        assert list(ver) == want
        if o.should_couple():
            assert o.couple() == 0
            t_y += 1
    assert t_y == 100
    e = hist.sum() / (smax + 1)
    assert ((hist - e) ** 2 / e).sum() < 21.1  # chi-square, 3 dof, 99.99 %


def test_stale_max_zero_reads_current_centre():
    o, *_ = _flat_oracle(K=2, d=3, tau=1, stale_max=0)
    for t in range(6):
        o.step(0.01, 0.0)
        _, stale, ver = o.read_schedule(t)
        assert (stale == 0).all() and (ver == t).all()
        assert o.couple() == 0


# ------------------------------------------------------------------------------------------- bf16
def test_bf16_round_matches_torch():
    rng = np.random.default_rng(0)
    vals = np.concatenate([
        rng.standard_normal(2000).astype(np.float32) * np.float32(10.0) ** rng.integers(-20, 20, 2000).astype(np.float32),
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.005859375, 1.01171875, 3.3895314e38, 1e-40, -1e-40], np.float32),
    ])
    want = torch.from_numpy(vals).to(torch.bfloat16).to(torch.float32).numpy()
    got = np.array([O.bf16_round(float(v)) for v in vals], np.float32)
    assert (got.view(np.uint32) == want.view(np.uint32)).all()


# ------------------------------------------------------------------------------------------- gradients
def test_lsq_gradient_closed_form():
    X, y, _ = synth.least_squares_data(200, 17, seed=1)
    cfg = O.make_config(O.MODEL_LSQ, widths=(17,), K=1, batch=9, n_samples=200)
    rng = np.random.default_rng(2)
    w = rng.standard_normal(17)
    idx = rng.integers(0, 200, 9).astype(np.int32)
    loss, g = O.loss_grad(cfg, X, y, w, idx)
    Xb, yb = X[idx].astype(np.float64), y[idx].astype(np.float64)
    r = Xb @ w - yb
    assert np.isclose(loss, 0.5 * np.mean(r**2), rtol=1e-13)
    np.testing.assert_allclose(g, Xb.T @ r / 9, rtol=1e-12, atol=1e-14)


def _torch_mlp_loss(widths, residual, params, Xb, yb):
    """Independent statement of the classifier with torch ops (float64), gradient by autograd."""
    p = torch.tensor(params, dtype=torch.float64, requires_grad=True)
    h = torch.tensor(Xb, dtype=torch.float64)
    off = 0
    L = len(widths) - 1
    for l in range(L):
        fi, fo = widths[l], widths[l + 1]
        W = p[off:off + fi * fo].reshape(fo, fi)
        off += fi * fo
        b = p[off:off + fo]
        off += fo
        z = h @ W.T + b
        if l == L - 1:
            h = z
        elif residual and fi == fo:
            h = h + torch.relu(z)
        else:
            h = torch.relu(z)
    loss = torch.nn.functional.cross_entropy(h, torch.tensor(yb, dtype=torch.long))
    loss.backward()
    return float(loss.detach()), p.grad.numpy(), h.detach().numpy()


@pytest.mark.parametrize("model,widths", [
    (O.MODEL_MLP, (6, 5, 3)),
    (O.MODEL_MLP, (7, 8, 8, 4)),
    (O.MODEL_RESMLP, (5, 6, 6, 6, 3)),
    (O.MODEL_MLP, (4, 3)),
])
def test_mlp_gradient_vs_autograd_and_finite_differences(model, widths):
    n, B = 50, 6
    X, labels = synth.gaussian_mixture(n, widths[0], widths[-1], seed=4)
    cfg = O.make_config(model, widths=widths, K=1, batch=B, n_samples=n)
    d = O.param_count(cfg)
    assert d == synth.mlp_param_count(widths)
    rng = np.random.default_rng(5)
    params = synth.mlp_init(widths, seed=1).astype(np.float64) + 0.1 * rng.standard_normal(d)
    idx = rng.integers(0, n, B).astype(np.int32)
    loss, g = O.loss_grad(cfg, X, labels, params, idx)
    # (a) torch autograd on an independently written forward pass
    tl, tg, tlogits = _torch_mlp_loss(widths, model == O.MODEL_RESMLP, params, X[idx], labels[idx])
    assert np.isclose(loss, tl, rtol=1e-12)
    np.testing.assert_allclose(g, tg, rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(O.forward(cfg, X, params, idx), tlogits, rtol=1e-12, atol=1e-13)
    # (b) central finite differences of the oracle's own loss on a sample of coordinates
    h = 1e-6
    for j in rng.choice(d, size=min(d, 25), replace=False):
        e = np.zeros(d)
        e[j] = h
        lp, _ = O.loss_grad(cfg, X, labels, params + e, idx)
        lm, _ = O.loss_grad(cfg, X, labels, params - e, idx)
        fd = (lp - lm) / (2 * h)
        assert abs(fd - g[j]) <= 1e-6 * max(1.0, abs(g[j])), (j, fd, g[j])


def test_residual_flag_only_on_square_hidden_layers():
    # widths 5-6-6-3: layer 0 (5->6) plain, layer 1 (6->6) residual, head plain; differs from the plain MLP
    widths = (5, 6, 6, 3)
    X, labels = synth.gaussian_mixture(20, 5, 3, seed=2)
    params = synth.mlp_init(widths, seed=3).astype(np.float64)
    idx = np.arange(4, dtype=np.int32)
    c_res = O.make_config(O.MODEL_RESMLP, widths=widths, K=1, batch=4, n_samples=20)
    c_mlp = O.make_config(O.MODEL_MLP, widths=widths, K=1, batch=4, n_samples=20)
    _, _, lg = _torch_mlp_loss(widths, True, params, X[idx], labels[idx])
    np.testing.assert_allclose(O.forward(c_res, X, params, idx), lg, rtol=1e-12)
    assert not np.allclose(O.forward(c_mlp, X, params, idx), lg)


def test_bf16_mode_exact_on_representable_values_and_close_otherwise():
    widths = (4, 4, 2)
    n, B = 8, 4
    rng = np.random.default_rng(0)
    # small dyadic values: every product, sum and stored activation is exact in bf16, so the forward pass agrees exactly
    X = (rng.integers(-2, 3, (n, 4)) * 0.5).astype(np.float32)
    labels = (np.arange(n) % 2).astype(np.int32)
    params = (rng.integers(-2, 3, synth.mlp_param_count(widths)) * 0.25).astype(np.float64)
    idx = np.arange(B, dtype=np.int32)
    c32 = O.make_config(O.MODEL_MLP, widths=widths, K=1, batch=B, n_samples=n)
    c16 = O.make_config(O.MODEL_MLP, widths=widths, K=1, batch=B, n_samples=n, gemm_dtype=O.GEMM_BF16)
    np.testing.assert_array_equal(O.forward(c32, X, params, idx), O.forward(c16, X, params, idx))
    # generic values: operands carry 8 significant bits, so the two gradients agree to a few 2^-8
    X2, labels2 = synth.gaussian_mixture(40, 4, 2, seed=1)
    p2 = synth.mlp_init(widths, seed=2).astype(np.float64)
    idx2 = np.arange(16, dtype=np.int32)
    c32b = O.make_config(O.MODEL_MLP, widths=widths, K=1, batch=16, n_samples=40)
    c16b = O.make_config(O.MODEL_MLP, widths=widths, K=1, batch=16, n_samples=40, gemm_dtype=O.GEMM_BF16)
    l32, g32 = O.loss_grad(c32b, X2, labels2, p2, idx2)
    l16, g16 = O.loss_grad(c16b, X2, labels2, p2, idx2)
    rel = np.linalg.norm(g16 - g32) / np.linalg.norm(g32)
    assert 0 < rel < 3e-2 and abs(l16 - l32) < 3e-2 * abs(l32)
    # parameters that are already bf16 values and a linear model: only the stored dz is rounded
    c1 = O.make_config(O.MODEL_MLP, widths=(4, 2), K=1, batch=16, n_samples=40, gemm_dtype=O.GEMM_BF16)
    c1f = O.make_config(O.MODEL_MLP, widths=(4, 2), K=1, batch=16, n_samples=40)
    p1 = np.array([O.bf16_round(float(v)) for v in synth.mlp_init((4, 2), seed=5)], np.float64)
    Xq = torch.from_numpy(X2).to(torch.bfloat16).to(torch.float32).numpy()
    lq, gq = O.loss_grad(c1, X2, labels2, p1, idx2)
    lf, gf = O.loss_grad(c1f, Xq, labels2, p1, idx2)
    assert np.isclose(lq, lf, rtol=1e-14)  # loss is taken before any backward rounding
    assert np.linalg.norm(gq - gf) / np.linalg.norm(gf) < 2 ** -8


def test_bf16_mode_step_keeps_gradients_and_optimiser_state_unrounded():
    # BF16 mode rounds matmul OPERANDS only.  Eq. 3 and the first update of Algorithm 1 know one gradient, so the
    # perturbation, the sampler and the centre update must be the FP32-mode arithmetic applied to that mode's gradients.
    # (a) Least squares on bf16-representable inputs: the only operand the mode rounds is the minibatch, so a whole
    #     trajectory (steps, stale centre reads, syncs) must be bit-equal to FP32 mode.  A rounding applied to g1, to its
    #     norm, to the perturbed point, to g2 or to G would break the equality.
    X, y, _ = synth.least_squares_data(64, 12, noise=0.01, seed=7)
    Xq = torch.from_numpy(X).to(torch.bfloat16).to(torch.float32).numpy()
    rng = np.random.default_rng(8)
    x0, y0 = rng.standard_normal((3, 12)), rng.standard_normal(12)
    runs = []
    for dt in (O.GEMM_FP32, O.GEMM_BF16):
        cfg = O.make_config(O.MODEL_LSQ, widths=(12,), K=3, batch=8, n_samples=64, gemm_dtype=dt, lam=0.3, tau=2, stale_max=2, seed=4)
        o = O.Oracle(cfg, Xq, y, x0, y0)
        for _ in range(7):
            o.step(0.05, 0.1)
            if o.should_couple():
                assert o.couple() == 0
        runs.append((o.read_state(), o.read_grads()))
    for key in ("x", "v", "y", "acc", "gprev"):
        np.testing.assert_array_equal(runs[0][0][key], runs[1][0][key])
    for a, b in zip(runs[0][1], runs[1][1]):
        np.testing.assert_array_equal(a, b)
    # and the mode does act on operands: with inputs that are not bf16 values the two modes differ
    o32 = O.Oracle(O.make_config(O.MODEL_LSQ, widths=(12,), K=3, batch=8, n_samples=64), X, y, x0, y0)
    o16 = O.Oracle(O.make_config(O.MODEL_LSQ, widths=(12,), K=3, batch=8, n_samples=64, gemm_dtype=O.GEMM_BF16), X, y, x0, y0)
    o32.step(0.05, 0.1)
    o16.step(0.05, 0.1)
    assert not np.array_equal(o32.read_state()["x"], o16.read_state()["x"])
    # (b) A classifier in BF16 mode: one step equals the gradient-fed (FLAT) step, which has no modes, driven with
    #     g1 = BF16-mode gradient at x and g2 = BF16-mode gradient at the UNROUNDED perturbed point x + rho g1/(|g1|+gamma)
    #     (the matmul rounds its own operand copy).  The FLAT model carries gradients as fp32, hence 1e-6, not equality.
    widths, K, B, n = (6, 8, 4), 2, 8, 40
    Xc, labels = synth.gaussian_mixture(n, widths[0], widths[-1], seed=1)
    w0 = synth.mlp_init(widths, seed=2).astype(np.float64)
    xs = np.stack([w0, w0 + 0.01 * rng.standard_normal(w0.shape)])
    yc = xs.mean(axis=0)
    kw = dict(K=K, lam=0.7, tau=4, seed=9)
    cfg = O.make_config(O.MODEL_MLP, widths=widths, batch=B, n_samples=n, gemm_dtype=O.GEMM_BF16, **kw)
    o = O.Oracle(cfg, Xc, labels, xs, yc)
    idx, _, _ = o.read_schedule(0)
    rho, gam = float(np.float32(0.1)), float(np.float32(1e-12))
    c1 = O.make_config(O.MODEL_MLP, widths=widths, K=1, batch=B, n_samples=n, gemm_dtype=O.GEMM_BF16)
    g1 = np.stack([O.loss_grad(c1, Xc, labels, xs[k], idx[k])[1] for k in range(K)])
    xp = np.stack([xs[k] + rho * g1[k] / (np.linalg.norm(g1[k]) + gam) for k in range(K)])
    g2 = np.stack([O.loss_grad(c1, Xc, labels, xp[k], idx[k])[1] for k in range(K)])
    o.step(0.05, 0.1)
    og1, og2, oxp = o.read_grads()
    np.testing.assert_allclose(og1, g1, rtol=1e-13, atol=1e-300)
    np.testing.assert_allclose(oxp, xp, rtol=1e-13)
    np.testing.assert_allclose(og2, g2, rtol=1e-12, atol=1e-300)
    f = O.Oracle(O.make_config(O.MODEL_FLAT, flat_d=len(w0), **kw), None, None, xs, yc)
    f.set_external_grads(g1, g2)
    f.step(0.05, 0.1)
    sf, so = f.read_state(), o.read_state()
    for key in ("x", "v", "acc"):
        assert np.linalg.norm(sf[key] - so[key]) <= 1e-6 * np.linalg.norm(so[key]), key
    # the gradients really are unrounded: they are not bf16 values
    assert np.mean([O.bf16_round(float(v)) == float(np.float32(v)) for v in og2[0][:200]]) < 0.2


# ------------------------------------------------------------------------------------------- S4: perturbation
def _lsq_oracle(K=2, B=8, n=64, f=12, noise=0.01, **kw):
    X, y, w_star = synth.least_squares_data(n, f, noise=noise, seed=7)
    cfg = O.make_config(O.MODEL_LSQ, widths=(f,), K=K, batch=B, n_samples=n, **kw)
    rng = np.random.default_rng(8)
    x0 = rng.standard_normal((K, f))
    y0 = x0.mean(axis=0)
    return O.Oracle(cfg, X, y, x0, y0), X, y, w_star, x0, y0


def test_perturbation_length_and_alignment():
    # ||x~ - x|| = rho n/(n+gamma) <= rho and g1.(x~ - x) = rho n^2/(n+gamma) >= 0 (proof of Proposition 7, steps 2-3)
    for gamma in (1e-12, 0.5):
        o, X, y, _, x0, _ = _lsq_oracle(gamma=gamma)
        rho = 0.05
        o.step(0.01, rho)
        g1, _, xp = o.read_grads()
        _, n1, _ = o.read_step_info()
        idx, _, _ = o.read_schedule(0)
        gam = float(np.float32(gamma))
        rho = float(np.float32(rho))
        for k in range(2):
            Xb, yb = X[idx[k]].astype(np.float64), y[idx[k]].astype(np.float64)
            g_closed = Xb.T @ (Xb @ x0[k] - yb) / len(yb)
            np.testing.assert_allclose(g1[k], g_closed, rtol=1e-12)
            n = np.linalg.norm(g_closed)
            assert np.isclose(n1[k], n, rtol=1e-13)
            delta = xp[k] - x0[k]
            assert np.isclose(np.linalg.norm(delta), rho * n / (n + gam), rtol=1e-11)
            assert np.linalg.norm(delta) <= rho * (1 + 1e-12)
            assert np.isclose(g_closed @ delta, rho * n * n / (n + gam), rtol=1e-11)


def test_sam_gradient_closed_form_on_least_squares():
    # g2 = X_b^T (X_b (w + eps) - y_b) / B on the SAME minibatch (Theorem 3)
    o, X, y, _, x0, _ = _lsq_oracle()
    o.step(0.01, 0.05)
    _, g2, _ = o.read_grads()
    idx, _, _ = o.read_schedule(0)
    rho = float(np.float32(0.05))
    for k in range(2):
        Xb, yb = X[idx[k]].astype(np.float64), y[idx[k]].astype(np.float64)
        g1 = Xb.T @ (Xb @ x0[k] - yb) / len(yb)
        eps = rho * g1 / (np.linalg.norm(g1) + float(np.float32(1e-12)))
        np.testing.assert_allclose(g2[k], Xb.T @ (Xb @ (x0[k] + eps) - yb) / len(yb), rtol=1e-11)


def test_stationary_point_gives_zero_perturbation_without_nan():
    # noise-free least squares at w = w*: the gradient vanishes and gamma keeps the map finite (Remark after Proposition 7)
    X, _, w_star = synth.least_squares_data(32, 6, noise=0.0, seed=3)
    y = (X.astype(np.float64) @ w_star.astype(np.float64)).astype(np.float32)
    # make the targets exactly consistent in double: use integer-valued data
    X = np.round(X * 4).astype(np.float32)
    w_int = np.round(w_star * 2).astype(np.float64)
    y = (X.astype(np.float64) @ w_int).astype(np.float32)
    cfg = O.make_config(O.MODEL_LSQ, widths=(6,), K=1, batch=8, n_samples=32, gamma=1e-12)
    o = O.Oracle(cfg, X, y, w_int[None, :], w_int)
    o.step(0.1, 0.05)
    g1, g2, xp = o.read_grads()
    assert np.all(g1 == 0) and np.all(g2 == 0) and np.all(np.isfinite(xp))
    np.testing.assert_array_equal(xp[0], w_int)
    np.testing.assert_array_equal(o.read_params(0), w_int)


# ------------------------------------------------------------------------------------------- S6: worker update
def test_update_matches_torch_sgd_when_no_pull():
    # lambda = 0: the sampler is a plain (Nesterov or heavy-ball) momentum step on g2; torch.optim.SGD states the same rule
    for nesterov in (1, 0):
        K, d = 2, 7
        o, x0, y0, g1, g2 = _flat_oracle(K=K, d=d, mu=0.9, nesterov=nesterov, lam=0.0, tau=100)
        p = torch.tensor(x0.astype(np.float64), requires_grad=True)
        opt = torch.optim.SGD([p], lr=float(np.float32(0.03)), momentum=float(np.float32(0.9)), nesterov=bool(nesterov))
        for _ in range(5):
            o.step(0.03, 0.05)
            p.grad = torch.tensor(g2.astype(np.float64))
            opt.step()
        np.testing.assert_allclose(o.read_state()["x"], p.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_rho_zero_is_momentum_sgd_on_proximal_objective():
    # rho = 0: g2 = g1 and the step is momentum SGD on f(x) + (lambda/2)||x - y||^2 (Algorithm 1, first update)
    o, X, y, _, x0, y0 = _lsq_oracle(K=2, mu=0.9, lam=0.3, tau=1000)
    eta, mu, lam = float(np.float32(0.02)), float(np.float32(0.9)), float(np.float32(0.3))
    x = x0.copy()
    v = np.zeros_like(x)
    for t in range(6):
        idx, _, _ = o.read_schedule(t)
        o.step(0.02, 0.0)
        for k in range(2):
            Xb, yb = X[idx[k]].astype(np.float64), y[idx[k]].astype(np.float64)
            G = Xb.T @ (Xb @ x[k] - yb) / len(yb) + lam * (x[k] - y0)
            v[k] = mu * v[k] + G
            x[k] = x[k] - eta * (G + mu * v[k])
    np.testing.assert_allclose(o.read_state()["x"], x, rtol=1e-11, atol=1e-13)
    g1, g2, xp = o.read_grads()
    np.testing.assert_array_equal(g1, g2)


def test_mu_zero_is_algorithm1_first_update():
    # mu = 0: x_{t+1} = x_t - eta (g_t + lambda (x_t - y_t)) exactly (Algorithm 1)
    o, x0, y0, g1, g2 = _flat_oracle(K=3, d=5, mu=0.0, lam=0.25, tau=100)
    eta, lam = float(np.float32(0.1)), float(np.float32(0.25))
    o.step(0.1, 0.05)
    want = x0.astype(np.float64) - eta * (g2.astype(np.float64) + lam * (x0.astype(np.float64) - y0.astype(np.float64)))
    np.testing.assert_allclose(o.read_state()["x"], want, rtol=1e-13, atol=1e-15)


def test_single_worker_without_coupling_is_plain_sam():
    # K = 1, lambda = 0: textbook SAM with momentum, written independently on the least-squares closed form
    o, X, y, _, x0, _ = _lsq_oracle(K=1, mu=0.9, lam=0.0, tau=10**6)
    eta, rho, mu, gam = (float(np.float32(a)) for a in (0.02, 0.05, 0.9, 1e-12))
    w = x0[0].copy()
    v = np.zeros_like(w)
    for t in range(8):
        idx, _, _ = o.read_schedule(t)
        o.step(0.02, 0.05)
        Xb, yb = X[idx[0]].astype(np.float64), y[idx[0]].astype(np.float64)
        g = Xb.T @ (Xb @ w - yb) / len(yb)
        wa = w + rho * g / (np.linalg.norm(g) + gam)
        gs = Xb.T @ (Xb @ wa - yb) / len(yb)
        v = mu * v + gs
        w = w - eta * (gs + mu * v)
    np.testing.assert_allclose(o.read_params(0), w, rtol=1e-11, atol=1e-13)


def test_pull_uses_the_stale_centre_version():
    # the worker's kernel term is lambda (x - y_ver) with y_ver the version its schedule entry names
    K, d, tau, smax = 3, 4, 1, 2
    o, x0, y0, g1, g2 = _flat_oracle(K=K, d=d, mu=0.0, lam=0.5, tau=tau, stale_max=smax, seed=21)
    eta, lam = float(np.float32(0.1)), float(np.float32(0.5))
    centres = [y0.astype(np.float64)]
    x = x0.astype(np.float64).copy()
    seen_stale = False
    for t in range(12):
        o.step(0.1, 0.0)
        _, stale, ver = o.read_schedule(t)
        for k in range(K):
            seen_stale |= ver[k] != len(centres) - 1
            x[k] = x[k] - eta * (g2[k].astype(np.float64) + lam * (x[k] - centres[ver[k]]))
        np.testing.assert_allclose(o.read_state()["x"], x, rtol=1e-12, atol=1e-14)
        assert o.couple() == 0
        centres.append(o.read_params(-1))
    assert seen_stale


# ------------------------------------------------------------------------------------------- S7: centre update
def test_centre_is_mean_of_iterates_when_beta0_etaprime1():
    # beta = 0, eta' = 1: y_new = y + (mean - y) = arithmetic mean of the n*tau post-update iterates (Algorithm 2, sync branch)
    K, d, tau = 3, 5, 4
    o, *_ = _flat_oracle(K=K, d=d, tau=tau, beta=0.0, eta_prime=1.0, lam=0.2)
    for rnd in range(3):
        iterates = []
        for s in range(tau):
            assert not o.should_couple()
            assert o.couple() != 0  # refused while the trigger is false
            o.step(0.05, 0.05)
            iterates.append(o.read_state()["x"].copy())
        assert o.should_couple()
        acc = o.read_state()["acc"]
        np.testing.assert_allclose(acc, np.sum(iterates, axis=0), rtol=1e-13)
        assert o.couple() == 0
        np.testing.assert_allclose(o.read_params(-1), np.mean(np.concatenate(iterates, axis=0), axis=0), rtol=1e-12, atol=1e-14)
        t, t_y, t_x = o.counters()
        assert t == (rnd + 1) * tau and t_y == rnd + 1 and (t_x == 0).all()
        assert np.all(o.read_state()["acc"] == 0)


def test_lookahead_direction_and_first_sync():
    # g = g' + beta (g' - g'_prev), with no difference term at the first sync (Algorithm 2; Section 4.2)
    K, d, tau = 2, 4, 2
    o, x0, y0, *_ = _flat_oracle(K=K, d=d, tau=tau, beta=0.9, eta_prime=0.7, lam=0.1)
    beta, etap = float(np.float32(0.9)), float(np.float32(0.7))
    y = y0.astype(np.float64)
    gprev = None
    for rnd in range(4):
        its = []
        for _ in range(tau):
            o.step(0.05, 0.05)
            its.append(o.read_state()["x"].copy())
        gp = np.sum(np.concatenate(its, axis=0), axis=0) / (K * tau) - y
        g = gp if gprev is None else gp + beta * (gp - gprev)
        y = y + etap * g
        gprev = gp
        assert o.couple() == 0
        np.testing.assert_allclose(o.read_params(-1), y, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(o.read_state()["gprev"], gp, rtol=1e-12, atol=1e-14)


def test_reduces_to_algorithm1_single_chain():
    # n = 1, tau = 1, beta = 0, mu = 0, eta' = alpha:  y_{t+1} = alpha x_{t+1} + (1 - alpha) y_t  (Algorithm 1), and
    # z_{t+1} = (1 - alpha) [ (1 - lambda eta) z_t - eta g_t ]  (proof of Lemma 5, step 1)
    alpha, lam, eta = 0.3, 0.4, 0.05
    o, X, yv, _, x0, y0 = _lsq_oracle(K=1, mu=0.0, lam=lam, tau=1, beta=0.0, eta_prime=alpha)
    a, l, e = (float(np.float32(v)) for v in (alpha, lam, eta))
    x = x0[0].copy()
    y = y0.copy()
    for t in range(10):
        z = x - y
        o.step(eta, 0.05)
        _, g2, _ = o.read_grads()
        x = x - e * (g2[0] + l * (x - y))
        y_new = a * x + (1 - a) * y
        assert o.couple() == 0
        np.testing.assert_allclose(o.read_params(0), x, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(o.read_params(-1), y_new, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(x - y_new, (1 - a) * ((1 - l * e) * z - e * g2[0]), rtol=1e-10, atol=1e-13)
        y = y_new


def test_workers_are_not_reset_at_sync():
    # the sync branch resets counters only; iterates and momentum buffers are untouched (Algorithm 2, last line of the branch)
    o, *_ = _flat_oracle(K=2, d=3, tau=1, lam=0.2)
    o.step(0.05, 0.05)
    before = o.read_state()
    assert o.couple() == 0
    after = o.read_state()
    np.testing.assert_array_equal(before["x"], after["x"])
    np.testing.assert_array_equal(before["v"], after["v"])


def test_lyapunov_identity_on_least_squares():
    # Phi_{t+1} = F_t(x_{t+1}) - (lambda/2)(1 - (1-alpha)^2) ||x_{t+1} - y_t||^2 with F_t(x) = f(x) + (lambda/2)||x - y_t||^2
    # (proof of Theorem 2): exercises the centre update through the full-data least-squares objective.
    alpha, lam, eta = 0.5, 0.3, 0.02
    o, X, yv, _, x0, y0 = _lsq_oracle(K=1, mu=0.0, lam=lam, tau=1, beta=0.0, eta_prime=alpha)
    a, l = float(np.float32(alpha)), float(np.float32(lam))
    Xd, yd = X.astype(np.float64), yv.astype(np.float64)
    f = lambda w: 0.5 * np.mean((Xd @ w - yd) ** 2)
    y = y0.copy()
    for t in range(5):
        o.step(eta, 0.0)
        assert o.couple() == 0
        x1, y1 = o.read_params(0), o.read_params(-1)
        phi = f(x1) + 0.5 * l * np.sum((x1 - y1) ** 2)
        F = f(x1) + 0.5 * l * np.sum((x1 - y) ** 2)
        assert np.isclose(phi, F - 0.5 * l * (1 - (1 - a) ** 2) * np.sum((x1 - y) ** 2), rtol=1e-11)
        y = y1


def test_constant_rho_plateau_bound_soft():
    # Theorem 3: average ||G_t||^2 <= 4 L^2 rho^2 + O(log T / sqrt T); soft check with full-batch gradients (sigma = 0)
    n, f = 64, 8
    X, yv, _ = synth.least_squares_data(n, f, noise=0.01, seed=9)
    Xd, yd = X.astype(np.float64), yv.astype(np.float64)
    Lc = np.linalg.eigvalsh(Xd.T @ Xd / n).max()
    lam, rho = 0.1, 0.05
    eta = 0.2 / (4 * (Lc + lam))
    cfg = O.make_config(O.MODEL_LSQ, widths=(f,), K=1, batch=n, n_samples=n, mu=0.0, lam=lam, tau=1, beta=0.0, eta_prime=0.5)
    o = O.Oracle(cfg, X, yv, np.zeros((1, f)), np.zeros(f))
    tail = []
    for t in range(400):
        x, y = o.read_params(0), o.read_params(-1)
        o.step(eta, rho)
        o.couple()
        if t >= 300:
            G = Xd.T @ (Xd @ x - yd) / n + float(np.float32(lam)) * (x - y)
            tail.append(G @ G)
    assert np.mean(tail) <= 4 * Lc**2 * rho**2 * 1.05


def test_invalid_configs_rejected():
    assert O.param_count(O.make_config(O.MODEL_FLAT, K=1, flat_d=0)) == -1
    assert O.param_count(O.make_config(O.MODEL_MLP, widths=(4, 0, 2), K=1, batch=1)) == -1
    assert O.param_count(O.make_config(O.MODEL_LSQ, widths=(256,), K=4, batch=32, n_samples=4096)) == 256
    assert O.param_count(O.make_config(O.MODEL_RESMLP, widths=(3072, 4096, 4096, 4096, 4096, 1000), K=1, batch=1)) == 67027944
    assert O.param_count(O.make_config(O.MODEL_MLP, widths=(3072, 2048, 2048, 2048, 100), K=1, batch=1)) == 14891108
    assert O.param_count(O.make_config(O.MODEL_MLP, widths=(784, 1024, 10), K=1, batch=1)) == 814090


# ------------------------------------------------------------------------------------------- asynchronous progress
def _expected_mask(seed, t, K, active_num, budget):
    """The stated rule, written out: ready if H_act mod 256 < active_num; served in (H_ord, k) order up to the budget."""
    ta, to = O.lib().oracle_tag_active(), O.lib().oracle_tag_order()
    ready = [O.hash5(seed, ta, t, k, 0) % 256 < active_num for k in range(K)]
    order = sorted((O.hash5(seed, to, t, k, 0), k) for k in range(K) if ready[k])
    served = {k for _, k in order[:max(budget, 0)]}
    return np.array([1 if k in served else 0 for k in range(K)], dtype=np.int32)


def test_async_progress_mask_counters_and_exact_trigger():
    # Algorithm 2: per-worker counters t_x^(i) advance independently and the sync fires when their sum reaches n tau
    K, tau, d, num, seed = 5, 3, 4, 128, 77
    o, x0, y0, g1, g2 = _flat_oracle(K=K, d=d, tau=tau, lam=0.2, seed=seed, active_num=num, beta=0.0, eta_prime=1.0)
    ready_hits, ready_trials, syncs, unequal = 0, 0, 0, False
    window = []
    for t in range(300):
        before = o.read_state()
        _, _, t_x = o.counters()
        budget = K * tau - int(t_x.sum())
        o.step(0.05, 0.05)
        act = o.read_active()
        np.testing.assert_array_equal(act, _expected_mask(seed, t, K, num, budget))
        after = o.read_state()
        _, _, t_x2 = o.counters()
        np.testing.assert_array_equal(t_x2 - t_x, act)
        assert t_x2.sum() <= K * tau
        for k in range(K):
            if act[k]:
                window.append(after["x"][k].copy())
            else:  # a waiting worker is untouched
                np.testing.assert_array_equal(after["x"][k], before["x"][k])
                np.testing.assert_array_equal(after["v"][k], before["v"][k])
        if budget >= K:  # the budget did not bind: activity is the plain Bernoulli(num/256) draw
            ready_hits += int(act.sum())
            ready_trials += K
        if o.should_couple():
            assert t_x2.sum() == K * tau and len(window) == K * tau
            unequal |= len(set(t_x2.tolist())) > 1
            assert o.couple() == 0
            # beta = 0, eta' = 1: the centre is the mean of exactly the n tau iterates collected, whoever produced them
            np.testing.assert_allclose(o.read_params(-1), np.mean(window, axis=0), rtol=1e-12, atol=1e-14)
            window = []
            syncs += 1
        else:
            assert t_x2.sum() < K * tau
    assert syncs > 20 and unequal
    p = ready_hits / ready_trials
    assert abs(p - 0.5) < 4 * np.sqrt(0.25 / ready_trials)


def test_always_ready_is_the_lock_step_schedule_and_waiting_for_sync_is_an_error():
    a, *_ = _flat_oracle(K=3, d=4, tau=2, lam=0.2, seed=5)
    b, *_ = _flat_oracle(K=3, d=4, tau=2, lam=0.2, seed=5, active_num=256)
    c, *_ = _flat_oracle(K=3, d=4, tau=2, lam=0.2, seed=5, active_num=0)
    for t in range(6):
        for o in (a, b, c):
            o.step(0.05, 0.05)
            assert (o.read_active() == 1).all()
            if o.should_couple():
                assert o.couple() == 0
    np.testing.assert_array_equal(a.read_state()["x"], b.read_state()["x"])
    np.testing.assert_array_equal(a.read_state()["x"], c.read_state()["x"])
    a.step(0.05, 0.05)
    a.step(0.05, 0.05)
    assert a.should_couple()
    x = a.read_state()["x"].copy()
    assert O.lib().oracle_step(a._h, 0.05, 0.05) == 4  # the sync is due: nobody may step
    np.testing.assert_array_equal(a.read_state()["x"], x)
    assert a.counters()[0] == 8


# ------------------------------------------------------------------------------------------- Langevin noise
def test_philox_matches_published_known_answers():
    for line in open(os.path.join(GOLD, "philox4x32_10_kat.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        v = [int(x, 16) for x in line.split()]
        assert O.philox(v[0:4], v[4:6]) == v[6:10]


def test_noise_is_standard_normal_and_keyed_by_all_of_its_arguments():
    z = np.array([O.noise4(9, 3, 2, 1, g) for g in range(50000)])  # 200000 draws
    flat = z.ravel()
    n = flat.size
    assert abs(flat.mean()) < 4 / np.sqrt(n)
    assert abs(flat.var() - 1) < 4 * np.sqrt(2 / n)
    assert abs(np.mean(flat**3)) < 4 * np.sqrt(15 / n)          # skewness 0
    assert abs(np.mean(flat**4) - 3) < 4 * np.sqrt(96 / n)      # kurtosis 3
    c = np.corrcoef(z.T)
    assert np.abs(c - np.eye(4)).max() < 4 / np.sqrt(len(z))   # the four lanes are uncorrelated
    # Kolmogorov distance to the normal CDF
    from scipy import stats
    assert stats.kstest(flat[:50000], "norm").pvalue > 1e-3
    base = O.noise4(9, 3, 2, 1, 7)
    for other in (O.noise4(10, 3, 2, 1, 7), O.noise4(9, 4, 2, 1, 7), O.noise4(9, 3, 3, 1, 7), O.noise4(9, 3, 2, 0, 7), O.noise4(9, 3, 2, 1, 8),
                  O.noise4(9 + 2**32, 3, 2, 1, 7), O.noise4(9, 3 + 2**32, 2, 1, 7)):
        assert not np.allclose(base, other)
    np.testing.assert_array_equal(base, O.noise4(9, 3, 2, 1, 7))


def test_langevin_step_adds_sqrt_2_eta_T_noise_and_samples_the_kernel_gibbs_density():
    # zero gradients, mu = 0, fixed centre: x_{t+1} = (1 - eta lambda) x_t + eta lambda y + sqrt(2 eta T) xi is an AR(1) chain whose
    # stationary law is N(y, 2 eta T / (1 - (1 - eta lambda)^2)) -> the Gibbs density exp(-(lambda/2)||x - y||^2 / T) as eta -> 0
    K, d, eta, lam, T = 2, 4000, 0.05, 2.0, 0.3
    cfg = O.make_config(O.MODEL_FLAT, K=K, flat_d=d, mu=0.0, lam=lam, tau=10**6, noise_temp=T, seed=4)
    y0 = np.full(d, 1.5)
    o = O.Oracle(cfg, None, None, np.tile(y0, (K, 1)), y0)
    z = np.zeros((K, d), np.float32)
    o.set_external_grads(z, z)
    e, l, Tf = (float(np.float32(v)) for v in (eta, lam, T))
    o.step(eta, 0.0)
    x1 = o.read_state()["x"]
    # first step from x = y: pure noise with variance 2 eta T, and exactly the tabulated normals
    want = np.concatenate([O.noise4(4, 0, 1, 0, g) for g in range(d // 4)])
    np.testing.assert_allclose(x1[1] - y0, np.sqrt(2 * e * Tf) * want, rtol=1e-12, atol=1e-15)
    assert abs((x1 - y0).var() / (2 * e * Tf) - 1) < 0.05
    for _ in range(150):
        o.step(eta, 0.0)
    var = (o.read_state()["x"] - y0).var()
    stationary = 2 * e * Tf / (1 - (1 - e * l) ** 2)
    assert abs(var / stationary - 1) < 0.05
    assert abs(stationary / (Tf / l) - 1) < 0.06  # close to the continuous-time Gibbs variance T / lambda


def test_zero_temperature_is_the_noise_free_step_and_noise_enters_the_iterate_sum():
    a, x0, y0, g1, g2 = _flat_oracle(K=2, d=9, tau=3, lam=0.2, seed=5)
    b, *_ = _flat_oracle(K=2, d=9, tau=3, lam=0.2, seed=5, noise_temp=0.0)
    c, *_ = _flat_oracle(K=2, d=9, tau=3, lam=0.2, seed=5, noise_temp=0.5)
    for o in (a, b, c):
        o.step(0.05, 0.05)
    np.testing.assert_array_equal(a.read_state()["x"], b.read_state()["x"])
    sc = c.read_state()
    assert not np.allclose(sc["x"], a.read_state()["x"])
    np.testing.assert_array_equal(sc["acc"], sc["x"])  # the accumulated iterate is the noisy one
    # d = 9: the last group is partial (one valid lane); segment 0, groups 0..2
    sigma = np.sqrt(2 * float(np.float32(0.05)) * float(np.float32(0.5)))
    z = np.concatenate([O.noise4(5, 0, 1, 0, g) for g in range(3)])[:9]
    np.testing.assert_allclose(sc["x"][1] - a.read_state()["x"][1], sigma * z, rtol=1e-9, atol=1e-14)


def test_noise_segments_follow_the_layers():
    # W_l is segment 2l and b_l segment 2l + 1; the group index restarts in every segment
    widths = (3, 5, 2)
    X, labels = synth.gaussian_mixture(20, 3, 2, seed=1)
    w0 = synth.mlp_init(widths, seed=1).astype(np.float64)
    mk = lambda T: O.Oracle(O.make_config(O.MODEL_MLP, widths=widths, K=1, batch=4, n_samples=20, mu=0.0, tau=100, seed=8, noise_temp=T), X, labels, w0[None], w0)
    a, b = mk(0.0), mk(1.0)
    a.step(0.1, 0.0)
    b.step(0.1, 0.0)
    diff = (b.read_params(0) - a.read_params(0)) / np.sqrt(2 * float(np.float32(0.1)))
    segs = [(0, 15), (1, 5), (2, 10), (3, 2)]
    off = 0
    for seg, ln in segs:
        z = np.concatenate([O.noise4(8, 0, 0, seg, g) for g in range((ln + 3) // 4)])[:ln]
        np.testing.assert_allclose(diff[off:off + ln], z, rtol=1e-9, atol=1e-12)
        off += ln


# ------------------------------------------------------------------------------------------- stationary kernels (Corollary 8)
KERNELS = [(O.KERNEL_GAUSSIAN, 0.0), (O.KERNEL_EXP_POWER, 1.0), (O.KERNEL_EXP_POWER, 1.5), (O.KERNEL_EXP_POWER, 2.0), (O.KERNEL_CAUCHY, 0.7), (O.KERNEL_MATERN32, 0.0)]


@pytest.mark.parametrize("kind,param", KERNELS)
def test_kernel_pull_is_the_gradient_of_the_kernel(kind, param):
    # grad_z phi(||z||) = w(||z||) z: central finite differences of the kernel itself against the weight the step uses
    rng = np.random.default_rng(kind * 10 + int(param * 4))
    lam = 0.8
    for scale in (0.05, 1.0, 7.0):
        z = scale * rng.standard_normal(6)
        w = O.kernel_weight(kind, lam, param, np.linalg.norm(z))
        for i in range(6):
            h = 1e-6 * max(1.0, abs(z[i]))
            zp, zm = z.copy(), z.copy()
            zp[i] += h
            zm[i] -= h
            fd = (O.kernel_phi(kind, lam, param, np.linalg.norm(zp)) - O.kernel_phi(kind, lam, param, np.linalg.norm(zm))) / (2 * h)
            assert abs(fd - w * z[i]) <= 1e-7 * max(1.0, abs(w * z[i])), (scale, i, fd, w * z[i])
    # the kernel vanishes at the centre and grows with the distance (a pull, never a push)
    assert O.kernel_phi(kind, lam, param, 0.0) == 0.0
    rs = np.linspace(0.01, 20, 200)
    assert all(O.kernel_weight(kind, lam, param, r) > 0 for r in rs)
    assert np.all(np.diff([O.kernel_phi(kind, lam, param, r) for r in rs]) > 0)


def test_kernel_family_members_and_their_gaussian_limits():
    from scipy.special import gamma as Gamma, kv

    lam = 1.7
    for r in (0.0, 0.3, 2.0, 11.0):
        # exponential-power family of the remark after Corollary 8, Gaussian when the exponent is 2
        assert O.kernel_phi(O.KERNEL_EXP_POWER, lam, 2.0, r) == O.kernel_phi(O.KERNEL_GAUSSIAN, lam, 0.0, r) == 0.5 * lam * r * r
        assert O.kernel_weight(O.KERNEL_EXP_POWER, lam, 2.0, r) == lam
        assert np.isclose(O.kernel_phi(O.KERNEL_EXP_POWER, lam, 1.0, r), lam * r, rtol=1e-15)
        # Cauchy: exp(-phi) is the Cauchy / Student profile (1 + r^2 / s^2)^(-lam s^2 / 2); wide scale -> Gaussian
        s = 0.9
        assert np.isclose(np.exp(-O.kernel_phi(O.KERNEL_CAUCHY, lam, s, r)), (1 + r * r / (s * s)) ** (-lam * s * s / 2), rtol=1e-13)
        assert np.isclose(O.kernel_weight(O.KERNEL_CAUCHY, lam, 1e9, r), lam, rtol=1e-12)
        # Matern class with smoothness 3/2 and length scale l: the textbook correlation 2^(1-nu)/Gamma(nu) u^nu K_nu(u), u = sqrt(2 nu) r / l
        if r > 0:
            nu, ell = 1.5, np.sqrt(3.0 / lam)
            u = np.sqrt(2 * nu) * r / ell
            assert np.isclose(np.exp(-O.kernel_phi(O.KERNEL_MATERN32, lam, 0.0, r)), 2 ** (1 - nu) / Gamma(nu) * u ** nu * kv(nu, u), rtol=1e-10)
    assert np.isclose(O.kernel_weight(O.KERNEL_MATERN32, lam, 0.0, 1e-9), lam, rtol=1e-8)
    # tail condition (i) of Corollary 8 (phi >= c r^a for large r) for the exponential-power and Matern members
    assert O.kernel_phi(O.KERNEL_MATERN32, lam, 0.0, 50.0) >= 0.5 * np.sqrt(lam) * 50.0
    # invalid parameters are refused
    for kind, param in ((O.KERNEL_EXP_POWER, 0.5), (O.KERNEL_EXP_POWER, 2.5), (O.KERNEL_CAUCHY, 0.0), (7, 0.0)):
        cfg = O.make_config(O.MODEL_FLAT, K=1, flat_d=3, kernel_kind=kind, kernel_param=param)
        assert not O.lib().oracle_create(O.C.byref(cfg), None, None, O._ptr(np.zeros(3)), O._ptr(np.zeros(3)), None)


@pytest.mark.parametrize("kind,param", KERNELS)
def test_worker_step_with_a_stationary_kernel(kind, param):
    K, d = 3, 9
    x0, y0, g1, g2 = synth.flat_problem(K, d, seed=5)
    lam = 0.6
    hp = dict(K=K, flat_d=d, lam=lam, tau=2, stale_max=1, seed=3)
    o = O.Oracle(O.make_config(O.MODEL_FLAT, kernel_kind=kind, kernel_param=param, **hp), None, None, x0, y0)
    o.set_external_grads(g1, g2)
    ref = O.Oracle(O.make_config(O.MODEL_FLAT, **hp), None, None, x0, y0)  # Gaussian kernel
    ref.set_external_grads(g1, g2)
    for t in range(5):
        before = o.read_state()
        _, _, ver = o.read_schedule(t) if t == 0 else (None, None, None)
        o.step(0.05, 0.1)
        w = o.read_pull_weights()
        # the weight is w(||x_k - y||) at the state before the step and the centre version the worker read (the current
        # one here except for stale reads, which the Gaussian run below covers through its identical schedule)
        if t == 0:
            r = np.linalg.norm(before["x"] - before["y"][None, :], axis=1)
            np.testing.assert_allclose(w, [O.kernel_weight(kind, float(np.float32(lam)), float(np.float32(param)), ri) for ri in r], rtol=1e-13)
        if o.should_couple():
            assert o.couple() == 0
        ref.step(0.05, 0.1)
        if ref.should_couple():
            assert ref.couple() == 0
        if kind == O.KERNEL_GAUSSIAN or (kind == O.KERNEL_EXP_POWER and param == 2.0):
            np.testing.assert_array_equal(o.read_state()["x"], ref.read_state()["x"])  # the Gaussian path, bit for bit
            np.testing.assert_array_equal(o.read_state()["y"], ref.read_state()["y"])
    if kind not in (O.KERNEL_GAUSSIAN,) and not (kind == O.KERNEL_EXP_POWER and param == 2.0):
        assert not np.allclose(o.read_state()["x"], ref.read_state()["x"])
    # one worker, one step: the step IS the Gaussian step with lambda replaced by this worker's weight (up to the fp32
    # value the configuration carries lambda in)
    a = O.Oracle(O.make_config(O.MODEL_FLAT, K=1, flat_d=d, lam=lam, kernel_kind=kind, kernel_param=param), None, None, x0[:1], y0)
    a.set_external_grads(g1[:1], g2[:1])
    a.step(0.05, 0.1)
    wk = a.read_pull_weights()[0]
    b = O.Oracle(O.make_config(O.MODEL_FLAT, K=1, flat_d=d, lam=wk), None, None, x0[:1], y0)
    b.set_external_grads(g1[:1], g2[:1])
    b.step(0.05, 0.1)
    np.testing.assert_allclose(a.read_state()["x"], b.read_state()["x"], rtol=1e-6)
    np.testing.assert_allclose(a.read_state()["v"], b.read_state()["v"], rtol=1e-6, atol=1e-9)


# ------------------------------------------------------------------------------------------- synchronous data parallelism (Section 5.2)
@pytest.mark.parametrize("model", ["lsq", "mlp"])
def test_dp_average_is_sam_on_the_union_of_the_workers_minibatches(model):
    # DP-SGD / DP-SAM aggregate the workers' gradients at every iteration: with equal minibatch sizes the mean of the K
    # per-worker gradients is the gradient of the mean loss over the union of the K minibatches, at both points of the SAM step
    K, B = 3, 8
    if model == "lsq":
        X, Y, _ = synth.least_squares_data(64, 12, noise=0.01, seed=7)
        w0 = np.random.default_rng(1).standard_normal(12)
        mk = dict(model=O.MODEL_LSQ, widths=(12,))
    else:
        widths = (6, 8, 4)
        X, Y = synth.gaussian_mixture(64, 6, 4, seed=1)
        w0 = synth.mlp_init(widths, seed=2).astype(np.float64)
        mk = dict(model=O.MODEL_MLP, widths=widths)
    d = len(w0)
    x0 = np.repeat(w0[None, :], K, axis=0)
    hp = dict(lam=0.0, tau=1, seed=11, mu=0.9)
    o = O.Oracle(O.make_config(mk["model"], widths=mk["widths"], K=K, batch=B, n_samples=64, dp_average=1, **hp), X, Y, x0, w0)
    idx, _, _ = o.read_schedule(0)
    union = idx.reshape(-1)
    cu = O.make_config(mk["model"], widths=mk["widths"], K=1, batch=K * B, n_samples=64)
    rho, gam = float(np.float32(0.1)), float(np.float32(1e-12))
    _, gb1 = O.loss_grad(cu, X, Y, w0, union)
    xp = w0 + rho * gb1 / (np.linalg.norm(gb1) + gam)
    _, gb2 = O.loss_grad(cu, X, Y, xp, union)
    o.step(0.05, 0.1)
    g1, g2, oxp = o.read_grads()
    for k in range(K):
        np.testing.assert_allclose(g1[k], gb1, rtol=1e-11, atol=1e-14)
        np.testing.assert_allclose(oxp[k], xp, rtol=1e-12)
        np.testing.assert_allclose(g2[k], gb2, rtol=1e-10, atol=1e-14)
    _, n1, _ = o.read_step_info()
    np.testing.assert_allclose(n1, np.linalg.norm(gb1), rtol=1e-12)
    # the update is the single-worker step driven by the union-batch gradients (gradient-fed model, which has no modes)
    f = O.Oracle(O.make_config(O.MODEL_FLAT, K=1, flat_d=d, **hp), None, None, w0[None, :], w0)
    f.set_external_grads(gb1[None, :], gb2[None, :])
    f.step(0.05, 0.1)
    s = o.read_state()
    for k in range(K):
        np.testing.assert_allclose(s["x"][k], f.read_state()["x"][0], rtol=1e-6, atol=1e-9)
        np.testing.assert_array_equal(s["x"][k], s["x"][0])  # the replicas of a data-parallel job stay identical
    # without the flag the workers use their own gradients and drift apart
    p = O.Oracle(O.make_config(mk["model"], widths=mk["widths"], K=K, batch=B, n_samples=64, **hp), X, Y, x0, w0)
    p.step(0.05, 0.1)
    assert not np.array_equal(p.read_state()["x"][1], p.read_state()["x"][0])
    # asynchronous progress contradicts the synchronous aggregation
    bad = O.make_config(O.MODEL_FLAT, K=2, flat_d=3, dp_average=1, active_num=100)
    assert not O.lib().oracle_create(O.C.byref(bad), None, None, O._ptr(np.zeros((2, 3))), O._ptr(np.zeros(3)), None)


# ------------------------------------------------------------------------------------------- convolutional model
def _torch_cnn_loss(channels, dense, H, W, params, Xb, yb):
    """Independent statement of the convolutional model with torch's own conv2d / max_pool2d (double), loss and autograd gradient."""
    import torch.nn.functional as F

    p = torch.tensor(params, dtype=torch.float64, requires_grad=True)
    x = torch.tensor(Xb, dtype=torch.float64).reshape(len(Xb), channels[0], H, W)
    off = 0
    for l in range(len(channels) - 1):
        ci, co = channels[l], channels[l + 1]
        Wt = p[off:off + co * ci * 9].reshape(co, ci, 3, 3)
        off += co * ci * 9
        b = p[off:off + co]
        off += co
        x = F.max_pool2d(F.relu(F.conv2d(x, Wt, b, stride=1, padding=1)), 2)
    x = x.flatten(1)
    widths = [x.shape[1]] + list(dense)
    for l in range(len(widths) - 1):
        Wl = p[off:off + widths[l] * widths[l + 1]].reshape(widths[l + 1], widths[l])
        off += widths[l] * widths[l + 1]
        b = p[off:off + widths[l + 1]]
        off += widths[l + 1]
        x = x @ Wl.T + b
        if l < len(widths) - 2:
            x = F.relu(x)
    assert off == len(params)
    loss = F.cross_entropy(x, torch.tensor(yb, dtype=torch.long))
    loss.backward()
    return float(loss.detach()), p.grad.numpy(), x.detach().numpy()


@pytest.mark.parametrize("channels,dense,H,W", [((2, 3), (5, 4), 4, 6), ((3, 4, 5), (7, 3), 8, 8), ((1, 2, 2, 3), (3,), 8, 8)])
def test_cnn_gradient_vs_torch_conv_autograd_and_finite_differences(channels, dense, H, W):
    n, B = 30, 5
    classes = dense[-1]
    X, labels = synth.gaussian_mixture(n, channels[0] * H * W, classes, seed=3)
    params = synth.cnn_init(channels, dense, H, W, seed=4).astype(np.float64)
    params += 0.05 * np.random.default_rng(5).standard_normal(params.shape)  # nonzero biases
    cfg = O.make_config(O.MODEL_CNN, widths=tuple(channels) + tuple(dense), K=1, batch=B, n_samples=n, n_conv=len(channels) - 1, img_h=H, img_w=W)
    assert O.param_count(cfg) == synth.cnn_param_count(channels, dense, H, W) == len(params)
    idx = np.array([3, 17, 0, 29, 11], dtype=np.int32)
    loss, grad = O.loss_grad(cfg, X, labels, params, idx)
    tl, tg, tlogits = _torch_cnn_loss(channels, dense, H, W, params, X[idx], labels[idx])
    np.testing.assert_allclose(O.forward(cfg, X, params, idx), tlogits, rtol=1e-11, atol=1e-12)
    assert abs(loss - tl) <= 1e-12 * abs(tl)
    np.testing.assert_allclose(grad, tg, rtol=1e-9, atol=1e-13)
    # central finite differences on a sample of coordinates of every parameter block
    rng = np.random.default_rng(6)
    for j in rng.choice(len(params), 25, replace=False):
        h = 1e-6
        pp, pm = params.copy(), params.copy()
        pp[j] += h
        pm[j] -= h
        fd = (O.loss_grad(cfg, X, labels, pp, idx)[0] - O.loss_grad(cfg, X, labels, pm, idx)[0]) / (2 * h)
        assert abs(fd - grad[j]) <= 1e-6 * max(1.0, abs(grad[j])), (j, fd, grad[j])
    # bf16 mode: exact where every operand is representable (dyadic inputs and weights, one convolution), close otherwise
    c16 = O.make_config(O.MODEL_CNN, widths=tuple(channels) + tuple(dense), K=1, batch=B, n_samples=n, n_conv=len(channels) - 1, img_h=H, img_w=W,
                        gemm_dtype=O.GEMM_BF16)
    l16, g16 = O.loss_grad(c16, X, labels, params, idx)
    assert 0 < np.linalg.norm(g16 - grad) / np.linalg.norm(grad) < 5e-2 and abs(l16 - loss) < 5e-2 * abs(loss)
    # invalid geometry is refused
    assert O.param_count(O.make_config(O.MODEL_CNN, widths=(2, 3, 4), K=1, batch=1, n_conv=1, img_h=5, img_w=4)) == -1
    assert O.param_count(O.make_config(O.MODEL_CNN, widths=(2, 3, 4), K=1, batch=1, n_conv=2, img_h=4, img_w=4)) == -1


def test_cnn_step_runs_the_same_sam_step_as_the_other_models():
    # the step itself is model-independent: with the convolutional model it equals the gradient-fed step driven by that model's gradients
    channels, dense, H, W = (2, 3), (4, 3), 4, 4
    n, B, K = 24, 6, 2
    X, labels = synth.gaussian_mixture(n, channels[0] * H * W, 3, seed=8)
    w0 = synth.cnn_init(channels, dense, H, W, seed=9).astype(np.float64)
    xs = np.stack([w0, w0 + 0.01 * np.random.default_rng(1).standard_normal(w0.shape)])
    kw = dict(K=K, lam=0.5, tau=2, seed=5)
    geo = dict(widths=channels + dense, n_conv=1, img_h=H, img_w=W, batch=B, n_samples=n)
    o = O.Oracle(O.make_config(O.MODEL_CNN, **geo, **kw), X, labels, xs, w0)
    idx, _, _ = o.read_schedule(0)
    c1 = O.make_config(O.MODEL_CNN, **dict(geo, batch=B), K=1)
    rho, gam = float(np.float32(0.1)), float(np.float32(1e-12))
    g1 = np.stack([O.loss_grad(c1, X, labels, xs[k], idx[k])[1] for k in range(K)])
    xp = np.stack([xs[k] + rho * g1[k] / (np.linalg.norm(g1[k]) + gam) for k in range(K)])
    g2 = np.stack([O.loss_grad(c1, X, labels, xp[k], idx[k])[1] for k in range(K)])
    o.step(0.05, 0.1)
    f = O.Oracle(O.make_config(O.MODEL_FLAT, flat_d=len(w0), **kw), None, None, xs, w0)
    f.set_external_grads(g1, g2)
    f.step(0.05, 0.1)
    for key in ("x", "v", "acc"):
        assert np.linalg.norm(f.read_state()[key] - o.read_state()[key]) <= 1e-6 * np.linalg.norm(o.read_state()[key]), key
