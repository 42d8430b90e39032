"""Pins for the oracle's cost functions and hand-derived derivatives.

Nothing here goes through the oracle's derivative code to produce an expected value:
expected values are central finite differences of the oracle's *cost*, reverse-mode
autodiff of a forward-only restatement of the cost in torch (fp64), library routines
(torch cross_entropy, scikit-learn's logistic regression) or dense linear algebra."""
import numpy as np
import pytest
import torch

import oracle
from oracle import Level
from oracle import levels as olv
from oracle.bf16 import round_to_bf16
import synth_inputs as si
from tests.oracle_build import logreg_levels, quadratic_levels, reweight_levels, three_levels



def central_fd(f, x, eps=1e-6):
    g = np.zeros_like(x)
    for j in range(x.size):
        e = np.zeros_like(x); e[j] = eps
        g[j] = (f(x + e) - f(x - e)) / (2 * eps)
    return g


def rel(a, b):
    return np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300)


# ------------------------------------------------------------------ bf16 rounding
def test_bf16_rounding_matches_library_conversion():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-20, 20, 20000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38]])
    x32 = x.astype(np.float32)
    ref = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(round_to_bf16(x32), ref)
    # ties go to the even mantissa: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert round_to_bf16(np.array([1.00390625]))[0] == 1.0
    assert round_to_bf16(np.array([1.01171875]))[0] == 1.015625


# ------------------------------------------------------------------ logistic family
def _small_logreg(n=40, d=6, seed=3):
    inp = si.logreg_bilevel(seed, n, d, 24)
    inp.lam = np.abs(si.normal_f32(seed, 77, (d,))) * 0.1 + 0.01
    inp.w0 = si.normal_f32(seed, 78, (d,)) * 0.3
    return logreg_levels(inp)


def test_logreg_cost_is_mean_logloss():
    lo, up = _small_logreg()
    w = lo.params
    z = torch.from_numpy(lo.X) @ torch.from_numpy(w)
    t = torch.from_numpy((lo.y + 1) / 2)
    ref = torch.nn.functional.binary_cross_entropy_with_logits(z, t).item()
    lam = up.params
    assert abs(oracle.levels.cost(lo) - (ref + 0.5 * np.sum(lam * w * w))) < 1e-14
    zv = torch.from_numpy(up.X) @ torch.from_numpy(w)
    refv = torch.nn.functional.binary_cross_entropy_with_logits(
        zv, torch.from_numpy((up.y + 1) / 2)).item()
    assert abs(oracle.levels.cost(up) - refv) < 1e-14


def test_logreg_grad_hvp_against_finite_differences():
    lo, up = _small_logreg()
    w = lo.params.copy()
    g_fd = central_fd(lambda x: olv.cost(lo, {id(lo): x}), w)
    assert rel(oracle.grad(lo, lo), g_fd) < 1e-8
    gl_fd = central_fd(lambda x: olv.cost(lo, {id(up): x}), up.params.copy())
    assert rel(oracle.grad(lo, up), gl_fd) < 1e-8
    gv_fd = central_fd(lambda x: olv.cost(up, {id(lo): x}), w)
    assert rel(oracle.grad(up, lo), gv_fd) < 1e-8
    assert np.all(oracle.grad(up, up) == 0.0)
    rng = np.random.default_rng(1)
    for _ in range(3):
        u = rng.standard_normal(w.size)
        eps = 1e-6
        hv_fd = (oracle.grad(lo, lo, {id(lo): w + eps * u})
                 - oracle.grad(lo, lo, {id(lo): w - eps * u})) / (2 * eps)
        assert rel(oracle.hvp(lo, u), hv_fd) < 1e-8
    # second difference of the cost itself pins u^T H u without using grad
    u = rng.standard_normal(w.size)
    e = 1e-4
    c0, cp, cm = olv.cost(lo), olv.cost(lo, {id(lo): w + e * u}), olv.cost(lo, {id(lo): w - e * u})
    assert abs(u @ oracle.hvp(lo, u) - (cp - 2 * c0 + cm) / e ** 2) < 1e-6


def test_logreg_dense_hessian_and_symmetry():
    lo, up = _small_logreg(d=5)
    d = lo.params.size
    H = np.stack([oracle.hvp(lo, np.eye(d)[j]) for j in range(d)], axis=1)
    np.testing.assert_allclose(H, H.T, atol=1e-15)
    Ht = torch.autograd.functional.hessian(
        lambda w: torch.nn.functional.softplus(
            -torch.from_numpy(lo.y) * (torch.from_numpy(lo.X) @ w)).mean()
        + 0.5 * (torch.from_numpy(up.params) * w * w).sum(), torch.from_numpy(lo.params))
    np.testing.assert_allclose(H, Ht.numpy(), atol=1e-13)
    assert np.all(np.linalg.eigvalsh(H) > 0)


def test_logreg_mixed_second_derivative():
    lo, up = _small_logreg()
    q = np.random.default_rng(2).standard_normal(lo.params.size)
    fd = central_fd(lambda lam: oracle.grad(lo, lo, {id(up): lam}) @ q, up.params.copy())
    assert rel(oracle.mixed_vjp(lo, up, q), fd) < 1e-8


def test_logreg_stationary_point_matches_sklearn():
    """With a uniform weight decay the lower problem is scikit-learn's L2 logistic regression
    (C = 1/(n*lambda), no intercept): the oracle gradient must vanish at sklearn's solution."""
    from sklearn.linear_model import LogisticRegression
    inp = si.logreg_bilevel(11, 200, 5, 16)
    lam0 = 0.05
    inp.lam[:] = lam0
    lo, up = logreg_levels(inp)
    clf = LogisticRegression(C=1.0 / (200 * lam0), fit_intercept=False, tol=1e-12, max_iter=5000)
    clf.fit(inp.X.astype(np.float64), inp.y)
    g = oracle.grad(lo, lo, {id(lo): clf.coef_.ravel()})
    assert np.linalg.norm(g) < 1e-6
    # and a few hundred oracle GD steps move towards the same point
    oracle.lower_step(lo, 3000)
    assert rel(lo.params, clf.coef_.ravel()) < 1e-4


# ------------------------------------------------------------------ quadratic family
def test_quadratic_closed_forms():
    rng = np.random.default_rng(5)
    A, b = rng.standard_normal((12, 5)), rng.standard_normal(12)
    lam = rng.random(5) + 0.1
    lo, up = quadratic_levels(A, b, lam, rng.standard_normal((7, 5)), rng.standard_normal(7))
    H = A.T @ A + np.diag(lam)
    wstar = np.linalg.solve(H, A.T @ b)
    assert np.linalg.norm(oracle.grad(lo, lo, {id(lo): wstar})) < 1e-12
    u = rng.standard_normal(5)
    np.testing.assert_allclose(oracle.hvp(lo, u), H @ u, atol=1e-13)
    w = rng.standard_normal(5)
    g_fd = central_fd(lambda x: olv.cost(lo, {id(lo): x}), w)
    assert rel(oracle.grad(lo, lo, {id(lo): w}), g_fd) < 1e-8
    gv_fd = central_fd(lambda x: olv.cost(up, {id(lo): x}), w)
    assert rel(oracle.grad(up, lo, {id(lo): w}), gv_fd) < 1e-8


# ------------------------------------------------------------------ MLP family vs autodiff
def _t(x):
    return torch.from_numpy(np.array(x, dtype=np.float64))


def _torch_act(name, a):
    return torch.relu(a) if name == "relu" else torch.nn.functional.gelu(a)


def _torch_mlp_logits(widths, act, flat, X):
    h, o = X, 0
    L = len(widths) - 1
    for l in range(L):
        fin, fout = widths[l], widths[l + 1]
        W = flat[o:o + fout * fin].reshape(fout, fin); o += fout * fin
        b = flat[o:o + fout]; o += fout
        h = torch.nn.functional.linear(h, W, b)
        if l < L - 1:
            h = _torch_act(act, h)
    return h


def _torch_weightnet(theta, ell):
    H = si.WEIGHTNET_HIDDEN
    a1, b1, a2, b2 = theta[:H], theta[H:2 * H], theta[2 * H:3 * H], theta[3 * H]
    return torch.sigmoid(torch.relu(ell[:, None] * a1 + b1) @ a2 + b2)


def _torch_reweight_cost(inp, w, theta, lam, detach=True):
    z = _torch_mlp_logits(inp.widths, inp.activation, w, _t(inp.train.X))
    ell = torch.nn.functional.cross_entropy(z, torch.from_numpy(inp.train.y.astype(np.int64)),
                                            reduction="none")
    r = _torch_weightnet(theta, ell.detach() if detach else ell)
    c = (r * ell).mean()
    if lam is not None:
        o = 0
        for l in range(len(inp.widths) - 1):
            n = inp.widths[l] * inp.widths[l + 1]
            c = c + 0.5 * torch.exp(lam[l]) * (w[o:o + n] ** 2).sum()
            o += n + inp.widths[l + 1]
    return c


def _tiny_reweight(act, seed=21, widths=(7, 6, 5, 4), B=12):
    inp = si.reweight_bilevel(seed, widths, B, 0.4, activation=act)
    inp.w = inp.w + si.normal_f32(seed, 300, inp.w.shape) * 0.05     # non-zero biases too
    inp.theta = si.weightnet_init(seed, 200) * 3.0
    inp.theta[si.WEIGHTNET_HIDDEN:2 * si.WEIGHTNET_HIDDEN] = \
        si.normal_f32(seed, 301, (si.WEIGHTNET_HIDDEN,)) * 0.2
    return inp


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_mlp_reweight_derivatives_against_autograd(act):
    inp = _tiny_reweight(act)
    w_lv, th_lv = reweight_levels(inp, bf16=False)
    lam_lv = Level(loss="mlp_ce", param_kind="logwd",
                   params=np.log([3e-2, 1e-2, 2e-2]), X=inp.val.X, y=inp.val.y,
                   constraints=[w_lv])
    w_lv.constraints = [th_lv, lam_lv]
    w = _t(inp.w).requires_grad_(True)
    th = _t(inp.theta).requires_grad_(True)
    lam = _t(lam_lv.params).requires_grad_(True)

    c = _torch_reweight_cost(inp, w, th, lam)
    assert abs(c.item() - olv.cost(w_lv)) < 1e-13
    gw, gth, glam = torch.autograd.grad(c, [w, th, lam], create_graph=True)
    assert rel(oracle.grad(w_lv, w_lv), gw.detach().numpy()) < 1e-12
    assert rel(oracle.grad(w_lv, th_lv), gth.detach().numpy()) < 1e-12
    assert rel(oracle.grad(w_lv, lam_lv), glam.detach().numpy()) < 1e-12

    rng = np.random.default_rng(4)
    for _ in range(2):
        u = rng.standard_normal(inp.w.size)
        hv, mth, mlam = torch.autograd.grad(gw @ _t(u), [w, th, lam], retain_graph=True)
        assert rel(oracle.hvp(w_lv, u), hv.numpy()) < 1e-11
        assert rel(oracle.mixed_vjp(w_lv, th_lv, u), mth.numpy()) < 1e-11
        assert rel(oracle.mixed_vjp(w_lv, lam_lv, u), mlam.numpy()) < 1e-11

    # upper cost: plain CE of the classifier on the clean batch
    zv = _torch_mlp_logits(inp.widths, act, w, _t(inp.val.X))
    cu = torch.nn.functional.cross_entropy(zv, torch.from_numpy(inp.val.y.astype(np.int64)))
    assert abs(cu.item() - olv.cost(th_lv)) < 1e-13
    (gu,) = torch.autograd.grad(cu, [w])
    assert rel(oracle.grad(th_lv, w_lv), gu.numpy()) < 1e-12
    assert np.all(oracle.grad(th_lv, th_lv) == 0.0)


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_mlp_reweight_frozen_costs_by_finite_differences(act):
    """Independent of autodiff: the two frozen cost functions differentiated numerically."""
    inp = _tiny_reweight(act, seed=22, widths=(5, 4, 3), B=9)
    w_lv, th_lv = reweight_levels(inp, bf16=False)
    M, Ws, bs, h, a, p, ell = olv._mlp_ce_state(w_lv, None)
    r = olv.wn_forward(th_lv.params, ell)[0]
    g_fd = central_fd(lambda x: olv.cost(w_lv, {id(w_lv): x}, r_fixed=r), w_lv.params.copy())
    assert rel(oracle.grad(w_lv, w_lv), g_fd) < 1e-7
    gt_fd = central_fd(lambda x: olv.cost(w_lv, {id(th_lv): x}, ell_fixed=ell),
                       th_lv.params.copy())
    assert rel(oracle.grad(w_lv, th_lv), gt_fd) < 1e-7
    # Hessian by columns is symmetric
    n = w_lv.params.size
    H = np.stack([oracle.hvp(w_lv, np.eye(n)[j]) for j in range(n)], axis=1)
    np.testing.assert_allclose(H, H.T, atol=1e-13)


def _tiny_three(act="gelu", seed=31, widths=(6, 5, 4, 3), B=10):
    inp = si.three_level(seed, widths, B, 0.3, activation=act)
    inp.w = inp.w + si.normal_f32(seed, 300, inp.w.shape) * 0.05
    inp.theta = si.weightnet_init(seed, 200) * 3.0
    inp.theta[si.WEIGHTNET_HIDDEN:2 * si.WEIGHTNET_HIDDEN] = \
        si.normal_f32(seed, 301, (si.WEIGHTNET_HIDDEN,)) * 0.2
    return inp


def _torch_detect_cost(widths, act, batch, w, theta, mu):
    z = _torch_mlp_logits(widths, act, w, _t(batch.X))
    ell = torch.nn.functional.cross_entropy(z, torch.from_numpy(batch.y.astype(np.int64)),
                                            reduction="none")
    r = _torch_weightnet(theta, ell)
    return ((r - _t(batch.clean)) ** 2).mean() + 0.5 * mu * (theta ** 2).sum()


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_weightnet_detect_derivatives_against_autograd(act):
    inp = _tiny_three(act)
    P1, P2, P3 = three_levels(inp, bf16=False)
    w = _t(inp.w).requires_grad_(True)
    th = _t(inp.theta).requires_grad_(True)
    c2 = _torch_detect_cost(inp.widths, act, inp.D2, w, th, inp.mu)
    assert abs(c2.item() - olv.cost(P2)) < 1e-13
    gth, gw = torch.autograd.grad(c2, [th, w], create_graph=True)
    assert rel(oracle.grad(P2, P2), gth.detach().numpy()) < 1e-12
    assert rel(oracle.grad(P2, P1), gw.detach().numpy()) < 1e-12
    rng = np.random.default_rng(6)
    for _ in range(2):
        q = rng.standard_normal(inp.theta.size)
        hv, mw = torch.autograd.grad(gth @ _t(q), [th, w], retain_graph=True)
        assert rel(oracle.hvp(P2, q), hv.numpy()) < 1e-11
        assert rel(oracle.mixed_vjp(P2, P1, q), mw.numpy()) < 1e-11
    # level 3 uses the same cost on its own batch without the mu term
    c3 = _torch_detect_cost(inp.widths, act, inp.D3, w, th, 0.0)
    assert abs(c3.item() - olv.cost(P3)) < 1e-13
    g3th, g3w = torch.autograd.grad(c3, [th, w])
    assert rel(oracle.grad(P3, P2), g3th.numpy()) < 1e-12
    assert rel(oracle.grad(P3, P1), g3w.numpy()) < 1e-12
    assert np.all(oracle.grad(P3, P3) == 0.0)


def test_three_level_classifier_cost_with_both_constraints():
    inp = _tiny_three("gelu")
    P1, P2, P3 = three_levels(inp, bf16=False)
    w = _t(inp.w).requires_grad_(True)
    th = _t(inp.theta).requires_grad_(True)
    lam = _t(inp.lam).requires_grad_(True)

    class _B:  # the classifier's own batch under the name the cost helper expects
        widths, activation, train = inp.widths, inp.activation, inp.D1
    c1 = _torch_reweight_cost(_B, w, th, lam)
    assert abs(c1.item() - olv.cost(P1)) < 1e-13
    gw, = torch.autograd.grad(c1, [w], create_graph=True)
    assert rel(oracle.grad(P1, P1), gw.detach().numpy()) < 1e-12
    q = np.random.default_rng(8).standard_normal(inp.w.size)
    hv, mlam, mth = torch.autograd.grad(gw @ _t(q), [w, lam, th])
    assert rel(oracle.hvp(P1, q), hv.numpy()) < 1e-11
    assert rel(oracle.mixed_vjp(P1, P3, q), mlam.numpy()) < 1e-11
    assert rel(oracle.mixed_vjp(P1, P2, q), mth.numpy()) < 1e-11


def test_bf16_level_quantises_matrices_and_hidden_activations():
    """A mixed-precision level evaluates its cost with bf16 operands in every matrix product:
    matrices and hidden activations rounded (torch's conversion is the reference), fp64
    everywhere else; the full-precision level does not."""
    inp = _tiny_reweight("relu", seed=23)
    inp.w = inp.w + si.normal_f32(23, 400, inp.w.shape) * 1e-3        # not bf16-representable
    w16, th16 = reweight_levels(inp, bf16=True)
    q = lambda t: t.to(torch.float32).to(torch.bfloat16).to(torch.float64)
    Ws, bs = olv.mlp_unpack(inp.widths, inp.w.astype(np.float64))
    h = _t(inp.train.X)
    for l, (W, b) in enumerate(zip(Ws, bs)):
        a = h @ q(_t(W)).T + _t(b)
        h = q(torch.relu(a)) if l < len(Ws) - 1 else a
    ell = torch.nn.functional.cross_entropy(h, torch.from_numpy(inp.train.y.astype(np.int64)),
                                            reduction="none")
    ref = (_torch_weightnet(_t(inp.theta), ell) * ell).mean().item()
    assert abs(olv.cost(w16) - ref) < 1e-13
    assert abs(olv.cost(reweight_levels(inp, bf16=False)[0]) - ref) > 1e-9
    # derivatives are straight-through: same formulas, evaluated on the quantised forward pass
    w64, th64 = reweight_levels(inp, bf16=False)
    assert rel(oracle.grad(w16, w16), oracle.grad(w64, w64)) < 5e-2


def test_fd_on_a_bf16_level_keeps_quantisation_offsets_frozen():
    """The finite difference on a mixed-precision level must see the perturbation, which is far
    below bf16 resolution: with frozen rounding offsets it agrees with the full-precision
    level's finite difference to within the quantisation error of the base point."""
    inp = _tiny_reweight("gelu", seed=29, widths=(8, 12, 10, 5), B=40)
    w16, th16 = reweight_levels(inp, bf16=True)
    w64, th64 = reweight_levels(inp, bf16=False)
    v = np.random.default_rng(3).standard_normal(inp.w.size)
    f16 = oracle.brj(w16, th16, v, "fd", eps0=1e-3, alpha=1.0)
    f64 = oracle.brj(w64, th64, v, "fd", eps0=1e-3, alpha=1.0)
    assert rel(f16, f64) < 5e-2
    # re-rounding the perturbed weights instead would wipe the perturbation out
    eps = 1e-3 / np.linalg.norm(v)
    naive = -(oracle.grad(w16, th16, {id(w16): w16.params + eps * v})
              - oracle.grad(w16, th16, {id(w16): w16.params - eps * v})) / (2 * eps)
    assert rel(naive, f64) > 10 * rel(f16, f64)


# ------------------------------------------------------------------ the two readings of a mixed-precision level
def _q(t):
    return t.to(torch.float32).to(torch.bfloat16).to(torch.float64)


def _theta_gradient_of_reweighted_mean(theta_np, ell):
    """d/dtheta mean_i sigmoid(net(ell_i)) * ell_i with the per-sample losses as data (autodiff)."""
    th = _t(theta_np).requires_grad_(True)
    c = (_torch_weightnet(th, ell.detach()) * ell.detach()).mean()
    (g,) = torch.autograd.grad(c, [th])
    return g.numpy()


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_plain_reading_rounds_the_matrices_only(act):
    """quant = "weights": the cost sees bf16-rounded matrices and nothing else rounded, and a
    finite-difference evaluation sees the displaced master with no rounding at all.  Expected values
    come from a forward-only restatement in torch and reverse-mode autodiff of it."""
    inp = _tiny_reweight(act, seed=37, widths=(8, 12, 10, 5), B=40)
    inp.w = inp.w + si.normal_f32(37, 400, inp.w.shape) * 1e-3        # master not bf16-representable
    w16, th16 = reweight_levels(inp, bf16=True, quant="weights")
    yt = torch.from_numpy(inp.train.y.astype(np.int64))

    def ell_at(flat, round_matrices):
        Ws, bs = olv.mlp_unpack(inp.widths, flat)
        h = _t(inp.train.X)
        for l, (W, b) in enumerate(zip(Ws, bs)):
            Wt = _q(_t(W)) if round_matrices else _t(W)
            a = h @ Wt.T + _t(b)
            h = _torch_act(act, a) if l < len(Ws) - 1 else a
        return torch.nn.functional.cross_entropy(h, yt, reduction="none")

    master = inp.w.astype(np.float64)
    ell = ell_at(master, True)
    ref = (_torch_weightnet(_t(inp.theta), ell) * ell).mean().item()
    assert abs(olv.cost(w16) - ref) < 1e-13
    # it differs from both the unrounded level and the bf16-operand reading
    assert abs(olv.cost(reweight_levels(inp, bf16=False)[0]) - ref) > 1e-9
    assert abs(olv.cost(reweight_levels(inp, bf16=True)[0]) - ref) > 1e-9
    # finite difference: master +- eps v, unrounded
    v = np.random.default_rng(5).standard_normal(inp.w.size)
    eps0 = 1e-3
    eps = eps0 / np.linalg.norm(v)
    gp = _theta_gradient_of_reweighted_mean(inp.theta, ell_at(master + eps * v, False))
    gm = _theta_gradient_of_reweighted_mean(inp.theta, ell_at(master - eps * v, False))
    got = oracle.brj(w16, th16, v, "fd", eps0=eps0, alpha=1.0)
    assert rel(got, -(gp - gm) / (2 * eps)) < 1e-9


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_operand_reading_displaces_layer_by_layer_with_frozen_offsets(act):
    """quant = "operands": in a finite-difference evaluation every hidden activation moves by exactly
    act(a+) - act(a) from its rounded base value, layer by layer, and the matrices by exactly eps V from
    their rounded values.  The restatement below carries base and displaced passes side by side and
    never forms a rounding offset; a wrong sign or a wrong layer index of one offset fails it."""
    inp = _tiny_reweight(act, seed=41, widths=(8, 12, 10, 9, 5), B=40)
    inp.w = inp.w + si.normal_f32(41, 400, inp.w.shape) * 1e-3
    w16, th16 = reweight_levels(inp, bf16=True)
    yt = torch.from_numpy(inp.train.y.astype(np.int64))
    master = inp.w.astype(np.float64)
    v = np.random.default_rng(6).standard_normal(inp.w.size)
    eps0 = 1e-3
    eps = eps0 / np.linalg.norm(v)
    Ws, bs = olv.mlp_unpack(inp.widths, master)
    Vs, cs = olv.mlp_unpack(inp.widths, v)
    nl = len(Ws)

    def displaced(sign):
        hb = hd = _t(inp.train.X)          # base (rounded) and displaced activations
        acts_b, acts_d = [], []
        for l in range(nl):
            Wq = _q(_t(Ws[l]))
            ab = hb @ Wq.T + _t(bs[l])
            ad = hd @ (Wq + sign * eps * _t(Vs[l])).T + _t(bs[l]) + sign * eps * _t(cs[l])
            acts_b.append(ab); acts_d.append(ad)
            if l < nl - 1:
                hb_next = _q(_torch_act(act, ab))
                hd = hb_next + (_torch_act(act, ad) - _torch_act(act, ab))
                hb = hb_next
        return acts_b, acts_d

    got_states = {}
    for sign in (+1.0, -1.0):
        acts_b, acts_d = displaced(sign)
        over = {id(w16): master + sign * eps * v, "frozen": {id(w16)}}
        M, _, _, h, a, p, ell = olv._mlp_ce_state(w16, over)
        _, _, _, hb, ab, _, _ = olv._mlp_ce_state(w16, None)
        for l in range(nl):
            np.testing.assert_allclose(a[l], acts_d[l].numpy(), rtol=0, atol=1e-13)
            np.testing.assert_allclose(ab[l], acts_b[l].numpy(), rtol=0, atol=1e-13)
            if l < nl - 1:       # h+- - h_base == act(a+-) - act(a_base), exactly this layer's
                lhs = h[l + 1] - hb[l + 1]
                rhs = (_torch_act(act, acts_d[l]) - _torch_act(act, acts_b[l])).numpy()
                np.testing.assert_allclose(lhs, rhs, rtol=0, atol=1e-15)
        got_states[sign] = torch.nn.functional.cross_entropy(acts_d[-1], yt, reduction="none")
    gp = _theta_gradient_of_reweighted_mean(inp.theta, got_states[+1.0])
    gm = _theta_gradient_of_reweighted_mean(inp.theta, got_states[-1.0])
    got = oracle.brj(w16, th16, v, "fd", eps0=eps0, alpha=1.0)
    assert rel(got, -(gp - gm) / (2 * eps)) < 1e-8
