"""Pins for the oracle's iterations and for the hypergradient they approximate.

Expected values come from dense linear algebra (matrix powers, numpy.linalg.solve, a
brute-force projected solve over the Krylov space), closed forms of a quadratic lower
level, brute-force finite differences of the upper loss after a converged lower solve, and
explicitly materialised Jacobians for the three-level chain."""
import numpy as np
import pytest
import torch

import oracle
from oracle import Level
from oracle import levels as olv
import synth_inputs as si
from tests.oracle_build import logreg_levels, quadratic_levels, three_levels
from tests.test_oracle_derivatives import (_t, _tiny_three, _torch_detect_cost,
                                           _torch_reweight_cost, central_fd, rel)



def _spd(d, seed, lo=0.2, hi=2.0):
    rng = np.random.default_rng(seed)
    Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    return Q @ np.diag(np.linspace(lo, hi, d)) @ Q.T


# ------------------------------------------------------------------ Neumann
def test_neumann_equals_truncated_matrix_power_series():
    H, v = _spd(7, 0), np.random.default_rng(1).standard_normal(7)
    for K, alpha in [(0, 0.3), (1, 0.3), (5, 0.4), (10, 0.01)]:
        A = np.eye(7) - alpha * H
        ref = alpha * sum(np.linalg.matrix_power(A, j) @ v for j in range(K + 1))
        np.testing.assert_allclose(oracle.neumann_solve(lambda t: H @ t, v, K, alpha), ref,
                                   rtol=0, atol=1e-13)


def test_neumann_error_bound_and_convergence_to_exact_solve():
    H, v = _spd(8, 2), np.random.default_rng(3).standard_normal(8)
    alpha = 1.0 / 2.0
    exact = np.linalg.solve(H, v)
    rho = np.linalg.norm(np.eye(8) - alpha * H, 2)
    prev = np.inf
    for K in [1, 4, 16, 64, 400]:
        err = np.linalg.norm(oracle.neumann_solve(lambda t: H @ t, v, K, alpha) - exact)
        assert err <= rho ** (K + 1) * np.linalg.norm(exact) * (1 + 1e-9) + 1e-14
        assert err < prev or err < 1e-13
        prev = err
    assert prev < 1e-12


# ------------------------------------------------------------------ CG
def test_cg_converges_in_d_steps_and_counts_iterations():
    H, v = _spd(8, 4), np.random.default_rng(5).standard_normal(8)
    q, it, status = oracle.cg_solve(lambda t: H @ t, v, 8)
    assert status == "ok" and it == 8
    np.testing.assert_allclose(q, np.linalg.solve(H, v), atol=1e-10)
    q, it, status = oracle.cg_solve(lambda t: H @ t, v, 50, tol=1e-6)
    assert status == "ok" and it <= 9
    assert np.linalg.norm(H @ q - v) <= 1e-6 * np.linalg.norm(v) * 1.0001


def test_cg_iterate_minimises_energy_norm_over_krylov_space():
    H, v = _spd(8, 6), np.random.default_rng(7).standard_normal(8)
    for K in [1, 2, 3, 5]:
        q, it, _ = oracle.cg_solve(lambda t: H @ t, v, K)
        V = np.stack([np.linalg.matrix_power(H, j) @ v for j in range(K)], axis=1)
        coef = np.linalg.solve(V.T @ H @ V, V.T @ v)          # Galerkin = H-norm projection
        np.testing.assert_allclose(q, V @ coef, atol=1e-9)
        assert it == K


def test_cg_reports_breakdown_on_indefinite_hessian():
    rng = np.random.default_rng(8)
    A, b = rng.standard_normal((6, 4)) * 0.1, rng.standard_normal(6)
    lo, up = quadratic_levels(A, b, np.array([-5.0, 0.3, 0.2, 0.1]), A, b)
    info = {}
    v = np.array([1.0, 0.0, 0.0, 0.0])
    out = oracle.brj(lo, up, v, "cg", K=5, info=info)
    assert info["status"] == "breakdown" and info["iters"] == 0
    np.testing.assert_array_equal(out, np.zeros(4))


# ------------------------------------------------------------------ finite difference
def test_fd_is_exact_for_the_weight_decay_constraint():
    """d/d(lambda) of the lower cost is 1/2 w^2, quadratic in w, so the central difference
    equals w * v (times alpha) for any epsilon."""
    inp = si.logreg_bilevel(13, 50, 6, 20)
    inp.w0 = si.normal_f32(13, 9, (6,))
    lo, up = logreg_levels(inp)
    v = np.random.default_rng(9).standard_normal(6)
    for eps0 in [1e-3, 0.01, 0.5]:
        np.testing.assert_allclose(oracle.brj(lo, up, v, "fd", eps0=eps0, alpha=0.7),
                                   -0.7 * lo.params * v, rtol=1e-9, atol=1e-14)
    assert np.all(oracle.brj(lo, up, np.zeros(6), "fd") == 0.0)


def test_fd_on_reweighting_tends_to_directional_derivative_of_the_theta_gradient():
    """As eps -> 0 the finite difference re-evaluates everything that depends on w, the
    detached weight-net input included, so its limit is the w-directional derivative of
    theta -> (1/B) sum_i l_i(w) d r(l_i(w); theta)/d theta, with O(eps^2) error."""
    from tests.test_oracle_derivatives import _tiny_reweight, _torch_mlp_logits, _torch_weightnet
    from tests.oracle_build import reweight_levels
    inp = _tiny_reweight("gelu", seed=41)
    w_lv, th_lv = reweight_levels(inp, bf16=False)
    v = np.random.default_rng(10).standard_normal(inp.w.size)
    w = _t(inp.w).requires_grad_(True)
    th = _t(inp.theta).requires_grad_(True)
    z = _torch_mlp_logits(inp.widths, "gelu", w, _t(inp.train.X))
    ell = torch.nn.functional.cross_entropy(z, torch.from_numpy(inp.train.y.astype(np.int64)),
                                            reduction="none")
    # G(w) = (1/B) sum_i l_i(w) * dr(l; theta)/dtheta at l = l_i(w): a vector-Jacobian product of
    # r w.r.t. theta with cotangent l/B, both factors kept attached to w
    r = _torch_weightnet(th, ell)
    G, = torch.autograd.grad(r, [th], grad_outputs=ell / ell.numel(), create_graph=True)
    limit = torch.stack([torch.autograd.grad(G[j], [w], retain_graph=True)[0] @ _t(v)
                         for j in range(inp.theta.size)]).numpy()
    errs = []
    nv = np.linalg.norm(v)
    # (small steps: the weight net's hidden ReLUs make the theta-gradient jump where a
    # per-sample loss crosses a kink, so the limit is approached only once no sample does)
    for eps in [1e-4, 1e-5]:
        out = oracle.brj(w_lv, th_lv, v, "fd", eps0=eps * nv, alpha=1.0)
        errs.append(np.linalg.norm(out + limit))
    assert errs[1] < errs[0] * 0.02 + 1e-12          # second-order in eps
    assert errs[1] < 1e-6 * max(1.0, np.linalg.norm(limit))


# ------------------------------------------------------------------ hypergradients
def _newton_solve_lower(lo, iters=60):
    d = lo.params.size
    for _ in range(iters):
        g = oracle.grad(lo, lo)
        H = np.stack([oracle.hvp(lo, np.eye(d)[j]) for j in range(d)], axis=1)
        lo.params = lo.params - np.linalg.solve(H, g)
    assert np.linalg.norm(oracle.grad(lo, lo)) <= 1e-12


def test_hypergradient_matches_brute_force_through_converged_lower_solve():
    """Eq. 1 with an exact inverse-Hessian solve equals d/d(lambda) C_upper(w*(lambda)),
    measured by central differences with the lower problem re-solved by Newton's method."""
    inp = si.logreg_bilevel(17, 60, 5, 30)
    inp.lam = (np.abs(si.normal_f32(17, 7, (5,))) * 0.1 + 0.02).astype(np.float32)
    lo, up = logreg_levels(inp)
    _newton_solve_lower(lo)

    def upper_of_lambda(lam):
        l2, u2 = logreg_levels(inp)
        u2.params = np.array(lam, dtype=np.float64)
        l2.params = lo.params.copy()
        _newton_solve_lower(l2, iters=25)
        return olv.cost(u2)

    brute = central_fd(upper_of_lambda, up.params.copy(), eps=1e-5)
    hg_cg = oracle.hypergrad_cg(lo, up, up, K=5)                 # d = 5: exact in 5 steps
    assert rel(hg_cg, brute) < 1e-6
    lmax = max(np.linalg.eigvalsh(np.stack([oracle.hvp(lo, e) for e in np.eye(5)], 1)))
    hg_nm = oracle.hypergrad_neumann(lo, up, up, K=4000, alpha=1.0 / lmax)
    assert rel(hg_nm, brute) < 1e-6
    # App. D.1: with few iterations CG is the closer of the two
    e_cg = rel(oracle.hypergrad_cg(lo, up, up, K=3), brute)
    e_nm = rel(oracle.hypergrad_neumann(lo, up, up, K=3, alpha=0.01), brute)
    assert e_cg < e_nm


def test_quadratic_lower_level_has_closed_form_best_response_and_hypergradient():
    rng = np.random.default_rng(11)
    A, b = rng.standard_normal((15, 6)), rng.standard_normal(15)
    Av, bv = rng.standard_normal((9, 6)), rng.standard_normal(9)
    lam = rng.random(6) + 0.1
    lo, up = quadratic_levels(A, b, lam, Av, bv)
    H = A.T @ A + np.diag(lam)
    wstar = np.linalg.solve(H, A.T @ b)
    lo.params = wstar.copy()
    # d w*/d lambda_j = -H^{-1} e_j w*_j  =>  d C_u / d lambda = -(w*) .* H^{-1} grad_w C_u
    closed = -wstar * np.linalg.solve(H, Av.T @ (Av @ wstar - bv))
    assert rel(oracle.hypergrad_cg(lo, up, up, K=6), closed) < 1e-9
    alpha = 1.0 / np.linalg.eigvalsh(H).max()
    assert rel(oracle.hypergrad_neumann(lo, up, up, K=20000, alpha=alpha), closed) < 1e-9
    # best response itself: many plain gradient steps reach the closed-form minimiser
    lo2, _ = quadratic_levels(A, b, lam, Av, bv)
    lo2.lr = alpha
    oracle.lower_step(lo2, 20000)
    assert rel(lo2.params, wstar) < 1e-9
    # and the Jacobian columns by brute force
    J = np.stack([(np.linalg.solve(H + np.diag(1e-6 * e), A.T @ b)
                   - np.linalg.solve(H - np.diag(1e-6 * e), A.T @ b)) / 2e-6 for e in np.eye(6)], 1)
    v = rng.standard_normal(6)
    assert rel(oracle.brj(lo, up, v, "cg", K=6), J.T @ v) < 1e-6


def test_lower_step_is_plain_gradient_descent():
    inp = si.logreg_bilevel(19, 30, 4, 10)
    lo, up = logreg_levels(inp)
    w = lo.params.copy()
    for _ in range(3):
        w = w - inp.lr * central_fd(lambda x: olv.cost(lo, {id(lo): x}), w)
    oracle.lower_step(lo, 3)
    assert rel(lo.params, w) < 1e-8


def test_itd_equals_autodiff_through_the_unrolled_steps():
    """ITD-RMAD against reverse-mode autodiff (torch, fp64) of the upper cost through T explicit
    gradient-descent steps of the lower cost, for the logistic problem and for the reweighted MLP."""
    # logistic weight decay
    inp = si.logreg_bilevel(23, 50, 6, 20)
    inp.lam = (np.abs(si.normal_f32(23, 7, (6,))) * 0.1 + 0.02).astype(np.float32)
    lo, up = logreg_levels(inp)
    X, y, Xv, yv = _t(inp.X), _t(inp.y), _t(inp.Xv), _t(inp.yv)
    lam = _t(inp.lam).requires_grad_(True)
    w = _t(inp.w0)
    sp = torch.nn.functional.softplus
    for _ in range(7):
        wg = w.detach().requires_grad_(True) if not w.requires_grad else w
        c = sp(-y * (X @ wg)).mean() + 0.5 * (lam * wg * wg).sum()
        g, = torch.autograd.grad(c, [wg], create_graph=True)
        w = wg - inp.lr * g
    cu = sp(-yv * (Xv @ w)).mean()
    ref, = torch.autograd.grad(cu, [lam])
    got = oracle.hypergrad_itd(lo, up, up, 7)
    assert rel(got, ref.numpy()) < 1e-10
    assert rel(lo.params, w.detach().numpy()) < 1e-12
    # reweighted MLP (stop-gradient on the weight net's input), gelu
    from tests.test_oracle_derivatives import _tiny_reweight, _torch_mlp_logits
    from tests.oracle_build import reweight_levels
    inp = _tiny_reweight("gelu", seed=43)
    w_lv, th_lv = reweight_levels(inp, bf16=False)
    th = _t(inp.theta).requires_grad_(True)
    w = _t(inp.w).requires_grad_(True)
    for _ in range(3):
        c = _torch_reweight_cost(inp, w, th, None)
        g, = torch.autograd.grad(c, [w], create_graph=True)
        w = w - inp.lr * g
    zv = _torch_mlp_logits(inp.widths, "gelu", w, _t(inp.val.X))
    cu = torch.nn.functional.cross_entropy(zv, torch.from_numpy(inp.val.y.astype(np.int64)))
    ref, = torch.autograd.grad(cu, [th])
    got = oracle.hypergrad_itd(w_lv, th_lv, th_lv, 3)
    assert rel(got, ref.numpy()) < 1e-9


# ------------------------------------------------------------------ chain (Eq. 2)
def _dense_three_level(inp):
    """Hessians and mixed second derivatives of a tiny three-level program by autodiff."""
    w = _t(inp.w).requires_grad_(True)
    th = _t(inp.theta).requires_grad_(True)
    lam = _t(inp.lam).requires_grad_(True)

    class _B:
        widths, activation, train = inp.widths, inp.activation, inp.D1
    c1 = _torch_reweight_cost(_B, w, th, lam)
    g1, = torch.autograd.grad(c1, [w], create_graph=True)
    H1 = torch.stack([torch.autograd.grad(g1[j], [w], retain_graph=True)[0]
                      for j in range(w.numel())]).numpy()
    M1lam = torch.stack([torch.autograd.grad(g1[j], [lam], retain_graph=True)[0]
                         for j in range(w.numel())]).numpy()
    c2 = _torch_detect_cost(inp.widths, inp.activation, inp.D2, w, th, inp.mu)
    g2, = torch.autograd.grad(c2, [th], create_graph=True)
    H2 = torch.stack([torch.autograd.grad(g2[j], [th], retain_graph=True)[0]
                      for j in range(th.numel())]).numpy()
    M2w = torch.stack([torch.autograd.grad(g2[j], [w], retain_graph=True)[0]
                       for j in range(th.numel())]).numpy()
    c3 = _torch_detect_cost(inp.widths, inp.activation, inp.D3, w, th, 0.0)
    v_th, v_w = torch.autograd.grad(c3, [th, w])
    return H1, M1lam, H2, M2w, v_th.numpy(), v_w.numpy()


def test_three_level_chain_equals_product_of_materialised_jacobians():
    """Right-to-left evaluation along a path (Eq. 2) against the explicit matrix product.

    The weight-net level is made strongly convex (mu) so that its edge can use an exact
    solve, J2 = -H2^{-1} M2.  The classifier's Hessian is singular by construction (adding a
    constant to all output biases leaves the softmax unchanged), so its edge is compared with
    the materialised truncated Neumann inverse S1 = alpha * sum_j (I - alpha H1)^j in place of
    H1^{-1}."""
    inp = _tiny_three("gelu", widths=(5, 4, 3), B=10)
    inp.lam = np.log(np.array([0.5, 0.7])).astype(np.float32)
    inp.mu = 0.5
    P1, P2, P3 = three_levels(inp, bf16=False)
    H1, M1lam, H2, M2w, v_th, v_w = _dense_three_level(inp)
    assert np.linalg.eigvalsh(H2).min() > 0
    nm = dict(method="neumann", K=6, alpha=0.05)
    S1 = 0.05 * sum(np.linalg.matrix_power(np.eye(H1.shape[0]) - 0.05 * H1, j) for j in range(7))
    J1 = -S1 @ M1lam                           # ~ d w*/d lambda     [d_w, 2]
    J2 = -np.linalg.solve(H2, M2w)             # d theta*/d w*       [301, d_w]
    levels = [P1, P2, P3]
    exact = dict(method="cg", K=400, tol=1e-14)
    # path lambda -> w* -> theta*
    out_b = oracle.chain_levels(levels, [2, 0, 1], [nm, exact])
    assert rel(out_b, J1.T @ (J2.T @ v_th)) < 1e-8
    # path lambda -> w*
    out_a = oracle.chain_levels(levels, [2, 0], [nm])
    assert rel(out_a, J1.T @ v_w) < 1e-10
    # merging the two paths at the w* node is the same as summing them (linearity)
    u = v_w + oracle.chain_levels(levels, [0, 1], [exact], v_in=v_th)
    merged = oracle.chain_levels(levels, [2, 0], [nm], v_in=u)
    assert rel(merged, out_a + out_b) < 1e-9
    # both edges truncated
    nm2 = dict(method="neumann", K=3, alpha=0.01)
    T1 = 0.01 * sum(np.linalg.matrix_power(np.eye(H1.shape[0]) - 0.01 * H1, j) for j in range(4))
    T2 = 0.01 * sum(np.linalg.matrix_power(np.eye(H2.shape[0]) - 0.01 * H2, j) for j in range(4))
    out_nm = oracle.chain_levels(levels, [2, 0, 1], [nm2, nm2])
    assert rel(out_nm, (-T1 @ M1lam).T @ ((-T2 @ M2w).T @ v_th)) < 1e-9
    # a wrong order of the factors or a missing transpose would not even have this shape
    assert out_nm.shape == (2,)


# ------------------------------------------------------------------ optimiser variants
@pytest.mark.parametrize("kind", ["momentum", "adam"])
def test_optimizer_steps_match_torch_optim(kind):
    """lower_step with SGD-momentum / Adam against torch.optim on autodiff gradients of the same cost."""
    inp = si.logreg_bilevel(29, 40, 5, 10)
    inp.w0 = si.normal_f32(29, 9, (5,)) * 0.3
    inp.lam = (np.abs(si.normal_f32(29, 7, (5,))) * 0.1 + 0.02).astype(np.float32)
    lo, up = logreg_levels(inp)
    lo.optimizer, lo.lr, lo.weight_decay = kind, 0.05, 0.01
    lo.momentum = 0.9
    w = _t(inp.w0).requires_grad_(True)
    opt = (torch.optim.SGD([w], lr=0.05, momentum=0.9, weight_decay=0.01) if kind == "momentum"
           else torch.optim.Adam([w], lr=0.05, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01))
    X, y, lam = _t(inp.X), _t(inp.y), _t(inp.lam)
    for _ in range(6):
        opt.zero_grad()
        c = torch.nn.functional.softplus(-y * (X @ w)).mean() + 0.5 * (lam * w * w).sum()
        c.backward()
        opt.step()
    oracle.lower_step(lo, 6)
    assert rel(lo.params, w.detach().numpy()) < 1e-10


# ------------------------------------------------------------------ step-size schedules
@pytest.mark.parametrize("sched", ["multistep", "cosine"])
def test_scheduled_steps_match_torch_lr_schedulers(sched):
    """The step size as a function of the step count against torch.optim.lr_scheduler (MultiStepLR: decay
    by a factor at given iterations; CosineAnnealingLR down to a minimum at T_max), value by value and
    through a momentum-SGD trajectory on autodiff gradients of the same cost."""
    from oracle.solvers import lr_at
    inp = si.logreg_bilevel(31, 40, 5, 10)
    inp.w0 = si.normal_f32(31, 9, (5,)) * 0.3
    lo, up = logreg_levels(inp)
    lo.optimizer, lo.lr, lo.momentum, lo.weight_decay = "momentum", 0.1, 0.9, 0.01
    lo.lr_schedule = sched
    lo.lr_milestones, lo.lr_gamma, lo.lr_t_max, lo.lr_min = (3, 7), 0.1, 10, 0.004
    w = _t(inp.w0).requires_grad_(True)
    opt = torch.optim.SGD([w], lr=0.1, momentum=0.9, weight_decay=0.01)
    sch = (torch.optim.lr_scheduler.MultiStepLR(opt, milestones=[3, 7], gamma=0.1) if sched == "multistep"
           else torch.optim.lr_scheduler.CosineAnnealingLR(opt, T_max=10, eta_min=0.004))
    X, y, lam = _t(inp.X), _t(inp.y), _t(inp.lam)
    for t in range(10):
        assert abs(lr_at(lo, t) - opt.param_groups[0]["lr"]) < 1e-12 * 0.1 + 1e-15, t
        opt.zero_grad()
        c = torch.nn.functional.softplus(-y * (X @ w)).mean() + 0.5 * (lam * w * w).sum()
        c.backward()
        opt.step()
        sch.step()
    oracle.lower_step(lo, 10)
    assert rel(lo.params, w.detach().numpy()) < 1e-10
    # a second call continues on the schedule when the caller advances lr_step0
    lo.lr_step0 = 10
    assert abs(lr_at(lo, 0) - (0.1 * 0.01 if sched == "multistep" else 0.004)) < 1e-15
    # beyond T_max the cosine schedule stays at its minimum; a constant schedule ignores every field
    assert sched != "cosine" or lr_at(lo, 25) == 0.004
    lo.lr_schedule = "constant"
    assert lr_at(lo, 3) == 0.1


def test_itd_with_a_schedule_matches_autodiff_through_the_unrolled_steps():
    """ITD-RMAD with a different step size per unrolled step against reverse-mode autodiff (torch, fp64)
    through the same steps."""
    inp = si.logreg_bilevel(33, 30, 4, 12)
    inp.w0 = si.normal_f32(33, 9, (4,)) * 0.2
    inp.lam = (np.abs(si.normal_f32(33, 7, (4,))) * 0.1 + 0.05).astype(np.float32)
    lo, up = logreg_levels(inp)
    lamL = lo.constraints[0]
    lo.lr, lo.lr_schedule, lo.lr_milestones, lo.lr_gamma = 0.5, "multistep", (2, 4), 0.5
    X, y, Xv, yv = _t(inp.X), _t(inp.y), _t(inp.Xv), _t(inp.yv)
    lam = _t(inp.lam).requires_grad_(True)
    w = _t(inp.w0)
    for t in range(5):
        lr = 0.5 * 0.5 ** sum(1 for m in (2, 4) if t >= m)
        wd = w.detach().requires_grad_(True) if t == 0 else w
        c = torch.nn.functional.softplus(-y * (X @ wd)).mean() + 0.5 * (lam * wd * wd).sum()
        (g,) = torch.autograd.grad(c, wd, create_graph=True)
        w = wd - lr * g
    cu = torch.nn.functional.softplus(-yv * (Xv @ w)).mean()
    (ref,) = torch.autograd.grad(cu, lam)
    out = oracle.hypergrad_itd(lo, up, lamL, 5)
    assert rel(out, ref.numpy()) < 1e-9


# ------------------------------------------------------------------ gradient accumulation
def test_accumulated_step_gradient_equals_full_batch_and_torch_accumulation():
    """Averaging the gradients of equal micro-batches is the full-batch gradient of a mean cost; the step
    it drives equals PyTorch's accumulation idiom (backward of cost/A per micro-batch, one optimiser step)."""
    from oracle.solvers import step_gradient
    inp = si.logreg_bilevel(35, 48, 5, 10)
    inp.w0 = si.normal_f32(35, 9, (5,)) * 0.3
    lo, up = logreg_levels(inp)
    full = oracle.grad(lo, lo)
    lo.grad_accum = 4
    assert rel(step_gradient(lo), full) < 1e-13
    lam = lo.constraints[0].params
    # weight decay is part of every micro-batch's cost: counted once in the average, not A times
    assert rel(step_gradient(lo) - lam * lo.params, full - lam * lo.params) < 1e-12
    w = _t(inp.w0).requires_grad_(True)
    opt = torch.optim.SGD([w], lr=0.1, momentum=0.9)
    lo.optimizer, lo.momentum, lo.lr = "momentum", 0.9, 0.1
    X, y, lamt = _t(inp.X), _t(inp.y), _t(inp.lam)
    for _ in range(3):
        opt.zero_grad()
        for a in range(4):
            Xa, ya = X[a * 12:(a + 1) * 12], y[a * 12:(a + 1) * 12]
            c = torch.nn.functional.softplus(-ya * (Xa @ w)).mean() + 0.5 * (lamt * w * w).sum()
            (c / 4).backward()
        opt.step()
    oracle.lower_step(lo, 3)
    assert rel(lo.params, w.detach().numpy()) < 1e-10
    lo.grad_accum = 5
    with pytest.raises(ValueError):
        step_gradient(lo)
