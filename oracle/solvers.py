"""Unrolled lower steps, best-response-Jacobian x vector products and their chaining (fp64).

TEST INFRASTRUCTURE (see the package docstring).

The paper names the approximations (Sec. 3.2: AID with Neumann series, AID with conjugate
gradient, AID with finite difference) and refers to the original works for their steps; the
steps below are the textbook form of each, applied to the implicit-function-theorem
expression  (dx*/dc)^T v = -M^T H^{-1} v  evaluated at the current (unrolled, approximate)
lower parameters x (Sec. 3.2; Sec. 5.4 for the finite difference being taken at the unrolled
weights).  Readings where the paper is silent:
  * Neumann(K, alpha): K Hessian-vector products, terms j = 0..K, the sum scaled by alpha, so
    that it tends to H^{-1} v when the spectral radius of (I - alpha H) is below one.
  * CG(K, tol): zero start, no preconditioner, stops after K iterations, or when the residual
    norm has fallen to tol*|v|, or (status "breakdown") when a search direction has p^T H p <= 0.
  * FD(eps0, alpha): eps = eps0/|v|_2; result -alpha*[dC/dc(x+eps v) - dC/dc(x-eps v)]/(2 eps),
    i.e. H^{-1} replaced by alpha*I; alpha defaults to 1.  On mixed-precision levels the two
    perturbed evaluations are not re-quantised.  Under the plain reading (Level.quant = "weights")
    x +- eps v is the displaced fp64 master, used unrounded; under the bf16-operand reading
    (Level.quant = "operands") it displaces the bf16 compute copy, and the rounding offsets of
    the hidden activations stay at their base-point values.
"""
from __future__ import annotations

import copy

import numpy as np

from . import levels as _lv
from .levels import Level

grad = _lv.grad
hvp = _lv.hvp
mixed_vjp = _lv.mixed_vjp


def lr_at(L: Level, step_in_call: int) -> float:
    """Step size of the problem's step number t = lr_step0 + step_in_call (App. C: the classifiers' step
    size is "decayed by a factor of 10" at stated iterations, or follows "the cosine annealing schedule"
    down to a minimum at the end of training; the weight net's is constant)."""
    t = int(L.lr_step0) + int(step_in_call)
    if L.lr_schedule == "constant":
        return float(L.lr)
    if L.lr_schedule == "multistep":
        passed = sum(1 for m in L.lr_milestones if m > 0 and t >= m)
        return float(L.lr) * float(L.lr_gamma) ** passed
    if L.lr_schedule == "cosine":
        u = min(t, L.lr_t_max) / float(L.lr_t_max)
        return float(L.lr_min) + (float(L.lr) - float(L.lr_min)) * 0.5 * (1.0 + np.cos(np.pi * u))
    raise ValueError(L.lr_schedule)


def apply_optimizer(L: Level, g: np.ndarray, step_in_call: int = 0) -> None:
    """One step of the problem's optimiser along gradient g (App. C names SGD with momentum and weight
    decay for the classifiers and Adam for the weight net; the update rules are the standard ones),
    with the step size of the schedule at this step."""
    x = L.params
    lr = lr_at(L, step_in_call)
    if L.optimizer == "gd":
        L.params = x - lr * g
        return
    gg = g + L.weight_decay * x
    st = L.opt_state
    if L.optimizer == "momentum":
        st["buf"] = L.momentum * st.get("buf", np.zeros_like(x)) + gg
        L.params = x - lr * st["buf"]
    elif L.optimizer == "adam":
        st["t"] = st.get("t", 0) + 1
        st["m"] = L.beta1 * st.get("m", np.zeros_like(x)) + (1.0 - L.beta1) * gg
        st["v"] = L.beta2 * st.get("v", np.zeros_like(x)) + (1.0 - L.beta2) * gg * gg
        mhat = st["m"] / (1.0 - L.beta1 ** st["t"])
        vhat = st["v"] / (1.0 - L.beta2 ** st["t"])
        L.params = x - lr * mhat / (np.sqrt(vhat) + L.adam_eps)
    else:
        raise ValueError(L.optimizer)


def step_gradient(L: Level) -> np.ndarray:
    """Gradient that a step of a problem without lower problems follows.  With gradient accumulation (one
    of the systems features Sec. 4 lists) the batch is taken as L.grad_accum equal micro-batches, one
    after the other, and their gradients are averaged before the optimiser step."""
    A = int(L.grad_accum)
    if A <= 1:
        return grad(L, L)
    n = L.X.shape[0]
    if n % A:
        raise ValueError("batch size must be a multiple of grad_accum")
    nb = n // A
    total = 0.0
    for a in range(A):
        Ls = copy.copy(L)
        Ls.X, Ls.y = L.X[a * nb:(a + 1) * nb], L.y[a * nb:(a + 1) * nb]
        if L.aux is not None:
            Ls.aux = L.aux[a * nb:(a + 1) * nb]
        total = total + grad(Ls, Ls)
    return total / A


def lower_step(L: Level, n_steps: int) -> None:
    """x <- x - lr * dC/dx, n_steps times on the level's fixed batch (Sec. 3.2: w* is
    approximated by a small number of unrolled gradient steps).  Updates L.params in place.
    For mixed-precision levels the gradient is taken at the bf16-rounded copy of the
    current master, which is re-derived at every step."""
    for s in range(int(n_steps)):
        g = step_gradient(L)
        if L.loss_scale is not None and not _loss_scaled_step_is_taken(L):
            continue
        apply_optimizer(L, g, s)


FP16_OVERFLOW = 65520.0      # magnitudes from here up round to infinity in IEEE binary16


def _loss_scaled_step_is_taken(L: Level) -> bool:
    """Loss scaling of a half-precision level (Sec. 4 lists mixed precision; the paper's listings switch it on
    with an fp16 flag and leave the scaling rule to the framework; the rule here is the usual dynamic one).
    State L.loss_scale = [S, good, G, skipped].  The backward pass multiplies its top-layer deltas by S and the
    gradient is divided by S again, which changes nothing in exact arithmetic, so only the overflow decision
    is modelled: the step overflows when S times the largest 16-bit backward operand rounds to infinity.  Then
    the update is skipped, S halves, `good` returns to 0 and `skipped` counts up.  Otherwise the step is
    taken, `good` counts up and, when it reaches G > 0, S doubles and `good` returns to 0."""
    st = L.loss_scale
    if st[0] * _lv.largest_backward_operand(L) >= FP16_OVERFLOW:
        st[0] *= 0.5
        st[1] = 0
        st[3] += 1
        return False
    st[1] += 1
    if st[2] > 0 and st[1] >= st[2]:
        st[0] *= 2.0
        st[1] = 0
    return True


def neumann_solve(hv, v, K: int, alpha: float) -> np.ndarray:
    """q = alpha * sum_{j=0..K} (I - alpha H)^j v, built with K products hv(.) = H(.)."""
    t = np.array(v, dtype=np.float64)
    s = t.copy()
    for _ in range(int(K)):
        t = t - alpha * hv(t)
        s = s + t
    return alpha * s


def cg_solve(hv, v, K: int, tol: float = 0.0):
    """Conjugate gradient on H q = v.  Returns (q, iterations done, status) with status
    'ok' or 'breakdown'."""
    v = np.asarray(v, dtype=np.float64)
    q = np.zeros_like(v)
    r = v.copy()
    p = r.copy()
    rho = r @ r
    stop = (tol * tol) * (v @ v)
    it = 0
    for _ in range(int(K)):
        if rho <= stop:
            break
        h = hv(p)
        gamma = p @ h
        if gamma <= 0.0:
            return q, it, "breakdown"
        a = rho / gamma
        q = q + a * p
        r = r - a * h
        rho_new = r @ r
        p = r + (rho_new / rho) * p
        rho = rho_new
        it += 1
    return q, it, "ok"


def brj(L: Level, wrt: Level, v, method: str, K: int = 0, alpha: float = 1.0,
        eps0: float = 0.01, tol: float = 0.0, info: dict | None = None) -> np.ndarray:
    """(d x*/d c)^T v for the problem L (own parameters x) and its constraint `wrt` (c):
    the base operation of Sec. 3.2, by the chosen approximation."""
    v = np.asarray(v, dtype=np.float64)
    if method == "neumann":
        q = neumann_solve(lambda t: hvp(L, t), v, K, alpha)
        return -mixed_vjp(L, wrt, q)
    if method == "cg":
        q, it, status = cg_solve(lambda t: hvp(L, t), v, K, tol)
        if info is not None:
            info["iters"], info["status"] = it, status
        return -mixed_vjp(L, wrt, q)
    if method == "fd":
        nv = np.sqrt(v @ v)
        if nv == 0.0:
            return np.zeros(wrt.params.size)
        eps = eps0 / nv
        # "frozen" marks a perturbed evaluation that is not re-quantised (either reading of a
        # mixed-precision level); for full-precision levels it has no effect
        gp = grad(L, wrt, over={id(L): L.params + eps * v, "frozen": {id(L)}})
        gm = grad(L, wrt, over={id(L): L.params - eps * v, "frozen": {id(L)}})
        return -alpha * (gp - gm) / (2.0 * eps)
    raise ValueError(method)


def _hypergrad(lower, upper, wrt, **kw):
    """Eq. 1 for one lower problem: direct gradient + best-response Jacobian x direct gradient."""
    v = grad(upper, lower)
    return grad(upper, wrt) + brj(lower, wrt, v, **kw)


def hypergrad_neumann(lower: Level, upper: Level, wrt: Level, K: int, alpha: float):
    return _hypergrad(lower, upper, wrt, method="neumann", K=K, alpha=alpha)


def hypergrad_cg(lower: Level, upper: Level, wrt: Level, K: int, tol: float = 0.0,
                 info: dict | None = None):
    return _hypergrad(lower, upper, wrt, method="cg", K=K, tol=tol, info=info)


def hypergrad_fd(lower: Level, upper: Level, wrt: Level, eps0: float = 0.01, alpha: float = 1.0):
    return _hypergrad(lower, upper, wrt, method="fd", eps0=eps0, alpha=alpha)


def hypergrad_itd(lower: Level, upper: Level, wrt: Level, n_steps: int) -> np.ndarray:
    """Iterative differentiation with reverse-mode autodiff (ITD-RMAD, Sec. 3.2): take n_steps
    unrolled gradient steps x_{t+1} = x_t - lr * g(x_t, c) from the current lower parameters
    (which are left at x_T), then differentiate C_upper(x_T(c), c) through the stored steps:

        a <- dC_u/dx at x_T;   out <- dC_u/dc
        for t = T-1 .. 0:   out <- out - lr * M_t^T a ;   a <- a - lr * H_t a

    with H_t, M_t the second derivatives of the lower cost at x_t (same stop-gradient and
    quantisation conventions as `hvp` / `mixed_vjp`)."""
    if lower.optimizer != "gd":
        raise ValueError("ITD-RMAD differentiates plain gradient-descent steps")
    xs = []
    for t in range(int(n_steps)):
        xs.append(lower.params.copy())
        lower.params = lower.params - lr_at(lower, t) * grad(lower, lower)
    a = grad(upper, lower)
    out = grad(upper, wrt).copy()
    for t in reversed(range(len(xs))):
        over = {id(lower): xs[t]}
        lr_t = lr_at(lower, t)
        out = out - lr_t * mixed_vjp(lower, wrt, a, over)
        a = a - lr_t * hvp(lower, a, over)
    return out


def chain_levels(levels, path, cfgs, v_in=None) -> np.ndarray:
    """One path term of Eq. 2, evaluated right to left (Sec. 3.2).

    path = [k, q(1), ..., q(m)] are indices into `levels`: the result is with respect to the
    parameters of levels[k]; q(1) is reached from k by the upper-to-lower edge and q(i+1)
    from q(i) by lower-to-upper edges.  The start vector is v_in, or dC_k/d theta_{q(m)} when
    v_in is None.  cfgs[i] (a dict of `brj` keyword arguments) configures the edge into
    q(i+1), i.e. cfgs[0] is the upper-to-lower edge.  The direct gradient of Eq. 2 is not
    added."""
    k, q = path[0], list(path[1:])
    if not q:
        raise ValueError("path needs at least one edge")
    v = grad(levels[k], levels[q[-1]]) if v_in is None else np.asarray(v_in, dtype=np.float64)
    for i in range(len(q) - 1, 0, -1):
        v = brj(levels[q[i]], levels[q[i - 1]], v, **cfgs[i])
    return brj(levels[q[0]], levels[k], v, **cfgs[0])
