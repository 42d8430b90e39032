"""Cost functions of the optimisation problems and their derivatives, in fp64.

TEST INFRASTRUCTURE (see the package docstring).  A `Level` is one problem P_k of the
multilevel program of Sec. 2: its own parameters theta_k, its cost C_k, one batch of data
D_k and the list of problems whose parameters constrain it (U_k and L_k, Def. 1).

Notation (own parameters x, one constraining block c):
    g = dC/dx,  H = d2C/dx2,  M = d(g)/dc,  so that  (dx*/dc)^T v = -M^T H^{-1} v
by the implicit function theorem at a stationary point of C in x (the base operation of
Sec. 3.2).  Every function below is the hand-derived formula for one cost family; the tests
pin each of them to central finite differences of `cost`.

Cost families
-------------
logreg_wd        App. D.1 lower problem: mean logistic loss + 1/2 w^T diag(lambda) w
logreg           App. D.1 upper problem: mean logistic loss of the lower w on validation data
quadratic_wd     1/2 |A w - b|^2 + 1/2 w^T diag(lambda) w   (closed-form best response)
quadratic        1/2 |A w - b|^2 of a constraining w          (upper loss for the above)
mlp_ce_reweight  App. A "Classifier": mean_i r_i * CE_i with r_i = sigmoid(weightnet(CE_i
                 detached)), plus 1/2 sum_l exp(lambda_l) |W_l|^2 when a log-weight-decay
                 constraint is attached
                 With a label-correction constraint attached (App. A "Correcting & Reweighting" listing) the
                 per-sample loss is the cross-entropy against the corrected soft label, see cn_forward.
mlp_ce_correct   App. A "Correct": mean CE of a constraining classifier on this level's batch plus the
                 mean CE of the correction net's own soft labels (its linear + softmax part) on the same batch
mlp_ce           App. A "Reweight": plain mean cross-entropy of a constraining classifier
weightnet_detect mean_j (sigmoid(weightnet(CE_j(w))) - clean_j)^2 + mu/2 |theta|^2, where the
                 per-sample loss is NOT detached (w is a constraining parameter of this cost)
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np
from scipy.special import erf, expit

from .bf16 import round_to_bf16, round_to_fp16

WN_H = 100  # hidden width of the 1-100-1 weight net (App. C, "Meta-Weight-Network")


@dataclass(eq=False)
class Level:
    loss: str
    param_kind: str                    # 'vector' | 'mlp' | 'weightnet' | 'logwd' | 'correctnet'
    params: np.ndarray                 # flat fp64 (master copy)
    X: Optional[np.ndarray] = None
    y: Optional[np.ndarray] = None
    aux: Optional[np.ndarray] = None   # weightnet_detect: 1.0 where the given label is clean
    widths: Optional[tuple] = None     # MLP layer widths (in, hidden..., classes)
    activation: str = "relu"
    lr: float = 0.1
    mu: float = 0.0
    bf16: bool = False                 # MLP matrices are used through a bf16-rounded copy
    quant: str = "operands"            # what a bf16 level rounds: "operands" | "weights" (see _mlp_ce_state)
    operand_dtype: str = "bf16"        # 16-bit format of a mixed-precision level: "bf16" | "fp16"
    loss_scale: Optional[list] = None  # fp16 levels: [scale, good steps, growth interval, skipped steps] (solvers.lower_step)
    constraints: list = field(default_factory=list)
    optimizer: str = "gd"              # 'gd' | 'momentum' | 'adam' (App. C: SGD with momentum / Adam per problem)
    momentum: float = 0.0
    beta1: float = 0.9
    beta2: float = 0.999
    adam_eps: float = 1e-8
    weight_decay: float = 0.0
    opt_state: dict = field(default_factory=dict)
    lr_schedule: str = "constant"      # 'constant' | 'multistep' | 'cosine' (App. C: decay by 10 at given iterations / cosine annealing)
    lr_step0: int = 0                  # steps taken before the present call
    lr_milestones: tuple = ()
    lr_gamma: float = 0.1
    lr_t_max: int = 1
    lr_min: float = 0.0
    grad_accum: int = 1                # micro-batches whose gradients are averaged into one step (Sec. 4)

    def __post_init__(self):
        self.params = np.array(self.params, dtype=np.float64).reshape(-1)
        if self.X is not None:
            self.X = np.asarray(self.X, dtype=np.float64)
        if self.y is not None and np.issubdtype(np.asarray(self.y).dtype, np.floating):
            self.y = np.asarray(self.y, dtype=np.float64)
        if self.aux is not None:
            self.aux = np.asarray(self.aux, dtype=np.float64)


def _p(level: Level, over) -> np.ndarray:
    if over is not None and id(level) in over:
        return np.asarray(over[id(level)], dtype=np.float64)
    return level.params


def _find(L: Level, kind: str, required: bool = True) -> Optional[Level]:
    for c in [L] + list(L.constraints):
        if c.param_kind == kind:
            return c
    if required:
        raise ValueError(f"level with loss {L.loss} has no participant of kind {kind}")
    return None


def _find_constraint(L: Level, kind: str, required: bool = True) -> Optional[Level]:
    for c in L.constraints:
        if c.param_kind == kind:
            return c
    if required:
        raise ValueError(f"level with loss {L.loss} has no constraint of kind {kind}")
    return None


# ------------------------------------------------------------------ scalar functions
def softplus(t):
    return np.maximum(t, 0.0) + np.log1p(np.exp(-np.abs(t)))


def _act(name, a):
    if name == "relu":
        return np.maximum(a, 0.0)
    if name == "gelu":
        return a * 0.5 * (1.0 + erf(a / np.sqrt(2.0)))
    raise ValueError(name)


def _act_d1(name, a):
    if name == "relu":
        return (a > 0.0).astype(np.float64)          # relu'(0) = 0
    pdf = np.exp(-0.5 * a * a) / np.sqrt(2.0 * np.pi)
    return 0.5 * (1.0 + erf(a / np.sqrt(2.0))) + a * pdf


def _act_d2(name, a):
    if name == "relu":
        return np.zeros_like(a)
    pdf = np.exp(-0.5 * a * a) / np.sqrt(2.0 * np.pi)
    return pdf * (2.0 - a * a)


# ------------------------------------------------------------------ MLP pieces
def mlp_unpack(widths, flat):
    """Flat [W_1, b_1, W_2, b_2, ...] -> lists of W_l [out,in] and b_l [out]."""
    Ws, bs, o = [], [], 0
    for l in range(len(widths) - 1):
        fin, fout = widths[l], widths[l + 1]
        Ws.append(flat[o:o + fout * fin].reshape(fout, fin)); o += fout * fin
        bs.append(flat[o:o + fout]); o += fout
    assert o == flat.size, "parameter vector does not match the layer widths"
    return Ws, bs


def mlp_pack(Ws, bs):
    return np.concatenate([np.concatenate([W.reshape(-1), b.reshape(-1)]) for W, b in zip(Ws, bs)])


def _round16(level: Level):
    """Rounding to the level's 16-bit operand format."""
    if level.operand_dtype == "bf16":
        return round_to_bf16
    if level.operand_dtype == "fp16":
        return round_to_fp16
    raise ValueError(level.operand_dtype)


def _mlp_weights(level: Level, flat):
    """The copy of the parameters the cost is evaluated at: matrices rounded to the 16-bit operand
    format for mixed-precision levels, biases as they are."""
    Ws, bs = mlp_unpack(level.widths, flat)
    if level.bf16:
        rnd = _round16(level)
        Ws = [rnd(W) for W in Ws]
    return Ws, bs


def _mlp_forward(Ws, bs, X, act, quant=False, offsets=None, rnd=round_to_bf16):
    """h[l] is the input of layer l (h[0] = X), a[l] its pre-activation; logits = a[-1].

    Mixed-precision levels (quant=True) feed every matrix product bf16 operands, so each hidden
    activation is rounded to bf16 before it enters the next layer; the rounding offsets
    round(h) - h are returned.  With `offsets` given, those offsets are added instead of
    rounding again: a perturbed evaluation keeps the base point's quantisation offsets frozen,
    the same straight-through convention under which the derivatives are taken."""
    h, a, offs = [X], [], []
    for l, (W, b) in enumerate(zip(Ws, bs)):
        a.append(h[-1] @ W.T + b)
        if l < len(Ws) - 1:
            hn = _act(act, a[-1])
            if offsets is not None:
                hn = hn + offsets[l]
            elif quant:
                hq = rnd(hn)
                offs.append(hq - hn)
                hn = hq
            h.append(hn)
    return h, a, offs


def _softmax_ce(z, y):
    zs = z - z.max(axis=1, keepdims=True)
    logp = zs - np.log(np.exp(zs).sum(axis=1, keepdims=True))
    p = np.exp(logp)
    ell = -logp[np.arange(z.shape[0]), y]
    return p, ell


def _onehot(y, C):
    e = np.zeros((y.shape[0], C))
    e[np.arange(y.shape[0]), y] = 1.0
    return e


def _mlp_backward(Ws, h, a, delta_top, act, extra_dh_last=None):
    """Reverse sweep from delta_top = dC/d(logits).  Returns gW, gb and the per-layer
    delta_l = dC/da_l and dh_l = dC/dh_l (dh[l] pairs with a[l-1]).  extra_dh_last: a further
    dependence of the cost on the last hidden activation (the input of the top layer), added to its dh."""
    L = len(Ws)
    gW, gb, deltas, dhs = [None] * L, [None] * L, [None] * L, [None] * L
    delta = delta_top
    for l in range(L - 1, -1, -1):
        deltas[l] = delta
        gW[l] = delta.T @ h[l]
        gb[l] = delta.sum(axis=0)
        if l > 0:
            dhs[l] = delta @ Ws[l]
            if l == L - 1 and extra_dh_last is not None:
                dhs[l] = dhs[l] + extra_dh_last
            delta = dhs[l] * _act_d1(act, a[l - 1])
    return gW, gb, deltas, dhs


def _mlp_rforward(Ws, h, a, Us, cs, act):
    """Directional derivative of the forward pass along (U_l, c_l): Ra[l] = d a_l."""
    Rh = np.zeros_like(h[0])
    Rhs, Ras = [], []
    for l in range(len(Ws)):
        Rhs.append(Rh)
        Ra = Rh @ Ws[l].T + h[l] @ Us[l].T + cs[l]
        Ras.append(Ra)
        if l < len(Ws) - 1:
            Rh = _act_d1(act, a[l]) * Ra
    return Rhs, Ras


# ------------------------------------------------------------------ weight net 1-100-1
def wn_unpack(theta):
    H = WN_H
    return theta[0:H], theta[H:2 * H], theta[2 * H:3 * H], theta[3 * H]


def wn_forward(theta, ell):
    """s = a2 . relu(a1*ell + b1) + b2 ; r = sigmoid(s).  Returns r, s, hidden, mask."""
    a1, b1, a2, b2 = wn_unpack(theta)
    pre = ell[:, None] * a1[None, :] + b1[None, :]
    mask = (pre > 0.0).astype(np.float64)
    hid = pre * mask
    s = hid @ a2 + b2
    return expit(s), s, hid, mask


def wn_grad_s(theta, ell, hid, mask):
    """Per-sample d s / d theta, shape [B, 301]."""
    a1, b1, a2, b2 = wn_unpack(theta)
    ma2 = mask * a2[None, :]
    return np.concatenate([ma2 * ell[:, None], ma2, hid, np.ones((ell.shape[0], 1))], axis=1)


def wn_ds_dell(theta, mask):
    a1, b1, a2, b2 = wn_unpack(theta)
    return (mask * (a1 * a2)[None, :]).sum(axis=1)


# ------------------------------------------------------------------ label-correction net
# Sec. 5.1 / App. C "Correct Network": it "takes the penultimate activation from the classification network, and
# outputs soft labels through the linear layer and the softmax layer", and these are "interpolated with the
# original labels via the reweighting scheme which is achieved with 2-layer MLP".  Reading: with h the last
# hidden activation of the classifier (width H) and y the given label,
#     s   = softmax(A h + a0)                       soft label, A [C, H]
#     rho = sigmoid(a2 . relu(A1 h + b1) + b2)      interpolation weight; hidden width 100 like the weight net;
#                                                   the paper does not name the MLP's input: the same h
#     new = rho * onehot(y) + (1 - rho) * s
# alpha = [A, a0, A1, b1, a2, b2] flat, C*H + C + 100*H + 201 parameters.
def cn_size(H, C):
    return C * H + C + WN_H * H + 2 * WN_H + 1


def cn_unpack(alpha, H, C):
    o = 0
    A = alpha[o:o + C * H].reshape(C, H); o += C * H
    a0 = alpha[o:o + C]; o += C
    A1 = alpha[o:o + WN_H * H].reshape(WN_H, H); o += WN_H * H
    b1 = alpha[o:o + WN_H]; o += WN_H
    a2 = alpha[o:o + WN_H]; o += WN_H
    b2 = alpha[o]; o += 1
    assert o == alpha.size, "correction-net vector does not match the classifier's widths"
    return A, a0, A1, b1, a2, b2


def cn_forward(alpha, hlast, y, C):
    """Returns s, rho, new labels and the hidden pieces (mask, hid) for the backward formulas."""
    A, a0, A1, b1, a2, b2 = cn_unpack(alpha, hlast.shape[1], C)
    t = hlast @ A.T + a0
    ts = t - t.max(axis=1, keepdims=True)
    s = np.exp(ts) / np.exp(ts).sum(axis=1, keepdims=True)
    pre = hlast @ A1.T + b1
    mask = (pre > 0.0).astype(np.float64)
    hid = pre * mask
    rho = expit(hid @ a2 + b2)
    new = rho[:, None] * _onehot(y, C) + (1.0 - rho)[:, None] * s
    return s, rho, new, mask, hid


def _cn_sample_derivs(alpha, hlast, y, C, logp, s, rho, mask):
    """Per-sample derivatives of l_i = -sum_c new_c log p_c with respect to the correction net's two
    pre-activations: dt = dl/d(A h + a0) [B, C] and dpre = dl/d(A1 h + b1) [B, 100], plus dm = dl/dm [B]."""
    A, a0, A1, b1, a2, b2 = cn_unpack(alpha, hlast.shape[1], C)
    g = -(1.0 - rho)[:, None] * logp                                  # dl/ds
    dt = s * (g - (s * g).sum(axis=1, keepdims=True))                 # back through the softmax
    D = -logp[np.arange(y.shape[0]), y] + (s * logp).sum(axis=1)      # dl/drho = -<onehot - s, log p>
    dm = D * rho * (1.0 - rho)
    dpre = mask * a2[None, :] * dm[:, None]
    return dt, dpre, dm


def _cn_pack_grad(coef, dt, dpre, dm, hlast, hid):
    """sum_i coef_i * d l_i / d alpha from the per-sample pieces."""
    gt, gp = coef[:, None] * dt, coef[:, None] * dpre
    return np.concatenate([(gt.T @ hlast).reshape(-1), gt.sum(axis=0), (gp.T @ hlast).reshape(-1), gp.sum(axis=0),
                           ((coef * dm)[:, None] * hid).sum(axis=0), [np.sum(coef * dm)]])


def _log_softmax(z):
    zs = z - z.max(axis=1, keepdims=True)
    return zs - np.log(np.exp(zs).sum(axis=1, keepdims=True))


def _corrected(L: Level, over, h, a, y):
    """Soft-label loss pieces of a classifier cost with a correction net attached, else None."""
    G = _find_constraint(L, "correctnet", required=False) if L.loss == "mlp_ce_reweight" else None
    if G is None:
        return None
    if len(h) < 2:
        raise ValueError("label correction needs a hidden layer")
    al = _p(G, over)
    C = a[-1].shape[1]
    logp = _log_softmax(a[-1])
    s, rho, new, mask, hid = cn_forward(al, h[-1], y, C)
    ell = -(new * logp).sum(axis=1)
    return dict(level=G, alpha=al, logp=logp, s=s, rho=rho, new=new, mask=mask, hid=hid, ell=ell, hlast=h[-1])


# ------------------------------------------------------------------ per-family evaluation
def _logreg_parts(L, over):
    if L.loss == "logreg_wd":
        w = _p(L, over)
        lam = _p(_find_constraint(L, "vector"), over)
    else:
        w = _p(_find_constraint(L, "vector"), over)
        lam = None
    return w, lam


def _mlp_ce_state(L: Level, over):
    """Forward pass of the classifier that takes part in cost L and the per-sample CE.

    A mixed-precision classifier (Sec. 4 lists mixed precision among the systems features; the
    paper does not say what is rounded) is evaluated under one of two stated readings:

    quant = "weights"   the plain reading.  The matrices are rounded to bf16 once per evaluation
                        of the cost; nothing else is rounded.  A finite-difference evaluation
                        (Sec. 3.2, AID-FD) displaces the fp64 master copy, x +- eps v, and uses
                        it as it is, with no rounding at all.
    quant = "operands"  every matrix product takes bf16 operands: the matrices and each hidden
                        activation are rounded.  A finite-difference evaluation displaces the
                        rounded matrices and keeps the base pass's rounding offsets of the hidden
                        activations (rounding is treated as the identity under differentiation).

    over["frozen"] (a set of level ids) marks the classifier's override as such a perturbed
    evaluation."""
    M = _find(L, "mlp")
    flat = _p(M, over)
    frozen = over is not None and id(M) in over.get("frozen", ())
    if M.bf16 and M.quant not in ("operands", "weights"):
        raise ValueError(M.quant)
    plain = M.bf16 and M.quant == "weights"
    if frozen and plain:
        Ws, bs = mlp_unpack(M.widths, flat)
        h, a, _ = _mlp_forward(Ws, bs, L.X, M.activation)
    elif frozen and M.bf16:
        Wb, bb = _mlp_weights(M, M.params)
        _, _, offs = _mlp_forward(Wb, bb, L.X, M.activation, quant=True, rnd=_round16(M))
        Wd, bd = mlp_unpack(M.widths, flat - M.params)
        Ws = [W0 + dW for W0, dW in zip(Wb, Wd)]
        bs = [b0 + db for b0, db in zip(bb, bd)]
        h, a, _ = _mlp_forward(Ws, bs, L.X, M.activation, offsets=offs)
    else:
        Ws, bs = _mlp_weights(M, flat)
        h, a, _ = _mlp_forward(Ws, bs, L.X, M.activation, quant=M.bf16 and not plain, rnd=_round16(M))
    p, ell = _softmax_ce(a[-1], np.asarray(L.y, dtype=np.int64))
    return M, Ws, bs, h, a, p, ell


def _reweight_r(L: Level, ell, over):
    T = _find_constraint(L, "weightnet", required=False)
    if T is None:
        return np.ones_like(ell), None
    r, s, hid, mask = wn_forward(_p(T, over), ell)
    return r, (T, s, hid, mask)


def _kappas(L: Level, over, nl):
    lamL = _find_constraint(L, "logwd", required=False)
    if lamL is None:
        return np.zeros(nl), None
    return np.exp(_p(lamL, over)), lamL


def cost(L: Level, over=None, r_fixed=None, ell_fixed=None) -> float:
    """C_k evaluated at the current (or overridden) parameters of all participants.

    mlp_ce_reweight carries a stop-gradient (the weight net sees the detached per-sample
    loss): `r_fixed` freezes the weights r_i (the function whose w-derivatives `grad`/`hvp`
    return) and `ell_fixed` freezes the per-sample losses (the function whose
    theta-derivative `grad` returns)."""
    if L.loss in ("logreg_wd", "logreg"):
        w, lam = _logreg_parts(L, over)
        c = softplus(-L.y * (L.X @ w)).mean()
        if lam is not None:
            c += 0.5 * np.sum(lam * w * w)
        return float(c)
    if L.loss in ("quadratic_wd", "quadratic"):
        if L.loss == "quadratic_wd":
            w, lam = _p(L, over), _p(_find_constraint(L, "vector"), over)
        else:
            w, lam = _p(_find_constraint(L, "vector"), over), None
        rres = L.X @ w - L.y
        c = 0.5 * rres @ rres
        if lam is not None:
            c += 0.5 * np.sum(lam * w * w)
        return float(c)
    if L.loss == "mlp_ce":
        _, _, _, _, _, _, ell = _mlp_ce_state(L, over)
        return float(ell.mean())
    if L.loss == "mlp_ce_correct":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        y = np.asarray(L.y, dtype=np.int64)
        s, _, _, _, _ = cn_forward(_p(_find(L, "correctnet"), over), h[-1], y, a[-1].shape[1])
        return float(ell.mean() - np.log(s[np.arange(y.shape[0]), y]).mean())
    if L.loss == "mlp_ce_reweight":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        cn = _corrected(L, over, h, a, np.asarray(L.y, dtype=np.int64))
        if cn is not None:
            ell = cn["ell"]
        if ell_fixed is not None:
            ell = np.asarray(ell_fixed, dtype=np.float64)
        r = _reweight_r(L, ell, over)[0] if r_fixed is None else np.asarray(r_fixed)
        kap, _ = _kappas(L, over, len(Ws))
        return float((r * ell).mean() + 0.5 * sum(k * np.sum(W * W) for k, W in zip(kap, Ws)))
    if L.loss == "weightnet_detect":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        T = _find(L, "weightnet")
        th = _p(T, over)
        r, _, _, _ = wn_forward(th, ell)
        return float(((r - L.aux) ** 2).mean() + 0.5 * L.mu * th @ th)
    raise ValueError(L.loss)


def grad(L: Level, wrt: Level, over=None) -> np.ndarray:
    """dC_L / d(params of `wrt`), `wrt` being L itself or one of its constraints.

    For mlp_ce_reweight the stop-gradient of the App. A listing applies: the derivative with
    respect to the classifier treats r_i as constants, the derivative with respect to the
    weight net treats the per-sample losses as data."""
    n_out = _p(wrt, over).size
    if L.loss in ("logreg_wd", "logreg"):
        w, lam = _logreg_parts(L, over)
        own_w = L if L.loss == "logreg_wd" else _find_constraint(L, "vector")
        if wrt is own_w:
            z = L.X @ w
            g = -(L.X.T @ (L.y * expit(-L.y * z))) / L.X.shape[0]
            return g + lam * w if lam is not None else g
        if L.loss == "logreg_wd" and wrt is _find_constraint(L, "vector"):
            return 0.5 * w * w
        return np.zeros(n_out)
    if L.loss in ("quadratic_wd", "quadratic"):
        own_w = L if L.loss == "quadratic_wd" else _find_constraint(L, "vector")
        w = _p(own_w, over)
        if wrt is own_w:
            g = L.X.T @ (L.X @ w - L.y)
            return g + _p(_find_constraint(L, "vector"), over) * w if L.loss == "quadratic_wd" else g
        if L.loss == "quadratic_wd" and wrt is _find_constraint(L, "vector"):
            return 0.5 * w * w
        return np.zeros(n_out)
    if L.loss == "mlp_ce":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        if wrt is not M:
            return np.zeros(n_out)
        B = L.X.shape[0]
        delta = (p - _onehot(np.asarray(L.y, np.int64), p.shape[1])) / B
        gW, gb, _, _ = _mlp_backward(Ws, h, a, delta, M.activation)
        return mlp_pack(gW, gb)
    if L.loss == "mlp_ce_correct":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        G = _find(L, "correctnet")
        al = _p(G, over)
        y = np.asarray(L.y, dtype=np.int64)
        B, C = L.X.shape[0], p.shape[1]
        s, _, _, _, _ = cn_forward(al, h[-1], y, C)
        dt = (s - _onehot(y, C)) / B                                  # d(mean CE of the soft label)/d(A h + a0)
        if wrt is G:
            out = np.zeros(al.size)
            H = h[-1].shape[1]
            out[:C * H] = (dt.T @ h[-1]).reshape(-1)
            out[C * H:C * H + C] = dt.sum(axis=0)
            return out
        if wrt is M:
            A = cn_unpack(al, h[-1].shape[1], C)[0]
            delta = (p - _onehot(y, C)) / B
            gW, gb, _, _ = _mlp_backward(Ws, h, a, delta, M.activation, extra_dh_last=dt @ A)
            return mlp_pack(gW, gb)
        return np.zeros(n_out)
    if L.loss == "mlp_ce_reweight":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        B = L.X.shape[0]
        y = np.asarray(L.y, np.int64)
        cn = _corrected(L, over, h, a, y)
        if cn is not None:
            ell = cn["ell"]
        r, wn = _reweight_r(L, ell, over)
        kap, lamL = _kappas(L, over, len(Ws))
        if cn is not None and (wrt is L or wrt is cn["level"]):
            dt, dpre, dm = _cn_sample_derivs(cn["alpha"], cn["hlast"], y, p.shape[1], cn["logp"], cn["s"], cn["rho"], cn["mask"])
            if wrt is cn["level"]:
                return _cn_pack_grad(r / B, dt, dpre, dm, cn["hlast"], cn["hid"])
            A, _, A1, _, _, _ = cn_unpack(cn["alpha"], cn["hlast"].shape[1], p.shape[1])
            delta = (r / B)[:, None] * (p - cn["new"])               # the soft label sums to one
            extra = (r / B)[:, None] * (dt @ A + dpre @ A1)          # the label itself moves with h (not detached)
            gW, gb, _, _ = _mlp_backward(Ws, h, a, delta, M.activation, extra_dh_last=extra)
            gW = [g + k * W for g, k, W in zip(gW, kap, Ws)]
            return mlp_pack(gW, gb)
        if wrt is L:
            delta = (r / B)[:, None] * (p - _onehot(np.asarray(L.y, np.int64), p.shape[1]))
            gW, gb, _, _ = _mlp_backward(Ws, h, a, delta, M.activation)
            gW = [g + k * W for g, k, W in zip(gW, kap, Ws)]
            return mlp_pack(gW, gb)
        if wn is not None and wrt is wn[0]:
            T, s, hid, mask = wn
            J = wn_grad_s(_p(T, over), ell, hid, mask)
            return ((r * (1.0 - r) * ell)[:, None] * J).sum(axis=0) / B
        if lamL is not None and wrt is lamL:
            return np.array([0.5 * k * np.sum(W * W) for k, W in zip(kap, Ws)])
        return np.zeros(n_out)
    if L.loss == "weightnet_detect":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        T = _find(L, "weightnet")
        th = _p(T, over)
        B = L.X.shape[0]
        r, s, hid, mask = wn_forward(th, ell)
        fp = 2.0 * (r - L.aux) * r * (1.0 - r)          # d/ds (sigmoid(s) - c)^2
        if wrt is T:
            return (fp[:, None] * wn_grad_s(th, ell, hid, mask)).sum(axis=0) / B + L.mu * th
        if wrt is M:
            kappa = fp * wn_ds_dell(th, mask) / B              # dC/d ell_j
            delta = kappa[:, None] * (p - _onehot(np.asarray(L.y, np.int64), p.shape[1]))
            gW, gb, _, _ = _mlp_backward(Ws, h, a, delta, M.activation)
            return mlp_pack(gW, gb)
        return np.zeros(n_out)
    raise ValueError(L.loss)


def largest_backward_operand(L: Level, over=None) -> float:
    """max over layers and entries of |delta_l| = |dC_L/da_l| in the gradient of the reweighted cross-entropy
    with respect to its own classifier: the quantities a mixed-precision backward pass holds in 16 bits.
    With fp16 operands and loss scale S, a step overflows when S times this reaches the format's range."""
    if L.loss != "mlp_ce_reweight":
        raise ValueError("loss scaling is defined for the classifier's own reweighted cross-entropy")
    M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
    B = L.X.shape[0]
    r, _ = _reweight_r(L, ell, over)
    delta_top = (r / B)[:, None] * (p - _onehot(np.asarray(L.y, np.int64), p.shape[1]))
    _, _, deltas, _ = _mlp_backward(Ws, h, a, delta_top, M.activation)
    return float(max(np.max(np.abs(d)) for d in deltas))


def hvp(L: Level, u: np.ndarray, over=None) -> np.ndarray:
    """H u with H = d2 C_L / d(own params)^2."""
    u = np.asarray(u, dtype=np.float64)
    if L.loss == "logreg_wd":
        w, lam = _logreg_parts(L, over)
        z = L.X @ w
        return L.X.T @ (expit(z) * expit(-z) * (L.X @ u)) / L.X.shape[0] + lam * u
    if L.loss == "quadratic_wd":
        lam = _p(_find_constraint(L, "vector"), over)
        return L.X.T @ (L.X @ u) + lam * u
    if L.loss == "mlp_ce_reweight":
        if _find_constraint(L, "correctnet", required=False) is not None:
            raise ValueError("second derivatives are not offered with label correction (the paper pairs it with AID-FD)")
        # R-operator (forward-over-reverse) through the classifier, r_i held constant.
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        act = M.activation
        B = L.X.shape[0]
        r, _ = _reweight_r(L, ell, over)
        kap, _ = _kappas(L, over, len(Ws))
        Us, cs = mlp_unpack(M.widths, u)
        delta_top = (r / B)[:, None] * (p - _onehot(np.asarray(L.y, np.int64), p.shape[1]))
        _, _, deltas, dhs = _mlp_backward(Ws, h, a, delta_top, act)
        Rhs, Ras = _mlp_rforward(Ws, h, a, Us, cs, act)
        Rdelta = (r / B)[:, None] * (p * Ras[-1] - p * (p * Ras[-1]).sum(axis=1, keepdims=True))
        nl = len(Ws)
        RgW, Rgb = [None] * nl, [None] * nl
        for l in range(nl - 1, -1, -1):
            RgW[l] = Rdelta.T @ h[l] + deltas[l].T @ Rhs[l] + kap[l] * Us[l]
            Rgb[l] = Rdelta.sum(axis=0)
            if l > 0:
                Rdh = Rdelta @ Ws[l] + deltas[l] @ Us[l]
                Rdelta = (Rdh * _act_d1(act, a[l - 1])
                          + dhs[l] * _act_d2(act, a[l - 1]) * Ras[l - 1])
        return mlp_pack(RgW, Rgb)
    if L.loss == "weightnet_detect" and L.param_kind == "weightnet":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        th = _p(L, over)
        a1, b1, a2, b2 = wn_unpack(th)
        ua1, ub1, ua2, ub2 = wn_unpack(u)
        B = L.X.shape[0]
        r, s, hid, mask = wn_forward(th, ell)
        c = L.aux
        rp = r * (1.0 - r)
        fp = 2.0 * (r - c) * rp
        fpp = 2.0 * rp * rp + 2.0 * (r - c) * rp * (1.0 - 2.0 * r)
        J = wn_grad_s(th, ell, hid, mask)                     # [B,301]
        Ju = J @ u
        # second derivative of s: only the (a2_k, a1_k) and (a2_k, b1_k) pairs are non-zero
        S2u = np.concatenate([
            mask * ua2[None, :] * ell[:, None],
            mask * ua2[None, :],
            mask * (ell[:, None] * ua1[None, :] + ub1[None, :]),
            np.zeros((B, 1))], axis=1)
        return ((fpp * Ju)[:, None] * J + fp[:, None] * S2u).sum(axis=0) / B + L.mu * u
    raise ValueError(f"no Hessian-vector product for loss {L.loss} / {L.param_kind}")


def mixed_vjp(L: Level, wrt: Level, q: np.ndarray, over=None) -> np.ndarray:
    """M^T q = d/dc < dC_L/dx , q > with q held fixed, c = params of the constraint `wrt`."""
    q = np.asarray(q, dtype=np.float64)
    if L.loss in ("logreg_wd", "quadratic_wd"):
        if wrt is _find_constraint(L, "vector"):
            return _p(L, over) * q
        raise ValueError("unknown constraint")
    if L.loss == "mlp_ce_reweight":
        if _find_constraint(L, "correctnet", required=False) is not None:
            raise ValueError("second derivatives are not offered with label correction (the paper pairs it with AID-FD)")
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        B = L.X.shape[0]
        r, wn = _reweight_r(L, ell, over)
        kap, lamL = _kappas(L, over, len(Ws))
        Qs, qc = mlp_unpack(M.widths, q)
        if wn is not None and wrt is wn[0]:
            T, s, hid, mask = wn
            _, Ras = _mlp_rforward(Ws, h, a, Qs, qc, M.activation)
            d = ((p - _onehot(np.asarray(L.y, np.int64), p.shape[1])) * Ras[-1]).sum(axis=1)
            J = wn_grad_s(_p(T, over), ell, hid, mask)
            return ((d * r * (1.0 - r))[:, None] * J).sum(axis=0) / B
        if lamL is not None and wrt is lamL:
            return np.array([k * np.sum(W * Q) for k, W, Q in zip(kap, Ws, Qs)])
        raise ValueError("unknown constraint")
    if L.loss == "weightnet_detect" and L.param_kind == "weightnet":
        M, Ws, bs, h, a, p, ell = _mlp_ce_state(L, over)
        if wrt is not M:
            raise ValueError("unknown constraint")
        th = _p(L, over)
        a1, b1, a2, b2 = wn_unpack(th)
        qa1, qb1, qa2, qb2 = wn_unpack(q)
        B = L.X.shape[0]
        r, s, hid, mask = wn_forward(th, ell)
        c = L.aux
        rp = r * (1.0 - r)
        fp = 2.0 * (r - c) * rp
        fpp = 2.0 * rp * rp + 2.0 * (r - c) * rp * (1.0 - 2.0 * r)
        Jq = wn_grad_s(th, ell, hid, mask) @ q
        dJq_dell = (mask * (a2 * qa1 + a1 * qa2)[None, :]).sum(axis=1)
        kappa = (fpp * wn_ds_dell(th, mask) * Jq + fp * dJq_dell) / B
        delta = kappa[:, None] * (p - _onehot(np.asarray(L.y, np.int64), p.shape[1]))
        gW, gb, _, _ = _mlp_backward(Ws, h, a, delta, M.activation)
        return mlp_pack(gW, gb)
    raise ValueError(f"no mixed second derivative for loss {L.loss}")
