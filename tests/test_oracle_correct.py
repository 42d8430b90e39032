"""Pins for the oracle's label-correction costs (the extended bilevel program of Sec. 5.1 and its App. A
listing): every expected value is reverse-mode autodiff of a forward-only restatement in torch, or a finite
difference of the oracle's cost."""
import numpy as np
import pytest
import torch

import oracle
from oracle import levels as olv
import synth_inputs as si
from tests.oracle_build import correct_reweight_levels
from tests.test_oracle_derivatives import _t, _torch_act, _torch_weightnet, central_fd, rel

HD = si.WEIGHTNET_HIDDEN


def _tiny(act, seed=61, widths=(7, 6, 5, 4), B=12):
    inp = si.correct_reweight(seed, widths, B, 0.4, activation=act)
    inp.w = inp.w + si.normal_f32(seed, 300, inp.w.shape) * 0.05
    inp.theta = si.weightnet_init(seed, 200) * 3.0
    inp.alpha = inp.alpha + si.normal_f32(seed, 310, inp.alpha.shape) * 0.3      # lively biases and mixing weights
    return inp


def _torch_forward(widths, act, flat, X):
    """logits and the last hidden activation"""
    h, o = X, 0
    L = len(widths) - 1
    hlast = None
    for l in range(L):
        fin, fout = widths[l], widths[l + 1]
        W = flat[o:o + fout * fin].reshape(fout, fin); o += fout * fin
        b = flat[o:o + fout]; o += fout
        if l == L - 1:
            hlast = h
        h = torch.nn.functional.linear(h, W, b)
        if l < L - 1:
            h = _torch_act(act, h)
    return h, hlast


def _torch_correct(alpha, hlast, y, C):
    H = hlast.shape[1]
    o = 0
    A = alpha[o:o + C * H].reshape(C, H); o += C * H
    a0 = alpha[o:o + C]; o += C
    A1 = alpha[o:o + HD * H].reshape(HD, H); o += HD * H
    b1 = alpha[o:o + HD]; o += HD
    a2 = alpha[o:o + HD]; o += HD
    b2 = alpha[o]
    s = torch.softmax(hlast @ A.T + a0, dim=1)
    rho = torch.sigmoid(torch.relu(hlast @ A1.T + b1) @ a2 + b2)
    onehot = torch.nn.functional.one_hot(y, C).to(torch.float64)
    return rho[:, None] * onehot + (1 - rho)[:, None] * s, hlast @ A.T + a0


def _classifier_cost(inp, w, th, al):
    """mean_i weight_i * (-sum_c new_ic log p_ic), the reweighting net fed the detached loss"""
    y = torch.from_numpy(inp.train.y.astype(np.int64))
    z, hlast = _torch_forward(inp.widths, inp.activation, w, _t(inp.train.X))
    new, _ = _torch_correct(al, hlast, y, inp.widths[-1])
    ell = -(new * torch.log_softmax(z, dim=1)).sum(dim=1)
    return (_torch_weightnet(th, ell.detach()) * ell).mean()


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_corrected_and_reweighted_classifier_cost_and_gradients_against_autograd(act):
    inp = _tiny(act)
    w_lv, th_lv, al_lv = correct_reweight_levels(inp, bf16=False)
    w = _t(inp.w).requires_grad_(True)
    th = _t(inp.theta).requires_grad_(True)
    al = _t(inp.alpha).requires_grad_(True)
    c = _classifier_cost(inp, w, th, al)
    assert abs(c.item() - olv.cost(w_lv)) < 1e-13
    gw, gth, gal = torch.autograd.grad(c, [w, th, al])
    assert rel(oracle.grad(w_lv, w_lv), gw.numpy()) < 1e-12          # includes the label's own dependence on h
    assert rel(oracle.grad(w_lv, al_lv), gal.numpy()) < 1e-12
    assert rel(oracle.grad(w_lv, th_lv), gth.numpy()) < 1e-12        # per-sample losses as data
    # the parameter count and the layout: a wrong slice would have failed above; the size is the stated one
    assert inp.alpha.size == si.correctnet_size(inp.widths[-2], inp.widths[-1]) == olv.cn_size(inp.widths[-2], inp.widths[-1])
    with pytest.raises(ValueError):
        oracle.hvp(w_lv, np.ones(inp.w.size))


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_correction_problem_cost_and_gradients_against_autograd(act):
    inp = _tiny(act, seed=63)
    w_lv, th_lv, al_lv = correct_reweight_levels(inp, bf16=False)
    w = _t(inp.w).requires_grad_(True)
    al = _t(inp.alpha).requires_grad_(True)
    y = torch.from_numpy(inp.val.y.astype(np.int64))
    z, hlast = _torch_forward(inp.widths, act, w, _t(inp.val.X))
    _, t = _torch_correct(al, hlast, y, inp.widths[-1])
    c = torch.nn.functional.cross_entropy(z, y) + torch.nn.functional.cross_entropy(t, y)
    assert abs(c.item() - olv.cost(al_lv)) < 1e-13
    gw, gal = torch.autograd.grad(c, [w, al])
    assert rel(oracle.grad(al_lv, w_lv), gw.numpy()) < 1e-12
    assert rel(oracle.grad(al_lv, al_lv), gal.numpy()) < 1e-12
    # the interpolation net takes no part in this cost
    H, C = inp.widths[-2], inp.widths[-1]
    assert np.all(oracle.grad(al_lv, al_lv)[C * H + C:] == 0.0)


def test_correction_gradients_by_finite_differences_and_the_finite_difference_hypergradient():
    inp = _tiny("gelu", seed=65, widths=(5, 4, 3), B=9)
    w_lv, th_lv, al_lv = correct_reweight_levels(inp, bf16=False)
    r = olv.wn_forward(th_lv.params, -np.ones(9))[0]      # any fixed weights: frozen for the w-derivative
    M, Ws, bs, h, a, p, ell = olv._mlp_ce_state(w_lv, None)
    cn = olv._corrected(w_lv, None, h, a, np.asarray(w_lv.y, np.int64))
    r = olv.wn_forward(th_lv.params, cn["ell"])[0]
    g_fd = central_fd(lambda x: olv.cost(w_lv, {id(w_lv): x}, r_fixed=r), w_lv.params.copy())
    assert rel(oracle.grad(w_lv, w_lv), g_fd) < 1e-7
    ga_fd = central_fd(lambda x: olv.cost(w_lv, {id(al_lv): x}, r_fixed=r), al_lv.params.copy())
    assert rel(oracle.grad(w_lv, al_lv), ga_fd) < 1e-7
    # Eq. 1 with the finite-difference Jacobian: direct gradient of the correction cost in alpha plus
    # -alpha_fd [grad_alpha C_lower(w + eps v) - grad_alpha C_lower(w - eps v)] / (2 eps), v = dC_corr/dw
    v = oracle.grad(al_lv, w_lv)
    eps = 0.01 / np.linalg.norm(v)
    gp = oracle.grad(w_lv, al_lv, {id(w_lv): w_lv.params + eps * v})
    gm = oracle.grad(w_lv, al_lv, {id(w_lv): w_lv.params - eps * v})
    ref = oracle.grad(al_lv, al_lv) - (gp - gm) / (2 * eps)
    assert rel(oracle.hypergrad_fd(w_lv, al_lv, al_lv, 0.01, 1.0), ref) < 1e-12
