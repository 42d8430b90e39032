"""Pins for the oracle's half-precision (IEEE binary16) reading of a mixed-precision level and for its loss
scaling rule.  Expected values come from torch's own conversion, reverse-mode autodiff of a restated cost, and
torch.amp.GradScaler, never from the oracle's formulas."""
import numpy as np
import pytest
import torch

import oracle
from oracle import levels as olv
from oracle import solvers as osv
from oracle.bf16 import round_to_fp16
import synth_inputs as si
from tests.oracle_build import reweight_levels
from tests.test_oracle_derivatives import _t, _tiny_reweight, _torch_act, _torch_weightnet, rel


def _h(t):
    return t.to(torch.float32).to(torch.float16).to(torch.float64)


def test_fp16_rounding_matches_library_conversion_and_overflows_where_the_format_does():
    x = np.concatenate([si.normal_f32(3, 1, (4096,)) * np.float32(s) for s in (1e-6, 1e-3, 1.0, 300.0, 7e4)])
    np.testing.assert_array_equal(round_to_fp16(x), torch.from_numpy(x).half().double().numpy())
    assert round_to_fp16(np.array([65519.0]))[0] == 65504.0
    assert np.isinf(round_to_fp16(np.array([65520.0]))[0])
    assert osv.FP16_OVERFLOW == 65520.0
    assert round_to_fp16(np.array([2.0 ** -25]))[0] == 0.0 and round_to_fp16(np.array([2.0 ** -24]))[0] == 2.0 ** -24


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_fp16_level_rounds_matrices_and_hidden_activations_to_binary16(act):
    inp = _tiny_reweight(act, seed=43)
    inp.w = inp.w + si.normal_f32(43, 400, inp.w.shape) * 1e-3
    w16, th16 = reweight_levels(inp, bf16=True, operand_dtype="fp16")
    Ws, bs = olv.mlp_unpack(inp.widths, inp.w.astype(np.float64))
    h = _t(inp.train.X)
    for l, (W, b) in enumerate(zip(Ws, bs)):
        a = h @ _h(_t(W)).T + _t(b)
        h = _h(_torch_act(act, a)) if l < len(Ws) - 1 else a
    ell = torch.nn.functional.cross_entropy(h, torch.from_numpy(inp.train.y.astype(np.int64)), reduction="none")
    ref = (_torch_weightnet(_t(inp.theta), ell) * ell).mean().item()
    assert abs(olv.cost(w16) - ref) < 1e-13
    assert abs(olv.cost(reweight_levels(inp, bf16=True)[0]) - ref) > 1e-9       # not the bfloat16 reading


def test_largest_backward_operand_is_the_largest_derivative_with_respect_to_a_pre_activation():
    inp = _tiny_reweight("gelu", seed=47, widths=(7, 9, 8, 5), B=20)
    w_lv, th_lv = reweight_levels(inp, bf16=False)
    Ws, bs = olv.mlp_unpack(inp.widths, inp.w.astype(np.float64))
    h = _t(inp.train.X)
    pre = []
    for l, (W, b) in enumerate(zip(Ws, bs)):
        a = (h @ _t(W).T + _t(b)).requires_grad_(True)
        a.retain_grad()
        pre.append(a)
        h = _torch_act("gelu", a) if l < len(Ws) - 1 else a
    ell = torch.nn.functional.cross_entropy(h, torch.from_numpy(inp.train.y.astype(np.int64)), reduction="none")
    c = (_torch_weightnet(_t(inp.theta), ell.detach()) * ell).mean()
    c.backward()
    ref = max(float(a.grad.abs().max()) for a in pre)
    assert abs(olv.largest_backward_operand(w_lv) - ref) < 1e-14 * max(1.0, ref)


def test_loss_scaling_follows_the_library_rule_and_leaves_taken_steps_unchanged():
    """Start far above what binary16 can hold: the first steps overflow and are skipped while the scale halves;
    then steps are taken, and after every `G` of them the scale doubles (and may overflow again).  The same
    overflow pattern replayed through torch.amp.GradScaler gives the same scales; the parameters after the
    run equal plain gradient descent with as many steps as were taken."""
    inp = _tiny_reweight("relu", seed=53, widths=(7, 9, 5), B=16)
    w, th = reweight_levels(inp, bf16=True, operand_dtype="fp16")
    plain, _ = reweight_levels(inp, bf16=True, operand_dtype="fp16")
    dmax = olv.largest_backward_operand(w)
    S0 = 2.0 ** np.ceil(np.log2(65520.0 / dmax) + 2.2)          # overflows for the first three steps
    G = 2
    w.loss_scale = [S0, 0, G, 0]
    scales, taken = [], []
    for step in range(9):
        before = w.params.copy()
        # the overflow decision is the format's: S * dmax converted to binary16 is infinite
        expect_overflow = bool(torch.isinf(torch.tensor(w.loss_scale[0] * olv.largest_backward_operand(w)).half()))
        oracle.lower_step(w, 1)
        moved = not np.array_equal(before, w.params)
        assert moved == (not expect_overflow)
        taken.append(moved)
        scales.append(w.loss_scale[0])
    assert taken[:3] == [False, False, False] and taken[3] and sum(taken) >= 4
    assert w.loss_scale[3] == taken.count(False)
    # the library's rule on the same pattern
    p = torch.nn.Parameter(torch.zeros(2))
    opt = torch.optim.SGD([p], lr=0.1)
    sc = torch.amp.GradScaler("cpu", init_scale=S0, growth_factor=2.0, backoff_factor=0.5, growth_interval=G)
    ref_scales = []
    for ok in taken:
        opt.zero_grad()
        sc.scale(p.sum()).backward()
        if not ok:
            p.grad[0] = float("inf")
        sc.step(opt)
        sc.update()
        ref_scales.append(sc.get_scale())
    assert scales == ref_scales
    assert abs(p.data[0].item() + 0.1 * sum(taken)) < 1e-6       # the library skipped exactly the overflowing steps
    oracle.lower_step(plain, sum(taken))
    assert rel(w.params, plain.params) < 1e-15
