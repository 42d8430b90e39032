"""The half-precision (IEEE binary16) operand variant of the MLP families and the loss scaling of its lower
steps, through the C ABI, against the fp64 oracle under the same reading (matrices and hidden activations
rounded to binary16).  Tolerance as for the bf16 paths: relative L2 error <= 2e-2; the loss-scaling state
(scale, counters) is integer / power-of-two work and must match exactly."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from oracle import levels as olv
from tests import oracle_build as ob

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _inputs(seed, widths, B, act):
    from tests.test_gpu_mlp import _perturb
    inp = _perturb(si.reweight_bilevel(seed, widths, B, 0.4, activation=act), seed)
    for b in (inp.train, inp.val):          # batches exactly representable in binary16 on both sides
        b.X = torch.from_numpy(np.ascontiguousarray(b.X, dtype=np.float32)).half().float().numpy()
    return inp


def _levels(inp):
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    w, th = cb.reweight_levels(inp, operand_dtype=torch.float16)
    ow, oth = ob.reweight_levels(inp, operand_dtype="fp16")
    return bt, cb, w, th, ow, oth


def _update_err(cb, w, ow, start):
    x0 = np.asarray(start, dtype=np.float64)
    return cb.rel_l2(w.params.double().cpu().numpy() - x0, ow.params - x0)


@pytest.mark.parametrize("act,widths,B", [("relu", (64, 96, 10), 128), ("gelu", (64, 96, 10), 128),
                                          ("gelu", (40, 130, 66, 12), 200)])
def test_fp16_primitives_and_hypergradients_match_oracle(act, widths, B, parity_record):
    inp = _inputs(101, widths, B, act)
    bt, cb, w, th, ow, oth = _levels(inp)
    ws = bt.Workspace([w, th])
    P = inp.w.size
    out = torch.empty(P, device="cuda")
    outt = torch.empty(si.WEIGHTNET_PARAMS, device="cuda")
    bt.betty_grad(w, w, out, ws)
    assert cb.rel_l2(out, oracle.grad(ow, ow)) < TOL
    bt.betty_grad(th, w, out, ws)
    g_up = oracle.grad(oth, ow)
    assert cb.rel_l2(out, g_up) < TOL
    bt.betty_hvp(w, cb.dev(g_up.astype(np.float32)), out, ws)
    assert cb.rel_l2(out, oracle.hvp(ow, g_up.astype(np.float32))) < TOL
    bt.betty_lower_step(w, 2, ws)                       # fused gradient steps
    oracle.lower_step(ow, 2)
    assert parity_record(f"fp16/{act}-B{B}/lower_update", _update_err(cb, w, ow, inp.w)) < TOL
    bt.betty_hypergrad_neumann(w, th, th, 3, 0.01, outt, ws)
    assert parity_record(f"fp16/{act}-B{B}/neumann", cb.rel_l2(outt, oracle.hypergrad_neumann(ow, oth, oth, 3, 0.01))) < TOL
    bt.betty_hypergrad_fd(w, th, th, 0.01, 1.0, outt, ws)
    assert parity_record(f"fp16/{act}-B{B}/fd", cb.rel_l2(outt, oracle.hypergrad_fd(ow, oth, oth, 0.01, 1.0))) < TOL
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_config3_shape_in_half_precision(parity_record):
    """Configuration 3's problem (3072 -> 1024 -> 10, batch 512) with binary16 operands: one lower step, then the
    finite-difference and Neumann hypergradients."""
    inp = si.config3()
    for b in (inp.train, inp.val):
        b.X = torch.from_numpy(np.ascontiguousarray(b.X, dtype=np.float32)).half().float().numpy()
    bt, cb, w, th, ow, oth = _levels(inp)
    ws = bt.Workspace([w, th])
    bt.betty_lower_step(w, inp.lower_steps, ws)
    oracle.lower_step(ow, inp.lower_steps)
    assert parity_record("fp16/config3/lower_update", _update_err(cb, w, ow, inp.w)) < TOL
    out = torch.empty(si.WEIGHTNET_PARAMS, device="cuda")
    bt.betty_hypergrad_fd(w, th, th, inp.eps0, inp.fd_alpha, out, ws)
    assert parity_record("fp16/config3/fd", cb.rel_l2(out, oracle.hypergrad_fd(ow, oth, oth, inp.eps0, inp.fd_alpha))) < TOL
    bt.betty_hypergrad_neumann(w, th, th, inp.K, inp.alpha, out, ws)
    assert parity_record("fp16/config3/neumann", cb.rel_l2(out, oracle.hypergrad_neumann(ow, oth, oth, inp.K, inp.alpha))) < TOL
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_dynamic_loss_scaling_skips_overflowing_steps_like_the_oracle():
    inp = _inputs(103, (64, 96, 10), 128, "relu")
    bt, cb, w, th, ow, oth = _levels(inp)
    dmax = olv.largest_backward_operand(ow)
    S0 = float(2.0 ** np.ceil(np.log2(65520.0 / dmax) + 2.5))      # the first three steps overflow, well clear of the edge
    w.set_loss_scale(S0, growth_interval=3)
    ow.loss_scale = [S0, 0, 3, 0]
    ws = bt.Workspace([w, th])
    w0 = w.params.clone()
    bt.betty_lower_step(w, 2, ws)
    oracle.lower_step(ow, 2)
    assert torch.equal(w.params, w0)                               # both steps were skipped
    assert w.loss_scale_state.tolist() == [S0 / 4, 0.0, 3.0, 2.0] == [float(x) for x in ow.loss_scale]
    bt.betty_lower_step(w, 7, ws)
    oracle.lower_step(ow, 7)
    assert w.loss_scale_state.tolist() == [float(x) for x in ow.loss_scale]
    assert ow.loss_scale[3] >= 3 and ow.loss_scale[3] < 9
    assert _update_err(cb, w, ow, inp.w) < TOL
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_static_loss_scale_recovers_gradients_that_underflow_without_it():
    """A cost scaled down until its top-layer deltas sit below binary16's smallest subnormal: without a loss
    scale the gradient step vanishes; with one the update matches the oracle.  The per-sample weights are what
    is made small (a weight net whose output bias is very negative), so the forward pass is unaffected."""
    inp = _inputs(107, (64, 96, 10), 128, "relu")
    inp.theta[:] = 0.0
    inp.theta[-1] = -17.0                                          # r_i = sigmoid(-17) ~ 4e-8: deltas ~ 3e-10
    bt, cb, w, th, ow, oth = _levels(inp)
    w.c.lr = ow.lr = 1e6
    ws = bt.Workspace([w, th])
    w0 = w.params.clone()
    w.set_loss_scale(1.0)
    bt.betty_lower_step(w, 1, ws)
    lost = _update_err(cb, w, ow_after := _stepped(ow, 1), inp.w)
    assert lost > 0.5                                              # most of the update never made it through 16 bits
    w.params.copy_(w0)
    w.set_loss_scale(2.0 ** 20)
    bt.betty_lower_step(w, 1, ws)
    assert _update_err(cb, w, ow_after, inp.w) < TOL
    assert w.loss_scale_state.tolist() == [2.0 ** 20, 1.0, 0.0, 0.0]
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def _stepped(olevel, n):
    oracle.lower_step(olevel, n)
    return olevel


def test_precision_and_loss_scale_arguments_are_checked():
    inp = _inputs(109, (64, 96, 10), 32, "relu")
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    w, th = cb.reweight_levels(inp)                               # bfloat16 level
    ws = bt.Workspace([w, th])
    w.set_loss_scale(1024.0)
    with pytest.raises(bt.BettyError) as e:
        bt.betty_lower_step(w, 1, ws)
    assert e.value.status == bt.BETTY_ERR_INVALID_ARG              # loss scaling belongs to binary16 blocks
    w.set_loss_scale(None)
    w.set_precision(bt.BETTY_F16)                                  # but its batch is bfloat16
    with pytest.raises(bt.BettyError) as e:
        bt.betty_lower_step(w, 1, ws)
    assert e.value.status == bt.BETTY_ERR_DTYPE
