"""The label-correction costs of the extended bilevel program (Sec. 5.1, "Correcting & reweighting corrupted
labels") on the GPU against the fp64 oracle: gradients with respect to every participant, lower steps, the
finite-difference hypergradients of both upper problems (the method the paper pairs this program with), and a run
of the whole program through the execution schedule.  bf16 matrix products: relative L2 error <= 2e-2."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests import oracle_build as ob

pytestmark = pytest.mark.gpu
TOL = 2e-2


def _inputs(seed, widths, B, act):
    inp = si.correct_reweight(seed, widths, B, 0.4, activation=act)
    inp.w = inp.w + si.to_bf16_values(si.normal_f32(seed, 300, inp.w.shape) * np.float32(0.02))
    inp.theta = (si.weightnet_init(seed, 200) * np.float32(3.0)).astype(np.float32)
    inp.alpha = (inp.alpha + si.normal_f32(seed, 310, inp.alpha.shape) * np.float32(0.1)).astype(np.float32)
    return inp


def _vec(n):
    return torch.empty(n, dtype=torch.float32, device="cuda")


@pytest.mark.parametrize("act,widths,B", [("relu", (24, 40, 16), 37), ("gelu", (64, 96, 10), 128),
                                          ("gelu", (16, 72, 64, 10), 130), ("relu", (40, 130, 66, 12), 200)])
def test_corrected_costs_match_oracle(act, widths, B, parity_record):
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = _inputs(201, widths, B, act)
    w, th, al = cb.correct_reweight_levels(inp)
    ow, oth, oal = ob.correct_reweight_levels(inp)
    ws = bt.Workspace([w, th, al])
    gw, gt, ga = _vec(inp.w.size), _vec(si.WEIGHTNET_PARAMS), _vec(inp.alpha.size)
    tag = f"correct/{act}-{'x'.join(map(str, widths))}"
    bt.betty_grad(w, w, gw, ws)
    assert parity_record(f"{tag}/grad_w", cb.rel_l2(gw, oracle.grad(ow, ow))) < TOL
    bt.betty_grad(w, al, ga, ws)
    assert parity_record(f"{tag}/grad_alpha", cb.rel_l2(ga, oracle.grad(ow, oal))) < TOL
    bt.betty_grad(w, th, gt, ws)
    assert cb.rel_l2(gt, oracle.grad(ow, oth)) < TOL
    bt.betty_grad(al, w, gw, ws)
    assert parity_record(f"{tag}/upper_grad_w", cb.rel_l2(gw, oracle.grad(oal, ow))) < TOL
    bt.betty_grad(al, al, ga, ws)
    assert cb.rel_l2(ga, oracle.grad(oal, oal)) < TOL
    H, C = widths[-2], widths[-1]
    assert torch.all(ga[C * H + C:] == 0)                   # the interpolation net takes no part in the upper cost
    bt.betty_grad(th, w, gw, ws)
    assert cb.rel_l2(gw, oracle.grad(oth, ow)) < TOL
    # second derivatives are not offered with label correction
    with pytest.raises(bt.BettyError) as e:
        bt.betty_hvp(w, cb.dev(inp.w), gw, ws)
    assert e.value.status == bt.BETTY_ERR_UNSUPPORTED
    # lower steps, then the finite-difference hypergradients of both upper problems
    bt.betty_lower_step(w, 2, ws)
    oracle.lower_step(ow, 2)
    w0 = inp.w.astype(np.float64)
    assert parity_record(f"{tag}/lower_update", cb.rel_l2(w.params.double().cpu().numpy() - w0, ow.params - w0)) < TOL
    # Both sides continue from the same lower parameters (the oracle's, as fp32).  A finite difference of gradients
    # through ReLU units is a discontinuous function of w: which of the few dozen units change side between
    # w + eps v and w - eps v decides the blocks of the result that belong to the interpolation net's first layer
    # (measured: parameters that differ by 1e-5 relative move those blocks by 20%, the rest by 5e-4), so the chain
    # "steps, then hypergradient" would compare two different sets of units, not the arithmetic.
    w.params.copy_(torch.from_numpy(ow.params.astype(np.float32)))
    ow.params = w.params.double().cpu().numpy()
    bt.betty_hypergrad_fd(w, al, al, 0.01, 1.0, ga, ws)
    assert parity_record(f"{tag}/fd_alpha", cb.rel_l2(ga, oracle.hypergrad_fd(ow, oal, oal, 0.01, 1.0))) < TOL
    bt.betty_hypergrad_fd(w, th, th, 0.01, 1.0, gt, ws)
    assert parity_record(f"{tag}/fd_theta", cb.rel_l2(gt, oracle.hypergrad_fd(ow, oth, oth, 0.01, 1.0))) < TOL
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_corrected_costs_at_configuration_3_size(parity_record):
    """The data-reweighting configuration's classifier (3072 -> 1024 -> 10, batch 512, 40% label noise) with the
    correction net attached (112,851 parameters): both upper problems' finite-difference hypergradients."""
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.correct_reweight(si.BASE_SEED + 3, (3072, 1024, 10), 512, 0.4, activation="relu")
    w, th, al = cb.correct_reweight_levels(inp)
    ow, oth, oal = ob.correct_reweight_levels(inp)
    ws = bt.Workspace([w, th, al])
    ga, gt = _vec(inp.alpha.size), _vec(si.WEIGHTNET_PARAMS)
    bt.betty_hypergrad_fd(w, al, al, 0.01, 1.0, ga, ws)
    assert parity_record("correct/config3-size/fd_alpha", cb.rel_l2(ga, oracle.hypergrad_fd(ow, oal, oal, 0.01, 1.0))) < TOL
    bt.betty_hypergrad_fd(w, th, th, 0.01, 1.0, gt, ws)
    assert parity_record("correct/config3-size/fd_theta", cb.rel_l2(gt, oracle.hypergrad_fd(ow, oth, oth, 0.01, 1.0))) < TOL
    bt.betty_lower_step(w, 1, ws)
    oracle.lower_step(ow, 1)
    w0 = inp.w.astype(np.float64)
    assert parity_record("correct/config3-size/lower_update", cb.rel_l2(w.params.double().cpu().numpy() - w0, ow.params - w0)) < TOL
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_extended_bilevel_program_runs_through_the_schedule():
    """Sec. 5.1's program as its App. A listing wires it: two upper problems (reweight, correct), each with an
    upper-to-lower edge into the classifier and a lower-to-upper edge out of it, finite-difference Jacobians,
    the classifier unrolled for a few steps between upper steps."""
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = _inputs(203, (64, 96, 10), 128, "gelu")
    w, th, al = cb.correct_reweight_levels(inp)
    ow, oth, oal = ob.correct_reweight_levels(inp)
    for lv, ol, lr in ((w, ow, 0.1), (th, oth, 0.05), (al, oal, 0.05)):
        lv.c.lr = ol.lr = lr
    u2l, l2u = [(1, 0), (2, 0)], [(0, 1), (0, 2)]
    assert bt.betty_find_paths(3, u2l, l2u, 2, [0]) == oracle.find_paths(u2l, l2u, 2, [0]) == [[2, 0]]
    cfg, ocfg = bt.MethodCfg(bt.BETTY_FD, eps0=0.01, alpha=1.0), dict(method="fd", eps0=0.01, alpha=1.0)
    ws = bt.Workspace([w, th, al])
    log = bt.betty_engine_run([w, th, al], u2l, l2u, [cfg] * 3, [2, 1, 1], 4, ws)
    assert log == oracle.engine_run([ow, oth, oal], u2l, l2u, [ocfg] * 3, [2, 1, 1], 4) == [0, 0, 1, 2, 0, 0, 1, 2]
    for lv, ol, x0 in ((w, ow, inp.w), (th, oth, inp.theta)):
        x0 = x0.astype(np.float64)
        assert cb.rel_l2(lv.params.double().cpu().numpy() - x0, ol.params - x0) < TOL
    # The correction net's update, block by block.  Here the two sides cannot be put on the same lower parameters
    # between the classifier's steps and the upper steps, so the blocks that a handful of ReLU units decide (the
    # interpolation net's first layer, see test_corrected_costs_match_oracle) are only held to the right size;
    # every other block is held to the tolerance.
    H, C, HD = inp.widths[-2], inp.widths[-1], si.WEIGHTNET_HIDDEN
    edges = [0, C * H + C, C * H + C + HD * H + HD, inp.alpha.size]          # [A, a0 | A1, b1 | a2, b2]
    got = al.params.double().cpu().numpy() - inp.alpha.astype(np.float64)
    ref = oal.params - inp.alpha.astype(np.float64)
    assert cb.rel_l2(got[edges[0]:edges[1]], ref[edges[0]:edges[1]]) < TOL
    assert cb.rel_l2(got[edges[2]:edges[3]], ref[edges[2]:edges[3]]) < TOL
    assert cb.rel_l2(got[edges[1]:edges[2]], ref[edges[1]:edges[2]]) < 0.6
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_correction_net_shape_is_checked():
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = _inputs(205, (24, 40, 16), 16, "relu")
    inp.alpha = inp.alpha[:-1]                              # one parameter short
    w, th, al = cb.correct_reweight_levels(inp)
    ws = bt.Workspace([w, th])
    with pytest.raises(bt.BettyError) as e:
        bt.betty_grad(w, w, _vec(inp.w.size), ws)
    assert e.value.status == bt.BETTY_ERR_SHAPE
