"""The execution schedule of Sec. 3.3 on the GPU against the oracle: the order of steps is integer
work and must match exactly; parameters after the run within the fp32 / bf16 tolerances."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests import oracle_build as ob

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def bt():
    import paper_2207_02849_b200 as bt
    return bt


def test_bilevel_logistic_run(bt):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(31, 300, 32, 80)
    w, lam = cb.logreg_levels(inp)
    ow, olam = ob.logreg_levels(inp)
    lam.c.lr = olam.lr = 0.5
    ws = bt.Workspace([w, lam])
    u2l, l2u = [(1, 0)], [(0, 1)]
    cfg = bt.MethodCfg(bt.BETTY_CG, K=8)
    ocfg = dict(method="cg", K=8)
    log = bt.betty_engine_run([w, lam], u2l, l2u, [cfg, cfg], [5, 1], 20, ws)
    olog = oracle.engine_run([ow, olam], u2l, l2u, [ocfg, ocfg], [5, 1], 20)
    assert log == olog and log.count(1) == 4
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    assert cb.rel_l2(lam.params, olam.params) < 1e-4
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


@pytest.mark.parametrize("unroll,iters", [([1, 1, 1], 2), ([2, 1, 1], 4), ([1, 2, 1], 2)])
def test_three_problem_schedules_match_exactly(bt, unroll, iters):
    from tests import cuda_build as cb
    rng = np.random.default_rng(0)
    A, b = rng.standard_normal((6, 4)).astype(np.float32), rng.standard_normal(6).astype(np.float32)
    f = lambda a: cb.dev(np.asarray(a, np.float32))
    P1 = bt.Level(bt.LOSS_QUADRATIC_WD, bt.PARAM_VECTOR, f(np.zeros(4)), X=f(A), y=f(b), lr=0.01)
    P2 = bt.Level(bt.LOSS_QUADRATIC, bt.PARAM_VECTOR, f(np.full(4, 0.1)), X=f(A), y=f(b), lr=0.01)
    P3 = bt.Level(bt.LOSS_QUADRATIC, bt.PARAM_VECTOR, f(np.full(4, 0.2)), X=f(A), y=f(b), lr=0.01)
    P1.set_constraints([P2]); P2.set_constraints([P1]); P3.set_constraints([P1])
    O1 = oracle.Level(loss="quadratic_wd", param_kind="vector", params=np.zeros(4), X=A, y=b, lr=0.01)
    O2 = oracle.Level(loss="quadratic", param_kind="vector", params=np.full(4, 0.1), X=A, y=b, lr=0.01, constraints=[O1])
    O3 = oracle.Level(loss="quadratic", param_kind="vector", params=np.full(4, 0.2), X=A, y=b, lr=0.01, constraints=[O1])
    O1.constraints = [O2]
    u2l, l2u = [(1, 0)], [(0, 1), (0, 2), (1, 2)]
    cfg, ocfg = bt.MethodCfg(bt.BETTY_NEUMANN, K=1, alpha=0.01), dict(method="neumann", K=1, alpha=0.01)
    ws = bt.Workspace([P1, P2, P3])
    log = bt.betty_engine_run([P1, P2, P3], u2l, l2u, [cfg] * 3, unroll, iters, ws)
    assert log == oracle.engine_run([O1, O2, O3], u2l, l2u, [ocfg] * 3, unroll, iters)
    for P, O in [(P1, O1), (P2, O2), (P3, O3)]:
        assert cb.rel_l2(P.params, O.params) < 1e-4 or np.linalg.norm(O.params) == 0


def test_three_level_mlp_run(bt):
    from tests import cuda_build as cb
    from tests.test_gpu_mlp import _three
    inp = _three("gelu")
    inp.lam = np.full(3, np.log(0.05), dtype=np.float32)     # decay strong enough for lambda's step to register in fp32
    P = cb.three_levels(inp)
    O = ob.three_levels(inp)
    for lv, ol, lr in zip(P, O, (0.1, 0.05, 500.0)):
        lv.c.lr = ol.lr = lr
    ws = bt.Workspace(list(P))
    u2l, l2u = [(2, 0), (1, 0)], [(0, 1), (0, 2), (1, 2)]
    cfg, ocfg = bt.MethodCfg(bt.BETTY_NEUMANN, K=3, alpha=0.01), dict(method="neumann", K=3, alpha=0.01)
    log = bt.betty_engine_run(list(P), u2l, l2u, [cfg] * 3, [2, 1, 1], 4, ws)
    assert log == oracle.engine_run(list(O), u2l, l2u, [ocfg] * 3, [2, 1, 1], 4) == [0, 0, 1, 2, 0, 0, 1, 2]
    assert cb.rel_l2(P[0].params - cb.dev(inp.w), O[0].params - inp.w.astype(np.float64)) < 2e-2       # the updates themselves
    assert cb.rel_l2(P[1].params - cb.dev(inp.theta), O[1].params - inp.theta.astype(np.float64)) < 2e-2
    assert np.linalg.norm(O[2].params - inp.lam) > 1e-4   # the step is well above fp32 resolution of lambda
    assert cb.rel_l2(P[2].params - cb.dev(inp.lam), O[2].params - inp.lam.astype(np.float64)) < 2e-2
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_two_upper_problems_share_one_lower_problem(bt):
    """The extended bilevel structure of the paper's noisy-label program (Sec. 5.1: a reweighting and a
    label-correcting problem above one classifier): two upper problems, each with an upper-to-lower edge
    into the classifier and a lower-to-upper edge out of it.  Built from the cost families at hand: the
    classifier's reweighted cross-entropy with per-layer decay, a weight net and a log-weight-decay vector
    above it, each with the plain cross-entropy of the classifier on a batch of its own."""
    from tests import cuda_build as cb
    from tests.test_gpu_mlp import _three
    inp = _three("gelu")
    inp.lam = np.full(3, np.log(0.05), dtype=np.float32)
    bf = torch.bfloat16
    P1 = bt.Level(bt.LOSS_MLP_CE_REWEIGHT, bt.PARAM_MLP, cb.dev(inp.w), X=cb.dev(inp.D1.X, bf), y=cb.dev(inp.D1.y),
                  widths=inp.widths, activation=bt.ACT_GELU, lr=0.1)
    P2 = bt.Level(bt.LOSS_MLP_CE, bt.PARAM_WEIGHTNET, cb.dev(inp.theta), X=cb.dev(inp.D2.X, bf), y=cb.dev(inp.D2.y_clean), lr=0.05)
    P3 = bt.Level(bt.LOSS_MLP_CE, bt.PARAM_LOGWD, cb.dev(inp.lam), X=cb.dev(inp.D3.X, bf), y=cb.dev(inp.D3.y_clean), lr=200.0)
    P1.set_constraints([P2, P3]); P2.set_constraints([P1]); P3.set_constraints([P1])
    O1 = oracle.Level(loss="mlp_ce_reweight", param_kind="mlp", params=inp.w, X=inp.D1.X, y=inp.D1.y, widths=inp.widths,
                      activation="gelu", lr=0.1, bf16=True)
    O2 = oracle.Level(loss="mlp_ce", param_kind="weightnet", params=inp.theta, X=inp.D2.X, y=inp.D2.y_clean, lr=0.05,
                      constraints=[O1])
    O3 = oracle.Level(loss="mlp_ce", param_kind="logwd", params=inp.lam, X=inp.D3.X, y=inp.D3.y_clean, lr=200.0,
                      constraints=[O1])
    O1.constraints = [O2, O3]
    u2l, l2u = [(1, 0), (2, 0)], [(0, 1), (0, 2)]
    # each upper parameter reaches the classifier's optimum along exactly one path
    assert bt.betty_find_paths(3, u2l, l2u, 1, [0]) == oracle.find_paths(u2l, l2u, 1, [0]) == [[1, 0]]
    assert bt.betty_find_paths(3, u2l, l2u, 2, [0]) == oracle.find_paths(u2l, l2u, 2, [0]) == [[2, 0]]
    cfg, ocfg = bt.MethodCfg(bt.BETTY_NEUMANN, K=3, alpha=0.01), dict(method="neumann", K=3, alpha=0.01)
    ws = bt.Workspace([P1, P2, P3])
    log = bt.betty_engine_run([P1, P2, P3], u2l, l2u, [cfg] * 3, [2, 1, 1], 4, ws)
    assert log == oracle.engine_run([O1, O2, O3], u2l, l2u, [ocfg] * 3, [2, 1, 1], 4) == [0, 0, 1, 2, 0, 0, 1, 2]
    assert cb.rel_l2(P1.params - cb.dev(inp.w), O1.params - inp.w.astype(np.float64)) < 2e-2
    assert cb.rel_l2(P2.params - cb.dev(inp.theta), O2.params - inp.theta.astype(np.float64)) < 2e-2
    assert np.linalg.norm(O3.params - inp.lam) > 1e-4
    assert cb.rel_l2(P3.params - cb.dev(inp.lam), O3.params - inp.lam.astype(np.float64)) < 2e-2
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
