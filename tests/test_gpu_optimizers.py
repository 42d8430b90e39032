"""Optimiser variants of a problem's step (SGD with momentum and weight decay, Adam) on the GPU
against the oracle, in betty_lower_step and inside the execution schedule."""
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


KINDS = {"momentum": 1, "adam": 2}


@pytest.mark.parametrize("kind", ["momentum", "adam"])
def test_lower_steps_logistic(bt, kind):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(37, 500, 48, 60)
    w, lam = cb.logreg_levels(inp)
    ow, olam = ob.logreg_levels(inp)
    w.c.lr = ow.lr = 0.05
    w.set_optimizer(KINDS[kind], momentum=0.9, weight_decay=0.01)
    ow.optimizer, ow.momentum, ow.weight_decay = kind, 0.9, 0.01
    ws = bt.Workspace([w, lam])
    bt.betty_lower_step(w, 12, ws)
    oracle.lower_step(ow, 12)
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
    out = torch.empty(48, dtype=torch.float32, device="cuda")
    with pytest.raises(bt.BettyError) as e:          # the reverse sweep of ITD assumes plain gradient steps
        bt.betty_hypergrad_itd(w, lam, lam, 2, out, ws)
    assert e.value.status == bt.BETTY_ERR_UNSUPPORTED


def test_reweighting_run_with_momentum_classifier_and_adam_weight_net(bt):
    """The optimiser pairing of the data-reweighting experiment (App. C): SGD with momentum and weight
    decay for the classifier, Adam for the weight net, run through the execution schedule."""
    from tests import cuda_build as cb
    from tests.test_gpu_mlp import _perturb
    inp = _perturb(si.reweight_bilevel(91, (64, 96, 10), 128, 0.4, activation="relu"), 91)
    w, th = cb.reweight_levels(inp)
    ow, oth = ob.reweight_levels(inp)
    w.c.lr = ow.lr = 0.1
    th.c.lr = oth.lr = 1e-3
    w.set_optimizer(bt.BETTY_OPT_MOMENTUM, momentum=0.9, weight_decay=5e-4)
    ow.optimizer, ow.momentum, ow.weight_decay = "momentum", 0.9, 5e-4
    th.set_optimizer(bt.BETTY_OPT_ADAM)
    oth.optimizer = "adam"
    ws = bt.Workspace([w, th])
    u2l, l2u = [(1, 0)], [(0, 1)]
    cfg, ocfg = bt.MethodCfg(bt.BETTY_NEUMANN, K=3, alpha=0.01), dict(method="neumann", K=3, alpha=0.01)
    log = bt.betty_engine_run([w, th], u2l, l2u, [cfg, cfg], [2, 1], 4, ws)
    assert log == oracle.engine_run([ow, oth], u2l, l2u, [ocfg, ocfg], [2, 1], 4) == [0, 0, 1, 0, 0, 1]
    assert cb.rel_l2(w.params - cb.dev(inp.w), ow.params - inp.w.astype(np.float64)) < 2e-2
    # Adam's first steps have magnitude lr whatever the gradient scale, so theta's displacement is well resolved
    assert cb.rel_l2(th.params - cb.dev(inp.theta), oth.params - inp.theta.astype(np.float64)) < 2e-2
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


# ------------------------------------------------------------------ step-size schedules
def _sched(level, olevel, bt, kind, step0=0):
    if kind == "multistep":
        level.set_lr_schedule(bt.BETTY_LR_MULTISTEP, step0=step0, milestones=[3, 7], gamma=0.1)
        olevel.lr_schedule, olevel.lr_milestones, olevel.lr_gamma = "multistep", (3, 7), 0.1
    else:
        level.set_lr_schedule(bt.BETTY_LR_COSINE, step0=step0, t_max=10, lr_min=0.004)
        olevel.lr_schedule, olevel.lr_t_max, olevel.lr_min = "cosine", 10, 0.004
    olevel.lr_step0 = step0


@pytest.mark.parametrize("sched", ["multistep", "cosine"])
@pytest.mark.parametrize("size", [(500, 48), (1024, 64)])     # the second one fits the on-chip whole-loop kernel
def test_scheduled_lower_steps_logistic(bt, sched, size):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(41, size[0], size[1], 60)
    w, lam = cb.logreg_levels(inp)
    ow, olam = ob.logreg_levels(inp)
    w.c.lr = ow.lr = 0.5
    _sched(w, ow, bt, sched)
    ws = bt.Workspace([w, lam])
    bt.betty_lower_step(w, 6, ws)
    oracle.lower_step(ow, 6)
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    _sched(w, ow, bt, sched, step0=6)                      # the next call continues on the schedule
    bt.betty_lower_step(w, 6, ws)
    oracle.lower_step(ow, 6)
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    # the schedule is not a no-op: constant steps end somewhere else
    oc, _ = ob.logreg_levels(inp)
    oc.lr = 0.5
    oracle.lower_step(oc, 12)
    assert cb.rel_l2(w.params, oc.params) > 1e-2
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_scheduled_itd_logistic(bt):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(43, 400, 32, 80)
    w, lam = cb.logreg_levels(inp)
    ow, olam = ob.logreg_levels(inp)
    w.c.lr = ow.lr = 0.5
    _sched(w, ow, bt, "multistep")
    T = 8
    ws = bt.Workspace([w, lam], extra_bytes=(T + 1) * (32 + 64) * 4)
    out = torch.empty(32, dtype=torch.float32, device="cuda")
    bt.betty_hypergrad_itd(w, lam, lam, T, out, ws)
    assert cb.rel_l2(out, oracle.hypergrad_itd(ow, olam, olam, T)) < 1e-4
    assert cb.rel_l2(w.params, ow.params) < 1e-4


@pytest.mark.parametrize("opt", ["gd", "momentum"])
def test_scheduled_lower_steps_mlp(bt, opt):
    """Cosine schedule on the classifier: plain steps take it inside the weight-gradient epilogues,
    momentum steps through the optimiser kernel."""
    from tests import cuda_build as cb
    from tests.test_gpu_mlp import _perturb
    inp = _perturb(si.reweight_bilevel(93, (64, 96, 10), 128, 0.4, activation="gelu"), 93)
    w, th = cb.reweight_levels(inp)
    ow, oth = ob.reweight_levels(inp)
    w.c.lr = ow.lr = 0.2
    if opt == "momentum":
        w.set_optimizer(bt.BETTY_OPT_MOMENTUM, momentum=0.9, weight_decay=5e-4)
        ow.optimizer, ow.momentum, ow.weight_decay = "momentum", 0.9, 5e-4
    _sched(w, ow, bt, "cosine")
    ws = bt.Workspace([w, th])
    bt.betty_lower_step(w, 8, ws)
    oracle.lower_step(ow, 8)
    w0 = cb.dev(inp.w)
    assert cb.rel_l2(w.params - w0, ow.params - inp.w.astype(np.float64)) < 2e-2
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_scheduled_run_through_the_execution_schedule(bt):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(45, 300, 24, 50)
    w, lam = cb.logreg_levels(inp)
    ow, olam = ob.logreg_levels(inp)
    w.c.lr = ow.lr = 0.5
    lam.c.lr = olam.lr = 0.05
    _sched(w, ow, bt, "multistep")
    lam.set_lr_schedule(bt.BETTY_LR_COSINE, t_max=4, lr_min=0.0)
    olam.lr_schedule, olam.lr_t_max, olam.lr_min = "cosine", 4, 0.0
    ws = bt.Workspace([w, lam])
    u2l, l2u = [(1, 0)], [(0, 1)]
    cfg, ocfg = bt.MethodCfg(bt.BETTY_CG, K=8), dict(method="cg", K=8, tol=0.0)
    log = bt.betty_engine_run([w, lam], u2l, l2u, [cfg, cfg], [3, 1], 9, ws)
    assert log == oracle.engine_run([ow, olam], u2l, l2u, [ocfg, ocfg], [3, 1], 9)
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    assert cb.rel_l2(lam.params - cb.dev(inp.lam), olam.params - inp.lam.astype(np.float64)) < 1e-3
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


# ------------------------------------------------------------------ gradient accumulation
@pytest.mark.parametrize("opt", ["gd", "momentum"])
def test_accumulated_steps_mlp(bt, opt):
    from tests import cuda_build as cb
    from tests.test_gpu_mlp import _perturb
    inp = _perturb(si.reweight_bilevel(95, (64, 96, 10), 128, 0.4, activation="gelu"), 95)
    w, th = cb.reweight_levels(inp)
    ow, oth = ob.reweight_levels(inp)
    w.c.lr = ow.lr = 0.2
    if opt == "momentum":
        w.set_optimizer(bt.BETTY_OPT_MOMENTUM, momentum=0.9, weight_decay=5e-4)
        ow.optimizer, ow.momentum, ow.weight_decay = "momentum", 0.9, 5e-4
    w.set_grad_accum(4)
    ow.grad_accum = 4
    ws = bt.Workspace([w, th])
    bt.betty_lower_step(w, 5, ws)
    oracle.lower_step(ow, 5)
    w0 = cb.dev(inp.w)
    assert cb.rel_l2(w.params - w0, ow.params - inp.w.astype(np.float64)) < 2e-2
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
    w.set_grad_accum(3)                                    # 128 rows do not split into 3 equal micro-batches
    with pytest.raises(bt.BettyError) as e:
        bt.betty_lower_step(w, 1, ws)
    assert e.value.status == bt.BETTY_ERR_SHAPE


def test_accumulated_steps_logistic_and_schedule_run(bt):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(47, 512, 32, 64)
    w, lam = cb.logreg_levels(inp)
    ow, olam = ob.logreg_levels(inp)
    w.c.lr = ow.lr = 0.5
    w.set_grad_accum(4)
    ow.grad_accum = 4
    ws = bt.Workspace([w, lam])
    bt.betty_lower_step(w, 6, ws)
    oracle.lower_step(ow, 6)
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    lam.c.lr = olam.lr = 0.2
    u2l, l2u = [(1, 0)], [(0, 1)]
    cfg, ocfg = bt.MethodCfg(bt.BETTY_CG, K=8), dict(method="cg", K=8, tol=0.0)
    log = bt.betty_engine_run([w, lam], u2l, l2u, [cfg, cfg], [3, 1], 6, ws)
    assert log == oracle.engine_run([ow, olam], u2l, l2u, [ocfg, ocfg], [3, 1], 6)
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    assert cb.rel_l2(lam.params - cb.dev(inp.lam), olam.params - inp.lam.astype(np.float64)) < 1e-3
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
