"""Level descriptors (device tensors) of the problem families the library serves, built from host
arrays: the logistic weight-decay pair of App. D.1, a least-squares pair, the data-reweighting pair of
the App. A listing and the three-level chain.  `inp` is any object with the named host arrays (the
seeded generators of the benchmark and the tests produce such objects).  Marshalling only."""
import numpy as np
import torch

from . import binding as bt


def dev(a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


def logreg_levels(inp):
    lam = bt.Level(bt.LOSS_LOGREG, bt.PARAM_VECTOR, dev(inp.lam), X=dev(inp.Xv), y=dev(inp.yv))
    w = bt.Level(bt.LOSS_LOGREG_WD, bt.PARAM_VECTOR, dev(inp.w0), X=dev(inp.X), y=dev(inp.y), lr=inp.lr)
    w.set_constraints([lam])
    lam.set_constraints([w])
    return w, lam


def quadratic_levels(A, b, lam, Av, bv, w0=None):
    f = lambda a: dev(np.asarray(a, dtype=np.float32))
    up = bt.Level(bt.LOSS_QUADRATIC, bt.PARAM_VECTOR, f(lam), X=f(Av), y=f(bv))
    lo = bt.Level(bt.LOSS_QUADRATIC_WD, bt.PARAM_VECTOR, f(np.zeros(A.shape[1]) if w0 is None else w0),
                  X=f(A), y=f(b))
    lo.set_constraints([up])
    up.set_constraints([lo])
    return lo, up


def _act(name):
    return bt.ACT_RELU if name == "relu" else bt.ACT_GELU


def reweight_levels(inp, operand_dtype=torch.bfloat16):
    """operand_dtype: torch.bfloat16 (default) or torch.float16, the type of the batches and of the classifier's
    matrix-product operands."""
    theta = bt.Level(bt.LOSS_MLP_CE, bt.PARAM_WEIGHTNET, dev(inp.theta), X=dev(inp.val.X, operand_dtype),
                     y=dev(inp.val.y))
    w = bt.Level(bt.LOSS_MLP_CE_REWEIGHT, bt.PARAM_MLP, dev(inp.w), X=dev(inp.train.X, operand_dtype),
                 y=dev(inp.train.y), widths=inp.widths, activation=_act(inp.activation), lr=inp.lr)
    if operand_dtype == torch.float16:
        w.set_precision(bt.BETTY_F16)
    w.set_constraints([theta])
    theta.set_constraints([w])
    return w, theta


def three_levels(inp):
    P1 = bt.Level(bt.LOSS_MLP_CE_REWEIGHT, bt.PARAM_MLP, dev(inp.w), X=dev(inp.D1.X, torch.bfloat16),
                  y=dev(inp.D1.y), widths=inp.widths, activation=_act(inp.activation), lr=inp.lr)
    P2 = bt.Level(bt.LOSS_WEIGHTNET_DETECT, bt.PARAM_WEIGHTNET, dev(inp.theta), X=dev(inp.D2.X, torch.bfloat16),
                  y=dev(inp.D2.y), aux=dev(inp.D2.clean), mu=inp.mu)
    P3 = bt.Level(bt.LOSS_WEIGHTNET_DETECT, bt.PARAM_LOGWD, dev(inp.lam), X=dev(inp.D3.X, torch.bfloat16),
                  y=dev(inp.D3.y), aux=dev(inp.D3.clean), mu=0.0)
    P1.set_constraints([P2, P3])
    P2.set_constraints([P1])
    P3.set_constraints([P2, P1])
    return P1, P2, P3


def correct_reweight_levels(inp):
    """The extended bilevel program of the noisy-label experiment: classifier below (labels corrected and
    reweighted), the reweighting net and the label-correction net above, both on the clean batch."""
    Xv, yv = dev(inp.val.X, torch.bfloat16), dev(inp.val.y)
    theta = bt.Level(bt.LOSS_MLP_CE, bt.PARAM_WEIGHTNET, dev(inp.theta), X=Xv, y=yv)
    alpha = bt.Level(bt.LOSS_MLP_CE_CORRECT, bt.PARAM_CORRECTNET, dev(inp.alpha), X=Xv, y=yv)
    w = bt.Level(bt.LOSS_MLP_CE_REWEIGHT, bt.PARAM_MLP, dev(inp.w), X=dev(inp.train.X, torch.bfloat16),
                 y=dev(inp.train.y), widths=inp.widths, activation=_act(inp.activation), lr=inp.lr)
    w.set_constraints([theta, alpha])
    theta.set_constraints([w])
    alpha.set_constraints([w])
    return w, theta, alpha
