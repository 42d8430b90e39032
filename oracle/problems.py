"""Oracle `Level` objects of the same problem families, built from the same host arrays.

TEST INFRASTRUCTURE (see the package docstring): no arithmetic of the method lives here."""
import numpy as np

from .levels import Level


def logreg_levels(inp):
    lam = Level(loss="logreg", param_kind="vector", params=inp.lam, X=inp.Xv, y=inp.yv)
    w = Level(loss="logreg_wd", param_kind="vector", params=inp.w0, X=inp.X, y=inp.y,
              lr=inp.lr, constraints=[lam])
    lam.constraints = [w]
    return w, lam


def quadratic_levels(A, b, lam, Av, bv, w0=None):
    up = Level(loss="quadratic", param_kind="vector", params=lam, X=Av, y=np.asarray(bv, float))
    lo = Level(loss="quadratic_wd", param_kind="vector",
               params=np.zeros(A.shape[1]) if w0 is None else w0, X=A,
               y=np.asarray(b, float), constraints=[up])
    up.constraints = [lo]
    return lo, up


def reweight_levels(inp, bf16=True, quant="operands", operand_dtype="bf16"):
    theta = Level(loss="mlp_ce", param_kind="weightnet", params=inp.theta, X=inp.val.X,
                  y=inp.val.y)
    w = Level(loss="mlp_ce_reweight", param_kind="mlp", params=inp.w, X=inp.train.X,
              y=inp.train.y, widths=inp.widths, activation=inp.activation, lr=inp.lr,
              bf16=bf16, quant=quant, operand_dtype=operand_dtype, constraints=[theta])
    theta.constraints = [w]
    return w, theta


def three_levels(inp, bf16=True, quant="operands"):
    """P1 classifier, P2 weight net (detector loss on D2), P3 log weight decay (detector
    loss on D3, no mu term)."""
    P1 = Level(loss="mlp_ce_reweight", param_kind="mlp", params=inp.w, X=inp.D1.X, y=inp.D1.y,
               widths=inp.widths, activation=inp.activation, lr=inp.lr, bf16=bf16, quant=quant)
    P2 = Level(loss="weightnet_detect", param_kind="weightnet", params=inp.theta, X=inp.D2.X,
               y=inp.D2.y, aux=inp.D2.clean.astype(np.float64), mu=inp.mu, constraints=[P1])
    P3 = Level(loss="weightnet_detect", param_kind="logwd", params=inp.lam, X=inp.D3.X,
               y=inp.D3.y, aux=inp.D3.clean.astype(np.float64), mu=0.0, constraints=[P2, P1])
    P1.constraints = [P2, P3]
    return P1, P2, P3


def correct_reweight_levels(inp, bf16=True, quant="operands"):
    """Classifier with corrected and reweighted labels below; the reweighting net (plain CE on the clean
    batch) and the correction net (CE of the classifier + CE of its own soft labels on the clean batch) above."""
    theta = Level(loss="mlp_ce", param_kind="weightnet", params=inp.theta, X=inp.val.X, y=inp.val.y)
    alpha = Level(loss="mlp_ce_correct", param_kind="correctnet", params=inp.alpha, X=inp.val.X, y=inp.val.y)
    w = Level(loss="mlp_ce_reweight", param_kind="mlp", params=inp.w, X=inp.train.X, y=inp.train.y,
              widths=inp.widths, activation=inp.activation, lr=inp.lr, bf16=bf16, quant=quant,
              constraints=[theta, alpha])
    theta.constraints = [w]
    alpha.constraints = [w]
    return w, theta, alpha
