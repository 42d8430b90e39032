"""Seeded synthetic inputs for the multilevel-optimization workloads.

This module only draws numbers and shapes them: it contains no loss, gradient,
Hessian or solver arithmetic.  It is the single piece of code that both the
fp64 CPU oracle's tests and the CUDA path's tests/benchmarks import, so that the
two are always fed bit-identical arrays.

Random numbers come from numpy's Philox (a counter-based generator) keyed by
(seed, stream id); every array has its own stream id so that shapes can change
without shifting other draws.

The five workloads mirror the structure of the paper's experiments (bilevel
hyper-parameter optimisation of a per-feature weight decay for logistic
regression, App. D.1; Meta-Weight-Net style data reweighting with a 1-100-1
weight net, Sec. 5.1 / App. A listing; a three-level chain, Sec. 5.3) with
synthetic data standing in for the public datasets.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

BASE_SEED = 20220702

WEIGHTNET_HIDDEN = 100
WEIGHTNET_PARAMS = 3 * WEIGHTNET_HIDDEN + 1


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def normal_f32(seed: int, stream: int, shape, chunk_rows: int = 16384) -> np.ndarray:
    """N(0,1) float32 array, generated in row chunks to bound temporary memory."""
    g = _rng(seed, stream)
    shape = tuple(int(s) for s in np.atleast_1d(shape))
    if len(shape) == 1 or shape[0] <= chunk_rows:
        return g.standard_normal(shape, dtype=np.float32)
    out = np.empty(shape, dtype=np.float32)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        out[r0:r1] = g.standard_normal((r1 - r0,) + shape[1:], dtype=np.float32)
    return out


def to_bf16_values(a: np.ndarray) -> np.ndarray:
    """Round a float32 array to the nearest bf16-representable value (ties to even),
    returned as float32.  Uses torch's conversion as the library routine."""
    import torch

    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


# --------------------------------------------------------------------------- logistic
@dataclass
class LogregBilevel:
    """Inputs of the bilevel weight-decay problem for binary logistic regression."""
    X: np.ndarray      # [n, d] float32 train features
    y: np.ndarray      # [n]    float32 in {-1,+1}
    Xv: np.ndarray     # [nv, d] float32 validation features
    yv: np.ndarray     # [nv]   float32 in {-1,+1}
    lam: np.ndarray    # [d] float32 per-feature weight decay (upper parameters)
    w0: np.ndarray     # [d] float32 lower start point
    lr: float = 0.1
    lower_steps: int = 100
    K: int = 10
    alpha: float = 0.01


def _planted_labels(X: np.ndarray, theta: np.ndarray, flip_u: np.ndarray, flip_p: float,
                    chunk_rows: int = 16384) -> np.ndarray:
    n = X.shape[0]
    y = np.empty(n, dtype=np.float32)
    t64 = theta.astype(np.float64)
    for r0 in range(0, n, chunk_rows):
        r1 = min(n, r0 + chunk_rows)
        s = X[r0:r1].astype(np.float64) @ t64
        y[r0:r1] = np.where(s >= 0.0, 1.0, -1.0)
    y[flip_u < flip_p] *= -1.0
    return y


def logreg_bilevel(seed: int, n: int, d: int, n_val: int, *, flip: float = 0.1,
                   lam0: float = 1e-2, lower_steps: int = 100, K: int = 10,
                   alpha: float = 0.01, lr: float = 0.1) -> LogregBilevel:
    theta = normal_f32(seed, 1, (d,))
    X = normal_f32(seed, 2, (n, d))
    Xv = normal_f32(seed, 3, (n_val, d))
    y = _planted_labels(X, theta, _rng(seed, 4).random(n), flip)
    yv = _planted_labels(Xv, theta, _rng(seed, 5).random(n_val), flip)
    return LogregBilevel(X=X, y=y, Xv=Xv, yv=yv,
                         lam=np.full(d, lam0, dtype=np.float32),
                         w0=np.zeros(d, dtype=np.float32),
                         lr=lr, lower_steps=lower_steps, K=K, alpha=alpha)


# --------------------------------------------------------------------------- classification
@dataclass
class ClassBatch:
    X: np.ndarray        # [B, d_in] float32 holding bf16-representable values
    y: np.ndarray        # [B] int32 labels as given to the learner (possibly noisy)
    y_clean: np.ndarray  # [B] int32 teacher labels
    clean: np.ndarray    # [B] float32 1.0 where y == teacher label was kept, else 0.0


def teacher(seed: int, d_in: int, n_classes: int) -> np.ndarray:
    return normal_f32(seed, 10, (d_in, n_classes))


def class_batch(seed: int, stream: int, B: int, d_in: int, n_classes: int, noise: float,
                T: np.ndarray) -> ClassBatch:
    """N(0,1) inputs rounded to bf16 values, labels = argmax of a planted linear
    teacher; with probability `noise` a label is replaced by a uniform draw from all classes."""
    X = to_bf16_values(normal_f32(seed, stream, (B, d_in)))
    scores = X.astype(np.float64) @ T.astype(np.float64)
    y_clean = np.argmax(scores, axis=1).astype(np.int32)
    g = _rng(seed, stream + 1000)
    replace = g.random(B) < noise
    draw = g.integers(0, n_classes, size=B, dtype=np.int64).astype(np.int32)
    y = np.where(replace, draw, y_clean).astype(np.int32)
    return ClassBatch(X=X, y=y, y_clean=y_clean, clean=(~replace).astype(np.float32))


def mlp_param_count(widths) -> int:
    return int(sum(widths[l + 1] * widths[l] + widths[l + 1] for l in range(len(widths) - 1)))


def mlp_init(seed: int, stream: int, widths) -> np.ndarray:
    """Flat fp32 parameter vector [W_1, b_1, W_2, b_2, ...] with W_l of shape
    [out_l, in_l] row-major ~ N(0, 1/in_l) rounded to bf16 values and b_l = 0."""
    parts = []
    for l in range(len(widths) - 1):
        fin, fout = int(widths[l]), int(widths[l + 1])
        W = normal_f32(seed, stream + l, (fout, fin)) * np.float32(1.0 / np.sqrt(fin))
        parts.append(to_bf16_values(W).reshape(-1))
        parts.append(np.zeros(fout, dtype=np.float32))
    return np.concatenate(parts)


def weightnet_init(seed: int, stream: int, *, b2: float = 0.0) -> np.ndarray:
    """Flat [a1(100), b1(100), a2(100), b2(1)]; a1, a2 ~ N(0, 1/100), biases 0."""
    H = WEIGHTNET_HIDDEN
    a1 = normal_f32(seed, stream, (H,)) * np.float32(0.1)
    a2 = normal_f32(seed, stream + 1, (H,)) * np.float32(0.1)
    return np.concatenate([a1, np.zeros(H, np.float32), a2, np.full(1, b2, np.float32)])


@dataclass
class ReweightBilevel:
    """Data reweighting: lower MLP classifier trained on a noisy batch with per-sample
    weights from a 1-100-1 net; upper loss = plain CE of the classifier on a clean batch."""
    widths: tuple
    activation: str
    w: np.ndarray            # flat MLP params
    theta: np.ndarray        # weight-net params (301)
    train: ClassBatch
    val: ClassBatch
    lr: float = 0.1
    lower_steps: int = 1
    K: int = 5
    alpha: float = 0.01
    eps0: float = 0.01
    fd_alpha: float = 1.0


def reweight_bilevel(seed: int, widths, B: int, noise: float, *, activation: str = "relu",
                     lower_steps: int = 1, K: int = 5, alpha: float = 0.01,
                     Bv: int | None = None) -> ReweightBilevel:
    widths = tuple(int(w) for w in widths)
    T = teacher(seed, widths[0], widths[-1])
    return ReweightBilevel(
        widths=widths, activation=activation,
        w=mlp_init(seed, 100, widths), theta=weightnet_init(seed, 200),
        train=class_batch(seed, 20, B, widths[0], widths[-1], noise, T),
        val=class_batch(seed, 30, Bv or B, widths[0], widths[-1], 0.0, T),
        lower_steps=lower_steps, K=K, alpha=alpha)


def correctnet_size(H: int, C: int) -> int:
    """Parameters of the label-correction net on a classifier with last hidden width H and C classes:
    a linear layer H -> C for the soft labels and an H-100-1 net for the interpolation weight."""
    return C * H + C + WEIGHTNET_HIDDEN * H + 2 * WEIGHTNET_HIDDEN + 1


def correctnet_init(seed: int, stream: int, H: int, C: int) -> np.ndarray:
    """[A (C x H), a0 (C), A1 (100 x H), b1 (100), a2 (100), b2]: matrices ~ N(0, 1/fan_in), biases 0."""
    Hd = WEIGHTNET_HIDDEN
    A = normal_f32(seed, stream, (C * H,)) * np.float32(1.0 / np.sqrt(H))
    A1 = normal_f32(seed, stream + 1, (Hd * H,)) * np.float32(1.0 / np.sqrt(H))
    a2 = normal_f32(seed, stream + 2, (Hd,)) * np.float32(1.0 / np.sqrt(Hd))
    return np.concatenate([A, np.zeros(C, np.float32), A1, np.zeros(Hd, np.float32), a2, np.zeros(1, np.float32)]).astype(np.float32)


@dataclass
class CorrectReweight:
    """The extended bilevel program of the paper's noisy-label experiment: one classifier below, a
    reweighting net and a label-correction net above it, both trained on the clean batch."""
    widths: tuple
    activation: str
    w: np.ndarray
    theta: np.ndarray        # reweighting net (301)
    alpha: np.ndarray        # correction net
    train: ClassBatch
    val: ClassBatch
    lr: float = 0.1
    eps0: float = 0.01
    fd_alpha: float = 1.0


def correct_reweight(seed: int, widths, B: int, noise: float, *, activation: str = "relu",
                     Bv: int | None = None) -> CorrectReweight:
    widths = tuple(int(w) for w in widths)
    T = teacher(seed, widths[0], widths[-1])
    return CorrectReweight(
        widths=widths, activation=activation, w=mlp_init(seed, 100, widths), theta=weightnet_init(seed, 200),
        alpha=correctnet_init(seed, 210, widths[-2], widths[-1]),
        train=class_batch(seed, 20, B, widths[0], widths[-1], noise, T),
        val=class_batch(seed, 30, Bv or B, widths[0], widths[-1], 0.0, T))


@dataclass
class ThreeLevel:
    """Three-level chain: P1 classifier w (loss reweighted CE + per-layer exp(lambda) weight
    decay), P2 weight net theta (clean-label detector loss on batch D2, coupled to w through the
    per-sample losses), P3 per-layer log weight decay lambda (detector loss on batch D3)."""
    widths: tuple
    activation: str
    w: np.ndarray
    theta: np.ndarray
    lam: np.ndarray          # [n_layers] log weight decay
    D1: ClassBatch
    D2: ClassBatch
    D3: ClassBatch
    mu: float = 1e-3
    lr: float = 0.1
    lower_steps: int = 1
    K: int = 3
    alpha: float = 0.01


def three_level(seed: int, widths, B: int, noise: float, *, activation: str = "relu",
                K: int = 3, alpha: float = 0.01) -> ThreeLevel:
    widths = tuple(int(w) for w in widths)
    T = teacher(seed, widths[0], widths[-1])
    L = len(widths) - 1
    return ThreeLevel(
        widths=widths, activation=activation,
        w=mlp_init(seed, 100, widths), theta=weightnet_init(seed, 200),
        lam=np.full(L, np.log(5e-4), dtype=np.float32),
        D1=class_batch(seed, 20, B, widths[0], widths[-1], noise, T),
        D2=class_batch(seed, 30, B, widths[0], widths[-1], noise, T),
        D3=class_batch(seed, 40, B, widths[0], widths[-1], noise, T),
        K=K, alpha=alpha)


# --------------------------------------------------------------------------- the five workloads
def config1(small: bool = False) -> LogregBilevel:
    return logreg_bilevel(BASE_SEED + 1, 1024, 64, 256, lower_steps=100, K=10, alpha=0.01)


def config2(scale: float = 1.0) -> LogregBilevel:
    """262144 x 4096 train (4 GiB fp32), 32768 x 4096 validation; `scale` < 1 shrinks the
    row counts only (used by tests that want the same column count on fewer rows)."""
    n = max(8, int(round(262144 * scale)))
    nv = max(8, int(round(32768 * scale)))
    return logreg_bilevel(BASE_SEED + 2, n, 4096, nv, lower_steps=20, K=20, alpha=0.01)


def config3() -> ReweightBilevel:
    return reweight_bilevel(BASE_SEED + 3, (3072, 1024, 10), 512, 0.4, lower_steps=1, K=5)


def config4() -> ThreeLevel:
    return three_level(BASE_SEED + 4, (784, 512, 512, 10), 1024, 0.3, K=3)


def config5(width: int = 4096, depth: int = 8, n_classes: int = 1000, B: int = 1024
            ) -> ReweightBilevel:
    widths = (width,) * (depth + 1) + (n_classes,)
    return reweight_bilevel(BASE_SEED + 5, widths, B, 0.2, activation="gelu",
                            lower_steps=4, K=3)
