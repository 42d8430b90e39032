"""Pins for the oracle's execution schedule (Sec. 3.3): the order of steps for hand-worked unroll
settings, and the upper-level trajectory against brute-force gradient descent on the closed-form
bilevel objective of a quadratic lower problem."""
import numpy as np

import oracle
from oracle import Level
from oracle import levels as olv
from tests.oracle_build import quadratic_levels


def _dummy_three_levels():
    """Three tiny quadratic-family problems wired like the three-level configuration; only the
    schedule is looked at, so every gradient just has to exist."""
    rng = np.random.default_rng(0)
    A, b = rng.standard_normal((6, 3)), rng.standard_normal(6)
    P1 = Level(loss="quadratic_wd", param_kind="vector", params=np.zeros(3), X=A, y=b, lr=0.01)
    P2 = Level(loss="quadratic", param_kind="vector", params=np.full(3, 0.1), X=A, y=b, lr=0.01, constraints=[P1])
    P3 = Level(loss="quadratic", param_kind="vector", params=np.full(3, 0.2), X=A, y=b, lr=0.01, constraints=[P1])
    P1.constraints = [P2]
    return [P1, P2, P3]


def test_schedule_orders_follow_section_3_3():
    l2u = [(0, 1), (0, 2), (1, 2)]          # P1 calls P2 and P3; P2 calls P3; P3 waits for both
    nm = dict(method="neumann", K=1, alpha=0.01)
    run = lambda unroll, iters: oracle.engine_run(_dummy_three_levels(), [(1, 0)], l2u, [nm] * 3, unroll, iters)
    # all unroll counts 1: every iteration steps P1, then P2 (called by P1), then P3 (both calls in)
    assert run([1, 1, 1], 2) == [0, 1, 2, 0, 1, 2]
    # P1 unrolls two steps before calling upwards
    assert run([2, 1, 1], 4) == [0, 0, 1, 2, 0, 0, 1, 2]
    # P2 calls P3 only after two of its own steps; P3 still needs P1's call as well
    assert run([1, 2, 1], 2) == [0, 1, 0, 1, 2]
    # a bilevel pair with 3 unrolled lower steps per upper step (App. A listing uses unroll_steps)
    lo, up = quadratic_levels(np.eye(2), np.ones(2), np.full(2, 0.5), np.eye(2), np.zeros(2))
    cg = dict(method="cg", K=2)
    assert oracle.engine_run([lo, up], [(1, 0)], [(0, 1)], [cg, cg], [3, 1], 7) == [0, 0, 0, 1, 0, 0, 0, 1, 0]


def test_upper_trajectory_equals_gradient_descent_on_the_closed_form_bilevel_objective():
    rng = np.random.default_rng(3)
    A, b = rng.standard_normal((12, 4)), rng.standard_normal(12)
    Av, bv = rng.standard_normal((9, 4)), rng.standard_normal(9)
    lam0 = rng.random(4) + 0.5
    lo, up = quadratic_levels(A, b, lam0, Av, bv)
    lo.lr = 0.9 / np.linalg.eigvalsh(A.T @ A + np.diag(lam0)).max()
    up.lr = 0.05
    unroll = 600                                           # the lower problem converges between upper steps

    def F(lam):
        w = np.linalg.solve(A.T @ A + np.diag(lam), A.T @ b)
        return 0.5 * np.sum((Av @ w - bv) ** 2)

    lam = lam0.copy()
    for _ in range(3):                                     # brute-force gradient descent on F
        g = np.array([(F(lam + 1e-6 * e) - F(lam - 1e-6 * e)) / 2e-6 for e in np.eye(4)])
        lam = lam - up.lr * g
    cg = dict(method="cg", K=4)
    log = oracle.engine_run([lo, up], [(1, 0)], [(0, 1)], [cg, cg], [unroll, 1], 3 * unroll)
    assert log.count(1) == 3 and log[unroll] == 1
    assert np.linalg.norm(up.params - lam) / np.linalg.norm(lam) < 1e-6
    assert F(up.params) < F(lam0)
