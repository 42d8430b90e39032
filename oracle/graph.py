"""The dataflow graph of Sec. 3.1 and Eq. 2 over it (fp64 oracle; TEST INFRASTRUCTURE).

Two kinds of directed edges between problems: upper-to-lower (theta_i constrains problem j) and
lower-to-upper (theta*_i constrains problem j).  A valid path from theta_k to theta*_l takes one
upper-to-lower edge first and lower-to-upper edges afterwards (Sec. 3.1)."""
from __future__ import annotations

import numpy as np

from .solvers import apply_optimizer, chain_levels, grad, step_gradient


def find_paths(u2l, l2u, k, targets):
    """All valid paths [k, q(1), ..., q(m)] from theta_k to a problem in `targets`, by depth-first
    search in edge order.  u2l / l2u are lists of (from, to) pairs."""
    targets = set(targets)
    out = []

    def visit(path):
        c = path[-1]
        if c in targets:
            out.append([k] + path)
        for a, b in l2u:
            if a == c and b != k and b not in path:
                visit(path + [b])

    for a, b in u2l:
        if a == k and b != k:
            visit([b])
    return out


def hypergrad_graph(levels, u2l, l2u, k, cfgs) -> np.ndarray:
    """Eq. 2 written out: direct gradient plus, for every lower problem l that constrains k through
    its optimal parameters and every valid path from theta_k to theta*_l, the path's Jacobian chain
    times dC_k/d theta*_l.  cfgs[q] holds the `brj` keyword arguments of problem q's Jacobians."""
    L_k = [a for a, b in l2u if b == k]
    total = grad(levels[k], levels[k]).copy()
    for path in find_paths(u2l, l2u, k, L_k):
        edge_cfgs = [cfgs[q] for q in path[1:]]
        total = total + chain_levels(levels, path, edge_cfgs)
    return total


def engine_run(levels, u2l, l2u, cfgs, unroll, n_iterations):
    """Execution of the whole program (Sec. 3.3).  Only the lowermost problems are stepped directly;
    a problem that has completed `unroll[j]` steps calls the problems it constrains through
    lower-to-upper edges; a called problem steps once every problem of its L set has called.  One
    step of problem j is one step of its optimiser along the gradient of Eq. 2.
    Returns the list of problem indices in the order they stepped."""
    n = len(levels)
    n_lower = [sum(1 for a, b in l2u if b == j) for j in range(n)]
    count, ready, log = [0] * n, [0] * n, []

    def step(j):
        log.append(j)
        if n_lower[j] == 0 and levels[j].grad_accum > 1:
            g = step_gradient(levels[j])
        else:
            g = hypergrad_graph(levels, u2l, l2u, j, cfgs)
        apply_optimizer(levels[j], g, count[j])
        count[j] += 1
        if count[j] % unroll[j] == 0:
            for a, b in l2u:
                if a == j:
                    ready[b] += 1
                    if ready[b] >= n_lower[b]:
                        ready[b] = 0
                        step(b)

    for _ in range(int(n_iterations)):
        for j in range(n):
            if n_lower[j] == 0:
                step(j)
    return log
