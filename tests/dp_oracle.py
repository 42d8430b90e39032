"""Test-side data-parallel evaluation with the fp64 oracle: what the row-sharded path must compute, written
from its definition.  Each rank holds oracle levels built on its own rows; a derivative of a sharded
level's cost is the rank's local derivative times its share of the rows, summed over the ranks by
`reduce` (an in-place sum over ranks of a numpy vector).  Solvers run on the replicated vectors."""
import numpy as np

import oracle


class ShardedOracle:
    def __init__(self, weights, reduce):
        self.weights = weights          # {id(level): row weight of this rank for that level}
        self.reduce = reduce

    def _sum(self, L, vec):
        w = self.weights.get(id(L))
        if w is None:
            return vec
        return self.reduce(np.ascontiguousarray(vec * w, dtype=np.float64))

    def grad(self, L, wrt):
        return self._sum(L, oracle.grad(L, wrt))

    def hvp(self, L, u):
        return self._sum(L, oracle.hvp(L, u))

    def mixed(self, L, wrt, q):
        return self._sum(L, oracle.mixed_vjp(L, wrt, q))

    def lower_step(self, L, n_steps):
        for _ in range(n_steps):
            L.params = L.params - L.lr * self.grad(L, L)

    def hypergrad(self, lower, upper, wrt, method, K=0, alpha=1.0, eps0=0.01):
        v = self.grad(upper, lower)
        direct = self.grad(upper, wrt)
        if method == "neumann":
            q = oracle.neumann_solve(lambda t: self.hvp(lower, t), v, K, alpha)
        elif method == "cg":
            q, _, _ = oracle.cg_solve(lambda t: self.hvp(lower, t), v, K, 0.0)
        else:
            nv = np.sqrt(v @ v)
            eps = eps0 / nv
            gp = oracle.grad(lower, wrt, over={id(lower): lower.params + eps * v, "frozen": {id(lower)}})
            gm = oracle.grad(lower, wrt, over={id(lower): lower.params - eps * v, "frozen": {id(lower)}})
            return direct + self._sum(lower, -alpha * (gp - gm) / (2.0 * eps))
        return direct - self.mixed(lower, wrt, q)
