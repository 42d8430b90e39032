"""fp64 CPU oracle for the multilevel-optimization hypergradient path.

TEST INFRASTRUCTURE ONLY.  This package is a slow, plain numpy/fp64 statement of what the
CUDA library computes.  It shares no code with the CUDA path and must never be imported by
the product package; only the test-suite, the smoke check and the benchmark's CPU-baseline
leg call it.

What each function follows:
  * levels.py  - the cost functions of the problems (Def. 1, Sec. 2 of the paper; App. D.1
                 for the logistic weight-decay problem; the App. A data-reweighting listing
                 for the reweighted cross-entropy) with their first and second derivatives
                 written out by hand.
  * graph.py   - the dataflow graph of Sec. 3.1: path enumeration and Eq. 2 summed over all paths.
  * solvers.py - unrolled lower-level gradient steps (Sec. 3.2), the best-response-Jacobian
                 times vector operation (Sec. 3.2) with Neumann-series, conjugate-gradient and
                 finite-difference approximations, Eq. 1 (hypergradient of a bilevel pair) and
                 the right-to-left product along one path of Eq. 2.

Pinning status.  Every derivative and the exact quantities the iterations approximate are
pinned by tests that do not go through this code (finite differences of the cost, dense
Hessians/Jacobians, numpy.linalg.solve, closed forms of a quadratic lower level, brute-force
finite differences of the upper loss after a converged lower solve).  The truncated
iterations themselves (Neumann with K terms and step alpha, CG stopped after K iterations,
the finite difference with a finite epsilon) have no values printed in the paper: for those,
parity is "parity unpinned" by the paper and pinned only by their mathematical definition
(matrix-power sums, Krylov optimality, the O(eps^2) limit).
"""
from .graph import engine_run, find_paths, hypergrad_graph  # noqa: F401
from .levels import Level  # noqa: F401
from .solvers import (  # noqa: F401
    brj, cg_solve, chain_levels, grad, hvp, hypergrad_cg, hypergrad_fd, hypergrad_itd, hypergrad_neumann,
    lower_step, mixed_vjp, neumann_solve,
)
