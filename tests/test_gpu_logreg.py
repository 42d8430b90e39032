"""Parity of the CUDA path with the fp64 oracle for the logistic / quadratic families
(App. D.1 problem): element-by-element on the same seeded inputs, through the C ABI.
Tolerance: relative L2 error <= 1e-4 for fp32 hypergradients."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests import oracle_build as ob

pytestmark = pytest.mark.gpu
TOL = 1e-4


@pytest.fixture(scope="module")
def bt():
    import paper_2207_02849_b200 as bt
    return bt


def _pair(inp):
    from tests import cuda_build as cb
    return cb.logreg_levels(inp), ob.logreg_levels(inp)


def _vec(n):
    return torch.empty(n, dtype=torch.float32, device="cuda")


SHAPES = [
    (1024, 64, 256),      # the small configuration
    (37, 64, 5),          # fewer rows than CTAs
    (2051, 4096, 513),    # full width, several tiles per CTA and a ragged last tile
    (1000, 2048, 300), (777, 1024, 100), (333, 516, 64),
    (257, 130, 33),       # d % 4 != 0: two-pass kernels
    (300, 4100, 40),      # d > 4096: two-pass kernels
    (1, 8, 1),
]


@pytest.mark.parametrize("n,d,nv", SHAPES)
def test_primitives_match_oracle(bt, n, d, nv):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(100 + n + d, n, d, nv)
    inp.w0 = si.normal_f32(7, 1, (d,)) * np.float32(0.5 / np.sqrt(d))
    inp.lam = (np.abs(si.normal_f32(7, 2, (d,))) * 0.05 + 0.01).astype(np.float32)
    (w, lam), (ow, olam) = _pair(inp)
    ws = bt.Workspace([w, lam])
    out = _vec(d)
    bt.betty_grad(w, w, out, ws)
    assert cb.rel_l2(out, oracle.grad(ow, ow)) < 2e-5
    bt.betty_grad(w, lam, out, ws)
    assert cb.rel_l2(out, oracle.grad(ow, olam)) < 1e-6
    bt.betty_grad(lam, w, out, ws)
    assert cb.rel_l2(out, oracle.grad(olam, ow)) < 2e-5
    bt.betty_grad(lam, lam, out, ws)
    assert torch.all(out == 0)
    u = si.normal_f32(9, 3, (d,))
    bt.betty_hvp(w, cb.dev(u), out, ws)
    assert cb.rel_l2(out, oracle.hvp(ow, u)) < 2e-5
    bt.betty_mixed_vjp(w, lam, cb.dev(u), out, ws)
    assert cb.rel_l2(out, oracle.mixed_vjp(ow, olam, u)) < 1e-6
    bt.betty_lower_step(w, 3, ws)
    oracle.lower_step(ow, 3)
    assert cb.rel_l2(w.params, ow.params) < 2e-5
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


@pytest.mark.parametrize("n,d,nv,steps,K", [(1024, 64, 256, 100, 10), (2051, 4096, 513, 20, 20),
                                             (513, 1028, 64, 10, 7)])
def test_hypergradients_match_oracle(bt, n, d, nv, steps, K):
    from tests import cuda_build as cb
    inp = si.config1() if (n, d) == (1024, 64) else si.logreg_bilevel(si.BASE_SEED + 2, n, d, nv)
    (w, lam), (ow, olam) = _pair(inp)
    ws = bt.Workspace([w, lam])
    bt.betty_lower_step(w, steps, ws)
    oracle.lower_step(ow, steps)
    assert cb.rel_l2(w.params, ow.params) < TOL
    out = _vec(d)
    bt.betty_hypergrad_neumann(w, lam, lam, K, 0.01, out, ws)
    assert cb.rel_l2(out, oracle.hypergrad_neumann(ow, olam, olam, K, 0.01)) < TOL
    bt.betty_hypergrad_cg(w, lam, lam, K, 0.0, out, ws)
    info = {}
    ref = oracle.hypergrad_cg(ow, olam, olam, K, 0.0, info=info)
    assert cb.rel_l2(out, ref) < TOL
    st, iters = bt.betty_poll_status(ws)
    assert st == bt.BETTY_OK and iters == info["iters"] == K          # integer work: exact
    bt.betty_hypergrad_fd(w, lam, lam, 0.01, 1.0, out, ws)
    assert cb.rel_l2(out, oracle.hypergrad_fd(ow, olam, olam, 0.01, 1.0)) < TOL
    # chain call on the one-edge path gives the Jacobian term alone (direct gradient is zero here)
    bt.betty_chain_levels([w, lam], [1, 0], [bt.MethodCfg(bt.BETTY_CG, K=K)], None, out, False, ws)
    assert cb.rel_l2(out, ref) < TOL


@pytest.mark.parametrize("n,d,nv", [(5, 8, 3), (1000, 50, 77), (777, 256, 100), (64, 33, 9), (2048, 128, 512),
                                    (999, 64, 77), (200, 256, 40), (300, 16, 10), (40, 32, 3), (1025, 64, 256),
                                    (500, 128, 40), (1000, 128, 64), (3000, 32, 100)])
def test_on_chip_whole_loop_kernel_matches_oracle(bt, n, d, nv):
    """Problems that fit a cluster's shared memory run each loop (all lower steps; a whole
    hypergradient) in one launch; ragged row counts, CTAs without rows and odd widths included.
    Power-of-two widths with few enough rows per CTA keep the rows in registers (the second line of
    cases, and the first one); the others, and 1025 x 64 with its 129 rows per CTA, in shared memory.
    The lower steps hold 64, 32 or 16 columns of a row per thread (widths 64 and 128; 32 and 256; 16), the
    hypergradient modes 8."""
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(900 + n + d, n, d, nv)
    inp.lam = (np.abs(si.normal_f32(11, 2, (d,))) * 0.05 + 0.01).astype(np.float32)
    (w, lam), (ow, olam) = _pair(inp)
    ws = bt.Workspace([w, lam])
    l0 = bt.betty_kernel_launches()
    bt.betty_lower_step(w, 30, ws)
    assert bt.betty_kernel_launches() - l0 == 1
    oracle.lower_step(ow, 30)
    assert cb.rel_l2(w.params, ow.params) < TOL
    out = _vec(d)
    for name, call, ref in [
        ("neumann", lambda: bt.betty_hypergrad_neumann(w, lam, lam, 7, 0.05, out, ws),
         lambda: oracle.hypergrad_neumann(ow, olam, olam, 7, 0.05)),
        ("cg", lambda: bt.betty_hypergrad_cg(w, lam, lam, min(d, 6), 0.0, out, ws),
         lambda: oracle.hypergrad_cg(ow, olam, olam, min(d, 6), 0.0)),
        ("fd", lambda: bt.betty_hypergrad_fd(w, lam, lam, 0.01, 0.5, out, ws),
         lambda: oracle.hypergrad_fd(ow, olam, olam, 0.01, 0.5)),
    ]:
        l0 = bt.betty_kernel_launches()
        call()
        assert bt.betty_kernel_launches() - l0 == 1, name
        assert cb.rel_l2(out, ref()) < TOL, name
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


@pytest.mark.parametrize("n,d,nv", [(1024, 64, 256), (999, 50, 77)])
def test_on_chip_kernel_is_bitwise_repeatable(bt, n, d, nv):
    """Every CTA of the cluster adds the same column sums in the same order, so two runs from the
    same state give the same bits (register form and shared-memory form)."""
    inp = si.logreg_bilevel(4242, n, d, nv)
    outs = []
    for _ in range(2):
        (w, lam), _o = _pair(inp)
        ws = bt.Workspace([w, lam], extra_bytes=41 * (d + 64) * 4)
        bt.betty_lower_step(w, 25, ws)
        a, b, c = _vec(d), _vec(d), _vec(d)
        bt.betty_hypergrad_cg(w, lam, lam, 5, 0.0, a, ws)
        bt.betty_hypergrad_neumann(w, lam, lam, 5, 0.05, b, ws)
        bt.betty_hypergrad_itd(w, lam, lam, 40, c, ws)
        outs.append((w.params.clone(), a, b, c))
    for x, y in zip(*outs):
        assert torch.equal(x, y)


def test_cg_early_stop_counts_iterations_like_the_oracle(bt):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(5, 400, 16, 100)
    (w, lam), (ow, olam) = _pair(inp)
    ws = bt.Workspace([w, lam])
    bt.betty_lower_step(w, 50, ws); oracle.lower_step(ow, 50)
    out = _vec(16)
    bt.betty_hypergrad_cg(w, lam, lam, 64, 1e-3, out, ws)
    info = {}
    ref = oracle.hypergrad_cg(ow, olam, olam, 64, 1e-3, info=info)
    st, iters = bt.betty_poll_status(ws)
    assert st == bt.BETTY_OK and iters == info["iters"] and iters < 64
    assert cb.rel_l2(out, ref) < TOL


def test_quadratic_family_and_cg_breakdown_status(bt):
    from tests import cuda_build as cb
    rng = np.random.default_rng(11)
    A, b = rng.standard_normal((150, 24)).astype(np.float32), rng.standard_normal(150).astype(np.float32)
    Av, bv = rng.standard_normal((90, 24)).astype(np.float32), rng.standard_normal(90).astype(np.float32)
    lamv = (rng.random(24) + 0.1).astype(np.float32)
    w0 = (rng.standard_normal(24) * 0.1).astype(np.float32)
    lo, up = cb.quadratic_levels(A, b, lamv, Av, bv, w0)
    olo, oup = ob.quadratic_levels(A, b, lamv, Av, bv, w0)
    ws = bt.Workspace([lo, up])
    out = _vec(24)
    bt.betty_hypergrad_cg(lo, up, up, 24, 0.0, out, ws)
    assert cb.rel_l2(out, oracle.hypergrad_cg(olo, oup, oup, 24, 0.0)) < 1e-3   # 24 fp32 CG steps
    bt.betty_hypergrad_neumann(lo, up, up, 8, 1e-3, out, ws)
    assert cb.rel_l2(out, oracle.hypergrad_neumann(olo, oup, oup, 8, 1e-3)) < TOL
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
    # an indefinite Hessian: the oracle reports breakdown at iteration 0, the device must too
    lam_bad = lamv.copy(); lam_bad[:] = -500.0
    lo2, up2 = cb.quadratic_levels(A, b, lam_bad, Av, bv, w0)
    olo2, oup2 = ob.quadratic_levels(A, b, lam_bad, Av, bv, w0)
    info = {}
    ref = oracle.hypergrad_cg(olo2, oup2, oup2, 5, 0.0, info=info)
    assert info["status"] == "breakdown"
    ws2 = bt.Workspace([lo2, up2])
    bt.betty_hypergrad_cg(lo2, up2, up2, 5, 0.0, out, ws2)
    st, iters = bt.betty_poll_status(ws2, raise_on_error=False)
    assert st == bt.BETTY_ERR_BREAKDOWN and iters == info["iters"]
    assert cb.rel_l2(out, ref) < TOL or np.linalg.norm(ref) == 0
    bt.betty_reset_status(ws2)
    assert bt.betty_poll_status(ws2)[0] == bt.BETTY_OK


def test_empty_batch_and_argument_errors(bt):
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(3, 16, 8, 4)
    (w, lam), _ = _pair(inp)
    ws = bt.Workspace([w, lam])
    out = _vec(8)
    empty = bt.Level(bt.LOSS_LOGREG_WD, bt.PARAM_VECTOR, cb.dev(inp.w0 + 1), X=torch.empty(0, 8, dtype=torch.float32, device="cuda"),
                     y=torch.empty(0, dtype=torch.float32, device="cuda"))
    empty.set_constraints([lam])
    bt.betty_grad(empty, empty, out, ws)            # only the weight-decay term is left
    assert cb.rel_l2(out, (inp.lam * (inp.w0 + 1)).astype(np.float64)) < 1e-6
    with pytest.raises(bt.BettyError) as e:
        bt.betty_hypergrad_cg(w, lam, w, 3, 0.0, out, ws)      # wrt must be a constraint of lower
    assert e.value.status == bt.BETTY_ERR_INVALID_ARG
    bad = bt.Level(bt.LOSS_LOGREG_WD, bt.PARAM_VECTOR, cb.dev(np.zeros(7, np.float32)), X=w.X, y=w.y)
    bad.set_constraints([lam])
    with pytest.raises(bt.BettyError) as e:
        bt.betty_grad(bad, bad, out, ws)
    assert e.value.status == bt.BETTY_ERR_SHAPE
    small = bt.Workspace([w, lam]); small.nbytes = 256
    with pytest.raises(bt.BettyError) as e:
        bt.betty_hvp(w, out, out, small)
    assert e.value.status == bt.BETTY_ERR_WORKSPACE


def test_misaligned_vectors_are_rejected_and_chain_start_vectors_match_oracle(bt):
    """Flat vector arguments must start on a 16-byte boundary: a start vector, a direction or an output
    one float off is refused with BETTY_ERR_ALIGNMENT by every entry point (the single-pass kernel and
    the curvature it leaves for the later HVPs of a solve rely on it).  With an aligned caller-supplied
    start vector the chain call agrees with the oracle for both solvers, on a full-width level (single
    pass, cached curvature) and on a width that takes the two-pass kernels (nothing cached)."""
    from tests import cuda_build as cb
    for n, d in [(1500, 4096), (400, 130)]:
        inp = si.logreg_bilevel(21, n, d, 32)
        (w, lam), (ow, olam) = _pair(inp)
        ws = bt.Workspace([w, lam])
        bt.betty_lower_step(w, 3, ws)
        oracle.lower_step(ow, 3)
        v = si.normal_f32(23, 5, (d,))
        buf = torch.zeros(d + 4, dtype=torch.float32, device="cuda")
        buf[1:d + 1] = cb.dev(v)
        out = _vec(d)
        for cfg, ocfg in [(bt.MethodCfg(bt.BETTY_NEUMANN, K=4, alpha=0.05), dict(method="neumann", K=4, alpha=0.05)),
                          (bt.MethodCfg(bt.BETTY_CG, K=4), dict(method="cg", K=4, tol=0.0))]:
            with pytest.raises(bt.BettyError) as e:
                bt.betty_chain_levels([w, lam], [1, 0], [cfg], buf[1:d + 1], out, False, ws)
            assert e.value.status == bt.BETTY_ERR_ALIGNMENT
            with pytest.raises(bt.BettyError) as e:
                bt.betty_chain_levels([w, lam], [1, 0], [cfg], cb.dev(v), buf[1:d + 1], False, ws)
            assert e.value.status == bt.BETTY_ERR_ALIGNMENT
            bt.betty_chain_levels([w, lam], [1, 0], [cfg], cb.dev(v), out, False, ws)
            assert cb.rel_l2(out, oracle.chain_levels([ow, olam], [1, 0], [ocfg], v_in=v)) < TOL
        for call in (lambda: bt.betty_grad(w, w, buf[1:d + 1], ws),
                     lambda: bt.betty_mixed_vjp(w, lam, buf[1:d + 1], out, ws),
                     lambda: bt.betty_hvp(w, buf[1:d + 1], out, ws),
                     lambda: bt.betty_hypergrad_cg(w, lam, lam, 2, 0.0, buf[1:d + 1], ws)):
            with pytest.raises(bt.BettyError) as e:
                call()
            assert e.value.status == bt.BETTY_ERR_ALIGNMENT
        assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_repeated_calls_are_bitwise_identical(bt):
    inp = si.logreg_bilevel(8, 3000, 4096, 64)
    (w, lam), _ = _pair(inp)
    ws = bt.Workspace([w, lam])
    u = torch.randn(4096, dtype=torch.float32, device="cuda")
    a, b = _vec(4096), _vec(4096)
    bt.betty_hvp(w, u, a, ws)
    bt.betty_hvp(w, u, b, ws)
    assert torch.equal(a, b)


@pytest.mark.parametrize("n,d,nv,T,on_chip", [
    (1024, 64, 256, 100, True),      # the small configuration: rows in registers, iterates in shared memory
    (999, 50, 77, 20, True),         # odd width: rows in shared memory
    (2048, 128, 256, 10, True),      # 256 rows per CTA: shared memory
    (300, 16, 10, 1, True),          # a single unrolled step
    (1024, 64, 256, 500, False),     # 500 stored iterates do not fit beside the rows: general path
    (700, 1028, 90, 12, False),      # too wide for the on-chip kernel
])
def test_itd_hypergradient_matches_oracle(bt, n, d, nv, T, on_chip):
    """ITD-RMAD: reverse sweep through the stored unrolled steps -- in one launch where the rows and
    the iterates fit on chip, else step by step with the iterates in the workspace."""
    from tests import cuda_build as cb
    inp = si.config1() if (n, d) == (1024, 64) else si.logreg_bilevel(77, n, d, nv)
    (w, lam), (ow, olam) = _pair(inp)
    ws = bt.Workspace([w, lam], extra_bytes=(T + 1) * (d + 64) * 4)
    out = _vec(d)
    l0 = bt.betty_kernel_launches()
    bt.betty_hypergrad_itd(w, lam, lam, T, out, ws)
    assert (bt.betty_kernel_launches() - l0 == 1) == on_chip
    ref = oracle.hypergrad_itd(ow, olam, olam, T)
    assert cb.rel_l2(w.params, ow.params) < TOL
    assert cb.rel_l2(out, ref) < TOL
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
