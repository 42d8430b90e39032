"""The allocation-free logistic HVP entry point.

Some users of the library cannot hand it a workspace: their process has given all device memory
to another allocator, or must not trigger the device-wide synchronisation that an allocation or
a free can cause.  `betty_hvp_logreg_static` serves them from a fixed scratch array built into
the library.  These tests call it through the C ABI twice in a row (the scratch keeps the first
call's contents, so the second call checks that stale data does no harm) and compare each result
with the fp64 oracle at the tolerance of the other logistic parity tests, and bit for bit with
`betty_hvp` on the same inputs (same kernels, same launch shape, same summation order).  The file
name keeps it last in collection order."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu
TOL = 2e-5


def _setup(n, d, seed):
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(seed, n, d, 8)
    inp.w0 = si.normal_f32(seed, 91, (d,)) * np.float32(0.5 / np.sqrt(d))
    inp.lam = (np.abs(si.normal_f32(seed, 92, (d,))) * 0.05 + 0.01).astype(np.float32)
    w, lam = cb.logreg_levels(inp)
    return bt, cb, w, lam, bt.Workspace([w, lam])


@pytest.mark.parametrize("n,d", [(3001, 4096), (1500, 2048), (777, 1024), (50, 64)])
def test_static_scratch_hvp_matches_oracle_and_workspace_hvp_on_two_calls_in_a_row(n, d):
    import oracle
    from tests import oracle_build as ob
    bt, cb, w, lam, ws = _setup(n, d, 500 + d)
    inp = si.logreg_bilevel(500 + d, n, d, 8)
    inp.w0 = w.params.cpu().numpy()
    inp.lam = lam.params.cpu().numpy()
    ow, _ = ob.logreg_levels(inp)
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    for call in range(2):
        u_host = si.normal_f32(600 + call, 93, (d,))
        u = cb.dev(u_host)
        ref = torch.empty(d, dtype=torch.float32, device="cuda")
        got = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
        bt.betty_hvp(w, u, ref, ws)
        bt.betty_hvp_logreg_static(w.X, w.params, lam.params, u, got, status)
        torch.cuda.synchronize()
        assert int(status.item()) == bt.BETTY_OK
        assert cb.rel_l2(got, oracle.hvp(ow, u_host)) < TOL
        assert torch.equal(got, ref)
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_static_scratch_hvp_of_an_empty_matrix_is_the_weight_decay_term():
    """n = 0: the data term vanishes, H u = lam . u exactly."""
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    d = 256
    X = torch.empty(0, d, dtype=torch.float32, device="cuda")
    w = cb.dev(si.normal_f32(7, 1, (d,)))
    lam = cb.dev(np.abs(si.normal_f32(7, 2, (d,))))
    u = cb.dev(si.normal_f32(7, 3, (d,)))
    got = torch.full((d,), float("nan"), dtype=torch.float32, device="cuda")
    status = torch.full((1,), -1, dtype=torch.int32, device="cuda")
    bt.betty_hvp_logreg_static(X, w, lam, u, got, status)
    torch.cuda.synchronize()
    assert int(status.item()) == bt.BETTY_OK
    assert torch.equal(got, lam * u)


def test_static_scratch_hvp_rejects_what_it_cannot_serve():
    import paper_2207_02849_b200 as bt
    # beyond the fixed scratch
    d = 4100
    X = torch.zeros(4, d, dtype=torch.float32, device="cuda")
    v = torch.zeros(d, dtype=torch.float32, device="cuda")
    with pytest.raises(bt.BettyError) as e:
        bt.betty_hvp_logreg_static(X, v, v, v, torch.empty_like(v))
    assert e.value.status == bt.BETTY_ERR_CAPACITY
    assert "scratch" in bt.betty_status_string(bt.BETTY_ERR_CAPACITY)
    # a width the single-pass kernel does not take
    d = 30
    X = torch.zeros(4, d, dtype=torch.float32, device="cuda")
    v = torch.zeros(d, dtype=torch.float32, device="cuda")
    with pytest.raises(bt.BettyError) as e:
        bt.betty_hvp_logreg_static(X, v, v, v, torch.empty_like(v))
    assert e.value.status == bt.BETTY_ERR_UNSUPPORTED
    # a direction that does not start on a 16-byte boundary
    d = 64
    X = torch.zeros(4, d, dtype=torch.float32, device="cuda")
    v = torch.zeros(d, dtype=torch.float32, device="cuda")
    shifted = torch.zeros(d + 1, dtype=torch.float32, device="cuda")[1:]
    with pytest.raises(bt.BettyError) as e:
        bt.betty_hvp_logreg_static(X, v, v, shifted, torch.empty_like(v))
    assert e.value.status == bt.BETTY_ERR_ALIGNMENT
    with pytest.raises(bt.BettyError) as e:
        bt.betty_hvp_logreg_static(X, v, v, v, shifted)
    assert e.value.status == bt.BETTY_ERR_ALIGNMENT
