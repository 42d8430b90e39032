"""Parity at the full sizes the benchmark times: configuration 2 (262144 x 4096 logistic, 20 lower
steps, CG K = 20) and configuration 5 (8 x 4096 GELU MLP + 1000-way head, batch 1024, 4 lower steps,
Neumann K = 3), in the launch configuration bench.py uses, against the fp64 oracle on the same seeded
inputs.  These two tests take a few minutes of host time for the oracle."""
import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests import oracle_build as ob

pytestmark = pytest.mark.gpu


def test_config2_full_size_hypergradient():
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.config2()
    w, lam = cb.logreg_levels(inp)
    ws = bt.Workspace([w, lam])
    bt.betty_lower_step(w, inp.lower_steps, ws)
    out = torch.empty(4096, dtype=torch.float32, device="cuda")
    bt.betty_hypergrad_cg(w, lam, lam, inp.K, 0.0, out, ws)
    st, iters = bt.betty_poll_status(ws)
    ow, olam = ob.logreg_levels(inp)
    oracle.lower_step(ow, inp.lower_steps)
    info = {}
    ref = oracle.hypergrad_cg(ow, olam, olam, inp.K, 0.0, info=info)
    assert st == bt.BETTY_OK and iters == info["iters"] == inp.K
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    assert cb.rel_l2(out, ref) < 1e-4


def test_config5_full_size_hypergradient(parity_record):
    """Held to 2e-2 against the oracle under both readings of a mixed-precision level (bf16 operands in
    every product; matrices rounded only), for the parameter update of the four lower steps and for the
    hypergradient (whole vector and largest single component)."""
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.config5()
    w, th = cb.reweight_levels(inp)
    ws = bt.Workspace([w, th])
    bt.betty_lower_step(w, inp.lower_steps, ws)
    out = torch.empty(si.WEIGHTNET_PARAMS, dtype=torch.float32, device="cuda")
    bt.betty_hypergrad_neumann(w, th, th, inp.K, inp.alpha, out, ws)
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
    got_w = w.params.double().cpu().numpy()
    w0 = inp.w.astype(np.float64)
    for quant in ("operands", "weights"):
        ow, oth = ob.reweight_levels(inp, quant=quant)
        oracle.lower_step(ow, inp.lower_steps)
        ref = oracle.hypergrad_neumann(ow, oth, oth, inp.K, inp.alpha)
        assert parity_record(f"config5/{quant}/lower_update", cb.rel_l2(got_w - w0, ow.params - w0)) < 2e-2
        assert parity_record(f"config5/{quant}/neumann", cb.rel_l2(out, ref)) < 2e-2
        assert parity_record(f"config5/{quant}/neumann_max", cb.rel_max(out, ref)) < 2e-2
