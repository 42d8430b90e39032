"""Device-side conditions reach the host through the status block, and the context stays usable:
an expired bounded wait (made on purpose with a barrier nothing arrives at), a non-finite value met
by a reduction, and clearing the block."""
import numpy as np
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_context_survives():
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(3, 64, 16, 8)
    w, lam = cb.logreg_levels(inp)
    ws = bt.Workspace([w, lam])
    bt.betty_selftest_wait_timeout(ws)
    st, _ = bt.betty_poll_status(ws, raise_on_error=False)
    assert st == bt.BETTY_ERR_TIMEOUT
    bt.betty_reset_status(ws)
    out = torch.empty(16, dtype=torch.float32, device="cuda")
    bt.betty_grad(w, w, out, ws)                       # ordinary work still runs afterwards
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK and torch.isfinite(out).all()


def test_non_finite_input_is_flagged_by_the_cg_reductions():
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(4, 3000, 512, 64)          # wide enough for the streaming path
    inp.Xv[5, 7] = np.nan
    w, lam = cb.logreg_levels(inp)
    ws = bt.Workspace([w, lam])
    out = torch.empty(512, dtype=torch.float32, device="cuda")
    bt.betty_hypergrad_cg(w, lam, lam, 4, 0.0, out, ws)
    st, iters = bt.betty_poll_status(ws, raise_on_error=False)
    assert st == bt.BETTY_ERR_NONFINITE and iters == 0
    with pytest.raises(bt.BettyError):
        bt.betty_poll_status(ws)
