"""The library's calls only enqueue work and keep solver scalars on the device, so a whole
hypergradient step can be captured into a CUDA graph and replayed: the replay must reproduce the
directly launched result bit for bit."""
import pytest
import torch

import synth_inputs as si

pytestmark = pytest.mark.gpu


def _capture(step):
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    return g


def test_logistic_step_replays_identically():
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.config1()
    w, lam = cb.logreg_levels(inp)
    w0 = w.params.clone()
    ws = bt.Workspace([w, lam])
    out = torch.empty(64, dtype=torch.float32, device="cuda")

    def step():
        w.params.copy_(w0)
        bt.betty_lower_step(w, inp.lower_steps, ws)
        bt.betty_hypergrad_cg(w, lam, lam, inp.K, 0.0, out, ws)

    step()
    torch.cuda.synchronize()
    direct = out.clone()
    g = _capture(step)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, direct)
    assert bt.betty_poll_status(ws) == (bt.BETTY_OK, inp.K)


def test_reweighting_step_replays_identically():
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.reweight_bilevel(61, (64, 128, 10), 128, 0.4)
    w, th = cb.reweight_levels(inp)
    w0 = w.params.clone()
    ws = bt.Workspace([w, th])
    out = torch.empty(si.WEIGHTNET_PARAMS, dtype=torch.float32, device="cuda")

    def step():
        w.params.copy_(w0)
        bt.betty_lower_step(w, 1, ws)
        bt.betty_hypergrad_neumann(w, th, th, 3, 0.01, out, ws)

    step()
    torch.cuda.synchronize()
    direct = out.clone()
    g = _capture(step)
    out.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, direct)
