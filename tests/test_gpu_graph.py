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


def test_one_stream_order_and_two_stream_order_give_the_same_bits():
    """The MLP families fork weight-gradient work to a second stream that each host thread gets at its
    first call outside a capture.  A thread whose first call is captured has none and launches
    everything in program order on the captured stream; both orders must give identical bits."""
    import threading
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    inp = si.reweight_bilevel(67, (72, 136, 64, 10), 200, 0.4, activation="gelu")
    w, th = cb.reweight_levels(inp)
    w0 = w.params.clone()
    ws = bt.Workspace([w, th])
    out = torch.empty(si.WEIGHTNET_PARAMS, dtype=torch.float32, device="cuda")

    def step():
        w.params.copy_(w0)
        bt.betty_lower_step(w, 2, ws)
        bt.betty_hypergrad_neumann(w, th, th, 3, 0.01, out, ws)

    step()          # this thread has made calls before: two streams
    step()
    torch.cuda.synchronize()
    direct_out, direct_w = out.clone(), w.params.clone()
    got = {}

    def worker():
        try:
            torch.cuda.set_device(0)
            s = torch.cuda.Stream()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s, capture_error_mode="thread_local"):
                step()
            out.zero_()
            torch.cuda.synchronize()
            g.replay()
            torch.cuda.synchronize()
            got["out"], got["w"] = out.clone(), w.params.clone()
        except Exception as e:      # surfaces in the asserting thread
            got["error"] = e

    t = threading.Thread(target=worker)
    t.start()
    t.join()
    assert "error" not in got, got.get("error")
    assert torch.equal(got["out"], direct_out)
    assert torch.equal(got["w"], direct_w)
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


@pytest.mark.parametrize("problem", ["fd", "neumann", "three_levels"])
def test_two_stream_steps_repeat_bit_for_bit(problem):
    """The calls fork independent work to a second stream (weight-gradient products beside the delta
    chain, the two finite-difference passes, a lower level's base pass beside the upper gradients).  A
    missing dependency between the streams would show as results that change from replay to replay:
    30 replays of one captured step must all give the bits of the directly launched step."""
    import paper_2207_02849_b200 as bt
    from tests import cuda_build as cb
    if problem == "three_levels":
        inp = si.three_level(83, (48, 72, 40, 10), 160, 0.3, activation="gelu")
        P = cb.three_levels(inp)
        w0 = P[0].params.clone()
        ws = bt.Workspace(list(P))
        out = torch.empty(inp.lam.size, dtype=torch.float32, device="cuda")
        cfg = bt.MethodCfg(bt.BETTY_NEUMANN, K=3, alpha=0.01)

        def step():
            P[0].params.copy_(w0)
            bt.betty_lower_step(P[0], 1, ws)
            bt.betty_hypergrad_graph(list(P), [(2, 0), (1, 0)], [(0, 1), (0, 2), (1, 2)], 2, [cfg] * 3, out, ws)
    else:
        inp = si.reweight_bilevel(79, (72, 136, 64, 10), 200, 0.4, activation="gelu")
        w, th = cb.reweight_levels(inp)
        w0 = w.params.clone()
        ws = bt.Workspace([w, th])
        out = torch.empty(si.WEIGHTNET_PARAMS, dtype=torch.float32, device="cuda")

        def step():
            w.params.copy_(w0)
            bt.betty_lower_step(w, 2, ws)
            if problem == "fd":
                bt.betty_hypergrad_fd(w, th, th, 0.01, 1.0, out, ws)
            else:
                bt.betty_hypergrad_neumann(w, th, th, 3, 0.01, out, ws)

    step()
    torch.cuda.synchronize()
    direct = out.clone()
    g = _capture(step)
    for _ in range(30):
        out.zero_()
        g.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, direct)
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
