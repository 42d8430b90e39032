"""The data-parallel hook of the library on a GPU: levels that hold a share of the rows, with the
all-reduce supplied by the caller.

One GPU is available to these tests, so the two ranks of the second test are two host threads, each with its
own levels, workspace and stream on that GPU; their all-reduce meets at a host-side barrier after each thread
has synchronised its own stream (no kernel ever waits for another), adds the two buffers and hands the sum
back to both.  Every rank's result must equal the one-rank oracle on the whole batch."""
import copy
import threading

import numpy as np
import pytest
import torch

import oracle
import synth_inputs as si
from tests import oracle_build as ob

pytestmark = pytest.mark.gpu


def _slice_batch(b, lo, hi):
    return type(b)(X=b.X[lo:hi], y=b.y[lo:hi], y_clean=b.y_clean[lo:hi], clean=b.clean[lo:hi])


def test_single_rank_with_the_hook_attached_matches_the_oracle():
    import paper_2207_02849_b200 as bt
    from paper_2207_02849_b200 import data_parallel as dp
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(5, 1027, 32, 255)
    w, lam = cb.logreg_levels(inp)
    ow, olam = ob.logreg_levels(inp)
    ar = dp.DeviceAllReduce()
    dp.shard_level(w, 1027, 0, 1, ar)
    dp.shard_level(lam, 255, 0, 1, ar)
    ws = bt.Workspace([w, lam])
    bt.betty_lower_step(w, 20, ws)
    oracle.lower_step(ow, 20)
    assert cb.rel_l2(w.params, ow.params) < 1e-4
    out = torch.empty(32, device="cuda")
    bt.betty_hypergrad_cg(w, lam, lam, 10, 0.0, out, ws)
    assert cb.rel_l2(out, oracle.hypergrad_cg(ow, olam, olam, 10, 0.0)) < 1e-4
    assert ar.calls == 20 + 2 + 10 + 1                 # steps, two direct gradients, ten products, the mixed product
    with pytest.raises(bt.BettyError) as e:
        bt.betty_hypergrad_itd(w, lam, lam, 3, out, ws)
    assert e.value.status == bt.BETTY_ERR_UNSUPPORTED
    assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK


def test_the_nccl_exchange_runs_on_the_library_buffers():
    """A one-rank NCCL job on this GPU: the collective is issued on the raw device buffers the library hands to
    the callback, on the stream the library is enqueuing on (a sum over one rank changes nothing, so the results
    must still equal the oracle's)."""
    import os
    import socket
    import torch.distributed as dist
    import paper_2207_02849_b200 as bt
    from paper_2207_02849_b200 import data_parallel as dp
    from tests import cuda_build as cb
    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        inp = si.logreg_bilevel(7, 1500, 4096, 300)
        w, lam = cb.logreg_levels(inp)
        ow, olam = ob.logreg_levels(inp)
        ar = dp.DeviceAllReduce(single_rank_too=True)
        dp.shard_level(w, 1500, 0, 1, ar)
        dp.shard_level(lam, 300, 0, 1, ar)
        ws = bt.Workspace([w, lam])
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):                      # not the default stream: the exchange must follow the library's
            bt.betty_lower_step(w, 3, ws)
            out = torch.empty(4096, device="cuda")
            bt.betty_hypergrad_cg(w, lam, lam, 5, 0.0, out, ws)
            side.synchronize()
        oracle.lower_step(ow, 3)
        assert cb.rel_l2(w.params, ow.params) < 1e-4
        assert cb.rel_l2(out, oracle.hypergrad_cg(ow, olam, olam, 5, 0.0)) < 1e-4
        assert ar.calls == 3 + 2 + 5 + 1
        assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
    finally:
        dist.destroy_process_group()


class _TwoThreadAllReduce:
    """Sum over two host threads that share one GPU (see the module docstring)."""

    def __init__(self):
        self.barrier = threading.Barrier(2, timeout=120)
        self.slots = [None, None]
        self.total = None

    def for_rank(self, rank):
        def allreduce(ptr, count, stream):
            from paper_2207_02849_b200.data_parallel import _RawDeviceBuffer
            t = torch.as_tensor(_RawDeviceBuffer(ptr, count), device="cuda")
            torch.cuda.ExternalStream(stream).synchronize() if stream else torch.cuda.synchronize()
            self.slots[rank] = t
            self.barrier.wait()
            if rank == 0:
                self.total = (self.slots[0] + self.slots[1])
                torch.cuda.synchronize()
            self.barrier.wait()
            t.copy_(self.total)
            torch.cuda.synchronize()
            self.barrier.wait()
        return allreduce


def _run_two_ranks(fn):
    ar = _TwoThreadAllReduce()
    results, errors = [None, None], [None, None]

    def body(rank):
        try:
            torch.cuda.set_device(0)
            with torch.cuda.stream(torch.cuda.Stream()):
                results[rank] = fn(rank, ar.for_rank(rank))
                torch.cuda.current_stream().synchronize()
        except BaseException as e:     # a failing rank breaks the barrier, which ends the other one too
            errors[rank] = e
            ar.barrier.abort()
    threads = [threading.Thread(target=body, args=(r,)) for r in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=600)
    for e in errors:
        if e is not None:
            raise e
    return results


def test_two_ranks_of_the_logistic_problem_match_the_one_rank_oracle():
    import paper_2207_02849_b200 as bt
    from paper_2207_02849_b200 import data_parallel as dp
    from tests import cuda_build as cb
    inp = si.logreg_bilevel(5, 2051, 4096, 513)          # full width: the single-pass kernel on each share
    ow, olam = ob.logreg_levels(inp)
    oracle.lower_step(ow, 5)
    refs = {"cg": oracle.hypergrad_cg(ow, olam, olam, 6, 0.0),
            "neumann": oracle.hypergrad_neumann(ow, olam, olam, 6, 0.01),
            "fd": oracle.hypergrad_fd(ow, olam, olam, 0.01, 1.0)}

    def rank_fn(rank, allreduce):
        sh = copy.copy(inp)
        lo, hi = dp.shard_rows(2051, rank, 2)
        lov, hiv = dp.shard_rows(513, rank, 2)
        sh.X, sh.y, sh.Xv, sh.yv = inp.X[lo:hi], inp.y[lo:hi], inp.Xv[lov:hiv], inp.yv[lov:hiv]
        w, lam = cb.logreg_levels(sh)
        dp.shard_level(w, 2051, rank, 2, allreduce)
        dp.shard_level(lam, 513, rank, 2, allreduce)
        ws = bt.Workspace([w, lam])
        bt.betty_lower_step(w, 5, ws)
        out = {}
        for m in ("cg", "neumann", "fd"):
            o = torch.empty(4096, device="cuda")
            if m == "cg":
                bt.betty_hypergrad_cg(w, lam, lam, 6, 0.0, o, ws)
            elif m == "neumann":
                bt.betty_hypergrad_neumann(w, lam, lam, 6, 0.01, o, ws)
            else:
                bt.betty_hypergrad_fd(w, lam, lam, 0.01, 1.0, o, ws)
            out[m] = o
        assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
        return w.params.clone(), out

    res = _run_two_ranks(rank_fn)
    for wp, out in res:
        assert cb.rel_l2(wp, ow.params) < 1e-4
        for m, ref in refs.items():
            assert cb.rel_l2(out[m], ref) < 1e-4, m
    # replicated state: both ranks hold the same bits
    assert torch.equal(res[0][0], res[1][0])
    for m in refs:
        assert torch.equal(res[0][1][m], res[1][1][m])


def test_two_ranks_of_the_reweighting_problem_match_the_one_rank_oracle():
    import paper_2207_02849_b200 as bt
    from paper_2207_02849_b200 import data_parallel as dp
    from tests import cuda_build as cb
    from tests.test_gpu_mlp import _perturb
    inp = _perturb(si.reweight_bilevel(61, (64, 96, 10), 256, 0.4, activation="gelu"), 61)
    ow, oth = ob.reweight_levels(inp)
    oracle.lower_step(ow, 2)
    refs = {"neumann": oracle.hypergrad_neumann(ow, oth, oth, 3, 0.01),
            "fd": oracle.hypergrad_fd(ow, oth, oth, 0.01, 1.0)}

    def rank_fn(rank, allreduce):
        sh = copy.copy(inp)
        lo, hi = dp.shard_rows(256, rank, 2)
        sh.train, sh.val = _slice_batch(inp.train, lo, hi), _slice_batch(inp.val, lo, hi)
        w, th = cb.reweight_levels(sh)
        dp.shard_level(w, 256, rank, 2, allreduce)
        dp.shard_level(th, 256, rank, 2, allreduce)
        ws = bt.Workspace([w, th])
        bt.betty_lower_step(w, 2, ws)
        out = {}
        for m in ("neumann", "fd"):
            o = torch.empty(si.WEIGHTNET_PARAMS, device="cuda")
            if m == "neumann":
                bt.betty_hypergrad_neumann(w, th, th, 3, 0.01, o, ws)
            else:
                bt.betty_hypergrad_fd(w, th, th, 0.01, 1.0, o, ws)
            out[m] = o
        assert bt.betty_poll_status(ws)[0] == bt.BETTY_OK
        return w.params.clone(), out

    res = _run_two_ranks(rank_fn)
    w0 = inp.w.astype(np.float64)
    for wp, out in res:
        assert cb.rel_l2(wp.double().cpu().numpy() - w0, ow.params - w0) < 2e-2
        for m, ref in refs.items():
            assert cb.rel_l2(out[m], ref) < 2e-2, m
    assert torch.equal(res[0][0], res[1][0])
