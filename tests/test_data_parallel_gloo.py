"""Row-sharded data-parallel evaluation on two gloo ranks (CPU): rows partitioned by
`data_parallel.shard_rows`, every derivative weighted by the rank's share of the rows and summed over the
ranks with the package's all-reduce, parameters and solver state replicated.  The sharded results must equal
the one-rank oracle on the whole batch: the weights sum to one, every row is held by exactly one rank, and
the terms that do not depend on the data (weight decay) are counted once."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _slice_batch(b, lo, hi):
    return type(b)(X=b.X[lo:hi], y=b.y[lo:hi], y_clean=b.y_clean[lo:hi], clean=b.clean[lo:hi])


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import copy
    import oracle
    import synth_inputs as si
    from oracle import problems as ob
    from paper_2207_02849_b200 import data_parallel as dp
    from tests.dp_oracle import ShardedOracle
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)

    def reduce(vec):
        t = torch.from_numpy(vec)
        dp.allreduce_sum_(t)
        return t.numpy()

    res = {}
    # ---- logistic weight-decay pair, a row count that does not divide evenly
    inp = si.logreg_bilevel(5, 1027, 32, 255)
    full_w, full_lam = ob.logreg_levels(inp)
    sh = copy.copy(inp)
    lo, hi = dp.shard_rows(1027, rank, world)
    lov, hiv = dp.shard_rows(255, rank, world)
    sh.X, sh.y, sh.Xv, sh.yv = inp.X[lo:hi], inp.y[lo:hi], inp.Xv[lov:hiv], inp.yv[lov:hiv]
    w, lam = ob.logreg_levels(sh)
    so = ShardedOracle({id(w): dp.row_weight(1027, rank, world), id(lam): dp.row_weight(255, rank, world)}, reduce)
    so.lower_step(w, 20)
    oracle.lower_step(full_w, 20)
    res["logreg_w"] = (w.params, full_w.params)
    res["logreg_cg"] = (so.hypergrad(w, lam, lam, "cg", K=10), oracle.hypergrad_cg(full_w, full_lam, full_lam, 10, 0.0))
    res["logreg_neumann"] = (so.hypergrad(w, lam, lam, "neumann", K=10, alpha=0.01),
                             oracle.hypergrad_neumann(full_w, full_lam, full_lam, 10, 0.01))
    res["logreg_fd"] = (so.hypergrad(w, lam, lam, "fd"), oracle.hypergrad_fd(full_w, full_lam, full_lam, 0.01, 1.0))
    # ---- data reweighting with an MLP classifier (unrounded arithmetic: the identity is exact)
    rinp = si.reweight_bilevel(9, (12, 16, 5), 37, 0.4, activation="gelu")
    rinp.theta = (si.weightnet_init(9, 200) * np.float32(3.0)).astype(np.float32)
    fw, fth = ob.reweight_levels(rinp, bf16=False)
    rs = copy.copy(rinp)
    lo, hi = dp.shard_rows(37, rank, world)
    rs.train, rs.val = _slice_batch(rinp.train, lo, hi), _slice_batch(rinp.val, lo, hi)
    sw, sth = ob.reweight_levels(rs, bf16=False)
    wgt = dp.row_weight(37, rank, world)
    so2 = ShardedOracle({id(sw): wgt, id(sth): wgt}, reduce)
    so2.lower_step(sw, 2)
    oracle.lower_step(fw, 2)
    res["mlp_w"] = (sw.params, fw.params)
    res["mlp_neumann"] = (so2.hypergrad(sw, sth, sth, "neumann", K=3, alpha=0.05),
                          oracle.hypergrad_neumann(fw, fth, fth, 3, 0.05))
    res["mlp_fd"] = (so2.hypergrad(sw, sth, sth, "fd"), oracle.hypergrad_fd(fw, fth, fth, 0.01, 1.0))
    errs = {k: float(np.linalg.norm(a - b) / np.linalg.norm(b)) for k, (a, b) in res.items()}
    out.put((rank, errs, [dp.shard_rows(1027, r, world) for r in range(world)]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_sharded_ranks_reproduce_the_one_rank_oracle():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=300) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, errs, shards in res:
        assert shards == [(0, 513), (513, 1027)]
        for name, e in errs.items():
            assert e < 1e-4, (rank, name, e)            # the stated bound; the identity holds to rounding
            assert e < 1e-10, (rank, name, e)


def test_row_shards_partition_the_rows_and_weights_sum_to_one():
    sys.path.insert(0, ROOT)
    from paper_2207_02849_b200 import data_parallel as dp
    for n in (0, 1, 7, 1024, 262144, 1027):
        for world in (1, 2, 3, 8):
            rows = [dp.shard_rows(n, r, world) for r in range(world)]
            assert rows[0][0] == 0 and rows[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(rows, rows[1:]))
            sizes = [hi - lo for lo, hi in rows]
            assert max(sizes) - min(sizes) <= 1
            assert abs(sum(dp.row_weight(n, r, world) for r in range(world)) - 1.0) < 1e-12
