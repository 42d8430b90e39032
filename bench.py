#!/usr/bin/env python
"""Benchmark of the hypergradient hot path.

`python bench.py --gpus N --steps K --warmup W` prints ONE JSON line.  A step is one pass of the
whole hot path over one batch of synthetic input: the unrolled lower-level gradient steps, the
direct gradients of the upper cost and the best-response-Jacobian product of the configuration's
method (default workload: the bilevel logistic weight-decay problem with X of 262144 x 4096 fp32,
20 lower steps, conjugate gradient with K = 20).  Inputs are resident in device memory for
`value`; `e2e` repeats the measurement with host (pinned) inputs copied in every step and the
result read back.  `--impl reference` times the fp64 CPU oracle on a bounded sample instead.
Under torchrun (N > 1) every rank runs an independent replica on its own GPU (the path has no
exchange step); value is the aggregate, time the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "hypergradient_steps_per_sec"
UNIT = "steps/s"
# datasheet figures of the part (HGX B200: HBM3e bandwidth, dense bf16), reported beside the measured peaks
NOMINAL_HBM_GBS = 7700.0
NOMINAL_BF16_TFLOPS = 2250.0
# (key, configuration, method, timed steps) of the short runs added to the default line
PER_CONFIG_RUNS = [("config1_cg", 1, "cg", 50), ("config1_neumann", 1, "neumann", 50), ("config3_fd", 3, "fd", 30),
                   ("config3_neumann", 3, "neumann", 30), ("config4", 4, "", 30), ("config5", 5, "neumann", 10)]


def _release(w):
    """Drop a workload's device tensors (its captured graph first)."""
    for k in list(w.__dict__):
        if k not in ("inp", "name", "dtype"):
            w.__dict__.pop(k, None)
    return None


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []
        self.t0 = self.t1 = None

    def mark_begin(self):
        self.t0 = time.time()

    def mark_end(self):
        self.t1 = time.time()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        t_wait = time.time()
        while not self.lines and time.time() - t_wait < 3.0:    # nvidia-smi needs about a second for its first line
            time.sleep(0.05)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [ln for (t, ln) in self.lines if self.t0 is not None and self.t0 <= t <= (self.t1 or t) + 0.05]
        short = not inside
        if short:           # region shorter than one sampling period: fall back to every sample taken
            inside = [ln for (_, ln) in self.lines]
        for ln in inside:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for nm, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        out = {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
               "samples": len(sm), "reasons": sorted(reasons)}
        if short:
            out["note"] = "timed region shorter than one sampling period: samples taken next to it"
        return out


# ------------------------------------------------------------------------------ workloads
class LogregWorkload:
    """Configs 1 and 2: bilevel weight decay for logistic regression (App. D.1 problem)."""

    def __init__(self, cfg: int, method: str, scale: float = 1.0, shard=None):
        import synth_inputs as si
        self.cfg = cfg
        self.inp = si.config1() if cfg == 1 else si.config2(scale)
        self.method = method or ("cg" if cfg == 2 else "cg")
        self.n, self.d = self.inp.X.shape
        self.nv = self.inp.Xv.shape[0]
        self.shard = shard
        if shard is not None:       # strong scaling: this rank keeps its share of the rows of both matrices
            from paper_2207_02849_b200 import data_parallel as dp
            import copy
            rank, world = shard
            self.n_global, self.nv_global = self.n, self.nv
            lo, hi = dp.shard_rows(self.n, rank, world)
            lov, hiv = dp.shard_rows(self.nv, rank, world)
            inp = copy.copy(self.inp)
            inp.X, inp.y, inp.Xv, inp.yv = self.inp.X[lo:hi], self.inp.y[lo:hi], self.inp.Xv[lov:hiv], self.inp.yv[lov:hiv]
            self.inp = inp
            self.n, self.nv = hi - lo, hiv - lov
        ng, nvg = (self.n_global, self.nv_global) if shard is not None else (self.n, self.nv)
        self.name = (f"config{cfg}: logistic weight-decay bilevel, X fp32 {ng}x{self.d} train / "
                     f"{nvg}x{self.d} val, {self.inp.lower_steps} lower GD steps, {self.method} K={self.inp.K}")
        self.dtype = "f32"

    # algorithmic bytes of one streaming pass over the train matrix (the dominant kernel)
    def pass_bytes(self):
        return self.n * self.d * 4

    def setup_device(self):
        import torch
        import paper_2207_02849_b200 as bt
        from paper_2207_02849_b200 import problems as cb
        self.bt, self.torch = bt, torch
        self.w, self.lam = cb.logreg_levels(self.inp)
        if self.shard is not None:
            from paper_2207_02849_b200 import data_parallel as dp
            self.allreduce = dp.DeviceAllReduce()
            dp.shard_level(self.w, self.n_global, self.shard[0], self.shard[1], self.allreduce)
            dp.shard_level(self.lam, self.nv_global, self.shard[0], self.shard[1], self.allreduce)
        self.w0 = self.w.params.clone()
        self.out = torch.empty(self.d, dtype=torch.float32, device="cuda")
        extra = (self.inp.lower_steps + 1) * (self.d + 64) * 4 if self.method == "itd" else 0
        self.ws = bt.Workspace([self.w, self.lam], extra_bytes=extra)

    def step(self):
        bt = self.bt
        self.w.params.copy_(self.w0)
        if self.method == "itd":      # the unrolled steps are part of the call
            bt.betty_hypergrad_itd(self.w, self.lam, self.lam, self.inp.lower_steps, self.out, self.ws)
            return
        bt.betty_lower_step(self.w, self.inp.lower_steps, self.ws)
        if self.method == "cg":
            bt.betty_hypergrad_cg(self.w, self.lam, self.lam, self.inp.K, 0.0, self.out, self.ws)
        elif self.method == "neumann":
            bt.betty_hypergrad_neumann(self.w, self.lam, self.lam, self.inp.K, self.inp.alpha, self.out, self.ws)
        else:
            bt.betty_hypergrad_fd(self.w, self.lam, self.lam, 0.01, 1.0, self.out, self.ws)

    # -- end-to-end: host buffers in, result out, through the same C-ABI calls
    def setup_host(self):
        torch = self.torch
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        self.h_in = [pin(self.inp.X), pin(self.inp.y), pin(self.inp.Xv), pin(self.inp.yv), pin(self.inp.lam),
                     pin(self.inp.w0)]
        self.d_in = [self.w.X, self.w.y, self.lam.X, self.lam.y, self.lam.params, self.w0]
        self.h_out = torch.empty(self.d, dtype=torch.float32).pin_memory()
        self.h2d = sum(t.numel() * t.element_size() for t in self.h_in)
        self.d2h = self.h_out.numel() * 4

    def step_e2e(self):
        for h, d in zip(self.h_in, self.d_in):
            d.copy_(h, non_blocking=True)
        self.step()
        self.h_out.copy_(self.out, non_blocking=True)

    def roofline_probe(self, reps: int):
        """Average duration of the dominant kernel (the fused HVP row-stream pass over the train
        matrix), timed alone with CUDA events around single betty_hvp calls; the tiny fixed-order
        reduction kernel that follows it is inside the bracket."""
        torch, bt = self.torch, self.bt
        u = torch.randn(self.d, dtype=torch.float32, device="cuda")
        hu = torch.empty_like(u)
        for _ in range(3):
            bt.betty_hvp(self.w, u, hu, self.ws)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in evs:
            a.record()
            bt.betty_hvp(self.w, u, hu, self.ws)
            b.record()
        torch.cuda.synchronize()
        ms = float(np.mean([a.elapsed_time(b) for a, b in evs]))
        # The same pass in its gradient form (one lower step = stream kernel + reduction; 21 of the step's 41
        # passes; the solve's 19 later HVPs, which reuse the first one's per-row curvature, run at its rate).
        keep = self.w.params.clone()
        for _ in range(2):
            bt.betty_lower_step(self.w, 1, self.ws)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in evs:
            a.record()
            bt.betty_lower_step(self.w, 1, self.ws)
            b.record()
        torch.cuda.synchronize()
        ms_g = float(np.mean([a.elapsed_time(b) for a, b in evs]))
        self.w.params.copy_(keep)
        return {"kernel": "k_logreg_stream<HVP>", "ms": ms, "bytes": self.pass_bytes(), "bound": "hbm",
                "also": {"kernel": "k_logreg_stream<gradient> (betty_lower_step, one step)", "ms": ms_g}}

    def parity(self):
        """Relative L2 error of one step's hypergradient against the fp64 oracle on the whole workload
        (small configurations only)."""
        import oracle
        from oracle import problems as ob
        self.step()
        got = self.out.double().cpu().numpy()
        ow, olam = ob.logreg_levels(self.inp)
        oracle.lower_step(ow, self.inp.lower_steps)
        if self.method == "cg":
            ref = oracle.hypergrad_cg(ow, olam, olam, self.inp.K, 0.0)
        elif self.method == "neumann":
            ref = oracle.hypergrad_neumann(ow, olam, olam, self.inp.K, self.inp.alpha)
        else:
            return None
        return float(np.linalg.norm(got - ref) / np.linalg.norm(ref))

    # -- oracle on a bounded sample of the same workload
    def oracle_sample(self, budget_rows: int):
        import oracle
        from oracle import problems as ob
        import synth_inputs as si
        import copy
        n_s = min(self.n, budget_rows)
        nv_s = max(1, min(self.nv, int(round(budget_rows * self.nv / self.n))))
        inp = copy.copy(self.inp)
        inp.X, inp.y, inp.Xv, inp.yv = self.inp.X[:n_s], self.inp.y[:n_s], self.inp.Xv[:nv_s], self.inp.yv[:nv_s]
        ow, olam = ob.logreg_levels(inp)
        t0 = time.perf_counter()
        if self.method == "itd":
            oracle.hypergrad_itd(ow, olam, olam, inp.lower_steps)
        else:
            oracle.lower_step(ow, inp.lower_steps)
        if self.method == "itd":
            pass
        elif self.method == "cg":
            oracle.hypergrad_cg(ow, olam, olam, inp.K, 0.0)
        elif self.method == "neumann":
            oracle.hypergrad_neumann(ow, olam, olam, inp.K, inp.alpha)
        else:
            oracle.hypergrad_fd(ow, olam, olam, 0.01, 1.0)
        dt = time.perf_counter() - t0
        frac = n_s / self.n
        return dt / frac, f"first {n_s} of {self.n} train rows and {nv_s} of {self.nv} validation rows, full step, time scaled by {1/frac:.0f}x"


class ReweightWorkload:
    """Configs 3 and 5: data reweighting (App. A listing): lower MLP classifier, upper 1-100-1 weight net."""

    def __init__(self, cfg: int, method: str, shard=None):
        import synth_inputs as si
        self.cfg = cfg
        self.inp = si.config3() if cfg == 3 else si.config5()
        self.method = method or ("fd" if cfg == 3 else "neumann")
        w = self.inp.widths
        self.B = self.inp.train.X.shape[0]
        self.shard = shard
        if shard is not None:       # strong scaling: this rank keeps its share of the rows of both batches
            from paper_2207_02849_b200 import data_parallel as dp
            import copy
            self.B_global = self.B
            lo, hi = dp.shard_rows(self.B, shard[0], shard[1])
            cut = lambda b: type(b)(X=b.X[lo:hi], y=b.y[lo:hi], y_clean=b.y_clean[lo:hi], clean=b.clean[lo:hi])
            inp = copy.copy(self.inp)
            inp.train, inp.val = cut(self.inp.train), cut(self.inp.val)
            self.inp = inp
        self.name = (f"config{cfg}: data reweighting, MLP {'x'.join(map(str, w)) if len(w) < 5 else f'{w[0]}->{len(w)-2}x{w[1]}->{w[-1]}'} "
                     f"{self.inp.activation} bf16/fp32-acc, batch {self.B}, {self.inp.lower_steps} lower SGD step(s), "
                     f"{self.method}" + (f" K={self.inp.K}" if self.method in ("neumann", "cg") else (" eps0=0.01" if self.method == "fd" else "")))
        self.dtype = "bf16"

    def setup_device(self):
        import torch
        import paper_2207_02849_b200 as bt
        from paper_2207_02849_b200 import problems as cb
        self.bt, self.torch = bt, torch
        self.w, self.th = cb.reweight_levels(self.inp)
        if self.shard is not None:
            from paper_2207_02849_b200 import data_parallel as dp
            self.allreduce = dp.DeviceAllReduce()
            dp.shard_level(self.w, self.B_global, self.shard[0], self.shard[1], self.allreduce)
            dp.shard_level(self.th, self.B_global, self.shard[0], self.shard[1], self.allreduce)
        self.w0 = self.w.params.clone()
        self.out = torch.empty(self.th.params.numel(), dtype=torch.float32, device="cuda")
        extra = (self.inp.lower_steps + 1) * (self.inp.w.size + 64) * 4 if self.method == "itd" else 0
        self.ws = bt.Workspace([self.w, self.th], extra_bytes=extra)

    def step(self):
        bt = self.bt
        self.w.params.copy_(self.w0)
        if self.method == "itd":
            bt.betty_hypergrad_itd(self.w, self.th, self.th, self.inp.lower_steps, self.out, self.ws)
            return
        bt.betty_lower_step(self.w, self.inp.lower_steps, self.ws)
        if self.method == "fd":
            bt.betty_hypergrad_fd(self.w, self.th, self.th, self.inp.eps0, self.inp.fd_alpha, self.out, self.ws)
        elif self.method == "neumann":
            bt.betty_hypergrad_neumann(self.w, self.th, self.th, self.inp.K, self.inp.alpha, self.out, self.ws)
        else:
            bt.betty_hypergrad_cg(self.w, self.th, self.th, self.inp.K, 0.0, self.out, self.ws)

    def setup_host(self):
        torch = self.torch
        pin = lambda t: t.detach().cpu().pin_memory()
        self.d_in = [self.w.X, self.w.y, self.th.X, self.th.y, self.th.params, self.w0]
        self.h_in = [pin(t) for t in self.d_in]
        self.h_out = torch.empty(self.out.numel(), dtype=torch.float32).pin_memory()
        self.h2d = sum(t.numel() * t.element_size() for t in self.h_in)
        self.d2h = self.h_out.numel() * 4

    def step_e2e(self):
        for h, d in zip(self.h_in, self.d_in):
            d.copy_(h, non_blocking=True)
        self.step()
        self.h_out.copy_(self.out, non_blocking=True)

    def roofline_probe(self, reps: int):
        """The dominant kernel is the tensor-core GEMM; its most frequent shape in this workload
        (batch x width x width, forward layout) is timed alone through the C ABI."""
        torch, bt = self.torch, self.bt
        w = self.inp.widths
        M, N, K = self.B, w[1], (w[1] if len(w) > 3 else w[0])
        A = torch.randn(M, K, device="cuda").to(torch.bfloat16)
        Bm = torch.randn(N, K, device="cuda").to(torch.bfloat16)
        Cm = torch.empty(M, N, dtype=torch.float32, device="cuda")
        pairs = [(A, K, 0, Bm, K, 1, K, 1.0)]
        for _ in range(3):
            bt.betty_gemm_bf16(M, N, pairs, Cm, N, 0.0, 2, self.ws)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in evs:
            a.record()
            bt.betty_gemm_bf16(M, N, pairs, Cm, N, 0.0, 2, self.ws)
            b.record()
        torch.cuda.synchronize()
        ms = float(np.mean([a.elapsed_time(b) for a, b in evs]))
        return {"kernel": f"k_gemm_tc {M}x{N}x{K}", "ms": ms, "flops": 2.0 * M * N * K, "bound": "tensor"}

    def whole_step_flops(self):
        """Matrix-product FLOPs of one step with the Neumann method: per layer U_l = 2 B in_l out_l; a
        gradient is forward + backward-data + weight-gradient products (3 sum U - U_1), a Hessian-vector
        product with the base pass cached is the R-forward, R-backward-data and two weight-gradient
        products per layer (6 sum U - 4 U_1: the input has no tangent), the mixed product one R-forward."""
        if self.method != "neumann":
            return None
        w = self.inp.widths
        U = [2.0 * self.B * w[l] * w[l + 1] for l in range(len(w) - 1)]
        grad, hvp, jvp = 3 * sum(U) - U[0], 6 * sum(U) - 4 * U[0], 2 * sum(U) - U[0]
        return (self.inp.lower_steps + 2) * grad + self.inp.K * hvp + jvp

    def parity(self):
        """Relative L2 error of one step's hypergradient against the fp64 oracle on the whole workload."""
        import oracle
        from oracle import problems as ob
        self.step()
        got = self.out.double().cpu().numpy()
        ow, oth = ob.reweight_levels(self.inp)
        oracle.lower_step(ow, self.inp.lower_steps)
        if self.method == "fd":
            ref = oracle.hypergrad_fd(ow, oth, oth, self.inp.eps0, self.inp.fd_alpha)
        elif self.method == "neumann":
            ref = oracle.hypergrad_neumann(ow, oth, oth, self.inp.K, self.inp.alpha)
        else:
            return None
        return float(np.linalg.norm(got - ref) / np.linalg.norm(ref))

    def oracle_sample(self, budget_rows: int):
        import copy
        import oracle
        from oracle import problems as ob
        frac = 1.0 if self.cfg == 3 else 1.0 / 8
        nb = max(1, int(self.B * frac))
        inp = copy.copy(self.inp)
        cut = lambda b: type(b)(X=b.X[:nb], y=b.y[:nb], y_clean=b.y_clean[:nb], clean=b.clean[:nb])
        inp.train, inp.val = cut(self.inp.train), cut(self.inp.val)
        ow, oth = ob.reweight_levels(inp)
        t0 = time.perf_counter()
        if self.method == "itd":
            oracle.hypergrad_itd(ow, oth, oth, inp.lower_steps)
        else:
            oracle.lower_step(ow, inp.lower_steps)
        if self.method == "itd":
            pass
        elif self.method == "fd":
            oracle.hypergrad_fd(ow, oth, oth, inp.eps0, inp.fd_alpha)
        elif self.method == "neumann":
            oracle.hypergrad_neumann(ow, oth, oth, inp.K, inp.alpha)
        else:
            oracle.hypergrad_cg(ow, oth, oth, inp.K, 0.0)
        dt = time.perf_counter() - t0
        return dt / frac, f"first {nb} of {self.B} rows of the train and validation batches, full step, time scaled by {1/frac:.0f}x"


class ThreeLevelWorkload:
    """Config 4: three-level chain; the timed unit is the level-3 hypergradient after one lower step."""

    def __init__(self, method: str):
        import synth_inputs as si
        self.inp = si.config4()
        self.method = "neumann"
        self.B = self.inp.D1.X.shape[0]
        self.name = (f"config4: three-level chain, MLP {'x'.join(map(str, self.inp.widths))} relu bf16/fp32-acc, batch "
                     f"{self.B}, weight net 1-100-1, per-layer log weight decay, two Neumann K={self.inp.K} edges")
        self.dtype = "bf16"

    def setup_device(self):
        import torch
        import paper_2207_02849_b200 as bt
        from paper_2207_02849_b200 import problems as cb
        self.bt, self.torch = bt, torch
        self.P = cb.three_levels(self.inp)
        self.w0 = self.P[0].params.clone()
        self.out = torch.empty(self.inp.lam.size, dtype=torch.float32, device="cuda")
        self.ws = bt.Workspace(list(self.P))
        self.cfgm = bt.MethodCfg(bt.BETTY_NEUMANN, K=self.inp.K, alpha=self.inp.alpha)
        self.u2l = [(2, 0), (1, 0)]              # lambda and theta constrain the classifier
        self.l2u = [(0, 1), (0, 2), (1, 2)]      # w* constrains P2 and P3, theta* constrains P3

    def step(self):
        bt, (P1, P2, P3) = self.bt, self.P
        P1.params.copy_(self.w0)
        bt.betty_lower_step(P1, 1, self.ws)
        # Eq. 2 over the program's dataflow graph, both paths from lambda merged at the w* node: one call
        bt.betty_hypergrad_graph(list(self.P), self.u2l, self.l2u, 2, [self.cfgm] * 3, self.out, self.ws)

    def setup_host(self):
        torch = self.torch
        P1, P2, P3 = self.P
        pin = lambda t: t.detach().cpu().pin_memory()
        self.d_in = [P1.X, P1.y, P2.X, P2.y, P2.aux, P3.X, P3.y, P3.aux, P2.params, P3.params, self.w0]
        self.h_in = [pin(t) for t in self.d_in]
        self.h_out = torch.empty(self.out.numel(), dtype=torch.float32).pin_memory()
        self.h2d = sum(t.numel() * t.element_size() for t in self.h_in)
        self.d2h = self.h_out.numel() * 4

    step_e2e = ReweightWorkload.step_e2e

    def roofline_probe(self, reps: int):
        self.inp.widths  # forward-layout GEMM batch x 512 x 784
        rw = ReweightWorkload.roofline_probe
        return rw(self, reps)

    def parity(self):
        import oracle
        from oracle import problems as ob
        self.step()
        got = self.out.double().cpu().numpy()
        O1, O2, O3 = ob.three_levels(self.inp)
        nm = dict(method="neumann", K=self.inp.K, alpha=self.inp.alpha)
        oracle.lower_step(O1, 1)
        u = oracle.grad(O3, O1) + oracle.chain_levels([O1, O2, O3], [0, 1], [nm], v_in=oracle.grad(O3, O2))
        ref = oracle.chain_levels([O1, O2, O3], [2, 0], [nm], v_in=u)
        return float(np.linalg.norm(got - ref) / np.linalg.norm(ref))

    def oracle_sample(self, budget_rows: int):
        import oracle
        from oracle import problems as ob
        O1, O2, O3 = ob.three_levels(self.inp)
        nm = dict(method="neumann", K=self.inp.K, alpha=self.inp.alpha)
        t0 = time.perf_counter()
        oracle.lower_step(O1, 1)
        u = oracle.grad(O3, O1) + oracle.chain_levels([O1, O2, O3], [0, 1], [nm], v_in=oracle.grad(O3, O2))
        oracle.chain_levels([O1, O2, O3], [2, 0], [nm], v_in=u)
        return time.perf_counter() - t0, "the full workload"


def make_workload(cfg: int, method: str, scale: float, shard=None):
    if cfg in (1, 2):
        return LogregWorkload(cfg, method, scale, shard)
    if cfg in (3, 5):
        return ReweightWorkload(cfg, method, shard)
    if cfg == 4:
        if shard is not None:
            raise SystemExit("strong scaling is offered for configurations 1, 2, 3 and 5")
        return ThreeLevelWorkload(method)
    raise SystemExit(f"unknown config {cfg}")


def max_over_ranks(ms: float, world: int, dist, device) -> float:
    """Step time of the job = the slowest rank's device time."""
    if world <= 1:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(ms_per_step: float, world: int) -> float:
    """Whole-job steps/s of `world` independent replicas that each finish a step every ms_per_step."""
    return world * 1e3 / ms_per_step


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


# ------------------------------------------------------------------------------ main
def run_reference(args, rank, world):
    if rank != 0:
        return
    wl = make_workload(args.config, args.method, args.scale)
    rows = args.oracle_rows
    times = []
    for i in range(args.warmup + args.steps):
        t, sample = wl.oracle_sample(rows)
        if i >= args.warmup:
            times.append(t)
    sec = float(np.mean(times))
    val = 1.0 / sec
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "note": "the fp64 oracle on the host cores of rank 0; no GPU is used"},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def gemm_probe(args, torch, bt):
    """Times `steps` back-to-back launches of one matrix product (queued behind a long memset so
    that host-side launch cost does not show) and prints achieved TFLOP/s."""
    f = [int(x) for x in args.gemm.split(",")]
    M, N, K = f[:3]
    ta, tb, npairs, path = (f[3:] + [0, 1, 1, 0][len(f) - 3:])[:4]
    A = torch.randn((K, M) if ta else (M, K), device="cuda").to(torch.bfloat16)
    B = torch.randn((N, K) if tb else (K, N), device="cuda").to(torch.bfloat16)
    C = torch.empty(M, N, dtype=torch.float32, device="cuda")
    pairs = [(A, A.shape[1], ta, B, B.shape[1], tb, K, 1.0)] * npairs
    lv = bt.Level(bt.LOSS_LOGREG, bt.PARAM_VECTOR, torch.zeros(8, device="cuda"))
    ws = bt.Workspace.__new__(bt.Workspace)
    ws.nbytes = 4096
    ws.buf = torch.zeros(4096 + 256, dtype=torch.uint8, device="cuda")
    ws.ptr = ws.buf.data_ptr() + (-ws.buf.data_ptr()) % 256
    for _ in range(max(args.warmup, 3)):
        bt.betty_gemm_bf16(M, N, pairs, C, N, 0.0, path, ws)
    big = torch.empty(1 << 28, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    big.zero_(); big.zero_()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        bt.betty_gemm_bf16(M, N, pairs, C, N, 0.0, path, ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    peaks = _peaks()
    tf = 2.0 * M * N * K * npairs / (ms * 1e-3) / 1e12
    print(json.dumps({"kernel": "betty_gemm_bf16", "M": M, "N": N, "K": K, "a_transposed": ta, "b_transposed": tb,
                      "n_pairs": npairs, "path": path, "us_per_launch": ms * 1e3, "tflops": tf,
                      "frac_of_bf16_peak": tf / peaks["bf16_tflops"], "peak_source": peaks["source"],
                      "device_status": bt.betty_status_string(bt.betty_poll_status(ws, raise_on_error=False)[0])}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--method", default="", choices=["", "cg", "neumann", "fd", "itd"])
    ap.add_argument("--scale", type=float, default=1.0, help="row-count scale of config 2 (tests/profiling only)")
    ap.add_argument("--oracle-rows", type=int, default=131072)
    ap.add_argument("--graph", type=int, default=-1,
                    help="replay the step from a CUDA graph captured from the C-ABI calls (default: on; 0 = plain calls)")
    ap.add_argument("--gemm", default="",
                    help="M,N,K[,a_transposed,b_transposed,n_pairs,path]: time only the bf16 matrix-product kernel "
                         "through betty_gemm_bf16 (kernel study; prints its own JSON line)")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="N > 1: weak = N independent replicas of the workload (default); strong = ONE workload "
                         "whose rows are sharded over the N ranks, one all-reduce of a parameter-sized vector per "
                         "gradient / Hessian-vector product / mixed product")
    ap.add_argument("--per-config", type=int, default=-1,
                    help="add short runs of the other configurations to the line (default: on for the plain "
                         "single-GPU configuration-2 run)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if args.steps > 3:
            args.steps = 3
        args.warmup = min(args.warmup, 1)
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: this path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    import paper_2207_02849_b200 as bt

    if args.gemm:
        gemm_probe(args, torch, bt)
        return
    warm = max(args.warmup, 3)
    peaks = _peaks()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    flush_buf = []

    def flush_for(cfg):
        """Configurations whose inputs fit in L2 get a flush (a 512 MiB write) before every step."""
        if cfg == 2:
            return None
        if not flush_buf:
            flush_buf.append(torch.empty(512 << 20, dtype=torch.uint8, device="cuda"))
        return flush_buf[0]

    def timed(fn, steps, warmup, flush, sampler=None, launches_per_replay=None):
        if sampler:
            sampler.start()     # the sampler starts during warm-up; only samples inside the timed region count
        for _ in range(warmup):
            fn()
        barrier()
        if sampler:
            sampler.mark_begin()
        l0 = bt.betty_kernel_launches()
        if flush is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                fn()
            e1.record()
            pairs = [(e0, e1)]
        else:
            pairs = []
            for _ in range(steps):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                pairs.append((e0, e1))
        barrier()
        if sampler:
            sampler.mark_end()
        launches = bt.betty_kernel_launches() - l0
        if launches_per_replay is not None:
            launches = launches_per_replay * steps
        clocks = sampler.stop() if sampler else None
        ms = sum(a.elapsed_time(b) for a, b in pairs)
        ms = max_over_ranks(ms, world, dist, "cuda")
        return ms, launches, clocks

    def capture(w):
        """The library's calls only enqueue work on the current stream and keep every scalar on the
        device, so a whole step can be captured once and replayed without host-side launch cost."""
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(2):
                w.step()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        l0 = bt.betty_kernel_launches()
        with torch.cuda.graph(graph):
            w.step()
        n = bt.betty_kernel_launches() - l0
        w.step = graph.replay
        w._graph = graph
        return n

    def roofline_of(w, reps=20):
        probe = w.roofline_probe(reps)
        if probe["bound"] == "hbm":
            achieved = probe["bytes"] / (probe["ms"] * 1e-3) / 1e9
            peak, unit, nominal = peaks["hbm_gbs"], "GB/s", NOMINAL_HBM_GBS
        else:
            achieved = probe["flops"] / (probe["ms"] * 1e-3) / 1e12
            peak, unit, nominal = peaks["bf16_tflops"], "TFLOP/s", NOMINAL_BF16_TFLOPS
        traffic = None
        tpath = os.path.join(ROOT, "profiles", "traffic.json")
        if os.path.exists(tpath):
            with open(tpath) as f:
                tj = json.load(f).get(probe["kernel"])
            if tj and tj.get("valid"):
                if "dram_bytes_per_launch" in tj:       # captured at the probe's own shape
                    traffic = float(tj["dram_bytes_per_launch"])
                else:                                   # captured on a smaller case; grows with the units streamed
                    traffic = tj["dram_bytes_per_unit"] * (probe["bytes"] / tj["unit_bytes"])
        r = {"bound": probe["bound"], "kernel": probe["kernel"], "achieved": achieved, "peak": peak, "unit": unit,
             "frac": achieved / peak, "traffic": traffic, "peak_source": f"{peaks['source']} (burst; kernel timed alone)",
             "nominal_peak": nominal, "frac_of_nominal": achieved / nominal,
             "kernel_ms": probe["ms"], "algorithmic_bytes_per_launch": probe.get("bytes"),
             "algorithmic_flops_per_launch": probe.get("flops")}
        if probe.get("also") and probe["bound"] == "hbm":
            a2 = probe["bytes"] / (probe["also"]["ms"] * 1e-3) / 1e9
            r["other_forms"] = [{"kernel": probe["also"]["kernel"], "kernel_ms": probe["also"]["ms"], "achieved": a2,
                                 "frac": a2 / peak, "frac_of_nominal": a2 / nominal}]
        return r

    def graph_default(cfg):
        return args.graph != 0

    strong = args.scaling == "strong"
    wl = make_workload(args.config, args.method, args.scale, (rank, world) if strong else None)
    wl.setup_device()
    flush = flush_for(args.config)
    l2_note = ("inputs (train matrix) larger than L2; no flush between steps" if flush is None
               else "L2 flushed (512 MiB write) before every step; each step timed by its own event pair, flush excluded")
    use_graph = graph_default(args.config) and not strong      # the all-reduce between kernels is not captured
    launches_per_replay = capture(wl) if use_graph else None
    step_dev, step_host = wl.step, wl.step_e2e

    sampler = ClockSampler(local) if rank == 0 else None
    ms, launches, clocks = timed(step_dev, args.steps, warm, flush, sampler, launches_per_replay)
    st, _ = bt.betty_poll_status(wl.ws)
    ms_per_step = ms / args.steps
    value = 1e3 / ms_per_step if strong else aggregate_value(ms_per_step, world)

    e2e = None
    wl2 = sets = None
    if not args.no_e2e:
        wl.setup_host()
        e_steps = max(1, min(args.steps, 5))
        if wl.h2d > (126 << 20):
            # Inputs larger than L2 (no flush needed): two device input sets, the copy of step i+1's inputs
            # runs on a second stream while step i computes; every step still copies all of its inputs from
            # pinned host memory and reads its result back, all inside the timed region.
            import copy
            wl2 = copy.copy(wl)                     # same generated inputs, own device tensors and workspace
            wl2.__dict__.pop("step", None)
            wl2.__dict__.pop("_graph", None)
            wl2.setup_device()
            if use_graph:
                capture(wl2)
            wl2.setup_host()
            wl2.h_in = wl.h_in                      # the same pinned host buffers
            sets = [wl, wl2]
            main_s, copy_s = torch.cuda.current_stream(), torch.cuda.Stream()
            ready = [torch.cuda.Event(), torch.cuda.Event()]
            free = [torch.cuda.Event(), torch.cuda.Event()]

            def issue_copy(i):
                b = i % 2
                copy_s.wait_event(free[b])          # the step that last used this set has finished
                with torch.cuda.stream(copy_s):
                    for h, d in zip(sets[b].h_in, sets[b].d_in):
                        d.copy_(h, non_blocking=True)
                    ready[b].record(copy_s)

            def run(n):
                for ev in free:
                    ev.record(main_s)
                issue_copy(0)
                for i in range(n):
                    b = i % 2
                    if i + 1 < n:
                        issue_copy(i + 1)
                    main_s.wait_event(ready[b])
                    sets[b].step()
                    sets[b].h_out.copy_(sets[b].out, non_blocking=True)
                    free[b].record(main_s)

            run(3)
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            run(e_steps)
            e1.record()
            barrier()
            ms_e = max_over_ranks(e0.elapsed_time(e1), world, dist, "cuda")
            how = "two device input sets: step i+1's host-to-device copy overlaps step i's kernels"
        else:
            ms_e, _, _ = timed(step_host, e_steps, 3, flush)
            how = "copy, compute and read-back in sequence on one stream"
        e2e = {"value": (1 if strong else world) * 1e3 / (ms_e / e_steps), "unit": UNIT, "h2d_bytes_per_step": int(wl.h2d),
               "d2h_bytes_per_step": int(wl.d2h), "how": how}

    roofline = roofline_of(wl)
    wl_name, wl_dtype = wl.name, wl.dtype

    # The other configurations, each as a short run of its own (the metric is quoted per configuration):
    # only on the default single-GPU run, after the headline workload has released its device memory.
    per_config = None
    if args.per_config == 1 or (args.per_config == -1 and world == 1 and args.config == 2 and not args.method
                                and args.scale == 1.0):
        cpu_early = None
        if not args.no_cpu_baseline and world == 1 and rank == 0:
            sec, sample = wl.oracle_sample(args.oracle_rows)
            cpu_early = {"value": 1.0 / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample}
        del step_dev, step_host
        if wl2 is not None:
            _release(wl2)
        wl2 = sets = None
        wl = _release(wl)
        torch.cuda.empty_cache()
        per_config = {}
        for key, cfg, method, steps_c in PER_CONFIG_RUNS:
            w = make_workload(cfg, method, 1.0)
            w.setup_device()
            lpr = capture(w) if graph_default(cfg) else None
            smp = ClockSampler(local)
            ms_c, launches_c, clocks_c = timed(w.step, steps_c, 3, flush_for(cfg), smp, lpr)
            st_c, _ = bt.betty_poll_status(w.ws)
            entry = {"workload": w.name, "steps": steps_c, "ms_per_step": ms_c / steps_c,
                     "steps_per_s": 1e3 * steps_c / ms_c, "gpu_launches_per_step": int(launches_c // steps_c),
                     "cuda_graph": lpr is not None, "device_status": bt.betty_status_string(st_c), "clocks": clocks_c,
                     "roofline": roofline_of(w, 10)}
            if hasattr(w, "whole_step_flops") and w.whole_step_flops():
                tf = w.whole_step_flops() / (ms_c / steps_c * 1e-3) / 1e12
                entry["whole_step"] = {"tflops": tf, "frac_of_burst_peak": tf / peaks["bf16_tflops"],
                                       "frac_of_sustained_peak": tf / peaks["bf16_tflops_sustained"]}
            if cfg in (1, 3, 4):
                entry["rel_l2_vs_oracle"] = w.parity()
            per_config[key] = entry
            w = _release(w)
            torch.cuda.empty_cache()
    else:
        cpu_early = None

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = cpu_early
    if cpu is None and not args.no_cpu_baseline and world == 1:
        sec, sample = wl.oracle_sample(args.oracle_rows)
        cpu = {"value": 1.0 / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": args.scaling, "vs_baseline": None,
            "dtype": wl_dtype, "data": "synthetic",
            "config": {"workload": wl_name, "l2": l2_note,
                       "replicas": 1 if strong else world,
                       "parallelism": (f"rows of every batch sharded over {world} rank(s); parameters and solver state "
                                       "replicated; one all-reduce (sum) of a parameter-sized vector per gradient, "
                                       "Hessian-vector product and mixed product") if strong
                       else f"{world} independent replica(s), no exchange in the data path",
                       "cuda_graph": bool(use_graph), "device_status": bt.betty_status_string(st)},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline, "cpu_baseline": cpu}
    if per_config is not None:
        line["per_config"] = per_config
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
