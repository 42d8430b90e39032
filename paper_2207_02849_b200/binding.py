"""ctypes binding of include/betty.h.  Argument marshalling only: every computation runs in
the CUDA library.  torch is used for device memory and the current stream."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))

# ---- enums (mirrors of betty.h) ----
BETTY_OK = 0
(BETTY_ERR_INVALID_ARG, BETTY_ERR_SHAPE, BETTY_ERR_DTYPE, BETTY_ERR_ALIGNMENT, BETTY_ERR_WORKSPACE,
 BETTY_ERR_CUDA, BETTY_ERR_NONFINITE, BETTY_ERR_BREAKDOWN, BETTY_ERR_TIMEOUT,
 BETTY_ERR_UNSUPPORTED, BETTY_ERR_CAPACITY) = range(1, 12)
(LOSS_LOGREG_WD, LOSS_LOGREG, LOSS_QUADRATIC_WD, LOSS_QUADRATIC, LOSS_MLP_CE_REWEIGHT, LOSS_MLP_CE,
 LOSS_WEIGHTNET_DETECT, LOSS_MLP_CE_CORRECT) = range(8)
PARAM_VECTOR, PARAM_MLP, PARAM_WEIGHTNET, PARAM_LOGWD, PARAM_CORRECTNET = range(5)
BETTY_NEUMANN, BETTY_CG, BETTY_FD = range(3)
ACT_RELU, ACT_GELU = range(2)
BETTY_F32, BETTY_BF16, BETTY_I32, BETTY_F16 = range(4)
BETTY_OPT_GD, BETTY_OPT_MOMENTUM, BETTY_OPT_ADAM = range(3)
BETTY_LR_CONSTANT, BETTY_LR_MULTISTEP, BETTY_LR_COSINE = range(3)


class BettyError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {betty_status_string(status)} (status {status})")


class _MethodCfg(C.Structure):
    _fields_ = [("method", C.c_int32), ("K", C.c_int32), ("alpha", C.c_float), ("eps0", C.c_float),
                ("tol", C.c_float)]


_ALLREDUCE = C.CFUNCTYPE(C.c_int32, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p)


class _Comm(C.Structure):
    _fields_ = [("allreduce", _ALLREDUCE), ("user", C.c_void_p), ("row_weight", C.c_float)]


class _Level(C.Structure):
    pass


_Level._fields_ = [
    ("loss", C.c_int32), ("param_kind", C.c_int32), ("params", C.c_void_p), ("n_params", C.c_int64),
    ("X", C.c_void_p), ("x_dtype", C.c_int32), ("n", C.c_int64), ("d", C.c_int64),
    ("y", C.c_void_p), ("aux", C.c_void_p), ("n_layers", C.c_int32), ("widths", C.POINTER(C.c_int64)),
    ("activation", C.c_int32), ("lr", C.c_float), ("mu", C.c_float), ("optimizer", C.c_int32),
    ("momentum", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("adam_eps", C.c_float),
    ("weight_decay", C.c_float), ("opt_state", C.c_void_p), ("n_constraints", C.c_int32),
    ("constraints", C.POINTER(C.POINTER(_Level))),
    ("lr_schedule", C.c_int32), ("lr_step0", C.c_int32), ("lr_t_max", C.c_int32), ("lr_milestones", C.c_int32 * 4),
    ("lr_gamma", C.c_float), ("lr_min", C.c_float), ("grad_accum", C.c_int32), ("comm", C.POINTER(_Comm)),
    ("precision", C.c_int32), ("loss_scale", C.c_void_p),
]

class _Edge(C.Structure):
    _fields_ = [("src", C.c_int32), ("dst", C.c_int32)]


class _GemmOperands(C.Structure):
    _fields_ = [("A", C.c_void_p), ("lda", C.c_int64), ("a_transposed", C.c_int32), ("B", C.c_void_p),
                ("ldb", C.c_int64), ("b_transposed", C.c_int32), ("K", C.c_int32), ("alpha", C.c_float)]


_lib = None


def lib_path() -> str:
    return os.path.join(_HERE, "libbetty.so")


def lib():
    """The loaded CUDA library.  Raises if it has not been built: nothing here falls back to
    another implementation."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -m paper_2207_02849_b200.build` "
                           "(nvcc, sm_100a); this package has no CPU fallback")
    L = C.CDLL(path)
    LP, VP, I32, SZ, F = C.POINTER(_Level), C.c_void_p, C.c_int32, C.c_size_t, C.c_float
    sig = {
        "betty_workspace_size": [C.POINTER(LP), I32, C.POINTER(SZ)],
        "betty_reset_status": [VP, SZ, VP],
        "betty_poll_status": [VP, VP, C.POINTER(I32)],
        "betty_lower_step": [LP, I32, VP, SZ, VP],
        "betty_grad": [LP, LP, VP, VP, SZ, VP],
        "betty_hvp": [LP, VP, VP, VP, SZ, VP],
        "betty_mixed_vjp": [LP, LP, VP, VP, VP, SZ, VP],
        "betty_hypergrad_neumann": [LP, LP, LP, I32, F, VP, VP, SZ, VP],
        "betty_hypergrad_cg": [LP, LP, LP, I32, F, VP, VP, SZ, VP],
        "betty_hypergrad_fd": [LP, LP, LP, F, F, VP, VP, SZ, VP],
        "betty_hypergrad_itd": [LP, LP, LP, I32, VP, VP, SZ, VP],
        "betty_chain_levels": [C.POINTER(LP), I32, C.POINTER(I32), I32, C.POINTER(_MethodCfg), VP, VP, I32,
                               VP, SZ, VP],
    }
    sig["betty_hvp_logreg_static"] = [VP, C.c_int64, C.c_int64, VP, VP, VP, VP, VP, VP]
    sig["betty_gemm_bf16"] = [I32, I32, I32, C.POINTER(_GemmOperands), VP, C.c_int64, F, I32, VP, SZ, VP]
    EP, IP = C.POINTER(_Edge), C.POINTER(I32)
    sig["betty_find_paths"] = [I32, EP, I32, EP, I32, I32, IP, I32, IP, I32, IP, IP]
    sig["betty_selftest_wait_timeout"] = [VP, SZ, VP]
    sig["betty_engine_run"] = [C.POINTER(LP), I32, EP, I32, EP, I32, C.POINTER(_MethodCfg), IP, I32, IP, I32, IP, VP, SZ, VP]
    sig["betty_hypergrad_graph"] = [C.POINTER(LP), I32, EP, I32, EP, I32, I32, C.POINTER(_MethodCfg), VP, VP, SZ, VP]
    for name, args in sig.items():
        fn = getattr(L, name)
        fn.argtypes, fn.restype = args, C.c_int
    L.betty_status_string.argtypes, L.betty_status_string.restype = [C.c_int], C.c_char_p
    L.betty_kernel_launches.argtypes, L.betty_kernel_launches.restype = [], C.c_uint64
    L.betty_selftest_smem_limit.argtypes = [I32, I32, C.c_uint64]
    L.betty_selftest_smem_limit.restype = I32
    _lib = L
    return L


def betty_status_string(status: int) -> str:
    return lib().betty_status_string(int(status)).decode()


def betty_kernel_launches() -> int:
    return int(lib().betty_kernel_launches())


_comm_error = [None]      # exception raised inside a data-parallel all-reduce callback, if any


def _check(status: int, where: str):
    if status != BETTY_OK:
        cause, _comm_error[0] = _comm_error[0], None
        if cause is not None:
            raise BettyError(status, where) from cause
        raise BettyError(status, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device tensors must be contiguous CUDA tensors")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


_DT = {torch.float32: BETTY_F32, torch.bfloat16: BETTY_BF16, torch.int32: BETTY_I32, torch.float16: BETTY_F16}


class Level:
    """Host-side descriptor of one problem P_k: keeps the tensors alive and owns the C struct."""

    def __init__(self, loss: int, param_kind: int, params: torch.Tensor, X: Optional[torch.Tensor] = None,
                 y: Optional[torch.Tensor] = None, aux: Optional[torch.Tensor] = None,
                 widths: Optional[Sequence[int]] = None, activation: int = ACT_RELU, lr: float = 0.1,
                 mu: float = 0.0):
        self.params, self.X, self.y, self.aux = params, X, y, aux
        self.widths = tuple(int(w) for w in widths) if widths is not None else None
        self.constraints: list[Level] = []
        s = _Level()
        s.loss, s.param_kind = int(loss), int(param_kind)
        s.params, s.n_params = _ptr(params), params.numel()
        s.X = _ptr(X)
        s.x_dtype = _DT.get(X.dtype, -1) if X is not None else BETTY_F32
        s.n, s.d = (X.shape[0], X.shape[1]) if X is not None else (0, 0)
        s.y, s.aux = _ptr(y), _ptr(aux)
        if self.widths is not None:
            self._widths = (C.c_int64 * len(self.widths))(*self.widths)
            s.n_layers, s.widths = len(self.widths) - 1, self._widths
        else:
            s.n_layers, s.widths = 0, None
        s.activation, s.lr, s.mu = int(activation), float(lr), float(mu)
        s.optimizer, s.opt_state = BETTY_OPT_GD, None
        self.opt_state = None
        s.n_constraints, s.constraints = 0, None
        self.c = s

    def set_constraints(self, levels: Sequence["Level"]) -> "Level":
        self.constraints = list(levels)
        self._carr = (C.POINTER(_Level) * max(1, len(levels)))(*[C.pointer(l.c) for l in levels])
        self.c.n_constraints = len(levels)
        self.c.constraints = self._carr if levels else None
        return self

    def set_optimizer(self, kind: int, momentum: float = 0.0, beta1: float = 0.9, beta2: float = 0.999,
                      eps: float = 1e-8, weight_decay: float = 0.0) -> "Level":
        """Chooses the optimiser of this problem's steps and allocates its zero-initialised state."""
        n = self.params.numel()
        size = {BETTY_OPT_GD: 0, BETTY_OPT_MOMENTUM: n, BETTY_OPT_ADAM: 2 * n + 1}[int(kind)]
        self.opt_state = torch.zeros(max(size, 1), dtype=torch.float32, device=self.params.device) if size else None
        self.c.optimizer, self.c.momentum = int(kind), float(momentum)
        self.c.beta1, self.c.beta2, self.c.adam_eps = float(beta1), float(beta2), float(eps)
        self.c.weight_decay = float(weight_decay)
        self.c.opt_state = _ptr(self.opt_state)
        return self

    def set_lr_schedule(self, kind: int, step0: int = 0, milestones: Sequence[int] = (), gamma: float = 0.1,
                        t_max: int = 1, lr_min: float = 0.0) -> "Level":
        """Step size as a function of the steps taken (betty_lr_schedule); step0 = steps taken before the
        next call."""
        if len(milestones) > 4:
            raise ValueError("at most 4 milestones")
        self.c.lr_schedule, self.c.lr_step0, self.c.lr_t_max = int(kind), int(step0), int(t_max)
        for i in range(4):
            self.c.lr_milestones[i] = int(milestones[i]) if i < len(milestones) else 0
        self.c.lr_gamma, self.c.lr_min = float(gamma), float(lr_min)
        return self

    def set_comm(self, allreduce, row_weight: float) -> "Level":
        """Marks this level as one rank's share of its problem's batch (betty_comm).  `allreduce(ptr, count,
        stream)` must sum `count` floats at device address `ptr` over all ranks, in place, ordered on the
        CUDA stream handle `stream`; an exception it raises surfaces as BETTY_ERR_CUDA from the library call
        (and is re-raised by the binding).  row_weight = this rank's rows / all rows.  None removes it."""
        if allreduce is None:
            self._comm = self._comm_cb = None
            self.c.comm = None
            return self
        self.comm_error = None

        def _cb(user, buf, count, stream):
            try:
                allreduce(int(buf), int(count), int(stream or 0))
                return 0
            except BaseException as e:           # never let an exception cross the C frames
                self.comm_error = _comm_error[0] = e
                return 1
        self._comm_cb = _ALLREDUCE(_cb)
        self._comm = _Comm(self._comm_cb, None, float(row_weight))
        self.c.comm = C.pointer(self._comm)
        return self

    def set_precision(self, dtype: int) -> "Level":
        """Operand type of an MLP block's matrix products: BETTY_BF16 (default) or BETTY_F16."""
        self.c.precision = int(dtype)
        return self

    def set_loss_scale(self, scale: Optional[float], growth_interval: int = 0) -> "Level":
        """Loss scaling of the lower steps of a BETTY_F16 block: allocates the four-float device state
        [scale, good steps, growth interval, skipped steps] (see betty.h); None switches it off."""
        if scale is None:
            self.loss_scale_state = None
            self.c.loss_scale = None
            return self
        self.loss_scale_state = torch.tensor([float(scale), 0.0, float(growth_interval), 0.0], dtype=torch.float32,
                                             device=self.params.device)
        self.c.loss_scale = _ptr(self.loss_scale_state)
        return self

    def set_grad_accum(self, n_micro: int) -> "Level":
        """Steps of this problem average the gradients of n_micro equal micro-batches of its batch."""
        self.c.grad_accum = int(n_micro)
        return self

    @property
    def ref(self):
        return C.byref(self.c)


class MethodCfg:
    def __init__(self, method: int, K: int = 0, alpha: float = 1.0, eps0: float = 0.01, tol: float = 0.0):
        self.c = _MethodCfg(int(method), int(K), float(alpha), float(eps0), float(tol))


def _level_array(levels: Sequence[Level]):
    return (C.POINTER(_Level) * len(levels))(*[C.pointer(l.c) for l in levels])


def betty_workspace_size(levels: Sequence[Level]) -> int:
    out = C.c_size_t(0)
    _check(lib().betty_workspace_size(_level_array(levels), len(levels), C.byref(out)), "betty_workspace_size")
    return int(out.value)


class Workspace:
    """Caller-owned scratch (a torch uint8 tensor) sized by betty_workspace_size."""

    def __init__(self, levels: Sequence[Level], device="cuda", extra_bytes: int = 0):
        self.nbytes = betty_workspace_size(levels) + int(extra_bytes)
        self.buf = torch.empty(self.nbytes + 256, dtype=torch.uint8, device=device)
        off = (-self.buf.data_ptr()) % 256
        self.ptr = self.buf.data_ptr() + off
        betty_reset_status(self)


def betty_reset_status(ws: Workspace, stream=None) -> None:
    _check(lib().betty_reset_status(ws.ptr, ws.nbytes, _stream(stream)), "betty_reset_status")


def betty_poll_status(ws: Workspace, stream=None, raise_on_error: bool = True):
    """Synchronises the stream; returns (status, cg_iters)."""
    it = C.c_int32(0)
    st = lib().betty_poll_status(ws.ptr, _stream(stream), C.byref(it))
    if raise_on_error:
        _check(st, "betty_poll_status")
    return st, int(it.value)


def betty_lower_step(L: Level, n_steps: int, ws: Workspace, stream=None) -> None:
    _check(lib().betty_lower_step(L.ref, int(n_steps), ws.ptr, ws.nbytes, _stream(stream)), "betty_lower_step")


def betty_grad(L: Level, wrt: Level, out: torch.Tensor, ws: Workspace, stream=None) -> None:
    _check(lib().betty_grad(L.ref, wrt.ref, _ptr(out), ws.ptr, ws.nbytes, _stream(stream)), "betty_grad")


def betty_hvp(L: Level, u: torch.Tensor, Hu: torch.Tensor, ws: Workspace, stream=None) -> None:
    _check(lib().betty_hvp(L.ref, _ptr(u), _ptr(Hu), ws.ptr, ws.nbytes, _stream(stream)), "betty_hvp")


def betty_mixed_vjp(L: Level, wrt: Level, q: torch.Tensor, out: torch.Tensor, ws: Workspace, stream=None) -> None:
    _check(lib().betty_mixed_vjp(L.ref, wrt.ref, _ptr(q), _ptr(out), ws.ptr, ws.nbytes, _stream(stream)),
           "betty_mixed_vjp")


def betty_hypergrad_neumann(lower: Level, upper: Level, wrt: Level, K: int, alpha: float, out: torch.Tensor,
                            ws: Workspace, stream=None) -> None:
    _check(lib().betty_hypergrad_neumann(lower.ref, upper.ref, wrt.ref, int(K), float(alpha), _ptr(out), ws.ptr,
                                         ws.nbytes, _stream(stream)), "betty_hypergrad_neumann")


def betty_hypergrad_cg(lower: Level, upper: Level, wrt: Level, K: int, tol: float, out: torch.Tensor,
                       ws: Workspace, stream=None) -> None:
    _check(lib().betty_hypergrad_cg(lower.ref, upper.ref, wrt.ref, int(K), float(tol), _ptr(out), ws.ptr, ws.nbytes,
                                    _stream(stream)), "betty_hypergrad_cg")


def betty_hypergrad_fd(lower: Level, upper: Level, wrt: Level, eps0: float, alpha: float, out: torch.Tensor,
                       ws: Workspace, stream=None) -> None:
    _check(lib().betty_hypergrad_fd(lower.ref, upper.ref, wrt.ref, float(eps0), float(alpha), _ptr(out), ws.ptr,
                                    ws.nbytes, _stream(stream)), "betty_hypergrad_fd")


def betty_hypergrad_itd(lower: Level, upper: Level, wrt: Level, n_steps: int, out: torch.Tensor, ws: Workspace,
                        stream=None) -> None:
    _check(lib().betty_hypergrad_itd(lower.ref, upper.ref, wrt.ref, int(n_steps), _ptr(out), ws.ptr, ws.nbytes,
                                     _stream(stream)), "betty_hypergrad_itd")


def betty_chain_levels(levels: Sequence[Level], path: Sequence[int], per_edge: Sequence[MethodCfg],
                       v_in: Optional[torch.Tensor], out: torch.Tensor, accumulate: bool, ws: Workspace,
                       stream=None) -> None:
    arr = _level_array(levels)
    p = (C.c_int32 * len(path))(*[int(i) for i in path])
    cfgs = (_MethodCfg * len(per_edge))(*[m.c for m in per_edge])
    _check(lib().betty_chain_levels(arr, len(levels), p, len(path), cfgs, _ptr(v_in), _ptr(out),
                                    1 if accumulate else 0, ws.ptr, ws.nbytes, _stream(stream)), "betty_chain_levels")


def betty_hvp_logreg_static(X: torch.Tensor, w: torch.Tensor, lam: torch.Tensor, u: torch.Tensor, Hu: torch.Tensor,
                            status_dev: Optional[torch.Tensor] = None, stream=None) -> None:
    """Logistic weight-decay HVP that uses the library's built-in scratch instead of a workspace
    (for callers that cannot allocate device memory); see betty.h for the limits."""
    n, d = X.shape
    _check(lib().betty_hvp_logreg_static(_ptr(X) if n else None, n, d, _ptr(w), _ptr(lam), _ptr(u), _ptr(Hu),
                                         _ptr(status_dev), _stream(stream)), "betty_hvp_logreg_static")


def betty_gemm_bf16(M: int, N: int, pairs, Cout: torch.Tensor, ldc: int, beta: float, path: int, ws: Workspace,
                    stream=None) -> None:
    """pairs: sequence of (A, lda, a_transposed, B, ldb, b_transposed, K, alpha) with bf16 device tensors."""
    arr = (_GemmOperands * len(pairs))()
    for i, (A, lda, ta, B, ldb, tb, K, alpha) in enumerate(pairs):
        arr[i] = _GemmOperands(_ptr(A), int(lda), int(bool(ta)), _ptr(B), int(ldb), int(bool(tb)), int(K), float(alpha))
    _check(lib().betty_gemm_bf16(int(M), int(N), len(pairs), arr, _ptr(Cout), int(ldc), float(beta), int(path), ws.ptr,
                                 ws.nbytes, _stream(stream)), "betty_gemm_bf16")


def _edges(pairs):
    arr = (_Edge * max(1, len(pairs)))()
    for i, (a, b) in enumerate(pairs):
        arr[i] = _Edge(int(a), int(b))
    return arr


def betty_find_paths(n_levels: int, u2l, l2u, k: int, targets) -> list:
    """Valid paths [k, q(1), ..., q(m)] of the dataflow graph (host-only call)."""
    t = (C.c_int32 * max(1, len(targets)))(*[int(x) for x in targets])
    n_paths, n_ints = C.c_int32(0), C.c_int32(0)
    eu, el = _edges(u2l), _edges(l2u)
    _check(lib().betty_find_paths(n_levels, eu, len(u2l), el, len(l2u), int(k), t, len(targets), None, 0,
                                  C.byref(n_paths), C.byref(n_ints)), "betty_find_paths")
    buf = (C.c_int32 * max(1, n_ints.value))()
    _check(lib().betty_find_paths(n_levels, eu, len(u2l), el, len(l2u), int(k), t, len(targets), buf, n_ints.value,
                                  C.byref(n_paths), C.byref(n_ints)), "betty_find_paths")
    out, i = [], 0
    for _ in range(n_paths.value):
        ln = buf[i]
        out.append([buf[i + 1 + j] for j in range(ln)])
        i += 1 + ln
    return out


def betty_hypergrad_graph(levels: Sequence[Level], u2l, l2u, k: int, per_level: Sequence[MethodCfg], out: torch.Tensor,
                          ws: Workspace, stream=None) -> None:
    arr = _level_array(levels)
    cfgs = (_MethodCfg * len(per_level))(*[m.c for m in per_level])
    _check(lib().betty_hypergrad_graph(arr, len(levels), _edges(u2l), len(u2l), _edges(l2u), len(l2u), int(k), cfgs,
                                       _ptr(out), ws.ptr, ws.nbytes, _stream(stream)), "betty_hypergrad_graph")


def betty_engine_run(levels: Sequence[Level], u2l, l2u, per_level: Sequence[MethodCfg], unroll_steps: Sequence[int],
                     n_iterations: int, ws: Workspace, stream=None, log_capacity: int = 65536) -> list:
    """Runs the program's execution schedule (Sec. 3.3); returns the order in which problems stepped."""
    arr = _level_array(levels)
    cfgs = (_MethodCfg * len(per_level))(*[m.c for m in per_level])
    un = (C.c_int32 * len(unroll_steps))(*[int(x) for x in unroll_steps])
    log = (C.c_int32 * log_capacity)()
    n = C.c_int32(0)
    _check(lib().betty_engine_run(arr, len(levels), _edges(u2l), len(u2l), _edges(l2u), len(l2u), cfgs, un,
                                  int(n_iterations), log, log_capacity, C.byref(n), ws.ptr, ws.nbytes, _stream(stream)),
           "betty_engine_run")
    return [log[i] for i in range(min(n.value, log_capacity))]


def betty_selftest_wait_timeout(ws: Workspace, stream=None) -> None:
    _check(lib().betty_selftest_wait_timeout(ws.ptr, ws.nbytes, _stream(stream)), "betty_selftest_wait_timeout")


def betty_selftest_smem_limit(reset: bool, device: int, nbytes: int) -> bool:
    """Host-only: would a launch needing `nbytes` of dynamic shared memory on `device` set the limit?"""
    return bool(lib().betty_selftest_smem_limit(1 if reset else 0, int(device), int(nbytes)))
