"""B200 (sm_100a) library for the hypergradient path of gradient-based multilevel optimisation
(arXiv 2207.02849): a C-ABI shared library of hand-written CUDA kernels plus this thin ctypes
binding.  Importing the package does not load the library; the first call does, and fails
loudly when the library is missing (there is no CPU fallback)."""
from .binding import (  # noqa: F401
    BettyError, Level, betty_gemm_bf16, MethodCfg, Workspace, betty_chain_levels, betty_grad, betty_hvp,
    betty_hvp_logreg_static, betty_hypergrad_cg, betty_engine_run, betty_find_paths, betty_hypergrad_fd, betty_hypergrad_graph, betty_hypergrad_itd, betty_hypergrad_neumann, betty_kernel_launches,
    betty_lower_step,
    betty_mixed_vjp, betty_poll_status, betty_reset_status, betty_selftest_smem_limit, betty_selftest_wait_timeout,
    betty_status_string,
    betty_workspace_size, lib, lib_path,
)
from . import binding as _b
from . import data_parallel  # noqa: F401

for _k, _v in vars(_b).items():
    if _k.startswith(("BETTY_", "LOSS_", "PARAM_", "ACT_")):
        globals()[_k] = _v
