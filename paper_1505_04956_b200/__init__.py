"""K-Means ASGD (Keuper & Pfreundt, arXiv 1505.04956) worker loop as CUDA kernels for B200.

`binding` wraps the C ABI of libasgd.so one to one; `inputs` draws seeded synthetic workloads;
`build` compiles the library in-tree.  Nothing here computes on the CPU.
"""
from .binding import (Asgd, AsgdConfig, AsgdError, make_config, asgd_workspace_bytes, asgd_fit_host,
                      asgd_fit_host_bytes, asgd_eval_noalloc, load, LIB_PATH, EXPORTS, PATH_AUTO, PATH_FP32, PATH_TC_FP16,
                      PATH_TC_BF16, PATH_FP32_GENERAL)

__all__ = ["Asgd", "AsgdConfig", "AsgdError", "make_config", "asgd_workspace_bytes", "asgd_fit_host",
           "asgd_fit_host_bytes", "asgd_eval_noalloc", "load", "LIB_PATH", "EXPORTS", "PATH_AUTO", "PATH_FP32", "PATH_TC_FP16",
           "PATH_TC_BF16", "PATH_FP32_GENERAL"]
