"""B200 (sm_100a) hybrid causal attention layer of Selective Attention Freezing: C-ABI library + binding."""
from .binding import (SAF_KERNEL_FWD, SAF_KERNEL_BWD, SAF_KERNEL_BWD_PREP, SAF_KERNEL_BWD_FINALIZE, SAF_KERNEL_LOGZ, SAF_KERNEL_SCALE,
                      SAF_KERNEL_PGRAD, SAF_KERNEL_FIT, SAF_KERNEL_FIT_MARGINALS, SAF_KERNEL_CALIB, SAF_KERNEL_CALIB_FINALIZE, SAF_ERR_INVALID_ARG, SAF_ERR_UNSUPPORTED,
                      SAF_ERR_CUDA, SAF_ERR_DEVICE_TIMEOUT, SAF_ERR_ARCH, SAF_ERR_NOMEM,
                      Context, SafError, SafProblem, SAF_BF16, SAF_F32, SAF_OK, load_library, make_problem,
                      saf_build_worklist, saf_pattern_logz_static, saf_version, status_string)

__all__ = ["Context", "SafError", "SafProblem", "SAF_BF16", "SAF_F32", "SAF_OK", "load_library", "make_problem",
           "saf_build_worklist", "saf_pattern_logz_static", "saf_version", "status_string"]
