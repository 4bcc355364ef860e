"""libtsr: the TSR-Adam (two-sided low-rank Adam) optimizer hot path for NVIDIA B200.

The compute lives in libtsr.so (CUDA, sm_100a; C ABI in include/tsr.h).  This package is the
thin ctypes binding.  There is no CPU fallback: without the built library, importing the
binding's `lib()` raises.
"""
from .binding import (  # noqa: F401
    EXPORTS, Hyper, MatDesc, MatPtrs, Plan, TsrError, TSR_BF16, TSR_F32, TSR_OK, TSR_RULE_ADAM, TSR_RULE_SGD, TSR_BLOCK_REEXPRESS_MOMENT, TSR_BLOCK_ONE_SIDED,
    lib, lib_path, make_hyper, dense_adamw, DenseTensor, project_core_static, STATIC_SCRATCH_FLOATS,
)
