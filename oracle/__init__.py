"""FP64 CPU oracle for the TSR-Adam hot path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the CPU-baseline / reference legs of the
benchmark may import this package.  The CUDA library never does, and this
package never imports the CUDA library or its Python binding.
"""
from .tsr_oracle import (  # noqa: F401
    OracleBlock,
    adam_core,
    backproject_apply,
    backproject_one_sided,
    build,
    core_bytes,
    dense_adamw,
    exact_svd_refresh,
    num_threads,
    orth,
    project_core,
    project_one_sided,
    reexpress_moment,
    rsvd_refresh,
    sgd_core,
    sketch_bytes,
    state_elems,
    svd_jacobi,
)
