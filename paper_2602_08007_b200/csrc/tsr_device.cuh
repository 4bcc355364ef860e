// Device-side helpers shared by the CUDA-core and the tensor-core kernels.
#pragma once
#include "tsr_internal.h"

namespace tsr {

// Core-space update of one entry (Section 3.4: moments, bias correction, normalised core; for
// the SGD rule of Algorithm 2 only the momentum).  Every rounding step is explicit so that all
// kernels that call it produce identical bits.
__device__ __forceinline__ float core_update_elem(float c, float &m1, float &m2, const StepScalars &sc)
{
    if (sc.rule == TSR_RULE_SGD) {
        m1 = __fmaf_rn(sc.beta1, m1, __fmul_rn(sc.omb1, c));
        return m1;
    }
    m1 = __fmaf_rn(sc.beta1, m1, __fmul_rn(sc.omb1, c));
    m2 = __fmaf_rn(sc.beta2, m2, __fmul_rn(sc.omb2, __fmul_rn(c, c)));
    const float mh = __fmul_rn(m1, sc.inv_bc1);
    const float vh = __fmul_rn(m2, sc.inv_bc2);
    return __fdiv_rn(mh, __fadd_rn(__fsqrt_rn(vh), sc.eps));
}

}  // namespace tsr
