// Device-side helpers shared by the CUDA-core and the tensor-core kernels.
#pragma once
#include "tsr_internal.h"

namespace tsr {

// Square root and quotient by the hardware's approximate units (errors of about one and two units
// in the last place): deterministic, so every kernel still produces the same bits, and a third of
// the instructions of the correctly rounded forms, which matters in the fused projection epilogue.
__device__ __forceinline__ float sqrt_approx(float x)
{
    float y;
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

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
    return __fdividef(mh, __fadd_rn(sqrt_approx(vh), sc.eps));
}

}  // namespace tsr
