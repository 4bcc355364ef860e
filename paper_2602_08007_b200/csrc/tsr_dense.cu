// Dense AdamW for the parameters that are not matrix blocks (biases, normalisation weights):
// Section 3.4 of the paper updates them "in dense form", i.e. with the textbook rule of Section 3.1.
// One multi-tensor launch per batch of up to DENSE_BATCH tensors; the table of pointers travels in
// the kernel's parameter space, so the call needs no context, no workspace and no allocation.
// HBM-bound: per parameter it reads p, g, m, v and writes p, m, v (28 bytes with FP32 gradients).
#include <math.h>

#include "tsr_device.cuh"
#include "tsr_internal.h"

namespace tsr {

constexpr int DENSE_BATCH = 48;
constexpr int DENSE_CHUNK = 1 << 14;   // elements per CTA

struct DenseBatch {
    float *p[DENSE_BATCH];
    const void *g[DENSE_BATCH];
    float *m[DENSE_BATCH];
    float *v[DENSE_BATCH];
    int64_t n[DENSE_BATCH];
    int32_t chunk_begin[DENSE_BATCH + 1];   // prefix sum of chunks per tensor
    int8_t g_bf16[DENSE_BATCH];
    int32_t count;
};

__global__ void __launch_bounds__(256)
dense_adamw_kernel(const __grid_constant__ DenseBatch b, StepScalars sc, float lr)
{
    // which tensor does this chunk belong to?
    int t = 0;
    while (t + 1 < b.count && (int)blockIdx.x >= b.chunk_begin[t + 1]) ++t;
    const int64_t e0 = (int64_t)((int)blockIdx.x - b.chunk_begin[t]) * DENSE_CHUNK;
    const int64_t e1 = min(b.n[t], e0 + DENSE_CHUNK);
    float *__restrict__ P = b.p[t];
    float *__restrict__ M = b.m[t];
    float *__restrict__ V = b.v[t];
    const float *gf = (const float *)b.g[t];
    const bf16 *gb = (const bf16 *)b.g[t];
    const bool is_bf16 = b.g_bf16[t] != 0;
    // vector path: four parameters per thread and access when everything is 16-byte aligned
    const bool vec = !is_bf16 && ((((uintptr_t)P | (uintptr_t)M | (uintptr_t)V | (uintptr_t)gf) & 15) == 0);
    int64_t e_scalar = e0;
    if (vec) {
        const int64_t nv = (e1 - e0) / 4;
        for (int64_t q = threadIdx.x; q < nv; q += blockDim.x) {
            const int64_t e = e0 + 4 * q;
            const float4 g4 = *(const float4 *)(gf + e);
            float4 m4 = *(const float4 *)(M + e), v4 = *(const float4 *)(V + e), p4 = *(const float4 *)(P + e);
            const float d0 = core_update_elem(g4.x, m4.x, v4.x, sc);
            const float d1 = core_update_elem(g4.y, m4.y, v4.y, sc);
            const float d2 = core_update_elem(g4.z, m4.z, v4.z, sc);
            const float d3 = core_update_elem(g4.w, m4.w, v4.w, sc);
            p4.x = __fmaf_rn(-lr, d0, __fmul_rn(sc.decay, p4.x));
            p4.y = __fmaf_rn(-lr, d1, __fmul_rn(sc.decay, p4.y));
            p4.z = __fmaf_rn(-lr, d2, __fmul_rn(sc.decay, p4.z));
            p4.w = __fmaf_rn(-lr, d3, __fmul_rn(sc.decay, p4.w));
            *(float4 *)(M + e) = m4;
            *(float4 *)(V + e) = v4;
            *(float4 *)(P + e) = p4;
        }
        e_scalar = e0 + 4 * nv;
    }
    for (int64_t e = e_scalar + threadIdx.x; e < e1; e += blockDim.x) {
        const float g = is_bf16 ? __bfloat162float(gb[e]) : gf[e];
        float m1 = M[e], m2 = V[e];
        const float d = core_update_elem(g, m1, m2, sc);      // m_hat / (sqrt(v_hat) + eps)
        M[e] = m1;
        V[e] = m2;
        P[e] = __fmaf_rn(-lr, d, __fmul_rn(sc.decay, P[e]));  // p - lr (d + wd p), decay = 1 - lr wd
    }
}

}  // namespace tsr

using namespace tsr;

extern "C" tsr_status tsr_dense_adamw(const tsr_dense_tensor *tensors, int32_t count, const tsr_hyper *h, void *stream)
{
    if (!tensors || count < 0 || !h) return TSR_ERR_INVALID_ARG;
    if (h->step < 1 || h->rule != TSR_RULE_ADAM) return TSR_ERR_INVALID_ARG;
    if (!(h->beta1 >= 0.f && h->beta1 < 1.f) || !(h->beta2 >= 0.f && h->beta2 < 1.f)) return TSR_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i) {
        const tsr_dense_tensor &t = tensors[i];
        if (t.count < 0) return TSR_ERR_SHAPE;
        if (t.count > 0 && (!t.param || !t.grad || !t.m || !t.v)) return TSR_ERR_INVALID_ARG;
        if (t.g_dtype != TSR_F32 && t.g_dtype != TSR_BF16) return TSR_ERR_UNSUPPORTED;
    }
    StepScalars sc;
    sc.beta1 = h->beta1; sc.beta2 = h->beta2; sc.eps = h->eps;
    sc.omb1 = (float)(1.0 - (double)h->beta1);
    sc.omb2 = (float)(1.0 - (double)h->beta2);
    sc.inv_bc1 = (float)(1.0 / (1.0 - pow((double)h->beta1, (double)h->step)));
    sc.inv_bc2 = (float)(1.0 / (1.0 - pow((double)h->beta2, (double)h->step)));
    sc.decay = 1.0f - h->lr * h->weight_decay;
    sc.step_scale = h->lr;
    sc.rule = TSR_RULE_ADAM;
    int i = 0;
    while (i < count) {
        DenseBatch b;
        b.count = 0;
        b.chunk_begin[0] = 0;
        while (i < count && b.count < DENSE_BATCH) {
            const tsr_dense_tensor &t = tensors[i++];
            if (t.count == 0) continue;
            const int c = b.count++;
            b.p[c] = t.param; b.g[c] = t.grad; b.m[c] = t.m; b.v[c] = t.v; b.n[c] = t.count;
            b.g_bf16[c] = (t.g_dtype == TSR_BF16);
            b.chunk_begin[c + 1] = b.chunk_begin[c] + (int32_t)((t.count + DENSE_CHUNK - 1) / DENSE_CHUNK);
        }
        if (b.count == 0) continue;
        dense_adamw_kernel<<<b.chunk_begin[b.count], 256, 0, (cudaStream_t)stream>>>(b, sc, h->lr);
        if (cudaGetLastError() != cudaSuccess) return TSR_ERR_CUDA;
    }
    return TSR_OK;
}
