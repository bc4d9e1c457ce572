// The steps on either side of the trellis pass in the paper's QAT loop (Algorithm 1): the Adam
// update of the continuous pre-image (and, optionally, of the table) and the computed Gaussian
// emission table of Section 3.1.  Element-wise, bound by HBM: 16-byte accesses, one pass.
#pragma once
#include "bcjr_common.cuh"

namespace bcjr {

// c(s) = Phi^-1((s + 1/2) / S) written out as a table (the same routine the kernels use for a null table)
__global__ void gaussian_table_kernel(float *c, int S)
{
    const int s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s < S) c[s] = gaussian_entry(s, S);
}

struct AdamParams {
    float *p;
    const float *g;
    float *m, *v;
    int64_t numel;
    float lr_c1;        // lr / (1 - beta1^t)
    float inv_c2;       // 1 / (1 - beta2^t)
    float beta1, beta2, eps;
};

__device__ __forceinline__ void adam_one(float &p, float g, float &m, float &v, const AdamParams &a)
{
    m = fmaf(a.beta1, m, (1.f - a.beta1) * g);
    v = fmaf(a.beta2, v, (1.f - a.beta2) * g * g);
    p -= a.lr_c1 * m / (sqrtf(v * a.inv_c2) + a.eps);
}

// grid-stride over float4 groups, scalar tail; grid = a multiple of the SM count
__global__ void __launch_bounds__(256) adam_kernel(AdamParams a)
{
    const int64_t n4 = a.numel / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    float4 *p4 = reinterpret_cast<float4 *>(a.p);
    const float4 *g4 = reinterpret_cast<const float4 *>(a.g);
    float4 *m4 = reinterpret_cast<float4 *>(a.m), *v4 = reinterpret_cast<float4 *>(a.v);
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += stride) {
        float4 p = p4[i], m = m4[i], v = v4[i];
        const float4 g = __ldg(g4 + i);
        adam_one(p.x, g.x, m.x, v.x, a); adam_one(p.y, g.y, m.y, v.y, a);
        adam_one(p.z, g.z, m.z, v.z, a); adam_one(p.w, g.w, m.w, v.w, a);
        p4[i] = p; m4[i] = m; v4[i] = v;
    }
    for (int64_t i = n4 * 4 + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < a.numel; i += stride) {
        float p = a.p[i], m = a.m[i], v = a.v[i];
        adam_one(p, a.g[i], m, v, a);
        a.p[i] = p; a.m[i] = m; a.v[i] = v;
    }
}

}  // namespace bcjr
