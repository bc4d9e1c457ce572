// Incoherence processing around the trellis pass (Section 3.1; Section 4, "Quantization
// configuration"): a random-sign Hadamard rotation on both sides of the weight matrix and a scale
// per group of 16 elements.  The paper names both without formulas; the forms used are
//     W~ = H_m diag(sL) W diag(sR) H_n / sqrt(m n),      W = diag(sL) H_m W~ H_n diag(sR) / sqrt(m n)
// with Sylvester-ordered Walsh-Hadamard matrices (entries +-1, H H = size I), and
//     scale(group) = sqrt(mean of the 16 squares),  W_scaled = W / scale.
// All of it is one or a few passes over the matrix: bound by HBM / L2 bandwidth.
//
// Fast Walsh-Hadamard transform in radix-8 passes: a pass takes three index bits [o, o+3), every
// thread holds the eight elements that differ in those bits and runs three butterfly stages in
// registers.  Rows (length n <= 8192) are transformed in shared memory, one row per CTA at a time;
// columns are transformed in place in global memory, one pass per launch, each thread working on
// eight rows x four adjacent columns (the matrix of a layer fits the 126 MB L2).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace bcjr {

// stages for bits s with first <= s < 3 of an 8-point transform (first = 0: all three)
template <typename T>
__device__ __forceinline__ void fwht8(T (&v)[8], int first)
{
    if (first <= 0) {
#pragma unroll
        for (int j = 0; j < 8; j += 2) { const T a = v[j], b = v[j + 1]; v[j] = a + b; v[j + 1] = a - b; }
    }
    if (first <= 1) {
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (!(j & 2)) { const T a = v[j], b = v[j + 2]; v[j] = a + b; v[j + 2] = a - b; }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) { const T a = v[j], b = v[j + 4]; v[j] = a + b; v[j + 4] = a - b; }
}

struct F4 {
    float4 f;
    __device__ __forceinline__ F4 operator+(const F4 &o) const { return F4{make_float4(f.x + o.f.x, f.y + o.f.y, f.z + o.f.z, f.w + o.f.w)}; }
    __device__ __forceinline__ F4 operator-(const F4 &o) const { return F4{make_float4(f.x - o.f.x, f.y - o.f.y, f.z - o.f.z, f.w - o.f.w)}; }
};

// shared-memory index with eight floats of padding per 64: keeps the stride-8 pass off a single bank group
__device__ __forceinline__ int rht_pad(int i) { return i + ((i >> 6) << 3); }

// Rows: out[r][:] = FWHT(in[r][:] * (pre ? s : 1)) * scale * (pre ? 1 : s);  n = 2^LOGN, blockDim = n / 8
template <int LOGN>
__global__ void fwht_rows_kernel(const float *in, float *out, const float *s, int m, float scale, int pre)
{
    constexpr int N = 1 << LOGN;
    extern __shared__ float row[];
    const int t = threadIdx.x;
    for (int r = blockIdx.x; r < m; r += gridDim.x) {
        const float *src = in + (size_t)r * N;
        float *dst = out + (size_t)r * N;
        float v[8];
        {   // bits 0..2 straight from global memory: eight consecutive elements per thread
            // plain loads: `out` may be `in` (in place), so the row is not read-only for the kernel
            const float4 a = reinterpret_cast<const float4 *>(src)[2 * t], b = reinterpret_cast<const float4 *>(src)[2 * t + 1];
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
            if (pre) {
                const float4 sa = __ldg(reinterpret_cast<const float4 *>(s) + 2 * t), sb = __ldg(reinterpret_cast<const float4 *>(s) + 2 * t + 1);
                v[0] *= sa.x; v[1] *= sa.y; v[2] *= sa.z; v[3] *= sa.w; v[4] *= sb.x; v[5] *= sb.y; v[6] *= sb.z; v[7] *= sb.w;
            }
            fwht8(v, 0);
        }
        if (LOGN == 3) {
#pragma unroll
            for (int j = 0; j < 8; ++j) dst[j] = v[j] * scale * (pre ? 1.f : s[j]);
            continue;
        }
        {
            float *p = row + rht_pad(8 * t);
            *reinterpret_cast<float4 *>(p) = make_float4(v[0], v[1], v[2], v[3]);
            *reinterpret_cast<float4 *>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
        }
        __syncthreads();
        // full radix-8 passes on bits [o, o+3), then one last pass on the top three bits that runs
        // only the stages of the bits not done yet; the last pass writes to global memory
        int o = 3;
        for (;; o += 3) {
            const bool last = o + 3 >= LOGN;
            const int oo = last ? LOGN - 3 : o;                 // bit offset of this pass
            const int first = o - oo;                            // stages below `first` were done by earlier passes
            const int lo = t & ((1 << oo) - 1), hi = t >> oo;
            const int base = (hi << (oo + 3)) | lo;
#pragma unroll
            for (int j = 0; j < 8; ++j) v[j] = row[rht_pad(base + (j << oo))];
            fwht8(v, first);
            if (last) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int i = base + (j << oo);
                    dst[i] = v[j] * scale * (pre ? 1.f : __ldg(s + i));
                }
                break;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) row[rht_pad(base + (j << oo))] = v[j];
            __syncthreads();
        }
        __syncthreads();                                         // the row buffer is reused by the next row
    }
}

// Columns, one radix-8 pass over row-index bits [o, o+3), in place: thread = (group of 8 rows, 4 adjacent columns).
// first: stages below it are skipped (last, partial pass).  sign_mode 1: multiply the inputs by s[row]
// (first pass of the forward rotation); 2: multiply the outputs by s[row] (last pass of the inverse).
__global__ void __launch_bounds__(256) fwht_cols_pass_kernel(float *W, const float *s, int m, int n4, int o, int first,
                                                                float scale, int sign_mode)
{
    const int64_t total = (int64_t)(m >> 3) * n4;
    for (int64_t id = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; id < total; id += (int64_t)gridDim.x * blockDim.x) {
        const int c4 = (int)(id % n4);
        const int g = (int)(id / n4);
        const int lo = g & ((1 << o) - 1), hi = g >> o;
        const int base = (hi << (o + 3)) | lo;
        float4 *p = reinterpret_cast<float4 *>(W) + c4;
        F4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int r = base + (j << o);
            v[j].f = p[(size_t)r * n4];
            if (sign_mode == 1) { const float sg = __ldg(s + r); v[j].f.x *= sg; v[j].f.y *= sg; v[j].f.z *= sg; v[j].f.w *= sg; }
        }
        fwht8(v, first);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int r = base + (j << o);
            const float k = scale * (sign_mode == 2 ? __ldg(s + r) : 1.f);
            p[(size_t)r * n4] = make_float4(v[j].f.x * k, v[j].f.y * k, v[j].f.z * k, v[j].f.w * k);
        }
    }
}

// scales[g] = sqrt(mean of the 16 squares of group g); out = W / scale (0 where the group is all zero)
__global__ void __launch_bounds__(256) group_scale_kernel(const float *W, float *scales, float *out, int64_t groups)
{
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += (int64_t)gridDim.x * blockDim.x) {
        const float4 *p = reinterpret_cast<const float4 *>(W) + 4 * g;
        float4 v[4];
        float ss = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) { v[i] = __ldg(p + i); ss += v[i].x * v[i].x + v[i].y * v[i].y + v[i].z * v[i].z + v[i].w * v[i].w; }
        const float sc = sqrtf(ss * (1.f / 16.f));
        const float inv = sc > 0.f ? 1.f / sc : 0.f;
        scales[g] = sc;
        float4 *q = reinterpret_cast<float4 *>(out) + 4 * g;
#pragma unroll
        for (int i = 0; i < 4; ++i) q[i] = make_float4(v[i].x * inv, v[i].y * inv, v[i].z * inv, v[i].w * inv);
    }
}

// out = W_scaled * scale of its group
__global__ void __launch_bounds__(256) group_unscale_kernel(const float *Ws, const float *scales, float *out, int64_t groups)
{
    for (int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; g < groups; g += (int64_t)gridDim.x * blockDim.x) {
        const float4 *p = reinterpret_cast<const float4 *>(Ws) + 4 * g;
        float4 *q = reinterpret_cast<float4 *>(out) + 4 * g;
        const float sc = __ldg(scales + g);
#pragma unroll
        for (int i = 0; i < 4; ++i) { const float4 v = __ldg(p + i); q[i] = make_float4(v.x * sc, v.y * sc, v.z * sc, v.w * sc); }
    }
}

}  // namespace bcjr
