// Pipe-rate micro-benchmarks: the denominators of the roofline the benchmark reports.
//
// The trellis recursions are bound by the special-function unit (ex2 / lg2 / rcp), the FP32
// pipe (packed f32x2 arithmetic) and, in the two-CTA backward kernel, by the per-step exchange
// between the CTAs of a cluster.  None of these has a vendor-stated figure one could divide by
// with a clear conscience (clocks sag under load, packed instructions occupy the pipe two
// cycles), so bcjr_measure_pipe_peaks measures them on the device the benchmark runs on, in
// well under a second:
//   - register-only chains (512 threads per SM, 8 independent chains per thread) for ex2, lg2,
//     fma.f32, fma.f32x2 and fma.f32x2 with one integer instruction beside each (does a packed instruction, two
//     cycles on the FP32 pipe, also hold the issue port for two?) (rcp shares the unit with ex2 and lg2; a chain of reciprocals is not measured
//     because the assembler simplifies it): results per clock per SM (clock64) and per second (CUDA events
//     over the whole grid, so the clock the GPU actually ran at is part of the number);
//   - st.async.v4 between the two CTAs of a cluster, both sending, on every SM: bytes landed per
//     clock per SM;
//   - one CTA-wide synchronisation round of 16 warps: named barrier, and mbarrier with one
//     arrival per warp and all warps polling.
// Every wait in here is bounded; a wait that runs out is reported as BCJR_ETIMEOUT.
#include "../../include/bcjr_microbench.h"

#include <cuda_runtime.h>

#include "bcjr_ptx.cuh"

using namespace bcjr;

namespace {

constexpr int MB_THREADS = 512, MB_CHAINS = 8;

enum { OP_EX2 = 0, OP_LG2, OP_FMA, OP_FMA2, OP_FMA2_ALU, OP_FMA2_MAX, OP_FMA2_EX2, OP_FMA2_F64, OP_COUNT };

template <int OP>
__global__ void __launch_bounds__(MB_THREADS, 1) chain_kernel(float *sink, unsigned long long *clk, int iters)
{
    float x[MB_CHAINS];
    float2 p[MB_CHAINS];
    unsigned u[MB_CHAINS];
    double dd[MB_CHAINS / 2];
#pragma unroll
    for (int i = 0; i < MB_CHAINS / 2; ++i) dd[i] = 1.0 + threadIdx.x * 1e-6 + i;
#pragma unroll
    for (int i = 0; i < MB_CHAINS; ++i) {
        x[i] = 1.0f + threadIdx.x * 1e-3f + i;
        p[i] = make_float2(x[i], x[i] + 1.f);
        u[i] = threadIdx.x * 2654435761u + i;
    }
    const float2 c1 = make_float2(1.0001f, 0.9999f), c2 = make_float2(1e-3f, 2e-3f);
    __syncthreads();
    const long long t0 = clock64();
    for (int it = 0; it < iters; ++it) {
        const float vary = 1.0f + 1e-3f * (float)it;               // an operand that changes every iteration, so that nothing folds
#pragma unroll
        for (int i = 0; i < MB_CHAINS; ++i) {
            if (OP == OP_EX2) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[i]));
            if (OP == OP_LG2) asm volatile("lg2.approx.ftz.f32 %0, %0;" : "+f"(x[i]));
            if (OP == OP_FMA) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(x[i]) : "f"(c1.x), "f"(c2.x));
            if (OP == OP_FMA2_ALU) asm volatile("xor.b32 %0, %0, %1;" : "+r"(u[i]) : "r"(0x9e3779b9u + (unsigned)it));   // an integer instruction per packed one
            if (OP == OP_FMA2_MAX) asm volatile("max.f32 %0, %0, %1;" : "+f"(x[i]) : "f"(vary));                          // a float maximum (integer pipe) per packed one
            if (OP == OP_FMA2_EX2 && (i & 3) == 0) asm volatile("ex2.approx.ftz.f32 %0, %0;" : "+f"(x[i]));                // a special-function instruction per four packed ones
            if (OP == OP_FMA2_F64 && (i & 1) == 0) asm volatile("fma.rn.f64 %0, %0, %1, %2;" : "+d"(dd[i >> 1]) : "d"(1.0000001), "d"(1e-9));   // an fp64 instruction per two packed ones
            if (OP >= OP_FMA2)
                asm volatile("{ .reg .b64 ra, rb, rc; mov.b64 ra, {%0, %1}; mov.b64 rb, {%2, %3}; mov.b64 rc, {%4, %5}; "
                             "fma.rn.f32x2 ra, ra, rb, rc; mov.b64 {%0, %1}, ra; }"
                             : "+f"(p[i].x), "+f"(p[i].y) : "f"(c1.x), "f"(c1.y), "f"(c2.x), "f"(c2.y));
        }
    }
    const long long t1 = clock64();
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < MB_CHAINS; ++i) s += x[i] + p[i].x + p[i].y + (float)(u[i] & 255u) + (float)dd[i >> 1];
    sink[blockIdx.x * MB_THREADS + threadIdx.x] = s;
    if (threadIdx.x == 0 && blockIdx.x == 0) clk[OP] = (unsigned long long)(t1 - t0);
}

// Two-CTA clusters, every thread sends `rounds` 16-byte st.async to the peer; the clock stops when all the bytes
// addressed to this CTA have landed (its mbarrier phase completes).
constexpr int XCHG_LAND_FLOATS = 16384;   // 64 KB landing zone
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(MB_THREADS, 1)
exchange_kernel(int rounds, unsigned long long *clk, int *err)
{
    extern __shared__ __align__(128) float land[];
    __shared__ __align__(8) unsigned long long bar;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t peer = cluster_ctarank() ^ 1u;
    const uint32_t bar_u = smem_u32(&bar);
    if (tid == 0) {
        mbar_init(bar_u, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (tid == 0) mbar_expect_tx(bar_u, (uint32_t)rounds * MB_THREADS * 16u);
    cluster_sync();
    const uint32_t pbar = mapa_u32(bar_u, peer), pdst = mapa_u32(smem_u32(land), peer);
    const long long t0 = clock64();
    for (int r = 0; r < rounds; ++r) {
        const uint32_t off = (uint32_t)(((r & 7) * 16 + warp) * 512 + lane * 16);
        st_async_v4(pdst + off, 1.f, 2.f, (float)r, 4.f, pbar);
    }
    bool ok = false;
    for (int it = 0; it < (1 << 22) && !ok; ++it) ok = mbar_try_wait(bar_u, 0u);
    const long long t1 = clock64();
    if (!ok && tid == 0) *err = 1;
    if (blockIdx.x == 0 && tid == 0) clk[0] = (unsigned long long)(t1 - t0);
    __syncthreads();
    cluster_sync();                       // nobody leaves while a peer may still be sending to it
}

template <int MODE>   // 0: named barrier, 1: mbarrier with one arrival per warp, every warp polling
__global__ void __launch_bounds__(MB_THREADS, 1) sync_kernel(int rounds, unsigned long long *clk, int *err)
{
    __shared__ __align__(8) unsigned long long bar[2];
    const int tid = threadIdx.x, lane = tid & 31;
    const uint32_t b0 = smem_u32(&bar[0]);
    if (tid == 0) {
        for (int s = 0; s < 2; ++s) mbar_init(b0 + 8u * s, MB_THREADS / 32);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t phase = 0;
    bool bad = false;
    const long long t0 = clock64();
    for (int r = 0; r < rounds && !bad; ++r) {
        if (MODE == 0) {
            asm volatile("bar.sync 1, 512;" ::: "memory");
        } else {
            const uint32_t b = b0 + 8u * (r & 1);
            __syncwarp();
            if (lane == 0) mbar_arrive_local(b);
            bool ok = false;
            for (int it = 0; it < (1 << 20) && !ok; ++it) ok = mbar_try_wait(b, (phase >> (r & 1)) & 1u);
            bad = !ok;
            phase ^= 1u << (r & 1);
        }
    }
    const long long t1 = clock64();
    if (bad) *err = 1;
    if (blockIdx.x == 0 && tid == 0) clk[0] = (unsigned long long)(t1 - t0);
}

struct DeviceScope {
    int prev = -1;
    bool ok = false;
    explicit DeviceScope(int dev) { ok = cudaGetDevice(&prev) == cudaSuccess && (prev == dev || cudaSetDevice(dev) == cudaSuccess); }
    ~DeviceScope() { if (ok && prev >= 0) cudaSetDevice(prev); }
};

template <int OP>
bool run_chain(int sms, int iters, float *sink, unsigned long long *clk, cudaStream_t st, double *per_clk_sm, double *per_s)
{
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) return false;
    double best_ms = 1e30;
    chain_kernel<OP><<<sms, MB_THREADS, 0, st>>>(sink, clk, iters);            // warm-up
    for (int rep = 0; rep < 3; ++rep) {
        cudaEventRecord(e0, st);
        chain_kernel<OP><<<sms, MB_THREADS, 0, st>>>(sink, clk, iters);
        cudaEventRecord(e1, st);
        if (cudaEventSynchronize(e1) != cudaSuccess) { cudaEventDestroy(e0); cudaEventDestroy(e1); return false; }
        float ms = 0.f;
        cudaEventElapsedTime(&ms, e0, e1);
        if (ms < best_ms) best_ms = ms;
    }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    unsigned long long h = 0;
    if (cudaMemcpy(&h, clk + OP, 8, cudaMemcpyDeviceToHost) != cudaSuccess || h == 0) return false;
    const double per_sm = (double)MB_THREADS * MB_CHAINS * iters;
    *per_clk_sm = per_sm / (double)h;
    *per_s = per_sm * sms / (best_ms * 1e-3);
    return true;
}

}  // namespace

extern "C" bcjr_status bcjr_measure_pipe_peaks(int device, bcjr_pipe_peaks *out, void *cuda_stream)
{
    if (!out) return BCJR_EINVAL;
    *out = bcjr_pipe_peaks{};
    DeviceScope scope(device);
    if (!scope.ok) { cudaGetLastError(); return BCJR_ECUDA; }
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || sms < 2) {
        cudaGetLastError();
        return BCJR_ECUDA;
    }
    cudaStream_t st = (cudaStream_t)cuda_stream;
    float *sink = nullptr;
    unsigned long long *clk = nullptr;
    int *err = nullptr;
    if (cudaMalloc(&sink, (size_t)sms * MB_THREADS * 4) != cudaSuccess || cudaMalloc(&clk, 64 * 8) != cudaSuccess ||
        cudaMalloc(&err, 4) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(sink); cudaFree(clk); cudaFree(err);
        return BCJR_ENOMEM;
    }
    cudaMemsetAsync(clk, 0, 64 * 8, st);
    cudaMemsetAsync(err, 0, 4, st);
    const int iters = 2000;
    bool ok = true;
    // let the clocks settle at their level under load before anything is timed (a GPU that was idle takes a few
    // milliseconds to get there, and a peak measured on the way up would flatter every fraction quoted against it)
    for (int rep = 0; rep < 40; ++rep) chain_kernel<OP_EX2><<<sms, MB_THREADS, 0, st>>>(sink, clk, iters);
    double per_s = 0.0, dummy = 0.0;
    ok = ok && run_chain<OP_EX2>(sms, iters, sink, clk, st, &out->ex2_per_clk_sm, &per_s);
    out->ex2_gops = per_s * 1e-9;
    ok = ok && run_chain<OP_LG2>(sms, iters, sink, clk, st, &out->lg2_per_clk_sm, &dummy);
    ok = ok && run_chain<OP_FMA>(sms, iters, sink, clk, st, &out->fma_f32_per_clk_sm, &dummy);
    ok = ok && run_chain<OP_FMA2>(sms, iters, sink, clk, st, &out->fma_f32x2_per_clk_sm, &per_s);
    out->fma_f32x2_gops = per_s * 1e-9;
    // one integer instruction (another pipe) beside every packed one: pairs per clock per SM again.  The same figure as
    // without them says the two pipes overlap; two thirds of it says they do not.
    ok = ok && run_chain<OP_FMA2_ALU>(sms, iters, sink, clk, st, &out->fma_f32x2_with_alu_per_clk_sm, &dummy);
    // the same question for a float maximum (integer pipe), a special-function instruction per four packed ones and
    // an fp64 instruction per two: packed pairs per clock per SM in each mix
    ok = ok && run_chain<OP_FMA2_MAX>(sms, iters, sink, clk, st, &out->fma_f32x2_with_max_per_clk_sm, &dummy);
    ok = ok && run_chain<OP_FMA2_EX2>(sms, iters, sink, clk, st, &out->fma_f32x2_with_ex2_per_clk_sm, &dummy);
    ok = ok && run_chain<OP_FMA2_F64>(sms, iters, sink, clk, st, &out->fma_f32x2_with_f64_per_clk_sm, &dummy);
    // the clock the chains ran at: results per second / (results per clock per SM * SMs)
    if (ok && out->ex2_per_clk_sm > 0.0) out->sm_clock_mhz = out->ex2_gops * 1e3 / (out->ex2_per_clk_sm * sms);
    out->num_sms = sms;
    unsigned long long h = 0;
    if (ok) {
        const int rounds = 96;            // 768 KB per CTA: the transaction count of an mbarrier stays below 2^20
        const size_t smem = (size_t)XCHG_LAND_FLOATS * 4;
        ok = cudaFuncSetAttribute(exchange_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess;
        for (int rep = 0; rep < 2 && ok; ++rep) exchange_kernel<<<sms / 2 * 2, MB_THREADS, smem, st>>>(rounds, clk + 32, err);
        ok = ok && cudaStreamSynchronize(st) == cudaSuccess && cudaMemcpy(&h, clk + 32, 8, cudaMemcpyDeviceToHost) == cudaSuccess && h > 0;
        if (ok) out->st_async_bytes_per_clk_sm = (double)rounds * MB_THREADS * 16 / (double)h;
    }
    if (ok) {
        const int rounds = 2000;
        for (int rep = 0; rep < 2; ++rep) sync_kernel<0><<<sms, MB_THREADS, 0, st>>>(rounds, clk + 33, err);
        for (int rep = 0; rep < 2; ++rep) sync_kernel<1><<<sms, MB_THREADS, 0, st>>>(rounds, clk + 34, err);
        unsigned long long hb[2] = {0, 0};
        ok = cudaStreamSynchronize(st) == cudaSuccess && cudaMemcpy(hb, clk + 33, 16, cudaMemcpyDeviceToHost) == cudaSuccess;
        if (ok) {
            out->cta_barrier_clk = (double)hb[0] / rounds;
            out->mbarrier_round_clk = (double)hb[1] / rounds;
        }
    }
    int herr = 0;
    const bool copied = cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost) == cudaSuccess;
    cudaFree(sink); cudaFree(clk); cudaFree(err);
    if (!ok || !copied) { cudaGetLastError(); return BCJR_ECUDA; }
    return herr ? BCJR_ETIMEOUT : BCJR_OK;
}
