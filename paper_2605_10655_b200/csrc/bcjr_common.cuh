// Shared device helpers and parameter blocks of the BCJR kernels (sm_100a).
//
// Notation (paper Section 3, with the state vector compressed by the trellis structure):
//   S = 2^Lb states, K = 2^k branches, Q = S / K groups.
//   The K states q*K + b (b < K) share one predecessor set {q + j*Q : j < K}; so
//     log alpha_t(s) = e_t(s) + L_t(s >> k),   L_{t+1}(q) = LSE_j [ L_t((q + jQ) >> k) + e_t(q + jQ) ]
//     log beta_t(s)  = M_t(s & (Q-1)),         M_{t-1}(q) = LSE_b [ M_t((qK + b) & (Q-1)) + e_t(qK + b) ]
//   with e_t(s) = -(w_t - c[s])^2 / (2T)  (Eq. 4-5).  Only L and M (Q values each) are carried.
//   All kernels work in base 2: every log-domain value is a log2, lam2 = log2(e) / (2T).
//   Each step an integer "gauge" offset is subtracted from L (and M) so that magnitudes stay
//   small; the integer sums O_t, P_t are exact, so log Z and the posterior normaliser
//   D_t = log2 Z - O_t - P_t are recovered without loss.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace bcjr {

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2f(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float rcpf(float x) {
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// one instruction on sm_100a (float min/max joined the warp-reduction instruction there)
__device__ __forceinline__ float warp_max(float v) {
    float r;
    asm volatile("redux.sync.max.f32 %0, %1, 0xffffffff;" : "=f"(r) : "f"(v));
    return r;
}
// Sums of several values over the warp in one butterfly: the first rounds halve the number of values a
// lane carries (it keeps one half, sends the other), the rest run on a single value.
// Two values, 5 shuffles: lanes 0-15 return the sum of a, lanes 16-31 the sum of b.
__device__ __forceinline__ float warp_sum2_split(float a, float b, int lane) {
    const bool hi = lane & 16;
    float v = (hi ? b : a) + __shfl_xor_sync(0xffffffffu, hi ? a : b, 16);
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
// Four values, 6 shuffles: lanes 0-7 return the sum of a, lanes 8-15 of b, lanes 16-23 of c, lanes 24-31 of d.
__device__ __forceinline__ float warp_sum4_split(float a, float b, float c, float d, int lane) {
    const bool hi = lane & 16, h8 = lane & 8;
    const float rx = __shfl_xor_sync(0xffffffffu, hi ? a : c, 16);
    const float ry = __shfl_xor_sync(0xffffffffu, hi ? b : d, 16);
    const float u = (hi ? c : a) + rx, w = (hi ? d : b) + ry;
    float v = (h8 ? w : u) + __shfl_xor_sync(0xffffffffu, h8 ? u : w, 8);
#pragma unroll
    for (int o = 4; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum3_split(float a, float b, float c, int lane) { return warp_sum4_split(a, b, c, 0.f, lane); }
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Device-side status / diagnostics block (one per context, in global memory).
struct DeviceDiag {
    int status;                  // first non-zero bcjr_status raised on the device
    unsigned int max_defect;     // float bits of max |sum gamma - 1|
    unsigned int max_logz_gap;   // float bits of max |log2 Z(alpha) - log2 Z(beta)|
    int pad;
    // configuration, written by the host when an option changes (not cleared by status queries)
    unsigned long long wait_limit_ns;   // budget of one device-side wait before it gives up
    int drop_history_load;              // test hook: CTA 0 never requests its first history chunk
    int pad2;
    float c_lo, c_hi;                   // smallest and largest table entry of the call in flight (table_range_kernel)
};
constexpr size_t DIAG_STATUS_BYTES = 16;   // the part bcjr_sync_status reads and clears

__device__ __forceinline__ void diag_max(unsigned int *slot, float v) {
    // v >= 0: float ordering equals unsigned ordering of the bit patterns
    if (!(v >= 0.0f)) v = __int_as_float(0x7f800000);   // NaN or negative -> +inf so it is seen
    atomicMax(slot, __float_as_uint(v));
}

// A non-finite log Z means non-finite inputs (or a table / temperature far outside fp32 range):
// recorded once as BCJR_ENUMERIC (-7); the outputs of that block are then meaningless.
__device__ __forceinline__ void diag_check_finite(DeviceDiag *diag, float v)
{
    if (!(fabsf(v) <= 3.0e38f)) atomicCAS(&diag->status, 0, -7);
}

// Energies without the step's common part.  A weight far outside the table's range (heavy-tailed inputs) puts
// lam2 (w - c)^2 in the tens of thousands for EVERY state, and a float32 rounded at that magnitude has lost the
// differences between states that the posterior is made of.  A constant of the step is a gauge (it shifts log Z
// and nothing else), so the kernels subtract one: with wc = w clamped to [c_lo, c_hi] and delta = w - wc,
//     (w - c)^2 - delta^2 = du (du - 2 delta),   du = c - wc,
// and the log2-potential is  e'(s) = du * (du * (-lam2) + kap),  kap = 2 lam2 delta -- two fused multiply-adds, as
// many operations as the plain square, small wherever c is near the weight (or near the end of the table the
// weight lies beyond).  Inside the range delta = 0 and this IS the plain square.  log Z gets lam2 delta^2 back.
struct StepEnergy {
    float wc;       // clamped weight
    float kap;      // 2 lam2 delta
    float delta;    // w - wc
};
__device__ __forceinline__ StepEnergy step_energy(float w, float lo, float hi, float lam2)
{
    StepEnergy e;
    e.wc = fminf(fmaxf(w, lo), hi);
    e.delta = w - e.wc;
    e.kap = 2.f * lam2 * e.delta;
    return e;
}

// Computed Gaussian emission of Section 3.1: c(s) = Phi^-1((s + 1/2) / S).  The cell centre is formed in double
// (exact), the inverse CDF in single precision; antisymmetric by construction (lower half evaluated, upper half
// mirrored).  A kernel given a null table pointer uses this instead of a load.
// (not inlined: the staging loops that call it are fully unrolled)
__device__ __noinline__ static float gaussian_entry(int s, int S)
{
    const int lo = s < S / 2 ? s : S - 1 - s;
    const float x = normcdfinvf((float)(((double)lo + 0.5) / (double)S));
    return s < S / 2 ? x : -x;
}
__device__ __forceinline__ float table_entry(const float *cb, int s, int S) { return cb ? __ldg(cb + s) : gaussian_entry(s, S); }

// smallest and largest entry of the table, for step_energy: one small block, launched ahead of the sweeps
static __global__ void __launch_bounds__(1024) table_range_kernel(const float *__restrict__ cb, int S, DeviceDiag *diag)
{
    __shared__ float lo_s[32], hi_s[32];
    float lo = __int_as_float(0x7f800000), hi = __int_as_float(0xff800000);
    if (!cb) {                                   // computed emission: monotone in s
        if (threadIdx.x == 0) { diag->c_lo = gaussian_entry(0, S); diag->c_hi = gaussian_entry(S - 1, S); }
        return;
    }
    for (int s = threadIdx.x; s < S; s += blockDim.x) {
        const float c = __ldg(cb + s);
        lo = fminf(lo, c); hi = fmaxf(hi, c);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if ((threadIdx.x & 31) == 0) { lo_s[threadIdx.x >> 5] = lo; hi_s[threadIdx.x >> 5] = hi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < (int)(blockDim.x >> 5); ++i) { lo = fminf(lo, lo_s[i]); hi = fmaxf(hi, hi_s[i]); }
        diag->c_lo = lo; diag->c_hi = hi;
    }
}

struct FwdParams {
    const float *W;          // [B*n]
    const float *cb;         // [S]
    const float *cb_beta;    // vector-emission kernels only: the table regrouped [K][Q][V] for the beta sweep
    float *soft;             // [B*n]
    float *soft_copy;        // [B*n] context-owned copy, read again by the backward pass
    float *logZ;             // [B] or null (natural log)
    float *hist;             // [grid][n*Q] gauge-fixed L_t, t = 1..n
    int *stepO;              // [grid][n+2] cumulative integer offsets O_t
    float *msg;              // [grid][2*Q] message ping-pong in global memory, or null (shared)
    float *blk_defect;       // [B] max_t |sum_s gamma_t(s) - 1| of every block, or null (not recorded)
    DeviceDiag *diag;
    int64_t B;
    int Lb, n;
    float lam2;              // log2(e) / (2T)
    int hist_every;          // checkpointing kernels: L_t is kept for every hist_every-th step (1 = every step)
};

struct BwdParams {
    const float *W;
    const float *cb;
    const float *cb_beta;    // vector-emission kernels only: the table regrouped [K][Q][V]
    const float *g;          // upstream gradient [B*n]
    const float *soft;       // saved soft codeword [B*n]
    float *gW;               // [B*n]
    float *gc_part;          // [grid][S] per-CTA partial of grad_codebook
    float *hist;             // [grid][2*n*Q]: L_t then Atilde_t
    int *stepO;
    float *msg;              // [grid][4*Q] or null
    DeviceDiag *diag;
    int64_t B;
    int Lb, n;
    float lam2;
    float invT;              // 1/T
};

struct VitParams {
    const float *W;
    const float *cb;
    uint8_t *path_bits;      // or null
    int64_t path_stride;
    uint16_t *states;        // or null
    float *hard;             // or null
    uint8_t *bp;             // [grid][n*Q] best branch per group per step
    double *msg;             // [grid][2*Q] or null (shared)
    int *path_ws;            // [grid][n] state sequence scratch
    DeviceDiag *diag;
    int64_t B;
    int Lb, n;
};

}  // namespace bcjr
