// Kernels for the trellis with VECTOR emissions: every state emits V numbers per step, a step
// consumes V weights and shifts KB = k*V bits into the state (the paper's "L=16, k=2, V=2"
// configuration: 128 steps per 256-weight block, 16 predecessors per state).
//
//   e_t(s) = -(1/(2T)) sum_v (w[V t + v] - c[s][v])^2        (Eq. 4 summed over the step's weights)
//   soft[V t + v] = sum_s c[s][v] gamma_t(s)                  (Eq. 7 per emitted component)
//
// Same structure as the scalar generic kernels (one thread block per weight block, a thread owns
// groups q = tid, tid + blockDim, ..., compressed messages L_t / M_t of Q = S / 2^KB entries in
// shared memory, gauge-fixed history of L_t in a per-CTA global buffer), with the per-step scalars
// (weight, upstream gradient, soft value, posterior sums) widened to V components.  The table is
// laid out [S][V] and read through the read-only cache.  The alpha sweep reads entry q + jQ for
// consecutive q (coalesced); the beta sweep reads entry qK + b, which for consecutive q is a
// 128-byte stride, so it reads a copy regrouped as [b][q][V] (made once per call by
// regroup_table_kernel) and keeps the per-CTA gradient accumulators in the same layout.
#pragma once
#include "bcjr_generic.cuh"

namespace bcjr {

template <int V>
struct VecOf {
    float v[V];
};
// V consecutive floats; for V = 2 one 8-byte load (the host checks the alignment of every array)
template <int V>
__device__ __forceinline__ VecOf<V> load_vec(const float *p)
{
    VecOf<V> r;
    if (V == 2) {
        const float2 t = __ldg(reinterpret_cast<const float2 *>(p));
        r.v[0] = t.x; r.v[V - 1] = t.y;
    } else {
#pragma unroll
        for (int i = 0; i < V; ++i) r.v[i] = __ldg(p + i);
    }
    return r;
}
// squared distance of the step's weights to the entry of state s
template <int V>
__device__ __forceinline__ float dist2(const VecOf<V> &w, const VecOf<V> &c)
{
    float e = 0.f;
#pragma unroll
    for (int i = 0; i < V; ++i) { const float d = w.v[i] - c.v[i]; e = fmaf(d, d, e); }
    return e;
}

// dst[(b*Q + q)*V + v] = src[((q << KB) + b)*V + v]
__global__ void regroup_table_kernel(const float *src, float *dst, int S, int KB, int V)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= S * V) return;
    const int v = i % V, u = i / V, Q = S >> KB, b = u / Q, q = u % Q;
    dst[i] = src[(size_t)((q << KB) + b) * V + v];
}
// Deterministic sum of the per-CTA gradient partials ([K][Q][V] each) into the table's own layout.
__global__ void reduce_gc_vec_kernel(const float *part, int nparts, int S, int KB, int V, float *out)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;       // index in the regrouped layout
    if (i >= S * V) return;
    const int v = i % V, u = i / V, Q = S >> KB, b = u / Q, q = u % Q;
    float acc = 0.f;
    for (int r = 0; r < nparts; ++r) acc += part[(size_t)r * S * V + i];
    out[(size_t)((q << KB) + b) * V + v] = acc;
}

constexpr int VEC_PART = 8;            // floats per per-warp slot of posterior sums (>= 2 + 2 V)
constexpr int VEC_SMEM_HEADER = 640;   // floats ahead of the message buffers: wmax 64, sums 512, log Z partials 32

// --------------------------------------------------------------------------------------
// Forward call: alpha sweep, log Z, beta sweep fused with the posterior and Eq. 7.
// p.n = weights per block (a multiple of V); nt = n / V steps.
// --------------------------------------------------------------------------------------
template <int KB, int V>
__global__ void __launch_bounds__(GEN_MAX_THREADS) fwd_vec_kernel(FwdParams p)
{
    constexpr int K = 1 << KB;
    extern __shared__ float smem[];
    const int S = 1 << p.Lb, Q = S >> KB, n = p.n, nt = n / V;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const float NEG_INF = __int_as_float(0xff800000);
    float *wmax = smem;             // [2][32]
    float *part = smem + 64;        // [2][32][VEC_PART]
    float *lzpart = smem + 64 + 2 * 32 * VEC_PART;     // [32]
    float *msgbuf = p.msg ? p.msg + (size_t)blockIdx.x * 2 * Q : smem + VEC_SMEM_HEADER;
    float *hist = p.hist + (size_t)blockIdx.x * nt * Q;
    int *stepO = p.stepO + (size_t)blockIdx.x * (nt + 2);
    const float lam2 = p.lam2;
    float defect = 0.f, zgap = 0.f;

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w = p.W + blk * n;
        float *Lin = msgbuf, *Lout = msgbuf + Q;
        for (int q = tid; q < Q; q += nthr) { Lin[q] = 0.f; hist[q] = 0.f; }   // L_1 = 0: free first state
        if (tid == 0) stepO[1] = 0;
        int O = 0;
        float off = 0.f, cmax = 0.f;
        __syncthreads();
        for (int t = 1; t <= nt; ++t) {
            const VecOf<V> wt = load_vec<V>(w + (size_t)(t - 1) * V);
            float tmax = NEG_INF;
            for (int q = tid; q < Q; q += nthr) {
                float a[K], m = NEG_INF;
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    const int s = q + j * Q;
                    a[j] = fmaf(dist2<V>(wt, load_vec<V>(p.cb + (size_t)s * V)), -lam2, Lin[s >> KB]);
                    m = fmaxf(m, a[j]);
                }
                float sum = 0.f;
#pragma unroll
                for (int j = 0; j < K; ++j) sum += ex2f(a[j] - m);
                const float out = m + lg2f(sum) - off;
                Lout[q] = out;
                if (t < nt) hist[(size_t)t * Q + q] = out;
                tmax = fmaxf(tmax, out);
            }
            tmax = warp_max(tmax);
            if (lane == 0) wmax[(t & 1) * 32 + warp] = tmax;
            O += (int)off;
            if (tid == 0) stepO[t + 1] = O;
            __syncthreads();
            cmax = warp_max(lane < nwarp ? wmax[(t & 1) * 32 + lane] : NEG_INF);
            off = rintf(cmax);
            float *sw = Lin; Lin = Lout; Lout = sw;
        }
        float ssum = 0.f;
        for (int q = tid; q < Q; q += nthr) ssum += ex2f(Lin[q] - cmax);
        ssum = warp_sum(ssum);
        if (lane == 0) lzpart[warp] = ssum;
        __syncthreads();
        float tot = 0.f;
        for (int i = 0; i < nwarp; ++i) tot += lzpart[i];
        const float lsefin = cmax + lg2f(tot);
        if (tid == 0) diag_check_finite(p.diag, lsefin);
        const int Ofin = O;
        if (tid == 0 && p.logZ) p.logZ[blk] = (float)(((double)Ofin + (double)lsefin) * 0.6931471805599453);
        float *Min = msgbuf, *Mout = msgbuf + Q;
        for (int q = tid; q < Q; q += nthr) Min[q] = 0.f;                      // M_nt = 0: free last state
        int P = 0;
        float offM = 0.f;
        __syncthreads();
        for (int t = nt; t >= 1; --t) {
            const VecOf<V> wt = load_vec<V>(w + (size_t)(t - 1) * V);
            const float D = (float)(Ofin - stepO[t] - P) + lsefin;
            float num[V], den = 0.f, tmax = NEG_INF;
#pragma unroll
            for (int v = 0; v < V; ++v) num[v] = 0.f;
            for (int q = tid; q < Q; q += nthr) {
                const float Ls = hist[(size_t)(t - 1) * Q + q];
                VecOf<V> c[K];
                float u[K], m = NEG_INF;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const int s = q * K + b;
                    c[b] = load_vec<V>(p.cb_beta + ((size_t)b * Q + q) * V);
                    u[b] = fmaf(dist2<V>(wt, c[b]), -lam2, Min[s & (Q - 1)]);
                    m = fmaxf(m, u[b]);
                }
                float sum = 0.f, craw[V];
#pragma unroll
                for (int v = 0; v < V; ++v) craw[v] = 0.f;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const float pb = ex2f(u[b] - m);
                    sum += pb;
#pragma unroll
                    for (int v = 0; v < V; ++v) craw[v] = fmaf(pb, c[b].v[v], craw[v]);
                }
                const float out = m + lg2f(sum) - offM;
                Mout[q] = out;
                tmax = fmaxf(tmax, out);
                const float f = ex2f(m + Ls - D);
                den = fmaf(f, sum, den);
#pragma unroll
                for (int v = 0; v < V; ++v) num[v] = fmaf(f, craw[v], num[v]);
            }
            den = warp_sum(den); tmax = warp_max(tmax);
#pragma unroll
            for (int v = 0; v < V; ++v) num[v] = warp_sum(num[v]);
            if (lane == 0) {
                wmax[(t & 1) * 32 + warp] = tmax;
                float *pp = part + ((t & 1) * 32 + warp) * VEC_PART;
                pp[0] = den;
#pragma unroll
                for (int v = 0; v < V; ++v) pp[1 + v] = num[v];
            }
            P += (int)offM;
            __syncthreads();
            cmax = warp_max(lane < nwarp ? wmax[(t & 1) * 32 + lane] : NEG_INF);
            offM = rintf(cmax);
            if (warp == 0) {
                const float *pp = part + ((t & 1) * 32 + lane) * VEC_PART;
                const float b = warp_sum(lane < nwarp ? pp[0] : 0.f);
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const float a = warp_sum(lane < nwarp ? pp[1 + v] : 0.f);
                    if (lane == 0) {
                        const float sw = a / b;
                        p.soft[blk * n + (size_t)(t - 1) * V + v] = sw;
                        if (p.soft_copy) p.soft_copy[blk * n + (size_t)(t - 1) * V + v] = sw;
                    }
                }
                if (lane == 0) defect = fmaxf(defect, fabsf(b - 1.f));
            }
            float *sw = Min; Min = Mout; Mout = sw;
        }
        ssum = 0.f;
        for (int q = tid; q < Q; q += nthr) ssum += ex2f(Min[q] - cmax);
        ssum = warp_sum(ssum);
        if (lane == 0) lzpart[warp] = ssum;
        __syncthreads();
        if (tid == 0) {
            float t2 = 0.f;
            for (int i = 0; i < nwarp; ++i) t2 += lzpart[i];
            const float lz_beta = cmax + lg2f(t2);
            zgap = fmaxf(zgap, fabsf((float)(P - Ofin) + (lz_beta - lsefin)));
        }
        __syncthreads();
    }
    if (tid == 0) {
        diag_max(&p.diag->max_defect, defect);
        diag_max(&p.diag->max_logz_gap, zgap);
    }
}

// --------------------------------------------------------------------------------------
// Backward call.  With h_t(s) = sum_v g[V t + v] (c[s][v] - soft[V t + v]) the recursions are those
// of the scalar kernel (first-order expectation semiring); per emitted component v
//   grad_W[V t + v]  = (1/T) Cov_gamma(r_t, c[.][v])
//   grad_c[u][v]    += gamma_t(u) [ g[V t + v] + (w[V t + v] - c[u][v]) r_t(u) / T ]
// --------------------------------------------------------------------------------------
template <int KB, int V>
__global__ void __launch_bounds__(GEN_MAX_THREADS) bwd_vec_kernel(BwdParams p)
{
    constexpr int K = 1 << KB;
    extern __shared__ float smem[];
    const int S = 1 << p.Lb, Q = S >> KB, n = p.n, nt = n / V;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const float NEG_INF = __int_as_float(0xff800000);
    float *wmax = smem;             // [2][32]
    float *part = smem + 64;        // [2][32][VEC_PART]: S0, S2, S1[v], S3[v]
    float *lzpart = smem + 64 + 2 * 32 * VEC_PART;
    float *msgbuf = p.msg ? p.msg + (size_t)blockIdx.x * 4 * Q : smem + VEC_SMEM_HEADER;
    float *histL = p.hist + (size_t)blockIdx.x * 2 * nt * Q;
    float *histA = histL + (size_t)nt * Q;
    int *stepO = p.stepO + (size_t)blockIdx.x * (nt + 2);
    float *gc = p.gc_part + (size_t)blockIdx.x * S * V;           // [K][Q][V], like cb_beta
    const float lam2 = p.lam2, invT = p.invT;
    float defect = 0.f;
    static_assert(2 + 2 * V <= VEC_PART, "posterior sums per warp slot");

    for (int i = tid; i < S * V; i += nthr) gc[i] = 0.f;

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w = p.W + blk * n, *g = p.g + blk * n, *sf = p.soft + blk * n;
        float *Lin = msgbuf, *Lout = msgbuf + Q, *Ain = msgbuf + 2 * Q, *Aout = msgbuf + 3 * Q;
        for (int q = tid; q < Q; q += nthr) { Lin[q] = 0.f; Ain[q] = 0.f; histL[q] = 0.f; histA[q] = 0.f; }
        if (tid == 0) stepO[1] = 0;
        int O = 0;
        float off = 0.f, cmax = 0.f;
        __syncthreads();
        for (int t = 1; t <= nt; ++t) {
            const VecOf<V> wt = load_vec<V>(w + (size_t)(t - 1) * V), gt = load_vec<V>(g + (size_t)(t - 1) * V);
            const VecOf<V> st = load_vec<V>(sf + (size_t)(t - 1) * V);
            float tmax = NEG_INF;
            for (int q = tid; q < Q; q += nthr) {
                float a[K], x[K], m = NEG_INF;
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    const int s = q + j * Q;
                    const VecOf<V> c = load_vec<V>(p.cb + (size_t)s * V);
                    a[j] = fmaf(dist2<V>(wt, c), -lam2, Lin[s >> KB]);
                    float h = Ain[s >> KB];
#pragma unroll
                    for (int v = 0; v < V; ++v) h = fmaf(gt.v[v], c.v[v] - st.v[v], h);
                    x[j] = h;
                    m = fmaxf(m, a[j]);
                }
                float sum = 0.f, acc = 0.f;
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    const float pj = ex2f(a[j] - m);
                    sum += pj;
                    acc = fmaf(pj, x[j], acc);
                }
                const float out = m + lg2f(sum) - off;
                const float aout = acc * rcpf(sum);
                Lout[q] = out; Aout[q] = aout;
                if (t < nt) { histL[(size_t)t * Q + q] = out; histA[(size_t)t * Q + q] = aout; }
                tmax = fmaxf(tmax, out);
            }
            tmax = warp_max(tmax);
            if (lane == 0) wmax[(t & 1) * 32 + warp] = tmax;
            O += (int)off;
            if (tid == 0) stepO[t + 1] = O;
            __syncthreads();
            cmax = warp_max(lane < nwarp ? wmax[(t & 1) * 32 + lane] : NEG_INF);
            off = rintf(cmax);
            float *sw = Lin; Lin = Lout; Lout = sw;
            sw = Ain; Ain = Aout; Aout = sw;
        }
        float ssum = 0.f;
        for (int q = tid; q < Q; q += nthr) ssum += ex2f(Lin[q] - cmax);
        ssum = warp_sum(ssum);
        if (lane == 0) lzpart[warp] = ssum;
        __syncthreads();
        float tot = 0.f;
        for (int i = 0; i < nwarp; ++i) tot += lzpart[i];
        const float lsefin = cmax + lg2f(tot);
        if (tid == 0) diag_check_finite(p.diag, lsefin);
        const int Ofin = O;
        float *Min = msgbuf, *Mout = msgbuf + Q, *Bin = msgbuf + 2 * Q, *Bout = msgbuf + 3 * Q;
        for (int q = tid; q < Q; q += nthr) { Min[q] = 0.f; Bin[q] = 0.f; }
        int P = 0;
        float offM = 0.f;
        __syncthreads();
        for (int t = nt; t >= 1; --t) {
            const VecOf<V> wt = load_vec<V>(w + (size_t)(t - 1) * V), gt = load_vec<V>(g + (size_t)(t - 1) * V);
            const VecOf<V> st = load_vec<V>(sf + (size_t)(t - 1) * V);
            const float D = (float)(Ofin - stepO[t] - P) + lsefin;
            float S0 = 0.f, S2 = 0.f, S1[V], S3[V], tmax = NEG_INF;
#pragma unroll
            for (int v = 0; v < V; ++v) { S1[v] = 0.f; S3[v] = 0.f; }
            for (int q = tid; q < Q; q += nthr) {
                const float Ls = histL[(size_t)(t - 1) * Q + q];
                const float At = histA[(size_t)(t - 1) * Q + q];
                VecOf<V> c[K];
                float u[K], y[K], m = NEG_INF;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const int s = q * K + b;
                    c[b] = load_vec<V>(p.cb_beta + ((size_t)b * Q + q) * V);
                    u[b] = fmaf(dist2<V>(wt, c[b]), -lam2, Min[s & (Q - 1)]);
                    float h = Bin[s & (Q - 1)];
#pragma unroll
                    for (int v = 0; v < V; ++v) h = fmaf(gt.v[v], c[b].v[v] - st.v[v], h);
                    y[b] = h;
                    m = fmaxf(m, u[b]);
                }
                float sum = 0.f, acc = 0.f;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    u[b] = ex2f(u[b] - m);                                 // rho(b|q) up to the group's sum
                    sum += u[b];
                    acc = fmaf(u[b], y[b], acc);
                }
                const float out = m + lg2f(sum) - offM;
                Mout[q] = out;
                Bout[q] = acc * rcpf(sum);
                tmax = fmaxf(tmax, out);
                const float f = ex2f(m + Ls - D);
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const float gam = u[b] * f;
                    const float r = y[b] + At;
                    const float gr = gam * r;
                    S0 += gam;
                    S2 += gr;
#pragma unroll
                    for (int v = 0; v < V; ++v) {
                        const float cm = c[b].v[v] - st.v[v];
                        S1[v] = fmaf(gam, cm, S1[v]);
                        S3[v] = fmaf(gr, cm, S3[v]);
                        gc[((size_t)b * Q + q) * V + v] += gam * fmaf(invT * (wt.v[v] - c[b].v[v]), r, gt.v[v]);
                    }
                }
            }
            S0 = warp_sum(S0); S2 = warp_sum(S2);
#pragma unroll
            for (int v = 0; v < V; ++v) { S1[v] = warp_sum(S1[v]); S3[v] = warp_sum(S3[v]); }
            tmax = warp_max(tmax);
            if (lane == 0) {
                wmax[(t & 1) * 32 + warp] = tmax;
                float *pp = part + ((t & 1) * 32 + warp) * VEC_PART;
                pp[0] = S0; pp[1] = S2;
#pragma unroll
                for (int v = 0; v < V; ++v) { pp[2 + v] = S1[v]; pp[2 + V + v] = S3[v]; }
            }
            P += (int)offM;
            __syncthreads();
            cmax = warp_max(lane < nwarp ? wmax[(t & 1) * 32 + lane] : NEG_INF);
            offM = rintf(cmax);
            if (warp == 0) {
                const float *pp = part + ((t & 1) * 32 + lane) * VEC_PART;
                const float a0 = warp_sum(lane < nwarp ? pp[0] : 0.f), a2 = warp_sum(lane < nwarp ? pp[1] : 0.f);
                const float i0 = 1.f / a0;
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const float a1 = warp_sum(lane < nwarp ? pp[2 + v] : 0.f);
                    const float a3 = warp_sum(lane < nwarp ? pp[2 + V + v] : 0.f);
                    if (lane == 0) p.gW[blk * n + (size_t)(t - 1) * V + v] = invT * (a3 * i0 - (a2 * i0) * (a1 * i0));
                }
                if (lane == 0) defect = fmaxf(defect, fabsf(a0 - 1.f));
            }
            float *sw = Min; Min = Mout; Mout = sw;
            sw = Bin; Bin = Bout; Bout = sw;
        }
        __syncthreads();
    }
    if (tid == 0) diag_max(&p.diag->max_defect, defect);
}

// --------------------------------------------------------------------------------------
// Viterbi with vector emissions.  Double metrics without fused multiply-add, components added
// in order: e = d_0 d_0, e += d_v d_v; m = min_j(...) + e; lowest branch / lowest state on ties.
// states: [B][nt] uint16; hard: [B][n] (the emitted numbers); path bits: Lb + KB (nt - 1).
// --------------------------------------------------------------------------------------
template <int V>
__device__ __forceinline__ double dist2_double(const VecOf<V> &w, const VecOf<V> &c)
{
    double e = 0.0;
#pragma unroll
    for (int i = 0; i < V; ++i) {
        const double d = __dsub_rn((double)w.v[i], (double)c.v[i]);
        const double dd = __dmul_rn(d, d);
        e = i == 0 ? dd : __dadd_rn(e, dd);
    }
    return e;
}

template <int KB, int V>
__global__ void __launch_bounds__(GEN_MAX_THREADS) viterbi_vec_kernel(VitParams p)
{
    constexpr int K = 1 << KB;
    extern __shared__ float smem[];
    const int S = 1 << p.Lb, Q = S >> KB, n = p.n, nt = n / V;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    double *redv = reinterpret_cast<double *>(smem);              // [32]
    int *redi = reinterpret_cast<int *>(smem + 64);               // [32]
    double *msgbuf = p.msg ? p.msg + (size_t)blockIdx.x * 2 * Q
                           : reinterpret_cast<double *>(smem + VEC_SMEM_HEADER);
    uint8_t *bp = p.bp + (size_t)blockIdx.x * nt * Q;
    int *path = p.path_ws + (size_t)blockIdx.x * nt;
    const int nbits = p.Lb + KB * (nt - 1);

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w = p.W + blk * n;
        double *in = msgbuf, *out = msgbuf + Q;
        for (int q = tid; q < Q; q += nthr) in[q] = 0.0;
        __syncthreads();
        for (int t = 1; t < nt; ++t) {
            const VecOf<V> wt = load_vec<V>(w + (size_t)(t - 1) * V);
            for (int q = tid; q < Q; q += nthr) {
                double bm = 0.0;
                int bj = 0;
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    const int s = q + j * Q;
                    const double mm = __dadd_rn(in[s >> KB], dist2_double<V>(wt, load_vec<V>(p.cb + (size_t)s * V)));
                    if (j == 0 || mm < bm) { bm = mm; bj = j; }
                }
                out[q] = bm;
                bp[(size_t)t * Q + q] = (uint8_t)bj;
            }
            __syncthreads();
            double *sw = in; in = out; out = sw;
        }
        {
            const VecOf<V> wt = load_vec<V>(w + (size_t)(nt - 1) * V);
            double bv = 0.0;
            int bi = 0x7fffffff;
            for (int q = tid; q < Q; q += nthr)
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const int s = q * K + b;
                    const double mm = __dadd_rn(in[q], dist2_double<V>(wt, load_vec<V>(p.cb + (size_t)s * V)));
                    if (bi == 0x7fffffff || mm < bv || (mm == bv && s < bi)) { bv = mm; bi = s; }
                }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const double ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (oi != 0x7fffffff && (bi == 0x7fffffff || ov < bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
            }
            if (lane == 0) { redv[warp] = bv; redi[warp] = bi; }
            __syncthreads();
            if (tid == 0) {
                double v = redv[0];
                int i = redi[0];
                for (int x = 1; x < nwarp; ++x) {
                    const double ov = redv[x];
                    const int oi = redi[x];
                    if (oi != 0x7fffffff && (i == 0x7fffffff || ov < v || (ov == v && oi < i))) { v = ov; i = oi; }
                }
                int s = i;
                path[nt - 1] = s;
                for (int t = nt - 1; t >= 1; --t) {
                    const int j = bp[(size_t)t * Q + (s >> KB)];
                    s = (s >> KB) + j * Q;
                    path[t - 1] = s;
                }
            }
            __syncthreads();
        }
        for (int t = tid; t < nt; t += nthr) {
            const int s = path[t];
            if (p.states) p.states[blk * nt + t] = (uint16_t)s;
            if (p.hard) {
                const VecOf<V> c = load_vec<V>(p.cb + (size_t)s * V);
#pragma unroll
                for (int v = 0; v < V; ++v) p.hard[blk * n + (size_t)t * V + v] = c.v[v];
            }
        }
        if (p.path_bits) {
            uint8_t *pb = p.path_bits + blk * p.path_stride;
            for (int64_t byte = tid; byte < p.path_stride; byte += nthr) {
                unsigned v = 0;
                for (int r = 0; r < 8; ++r) {
                    const int64_t pos = byte * 8 + r;
                    int bit = 0;
                    if (pos < p.Lb) bit = (path[0] >> (p.Lb - 1 - (int)pos)) & 1;
                    else if (pos < nbits) {
                        const int rel = (int)pos - p.Lb;
                        bit = (path[1 + rel / KB] >> (KB - 1 - rel % KB)) & 1;
                    }
                    v |= (unsigned)bit << (7 - r);
                }
                pb[byte] = (uint8_t)v;
            }
        }
        __syncthreads();
    }
}

}  // namespace bcjr
