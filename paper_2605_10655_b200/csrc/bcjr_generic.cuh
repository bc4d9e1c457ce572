// Generic kernels: one thread block per weight block, any (Lb, k) with Lb - k <= 14.
// They are the cover-everything path (small trellises, odd shapes); the cluster kernels in
// bcjr_cluster.cuh take over for the 2^16-state trellis.
//
// Work split: a thread owns groups q = tid, tid + blockDim, ...  The compressed messages
// (Q floats each) ping-pong through shared memory (or through a per-CTA global scratch when
// they do not fit); the gauge-fixed forward messages of every step are spilled to a per-CTA
// history in global memory and read back by the beta sweep, which fuses the posterior, the
// codeword expectation (Eq. 7) and, in the backward pass, the gradient contraction.
#pragma once
#include "bcjr_common.cuh"

namespace bcjr {

constexpr int GEN_SMEM_HEADER = 512;   // floats reserved ahead of the message buffers
constexpr int GEN_MAX_THREADS = 512;

// --------------------------------------------------------------------------------------
// Forward call: alpha sweep (Eq. 5, log domain) then beta sweep fused with Eq. 6-7.
// --------------------------------------------------------------------------------------
template <int KB>
__global__ void __launch_bounds__(GEN_MAX_THREADS, (KB == 2 || KB == 3) ? 2 : 1) fwd_generic_kernel(FwdParams p)
{
    constexpr int K = 1 << KB;
    extern __shared__ float smem[];
    const int S = 1 << p.Lb, Q = S >> KB, n = p.n;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const float NEG_INF = __int_as_float(0xff800000);
    float *wmax = smem;             // [2][32]
    float *part = smem + 64;        // [2][32][2]
    float *lzpart = smem + 192;     // [32]
    float *msgbuf = p.msg ? p.msg + (size_t)blockIdx.x * 2 * Q : smem + GEN_SMEM_HEADER;
    float *hist = p.hist + (size_t)blockIdx.x * n * Q;
    int *stepO = p.stepO + (size_t)blockIdx.x * (n + 2);
    const float lam2 = p.lam2;
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;
    float defect = 0.f, zgap = 0.f;

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w = p.W + blk * n;
        float *Lin = msgbuf, *Lout = msgbuf + Q;
        for (int q = tid; q < Q; q += nthr) { Lin[q] = 0.f; hist[q] = 0.f; }   // L_1 = 0: free first state
        if (tid == 0) stepO[1] = 0;
        int O = 0;
        float off = 0.f, cmax = 0.f, bdef = 0.f;
        double zshift = 0.0;                     // sum_t lam2 delta_t^2: what step_energy leaves out of log2 Z
        __syncthreads();
        // ---- alpha: from L_t to L_{t+1}, t = 1..n (the last one only feeds log Z)
        for (int t = 1; t <= n; ++t) {
            const StepEnergy se = step_energy(__ldg(w + t - 1), c_lo, c_hi, lam2);
            zshift += (double)lam2 * (double)se.delta * (double)se.delta;
            float tmax = NEG_INF;
            for (int q = tid; q < Q; q += nthr) {
                float a[K], m = NEG_INF;
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    const int s = q + j * Q;
                    const float du = __ldg(p.cb + s) - se.wc;
                    a[j] = fmaf(du, fmaf(du, -lam2, se.kap), Lin[s >> KB]);
                    m = fmaxf(m, a[j]);
                }
                float sum = 0.f;
#pragma unroll
                for (int j = 0; j < K; ++j) sum += ex2f(a[j] - m);
                const float out = m + lg2f(sum) - off;
                Lout[q] = out;
                if (t < n) hist[(size_t)t * Q + q] = out;
                tmax = fmaxf(tmax, out);
            }
            tmax = warp_max(tmax);
            if (lane == 0) wmax[(t & 1) * 32 + warp] = tmax;
            O += (int)off;                       // O_{t+1}
            if (tid == 0) stepO[t + 1] = O;
            __syncthreads();
            cmax = warp_max(lane < nwarp ? wmax[(t & 1) * 32 + lane] : NEG_INF);
            off = rintf(cmax);
            float *sw = Lin; Lin = Lout; Lout = sw;
        }
        // ---- log2 Z = O_{n+1} + LSE_q L_{n+1}(q)
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
        if (tid == 0 && p.logZ) p.logZ[blk] = (float)(((double)Ofin + (double)lsefin - zshift) * 0.6931471805599453);
        // ---- beta sweep fused with the posterior and the expectation
        float *Min = msgbuf, *Mout = msgbuf + Q;
        for (int q = tid; q < Q; q += nthr) Min[q] = 0.f;                      // M_n = 0: free last state
        int P = 0;
        float offM = 0.f;
        __syncthreads();
        for (int t = n; t >= 1; --t) {
            const StepEnergy se = step_energy(__ldg(w + t - 1), c_lo, c_hi, lam2);
            const float D = (float)(Ofin - stepO[t] - P) + lsefin;
            float num = 0.f, den = 0.f, tmax = NEG_INF;
            for (int q = tid; q < Q; q += nthr) {
                const float Ls = hist[(size_t)(t - 1) * Q + q];
                float u[K], c[K], m = NEG_INF;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const int s = q * K + b;
                    c[b] = __ldg(p.cb + s);
                    const float du = c[b] - se.wc;
                    u[b] = fmaf(du, fmaf(du, -lam2, se.kap), Min[s & (Q - 1)]);
                    m = fmaxf(m, u[b]);
                }
                float sum = 0.f, craw = 0.f;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const float pb = ex2f(u[b] - m);
                    sum += pb;
                    craw = fmaf(pb, c[b], craw);
                }
                const float out = m + lg2f(sum) - offM;
                Mout[q] = out;
                tmax = fmaxf(tmax, out);
                const float f = ex2f(m + Ls - D);
                den = fmaf(f, sum, den);
                num = fmaf(f, craw, num);
            }
            num = warp_sum(num); den = warp_sum(den); tmax = warp_max(tmax);
            if (lane == 0) {
                wmax[(t & 1) * 32 + warp] = tmax;
                part[((t & 1) * 32 + warp) * 2] = num;
                part[((t & 1) * 32 + warp) * 2 + 1] = den;
            }
            P += (int)offM;                      // P_{t-1}
            __syncthreads();
            cmax = warp_max(lane < nwarp ? wmax[(t & 1) * 32 + lane] : NEG_INF);
            offM = rintf(cmax);
            if (warp == 0) {
                float a = lane < nwarp ? part[((t & 1) * 32 + lane) * 2] : 0.f;
                float b = lane < nwarp ? part[((t & 1) * 32 + lane) * 2 + 1] : 0.f;
                a = warp_sum(a); b = warp_sum(b);
                if (lane == 0) {
                    const float sw = a / b;
                    p.soft[blk * n + t - 1] = sw;
                    if (p.soft_copy) p.soft_copy[blk * n + t - 1] = sw;
                    bdef = fmaxf(bdef, fabsf(b - 1.f));
                }
            }
            float *sw = Min; Min = Mout; Mout = sw;
        }
        // ---- consistency: P_0 + LSE_q M_0(q) must equal log2 Z
        ssum = 0.f;
        for (int q = tid; q < Q; q += nthr) ssum += ex2f(Min[q] - cmax);
        ssum = warp_sum(ssum);
        if (lane == 0) lzpart[warp] = ssum;
        __syncthreads();
        if (tid == 0) {
            defect = fmaxf(defect, bdef);
            if (p.blk_defect) p.blk_defect[blk] = bdef;
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
// Backward call: the two sweeps again, carrying the conditional expectations of the centred
// emitted sum next to the messages (first-order expectation semiring), fused with the
// gradient contraction.  With h_t(s) = g_t (c[s] - soft_t):
//   At_{t+1}(q) = sum_j pi(j|q) [ h_t(q + jQ) + At_t((q + jQ) >> k) ],        At_1 = 0
//   Bt_{t-1}(q) = sum_b rho(b|q) [ h_t(qK + b) + Bt_t((qK + b) & (Q-1)) ],    Bt_n = 0
//   r_t(s) = h_t(s) + At_t(s >> k) + Bt_t(s & (Q-1))  =  E[G | s_t = s] - E[G]
//   grad_W[t]  = (1/T) Cov_gamma(r_t, c)
//   grad_c[u] += gamma_t(u) [ g_t + (w_t - c[u]) r_t(u) / T ]
// --------------------------------------------------------------------------------------
template <int KB>
__global__ void __launch_bounds__(GEN_MAX_THREADS, KB == 2 ? 2 : 1) bwd_generic_kernel(BwdParams p)
{
    constexpr int K = 1 << KB;
    extern __shared__ float smem[];
    const int S = 1 << p.Lb, Q = S >> KB, n = p.n;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    const float NEG_INF = __int_as_float(0xff800000);
    float *wmax = smem;             // [2][32]
    float *part = smem + 64;        // [2][32][4]
    float *lzpart = smem + 320;     // [32]
    float *msgbuf = p.msg ? p.msg + (size_t)blockIdx.x * 4 * Q : smem + GEN_SMEM_HEADER;
    float *histL = p.hist + (size_t)blockIdx.x * 2 * n * Q;
    float *histA = histL + (size_t)n * Q;
    int *stepO = p.stepO + (size_t)blockIdx.x * (n + 2);
    float *gc = p.gc_part + (size_t)blockIdx.x * S;
    const float lam2 = p.lam2, invT = p.invT;
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;
    float defect = 0.f;

    for (int q = tid; q < Q; q += nthr)
#pragma unroll
        for (int b = 0; b < K; ++b) gc[q * K + b] = 0.f;

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w = p.W + blk * n, *g = p.g + blk * n, *sf = p.soft + blk * n;
        float *Lin = msgbuf, *Lout = msgbuf + Q, *Ain = msgbuf + 2 * Q, *Aout = msgbuf + 3 * Q;
        for (int q = tid; q < Q; q += nthr) { Lin[q] = 0.f; Ain[q] = 0.f; histL[q] = 0.f; histA[q] = 0.f; }
        if (tid == 0) stepO[1] = 0;
        int O = 0;
        float off = 0.f, cmax = 0.f;
        __syncthreads();
        for (int t = 1; t <= n; ++t) {
            const float gt = __ldg(g + t - 1), st = __ldg(sf + t - 1);
            const StepEnergy se = step_energy(__ldg(w + t - 1), c_lo, c_hi, lam2);
            float tmax = NEG_INF;
            for (int q = tid; q < Q; q += nthr) {
                float a[K], x[K], m = NEG_INF;
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    const int s = q + j * Q;
                    const float c = __ldg(p.cb + s);
                    const float du = c - se.wc;
                    a[j] = fmaf(du, fmaf(du, -lam2, se.kap), Lin[s >> KB]);
                    x[j] = fmaf(gt, c - st, Ain[s >> KB]);
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
                if (t < n) { histL[(size_t)t * Q + q] = out; histA[(size_t)t * Q + q] = aout; }
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
        for (int t = n; t >= 1; --t) {
            const float gt = __ldg(g + t - 1), st = __ldg(sf + t - 1);
            const StepEnergy se = step_energy(__ldg(w + t - 1), c_lo, c_hi, lam2);
            const float D = (float)(Ofin - stepO[t] - P) + lsefin;
            float S0 = 0.f, S1 = 0.f, S2 = 0.f, S3 = 0.f, tmax = NEG_INF;
            for (int q = tid; q < Q; q += nthr) {
                const float Ls = histL[(size_t)(t - 1) * Q + q];
                const float At = histA[(size_t)(t - 1) * Q + q];
                float u[K], d[K], cm[K], y[K], m = NEG_INF;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const int s = q * K + b;
                    const float c = __ldg(p.cb + s);
                    const float du = c - se.wc;
                    d[b] = se.delta - du;                       // w - c
                    cm[b] = c - st;
                    u[b] = fmaf(du, fmaf(du, -lam2, se.kap), Min[s & (Q - 1)]);
                    y[b] = fmaf(gt, cm[b], Bin[s & (Q - 1)]);
                    m = fmaxf(m, u[b]);
                }
                float pb[K], sum = 0.f, acc = 0.f;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    pb[b] = ex2f(u[b] - m);
                    sum += pb[b];
                    acc = fmaf(pb[b], y[b], acc);
                }
                const float out = m + lg2f(sum) - offM;
                Mout[q] = out;
                Bout[q] = acc * rcpf(sum);
                tmax = fmaxf(tmax, out);
                const float f = ex2f(m + Ls - D);
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const float gam = pb[b] * f;
                    const float r = y[b] + At;
                    const float gr = gam * r;
                    S0 += gam;
                    S1 = fmaf(gam, cm[b], S1);
                    S2 += gr;
                    S3 = fmaf(gr, cm[b], S3);
                    gc[q * K + b] += gam * fmaf(invT * d[b], r, gt);
                }
            }
            S0 = warp_sum(S0); S1 = warp_sum(S1); S2 = warp_sum(S2); S3 = warp_sum(S3);
            tmax = warp_max(tmax);
            if (lane == 0) {
                wmax[(t & 1) * 32 + warp] = tmax;
                float *pp = part + ((t & 1) * 32 + warp) * 4;
                pp[0] = S0; pp[1] = S1; pp[2] = S2; pp[3] = S3;
            }
            P += (int)offM;
            __syncthreads();
            cmax = warp_max(lane < nwarp ? wmax[(t & 1) * 32 + lane] : NEG_INF);
            offM = rintf(cmax);
            if (warp == 0) {
                const float *pp = part + ((t & 1) * 32 + lane) * 4;
                float a0 = lane < nwarp ? pp[0] : 0.f, a1 = lane < nwarp ? pp[1] : 0.f;
                float a2 = lane < nwarp ? pp[2] : 0.f, a3 = lane < nwarp ? pp[3] : 0.f;
                a0 = warp_sum(a0); a1 = warp_sum(a1); a2 = warp_sum(a2); a3 = warp_sum(a3);
                if (lane == 0) {
                    const float i0 = 1.f / a0;
                    p.gW[blk * n + t - 1] = invT * (a3 * i0 - (a2 * i0) * (a1 * i0));
                    defect = fmaxf(defect, fabsf(a0 - 1.f));
                }
            }
            float *sw = Min; Min = Mout; Mout = sw;
            sw = Bin; Bin = Bout; Bout = sw;
        }
        __syncthreads();
    }
    if (tid == 0) diag_max(&p.diag->max_defect, defect);
}

// Deterministic (fixed-order) sum of the per-CTA partial codebook gradients.
static __global__ void reduce_gc_kernel(const float *part, int nparts, int S, float *out)
{
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= S) return;
    float acc = 0.f;
    for (int i = 0; i < nparts; ++i) acc += part[(size_t)i * S + u];
    out[u] = acc;
}

// --------------------------------------------------------------------------------------
// Viterbi (Section 3.2) with double metrics.  mv_t(q) = min_j m_{t-1}(q + jQ) is shared by
// the K states of group q, so one branch index per group per step is kept for the backtrack.
// --------------------------------------------------------------------------------------
template <int KB>
__global__ void __launch_bounds__(GEN_MAX_THREADS) viterbi_generic_kernel(VitParams p)
{
    constexpr int K = 1 << KB;
    extern __shared__ float smem[];
    const int S = 1 << p.Lb, Q = S >> KB, n = p.n;
    const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
    double *redv = reinterpret_cast<double *>(smem);              // [32]
    int *redi = reinterpret_cast<int *>(smem + 64);               // [32]
    int *sbest = reinterpret_cast<int *>(smem + 96);
    double *msgbuf = p.msg ? p.msg + (size_t)blockIdx.x * 2 * Q
                           : reinterpret_cast<double *>(smem + GEN_SMEM_HEADER);
    uint8_t *bp = p.bp + (size_t)blockIdx.x * n * Q;
    int *path = p.path_ws + (size_t)blockIdx.x * n;
    const int nbits = p.Lb + KB * (n - 1);

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w = p.W + blk * n;
        double *in = msgbuf, *out = msgbuf + Q;
        for (int q = tid; q < Q; q += nthr) in[q] = 0.0;
        __syncthreads();
        for (int t = 1; t < n; ++t) {
            const double wt = (double)__ldg(w + t - 1);
            for (int q = tid; q < Q; q += nthr) {
                double bm = 0.0;
                int bj = 0;
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    const int s = q + j * Q;
                    const double d = __dsub_rn(wt, (double)__ldg(p.cb + s));
                    const double mm = __dadd_rn(in[s >> KB], __dmul_rn(d, d));
                    if (j == 0 || mm < bm) { bm = mm; bj = j; }
                }
                out[q] = bm;
                bp[(size_t)t * Q + q] = (uint8_t)bj;
            }
            __syncthreads();
            double *sw = in; in = out; out = sw;
        }
        // final metrics m_n(s) = mv_n(s >> k) + (w_n - c[s])^2, lowest s among the minima
        {
            const double wt = (double)__ldg(w + n - 1);
            double bv = 0.0;
            int bi = 0x7fffffff;
            for (int q = tid; q < Q; q += nthr)
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    const int s = q * K + b;
                    const double d = __dsub_rn(wt, (double)__ldg(p.cb + s));
                    const double mm = __dadd_rn(in[q], __dmul_rn(d, d));
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
                // backtrack: predecessor of s at step t is (s >> k) + j*Q with j the stored branch
                int s = i;
                path[n - 1] = s;
                for (int t = n - 1; t >= 1; --t) {
                    const int j = bp[(size_t)t * Q + (s >> KB)];
                    s = (s >> KB) + j * Q;
                    path[t - 1] = s;
                }
                *sbest = i;
            }
            __syncthreads();
        }
        for (int t = tid; t < n; t += nthr) {
            const int s = path[t];
            if (p.states) p.states[blk * n + t] = (uint16_t)s;
            if (p.hard) p.hard[blk * n + t] = __ldg(p.cb + s);
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
