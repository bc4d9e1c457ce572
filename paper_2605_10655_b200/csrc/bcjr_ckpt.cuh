// Forward call with checkpointed forward messages (Lb = 16, k = 2): the one-CTA tensor-memory kernel of
// bcjr_solo.cuh, except that the alpha sweep keeps L_t only for every m-th step and the beta sweep recomputes
// the m - 1 steps in between.
//
// bcjr_solo.cuh stores L_t of every step (n Q floats per block, 16 MB at k = 2, n = 256) and streams it back:
// history traffic n Q 8 bytes per block through HBM.  Here the alpha sweep stores L_t for t = 1, m+1, 2m+1, ...
// only.  The beta sweep walks the segments [cm+1, (c+1)m] from the last to the first; for each it reloads the
// checkpoint L_{cm+1}, runs the alpha recursion forward again through the segment -- same instructions, same
// recorded gauge offsets, hence bit-identical messages -- writing L_t of the segment's steps to a scratch of
// m rows that is reused by every segment (and therefore lives in L2), and then takes the segment's beta steps
// from that scratch.  HBM history traffic drops to 1/m; the price is (m-1)/m of an alpha sweep more
// special-function work per block, which is why m = 1 is the default on this GPU.
//
// Shared memory: three message buffers instead of two -- while a segment is recomputed the current M must
// survive next to the alpha ping-pong -- so the history staging is two butterflies deep instead of eight and
// blocks are limited to 512 steps.
#pragma once
#include "bcjr_solo.cuh"

namespace bcjr {

template <int KB_>
struct CkptCfg {
    using B = SoloCfg<KB_>;
    static constexpr int LB = 16, KB = KB_, K = B::K, S = B::S, Q = B::Q, NB = B::NB;
    static constexpr int CTHREADS = 512, THREADS = 512, NWARP = 16, BPT = B::BPT, UNITS = B::UNITS, HPU = B::HPU, NCH = B::NCH;
    static constexpr int RD = 2;                               // staging depth in butterflies
    static constexpr int MAX_N = 512, MAX_M = 16;
    static constexpr int OFF_MSG = 0;                          // [3][Q]
    static constexpr int OFF_RING = OFF_MSG + 3 * Q;           // float4 [RD][NCH][CTHREADS]
    static constexpr int OFF_W = OFF_RING + RD * NCH * CTHREADS * 4;   // [2][MAX_N] clamped weight, kap (step_energy)
    static constexpr int OFF_GAUGE = OFF_W + 2 * MAX_N;        // [MAX_N + 2] gauge offset used by alpha step t
    static constexpr int OFF_O = OFF_GAUGE + MAX_N + 2;        // int [MAX_N + 2]
    static constexpr int OFF_WMAX = OFF_O + MAX_N + 2;         // [2][32]
    static constexpr int OFF_PART = OFF_WMAX + 64;             // [2][32][2]
    static constexpr int OFF_LZ = OFF_PART + 128;              // [32]
    static constexpr int OFF_TMEM = OFF_LZ + 32;
    static constexpr int SMEM_FLOATS = OFF_TMEM + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(OFF_RING % 4 == 0, "staging alignment");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");
    static_assert(KB_ == 2 && NCH == 1, "the alpha step on the beta-paired table is written for K = 4");
    __host__ __device__ static constexpr int a_idx(int j, int h) { return B::a_idx(j, h); }
    __host__ __device__ static constexpr int b_idx(int jh, int b) { return B::b_idx(jh, b); }
    // history rows per CTA: the checkpoints, then the segment scratch
    __host__ __device__ static constexpr int rows(int n, int m) { return (n + m - 1) / m + m; }
};

template <int KB>
__global__ void __launch_bounds__(CkptCfg<KB>::THREADS, 1) fwd_ckpt_kernel(FwdParams p)
{
    using C = CkptCfg<KB>;
    constexpr int K = C::K, NB = C::NB, Q = C::Q, BPT = C::BPT, NWARP = C::NWARP, CT = C::CTHREADS, NCH = C::NCH, RD = C::RD;
    constexpr int UNITS = C::UNITS, HPU = C::HPU, NU = BPT * UNITS;
    constexpr int ROW = BPT * NCH * CT;                          // float4 per history row
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.n, m = p.hist_every;
    const int NC = (n + m - 1) / m;
    const float NEG_INF = __int_as_float(0xff800000);
    const float2 nl2 = splat2(-p.lam2);

    float *msg = smem + C::OFF_MSG;
    float4 *stage4 = reinterpret_cast<float4 *>(smem + C::OFF_RING);
    float *w_s = smem + C::OFF_W, *kap_s = w_s + C::MAX_N;
    float *gauge_s = smem + C::OFF_GAUGE;
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);
    const uint32_t stage_u32 = smem_u32(stage4) + (uint32_t)tid * 16u;
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;

    // history of this CTA: float4 [NC + m][BPT][NCH][CT]; rows 0 .. NC-1 = checkpoints L_{cm+1}, rows NC .. = scratch of a segment
    float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)blockIdx.x * C::rows(n, m) * Q) + tid;

    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    int push_a[BPT];
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int x = i * CT + tid;
        const int q2 = x * K, j2 = q2 / NB, x2 = q2 % NB;
        push_a[i] = ((x2 / CT) * K + j2) * CT + (x2 % CT);
    }
    float defect = 0.f, zgap = 0.f;

    // One alpha step: L_{t+1} from L_t (Lin, thread-private entries) into Lout (the consumers' entries); the inputs are
    // stored to hrow when it is not null.  Used by the alpha sweep and, unchanged, by the recomputation, so both give
    // the same bits.  It works on the table as the BETA sweep pairs it -- (c[2jh|x|b], c[2jh+1|x|b]) -- so that the
    // table is staged once per block and never re-paired: the sum over the predecessors j of output b is then a sum
    // over the two halves of two packed values instead of over four packed values.
    auto alpha_step = [&](const float *Lin, float *Lout, float4 *hrow, float wc, float kap, float off) -> float {
        const float2 w2 = splat2(wc), kap2 = splat2(kap);
        float tmax = NEG_INF;
        float2 cb[2][8];
        tmem_ld16(tm, cb[0]);
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            float Lj[K];
#pragma unroll
            for (int j = 0; j < K; ++j) Lj[j] = Lin[(i * K + j) * CT + tid];
            if (hrow) hrow[i * CT] = make_float4(Lj[0], Lj[1], Lj[2], Lj[3]);
            tmem_wait_ld(cb[i & 1]);
            if (i + 1 < BPT) tmem_ld16(tm + 16u * (i + 1), cb[(i + 1) & 1]);
            const float2 L01 = make_float2(Lj[0], Lj[1]), L23 = make_float2(Lj[2], Lj[3]);
            float out[K];
#pragma unroll
            for (int b = 0; b < K; ++b) {
                const float2 d0 = sub2(cb[i & 1][C::b_idx(0, b)], w2), d1 = sub2(cb[i & 1][C::b_idx(1, b)], w2);
                const float2 a0 = energy2(d0, nl2, kap2, L01), a1 = energy2(d1, nl2, kap2, L23);
                const float mx = fmaxf(max3f(a0.x, a0.y, a1.x), a1.y);
                const float2 m2 = splat2(mx);
                const float2 s2 = add2(ex2f2(sub2(a0, m2)), ex2f2(sub2(a1, m2)));
                out[b] = (mx - off) + lg2f(s2.x + s2.y);
                tmax = fmaxf(tmax, mx);
            }
            *reinterpret_cast<float4 *>(Lout + push_a[i]) = make_float4(out[0], out[1], out[2], out[3]);
        }
        return tmax;
    };

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w = p.W + blk * n;
        for (int t = tid; t < n; t += CT) {
            const StepEnergy se = step_energy(__ldg(w + t), c_lo, c_hi, p.lam2);
            w_s[t] = se.wc; kap_s[t] = se.kap;
        }
        for (int q = tid; q < Q; q += CT) msg[q] = 0.f;                      // L_1 = 0 in buffer 0
        if (tid == 0) O_s[1] = 0;
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * CT + tid, tm + (uint32_t)(K * K * i), true);   // beta pairing, for both sweeps
        tmem_wait_st();
        int O = 0;
        float off = 0.f, cmax = 0.f, bdef = 0.f;
        compute_barrier(CT);
        // ================= alpha sweep: checkpoints only
        {
            int since = 0, ci = 0;                                           // (t - 1) mod m, (t - 1) / m
            for (int t = 1; t <= n; ++t) {
                const int cur = (t - 1) & 1;
                if (t > 1) {
                    cmax = warp_max(lane < NWARP ? wmax[cur * 32 + lane] : NEG_INF) - off;
                    off = rintf(cmax);
                }
                if (tid == 0) gauge_s[t] = off;
                float4 *hrow = since == 0 ? hist4 + (size_t)ci * ROW : nullptr;
                float tmax = alpha_step(msg + cur * Q, msg + (cur ^ 1) * Q, hrow, w_s[t - 1], kap_s[t - 1], off);
                tmax = warp_max(tmax);
                if (lane == 0) wmax[(cur ^ 1) * 32 + warp] = tmax;
                O += (int)off;
                if (tid == 0) O_s[t + 1] = O;
                if (++since == m) { since = 0; ++ci; }
                compute_barrier(CT);
            }
        }
        // ================= log2 Z = O_{n+1} + LSE_q L_{n+1}(q); L_{n+1} sits in buffer n&1
        cmax = warp_max(lane < NWARP ? wmax[(n & 1) * 32 + lane] : NEG_INF) - off;
        {
            const float *Lfin = msg + (n & 1) * Q;
            float ssum = 0.f;
            for (int q = tid; q < Q; q += CT) ssum += ex2f(Lfin[q] - cmax);
            ssum = warp_sum(ssum);
            if (lane == 0) lz[warp] = ssum;
            compute_barrier(CT);
        }
        const float lsefin = cmax + lg2f(warp_sum(lane < NWARP ? lz[lane] : 0.f));
        if (tid == 0) diag_check_finite(p.diag, lsefin);
        const int Ofin = O;
        if (tid == 0 && p.logZ) {
            double zshift = 0.0;                                             // what step_energy leaves out of log2 Z
            for (int t = 0; t < n; ++t) zshift += (double)kap_s[t] * (double)kap_s[t];
            zshift /= 4.0 * (double)p.lam2;
            p.logZ[blk] = (float)(((double)Ofin + (double)lsefin - zshift) * 0.6931471805599453);
        }
        // ================= beta sweep, segment by segment
        for (int q = tid; q < Q; q += CT) msg[q] = 0.f;                      // M_n = 0 in buffer 0
        int P = 0, mb = 0;                                                   // mb: buffer that holds the current M
        float offM = 0.f;
        int par = 0;                                                         // parity of the wmax / part slots
        bool first = true;
        compute_barrier(CT);
        for (int c = NC - 1; c >= 0; --c) {
            const int t0 = c * m + 1, t_end = min(t0 + m - 1, n), len = t_end - t0 + 1;
            float4 *seg = hist4 + (size_t)NC * ROW;                          // row s = L_{t0 + s}, s >= 1
            if (len > 1) {
                // ---- recompute L_{t0+1} .. L_{t_end} from the checkpoint, in the two buffers that do not hold M
                const int a0 = mb == 0 ? 1 : 0, a1 = 3 - mb - a0;
                {
                    float *A = msg + a0 * Q;
                    const float4 *ck = hist4 + (size_t)c * ROW;
#pragma unroll
                    for (int i = 0; i < BPT; ++i)
#pragma unroll
                        for (int q = 0; q < NCH; ++q) {
                            const float4 v = __ldcg(ck + (i * NCH + q) * CT);
                            A[(i * K + 4 * q) * CT + tid] = v.x; A[(i * K + 4 * q + 1) * CT + tid] = v.y;
                            A[(i * K + 4 * q + 2) * CT + tid] = v.z; A[(i * K + 4 * q + 3) * CT + tid] = v.w;
                        }
                }
                for (int s = 0; s + 1 < len; ++s) {
                    const int t = t0 + s;
                    const float *Lin = msg + ((s & 1) ? a1 : a0) * Q;
                    float *Lout = msg + ((s & 1) ? a0 : a1) * Q;
                    alpha_step(Lin, Lout, s > 0 ? seg + (size_t)s * ROW : nullptr, w_s[t - 1], kap_s[t - 1], gauge_s[t]);
                    compute_barrier(CT);
                }
                {
                    const float *Lin = msg + (((len - 1) & 1) ? a1 : a0) * Q;    // L_{t_end}: this thread's entries
                    float4 *hrow = seg + (size_t)(len - 1) * ROW;
#pragma unroll
                    for (int i = 0; i < BPT; ++i)
#pragma unroll
                        for (int q = 0; q < NCH; ++q)
                            hrow[(i * NCH + q) * CT] = make_float4(Lin[(i * K + 4 * q) * CT + tid], Lin[(i * K + 4 * q + 1) * CT + tid],
                                                                   Lin[(i * K + 4 * q + 2) * CT + tid], Lin[(i * K + 4 * q + 3) * CT + tid]);
                }
                compute_barrier(CT);                                         // the recomputation's buffers are free for M again
            }
            // ---- the segment's beta steps, t = t_end .. t0; L_t from the scratch (row t - t0) or the checkpoint (t = t0)
            auto row_of = [&](int t) -> const float4 * { return t == t0 ? hist4 + (size_t)c * ROW : seg + (size_t)(t - t0) * ROW; };
            int nt = t_end, ni = 0;                                          // next chunk to request: butterfly ni of step nt
            auto issue_chunk = [&](uint32_t slot) {
                const float4 *src = row_of(nt) + ni * NCH * CT;
                const uint32_t dst = stage_u32 + slot * (uint32_t)(NCH * CT * 16);
#pragma unroll
                for (int q = 0; q < NCH; ++q)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)(q * CT * 16)), "l"(src + q * CT) : "memory");
                asm volatile("cp.async.commit_group;" ::: "memory");
                if (++ni == BPT) { ni = 0; if (nt > t0) --nt; }              // past the segment's end: the last step again, unread
            };
#pragma unroll
            for (uint32_t cnk = 0; cnk + 1 < RD; ++cnk) issue_chunk(cnk);
            uint32_t slot = 0;
            for (int t = t_end; t >= t0; --t) {
                const int mo = mb == 0 ? 1 : 0;                              // output buffer: ping-pong between two of the three
                const float *Min = msg + mb * Q;
                float *Mout = msg + mo * Q;
                if (!first) {
                    cmax = warp_max(lane < NWARP ? wmax[par * 32 + lane] : NEG_INF);
                    P += (int)offM;
                    offM = rintf(cmax);
                    if (warp == 0) {                                         // soft[t+1] from the partial sums
                        float a = lane < NWARP ? part[(par * 32 + lane) * 2] : 0.f;
                        float cc = lane < NWARP ? part[(par * 32 + lane) * 2 + 1] : 0.f;
                        a = warp_sum(a); cc = warp_sum(cc);
                        if (lane == 0) {
                            const float sw = a / cc;
                            p.soft[blk * n + t] = sw;
                            if (p.soft_copy) p.soft_copy[blk * n + t] = sw;
                            bdef = fmaxf(bdef, fabsf(cc - 1.f));
                        }
                    }
                }
                first = false;
                const float2 w2 = splat2(w_s[t - 1]), kap2 = splat2(kap_s[t - 1]);
                const float2 offM2 = splat2(offM);
                const float2 Dm2 = splat2((float)(Ofin - O_s[t] - P) + lsefin);
                float2 num2 = make_float2(0.f, 0.f), den2 = make_float2(0.f, 0.f);
                float tmax = NEG_INF;
                float2 cb[2][8];
                tmem_ld16(tm, cb[0]);
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    issue_chunk(slot == 0 ? RD - 1 : slot - 1);              // refill the slot consumed last
                    asm volatile("cp.async.wait_group %0;" ::"n"(RD - 1) : "memory");
                    float Lh[K];
#pragma unroll
                    for (int q = 0; q < NCH; ++q) {
                        const float4 l4 = stage4[(slot * NCH + q) * CT + tid];
                        Lh[4 * q] = l4.x; Lh[4 * q + 1] = l4.y; Lh[4 * q + 2] = l4.z; Lh[4 * q + 3] = l4.w;
                    }
                    slot = slot + 1 == RD ? 0 : slot + 1;
                    float Mb[K];
#pragma unroll
                    for (int b = 0; b < K; b += 4) {
                        const float4 v = *reinterpret_cast<const float4 *>(Min + (i * CT + tid) * K + b);
                        Mb[b] = v.x; Mb[b + 1] = v.y; Mb[b + 2] = v.z; Mb[b + 3] = v.w;
                    }
#pragma unroll
                    for (int u = 0; u < UNITS; ++u) {
                        const int g = i * UNITS + u;
                        tmem_wait_ld(cb[g & 1]);
                        if (g + 1 < NU) tmem_ld16(tm + 16u * (g + 1), cb[(g + 1) & 1]);
#pragma unroll
                        for (int hh = 0; hh < HPU; ++hh) {
                            const int jh = u * HPU + hh;
                            float2 uu[K];
#pragma unroll
                            for (int b = 0; b < K; ++b) {
                                const float2 du = sub2(cb[g & 1][C::b_idx(hh, b)], w2);
                                uu[b] = energy2(du, nl2, kap2, splat2(Mb[b]));
                            }
                            const float2 mx = max_pairs<K>(uu);
                            const float2 Lhj = make_float2(Lh[2 * jh], Lh[2 * jh + 1]);
                            const float2 f = ex2f2(add2(sub2(mx, Dm2), Lhj));
                            float2 pb = ex2f2(sub2(uu[0], mx));
                            float2 sum = pb, craw = mul2(pb, cb[g & 1][C::b_idx(hh, 0)]);
#pragma unroll
                            for (int b = 1; b < K; ++b) {
                                pb = ex2f2(sub2(uu[b], mx));
                                sum = add2(sum, pb);
                                craw = fma2(pb, cb[g & 1][C::b_idx(hh, b)], craw);
                            }
                            const float2 out = add2(sub2(mx, offM2), lg2f2(sum));
                            tmax = max3f(tmax, mx.x, mx.y);
                            Mout[((2 * jh) * (NB / K) + (i * CT + tid) / K) * K + (tid % K)] = out.x;
                            Mout[((2 * jh + 1) * (NB / K) + (i * CT + tid) / K) * K + (tid % K)] = out.y;
                            num2 = fma2(f, craw, num2);
                            den2 = fma2(f, sum, den2);
                        }
                    }
                }
                const float nd = warp_sum2_split(num2.x + num2.y, den2.x + den2.y, lane);
                tmax = warp_max(tmax) - offM;
                par ^= 1;
                if (lane == 0) wmax[par * 32 + warp] = tmax;
                if ((lane & 15) == 0) part[(par * 32 + warp) * 2 + (lane >> 4)] = nd;
                mb = mo;
                compute_barrier(CT);
            }
            asm volatile("cp.async.wait_all;" ::: "memory");                 // the unread tail requests of this segment
        }
        {
            cmax = warp_max(lane < NWARP ? wmax[par * 32 + lane] : NEG_INF);  // M_0 and the sums of step 1
            P += (int)offM;
            if (warp == 0) {
                float a = lane < NWARP ? part[(par * 32 + lane) * 2] : 0.f;
                float cc = lane < NWARP ? part[(par * 32 + lane) * 2 + 1] : 0.f;
                a = warp_sum(a); cc = warp_sum(cc);
                if (lane == 0) {
                    const float sw = a / cc;
                    p.soft[blk * n] = sw;
                    if (p.soft_copy) p.soft_copy[blk * n] = sw;
                    bdef = fmaxf(bdef, fabsf(cc - 1.f));
                    defect = fmaxf(defect, bdef);
                    if (p.blk_defect) p.blk_defect[blk] = bdef;
                }
            }
            // consistency: P_0 + LSE_q M_0(q) against log2 Z
            const float *Mfin = msg + mb * Q;
            float ssum = 0.f;
            for (int q = tid; q < Q; q += CT) ssum += ex2f(Mfin[q] - cmax);
            ssum = warp_sum(ssum);
            compute_barrier(CT);                                             // lz is free again
            if (lane == 0) lz[warp] = ssum;
            compute_barrier(CT);
            const float lz_beta = cmax + lg2f(warp_sum(lane < NWARP ? lz[lane] : 0.f));
            zgap = fmaxf(zgap, fabsf((float)(P - Ofin) + (lz_beta - lsefin)));
            compute_barrier(CT);
        }
    }
    if (tid == 0) {
        diag_max(&p.diag->max_defect, defect);
        diag_max(&p.diag->max_logz_gap, zgap);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
