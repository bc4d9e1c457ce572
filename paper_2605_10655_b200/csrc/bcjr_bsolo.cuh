// Backward call without grad_codebook (2^16 states, k = 2) on ONE CTA per block.
//
// The two-CTA backward kernels exist because the gradient accumulators of the codebook need a second SM's tensor
// memory.  A call that does not ask for grad_codebook (the table is fixed, or computed: Section 3.1) has no
// accumulators, so the whole backward pass of a block fits one SM, like the forward pass: the alpha sweep of
// bwd_alpha_kernel, then a beta sweep carrying (M, Bt) IN PLACE in the same two arrays, one CTA barrier per step
// and eight butterflies per thread to hide it behind.
//
// In-place beta sweep.  Butterfly x reads M_t([x|b]), b = 0..K-1, and writes M_{t-1}([j|x]), j = 0..K-1; output j
// takes the slot of input b = j.  Group index q of step t therefore lives at
//     slot_t(q) = swz(rotr(q, rr_t)),   rr_n = 0,   rr_{t-1} = rr_t - k  (mod Lb - k)
// (the alpha sweep's rotation run backwards), with the same bank swizzle: a warp's 32 butterflies differ in index
// bits k..k+4, which the rotation moves to a window of five consecutive bits at an even position, exactly the
// windows the swizzle was built for.
//
// History: written and read by the same thread (butterfly i * 512 + tid in both sweeps), float4
// [n][butterfly slot][L | At][thread] per resident CTA, streamed back through a four-deep cp.async ring.
#pragma once
#include "bcjr_alpha.cuh"

namespace bcjr {

struct BSoloCfg : AlphaCfg<2> {
    using A = AlphaCfg<2>;
    static constexpr int NCH = 2 * K / 4;                      // 16-byte chunks per butterfly and thread: K values of L, K of At
    static constexpr int RD = 4;                               // staging ring: butterflies in flight
    static constexpr int MAX_N = 1024;
    static constexpr int OFF_M = 0;                            // [Q]  L, then M
    static constexpr int OFF_B = OFF_M + Q;                    // [Q]  At, then Bt
    static constexpr int OFF_RING = OFF_B + Q;                 // float4 [RD][NCH][THREADS]
    static constexpr int OFF_TABA = OFF_RING + RD * NCH * THREADS * 4;   // uint32 [NROT][16]: alpha sweep, T_i (BPT) and T_j (K) from entry 8
    static constexpr int OFF_TABB = OFF_TABA + NROT * 16;      // uint32 [NROT][16]: beta sweep, T_i (BPT) and T_b (K) from entry 8
    static constexpr int OFF_O = OFF_TABB + NROT * 16;         // int [MAX_N + 2]
    static constexpr int OFF_WMAX = OFF_O + MAX_N + 2 + 2;     // [2][32]
    static constexpr int OFF_PART = OFF_WMAX + 64;             // [2][32][4]
    static constexpr int OFF_LZ = OFF_PART + 256;              // [32]
    static constexpr int OFF_TMEM = OFF_LZ + 32;
    static constexpr int SMEM_FLOATS = OFF_TMEM + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(K == 4 && BPT == 8 && BPT % RD == 0, "ring slot of butterfly i is i mod RD");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory of one CTA");
    // beta sweep: input b of butterfly x = i * 512 + tid is group (x << k) | b
    __host__ __device__ static constexpr uint32_t beta_q(int i, int tid, int b) { return ((uint32_t)(i * THREADS + tid) << KB) | (uint32_t)b; }
};

__global__ void __launch_bounds__(BSoloCfg::THREADS, 1) bwd_solo_kernel(BwdParams p)
{
    using C = BSoloCfg;
    constexpr int KB = C::KB, K = C::K, Q = C::Q, BPT = C::BPT, NWARP = C::NWARP, CT = C::CTHREADS, NCH = C::NCH, RD = C::RD;
    constexpr ptrdiff_t HSTEP = 2 * Q / 4;                      // float4 per step: (L, At) of every group
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float2 nl2 = splat2(-p.lam2);
    const float invT = p.invT;
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;

    float *Ms = smem + C::OFF_M, *Bs = smem + C::OFF_B;
    const float4 *stage4 = reinterpret_cast<const float4 *>(smem + C::OFF_RING);
    const uint32_t stage_u32 = smem_u32(smem + C::OFF_RING) + (uint32_t)tid * 16u;
    uint32_t *tabA = reinterpret_cast<uint32_t *>(smem + C::OFF_TABA);
    uint32_t *tabB = reinterpret_cast<uint32_t *>(smem + C::OFF_TABB);
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);

    if (tid < C::NROT * 16) {
        const int r = tid >> 4, e = tid & 15;                            // table row = the rotation itself
        uint32_t va = 0, vb = 0;
        if (e < BPT) {
            va = C::slot((uint32_t)e << 9, r);                           // alpha: butterfly bits above the thread index
            vb = C::slot(C::beta_q(e, 0, 0), r);                         // beta: the same bits, k positions higher
        } else if (e >= 8 && e < 8 + K) {
            va = C::slot((uint32_t)(e - 8) << (C::QB - KB), r);          // alpha: the input's branch bits on top
            vb = C::slot((uint32_t)(e - 8), r);                          // beta: the input's branch bits at the bottom
        }
        tabA[tid] = va;
        tabB[tid] = vb;
    }
    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)blockIdx.x * n * 2 * Q) + tid;   // this thread's entries
    float defect = 0.f;

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w_s = p.W + blk * n, *g_s = p.g + blk * n, *sf_s = p.soft + blk * n;
        {
            const float gsh1 = -__ldg(g_s) * __ldg(sf_s);             // L_1 = 0; the At array carries At + gsh (see bcjr_duo.cuh)
            for (int q = tid; q < Q; q += CT) { Ms[q] = 0.f; Bs[q] = gsh1; }
        }
        if (tid == 0) O_s[1] = 0;
        int outside = 0;
        for (int t = tid; t < n; t += CT) {
            const float wv = __ldg(w_s + t);
            outside |= !(wv >= c_lo && wv <= c_hi);
        }
        const bool recentre = __syncthreads_or(outside) != 0;
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * CT + tid, tm + (uint32_t)(K * K * i), false);
        tmem_wait_st();
        int O = 0;
        float off = 0.f, cmax = 0.f;
        compute_barrier(CT);
        // ================= alpha sweep carrying (L, At); every step's inputs go to the history
        auto alpha_sweep = [&](auto rc_tag) {
            constexpr bool RC = decltype(rc_tag)::value;
            int r = 0;                                                // k (t - 1) mod (Lb - k)
            for (int t = 1; t <= n; ++t) {
                const int cur = (t - 1) & 1;
                float2 cb[8];
                tmem_ld16(tm, cb);
                const float gt = __ldg(g_s + t - 1), wt = __ldg(w_s + t - 1);
                const float gshn = t < n ? -__ldg(g_s + t) * __ldg(sf_s + t) : 0.f;
                if (t > 1) {
                    cmax = warp_max(lane < NWARP ? wmax[cur * 32 + lane] : NEG_INF) - off;
                    off = rintf(cmax);
                }
                const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
                const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), off2 = splat2(off), gshn2 = splat2(gshn);
                const uint32_t *tb = tabA + r * 16;
                const uint32_t st = C::slot((uint32_t)tid, r);
                uint32_t TJ[K];
#pragma unroll
                for (int j = 0; j < K; ++j) TJ[j] = tb[8 + j] ^ st;
                float4 *hrow = hist4 + (size_t)(t - 1) * HSTEP;
                float tmax = NEG_INF;
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    const uint32_t ti = tb[i];
                    float Lj[K], Aj[K];
#pragma unroll
                    for (int j = 0; j < K; ++j) {
                        Lj[j] = Ms[ti ^ TJ[j]];
                        Aj[j] = Bs[ti ^ TJ[j]];
                    }
                    hrow[(i * NCH) * CT] = make_float4(Lj[0], Lj[1], Lj[2], Lj[3]);
                    hrow[(i * NCH + 1) * CT] = make_float4(Aj[0], Aj[1], Aj[2], Aj[3]);
                    tmem_wait_ld(cb);
                    float2 outL[K / 2], outA[K / 2];
#pragma unroll
                    for (int h = 0; h < K / 2; ++h) {
                        float2 a[K];
#pragma unroll
                        for (int j = 0; j < K; ++j) {
                            const float2 du = sub2(cb[C::a_idx(j, h)], w2);
                            a[j] = RC ? energy2(du, nl2, kap2, splat2(Lj[j])) : fma2(mul2(du, du), nl2, splat2(Lj[j]));
                        }
                        const float2 m = max_pairs<K>(a);
                        float2 pj = ex2f2(sub2(a[0], m));
                        float2 sum = pj, ax = mul2(pj, fma2(g2, cb[C::a_idx(0, h)], splat2(Aj[0])));
#pragma unroll
                        for (int j = 1; j < K; ++j) {
                            pj = ex2f2(sub2(a[j], m));
                            sum = add2(sum, pj);
                            ax = fma2(pj, fma2(g2, cb[C::a_idx(j, h)], splat2(Aj[j])), ax);
                        }
                        outL[h] = add2(sub2(m, off2), lg2f2(sum));
                        outA[h] = fma2(ax, rcpf2(sum), gshn2);
                        tmax = max3f(tmax, m.x, m.y);
                    }
                    if (i + 1 < BPT) tmem_ld16(tm + 16u * (i + 1), cb);
                    // output [x|l] takes the place of input [l|x]
#pragma unroll
                    for (int h = 0; h < K / 2; ++h) {
                        Ms[ti ^ TJ[2 * h]] = outL[h].x; Ms[ti ^ TJ[2 * h + 1]] = outL[h].y;
                        Bs[ti ^ TJ[2 * h]] = outA[h].x; Bs[ti ^ TJ[2 * h + 1]] = outA[h].y;
                    }
                }
                tmax = warp_max(tmax);
                if (lane == 0) wmax[(cur ^ 1) * 32 + warp] = tmax;
                O += (int)off;
                if (tid == 0) O_s[t + 1] = O;
                r += KB; r = r >= C::QB ? r - C::QB : r;
                compute_barrier(CT);
            }
        };
        if (recentre) alpha_sweep(std::true_type{}); else alpha_sweep(std::false_type{});
        // log2 Z = O_{n+1} + LSE_q L_{n+1}(q)
        cmax = warp_max(lane < NWARP ? wmax[(n & 1) * 32 + lane] : NEG_INF) - off;
        {
            float ssum = 0.f;
            for (int q = tid; q < Q; q += CT) ssum += ex2f(Ms[q] - cmax);
            ssum = warp_sum(ssum);
            if (lane == 0) lz[warp] = ssum;
            compute_barrier(CT);
        }
        const float lsefin = cmax + lg2f(warp_sum(lane < NWARP ? lz[lane] : 0.f));
        const int Ofin = O;
        if (tid == 0) diag_check_finite(p.diag, lsefin);
        // ================= beta sweep carrying (M, Bt) in place, with the contraction for grad_W
        {
            const float gshn = -__ldg(g_s + n - 1) * __ldg(sf_s + n - 1);     // M_n = 0, Bt_n = 0 (+ centring shift)
            for (int q = tid; q < Q; q += CT) { Ms[q] = 0.f; Bs[q] = gshn; }
        }
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * CT + tid, tm + (uint32_t)(K * K * i), true);   // beta pairing
        tmem_wait_st();
        // history stream: butterfly i of step t is requested three butterflies ahead, into ring slot i mod RD
        auto issue = [&](const float4 *row, int i) {                 // butterfly i of the step whose history starts at row
            const uint32_t dst = stage_u32 + (uint32_t)(i & (RD - 1)) * (uint32_t)(NCH * CT * 16);
#pragma unroll
            for (int q = 0; q < NCH; ++q)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)(q * CT * 16)), "l"(row + (i * NCH + q) * CT) : "memory");
        };
#pragma unroll
        for (int i = 0; i < RD - 1; ++i) {
            issue(hist4 + (size_t)(n - 1) * HSTEP, i);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        int P = 0;
        float offM = 0.f;
        compute_barrier(CT);
        // last warp: turn the sums of step t (slots of parity b) into grad_W[t]
        auto finish_step = [&](int t, int b) {
            if (warp == NWARP - 1) {
                const float *pp = part + (b * 32 + lane) * 4;
                float a0 = lane < NWARP ? pp[0] : 0.f, a2 = lane < NWARP ? pp[1] : 0.f, az = lane < NWARP ? pp[2] : 0.f;
                a0 = warp_sum(a0); a2 = warp_sum(a2); az = warp_sum(az);
                if (lane == 0) {
                    const float i0 = 1.f / a0;
                    p.gW[blk * n + t - 1] = (__ldg(g_s + t - 1) - az * i0) + (a2 * i0) * (__ldg(w_s + t - 1) - __ldg(sf_s + t - 1)) * invT;
                    defect = fmaxf(defect, fabsf(a0 - 1.f));
                }
            }
        };
        auto beta_sweep = [&](auto rc_tag) {
            constexpr bool RC = decltype(rc_tag)::value;
            int rr = 0;                                               // -k (n - t) mod (Lb - k)
            for (int t = n; t >= 1; --t) {
                const int par = t & 1;
                float2 cb[8];                                     // one set of table registers (see bcjr_skew.cuh)
                tmem_ld16(tm, cb);
                const float wt = __ldg(w_s + t - 1), gt = __ldg(g_s + t - 1);
                const float gsh = -gt * __ldg(sf_s + t - 1);                      // shift carried by the stored At
                const float gshp = t > 1 ? -__ldg(g_s + t - 2) * __ldg(sf_s + t - 2) : 0.f;   // for step t-1
                const int Ot = O_s[t];
                if (t < n) {
                    P += (int)offM;                                   // offsets carried by this step's inputs M_t
                    cmax = warp_max(lane < NWARP ? wmax[(par ^ 1) * 32 + lane] : NEG_INF);
                    offM = rintf(cmax);
                    finish_step(t + 1, par ^ 1);
                }
                const float2 gsh2 = splat2(gsh), gshp2 = splat2(gshp), offM2 = splat2(offM);
                const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
                const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), ngi2 = splat2(-invT), gid2 = splat2(invT * se.delta);
                const float2 Dm2 = splat2((float)(Ofin - Ot - P) + lsefin);
                const uint32_t *tb = tabB + rr * 16;
                const uint32_t st = C::slot(C::beta_q(0, tid, 0), rr);
                const float4 *hrow = hist4 + (size_t)(t - 1) * HSTEP;
                uint32_t TB[K];
#pragma unroll
                for (int b = 0; b < K; ++b) TB[b] = tb[8 + b] ^ st;
                float2 S0 = make_float2(0.f, 0.f), S2 = S0, ZS = S0;
                float tmax = NEG_INF;
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    const uint32_t ti = tb[i];
                    asm volatile("cp.async.wait_group %0;" ::"n"(RD - 2) : "memory");
                    float Lh[K], Ah[K];
                    {
                        const float4 l4 = stage4[((i & (RD - 1)) * NCH) * CT + tid], a4 = stage4[((i & (RD - 1)) * NCH + 1) * CT + tid];
                        Lh[0] = l4.x; Lh[1] = l4.y; Lh[2] = l4.z; Lh[3] = l4.w;
                        Ah[0] = a4.x; Ah[1] = a4.y; Ah[2] = a4.z; Ah[3] = a4.w;
                    }
                    {                                                 // RD - 1 butterflies ahead, into the slot the previous one was read from
                        const int ahead = i + RD - 1;
                        if (ahead < BPT) issue(hrow, ahead);
                        else if (t > 1) issue(hrow - HSTEP, ahead - BPT);
                        asm volatile("cp.async.commit_group;" ::: "memory");
                    }
                    float Mb[K], Yb[K];
#pragma unroll
                    for (int b = 0; b < K; ++b) {
                        Mb[b] = Ms[ti ^ TB[b]];
                        Yb[b] = Bs[ti ^ TB[b]];
                    }
                    tmem_wait_ld(cb);
                    float2 outM[K / 2], outB[K / 2];
#pragma unroll
                    for (int jh = 0; jh < K / 2; ++jh) {
                        float2 uu[K], d[K];
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            d[b] = sub2(cb[C::b_idx(jh, b)], w2);              // du = c - wc
                            uu[b] = RC ? energy2(d[b], nl2, kap2, splat2(Mb[b])) : fma2(mul2(d[b], d[b]), nl2, splat2(Mb[b]));
                        }
                        const float2 m = max_pairs<K>(uu);
                        const float2 Ahj = sub2(make_float2(Ah[2 * jh], Ah[2 * jh + 1]), gsh2);
                        const float2 Lhj = make_float2(Lh[2 * jh], Lh[2 * jh + 1]);
                        const float2 f = ex2f2(add2(sub2(m, Dm2), Lhj));
                        // f (w - c) / T = f delta / T - (f / T) du
                        const float2 fg = mul2(f, g2), nfi = mul2(f, ngi2), fid = RC ? mul2(f, gid2) : make_float2(0.f, 0.f);
                        const float2 nfiA = mul2(nfi, Ahj);                 // plain square: f (w - c) r / T = du (nfi y + nfi At)
                        float2 sum = make_float2(0.f, 0.f), ya = sum, zs = sum;
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            const float2 pb = ex2f2(sub2(uu[b], m));
                            const float2 y = fma2(g2, cb[C::b_idx(jh, b)], splat2(Yb[b]));   // h + Bt
                            const float2 z = RC ? fma2(fma2(nfi, d[b], fid), add2(y, Ahj), fg) : fma2(d[b], fma2(nfi, y, nfiA), fg);   // f (g + (w - c) r / T)
                            sum = add2(sum, pb);
                            ya = fma2(pb, y, ya);
                            zs = fma2(pb, z, zs);
                        }
                        outM[jh] = sub2(add2(m, lg2f2(sum)), offM2);
                        outB[jh] = fma2(ya, rcpf2(sum), gshp2);
                        tmax = max3f(tmax, m.x, m.y);
                        S0 = fma2(f, sum, S0);
                        S2 = fma2(f, fma2(Ahj, sum, ya), S2);
                        ZS = add2(ZS, zs);
                    }
                    if (i + 1 < BPT) tmem_ld16(tm + 16u * (i + 1), cb);
                    // output [j|x] takes the place of input [x|j]
#pragma unroll
                    for (int jh = 0; jh < K / 2; ++jh) {
                        Ms[ti ^ TB[2 * jh]] = outM[jh].x; Ms[ti ^ TB[2 * jh + 1]] = outM[jh].y;
                        Bs[ti ^ TB[2 * jh]] = outB[jh].x; Bs[ti ^ TB[2 * jh + 1]] = outB[jh].y;
                    }
                }
                tmax = warp_max(tmax) - offM;
                if (lane == 0) wmax[par * 32 + warp] = tmax;
                const float s3 = warp_sum3_split(S0.x + S0.y, S2.x + S2.y, ZS.x + ZS.y, lane);
                if ((lane & 7) == 0 && lane < 24) part[(par * 32 + warp) * 4 + (lane >> 3)] = s3;
                rr = rr == 0 ? C::QB - KB : rr - KB;
                compute_barrier(CT);
            }
        };
        if (recentre) beta_sweep(std::true_type{}); else beta_sweep(std::false_type{});
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        finish_step(1, 1);
        compute_barrier(CT);                                          // part, wmax, lz and the messages are free for the next block
    }
    if (tid == CT - 32) diag_max(&p.diag->max_defect, defect);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
