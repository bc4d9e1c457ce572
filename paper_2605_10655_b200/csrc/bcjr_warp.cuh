// Mid-size trellises (Lb = 11, 12, 13; k = 2): one WARP per weight block.
//
// At 2^12 states a trellis step is 1/16 of the 2^16-state step.  Spread over a CTA it is a few states per thread
// between two CTA barriers, and the barriers dominate (the generic kernels sit at 15 % of the special-function peak
// there).  Given to a single warp, a step is eight butterflies of sixteen states per lane -- the same work per thread
// and step as in the 2^16-state forward kernel -- and the exchange between steps needs no barrier at all: a lane's
// outputs are some other lane's inputs of the same warp, so __syncwarp() orders them.  Sixteen warps per CTA run
// sixteen independent blocks; nothing is shared between them but the SM.
//
// The table lives where it does in the large-trellis kernels: in tensor memory, lane-private.  Every warp holds the
// WHOLE table (2^Lb floats = 32 lanes x 2^(Lb-5) columns) in its own quarter of the lanes and its own column range;
// at Lb = 12 sixteen warps x 128 columns fill the SM's 256 KB exactly.  The backward kernel keeps the gradient
// accumulators next to it (twice the columns, half the warps) and sums the warps' partials at the end.
//
// Messages are indexed by the group index itself: alpha inputs L([j|x]) at j NB + x, outputs L'([x|l]) at 4x + l
// (one 16-byte store); beta the other way round.  History is thread-private as in the large-trellis kernels.
#pragma once
#include "bcjr_solo.cuh"

namespace bcjr {

template <int LB_, bool BWD>
struct WarpCfg {
    static constexpr int LB = LB_, KB = 2, K = 4, S = 1 << LB, Q = S >> KB, NB = S >> (2 * KB);
    static constexpr int BPT = NB / 32;                        // butterflies per lane: 4 / 8 / 16
    static constexpr int UNITS = 1, HPU = 2;
    static constexpr int COLS = (BWD ? 32 : 16) * BPT;         // tensor-memory columns per thread: table (+ accumulators)
    static constexpr int NWARP = 2048 / COLS < 16 ? 2048 / COLS : 16;   // 4 lane quarters x (512 / COLS) column ranges
    static constexpr int THREADS = 32 * NWARP;
    static constexpr int NCH = BWD ? 2 : 1;                    // 16-byte history chunks per butterfly: L (and At)
    static constexpr int RD = BPT < 8 ? BPT : 8;               // history staging depth in butterflies
    static constexpr int MSG = (BWD ? 4 : 2) * Q;              // floats per warp: two parities of L (and At)
    static constexpr int RING = RD * NCH * 32 * 4;             // floats per warp
    static constexpr int PER_WARP = MSG + RING;
    static constexpr int OFF_TMEM = NWARP * PER_WARP;
    static constexpr int SMEM_FLOATS = OFF_TMEM + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(LB >= 11 && LB <= 13, "one warp per block is built for 2^11 .. 2^13 states");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");
    __host__ __device__ static constexpr int a_idx(int j, int h) { return 2 * j + h; }
    __host__ __device__ static constexpr int b_idx(int jh, int b) { return 4 * jh + b; }
};

// Forward call: alpha sweep, log Z, beta sweep with posterior and expectation (Eq. 5-7); p.stepO holds the gauge
// offsets O_t of every resident warp ([warps][n + 2]), p.hist its history ([warps][n][BPT][32] float4).
template <int LB>
__global__ void __launch_bounds__(WarpCfg<LB, false>::THREADS, 1) fwd_warp_kernel(FwdParams p)
{
    using C = WarpCfg<LB, false>;
    constexpr int K = C::K, NB = C::NB, Q = C::Q, BPT = C::BPT, RD = C::RD;
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float2 nl2 = splat2(-p.lam2);
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);

    float *msg = smem + warp * C::PER_WARP;
    float4 *stage4 = reinterpret_cast<float4 *>(msg + C::MSG);          // [RD][32], thread-private entries
    const uint32_t stage_u32 = smem_u32(stage4) + (uint32_t)lane * 16u;
    const int64_t wg = (int64_t)blockIdx.x * C::NWARP + warp, nwg = (int64_t)gridDim.x * C::NWARP;
    float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)wg * n * Q) + lane;    // row t: [BPT][32]
    int *O_g = p.stepO + (size_t)wg * (n + 2);

    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * C::COLS);
    float defect = 0.f, zgap = 0.f;

    for (int64_t blk = wg; blk < p.B; blk += nwg) {
        const float *w = p.W + blk * n;
        for (int q = lane; q < Q; q += 32) msg[q] = 0.f;                   // L_1 = 0 in buffer 0
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * 32 + lane, tm + (uint32_t)(16 * i), false);
        tmem_wait_st();
        int O = 0;
        float off = 0.f, cmax = 0.f, bdef = 0.f;
        double zshift = 0.0;
        if (lane == 0) O_g[1] = 0;
        __syncwarp();
        // ================= alpha sweep
        for (int t = 1; t <= n; ++t) {
            const int cur = (t - 1) & 1;
            const float *Lin = msg + cur * Q;
            float *Lout = msg + (cur ^ 1) * Q;
            float2 cb[2][8];
            tmem_ld16(tm, cb[0]);
            const StepEnergy se = step_energy(__ldg(w + t - 1), c_lo, c_hi, p.lam2);
            zshift += (double)p.lam2 * (double)se.delta * (double)se.delta;
            if (t > 1) off = rintf(cmax);
            const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), off2 = splat2(off);
            float4 *hrow = hist4 + (size_t)(t - 1) * (BPT * 32);
            float tmax = NEG_INF;
#pragma unroll
            for (int i = 0; i < BPT; ++i) {
                float Lj[K];
#pragma unroll
                for (int j = 0; j < K; ++j) Lj[j] = Lin[j * NB + i * 32 + lane];
                hrow[i * 32] = make_float4(Lj[0], Lj[1], Lj[2], Lj[3]);
                tmem_wait_ld(cb[i & 1]);
                if (i + 1 < BPT) tmem_ld16(tm + 16u * (i + 1), cb[(i + 1) & 1]);
                float2 out[K / 2];
#pragma unroll
                for (int h = 0; h < K / 2; ++h) {
                    float2 a[K];
#pragma unroll
                    for (int j = 0; j < K; ++j) a[j] = energy2(sub2(cb[i & 1][C::a_idx(j, h)], w2), nl2, kap2, splat2(Lj[j]));
                    const float2 m = max_pairs<K>(a);
                    float2 sum = ex2f2(sub2(a[0], m));
#pragma unroll
                    for (int j = 1; j < K; ++j) sum = add2(sum, ex2f2(sub2(a[j], m)));
                    out[h] = add2(sub2(m, off2), lg2f2(sum));
                    tmax = max3f(tmax, m.x, m.y);
                }
                *reinterpret_cast<float4 *>(Lout + (i * 32 + lane) * K) = make_float4(out[0].x, out[0].y, out[1].x, out[1].y);
            }
            cmax = warp_max(tmax) - off;                                   // maximum of the outputs as stored
            O += (int)off;
            if (lane == 0) O_g[t + 1] = O;
            __syncwarp();
        }
        // ================= log2 Z = O_{n+1} + LSE_q L_{n+1}(q); L_{n+1} sits in buffer n & 1
        float lsefin;
        {
            const float *Lfin = msg + (n & 1) * Q;
            float ssum = 0.f;
            for (int q = lane; q < Q; q += 32) ssum += ex2f(Lfin[q] - cmax);
            lsefin = cmax + lg2f(warp_sum(ssum));
        }
        if (lane == 0) diag_check_finite(p.diag, lsefin);
        const int Ofin = O;
        if (lane == 0 && p.logZ) p.logZ[blk] = (float)(((double)Ofin + (double)lsefin - zshift) * 0.6931471805599453);
        __syncwarp();
        // ================= beta sweep
        for (int q = lane; q < Q; q += 32) msg[q] = 0.f;                   // M_n = 0 in buffer 0
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * 32 + lane, tm + (uint32_t)(16 * i), true);
        tmem_wait_st();
        int P = 0;
        float offM = 0.f;
        // history stream: chunk c = butterfly (t = n - c / BPT, i = c % BPT), staged RD - 1 ahead with cp.async
        int nt = n, ni = 0;
        auto issue_chunk = [&](uint32_t slot) {
            const float4 *src = hist4 + (size_t)(nt - 1) * (BPT * 32) + ni * 32;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(stage_u32 + slot * 512u), "l"(src) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
            if (++ni == BPT) { ni = 0; if (nt > 1) --nt; }                 // past the end: the last step again, unread
        };
#pragma unroll
        for (uint32_t c = 0; c + 1 < RD; ++c) issue_chunk(c);
        uint32_t slot = 0;
        int Ot = O_g[n];
        __syncwarp();
        for (int t = n; t >= 1; --t) {
            const int cur = (n - t) & 1;
            const float *Min = msg + cur * Q;
            float *Mout = msg + (cur ^ 1) * Q;
            const int Onext = t > 1 ? O_g[t - 1] : 0;                      // requested a step ahead
            if (t < n) { P += (int)offM; offM = rintf(cmax); }
            const StepEnergy se = step_energy(__ldg(w + t - 1), c_lo, c_hi, p.lam2);
            const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), offM2 = splat2(offM);
            const float2 Dm2 = splat2((float)(Ofin - Ot - P) + lsefin);
            float2 num2 = make_float2(0.f, 0.f), den2 = make_float2(0.f, 0.f);
            float tmax = NEG_INF;
            float2 cb[2][8];
            tmem_ld16(tm, cb[0]);
#pragma unroll
            for (int i = 0; i < BPT; ++i) {
                issue_chunk(slot == 0 ? RD - 1 : slot - 1);                // refill the slot consumed last
                asm volatile("cp.async.wait_group %0;" ::"n"(RD - 1) : "memory");
                const float4 l4 = stage4[slot * 32 + lane];
                const float Lh[K] = {l4.x, l4.y, l4.z, l4.w};
                slot = slot + 1 == RD ? 0 : slot + 1;
                const float4 mv = *reinterpret_cast<const float4 *>(Min + (i * 32 + lane) * K);
                const float Mb[K] = {mv.x, mv.y, mv.z, mv.w};
                tmem_wait_ld(cb[i & 1]);
                if (i + 1 < BPT) tmem_ld16(tm + 16u * (i + 1), cb[(i + 1) & 1]);
#pragma unroll
                for (int jh = 0; jh < K / 2; ++jh) {
                    float2 uu[K];
#pragma unroll
                    for (int b = 0; b < K; ++b) uu[b] = energy2(sub2(cb[i & 1][C::b_idx(jh, b)], w2), nl2, kap2, splat2(Mb[b]));
                    const float2 m = max_pairs<K>(uu);
                    const float2 f = ex2f2(add2(sub2(m, Dm2), make_float2(Lh[2 * jh], Lh[2 * jh + 1])));
                    float2 pb = ex2f2(sub2(uu[0], m));
                    float2 sum = pb, craw = mul2(pb, cb[i & 1][C::b_idx(jh, 0)]);
#pragma unroll
                    for (int b = 1; b < K; ++b) {
                        pb = ex2f2(sub2(uu[b], m));
                        sum = add2(sum, pb);
                        craw = fma2(pb, cb[i & 1][C::b_idx(jh, b)], craw);
                    }
                    const float2 out = add2(sub2(m, offM2), lg2f2(sum));
                    tmax = max3f(tmax, m.x, m.y);
                    Mout[(2 * jh) * NB + i * 32 + lane] = out.x;            // M([j|x]) at j NB + x
                    Mout[(2 * jh + 1) * NB + i * 32 + lane] = out.y;
                    num2 = fma2(f, craw, num2);
                    den2 = fma2(f, sum, den2);
                }
            }
            const float nd = warp_sum2_split(num2.x + num2.y, den2.x + den2.y, lane);   // lane 0: numerator, lane 16: denominator
            const float den = __shfl_sync(0xffffffffu, nd, 16);
            cmax = warp_max(tmax) - offM;                                  // maximum of the outputs as stored
            if (lane == 0) {
                const float sw = nd / den;
                p.soft[blk * n + t - 1] = sw;
                if (p.soft_copy) p.soft_copy[blk * n + t - 1] = sw;
                bdef = fmaxf(bdef, fabsf(den - 1.f));
            }
            Ot = Onext;
            __syncwarp();
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        {
            // consistency: P_0 + LSE_q M_0(q) against log2 Z; M_0 sits in buffer n & 1
            P += (int)offM;
            const float *Mfin = msg + (n & 1) * Q;
            float ssum = 0.f;
            for (int q = lane; q < Q; q += 32) ssum += ex2f(Mfin[q] - cmax);
            const float lz_beta = cmax + lg2f(warp_sum(ssum));
            zgap = fmaxf(zgap, fabsf((float)(P - Ofin) + (lz_beta - lsefin)));
            defect = fmaxf(defect, bdef);
            if (lane == 0 && p.blk_defect) p.blk_defect[blk] = bdef;
        }
        __syncwarp();
    }
    if (lane == 0) {
        diag_max(&p.diag->max_defect, defect);
        diag_max(&p.diag->max_logz_gap, zgap);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

// Backward call: alpha sweep carrying (L, At), log Z, beta sweep carrying (M, Bt) with the gradient contraction
// (see bcjr_duo.cuh for the arithmetic); table and gradient accumulators in the warp's tensor-memory columns.
// p.gc_part: [warps][S] partial codebook gradients (one per resident warp, written once at the end); p.hist:
// [warps][n][BPT][2][32] float4; p.stepO: [warps][n + 2].
template <int LB, bool ACC>
__global__ void __launch_bounds__(WarpCfg<LB, true>::THREADS, 1) bwd_warp_kernel(BwdParams p)
{
    using C = WarpCfg<LB, true>;
    constexpr int K = C::K, NB = C::NB, Q = C::Q, BPT = C::BPT, RD = C::RD;
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float invT = p.invT;
    const float2 nl2 = splat2(-p.lam2);
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);

    float *msg = smem + warp * C::PER_WARP;                               // [2 parities][L | At][Q]
    float4 *stage4 = reinterpret_cast<float4 *>(msg + C::MSG);          // [RD][2][32], thread-private entries
    const uint32_t stage_u32 = smem_u32(stage4) + (uint32_t)lane * 16u;
    const int64_t wg = (int64_t)blockIdx.x * C::NWARP + warp, nwg = (int64_t)gridDim.x * C::NWARP;
    float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)wg * n * 2 * Q) + lane;   // row t: [BPT][2][32]
    int *O_g = p.stepO + (size_t)wg * (n + 2);

    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm_cb = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * C::COLS);
    const uint32_t tm_acc = tm_cb + 16u * BPT;
    if (ACC) {
        float2 z[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < BPT; ++i) tmem_st16(tm_acc + 16u * i, z);
        tmem_wait_st();
    }
    float defect = 0.f;

    for (int64_t blk = wg; blk < p.B; blk += nwg) {
        const float *w_s = p.W + blk * n, *g_s = p.g + blk * n, *sf_s = p.soft + blk * n;
        {
            const float gsh1 = -__ldg(g_s) * __ldg(sf_s);                 // L_1 = 0; the At array carries At + gsh (see bcjr_duo.cuh)
            for (int q = lane; q < Q; q += 32) { msg[q] = 0.f; msg[Q + q] = gsh1; }
        }
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * 32 + lane, tm_cb + (uint32_t)(16 * i), false);
        tmem_wait_st();
        int O = 0;
        float off = 0.f, cmax = 0.f;
        if (lane == 0) O_g[1] = 0;
        __syncwarp();
        // ================= alpha sweep carrying (L, At)
        for (int t = 1; t <= n; ++t) {
            const int cur = (t - 1) & 1;
            const float *Lin = msg + cur * 2 * Q, *Ain = Lin + Q;
            float *Lout = msg + (cur ^ 1) * 2 * Q, *Aout = Lout + Q;
            float2 cb[2][8];
            tmem_ld16(tm_cb, cb[0]);
            const float gt = __ldg(g_s + t - 1);
            const float gshn = t < n ? -__ldg(g_s + t) * __ldg(sf_s + t) : 0.f;
            const StepEnergy se = step_energy(__ldg(w_s + t - 1), c_lo, c_hi, p.lam2);
            if (t > 1) off = rintf(cmax);
            const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), off2 = splat2(off), gshn2 = splat2(gshn);
            float4 *hrow = hist4 + (size_t)(t - 1) * (BPT * 2 * 32);
            float tmax = NEG_INF;
#pragma unroll
            for (int i = 0; i < BPT; ++i) {
                float Lj[K], Aj[K];
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    Lj[j] = Lin[j * NB + i * 32 + lane];
                    Aj[j] = Ain[j * NB + i * 32 + lane];
                }
                hrow[(i * 2) * 32] = make_float4(Lj[0], Lj[1], Lj[2], Lj[3]);
                hrow[(i * 2 + 1) * 32] = make_float4(Aj[0], Aj[1], Aj[2], Aj[3]);
                tmem_wait_ld(cb[i & 1]);
                if (i + 1 < BPT) tmem_ld16(tm_cb + 16u * (i + 1), cb[(i + 1) & 1]);
                float2 outL[K / 2], outA[K / 2];
#pragma unroll
                for (int h = 0; h < K / 2; ++h) {
                    float2 a[K];
#pragma unroll
                    for (int j = 0; j < K; ++j) a[j] = energy2(sub2(cb[i & 1][C::a_idx(j, h)], w2), nl2, kap2, splat2(Lj[j]));
                    const float2 m = max_pairs<K>(a);
                    float2 pj = ex2f2(sub2(a[0], m));
                    float2 sum = pj, ax = mul2(pj, fma2(g2, cb[i & 1][C::a_idx(0, h)], splat2(Aj[0])));
#pragma unroll
                    for (int j = 1; j < K; ++j) {
                        pj = ex2f2(sub2(a[j], m));
                        sum = add2(sum, pj);
                        ax = fma2(pj, fma2(g2, cb[i & 1][C::a_idx(j, h)], splat2(Aj[j])), ax);
                    }
                    outL[h] = add2(sub2(m, off2), lg2f2(sum));
                    outA[h] = fma2(ax, rcpf2(sum), gshn2);
                    tmax = max3f(tmax, m.x, m.y);
                }
                *reinterpret_cast<float4 *>(Lout + (i * 32 + lane) * K) = make_float4(outL[0].x, outL[0].y, outL[1].x, outL[1].y);
                *reinterpret_cast<float4 *>(Aout + (i * 32 + lane) * K) = make_float4(outA[0].x, outA[0].y, outA[1].x, outA[1].y);
            }
            cmax = warp_max(tmax) - off;
            O += (int)off;
            if (lane == 0) O_g[t + 1] = O;
            __syncwarp();
        }
        // ================= log2 Z
        float lsefin;
        {
            const float *Lfin = msg + (n & 1) * 2 * Q;
            float ssum = 0.f;
            for (int q = lane; q < Q; q += 32) ssum += ex2f(Lfin[q] - cmax);
            lsefin = cmax + lg2f(warp_sum(ssum));
        }
        if (lane == 0) diag_check_finite(p.diag, lsefin);
        const int Ofin = O;
        __syncwarp();
        // ================= beta sweep carrying (M, Bt), with the gradient contraction
        {
            const float gshn = -__ldg(g_s + n - 1) * __ldg(sf_s + n - 1);   // M_n = 0, Bt_n = 0 (+ centring shift)
            for (int q = lane; q < Q; q += 32) { msg[q] = 0.f; msg[Q + q] = gshn; }
        }
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * 32 + lane, tm_cb + (uint32_t)(16 * i), true);
        tmem_wait_st();
        int P = 0;
        float offM = 0.f;
        int nt = n, ni = 0;
        auto issue_chunk = [&](uint32_t slot) {
            const float4 *src = hist4 + (size_t)(nt - 1) * (BPT * 2 * 32) + ni * 64;
            const uint32_t dst = stage_u32 + slot * 1024u;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 512u), "l"(src + 32) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
            if (++ni == BPT) { ni = 0; if (nt > 1) --nt; }
        };
#pragma unroll
        for (uint32_t c = 0; c + 1 < RD; ++c) issue_chunk(c);
        uint32_t slot = 0;
        int Ot = O_g[n];
        __syncwarp();
        for (int t = n; t >= 1; --t) {
            const int cur = (n - t) & 1;
            const float *Min = msg + cur * 2 * Q, *Bin = Min + Q;
            float *Mout = msg + (cur ^ 1) * 2 * Q, *Bout = Mout + Q;
            const int Onext = t > 1 ? O_g[t - 1] : 0;
            if (t < n) { P += (int)offM; offM = rintf(cmax); }
            const float wt = __ldg(w_s + t - 1), gt = __ldg(g_s + t - 1), st = __ldg(sf_s + t - 1);
            const float gsh = -gt * st;                                     // shift carried by the stored At
            const float gshp = t > 1 ? -__ldg(g_s + t - 2) * __ldg(sf_s + t - 2) : 0.f;   // for step t-1
            const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
            const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), ngi2 = splat2(-invT), gid2 = splat2(invT * se.delta);
            const float2 gsh2 = splat2(gsh), gshp2 = splat2(gshp), offM2 = splat2(offM);
            const float2 Dm2 = splat2((float)(Ofin - Ot - P) + lsefin);
            float2 S0 = make_float2(0.f, 0.f), S2 = S0, ZS = S0;
            float tmax = NEG_INF;
            float2 cb[2][8];
            tmem_ld16(tm_cb, cb[0]);
#pragma unroll
            for (int i = 0; i < BPT; ++i) {
                issue_chunk(slot == 0 ? RD - 1 : slot - 1);
                asm volatile("cp.async.wait_group %0;" ::"n"(RD - 1) : "memory");
                const float4 l4 = stage4[slot * 64 + lane], a4 = stage4[slot * 64 + 32 + lane];
                const float Lh[K] = {l4.x, l4.y, l4.z, l4.w}, Ah[K] = {a4.x, a4.y, a4.z, a4.w};
                slot = slot + 1 == RD ? 0 : slot + 1;
                const float4 mv = *reinterpret_cast<const float4 *>(Min + (i * 32 + lane) * K);
                const float4 bv = *reinterpret_cast<const float4 *>(Bin + (i * 32 + lane) * K);
                const float Mb[K] = {mv.x, mv.y, mv.z, mv.w}, Yb[K] = {bv.x, bv.y, bv.z, bv.w};
                float2 acc[8];
                tmem_wait_ld(cb[i & 1]);
                if (ACC) tmem_ld16(tm_acc + 16u * i, acc);
                if (i + 1 < BPT) tmem_ld16(tm_cb + 16u * (i + 1), cb[(i + 1) & 1]);
                bool acc_ready = !ACC;
#pragma unroll
                for (int jh = 0; jh < K / 2; ++jh) {
                    float2 uu[K], d[K];
#pragma unroll
                    for (int b = 0; b < K; ++b) {
                        d[b] = sub2(cb[i & 1][C::b_idx(jh, b)], w2);        // du = c - wc
                        uu[b] = energy2(d[b], nl2, kap2, splat2(Mb[b]));
                    }
                    const float2 m = max_pairs<K>(uu);
                    const float2 Ahj = sub2(make_float2(Ah[2 * jh], Ah[2 * jh + 1]), gsh2);
                    const float2 f = ex2f2(add2(sub2(m, Dm2), make_float2(Lh[2 * jh], Lh[2 * jh + 1])));
                    const float2 fg = mul2(f, g2), nfi = mul2(f, ngi2), fid = mul2(f, gid2);   // f (w - c) / T = f delta / T - (f / T) du
                    if (!acc_ready) { tmem_wait_ld(acc); acc_ready = true; }
                    float2 sum = make_float2(0.f, 0.f), ya = sum, zs = sum;
#pragma unroll
                    for (int b = 0; b < K; ++b) {
                        const float2 pb = ex2f2(sub2(uu[b], m));
                        const float2 y = fma2(g2, cb[i & 1][C::b_idx(jh, b)], splat2(Yb[b]));   // h + Bt
                        const float2 z = fma2(fma2(nfi, d[b], fid), add2(y, Ahj), fg);            // f (g + (w - c) r / T)
                        sum = add2(sum, pb);
                        ya = fma2(pb, y, ya);
                        zs = fma2(pb, z, zs);
                        if (ACC) acc[C::b_idx(jh, b)] = fma2(pb, z, acc[C::b_idx(jh, b)]);
                    }
                    const float2 outM = add2(sub2(m, offM2), lg2f2(sum));
                    const float2 outB = fma2(ya, rcpf2(sum), gshp2);
                    tmax = max3f(tmax, m.x, m.y);
                    Mout[(2 * jh) * NB + i * 32 + lane] = outM.x; Mout[(2 * jh + 1) * NB + i * 32 + lane] = outM.y;
                    Bout[(2 * jh) * NB + i * 32 + lane] = outB.x; Bout[(2 * jh + 1) * NB + i * 32 + lane] = outB.y;
                    S0 = fma2(f, sum, S0);
                    S2 = fma2(f, fma2(Ahj, sum, ya), S2);
                    ZS = add2(ZS, zs);
                }
                if (ACC) tmem_st16(tm_acc + 16u * i, acc);
            }
            if (ACC) tmem_wait_st();
            cmax = warp_max(tmax) - offM;
            // lanes 0-7 hold sum gamma, 8-15 sum gamma r, 16-23 sum gamma z
            const float s3 = warp_sum3_split(S0.x + S0.y, S2.x + S2.y, ZS.x + ZS.y, lane);
            const float a2 = __shfl_sync(0xffffffffu, s3, 8), az = __shfl_sync(0xffffffffu, s3, 16);
            if (lane == 0) {
                const float i0 = 1.f / s3;
                p.gW[blk * n + t - 1] = (gt - az * i0) + (a2 * i0) * (wt - st) * invT;
                defect = fmaxf(defect, fabsf(s3 - 1.f));
            }
            Ot = Onext;
            __syncwarp();
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncwarp();
    }
    if (ACC) {
        // this warp's partial of grad_codebook: beta pair (jh, b) of butterfly x holds states [2jh | x | b], [2jh+1 | x | b]
        float *gc = p.gc_part + (size_t)wg * C::S;
        tmem_wait_st();
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            const int x = i * 32 + lane;
            float2 acc[8];
            tmem_ld16(tm_acc + 16u * i, acc);
            tmem_wait_ld(acc);
#pragma unroll
            for (int jh = 0; jh < K / 2; ++jh)
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    gc[(size_t)(2 * jh) * Q + (size_t)x * K + b] = acc[C::b_idx(jh, b)].x;
                    gc[(size_t)(2 * jh + 1) * Q + (size_t)x * K + b] = acc[C::b_idx(jh, b)].y;
                }
        }
    }
    if (lane == 0) diag_max(&p.diag->max_defect, defect);
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

// Backward call with grad_codebook at Lb = 12, 13: TWO warps per weight block.
//
// Table plus accumulators are 2 x 2^Lb floats per block; with one warp per block that is 256 (Lb = 12) or 512 (Lb = 13)
// columns per lane, so only eight or four warps fit an SM and the schedulers run short of warps to pick from (issue
// slots two thirds used).  Here the butterflies of a block are split between two warps -- half the columns each, twice
// the warps per SM for the same number of resident blocks.  The pair shares the block's message buffers; one named
// barrier of 64 threads per step orders them (the gauge maximum and the posterior sums of the two warps meet in a few
// words of shared memory, read after that barrier).  Everything else is bwd_warp_kernel.
template <int LB_>
struct Warp2Cfg {
    using W = WarpCfg<LB_, true>;
    static constexpr int LB = LB_, KB = 2, K = 4, S = W::S, Q = W::Q, NB = W::NB;
    static constexpr int BPT = W::BPT / 2;                     // butterflies per lane and warp: 4 (Lb = 12), 8 (Lb = 13)
    static constexpr int UNITS = 1, HPU = 2;
    static constexpr int COLS = 32 * BPT;                      // table + accumulators
    static constexpr int NWARP = 2048 / COLS < 16 ? 2048 / COLS : 16;
    static constexpr int NPAIR = NWARP / 2, THREADS = 32 * NWARP;
    static constexpr int RD = BPT < 8 ? BPT : 8;
    static constexpr int MSG = 4 * Q;                          // floats per pair: two parities of (L, At)
    static constexpr int RING = RD * 2 * 32 * 4;               // floats per warp
    static constexpr int XCH = 32;                             // floats per pair: gauge maxima [2][2], sums [2][2][4], log Z partials [2]
    static constexpr int PER_PAIR = MSG + 2 * RING + XCH;
    static constexpr int OFF_TMEM = NPAIR * PER_PAIR;
    static constexpr int SMEM_FLOATS = OFF_TMEM + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(LB == 12 || LB == 13, "two warps per block: 2^12 and 2^13 states");
    static_assert(SMEM_BYTES <= 227 * 1024, "shared memory");
    static_assert(NPAIR + 1 <= 15, "one named barrier per pair");
    __host__ __device__ static constexpr int a_idx(int j, int h) { return 2 * j + h; }
    __host__ __device__ static constexpr int b_idx(int jh, int b) { return 4 * jh + b; }
};

__device__ __forceinline__ void pair_barrier(int pair)
{
    asm volatile("bar.sync %0, 64;" ::"r"(pair + 1) : "memory");
}

// p.gc_part: [pairs][S]; p.hist: [pairs][n][2 warps][BPT][2][32] float4; p.stepO: [pairs][n + 2].
template <int LB>
__global__ void __launch_bounds__(Warp2Cfg<LB>::THREADS, 1) bwd_warp2_kernel(BwdParams p)
{
    using C = Warp2Cfg<LB>;
    constexpr int K = C::K, NB = C::NB, Q = C::Q, BPT = C::BPT, RD = C::RD;
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, pw = warp & 1, pair = warp >> 1;
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float invT = p.invT;
    const float2 nl2 = splat2(-p.lam2);
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);

    float *msg = smem + pair * C::PER_PAIR;                               // [2 parities][L | At][Q], shared by the pair
    float4 *stage4 = reinterpret_cast<float4 *>(msg + C::MSG + pw * C::RING);   // [RD][2][32], thread-private entries
    float *xch = msg + C::MSG + 2 * C::RING;
    float *wm = xch;                                                      // [2 parities][2 warps]
    float *part = xch + 4;                                                // [2 parities][2 warps][4]
    float *lzp = xch + 20;                                                // [2 warps]
    const uint32_t stage_u32 = smem_u32(stage4) + (uint32_t)lane * 16u;
    const int64_t pg = (int64_t)blockIdx.x * C::NPAIR + pair, npg = (int64_t)gridDim.x * C::NPAIR;
    const int x0 = pw * BPT * 32 + lane;                                  // this thread's butterflies: x0 + 32 i
    float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)pg * n * 2 * Q) + pw * (BPT * 2 * 32) + lane;   // row t: [2][BPT][2][32]
    constexpr int HROW = 2 * BPT * 2 * 32;
    int *O_g = p.stepO + (size_t)pg * (n + 2);

    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm_cb = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * C::COLS);
    const uint32_t tm_acc = tm_cb + 16u * BPT;
    {
        float2 z[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = make_float2(0.f, 0.f);
#pragma unroll
        for (int i = 0; i < BPT; ++i) tmem_st16(tm_acc + 16u * i, z);
        tmem_wait_st();
    }
    float defect = 0.f;

    for (int64_t blk = pg; blk < p.B; blk += npg) {
        const float *w_s = p.W + blk * n, *g_s = p.g + blk * n, *sf_s = p.soft + blk * n;
        {
            const float gsh1 = -__ldg(g_s) * __ldg(sf_s);                 // L_1 = 0; the At array carries At + gsh (see bcjr_duo.cuh)
            for (int q = pw * 32 + lane; q < Q; q += 64) { msg[q] = 0.f; msg[Q + q] = gsh1; }
        }
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, x0 + 32 * i, tm_cb + (uint32_t)(16 * i), false);
        tmem_wait_st();
        int O = 0;
        float off = 0.f, cmax = 0.f;
        if (pw == 0 && lane == 0) O_g[1] = 0;
        pair_barrier(pair);
        // ================= alpha sweep carrying (L, At)
        for (int t = 1; t <= n; ++t) {
            const int cur = (t - 1) & 1;
            const float *Lin = msg + cur * 2 * Q, *Ain = Lin + Q;
            float *Lout = msg + (cur ^ 1) * 2 * Q, *Aout = Lout + Q;
            float2 cb[2][8];
            tmem_ld16(tm_cb, cb[0]);
            const float gt = __ldg(g_s + t - 1);
            const float gshn = t < n ? -__ldg(g_s + t) * __ldg(sf_s + t) : 0.f;
            const StepEnergy se = step_energy(__ldg(w_s + t - 1), c_lo, c_hi, p.lam2);
            if (t > 1) {
                cmax = fmaxf(wm[cur * 2], wm[cur * 2 + 1]) - off;            // maximum of this step's inputs as stored
                off = rintf(cmax);
            }
            const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), off2 = splat2(off), gshn2 = splat2(gshn);
            float4 *hrow = hist4 + (size_t)(t - 1) * HROW;
            float tmax = NEG_INF;
#pragma unroll
            for (int i = 0; i < BPT; ++i) {
                const int x = x0 + 32 * i;
                float Lj[K], Aj[K];
#pragma unroll
                for (int j = 0; j < K; ++j) {
                    Lj[j] = Lin[j * NB + x];
                    Aj[j] = Ain[j * NB + x];
                }
                hrow[(i * 2) * 32] = make_float4(Lj[0], Lj[1], Lj[2], Lj[3]);
                hrow[(i * 2 + 1) * 32] = make_float4(Aj[0], Aj[1], Aj[2], Aj[3]);
                tmem_wait_ld(cb[i & 1]);
                if (i + 1 < BPT) tmem_ld16(tm_cb + 16u * (i + 1), cb[(i + 1) & 1]);
                float2 outL[K / 2], outA[K / 2];
#pragma unroll
                for (int h = 0; h < K / 2; ++h) {
                    float2 a[K];
#pragma unroll
                    for (int j = 0; j < K; ++j) a[j] = energy2(sub2(cb[i & 1][C::a_idx(j, h)], w2), nl2, kap2, splat2(Lj[j]));
                    const float2 m = max_pairs<K>(a);
                    float2 pj = ex2f2(sub2(a[0], m));
                    float2 sum = pj, ax = mul2(pj, fma2(g2, cb[i & 1][C::a_idx(0, h)], splat2(Aj[0])));
#pragma unroll
                    for (int j = 1; j < K; ++j) {
                        pj = ex2f2(sub2(a[j], m));
                        sum = add2(sum, pj);
                        ax = fma2(pj, fma2(g2, cb[i & 1][C::a_idx(j, h)], splat2(Aj[j])), ax);
                    }
                    outL[h] = add2(sub2(m, off2), lg2f2(sum));
                    outA[h] = fma2(ax, rcpf2(sum), gshn2);
                    tmax = max3f(tmax, m.x, m.y);
                }
                *reinterpret_cast<float4 *>(Lout + x * K) = make_float4(outL[0].x, outL[0].y, outL[1].x, outL[1].y);
                *reinterpret_cast<float4 *>(Aout + x * K) = make_float4(outA[0].x, outA[0].y, outA[1].x, outA[1].y);
            }
            tmax = warp_max(tmax);
            if (lane == 0) wm[(cur ^ 1) * 2 + pw] = tmax;
            O += (int)off;
            if (pw == 0 && lane == 0) O_g[t + 1] = O;
            pair_barrier(pair);
        }
        // ================= log2 Z
        cmax = fmaxf(wm[(n & 1) * 2], wm[(n & 1) * 2 + 1]) - off;
        float lsefin;
        {
            const float *Lfin = msg + (n & 1) * 2 * Q;
            float ssum = 0.f;
            for (int q = pw * 32 + lane; q < Q; q += 64) ssum += ex2f(Lfin[q] - cmax);
            ssum = warp_sum(ssum);
            if (lane == 0) lzp[pw] = ssum;
            pair_barrier(pair);
            lsefin = cmax + lg2f(lzp[0] + lzp[1]);
        }
        if (pw == 0 && lane == 0) diag_check_finite(p.diag, lsefin);
        const int Ofin = O;
        pair_barrier(pair);                                               // everybody has read the last alpha messages and lzp
        // ================= beta sweep carrying (M, Bt), with the gradient contraction
        {
            const float gshn = -__ldg(g_s + n - 1) * __ldg(sf_s + n - 1);   // M_n = 0, Bt_n = 0 (+ centring shift)
            for (int q = pw * 32 + lane; q < Q; q += 64) { msg[q] = 0.f; msg[Q + q] = gshn; }
        }
#pragma unroll
        for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, x0 + 32 * i, tm_cb + (uint32_t)(16 * i), true);
        tmem_wait_st();
        int P = 0;
        float offM = 0.f;
        int nt = n, ni = 0;
        auto issue_chunk = [&](uint32_t slot) {
            const float4 *src = hist4 + (size_t)(nt - 1) * HROW + ni * 64;
            const uint32_t dst = stage_u32 + slot * 1024u;
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
            asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 512u), "l"(src + 32) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
            if (++ni == BPT) { ni = 0; if (nt > 1) --nt; }
        };
#pragma unroll
        for (uint32_t c = 0; c + 1 < RD; ++c) issue_chunk(c);
        uint32_t slot = 0;
        int Ot = O_g[n];
        // pair, warp 0, lane 0: turn the sums of step t (slots of parity b) into grad_W[t]
        auto finish_step = [&](int t, int b) {
            if (pw == 0 && lane == 0) {
                const float *pp = part + b * 8;
                const float a0 = pp[0] + pp[4], a2 = pp[1] + pp[5], az = pp[2] + pp[6];
                const float i0 = 1.f / a0;
                p.gW[blk * n + t - 1] = (__ldg(g_s + t - 1) - az * i0) + (a2 * i0) * (__ldg(w_s + t - 1) - __ldg(sf_s + t - 1)) * invT;
                defect = fmaxf(defect, fabsf(a0 - 1.f));
            }
        };
        pair_barrier(pair);
        for (int t = n; t >= 1; --t) {
            const int cur = (n - t) & 1;
            const float *Min = msg + cur * 2 * Q, *Bin = Min + Q;
            float *Mout = msg + (cur ^ 1) * 2 * Q, *Bout = Mout + Q;
            const int Onext = t > 1 ? O_g[t - 1] : 0;
            if (t < n) {
                P += (int)offM;
                cmax = fmaxf(wm[cur * 2], wm[cur * 2 + 1]);
                offM = rintf(cmax);
                finish_step(t + 1, cur);
            }
            const float wt = __ldg(w_s + t - 1), gt = __ldg(g_s + t - 1), st = __ldg(sf_s + t - 1);
            const float gsh = -gt * st;                                     // shift carried by the stored At
            const float gshp = t > 1 ? -__ldg(g_s + t - 2) * __ldg(sf_s + t - 2) : 0.f;   // for step t-1
            const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
            const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), ngi2 = splat2(-invT), gid2 = splat2(invT * se.delta);
            const float2 gsh2 = splat2(gsh), gshp2 = splat2(gshp), offM2 = splat2(offM);
            const float2 Dm2 = splat2((float)(Ofin - Ot - P) + lsefin);
            float2 S0 = make_float2(0.f, 0.f), S2 = S0, ZS = S0;
            float tmax = NEG_INF;
            float2 cb[2][8];
            tmem_ld16(tm_cb, cb[0]);
#pragma unroll
            for (int i = 0; i < BPT; ++i) {
                const int x = x0 + 32 * i;
                issue_chunk(slot == 0 ? RD - 1 : slot - 1);
                asm volatile("cp.async.wait_group %0;" ::"n"(RD - 1) : "memory");
                const float4 l4 = stage4[slot * 64 + lane], a4 = stage4[slot * 64 + 32 + lane];
                const float Lh[K] = {l4.x, l4.y, l4.z, l4.w}, Ah[K] = {a4.x, a4.y, a4.z, a4.w};
                slot = slot + 1 == RD ? 0 : slot + 1;
                const float4 mv = *reinterpret_cast<const float4 *>(Min + x * K);
                const float4 bv = *reinterpret_cast<const float4 *>(Bin + x * K);
                const float Mb[K] = {mv.x, mv.y, mv.z, mv.w}, Yb[K] = {bv.x, bv.y, bv.z, bv.w};
                float2 acc[8];
                tmem_wait_ld(cb[i & 1]);
                tmem_ld16(tm_acc + 16u * i, acc);
                if (i + 1 < BPT) tmem_ld16(tm_cb + 16u * (i + 1), cb[(i + 1) & 1]);
                bool acc_ready = false;
#pragma unroll
                for (int jh = 0; jh < K / 2; ++jh) {
                    float2 uu[K], d[K];
#pragma unroll
                    for (int b = 0; b < K; ++b) {
                        d[b] = sub2(cb[i & 1][C::b_idx(jh, b)], w2);        // du = c - wc
                        uu[b] = energy2(d[b], nl2, kap2, splat2(Mb[b]));
                    }
                    const float2 m = max_pairs<K>(uu);
                    const float2 Ahj = sub2(make_float2(Ah[2 * jh], Ah[2 * jh + 1]), gsh2);
                    const float2 f = ex2f2(add2(sub2(m, Dm2), make_float2(Lh[2 * jh], Lh[2 * jh + 1])));
                    const float2 fg = mul2(f, g2), nfi = mul2(f, ngi2), fid = mul2(f, gid2);   // f (w - c) / T = f delta / T - (f / T) du
                    if (!acc_ready) { tmem_wait_ld(acc); acc_ready = true; }
                    float2 sum = make_float2(0.f, 0.f), ya = sum, zs = sum;
#pragma unroll
                    for (int b = 0; b < K; ++b) {
                        const float2 pb = ex2f2(sub2(uu[b], m));
                        const float2 y = fma2(g2, cb[i & 1][C::b_idx(jh, b)], splat2(Yb[b]));   // h + Bt
                        const float2 z = fma2(fma2(nfi, d[b], fid), add2(y, Ahj), fg);            // f (g + (w - c) r / T)
                        sum = add2(sum, pb);
                        ya = fma2(pb, y, ya);
                        zs = fma2(pb, z, zs);
                        acc[C::b_idx(jh, b)] = fma2(pb, z, acc[C::b_idx(jh, b)]);
                    }
                    const float2 outM = add2(sub2(m, offM2), lg2f2(sum));
                    const float2 outB = fma2(ya, rcpf2(sum), gshp2);
                    tmax = max3f(tmax, m.x, m.y);
                    Mout[(2 * jh) * NB + x] = outM.x; Mout[(2 * jh + 1) * NB + x] = outM.y;
                    Bout[(2 * jh) * NB + x] = outB.x; Bout[(2 * jh + 1) * NB + x] = outB.y;
                    S0 = fma2(f, sum, S0);
                    S2 = fma2(f, fma2(Ahj, sum, ya), S2);
                    ZS = add2(ZS, zs);
                }
                tmem_st16(tm_acc + 16u * i, acc);
            }
            tmem_wait_st();
            tmax = warp_max(tmax) - offM;
            // lanes 0-7 hold sum gamma, 8-15 sum gamma r, 16-23 sum gamma z
            const float s3 = warp_sum3_split(S0.x + S0.y, S2.x + S2.y, ZS.x + ZS.y, lane);
            if (lane == 0) wm[(cur ^ 1) * 2 + pw] = tmax;
            if ((lane & 7) == 0 && lane < 24) part[(cur ^ 1) * 8 + pw * 4 + (lane >> 3)] = s3;
            Ot = Onext;
            pair_barrier(pair);
        }
        finish_step(1, n & 1);
        asm volatile("cp.async.wait_all;" ::: "memory");
        pair_barrier(pair);                                               // the exchange words are free for the next block
    }
    {
        // this pair's partial of grad_codebook: beta pair (jh, b) of butterfly x holds states [2jh | x | b], [2jh+1 | x | b]
        float *gc = p.gc_part + (size_t)pg * C::S;
        tmem_wait_st();
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            const int x = x0 + 32 * i;
            float2 acc[8];
            tmem_ld16(tm_acc + 16u * i, acc);
            tmem_wait_ld(acc);
#pragma unroll
            for (int jh = 0; jh < K / 2; ++jh)
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    gc[(size_t)(2 * jh) * Q + (size_t)x * K + b] = acc[C::b_idx(jh, b)].x;
                    gc[(size_t)(2 * jh + 1) * Q + (size_t)x * K + b] = acc[C::b_idx(jh, b)].y;
                }
        }
    }
    if (pw == 0 && lane == 0) diag_max(&p.diag->max_defect, defect);
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
