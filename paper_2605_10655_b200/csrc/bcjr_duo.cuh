// Backward call for the 2^16-state trellis (k = 2): one weight block per cluster of TWO CTAs,
// codebook AND codebook-gradient accumulators in tensor memory.
//
// The backward pass needs, per state, the codebook entry and a gradient accumulator (2 x 256 KB
// per block) next to the (L, At) / (M, Bt) message pairs.  A pair of SMs holds that only if the
// tensor memory is used: each CTA keeps its half of the codebook (64 columns per thread) and its
// half of the accumulators (64 columns per thread) in TMEM, lane-private, exactly the access
// pattern of a thread that owns the same butterflies for the whole kernel.  Registers are then
// free for the arithmetic, shared memory for the messages and the history staging, and clusters
// of two fill all 148 SMs (clusters of four, needed when the accumulators live in registers,
// fill only 132).
//
// Step protocol.  Messages are double-buffered.  Half of a CTA's outputs are consumed by the CTA
// itself, half by its peer (the perfect shuffle leaves no better split).  The peer's half is
// pushed with st.async into the peer's buffer `ob` and credits the peer's mbarrier full[ob] with
// its bytes; the own half is written with plain shared-memory stores, because st.async sustains
// only ~10 bytes per clock per SM, whatever the destination: with all 64 KB of a step's outputs
// on it, it alone set the step time (6.9 k clocks per step; 5.3 k with the own half off it).  A
// phase of full[ob] completes when (a) the peer's bytes have landed and (b) every warp of the
// cluster has arrived on it after its last butterfly of the step -- so nobody still reads the
// other buffer when the next step starts overwriting it.  A warp arrives on its own CTA's
// barrier with release semantics at CTA scope (that publishes its plain stores to the warps that
// wait on the barrier) and on the peer's barrier relaxed: there it has nothing to publish (the
// data travels with st.async and is accounted in bytes), and the reads the arrival has to follow
// are complete when it issues, because every value a warp reads from its input buffer feeds,
// through register dependences, a store that precedes the arrival in program order.  (A release
// arrival at cluster scope per warp costs a fence: 8 % of the kernel.)
//
// History.  The inputs (L, At) of a butterfly in the alpha sweep are exactly what the same thread
// needs for that butterfly in the beta sweep, so the history is thread-private: the thread stores
// its inputs with 16-byte global stores ([step][CTA][butterfly slot][16-byte chunk][thread]) and
// streams them back with cp.async into its own staging slots, a whole step ahead (one
// cp.async.wait_group per step; no mbarrier, no producer thread, no branch in the butterfly loop).
#pragma once
#include "bcjr_solo.cuh"

namespace bcjr {



template <int KB_>
struct DuoCfg {
    static constexpr int LB = 16, KB = KB_, K = 1 << KB, S = 1 << LB, Q = S >> KB, NB = S >> (2 * KB);
    static constexpr int CL = 2;
    static constexpr int NBC = NB / CL, QC = Q / CL;
    static constexpr int THREADS = 512, NWARP = THREADS / 32;
    static constexpr int BPT = NBC / THREADS;                  // butterflies per thread: 4 (k = 2), 1 (k = 3)
    static constexpr int UNITS = K * K / 16;                   // 16-column TMEM units per butterfly
    static constexpr int HPU = (K / 2) / UNITS;                // pairs h (alpha) / jh (beta) per unit
    static constexpr int SLOTS = CL * NWARP;                   // 32 per-warp partial slots
    static constexpr int NCH = 2 * K / 4;                      // 16-byte chunks per butterfly and thread: K values of L, K of At
    static constexpr int RD = BPT;                             // staging slots: one per butterfly of a step
    static constexpr int MAX_N = 1024;
    static constexpr int ARRIVALS = 1 + SLOTS;                 // armer + one arrival per warp of the cluster
    static constexpr int OFF_MSG = 0;                          // [2 parity][2 arrays][QC]
    static constexpr int OFF_RING = OFF_MSG + 4 * QC;          // float4 [RD][NCH][THREADS]
    static constexpr int OFF_O = OFF_RING + RD * NCH * THREADS * 4;   // int [MAX_N + 2]
    static constexpr int OFF_WMAX = OFF_O + MAX_N + 2 + 2;     // [2][32]
    static constexpr int OFF_PART = OFF_WMAX + 64;             // [2][32][4]
    static constexpr int OFF_LZ = OFF_PART + 256;              // [32]
    static constexpr int OFF_MBAR = OFF_LZ + 32;               // uint64: full[2]
    static constexpr int NMBAR = 2;
    static constexpr int OFF_TMEM = OFF_MBAR + 2 * NMBAR;
    static constexpr int OFF_FLAG = OFF_TMEM + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 2;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(OFF_MBAR % 2 == 0, "mbarrier alignment");
    static_assert(2 * BPT * K * K == 128, "codebook + accumulators fill the thread's 128 TMEM columns");
    static_assert(CL == 2 && K % (2 * CL) == 0, "beta destinations: CTA of output j is j*CL/K");
    static_assert(UNITS * HPU == K / 2 && (K == 4 || K == 8), "unit decomposition");
    __host__ __device__ static constexpr int a_idx(int j, int h) { return K == 4 ? 2 * j + h : j; }
    __host__ __device__ static constexpr int b_idx(int jh, int b) { return K == 4 ? 4 * jh + b : b; }
};

// BETA_ONLY = true: the beta sweeps alone, on the history, gauge offsets and log Z tail that bwd_alpha_kernel
// (bcjr_alpha.cuh) wrote for the same blocks (block b of the call: history at p.hist + b n 2Q, offsets at
// p.stepO + b (MAX_N + 4)); the partial codebook gradient is then ADDED to p.gc_part.
template <int KB, bool BETA_ONLY = false>
__global__ void __launch_bounds__(DuoCfg<KB>::THREADS, 1) bwd_duo_kernel(BwdParams p)
{
    using C = DuoCfg<KB>;
    constexpr int K = C::K, NB = C::NB, NBC = C::NBC, QC = C::QC, BPT = C::BPT, NWARP = C::NWARP, CT = C::THREADS;
    constexpr int CL = C::CL, SLOTS = C::SLOTS, NCH = C::NCH, RD = C::RD, UNITS = C::UNITS, HPU = C::HPU, NU = BPT * UNITS;
    constexpr int KK = K * K;
    constexpr uint32_t BUF_BYTES = 2u * QC * 4u;                 // (L, At) of one parity
    constexpr uint32_t TX_MSG = BUF_BYTES / 2 + SLOTS * 4u;      // the peer's half of the messages + gauge slots
    constexpr uint32_t TX_PART = SLOTS * 12u;                    // posterior sums (rank 0 only)
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();
    const uint32_t cid = cluster_id_x(), ncl = cluster_count_x();
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float invT = p.invT;
    const float2 nl2 = splat2(-p.lam2);
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;

    float *msg = smem + C::OFF_MSG;
    float4 *stage4 = reinterpret_cast<float4 *>(smem + C::OFF_RING);      // [RD][NCH][CT], thread-private entries
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAG);
    Proto pr{1u, abort_flag, p.diag};
    const uint32_t mbar_full = smem_u32(smem + C::OFF_MBAR);     // [2], one per message parity
    const uint32_t msg_u32 = smem_u32(msg), stage_u32 = smem_u32(stage4) + (uint32_t)tid * 16u;
    const uint32_t wmax_u32 = smem_u32(wmax), part_u32 = smem_u32(part), lz_u32 = smem_u32(lz);

    // history of this cluster: float4 [n][CL][BPT][NCH][CT]; this thread's entries
    float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)cid * n * 2 * C::Q) + tid;

    uint32_t full_of[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) full_of[r] = mapa_u32(mbar_full, (uint32_t)r);

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) mbar_init(mbar_full + 8u * s, C::ARRIVALS);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    uint32_t full_phase = 0;       // bit b = parity to wait for on full[b]
    auto wait_inputs = [&](int b) {
        pr.wait(mbar_full + 8u * b, (full_phase >> b) & 1u);
        full_phase ^= 1u << b;
    };

    const uint32_t tm_cb = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    const uint32_t tm_acc = tm_cb + 64u;
    uint32_t push_a[BPT], push_a_mbar[BPT], push_b[BPT][K];
    uint32_t own_a = 0;                                          // bit i: the alpha outputs of butterfly slot i stay in this CTA
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int x = (int)rank * NBC + i * CT + tid;
        {
            // L([x|l]) -> butterfly x2 = (x*K) mod NB, input j2 = (x*K) / NB, at [(i2*K + j2)*CT + tid2 .. +K)
            const int q2 = x * K, j2 = q2 / NB, x2 = q2 % NB;
            const int r2 = x2 / NBC, xl2 = x2 % NBC;
            const uint32_t a2 = msg_u32 + (uint32_t)(((xl2 / CT) * K + j2) * CT + xl2 % CT) * 4u;
            push_a[i] = r2 == (int)rank ? a2 : mapa_u32(a2, (uint32_t)r2);     // own CTA: plain address, plain stores
            push_a_mbar[i] = full_of[r2];
            own_a |= (r2 == (int)rank ? 1u : 0u) << i;
        }
#pragma unroll
        for (int j = 0; j < K; ++j) {
            // (M, Bt)([j|x]) -> butterfly x1 = (j*NB + x) / K, input b1 = x mod K, CTA j*CL/K.  The pair travels
            // as one 8-byte store; inputs 2e, 2e+1 of a butterfly share a 16-byte entry of plane e:
            // float4 [K/2][NBC] = (M_2e, Bt_2e, M_2e+1, Bt_2e+1)
            const int q1 = j * NB + x, x1 = q1 / K, b1 = q1 % K;
            const int r1 = x1 / NBC, xl1 = x1 % NBC;
            const uint32_t a1 = msg_u32 + (uint32_t)(((b1 >> 1) * NBC + xl1) * 4 + (b1 & 1) * 2) * 4u;
            push_b[i][j] = r1 == (int)rank ? a1 : mapa_u32(a1, (uint32_t)r1);  // r1 = j*CL/K for every x
        }
    }
    uint32_t wmax_dst[CL], lz_dst[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        wmax_dst[r] = mapa_u32(wmax_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
        lz_dst[r] = mapa_u32(lz_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
    }
    const uint32_t part_dst = mapa_u32(part_u32 + (uint32_t)((int)rank * NWARP + warp) * 16u, 0u);
    // zero the accumulators (laid out like the beta-paired codebook, 64 columns further)
    {
        float2 z[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = make_float2(0.f, 0.f);
#pragma unroll
        for (int g = 0; g < NU; ++g) tmem_st16(tm_acc + 16u * g, z);
        tmem_wait_st();
    }
    // test hook for the waits' abort path: one warp of CTA 0 withholds an arrival of its first block
    const bool drop_hook = blockIdx.x == 0 && warp == 1 && p.diag->drop_history_load != 0;
    float defect = 0.f;

    for (int64_t blk = cid; blk < p.B; blk += ncl) {
        int ib = 0;
        // per-step scalars of this block (read through the read-only cache, one line per warp)
        const float *w_s = p.W + blk * n, *g_s = p.g + blk * n, *sf_s = p.soft + blk * n;
        int O = 0, Ofin = 0;
        float off = 0.f, cmax = 0.f, lsefin = 0.f;
        if constexpr (BETA_ONLY) {
            hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)blk * n * 2 * C::Q) + tid;
            const int *aux = p.stepO + (size_t)blk * (C::MAX_N + 4);
            for (int t = 1 + tid; t <= n + 1; t += CT) O_s[t] = aux[t];
            __syncthreads();
            Ofin = O_s[n + 1];
            lsefin = __int_as_float(aux[n + 2]);
        } else {
            // L_1 = 0; the At array carries At + gsh (gsh_t = -g_t soft_t centres h_t = g_t c - g_t soft_t)
            {
                const float gsh1 = -__ldg(g_s) * __ldg(sf_s);
                for (int q = tid; q < QC; q += CT) { msg[q] = 0.f; msg[QC + q] = gsh1; }
            }
            if (tid == 0) O_s[1] = 0;
#pragma unroll
            for (int i = 0; i < BPT; ++i)                             // codebook -> TMEM, alpha pairing
                stage_codebook<C>(p.cb, (int)rank * NBC + i * CT + tid, tm_cb + (uint32_t)(KK * i), false);
            tmem_wait_st();
            cluster_sync();                                          // block start
            // ================= alpha sweep carrying (L, At)
            for (int t = 1; t <= n; ++t) {
                const int ob = ib ^ 1;
                // what does not depend on the step's inputs is requested before the wait for them: the first
                // codebook unit from tensor memory and the step's scalars (their latency hides under the wait)
                float2 cb[2][8];
                tmem_ld16(tm_cb, cb[0]);
                const float gt = __ldg(g_s + t - 1), wt = __ldg(w_s + t - 1);
                const float gshn = t < n ? -__ldg(g_s + t) * __ldg(sf_s + t) : 0.f;
                if (t > 1) {
                    wait_inputs(ib);
                    cmax = warp_max(lane < SLOTS ? wmax[ib * 32 + lane] : NEG_INF) - off;
                    off = rintf(cmax);
                }
                if (!pr.warp_live()) { tmem_wait_ld(cb[0]); break; } // a wait ran out: this warp issues nothing more
                const float *Lin = msg + ib * 2 * QC, *Ain = Lin + QC;
                const uint32_t ob_off = (uint32_t)ob * BUF_BYTES, ob_mbar = 8u * ob;
                if (tid == 0) mbar_expect_tx(mbar_full + ob_mbar, TX_MSG);
                float4 *hrow = hist4 + ((size_t)(t - 1) * CL + rank) * (BPT * NCH * CT);      // (L_t, At_t) of this thread's butterflies
                // gshn: shift for the consumers of this step's At (step t+1); unused at t = n
                const float2 gshn2 = splat2(gshn);
                const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
                const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), off2 = splat2(off);
                float tmax = NEG_INF;
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    float2 outL[K / 2], outA[K / 2];
                    float Lj[K], Aj[K];
#pragma unroll
                    for (int j = 0; j < K; ++j) {
                        Lj[j] = Lin[(i * K + j) * CT + tid];
                        Aj[j] = Ain[(i * K + j) * CT + tid];
                    }
#pragma unroll
                    for (int q = 0; q < K / 4; ++q) {
                        hrow[(i * NCH + q) * CT] = make_float4(Lj[4 * q], Lj[4 * q + 1], Lj[4 * q + 2], Lj[4 * q + 3]);
                        hrow[(i * NCH + K / 4 + q) * CT] = make_float4(Aj[4 * q], Aj[4 * q + 1], Aj[4 * q + 2], Aj[4 * q + 3]);
                    }
#pragma unroll
                    for (int u = 0; u < UNITS; ++u) {
                        const int g = i * UNITS + u;
                        tmem_wait_ld(cb[g & 1]);
                        if (g + 1 < NU) tmem_ld16(tm_cb + 16u * (g + 1), cb[(g + 1) & 1]);
#pragma unroll
                        for (int hh = 0; hh < HPU; ++hh) {
                            const int h = u * HPU + hh;
                            float2 a[K];
#pragma unroll
                            for (int j = 0; j < K; ++j) {
                                const float2 du = sub2(cb[g & 1][C::a_idx(j, hh)], w2);
                                a[j] = energy2(du, nl2, kap2, splat2(Lj[j]));
                            }
                            const float2 m = max_pairs<K>(a);
                            float2 pj = ex2f2(sub2(a[0], m));
                            float2 sum = pj, ax = mul2(pj, fma2(g2, cb[g & 1][C::a_idx(0, hh)], splat2(Aj[0])));
#pragma unroll
                            for (int j = 1; j < K; ++j) {
                                // one in eight exponentials on the FP32 pipe (none: 13.17 ms, one in four: 13.14, one in eight: 13.04 per 592 blocks); no gain at K = 8
                                pj = (KB == 2 && j % 4 == 3 && (hh & 1)) ? ex2_poly2(sub2(a[j], m)) : ex2f2(sub2(a[j], m));
                                sum = add2(sum, pj);
                                ax = fma2(pj, fma2(g2, cb[g & 1][C::a_idx(j, hh)], splat2(Aj[j])), ax);
                            }
                            outL[h] = add2(sub2(m, off2), lg2f2(sum));
                            outA[h] = fma2(ax, rcpf2(sum), gshn2);
                            tmax = max3f(tmax, m.x, m.y);
                        }
                    }
                    const uint32_t mb = push_a_mbar[i] + ob_mbar;
                    // k = 2: the outputs of slot i go to CTA i & 1 whatever the thread (x*K mod NB = (i & 1)*NBC + 4 tid);
                    // said this way the choice is uniform for the compiler too
                    const bool own = BPT >= 2 ? (i & 1) == (int)rank : (own_a >> i) & 1u;
#pragma unroll
                    for (int h = 0; h < K / 2; h += 2) {
                        push_v4(own, push_a[i] + ob_off + 8u * h, outL[h].x, outL[h].y, outL[h + 1].x, outL[h + 1].y, mb);
                        push_v4(own, push_a[i] + ob_off + QC * 4u + 8u * h, outA[h].x, outA[h].y, outA[h + 1].x, outA[h + 1].y, mb);
                    }
                }
                tmax = warp_max(tmax);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_async_f32(wmax_dst[r] + (uint32_t)(ob * 32) * 4u, tmax, full_of[r] + ob_mbar);
                }
                O += (int)off;
                if (tid == 0) O_s[t + 1] = O;
                __syncwarp();
                if (lane == 0) {                                     // this warp has read all its inputs and written its outputs
                    mbar_arrive_local(mbar_full + ob_mbar);
                    mbar_arrive_remote(full_of[rank ^ 1u] + ob_mbar);
                }
                ib = ob;
            }
            // ================= log2 Z
            wait_inputs(ib);
            cmax = warp_max(lane < SLOTS ? wmax[ib * 32 + lane] : NEG_INF) - off;
            {
                const float *Lfin = msg + ib * 2 * QC;
                float ssum = 0.f;
                for (int q = tid; q < QC; q += CT) ssum += ex2f(Lfin[q] - cmax);
                ssum = warp_sum(ssum);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r], ssum);
                }
                cluster_sync();                                      // log Z exchange
            }
            lsefin = cmax + lg2f(warp_sum(lane < SLOTS ? lz[lane] : 0.f));
            if (tid == 0) diag_check_finite(p.diag, lsefin);
            Ofin = O;
        }
        // ================= beta sweep carrying (M, Bt), with the gradient contraction
        {
            const float gshn = -__ldg(g_s + n - 1) * __ldg(sf_s + n - 1);     // M_n = 0, Bt_n = 0 (+ centring shift)
            for (int f = tid; f < 2 * QC; f += CT) msg[ib * 2 * QC + f] = (f & 1) ? gshn : 0.f;
        }
#pragma unroll
        for (int i = 0; i < BPT; ++i)                             // codebook -> TMEM, beta pairing
            stage_codebook<C>(p.cb, (int)rank * NBC + i * CT + tid, tm_cb + (uint32_t)(KK * i), true);
        tmem_wait_st();
        int P = 0;
        float offM = 0.f;
        // history stream: chunk c of this block = butterfly (t = n - c / BPT, i = c % BPT), staged one step ahead
        const uint32_t nchunks = (uint32_t)n * BPT;
        // running source pointer of the next chunk to request: butterflies i = 0..BPT-1 of step t, then step t - 1
        const float4 *nsrc = hist4 + ((size_t)(n - 1) * CL + rank) * (BPT * NCH * CT);
        uint32_t nleft = nchunks;                                // chunks not yet requested
        int ni = 0;
        auto issue_chunk = [&](uint32_t slot) {
            // branch-free: once every chunk has been requested the last one is simply requested again
            // (into a slot nobody reads any more)
            const uint32_t dst = stage_u32 + slot * (uint32_t)(NCH * CT * 16);
#pragma unroll
            for (int q = 0; q < NCH; ++q)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)(q * CT * 16)), "l"(nsrc + q * CT) : "memory");
            asm volatile("cp.async.commit_group;" ::: "memory");
            const bool more = nleft > 1;
            const bool wrap = ni == BPT - 1;
            const ptrdiff_t adv = wrap ? -(ptrdiff_t)((size_t)(CL * BPT + BPT - 1) * (NCH * CT)) : (ptrdiff_t)(NCH * CT);
            nsrc += more ? adv : 0;
            ni = wrap ? 0 : ni + 1;
            nleft -= more ? 1u : 0u;
        };
#pragma unroll
        for (uint32_t c = 0; c < RD; ++c) issue_chunk(c);           // the first step's butterflies
        uint32_t chunk = 0;
        cluster_sync();                                          // beta start
        // rank 0, warp 0: turn the sums of step t (slots of parity b) into grad_W[t]
        auto finish_step = [&](int t, int b) {
            if (rank == 0 && warp == NWARP - 1) {                // the warps with the highest index finish a step first: slack
                const float *pp = part + (b * 32 + lane) * 4;
                float a0 = lane < SLOTS ? pp[0] : 0.f, a2 = lane < SLOTS ? pp[1] : 0.f, az = lane < SLOTS ? pp[2] : 0.f;
                a0 = warp_sum(a0); a2 = warp_sum(a2); az = warp_sum(az);
                if (lane == 0) {
                    const float i0 = 1.f / a0;
                    p.gW[blk * n + t - 1] = (__ldg(g_s + t - 1) - az * i0) + (a2 * i0) * (__ldg(w_s + t - 1) - __ldg(sf_s + t - 1)) * invT;
                    defect = fmaxf(defect, fabsf(a0 - 1.f));
                }
            }
        };
        for (int t = n; t >= 1; --t) {
            const int ob = ib ^ 1;
            // requested before the wait for the step's inputs, like in the alpha sweep
            float2 cb[2][8];
            tmem_ld16(tm_cb, cb[0]);
            const float wt = __ldg(w_s + t - 1), gt = __ldg(g_s + t - 1);
            const float gsh = -gt * __ldg(sf_s + t - 1);                      // shift carried by the stored At
            const float gshp = t > 1 ? -__ldg(g_s + t - 2) * __ldg(sf_s + t - 2) : 0.f;   // for step t-1
            const int Ot = O_s[t];
            asm volatile("cp.async.wait_group 0;" ::: "memory");    // this step's history, requested during the previous step
            float Lh0[K], Ah0[K];                                   // the first butterfly's, read before the wait as well
#pragma unroll
            for (int q = 0; q < K / 4; ++q) {
                const float4 l4 = stage4[q * CT + tid], a4 = stage4[(K / 4 + q) * CT + tid];
                Lh0[4 * q] = l4.x; Lh0[4 * q + 1] = l4.y; Lh0[4 * q + 2] = l4.z; Lh0[4 * q + 3] = l4.w;
                Ah0[4 * q] = a4.x; Ah0[4 * q + 1] = a4.y; Ah0[4 * q + 2] = a4.z; Ah0[4 * q + 3] = a4.w;
            }
            issue_chunk(0);
            if (t < n) {
                wait_inputs(ib);
                cmax = warp_max(lane < SLOTS ? wmax[ib * 32 + lane] : NEG_INF);
                P += (int)offM;
                offM = rintf(cmax);
                finish_step(t + 1, ib);
            }
            if (!pr.warp_live()) { tmem_wait_ld(cb[0]); break; } // a wait ran out: this warp issues nothing more
            const float4 *MBin = reinterpret_cast<const float4 *>(msg + ib * 2 * QC);
            const uint32_t ob_off = (uint32_t)ob * BUF_BYTES, ob_mbar = 8u * ob;
            if (tid == 0) mbar_expect_tx(mbar_full + ob_mbar, rank == 0 ? TX_MSG + TX_PART : TX_MSG);
            const float2 gsh2 = splat2(gsh), gshp2 = splat2(gshp);
            const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
            const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), ngi2 = splat2(-invT), gid2 = splat2(invT * se.delta), offM2 = splat2(offM);
            const float2 Dm2 = splat2((float)(Ofin - Ot - P) + lsefin);
            float2 S0 = make_float2(0.f, 0.f), S2 = S0, ZS = S0;
            float tmax = NEG_INF;
#pragma unroll
            for (int i = 0; i < BPT; ++i, ++chunk) {
                float Lh[K], Ah[K];
                if (i == 0) {
#pragma unroll
                    for (int j = 0; j < K; ++j) { Lh[j] = Lh0[j]; Ah[j] = Ah0[j]; }
                } else {
#pragma unroll
                    for (int q = 0; q < K / 4; ++q) {
                        const float4 l4 = stage4[(i * NCH + q) * CT + tid], a4 = stage4[(i * NCH + K / 4 + q) * CT + tid];
                        Lh[4 * q] = l4.x; Lh[4 * q + 1] = l4.y; Lh[4 * q + 2] = l4.z; Lh[4 * q + 3] = l4.w;
                        Ah[4 * q] = a4.x; Ah[4 * q + 1] = a4.y; Ah[4 * q + 2] = a4.z; Ah[4 * q + 3] = a4.w;
                    }
                    issue_chunk(i);                                  // this slot's entry for the next step (a whole step ahead)
                }
                float Mb[K], Yb[K];
#pragma unroll
                for (int e = 0; e < K / 2; ++e) {
                    const float4 v = MBin[e * NBC + i * CT + tid];
                    Mb[2 * e] = v.x; Yb[2 * e] = v.y; Mb[2 * e + 1] = v.z; Yb[2 * e + 1] = v.w;
                }
#pragma unroll
                for (int u = 0; u < UNITS; ++u) {
                    const int g = i * UNITS + u;
                    float2 acc[8];
                    tmem_wait_ld(cb[g & 1]);
                    tmem_ld16(tm_acc + 16u * g, acc);
                    if (g + 1 < NU) tmem_ld16(tm_cb + 16u * (g + 1), cb[(g + 1) & 1]);
                    bool acc_ready = false;
#pragma unroll
                    for (int hh = 0; hh < HPU; ++hh) {
                        const int jh = u * HPU + hh;
                        float2 uu[K], d[K];
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            d[b] = sub2(cb[g & 1][C::b_idx(hh, b)], w2);            // du = c - wc
                            uu[b] = energy2(d[b], nl2, kap2, splat2(Mb[b]));
                        }
                        const float2 m = max_pairs<K>(uu);
                        const float2 Ahj = sub2(make_float2(Ah[2 * jh], Ah[2 * jh + 1]), gsh2);
                        const float2 Lhj = make_float2(Lh[2 * jh], Lh[2 * jh + 1]);
                        const float2 f = ex2f2(add2(sub2(m, Dm2), Lhj));
                        // f (w - c) / T = f delta / T - (f / T) du
                        const float2 fg = mul2(f, g2), nfi = mul2(f, ngi2), fid = mul2(f, gid2);
                        if (!acc_ready) { tmem_wait_ld(acc); acc_ready = true; }
                        float2 sum = make_float2(0.f, 0.f), ya = sum, zs = sum;
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            const float2 pb = ex2f2(sub2(uu[b], m));
                            const float2 y = fma2(g2, cb[g & 1][C::b_idx(hh, b)], splat2(Yb[b]));   // h + Bt
                            const float2 z = fma2(fma2(nfi, d[b], fid), add2(y, Ahj), fg);            // f (g + (w - c) r / T)
                            sum = add2(sum, pb);
                            ya = fma2(pb, y, ya);
                            zs = fma2(pb, z, zs);
                            acc[C::b_idx(hh, b)] = fma2(pb, z, acc[C::b_idx(hh, b)]);
                        }
                        const float2 outM = add2(sub2(m, offM2), lg2f2(sum));
                        const float2 outB = fma2(ya, rcpf2(sum), gshp2);
                        tmax = max3f(tmax, m.x, m.y);
                        const uint32_t mb0 = full_of[(2 * jh) * CL / K] + ob_mbar, mb1 = full_of[(2 * jh + 1) * CL / K] + ob_mbar;
                        const bool own = (2 * jh) * CL / K == (int)rank;         // both outputs of the pair go to the same CTA
                        push_v2(own, push_b[i][2 * jh] + ob_off, outM.x, outB.x, mb0);
                        push_v2(own, push_b[i][2 * jh + 1] + ob_off, outM.y, outB.y, mb1);
                        S0 = fma2(f, sum, S0);
                        S2 = fma2(f, fma2(Ahj, sum, ya), S2);
                        ZS = add2(ZS, zs);
                    }
                    tmem_st16(tm_acc + 16u * g, acc);
                }
            }
            tmem_wait_st();
            tmax = warp_max(tmax) - offM;
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < CL; ++r) st_async_f32(wmax_dst[r] + (uint32_t)(ob * 32) * 4u, tmax, full_of[r] + ob_mbar);
            }
            __syncwarp();
            if (lane == 0 && !(drop_hook && t == n && blk == cid)) {   // this warp has read all its inputs and written its outputs
                mbar_arrive_local(mbar_full + ob_mbar);
                mbar_arrive_remote(full_of[rank ^ 1u] + ob_mbar);
            }
            // the posterior sums follow the arrival: the phase cannot complete before their bytes have landed
            // (they are part of rank 0's expected count), and nobody waits for this warp's shuffles
            const float s3 = warp_sum3_split(S0.x + S0.y, S2.x + S2.y, ZS.x + ZS.y, lane);
            if ((lane & 7) == 0 && lane < 24)
                st_async_f32(part_dst + (uint32_t)(ob * 128 + (lane >> 3)) * 4u, s3, full_of[0] + ob_mbar);
            ib = ob;
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        wait_inputs(ib);                                         // the sums of step 1
        finish_step(1, ib);
        cluster_sync();                                          // block end
    }
    // this cluster's partial of grad_codebook: beta pair (jh, b) of butterfly x holds states [2jh | x | b], [2jh+1 | x | b]
    float *gc = p.gc_part + (size_t)cid * C::S;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int x = (int)rank * NBC + i * CT + tid;
#pragma unroll
        for (int u = 0; u < UNITS; ++u) {
            float2 acc[8];
            tmem_ld16(tm_acc + 16u * (i * UNITS + u), acc);
            tmem_wait_ld(acc);
#pragma unroll
            for (int hh = 0; hh < HPU; ++hh) {
                const int jh = u * HPU + hh;
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    float *g0 = gc + (size_t)(2 * jh) * C::Q + (size_t)x * K + b, *g1 = gc + (size_t)(2 * jh + 1) * C::Q + (size_t)x * K + b;
                    *g0 = BETA_ONLY ? *g0 + acc[C::b_idx(hh, b)].x : acc[C::b_idx(hh, b)].x;
                    *g1 = BETA_ONLY ? *g1 + acc[C::b_idx(hh, b)].y : acc[C::b_idx(hh, b)].y;
                }
            }
        }
    }
    if (tid == CT - 32 && rank == 0) diag_max(&p.diag->max_defect, defect);
    asm volatile("cp.async.wait_all;" ::: "memory");           // no copy may be in flight at exit (a warp may have left the loop early)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync();             // no CTA leaves while a peer may still address its shared memory
    if (*abort_flag) settle_after_abort();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
