// Backward call for the 2^16-state, k = 2 trellis: the two-CTA tensor-memory kernel of bcjr_duo.cuh with
// the butterflies of a thread ordered so that a step never has to wait for the whole cluster.
//
// What bcjr_duo.cuh does at every step boundary is a barrier in disguise: a warp may start step t+1 only
// when all 32 warps of the cluster have finished step t, so each warp idles from the moment it is done
// until the slowest one is (several hundred clocks per step, 8-9 % of the kernel).  The dependences of
// the trellis do not ask for that.  One output of butterfly x is one input of one butterfly of the next
// step, and which butterflies feed which is fixed by the bitshift structure:
//     alpha:  L'([x|l]) is input j = x >> 10 of butterfly ((x & 1023) << 2) | l
//     beta :  M'([j|x]) is input b = x & 3   of butterfly (j << 10) | (x >> 2)
// so the assignment of butterflies to (thread, slot) and the order in which a thread walks its four
// slots decide how early a step's first butterfly can start.  Here, with x = [b1 b0 | a1 a0 | r] (r the low
// eight bits), CTA = b1 and
//     slot 0: a1 =  b1, b0 = 0          slot 2: a1 = !b1, a0 = 0
//     slot 1: a1 =  b1, b0 = 1          slot 3: a1 = !b1, a0 = 1          (the free bit and r make up the thread)
// the alpha sweep walks the slots 0,1,2,3 and the beta sweep 2,0,3,1, and then
//   * the butterfly a thread computes FIRST in a step needs nothing from the butterflies the threads
//     computed LAST in the step before (alpha: slot 0 reads slots 0,1 of its own CTA and slot 2 of the peer;
//     beta: slot 2 reads slots 0,2,3 of the peer);
//   * in the alpha sweep slots 0,1 send all their outputs to the own CTA (plain shared stores) and slots
//     2,3 all theirs to the peer (st.async); in the beta sweep every butterfly sends half and half.
// Each message buffer therefore has two mbarriers: "early" completes when what the first butterfly needs
// has arrived, "late" when everything has and every warp of the cluster is done with the step.  A warp
// waits for "early" at the top of a step, computes its first butterfly, waits for "late" (which by then
// has had a whole butterfly's time to complete), and only then writes outputs -- the first write of step
// t+1 goes into the buffer step t read, so "late" is also what makes that overwrite safe.  The gauge offset
// (rounded maximum of the previous step's outputs) enters only when outputs are formed, so it too is taken
// after the "late" wait and stays exact.
//
// Everything else -- tensor-memory tables and accumulators, thread-private history, bounded waits, the
// arithmetic itself -- is that of bcjr_duo.cuh.  ACC = false leaves out the gradient accumulators (a call
// that does not ask for grad_codebook).  BETA_ONLY = true runs the beta sweeps alone, on the history, gauge
// offsets and log Z that bwd_alpha_kernel (bcjr_alpha.cuh) wrote for the same blocks; block b of the call then
// has its history at p.hist + b n 2Q and its offsets at p.stepO + b (MAX_N + 4), and the partial codebook
// gradient is ADDED to p.gc_part (several launches share it).
#pragma once
#include <type_traits>

#include "bcjr_duo.cuh"

namespace bcjr {

struct SkewCfg {
    static constexpr int LB = 16, KB = 2, K = 4, S = 1 << LB, Q = S >> KB, NB = S >> (2 * KB);
    static constexpr int CL = 2, NBC = NB / CL, QC = Q / CL;
    static constexpr int THREADS = 512, NWARP = THREADS / 32, BPT = NBC / THREADS;   // 4 butterflies per thread
    static constexpr int UNITS = 1, HPU = 2;
    static constexpr int SLOTS = CL * NWARP;
    static constexpr int NCH = 2 * K / 4;                      // 16-byte chunks per butterfly and thread: K values of L, K of At
    static constexpr int MAX_N = 1024;
    static constexpr int BUF = 2 * QC + 16;                    // floats of one message buffer: (L, At), or the two planes of (M, Bt) pairs + padding
    static constexpr int PLANE = NBC + 4;                      // float4 between the planes: a half-warp's 8-byte stores then reach all 32 banks
    static constexpr int OFF_MSG = 0;                          // [2 parity][BUF]
    static constexpr int OFF_RING = OFF_MSG + 2 * BUF;         // float4 [BPT][NCH][THREADS]
    static constexpr int OFF_O = OFF_RING + BPT * NCH * THREADS * 4;   // int [MAX_N + 2]
    static constexpr int OFF_WMAX = OFF_O + MAX_N + 2 + 2;     // [2][32]
    static constexpr int OFF_PART = OFF_WMAX + 64;             // [2][32][4]
    static constexpr int OFF_LZ = OFF_PART + 256;              // [32]
    static constexpr int OFF_MBAR = OFF_LZ + 32;               // uint64: early[2], late[2]
    static constexpr int OFF_TMEM = OFF_MBAR + 8;
    static constexpr int OFF_FLAG = OFF_TMEM + 2;
    static constexpr int OFF_PUSH = OFF_FLAG + 2;              // uint32 [2 BPT][THREADS]: beta push addresses of every thread and slot
    static constexpr int SMEM_FLOATS = OFF_PUSH + 2 * BPT * THREADS;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(OFF_MBAR % 2 == 0, "mbarrier alignment");
    static_assert(BPT == 4 && K == 4, "slot scheme is written for four butterflies of sixteen states per thread");
    __host__ __device__ static constexpr int a_idx(int j, int h) { return 2 * j + h; }
    __host__ __device__ static constexpr int b_idx(int jh, int b) { return 4 * jh + b; }
    // butterfly of (CTA, thread, slot) and back
    __host__ __device__ static constexpr int x_of(int rank, int tid, int slot)
    {
        return slot < 2 ? (rank << 11) | (slot << 10) | (rank << 9) | ((tid >> 8) << 8) | (tid & 255)
                        : (rank << 11) | ((tid >> 8) << 10) | ((rank ^ 1) << 9) | ((slot & 1) << 8) | (tid & 255);
    }
    __host__ __device__ static constexpr int rank_of(int x) { return (x >> 11) & 1; }
    __host__ __device__ static constexpr int slot_of(int x)
    {
        return ((x >> 9) & 1) == ((x >> 11) & 1) ? (x >> 10) & 1 : 2 + ((x >> 8) & 1);
    }
    __host__ __device__ static constexpr int tid_of(int x)
    {
        return ((x >> 9) & 1) == ((x >> 11) & 1) ? (((x >> 8) & 1) << 8) | (x & 255) : (((x >> 10) & 1) << 8) | (x & 255);
    }
};

template <bool ACC, bool BETA_ONLY>
__global__ void __launch_bounds__(SkewCfg::THREADS, 1) bwd_skew_kernel(BwdParams p)
{
    using C = SkewCfg;
    constexpr int K = C::K, NBC = C::NBC, QC = C::QC, BPT = C::BPT, NWARP = C::NWARP, CT = C::THREADS;
    constexpr int CL = C::CL, SLOTS = C::SLOTS, NCH = C::NCH;
    constexpr uint32_t BUF_BYTES = (uint32_t)C::BUF * 4u;        // one parity
    constexpr int PLANE = C::PLANE;
    // bytes the peer sends into a buffer of this CTA per step: alpha, one slot = 512 threads x (16 + 16) bytes;
    // beta, one slot = 512 threads x 2 outputs x 8 bytes; the gauge slots (32 x 4) and, on CTA 0, the posterior
    // sums (32 x 12) travel with the "late" part
    constexpr uint32_t TX_A_EARLY = CT * 32u, TX_A_LATE = CT * 32u + SLOTS * 4u;
    constexpr uint32_t TX_B_EARLY = 3u * CT * 16u, TX_B_LATE = CT * 16u + SLOTS * 4u, TX_PART = SLOTS * 12u;
    constexpr int ORD_B0 = 2, ORD_B1 = 0, ORD_B2 = 3, ORD_B3 = 1;   // beta sweep: slot walked at position 0..3
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
    float4 *stage4 = reinterpret_cast<float4 *>(smem + C::OFF_RING);      // [BPT][NCH][CT], thread-private entries
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAG);
    Proto pr{1u, abort_flag, p.diag};
    const uint32_t mb_early = smem_u32(smem + C::OFF_MBAR), mb_late = mb_early + 16u;   // [2] each, one per parity
    const uint32_t msg_u32 = smem_u32(msg), stage_u32 = smem_u32(stage4) + (uint32_t)tid * 16u;
    const uint32_t wmax_u32 = smem_u32(wmax), part_u32 = smem_u32(part), lz_u32 = smem_u32(lz);

    // history of this cluster (BETA_ONLY: of the block at hand): float4 [n][CL][BPT][NCH][CT]; this thread's entries
    float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)cid * n * 2 * C::Q) + tid;
    constexpr ptrdiff_t HSTEP = (ptrdiff_t)CL * BPT * NCH * CT;     // float4 per step

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(mb_early + 8u * s, 1 + NWARP); mbar_init(mb_late + 8u * s, 1 + SLOTS); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    uint32_t phase = 0;            // bit b: parity to wait for on early[b]; bit 2 + b: on late[b]
    auto wait_early = [&](int b) { pr.wait(mb_early + 8u * b, (phase >> b) & 1u); phase ^= 1u << b; };
    auto wait_late = [&](int b) { pr.wait(mb_late + 8u * b, (phase >> (2 + b)) & 1u); phase ^= 4u << b; };

    const uint32_t tm_cb = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    const uint32_t tm_acc = tm_cb + 64u;
    const uint32_t peer = rank ^ 1u;
    const uint32_t peer_early = mapa_u32(mb_early, peer), peer_late = mapa_u32(mb_late, peer);
    uint32_t late_of[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) late_of[r] = mapa_u32(mb_late, (uint32_t)r);
    // where the outputs go
    uint32_t push_a[BPT];          // alpha: slots 0,1 own CTA (plain address), slots 2,3 the peer (cluster address)
    uint32_t push_bl[BPT], push_br[BPT];   // beta: outputs j = (rank, 0) [+8 KB for (rank, 1)] and j = (!rank, 0) [+4 KB for (!rank, 1)]
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int x = C::x_of((int)rank, tid, i);
        {
            const int x2 = (x & 1023) << 2, j2 = x >> 10;
            const uint32_t a2 = msg_u32 + (uint32_t)((C::slot_of(x2) * K + j2) * CT + C::tid_of(x2)) * 4u;
            push_a[i] = i < 2 ? a2 : mapa_u32(a2, peer);
        }
        {
            const int bin = x & 3;
            const int xl = ((int)rank << 11) | (x >> 2), xr = ((int)peer << 11) | (x >> 2);     // consumer butterflies of outputs j = (CTA, 0)
            const uint32_t al = msg_u32 + (uint32_t)(((bin >> 1) * PLANE + C::slot_of(xl) * CT + C::tid_of(xl)) * 4 + (bin & 1) * 2) * 4u;
            const uint32_t ar = msg_u32 + (uint32_t)(((bin >> 1) * PLANE + C::slot_of(xr) * CT + C::tid_of(xr)) * 4 + (bin & 1) * 2) * 4u;
            push_bl[i] = al;
            push_br[i] = mapa_u32(ar, peer);
            if (BETA_ONLY) {
                reinterpret_cast<uint32_t *>(smem + C::OFF_PUSH)[(2 * i) * CT + tid] = push_bl[i];
                reinterpret_cast<uint32_t *>(smem + C::OFF_PUSH)[(2 * i + 1) * CT + tid] = push_br[i];
            }
        }
    }
    const uint32_t *pushtab = reinterpret_cast<const uint32_t *>(smem + C::OFF_PUSH) + tid;
    constexpr uint32_t BL_STEP = CT * 16u, BR_STEP = 256u * 16u;     // j0 = 1: next slot (own CTA) / upper half of the threads (peer)
    uint32_t wmax_dst[CL], lz_dst[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        wmax_dst[r] = mapa_u32(wmax_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
        lz_dst[r] = mapa_u32(lz_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
    }
    const uint32_t part_dst = mapa_u32(part_u32 + (uint32_t)((int)rank * NWARP + warp) * 16u, 0u);
    if (ACC) {                                                   // zero the accumulators (laid out like the beta-paired codebook)
        float2 z[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = make_float2(0.f, 0.f);
#pragma unroll
        for (int g = 0; g < BPT; ++g) tmem_st16(tm_acc + 16u * g, z);
        tmem_wait_st();
    }
    // test hook for the waits' abort path: one warp of CTA 0 withholds an arrival of its first block
    const bool drop_hook = blockIdx.x == 0 && warp == 1 && p.diag->drop_history_load != 0;
    float defect = 0.f;

    for (int64_t blk = cid; blk < p.B; blk += ncl) {
        int ib = 0;
        const float *w_s = p.W + blk * n, *g_s = p.g + blk * n, *sf_s = p.soft + blk * n;
        if (BETA_ONLY) {
            // the alpha sweep of this block was run by bwd_alpha_kernel: its history, gauge offsets and log Z tail
            hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)blk * n * 2 * C::Q) + tid;
            const int *aux = p.stepO + (size_t)blk * (C::MAX_N + 4);
            for (int t = 1 + tid; t <= n + 1; t += CT) O_s[t] = aux[t];
        } else {
            // L_1 = 0; the At array carries At + gsh (gsh_t = -g_t soft_t centres h_t = g_t c - g_t soft_t)
            const float gsh1 = -__ldg(g_s) * __ldg(sf_s);
            for (int q = tid; q < QC; q += CT) { msg[q] = 0.f; msg[QC + q] = gsh1; }
            if (tid == 0) O_s[1] = 0;
        }
        // a block whose weights all lie inside the table's range (nearly every block of Gaussian weights) takes the
        // sweeps with the plain square; any other block the form of step_energy (both CTAs decide alike)
        int outside = 0;
        for (int t = tid; t < n; t += CT) {
            const float wv = __ldg(w_s + t);
            outside |= !(wv >= c_lo && wv <= c_hi);
        }
        const bool recentre = __syncthreads_or(outside) != 0;
        int O = 0, Ofin = 0;
        float off = 0.f, cmax = 0.f, lsefin = 0.f;
        bool dead = false;
        if constexpr (!BETA_ONLY) {
#pragma unroll
            for (int i = 0; i < BPT; ++i)                             // codebook -> TMEM, alpha pairing
                stage_codebook<C>(p.cb, C::x_of((int)rank, tid, i), tm_cb + (uint32_t)(16 * i), false);
            tmem_wait_st();
            cluster_sync();                                          // block start
            // ================= alpha sweep carrying (L, At)
            auto alpha_sweep = [&](auto rc_tag) {
            constexpr bool RC = decltype(rc_tag)::value;
            for (int t = 1; t <= n; ++t) {
                const int ob = ib ^ 1;
                float2 cb[2][8];
                tmem_ld16(tm_cb, cb[0]);
                const float gt = __ldg(g_s + t - 1), wt = __ldg(w_s + t - 1);
                const float gshn = t < n ? -__ldg(g_s + t) * __ldg(sf_s + t) : 0.f;
                if (t > 1) wait_early(ib);
                if (!pr.warp_live()) { tmem_wait_ld(cb[0]); dead = true; break; }
                const float *Lin = msg + ib * C::BUF, *Ain = Lin + QC;
                const uint32_t ob_off = (uint32_t)ob * BUF_BYTES, ob_mbar = 8u * ob;
                if (tid == 0) {
                    mbar_expect_tx(mb_early + ob_mbar, TX_A_EARLY);
                    mbar_expect_tx(mb_late + ob_mbar, TX_A_LATE);
                }
                float4 *hrow = hist4 + (size_t)(t - 1) * HSTEP + (size_t)rank * (BPT * NCH * CT);   // (L_t, At_t) of this thread's butterflies
                const float2 gshn2 = splat2(gshn);
                const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
                const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt);
                float2 off2 = splat2(off);
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
                    hrow[(i * NCH) * CT] = make_float4(Lj[0], Lj[1], Lj[2], Lj[3]);
                    hrow[(i * NCH + 1) * CT] = make_float4(Aj[0], Aj[1], Aj[2], Aj[3]);
                    tmem_wait_ld(cb[i & 1]);
                    if (i + 1 < BPT) tmem_ld16(tm_cb + 16u * (i + 1), cb[(i + 1) & 1]);
#pragma unroll
                    for (int h = 0; h < K / 2; ++h) {
                        float2 a[K];
#pragma unroll
                        for (int j = 0; j < K; ++j) {
                            const float2 du = sub2(cb[i & 1][C::a_idx(j, h)], w2);
                            a[j] = RC ? energy2(du, nl2, kap2, splat2(Lj[j])) : fma2(mul2(du, du), nl2, splat2(Lj[j]));
                        }
                        const float2 m = max_pairs<K>(a);
                        float2 pj = ex2f2(sub2(a[0], m));
                        float2 sum = pj, ax = mul2(pj, fma2(g2, cb[i & 1][C::a_idx(0, h)], splat2(Aj[0])));
#pragma unroll
                        for (int j = 1; j < K; ++j) {
                            pj = (j == 3 && (h & 1)) ? ex2_poly2(sub2(a[j], m)) : ex2f2(sub2(a[j], m));   // one in eight on the FP32 pipe
                            sum = add2(sum, pj);
                            ax = fma2(pj, fma2(g2, cb[i & 1][C::a_idx(j, h)], splat2(Aj[j])), ax);
                        }
                        outL[h] = add2(m, lg2f2(sum));               // the gauge offset is subtracted below
                        outA[h] = fma2(ax, rcpf2(sum), gshn2);
                        tmax = max3f(tmax, m.x, m.y);
                    }
                    if (i == 0) {
                        // everything of the previous step has arrived and every warp of the cluster is done with it:
                        // the gauge of this step's outputs, and leave to overwrite the buffer that step read
                        if (t > 1) {
                            wait_late(ib);
                            cmax = warp_max(lane < SLOTS ? wmax[ib * 32 + lane] : NEG_INF) - off;
                            off = rintf(cmax);
                            off2 = splat2(off);
                        }
                        if (!pr.warp_live()) { dead = true; break; }
                    }
                    outL[0] = sub2(outL[0], off2); outL[1] = sub2(outL[1], off2);
                    if (i < 2) {
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(push_a[i] + ob_off), "f"(outL[0].x), "f"(outL[0].y),
                                     "f"(outL[1].x), "f"(outL[1].y) : "memory");
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(push_a[i] + ob_off + QC * 4u), "f"(outA[0].x),
                                     "f"(outA[0].y), "f"(outA[1].x), "f"(outA[1].y) : "memory");
                    } else {
                        const uint32_t mb = (i == 2 ? peer_early : peer_late) + ob_mbar;
                        st_async_v4(push_a[i] + ob_off, outL[0].x, outL[0].y, outL[1].x, outL[1].y, mb);
                        st_async_v4(push_a[i] + ob_off + QC * 4u, outA[0].x, outA[0].y, outA[1].x, outA[1].y, mb);
                    }
                    if (i == 1) {                                     // slots 0 and 1 are in this CTA's buffer: publish them
                        __syncwarp();
                        if (lane == 0) mbar_arrive_local(mb_early + ob_mbar);
                    }
                }
                if (dead) { tmem_wait_ld(cb[0]); tmem_wait_ld(cb[1]); break; }
                tmax = warp_max(tmax);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_async_f32(wmax_dst[r] + (uint32_t)(ob * 32) * 4u, tmax, late_of[r] + ob_mbar);
                }
                O += (int)off;
                if (tid == 0) O_s[t + 1] = O;
                __syncwarp();
                if (lane == 0) {                                     // this warp has read all its inputs and written its outputs
                    mbar_arrive_local(mb_late + ob_mbar);
                    mbar_arrive_remote(peer_late + ob_mbar);
                }
                ib = ob;
            }
            };
            if (recentre) alpha_sweep(std::true_type{}); else alpha_sweep(std::false_type{});
            // ================= log2 Z
            wait_early(ib);
            wait_late(ib);
            cmax = warp_max(lane < SLOTS ? wmax[ib * 32 + lane] : NEG_INF) - off;
            {
                const float *Lfin = msg + ib * C::BUF;
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
        } else {
            __syncthreads();                                     // the offsets loaded above
            Ofin = O_s[n + 1];
            lsefin = __int_as_float(p.stepO[(size_t)blk * (C::MAX_N + 4) + n + 2]);
        }
        // ================= beta sweep carrying (M, Bt), with the gradient contraction
        {
            const float gshn = -__ldg(g_s + n - 1) * __ldg(sf_s + n - 1);     // M_n = 0, Bt_n = 0 (+ centring shift)
            for (int f = tid; f < C::BUF; f += CT) msg[ib * C::BUF + f] = (f & 1) ? gshn : 0.f;
        }
#pragma unroll
        for (int i = 0; i < BPT; ++i)                             // codebook -> TMEM, beta pairing
            stage_codebook<C>(p.cb, C::x_of((int)rank, tid, i), tm_cb + (uint32_t)(16 * i), true);
        tmem_wait_st();
        int P = 0;
        float offM = 0.f;
        // history stream: the four butterflies of step t are requested during step t + 1, each into its own staging slot
        const float4 *hsrc = hist4 + (size_t)(n - 1) * HSTEP + (size_t)rank * (BPT * NCH * CT);    // step being requested next
        auto issue_chunk = [&](int slot) {
            const uint32_t dst = stage_u32 + (uint32_t)slot * (uint32_t)(NCH * CT * 16);
#pragma unroll
            for (int q = 0; q < NCH; ++q)
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)(q * CT * 16)), "l"(hsrc + (slot * NCH + q) * CT) : "memory");
        };
#pragma unroll
        for (int i = 0; i < BPT; ++i) issue_chunk(i);           // the first step's butterflies
        asm volatile("cp.async.commit_group;" ::: "memory");
        cluster_sync();                                          // beta start
        // rank 0, last warp: turn the sums of step t (slots of parity b) into grad_W[t]
        auto finish_step = [&](int t, int b) {
            if (rank == 0 && warp == NWARP - 1) {
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
        auto beta_sweep = [&](auto rc_tag) {
        constexpr bool RC = decltype(rc_tag)::value;
        for (int t = n; t >= 1 && !dead; --t) {
            const int ob = ib ^ 1;
            // one set of table registers: the next butterfly's entries are requested when this one's arithmetic is done
            // (a second set, loaded a butterfly ahead, costs sixteen registers the scheduler makes better use of: 11.74 -> 11.63 ms)
            float2 cb[8];
            tmem_ld16(tm_cb + 16u * ORD_B0, cb);
            const float wt = __ldg(w_s + t - 1), gt = __ldg(g_s + t - 1);
            const float gsh = -gt * __ldg(sf_s + t - 1);                      // shift carried by the stored At
            const float gshp = t > 1 ? -__ldg(g_s + t - 2) * __ldg(sf_s + t - 2) : 0.f;   // for step t-1
            const int Ot = O_s[t];
            asm volatile("cp.async.wait_group 0;" ::: "memory");    // this step's history, requested during the previous step
            hsrc -= t > 1 ? HSTEP : 0;                              // next requests: step t - 1 (at t = 1: step 1 again, unread)
            if (t < n) wait_early(ib);
            if (!pr.warp_live()) { tmem_wait_ld(cb); dead = true; break; }
            P += (int)offM;                                         // offsets carried by this step's inputs M_t
            const float4 *MBin = reinterpret_cast<const float4 *>(msg + ib * C::BUF);
            const uint32_t ob_off = (uint32_t)ob * BUF_BYTES, ob_mbar = 8u * ob;
            if (tid == 0) {
                mbar_expect_tx(mb_early + ob_mbar, TX_B_EARLY);
                mbar_expect_tx(mb_late + ob_mbar, rank == 0 ? TX_B_LATE + TX_PART : TX_B_LATE);
            }
            const float2 gsh2 = splat2(gsh), gshp2 = splat2(gshp);
            const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
            const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), ngi2 = splat2(-invT), gid2 = splat2(invT * se.delta);
            float2 offM2 = splat2(offM);
            const float2 Dm2 = splat2((float)(Ofin - Ot - P) + lsefin);
            float2 S0 = make_float2(0.f, 0.f), S2 = S0, ZS = S0;
            float tmax = NEG_INF;
#pragma unroll
            for (int pos = 0; pos < BPT; ++pos) {
                const int i = pos == 0 ? ORD_B0 : pos == 1 ? ORD_B1 : pos == 2 ? ORD_B2 : ORD_B3;
                const int inext = pos == 0 ? ORD_B1 : pos == 1 ? ORD_B2 : ORD_B3;
                float Lh[K], Ah[K];
                {
                    const float4 l4 = stage4[(i * NCH) * CT + tid], a4 = stage4[(i * NCH + 1) * CT + tid];
                    Lh[0] = l4.x; Lh[1] = l4.y; Lh[2] = l4.z; Lh[3] = l4.w;
                    Ah[0] = a4.x; Ah[1] = a4.y; Ah[2] = a4.z; Ah[3] = a4.w;
                }
                issue_chunk(i);                                     // this slot's entry for the next step (a whole step ahead)
                if (pos == BPT - 1) asm volatile("cp.async.commit_group;" ::: "memory");
                float Mb[K], Yb[K];
#pragma unroll
                for (int e = 0; e < K / 2; ++e) {
                    const float4 v = MBin[e * PLANE + i * CT + tid];
                    Mb[2 * e] = v.x; Yb[2 * e] = v.y; Mb[2 * e + 1] = v.z; Yb[2 * e + 1] = v.w;
                }
                float2 acc[8];
                tmem_wait_ld(cb);
                if (ACC) tmem_ld16(tm_acc + 16u * i, acc);
                bool acc_ready = !ACC;
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
                    if (!acc_ready) { tmem_wait_ld(acc); acc_ready = true; }
                    float2 sum = make_float2(0.f, 0.f), ya = sum, zs = sum;
#pragma unroll
                    for (int b = 0; b < K; ++b) {
                        const float2 pb = ex2f2(sub2(uu[b], m));
                        const float2 y = fma2(g2, cb[C::b_idx(jh, b)], splat2(Yb[b]));   // h + Bt
                        const float2 z = RC ? fma2(fma2(nfi, d[b], fid), add2(y, Ahj), fg) : fma2(d[b], fma2(nfi, y, nfiA), fg);   // f (g + (w - c) r / T)
                        sum = add2(sum, pb);
                        ya = fma2(pb, y, ya);
                        zs = fma2(pb, z, zs);
                        if (ACC) acc[C::b_idx(jh, b)] = fma2(pb, z, acc[C::b_idx(jh, b)]);
                    }
                    outM[jh] = add2(m, lg2f2(sum));               // the gauge offset is subtracted below
                    outB[jh] = fma2(ya, rcpf2(sum), gshp2);
                    tmax = max3f(tmax, m.x, m.y);
                    S0 = fma2(f, sum, S0);
                    S2 = fma2(f, fma2(Ahj, sum, ya), S2);
                    ZS = add2(ZS, zs);
                }
                if (ACC) tmem_st16(tm_acc + 16u * i, acc);
                if (pos == 0) {
                    if (t < n) {
                        wait_late(ib);
                        cmax = warp_max(lane < SLOTS ? wmax[ib * 32 + lane] : NEG_INF);
                        offM = rintf(cmax);
                        offM2 = splat2(offM);
                        finish_step(t + 1, ib);
                    }
                    if (!pr.warp_live()) { dead = true; break; }
                }
                if (pos + 1 < BPT) tmem_ld16(tm_cb + 16u * inext, cb);
                // outputs j = 2 jh, 2 jh + 1 go to CTA jh: own CTA by plain stores, the peer by st.async
                const uint32_t mbp = (pos == BPT - 1 ? peer_late : peer_early) + ob_mbar;
#pragma unroll
                for (int jh = 0; jh < K / 2; ++jh) {
                    const float2 oM = sub2(outM[jh], offM2);
                    if (jh == (int)rank) {
                        const uint32_t pl = (BETA_ONLY ? pushtab[(2 * i) * CT] : push_bl[i]) + ob_off;
                        asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(pl), "f"(oM.x), "f"(outB[jh].x) : "memory");
                        asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(pl + BL_STEP), "f"(oM.y), "f"(outB[jh].y) : "memory");
                    } else {
                        const uint32_t prm = (BETA_ONLY ? pushtab[(2 * i + 1) * CT] : push_br[i]) + ob_off;
                        st_async_v2(prm, oM.x, outB[jh].x, mbp);
                        st_async_v2(prm + BR_STEP, oM.y, outB[jh].y, mbp);
                    }
                }
                if (pos == BPT - 2) {                             // "early" also counts the local warps (its arrival count is fixed)
                    __syncwarp();
                    if (lane == 0) mbar_arrive_local(mb_early + ob_mbar);
                }
            }
            if (dead) { tmem_wait_ld(cb); break; }
            if (ACC) tmem_wait_st();
            tmax = warp_max(tmax) - offM;
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < CL; ++r) st_async_f32(wmax_dst[r] + (uint32_t)(ob * 32) * 4u, tmax, late_of[r] + ob_mbar);
            }
            __syncwarp();
            if (lane == 0 && !(drop_hook && t == n && blk == cid)) {   // this warp has read all its inputs and written its outputs
                mbar_arrive_local(mb_late + ob_mbar);
                mbar_arrive_remote(peer_late + ob_mbar);
            }
            // the posterior sums follow the arrival: the phase cannot complete before their bytes have landed
            // (they are part of rank 0's expected count), and nobody waits for this warp's shuffles
            const float s3 = warp_sum3_split(S0.x + S0.y, S2.x + S2.y, ZS.x + ZS.y, lane);
            if ((lane & 7) == 0 && lane < 24)
                st_async_f32(part_dst + (uint32_t)(ob * 128 + (lane >> 3)) * 4u, s3, late_of[0] + ob_mbar);
            ib = ob;
        }
        };
        if (recentre) beta_sweep(std::true_type{}); else beta_sweep(std::false_type{});
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        if (!dead) {
            wait_early(ib);
            wait_late(ib);                                       // the sums of step 1
            finish_step(1, ib);
        }
        cluster_sync();                                          // block end
    }
    // this cluster's partial of grad_codebook: beta pair (jh, b) of butterfly x holds states [2jh | x | b], [2jh+1 | x | b]
    if (ACC) {
        float *gc = p.gc_part + (size_t)cid * C::S;
        tmem_wait_st();
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            const int x = C::x_of((int)rank, tid, i);
            float2 acc[8];
            tmem_ld16(tm_acc + 16u * i, acc);
            tmem_wait_ld(acc);
#pragma unroll
            for (int jh = 0; jh < K / 2; ++jh)
#pragma unroll
                for (int b = 0; b < K; ++b) {
                    float *g0 = gc + (size_t)(2 * jh) * C::Q + (size_t)x * K + b, *g1 = gc + (size_t)(2 * jh + 1) * C::Q + (size_t)x * K + b;
                    *g0 = BETA_ONLY ? *g0 + acc[C::b_idx(jh, b)].x : acc[C::b_idx(jh, b)].x;
                    *g1 = BETA_ONLY ? *g1 + acc[C::b_idx(jh, b)].y : acc[C::b_idx(jh, b)].y;
                }
        }
    }
    if (tid == CT - 32 && rank == 0) diag_max(&p.diag->max_defect, defect);
    asm volatile("cp.async.wait_all;" ::: "memory");           // no copy may be in flight at exit (a warp may have left the loop early)
    tmem_wait_st();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync();             // no CTA leaves while a peer may still address its shared memory
    if (*abort_flag) settle_after_abort();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
