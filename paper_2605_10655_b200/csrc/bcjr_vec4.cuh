// Vector-emission trellis with 16 state bits, 4 bits and V = 2 weights per step (the paper's
// "L=16, k=2, V=2"): one weight block per cluster of FOUR CTAs, table slice resident in shared
// memory.
//
// Ownership.  Q = 4096 groups, 1024 per CTA, an adjacent pair per thread; which groups a CTA owns
// is chosen per sweep so that it reads only a quarter of the messages:
//   alpha:  L_{t+1}(q) = LSE_j [ L_t((q >> 4) + 256 j) + e_t(q + jQ) ]              CTA r owns q >> 10 == r
//           and reads the entries i of L_t with ((i & 255) >> 6) == r;
//   beta :  M_{t-1}(q) = LSE_b [ M_t(((q & 255) << 4) | b) + e_t(16 q + b) ]        CTA r owns ((q & 255) >> 6) == r
//           and reads the entries i of M_t with (i >> 10) == r.
// Hence every output has exactly one consumer CTA: one st.async (the thread's pair) per thread
// and step.  The table slice of a sweep is 16 entries x 2 groups x 2 floats per thread,
// thread-private: 128 KB per CTA, staged at the start of each sweep (alpha from the table itself,
// which is [j][q][V] in memory; beta from the copy regrouped [b][q][V]) as one float4 per
// (j, thread): (c0.x, c1.x, c0.y, c1.y) for the thread's two groups, i.e. ready-made f32x2 pairs.
//
// Message buffers (three, completed through the consumer's mbarrier by byte count: the protocol of
// fwd_cluster_kernel; gauge maximum and posterior sums travel the same way).  Alpha entries keep
// their index.  The beta quarter of a CTA is stored as [b >> 1][x][b & 1] with x = (i >> 4) & 63,
// b = i & 15: a thread's two outputs are adjacent (one 8-byte push) and its reads of
// M(x, b), M(x, b+1), M(x+1, b), M(x+1, b+1) are one conflict-free 16-byte load.
//
// History.  L_t(q) is written by its alpha owner and read back by its beta owner (another CTA of
// the cluster, after the cluster barriers between the sweeps): plain coalesced global stores /
// L2 loads, 8 bytes per thread and step, prefetched one step ahead.
#pragma once
#include "bcjr_cluster.cuh"

namespace bcjr {

struct Vec4Cfg {
    static constexpr int LB = 16, KB = 4, V = 2, K = 16, S = 1 << LB, Q = S >> KB;
    static constexpr int CL = 4, THREADS = 512, NWARP = THREADS / 32, QC = Q / CL;
    static constexpr int SLOTS = CL * NWARP;                   // 64 per-warp partial slots
    static constexpr int NBUF = 3;
    static constexpr int MAX_N = 2048, MAX_NT = MAX_N / V;     // weights / steps per block
    static constexpr int OFF_TAB = 0;                          // float4 [K][THREADS]
    static constexpr int OFF_MSG = OFF_TAB + 4 * K * THREADS;  // [NBUF][Q]
    static constexpr int OFF_W = OFF_MSG + NBUF * Q;           // [MAX_N]
    static constexpr int OFF_O = OFF_W + MAX_N;                // int [MAX_NT + 2]
    static constexpr int OFF_WMAX = OFF_O + MAX_NT + 4;        // [NBUF][64]
    static constexpr int OFF_PART = OFF_WMAX + NBUF * 64;      // [NBUF][64][4]: den, num_0, num_1
    static constexpr int OFF_LZ = OFF_PART + NBUF * 64 * 4;    // [2][64]
    static constexpr int OFF_MBAR = OFF_LZ + 128;              // uint64 [NBUF]
    static constexpr int OFF_FLAG = OFF_MBAR + 2 * NBUF + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(QC == 2 * THREADS, "a thread owns two adjacent groups");
    static_assert(OFF_MBAR % 2 == 0 && OFF_TAB % 4 == 0 && OFF_MSG % 4 == 0, "alignment");
};

// table slice for one sweep: src is [16][Q][2]; entry (j, tid) = the rows of the thread's groups q0, q0 + 1
__device__ __forceinline__ void vec4_stage_table(float4 *tab, const float *src, int q0, int tid)
{
    using C = Vec4Cfg;
#pragma unroll 4
    for (int j = 0; j < C::K; ++j) {
        const float4 v = __ldg(reinterpret_cast<const float4 *>(src + ((size_t)j * C::Q + q0) * 2));
        tab[j * C::THREADS + tid] = make_float4(v.x, v.z, v.y, v.w);        // (c0.x, c1.x, c0.y, c1.y)
    }
}

__global__ void __launch_bounds__(Vec4Cfg::THREADS, 1) fwd_vec4_kernel(FwdParams p)
{
    using C = Vec4Cfg;
    constexpr int K = C::K, Q = C::Q, QC = C::QC, CL = C::CL, NWARP = C::NWARP, NBUF = C::NBUF, SLOTS = C::SLOTS, CT = C::THREADS;
    constexpr uint32_t TX_ALPHA = QC * 4u + SLOTS * 4u;          // a quarter of L + gauge slots
    constexpr uint32_t TX_BETA = QC * 4u + SLOTS * 4u;           // a quarter of M + gauge slots
    constexpr uint32_t TX_PART = SLOTS * 16u;                    // posterior sums (rank 0 only)
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();
    const uint32_t cid = cluster_id_x(), ncl = cluster_count_x();
    const int n = p.n, nt = n / C::V;
    const float NEG_INF = __int_as_float(0xff800000);
    const float2 nl2 = splat2(-p.lam2);

    float4 *tab = reinterpret_cast<float4 *>(smem + C::OFF_TAB);
    float *msg = smem + C::OFF_MSG;
    float *w_s = smem + C::OFF_W;
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAG);
    Proto pr{1u, abort_flag, p.diag};
    const uint32_t mbar_full = smem_u32(smem + C::OFF_MBAR);
    const uint32_t msg_u32 = smem_u32(msg), wmax_u32 = smem_u32(wmax), part_u32 = smem_u32(part), lz_u32 = smem_u32(lz);

    const int q0 = (int)rank * QC + 2 * tid;                     // alpha sweep: this thread's groups q0, q0 + 1
    const int q0b = warp * 256 + (int)rank * 64 + 2 * lane;      // beta sweep: groups q0b, q0b + 1
    float *hist = p.hist + (size_t)cid * nt * Q;                 // [nt][Q]: row t = L_{t+1}

    uint32_t full_of[CL], msg_of[CL], wmax_dst[CL], lz_dst[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        full_of[r] = mapa_u32(mbar_full, (uint32_t)r);
        msg_of[r] = mapa_u32(msg_u32, (uint32_t)r);
        wmax_dst[r] = mapa_u32(wmax_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
        lz_dst[r] = mapa_u32(lz_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
    }
    const uint32_t part_dst = mapa_u32(part_u32 + (uint32_t)((int)rank * NWARP + warp) * 16u, 0u);
    // alpha: the pair (q0, q0 + 1) is read by CTA (q0 & 255) >> 6, under its own index
    const int ra = (q0 & 255) >> 6;
    const uint32_t push_a = (ra == 0 ? msg_of[0] : ra == 1 ? msg_of[1] : ra == 2 ? msg_of[2] : msg_of[3]) + (uint32_t)q0 * 4u;
    const uint32_t push_a_mbar = ra == 0 ? full_of[0] : ra == 1 ? full_of[1] : ra == 2 ? full_of[2] : full_of[3];
    // beta: the pair (q0b, q0b + 1) = entries (x', b'), (x', b' + 1) with x' = q0b >> 4, b' = q0b & 15 (even)
    // is read by CTA x' >> 6 = warp >> 2 at [b' >> 1][x' & 63][b' & 1]
    const int rb = warp >> 2;
    const uint32_t push_b = (rb == 0 ? msg_of[0] : rb == 1 ? msg_of[1] : rb == 2 ? msg_of[2] : msg_of[3])
                            + (uint32_t)(((q0b & 15) >> 1) * 128 + 2 * ((q0b >> 4) & 63)) * 4u;
    const uint32_t push_b_mbar = rb == 0 ? full_of[0] : rb == 1 ? full_of[1] : rb == 2 ? full_of[2] : full_of[3];

    if (tid == 0) {
        for (int s = 0; s < NBUF; ++s) mbar_init(mbar_full + 8u * s, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t full_phase = 0;
    int ib = 0;
    float defect = 0.f, zgap = 0.f;
    auto wait_inputs = [&](int b) {
        pr.wait(mbar_full + 8u * b, (full_phase >> b) & 1u);
        full_phase ^= 1u << b;
    };

    for (int64_t blk = cid; blk < p.B; blk += ncl) {
        const float *w = p.W + blk * n;
        for (int t = tid; t < n; t += CT) w_s[t] = __ldg(w + t);
        for (int q = tid; q < Q; q += CT) msg[ib * Q + q] = 0.f;             // L_1 = 0
        if (tid == 0) O_s[1] = 0;
        vec4_stage_table(tab, p.cb, q0, tid);
        int O = 0;
        float off = 0.f, cmax = 0.f;
        cluster_sync();
        // ================= alpha sweep: step t maps L_t to L_{t+1}
        for (int t = 1; t <= nt; ++t) {
            const int ob = ib == NBUF - 1 ? 0 : ib + 1;
            if (t > 1) {
                wait_inputs(ib);
                cmax = warp_max(slot_max(wmax + ib * 64, lane, SLOTS)) - off;
                off = rintf(cmax);
            }
            const float *Lin = msg + ib * Q + (q0 >> 4);
            const uint32_t ob_off = (uint32_t)(ob * Q) * 4u, ob_mbar = 8u * ob;
            if (tid == 0) pr.expect_tx(mbar_full + ob_mbar, TX_ALPHA);
            const float2 wx = splat2(w_s[2 * (t - 1)]), wy = splat2(w_s[2 * (t - 1) + 1]);
            float2 a[K];
#pragma unroll
            for (int j = 0; j < K; ++j) {
                const float4 c = tab[j * CT + tid];
                const float2 dx = sub2(make_float2(c.x, c.y), wx), dy = sub2(make_float2(c.z, c.w), wy);
                a[j] = fma2(fma2(dy, dy, mul2(dx, dx)), nl2, splat2(Lin[256 * j]));
            }
            const float2 m = max_pairs<K>(a);
            float2 sum = ex2f2(sub2(a[0], m));
#pragma unroll
            for (int j = 1; j < K; ++j) sum = add2(sum, ex2f2(sub2(a[j], m)));
            const float2 out = add2(sub2(m, splat2(off)), lg2f2(sum));
            pr.async_v2(push_a + ob_off, out.x, out.y, push_a_mbar + ob_mbar);
            if (t < nt) *reinterpret_cast<float2 *>(hist + (size_t)t * Q + q0) = out;
            const float tmax = warp_max(fmaxf(m.x, m.y));
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(ob * 64) * 4u, tmax, full_of[r] + ob_mbar);
            }
            O += (int)off;
            if (tid == 0) O_s[t + 1] = O;
            ib = ob;
        }
        // ================= log2 Z = O_{nt+1} + LSE_q L_{nt+1}(q); this CTA holds the quarter it would read
        wait_inputs(ib);
        cmax = warp_max(slot_max(wmax + ib * 64, lane, SLOTS)) - off;
        {
            // entries addressed to this CTA: indices i with ((i & 255) >> 6) == rank
            const float *Lfin = msg + ib * Q;
            float ssum = 0.f;
            for (int e = tid; e < QC; e += CT) ssum += ex2f(Lfin[(e >> 6) * 256 + (int)rank * 64 + (e & 63)] - cmax);
            ssum = warp_sum(ssum);
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r], ssum);
            }
            cluster_sync();
        }
        float lsefin;
        {
            float v = (lane < SLOTS ? lz[lane] : 0.f) + (lane + 32 < SLOTS ? lz[lane + 32] : 0.f);
            v = warp_sum(v);
            lsefin = cmax + lg2f(v);
            if (tid == 0) diag_check_finite(p.diag, lsefin);
        }
        const int Ofin = O;
        if (tid == 0 && rank == 0 && p.logZ) p.logZ[blk] = (float)(((double)Ofin + (double)lsefin) * 0.6931471805599453);
        // ================= beta sweep: step t maps M_t to M_{t-1}
        for (int q = tid; q < QC; q += CT) msg[ib * Q + q] = 0.f;            // M_nt = 0 (this CTA's quarter)
        vec4_stage_table(tab, p.cb_beta, q0b, tid);
        int P = 0;
        float offM = 0.f;
        float2 Ls = nt > 1 ? __ldcg(reinterpret_cast<const float2 *>(hist + (size_t)(nt - 1) * Q + q0b)) : make_float2(0.f, 0.f);
        cluster_sync();
        auto finish_step = [&](int t, int b) {
            if (rank == 0 && warp == 0) {
                float4 s4 = lane < SLOTS ? *reinterpret_cast<const float4 *>(part + (b * 64 + lane) * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
                if (lane + 32 < SLOTS) {
                    const float4 o = *reinterpret_cast<const float4 *>(part + (b * 64 + lane + 32) * 4);
                    s4.x += o.x; s4.y += o.y; s4.z += o.z;
                }
                const float den = warp_sum(s4.x), n0 = warp_sum(s4.y), n1 = warp_sum(s4.z);
                if (lane == 0) {
                    const float s0 = n0 / den, s1 = n1 / den;
                    *reinterpret_cast<float2 *>(p.soft + blk * n + 2 * (t - 1)) = make_float2(s0, s1);
                    if (p.soft_copy) *reinterpret_cast<float2 *>(p.soft_copy + blk * n + 2 * (t - 1)) = make_float2(s0, s1);
                    defect = fmaxf(defect, fabsf(den - 1.f));
                }
            }
        };
        for (int t = nt; t >= 1; --t) {
            const int ob = ib == NBUF - 1 ? 0 : ib + 1;
            if (t < nt) {
                wait_inputs(ib);
                cmax = warp_max(slot_max(wmax + ib * 64, lane, SLOTS));
                P += (int)offM;
                offM = rintf(cmax);
                finish_step(t + 1, ib);
            }
            const float *Min = msg + ib * Q + 4 * lane;                          // [b >> 1][x][b & 1], x = 2 lane, 2 lane + 1
            const uint32_t ob_off = (uint32_t)(ob * Q) * 4u, ob_mbar = 8u * ob;
            if (tid == 0) pr.expect_tx(mbar_full + ob_mbar, rank == 0 ? TX_BETA + TX_PART : TX_BETA);
            // history of the next step, one step ahead (row t - 2 = L_{t-1}; L_1 = 0)
            const float2 Ls_next = t > 2 ? __ldcg(reinterpret_cast<const float2 *>(hist + (size_t)(t - 2) * Q + q0b)) : make_float2(0.f, 0.f);
            const float2 wx = splat2(w_s[2 * (t - 1)]), wy = splat2(w_s[2 * (t - 1) + 1]);
            const float Dm = ((float)(Ofin - O_s[t] - P) + lsefin) - offM;       // outputs are shifted by offM: fold it in
            const float2 offM2 = splat2(offM);
            float2 u[K];
#pragma unroll
            for (int b = 0; b < K; b += 2) {
                const float4 Mv = *reinterpret_cast<const float4 *>(Min + 128 * (b >> 1));   // M(x,b), M(x,b+1), M(x+1,b), M(x+1,b+1)
#pragma unroll
                for (int bb = 0; bb < 2; ++bb) {
                    const float4 c = tab[(b + bb) * CT + tid];
                    const float2 dx = sub2(make_float2(c.x, c.y), wx), dy = sub2(make_float2(c.z, c.w), wy);
                    const float2 Mb = bb == 0 ? make_float2(Mv.x, Mv.z) : make_float2(Mv.y, Mv.w);
                    u[b + bb] = fma2(fma2(dy, dy, mul2(dx, dx)), nl2, sub2(Mb, offM2));
                }
            }
            const float2 m = max_pairs<K>(u);
            float2 sum = make_float2(0.f, 0.f), cx = sum, cy = sum;
#pragma unroll
            for (int b = 0; b < K; ++b) {
                const float2 pb = ex2f2(sub2(u[b], m));
                const float4 c = tab[b * CT + tid];
                sum = add2(sum, pb);
                cx = fma2(pb, make_float2(c.x, c.y), cx);
                cy = fma2(pb, make_float2(c.z, c.w), cy);
            }
            const float2 out = add2(m, lg2f2(sum));
            const float2 f = ex2f2(add2(m, sub2(Ls, splat2(Dm))));
            pr.async_v2(push_b + ob_off, out.x, out.y, push_b_mbar + ob_mbar);
            const float2 fd = mul2(f, sum), fx = mul2(f, cx), fy = mul2(f, cy);
            const float den = warp_sum(fd.x + fd.y), n0 = warp_sum(fx.x + fx.y), n1 = warp_sum(fy.x + fy.y);
            const float tmax = warp_max(fmaxf(m.x, m.y));
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(ob * 64) * 4u, tmax, full_of[r] + ob_mbar);
                pr.async_v4(part_dst + (uint32_t)(ob * 256) * 4u, den, n0, n1, 0.f, full_of[0] + ob_mbar);
            }
            Ls = Ls_next;
            ib = ob;
        }
        wait_inputs(ib);                                                     // M_0 and the sums of step 1
        cmax = warp_max(slot_max(wmax + ib * 64, lane, SLOTS));
        P += (int)offM;
        finish_step(1, ib);
        // ================= consistency: P_0 + LSE_q M_0(q) against log2 Z (every CTA holds a quarter of M_0)
        {
            const float *Mfin = msg + ib * Q;
            float ssum = 0.f;
            for (int e = tid; e < QC; e += CT) ssum += ex2f(Mfin[e] - cmax);
            ssum = warp_sum(ssum);
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r] + 64u * 4u, ssum);
            }
            cluster_sync();
            float v = (lane < SLOTS ? lz[64 + lane] : 0.f) + (lane + 32 < SLOTS ? lz[96 + lane] : 0.f);
            v = warp_sum(v);
            const float lz_beta = cmax + lg2f(v);
            zgap = fmaxf(zgap, fabsf((float)(P - Ofin) + (lz_beta - lsefin)));
            cluster_sync();     // nobody still reads this block's buffers when the next block starts
        }
    }
    if (tid == 0 && rank == 0) {
        diag_max(&p.diag->max_defect, defect);
        diag_max(&p.diag->max_logz_gap, zgap);
    }
    __syncthreads();
    cluster_sync();             // no CTA leaves while a peer may still address its shared memory
    if (*abort_flag) settle_after_abort();
}

}  // namespace bcjr
