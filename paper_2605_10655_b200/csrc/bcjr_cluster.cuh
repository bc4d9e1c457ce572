// Cluster kernels for the large trellis (S = 2^LB states, LB >= 2k): one weight block per
// thread-block cluster, the state vector spread over the cluster's shared memories.
//
// Butterfly form of the recursions.  Write a state as s = [j | x | l] with j and l of k bits
// and x of LB-2k bits.  One trellis step couples, for fixed x, the K inputs L_t([j|x]) with the
// K outputs L_{t+1}([x|l]) through the K*K states [j|x|l]:
//     L_{t+1}([x|l]) = LSE_j ( L_t([j|x]) + e_t([j|x|l]) )
//     M_{t-1}([j|x]) = LSE_b ( M_t([x|b]) + e_t([j|x|b]) )
// and the posterior of state [j|x|b] at step t is proportional to
//     exp( L_t([j|x]) + e_t([j|x|b]) + M_t([x|b]) ).
// A thread owns the same butterflies x for every step, both sweeps and every block, so the
// K*K codebook entries of each of its butterflies stay in registers for the whole kernel.
// Each output has exactly one consumer butterfly; it is pushed straight into the consumer
// CTA's shared memory (st.shared::cluster), and one cluster barrier closes the step.
//
// History: the beta sweep needs L_t([j|x]) again.  The input buffer of alpha step t is exactly
// that data in the layout the owner reads it, so one elected thread streams the whole buffer
// to a per-cluster history in global memory with a bulk copy (TMA, shared -> global), and the
// beta sweep prefetches it back two steps ahead (global -> shared, mbarrier completion).
#pragma once
#include "bcjr_ptx.cuh"

namespace bcjr {

template <int LB, int KB, int CL, int THREADS>
struct ClusterCfg {
    static constexpr int K = 1 << KB;
    static constexpr int S = 1 << LB;
    static constexpr int Q = S >> KB;                 // groups = message length
    static constexpr int NB = S >> (2 * KB);          // butterflies
    static constexpr int NBC = NB / CL;               // butterflies per CTA
    static constexpr int BPT = NBC / THREADS;         // butterflies per thread
    static constexpr int QC = Q / CL;                 // message entries held per CTA
    static constexpr int NWARP = THREADS / 32;
    static constexpr int THREADS_ = THREADS;
    static constexpr int NSTAGE = 3;
    static constexpr int MAX_N = 2048;
    static_assert(LB >= 2 * KB, "butterfly form needs LB >= 2k");
    static_assert(NBC % THREADS == 0 && BPT >= 1, "butterflies must divide evenly");
    static_assert(CL * NWARP <= 64, "at most two partials per lane");
    static_assert(NBC % K == 0 || CL == 1, "vector pushes must stay inside one CTA");
    // shared memory carve-up (floats unless noted)
    static constexpr int NBUF = 3;                            // message buffers (see the step protocol)
    static constexpr int OFF_MSG = 0;                         // [NBUF][QC]
    static constexpr int OFF_STAGE = OFF_MSG + NBUF * QC;     // [NSTAGE][QC]
    static constexpr int OFF_W = OFF_STAGE + NSTAGE * QC;     // [MAX_N]
    static constexpr int OFF_O = OFF_W + MAX_N;               // int [MAX_N + 2]
    static constexpr int OFF_WMAX = OFF_O + MAX_N + 2 + 2;    // [NBUF][64]
    static constexpr int OFF_PART = OFF_WMAX + 192;           // [NBUF][64][2]
    static constexpr int OFF_LZ = OFF_PART + 384;             // [2][64]
    static constexpr int OFF_MBAR = OFF_LZ + 128;             // uint64 [NSTAGE] history ring, then [NBUF] message buffers
    static constexpr int OFF_FLAG = OFF_MBAR + 2 * (NSTAGE + NBUF) + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(OFF_MBAR % 2 == 0, "mbarrier alignment");
    static_assert((QC * 4) % 16 == 0, "bulk copies move multiples of 16 bytes");
};

// Codebook of the owned butterflies, in the pairing a sweep wants.  Alpha pairs neighbouring
// outputs l: A[i][j][h] = (c[j|x|2h], c[j|x|2h+1]);  beta pairs neighbouring inputs j:
// B[i][jh][b] = (c[2jh|x|b], c[2jh+1|x|b]).  Reloaded (from L2) at the start of each sweep.
template <typename C>
__device__ __forceinline__ void load_cb_alpha(float2 (&A)[C::BPT][C::K][C::K / 2], const float *cbk, int rank, int tid)
{
#pragma unroll
    for (int i = 0; i < C::BPT; ++i) {
        const int x = rank * C::NBC + i * C::THREADS_ + tid;
#pragma unroll
        for (int j = 0; j < C::K; ++j)
#pragma unroll
            for (int h = 0; h < C::K / 2; h += 2) {
                const float4 v = __ldg(reinterpret_cast<const float4 *>(cbk + (size_t)j * C::Q + (size_t)x * C::K) + h / 2);
                A[i][j][h] = make_float2(v.x, v.y);
                A[i][j][h + 1] = make_float2(v.z, v.w);
            }
    }
}
template <typename C>
__device__ __forceinline__ void load_cb_beta(float2 (&B)[C::BPT][C::K / 2][C::K], const float *cbk, int rank, int tid)
{
#pragma unroll
    for (int i = 0; i < C::BPT; ++i) {
        const int x = rank * C::NBC + i * C::THREADS_ + tid;
#pragma unroll
        for (int jh = 0; jh < C::K / 2; ++jh)
#pragma unroll
            for (int b = 0; b < C::K; b += 4) {
                const float4 v0 = __ldg(reinterpret_cast<const float4 *>(cbk + (size_t)(2 * jh) * C::Q + (size_t)x * C::K) + b / 4);
                const float4 v1 = __ldg(reinterpret_cast<const float4 *>(cbk + (size_t)(2 * jh + 1) * C::Q + (size_t)x * C::K) + b / 4);
                B[i][jh][b] = make_float2(v0.x, v1.x);
                B[i][jh][b + 1] = make_float2(v0.y, v1.y);
                B[i][jh][b + 2] = make_float2(v0.z, v1.z);
                B[i][jh][b + 3] = make_float2(v0.w, v1.w);
            }
    }
}

// --------------------------------------------------------------------------------------
// Forward call on a cluster: alpha sweep, log Z, beta sweep fused with Eq. 6-7.
//
// Step protocol (no per-step barrier).  The messages live in three buffers.  Step s reads
// buffer s%3 and every thread pushes its outputs, with st.async, into buffer (s+1)%3 of the
// consumer's CTA, crediting that CTA's mbarrier full[(s+1)%3].  A thread starts step s+1 when
// full[(s+1)%3] of its own CTA completes, i.e. when every input of its CTA has landed.
// Three buffers make this safe without any further handshake: a thread can only be writing
// buffer b again (step s+3) after every thread of the cluster has finished step s+2, hence
// has long finished reading b (step s+1).  The per-warp partial results (gauge maximum,
// posterior sums) travel the same way into small slot arrays.  One thread per CTA arms each
// phase (arrive.expect_tx) and moves the history with bulk copies.
// --------------------------------------------------------------------------------------
template <int LB, int KB, int CL, int THREADS>
__global__ void __launch_bounds__(THREADS, 1) fwd_cluster_kernel(FwdParams p)
{
    using C = ClusterCfg<LB, KB, CL, THREADS>;
    constexpr int K = C::K, NB = C::NB, NBC = C::NBC, BPT = C::BPT, QC = C::QC, NWARP = C::NWARP;
    constexpr int NBUF = C::NBUF, SLOTS = CL * NWARP;
    constexpr uint32_t TX_MSG = QC * 4u + SLOTS * 4u;            // messages + gauge slots per phase
    constexpr uint32_t TX_PART = SLOTS * 8u;                     // posterior partial sums (rank 0 only)
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();
    const uint32_t cid = cluster_id_x(), ncl = cluster_count_x();
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float2 nl2 = splat2(-p.lam2);

    float *msg = smem + C::OFF_MSG;
    float *stage = smem + C::OFF_STAGE;
    float *w_s = smem + C::OFF_W;
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAG);
    Proto pr{1u, abort_flag, p.diag};
    const uint32_t mbar_stage = smem_u32(smem + C::OFF_MBAR);
    const uint32_t mbar_full = mbar_stage + 8u * C::NSTAGE;
    const uint32_t msg_u32 = smem_u32(msg), stage_u32 = smem_u32(stage);
    const uint32_t wmax_u32 = smem_u32(wmax), part_u32 = smem_u32(part), lz_u32 = smem_u32(lz);

    float *hist = p.hist + (size_t)cid * n * C::Q;      // history of this cluster: [n][CL][QC]

    // Destinations.  alpha: the K outputs of butterfly x are L([x|l]) = index x*K + l; their
    // consumer is butterfly (x*K) mod NB, input slot (x*K) / NB, one CTA, contiguous.  beta: the
    // output M([j|x]) = index j*NB + x goes to butterfly (j*NB + x) / K as its input x mod K;
    // its CTA is floor(j*CL/K), a compile-time function of j.
    uint32_t push_a[BPT], push_a_mbar[BPT], push_b[BPT][K], full_of[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) full_of[r] = mapa_u32(mbar_full, (uint32_t)r);
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int x = (int)rank * NBC + i * THREADS + tid;
        {
            const int q2 = x * K;
            const int j2 = q2 / NB, x2 = q2 % NB;
            const int r2 = x2 / NBC, xl2 = x2 % NBC;
            push_a[i] = mapa_u32(msg_u32 + (uint32_t)(j2 * NBC + xl2) * 4u, (uint32_t)r2);
            push_a_mbar[i] = mapa_u32(mbar_full, (uint32_t)r2);
        }
#pragma unroll
        for (int j = 0; j < K; ++j) {
            const int q1 = j * NB + x;
            const int x1 = q1 / K, b1 = q1 % K;
            const int r1 = x1 / NBC, xl1 = x1 % NBC;
            push_b[i][j] = mapa_u32(msg_u32 + (uint32_t)(xl1 * K + b1) * 4u, (uint32_t)r1);
        }
    }
    static_assert(K % CL == 0, "beta destinations: CTA of output j is j*CL/K");
    // partial-result slots: every warp of every CTA writes one entry into every CTA's array
    uint32_t wmax_dst[CL], lz_dst[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        wmax_dst[r] = mapa_u32(wmax_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
        lz_dst[r] = mapa_u32(lz_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
    }
    const uint32_t part_dst = mapa_u32(part_u32 + (uint32_t)((int)rank * NWARP + warp) * 8u, 0u);

    if (tid == 0) {
        for (int s = 0; s < C::NSTAGE + NBUF; ++s) mbar_init(mbar_stage + 8u * s, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t loads_done = 0;       // bulk loads consumed so far (stage = count % NSTAGE, parity = (count / NSTAGE) & 1)
    uint32_t loads_issued = 0;
    uint32_t full_phase = 0;       // bit b = parity to wait for on full[b]
    int ib = 0;                    // buffer holding the inputs of the next step
    float defect = 0.f, zgap = 0.f;

    // wait until every input of this CTA for the coming step has landed in buffer b
    auto wait_inputs = [&](int b) {
        pr.wait(mbar_full + 8u * b, (full_phase >> b) & 1u);
        full_phase ^= 1u << b;
    };

    for (int64_t blk = cid; blk < p.B; blk += ncl) {
        const float *w = p.W + blk * n;
        for (int t = tid; t < n; t += THREADS) w_s[t] = __ldg(w + t);
        for (int q = tid; q < QC; q += THREADS) msg[ib * QC + q] = 0.f;      // L_1 = 0
        if (tid == 0) O_s[1] = 0;
        int O = 0;
        float off = 0.f, cmax = 0.f;
        cluster_sync();
        // ================= alpha sweep: step t maps L_t to L_{t+1}
        {
            float2 cbA[BPT][K][K / 2];
            load_cb_alpha<C>(cbA, p.cb, (int)rank, tid);
            for (int t = 1; t <= n; ++t) {
                const int ob = ib == NBUF - 1 ? 0 : ib + 1;
                if (t > 1) {
                    wait_inputs(ib);
                    // gauge: rounded maximum of the group maxima of the previous step (within
                    // log2 K of the maximum of L_t, which is all a gauge needs)
                    cmax = warp_max(slot_max(wmax + ib * 64, lane, SLOTS)) - off;
                    off = rintf(cmax);
                }
                const float *Lin = msg + ib * QC;
                const uint32_t ob_off = (uint32_t)(ob * QC) * 4u, ob_mbar = 8u * ob;
                if (tid == 0) {
                    pr.expect_tx(mbar_full + ob_mbar, TX_MSG);
                    bulk_wait_read0();                                   // previous spill has left its buffer
                    fence_proxy_async();
                    pr.store(hist + ((size_t)(t - 1) * CL + rank) * QC, msg_u32 + (uint32_t)(ib * QC) * 4u, QC * 4u);
                    bulk_commit();
                }
                const float2 w2 = splat2(w_s[t - 1]);
                const float2 off2 = splat2(off);
                float tmax = NEG_INF;
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    const int xl = i * THREADS + tid;
                    float2 Lj[K];
#pragma unroll
                    for (int j = 0; j < K; ++j) Lj[j] = splat2(Lin[j * NBC + xl]);
                    float2 out[K / 2];
#pragma unroll
                    for (int h = 0; h < K / 2; ++h) {
                        float2 a[K];
#pragma unroll
                        for (int j = 0; j < K; ++j) {
                            const float2 d = sub2(cbA[i][j][h], w2);
                            a[j] = fma2(mul2(d, d), nl2, Lj[j]);
                        }
                        const float2 m = max_pairs<K>(a);
                        float2 sum = ex2f2(sub2(a[0], m));
#pragma unroll
                        for (int j = 1; j < K; ++j) sum = add2(sum, ex2f2(sub2(a[j], m)));
                        out[h] = add2(sub2(m, off2), lg2f2(sum));
                        tmax = max3f(tmax, m.x, m.y);
                    }
#pragma unroll
                    for (int h = 0; h < K / 2; h += 2)
                        pr.async_v4(push_a[i] + ob_off + 8u * h, out[h].x, out[h].y, out[h + 1].x, out[h + 1].y,
                                    push_a_mbar[i] + ob_mbar);
                }
                tmax = warp_max(tmax);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(ob * 64) * 4u, tmax, full_of[r] + ob_mbar);
                }
                O += (int)off;
                if (tid == 0) O_s[t + 1] = O;
                ib = ob;
            }
        }
        // ================= log2 Z = O_{n+1} + LSE_q L_{n+1}(q); L_{n+1} sits in buffer ib
        wait_inputs(ib);
        cmax = warp_max(slot_max(wmax + ib * 64, lane, SLOTS)) - off;
        {
            const float *Lfin = msg + ib * QC;
            float ssum = 0.f;
            for (int q = tid; q < QC; q += THREADS) ssum += ex2f(Lfin[q] - cmax);
            ssum = warp_sum(ssum);
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r], ssum);
            }
            if (tid == 0) bulk_wait_all0();                          // history fully written
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
        if (tid == 0 && rank == 0 && p.logZ)
            p.logZ[blk] = (float)(((double)Ofin + (double)lsefin) * 0.6931471805599453);
        // ================= beta sweep: step t maps M_t to M_{t-1}
        for (int q = tid; q < QC; q += THREADS) msg[ib * QC + q] = 0.f;      // M_n = 0
        if (tid == 0) {                                              // prefetch L_n and L_{n-1}
            fence_proxy_async();
            for (int d = 0; d < 2 && n - d >= 1; ++d) {
                const uint32_t s = loads_issued % C::NSTAGE;
                pr.expect_tx(mbar_stage + 8u * s, QC * 4u);
                pr.load(stage_u32 + s * QC * 4u, hist + ((size_t)(n - d - 1) * CL + rank) * QC, QC * 4u, mbar_stage + 8u * s);
                loads_issued += pr.live ? 1u : 0u;
            }
        }
        int P = 0;
        float offM = 0.f;
        cluster_sync();
        {
            float2 cbB[BPT][K / 2][K];
            load_cb_beta<C>(cbB, p.cb, (int)rank, tid);
            // rank 0, warp 0: turn the partial sums of step t (slots of buffer b) into soft[t]
            auto finish_step = [&](int t, int b) {
                if (rank == 0 && warp == 0) {
                    float a = lane < SLOTS ? part[(b * 64 + lane) * 2] : 0.f;
                    float c = lane < SLOTS ? part[(b * 64 + lane) * 2 + 1] : 0.f;
                    if (lane + 32 < SLOTS) { a += part[(b * 64 + lane + 32) * 2]; c += part[(b * 64 + lane + 32) * 2 + 1]; }
                    a = warp_sum(a); c = warp_sum(c);
                    if (lane == 0) {
                        const float sw = a / c;
                        p.soft[blk * n + t - 1] = sw;
                        if (p.soft_copy) p.soft_copy[blk * n + t - 1] = sw;
                        defect = fmaxf(defect, fabsf(c - 1.f));
                    }
                }
            };
            for (int t = n; t >= 1; --t) {
                const int ob = ib == NBUF - 1 ? 0 : ib + 1;
                if (t < n) {
                    wait_inputs(ib);
                    cmax = warp_max(slot_max(wmax + ib * 64, lane, SLOTS));
                    P += (int)offM;                                      // P_t
                    offM = rintf(cmax);
                    finish_step(t + 1, ib);
                }
                const float *Min = msg + ib * QC;
                const uint32_t ob_off = (uint32_t)(ob * QC) * 4u, ob_mbar = 8u * ob;
                if (tid == 0) {
                    pr.expect_tx(mbar_full + ob_mbar, rank == 0 ? TX_MSG + TX_PART : TX_MSG);
                    if (t - 2 >= 1) {                                    // prefetch L_{t-2}
                        fence_proxy_async();
                        const uint32_t s = loads_issued % C::NSTAGE;
                        pr.expect_tx(mbar_stage + 8u * s, QC * 4u);
                        pr.load(stage_u32 + s * QC * 4u, hist + ((size_t)(t - 3) * CL + rank) * QC, QC * 4u, mbar_stage + 8u * s);
                        loads_issued += pr.live ? 1u : 0u;
                    }
                }
                const uint32_t st = loads_done % C::NSTAGE;
                pr.wait(mbar_stage + 8u * st, (loads_done / C::NSTAGE) & 1u);
                ++loads_done;
                const float *Lh = stage + st * QC;
                const float2 w2 = splat2(w_s[t - 1]);
                // the outputs are gauge-shifted by offM; fold the shift into the inputs and into D
                const float Dm = ((float)(Ofin - O_s[t] - P) + lsefin) - offM;
                float2 num2 = make_float2(0.f, 0.f), den2 = make_float2(0.f, 0.f);
                float tmax = NEG_INF;
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    const int xl = i * THREADS + tid;
                    float2 Mb[K];
#pragma unroll
                    for (int b = 0; b < K; b += 4) {
                        const float4 v = *reinterpret_cast<const float4 *>(Min + xl * K + b);
                        Mb[b] = splat2(v.x - offM); Mb[b + 1] = splat2(v.y - offM);
                        Mb[b + 2] = splat2(v.z - offM); Mb[b + 3] = splat2(v.w - offM);
                    }
#pragma unroll
                    for (int jh = 0; jh < K / 2; ++jh) {
                        float2 u[K];
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            const float2 d = sub2(cbB[i][jh][b], w2);
                            u[b] = fma2(mul2(d, d), nl2, Mb[b]);
                        }
                        const float2 m = max_pairs<K>(u);
                        const float2 LhD = make_float2(Lh[(2 * jh) * NBC + xl] - Dm, Lh[(2 * jh + 1) * NBC + xl] - Dm);
                        const float2 f = ex2f2(add2(m, LhD));
                        float2 pb = ex2f2(sub2(u[0], m));
                        float2 sum = pb, craw = mul2(pb, cbB[i][jh][0]);
#pragma unroll
                        for (int b = 1; b < K; ++b) {
                            pb = ex2f2(sub2(u[b], m));
                            sum = add2(sum, pb);
                            craw = fma2(pb, cbB[i][jh][b], craw);
                        }
                        const float2 out = add2(m, lg2f2(sum));
                        tmax = max3f(tmax, m.x, m.y);
                        pr.async_f32(push_b[i][2 * jh] + ob_off, out.x, full_of[(2 * jh) * CL / K] + ob_mbar);
                        pr.async_f32(push_b[i][2 * jh + 1] + ob_off, out.y, full_of[(2 * jh + 1) * CL / K] + ob_mbar);
                        num2 = fma2(f, craw, num2);
                        den2 = fma2(f, sum, den2);
                    }
                }
                const float num = warp_sum(num2.x + num2.y), den = warp_sum(den2.x + den2.y);
                tmax = warp_max(tmax);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(ob * 64) * 4u, tmax, full_of[r] + ob_mbar);
                    pr.async_v2(part_dst + (uint32_t)(ob * 128) * 4u, num, den, full_of[0] + ob_mbar);
                }
                ib = ob;
            }
            wait_inputs(ib);                                             // M_0 and the sums of step 1
            cmax = warp_max(slot_max(wmax + ib * 64, lane, SLOTS));
            P += (int)offM;                                              // P_0
            finish_step(1, ib);
        }
        // ================= consistency: P_0 + LSE_q M_0(q) against log2 Z (M_0 in buffer ib)
        {
            const float *Mfin = msg + ib * QC;
            float ssum = 0.f;
            for (int q = tid; q < QC; q += THREADS) ssum += ex2f(Mfin[q] - cmax);
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
    if (*abort_flag && tid == 0) drain_bulk_loads(mbar_stage, loads_issued, C::NSTAGE, p.diag);
    __syncthreads();
    cluster_sync();             // no CTA leaves while a peer may still address its shared memory
    if (*abort_flag) settle_after_abort();
}

// --------------------------------------------------------------------------------------
// Backward call on a cluster.  Same butterflies; each message now carries a second value, the
// conditional expectation of the centred emitted sum (At on the alpha side, Bt on the beta
// side, see bcjr_generic.cuh for the recursions).  The codebook gradient of a state is owned
// by the thread that owns the state, for every step and every block, so it accumulates in
// registers and is written once, at the end, to this cluster's partial sum.
//
// Per step the beta sweep hands three sums over the posterior to rank 0:
//   S0 = sum gamma,   S2 = sum gamma r,   ZS = sum gamma (g_t + (w_t - c) r / T)
// (ZS is the sum over states of exactly what is added to the codebook-gradient accumulators)
// and  grad_W[t] = -(1/T) Cov(r, w_t - c) = g_t - ZS/S0 + (S2/S0) (w_t - soft_t) / T.
// --------------------------------------------------------------------------------------
template <int LB, int KB, int CL, int THREADS>
struct BwdClusterCfg {
    using F = ClusterCfg<LB, KB, CL, THREADS>;
    static constexpr int QC = F::QC;
    static constexpr int NSTAGE = 3;
    static constexpr int MAX_N = 2048;
    static constexpr int OFF_MSG = 0;                          // [2 parity][2 arrays][QC]
    static constexpr int OFF_STAGE = OFF_MSG + 4 * QC;         // [NSTAGE][2][QC]
    static constexpr int OFF_W = OFF_STAGE + NSTAGE * 2 * QC;  // w, g, soft: [3][MAX_N]
    static constexpr int OFF_O = OFF_W + 3 * MAX_N;            // int [MAX_N + 4]
    static constexpr int OFF_WMAX = OFF_O + MAX_N + 4;         // [2][64]
    static constexpr int OFF_PART = OFF_WMAX + 128;            // [2][64][4]
    static constexpr int OFF_LZ = OFF_PART + 512;              // [64]
    static constexpr int OFF_MBAR = OFF_LZ + 64;               // uint64 [NSTAGE]
    static constexpr int OFF_FLAG = OFF_MBAR + 2 * NSTAGE + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(OFF_MBAR % 2 == 0, "mbarrier alignment");
};

template <int LB, int KB, int CL, int THREADS>
__global__ void __launch_bounds__(THREADS, 1) bwd_cluster_kernel(BwdParams p)
{
    using C = ClusterCfg<LB, KB, CL, THREADS>;
    using BC = BwdClusterCfg<LB, KB, CL, THREADS>;
    constexpr int K = C::K, NB = C::NB, NBC = C::NBC, BPT = C::BPT, QC = C::QC, NWARP = C::NWARP;
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();
    const uint32_t cid = cluster_id_x(), ncl = cluster_count_x();
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float invT = p.invT;
    const float2 nl2 = splat2(-p.lam2);

    float *msg = smem + BC::OFF_MSG;
    float *stage = smem + BC::OFF_STAGE;
    float *w_s = smem + BC::OFF_W, *g_s = w_s + BC::MAX_N, *sf_s = g_s + BC::MAX_N;
    int *O_s = reinterpret_cast<int *>(smem + BC::OFF_O);
    float *wmax = smem + BC::OFF_WMAX;
    float *part = smem + BC::OFF_PART;
    float *lz = smem + BC::OFF_LZ;
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + BC::OFF_FLAG);
    Proto pr{1u, abort_flag, p.diag};
    const uint32_t mbar0 = smem_u32(smem + BC::OFF_MBAR);
    const uint32_t msg_u32 = smem_u32(msg), stage_u32 = smem_u32(stage);
    const uint32_t wmax_u32 = smem_u32(wmax), part_u32 = smem_u32(part), lz_u32 = smem_u32(lz);
    constexpr uint32_t STEP_BYTES = 2u * QC * 4u;            // both arrays of one parity / one stage

    float *hist = p.hist + (size_t)cid * n * 2 * C::Q;       // [n][CL][2][QC]

    float2 acc[BPT][K / 2][K];                               // grad_codebook of the owned states, paired like cbB
    uint32_t push_a[BPT], push_b[BPT][K];
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int x = (int)rank * NBC + i * THREADS + tid;
#pragma unroll
        for (int jh = 0; jh < K / 2; ++jh)
#pragma unroll
            for (int b = 0; b < K; ++b) acc[i][jh][b] = make_float2(0.f, 0.f);
        {
            const int q2 = x * K;
            const int j2 = q2 / NB, x2 = q2 % NB;
            const int r2 = x2 / NBC, xl2 = x2 % NBC;
            push_a[i] = mapa_u32(msg_u32 + (uint32_t)(j2 * NBC + xl2) * 4u, (uint32_t)r2);
        }
#pragma unroll
        for (int j = 0; j < K; ++j) {
            const int q1 = j * NB + x;
            const int x1 = q1 / K, b1 = q1 % K;
            const int r1 = x1 / NBC, xl1 = x1 % NBC;
            push_b[i][j] = mapa_u32(msg_u32 + (uint32_t)(xl1 * K + b1) * 4u, (uint32_t)r1);
        }
    }
    uint32_t wmax_dst[CL], lz_dst[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        wmax_dst[r] = mapa_u32(wmax_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
        lz_dst[r] = mapa_u32(lz_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
    }
    const uint32_t part_dst = mapa_u32(part_u32 + (uint32_t)((int)rank * NWARP + warp) * 16u, 0u);

    if (tid == 0) {
        for (int s = 0; s < BC::NSTAGE; ++s) mbar_init(mbar0 + 8u * s, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    uint32_t loads_done = 0, loads_issued = 0;
    float defect = 0.f;

    for (int64_t blk = cid; blk < p.B; blk += ncl) {
        for (int t = tid; t < n; t += THREADS) {
            w_s[t] = __ldg(p.W + blk * n + t);
            g_s[t] = __ldg(p.g + blk * n + t);
            sf_s[t] = __ldg(p.soft + blk * n + t);
        }
        for (int q = tid; q < 2 * QC; q += THREADS) msg[q] = 0.f;    // L_1 = 0, At_1 = 0 (parity 0)
        if (tid == 0) O_s[1] = 0;
        int O = 0;
        float off = 0.f, cmax = 0.f;
        cluster_sync();
        // ================= alpha sweep carrying (L, At)
        {
            float2 cbA[BPT][K][K / 2];
            load_cb_alpha<C>(cbA, p.cb, (int)rank, tid);
            for (int t = 1; t <= n; ++t) {
                const int cur = (t - 1) & 1;
                const float *Lin = msg + cur * 2 * QC, *Ain = Lin + QC;
                const uint32_t nxt_off = (uint32_t)((t & 1) * 2 * QC) * 4u;
                if (tid == 0) {
                    fence_proxy_async();
                    pr.store(hist + ((size_t)(t - 1) * CL + rank) * 2 * QC, msg_u32 + (uint32_t)(cur * 2 * QC) * 4u, STEP_BYTES);
                    bulk_commit();
                }
                const float gt = g_s[t - 1];
                const float gsh = -gt * sf_s[t - 1];                      // centring: h = g c - g soft
                const float2 w2 = splat2(w_s[t - 1]), g2 = splat2(gt), off2 = splat2(off);
                float tmax = NEG_INF;
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    const int xl = i * THREADS + tid;
                    float2 Lj[K], Aj[K];
#pragma unroll
                    for (int j = 0; j < K; ++j) { Lj[j] = splat2(Lin[j * NBC + xl]); Aj[j] = splat2(Ain[j * NBC + xl] + gsh); }
                    float2 outL[K / 2], outA[K / 2];
#pragma unroll
                    for (int h = 0; h < K / 2; ++h) {
                        float2 a[K];
#pragma unroll
                        for (int j = 0; j < K; ++j) {
                            const float2 d = sub2(cbA[i][j][h], w2);
                            a[j] = fma2(mul2(d, d), nl2, Lj[j]);
                        }
                        const float2 m = max_pairs<K>(a);
                        float2 pj = ex2f2(sub2(a[0], m));
                        float2 sum = pj, ax = mul2(pj, fma2(g2, cbA[i][0][h], Aj[0]));
#pragma unroll
                        for (int j = 1; j < K; ++j) {
                            pj = ex2f2(sub2(a[j], m));
                            sum = add2(sum, pj);
                            ax = fma2(pj, fma2(g2, cbA[i][j][h], Aj[j]), ax);
                        }
                        outL[h] = add2(sub2(m, off2), lg2f2(sum));
                        outA[h] = mul2(ax, rcpf2(sum));
                        tmax = max3f(tmax, m.x, m.y);
                    }
#pragma unroll
                    for (int h = 0; h < K / 2; h += 2) {
                        st_cluster_v4(push_a[i] + nxt_off + 8u * h, outL[h].x, outL[h].y, outL[h + 1].x, outL[h + 1].y);
                        st_cluster_v4(push_a[i] + nxt_off + QC * 4u + 8u * h, outA[h].x, outA[h].y, outA[h + 1].x, outA[h + 1].y);
                    }
                }
                tmax = warp_max(tmax);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_cluster_f32(wmax_dst[r] + (uint32_t)((t & 1) * 64) * 4u, tmax);
                }
                O += (int)off;
                if (tid == 0) {
                    O_s[t + 1] = O;
                    bulk_wait_read0();
                }
                cluster_sync();
                cmax = warp_max(slot_max(wmax + (t & 1) * 64, lane, CL * NWARP)) - off;
                off = rintf(cmax);
            }
        }
        // ================= log2 Z
        {
            const float *Lfin = msg + (n & 1) * 2 * QC;
            float ssum = 0.f;
            for (int q = tid; q < QC; q += THREADS) ssum += ex2f(Lfin[q] - cmax);
            ssum = warp_sum(ssum);
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r], ssum);
            }
            if (tid == 0) bulk_wait_all0();
            cluster_sync();
        }
        float lsefin;
        {
            float v = (lane < CL * NWARP ? lz[lane] : 0.f) + (lane + 32 < CL * NWARP ? lz[lane + 32] : 0.f);
            v = warp_sum(v);
            lsefin = cmax + lg2f(v);
            if (tid == 0) diag_check_finite(p.diag, lsefin);
        }
        const int Ofin = O;
        // ================= beta sweep carrying (M, Bt), with the gradient contraction
        for (int q = tid; q < 2 * QC; q += THREADS) msg[q] = 0.f;    // M_n = 0, Bt_n = 0 (parity 0)
        if (tid == 0) {
            fence_proxy_async();
            for (int d = 0; d < 2 && n - d >= 1; ++d) {
                const uint32_t s = loads_issued % BC::NSTAGE;
                pr.expect_tx(mbar0 + 8u * s, STEP_BYTES);
                pr.load(stage_u32 + s * STEP_BYTES, hist + ((size_t)(n - d - 1) * CL + rank) * 2 * QC, STEP_BYTES, mbar0 + 8u * s);
                loads_issued += pr.live ? 1u : 0u;
            }
        }
        int P = 0;
        float offM = 0.f;
        cluster_sync();
        {
            float2 cbB[BPT][K / 2][K];
            load_cb_beta<C>(cbB, p.cb, (int)rank, tid);
            for (int t = n; t >= 1; --t) {
                const int cur = (n - t) & 1;
                const float *Min = msg + cur * 2 * QC, *Bin = Min + QC;
                const uint32_t nxt_off = (uint32_t)((cur ^ 1) * 2 * QC) * 4u;
                if (tid == 0 && t - 2 >= 1) {
                    fence_proxy_async();
                    const uint32_t s = loads_issued % BC::NSTAGE;
                    pr.expect_tx(mbar0 + 8u * s, STEP_BYTES);
                    pr.load(stage_u32 + s * STEP_BYTES, hist + ((size_t)(t - 3) * CL + rank) * 2 * QC, STEP_BYTES, mbar0 + 8u * s);
                    loads_issued += pr.live ? 1u : 0u;
                }
                const uint32_t st = loads_done % BC::NSTAGE;
                pr.wait(mbar0 + 8u * st, (loads_done / BC::NSTAGE) & 1u);
                ++loads_done;
                const float *Lh = stage + st * 2 * QC, *Ah = Lh + QC;
                const float wt = w_s[t - 1], gt = g_s[t - 1], sft = sf_s[t - 1];
                const float gsh = -gt * sft;
                const float2 w2 = splat2(wt), g2 = splat2(gt), gi2 = splat2(invT);
                const float Dm = ((float)(Ofin - O_s[t] - P) + lsefin) - offM;
                float2 S0 = make_float2(0.f, 0.f), S2 = S0, ZS = S0;
                float tmax = NEG_INF;
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    const int xl = i * THREADS + tid;
                    float2 Mb[K], Yb[K];
#pragma unroll
                    for (int b = 0; b < K; b += 4) {
                        const float4 v = *reinterpret_cast<const float4 *>(Min + xl * K + b);
                        Mb[b] = splat2(v.x - offM); Mb[b + 1] = splat2(v.y - offM);
                        Mb[b + 2] = splat2(v.z - offM); Mb[b + 3] = splat2(v.w - offM);
                        const float4 y = *reinterpret_cast<const float4 *>(Bin + xl * K + b);
                        Yb[b] = splat2(y.x + gsh); Yb[b + 1] = splat2(y.y + gsh);
                        Yb[b + 2] = splat2(y.z + gsh); Yb[b + 3] = splat2(y.w + gsh);
                    }
#pragma unroll
                    for (int jh = 0; jh < K / 2; ++jh) {
                        float2 u[K], d[K];
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            d[b] = sub2(w2, cbB[i][jh][b]);
                            u[b] = fma2(mul2(d[b], d[b]), nl2, Mb[b]);
                        }
                        const float2 m = max_pairs<K>(u);
                        const float2 Ahj = make_float2(Ah[(2 * jh) * NBC + xl], Ah[(2 * jh + 1) * NBC + xl]);
                        const float2 LhD = make_float2(Lh[(2 * jh) * NBC + xl] - Dm, Lh[(2 * jh + 1) * NBC + xl] - Dm);
                        const float2 f = ex2f2(add2(m, LhD));
                        const float2 fg = mul2(f, g2), fi = mul2(f, gi2);
                        float2 sum = make_float2(0.f, 0.f), ya = sum, zs = sum;
#pragma unroll
                        for (int b = 0; b < K; ++b) {
                            const float2 pb = ex2f2(sub2(u[b], m));
                            const float2 y = fma2(g2, cbB[i][jh][b], Yb[b]);            // h + Bt
                            const float2 z = fma2(mul2(fi, d[b]), add2(y, Ahj), fg);      // f (g + (w - c) r / T)
                            sum = add2(sum, pb);
                            ya = fma2(pb, y, ya);
                            zs = fma2(pb, z, zs);
                            acc[i][jh][b] = fma2(pb, z, acc[i][jh][b]);
                        }
                        const float2 outM = add2(m, lg2f2(sum));
                        const float2 outB = mul2(ya, rcpf2(sum));
                        tmax = max3f(tmax, m.x, m.y);
                        st_cluster_f32(push_b[i][2 * jh] + nxt_off, outM.x);
                        st_cluster_f32(push_b[i][2 * jh + 1] + nxt_off, outM.y);
                        st_cluster_f32(push_b[i][2 * jh] + nxt_off + QC * 4u, outB.x);
                        st_cluster_f32(push_b[i][2 * jh + 1] + nxt_off + QC * 4u, outB.y);
                        S0 = fma2(f, sum, S0);
                        S2 = fma2(f, fma2(Ahj, sum, ya), S2);
                        ZS = add2(ZS, zs);
                    }
                }
                const float s0 = warp_sum(S0.x + S0.y), s2 = warp_sum(S2.x + S2.y), zz = warp_sum(ZS.x + ZS.y);
                tmax = warp_max(tmax);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_cluster_f32(wmax_dst[r] + (uint32_t)((t & 1) * 64) * 4u, tmax);
                    const uint32_t pd = part_dst + (uint32_t)((t & 1) * 256) * 4u;
                    st_cluster_f32(pd, s0); st_cluster_f32(pd + 4u, s2); st_cluster_f32(pd + 8u, zz);
                }
                P += (int)offM;
                cluster_sync();
                cmax = warp_max(slot_max(wmax + (t & 1) * 64, lane, CL * NWARP));
                offM = rintf(cmax);
                if (rank == 0 && warp == 0) {
                    const float *pp = part + (t & 1) * 256 + lane * 4;
                    const bool on = lane < CL * NWARP, on2 = lane + 32 < CL * NWARP;
                    float a0 = on ? pp[0] : 0.f, a2 = on ? pp[1] : 0.f, az = on ? pp[2] : 0.f;
                    if (on2) { a0 += pp[128]; a2 += pp[129]; az += pp[130]; }
                    a0 = warp_sum(a0); a2 = warp_sum(a2); az = warp_sum(az);
                    if (lane == 0) {
                        const float i0 = 1.f / a0;
                        p.gW[blk * n + t - 1] = (gt - az * i0) + (a2 * i0) * (wt - sft) * invT;
                        defect = fmaxf(defect, fabsf(a0 - 1.f));
                    }
                }
            }
        }
        cluster_sync();
    }
    // this cluster's partial of grad_codebook: state [j|x|b] = j*Q + x*K + b
    float *gc = p.gc_part + (size_t)cid * C::S;
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int x = (int)rank * NBC + i * THREADS + tid;
#pragma unroll
        for (int jh = 0; jh < K / 2; ++jh)
#pragma unroll
            for (int b = 0; b < K; ++b) {
                gc[(size_t)(2 * jh) * C::Q + (size_t)x * K + b] = acc[i][jh][b].x;
                gc[(size_t)(2 * jh + 1) * C::Q + (size_t)x * K + b] = acc[i][jh][b].y;
            }
    }
    if (tid == 0 && rank == 0) diag_max(&p.diag->max_defect, defect);
    if (*abort_flag && tid == 0) drain_bulk_loads(mbar0, loads_issued, BC::NSTAGE, p.diag);
    __syncthreads();
    cluster_sync();             // no CTA leaves while a peer may still address its shared memory
    if (*abort_flag) settle_after_abort();
}

// ---------------------------------------------------------------------------- host side
inline bool cluster_supported(int Lb, int k) { return Lb == 16 && (k == 2 || k == 3); }

}  // namespace bcjr
