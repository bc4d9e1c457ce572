// Vector-emission trellis with 16 state bits, 4 bits and V = 2 weights per step (the paper's
// "L=16, k=2, V=2"): weight blocks on clusters of FOUR CTAs, table slice resident in tensor memory.
//
// Ownership.  Q = 4096 groups, 1024 per CTA, an adjacent pair per thread; which groups a CTA owns
// is chosen per sweep so that it reads only a quarter of the messages:
//   alpha:  L_{t+1}(q) = LSE_j [ L_t((q >> 4) + 256 j) + e_t(q + jQ) ]              CTA r owns q >> 10 == r
//           and reads the entries i of L_t with ((i & 255) >> 6) == r;
//   beta :  M_{t-1}(q) = LSE_b [ M_t(((q & 255) << 4) | b) + e_t(16 q + b) ]        CTA r owns ((q & 255) >> 6) == r
//           and reads the entries i of M_t with (i >> 10) == r.
// Hence every output has exactly one consumer CTA: one st.async (the thread's pair) per thread
// and step.  The table slice of a sweep is 16 entries x 2 groups x 2 floats per thread,
// thread-private: 128 KB per CTA = 64 TMEM columns per thread (lane-private scratchpad use of
// tensor memory, as in the scalar kernels; shared memory would spend its whole bandwidth on
// these reads), staged at the start of each sweep (alpha from the table itself, which is
// [j][q][V] in memory; beta from the copy regrouped [b][q][V]) as (c0.x, c1.x), (c0.y, c1.y) per
// entry for the thread's two groups, i.e. ready-made f32x2 pairs, four entries per 16-column unit.
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
#include "bcjr_solo.cuh"

namespace bcjr {

template <int NBLK_>
struct Vec4Cfg {
    static constexpr int LB = 16, KB = 4, V = 2, K = 16, S = 1 << LB, Q = S >> KB;
    static constexpr int CL = 4, THREADS = 512, NWARP = THREADS / 32, QC = Q / CL;
    static constexpr int SLOTS = CL * NWARP;                   // 64 per-warp partial slots
    static constexpr int NBUF = 3;
    static constexpr int NBLK = NBLK_;                         // weight blocks in flight per cluster
    static constexpr int UNITS = 4;                            // 16-column TMEM units: 4 table entries (x 2 groups x 2 floats) each
    static constexpr int MAX_N = 2048, MAX_NT = MAX_N / V;     // weights / steps per block
    static constexpr int OFF_MSG = 0;                                  // [NBUF][NBLK][QC]
    static constexpr int OFF_W = OFF_MSG + NBUF * NBLK * QC;           // [NBLK][MAX_N]
    static constexpr int OFF_O = OFF_W + NBLK * MAX_N;                 // int [NBLK][MAX_NT + 4]
    static constexpr int OFF_WMAX = OFF_O + NBLK * (MAX_NT + 4);       // [NBUF][NBLK][64]
    static constexpr int OFF_PART = OFF_WMAX + NBUF * NBLK * 64;       // [NBUF][NBLK][64][4]: den, num_0, num_1
    static constexpr int OFF_LZ = OFF_PART + NBUF * NBLK * 64 * 4;     // [2][NBLK][64]
    static constexpr int OFF_MBAR = OFF_LZ + 2 * NBLK * 64;            // uint64 [NBUF][NBLK]
    static constexpr int OFF_TMEM = OFF_MBAR + 2 * NBUF * NBLK + 2;
    static constexpr int OFF_FLAG = OFF_TMEM + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(QC == 2 * THREADS, "a thread owns two adjacent groups");
    static_assert(OFF_MBAR % 2 == 0 && OFF_MSG % 4 == 0 && OFF_PART % 4 == 0, "alignment");
    static_assert(SMEM_BYTES <= 232448, "shared memory of one CTA");
    static_assert(NBLK <= NWARP && NBUF * NBLK <= 32, "one finishing warp per block in flight; phase bits");
};

// table slice for one sweep into the thread's TMEM columns: src is [16][Q][2]; entry j of the
// thread's groups q0, q0 + 1 becomes the pairs (c0.x, c1.x), (c0.y, c1.y) at columns 4 j .. 4 j + 3
__device__ __forceinline__ void vec4_stage_table(uint32_t tm, const float *src, int q0)
{
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        float2 v[8];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float4 c = __ldg(reinterpret_cast<const float4 *>(src + ((size_t)(4 * u + e) * 4096 + q0) * 2));
            v[2 * e] = make_float2(c.x, c.z);
            v[2 * e + 1] = make_float2(c.y, c.w);
        }
        tmem_st16(tm + 16u * u, v);
    }
    tmem_wait_st();
}

// Several weight blocks (NBLK) are in flight per cluster, all in the same step of the same sweep:
// a step of the trellis is short (32 states per thread) against the latency of the exchange, so
// the cluster works through "block 0 step t, block 1 step t, ..." and the messages of a block
// travel while the other blocks compute.  The table slice is shared by the blocks in flight.
template <int NBLK_>
__global__ void __launch_bounds__(Vec4Cfg<NBLK_>::THREADS, 1) fwd_vec4_kernel(FwdParams p)
{
    using C = Vec4Cfg<NBLK_>;
    constexpr int K = C::K, Q = C::Q, QC = C::QC, CL = C::CL, NWARP = C::NWARP, NBUF = C::NBUF, SLOTS = C::SLOTS, CT = C::THREADS;
    constexpr int NBLK = C::NBLK, OSTR = C::MAX_NT + 4;
    constexpr uint32_t TX_MSG = QC * 4u + SLOTS * 4u;            // a quarter of the messages + gauge slots
    constexpr uint32_t TX_PART = SLOTS * 16u;                    // posterior sums (rank 0 only)
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();
    const uint32_t cid = cluster_id_x(), ncl = cluster_count_x();
    const int n = p.n, nt = n / C::V;
    const float2 nl2 = splat2(-p.lam2);

    float *msg = smem + C::OFF_MSG;
    float *w_s = smem + C::OFF_W;
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAG);
    Proto pr{1u, abort_flag, p.diag};
    const uint32_t mbar_full = smem_u32(smem + C::OFF_MBAR);     // [NBUF][NBLK]
    const uint32_t msg_u32 = smem_u32(msg), wmax_u32 = smem_u32(wmax), part_u32 = smem_u32(part), lz_u32 = smem_u32(lz);

    const int q0 = (int)rank * QC + 2 * tid;                     // alpha sweep: this thread's groups q0, q0 + 1
    const int q0b = warp * 256 + (int)rank * 64 + 2 * lane;      // beta sweep: groups q0b, q0b + 1
    float *hist = p.hist + (size_t)cid * NBLK * nt * Q;          // [NBLK][nt][Q]: row t = L_{t+1}

    uint32_t full_of[CL], msg_of[CL], wmax_dst[CL], lz_dst[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        full_of[r] = mapa_u32(mbar_full, (uint32_t)r);
        msg_of[r] = mapa_u32(msg_u32, (uint32_t)r);
        wmax_dst[r] = mapa_u32(wmax_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
        lz_dst[r] = mapa_u32(lz_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
    }
    const uint32_t part_dst = mapa_u32(part_u32 + (uint32_t)((int)rank * NWARP + warp) * 16u, 0u);
    // alpha: entry i of L is read by CTA (i & 255) >> 6, which keeps its quarter as [i >> 8][i & 63];
    // the thread's outputs (q0, q0 + 1) are adjacent there
    const int ra = (q0 & 255) >> 6;
    const uint32_t push_a = (ra == 0 ? msg_of[0] : ra == 1 ? msg_of[1] : ra == 2 ? msg_of[2] : msg_of[3])
                            + (uint32_t)((q0 >> 8) * 64 + (q0 & 63)) * 4u;
    const uint32_t push_a_mbar = ra == 0 ? full_of[0] : ra == 1 ? full_of[1] : ra == 2 ? full_of[2] : full_of[3];
    // beta: entry i = (x', b') of M (x' = i >> 4, b' = i & 15) is read by CTA x' >> 6, kept as
    // [b' >> 1][x' & 63][b' & 1]; the thread's outputs are (x', b'), (x', b' + 1) with b' even
    const int rb = warp >> 2;
    const uint32_t push_b = (rb == 0 ? msg_of[0] : rb == 1 ? msg_of[1] : rb == 2 ? msg_of[2] : msg_of[3])
                            + (uint32_t)(((q0b & 15) >> 1) * 128 + 2 * ((q0b >> 4) & 63)) * 4u;
    const uint32_t push_b_mbar = rb == 0 ? full_of[0] : rb == 1 ? full_of[1] : rb == 2 ? full_of[2] : full_of[3];

    if (tid == 0) {
        for (int s = 0; s < NBUF * NBLK; ++s) mbar_init(mbar_full + 8u * s, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    uint32_t full_phase = 0;       // bit (b * NBLK + k) = parity to wait for on full[b][k]
    int ib = 0;
    float defect = 0.f, zgap = 0.f;
    auto wait_inputs = [&](int b, int k) {
        const int s = b * NBLK + k;
        pr.wait(mbar_full + 8u * s, (full_phase >> s) & 1u);
        full_phase ^= 1u << s;
    };

    for (int64_t base = (int64_t)cid * NBLK; base < p.B; base += (int64_t)ncl * NBLK) {
        const int nact = (int)(p.B - base < NBLK ? p.B - base : NBLK);        // blocks in flight in this batch
        for (int k = 0; k < nact; ++k) {
            const float *w = p.W + (base + k) * n;
            for (int t = tid; t < n; t += CT) w_s[k * C::MAX_N + t] = __ldg(w + t);
            for (int q = tid; q < QC; q += CT) msg[(ib * NBLK + k) * QC + q] = 0.f;      // L_1 = 0
            if (tid == 0) O_s[k * OSTR + 1] = 0;
        }
        vec4_stage_table(tm, p.cb, q0);
        int O[NBLK];
        float off[NBLK], cmax[NBLK];
#pragma unroll
        for (int k = 0; k < NBLK; ++k) { O[k] = 0; off[k] = 0.f; cmax[k] = 0.f; }
        cluster_sync();
        // ================= alpha sweep: step t maps L_t to L_{t+1}
        for (int t = 1; t <= nt; ++t) {
            const int ob = ib == NBUF - 1 ? 0 : ib + 1;
#pragma unroll
            for (int k = 0; k < NBLK; ++k) {
                if (k < nact) {
                    const int si = ib * NBLK + k, so = ob * NBLK + k;
                    // the first table unit and the step's weights do not depend on the step's inputs: requested before the wait
                    float2 a[K], cb[2][8];
                    tmem_ld16(tm, cb[0]);
                    const float *wk = w_s + k * C::MAX_N + 2 * (t - 1);
                    const float2 wx = splat2(wk[0]), wy = splat2(wk[1]);
                    if (t > 1) {
                        wait_inputs(ib, k);
                        cmax[k] = warp_max(slot_max(wmax + si * 64, lane, SLOTS)) - off[k];
                        off[k] = rintf(cmax[k]);
                    }
                    const float *Lin = msg + si * QC + (tid >> 3);            // [j][x], x = (q0 >> 4) & 63
                    if (tid == 0) pr.expect_tx(mbar_full + 8u * so, TX_MSG);
#pragma unroll
                    for (int u = 0; u < C::UNITS; ++u) {
                        tmem_wait_ld(cb[u & 1]);
                        if (u + 1 < C::UNITS) tmem_ld16(tm + 16u * (u + 1), cb[(u + 1) & 1]);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int j = 4 * u + e;
                            const float2 dx = sub2(cb[u & 1][2 * e], wx), dy = sub2(cb[u & 1][2 * e + 1], wy);
                            a[j] = fma2(fma2(dy, dy, mul2(dx, dx)), nl2, splat2(Lin[64 * j]));
                        }
                    }
                    const float2 m = max_pairs<K>(a);
                    float2 sum = ex2f2(sub2(a[0], m));
#pragma unroll
                    for (int j = 1; j < K; ++j) sum = add2(sum, ex2f2(sub2(a[j], m)));
                    const float2 out = add2(sub2(m, splat2(off[k])), lg2f2(sum));
                    pr.async_v2(push_a + (uint32_t)(so * QC) * 4u, out.x, out.y, push_a_mbar + 8u * so);
                    if (t < nt) *reinterpret_cast<float2 *>(hist + ((size_t)k * nt + t) * Q + q0) = out;
                    const float tmax = warp_max(fmaxf(m.x, m.y));
                    if (lane == 0) {
#pragma unroll
                        for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(so * 64) * 4u, tmax, full_of[r] + 8u * so);
                    }
                    O[k] += (int)off[k];
                    if (tid == 0) O_s[k * OSTR + t + 1] = O[k];
                }
            }
            ib = ob;
        }
        // ================= log2 Z = O_{nt+1} + LSE_q L_{nt+1}(q), each CTA sums the quarter it holds
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            if (k < nact) {
                const int si = ib * NBLK + k;
                wait_inputs(ib, k);
                cmax[k] = warp_max(slot_max(wmax + si * 64, lane, SLOTS)) - off[k];
                const float *Lfin = msg + si * QC;
                float ssum = 0.f;
                for (int e = tid; e < QC; e += CT) ssum += ex2f(Lfin[e] - cmax[k]);
                ssum = warp_sum(ssum);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r] + (uint32_t)(k * 64) * 4u, ssum);
                }
            }
        }
        cluster_sync();
        float lsefin[NBLK];
        int Ofin[NBLK];
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            lsefin[k] = 0.f; Ofin[k] = O[k];
            if (k < nact) {
                float v = (lane < SLOTS ? lz[k * 64 + lane] : 0.f) + (lane + 32 < SLOTS ? lz[k * 64 + lane + 32] : 0.f);
                v = warp_sum(v);
                lsefin[k] = cmax[k] + lg2f(v);
                if (tid == 0) diag_check_finite(p.diag, lsefin[k]);
                if (tid == 0 && rank == 0 && p.logZ)
                    p.logZ[base + k] = (float)(((double)Ofin[k] + (double)lsefin[k]) * 0.6931471805599453);
            }
        }
        // ================= beta sweep: step t maps M_t to M_{t-1}
        for (int k = 0; k < nact; ++k)
            for (int q = tid; q < QC; q += CT) msg[(ib * NBLK + k) * QC + q] = 0.f;      // M_nt = 0
        vec4_stage_table(tm, p.cb_beta, q0b);
        int P[NBLK];
        float offM[NBLK];
        float2 Ls[NBLK];
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            P[k] = 0; offM[k] = 0.f;
            Ls[k] = (k < nact && nt > 1) ? __ldcg(reinterpret_cast<const float2 *>(hist + ((size_t)k * nt + nt - 1) * Q + q0b))
                                          : make_float2(0.f, 0.f);
        }
        cluster_sync();
        // rank 0, warp k: turn the sums of step t of block k (slots of buffer b) into soft[t]
        auto finish_step = [&](int t, int b, int k) {
            if (rank == 0 && warp == k) {
                const float *pp = part + (size_t)((b * NBLK + k) * 64) * 4;
                float4 s4 = *reinterpret_cast<const float4 *>(pp + lane * 4);
                const float4 o = *reinterpret_cast<const float4 *>(pp + (lane + 32) * 4);
                const float den = warp_sum(s4.x + o.x), n0 = warp_sum(s4.y + o.y), n1 = warp_sum(s4.z + o.z);
                if (lane == 0) {
                    const float s0 = n0 / den, s1 = n1 / den;
                    *reinterpret_cast<float2 *>(p.soft + (base + k) * n + 2 * (t - 1)) = make_float2(s0, s1);
                    if (p.soft_copy) *reinterpret_cast<float2 *>(p.soft_copy + (base + k) * n + 2 * (t - 1)) = make_float2(s0, s1);
                    defect = fmaxf(defect, fabsf(den - 1.f));
                }
            }
        };
        for (int t = nt; t >= 1; --t) {
            const int ob = ib == NBUF - 1 ? 0 : ib + 1;
#pragma unroll
            for (int k = 0; k < NBLK; ++k) {
                if (k < nact) {
                    const int si = ib * NBLK + k, so = ob * NBLK + k;
                    float2 u[K], cb[2][8];
                    tmem_ld16(tm, cb[0]);                                     // requested before the wait for the step's inputs
                    if (t < nt) {
                        wait_inputs(ib, k);
                        cmax[k] = warp_max(slot_max(wmax + si * 64, lane, SLOTS));
                        P[k] += (int)offM[k];
                        offM[k] = rintf(cmax[k]);
                        finish_step(t + 1, ib, k);
                    }
                    const float *Min = msg + si * QC + 4 * lane;              // [b >> 1][x][b & 1], x = 2 lane, 2 lane + 1
                    if (tid == 0) pr.expect_tx(mbar_full + 8u * so, rank == 0 ? TX_MSG + TX_PART : TX_MSG);
                    // history of the next step, one step ahead (row t - 2 = L_{t-1}; L_1 = 0)
                    const float2 Ls_next = t > 2 ? __ldcg(reinterpret_cast<const float2 *>(hist + ((size_t)k * nt + t - 2) * Q + q0b))
                                                 : make_float2(0.f, 0.f);
                    const float *wk = w_s + k * C::MAX_N + 2 * (t - 1);
                    const float2 wx = splat2(wk[0]), wy = splat2(wk[1]);
                    // the outputs are shifted by offM (once per group, below); D refers to the unshifted inputs
                    const float Dm = ((float)(Ofin[k] - O_s[k * OSTR + t] - P[k]) + lsefin[k]);
                    const float2 offM2 = splat2(offM[k]);
#pragma unroll
                    for (int un = 0; un < C::UNITS; ++un) {
                        tmem_wait_ld(cb[un & 1]);
                        tmem_ld16(tm + 16u * ((un + 1) % C::UNITS), cb[(un + 1) & 1]);       // wraps round for the second pass
#pragma unroll
                        for (int e = 0; e < 4; e += 2) {
                            const int b = 4 * un + e;
                            const float4 Mv = *reinterpret_cast<const float4 *>(Min + 128 * (b >> 1));   // M(x,b), M(x,b+1), M(x+1,b), M(x+1,b+1)
#pragma unroll
                            for (int bb = 0; bb < 2; ++bb) {
                                const float2 dx = sub2(cb[un & 1][2 * (e + bb)], wx), dy = sub2(cb[un & 1][2 * (e + bb) + 1], wy);
                                const float2 Mb = bb == 0 ? make_float2(Mv.x, Mv.z) : make_float2(Mv.y, Mv.w);
                                u[b + bb] = fma2(fma2(dy, dy, mul2(dx, dx)), nl2, Mb);
                            }
                        }
                    }
                    const float2 m = max_pairs<K>(u);
                    float2 sum = make_float2(0.f, 0.f), cx = sum, cy = sum;
#pragma unroll
                    for (int un = 0; un < C::UNITS; ++un) {                                  // second pass over the table slice
                        tmem_wait_ld(cb[un & 1]);
                        if (un + 1 < C::UNITS) tmem_ld16(tm + 16u * (un + 1), cb[(un + 1) & 1]);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float2 pb = ex2f2(sub2(u[4 * un + e], m));
                            sum = add2(sum, pb);
                            cx = fma2(pb, cb[un & 1][2 * e], cx);
                            cy = fma2(pb, cb[un & 1][2 * e + 1], cy);
                        }
                    }
                    const float2 out = add2(sub2(m, offM2), lg2f2(sum));
                    const float2 f = ex2f2(add2(m, sub2(Ls[k], splat2(Dm))));
                    pr.async_v2(push_b + (uint32_t)(so * QC) * 4u, out.x, out.y, push_b_mbar + 8u * so);
                    const float2 fd = mul2(f, sum), fx = mul2(f, cx), fy = mul2(f, cy);
                    const float den = warp_sum(fd.x + fd.y), n0 = warp_sum(fx.x + fx.y), n1 = warp_sum(fy.x + fy.y);
                    const float tmax = warp_max(fmaxf(m.x, m.y)) - offM[k];
                    if (lane == 0) {
#pragma unroll
                        for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(so * 64) * 4u, tmax, full_of[r] + 8u * so);
                        pr.async_v4(part_dst + (uint32_t)(so * 256) * 4u, den, n0, n1, 0.f, full_of[0] + 8u * so);
                    }
                    Ls[k] = Ls_next;
                }
            }
            ib = ob;
        }
        // ================= M_0, the sums of step 1, and the consistency check P_0 + LSE_q M_0(q) = log2 Z
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            if (k < nact) {
                const int si = ib * NBLK + k;
                wait_inputs(ib, k);
                cmax[k] = warp_max(slot_max(wmax + si * 64, lane, SLOTS));
                P[k] += (int)offM[k];
                finish_step(1, ib, k);
                const float *Mfin = msg + si * QC;
                float ssum = 0.f;
                for (int e = tid; e < QC; e += CT) ssum += ex2f(Mfin[e] - cmax[k]);
                ssum = warp_sum(ssum);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r] + (uint32_t)((NBLK + k) * 64) * 4u, ssum);
                }
            }
        }
        cluster_sync();
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            if (k < nact) {
                float v = (lane < SLOTS ? lz[(NBLK + k) * 64 + lane] : 0.f) + (lane + 32 < SLOTS ? lz[(NBLK + k) * 64 + lane + 32] : 0.f);
                v = warp_sum(v);
                const float lz_beta = cmax[k] + lg2f(v);
                zgap = fmaxf(zgap, fabsf((float)(P[k] - Ofin[k]) + (lz_beta - lsefin[k])));
            }
        }
        cluster_sync();         // nobody still reads this batch's buffers when the next batch starts
    }
    // defect lives in warps 0..NBLK-1 of rank 0, zgap everywhere
    if (rank == 0 && lane == 0 && warp < NBLK) diag_max(&p.diag->max_defect, defect);
    if (tid == 0 && rank == 0) diag_max(&p.diag->max_logz_gap, zgap);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync();             // no CTA leaves while a peer may still address its shared memory
    if (*abort_flag) settle_after_abort();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

// --------------------------------------------------------------------------------------
// Backward call on the same clusters.  Every message carries a second value, the conditional
// expectation of the centred emitted sum (first-order expectation semiring; the recursions are
// those of bwd_vec_kernel).  Per thread the tensor memory holds the table slice (64 columns) and,
// next to it, the gradient accumulators of the thread's beta-sweep states (64 columns, same
// layout), kept over all steps and all blocks and written once to this cluster's partial sum.
//   h_t(s) = sum_v g[V t + v] (c[s][v] - soft[V t + v]); the constant -g.soft of the consumer's
//   step is added by the producer of At / Bt, so a consumer forms g.c + (carried value) only.
//   z_v(s) = gamma_t(s) (g_v + (w_v - c[s][v]) r_t(s) / T)  is the accumulator increment;
//   grad_W[V t + v] = g_v - (sum_s z_v) / S0 + (S2 / S0) (w_v - soft_v) / T,  S0 = sum gamma, S2 = sum gamma r.
// --------------------------------------------------------------------------------------
template <int NBLK_>
struct Vec4BwdCfg {
    using F = Vec4Cfg<NBLK_>;
    static constexpr int Q = F::Q, QC = F::QC, CL = F::CL, THREADS = F::THREADS, NWARP = F::NWARP, SLOTS = F::SLOTS, K = F::K;
    static constexpr int NBUF = 3, NBLK = NBLK_, UNITS = 4;
    static constexpr int MAX_N = 1024, MAX_NT = MAX_N / 2;
    static constexpr int OFF_MSG = 0;                                  // [NBUF][NBLK][2][QC]: (L, At) or (M, Bt)
    static constexpr int OFF_W = OFF_MSG + NBUF * NBLK * 2 * QC;       // [NBLK][3][MAX_N]: w, g, soft
    static constexpr int OFF_O = OFF_W + NBLK * 3 * MAX_N;             // int [NBLK][MAX_NT + 4]
    static constexpr int OFF_WMAX = OFF_O + NBLK * (MAX_NT + 4);       // [NBUF][NBLK][64]
    static constexpr int OFF_PART = OFF_WMAX + NBUF * NBLK * 64;       // [NBUF][NBLK][64][4]: S0, S2, ZS_0, ZS_1
    static constexpr int OFF_LZ = OFF_PART + NBUF * NBLK * 64 * 4;     // [NBLK][64]
    static constexpr int OFF_MBAR = OFF_LZ + NBLK * 64;                // uint64 [NBUF][NBLK]
    static constexpr int OFF_TMEM = OFF_MBAR + 2 * NBUF * NBLK + 2;
    static constexpr int OFF_FLAG = OFF_TMEM + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(OFF_MBAR % 2 == 0 && OFF_MSG % 4 == 0 && OFF_PART % 4 == 0, "alignment");
    static_assert(SMEM_BYTES <= 232448, "shared memory of one CTA");
    static_assert(NBLK <= NWARP && NBUF * NBLK <= 32, "one finishing warp per block in flight; phase bits");
};

template <int NBLK_>
__global__ void __launch_bounds__(Vec4BwdCfg<NBLK_>::THREADS, 1) bwd_vec4_kernel(BwdParams p)
{
    using C = Vec4BwdCfg<NBLK_>;
    constexpr int K = C::K, Q = C::Q, QC = C::QC, CL = C::CL, NWARP = C::NWARP, NBUF = C::NBUF, SLOTS = C::SLOTS, CT = C::THREADS;
    constexpr int NBLK = C::NBLK, OSTR = C::MAX_NT + 4, UNITS = C::UNITS, MAXN = C::MAX_N;
    constexpr uint32_t TX_MSG = 2u * QC * 4u + SLOTS * 4u;       // a quarter of both message arrays + gauge slots
    constexpr uint32_t TX_PART = SLOTS * 16u;                    // posterior sums (rank 0 only)
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t rank = cluster_ctarank();
    const uint32_t cid = cluster_id_x(), ncl = cluster_count_x();
    const int n = p.n, nt = n / 2;
    const float2 nl2 = splat2(-p.lam2);
    const float invT = p.invT;

    float *msg = smem + C::OFF_MSG;
    float *w_s = smem + C::OFF_W;
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAG);
    Proto pr{1u, abort_flag, p.diag};
    const uint32_t mbar_full = smem_u32(smem + C::OFF_MBAR);
    const uint32_t msg_u32 = smem_u32(msg), wmax_u32 = smem_u32(wmax), part_u32 = smem_u32(part), lz_u32 = smem_u32(lz);

    const int q0 = (int)rank * QC + 2 * tid;                     // alpha sweep: groups q0, q0 + 1
    const int q0b = warp * 256 + (int)rank * 64 + 2 * lane;      // beta sweep: groups q0b, q0b + 1
    float *histL = p.hist + (size_t)cid * NBLK * 2 * nt * Q;     // [NBLK][nt][Q]: row t = L_{t+1}
    float *histA = histL + (size_t)NBLK * nt * Q;                // same shape: At_{t+1} (with the consumer's shift)

    uint32_t full_of[CL], msg_of[CL], wmax_dst[CL], lz_dst[CL];
#pragma unroll
    for (int r = 0; r < CL; ++r) {
        full_of[r] = mapa_u32(mbar_full, (uint32_t)r);
        msg_of[r] = mapa_u32(msg_u32, (uint32_t)r);
        wmax_dst[r] = mapa_u32(wmax_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
        lz_dst[r] = mapa_u32(lz_u32 + (uint32_t)((int)rank * NWARP + warp) * 4u, (uint32_t)r);
    }
    const uint32_t part_dst = mapa_u32(part_u32 + (uint32_t)((int)rank * NWARP + warp) * 16u, 0u);
    const int ra = (q0 & 255) >> 6;
    const uint32_t push_a = (ra == 0 ? msg_of[0] : ra == 1 ? msg_of[1] : ra == 2 ? msg_of[2] : msg_of[3])
                            + (uint32_t)((q0 >> 8) * 64 + (q0 & 63)) * 4u;
    const uint32_t push_a_mbar = ra == 0 ? full_of[0] : ra == 1 ? full_of[1] : ra == 2 ? full_of[2] : full_of[3];
    const int rb = warp >> 2;
    const uint32_t push_b = (rb == 0 ? msg_of[0] : rb == 1 ? msg_of[1] : rb == 2 ? msg_of[2] : msg_of[3])
                            + (uint32_t)(((q0b & 15) >> 1) * 128 + 2 * ((q0b >> 4) & 63)) * 4u;
    const uint32_t push_b_mbar = rb == 0 ? full_of[0] : rb == 1 ? full_of[1] : rb == 2 ? full_of[2] : full_of[3];

    if (tid == 0) {
        for (int s = 0; s < NBUF * NBLK; ++s) mbar_init(mbar_full + 8u * s, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    const uint32_t tm_acc = tm + 64u;
    {
        float2 z[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) z[e] = make_float2(0.f, 0.f);
#pragma unroll
        for (int u = 0; u < UNITS; ++u) tmem_st16(tm_acc + 16u * u, z);
        tmem_wait_st();
    }
    uint32_t full_phase = 0;
    int ib = 0;
    float defect = 0.f;
    auto wait_inputs = [&](int b, int k) {
        const int s = b * NBLK + k;
        pr.wait(mbar_full + 8u * s, (full_phase >> s) & 1u);
        full_phase ^= 1u << s;
    };

    for (int64_t base = (int64_t)cid * NBLK; base < p.B; base += (int64_t)ncl * NBLK) {
        const int nact = (int)(p.B - base < NBLK ? p.B - base : NBLK);
        for (int k = 0; k < nact; ++k) {
            const float *w = p.W + (base + k) * n, *g = p.g + (base + k) * n, *sf = p.soft + (base + k) * n;
            float *wk = w_s + k * 3 * MAXN;
            for (int t = tid; t < n; t += CT) { wk[t] = __ldg(w + t); wk[MAXN + t] = __ldg(g + t); wk[2 * MAXN + t] = __ldg(sf + t); }
            if (tid == 0) O_s[k * OSTR + 1] = 0;
        }
        __syncthreads();
        for (int k = 0; k < nact; ++k) {
            // L_1 = 0; the At array carries At + (shift of the consumer's step): At_1 = 0, shift -g_1.soft_1
            const float *wk = w_s + k * 3 * MAXN;
            const float gs1 = -(wk[MAXN] * wk[2 * MAXN] + wk[MAXN + 1] * wk[2 * MAXN + 1]);
            float *m0 = msg + (size_t)(ib * NBLK + k) * 2 * QC;
            for (int q = tid; q < QC; q += CT) { m0[q] = 0.f; m0[QC + q] = gs1; }
        }
        vec4_stage_table(tm, p.cb, q0);
        int O[NBLK];
        float off[NBLK], cmax[NBLK];
#pragma unroll
        for (int k = 0; k < NBLK; ++k) { O[k] = 0; off[k] = 0.f; cmax[k] = 0.f; }
        cluster_sync();
        // ================= alpha sweep carrying (L, At)
        for (int t = 1; t <= nt; ++t) {
            const int ob = ib == NBUF - 1 ? 0 : ib + 1;
#pragma unroll
            for (int k = 0; k < NBLK; ++k) {
                if (k < nact) {
                    const int si = ib * NBLK + k, so = ob * NBLK + k;
                    if (t > 1) {
                        wait_inputs(ib, k);
                        cmax[k] = warp_max(slot_max(wmax + si * 64, lane, SLOTS)) - off[k];
                        off[k] = rintf(cmax[k]);
                    }
                    const float *Lin = msg + (size_t)si * 2 * QC + (tid >> 3), *Ain = Lin + QC;
                    if (tid == 0) pr.expect_tx(mbar_full + 8u * so, TX_MSG);
                    const float *wk = w_s + k * 3 * MAXN + 2 * (t - 1);
                    const float2 wx = splat2(wk[0]), wy = splat2(wk[1]);
                    const float2 gx = splat2(wk[MAXN]), gy = splat2(wk[MAXN + 1]);
                    // shift for the consumers of this step's At (step t + 1); unused at t = nt
                    const float gsn = t < nt ? -(wk[MAXN + 2] * wk[2 * MAXN + 2] + wk[MAXN + 3] * wk[2 * MAXN + 3]) : 0.f;
                    float2 a[K], x[K], cb[2][8];
                    tmem_ld16(tm, cb[0]);
#pragma unroll
                    for (int u = 0; u < UNITS; ++u) {
                        tmem_wait_ld(cb[u & 1]);
                        if (u + 1 < UNITS) tmem_ld16(tm + 16u * (u + 1), cb[(u + 1) & 1]);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int j = 4 * u + e;
                            const float2 cx = cb[u & 1][2 * e], cy = cb[u & 1][2 * e + 1];
                            const float2 dx = sub2(cx, wx), dy = sub2(cy, wy);
                            a[j] = fma2(fma2(dy, dy, mul2(dx, dx)), nl2, splat2(Lin[64 * j]));
                            x[j] = fma2(gx, cx, fma2(gy, cy, splat2(Ain[64 * j])));      // g.c + (At - g.soft)
                        }
                    }
                    const float2 m = max_pairs<K>(a);
                    float2 sum = make_float2(0.f, 0.f), ax = sum;
#pragma unroll
                    for (int j = 0; j < K; ++j) {
                        const float2 pj = ex2f2(sub2(a[j], m));
                        sum = add2(sum, pj);
                        ax = fma2(pj, x[j], ax);
                    }
                    const float2 outL = add2(sub2(m, splat2(off[k])), lg2f2(sum));
                    const float2 outA = fma2(ax, rcpf2(sum), splat2(gsn));
                    pr.async_v2(push_a + (uint32_t)(so * 2 * QC) * 4u, outL.x, outL.y, push_a_mbar + 8u * so);
                    pr.async_v2(push_a + (uint32_t)(so * 2 * QC + QC) * 4u, outA.x, outA.y, push_a_mbar + 8u * so);
                    if (t < nt) {
                        *reinterpret_cast<float2 *>(histL + ((size_t)k * nt + t) * Q + q0) = outL;
                        *reinterpret_cast<float2 *>(histA + ((size_t)k * nt + t) * Q + q0) = outA;
                    }
                    const float tmax = warp_max(fmaxf(m.x, m.y));
                    if (lane == 0) {
#pragma unroll
                        for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(so * 64) * 4u, tmax, full_of[r] + 8u * so);
                    }
                    O[k] += (int)off[k];
                    if (tid == 0) O_s[k * OSTR + t + 1] = O[k];
                }
            }
            ib = ob;
        }
        // ================= log2 Z
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            if (k < nact) {
                const int si = ib * NBLK + k;
                wait_inputs(ib, k);
                cmax[k] = warp_max(slot_max(wmax + si * 64, lane, SLOTS)) - off[k];
                const float *Lfin = msg + (size_t)si * 2 * QC;
                float ssum = 0.f;
                for (int e = tid; e < QC; e += CT) ssum += ex2f(Lfin[e] - cmax[k]);
                ssum = warp_sum(ssum);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r] + (uint32_t)(k * 64) * 4u, ssum);
                }
            }
        }
        cluster_sync();
        float lsefin[NBLK];
        int Ofin[NBLK];
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            lsefin[k] = 0.f; Ofin[k] = O[k];
            if (k < nact) {
                float v = (lane < SLOTS ? lz[k * 64 + lane] : 0.f) + (lane + 32 < SLOTS ? lz[k * 64 + lane + 32] : 0.f);
                v = warp_sum(v);
                lsefin[k] = cmax[k] + lg2f(v);
                if (tid == 0) diag_check_finite(p.diag, lsefin[k]);
            }
        }
        // ================= beta sweep carrying (M, Bt), with the gradient contraction
        for (int k = 0; k < nact; ++k) {
            // M_nt = 0, Bt_nt = 0 (+ the shift of step nt)
            const float *wk = w_s + k * 3 * MAXN;
            const float gsl = -(wk[MAXN + n - 2] * wk[2 * MAXN + n - 2] + wk[MAXN + n - 1] * wk[2 * MAXN + n - 1]);
            float *m0 = msg + (size_t)(ib * NBLK + k) * 2 * QC;
            for (int q = tid; q < QC; q += CT) { m0[q] = 0.f; m0[QC + q] = gsl; }
        }
        vec4_stage_table(tm, p.cb_beta, q0b);
        int P[NBLK];
        float offM[NBLK];
        float2 Ls[NBLK], As[NBLK];
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            P[k] = 0; offM[k] = 0.f;
            const bool have = k < nact && nt > 1;
            Ls[k] = have ? __ldcg(reinterpret_cast<const float2 *>(histL + ((size_t)k * nt + nt - 1) * Q + q0b)) : make_float2(0.f, 0.f);
            // At_1 = 0 carries the shift of step 1 like every other row
            As[k] = have ? __ldcg(reinterpret_cast<const float2 *>(histA + ((size_t)k * nt + nt - 1) * Q + q0b))
                         : splat2(k < nact ? -(w_s[k * 3 * MAXN + MAXN] * w_s[k * 3 * MAXN + 2 * MAXN] + w_s[k * 3 * MAXN + MAXN + 1] * w_s[k * 3 * MAXN + 2 * MAXN + 1]) : 0.f);
        }
        cluster_sync();
        // rank 0, warp k: turn the sums of step t of block k (slots of buffer b) into grad_W of that step
        auto finish_step = [&](int t, int b, int k) {
            if (rank == 0 && warp == k) {
                const float *pp = part + (size_t)((b * NBLK + k) * 64) * 4;
                const float4 s4 = *reinterpret_cast<const float4 *>(pp + lane * 4);
                const float4 o = *reinterpret_cast<const float4 *>(pp + (lane + 32) * 4);
                const float v4 = warp_sum4_split(s4.x + o.x, s4.y + o.y, s4.z + o.z, s4.w + o.w, lane);
                const float a0 = __shfl_sync(0xffffffffu, v4, 0), a2 = __shfl_sync(0xffffffffu, v4, 8);
                const float z0 = __shfl_sync(0xffffffffu, v4, 16), z1 = __shfl_sync(0xffffffffu, v4, 24);
                if (lane == 0) {
                    const float *wk = w_s + k * 3 * MAXN + 2 * (t - 1);
                    const float i0 = 1.f / a0;
                    const float gw0 = (wk[MAXN] - z0 * i0) + (a2 * i0) * (wk[0] - wk[2 * MAXN]) * invT;
                    const float gw1 = (wk[MAXN + 1] - z1 * i0) + (a2 * i0) * (wk[1] - wk[2 * MAXN + 1]) * invT;
                    *reinterpret_cast<float2 *>(p.gW + (base + k) * n + 2 * (t - 1)) = make_float2(gw0, gw1);
                    defect = fmaxf(defect, fabsf(a0 - 1.f));
                }
            }
        };
        for (int t = nt; t >= 1; --t) {
            const int ob = ib == NBUF - 1 ? 0 : ib + 1;
#pragma unroll
            for (int k = 0; k < NBLK; ++k) {
                if (k < nact) {
                    const int si = ib * NBLK + k, so = ob * NBLK + k;
                    if (t < nt) {
                        wait_inputs(ib, k);
                        cmax[k] = warp_max(slot_max(wmax + si * 64, lane, SLOTS));
                        P[k] += (int)offM[k];
                        offM[k] = rintf(cmax[k]);
                        finish_step(t + 1, ib, k);
                    }
                    const float *Min = msg + (size_t)si * 2 * QC + 4 * lane, *Bin = Min + QC;
                    if (tid == 0) pr.expect_tx(mbar_full + 8u * so, rank == 0 ? TX_MSG + TX_PART : TX_MSG);
                    const float *wk = w_s + k * 3 * MAXN + 2 * (t - 1);
                    const float2 wx = splat2(wk[0]), wy = splat2(wk[1]);
                    const float2 gx = splat2(wk[MAXN]), gy = splat2(wk[MAXN + 1]);
                    const float gs = -(wk[MAXN] * wk[2 * MAXN] + wk[MAXN + 1] * wk[2 * MAXN + 1]);              // shift carried by the stored At
                    const float gsp = t > 1 ? -(wk[MAXN - 2] * wk[2 * MAXN - 2] + wk[MAXN - 1] * wk[2 * MAXN - 1]) : 0.f;   // for step t - 1
                    float2 Ls_next = make_float2(0.f, 0.f), As_next = Ls_next;
                    if (t > 2) {
                        Ls_next = __ldcg(reinterpret_cast<const float2 *>(histL + ((size_t)k * nt + t - 2) * Q + q0b));
                        As_next = __ldcg(reinterpret_cast<const float2 *>(histA + ((size_t)k * nt + t - 2) * Q + q0b));
                    } else if (t == 2) {
                        As_next = splat2(-(wk[MAXN - 2] * wk[2 * MAXN - 2] + wk[MAXN - 1] * wk[2 * MAXN - 1]));          // At_1 = 0 + shift of step 1
                    }
                    const float Dm = ((float)(Ofin[k] - O_s[k * OSTR + t] - P[k]) + lsefin[k]);
                    const float2 offM2 = splat2(offM[k]);
                    float2 u[K], cb[8];
#pragma unroll
                    for (int un = 0; un < UNITS; ++un) {
                        tmem_ld16(tm + 16u * un, cb);
                        tmem_wait_ld(cb);
#pragma unroll
                        for (int e = 0; e < 4; e += 2) {
                            const int b = 4 * un + e;
                            const float4 Mv = *reinterpret_cast<const float4 *>(Min + 128 * (b >> 1));
#pragma unroll
                            for (int bb = 0; bb < 2; ++bb) {
                                const float2 dx = sub2(cb[2 * (e + bb)], wx), dy = sub2(cb[2 * (e + bb) + 1], wy);
                                const float2 Mb = bb == 0 ? make_float2(Mv.x, Mv.z) : make_float2(Mv.y, Mv.w);
                                u[b + bb] = fma2(fma2(dy, dy, mul2(dx, dx)), nl2, Mb);
                            }
                        }
                    }
                    const float2 m = max_pairs<K>(u);
                    const float2 f = ex2f2(add2(m, sub2(Ls[k], splat2(Dm))));
                    const float2 iT2 = splat2(invT);
                    const float2 Ahj = sub2(As[k], splat2(gs));                        // At_t without the shift
                    float2 sum = make_float2(0.f, 0.f), ya = sum, Z0 = sum, Z1 = sum;
#pragma unroll
                    for (int un = 0; un < UNITS; ++un) {                                   // second pass, with the accumulators
                        float2 acc[8];
                        tmem_ld16(tm + 16u * un, cb);
                        tmem_ld16(tm_acc + 16u * un, acc);
                        tmem_wait_ld(cb);
                        tmem_wait_ld(acc);
#pragma unroll
                        for (int e = 0; e < 4; e += 2) {
                            const int b = 4 * un + e;
                            const float4 Bv = *reinterpret_cast<const float4 *>(Bin + 128 * (b >> 1));
#pragma unroll
                            for (int bb = 0; bb < 2; ++bb) {
                                const float2 cx = cb[2 * (e + bb)], cy = cb[2 * (e + bb) + 1];
                                const float2 Bb = bb == 0 ? make_float2(Bv.x, Bv.z) : make_float2(Bv.y, Bv.w);
                                const float2 y = fma2(gx, cx, fma2(gy, cy, Bb));             // g.c + (Bt - g.soft) = h + Bt
                                const float2 pb = ex2f2(sub2(u[b + bb], m));
                                sum = add2(sum, pb);
                                ya = fma2(pb, y, ya);
                                const float2 rT = mul2(add2(y, Ahj), iT2);                 // r / T
                                const float2 gam = mul2(pb, f);                            // gamma
                                const float2 ix = fma2(rT, sub2(wx, cx), gx), iy = fma2(rT, sub2(wy, cy), gy);   // g_v + (w_v - c_v) r / T
                                Z0 = fma2(gam, ix, Z0); Z1 = fma2(gam, iy, Z1);                                  // z_v = gamma (g_v + (w_v - c_v) r / T)
                                acc[2 * (e + bb)] = fma2(gam, ix, acc[2 * (e + bb)]);
                                acc[2 * (e + bb) + 1] = fma2(gam, iy, acc[2 * (e + bb) + 1]);
                            }
                        }
                        tmem_st16(tm_acc + 16u * un, acc);
                    }
                    tmem_wait_st();
                    // S0 = sum gamma = f sum rho;  S2 = sum gamma r = f (sum rho y + At sum rho)
                    const float2 S0 = mul2(f, sum), S2 = mul2(f, fma2(Ahj, sum, ya));
                    const float2 outM = add2(sub2(m, offM2), lg2f2(sum));
                    const float2 outB = fma2(ya, rcpf2(sum), splat2(gsp));
                    pr.async_v2(push_b + (uint32_t)(so * 2 * QC) * 4u, outM.x, outM.y, push_b_mbar + 8u * so);
                    pr.async_v2(push_b + (uint32_t)(so * 2 * QC + QC) * 4u, outB.x, outB.y, push_b_mbar + 8u * so);
                    const float v4 = warp_sum4_split(S0.x + S0.y, S2.x + S2.y, Z0.x + Z0.y, Z1.x + Z1.y, lane);   // lanes 0, 8, 16, 24
                    const float tmax = warp_max(fmaxf(m.x, m.y)) - offM[k];
                    if (lane == 0) {
#pragma unroll
                        for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(so * 64) * 4u, tmax, full_of[r] + 8u * so);
                    }
                    if ((lane & 7) == 0)
                        pr.async_f32(part_dst + (uint32_t)(so * 256 + (lane >> 3)) * 4u, v4, full_of[0] + 8u * so);
                    Ls[k] = Ls_next; As[k] = As_next;
                }
            }
            ib = ob;
        }
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            if (k < nact) {
                wait_inputs(ib, k);                                          // the sums of step 1
                finish_step(1, ib, k);
            }
        }
        cluster_sync();         // nobody still reads this batch's buffers when the next batch starts
    }
    // this cluster's partial of the table gradient, in the regrouped layout [b][q][V]
    {
        float *gc = p.gc_part + (size_t)cid * C::F::S * 2;
#pragma unroll
        for (int un = 0; un < UNITS; ++un) {
            float2 acc[8];
            tmem_ld16(tm_acc + 16u * un, acc);
            tmem_wait_ld(acc);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int b = 4 * un + e;
                *reinterpret_cast<float4 *>(gc + ((size_t)b * Q + q0b) * 2) =
                    make_float4(acc[2 * e].x, acc[2 * e + 1].x, acc[2 * e].y, acc[2 * e + 1].y);   // (z0.x, z0.y, z1.x, z1.y)
            }
        }
    }
    if (rank == 0 && lane == 0 && warp < NBLK) diag_max(&p.diag->max_defect, defect);
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    cluster_sync();             // no CTA leaves while a peer may still address its shared memory
    if (*abort_flag) settle_after_abort();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
