// Vector-emission trellis with 16 state bits, 4 bits and V = 2 weights per step: forward call on clusters of
// TWO CTAs.
//
// The table of this trellis is S x V floats = 512 KB, the tensor memory of two SMs.  fwd_vec4_kernel spreads it
// over four (it shares the cluster shape with the backward kernel, which needs the gradient accumulators too), but
// clusters of four fit 33 times on the GPU (132 of 148 SMs) and leave a thread 32 states per step to hide the
// per-step hand-over behind.  The forward call needs the table alone: here two CTAs hold it whole (128 columns per
// thread), 74 clusters fill the GPU, and a thread has 64 states per step -- two packed pairs of groups that share
// their sixteen inputs.
//
// Ownership (Q = 4096 groups, 2048 per CTA, four per thread).
//   alpha:  L_{t+1}(q) = LSE_j [ L_t((q >> 4) + 256 j) + e_t(q + jQ) ]              CTA r owns q >> 11 == r,
//           thread tid the groups q0 .. q0 + 3, q0 = 2048 r + 4 tid (one butterfly x = q0 >> 4, outputs l = q0 & 15 ..),
//           and reads the entries i of L_t with ((i & 255) >> 7) == r, kept as [i >> 8][i & 127];
//   beta :  M_{t-1}(q) = LSE_b [ M_t(((q & 255) << 4) | b) + e_t(16 q + b) ]        CTA r owns ((q & 255) >> 7) == r,
//           thread (xp = lane + 32 (warp & 1), jp = warp >> 1) the groups [j | x] with j in {2 jp, 2 jp + 1} and
//           x in {128 r + 2 xp, + 1} (two butterflies, two outputs each, sharing the inputs M(x, b), M(x + 1, b)),
//           and reads the entries i = (x', b') of M_t with (i >> 11) == r, kept as [b' >> 1][x' & 127][b' & 1].
// Every output has exactly one consumer CTA: one 16-byte st.async per thread and step in the alpha sweep, two
// 8-byte ones in the beta sweep.  Table slice per sweep and pair: the layout of vec4_stage_table, pair p at columns
// 64 p.  Message buffers, gauge slots, posterior sums, history and the blocks-in-flight schedule are those of
// fwd_vec4_kernel.
#pragma once
#include "bcjr_vec4.cuh"

namespace bcjr {

template <int NBLK_>
struct Vec2Cfg {
    static constexpr int LB = 16, KB = 4, V = 2, K = 16, S = 1 << LB, Q = S >> KB;
    static constexpr int CL = 2, THREADS = 512, NWARP = THREADS / 32, QC = Q / CL;
    static constexpr int SLOTS = CL * NWARP;                   // 32 per-warp partial slots
    static constexpr int NBUF = 3;
    static constexpr int NBLK = NBLK_;                         // weight blocks in flight per cluster
    static constexpr int PP = 2;                               // packed pairs of groups per thread
    static constexpr int UNITS = 4;                            // 16-column TMEM units per pair: 4 table entries (x 2 groups x 2 floats) each
    static constexpr int MAX_N = 2048, MAX_NT = MAX_N / V;     // weights / steps per block
    static constexpr int OFF_MSG = 0;                                  // [NBUF][NBLK][QC]
    static constexpr int OFF_W = OFF_MSG + NBUF * NBLK * QC;           // [NBLK][MAX_N]
    static constexpr int OFF_O = OFF_W + NBLK * MAX_N;                 // int [NBLK][MAX_NT + 4]
    static constexpr int OFF_WMAX = OFF_O + NBLK * (MAX_NT + 4);       // [NBUF][NBLK][SLOTS]
    static constexpr int OFF_PART = OFF_WMAX + NBUF * NBLK * SLOTS;    // [NBUF][NBLK][SLOTS][4]: den, num_0, num_1
    static constexpr int OFF_LZ = OFF_PART + NBUF * NBLK * SLOTS * 4;  // [2][NBLK][SLOTS]
    static constexpr int OFF_MBAR = OFF_LZ + 2 * NBLK * SLOTS;         // uint64 [NBUF][NBLK]
    static constexpr int OFF_TMEM = OFF_MBAR + 2 * NBUF * NBLK + 2;
    static constexpr int OFF_FLAG = OFF_TMEM + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(QC == 2 * PP * THREADS, "a thread owns two packed pairs of groups");
    static_assert(SLOTS == 32, "one gauge slot per lane");
    static_assert(OFF_MBAR % 2 == 0 && OFF_MSG % 4 == 0 && OFF_PART % 4 == 0, "alignment");
    static_assert(SMEM_BYTES <= 232448, "shared memory of one CTA");
    static_assert(NBLK <= NWARP && NBUF * NBLK <= 32, "one finishing warp per block in flight; phase bits");
    // index arithmetic of the two sweeps (host-checkable)
    __host__ __device__ static constexpr int alpha_q0(int rank, int tid) { return rank * QC + 4 * tid; }
    __host__ __device__ static constexpr int alpha_in(int tid) { return tid >> 2; }                        // + 128 j: input j of the thread's butterfly
    __host__ __device__ static constexpr int alpha_dst_rank(int q0) { return (q0 & 255) >> 7; }
    __host__ __device__ static constexpr int alpha_dst_off(int q0) { return (q0 >> 8) * 128 + (q0 & 127); }
    __host__ __device__ static constexpr int beta_q0(int rank, int warp, int lane, int p)
    {
        return (2 * (warp >> 1) + p) * 256 + rank * 128 + 2 * (lane + 32 * (warp & 1));
    }
    __host__ __device__ static constexpr int beta_in(int warp, int lane) { return 4 * (lane + 32 * (warp & 1)); }   // + 256 (b >> 1): M(x,b), M(x,b+1), M(x+1,b), M(x+1,b+1)
    __host__ __device__ static constexpr int beta_dst_rank(int q) { return q >> 11; }
    __host__ __device__ static constexpr int beta_dst_off(int q) { return ((q & 15) >> 1) * 256 + 2 * ((q >> 4) & 127) + (q & 1); }
};

template <int NBLK_>
__global__ void __launch_bounds__(Vec2Cfg<NBLK_>::THREADS, 1) fwd_vec2_kernel(FwdParams p)
{
    using C = Vec2Cfg<NBLK_>;
    constexpr int K = C::K, Q = C::Q, QC = C::QC, CL = C::CL, NWARP = C::NWARP, NBUF = C::NBUF, SLOTS = C::SLOTS, CT = C::THREADS;
    constexpr int NBLK = C::NBLK, OSTR = C::MAX_NT + 4, PP = C::PP;
    constexpr uint32_t TX_MSG = QC * 4u + SLOTS * 4u;            // half of the messages + gauge slots
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

    const int q0 = C::alpha_q0((int)rank, tid);                  // alpha sweep: this thread's groups q0 .. q0 + 3
    const int q0b = C::beta_q0((int)rank, warp, lane, 0);        // beta sweep: groups q0b, q0b + 1 and q0b + 256, q0b + 257
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
    const int ra = C::alpha_dst_rank(q0);
    const uint32_t push_a = (ra == 0 ? msg_of[0] : msg_of[1]) + (uint32_t)C::alpha_dst_off(q0) * 4u;
    const uint32_t push_a_mbar = ra == 0 ? full_of[0] : full_of[1];
    const int rb = C::beta_dst_rank(q0b);                        // the same for the thread's second pair
    const uint32_t push_b = (rb == 0 ? msg_of[0] : msg_of[1]) + (uint32_t)C::beta_dst_off(q0b) * 4u;
    constexpr uint32_t PUSH_B_PAIR = (uint32_t)(C::beta_dst_off(256) - C::beta_dst_off(0)) * 4u;   // second pair: j + 1
    const uint32_t push_b_mbar = rb == 0 ? full_of[0] : full_of[1];

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
#pragma unroll
        for (int pp = 0; pp < PP; ++pp) vec4_stage_table(tm + 64u * pp, p.cb, q0 + 2 * pp);
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
                    float2 cb[2][8];
                    tmem_ld16(tm, cb[0]);
                    const float *wk = w_s + k * C::MAX_N + 2 * (t - 1);
                    const float2 wx = splat2(wk[0]), wy = splat2(wk[1]);
                    if (t > 1) {
                        wait_inputs(ib, k);
                        cmax[k] = warp_max(wmax[si * SLOTS + lane]) - off[k];
                        off[k] = rintf(cmax[k]);
                    }
                    const float *Lin = msg + si * QC + C::alpha_in(tid);      // [j][x & 127]
                    if (tid == 0) pr.expect_tx(mbar_full + 8u * so, TX_MSG);
                    float2 out[PP];
                    float tmax = __int_as_float(0xff800000);
#pragma unroll
                    for (int pp = 0; pp < PP; ++pp) {
                        float2 a[K];
#pragma unroll
                        for (int u = 0; u < C::UNITS; ++u) {
                            const int g = pp * C::UNITS + u;
                            tmem_wait_ld(cb[g & 1]);
                            if (g + 1 < PP * C::UNITS) tmem_ld16(tm + 16u * (g + 1), cb[(g + 1) & 1]);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int j = 4 * u + e;
                                const float2 dx = sub2(cb[g & 1][2 * e], wx), dy = sub2(cb[g & 1][2 * e + 1], wy);
                                a[j] = fma2(fma2(dy, dy, mul2(dx, dx)), nl2, splat2(Lin[128 * j]));
                            }
                        }
                        const float2 m = max_pairs<K>(a);
                        float2 sum = ex2f2(sub2(a[0], m));
#pragma unroll
                        for (int j = 1; j < K; ++j) sum = add2(sum, ex2f2(sub2(a[j], m)));
                        out[pp] = add2(sub2(m, splat2(off[k])), lg2f2(sum));
                        tmax = max3f(tmax, m.x, m.y);
                    }
                    pr.async_v4(push_a + (uint32_t)(so * QC) * 4u, out[0].x, out[0].y, out[1].x, out[1].y, push_a_mbar + 8u * so);
                    if (t < nt) *reinterpret_cast<float4 *>(hist + ((size_t)k * nt + t) * Q + q0) = make_float4(out[0].x, out[0].y, out[1].x, out[1].y);
                    tmax = warp_max(tmax);
                    if (lane == 0) {
#pragma unroll
                        for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(so * SLOTS) * 4u, tmax, full_of[r] + 8u * so);
                    }
                    O[k] += (int)off[k];
                    if (tid == 0) O_s[k * OSTR + t + 1] = O[k];
                }
            }
            ib = ob;
        }
        // ================= log2 Z = O_{nt+1} + LSE_q L_{nt+1}(q), each CTA sums the half it holds
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            if (k < nact) {
                const int si = ib * NBLK + k;
                wait_inputs(ib, k);
                cmax[k] = warp_max(wmax[si * SLOTS + lane]) - off[k];
                const float *Lfin = msg + si * QC;
                float ssum = 0.f;
                for (int e = tid; e < QC; e += CT) ssum += ex2f(Lfin[e] - cmax[k]);
                ssum = warp_sum(ssum);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r] + (uint32_t)(k * SLOTS) * 4u, ssum);
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
                const float v = warp_sum(lz[k * SLOTS + lane]);
                lsefin[k] = cmax[k] + lg2f(v);
                if (tid == 0) diag_check_finite(p.diag, lsefin[k]);
                if (tid == 0 && rank == 0 && p.logZ)
                    p.logZ[base + k] = (float)(((double)Ofin[k] + (double)lsefin[k]) * 0.6931471805599453);
            }
        }
        // ================= beta sweep: step t maps M_t to M_{t-1}
        for (int k = 0; k < nact; ++k)
            for (int q = tid; q < QC; q += CT) msg[(ib * NBLK + k) * QC + q] = 0.f;      // M_nt = 0
#pragma unroll
        for (int pp = 0; pp < PP; ++pp) vec4_stage_table(tm + 64u * pp, p.cb_beta, q0b + 256 * pp);
        int P[NBLK];
        float offM[NBLK];
        float2 Ls[NBLK][PP];
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            P[k] = 0; offM[k] = 0.f;
#pragma unroll
            for (int pp = 0; pp < PP; ++pp)
                Ls[k][pp] = (k < nact && nt > 1) ? __ldcg(reinterpret_cast<const float2 *>(hist + ((size_t)k * nt + nt - 1) * Q + q0b + 256 * pp))
                                                 : make_float2(0.f, 0.f);
        }
        cluster_sync();
        // rank 0, warp k: turn the sums of step t of block k (slots of buffer b) into soft[t]
        auto finish_step = [&](int t, int b, int k) {
            if (rank == 0 && warp == k) {
                const float4 s4 = *reinterpret_cast<const float4 *>(part + (size_t)((b * NBLK + k) * SLOTS + lane) * 4);
                const float den = warp_sum(s4.x), n0 = warp_sum(s4.y), n1 = warp_sum(s4.z);
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
                    float2 cb[2][8];
                    tmem_ld16(tm, cb[0]);                                     // requested before the wait for the step's inputs
                    if (t < nt) {
                        wait_inputs(ib, k);
                        cmax[k] = warp_max(wmax[si * SLOTS + lane]);
                        P[k] += (int)offM[k];
                        offM[k] = rintf(cmax[k]);
                        finish_step(t + 1, ib, k);
                    }
                    const float *Min = msg + si * QC + C::beta_in(warp, lane);   // [b >> 1][x & 127][b & 1], x = 2 xp, 2 xp + 1
                    if (tid == 0) pr.expect_tx(mbar_full + 8u * so, rank == 0 ? TX_MSG + TX_PART : TX_MSG);
                    // history of the next step, one step ahead (row t - 2 = L_{t-1}; L_1 = 0)
                    float2 Ls_next[PP];
#pragma unroll
                    for (int pp = 0; pp < PP; ++pp)
                        Ls_next[pp] = t > 2 ? __ldcg(reinterpret_cast<const float2 *>(hist + ((size_t)k * nt + t - 2) * Q + q0b + 256 * pp))
                                            : make_float2(0.f, 0.f);
                    const float *wk = w_s + k * C::MAX_N + 2 * (t - 1);
                    const float2 wx = splat2(wk[0]), wy = splat2(wk[1]);
                    // the outputs are shifted by offM (once per group, below); D refers to the unshifted inputs
                    const float Dm = ((float)(Ofin[k] - O_s[k * OSTR + t] - P[k]) + lsefin[k]);
                    const float2 offM2 = splat2(offM[k]);
                    float2 fd = make_float2(0.f, 0.f), fx = fd, fy = fd;
                    float tmax = __int_as_float(0xff800000);
#pragma unroll
                    for (int pp = 0; pp < PP; ++pp) {
                        float2 u[K];
#pragma unroll
                        for (int un = 0; un < C::UNITS; ++un) {
                            const int g = 2 * pp * C::UNITS + un;                             // every pair walks its table slice twice
                            tmem_wait_ld(cb[g & 1]);
                            tmem_ld16(tm + 64u * pp + 16u * ((un + 1) % C::UNITS), cb[(g + 1) & 1]);   // wraps round for the second pass
#pragma unroll
                            for (int e = 0; e < 4; e += 2) {
                                const int b = 4 * un + e;
                                const float4 Mv = *reinterpret_cast<const float4 *>(Min + 256 * (b >> 1));   // M(x,b), M(x,b+1), M(x+1,b), M(x+1,b+1)
#pragma unroll
                                for (int bb = 0; bb < 2; ++bb) {
                                    const float2 dx = sub2(cb[g & 1][2 * (e + bb)], wx), dy = sub2(cb[g & 1][2 * (e + bb) + 1], wy);
                                    const float2 Mb = bb == 0 ? make_float2(Mv.x, Mv.z) : make_float2(Mv.y, Mv.w);
                                    u[b + bb] = fma2(fma2(dy, dy, mul2(dx, dx)), nl2, Mb);
                                }
                            }
                        }
                        const float2 m = max_pairs<K>(u);
                        float2 sum = make_float2(0.f, 0.f), cx = sum, cy = sum;
#pragma unroll
                        for (int un = 0; un < C::UNITS; ++un) {                                  // second pass over the table slice
                            const int g = (2 * pp + 1) * C::UNITS + un;
                            tmem_wait_ld(cb[g & 1]);
                            if (un + 1 < C::UNITS) tmem_ld16(tm + 64u * pp + 16u * (un + 1), cb[(g + 1) & 1]);
                            else if (pp + 1 < PP) tmem_ld16(tm + 64u * (pp + 1), cb[(g + 1) & 1]);   // first unit of the next pair
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 pb = ex2f2(sub2(u[4 * un + e], m));
                                sum = add2(sum, pb);
                                cx = fma2(pb, cb[g & 1][2 * e], cx);
                                cy = fma2(pb, cb[g & 1][2 * e + 1], cy);
                            }
                        }
                        const float2 out = add2(sub2(m, offM2), lg2f2(sum));
                        const float2 f = ex2f2(add2(m, sub2(Ls[k][pp], splat2(Dm))));
                        pr.async_v2(push_b + PUSH_B_PAIR * pp + (uint32_t)(so * QC) * 4u, out.x, out.y, push_b_mbar + 8u * so);
                        fd = fma2(f, sum, fd); fx = fma2(f, cx, fx); fy = fma2(f, cy, fy);
                        tmax = max3f(tmax, m.x, m.y);
                        Ls[k][pp] = Ls_next[pp];
                    }
                    const float s3 = warp_sum3_split(fd.x + fd.y, fx.x + fx.y, fy.x + fy.y, lane);   // lanes 0, 8, 16: den, num_0, num_1
                    tmax = warp_max(tmax) - offM[k];
                    if (lane == 0) {
#pragma unroll
                        for (int r = 0; r < CL; ++r) pr.async_f32(wmax_dst[r] + (uint32_t)(so * SLOTS) * 4u, tmax, full_of[r] + 8u * so);
                    }
                    if ((lane & 7) == 0) pr.async_f32(part_dst + (uint32_t)(so * SLOTS * 4 + (lane >> 3)) * 4u, lane < 24 ? s3 : 0.f, full_of[0] + 8u * so);
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
                cmax[k] = warp_max(wmax[si * SLOTS + lane]);
                P[k] += (int)offM[k];
                finish_step(1, ib, k);
                const float *Mfin = msg + si * QC;
                float ssum = 0.f;
                for (int e = tid; e < QC; e += CT) ssum += ex2f(Mfin[e] - cmax[k]);
                ssum = warp_sum(ssum);
                if (lane == 0) {
#pragma unroll
                    for (int r = 0; r < CL; ++r) st_cluster_f32(lz_dst[r] + (uint32_t)((NBLK + k) * SLOTS) * 4u, ssum);
                }
            }
        }
        cluster_sync();
#pragma unroll
        for (int k = 0; k < NBLK; ++k) {
            if (k < nact) {
                const float v = warp_sum(lz[(NBLK + k) * SLOTS + lane]);
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

}  // namespace bcjr
