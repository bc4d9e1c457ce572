// Forward call, one CTA per weight block, for the 2^16-state trellis (k = 2).
//
// The whole codebook (2^16 floats = 256 KB) does not fit one SM's registers next to anything
// else, and not its shared memory either -- but it is exactly the size of the SM's tensor
// memory (TMEM, 512 columns x 128 lanes x 32 bit), which this path does not otherwise use.
// TMEM is lane-private (a warp reaches only the 32 lanes of its sub-partition) and that is
// precisely the access pattern here: a thread owns the same butterflies for the whole kernel
// (see bcjr_cluster.cuh for the butterfly form), so the K*K codebook entries of each of its
// butterflies sit in "its" TMEM lane and are fetched with tcgen05.ld, sixteen columns at a
// time, one butterfly ahead of the arithmetic.  With the codebook out of the register file and
// the compressed message vector (64 KB) double-buffered in shared memory, one SM handles a
// block alone: the per-step exchange is a CTA barrier instead of a cluster-wide handshake.
//
// 16 warps (512 threads, 8 butterflies each at k = 2), all computing.  The history is
// thread-private: the alpha inputs L_t of a butterfly are what the same thread needs for that
// butterfly in the beta sweep, so it stores them with 16-byte global stores
// ([step][butterfly slot][16-byte chunk][thread]) and streams them back with cp.async into its own
// staging slots, RD - 1 butterflies ahead (cp.async.wait_group: no mbarrier, no copy warp, no
// branch in the butterfly loop).  No thread of this kernel spins on anything.
#pragma once
#include <type_traits>

#include "bcjr_ptx.cuh"


namespace bcjr {

// ---------------------------------------------------------------------------- TMEM helpers
__device__ __forceinline__ void tmem_alloc_512(uint32_t smem_dst)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_dst) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_512(uint32_t taddr)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(taddr) : "memory");
}
// wait for this thread's outstanding tcgen05.ld; the loaded registers are operands so that no
// use of them can be scheduled ahead of the wait
__device__ __forceinline__ void tmem_wait_ld(float2 (&v)[8])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+f"(v[0].x), "+f"(v[0].y), "+f"(v[1].x), "+f"(v[1].y), "+f"(v[2].x), "+f"(v[2].y), "+f"(v[3].x), "+f"(v[3].y),
                   "+f"(v[4].x), "+f"(v[4].y), "+f"(v[5].x), "+f"(v[5].y), "+f"(v[6].x), "+f"(v[6].y), "+f"(v[7].x), "+f"(v[7].y)
                 :
                 : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// sixteen consecutive columns of the calling thread's lane, as eight packed pairs
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const float2 (&v)[8])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "f"(v[0].x), "f"(v[0].y), "f"(v[1].x), "f"(v[1].y), "f"(v[2].x), "f"(v[2].y), "f"(v[3].x), "f"(v[3].y), "f"(v[4].x),
        "f"(v[4].y), "f"(v[5].x), "f"(v[5].y), "f"(v[6].x), "f"(v[6].y), "f"(v[7].x), "f"(v[7].y)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float2 (&v)[8])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=f"(v[0].x), "=f"(v[0].y), "=f"(v[1].x), "=f"(v[1].y), "=f"(v[2].x), "=f"(v[2].y), "=f"(v[3].x), "=f"(v[3].y),
          "=f"(v[4].x), "=f"(v[4].y), "=f"(v[5].x), "=f"(v[5].y), "=f"(v[6].x), "=f"(v[6].y), "=f"(v[7].x), "=f"(v[7].y)
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void compute_barrier(int nthreads)
{
    asm volatile("bar.sync 1, %0;" ::"r"(nthreads) : "memory");
}

// KB = 2: 8 butterflies of 16 states per thread; KB = 3: 2 butterflies of 64 states per thread.
// A butterfly's K*K codebook entries are fetched in units of sixteen TMEM columns (eight packed
// pairs): with K = 4 one unit is the whole butterfly, with K = 8 a unit is one output pair h of
// the alpha sweep (pairs over j) or one input pair jh of the beta sweep (pairs over b).
template <int KB_>
struct SoloCfg {
    static constexpr int LB = 16, KB = KB_, K = 1 << KB, S = 1 << LB, Q = S >> KB, NB = S >> (2 * KB);
    static constexpr int CTHREADS = 512;                       // every thread computes
    static constexpr int THREADS = CTHREADS;
    static constexpr int NWARP = CTHREADS / 32;
    static constexpr int BPT = NB / CTHREADS;                  // butterflies per thread
    static constexpr int UNITS = K * K / 16;                   // 16-column units per butterfly
    static constexpr int HPU = (K / 2) / UNITS;                // pairs h (alpha) or jh (beta) covered by one unit
    static constexpr int NCH = K / 4;                          // 16-byte chunks per butterfly and thread (K values of L)
    static constexpr int RD = KB == 2 ? BPT : 4;               // staging depth in butterflies
    static constexpr int MAX_N = 2048;
    static constexpr int OFF_MSG = 0;                          // [2][Q]
    static constexpr int OFF_RING = OFF_MSG + 2 * Q;           // float4 [RD][NCH][CTHREADS], thread-private entries
    static constexpr int OFF_W = OFF_RING + RD * NCH * CTHREADS * 4;   // [2][MAX_N]: clamped weight and kap of every step (step_energy)
    static constexpr int OFF_O = OFF_W + 2 * MAX_N;            // int [MAX_N + 2]
    static constexpr int OFF_WMAX = OFF_O + MAX_N + 2 + 2;     // [2][32]
    static constexpr int OFF_PART = OFF_WMAX + 64;             // [2][32][2]
    static constexpr int OFF_LZ = OFF_PART + 128;              // [32]
    static constexpr int OFF_MBAR = OFF_LZ + 32;               // (no mbarrier left in this kernel; kept 8-byte aligned)
    static constexpr int OFF_TMEM = OFF_MBAR + 2;              // uint32 TMEM base
    static constexpr int OFF_FLAG = OFF_TMEM + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 2;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(OFF_MBAR % 2 == 0, "mbarrier alignment");
    static_assert(BPT * K * K == 128, "a thread's codebook slice fills its 128 TMEM columns");
    static_assert(UNITS * HPU == K / 2 && (K == 4 || K == 8), "unit decomposition");
    // pair index inside a unit: alpha pair (j, h), beta pair (jh, b)
    __host__ __device__ static constexpr int a_idx(int j, int h) { return K == 4 ? 2 * j + h : j; }
    __host__ __device__ static constexpr int b_idx(int jh, int b) { return K == 4 ? 4 * jh + b : b; }
};

// stage one butterfly's codebook entries into TMEM in the pairing of a sweep; a null table means the computed
// Gaussian emission (Section 3.1), evaluated here instead of loaded
template <typename C>
__device__ __forceinline__ void stage_codebook(const float *cbk, int x, uint32_t tm_butterfly, bool beta)
{
    constexpr int K = C::K;
#pragma unroll
    for (int u = 0; u < C::UNITS; ++u) {
        float2 v[8];
#pragma unroll
        for (int hh = 0; hh < C::HPU; ++hh) {
            const int h = u * C::HPU + hh;                     // alpha: output pair (2h, 2h+1); beta: input pair (2h, 2h+1)
#pragma unroll
            for (int o = 0; o < K; ++o) {
                // alpha: pair (j = o, h) = (c[o | x | 2h], c[o | x | 2h+1]);  beta: pair (jh = h, b = o) = (c[2h | x | o], c[2h+1 | x | o])
                const int slo = beta ? (2 * h) * C::Q + x * K + o : o * C::Q + x * K + 2 * h;
                const int shi = beta ? (2 * h + 1) * C::Q + x * K + o : o * C::Q + x * K + 2 * h + 1;
                const float lo = table_entry(cbk, slo, C::S), hi = table_entry(cbk, shi, C::S);
                v[beta ? C::b_idx(hh, o) : C::a_idx(o, hh)] = make_float2(lo, hi);
            }
        }
        tmem_st16(tm_butterfly + 16u * u, v);
    }
}

template <int KB>
__global__ void __launch_bounds__(SoloCfg<KB>::THREADS, 1) fwd_solo_kernel(FwdParams p)
{
    using C = SoloCfg<KB>;
    constexpr int K = C::K, NB = C::NB, Q = C::Q, BPT = C::BPT, NWARP = C::NWARP, CT = C::CTHREADS, NCH = C::NCH, RD = C::RD;
    constexpr int UNITS = C::UNITS, HPU = C::HPU, NU = BPT * UNITS;
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float2 nl2 = splat2(-p.lam2);

    float *msg = smem + C::OFF_MSG;
    float4 *stage4 = reinterpret_cast<float4 *>(smem + C::OFF_RING);
    float *w_s = smem + C::OFF_W, *kap_s = w_s + C::MAX_N;
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;
    int *O_s = reinterpret_cast<int *>(smem + C::OFF_O);
    float *wmax = smem + C::OFF_WMAX;
    float *part = smem + C::OFF_PART;
    float *lz = smem + C::OFF_LZ;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);
    const uint32_t stage_u32 = smem_u32(stage4) + (uint32_t)tid * 16u;

    // history of this CTA: float4 [n][BPT][NCH][CT], row t = the alpha inputs L_t of every butterfly;
    // a thread writes and reads back only its own entries
    float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)blockIdx.x * n * Q) + tid;

    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    {
        // ============================ compute warps ============================
        // TMEM: lanes of this warp's sub-partition, 128 columns per thread
        const uint32_t tm = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
        // destinations of the outputs (floats from the start of a message buffer)
        //   alpha: L([x|l]) -> butterfly x2 = (x*K) mod NB, input j2 = (x*K) / NB: [(i2*K + j2)*CT + tid2 .. +K)
        //   beta : M([j|x]) -> butterfly x1 = (j*NB + x) / K, input b1 = x mod K:  [x1*K + b1]
        int push_a[BPT];
#pragma unroll
        for (int i = 0; i < BPT; ++i) {
            const int x = i * CT + tid;
            const int q2 = x * K, j2 = q2 / NB, x2 = q2 % NB;
            push_a[i] = ((x2 / CT) * K + j2) * CT + (x2 % CT);
        }
        float defect = 0.f, zgap = 0.f;

        for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
            const float *w = p.W + blk * n;
            // A block whose weights all lie inside the table's range (delta = 0 at every step, nearly every block of
            // Gaussian weights) takes the sweeps with the plain square: one multiply instead of a fused multiply-add
            // per pair of states, 5 % of the kernel.  Any other block takes the form of step_energy.
            int outside = 0;
            for (int t = tid; t < n; t += CT) {
                const StepEnergy se = step_energy(__ldg(w + t), c_lo, c_hi, p.lam2);
                w_s[t] = se.wc; kap_s[t] = se.kap;
                outside |= se.delta != 0.f;
            }
            const bool recentre = __syncthreads_or(outside) != 0;
            for (int q = tid; q < Q; q += CT) msg[q] = 0.f;                      // L_1 = 0 in buffer 0
            if (tid == 0) O_s[1] = 0;
#pragma unroll
            for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * CT + tid, tm + (uint32_t)(K * K * i), false);
            tmem_wait_st();
            int O = 0;
            float off = 0.f, cmax = 0.f, bdef = 0.f;
            compute_barrier(CT);
            // ================= alpha sweep
            auto alpha_sweep = [&](auto rc_tag) {
            constexpr bool RC = decltype(rc_tag)::value;
            for (int t = 1; t <= n; ++t) {
                const int cur = (t - 1) & 1;
                const float *Lin = msg + cur * Q;
                float *Lout = msg + (cur ^ 1) * Q;
                if (t > 1) {
                    cmax = warp_max(lane < NWARP ? wmax[cur * 32 + lane] : NEG_INF) - off;
                    off = rintf(cmax);
                }
                float4 *hrow = hist4 + (size_t)(t - 1) * (BPT * NCH * CT);
                const float2 w2 = splat2(w_s[t - 1]), kap2 = splat2(kap_s[t - 1]);
                const float2 off2 = splat2(off);
                float tmax = NEG_INF;
                float2 cb[2][8];
                tmem_ld16(tm, cb[0]);
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    float Lj[K];
#pragma unroll
                    for (int j = 0; j < K; ++j) Lj[j] = Lin[(i * K + j) * CT + tid];
#pragma unroll
                    for (int q = 0; q < NCH; ++q)
                        hrow[(i * NCH + q) * CT] = make_float4(Lj[4 * q], Lj[4 * q + 1], Lj[4 * q + 2], Lj[4 * q + 3]);
                    float2 out[K / 2];
#pragma unroll
                    for (int u = 0; u < UNITS; ++u) {
                        const int g = i * UNITS + u;                             // unit counter (compile time after unrolling)
                        tmem_wait_ld(cb[g & 1]);
                        if (g + 1 < NU) tmem_ld16(tm + 16u * (g + 1), cb[(g + 1) & 1]);
#pragma unroll
                        for (int hh = 0; hh < HPU; ++hh) {
                            const int h = u * HPU + hh;
                            float2 a[K];
#pragma unroll
                            for (int j = 0; j < K; ++j) {
                                const float2 du = sub2(cb[g & 1][C::a_idx(j, hh)], w2);
                                a[j] = RC ? energy2(du, nl2, kap2, splat2(Lj[j])) : fma2(mul2(du, du), nl2, splat2(Lj[j]));
                            }
                            const float2 m = max_pairs<K>(a);
                            float2 sum = ex2f2(sub2(a[0], m));
#pragma unroll
                            for (int j = 1; j < K; ++j)      // every fourth exponential on the FP32 pipe: the MUFU is this sweep's bottleneck
                                sum = add2(sum, (j % 4 == 3) ? ex2_poly2(sub2(a[j], m)) : ex2f2(sub2(a[j], m)));
                            out[h] = add2(sub2(m, off2), lg2f2(sum));
                            tmax = max3f(tmax, m.x, m.y);
                        }
                    }
#pragma unroll
                    for (int h = 0; h < K / 2; h += 2)
                        *reinterpret_cast<float4 *>(Lout + push_a[i] + 2 * h) = make_float4(out[h].x, out[h].y, out[h + 1].x, out[h + 1].y);
                }
                tmax = warp_max(tmax);
                if (lane == 0) wmax[(cur ^ 1) * 32 + warp] = tmax;
                O += (int)off;
                if (tid == 0) O_s[t + 1] = O;
                compute_barrier(CT);
            }
            };
            if (recentre) alpha_sweep(std::true_type{}); else alpha_sweep(std::false_type{});
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
                double zshift = 0.0;                             // sum_t lam2 delta_t^2 = sum_t kap_t^2 / (4 lam2): left out by step_energy
                for (int t = 0; t < n; ++t) zshift += (double)kap_s[t] * (double)kap_s[t];
                zshift /= 4.0 * (double)p.lam2;
                p.logZ[blk] = (float)(((double)Ofin + (double)lsefin - zshift) * 0.6931471805599453);
            }
            // ================= beta sweep
            for (int q = tid; q < Q; q += CT) msg[q] = 0.f;                      // M_n = 0 in buffer 0
#pragma unroll
            for (int i = 0; i < BPT; ++i) stage_codebook<C>(p.cb, i * CT + tid, tm + (uint32_t)(K * K * i), true);
            tmem_wait_st();
            int P = 0;
            float offM = 0.f;
            // history stream: chunk c = butterfly (t = n - c / BPT, i = c % BPT), staged RD - 1 ahead with cp.async
            const uint32_t nchunks = (uint32_t)n * BPT;
            // running source pointer of the next chunk to request: butterflies i = 0..BPT-1 of step t, then step t - 1
            const float4 *nsrc = hist4 + (size_t)(n - 1) * (BPT * NCH * CT);
            uint32_t nleft = nchunks;                            // chunks not yet requested
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
                const ptrdiff_t adv = wrap ? -(ptrdiff_t)((size_t)(2 * BPT - 1) * (NCH * CT)) : (ptrdiff_t)(NCH * CT);
                nsrc += more ? adv : 0;
                ni = wrap ? 0 : ni + 1;
                nleft -= more ? 1u : 0u;
            };
            // RD == BPT (k = 2): the ring slot of a butterfly is its index in the step, and everything about a request is
            // known at compile time but the step
            constexpr bool STATIC_RING = RD == BPT;
            constexpr ptrdiff_t HROW = (ptrdiff_t)BPT * NCH * CT;
            auto issue_static = [&](const float4 *row, int i) {           // butterfly i of the step whose history starts at row
                const uint32_t dst = stage_u32 + (uint32_t)i * (uint32_t)(NCH * CT * 16);
#pragma unroll
                for (int q = 0; q < NCH; ++q)
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (uint32_t)(q * CT * 16)), "l"(row + (i * NCH + q) * CT) : "memory");
            };
#pragma unroll
            for (uint32_t c = 0; c + 1 < RD; ++c) {
                if (STATIC_RING) { issue_static(hist4 + (size_t)(n - 1) * HROW, (int)c); asm volatile("cp.async.commit_group;" ::: "memory"); }
                else issue_chunk(c);
            }
            uint32_t chunk = 0, slot = 0;
            compute_barrier(CT);
            auto beta_sweep = [&](auto rc_tag) {
            constexpr bool RC = decltype(rc_tag)::value;
            for (int t = n; t >= 1; --t) {
                const int cur = (n - t) & 1;
                const float *Min = msg + cur * Q;
                float *Mout = msg + (cur ^ 1) * Q;
                if (t < n) {
                    cmax = warp_max(lane < NWARP ? wmax[cur * 32 + lane] : NEG_INF);
                    P += (int)offM;
                    offM = rintf(cmax);
                    if (warp == 0) {                                             // soft[t+1] from the partial sums
                        float a = lane < NWARP ? part[(cur * 32 + lane) * 2] : 0.f;
                        float c = lane < NWARP ? part[(cur * 32 + lane) * 2 + 1] : 0.f;
                        a = warp_sum(a); c = warp_sum(c);
                        if (lane == 0) {
                            const float sw = a / c;
                            p.soft[blk * n + t] = sw;
                            if (p.soft_copy) p.soft_copy[blk * n + t] = sw;
                            bdef = fmaxf(bdef, fabsf(c - 1.f));
                        }
                    }
                }
                const float2 w2 = splat2(w_s[t - 1]), kap2 = splat2(kap_s[t - 1]);
                const float2 offM2 = splat2(offM);
                const float2 Dm2 = splat2((float)(Ofin - O_s[t] - P) + lsefin);
                float2 num2 = make_float2(0.f, 0.f), den2 = make_float2(0.f, 0.f);
                float tmax = NEG_INF;
                float2 cb[2][8];
                tmem_ld16(tm, cb[0]);
#pragma unroll
                for (int i = 0; i < BPT; ++i, ++chunk) {
                    if (STATIC_RING) {                               // RD - 1 butterflies ahead, into the slot consumed last
                        const float4 *hrow = hist4 + (size_t)(t - 1) * HROW;
                        if (i == 0) issue_static(hrow, BPT - 1);
                        else if (t > 1) issue_static(hrow - HROW, i - 1);
                        asm volatile("cp.async.commit_group;" ::: "memory");
                    } else {
                        issue_chunk(slot == 0 ? RD - 1 : slot - 1);  // refill the slot consumed last
                    }
                    asm volatile("cp.async.wait_group %0;" ::"n"(RD - 1) : "memory"); // chunk `chunk` has landed
                    const uint32_t sl = STATIC_RING ? (uint32_t)i : slot;
                    float Lh[K];
#pragma unroll
                    for (int q = 0; q < NCH; ++q) {
                        const float4 l4 = stage4[(sl * NCH + q) * CT + tid];
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
                                uu[b] = RC ? energy2(du, nl2, kap2, splat2(Mb[b])) : fma2(mul2(du, du), nl2, splat2(Mb[b]));
                            }
                            const float2 m = max_pairs<K>(uu);
                            const float2 Lhj = make_float2(Lh[2 * jh], Lh[2 * jh + 1]);
                            const float2 f = ex2f2(add2(sub2(m, Dm2), Lhj));
                            float2 pb = ex2f2(sub2(uu[0], m));
                            float2 sum = pb, craw = mul2(pb, cb[g & 1][C::b_idx(hh, 0)]);
#pragma unroll
                            for (int b = 1; b < K; ++b) {
                                pb = ex2f2(sub2(uu[b], m));
                                sum = add2(sum, pb);
                                craw = fma2(pb, cb[g & 1][C::b_idx(hh, b)], craw);
                            }
                            const float2 out = add2(sub2(m, offM2), lg2f2(sum));
                            tmax = max3f(tmax, m.x, m.y);
                            // M([j|x]) with x = i*CT + tid goes to [x1*K + b1], x1 = j*(NB/K) + x/K, b1 = x%K
                            Mout[((2 * jh) * (NB / K) + (i * CT + tid) / K) * K + (tid % K)] = out.x;
                            Mout[((2 * jh + 1) * (NB / K) + (i * CT + tid) / K) * K + (tid % K)] = out.y;
                            num2 = fma2(f, craw, num2);
                            den2 = fma2(f, sum, den2);
                        }
                    }
                }
                const float nd = warp_sum2_split(num2.x + num2.y, den2.x + den2.y, lane);   // lane 0: numerator, lane 16: denominator
                tmax = warp_max(tmax) - offM;
                if (lane == 0) wmax[(cur ^ 1) * 32 + warp] = tmax;
                if ((lane & 15) == 0) part[((cur ^ 1) * 32 + warp) * 2 + (lane >> 4)] = nd;
                compute_barrier(CT);
            }
            };
            if (recentre) beta_sweep(std::true_type{}); else beta_sweep(std::false_type{});
            {
                const int fin = n & 1;                                           // M_0 and the sums of step 1
                cmax = warp_max(lane < NWARP ? wmax[fin * 32 + lane] : NEG_INF);
                P += (int)offM;
                if (warp == 0) {
                    float a = lane < NWARP ? part[(fin * 32 + lane) * 2] : 0.f;
                    float c = lane < NWARP ? part[(fin * 32 + lane) * 2 + 1] : 0.f;
                    a = warp_sum(a); c = warp_sum(c);
                    if (lane == 0) {
                        const float sw = a / c;
                        p.soft[blk * n] = sw;
                        if (p.soft_copy) p.soft_copy[blk * n] = sw;
                        bdef = fmaxf(bdef, fabsf(c - 1.f));
                        defect = fmaxf(defect, bdef);
                        if (p.blk_defect) p.blk_defect[blk] = bdef;
                    }
                }
                // consistency: P_0 + LSE_q M_0(q) against log2 Z
                const float *Mfin = msg + fin * Q;
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
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
