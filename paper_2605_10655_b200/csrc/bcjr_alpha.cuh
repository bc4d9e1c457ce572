// Backward call, first half (2^16 states; k = 2, 3): the alpha sweep carrying (L, At) on ONE CTA per block.
//
// The backward pass needs gradient accumulators next to the codebook only in its beta sweep.  Its alpha sweep
// -- the forward messages L_t and the conditional expectations At_t of every step, which the beta sweep reads
// back -- needs the codebook alone, and the codebook alone fits one SM's tensor memory.  Run on one SM, a step is
// one CTA barrier instead of a cluster handshake and a thread has eight butterflies per step instead of four to
// hide it behind, which is why the forward kernel reaches a higher fraction of the special-function peak than
// the two-CTA backward kernel.  So the backward call is split: this kernel writes the history of a chunk of
// blocks (one block per SM), bwd_skew_kernel<ACC, true> (k = 2) or bwd_duo_kernel<3, true> (k = 3) then runs the beta
// sweeps of the same chunk on two-CTA clusters.
//
// Messages in place.  (L, At) double-buffered would be 256 KB; here each array has ONE buffer of Q floats.  A
// butterfly's four inputs have no other reader, so its four outputs overwrite them (output [x|l] takes the place
// of input [l|x]); the price is that group index q lives at a step-dependent slot,
//     slot_t(q) = swz(rotr(q, 2 (t-1) mod 14))      (the perfect shuffle undone one step at a time),
// where swz XORs the upper index bits into the five bank bits through a matrix chosen so that, at every one of the
// seven rotations, the five index bits that vary across a warp reach five different bank bits.  (L and At are two
// arrays of floats, not one array of pairs: 8-byte elements, with a swizzle made for them, measured 2 % slower.)  rotr and swz are
// XOR-linear over disjoint bit fields, so a thread's addresses are  T_i ^ s_tid ^ T_j  with two small per-step
// tables and one value per thread and step.
//
// History layout: exactly what the beta kernel's threads read (float4 [n][CTA][slot][L | At][thread] in ITS
// assignment of butterflies to threads), so each butterfly's rows are written where its beta-sweep owner looks.
#pragma once
#include "bcjr_skew.cuh"

namespace bcjr {

template <int KB_>
struct AlphaCfg {
    static constexpr int LB = 16, KB = KB_, K = 1 << KB, S = 1 << LB, Q = S >> KB, NB = S >> (2 * KB), QB = LB - KB;
    static constexpr int CTHREADS = 512, THREADS = 512, NWARP = 16, BPT = NB / CTHREADS;   // butterflies per thread: x = i * 512 + tid
    static constexpr int UNITS = K * K / 16, HPU = (K / 2) / UNITS;                       // 16-column table units per butterfly
    static constexpr int MAX_N = 1024, NROT = QB;              // rotations: k (t-1) mod (Lb - k) takes 7 values at k = 2, all 13 at k = 3
    static constexpr int OFF_L = 0;                            // [Q]
    static constexpr int OFF_A = OFF_L + Q;                    // [Q]
    static constexpr int OFF_TAB = OFF_A + Q;                  // uint32 [NROT][16]: T_i (BPT), T_j (K) from entry 8
    static constexpr int OFF_WMAX = OFF_TAB + NROT * 16;       // [2][32]
    static constexpr int OFF_LZ = OFF_WMAX + 64;               // [32]
    static constexpr int OFF_TMEM = OFF_LZ + 32;
    static constexpr int SMEM_FLOATS = OFF_TMEM + 4;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static constexpr int AUX_INTS = MAX_N + 4;                 // per block: O_t (t = 1 .. n+1), then the bits of the log2 Z tail
    static_assert(BPT * K * K == 128 && BPT <= 8 && K <= 8, "a thread's table slice fills its 128 tensor-memory columns");
    __host__ __device__ static constexpr int a_idx(int j, int h) { return K == 4 ? 2 * j + h : j; }
    __host__ __device__ static constexpr int b_idx(int jh, int b) { return K == 4 ? 4 * jh + b : b; }
    __host__ __device__ static constexpr uint32_t rotr(uint32_t v, int r) { return ((v >> r) | (v << (QB - r))) & ((1u << QB) - 1u); }
    // bank bits ^= M * (upper index bits).  The columns of M were chosen (by hand at k = 2, by search at k = 3; both
    // checked exhaustively) so that at every rotation the five index bits that vary across a warp reach five
    // independent vectors: e0..e4 for index bits 5..9, then e0+e1, e2, e0+e3, e4 for bits 10..13 (k = 2, 14 index bits)
    // or e0+e2, e1+e3, e0+e1+e4 for bits 10..12 (k = 3, 13 index bits).
    __host__ __device__ static constexpr uint32_t swz(uint32_t v)
    {
        const uint32_t h = v >> 10;
        const uint32_t top = KB == 2 ? ((h & 1u) * 3u) ^ ((h & 2u) << 1) ^ (((h >> 2) & 1u) * 9u) ^ ((h & 8u) << 1)
                                     : ((h & 1u) * 5u) ^ (((h >> 1) & 1u) * 10u) ^ (((h >> 2) & 1u) * 19u);
        return v ^ ((v >> 5) & 31u) ^ top;
    }
    __host__ __device__ static constexpr uint32_t slot(uint32_t q, int r) { return swz(rotr(q, r)); }
};

// HL: the beta kernel's history layout (SkewCfg at k = 2, DuoCfg<3> at k = 3): float4 index of chunk 0 of butterfly x inside a step
template <int KB>
__device__ __forceinline__ int beta_history_pos(int x)
{
    if (KB == 2) return SkewCfg::rank_of(x) * (SkewCfg::BPT * SkewCfg::NCH * SkewCfg::THREADS) + SkewCfg::slot_of(x) * SkewCfg::NCH * SkewCfg::THREADS + SkewCfg::tid_of(x);
    using D = DuoCfg<3>;                                        // x = rank * NBC + tid, one butterfly per thread
    return (x / D::NBC) * (D::BPT * D::NCH * D::THREADS) + (x % D::NBC);
}

template <int KB>
__global__ void __launch_bounds__(AlphaCfg<KB>::THREADS, 1) bwd_alpha_kernel(BwdParams p)
{
    using C = AlphaCfg<KB>;
    constexpr int K = C::K, Q = C::Q, BPT = C::BPT, NWARP = C::NWARP, CT = C::CTHREADS, UNITS = C::UNITS, HPU = C::HPU, NU = BPT * UNITS;
    constexpr ptrdiff_t HSTEP = 2 * Q / 4;                      // float4 per step: (L, At) of every group
    constexpr int HCH = CT;                                     // float4 between the 16-byte chunks of a butterfly (both layouts: 512 threads)
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.n;
    const float NEG_INF = __int_as_float(0xff800000);
    const float2 nl2 = splat2(-p.lam2);
    const float c_lo = p.diag->c_lo, c_hi = p.diag->c_hi;

    float *Ls = smem + C::OFF_L, *As = smem + C::OFF_A;
    uint32_t *tab = reinterpret_cast<uint32_t *>(smem + C::OFF_TAB);
    float *wmax = smem + C::OFF_WMAX;
    float *lz = smem + C::OFF_LZ;
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);

    if (tid < C::NROT * 16) {
        const int r = tid >> 4, e = tid & 15;                            // table row = the rotation itself
        uint32_t v = 0;
        if (e < BPT) v = C::slot((uint32_t)e << 9, r);                   // T_i: butterfly bits above the thread index
        else if (e >= 8 && e < 8 + K) v = C::slot((uint32_t)(e - 8) << (C::QB - KB), r);   // T_j: the input's branch bits
        tab[tid] = v;
    }
    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t tm = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
    // where the beta kernel's owner of butterfly x_i reads its history: float4 index inside a step
    int hpos[BPT];
#pragma unroll
    for (int i = 0; i < BPT; ++i) {
        const int x = i * CT + tid;
        hpos[i] = beta_history_pos<KB>(x);
    }

    for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x) {
        const float *w_s = p.W + blk * n, *g_s = p.g + blk * n, *sf_s = p.soft + blk * n;
        float4 *hist4 = reinterpret_cast<float4 *>(p.hist + (size_t)blk * n * 2 * Q);
        int *aux = p.stepO + (size_t)blk * C::AUX_INTS;
        {
            const float gsh1 = -__ldg(g_s) * __ldg(sf_s);             // L_1 = 0; the At array carries At + gsh (see bcjr_duo.cuh)
            for (int q = tid; q < Q; q += CT) { Ls[q] = 0.f; As[q] = gsh1; }
        }
        if (tid == 0) aux[1] = 0;
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
        auto alpha_sweep = [&](auto rc_tag) {
            constexpr bool RC = decltype(rc_tag)::value;
            int r = 0;                                                // k (t - 1) mod (Lb - k)
            for (int t = 1; t <= n; ++t) {
                const int cur = (t - 1) & 1;
                float2 cb[2][8];
                tmem_ld16(tm, cb[0]);
                const float gt = __ldg(g_s + t - 1), wt = __ldg(w_s + t - 1);
                const float gshn = t < n ? -__ldg(g_s + t) * __ldg(sf_s + t) : 0.f;
                if (t > 1) {
                    cmax = warp_max(lane < NWARP ? wmax[cur * 32 + lane] : NEG_INF) - off;
                    off = rintf(cmax);
                }
                const StepEnergy se = step_energy(wt, c_lo, c_hi, p.lam2);
                const float2 w2 = splat2(se.wc), kap2 = splat2(se.kap), g2 = splat2(gt), off2 = splat2(off), gshn2 = splat2(gshn);
                const uint32_t *tb = tab + r * 16;
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
                        Lj[j] = Ls[ti ^ TJ[j]];
                        Aj[j] = As[ti ^ TJ[j]];
                    }
#pragma unroll
                    for (int q = 0; q < K / 4; ++q) {
                        hrow[hpos[i] + q * HCH] = make_float4(Lj[4 * q], Lj[4 * q + 1], Lj[4 * q + 2], Lj[4 * q + 3]);
                        hrow[hpos[i] + (K / 4 + q) * HCH] = make_float4(Aj[4 * q], Aj[4 * q + 1], Aj[4 * q + 2], Aj[4 * q + 3]);
                    }
                    float2 outL[K / 2], outA[K / 2];
#pragma unroll
                    for (int u = 0; u < UNITS; ++u) {
                        const int g = i * UNITS + u;
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
                            float2 pj = ex2f2(sub2(a[0], m));
                            float2 sum = pj, ax = mul2(pj, fma2(g2, cb[g & 1][C::a_idx(0, hh)], splat2(Aj[0])));
#pragma unroll
                            for (int j = 1; j < K; ++j) {
                                // (no exponential goes to the FP32 pipe here, unlike the forward kernel's alpha sweep: with the
                                // conditional expectations riding along this sweep is short of issue slots, not of the special-function unit)
                                pj = ex2f2(sub2(a[j], m));
                                sum = add2(sum, pj);
                                ax = fma2(pj, fma2(g2, cb[g & 1][C::a_idx(j, hh)], splat2(Aj[j])), ax);
                            }
                            outL[h] = add2(sub2(m, off2), lg2f2(sum));
                            outA[h] = fma2(ax, rcpf2(sum), gshn2);
                            tmax = max3f(tmax, m.x, m.y);
                        }
                    }
                    // output [x|l] takes the place of input [l|x]
#pragma unroll
                    for (int h = 0; h < K / 2; ++h) {
                        Ls[ti ^ TJ[2 * h]] = outL[h].x; Ls[ti ^ TJ[2 * h + 1]] = outL[h].y;
                        As[ti ^ TJ[2 * h]] = outA[h].x; As[ti ^ TJ[2 * h + 1]] = outA[h].y;
                    }
                }
                tmax = warp_max(tmax);
                if (lane == 0) wmax[(cur ^ 1) * 32 + warp] = tmax;
                O += (int)off;
                if (tid == 0) aux[t + 1] = O;
                r += KB; r = r >= C::QB ? r - C::QB : r;
                compute_barrier(CT);
            }
        };
        if (recentre) alpha_sweep(std::true_type{}); else alpha_sweep(std::false_type{});
        // log2 Z = O_{n+1} + LSE_q L_{n+1}(q): the beta kernel needs the tail LSE_q L_{n+1}(q)
        cmax = warp_max(lane < NWARP ? wmax[(n & 1) * 32 + lane] : NEG_INF) - off;
        {
            float ssum = 0.f;
            for (int q = tid; q < Q; q += CT) ssum += ex2f(Ls[q] - cmax);
            ssum = warp_sum(ssum);
            if (lane == 0) lz[warp] = ssum;
            compute_barrier(CT);
        }
        const float lsefin = cmax + lg2f(warp_sum(lane < NWARP ? lz[lane] : 0.f));
        if (tid == 0) {
            diag_check_finite(p.diag, lsefin);
            aux[n + 2] = __float_as_int(lsefin);
        }
        compute_barrier(CT);                                          // lz, wmax and the messages are free for the next block
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
