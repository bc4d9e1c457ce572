// Viterbi hard code for the 2^16-state trellis (k = 2 or 3): one CTA per weight block.
//
// Same butterfly ownership as the sum-product kernels, in the (min, +) semiring and in IEEE
// double (bit-identical with a sequential double implementation: d = (double)w - (double)c,
// m = min_j(...) + d*d, no fused multiply-add; the lowest branch wins ties):
//     mv_{t+1}([x|l]) = min_j ( mv_t([j|x]) + (w_t - c[j|x|l])^2 ),   best branch j kept per group.
//   - codebook: tensor memory (the fp32 table is exactly the SM's 256 KB of TMEM);
//   - metrics: Q doubles = 128 KB, ONE buffer, updated in place.  A butterfly's four inputs
//     have no other reader, so its four outputs overwrite them; the price is that the logical
//     index q lives at a step-dependent address, rotr(q, k*step) on the Lb-k index bits (the
//     perfect shuffle undone one step at a time), XOR-swizzled so that whichever five index bits
//     vary across a warp land on different banks.  One CTA barrier per step;
//   - backpointers: one word per butterfly and step (K branches of k bits: a byte for k = 2, 32
//     bits for k = 3), 4 KB per step and 1 MB per 256-step block, streamed to global memory; an extra warp backtracks block b, and writes its outputs,
//     while the compute warps already run block b+1 (two backpointer buffers per CTA).
#pragma once
#include "bcjr_solo.cuh"

namespace bcjr {

template <int KB_>
struct VitSoloCfg {
    static constexpr int LB = 16, KB = KB_, K = 1 << KB, S = 1 << LB, Q = S >> KB, NB = S >> (2 * KB);
    static constexpr int QB = LB - KB;                          // index bits of a group
    static constexpr int CTHREADS = 512, THREADS = CTHREADS + 32, NWARP = CTHREADS / 32;
    static constexpr int BPT = NB / CTHREADS;                   // butterflies per thread (8 / 2): x = tid*BPT + i
    static constexpr int UNITS = K * K / 16;                    // 16-column TMEM units per butterfly
    static constexpr int JPU = K / UNITS;                       // predecessors j covered by one unit
    static constexpr int WORD_BITS = 64 / BPT;                  // backpointer word of one butterfly (8 / 32 bits)
    static constexpr int ROW_BYTES = NB * WORD_BITS / 8;        // backpointers of one step
    static constexpr int MAX_N = 4096;
    static constexpr int OFF_MV = 0;                            // double [Q]  (2 floats each)
    static constexpr int OFF_PATH = OFF_MV + 2 * Q;             // int [MAX_N] state sequence of the block being traced
    static constexpr int OFF_RED = OFF_PATH + MAX_N;            // double [32] + int [32]
    static constexpr int OFF_BEST = OFF_RED + 96;               // int [2] final state per buffer parity
    static constexpr int OFF_MBAR = OFF_BEST + 2;               // uint64: tb_ready[2], tb_done[2]
    static constexpr int OFF_TMEM = OFF_MBAR + 8;
    static constexpr int OFF_FLAG = OFF_TMEM + 2;
    static constexpr int SMEM_FLOATS = OFF_FLAG + 2;
    static constexpr size_t SMEM_BYTES = (size_t)SMEM_FLOATS * 4;
    static_assert(OFF_MBAR % 2 == 0 && OFF_RED % 2 == 0, "8-byte alignment");
    static_assert(BPT * K * K == 128, "a thread's codebook slice fills its 128 TMEM columns");
    static_assert(K * KB <= WORD_BITS && (WORD_BITS == 8 || WORD_BITS == 32), "backpointer word");
};

// step-dependent physical slot of a QB-bit group index: rotate right, then fold the upper bits
// into the bank bits (XOR-linear, so it distributes over disjoint bit fields)
template <int QB>
__device__ __forceinline__ uint32_t vit_rotr(uint32_t v, int r)
{
    constexpr uint32_t M = (1u << QB) - 1u;
    return ((v >> r) | (v << (QB - r))) & M;
}
__device__ __forceinline__ uint32_t vit_swz(uint32_t v) { return v ^ ((v >> 5) & 31u) ^ ((v >> 10) & 15u); }

template <int KB>
__global__ void __launch_bounds__(VitSoloCfg<KB>::THREADS, 1) viterbi_solo_kernel(VitParams p)
{
    using C = VitSoloCfg<KB>;
    constexpr int K = C::K, Q = C::Q, BPT = C::BPT, NWARP = C::NWARP, CT = C::CTHREADS, QB = C::QB;
    constexpr int UNITS = C::UNITS, JPU = C::JPU, WB = C::WORD_BITS, ROWB = C::ROW_BYTES;
    extern __shared__ __align__(16) float smem[];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int n = p.n;
    double *mv = reinterpret_cast<double *>(smem + C::OFF_MV);
    int *path = reinterpret_cast<int *>(smem + C::OFF_PATH);
    double *redv = reinterpret_cast<double *>(smem + C::OFF_RED);
    int *redi = reinterpret_cast<int *>(smem + C::OFF_RED + 64);
    volatile int *best = reinterpret_cast<volatile int *>(smem + C::OFF_BEST);
    volatile uint32_t *tmem_slot = reinterpret_cast<volatile uint32_t *>(smem + C::OFF_TMEM);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + C::OFF_FLAG);
    Proto pr{1u, abort_flag, p.diag};
    const uint32_t tb_ready = smem_u32(smem + C::OFF_MBAR);      // [2] compute -> trace warp
    const uint32_t tb_done = tb_ready + 16u;                     // [2] trace warp -> compute
    // backpointers of this CTA: [2 parities][n][ROWB] bytes
    uint8_t *bp_base = p.bp + (size_t)blockIdx.x * 2 * (size_t)n * ROWB;
    const int nbits = C::LB + KB * (n - 1);

    if (tid == 0) {
        for (int s = 0; s < 2; ++s) { mbar_init(tb_ready + 8u * s, NWARP); mbar_init(tb_done + 8u * s, 1); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc_512(smem_u32(const_cast<uint32_t *>(tmem_slot)));
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;

    if (warp == NWARP) {
        // ============================ trace warp ============================
        uint32_t it = 0;
        for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x, ++it) {
            const uint32_t par = it & 1u;
            pr.wait(tb_ready + 8u * par, (it >> 1) & 1u);
            if (!__all_sync(0xffffffffu, pr.live)) continue;     // a wait ran out: nothing valid to trace
            const uint8_t *bp = bp_base + (size_t)par * n * ROWB;
            if (lane == 0) {
                // predecessor of s at step t+1 is j*Q + (s >> k), j = branch stored for group s >> k
                int s = best[par] & (C::S - 1);
                path[n - 1] = s;
                for (int t = n - 1; t >= 1; --t) {
                    const int q = s >> KB;
                    unsigned word;
                    if (WB == 8) word = __ldcg(bp + (size_t)t * ROWB + (q >> KB));
                    else word = __ldcg(reinterpret_cast<const unsigned *>(bp + (size_t)t * ROWB) + (q >> KB));
                    const int j = (int)(word >> (KB * (q & (K - 1)))) & (K - 1);
                    s = j * Q + q;
                    path[t - 1] = s;
                }
            }
            __syncwarp();
            for (int t = lane; t < n; t += 32) {
                const int s = path[t];
                if (p.states) p.states[blk * n + t] = (uint16_t)s;
                if (p.hard) p.hard[blk * n + t] = table_entry(p.cb, s, C::S);
            }
            if (p.path_bits) {
                uint8_t *pb = p.path_bits + blk * p.path_stride;
                for (int64_t byte = lane; byte < p.path_stride; byte += 32) {
                    unsigned v = 0;
                    for (int r = 0; r < 8; ++r) {
                        const int64_t pos = byte * 8 + r;
                        int bit = 0;
                        if (pos < C::LB) bit = (path[0] >> (C::LB - 1 - (int)pos)) & 1;
                        else if (pos < nbits) {
                            const int rel = (int)pos - C::LB;
                            bit = (path[1 + rel / KB] >> (KB - 1 - rel % KB)) & 1;
                        }
                        v |= (unsigned)bit << (7 - r);
                    }
                    pb[byte] = (uint8_t)v;
                }
            }
            __syncwarp();
            if (lane == 0) pr.arrive(tb_done + 8u * par);      // this backpointer buffer may be reused
        }
    } else {
        // ============================ compute warps ============================
        const uint32_t tm = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)((warp >> 2) * 128);
        // codebook -> TMEM: column K*K*i + K*j + l = c[j | x_i | l], x_i = tid*BPT + i
#pragma unroll
        for (int i = 0; i < BPT; ++i)
#pragma unroll
            for (int u = 0; u < UNITS; ++u) {
                float2 v[8];
#pragma unroll
                for (int jj = 0; jj < JPU; ++jj)
#pragma unroll
                    for (int l4 = 0; l4 < K; l4 += 4) {
                        const int s0 = (u * JPU + jj) * Q + (tid * BPT + i) * K + l4;
                        float4 c4;
                        if (p.cb) c4 = __ldg(reinterpret_cast<const float4 *>(p.cb + s0));
                        else c4 = make_float4(gaussian_entry(s0, C::S), gaussian_entry(s0 + 1, C::S), gaussian_entry(s0 + 2, C::S), gaussian_entry(s0 + 3, C::S));
                        v[jj * (K / 2) + l4 / 2] = make_float2(c4.x, c4.y);
                        v[jj * (K / 2) + l4 / 2 + 1] = make_float2(c4.z, c4.w);
                    }
                tmem_st16(tm + 16u * (i * UNITS + u), v);
            }
        tmem_wait_st();
        uint32_t it = 0;
        for (int64_t blk = blockIdx.x; blk < p.B; blk += gridDim.x, ++it) {
            const uint32_t par = it & 1u;
            const float *w = p.W + blk * n;
            // the backpointer buffer of this parity was last used two blocks ago: wait until traced
            if (it >= 2) pr.wait(tb_done + 8u * par, ((it >> 1) - 1u) & 1u);
            uint8_t *bp = bp_base + (size_t)par * n * ROWB;
            for (int q = tid; q < Q; q += CT) mv[q] = 0.0;           // mv_1 = 0: free first state
            compute_barrier(CT);
            for (int t = 1; t <= n; ++t) {
                // step t < n: mv_{t+1} from mv_t and w_t;  t = n: final metrics and their argmin
                const int r = (KB * (t - 1)) % QB;
                const double wt = (double)__ldg(w + t - 1);
                uint32_t SJ[K];
#pragma unroll
                for (int j = 0; j < K; ++j) SJ[j] = vit_swz(vit_rotr<QB>((uint32_t)j << (QB - KB), r));
                unsigned long long bytes = 0ull;
                double bv = 0.0;
                int bi = 0x7fffffff;
                float2 cb[2][8];
                tmem_ld16(tm, cb[0]);
#pragma unroll
                for (int i = 0; i < BPT; ++i) {
                    const uint32_t x = (uint32_t)(tid * BPT + i);
                    const uint32_t sx = vit_swz(vit_rotr<QB>(x, r));
                    double in[K], bm[K];
                    unsigned word = 0;                               // branch of output l in bits [KB*l, KB*l + KB)
#pragma unroll
                    for (int j = 0; j < K; ++j) in[j] = mv[sx ^ SJ[j]];
#pragma unroll
                    for (int u = 0; u < UNITS; ++u) {
                        const int g = i * UNITS + u;
                        tmem_wait_ld(cb[g & 1]);
                        if (g + 1 < BPT * UNITS) tmem_ld16(tm + 16u * (g + 1), cb[(g + 1) & 1]);
#pragma unroll
                        for (int jj = 0; jj < JPU; ++jj) {
                            const int j = u * JPU + jj;              // ascending: the lowest branch wins ties
#pragma unroll
                            for (int l = 0; l < K; ++l) {
                                const float2 cp = cb[g & 1][jj * (K / 2) + (l >> 1)];
                                const float c = (l & 1) ? cp.y : cp.x;
                                const double d = __dsub_rn(wt, (double)c);
                                const double mm = __dadd_rn(in[j], __dmul_rn(d, d));
                                if (t < n) {
                                    if (j == 0 || mm < bm[l]) {
                                        bm[l] = mm;
                                        word = (word & ~((unsigned)(K - 1) << (KB * l))) | ((unsigned)j << (KB * l));
                                    }
                                } else {
                                    const int s = (int)((uint32_t)j * Q + x * K + l);
                                    if (bi == 0x7fffffff || mm < bv || (mm == bv && s < bi)) { bv = mm; bi = s; }
                                }
                            }
                        }
                    }
                    if (t < n) {
                        // output [x|l] takes the slot of input [l|x]
#pragma unroll
                        for (int l = 0; l < K; ++l) mv[sx ^ SJ[l]] = bm[l];
                        bytes |= (unsigned long long)word << (WB * i);
                    }
                }
                if (t < n) {
                    // backpointers of step t+1 (row t): 8 contiguous bytes per thread
                    *reinterpret_cast<unsigned long long *>(bp + (size_t)t * ROWB + (size_t)tid * 8) = bytes;
                    compute_barrier(CT);
                } else {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const double ov = __shfl_xor_sync(0xffffffffu, bv, o);
                        const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                        if (ov < bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
                    }
                    if (lane == 0) { redv[warp] = bv; redi[warp] = bi; }
                    compute_barrier(CT);
                    if (tid == 0) {
                        double v = redv[0];
                        int bs = redi[0];
                        for (int z = 1; z < NWARP; ++z)
                            if (redv[z] < v || (redv[z] == v && redi[z] < bs)) { v = redv[z]; bs = redi[z]; }
                        best[par] = bs;
                    }
                    compute_barrier(CT);                             // best[] and every backpointer are written
                }
            }
            __syncwarp();
            if (lane == 0) pr.arrive(tb_ready + 8u * par);         // hand the block to the trace warp
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) tmem_dealloc_512(tmem_base);
}

}  // namespace bcjr
