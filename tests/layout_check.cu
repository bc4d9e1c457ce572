// Host-side check of the index arithmetic the 2^16-state backward kernels rely on (no GPU needed): the
// functions below are the kernels' own (constexpr, host and device), compiled here for the host.
//   1. bwd_skew_kernel: (CTA, thread, slot) <-> butterfly is a bijection; every output has one destination entry;
//      the butterfly a thread computes FIRST in a step depends on none of those computed LAST in the step before
//      (alpha order 0,1,2,3; beta order 2,0,3,1); alpha slots 0,1 feed the own CTA, slots 2,3 the peer.
//   3. fwd_vec2_kernel: production, consumer CTA and reader's address of every group in both sweeps.
//   2. bwd_alpha_kernel<2>, <3> (and the same sweeps inside bwd_solo_kernel, whose in-place beta sweep is checked too): the in-place slot function is a bijection, XOR-linear over the bit fields the
//      kernel combines, consistent from one step to the next (output [x|l] takes the slot of input [l|x]), and a
//      warp's 32 lanes always reach 32 different banks.
#include <cstdio>
#include <set>
#include <vector>

#include "../paper_2605_10655_b200/csrc/bcjr_bsolo.cuh"
#include "../paper_2605_10655_b200/csrc/bcjr_vec2.cuh"

using namespace bcjr;

static int fails = 0;
#define CHECK(cond, ...) do { if (!(cond)) { if (fails < 20) { std::printf("FAIL %s:%d: ", __FILE__, __LINE__); std::printf(__VA_ARGS__); std::printf("\n"); } ++fails; } } while (0)

static void check_skew()
{
    using C = SkewCfg;
    std::set<int> seen;
    for (int r = 0; r < 2; ++r)
        for (int t = 0; t < 512; ++t)
            for (int s = 0; s < 4; ++s) {
                const int x = C::x_of(r, t, s);
                CHECK(x >= 0 && x < C::NB && seen.insert(x).second, "x_of not injective at (%d,%d,%d)", r, t, s);
                CHECK(C::rank_of(x) == r && C::slot_of(x) == s && C::tid_of(x) == t, "inverse of x_of at %d", x);
            }
    const int beta_pos[4] = {1, 3, 0, 2};                 // position of slot s in the beta order 2,0,3,1
    std::set<long> dest_a, dest_b;
    for (int x = 0; x < C::NB; ++x) {
        const int r = C::rank_of(x), s = C::slot_of(x);
        for (int l = 0; l < 4; ++l) {                     // alpha: L'([x|l]) is input x >> 10 of butterfly ((x & 1023) << 2) | l
            const int x2 = ((x & 1023) << 2) | l, j2 = x >> 10;
            CHECK((C::rank_of(x2) == r) == (s < 2), "alpha destination CTA of slot %d", s);
            dest_a.insert((long)C::rank_of(x2) * 65536 + (C::slot_of(x2) * 4 + j2) * 512 + C::tid_of(x2));
            CHECK(!(C::slot_of(x2) == 0 && s == 3), "alpha: first butterfly depends on a last one (x=%d)", x);
            CHECK(C::tid_of((x & 1023) << 2) % 4 == 0 && C::tid_of(x2) == C::tid_of((x & 1023) << 2) + l, "alpha outputs not one 16-byte entry");
        }
        for (int j = 0; j < 4; ++j) {                     // beta: M'([j|x]) is input x & 3 of butterfly (j << 10) | (x >> 2)
            const int x1 = (j << 10) | (x >> 2);
            CHECK(C::rank_of(x1) == (j >> 1), "beta destination CTA");
            dest_b.insert((long)C::rank_of(x1) * 65536 + ((x & 3) * 2048 + C::slot_of(x1) * 512 + C::tid_of(x1)));
            CHECK(!(beta_pos[C::slot_of(x1)] == 0 && beta_pos[s] == 3), "beta: first butterfly depends on a last one (x=%d)", x);
            // what the kernel assumes about the two outputs of a pair: next slot (own CTA) / upper half of the threads (peer)
            if ((j & 1) == 0) {
                const int y = ((j + 1) << 10) | (x >> 2);
                if (C::rank_of(x1) == r) CHECK(C::slot_of(y) == C::slot_of(x1) + 1 && C::tid_of(y) == C::tid_of(x1), "beta own-CTA pair");
                else CHECK(C::slot_of(y) == C::slot_of(x1) && C::tid_of(y) == C::tid_of(x1) + 256, "beta peer pair");
            }
        }
    }
    CHECK(dest_a.size() == 2u * 8192u && dest_b.size() == 2u * 8192u, "destinations not a bijection");
}

template <int KB>
static void check_alpha()
{
    using C = AlphaCfg<KB>;
    constexpr int QB = C::QB, K = C::K;
    for (int step = 0; step < 3 * QB; ++step) {
        const int r = (KB * step) % QB, r2 = (KB * (step + 1)) % QB;
        std::vector<char> used(1 << QB, 0);
        for (uint32_t q = 0; q < (1u << QB); ++q) {
            const uint32_t s = C::slot(q, r);
            CHECK(s < (1u << QB) && !used[s], "slot not a bijection (k=%d r=%d)", KB, r);
            used[s] = 1;
        }
        for (int i = 0; i < C::BPT; ++i)
            for (int j = 0; j < K; ++j)
                for (int w = 0; w < 16; ++w) {
                    std::set<uint32_t> banks;
                    for (int l = 0; l < 32; ++l) {
                        const uint32_t tid = w * 32 + l, x = ((uint32_t)i << 9) | tid, q = ((uint32_t)j << (QB - KB)) | x;
                        const uint32_t s = C::slot(q, r);
                        CHECK(s == (C::slot((uint32_t)i << 9, r) ^ C::slot(tid, r) ^ C::slot((uint32_t)j << (QB - KB), r)), "slot not XOR-linear");
                        banks.insert(s & 31u);
                        // in place: output [x|l'] of this step is found next step where input [l'|x] was
                        CHECK(C::slot(((x << KB) | (uint32_t)j) & ((1u << QB) - 1u), r2) == s, "in-place slots inconsistent (k=%d)", KB);
                    }
                    CHECK(banks.size() == 32u, "bank conflict (k=%d r=%d)", KB, r);
                }
    }
}

// bwd_solo_kernel's in-place beta sweep: input b of butterfly x is group (x << k) | b at rotation rr; output j takes
// the slot of input j and must be where the next step (rotation rr - k) looks for group (j << (QB - k)) | x.
static void check_beta_in_place()
{
    using C = BSoloCfg;
    constexpr int QB = C::QB, K = C::K, KB = C::KB;
    int rr = 0;
    for (int step = 0; step < 3 * QB; ++step) {
        const int rr2 = rr == 0 ? QB - KB : rr - KB;
        for (int i = 0; i < C::BPT; ++i)
            for (int b = 0; b < K; ++b)
                for (int w = 0; w < 16; ++w) {
                    std::set<uint32_t> banks;
                    for (int l = 0; l < 32; ++l) {
                        const int tid = w * 32 + l;
                        const uint32_t x = (uint32_t)(i * C::THREADS + tid), q = C::beta_q(i, tid, b);
                        const uint32_t s = C::slot(q, rr);
                        CHECK(s == (C::slot(C::beta_q(i, 0, 0), rr) ^ C::slot(C::beta_q(0, tid, 0), rr) ^ C::slot((uint32_t)b, rr)), "beta slot not XOR-linear");
                        banks.insert(s & 31u);
                        CHECK(C::slot(((uint32_t)b << (QB - KB)) | x, rr2) == s, "beta in-place slots inconsistent (rr=%d)", rr);
                    }
                    CHECK(banks.size() == 32u, "beta bank conflict (rr=%d)", rr);
                }
        rr = rr2;
    }
}

// fwd_vec2_kernel: every group is produced once per sweep, lands in the CTA that reads it, at the place its reader looks
static void check_vec2()
{
    using C = Vec2Cfg<3>;
    // alpha: entry i = j * 256 + x of L is read by the threads of butterfly x as input j
    std::vector<int> seen(C::Q, 0);
    for (int rank = 0; rank < 2; ++rank)
        for (int tid = 0; tid < C::THREADS; ++tid) {
            const int q0 = C::alpha_q0(rank, tid);
            for (int e = 0; e < 4; ++e) {
                const int i = q0 + e, j = i >> 8, x = i & 255, rc = x >> 7;
                ++seen[i];
                CHECK(C::alpha_dst_rank(q0) == rc, "alpha: consumer CTA of group %d", i);
                // a reader of butterfly x in CTA rc: tid' with (rc * 2048 + 4 tid') >> 4 == x
                const int tidr = (x & 127) << 2;
                CHECK((C::alpha_q0(rc, tidr) >> 4) == x && C::alpha_dst_off(q0) + e == C::alpha_in(tidr) + 128 * j, "alpha: group %d not where its reader looks", i);
            }
            CHECK(C::alpha_dst_off(q0) % 4 == 0, "alpha push not 16-byte aligned");
        }
    for (int i = 0; i < C::Q; ++i) CHECK(seen[i] == 1, "alpha: group %d produced %d times", i, seen[i]);
    // beta: entry i = (x << 4) | b of M is read by the thread that owns butterflies 2 xp, 2 xp + 1 (x >> 1 == xp) as part of one float4
    std::fill(seen.begin(), seen.end(), 0);
    for (int rank = 0; rank < 2; ++rank)
        for (int warp = 0; warp < 16; ++warp)
            for (int lane = 0; lane < 32; ++lane)
                for (int pp = 0; pp < 2; ++pp) {
                    const int q = C::beta_q0(rank, warp, lane, pp);
                    CHECK(q == C::beta_q0(rank, warp, lane, 0) + 256 * pp && ((q & 255) >> 7) == rank && q % 2 == 0, "beta: ownership of group %d", q);
                    CHECK(C::beta_dst_rank(q) == C::beta_dst_rank(C::beta_q0(rank, warp, lane, 0)), "beta: the two pairs of a thread go to different CTAs");
                    CHECK(C::beta_dst_off(q) - C::beta_dst_off(C::beta_q0(rank, warp, lane, 0)) == pp * (C::beta_dst_off(256) - C::beta_dst_off(0)), "beta: pair offset");
                    for (int e = 0; e < 2; ++e) {
                        const int i = q + e, x = i >> 4, b = i & 15, rc = x >> 7;
                        ++seen[i];
                        CHECK(C::beta_dst_rank(q) == rc && C::beta_dst_off(q) + e == C::beta_dst_off(i), "beta: consumer of group %d", i);
                        // the reader: CTA rc, xp = (x & 127) >> 1 -> lane' = xp & 31, warp' & 1 = xp >> 5
                        const int xp = (x & 127) >> 1;
                        const int want = C::beta_in(xp >> 5, xp & 31) + 256 * (b >> 1) + 2 * (x & 1) + (b & 1);
                        CHECK(C::beta_dst_off(i) == want, "beta: group %d not where its reader looks", i);
                    }
                    CHECK(C::beta_dst_off(q) % 2 == 0, "beta push not 8-byte aligned");
                }
    for (int i = 0; i < C::Q; ++i) CHECK(seen[i] == 1, "beta: group %d produced %d times", i, seen[i]);
}

int main()
{
    check_vec2();
    check_beta_in_place();
    check_skew();
    check_alpha<2>();
    check_alpha<3>();
    if (fails) std::printf("%d checks failed\n", fails);
    else std::printf("layouts ok\n");
    return fails ? 1 : 0;
}
