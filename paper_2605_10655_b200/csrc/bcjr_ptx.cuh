// Inline-PTX helpers shared by the large-trellis kernels (sm_100a): shared-memory and cluster addressing,
// asynchronous remote stores with mbarrier byte accounting, bulk copies, the bounded-wait protocol, packed
// fp32-pair arithmetic and the polynomial exponential.
#pragma once
#include "bcjr_common.cuh"

namespace bcjr {

// ---------------------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v)
{
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, float a, float b, float c, float d)
{
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(a), "f"(b), "f"(c), "f"(d)
                 : "memory");
}
// Asynchronous remote stores: the data lands in the destination CTA's shared memory and the
// destination's mbarrier is credited with the bytes, so the consumer learns that its inputs are
// complete from the mbarrier alone -- no cluster-wide barrier and no fence on the producer side.
__device__ __forceinline__ void st_async_f32(uint32_t addr, float v, uint32_t mbar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(addr), "f"(v), "r"(mbar)
                 : "memory");
}
__device__ __forceinline__ void st_async_v2(uint32_t addr, float a, float b, uint32_t mbar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];" ::"r"(addr), "f"(a),
                 "f"(b), "r"(mbar)
                 : "memory");
}
__device__ __forceinline__ void st_async_v4(uint32_t addr, float a, float b, float c, float d, uint32_t mbar)
{
    asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
                 "f"(a), "f"(b), "f"(c), "f"(d), "r"(mbar)
                 : "memory");
}
// One output either way: a plain store into this CTA's shared memory (own = true, addr in the CTA's
// window) or st.async into a peer's (addr in the cluster window, bytes credited to mbar).  No branch.
__device__ __forceinline__ void push_v2(bool own, uint32_t addr, float a, float b, uint32_t mbar)
{
    asm volatile(
        "{ .reg .pred p; setp.ne.u32 p, %0, 0;\n"
        "@p st.shared.v2.f32 [%1], {%2, %3};\n"
        "@!p st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%1], {%2, %3}, [%4]; }" ::"r"((uint32_t)own),
        "r"(addr), "f"(a), "f"(b), "r"(mbar)
        : "memory");
}
__device__ __forceinline__ void push_v4(bool own, uint32_t addr, float a, float b, float c, float d, uint32_t mbar)
{
    asm volatile(
        "{ .reg .pred p; setp.ne.u32 p, %0, 0;\n"
        "@p st.shared.v4.f32 [%1], {%2, %3, %4, %5};\n"
        "@!p st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%1], {%2, %3, %4, %5}, [%6]; }" ::"r"((uint32_t)own),
        "r"(addr), "f"(a), "f"(b), "f"(c), "f"(d), "r"(mbar)
        : "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_sync() { cluster_arrive(); cluster_wait(); }
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_id_x()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_count_x()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_store(void *gdst, uint32_t ssrc, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(ssrc), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read0() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all0() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_load(uint32_t sdst, const void *gsrc, uint32_t bytes, uint32_t mbar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(sdst),
                 "l"(gsrc), "r"(bytes), "r"(mbar)
                 : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t mbar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(mbar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t mbar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(mbar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t mbar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
    return ok != 0;
}
// The same probe, but the thread may be parked by the hardware for up to `ns` nanoseconds while the phase is
// incomplete: a waiting warp then costs the SM's schedulers a handful of instructions instead of a busy loop.
__device__ __forceinline__ bool mbar_try_wait_parked(uint32_t mbar, uint32_t parity, uint32_t ns)
{
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok) : "r"(mbar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
// Device-side waits are bounded by wall time (the context's wait budget, default 2 s): a wait that
// runs out raises BCJR_ETIMEOUT (-6) in the diagnostics and sets the CTA-wide abort flag; the kernel
// then runs to its end on meaningless numbers instead of hanging (see Proto below).
__device__ __forceinline__ unsigned long long global_timer_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// After a wait has run out the threads no longer wait for their inputs, so asynchronous copies may
// still be on their way into this CTA's shared memory when the kernel reaches its end.  Leaving
// with copies in flight is not allowed: the thread that requested bulk loads waits for each of the
// last `depth` of them (time-bounded, ignoring the abort flag), and every thread lets the
// st.async traffic addressed to this CTA land (a fixed, short delay) before the CTA exits.
__device__ __forceinline__ void drain_bulk_loads(uint32_t mbar_base, uint32_t issued, uint32_t depth, DeviceDiag *diag)
{
    const unsigned long long limit = diag->wait_limit_ns;
    for (uint32_t c = issued > depth ? issued - depth : 0u; c < issued; ++c) {
        const uint32_t mbar = mbar_base + 8u * (c % depth), parity = (c / depth) & 1u;
        const unsigned long long t0 = global_timer_ns();
        for (int outer = 0; outer < (1 << 22); ++outer) {
            if (mbar_try_wait(mbar, parity)) break;
            if (global_timer_ns() - t0 > limit) break;
        }
    }
}
__device__ __forceinline__ void settle_after_abort()
{
    const unsigned long long t0 = global_timer_ns();
    for (int i = 0; i < (1 << 16) && global_timer_ns() - t0 < 200000ull; ++i) __nanosleep(1000);
}
__device__ __forceinline__ void mbar_arrive_local(uint32_t mbar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
}
// Relaxed arrival on a (possibly remote) mbarrier of the cluster: it publishes nothing by itself.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t remote_mbar)
{
    asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_mbar) : "memory");
}
// Protocol operations of one thread.  `live` turns false when one of this thread's waits runs out
// (or finds that another thread of the CTA has given up).  A thread that is not live issues no
// further mbarrier arrivals, transaction announcements, asynchronous stores or bulk copies, but
// still reaches every CTA and cluster barrier, on meaningless numbers.  Two forms are used:
//   * per operation: the guarded members below (arrive, expect_tx, load, store, async_*);
//   * per step: the hot kernels take a warp-uniform vote (warp_live) right after the step's first
//     wait and skip the step's work when a lane is dead; inside an admitted step the operations
//     are issued unguarded, so a wait that runs out in mid-step lets the thread finish that one
//     step.  Either way a thread is at most one step ahead of the last completed phase when it
//     stops, so no transaction count runs away and nothing is issued after the last barrier.
struct Proto {
    uint32_t live;
    volatile int *abort_flag;
    DeviceDiag *diag;
    __device__ __forceinline__ void wait(uint32_t mbar, uint32_t parity)
    {
        if (mbar_try_wait(mbar, parity)) return;                 // fast path: one probe
        if (!live) return;
        if (*abort_flag) { live = 0u; return; }
        unsigned long long t0 = 0;
        for (int i = 0; i < (1 << 22); ++i) {                    // hard cap besides the time budget
            if (mbar_try_wait_parked(mbar, parity, 4000u)) return;
            if ((i & 63) == 63) {
                const unsigned long long now = global_timer_ns();
                if (t0 == 0) t0 = now;
                if (*abort_flag || now - t0 > diag->wait_limit_ns) break;
            }
        }
        live = 0u;
        *abort_flag = 1;
        atomicCAS(&diag->status, 0, -6);
    }
    // warp-uniform liveness, taken once per step: a warp with a dead lane stops as a whole
    __device__ __forceinline__ bool warp_live()
    {
        live = __all_sync(0xffffffffu, live != 0u) ? 1u : 0u;
        return live != 0u;
    }
    __device__ __forceinline__ void arrive(uint32_t mbar) const
    {
        if (live) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(mbar) : "memory");
    }
    __device__ __forceinline__ void arrive_cluster(uint32_t remote_mbar) const
    {
        if (live) asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote_mbar) : "memory");
    }
    __device__ __forceinline__ void expect_tx(uint32_t mbar, uint32_t bytes) const { if (live) mbar_expect_tx(mbar, bytes); }
    __device__ __forceinline__ void load(uint32_t sdst, const void *gsrc, uint32_t bytes, uint32_t mbar) const
    {
        if (live) bulk_load(sdst, gsrc, bytes, mbar);
    }
    __device__ __forceinline__ void store(void *gdst, uint32_t ssrc, uint32_t bytes) const { if (live) bulk_store(gdst, ssrc, bytes); }
    __device__ __forceinline__ void async_f32(uint32_t addr, float v, uint32_t mbar) const { if (live) st_async_f32(addr, v, mbar); }
    __device__ __forceinline__ void async_v2(uint32_t addr, float a, float b, uint32_t mbar) const { if (live) st_async_v2(addr, a, b, mbar); }
    __device__ __forceinline__ void async_v4(uint32_t addr, float a, float b, float c, float d, uint32_t mbar) const
    {
        if (live) st_async_v4(addr, a, b, c, d, mbar);
    }
};

// non-blocking probe of a phase
__device__ __forceinline__ bool mbar_test(uint32_t mbar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok) : "r"(mbar), "r"(parity) : "memory");
    return ok != 0;
}

// ---------------------------------------------------------------------------- packed fp32 pairs
// sm_100 executes add/mul/fma on two packed fp32 values per instruction (f32x2): the kernels
// keep every per-state quantity as a pair so that the FP32 instruction count per state halves
// and the special-function unit, not instruction issue, is the binding pipe.
__device__ __forceinline__ float2 add2(float2 a, float2 b)
{
    float2 d;
    asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; add.rn.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 sub2(float2 a, float2 b)
{
    float2 d;
    asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; sub.rn.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b)
{
    float2 d;
    asm("{ .reg .b64 ra, rb, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mul.rn.f32x2 rd, ra, rb; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y));
    return d;
}
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c)
{
    float2 d;
    asm("{ .reg .b64 ra, rb, rc, rd; mov.b64 ra, {%2, %3}; mov.b64 rb, {%4, %5}; mov.b64 rc, {%6, %7}; "
        "fma.rn.f32x2 rd, ra, rb, rc; mov.b64 {%0, %1}, rd; }"
        : "=f"(d.x), "=f"(d.y) : "f"(a.x), "f"(a.y), "f"(b.x), "f"(b.y), "f"(c.x), "f"(c.y));
    return d;
}
__device__ __forceinline__ float2 splat2(float v) { return make_float2(v, v); }
// log2-potential of a pair of states plus a message: du (du (-lam2) + kap) + msg, see step_energy
__device__ __forceinline__ float2 energy2(float2 du, float2 nl2, float2 kap2, float2 msg)
{
    return fma2(du, fma2(du, nl2, kap2), msg);
}
__device__ __forceinline__ float2 ex2f2(float2 a) { return make_float2(ex2f(a.x), ex2f(a.y)); }
__device__ __forceinline__ float2 lg2f2(float2 a) { return make_float2(lg2f(a.x), lg2f(a.y)); }
__device__ __forceinline__ float2 rcpf2(float2 a) { return make_float2(rcpf(a.x), rcpf(a.y)); }
// 2^x for x <= 0 on the FP32 pipe (no special-function instruction): x = n + f with n the nearest
// integer and |f| <= 1/2, 2^f by the degree-5 interpolant at the Chebyshev nodes of [-1/2, 1/2] (relative
// error 2.4e-7 evaluated in float32, about that of ex2.approx), the
// factor 2^n by an add on the exponent field.  Arguments below -125 are clamped (the result there
// is ~2e-38 against a group maximum of 1, far below anything the sums can see).
__device__ __forceinline__ float2 ex2_poly2(float2 x)
{
    x.x = fmaxf(x.x, -125.f); x.y = fmaxf(x.y, -125.f);
    const float2 magic = splat2(12582912.f);                     // 1.5 * 2^23: adding it rounds to the nearest integer
    const float2 t = add2(x, magic);
    const float2 n = sub2(t, magic);
    const float2 f = sub2(x, n);
    float2 p = fma2(splat2(1.3390863e-3f), f, splat2(9.6760318e-3f));
    p = fma2(p, f, splat2(5.5503570e-2f));
    p = fma2(p, f, splat2(2.4022107e-1f));
    p = fma2(p, f, splat2(6.9314718e-1f));
    p = fma2(p, f, splat2(1.0000001f));
    // t = 1.5 * 2^23 + n exactly, so its low mantissa bits hold n (two's complement): shift them onto the exponent
    p.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
    p.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
    return p;
}
__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// elementwise max over N pairs
template <int N>
__device__ __forceinline__ float2 max_pairs(const float2 (&a)[N])
{
    float2 m = a[0];
    int j = 1;
#pragma unroll
    for (; j + 1 < N; j += 2) { m.x = max3f(m.x, a[j].x, a[j + 1].x); m.y = max3f(m.y, a[j].y, a[j + 1].y); }
    if (j < N) { m.x = fmaxf(m.x, a[j].x); m.y = fmaxf(m.y, a[j].y); }
    return m;
}

// max over up to 64 per-warp slots, two per lane
__device__ __forceinline__ float slot_max(const float *slots, int lane, int count)
{
    float v = lane < count ? slots[lane] : __int_as_float(0xff800000);
    if (lane + 32 < count) v = fmaxf(v, slots[lane + 32]);
    return v;
}

}  // namespace bcjr
