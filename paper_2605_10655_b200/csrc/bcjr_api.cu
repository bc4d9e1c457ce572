// Host side of the C ABI declared in include/bcjr_b200.h: argument checks, scratch
// management, kernel selection and launches.  No compute happens on the host.
#include "../../include/bcjr_b200.h"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>

#include "bcjr_common.cuh"
#include "bcjr_generic.cuh"
#ifndef BCJR_NO_CLUSTER
#include "bcjr_cluster.cuh"
#include "bcjr_vec.cuh"
#include "bcjr_vec4.cuh"
#include "bcjr_vec2.cuh"
#include "bcjr_qat.cuh"
#include "bcjr_rht.cuh"
#include "bcjr_solo.cuh"
#include "bcjr_duo.cuh"
#include "bcjr_skew.cuh"
#include "bcjr_alpha.cuh"
#include "bcjr_bsolo.cuh"
#include "bcjr_ckpt.cuh"
#include "bcjr_warp.cuh"
#include "bcjr_viterbi.cuh"
#endif

using namespace bcjr;

namespace {

const unsigned long long kDefaultWaitLimitNs = 2000000000ull;   // 2 s per device-side wait

struct Buffer {
    void *ptr = nullptr;
    size_t bytes = 0;
};

}  // namespace

struct bcjr_ctx {
    int device = 0;
    int num_sms = 0;
    int max_smem_optin = 0;
    Buffer hist, stepO, msg, gc_part, soft_copy, bp, path_ws, cb_beta, grad_w, grad_c, blk_defect, gauss_cb, staging[6];
    DeviceDiag *diag = nullptr;
    // saved by bcjr_soft_quantize for bcjr_backward
    bool have_fwd = false;
    bool cb_computed = false;  // the call in flight (and the saved forward state) uses the computed Gaussian emission
    const float *W = nullptr, *cb = nullptr;
    int Lb = 0, k = 0, n = 0;
    int V = 1;                 // numbers emitted per state and step by the saved forward call
    int64_t B = 0;
    float T = 0.f;
    // options
    int opt_path = 0;
    int opt_max_ctas = 0;
    int opt_bwd_variant = 0;   // 0 = alpha kernel + two-CTA beta kernel (without grad_codebook at k = 2: one-CTA kernel), 1 = register-accumulator
                               // cluster kernel, 2 = fused two-CTA TMEM kernel, 3 = fused with skewed slot order, 4 = two-kernel call always
    int opt_fwd_variant = 0;   // 0 = TMEM single-CTA forward kernel where it applies, 1 = cluster forward kernel
    int opt_record_defect = 0; // forward calls record the posterior defect of every block
    int opt_hist_every = 1;    // large-trellis forward call: keep L_t of every m-th step, recompute the others in the beta sweep
    int64_t defect_blocks = 0; // blocks covered by the last recording
    int launches = 0;
    int last_path = 0;
    std::string cuda_error;
};

namespace {

bcjr_status cuda_fail(bcjr_ctx *ctx, cudaError_t e, const char *what)
{
    ctx->cuda_error = std::string(what) + ": " + cudaGetErrorString(e);
    cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? BCJR_ENOMEM : BCJR_ECUDA;
}

#define CU(call)                                                        \
    do {                                                                \
        cudaError_t e__ = (call);                                       \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, #call);      \
    } while (0)

bcjr_status ensure(bcjr_ctx *ctx, Buffer &b, size_t bytes)
{
    if (bytes <= b.bytes) return BCJR_OK;
    if (b.ptr) { CU(cudaFree(b.ptr)); b.ptr = nullptr; b.bytes = 0; }
    CU(cudaMalloc(&b.ptr, bytes));
    b.bytes = bytes;
    return BCJR_OK;
}

// Computed Gaussian emission (a NULL codebook): the tensor-memory kernels evaluate the entries themselves while
// staging; every other kernel reads a table, so the context keeps one written by gaussian_table_kernel.
bcjr_status computed_table(bcjr_ctx *ctx, int Lb, cudaStream_t st, const float **table)
{
    const int S = 1 << Lb;
    bcjr_status rc = ensure(ctx, ctx->gauss_cb, (size_t)(1 << 16) * 4);
    if (rc) return rc;
    gaussian_table_kernel<<<(S + 255) / 256, 256, 0, st>>>((float *)ctx->gauss_cb.ptr, S);
    ctx->launches += 1;
    CU(cudaGetLastError());
    *table = (const float *)ctx->gauss_cb.ptr;
    return BCJR_OK;
}

bcjr_status check_dims(int Lb, int k, int n, int64_t B)
{
    if (k < 1 || k > 4 || Lb < k || Lb > 16 || n < 1 || B < 0) return BCJR_EINVAL;
    if (Lb - k > 14) return BCJR_EUNSUPPORTED;
    if ((int64_t)n * (int64_t)(1 << (Lb - k)) > ((int64_t)1 << 31)) return BCJR_EUNSUPPORTED;
    return BCJR_OK;
}

int generic_threads(int Q)
{
    int t = (Q + 31) / 32 * 32;
    if (t < 32) t = 32;
    return t > GEN_MAX_THREADS ? GEN_MAX_THREADS : t;
}

struct GenericLaunch {
    int threads, grid;
    size_t smem;
    bool msg_global;
};

template <typename Kern>
bcjr_status plan_generic(bcjr_ctx *ctx, Kern kern, int Q, size_t msg_bytes, int64_t B, GenericLaunch *out,
                         int header_floats = GEN_SMEM_HEADER)
{
    out->threads = generic_threads(Q);
    const size_t header = (size_t)header_floats * sizeof(float);
    const size_t budget = (size_t)ctx->max_smem_optin - 1024;
    out->msg_global = header + msg_bytes > budget;
    out->smem = out->msg_global ? header : header + msg_bytes;
    CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    int occ = 0;
    CU(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kern, out->threads, out->smem));
    if (occ < 1) occ = 1;
    int64_t grid = (int64_t)occ * ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && grid > ctx->opt_max_ctas) grid = ctx->opt_max_ctas;
    if (grid > B) grid = B;
    if (grid < 1) grid = 1;
    out->grid = (int)grid;
    return BCJR_OK;
}

template <int KB>
bcjr_status launch_fwd_generic(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    const int Q = 1 << (p.Lb - KB);
    GenericLaunch gl;
    bcjr_status rc = plan_generic(ctx, fwd_generic_kernel<KB>, Q, (size_t)2 * Q * 4, p.B, &gl);
    if (rc) return rc;
    if ((rc = ensure(ctx, ctx->hist, (size_t)gl.grid * p.n * Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->stepO, (size_t)gl.grid * (p.n + 2) * 4))) return rc;
    if (gl.msg_global && (rc = ensure(ctx, ctx->msg, (size_t)gl.grid * 2 * Q * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.stepO = (int *)ctx->stepO.ptr;
    p.msg = gl.msg_global ? (float *)ctx->msg.ptr : nullptr;
    fwd_generic_kernel<KB><<<gl.grid, gl.threads, gl.smem, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

template <int KB>
bcjr_status launch_bwd_generic(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st)
{
    const int S = 1 << p.Lb, Q = S >> KB;
    GenericLaunch gl;
    bcjr_status rc = plan_generic(ctx, bwd_generic_kernel<KB>, Q, (size_t)4 * Q * 4, p.B, &gl);
    if (rc) return rc;
    if ((rc = ensure(ctx, ctx->hist, (size_t)gl.grid * 2 * p.n * Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->stepO, (size_t)gl.grid * (p.n + 2) * 4))) return rc;
    if ((rc = ensure(ctx, ctx->gc_part, (size_t)gl.grid * S * 4))) return rc;
    if (gl.msg_global && (rc = ensure(ctx, ctx->msg, (size_t)gl.grid * 4 * Q * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.stepO = (int *)ctx->stepO.ptr;
    p.gc_part = (float *)ctx->gc_part.ptr;
    p.msg = gl.msg_global ? (float *)ctx->msg.ptr : nullptr;
    bwd_generic_kernel<KB><<<gl.grid, gl.threads, gl.smem, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    if (grad_codebook) {
        reduce_gc_kernel<<<(S + 255) / 256, 256, 0, st>>>(p.gc_part, gl.grid, S, grad_codebook);
        ctx->launches += 1;
        CU(cudaGetLastError());
    }
    return BCJR_OK;
}

template <int KB>
bcjr_status launch_vit_generic(bcjr_ctx *ctx, VitParams p, cudaStream_t st)
{
    const int Q = 1 << (p.Lb - KB);
    GenericLaunch gl;
    bcjr_status rc = plan_generic(ctx, viterbi_generic_kernel<KB>, Q, (size_t)2 * Q * 8, p.B, &gl);
    if (rc) return rc;
    if ((rc = ensure(ctx, ctx->bp, (size_t)gl.grid * p.n * Q))) return rc;
    if ((rc = ensure(ctx, ctx->path_ws, (size_t)gl.grid * p.n * 4))) return rc;
    if (gl.msg_global && (rc = ensure(ctx, ctx->msg, (size_t)gl.grid * 2 * Q * 8))) return rc;
    p.bp = (uint8_t *)ctx->bp.ptr;
    p.path_ws = (int *)ctx->path_ws.ptr;
    p.msg = gl.msg_global ? (double *)ctx->msg.ptr : nullptr;
    viterbi_generic_kernel<KB><<<gl.grid, gl.threads, gl.smem, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

// ---- vector emissions (V weights per step, KB = k V bits per step): one CTA per block
template <int KB, int V>
bcjr_status launch_fwd_vec(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    const int Q = 1 << (p.Lb - KB), nt = p.n / V;
    GenericLaunch gl;
    bcjr_status rc = plan_generic(ctx, fwd_vec_kernel<KB, V>, Q, (size_t)2 * Q * 4, p.B, &gl, VEC_SMEM_HEADER);
    if (rc) return rc;
    if ((rc = ensure(ctx, ctx->hist, (size_t)gl.grid * nt * Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->stepO, (size_t)gl.grid * (nt + 2) * 4))) return rc;
    if (gl.msg_global && (rc = ensure(ctx, ctx->msg, (size_t)gl.grid * 2 * Q * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.stepO = (int *)ctx->stepO.ptr;
    p.msg = gl.msg_global ? (float *)ctx->msg.ptr : nullptr;
    const int SV = (1 << p.Lb) * V;
    if ((rc = ensure(ctx, ctx->cb_beta, (size_t)SV * 4))) return rc;
    regroup_table_kernel<<<(SV + 255) / 256, 256, 0, st>>>(p.cb, (float *)ctx->cb_beta.ptr, 1 << p.Lb, KB, V);
    p.cb_beta = (const float *)ctx->cb_beta.ptr;
    fwd_vec_kernel<KB, V><<<gl.grid, gl.threads, gl.smem, st>>>(p);
    ctx->launches += 2;
    CU(cudaGetLastError());
    return BCJR_OK;
}

template <int KB, int V>
bcjr_status launch_bwd_vec(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st)
{
    const int S = 1 << p.Lb, Q = S >> KB, nt = p.n / V;
    GenericLaunch gl;
    bcjr_status rc = plan_generic(ctx, bwd_vec_kernel<KB, V>, Q, (size_t)4 * Q * 4, p.B, &gl, VEC_SMEM_HEADER);
    if (rc) return rc;
    if ((rc = ensure(ctx, ctx->hist, (size_t)gl.grid * 2 * nt * Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->stepO, (size_t)gl.grid * (nt + 2) * 4))) return rc;
    if ((rc = ensure(ctx, ctx->gc_part, (size_t)gl.grid * S * V * 4))) return rc;
    if (gl.msg_global && (rc = ensure(ctx, ctx->msg, (size_t)gl.grid * 4 * Q * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.stepO = (int *)ctx->stepO.ptr;
    p.gc_part = (float *)ctx->gc_part.ptr;
    p.msg = gl.msg_global ? (float *)ctx->msg.ptr : nullptr;
    // the regrouped table of the forward call may be stale (another call in between): rebuild it
    if ((rc = ensure(ctx, ctx->cb_beta, (size_t)S * V * 4))) return rc;
    regroup_table_kernel<<<(S * V + 255) / 256, 256, 0, st>>>(p.cb, (float *)ctx->cb_beta.ptr, S, KB, V);
    p.cb_beta = (const float *)ctx->cb_beta.ptr;
    bwd_vec_kernel<KB, V><<<gl.grid, gl.threads, gl.smem, st>>>(p);
    ctx->launches += 2;
    CU(cudaGetLastError());
    if (grad_codebook) {
        reduce_gc_vec_kernel<<<(S * V + 255) / 256, 256, 0, st>>>(p.gc_part, gl.grid, S, KB, V, grad_codebook);
        ctx->launches += 1;
        CU(cudaGetLastError());
    }
    return BCJR_OK;
}

template <int KB, int V>
bcjr_status launch_vit_vec(bcjr_ctx *ctx, VitParams p, cudaStream_t st)
{
    const int Q = 1 << (p.Lb - KB), nt = p.n / V;
    GenericLaunch gl;
    bcjr_status rc = plan_generic(ctx, viterbi_vec_kernel<KB, V>, Q, (size_t)2 * Q * 8, p.B, &gl, VEC_SMEM_HEADER);
    if (rc) return rc;
    if ((rc = ensure(ctx, ctx->bp, (size_t)gl.grid * nt * Q))) return rc;
    if ((rc = ensure(ctx, ctx->path_ws, (size_t)gl.grid * nt * 4))) return rc;
    if (gl.msg_global && (rc = ensure(ctx, ctx->msg, (size_t)gl.grid * 2 * Q * 8))) return rc;
    p.bp = (uint8_t *)ctx->bp.ptr;
    p.path_ws = (int *)ctx->path_ws.ptr;
    p.msg = gl.msg_global ? (double *)ctx->msg.ptr : nullptr;
    viterbi_vec_kernel<KB, V><<<gl.grid, gl.threads, gl.smem, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

// V = 2 only: (k, V) = (1, 2) and (2, 2); every array that is read two floats at a time must be 8-byte aligned
bcjr_status check_vec(int Lb, int k, int V, int n, int64_t B)
{
    if (V < 1 || k < 1 || n < 1 || B < 0 || n % V) return BCJR_EINVAL;
    if (V != 2 || k > 2) return BCJR_EUNSUPPORTED;
    return check_dims(Lb, k * V, n / V, B);
}
bool aligned8(const void *p) { return ((uintptr_t)p & 7u) == 0; }

#ifndef BCJR_NO_CLUSTER
#ifndef FWD_THREADS_K2
#define FWD_THREADS_K2 512
#endif
#ifndef FWD_CL_K2
#define FWD_CL_K2 2
#endif
// One cluster of CL CTAs per weight block in flight; the grid is the number of clusters the
// GPU can hold at once (persistent loop over blocks inside the kernel).
template <typename Kern>
bcjr_status plan_cluster(bcjr_ctx *ctx, Kern kern, int CL, int threads, size_t smem, int64_t B,
                         cudaLaunchConfig_t *cfg, cudaLaunchAttribute *attr, cudaStream_t st)
{
    CU(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = CL;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg->gridDim = dim3(CL * ctx->num_sms, 1, 1);
    cfg->blockDim = dim3(threads, 1, 1);
    cfg->dynamicSmemBytes = smem;
    cfg->stream = st;
    cfg->attrs = attr;
    cfg->numAttrs = 1;
    int ncl = 0;
    CU(cudaOccupancyMaxActiveClusters(&ncl, kern, cfg));
    if (ncl < 1) return BCJR_EUNSUPPORTED;
    if (ctx->opt_max_ctas > 0 && ncl > ctx->opt_max_ctas / CL) ncl = ctx->opt_max_ctas / CL > 0 ? ctx->opt_max_ctas / CL : 1;
    if (ncl > B) ncl = (int)B;
    cfg->gridDim = dim3(CL * ncl, 1, 1);
    return BCJR_OK;
}

// Lb = 16, 4 bits and 2 weights per step: one block per cluster of four CTAs, table slice in shared memory
// blocks in flight per cluster: three hide the exchange best in the forward kernel (6.6 -> 6.4 ms per 592 blocks),
// the backward kernel has no registers for a third (9.55 -> 10.1 ms)
#ifndef VEC4_FWD_NBLK
#define VEC4_FWD_NBLK 3
#endif
#ifndef VEC2_FWD_NBLK
#define VEC2_FWD_NBLK 4
#endif
#ifndef VEC4_BWD_NBLK
#define VEC4_BWD_NBLK 2
#endif
bcjr_status launch_fwd_vec4(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    using C = Vec4Cfg<VEC4_FWD_NBLK>;
    if (p.n > C::MAX_N || ((uintptr_t)p.cb & 15u)) return BCJR_EUNSUPPORTED;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    auto kern = fwd_vec4_kernel<VEC4_FWD_NBLK>;
    bcjr_status rc = plan_cluster(ctx, kern, C::CL, C::THREADS, C::SMEM_BYTES, (p.B + C::NBLK - 1) / C::NBLK, &cfg, attr, st);
    if (rc) return rc;
    const int ncl = cfg.gridDim.x / C::CL, nt = p.n / C::V;
    if ((rc = ensure(ctx, ctx->hist, (size_t)ncl * C::NBLK * nt * C::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->cb_beta, (size_t)C::S * C::V * 4))) return rc;
    regroup_table_kernel<<<(C::S * C::V + 255) / 256, 256, 0, st>>>(p.cb, (float *)ctx->cb_beta.ptr, C::S, C::KB, C::V);
    p.hist = (float *)ctx->hist.ptr;
    p.cb_beta = (const float *)ctx->cb_beta.ptr;
    CU(cudaLaunchKernelEx(&cfg, kern, p));
    ctx->launches += 2;
    return BCJR_OK;
}

// Forward call of the same trellis on clusters of two CTAs (the table alone fits two tensor memories): the default.
bcjr_status launch_fwd_vec2(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    using C = Vec2Cfg<VEC2_FWD_NBLK>;
    if (p.n > C::MAX_N || ((uintptr_t)p.cb & 15u)) return BCJR_EUNSUPPORTED;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    auto kern = fwd_vec2_kernel<VEC2_FWD_NBLK>;
    bcjr_status rc = plan_cluster(ctx, kern, C::CL, C::THREADS, C::SMEM_BYTES, (p.B + C::NBLK - 1) / C::NBLK, &cfg, attr, st);
    if (rc) return rc;
    const int ncl = cfg.gridDim.x / C::CL, nt = p.n / C::V;
    if ((rc = ensure(ctx, ctx->hist, (size_t)ncl * C::NBLK * nt * C::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->cb_beta, (size_t)C::S * C::V * 4))) return rc;
    regroup_table_kernel<<<(C::S * C::V + 255) / 256, 256, 0, st>>>(p.cb, (float *)ctx->cb_beta.ptr, C::S, C::KB, C::V);
    p.hist = (float *)ctx->hist.ptr;
    p.cb_beta = (const float *)ctx->cb_beta.ptr;
    CU(cudaLaunchKernelEx(&cfg, kern, p));
    ctx->launches += 2;
    return BCJR_OK;
}

bcjr_status launch_bwd_vec4(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st)
{
    using C = Vec4BwdCfg<VEC4_BWD_NBLK>;
    constexpr int S = C::F::S, V = 2, KB = 4;
    if (p.n > C::MAX_N || ((uintptr_t)p.cb & 15u)) return BCJR_EUNSUPPORTED;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    auto kern = bwd_vec4_kernel<VEC4_BWD_NBLK>;
    bcjr_status rc = plan_cluster(ctx, kern, C::CL, C::THREADS, C::SMEM_BYTES, (p.B + C::NBLK - 1) / C::NBLK, &cfg, attr, st);
    if (rc) return rc;
    const int ncl = cfg.gridDim.x / C::CL, nt = p.n / V;
    if ((rc = ensure(ctx, ctx->hist, (size_t)ncl * C::NBLK * 2 * nt * C::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->gc_part, (size_t)ncl * S * V * 4))) return rc;
    if ((rc = ensure(ctx, ctx->cb_beta, (size_t)S * V * 4))) return rc;
    regroup_table_kernel<<<(S * V + 255) / 256, 256, 0, st>>>(p.cb, (float *)ctx->cb_beta.ptr, S, KB, V);
    p.hist = (float *)ctx->hist.ptr;
    p.gc_part = (float *)ctx->gc_part.ptr;
    p.cb_beta = (const float *)ctx->cb_beta.ptr;
    CU(cudaLaunchKernelEx(&cfg, kern, p));
    ctx->launches += 2;
    if (grad_codebook) {
        reduce_gc_vec_kernel<<<(S * V + 255) / 256, 256, 0, st>>>(p.gc_part, ncl, S, KB, V, grad_codebook);
        ctx->launches += 1;
        CU(cudaGetLastError());
    }
    return BCJR_OK;
}

template <int LB, int KB, int CL, int THREADS>
bcjr_status launch_fwd_cluster_t(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    using C = ClusterCfg<LB, KB, CL, THREADS>;
    if (p.n > C::MAX_N) return BCJR_EUNSUPPORTED;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    auto kern = fwd_cluster_kernel<LB, KB, CL, THREADS>;
    bcjr_status rc = plan_cluster(ctx, kern, CL, THREADS, C::SMEM_BYTES, p.B, &cfg, attr, st);
    if (rc) return rc;
    const int ncl = cfg.gridDim.x / CL;
    if ((rc = ensure(ctx, ctx->hist, (size_t)ncl * p.n * C::Q * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    CU(cudaLaunchKernelEx(&cfg, kern, p));
    ctx->launches += 1;
    return BCJR_OK;
}

template <int LB, int KB, int CL, int THREADS>
bcjr_status launch_bwd_cluster_t(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st)
{
    using C = ClusterCfg<LB, KB, CL, THREADS>;
    using BC = BwdClusterCfg<LB, KB, CL, THREADS>;
    if (p.n > BC::MAX_N) return BCJR_EUNSUPPORTED;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    auto kern = bwd_cluster_kernel<LB, KB, CL, THREADS>;
    bcjr_status rc = plan_cluster(ctx, kern, CL, THREADS, BC::SMEM_BYTES, p.B, &cfg, attr, st);
    if (rc) return rc;
    const int ncl = cfg.gridDim.x / CL;
    if ((rc = ensure(ctx, ctx->hist, (size_t)ncl * p.n * 2 * C::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->gc_part, (size_t)ncl * C::S * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.gc_part = (float *)ctx->gc_part.ptr;
    CU(cudaLaunchKernelEx(&cfg, kern, p));
    ctx->launches += 1;
    if (grad_codebook) {
        reduce_gc_kernel<<<(C::S + 255) / 256, 256, 0, st>>>(p.gc_part, ncl, C::S, grad_codebook);
        ctx->launches += 1;
        CU(cudaGetLastError());
    }
    return BCJR_OK;
}

// Backward call, clusters of two with codebook and accumulators in tensor memory (Lb = 16; k = 2, 3).
template <int KB>
bcjr_status launch_bwd_duo(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st)
{
    using C = DuoCfg<KB>;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    bcjr_status rc = plan_cluster(ctx, bwd_duo_kernel<KB>, C::CL, C::THREADS, C::SMEM_BYTES, p.B, &cfg, attr, st);
    if (rc) return rc;
    const int ncl = cfg.gridDim.x / C::CL;
    if ((rc = ensure(ctx, ctx->hist, (size_t)ncl * p.n * 2 * C::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->gc_part, (size_t)ncl * C::S * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.gc_part = (float *)ctx->gc_part.ptr;
    if (ctx->cb_computed) p.cb = nullptr;                    // entries are evaluated while staging
    CU(cudaLaunchKernelEx(&cfg, bwd_duo_kernel<KB>, p));
    ctx->launches += 1;
    if (grad_codebook) {
        reduce_gc_kernel<<<(C::S + 255) / 256, 256, 0, st>>>(p.gc_part, ncl, C::S, grad_codebook);
        ctx->launches += 1;
        CU(cudaGetLastError());
    }
    return BCJR_OK;
}

// Backward call for k = 2: the two-CTA tensor-memory kernel with the skewed slot order; without grad_codebook the
// accumulator half of the kernel is compiled out.
template <bool ACC>
bcjr_status launch_bwd_skew(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st)
{
    using C = SkewCfg;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    bcjr_status rc = plan_cluster(ctx, bwd_skew_kernel<ACC, false>, C::CL, C::THREADS, C::SMEM_BYTES, p.B, &cfg, attr, st);
    if (rc) return rc;
    const int ncl = cfg.gridDim.x / C::CL;
    if ((rc = ensure(ctx, ctx->hist, (size_t)ncl * p.n * 2 * C::Q * 4))) return rc;
    if (ACC && (rc = ensure(ctx, ctx->gc_part, (size_t)ncl * C::S * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.gc_part = ACC ? (float *)ctx->gc_part.ptr : nullptr;
    if (ctx->cb_computed) p.cb = nullptr;                    // entries are evaluated while staging
    CU(cudaLaunchKernelEx(&cfg, bwd_skew_kernel<ACC, false>, p));
    ctx->launches += 1;
    if (ACC) {
        reduce_gc_kernel<<<(C::S + 255) / 256, 256, 0, st>>>(p.gc_part, ncl, C::S, grad_codebook);
        ctx->launches += 1;
        CU(cudaGetLastError());
    }
    return BCJR_OK;
}

// Backward call in two kernels per chunk of blocks: the alpha sweeps on one CTA per block (bwd_alpha_kernel), then the
// beta sweeps of the same blocks on two-CTA clusters (k = 2: bwd_skew_kernel<ACC, true>; k = 3: bwd_duo_kernel<3, true>).
// A chunk is as many blocks as the GPU has SMs; the history of a chunk (32 MB per block at n = 256) is the hand-over.
template <int KB, bool ACC, typename BetaKernel>
bcjr_status launch_bwd_split(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st, BetaKernel beta, size_t beta_smem)
{
    using A = AlphaCfg<KB>;
    constexpr int CL = 2, THREADS = 512;
    cudaLaunchConfig_t cfg{};
    cudaLaunchAttribute attr[1];
    bcjr_status rc = plan_cluster(ctx, beta, CL, THREADS, beta_smem, p.B, &cfg, attr, st);
    if (rc) return rc;
    CU(cudaFuncSetAttribute(bwd_alpha_kernel<KB>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    const int ncl = cfg.gridDim.x / CL;
    int64_t chunk = ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && chunk > ctx->opt_max_ctas) chunk = ctx->opt_max_ctas;
    if (chunk > p.B) chunk = p.B;
    if ((rc = ensure(ctx, ctx->hist, (size_t)chunk * p.n * 2 * A::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->stepO, (size_t)chunk * A::AUX_INTS * 4))) return rc;
    if (ACC) {
        if ((rc = ensure(ctx, ctx->gc_part, (size_t)ncl * A::S * 4))) return rc;
        CU(cudaMemsetAsync(ctx->gc_part.ptr, 0, (size_t)ncl * A::S * 4, st));     // the beta launches add into it
    }
    p.hist = (float *)ctx->hist.ptr;
    p.stepO = (int *)ctx->stepO.ptr;
    p.gc_part = ACC ? (float *)ctx->gc_part.ptr : nullptr;
    if (ctx->cb_computed) p.cb = nullptr;                    // entries are evaluated while staging
    const int64_t B = p.B;
    const float *W = p.W, *g = p.g, *soft = p.soft;
    float *gW = p.gW;
    for (int64_t b0 = 0; b0 < B; b0 += chunk) {
        const int64_t nb = B - b0 < chunk ? B - b0 : chunk;
        p.B = nb;
        p.W = W + b0 * p.n; p.g = g + b0 * p.n; p.soft = soft + b0 * p.n; p.gW = gW + b0 * p.n;
        bwd_alpha_kernel<KB><<<(int)nb, A::THREADS, A::SMEM_BYTES, st>>>(p);
        CU(cudaGetLastError());
        cfg.gridDim = dim3((unsigned)(CL * (nb < ncl ? nb : ncl)), 1, 1);
        CU(cudaLaunchKernelEx(&cfg, beta, p));
        ctx->launches += 2;
    }
    if (ACC && grad_codebook) {
        reduce_gc_kernel<<<(A::S + 255) / 256, 256, 0, st>>>(p.gc_part, ncl, A::S, grad_codebook);
        ctx->launches += 1;
        CU(cudaGetLastError());
    }
    return BCJR_OK;
}

// Backward call without grad_codebook (Lb = 16, k = 2): both sweeps on one CTA per block.
bcjr_status launch_bwd_solo(bcjr_ctx *ctx, BwdParams p, cudaStream_t st)
{
    using C = BSoloCfg;
    CU(cudaFuncSetAttribute(bwd_solo_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    int64_t grid = ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && grid > ctx->opt_max_ctas) grid = ctx->opt_max_ctas;
    if (grid > p.B) grid = p.B;
    bcjr_status rc = ensure(ctx, ctx->hist, (size_t)grid * p.n * 2 * C::Q * 4);
    if (rc) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.gc_part = nullptr;
    if (ctx->cb_computed) p.cb = nullptr;                    // entries are evaluated while staging
    bwd_solo_kernel<<<(int)grid, C::THREADS, C::SMEM_BYTES, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

bcjr_status launch_bwd_cluster(bcjr_ctx *ctx, BwdParams p, int k, float *grad_codebook, cudaStream_t st)
{
    if (p.Lb != 16) return BCJR_EUNSUPPORTED;
    if (k == 2 && ctx->opt_bwd_variant == 0 && !grad_codebook && p.n <= BSoloCfg::MAX_N) return launch_bwd_solo(ctx, p, st);
    if (k == 2 && (ctx->opt_bwd_variant == 0 || ctx->opt_bwd_variant == 4) && p.n <= SkewCfg::MAX_N)
        return grad_codebook ? launch_bwd_split<2, true>(ctx, p, grad_codebook, st, bwd_skew_kernel<true, true>, SkewCfg::SMEM_BYTES)
                             : launch_bwd_split<2, false>(ctx, p, nullptr, st, bwd_skew_kernel<false, true>, SkewCfg::SMEM_BYTES);
    if (k == 3 && (ctx->opt_bwd_variant == 0 || ctx->opt_bwd_variant == 4) && p.n <= DuoCfg<3>::MAX_N)   // without grad_codebook the partial sums are formed and dropped
        return launch_bwd_split<3, true>(ctx, p, grad_codebook, st, bwd_duo_kernel<3, true>, DuoCfg<3>::SMEM_BYTES);
    if (k == 2 && ctx->opt_bwd_variant == 3 && p.n <= SkewCfg::MAX_N)
        return grad_codebook ? launch_bwd_skew<true>(ctx, p, grad_codebook, st) : launch_bwd_skew<false>(ctx, p, nullptr, st);
    if (k == 2 && ctx->opt_bwd_variant != 1 && p.n <= DuoCfg<2>::MAX_N) return launch_bwd_duo<2>(ctx, p, grad_codebook, st);
    if (k == 3 && ctx->opt_bwd_variant != 1 && p.n <= DuoCfg<3>::MAX_N) return launch_bwd_duo<3>(ctx, p, grad_codebook, st);   // variants 2, 3; no grad_codebook
    if (k == 2) return launch_bwd_cluster_t<16, 2, 4, 512>(ctx, p, grad_codebook, st);
    if (k == 3) return launch_bwd_cluster_t<16, 3, 4, 256>(ctx, p, grad_codebook, st);
    return BCJR_EUNSUPPORTED;
}

// Viterbi, one CTA per block with the codebook in tensor memory (Lb = 16; k = 2, 3).
template <int KB>
bcjr_status launch_vit_solo(bcjr_ctx *ctx, VitParams p, cudaStream_t st)
{
    using C = VitSoloCfg<KB>;
    if (p.n > C::MAX_N) return BCJR_EUNSUPPORTED;
    CU(cudaFuncSetAttribute(viterbi_solo_kernel<KB>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    int64_t grid = ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && grid > ctx->opt_max_ctas) grid = ctx->opt_max_ctas;
    if (grid > p.B) grid = p.B;
    bcjr_status rc = ensure(ctx, ctx->bp, (size_t)grid * 2 * p.n * C::ROW_BYTES);
    if (rc) return rc;
    p.bp = (uint8_t *)ctx->bp.ptr;
    p.diag = ctx->diag;
    if (ctx->cb_computed) p.cb = nullptr;                    // entries are evaluated while staging
    viterbi_solo_kernel<KB><<<(int)grid, C::THREADS, C::SMEM_BYTES, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

// Forward call, one CTA per block with the codebook in tensor memory (Lb = 16; k = 2, 3).
template <int KB>
bcjr_status launch_fwd_solo(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    using C = SoloCfg<KB>;
    if (p.n > C::MAX_N) return BCJR_EUNSUPPORTED;
    CU(cudaFuncSetAttribute(fwd_solo_kernel<KB>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    int64_t grid = ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && grid > ctx->opt_max_ctas) grid = ctx->opt_max_ctas;
    if (grid > p.B) grid = p.B;
    bcjr_status rc = ensure(ctx, ctx->hist, (size_t)grid * p.n * C::Q * 4);
    if (rc) return rc;
    p.hist = (float *)ctx->hist.ptr;
    if (ctx->cb_computed) p.cb = nullptr;                    // entries are evaluated while staging
    fwd_solo_kernel<KB><<<(int)grid, C::THREADS, C::SMEM_BYTES, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

// Forward call with checkpointed history (option history_every_m > 1; Lb = 16, k = 2, n <= 512).
template <int KB>
bcjr_status launch_fwd_ckpt(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    using C = CkptCfg<KB>;
    CU(cudaFuncSetAttribute(fwd_ckpt_kernel<KB>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    int64_t grid = ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && grid > ctx->opt_max_ctas) grid = ctx->opt_max_ctas;
    if (grid > p.B) grid = p.B;
    p.hist_every = ctx->opt_hist_every;
    bcjr_status rc = ensure(ctx, ctx->hist, (size_t)grid * C::rows(p.n, p.hist_every) * C::Q * 4);
    if (rc) return rc;
    p.hist = (float *)ctx->hist.ptr;
    if (ctx->cb_computed) p.cb = nullptr;                    // entries are evaluated while staging
    fwd_ckpt_kernel<KB><<<(int)grid, C::THREADS, C::SMEM_BYTES, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

// Mid-size trellises (Lb = 11 .. 13, k = 2): one warp per block, table (and accumulators) in tensor memory.
inline bool warp_supported(int Lb, int k) { return k == 2 && Lb >= 11 && Lb <= 13; }

template <int LB>
bcjr_status launch_fwd_warp(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    using C = WarpCfg<LB, false>;
    CU(cudaFuncSetAttribute(fwd_warp_kernel<LB>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    int64_t grid = ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && grid > ctx->opt_max_ctas) grid = ctx->opt_max_ctas;
    const int64_t need = (p.B + C::NWARP - 1) / C::NWARP;
    if (grid > need) grid = need;
    const size_t warps = (size_t)grid * C::NWARP;
    bcjr_status rc;
    if ((rc = ensure(ctx, ctx->hist, warps * p.n * C::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->stepO, warps * ((size_t)p.n + 2) * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.stepO = (int *)ctx->stepO.ptr;
    if (ctx->cb_computed) p.cb = nullptr;                    // entries are evaluated while staging
    fwd_warp_kernel<LB><<<(int)grid, C::THREADS, C::SMEM_BYTES, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

template <int LB, bool ACC>
bcjr_status launch_bwd_warp(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st)
{
    using C = WarpCfg<LB, true>;
    CU(cudaFuncSetAttribute(bwd_warp_kernel<LB, ACC>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    int64_t grid = ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && grid > ctx->opt_max_ctas) grid = ctx->opt_max_ctas;
    const int64_t need = (p.B + C::NWARP - 1) / C::NWARP;
    if (grid > need) grid = need;
    const size_t warps = (size_t)grid * C::NWARP;
    bcjr_status rc;
    if ((rc = ensure(ctx, ctx->hist, warps * p.n * 2 * C::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->stepO, warps * ((size_t)p.n + 2) * 4))) return rc;
    if (ACC && (rc = ensure(ctx, ctx->gc_part, warps * C::S * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.stepO = (int *)ctx->stepO.ptr;
    p.gc_part = ACC ? (float *)ctx->gc_part.ptr : nullptr;
    if (ctx->cb_computed) p.cb = nullptr;
    bwd_warp_kernel<LB, ACC><<<(int)grid, C::THREADS, C::SMEM_BYTES, st>>>(p);
    ctx->launches += 1;
    CU(cudaGetLastError());
    if (ACC) {
        reduce_gc_kernel<<<(C::S + 255) / 256, 256, 0, st>>>(p.gc_part, (int)warps, C::S, grad_codebook);
        ctx->launches += 1;
        CU(cudaGetLastError());
    }
    return BCJR_OK;
}

// Backward call with grad_codebook at Lb = 12, 13: two warps per block (twice the warps per SM for the same tensor memory).
template <int LB>
bcjr_status launch_bwd_warp2(bcjr_ctx *ctx, BwdParams p, float *grad_codebook, cudaStream_t st)
{
    using C = Warp2Cfg<LB>;
    CU(cudaFuncSetAttribute(bwd_warp2_kernel<LB>, cudaFuncAttributeMaxDynamicSharedMemorySize, ctx->max_smem_optin));
    int64_t grid = ctx->num_sms;
    if (ctx->opt_max_ctas > 0 && grid > ctx->opt_max_ctas) grid = ctx->opt_max_ctas;
    const int64_t need = (p.B + C::NPAIR - 1) / C::NPAIR;
    if (grid > need) grid = need;
    const size_t pairs = (size_t)grid * C::NPAIR;
    bcjr_status rc;
    if ((rc = ensure(ctx, ctx->hist, pairs * p.n * 2 * C::Q * 4))) return rc;
    if ((rc = ensure(ctx, ctx->stepO, pairs * ((size_t)p.n + 2) * 4))) return rc;
    if ((rc = ensure(ctx, ctx->gc_part, pairs * C::S * 4))) return rc;
    p.hist = (float *)ctx->hist.ptr;
    p.stepO = (int *)ctx->stepO.ptr;
    p.gc_part = (float *)ctx->gc_part.ptr;
    if (ctx->cb_computed) p.cb = nullptr;
    bwd_warp2_kernel<LB><<<(int)grid, C::THREADS, C::SMEM_BYTES, st>>>(p);
    CU(cudaGetLastError());
    reduce_gc_kernel<<<(C::S + 255) / 256, 256, 0, st>>>(p.gc_part, (int)pairs, C::S, grad_codebook);
    ctx->launches += 2;
    CU(cudaGetLastError());
    return BCJR_OK;
}

bcjr_status launch_fwd_warp_any(bcjr_ctx *ctx, FwdParams p, cudaStream_t st)
{
    switch (p.Lb) {
        case 11: return launch_fwd_warp<11>(ctx, p, st);
        case 12: return launch_fwd_warp<12>(ctx, p, st);
        default: return launch_fwd_warp<13>(ctx, p, st);
    }
}

bcjr_status launch_bwd_warp_any(bcjr_ctx *ctx, BwdParams p, float *gc, cudaStream_t st)
{
    switch (p.Lb) {
        case 11: return gc ? launch_bwd_warp<11, true>(ctx, p, gc, st) : launch_bwd_warp<11, false>(ctx, p, gc, st);
        case 12:
            if (gc && ctx->opt_bwd_variant != 1) return launch_bwd_warp2<12>(ctx, p, gc, st);
            return gc ? launch_bwd_warp<12, true>(ctx, p, gc, st) : launch_bwd_warp<12, false>(ctx, p, gc, st);
        default:
            if (gc && ctx->opt_bwd_variant != 1) return launch_bwd_warp2<13>(ctx, p, gc, st);
            return gc ? launch_bwd_warp<13, true>(ctx, p, gc, st) : launch_bwd_warp<13, false>(ctx, p, gc, st);
    }
}

bcjr_status launch_fwd_cluster(bcjr_ctx *ctx, FwdParams p, int k, cudaStream_t st)
{
    if (p.Lb != 16) return BCJR_EUNSUPPORTED;
    if (ctx->opt_hist_every > 1 && ctx->opt_fwd_variant != 1 && k == 2 && p.n <= CkptCfg<2>::MAX_N) return launch_fwd_ckpt<2>(ctx, p, st);
    if (k == 2 && ctx->opt_fwd_variant != 1) return launch_fwd_solo<2>(ctx, p, st);
    if (k == 3 && ctx->opt_fwd_variant != 1) return launch_fwd_solo<3>(ctx, p, st);
    if (k == 2) return launch_fwd_cluster_t<16, 2, FWD_CL_K2, FWD_THREADS_K2>(ctx, p, st);
    if (k == 3) return launch_fwd_cluster_t<16, 3, 2, 512>(ctx, p, st);
    return BCJR_EUNSUPPORTED;
}
#endif

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev)
    {
        if (cudaGetDevice(&prev) == cudaSuccess && (prev == dev || cudaSetDevice(dev) == cudaSuccess)) ok = true;
    }
    ~DeviceGuard() { if (ok && prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

namespace {
int log2_exact(int64_t v)
{
    if (v < 1 || (v & (v - 1))) return -1;
    int l = 0;
    while ((((int64_t)1) << l) < v) ++l;
    return l;
}
template <int LOGN>
void launch_fwht_rows(const float *in, float *out, const float *s, int m, float scale, int pre, int sms, cudaStream_t st)
{
    constexpr int N = 1 << LOGN, T = N / 8;
    int grid = sms * (T >= 1024 ? 1 : 1024 / T);
    if (grid > m) grid = m;
    fwht_rows_kernel<LOGN><<<grid, T, (size_t)(N + N / 8) * 4, st>>>(in, out, s, m, scale, pre);
}
}  // namespace

extern "C" {

bcjr_status bcjr_create(bcjr_ctx **out, int device_ordinal)
{
    if (!out) return BCJR_EINVAL;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device_ordinal < 0 || device_ordinal >= count) {
        cudaGetLastError();
        return BCJR_ECUDA;
    }
    bcjr_ctx *ctx = new (std::nothrow) bcjr_ctx();
    if (!ctx) return BCJR_ENOMEM;
    ctx->device = device_ordinal;
    DeviceGuard guard(device_ordinal);
    cudaDeviceProp prop;
    if (!guard.ok || cudaGetDeviceProperties(&prop, device_ordinal) != cudaSuccess ||
        cudaMalloc((void **)&ctx->diag, sizeof(DeviceDiag)) != cudaSuccess ||
        cudaMemset(ctx->diag, 0, sizeof(DeviceDiag)) != cudaSuccess ||
        cudaMemcpy(&ctx->diag->wait_limit_ns, &kDefaultWaitLimitNs, sizeof(kDefaultWaitLimitNs), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError();
        delete ctx;
        return BCJR_ECUDA;
    }
    ctx->num_sms = prop.multiProcessorCount;
    ctx->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    *out = ctx;
    return BCJR_OK;
}

bcjr_status bcjr_destroy(bcjr_ctx *ctx)
{
    if (!ctx) return BCJR_EINVAL;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    Buffer *all[] = {&ctx->hist, &ctx->stepO, &ctx->msg, &ctx->gc_part, &ctx->soft_copy, &ctx->bp, &ctx->path_ws,
                     &ctx->cb_beta, &ctx->grad_w, &ctx->grad_c, &ctx->blk_defect, &ctx->gauss_cb, &ctx->staging[0], &ctx->staging[1], &ctx->staging[2], &ctx->staging[3], &ctx->staging[4],
                     &ctx->staging[5]};
    for (Buffer *b : all)
        if (b->ptr) cudaFree(b->ptr);
    if (ctx->diag) cudaFree(ctx->diag);
    cudaGetLastError();
    delete ctx;
    return BCJR_OK;
}

bcjr_status bcjr_set_option(bcjr_ctx *ctx, const char *name, int64_t value)
{
    if (!ctx || !name) return BCJR_EINVAL;
    if (!strcmp(name, "path")) {
        if (value < 0 || value > 2) return BCJR_EINVAL;
        ctx->opt_path = (int)value;
        return BCJR_OK;
    }
    if (!strcmp(name, "bwd_variant")) {
        if (value < 0 || value > 4) return BCJR_EINVAL;
        ctx->opt_bwd_variant = (int)value;
        return BCJR_OK;
    }
    if (!strcmp(name, "fwd_variant")) {
        if (value < 0 || value > 1) return BCJR_EINVAL;
        ctx->opt_fwd_variant = (int)value;
        return BCJR_OK;
    }
    if (!strcmp(name, "wait_limit_ms") || !strcmp(name, "debug_drop_history_load")) {
        // device-side configuration: written behind everything already queued on the device
        DeviceGuard guard(ctx->device);
        if (!guard.ok || value < 0 || value > 600000) return BCJR_EINVAL;
        CU(cudaDeviceSynchronize());
        if (name[0] == 'w') {
            const unsigned long long ns = (unsigned long long)(value > 0 ? value : 1) * 1000000ull;
            CU(cudaMemcpy(&ctx->diag->wait_limit_ns, &ns, sizeof(ns), cudaMemcpyHostToDevice));
        } else {
            const int flag = value != 0;
            CU(cudaMemcpy(&ctx->diag->drop_history_load, &flag, sizeof(flag), cudaMemcpyHostToDevice));
        }
        return BCJR_OK;
    }
    if (!strcmp(name, "history_every_m")) {
        if (value < 1 || value > 16) return BCJR_EINVAL;
        ctx->opt_hist_every = (int)value;
        return BCJR_OK;
    }
    if (!strcmp(name, "record_block_defect")) {
        if (value < 0 || value > 1) return BCJR_EINVAL;
        ctx->opt_record_defect = (int)value;
        return BCJR_OK;
    }
    if (!strcmp(name, "max_ctas")) {
        if (value < 0 || value > (1 << 20)) return BCJR_EINVAL;
        ctx->opt_max_ctas = (int)value;
        return BCJR_OK;
    }
    return BCJR_EINVAL;
}

bcjr_status bcjr_soft_quantize(bcjr_ctx *ctx, const float *W, const float *codebook, int Lb, int k, int n,
                               int64_t num_blocks, float T, float *soft, float *logZ, void *cuda_stream)
{
    if (!ctx) return BCJR_EINVAL;
    if (!(T > 0.f) || !std::isfinite(T)) return BCJR_EINVAL;
    bcjr_status rc = check_dims(Lb, k, n, num_blocks);
    if (rc) return rc;
    if (num_blocks > 0 && (!W || !soft)) return BCJR_EINVAL;   // empty input: pointers unused; codebook NULL = computed emission
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    ctx->have_fwd = false;
    ctx->cb_computed = codebook == nullptr;
    if (num_blocks == 0) {
        ctx->W = W; ctx->cb = codebook; ctx->Lb = Lb; ctx->k = k; ctx->n = n; ctx->B = 0; ctx->T = T;
        ctx->V = 1;
        ctx->have_fwd = true;
        return BCJR_OK;
    }
    if (ctx->cb_computed && (rc = computed_table(ctx, Lb, st, &codebook))) return rc;
    if ((rc = ensure(ctx, ctx->soft_copy, (size_t)num_blocks * n * 4))) return rc;
    FwdParams p{};
    p.W = W; p.cb = codebook; p.soft = soft; p.soft_copy = (float *)ctx->soft_copy.ptr; p.logZ = logZ;
    p.diag = ctx->diag; p.B = num_blocks; p.Lb = Lb; p.n = n;
    p.lam2 = (float)(1.4426950408889634 / (2.0 * (double)T));
    table_range_kernel<<<1, 1024, 0, st>>>(codebook, 1 << Lb, ctx->diag);     // c_lo, c_hi for step_energy
    ctx->launches += 1;
    ctx->defect_blocks = 0;
    if (ctx->opt_record_defect) {
        if ((rc = ensure(ctx, ctx->blk_defect, (size_t)num_blocks * 4))) return rc;
        CU(cudaMemsetAsync(ctx->blk_defect.ptr, 0xff, (size_t)num_blocks * 4, st));   // NaN = not recorded by this kernel
        p.blk_defect = (float *)ctx->blk_defect.ptr;
        ctx->defect_blocks = num_blocks;
    }
    bool use_cluster = false;
#ifndef BCJR_NO_CLUSTER
    use_cluster = ctx->opt_path != 1 && cluster_supported(Lb, k);
    if (ctx->opt_path == 2 && !use_cluster) return BCJR_EUNSUPPORTED;
    if (use_cluster) {
        rc = launch_fwd_cluster(ctx, p, k, st);
        if (rc == BCJR_EUNSUPPORTED && ctx->opt_path != 2) { use_cluster = false; rc = BCJR_OK; }   // e.g. n too long
    }
    bool use_warp = !use_cluster && ctx->opt_path == 0 && warp_supported(Lb, k);
    if (use_warp) rc = launch_fwd_warp_any(ctx, p, st);
#else
    if (ctx->opt_path == 2) return BCJR_EUNSUPPORTED;
    const bool use_warp = false;
#endif
    if (!use_cluster && !use_warp) {
        switch (k) {
            case 1: rc = launch_fwd_generic<1>(ctx, p, st); break;
            case 2: rc = launch_fwd_generic<2>(ctx, p, st); break;
            case 3: rc = launch_fwd_generic<3>(ctx, p, st); break;
            default: rc = launch_fwd_generic<4>(ctx, p, st); break;
        }
    }
    if (rc) return rc;
    ctx->last_path = use_cluster ? 1 : use_warp ? 2 : 0;
    ctx->W = W; ctx->cb = codebook; ctx->Lb = Lb; ctx->k = k; ctx->n = n; ctx->B = num_blocks; ctx->T = T;
    ctx->V = 1;
    ctx->have_fwd = true;
    return BCJR_OK;
}

bcjr_status bcjr_backward(bcjr_ctx *ctx, const float *grad_soft, float *grad_W, float *grad_codebook,
                          void *cuda_stream)
{
    if (!ctx) return BCJR_EINVAL;
    if (!ctx->have_fwd) return BCJR_ESTATE;
    if (ctx->B > 0 && (!grad_soft || !grad_W)) return BCJR_EINVAL;
    if (ctx->cb_computed && ctx->V == 1 && grad_codebook) return BCJR_EINVAL;   // a computed emission has no table to differentiate
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int S = 1 << ctx->Lb;
    if (ctx->B == 0) {
        if (grad_codebook) CU(cudaMemsetAsync(grad_codebook, 0, (size_t)S * ctx->V * 4, st));
        return BCJR_OK;
    }
    BwdParams p{};
    p.W = ctx->W; p.cb = ctx->cb; p.g = grad_soft; p.soft = (const float *)ctx->soft_copy.ptr; p.gW = grad_W;
    p.diag = ctx->diag; p.B = ctx->B; p.Lb = ctx->Lb; p.n = ctx->n;
    p.lam2 = (float)(1.4426950408889634 / (2.0 * (double)ctx->T));
    p.invT = (float)(1.0 / (double)ctx->T);
    bcjr_status rc = BCJR_OK;
    if (ctx->V == 1) {
        table_range_kernel<<<1, 1024, 0, st>>>(ctx->cb, S, ctx->diag);          // c_lo, c_hi for step_energy
        ctx->launches += 1;
    }
    if (ctx->V == 2) {                                   // saved by bcjr_soft_quantize_vec: k bits per weight
        if (!aligned8(grad_soft) || !aligned8(grad_W)) return BCJR_EINVAL;
        bool large = false;
#ifndef BCJR_NO_CLUSTER
        large = ctx->opt_path != 1 && ctx->Lb == 16 && ctx->k == 2;
        if (ctx->opt_path == 2 && !large) return BCJR_EUNSUPPORTED;
        if (large) {
            rc = launch_bwd_vec4(ctx, p, grad_codebook, st);
            if (rc == BCJR_EUNSUPPORTED && ctx->opt_path != 2) { large = false; rc = BCJR_OK; }
        }
#else
        if (ctx->opt_path == 2) return BCJR_EUNSUPPORTED;
#endif
        if (!large)
            rc = ctx->k == 1 ? launch_bwd_vec<2, 2>(ctx, p, grad_codebook, st) : launch_bwd_vec<4, 2>(ctx, p, grad_codebook, st);
        if (rc) return rc;
        ctx->last_path = large ? 1 : 0;
        return BCJR_OK;
    }
    bool use_cluster = false;
#ifndef BCJR_NO_CLUSTER
    use_cluster = ctx->opt_path != 1 && cluster_supported(ctx->Lb, ctx->k);
    if (ctx->opt_path == 2 && !use_cluster) return BCJR_EUNSUPPORTED;
    if (use_cluster) {
        rc = launch_bwd_cluster(ctx, p, ctx->k, grad_codebook, st);
        if (rc == BCJR_EUNSUPPORTED && ctx->opt_path != 2) { use_cluster = false; rc = BCJR_OK; }
    }
    const bool use_warp = !use_cluster && ctx->opt_path == 0 && warp_supported(ctx->Lb, ctx->k);
    if (use_warp) rc = launch_bwd_warp_any(ctx, p, grad_codebook, st);
#else
    if (ctx->opt_path == 2) return BCJR_EUNSUPPORTED;
    const bool use_warp = false;
#endif
    if (!use_cluster && !use_warp) {
        switch (ctx->k) {
            case 1: rc = launch_bwd_generic<1>(ctx, p, grad_codebook, st); break;
            case 2: rc = launch_bwd_generic<2>(ctx, p, grad_codebook, st); break;
            case 3: rc = launch_bwd_generic<3>(ctx, p, grad_codebook, st); break;
            default: rc = launch_bwd_generic<4>(ctx, p, grad_codebook, st); break;
        }
    }
    if (rc) return rc;
    ctx->last_path = use_cluster ? 1 : use_warp ? 2 : 0;
    return BCJR_OK;
}

bcjr_status viterbi_hard(bcjr_ctx *ctx, const float *W, const float *codebook, int Lb, int k, int n,
                         int64_t num_blocks, uint8_t *path_bits, int64_t path_stride_bytes, uint16_t *states,
                         float *hard, void *cuda_stream)
{
    if (!ctx) return BCJR_EINVAL;
    bcjr_status rc = check_dims(Lb, k, n, num_blocks);
    if (rc) return rc;
    if (num_blocks > 0 && !W) return BCJR_EINVAL;                // codebook NULL = computed emission
    const int64_t nbits = Lb + (int64_t)k * (n - 1);
    if (path_bits && path_stride_bytes < (nbits + 7) / 8) return BCJR_EINVAL;
    if (num_blocks == 0) return BCJR_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const bool saved_computed = ctx->cb_computed;                // belongs to the saved forward state: restored below
    struct Restore { bcjr_ctx *c; bool v; ~Restore() { c->cb_computed = v; } } restore{ctx, saved_computed};
    ctx->cb_computed = codebook == nullptr;
    if (ctx->cb_computed) {
        // the context has one computed table: a saved forward state that relies on another size of it ends here
        if (ctx->have_fwd && saved_computed && ctx->Lb != Lb) ctx->have_fwd = false;
        if ((rc = computed_table(ctx, Lb, st, &codebook))) return rc;
    }
    VitParams p{};
    p.W = W; p.cb = codebook; p.path_bits = path_bits; p.path_stride = path_stride_bytes;
    p.states = states; p.hard = hard; p.B = num_blocks; p.Lb = Lb; p.n = n;
    bool use_large = false;
#ifndef BCJR_NO_CLUSTER
    use_large = ctx->opt_path != 1 && Lb == 16 && (k == 2 || k == 3);
    if (ctx->opt_path == 2 && !use_large) return BCJR_EUNSUPPORTED;
    if (use_large) {
        rc = k == 2 ? launch_vit_solo<2>(ctx, p, st) : launch_vit_solo<3>(ctx, p, st);
        if (rc == BCJR_EUNSUPPORTED && ctx->opt_path != 2) { use_large = false; rc = BCJR_OK; }
    }
#else
    if (ctx->opt_path == 2) return BCJR_EUNSUPPORTED;
#endif
    if (!use_large) {
        switch (k) {
            case 1: rc = launch_vit_generic<1>(ctx, p, st); break;
            case 2: rc = launch_vit_generic<2>(ctx, p, st); break;
            case 3: rc = launch_vit_generic<3>(ctx, p, st); break;
            default: rc = launch_vit_generic<4>(ctx, p, st); break;
        }
    }
    if (rc) return rc;
    ctx->last_path = use_large ? 1 : 0;
    return BCJR_OK;
}

bcjr_status bcjr_soft_quantize_vec(bcjr_ctx *ctx, const float *W, const float *codebook, int Lb, int k, int V,
                                   int n, int64_t num_blocks, float T, float *soft, float *logZ, void *cuda_stream)
{
    if (!ctx) return BCJR_EINVAL;
    if (V == 1) return bcjr_soft_quantize(ctx, W, codebook, Lb, k, n, num_blocks, T, soft, logZ, cuda_stream);
    if (!(T > 0.f) || !std::isfinite(T)) return BCJR_EINVAL;
    bcjr_status rc = check_vec(Lb, k, V, n, num_blocks);
    if (rc) return rc;
    if (num_blocks > 0 && (!W || !codebook || !soft)) return BCJR_EINVAL;
    if (!aligned8(W) || !aligned8(codebook) || !aligned8(soft)) return BCJR_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    ctx->have_fwd = false;
    if (num_blocks > 0) {
        if ((rc = ensure(ctx, ctx->soft_copy, (size_t)num_blocks * n * 4))) return rc;
        FwdParams p{};
        p.W = W; p.cb = codebook; p.soft = soft; p.soft_copy = (float *)ctx->soft_copy.ptr; p.logZ = logZ;
        p.diag = ctx->diag; p.B = num_blocks; p.Lb = Lb; p.n = n;
        p.lam2 = (float)(1.4426950408889634 / (2.0 * (double)T));
        bool large = false;
#ifndef BCJR_NO_CLUSTER
        large = ctx->opt_path != 1 && Lb == 16 && k == 2;
        if (ctx->opt_path == 2 && !large) return BCJR_EUNSUPPORTED;
        if (large) {
            rc = ctx->opt_fwd_variant == 1 ? launch_fwd_vec4(ctx, p, st) : launch_fwd_vec2(ctx, p, st);
            if (rc == BCJR_EUNSUPPORTED && ctx->opt_path != 2) { large = false; rc = BCJR_OK; }   // e.g. n too long
        }
#else
        if (ctx->opt_path == 2) return BCJR_EUNSUPPORTED;
#endif
        if (!large) rc = k == 1 ? launch_fwd_vec<2, 2>(ctx, p, st) : launch_fwd_vec<4, 2>(ctx, p, st);
        if (rc) return rc;
        ctx->last_path = large ? 1 : 0;
    }
    ctx->W = W; ctx->cb = codebook; ctx->Lb = Lb; ctx->k = k; ctx->n = n; ctx->B = num_blocks; ctx->T = T;
    ctx->V = V;
    ctx->have_fwd = true;
    return BCJR_OK;
}

bcjr_status viterbi_hard_vec(bcjr_ctx *ctx, const float *W, const float *codebook, int Lb, int k, int V, int n,
                             int64_t num_blocks, uint8_t *path_bits, int64_t path_stride_bytes, uint16_t *states,
                             float *hard, void *cuda_stream)
{
    if (!ctx) return BCJR_EINVAL;
    if (V == 1)
        return viterbi_hard(ctx, W, codebook, Lb, k, n, num_blocks, path_bits, path_stride_bytes, states, hard, cuda_stream);
    bcjr_status rc = check_vec(Lb, k, V, n, num_blocks);
    if (rc) return rc;
    if (num_blocks > 0 && (!W || !codebook)) return BCJR_EINVAL;
    if (!aligned8(W) || !aligned8(codebook)) return BCJR_EINVAL;
    const int64_t nbits = Lb + (int64_t)k * V * (n / V - 1);
    if (path_bits && path_stride_bytes < (nbits + 7) / 8) return BCJR_EINVAL;
    if (num_blocks == 0) return BCJR_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    VitParams p{};
    p.W = W; p.cb = codebook; p.path_bits = path_bits; p.path_stride = path_stride_bytes;
    p.states = states; p.hard = hard; p.B = num_blocks; p.Lb = Lb; p.n = n;
    rc = k == 1 ? launch_vit_vec<2, 2>(ctx, p, st) : launch_vit_vec<4, 2>(ctx, p, st);
    if (rc) return rc;
    ctx->last_path = 0;
    return BCJR_OK;
}

bcjr_status bcjr_ste_forward(bcjr_ctx *ctx, const float *W, const float *codebook, int Lb, int k, int n,
                             int64_t num_blocks, float T, float *hard, uint16_t *states, float *soft,
                             void *cuda_stream)
{
    if (!ctx) return BCJR_EINVAL;
    if (!(T > 0.f) || !std::isfinite(T)) return BCJR_EINVAL;
    bcjr_status rc = check_dims(Lb, k, n, num_blocks);
    if (rc) return rc;
    if (num_blocks > 0 && (!W || !hard)) return BCJR_EINVAL;
    float *soft_out = soft;
    if (!soft_out && num_blocks > 0) {
        // the relaxation's output is only needed as saved state: let it land in the context's own copy
        DeviceGuard guard(ctx->device);
        if (!guard.ok) return BCJR_ECUDA;
        if ((rc = ensure(ctx, ctx->soft_copy, (size_t)num_blocks * n * 4))) return rc;
        soft_out = (float *)ctx->soft_copy.ptr;
    }
    if ((rc = bcjr_soft_quantize(ctx, W, codebook, Lb, k, n, num_blocks, T, soft_out, nullptr, cuda_stream))) return rc;
    rc = viterbi_hard(ctx, W, codebook, Lb, k, n, num_blocks, nullptr, 0, states, hard, cuda_stream);
    if (rc) ctx->have_fwd = false;
    return rc;
}

double bcjr_temperature(double T0, double T_end, int t, int n_steps)
{
    if (!(T0 > 0.0) || !(T_end > 0.0) || n_steps < 1) return 0.0;
    return T0 * std::pow(T_end / T0, (double)t / (double)n_steps);
}

bcjr_status bcjr_gaussian_codebook(bcjr_ctx *ctx, int Lb, float *codebook, void *cuda_stream)
{
    if (!ctx || !codebook || Lb < 1 || Lb > 16) return BCJR_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    const int S = 1 << Lb;
    gaussian_table_kernel<<<(S + 255) / 256, 256, 0, (cudaStream_t)cuda_stream>>>(codebook, S);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

bcjr_status bcjr_adam_update(bcjr_ctx *ctx, float *param, const float *grad, float *m, float *v, int64_t numel,
                             int t, float lr, float beta1, float beta2, float eps, void *cuda_stream)
{
    if (!ctx || numel < 0 || t < 1) return BCJR_EINVAL;
    if (!(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) || !(eps > 0.f) || !std::isfinite(lr)) return BCJR_EINVAL;
    if (numel == 0) return BCJR_OK;
    if (!param || !grad || !m || !v) return BCJR_EINVAL;
    if (((uintptr_t)param | (uintptr_t)grad | (uintptr_t)m | (uintptr_t)v) & 15u) return BCJR_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    AdamParams a{};
    a.p = param; a.g = grad; a.m = m; a.v = v; a.numel = numel;
    a.lr_c1 = (float)((double)lr / (1.0 - std::pow((double)beta1, (double)t)));
    a.inv_c2 = (float)(1.0 / (1.0 - std::pow((double)beta2, (double)t)));
    a.beta1 = beta1; a.beta2 = beta2; a.eps = eps;
    int64_t blocks = (numel / 4 + 255) / 256;
    const int64_t cap = (int64_t)ctx->num_sms * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    adam_kernel<<<(int)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(a);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

bcjr_status bcjr_backward_adam(bcjr_ctx *ctx, const float *grad_soft, float *W_latent, float *m_W, float *v_W,
                               float *codebook, float *m_c, float *v_c, int t, float lr_W, float lr_c,
                               float beta1, float beta2, float eps, void *cuda_stream)
{
    if (!ctx) return BCJR_EINVAL;
    if (!ctx->have_fwd) return BCJR_ESTATE;
    if (W_latent != ctx->W || (codebook && codebook != ctx->cb)) return BCJR_EINVAL;   // must be the saved tensors
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    const int64_t numel = ctx->B * ctx->n, csize = ((int64_t)1 << ctx->Lb) * ctx->V;
    bcjr_status rc;
    if ((rc = ensure(ctx, ctx->grad_w, (size_t)(numel > 0 ? numel : 1) * 4))) return rc;
    if ((rc = ensure(ctx, ctx->grad_c, (size_t)csize * 4))) return rc;
    float *gW = (float *)ctx->grad_w.ptr, *gc = (float *)ctx->grad_c.ptr;
    if ((rc = bcjr_backward(ctx, grad_soft, gW, codebook ? gc : nullptr, cuda_stream))) return rc;
    if ((rc = bcjr_adam_update(ctx, W_latent, gW, m_W, v_W, numel, t, lr_W, beta1, beta2, eps, cuda_stream))) return rc;
    if (codebook && (rc = bcjr_adam_update(ctx, codebook, gc, m_c, v_c, csize, t, lr_c, beta1, beta2, eps, cuda_stream))) return rc;
    ctx->have_fwd = false;      // the saved inputs have changed: a new forward call is needed
    return BCJR_OK;
}

bcjr_status bcjr_rht(bcjr_ctx *ctx, const float *W, float *out, int m, int n, const float *sign_rows,
                     const float *sign_cols, int inverse, void *cuda_stream)
{
    if (!ctx || !W || !out || !sign_rows || !sign_cols) return BCJR_EINVAL;
    const int lm = log2_exact(m), ln = log2_exact(n);
    if (lm < 3 || ln < 3) return BCJR_EINVAL;                     // powers of two, at least 8
    if (ln > 13 || lm > 24) return BCJR_EUNSUPPORTED;            // a row must fit shared memory
    if (((uintptr_t)W | (uintptr_t)out | (uintptr_t)sign_cols) & 15u) return BCJR_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int pre = inverse ? 0 : 1;
    const float srow = (float)(1.0 / std::sqrt((double)n)), scol = (float)(1.0 / std::sqrt((double)m));
    switch (ln) {
        case 3: launch_fwht_rows<3>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 4: launch_fwht_rows<4>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 5: launch_fwht_rows<5>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 6: launch_fwht_rows<6>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 7: launch_fwht_rows<7>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 8: launch_fwht_rows<8>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 9: launch_fwht_rows<9>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 10: launch_fwht_rows<10>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 11: launch_fwht_rows<11>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        case 12: launch_fwht_rows<12>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
        default: launch_fwht_rows<13>(W, out, sign_cols, m, srow, pre, ctx->num_sms, st); break;
    }
    ctx->launches += 1;
    CU(cudaGetLastError());
    // columns: radix-8 passes over the row-index bits, in place on `out`
    const int n4 = n / 4;
    const int64_t total = (int64_t)(m / 8) * n4;
    int blocks = (int)((total + 255) / 256 < (int64_t)ctx->num_sms * 8 ? (total + 255) / 256 : (int64_t)ctx->num_sms * 8);
    if (blocks < 1) blocks = 1;
    for (int o = 0;; o += 3) {
        const bool last = o + 3 >= lm;
        const int oo = last ? lm - 3 : o, first = o - oo;
        const int mode = (!inverse && o == 0) ? 1 : (inverse && last) ? 2 : 0;
        fwht_cols_pass_kernel<<<blocks, 256, 0, st>>>(out, sign_rows, m, n4, oo, first, last ? scol : 1.f, mode);
        ctx->launches += 1;
        CU(cudaGetLastError());
        if (last) break;
    }
    return BCJR_OK;
}

bcjr_status bcjr_group_scale(bcjr_ctx *ctx, const float *W, float *scales, float *W_scaled, int64_t numel, void *cuda_stream)
{
    if (!ctx || numel < 0 || numel % 16) return BCJR_EINVAL;
    if (numel == 0) return BCJR_OK;
    if (!W || !scales || !W_scaled || (((uintptr_t)W | (uintptr_t)W_scaled) & 15u)) return BCJR_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    const int64_t groups = numel / 16;
    int64_t blocks = (groups + 255) / 256;
    if (blocks > (int64_t)ctx->num_sms * 16) blocks = (int64_t)ctx->num_sms * 16;
    group_scale_kernel<<<(int)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(W, scales, W_scaled, groups);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

bcjr_status bcjr_group_unscale(bcjr_ctx *ctx, const float *W_scaled, const float *scales, float *W, int64_t numel, void *cuda_stream)
{
    if (!ctx || numel < 0 || numel % 16) return BCJR_EINVAL;
    if (numel == 0) return BCJR_OK;
    if (!W || !scales || !W_scaled || (((uintptr_t)W | (uintptr_t)W_scaled) & 15u)) return BCJR_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    const int64_t groups = numel / 16;
    int64_t blocks = (groups + 255) / 256;
    if (blocks > (int64_t)ctx->num_sms * 16) blocks = (int64_t)ctx->num_sms * 16;
    group_unscale_kernel<<<(int)blocks, 256, 0, (cudaStream_t)cuda_stream>>>(W_scaled, scales, W, groups);
    ctx->launches += 1;
    CU(cudaGetLastError());
    return BCJR_OK;
}

bcjr_status bcjr_step_host(bcjr_ctx *ctx, const float *W_host, const float *codebook_host,
                           const float *grad_soft_host, int Lb, int k, int n, int64_t num_blocks, float T,
                           float *soft_host, float *grad_W_host, float *grad_codebook_host, void *cuda_stream)
{
    if (!ctx || !W_host || !codebook_host || !grad_soft_host) return BCJR_EINVAL;
    bcjr_status rc = check_dims(Lb, k, n, num_blocks);
    if (rc) return rc;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const size_t wbytes = (size_t)num_blocks * n * 4, cbytes = ((size_t)1 << Lb) * 4;
    const size_t sizes[6] = {wbytes, cbytes, wbytes, wbytes, wbytes, cbytes};
    for (int i = 0; i < 6; ++i)
        if ((rc = ensure(ctx, ctx->staging[i], sizes[i] ? sizes[i] : 4))) return rc;
    float *dW = (float *)ctx->staging[0].ptr, *dcb = (float *)ctx->staging[1].ptr;
    float *dg = (float *)ctx->staging[2].ptr, *dsoft = (float *)ctx->staging[3].ptr;
    float *dgW = (float *)ctx->staging[4].ptr, *dgc = (float *)ctx->staging[5].ptr;
    if (wbytes) CU(cudaMemcpyAsync(dW, W_host, wbytes, cudaMemcpyHostToDevice, st));
    CU(cudaMemcpyAsync(dcb, codebook_host, cbytes, cudaMemcpyHostToDevice, st));
    if (wbytes) CU(cudaMemcpyAsync(dg, grad_soft_host, wbytes, cudaMemcpyHostToDevice, st));
    if ((rc = bcjr_soft_quantize(ctx, dW, dcb, Lb, k, n, num_blocks, T, dsoft, nullptr, cuda_stream))) return rc;
    if ((rc = bcjr_backward(ctx, dg, dgW, dgc, cuda_stream))) return rc;
    if (soft_host && wbytes) CU(cudaMemcpyAsync(soft_host, dsoft, wbytes, cudaMemcpyDeviceToHost, st));
    if (grad_W_host && wbytes) CU(cudaMemcpyAsync(grad_W_host, dgW, wbytes, cudaMemcpyDeviceToHost, st));
    if (grad_codebook_host) CU(cudaMemcpyAsync(grad_codebook_host, dgc, cbytes, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamSynchronize(st));
    return BCJR_OK;
}

bcjr_status bcjr_sync_status(bcjr_ctx *ctx, void *cuda_stream, bcjr_diag *out)
{
    if (!ctx) return BCJR_EINVAL;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    CU(cudaStreamSynchronize(st));
    DeviceDiag h;
    CU(cudaMemcpy(&h, ctx->diag, DIAG_STATUS_BYTES, cudaMemcpyDeviceToHost));
    CU(cudaMemset(ctx->diag, 0, DIAG_STATUS_BYTES));
    if (out) {
        out->device_status = h.status;
        float f;
        memcpy(&f, &h.max_defect, 4);
        out->max_posterior_defect = f;
        memcpy(&f, &h.max_logz_gap, 4);
        out->max_logz_mismatch = f * 0.6931472f;
        out->kernel_launches = ctx->launches;
        out->last_path = ctx->last_path;
    }
    return (bcjr_status)h.status;
}

bcjr_status bcjr_block_defects(bcjr_ctx *ctx, float *host_out, int64_t count, void *cuda_stream)
{
    if (!ctx || count < 0 || (count > 0 && !host_out)) return BCJR_EINVAL;
    if (count > ctx->defect_blocks) return BCJR_ESTATE;
    if (count == 0) return BCJR_OK;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return BCJR_ECUDA;
    CU(cudaStreamSynchronize((cudaStream_t)cuda_stream));
    CU(cudaMemcpy(host_out, ctx->blk_defect.ptr, (size_t)count * 4, cudaMemcpyDeviceToHost));
    return BCJR_OK;
}

int64_t bcjr_workspace_bytes(const bcjr_ctx *ctx)
{
    if (!ctx) return 0;
    const Buffer *all[] = {&ctx->hist, &ctx->stepO, &ctx->msg, &ctx->gc_part, &ctx->soft_copy, &ctx->bp,
                           &ctx->path_ws, &ctx->cb_beta, &ctx->grad_w, &ctx->grad_c, &ctx->blk_defect, &ctx->gauss_cb, &ctx->staging[0], &ctx->staging[1], &ctx->staging[2], &ctx->staging[3],
                           &ctx->staging[4], &ctx->staging[5]};
    int64_t tot = 0;
    for (const Buffer *b : all) tot += (int64_t)b->bytes;
    return tot;
}

const char *bcjr_last_cuda_error(const bcjr_ctx *ctx) { return ctx ? ctx->cuda_error.c_str() : ""; }

const char *bcjr_status_string(bcjr_status s)
{
    switch (s) {
        case BCJR_OK: return "ok";
        case BCJR_EINVAL: return "invalid argument";
        case BCJR_ENOMEM: return "out of device memory";
        case BCJR_ECUDA: return "CUDA runtime error";
        case BCJR_ESTATE: return "bcjr_backward called without a saved forward pass";
        case BCJR_EUNSUPPORTED: return "unsupported (Lb, k, n) combination";
        case BCJR_ETIMEOUT: return "device-side wait timed out";
        case BCJR_ENUMERIC: return "non-finite values on the device";
        case BCJR_ETOOLARGE: return "problem exceeds the fixed scratch of bcjr_soft_quantize_static";
    }
    return "unknown status";
}

}  // extern "C"
