// bcjr_soft_quantize_static: the forward call for callers that may not allocate device memory.
//
// Who this is for: code that runs where cudaMalloc / cudaFree are off limits -- a host loop that
// must never take the device-wide synchronisation an allocation or a free implies, a process
// whose device memory has all been handed to another allocator up front, a plug-in that is only
// allowed to launch work on buffers it was given.  The regular entry points grow a per-context
// scratch area with cudaMalloc on demand; this one owns a fixed scratch array that is part of
// the library image instead, so nothing is allocated or freed, ever, on any path through it.
//
// The price is a size limit (see BCJR_STATIC_SCRATCH_BYTES) and a single shared scratch area:
// every call on a device uses the same array, so two calls whose kernels overlap on the GPU
// (different streams, different host threads) would overwrite each other's history.  Issue
// them on one stream, or otherwise make sure one has finished before the next starts.
#include "../../include/bcjr_b200.h"

#include <cmath>
#include <mutex>

#include "bcjr_common.cuh"
#include "bcjr_generic.cuh"

using namespace bcjr;

namespace {

// Scratch of the static entry point: a small header (device diagnostics) followed by the
// per-CTA step offsets and the per-CTA message history of the generic forward kernel.
// Every GPU that loads the library holds this array until the process exits.
constexpr size_t kStaticScratchBytes = BCJR_STATIC_SCRATCH_BYTES;
constexpr size_t kHeaderBytes = 256;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char *g_scratch_ptr[kMaxDevices] = {};   // device address of g_static_scratch, per device
int g_num_sms[kMaxDevices] = {};
int g_smem_optin[kMaxDevices] = {};

// In host code `g_static_scratch` is only a handle for the symbol, not a device address: the
// address the kernel needs comes from cudaGetSymbolAddress, asked once per device while that
// device is current.
bcjr_status resolve_scratch(int dev, unsigned char **out)
{
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_ptr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return BCJR_ECUDA;
        }
        int sms = 0, smem = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) {
            cudaGetLastError();
            return BCJR_ECUDA;
        }
        g_num_sms[dev] = sms;
        g_smem_optin[dev] = smem;
        g_scratch_ptr[dev] = static_cast<unsigned char *>(ptr);
    }
    *out = g_scratch_ptr[dev];
    return BCJR_OK;
}

template <int KB>
bcjr_status launch_static(int dev, unsigned char *scratch, FwdParams p, cudaStream_t st)
{
    const int Q = 1 << (p.Lb - KB);
    int threads = (Q + 31) / 32 * 32;
    if (threads > GEN_MAX_THREADS) threads = GEN_MAX_THREADS;
    const size_t smem = (size_t)(GEN_SMEM_HEADER + 2 * Q) * sizeof(float);
    if (smem + 1024 > (size_t)g_smem_optin[dev]) return BCJR_EUNSUPPORTED;   // messages must fit shared memory
    // per CTA: n*Q floats of history, n+2 ints of step offsets (rounded up to 256 bytes)
    const size_t hist_bytes = (size_t)p.n * Q * 4;
    const size_t step_bytes = (((size_t)p.n + 2) * 4 + 255) / 256 * 256;
    const size_t per_cta = hist_bytes + step_bytes;
    const size_t room = kStaticScratchBytes - kHeaderBytes;
    if (per_cta > room) return BCJR_ETOOLARGE;                               // one block alone does not fit
    // always the device's opt-in maximum, never this call's own size: the attribute belongs to the kernel, not to a
    // call, and a smaller value set here could undercut a launch another host thread is about to make
    if (cudaFuncSetAttribute(fwd_generic_kernel<KB>, cudaFuncAttributeMaxDynamicSharedMemorySize, g_smem_optin[dev]) != cudaSuccess) {
        cudaGetLastError();
        return BCJR_ECUDA;
    }
    int occ = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, fwd_generic_kernel<KB>, threads, smem) != cudaSuccess) {
        cudaGetLastError();
        return BCJR_ECUDA;
    }
    // as many CTAs as the GPU can hold, as the work needs, and as the scratch has room for
    int64_t grid = (int64_t)(occ < 1 ? 1 : occ) * g_num_sms[dev];
    if (grid > p.B) grid = p.B;
    if ((size_t)grid > room / per_cta) grid = (int64_t)(room / per_cta);
    if (grid < 1) return BCJR_ETOOLARGE;
    // layout: [header][grid x (n+2) ints, padded to 256 bytes][grid x n*Q floats]
    const size_t step_total = ((size_t)grid * ((size_t)p.n + 2) * 4 + 255) / 256 * 256;
    p.diag = reinterpret_cast<DeviceDiag *>(scratch);
    p.stepO = reinterpret_cast<int *>(scratch + kHeaderBytes);
    p.hist = reinterpret_cast<float *>(scratch + kHeaderBytes + step_total);
    p.msg = nullptr;
    p.soft_copy = nullptr;
    // The array keeps whatever the previous call left.  History and step offsets are always
    // written before they are read; only the diagnostics header accumulates, so clear it.
    if (cudaMemsetAsync(scratch, 0, kHeaderBytes, st) != cudaSuccess) {
        cudaGetLastError();
        return BCJR_ECUDA;
    }
    table_range_kernel<<<1, 1024, 0, st>>>(p.cb, 1 << p.Lb, p.diag);          // c_lo, c_hi for step_energy
    fwd_generic_kernel<KB><<<(int)grid, threads, smem, st>>>(p);
    if (cudaGetLastError() != cudaSuccess) return BCJR_ECUDA;
    return BCJR_OK;
}

}  // namespace

extern "C" bcjr_status bcjr_soft_quantize_static(const float *W, const float *codebook, int Lb, int k, int n,
                                                 int64_t num_blocks, float T, float *soft, float *logZ,
                                                 void *cuda_stream)
{
    if (k < 1 || k > 4 || Lb < k || Lb > 16 || n < 1 || num_blocks < 0) return BCJR_EINVAL;
    if (!(T > 0.f) || !std::isfinite(T)) return BCJR_EINVAL;
    if (num_blocks == 0) return BCJR_OK;
    if (!W || !codebook || !soft) return BCJR_EINVAL;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return BCJR_ECUDA;
    }
    unsigned char *scratch = nullptr;
    bcjr_status rc = resolve_scratch(dev, &scratch);
    if (rc) return rc;
    FwdParams p{};
    p.W = W; p.cb = codebook; p.soft = soft; p.logZ = logZ;
    p.B = num_blocks; p.Lb = Lb; p.n = n;
    p.lam2 = (float)(1.4426950408889634 / (2.0 * (double)T));
    cudaStream_t st = (cudaStream_t)cuda_stream;
    switch (k) {
        case 1: return launch_static<1>(dev, scratch, p, st);
        case 2: return launch_static<2>(dev, scratch, p, st);
        case 3: return launch_static<3>(dev, scratch, p, st);
        default: return launch_static<4>(dev, scratch, p, st);
    }
}

extern "C" int64_t bcjr_static_scratch_bytes(void) { return (int64_t)kStaticScratchBytes; }
