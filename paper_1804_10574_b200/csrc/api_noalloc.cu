// Batch-norm forward for callers that must not allocate.
//
// Some callers of this library run where device allocation is off limits: inside a memory pool they do not own,
// in a real-time loop where cudaMalloc's implicit synchronisation is unacceptable, or in a process whose device
// memory is fully budgeted up front.  ddg_bn_fwd needs a scratch buffer (per-CTA partial sums and a ticket
// counter) that such a caller cannot provide without allocating.  This entry point carries that scratch inside
// the library image instead: a file-scope device array of a fixed, modest size, so the call allocates nothing.
#include <mutex>

#include "../../include/ddg.h"
#include "common.cuh"
#include "kernels.h"

using namespace ddg;

namespace ddg { void set_global_error(const char *msg); }

namespace {

constexpr int kNoAllocMaxC = 64;
// bn_scratch_elems(64) floats: 32 for the ticket counter + 592 CTAs x 2 sums x 64 channels x 2 (fp64 partials of the
// fp32 mode).  About 592 KiB; every GPU that loads the library holds it until the process exits.
constexpr size_t kNoAllocScratchElems = 32 + (size_t)592 * 2 * kNoAllocMaxC * 2;

static __device__ __align__(256) float g_bn_noalloc_scratch[kNoAllocScratchElems];

constexpr int kMaxDevices = 64;
float *g_scratch_addr[kMaxDevices] = {};  // device address of the array, per device, resolved on first use
std::mutex g_scratch_mu;

// In host code the array's name is only a handle: the device address has to be asked for, per device, with that
// device current.
ddg_status scratch_for_current_device(float **out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_global_error("ddg_bn_fwd_noalloc: no current CUDA device");
        return DDG_ERR_CUDA;
    }
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    if (!g_scratch_addr[dev]) {
        void *p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_bn_noalloc_scratch);
        if (e != cudaSuccess || !p) {
            set_global_error("ddg_bn_fwd_noalloc: cudaGetSymbolAddress failed for the built-in scratch array");
            return DDG_ERR_CUDA;
        }
        g_scratch_addr[dev] = static_cast<float *>(p);
    }
    *out = g_scratch_addr[dev];
    return DDG_OK;
}

}  // namespace

extern "C" ddg_status ddg_bn_fwd_noalloc(int precision, const void *x, const void *gamma, const void *beta,
                                         const void *res, void *y, float *mean, float *invstd, int B, int HW, int C,
                                         int relu, void *stream) {
    if ((precision != DDG_FP32 && precision != DDG_BF16) || !x || !gamma || !beta || !y || !mean || !invstd)
        return DDG_ERR_INVALID_ARG;
    if (B < 1 || HW < 1 || C < 1) return DDG_ERR_INVALID_ARG;
    if (C > kNoAllocMaxC || bn_scratch_elems(C) > kNoAllocScratchElems) {
        set_global_error("ddg_bn_fwd_noalloc: C exceeds the built-in scratch (at most 64 channels); use ddg_bn_fwd "
                         "with caller-provided scratch");
        return DDG_ERR_UNSUPPORTED;
    }
    {   // an error left pending by an earlier call must not be blamed on (or cleared by) this one
        const cudaError_t before = cudaPeekAtLastError();
        if (before != cudaSuccess) {
            set_global_error("ddg_bn_fwd_noalloc: an earlier CUDA error is still pending");
            return DDG_ERR_CUDA;
        }
    }
    float *scratch = nullptr;
    ddg_status st = scratch_for_current_device(&scratch);
    if (st != DDG_OK) return st;
    cudaStream_t s = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the CTA ticket counter must start at zero
    if (cudaMemsetAsync(scratch, 0, 128, s) != cudaSuccess) return DDG_ERR_CUDA;
    launch_bn_stats(precision, x, mean, invstd, scratch, (long)B * HW, C, s);
    Shortcut sc{};
    if (res) { sc.mode = 1; sc.a = res; }
    launch_bn_apply(precision, x, gamma, beta, mean, invstd, sc, y, B, HW, 1, C, relu, s);
    return cudaGetLastError() == cudaSuccess ? DDG_OK : DDG_ERR_CUDA;
}
