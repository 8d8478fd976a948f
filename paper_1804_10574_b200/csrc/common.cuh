// Shared device/host helpers of the DDG CUDA library (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

#include "kernels.h"

namespace ddg {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f<bf16>(float v) { return __float2bfloat16_rn(v); }

// Arithmetic type between storage points: bf16 tensors are computed in fp32; fp32 tensors (the parity mode) in
// fp64, so that the fp32 mode differs from an fp64 evaluation only by the fp32 rounding of what is stored.
template <typename T> struct AccOf { typedef float type; };
template <> struct AccOf<float> { typedef double type; };
template <typename T> __device__ __forceinline__ T from_a(float v) { return from_f<T>(v); }
template <typename T> __device__ __forceinline__ T from_a(double v);
template <> __device__ __forceinline__ float from_a<float>(double v) { return (float)v; }
template <> __device__ __forceinline__ bf16 from_a<bf16>(double v) { return __float2bfloat16_rn((float)v); }

// A 16-byte vector of elements of T: 4 floats or 8 bf16.
template <typename T> struct Vec16 { static constexpr int N = 16 / sizeof(T); };

template <typename T, int N> struct alignas(sizeof(T) * N) Pack { T v[N]; };

template <typename T, int N> __device__ __forceinline__ void load_f(const T *p, float (&out)[N]) {
    Pack<T, N> q = *reinterpret_cast<const Pack<T, N> *>(p);
#pragma unroll
    for (int i = 0; i < N; ++i) out[i] = to_f(q.v[i]);
}
template <typename T, int N> __device__ __forceinline__ void store_f(T *p, const float (&in)[N]) {
    Pack<T, N> q;
#pragma unroll
    for (int i = 0; i < N; ++i) q.v[i] = from_f<T>(in[i]);
    *reinterpret_cast<Pack<T, N> *>(p) = q;
}
template <typename T, typename A, int N> __device__ __forceinline__ void load_a(const T *p, A (&out)[N]) {
    Pack<T, N> q = *reinterpret_cast<const Pack<T, N> *>(p);
#pragma unroll
    for (int i = 0; i < N; ++i) out[i] = (A)to_f(q.v[i]);
}
template <typename T, typename A, int N> __device__ __forceinline__ void store_a(T *p, const A (&in)[N]) {
    Pack<T, N> q;
#pragma unroll
    for (int i = 0; i < N; ++i) q.v[i] = from_a<T>(in[i]);
    *reinterpret_cast<Pack<T, N> *>(p) = q;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Totals of n_part rows of nval = 2C per-CTA partial sums, by the first THREADS threads of a CTA (all threads of the CTA must call), in a fixed order: the
// rows are read as one flat array of 16-byte vectors (THREADS * 4 values per pass is a multiple of nval, so a thread
// always meets the same four columns), up to eight independent loads in flight per thread, accumulated in double in
// pass order; the threads that share a column are then added in index order.  Result: tot[0..nval) in shared memory.
// fold: THREADS * 4 doubles of shared memory.  The convolution's last CTA and the element-wise passes use the same routine
// with the same THREADS, so both ways of folding give the same bits.
template <int THREADS>
__device__ __forceinline__ void fold_partials(const float *__restrict__ part, int n_part, int nval, double *fold, double *tot) {
    const int t = threadIdx.x;
    const int total4 = n_part * nval / 4;
    if (t < THREADS) {
        double a[4] = {0.0, 0.0, 0.0, 0.0};
        const float4 *p4 = reinterpret_cast<const float4 *>(part);
        for (int i0 = t; i0 < total4; i0 += 8 * THREADS) {
            float4 q[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int i = i0 + u * THREADS;
                q[u] = i < total4 ? __ldcg(p4 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) { a[0] += (double)q[u].x; a[1] += (double)q[u].y; a[2] += (double)q[u].z; a[3] += (double)q[u].w; }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) fold[t * 4 + j] = a[j];
    }
    __syncthreads();
    if (t < nval) {
        // column t lives in the threads whose first vector covers it: thread (t / 4) + k * (nval / 4), element t % 4
        double sum = 0.0;
        for (int k = t / 4; k < THREADS; k += nval / 4) sum += fold[k * 4 + (t & 3)];
        tot[t] = sum;
    }
    __syncthreads();
}


static inline int ceil_div(long a, long b) { return (int)((a + b - 1) / b); }

// Programmatic dependent launch.  A kernel launched with programmatic stream serialisation may be scheduled while the
// previous kernel of its stream is still running, so that its launch latency and its prologue overlap that kernel's
// tail.  The contract that keeps this correct: every kernel executes pdl_wait() before its first access to global
// memory that an earlier kernel may write or still read; the wait returns when all preceding kernels of the stream have
// completed and their writes are visible.  pdl_launch() tells the scheduler that the next kernel may start being placed.
// Which launches carry the attribute is the caller's policy (Launch::pdl in kernels.h).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// asks_pdl: the kernel is one of those that keep the attribute under Launch::pdl == 2
template <typename... KArgs, typename... Args>
inline void launch_kp(bool asks_pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, const Launch &L,
                      Args &&...args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = L.s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (L.pdl == 1 || (L.pdl == 2 && asks_pdl)) ? 1 : 0;
    cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
template <typename... KArgs, typename... Args>
inline void launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, const Launch &L, Args &&...args) {
    launch_kp(false, kernel, grid, block, smem, L, std::forward<Args>(args)...);
}

}  // namespace ddg
