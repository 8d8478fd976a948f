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
