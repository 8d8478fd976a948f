// Memory-bound kernels of the DDG step: layout shim, batch-norm statistics / apply / backward, ReLU, global
// mean pool, small FC layers, softmax cross-entropy, and the fused delayed-gradient optimiser update.
// All are coalesced 16-byte-vector kernels with fp32 arithmetic; reductions are two-stage with a fixed
// summation order (per-CTA partials, last CTA folds them), so results are reproducible run to run.
#include "common.cuh"
#include "kernels.h"

namespace ddg {

static constexpr int kThreads = 256;
static constexpr int kMaxPartials = 592;  // 4 CTAs per SM on 148 SMs
static constexpr float kBnEps = 1e-5f;

#define DISPATCH_PREC(prec, ...)                       \
    do {                                               \
        if ((prec) == P_BF16) { typedef bf16 T; __VA_ARGS__; } \
        else { typedef float T; __VA_ARGS__; }         \
    } while (0)

// ------------------------------------------------------------------------------------------------------
// input shim: NCHW fp32 -> NHWC T
// ------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void shim_kernel(const float *__restrict__ x, T *__restrict__ out, int B, int C, int HW, int Cpad) {
    pdl_launch();
    pdl_wait();
    long i = (long)blockIdx.x * blockDim.x + threadIdx.x;  // (n, p)
    if (i >= (long)B * HW) return;
    long n = i / HW, p = i % HW;
    for (int c = 0; c < C; ++c) out[i * Cpad + c] = from_f<T>(x[(n * C + c) * HW + p]);
    for (int c = C; c < Cpad; ++c) out[i * Cpad + c] = from_f<T>(0.f);  // zero channels up to the padded width
}

int launch_shim(int prec, const float *x, void *out, int B, int C, int H, int W, int Cpad, Launch s) {
    long n = (long)B * H * W;
    DISPATCH_PREC(prec, launch_k(shim_kernel<T>, ceil_div(n, kThreads), kThreads, 0, s, x, (T *)out, B, C, H * W, Cpad));
    return 1;
}

// ------------------------------------------------------------------------------------------------------
// ReLU
// ------------------------------------------------------------------------------------------------------
template <typename T> __global__ void relu_fwd_kernel(const T *x, T *y, size_t n) {
    pdl_launch();
    pdl_wait();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) { float v = to_f(x[i]); y[i] = from_f<T>(v > 0.f ? v : 0.f); }
}
template <typename T> __global__ void relu_bwd_kernel(const T *y, const T *dy, T *dx, size_t n) {
    pdl_launch();
    pdl_wait();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dx[i] = to_f(y[i]) > 0.f ? dy[i] : from_f<T>(0.f);
}
int launch_relu_fwd(int prec, const void *x, void *y, size_t n, Launch s) {
    DISPATCH_PREC(prec, launch_k(relu_fwd_kernel<T>, ceil_div(n, kThreads), kThreads, 0, s, (const T *)x, (T *)y, n));
    return 1;
}
int launch_relu_bwd(int prec, const void *y, const void *dy, void *dx, size_t n, Launch s) {
    DISPATCH_PREC(prec, launch_k(relu_bwd_kernel<T>, ceil_div(n, kThreads), kThreads, 0, s, (const T *)y, (const T *)dy,
                                                                                      (T *)dx, n));
    return 1;
}

// ------------------------------------------------------------------------------------------------------
// global mean pool: x [B][HW][C] -> y [B][C]
// ------------------------------------------------------------------------------------------------------
template <typename T> __global__ void avgpool_fwd_kernel(const T *x, T *y, int HW, int C) {
    pdl_launch();
    pdl_wait();
    typedef typename AccOf<T>::type A;
    __shared__ A sm[kThreads];
    const int n = blockIdx.x, lanes = blockDim.x / C;  // host guarantees C <= blockDim
    const int c = threadIdx.x % C, lane = threadIdx.x / C;
    A acc = 0;
    if (lane < lanes)
        for (int p = lane; p < HW; p += lanes) acc += (A)to_f(x[((size_t)n * HW + p) * C + c]);
    sm[threadIdx.x] = acc;
    __syncthreads();
    if (threadIdx.x < C) {
        A t = 0;
        for (int l = 0; l < lanes; ++l) t += sm[l * C + c];
        y[(size_t)n * C + c] = from_a<T>(t / (A)HW);
    }
}
template <typename T> __global__ void avgpool_bwd_kernel(const T *dy, T *dx, int HW, int C, size_t n) {
    pdl_launch();
    pdl_wait();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    size_t b = i / ((size_t)HW * C);
    int c = (int)(i % C);
    typedef typename AccOf<T>::type A;
    dx[i] = from_a<T>((A)to_f(dy[b * C + c]) / (A)HW);
}
int launch_avgpool_fwd(int prec, const void *x, void *y, int B, int HW, int C, Launch s) {
    DISPATCH_PREC(prec, launch_k(avgpool_fwd_kernel<T>, B, kThreads, 0, s, (const T *)x, (T *)y, HW, C));
    return 1;
}
int launch_avgpool_bwd(int prec, const void *dy, void *dx, int B, int HW, int C, Launch s) {
    size_t n = (size_t)B * HW * C;
    DISPATCH_PREC(prec, launch_k(avgpool_bwd_kernel<T>, ceil_div(n, kThreads), kThreads, 0, s, (const T *)dy, (T *)dx, HW,
                                                                                        C, n));
    return 1;
}

// ------------------------------------------------------------------------------------------------------
// small FC layers (CUDA cores; the FC layers of these networks are a few MFLOP)
// ------------------------------------------------------------------------------------------------------
// one warp per output element y[b][o]
template <typename T, typename TO>
__global__ void fc_fwd_kernel(const T *x, const T *W, const T *bias, TO *y, int B, int in, int out, int relu) {
    pdl_launch();
    pdl_wait();
    long warp = ((long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    if (warp >= (long)B * out) return;
    typedef typename AccOf<T>::type A;
    int b = (int)(warp / out), o = (int)(warp % out);
    A acc = 0;
    for (int i = lane; i < in; i += 32) acc += (A)to_f(x[(size_t)b * in + i]) * (A)to_f(W[(size_t)o * in + i]);
    acc = warp_sum(acc);
    if (lane == 0) {
        if (bias) acc += (A)to_f(bias[o]);
        if (relu && acc < 0) acc = 0;
        y[(size_t)b * out + o] = from_a<TO>(acc);
    }
}
template <typename TO> __device__ __forceinline__ float masked_dy(const TO *y, const TO *dy, size_t i, int relu) {
    float d = to_f(dy[i]);
    if (relu && !(to_f(y[i]) > 0.f)) d = 0.f;
    return d;
}
// dx[b][i] = sum_o dz[b][o] W[o][i]
template <typename T, typename TO>
__global__ void fc_dx_kernel(const T *W, const TO *y, const TO *dy, T *dx, int B, int in, int out, int relu) {
    pdl_launch();
    pdl_wait();
    long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= (long)B * in) return;
    typedef typename AccOf<T>::type A;
    int b = (int)(idx / in), i = (int)(idx % in);
    A acc = 0;
    for (int o = 0; o < out; ++o)
        acc += (A)masked_dy(y, dy, (size_t)b * out + o, relu) * (A)to_f(W[(size_t)o * in + i]);
    dx[idx] = from_a<T>(acc);
}
// dW[o][i] = sum_b dz[b][o] x[b][i]; db[o] = sum_b dz[b][o]   (thread per (o, i); i == in handles the bias)
template <typename T, typename TO>
__global__ void fc_dw_kernel(const T *x, const TO *y, const TO *dy, float *dW, float *db, int B, int in, int out,
                             int relu) {
    pdl_launch();
    pdl_wait();
    long idx = (long)blockIdx.x * blockDim.x + threadIdx.x;
    int cols = in + 1;
    if (idx >= (long)out * cols) return;
    typedef typename AccOf<T>::type A;
    int o = (int)(idx / cols), i = (int)(idx % cols);
    A acc = 0;
    if (i < in) {
        for (int b = 0; b < B; ++b)
            acc += (A)masked_dy(y, dy, (size_t)b * out + o, relu) * (A)to_f(x[(size_t)b * in + i]);
        dW[(size_t)o * in + i] = (float)acc;
    } else if (db) {
        for (int b = 0; b < B; ++b) acc += (A)masked_dy(y, dy, (size_t)b * out + o, relu);
        db[o] = (float)acc;
    }
}
int launch_fc_fwd(int prec, const void *x, const void *W, const void *bias, void *y, int B, int in, int out, int relu,
                  int out_f32, Launch s) {
    long threads = (long)B * out * 32;
    DISPATCH_PREC(prec, {
        if (out_f32)
            launch_k(fc_fwd_kernel<T, float>, ceil_div(threads, kThreads), kThreads, 0, s, (const T *)x, (const T *)W,
                                                                                    (const T *)bias, (float *)y, B, in,
                                                                                    out, relu);
        else
            launch_k(fc_fwd_kernel<T, T>, ceil_div(threads, kThreads), kThreads, 0, s, (const T *)x, (const T *)W,
                                                                                (const T *)bias, (T *)y, B, in, out,
                                                                                relu);
    });
    return 1;
}
int launch_fc_bwd(int prec, const void *x, const void *W, const void *y, const void *dy, void *dx, float *dW, float *db,
                  int B, int in, int out, int relu, int out_f32, Launch s) {
    int n = 0;
    DISPATCH_PREC(prec, {
        if (out_f32) {
            if (dx) { launch_k(fc_dx_kernel<T, float>, ceil_div((long)B * in, kThreads), kThreads, 0, s, (const T *)W, (const float *)y, (const float *)dy, (T *)dx, B, in, out, relu); ++n; }
            launch_k(fc_dw_kernel<T, float>, ceil_div((long)out * (in + 1), kThreads), kThreads, 0, s, (const T *)x, (const float *)y, (const float *)dy, dW, db, B, in, out, relu);
        } else {
            if (dx) { launch_k(fc_dx_kernel<T, T>, ceil_div((long)B * in, kThreads), kThreads, 0, s, (const T *)W, (const T *)y, (const T *)dy, (T *)dx, B, in, out, relu); ++n; }
            launch_k(fc_dw_kernel<T, T>, ceil_div((long)out * (in + 1), kThreads), kThreads, 0, s, (const T *)x, (const T *)y, (const T *)dy, dW, db, B, in, out, relu);
        }
    });
    return n + 1;
}

// ------------------------------------------------------------------------------------------------------
// softmax cross-entropy: one CTA, one warp per row, fixed-order final sum
// ------------------------------------------------------------------------------------------------------
__device__ __forceinline__ float exp_a(float v) { return expf(v); }
__device__ __forceinline__ double exp_a(double v) { return exp(v); }
__device__ __forceinline__ float log_a(float v) { return logf(v); }
__device__ __forceinline__ double log_a(double v) { return log(v); }

template <typename A>
__global__ void softmax_ce_kernel(const float *logits, const int *labels, float *loss, float *dlogits, int B, int C) {
    pdl_launch();
    pdl_wait();
    __shared__ A wsum[32];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    A acc = 0;
    for (int b = warp; b < B; b += nw) {
        const float *z = logits + (size_t)b * C;
        float mx = -INFINITY;
        for (int c = lane; c < C; c += 32) mx = fmaxf(mx, z[c]);
        mx = warp_max(mx);
        A se = 0;
        for (int c = lane; c < C; c += 32) se += exp_a((A)z[c] - (A)mx);
        se = warp_sum(se);
        const int y = labels[b];
        for (int c = lane; c < C; c += 32)
            dlogits[(size_t)b * C + c] = (float)((exp_a((A)z[c] - (A)mx) / se - (c == y ? (A)1 : (A)0)) / (A)B);
        acc += log_a(se) + (A)mx - (A)z[y];
    }
    if (lane == 0) wsum[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        A t = 0;
        for (int w = 0; w < nw; ++w) t += wsum[w];
        *loss = (float)(t / (A)B);
    }
}
int launch_softmax_ce(int prec, const float *logits, const int *labels, float *loss, float *dlogits, int B, int C,
                      Launch s) {
    if (prec == P_BF16) launch_k(softmax_ce_kernel<float>, 1, 1024, 0, s, logits, labels, loss, dlogits, B, C);
    else launch_k(softmax_ce_kernel<double>, 1, 1024, 0, s, logits, labels, loss, dlogits, B, C);
    return 1;
}

// ------------------------------------------------------------------------------------------------------
// batch norm
// ------------------------------------------------------------------------------------------------------
// ticket counter (32 floats) + per-CTA partial sums, sized for the fp64 partials of the fp32 mode
size_t bn_scratch_elems(int C) { return 32 + (size_t)kMaxPartials * 2 * C * 2; }

static int bn_grid(long npix, int lanes) {
    long g = (npix + (long)lanes * 8 - 1) / ((long)lanes * 8);
    if (g < 1) g = 1;
    if (g > kMaxPartials) g = kMaxPartials;
    return (int)g;
}

// Two per-channel sums over all pixels.  MODE 0: (sum x, sum x^2) -> mean, invstd.
// MODE 1: (sum dz, sum dz*xhat) -> dbeta, dgamma, with dz = dout * [out > 0] when relu.
template <typename T, int VEC, int MODE>
__global__ void __launch_bounds__(kThreads)
bn_reduce_kernel(const T *__restrict__ x, const T *__restrict__ dout, const T *__restrict__ out,
                 const float *__restrict__ mean_in, const float *__restrict__ invstd_in, float *o0, float *o1,
                 float *scratch, long npix, int C, int relu) {
    pdl_launch();
    pdl_wait();
    typedef typename AccOf<T>::type A;
    __shared__ A sm[kThreads * VEC];
    __shared__ bool is_last;
    unsigned *counter = reinterpret_cast<unsigned *>(scratch);
    A *part = reinterpret_cast<A *>(scratch + 32);
    const int groups = C / VEC, lanes = kThreads / groups;
    const int g = threadIdx.x % groups, lane = threadIdx.x / groups;
    A s0[VEC], s1[VEC], mu[VEC], is[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) { s0[j] = 0; s1[j] = 0; mu[j] = 0; is[j] = 0; }
    if (MODE == 1 && lane < lanes) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) { mu[j] = mean_in[g * VEC + j]; is[j] = invstd_in[g * VEC + j]; }
    }
    if (lane < lanes) {
        for (long p = (long)blockIdx.x * lanes + lane; p < npix; p += (long)gridDim.x * lanes) {
            A xv[VEC];
            load_a<T, A, VEC>(x + p * C + g * VEC, xv);
            if (MODE == 0) {
#pragma unroll
                for (int j = 0; j < VEC; ++j) { s0[j] += xv[j]; s1[j] += xv[j] * xv[j]; }
            } else {
                A dv[VEC];
                load_a<T, A, VEC>(dout + p * C + g * VEC, dv);
                if (relu) {
                    float ov[VEC];
                    load_f<T, VEC>(out + p * C + g * VEC, ov);
#pragma unroll
                    for (int j = 0; j < VEC; ++j) if (!(ov[j] > 0.f)) dv[j] = 0;
                }
#pragma unroll
                for (int j = 0; j < VEC; ++j) { s0[j] += dv[j]; s1[j] += dv[j] * (xv[j] - mu[j]) * is[j]; }
            }
        }
    }
    // fold the pixel lanes of this CTA in a fixed order
    for (int pass = 0; pass < 2; ++pass) {
        __syncthreads();
        if (lane < lanes) {
#pragma unroll
            for (int j = 0; j < VEC; ++j) sm[lane * C + g * VEC + j] = pass == 0 ? s0[j] : s1[j];
        }
        __syncthreads();
        if (threadIdx.x < C) {
            A t = 0;
            for (int l = 0; l < lanes; ++l) t += sm[l * C + threadIdx.x];
            part[(size_t)blockIdx.x * 2 * C + pass * C + threadIdx.x] = t;
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(counter, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // fold the per-CTA partials with the whole CTA: value v (0..2C) is summed by kThreads/(2C) threads over interleaved
    // partials (several loads in flight each), then combined in a fixed order
    __shared__ double fold[kThreads];
    const int nval = 2 * C;
    const int ways = kThreads / nval;  // >= 1: C <= 128 on this path, checked by the host
    const int v = threadIdx.x % nval, way = threadIdx.x / nval;
    double acc = 0.0;
    if (way < ways)
        for (unsigned i = way; i < gridDim.x; i += ways) acc += (double)__ldcg(part + (size_t)i * 2 * C + v);
    fold[threadIdx.x] = acc;
    __syncthreads();
    for (int c = threadIdx.x; c < C; c += kThreads) {
        double a = 0.0, b = 0.0;
        for (int w = 0; w < ways; ++w) { a += fold[w * nval + c]; b += fold[w * nval + C + c]; }
        if (MODE == 0) {
            double m = a / (double)npix, var = b / (double)npix - m * m;
            if (var < 0.0) var = 0.0;
            o0[c] = (float)m;
            o1[c] = (float)(1.0 / sqrt(var + (double)kBnEps));
        } else {
            o0[c] = (float)a;  // dbeta
            o1[c] = (float)b;  // dgamma
        }
    }
    if (threadIdx.x == 0) *counter = 0u;
}

// Fast path of the per-channel reductions (C/VEC a power of two <= 32): 512-thread CTAs, at most one per SM; the
// tensor is walked as a flat array of 16-byte vectors with a stride that is a multiple of the vectors per pixel, so a
// thread always sees the same channels; four vectors per trip with all loads issued first.  Folding order is fixed:
// lanes of a warp by xor-shuffles, warps of a CTA in index order, CTAs in index order by the last CTA to finish.
static constexpr int kRedThreads = 512;

template <typename T, int VEC, int MODE, int U>
__global__ void __launch_bounds__(kRedThreads, U == 2 ? 2 : 1)
bn_reduce_fast_kernel(const T *__restrict__ x, const T *__restrict__ dout, const T *__restrict__ out,
                      const float *__restrict__ mean_in, const float *__restrict__ invstd_in, float *o0, float *o1,
                      float *scratch, long npix, int C, int relu) {
    pdl_launch();
    pdl_wait();
    typedef typename AccOf<T>::type A;
    constexpr int kWarps = kRedThreads / 32;
    __shared__ A sm[kWarps][2 * 128];  // per-warp sums of the 2C values (C <= 128)
    __shared__ bool is_last;
    unsigned *counter = reinterpret_cast<unsigned *>(scratch);
    A *part = reinterpret_cast<A *>(scratch + 32);
    const int groups = C / VEC;
    const long nvec = npix * groups;
    const long tid = (long)blockIdx.x * kRedThreads + threadIdx.x, stride = (long)gridDim.x * kRedThreads;
    const int grp = (int)(tid & (groups - 1)), c0 = grp * VEC;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    A s0[VEC], s1[VEC], mu[VEC], is[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        s0[j] = 0; s1[j] = 0;
        mu[j] = MODE == 1 ? (A)mean_in[c0 + j] : (A)0;
        is[j] = MODE == 1 ? (A)invstd_in[c0 + j] : (A)0;
    }
    // U vectors per trip: 4 with one CTA per SM (small tensors: one trip, lowest latency), 2 with two CTAs per SM
    // (large tensors: more loads in flight per SM)
    for (long i0 = tid; i0 < nvec; i0 += U * stride) {
        A xv[U][VEC], dv[U][VEC];
        float ov[U][VEC];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long i = i0 + u * stride;
            if (i < nvec) {
                load_a<T, A, VEC>(x + i * VEC, xv[u]);
                if (MODE == 1) {
                    load_a<T, A, VEC>(dout + i * VEC, dv[u]);
                    if (relu) load_f<T, VEC>(out + i * VEC, ov[u]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i0 + u * stride < nvec) {
#pragma unroll
                for (int j = 0; j < VEC; ++j) {
                    if (MODE == 0) { s0[j] += xv[u][j]; s1[j] += xv[u][j] * xv[u][j]; }
                    else {
                        A d = dv[u][j];
                        if (relu && !(ov[u][j] > 0.f)) d = 0;
                        s0[j] += d; s1[j] += d * (xv[u][j] - mu[j]) * is[j];
                    }
                }
            }
        }
    }
    // lanes of a warp that hold the same channels: lane ids equal modulo `groups`
    for (int o = 16; o >= groups; o >>= 1) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) {
            s0[j] += __shfl_xor_sync(0xffffffffu, s0[j], o);
            s1[j] += __shfl_xor_sync(0xffffffffu, s1[j], o);
        }
    }
    if (lane < groups) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) { sm[warp][c0 + j] = s0[j]; sm[warp][C + c0 + j] = s1[j]; }
    }
    __syncthreads();
    if (threadIdx.x < 2 * C) {
        A t = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t += sm[w][threadIdx.x];
        part[(size_t)blockIdx.x * 2 * C + threadIdx.x] = t;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(counter, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    __shared__ double fold[kRedThreads];
    const int nval = 2 * C, ways = kRedThreads / nval;
    if (sizeof(A) == 4) {
        // fp32 partials (bf16 tensors): all rows in batches of 16-byte loads, eight in flight per thread.  A thread of the
        // walk below adds its rows one after the other, four loads in flight: with 148 rows of 128 values that alone
        // was 7 us of an 11 us kernel.  The per-warp sums are consumed: their 16 KB hold the per-thread totals.
        fold_partials<kRedThreads>(reinterpret_cast<const float *>(part), (int)gridDim.x, nval, reinterpret_cast<double *>(&sm[0][0]), fold);
    } else {
        const int v = threadIdx.x % nval, way = threadIdx.x / nval;
        double acc = 0.0;
        if (way < ways) {
            double a4[4] = {0.0, 0.0, 0.0, 0.0};
            unsigned i = way;
            for (; i + 3 * ways < gridDim.x; i += 4 * ways) {
#pragma unroll
                for (int u = 0; u < 4; ++u) a4[u] += (double)__ldcg(part + (size_t)(i + u * ways) * nval + v);
            }
            for (; i < gridDim.x; i += ways) a4[0] += (double)__ldcg(part + (size_t)i * nval + v);
            acc = (a4[0] + a4[1]) + (a4[2] + a4[3]);
        }
        fold[threadIdx.x] = acc;
        __syncthreads();
    }
    if (threadIdx.x < C) {
        const int c = threadIdx.x;
        double a = 0.0, b = 0.0;
        if (sizeof(A) == 4) { a = fold[c]; b = fold[C + c]; }
        else for (int w = 0; w < ways; ++w) { a += fold[w * nval + c]; b += fold[w * nval + C + c]; }
        if (MODE == 0) {
            double m = a / (double)npix, var = b / (double)npix - m * m;
            if (var < 0.0) var = 0.0;
            o0[c] = (float)m;
            o1[c] = (float)(1.0 / sqrt(var + (double)kBnEps));
        } else {
            o0[c] = (float)a;  // dbeta
            o1[c] = (float)b;  // dgamma
        }
    }
    if (threadIdx.x == 0) *counter = 0u;
}

static bool red_fast_ok(int C, int V) {
    if (C % V != 0 || C > 128) return false;
    const int groups = C / V;
    return (groups & (groups - 1)) == 0 && groups <= 32;
}
static int red_fast_grid(long nvec, int per_sm) {
    long g = (nvec + 4L * kRedThreads - 1) / (4L * kRedThreads);
    if (g > 148 * per_sm) g = 148 * per_sm;
    return (int)(g < 1 ? 1 : g);
}

__device__ __forceinline__ void unpack_bf16x8(const uint4 &q, float (&f)[8]) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        f[2 * k] = __uint_as_float(w[k] << 16);
        f[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
}
__device__ __forceinline__ uint4 pack_bf16x8(const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
        w[k] = *reinterpret_cast<const uint32_t *>(&h);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
}


// Reductions over large bf16 tensors (more vectors than one trip of the kernel above covers): one 768-thread CTA per
// SM (few partials for the last CTA to fold), operands kept as raw 16-byte registers with the loads of U vectors of
// each issued before the first use, so that an SM has ~70 KB of loads in flight.  The second backward sum is accumulated as sum dz*(x - mean) and scaled by
// invstd once at the end.  Same fixed folding order as above: lanes, warps, then CTAs in index order by the last CTA.
static constexpr int kBigThreads = 768;

template <int MODE, int U>
__global__ void __launch_bounds__(kBigThreads, 1)
bn_reduce_big_kernel(const bf16 *__restrict__ x, const bf16 *__restrict__ dout, const bf16 *__restrict__ out,
                     const float *__restrict__ mean_in, const float *__restrict__ invstd_in, float *o0, float *o1,
                     float *scratch, long npix, int C, int relu) {
    pdl_launch();
    pdl_wait();
    constexpr int kWarps = kBigThreads / 32;
    __shared__ float sm[kWarps][2 * 128];
    __shared__ bool is_last;
    __shared__ double fold[kBigThreads];
    unsigned *counter = reinterpret_cast<unsigned *>(scratch);
    float *part = scratch + 32;
    const int groups = C / 8;
    const long nvec = npix * groups;
    const long tid = (long)blockIdx.x * kBigThreads + threadIdx.x, stride = (long)gridDim.x * kBigThreads;
    const int c0 = (int)(tid & (groups - 1)) * 8;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float s0[8], s1[8], mu[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { s0[j] = 0.f; s1[j] = 0.f; mu[j] = MODE == 1 ? mean_in[c0 + j] : 0.f; }
    const uint4 *x4 = reinterpret_cast<const uint4 *>(x), *d4 = reinterpret_cast<const uint4 *>(dout),
                *o4 = reinterpret_cast<const uint4 *>(out);
    for (long i0 = tid; i0 < nvec; i0 += U * stride) {
        uint4 xq[U], dq[U], oq[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long i = i0 + u * stride;
            if (i < nvec) {
                xq[u] = x4[i];
                if (MODE == 1) {
                    dq[u] = d4[i];
                    if (relu) oq[u] = o4[i];
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (i0 + u * stride < nvec) {
                float xv[8], dv[8], ov[8];
                unpack_bf16x8(xq[u], xv);
                if (MODE == 1) {
                    unpack_bf16x8(dq[u], dv);
                    if (relu) unpack_bf16x8(oq[u], ov);
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (MODE == 0) { s0[j] += xv[j]; s1[j] = fmaf(xv[j], xv[j], s1[j]); }
                    else {
                        const float d = (relu && !(ov[j] > 0.f)) ? 0.f : dv[j];
                        s0[j] += d;
                        s1[j] = fmaf(d, xv[j] - mu[j], s1[j]);
                    }
                }
            }
        }
    }
    for (int o = 16; o >= groups; o >>= 1) {
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            s0[j] += __shfl_xor_sync(0xffffffffu, s0[j], o);
            s1[j] += __shfl_xor_sync(0xffffffffu, s1[j], o);
        }
    }
    if (lane < groups) {
#pragma unroll
        for (int j = 0; j < 8; ++j) { sm[warp][c0 + j] = s0[j]; sm[warp][C + c0 + j] = s1[j]; }
    }
    __syncthreads();
    if (threadIdx.x < 2 * C) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t += sm[w][threadIdx.x];
        part[(size_t)blockIdx.x * 2 * C + threadIdx.x] = t;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = (atomicAdd(counter, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    // all partial rows in one batch of 16-byte loads; the per-warp sums are consumed, their 24 KB hold the per-thread totals
    fold_partials<kBigThreads>(part, (int)gridDim.x, 2 * C, reinterpret_cast<double *>(&sm[0][0]), fold);
    if (threadIdx.x < C) {
        const int c = threadIdx.x;
        const double a = fold[c], b = fold[C + c];
        if (MODE == 0) {
            double m = a / (double)npix, var = b / (double)npix - m * m;
            if (var < 0.0) var = 0.0;
            o0[c] = (float)m;
            o1[c] = (float)(1.0 / sqrt(var + (double)kBnEps));
        } else {
            o0[c] = (float)a;                             // dbeta
            o1[c] = (float)(b * (double)invstd_in[c]);  // dgamma
        }
    }
    if (threadIdx.x == 0) *counter = 0u;
}

static bool red_big_ok(int prec, long nvec, int C) {
    return prec == P_BF16 && C % 8 == 0 && C <= 128 && red_fast_ok(C, 8) && nvec > 16L * 148 * kRedThreads;
}
static int red_big_grid(long nvec, int U) {
    long g = (nvec + (long)kBigThreads * U - 1) / ((long)kBigThreads * U);
    return (int)(g > 148 ? 148 : g);
}

template <typename T> static int vec_for(int C) { return (C % Vec16<T>::N == 0) ? Vec16<T>::N : 1; }

int launch_bn_stats(int prec, const void *x, float *mean, float *invstd, float *scratch, long npix, int C,
                    Launch s) {
    if (red_big_ok(prec, npix * (C / 8), C)) {
        launch_k(bn_reduce_big_kernel<0, 4>, red_big_grid(npix * (C / 8), 4), kBigThreads, 0, s, (const bf16 *)x, (const bf16 *)nullptr,
                 (const bf16 *)nullptr, (const float *)nullptr, (const float *)nullptr, mean, invstd, scratch, npix, C, 0);
        return 1;
    }
    DISPATCH_PREC(prec, {
        if (red_fast_ok(C, Vec16<T>::N)) {
            constexpr int V = Vec16<T>::N;
            launch_k(bn_reduce_fast_kernel<T, V, 0, 4>, red_fast_grid(npix * (C / V), 1), kRedThreads, 0, s, (const T *)x,
                     nullptr, nullptr, nullptr, nullptr, mean, invstd, scratch, npix, C, 0);
        } else if (vec_for<T>(C) > 1) {
            constexpr int V = Vec16<T>::N;
            launch_k(bn_reduce_kernel<T, V, 0>, bn_grid(npix, kThreads / (C / V)), kThreads, 0, s, (const T *)x, nullptr, nullptr, nullptr, nullptr, mean, invstd, scratch, npix, C, 0);
        } else {
            launch_k(bn_reduce_kernel<T, 1, 0>, bn_grid(npix, kThreads / C), kThreads, 0, s, (const T *)x, nullptr, nullptr, nullptr, nullptr, mean, invstd, scratch, npix, C, 0);
        }
    });
    return 1;
}

int launch_bn_bwd_reduce(int prec, const void *dout, const void *out, const void *x, const float *mean,
                         const float *invstd, float *dgamma, float *dbeta, float *scratch, long npix, int C, int relu,
                         Launch s) {
    if (red_big_ok(prec, npix * (C / 8), C)) {
        launch_k(bn_reduce_big_kernel<1, 2>, red_big_grid(npix * (C / 8), 2), kBigThreads, 0, s, (const bf16 *)x, (const bf16 *)dout,
                 (const bf16 *)out, mean, invstd, dbeta, dgamma, scratch, npix, C, relu);
        return 1;
    }
    DISPATCH_PREC(prec, {
        if (red_fast_ok(C, Vec16<T>::N)) {
            constexpr int V = Vec16<T>::N;
            const long nvec = npix * (C / V);
            if (nvec > 16L * 148 * kRedThreads)  // large: two CTAs per SM keep more loads in flight
                launch_k(bn_reduce_fast_kernel<T, V, 1, 2>, red_fast_grid(nvec, 2), kRedThreads, 0, s, (const T *)x,
                         (const T *)dout, (const T *)out, mean, invstd, dbeta, dgamma, scratch, npix, C, relu);
            else
                launch_k(bn_reduce_fast_kernel<T, V, 1, 4>, red_fast_grid(nvec, 1), kRedThreads, 0, s, (const T *)x,
                         (const T *)dout, (const T *)out, mean, invstd, dbeta, dgamma, scratch, npix, C, relu);
        } else if (vec_for<T>(C) > 1) {
            constexpr int V = Vec16<T>::N;
            launch_k(bn_reduce_kernel<T, V, 1>, bn_grid(npix, kThreads / (C / V)), kThreads, 0, s, (const T *)x, (const T *)dout, (const T *)out, mean, invstd, dbeta, dgamma, scratch, npix, C, relu);
        } else {
            launch_k(bn_reduce_kernel<T, 1, 1>, bn_grid(npix, kThreads / C), kThreads, 0, s, (const T *)x, (const T *)dout, (const T *)out, mean, invstd, dbeta, dgamma, scratch, npix, C, relu);
        }
    });
    return 1;
}

// y = [relu](gamma*(x-mean)*invstd + beta + shortcut)
template <typename T, int VEC>
__global__ void __launch_bounds__(kThreads)
bn_apply_kernel(const T *__restrict__ x, const T *__restrict__ gamma, const T *__restrict__ beta,
                const float *__restrict__ mean, const float *__restrict__ invstd, Shortcut sc, T *__restrict__ y,
                long nvec, int H, int W, int C, int relu) {
    pdl_launch();
    pdl_wait();
    long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nvec) return;
    const int groups = C / VEC;
    const int c0 = (int)(i % groups) * VEC;
    const long p = i / groups;
    typedef typename AccOf<T>::type A;
    A v[VEC];
    load_a<T, A, VEC>(x + p * C + c0, v);
#pragma unroll
    for (int j = 0; j < VEC; ++j)
        v[j] = (A)to_f(gamma[c0 + j]) * (v[j] - (A)mean[c0 + j]) * (A)invstd[c0 + j] + (A)to_f(beta[c0 + j]);
    if (sc.mode == 1) {
        A r[VEC];
        load_a<T, A, VEC>((const T *)sc.a + p * C + c0, r);
#pragma unroll
        for (int j = 0; j < VEC; ++j) v[j] += r[j];
    } else if (sc.mode == 2) {
        if (c0 < sc.c_small) {  // host guarantees c_small % VEC == 0 on the vector path
            const int wo = (int)(p % W), ho = (int)((p / W) % H);
            const long n = p / ((long)W * H);
            const long q = (n * sc.h_big + 2 * ho) * sc.w_big + 2 * wo;
            A r[VEC];
            load_a<T, A, VEC>((const T *)sc.a + q * sc.c_small + c0, r);
#pragma unroll
            for (int j = 0; j < VEC; ++j) if (c0 + j < sc.c_small) v[j] += r[j];
        }
    }
    if (relu) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) v[j] = v[j] > 0 ? v[j] : (A)0;
    }
    store_a<T, A, VEC>(y + p * C + c0, v);
}

// Fast path of the element-wise pass for bf16 tensors (no shortcut or the identity shortcut; C/8 a power of two):
// the per-channel constants are folded once per CTA into scale = gamma*invstd and shift = beta - mean*scale (shared
// memory, then registers: the flat 16-byte-vector walk keeps a thread on the same 8 channels), a thread issues the
// loads of U vectors of every operand, kept as raw 16-byte registers, before it uses the first, and the grid is
// capped at three CTAs per SM.
static constexpr int kApplyCtasPerSm = 3;

// FOLD: the statistics come as per-CTA partial sums that this kernel adds up first (an instantiation of its own: the
// 10 KB of shared memory the fold needs would otherwise sit in every launch and keep other streams' CTAs off the SM)
template <int U, bool FOLD>
__global__ void __launch_bounds__(kThreads, kApplyCtasPerSm)
bn_apply_fast_kernel(const bf16 *__restrict__ x, const bf16 *__restrict__ gamma, const bf16 *__restrict__ beta,
                     float *__restrict__ mean, float *__restrict__ invstd, const bf16 *__restrict__ res,
                     bf16 *__restrict__ y, long nvec, int C, int relu, const float *__restrict__ part, int n_part) {
    __shared__ float sm_scale[128], sm_shift[128];
    pdl_launch();
    pdl_wait();
    if (FOLD) {
        // statistics from the convolution epilogue's partial sums (sum x, sum x^2): every CTA folds them the same way
        __shared__ double sm_fold[kThreads * 4], sm_tot[256];
        fold_partials<kThreads>(part, n_part, 2 * C, sm_fold, sm_tot);
        const double npix = (double)(nvec / (C / 8));
        for (int c = threadIdx.x; c < C; c += kThreads) {
            const double m = sm_tot[c] / npix;
            double var = sm_tot[C + c] / npix - m * m;
            if (var < 0.0) var = 0.0;
            const float mf = (float)m, isf = (float)(1.0 / sqrt(var + (double)kBnEps));
            if (blockIdx.x == 0) { mean[c] = mf; invstd[c] = isf; }  // the backward sweep reads them
            const float sc = to_f(gamma[c]) * isf;
            sm_scale[c] = sc;
            sm_shift[c] = to_f(beta[c]) - mf * sc;
        }
    } else {
        for (int c = threadIdx.x; c < C; c += kThreads) {
            const float sc = to_f(gamma[c]) * invstd[c];
            sm_scale[c] = sc;
            sm_shift[c] = to_f(beta[c]) - mean[c] * sc;
        }
    }
    __syncthreads();
    const int groups = C / 8;
    const long tid = (long)blockIdx.x * kThreads + threadIdx.x, stride = (long)gridDim.x * kThreads;
    const int c0 = (int)(tid & (groups - 1)) * 8;
    float sc[8], sh[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { sc[j] = sm_scale[c0 + j]; sh[j] = sm_shift[c0 + j]; }
    const uint4 *x4 = reinterpret_cast<const uint4 *>(x), *r4 = reinterpret_cast<const uint4 *>(res);
    uint4 *y4 = reinterpret_cast<uint4 *>(y);
    for (long i0 = tid; i0 < nvec; i0 += U * stride) {
        uint4 xq[U], rq[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long i = i0 + u * stride;
            if (i < nvec) {
                xq[u] = x4[i];
                if (res != nullptr) rq[u] = r4[i];
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long i = i0 + u * stride;
            if (i < nvec) {
                float v[8], r[8];
                unpack_bf16x8(xq[u], v);
                if (res != nullptr) unpack_bf16x8(rq[u], r);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float t = fmaf(v[j], sc[j], sh[j]);
                    if (res != nullptr) t += r[j];
                    v[j] = (relu && !(t > 0.f)) ? 0.f : t;
                }
                y4[i] = pack_bf16x8(v);
            }
        }
    }
}

static bool apply_fast_ok(int C, int V) {
    if (C % V != 0 || C > 128) return false;
    const int groups = C / V;
    return (groups & (groups - 1)) == 0 && groups <= 32;
}
// vectors per thread and trip: as many as still leave every SM its three CTAs
static int apply_unroll(long nvec) {
    const long full = 148L * kApplyCtasPerSm * kThreads;
    return nvec >= 4 * full ? 4 : (nvec >= 2 * full ? 2 : 1);
}
static int apply_grid(long nvec, int U) {
    long g = (nvec + (long)kThreads * U - 1) / ((long)kThreads * U);
    // tensors of the training step's size: two CTAs per SM, which leaves registers for a convolution CTA of another
    // stream beside them (K = 4 step 0.8 % faster than with three); large tensors: three, for the loads in flight
    const int cap = U == 4 ? kApplyCtasPerSm : 2;
    if (g > 148L * cap) g = 148L * cap;
    return (int)(g < 1 ? 1 : g);
}

bool bn_apply_takes_partials(int prec, int C, int shortcut_mode) {
    return prec == P_BF16 && shortcut_mode != 2 && apply_fast_ok(C, Vec16<bf16>::N) && (1024 % (2 * C)) == 0;
}

int launch_bn_apply(int prec, const void *x, const void *gamma, const void *beta, float *mean, float *invstd,
                    Shortcut sc, void *y, int B, int H, int W, int C, int relu, Launch s, BnPartials bp) {
    const long npix = (long)B * H * W;
    if (bp.part != nullptr && !bn_apply_takes_partials(prec, C, sc.mode)) return -1;
    if (prec == P_BF16 && sc.mode != 2 && apply_fast_ok(C, Vec16<bf16>::N)) {
        typedef bf16 T;
        constexpr int V = Vec16<T>::N;
        const long nvec = npix * (C / V);
        const int U = apply_unroll(nvec);
        const T *res = sc.mode == 1 ? (const T *)sc.a : nullptr;
        auto k = U == 4 ? bn_apply_fast_kernel<4, false> : (U == 2 ? bn_apply_fast_kernel<2, false> : bn_apply_fast_kernel<1, false>);
        if (bp.part != nullptr)
            k = U == 4 ? bn_apply_fast_kernel<4, true> : (U == 2 ? bn_apply_fast_kernel<2, true> : bn_apply_fast_kernel<1, true>);
        launch_k(k, apply_grid(nvec, U), kThreads, 0, s, (const T *)x, (const T *)gamma, (const T *)beta, mean, invstd, res,
                 (T *)y, nvec, C, relu, bp.part, bp.n);
        return 1;
    }
    DISPATCH_PREC(prec, {
        constexpr int V = Vec16<T>::N;
        if (C % V == 0 && (sc.mode != 2 || sc.c_small % V == 0)) {
            long nvec = npix * (C / V);
            launch_k(bn_apply_kernel<T, V>, ceil_div(nvec, kThreads), kThreads, 0, s, (const T *)x, (const T *)gamma, (const T *)beta, mean, invstd, sc, (T *)y, nvec, H, W, C, relu);
        } else {
            long nvec = npix * C;
            launch_k(bn_apply_kernel<T, 1>, ceil_div(nvec, kThreads), kThreads, 0, s, (const T *)x, (const T *)gamma, (const T *)beta, mean, invstd, sc, (T *)y, nvec, H, W, C, relu);
        }
    });
    return 1;
}

// dx = gamma*invstd*(dz - dbeta/n - xhat*dgamma/n)
template <typename T, int VEC>
__global__ void __launch_bounds__(kThreads)
bn_bwd_apply_kernel(const T *__restrict__ dout, const T *__restrict__ out, const T *__restrict__ x,
                    const T *__restrict__ gamma, const float *__restrict__ mean, const float *__restrict__ invstd,
                    const float *__restrict__ dgamma, const float *__restrict__ dbeta, T *__restrict__ dx, long nvec,
                    long npix, int C, int relu) {
    pdl_launch();
    pdl_wait();
    long i = (long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= nvec) return;
    const int groups = C / VEC;
    const int c0 = (int)(i % groups) * VEC;
    const long p = i / groups;
    typedef typename AccOf<T>::type A;
    A xv[VEC], dv[VEC];
    load_a<T, A, VEC>(x + p * C + c0, xv);
    load_a<T, A, VEC>(dout + p * C + c0, dv);
    if (relu) {
        float ov[VEC];
        load_f<T, VEC>(out + p * C + c0, ov);
#pragma unroll
        for (int j = 0; j < VEC; ++j) if (!(ov[j] > 0.f)) dv[j] = 0;
    }
    const A cnt = (A)npix;
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        const int c = c0 + j;
        const A xh = (xv[j] - (A)mean[c]) * (A)invstd[c];
        dv[j] = (A)to_f(gamma[c]) * (A)invstd[c] * (dv[j] - (A)dbeta[c] / cnt - xh * (A)dgamma[c] / cnt);
    }
    store_a<T, A, VEC>(dx + p * C + c0, dv);
}

// Fast path for bf16 tensors, laid out like bn_apply_fast_kernel.  With gi = gamma*invstd and n pixels,
//   dx = gi*(dz - dbeta/n - xhat*dgamma/n) = gi*dz + k1*x + k0,  k1 = -gi*invstd*dgamma/n,  k0 = -gi*dbeta/n - k1*mean.
template <int U, bool FOLD>
__global__ void __launch_bounds__(kThreads, kApplyCtasPerSm)
bn_bwd_apply_fast_kernel(const bf16 *__restrict__ dout, const bf16 *__restrict__ out, const bf16 *__restrict__ x,
                         const bf16 *__restrict__ gamma, const float *__restrict__ mean, const float *__restrict__ invstd,
                         float *__restrict__ dgamma, float *__restrict__ dbeta, bf16 *__restrict__ dx,
                         long nvec, long npix, int C, int relu, const float *__restrict__ part, int n_part) {
    __shared__ float sm_gi[128], sm_k1[128], sm_k0[128];
    pdl_launch();
    pdl_wait();
    __shared__ double sm_tot[FOLD ? 256 : 1];
    if (FOLD) {
        // (sum dz, sum dz * xhat) from the partial sums of the input-gradient convolution's epilogue
        __shared__ double sm_fold[kThreads * 4];
        fold_partials<kThreads>(part, n_part, 2 * C, sm_fold, sm_tot);
    }
    for (int c = threadIdx.x; c < C; c += kThreads) {
        float db, dg;
        if (FOLD) {
            db = (float)sm_tot[c]; dg = (float)sm_tot[C + c];
            if (blockIdx.x == 0) { dbeta[c] = db; dgamma[c] = dg; }  // the parameter gradients of this batch norm
        } else {
            db = dbeta[c]; dg = dgamma[c];
        }
        const float inv_n = 1.f / (float)npix;
        const float gi = to_f(gamma[c]) * invstd[c];
        const float k1 = -gi * invstd[c] * dg * inv_n;
        sm_gi[c] = gi;
        sm_k1[c] = k1;
        sm_k0[c] = -gi * db * inv_n - k1 * mean[c];
    }
    __syncthreads();
    const int groups = C / 8;
    const long tid = (long)blockIdx.x * kThreads + threadIdx.x, stride = (long)gridDim.x * kThreads;
    const int c0 = (int)(tid & (groups - 1)) * 8;
    float gi[8], k1[8], k0[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) { gi[j] = sm_gi[c0 + j]; k1[j] = sm_k1[c0 + j]; k0[j] = sm_k0[c0 + j]; }
    const uint4 *x4 = reinterpret_cast<const uint4 *>(x), *d4 = reinterpret_cast<const uint4 *>(dout),
                *o4 = reinterpret_cast<const uint4 *>(out);
    uint4 *dx4 = reinterpret_cast<uint4 *>(dx);
    for (long i0 = tid; i0 < nvec; i0 += U * stride) {
        uint4 xq[U], dq[U], oq[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long i = i0 + u * stride;
            if (i < nvec) {
                xq[u] = x4[i];
                dq[u] = d4[i];
                if (relu) oq[u] = o4[i];
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long i = i0 + u * stride;
            if (i < nvec) {
                float xv[8], dv[8], ov[8];
                unpack_bf16x8(xq[u], xv);
                unpack_bf16x8(dq[u], dv);
                if (relu) unpack_bf16x8(oq[u], ov);
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const float d = (relu && !(ov[j] > 0.f)) ? 0.f : dv[j];
                    dv[j] = fmaf(gi[j], d, fmaf(k1[j], xv[j], k0[j]));
                }
                dx4[i] = pack_bf16x8(dv);
            }
        }
    }
}

int launch_bn_bwd_apply(int prec, const void *dout, const void *out, const void *x, const void *gamma,
                        const float *mean, const float *invstd, float *dgamma, float *dbeta, void *dx,
                        long npix, int C, int relu, Launch s, BnPartials bp) {
    if (bp.part != nullptr && !bn_apply_takes_partials(prec, C, 0)) return -1;
    if (prec == P_BF16 && apply_fast_ok(C, Vec16<bf16>::N)) {
        typedef bf16 T;
        constexpr int V = Vec16<T>::N;
        const long nvec = npix * (C / V);
        const int U = apply_unroll(nvec) >= 2 ? 2 : 1;  // three operands: two vectors of each in flight per thread
        auto k = U == 2 ? bn_bwd_apply_fast_kernel<2, false> : bn_bwd_apply_fast_kernel<1, false>;
        if (bp.part != nullptr) k = U == 2 ? bn_bwd_apply_fast_kernel<2, true> : bn_bwd_apply_fast_kernel<1, true>;
        launch_k(k, apply_grid(nvec, U), kThreads, 0, s, (const T *)dout, (const T *)out, (const T *)x, (const T *)gamma, mean,
                 invstd, dgamma, dbeta, (T *)dx, nvec, npix, C, relu, bp.part, bp.n);
        return 1;
    }
    DISPATCH_PREC(prec, {
        constexpr int V = Vec16<T>::N;
        if (C % V == 0) {
            long nvec = npix * (C / V);
            launch_k(bn_bwd_apply_kernel<T, V>, ceil_div(nvec, kThreads), kThreads, 0, s, (const T *)dout, (const T *)out, (const T *)x, (const T *)gamma, mean, invstd, dgamma, dbeta, (T *)dx,
                nvec, npix, C, relu);
        } else {
            long nvec = npix * C;
            launch_k(bn_bwd_apply_kernel<T, 1>, ceil_div(nvec, kThreads), kThreads, 0, s, (const T *)dout, (const T *)out, (const T *)x, (const T *)gamma, mean, invstd, dgamma, dbeta, (T *)dx,
                nvec, npix, C, relu);
        }
    });
    return 1;
}

// ------------------------------------------------------------------------------------------------------
// optimiser update with the delayed gradient (Eq. 9 / Algorithm 1, Algorithm 2) + weight-version refresh
// ------------------------------------------------------------------------------------------------------
static constexpr int kUpdVecs = 2;  // float4 groups per thread, all loads issued before the first use

// one parameter: master weight, first (and second) moment, gradient
// lr, c1c, c2c: the step size and Adam's bias corrections of this iteration (by value or from the device block)
template <typename A>
__device__ __forceinline__ void update_one(float &w, float &v, float &m2, float g, const UpdateArgs &a, A lr, A c1c, A c2c) {
    if (a.mode == 0) {
        const A d = (A)g + (A)a.wd * (A)w;
        const A vn = (A)a.mu * (A)v + d;
        v = (float)vn;
        w = (float)((A)w - lr * vn);
    } else if (a.mode == 1) {
        const A m1 = (A)a.b1 * (A)v + ((A)1 - (A)a.b1) * (A)g;
        const A m2n = (A)a.b2 * (A)m2 + ((A)1 - (A)a.b2) * (A)g * (A)g;
        v = (float)m1;
        m2 = (float)m2n;
        w = (float)((A)w - lr * (m1 / c1c) / (sqrt(m2n / c2c) + (A)a.eps));
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
update_kernel(float *__restrict__ w, float *__restrict__ v, float *__restrict__ m2, const float *__restrict__ g,
              T *__restrict__ wv, size_t n, UpdateArgs a) {
    pdl_launch();
    pdl_wait();
    typedef typename AccOf<T>::type A;  // the master state is fp32 either way; A is the arithmetic in between
    const A lr = a.dyn ? (A)a.dyn[0] : (A)a.lr;
    const A c1c = a.dyn ? (A)a.dyn[1] : (A)a.c1c, c2c = a.dyn ? (A)a.dyn[2] : (A)a.c2c;
    const size_t span = (size_t)gridDim.x * blockDim.x * 4;  // elements one pass of the grid covers
    const size_t base = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(g) |
                           reinterpret_cast<uintptr_t>(m2) | (reinterpret_cast<uintptr_t>(wv) * (16 / (4 * sizeof(T))));
    if ((bits & 15) == 0 && base + (kUpdVecs - 1) * span + 4 <= n) {
        float4 W[kUpdVecs], V[kUpdVecs], G[kUpdVecs], M[kUpdVecs];
#pragma unroll
        for (int u = 0; u < kUpdVecs; ++u) {
            const size_t i = base + u * span;
            W[u] = *reinterpret_cast<const float4 *>(w + i);
            if (a.mode != 2) {
                V[u] = *reinterpret_cast<const float4 *>(v + i);
                G[u] = *reinterpret_cast<const float4 *>(g + i);
                if (a.mode == 1) M[u] = *reinterpret_cast<const float4 *>(m2 + i);
            }
        }
#pragma unroll
        for (int u = 0; u < kUpdVecs; ++u) {
            const size_t i = base + u * span;
            update_one<A>(W[u].x, V[u].x, M[u].x, G[u].x, a, lr, c1c, c2c);
            update_one<A>(W[u].y, V[u].y, M[u].y, G[u].y, a, lr, c1c, c2c);
            update_one<A>(W[u].z, V[u].z, M[u].z, G[u].z, a, lr, c1c, c2c);
            update_one<A>(W[u].w, V[u].w, M[u].w, G[u].w, a, lr, c1c, c2c);
            if (a.mode != 2) {
                *reinterpret_cast<float4 *>(w + i) = W[u];
                *reinterpret_cast<float4 *>(v + i) = V[u];
                if (a.mode == 1) *reinterpret_cast<float4 *>(m2 + i) = M[u];
            }
            const float o[4] = {W[u].x, W[u].y, W[u].z, W[u].w};
            store_f<T, 4>(wv + i, o);
        }
        return;
    }
    for (int u = 0; u < kUpdVecs; ++u) {  // ragged end or unaligned arrays: element by element
        for (int j = 0; j < 4; ++j) {
            const size_t i = base + u * span + j;
            if (i >= n) break;
            float wi = w[i], vi = 0.f, mi = 0.f, gi = 0.f;
            if (a.mode != 2) { vi = v[i]; gi = g[i]; if (a.mode == 1) mi = m2[i]; }
            update_one<A>(wi, vi, mi, gi, a, lr, c1c, c2c);
            if (a.mode != 2) { w[i] = wi; v[i] = vi; if (a.mode == 1) m2[i] = mi; }
            wv[i] = from_f<T>(wi);
        }
    }
}

int launch_update(int prec, float *w, float *v, float *m2, const float *g, void *wv, size_t n, UpdateArgs a,
                  Launch s) {
    if (n == 0) return 0;
    DISPATCH_PREC(prec, launch_k(update_kernel<T>, ceil_div((n + 3) / 4, (long)kThreads * kUpdVecs), kThreads, 0, s, w, v, m2, g, (T *)wv, n, a));
    return 1;
}

__global__ void set_opt_scalars_kernel(double *dyn, double lr, double c1c, double c2c) {
    pdl_launch();
    pdl_wait();
    if (threadIdx.x == 0) { dyn[0] = lr; dyn[1] = c1c; dyn[2] = c2c; }
}
int launch_set_opt_scalars(double *dyn, double lr, double c1c, double c2c, Launch s) {
    launch_k(set_opt_scalars_kernel, 1, 32, 0, s, dyn, lr, c1c, c2c);
    return 1;
}

__global__ void stamp_kernel(StampOp op) {
    pdl_launch();
    pdl_wait();
    if (threadIdx.x != 0) return;
    const long long now = *op.counter;
    for (int i = 0; i < 3; ++i)
        if (op.check[i] != nullptr && *op.check[i] != now) atomicCAS(op.err, 0, op.code + i);
    for (int i = 0; i < 2; ++i)
        if (op.set[i] != nullptr) *op.set[i] = now + op.set_add;
    *op.counter = now + op.advance;
}
int launch_stamp(StampOp op, Launch s) {
    launch_k(stamp_kernel, 1, 32, 0, s, op);
    return 1;
}
__global__ void add_to_counter_kernel(long long *counter, long long delta) {
    pdl_launch();
    pdl_wait();
    if (threadIdx.x == 0) *counter += delta;
}
int launch_add_to_counter(long long *counter, long long delta, Launch s) {
    launch_k(add_to_counter_kernel, 1, 32, 0, s, counter, delta);
    return 1;
}

int launch_cast(int prec, const float *src, void *dst, size_t n, Launch s) {
    UpdateArgs a = {};
    a.mode = 2;
    return launch_update(prec, const_cast<float *>(src), nullptr, nullptr, nullptr, dst, n, a, s);
}

// ------------------------------------------------------------------------------------------------------
// weight initialisation: counter-based normal draws (splitmix64 hash of (seed, stream, index) + Box-Muller)
// ------------------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
    z += 0x9e3779b97f4a7c15ull;
    z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ull;
    z = (z ^ (z >> 27)) * 0x94d049bb133111ebull;
    return z ^ (z >> 31);
}
__global__ void fill_normal_kernel(float *dst, size_t n, float stddev, unsigned long long seed,
                                   unsigned long long stream_id) {
    pdl_launch();
    pdl_wait();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    unsigned long long h = mix64(mix64(seed ^ (stream_id * 0xd1342543de82ef95ull)) + i);
    unsigned long long h2 = mix64(h);
    float u1 = ((h >> 40) + 1.0f) * (1.0f / 16777217.0f);  // (0, 1)
    float u2 = (h2 >> 40) * (1.0f / 16777216.0f);
    dst[i] = stddev * sqrtf(-2.f * logf(u1)) * cospif(2.f * u2);
}
__global__ void fill_const_kernel(float *dst, size_t n, float v) {
    pdl_launch();
    pdl_wait();
    size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) dst[i] = v;
}
int launch_fill_normal(float *dst, size_t n, float stddev, unsigned long long seed, unsigned long long stream_id,
                       Launch s) {
    if (n == 0) return 0;
    launch_k(fill_normal_kernel, ceil_div(n, kThreads), kThreads, 0, s, dst, n, stddev, seed, stream_id);
    return 1;
}
int launch_fill_const(float *dst, size_t n, float v, Launch s) {
    if (n == 0) return 0;
    launch_k(fill_const_kernel, ceil_div(n, kThreads), kThreads, 0, s, dst, n, v);
    return 1;
}

}  // namespace ddg
