// CUDA-core 3x3 convolution kernels (forward, input gradient, weight gradient) for NHWC tensors of any shape.
// They carry the fp32 mode and every shape the tensor-core path does not take (stride 2, the 3-channel stem).
#include "common.cuh"
#include "conv_tc.h"
#include "kernels.h"

namespace ddg {

#define DISPATCH_PREC(prec, ...)                       \
    do {                                               \
        if ((prec) == P_BF16) { typedef bf16 T; __VA_ARGS__; } \
        else { typedef float T; __VA_ARGS__; }         \
    } while (0)

static constexpr int kConvThreads = 256;
static constexpr int kCdt = 8;  // destination channels per thread

// One kernel for both directions.  "src" is x (forward) or dy (input gradient); "dst" is y or dx.
//   forward : dst pixel (ho,wo) reads src pixel (s*ho+ky-1, s*wo+kx-1)
//   dgrad   : dst pixel (hi,wi) reads src pixel ((hi+1-ky)/s, (wi+1-kx)/s) when both divisions are exact
// Weights are staged in shared memory as float [tap][Cs][Cd].
template <typename T, int DGRAD>
__global__ void __launch_bounds__(kConvThreads)
conv3x3_direct_kernel(const T *__restrict__ src, const T *__restrict__ w, T *__restrict__ dst, int B, int Hs, int Ws,
                      int Cs, int Hd, int Wd, int Cd, int stride, int relu, Shortcut sc) {
    pdl_launch();
    pdl_wait();
    extern __shared__ float wsm[];
    const int Cin = DGRAD ? Cd : Cs, Cout = DGRAD ? Cs : Cd;
    for (int i = threadIdx.x; i < 9 * Cs * Cd; i += blockDim.x) {
        const int cd = i % Cd, cs = (i / Cd) % Cs, tap = i / (Cd * Cs);
        const int ci = DGRAD ? cd : cs, co = DGRAD ? cs : cd;
        wsm[i] = to_f(w[((size_t)co * Cin + ci) * 9 + tap]);
    }
    __syncthreads();
    const int groups = (Cd + kCdt - 1) / kCdt;
    const int pix_per_cta = kConvThreads / groups;
    const int grp = threadIdx.x / pix_per_cta, pl = threadIdx.x % pix_per_cta;
    if (grp >= groups) return;
    const long npix = (long)B * Hd * Wd;
    const long p = (long)blockIdx.x * pix_per_cta + pl;
    if (p >= npix) return;
    const int wd = (int)(p % Wd), hd = (int)((p / Wd) % Hd);
    const long n = p / ((long)Wd * Hd);
    const int cd0 = grp * kCdt;
    typedef typename AccOf<T>::type A;
    A acc[kCdt];
#pragma unroll
    for (int j = 0; j < kCdt; ++j) acc[j] = 0;
    constexpr int V = Vec16<T>::N;
    const bool vec_ok = (Cs % V) == 0;
    for (int ky = 0; ky < 3; ++ky) {
        int hs;
        if (DGRAD) {
            const int a = hd + 1 - ky;
            if (a < 0 || (a % stride) != 0) continue;
            hs = a / stride;
        } else {
            hs = stride * hd + ky - 1;
        }
        if (hs < 0 || hs >= Hs) continue;
        for (int kx = 0; kx < 3; ++kx) {
            int ws;
            if (DGRAD) {
                const int b = wd + 1 - kx;
                if (b < 0 || (b % stride) != 0) continue;
                ws = b / stride;
            } else {
                ws = stride * wd + kx - 1;
            }
            if (ws < 0 || ws >= Ws) continue;
            const T *sp = src + ((n * Hs + hs) * Ws + ws) * Cs;
            const float *wt = wsm + (size_t)(ky * 3 + kx) * Cs * Cd + cd0;
            if (vec_ok) {
                for (int cs = 0; cs < Cs; cs += V) {
                    float sv[V];
                    load_f<T, V>(sp + cs, sv);
#pragma unroll
                    for (int u = 0; u < V; ++u) {
                        const float *wr = wt + (size_t)(cs + u) * Cd;
#pragma unroll
                        for (int j = 0; j < kCdt; ++j)
                            if (cd0 + j < Cd) acc[j] += (A)sv[u] * (A)wr[j];
                    }
                }
            } else {
                for (int cs = 0; cs < Cs; ++cs) {
                    const float sv = to_f(sp[cs]);
                    const float *wr = wt + (size_t)cs * Cd;
#pragma unroll
                    for (int j = 0; j < kCdt; ++j)
                        if (cd0 + j < Cd) acc[j] += (A)sv * (A)wr[j];
                }
            }
        }
    }
    // epilogue: shortcut gradient (dgrad of a residual block's first conv), ReLU (forward of a conv+ReLU layer)
    if (DGRAD && sc.mode != 0) {
        const T *dout = (const T *)sc.a, *out = (const T *)sc.b;
        if (sc.mode == 1) {
#pragma unroll
            for (int j = 0; j < kCdt; ++j)
                if (cd0 + j < Cd) {
                    const size_t q = (size_t)p * Cd + cd0 + j;
                    if (to_f(out[q]) > 0.f) acc[j] += (A)to_f(dout[q]);
                }
        } else if (sc.mode == 3) {
            // 1x1-projection shortcut with this convolution's stride: input pixel (s*h, s*w) fed output pixel (h, w)
            if ((hd % stride) == 0 && (wd % stride) == 0) {
                const T *ws = (const T *)sc.w;  // [Cout][Cin]
                const size_t q0 = ((n * Hs + hd / stride) * Ws + wd / stride) * (size_t)Cout;
                for (int co = 0; co < Cout; ++co) {
                    if (!(to_f(out[q0 + co]) > 0.f)) continue;
                    const A d = (A)to_f(dout[q0 + co]);
#pragma unroll
                    for (int j = 0; j < kCdt; ++j)
                        if (cd0 + j < Cd) acc[j] += d * (A)to_f(ws[(size_t)co * Cin + cd0 + j]);
                }
            }
        } else if ((hd % 2) == 0 && (wd % 2) == 0) {
            // block output is [B][Hs][Ws][Cout]; channel c < Cin of the input maps to the same channel
            const size_t q0 = ((n * Hs + hd / 2) * Ws + wd / 2) * (size_t)Cout;
#pragma unroll
            for (int j = 0; j < kCdt; ++j)
                if (cd0 + j < Cd && cd0 + j < Cout) {
                    if (to_f(out[q0 + cd0 + j]) > 0.f) acc[j] += (A)to_f(dout[q0 + cd0 + j]);
                }
        }
    }
#pragma unroll
    for (int j = 0; j < kCdt; ++j)
        if (cd0 + j < Cd) {
            A v = acc[j];
            if (relu && v < 0) v = 0;
            dst[(size_t)p * Cd + cd0 + j] = from_a<T>(v);
        }
}

template <typename T, int DGRAD>
static void conv_direct_launch(const void *src, const void *w, void *dst, int B, int Hs, int Ws, int Cs, int Hd,
                               int Wd, int Cd, int stride, int relu, Shortcut sc, Launch s) {
    const size_t smem = (size_t)9 * Cs * Cd * sizeof(float);
    const int groups = (Cd + kCdt - 1) / kCdt;
    const int pix_per_cta = kConvThreads / groups;
    const long npix = (long)B * Hd * Wd;
    launch_k(conv3x3_direct_kernel<T, DGRAD>, ceil_div(npix, pix_per_cta), kConvThreads, smem, s, (const T *)src, (const T *)w, (T *)dst, B, Hs, Ws, Cs, Hd, Wd, Cd, stride, relu, sc);
}

int conv_direct_init() {
    cudaError_t e = cudaSuccess;
    auto set = [&](const void *f) {
        cudaError_t r = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e == cudaSuccess) e = r;
    };
    set((const void *)conv3x3_direct_kernel<float, 0>);
    set((const void *)conv3x3_direct_kernel<float, 1>);
    set((const void *)conv3x3_direct_kernel<bf16, 0>);
    set((const void *)conv3x3_direct_kernel<bf16, 1>);
    return (int)e;
}

int launch_conv_fwd_direct(int prec, const void *x, const void *w, void *y, int B, int H, int W, int Cin, int Cout,
                           int stride, int relu, Launch s) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    Shortcut none = {};
    DISPATCH_PREC(prec, (conv_direct_launch<T, 0>(x, w, y, B, H, W, Cin, Ho, Wo, Cout, stride, relu, none, s)));
    return 1;
}

int launch_conv_dgrad_direct(int prec, const void *dy, const void *w, void *dx, int B, int H, int W, int Cin, int Cout,
                             int stride, Shortcut sc, Launch s) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    DISPATCH_PREC(prec, (conv_direct_launch<T, 1>(dy, w, dx, B, Ho, Wo, Cout, H, W, Cin, stride, 0, sc, s)));
    return 1;
}

// ------------------------------------------------------------------------------------------------------
// weight gradient: dw[co][ci][ky][kx] = sum_{n,ho,wo} dy[n,ho,wo,co] * x[n, s*ho+ky-1, s*wo+kx-1, ci]
// grid = (row chunks, 3 kernel rows).  Each CTA accumulates its chunk of output rows in registers and writes a
// partial [kx][ci][co] block to scratch; a second kernel folds the partials in a fixed order.
// ------------------------------------------------------------------------------------------------------
static constexpr int kWgThreads = 256;
static constexpr int kWgMaxCiPer = 16;

static int wgrad_chunks(int B, int Ho) {
    const long rows = (long)B * Ho;
    long chunks = rows < 96 ? rows : 96;
    return (int)chunks;
}

// fp32 elements; sized for the fp64 partials of the fp32 mode
size_t conv_wgrad_scratch_elems(int B, int H, int W, int Cin, int Cout, int stride) {
    const int Ho = (H - 1) / stride + 1;
    return (size_t)wgrad_chunks(B, Ho) * 9 * Cin * Cout * 2;
}

template <typename T>
__global__ void __launch_bounds__(kWgThreads)
conv3x3_wgrad_partial_kernel(const T *__restrict__ x, const T *__restrict__ dy,
                             typename AccOf<T>::type *__restrict__ part, int B, int H, int W, int Cin, int Ho, int Wo,
                             int Cout, int stride, int ci_per) {
    pdl_launch();
    pdl_wait();
    typedef typename AccOf<T>::type A;
    extern __shared__ float sm[];
    float *xs = sm;                         // [(W+2)][Cin] with a zero halo column on each side
    float *dys = sm + (size_t)(W + 2) * Cin;  // [Wo][Cout]
    const int ky = blockIdx.y;
    const int co = threadIdx.x % Cout, cig = threadIdx.x / Cout;
    const int ci0 = cig * ci_per;
    const bool active = (threadIdx.x < (kWgThreads / Cout) * Cout) && ci0 < Cin;
    A acc[3][kWgMaxCiPer];
#pragma unroll
    for (int a = 0; a < 3; ++a)
#pragma unroll
        for (int j = 0; j < kWgMaxCiPer; ++j) acc[a][j] = 0;
    const long rows = (long)B * Ho;
    const long r0 = rows * blockIdx.x / gridDim.x, r1 = rows * (blockIdx.x + 1) / gridDim.x;
    for (long r = r0; r < r1; ++r) {
        const int ho = (int)(r % Ho);
        const long n = r / Ho;
        const int hi = stride * ho + ky - 1;
        if (hi < 0 || hi >= H) continue;  // uniform across the CTA
        __syncthreads();
        const T *xrow = x + ((n * H + hi) * W) * (size_t)Cin;
        for (int i = threadIdx.x; i < (W + 2) * Cin; i += blockDim.x) {
            const int wcol = i / Cin - 1;
            xs[i] = (wcol >= 0 && wcol < W) ? to_f(xrow[(size_t)wcol * Cin + (i % Cin)]) : 0.f;
        }
        const T *dyrow = dy + (r * Wo) * (size_t)Cout;
        for (int i = threadIdx.x; i < Wo * Cout; i += blockDim.x) dys[i] = to_f(dyrow[i]);
        __syncthreads();
        if (!active) continue;
        for (int wo = 0; wo < Wo; ++wo) {
            const A d = (A)dys[wo * Cout + co];
            const float *xp = xs + (size_t)(stride * wo) * Cin + ci0;  // column (s*wo + kx - 1) + 1 halo
#pragma unroll
            for (int kx = 0; kx < 3; ++kx)
#pragma unroll
                for (int j = 0; j < kWgMaxCiPer; ++j)
                    if (j < ci_per && ci0 + j < Cin) acc[kx][j] += d * (A)xp[kx * Cin + j];
        }
    }
    if (!active) return;
    A *out = part + (size_t)blockIdx.x * 9 * Cin * Cout;
#pragma unroll
    for (int kx = 0; kx < 3; ++kx)
#pragma unroll
        for (int j = 0; j < kWgMaxCiPer; ++j)
            if (j < ci_per && ci0 + j < Cin)
                out[((size_t)(ky * 3 + kx) * Cin + ci0 + j) * Cout + co] = acc[kx][j];
}

template <typename A>
__global__ void conv3x3_wgrad_fold_kernel(const A *__restrict__ part, float *__restrict__ dw, int chunks, int Cin,
                                          int Cout) {
    pdl_launch();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;  // index into [tap][ci][co]
    const int total = 9 * Cin * Cout;
    if (i >= total) return;
    A t = 0;
    for (int c = 0; c < chunks; ++c) t += part[(size_t)c * total + i];
    const int co = i % Cout, ci = (i / Cout) % Cin, tap = i / (Cout * Cin);
    dw[((size_t)co * Cin + ci) * 9 + tap] = (float)t;
}

int launch_conv_wgrad_direct(int prec, const void *x, const void *dy, float *dw, float *scratch, int B, int H, int W,
                             int Cin, int Cout, int stride, Launch s) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    const int chunks = wgrad_chunks(B, Ho);
    const int cigs = kWgThreads / Cout;  // host guarantees Cout <= 256
    const int ci_per = (Cin + cigs - 1) / cigs;
    // ci_per <= kWgMaxCiPer is checked by the caller (Cin*Cout <= 4096)
    const size_t smem = ((size_t)(W + 2) * Cin + (size_t)Wo * Cout) * sizeof(float);
    dim3 grid(chunks, 3);
    DISPATCH_PREC(prec, {
        typedef typename AccOf<T>::type A;
        launch_k(conv3x3_wgrad_partial_kernel<T>, grid, kWgThreads, smem, s, (const T *)x, (const T *)dy, (A *)scratch, B, H, W,
                                                                     Cin, Ho, Wo, Cout, stride, ci_per);
        launch_k(conv3x3_wgrad_fold_kernel<A>, ceil_div(9 * Cin * Cout, 256), 256, 0, s, (const A *)scratch, dw, chunks, Cin,
                                                                                  Cout);
    });
    return 2;
}

// ------------------------------------------------------------------------------------------------------
// 1x1 convolution with a spatial stride (projection shortcut).  A few MFLOP per call: plain CUDA-core kernels.
// ------------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
conv1x1_fwd_kernel(const T *__restrict__ x, const T *__restrict__ w, T *__restrict__ y, long npix, int H, int W, int Cin,
                   int Ho, int Wo, int Cout, int stride) {
    pdl_launch();
    pdl_wait();
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;  // (output pixel, co)
    if (i >= npix * Cout) return;
    typedef typename AccOf<T>::type A;
    const int co = (int)(i % Cout);
    const long p = i / Cout;
    const int wo = (int)(p % Wo), ho = (int)((p / Wo) % Ho);
    const long n = p / ((long)Wo * Ho);
    const T *xp = x + ((n * H + (long)stride * ho) * W + (long)stride * wo) * Cin;
    const T *wp = w + (size_t)co * Cin;
    A acc = 0;
    for (int ci = 0; ci < Cin; ++ci) acc += (A)to_f(xp[ci]) * (A)to_f(wp[ci]);
    y[i] = from_a<T>(acc);
}

template <typename T>
__global__ void __launch_bounds__(256)
conv1x1_dgrad_add_kernel(const T *__restrict__ dout, const T *__restrict__ out, const T *__restrict__ w, T *__restrict__ dx,
                         long npix, int H, int W, int Cin, int Ho, int Wo, int Cout, int stride) {
    pdl_launch();
    pdl_wait();
    const long i = (long)blockIdx.x * blockDim.x + threadIdx.x;  // (output pixel, ci)
    if (i >= npix * Cin) return;
    typedef typename AccOf<T>::type A;
    const int ci = (int)(i % Cin);
    const long p = i / Cin;
    const int wo = (int)(p % Wo), ho = (int)((p / Wo) % Ho);
    const long n = p / ((long)Wo * Ho);
    T *dst = dx + ((n * H + (long)stride * ho) * W + (long)stride * wo) * Cin + ci;
    A acc = (A)to_f(*dst);
    for (int co = 0; co < Cout; ++co) {
        if (out != nullptr && !(to_f(out[p * Cout + co]) > 0.f)) continue;
        acc += (A)to_f(dout[p * Cout + co]) * (A)to_f(w[(size_t)co * Cin + ci]);
    }
    *dst = from_a<T>(acc);
}

static constexpr int k1x1Chunks = 64;
size_t conv1x1_wgrad_scratch_elems(int Cin, int Cout) { return (size_t)k1x1Chunks * Cin * Cout * 2; }  // fp64 partials in fp32 mode

// one CTA per chunk of output pixels; thread t owns the (co, ci) pairs t, t + 256, ...
template <typename T>
__global__ void __launch_bounds__(256)
conv1x1_wgrad_partial_kernel(const T *__restrict__ x, const T *__restrict__ dout, const T *__restrict__ out,
                             typename AccOf<T>::type *__restrict__ part, long npix, int H, int W, int Cin, int Ho, int Wo,
                             int Cout, int stride) {
    pdl_launch();
    pdl_wait();
    typedef typename AccOf<T>::type A;
    constexpr int kMaxPairs = 16;  // Cin * Cout <= 4096
    const int pairs = Cin * Cout;
    A acc[kMaxPairs];
#pragma unroll
    for (int j = 0; j < kMaxPairs; ++j) acc[j] = 0;
    const long p0 = npix * blockIdx.x / gridDim.x, p1 = npix * (blockIdx.x + 1) / gridDim.x;
    for (long p = p0; p < p1; ++p) {
        const int wo = (int)(p % Wo), ho = (int)((p / Wo) % Ho);
        const long n = p / ((long)Wo * Ho);
        const T *xp = x + ((n * H + (long)stride * ho) * W + (long)stride * wo) * Cin;
#pragma unroll
        for (int j = 0; j < kMaxPairs; ++j) {
            const int q = threadIdx.x + j * 256;
            if (q < pairs) {
                const int co = q / Cin, ci = q % Cin;
                float d = to_f(dout[p * Cout + co]);
                if (out != nullptr && !(to_f(out[p * Cout + co]) > 0.f)) d = 0.f;
                acc[j] += (A)d * (A)to_f(xp[ci]);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < kMaxPairs; ++j) {
        const int q = threadIdx.x + j * 256;
        if (q < pairs) part[(size_t)blockIdx.x * pairs + q] = acc[j];
    }
}

template <typename A>
__global__ void conv1x1_wgrad_fold_kernel(const A *__restrict__ part, float *__restrict__ dw, int chunks, int pairs) {
    pdl_launch();
    pdl_wait();
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q >= pairs) return;
    A t = 0;
    for (int c = 0; c < chunks; ++c) t += part[(size_t)c * pairs + q];
    dw[q] = (float)t;
}

int launch_conv1x1_fwd(int prec, const void *x, const void *w, void *y, int B, int H, int W, int Cin, int Cout, int stride,
                       Launch s) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    const long npix = (long)B * Ho * Wo;
    DISPATCH_PREC(prec, launch_k(conv1x1_fwd_kernel<T>, ceil_div(npix * Cout, 256), 256, 0, s, (const T *)x, (const T *)w, (T *)y,
                                 npix, H, W, Cin, Ho, Wo, Cout, stride));
    return 1;
}

int launch_conv1x1_dgrad_add(int prec, const void *dout, const void *out, const void *w, void *dx, int B, int H, int W,
                             int Cin, int Cout, int stride, Launch s) {
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    const long npix = (long)B * Ho * Wo;
    DISPATCH_PREC(prec, launch_k(conv1x1_dgrad_add_kernel<T>, ceil_div(npix * Cin, 256), 256, 0, s, (const T *)dout,
                                 (const T *)out, (const T *)w, (T *)dx, npix, H, W, Cin, Ho, Wo, Cout, stride));
    return 1;
}

int launch_conv1x1_wgrad(int prec, const void *x, const void *dout, const void *out, float *dw, float *scratch, int B,
                         int H, int W, int Cin, int Cout, int stride, Launch s) {
    if ((long)Cin * Cout > 4096) return -1;
    const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
    const long npix = (long)B * Ho * Wo;
    const int chunks = npix < k1x1Chunks ? (int)npix : k1x1Chunks;
    DISPATCH_PREC(prec, {
        typedef typename AccOf<T>::type A;
        launch_k(conv1x1_wgrad_partial_kernel<T>, chunks, 256, 0, s, (const T *)x, (const T *)dout, (const T *)out, (A *)scratch,
                 npix, H, W, Cin, Ho, Wo, Cout, stride);
        launch_k(conv1x1_wgrad_fold_kernel<A>, ceil_div(Cin * Cout, 256), 256, 0, s, (const A *)scratch, dw, chunks, Cin * Cout);
    });
    return 2;
}

}  // namespace ddg
