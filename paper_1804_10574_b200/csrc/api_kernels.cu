// Single-kernel C-ABI entry points (per-kernel parity tests and roofline measurements).
#include "../../include/ddg.h"
#include "common.cuh"
#include "conv_tc.h"
#include <stdio.h>

#include "kernels.h"

using namespace ddg;

namespace ddg { void set_global_error(const char *msg); }

namespace {
bool bad_prec(int p) { return p != DDG_FP32 && p != DDG_BF16; }
ddg_status init_once() {
    static int rc = -1;
    if (rc < 0) { rc = conv_direct_init(); if (rc == 0) rc = conv_tc_init(); }
    return rc == 0 ? DDG_OK : DDG_ERR_CUDA;
}
// An error left pending by an earlier, unrelated CUDA call would otherwise be blamed on (and cleared by) this entry
// point: refuse to launch on top of it and name it.
bool pending_error() {
    const cudaError_t e = cudaPeekAtLastError();
    if (e == cudaSuccess) return false;
    static thread_local char msg[256];
    snprintf(msg, sizeof(msg), "an earlier CUDA error is still pending: %s", cudaGetErrorString(e));
    set_global_error(msg);
    return true;
}
// r: what the launcher returned (negative: it refused the launch)
ddg_status done(int r = 0) {
    if (r < 0) {
        set_global_error("the kernel launcher refused the launch (tensor map or shared-memory plan)");
        return DDG_ERR_CUDA;
    }
    const cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) return DDG_OK;
    set_global_error(cudaGetErrorString(e));
    return DDG_ERR_CUDA;
}
bool conv_shape_ok(int B, int H, int W, int Cin, int Cout, int stride) {
    return B >= 1 && H >= 1 && W >= 1 && Cin >= 1 && Cout >= 1 && (stride == 1 || stride == 2) && Cin <= 256 &&
           Cout <= 256 && (size_t)Cin * Cout <= 4096;
}
}  // namespace

extern "C" {

int ddg_tensor_core_path(int B, int H, int W, int Cin, int Cout, int stride) {
    if (init_once() != DDG_OK) return 0;
    if (conv_tc_s2_supported(B, H, W, Cin, Cout, stride)) return 3;
    return (conv_tc_supported(B, H, W, Cin, Cout, stride) ? 1 : 0) | (wgrad_tc_supported(B, H, W, Cin, Cout, stride) ? 2 : 0);
}

ddg_status ddg_conv3x3_fwd(int precision, const void *x, const void *w, void *y, int B, int H, int W, int Cin,
                           int Cout, int stride, void *stream) {
    if (bad_prec(precision) || !x || !w || !y) return DDG_ERR_INVALID_ARG;
    if (!conv_shape_ok(B, H, W, Cin, Cout, stride)) return DDG_ERR_UNSUPPORTED;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    int r;
    if (precision == DDG_BF16 && conv_tc_supported(B, H, W, Cin, Cout, stride))
        r = launch_conv_tc(0, x, w, nullptr, y, B, H, W, Cin, Shortcut{}, s);
    else if (precision == DDG_BF16 && conv_tc_s2_supported(B, H, W, Cin, Cout, stride))
        r = launch_conv_tc_s2(0, x, w, nullptr, y, B, H, W, Cin, Shortcut{}, s);
    else
        r = launch_conv_fwd_direct(precision, x, w, y, B, H, W, Cin, Cout, stride, 0, s);
    return done(r);
}

ddg_status ddg_conv3x3_dgrad(int precision, const void *dy, const void *w, void *dx, int B, int H, int W, int Cin,
                             int Cout, int stride, void *stream) {
    if (bad_prec(precision) || !dy || !w || !dx) return DDG_ERR_INVALID_ARG;
    if (!conv_shape_ok(B, H, W, Cin, Cout, stride)) return DDG_ERR_UNSUPPORTED;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    int r;
    if (precision == DDG_BF16 && conv_tc_supported(B, H, W, Cin, Cout, stride))
        r = launch_conv_tc(1, dy, w, nullptr, dx, B, H, W, Cin, Shortcut{}, s);
    else if (precision == DDG_BF16 && conv_tc_s2_supported(B, H, W, Cin, Cout, stride))
        r = launch_conv_tc_s2(1, dy, w, nullptr, dx, B, H, W, Cin, Shortcut{}, s);
    else
        r = launch_conv_dgrad_direct(precision, dy, w, dx, B, H, W, Cin, Cout, stride, Shortcut{}, s);
    return done(r);
}

size_t ddg_conv3x3_packed_bytes(int B, int H, int W, int C) {
    if (init_once() != DDG_OK || !conv_tc_supported(B, H, W, C, C, 1)) return 0;
    return tc_packed_bytes(C);
}

ddg_status ddg_conv3x3_pack(const void *w, void *packed, int C, void *stream) {
    if (!w || !packed) return DDG_ERR_INVALID_ARG;
    if (C != 16 && C != 32 && C != 64) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    return done(launch_pack_one(w, packed, C, (cudaStream_t)stream));
}

ddg_status ddg_conv3x3_packed(int dgrad, const void *src, const void *w, const void *packed, void *dst, int B, int H,
                              int W, int C, void *stream) {
    if (!src || !w || !packed || !dst) return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_supported(B, H, W, C, C, 1)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    return done(launch_conv_tc(dgrad ? 1 : 0, src, w, packed, dst, B, H, W, C, Shortcut{}, (cudaStream_t)stream));
}

size_t ddg_conv3x3_fused_scratch_elems(int B, int H, int W, int C) {
    if (init_once() != DDG_OK || !conv_tc_supported(B, H, W, C, C, 1)) return 0;
    return 32 + (size_t)conv_tc_grid(B, H, W) * 2 * C;  // ticket counter, then one partial [2C] per CTA
}

ddg_status ddg_conv3x3_fwd_stats(const void *x, const void *w, const void *packed, void *y, float *mean, float *invstd,
                                 float *scratch, int B, int H, int W, int C, void *stream) {
    if (!x || !w || !y || !mean || !invstd || !scratch) return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_supported(B, H, W, C, C, 1)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(scratch, 0, 128, s) != cudaSuccess) return DDG_ERR_CUDA;  // the CTA ticket counter
    BnFuse bf;
    bf.counter = reinterpret_cast<unsigned *>(scratch); bf.part = scratch + 32; bf.o0 = mean; bf.o1 = invstd;
    return done(launch_conv_tc(0, x, w, packed, y, B, H, W, C, Shortcut{}, s, bf));
}

ddg_status ddg_conv3x3_fwd_stats_prepared(const void *x, const void *w, const void *packed, void *y, float *mean,
                                          float *invstd, float *scratch, int B, int H, int W, int C, void *stream) {
    if (!x || !w || !y || !mean || !invstd || !scratch) return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_supported(B, H, W, C, C, 1)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    BnFuse bf;
    bf.counter = reinterpret_cast<unsigned *>(scratch); bf.part = scratch + 32; bf.o0 = mean; bf.o1 = invstd;
    return done(launch_conv_tc(0, x, w, packed, y, B, H, W, C, Shortcut{}, (cudaStream_t)stream, bf));
}

ddg_status ddg_conv3x3_fwd_stats_shared(const void *x, const void *w, const void *packed, void *y, float *mean,
                                        float *invstd, float *scratch, int B, int H, int W, int C, void *stream) {
    if (!x || !w || !y || !mean || !invstd || !scratch) return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_supported(B, H, W, C, C, 1)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    BnFuse bf;
    bf.counter = reinterpret_cast<unsigned *>(scratch); bf.part = scratch + 32; bf.o0 = mean; bf.o1 = invstd;
    const Launch shared((cudaStream_t)stream, 2, true, nullptr);  // what the engine passes for K > 1
    return done(launch_conv_tc(0, x, w, packed, y, B, H, W, C, Shortcut{}, shared, bf));
}

ddg_status ddg_conv3x3_fwd_partials(const void *x, const void *w, const void *packed, void *y, float *part,
                                    int *n_part_host, int B, int H, int W, int C, void *stream) {
    if (!x || !w || !y || !part || !n_part_host) return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_supported(B, H, W, C, C, 1)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    BnFuse bf;
    bf.part = part; bf.n_part_out = n_part_host;
    return done(launch_conv_tc(0, x, w, packed, y, B, H, W, C, Shortcut{}, (cudaStream_t)stream, bf));
}

ddg_status ddg_bn_fwd_partials(const void *y, const void *gamma, const void *beta, const void *res, void *out,
                               const float *part, int n_part, float *mean, float *invstd, int B, int HW, int C, int relu,
                               void *stream) {
    if (!y || !gamma || !beta || !out || !part || n_part < 1 || !mean || !invstd) return DDG_ERR_INVALID_ARG;
    if (B < 1 || HW < 1 || !bn_apply_takes_partials(DDG_BF16, C, res ? 1 : 0)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    Shortcut sc{};
    if (res) { sc.mode = 1; sc.a = res; }
    BnPartials bp;
    bp.part = part; bp.n = n_part;
    return done(launch_bn_apply(DDG_BF16, y, gamma, beta, mean, invstd, sc, out, B, HW, 1, C, relu, (cudaStream_t)stream, bp));
}

ddg_status ddg_conv3x3_dgrad_partials(const void *dy, const void *w, const void *packed, void *dx, const void *res_dout,
                                      const void *res_out, const void *bn_mask, const void *bn_x, const float *bn_mean,
                                      const float *bn_invstd, float *part, int *n_part_host, int B, int H, int W, int C,
                                      void *stream) {
    if (!dy || !w || !dx || !bn_mask || !bn_x || !bn_mean || !bn_invstd || !part || !n_part_host) return DDG_ERR_INVALID_ARG;
    if ((res_dout == nullptr) != (res_out == nullptr)) return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_supported(B, H, W, C, C, 1)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    Shortcut sc{};
    if (res_dout) { sc.mode = 1; sc.a = res_dout; sc.b = res_out; }
    BnFuse bf;
    bf.part = part; bf.n_part_out = n_part_host;
    bf.mask = bn_mask; bf.x = bn_x; bf.mean = bn_mean; bf.invstd = bn_invstd;
    return done(launch_conv_tc(1, dy, w, packed, dx, B, H, W, C, sc, (cudaStream_t)stream, bf));
}

ddg_status ddg_bn_bwd_partials(const void *dout, const void *out, const void *x, const void *gamma, const float *mean,
                               const float *invstd, void *dx, float *dgamma, float *dbeta, const float *part, int n_part,
                               int B, int HW, int C, int relu, void *stream) {
    if (!dout || !x || !gamma || !mean || !invstd || !dx || !dgamma || !dbeta || !part || n_part < 1 || (relu && !out))
        return DDG_ERR_INVALID_ARG;
    if (B < 1 || HW < 1 || !bn_apply_takes_partials(DDG_BF16, C, 0)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    BnPartials bp;
    bp.part = part; bp.n = n_part;
    return done(launch_bn_bwd_apply(DDG_BF16, dout, out, x, gamma, mean, invstd, dgamma, dbeta, dx, (long)B * HW, C, relu,
                                    (cudaStream_t)stream, bp));
}

ddg_status ddg_conv3x3_bnrelu_fwd_stats(const void *x, const void *res, const void *gamma, const void *beta,
                                        const float *mean_in, const float *invstd_in, void *a_out, const void *w,
                                        const void *packed, void *y,
                                        float *mean, float *invstd, float *scratch, int B, int H, int W, int C,
                                        void *stream) {
    if (!x || !gamma || !beta || !mean_in || !invstd_in || !a_out || !w || !y || !mean || !invstd || !scratch)
        return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_xform_supported(B, H, W, C, false)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(scratch, 0, 128, s) != cudaSuccess) return DDG_ERR_CUDA;
    BnFuse bf;
    bf.counter = reinterpret_cast<unsigned *>(scratch); bf.part = scratch + 32; bf.o0 = mean; bf.o1 = invstd;
    InXform xf;
    xf.gamma = gamma; xf.beta = beta; xf.mean = mean_in; xf.invstd = invstd_in; xf.a_out = a_out; xf.res = res;
    return done(launch_conv_tc(0, x, w, packed, y, B, H, W, C, Shortcut{}, s, bf, xf));
}

namespace {
ddg_status dgrad_fused(const void *dy, const void *w, const void *packed, void *dx, const void *res_dout,
                       const void *res_out, const void *bn_mask, const void *bn_x, const float *bn_mean,
                       const float *bn_invstd, float *dbeta, float *dgamma, float *scratch, int B, int H, int W, int C,
                       void *stream, bool shared);
}
ddg_status ddg_conv3x3_dgrad_fused(const void *dy, const void *w, const void *packed, void *dx, const void *res_dout,
                                   const void *res_out, const void *bn_mask, const void *bn_x, const float *bn_mean,
                                   const float *bn_invstd, float *dbeta, float *dgamma, float *scratch, int B, int H,
                                   int W, int C, void *stream) {
    return dgrad_fused(dy, w, packed, dx, res_dout, res_out, bn_mask, bn_x, bn_mean, bn_invstd, dbeta, dgamma, scratch, B, H,
                       W, C, stream, false);
}
ddg_status ddg_conv3x3_dgrad_fused_shared(const void *dy, const void *w, const void *packed, void *dx,
                                          const void *res_dout, const void *res_out, const void *bn_mask, const void *bn_x,
                                          const float *bn_mean, const float *bn_invstd, float *dbeta, float *dgamma,
                                          float *scratch, int B, int H, int W, int C, void *stream) {
    return dgrad_fused(dy, w, packed, dx, res_dout, res_out, bn_mask, bn_x, bn_mean, bn_invstd, dbeta, dgamma, scratch, B, H,
                       W, C, stream, true);
}
}  // extern "C"
namespace {
ddg_status dgrad_fused(const void *dy, const void *w, const void *packed, void *dx, const void *res_dout,
                       const void *res_out, const void *bn_mask, const void *bn_x, const float *bn_mean,
                       const float *bn_invstd, float *dbeta, float *dgamma, float *scratch, int B, int H, int W, int C,
                       void *stream, bool shared) {
    if (!dy || !w || !dx || !scratch) return DDG_ERR_INVALID_ARG;
    if ((res_dout == nullptr) != (res_out == nullptr)) return DDG_ERR_INVALID_ARG;
    const bool sums = bn_mask || bn_x || bn_mean || bn_invstd || dbeta || dgamma;
    if (sums && !(bn_mask && bn_x && bn_mean && bn_invstd && dbeta && dgamma)) return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_supported(B, H, W, C, C, 1)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(scratch, 0, 128, s) != cudaSuccess) return DDG_ERR_CUDA;
    Shortcut sc{};
    if (res_dout) { sc.mode = 1; sc.a = res_dout; sc.b = res_out; }
    BnFuse bf;
    if (sums) {
        bf.counter = reinterpret_cast<unsigned *>(scratch); bf.part = scratch + 32; bf.o0 = dbeta; bf.o1 = dgamma;
        bf.mask = bn_mask; bf.x = bn_x; bf.mean = bn_mean; bf.invstd = bn_invstd;
    }
    // shared: the launch plan and launch attribute policy the engine uses while K > 1 module streams share the GPU
    return done(launch_conv_tc(1, dy, w, packed, dx, B, H, W, C, sc, shared ? Launch(s, 2, true, nullptr) : Launch(s), bf));
}
}  // namespace
extern "C" {

ddg_status ddg_conv3x3_s2_dgrad_shortcut(const void *dy, const void *w, void *dx, const void *res_dout,
                                         const void *res_out, int B, int H, int W, int Cin, void *stream) {
    if (!dy || !w || !dx || (res_dout == nullptr) != (res_out == nullptr)) return DDG_ERR_INVALID_ARG;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (!conv_tc_s2_supported(B, H, W, Cin, 2 * Cin, 2)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    Shortcut sc{};
    if (res_dout) { sc.mode = 2; sc.a = res_dout; sc.b = res_out; sc.c_small = Cin; sc.h_big = H; sc.w_big = W; }
    return done(launch_conv_tc_s2(1, dy, w, nullptr, dx, B, H, W, Cin, sc, (cudaStream_t)stream));
}

ddg_status ddg_conv1x1_fwd(int precision, const void *x, const void *w, void *y, int B, int H, int W, int Cin, int Cout,
                           int stride, void *stream) {
    if (bad_prec(precision) || !x || !w || !y) return DDG_ERR_INVALID_ARG;
    if (!conv_shape_ok(B, H, W, Cin, Cout, stride)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    return done(launch_conv1x1_fwd(precision, x, w, y, B, H, W, Cin, Cout, stride, (cudaStream_t)stream));
}

ddg_status ddg_conv1x1_dgrad_add(int precision, const void *dout, const void *out, const void *w, void *dx, int B, int H,
                                 int W, int Cin, int Cout, int stride, void *stream) {
    if (bad_prec(precision) || !dout || !w || !dx) return DDG_ERR_INVALID_ARG;
    if (!conv_shape_ok(B, H, W, Cin, Cout, stride)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    return done(launch_conv1x1_dgrad_add(precision, dout, out, w, dx, B, H, W, Cin, Cout, stride, (cudaStream_t)stream));
}

size_t ddg_conv1x1_wgrad_scratch_elems(int Cin, int Cout) {
    return (Cin >= 1 && Cout >= 1 && (size_t)Cin * Cout <= 4096) ? conv1x1_wgrad_scratch_elems(Cin, Cout) : 0;
}

ddg_status ddg_conv1x1_wgrad(int precision, const void *x, const void *dout, const void *out, float *dw, float *scratch,
                             int B, int H, int W, int Cin, int Cout, int stride, void *stream) {
    if (bad_prec(precision) || !x || !dout || !dw || !scratch) return DDG_ERR_INVALID_ARG;
    if (!conv_shape_ok(B, H, W, Cin, Cout, stride)) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    return done(launch_conv1x1_wgrad(precision, x, dout, out, dw, scratch, B, H, W, Cin, Cout, stride, (cudaStream_t)stream));
}

size_t ddg_conv3x3_wgrad_scratch_elems(int B, int H, int W, int Cin, int Cout, int stride) {
    if (!conv_shape_ok(B, H, W, Cin, Cout, stride)) return 0;
    size_t a = conv_wgrad_scratch_elems(B, H, W, Cin, Cout, stride), b = wgrad_tc_scratch_elems();
    return a > b ? a : b;
}

ddg_status ddg_conv3x3_wgrad(int precision, const void *x, const void *dy, float *dw, float *scratch, int B, int H,
                             int W, int Cin, int Cout, int stride, void *stream) {
    if (bad_prec(precision) || !x || !dy || !dw || !scratch) return DDG_ERR_INVALID_ARG;
    if (!conv_shape_ok(B, H, W, Cin, Cout, stride)) return DDG_ERR_UNSUPPORTED;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    int r;
    if (precision == DDG_BF16 && wgrad_tc_supported(B, H, W, Cin, Cout, stride))
        r = launch_wgrad_tc(x, dy, dw, scratch, B, H, W, Cin, Cin, s);
    else if (precision == DDG_BF16 && conv_tc_s2_supported(B, H, W, Cin, Cout, stride))
        r = launch_wgrad_tc_s2(x, dy, dw, scratch, B, H, W, Cin, s);
    else
        r = launch_conv_wgrad_direct(precision, x, dy, dw, scratch, B, H, W, Cin, Cout, stride, s);
    return done(r);
}

int ddg_fc_tensor_core_path(int B, int in, int out) {
    if (init_once() != DDG_OK) return 0;
    return fc_tc_shape_supported(B, in, out) ? 1 : 0;
}

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

ddg_status ddg_fc_fwd(int precision, const void *x, const void *W, const void *bias, void *y, int B, int in, int out,
                      int relu, int out_f32, void *stream) {
    if (bad_prec(precision) || !x || !W || !y) return DDG_ERR_INVALID_ARG;
    if (B < 1 || in < 1 || out < 1) return DDG_ERR_UNSUPPORTED;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (precision == DDG_BF16 && fc_tc_supported(x, W, B, in, out))
        return done(launch_fc_fwd_tc(x, W, bias, y, B, in, out, relu, out_f32, s));
    return done(launch_fc_fwd(precision, x, W, bias, y, B, in, out, relu, out_f32, s));
}

ddg_status ddg_fc_bwd(int precision, const void *x, const void *W, const void *y, const void *dy, void *dx, float *dW,
                      float *db, int B, int in, int out, int relu, int out_f32, void *stream) {
    if (bad_prec(precision) || !x || !W || !dy || !dW || (relu && !y)) return DDG_ERR_INVALID_ARG;
    if (B < 1 || in < 1 || out < 1) return DDG_ERR_UNSUPPORTED;
    if (init_once() != DDG_OK) return DDG_ERR_CUDA;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (precision == DDG_BF16 && fc_tc_supported(x, W, B, in, out) && aligned16(dW) && aligned16(dx))
        return done(launch_fc_bwd_tc(x, W, y, dy, dx, dW, db, B, in, out, relu, out_f32, s));
    return done(launch_fc_bwd(precision, x, W, y, dy, dx, dW, db, B, in, out, relu, out_f32, s));
}

size_t ddg_bn_scratch_elems(int C) { return C >= 1 && C <= 128 ? bn_scratch_elems(C) : 0; }

ddg_status ddg_bn_fwd(int precision, const void *x, const void *gamma, const void *beta, const void *res, void *y,
                      float *mean, float *invstd, float *scratch, int B, int HW, int C, int relu, void *stream) {
    if (bad_prec(precision) || !x || !gamma || !beta || !y || !mean || !invstd || !scratch) return DDG_ERR_INVALID_ARG;
    if (B < 1 || HW < 1 || C < 1 || C > 128) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(scratch, 0, 128, s) != cudaSuccess) return DDG_ERR_CUDA;  // the CTA ticket counter
    launch_bn_stats(precision, x, mean, invstd, scratch, (long)B * HW, C, s);
    Shortcut sc{};
    if (res) { sc.mode = 1; sc.a = res; }
    launch_bn_apply(precision, x, gamma, beta, mean, invstd, sc, y, B, HW, 1, C, relu, s);
    return done();
}

ddg_status ddg_bn_bwd(int precision, const void *dout, const void *out, const void *x, const void *gamma,
                      const float *mean, const float *invstd, void *dx, float *dgamma, float *dbeta, float *scratch,
                      int B, int HW, int C, int relu, void *stream) {
    if (bad_prec(precision) || !dout || !x || !gamma || !mean || !invstd || !dx || !dgamma || !dbeta || !scratch ||
        (relu && !out))
        return DDG_ERR_INVALID_ARG;
    if (B < 1 || HW < 1 || C < 1 || C > 128) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(scratch, 0, 128, s) != cudaSuccess) return DDG_ERR_CUDA;
    launch_bn_bwd_reduce(precision, dout, out, x, mean, invstd, dgamma, dbeta, scratch, (long)B * HW, C, relu, s);
    launch_bn_bwd_apply(precision, dout, out, x, gamma, mean, invstd, dgamma, dbeta, dx, (long)B * HW, C, relu, s);
    return done();
}

ddg_status ddg_bn_bwd_reduce(int precision, const void *dout, const void *out, const void *x, const float *mean,
                             const float *invstd, float *dgamma, float *dbeta, float *scratch, int B, int HW, int C,
                             int relu, void *stream) {
    if (bad_prec(precision) || !dout || !x || !mean || !invstd || !dgamma || !dbeta || !scratch || (relu && !out))
        return DDG_ERR_INVALID_ARG;
    if (B < 1 || HW < 1 || C < 1 || C > 128) return DDG_ERR_UNSUPPORTED;
    if (pending_error()) return DDG_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(scratch, 0, 128, s) != cudaSuccess) return DDG_ERR_CUDA;
    launch_bn_bwd_reduce(precision, dout, out, x, mean, invstd, dgamma, dbeta, scratch, (long)B * HW, C, relu, s);
    return done();
}

ddg_status ddg_sgd_update(int precision, float *w, float *v, const float *g, void *w_version, size_t n, float lr,
                          float momentum, float weight_decay, void *stream) {
    if (bad_prec(precision) || !w || !v || !g || !w_version) return DDG_ERR_INVALID_ARG;
    if (pending_error()) return DDG_ERR_CUDA;
    UpdateArgs a{};
    a.mode = 0; a.lr = lr; a.mu = momentum; a.wd = weight_decay;
    launch_update(precision, w, v, nullptr, g, w_version, n, a, (cudaStream_t)stream);
    return done();
}

}  // extern "C"
