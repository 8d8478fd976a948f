// Internal launcher interface between the host engine and the kernels.  Every launcher only enqueues on the
// given stream and returns the number of kernel launches it issued.  `prec` is 0 (fp32 tensors) or 1 (bf16).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

namespace ddg {

enum { P_F32 = 0, P_BF16 = 1 };

static inline size_t elem_size(int prec) { return prec == P_BF16 ? 2 : 4; }

// Where and how a launcher enqueues its kernels.  A bare stream converts to the single-kernel default: the
// programmatic launch attribute on every launch, the GPU not shared with other module streams, and the library's
// process-wide error word.  The engine builds one per module from its configuration.
//   pdl    programmatic dependent launch: 0 = never, 1 = every kernel, 2 = only the kernels that ask for it (the
//          forward / input-gradient convolution), which is what pays while several module streams share the GPU
//   shared several module streams share the GPU: launchers size grids so that SMs are left over for the other modules'
//          kernels where that costs the kernel itself nothing
//   err    device word that a bounded wait which ran out reports into (nullptr: the process-wide word)
struct Launch {
    cudaStream_t s;
    int pdl;
    bool shared;
    int *err;
    Launch(cudaStream_t st = nullptr, int pdl_ = 1, bool shared_ = false, int *err_ = nullptr)
        : s(st), pdl(pdl_), shared(shared_), err(err_) {}
    operator cudaStream_t() const { return s; }
    Launch on(cudaStream_t other) const { return Launch(other, pdl, shared, err); }  // same policy, another stream
};

// Shortcut input of a residual add (forward) or its gradient (backward).
//   mode 0: none.  mode 1: identity (same shape as the tensor it is added to).
//   mode 2: parameter-free down-sampling shortcut: spatial stride 2, channels >= c_small are zero.
//   mode 3 (backward, CUDA-core input gradient only): 1x1-projection shortcut W_s [Cout][c_small] with the convolution's
//           stride: dx[n][s*h][s*w][ci] += sum_co a[n][h][w][co] * [b > 0] * w[co][ci].
struct Shortcut {
    int mode;
    const void *a;   // forward: block input x.          backward: error gradient of the block output
    const void *b;   // forward: unused.                 backward: block output (for the ReLU mask)
    int c_small;     // channels of the narrower tensor (block input)
    int h_big, w_big;  // spatial size of the block input (the larger map)
    const void *w;   // mode 3: the projection filter
};

// ---- layout / small layers --------------------------------------------------------------------------
// Cpad >= C: channels per pixel of the output; the extra channels are written as zero.
int launch_shim(int prec, const float *x_nchw, void *out_nhwc, int B, int C, int H, int W, int Cpad, Launch s);
int launch_relu_fwd(int prec, const void *x, void *y, size_t n, Launch s);
int launch_relu_bwd(int prec, const void *y, const void *dy, void *dx, size_t n, Launch s);
int launch_avgpool_fwd(int prec, const void *x, void *y, int B, int HW, int C, Launch s);
int launch_avgpool_bwd(int prec, const void *dy, void *dx, int B, int HW, int C, Launch s);

// FC: x [B][in] (prec), W [out][in] (prec), bias [out] (prec, nullable).  out_f32: y (and dy) are fp32.
int launch_fc_fwd(int prec, const void *x, const void *W, const void *bias, void *y, int B, int in, int out,
                  int relu, int out_f32, Launch s);
// dx nullable.  y is the forward output (needed when relu).  dW/db fp32.
int launch_fc_bwd(int prec, const void *x, const void *W, const void *y, const void *dy, void *dx, float *dW,
                  float *db, int B, int in, int out, int relu, int out_f32, Launch s);

// loss = mean CE, dlogits = (softmax - onehot)/B; logits/dlogits fp32 [B][C].
int launch_softmax_ce(int prec, const float *logits, const int *labels, float *loss, float *dlogits, int B, int C,
                      Launch s);

// ---- batch norm -------------------------------------------------------------------------------------
size_t bn_scratch_elems(int C);
int launch_bn_stats(int prec, const void *x, float *mean, float *invstd, float *scratch, long npix, int C,
                    Launch s);
// Per-CTA partial sums left by the epilogue of the convolution that produced a batch norm's input (or incoming gradient):
// part[n][2C] fp32, rows in CTA order.  The element-wise pass that consumes the sums folds them itself, every CTA the
// same rows in the same fixed order (so all CTAs hold identical totals and nothing has to be waited for or
// broadcast), and its first CTA also stores the folded pair (mean, invstd) or (dbeta, dgamma) where the separate
// reduction would have put it.  part == nullptr: the sums are already in place.
struct BnPartials {
    const float *part = nullptr;
    int n = 0;
};
// true when launch_bn_apply / launch_bn_bwd_apply take partials for this case (the bf16 fast kernels)
bool bn_apply_takes_partials(int prec, int C, int shortcut_mode);
// y = [relu](gamma*(x-mean)*invstd + beta + shortcut).  y is [B][H][W][C].  With partials (sum x, sum x^2) the kernel
// computes mean / invstd itself and WRITES them to `mean` / `invstd`.
int launch_bn_apply(int prec, const void *x, const void *gamma, const void *beta, float *mean, float *invstd,
                    Shortcut sc, void *y, int B, int H, int W, int C, int relu, Launch s, BnPartials bp = BnPartials());
// sums[0..C) = sum dz, sums[C..2C) = sum dz*xhat with dz = dout*[out>0] (relu) ; also written to dbeta/dgamma.
int launch_bn_bwd_reduce(int prec, const void *dout, const void *out, const void *x, const float *mean,
                         const float *invstd, float *dgamma, float *dbeta, float *scratch, long npix, int C, int relu,
                         Launch s);
// With partials (sum dz, sum dz*xhat) the kernel folds them itself and WRITES dbeta / dgamma.
int launch_bn_bwd_apply(int prec, const void *dout, const void *out, const void *x, const void *gamma,
                        const float *mean, const float *invstd, float *dgamma, float *dbeta, void *dx,
                        long npix, int C, int relu, Launch s, BnPartials bp = BnPartials());

// ---- 3x3 convolution, CUDA-core kernels (any shape; used for fp32 and for shapes the tensor-core path skips) --
int launch_conv_fwd_direct(int prec, const void *x, const void *w, void *y, int B, int H, int W, int Cin, int Cout,
                           int stride, int relu, Launch s);
int launch_conv_dgrad_direct(int prec, const void *dy, const void *w, void *dx, int B, int H, int W, int Cin,
                             int Cout, int stride, Shortcut sc, Launch s);
size_t conv_wgrad_scratch_elems(int B, int H, int W, int Cin, int Cout, int stride);
int launch_conv_wgrad_direct(int prec, const void *x, const void *dy, float *dw, float *scratch, int B, int H, int W,
                             int Cin, int Cout, int stride, Launch s);

// ---- 1x1 convolution with a spatial stride, no bias (projection shortcut of a shape-changing block), CUDA cores ----
// x [B][H][W][Cin], w [Cout][Cin], y [B][Ho][Wo][Cout], Ho = (H-1)/stride+1.
int launch_conv1x1_fwd(int prec, const void *x, const void *w, void *y, int B, int H, int W, int Cin, int Cout, int stride,
                       Launch s);
// dx[n][s*h][s*w][ci] += sum_co dz[n][h][w][co] * w[co][ci], dz = dout * [out > 0] (out nullable: no mask); dx is read,
// added to and stored in its element type.
int launch_conv1x1_dgrad_add(int prec, const void *dout, const void *out, const void *w, void *dx, int B, int H, int W,
                             int Cin, int Cout, int stride, Launch s);
// dw[co][ci] = sum over output pixels of dz[p][co] * x[s*p][ci]; per-chunk partials in scratch, folded in a fixed order.
size_t conv1x1_wgrad_scratch_elems(int Cin, int Cout);
int launch_conv1x1_wgrad(int prec, const void *x, const void *dout, const void *out, float *dw, float *scratch, int B,
                         int H, int W, int Cin, int Cout, int stride, Launch s);

// ---- optimiser --------------------------------------------------------------------------------------
// mode 0: SGD momentum/decay step.  mode 1: Adam step (c1, c2 = bias corrections).  mode 2: no step, only
// refresh the weight version.  w/v/m2 fp32 master state, g fp32, wv = version slot in `prec`.
// dyn (device, nullable): three doubles {lr, c1c, c2c} that replace the by-value fields of the same names.  The engine
// keeps them in device memory so that a recorded update (CUDA graph) follows the step size sequence and Adam's
// iteration-dependent bias corrections without being re-recorded; launch_set_opt_scalars writes them in stream order.
struct UpdateArgs {
    int mode;
    float lr, mu, wd, b1, b2, eps;
    double c1c, c2c;  // Adam bias corrections 1-beta1^(t+1), 1-beta2^(t+1)
    const double *dyn;
};
int launch_update(int prec, float *w, float *v, float *m2, const float *g, void *wv, size_t n, UpdateArgs a,
                  Launch s);
int launch_set_opt_scalars(double *dyn, double lr, double c1c, double c2c, Launch s);

// Ring-slot stamps (debug aid of the engine).  One single-thread kernel per piece of an iteration: compares up to three
// stamps with *expect (a device-resident counter) and raises *err with `code + i` (first mismatch wins, never a trap),
// stores the counter's value into up to two stamps, then adds `advance` to the counter.
struct StampOp {
    long long *counter;          // device counter of the piece (sample or iteration index)
    const long long *check[3];   // stamps that must equal *counter (nullptr = unused)
    long long *set[2];           // stamps that receive *counter + set_add (nullptr = unused)
    int set_add;
    int advance;
    int code;
    int *err;
};
int launch_stamp(StampOp op, Launch s);
int launch_add_to_counter(long long *counter, long long delta, Launch s);
int launch_cast(int prec, const float *src, void *dst, size_t n, Launch s);
int launch_fill_normal(float *dst, size_t n, float stddev, unsigned long long seed, unsigned long long stream_id,
                       Launch s);
int launch_fill_const(float *dst, size_t n, float v, Launch s);

}  // namespace ddg
