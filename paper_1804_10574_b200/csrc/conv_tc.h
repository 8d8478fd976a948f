// Tensor-core (tcgen05 / TMEM / TMA) 3x3 convolution path for bf16 NHWC tensors on sm_100a.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>

#include "kernels.h"

namespace ddg {

// Shapes the tensor-core kernels take: stride 1, Cin == Cout in {16, 32, 64}, 128-pixel tiles that cover whole
// image rows (W in {8, 16, 32}, and B*H*W a multiple of 128).
bool conv_tc_supported(int B, int H, int W, int Cin, int Cout, int stride);
// dir 0: dst = conv3x3(src, w) (forward).  dir 1: dst = input gradient of conv3x3 given src = dy; with
// sc.mode == 1 the identity-shortcut gradient sc.a * [sc.b > 0] is added before the store.
// w: filter in canonical [Cout][Cin][3][3] order.  w_packed (nullable): the pre-arranged filter images written by
// launch_pack_filters for this convolution (tc_packed_bytes(C) bytes: forward image, then input-gradient image); when
// given, the kernel fetches its filter with one bulk copy instead of re-arranging the canonical one itself.
// bf.part != nullptr: the kernel also reduces its output for the batch norm that consumes it.  Per-CTA partial sums
// go to bf.part[conv_tc_grid(B, H, W)][2C]; the CTA that finishes last (ticket in *bf.counter, zero before and after)
// adds them in a fixed order and stores the result.  With bf.x == nullptr the sums are (sum y, sum y^2) per channel and
// the result is the forward statistics bf.o0 = mean, bf.o1 = 1/sqrt(var + 1e-5).  Otherwise they are (sum dz, sum dz *
// xhat), dz = output * [bf.mask > 0], xhat = (bf.x - bf.mean) * bf.invstd: the two reductions of the batch-norm
// backward whose incoming gradient is this kernel's output; bf.o0 = dbeta, bf.o1 = dgamma.
// counter == nullptr: the kernel only leaves the per-CTA partials (*n_part_out rows, one per CTA of its grid) and the
// element-wise pass that consumes the sums folds them (BnPartials in kernels.h): no ticket, no serial tail in this kernel.
struct BnFuse {
    float *part = nullptr;
    unsigned *counter = nullptr;
    int *n_part_out = nullptr;
    float *o0 = nullptr, *o1 = nullptr;
    const void *mask = nullptr, *x = nullptr;
    const float *mean = nullptr, *invstd = nullptr;
};
// Input transform on the operand path of the forward convolution (gamma != nullptr): src holds the raw output y of the
// previous convolution and the kernel applies that convolution's batch norm and ReLU itself, a = relu(y * scale + shift)
// with scale = gamma * invstd and shift = beta - mean * scale, in shared memory between the TMA box and the MMAs (rows
// outside the image stay zero: they are this convolution's padding), and stores a to a_out (same shape as src) for the
// backward sweep.  The arithmetic is that of the element-wise batch-norm pass, value for value.  Available where
// conv_tc_xform_supported says so (the plan's thread count, with four transform warps per pipeline, fits the kernel).
// res != nullptr: the batch norm closes a residual block, a = relu(y * scale + shift + res) (res: same shape as src,
// fetched by a second TMA box per stage).
struct InXform {
    const void *gamma = nullptr, *beta = nullptr;
    const float *mean = nullptr, *invstd = nullptr;
    void *a_out = nullptr;
    const void *res = nullptr;
};
bool conv_tc_xform_supported(int B, int H, int W, int C, bool shared);
// true where the transform warps fit beside the launch plan the kernel would take anyway (the training step's sizes); at
// very large batches the plan is cut down to make room for them, and the separate element-wise kernel is the better choice
bool conv_tc_xform_keeps_plan(int B, int H, int W, int C, bool shared);
int launch_conv_tc(int dir, const void *src, const void *w, const void *w_packed, void *dst, int B, int H, int W, int C,
                   Shortcut sc, Launch s, BnFuse bf = BnFuse(), InXform xf = InXform());
int conv_tc_grid(int B, int H, int W);
size_t tc_packed_bytes(int C);
// One launch that re-arranges the filters of many convolutions of one weight version.
// element offset in wver, byte offset in packed; pad_ = job kind: 0 stride-1 C x C filter, 1 stride-2 C -> 2C filter
struct PackJobHost { long src_off; long dst_off; int C; int first_elem; int cin_real; int pad_; };
int launch_pack_one(const void *w, void *packed, int C, Launch s);
int launch_pack_filters(const void *wver, void *packed, const void *jobs_dev, int n_jobs, int total_elems,
                        Launch s);

// Stride-2 convolutions of the down-sampling blocks: Cout = 2 Cin, Cin in {16, 32}, even H and W, output map in whole
// 128-pixel tiles.  H, W are the input size.  dir as above; in dir 1 sc.mode == 2 adds the gradient of the
// parameter-free shortcut (sc.a = gradient of the block output, sc.b = block output).  w_packed (nullable):
// tc_s2_packed_bytes(Cin) bytes written by launch_pack_filters for a job of kind 1.
bool conv_tc_s2_supported(int B, int H, int W, int Cin, int Cout, int stride);
size_t tc_s2_packed_bytes(int Cin);
int launch_conv_tc_s2(int dir, const void *src, const void *w, const void *w_packed, void *dst, int B, int H, int W, int Cin,
                      Shortcut sc, Launch s);
int launch_wgrad_tc_s2(const void *x, const void *dy, float *dw, float *scratch, int B, int H, int W, int Cin, Launch s);

bool wgrad_tc_supported(int B, int H, int W, int Cin, int Cout, int stride);
size_t wgrad_tc_scratch_elems();
// cin_real < C: x was zero-padded from cin_real to C channels; dw is the canonical [C][cin_real][3][3] gradient.
int launch_wgrad_tc(const void *x, const void *dy, float *dw, float *scratch, int B, int H, int W, int C, int cin_real,
                    Launch s);

// Fully connected layers on the tensor cores (fc_tc.cu): x [B][in] and W [out][in] row-major bf16, read in place by TMA.
// Shapes taken: in a multiple of 64 up to 256, out up to 128; x and W must start on a 16-byte boundary, dx and dW too.
// y / dy are fp32 when out_f32 (the network's last layer: logits and loss gradient), else bf16; dW / db fp32; dx (nullable)
// bf16; y is only read when relu.  The backward launch produces dx, dW and db in one kernel.
bool fc_tc_shape_supported(int B, int in, int out);
bool fc_tc_supported(const void *x, const void *W, int B, int in, int out);
int launch_fc_fwd_tc(const void *x, const void *W, const void *bias, void *y, int B, int in, int out, int relu, int out_f32,
                     Launch s);
int launch_fc_bwd_tc(const void *x, const void *W, const void *y, const void *dy, void *dx, float *dW, float *db, int B,
                     int in, int out, int relu, int out_f32, Launch s);
int fc_tc_init();

// One-time per-process set-up (function attributes, driver entry points).  Returns a cudaError_t value.
int conv_tc_init();
// The process-wide error word that kernels launched without a context's own word (Launch::err == nullptr) raise when a
// bounded wait runs out (0 = none, -1 = cannot be read).
int conv_tc_error();
// Test aid: one CTA that waits, with a limit of `polls` polls, on a barrier nothing arrives on, then raises the error
// word of `s` with code 99 and returns.
int launch_wait_probe(unsigned polls, Launch s);
int conv_direct_init();

}  // namespace ddg
