// Host side of the DDG library: network planning, per-module ring buffers, the K-stream schedule of one DDG
// iteration (Algorithm 1 with the sweeps of Eq. 3 and Eq. 6-7), CUDA-graph replay, and the C ABI.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <memory>
#include <string>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "../../include/ddg.h"
#include "common.cuh"
#include "conv_tc.h"
#include "kernels.h"

using namespace ddg;

namespace {

thread_local std::string g_create_error;

struct TensorRef {
    int module;   // arena that holds the tensor (-1: none)
    size_t off;   // byte offset inside one arena slot
};

struct LayerPlan {
    ddg_layer spec;
    int Cin, Hin, Win, Cout, Hout, Wout;
    int module;
    size_t p_off;  // element offset of the layer's parameters inside its module's parameter slice
    size_t p_cnt;
    TensorRef in, out;            // layer input (may live in the previous module's arena) and output
    TensorRef y1, a1, y2, stats;  // basic block intermediates; stats = fp32 [4][C] (mean1,invstd1,mean2,invstd2)
    long pk1 = -1, pk2 = -1;      // byte offsets of the pre-arranged filter images (conv / conv1, conv2), -1 = none
    int pad_c = 0;                // first conv only: its input is stored zero-padded to this many channels (0 = as is)
    bool is_first, is_last;
};

struct Module {
    int first, last;            // layer range
    int R;                      // ring length K-k+1 (k 1-based): activation slots and weight versions
    size_t P;                   // parameter count
    size_t p_off_global;        // offset of the slice in the canonical flat vector
    size_t arena_bytes;         // one activation slot
    char *arena = nullptr;      // R slots
    float *w = nullptr, *v = nullptr, *m2 = nullptr, *g = nullptr;
    char *wver = nullptr;       // R weight versions in the compute precision
    char *packed = nullptr;     // R sets of pre-arranged filter images for the tensor-core kernels
    size_t packed_bytes = 0;
    void *pack_jobs = nullptr;  // device table of PackJobHost
    int n_pack_jobs = 0, pack_elems = 0;
    char *tmp[3] = {nullptr, nullptr, nullptr};  // error-gradient temporaries of the backward sweep
    size_t tmp_bytes = 0;
    float *bn_scratch = nullptr, *wg_scratch = nullptr;
    char *delta_out[2] = {nullptr, nullptr};  // error gradient w.r.t. this module's input, double buffered
    size_t delta_bytes = 0;
    long last_sample = -1;
    cudaStream_t stream = nullptr;
    bool own_stream = false;
    cudaEvent_t ev_fwd = nullptr, ev_bwd = nullptr, ev_join = nullptr;
    cudaEvent_t ev_time[4] = {nullptr, nullptr, nullptr, nullptr};  // time_pieces: forward begin / end, backward begin / end
    // weight gradients run beside the error-gradient chain, on a second stream of the module
    cudaStream_t side = nullptr;
    cudaEvent_t ev_fork = nullptr, ev_side[4] = {nullptr, nullptr, nullptr, nullptr};
    char *dyring[4] = {nullptr, nullptr, nullptr, nullptr};  // conv-output error gradients, kept until their wgrad ran
    // step size and Adam bias corrections of the update that runs next, device resident (recorded updates read them)
    double *opt_dyn = nullptr;
    double dyn_sent[3] = {0.0, 0.0, 0.0};
    bool dyn_valid = false;
    // debug_checks: device counters {forward iteration, backward sample, update iteration} and one stamp per activation
    // slot, weight-version slot and error-gradient buffer: [3 counters][R][R][2]
    long long *stamps = nullptr;
    long long *fcount() const { return stamps; }
    long long *bcount() const { return stamps + 1; }
    long long *ucount() const { return stamps + 2; }
    long long *astamp(long i) const { return stamps + 3 + i % R; }
    long long *wstamp(long i) const { return stamps + 3 + R + i % R; }
    long long *dstamp(long i) const { return stamps + 3 + 2 * R + i % 2; }
};

// launch counter that remembers a launcher's refusal (negative return) instead of adding it
struct Count {
    long n = 0;
    bool failed = false;
    void operator+=(int r) { if (r < 0) failed = true; else n += r; }
    void operator+=(const Count &o) { n += o.n; failed = failed || o.failed; }
};

}  // namespace

struct ddg_ctx {
    int K = 0, n_layers = 0, prec = 0, B = 0, in_c = 0, in_h = 0, in_w = 0, classes = 0;
    ddg_opt opt{};
    ddg_cfg cfg{};
    std::vector<LayerPlan> layers;
    std::vector<Module> mods;
    size_t P = 0;
    long t = 0;
    int period = 1;
    float *x_stage = nullptr;  // K staged copies of the input batch (fp32 NCHW) and labels
    int *y_stage = nullptr;
    size_t x_elems = 0;
    float *dlogits = nullptr, *loss_dev = nullptr;
    float *pinned_loss = nullptr;
    cudaStream_t loss_stream = nullptr;  // carries the loss read-back, so that it waits for the forward sweep only
    // pipelined loss read-back (ddg_step_host_pipelined): iteration t's loss and error word land in slot t mod 2 of a
    // pinned ring, ev_loss[t mod 2] marks the copy, and the last module's next forward sweep waits for it before it
    // overwrites the device scalar
    float *pinned_ring = nullptr;
    cudaEvent_t ev_loss[2] = {nullptr, nullptr};
    long loss_pending = -1;  // iteration whose copy is the latest enqueued (-1: none)
    std::vector<cudaGraphExec_t> graphs;
    std::vector<long> graph_launches;
    bool graphs_ready = false;
    long launches = 0;
    int *err_word = nullptr;  // device: raised by a kernel whose bounded wait ran out or by a ring-stamp mismatch
    bool broken = false;
    std::string err;
    // the element-wise batch-norm passes fold the convolution epilogues' partial sums themselves (ddg_cfg.bn_fold)
    bool fold_in_consumer() const { return cfg.bn_fold == 2 || (cfg.bn_fold == 0 && K == 1); }
    // how this context's kernels are launched on stream st (Launch in kernels.h)
    Launch lx(cudaStream_t st) const {
        const int pdl = cfg.launch_overlap == 1 ? 0 : (cfg.launch_overlap == 2 ? 1 : (K == 1 ? 1 : 2));
        return Launch(st, pdl, K > 1, err_word);
    }
};

namespace {

void set_err(ddg_ctx *c, const char *fmt, ...) {
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof(buf), fmt, ap);
    va_end(ap);
    if (c) c->err = buf;
    g_create_error = buf;
}

#define CU(call)                                                                                     \
    do {                                                                                             \
        cudaError_t e_ = (call);                                                                     \
        if (e_ != cudaSuccess) {                                                                     \
            set_err(ctx, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), __FILE__, __LINE__); \
            if (ctx) ctx->broken = true;                                                             \
            return e_ == cudaErrorMemoryAllocation ? DDG_ERR_OOM : DDG_ERR_CUDA;                     \
        }                                                                                            \
    } while (0)

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

size_t layer_params(const ddg_layer &s) {
    switch (s.kind) {
    case DDG_FC: return (size_t)s.c_in * s.c_out + (s.has_bias ? s.c_out : 0);
    case DDG_CONV3X3: return (size_t)s.c_in * s.c_out * 9;
    case DDG_BN: return 2 * (size_t)s.c_in;
    case DDG_BASIC_BLOCK: return (size_t)s.c_in * s.c_out * 9 + (size_t)s.c_out * s.c_out * 9 + 4 * (size_t)s.c_out;
    case DDG_BASIC_BLOCK_PROJ:
        return (size_t)s.c_in * s.c_out * 9 + (size_t)s.c_out * s.c_out * 9 + 4 * (size_t)s.c_out + (size_t)s.c_in * s.c_out;
    default: return 0;
    }
}

bool is_block(int kind) { return kind == DDG_BASIC_BLOCK || kind == DDG_BASIC_BLOCK_PROJ; }

int gcd_i(int a, int b) { return b ? gcd_i(b, a % b) : a; }

char *slot_ptr(ddg_ctx *c, TensorRef r, long iter) {
    Module &m = c->mods[r.module];
    return m.arena + (size_t)(iter % m.R) * m.arena_bytes + r.off;
}

// ---- convolution dispatch: tensor-core path where it applies, CUDA cores otherwise --------------------
int conv_fwd(ddg_ctx *c, const void *x, const void *w, const void *wp, void *y, int H, int W, int Cin, int Cout,
             int stride, int relu, Launch s) {
    if (c->prec == P_BF16 && !relu && conv_tc_supported(c->B, H, W, Cin, Cout, stride))
        return launch_conv_tc(0, x, w, wp, y, c->B, H, W, Cin, Shortcut{}, s);
    if (c->prec == P_BF16 && !relu && conv_tc_s2_supported(c->B, H, W, Cin, Cout, stride))
        return launch_conv_tc_s2(0, x, w, wp, y, c->B, H, W, Cin, Shortcut{}, s);
    return launch_conv_fwd_direct(c->prec, x, w, y, c->B, H, W, Cin, Cout, stride, relu, s);
}
int conv_dgrad(ddg_ctx *c, const void *dy, const void *w, const void *wp, void *dx, int H, int W, int Cin, int Cout,
               int stride, Shortcut sc, Launch s) {
    if (c->prec == P_BF16 && sc.mode != 2 && conv_tc_supported(c->B, H, W, Cin, Cout, stride))
        return launch_conv_tc(1, dy, w, wp, dx, c->B, H, W, Cin, sc, s);
    if (c->prec == P_BF16 && sc.mode != 1 && conv_tc_s2_supported(c->B, H, W, Cin, Cout, stride))
        return launch_conv_tc_s2(1, dy, w, wp, dx, c->B, H, W, Cin, sc, s);
    return launch_conv_dgrad_direct(c->prec, dy, w, dx, c->B, H, W, Cin, Cout, stride, sc, s);
}
int conv_wgrad(ddg_ctx *c, Module &m, const void *x, const void *dy, float *dw, int H, int W, int Cin, int Cout,
               int stride, Launch s) {
    if (c->prec == P_BF16 && wgrad_tc_supported(c->B, H, W, Cin, Cout, stride))
        return launch_wgrad_tc(x, dy, dw, m.wg_scratch, c->B, H, W, Cin, Cin, s);
    if (c->prec == P_BF16 && conv_tc_s2_supported(c->B, H, W, Cin, Cout, stride))
        return launch_wgrad_tc_s2(x, dy, dw, m.wg_scratch, c->B, H, W, Cin, s);
    return launch_conv_wgrad_direct(c->prec, x, dy, dw, m.wg_scratch, c->B, H, W, Cin, Cout, stride, s);
}

// ---- FC dispatch: tensor-core kernels in bf16 mode where shape and alignment allow, CUDA cores otherwise -----------
bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
int fc_fwd(ddg_ctx *c, const void *x, const void *W, const void *bias, void *y, int in, int out, int relu, int out_f32,
           Launch s) {
    if (c->prec == P_BF16 && fc_tc_supported(x, W, c->B, in, out))
        return launch_fc_fwd_tc(x, W, bias, y, c->B, in, out, relu, out_f32, s);
    return launch_fc_fwd(c->prec, x, W, bias, y, c->B, in, out, relu, out_f32, s);
}
int fc_bwd(ddg_ctx *c, const void *x, const void *W, const void *y, const void *dy, void *dx, float *dW, float *db, int in,
           int out, int relu, int out_f32, Launch s) {
    if (c->prec == P_BF16 && fc_tc_supported(x, W, c->B, in, out) && aligned16(dW) && aligned16(dx))
        return launch_fc_bwd_tc(x, W, y, dy, dx, dW, db, c->B, in, out, relu, out_f32, s);
    return launch_fc_bwd(c->prec, x, W, y, dy, dx, dW, db, c->B, in, out, relu, out_f32, s);
}

// ---- forward sweep of module k on the minibatch of iteration t (Eq. 3) --------------------------------
Count forward_module(ddg_ctx *c, int k, long t) {
    Module &m = c->mods[k];
    const Launch s = c->lx(m.stream);
    const size_t es = elem_size(c->prec);
    const char *wv = m.wver + (size_t)(t % m.R) * m.P * es;
    const char *pk = m.packed ? m.packed + (size_t)(t % m.R) * m.packed_bytes : nullptr;
    auto pkp = [&](long off) -> const void * { return (pk && off >= 0) ? pk + off : nullptr; };
    Count n;
    const bool fuse_bn = !c->cfg.separate_bn_sums;
    // A block's closing pass out = relu(bn2(y2) + x) may be left to the first convolution of the next block, which then
    // reads y2 and x, computes `out` on its operand path and stores it: `owed` describes such a pass.
    InXform owed;
    const void *owed_src = nullptr;
    for (int l = m.first; l <= m.last; ++l) {
        LayerPlan &L = c->layers[l];
        const char *w = wv + L.p_off * es;
        const void *in;
        if (L.is_first) {  // layout shim: staged NCHW fp32 -> NHWC in the compute precision, kept in the arena
            char *xin = slot_ptr(c, L.in, t);
            n += launch_shim(c->prec, c->x_stage + (size_t)(t % c->K) * c->x_elems, xin, c->B, c->in_c, c->in_h,
                             c->in_w, L.pad_c ? L.pad_c : c->in_c, s);
            in = xin;
        } else {
            in = slot_ptr(c, L.in, t);
        }
        char *out = slot_ptr(c, L.out, t);
        const int B = c->B;
        switch (L.spec.kind) {
        case DDG_FC:
            n += fc_fwd(c, in, w, L.spec.has_bias ? w + (size_t)L.Cin * L.Cout * es : nullptr, out, L.Cin, L.Cout,
                        L.spec.relu_after, L.is_last, s);
            break;
        case DDG_CONV3X3:
            if (L.pad_c)  // stem on the tensor cores: input and filter image zero-padded to pad_c channels
                n += launch_conv_tc(0, in, w, pkp(L.pk1), out, B, L.Hin, L.Win, L.pad_c, Shortcut{}, s);
            else
                n += conv_fwd(c, in, w, pkp(L.pk1), out, L.Hin, L.Win, L.Cin, L.Cout, L.spec.stride, L.spec.relu_after, s);
            break;
        case DDG_BN: {
            float *st = (float *)slot_ptr(c, L.stats, t);
            n += launch_bn_stats(c->prec, in, st, st + L.Cin, m.bn_scratch, (long)B * L.Hin * L.Win, L.Cin, s);
            n += launch_bn_apply(c->prec, in, w, w + (size_t)L.Cin * es, st, st + L.Cin, Shortcut{}, out, B, L.Hin,
                                 L.Win, L.Cin, L.spec.relu_after, s);
            break;
        }
        case DDG_RELU:
            n += launch_relu_fwd(c->prec, in, out, (size_t)B * L.Cin * L.Hin * L.Win, s);
            break;
        case DDG_GLOBAL_AVGPOOL:
            n += launch_avgpool_fwd(c->prec, in, out, B, L.Hin * L.Win, L.Cin, s);
            break;
        case DDG_BASIC_BLOCK:
        case DDG_BASIC_BLOCK_PROJ: {
            const int Ci = L.Cin, Co = L.Cout, st = L.spec.stride;
            const char *w1 = w, *g1 = w1 + (size_t)Co * Ci * 9 * es, *b1 = g1 + (size_t)Co * es;
            const char *w2 = b1 + (size_t)Co * es, *g2 = w2 + (size_t)Co * Co * 9 * es, *b2 = g2 + (size_t)Co * es;
            const char *ws = b2 + (size_t)Co * es;  // projection filter, DDG_BASIC_BLOCK_PROJ only
            char *y1 = slot_ptr(c, L.y1, t), *a1 = slot_ptr(c, L.a1, t), *y2 = slot_ptr(c, L.y2, t);
            float *stt = (float *)slot_ptr(c, L.stats, t);
            const long npix = (long)B * L.Hout * L.Wout;
            // convolution followed by its batch norm; the statistics come from the convolution's epilogue where the
            // tensor-core kernel runs, from a reduction kernel otherwise
            // a convolution and the statistics of the batch norm that follows it; xf: an input transform for it to carry
            // leave_partials: the pass that consumes the statistics is an element-wise kernel that folds the epilogue's
            // per-CTA partial sums itself (no serial fold at the end of the convolution); returns them
            auto conv_stats = [&](const void *xin, const void *wc, const void *wp, void *yc, int H, int W, int Cic, int strd,
                                  float *mean, float *invstd, InXform xf, bool leave_partials) -> BnPartials {
                BnPartials bp;
                if (fuse_bn && c->prec == P_BF16 && conv_tc_supported(B, H, W, Cic, Co, strd)) {
                    BnFuse bf;
                    bf.part = m.bn_scratch + 32; bf.o0 = mean; bf.o1 = invstd;
                    if (leave_partials) { bf.n_part_out = &bp.n; bp.part = bf.part; }
                    else bf.counter = (unsigned *)m.bn_scratch;
                    n += launch_conv_tc(0, xin, wc, wp, yc, B, H, W, Cic, Shortcut{}, s, bf, xf);
                } else {
                    n += conv_fwd(c, xin, wc, wp, yc, H, W, Cic, Co, strd, 0, s);
                    n += launch_bn_stats(c->prec, yc, mean, invstd, m.bn_scratch, npix, Co, s);
                }
                return bp;
            };
            // bn1's normalise + ReLU pass rides on conv2's operand path where the tensor-core kernel can take it: conv2
            // then reads the raw y1, computes a1 in shared memory and stores it for the backward sweep
            const bool ride = c->cfg.fuse_bn_apply >= 1 && fuse_bn && c->prec == P_BF16 &&
                              conv_tc_xform_keeps_plan(B, L.Hout, L.Wout, Co, s.shared);
            const BnPartials bp1 = conv_stats(owed_src ? owed_src : in, w1, pkp(L.pk1), y1, L.Hin, L.Win, Ci, st, stt, stt + Co,
                                              owed, !ride && c->fold_in_consumer() && bn_apply_takes_partials(c->prec, Co, 0));
            owed = InXform{};
            owed_src = nullptr;
            if (!ride) n += launch_bn_apply(c->prec, y1, g1, b1, stt, stt + Co, Shortcut{}, a1, B, L.Hout, L.Wout, Co, 1, s, bp1);
            Shortcut sc{};
            sc.mode = (st == 1 && Ci == Co) ? 1 : 2;
            sc.a = in; sc.c_small = Ci; sc.h_big = L.Hin; sc.w_big = L.Win;
            if (L.spec.kind == DDG_BASIC_BLOCK_PROJ) {
                // projected shortcut W_s x into a temporary of the module (only this forward sweep reads it), then added
                // like an identity shortcut
                n += launch_conv1x1_fwd(c->prec, in, ws, m.tmp[0], B, L.Hin, L.Win, Ci, Co, st, s);
                sc.mode = 1; sc.a = m.tmp[0];
            }
            InXform xf;
            if (ride) { xf.gamma = g1; xf.beta = b1; xf.mean = stt; xf.invstd = stt + Co; xf.a_out = a1; }
            // the closing pass goes to the next block's first convolution when that is a plain stride-1 block of the same
            // width in this module and the shortcut is the identity (the residual box then has the shape of y2)
            bool defer = false;
            if (ride && c->cfg.fuse_bn_apply >= 2 && sc.mode == 1 && L.spec.kind == DDG_BASIC_BLOCK && l + 1 <= m.last) {
                const LayerPlan &Nx = c->layers[l + 1];
                defer = Nx.spec.kind == DDG_BASIC_BLOCK && Nx.spec.stride == 1 && Nx.Cin == Nx.Cout && Nx.Cin == Co &&
                        conv_tc_xform_keeps_plan(B, Nx.Hin, Nx.Win, Nx.Cin, s.shared);
            }
            const BnPartials bp2 = conv_stats(ride ? y1 : a1, w2, pkp(L.pk2), y2, L.Hout, L.Wout, Co, 1, stt + 2 * Co, stt + 3 * Co,
                                              xf, !defer && c->fold_in_consumer() && bn_apply_takes_partials(c->prec, Co, sc.mode));
            if (defer) {
                owed.gamma = g2; owed.beta = b2; owed.mean = stt + 2 * Co; owed.invstd = stt + 3 * Co;
                owed.a_out = out; owed.res = in;
                owed_src = y2;
            } else {
                n += launch_bn_apply(c->prec, y2, g2, b2, stt + 2 * Co, stt + 3 * Co, sc, out, B, L.Hout, L.Wout, Co, 1, s, bp2);
            }
            break;
        }
        }
    }
    if (k == c->K - 1) {  // loss f and the up-to-date error gradient of the last module
        LayerPlan &L = c->layers[m.last];
        n += launch_softmax_ce(c->prec, (const float *)slot_ptr(c, L.out, t), c->y_stage + (size_t)(t % c->K) * c->B,
                               c->loss_dev, c->dlogits, c->B, c->classes, s);
    }
    if (c->cfg.debug_checks) {
        // the weight version read must be the one written for iteration t; the activation slot now holds iteration t
        StampOp op{};
        op.counter = m.fcount(); op.check[0] = m.wstamp(t); op.set[0] = m.astamp(t);
        op.advance = 1; op.code = 1000 + 100 * k; op.err = c->err_word;
        n += launch_stamp(op, s);
    }
    return n;
}

// ---- backward sweep of module k at iteration t on the stored sample sidx = t-K+k (Eq. 6-7) ------------
Count backward_module(ddg_ctx *c, int k, long t, long sidx) {
    Module &m = c->mods[k];
    const Launch s = c->lx(m.stream), side = s.on(m.side);
    const size_t es = elem_size(c->prec);
    const char *wv = m.wver + (size_t)(sidx % m.R) * m.P * es;  // the weights w^s of the stored iteration
    const char *pk = m.packed ? m.packed + (size_t)(sidx % m.R) * m.packed_bytes : nullptr;
    auto pkp = [&](long off) -> const void * { return (pk && off >= 0) ? pk + off : nullptr; };
    Count n;
    const int B = c->B;
    if (c->cfg.debug_checks) {
        // activation slot and weight version must be those of sample sidx, and the incoming error gradient the one
        // module k+1 produced for that sample; the outgoing buffer is stamped with it
        StampOp op{};
        op.counter = m.bcount(); op.check[0] = m.astamp(sidx); op.check[1] = m.wstamp(sidx);
        if (k < c->K - 1) op.check[2] = c->mods[k + 1].dstamp(t + 1);
        if (k > 0) op.set[0] = m.dstamp(t);
        op.advance = 1; op.code = 1000 + 100 * k + 10; op.err = c->err_word;
        n += launch_stamp(op, s);
    }
    const char *cur = (k == c->K - 1) ? (const char *)c->dlogits : c->mods[k + 1].delta_out[(t + 1) % 2];
    int cur_tmp = -1;
    auto pick = [&](int e1, int e2) { for (int i = 0; i < 3; ++i) if (i != e1 && i != e2) return i; return 0; };
    // The weight gradient of a convolution needs only (layer input, dy); nothing on the way down to the module input
    // waits for it.  It runs on the module's side stream; dy lives in a ring of four buffers so that the chain can move
    // on, and the chain only waits when it comes back to a buffer whose weight gradient has not finished.
    // true when the kernel that produced `cur` already left the two sums (dbeta, dgamma) of the batch norm that
    // consumes it in that batch norm's gradient slots
    bool cur_sums = false;
    BnPartials cur_parts;  // ... as per-CTA partials that the element-wise pass folds (cur_sums is true as well)
    float *bn_part = m.bn_scratch + 32;
    unsigned *bn_counter = (unsigned *)m.bn_scratch;
    const bool fuse = !c->cfg.separate_bn_sums && c->prec == P_BF16;
    int dy_i = 0, last_side = -1;
    bool ring_used[4] = {false, false, false, false};
    auto ring_next = [&]() -> int {
        const int j = dy_i++ & 3;
        if (ring_used[j]) cudaStreamWaitEvent(s, m.ev_side[j], 0);
        return j;
    };
    auto side_wgrad = [&](int j, const void *x_in, const void *dy, float *gwp, int H, int W, int Ci, int Co, int st) {
        cudaEventRecord(m.ev_fork, s);
        cudaStreamWaitEvent(m.side, m.ev_fork, 0);
        n += conv_wgrad(c, m, x_in, dy, gwp, H, W, Ci, Co, st, side);
        cudaEventRecord(m.ev_side[j], m.side);
        ring_used[j] = true;
        last_side = j;
    };
    auto side_join = [&]() { if (last_side >= 0) cudaStreamWaitEvent(s, m.ev_side[last_side], 0); };
    for (int l = m.last; l >= m.first; --l) {
        LayerPlan &L = c->layers[l];
        const char *w = wv + L.p_off * es;
        float *gw = m.g + L.p_off;
        const char *in = slot_ptr(c, L.in, sidx);
        const char *out = slot_ptr(c, L.out, sidx);
        const bool mod_first = (l == m.first);
        const bool need_dx = !L.is_first;
        // destination of the error gradient w.r.t. the layer input
        int dst_tmp = -1;
        bool next_sums = false;
        BnPartials next_parts;
        char *dst = nullptr;
        if (need_dx) {
            if (mod_first) dst = m.delta_out[t % 2];
            else { dst_tmp = pick(cur_tmp, -1); dst = m.tmp[dst_tmp]; }
        }
        switch (L.spec.kind) {
        case DDG_FC:
            n += fc_bwd(c, in, w, out, cur, dst, gw, L.spec.has_bias ? gw + (size_t)L.Cin * L.Cout : nullptr, L.Cin,
                        L.Cout, L.spec.relu_after, L.is_last, s);
            break;
        case DDG_CONV3X3: {
            const char *dy = cur;
            if (L.spec.relu_after) {
                int tm = pick(cur_tmp, dst_tmp);
                n += launch_relu_bwd(c->prec, out, cur, m.tmp[tm], (size_t)B * L.Cout * L.Hout * L.Wout, s);
                dy = m.tmp[tm];
            }
            if (need_dx)
                n += conv_dgrad(c, dy, w, pkp(L.pk1), dst, L.Hin, L.Win, L.Cin, L.Cout, L.spec.stride, Shortcut{}, s);
            side_join();  // this one runs on the chain's own stream and shares the weight-gradient scratch
            if (L.pad_c) n += launch_wgrad_tc(in, dy, gw, m.wg_scratch, B, L.Hin, L.Win, L.pad_c, L.Cin, s);
            else n += conv_wgrad(c, m, in, dy, gw, L.Hin, L.Win, L.Cin, L.Cout, L.spec.stride, s);
            break;
        }
        case DDG_BN: {
            const float *st = (const float *)slot_ptr(c, L.stats, sidx);
            const long npix = (long)B * L.Hin * L.Win;
            n += launch_bn_bwd_reduce(c->prec, cur, out, in, st, st + L.Cin, gw, gw + L.Cin, m.bn_scratch, npix, L.Cin,
                                      L.spec.relu_after, s);
            char *d = dst ? dst : m.tmp[pick(cur_tmp, -1)];
            n += launch_bn_bwd_apply(c->prec, cur, out, in, w, st, st + L.Cin, gw, gw + L.Cin, d, npix, L.Cin,
                                     L.spec.relu_after, s);
            break;
        }
        case DDG_RELU:
            if (need_dx) n += launch_relu_bwd(c->prec, out, cur, dst, (size_t)B * L.Cin * L.Hin * L.Win, s);
            break;
        case DDG_GLOBAL_AVGPOOL:
            if (need_dx) n += launch_avgpool_bwd(c->prec, cur, dst, B, L.Hin * L.Win, L.Cin, s);
            break;
        case DDG_BASIC_BLOCK:
        case DDG_BASIC_BLOCK_PROJ: {
            const int Ci = L.Cin, Co = L.Cout, st = L.spec.stride;
            const bool proj = L.spec.kind == DDG_BASIC_BLOCK_PROJ;
            const size_t nw1 = (size_t)Co * Ci * 9, nw2 = (size_t)Co * Co * 9;
            const char *w1 = w, *g1 = w1 + nw1 * es, *w2 = g1 + 2 * (size_t)Co * es, *g2 = w2 + nw2 * es;
            const char *ws = g2 + 2 * (size_t)Co * es;
            float *gw1 = gw, *gg1 = gw1 + nw1, *gb1 = gg1 + Co, *gw2 = gb1 + Co, *gg2 = gw2 + nw2, *gb2 = gg2 + Co;
            float *gws = gb2 + Co;
            const char *y1 = slot_ptr(c, L.y1, sidx), *a1 = slot_ptr(c, L.a1, sidx), *y2 = slot_ptr(c, L.y2, sidx);
            const float *stt = (const float *)slot_ptr(c, L.stats, sidx);
            const long npix = (long)B * L.Hout * L.Wout;
            // the two scratch temporaries are the ones not holding the incoming error gradient
            const int tA = pick(cur_tmp, -1), tB = pick(cur_tmp, tA);
            (void)tA;
            const int j2 = ring_next();
            char *dy2 = m.dyring[j2], *da1 = m.tmp[tB];
            if (!cur_sums)
                n += launch_bn_bwd_reduce(c->prec, cur, out, y2, stt + 2 * Co, stt + 3 * Co, gg2, gb2, m.bn_scratch, npix, Co,
                                          1, s);
            n += launch_bn_bwd_apply(c->prec, cur, out, y2, g2, stt + 2 * Co, stt + 3 * Co, gg2, gb2, dy2, npix, Co, 1, s,
                                     cur_sums ? cur_parts : BnPartials());
            side_wgrad(j2, a1, dy2, gw2, L.Hout, L.Wout, Co, Co, 1);
            const int j1 = ring_next();
            char *dy1 = m.dyring[j1];
            BnPartials parts1;
            if (fuse && conv_tc_supported(B, L.Hout, L.Wout, Co, Co, 1)) {
                // the input gradient of conv2 is the incoming gradient of bn1: its two sums come out of the same kernel
                BnFuse bf;
                bf.part = bn_part; bf.o0 = gb1; bf.o1 = gg1;
                bf.mask = a1; bf.x = y1; bf.mean = stt; bf.invstd = stt + Co;
                if (c->fold_in_consumer() && bn_apply_takes_partials(c->prec, Co, 0)) { bf.n_part_out = &parts1.n; parts1.part = bn_part; }
                else bf.counter = bn_counter;
                n += launch_conv_tc(1, dy2, w2, pkp(L.pk2), da1, B, L.Hout, L.Wout, Co, Shortcut{}, s, bf);
            } else {
                n += conv_dgrad(c, dy2, w2, pkp(L.pk2), da1, L.Hout, L.Wout, Co, Co, 1, Shortcut{}, s);
                n += launch_bn_bwd_reduce(c->prec, da1, a1, y1, stt, stt + Co, gg1, gb1, m.bn_scratch, npix, Co, 1, s);
            }
            n += launch_bn_bwd_apply(c->prec, da1, a1, y1, g1, stt, stt + Co, gg1, gb1, dy1, npix, Co, 1, s, parts1);
            side_wgrad(j1, in, dy1, gw1, L.Hin, L.Win, Ci, Co, st);
            if (proj) {
                // weight gradient of the projection, on the chain's own stream (it reads the incoming gradient in place
                // and shares the weight-gradient scratch with the side stream: wait for what runs there first)
                side_join();
                n += launch_conv1x1_wgrad(c->prec, in, cur, out, gws, m.wg_scratch, B, L.Hin, L.Win, Ci, Co, st, s);
            }
            if (need_dx && proj) {
                char *dx = mod_first ? dst : da1;
                if (c->prec == P_BF16) {
                    // tensor-core input gradient of conv1, then the projection's share added in place
                    n += conv_dgrad(c, dy1, w1, pkp(L.pk1), dx, L.Hin, L.Win, Ci, Co, st, Shortcut{}, s);
                    n += launch_conv1x1_dgrad_add(c->prec, cur, out, ws, dx, B, L.Hin, L.Win, Ci, Co, st, s);
                } else {
                    // one kernel, one rounding: the CUDA-core input gradient adds W_s^T dz before it stores
                    Shortcut sc{};
                    sc.mode = 3; sc.a = cur; sc.b = out; sc.c_small = Ci; sc.h_big = L.Hin; sc.w_big = L.Win; sc.w = ws;
                    n += launch_conv_dgrad_direct(c->prec, dy1, w1, dx, B, L.Hin, L.Win, Ci, Co, st, sc, s);
                }
                if (!mod_first) { dst = dx; dst_tmp = tB; }
            } else if (need_dx) {
                Shortcut sc{};
                sc.mode = (st == 1 && Ci == Co) ? 1 : 2;
                sc.a = cur; sc.b = out; sc.c_small = Ci; sc.h_big = L.Hin; sc.w_big = L.Win;
                char *dx = mod_first ? dst : da1;  // da1 is dead once bn1's backward has run
                const LayerPlan *Pv = mod_first ? nullptr : &c->layers[l - 1];
                if (fuse && Pv && is_block(Pv->spec.kind) && sc.mode == 1 &&
                    conv_tc_supported(B, L.Hin, L.Win, Ci, Co, st)) {
                    // dx is the incoming gradient of the block below, whose second batch norm reduces it first: take
                    // those sums here (its output is this block's input, its bn2 input and statistics are in its slots)
                    const float *pst = (const float *)slot_ptr(c, Pv->stats, sidx);
                    // gradient slots of the block below: conv1, gamma1, beta1, conv2, gamma2, beta2
                    float *pg2 = m.g + Pv->p_off + (size_t)Ci * Pv->Cin * 9 + 2 * (size_t)Ci + (size_t)Ci * Ci * 9;
                    BnFuse bf;
                    bf.part = bn_part; bf.o1 = pg2; bf.o0 = pg2 + Ci;
                    bf.mask = in; bf.x = slot_ptr(c, Pv->y2, sidx);
                    bf.mean = pst + 2 * Ci; bf.invstd = pst + 3 * Ci;
                    next_parts = BnPartials();
                    if (c->fold_in_consumer() && bn_apply_takes_partials(c->prec, Ci, 0)) { bf.n_part_out = &next_parts.n; next_parts.part = bn_part; }
                    else bf.counter = bn_counter;
                    n += launch_conv_tc(1, dy1, w1, pkp(L.pk1), dx, B, L.Hin, L.Win, Ci, sc, s, bf);
                    next_sums = true;
                } else {
                    n += conv_dgrad(c, dy1, w1, pkp(L.pk1), dx, L.Hin, L.Win, Ci, Co, st, sc, s);
                }
                if (!mod_first) { dst = dx; dst_tmp = tB; }
            }
            break;
        }
        }
        cur = dst;
        cur_tmp = dst_tmp;
        cur_sums = next_sums;
        cur_parts = next_parts;
    }
    side_join();  // the update that follows reads every gradient of the module
    return n;
}

// Re-arrange the filters of weight version `slot` into the images the tensor-core kernels copy in one piece.
int pack_module(ddg_ctx *c, Module &m, int slot) {
    if (!m.packed || m.n_pack_jobs == 0) return 0;
    const size_t es = elem_size(c->prec);
    return launch_pack_filters(m.wver + (size_t)slot * m.P * es, m.packed + (size_t)slot * m.packed_bytes, m.pack_jobs,
                               m.n_pack_jobs, m.pack_elems, c->lx(m.stream));
}

// Step size and Adam bias corrections of iteration t (Algorithm 1: gamma_t; Algorithm 2: 1 - beta^(t+1) with the
// global t), as the doubles the update kernel computes with.
void opt_scalars(const ddg_ctx *c, long t, double out[3]) {
    out[0] = (double)c->opt.lr;
    out[1] = out[2] = 1.0;
    if (c->opt.kind == DDG_OPT_ADAM) {
        out[1] = 1.0 - pow((double)c->opt.beta1, (double)(t + 1));
        out[2] = 1.0 - pow((double)c->opt.beta2, (double)(t + 1));
    }
}

// Bring module k's device block of optimiser scalars up to iteration t, in stream order before its update.  Never
// called inside a capture: the recorded update reads the block, so one recording serves every step size and iteration.
int push_opt_scalars(ddg_ctx *c, int k, long t) {
    Module &m = c->mods[k];
    double v[3];
    opt_scalars(c, t, v);
    if (m.dyn_valid && v[0] == m.dyn_sent[0] && v[1] == m.dyn_sent[1] && v[2] == m.dyn_sent[2]) return 0;
    m.dyn_valid = true;
    for (int i = 0; i < 3; ++i) m.dyn_sent[i] = v[i];
    return launch_set_opt_scalars(m.opt_dyn, v[0], v[1], v[2], c->lx(m.stream));
}

// ---- update of module k with its delayed gradient (Eq. 8-9; Algorithm 1 / 2) --------------------------
Count update_module(ddg_ctx *c, int k, long t, bool have_grad) {
    Module &m = c->mods[k];
    const Launch s = c->lx(m.stream);
    Count n;
    UpdateArgs a{};
    a.mu = c->opt.momentum; a.wd = c->opt.weight_decay;
    a.b1 = c->opt.beta1; a.b2 = c->opt.beta2; a.eps = c->opt.eps;
    a.dyn = m.opt_dyn;
    if (!have_grad) a.mode = 2;  // Eq. 8: the delayed gradient does not exist yet; leave the module untouched
    else a.mode = c->opt.kind == DDG_OPT_ADAM ? 1 : 0;
    if (c->cfg.debug_checks) {  // the slot written below holds the weights of iteration t+1
        StampOp op{};
        op.counter = m.ucount(); op.set[0] = m.wstamp(t + 1); op.set_add = 1;
        op.advance = 1; op.code = 1000 + 100 * k + 20; op.err = c->err_word;
        n += launch_stamp(op, s);
    }
    if (a.mode == 2 && m.R == 1) return n;
    char *wv = m.wver + (size_t)((t + 1) % m.R) * m.P * elem_size(c->prec);
    n += launch_update(c->prec, m.w, m.v, m.m2, m.g, wv, m.P, a, s);
    n += pack_module(c, m, (int)((t + 1) % m.R));
    return n;
}

// One schedulable piece of an iteration: the forward sweep of module k (seg 0) or its backward sweep + update
// (seg 1).  Inside a piece the kernels form a chain on the module's stream.
ddg_status enqueue_segment(ddg_ctx *ctx, int k, int seg, long t, long *launches) {
    const long sidx = t - ctx->K + (k + 1);
    Count n;
    if (seg == 0) n += forward_module(ctx, k, t);
    else {
        if (sidx >= 0) n += backward_module(ctx, k, t, sidx);
        n += update_module(ctx, k, t, sidx >= 0);
    }
    if (n.failed) {
        set_err(ctx, "a kernel launcher refused its launch (tensor map or shared-memory plan) in module %d", k);
        return DDG_ERR_CUDA;
    }
    CU(cudaGetLastError());
    *launches = n.n;
    return DDG_OK;
}

// Record the CUDA graph of piece (k, seg) for the ring phase of iteration t (nothing runs).
ddg_status capture_segment(ddg_ctx *ctx, int k, int seg, long t) {
    Module &m = ctx->mods[k];
    const size_t idx = ((size_t)(t % ctx->period) * ctx->K + k) * 2 + seg;
    if (ctx->graphs[idx]) return DDG_OK;
    CU(cudaStreamBeginCapture(m.stream, cudaStreamCaptureModeThreadLocal));
    long n = 0;
    ddg_status st = enqueue_segment(ctx, k, seg, t, &n);
    cudaGraph_t graph = nullptr;
    cudaError_t e2 = cudaStreamEndCapture(m.stream, &graph);
    if (st != DDG_OK) { if (graph) cudaGraphDestroy(graph); return st; }
    CU(e2);
    cudaGraphExec_t exec = nullptr;
    cudaError_t e3 = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    CU(e3);
    ctx->graphs[idx] = exec;
    ctx->graph_launches[idx] = n;
    return DDG_OK;
}

// Record every piece of every ring phase at once, at the first steady-state iteration t0: what a piece launches
// depends on the iteration only through its ring slots (t mod R_k, t mod K, t mod 2), which repeat with the period, so
// phase p is recorded from the first iteration >= t0 that falls into it.  Afterwards every iteration is replay only.
ddg_status capture_all(ddg_ctx *ctx, long t0) {
    for (long t = t0; t < t0 + ctx->period; ++t)
        for (int k = 0; k < ctx->K; ++k)
            for (int seg = 0; seg < 2; ++seg) {
                ddg_status st = capture_segment(ctx, k, seg, t);
                if (st != DDG_OK) return st;
            }
    ctx->graphs_ready = true;
    return DDG_OK;
}

// Run a piece: directly, or as a replay of the CUDA graph recorded for (ring phase, module, piece).  The graph holds
// only the module's own chain; what orders the pieces against each other (module k+1's forward after module k's,
// module k's backward after the error gradient module k+1 produced one iteration earlier) stays outside as stream
// events, so consecutive iterations overlap exactly as they do without graphs.
ddg_status run_segment(ddg_ctx *ctx, int k, int seg, long t, bool use_graph, long *launches) {
    Module &m = ctx->mods[k];
    long extra = 0;
    if (seg == 1 && t - ctx->K + (k + 1) >= 0) extra = push_opt_scalars(ctx, k, t);
    if (!use_graph) {
        ddg_status st = enqueue_segment(ctx, k, seg, t, launches);
        *launches += extra;
        return st;
    }
    const size_t idx = ((size_t)(t % ctx->period) * ctx->K + k) * 2 + seg;
    CU(cudaGraphLaunch(ctx->graphs[idx], m.stream));
    *launches = ctx->graph_launches[idx] + extra;
    return DDG_OK;
}

// A piece as a timeline tool and the piece timer see it: an NVTX range on the enqueuing thread ("F2", "B2+U2") and,
// in contexts created with time_pieces, a timing event on the module's stream on either side.
struct PieceRange {
    ddg_ctx *ctx;
    Module &m;
    const int seg;
    bool open = true;
    PieceRange(ddg_ctx *c, int k, int s) : ctx(c), m(c->mods[k]), seg(s) {
        char name[24];
        snprintf(name, sizeof name, seg == 0 ? "F%d" : "B%d+U%d", k + 1, k + 1);
        nvtxRangePushA(name);
        if (m.ev_time[0]) cudaEventRecord(m.ev_time[2 * seg], m.stream);
    }
    cudaError_t close() {
        open = false;
        nvtxRangePop();
        return m.ev_time[0] ? cudaEventRecord(m.ev_time[2 * seg + 1], m.stream) : cudaSuccess;
    }
    ~PieceRange() { if (open) nvtxRangePop(); }
};

// Enqueue one whole iteration on the K streams.
ddg_status enqueue_iteration(ddg_ctx *ctx, long t, bool use_graph, long *launches) {
    const int K = ctx->K;
    long total = 0, n = 0;
    // forward sweep, module 1..K in order; module k+1 waits for module k's output
    for (int k = 0; k < K; ++k) {
        Module &m = ctx->mods[k];
        if (k > 0) CU(cudaStreamWaitEvent(m.stream, ctx->mods[k - 1].ev_fwd, 0));
        // a pipelined read-back of the previous loss must have left the device scalar before this sweep rewrites it
        if (k == K - 1 && ctx->loss_pending >= 0) CU(cudaStreamWaitEvent(m.stream, ctx->ev_loss[ctx->loss_pending & 1], 0));
        PieceRange range(ctx, k, 0);
        ddg_status st = run_segment(ctx, k, 0, t, use_graph, &n);
        if (st != DDG_OK) return st;
        total += n;
        if (range.close() != cudaSuccess) return DDG_ERR_CUDA;
        CU(cudaEventRecord(m.ev_fwd, m.stream));  // for module k+1; the last module's marks the loss
    }
    // backward sweeps and updates: independent across modules within the iteration ("for k in parallel").  Ascending
    // k, so that module k waits for the error gradient module k+1 recorded in the PREVIOUS iteration.
    for (int k = 0; k < K; ++k) {
        Module &m = ctx->mods[k];
        const long sidx = t - K + (k + 1);
        if (sidx >= 0 && k < K - 1) CU(cudaStreamWaitEvent(m.stream, ctx->mods[k + 1].ev_bwd, 0));
        PieceRange range(ctx, k, 1);
        ddg_status st = run_segment(ctx, k, 1, t, use_graph, &n);
        if (st != DDG_OK) return st;
        total += n;
        if (range.close() != cudaSuccess) return DDG_ERR_CUDA;
        if (sidx >= 0 && k > 0) CU(cudaEventRecord(m.ev_bwd, m.stream));
        m.last_sample = sidx >= 0 ? sidx : -1;
    }
    *launches = total;
    return DDG_OK;
}

ddg_status init_weights(ddg_ctx *ctx) {
    for (int l = 0; l < ctx->n_layers; ++l) {
        LayerPlan &L = ctx->layers[l];
        Module &m = ctx->mods[L.module];
        float *w = m.w + L.p_off;
        cudaStream_t s = m.stream;
        const unsigned long long seed = ctx->cfg.seed;
        switch (L.spec.kind) {
        case DDG_FC:
            launch_fill_normal(w, (size_t)L.Cin * L.Cout, sqrtf(2.f / L.Cin), seed, 2 * l, s);
            if (L.spec.has_bias) launch_fill_const(w + (size_t)L.Cin * L.Cout, L.Cout, 0.f, s);
            break;
        case DDG_CONV3X3:
            launch_fill_normal(w, (size_t)L.Cin * L.Cout * 9, sqrtf(2.f / (9 * L.Cin)), seed, 2 * l, s);
            break;
        case DDG_BN:
            launch_fill_const(w, L.Cin, 1.f, s);
            launch_fill_const(w + L.Cin, L.Cin, 0.f, s);
            break;
        case DDG_BASIC_BLOCK:
        case DDG_BASIC_BLOCK_PROJ: {
            const size_t nw1 = (size_t)L.Cout * L.Cin * 9, nw2 = (size_t)L.Cout * L.Cout * 9;
            if (L.spec.kind == DDG_BASIC_BLOCK_PROJ)
                launch_fill_normal(w + nw1 + 4 * L.Cout + nw2, (size_t)L.Cout * L.Cin, sqrtf(2.f / L.Cin), seed,
                                   2 * l + 1000003, s);
            launch_fill_normal(w, nw1, sqrtf(2.f / (9 * L.Cin)), seed, 2 * l, s);
            launch_fill_const(w + nw1, L.Cout, 1.f, s);
            launch_fill_const(w + nw1 + L.Cout, L.Cout, 0.f, s);
            launch_fill_normal(w + nw1 + 2 * L.Cout, nw2, sqrtf(2.f / (9 * L.Cout)), seed, 2 * l + 1, s);
            launch_fill_const(w + nw1 + 2 * L.Cout + nw2, L.Cout, 1.f, s);
            launch_fill_const(w + nw1 + 3 * L.Cout + nw2, L.Cout, 0.f, s);
            break;
        }
        default: break;
        }
    }
    for (auto &m : ctx->mods) { launch_cast(ctx->prec, m.w, m.wver, m.P, m.stream); pack_module(ctx, m, 0); }
    CU(cudaGetLastError());
    for (auto &m : ctx->mods) CU(cudaStreamSynchronize(m.stream));
    return DDG_OK;
}

// Turn a raised error word into the context's error state.  Codes below 1000: the bounded wait with that code ran
// out.  1000 + 100 * module + check: a ring-slot stamp did not match (debug_checks).
ddg_status report_error_word(ddg_ctx *ctx, int code) {
    if (code == 0) return DDG_OK;
    ctx->broken = true;
    if (code >= 1000) {
        static const char *const what[] = {"weight version read by the forward sweep", "?", "?", "?", "?", "?", "?", "?", "?", "?",
                                           "activation slot read by the backward sweep",
                                           "weight version read by the backward sweep",
                                           "error gradient received from the next module"};
        const int which = (code - 1000) % 100;
        set_err(ctx, "ring stamp mismatch in module %d: %s is not the one the iteration expects", (code - 1000) / 100,
                which < 13 ? what[which] : "?");
        return DDG_ERR_STATE;
    }
    set_err(ctx, "a kernel gave up on a bounded wait (code %d)", code);
    return DDG_ERR_TIMEOUT;
}

// reads the error word as it is now (does not wait for work in flight)
ddg_status check_kernel_errors(ddg_ctx *ctx) {
    int code = 0;
    CU(cudaMemcpy(&code, ctx->err_word, sizeof(int), cudaMemcpyDeviceToHost));
    return report_error_word(ctx, code);
}

ddg_status sync_all(ddg_ctx *ctx) {
    for (auto &m : ctx->mods) CU(cudaStreamSynchronize(m.stream));
    return check_kernel_errors(ctx);
}

}  // namespace

namespace ddg {
// lets the other translation units leave a message for ddg_last_error(NULL)
void set_global_error(const char *msg) { g_create_error = msg; }
}  // namespace ddg

// ========================================================================================================
// C ABI
// ========================================================================================================
extern "C" {

const char *ddg_last_error(const ddg_ctx *ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

void ddg_destroy(ddg_ctx *ctx) {
    if (!ctx) return;
    for (auto &m : ctx->mods)
        if (m.stream) cudaStreamSynchronize(m.stream);
    for (auto g : ctx->graphs)
        if (g) cudaGraphExecDestroy(g);
    for (auto &m : ctx->mods) {
        cudaFree(m.packed); cudaFree(m.pack_jobs);
        cudaFree(m.arena); cudaFree(m.w); cudaFree(m.v); cudaFree(m.m2); cudaFree(m.g); cudaFree(m.wver);
        for (char *p : m.tmp) cudaFree(p);
        for (char *p : m.dyring) cudaFree(p);
        if (m.side) { cudaStreamSynchronize(m.side); cudaStreamDestroy(m.side); }
        if (m.ev_fork) cudaEventDestroy(m.ev_fork);
        for (auto e : m.ev_side) if (e) cudaEventDestroy(e);
        cudaFree(m.bn_scratch); cudaFree(m.wg_scratch);
        cudaFree(m.opt_dyn); cudaFree(m.stamps);
        cudaFree(m.delta_out[0]); cudaFree(m.delta_out[1]);
        if (m.ev_fwd) cudaEventDestroy(m.ev_fwd);
        if (m.ev_bwd) cudaEventDestroy(m.ev_bwd);
        if (m.ev_join) cudaEventDestroy(m.ev_join);
        for (auto e : m.ev_time) if (e) cudaEventDestroy(e);
        if (m.own_stream && m.stream) cudaStreamDestroy(m.stream);
    }
    cudaFree(ctx->x_stage); cudaFree(ctx->y_stage); cudaFree(ctx->dlogits); cudaFree(ctx->loss_dev);
    cudaFree(ctx->err_word);
    if (ctx->pinned_loss) cudaFreeHost(ctx->pinned_loss);
    if (ctx->pinned_ring) cudaFreeHost(ctx->pinned_ring);
    for (auto e : ctx->ev_loss) if (e) cudaEventDestroy(e);
    if (ctx->loss_stream) cudaStreamDestroy(ctx->loss_stream);
    delete ctx;
}

ddg_status ddg_create(const ddg_layer *layers, int n_layers, const int *split_after, int K, const ddg_opt *opt,
                      const ddg_cfg *cfg, ddg_ctx **out) {
    ddg_ctx *ctx = nullptr;  // CU() reports into the thread-local create error while this is null
    if (!layers || !opt || !cfg || !out || n_layers < 1 || K < 1 || (K > 1 && !split_after)) {
        set_err(nullptr, "ddg_create: NULL argument or non-positive count");
        return DDG_ERR_INVALID_ARG;
    }
    *out = nullptr;
    if (K > n_layers || K > 8) { set_err(nullptr, "ddg_create: K=%d out of range (1..min(8, layers))", K); return DDG_ERR_BAD_SPEC; }
    if (cfg->batch < 1 || cfg->in_c < 1 || cfg->in_h < 1 || cfg->in_w < 1 || cfg->num_classes < 1 ||
        (cfg->precision != DDG_FP32 && cfg->precision != DDG_BF16)) {
        set_err(nullptr, "ddg_create: bad configuration");
        return DDG_ERR_INVALID_ARG;
    }
    if (opt->kind != DDG_OPT_SGD && opt->kind != DDG_OPT_ADAM) { set_err(nullptr, "ddg_create: unknown optimiser"); return DDG_ERR_INVALID_ARG; }
    if (cfg->bn_fold < 0 || cfg->bn_fold > 2 || cfg->fuse_bn_apply < 0 || cfg->fuse_bn_apply > 2) { set_err(nullptr, "ddg_create: bn_fold and fuse_bn_apply must be 0, 1 or 2"); return DDG_ERR_INVALID_ARG; }
    if (cfg->launch_overlap < 0 || cfg->launch_overlap > 2) { set_err(nullptr, "ddg_create: launch_overlap must be 0, 1 or 2"); return DDG_ERR_INVALID_ARG; }
    for (int k = 0; k + 1 < K; ++k)
        if (split_after[k] < 0 || split_after[k] >= n_layers - 1 || (k > 0 && split_after[k] <= split_after[k - 1])) {
            set_err(nullptr, "ddg_create: split points must be strictly increasing layer indices in [0, n_layers-2]");
            return DDG_ERR_BAD_SPEC;
        }
    int dev_count = 0;
    if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count == 0) {
        set_err(nullptr, "ddg_create: no CUDA device; this library has no CPU path");
        return DDG_ERR_CUDA;
    }
    int dev = 0, major = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (major != 10) { set_err(nullptr, "ddg_create: needs a compute-capability 10.x device (found %d.x)", major); return DDG_ERR_UNSUPPORTED; }

    {
        cudaError_t ie = (cudaError_t)conv_direct_init();
        if (ie == cudaSuccess) ie = (cudaError_t)conv_tc_init();
        if (ie != cudaSuccess) { set_err(nullptr, "kernel set-up failed: %s", cudaGetErrorString(ie)); return DDG_ERR_CUDA; }
    }
    std::unique_ptr<ddg_ctx, void (*)(ddg_ctx *)> holder(new ddg_ctx, ddg_destroy);
    ddg_ctx *c = holder.get();
    c->K = K; c->n_layers = n_layers; c->prec = cfg->precision == DDG_BF16 ? P_BF16 : P_F32;
    c->B = cfg->batch; c->in_c = cfg->in_c; c->in_h = cfg->in_h; c->in_w = cfg->in_w; c->classes = cfg->num_classes;
    c->opt = *opt; c->cfg = *cfg;
    const size_t es = elem_size(c->prec);

    // ---- shapes and validation (Section 2: a chain of L layers) ----
    c->layers.resize(n_layers);
    int C = c->in_c, H = c->in_h, W = c->in_w;
    for (int l = 0; l < n_layers; ++l) {
        LayerPlan &L = c->layers[l];
        L.spec = layers[l];
        L.Cin = C; L.Hin = H; L.Win = W;
        L.is_first = (l == 0); L.is_last = (l == n_layers - 1);
        const ddg_layer &s = layers[l];
        bool ok = true;
        switch (s.kind) {
        case DDG_FC: ok = (H == 1 && W == 1 && s.c_in == C && s.c_out >= 1); C = s.c_out; break;
        case DDG_CONV3X3:
            ok = (s.c_in == C && s.c_out >= 1 && (s.stride == 1 || s.stride == 2));
            if (ok && s.has_bias) { set_err(nullptr, "layer %d: convolution bias is not supported", l); return DDG_ERR_UNSUPPORTED; }
            C = s.c_out; H = (H - 1) / s.stride + 1; W = (W - 1) / s.stride + 1; break;
        case DDG_BASIC_BLOCK:
            ok = (s.c_in == C && s.c_out >= s.c_in && (s.stride == 1 || s.stride == 2) &&
                  (s.stride == 2 || s.c_out == s.c_in));
            C = s.c_out; H = (H - 1) / s.stride + 1; W = (W - 1) / s.stride + 1; break;
        case DDG_BASIC_BLOCK_PROJ:
            ok = (s.c_in == C && s.c_out >= 1 && (s.stride == 1 || s.stride == 2));
            C = s.c_out; H = (H - 1) / s.stride + 1; W = (W - 1) / s.stride + 1; break;
        case DDG_BN: ok = (s.c_in == C); break;
        case DDG_RELU: break;
        case DDG_GLOBAL_AVGPOOL: H = 1; W = 1; break;
        default: ok = false;
        }
        if (!ok) { set_err(nullptr, "layer %d: specification does not fit its input [%d,%d,%d]", l, L.Cin, L.Hin, L.Win); return DDG_ERR_BAD_SPEC; }
        if ((s.kind == DDG_CONV3X3 || is_block(s.kind) || s.kind == DDG_BN || s.kind == DDG_GLOBAL_AVGPOOL) &&
            (C > 128 || L.Cin > 128 || (size_t)L.Cin * C > 4096)) {
            set_err(nullptr, "layer %d: channel counts above 64x64 (or 128 for BN / pooling) are not supported", l);
            return DDG_ERR_UNSUPPORTED;
        }
        L.Cout = C; L.Hout = H; L.Wout = W;
        L.p_cnt = layer_params(s);
    }
    if (layers[n_layers - 1].kind != DDG_FC || C != c->classes) {
        set_err(nullptr, "the last layer must be an FC layer with num_classes outputs");
        return DDG_ERR_BAD_SPEC;
    }

    // ---- modules (Section 3: K groups of consecutive layers) and arena layout ----
    c->mods.resize(K);
    size_t p_global = 0;
    for (int k = 0; k < K; ++k) {
        Module &m = c->mods[k];
        m.first = k == 0 ? 0 : split_after[k - 1] + 1;
        m.last = k == K - 1 ? n_layers - 1 : split_after[k];
        m.R = K - k;  // K-k+1 with 1-based k
        m.p_off_global = p_global;
        size_t off = 0, p = 0;
        auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
        for (int l = m.first; l <= m.last; ++l) {
            LayerPlan &L = c->layers[l];
            L.module = k;
            L.p_off = p;
            p += L.p_cnt;
            size_t n_in = (size_t)c->B * L.Cin * L.Hin * L.Win;
            const size_t n_out = (size_t)c->B * L.Cout * L.Hout * L.Wout;
            if (l == 0 && c->prec == P_BF16 && L.spec.kind == DDG_CONV3X3 && !L.spec.relu_after && L.spec.stride == 1 &&
                L.Cin < 16 && L.Cout == 16 && conv_tc_supported(c->B, L.Hin, L.Win, 16, 16, 1)) {
                // a narrow first convolution (3 input channels) runs on the tensor-core kernels with its input stored
                // zero-padded to 16 channels
                L.pad_c = 16;
                n_in = (size_t)c->B * 16 * L.Hin * L.Win;
            }
            if (l == 0) L.in = {0, take(n_in * es)};                      // the shimmed input lives in module 1's arena
            else L.in = c->layers[l - 1].out;                             // may point into the previous module's arena
            L.out = {k, take(L.is_last ? n_out * sizeof(float) : n_out * es)};
            if (is_block(L.spec.kind)) {
                L.y1 = {k, take(n_out * es)}; L.a1 = {k, take(n_out * es)}; L.y2 = {k, take(n_out * es)};
                L.stats = {k, take(4 * (size_t)L.Cout * sizeof(float))};
            } else if (L.spec.kind == DDG_BN) {
                L.stats = {k, take(2 * (size_t)L.Cin * sizeof(float))};
            }
            m.tmp_bytes = std::max(m.tmp_bytes, std::max(n_in, n_out) * es);
        }
        m.P = p;
        m.arena_bytes = off;
        p_global += p;
    }
    c->P = p_global;
    c->period = 2;
    for (int k = 0; k < K; ++k) c->period = c->period / gcd_i(c->period, c->mods[k].R) * c->mods[k].R;
    c->graphs.assign((size_t)c->period * K * 2, nullptr);
    c->graph_launches.assign((size_t)c->period * K * 2, 0);

    // ---- device state ----
    ctx = c;  // from here on CU() records into the context
    for (int k = 0; k < K; ++k) {
        Module &m = c->mods[k];
        if (cfg->streams) m.stream = (cudaStream_t)cfg->streams[k];
        else { CU(cudaStreamCreateWithFlags(&m.stream, cudaStreamNonBlocking)); m.own_stream = true; }
        CU(cudaEventCreateWithFlags(&m.ev_fwd, cudaEventDisableTiming));
        CU(cudaEventCreateWithFlags(&m.ev_bwd, cudaEventDisableTiming));
        CU(cudaEventCreateWithFlags(&m.ev_join, cudaEventDisableTiming));
        if (cfg->time_pieces) for (auto &e : m.ev_time) CU(cudaEventCreate(&e));
        const size_t pn = std::max<size_t>(m.P, 1);
        CU(cudaMalloc(&m.arena, m.arena_bytes * m.R));
        CU(cudaMemset(m.arena, 0, m.arena_bytes * m.R));
        CU(cudaMalloc(&m.w, pn * 4)); CU(cudaMalloc(&m.v, pn * 4)); CU(cudaMalloc(&m.g, pn * 4));
        CU(cudaMemset(m.v, 0, pn * 4)); CU(cudaMemset(m.g, 0, pn * 4)); CU(cudaMemset(m.w, 0, pn * 4));
        if (opt->kind == DDG_OPT_ADAM) { CU(cudaMalloc(&m.m2, pn * 4)); CU(cudaMemset(m.m2, 0, pn * 4)); }
        CU(cudaMalloc(&m.wver, pn * es * m.R));
        CU(cudaMemset(m.wver, 0, pn * es * m.R));
        for (auto &p : m.tmp) CU(cudaMalloc(&p, m.tmp_bytes));
        for (auto &p : m.dyring) CU(cudaMalloc(&p, m.tmp_bytes));
        CU(cudaMalloc(&m.opt_dyn, 3 * sizeof(double)));
        CU(cudaMemset(m.opt_dyn, 0, 3 * sizeof(double)));
        {   // ring stamps: counters 0; activation stamps -1 (nothing written); weight version 0 sits in slot 0
            std::vector<long long> init(3 + 2 * (size_t)m.R + 2, -1);
            init[0] = init[1] = init[2] = 0;
            init[3 + m.R] = 0;
            CU(cudaMalloc(&m.stamps, init.size() * sizeof(long long)));
            CU(cudaMemcpy(m.stamps, init.data(), init.size() * sizeof(long long), cudaMemcpyHostToDevice));
        }
        {   // the side stream inherits the priority of the module's stream (the caller may rank the modules)
            int prio = 0;
            CU(cudaStreamGetPriority(m.stream, &prio));
            CU(cudaStreamCreateWithPriority(&m.side, cudaStreamNonBlocking, prio));
        }
        CU(cudaEventCreateWithFlags(&m.ev_fork, cudaEventDisableTiming));
        for (auto &e : m.ev_side) CU(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
        size_t bn_max = 0, wg_max = 0;
        for (int l = m.first; l <= m.last; ++l) {
            LayerPlan &L = c->layers[l];
            if (L.spec.kind == DDG_BN || is_block(L.spec.kind)) bn_max = std::max(bn_max, bn_scratch_elems(L.Cout));
            if (L.spec.kind == DDG_BASIC_BLOCK_PROJ) wg_max = std::max(wg_max, conv1x1_wgrad_scratch_elems(L.Cin, L.Cout));
            if (L.spec.kind == DDG_CONV3X3)
                wg_max = std::max(wg_max, conv_wgrad_scratch_elems(c->B, L.Hin, L.Win, L.Cin, L.Cout, L.spec.stride));
            if (is_block(L.spec.kind)) {
                wg_max = std::max(wg_max, conv_wgrad_scratch_elems(c->B, L.Hin, L.Win, L.Cin, L.Cout, L.spec.stride));
                wg_max = std::max(wg_max, conv_wgrad_scratch_elems(c->B, L.Hout, L.Wout, L.Cout, L.Cout, 1));
            }
        }
        wg_max = std::max(wg_max, wgrad_tc_scratch_elems());
        if (c->prec == P_BF16) {  // pre-arranged filter images for the convolutions the tensor-core kernels take
            std::vector<PackJobHost> jobs;
            size_t pk_off = 0;
            int elems = 0;
            auto plan = [&](long *slot, size_t w_off, int H, int W, int Ci, int Co, int stride, int cin_real = 0) {
                if (conv_tc_s2_supported(c->B, H, W, Ci, Co, stride)) {
                    *slot = (long)pk_off;
                    jobs.push_back(PackJobHost{(long)w_off, (long)pk_off, Ci, elems, Ci, 1});
                    pk_off += tc_s2_packed_bytes(Ci);
                    elems += 9 * Ci * Co;
                    return;
                }
                if (!conv_tc_supported(c->B, H, W, Ci, Co, stride)) return;
                *slot = (long)pk_off;
                jobs.push_back(PackJobHost{(long)w_off, (long)pk_off, Ci, elems, cin_real ? cin_real : Ci, 0});
                pk_off += tc_packed_bytes(Ci);
                elems += 9 * Ci * Ci;
            };
            for (int l = m.first; l <= m.last; ++l) {
                LayerPlan &L = c->layers[l];
                if (L.spec.kind == DDG_CONV3X3 && L.pad_c)
                    plan(&L.pk1, L.p_off, L.Hin, L.Win, L.pad_c, L.Cout, 1, L.Cin);
                else if (L.spec.kind == DDG_CONV3X3 && !L.spec.relu_after)
                    plan(&L.pk1, L.p_off, L.Hin, L.Win, L.Cin, L.Cout, L.spec.stride);
                if (is_block(L.spec.kind)) {
                    plan(&L.pk1, L.p_off, L.Hin, L.Win, L.Cin, L.Cout, L.spec.stride);
                    plan(&L.pk2, L.p_off + (size_t)L.Cout * L.Cin * 9 + 2 * (size_t)L.Cout, L.Hout, L.Wout, L.Cout, L.Cout, 1);
                }
            }
            if (!jobs.empty()) {
                m.packed_bytes = pk_off;
                m.n_pack_jobs = (int)jobs.size();
                m.pack_elems = elems;
                CU(cudaMalloc(&m.packed, pk_off * m.R));
                CU(cudaMalloc(&m.pack_jobs, jobs.size() * sizeof(PackJobHost)));
                CU(cudaMemcpy(m.pack_jobs, jobs.data(), jobs.size() * sizeof(PackJobHost), cudaMemcpyHostToDevice));
            }
        }
        CU(cudaMalloc(&m.bn_scratch, std::max<size_t>(bn_max, 64) * 4));
        CU(cudaMemset(m.bn_scratch, 0, std::max<size_t>(bn_max, 64) * 4));
        CU(cudaMalloc(&m.wg_scratch, std::max<size_t>(wg_max, 64) * 4));
        CU(cudaMemset(m.wg_scratch, 0, std::max<size_t>(wg_max, 64) * 4));
        if (k > 0) {
            LayerPlan &L = c->layers[m.first];
            m.delta_bytes = (size_t)c->B * L.Cin * L.Hin * L.Win * es;
            for (auto &p : m.delta_out) { CU(cudaMalloc(&p, m.delta_bytes)); CU(cudaMemset(p, 0, m.delta_bytes)); }
        }
    }
    c->x_elems = (size_t)c->B * c->in_c * c->in_h * c->in_w;
    CU(cudaMalloc(&c->x_stage, c->x_elems * 4 * K));
    CU(cudaMalloc(&c->y_stage, (size_t)c->B * 4 * K));
    CU(cudaMalloc(&c->dlogits, (size_t)c->B * c->classes * 4));
    CU(cudaMalloc(&c->loss_dev, 4));
    CU(cudaMemset(c->loss_dev, 0, 4));
    CU(cudaMalloc(&c->err_word, sizeof(int)));  // this context's own error word, clear at creation
    CU(cudaMemset(c->err_word, 0, sizeof(int)));
    CU(cudaMallocHost(&c->pinned_loss, 8));  // the loss, and the tensor-core kernels' error word read with it
    CU(cudaMallocHost(&c->pinned_ring, 16));
    for (auto &e : c->ev_loss) CU(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    CU(cudaStreamCreateWithFlags(&c->loss_stream, cudaStreamNonBlocking));
    // the memsets above ran on the legacy default stream, which the non-blocking module streams do not wait for
    CU(cudaDeviceSynchronize());
    ddg_status st = init_weights(c);
    if (st != DDG_OK) { g_create_error = c->err; return st; }
    *out = holder.release();
    return DDG_OK;
}

static ddg_status step_common(ddg_ctx *ctx, const float *x, const int *y, float *loss_host, cudaMemcpyKind kind,
                              bool pipelined = false) {
    if (!ctx || !x || !y) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    const long t = ctx->t;
    const int K = ctx->K;
    cudaStream_t s0 = ctx->mods[0].stream;
    // stage the batch: the sweeps (and graph replays) read library-owned buffers
    CU(cudaMemcpyAsync(ctx->x_stage + (size_t)(t % K) * ctx->x_elems, x, ctx->x_elems * 4, kind, s0));
    CU(cudaMemcpyAsync(ctx->y_stage + (size_t)(t % K) * ctx->B, y, (size_t)ctx->B * 4, kind, s0));
    // the first K-1 iterations have modules in warm-up and a different shape: they are not recorded
    const bool steady = t >= K - 1;
    if (ctx->cfg.use_graph && steady && !ctx->graphs_ready) {
        ddg_status cs = capture_all(ctx, t);
        if (cs != DDG_OK) { ctx->broken = true; return cs; }
    }
    ddg_status st = enqueue_iteration(ctx, t, ctx->cfg.use_graph && steady, &ctx->launches);
    if (st != DDG_OK) { ctx->broken = true; return st; }
    ctx->t = t + 1;
    if (pipelined) {
        // enqueue the read-back of this iteration's loss, hand out the previous iteration's (long complete)
        float *slot = ctx->pinned_ring + 2 * (t & 1);
        CU(cudaStreamWaitEvent(ctx->loss_stream, ctx->mods[K - 1].ev_fwd, 0));
        CU(cudaMemcpyAsync(slot, ctx->loss_dev, 4, cudaMemcpyDeviceToHost, ctx->loss_stream));
        CU(cudaMemcpyAsync(slot + 1, ctx->err_word, sizeof(int), cudaMemcpyDeviceToHost, ctx->loss_stream));
        CU(cudaEventRecord(ctx->ev_loss[t & 1], ctx->loss_stream));
        const long prev = ctx->loss_pending;
        ctx->loss_pending = t;
        if (loss_host) {
            if (prev < 0) *loss_host = nanf("");
            else {
                CU(cudaEventSynchronize(ctx->ev_loss[prev & 1]));
                const float *p = ctx->pinned_ring + 2 * (prev & 1);
                *loss_host = p[0];
                const int flag = *reinterpret_cast<const int *>(p + 1);
                if (flag != 0) return report_error_word(ctx, flag);
            }
        }
        return DDG_OK;
    }
    if (loss_host) {
        // The loss exists once the last module's forward sweep is done: wait for that only.  The backward sweeps and
        // updates of this iteration stay in flight and overlap the caller's next step (the decoupling DDG is about).
        CU(cudaStreamWaitEvent(ctx->loss_stream, ctx->mods[K - 1].ev_fwd, 0));
        CU(cudaMemcpyAsync(ctx->pinned_loss, ctx->loss_dev, 4, cudaMemcpyDeviceToHost, ctx->loss_stream));
        // error flags raised so far ride along (a later call or ddg_sync reports what is still running): one host wait
        int *flag = reinterpret_cast<int *>(ctx->pinned_loss + 1);
        *flag = 0;
        CU(cudaMemcpyAsync(flag, ctx->err_word, sizeof(int), cudaMemcpyDeviceToHost, ctx->loss_stream));
        CU(cudaStreamSynchronize(ctx->loss_stream));
        *loss_host = *ctx->pinned_loss;
        if (*flag != 0) return report_error_word(ctx, *flag);
    }
    return DDG_OK;
}

ddg_status ddg_step(ddg_ctx *ctx, const float *x_dev, const int *y_dev, float *loss_host) {
    return step_common(ctx, x_dev, y_dev, loss_host, cudaMemcpyDeviceToDevice);
}

ddg_status ddg_step_host(ddg_ctx *ctx, const float *x_host, const int *y_host, float *loss_host) {
    return step_common(ctx, x_host, y_host, loss_host, cudaMemcpyHostToDevice);
}

ddg_status ddg_step_host_pipelined(ddg_ctx *ctx, const float *x_host, const int *y_host, float *loss_prev_host) {
    return step_common(ctx, x_host, y_host, loss_prev_host, cudaMemcpyHostToDevice, true);
}

ddg_status ddg_pipelined_loss(ddg_ctx *ctx, float *loss_host) {
    if (!ctx || !loss_host) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    if (ctx->loss_pending < 0) {
        set_err(ctx, "ddg_pipelined_loss: no ddg_step_host_pipelined call has been made");
        return DDG_ERR_INVALID_ARG;
    }
    CU(cudaEventSynchronize(ctx->ev_loss[ctx->loss_pending & 1]));
    const float *p = ctx->pinned_ring + 2 * (ctx->loss_pending & 1);
    *loss_host = p[0];
    const int flag = *reinterpret_cast<const int *>(p + 1);
    if (flag != 0) return report_error_word(ctx, flag);
    return DDG_OK;
}

ddg_status ddg_set_lr(ddg_ctx *ctx, float lr) {
    if (!ctx) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    // the updates (recorded or not) read the step size from a device block that each module's stream refreshes, in
    // order, before its next update: nothing in flight is disturbed and nothing is re-recorded
    ctx->opt.lr = lr;
    return DDG_OK;
}

ddg_status ddg_param_count(const ddg_ctx *ctx, size_t *n, size_t *per_module) {
    if (!ctx || !n) return DDG_ERR_INVALID_ARG;
    *n = ctx->P;
    if (per_module) for (int k = 0; k < ctx->K; ++k) per_module[k] = ctx->mods[k].P;
    return DDG_OK;
}

ddg_status ddg_get_weights(ddg_ctx *ctx, float *dst, size_t n, int on_device) {
    if (!ctx || !dst || n != ctx->P) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    ddg_status st = sync_all(ctx);
    if (st != DDG_OK) return st;
    for (auto &m : ctx->mods)
        CU(cudaMemcpy(dst + m.p_off_global, m.w, m.P * 4, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost));
    if (on_device) CU(cudaDeviceSynchronize());
    return DDG_OK;
}

ddg_status ddg_set_weights(ddg_ctx *ctx, const float *src, size_t n, int on_device) {
    if (!ctx || !src || n != ctx->P) return DDG_ERR_INVALID_ARG;
    if (ctx->broken || ctx->t != 0) { if (ctx) set_err(ctx, "ddg_set_weights is only allowed before the first step"); return DDG_ERR_STATE; }
    ddg_status st = sync_all(ctx);
    if (st != DDG_OK) return st;
    for (auto &m : ctx->mods) {
        CU(cudaMemcpy(m.w, src + m.p_off_global, m.P * 4, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice));
        CU(cudaMemset(m.v, 0, m.P * 4));
        if (m.m2) CU(cudaMemset(m.m2, 0, m.P * 4));
    }
    CU(cudaDeviceSynchronize());  // default-stream copies and memsets are not ordered against the module streams
    for (auto &m : ctx->mods) { launch_cast(ctx->prec, m.w, m.wver, m.P, m.stream); pack_module(ctx, m, 0); }
    CU(cudaGetLastError());
    return sync_all(ctx);
}

ddg_status ddg_get_grads(ddg_ctx *ctx, int k, float *dst, size_t n, int on_device, long *sample) {
    if (!ctx || !dst || k < 0 || k >= ctx->K || n != ctx->mods[k].P) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    ddg_status st = sync_all(ctx);
    if (st != DDG_OK) return st;
    Module &m = ctx->mods[k];
    if (sample) *sample = m.last_sample;
    if (m.last_sample < 0) {
        if (on_device) { CU(cudaMemset(dst, 0, n * 4)); CU(cudaDeviceSynchronize()); } else memset(dst, 0, n * 4);
        return DDG_OK;
    }
    CU(cudaMemcpy(dst, m.g, n * 4, on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyDeviceToHost));
    if (on_device) CU(cudaDeviceSynchronize());
    return DDG_OK;
}

ddg_status ddg_get_loss_dev(ddg_ctx *ctx, const float **loss_dev) {
    if (!ctx || !loss_dev) return DDG_ERR_INVALID_ARG;
    *loss_dev = ctx->loss_dev;
    return DDG_OK;
}

ddg_status ddg_piece_times(ddg_ctx *ctx, float *fwd_ms, float *bwd_ms) {
    if (!ctx || !fwd_ms || !bwd_ms) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    if (!ctx->cfg.time_pieces || ctx->t == 0) {
        set_err(ctx, "ddg_piece_times needs a context created with time_pieces and at least one iteration");
        return DDG_ERR_INVALID_ARG;
    }
    ddg_status st = sync_all(ctx);
    if (st != DDG_OK) return st;
    for (int k = 0; k < ctx->K; ++k) {
        Module &m = ctx->mods[k];
        CU(cudaEventElapsedTime(&fwd_ms[k], m.ev_time[0], m.ev_time[1]));
        CU(cudaEventElapsedTime(&bwd_ms[k], m.ev_time[2], m.ev_time[3]));
    }
    return DDG_OK;
}

ddg_status ddg_last_step_launches(const ddg_ctx *ctx, long *launches) {
    if (!ctx || !launches) return DDG_ERR_INVALID_ARG;
    *launches = ctx->launches;
    return DDG_OK;
}

// ---- checkpoint / resume -------------------------------------------------------------------------------------
namespace {
struct StateHeader {
    unsigned long long magic;
    int version, K, n_layers, prec, B, opt_kind, classes, pad_;
    unsigned long long P, body_bytes;
    long t;
};
constexpr unsigned long long kStateMagic = 0x4444475f53544154ull;  // "DDG_STAT"

// every device buffer that carries state from one iteration to the next, in a fixed order
void state_regions(ddg_ctx *c, std::vector<std::pair<void *, size_t>> *out) {
    const size_t es = elem_size(c->prec);
    for (auto &m : c->mods) {
        const size_t pn = m.P;
        out->push_back({m.w, pn * 4}); out->push_back({m.v, pn * 4}); out->push_back({m.g, pn * 4});
        if (m.m2) out->push_back({m.m2, pn * 4});
        out->push_back({m.wver, pn * es * m.R});
        out->push_back({m.arena, m.arena_bytes * m.R});
        if (m.packed) out->push_back({m.packed, m.packed_bytes * m.R});
        for (char *d : m.delta_out) if (d) out->push_back({d, m.delta_bytes});
        out->push_back({m.stamps, (3 + 2 * (size_t)m.R + 2) * sizeof(long long)});
    }
    out->push_back({c->loss_dev, 4});
}
size_t state_body_bytes(ddg_ctx *c) {
    std::vector<std::pair<void *, size_t>> r;
    state_regions(c, &r);
    size_t n = (size_t)c->K * sizeof(long);  // last_sample per module
    for (auto &p : r) n += p.second;
    return n;
}
}  // namespace

ddg_status ddg_state_bytes(const ddg_ctx *ctx, size_t *bytes) {
    if (!ctx || !bytes) return DDG_ERR_INVALID_ARG;
    *bytes = sizeof(StateHeader) + state_body_bytes(const_cast<ddg_ctx *>(ctx));
    return DDG_OK;
}

ddg_status ddg_save_state(ddg_ctx *ctx, void *dst_host, size_t bytes) {
    if (!ctx || !dst_host) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    const size_t body = state_body_bytes(ctx);
    if (bytes != sizeof(StateHeader) + body) { set_err(ctx, "ddg_save_state: buffer size does not match ddg_state_bytes"); return DDG_ERR_INVALID_ARG; }
    ddg_status st = sync_all(ctx);
    if (st != DDG_OK) return st;
    StateHeader h{};
    h.magic = kStateMagic; h.version = 1; h.K = ctx->K; h.n_layers = ctx->n_layers; h.prec = ctx->prec; h.B = ctx->B;
    h.opt_kind = ctx->opt.kind; h.classes = ctx->classes; h.P = ctx->P; h.body_bytes = body; h.t = ctx->t;
    char *p = static_cast<char *>(dst_host);
    memcpy(p, &h, sizeof(h)); p += sizeof(h);
    for (auto &m : ctx->mods) { memcpy(p, &m.last_sample, sizeof(long)); p += sizeof(long); }
    std::vector<std::pair<void *, size_t>> r;
    state_regions(ctx, &r);
    for (auto &q : r) { CU(cudaMemcpy(p, q.first, q.second, cudaMemcpyDeviceToHost)); p += q.second; }
    return DDG_OK;
}

ddg_status ddg_load_state(ddg_ctx *ctx, const void *src_host, size_t bytes) {
    if (!ctx || !src_host || bytes < sizeof(StateHeader)) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    StateHeader h;
    memcpy(&h, src_host, sizeof(h));
    const size_t body = state_body_bytes(ctx);
    if (h.magic != kStateMagic || h.version != 1 || h.K != ctx->K || h.n_layers != ctx->n_layers || h.prec != ctx->prec ||
        h.B != ctx->B || h.opt_kind != ctx->opt.kind || h.classes != ctx->classes || h.P != ctx->P || h.body_bytes != body ||
        bytes != sizeof(StateHeader) + body || h.t < 0) {
        set_err(ctx, "ddg_load_state: the checkpoint was not written by a context of this shape");
        return DDG_ERR_INVALID_ARG;
    }
    ddg_status st = sync_all(ctx);
    if (st != DDG_OK) return st;
    const char *p = static_cast<const char *>(src_host) + sizeof(h);
    for (auto &m : ctx->mods) { memcpy(&m.last_sample, p, sizeof(long)); p += sizeof(long); m.dyn_valid = false; }
    std::vector<std::pair<void *, size_t>> r;
    state_regions(ctx, &r);
    for (auto &q : r) { CU(cudaMemcpy(q.first, p, q.second, cudaMemcpyHostToDevice)); p += q.second; }
    CU(cudaDeviceSynchronize());  // the copies ran on the default stream; the module streams do not wait for it
    ctx->t = h.t;
    ctx->loss_pending = -1;  // a read-back enqueued before the restore belongs to the run that was replaced
    return DDG_OK;
}

ddg_status ddg_debug_wait_timeout(ddg_ctx *ctx, unsigned polls) {
    if (!ctx || polls == 0) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    if (launch_wait_probe(polls, ctx->lx(ctx->mods[0].stream)) < 0) {
        set_err(ctx, "ddg_debug_wait_timeout: the tensor-core path is not initialised");
        return DDG_ERR_CUDA;
    }
    CU(cudaGetLastError());
    return DDG_OK;
}

ddg_status ddg_debug_shift_stamps(ddg_ctx *ctx, int k, long delta) {
    if (!ctx || k < 0 || k >= ctx->K) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    if (!ctx->cfg.debug_checks) { set_err(ctx, "ddg_debug_shift_stamps: the context was created without debug_checks"); return DDG_ERR_STATE; }
    launch_add_to_counter(ctx->mods[k].fcount(), (long long)delta, ctx->lx(ctx->mods[k].stream));
    CU(cudaGetLastError());
    return DDG_OK;
}

ddg_status ddg_sync(ddg_ctx *ctx) {
    if (!ctx) return DDG_ERR_INVALID_ARG;
    if (ctx->broken) return DDG_ERR_STATE;
    ddg_status st = sync_all(ctx);
    if (st != DDG_OK) return st;
    CU(cudaGetLastError());
    return DDG_OK;
}

}  // extern "C"
