// Tensor-core 3x3 convolution for bf16 NHWC tensors on sm_100a: implicit GEMM on tcgen05 with TMEM accumulators,
// the im2col operand streamed by TMA (one shifted, zero-filled box per filter tap), the filter resident in shared
// memory for the life of a persistent CTA.
//
//   forward  y[p][co]  = sum_{tap,ci} x[p + tap][ci]  * w[co][ci][tap]
//   dgrad    dx[p][ci] = sum_{tap,co} dy[p + tap][co] * w[co][ci][8 - tap]     (stride 1: the same kernel, filter flipped)
//
// One CTA tile is 128 consecutive output pixels (whole image rows) x C channels.  The input rows are loaded ONCE per
// tile, unshifted in the column direction: the MMAs produce, per filter column kx, the partial result
// P_kx[p][co] = sum_{ky,ci} x[p + (ky-1) rows][ci] * w[co][ci][ky][kx] at the INPUT column (UMMA M=128, N=3C, K=16 per
// instruction, the three filter columns stacked along N, chunk of 16 output channels by chunk), and the epilogue adds the three partials across
// neighbouring pixels, y[h][w] = P_0[h][w-1] + P_1[h][w] + P_2[h][w+1], with warp shuffles (a warp holds whole image
// rows; the image border contributes zero).  The filter-row shift costs nothing: the three rows read the same TMA box
// at offsets of 0, W and 2W pixels, which are whole swizzle periods, so only the descriptor start address moves.
// Warp roles: a CTA runs P independent pipelines (1, 2 or 4) over interleaved tiles, each with its own TMA-issuing
// warp (warps 0..P-1), MMA-issuing warp (warps P..2P-1), share of the stage ring and TMEM accumulators; the remaining
// warps are epilogue groups of four (one warp per TMEM lane quarter) that drain TMEM, combine, add the shortcut gradient
// where asked, convert to bf16 and store, shared out among the pipelines as EpiPlan says.  Why several pipelines: the
// cost of a tile is the chain of barrier hand-offs and tcgen05 instruction issue of its single MMA thread (150-200
// cycles per operation, a thousand and more per tile), not data movement, tensor-core or epilogue time (removing the
// stores, the shuffles and two of the three TMEM loads of the epilogue changes the kernel's time by under 10 %), so
// chains side by side raise the tile rate of an SM.  Every mbarrier wait is bounded: when one runs out, the CTA raises
// an error word that the host reads at its next sync point, and leaves.
#include <cstdlib>
#include <map>
#include <mutex>
#include <tuple>

#include "common.cuh"
#include "conv_tc.h"
#include "tc_common.cuh"

namespace ddg {

namespace {

constexpr int kTcMaxThreads = 768;  // convolution: at most four pipelines (TMA warp, MMA warp, four epilogue warps each)
constexpr int kS2Threads = 320;   // stride-2 convolution: TMA warp, MMA warp, two groups of four epilogue warps
constexpr int kWgThreads = 192;   // weight gradient: TMA warp, MMA warp, four epilogue warps

__device__ int g_tc_error = 0;  // 0 = fine; otherwise the code of the wait that ran out

// Shared-memory plan of the convolution kernel (all offsets from a 1024-byte aligned base).
struct ConvSmem {
    uint32_t w_off, a_off, tail_off;
};
template <int C> __host__ __device__ inline ConvSmem conv_smem_plan(int n_stages, int stage_bytes) {
    ConvSmem p;
    p.w_off = 0;
    p.a_off = (TcCfg<C>::w_bytes + 1023u) & ~1023u;
    p.tail_off = p.a_off + (uint32_t)n_stages * (uint32_t)stage_bytes;
    return p;
}
// after the pipeline stages: 512 bytes of barriers and flags, 8 KB of per-warp batch-norm sums (up to 16 epilogue
// warps x 4 channel chunks x 32 lanes), 512 bytes of per-channel mean / invstd, 512 bytes of per-channel scale / shift
// of the input transform
constexpr int kTailBytes = 512 + 8192 + 512 + 512;
template <int C> inline size_t conv_smem_bytes(int n_stages, int stage_bytes) {
    return 1024 + conv_smem_plan<C>(n_stages, stage_bytes).tail_off + kTailBytes;
}

// Sum of v[i] over the 32 lanes of a warp for 32 values at once: after the call lane l holds the total of v[l] in
// v[0].  Each step halves the values a lane keeps (31 shuffles in all instead of 32 x 5).
__device__ __forceinline__ void warp_transpose_sum32(float (&v)[32], int lane) {
#pragma unroll
    for (int step = 16; step >= 1; step >>= 1) {
        const bool upper = (lane & step) != 0;
#pragma unroll
        for (int i = 0; i < step; ++i) {
            const float send = upper ? v[i] : v[i + step];
            const float keep = upper ? v[i + step] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, step);
        }
    }
}

// Filter images for the tensor-core kernels: per convolution two blocks of 3 swizzled K-major [3C][C] bf16 tiles (one
// per filter row; rows = filter column x channel of this pass, k = contraction channel): the forward one (row =
// output channel, k = input channel) and the input-gradient one (row = input channel, k = output channel, taps
// flipped).  One thread per (tap, row, k).
struct PackJob { long src_off; long dst_off; int C; int first_elem; int cin_real; int pad_; };

// image element (tap = ky*3+kx, row r, k): filter row tile ky; within it the rows (= accumulator columns) are ordered
// (16-channel chunk of r, kx, r mod 16), so that the three filter-column partials of a chunk are 48 consecutive
// accumulator columns and the epilogue fetches them with two TMEM loads
template <int C> __device__ __forceinline__ uint32_t w_img_off(int tap, int r, int k) {
    return (uint32_t)(tap / 3) * TcCfg<C>::w_row_tile_bytes + swz_off<C>((r >> 4) * 48 + (tap % 3) * 16 + (r & 15), k);
}
// cin: input channels the canonical filter really has; channels cin..C-1 of the images are zero (a first layer whose
// input was zero-padded to C channels)
template <int C> __device__ __forceinline__ void pack_one(const bf16 *w, uint8_t *dst, int i, int cin) {
    const int tap = i / (C * C), r = (i / C) % C, k = i % C;
    const uint32_t o = w_img_off<C>(tap, r, k);
    const bf16 zero = __float2bfloat16_rn(0.f);
    *reinterpret_cast<bf16 *>(dst + o) = k < cin ? w[(size_t)(r * cin + k) * 9 + tap] : zero;
    *reinterpret_cast<bf16 *>(dst + TcCfg<C>::w_bytes + o) = r < cin ? w[(size_t)(k * cin + r) * 9 + (8 - tap)] : zero;
}

// filter images of a stride-2 convolution with Ci input channels (Co = 2 Ci): nine [Co][Ci] K-major tiles for the forward
// pass, then nine [Ci][Co] K-major tiles for the input gradient; tile index = ky*3+kx in both
template <int CI> struct S2Cfg {
    static constexpr int CO = 2 * CI;
    static constexpr int tap_bytes = CO * CI * 2;
    static constexpr int img_bytes = 9 * tap_bytes;
};
template <int CI> __device__ __forceinline__ void pack_s2_one(const bf16 *w, uint8_t *dst, int i) {
    constexpr int CO = 2 * CI;
    const int tap = i / (CO * CI), co = (i / CI) % CO, ci = i % CI;
    const bf16 v = w[(size_t)(co * CI + ci) * 9 + tap];
    *reinterpret_cast<bf16 *>(dst + tap * S2Cfg<CI>::tap_bytes + swz_off<CI>(co, ci)) = v;
    *reinterpret_cast<bf16 *>(dst + S2Cfg<CI>::img_bytes + tap * S2Cfg<CI>::tap_bytes + swz_off<CO>(ci, co)) = v;
}

__global__ void pack_filters_kernel(const bf16 *__restrict__ wver, uint8_t *__restrict__ packed,
                                    const PackJob *__restrict__ jobs, int n_jobs, int total) {
    pdl_launch();
    pdl_wait();
    const int e = blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= total) return;
    int lo = 0, hi = n_jobs - 1;  // last job whose first element is <= e
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (jobs[mid].first_elem <= e) lo = mid; else hi = mid - 1;
    }
    const PackJob j = jobs[lo];
    const int i = e - j.first_elem;
    if (j.pad_ == 1) {  // stride-2 convolution with C input channels
        if (j.C == 16) pack_s2_one<16>(wver + j.src_off, packed + j.dst_off, i);
        else pack_s2_one<32>(wver + j.src_off, packed + j.dst_off, i);
        return;
    }
    if (j.C == 16) pack_one<16>(wver + j.src_off, packed + j.dst_off, i, j.cin_real);
    else if (j.C == 32) pack_one<32>(wver + j.src_off, packed + j.dst_off, i, j.cin_real);
    else pack_one<64>(wver + j.src_off, packed + j.dst_off, i, j.cin_real);
}

// the same for one convolution, job passed by value
__global__ void pack_one_filter_kernel(const bf16 *__restrict__ w, uint8_t *__restrict__ packed, int C) {
    pdl_launch();
    pdl_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= 9 * C * C) return;
    if (C == 16) pack_one<16>(w, packed, i, C);
    else if (C == 32) pack_one<32>(w, packed, i, C);
    else pack_one<64>(w, packed, i, C);
}

// ---------------------------------------------------------------------------------------------------------
// forward / input gradient.
//   slab == 1 (tile inside one image): one TMA box of (rows+2) image rows per tile; filter row ky reads it at an offset
//              of ky*W pixels.
//   slab == 0 (tile = several whole small images): one TMA box of the tile shifted by ky-1 rows per filter row (3 per
//              tile), zero-filled at the image border.
// ---------------------------------------------------------------------------------------------------------
// How the epilogue warp groups (four warps each, one per TMEM lane quarter; the warps after the 2 * n_pipes issuing
// warps) share the tiles of a pipeline.  A pipeline numbers its tiles it = 0, 1, ...; tile `it` accumulates in the
// pipeline's accumulator it % n_acc and is drained by the `split` groups of slot it % n_slots, each of which takes an
// equal share of the tile's 16-channel chunks.
//   n_slots = 2, split = 1: two groups take alternate tiles (the epilogue of one overlaps the next one's);
//   n_slots = 1, split = 2: two groups halve every tile (shorter epilogue where a CTA has one or two tiles).
struct EpiPlan { int n_pipes, n_acc, n_slots, split; };

// (bound of 768 threads: caps the kernel at 80 registers, so that two 384-thread CTAs of different streams share an SM)
template <int C>
__global__ void __launch_bounds__(768, 1)
conv3x3_tc_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap_res,
                  const bf16 *__restrict__ w, const uint8_t *__restrict__ w_packed,
                  bf16 *__restrict__ dst, int dgrad, int H, int W, int rows_per_tile, int imgs_per_tile, int n_tiles,
                  int slab, int n_stages, int stage_bytes, int tmem_cols, EpiPlan plan_e, const bf16 *__restrict__ res_dout,
                  const bf16 *__restrict__ res_out, float *__restrict__ stat_part, unsigned *__restrict__ stat_counter,
                  float *__restrict__ stat_o0, float *__restrict__ stat_o1, const bf16 *__restrict__ bn_mask,
                  const bf16 *__restrict__ bn_x, const float *__restrict__ bn_mean, const float *__restrict__ bn_invstd,
                  const bf16 *__restrict__ xf_gamma, const bf16 *__restrict__ xf_beta, const float *__restrict__ xf_mean,
                  const float *__restrict__ xf_invstd, bf16 *__restrict__ xf_out, int xf_res, int xf_warps, int *__restrict__ err_word) {
    // xf_gamma != nullptr (forward only): the source tensor is the raw output y of the previous convolution and this
    // kernel applies that convolution's batch norm and ReLU on its own operand path: xf_warps transform warps per pipeline
    // turn every TMA box, in place in shared memory, into a = relu(y * scale + shift) (scale = gamma * invstd, shift =
    // beta - mean * scale; rows outside the image stay zero: they are the convolution's padding), store the tile's own
    // rows of a to xf_out (the backward sweep reads them) and only then hand the stage to the MMA warp.  xf_res != 0: the
    // batch norm closes a residual block, a = relu(y * scale + shift + res): the stage holds a second box, fetched through
    // tmap_res with the same coordinates, right behind the first.
    // stat_part != nullptr: the epilogue also reduces, per channel over the pixels of this CTA's tiles, the two sums the
    // batch norm that follows needs, from the values as stored (rounded to bf16), writes them to
    // stat_part[blockIdx.x][2C], and the CTA that finishes last adds the partials in a fixed order:
    //   bn_x == nullptr: (sum y, sum y^2) -> stat_o0 = mean, stat_o1 = 1/sqrt(var + eps) (forward statistics);
    //   otherwise (sum dz, sum dz * xhat) with dz = result * [bn_mask > 0], xhat = (bn_x - mean) * invstd -> stat_o0 =
    //   dbeta, stat_o1 = dgamma: the sums of the batch-norm backward whose incoming gradient this kernel produces.
    typedef TcCfg<C> Cfg;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const ConvSmem plan = conv_smem_plan<C>(n_stages, stage_bytes);
    const uint32_t w_base = base + plan.w_off, a_base = base + plan.a_off;
    uint8_t *tail = smem + plan.tail_off;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tail);  // full[16], empty[16], tfull[4], tempty[4], wbar, raw[16]
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(tail + (3 * kMaxStages + 9) * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tail + (3 * kMaxStages + 9) * 8 + 8);
    const Waiter wt{abort_flag, err_word, kSpinLimit};
    float (*sm_run)[4][32] = reinterpret_cast<float (*)[4][32]>(tail + 512);  // [epilogue warp][channel chunk][lane]
    float *sm_stat = reinterpret_cast<float *>(tail + 512 + 8192);            // mean[C], invstd[C]
    float *sm_xf = reinterpret_cast<float *>(tail + 512 + 8192 + 512);        // scale[C], shift[C] of the input transform
    const bool xform = xf_gamma != nullptr;
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + 4 + a); };
    const uint32_t w_bar = bar0 + 8u * (2 * kMaxStages + 8);
    auto raw_bar = [&](int s) { return bar0 + 8u * (2 * kMaxStages + 9 + s); };  // box landed, not yet transformed

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (stat_part != nullptr)
        for (int i = threadIdx.x; i < 16 * 4 * 32; i += blockDim.x) (&sm_run[0][0][0])[i] = 0.f;
    if (threadIdx.x == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmap) : "memory");  // the first TMA would otherwise wait for its descriptor
        // with the input transform a stage is full once each of the pipeline's transform warps has arrived
        for (int s = 0; s < n_stages; ++s) { mbar_init(full_bar(s), xform ? xf_warps : 1); mbar_init(empty_bar(s), 1); mbar_init(raw_bar(s), 1); }
        for (int a = 0; a < 4; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4 * plan_e.split); }
        mbar_init(w_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {  // TMEM allocation is a whole-warp operation; the same warp frees it at the end
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // launch latency, barrier set-up and the TMEM allocation above overlap the previous kernel's tail; nothing before
    // this point touches global memory
    pdl_launch();
    pdl_wait();
    if (bn_x != nullptr && threadIdx.x < 2 * C)
        sm_stat[threadIdx.x] = threadIdx.x < C ? bn_mean[threadIdx.x] : bn_invstd[threadIdx.x - C];
    if (xform && threadIdx.x < C) {  // the same two constants, computed the same way, as the element-wise batch-norm pass
        const float sc = to_f(xf_gamma[threadIdx.x]) * xf_invstd[threadIdx.x];
        sm_xf[threadIdx.x] = sc;
        sm_xf[C + threadIdx.x] = to_f(xf_beta[threadIdx.x]) - xf_mean[threadIdx.x] * sc;
    }
    if (w_packed == nullptr) {
        // filter in canonical order: stage it here as 9 K-major [C rows = output channel of this pass][C] tiles
        for (int i = threadIdx.x; i < 9 * C * C; i += blockDim.x) {
            const int tap = i / (C * C), r = (i / C) % C, k = i % C;
            const size_t g = dgrad ? ((size_t)(k * C + r) * 9 + (8 - tap)) : ((size_t)(r * C + k) * 9 + tap);
            *reinterpret_cast<bf16 *>(smem + plan.w_off + w_img_off<C>(tap, r, k)) = w[g];
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const int tiles_per_img = H / rows_per_tile;  // tiles per image when a tile lies inside one image
    const int loads_per_tile = slab ? 1 : 3;

    // pipeline g owns stages [g*ring, (g+1)*ring) and takes every tile_step-th tile
    const int n_pipes = plan_e.n_pipes;
    const int ring = n_stages / n_pipes;
    const int tile_step = n_pipes * gridDim.x;
    const int n_epi_groups_plan = n_pipes * plan_e.n_slots * plan_e.split;
    const int n_epi_groups = n_epi_groups_plan < 2 ? 2 : n_epi_groups_plan;  // warps launched for the epilogue: 4 per group
    if (warp < n_pipes) {
        // ---------------- TMA producers ----------------
        const int g = warp;
        if (lane == 0) {
            if (g == 0 && w_packed != nullptr) {  // pre-arranged filter image: one bulk copy
                mbar_expect_tx(w_bar, Cfg::w_bytes);
                bulk_copy_g2s(w_base, w_packed + (dgrad ? Cfg::w_bytes : 0), Cfg::w_bytes, w_bar);
            }
            int ls = 0;
            uint32_t ph = 0;
            bool ok = true;
            // tile -> (first image, first row): divided once, then stepped (an integer division per tile is a hundred
            // cycles of this thread's chain)
            const int tile0 = blockIdx.x + g * gridDim.x;
            const int step_n = tile_step / tiles_per_img, step_t = tile_step % tiles_per_img;
            int n_img = tile0 / tiles_per_img, t_img = tile0 % tiles_per_img;
            for (int tile = tile0; tile < n_tiles && ok; tile += tile_step) {
                int n0, h0;
                if (imgs_per_tile > 1) { n0 = tile * imgs_per_tile; h0 = 0; }  // a tile spans whole images
                else { n0 = n_img; h0 = t_img * rows_per_tile; }
                n_img += step_n; t_img += step_t;
                if (t_img >= tiles_per_img) { t_img -= tiles_per_img; ++n_img; }
                for (int j = 0; j < loads_per_tile && ok; ++j) {
                    const int s = g * ring + ls;
                    ok = mbar_wait(empty_bar(s), ph ^ 1u, wt, 1);
                    if (!ok) break;
                    const uint32_t land = xform ? raw_bar(s) : full_bar(s);
                    mbar_expect_tx(land, (uint32_t)stage_bytes);
                    tma_load_4d(a_base + s * stage_bytes, &tmap, land, 0, 0, slab ? h0 - 1 : h0 + j - 1, n0);
                    if (xf_res)  // the residual's box behind it (a stage is then two boxes)
                        tma_load_4d(a_base + s * stage_bytes + stage_bytes / 2, &tmap_res, land, 0, 0, slab ? h0 - 1 : h0 + j - 1, n0);
                    if (++ls == ring) { ls = 0; ph ^= 1u; }
                }
            }
            if (!ok) {  // let copies already in flight land before the CTA can exit
                for (int i = 0; i < 2000; ++i) __nanosleep(100);
            }
        }
    } else if (warp < 2 * n_pipes) {
        // ---------------- MMA issuers ----------------
        const int g = warp - n_pipes;
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((3 * C) >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
            int ls = 0, it = 0;
            uint32_t ph = 0;
            bool ok = true;
            if (w_packed != nullptr) ok = mbar_wait(w_bar, 0, wt, 5);
            int acc_i = 0;        // it % n_acc and the parity of it / n_acc, stepped instead of divided
            uint32_t aph = 0;
            for (int tile = blockIdx.x + g * gridDim.x; tile < n_tiles && ok; tile += tile_step, ++it) {
                // the pipeline's accumulators in turn
                const int a = g * plan_e.n_acc + acc_i;
                ok = mbar_wait(tempty_bar(a), aph ^ 1u, wt, 2);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * 3 * C);
                for (int j = 0; j < loads_per_tile && ok; ++j) {
                    const int s = g * ring + ls;
                    ok = mbar_wait(full_bar(s), ph, wt, 3);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t a_addr = a_base + s * stage_bytes;
                    const int n_sub = slab ? 3 : 1;
                    for (int i = 0; i < n_sub; ++i) {
                        const int ky = slab ? i : j;
                        const uint64_t adesc = make_desc(a_addr + (uint32_t)(i * W) * Cfg::row_bytes, 8 * Cfg::row_bytes, Cfg::layout);
                        const uint64_t bdesc = make_desc(w_base + ky * Cfg::w_row_tile_bytes, 8 * Cfg::row_bytes, Cfg::layout);
#pragma unroll
                        for (int k = 0; k < C / 16; ++k)  // 16 channels = 32 bytes further along the contraction axis
                            tc_mma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (ky | k) != 0);
                    }
                    tc_commit(empty_bar(s));  // the stage is free once these MMAs have read it
                    if (++ls == ring) { ls = 0; ph ^= 1u; }
                }
                if (ok) tc_commit(tfull_bar(a));
                if (++acc_i == plan_e.n_acc) { acc_i = 0; aph ^= 1u; }
            }
        }
    } else if (xform && warp >= 2 * n_pipes + 4 * n_epi_groups) {
        // ---------------- input transform: raw box -> relu(batch norm) in place, the tile's own rows also to global ------
        const int tw = warp - 2 * n_pipes - 4 * n_epi_groups;
        const int g = tw / xf_warps, t128 = 32 * (tw % xf_warps) + lane;  // pipeline, thread among its transform threads
        const int xf_threads = 32 * xf_warps;
        constexpr int kCg = C / 8;                            // 16-byte cells (8 channels) per pixel
        const int box_rows_img = slab ? rows_per_tile + 2 : rows_per_tile;  // image rows of a box, per image
        const int n_pix = box_rows_img * imgs_per_tile * W;
        // W and (image-pair tiles) H are powers of two; a thread keeps its cell of the pixel (the thread count is a
        // multiple of the cells per pixel) and walks the pixels
        const int log_w = 31 - __clz(W), log_h = 31 - __clz(H);
        const int cg = t128 % kCg, p_first = t128 / kCg, p_step = xf_threads / kCg;
        float sc[8], sh[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) { sc[k] = sm_xf[8 * cg + k]; sh[k] = sm_xf[C + 8 * cg + k]; }
        int ls = 0;
        uint32_t ph = 0;
        bool ok = g < n_pipes;
        for (int tile = blockIdx.x + g * gridDim.x; tile < n_tiles && ok; tile += tile_step) {
            int n0, h0;
            if (imgs_per_tile > 1) { n0 = tile * imgs_per_tile; h0 = 0; }
            else { n0 = tile / tiles_per_img; h0 = (tile % tiles_per_img) * rows_per_tile; }
            for (int j = 0; j < loads_per_tile && ok; ++j) {
                const int s = g * ring + ls;
                ok = mbar_wait(raw_bar(s), ph, wt, 6);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                uint8_t *stage = smem + plan.a_off + (size_t)s * stage_bytes;
                const int row_first = slab ? h0 - 1 : j - 1;   // image row of the box's first row
                const bool owns = slab || j == 1;              // the unshifted box holds the tile's own pixels
                constexpr int U = 2;                           // cells in flight per thread
                for (int pb = p_first; pb < n_pix; pb += U * p_step) {
                    uint4 q[U], rr[U];
                    int hh[U];
                    uint32_t off[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        const int p = pb + u * p_step;
                        const int r = slab ? (p >> log_w) : ((p >> log_w) & (H - 1));
                        hh[u] = (p < n_pix) ? row_first + r : -1;   // -1: nothing to do (past the box, or padding)
                        if (hh[u] >= H) hh[u] = -1;
                        off[u] = swz_off<C>(p, 8 * cg);
                        if (hh[u] >= 0) {
                            q[u] = *reinterpret_cast<const uint4 *>(stage + off[u]);
                            if (xf_res) rr[u] = *reinterpret_cast<const uint4 *>(stage + stage_bytes / 2 + off[u]);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < U; ++u) {
                        if (hh[u] < 0) continue;               // padding rows: the zero fill stays
                        const uint32_t wq[4] = {q[u].x, q[u].y, q[u].z, q[u].w};
                        const uint32_t rq[4] = {rr[u].x, rr[u].y, rr[u].z, rr[u].w};
                        uint32_t o[4];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            float a = fmaf(__uint_as_float(wq[k] << 16), sc[2 * k], sh[2 * k]);
                            float b = fmaf(__uint_as_float(wq[k] & 0xffff0000u), sc[2 * k + 1], sh[2 * k + 1]);
                            if (xf_res) { a += __uint_as_float(rq[k] << 16); b += __uint_as_float(rq[k] & 0xffff0000u); }
                            a = a > 0.f ? a : 0.f;
                            b = b > 0.f ? b : 0.f;
                            const __nv_bfloat162 h2 = __floats2bfloat162_rn(a, b);
                            o[k] = *reinterpret_cast<const uint32_t *>(&h2);
                        }
                        const uint4 res = make_uint4(o[0], o[1], o[2], o[3]);
                        *reinterpret_cast<uint4 *>(stage + off[u]) = res;
                        const int p = pb + u * p_step;
                        const int r = slab ? (p >> log_w) : ((p >> log_w) & (H - 1));
                        if (owns && (!slab || (r >= 1 && r <= rows_per_tile))) {
                            const int img = slab ? 0 : (p >> (log_w + log_h));
                            const size_t pix = ((size_t)(n0 + img) * H + hh[u]) * W + (p & (W - 1));
                            *reinterpret_cast<uint4 *>(xf_out + pix * C + 8 * cg) = res;
                        }
                    }
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
                __syncwarp();
                if (lane == 0) mbar_arrive(full_bar(s));
                if (++ls == ring) { ls = 0; ph ^= 1u; }
            }
        }
    } else if (warp < 2 * n_pipes + 4 * n_epi_groups) {
        // ---------------- epilogue: TMEM -> registers -> bf16 -> global ----------------
        const int q = warp & 3;  // a warp may only touch TMEM lanes [32*(warp%4), +32)
        const int ew = warp - 2 * n_pipes;  // index among the epilogue warps
        const int grp = ew >> 2;
        const int per_pipe = plan_e.n_slots * plan_e.split;
        const int pipe = grp / per_pipe, slot = (grp % per_pipe) / plan_e.split, share = grp % plan_e.split;
        constexpr int kChunks = C / 16;
        const int c_begin = 16 * (share * kChunks / plan_e.split), c_end = 16 * ((share + 1) * kChunks / plan_e.split);
        bool ok = pipe < n_pipes;  // a group the plan has no work for leaves at once
        const int wcol = lane % W;  // W divides 32: a warp holds whole image rows
        int acc_i = slot % plan_e.n_acc;                       // it % n_acc and the parity of it / n_acc, stepped
        uint32_t aph = (uint32_t)(slot / plan_e.n_acc) & 1u;
        int tile = blockIdx.x + pipe * gridDim.x + slot * tile_step;
        const int tile_stride = plan_e.n_slots * tile_step;
        for (; ok; tile += tile_stride) {
            if (tile >= n_tiles) break;
            const int a = pipe * plan_e.n_acc + acc_i;
            const uint32_t aph_now = aph;
            acc_i += plan_e.n_slots;
            while (acc_i >= plan_e.n_acc) { acc_i -= plan_e.n_acc; aph ^= 1u; }
            const size_t pix = (size_t)tile * kTileM + 32 * q + lane;
            // what the epilogue reads from global memory for this pixel (shortcut gradient, batch-norm mask and input) was
            // written long ago: start fetching it now, under the TMA and MMA latency of the tile
            if (res_dout != nullptr) {
#pragma unroll
                for (int o = 0; o < C * 2; o += 128) {
                    prefetch_l1(reinterpret_cast<const char *>(res_dout + pix * C) + o);
                    prefetch_l1(reinterpret_cast<const char *>(res_out + pix * C) + o);
                }
            }
            if (bn_x != nullptr) {
#pragma unroll
                for (int o = 0; o < C * 2; o += 128) {
                    prefetch_l1(reinterpret_cast<const char *>(bn_mask + pix * C) + o);
                    prefetch_l1(reinterpret_cast<const char *>(bn_x + pix * C) + o);
                }
            }
            ok = mbar_wait(tfull_bar(a), aph_now, wt, 4);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(a * 3 * C);
#pragma unroll 1
            for (int c0 = c_begin; c0 < c_end; c0 += 16) {
                float p0[16], p1[16], p2[16];
                // p0: filter column 0, belongs to the pixel on the right; p2: filter column 2, to the pixel on the left
                tc_ld32(t_row + (uint32_t)(3 * c0), p0, p1);  // the chunk's three pieces are 48 consecutive columns
                tc_ld16(t_row + (uint32_t)(3 * c0) + 32u, p2);
                tc_wait_ld();
                if (c0 + 16 >= c_end) {  // this group's last read of the accumulator: hand it back to the MMA warp
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(a));
                }
                float acc[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const float left = __shfl_up_sync(0xffffffffu, p0[j], 1);
                    const float right = __shfl_down_sync(0xffffffffu, p2[j], 1);
                    acc[j] = p1[j] + (wcol > 0 ? left : 0.f) + (wcol < W - 1 ? right : 0.f);
                }
                if (res_dout != nullptr) {  // identity-shortcut gradient: + dout * [out > 0]
                    float d[16], o[16];
                    ld_global_32(res_dout + pix * C + c0, d);
                    ld_global_32(res_out + pix * C + c0, o);
#pragma unroll
                    for (int j = 0; j < 16; ++j) if (o[j] > 0.f) acc[j] += d[j];
                }
                {
                    uint32_t pk[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const __nv_bfloat162 b2 = __floats2bfloat162_rn(acc[2 * j], acc[2 * j + 1]);
                        pk[j] = *reinterpret_cast<const uint32_t *>(&b2);
                    }
                    st_global_32(dst + pix * C + c0, pk);
                }
                if (stat_part != nullptr) {
                    float v[32];
                    if (bn_x == nullptr) {
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            const float r = __bfloat162float(__float2bfloat16_rn(acc[j]));
                            v[j] = r;
                            v[16 + j] = r * r;
                        }
                    } else {
                        float mk[16], xv[16];
                        ld_global_32(bn_mask + pix * C + c0, mk);
                        ld_global_32(bn_x + pix * C + c0, xv);
#pragma unroll
                        for (int j = 0; j < 16; ++j) {
                            float d = __bfloat162float(__float2bfloat16_rn(acc[j]));
                            if (!(mk[j] > 0.f)) d = 0.f;
                            v[j] = d;
                            v[16 + j] = d * (xv[j] - sm_stat[c0 + j]) * sm_stat[C + c0 + j];
                        }
                    }
                    warp_transpose_sum32(v, lane);
                    sm_run[ew][c0 >> 4][lane] += v[0];  // lane l < 16: first sum of channel c0+l; else second sum
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tmem_cols)
                     : "memory");
    }
    if (stat_part == nullptr) return;
    if (threadIdx.x < 2 * C) {  // the epilogue warps' sums in a fixed order
        const int c = threadIdx.x % C, l = (c & 15) + 16 * (threadIdx.x / C);
        float t = 0.f;
#pragma unroll
        for (int wq = 0; wq < 16; ++wq) t += sm_run[wq][c >> 4][l];
        stat_part[(size_t)blockIdx.x * 2 * C + threadIdx.x] = t;
    }
    if (stat_counter == nullptr) return;  // the kernel that consumes the sums folds the partials itself
    __syncthreads();  // the partial stores above are ordered before thread 0's release below by this barrier
    int *is_last = reinterpret_cast<int *>(sm_stat);  // free again: the epilogue is over
    if (threadIdx.x == 0) {
        unsigned old;
        asm volatile("atom.add.acq_rel.gpu.global.u32 %0, [%1], 1;" : "=r"(old) : "l"(stat_counter) : "memory");
        *is_last = (old == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!*is_last) return;
    // last CTA: the partials of all CTAs, added up exactly as the element-wise passes do it (same routine, 256 threads)
    double *fold = reinterpret_cast<double *>(&sm_run[0][0][0]);  // 256 x 4 doubles = the 8 KB of the per-warp sums
    double *tot = reinterpret_cast<double *>(smem + plan.a_off);     // the stage ring is idle by now
    fold_partials<256>(stat_part, (int)gridDim.x, 2 * C, fold, tot);
    if (threadIdx.x < C) {
        const int c = threadIdx.x;
        const double a = tot[c], b = tot[C + c];
        if (bn_x == nullptr) {
            const double npix = (double)n_tiles * kTileM;
            double m = a / npix, var = b / npix - m * m;
            if (var < 0.0) var = 0.0;
            stat_o0[c] = (float)m;
            stat_o1[c] = (float)(1.0 / sqrt(var + (double)1e-5f));  // the element-wise passes' constant, bit for bit
        } else {
            stat_o0[c] = (float)a;
            stat_o1[c] = (float)b;
        }
    }
    if (threadIdx.x == 0) *stat_counter = 0u;
}

// ---------------------------------------------------------------------------------------------------------
// Weight gradient on the tensor cores:  dw[co][ci][ky][kx] = sum_p dy[p][co] * x[p + (ky-1, kx-1)][ci].
// The contraction runs over pixels, so both operands are used "MN-major": a TMA tile [pixels][C channels] is read by
// the MMA with the channel axis as its M (or N) axis and the pixel axis as K, 16 pixels per instruction.  The MMA
// shape is M=128 whatever C is: rows >= C of the accumulator are never read (their operand rows alias other rows of
// the same dy tile).  N = 3C: three filter taps stacked through the descriptor's leading-dimension offset.
//   slab == 0: grid (pixel chunks, 3 filter rows); per tile the dy box and three shifted x boxes (one per filter
//              column); the three stacked taps are the filter columns.  TMEM holds D[co][(kx, ci)].
//   slab == 1: grid (pixel chunks, 1); per tile the dy box and three x boxes of (rows+2) image rows (one per filter
//              column); the three stacked taps are the filter rows (row offsets 0, W, 2W pixels inside the box).  TMEM
//              holds all nine taps D[co][(kx, ky, ci)].
// A CTA accumulates over all of its pixel tiles in TMEM, then writes one fp32 partial; the fold kernel sums the chunks
// in a fixed order.
// ---------------------------------------------------------------------------------------------------------
constexpr int kWgMaxChunks = 148;

struct WgSmem { uint32_t tail_off; };

template <int C>
__global__ void __launch_bounds__(kWgThreads, 1)
wgrad_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_dy,
                float *__restrict__ part, int H, int W, int rows_per_tile, int imgs_per_tile, int n_tiles, int slab,
                int n_stages, int x_box_bytes, int tmem_cols, int wide, int tall, int *__restrict__ err_word) {
    typedef TcCfg<C> Cfg;
    const int stage_bytes = Cfg::tile_bytes + 3 * x_box_bytes;
    const int box_rows = rows_per_tile + 2;  // image rows of a column box in slab mode
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *tail = smem_raw + (base - raw) + (size_t)n_stages * stage_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tail);  // full[16], empty[16], done
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(tail + (2 * kMaxStages + 1) * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tail + (2 * kMaxStages + 1) * 8 + 8);
    const Waiter wt{abort_flag, err_word, kSpinLimit};
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
    const uint32_t done_bar = bar0 + 8u * (2 * kMaxStages);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int ky_cta = blockIdx.y;
    const int t0 = (int)((long)n_tiles * blockIdx.x / gridDim.x), t1 = (int)((long)n_tiles * (blockIdx.x + 1) / gridDim.x);

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(done_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch();
    pdl_wait();  // everything above is on-chip set-up; global memory is first touched below
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const int tiles_per_img = H / rows_per_tile;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            int n_img = t0 / tiles_per_img, t_img = t0 % tiles_per_img;  // divided once, then stepped
            for (int tile = t0; tile < t1 && ok; ++tile) {
                int n0, h0;
                if (imgs_per_tile > 1) { n0 = tile * imgs_per_tile; h0 = 0; }
                else { n0 = n_img; h0 = t_img * rows_per_tile; }
                if (++t_img == tiles_per_img) { t_img = 0; ++n_img; }
                ok = mbar_wait(empty_bar(s), ph ^ 1u, wt, 11);
                if (!ok) break;
                const uint32_t st = base + s * stage_bytes;
                mbar_expect_tx(full_bar(s), (uint32_t)stage_bytes);
                tma_load_4d(st, &tmap_dy, full_bar(s), 0, 0, h0, n0);
                for (int kx = 0; kx < 3; ++kx)
                    tma_load_4d(st + Cfg::tile_bytes + kx * x_box_bytes, &tmap_x, full_bar(s), 0, kx - 1,
                                slab ? h0 - 1 : h0 + ky_cta - 1, n0);
                if (++s == n_stages) { s = 0; ph ^= 1u; }
            }
            if (!ok) for (int i = 0; i < 2000; ++i) __nanosleep(100);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // both operands MN-major (bits 15, 16); fp32 accumulate; bf16 inputs; M = 128, N = 3C
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                                   ((uint32_t)((3 * C) >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
            const uint32_t idesc_wide = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                                        ((uint32_t)(((2 * box_rows + 3) * C) >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
            const uint32_t idesc_tall = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) |
                                        ((uint32_t)(C >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = t0; tile < t1 && ok; ++tile) {
                ok = mbar_wait(full_bar(s), ph, wt, 12);
                if (!ok) break;
                tc_fence_after();
                const uint32_t st = base + s * stage_bytes;
                if (slab && wide) {
                    // one instruction per 16 pixels: N runs over the three column boxes in one go (they are contiguous
                    // and each is box_rows image rows of W pixels), block b = kx*box_rows + ky; only ky < 3 is read back
#pragma unroll
                    for (int k = 0; k < kTileM / 16; ++k) {
                        const uint32_t koff = (uint32_t)k * 16 * Cfg::row_bytes;
                        const uint64_t adesc = make_desc(st + koff, 8 * Cfg::row_bytes, Cfg::layout, 2 * C * C);
                        const uint64_t bdesc = make_desc(st + Cfg::tile_bytes + koff, 8 * Cfg::row_bytes, Cfg::layout,
                                                         (uint32_t)W * Cfg::row_bytes);
                        tc_mma_bf16(tmem_base, adesc, bdesc, idesc_wide, (tile != t0) || (k != 0));
                    }
                } else if (slab && tall) {
                    // operands swapped: M runs over (filter row, input channel) = the rows of column box kx, N over the
                    // C output channels; 3 instructions per 16 pixels, C accumulator columns each
                    for (int kx = 0; kx < 3; ++kx) {
#pragma unroll
                        for (int k = 0; k < kTileM / 16; ++k) {
                            const uint32_t koff = (uint32_t)k * 16 * Cfg::row_bytes;
                            const uint64_t adesc = make_desc(st + Cfg::tile_bytes + kx * x_box_bytes + koff, 8 * Cfg::row_bytes,
                                                             Cfg::layout, (uint32_t)W * Cfg::row_bytes);
                            const uint64_t bdesc = make_desc(st + koff, 8 * Cfg::row_bytes, Cfg::layout, 2 * C * C);
                            tc_mma_bf16(tmem_base + (uint32_t)(kx * C), adesc, bdesc, idesc_tall, (tile != t0) || (k != 0));
                        }
                    }
                } else if (slab) {
                    for (int kx = 0; kx < 3; ++kx) {
#pragma unroll
                        for (int k = 0; k < kTileM / 16; ++k) {
                            const uint32_t koff = (uint32_t)k * 16 * Cfg::row_bytes;  // 16 pixels along the contraction axis
                            const uint64_t adesc = make_desc(st + koff, 8 * Cfg::row_bytes, Cfg::layout, 2 * C * C);
                            // N walks the C channels, then the next filter row: W pixels further down the same box
                            const uint64_t bdesc = make_desc(st + Cfg::tile_bytes + kx * x_box_bytes + koff, 8 * Cfg::row_bytes,
                                                             Cfg::layout, (uint32_t)W * Cfg::row_bytes);
                            tc_mma_bf16(tmem_base + (uint32_t)(kx * 3 * C), adesc, bdesc, idesc, (tile != t0) || (k != 0));
                        }
                    }
                } else {
#pragma unroll
                    for (int k = 0; k < kTileM / 16; ++k) {
                        const uint32_t koff = (uint32_t)k * 16 * Cfg::row_bytes;
                        // dy: M walks the C channels of a row, then (rows >= C, ignored) other rows of the same tile
                        const uint64_t adesc = make_desc(st + koff, 8 * Cfg::row_bytes, Cfg::layout, 2 * C * C);
                        // x: N walks the C channels, then the next filter column's box
                        const uint64_t bdesc = make_desc(st + Cfg::tile_bytes + koff, 8 * Cfg::row_bytes, Cfg::layout,
                                                         (uint32_t)x_box_bytes);
                        tc_mma_bf16(tmem_base, adesc, bdesc, idesc, (tile != t0) || (k != 0));
                    }
                }
                tc_commit(empty_bar(s));
                if (++s == n_stages) { s = 0; ph ^= 1u; }
            }
            if (ok) tc_commit(done_bar);
        }
    } else {
        const int q = warp & 3;
        bool ok = mbar_wait(done_bar, 0, wt, 13);
        ok = __all_sync(0xffffffffu, ok);
        if (ok && tall) {
            // accumulator row = ky*C + ci (rows >= 3C unused), column = kx*C + co: each thread writes runs of output channels
            tc_fence_after();
            const int r = 32 * q + lane, ky = r / C, ci = r % C;
            float *out = part + (size_t)blockIdx.x * 9 * C * C;
#pragma unroll 1
            for (int c0 = 0; c0 < 3 * C; c0 += 16) {
                float v[16];
                tc_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c0, v);
                tc_wait_ld();
                if (ky < 3) {
                    const int kx = c0 / C, co0 = c0 % C;
                    float4 *o4 = reinterpret_cast<float4 *>(out + ((size_t)(ky * 3 + kx) * C + ci) * C + co0);
#pragma unroll
                    for (int j = 0; j < 4; ++j) o4[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                }
            }
        } else if (ok && 32 * q < C) {  // only accumulator rows < C carry the result
            tc_fence_after();
            const int co = 32 * q + lane;
            float *out = part + (size_t)blockIdx.x * 9 * C * C;
            const int ncols = slab ? 9 * C : 3 * C;
#pragma unroll 1
            for (int c0 = 0; c0 < ncols; c0 += 16) {
                float v[16];
                // accumulator column of these 16 input channels: tap group g = c0 / C; in the wide layout group (kx, ky)
                // sits at block kx*box_rows + ky
                const int gq = c0 / C;
                const int col = wide ? ((gq / 3) * box_rows + gq % 3) * C + c0 % C : c0;
                tc_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)col, v);
                tc_wait_ld();
                if (co < C) {
                    // column c0..c0+15 = 16 input channels of one tap
                    const int g = c0 / C, ci0 = c0 % C;
                    const int tap = slab ? (g % 3) * 3 + g / 3 : ky_cta * 3 + g;   // slab: g = kx*3 + ky
#pragma unroll
                    for (int j = 0; j < 16; ++j) out[((size_t)tap * C + ci0 + j) * C + co] = v[j];  // [tap][ci][co]
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tmem_cols)
                     : "memory");
    }
}

// ---------------------------------------------------------------------------------------------------------
// Stride-2 3x3 convolution (the first convolution of a down-sampling residual block, Cout = 2 Cin) on the tensor
// cores.  Output pixel (oy, ox) reads input pixels (2oy+ky-1, 2ox+kx-1): for one filter tap these are every second
// pixel of every second row, which one TMA box fetches when the input [B][H][W][Ci] is described as the 5-D tensor
// (2 Ci, W/2, 2, H/2, B): a pixel PAIR is the innermost axis (the column parity px selects its first or second half),
// the row parity py is an axis of extent 2, and the zero fill of the pair axis and the half-row axis gives the padding.
//   forward : per tile of 128 output pixels, nine tap boxes [128][Ci], nine MMAs (M=128, N=Co, K=Ci) into one
//             accumulator.
//   dgrad   : the input pixels fall into four parity classes (py, px); a class-(py,px) pixel (2j+py, 2i+px) receives
//             taps ky = 1 (py = 0) or ky in {0, 2} (py = 1) from output rows j+1 / j, and likewise in x.  A tile is 128
//             input pixels of one class; its (1+py)(1+px) operand boxes are the dy tile shifted by 0/1 rows and columns
//             (zero-filled past the last row / column), MMAs M=128, N=Ci, K=Co.
// The pipeline (TMA warp, MMA warp, two epilogue groups, bounded waits) is that of the stride-1 kernel; one pipeline
// stage is one operand box.
// ---------------------------------------------------------------------------------------------------------
__device__ __forceinline__ void tma_load_5d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2,
                                            int c3, int c4) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6, %7}], "
        "[%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4)
        : "memory");
}

// KC: contraction channels (channels of the operand tensor); NC: channels of the result.  MODE 0 forward (KC = Ci,
// NC = Co), MODE 1 input gradient (KC = Co, NC = Ci).  Hs x Ws is the SMALL (output-resolution) map; rows_per_tile /
// imgs_per_tile describe a 128-pixel tile of it.  n_sp = number of such tiles.
template <int KC, int NC, int MODE>
__global__ void __launch_bounds__(kS2Threads, 1)
conv3x3_s2_tc_kernel(const __grid_constant__ CUtensorMap tmap, const bf16 *__restrict__ w, const uint8_t *__restrict__ w_packed,
                     bf16 *__restrict__ dst, int Hs, int Ws, int rows_per_tile, int imgs_per_tile, int n_sp, int n_stages,
                     const bf16 *__restrict__ res_dout, const bf16 *__restrict__ res_out, int *__restrict__ err_word) {
    typedef TcCfg<KC> Cfg;
    constexpr int CI = MODE == 0 ? KC : NC;
    constexpr int tap_bytes = KC * NC * 2;
    constexpr int w_bytes = 9 * tap_bytes;
    constexpr int stage_bytes = Cfg::tile_bytes;
    constexpr int tmem_cols = 2 * NC < 32 ? 32 : 2 * NC;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const uint32_t w_base = base, a_base = base + ((w_bytes + 1023u) & ~1023u);
    uint8_t *tail = smem + ((w_bytes + 1023u) & ~1023u) + (size_t)n_stages * stage_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tail);  // full[16], empty[16], tfull[4], tempty[4], wbar
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(tail + (2 * kMaxStages + 9) * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tail + (2 * kMaxStages + 9) * 8 + 8);
    const Waiter wt{abort_flag, err_word, kSpinLimit};
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
    auto tfull_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + a); };
    auto tempty_bar = [&](int a) { return bar0 + 8u * (2 * kMaxStages + 4 + a); };
    const uint32_t w_bar = bar0 + 8u * (2 * kMaxStages + 8);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int n_tiles = MODE == 0 ? n_sp : 4 * n_sp;

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), 4); }
        mbar_init(w_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch();
    pdl_wait();  // nothing above touches global memory
    if (w_packed == nullptr) {  // canonical filter [Co][Ci][3][3]: arrange the nine tiles of this pass here
        constexpr int CO = 2 * CI;
        for (int i = threadIdx.x; i < 9 * CO * CI; i += kS2Threads) {
            const int tap = i / (CO * CI), co = (i / CI) % CO, ci = i % CI;
            const uint32_t o = (uint32_t)tap * tap_bytes + (MODE == 0 ? swz_off<KC>(co, ci) : swz_off<KC>(ci, co));
            *reinterpret_cast<bf16 *>(smem + o) = w[(size_t)(co * CI + ci) * 9 + tap];
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const int tiles_per_img = Hs / rows_per_tile;
    // spatial tile -> (first image, first row of the small map)
    auto tile_origin = [&](int sp, int *n0, int *h0) {
        if (imgs_per_tile > 1) { *n0 = sp * imgs_per_tile; *h0 = 0; }
        else { *n0 = sp / tiles_per_img; *h0 = (sp % tiles_per_img) * rows_per_tile; }
    };

    if (warp == 0) {
        if (lane == 0) {
            if (w_packed != nullptr) {
                mbar_expect_tx(w_bar, w_bytes);
                bulk_copy_g2s(w_base, w_packed, w_bytes, w_bar);
            }
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x) {
                const int cls = MODE == 0 ? 0 : tile / n_sp, sp = MODE == 0 ? tile : tile % n_sp;
                const int py = cls >> 1, px = cls & 1;
                int n0, h0;
                tile_origin(sp, &n0, &h0);
                const int n_loads = MODE == 0 ? 9 : (1 + py) * (1 + px);
                for (int j = 0; j < n_loads && ok; ++j) {
                    ok = mbar_wait(empty_bar(s), ph ^ 1u, wt, 21);
                    if (!ok) break;
                    mbar_expect_tx(full_bar(s), (uint32_t)stage_bytes);
                    const uint32_t d = a_base + s * stage_bytes;
                    if (MODE == 0) {
                        const int ky = j / 3, kx = j % 3;
                        // column 2ox+kx-1: kx = 1 -> first pixel of pair ox; kx = 0 / 2 -> second pixel of pair ox-1 / ox
                        tma_load_5d(d, &tmap, full_bar(s), kx == 1 ? 0 : KC, kx == 0 ? -1 : 0, ky == 1 ? 0 : 1,
                                    h0 + (ky == 0 ? -1 : 0), n0);
                    } else {
                        const int sy = px ? j >> 1 : j, sx = px ? j & 1 : 0;
                        tma_load_4d(d, &tmap, full_bar(s), 0, sx, h0 + sy, n0);
                    }
                    if (++s == n_stages) { s = 0; ph ^= 1u; }
                }
            }
            if (!ok) for (int i = 0; i < 2000; ++i) __nanosleep(100);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(NC >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
            int s = 0;
            uint32_t ph = 0;
            int it = 0;
            bool ok = true;
            if (w_packed != nullptr) ok = mbar_wait(w_bar, 0, wt, 25);
            for (int tile = blockIdx.x; tile < n_tiles && ok; tile += gridDim.x, ++it) {
                const int cls = MODE == 0 ? 0 : tile / n_sp;
                const int py = cls >> 1, px = cls & 1;
                const int n_loads = MODE == 0 ? 9 : (1 + py) * (1 + px);
                const int a = it & 1;
                const uint32_t aph = (it >> 1) & 1u;
                ok = mbar_wait(tempty_bar(a), aph ^ 1u, wt, 22);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)(a * NC);
                for (int j = 0; j < n_loads && ok; ++j) {
                    ok = mbar_wait(full_bar(s), ph, wt, 23);
                    if (!ok) break;
                    tc_fence_after();
                    int tap = j;
                    if (MODE == 1) {
                        const int sy = px ? j >> 1 : j, sx = px ? j & 1 : 0;
                        // dx row 2j'+1 takes ky = 0 from output row j'+1 (the shifted box) and ky = 2 from row j'
                        const int ky = py ? (sy ? 0 : 2) : 1, kx = px ? (sx ? 0 : 2) : 1;
                        tap = ky * 3 + kx;
                    }
                    const uint64_t adesc = make_desc(a_base + s * stage_bytes, 8 * Cfg::row_bytes, Cfg::layout);
                    const uint64_t bdesc = make_desc(w_base + tap * tap_bytes, 8 * Cfg::row_bytes, Cfg::layout);
#pragma unroll
                    for (int k = 0; k < KC / 16; ++k) tc_mma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (j | k) != 0);
                    tc_commit(empty_bar(s));
                    if (++s == n_stages) { s = 0; ph ^= 1u; }
                }
                if (ok) tc_commit(tfull_bar(a));
            }
        }
    } else {
        const int q = warp & 3;
        const int grp = (warp - 2) >> 2;
        int it = grp;
        bool ok = true;
        for (int tile = blockIdx.x + grp * gridDim.x; tile < n_tiles && ok; tile += 2 * gridDim.x, it += 2) {
            const int a = it & 1;
            const uint32_t aph = (it >> 1) & 1u;
            ok = mbar_wait(tfull_bar(a), aph, wt, 24);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int cls = MODE == 0 ? 0 : tile / n_sp, sp = MODE == 0 ? tile : tile % n_sp;
            const int pl = 32 * q + lane;
            const size_t pix_small = (size_t)sp * kTileM + pl;  // pixel of the small map, linear over [B][Hs][Ws]
            size_t pix_dst = pix_small;
            if (MODE == 1) {
                const int py = cls >> 1, px = cls & 1;
                int n0, h0;
                tile_origin(sp, &n0, &h0);
                const int i = pl % Ws, jr = (pl / Ws) % rows_per_tile, nl = pl / (Ws * rows_per_tile);
                pix_dst = ((size_t)(n0 + nl) * (2 * Hs) + 2 * (h0 + jr) + py) * (size_t)(2 * Ws) + 2 * i + px;
            }
            const uint32_t t_row = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(a * NC);
#pragma unroll 1
            for (int c0 = 0; c0 < NC; c0 += 16) {
                float acc[16];
                tc_ld16(t_row + (uint32_t)c0, acc);
                tc_wait_ld();
                if (c0 + 16 >= NC) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(tempty_bar(a));
                }
                if (MODE == 1 && cls == 0 && res_dout != nullptr) {
                    // gradient of the parameter-free shortcut: the block input at (2j, 2i), channel c, was added to channel
                    // c of the block output at (j, i); the output has KC channels
#pragma unroll
                    for (int h = 0; h < 16; h += 8) {
                        float d[8], o[8];
                        load_f<bf16, 8>(res_dout + pix_small * KC + c0 + h, d);
                        load_f<bf16, 8>(res_out + pix_small * KC + c0 + h, o);
#pragma unroll
                        for (int j = 0; j < 8; ++j) if (o[j] > 0.f) acc[h + j] += d[j];
                    }
                }
#pragma unroll
                for (int h = 0; h < 16; h += 8) {
                    float v[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) v[j] = acc[h + j];
                    store_f<bf16, 8>(dst + pix_dst * NC + c0 + h, v);
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tmem_cols)
                     : "memory");
    }
}

// Weight gradient of the stride-2 convolution: dw[co][ci][tap] = sum_p dy[p][co] * x[tap box][p][ci].  Per tile of 128
// output pixels one dy box and the nine tap boxes of the forward pass; both operands MN-major (pixels are the
// contraction axis), M = 128 (rows >= Co unused), the taps stacked along N through the leading-dimension offset
// (N = 9 Ci, split in two instructions when it exceeds 256).  A CTA accumulates its tiles in TMEM and writes one fp32
// partial [tap][ci][co].
template <int CI>
__global__ void __launch_bounds__(kWgThreads, 1)
wgrad_s2_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_dy,
                   float *__restrict__ part, int Hs, int Ws, int rows_per_tile, int imgs_per_tile, int n_tiles, int n_stages,
                   int *__restrict__ err_word) {
    constexpr int CO = 2 * CI;
    typedef TcCfg<CI> CfgX;
    typedef TcCfg<CO> CfgY;
    constexpr int stage_bytes = CfgY::tile_bytes + 9 * CfgX::tile_bytes;
    constexpr int n_total = 9 * CI;
    constexpr int n_first = n_total <= 256 ? n_total : 5 * CI;  // taps 0-4, then taps 5-8
    constexpr int tmem_cols = n_total <= 256 ? 256 : 512;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *tail = smem_raw + (base - raw) + (size_t)n_stages * stage_bytes;
    uint64_t *bars = reinterpret_cast<uint64_t *>(tail);
    uint32_t *tmem_holder = reinterpret_cast<uint32_t *>(tail + (2 * kMaxStages + 1) * 8);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tail + (2 * kMaxStages + 1) * 8 + 8);
    const Waiter wt{abort_flag, err_word, kSpinLimit};
    const uint32_t bar0 = smem_u32(bars);
    auto full_bar = [&](int s) { return bar0 + 8u * s; };
    auto empty_bar = [&](int s) { return bar0 + 8u * (kMaxStages + s); };
    const uint32_t done_bar = bar0 + 8u * (2 * kMaxStages);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int t0 = (int)((long)n_tiles * blockIdx.x / gridDim.x), t1 = (int)((long)n_tiles * (blockIdx.x + 1) / gridDim.x);

    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
        mbar_init(done_bar, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)),
                     "r"((uint32_t)tmem_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    pdl_launch();
    pdl_wait();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_holder;
    const int tiles_per_img = Hs / rows_per_tile;

    if (warp == 0) {
        if (lane == 0) {
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = t0; tile < t1 && ok; ++tile) {
                int n0, h0;
                if (imgs_per_tile > 1) { n0 = tile * imgs_per_tile; h0 = 0; }
                else { n0 = tile / tiles_per_img; h0 = (tile % tiles_per_img) * rows_per_tile; }
                ok = mbar_wait(empty_bar(s), ph ^ 1u, wt, 31);
                if (!ok) break;
                const uint32_t st = base + s * stage_bytes;
                mbar_expect_tx(full_bar(s), (uint32_t)stage_bytes);
                tma_load_4d(st, &tmap_dy, full_bar(s), 0, 0, h0, n0);
                for (int tap = 0; tap < 9; ++tap) {
                    const int ky = tap / 3, kx = tap % 3;
                    tma_load_5d(st + CfgY::tile_bytes + tap * CfgX::tile_bytes, &tmap_x, full_bar(s), kx == 1 ? 0 : CI,
                                kx == 0 ? -1 : 0, ky == 1 ? 0 : 1, h0 + (ky == 0 ? -1 : 0), n0);
                }
                if (++s == n_stages) { s = 0; ph ^= 1u; }
            }
            if (!ok) for (int i = 0; i < 2000; ++i) __nanosleep(100);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc0 = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(kTileM >> 4) << 24);
            const uint32_t idesc_a = idesc0 | ((uint32_t)(n_first >> 3) << 17);
            const uint32_t idesc_b = idesc0 | ((uint32_t)((n_total - n_first) >> 3) << 17);
            int s = 0;
            uint32_t ph = 0;
            bool ok = true;
            for (int tile = t0; tile < t1 && ok; ++tile) {
                ok = mbar_wait(full_bar(s), ph, wt, 32);
                if (!ok) break;
                tc_fence_after();
                const uint32_t st = base + s * stage_bytes;
#pragma unroll
                for (int k = 0; k < kTileM / 16; ++k) {
                    // 16 pixels further along the contraction axis in each operand
                    const uint64_t adesc = make_desc(st + (uint32_t)k * 16 * CfgY::row_bytes, 8 * CfgY::row_bytes, CfgY::layout, 2 * CO * CO);
                    const uint32_t xb = st + CfgY::tile_bytes + (uint32_t)k * 16 * CfgX::row_bytes;
                    const uint64_t bdesc = make_desc(xb, 8 * CfgX::row_bytes, CfgX::layout, CfgX::tile_bytes);
                    tc_mma_bf16(tmem_base, adesc, bdesc, idesc_a, (tile != t0) || (k != 0));
                    if (n_first < n_total) {
                        const uint64_t bdesc2 = make_desc(xb + 5 * CfgX::tile_bytes, 8 * CfgX::row_bytes, CfgX::layout, CfgX::tile_bytes);
                        tc_mma_bf16(tmem_base + (uint32_t)n_first, adesc, bdesc2, idesc_b, (tile != t0) || (k != 0));
                    }
                }
                tc_commit(empty_bar(s));
                if (++s == n_stages) { s = 0; ph ^= 1u; }
            }
            if (ok) tc_commit(done_bar);
        }
    } else {
        const int q = warp & 3;
        bool ok = mbar_wait(done_bar, 0, wt, 33);
        ok = __all_sync(0xffffffffu, ok);
        if (ok && 32 * q < CO) {
            tc_fence_after();
            const int co = 32 * q + lane;
            float *out = part + (size_t)blockIdx.x * 9 * CI * CO;
#pragma unroll 1
            for (int c0 = 0; c0 < n_total; c0 += 16) {
                float v[16];
                tc_ld16(tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)c0, v);
                tc_wait_ld();
#pragma unroll
                for (int j = 0; j < 16; ++j) out[(size_t)(c0 + j) * CO + co] = v[j];  // column = tap*Ci + ci
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)tmem_cols)
                     : "memory");
    }
}

// dw[co][ci][tap] = sum over chunks of part[chunk][tap][ci][co].  64 outputs per CTA, four threads per output: thread g
// adds chunks g, g+4, ... (four independent loads in flight per thread), the four sums are combined in a fixed order.
// C = input channels of the partials, Co = output channels, cin <= C = input channels of dw.
__global__ void __launch_bounds__(256) wgrad_tc_fold_kernel(const float *__restrict__ part, float *__restrict__ dw, int chunks, int C,
                                                            int Co, int cin) {
    pdl_launch();
    pdl_wait();
    __shared__ float sm[4][64];
    const int total = 9 * C * Co;
    const int o = threadIdx.x & 63, g = threadIdx.x >> 6;
    const int i = blockIdx.x * 64 + o;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (i < total) {
        // batches of eight loads in flight per thread (the kernel is a chain of L2 round trips), the last one predicated
        for (int c = g; c < chunks; c += 32) {
            float q[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) q[u] = (c + 4 * u < chunks) ? __ldcg(part + (size_t)(c + 4 * u) * total + i) : 0.f;
#pragma unroll
            for (int u = 0; u < 8; ++u) acc[u] += q[u];
        }
    }
    sm[g][o] = ((acc[0] + acc[1]) + (acc[2] + acc[3])) + ((acc[4] + acc[5]) + (acc[6] + acc[7]));
    __syncthreads();
    if (g == 0 && i < total) {
        const float t = (sm[0][o] + sm[1][o]) + (sm[2][o] + sm[3][o]);
        const int co = i % Co, ci = (i / Co) % C, tap = i / (C * Co);
        if (ci < cin) dw[((size_t)co * cin + ci) * 9 + tap] = t;  // cin < C: the input was zero-padded to C channels
    }
}

// ---- host side: tensor maps ------------------------------------------------------------------------------
PFN_cuTensorMapEncodeTiled_v12000 g_encode = nullptr;

struct MapKey {
    const void *ptr; int B, H, W, C, rows, imgs;
    bool operator<(const MapKey &o) const {
        return std::tie(ptr, B, H, W, C, rows, imgs) < std::tie(o.ptr, o.B, o.H, o.W, o.C, o.rows, o.imgs);
    }
};
std::map<MapKey, CUtensorMap> g_maps;
std::mutex g_maps_mu;

void tile_geometry(int H, int W, int *rows_per_tile, int *imgs_per_tile) {
    int r = kTileM / W;
    if (r > H) r = H;
    *rows_per_tile = r;
    *imgs_per_tile = kTileM / (W * r);
}

// Tensor map of an NHWC bf16 tensor with a box of (C, W, rows, imgs), zero fill outside the tensor.
bool get_map(const void *ptr, int B, int H, int W, int C, int rows, int imgs, CUtensorMap *out) {
    std::lock_guard<std::mutex> lock(g_maps_mu);
    MapKey key{ptr, B, H, W, C, rows, imgs};
    auto it = g_maps.find(key);
    if (it != g_maps.end()) { *out = it->second; return true; }
    cuuint64_t dims[4] = {(cuuint64_t)C, (cuuint64_t)W, (cuuint64_t)H, (cuuint64_t)B};
    cuuint64_t strides[3] = {(cuuint64_t)C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)H * W * C * 2};
    cuuint32_t box[4] = {(cuuint32_t)C, (cuuint32_t)W, (cuuint32_t)rows, (cuuint32_t)imgs};
    cuuint32_t estr[4] = {1, 1, 1, 1};
    CUtensorMapSwizzle swz = C == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (C == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    CUtensorMap m;
    CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (g_maps.size() > 8192) g_maps.clear();
    g_maps[key] = m;
    *out = m;
    return true;
}

// Tensor map of the stride-2 view of an NHWC bf16 tensor [B][H][W][C]: axes (pixel pair = 2C, W/2, row parity, H/2, B),
// box (C, W/2, 1, rows, imgs): one column parity of one row parity.
std::map<MapKey, CUtensorMap> g_maps_s2;
bool get_map_s2(const void *ptr, int B, int H, int W, int C, int rows, int imgs, CUtensorMap *out) {
    std::lock_guard<std::mutex> lock(g_maps_mu);
    MapKey key{ptr, B, H, W, C, rows, imgs};
    auto it = g_maps_s2.find(key);
    if (it != g_maps_s2.end()) { *out = it->second; return true; }
    cuuint64_t dims[5] = {(cuuint64_t)2 * C, (cuuint64_t)W / 2, 2, (cuuint64_t)H / 2, (cuuint64_t)B};
    cuuint64_t strides[4] = {(cuuint64_t)2 * C * 2, (cuuint64_t)W * C * 2, (cuuint64_t)2 * W * C * 2, (cuuint64_t)H * W * C * 2};
    cuuint32_t box[5] = {(cuuint32_t)C, (cuuint32_t)(W / 2), 1, (cuuint32_t)rows, (cuuint32_t)imgs};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    CUtensorMapSwizzle swz = C == 64 ? CU_TENSOR_MAP_SWIZZLE_128B : (C == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_32B);
    CUtensorMap m;
    CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void *>(ptr), dims, strides, box, estr,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, swz, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (g_maps_s2.size() > 1024) g_maps_s2.clear();
    g_maps_s2[key] = m;
    *out = m;
    return true;
}

int g_num_sms = 148;
// device address of the process-wide error word (single-kernel entry points); contexts bring their own
int *g_tc_error_addr = nullptr;
int *err_word_of(const Launch &L) { return L.err ? L.err : g_tc_error_addr; }
// Shared memory a CTA may take for its pipeline stages: less than half an SM, so that kernels of two modules (streams)
// can share an SM instead of queueing behind each other (K = 4 step, ms per iteration at 56 / 64 / 72 / 80 / 100 / 128
// KB: 1.870 / 1.884 / 1.844 / 1.844 - 1.857 / 1.874 / 2.068).
constexpr int kSmemBudget = 80 * 1024;
constexpr int kSmemMax = 227 * 1024;

// Launch plan of the forward / input-gradient kernel for n_tiles tiles: pipelines per CTA, epilogue groups, grid.
//   C = 16 (one 16-channel chunk per tile): two pipelines where an SM has at least four tiles, four where it has at
//   least sixteen (large batches); below that one pipeline whose two epilogue groups take alternate tiles.
//   C >= 32: one pipeline whose two groups halve every tile where an SM has a single tile (shorter epilogue); for
//   C = 32 two pipelines with one group each where it has two (both tiles side by side; C = 64 would need all 512
//   TMEM columns for that).  Three tiles or more: C = 64 two pipelines whose two groups halve every tile; C = 32 two
//   pipelines with two accumulators and one group each (the MMAs of the next tile run under the epilogue of this one;
//   batch 256 / 1024 / 4096: 11.9 / 17.5 / 39.4 -> 10.8 / 16.5 / 36.5 us against two groups halving the tile), and
//   four pipelines from sixteen tiles per SM on (batch 4096: 35.4 us).
// A pipeline with a single tile uses one accumulator: fewer TMEM columns, so that CTAs of other streams fit beside it.
// Several module streams (shared): as few CTAs as give every pipeline the same number of tiles as a full grid would give
// the busiest one; the kernel's critical path is as long, and the SMs left over are free for the other streams (K = 4
// step -2 %).  A kernel that has the GPU to itself takes every SM (a few pipelines then finish early).
struct TcPlan { EpiPlan ep; int grid, threads, xf_warps; };
TcPlan tc_plan(int C, int n_tiles, int slab, bool shared, bool xform) {
    const int sms = g_num_sms;
    EpiPlan ep;
    if (C == 16) {
        const int P = !slab ? 1 : (n_tiles >= 16 * sms ? 4 : (n_tiles >= 4 * sms ? 2 : 1));
        const int n_acc = P > 1 ? 1 : (n_tiles <= sms ? 1 : 2);
        ep = EpiPlan{P, n_acc, n_acc, 1};
    } else if (n_tiles >= 3 * sms) {
        if (C == 64) ep = EpiPlan{2, 1, 1, 2};  // 2 x 2 x 192 columns would not fit
        else ep = n_tiles >= 16 * sms ? EpiPlan{4, 1, 1, 1} : EpiPlan{2, 2, 1, 1};
    } else if (C == 32 && n_tiles > sms) {
        ep = EpiPlan{2, 1, 1, 1};
    } else {
        ep = EpiPlan{1, n_tiles <= sms ? 1 : 2, 1, 2};
    }
    if (xform) {
        // four transform warps per pipeline must fit the kernel's 768 threads: at most two pipelines, one epilogue group
        // each where the plan above would launch two
        if (ep.n_pipes > 2) ep = EpiPlan{2, 1, 1, 1};
        if (2 * ep.n_pipes + 4 * ep.n_pipes * ep.n_slots * ep.split + 4 * ep.n_pipes > 24) ep = EpiPlan{2, ep.n_acc, 1, 1};
    }
    TcPlan p;
    p.ep = ep;
    int per_pipe = (n_tiles + sms * ep.n_pipes - 1) / (sms * ep.n_pipes);
    // ... and never a single tile per pipeline: a CTA's set-up and wind-down (barriers, TMEM, filter image, partial sums)
    // cost as much SM time as three or four tiles, and under sharing the SM time a kernel takes is what the other
    // streams wait for.  Half the CTAs with two tiles each: the 32- and 64-channel convolutions of the K = 4 step (256
    // and 64 tiles) take longer alone, the iteration 6 % less (1.758 -> 1.650 ms); three tiles: 1.675; doubling the 16-
    // channel kernels' four tiles per pipeline: 1.84.
    if (shared && per_pipe < 2) per_pipe = 2;
    const int balanced = (n_tiles + per_pipe * ep.n_pipes - 1) / (per_pipe * ep.n_pipes);
    const int full = (n_tiles + ep.n_pipes - 1) / ep.n_pipes < sms ? (n_tiles + ep.n_pipes - 1) / ep.n_pipes : sms;
    p.grid = shared ? balanced : full;
    const int groups = ep.n_pipes * ep.n_slots * ep.split;
    // Transform warps per pipeline: every thread a CTA launches is given the kernel's 80 registers, so these warps cost
    // register file that CTAs of the other module streams would otherwise use; one warp keeps up with a 16-channel tile
    // (12 - 24 16-byte cells per lane), the wider tiles get two and four.
    p.xf_warps = xform ? (C == 16 ? 1 : (C == 32 ? 2 : 4)) : 0;
    // issuing warps, four warps per epilogue group, and the transform warps
    p.threads = 32 * (2 * ep.n_pipes + 4 * (groups < 2 ? 2 : groups) + p.xf_warps * ep.n_pipes);
    return p;
}

template <int C>
int launch_tc(int dir, const void *src, const void *w, const void *w_packed, void *dst, int B, int H, int W,
              Shortcut sc, BnFuse bf, InXform xf, Launch s) {
    int rows, imgs;
    tile_geometry(H, W, &rows, &imgs);
    const int slab = (imgs == 1) ? 1 : 0;
    const int box_rows = slab ? rows + 2 : rows;
    CUtensorMap map;
    if (32 % W != 0 || !get_map(src, B, H, W, C, box_rows, imgs, &map)) return -1;
    const bool xform = xf.gamma != nullptr;
    if (xform && dir != 0) return -1;
    CUtensorMap map_res = map;
    if (xform && xf.res != nullptr && !get_map(xf.res, B, H, W, C, box_rows, imgs, &map_res)) return -1;
    const int stage_bytes = box_rows * imgs * W * C * 2 * (xform && xf.res != nullptr ? 2 : 1);
    const int n_tiles = (int)((long)B * H * W / kTileM);
    const TcPlan pl = tc_plan(C, n_tiles, slab, s.shared, xform);
    const EpiPlan ep = pl.ep;
    const int grid = pl.grid, threads = pl.threads;
    if (threads > 768) return -1;  // the kernel's launch bound
    // CTAs with many tiles take the whole SM's shared memory for the stage ring; the others about half of it
    const int budget = n_tiles >= 8 * grid ? kSmemMax - 1024 - kTailBytes : kSmemBudget;
    int n_stages = (budget - (int)conv_smem_plan<C>(0, 0).a_off) / stage_bytes;
    if (n_stages > kMaxStages) n_stages = kMaxStages;
    int min_ring = 3;
    if (conv_smem_bytes<C>(min_ring * ep.n_pipes, stage_bytes) > (size_t)kSmemMax) min_ring = 2;  // two-box stages of wide tiles
    if (n_stages < min_ring * ep.n_pipes) n_stages = min_ring * ep.n_pipes;
    n_stages -= n_stages % ep.n_pipes;
    const int acc_cols = ep.n_pipes * ep.n_acc * 3 * C;
    int tmem_cols = 32;
    while (tmem_cols < acc_cols) tmem_cols <<= 1;
    if (tmem_cols > 512 || conv_smem_bytes<C>(n_stages, stage_bytes) > (size_t)kSmemMax) return -1;
    if (bf.n_part_out != nullptr) *bf.n_part_out = grid;
    launch_kp(true, conv3x3_tc_kernel<C>, grid, threads, conv_smem_bytes<C>(n_stages, stage_bytes), s, map, map_res, (const bf16 *)w, (const uint8_t *)w_packed, (bf16 *)dst, dir, H, W, rows, imgs, n_tiles, slab, n_stages,
        stage_bytes, tmem_cols, ep, sc.mode == 1 ? (const bf16 *)sc.a : nullptr, sc.mode == 1 ? (const bf16 *)sc.b : nullptr, bf.part,
        bf.counter, bf.o0, bf.o1, (const bf16 *)bf.mask, (const bf16 *)bf.x, bf.mean, bf.invstd, (const bf16 *)xf.gamma,
        (const bf16 *)xf.beta, xf.mean, xf.invstd, (bf16 *)xf.a_out, (xform && xf.res != nullptr) ? 1 : 0, pl.xf_warps, err_word_of(s));
    return 1;
}

template <int C>
int launch_wg(const void *x, const void *dy, float *dw, float *scratch, int B, int H, int W, int cin, Launch s) {
    int rows, imgs;
    tile_geometry(H, W, &rows, &imgs);
    const int slab = (imgs == 1 && 9 * C <= 512) ? 1 : 0;
    CUtensorMap mx, md;
    if (!get_map(x, B, H, W, C, slab ? rows + 2 : rows, imgs, &mx) || !get_map(dy, B, H, W, C, rows, imgs, &md)) return -1;
    const int x_box_bytes = (slab ? rows + 2 : rows) * imgs * W * C * 2;
    const int stage_bytes = TcCfg<C>::tile_bytes + 3 * x_box_bytes;
    const int n_tiles_all = (int)((long)B * H * W / kTileM);
    // many tiles per CTA (large batches): the whole SM's shared memory for the stage ring, so that the loads of the next
    // tiles are in flight while this one is multiplied (batch 4096: 72 -> 68 us at 32 channels, 53 -> 44 us at 64);
    // otherwise the half-SM budget: taking more in the training step cost 4 % of the K = 4 iteration
    // 32 channels, very large batches: two CTAs per SM (half the shared memory each, twice the pixel chunks): the MMA
    // thread of this operand-swapped form is issue-bound, a second one per SM takes batch 4096 from 70.6 to 61.6 us
    // (the 16-channel form is bound by the tensor pipe and the 64-channel one by its fold: both lose with two)
    const bool pair = C == 32 && n_tiles_all >= 32 * g_num_sms;
    // training-step sizes: the half-SM budget (two stages of 32 or 64 channels); the 16-channel kernel, whose tile is
    // eight tensor-bound instructions, wants a fourth stage of loads in flight (K = 1 / 3 / 4 iteration -1.7 / -0.8 /
    // -1.6 %; two, five or six stages lose)
    const int small_budget = C == 16 ? 100 * 1024 : kSmemBudget;
    const int budget = pair ? 110 * 1024 : (n_tiles_all >= 8 * g_num_sms ? kSmemMax - 2048 - (C == 32 ? 4096 : 0) : small_budget);
    int n_stages = budget / stage_bytes;
    if (n_stages > kMaxStages) n_stages = kMaxStages;
    if (n_stages < 2) n_stages = 2;
    // slab mode with narrow channels: all nine taps from one instruction per 16 pixels when the three column boxes
    // (contiguous, box_rows blocks of C columns each) fit one N <= 256
    const int wide = (slab && (2 * (rows + 2) + 3) * C <= 256) ? 1 : 0;
    // otherwise, where 128 accumulator rows hold three filter rows (C = 32), the operands are swapped: 3C columns
    // instead of 9C, so that the kernel takes a quarter of the TMEM and leaves room for other streams' CTAs
    const int tall = (slab && !wide && 3 * C <= kTileM) ? 1 : 0;
    const int ncols = wide ? (2 * (rows + 2) + 3) * C : ((slab && !tall) ? 9 * C : 3 * C);
    const int tmem_cols = ncols <= 64 ? 64 : (ncols <= 128 ? 128 : (ncols <= 256 ? 256 : 512));
    const int n_tiles = (int)((long)B * H * W / kTileM);
    // pixel chunks (= CTAs, = partials to fold): few at the training step's sizes, where the kernel shares the GPU with
    // the other streams and the fold should stay small; one per 16 tiles, up to a CTA per SM, for large batches
    // (64 channels, whose launch has three CTAs per chunk, one per filter row: half as many chunks while several module
    // streams share the GPU - K = 4 iteration 1.629 -> 1.607 ms, K = 2, 3 unchanged; the 16- and 32-channel counts lose
    // in both directions)
    const int max_chunks = slab ? (C == 16 ? 74 : 37) : (s.shared ? 12 : 24);
    int chunks = n_tiles < max_chunks ? n_tiles : max_chunks;
    const int cap = slab ? (pair ? 2 * kWgMaxChunks : kWgMaxChunks) : 48;
    const int big = n_tiles / 16 < cap ? n_tiles / 16 : cap;
    if (big > chunks) chunks = big;
    // tall: the unused accumulator rows (filter rows >= 3) read up to 128 - 3C pixel rows past the last column box
    launch_k(wgrad_tc_kernel<C>, dim3(chunks, slab ? 1 : 3), kWgThreads, 1024 + (size_t)n_stages * stage_bytes + 512 + (tall ? 4096 : 0), s, mx, md, scratch, H, W, rows, imgs, n_tiles, slab, n_stages, x_box_bytes, tmem_cols, wide, tall, err_word_of(s));
    launch_k(wgrad_tc_fold_kernel, ceil_div(9 * C * C, 64), 256, 0, s, scratch, dw, chunks, C, C, cin);
    return 2;
}

template <int KC, int NC, int MODE>
size_t s2_smem_bytes(int n_stages) {
    return 1024 + ((9 * KC * NC * 2 + 1023) & ~1023) + (size_t)n_stages * TcCfg<KC>::tile_bytes + 512;
}
// H, W: the large (input-resolution) map.  dir 0: src = x [B][H][W][CI] -> dst = y [B][H/2][W/2][2CI];
// dir 1: src = dy -> dst = dx, plus the parameter-free shortcut's gradient when sc.mode == 2.
template <int CI>
int launch_tc_s2(int dir, const void *src, const void *w, const void *w_packed, void *dst, int B, int H, int W, Shortcut sc,
                 Launch s) {
    constexpr int CO = 2 * CI;
    const int Hs = H / 2, Ws = W / 2;
    int rows, imgs;
    tile_geometry(Hs, Ws, &rows, &imgs);
    const int n_sp = (int)((long)B * Hs * Ws / kTileM);
    const uint8_t *pk = (const uint8_t *)w_packed;
    CUtensorMap map;
    if (dir == 0) {
        if (!get_map_s2(src, B, H, W, CI, rows, imgs, &map)) return -1;
        int n_stages = kSmemBudget / TcCfg<CI>::tile_bytes;
        if (n_stages > kMaxStages) n_stages = kMaxStages;
        // two CTAs per SM where a CTA's single pipeline leaves the SM idle between hand-offs (16 -> 32 channels, batch
        // 1024 / 4096: 39 / 126 -> 25 / 70 us); the 32 -> 64 forward is faster with one (22 / 46 against 27 / 51 us)
        const int cap = (CI == 16 ? 2 : 1) * g_num_sms;
        const int grid = n_sp < cap ? n_sp : cap;
        launch_k(conv3x3_s2_tc_kernel<CI, CO, 0>, grid, kS2Threads, s2_smem_bytes<CI, CO, 0>(n_stages), s, map, (const bf16 *)w, pk,
                 (bf16 *)dst, Hs, Ws, rows, imgs, n_sp, n_stages, (const bf16 *)nullptr, (const bf16 *)nullptr, err_word_of(s));
    } else {
        if (!get_map(src, B, Hs, Ws, CO, rows, imgs, &map)) return -1;
        int n_stages = (kSmemBudget - 9 * CI * CO * 2) / TcCfg<CO>::tile_bytes;
        if (n_stages > kMaxStages) n_stages = kMaxStages;
        if (n_stages < 3) n_stages = 3;
        const int n_tiles = 4 * n_sp;
        // two CTAs per SM (batch 1024 / 4096: 59 / 208 -> 37 / 121 us for 16 <- 32 channels, 27 / 73 -> 23 / 51 us for
        // 32 <- 64)
        const int grid = n_tiles < 2 * g_num_sms ? n_tiles : 2 * g_num_sms;
        launch_k(conv3x3_s2_tc_kernel<CO, CI, 1>, grid, kS2Threads, s2_smem_bytes<CO, CI, 1>(n_stages), s, map, (const bf16 *)w,
                 pk ? pk + S2Cfg<CI>::img_bytes : pk, (bf16 *)dst, Hs, Ws, rows, imgs, n_sp, n_stages,
                 sc.mode == 2 ? (const bf16 *)sc.a : nullptr, sc.mode == 2 ? (const bf16 *)sc.b : nullptr, err_word_of(s));
    }
    return 1;
}

template <int CI>
int launch_wg_s2(const void *x, const void *dy, float *dw, float *scratch, int B, int H, int W, Launch s) {
    constexpr int CO = 2 * CI;
    const int Hs = H / 2, Ws = W / 2;
    int rows, imgs;
    tile_geometry(Hs, Ws, &rows, &imgs);
    CUtensorMap mx, md;
    if (!get_map_s2(x, B, H, W, CI, rows, imgs, &mx) || !get_map(dy, B, Hs, Ws, CO, rows, imgs, &md)) return -1;
    const int stage_bytes = TcCfg<CO>::tile_bytes + 9 * TcCfg<CI>::tile_bytes;
    int n_stages = (200 * 1024) / stage_bytes;
    if (n_stages > 4) n_stages = 4;
    const int n_tiles = (int)((long)B * Hs * Ws / kTileM);
    // pixel chunks = CTAs: 64 at the training step's sizes (a small fold), one per SM from four tiles per SM on (batch
    // 1024 / 4096, 16 -> 32 channels: 36 / 103 -> 31 / 74 us; 32 -> 64: 23.5 / 52 -> 22 / 40 us)
    const int max_chunks = n_tiles >= 512 ? kWgMaxChunks : 64;
    const int chunks = n_tiles < max_chunks ? n_tiles : max_chunks;
    launch_k(wgrad_s2_tc_kernel<CI>, chunks, kWgThreads, 1024 + (size_t)n_stages * stage_bytes + 512, s, mx, md, scratch, Hs, Ws,
             rows, imgs, n_tiles, n_stages, err_word_of(s));
    launch_k(wgrad_tc_fold_kernel, ceil_div(9 * CI * CO, 64), 256, 0, s, scratch, dw, chunks, CI, CO, CI);
    return 2;
}

}  // namespace

// stride 2, Cout = 2 Cin, Cin in {16, 32}, output map 16x16 or 8x8 in whole 128-pixel tiles
bool conv_tc_s2_supported(int B, int H, int W, int Cin, int Cout, int stride) {
    if (!g_encode) return false;
    if (stride != 2 || Cout != 2 * Cin || (Cin != 16 && Cin != 32)) return false;
    if ((H & 1) || (W & 1)) return false;
    const int Hs = H / 2, Ws = W / 2;
    if (Ws < 4 || Ws > 32 || kTileM % Ws != 0) return false;
    const int r = kTileM / Ws;
    if (r <= Hs) { if (Hs % r != 0) return false; }
    else { if (kTileM % (Hs * Ws) != 0 || B % (kTileM / (Hs * Ws)) != 0) return false; }
    return ((long)B * Hs * Ws) % kTileM == 0;
}
size_t tc_s2_packed_bytes(int Cin) { return 2 * (size_t)9 * Cin * 2 * Cin * 2; }

int launch_conv_tc_s2(int dir, const void *src, const void *w, const void *w_packed, void *dst, int B, int H, int W, int Cin,
                      Shortcut sc, Launch s) {
    if (Cin == 16) return launch_tc_s2<16>(dir, src, w, w_packed, dst, B, H, W, sc, s);
    if (Cin == 32) return launch_tc_s2<32>(dir, src, w, w_packed, dst, B, H, W, sc, s);
    return -1;
}
int launch_wgrad_tc_s2(const void *x, const void *dy, float *dw, float *scratch, int B, int H, int W, int Cin, Launch s) {
    if (Cin == 16) return launch_wg_s2<16>(x, dy, dw, scratch, B, H, W, s);
    if (Cin == 32) return launch_wg_s2<32>(x, dy, dw, scratch, B, H, W, s);
    return -1;
}

bool conv_tc_supported(int B, int H, int W, int Cin, int Cout, int stride) {
    if (!g_encode) return false;
    if (stride != 1 || Cin != Cout || (Cin != 16 && Cin != 32 && Cin != 64)) return false;
    if (W > 32 || 32 % W != 0) return false;  // a warp of the epilogue must hold whole image rows
    const int r = kTileM / W;
    if (r <= H) { if (H % r != 0) return false; }
    else { if (kTileM % (H * W) != 0 || B % (kTileM / (H * W)) != 0) return false; }
    return ((long)B * H * W) % kTileM == 0;
}

size_t tc_packed_bytes(int C) { return 2 * (size_t)9 * C * C * 2; }

int launch_conv_tc(int dir, const void *src, const void *w, const void *w_packed, void *dst, int B, int H, int W, int C,
                   Shortcut sc, Launch s, BnFuse bf, InXform xf) {
    switch (C) {
    case 16: return launch_tc<16>(dir, src, w, w_packed, dst, B, H, W, sc, bf, xf, s);
    case 32: return launch_tc<32>(dir, src, w, w_packed, dst, B, H, W, sc, bf, xf, s);
    case 64: return launch_tc<64>(dir, src, w, w_packed, dst, B, H, W, sc, bf, xf, s);
    }
    return -1;
}

bool conv_tc_xform_supported(int B, int H, int W, int C, bool shared) {
    if (!conv_tc_supported(B, H, W, C, C, 1)) return false;
    int rows, imgs;
    tile_geometry(H, W, &rows, &imgs);
    return tc_plan(C, (int)((long)B * H * W / kTileM), imgs == 1 ? 1 : 0, shared, true).threads <= 768;
}

bool conv_tc_xform_keeps_plan(int B, int H, int W, int C, bool shared) {
    if (!conv_tc_xform_supported(B, H, W, C, shared)) return false;
    int rows, imgs;
    tile_geometry(H, W, &rows, &imgs);
    const int n_tiles = (int)((long)B * H * W / kTileM), slab = imgs == 1 ? 1 : 0;
    const EpiPlan a = tc_plan(C, n_tiles, slab, shared, true).ep, b = tc_plan(C, n_tiles, slab, shared, false).ep;
    return a.n_pipes == b.n_pipes && a.n_acc == b.n_acc && a.n_slots == b.n_slots && a.split == b.split;
}

int conv_tc_grid(int B, int H, int W) {
    const int n_tiles = (int)((long)B * H * W / kTileM);
    return n_tiles < g_num_sms ? n_tiles : g_num_sms;
}

int launch_pack_filters(const void *wver, void *packed, const void *jobs_dev, int n_jobs, int total_elems,
                        Launch s) {
    if (n_jobs == 0) return 0;
    launch_k(pack_filters_kernel, ceil_div(total_elems, 256), 256, 0, s, (const bf16 *)wver, (uint8_t *)packed,
                                                                  (const PackJob *)jobs_dev, n_jobs, total_elems);
    return 1;
}

int launch_pack_one(const void *w, void *packed, int C, Launch s) {
    launch_k(pack_one_filter_kernel, ceil_div(9 * C * C, 256), 256, 0, s, (const bf16 *)w, (uint8_t *)packed, C);
    return 1;
}

bool wgrad_tc_supported(int B, int H, int W, int Cin, int Cout, int stride) {
    return conv_tc_supported(B, H, W, Cin, Cout, stride);
}
// the most partials any launch leaves: 2 x 148 chunks of 9 x 32 x 32 (paired 32-channel CTAs) = 148 chunks of 9 x 32 x 64
// (stride 2); 64 channels: 49 chunks
size_t wgrad_tc_scratch_elems() { return (size_t)2 * kWgMaxChunks * 9 * 32 * 32; }

int launch_wgrad_tc(const void *x, const void *dy, float *dw, float *scratch, int B, int H, int W, int C, int cin_real,
                    Launch s) {
    switch (C) {
    case 16: return launch_wg<16>(x, dy, dw, scratch, B, H, W, cin_real, s);
    case 32: return launch_wg<32>(x, dy, dw, scratch, B, H, W, cin_real, s);
    case 64: return launch_wg<64>(x, dy, dw, scratch, B, H, W, cin_real, s);
    }
    return -1;
}

PFN_cuTensorMapEncodeTiled_v12000 tc_encode_fn() { return g_encode; }
int *tc_err_word_of(const Launch &L) { return err_word_of(L); }

int conv_tc_error() {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(int)) != cudaSuccess) return -1;
    return v;
}

// A one-CTA kernel whose only work is a bounded wait on a barrier nothing ever arrives on: no TMA, no MMA, no TMEM.
// The wait gives up after `polls` polls, raises the error word with code 99 and the kernel returns.  It exists so that
// the path from a wait that ran out to the host's error status can be exercised without a stuck pipeline.
__global__ void wait_probe_kernel(int *err_word, unsigned polls) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    pdl_launch();
    pdl_wait();
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        const Waiter wt{&abort_flag, err_word, polls};
        mbar_wait(smem_u32(&bar), 0, wt, 99);
    }
}
int launch_wait_probe(unsigned polls, Launch s) {
    if (!g_tc_error_addr) return -1;
    launch_k(wait_probe_kernel, 1, 32, 0, s, err_word_of(s), polls);
    return 1;
}

int conv_tc_init() {
    static int rc = -1;
    if (rc >= 0) return rc;
    cudaDriverEntryPointQueryResult q;
    void *fn = nullptr;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) { cudaGetLastError(); rc = 0; return rc; }  // path stays off
    g_encode = (PFN_cuTensorMapEncodeTiled_v12000)fn;
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&g_num_sms, cudaDevAttrMultiProcessorCount, dev);
    {
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_tc_error);
        if (e != cudaSuccess) { rc = (int)e; return rc; }
        g_tc_error_addr = static_cast<int *>(p);
    }
    const void *fns[12] = {(const void *)conv3x3_tc_kernel<16>, (const void *)conv3x3_tc_kernel<32>,
                           (const void *)conv3x3_tc_kernel<64>, (const void *)wgrad_tc_kernel<16>,
                           (const void *)wgrad_tc_kernel<32>, (const void *)wgrad_tc_kernel<64>,
                           (const void *)conv3x3_s2_tc_kernel<16, 32, 0>, (const void *)conv3x3_s2_tc_kernel<32, 64, 0>,
                           (const void *)conv3x3_s2_tc_kernel<32, 16, 1>, (const void *)conv3x3_s2_tc_kernel<64, 32, 1>,
                           (const void *)wgrad_s2_tc_kernel<16>, (const void *)wgrad_s2_tc_kernel<32>};
    for (const void *f : fns) {
        e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemMax);
        if (e != cudaSuccess) break;
    }
    if (e == cudaSuccess) e = (cudaError_t)fc_tc_init();
    rc = (int)e;
    return rc;
}

}  // namespace ddg
