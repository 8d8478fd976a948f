// Fully connected layers on the tensor cores (sm_100a): bf16 operands fetched by TMA, tcgen05 MMAs with fp32
// accumulators in TMEM, bias / ReLU / masking in the epilogue.  Eq. 3 (forward) and Eq. 4-5 / Eq. 6-7 (backward) for
// h = x W^T + b.
//
//   forward   y[b][o]  = sum_i x[b][i] W[o][i] + bias[o]            M = 128 batch rows, N = out (padded to 16), K = in
//   dx        dx[b][i] = sum_o dz[b][o] W[o][i]                      M = 128 batch rows, N = in, K = out (padded to 16)
//   dW        dW[o][i] = sum_b dz[b][o] x[b][i]                      M = out (<= 128), N = in, K = batch (128 per tile)
//   db        db[o]    = sum_b dz[b][o]                              plain sums (a few thousand values)
// with dz = dy * [y > 0] where the layer has a ReLU.
//
// x [B][in] and W [out][in] are row-major with the contraction axis of the forward pass innermost, so TMA boxes of 64
// columns (one 128-byte swizzle row) feed the forward MMAs as K-major operands directly.  The backward pass reads the
// SAME shared-memory images the other way round: W as an MN-major B operand for dx (N = in runs along the rows' bytes,
// K = out across rows), x as an MN-major B operand for dW (K = batch across rows).  dz is built by the CTA itself in
// 16-column slabs [128 batch rows][16 outputs] of 32-byte rows: a slab is a K-major A tile for dx (K = its 16 outputs)
// and, read across rows, an MN-major A tile for dW (M = its 16 outputs, K = batch).  An fp32 dy (the loss gradient of the
// last layer) is split into two bf16 terms, dz = hi + lo, multiplied one after the other into the same accumulator, so
// that the tensor-core path keeps ~16 mantissa bits of the loss gradient instead of 8.
// One CTA of four warps per 128 batch rows in the forward pass; one CTA walks all batch tiles in the backward pass
// (dW accumulates over them in TMEM).  These layers are a few MFLOP: the kernels are not pipelined.
#include <map>
#include <mutex>
#include <tuple>

#include "common.cuh"
#include "conv_tc.h"
#include "tc_common.cuh"

namespace ddg {

namespace {

constexpr int kFcThreads = 128;
constexpr int kFcKBox = 64;                      // columns of a TMA box: 128 bytes, one swizzle row
constexpr int kFcXBlock = kTileM * kFcKBox * 2;  // bytes of one [128][64] bf16 block
constexpr int kFcSlab = kTileM * 16 * 2;         // bytes of one dz slab [128][16]
constexpr int kFcDzPart = 8 * kFcSlab;           // eight slabs: all 128 rows of the dW accumulator

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTileM >> 4) << 24);  // fp32 += bf16 x bf16, M = 128

__device__ __forceinline__ void tmem_alloc(uint32_t *holder, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(holder)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t base, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(base), "r"(cols) : "memory");
}

// ---- forward ----------------------------------------------------------------------------------------------
template <typename TO>
__global__ void __launch_bounds__(kFcThreads, 1)
fc_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                 const bf16 *__restrict__ bias, TO *__restrict__ y, int B, int in, int out, int n_pad, int relu,
                 int tmem_cols, int *__restrict__ err_word) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[2];  // operands landed, accumulator complete
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    const int kb = in / kFcKBox;
    const uint32_t x_base = base, w_base = base + (uint32_t)kb * kFcXBlock;
    const uint32_t w_block = (uint32_t)n_pad * 128u;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Waiter wt{&abort_flag, err_word, kSpinLimit};
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bars[0]), 1);
        mbar_init(smem_u32(&bars[1]), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_holder, (uint32_t)tmem_cols);
    pdl_launch();
    pdl_wait();  // nothing above touches global memory
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;
    const int row0 = blockIdx.x * kTileM;
    const uint32_t ld_bar = smem_u32(&bars[0]), mma_bar = smem_u32(&bars[1]);
    if (threadIdx.x == 0) {
        mbar_expect_tx(ld_bar, (uint32_t)kb * (kFcXBlock + w_block));
        for (int j = 0; j < kb; ++j) {
            tma_load_2d(x_base + j * kFcXBlock, &tmap_x, ld_bar, j * kFcKBox, row0);  // rows >= B: zero fill
            tma_load_2d(w_base + j * w_block, &tmap_w, ld_bar, j * kFcKBox, 0);       // rows >= out: zero fill
        }
        if (mbar_wait(ld_bar, 0, wt, 41)) {
            tc_fence_after();
            const uint32_t idesc = kIdescBase | ((uint32_t)(n_pad >> 3) << 17);
            for (int j = 0; j < kb; ++j) {
                const uint64_t adesc = make_desc(x_base + j * kFcXBlock, 1024, 2u);
                const uint64_t bdesc = make_desc(w_base + j * w_block, 1024, 2u);
#pragma unroll
                for (int k = 0; k < kFcKBox / 16; ++k) tc_mma_bf16(tmem_base, adesc + 2 * k, bdesc + 2 * k, idesc, (j | k) != 0);
            }
            tc_commit(mma_bar);
        } else {
            for (int i = 0; i < 2000; ++i) __nanosleep(100);  // let copies in flight land before the CTA can exit
        }
    }
    __syncwarp();
    bool ok = mbar_wait(mma_bar, 0, wt, 42);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
        tc_fence_after();
        const int b = row0 + 32 * warp + lane;
        for (int c0 = 0; c0 < n_pad; c0 += 16) {
            float v[16];
            tc_ld16(tmem_base + ((uint32_t)(32 * warp) << 16) + (uint32_t)c0, v);
            tc_wait_ld();
            if (b < B) {
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int o = c0 + j;
                    if (o < out) {
                        float t = v[j] + (bias != nullptr ? to_f(bias[o]) : 0.f);
                        if (relu && t < 0.f) t = 0.f;
                        y[(size_t)b * out + o] = from_f<TO>(t);
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_free(tmem_base, (uint32_t)tmem_cols); }
}

// ---- backward ---------------------------------------------------------------------------------------------
// TO: element type of y and dy (float for the last layer, whose dy is the loss gradient; bf16 for hidden layers).
// parts = 2: dz is split into two bf16 terms.  dx == nullptr: the layer is the network's first, only dW / db.
template <typename TO>
__global__ void __launch_bounds__(kFcThreads, 1)
fc_bwd_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                 const TO *__restrict__ y, const TO *__restrict__ dy, bf16 *__restrict__ dx, float *__restrict__ dW,
                 float *__restrict__ db, int B, int in, int out, int k_pad, int relu, int parts, int tmem_cols,
                 int *__restrict__ err_word) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bars[3];  // W landed, x tile landed, MMAs of the tile done
    __shared__ uint32_t tmem_holder;
    __shared__ int abort_flag;
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    uint8_t *smem = smem_raw + (base - raw);
    const int nb = in / kFcKBox;
    const uint32_t w_block = (uint32_t)k_pad * 128u;
    const uint32_t x_base = base, w_base = x_base + (uint32_t)nb * kFcXBlock, dz_base = w_base + (uint32_t)nb * w_block;
    uint8_t *dz_smem = smem + (dz_base - base);
    const uint32_t w_bar = smem_u32(&bars[0]), x_bar = smem_u32(&bars[1]), mma_bar = smem_u32(&bars[2]);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Waiter wt{&abort_flag, err_word, kSpinLimit};
    if (threadIdx.x == 0) {
        mbar_init(w_bar, 1); mbar_init(x_bar, 1); mbar_init(mma_bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_holder, (uint32_t)tmem_cols);
    pdl_launch();
    pdl_wait();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_holder;
    const uint32_t acc_dx = tmem_base, acc_dw = tmem_base + (uint32_t)in;
    const int n_tiles = (B + kTileM - 1) / kTileM;
    if (threadIdx.x == 0 && dx != nullptr) {
        mbar_expect_tx(w_bar, (uint32_t)nb * w_block);
        for (int j = 0; j < nb; ++j) tma_load_2d(w_base + j * w_block, &tmap_w, w_bar, j * kFcKBox, 0);
    }
    bool ok = true;
    for (int tile = 0; tile < n_tiles && ok; ++tile) {
        const int row0 = tile * kTileM;
        const uint32_t ph = (uint32_t)tile & 1u;
        if (threadIdx.x == 0) {
            mbar_expect_tx(x_bar, (uint32_t)nb * kFcXBlock);
            for (int j = 0; j < nb; ++j) tma_load_2d(x_base + j * kFcXBlock, &tmap_x, x_bar, j * kFcKBox, row0);
        }
        {   // dz of batch row r = threadIdx.x: eight slabs of 16 outputs, zero beyond out and beyond the batch
            const int r = threadIdx.x, b = row0 + r;
            for (int s = 0; s < 8; ++s) {
                uint32_t hi[8], lo[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    float d[2];
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int o = 16 * s + 2 * j + h;
                        float t = 0.f;
                        if (b < B && o < out) {
                            t = to_f(dy[(size_t)b * out + o]);
                            if (relu && !(to_f(y[(size_t)b * out + o]) > 0.f)) t = 0.f;
                        }
                        d[h] = t;
                    }
                    const __nv_bfloat162 h2 = __floats2bfloat162_rn(d[0], d[1]);
                    hi[j] = *reinterpret_cast<const uint32_t *>(&h2);
                    const __nv_bfloat162 l2 = __floats2bfloat162_rn(d[0] - __low2float(h2), d[1] - __high2float(h2));
                    lo[j] = *reinterpret_cast<const uint32_t *>(&l2);
                }
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    const uint32_t off = (uint32_t)s * kFcSlab + swz_off<16>(r, 8 * half);
                    *reinterpret_cast<uint4 *>(dz_smem + off) = make_uint4(hi[4 * half], hi[4 * half + 1], hi[4 * half + 2], hi[4 * half + 3]);
                    if (parts == 2)
                        *reinterpret_cast<uint4 *>(dz_smem + kFcDzPart + off) =
                            make_uint4(lo[4 * half], lo[4 * half + 1], lo[4 * half + 2], lo[4 * half + 3]);
                }
            }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
        __syncthreads();
        if (threadIdx.x == 0) {
            bool go = true;
            if (tile == 0 && dx != nullptr) go = mbar_wait(w_bar, 0, wt, 43);
            if (go) go = mbar_wait(x_bar, ph, wt, 44);
            if (go) {
                tc_fence_after();
                if (dx != nullptr) {
                    // dx: A = dz slabs, K-major; B = W blocks read MN-major (N = in along the bytes of a row, next 64
                    // columns one block further), 16 rows (outputs) per instruction
                    const uint32_t idesc = kIdescBase | (1u << 16) | ((uint32_t)(in >> 3) << 17);
                    int first = 1;
                    for (int p = 0; p < parts; ++p)
                        for (int s = 0; s < k_pad / 16; ++s) {
                            const uint64_t adesc = make_desc(dz_base + p * kFcDzPart + s * kFcSlab, 256, 6u);
                            const uint64_t bdesc = make_desc(w_base + s * 16 * 128, 1024, 2u, w_block);
                            tc_mma_bf16(acc_dx, adesc, bdesc, idesc, first ? 0u : 1u);
                            first = 0;
                        }
                }
                {
                    // dW: A = dz read MN-major (M = outputs: 16 per slab, next slab 4 KB further), B = x blocks read
                    // MN-major, 16 batch rows per instruction; accumulates over all tiles
                    const uint32_t idesc = kIdescBase | (1u << 15) | (1u << 16) | ((uint32_t)(in >> 3) << 17);
                    for (int p = 0; p < parts; ++p)
                        for (int k = 0; k < kTileM / 16; ++k) {
                            const uint64_t adesc = make_desc(dz_base + p * kFcDzPart + k * 16 * 32, 256, 6u, kFcSlab);
                            const uint64_t bdesc = make_desc(x_base + k * 16 * 128, 1024, 2u, kFcXBlock);
                            tc_mma_bf16(acc_dw, adesc, bdesc, idesc, (tile | p | k) != 0 ? 1u : 0u);
                        }
                }
                tc_commit(mma_bar);
            } else {
                for (int i = 0; i < 2000; ++i) __nanosleep(100);
            }
        }
        __syncwarp();
        ok = mbar_wait(mma_bar, ph, wt, 45);
        ok = __syncthreads_and(ok ? 1 : 0) != 0;
        if (!ok) break;
        tc_fence_after();
        if (dx != nullptr) {
            const int b = row0 + 32 * warp + lane;
            for (int c0 = 0; c0 < in; c0 += 16) {
                float v[16];
                tc_ld16(acc_dx + ((uint32_t)(32 * warp) << 16) + (uint32_t)c0, v);
                tc_wait_ld();
                if (b < B) {
                    store_f<bf16, 8>(dx + (size_t)b * in + c0, reinterpret_cast<const float(&)[8]>(v[0]));
                    store_f<bf16, 8>(dx + (size_t)b * in + c0 + 8, reinterpret_cast<const float(&)[8]>(v[8]));
                }
            }
        }
        tc_fence_before();
        __syncthreads();  // the next tile's MMAs overwrite the dx accumulator and the dz / x images
    }
    if (ok) {
        tc_fence_after();
        const int o = 32 * warp + lane;
        for (int c0 = 0; c0 < in; c0 += 16) {
            float v[16];
            tc_ld16(acc_dw + ((uint32_t)(32 * warp) << 16) + (uint32_t)c0, v);
            tc_wait_ld();
            if (o < out) {
                float4 *o4 = reinterpret_cast<float4 *>(dW + (size_t)o * in + c0);
#pragma unroll
                for (int j = 0; j < 4; ++j) o4[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            }
        }
        if (db != nullptr && o < out) {  // bias gradient: batch rows in index order
            float acc = 0.f;
            for (int b = 0; b < B; ++b) {
                float t = to_f(dy[(size_t)b * out + o]);
                if (relu && !(to_f(y[(size_t)b * out + o]) > 0.f)) t = 0.f;
                acc += t;
            }
            db[o] = acc;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) { tc_fence_after(); tmem_free(tmem_base, (uint32_t)tmem_cols); }
}

// ---- host side --------------------------------------------------------------------------------------------
struct Map2Key {
    const void *ptr; int rows, cols, box_rows;
    bool operator<(const Map2Key &o) const { return std::tie(ptr, rows, cols, box_rows) < std::tie(o.ptr, o.rows, o.cols, o.box_rows); }
};
std::map<Map2Key, CUtensorMap> g_maps2;
std::mutex g_maps2_mu;

// Tensor map of a row-major bf16 matrix [rows][cols] with a box of (64 columns, box_rows rows), 128-byte swizzle,
// zero fill outside the matrix.
bool get_map_2d(const void *ptr, int rows, int cols, int box_rows, CUtensorMap *out) {
    PFN_cuTensorMapEncodeTiled_v12000 enc = tc_encode_fn();
    if (!enc) return false;
    std::lock_guard<std::mutex> lock(g_maps2_mu);
    Map2Key key{ptr, rows, cols, box_rows};
    auto it = g_maps2.find(key);
    if (it != g_maps2.end()) { *out = it->second; return true; }
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)kFcKBox, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUtensorMap m;
    CUresult r = enc(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    if (g_maps2.size() > 2048) g_maps2.clear();
    g_maps2[key] = m;
    *out = m;
    return true;
}

int pad16(int v) { return (v + 15) / 16 * 16; }
int pow2_cols(int need) { int c = 32; while (c < need) c <<= 1; return c; }
size_t fwd_smem(int in, int out) { return 1024 + (size_t)(in / kFcKBox) * (kFcXBlock + (size_t)pad16(out) * 128); }
size_t bwd_smem(int in, int out, int parts) {
    return 1024 + (size_t)(in / kFcKBox) * (kFcXBlock + (size_t)pad16(out) * 128) + (size_t)parts * kFcDzPart;
}
constexpr size_t kFcSmemMax = 227 * 1024 - 256;  // the kernels' static shared memory comes on top

}  // namespace

bool fc_tc_shape_supported(int B, int in, int out) {
    if (!tc_encode_fn()) return false;
    if (B < 1 || in < kFcKBox || in % kFcKBox != 0 || in > 256 || out < 1 || out > 128) return false;
    return bwd_smem(in, out, 2) <= kFcSmemMax && fwd_smem(in, out) <= kFcSmemMax;
}

bool fc_tc_supported(const void *x, const void *W, int B, int in, int out) {
    // TMA reads x and W in place: both must start on a 16-byte boundary (their rows are in * 2 bytes, a multiple of 128)
    return fc_tc_shape_supported(B, in, out) && (reinterpret_cast<uintptr_t>(x) & 15) == 0 && (reinterpret_cast<uintptr_t>(W) & 15) == 0;
}

int launch_fc_fwd_tc(const void *x, const void *W, const void *bias, void *y, int B, int in, int out, int relu, int out_f32,
                     Launch s) {
    const int n_pad = pad16(out);
    CUtensorMap mx, mw;
    if (!get_map_2d(x, B, in, kTileM, &mx) || !get_map_2d(W, out, in, n_pad, &mw)) return -1;
    const int cols = pow2_cols(n_pad);
    const int grid = (B + kTileM - 1) / kTileM;
    if (out_f32)
        launch_k(fc_fwd_tc_kernel<float>, grid, kFcThreads, fwd_smem(in, out), s, mx, mw, (const bf16 *)bias, (float *)y, B, in, out,
                 n_pad, relu, cols, tc_err_word_of(s));
    else
        launch_k(fc_fwd_tc_kernel<bf16>, grid, kFcThreads, fwd_smem(in, out), s, mx, mw, (const bf16 *)bias, (bf16 *)y, B, in, out,
                 n_pad, relu, cols, tc_err_word_of(s));
    return 1;
}

int launch_fc_bwd_tc(const void *x, const void *W, const void *y, const void *dy, void *dx, float *dW, float *db, int B,
                     int in, int out, int relu, int out_f32, Launch s) {
    const int k_pad = pad16(out);
    CUtensorMap mx, mw;
    if (!get_map_2d(x, B, in, kTileM, &mx) || !get_map_2d(W, out, in, k_pad, &mw)) return -1;
    const int parts = out_f32 ? 2 : 1;
    const int cols = pow2_cols(2 * in);
    if (out_f32)
        launch_k(fc_bwd_tc_kernel<float>, 1, kFcThreads, bwd_smem(in, out, parts), s, mx, mw, (const float *)y, (const float *)dy,
                 (bf16 *)dx, dW, db, B, in, out, k_pad, relu, parts, cols, tc_err_word_of(s));
    else
        launch_k(fc_bwd_tc_kernel<bf16>, 1, kFcThreads, bwd_smem(in, out, parts), s, mx, mw, (const bf16 *)y, (const bf16 *)dy,
                 (bf16 *)dx, dW, db, B, in, out, k_pad, relu, parts, cols, tc_err_word_of(s));
    return 1;
}

int fc_tc_init() {
    const void *fns[4] = {(const void *)fc_fwd_tc_kernel<float>, (const void *)fc_fwd_tc_kernel<bf16>,
                          (const void *)fc_bwd_tc_kernel<float>, (const void *)fc_bwd_tc_kernel<bf16>};
    for (const void *f : fns) {
        cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024 - 256);
        if (e != cudaSuccess) return (int)e;
    }
    return 0;
}

}  // namespace ddg
