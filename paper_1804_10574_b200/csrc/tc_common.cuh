// Device-side building blocks shared by the tensor-core kernels (tcgen05 / TMEM / TMA on sm_100a): thin PTX wrappers,
// the bounded mbarrier wait, shared-memory matrix descriptors and the swizzled tile layouts.
#pragma once
#include <cuda.h>
#include <cudaTypedefs.h>
#include <stdint.h>

#include "common.cuh"

namespace ddg {

constexpr int kTileM = 128;
constexpr unsigned kSpinLimit = 1u << 24;  // bounded waits: ~ a second at worst, then the CTA gives up

// ---- thin PTX wrappers ---------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// One try: the thread may sleep inside the instruction for up to about `hint_ns` until the phase completes (it is woken
// when it does), so that a waiting warp issues few instructions and leaves the SM's shared-memory pipe to the others.
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity, uint32_t hint_ns = 300u) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false (and raises the error word and the CTA's abort flag) when the limit is hit.
struct Waiter {
    volatile int *abort_flag;  // shared memory: set by the first wait of the CTA that gives up, seen by the others
    int *err;                  // global memory: the error word the host reads at its next sync point
    unsigned limit;            // polls before a wait gives up
};
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const Waiter &wt, int code) {
    for (unsigned i = 0; i < wt.limit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 15u) == 15u && *wt.abort_flag) return false;
        if (i > 4096) __nanosleep(64);
    }
    *wt.abort_flag = 1;
    atomicCAS(wt.err, 0, code);
    return false;
}

__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], "
        "[%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}

// one 32-byte store (16 bf16 channels of a pixel): every 32-byte sector of the output is written whole, by one request
__device__ __forceinline__ void st_global_32(void *p, const uint32_t (&v)[8]) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"l"(p), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7])
                 : "memory");
}

// the matching 32-byte load, unpacked to 16 floats
__device__ __forceinline__ void ld_global_32(const bf16 *p, float (&f)[16]) {
    uint32_t v[8];
    asm volatile("ld.global.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "l"(p));
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        f[2 * k] = __uint_as_float(v[k] << 16);
        f[2 * k + 1] = __uint_as_float(v[k] & 0xffff0000u);
    }
}

__device__ __forceinline__ void prefetch_l1(const void *p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                            uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, "
        "[%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
#pragma unroll
    for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// 32 consecutive columns into two 16-value halves (one instruction: issuing a tcgen05.ld costs its warp ~70 ns)
__device__ __forceinline__ void tc_ld32(uint32_t taddr, float (&a)[16], float (&b)[16]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
          "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
          "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
#pragma unroll
    for (int i = 0; i < 16; ++i) { a[i] = __uint_as_float(r[i]); b[i] = __uint_as_float(r[16 + i]); }
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major (or MN-major) bf16 tile whose rows are one swizzle span wide
// (32, 64 or 128 bytes): 8-row groups are `sbo` bytes apart; the leading-dimension field is not used by these
// layouts and carries its canonical value 1.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t sbo_bytes, uint32_t layout_type,
                                              uint32_t lbo_bytes = 16) {
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3fff);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3fff) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3fff) << 32;
    d |= (uint64_t)1 << 46;  // descriptor version of this architecture
    d |= (uint64_t)layout_type << 61;
    return d;
}

constexpr int kMaxStages = 16;

template <int C> struct TcCfg {
    static constexpr int row_bytes = C * 2;                           // one pixel's channels = one swizzle span
    static constexpr uint32_t layout = C == 64 ? 2u : (C == 32 ? 4u : 6u);  // 128B / 64B / 32B swizzle
    static constexpr uint32_t swz_mask = C == 64 ? 7u : (C == 32 ? 3u : 1u);
    static constexpr int w_row_tile_bytes = 3 * C * C * 2;            // one filter row: [3C rows = (chunk, kx, out ch % 16)][C]
    static constexpr int w_bytes = 3 * w_row_tile_bytes;
    static constexpr int tile_bytes = kTileM * C * 2;
    static constexpr int acc_stages = 2;                              // TMEM accumulator stages of 3C columns each
    static constexpr int tmem_cols = C == 16 ? 128 : (C == 32 ? 256 : 512);  // 2 * 3C rounded up to a power of two
};

// byte offset of element (row, k) inside a swizzled tile whose rows are row_bytes wide
template <int C> __host__ __device__ __forceinline__ uint32_t swz_off(int row, int k) {
    uint32_t off = (uint32_t)row * TcCfg<C>::row_bytes + (uint32_t)k * 2;
    return off ^ (((off >> 7) & TcCfg<C>::swz_mask) << 4);
}

__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}


// ---- host side -------------------------------------------------------------------------------------------
// cuTensorMapEncodeTiled, resolved through the runtime by conv_tc_init (nullptr until then / when unavailable)
PFN_cuTensorMapEncodeTiled_v12000 tc_encode_fn();
// the error word a launch reports into: the context's own, or the process-wide one
int *tc_err_word_of(const Launch &L);

}  // namespace ddg
