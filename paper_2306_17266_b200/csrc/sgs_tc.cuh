// Device-side building blocks shared by the tensor-core convolution kernels: PTX wrappers for
// mbarriers, TMA tensor copies and tcgen05 (allocation, MMA, commit, tensor-memory loads), the
// shared-memory matrix descriptor of the 128-byte-swizzled K-major tiles, and the fused epilogue.
#pragma once

#include "sgs_internal.h"

namespace sgs {

constexpr int TILE_M = 128;   // output pixels per CTA (TMEM lanes)
constexpr int CHUNK_C = 64;   // channels per pipeline stage (64 bf16 = one 128-byte swizzle row)
constexpr int A_STAGE_BYTES = TILE_M * CHUNK_C * 2;
constexpr unsigned long long WAIT_LIMIT_NS = 2000000000ull;  // 2 s per wait

struct TcParams {
    CUtensorMap tmA[4];  // activation views: [0] stride 1, or [ph*2+pw] parity views for stride 2
    CUtensorMap tmW;     // sliced weight view (C', R*R, K')
    const float *scale, *shift;
    const __nv_bfloat16 *res;
    __nv_bfloat16 *y;
    float *ws;               // split-K workspace: [splits][M][K] fp32 partial tiles
    size_t slice;            // M*K, elements of one workspace slice
    int *status;             // device status word: nonzero after a bounded wait ran out
    int N, Ho, Wo, K, C;     // output dims, sliced filters, sliced channels
    int k, stride, R, o, p;  // kernel size, stride, stored kernel size, crop offset, padding
    int bw, bh, bn;          // tile box in output pixels
    int tiles_w, tiles_h;    // tiles along w and h (tiles along n = gridDim.x / (tiles_w*tiles_h))
    int cchunks, iters;      // channel chunks per tap, total pipeline iterations (k*k*cchunks)
    int splits, act;
    int cacheK, cacheC, weight_policy;
    const int *cache_tbl;    // optional device table overriding the three values above (see ConvArgs)
    int layer;
    // int8 layers (8-bit operands, int32 accumulator): per-filter requantisation parameters and the integer epilogue
    //   v = rshift_round(acc * q_mult[f], 31 + q_shift[f]) + q_bias[f] + rshift_round((res - q_zr) * q_res_mult, 31 + q_res_shift) + q_zy
    const int *q_mult, *q_shift, *q_bias;
    int q_zy, q_zr, q_res_mult, q_res_shift;
    int q_flags;             // bit 0: x signed, bit 1: y signed, bit 2: res signed, bit 3: ReLU (max with q_zy)
    int q_ldy;               // bytes per pixel of y and res (>= K; the bytes beyond K are written as zeros)
};

namespace {

// ---------------------------------------------------------------------------------------------
// PTX wrappers
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: false if the phase did not complete within limit_ns or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag,
                                          unsigned long long limit_ns = WAIT_LIMIT_NS) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    for (;;) {
        for (int i = 0; i < 64; i++)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (global_ns() - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
}
__device__ __forceinline__ uint64_t make_policy(int kind) {  // 0 normal, 1 evict-last, 2 evict-first
    uint64_t pol;
    if (kind == 1) asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    else if (kind == 2) asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    else asm volatile("createpolicy.fractional.L2::evict_normal.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_4d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2,
                                            int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "r"(c3)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d_hint(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%3, %4, %5}], "
        "[%2], %6;"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(void *dst, const CUtensorMap *map, uint64_t *bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
// A tensor map that lives in global memory and was written by the host (cudaMemcpy) must be acquired
// by the thread that is going to use it, before its first use in that thread.
__device__ __forceinline__ void tensormap_acquire(const CUtensorMap *map) {
    asm volatile("fence.proxy.tensormap::generic.acquire.sys [%0], 128;" ::"l"(map) : "memory");
}
// True in exactly one lane of a converged warp (the same lane every time).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred P;\n\t"
        "elect.sync _|P, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, P;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
// Programmatic dependent launch: wait() returns once the grids this one depends on have completed and
// their writes are visible; launch_dependents() lets the next grid in the stream start its own prologue
// early.  Both are no-ops for a grid that was launched without the attribute.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(uint32_t *dst_smem, uint32_t cols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t cols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(cols) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 8-bit operands (signedness in the instruction descriptor), int32 accumulator; K = 32 per instruction
__device__ __forceinline__ void umma_i8(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t *v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t *v) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes with the 128-byte
// swizzle: start address >> 4, leading offset 1 (unused for swizzled K-major), stride offset
// 1024 B (8 rows) >> 4, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr) {
    return (uint64_t)((saddr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ float act_fn(float v, int act) {
    if (act == ACT_RELU) return fmaxf(v, 0.f);
    if (act == ACT_HSWISH) return v * fminf(fmaxf(v + 3.f, 0.f), 6.f) * (1.f / 6.f);
    return v;
}

// Residual, activation and bf16 store of 8 consecutive filters of one pixel (o already holds
// accumulator * scale + shift).
__device__ __forceinline__ void finish_store(float *o, const __nv_bfloat16 *res, __nv_bfloat16 *y, size_t oi, int act) {
    if (res) {
        uint4 rv = *reinterpret_cast<const uint4 *>(res + oi);
        const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv);
#pragma unroll
        for (int j = 0; j < 4; j++) { float2 t = __bfloat1622float2(rb[j]); o[2 * j] += t.x; o[2 * j + 1] += t.y; }
    }
    uint4 ov;
    __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
    for (int j = 0; j < 4; j++) ob[j] = __floats2bfloat162_rn(act_fn(o[2 * j], act), act_fn(o[2 * j + 1], act));
    *reinterpret_cast<uint4 *>(y + oi) = ov;
}

}  // namespace

// Rounding right shift of the integer epilogue: floor((v + 2^(s-1)) / 2^s), 1 <= s <= 62 (ties go up).
__host__ __device__ __forceinline__ long long rshift_round(long long v, int s) { return (v + (1ll << (s - 1))) >> s; }

struct TcConvPlan {
    TcParams prm;
    int i8 = 0;          // 8-bit operands: 128 channels per stage, 32 per MMA
    dim3 grid;
    int bn_tile = 128;   // filters per tile
    int swap = 0;        // grouped launches only: filters on the MMA's row side, all pixels on the column side
    int kw = 1;          // taps along x (k for square kernels, 1 for the window view of a stem)
    size_t ws_elems = 0;
};

}  // namespace sgs
