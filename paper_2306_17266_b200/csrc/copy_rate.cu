// Stand-alone microbenchmark (not part of libsgs): rate of asynchronous copies into shared memory per SM.
// Tiled TMA boxes of 256 rows x 128 B (128-byte swizzle, rows 9 KB apart, the shape of a weight stage of
// the grouped convolution) against contiguous 32 KB bulk copies of the same tensor, which fits L2.
// One CTA per SM, one thread issues and keeps 4 copies in flight; every wait is bounded.
// Build and run: python -m paper_2306_17266_b200.microbench copy-rate
#include <cuda.h>
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdint>
#include <cstdlib>
#include <dlfcn.h>

__device__ __forceinline__ uint32_t s32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool try_wait(uint64_t *bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(s32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool wait_bounded(uint64_t *bar, uint32_t parity) {
    for (long long i = 0; i < 20000000; i++) if (try_wait(bar, parity)) return true;
    return false;
}
constexpr int STAGES = 4, BYTES = 32768;

template <int MODE>  // 0: tensor box 3D {64, 1, 256}; 1: bulk contiguous
__global__ void __launch_bounds__(32, 1) rate_kernel(const __grid_constant__ CUtensorMap map, const uint8_t *base, size_t span, int iters, int rows_total, unsigned long long *cycles, int *err) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t *smem = (uint8_t *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(8) uint64_t bar[STAGES];
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(s32(&bar[s])));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x != 0) return;
    const long long t0 = clock64();
    uint32_t phase[STAGES] = {0, 0, 0, 0};
    for (int i = 0; i < iters + STAGES; i++) {
        const int s = i % STAGES;
        if (i >= STAGES) {
            if (!wait_bounded(&bar[s], phase[s])) { *err = 1; return; }
            phase[s] ^= 1;
        }
        if (i < iters) {
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(&bar[s])), "r"(BYTES) : "memory");
            // every CTA walks its own region; consecutive copies are different data
            const unsigned blk = (unsigned)((blockIdx.x * 131u + (unsigned)i * 7u) % (unsigned)(rows_total / 256));
            if (MODE == 0) {
                asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
                             ::"r"(s32(smem + s * BYTES)), "l"(&map), "r"(s32(&bar[s])), "r"(0), "r"(0), "r"((int)(blk * 256)) : "memory");
            } else {
                asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                             ::"r"(s32(smem + s * BYTES)), "l"(base + (size_t)blk * 2359296), "r"(BYTES), "r"(s32(&bar[s])) : "memory");
            }
        }
    }
    cycles[blockIdx.x] = (unsigned long long)(clock64() - t0);
}

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int main(int argc, char **argv) {
    const int iters = 2000;
    // weights-like tensor: [rows][taps = 9][C = 512] bf16; a box takes 64 channels of one tap of 256 rows: row pitch 9 * 512 * 2 B
    const int rows_total = 8192, taps = 9, C = 512;
    const size_t bytes = (size_t)rows_total * taps * C * 2;  // 75 MB: fits L2
    uint8_t *d; cudaMalloc(&d, bytes); cudaMemset(d, 1, bytes);
    unsigned long long *cyc; cudaMalloc(&cyc, 148 * 8);
    int *err; cudaMalloc(&err, 4); cudaMemset(err, 0, 4);
    void *fn = nullptr; cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qr) != cudaSuccess || !fn) { printf("no encode\n"); return 1; }
    CUtensorMap map;
    cuuint64_t dims[3] = {(cuuint64_t)C, (cuuint64_t)taps, (cuuint64_t)rows_total};
    cuuint64_t str[2] = {(cuuint64_t)C * 2, (cuuint64_t)taps * C * 2};
    cuuint32_t box[3] = {64, 1, 256}, es[3] = {1, 1, 1};
    CUresult r = ((EncodeFn)fn)(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, d, dims, str, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { printf("encode failed %d\n", (int)r); return 1; }
    const int smem = STAGES * BYTES + 1024;
    cudaFuncSetAttribute(rate_kernel<0>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    cudaFuncSetAttribute(rate_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    for (int ctas : {1, 32, 148}) {
        for (int mode = 0; mode < 2; mode++) {
            for (int rep = 0; rep < 2; rep++) {
                if (mode == 0) rate_kernel<0><<<ctas, 32, smem>>>(map, d, bytes, iters, rows_total, cyc, err);
                else rate_kernel<1><<<ctas, 32, smem>>>(map, d, bytes, iters, rows_total, cyc, err);
                cudaError_t e = cudaDeviceSynchronize();
                if (e != cudaSuccess) { printf("cuda error %s\n", cudaGetErrorString(e)); return 1; }
            }
            unsigned long long h[148]; int he = 0;
            cudaMemcpy(h, cyc, ctas * 8, cudaMemcpyDeviceToHost); cudaMemcpy(&he, err, 4, cudaMemcpyDeviceToHost);
            double mx = 0; for (int i = 0; i < ctas; i++) mx = h[i] > mx ? (double)h[i] : mx;
            printf("ctas %3d mode %s: %.1f B/clk/SM (%.0f clk per 32 KB copy)%s\n", ctas, mode ? "bulk-contiguous" : "tensor-256rows", (double)iters * BYTES / mx, mx / iters, he ? " WAIT RAN OUT" : "");
        }
    }
    return 0;
}
