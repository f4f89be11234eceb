// Sliced convolution as an implicit GEMM on the 5th-generation tensor cores (tcgen05) of sm_100a.
//
//   D[m][f] = sum_{r,s} sum_{c<C'} x[n][ho*st + r - p][wo*st + s - p][c] * w[f][o+r][o+s][c],  f < K'
//
// GEMM view: M = output pixels (128 TMEM lanes per CTA), N = output filters (BN columns), K = taps x
// channels.  Operands are staged in shared memory by TMA with the 128-byte swizzle; the accumulator
// lives in tensor memory; an epilogue applies the folded batch norm, residual and activation and
// stores bf16 NHWC.
//
// Slicing is folded into the TMA descriptors (paper Section 2.1: a SubNet only *selects* weights of
// the SuperNet; Section 1: no SubNet is extracted): the weight map has the extents (C', R*R, K') of
// the slice and the strides of the stored [Kmax][R][R][Cmax] tensor, so a tile that overhangs the
// slice is zero-filled by the hardware and no sliced copy of a weight exists anywhere.
//
// Activation tiles are rectangular boxes (bw x bh x bn output pixels, <= 128) fetched per filter tap
// with shifted box coordinates; image borders are the hardware's out-of-bounds zero fill.  Stride 2
// reads one of four "parity" views of the input (even/odd rows x even/odd columns), each a plain
// tensor map with doubled strides.
//
// SubGraph-Stationary reuse (paper Section 2.2, Section 4.2 Persistent / Dynamic Buffer): weight tiles
// inside the cached SubGraph's prefix box (filter < cacheK and channel < cacheC) are loaded with an
// L2 evict-last policy so that the shared weights stay on chip across queries; the distinct weights
// of each SubNet take the default replacement.
//
// Warp roles (192 threads): warp 0 = TMA producer, warp 1 = MMA issuer and TMEM owner, warps 2..5 =
// epilogue (one TMEM lane quadrant each).  Every wait is bounded; when one runs out the kernel sets
// a status word, lets its in-flight copies land, frees its tensor memory and returns.
#include "sgs_tc.cuh"

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <unordered_map>

namespace sgs {

namespace {

// ---------------------------------------------------------------------------------------------
// The kernel.  grid = (m tiles, n tiles, K splits), block = 192.
// Dynamic shared memory (1024-byte aligned): STAGES x [A tile 16 KB | B tile BN*128 B].
// ---------------------------------------------------------------------------------------------
template <int BN, int STAGES, bool I8>
__global__ void __launch_bounds__(192, 1) conv_tc_kernel(const __grid_constant__ TcParams p) {
    // (a stage row is 128 bytes either way: 64 bf16 or 128 8-bit channels; an MMA takes 32 bytes of it)
    constexpr int CH = I8 ? 2 * CHUNK_C : CHUNK_C, KS = I8 ? 32 : 16;
    constexpr int B_STAGE_BYTES = BN * CHUNK_C * 2;
    constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    __shared__ int row_m[TILE_M];  // output pixel index of each tile row, -1 outside the tensor
    __shared__ __align__(8) uint64_t full_bar[STAGES], empty_bar[STAGES], accum_bar;
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;
    __shared__ float scale_s[BN], shift_s[BN];  // folded batch norm (8-bit layers: multiplier and shift as integers, plus the bias)
    __shared__ int bias_s[I8 ? BN : 1];

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    volatile int *abort_flag = &abort_s;

    // tile coordinates
    const int tiles_hw = p.tiles_w * p.tiles_h;
    const int tn = blockIdx.x / tiles_hw, th = (blockIdx.x % tiles_hw) / p.tiles_w, tw = blockIdx.x % p.tiles_w;
    const int n0 = tn * p.bn, h0 = th * p.bh, w0 = tw * p.bw;
    const int f0 = blockIdx.y * BN;
    // MMA shape: M = 128, N = this tile's filters rounded up to 16, bf16 x bf16 -> fp32, both K-major
    const int n_mma = min(BN, (p.K - f0 + 15) & ~15);
    // instruction descriptor: accumulator format (1 fp32, 2 int32) at bit 4, A / B formats at bits 7 / 10 (bf16 = 1;
    // 8-bit: 0 unsigned, 1 signed), N >> 3 at bit 17, M >> 4 at bit 24; both operands K-major
    const uint32_t IDESC = I8 ? ((2u << 4) | ((uint32_t)(p.q_flags & 1) << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24))
                              : ((1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24));
    // K range of this split
    const int per = (p.iters + p.splits - 1) / p.splits;
    const int it_begin = blockIdx.z * per, it_end = min(p.iters, it_begin + per);
    const int n_it = max(0, it_end - it_begin);

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; s++) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        mbar_init(&accum_bar, 1);
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_base_s, BN);
    if (warp >= 2) {
        for (int j = threadIdx.x - 64; j < BN; j += 128) {
            int f = f0 + j;
            if (I8) {
                reinterpret_cast<int *>(scale_s)[j] = f < p.K ? p.q_mult[f] : 0;
                reinterpret_cast<int *>(shift_s)[j] = f < p.K ? min(max(p.q_shift[f], 0), 31) : 0;  // (0..31 by contract)
                bias_s[I8 ? j : 0] = f < p.K ? p.q_bias[f] : 0;
            } else {
                scale_s[j] = f < p.K ? p.scale[f] : 0.f;
                shift_s[j] = f < p.K ? p.shift[f] : 0.f;
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    pdl_launch_dependents();  // the next layer may start its prologue and its weight loads now

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        // The whole warp runs the loop converged, so every operand of the copy instructions is a
        // warp-uniform value; only the copy instructions themselves are issued by one elected lane.
        const uint64_t pol_keep = make_policy(1), pol_stream = make_policy(2);
        const uint32_t tx = (uint32_t)(p.bw * p.bh * p.bn * CHUNK_C * 2 + B_STAGE_BYTES);
        int weight_policy = p.weight_policy, cacheK = p.cacheK, cacheC = p.cacheC;
        if (p.cache_tbl) {
            weight_policy = __ldg(p.cache_tbl);
            cacheK = __ldg(p.cache_tbl + 1 + 2 * p.layer);
            cacheC = __ldg(p.cache_tbl + 2 + 2 * p.layer);
        }
        // (tap row r, tap column sx, channel chunk cc) of iteration it_begin, then stepped
        int cc = it_begin % p.cchunks, tap = it_begin / p.cchunks;
        int r = tap / p.k, sx = tap % p.k;
        auto load_weights = [&](int s, int c0, int tapw) {
            uint8_t *sb = smem + s * STAGE_BYTES + A_STAGE_BYTES;
            mbar_expect_tx(&full_bar[s], tx);
            // policy 1: tiles of the cached SubGraph are kept (evict-last), the rest take the default
            // replacement (measured: marking them evict-first loses to plain LRU whenever the SuperNet
            // fits in L2); policy 2: everything evict-first (the "no reuse at all" reference point)
            const bool in_box = weight_policy == 1 && f0 < cacheK && c0 < cacheC;
            if (weight_policy == 2) tma_load_3d_hint(sb, &p.tmW, &full_bar[s], c0, tapw, f0, pol_stream);
            else if (in_box) tma_load_3d_hint(sb, &p.tmW, &full_bar[s], c0, tapw, f0, pol_keep);
            else tma_load_3d(sb, &p.tmW, &full_bar[s], c0, tapw, f0);
        };
        // Weights do not depend on the previous layer: fill the first stages' weight halves before
        // waiting for it, so that their latency overlaps the previous layer's tail.
        {
            int cc2 = cc, r2 = r, sx2 = sx;
            const int pre = min(n_it, STAGES);
            for (int i = 0; i < pre; i++) {
                if (elect_one()) load_weights(i, cc2 * CH, (p.o + r2) * p.R + (p.o + sx2));
                __syncwarp();
                if (++cc2 == p.cchunks) { cc2 = 0; if (++sx2 == p.k) { sx2 = 0; ++r2; } }
            }
        }
        pdl_wait();  // activations (and the buffers this layer overwrites) belong to the previous layers until here
        for (int i = 0; i < n_it; i++) {
            const int s = i % STAGES, round = i / STAGES;
            bool ok = round == 0 || mbar_wait(&empty_bar[s], (round - 1) & 1, abort_flag);
            if (!__all_sync(0xffffffffu, ok)) break;
            const int c0 = cc * CH;
            uint8_t *sa = smem + s * STAGE_BYTES;
            const int dh = r - p.p, dw = sx - p.p;
            if (elect_one()) {
                if (round > 0) load_weights(s, c0, (p.o + r) * p.R + (p.o + sx));
                if (p.stride == 1) {
                    tma_load_4d(sa, &p.tmA[0], &full_bar[s], c0, w0 + dw, h0 + dh, n0);
                } else {
                    const int ph = dh & 1, pw = dw & 1;
                    tma_load_4d(sa, &p.tmA[ph * 2 + pw], &full_bar[s], c0, w0 + ((dw - pw) >> 1), h0 + ((dh - ph) >> 1), n0);
                }
            }
            __syncwarp();
            if (++cc == p.cchunks) { cc = 0; if (++sx == p.k) { sx = 0; ++r; } }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        // Same structure: converged warp, one elected lane issues the MMAs and their commits.
        bool ok = true;
        int cc = it_begin % p.cchunks;
        for (int i = 0; i < n_it; i++) {
            const int s = i % STAGES, round = i / STAGES;
            ok = __all_sync(0xffffffffu, mbar_wait(&full_bar[s], round & 1, abort_flag));
            if (!ok) break;
            tc_fence_after();
            const int ksteps = (min(CH, p.C - cc * CH) + KS - 1) / KS;
            const uint32_t sa = smem_u32(smem + s * STAGE_BYTES), sb = sa + A_STAGE_BYTES;
            const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
            if (elect_one()) {
                for (int q = 0; q < ksteps; q++) {
                    if (I8) umma_i8(tmem_base, da + (uint64_t)(2 * q), db + (uint64_t)(2 * q), IDESC, (i > 0 || q > 0) ? 1u : 0u);
                    else umma_bf16(tmem_base, da + (uint64_t)(2 * q), db + (uint64_t)(2 * q), IDESC, (i > 0 || q > 0) ? 1u : 0u);
                }
                umma_commit(&empty_bar[s]);  // frees the stage once these MMAs have read it
                if (i == n_it - 1) umma_commit(&accum_bar);  // accumulator complete
            }
            __syncwarp();
            if (++cc == p.cchunks) cc = 0;
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        // Each thread owns one tile row (= TMEM lane = output pixel).
        const int quad = warp & 3;            // TMEM lane quadrant this warp may read
        const int row = quad * 32 + lane;     // tile row = output pixel within the box
        {
            const int rows = p.bw * p.bh * p.bn;
            const int dn = row / (p.bh * p.bw), dhh = (row / p.bw) % p.bh, dww = row % p.bw;
            const int n = n0 + dn, h = h0 + dhh, w = w0 + dww;
            const bool valid = row < rows && n < p.N && h < p.Ho && w < p.Wo;
            row_m[row] = valid ? (int)(((size_t)n * p.Ho + h) * p.Wo + w) : -1;
        }
        pdl_wait();  // residual reads and output writes must not pass the previous layers
        bool ok = n_it > 0 ? mbar_wait(&accum_bar, 0, abort_flag) : true;
        ok = __all_sync(0xffffffffu, ok);
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const int ncols = min(BN, p.K - f0);  // filters of this tile, a multiple of 8
        if (I8) {
            // integer epilogue: requantise the int32 accumulator per filter, add bias, residual and the output
            // zero point, ReLU as a maximum with the zero point, saturate, store 8 filters (8 bytes) at a time
            if (ok) {
                const int m = row_m[row];
                const int *mult = reinterpret_cast<const int *>(scale_s), *shf = reinterpret_cast<const int *>(shift_s);
                const uint8_t *res8 = reinterpret_cast<const uint8_t *>(p.res);
                uint8_t *y8 = reinterpret_cast<uint8_t *>(p.y);
                const bool ysig = p.q_flags & 2, rsig = p.q_flags & 4, relu = p.q_flags & 8;
                const int lo = ysig ? -128 : 0, hi = ysig ? 127 : 255;
#pragma unroll 1
                for (int j0 = 0; j0 < ncols; j0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(taddr + j0, v);
                    tmem_ld_wait();
                    if (m >= 0) {
#pragma unroll
                        for (int g = 0; g < 4; g++) {
                            const int c = j0 + 8 * g;
                            if (c < ncols) {
                                const size_t oi = (size_t)m * p.q_ldy + f0 + c;
                                uint2 rraw = make_uint2(0u, 0u);
                                if (res8) rraw = *reinterpret_cast<const uint2 *>(res8 + oi);
                                uint2 outw = make_uint2(0u, 0u);
#pragma unroll
                                for (int j = 0; j < 8; j++) {
                                    long long t = rshift_round((long long)(int)v[8 * g + j] * (long long)mult[c + j], 31 + shf[c + j]) + (long long)bias_s[I8 ? c + j : 0];
                                    if (res8) {
                                        const uint32_t rb = ((j < 4 ? rraw.x : rraw.y) >> (8 * (j & 3))) & 0xffu;
                                        const int rq = rsig ? (int)(signed char)rb : (int)rb;
                                        t += rshift_round((long long)(rq - p.q_zr) * (long long)p.q_res_mult, 31 + p.q_res_shift);
                                    }
                                    t += p.q_zy;
                                    if (relu && t < p.q_zy) t = p.q_zy;
                                    const int q8 = (int)(t < lo ? lo : (t > hi ? hi : t));
                                    const uint32_t byte = (uint32_t)q8 & 0xffu;
                                    if (j < 4) outw.x |= byte << (8 * j); else outw.y |= byte << (8 * (j - 4));
                                }
                                *reinterpret_cast<uint2 *>(y8 + oi) = outw;
                            }
                        }
                    }
                }
                // a padded pixel (16-byte multiples for the next layer's copies): the 8 bytes beyond the last filter are zeros
                if (m >= 0 && f0 + ncols == p.K && p.q_ldy > p.K) *reinterpret_cast<uint2 *>(y8 + (size_t)m * p.q_ldy + p.K) = make_uint2(0u, 0u);
            }
        } else if (p.splits == 1) {
            // straight from tensor memory to global memory: each thread finishes its own pixel row,
            // 8 filters (16 bytes) per store
            if (ok) {
                const int m = row_m[row];
#pragma unroll 1
                for (int j0 = 0; j0 < ncols; j0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(taddr + j0, v);
                    tmem_ld_wait();
                    if (m >= 0) {
#pragma unroll
                        for (int g = 0; g < 4; g++) {
                            const int c = j0 + 8 * g;
                            if (c < ncols) {
                                float o[8];
#pragma unroll
                                for (int j = 0; j < 8; j++) o[j] = __uint_as_float(v[8 * g + j]) * scale_s[c + j] + shift_s[c + j];
                                finish_store(o, p.res, p.y, (size_t)m * p.K + f0 + c, p.act);
                            }
                        }
                    }
                }
            }
        } else {
            // split K: this CTA covers only part of the reduction; it stores its fp32 partial tile into
            // its own slice of the workspace and splitk_finish_kernel adds the slices in split order.
            if (ok && n_it > 0) {
                const int m = row_m[row];
                float *part = p.ws + (size_t)blockIdx.z * p.slice + (size_t)(m < 0 ? 0 : m) * p.K + f0;
#pragma unroll 1
                for (int j0 = 0; j0 < ncols; j0 += 32) {
                    uint32_t v[32];
                    tmem_ld32(taddr + j0, v);
                    tmem_ld_wait();
                    if (m >= 0) {
#pragma unroll
                        for (int g = 0; g < 8; g++) {
                            const int c = j0 + 4 * g;
                            if (c < ncols)
                                __stcg(reinterpret_cast<float4 *>(part + c),
                                       make_float4(__uint_as_float(v[4 * g]), __uint_as_float(v[4 * g + 1]),
                                                   __uint_as_float(v[4 * g + 2]), __uint_as_float(v[4 * g + 3])));
                        }
                    }
                }
            }
        }
    }
    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (abort_s) {
        // a wait ran out: report, give copies that may still be in flight time to land in this
        // CTA's shared memory, then release the tensor memory
        if (threadIdx.x == 0) atomicExch(p.status, 1);
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, BN); }
}

// Second step of a split reduction: out = act(scale * (slice_0 + slice_1 + ...) + shift + res), the
// slices added in split order so that the result is the same on every run.  One thread per 8 filters
// of one pixel; all of a thread's loads are issued before the first add.
__global__ void __launch_bounds__(256) splitk_finish_kernel(const float *__restrict__ ws, size_t slice, int live,
                                                            const float *__restrict__ scale, const float *__restrict__ shift,
                                                            const __nv_bfloat16 *res, __nv_bfloat16 *y, size_t groups, int K,
                                                            int act) {
    const size_t g = blockIdx.x * (size_t)blockDim.x + threadIdx.x;
    if (g >= groups) return;
    const size_t oi = g * 8;
    const int f = (int)(oi % (size_t)K);
    float4 q[8][2];
#pragma unroll
    for (int z = 0; z < 8; z++) {
        if (z < live) {
            const float *src = ws + (size_t)z * slice + oi;
            q[z][0] = __ldcg(reinterpret_cast<const float4 *>(src));
            q[z][1] = __ldcg(reinterpret_cast<const float4 *>(src + 4));
        }
    }
    float o[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int z = 0; z < 8; z++) {
        if (z < live) {
            o[0] += q[z][0].x; o[1] += q[z][0].y; o[2] += q[z][0].z; o[3] += q[z][0].w;
            o[4] += q[z][1].x; o[5] += q[z][1].y; o[6] += q[z][1].z; o[7] += q[z][1].w;
        }
    }
#pragma unroll
    for (int j = 0; j < 8; j++) o[j] = o[j] * scale[f + j] + shift[f + j];
    finish_store(o, res, y, oi, act);
}

// ---------------------------------------------------------------------------------------------
// Host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

// Encoded tensor maps by their defining numbers.  A SubNet never seen before still slices the same stored layers
// into one of a few (K', C') boxes and reads the same workspaces at one of a few channel counts, so most of its
// maps were encoded for an earlier SubNet already; planning a new config then costs look-ups instead of driver calls.
struct MapKey {
    uint64_t v[15];
    bool operator==(const MapKey &o) const { return std::memcmp(v, o.v, sizeof v) == 0; }
};
struct MapKeyHash {
    size_t operator()(const MapKey &k) const {
        uint64_t h = 1469598103934665603ull;
        for (uint64_t x : k.v) { h ^= x; h *= 1099511628211ull; h ^= h >> 29; }
        return (size_t)h;
    }
};
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_map_cache;
std::mutex g_map_mu;

bool encode_map(CUtensorMap *m, const void *base, int rank, const uint64_t *dims, const uint64_t *strides_bytes,
                const uint32_t *box, bool bytes = false) {
    MapKey key;
    std::memset(&key, 0, sizeof key);
    key.v[0] = reinterpret_cast<uint64_t>(base);
    key.v[1] = (uint64_t)rank | (bytes ? 256u : 0u);
    for (int i = 0; i < rank; i++) { key.v[2 + i] = dims[i]; key.v[11 + (i >> 1)] |= (uint64_t)box[i] << (32 * (i & 1)); }
    for (int i = 0; i + 1 < rank; i++) key.v[7 + i] = strides_bytes[i];
    {
        std::lock_guard<std::mutex> lk(g_map_mu);
        auto it = g_map_cache.find(key);
        if (it != g_map_cache.end()) { *m = it->second; return true; }
    }
    cuuint64_t gd[5], gs[4];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; i++) { gd[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
    for (int i = 0; i + 1 < rank; i++) gs[i] = strides_bytes[i];
    CUresult r = encode_fn()(m, bytes ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void *>(base), gd, gs, bx, es,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    std::lock_guard<std::mutex> lk(g_map_mu);
    if (g_map_cache.size() < (1u << 20)) g_map_cache.emplace(key, *m);  // (128 bytes each; bounded)
    return true;
}

struct DeviceScratch {
    int *status = nullptr;
    int sms = 0;
    bool attrs_set = false;
};
DeviceScratch g_dev[64];
std::mutex g_mu;
int g_status_seen = 0;

template <int BN, int STAGES> constexpr int smem_bytes() { return STAGES * (A_STAGE_BYTES + BN * CHUNK_C * 2) + 1024; }

}  // namespace

bool tc_available() { return encode_fn() != nullptr; }
size_t tc_conv_ws_elems(const TcConvPlan &p) { return p.ws_elems; }

int *tc_status_word(int device) {
    if (device < 0 || device >= 64) return nullptr;
    std::lock_guard<std::mutex> lk(g_mu);
    return g_dev[device].status;
}

int *static_status_word(int device);  // status word inside the fixed scratch array (below); nullptr before its set-up

// Both status words of the current device (the allocated one and the one inside the fixed scratch array of the
// allocation-free entry point); a word of another device is readable only while that device is current.
int tc_conv_status() {
    std::lock_guard<std::mutex> lk(g_mu);
    int cur = -1;
    if (cudaGetDevice(&cur) != cudaSuccess || cur < 0 || cur >= 64) return g_status_seen;
    int *words[2] = {g_dev[cur].status, static_status_word(cur)};
    for (int *w : words) {
        int v = 0;
        if (w && cudaMemcpy(&v, w, sizeof(int), cudaMemcpyDeviceToHost) == cudaSuccess && v) g_status_seen = 1;
    }
    return g_status_seen;
}

cudaError_t tc_conv_status_clear() {
    std::lock_guard<std::mutex> lk(g_mu);
    int cur = -1;
    cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return e;
    if (cur < 0 || cur >= 64) return cudaErrorInvalidDevice;
    if ((e = cudaDeviceSynchronize()) != cudaSuccess) return e;
    int *words[2] = {g_dev[cur].status, static_status_word(cur)};
    for (int *w : words)
        if (w && (e = cudaMemset(w, 0, sizeof(int))) != cudaSuccess) return e;
    g_status_seen = 0;
    return cudaSuccess;
}

namespace {
// One block whose single wait can never be satisfied (nothing arrives at the barrier): it gives up after
// limit_ns, records that in the status word like the convolution kernels do, and returns.
__global__ void expire_wait_kernel(unsigned long long limit_ns, int *status) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_s;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    volatile int *abort_flag = &abort_s;
    const bool ok = mbar_wait(&bar, 0, abort_flag, limit_ns);
    __syncthreads();
    if (threadIdx.x == 0 && (!ok || abort_s)) atomicExch(status, 1);
}
}  // namespace

cudaError_t tc_expire_wait(unsigned limit_us, cudaStream_t st) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = tc_conv_init(dev)) != cudaSuccess) return e;
    expire_wait_kernel<<<1, 64, 0, st>>>((unsigned long long)limit_us * 1000ull, g_dev[dev].status);
    return cudaGetLastError();
}

// Picks the output-pixel box (bw, bh, bn), bw*bh*bn <= 128, that wastes the fewest tile rows.
static void choose_box(int N, int Ho, int Wo, int *bw_, int *bh_, int *bn_) {
    // (the search visits a few hundred candidates; a stream of never-seen SubNets asks for the same few shapes)
    static std::unordered_map<uint64_t, uint32_t> memo;
    static std::mutex memo_mu;
    const uint64_t key = ((uint64_t)(uint32_t)N << 40) | ((uint64_t)(uint32_t)Ho << 20) | (uint32_t)Wo;
    {
        std::lock_guard<std::mutex> lk(memo_mu);
        auto it = memo.find(key);
        if (it != memo.end()) { *bw_ = it->second & 0xff; *bh_ = (it->second >> 8) & 0xff; *bn_ = (it->second >> 16) & 0xff; return; }
    }
    double best = -1;
    int bbw = 1, bbh = 1, bbn = 1;
    for (int bw = 1; bw <= std::min(Wo, TILE_M); bw++) {
        for (int bh = 1; bh <= std::min(Ho, TILE_M / bw); bh++) {
            int bn = std::min(N, TILE_M / (bw * bh));
            if (bn < 1) continue;
            long long tiles = (long long)((Wo + bw - 1) / bw) * ((Ho + bh - 1) / bh) * ((N + bn - 1) / bn);
            double util = (double)N * Ho * Wo / (double)(tiles * TILE_M);
            double score = util + 1e-6 * bw;  // prefer long contiguous runs
            if (score > best) { best = score; bbw = bw; bbh = bh; bbn = bn; }
        }
    }
    *bw_ = bbw; *bh_ = bbh; *bn_ = bbn;
    if (N < (1 << 20) && Ho < (1 << 20) && Wo < (1 << 20)) {
        std::lock_guard<std::mutex> lk(memo_mu);
        if (memo.size() < 65536) memo.emplace(key, (uint32_t)bbw | ((uint32_t)bbh << 8) | ((uint32_t)bbn << 16));
    }
}

std::shared_ptr<TcConvPlan> tc_conv_prepare(const ConvArgs &a, int device, std::string *why) {
    auto no = [&](const char *msg) { if (why) *why = msg; return std::shared_ptr<TcConvPlan>(); };
    if (!encode_fn()) return no("cuTensorMapEncodeTiled unavailable");
    if (a.C % 8 || a.K % 8 || a.Cmax % 8) return no("channel counts must be multiples of 8");
    if (a.i8 && ((a.ldx ? a.ldx : a.C) % 16 || a.C % 8 || a.Cmax % 16 || a.throughput || a.win || (a.ldy && (a.ldy % 16 || a.ldy < a.K || a.ldy - a.K >= 16)) || (!a.ldy && a.K % 8)))
        return no("8-bit layers: pixels in multiples of 16 bytes, single launches");
    if (a.C < 8 || a.K < 8) return no("too few channels");
    if (a.k % 2 == 0 || a.k > a.R) return no("kernel size");
    if (a.stride != 1 && a.stride != 2) return no("stride");
    if (a.stride == 2 && ((a.H | a.W) & 1)) return no("stride 2 needs even input sizes");
    if ((reinterpret_cast<uintptr_t>(a.x) | reinterpret_cast<uintptr_t>(a.w) | reinterpret_cast<uintptr_t>(a.y) |
         reinterpret_cast<uintptr_t>(a.res)) & 15)
        return no("pointers must be 16-byte aligned");
    if (device < 0 || device >= 64) return no("device index");
    if ((a.ldx || a.ldy) && a.throughput != 2 && !a.i8) return no("padded pixels are for grouped launches and 8-bit layers");
    if ((a.ldx && (a.ldx < a.C || a.ldx % 8)) || (a.ldy && (a.ldy < a.K || a.ldy % 8))) return no("channel pitch");

    auto plan = std::make_shared<TcConvPlan>();
    TcParams &p = plan->prm;
    std::memset(&p, 0, sizeof(p));
    p.N = a.N; p.Ho = a.Ho; p.Wo = a.Wo; p.K = a.K; p.C = a.C;
    p.k = a.k; p.stride = a.stride; p.R = a.R; p.o = (a.R - a.k) / 2; p.p = (a.k - 1) / 2;
    plan->kw = a.k;
    if (a.win) {
        // window view of a stem: taps = the k filter rows, no arithmetic padding (the margin is in the buffer)
        if (a.throughput != 2 || a.C != CHUNK_C || a.Cmax != CHUNK_C) return no("window view");
        plan->kw = 1; p.R = 1; p.o = 0; p.p = 0;
    }
    p.act = a.act;
    const bool flat = a.k == 1 && a.stride == 1;
    // C = channels per pixel of x as stored (pitch and extent of the activation maps): with padded pixels the
    // channels beyond the slice are zeros, so the maps may show them and no row ends inside a 32-byte sector
    const uint64_t C = (uint64_t)(a.ldx ? a.ldx : a.C), eb = a.i8 ? 1 : 2;
    const uint32_t CH = a.i8 ? 2 * CHUNK_C : CHUNK_C;  // channels per stage (128 bytes)
    const bool b8 = a.i8 != 0;
    plan->i8 = a.i8;
    // Grouped launches (throughput == 2) run a layer with very few output pixels "swapped": the filters
    // take the 128-row side of the MMA and ALL pixels of the member form the other operand (one pixel
    // tile), so that no MMA rows are wasted on a 2x2 or 4x4 map.  (The kernel takes up to 256 pixels
    // this way; measured on 7x7 and 14x14 maps it was no faster than pixel rows, so the limit is 32.)
    const long long m_total = (long long)a.N * a.Ho * a.Wo;
    const bool swap = a.throughput == 2 && m_total <= 32;
    plan->swap = swap ? 1 : 0;
    if (flat) {
        // 1x1 stride 1: the activation tensor is a plain [M][C] matrix, tiles are 128 consecutive pixels
        const uint64_t M = (uint64_t)a.N * a.H * a.W;
        // (a member of a grouped launch with fewer than 128 pixels gets a box of exactly its pixels, so that
        // two such members can share the 128 rows of a tile)
        p.bw = swap ? (int)M : a.throughput == 2 ? (int)std::min<uint64_t>(M, TILE_M) : TILE_M; p.bh = 1; p.bn = 1;
        p.N = 1; p.Ho = 1; p.Wo = (int)M;
        uint64_t dims[4] = {C, M, 1, 1}, str[3] = {C * eb, M * C * eb, M * C * eb};
        uint32_t box[4] = {CH, (uint32_t)p.bw, 1, 1};
        if (!encode_map(&p.tmA[0], a.x, 4, dims, str, box, b8)) return no("activation tensor map");
    } else {
        if (swap) { p.bw = a.Wo; p.bh = a.Ho; p.bn = a.N; }
        else choose_box(a.N, a.Ho, a.Wo, &p.bw, &p.bh, &p.bn);
        if (a.win) {
            // dim 0 = the 64-element window of output column wo (starts at padded pixel wo * stride), dim 1 = wo,
            // dim 2 = input row (stride 2: rows of one parity), dim 3 = image
            uint32_t wbox[4] = {CHUNK_C, (uint32_t)p.bw, (uint32_t)p.bh, (uint32_t)p.bn};
            const uint64_t px = 8 * eb, st = (uint64_t)a.stride;
            for (int ph = 0; ph < a.stride; ph++) {
                const char *base = static_cast<const char *>(a.x) + (size_t)ph * a.W * px;
                uint64_t dims[4] = {CHUNK_C, (uint64_t)a.Wo, (uint64_t)(a.H - ph + a.stride - 1) / st, (uint64_t)a.N};
                uint64_t str[3] = {st * px, st * (uint64_t)a.W * px, (uint64_t)a.H * a.W * px};
                if (!encode_map(&p.tmA[ph * 2], base, 4, dims, str, wbox)) return no("window tensor map");
            }
        }
        uint32_t box[4] = {CH, (uint32_t)p.bw, (uint32_t)p.bh, (uint32_t)p.bn};
        if (a.win) {
            // (encoded above)
        } else if (a.stride == 1) {
            uint64_t dims[4] = {C, (uint64_t)a.W, (uint64_t)a.H, (uint64_t)a.N};
            uint64_t str[3] = {C * eb, (uint64_t)a.W * C * eb, (uint64_t)a.H * a.W * C * eb};
            if (!encode_map(&p.tmA[0], a.x, 4, dims, str, box, b8)) return no("activation tensor map");
        } else {
            for (int ph = 0; ph < 2; ph++)
                for (int pw = 0; pw < 2; pw++) {
                    const char *base = static_cast<const char *>(a.x) + ((size_t)ph * a.W + pw) * C * eb;
                    uint64_t dims[4] = {C, (uint64_t)a.W / 2, (uint64_t)a.H / 2, (uint64_t)a.N};
                    uint64_t str[3] = {2 * C * eb, 2 * (uint64_t)a.W * C * eb, (uint64_t)a.H * a.W * C * eb};
                    if (!encode_map(&p.tmA[ph * 2 + pw], base, 4, dims, str, box, b8)) return no("activation tensor map");
                }
        }
    }
    p.tiles_w = (p.Wo + p.bw - 1) / p.bw;
    p.tiles_h = (p.Ho + p.bh - 1) / p.bh;
    const int tiles_n = (p.N + p.bn - 1) / p.bn;
    const int mtiles = p.tiles_w * p.tiles_h * tiles_n;

    // filter tile: 128 wide unless the layer is narrow or too few CTAs would stream the weights
    int sms = 148;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        DeviceScratch &ds = g_dev[device];
        if (!ds.sms) cudaDeviceGetAttribute(&ds.sms, cudaDevAttrMultiProcessorCount, device);
        if (ds.sms > 0) sms = ds.sms;
    }
    p.cchunks = (a.C + (int)CH - 1) / (int)CH;
    p.iters = a.k * plan->kw * p.cchunks;
    // Filter tile.  Issuing one MMA costs the issuing thread about the same whatever its width, so wide
    // tiles are preferred as long as tiles x K splits can still occupy every SM.
    // a split costs a second (small) kernel, so it has to save at least a dozen pipeline iterations
    int max_splits = p.iters >= 16 ? std::min(8, p.iters / 4) : 1;
    int BN = 64;
    for (int cand : {128}) {  // 256-wide tiles leave one CTA per SM, which this non-persistent kernel cannot afford
        if (a.K <= cand / 2) continue;  // would be mostly padding
        if ((long long)mtiles * ((a.K + cand - 1) / cand) * max_splits >= sms) { BN = cand; break; }
    }
    if (a.throughput) {
        // Many independent launches share the GPU (queries in flight): filling every SM from one launch
        // no longer matters, work per issued MMA does.  Wide tiles, splits only for very long K loops.
        // Measured on the batch-1 stream with 16 queries in flight: +13 % queries/s.
        BN = a.K > 64 ? 128 : 64;
        max_splits = p.iters >= 32 ? std::min(4, p.iters / 8) : 1;
    }
    if (a.throughput == 2) {
        // grouped launch: no split; filter tile = the narrowest of 64 / 128 / 256 that holds the layer
        // (256 at most), or 128 filters on the MMA's row side when swapped
        max_splits = 1;
        BN = swap ? 128 : a.K <= 64 ? 64 : a.K <= 128 ? 128 : 256;
    }
    if (a.i8) max_splits = 1;  // (the integer epilogue has no second step)
    plan->bn_tile = BN;
    {
        const uint64_t taps = a.win ? (uint64_t)a.k : (uint64_t)a.R * a.R;  // stored taps per filter
        // (padded pixels: the weight map shows the stored channels up to the pixel's pitch; they meet zeros)
        const uint64_t Cw = a.ldx ? std::min<uint64_t>((uint64_t)a.ldx, (uint64_t)a.Cmax) : (uint64_t)a.C;
        uint64_t dims[3] = {Cw, taps, (uint64_t)a.K};
        uint64_t str[2] = {(uint64_t)a.Cmax * eb, taps * a.Cmax * eb};
        uint32_t box[3] = {CH, 1, (uint32_t)BN};
        if (!encode_map(&p.tmW, a.w, 3, dims, str, box, b8)) return no("weight tensor map");
    }
    const int ntiles = (a.K + BN - 1) / BN;
    // split the K loop when the tiles alone cannot fill the machine
    int splits = 1;
    const int ctas = mtiles * ntiles;
    if (ctas < sms && max_splits > 1) {
        splits = std::min((sms + ctas - 1) / ctas, max_splits);
        if (splits < 1) splits = 1;
        // every split must own at least one iteration
        while (splits > 1 && (p.iters + splits - 1) / splits * (splits - 1) >= p.iters) splits--;
    }
    p.splits = splits;
    p.slice = (size_t)a.N * a.Ho * a.Wo * a.K;
    plan->grid = dim3((unsigned)mtiles, (unsigned)ntiles, (unsigned)splits);
    plan->ws_elems = splits > 1 ? (size_t)splits * a.N * a.Ho * a.Wo * a.K : 0;
    return plan;
}

// Launches the second step of a split reduction for the layer described by prm.
static cudaError_t launch_finish(const TcParams &prm, cudaStream_t st) {
    const int per = (prm.iters + prm.splits - 1) / prm.splits;
    const int live = (prm.iters + per - 1) / per;  // splits that own at least one iteration
    const size_t groups = prm.slice / 8;
    splitk_finish_kernel<<<(unsigned)((groups + 255) / 256), 256, 0, st>>>(prm.ws, prm.slice, live, prm.scale, prm.shift, prm.res,
                                                                         prm.y, groups, prm.K, prm.act);
    return cudaGetLastError();
}

template <int BN, int STAGES, bool I8 = false> static cudaError_t launch_variant(const TcConvPlan &pl, const TcParams &prm, cudaStream_t st) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = pl.grid;
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = smem_bytes<BN, STAGES>();
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, conv_tc_kernel<BN, STAGES, I8>, prm);
}

// One-time set-up of the current device: status word and the kernels' shared-memory limits.  Must
// run outside stream capture (it allocates).
cudaError_t tc_conv_init(int dev) {
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lk(g_mu);
    DeviceScratch &ds = g_dev[dev];
    if (ds.attrs_set && ds.status) return cudaSuccess;
    cudaError_t e;
    if (!ds.status) {
        if ((e = cudaMalloc(&ds.status, sizeof(int))) != cudaSuccess) return e;
        if ((e = cudaMemset(ds.status, 0, sizeof(int))) != cudaSuccess) return e;
    }
    if ((e = cudaFuncSetAttribute(conv_tc_kernel<64, 3, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<64, 3>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(conv_tc_kernel<128, 3, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<128, 3>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(conv_tc_kernel<256, 4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<256, 4>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(conv_tc_kernel<64, 3, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<64, 3>())) != cudaSuccess) return e;
    if ((e = cudaFuncSetAttribute(conv_tc_kernel<128, 3, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<128, 3>())) != cudaSuccess) return e;
    if ((e = tc_group_init(dev)) != cudaSuccess) return e;
    if ((e = subnet_kernel_init(dev)) != cudaSuccess) return e;
    ds.attrs_set = true;
    return cudaSuccess;
}

cudaError_t tc_conv_launch(const TcConvPlan &pl, const ConvArgs &a, cudaStream_t st, int *launches) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if ((e = tc_conv_init(dev)) != cudaSuccess) return e;
    TcParams prm = pl.prm;
    prm.scale = a.scale; prm.shift = a.shift;
    prm.res = static_cast<const __nv_bfloat16 *>(a.res);
    prm.y = static_cast<__nv_bfloat16 *>(a.y);
    prm.status = g_dev[dev].status;
    prm.cacheK = a.cacheK; prm.cacheC = a.cacheC; prm.weight_policy = a.weight_policy;
    prm.cache_tbl = a.cache_tbl; prm.layer = a.layer;
    prm.ws = a.ws;
    if (prm.splits > 1 && (!a.ws || a.ws_elems < pl.ws_elems)) prm.splits = 1;  // no workspace: run unsplit
    TcConvPlan run = pl;
    run.grid.z = (unsigned)prm.splits;
    if (pl.i8) {
        if (!a.q_mult || !a.q_shift || !a.q_bias || pl.bn_tile > 128 || prm.splits != 1) return cudaErrorInvalidValue;
        prm.q_mult = a.q_mult; prm.q_shift = a.q_shift; prm.q_bias = a.q_bias;
        prm.q_zy = a.q_zy; prm.q_zr = a.q_zr; prm.q_res_mult = a.q_res_mult; prm.q_res_shift = a.q_res_shift; prm.q_flags = a.q_flags;
        prm.q_ldy = a.ldy ? a.ldy : a.K;
        e = pl.bn_tile == 64 ? launch_variant<64, 3, true>(run, prm, st) : launch_variant<128, 3, true>(run, prm, st);
        if (launches) *launches = 1;
        return e;
    }
    if (pl.bn_tile == 64) e = launch_variant<64, 3>(run, prm, st);
    else if (pl.bn_tile == 128) e = launch_variant<128, 3>(run, prm, st);
    else e = launch_variant<256, 4>(run, prm, st);
    if (launches) *launches = 1;
    if (e != cudaSuccess || prm.splits == 1) return e;
    e = launch_finish(prm, st);
    if (launches) *launches = 2;
    return e;
}

}  // namespace sgs

// =============================================================================================
// Sliced convolution for callers that must not allocate device memory.
//
// Some users of this library run where cudaMalloc is off limits: inside a serving process whose
// whole device memory was handed to a pool at start-up, or in a latency-critical loop where an
// implicit device synchronisation (which cudaMalloc / cudaFree cause) is not acceptable.  For them the split-reduction scratch of the
// tensor-core kernel lives in a fixed array that is part of the loaded library image.
// =============================================================================================
namespace sgs {
namespace {

constexpr size_t STATIC_WS_FLOATS = SGS_STATIC_SCRATCH_BYTES / sizeof(float);

struct StaticScratch {
    float ws[STATIC_WS_FLOATS];  // partial tiles of the split reduction
    int status;                  // set by a kernel whose bounded wait ran out
};
// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) StaticScratch g_static_scratch;

// Device address of the array per device.  In host code the symbol's name is only a handle; the
// address a kernel can use has to be asked for with cudaGetSymbolAddress while that device is current.
StaticScratch *g_static_ptr[64] = {};
std::mutex g_static_mu;

cudaError_t static_scratch_setup(int dev, StaticScratch **out) {
    std::lock_guard<std::mutex> lk(g_static_mu);
    if (!g_static_ptr[dev]) {
        StaticScratch *ptr = nullptr;
        cudaError_t e = cudaGetSymbolAddress((void **)&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(conv_tc_kernel<64, 3, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<64, 3>())) != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(conv_tc_kernel<128, 3, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<128, 3>())) != cudaSuccess) return e;
        if ((e = cudaFuncSetAttribute(conv_tc_kernel<256, 4, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<256, 4>())) != cudaSuccess) return e;
        if ((e = cudaMemset(&ptr->status, 0, sizeof(int))) != cudaSuccess) return e;
        g_static_ptr[dev] = ptr;
    }
    *out = g_static_ptr[dev];
    return cudaSuccess;
}

}  // namespace

int *static_status_word(int device) {
    std::lock_guard<std::mutex> lk(g_static_mu);
    return (device >= 0 && device < 64 && g_static_ptr[device]) ? &g_static_ptr[device]->status : nullptr;
}
}  // namespace sgs

extern "C" sgs_status_t sgs_conv2d_sliced_static(const sgs_conv_desc_t *d, const void *d_x, const void *d_w,
                                                 const float *d_scale, const float *d_shift, const void *d_res, void *d_y,
                                                 void *cuda_stream) {
    using namespace sgs;
    if (!d || !d_x || !d_w || !d_scale || !d_shift || !d_y) return SGS_EINVAL;
    if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->C <= 0 || d->K <= 0 || d->k <= 0 || (d->k & 1) == 0 || d->k > d->R ||
        ((d->R - d->k) & 1) || d->K > d->Kmax || d->C > d->Cmax || (d->stride != 1 && d->stride != 2) || d->act < 0 || d->act > 2)
        return SGS_EINVAL;
    if (d->impl < 0 || d->impl > 2) return SGS_EINVAL;
    if (d->dtype != SGS_BF16 || d->depthwise || d->impl == 1 || !tc_available()) return SGS_EUNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SGS_ECUDA;
    StaticScratch *sc = nullptr;
    if (static_scratch_setup(dev, &sc) != cudaSuccess) return SGS_ECUDA;

    ConvArgs a;
    a.x = d_x; a.w = d_w; a.scale = d_scale; a.shift = d_shift; a.res = d_res; a.y = d_y;
    a.N = d->N; a.H = d->H; a.W = d->W; a.C = d->C; a.K = d->K;
    a.Kmax = d->Kmax; a.Cmax = d->Cmax; a.R = d->R; a.k = d->k; a.stride = d->stride; a.act = d->act;
    const int p = (d->k - 1) / 2;
    a.Ho = (d->H + 2 * p - d->k) / d->stride + 1;
    a.Wo = (d->W + 2 * p - d->k) / d->stride + 1;
    a.cacheK = d->cache_k; a.cacheC = d->cache_c; a.weight_policy = d->weight_policy;
    std::shared_ptr<TcConvPlan> plan = tc_conv_prepare(a, dev, nullptr);  // host memory only
    if (!plan) return SGS_EUNSUPPORTED;
    TcParams prm = plan->prm;
    if (d->split_k_off) prm.splits = 1;
    if (prm.splits > 1 && plan->ws_elems > STATIC_WS_FLOATS)
        return SGS_ENOMEM;  // the layer's split reduction does not fit SGS_STATIC_SCRATCH_BYTES
    cudaStream_t st = (cudaStream_t)cuda_stream;
    // Nothing in the array has to start at zero: every partial-tile element that is read back by the
    // second step is written by the first step of the same call.
    prm.scale = a.scale; prm.shift = a.shift;
    prm.res = static_cast<const __nv_bfloat16 *>(a.res);
    prm.y = static_cast<__nv_bfloat16 *>(a.y);
    prm.status = &sc->status;
    prm.cacheK = a.cacheK; prm.cacheC = a.cacheC; prm.weight_policy = a.weight_policy;
    prm.cache_tbl = nullptr; prm.layer = 0;
    prm.ws = sc->ws;
    TcConvPlan run = *plan;
    run.grid.z = (unsigned)prm.splits;
    cudaError_t e = plan->bn_tile == 64    ? launch_variant<64, 3>(run, prm, st)
                    : plan->bn_tile == 128 ? launch_variant<128, 3>(run, prm, st)
                                           : launch_variant<256, 4>(run, prm, st);
    if (e == cudaSuccess && prm.splits > 1) e = launch_finish(prm, st);
    return e == cudaSuccess ? SGS_OK : SGS_ECUDA;
}
