// Persistent SubNet kernel for the MobileNetV3-shaped family (bf16, one image per query).
//
// The paper's accelerator serves one query per pass and keeps the weights it will need again on chip
// (Section 3.1, Section 4.2 "Persistent Buffer").  On this GPU a one-image MobileNetV3-sized SubNet is far too
// small to fill the machine layer by layer: a wave of 32 such queries needs about a hundred dependent launches of
// 10 - 20 us each.  Here the whole stream is ONE launch instead.  Every block (one per SM, 512 threads) takes the
// next unserved query from a counter and runs all layers of that query's SubNet by itself, image to logits:
//   * pointwise (1x1) convolutions on the tensor cores: tcgen05.mma with the fp32 accumulator in tensor memory
//     (two 256-column buffers, so the epilogue of one tile overlaps the MMAs of the next); the operands are
//     brought into 128-byte-swizzled shared-memory tiles by the block's own threads with 16-byte asynchronous
//     copies (a ring of three stages, copies two stages ahead of the MMAs) - the tiles of one query are too
//     small and too many to be worth a tensor map each;
//   * depthwise convolutions, the 3-channel stem, pooling, the squeeze-excite gate and the linear layers on the
//     CUDA cores, with 16-byte accesses;
//   * activations in a private scratch area of the block in global memory (written and read back by the same
//     SM, so they stay in L1 / L2); pooled vectors and gates in shared memory.
//   * optionally a weight buffer in shared memory, filled once per block at the start of the launch with the
//     cached SubGraph's boxes of the first pointwise layers (the first filters x first channels of their stored
//     rows) and read in place by the MMAs of every query the block serves; filters and channels of a query's
//     slice beyond the box are streamed through the ring as usual (the SubGraph-stationary dataflow of
//     Section 4.3: what the queries share is fetched once, the rest per query).
// Nothing waits on another block, so the kernel needs no co-scheduling guarantee; its only waits are on its own
// copies and MMAs, and they are bounded like those of the other tensor-core kernels.
// Slicing is the same as everywhere else in the library: the first K' filters and C' channels of the stored rows,
// the centre k x k taps of a stored depthwise filter; no sliced copy of a weight exists.

#include "sgs_tc.cuh"

namespace sgs {

namespace {

using bf16 = __nv_bfloat16;

constexpr int PQ_THREADS = 512;
constexpr int PQ_BLOCKS_PER_SM = 1;          // (measured: two blocks of 256 threads per SM with 96-filter tiles serve 28k queries/s, one of 512 serves 42k)
constexpr int PQ_WARPS = PQ_THREADS / 32;
constexpr int PQ_ROWS = PQ_THREADS / 8;      // rows of 128 bytes one round of 16-byte copies covers
constexpr int PQ_MAX_K = 1024;               // widest pointwise layer (folded batch norm staged in shared memory)
constexpr int PQ_MAX_BN = 256;               // filters per tile
constexpr int PQ_RING_BYTES = 144 * 1024;    // operand ring: 3 stages of pixel tile (16 KB) + filter tile (up to 32 KB), or 4 smaller ones
constexpr int PQ_LAG = 2;                    // copies run this many stages ahead of the MMAs
constexpr int PQ_VEC = 1280;                 // longest fp32 vector held in shared memory (the head's width)
constexpr int PQ_ACC_COLS = 256;             // tensor-memory columns of one accumulator buffer
constexpr int PQ_HELD_MAX = 56 * 1024;       // largest weight buffer (dynamic shared memory beyond the ring)
constexpr unsigned long long PQ_WAIT_NS = 2000000000ull;

// Completed phases of the block's barriers since the kernel started (the same in every thread; only ever
// indexed with constants, so they live in registers).
struct PipeState {
    uint32_t use[4];  // commits issued to free_bar[s]
    uint32_t acc[2];  // commits issued to acc_bar[b]
    uint32_t tiles;   // output tiles started (buffer = tiles & 1)
};
__device__ __forceinline__ uint32_t get4(const uint32_t (&a)[4], int s) { return s == 0 ? a[0] : s == 1 ? a[1] : s == 2 ? a[2] : a[3]; }
__device__ __forceinline__ void inc4(uint32_t (&a)[4], int s) { a[0] += s == 0; a[1] += s == 1; a[2] += s == 2; a[3] += s == 3; }

// 16-byte asynchronous copy into shared memory; `valid` false writes zeros (nothing is read).
__device__ __forceinline__ void cp16_cg(uint32_t dst, const void *src, bool valid) {
    const int n = valid ? 16 : 0;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp16_ca(uint32_t dst, const void *src, bool valid) {
    const int n = valid ? 16 : 0;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ float2 unpack2(uint32_t u) { return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u)); }

__device__ __forceinline__ float dot8w(uint4 wv, float4 x0, float4 x1, float s) {
    const float2 a = unpack2(wv.x), b = unpack2(wv.y), c = unpack2(wv.z), d = unpack2(wv.w);
    s = fmaf(a.x, x0.x, s); s = fmaf(a.y, x0.y, s); s = fmaf(b.x, x0.z, s); s = fmaf(b.y, x0.w, s);
    s = fmaf(c.x, x1.x, s); s = fmaf(c.y, x1.y, s); s = fmaf(d.x, x1.z, s); s = fmaf(d.y, x1.w, s);
    return s;
}

// ---------------------------------------------------------------------------------------------
// Pointwise convolution  y[m][f] = act(scale[f] * sum_c x[m][c] * w[f][c] + shift[f]) (+ res[m][f])
// M = H * W pixels of the one image, tiles of 128 pixels x BN filters (BN <= PQ_MAX_BN), channels in chunks of 64;
// a ring of three stages, each the pixel tile's and the filter tile's 64-channel chunk.
// (Measured alternatives, both slower: the layer's whole weight matrix copied once and read in place by every pixel
// tile - the larger shared-memory footprint costs the depthwise layers their L1; and the epilogue's results
// gathered in a shared-memory tile and written out with fully coalesced stores - the epilogue is bound by its
// arithmetic, not by its 16-byte stores.)
// ---------------------------------------------------------------------------------------------
struct PwShape {
    int M, C, K, n_tiles, BN, cchunks, m_tiles, stage_bytes, S;
};
__device__ __forceinline__ PwShape pw_shape(const PqOp &op) {
    PwShape s;
    s.M = op.Ho * op.Wo; s.C = op.C; s.K = op.K;
    s.n_tiles = (s.K + PQ_MAX_BN - 1) / PQ_MAX_BN;
    s.BN = (((s.K + s.n_tiles - 1) / s.n_tiles) + 15) & ~15;  // MMA width: a multiple of 16, at most PQ_MAX_BN
    s.cchunks = (s.C + 63) >> 6;
    s.m_tiles = (s.M + 127) >> 7;
    s.stage_bytes = A_STAGE_BYTES + s.BN * 128;
    s.S = min(4, PQ_RING_BYTES / s.stage_bytes);
    return s;
}

// Epilogue arithmetic of 16 consecutive filters of one pixel, two values at a time (packed fp32 instructions).
// Hard swish is x * sat(x / 6 + 1 / 2): one saturating multiply-add and one multiply.
__device__ __forceinline__ void pw_store16(const PwShape &s, const float *bn, const uint32_t *v, const bf16 *res, bf16 *y, int m, int f0,
                                           int c, int cols, int act) {
#pragma unroll
    for (int h = 0; h < 2; h++) {
        const int cc = c + h * 8;
        if (cc < cols) {
            const int f = f0 + cc;
            const size_t oi = (size_t)m * s.K + f;
            const float4 s0 = *reinterpret_cast<const float4 *>(bn + f), s1 = *reinterpret_cast<const float4 *>(bn + f + 4);
            const float4 h0 = *reinterpret_cast<const float4 *>(bn + PQ_MAX_K + f), h1 = *reinterpret_cast<const float4 *>(bn + PQ_MAX_K + f + 4);
            float2 o[4];
            o[0] = __ffma2_rn(make_float2(__uint_as_float(v[h * 8 + 0]), __uint_as_float(v[h * 8 + 1])), make_float2(s0.x, s0.y), make_float2(h0.x, h0.y));
            o[1] = __ffma2_rn(make_float2(__uint_as_float(v[h * 8 + 2]), __uint_as_float(v[h * 8 + 3])), make_float2(s0.z, s0.w), make_float2(h0.z, h0.w));
            o[2] = __ffma2_rn(make_float2(__uint_as_float(v[h * 8 + 4]), __uint_as_float(v[h * 8 + 5])), make_float2(s1.x, s1.y), make_float2(h1.x, h1.y));
            o[3] = __ffma2_rn(make_float2(__uint_as_float(v[h * 8 + 6]), __uint_as_float(v[h * 8 + 7])), make_float2(s1.z, s1.w), make_float2(h1.z, h1.w));
            if (res) {
                const uint4 rv = *reinterpret_cast<const uint4 *>(res + oi);
                o[0] = __fadd2_rn(o[0], unpack2(rv.x)); o[1] = __fadd2_rn(o[1], unpack2(rv.y));
                o[2] = __fadd2_rn(o[2], unpack2(rv.z)); o[3] = __fadd2_rn(o[3], unpack2(rv.w));
            }
            uint4 ov;
            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
            for (int j = 0; j < 4; j++) {
                if (act == ACT_RELU) {
                    o[j].x = fmaxf(o[j].x, 0.f); o[j].y = fmaxf(o[j].y, 0.f);
                } else if (act == ACT_HSWISH) {
                    const float2 t = make_float2(__saturatef(fmaf(o[j].x, 1.f / 6.f, 0.5f)), __saturatef(fmaf(o[j].y, 1.f / 6.f, 0.5f)));
                    o[j] = __fmul2_rn(o[j], t);
                }
                ob[j] = __floats2bfloat162_rn(o[j].x, o[j].y);
            }
            *reinterpret_cast<uint4 *>(y + oi) = ov;
        }
    }
}

// Epilogue of tile (mt, nt) out of an accumulator buffer: warp w reads lane quadrant w % 4 (its 32 pixels) and the
// groups of 16 filters g with g % (warps / 4) == w / 4, two groups per tensor-memory wait.  bn: the layer's folded
// batch norm in shared memory, scale at [f], shift at [PQ_MAX_K + f].
__device__ __forceinline__ bool pw_epilogue(const PqOp &op, const PwShape &s, const float *bn, const bf16 *res, bf16 *y, int mt, int nt,
                                            uint32_t tmem_acc, uint64_t *bar, uint32_t parity, volatile int *abort_flag) {
    constexpr int CG = PQ_WARPS / 4;  // column groups the warps of one quadrant share
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, quad = warp & 3, cgrp = warp >> 2;
    if (!__all_sync(0xffffffffu, mbar_wait(bar, parity, abort_flag, PQ_WAIT_NS))) return false;
    tc_fence_after();
    const int m = mt * 128 + quad * 32 + lane, act = op.act;
    const int f0 = nt * s.BN, cols = min(s.BN, s.K - f0);  // a multiple of 8
    const uint32_t t = tmem_acc + ((uint32_t)(quad * 32) << 16);
    for (int g = cgrp; g * 16 < cols; g += 2 * CG) {
        uint32_t v0[16], v1[16];
        const bool two = (g + CG) * 16 < cols;  // (the same in every lane)
        tmem_ld16(t + (uint32_t)(g * 16), v0);
        if (two) tmem_ld16(t + (uint32_t)((g + CG) * 16), v1);
        tmem_ld_wait();
        if (m < s.M) {
            pw_store16(s, bn, v0, res, y, m, f0, g * 16, cols, act);
            if (two) pw_store16(s, bn, v1, res, y, m, f0, (g + CG) * 16, cols, act);
        }
    }
    tc_fence_before();  // the buffer's next MMAs are issued after a block barrier
    return true;
}
// Returns false when a wait ran out (the caller leaves at its next block barrier).
__device__ __forceinline__ bool pq_pointwise(const PqOp &op, const bf16 *x, const bf16 *res, bf16 *y, uint8_t *ring, float *bn,
                                             uint32_t held_u32, uint64_t *free_bar, uint64_t *acc_bar, uint32_t tmem_base, PipeState &ps,
                                             volatile int *abort_flag) {
    const int tid = threadIdx.x;
    const PwShape s = pw_shape(op);
    const int S = s.S;
    const int total = s.n_tiles * s.m_tiles * s.cchunks;
    // instruction descriptor: fp32 accumulator, bf16 x bf16, both K-major, N = BN, M = 128
    const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(s.BN >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
    const uint32_t ring_u32 = smem_u32(ring);
    const bf16 *w = static_cast<const bf16 *>(op.w);
    // the layer's folded batch norm, read by every epilogue (visible after the first block barrier of the loop)
    for (int f = tid; f < s.K; f += PQ_THREADS) { bn[f] = __ldg(op.scale + f); bn[PQ_MAX_K + f] = __ldg(op.shift + f); }
    // this thread's 16-byte piece of every 128-byte row it copies: rows tid / 8 + PQ_ROWS j, piece tid % 8 (the
    // swizzle term row % 8 is then the same for all of them)
    const int c16 = tid & 7, r0 = tid >> 3;
    const uint32_t piece = (uint32_t)((c16 ^ (r0 & 7)) << 4);
    // Weight buffer: of this layer's box the query can use the first hK filters (a multiple of 16) in every channel
    // chunk whose channels - as far as the query takes them - lie inside the box; those need no copy and are
    // multiplied in place, the tile's other filters come through the ring and get an MMA of their own.
    const int hK = (held_u32 != 0u && op.cache_off >= 0 && s.n_tiles == 1) ? (min(op.cache_rows, s.K) & ~15) : 0;
    const uint32_t box_u32 = held_u32 + (uint32_t)(op.cache_off < 0 ? 0 : op.cache_off);
    const uint32_t idesc_h = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(hK >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
    const uint32_t idesc_r = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((s.BN - hK) >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
    auto chunk_held = [&](int ch) { return hK > 0 && min(s.C, (ch + 1) * 64) <= op.ld2; };

    bool ok = true;
    int p_chunk = 0, p_mt = 0, p_nt = 0, p_stage = 0;  // next iteration to copy
    int c_chunk = 0, c_mt = 0, c_nt = 0, c_stage = 0;  // next iteration to multiply
    int e_mt = -1, e_nt = 0;                           // finished tile whose epilogue is still to run
    uint32_t e_buf = 0;
    for (int i = 0; i < total + PQ_LAG; i++) {
        if (i >= PQ_LAG) {
            cp_wait<PQ_LAG - 1>();  // this thread's copies of iteration i - LAG have landed
            fence_async_smem();     // ... and are visible to the tensor core's reads
            tc_fence_before();
            __syncthreads();        // ... and so are everybody else's
            const uint32_t buf = ps.tiles & 1u;
            if (tid == 0) {
                tc_fence_after();
                const uint32_t sa = ring_u32 + (uint32_t)(c_stage * s.stage_bytes), sb = sa + A_STAGE_BYTES;
                const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
                const int ksteps = (min(64, s.C - c_chunk * 64) + 15) >> 4;
                if (chunk_held(c_chunk)) {
                    const uint64_t dh = smem_desc_sw128(box_u32 + (uint32_t)(c_chunk * op.cache_rows * 128));
                    const uint64_t dr = smem_desc_sw128(sb + (uint32_t)(hK * 128));
                    for (int q = 0; q < ksteps; q++) {
                        umma_bf16(tmem_base + buf * PQ_ACC_COLS, da + (uint64_t)(2 * q), dh + (uint64_t)(2 * q), idesc_h, (c_chunk > 0 || q > 0) ? 1u : 0u);
                        if (s.BN > hK)
                            umma_bf16(tmem_base + buf * PQ_ACC_COLS + (uint32_t)hK, da + (uint64_t)(2 * q), dr + (uint64_t)(2 * q), idesc_r, (c_chunk > 0 || q > 0) ? 1u : 0u);
                    }
                } else {
                    for (int q = 0; q < ksteps; q++)
                        umma_bf16(tmem_base + buf * PQ_ACC_COLS, da + (uint64_t)(2 * q), db + (uint64_t)(2 * q), idesc, (c_chunk > 0 || q > 0) ? 1u : 0u);
                }
                umma_commit(&free_bar[c_stage]);
                if (c_chunk == s.cchunks - 1) umma_commit(&acc_bar[buf]);
            }
            inc4(ps.use, c_stage);
            // the previous tile's epilogue runs while this tile's MMAs do
            if (c_chunk == 0 && e_mt >= 0) {
                const uint32_t n_acc = e_buf ? ps.acc[1] : ps.acc[0];
                ok = pw_epilogue(op, s, bn, res, y, e_mt, e_nt, tmem_base + e_buf * PQ_ACC_COLS, &acc_bar[e_buf], (n_acc - 1) & 1u, abort_flag) && ok;
                e_mt = -1;
            }
            if (c_chunk == s.cchunks - 1) {
                if (buf) ps.acc[1]++; else ps.acc[0]++;
                ps.tiles++;
                e_mt = c_mt; e_nt = c_nt; e_buf = buf;
            }
            if (++c_stage == S) c_stage = 0;
            if (++c_chunk == s.cchunks) { c_chunk = 0; if (++c_mt == s.m_tiles) { c_mt = 0; ++c_nt; } }
        }
        if (i < total) {
            // the stage was last read by the MMAs of iteration i - S, issued in the previous step
            const uint32_t u = get4(ps.use, p_stage);
            if (i >= S && u > 0) ok = mbar_wait(&free_bar[p_stage], (u - 1) & 1u, abort_flag, PQ_WAIT_NS) && ok;
            const uint32_t sa = ring_u32 + (uint32_t)(p_stage * s.stage_bytes), sb = sa + A_STAGE_BYTES;
            const int c0 = p_chunk * 64 + c16 * 8;
            const bool cvalid = c0 < s.C;
#pragma unroll
            for (int j = 0; j < 128 / PQ_ROWS; j++) {
                const int row = r0 + PQ_ROWS * j, m = p_mt * 128 + row;
                const bool v = cvalid && m < s.M;
                cp16_cg(sa + (uint32_t)(row * 128) + piece, v ? x + (size_t)m * s.C + c0 : x, v);
            }
            for (int row = r0 + (chunk_held(p_chunk) ? hK : 0); row < s.BN; row += PQ_ROWS) {
                const int f = p_nt * s.BN + row;
                const bool v = cvalid && f < s.K;
                cp16_ca(sb + (uint32_t)(row * 128) + piece, v ? w + (size_t)f * op.ld + c0 : w, v);
            }
            if (++p_stage == S) p_stage = 0;
            if (++p_chunk == s.cchunks) { p_chunk = 0; if (++p_mt == s.m_tiles) { p_mt = 0; ++p_nt; } }
        }
        cp_commit();  // (an empty group in the drain steps keeps the group count in step with i)
    }
    if (e_mt >= 0) {
        const uint32_t n_acc = e_buf ? ps.acc[1] : ps.acc[0];
        ok = pw_epilogue(op, s, bn, res, y, e_mt, e_nt, tmem_base + e_buf * PQ_ACC_COLS, &acc_bar[e_buf], (n_acc - 1) & 1u, abort_flag) && ok;
    }
    cp_wait<0>();
    return ok;
}

// ---------------------------------------------------------------------------------------------
// Depthwise convolution: a thread owns 8 channels of 4 (2) neighbouring output pixels of one output row and walks
// the filter rows; per filter row it loads the input columns once and uses each for every tap it belongs to.
// (Plain loads: the input was written by this block a moment ago.  Measured alternatives: the layer's filters
// converted to fp32 once and read from shared memory, two 16-byte reads per tap instead of one global load and its
// unpacking: 41k queries/s against 44k; channel blocks of 64 outermost so that the rows a block needs again stay in
// L1: slower as well.)
// ---------------------------------------------------------------------------------------------
template <int K, int ST>
__device__ __noinline__ void pq_depthwise(const PqOp &op, const bf16 *x, bf16 *y) {
    constexpr int TW = (ST == 2 && K > 3) ? 2 : 4;  // (the wide stride-2 windows would not fit the register budget of 512 threads)
    constexpr int NCOL = (TW - 1) * ST + K, P = (K - 1) / 2;
    constexpr int RU = K == 7 ? 1 : K;  // filter rows unrolled together (all 7 rows of the widest filter at once would spill)
    const int Cn = op.K, groups = Cn >> 3, wblocks = (op.Wo + TW - 1) / TW;
    const int per_row = groups * wblocks, total = per_row * op.Ho;
    const int o = (op.R - K) / 2;
    const bf16 *__restrict__ w = static_cast<const bf16 *>(op.w);
    for (int it = threadIdx.x; it < total; it += PQ_THREADS) {
        const int ho = it / per_row, idx = it - ho * per_row;
        const int cg = idx % groups, wb = idx / groups;
        const int c0 = cg * 8, wo0 = wb * TW;
        float2 acc[TW][4];
#pragma unroll
        for (int t = 0; t < TW; t++)
#pragma unroll
            for (int j = 0; j < 4; j++) acc[t][j] = make_float2(0.f, 0.f);
#pragma unroll RU
        for (int r = 0; r < K; r++) {
            const int hi = ho * ST + r - P;
            if (hi < 0 || hi >= op.H) continue;
            const bf16 *xrow = x + (size_t)hi * op.W * Cn + c0;
            uint4 col[NCOL];
#pragma unroll
            for (int j = 0; j < NCOL; j++) {
                const int wi = wo0 * ST + j - P;
                col[j] = (wi >= 0 && wi < op.W) ? *reinterpret_cast<const uint4 *>(xrow + (size_t)wi * Cn) : make_uint4(0u, 0u, 0u, 0u);
            }
            const bf16 *wrow = w + ((size_t)(o + r) * op.R + o) * op.Kmax + c0;
#pragma unroll
            for (int sx = 0; sx < K; sx++) {
                const uint4 wv = __ldg(reinterpret_cast<const uint4 *>(wrow + (size_t)sx * op.Kmax));
                const float2 w0 = unpack2(wv.x), w1 = unpack2(wv.y), w2 = unpack2(wv.z), w3 = unpack2(wv.w);
#pragma unroll
                for (int t = 0; t < TW; t++) {
                    const uint4 xv = col[t * ST + sx];
                    acc[t][0] = __ffma2_rn(unpack2(xv.x), w0, acc[t][0]);
                    acc[t][1] = __ffma2_rn(unpack2(xv.y), w1, acc[t][1]);
                    acc[t][2] = __ffma2_rn(unpack2(xv.z), w2, acc[t][2]);
                    acc[t][3] = __ffma2_rn(unpack2(xv.w), w3, acc[t][3]);
                }
            }
        }
        const float4 s0 = __ldg(reinterpret_cast<const float4 *>(op.scale + c0)), s1 = __ldg(reinterpret_cast<const float4 *>(op.scale + c0 + 4));
        const float4 h0 = __ldg(reinterpret_cast<const float4 *>(op.shift + c0)), h1 = __ldg(reinterpret_cast<const float4 *>(op.shift + c0 + 4));
        bf16 *yrow = y + ((size_t)ho * op.Wo) * Cn + c0;
#pragma unroll
        for (int t = 0; t < TW; t++) {
            const int wo = wo0 + t;
            if (wo < op.Wo) {
                const float v[8] = {acc[t][0].x * s0.x + h0.x, acc[t][0].y * s0.y + h0.y, acc[t][1].x * s0.z + h0.z, acc[t][1].y * s0.w + h0.w,
                                    acc[t][2].x * s1.x + h1.x, acc[t][2].y * s1.y + h1.y, acc[t][3].x * s1.z + h1.z, acc[t][3].y * s1.w + h1.w};
                uint4 ov;
                __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
                for (int j = 0; j < 4; j++) ob[j] = __floats2bfloat162_rn(act_fn(v[2 * j], op.act), act_fn(v[2 * j + 1], op.act));
                *reinterpret_cast<uint4 *>(yrow + (size_t)wo * Cn) = ov;
            }
        }
    }
}

// Stem: 3-channel image, k x k taps (k <= 3 here), stride `stride`, direct on the CUDA cores; a thread owns one
// output pixel and produces the filters eight at a time.  wsm: k * k * 3 * K floats of shared memory.
__device__ __noinline__ void pq_stem(const PqOp &op, const bf16 *img, bf16 *y, float *wsm) {
    const int k = op.k, K = op.K, taps = k * k * 3, o = (op.R - k) / 2, P = (k - 1) / 2;
    const bf16 *w = static_cast<const bf16 *>(op.w);
    for (int i = threadIdx.x; i < taps * K; i += PQ_THREADS) {
        const int f = i % K, t = i / K, c = t % 3, sx = (t / 3) % k, r = t / (3 * k);
        wsm[i] = __bfloat162float(__ldg(w + (((size_t)f * op.R + (o + r)) * op.R + (o + sx)) * op.ld + c));
    }
    __syncthreads();
    const int npx = op.Ho * op.Wo;
    for (int px = threadIdx.x; px < npx; px += PQ_THREADS) {
        const int ho = px / op.Wo, wo = px - ho * op.Wo;
        float in[27];
#pragma unroll
        for (int t = 0; t < 27; t++) in[t] = 0.f;
#pragma unroll
        for (int r = 0; r < 3; r++)
#pragma unroll
            for (int sx = 0; sx < 3; sx++) {
                const int hi = ho * op.stride + r - P, wi = wo * op.stride + sx - P;
                if (r < k && sx < k && hi >= 0 && hi < op.H && wi >= 0 && wi < op.W) {
                    const bf16 *pp = img + ((size_t)hi * op.W + wi) * 3;
#pragma unroll
                    for (int c = 0; c < 3; c++) in[(r * 3 + sx) * 3 + c] = __bfloat162float(__ldg(pp + c));
                }
            }
        for (int f0 = 0; f0 < K; f0 += 8) {
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int r = 0; r < 3; r++)
#pragma unroll
                for (int sx = 0; sx < 3; sx++)
                    if (r < k && sx < k) {
#pragma unroll
                        for (int c = 0; c < 3; c++) {
                            const float xv = in[(r * 3 + sx) * 3 + c];
                            const float4 *wp = reinterpret_cast<const float4 *>(wsm + ((r * k + sx) * 3 + c) * K + f0);  // (every lane the same address)
                            const float4 wa = wp[0], wb = wp[1];
                            acc[0] = fmaf(xv, wa.x, acc[0]); acc[1] = fmaf(xv, wa.y, acc[1]); acc[2] = fmaf(xv, wa.z, acc[2]); acc[3] = fmaf(xv, wa.w, acc[3]);
                            acc[4] = fmaf(xv, wb.x, acc[4]); acc[5] = fmaf(xv, wb.y, acc[5]); acc[6] = fmaf(xv, wb.z, acc[6]); acc[7] = fmaf(xv, wb.w, acc[7]);
                        }
                    }
            float ov[8];
#pragma unroll
            for (int q = 0; q < 8; q++) ov[q] = acc[q] * __ldg(op.scale + f0 + q) + __ldg(op.shift + f0 + q);
            finish_store(ov, nullptr, y, (size_t)px * K + f0, op.act);
        }
    }
}

// Global average pool into a shared-memory vector: a warp per 8-channel vector.
__device__ __forceinline__ void pq_gap(const PqOp &op, const bf16 *x, float *out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, cvecs = op.C >> 3, HW = op.H * op.W;
    const float inv = 1.f / (float)HW;
    for (int cv = warp; cv < cvecs; cv += PQ_WARPS) {
        const bf16 *base = x + cv * 8;
        float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int i = lane; i < HW; i += 32) {
            const uint4 v = *reinterpret_cast<const uint4 *>(base + (size_t)i * op.C);
            const float2 a = unpack2(v.x), b = unpack2(v.y), c = unpack2(v.z), d = unpack2(v.w);
            acc[0] += a.x; acc[1] += a.y; acc[2] += b.x; acc[3] += b.y; acc[4] += c.x; acc[5] += c.y; acc[6] += d.x; acc[7] += d.y;
        }
#pragma unroll
        for (int j = 0; j < 8; j++) {
#pragma unroll
            for (int o = 16; o; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
        }
        if (lane == 0) {
#pragma unroll
            for (int j = 0; j < 8; j++) out[cv * 8 + j] = acc[j] * inv;
        }
    }
}

// y[j] = f(bias[j] + sum_c w[j][c] * v[c]) for j < K: a warp takes JB outputs at a time and has the 16-byte weight
// loads of all of them in flight together.  HS: hard sigmoid (the squeeze-excite gate) instead of `act`.
template <int JB, bool HS>
__device__ __noinline__ void pq_matvec(const bf16 *w, int ld, const float *bias, const float *v, float *y, int C, int K, int act) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int j0 = warp * JB; j0 < K; j0 += PQ_WARPS * JB) {
        float s[JB];
#pragma unroll
        for (int u = 0; u < JB; u++) s[u] = 0.f;
        for (int c = lane * 8; c < C; c += 256) {
            uint4 wv[JB];
#pragma unroll
            for (int u = 0; u < JB; u++)
                wv[u] = j0 + u < K ? __ldg(reinterpret_cast<const uint4 *>(w + (size_t)(j0 + u) * ld + c)) : make_uint4(0u, 0u, 0u, 0u);
            const float4 x0 = *reinterpret_cast<const float4 *>(v + c), x1 = *reinterpret_cast<const float4 *>(v + c + 4);
#pragma unroll
            for (int u = 0; u < JB; u++) s[u] = dot8w(wv[u], x0, x1, s[u]);
        }
#pragma unroll
        for (int u = 0; u < JB; u++) {
#pragma unroll
            for (int o = 16; o; o >>= 1) s[u] += __shfl_xor_sync(0xffffffffu, s[u], o);
            if (lane == 0 && j0 + u < K) {
                const float t = s[u] + __ldg(bias + j0 + u);
                y[j0 + u] = HS ? fminf(fmaxf(t + 3.f, 0.f), 6.f) / 6.f : act_fn(t, act);
            }
        }
    }
}

// In-place squeeze-excite scale: x[p][c] *= gate[c].
__device__ __forceinline__ void pq_scale(const PqOp &op, bf16 *x, const float *gate) {
    const int cvecs = op.C >> 3, total = op.H * op.W * cvecs;
    for (int i = threadIdx.x; i < total; i += PQ_THREADS) {
        const int cv = i % cvecs;
        const uint4 v = *reinterpret_cast<const uint4 *>(x + (size_t)i * 8);
        const float4 g0 = *reinterpret_cast<const float4 *>(gate + cv * 8), g1 = *reinterpret_cast<const float4 *>(gate + cv * 8 + 4);
        const float2 a = unpack2(v.x), b = unpack2(v.y), c = unpack2(v.z), d = unpack2(v.w);
        uint4 o;
        __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&o);
        ob[0] = __floats2bfloat162_rn(a.x * g0.x, a.y * g0.y);
        ob[1] = __floats2bfloat162_rn(b.x * g0.z, b.y * g0.w);
        ob[2] = __floats2bfloat162_rn(c.x * g1.x, c.y * g1.y);
        ob[3] = __floats2bfloat162_rn(d.x * g1.z, d.y * g1.w);
        *reinterpret_cast<uint4 *>(x + (size_t)i * 8) = o;
    }
}

__global__ void __launch_bounds__(PQ_THREADS, PQ_BLOCKS_PER_SM) subnet_kernel(const PqParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t *ring = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    __shared__ __align__(16) float vec_s[3][PQ_VEC];
    __shared__ __align__(16) float bn_s[2 * PQ_MAX_K];
    __shared__ __align__(16) PqOp op_s;
    __shared__ __align__(16) PqQuery q_s;
    __shared__ __align__(8) uint64_t free_bar[4], acc_bar[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s, next_s;
    volatile int *abort_flag = &abort_s;
    const int tid = threadIdx.x, warp = tid >> 5;

    if (tid == 0) {
        for (int s = 0; s < 4; s++) mbar_init(&free_bar[s], 1);
        mbar_init(&acc_bar[0], 1);
        mbar_init(&acc_bar[1], 1);
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) tmem_alloc(&tmem_base_s, 2 * PQ_ACC_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    PipeState ps;
    ps.use[0] = ps.use[1] = ps.use[2] = ps.use[3] = 0u; ps.acc[0] = ps.acc[1] = 0u; ps.tiles = 0u;
    uint8_t *slot = p.scratch + (size_t)blockIdx.x * p.slot_bytes;
    bool ok = true;
    // the weight buffer: behind the ring, filled once
    const uint32_t held_u32 = p.n_held > 0 ? smem_u32(ring + PQ_RING_BYTES) : 0u;
    if (p.n_held > 0) {
        const int c16 = tid & 7, r0 = tid >> 3;
        const uint32_t piece = (uint32_t)((c16 ^ (r0 & 7)) << 4);
        for (int e = 0; e < p.n_held; e++) {
            const PqHeld h = p.held[e];
            const bf16 *hw = static_cast<const bf16 *>(h.w);
            for (int ch = 0; ch < h.chunks; ch++) {
                const int c0 = ch * 64 + c16 * 8;
                const uint32_t dst = held_u32 + h.off + (uint32_t)(ch * h.rows * 128);
                for (int row = r0; row < h.rows; row += PQ_ROWS) cp16_cg(dst + (uint32_t)(row * 128) + piece, c0 < h.C ? hw + (size_t)row * h.ld + c0 : hw, c0 < h.C);
            }
        }
        cp_commit();
        cp_wait<0>();
        fence_async_smem();
        __syncthreads();
    }

    for (;;) {
        if (tid == 0) next_s = atomicAdd(p.counter, 1);
        __syncthreads();
        const int qi = next_s;
        if (qi >= p.n_queries || *abort_flag) break;
        if (tid < 2) reinterpret_cast<uint4 *>(&q_s)[tid] = __ldg(reinterpret_cast<const uint4 *>(p.queries + qi) + tid);
        __syncthreads();
        const int op_begin = q_s.op_begin, op_count = q_s.op_count;
        for (int oi = 0; oi < op_count; oi++) {
            __syncthreads();  // the previous layer is complete: its outputs are visible, its record is free
            if (*abort_flag) break;
            if (tid < 8) reinterpret_cast<uint4 *>(&op_s)[tid] = __ldg(reinterpret_cast<const uint4 *>(p.ops + op_begin + oi) + tid);
            __syncthreads();
            const PqOp &op = op_s;
            const bf16 *x = op.in < 0 ? static_cast<const bf16 *>(q_s.x) : reinterpret_cast<const bf16 *>(slot + (size_t)op.in * p.act_bytes);
            bf16 *y = op.out < 0 ? nullptr : reinterpret_cast<bf16 *>(slot + (size_t)op.out * p.act_bytes);
            const bf16 *res = op.res < 0 ? nullptr : reinterpret_cast<const bf16 *>(slot + (size_t)op.res * p.act_bytes);
            switch (op.type) {
            case PQ_STEM: pq_stem(op, x, y, reinterpret_cast<float *>(ring)); break;
            case PQ_PW: ok = pq_pointwise(op, x, res, y, ring, bn_s, held_u32, free_bar, acc_bar, tmem_base, ps, abort_flag) && ok; break;
            case PQ_DW:
                if (op.stride == 1) {
                    if (op.k == 3) pq_depthwise<3, 1>(op, x, y);
                    else if (op.k == 5) pq_depthwise<5, 1>(op, x, y);
                    else pq_depthwise<7, 1>(op, x, y);
                } else {
                    if (op.k == 3) pq_depthwise<3, 2>(op, x, y);
                    else if (op.k == 5) pq_depthwise<5, 2>(op, x, y);
                    else pq_depthwise<7, 2>(op, x, y);
                }
                break;
            case PQ_GAP: pq_gap(op, x, vec_s[op.vout]); break;
            case PQ_SE_GATE:
                // first FC (ReLU) into the third vector, second FC (hard sigmoid) into the gate
                pq_matvec<4, false>(static_cast<const bf16 *>(op.w), op.ld, op.shift, vec_s[op.vin], vec_s[2], op.C, op.K, ACT_RELU);
                __syncthreads();
                pq_matvec<8, true>(static_cast<const bf16 *>(op.w2), op.ld2, op.bias2, vec_s[2], vec_s[op.vout], op.K, op.C, 0);
                break;
            case PQ_SCALE: pq_scale(op, y, vec_s[op.vin]); break;
            case PQ_LINEAR:
                pq_matvec<8, false>(static_cast<const bf16 *>(op.w), op.ld, op.shift, vec_s[op.vin], op.vout < 0 ? q_s.logits : vec_s[op.vout], op.C, op.K, op.act);
                break;
            default: break;
            }
        }
        __syncthreads();  // (also keeps next_s and q_s until every thread is done with them)
        if (*abort_flag) break;
    }
    // (every thread left the loops after the same block barrier; the flag is only written inside waits)
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem_base, 2 * PQ_ACC_COLS);
    if (tid == 0 && (*abort_flag || !ok)) atomicExch(p.status, 1);
}

}  // namespace

size_t subnet_kernel_smem() { return (size_t)PQ_RING_BYTES + 1024; }
size_t subnet_kernel_held_max() { return (size_t)PQ_HELD_MAX; }
int subnet_kernel_blocks_per_sm() { return PQ_BLOCKS_PER_SM; }

cudaError_t subnet_kernel_init(int device) {
    (void)device;
    return cudaFuncSetAttribute(subnet_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(subnet_kernel_smem() + PQ_HELD_MAX));
}

cudaError_t subnet_kernel_launch(const PqParams &p, int blocks, cudaStream_t st) {
    if (blocks <= 0) return cudaSuccess;
    if (p.held_bytes > (unsigned)PQ_HELD_MAX || (p.held_bytes & 1023u)) return cudaErrorInvalidValue;
    subnet_kernel<<<blocks, PQ_THREADS, subnet_kernel_smem() + (p.n_held > 0 ? p.held_bytes : 0u), st>>>(p);
    return cudaGetLastError();
}

}  // namespace sgs
