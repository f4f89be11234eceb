// Grouped sliced convolution: ONE launch runs the same stored layer for many queries in flight, each
// with its own SubNet slice (paper Section 2.1: every query selects its own filters / channels of the
// shared layer; Section 3.1: a stream of such queries).  A launch gets a table with one entry per
// member (query): its tensor maps, slice extents, tile geometry and buffers.  All members' output tiles
// form one list of tiles; persistent CTAs (one per SM) walk that list with a fixed stride.
//
// Per CTA: warp 0 = weight producer, warp 10 = activation producer, warp 1 = MMA issuer, warps 2..9 =
// two epilogue groups.  The shared-memory ring of operand stages runs on across tiles, and the fp32
// accumulator in tensor memory is double buffered (2 x 256 columns, one buffer per epilogue group), so the
// epilogues of tiles j and j + 1 (tensor memory -> folded batch norm -> residual -> activation -> bf16
// NHWC) overlap each other and the loads and MMAs of the tiles that follow.
//
// The arithmetic of one tile is that of conv_tc_kernel (sgs_conv_tc.cu): implicit GEMM with
// 128 output pixels x up to 256 filters, 64 channels per stage, slicing through the tensor maps'
// extents.  The reduction is never split here: with many members in flight the tiles alone fill the GPU.
#include "sgs_tc.cuh"

#include <algorithm>
#include <cstring>

namespace sgs {

namespace {

constexpr int G_MAX_STAGES = 8;
constexpr int G_X_BYTES = 128 * CHUNK_C * 2;  // operand on the MMA's row side: 128 rows
constexpr int G_RING_BYTES = 192 * 1024;      // operand ring: 8 stages of 16 + 8 KB (tiles of at most 64 columns), 6 of 16 + 16 KB, or 4 of 16 + 32 KB (256-column tiles)
constexpr int G_SMEM_BYTES = G_RING_BYTES + 1024;
constexpr int G_ACC_COLS = 256;                   // tensor-memory columns of one accumulator buffer
constexpr int G_EPI_WARPS = 8;                    // two groups of four (one warp per tensor-memory lane quadrant)
constexpr int G_THREADS = 64 + 32 * G_EPI_WARPS + 32;  // weight producer, MMA warp, epilogue warps, pixel producer
constexpr int G_PIX_WARP = 2 + G_EPI_WARPS;

// One member (query) of a grouped launch.
//   normal  : MMA rows = a box of <= 128 output pixels, MMA columns = bn_tile (64 / 128 / 256) filters
//   swapped : MMA rows = 128 filters, MMA columns = ALL output pixels of the member (<= 256, padded to 16)
struct __align__(16) GroupEntry {
    const float *scale, *shift;
    const __nv_bfloat16 *res;
    __nv_bfloat16 *y;
    int map_a, map_w;        // indices into the launch's tensor maps: activation view(s) (4 for stride-2 kernels
                             // larger than 1x1: the parity views; else 1) and the sliced weight view
    int tile_begin;          // index of this member's first tile in the launch's tile list
    int mtiles;              // pixel tiles of this member (tile = filter tile * mtiles + pixel tile)
    int N, Ho, Wo, K, C;
    int R, tap0;             // stored kernel size; tap index of the cropped kernel's first tap
    int tiles_w, tiles_hw, cchunks, iters, layer;
    short bw, bh, bn;        // pixel box
    short bn_tile;           // MMA columns of a full tile
    short pix_rows;          // rows of the pixel box (bw * bh * bn)
    short pad0_;
    unsigned char k, stride, p, act, swap, kw;  // k x kw taps
    // Two members with at most 64 output pixels each can share a tile: the first ("pair") owns the tile's
    // geometry, filters and weight map and takes MMA rows 0..63, the entry after it ("second") takes rows
    // 64..127 with its own activation map, outputs and filter count (not larger than the first's).
    unsigned char pair, second;
    int ldk;                 // channels per pixel of y and res as stored (>= K; the kernel writes zeros into K..ldk-1)
    // SubGraph cache box of this member's query (the cached SubGraph in force when the query is served, in stream
    // order): weight tiles with filter < cacheK and channel < cacheC are loaded evict-last; cacheK == -1: every
    // weight load evict-first; 0: no hint
    int cacheK, cacheC;
};
static_assert(sizeof(GroupEntry) == TC_GROUP_ENTRY_BYTES, "entry size");

// Index of the entry that owns tile t (entries are sorted by tile_begin); the whole warp calls it.
__device__ __forceinline__ int find_entry(const GroupEntry *es, int n, int t, int lane) {
    const unsigned b0 = __ballot_sync(0xffffffffu, lane < n && es[lane].tile_begin <= t);
    const unsigned b1 = __ballot_sync(0xffffffffu, lane + 32 < n && es[lane + 32].tile_begin <= t);
    return __popc(b0) + __popc(b1) - 1;
}
// Same for one thread.
__device__ __forceinline__ int find_entry_serial(const GroupEntry *es, int n, int t) {
    int lo = 0, hi = n - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (es[mid].tile_begin <= t) lo = mid; else hi = mid - 1;
    }
    return es[lo].second ? lo - 1 : lo;
}
// The entry that owns tile t's geometry (the first member of a pair); the whole warp calls it.
__device__ __forceinline__ int tile_entry(const GroupEntry *es, int n, int t, int lane) {
    const int i = find_entry(es, n, t, lane);
    return es[i].second ? i - 1 : i;
}

// Named barrier of one epilogue group (4 warps): id 1 or 2.
__device__ __forceinline__ void group_bar(int grp) { asm volatile("bar.sync %0, 128;" ::"r"(grp + 1) : "memory"); }
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap *m) { asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory"); }


// Kernel parameters.  The tensor maps travel in the parameter block (the TMA unit reads them from
// there); the per-member records travel in a device table.
template <int NMAPS> struct GroupParams {
    const GroupEntry *entries;
    const void *unused_;
    int *status;
    int n_entries, total_tiles;
    int n_stages, stage_bytes;  // operand ring of this launch
    int group;                  // consecutive stages that share one pair of barriers (n_stages is a multiple of it)
    int pad_[5];
    CUtensorMap maps[NMAPS];
};
static_assert(sizeof(GroupParams<TC_GROUP_MAPS_LARGE>) <= 32764, "kernel parameter block");

template <int NMAPS>
__global__ void __launch_bounds__(G_THREADS, 1) conv_group_kernel(const __grid_constant__ GroupParams<NMAPS> P) {
    const GroupEntry *__restrict__ entries = P.entries;
    const int n_entries = P.n_entries, total_tiles = P.total_tiles;
    int *status = P.status;
    extern __shared__ uint8_t smem_raw[];
    __shared__ GroupEntry es[TC_GROUP_MAX_ENTRIES];
    __shared__ float scale_s[2][2][G_ACC_COLS], shift_s[2][2][G_ACC_COLS];  // per epilogue group: folded batch norm of its current / next tile's filters
    __shared__ __align__(8) uint64_t full_bar[G_MAX_STAGES], empty_bar[G_MAX_STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int abort_s;

    uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    volatile int *abort_flag = &abort_s;

    // The table was uploaded before the first kernel of the stream segment, so it may be read before
    // the wait on the previous layer.
    for (int i = threadIdx.x; i < n_entries * (int)(sizeof(GroupEntry) / 16); i += blockDim.x)
        reinterpret_cast<uint4 *>(es)[i] = __ldg(reinterpret_cast<const uint4 *>(entries) + i);
    if (threadIdx.x == 0) {
        // Barriers are per GROUP of consecutive stages: a group is full once both producers' copies of all its
        // stages have landed (each producer arrives once per stage), and empty once the MMAs of its last stage
        // have read it.  One wait and one commit then serve `group` stages: the issuing threads pay their fixed
        // cost per wait (a few hundred cycles) once per group instead of once per 64 channels.
        for (int s = 0; s < G_MAX_STAGES; s++) { mbar_init(&full_bar[s], 2 * (uint32_t)P.group); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; b++) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], G_EPI_WARPS / 2); }
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_base_s, 2 * G_ACC_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const int n_stages = P.n_stages, stage_bytes = P.stage_bytes, gsz = P.group;
    pdl_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------------ weight producer
        // Weights do not depend on the previous layer, so this warp never waits for it: it runs ahead
        // as far as the ring allows.  The warp runs its loop converged; one elected lane issues.
        const uint64_t pol_keep = make_policy(1), pol_stream = make_policy(2);
        int s = 0, g = 0, gi = 0;  // stage, its group, its position in the group
        uint32_t phase = 0;
        bool wrapped = false, ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const GroupEntry &e = es[tile_entry(es, n_entries, t, lane)];
            const int nt = (t - e.tile_begin) / e.mtiles;
            const int wrows = e.swap ? 128 : e.bn_tile;  // rows of the weight box
            const int f0 = nt * wrows;
            const uint32_t w_bytes = (uint32_t)(wrows * CHUNK_C * 2);
            uint8_t *dst0 = smem + (e.swap ? 0 : G_X_BYTES);
            const CUtensorMap *map_w = &P.maps[e.map_w];
            const int k = e.k, kw = e.kw, cchunks = e.cchunks, R = e.R;
            int kind = 0;  // 0 default replacement, 1 keep (inside the cached SubGraph's box, up to channel cacheC), 2 stream
            int cacheC = 0;
            if (e.cacheK < 0) kind = 2;
            else if (f0 < e.cacheK) { kind = 1; cacheC = e.cacheC; }
            int tap_row = e.tap0;
            for (int r = 0; r < k && ok; r++, tap_row += R) {
                for (int sx = 0; sx < kw && ok; sx++) {
                    for (int cc = 0, c0 = 0; cc < cchunks; cc++, c0 += CHUNK_C) {
                        if (wrapped && gi == 0) ok = __all_sync(0xffffffffu, mbar_wait(&empty_bar[g], phase ^ 1, abort_flag));
                        if (!ok) break;
                        if (elect_one()) {
                            uint8_t *sb = dst0 + s * stage_bytes;
                            mbar_expect_tx(&full_bar[g], w_bytes);
                            if (kind == 2) tma_load_3d_hint(sb, map_w, &full_bar[g], c0, tap_row + sx, f0, pol_stream);
                            else if (kind == 1 && c0 < cacheC) tma_load_3d_hint(sb, map_w, &full_bar[g], c0, tap_row + sx, f0, pol_keep);
                            else tma_load_3d(sb, map_w, &full_bar[g], c0, tap_row + sx, f0);
                        }
                        __syncwarp();
                        if (++gi == gsz) { gi = 0; ++g; }
                        if (++s == n_stages) { s = 0; g = 0; phase ^= 1; wrapped = true; }
                    }
                }
            }
            const int tn = t + (int)gridDim.x;
            if (ok && tn < total_tiles && elect_one()) prefetch_tensormap(&P.maps[es[find_entry_serial(es, n_entries, tn)].map_w]);
            __syncwarp();
        }
        // the CTA's last group may be partial: arrive for the stages it does not have
        if (gi != 0 && elect_one())
            for (; gi < gsz; gi++) mbar_arrive(&full_bar[g]);
    } else if (warp == G_PIX_WARP) {
        // ------------------------------------------------------------------ activation producer
        int s = 0, g = 0, gi = 0;
        uint32_t phase = 0;
        bool wrapped = false, ok = true;
        pdl_wait();  // activations (and the buffers this layer overwrites) belong to the previous layers until here
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const GroupEntry &e = es[tile_entry(es, n_entries, t, lane)];
            const int mt = (t - e.tile_begin) % e.mtiles;
            const int n0 = (mt / e.tiles_hw) * e.bn, h0 = ((mt % e.tiles_hw) / e.tiles_w) * e.bh, w0 = (mt % e.tiles_w) * e.bw;
            const uint32_t pix_bytes = (uint32_t)(e.pix_rows * CHUNK_C * 2);
            uint8_t *dst0 = smem + (e.swap ? G_X_BYTES : 0);
            const CUtensorMap *map_a = &P.maps[e.map_a];
            const uint32_t pix_bytes2 = e.pair ? (uint32_t)((&e)[1].pix_rows * CHUNK_C * 2) : 0u;
            const CUtensorMap *map_a2 = &P.maps[e.pair ? (&e)[1].map_a : e.map_a];
            const int k = e.k, kw = e.kw, cchunks = e.cchunks, pad = e.p, stride = e.stride;
            for (int r = 0; r < k && ok; r++) {
                for (int sx = 0; sx < kw && ok; sx++) {
                    const int dh = r - pad, dw = sx - pad;
                    // stride 2: one of the four parity views, at half the offset
                    const int ph = stride == 2 ? (dh & 1) : 0, pw = stride == 2 ? (dw & 1) : 0;
                    const CUtensorMap *m = map_a + ph * 2 + pw;
                    const int cw = stride == 2 ? w0 + ((dw - pw) >> 1) : w0 + dw, ch = stride == 2 ? h0 + ((dh - ph) >> 1) : h0 + dh;
                    for (int cc = 0, c0 = 0; cc < cchunks; cc++, c0 += CHUNK_C) {
                        if (wrapped && gi == 0) ok = __all_sync(0xffffffffu, mbar_wait(&empty_bar[g], phase ^ 1, abort_flag));
                        if (!ok) break;
                        if (elect_one()) {
                            mbar_expect_tx(&full_bar[g], pix_bytes + pix_bytes2);
                            tma_load_4d(dst0 + s * stage_bytes, m, &full_bar[g], c0, cw, ch, n0);
                            // (a pair is a single tile of one layer: same tap offsets and parity view, box origin 0)
                            if (pix_bytes2) tma_load_4d(dst0 + s * stage_bytes + 64 * CHUNK_C * 2, map_a2 + (m - map_a), &full_bar[g], c0, cw, ch, n0);
                        }
                        __syncwarp();
                        if (++gi == gsz) { gi = 0; ++g; }
                        if (++s == n_stages) { s = 0; g = 0; phase ^= 1; wrapped = true; }
                    }
                }
            }
            const int tn = t + (int)gridDim.x;
            if (ok && tn < total_tiles && elect_one()) prefetch_tensormap(&P.maps[es[find_entry_serial(es, n_entries, tn)].map_a]);
            __syncwarp();
        }
        if (gi != 0 && elect_one())
            for (; gi < gsz; gi++) mbar_arrive(&full_bar[g]);
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        int s = 0, g = 0, gi = 0;
        uint32_t phase = 0;
        int j = 0;
        const uint32_t ring = smem_u32(smem);
        bool ok = true;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x, j++) {
            const GroupEntry &e = es[tile_entry(es, n_entries, t, lane)];
            const int nt = (t - e.tile_begin) / e.mtiles;
            // MMA shape: 128 rows; columns = this tile's filters (normal) or the member's pixels (swapped),
            // rounded up to 16; bf16 x bf16 -> fp32, both operands K-major
            const int n_mma = e.swap ? e.bn_tile : min((int)e.bn_tile, (e.K - nt * e.bn_tile + 15) & ~15);
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
            const int buf = j & 1;
            const int cchunks = e.cchunks, taps = e.k * e.kw;
            const int last_ksteps = (e.C - (cchunks - 1) * CHUNK_C + 15) / 16;  // 16-channel steps of a tap's last chunk
            ok = j < 2 || mbar_wait(&acc_empty[buf], ((j >> 1) - 1) & 1, abort_flag);  // epilogue drained this buffer
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * G_ACC_COLS);
            uint32_t accumulate = 0;
            for (int tap = 0; tap < taps && ok; tap++) {
                for (int cc = 0; cc < cchunks; cc++) {
                    if (gi == 0) {
                        ok = __all_sync(0xffffffffu, mbar_wait(&full_bar[g], phase, abort_flag));
                        if (!ok) break;
                        tc_fence_after();
                    }
                    const int ksteps = cc == cchunks - 1 ? last_ksteps : CHUNK_C / 16;
                    const uint32_t sx_ = ring + (uint32_t)(s * stage_bytes);
                    const uint64_t da = smem_desc_sw128(sx_), db = smem_desc_sw128(sx_ + G_X_BYTES);
                    if (elect_one()) {
                        for (int q = 0; q < ksteps; q++) { umma_bf16(d_tmem, da + (uint64_t)(2 * q), db + (uint64_t)(2 * q), idesc, accumulate); accumulate = 1; }
                        if (gi == gsz - 1) umma_commit(&empty_bar[g]);  // frees the group once the MMAs of all its stages have read it
                        if (tap == taps - 1 && cc == cchunks - 1) umma_commit(&acc_full[buf]);  // accumulator complete
                    }
                    __syncwarp();
                    accumulate = 1;
                    if (++gi == gsz) { gi = 0; ++g; }
                    if (++s == n_stages) { s = 0; g = 0; phase ^= 1; }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..9)
        // Two groups of four warps (one per tensor-memory lane quadrant).  Group g owns accumulator buffer g
        // and takes the CTA's tiles j with j % 2 == g, so the epilogues of two consecutive tiles run side by
        // side; a thread handles one accumulator row and all of the tile's columns, 32 at a time.
        const int quad = warp & 3;                // tensor-memory lane quadrant this warp may read
        const int grp = (warp - 2) >> 2;          // epilogue group = accumulator buffer
        const int row_all = quad * 32 + lane;     // accumulator row: output pixel (normal) or filter (swapped)
        const int et = (threadIdx.x - 64) & 127;  // thread within the group
        float(*scale_g)[G_ACC_COLS] = scale_s[grp];
        float(*shift_g)[G_ACC_COLS] = shift_s[grp];
        const int stride2 = 2 * (int)gridDim.x;
        pdl_wait();  // residual reads and output writes must not pass the previous layers
        bool alive = true;  // after a failed wait the warp only keeps the named barrier in step
        // folded batch norm of a normal tile: thread et fetches the scale and shift of filters et and et + 128
        auto fetch_bn = [&](int tile, float *v) {
            v[0] = v[1] = v[2] = v[3] = 0.f;
            if (tile >= total_tiles) return;
            const GroupEntry &e = es[tile_entry(es, n_entries, tile, lane)];
            if (e.swap) return;
            const int f = ((tile - e.tile_begin) / e.mtiles) * e.bn_tile + et;
            if (et < e.bn_tile && f < e.K) { v[0] = __ldg(e.scale + f); v[1] = __ldg(e.shift + f); }
            if (et + 128 < e.bn_tile && f + 128 < e.K) { v[2] = __ldg(e.scale + f + 128); v[3] = __ldg(e.shift + f + 128); }
        };
        auto store_bn = [&](int b, const float *v) {
            scale_g[b][et] = v[0]; shift_g[b][et] = v[1]; scale_g[b][et + 128] = v[2]; shift_g[b][et + 128] = v[3];
        };
        {
            float v[4];
            fetch_bn((int)blockIdx.x + grp * (int)gridDim.x, v);
            store_bn(0, v);
        }
        int jj = 0;  // tiles this group has taken
        for (int t = (int)blockIdx.x + grp * (int)gridDim.x; t < total_tiles; t += stride2, jj++) {
            const GroupEntry &e0 = es[tile_entry(es, n_entries, t, lane)];
            const int local = t - e0.tile_begin, nt = local / e0.mtiles, mt = local % e0.mtiles;
            // rows 64..127 of a pair's tile belong to the second member (a warp lies on one side)
            const bool second_half = e0.pair && quad >= 2;
            const GroupEntry &e = second_half ? (&e0)[1] : e0;
            const int row = second_half ? row_all - 64 : row_all;
            const int K = e.K, ldk = e.ldk, act = e.act;
            const __nv_bfloat16 *res = e.res;
            __nv_bfloat16 *y = e.y;
            const int sb = jj & 1;  // which of the group's two scale / shift tables
            const uint32_t tacc = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(grp * G_ACC_COLS);
            float nbn[4];
            fetch_bn(t + stride2, nbn);  // requested now, stored after this tile's work
            if (!e.swap) {
                // ---- normal tile: this thread owns output pixel `m`, columns are filters
                const int n0 = (mt / e.tiles_hw) * e.bn, h0 = ((mt % e.tiles_hw) / e.tiles_w) * e.bh, w0 = (mt % e.tiles_w) * e.bw;
                const int f0 = nt * e0.bn_tile;
                int m;
                {
                    const int dn = row / (e.bh * e.bw), dhh = (row / e.bw) % e.bh, dww = row % e.bw;
                    const int n = n0 + dn, h = h0 + dhh, w = w0 + dww;
                    const bool valid = row < e.pix_rows && n < e.N && h < e.Ho && w < e.Wo;
                    m = valid ? (int)(((size_t)n * e.Ho + h) * e.Wo + w) : -1;
                }
                const int cend = min((int)e0.bn_tile, K - f0);  // filters of this tile, a multiple of 8 (<= 0: none of this member's)
                const int cpad = min((int)e0.bn_tile, ldk - f0);  // ... and the end of the pixel's padding, written as zeros
                const size_t obase = (size_t)(m < 0 ? 0 : m) * ldk + f0;
                // the residual does not depend on the accumulator: the first 64 columns' part is requested
                // before waiting, every further part two steps ahead of its use (a thread then has 8 loads of
                // 16 bytes in flight: the epilogue of a tile with a residual is bound by their latency).
                // (Measured alternative: transposing the accesses through a warp-private staging block so that a
                // warp touches 8 rows x 64 contiguous bytes instead of 32 rows x 16 bytes changed no layer's time
                // at 16 images per member and cost 1.7 % on the batch-1 stream.)
                auto load_res = [&](int c0, uint4 *rv) {
#pragma unroll
                    for (int g = 0; g < 4; g++) {
                        const int c = c0 + 8 * g;
                        rv[g] = (res && m >= 0 && c < cend) ? __ldg(reinterpret_cast<const uint4 *>(res + obase + c)) : make_uint4(0u, 0u, 0u, 0u);
                    }
                };
                uint4 rv[4], rn[4];
                load_res(0, rv);
                load_res(32, rn);
                group_bar(grp);  // this tile's scale / shift (written during the group's previous tile) are visible
                const float *sc = scale_g[sb], *sh = shift_g[sb];
                if (alive) alive = __all_sync(0xffffffffu, mbar_wait(&acc_full[grp], jj & 1, abort_flag));
                if (alive) {
                    tc_fence_after();
#pragma unroll 1
                    for (int c0 = 0; c0 < cpad; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld32(tacc + c0, v);
                        uint4 rf[4];
                        load_res(c0 + 64, rf);
                        tmem_ld_wait();
                        if (m >= 0) {
#pragma unroll
                            for (int g = 0; g < 4; g++) {
                                const int c = c0 + 8 * g;
                                if (c >= cend && c < cpad) *reinterpret_cast<uint4 *>(y + obase + c) = make_uint4(0u, 0u, 0u, 0u);
                                if (c < cend) {
                                    float ov[8];
#pragma unroll
                                    for (int q = 0; q < 8; q++) ov[q] = __uint_as_float(v[8 * g + q]) * sc[c + q] + sh[c + q];
                                    const __nv_bfloat162 *rb = reinterpret_cast<const __nv_bfloat162 *>(&rv[g]);
#pragma unroll
                                    for (int q = 0; q < 4; q++) { const float2 f2 = __bfloat1622float2(rb[q]); ov[2 * q] += f2.x; ov[2 * q + 1] += f2.y; }
                                    finish_store(ov, nullptr, y, obase + c, act);
                                }
                            }
                        }
#pragma unroll
                        for (int g = 0; g < 4; g++) { rv[g] = rn[g]; rn[g] = rf[g]; }
                    }
                }
            } else {
                // ---- swapped tile: this thread owns filter `f`, columns are the member's output pixels
                const int f = nt * 128 + row;
                const bool fvalid = f < K, fpad = f >= K && f < ldk;
                const int cend = e.pix_rows;  // == N * Ho * Wo: the pixel tile is the whole member
                float sc = 0.f, sh = 0.f;
                if (fvalid) { sc = __ldg(e.scale + f); sh = __ldg(e.shift + f); }
                const unsigned short *resu = reinterpret_cast<const unsigned short *>(res);
                auto load_res = [&](int c0, uint32_t *rv) {  // 32 pixels, two per register
#pragma unroll
                    for (int q = 0; q < 16; q++) {
                        const int p0 = c0 + 2 * q;
                        uint32_t lo = 0, hi = 0;
                        if (res && fvalid && p0 < cend) lo = __ldg(resu + (size_t)p0 * ldk + f);
                        if (res && fvalid && p0 + 1 < cend) hi = __ldg(resu + (size_t)(p0 + 1) * ldk + f);
                        rv[q] = lo | (hi << 16);
                    }
                };
                uint32_t rv[16];
                load_res(0, rv);
                group_bar(grp);
                if (alive) alive = __all_sync(0xffffffffu, mbar_wait(&acc_full[grp], jj & 1, abort_flag));
                if (alive) {
                    tc_fence_after();
#pragma unroll 1
                    for (int c0 = 0; c0 < cend; c0 += 32) {
                        uint32_t v[32];
                        tmem_ld32(tacc + c0, v);
                        uint32_t rn[16];
                        load_res(c0 + 32, rn);
                        tmem_ld_wait();
                        if (fvalid) {
#pragma unroll
                            for (int q = 0; q < 32; q++) {
                                const int px = c0 + q;
                                if (px < cend) {
                                    const uint32_t rbits = (q & 1) ? (rv[q >> 1] & 0xffff0000u) : (rv[q >> 1] << 16);
                                    const float o = act_fn(__uint_as_float(v[q]) * sc + sh + __uint_as_float(rbits), act);
                                    y[(size_t)px * ldk + f] = __float2bfloat16_rn(o);
                                }
                            }
                        } else if (fpad) {
#pragma unroll
                            for (int q = 0; q < 32; q++)
                                if (c0 + q < cend) y[(size_t)(c0 + q) * ldk + f] = __float2bfloat16_rn(0.f);
                        }
#pragma unroll
                        for (int q = 0; q < 16; q++) rv[q] = rn[q];
                    }
                }
            }
            if (alive) {
                // hand the accumulator buffer back to the MMA warp
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&acc_empty[grp]);
            }
            // the group read table sb ^ 1 for the last time during its previous tile, which all of its
            // threads have left (barrier above)
            store_bn(sb ^ 1, nbn);
        }
    }
    // ---------------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (abort_s) {
        if (threadIdx.x == 0) atomicExch(status, 1);
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 2000000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 2 * G_ACC_COLS); }
}

}  // namespace

// Number of activation views a member needs: the four parity views only when a stride-2 kernel
// reaches odd offsets, i.e. for kernels larger than 1x1.
static int views_of(const TcParams &p) { return (p.stride == 2 && p.k > 1) ? 4 : 1; }  // (a stride-2 window view uses views 0 and 2 of 4)

struct GroupLaunch::Impl {
    GroupParams<TC_GROUP_MAPS_LARGE> prm;  // host image of the parameter block (the small variant is a prefix)
    int n_maps = 0;
    int col_rows = 0;   // most rows any member's column-side operand has (64, 128 or 256: sizes the stages)
    const void *win_base = nullptr;  // largest cached filter prefix among the members' stored layers
    size_t win_bytes = 0;
};

GroupLaunch::GroupLaunch() : impl(new Impl) { reset(nullptr); }
GroupLaunch::~GroupLaunch() { delete impl; }

void GroupLaunch::reset(const void *d_entries) {
    impl->n_maps = 0;
    impl->col_rows = 0;
    impl->win_base = nullptr;
    impl->win_bytes = 0;
    impl->prm.entries = static_cast<const GroupEntry *>(d_entries);
    impl->prm.n_entries = 0;
    impl->prm.total_tiles = 0;
}
int GroupLaunch::members() const { return impl->prm.n_entries; }
int GroupLaunch::maps() const { return impl->n_maps; }
int GroupLaunch::tiles() const { return impl->prm.total_tiles; }

bool GroupLaunch::fits(const TcConvPlan &pl) const {
    return impl->prm.n_entries < TC_GROUP_MAX_ENTRIES && impl->n_maps + views_of(pl.prm) + 1 <= TC_GROUP_MAPS_LARGE;
}

void GroupLaunch::add(void *host_entry, const TcConvPlan &pl, const ConvArgs &a) {
    const TcParams &p = pl.prm;
    GroupEntry e;
    std::memset(&e, 0, sizeof e);
    const int views = views_of(p);
    e.map_a = impl->n_maps;
    std::memcpy(&impl->prm.maps[impl->n_maps], p.tmA, (size_t)views * sizeof(CUtensorMap));
    impl->n_maps += views;
    e.map_w = impl->n_maps;
    std::memcpy(&impl->prm.maps[impl->n_maps], &p.tmW, sizeof(CUtensorMap));
    impl->n_maps += 1;
    e.scale = a.scale; e.shift = a.shift;
    e.res = static_cast<const __nv_bfloat16 *>(a.res);
    e.y = static_cast<__nv_bfloat16 *>(a.y);
    e.tile_begin = impl->prm.total_tiles;
    e.mtiles = (int)pl.grid.x;
    e.N = p.N; e.Ho = p.Ho; e.Wo = p.Wo; e.K = p.K; e.C = p.C;
    e.ldk = a.ldy ? a.ldy : p.K;
    // weight_policy 1: per-tile hints from the box; 2: all evict-first; 3: the box only feeds the launch's window
    e.cacheK = a.weight_policy == 2 ? -1 : a.weight_policy == 1 ? a.cacheK : 0;
    e.cacheC = a.weight_policy == 1 ? a.cacheC : 0;
    if ((a.weight_policy == 1 || a.weight_policy == 3) && a.cacheK > 0) {
        // the launch's access-policy window (optional mechanism): the filters [0, cacheK) of this stored layer, whole rows
        const size_t bytes = (size_t)a.cacheK * a.R * a.R * a.Cmax * 2;
        if (bytes > impl->win_bytes) { impl->win_base = a.w; impl->win_bytes = bytes; }
    }
    e.R = p.R; e.tap0 = p.o * p.R + p.o;
    e.tiles_w = p.tiles_w; e.tiles_hw = p.tiles_w * p.tiles_h;
    e.cchunks = p.cchunks; e.iters = p.iters; e.layer = a.layer;
    e.bw = (short)p.bw; e.bh = (short)p.bh; e.bn = (short)p.bn;
    e.pix_rows = (short)(p.bw * p.bh * p.bn);
    e.swap = (unsigned char)pl.swap;
    e.bn_tile = (short)(pl.swap ? (e.pix_rows + 15) / 16 * 16 : pl.bn_tile);
    e.k = (unsigned char)p.k; e.kw = (unsigned char)pl.kw; e.stride = (unsigned char)p.stride; e.p = (unsigned char)p.p; e.act = (unsigned char)p.act;
    impl->col_rows = std::max(impl->col_rows, (int)(pl.swap ? e.pix_rows : e.bn_tile));
    impl->prm.n_entries++;
    // Pairing: this member and the previous one of the launch each fit the lower / upper half of a tile's 128
    // rows, run the same stored layer, and one's slice contains the other's (filters and channels): they
    // share the larger one's tiles and weight copies.
    auto half = [](const GroupEntry &g) { return !g.swap && g.mtiles == 1 && g.pix_rows <= 64 && g.kw == g.k; };
    GroupEntry *prev = impl->prm.n_entries >= 2 ? static_cast<GroupEntry *>(host_entry) - 1 : nullptr;
    if (prev && !a.win && half(e) && half(*prev) && !prev->pair && !prev->second && prev->layer == e.layer && prev->k == e.k &&
        prev->stride == e.stride && prev->act == e.act && ((prev->K >= e.K && prev->C >= e.C) || (e.K >= prev->K && e.C >= prev->C))) {
        GroupEntry first = *prev, second = e;
        if (!(prev->K >= e.K && prev->C >= e.C)) { first = e; second = *prev; }
        first.tile_begin = second.tile_begin = prev->tile_begin;
        first.pair = 1; first.second = 0;
        second.pair = 0; second.second = 1;
        const int ntiles = (first.K + first.bn_tile - 1) / first.bn_tile;
        impl->prm.total_tiles = first.tile_begin + ntiles;
        *prev = first;
        std::memcpy(host_entry, &second, sizeof second);
        return;
    }
    std::memcpy(host_entry, &e, sizeof e);
    impl->prm.total_tiles += e.mtiles * (int)pl.grid.y;
}

static int g_group_stages = 0;  // 0 = default
void tc_group_set_stage_group(int stages) { g_group_stages = stages; }

cudaError_t tc_group_init(int) {
    cudaError_t e = cudaFuncSetAttribute(conv_group_kernel<TC_GROUP_MAPS_SMALL>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(conv_group_kernel<TC_GROUP_MAPS_LARGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM_BYTES);
}

cudaError_t GroupLaunch::launch(size_t window_max, int sms, cudaStream_t st) {
    if (impl->prm.n_entries <= 0 || impl->prm.total_tiles <= 0) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    impl->prm.status = tc_status_word(dev);
    if (!impl->prm.status) return cudaErrorInitializationError;
    impl->prm.unused_ = nullptr;
    // stage = 16 KB for the row-side operand + room for the widest column-side operand of the launch
    const int col_rows = impl->col_rows <= 64 ? 64 : impl->col_rows <= 128 ? 128 : 256;
    impl->prm.stage_bytes = G_X_BYTES + col_rows * CHUNK_C * 2;
    impl->prm.n_stages = G_RING_BYTES / impl->prm.stage_bytes;  // 8, 6 or 4
    const int want = g_group_stages > 0 ? g_group_stages : 1;  // (measured on batch-16 members: 2 or 4 stages per barrier pair change nothing for narrow tiles and cost 10-25 % on 256-column tiles)
    impl->prm.group = (want <= impl->prm.n_stages / 2 && impl->prm.n_stages % want == 0) ? want : 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)std::min(impl->prm.total_tiles, std::max(1, sms)));
    cfg.blockDim = dim3(G_THREADS);
    cfg.dynamicSmemBytes = G_SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (window_max && impl->win_base && impl->win_bytes) {
        // Access-policy window of this launch: L2 lines of the cached filter prefix that the launch touches are
        // kept with the persisting property (they live in the L2 carve-out the handle sized to the cache budget),
        // everything else is accessed normally.
        attr[1].id = cudaLaunchAttributeAccessPolicyWindow;
        attr[1].val.accessPolicyWindow.base_ptr = const_cast<void *>(impl->win_base);
        attr[1].val.accessPolicyWindow.num_bytes = std::min(impl->win_bytes, window_max);
        attr[1].val.accessPolicyWindow.hitRatio = 1.0f;
        attr[1].val.accessPolicyWindow.hitProp = cudaAccessPropertyPersisting;
        attr[1].val.accessPolicyWindow.missProp = cudaAccessPropertyNormal;
        cfg.numAttrs = 2;
    }
    if (impl->n_maps <= TC_GROUP_MAPS_SMALL) {
        // the small parameter block is a prefix of the large one (same header, fewer maps)
        void *args[1] = {&impl->prm};
        return cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(conv_group_kernel<TC_GROUP_MAPS_SMALL>), args);
    }
    void *args[1] = {&impl->prm};
    return cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(conv_group_kernel<TC_GROUP_MAPS_LARGE>), args);
}

}  // namespace sgs
