// Grouped sliced convolution: ONE launch runs the same stored layer for many queries in flight, each
// with its own SubNet slice (paper Section 2.1: every query selects its own filters / channels of the
// shared layer; Section 3.1: a stream of such queries).  A launch gets a table with one entry per
// member (query): its tensor maps, slice extents, tile geometry and buffers.  All members' output tiles
// form one list of tiles; persistent CTAs (two per SM) walk that list with a fixed stride.
//
// Per CTA: warp 0 = TMA producer, warp 1 = MMA issuer, warps 2..5 = epilogue.  The shared-memory ring
// of operand stages runs on across tiles, and the fp32 accumulator in tensor memory is double
// buffered (2 x 128 columns), so the epilogue of tile j (tensor memory -> folded batch norm ->
// residual -> activation -> bf16 NHWC) overlaps the loads and MMAs of tile j + 1.
//
// The arithmetic of one tile is that of conv_tc_kernel (sgs_conv_tc.cu): implicit GEMM with
// 128 output pixels x up to 128 filters, 64 channels per stage, slicing through the tensor maps'
// extents.  The reduction is never split here: with many members in flight the tiles alone fill the GPU.
#include "sgs_tc.cuh"

#include <algorithm>
#include <cstring>

namespace sgs {

namespace {

constexpr int G_BN = 128;
constexpr int G_STAGES = 3;
constexpr int G_STAGE_BYTES = A_STAGE_BYTES + G_BN * CHUNK_C * 2;
constexpr int G_SMEM_BYTES = G_STAGES * G_STAGE_BYTES + 1024;

struct __align__(16) GroupEntry {
    int map_a, map_w;        // indices into the launch's tensor maps: activation view(s) (4 for stride-2 kernels
                             // larger than 1x1: the parity views; else 1) and the sliced weight view
    const float *scale, *shift;
    const __nv_bfloat16 *res;
    __nv_bfloat16 *y;
    int tile_begin;          // index of this member's first tile in the launch's tile list
    int mtiles, ntiles;      // pixel tiles and filter tiles of this member
    int N, Ho, Wo, K, C;
    int k, stride, R, o, p;
    int bw, bh, bn, tiles_w, tiles_h;
    int cchunks, iters, act, layer;
};
static_assert(sizeof(GroupEntry) == TC_GROUP_ENTRY_BYTES, "entry size");

// Index of the entry that owns tile t (entries are sorted by tile_begin); the whole warp calls it.
__device__ __forceinline__ int find_entry(const GroupEntry *es, int n, int t, int lane) {
    const unsigned b0 = __ballot_sync(0xffffffffu, lane < n && es[lane].tile_begin <= t);
    const unsigned b1 = __ballot_sync(0xffffffffu, lane + 32 < n && es[lane + 32].tile_begin <= t);
    return __popc(b0) + __popc(b1) - 1;
}

__device__ __forceinline__ void epilogue_bar() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Kernel parameters.  The tensor maps travel in the parameter block (the TMA unit reads them from
// there); the per-member records travel in a device table.
template <int NMAPS> struct GroupParams {
    const GroupEntry *entries;
    const int *cache_tbl;
    int *status;
    int n_entries, total_tiles;
    int pad_[8];
    CUtensorMap maps[NMAPS];
};
static_assert(sizeof(GroupParams<TC_GROUP_MAPS_LARGE>) <= 32764, "kernel parameter block");

template <int NMAPS>
__global__ void __launch_bounds__(192, 1) conv_group_kernel(const __grid_constant__ GroupParams<NMAPS> P) {
    const GroupEntry *__restrict__ entries = P.entries;
    const int n_entries = P.n_entries, total_tiles = P.total_tiles;
    const int *__restrict__ cache_tbl = P.cache_tbl;
    int *status = P.status;
    extern __shared__ uint8_t smem_raw[];
    __shared__ GroupEntry es[TC_GROUP_MAX_ENTRIES];
    __shared__ int row_m[TILE_M];  // output pixel index of each tile row, -1 outside the tensor
    __shared__ float scale_s[G_BN], shift_s[G_BN];
    __shared__ __align__(8) uint64_t full_bar[G_STAGES], empty_bar[G_STAGES], acc_full[2], acc_empty[2];
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
        for (int s = 0; s < G_STAGES; s++) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
        for (int b = 0; b < 2; b++) { mbar_init(&acc_full[b], 1); mbar_init(&acc_empty[b], 4); }
        abort_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) tmem_alloc(&tmem_base_s, 2 * G_BN);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    pdl_launch_dependents();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        const uint64_t pol_keep = make_policy(1), pol_stream = make_policy(2);
        const int weight_policy = cache_tbl ? __ldg(cache_tbl) : 0;
        uint32_t it = 0;
        bool first = true;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
            const GroupEntry &e = es[find_entry(es, n_entries, t, lane)];
            const int local = t - e.tile_begin, nt = local / e.mtiles, mt = local % e.mtiles;
            const int tiles_hw = e.tiles_w * e.tiles_h;
            const int n0 = (mt / tiles_hw) * e.bn, h0 = ((mt % tiles_hw) / e.tiles_w) * e.bh, w0 = (mt % e.tiles_w) * e.bw;
            const int f0 = nt * G_BN;
            const uint32_t tx = (uint32_t)(e.bw * e.bh * e.bn * CHUNK_C * 2 + G_BN * CHUNK_C * 2);
            const CUtensorMap *map_a = &P.maps[e.map_a], *map_w = &P.maps[e.map_w];
            const int k = e.k, cchunks = e.cchunks, iters = e.iters, R = e.R, o = e.o, pad = e.p, stride = e.stride;
            int cacheK = 0, cacheC = 0;
            if (weight_policy == 1) { cacheK = __ldg(cache_tbl + 1 + 2 * e.layer); cacheC = __ldg(cache_tbl + 2 + 2 * e.layer); }
            auto load_weights = [&](int s, int c0, int tapw) {
                uint8_t *sb = smem + s * G_STAGE_BYTES + A_STAGE_BYTES;
                mbar_expect_tx(&full_bar[s], tx);
                // weight tiles inside the cached SubGraph's box are kept in L2 (evict-last); policy 2
                // marks every weight load evict-first (the "no reuse" reference point)
                if (weight_policy == 2) tma_load_3d_hint(sb, map_w, &full_bar[s], c0, tapw, f0, pol_stream);
                else if (weight_policy == 1 && f0 < cacheK && c0 < cacheC) tma_load_3d_hint(sb, map_w, &full_bar[s], c0, tapw, f0, pol_keep);
                else tma_load_3d(sb, map_w, &full_bar[s], c0, tapw, f0);
            };
            int pre = 0;
            if (first) {
                // Weights do not depend on the previous layer: the first stages' weight halves are
                // requested before waiting for it.
                first = false;
                pre = min(iters, G_STAGES);
                int cc2 = 0, r2 = 0, sx2 = 0;
                for (int i = 0; i < pre; i++) {
                    if (elect_one()) load_weights(i, cc2 * CHUNK_C, (o + r2) * R + (o + sx2));
                    __syncwarp();
                    if (++cc2 == cchunks) { cc2 = 0; if (++sx2 == k) { sx2 = 0; ++r2; } }
                }
                pdl_wait();
            }
            int cc = 0, r = 0, sx = 0;
            bool ok = true;
            for (int i = 0; i < iters; i++, it++) {
                const int s = it % G_STAGES;
                const uint32_t round = it / G_STAGES;
                ok = round == 0 || mbar_wait(&empty_bar[s], (round - 1) & 1, abort_flag);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const int c0 = cc * CHUNK_C;
                uint8_t *sa = smem + s * G_STAGE_BYTES;
                const int dh = r - pad, dw = sx - pad;
                if (elect_one()) {
                    if (i >= pre) load_weights(s, c0, (o + r) * R + (o + sx));
                    if (stride == 1) {
                        tma_load_4d(sa, map_a, &full_bar[s], c0, w0 + dw, h0 + dh, n0);
                    } else {
                        const int ph = dh & 1, pw = dw & 1;
                        tma_load_4d(sa, map_a + ph * 2 + pw, &full_bar[s], c0, w0 + ((dw - pw) >> 1), h0 + ((dh - ph) >> 1), n0);
                    }
                }
                __syncwarp();
                if (++cc == cchunks) { cc = 0; if (++sx == k) { sx = 0; ++r; } }
            }
            if (!ok) break;
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        uint32_t it = 0;
        int j = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, j++) {
            const GroupEntry &e = es[find_entry(es, n_entries, t, lane)];
            const int nt = (t - e.tile_begin) / e.mtiles;
            const int f0 = nt * G_BN;
            const int n_mma = min(G_BN, (e.K - f0 + 15) & ~15);
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(TILE_M >> 4) << 24);
            const int buf = j & 1;
            const int C = e.C, cchunks = e.cchunks, iters = e.iters;
            bool ok = j < 2 || mbar_wait(&acc_empty[buf], ((j >> 1) - 1) & 1, abort_flag);  // epilogue drained this buffer
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem_base + (uint32_t)(buf * G_BN);
            int cc = 0;
            for (int i = 0; i < iters; i++, it++) {
                const int s = it % G_STAGES;
                const uint32_t round = it / G_STAGES;
                ok = __all_sync(0xffffffffu, mbar_wait(&full_bar[s], round & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                const int ksteps = (min(CHUNK_C, C - cc * CHUNK_C) + 15) / 16;
                const uint32_t sa = smem_u32(smem + s * G_STAGE_BYTES), sb = sa + A_STAGE_BYTES;
                const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
                if (elect_one()) {
                    for (int q = 0; q < ksteps; q++)
                        umma_bf16(d_tmem, da + (uint64_t)(2 * q), db + (uint64_t)(2 * q), idesc, (i > 0 || q > 0) ? 1u : 0u);
                    umma_commit(&empty_bar[s]);
                    if (i == iters - 1) umma_commit(&acc_full[buf]);
                }
                __syncwarp();
                if (++cc == cchunks) cc = 0;
            }
            if (!ok) break;
        }
    } else {
        // ------------------------------------------------------------------ epilogue (warps 2..5)
        const int quad = warp & 3;         // TMEM lane quadrant this warp may read
        const int row = quad * 32 + lane;  // tile row = output pixel within the box
        const int et = threadIdx.x - 64;   // 0..127
        pdl_wait();  // residual reads and output writes must not pass the previous layers
        bool alive = true;  // after a failed wait the warp only keeps the named barriers in step
        int j = 0;
        for (int t = blockIdx.x; t < total_tiles; t += gridDim.x, j++) {
            const GroupEntry &e = es[find_entry(es, n_entries, t, lane)];
            const int local = t - e.tile_begin, nt = local / e.mtiles, mt = local % e.mtiles;
            const int tiles_hw = e.tiles_w * e.tiles_h;
            const int n0 = (mt / tiles_hw) * e.bn, h0 = ((mt % tiles_hw) / e.tiles_w) * e.bh, w0 = (mt % e.tiles_w) * e.bw;
            const int f0 = nt * G_BN;
            const int K = e.K, act = e.act;
            const __nv_bfloat16 *res = e.res;
            __nv_bfloat16 *y = e.y;
            epilogue_bar();  // every epilogue thread is done with the previous tile's tables
            {
                const int rows = e.bw * e.bh * e.bn;
                const int dn = row / (e.bh * e.bw), dhh = (row / e.bw) % e.bh, dww = row % e.bw;
                const int n = n0 + dn, h = h0 + dhh, w = w0 + dww;
                const bool valid = row < rows && n < e.N && h < e.Ho && w < e.Wo;
                row_m[row] = valid ? (int)(((size_t)n * e.Ho + h) * e.Wo + w) : -1;
                const int f = f0 + et;
                scale_s[et] = f < K ? __ldg(e.scale + f) : 0.f;
                shift_s[et] = f < K ? __ldg(e.shift + f) : 0.f;
            }
            epilogue_bar();
            const int buf = j & 1;
            if (alive) {
                bool ok = mbar_wait(&acc_full[buf], (j >> 1) & 1, abort_flag);
                alive = __all_sync(0xffffffffu, ok);
            }
            if (!alive) continue;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * G_BN);
            const int ncols = min(G_BN, K - f0);  // filters of this tile, a multiple of 8
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
                            float ov[8];
#pragma unroll
                            for (int q = 0; q < 8; q++) ov[q] = __uint_as_float(v[8 * g + q]) * scale_s[c + q] + shift_s[c + q];
                            finish_store(ov, res, y, (size_t)m * K + f0 + c, act);
                        }
                    }
                }
            }
            // hand the accumulator buffer back to the MMA warp
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
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
    if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, 2 * G_BN); }
}

}  // namespace

// Number of activation views a member needs: the four parity views only when a stride-2 kernel
// reaches odd offsets, i.e. for kernels larger than 1x1.
static int views_of(const TcParams &p) { return (p.stride == 2 && p.k > 1) ? 4 : 1; }

struct GroupLaunch::Impl {
    GroupParams<TC_GROUP_MAPS_LARGE> prm;  // host image of the parameter block (the small variant is a prefix)
    int n_maps = 0;
};

GroupLaunch::GroupLaunch() : impl(new Impl) { reset(nullptr); }
GroupLaunch::~GroupLaunch() { delete impl; }

void GroupLaunch::reset(const void *d_entries) {
    impl->n_maps = 0;
    impl->prm.entries = static_cast<const GroupEntry *>(d_entries);
    impl->prm.n_entries = 0;
    impl->prm.total_tiles = 0;
}
int GroupLaunch::members() const { return impl->prm.n_entries; }
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
    e.ntiles = (a.K + G_BN - 1) / G_BN;
    e.N = p.N; e.Ho = p.Ho; e.Wo = p.Wo; e.K = p.K; e.C = p.C;
    e.k = p.k; e.stride = p.stride; e.R = p.R; e.o = p.o; e.p = p.p;
    e.bw = p.bw; e.bh = p.bh; e.bn = p.bn; e.tiles_w = p.tiles_w; e.tiles_h = p.tiles_h;
    e.cchunks = p.cchunks; e.iters = p.iters; e.act = p.act; e.layer = a.layer;
    std::memcpy(host_entry, &e, sizeof e);
    impl->prm.n_entries++;
    impl->prm.total_tiles += e.mtiles * e.ntiles;
}

cudaError_t tc_group_init(int) {
    cudaError_t e = cudaFuncSetAttribute(conv_group_kernel<TC_GROUP_MAPS_SMALL>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM_BYTES);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(conv_group_kernel<TC_GROUP_MAPS_LARGE>, cudaFuncAttributeMaxDynamicSharedMemorySize, G_SMEM_BYTES);
}

cudaError_t GroupLaunch::launch(const int *cache_tbl, int sms, cudaStream_t st) {
    if (impl->prm.n_entries <= 0 || impl->prm.total_tiles <= 0) return cudaSuccess;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    impl->prm.status = tc_status_word(dev);
    if (!impl->prm.status) return cudaErrorInitializationError;
    impl->prm.cache_tbl = cache_tbl;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)std::min(impl->prm.total_tiles, 2 * std::max(1, sms)));
    cfg.blockDim = dim3(192);
    cfg.dynamicSmemBytes = G_SMEM_BYTES;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (impl->n_maps <= TC_GROUP_MAPS_SMALL) {
        // the small parameter block is a prefix of the large one (same header, fewer maps)
        void *args[1] = {&impl->prm};
        return cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(conv_group_kernel<TC_GROUP_MAPS_SMALL>), args);
    }
    void *args[1] = {&impl->prm};
    return cudaLaunchKernelExC(&cfg, reinterpret_cast<const void *>(conv_group_kernel<TC_GROUP_MAPS_LARGE>), args);
}

}  // namespace sgs
