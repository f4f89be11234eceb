// Plain CUDA-core kernels: sliced convolution (shared-memory implicit GEMM in fp32), depthwise
// convolution with centre-cropped kernels, pooling, squeeze-excite, linear layers, and the
// load-time re-layout / batch-norm folding kernels.
//
// These are the complete path in fp32 mode and, in bf16 mode, serve the layers the tensor-core
// kernel does not take (3-channel stems, channel counts that are not multiples of 8).
#include "sgs_internal.h"

#include <algorithm>
#include <cooperative_groups.h>

namespace sgs {

template <typename T> __device__ __forceinline__ float to_f(T v);
template <> __device__ __forceinline__ float to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f(float v);
template <> __device__ __forceinline__ float from_f<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float apply_act(float v, int act) {
    if (act == ACT_RELU) return fmaxf(v, 0.f);
    if (act == ACT_HSWISH) return v * fminf(fmaxf(v + 3.f, 0.f), 6.f) * (1.f / 6.f);
    return v;
}

// ---------------------------------------------------------------------------------------------
// Sliced convolution as an implicit GEMM on CUDA cores.
//   D[m][f] = sum_kk A[m][kk] * B[f][kk],  m = output pixel, f < K', kk = (r*k + s)*C' + c
//   A[m][kk] = x[n][ho*st + r - p][wo*st + s - p][c]   (zero outside the image)
//   B[f][kk] = w[f][o + r][o + s][c]                   (stored [Kmax][R][R][Cmax], o = (R-k)/2)
// 64 x 64 output tile per block, 16-wide k chunks, 4 x 4 outputs per thread.
// ---------------------------------------------------------------------------------------------
constexpr int PT_M = 64, PT_N = 64, PT_K = 16;

template <typename T>
__global__ void __launch_bounds__(256) conv_plain_kernel(ConvArgs a) {
    __shared__ float As[PT_K][PT_M + 4];
    __shared__ float Bs[PT_K][PT_N + 4];
    const T *__restrict__ x = static_cast<const T *>(a.x);
    const T *__restrict__ w = static_cast<const T *>(a.w);
    const int M = a.N * a.Ho * a.Wo;
    const int KK = a.k * a.k * a.C;
    const int p = (a.k - 1) / 2, o = (a.R - a.k) / 2;
    const int m0 = blockIdx.x * PT_M, f0 = blockIdx.y * PT_N;
    const int t = threadIdx.x;
    const int lk = t % PT_K, lrow = t / PT_K;  // loader coordinates
    const int tx = t % 16, ty = t / 16;        // compute coordinates

    // decode the four pixels this thread loads
    int pn[4], ph[4], pw[4];
    bool pv[4];
#pragma unroll
    for (int j = 0; j < 4; j++) {
        int m = m0 + lrow + 16 * j;
        pv[j] = m < M;
        int mm = pv[j] ? m : 0;
        pw[j] = mm % a.Wo;
        ph[j] = (mm / a.Wo) % a.Ho;
        pn[j] = mm / (a.Wo * a.Ho);
    }
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; i++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[i][j] = 0.f;

    for (int kk0 = 0; kk0 < KK; kk0 += PT_K) {
        const int kk = kk0 + lk;
        const bool kv = kk < KK;
        int c = 0, r = 0, s = 0;
        if (kv) {
            c = kk % a.C;
            int rs = kk / a.C;
            s = rs % a.k;
            r = rs / a.k;
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            float v = 0.f;
            if (kv && pv[j]) {
                int hi = ph[j] * a.stride + r - p, wi = pw[j] * a.stride + s - p;
                if (hi >= 0 && hi < a.H && wi >= 0 && wi < a.W)
                    v = to_f<T>(x[(((size_t)pn[j] * a.H + hi) * a.W + wi) * a.C + c]);
            }
            As[lk][lrow + 16 * j] = v;
        }
#pragma unroll
        for (int j = 0; j < 4; j++) {
            int f = f0 + lrow + 16 * j;
            float v = 0.f;
            if (kv && f < a.K) v = to_f<T>(w[(((size_t)f * a.R + (o + r)) * a.R + (o + s)) * a.Cmax + c]);
            Bs[lk][lrow + 16 * j] = v;
        }
        __syncthreads();
#pragma unroll
        for (int q = 0; q < PT_K; q++) {
            float av[4], bv[4];
#pragma unroll
            for (int i = 0; i < 4; i++) av[i] = As[q][ty * 4 + i];
#pragma unroll
            for (int j = 0; j < 4; j++) bv[j] = Bs[q][tx * 4 + j];
#pragma unroll
            for (int i = 0; i < 4; i++)
#pragma unroll
                for (int j = 0; j < 4; j++) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    const T *__restrict__ res = static_cast<const T *>(a.res);
    T *__restrict__ y = static_cast<T *>(a.y);
#pragma unroll
    for (int i = 0; i < 4; i++) {
        int m = m0 + ty * 4 + i;
        if (m >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; j++) {
            int f = f0 + tx * 4 + j;
            if (f >= a.K) continue;
            float v = acc[i][j] * a.scale[f] + a.shift[f];
            size_t oi = (size_t)m * a.K + f;
            if (res) v += to_f<T>(res[oi]);
            y[oi] = from_f<T>(apply_act(v, a.act));
        }
    }
}

template <typename T> cudaError_t launch_conv_plain(const ConvArgs &a, cudaStream_t st) {
    int M = a.N * a.Ho * a.Wo;
    if (M <= 0 || a.K <= 0) return cudaSuccess;
    dim3 grid((M + PT_M - 1) / PT_M, (a.K + PT_N - 1) / PT_N);
    conv_plain_kernel<T><<<grid, 256, 0, st>>>(a);
    return cudaGetLastError();
}
template cudaError_t launch_conv_plain<float>(const ConvArgs &, cudaStream_t);
template cudaError_t launch_conv_plain<__nv_bfloat16>(const ConvArgs &, cudaStream_t);

// ---------------------------------------------------------------------------------------------
// Depthwise k x k convolution, kernel = centre window of the stored R x R kernel, weights
// [R][R][Kmax].  One thread per (pixel, channel), channels fastest (coalesced NHWC).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) dw_plain_kernel(ConvArgs a) {
    const T *__restrict__ x = static_cast<const T *>(a.x);
    const T *__restrict__ w = static_cast<const T *>(a.w);
    T *__restrict__ y = static_cast<T *>(a.y);
    const size_t total = (size_t)a.N * a.Ho * a.Wo * a.K;
    const int p = (a.k - 1) / 2, o = (a.R - a.k) / 2;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int c = (int)(i % a.K);
        size_t m = i / a.K;
        int wo = (int)(m % a.Wo), ho = (int)((m / a.Wo) % a.Ho), n = (int)(m / ((size_t)a.Wo * a.Ho));
        float acc = 0.f;
        for (int r = 0; r < a.k; r++) {
            int hi = ho * a.stride + r - p;
            if (hi < 0 || hi >= a.H) continue;
            for (int s = 0; s < a.k; s++) {
                int wi = wo * a.stride + s - p;
                if (wi < 0 || wi >= a.W) continue;
                acc = fmaf(to_f<T>(x[(((size_t)n * a.H + hi) * a.W + wi) * a.K + c]),
                           to_f<T>(w[((size_t)(o + r) * a.R + (o + s)) * a.Kmax + c]), acc);
            }
        }
        float v = acc * a.scale[c] + a.shift[c];
        y[i] = from_f<T>(apply_act(v, a.act));
    }
}

// Vectorised bf16 depthwise convolution.  A thread owns 8 channels (one 16-byte vector) of TW = 4
// neighbouring output pixels of one output row: per filter row it loads the (TW-1)*ST + K input
// columns once and uses each for every tap it belongs to, so global loads per output drop from K*K
// to about K*(1 + (K-1)/(TW*ST)); neighbouring threads cover neighbouring channel vectors, so every
// load and store of a warp is one contiguous run.  fp32 accumulation with packed 2-wide FMAs.
// HBM traffic per output element: 2 B read + 2 B written (rows are re-read from L1/L2, not DRAM).
__device__ __forceinline__ float2 bf2_lo(uint32_t u) { return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u)); }

// Argument record of a depthwise kernel: by value, or (GROUP: one launch for many queries in flight) from a
// device table with DW_ENTRY_BYTES per member, blockIdx.z = member * images + image.
#define SGS_DW_ARGS()                                                                                          \
    __shared__ __align__(16) unsigned char a_raw_[sizeof(ConvArgs)];                                           \
    if (GROUP) {                                                                                               \
        const uint32_t *src_ = reinterpret_cast<const uint32_t *>(tbl + (size_t)(blockIdx.z / n_img) * DW_ENTRY_BYTES); \
        for (int i_ = threadIdx.x; i_ < (int)(sizeof(ConvArgs) / 4); i_ += blockDim.x) reinterpret_cast<uint32_t *>(a_raw_)[i_] = __ldg(src_ + i_); \
        __syncthreads();                                                                                       \
    }                                                                                                          \
    const ConvArgs &a = GROUP ? *reinterpret_cast<const ConvArgs *>(a_raw_) : a1;                              \
    const int n = GROUP ? (int)(blockIdx.z % n_img) : (int)blockIdx.z;
static_assert(sizeof(ConvArgs) % 4 == 0 && sizeof(ConvArgs) <= DW_ENTRY_BYTES, "depthwise table record");

template <int K, int ST>
__device__ __forceinline__ void dw_vec_body(const ConvArgs &a, const int n) {
    constexpr int TW = 4, NCOL = (TW - 1) * ST + K, P = (K - 1) / 2;
    // grid: x covers (channel vector, pixel block) of one output row, y = output row, z = image;
    // all index arithmetic stays in 32 bits
    const int groups = a.K / 8, wblocks = (a.Wo + TW - 1) / TW;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= groups * wblocks) return;
    const int cg = idx % groups, wb = idx / groups;
    const int ho = blockIdx.y;
    const int c0 = cg * 8, wo0 = wb * TW, o = (a.R - K) / 2;
    const __nv_bfloat16 *__restrict__ x = static_cast<const __nv_bfloat16 *>(a.x);
    const __nv_bfloat16 *__restrict__ w = static_cast<const __nv_bfloat16 *>(a.w);

    float2 acc[TW][4];
#pragma unroll
    for (int t = 0; t < TW; t++)
#pragma unroll
        for (int j = 0; j < 4; j++) acc[t][j] = make_float2(0.f, 0.f);

    const __nv_bfloat16 *ximg = x + ((size_t)n * a.H) * a.W * a.K + c0;
#pragma unroll
    for (int r = 0; r < K; r++) {
        const int hi = ho * ST + r - P;
        if (hi < 0 || hi >= a.H) continue;
        const __nv_bfloat16 *xrow = ximg + (size_t)hi * a.W * a.K;
        uint4 col[NCOL];
#pragma unroll
        for (int j = 0; j < NCOL; j++) {
            const int wi = wo0 * ST + j - P;
            col[j] = (wi >= 0 && wi < a.W) ? __ldg(reinterpret_cast<const uint4 *>(xrow + wi * a.K)) : make_uint4(0u, 0u, 0u, 0u);
        }
        const __nv_bfloat16 *wrow = w + ((o + r) * a.R + o) * a.Kmax + c0;
#pragma unroll
        for (int s = 0; s < K; s++) {
            const uint4 wv = __ldg(reinterpret_cast<const uint4 *>(wrow + s * a.Kmax));
            const float2 w0 = bf2_lo(wv.x), w1 = bf2_lo(wv.y), w2 = bf2_lo(wv.z), w3 = bf2_lo(wv.w);
#pragma unroll
            for (int t = 0; t < TW; t++) {
                const uint4 xv = col[t * ST + s];
                acc[t][0] = __ffma2_rn(bf2_lo(xv.x), w0, acc[t][0]);
                acc[t][1] = __ffma2_rn(bf2_lo(xv.y), w1, acc[t][1]);
                acc[t][2] = __ffma2_rn(bf2_lo(xv.z), w2, acc[t][2]);
                acc[t][3] = __ffma2_rn(bf2_lo(xv.w), w3, acc[t][3]);
            }
        }
    }
    const float4 s0 = __ldg(reinterpret_cast<const float4 *>(a.scale + c0)), s1 = __ldg(reinterpret_cast<const float4 *>(a.scale + c0 + 4));
    const float4 h0 = __ldg(reinterpret_cast<const float4 *>(a.shift + c0)), h1 = __ldg(reinterpret_cast<const float4 *>(a.shift + c0 + 4));
    __nv_bfloat16 *yrow = static_cast<__nv_bfloat16 *>(a.y) + (((size_t)n * a.Ho + ho) * a.Wo) * a.K + c0;
#pragma unroll
    for (int t = 0; t < TW; t++) {
        const int wo = wo0 + t;
        if (wo >= a.Wo) break;
        float v[8] = {acc[t][0].x * s0.x + h0.x, acc[t][0].y * s0.y + h0.y, acc[t][1].x * s0.z + h0.z, acc[t][1].y * s0.w + h0.w,
                      acc[t][2].x * s1.x + h1.x, acc[t][2].y * s1.y + h1.y, acc[t][3].x * s1.z + h1.z, acc[t][3].y * s1.w + h1.w};
        uint4 ov;
        __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
        for (int j = 0; j < 4; j++) ob[j] = __floats2bfloat162_rn(apply_act(v[2 * j], a.act), apply_act(v[2 * j + 1], a.act));
        *reinterpret_cast<uint4 *>(yrow + wo * a.K) = ov;
    }
}
template <int K, int ST, bool GROUP>
__global__ void __launch_bounds__(256) dw_vec_kernel(const ConvArgs a1, const char *__restrict__ tbl, int n_img) {
    SGS_DW_ARGS()
    dw_vec_body<K, ST>(a, n);
}

// Tiled variant: a thread owns 8 channels of a TH x TW patch of output pixels.  Every vector of the
// patch's halo is loaded and unpacked ONCE and used for all the output rows and taps it belongs to, so
// the instruction count per output element (the limit of the row-at-a-time kernel above) drops to about
// ((TH-1)*ST+K)*((TW-1)*ST+K)/(TH*TW) unpacks + K*K packed FMAs per 8 channels.  With PRELOAD every load
// of the halo is issued before the first use (memory latency is then hidden by the loads a thread has
// in flight, not by occupancy).  Patches whose halo lies inside the image take a path without bounds
// tests.  The epilogue is packed: one FMA for the folded batch norm per channel pair, and h-swish as
// x * clamp(x / 6 + 0.5, 0, 1) (= x * relu6(x + 3) / 6): one saturating FMA and one packed multiply.
template <int K, int ST, int TH, int TW, bool PRELOAD, int ACT>
__device__ __forceinline__ void dw_tile_body(const ConvArgs &a, const int n) {
    constexpr int P = (K - 1) / 2, NCOL = (TW - 1) * ST + K, NROW = (TH - 1) * ST + K;
    const int groups = a.K / 8, wblocks = (a.Wo + TW - 1) / TW;
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= groups * wblocks || (int)blockIdx.y * TH >= a.Ho) return;
    const int cg = idx % groups, wb = idx / groups;
    const int ho0 = blockIdx.y * TH;
    const int c0 = cg * 8, wo0 = wb * TW, o = (a.R - K) / 2;
    const __nv_bfloat16 *__restrict__ x = static_cast<const __nv_bfloat16 *>(a.x);
    const __nv_bfloat16 *__restrict__ w = static_cast<const __nv_bfloat16 *>(a.w);

    // weights stay packed in registers and are unpacked at use
    constexpr bool WUNPACK = false;  // (unpacking the weights once costs 72 registers for K = 3 and measured slower)
    uint4 wv[WUNPACK ? 1 : K * K];
    float2 wf[WUNPACK ? K * K : 1][4];
#pragma unroll
    for (int r = 0; r < K; r++)
#pragma unroll
        for (int s = 0; s < K; s++) {
            const uint4 q = __ldg(reinterpret_cast<const uint4 *>(w + ((o + r) * a.R + o + s) * a.Kmax + c0));
            if (WUNPACK) {
                float2 *d = wf[WUNPACK ? r * K + s : 0];
                d[0] = bf2_lo(q.x); d[1] = bf2_lo(q.y); d[2] = bf2_lo(q.z); d[3] = bf2_lo(q.w);
            } else {
                wv[WUNPACK ? 0 : r * K + s] = q;
            }
        }

    float2 acc[TH][TW][4];
#pragma unroll
    for (int i = 0; i < TH; i++)
#pragma unroll
        for (int t = 0; t < TW; t++)
#pragma unroll
            for (int j = 0; j < 4; j++) acc[i][t][j] = make_float2(0.f, 0.f);

    const __nv_bfloat16 *ximg = x + ((size_t)n * a.H) * a.W * a.K + c0;
    const int wi0 = wo0 * ST - P, hi0 = ho0 * ST - P;
    const bool interior = hi0 >= 0 && hi0 + NROW <= a.H && wi0 >= 0 && wi0 + NCOL <= a.W;
    uint4 raw[PRELOAD ? NROW : 1][NCOL];
    if (PRELOAD) {
#pragma unroll
        for (int ir = 0; ir < NROW; ir++) {
            const int hi = hi0 + ir;
            const bool rok = hi >= 0 && hi < a.H;
            const __nv_bfloat16 *xrow = ximg + (size_t)(rok ? hi : 0) * a.W * a.K;
#pragma unroll
            for (int j = 0; j < NCOL; j++) {
                const int wi = wi0 + j;
                raw[PRELOAD ? ir : 0][j] = (rok && wi >= 0 && wi < a.W) ? __ldg(reinterpret_cast<const uint4 *>(xrow + wi * a.K)) : make_uint4(0u, 0u, 0u, 0u);
            }
        }
    }
#pragma unroll
    for (int ir = 0; ir < NROW; ir++) {
        const int hi = hi0 + ir;
        if (!PRELOAD && (hi < 0 || hi >= a.H)) continue;
        const __nv_bfloat16 *xrow = ximg + (size_t)hi * a.W * a.K;
        float2 xc[NCOL][4];
#pragma unroll
        for (int j = 0; j < NCOL; j++) {
            const int wi = wi0 + j;
            uint4 v;
            if (PRELOAD) v = raw[PRELOAD ? ir : 0][j];
            else if (interior) v = __ldg(reinterpret_cast<const uint4 *>(xrow + wi * a.K));
            else v = (wi >= 0 && wi < a.W) ? __ldg(reinterpret_cast<const uint4 *>(xrow + wi * a.K)) : make_uint4(0u, 0u, 0u, 0u);
            xc[j][0] = bf2_lo(v.x); xc[j][1] = bf2_lo(v.y); xc[j][2] = bf2_lo(v.z); xc[j][3] = bf2_lo(v.w);
        }
#pragma unroll
        for (int oh = 0; oh < TH; oh++) {
            const int r = ir - oh * ST;  // filter row this input row meets in output row oh
            if (r < 0 || r >= K) continue;
#pragma unroll
            for (int s = 0; s < K; s++) {
                float2 w0, w1, w2, w3;
                if (WUNPACK) {
                    const float2 *d = wf[WUNPACK ? r * K + s : 0];
                    w0 = d[0]; w1 = d[1]; w2 = d[2]; w3 = d[3];
                } else {
                    const uint4 q = wv[WUNPACK ? 0 : r * K + s];
                    w0 = bf2_lo(q.x); w1 = bf2_lo(q.y); w2 = bf2_lo(q.z); w3 = bf2_lo(q.w);
                }
#pragma unroll
                for (int t = 0; t < TW; t++) {
                    acc[oh][t][0] = __ffma2_rn(xc[t * ST + s][0], w0, acc[oh][t][0]);
                    acc[oh][t][1] = __ffma2_rn(xc[t * ST + s][1], w1, acc[oh][t][1]);
                    acc[oh][t][2] = __ffma2_rn(xc[t * ST + s][2], w2, acc[oh][t][2]);
                    acc[oh][t][3] = __ffma2_rn(xc[t * ST + s][3], w3, acc[oh][t][3]);
                }
            }
        }
    }
    const float4 s0 = __ldg(reinterpret_cast<const float4 *>(a.scale + c0)), s1 = __ldg(reinterpret_cast<const float4 *>(a.scale + c0 + 4));
    const float4 h0 = __ldg(reinterpret_cast<const float4 *>(a.shift + c0)), h1 = __ldg(reinterpret_cast<const float4 *>(a.shift + c0 + 4));
    const float2 sc[4] = {make_float2(s0.x, s0.y), make_float2(s0.z, s0.w), make_float2(s1.x, s1.y), make_float2(s1.z, s1.w)};
    const float2 sh[4] = {make_float2(h0.x, h0.y), make_float2(h0.z, h0.w), make_float2(h1.x, h1.y), make_float2(h1.z, h1.w)};
#pragma unroll
    for (int oh = 0; oh < TH; oh++) {
        const int ho = ho0 + oh;
        if (ho >= a.Ho) break;
        __nv_bfloat16 *yrow = static_cast<__nv_bfloat16 *>(a.y) + (((size_t)n * a.Ho + ho) * a.Wo) * a.K + c0;
#pragma unroll
        for (int t = 0; t < TW; t++) {
            const int wo = wo0 + t;
            if (wo >= a.Wo) break;
            uint4 ov;
            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
            for (int j = 0; j < 4; j++) {
                float2 v = __ffma2_rn(acc[oh][t][j], sc[j], sh[j]);
                if (ACT == ACT_RELU) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); }
                if (ACT == ACT_HSWISH) {
                    const float2 g = make_float2(__saturatef(fmaf(v.x, 1.f / 6.f, 0.5f)), __saturatef(fmaf(v.y, 1.f / 6.f, 0.5f)));
                    v = __fmul2_rn(v, g);
                }
                ob[j] = __float22bfloat162_rn(v);
            }
            *reinterpret_cast<uint4 *>(yrow + wo * a.K) = ov;
        }
    }
}
template <int K, int ST, int TH, int TW, bool PRELOAD, int ACT, bool GROUP>
__global__ void __launch_bounds__(128) dw_tile_kernel(const ConvArgs a1, const char *__restrict__ tbl, int n_img) {
    SGS_DW_ARGS()
    if (GROUP) { const ConvArgs al = a; dw_tile_body<K, ST, TH, TW, PRELOAD, ACT>(al, n); }  // (register copy, see dw_mixed_kernel)
    else dw_tile_body<K, ST, TH, TW, PRELOAD, ACT>(a, n);
}
// Stride-1 depthwise convolution that WALKS down the image behind a ring of input rows in shared memory (the
// B200 form of a line buffer: paper Section 4.2 keeps the rows a sliding window needs on chip).  A block owns 128
// channels x a tile of 4 * TW output columns x a segment of SEG output rows.  Its 128 threads copy one input row of
// the tile at a time into a ring of RING rows with 16-byte asynchronous copies (zero fill for rows, columns and
// channels outside the tensor, so the arithmetic has no bounds tests), RING - 1 rows ahead of the row being used:
// memory latency is covered by the ring, not by registers or occupancy.  A thread owns 4 channels (an 8-byte vector)
// of a strip of TW columns: per input row it reads TW + K - 1 vectors from the ring, unpacks each ONCE, and
// scatters it into the K output rows it belongs to.  The K live output rows rotate through K accumulator slots; the
// row loop is unrolled by K so that every slot index is static: input row hi = base + u meets filter row r in output
// row hi + P - r, slot (u - r) mod K.  Filter row 0 STARTS an output row (a product instead of an accumulate: slots
// never need clearing, rows outside the segment never need a test), filter row K - 1 completes it.  The weights of
// the block's 128 channels sit unpacked (fp32) in shared memory; a lane reads its four per tap with one 16-byte load.
// Grid: x = channel blocks x column tiles, y = row segments, z = image (x member).
#ifndef DW_WALK_SEG_ROWS
#define DW_WALK_SEG_ROWS 56
#endif
constexpr int DW_WALK_SEG = DW_WALK_SEG_ROWS;  // output rows per segment (halo: K - 1 extra input rows per segment)
template <int K> struct DwWalkShape {
    static constexpr int TW = K == 3 ? 4 : 2;          // output columns per thread
    static constexpr int ICOL = 4 * TW + K - 1;        // input columns of a block's tile
    static constexpr int RING = K == 7 ? 6 : 8;        // input rows in the ring
    static constexpr int ROW_BYTES = ICOL * 256;       // 128 channels x 2 bytes per column
    static constexpr int SMEM = K * K * 128 * 4 + RING * ROW_BYTES;
};

__device__ __forceinline__ void cp_async16(void *dst, const void *src, bool valid) {
    const unsigned n = valid ? 16u : 0u;  // 0 source bytes: the 16 destination bytes are zero-filled
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((unsigned)__cvta_generic_to_shared(dst)), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int K, int ACT>
__device__ __forceinline__ void dw_walk_body(const ConvArgs &a, const int n, unsigned char *smem, const int chblocks) {
    using S = DwWalkShape<K>;
    constexpr int TW = S::TW, P = (K - 1) / 2, NCOL = TW + K - 1, ICOL = S::ICOL, RING = S::RING;
    float *wsm = reinterpret_cast<float *>(smem);
    unsigned char *ring = smem + K * K * 128 * 4;
    const int lane = threadIdx.x & 31, wrp = threadIdx.x >> 5;
    const int groups = a.K / 4, tiles_w = (a.Wo + 4 * TW - 1) / (4 * TW);
    // (chblocks = channel blocks of the GRID: a launch over several members is sized for the widest of them)
    const int cb = blockIdx.x % chblocks, tb = blockIdx.x / chblocks;
    const int ho_begin = blockIdx.y * DW_WALK_SEG, ho_end = min(a.Ho, ho_begin + DW_WALK_SEG);
    if (cb * 32 >= groups || tb >= tiles_w || ho_begin >= a.Ho) return;  // (whole blocks only: no barrier is skipped)
    const int o = (a.R - K) / 2;
    const __nv_bfloat16 *__restrict__ w = static_cast<const __nv_bfloat16 *>(a.w);
    // the block's weights: wsm[tap][lane * 4 + j] = w[o + r][o + s][cb * 128 + lane * 4 + j] (zero beyond the slice)
    for (int i = threadIdx.x; i < K * K * 32; i += blockDim.x) {
        const int tap = i >> 5, l = i & 31, c = cb * 128 + l * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c < a.K) {
            const uint2 q = __ldg(reinterpret_cast<const uint2 *>(w + ((size_t)((o + tap / K) * a.R + o + tap % K)) * a.Kmax + c));
            const float2 lo = bf2_lo(q.x), hi = bf2_lo(q.y);
            v = make_float4(lo.x, lo.y, hi.x, hi.y);
        }
        reinterpret_cast<float4 *>(wsm)[tap * 32 + l] = v;
    }
    const int cg = cb * 32 + lane;
    const int c0 = cg * 4, wt0 = tb * 4 * TW, wo0 = wt0 + wrp * TW;
    const bool active = cg < groups;  // (lanes beyond the slice compute zeros and store nothing)
    const __nv_bfloat16 *ximg = static_cast<const __nv_bfloat16 *>(a.x) + ((size_t)n * a.H) * a.W * a.K;
    __nv_bfloat16 *yimg = static_cast<__nv_bfloat16 *>(a.y) + ((size_t)n * a.Ho) * a.Wo * a.K + c0;
    float4 sc4 = make_float4(0.f, 0.f, 0.f, 0.f), sh4 = sc4;
    if (active) { sc4 = __ldg(reinterpret_cast<const float4 *>(a.scale + c0)); sh4 = __ldg(reinterpret_cast<const float4 *>(a.shift + c0)); }
    const float2 sc[2] = {make_float2(sc4.x, sc4.y), make_float2(sc4.z, sc4.w)}, sh[2] = {make_float2(sh4.x, sh4.y), make_float2(sh4.z, sh4.w)};
    const float4 *wl = reinterpret_cast<const float4 *>(wsm) + lane;

    const int hi_first = ho_begin - P, hi_last = ho_end - 1 + P;  // input rows that meet the segment (may lie outside the image)
    // One input row of the tile -> ring slot (hi - hi_first) % RING, 16 chunks of 16 bytes per column.  A thread
    // copies the same (column, channel) chunks of every row: their offsets and whether they lie inside the tensor
    // are fixed before the row loop.
    constexpr int NCH = (ICOL * 16 + 127) / 128;  // chunks per thread and row
    int src_off[NCH], dst_off[NCH];               // element offset inside an input row (-1: outside), byte offset in the slot
#pragma unroll
    for (int i = 0; i < NCH; i++) {
        const int q = threadIdx.x + i * 128;
        const int j = q >> 4, part = q & 15;
        const int wi = wt0 - P + j, c = cb * 128 + part * 8;
        dst_off[i] = q < ICOL * 16 ? q * 16 : -1;
        src_off[i] = (q < ICOL * 16 && wi >= 0 && wi < a.W && c < a.K) ? wi * a.K + c : -1;
    }
    auto copy_row = [&](int hi) {
        if (hi <= hi_last) {
            unsigned char *dst = ring + ((hi - hi_first) % RING) * S::ROW_BYTES;
            const bool rok = hi >= 0 && hi < a.H;
            const __nv_bfloat16 *xrow = ximg + (size_t)(rok ? hi : 0) * a.W * a.K;
#pragma unroll
            for (int i = 0; i < NCH; i++) {
                if (dst_off[i] >= 0) {
                    const bool ok = rok && src_off[i] >= 0;
                    cp_async16(dst + dst_off[i], ok ? (const void *)(xrow + src_off[i]) : (const void *)ximg, ok);
                }
            }
        }
        cp_async_commit();  // (a group per row, also when it is empty: the wait below counts groups)
    };
#pragma unroll 1
    for (int d = 0; d < RING - 1; d++) copy_row(hi_first + d);

    float2 acc[K][TW][2];
    for (int base = hi_first; base <= hi_last; base += K) {
#pragma unroll
        for (int u = 0; u < K; u++) {
            const int hi = base + u;
            if (hi <= hi_last) {  // (block-uniform)
                cp_async_wait<RING - 2>();  // this thread's copies of row hi have landed ...
                __syncthreads();            // ... and everybody's; everybody has also finished with row hi - 1
                copy_row(hi + RING - 1);    // into the slot row hi - 1 used
                const unsigned char *row = ring + ((hi - hi_first) % RING) * S::ROW_BYTES + (wrp * TW) * 256 + lane * 8;
                float2 xc[NCOL][2];
#pragma unroll
                for (int j = 0; j < NCOL; j++) {
                    const uint2 v = *reinterpret_cast<const uint2 *>(row + j * 256);
                    xc[j][0] = bf2_lo(v.x); xc[j][1] = bf2_lo(v.y);
                }
#pragma unroll
                for (int r = 0; r < K; r++) {
                    constexpr int KK = K;
                    const int slot = ((u - r) % KK + KK) % KK;
#pragma unroll
                    for (int s2 = 0; s2 < K; s2++) {
                        const float4 wq = wl[(r * K + s2) * 32];
                        const float2 w0 = make_float2(wq.x, wq.y), w1 = make_float2(wq.z, wq.w);
#pragma unroll
                        for (int t = 0; t < TW; t++) {
                            if (r == 0 && s2 == 0) {
                                acc[slot][t][0] = __fmul2_rn(xc[t + s2][0], w0);
                                acc[slot][t][1] = __fmul2_rn(xc[t + s2][1], w1);
                            } else {
                                acc[slot][t][0] = __ffma2_rn(xc[t + s2][0], w0, acc[slot][t][0]);
                                acc[slot][t][1] = __ffma2_rn(xc[t + s2][1], w1, acc[slot][t][1]);
                            }
                        }
                    }
                }
                // the output row this input row completes (filter row K - 1): hi - P
                const int oh = hi - P;
                if (active && oh >= ho_begin && oh < ho_end) {
                    constexpr int KK = K;
                    const int slot = ((u - (K - 1)) % KK + KK) % KK;
                    __nv_bfloat16 *yrow = yimg + (size_t)oh * a.Wo * a.K;
#pragma unroll
                    for (int t = 0; t < TW; t++) {
                        if (wo0 + t < a.Wo) {
                            uint2 ov;
                            __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&ov);
#pragma unroll
                            for (int j = 0; j < 2; j++) {
                                float2 v = __ffma2_rn(acc[slot][t][j], sc[j], sh[j]);
                                if (ACT == ACT_RELU) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); }
                                if (ACT == ACT_HSWISH) {
                                    const float2 g = make_float2(__saturatef(fmaf(v.x, 1.f / 6.f, 0.5f)), __saturatef(fmaf(v.y, 1.f / 6.f, 0.5f)));
                                    v = __fmul2_rn(v, g);
                                }
                                ob[j] = __float22bfloat162_rn(v);
                            }
                            *reinterpret_cast<uint2 *>(yrow + (size_t)(wo0 + t) * a.K) = ov;
                        }
                    }
                }
            }
        }
    }
    cp_async_wait<0>();
}
template <int K, int ACT, bool GROUP>
__global__ void __launch_bounds__(128, K == 7 ? 3 : 4) dw_walk_kernel(const ConvArgs a1, const char *__restrict__ tbl, int n_img, int chblocks) {
    __shared__ __align__(16) unsigned char smem[DwWalkShape<K>::SMEM];
    SGS_DW_ARGS()
    if (GROUP) { const ConvArgs al = a; dw_walk_body<K, ACT>(al, n, smem, chblocks); }
    else dw_walk_body<K, ACT>(a, n, smem, chblocks);
}
// grid of the walking kernel for a member with `kmax` channels at most
static dim3 dw_walk_grid(const ConvArgs &a, int kmax, int TW, int images) {
    const int chblocks = (kmax / 4 + 31) / 32, tiles_w = (a.Wo + 4 * TW - 1) / (4 * TW);
    return dim3((unsigned)(chblocks * tiles_w), (unsigned)((a.Ho + DW_WALK_SEG - 1) / DW_WALK_SEG), (unsigned)images);
}

// Members of one launch with different kernel sizes (a wave's depthwise layer: every member crops its own
// k x k window out of the stored 7x7): each block runs the body of its member's kernel size.  The grid
// covers the largest member; blocks beyond a member's own extent leave at once.
// Stride 1: the walking bodies on the walking kernel's grid (sized for strips of 2 columns and the widest member);
// stride 2: the patch / row bodies on their grid.
template <int ST, int ACT, bool WALK> __device__ __forceinline__ void dw_mixed_dispatch(const ConvArgs &a, const int n, unsigned char *wsm, int chblocks);
template <int ST, int ACT, bool WALK>
__global__ void __launch_bounds__(128, 3) dw_mixed_kernel(const char *__restrict__ tbl, int n_img, int chblocks) {
    constexpr bool GROUP = true;
    __shared__ __align__(16) unsigned char wsm[WALK ? DwWalkShape<7>::SMEM : 16];  // (7x7 needs the most; 5x5: 37376, 3x3: 41472 bytes)
    static_assert(DwWalkShape<7>::SMEM >= DwWalkShape<5>::SMEM && DwWalkShape<7>::SMEM >= DwWalkShape<3>::SMEM && DwWalkShape<7>::SMEM <= 48 * 1024, "ring sizes");
    const ConvArgs a1 = ConvArgs();
    SGS_DW_ARGS()
    const ConvArgs al = a;  // (a copy in registers: reading the fields from shared memory at every use costs the tiled bodies 100 registers more)
    dw_mixed_dispatch<ST, ACT, WALK>(al, n, wsm, chblocks);
}
template <int ST, int ACT, bool WALK>
__device__ __forceinline__ void dw_mixed_dispatch(const ConvArgs &a, const int n, unsigned char *wsm, int chblocks) {
    if (WALK) {
        if (a.k == 3) dw_walk_body<3, ACT>(a, n, wsm, chblocks);
        else if (a.k == 5) dw_walk_body<5, ACT>(a, n, wsm, chblocks);
        else dw_walk_body<7, ACT>(a, n, wsm, chblocks);
    } else if (ST == 1) {
        if (a.k == 3) dw_tile_body<3, 1, 2, 4, true, ACT>(a, n);
        else if (a.k == 5) dw_tile_body<5, 1, 1, 4, true, ACT>(a, n);
        else dw_vec_body<7, 1>(a, n);
    } else {
        if (a.k == 3) dw_tile_body<3, 2, 1, 4, false, ACT>(a, n);
        else if (a.k == 5) dw_vec_body<5, 2>(a, n);
        else dw_vec_body<7, 2>(a, n);
    }
}

// `a` = the (first) member; grouped: kmax = the widest member's channel count, tbl = device table, members > 0
template <int K, int ST, int TH, int TW, bool PRELOAD, bool GROUP>
static cudaError_t launch_dw_tile(const ConvArgs &a, int kmax, const char *tbl, int members, cudaStream_t st) {
    const int per_row = ((a.Wo + TW - 1) / TW) * (kmax / 8);
    dim3 grid((per_row + 127) / 128, (a.Ho + TH - 1) / TH, a.N * (GROUP ? members : 1));
    if (a.act == ACT_RELU) dw_tile_kernel<K, ST, TH, TW, PRELOAD, ACT_RELU, GROUP><<<grid, 128, 0, st>>>(a, tbl, a.N);
    else if (a.act == ACT_HSWISH) dw_tile_kernel<K, ST, TH, TW, PRELOAD, ACT_HSWISH, GROUP><<<grid, 128, 0, st>>>(a, tbl, a.N);
    else dw_tile_kernel<K, ST, TH, TW, PRELOAD, ACT_NONE, GROUP><<<grid, 128, 0, st>>>(a, tbl, a.N);
    return cudaGetLastError();
}

template <int K, bool GROUP>
static cudaError_t launch_dw_walk(const ConvArgs &a, int kmax, const char *tbl, int members, cudaStream_t st) {
    const dim3 grid = dw_walk_grid(a, kmax, DwWalkShape<K>::TW, a.N * (GROUP ? members : 1));
    const int chblocks = (kmax / 4 + 31) / 32;
    if (a.act == ACT_RELU) dw_walk_kernel<K, ACT_RELU, GROUP><<<grid, 128, 0, st>>>(a, tbl, a.N, chblocks);
    else if (a.act == ACT_HSWISH) dw_walk_kernel<K, ACT_HSWISH, GROUP><<<grid, 128, 0, st>>>(a, tbl, a.N, chblocks);
    else dw_walk_kernel<K, ACT_NONE, GROUP><<<grid, 128, 0, st>>>(a, tbl, a.N, chblocks);
    return cudaGetLastError();
}

template <int K, int ST, bool GROUP>
static cudaError_t launch_dw_vec(const ConvArgs &a, int kmax, const char *tbl, int members, cudaStream_t st) {
    const int per_row = ((a.Wo + 3) / 4) * (kmax / 8);
    const int block = per_row >= 256 ? 256 : per_row >= 128 ? 128 : 64;
    dim3 grid((per_row + block - 1) / block, a.Ho, a.N * (GROUP ? members : 1));
    dw_vec_kernel<K, ST, GROUP><<<grid, block, 0, st>>>(a, tbl, a.N);
    return cudaGetLastError();
}

static bool dw_vec_eligible(const ConvArgs &a) {
    return a.K % 8 == 0 && a.Kmax % 8 == 0 && (a.stride == 1 || a.stride == 2) && a.Ho <= 65535 && a.N <= 65535 &&
           (size_t)a.W * a.K < (1u << 30) &&
           ((reinterpret_cast<uintptr_t>(a.x) | reinterpret_cast<uintptr_t>(a.w) | reinterpret_cast<uintptr_t>(a.y)) & 15) == 0 &&
           ((reinterpret_cast<uintptr_t>(a.scale) | reinterpret_cast<uintptr_t>(a.shift)) & 15) == 0;
}

// Stride-1 layers take the walking kernel when the launch is large: at least this many million output elements over
// all images and members, on maps at least 28 wide.  A block walks up to 56 rows one after the other, which pays on
// working sets that stream from HBM (64 x 56 x 56 x 480: +6 % for 3x3, +13 % for 7x7 over the patch / row kernels) and
// loses on the small launches of batch-1 waves (MobileNetV3-shaped stream: 34.7k queries/s without it, 32.3k with it
// everywhere), where the patch kernels' many short threads win.  0 = never, negative = always; tuning aid.
static int g_dw_walk_min_melems = 48;
void dw_set_walk(int min_million_elements) { g_dw_walk_min_melems = min_million_elements; }
static bool dw_walks(const ConvArgs &a, int kmax, int members) {
    if (g_dw_walk_min_melems < 0) return true;  // (tests: every stride-1 shape through the walking kernel)
    return g_dw_walk_min_melems > 0 && a.Wo >= 28 &&
           (long long)a.N * members * a.Ho * a.Wo * kmax >= (long long)g_dw_walk_min_melems * 1000000ll;
}

// The vectorised bf16 kernel of a (kernel size, stride) pair; measured on working sets beyond L2
// (N64 56x56 C480) the tiled kernel wins for k3 and for k5 stride 1.
template <bool GROUP>
static cudaError_t launch_dw_bf16(const ConvArgs &a, int kmax, const char *tbl, int members, cudaStream_t st) {
    switch (a.k * 10 + a.stride) {
    case 31: return dw_walks(a, kmax, GROUP ? members : 1) ? launch_dw_walk<3, GROUP>(a, kmax, tbl, members, st) : launch_dw_tile<3, 1, 2, 4, true, GROUP>(a, kmax, tbl, members, st);
    case 32: return launch_dw_tile<3, 2, 1, 4, false, GROUP>(a, kmax, tbl, members, st);
    case 51: return dw_walks(a, kmax, GROUP ? members : 1) ? launch_dw_walk<5, GROUP>(a, kmax, tbl, members, st) : launch_dw_tile<5, 1, 1, 4, true, GROUP>(a, kmax, tbl, members, st);
    case 52: return launch_dw_vec<5, 2, GROUP>(a, kmax, tbl, members, st);
    case 71: return dw_walks(a, kmax, GROUP ? members : 1) ? launch_dw_walk<7, GROUP>(a, kmax, tbl, members, st) : launch_dw_vec<7, 1, GROUP>(a, kmax, tbl, members, st);
    case 72: return launch_dw_vec<7, 2, GROUP>(a, kmax, tbl, members, st);
    default: return cudaErrorNotSupported;
    }
}

cudaError_t launch_dw_group(const char *h_tbl, const char *d_tbl, int members, cudaStream_t st) {
    if (members <= 0) return cudaSuccess;
    const ConvArgs &a0 = *reinterpret_cast<const ConvArgs *>(h_tbl);
    int kmax = 0;
    bool mixed = false;
    for (int i = 0; i < members; i++) {
        const ConvArgs &a = *reinterpret_cast<const ConvArgs *>(h_tbl + (size_t)i * DW_ENTRY_BYTES);
        if (!dw_vec_eligible(a) || (a.k != 3 && a.k != 5 && a.k != 7) || a.stride != a0.stride || a.act != a0.act || a.N != a0.N ||
            a.H != a0.H || a.W != a0.W)
            return cudaErrorNotSupported;
        kmax = std::max(kmax, a.K);
        mixed = mixed || a.k != a0.k;
    }
    if ((long long)a0.N * members > 65535) return cudaErrorNotSupported;
    if (!mixed) return launch_dw_bf16<true>(a0, kmax, d_tbl, members, st);
    // (same input size and stride, odd kernels with padding (k - 1) / 2: every member has the same output size)
    const int per_row = ((a0.Wo + 3) / 4) * (kmax / 8);
    const int chblocks = (kmax / 4 + 31) / 32;
    if (a0.stride == 1 && dw_walks(a0, kmax, members)) {
        const dim3 grid = dw_walk_grid(a0, kmax, 2, a0.N * members);
        if (a0.act == ACT_RELU) dw_mixed_kernel<1, ACT_RELU, true><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
        else if (a0.act == ACT_HSWISH) dw_mixed_kernel<1, ACT_HSWISH, true><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
        else dw_mixed_kernel<1, ACT_NONE, true><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
    } else if (a0.stride == 1) {
        // (the patch bodies of 3x3 and 5x5 own 2 resp. 1 output rows per block row: the grid covers single rows,
        // blocks beyond a member's own extent leave at once)
        dim3 grid((per_row + 127) / 128, a0.Ho, a0.N * members);
        if (a0.act == ACT_RELU) dw_mixed_kernel<1, ACT_RELU, false><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
        else if (a0.act == ACT_HSWISH) dw_mixed_kernel<1, ACT_HSWISH, false><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
        else dw_mixed_kernel<1, ACT_NONE, false><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
    } else {
        dim3 grid((per_row + 127) / 128, a0.Ho, a0.N * members);
        if (a0.act == ACT_RELU) dw_mixed_kernel<2, ACT_RELU, false><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
        else if (a0.act == ACT_HSWISH) dw_mixed_kernel<2, ACT_HSWISH, false><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
        else dw_mixed_kernel<2, ACT_NONE, false><<<grid, 128, 0, st>>>(d_tbl, a0.N, chblocks);
    }
    return cudaGetLastError();
}

template <typename T> cudaError_t launch_dw(const ConvArgs &a, cudaStream_t st) {
    size_t total = (size_t)a.N * a.Ho * a.Wo * a.K;
    if (!total) return cudaSuccess;
    if (sizeof(T) == 2 && dw_vec_eligible(a)) {
        cudaError_t e = launch_dw_bf16<false>(a, a.K, nullptr, 1, st);
        if (e != cudaErrorNotSupported) return e;
    }
    int blocks = (int)std::min<size_t>((total + 255) / 256, 148 * 16);
    dw_plain_kernel<T><<<blocks, 256, 0, st>>>(a);
    return cudaGetLastError();
}
template cudaError_t launch_dw<float>(const ConvArgs &, cudaStream_t);
template cudaError_t launch_dw<__nv_bfloat16>(const ConvArgs &, cudaStream_t);

// ---------------------------------------------------------------------------------------------
// 3x3 stride-2 max pool, padding 1 (only in-image taps compared)
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void maxpool_kernel(const T *__restrict__ x, T *__restrict__ y, int N, int H, int W, int C, int Ho, int Wo) {
    size_t total = (size_t)N * Ho * Wo * C;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int c = (int)(i % C);
        size_t m = i / C;
        int wo = (int)(m % Wo), ho = (int)((m / Wo) % Ho), n = (int)(m / ((size_t)Wo * Ho));
        float best = -INFINITY;
        for (int r = 0; r < 3; r++) {
            int hi = 2 * ho + r - 1;
            if (hi < 0 || hi >= H) continue;
            for (int s = 0; s < 3; s++) {
                int wi = 2 * wo + s - 1;
                if (wi < 0 || wi >= W) continue;
                best = fmaxf(best, to_f<T>(x[(((size_t)n * H + hi) * W + wi) * C + c]));
            }
        }
        y[i] = from_f<T>(best);
    }
}
template <typename T> cudaError_t launch_maxpool3s2(const T *x, T *y, int N, int H, int W, int C, cudaStream_t st) {
    int Ho = (H - 1) / 2 + 1, Wo = (W - 1) / 2 + 1;
    size_t total = (size_t)N * Ho * Wo * C;
    if (!total) return cudaSuccess;
    int blocks = (int)std::min<size_t>((total + 255) / 256, 148 * 16);
    maxpool_kernel<T><<<blocks, 256, 0, st>>>(x, y, N, H, W, C, Ho, Wo);
    return cudaGetLastError();
}
template cudaError_t launch_maxpool3s2<float>(const float *, float *, int, int, int, int, cudaStream_t);
template cudaError_t launch_maxpool3s2<__nv_bfloat16>(const __nv_bfloat16 *, __nv_bfloat16 *, int, int, int, int, cudaStream_t);

// ---------------------------------------------------------------------------------------------
// Global average pool: g[n][c] = mean_{hw} x[n][hw][c], fp32 result.
// grid (ceil(C/32), N), block (32, 8): 8 pixel lanes per channel, reduced through shared memory.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void gap_kernel(const T *__restrict__ x, float *__restrict__ g, int HW, int C) {
    __shared__ float part[8][33];
    int c = blockIdx.x * 32 + threadIdx.x, n = blockIdx.y;
    float s = 0.f;
    if (c < C)
        for (int i = threadIdx.y; i < HW; i += 8) s += to_f<T>(x[((size_t)n * HW + i) * C + c]);
    part[threadIdx.y][threadIdx.x] = s;
    __syncthreads();
    if (threadIdx.y == 0 && c < C) {
        float tot = 0.f;
#pragma unroll
        for (int j = 0; j < 8; j++) tot += part[j][threadIdx.x];
        g[(size_t)n * C + c] = tot / (float)HW;
    }
}
// bf16, C % 8 == 0: one warp per (image, 8-channel vector); lanes stride over the pixels with 16-byte
// loads and the lane sums are combined by a fixed shuffle tree (same result every run).
__device__ __forceinline__ float2 bf2f(uint32_t u) { return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u)); }

__global__ void __launch_bounds__(256) gap_vec_kernel(const __nv_bfloat16 *__restrict__ x, float *__restrict__ g, int N, int HW, int C) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int cvecs = C >> 3;
    if (warp >= N * cvecs) return;
    const int n = warp / cvecs, cv = warp % cvecs;
    const __nv_bfloat16 *base = x + (size_t)n * HW * C + cv * 8;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int i = lane; i < HW; i += 32) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(base + (size_t)i * C));
        const float2 a = bf2f(v.x), b = bf2f(v.y), c = bf2f(v.z), d = bf2f(v.w);
        acc[0] += a.x; acc[1] += a.y; acc[2] += b.x; acc[3] += b.y; acc[4] += c.x; acc[5] += c.y; acc[6] += d.x; acc[7] += d.y;
    }
#pragma unroll
    for (int j = 0; j < 8; j++)
#pragma unroll
        for (int o = 16; o; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
    if (lane == 0) {
        const float inv = 1.f / (float)HW;
        float4 *dst = reinterpret_cast<float4 *>(g + (size_t)n * C + cv * 8);
        dst[0] = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
        dst[1] = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
    }
}

template <typename T> cudaError_t launch_gap(const T *x, float *g, int N, int HW, int C, cudaStream_t st) {
    if (N <= 0 || C <= 0) return cudaSuccess;
    if (sizeof(T) == 2 && C % 8 == 0 && (reinterpret_cast<uintptr_t>(x) & 15) == 0 && (reinterpret_cast<uintptr_t>(g) & 15) == 0) {
        const int warps = N * (C / 8);
        gap_vec_kernel<<<(warps * 32 + 255) / 256, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16 *>(x), g, N, HW, C);
        return cudaGetLastError();
    }
    dim3 grid((C + 31) / 32, N), block(32, 8);
    gap_kernel<T><<<grid, block, 0, st>>>(x, g, HW, C);
    return cudaGetLastError();
}
template cudaError_t launch_gap<float>(const float *, float *, int, int, int, cudaStream_t);
template cudaError_t launch_gap<__nv_bfloat16>(const __nv_bfloat16 *, float *, int, int, int, cudaStream_t);

// ---------------------------------------------------------------------------------------------
// Squeeze-excite gate: z = relu(W1[:sq,:mid] g + b1), gate = hsigmoid(W2[:mid,:sq] z + b2).
// One block per image; warps stride over outputs and reduce with shuffles.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(1024) se_gate_kernel(const float *__restrict__ g, const T *__restrict__ w1,
                                                      const float *__restrict__ b1, const T *__restrict__ w2,
                                                      const float *__restrict__ b2, float *__restrict__ gate, int mid,
                                                      int sq, int w1_ld, int w2_ld) {
    extern __shared__ float sm[];
    float *gs = sm, *zs = sm + mid;
    int n = blockIdx.x, lane = threadIdx.x % 32, warp = threadIdx.x / 32, nw = blockDim.x / 32;
    for (int c = threadIdx.x; c < mid; c += blockDim.x) gs[c] = g[(size_t)n * mid + c];
    __syncthreads();
    for (int j = warp; j < sq; j += nw) {
        float s = 0.f;
        for (int c = lane; c < mid; c += 32) s = fmaf(to_f<T>(w1[(size_t)j * w1_ld + c]), gs[c], s);
#pragma unroll
        for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) zs[j] = fmaxf(s + b1[j], 0.f);
    }
    __syncthreads();
    for (int c = warp; c < mid; c += nw) {
        float s = 0.f;
        for (int j = lane; j < sq; j += 32) s = fmaf(to_f<T>(w2[(size_t)c * w2_ld + j]), zs[j], s);
#pragma unroll
        for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) gate[(size_t)n * mid + c] = fminf(fmaxf(s + b2[c] + 3.f, 0.f), 6.f) / 6.f;
    }
}
template <typename T>
cudaError_t launch_se_gate(const float *g, const T *w1, const float *b1, const T *w2, const float *b2, float *gate,
                           int N, int mid, int sq, int w1_ld, int w2_ld, cudaStream_t st) {
    if (N <= 0) return cudaSuccess;
    se_gate_kernel<T><<<N, 1024, (size_t)(mid + sq) * sizeof(float), st>>>(g, w1, b1, w2, b2, gate, mid, sq, w1_ld, w2_ld);
    return cudaGetLastError();
}
template cudaError_t launch_se_gate<float>(const float *, const float *, const float *, const float *, const float *, float *, int, int, int, int, int, cudaStream_t);
template cudaError_t launch_se_gate<__nv_bfloat16>(const float *, const __nv_bfloat16 *, const float *, const __nv_bfloat16 *, const float *, float *, int, int, int, int, int, cudaStream_t);

// y[n][hw][c] = x[n][hw][c] * gate[n][c]
template <typename T>
__global__ void scale_kernel(const T *__restrict__ x, const float *__restrict__ gate, T *__restrict__ y, size_t total,
                             int HW, int C) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        int c = (int)(i % C);
        size_t n = i / ((size_t)HW * C);
        y[i] = from_f<T>(to_f<T>(x[i]) * gate[n * C + c]);
    }
}
__global__ void __launch_bounds__(256) scale_vec_kernel(const __nv_bfloat16 *__restrict__ x, const float *__restrict__ gate,
                                                        __nv_bfloat16 *__restrict__ y, int vecs_per_image, int cvecs, int C, int total) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;  // one 8-channel vector
    if (i >= total) return;
    const int n = i / vecs_per_image, cv = i % cvecs;
    const uint4 v = *reinterpret_cast<const uint4 *>(x + (size_t)i * 8);
    const float4 g0 = __ldg(reinterpret_cast<const float4 *>(gate + (size_t)n * C + cv * 8));
    const float4 g1 = __ldg(reinterpret_cast<const float4 *>(gate + (size_t)n * C + cv * 8 + 4));
    const float2 a = bf2f(v.x), b = bf2f(v.y), c = bf2f(v.z), d = bf2f(v.w);
    uint4 o;
    __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&o);
    ob[0] = __floats2bfloat162_rn(a.x * g0.x, a.y * g0.y);
    ob[1] = __floats2bfloat162_rn(b.x * g0.z, b.y * g0.w);
    ob[2] = __floats2bfloat162_rn(c.x * g1.x, c.y * g1.y);
    ob[3] = __floats2bfloat162_rn(d.x * g1.z, d.y * g1.w);
    *reinterpret_cast<uint4 *>(y + (size_t)i * 8) = o;
}

template <typename T> cudaError_t launch_scale(const T *x, const float *gate, T *y, int N, int HW, int C, cudaStream_t st) {
    size_t total = (size_t)N * HW * C;
    if (!total) return cudaSuccess;
    if (sizeof(T) == 2 && C % 8 == 0 && total / 8 < (1u << 30) &&
        ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y) | reinterpret_cast<uintptr_t>(gate)) & 15) == 0) {
        const int tv = (int)(total / 8);
        scale_vec_kernel<<<(tv + 255) / 256, 256, 0, st>>>(reinterpret_cast<const __nv_bfloat16 *>(x), gate,
                                                          reinterpret_cast<__nv_bfloat16 *>(y), HW * (C / 8), C / 8, C, tv);
        return cudaGetLastError();
    }
    int blocks = (int)std::min<size_t>((total + 255) / 256, 148 * 16);
    scale_kernel<T><<<blocks, 256, 0, st>>>(x, gate, y, total, HW, C);
    return cudaGetLastError();
}
template cudaError_t launch_scale<float>(const float *, const float *, float *, int, int, int, cudaStream_t);
template cudaError_t launch_scale<__nv_bfloat16>(const __nv_bfloat16 *, const float *, __nv_bfloat16 *, int, int, int, cudaStream_t);

// ---------------------------------------------------------------------------------------------
// Sliced linear layer on fp32 vectors: y[n][j] = act(sum_{c<C} w[j][c] v[n][c] + bias[j]), j < K.
// One warp per (n, j).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256) linear_kernel(const float *__restrict__ v, const T *__restrict__ w,
                                                     const float *__restrict__ bias, float *__restrict__ y, int N,
                                                     int C, int K, int ld, int act) {
    int warp = (blockIdx.x * blockDim.x + threadIdx.x) / 32, lane = threadIdx.x % 32;
    if (warp >= N * K) return;
    int n = warp / K, j = warp % K;
    float s = 0.f;
    for (int c = lane; c < C; c += 32) s = fmaf(to_f<T>(w[(size_t)j * ld + c]), v[(size_t)n * C + c], s);
#pragma unroll
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) y[(size_t)n * K + j] = apply_act(s + bias[j], act);
}
// bf16 weights, C % 8 == 0, ld % 8 == 0: each lane takes 8 weights (16 bytes) and 8 inputs per step
__global__ void __launch_bounds__(256) linear_vec_kernel(const float *__restrict__ v, const __nv_bfloat16 *__restrict__ w,
                                                         const float *__restrict__ bias, float *__restrict__ y, int N, int C,
                                                         int K, int ld, int act) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= N * K) return;
    const int n = warp / K, j = warp % K;
    const __nv_bfloat16 *wr = w + (size_t)j * ld;
    const float *vr = v + (size_t)n * C;
    float s = 0.f;
    for (int c = lane * 8; c < C; c += 256) {
        const uint4 wv = __ldg(reinterpret_cast<const uint4 *>(wr + c));
        const float4 x0 = *reinterpret_cast<const float4 *>(vr + c), x1 = *reinterpret_cast<const float4 *>(vr + c + 4);
        const float2 a = bf2f(wv.x), b = bf2f(wv.y), cc = bf2f(wv.z), d = bf2f(wv.w);
        s = fmaf(a.x, x0.x, s); s = fmaf(a.y, x0.y, s); s = fmaf(b.x, x0.z, s); s = fmaf(b.y, x0.w, s);
        s = fmaf(cc.x, x1.x, s); s = fmaf(cc.y, x1.y, s); s = fmaf(d.x, x1.z, s); s = fmaf(d.y, x1.w, s);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) y[(size_t)n * K + j] = apply_act(s + bias[j], act);
}

template <typename T>
cudaError_t launch_linear(const float *v, const T *w, const float *bias, float *y, int N, int C, int K, int ld, int act,
                          cudaStream_t st) {
    long long warps = (long long)N * K;
    if (warps <= 0) return cudaSuccess;
    if (sizeof(T) == 2 && C % 8 == 0 && ld % 8 == 0 && ((reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(v)) & 15) == 0) {
        linear_vec_kernel<<<(unsigned)((warps * 32 + 255) / 256), 256, 0, st>>>(v, reinterpret_cast<const __nv_bfloat16 *>(w), bias, y, N,
                                                                               C, K, ld, act);
        return cudaGetLastError();
    }
    int blocks = (int)((warps * 32 + 255) / 256);
    linear_kernel<T><<<blocks, 256, 0, st>>>(v, w, bias, y, N, C, K, ld, act);
    return cudaGetLastError();
}
template cudaError_t launch_linear<float>(const float *, const float *, const float *, float *, int, int, int, int, int, cudaStream_t);
template cudaError_t launch_linear<__nv_bfloat16>(const float *, const __nv_bfloat16 *, const float *, float *, int, int, int, int, int, cudaStream_t);

// ---------------------------------------------------------------------------------------------
// Record-driven bf16 kernels (see SmallEntry): each body works on one member; the `single` kernels get
// the record by value, the `group` kernels pick it from a device table with blockIdx.y.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t bf2_max(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmax2(*reinterpret_cast<const __nv_bfloat162 *>(&a), *reinterpret_cast<const __nv_bfloat162 *>(&b));
    return *reinterpret_cast<uint32_t *>(&r);
}

// 3x3 stride-2 max pool, padding 1: a thread owns 8 channels of one output pixel.
__device__ __forceinline__ void maxpool_body(const SmallEntry &e, int bx, int nbx) {
    const int cv = e.C >> 3;
    const int total = e.N * e.Ho * e.Wo * cv;
    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(e.x);
    __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(e.y);
    for (int i = bx * blockDim.x + threadIdx.x; i < total; i += nbx * blockDim.x) {
        const int c = i % cv, m = i / cv;
        const int wo = m % e.Wo, ho = (m / e.Wo) % e.Ho, n = m / (e.Wo * e.Ho);
        uint4 best = make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);  // -inf pairs
#pragma unroll
        for (int r = 0; r < 3; r++) {
            const int hi = 2 * ho + r - 1;
            if (hi < 0 || hi >= e.H) continue;
#pragma unroll
            for (int s = 0; s < 3; s++) {
                const int wi = 2 * wo + s - 1;
                if (wi < 0 || wi >= e.W) continue;
                const uint4 v = __ldg(reinterpret_cast<const uint4 *>(x + (((size_t)n * e.H + hi) * e.W + wi) * e.C) + c);
                best.x = bf2_max(best.x, v.x); best.y = bf2_max(best.y, v.y); best.z = bf2_max(best.z, v.z); best.w = bf2_max(best.w, v.w);
            }
        }
        reinterpret_cast<uint4 *>(y + (size_t)m * e.C)[c] = best;
    }
}

// Global average pool: one warp per 8-channel vector of one image (fixed shuffle tree).
__device__ __forceinline__ void gap_body(const SmallEntry &e, int bx) {
    const int warp = (bx * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const int cvecs = e.C >> 3, HW = e.H * e.W;
    if (warp >= e.N * cvecs) return;
    const int n = warp / cvecs, cv = warp % cvecs;
    const __nv_bfloat16 *base = static_cast<const __nv_bfloat16 *>(e.x) + (size_t)n * HW * e.C + cv * 8;
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int i = lane; i < HW; i += 32) {
        const uint4 v = __ldg(reinterpret_cast<const uint4 *>(base + (size_t)i * e.C));
        const float2 a = bf2f(v.x), b = bf2f(v.y), c = bf2f(v.z), d = bf2f(v.w);
        acc[0] += a.x; acc[1] += a.y; acc[2] += b.x; acc[3] += b.y; acc[4] += c.x; acc[5] += c.y; acc[6] += d.x; acc[7] += d.y;
    }
#pragma unroll
    for (int j = 0; j < 8; j++)
#pragma unroll
        for (int o = 16; o; o >>= 1) acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], o);
    if (lane == 0) {
        const float inv = 1.f / (float)HW;
        float4 *dst = reinterpret_cast<float4 *>(static_cast<float *>(e.y) + (size_t)n * e.C + cv * 8);
        dst[0] = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
        dst[1] = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
    }
}

// y[n][hw][c] = x[n][hw][c] * gate[n][c] (gate = e.w, fp32): a thread scales one 8-channel vector.
__device__ __forceinline__ void scale_body(const SmallEntry &e, int bx, int nbx) {
    const int cvecs = e.C >> 3, per_image = e.H * e.W * cvecs, total = e.N * per_image;
    const __nv_bfloat16 *x = static_cast<const __nv_bfloat16 *>(e.x);
    const float *gate = static_cast<const float *>(e.w);
    __nv_bfloat16 *y = static_cast<__nv_bfloat16 *>(e.y);
    for (int i = bx * blockDim.x + threadIdx.x; i < total; i += nbx * blockDim.x) {
        const int n = i / per_image, cv = i % cvecs;
        const uint4 v = *reinterpret_cast<const uint4 *>(x + (size_t)i * 8);
        const float4 g0 = __ldg(reinterpret_cast<const float4 *>(gate + (size_t)n * e.C + cv * 8));
        const float4 g1 = __ldg(reinterpret_cast<const float4 *>(gate + (size_t)n * e.C + cv * 8 + 4));
        const float2 a = bf2f(v.x), b = bf2f(v.y), c = bf2f(v.z), d = bf2f(v.w);
        uint4 o;
        __nv_bfloat162 *ob = reinterpret_cast<__nv_bfloat162 *>(&o);
        ob[0] = __floats2bfloat162_rn(a.x * g0.x, a.y * g0.y);
        ob[1] = __floats2bfloat162_rn(b.x * g0.z, b.y * g0.w);
        ob[2] = __floats2bfloat162_rn(c.x * g1.x, c.y * g1.y);
        ob[3] = __floats2bfloat162_rn(d.x * g1.z, d.y * g1.w);
        *reinterpret_cast<uint4 *>(y + (size_t)i * 8) = o;
    }
}

// Dot product of 8 bf16 weights (one 16-byte vector) with 8 fp32 values.
__device__ __forceinline__ float dot8(uint4 wv, float4 x0, float4 x1, float s) {
    const float2 a = bf2f(wv.x), b = bf2f(wv.y), c = bf2f(wv.z), d = bf2f(wv.w);
    s = fmaf(a.x, x0.x, s); s = fmaf(a.y, x0.y, s); s = fmaf(b.x, x0.z, s); s = fmaf(b.y, x0.w, s);
    s = fmaf(c.x, x1.x, s); s = fmaf(c.y, x1.y, s); s = fmaf(d.x, x1.z, s); s = fmaf(d.y, x1.w, s);
    return s;
}

// Squeeze-excite gate of one image of one member (se_gate_kernel's arithmetic, other summation order):
// x = pooled vector, w / bias = first FC (K = squeeze width, ld), w2 / bias2 = second FC (ld2), y = gate;
// C = mid channels.  Both FCs are a few hundred short dot products: a warp takes JB outputs at a time and
// issues the 16-byte weight loads of all of them before the first use, so a block pays the memory
// latency a handful of times instead of once per output.  The gate of one image is the work of a cluster
// of SE_SPLIT blocks (one block alone streams both weight matrices through a single SM): every block
// computes a share of the first FC's outputs and writes them into all the blocks' shared memory, and
// after the cluster barrier a share of the second FC's.
constexpr int SE_SPLIT = 4, SE_THREADS = 512;
__global__ void __cluster_dims__(SE_SPLIT, 1, 1) __launch_bounds__(SE_THREADS) se_gate_group_kernel(const SmallEntry *__restrict__ tbl) {
    extern __shared__ __align__(16) float sm[];
    __shared__ SmallEntry e;
    cooperative_groups::cluster_group cluster = cooperative_groups::this_cluster();
    const int rank = (int)cluster.block_rank();
    if (threadIdx.x < 8) reinterpret_cast<uint4 *>(&e)[threadIdx.x] = __ldg(reinterpret_cast<const uint4 *>(tbl + blockIdx.y) + threadIdx.x);
    __syncthreads();
    const int mid = e.C, sq = e.K;
    float *gs = sm, *zs = sm + mid;
    const int n = blockIdx.x / SE_SPLIT, lane = threadIdx.x % 32, nwb = blockDim.x / 32;
    const int warp = rank * nwb + threadIdx.x / 32, nw = nwb * SE_SPLIT;  // warps of the whole cluster share the outputs
    if (n >= e.N) return;  // (the same for every block of a cluster)
    float *zs_peer = cluster.map_shared_rank(zs, lane < SE_SPLIT ? lane : 0);  // lanes 0..SE_SPLIT-1 each write one block's copy
    const float *g = static_cast<const float *>(e.x);
    const __nv_bfloat16 *w1 = static_cast<const __nv_bfloat16 *>(e.w), *w2 = static_cast<const __nv_bfloat16 *>(e.w2);
    float *gate = static_cast<float *>(e.y);
    for (int c = threadIdx.x; c < mid; c += blockDim.x) gs[c] = g[(size_t)n * mid + c];
    __syncthreads();
    const bool vec = ((mid | sq | e.ld | e.ld2) & 7) == 0 && ((reinterpret_cast<uintptr_t>(w1) | reinterpret_cast<uintptr_t>(w2)) & 15) == 0;
    if (vec) {
        constexpr int JB = 4;
        for (int j0 = warp * JB; j0 < sq; j0 += nw * JB) {
            float s[JB];
#pragma unroll
            for (int u = 0; u < JB; u++) s[u] = 0.f;
            for (int c = lane * 8; c < mid; c += 256) {
                uint4 wv[JB];
#pragma unroll
                for (int u = 0; u < JB; u++)
                    wv[u] = j0 + u < sq ? __ldg(reinterpret_cast<const uint4 *>(w1 + (size_t)(j0 + u) * e.ld + c)) : make_uint4(0u, 0u, 0u, 0u);
                const float4 x0 = *reinterpret_cast<const float4 *>(gs + c), x1 = *reinterpret_cast<const float4 *>(gs + c + 4);
#pragma unroll
                for (int u = 0; u < JB; u++) s[u] = dot8(wv[u], x0, x1, s[u]);
            }
#pragma unroll
            for (int u = 0; u < JB; u++) {
#pragma unroll
                for (int o = 16; o; o >>= 1) s[u] += __shfl_xor_sync(0xffffffffu, s[u], o);
                if (lane < SE_SPLIT && j0 + u < sq) zs_peer[j0 + u] = fmaxf(s[u] + e.bias[j0 + u], 0.f);
            }
        }
    } else {
        for (int j = warp; j < sq; j += nw) {
            float s = 0.f;
            for (int c = lane; c < mid; c += 32) s = fmaf(__bfloat162float(w1[(size_t)j * e.ld + c]), gs[c], s);
#pragma unroll
            for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane < SE_SPLIT) zs_peer[j] = fmaxf(s + e.bias[j], 0.f);
        }
    }
    cluster.sync();  // every block's zs is complete (and no block leaves while others may still write into it)
    if (vec) {
        constexpr int JB = 8;
        for (int c0 = warp * JB; c0 < mid; c0 += nw * JB) {
            float s[JB];
#pragma unroll
            for (int u = 0; u < JB; u++) s[u] = 0.f;
            for (int j = lane * 8; j < sq; j += 256) {
                uint4 wv[JB];
#pragma unroll
                for (int u = 0; u < JB; u++)
                    wv[u] = c0 + u < mid ? __ldg(reinterpret_cast<const uint4 *>(w2 + (size_t)(c0 + u) * e.ld2 + j)) : make_uint4(0u, 0u, 0u, 0u);
                const float4 x0 = *reinterpret_cast<const float4 *>(zs + j), x1 = *reinterpret_cast<const float4 *>(zs + j + 4);
#pragma unroll
                for (int u = 0; u < JB; u++) s[u] = dot8(wv[u], x0, x1, s[u]);
            }
#pragma unroll
            for (int u = 0; u < JB; u++) {
#pragma unroll
                for (int o = 16; o; o >>= 1) s[u] += __shfl_xor_sync(0xffffffffu, s[u], o);
                if (lane == 0 && c0 + u < mid) gate[(size_t)n * mid + c0 + u] = fminf(fmaxf(s[u] + e.bias2[c0 + u] + 3.f, 0.f), 6.f) / 6.f;
            }
        }
    } else {
        for (int c = warp; c < mid; c += nw) {
            float s = 0.f;
            for (int j = lane; j < sq; j += 32) s = fmaf(__bfloat162float(w2[(size_t)c * e.ld2 + j]), zs[j], s);
#pragma unroll
            for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0) gate[(size_t)n * mid + c] = fminf(fmaxf(s + e.bias2[c] + 3.f, 0.f), 6.f) / 6.f;
        }
    }
}

// Sliced linear layer on fp32 vectors: one warp per (image, output), 16-byte weight loads.
__device__ __forceinline__ void linear_body(const SmallEntry &e, int bx) {
    const int warp = (bx * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= e.N * e.K) return;
    const int n = warp / e.K, j = warp % e.K;
    const __nv_bfloat16 *wr = static_cast<const __nv_bfloat16 *>(e.w) + (size_t)j * e.ld;
    const float *vr = static_cast<const float *>(e.x) + (size_t)n * e.C;
    float s = 0.f;
    for (int c = lane * 8; c < e.C; c += 256) {
        const uint4 wv = __ldg(reinterpret_cast<const uint4 *>(wr + c));
        const float4 x0 = *reinterpret_cast<const float4 *>(vr + c), x1 = *reinterpret_cast<const float4 *>(vr + c + 4);
        const float2 a = bf2f(wv.x), b = bf2f(wv.y), cc = bf2f(wv.z), d = bf2f(wv.w);
        s = fmaf(a.x, x0.x, s); s = fmaf(a.y, x0.y, s); s = fmaf(b.x, x0.z, s); s = fmaf(b.y, x0.w, s);
        s = fmaf(cc.x, x1.x, s); s = fmaf(cc.y, x1.y, s); s = fmaf(d.x, x1.z, s); s = fmaf(d.y, x1.w, s);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) static_cast<float *>(e.y)[(size_t)n * e.K + j] = apply_act(s + e.bias[j], e.act);
}

// Patch matrix of a convolution with 3 input channels (the stems): row m = output pixel, column
// kk = (r * k + s) * 3 + c holds x[n][ho*st + r - p][wo*st + s - p][c] (0 outside the image and for the
// padding columns kk >= k*k*3).  With it the stem is a GEMM on the tensor cores like every other layer.
// A block owns one output row of one image: it stages the k input rows in shared memory (16-byte
// loads), then every thread assembles 8 consecutive columns of a patch row and writes them with one
// 16-byte store, consecutive threads to consecutive addresses.
constexpr int IM2COL_MAX_W = 1024;  // widest input row the shared-memory staging holds (7 rows x 3 channels)
template <int K, int ST>
__device__ __forceinline__ void im2col_body(const SmallEntry &e, int bx) {
    constexpr int P = (K - 1) / 2, KK = K * K * 3;
    constexpr int ROWLEN = (IM2COL_MAX_W + 2 * P) * 3;  // a staged row with P zero pixels on either side
    // rows[r] = input row ho*ST + r - P, shifted right by P pixels and zero outside the image, so that the
    // patch element (r, s, c) of output column wo is rows[r][(wo*ST + s) * 3 + c] without any bounds test
    __shared__ __align__(16) unsigned short rows[K][ROWLEN];
    if (bx >= e.N * e.Ho) return;
    const int n = bx / e.Ho, ho = bx % e.Ho;
    const int rowlen = e.W * 3;  // elements; a multiple of 8 (checked by the host)
    const unsigned short *ximg = static_cast<const unsigned short *>(e.x) + (size_t)n * e.H * rowlen;
    const int padded = rowlen + 2 * P * 3;
#pragma unroll
    for (int r = 0; r < K; r++) {
        const int hi = ho * ST + r - P;
        const bool rok = hi >= 0 && hi < e.H;
        const unsigned short *src = ximg + (size_t)(rok ? hi : 0) * rowlen;
        for (int i = threadIdx.x; i < padded; i += blockDim.x) {
            const int j = i - P * 3;
            rows[r][i] = (rok && j >= 0 && j < rowlen) ? __ldg(src + j) : (unsigned short)0;
        }
    }
    __syncthreads();
    // a thread keeps one group of 8 patch columns (their 8 offsets into `rows` stay in registers) and walks
    // the output columns; neighbouring threads write neighbouring 16-byte pieces
    const int gv = e.KKp >> 3;
    const int lanes_w = blockDim.x / gv;  // output columns in flight per block
    const int g = threadIdx.x % gv, wl = threadIdx.x / gv;
    if (wl >= lanes_w) return;
    int off[8];
#pragma unroll
    for (int q = 0; q < 8; q++) {
        const int kk = g * 8 + q;
        const int c = kk % 3, rs = kk / 3, s = rs % K, r = rs / K;
        off[q] = kk < KK ? r * ROWLEN + s * 3 + c : -1;  // -1: padding column, always zero
    }
    uint4 *y = static_cast<uint4 *>(e.y) + ((size_t)n * e.Ho + ho) * e.Wo * gv;
    const unsigned short *base = &rows[0][0];
    for (int wo = wl; wo < e.Wo; wo += lanes_w) {
        const unsigned short *p = base + wo * ST * 3;
        unsigned short v[8];
#pragma unroll
        for (int q = 0; q < 8; q++) v[q] = off[q] >= 0 ? p[off[q]] : (unsigned short)0;
        y[wo * gv + g] = make_uint4(v[0] | ((uint32_t)v[1] << 16), v[2] | ((uint32_t)v[3] << 16), v[4] | ((uint32_t)v[5] << 16), v[6] | ((uint32_t)v[7] << 16));
    }
}

// 3-channel image -> [N][Ho][Wo][8] with the image at (k, k) and zeros elsewhere (margins and channels 3..7):
// the input of the window-view stem.  A thread writes one padded pixel (16 bytes).
__device__ __forceinline__ void pad8_body(const SmallEntry &e, int bx, int nbx) {
    const int total = e.N * e.Ho * e.Wo;
    const unsigned short *x = static_cast<const unsigned short *>(e.x);
    uint4 *y = static_cast<uint4 *>(e.y);
    for (int i = bx * blockDim.x + threadIdx.x; i < total; i += nbx * blockDim.x) {
        const int wp = i % e.Wo, hp = (i / e.Wo) % e.Ho, n = i / (e.Wo * e.Ho);
        const int h = hp - e.k, w = wp - e.k;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (h >= 0 && h < e.H && w >= 0 && w < e.W) {
            const unsigned short *p = x + (((size_t)n * e.H + h) * e.W + w) * 3;
            v.x = __ldg(p) | ((uint32_t)__ldg(p + 1) << 16);
            v.y = __ldg(p + 2);
        }
        y[i] = v;
    }
}

template <int KIND, int K, int ST> __device__ __forceinline__ void small_body(const SmallEntry &e, int bx, int nbx) {
    if constexpr (KIND == OP_MAXPOOL) maxpool_body(e, bx, nbx);
    else if constexpr (KIND == OP_GAP) gap_body(e, bx);
    else if constexpr (KIND == OP_LINEAR) linear_body(e, bx);
    else if constexpr (KIND == OP_SCALE) scale_body(e, bx, nbx);
    else if constexpr (KIND == OP_PAD8) pad8_body(e, bx, nbx);
    else im2col_body<K, ST>(e, bx);
}
template <int KIND, int K, int ST> __global__ void __launch_bounds__(256) small_single_kernel(const SmallEntry e) {
    small_body<KIND, K, ST>(e, blockIdx.x, gridDim.x);
}
template <int KIND, int K, int ST> __global__ void __launch_bounds__(256) small_group_kernel(const SmallEntry *__restrict__ tbl) {
    __shared__ SmallEntry e;
    if (threadIdx.x < 8) reinterpret_cast<uint4 *>(&e)[threadIdx.x] = __ldg(reinterpret_cast<const uint4 *>(tbl + blockIdx.y) + threadIdx.x);
    __syncthreads();
    small_body<KIND, K, ST>(e, blockIdx.x, gridDim.x);
}

// Linear layer for several members that use the SAME stored layer (same weights, outputs, batch): a warp
// owns one (image, output) pair for up to LIN_CHUNK members, loads every 16-byte piece of the weight row
// once and uses it for each member whose (sliced) input is that long.  Per member the arithmetic and its
// order are those of linear_body.
constexpr int LIN_CHUNK = 8;
__global__ void __launch_bounds__(256) linear_multi_kernel(const SmallEntry *__restrict__ tbl, int n_members) {
    __shared__ SmallEntry es[LIN_CHUNK];
    const int m0 = blockIdx.y * LIN_CHUNK, nm = min(LIN_CHUNK, n_members - m0);
    if ((int)threadIdx.x < nm * 8) reinterpret_cast<uint4 *>(es)[threadIdx.x] = __ldg(reinterpret_cast<const uint4 *>(tbl + m0) + threadIdx.x);
    __syncthreads();
    const SmallEntry &e0 = es[0];
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (warp >= e0.N * e0.K) return;
    const int n = warp / e0.K, j = warp % e0.K;
    const __nv_bfloat16 *wr = static_cast<const __nv_bfloat16 *>(e0.w) + (size_t)j * e0.ld;
    int Cmax = 0;
    for (int m = 0; m < nm; m++) Cmax = max(Cmax, es[m].C);
    float s[LIN_CHUNK];
#pragma unroll
    for (int m = 0; m < LIN_CHUNK; m++) s[m] = 0.f;
    for (int c = lane * 8; c < Cmax; c += 256) {
        const uint4 wv = __ldg(reinterpret_cast<const uint4 *>(wr + c));
        const float2 a = bf2f(wv.x), b = bf2f(wv.y), cc = bf2f(wv.z), d = bf2f(wv.w);
#pragma unroll
        for (int m = 0; m < LIN_CHUNK; m++) {
            if (m < nm && c < es[m].C) {
                const float *vr = static_cast<const float *>(es[m].x) + (size_t)n * es[m].C + c;
                const float4 x0 = *reinterpret_cast<const float4 *>(vr), x1 = *reinterpret_cast<const float4 *>(vr + 4);
                float t = s[m];
                t = fmaf(a.x, x0.x, t); t = fmaf(a.y, x0.y, t); t = fmaf(b.x, x0.z, t); t = fmaf(b.y, x0.w, t);
                t = fmaf(cc.x, x1.x, t); t = fmaf(cc.y, x1.y, t); t = fmaf(d.x, x1.z, t); t = fmaf(d.y, x1.w, t);
                s[m] = t;
            }
        }
    }
    const float bias = e0.bias[j];
#pragma unroll
    for (int m = 0; m < LIN_CHUNK; m++) {
        float t = s[m];
#pragma unroll
        for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0 && m < nm) static_cast<float *>(es[m].y)[(size_t)n * e0.K + j] = apply_act(t + bias, e0.act);
    }
}

bool small_supported(int kind, const SmallEntry &e) {
    auto al = [](const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; };
    if (!al(e.x) || !al(e.y)) return false;
    switch (kind) {
    case OP_MAXPOOL: return e.C % 8 == 0 && (long long)e.N * e.Ho * e.Wo * (e.C / 8) < (1ll << 31);
    case OP_GAP: return e.C % 8 == 0;
    case OP_SCALE: return e.C % 8 == 0 && al(e.w) && (long long)e.N * e.H * e.W * (e.C / 8) < (1ll << 31);
    case OP_SE_GATE: return e.w2 != nullptr;
    case OP_PAD8: return (long long)e.N * e.Ho * e.Wo < (1ll << 31);
    case OP_LINEAR: return e.C % 8 == 0 && e.ld % 8 == 0 && al(e.w);
    case OP_IM2COL: return (e.k == 3 || e.k == 7) && (e.stride == 1 || e.stride == 2) && e.KKp % 8 == 0 && e.KKp >= e.k * e.k * 3 &&
                           e.W % 8 == 0 && e.W <= IM2COL_MAX_W && (long long)e.N * e.Ho < (1ll << 31) && (long long)e.Wo * (e.KKp / 8) < (1ll << 31);
    default: return false;
    }
}

// blocks along x that one member needs
static long long small_blocks(int kind, const SmallEntry &e) {
    switch (kind) {
    case OP_MAXPOOL: return ((long long)e.N * e.Ho * e.Wo * (e.C / 8) + 255) / 256;
    case OP_GAP: return ((long long)e.N * (e.C / 8) * 32 + 255) / 256;
    case OP_SCALE: return ((long long)e.N * e.H * e.W * (e.C / 8) + 255) / 256;
    case OP_PAD8: return ((long long)e.N * e.Ho * e.Wo + 255) / 256;
    case OP_LINEAR: return ((long long)e.N * e.K * 32 + 255) / 256;
    default: return (long long)e.N * e.Ho;  // patch matrix: one block per output row
    }
}

template <int KIND, int K, int ST>
static cudaError_t launch_small_t(const SmallEntry *h, const SmallEntry *d, int n, unsigned bx, cudaStream_t st) {
    if (d) small_group_kernel<KIND, K, ST><<<dim3(bx, (unsigned)n), 256, 0, st>>>(d);
    else small_single_kernel<KIND, K, ST><<<bx, 256, 0, st>>>(*h);
    return cudaGetLastError();
}

cudaError_t launch_small(int kind, const SmallEntry *h, const SmallEntry *d, int n, cudaStream_t st) {
    if (n <= 0) return cudaSuccess;
    if ((!d && n != 1) || n > 65535) return cudaErrorInvalidValue;
    long long blocks = 1;
    for (int i = 0; i < n; i++) blocks = std::max(blocks, small_blocks(kind, h[i]));
    // the grid-stride kernels (max pool, SE scale) need not cover every element with a block of their own
    if (kind == OP_MAXPOOL || kind == OP_SCALE || kind == OP_PAD8) blocks = std::min<long long>(blocks, 148 * 16);
    const unsigned bx = (unsigned)blocks;
    switch (kind) {
    case OP_MAXPOOL: return launch_small_t<OP_MAXPOOL, 0, 0>(h, d, n, bx, st);
    case OP_GAP: return launch_small_t<OP_GAP, 0, 0>(h, d, n, bx, st);
    case OP_SCALE: return launch_small_t<OP_SCALE, 0, 0>(h, d, n, bx, st);
    case OP_PAD8: return launch_small_t<OP_PAD8, 0, 0>(h, d, n, bx, st);
    case OP_SE_GATE: {
        if (!d) return cudaErrorInvalidValue;
        int nimg = 0, fl = 0;
        for (int i = 0; i < n; i++) { nimg = std::max(nimg, h[i].N); fl = std::max(fl, h[i].C + h[i].K); }
        se_gate_group_kernel<<<dim3((unsigned)nimg * SE_SPLIT, (unsigned)n), SE_THREADS, (size_t)fl * sizeof(float), st>>>(d);
        return cudaGetLastError();
    }
    case OP_LINEAR: {
        bool same = d != nullptr && n > 1;
        for (int i = 1; i < n && same; i++)
            same = h[i].w == h[0].w && h[i].K == h[0].K && h[i].ld == h[0].ld && h[i].N == h[0].N && h[i].act == h[0].act && h[i].bias == h[0].bias;
        if (same) {  // one stored layer for all members: share its weight rows
            linear_multi_kernel<<<dim3(bx, (unsigned)((n + LIN_CHUNK - 1) / LIN_CHUNK)), 256, 0, st>>>(d, n);
            return cudaGetLastError();
        }
        return launch_small_t<OP_LINEAR, 0, 0>(h, d, n, bx, st);
    }
    case OP_IM2COL: {
        const int key = h[0].k * 10 + h[0].stride;
        for (int i = 1; i < n; i++)
            if (h[i].k * 10 + h[i].stride != key) return cudaErrorInvalidValue;
        if (key == 72) return launch_small_t<OP_IM2COL, 7, 2>(h, d, n, bx, st);
        if (key == 71) return launch_small_t<OP_IM2COL, 7, 1>(h, d, n, bx, st);
        if (key == 32) return launch_small_t<OP_IM2COL, 3, 2>(h, d, n, bx, st);
        if (key == 31) return launch_small_t<OP_IM2COL, 3, 1>(h, d, n, bx, st);
        return cudaErrorInvalidValue;
    }
    default: return cudaErrorInvalidValue;
    }
}

__global__ void stem_gemm_weights_kernel(const __nv_bfloat16 *__restrict__ src, __nv_bfloat16 *__restrict__ dst, int K, int KK, int KKp) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= K * KKp) return;
    const int f = i / KKp, kk = i % KKp;
    dst[i] = kk < KK ? src[(size_t)f * KK + kk] : __float2bfloat16_rn(0.f);
}
__global__ void stem_window_weights_kernel(const __nv_bfloat16 *__restrict__ src, __nv_bfloat16 *__restrict__ dst, int K, int k) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;  // dst index [f][r][px][c8]
    if (i >= K * k * 64) return;
    const int c = i % 8, px = (i / 8) % 8, r = (i / 64) % k, f = i / (64 * k);
    dst[i] = (px < k && c < 3) ? src[(((size_t)f * k + r) * k + px) * 3 + c] : __float2bfloat16_rn(0.f);
}
cudaError_t launch_stem_window_weights(const void *src, void *dst, int K, int k, cudaStream_t st) {
    const int total = K * k * 64;
    stem_window_weights_kernel<<<(total + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(src), static_cast<__nv_bfloat16 *>(dst), K, k);
    return cudaGetLastError();
}
cudaError_t launch_stem_gemm_weights(const void *src, void *dst, int K, int KK, int KKp, cudaStream_t st) {
    const int total = K * KKp;
    stem_gemm_weights_kernel<<<(total + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16 *>(src), static_cast<__nv_bfloat16 *>(dst), K, KK, KKp);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Load-time kernels
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void relayout_conv_kernel(const float *__restrict__ src, T *__restrict__ dst, int K, int C, int Cp, int R, int S) {
    size_t total = (size_t)K * Cp * R * S;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        // i indexes dst [K][R][S][Cp]; channels C..Cp-1 of a row are zero
        int c = (int)(i % Cp);
        size_t q = i / Cp;
        int s = (int)(q % S), r = (int)((q / S) % R), f = (int)(q / ((size_t)S * R));
        dst[i] = from_f<T>(c < C ? src[(((size_t)f * C + c) * R + r) * S + s] : 0.f);
    }
}
cudaError_t launch_relayout_conv(const float *src, void *dst, int K, int C, int Cp, int R, int S, int bf16, cudaStream_t st) {
    size_t total = (size_t)K * Cp * R * S;
    int blocks = (int)std::min<size_t>((total + 255) / 256, 148 * 32);
    if (bf16) relayout_conv_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(src, static_cast<__nv_bfloat16 *>(dst), K, C, Cp, R, S);
    else relayout_conv_kernel<float><<<blocks, 256, 0, st>>>(src, static_cast<float *>(dst), K, C, Cp, R, S);
    return cudaGetLastError();
}

template <typename T>
__global__ void relayout_dw_kernel(const float *__restrict__ src, T *__restrict__ dst, int K, int R, int S) {
    size_t total = (size_t)K * R * S;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        // dst [R][S][K], src [K][1][R][S]
        int f = (int)(i % K);
        size_t q = i / K;
        dst[i] = from_f<T>(src[(size_t)f * R * S + q]);
    }
}
cudaError_t launch_relayout_dw(const float *src, void *dst, int K, int R, int S, int bf16, cudaStream_t st) {
    size_t total = (size_t)K * R * S;
    int blocks = (int)std::min<size_t>((total + 255) / 256, 148 * 32);
    if (bf16) relayout_dw_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(src, static_cast<__nv_bfloat16 *>(dst), K, R, S);
    else relayout_dw_kernel<float><<<blocks, 256, 0, st>>>(src, static_cast<float *>(dst), K, R, S);
    return cudaGetLastError();
}

template <typename T> __global__ void convert_kernel(const float *__restrict__ src, T *__restrict__ dst, size_t n) {
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = from_f<T>(src[i]);
}
cudaError_t launch_convert(const float *src, void *dst, size_t n, int bf16, cudaStream_t st) {
    if (!n) return cudaSuccess;
    int blocks = (int)std::min<size_t>((n + 255) / 256, 148 * 32);
    if (bf16) convert_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(src, static_cast<__nv_bfloat16 *>(dst), n);
    else convert_kernel<float><<<blocks, 256, 0, st>>>(src, static_cast<float *>(dst), n);
    return cudaGetLastError();
}

// Holds a stream for about `us` microseconds (bounded: the loop ends on its own).
__global__ void delay_kernel(unsigned us) {
    unsigned long long t0, t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t0));
    do {
        __nanosleep(2000);
        asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    } while (t - t0 < (unsigned long long)us * 1000ull);
}
cudaError_t launch_delay(unsigned microseconds, cudaStream_t st) {
    delay_kernel<<<1, 1, 0, st>>>(microseconds > 50000u ? 50000u : microseconds);
    return cudaGetLastError();
}

// Measurement aid: fp32 FMA rate of the CUDA cores.  Every thread runs `iters` rounds of 16 independent
// fused multiply-adds on registers (no memory traffic, no dependence between the 16 chains inside a round);
// the sum is stored so that the loop cannot be removed.
__global__ void __launch_bounds__(256) fma_rate_kernel(float *out, int iters, float a, float b) {
    float x[16];
#pragma unroll
    for (int j = 0; j < 16; j++) x[j] = (float)(threadIdx.x + j) * 1e-3f;
    for (int i = 0; i < iters; i++) {
#pragma unroll
        for (int j = 0; j < 16; j++) x[j] = fmaf(x[j], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < 16; j++) s += x[j];
    out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}
cudaError_t measure_fma_rate(double *tflops, cudaStream_t st) {
    const int blocks = 148 * 8, threads = 256, iters = 4096;
    float *out = nullptr;
    cudaError_t e = cudaMalloc((void **)&out, (size_t)blocks * threads * sizeof(float));
    if (e != cudaSuccess) return e;
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    float best = 0.f;
    for (int rep = 0; rep < 5 && e == cudaSuccess; rep++) {
        cudaEventRecord(e0, st);
        fma_rate_kernel<<<blocks, threads, 0, st>>>(out, iters, 0.999f, 1e-3f);
        cudaEventRecord(e1, st);
        e = cudaEventSynchronize(e1);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e == cudaSuccess && rep > 0 && (best == 0.f || ms < best)) best = ms;  // (first round: warm-up)
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(out);
    if (e != cudaSuccess) return e;
    *tflops = best > 0.f ? 2.0 * blocks * threads * 16.0 * iters / (best * 1e-3) / 1e12 : 0.0;
    return cudaSuccess;
}

// Batch-norm folding: scale = gamma / sqrt(var + 1e-5), shift = beta - mean * scale (+ bias).
__global__ void fold_bn_kernel(const float *gamma, const float *beta, const float *mean, const float *var,
                               const float *bias, float *scale, float *shift, int K) {
    int f = blockIdx.x * blockDim.x + threadIdx.x;
    if (f >= K) return;
    float sc = 1.f, sh = 0.f;
    if (gamma) {
        sc = gamma[f] / sqrtf(var[f] + 1e-5f);
        sh = beta[f] - mean[f] * sc;
    }
    if (bias) sh += bias[f];
    scale[f] = sc;
    shift[f] = sh;
}
cudaError_t launch_fold_bn(const float *gamma, const float *beta, const float *mean, const float *var,
                           const float *bias, float *scale, float *shift, int K, cudaStream_t st) {
    fold_bn_kernel<<<(K + 127) / 128, 128, 0, st>>>(gamma, beta, mean, var, bias, scale, shift, K);
    return cudaGetLastError();
}

}  // namespace sgs
