// Internal declarations shared by the translation units of libsgs (host side).
#pragma once

#include <cuda_runtime.h>
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdint>
#include <cstddef>
#include <string>
#include <unordered_map>
#include <vector>
#include <memory>

#include "sgs.h"

namespace sgs {

enum LayerKind { KIND_CONV = 0, KIND_DW = 1, KIND_LINEAR = 2 };
enum Act { ACT_NONE = 0, ACT_RELU = 1, ACT_HSWISH = 2 };

// One stored SuperNet layer on the device.
//   conv      w = [K][R][S][C]   (filters outermost, channels innermost)
//   depthwise w = [R][S][K]      (channels innermost so NHWC threads read contiguous weights)
//   linear    w = [K][C]
// element type = the handle's compute dtype.  scale/shift hold the folded batch norm
// (scale = gamma / sqrt(var + eps), shift = beta - mean * scale), or scale = 1, shift = bias.
struct StoredLayer {
    int kind = 0, K = 0, C = 0, R = 0, S = 0;
    bool has_bn = false, has_bias = false;
    void *w = nullptr;
    float *scale = nullptr, *shift = nullptr;
    size_t w_bytes = 0;
    std::string name;
};

struct Slice {  // the part of a stored layer a SubNet uses
    int active = 0, K = 0, C = 0, k = 0;
};

// Arguments of one convolution launch (regular or depthwise), any implementation.
struct ConvArgs {
    const void *x = nullptr;   // [N][H][W][C]
    const void *w = nullptr;   // stored layer weights
    const float *scale = nullptr, *shift = nullptr;
    const void *res = nullptr; // optional residual [N][Ho][Wo][K]
    void *y = nullptr;         // [N][Ho][Wo][K]
    int N = 0, H = 0, W = 0, C = 0, Ho = 0, Wo = 0, K = 0;
    int Kmax = 0, Cmax = 0, R = 0;  // stored dims (square kernels)
    int k = 1, stride = 1, act = 0;
    // SubGraph cache box of this layer: weight tiles with filter < cacheK and channel < cacheC are
    // loaded with an evict-last L2 policy; weight_policy 0 = none, 1 = use the box, 2 = all evict-first
    int cacheK = 0, cacheC = 0, weight_policy = 0;
    // when set, the three values above are read by the kernel from device memory instead:
    // cache_tbl[0] = weight_policy, cache_tbl[1 + 2*layer] = cacheK, cache_tbl[2 + 2*layer] = cacheC
    // (lets a captured graph follow cache updates without being re-captured)
    const int *cache_tbl = nullptr;
    int layer = 0;
    int throughput = 0;  // 1: pick tiles for aggregate throughput (many launches in flight), 0: for the latency of this launch
    // split-K scratch of the tensor-core kernel: fp32 partial tiles [splits][M][K]
    float *ws = nullptr;
    size_t ws_elems = 0;
};

enum OpType { OP_CONV, OP_DW, OP_MAXPOOL, OP_GAP, OP_SE_GATE, OP_SCALE, OP_LINEAR };

struct TcConvPlan;  // tensor-core launch description (sgs_conv_tc.cu)

struct Op {
    OpType type = OP_CONV;
    int layer = -1, layer2 = -1;
    int in = -1, out = -1, res = -1;  // activation buffer ids; -1 input tensor / none
    int vin = -1, vout = -1;          // vector buffer ids (fp32)
    ConvArgs conv;
    int N = 0, H = 0, W = 0, C = 0, K = 0, act = 0;
    int impl = 0;                     // 0 plain CUDA-core kernel, 1 tensor-core kernel
    double alg_bytes = 0, flops = 0;  // algorithmic traffic (weights + input + output + residual) and useful FLOPs
    std::shared_ptr<TcConvPlan> tc;
};

struct Plan {
    std::vector<Op> ops;
    int batch = 0, res = 0;
    double flops = 0, weight_bytes = 0, act_bytes = 0;
    std::vector<Slice> slices;
    std::vector<int> enc;  // (K, C, k) per stored layer: the SubNet's vector encoding
    size_t act_elems = 0;  // elements each activation buffer must hold
    cudaGraphExec_t graph = nullptr;  // ops [1, n-1): everything that touches only internal buffers
    std::vector<cudaEvent_t> prof_ev;      // start / end event of every op (profiling)
    int launches = 0;
    bool prepared = false;  // implementations chosen and buffer addresses fixed
    int slot = 0;           // which set of workspaces the plan's buffer addresses refer to
    int throughput = 0;     // tile choice of the plan's convolutions (see ConvArgs::throughput)
};

// ---- launchers implemented in sgs_kernels.cu (T = float or __nv_bfloat16) -------------------
template <typename T> cudaError_t launch_conv_plain(const ConvArgs &a, cudaStream_t st);
template <typename T> cudaError_t launch_dw(const ConvArgs &a, cudaStream_t st);
template <typename T> cudaError_t launch_maxpool3s2(const T *x, T *y, int N, int H, int W, int C, cudaStream_t st);
template <typename T> cudaError_t launch_gap(const T *x, float *g, int N, int HW, int C, cudaStream_t st);
template <typename T>
cudaError_t launch_se_gate(const float *g, const T *w1, const float *b1, const T *w2, const float *b2, float *gate,
                           int N, int mid, int sq, int w1_ld, int w2_ld, cudaStream_t st);
template <typename T> cudaError_t launch_scale(const T *x, const float *gate, T *y, int N, int HW, int C, cudaStream_t st);
template <typename T>
cudaError_t launch_linear(const float *v, const T *w, const float *bias, float *y, int N, int C, int K, int ld, int act,
                          cudaStream_t st);
cudaError_t launch_relayout_conv(const float *src, void *dst, int K, int C, int R, int S, int bf16, cudaStream_t st);
cudaError_t launch_relayout_dw(const float *src, void *dst, int K, int R, int S, int bf16, cudaStream_t st);
cudaError_t launch_convert(const float *src, void *dst, size_t n, int bf16, cudaStream_t st);
cudaError_t launch_delay(unsigned microseconds, cudaStream_t st);  // one thread sleeping for a bounded time
cudaError_t launch_fold_bn(const float *gamma, const float *beta, const float *mean, const float *var,
                           const float *bias, float *scale, float *shift, int K, cudaStream_t st);

// ---- tensor-core convolution (sgs_conv_tc.cu) -----------------------------------------------
// Returns nullptr when the shape is not handled by the tensor-core kernel (caller falls back).
std::shared_ptr<TcConvPlan> tc_conv_prepare(const ConvArgs &a, int device, std::string *why);
size_t tc_conv_ws_elems(const TcConvPlan &p);      // fp32 elements of split-K scratch the plan wants (0 = none)
cudaError_t tc_conv_launch(const TcConvPlan &p, const ConvArgs &a, cudaStream_t st, int *launches);
cudaError_t tc_conv_init(int device);  // one-time device set-up; call outside stream capture
bool tc_available();
int tc_conv_status();  // nonzero once any tensor-core kernel reported a bounded wait running out

}  // namespace sgs
