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
    int Cp = 0;  // conv: channels per (filter, tap) row as stored (>= C; the rest of a row is zero), else C
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
    int Kmax = 0, Cmax = 0, R = 0;  // stored dims (square kernels); Cmax = channels per stored (filter, tap) row
    // Channel pitch (elements per pixel) of x and of y / res when a pixel holds more than the sliced channels:
    // 0 = dense (C resp. K).  Padded tensors keep their pixels at a multiple of 16 channels (32 bytes) and the
    // channels beyond the slice are ZERO: the copy unit moves rows whose ends fall inside a 32-byte sector at a
    // third of the rate (measured on sm_100a), and C, K are multiples of 8 only.  Tensor-core kernels of grouped
    // launches only; they write the zeros of y.
    int ldx = 0, ldy = 0;
    int i8 = 0;  // 8-bit operands (x, w, res, y one byte per element; sgs_conv2d_sliced_i8): tensor-core kernel only
    const int *q_mult = nullptr, *q_shift = nullptr, *q_bias = nullptr;  // ... with the integer epilogue of TcParams
    int q_zy = 0, q_zr = 0, q_res_mult = 0, q_res_shift = 0, q_flags = 0;
    int k = 1, stride = 1, act = 0;
    // Window view of a 3-channel stem (grouped launches): x is the input padded to 8 channels with a zero
    // margin, [N][H][W][8] with H, W the PADDED sizes; an "input channel" chunk is the 8-pixel x 8-channel
    // window that starts at output column wo * stride (64 contiguous elements), the taps are the k filter ROWS
    // only (C = Cmax = 64, R = 1), and the weights are [Kmax][k][64] with zeros where the window has no tap.
    int win = 0;
    // SubGraph cache box of this layer: weight tiles with filter < cacheK and channel < cacheC are
    // loaded with an evict-last L2 policy; weight_policy 0 = none, 1 = use the box, 2 = all evict-first
    int cacheK = 0, cacheC = 0, weight_policy = 0;
    // when set, the three values above are read by the kernel from device memory instead:
    // cache_tbl[0] = weight_policy, cache_tbl[1 + 2*layer] = cacheK, cache_tbl[2 + 2*layer] = cacheC
    // (lets a captured graph follow cache updates without being re-captured)
    const int *cache_tbl = nullptr;
    int layer = 0;
    int throughput = 0;  // 0: tiles for the latency of this launch; 1: for aggregate throughput (many launches in flight);
                         // 2: member of a grouped launch (128-filter tiles, reduction never split)
    // split-K scratch of the tensor-core kernel: fp32 partial tiles [splits][M][K]
    float *ws = nullptr;
    size_t ws_elems = 0;
};

// ---- persistent SubNet kernel (sgs_subnet_kernel.cu) ------------------------------------------
// One launch serves a whole stream of one-image queries of the MobileNetV3-shaped family: every block (one per
// SM) takes the next unserved query and runs ALL layers of that query's SubNet by itself, from the image to the
// logits, out of a private scratch area; the layers are the records of an op list the host wrote for the config.
enum PqType { PQ_STEM = 0, PQ_PW = 1, PQ_DW = 2, PQ_GAP = 3, PQ_SE_GATE = 4, PQ_SCALE = 5, PQ_LINEAR = 6 };
struct alignas(16) PqOp {
    int type;
    int in, out, res;     // activation buffers of the block's scratch area (-1: the query's image / none)
    int vin, vout;        // fp32 vectors held in shared memory (vout -1: the query's logits)
    int H, W, C, K;       // input map, sliced input channels, sliced filters (depthwise: C == K channels)
    int Ho, Wo, k, stride;
    int act, R, Kmax, ld; // stored kernel size, stored filter count (depthwise pitch), row pitch of w in elements
    int ld2, cache_rows;  // SE gate: pitch of the second FC; pointwise: channels (ld2) and filters (cache_rows) of this layer held in the block's weight buffer
    const void *w;        // stored weights of the layer (sliced by prefix / centre crop inside the kernel)
    const float *scale, *shift;  // folded batch norm, or shift = bias
    const void *w2;       // SE gate: second FC
    const float *bias2;
    long long cache_off;  // pointwise: byte offset of this layer's rows in the block's weight buffer (-1: not held)
};
static_assert(sizeof(PqOp) == 128, "record size");
struct alignas(16) PqQuery {
    const void *x;   // [res][res][3] bf16
    float *logits;   // [classes]
    int op_begin, op_count;
    int pad_[2];
};
static_assert(sizeof(PqQuery) == 32, "record size");
// One layer's box in the weight buffer every block keeps in shared memory for the whole launch (Section 4.2,
// Persistent Buffer): the first `rows` filters (a multiple of 16) x the first C channels of a pointwise layer, stored as
// `chunks` tiles of rows x 128 bytes (64 channels each, zero beyond C) in the layout the tensor core reads.
struct alignas(16) PqHeld {
    const void *w;
    int ld, rows, chunks, C;
    unsigned off;
    int pad_;
};
static_assert(sizeof(PqHeld) == 32, "record size");
struct PqParams {
    const PqHeld *held;      // n_held boxes, held_bytes in total (0: no weight buffer)
    int n_held;
    unsigned held_bytes;
    const PqQuery *queries;
    const PqOp *ops;
    int n_queries;
    int *counter;            // next unserved query (zeroed before the launch)
    unsigned char *scratch;  // blocks x slot_bytes: four activation buffers of act_bytes per block
    size_t slot_bytes, act_bytes;
    int *status;             // device status word: nonzero after a bounded wait ran out
};

enum OpType { OP_CONV, OP_DW, OP_MAXPOOL, OP_GAP, OP_SE_GATE, OP_SCALE, OP_LINEAR, OP_IM2COL, OP_PAD8 };

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
    int rank = -1;                    // position of this op in the largest SubNet's op list (wave merging)
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
    bool padded = false;    // activation tensors hold 16-channel-padded pixels (ConvArgs::ldx, ldy)
    int slot = 0;           // which set of workspaces the plan's buffer addresses refer to
    int throughput = 0;     // tile choice of the plan's convolutions (see ConvArgs::throughput)
    std::vector<PqOp> pq;  // the plan as an op list of the persistent SubNet kernel (built on first use)
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
cudaError_t launch_relayout_conv(const float *src, void *dst, int K, int C, int Cp, int R, int S, int bf16, cudaStream_t st);  // dst [K][R][S][Cp], zero beyond C
cudaError_t launch_relayout_dw(const float *src, void *dst, int K, int R, int S, int bf16, cudaStream_t st);
cudaError_t launch_convert(const float *src, void *dst, size_t n, int bf16, cudaStream_t st);
cudaError_t measure_fma_rate(double *tflops, cudaStream_t st);  // fp32 FMA rate of the CUDA cores (2 FLOP per FMA), best of 4 timed launches
cudaError_t launch_delay(unsigned microseconds, cudaStream_t st);  // one thread sleeping for a bounded time
cudaError_t launch_fold_bn(const float *gamma, const float *beta, const float *mean, const float *var,
                           const float *bias, float *scale, float *shift, int K, cudaStream_t st);

// ---- bf16 kernels that take their arguments as a record, alone or as one member of a grouped launch
// (one launch serves many queries in flight: blockIdx.y selects the member's record in a device table)
struct alignas(16) SmallEntry {
    const void *x;       // input tensor / vector
    void *y;             // output tensor / vector
    const void *w;       // linear: weights [K][ld] bf16
    const float *bias;   // linear: bias [K]
    int N, H, W, C;      // input dims (linear: C inputs; gap: H*W pixels)
    int K, ld, act;      // linear: outputs, row pitch of w, activation
    int Ho, Wo;          // output dims (max pool, patch matrix)
    int k, stride, KKp;  // patch matrix: kernel size, stride, padded row length
    const void *w2;      // SE gate: second FC weights [C][ld2] bf16 (first FC: w [K][ld], K = squeeze width)
    const float *bias2;  // SE gate: second FC bias [C]
    int ld2;
    int pad_[7];
};
static_assert(sizeof(SmallEntry) == 128, "record size");
// kind: OP_MAXPOOL (3x3 stride 2, C % 8 == 0), OP_GAP (C % 8 == 0), OP_LINEAR (C % 8 == 0, ld % 8 == 0),
// OP_SCALE (SE scale, gate vector in w; C % 8 == 0), OP_SE_GATE (grouped launches only),
// OP_IM2COL (3 input channels; k in {3, 7}; stride in {1, 2}), OP_PAD8 (3-channel image -> 8 channels with a
// zero margin: k = margin left / top, Ho x Wo = padded size).  `h` is the host image of the `n` records
// at device address `d` (it sizes the grid); with d == nullptr, n must be 1 and the record is passed by value.
bool small_supported(int kind, const SmallEntry &e);
cudaError_t launch_small(int kind, const SmallEntry *h, const SmallEntry *d, int n, cudaStream_t st);
// Depthwise convolution of several members in one launch: h_tbl / d_tbl = host image and device copy of
// `members` ConvArgs records, DW_ENTRY_BYTES apart.  All members must share stride, activation and image dims
// and take the vectorised bf16 kernels (kernel sizes 3, 5, 7 may be mixed); otherwise cudaErrorNotSupported and
// nothing is launched.
constexpr int DW_ENTRY_BYTES = 256;
void dw_set_walk(int min_million_elements);  // tuning aid: stride-1 depthwise launches of at least this many million outputs take the walking kernel (0 = never)
cudaError_t launch_dw_group(const char *h_tbl, const char *d_tbl, int members, cudaStream_t st);
// Stem weights for the window view: dst[f][r][px * 8 + c] = src[f][r][px][c] (px < k, c < 3), else 0; dst [K][k][64].
cudaError_t launch_stem_window_weights(const void *src, void *dst, int K, int k, cudaStream_t st);
// Stem weights as a GEMM operand: dst[f][kk] = src[f][kk] for kk < KK (the stored [K][R][R][3] row), 0 up to KKp.
cudaError_t launch_stem_gemm_weights(const void *src, void *dst, int K, int KK, int KKp, cudaStream_t st);

// ---- tensor-core convolution (sgs_conv_tc.cu) -----------------------------------------------
// Returns nullptr when the shape is not handled by the tensor-core kernel (caller falls back).
std::shared_ptr<TcConvPlan> tc_conv_prepare(const ConvArgs &a, int device, std::string *why);
size_t tc_conv_ws_elems(const TcConvPlan &p);      // fp32 elements of split-K scratch the plan wants (0 = none)
cudaError_t tc_conv_launch(const TcConvPlan &p, const ConvArgs &a, cudaStream_t st, int *launches);
cudaError_t tc_conv_init(int device);  // one-time device set-up; call outside stream capture
bool tc_available();
int tc_conv_status();  // nonzero once any tensor-core kernel reported a bounded wait running out
int *tc_status_word(int device);  // device address of that status word (after tc_conv_init), else nullptr
cudaError_t tc_conv_status_clear();  // synchronises the current device, then zeroes its status words and the sticky flag
cudaError_t tc_expire_wait(unsigned limit_us, cudaStream_t st);  // a kernel whose only wait runs out after limit_us (test of the time-out path)

// ---- grouped tensor-core convolution (sgs_conv_group.cu) -------------------------------------
// One launch runs the same stored layer for up to TC_GROUP_MAX_ENTRIES members (queries in flight).
// A member is described by a TC_GROUP_ENTRY_BYTES record in a device table and by its tensor maps,
// which travel in the kernel's parameter block.  Plans for it are prepared with
// ConvArgs::throughput == 2 (128-filter tiles, reduction never split).
constexpr int TC_GROUP_ENTRY_BYTES = 128;
constexpr int TC_GROUP_MAX_ENTRIES = 64;
constexpr int TC_GROUP_MAPS_SMALL = 64, TC_GROUP_MAPS_LARGE = 248;  // tensor maps per launch (two kernel variants)
class GroupLaunch {
public:
    GroupLaunch();
    ~GroupLaunch();
    GroupLaunch(const GroupLaunch &) = delete;
    GroupLaunch &operator=(const GroupLaunch &) = delete;
    void reset(const void *d_entries);       // start a launch whose member records will live at d_entries
    bool fits(const TcConvPlan &p) const;   // room for one more member (records and tensor maps)?
    // Adds a member: writes its record to host_entry (the host image of the next device record).
    void add(void *host_entry, const TcConvPlan &p, const ConvArgs &a);
    int members() const;
    int maps() const;                       // tensor maps used so far
    int tiles() const;
    // window_max > 0: also mark the launch's cached filter prefix with an access-policy window of at most that many bytes
    cudaError_t launch(size_t window_max, int sms, cudaStream_t st);
private:
    struct Impl;
    Impl *impl;
};
cudaError_t tc_group_init(int device);

cudaError_t subnet_kernel_init(int device);
size_t subnet_kernel_smem();  // dynamic shared memory of a block
int subnet_kernel_blocks_per_sm();
cudaError_t subnet_kernel_launch(const PqParams &p, int blocks, cudaStream_t st);
size_t subnet_kernel_held_max();  // largest weight buffer a block can keep
void tc_group_set_stage_group(int stages);  // tuning: stages per barrier pair of the grouped kernel (0 = default)

}  // namespace sgs
