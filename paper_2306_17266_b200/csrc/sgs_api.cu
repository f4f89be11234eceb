// Host side of libsgs: the C interface, SuperNet loading, SubNet slice plans, plan execution,
// query streams and the SubGraph cache policy.
#include "sgs_internal.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <cstdlib>
#include <deque>
#include <map>
#include <chrono>
#include <nvtx3/nvToolsExt.h>
#include <mutex>

using namespace sgs;

namespace {

constexpr uint32_t BLOB_MAGIC = 0x42534753u;  // 'SGSB'

struct LayerSpec {
    std::string name;
    int kind, K, C, R;
    bool bn, bias;
};

// nearest multiple of 8 to num/den (ties up), at least 8
int round8(long long num, long long den) {
    long long q = (2 * num + 8 * den) / (16 * den);
    return (int)std::max<long long>(8, 8 * q);
}
int per_mille(float f) { return (int)std::floor((double)f * 1000.0 + 0.5); }

struct FamilyDef {
    int n_stages = 0;
    std::vector<int> width, max_depth, base_depth, stride, act, se;
    int stem = 0, classes = 0, max_kernel = 0;
};

FamilyDef family_def(int family) {
    FamilyDef d;
    if (family == SGS_TINY) {
        d.n_stages = 3; d.width = {16, 32, 64}; d.max_depth = {3, 3, 3}; d.base_depth = {1, 1, 1};
        d.stride = {1, 2, 2}; d.stem = 16; d.classes = 10; d.max_kernel = 3;
    } else if (family == SGS_RESNET) {
        d.n_stages = 4; d.width = {256, 512, 1024, 2048}; d.base_depth = {2, 2, 4, 2}; d.max_depth = {4, 4, 6, 4};
        d.stride = {1, 2, 2, 2}; d.stem = 64; d.classes = 1000; d.max_kernel = 7;
    } else if (family == SGS_MBV3) {
        d.n_stages = 5; d.width = {24, 40, 80, 112, 160}; d.max_depth = {4, 4, 4, 4, 4}; d.base_depth = {2, 2, 2, 2, 2};
        d.stride = {2, 2, 2, 1, 2}; d.act = {ACT_RELU, ACT_RELU, ACT_HSWISH, ACT_HSWISH, ACT_HSWISH};
        d.se = {0, 1, 0, 1, 1}; d.stem = 16; d.classes = 1000; d.max_kernel = 7;
    }
    return d;
}

std::string bname(int s, int b, const char *leaf) {
    char buf[64];
    snprintf(buf, sizeof buf, "s%db%d.%s", s, b, leaf);
    return buf;
}

// Stored layers in blob order.
std::vector<LayerSpec> stored_layers(int family) {
    FamilyDef d = family_def(family);
    std::vector<LayerSpec> v;
    auto conv = [&](std::string n, int K, int C, int R) { v.push_back({std::move(n), KIND_CONV, K, C, R, true, false}); };
    auto lin = [&](std::string n, int K, int C) { v.push_back({std::move(n), KIND_LINEAR, K, C, 1, false, true}); };
    auto dw = [&](std::string n, int K, int R) { v.push_back({std::move(n), KIND_DW, K, 1, R, true, false}); };
    if (family == SGS_TINY) {
        conv("stem", d.stem, 3, 3);
        int in = d.stem;
        for (int s = 0; s < d.n_stages; s++) {
            for (int b = 0; b < d.max_depth[s]; b++) {
                int cin = b ? d.width[s] : in;
                conv(bname(s, b, "conv1"), d.width[s], cin, 3);
                conv(bname(s, b, "conv2"), d.width[s], d.width[s], 3);
                if (b == 0 && s > 0) conv(bname(s, b, "proj"), d.width[s], cin, 1);
            }
            in = d.width[s];
        }
        lin("fc", d.classes, in);
    } else if (family == SGS_RESNET) {
        conv("stem", d.stem, 3, 7);
        int in = d.stem;
        for (int s = 0; s < d.n_stages; s++) {
            int mid = round8((long long)d.width[s] * 350, 1000);
            for (int b = 0; b < d.max_depth[s]; b++) {
                int cin = b ? d.width[s] : in;
                conv(bname(s, b, "conv1"), mid, cin, 1);
                conv(bname(s, b, "conv2"), mid, mid, 3);
                conv(bname(s, b, "conv3"), d.width[s], mid, 1);
                if (b == 0) conv(bname(s, b, "proj"), d.width[s], cin, 1);
            }
            in = d.width[s];
        }
        lin("fc", d.classes, in);
    } else if (family == SGS_MBV3) {
        conv("stem", d.stem, 3, 3);
        dw("first.dw", d.stem, 3);
        conv("first.pw", d.stem, d.stem, 1);
        int in = d.stem;
        for (int s = 0; s < d.n_stages; s++) {
            for (int b = 0; b < d.max_depth[s]; b++) {
                int cin = b ? d.width[s] : in, mid = 6 * cin;
                conv(bname(s, b, "expand"), mid, cin, 1);
                dw(bname(s, b, "dw"), mid, 7);
                if (d.se[s]) {
                    int sq = round8(mid, 4);
                    lin(bname(s, b, "se1"), sq, mid);
                    lin(bname(s, b, "se2"), mid, sq);
                }
                conv(bname(s, b, "project"), d.width[s], mid, 1);
            }
            in = d.width[s];
        }
        conv("head.conv", 960, in, 1);
        lin("head.mix", 1280, 960);
        lin("fc", d.classes, 1280);
    }
    return v;
}

// Channels per stored (filter, tap) row of a convolution: bf16 rows are padded with zeros to a multiple of 16
// channels (32 bytes), so that tensor-map rows start and end on 32-byte sectors (the 3-channel stem keeps its rows).
int stored_row(int kind, int C, int dtype) { return (kind == KIND_CONV && dtype == SGS_BF16 && C >= 8) ? (C + 15) / 16 * 16 : C; }

struct DeviceGuard {
    int prev = -1;
    bool ok = true;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) prev = -1;
        if (prev != dev) ok = cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

struct CacheState {
    bool enabled = false;
    int window_q = 4;
    size_t budget = 0;
    std::deque<std::vector<int>> window;  // last encodings (3 ints per layer)
    std::vector<int> G;                   // cached SubGraph encoding, clipped to the budget
    size_t G_bytes = 0;
    int epoch = 0;                        // bumped whenever G changes
    int since_update = 0;
    int evict_first_when_off = 0;
    int policy = 0;                       // 0: intersection of the window; 1: candidate nearest to the window's average;
                                          // 2: pinned by a scheduler object (observations change nothing)
    std::vector<std::vector<int>> cand_raw, cand;  // candidate SubGraph encodings as given / clipped to the budget
    std::vector<size_t> cand_bytes;
    int decisions = 0, last_choice = -1;
};

}  // namespace

struct sgs_supernet {
    int family = 0, device = 0;
    sgs_dtype_t dtype = SGS_BF16;
    FamilyDef def;
    std::vector<StoredLayer> layers;
    std::map<std::string, int> by_name;
    char *weight_arena = nullptr;
    size_t weight_arena_bytes = 0;
    float *param_arena = nullptr;  // folded scale / shift
    size_t param_arena_bytes = 0;
    // bf16 handles: the stem's weights once more as a GEMM operand [K][stem_kkp] (rows = the stored
    // (r, s, c) order, zero padded to a multiple of 8), used with the patch matrix of the input
    void *stem_gemm_w = nullptr;
    int stem_kkp = 0;
    // ... and as [K][k][64] for the window view used by waves: per filter row an 8-pixel x 8-channel window
    void *stem_win_w = nullptr;
    // Workspaces of the queries in flight.  Queries of a stream are independent, so up to
    // `concurrency` of them run at the same time, each in its own slot (own activation buffers, own
    // scratch, own CUDA stream); slot 0 runs on the caller's stream.
    struct Slot {
        void *act[4] = {nullptr, nullptr, nullptr, nullptr};
        float *vec[3] = {nullptr, nullptr, nullptr};
        float *ws = nullptr;        // split-K scratch of the tensor-core kernel
        void *stage_in = nullptr;   // device staging for host-buffer streams
        float *stage_out = nullptr;
        cudaStream_t st = nullptr;  // internal stream (slots >= 1)
        cudaEvent_t ev = nullptr;
    };
    std::vector<Slot> slots;
    // Wave execution (many queries advance through the layers together, one grouped launch per layer):
    // each wave in flight has its own stream, launch-table buffers and staging buffers.
    struct WaveCtx {
        cudaStream_t st = nullptr;
        cudaEvent_t done = nullptr;  // everything issued for the last wave of this context has finished
        char *h_tbl = nullptr, *d_tbl = nullptr;  // launch tables of one wave: pinned host image and device copy
        size_t tbl_bytes = 0;
        void *stage_in = nullptr;    // host-buffer streams: the wave's inputs / logits on the device
        float *stage_out = nullptr;
        size_t stage_in_bytes = 0, stage_out_bytes = 0;
        bool busy = false;
    };
    std::vector<WaveCtx> waves;
    std::vector<std::unique_ptr<GroupLaunch>> group_pool;  // parameter blocks of a wave's grouped launches (reused)
    std::unordered_map<long long, int> op_rank;        // (op type, anchor layer) -> position in the largest SubNet
    int sms = 148;
    size_t act_elems = 0;
    size_t vec_elems = 0;
    int *cache_tbl = nullptr;       // device: [policy, K_0, C_0, K_1, C_1, ...] read by the conv kernels
    int cache_tbl_epoch = -1;       // cache epoch the device table reflects
    int *tbl_ring = nullptr;        // pinned host ring of table images (async uploads need stable sources)
    cudaEvent_t tbl_ring_ev[16] = {};  // upload of ring entry i has completed
    int tbl_ring_pos = 0;
    size_t splitk_ws_elems = 0;
    size_t stage_in_bytes = 0, stage_out_bytes = 0;
    size_t device_bytes = 0;
    std::unordered_map<std::string, std::unique_ptr<Plan>> plans;
    CacheState cache;
    size_t l2_bytes = 0, persist_max = 0, window_max = 0;
    long long kernel_launches = 0;
    int plan_hits = 0, plan_misses = 0;
    int force_plain = 0;
    // persistent SubNet kernel: scratch of its blocks, op / query tables (pinned host image and device copy), query counter
    unsigned char *pq_scratch = nullptr;
    size_t pq_scratch_bytes = 0;
    char *pq_h_tbl = nullptr, *pq_d_tbl = nullptr;
    size_t pq_tbl_bytes = 0;
    int *pq_counter = nullptr;
    void *pq_stage_in = nullptr;
    float *pq_stage_out = nullptr;
    size_t pq_stage_in_bytes = 0, pq_stage_out_bytes = 0;
    size_t persist_limit_set = 0;  // cudaLimitPersistingL2CacheSize as last set by this handle
    int nvtx = 0;  // 1: NVTX ranges named after the stored layer around every launch
    int persistent_held_kb = 16;  // persistent execution: shared memory per SM for the cached SubGraph's first layers (0: none)
    long long fail_alloc_after = -1;  // < 0: off; else device allocations left before they start failing (test aid)
    int cache_mech = 0;    // how grouped launches keep the cached SubGraph in L2: 0 per-tile hints, 1 access-policy window of the launch, 2 both
    int pad_channels = 1;  // waves of the ResNet-shaped family keep activation pixels at multiples of 16 channels
    int throughput_mode = 0;  // set by streams that keep many queries in flight; part of the plan key
    double host_us_graph = 0, host_us_direct = 0, host_us_stream = 0, host_us_query = 0, host_us_table = 0;  // host time spent issuing work (diagnostic counters)
    // per-kernel-class timing (option "profile"): 0 tensor-core conv, 1 CUDA-core conv, 2 depthwise, 3 other
    int profile = 0;
    std::vector<Plan *> prof_used;  // plans run since the last fold, in order
    double prof_ms[4] = {0, 0, 0, 0}, prof_bytes[4] = {0, 0, 0, 0}, prof_flops[4] = {0, 0, 0, 0};
    long long prof_launches[4] = {0, 0, 0, 0};
    std::vector<sgs_launch_record_t> prof_trace;  // waves: one record per launch of the profiled passes (bounded)
    mutable std::string err;
    size_t elem() const { return dtype == SGS_BF16 ? 2 : 4; }
    int idx(const std::string &n) const {
        auto it = by_name.find(n);
        return it == by_name.end() ? -1 : it->second;
    }
};

namespace {

sgs_status_t fail(const sgs_supernet *n, sgs_status_t st, const std::string &msg) {
    if (n) n->err = msg;
    return st;
}
#define CU(call)                                                                                        \
    do {                                                                                                \
        cudaError_t e_ = (call);                                                                        \
        if (e_ != cudaSuccess)                                                                          \
            return fail(net, e_ == cudaErrorMemoryAllocation ? SGS_ENOMEM : SGS_ECUDA,                  \
                        std::string(#call) + ": " + cudaGetErrorString(e_));                            \
    } while (0)

sgs_status_t dev_alloc(sgs_supernet *net, void **p, size_t bytes) {
    // (fault injection on the host, option "fail_alloc_after": the n-th allocation from now on and every later one fail)
    if (net->fail_alloc_after >= 0 && net->fail_alloc_after-- == 0) {
        net->fail_alloc_after = 0;
        *p = nullptr;
        return fail(net, SGS_ENOMEM, "device allocation failed (injected)");
    }
    if (cudaMalloc(p, bytes) != cudaSuccess) {
        cudaGetLastError();
        *p = nullptr;
        return fail(net, SGS_ENOMEM, "device allocation of " + std::to_string(bytes) + " bytes failed");
    }
    net->device_bytes += bytes;
    return SGS_OK;
}
void dev_free(sgs_supernet *net, void *p, size_t bytes) {
    if (!p) return;
    cudaFree(p);
    net->device_bytes -= bytes;
}
void drop_graphs(sgs_supernet *net) {
    for (auto &kv : net->plans) {
        if (kv.second->graph) { cudaGraphExecDestroy(kv.second->graph); kv.second->graph = nullptr; }
    }
}

// ------------------------------------------------------------------------------------------
// Config -> per-layer slices (paper Section 2.1: elastic depth, width / expand ratio, kernel)
// ------------------------------------------------------------------------------------------
bool in_set(int v, std::initializer_list<int> s) { return std::find(s.begin(), s.end(), v) != s.end(); }

bool cfg_valid(const sgs_supernet *net, const sgs_subnet_cfg_t *c) {
    const FamilyDef &d = net->def;
    for (int s = 0; s < d.n_stages; s++) {
        int dep = c->depth[s];
        if (net->family == SGS_TINY) {
            if (!in_set(dep, {1, 2, 3}) || !in_set(per_mille(c->width[s + 1]), {500, 750, 1000})) return false;
        } else if (net->family == SGS_RESNET) {
            if (dep < d.base_depth[s] || dep > d.max_depth[s]) return false;
            if (!in_set(per_mille(c->width[s + 1]), {650, 800, 1000})) return false;
            for (int b = 0; b < dep; b++)
                if (!in_set(per_mille(c->expand[s][b]), {200, 250, 350})) return false;
        } else {
            if (!in_set(dep, {2, 3, 4})) return false;
            for (int b = 0; b < dep; b++) {
                if (!in_set(per_mille(c->expand[s][b]), {3000, 4000, 6000})) return false;
                if (!in_set(c->kernel[s][b], {3, 5, 7})) return false;
            }
        }
    }
    if (net->family == SGS_RESNET && !in_set(per_mille(c->width[0]), {650, 800, 1000})) return false;
    return true;
}

std::vector<Slice> slices_for(const sgs_supernet *net, const sgs_subnet_cfg_t *c) {
    const FamilyDef &d = net->def;
    std::vector<Slice> sl(net->layers.size());
    auto use = [&](const std::string &name, int K, int C, int k) {
        int i = net->idx(name);
        sl[i].active = 1; sl[i].K = K; sl[i].C = C; sl[i].k = k;
    };
    if (net->family == SGS_TINY) {
        std::vector<int> w(3);
        for (int s = 0; s < 3; s++) w[s] = d.width[s] * per_mille(c->width[s + 1]) / 1000;
        use("stem", w[0], 3, 3);
        int in = w[0];
        for (int s = 0; s < 3; s++) {
            for (int b = 0; b < c->depth[s]; b++) {
                int cin = b ? w[s] : in;
                use(bname(s, b, "conv1"), w[s], cin, 3);
                use(bname(s, b, "conv2"), w[s], w[s], 3);
                if (b == 0 && s > 0) use(bname(s, b, "proj"), w[s], cin, 1);
            }
            in = w[s];
        }
        use("fc", d.classes, in, 1);
    } else if (net->family == SGS_RESNET) {
        int in = round8((long long)d.stem * per_mille(c->width[0]), 1000);
        use("stem", in, 3, 7);
        for (int s = 0; s < 4; s++) {
            int out = round8((long long)d.width[s] * per_mille(c->width[s + 1]), 1000);
            for (int b = 0; b < c->depth[s]; b++) {
                int cin = b ? out : in;
                int mid = round8((long long)out * per_mille(c->expand[s][b]), 1000);
                use(bname(s, b, "conv1"), mid, cin, 1);
                use(bname(s, b, "conv2"), mid, mid, 3);
                use(bname(s, b, "conv3"), out, mid, 1);
                if (b == 0) use(bname(s, b, "proj"), out, cin, 1);
            }
            in = out;
        }
        use("fc", d.classes, in, 1);
    } else {
        use("stem", d.stem, 3, 3);
        use("first.dw", d.stem, 1, 3);
        use("first.pw", d.stem, d.stem, 1);
        int in = d.stem;
        for (int s = 0; s < 5; s++) {
            for (int b = 0; b < c->depth[s]; b++) {
                int cin = b ? d.width[s] : in;
                int mid = round8((long long)cin * per_mille(c->expand[s][b]), 1000);
                use(bname(s, b, "expand"), mid, cin, 1);
                use(bname(s, b, "dw"), mid, 1, c->kernel[s][b]);
                if (d.se[s]) {
                    int sq = round8(mid, 4);
                    use(bname(s, b, "se1"), sq, mid, 1);
                    use(bname(s, b, "se2"), mid, sq, 1);
                }
                use(bname(s, b, "project"), d.width[s], mid, 1);
            }
            in = d.width[s];
        }
        use("head.conv", 960, in, 1);
        use("head.mix", 1280, 960, 1);
        use("fc", d.classes, 1280, 1);
    }
    return sl;
}

std::vector<int> encoding_of(const std::vector<Slice> &sl) {
    std::vector<int> e(3 * sl.size());
    for (size_t i = 0; i < sl.size(); i++) { e[3 * i] = sl[i].K; e[3 * i + 1] = sl[i].C; e[3 * i + 2] = sl[i].k; }
    return e;
}

// ------------------------------------------------------------------------------------------
// Plan construction
// ------------------------------------------------------------------------------------------
struct Builder {
    sgs_supernet *net;
    Plan *plan;
    int N;
    size_t max_elems = 0;
    bool padded = false;  // activation tensors keep pixels at a multiple of 16 channels (see ConvArgs::ldx)

    void note(size_t elems) { max_elems = std::max(max_elems, elems); }
    int phys(int channels) const { return padded ? (channels + 15) / 16 * 16 : channels; }

    // convolution (regular or depthwise) of stored layer `name`
    void conv(const std::string &name, int in, int out, int res, int &H, int &W, int stride, int act) {
        int li = net->idx(name);
        const StoredLayer &L = net->layers[li];
        const Slice &s = plan->slices[li];
        Op op;
        op.type = L.kind == KIND_DW ? OP_DW : OP_CONV;
        op.layer = li; op.in = in; op.out = out; op.res = res;
        ConvArgs &a = op.conv;
        a.w = L.w; a.scale = L.scale; a.shift = L.shift;
        a.N = N; a.H = H; a.W = W; a.C = L.kind == KIND_DW ? s.K : s.C; a.K = s.K;
        a.k = s.k; a.stride = stride; a.act = act;
        int p = (s.k - 1) / 2;
        a.Ho = (H + 2 * p - s.k) / stride + 1;
        a.Wo = (W + 2 * p - s.k) / stride + 1;
        a.Kmax = L.K; a.Cmax = L.kind == KIND_CONV ? L.Cp : L.C; a.R = L.R;
        if (padded && op.type == OP_CONV) { a.ldx = in >= 0 ? phys(a.C) : 0; a.ldy = phys(a.K); }
        double M = (double)N * a.Ho * a.Wo;
        double per_out = L.kind == KIND_DW ? (double)s.k * s.k : (double)s.C * s.k * s.k;
        op.flops = 2.0 * M * s.K * per_out;
        op.alg_bytes = ((double)s.K * per_out + (double)N * H * W * a.C + M * s.K * (res >= 0 ? 2 : 1)) * net->elem();
        plan->flops += op.flops;
        plan->weight_bytes += (double)s.K * per_out * net->elem();
        plan->act_bytes += ((double)N * H * W * a.C + M * s.K * (res >= 0 ? 2 : 1)) * net->elem();
        note((size_t)M * phys(s.K));
        H = a.Ho; W = a.Wo;
        plan->ops.push_back(op);
    }
    // Stem (3 input channels): on bf16 handles with a filter count that is a multiple of 8 it runs on the
    // tensor cores as patch matrix (tmp) x GEMM weights; otherwise as a direct convolution.
    void stem(const std::string &name, int out, int tmp, int &H, int &W, int stride, int act) {
        const int li = net->idx(name);
        const StoredLayer &L = net->layers[li];
        const Slice &s = plan->slices[li];
        const size_t first = plan->ops.size();
        const int Hin = H, Win = W;
        conv(name, -1, out, -1, H, W, stride, act);
        // (the patch-matrix kernel stages whole input rows with 16-byte loads: widths that are multiples of 8)
        if (net->throughput_mode == 2 && net->stem_win_w && !net->force_plain && s.K % 8 == 0 && (s.k == 3 || s.k == 7)) {
            // Waves: no patch matrix.  The image is copied once into an 8-channel buffer with a zero margin
            // (16 bytes per pixel, so that pixels can be TMA rows); the 64 contiguous elements that start at
            // padded pixel wo * stride are the 8-pixel window of output column wo, and the stem becomes a
            // convolution over the k filter ROWS with 64 "channels" per row.
            Op &cv = plan->ops[first];
            const int P = (s.k - 1) / 2;
            int Hp = std::max((H - 1) * stride + s.k, Hin + P), Wp = std::max((W - 1) * stride + 8, Win + P);
            Hp += Hp & 1; Wp += Wp & 1;
            Op pd;
            pd.type = OP_PAD8; pd.layer = li; pd.in = -1; pd.out = tmp;
            pd.N = N; pd.H = Hin; pd.W = Win; pd.C = 3; pd.K = P;
            pd.conv.Ho = Hp; pd.conv.Wo = Wp;
            pd.alg_bytes = ((double)N * Hin * Win * 3 + (double)N * Hp * Wp * 8) * net->elem();
            cv.in = tmp;
            ConvArgs &a = cv.conv;
            a.w = net->stem_win_w;
            a.H = Hp; a.W = Wp; a.C = 64; a.Cmax = 64; a.win = 1; a.ldx = 0;
            note((size_t)N * Hp * Wp * 8);
            plan->ops.insert(plan->ops.begin() + (long)first, pd);
            return;
        }
        if (!net->stem_gemm_w || net->force_plain || s.K % 8 || (s.k != 3 && s.k != 7) || Win % 8 || Win > 1024) return;
        Op &cv = plan->ops[first];
        const int KKp = net->stem_kkp;
        Op im;
        im.type = OP_IM2COL; im.layer = li; im.in = -1; im.out = tmp;
        im.N = N; im.H = Hin; im.W = Win; im.C = 3; im.K = KKp;
        im.conv = cv.conv;  // geometry (k, stride, output dims)
        im.alg_bytes = ((double)N * Hin * Win * 3 + (double)N * H * W * KKp) * net->elem();
        cv.in = tmp;
        ConvArgs &a = cv.conv;
        a.w = net->stem_gemm_w;
        a.H = H; a.W = W; a.C = KKp; a.Cmax = KKp; a.R = 1; a.k = 1; a.stride = 1;
        note((size_t)N * H * W * KKp);
        plan->ops.insert(plan->ops.begin() + (long)first, im);
        (void)L;
    }
    void linear(const std::string &name, int vin, int vout, int act, bool vin_padded = false) {
        int li = net->idx(name);
        const Slice &s = plan->slices[li];
        Op op;
        // (a padded pooled vector carries zeros beyond the slice; the extra stored weights they meet exist: row pitch >= 16-multiple)
        op.type = OP_LINEAR; op.layer = li; op.vin = vin; op.vout = vout; op.N = N; op.C = vin_padded ? std::min(phys(s.C), net->layers[li].C) : s.C; op.K = s.K; op.act = act;
        op.flops = 2.0 * N * s.K * s.C;
        op.alg_bytes = (double)s.K * s.C * net->elem() + 4.0 * N * (s.K + s.C);
        plan->flops += op.flops;
        plan->weight_bytes += (double)s.K * s.C * net->elem();
        plan->ops.push_back(op);
    }
    void gap(int in, int vout, int H, int W, int C) {
        Op op;
        op.type = OP_GAP; op.in = in; op.vout = vout; op.N = N; op.H = H; op.W = W; op.C = phys(C);
        op.alg_bytes = (double)N * H * W * C * net->elem() + 4.0 * N * C;
        plan->ops.push_back(op);
    }
};

sgs_status_t build_plan(sgs_supernet *net, const sgs_subnet_cfg_t *cfg, int batch, int res, Plan *plan) {
    const FamilyDef &d = net->def;
    plan->batch = batch; plan->res = res;
    plan->slices = slices_for(net, cfg);
    Builder B{net, plan, batch};
    // Waves of the ResNet-shaped family on bf16 handles: every convolution runs in the grouped tensor-core kernel
    // (all channel counts are multiples of 8, and with res % 32 == 0 every stride-2 layer sees even sizes), so the
    // activation tensors can be padded to 16-channel pixels.  choose_impls refuses a padded plan otherwise.
    B.padded = net->family == SGS_RESNET && net->throughput_mode == 2 && net->dtype == SGS_BF16 && !net->force_plain &&
               tc_available() && res % 32 == 0 && net->stem_win_w != nullptr && net->pad_channels;
    plan->padded = B.padded;
    int H = res, W = res;
    // activation buffers: X current tensor, T1/T2 temporaries, SC shortcut
    int X = 0, T1 = 1, T2 = 2, SC = 3;
    if (net->family == SGS_TINY) {
        B.stem("stem", X, T1, H, W, 1, ACT_RELU);
        for (int s = 0; s < 3; s++)
            for (int b = 0; b < cfg->depth[s]; b++) {
                int st = b == 0 ? d.stride[s] : 1, shortcut = X;
                int h1 = H, w1 = W;
                if (b == 0 && s > 0) { int h = H, w = W; B.conv(bname(s, b, "proj"), X, SC, -1, h, w, st, ACT_NONE); shortcut = SC; }
                B.conv(bname(s, b, "conv1"), X, T1, -1, h1, w1, st, ACT_RELU);
                B.conv(bname(s, b, "conv2"), T1, T2, shortcut, h1, w1, 1, ACT_RELU);
                std::swap(X, T2); H = h1; W = w1;
            }
        int C = plan->slices[net->idx("fc")].C;
        B.gap(X, 0, H, W, C);
        B.linear("fc", 0, -1, ACT_NONE);
    } else if (net->family == SGS_RESNET) {
        B.stem("stem", T1, T2, H, W, 2, ACT_RELU);
        {
            Op op;
            op.type = OP_MAXPOOL; op.in = T1; op.out = X; op.N = batch; op.H = H; op.W = W; op.C = B.phys(plan->slices[net->idx("stem")].K);
            int Hp = (H - 1) / 2 + 1, Wp = (W - 1) / 2 + 1;
            op.alg_bytes = ((double)batch * H * W + (double)batch * Hp * Wp) * plan->slices[net->idx("stem")].K * net->elem();
            plan->ops.push_back(op);
            H = Hp; W = Wp;
            B.note((size_t)batch * H * W * op.C);
        }
        for (int s = 0; s < 4; s++)
            for (int b = 0; b < cfg->depth[s]; b++) {
                int st = b == 0 ? d.stride[s] : 1, shortcut = X;
                int h = H, w = W;
                if (b == 0) { int h0 = H, w0 = W; B.conv(bname(s, b, "proj"), X, SC, -1, h0, w0, st, ACT_NONE); shortcut = SC; }
                B.conv(bname(s, b, "conv1"), X, T1, -1, h, w, 1, ACT_RELU);
                B.conv(bname(s, b, "conv2"), T1, T2, -1, h, w, st, ACT_RELU);
                B.conv(bname(s, b, "conv3"), T2, T1, shortcut, h, w, 1, ACT_RELU);
                std::swap(X, T1); H = h; W = w;
            }
        int C = plan->slices[net->idx("fc")].C;
        B.gap(X, 0, H, W, C);
        B.linear("fc", 0, -1, ACT_NONE, B.padded);
    } else {
        B.stem("stem", X, T1, H, W, 2, ACT_HSWISH);
        { int h = H, w = W; B.conv("first.dw", X, T1, -1, h, w, 1, ACT_RELU); }
        { int h = H, w = W; B.conv("first.pw", T1, T2, X, h, w, 1, ACT_NONE); }
        std::swap(X, T2);
        int C = d.stem;
        for (int s = 0; s < 5; s++)
            for (int b = 0; b < cfg->depth[s]; b++) {
                int st = b == 0 ? d.stride[s] : 1, out = d.width[s];
                int mid = plan->slices[net->idx(bname(s, b, "expand"))].K;
                int h = H, w = W;
                B.conv(bname(s, b, "expand"), X, T1, -1, h, w, 1, d.act[s]);
                B.conv(bname(s, b, "dw"), T1, T2, -1, h, w, st, d.act[s]);
                if (d.se[s]) {
                    B.gap(T2, 0, h, w, mid);
                    Op g;
                    g.type = OP_SE_GATE; g.layer = net->idx(bname(s, b, "se1")); g.layer2 = net->idx(bname(s, b, "se2"));
                    g.vin = 0; g.vout = 1; g.N = batch; g.C = mid; g.K = plan->slices[g.layer].K;
                    g.flops = 4.0 * batch * mid * g.K;
                    g.alg_bytes = 2.0 * mid * g.K * net->elem();
                    plan->flops += g.flops;
                    plan->weight_bytes += 2.0 * mid * g.K * net->elem();
                    plan->ops.push_back(g);
                    Op sc;
                    sc.type = OP_SCALE; sc.in = T2; sc.out = T2; sc.vin = 1; sc.N = batch; sc.H = h; sc.W = w; sc.C = mid;
                    sc.alg_bytes = 2.0 * batch * h * w * mid * net->elem();
                    plan->ops.push_back(sc);
                }
                int resid = (st == 1 && C == out) ? X : -1;
                B.conv(bname(s, b, "project"), T2, T1, resid, h, w, 1, ACT_NONE);
                std::swap(X, T1); H = h; W = w; C = out;
            }
        { int h = H, w = W; B.conv("head.conv", X, T1, -1, h, w, 1, ACT_HSWISH); }
        B.gap(T1, 0, H, W, 960);
        B.linear("head.mix", 0, 1, ACT_HSWISH);
        B.linear("fc", 1, -1, ACT_NONE);
    }
    plan->act_elems = B.max_elems;
    return SGS_OK;
}

// Makes sure `n_slots` slots exist, each with buffers for the sizes in use.
// Frees the activation / vector / split-reduction buffers of a slot (the sizes are the handle's current ones).
void release_slot_buffers(sgs_supernet *net, sgs_supernet::Slot &sl, bool act, bool vec, bool ws) {
    for (int i = 0; i < 4 && act; i++) { dev_free(net, sl.act[i], net->act_elems * net->elem() + 256); sl.act[i] = nullptr; }
    for (int i = 0; i < 3 && vec; i++) { dev_free(net, sl.vec[i], net->vec_elems * 4); sl.vec[i] = nullptr; }
    if (ws) { dev_free(net, sl.ws, net->splitk_ws_elems * 4); sl.ws = nullptr; }
}

sgs_status_t ensure_slots(sgs_supernet *net, int n_slots) {
    while ((int)net->slots.size() < n_slots) {
        sgs_supernet::Slot sl;
        if (!net->slots.empty()) {
            CU(cudaStreamCreateWithFlags(&sl.st, cudaStreamNonBlocking));
            CU(cudaEventCreateWithFlags(&sl.ev, cudaEventDisableTiming));
        }
        sgs_status_t st = SGS_OK;
        for (int i = 0; i < 4 && net->act_elems && st == SGS_OK; i++) st = dev_alloc(net, &sl.act[i], net->act_elems * net->elem() + 256);
        for (int i = 0; i < 3 && net->vec_elems && st == SGS_OK; i++) st = dev_alloc(net, (void **)&sl.vec[i], net->vec_elems * 4);
        if (net->splitk_ws_elems && st == SGS_OK) st = dev_alloc(net, (void **)&sl.ws, net->splitk_ws_elems * 4);
        if (st != SGS_OK) {  // nothing of a half-built slot stays behind
            release_slot_buffers(net, sl, true, true, true);
            if (sl.st) cudaStreamDestroy(sl.st);
            if (sl.ev) cudaEventDestroy(sl.ev);
            return st;
        }
        net->slots.push_back(sl);
    }
    return SGS_OK;
}

// Grows the workspaces of every slot.  If an allocation fails, ALL slots give up the kind of buffer that was being
// grown and the handle's size for it returns to zero, so that the next call starts from a consistent state (no slot
// is ever left with a missing or a smaller buffer than the handle believes).
sgs_status_t ensure_workspace(sgs_supernet *net, size_t act_elems, int batch) {
    if (net->slots.empty()) { sgs_status_t st = ensure_slots(net, 1); if (st != SGS_OK) return st; }
    if (act_elems > net->act_elems) {
        drop_graphs(net);
        for (auto &kv : net->plans) kv.second->prepared = false;
        for (auto &sl : net->slots) release_slot_buffers(net, sl, true, false, false);
        net->act_elems = act_elems;
        sgs_status_t st = SGS_OK;
        for (auto &sl : net->slots)
            for (int i = 0; i < 4 && st == SGS_OK; i++) st = dev_alloc(net, &sl.act[i], act_elems * net->elem() + 256);
        if (st != SGS_OK) {
            for (auto &sl : net->slots) release_slot_buffers(net, sl, true, false, false);
            net->act_elems = 0;
            return st;
        }
    }
    size_t vneed = (size_t)batch * 2048;
    if (vneed > net->vec_elems) {
        drop_graphs(net);
        for (auto &sl : net->slots) release_slot_buffers(net, sl, false, true, false);
        net->vec_elems = vneed;
        sgs_status_t st = SGS_OK;
        for (auto &sl : net->slots)
            for (int i = 0; i < 3 && st == SGS_OK; i++) st = dev_alloc(net, (void **)&sl.vec[i], vneed * 4);
        if (st != SGS_OK) {
            for (auto &sl : net->slots) release_slot_buffers(net, sl, false, true, false);
            net->vec_elems = 0;
            return st;
        }
    }
    return SGS_OK;
}

// Chooses the implementation of every convolution of a plan and fixes its buffer addresses (the
// tensor maps of the tensor-core kernel hold absolute addresses of the activation workspaces).
// prepare_impls touches nothing but the plan (several plans may be prepared at the same time by different threads);
// choose_impls = prepare + the part that may grow the handle's split-reduction scratch.
sgs_status_t prepare_impls(const sgs_supernet *net, Plan *plan, size_t *ws_need_out, std::string *err) {
    size_t ws_need = 0;
    for (Op &op : plan->ops) {
        if (op.type != OP_CONV && op.type != OP_DW) continue;
        const sgs_supernet::Slot &sl = net->slots[plan->slot];
        op.conv.x = op.in >= 0 ? sl.act[op.in] : nullptr;
        op.conv.y = sl.act[op.out];
        op.conv.res = op.res >= 0 ? sl.act[op.res] : nullptr;
        op.impl = 0;
        op.tc.reset();
        op.conv.throughput = plan->throughput;
        if (op.type != OP_CONV || op.in < 0) continue;
        if (net->dtype != SGS_BF16 || net->force_plain || !tc_available()) continue;
        std::string why;
        op.tc = tc_conv_prepare(op.conv, net->device, &why);
        if (!op.tc && op.conv.win) { *err = "window view of the stem: " + why; return SGS_EUNSUPPORTED; }
        if (!op.tc && plan->padded) { *err = "padded activation layout needs the tensor-core kernel: " + why; return SGS_EUNSUPPORTED; }
        if (op.tc) {
            op.impl = 1;
            ws_need = std::max(ws_need, tc_conv_ws_elems(*op.tc));
        }
    }
    *ws_need_out = ws_need;
    return SGS_OK;
}

sgs_status_t grow_splitk_scratch(sgs_supernet *net, size_t ws_need) {
    if (ws_need > net->splitk_ws_elems) {
        drop_graphs(net);
        for (auto &sl : net->slots) release_slot_buffers(net, sl, false, false, true);  // (cudaFree waits for work in flight)
        net->splitk_ws_elems = ws_need;
        sgs_status_t st = SGS_OK;
        for (auto &sl : net->slots)
            if (st == SGS_OK) st = dev_alloc(net, (void **)&sl.ws, ws_need * 4);
        if (st != SGS_OK) {
            for (auto &sl : net->slots) release_slot_buffers(net, sl, false, false, true);
            net->splitk_ws_elems = 0;
            for (auto &kv : net->plans) kv.second->prepared = false;  // (plans that counted on the scratch choose again)
            return st;
        }
    }
    return SGS_OK;
}

sgs_status_t choose_impls(sgs_supernet *net, Plan *plan) {
    size_t ws_need = 0;
    std::string err;
    sgs_status_t st = prepare_impls(net, plan, &ws_need, &err);
    if (st != SGS_OK) return fail(net, st, err);
    if ((st = grow_splitk_scratch(net, ws_need)) != SGS_OK) return st;
    plan->prepared = true;
    return SGS_OK;
}

// NVTX range around the launches of one layer (option "nvtx"; a no-op unless a tool that listens is attached).
struct LayerRange {
    bool on;
    LayerRange(const sgs_supernet *net, int layer, const char *what) : on(net->nvtx != 0) {
        if (!on) return;
        const std::string name = layer >= 0 && layer < (int)net->layers.size() ? net->layers[(size_t)layer].name : std::string(what);
        nvtxRangePushA(name.c_str());
    }
    ~LayerRange() { if (on) nvtxRangePop(); }
    LayerRange(const LayerRange &) = delete;
    LayerRange &operator=(const LayerRange &) = delete;
};

// Key of an op that is the same for every SubNet: its type and the stored layer it uses; ops without
// a layer (pools, the SE scale) are anchored to the next op that has one.
long long op_key(const Plan &p, size_t oi) {
    int anchor = p.ops[oi].layer;
    for (size_t j = oi + 1; anchor < 0 && j < p.ops.size(); j++) anchor = p.ops[j].layer;
    return ((long long)p.ops[oi].type << 32) | (unsigned)anchor;
}

// The largest SubNet runs every op any SubNet runs, in the same relative order (depth keeps the first
// blocks of a stage), so the position of an op in its op list orders the ops of all SubNets.
sgs_status_t ensure_ranks(sgs_supernet *net) {
    if (!net->op_rank.empty()) return SGS_OK;
    sgs_subnet_cfg_t c;
    std::memset(&c, 0, sizeof c);
    const FamilyDef &d = net->def;
    for (int s = 0; s < d.n_stages; s++) {
        c.depth[s] = d.max_depth[s];
        c.width[s + 1] = 1.0f;
        for (int b = 0; b < SGS_MAX_BLOCKS; b++) { c.expand[s][b] = net->family == SGS_MBV3 ? 6.0f : 0.35f; c.kernel[s][b] = 7; }
    }
    c.width[0] = 1.0f;
    // (the stem has two forms, patch matrix + GEMM and padded copy + window view: both are ranked)
    const int mode = net->throughput_mode;
    for (int m : {0, 2}) {
        net->throughput_mode = m;
        Plan p;
        sgs_status_t st = build_plan(net, &c, 1, 64, &p);
        if (st != SGS_OK) { net->throughput_mode = mode; return st; }
        for (size_t i = 0; i < p.ops.size(); i++) net->op_rank.emplace(op_key(p, i), (int)i);
    }
    net->throughput_mode = mode;
    return SGS_OK;
}

sgs_status_t get_plan(sgs_supernet *net, const sgs_subnet_cfg_t *cfg, int batch, int res, int slot, Plan **out) {
    std::string key(reinterpret_cast<const char *>(cfg), sizeof(*cfg));
    key.append(reinterpret_cast<const char *>(&batch), sizeof batch);
    key.append(reinterpret_cast<const char *>(&res), sizeof res);
    key.append(reinterpret_cast<const char *>(&slot), sizeof slot);
    key.append(reinterpret_cast<const char *>(&net->throughput_mode), sizeof net->throughput_mode);
    auto it = net->plans.find(key);
    if (it != net->plans.end()) { net->plan_hits++; *out = it->second.get(); return SGS_OK; }
    if (!cfg_valid(net, cfg)) return fail(net, SGS_ECONFIG, "SubNet config outside the elastic sets of this SuperNet");
    net->plan_misses++;
    std::unique_ptr<Plan> p(new Plan);
    sgs_status_t st = build_plan(net, cfg, batch, res, p.get());
    if (st != SGS_OK) return st;
    p->slot = slot;
    p->throughput = net->throughput_mode;
    p->enc = encoding_of(p->slices);
    if ((st = ensure_ranks(net)) != SGS_OK) return st;
    for (size_t i = 0; i < p->ops.size(); i++) {
        auto it = net->op_rank.find(op_key(*p, i));
        if (it == net->op_rank.end()) return fail(net, SGS_ECONFIG, "op outside the largest SubNet");
        p->ops[i].rank = it->second;
    }
    *out = p.get();
    net->plans.emplace(std::move(key), std::move(p));
    return SGS_OK;
}

// Argument record of a max pool, global average pool, linear or patch-matrix op (bf16 handles).
SmallEntry small_entry(const sgs_supernet *net, const Plan *plan, const Op &op, const void *d_input, void *d_logits) {
    const sgs_supernet::Slot &sl = net->slots[plan->slot];
    SmallEntry e;
    std::memset(&e, 0, sizeof e);
    switch (op.type) {
    case OP_MAXPOOL:
        e.x = op.in < 0 ? d_input : sl.act[op.in]; e.y = sl.act[op.out];
        e.N = op.N; e.H = op.H; e.W = op.W; e.C = op.C; e.Ho = (op.H - 1) / 2 + 1; e.Wo = (op.W - 1) / 2 + 1;
        break;
    case OP_GAP:
        e.x = op.in < 0 ? d_input : sl.act[op.in]; e.y = sl.vec[op.vout];
        e.N = op.N; e.H = op.H; e.W = op.W; e.C = op.C;
        break;
    case OP_LINEAR: {
        const StoredLayer &L = net->layers[op.layer];
        e.x = sl.vec[op.vin]; e.y = op.vout < 0 ? d_logits : (void *)sl.vec[op.vout];
        e.w = L.w; e.bias = L.shift;
        e.N = op.N; e.C = op.C; e.K = op.K; e.ld = L.C; e.act = op.act;
        break;
    }
    case OP_SCALE:
        e.x = sl.act[op.in]; e.y = sl.act[op.out]; e.w = sl.vec[op.vin];
        e.N = op.N; e.H = op.H; e.W = op.W; e.C = op.C;
        break;
    case OP_SE_GATE: {
        const StoredLayer &L1 = net->layers[op.layer], &L2 = net->layers[op.layer2];
        e.x = sl.vec[op.vin]; e.y = sl.vec[op.vout];
        e.w = L1.w; e.bias = L1.shift; e.ld = L1.C; e.w2 = L2.w; e.bias2 = L2.shift; e.ld2 = L2.C;
        e.N = op.N; e.C = op.C; e.K = op.K;
        break;
    }
    case OP_PAD8:
        e.x = d_input; e.y = sl.act[op.out];
        e.N = op.N; e.H = op.H; e.W = op.W; e.C = 3; e.k = op.K; e.Ho = op.conv.Ho; e.Wo = op.conv.Wo;
        break;
    case OP_IM2COL:
        e.x = d_input; e.y = sl.act[op.out];
        e.N = op.N; e.H = op.H; e.W = op.W; e.C = 3;
        e.Ho = op.conv.Ho; e.Wo = op.conv.Wo; e.k = op.conv.k; e.stride = op.conv.stride; e.KKp = op.K;
        break;
    default: break;
    }
    return e;
}

// Launches one op of a plan on `st`.
template <typename T>
sgs_status_t launch_op(sgs_supernet *net, Plan *plan, Op &op, const void *d_input, void *d_logits, cudaStream_t st) {
    const sgs_supernet::Slot &sl = net->slots[plan->slot];
    auto abuf = [&](int id) -> void * { return id < 0 ? const_cast<void *>(d_input) : sl.act[id]; };
    LayerRange range(net, op.layer, "layer without weights");
    switch (op.type) {
    case OP_CONV:
    case OP_DW: {
        ConvArgs a = op.conv;
        if (op.in < 0) a.x = d_input;
        a.cache_tbl = net->cache_tbl; a.layer = op.layer;
        a.ws = sl.ws; a.ws_elems = net->splitk_ws_elems;
        if (op.type == OP_DW) { CU(launch_dw<T>(a, st)); net->kernel_launches++; }
        else if (op.impl == 1) { int n = 0; CU(tc_conv_launch(*op.tc, a, st, &n)); net->kernel_launches += n; }
        else { CU(launch_conv_plain<T>(a, st)); net->kernel_launches++; }
        break;
    }
    case OP_PAD8:
    case OP_IM2COL: {
        SmallEntry e = small_entry(net, plan, op, d_input, d_logits);
        CU(launch_small(op.type, &e, nullptr, 1, st));
        net->kernel_launches++;
        break;
    }
    case OP_MAXPOOL:
        CU(launch_maxpool3s2<T>((const T *)abuf(op.in), (T *)sl.act[op.out], op.N, op.H, op.W, op.C, st));
        net->kernel_launches++;
        break;
    case OP_GAP:
        CU(launch_gap<T>((const T *)abuf(op.in), sl.vec[op.vout], op.N, op.H * op.W, op.C, st));
        net->kernel_launches++;
        break;
    case OP_SE_GATE: {
        const StoredLayer &L1 = net->layers[op.layer], &L2 = net->layers[op.layer2];
        CU(launch_se_gate<T>(sl.vec[op.vin], (const T *)L1.w, L1.shift, (const T *)L2.w, L2.shift, sl.vec[op.vout],
                             op.N, op.C, op.K, L1.C, L2.C, st));
        net->kernel_launches++;
        break;
    }
    case OP_SCALE:
        CU(launch_scale<T>((const T *)sl.act[op.in], sl.vec[op.vin], (T *)sl.act[op.out], op.N, op.H * op.W, op.C, st));
        net->kernel_launches++;
        break;
    case OP_LINEAR: {
        const StoredLayer &L = net->layers[op.layer];
        float *y = op.vout < 0 ? static_cast<float *>(d_logits) : sl.vec[op.vout];
        CU(launch_linear<T>(sl.vec[op.vin], (const T *)L.w, L.shift, y, op.N, op.C, op.K, L.C, op.act, st));
        net->kernel_launches++;
        break;
    }
    }
    return SGS_OK;
}

template <typename T>
sgs_status_t run_ops(sgs_supernet *net, Plan *plan, const void *d_input, void *d_logits, cudaStream_t st, size_t first,
                     size_t last) {
    for (size_t oi = first; oi < last; oi++) {
        Op &op = plan->ops[oi];
        if (net->profile) {
            // one event pair per op of the plan
            if (plan->prof_ev.size() != 2 * plan->ops.size()) {
                for (cudaEvent_t e : plan->prof_ev) cudaEventDestroy(e);
                plan->prof_ev.assign(2 * plan->ops.size(), nullptr);
                for (auto &e : plan->prof_ev) CU(cudaEventCreate(&e));
            }
            CU(cudaEventRecord(plan->prof_ev[2 * oi], st));
        }
        sgs_status_t rc = launch_op<T>(net, plan, op, d_input, d_logits, st);
        if (rc != SGS_OK) return rc;
        if (net->profile) CU(cudaEventRecord(plan->prof_ev[2 * oi + 1], st));
    }
    return SGS_OK;
}

// Adds the per-op durations of every plan run since the last fold to the per-class totals.  A plan
// that ran several times contributes its latest timestamps once per run.
void fold_profile(sgs_supernet *net) {
    if (net->prof_used.empty()) return;
    cudaDeviceSynchronize();
    for (Plan *plan : net->prof_used) {
        if (plan->prof_ev.size() != 2 * plan->ops.size()) continue;
        for (size_t oi = 0; oi < plan->ops.size(); oi++) {
            const Op &op = plan->ops[oi];
            const int cls = op.type == OP_CONV ? (op.impl == 1 ? 0 : 1) : op.type == OP_DW ? 2 : 3;
            float ms = 0;
            if (cudaEventElapsedTime(&ms, plan->prof_ev[2 * oi], plan->prof_ev[2 * oi + 1]) == cudaSuccess) {
                net->prof_ms[cls] += ms; net->prof_bytes[cls] += op.alg_bytes; net->prof_flops[cls] += op.flops;
                net->prof_launches[cls]++;
            }
        }
    }
    net->prof_used.clear();
}

void destroy_plan_resources(Plan *plan) {
    if (plan->graph) cudaGraphExecDestroy(plan->graph);
    plan->graph = nullptr;
    for (cudaEvent_t e : plan->prof_ev) cudaEventDestroy(e);
    plan->prof_ev.clear();
}

sgs_status_t run_plan(sgs_supernet *net, Plan *plan, const void *d_input, void *d_logits, cudaStream_t st, size_t first,
                      size_t last) {
    return net->dtype == SGS_BF16 ? run_ops<__nv_bfloat16>(net, plan, d_input, d_logits, st, first, last)
                                  : run_ops<float>(net, plan, d_input, d_logits, st, first, last);
}

// Brings the device copy of the cache table up to date with the host policy state.  The image is
// built in a pinned ring entry so that the copy is truly asynchronous.
sgs_status_t push_cache_table(sgs_supernet *net, cudaStream_t st) {
    const CacheState &cs = net->cache;
    if (net->cache_tbl_epoch == cs.epoch) return SGS_OK;
    const size_t n = 1 + 2 * net->layers.size();
    const int slot = net->tbl_ring_pos;
    net->tbl_ring_pos = (slot + 1) % 16;
    CU(cudaEventSynchronize(net->tbl_ring_ev[slot]));  // the upload that last used this entry (16 updates ago)
    int *tbl = net->tbl_ring + (size_t)slot * n;
    std::memset(tbl, 0, n * sizeof(int));
    if (cs.enabled && !cs.G.empty()) {
        tbl[0] = 1;
        for (size_t li = 0; li < net->layers.size(); li++) { tbl[1 + 2 * li] = cs.G[3 * li]; tbl[2 + 2 * li] = cs.G[3 * li + 1]; }
    } else if (!cs.enabled && cs.evict_first_when_off) {
        tbl[0] = 2;
    }
    CU(cudaMemcpyAsync(net->cache_tbl, tbl, n * sizeof(int), cudaMemcpyHostToDevice, st));
    CU(cudaEventRecord(net->tbl_ring_ev[slot], st));
    net->cache_tbl_epoch = cs.epoch;
    return SGS_OK;
}

// Run one query.  With graphs, the first op (reads the caller's input) and the last op (writes the
// caller's logits) are launched directly; everything between touches only buffers the handle owns and
// is replayed as one captured graph per plan, independent of the caller's pointers and of the cache
// state (kernels read the cache box from device memory).
sgs_status_t run_query(sgs_supernet *net, const sgs_subnet_cfg_t *cfg, const void *d_input, int batch, int res,
                       void *d_logits, cudaStream_t st, bool use_graph, int slot, Plan **plan_out) {
    Plan *plan = nullptr;
    sgs_status_t rc = get_plan(net, cfg, batch, res, slot, &plan);
    if (rc != SGS_OK) return rc;
    rc = ensure_workspace(net, plan->act_elems, batch);
    if (rc != SGS_OK) return rc;
    if (!plan->prepared) {
        rc = choose_impls(net, plan);
        if (rc != SGS_OK) return rc;
    }
    if (plan_out) *plan_out = plan;
    {
        const auto p0 = std::chrono::steady_clock::now();
        rc = push_cache_table(net, st);
        net->host_us_table += std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - p0).count();
    }
    if (rc != SGS_OK) return rc;
    const size_t n_ops = plan->ops.size();
    if (net->profile) net->prof_used.push_back(plan);
    if (!use_graph || net->profile || n_ops < 3) {
        long long before = net->kernel_launches;
        rc = run_plan(net, plan, d_input, d_logits, st, 0, n_ops);
        plan->launches = (int)(net->kernel_launches - before);
        return rc;
    }
    cudaGraphExec_t &graph = plan->graph;
    if (!graph) {
        cudaGraph_t g = nullptr;
        CU(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
        long long before = net->kernel_launches;
        rc = run_plan(net, plan, d_input, d_logits, st, 1, n_ops - 1);
        plan->launches = (int)(net->kernel_launches - before) + 2;
        net->kernel_launches = before;
        cudaError_t e = cudaStreamEndCapture(st, &g);
        if (rc != SGS_OK) { if (g) cudaGraphDestroy(g); return rc; }
        if (e != cudaSuccess) return fail(net, SGS_ECUDA, std::string("graph capture: ") + cudaGetErrorString(e));
        e = cudaGraphInstantiate(&graph, g, 0);
        cudaGraphDestroy(g);
        if (e != cudaSuccess) return fail(net, SGS_ECUDA, std::string("graph instantiate: ") + cudaGetErrorString(e));
    }
    long long before = net->kernel_launches;
    auto t0 = std::chrono::steady_clock::now();
    rc = run_plan(net, plan, d_input, d_logits, st, 0, 1);
    if (rc != SGS_OK) return rc;
    auto t1 = std::chrono::steady_clock::now();
    CU(cudaGraphLaunch(graph, st));
    auto t2 = std::chrono::steady_clock::now();
    rc = run_plan(net, plan, d_input, d_logits, st, n_ops - 1, n_ops);
    auto t3 = std::chrono::steady_clock::now();
    net->host_us_graph += std::chrono::duration<double, std::micro>(t2 - t1).count();
    net->host_us_direct += std::chrono::duration<double, std::micro>(t1 - t0).count() + std::chrono::duration<double, std::micro>(t3 - t2).count();
    net->kernel_launches = before + plan->launches;
    return rc;
}

// ------------------------------------------------------------------------------------------
// SubGraph cache policy (paper Section 2.2, 3.3, Appendix A.1 and A.4)
// ------------------------------------------------------------------------------------------
size_t layer_box_bytes(const sgs_supernet *net, int li, int K, int C, int k) {
    const StoredLayer &L = net->layers[li];
    size_t per = L.kind == KIND_DW ? (size_t)k * k : (size_t)C * k * k;
    return (size_t)K * per * net->elem();
}

// G = element-wise minimum of the encodings in the window (the exact intersection of those SubNets,
// because every slice is a prefix / centred window), kept layer by layer in network order while it
// fits the byte budget.
// Keeps the layers of `g` in network order while they fit the byte budget; returns the bytes kept.
size_t clip_to_budget(const sgs_supernet *net, std::vector<int> &g, size_t budget) {
    size_t used = 0;
    for (size_t li = 0; li < net->layers.size(); li++) {
        size_t b = layer_box_bytes(net, (int)li, g[3 * li], g[3 * li + 1], g[3 * li + 2]);
        if (used + b > budget) { g[3 * li] = g[3 * li + 1] = g[3 * li + 2] = 0; continue; }
        used += b;
    }
    return used;
}

void clip_candidates(sgs_supernet *net) {
    CacheState &cs = net->cache;
    cs.cand = cs.cand_raw;
    cs.cand_bytes.assign(cs.cand.size(), 0);
    for (size_t j = 0; j < cs.cand.size(); j++) cs.cand_bytes[j] = clip_to_budget(net, cs.cand[j], cs.budget);
}

// Algorithm 1's caching decision: AvgNet = mean of the window's encodings; the cached SubGraph becomes
// the candidate G_j with the smallest Euclidean distance to it on the (K_i, C_i) entries (Section 3.3).
// With Q = window length and S = element-wise sum, Q^2 * Dist^2 = sum_i (Q * G_ji - S_i)^2 is compared
// exactly in 64-bit integers; ties go to the lowest index.
int nearest_candidate(const std::deque<std::vector<int>> &window, const std::vector<std::vector<int>> &cand) {
    const long long Q = (long long)window.size();
    const size_t n = window.front().size();
    std::vector<long long> S(n, 0);
    for (const auto &e : window)
        for (size_t i = 0; i < n; i++) S[i] += e[i];
    int best = -1;
    unsigned long long best_d = 0;
    for (size_t j = 0; j < cand.size(); j++) {
        unsigned long long d = 0;
        for (size_t i = 0; i < n; i++) {
            if (i % 3 == 2) continue;  // the kernel-size entry takes no part in the distance
            long long t = Q * cand[j][i] - S[i];
            d += (unsigned long long)(t * t);
        }
        if (best < 0 || d < best_d) { best = (int)j; best_d = d; }
    }
    return best;
}

void choose_nearest_candidate(sgs_supernet *net) {
    CacheState &cs = net->cache;
    const int best = nearest_candidate(cs.window, cs.cand);
    cs.decisions++;
    cs.last_choice = best;
    if (cs.cand[best] != cs.G) { cs.G = cs.cand[best]; cs.epoch++; }
    cs.G_bytes = cs.cand_bytes[best];
}

void recompute_cached_subgraph(sgs_supernet *net) {
    CacheState &cs = net->cache;
    if (cs.window.empty()) return;
    if (cs.policy == 1 && !cs.cand.empty()) { choose_nearest_candidate(net); return; }
    std::vector<int> g = cs.window.front();
    for (const auto &e : cs.window)
        for (size_t i = 0; i < g.size(); i++) g[i] = std::min(g[i], e[i]);
    size_t used = clip_to_budget(net, g, cs.budget);
    cs.decisions++;
    if (g != cs.G) { cs.G = std::move(g); cs.epoch++; }
    cs.G_bytes = used;
}

struct QueryAccount { double weight_bytes = 0, miss_bytes = 0, hit_ratio = 0; };

QueryAccount account_query(const sgs_supernet *net, const std::vector<int> &sn) {
    const CacheState &cs = net->cache;
    QueryAccount a;
    double num = 0, den = 0;
    for (size_t li = 0; li < net->layers.size(); li++) {
        int K = sn[3 * li], C = sn[3 * li + 1], k = sn[3 * li + 2];
        if (!K) continue;
        size_t all = layer_box_bytes(net, (int)li, K, C, k), common = 0;
        int gK = 0, gC = 0;
        if (cs.enabled && !cs.G.empty()) {
            gK = std::min(K, cs.G[3 * li]); gC = std::min(C, cs.G[3 * li + 1]);
            int gk = std::min(k, cs.G[3 * li + 2]);
            common = layer_box_bytes(net, (int)li, gK, gC, gk);
        }
        a.weight_bytes += (double)all;
        a.miss_bytes += (double)(all - common);
        num += (double)gK * gK + (double)gC * gC;
        den += (double)K * K + (double)C * C;
    }
    a.hit_ratio = den > 0 ? std::sqrt(num) / std::sqrt(den) : 0;
    return a;
}

// The cached SubGraph becomes candidate j (anything outside [0, |S|) empties the cache) and stays until the
// next pin: observations no longer move it.
void cache_pin(sgs_supernet *net, int j) {
    CacheState &cs = net->cache;
    cs.enabled = true;
    cs.policy = 2;
    std::vector<int> g;
    size_t bytes = 0;
    if (j >= 0 && j < (int)cs.cand.size()) { g = cs.cand[j]; bytes = cs.cand_bytes[j]; }
    else j = -1;
    if (g != cs.G) { cs.G = std::move(g); cs.epoch++; }
    cs.G_bytes = bytes;
    cs.last_choice = j;
}

void cache_observe(sgs_supernet *net, const std::vector<int> &enc) {
    CacheState &cs = net->cache;
    if (cs.policy == 2) return;
    cs.window.push_back(enc);
    while ((int)cs.window.size() > cs.window_q) cs.window.pop_front();
    if (++cs.since_update >= cs.window_q) {
        cs.since_update = 0;
        recompute_cached_subgraph(net);
    }
}

void cache_reset(sgs_supernet *net, bool enabled, size_t budget, int window_q) {
    CacheState &cs = net->cache;
    cs.enabled = enabled;
    cs.window_q = std::max(1, window_q);
    size_t cap = net->persist_max ? net->persist_max : net->l2_bytes;
    cs.budget = budget ? std::min(budget, net->l2_bytes ? net->l2_bytes : budget) : cap;
    cs.window.clear();
    cs.G.clear();
    cs.G_bytes = 0;
    cs.since_update = 0;
    cs.decisions = 0;
    cs.last_choice = -1;
    cs.epoch++;
    clip_candidates(net);
}

}  // namespace

// =============================================================================================
// C interface
// =============================================================================================
extern "C" {

sgs_status_t sgs_supernet_load(const sgs_arch_desc_t *arch, const void *host_blob, size_t nbytes,
                               sgs_dtype_t compute_dtype, int device, sgs_supernet_t **out) {
    if (!arch || !host_blob || !out || nbytes < 32 || nbytes % 4) return SGS_EINVAL;
    if (compute_dtype != SGS_F32 && compute_dtype != SGS_BF16) return SGS_EINVAL;
    if (arch->family < SGS_TINY || arch->family > SGS_MBV3) return SGS_EINVAL;
    *out = nullptr;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device < 0 || device >= ndev) return SGS_ECUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return SGS_ECUDA;
    if (prop.major != 10) return SGS_EUNSUPPORTED;
    const uint32_t *words = static_cast<const uint32_t *>(host_blob);
    if (words[0] != BLOB_MAGIC || words[1] != 1u || (int)words[2] != arch->family) return SGS_EINVAL;

    std::unique_ptr<sgs_supernet> holder(new (std::nothrow) sgs_supernet);
    if (!holder) return SGS_ENOMEM;
    sgs_supernet *net = holder.get();
    net->family = arch->family; net->device = device; net->dtype = compute_dtype;
    net->def = family_def(arch->family);
    // optional cross-checks of the descriptor
    if (arch->n_stages && arch->n_stages != net->def.n_stages) return SGS_EINVAL;
    if (arch->n_classes && arch->n_classes != net->def.classes) return SGS_EINVAL;
    if (arch->stem_width && arch->stem_width != net->def.stem) return SGS_EINVAL;
    for (int s = 0; s < net->def.n_stages; s++) {
        if (arch->max_depth[s] && arch->max_depth[s] != net->def.max_depth[s]) return SGS_EINVAL;
        if (arch->base_width[s] && arch->base_width[s] != net->def.width[s]) return SGS_EINVAL;
    }
    DeviceGuard guard(device);
    if (!guard.ok) return SGS_ECUDA;

    // walk the records against the family definition
    std::vector<LayerSpec> specs = stored_layers(arch->family);
    if ((size_t)words[3] != specs.size()) return SGS_EINVAL;
    size_t pos = 8, total_words = nbytes / 4;
    struct Rec { size_t w_off, bn_off, bias_off; };
    std::vector<Rec> recs;
    size_t arena = 0, params = 0;
    for (const LayerSpec &sp : specs) {
        if (pos + 8 > total_words) return SGS_EINVAL;
        const uint32_t *h = words + pos;
        if ((int)h[0] != sp.kind || (int)h[1] != sp.K || (int)h[2] != sp.C || (int)h[3] != sp.R || (int)h[4] != sp.R ||
            (h[5] != 0) != sp.bn || (h[6] != 0) != sp.bias)
            return SGS_EINVAL;
        size_t nw = (size_t)sp.K * sp.C * sp.R * sp.R;
        const size_t nw_stored = (size_t)sp.K * stored_row(sp.kind, sp.C, compute_dtype) * sp.R * sp.R;
        Rec r{pos + 8, 0, 0};
        size_t q = pos + 8 + nw;
        if (sp.bn) { r.bn_off = q; q += 4 * (size_t)sp.K; }
        if (sp.bias) { r.bias_off = q; q += sp.K; }
        if (q > total_words) return SGS_EINVAL;
        pos = q;
        recs.push_back(r);
        arena += (nw_stored * (compute_dtype == SGS_BF16 ? 2 : 4) + 255) / 256 * 256;
        params += ((size_t)sp.K + 63) / 64 * 64 * 2;
    }
    if (pos != total_words) return SGS_EINVAL;

    sgs_status_t st;
    float *stage = nullptr;
    if ((st = dev_alloc(net, (void **)&stage, nbytes)) != SGS_OK) return st;
    auto cleanup_stage = [&]() { dev_free(net, stage, nbytes); };
    if ((st = dev_alloc(net, (void **)&net->weight_arena, arena)) != SGS_OK) { cleanup_stage(); sgs_supernet_free(holder.release()); return st; }
    net->weight_arena_bytes = arena;
    if ((st = dev_alloc(net, (void **)&net->param_arena, params * 4)) != SGS_OK) { cleanup_stage(); sgs_supernet_free(holder.release()); return st; }
    net->param_arena_bytes = params * 4;
    cudaError_t e = cudaMemcpy(stage, host_blob, nbytes, cudaMemcpyHostToDevice);
    size_t aoff = 0, poff = 0;
    const int bf = compute_dtype == SGS_BF16;
    for (size_t i = 0; i < specs.size() && e == cudaSuccess; i++) {
        const LayerSpec &sp = specs[i];
        StoredLayer L;
        L.kind = sp.kind; L.K = sp.K; L.C = sp.C; L.R = sp.R; L.S = sp.R; L.has_bn = sp.bn; L.has_bias = sp.bias; L.name = sp.name;
        size_t nw = (size_t)sp.K * sp.C * sp.R * sp.R;
        L.Cp = stored_row(sp.kind, sp.C, compute_dtype);
        L.w = net->weight_arena + aoff;
        L.w_bytes = nw * net->elem();
        aoff += ((size_t)sp.K * L.Cp * sp.R * sp.R * net->elem() + 255) / 256 * 256;
        L.scale = net->param_arena + poff;
        L.shift = L.scale + ((size_t)sp.K + 63) / 64 * 64;
        poff += ((size_t)sp.K + 63) / 64 * 64 * 2;
        const float *src = stage + recs[i].w_off;
        if (sp.kind == KIND_CONV) e = launch_relayout_conv(src, L.w, sp.K, sp.C, L.Cp, sp.R, sp.R, bf, 0);
        else if (sp.kind == KIND_DW) e = launch_relayout_dw(src, L.w, sp.K, sp.R, sp.R, bf, 0);
        else e = launch_convert(src, L.w, nw, bf, 0);
        if (e != cudaSuccess) break;
        const float *bn = sp.bn ? stage + recs[i].bn_off : nullptr;
        const float *bias = sp.bias ? stage + recs[i].bias_off : nullptr;
        e = launch_fold_bn(bn, bn ? bn + sp.K : nullptr, bn ? bn + 2 * sp.K : nullptr, bn ? bn + 3 * sp.K : nullptr, bias,
                           L.scale, L.shift, sp.K, 0);
        net->by_name[sp.name] = (int)net->layers.size();
        net->layers.push_back(L);
    }
    if (e == cudaSuccess && bf && !net->layers.empty() && net->layers[0].kind == KIND_CONV && net->layers[0].C == 3) {
        const StoredLayer &L = net->layers[0];
        const int KK = L.R * L.R * 3;
        net->stem_kkp = (KK + 7) / 8 * 8;
        if (dev_alloc(net, &net->stem_gemm_w, (size_t)L.K * net->stem_kkp * 2) != SGS_OK) e = cudaErrorMemoryAllocation;
        else e = launch_stem_gemm_weights(L.w, net->stem_gemm_w, L.K, KK, net->stem_kkp, 0);
        if (e == cudaSuccess && L.R <= 8) {
            if (dev_alloc(net, &net->stem_win_w, (size_t)L.K * L.R * 64 * 2) != SGS_OK) e = cudaErrorMemoryAllocation;
            else e = launch_stem_window_weights(L.w, net->stem_win_w, L.K, L.R, 0);
        }
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    cleanup_stage();
    if (e != cudaSuccess) { sgs_supernet_free(holder.release()); return e == cudaErrorMemoryAllocation ? SGS_ENOMEM : SGS_ECUDA; }

    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, device) == cudaSuccess && v > 0) net->sms = v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrL2CacheSize, device) == cudaSuccess) net->l2_bytes = (size_t)v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxPersistingL2CacheSize, device) == cudaSuccess) net->persist_max = (size_t)v;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxAccessPolicyWindowSize, device) == cudaSuccess) net->window_max = (size_t)v;
    {
        size_t n = 1 + 2 * net->layers.size();
        bool ok = dev_alloc(net, (void **)&net->cache_tbl, n * sizeof(int)) == SGS_OK &&
                  cudaMemset(net->cache_tbl, 0, n * sizeof(int)) == cudaSuccess &&
                  cudaMallocHost((void **)&net->tbl_ring, 16 * n * sizeof(int)) == cudaSuccess;
        for (int i = 0; i < 16 && ok; i++) ok = cudaEventCreateWithFlags(&net->tbl_ring_ev[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            sgs_supernet_free(holder.release());
            return SGS_ENOMEM;
        }
    }
    if (compute_dtype == SGS_BF16 && tc_available() && tc_conv_init(device) != cudaSuccess) {
        sgs_supernet_free(holder.release());
        return SGS_ECUDA;
    }
    cache_reset(net, false, 0, 4);
    *out = holder.release();
    return SGS_OK;
}

void sgs_supernet_free(sgs_supernet_t *net) {
    if (!net) return;
    DeviceGuard guard(net->device);
    cudaDeviceSynchronize();
    for (auto &kv : net->plans) destroy_plan_resources(kv.second.get());
    net->plans.clear();
    net->prof_used.clear();
    cudaFree(net->weight_arena);
    cudaFree(net->param_arena);
    cudaFree(net->stem_gemm_w);
    cudaFree(net->stem_win_w);
    for (auto &sl : net->slots) {
        for (int i = 0; i < 4; i++) cudaFree(sl.act[i]);
        for (int i = 0; i < 3; i++) cudaFree(sl.vec[i]);
        cudaFree(sl.ws);
        cudaFree(sl.stage_in);
        cudaFree(sl.stage_out);
        if (sl.ev) cudaEventDestroy(sl.ev);
        if (sl.st) cudaStreamDestroy(sl.st);
    }
    for (auto &w : net->waves) {
        cudaFree(w.d_tbl);
        cudaFreeHost(w.h_tbl);
        cudaFree(w.stage_in);
        cudaFree(w.stage_out);
        if (w.done) cudaEventDestroy(w.done);
        if (w.st) cudaStreamDestroy(w.st);
    }
    cudaFree(net->pq_scratch);
    cudaFree(net->pq_d_tbl);
    cudaFreeHost(net->pq_h_tbl);
    cudaFree(net->pq_counter);
    cudaFree(net->pq_stage_in);
    cudaFree(net->pq_stage_out);
    cudaFree(net->cache_tbl);
    cudaFreeHost(net->tbl_ring);
    for (int i = 0; i < 16; i++)
        if (net->tbl_ring_ev[i]) cudaEventDestroy(net->tbl_ring_ev[i]);
    delete net;
}

sgs_status_t sgs_subnet_validate(const sgs_supernet_t *net, const sgs_subnet_cfg_t *cfg) {
    if (!net || !cfg) return SGS_EINVAL;
    return cfg_valid(net, cfg) ? SGS_OK : fail(net, SGS_ECONFIG, "SubNet config outside the elastic sets of this SuperNet");
}

int sgs_num_layers(const sgs_supernet_t *net) { return net ? (int)net->layers.size() : 0; }

sgs_status_t sgs_subnet_encode(const sgs_supernet_t *net, const sgs_subnet_cfg_t *cfg, int *out) {
    if (!net || !cfg || !out) return SGS_EINVAL;
    if (!cfg_valid(net, cfg)) return fail(net, SGS_ECONFIG, "SubNet config outside the elastic sets of this SuperNet");
    std::vector<int> e = encoding_of(slices_for(net, cfg));
    std::memcpy(out, e.data(), e.size() * sizeof(int));
    return SGS_OK;
}

sgs_status_t sgs_subnet_cost(const sgs_supernet_t *cnet, const sgs_subnet_cfg_t *cfg, int batch, int res, double *flops,
                             double *weight_bytes, double *activation_bytes) {
    sgs_supernet *net = const_cast<sgs_supernet *>(cnet);
    if (!net || !cfg || batch <= 0 || res <= 0) return SGS_EINVAL;
    if (!cfg_valid(net, cfg)) return fail(net, SGS_ECONFIG, "SubNet config outside the elastic sets of this SuperNet");
    Plan p;
    sgs_status_t st = build_plan(net, cfg, batch, res, &p);
    if (st != SGS_OK) return st;
    if (flops) *flops = p.flops;
    if (weight_bytes) *weight_bytes = p.weight_bytes;
    if (activation_bytes) *activation_bytes = p.act_bytes;
    return SGS_OK;
}

sgs_status_t sgs_subnet_run(sgs_supernet_t *net, const sgs_subnet_cfg_t *cfg, const void *d_input, int batch, int res,
                            void *d_logits, void *cuda_stream) {
    if (!net) return SGS_EINVAL;
    if (!cfg || !d_input || !d_logits || batch <= 0 || res < 8 || res > 1024) return fail(net, SGS_EINVAL, "bad argument");
    DeviceGuard guard(net->device);
    if (!guard.ok) return fail(net, SGS_ECUDA, "cudaSetDevice failed");
    Plan *plan = nullptr;
    sgs_status_t rc = run_query(net, cfg, d_input, batch, res, d_logits, (cudaStream_t)cuda_stream, false, 0, &plan);
    if (rc != SGS_OK) return rc;
    if (net->cache.enabled) cache_observe(net, plan->enc);
    return SGS_OK;
}

// ------------------------------------------------------------------------------------------
// Wave execution of a stream.  `G` consecutive queries form a wave; the wave walks the op list of the
// largest SubNet, and at every position the members whose SubNet has that op run it together: the
// tensor-core convolutions of all members are ONE grouped launch (sgs_conv_group.cu), the remaining op
// types are launched per member.  Up to `W` waves are in flight on their own streams.
// ------------------------------------------------------------------------------------------
static sgs_status_t ensure_waves(sgs_supernet *net, int W) {
    while ((int)net->waves.size() < W) {
        sgs_supernet::WaveCtx w;
        CU(cudaStreamCreateWithFlags(&w.st, cudaStreamNonBlocking));
        CU(cudaEventCreateWithFlags(&w.done, cudaEventDisableTiming));
        net->waves.push_back(w);
    }
    return SGS_OK;
}

static sgs_status_t wave_impl(sgs_supernet_t *net, int n_queries, const sgs_subnet_cfg_t *cfgs, const void *inputs, int batch,
                              int res, void *logits, const sgs_stream_opts_t &o, sgs_stream_stats_t *stats, cudaStream_t st,
                              bool host_buffers) {
    const int G = std::min(o.wave, TC_GROUP_MAX_ENTRIES);
    // per-launch timing (option "profile") wants the launches of one wave at a time
    const int W = net->profile ? 1 : std::max(1, std::min(o.concurrency ? o.concurrency : 2, 8));
    struct ProfRec { cudaEvent_t e0, e1; int cls; double bytes, flops; int layer, members, tiles; };
    std::vector<ProfRec> prof;
    sgs_status_t rc = ensure_slots(net, G * W);
    if (rc != SGS_OK) return rc;
    if ((rc = ensure_waves(net, W)) != SGS_OK) return rc;
    if ((rc = ensure_ranks(net)) != SGS_OK) return rc;
    net->throughput_mode = 2;
    if (net->cache.enabled && net->cache_mech != 0 && net->persist_max) {
        // the window mechanism keeps its lines in the L2 carve-out for persisting accesses: size it to the budget
        // (a limit of this process's context; lines of an earlier stream go back to normal first)
        const size_t want = std::min(net->cache.budget, net->persist_max);
        if (want != net->persist_limit_set) {
            CU(cudaDeviceSetLimit(cudaLimitPersistingL2CacheSize, want));
            net->persist_limit_set = want;
        }
        cudaCtxResetPersistingL2Cache();
    }
    const size_t in_bytes = (size_t)batch * res * res * 3 * net->elem();
    const size_t out_bytes = (size_t)batch * net->def.classes * sizeof(float);
    const int n_ranks = (int)net->op_rank.size();
    const int n_waves = (n_queries + G - 1) / G;
    std::vector<cudaEvent_t> ev;  // per wave: start and end on the wave's stream
    if (o.record_latency) {
        ev.resize(2 * (size_t)n_waves);
        for (auto &e : ev) CU(cudaEventCreate(&e));
    }
    cudaEvent_t e0, e1;
    CU(cudaEventCreate(&e0));
    CU(cudaEventCreate(&e1));
    const long long launches0 = net->kernel_launches;
    const int hits0 = net->plan_hits, miss0 = net->plan_misses;
    double flops = 0, wbytes = 0, miss_bytes = 0, hit = 0;
    int updates = 0;
    CU(cudaEventRecord(e0, st));
    for (int w = 0; w < W; w++) { CU(cudaStreamWaitEvent(net->waves[w].st, e0, 0)); net->waves[w].busy = false; }
    const auto host_t0 = std::chrono::steady_clock::now();
    std::vector<Plan *> plans((size_t)G);
    std::vector<std::shared_ptr<const std::vector<int>>> boxes((size_t)G);  // per member: the cached SubGraph its query is served under
    std::vector<int> box_epoch((size_t)G, -1);
    std::vector<std::vector<std::pair<int, int>>> buckets((size_t)n_ranks);  // per rank: (member, op index)
    struct Launch { int rank; GroupLaunch *group; int small_kind; size_t off; int count; int rank2 = -1; };  // rank2: a second bucket merged into this launch;  // group == nullptr && small_kind < 0: the bucket's ungrouped ops, per member
    std::vector<Launch> launches;
    std::vector<char> merged;  // per rank: its bucket went into the previous bucket's launch
    for (int wv = 0; wv < n_waves && rc == SGS_OK; wv++) {
        const int ci = wv % W, q0 = wv * G, members = std::min(G, n_queries - q0);
        auto tick = [](std::chrono::steady_clock::time_point &t0) {
            const auto now = std::chrono::steady_clock::now();
            const double us = std::chrono::duration<double, std::micro>(now - t0).count();
            t0 = now;
            return us;
        };
        auto tp = std::chrono::steady_clock::now();
        // plans of the members (each member owns slot ci * G + m)
        for (int m = 0; m < members && rc == SGS_OK; m++) {
            rc = get_plan(net, &cfgs[q0 + m], batch, res, ci * G + m, &plans[m]);
            if (rc == SGS_OK) rc = ensure_workspace(net, plans[m]->act_elems, batch);
        }
        // members whose plan is new: tensor maps and tile choices.  (Preparing them on several host threads at once was
        // measured slower, 102 us against 67 us per never-seen config: the driver's tensor-map encoder serialises.)
        for (int m = 0; m < members && rc == SGS_OK; m++)
            if (!plans[m]->prepared) rc = choose_impls(net, plans[m]);
        if (rc != SGS_OK) break;
        net->host_us_query += tick(tp);
        sgs_supernet::WaveCtx &cx = net->waves[ci];  // (taken after ensure_*: the vector does not move later)
        if (cx.busy) CU(cudaEventSynchronize(cx.done));  // its table image and staging buffers are free again
        net->host_us_direct += tick(tp);
        if (host_buffers) {
            const size_t need_in = (size_t)G * in_bytes, need_out = (size_t)G * out_bytes;
            if (cx.stage_in_bytes < need_in) {
                dev_free(net, cx.stage_in, cx.stage_in_bytes); cx.stage_in = nullptr; cx.stage_in_bytes = 0;
                if ((rc = dev_alloc(net, &cx.stage_in, need_in)) != SGS_OK) break;
                cx.stage_in_bytes = need_in;
            }
            if (cx.stage_out_bytes < need_out) {
                dev_free(net, cx.stage_out, cx.stage_out_bytes); cx.stage_out = nullptr; cx.stage_out_bytes = 0;
                if ((rc = dev_alloc(net, (void **)&cx.stage_out, need_out)) != SGS_OK) break;
                cx.stage_out_bytes = need_out;
            }
        }
        // Accounting and cache policy follow the stream order.  Every member keeps the cached SubGraph that is in
        // force when its query is served (snapshots are shared between the members of one caching decision): its
        // convolutions carry that box in their launch records, so the L2 hints of a wave change with the policy
        // from one member to the next, not from one wave to the next.
        const int epoch_at_issue = net->cache.epoch;
        for (int m = 0; m < members; m++) {
            const int epoch_before = net->cache.epoch;
            if (!boxes[m] || box_epoch[m] != epoch_before) {
                if (m > 0 && box_epoch[m - 1] == epoch_before && boxes[m - 1]) boxes[m] = boxes[m - 1];
                else boxes[m] = std::make_shared<const std::vector<int>>(net->cache.enabled ? net->cache.G : std::vector<int>());
                box_epoch[m] = epoch_before;
            }
            QueryAccount qa = account_query(net, plans[m]->enc);
            flops += plans[m]->flops; wbytes += qa.weight_bytes; miss_bytes += qa.miss_bytes; hit += qa.hit_ratio;
            if (net->cache.enabled) {
                cache_observe(net, plans[m]->enc);
                if (net->cache.epoch != epoch_before) updates++;
            }
        }
        // persisting L2 lines of SubGraphs that are no longer cached go back to normal replacement
        if (net->cache.enabled && net->cache_mech != 0 && net->cache.epoch != epoch_at_issue) cudaCtxResetPersistingL2Cache();
        const int box_policy = !net->cache.enabled ? (net->cache.evict_first_when_off ? 2 : 0) : (net->cache_mech == 1 ? 3 : 1);
        auto set_box = [&](ConvArgs &a, int member, int layer) {
            a.weight_policy = box_policy; a.cacheK = a.cacheC = 0;
            const std::vector<int> &G = *boxes[(size_t)member];
            if ((box_policy == 1 || box_policy == 3) && !G.empty()) { a.cacheK = G[3 * (size_t)layer]; a.cacheC = G[3 * (size_t)layer + 1]; }
            else if (box_policy == 1 || box_policy == 3) a.weight_policy = 0;
        };
        // merge the members' op lists by rank
        for (auto &b : buckets) b.clear();
        size_t n_tc = 0;
        for (int m = 0; m < members; m++)
            for (size_t oi = 0; oi < plans[m]->ops.size(); oi++) {
                buckets[(size_t)plans[m]->ops[oi].rank].emplace_back(m, (int)oi);
                n_tc += plans[m]->ops[oi].impl == 1 && plans[m]->ops[oi].type == OP_CONV;
            }
        size_t n_small = 0;
        for (int m = 0; m < members; m++) n_small += plans[m]->ops.size();
        const size_t need_tbl = (n_tc + 2 * n_small) * TC_GROUP_ENTRY_BYTES + 256;  // (depthwise records take two slots)
        if (cx.tbl_bytes < need_tbl) {
            cudaFreeHost(cx.h_tbl); cx.h_tbl = nullptr;
            dev_free(net, cx.d_tbl, cx.tbl_bytes); cx.d_tbl = nullptr; cx.tbl_bytes = 0;
            const size_t bytes = need_tbl * 2;
            if (cudaMallocHost((void **)&cx.h_tbl, bytes) != cudaSuccess) { rc = fail(net, SGS_ENOMEM, "pinned launch table"); break; }
            if ((rc = dev_alloc(net, (void **)&cx.d_tbl, bytes)) != SGS_OK) break;
            cx.tbl_bytes = bytes;
        }
        const void *din0 = static_cast<const char *>(inputs) + (size_t)q0 * in_bytes;
        void *dout0 = static_cast<char *>(logits) + (size_t)q0 * out_bytes;
        // tables and parameter blocks of the grouped launches
        launches.clear();
        size_t off = 0, used = 0;
        auto next_group = [&]() -> GroupLaunch * {
            if (used == net->group_pool.size()) net->group_pool.emplace_back(new GroupLaunch);
            GroupLaunch *g = net->group_pool[used++].get();
            g->reset(cx.d_tbl + off);
            return g;
        };
        merged.assign((size_t)n_ranks, 0);
        for (int r = 0; r < n_ranks; r++) {
            const auto &b = buckets[(size_t)r];
            if (b.empty() || merged[(size_t)r]) continue;
            GroupLaunch *g = nullptr;
            const size_t first_launch = launches.size();
            // Members with at most 64 output pixels can share a tile in pairs if one's slice (filters and channels)
            // contains the other's, and a pair is two consecutive records: order such a bucket so that every
            // member is followed by the largest not yet placed member it contains.
            std::vector<std::pair<int, int>> order(b.begin(), b.end());
            {
                const Op &o0 = plans[b[0].first]->ops[(size_t)b[0].second];
                if (o0.type == OP_CONV && o0.impl == 1 && (long long)o0.conv.N * o0.conv.Ho * o0.conv.Wo <= 64 && b.size() > 2) {
                    auto opof = [&](const std::pair<int, int> &mo) -> const Op & { return plans[mo.first]->ops[(size_t)mo.second]; };
                    std::stable_sort(order.begin(), order.end(), [&](const std::pair<int, int> &x, const std::pair<int, int> &y) {
                        const ConvArgs &cx_ = opof(x).conv, &cy_ = opof(y).conv;
                        return cx_.K != cy_.K ? cx_.K > cy_.K : cx_.C > cy_.C;
                    });
                    std::vector<std::pair<int, int>> placed;
                    std::vector<char> used_m(order.size(), 0);
                    for (size_t i = 0; i < order.size(); i++) {
                        if (used_m[i]) continue;
                        used_m[i] = 1;
                        placed.push_back(order[i]);
                        for (size_t j = i + 1; j < order.size(); j++) {
                            if (used_m[j] || opof(order[j]).conv.C > opof(order[i]).conv.C) continue;
                            used_m[j] = 1;
                            placed.push_back(order[j]);
                            break;
                        }
                    }
                    order.swap(placed);
                }
            }
            for (const auto &mo : order) {
                Plan *pl = plans[mo.first];
                const Op &op = pl->ops[(size_t)mo.second];
                if (op.type != OP_CONV || op.impl != 1) continue;  // launched per member below
                if (!g || !g->fits(*op.tc)) { g = next_group(); launches.push_back({r, g, -1, 0, 0}); }
                ConvArgs a = op.conv;
                a.layer = op.layer;
                set_box(a, mo.first, op.layer);
                g->add(cx.h_tbl + off, *op.tc, a);
                off += TC_GROUP_ENTRY_BYTES;
            }
            // Two consecutive convolution layers that do not depend on each other (a block's projection
            // shortcut and its first convolution both read the block input) share one launch when they fit.
            if (g && launches.size() == first_launch + 1) {
                int r2 = r + 1;
                while (r2 < n_ranks && buckets[(size_t)r2].empty()) r2++;
                if (r2 < n_ranks) {
                    auto all_tc = [&](const std::vector<std::pair<int, int>> &bb) {
                        for (const auto &mo : bb) {
                            const Op &op = plans[mo.first]->ops[(size_t)mo.second];
                            if (op.type != OP_CONV || op.impl != 1) return false;
                        }
                        return true;
                    };
                    const auto &b2 = buckets[(size_t)r2];
                    bool ok = all_tc(b) && all_tc(b2) && g->members() + (int)b2.size() <= TC_GROUP_MAX_ENTRIES;
                    for (const auto &m2 : b2) {
                        if (!ok) break;
                        const Op &o2 = plans[m2.first]->ops[(size_t)m2.second];
                        for (const auto &m1 : b) {
                            if (m1.first != m2.first) continue;
                            const Op &o1 = plans[m1.first]->ops[(size_t)m1.second];
                            // same member: no read-after-write, write-after-read or write-after-write between them
                            if (o2.in == o1.out || o2.res == o1.out || o2.out == o1.out || o2.out == o1.in || (o1.res >= 0 && o2.out == o1.res)) ok = false;
                        }
                    }
                    if (ok) {
                        // (fits() also bounds the tensor maps; checked entry by entry, undone as a whole is not
                        // possible, so test the worst case first: 5 maps per member)
                        ok = g->members() + (int)b2.size() <= TC_GROUP_MAX_ENTRIES && g->maps() + 5 * (int)b2.size() <= TC_GROUP_MAPS_LARGE;
                    }
                    if (ok) {
                        for (const auto &mo : b2) {
                            const Op &op = plans[mo.first]->ops[(size_t)mo.second];
                            ConvArgs a = op.conv;
                            a.layer = op.layer;
                            set_box(a, mo.first, op.layer);
                            g->add(cx.h_tbl + off, *op.tc, a);
                            off += TC_GROUP_ENTRY_BYTES;
                        }
                        launches.back().rank2 = r2;
                        merged[(size_t)r2] = 1;
                    }
                }
            }
            // max pool / average pool / linear / patch matrix: one launch over the members when every
            // member's op has the vectorised form; the remaining ops run member by member
            const Op &op0 = plans[b[0].first]->ops[(size_t)b[0].second];
            const int kind = op0.type;
            bool grouped = kind == OP_MAXPOOL || kind == OP_GAP || kind == OP_LINEAR || kind == OP_IM2COL || kind == OP_SCALE || kind == OP_SE_GATE || kind == OP_PAD8;
            if (grouped) {
                const size_t off0 = off;
                for (const auto &mo : b) {
                    const void *xin = static_cast<const char *>(host_buffers ? cx.stage_in : din0) + (size_t)mo.first * in_bytes;
                    void *yout = static_cast<char *>(host_buffers ? (void *)cx.stage_out : dout0) + (size_t)mo.first * out_bytes;
                    SmallEntry se = small_entry(net, plans[mo.first], plans[mo.first]->ops[(size_t)mo.second], xin, yout);
                    grouped = grouped && small_supported(kind, se);
                    std::memcpy(cx.h_tbl + off, &se, sizeof se);
                    off += sizeof se;
                }
                if (grouped) { launches.push_back({r, nullptr, kind, off0, (int)b.size()}); continue; }
                off = off0;
            }
            if (kind == OP_DW) {
                // depthwise: all members share a launch, ordered by kernel size (stride, activation and image
                // size are the layer's); a member the vectorised kernels do not take sends the bucket back
                // to member-by-member launches
                const size_t off0 = off;
                const size_t l0 = launches.size();
                bool ok = true;
                int total_dw = 0;
                for (int kk : {3, 5, 7}) {
                    const size_t offk = off;
                    int cnt = 0;
                    for (const auto &mo : b) {
                        const Op &op = plans[mo.first]->ops[(size_t)mo.second];
                        if (op.conv.k != kk) continue;
                        ConvArgs a = op.conv;
                        a.layer = op.layer;
                        std::memcpy(cx.h_tbl + off, &a, sizeof a);
                        off += DW_ENTRY_BYTES;
                        cnt++;
                    }
                    (void)offk;
                    total_dw += cnt;
                }
                // one launch for the layer: blocks pick the kernel body of their member's kernel size
                if (total_dw) launches.push_back({r, nullptr, OP_DW, off0, total_dw});
                size_t total = 0;
                for (size_t i = l0; i < launches.size(); i++) total += (size_t)launches[i].count;
                ok = total == b.size() && net->dtype == SGS_BF16;
                for (size_t i = l0; i < launches.size() && ok; i++) {
                    // dry check with the launcher's own rules (it launches nothing when it refuses)
                    const ConvArgs &a0 = *reinterpret_cast<const ConvArgs *>(cx.h_tbl + launches[i].off);
                    ok = a0.K % 8 == 0 && (long long)a0.N * launches[i].count <= 65535;
                }
                if (ok) continue;
                launches.resize(l0);
                off = off0;
            }
            launches.push_back({r, nullptr, -1, 0, 0});  // the bucket's remaining ops, member by member
        }
        net->host_us_table += tick(tp);
        cudaStream_t ws = cx.st;
        const void *din = din0;
        void *dout = dout0;
        if (off) CU(cudaMemcpyAsync(cx.d_tbl, cx.h_tbl, off, cudaMemcpyHostToDevice, ws));
        if ((rc = push_cache_table(net, ws)) != SGS_OK) break;
        if (o.record_latency) CU(cudaEventRecord(ev[2 * (size_t)wv], ws));
        if (host_buffers) {
            CU(cudaMemcpyAsync(cx.stage_in, din, (size_t)members * in_bytes, cudaMemcpyHostToDevice, ws));
            din = cx.stage_in;
        }
        // Profiling brackets every launch with events.  A sleeping kernel first holds the stream while the
        // host queues the whole wave, so that the intervals hold device time, not launch latency.
        if (net->profile) CU(launch_delay(1500, ws));
        auto prof_begin = [&](int cls, double bytes, double fl, int layer, int members, int tiles) -> sgs_status_t {
            if (!net->profile) return SGS_OK;
            ProfRec r{nullptr, nullptr, cls, bytes, fl, layer, members, tiles};
            CU(cudaEventCreate(&r.e0));
            CU(cudaEventCreate(&r.e1));
            CU(cudaEventRecord(r.e0, ws));
            prof.push_back(r);
            return SGS_OK;
        };
        auto prof_end = [&]() -> sgs_status_t {
            if (net->profile) CU(cudaEventRecord(prof.back().e1, ws));
            return SGS_OK;
        };
        auto first_layer = [&](int rank) -> int {  // stored layer of the launch's first member (-1: an op without weights)
            const auto &b = buckets[(size_t)rank];
            return b.empty() ? -1 : plans[b.front().first]->ops[(size_t)b.front().second].layer;
        };
        auto bucket_cost = [&](int rank, bool tc, double *bytes, double *fl) {
            *bytes = 0; *fl = 0;
            for (const auto &mo : buckets[(size_t)rank]) {
                const Op &op = plans[mo.first]->ops[(size_t)mo.second];
                if ((op.type == OP_CONV && op.impl == 1) != tc) continue;
                *bytes += op.alg_bytes; *fl += op.flops;
            }
        };
        void *dlog = host_buffers ? (void *)cx.stage_out : dout;
        for (const Launch &L : launches) {
            double pb = 0, pf = 0;
            LayerRange range(net, first_layer(L.rank), "layer without weights");
            if (L.group) {
                // (a bucket split over several launches books its whole cost on each: buckets of more than
                // 64 members or 248 tensor maps do not occur while profiling waves of <= 64)
                bucket_cost(L.rank, true, &pb, &pf);
                if (L.rank2 >= 0) { double b2 = 0, f2 = 0; bucket_cost(L.rank2, true, &b2, &f2); pb += b2; pf += f2; }
                if ((rc = prof_begin(0, pb, pf, first_layer(L.rank), L.group->members(), L.group->tiles())) != SGS_OK) break;
                CU(L.group->launch(net->cache.enabled && net->cache_mech != 0 ? net->window_max : 0, net->sms, ws));
                if ((rc = prof_end()) != SGS_OK) break;
                net->kernel_launches++;
                continue;
            }
            if (L.small_kind == OP_DW) {
                bucket_cost(L.rank, false, &pb, &pf);
                if ((rc = prof_begin(2, pb, pf, first_layer(L.rank), L.count, 0)) != SGS_OK) break;
                cudaError_t de = launch_dw_group(cx.h_tbl + L.off, cx.d_tbl + L.off, L.count, ws);
                if (de == cudaErrorNotSupported) {
                    // (not expected after the checks above) run these members one by one
                    for (int i = 0; i < L.count && rc == SGS_OK; i++) {
                        const ConvArgs &a = *reinterpret_cast<const ConvArgs *>(cx.h_tbl + L.off + (size_t)i * DW_ENTRY_BYTES);
                        CU(launch_dw<__nv_bfloat16>(a, ws));
                        net->kernel_launches++;
                    }
                } else {
                    CU(de);
                    net->kernel_launches++;
                }
                if ((rc = prof_end()) != SGS_OK) break;
                continue;
            }
            if (L.small_kind >= 0) {
                bucket_cost(L.rank, false, &pb, &pf);
                if ((rc = prof_begin(3, pb, pf, first_layer(L.rank), L.count, 0)) != SGS_OK) break;
                CU(launch_small(L.small_kind, reinterpret_cast<const SmallEntry *>(cx.h_tbl + L.off),
                                reinterpret_cast<const SmallEntry *>(cx.d_tbl + L.off), L.count, ws));
                if ((rc = prof_end()) != SGS_OK) break;
                net->kernel_launches++;
                continue;
            }
            for (const auto &mo : buckets[(size_t)L.rank]) {
                Plan *pl = plans[mo.first];
                Op &op = pl->ops[(size_t)mo.second];
                if (op.type == OP_CONV && op.impl == 1) continue;
                const void *xin = static_cast<const char *>(din) + (size_t)mo.first * in_bytes;
                void *yout = static_cast<char *>(dlog) + (size_t)mo.first * out_bytes;
                rc = net->dtype == SGS_BF16 ? launch_op<__nv_bfloat16>(net, pl, op, xin, yout, ws) : launch_op<float>(net, pl, op, xin, yout, ws);
                if (rc != SGS_OK) break;
            }
            if (rc != SGS_OK) break;
        }
        if (rc != SGS_OK) break;
        if (host_buffers) CU(cudaMemcpyAsync(dout, cx.stage_out, (size_t)members * out_bytes, cudaMemcpyDeviceToHost, ws));
        if (o.record_latency) CU(cudaEventRecord(ev[2 * (size_t)wv + 1], ws));
        CU(cudaEventRecord(cx.done, ws));
        cx.busy = true;
        net->host_us_graph += tick(tp);
    }
    net->host_us_stream += std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - host_t0).count();
    for (int w = 0; w < W; w++) {  // join
        cudaEventRecord(net->waves[w].done, net->waves[w].st);
        cudaStreamWaitEvent(st, net->waves[w].done, 0);
    }
    cudaError_t ce = cudaEventRecord(e1, st);
    cudaError_t se = cudaStreamSynchronize(st);
    if (rc == SGS_OK && (ce != cudaSuccess || se != cudaSuccess))
        rc = fail(net, SGS_ECUDA, std::string("stream: ") + cudaGetErrorString(se != cudaSuccess ? se : ce));
    if (rc != SGS_OK) cudaDeviceSynchronize();
    for (ProfRec &r : prof) {
        float ms = 0;
        if (rc == SGS_OK && r.e1 && cudaEventElapsedTime(&ms, r.e0, r.e1) == cudaSuccess) {
            net->prof_ms[r.cls] += ms; net->prof_bytes[r.cls] += r.bytes; net->prof_flops[r.cls] += r.flops; net->prof_launches[r.cls]++;
            if (net->prof_trace.size() < 65536) {
                sgs_launch_record_t tr;
                tr.kernel_class = r.cls; tr.layer = r.layer; tr.members = r.members; tr.tiles = r.tiles;
                tr.ms = ms; tr.alg_bytes = r.bytes; tr.flops = r.flops;
                net->prof_trace.push_back(tr);
            }
        }
        if (r.e0) cudaEventDestroy(r.e0);
        if (r.e1) cudaEventDestroy(r.e1);
    }
    if (rc == SGS_OK && tc_conv_status()) rc = fail(net, SGS_ETIMEOUT, "a bounded device-side wait ran out in the tensor-core kernel");
    if (rc == SGS_OK && stats) {
        std::memset(stats, 0, sizeof(*stats));
        float ms = 0;
        cudaEventElapsedTime(&ms, e0, e1);
        stats->n_queries = n_queries;
        stats->total_ms = ms;
        stats->queries_per_s = ms > 0 ? n_queries / (ms * 1e-3) : 0;
        stats->images_per_s = stats->queries_per_s * batch;
        if (o.record_latency && n_queries) {
            // every query of a wave starts and ends with its wave
            std::vector<float> lat;
            double sum = 0;
            for (int wv = 0; wv < n_waves; wv++) {
                float l = 0;
                cudaEventElapsedTime(&l, ev[2 * (size_t)wv], ev[2 * (size_t)wv + 1]);
                const int members = std::min(G, n_queries - wv * G);
                for (int m = 0; m < members; m++) { lat.push_back(l); sum += l; }
            }
            std::sort(lat.begin(), lat.end());
            stats->p50_ms = lat[(size_t)(n_queries - 1) / 2];
            stats->p99_ms = lat[(size_t)std::min<long long>(n_queries - 1, (long long)std::ceil(0.99 * n_queries) - 1)];
            stats->mean_ms = sum / n_queries;
        }
        stats->useful_flops = flops;
        stats->weight_bytes = wbytes;
        stats->hbm_weight_bytes = miss_bytes;
        stats->hit_ratio = n_queries ? hit / n_queries : 0;
        stats->byte_hit_ratio = wbytes > 0 ? 1.0 - miss_bytes / wbytes : 0;
        stats->kernel_launches = net->kernel_launches - launches0;
        stats->plan_hits = net->plan_hits - hits0;
        stats->plan_misses = net->plan_misses - miss0;
        stats->cache_updates = updates;
    }
    for (auto &e : ev) cudaEventDestroy(e);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    net->throughput_mode = 0;
    return rc;
}

// ---------------------------------------------------------------------------------------------
// Persistent execution (sgs_stream_opts_t::persistent): the whole stream is one launch of the SubNet kernel.
// ---------------------------------------------------------------------------------------------
// The plan of a config as the op list the kernel interprets (one record per layer; the patch-matrix / padding ops
// that the layer-by-layer paths put in front of the stem are dropped, the kernel convolves the image directly).
static sgs_status_t build_pq_ops(sgs_supernet *net, Plan *plan) {
    plan->pq.clear();
    const int stem_li = net->idx("stem");
    auto mult8 = [](int v) { return v > 0 && v % 8 == 0; };
    for (const Op &op : plan->ops) {
        PqOp q;
        std::memset(&q, 0, sizeof q);
        q.in = q.out = q.res = q.vin = q.vout = -1;
        q.cache_off = -1;
        switch (op.type) {
        case OP_IM2COL:
        case OP_PAD8: continue;
        case OP_CONV: {
            const StoredLayer &L = net->layers[op.layer];
            const Slice &s = plan->slices[op.layer];
            const ConvArgs &a = op.conv;
            q.w = L.w; q.scale = L.scale; q.shift = L.shift; q.act = a.act; q.out = op.out;
            q.Ho = a.Ho; q.Wo = a.Wo; q.K = s.K; q.R = L.R; q.Kmax = L.K; q.ld = L.Cp;
            if (op.layer == stem_li) {
                if (s.k > 3 || !mult8(s.K) || s.K > 64 || L.C != 3) return fail(net, SGS_EUNSUPPORTED, "persistent kernel: stem shape");
                q.type = PQ_STEM; q.H = plan->res; q.W = plan->res; q.C = 3; q.k = s.k; q.stride = 2;  // (the stem of this family)
            } else {
                if (s.k != 1 || a.stride != 1 || !mult8(s.C) || !mult8(s.K) || s.K > 1024) return fail(net, SGS_EUNSUPPORTED, "persistent kernel: convolution shape");
                q.type = PQ_PW; q.in = op.in; q.res = op.res; q.H = a.H; q.W = a.W; q.C = s.C; q.k = 1; q.stride = 1;
            }
            break;
        }
        case OP_DW: {
            const StoredLayer &L = net->layers[op.layer];
            const ConvArgs &a = op.conv;
            if (!mult8(a.K) || (a.k != 3 && a.k != 5 && a.k != 7) || (a.stride != 1 && a.stride != 2)) return fail(net, SGS_EUNSUPPORTED, "persistent kernel: depthwise shape");
            q.type = PQ_DW; q.in = op.in; q.out = op.out; q.H = a.H; q.W = a.W; q.Ho = a.Ho; q.Wo = a.Wo; q.C = a.K; q.K = a.K;
            q.k = a.k; q.stride = a.stride; q.act = a.act; q.R = L.R; q.Kmax = L.K; q.ld = L.K;
            q.w = L.w; q.scale = L.scale; q.shift = L.shift;
            break;
        }
        case OP_GAP:
            if (!mult8(op.C) || op.C > 1280) return fail(net, SGS_EUNSUPPORTED, "persistent kernel: pooled width");
            q.type = PQ_GAP; q.in = op.in; q.vout = op.vout; q.H = op.H; q.W = op.W; q.C = op.C;
            break;
        case OP_SE_GATE: {
            const StoredLayer &L1 = net->layers[op.layer], &L2 = net->layers[op.layer2];
            if (!mult8(op.C) || !mult8(op.K) || !mult8(L1.C) || !mult8(L2.C) || op.C > 1280 || op.K > 1280) return fail(net, SGS_EUNSUPPORTED, "persistent kernel: squeeze-excite shape");
            q.type = PQ_SE_GATE; q.vin = op.vin; q.vout = op.vout; q.C = op.C; q.K = op.K;
            q.w = L1.w; q.ld = L1.C; q.shift = L1.shift; q.w2 = L2.w; q.ld2 = L2.C; q.bias2 = L2.shift;
            break;
        }
        case OP_SCALE:
            q.type = PQ_SCALE; q.in = op.in; q.out = op.out; q.vin = op.vin; q.H = op.H; q.W = op.W; q.C = op.C;
            break;
        case OP_LINEAR: {
            const StoredLayer &L = net->layers[op.layer];
            if (!mult8(op.C) || !mult8(L.C) || op.C > 1280 || (op.vout >= 0 && op.K > 1280)) return fail(net, SGS_EUNSUPPORTED, "persistent kernel: linear shape");
            q.type = PQ_LINEAR; q.vin = op.vin; q.vout = op.vout; q.C = op.C; q.K = op.K; q.act = op.act;
            q.w = L.w; q.ld = L.C; q.shift = L.shift;
            break;
        }
        default: return fail(net, SGS_EUNSUPPORTED, "persistent kernel: layer type");
        }
        if (q.vin > 1 || q.vout > 1 || q.in > 3 || q.out > 3 || q.res > 3) return fail(net, SGS_EUNSUPPORTED, "persistent kernel: buffer id");
        plan->pq.push_back(q);
    }
    return SGS_OK;
}

static sgs_status_t persistent_impl(sgs_supernet_t *net, int n_queries, const sgs_subnet_cfg_t *cfgs, const void *inputs, int res,
                                    void *logits, const sgs_stream_opts_t &o, sgs_stream_stats_t *stats, cudaStream_t st,
                                    bool host_buffers) {
    if (net->family != SGS_MBV3 || net->dtype != SGS_BF16 || !tc_available())
        return fail(net, SGS_EUNSUPPORTED, "persistent execution serves bf16 handles of the MobileNetV3-shaped family on a tensor-core device");
    net->throughput_mode = 0;
    const int hits0 = net->plan_hits, miss0 = net->plan_misses;
    const long long launches0 = net->kernel_launches;
    const size_t in_bytes = (size_t)res * res * 3 * net->elem(), out_bytes = (size_t)net->def.classes * sizeof(float);
    // plans and op lists (one list per distinct config of the call)
    std::vector<Plan *> plans((size_t)n_queries);
    std::unordered_map<Plan *, int> begin;
    std::vector<PqOp> ops;
    std::vector<PqQuery> qs((size_t)n_queries);
    size_t act_elems = 0;
    double flops = 0, wbytes = 0, miss_bytes = 0, hit = 0;
    int updates = 0;
    for (int t = 0; t < n_queries; t++) {
        Plan *pl = nullptr;
        sgs_status_t rc = get_plan(net, &cfgs[t], 1, res, 0, &pl);
        if (rc != SGS_OK) return rc;
        if (pl->pq.empty() && (rc = build_pq_ops(net, pl)) != SGS_OK) return rc;
        plans[(size_t)t] = pl;
        act_elems = std::max(act_elems, pl->act_elems);
    }
    // The weight buffer of this launch: the SubGraph the cache policy chooses from the call's first window_q queries
    // (their intersection, or the candidate nearest to their average), of which every block keeps the pointwise layers'
    // boxes in shared memory, front layers first, as far as the buffer reaches.  One launch has one choice; the
    // accounting below is against what is actually held.
    std::vector<PqHeld> held;
    std::unordered_map<const void *, size_t> held_of;  // stored weights -> entry
    unsigned held_bytes = 0;
    if (net->cache.enabled && net->persistent_held_kb > 0 && n_queries > 0) {
        const int first = std::min(n_queries, net->cache.window_q);
        for (int t = 0; t < first; t++) net->cache.window.push_back(plans[(size_t)t]->enc);
        recompute_cached_subgraph(net);
        std::vector<int> g = net->cache.G, kept(g.size(), 0);
        const size_t budget = (size_t)net->persistent_held_kb * 1024;
        for (size_t li = 0; li < net->layers.size() && !g.empty(); li++) {
            const StoredLayer &L = net->layers[li];
            if (L.kind != KIND_CONV || L.R != 1 || L.C < 8) continue;
            const int rows = g[3 * li] & ~15, C = g[3 * li + 1];
            if (rows < 16 || rows > 256 || C < 8) continue;
            const int chunks = (C + 63) / 64;
            const size_t bytes = (size_t)chunks * rows * 128;
            if (held_bytes + bytes > budget) break;  // from the front, as the byte budget of the L2 policy is spent
            PqHeld h;
            std::memset(&h, 0, sizeof h);
            h.w = L.w; h.ld = L.Cp; h.rows = rows; h.chunks = chunks; h.C = C; h.off = held_bytes;
            held_of.emplace(L.w, held.size());
            held.push_back(h);
            held_bytes += (unsigned)bytes;
            kept[3 * li] = rows; kept[3 * li + 1] = C; kept[3 * li + 2] = 1;
        }
        held_bytes = (held_bytes + 1023u) & ~1023u;
        net->cache.G = kept;
        net->cache.epoch++;
        updates = 1;
    }
    for (int t = 0; t < n_queries; t++) {
        Plan *pl = plans[(size_t)t];
        auto it = begin.find(pl);
        if (it == begin.end()) {
            it = begin.emplace(pl, (int)ops.size()).first;
            for (PqOp q : pl->pq) {
                if (q.type == PQ_PW) {
                    auto h = held_of.find(q.w);
                    if (h != held_of.end()) { const PqHeld &e = held[h->second]; q.cache_off = e.off; q.cache_rows = e.rows; q.ld2 = e.C; }
                }
                ops.push_back(q);
            }
        }
        PqQuery &q = qs[(size_t)t];
        std::memset(&q, 0, sizeof q);
        q.op_begin = it->second; q.op_count = (int)pl->pq.size();
        QueryAccount qa = account_query(net, pl->enc);
        flops += pl->flops; wbytes += qa.weight_bytes; miss_bytes += qa.miss_bytes; hit += qa.hit_ratio;
    }
    // device resources: scratch of the blocks, tables, counter, staging for host buffers
    const int blocks_max = std::max(1, net->sms) * subnet_kernel_blocks_per_sm();
    const size_t act_bytes = (act_elems * net->elem() + 255) / 256 * 256, slot_bytes = 4 * act_bytes;
    if (net->pq_scratch_bytes < slot_bytes * blocks_max) {
        CU(cudaStreamSynchronize(st));
        dev_free(net, net->pq_scratch, net->pq_scratch_bytes); net->pq_scratch = nullptr; net->pq_scratch_bytes = 0;
        sgs_status_t rc = dev_alloc(net, (void **)&net->pq_scratch, slot_bytes * blocks_max);
        if (rc != SGS_OK) return rc;
        net->pq_scratch_bytes = slot_bytes * blocks_max;
    }
    const size_t ops_bytes = ops.size() * sizeof(PqOp), q_bytes = qs.size() * sizeof(PqQuery), h_bytes = held.size() * sizeof(PqHeld);
    const size_t tbl_need = ops_bytes + q_bytes + h_bytes;
    if (net->pq_tbl_bytes < tbl_need) {
        CU(cudaStreamSynchronize(st));
        dev_free(net, net->pq_d_tbl, net->pq_tbl_bytes); net->pq_d_tbl = nullptr;
        cudaFreeHost(net->pq_h_tbl); net->pq_h_tbl = nullptr;
        net->pq_tbl_bytes = 0;
        const size_t cap = tbl_need + tbl_need / 2;
        if (cudaMallocHost((void **)&net->pq_h_tbl, cap) != cudaSuccess) return fail(net, SGS_ENOMEM, "pinned table of the persistent kernel");
        sgs_status_t rc = dev_alloc(net, (void **)&net->pq_d_tbl, cap);
        if (rc != SGS_OK) { cudaFreeHost(net->pq_h_tbl); net->pq_h_tbl = nullptr; return rc; }
        net->pq_tbl_bytes = cap;
    }
    if (!net->pq_counter) {
        sgs_status_t rc = dev_alloc(net, (void **)&net->pq_counter, 256);
        if (rc != SGS_OK) return rc;
    }
    if (host_buffers) {
        const size_t need_in = in_bytes * (size_t)n_queries, need_out = out_bytes * (size_t)n_queries;
        if (net->pq_stage_in_bytes < need_in) {
            CU(cudaStreamSynchronize(st));
            dev_free(net, net->pq_stage_in, net->pq_stage_in_bytes); net->pq_stage_in = nullptr; net->pq_stage_in_bytes = 0;
            sgs_status_t rc = dev_alloc(net, &net->pq_stage_in, need_in);
            if (rc != SGS_OK) return rc;
            net->pq_stage_in_bytes = need_in;
        }
        if (net->pq_stage_out_bytes < need_out) {
            CU(cudaStreamSynchronize(st));
            dev_free(net, net->pq_stage_out, net->pq_stage_out_bytes); net->pq_stage_out = nullptr; net->pq_stage_out_bytes = 0;
            sgs_status_t rc = dev_alloc(net, (void **)&net->pq_stage_out, need_out);
            if (rc != SGS_OK) return rc;
            net->pq_stage_out_bytes = need_out;
        }
    }
    const char *din = host_buffers ? static_cast<const char *>(net->pq_stage_in) : static_cast<const char *>(inputs);
    char *dout = host_buffers ? reinterpret_cast<char *>(net->pq_stage_out) : static_cast<char *>(logits);
    for (int t = 0; t < n_queries; t++) {
        qs[(size_t)t].x = din + (size_t)t * in_bytes;
        qs[(size_t)t].logits = reinterpret_cast<float *>(dout + (size_t)t * out_bytes);
    }
    CU(cudaStreamSynchronize(st));  // the pinned table image may still be the source of an earlier call's copy
    if (tbl_need) {
        std::memcpy(net->pq_h_tbl, ops.data(), ops_bytes);
        std::memcpy(net->pq_h_tbl + ops_bytes, qs.data(), q_bytes);
        if (h_bytes) std::memcpy(net->pq_h_tbl + ops_bytes + q_bytes, held.data(), h_bytes);
    }

    cudaEvent_t e0, e1;
    CU(cudaEventCreate(&e0));
    CU(cudaEventCreate(&e1));
    sgs_status_t rc = SGS_OK;
    cudaError_t ce = cudaEventRecord(e0, st);
    if (ce == cudaSuccess && host_buffers && n_queries) ce = cudaMemcpyAsync(net->pq_stage_in, inputs, in_bytes * (size_t)n_queries, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess && tbl_need) ce = cudaMemcpyAsync(net->pq_d_tbl, net->pq_h_tbl, tbl_need, cudaMemcpyHostToDevice, st);
    if (ce == cudaSuccess) ce = cudaMemsetAsync(net->pq_counter, 0, sizeof(int), st);
    if (ce == cudaSuccess && n_queries) {
        PqParams p;
        p.ops = reinterpret_cast<const PqOp *>(net->pq_d_tbl);
        p.queries = reinterpret_cast<const PqQuery *>(net->pq_d_tbl + ops_bytes);
        p.held = reinterpret_cast<const PqHeld *>(net->pq_d_tbl + ops_bytes + q_bytes);
        p.n_held = (int)held.size();
        p.held_bytes = held_bytes;
        p.n_queries = n_queries;
        p.counter = net->pq_counter;
        p.scratch = net->pq_scratch;
        p.slot_bytes = slot_bytes; p.act_bytes = act_bytes;
        p.status = tc_status_word(net->device);
        LayerRange range(net, -1, "persistent SubNet kernel");
        ce = subnet_kernel_launch(p, std::min(blocks_max, n_queries), st);
        net->kernel_launches++;
    }
    if (ce == cudaSuccess && host_buffers && n_queries) ce = cudaMemcpyAsync(logits, net->pq_stage_out, out_bytes * (size_t)n_queries, cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaEventRecord(e1, st);
    cudaError_t se = cudaStreamSynchronize(st);
    if (ce != cudaSuccess || se != cudaSuccess) rc = fail(net, SGS_ECUDA, std::string("persistent stream: ") + cudaGetErrorString(se != cudaSuccess ? se : ce));
    if (rc == SGS_OK && tc_conv_status()) rc = fail(net, SGS_ETIMEOUT, "a bounded device-side wait ran out in the persistent SubNet kernel");
    if (rc == SGS_OK && stats) {
        std::memset(stats, 0, sizeof(*stats));
        float ms = 0;
        cudaEventElapsedTime(&ms, e0, e1);
        stats->n_queries = n_queries;
        stats->total_ms = ms;
        stats->queries_per_s = ms > 0 ? n_queries / (ms * 1e-3) : 0;
        stats->images_per_s = stats->queries_per_s;
        if (o.record_latency && n_queries) stats->p50_ms = stats->p99_ms = stats->mean_ms = ms;  // every query starts and ends with the launch
        stats->useful_flops = flops;
        stats->weight_bytes = wbytes;
        stats->hbm_weight_bytes = miss_bytes;
        stats->hit_ratio = n_queries ? hit / n_queries : 0;
        stats->byte_hit_ratio = wbytes > 0 ? 1.0 - miss_bytes / wbytes : 0;
        stats->kernel_launches = net->kernel_launches - launches0;
        stats->plan_hits = net->plan_hits - hits0;
        stats->plan_misses = net->plan_misses - miss0;
        stats->cache_updates = updates;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    return rc;
}

static sgs_status_t stream_impl(sgs_supernet_t *net, int n_queries, const sgs_subnet_cfg_t *cfgs, const void *inputs,
                                int batch, int res, void *logits, const sgs_stream_opts_t *opts,
                                sgs_stream_stats_t *stats, cudaStream_t st, bool host_buffers) {
    if (!net) return SGS_EINVAL;
    if (n_queries < 0 || (n_queries && (!cfgs || !inputs || !logits)) || batch <= 0 || res < 8 || res > 1024)
        return fail(net, SGS_EINVAL, "bad argument");
    DeviceGuard guard(net->device);
    if (!guard.ok) return fail(net, SGS_ECUDA, "cudaSetDevice failed");
    sgs_stream_opts_t o;
    if (opts) o = *opts;
    else { o.cache_enabled = 1; o.window_q = 4; o.cache_budget_bytes = 0; o.use_graphs = 1; o.record_latency = 1; o.weights_evict_first = 0; o.concurrency = 1; o.wave = 0; o.policy = 0; o.persistent = 0; }
    if (o.window_q < 1) return fail(net, SGS_EINVAL, "window_q must be >= 1");
    if (o.concurrency < 0 || o.concurrency > 16) return fail(net, SGS_EINVAL, "concurrency must be in [0, 16]");
    for (int t = 0; t < n_queries; t++)
        if (!cfg_valid(net, &cfgs[t])) return fail(net, SGS_ECONFIG, "query " + std::to_string(t) + ": config outside the elastic sets");
    if (o.wave < 0) return fail(net, SGS_EINVAL, "wave must be >= 0");
    if (o.policy != SGS_POLICY_INTERSECTION && o.policy != SGS_POLICY_AVGNET) return fail(net, SGS_EINVAL, "unknown cache policy");
    if (o.policy == SGS_POLICY_AVGNET && o.cache_enabled && net->cache.cand_raw.empty())
        return fail(net, SGS_EINVAL, "the AvgNet policy needs a candidate set (sgs_cache_set_candidates)");
    net->cache.policy = o.policy;
    cache_reset(net, o.cache_enabled != 0, o.cache_budget_bytes, o.window_q);
    net->cache.evict_first_when_off = (!o.cache_enabled && o.weights_evict_first) ? 1 : 0;
    if (o.persistent) {
        if (batch != 1) return fail(net, SGS_EINVAL, "persistent execution takes one image per query");
        return persistent_impl(net, n_queries, cfgs, inputs, res, logits, o, stats, st, host_buffers);
    }
    if (o.wave > 0 && n_queries > 0 && net->dtype == SGS_BF16 && tc_available() && !net->force_plain)
        return wave_impl(net, n_queries, cfgs, inputs, batch, res, logits, o, stats, st, host_buffers);
    // queries in flight at once: each runs in its own slot; per-kernel profiling wants them one by one
    const int S = net->profile ? 1 : std::max(1, std::min(o.concurrency ? o.concurrency : 1, std::max(1, n_queries)));
    {
        sgs_status_t rc = ensure_slots(net, S);
        if (rc != SGS_OK) return rc;
    }
    net->throughput_mode = S >= 12 ? 1 : 0;

    const size_t in_elems = (size_t)batch * res * res * 3, in_bytes = in_elems * net->elem();
    const size_t out_bytes = (size_t)batch * net->def.classes * sizeof(float);
    if (host_buffers) {
        // one staging pair per slot: consecutive queries of a slot are ordered by the slot's stream
        if (net->stage_in_bytes < in_bytes || net->stage_out_bytes < out_bytes) {
            for (auto &sl : net->slots) {
                dev_free(net, sl.stage_in, net->stage_in_bytes); sl.stage_in = nullptr;
                dev_free(net, sl.stage_out, net->stage_out_bytes); sl.stage_out = nullptr;
            }
            net->stage_in_bytes = std::max(net->stage_in_bytes, in_bytes);
            net->stage_out_bytes = std::max(net->stage_out_bytes, out_bytes);
        }
        for (auto &sl : net->slots) {
            if (!sl.stage_in) { sgs_status_t rc = dev_alloc(net, &sl.stage_in, net->stage_in_bytes); if (rc != SGS_OK) return rc; }
            if (!sl.stage_out) { sgs_status_t rc = dev_alloc(net, (void **)&sl.stage_out, net->stage_out_bytes); if (rc != SGS_OK) return rc; }
        }
    }
    std::vector<cudaEvent_t> ev;  // per query: start and end on the query's stream
    if (o.record_latency) {
        ev.resize(2 * (size_t)n_queries);
        for (auto &e : ev) CU(cudaEventCreate(&e));
    }
    cudaEvent_t e0, e1;
    CU(cudaEventCreate(&e0));
    CU(cudaEventCreate(&e1));
    const long long launches0 = net->kernel_launches;
    const int hits0 = net->plan_hits, miss0 = net->plan_misses;
    double flops = 0, wbytes = 0, miss_bytes = 0, hit = 0;
    int updates = 0;
    sgs_status_t rc = SGS_OK;
    CU(cudaEventRecord(e0, st));
    const auto host_t0 = std::chrono::steady_clock::now();
    for (int sidx = 1; sidx < S; sidx++) CU(cudaStreamWaitEvent(net->slots[sidx].st, e0, 0));  // fork
    for (int t = 0; t < n_queries && rc == SGS_OK; t++) {
        const int slot = t % S;
        sgs_supernet::Slot &sl = net->slots[slot];
        cudaStream_t qs = slot == 0 ? st : sl.st;
        const void *din;
        void *dout;
        if (o.record_latency) {
            cudaError_t ce = cudaEventRecord(ev[2 * (size_t)t], qs);
            if (ce != cudaSuccess) { rc = fail(net, SGS_ECUDA, cudaGetErrorString(ce)); break; }
        }
        if (host_buffers) {
            din = sl.stage_in;
            dout = sl.stage_out;
            cudaError_t ce = cudaMemcpyAsync(sl.stage_in, static_cast<const char *>(inputs) + (size_t)t * in_bytes, in_bytes,
                                             cudaMemcpyHostToDevice, qs);
            if (ce != cudaSuccess) { rc = fail(net, SGS_ECUDA, cudaGetErrorString(ce)); break; }
        } else {
            din = static_cast<const char *>(inputs) + (size_t)t * in_bytes;
            dout = static_cast<char *>(logits) + (size_t)t * out_bytes;
        }
        // Profiling brackets every launch with events.  To keep the host's launch latency out of those
        // intervals the stream is first held for a few milliseconds by a sleeping kernel, so that the
        // launches of the next 8 queries are already queued when the GPU reaches them.
        if (net->profile && t % 8 == 0) {
            cudaError_t ce = launch_delay(6000, qs);
            if (ce != cudaSuccess) { rc = fail(net, SGS_ECUDA, cudaGetErrorString(ce)); break; }
        }
        Plan *plan = nullptr;
        const int epoch_before = net->cache.epoch;
        // the legacy default stream cannot be captured: run it without graphs
        const auto q0 = std::chrono::steady_clock::now();
        rc = run_query(net, &cfgs[t], din, batch, res, dout, qs, o.use_graphs != 0 && qs != nullptr, slot, &plan);
        net->host_us_query += std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - q0).count();
        if (rc != SGS_OK) break;
        if (host_buffers) {
            cudaError_t ce = cudaMemcpyAsync(static_cast<char *>(logits) + (size_t)t * out_bytes, dout, out_bytes,
                                             cudaMemcpyDeviceToHost, qs);
            if (ce != cudaSuccess) { rc = fail(net, SGS_ECUDA, cudaGetErrorString(ce)); break; }
        }
        if (o.record_latency) {
            cudaError_t ce = cudaEventRecord(ev[2 * (size_t)t + 1], qs);
            if (ce != cudaSuccess) { rc = fail(net, SGS_ECUDA, cudaGetErrorString(ce)); break; }
        }
        const std::vector<int> &enc = plan->enc;
        QueryAccount qa = account_query(net, enc);
        flops += plan->flops; wbytes += qa.weight_bytes; miss_bytes += qa.miss_bytes; hit += qa.hit_ratio;
        if (net->cache.enabled) {
            cache_observe(net, enc);
            if (net->cache.epoch != epoch_before) updates++;
        }
    }
    net->host_us_stream += std::chrono::duration<double, std::micro>(std::chrono::steady_clock::now() - host_t0).count();
    for (int sidx = 1; sidx < S; sidx++) {  // join
        cudaEventRecord(net->slots[sidx].ev, net->slots[sidx].st);
        cudaStreamWaitEvent(st, net->slots[sidx].ev, 0);
    }
    cudaError_t ce = cudaEventRecord(e1, st);
    cudaError_t se = cudaStreamSynchronize(st);
    if (rc == SGS_OK && (ce != cudaSuccess || se != cudaSuccess))
        rc = fail(net, SGS_ECUDA, std::string("stream: ") + cudaGetErrorString(se != cudaSuccess ? se : ce));
    if (rc != SGS_OK) cudaDeviceSynchronize();  // leave no work of the other slots behind
    if (rc == SGS_OK && tc_conv_status()) rc = fail(net, SGS_ETIMEOUT, "a bounded device-side wait ran out in the tensor-core kernel");
    if (rc == SGS_OK && stats) {
        std::memset(stats, 0, sizeof(*stats));
        float ms = 0;
        cudaEventElapsedTime(&ms, e0, e1);
        stats->n_queries = n_queries;
        stats->total_ms = ms;
        stats->queries_per_s = ms > 0 ? n_queries / (ms * 1e-3) : 0;
        stats->images_per_s = stats->queries_per_s * batch;
        if (o.record_latency && n_queries) {
            std::vector<float> lat((size_t)n_queries);
            double sum = 0;
            for (int t = 0; t < n_queries; t++) { cudaEventElapsedTime(&lat[t], ev[2 * (size_t)t], ev[2 * (size_t)t + 1]); sum += lat[t]; }
            std::sort(lat.begin(), lat.end());
            stats->p50_ms = lat[(size_t)(n_queries - 1) / 2];
            stats->p99_ms = lat[(size_t)std::min<long long>(n_queries - 1, (long long)std::ceil(0.99 * n_queries) - 1)];
            stats->mean_ms = sum / n_queries;
        }
        stats->useful_flops = flops;
        stats->weight_bytes = wbytes;
        stats->hbm_weight_bytes = miss_bytes;
        stats->hit_ratio = n_queries ? hit / n_queries : 0;
        stats->byte_hit_ratio = wbytes > 0 ? 1.0 - miss_bytes / wbytes : 0;
        stats->kernel_launches = net->kernel_launches - launches0;
        stats->plan_hits = net->plan_hits - hits0;
        stats->plan_misses = net->plan_misses - miss0;
        stats->cache_updates = updates;
    }
    for (auto &e : ev) cudaEventDestroy(e);
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    net->throughput_mode = 0;
    return rc;
}

sgs_status_t sgs_stream_run(sgs_supernet_t *net, int n_queries, const sgs_subnet_cfg_t *cfgs, const void *d_inputs,
                            int batch_per_query, int res, void *d_logits, const sgs_stream_opts_t *opts,
                            sgs_stream_stats_t *stats, void *cuda_stream) {
    return stream_impl(net, n_queries, cfgs, d_inputs, batch_per_query, res, d_logits, opts, stats, (cudaStream_t)cuda_stream, false);
}

sgs_status_t sgs_stream_run_host(sgs_supernet_t *net, int n_queries, const sgs_subnet_cfg_t *cfgs, const void *h_inputs,
                                 int batch_per_query, int res, void *h_logits, const sgs_stream_opts_t *opts,
                                 sgs_stream_stats_t *stats, void *cuda_stream) {
    return stream_impl(net, n_queries, cfgs, h_inputs, batch_per_query, res, h_logits, opts, stats, (cudaStream_t)cuda_stream, true);
}

sgs_status_t sgs_cache_configure(sgs_supernet_t *net, int enabled, size_t budget_bytes, int window_q) {
    if (!net) return SGS_EINVAL;
    if (window_q < 1) return fail(net, SGS_EINVAL, "window_q must be >= 1");
    cache_reset(net, enabled != 0, budget_bytes, window_q);
    return SGS_OK;
}

sgs_status_t sgs_cache_set_candidates(sgs_supernet_t *net, const sgs_subnet_cfg_t *cfgs, int n) {
    if (!net || n < 0 || (n && !cfgs)) return SGS_EINVAL;
    std::vector<std::vector<int>> raw;
    for (int j = 0; j < n; j++) {
        if (!cfg_valid(net, &cfgs[j])) return fail(net, SGS_ECONFIG, "candidate " + std::to_string(j) + ": config outside the elastic sets");
        raw.push_back(encoding_of(slices_for(net, &cfgs[j])));
    }
    net->cache.cand_raw = std::move(raw);
    clip_candidates(net);
    if (n == 0) net->cache.policy = 0;
    return SGS_OK;
}

sgs_status_t sgs_cache_set_policy(sgs_supernet_t *net, int policy) {
    if (!net) return SGS_EINVAL;
    if (policy != SGS_POLICY_INTERSECTION && policy != SGS_POLICY_AVGNET) return fail(net, SGS_EINVAL, "unknown cache policy");
    if (policy == SGS_POLICY_AVGNET && net->cache.cand_raw.empty())
        return fail(net, SGS_EINVAL, "the AvgNet policy needs a candidate set (sgs_cache_set_candidates)");
    net->cache.policy = policy;
    return SGS_OK;
}

// ------------------------------------------------------------------------------------------
// Scheduler object: Algorithm 1 (Section 3.3) over a latency table (Section 3.2)
// ------------------------------------------------------------------------------------------
}  // extern "C"

struct sgs_sched {
    sgs_supernet *net = nullptr;
    int N = 0, M = 0, q = 1;
    std::vector<sgs_subnet_cfg_t> subnets;
    std::vector<std::vector<int>> encs;
    std::vector<double> acc, table;  // table[i * (M + 1) + j]; column M = nothing cached
    std::deque<std::vector<int>> window;
    int since = 0, state = 0;
    void *flush = nullptr;
    size_t flush_bytes = 0;
};

namespace {
int sched_select(const sgs_sched *s, int policy, double a_t, double l_t) {
    const int W = s->M + 1;
    int best = -1;
    bool best_feasible = false;
    for (int i = 0; i < s->N; i++) {
        const double lat = s->table[(size_t)i * W + s->state], acc = s->acc[i];
        const bool feasible = policy == SGS_STRICT_ACCURACY ? acc >= a_t : lat <= l_t;
        if (best < 0) { best = i; best_feasible = feasible; continue; }
        if (feasible != best_feasible) { if (feasible) { best = i; best_feasible = true; } continue; }
        const double blat = s->table[(size_t)best * W + s->state], bacc = s->acc[best];
        // among feasible SubNets: the fastest (STRICT_ACCURACY) / the most accurate (STRICT_LATENCY); with no
        // feasible SubNet the roles swap (the most accurate / the fastest); ties by the other quantity
        const bool by_latency = (policy == SGS_STRICT_ACCURACY) == feasible;
        const bool better = by_latency ? (lat < blat || (lat == blat && acc > bacc)) : (acc > bacc || (acc == bacc && lat < blat));
        if (better) best = i;
    }
    return best;
}
}  // namespace

extern "C" {

sgs_status_t sgs_sched_create(sgs_supernet_t *net, const sgs_subnet_cfg_t *subnets, const double *accuracy, int n_subnets,
                              int window_q, sgs_sched_t **out) {
    if (!net || !out) return SGS_EINVAL;
    if (!subnets || !accuracy || n_subnets < 1 || window_q < 1) return fail(net, SGS_EINVAL, "bad argument");
    if (net->cache.cand_raw.empty()) return fail(net, SGS_EINVAL, "a scheduler needs a candidate set (sgs_cache_set_candidates)");
    std::unique_ptr<sgs_sched> s(new (std::nothrow) sgs_sched);
    if (!s) return SGS_ENOMEM;
    s->net = net; s->N = n_subnets; s->M = (int)net->cache.cand_raw.size(); s->q = window_q;
    for (int i = 0; i < n_subnets; i++) {
        if (!cfg_valid(net, &subnets[i])) return fail(net, SGS_ECONFIG, "SubNet " + std::to_string(i) + ": config outside the elastic sets");
        s->subnets.push_back(subnets[i]);
        s->encs.push_back(encoding_of(slices_for(net, &subnets[i])));
        s->acc.push_back(accuracy[i]);
    }
    s->table.assign((size_t)s->N * (s->M + 1), 0.0);
    s->state = s->M;
    cache_pin(net, -1);
    *out = s.release();
    return SGS_OK;
}

void sgs_sched_free(sgs_sched_t *s) {
    if (!s) return;
    if (s->flush) {
        DeviceGuard guard(s->net->device);
        cudaDeviceSynchronize();
        dev_free(s->net, s->flush, s->flush_bytes);
    }
    if (s->net->cache.policy == 2) { s->net->cache.policy = 0; cache_reset(s->net, false, s->net->cache.budget, s->net->cache.window_q); }
    delete s;
}

sgs_status_t sgs_sched_dims(const sgs_sched_t *s, int *n_subnets, int *n_columns) {
    if (!s) return SGS_EINVAL;
    if (n_subnets) *n_subnets = s->N;
    if (n_columns) *n_columns = s->M + 1;
    return SGS_OK;
}

sgs_status_t sgs_sched_set_table(sgs_sched_t *s, const double *latency) {
    if (!s || !latency) return SGS_EINVAL;
    std::copy(latency, latency + s->table.size(), s->table.begin());
    return SGS_OK;
}

sgs_status_t sgs_sched_get_table(const sgs_sched_t *s, double *latency) {
    if (!s || !latency) return SGS_EINVAL;
    std::copy(s->table.begin(), s->table.end(), latency);
    return SGS_OK;
}

sgs_status_t sgs_sched_measure(sgs_sched_t *s, const void *d_input, int batch, int res, void *d_logits, int reps,
                               size_t flush_bytes, void *cuda_stream) {
    if (!s) return SGS_EINVAL;
    sgs_supernet *net = s->net;
    if (!d_input || !d_logits || batch <= 0 || res < 8 || res > 1024 || reps < 1 || reps > 1000) return fail(net, SGS_EINVAL, "bad argument");
    if ((int)net->cache.cand.size() != s->M) return fail(net, SGS_EINVAL, "the candidate set changed under the scheduler");
    DeviceGuard guard(net->device);
    if (!guard.ok) return fail(net, SGS_ECUDA, "cudaSetDevice failed");
    cudaStream_t st = (cudaStream_t)cuda_stream;
    if (flush_bytes > s->flush_bytes) {
        CU(cudaStreamSynchronize(st));
        dev_free(net, s->flush, s->flush_bytes);
        s->flush = nullptr; s->flush_bytes = 0;
        sgs_status_t rc = dev_alloc(net, &s->flush, flush_bytes);
        if (rc != SGS_OK) return rc;
        s->flush_bytes = flush_bytes;
    }
    std::vector<cudaEvent_t> ev(2 * (size_t)reps);
    for (auto &e : ev) CU(cudaEventCreate(&e));
    sgs_status_t rc = SGS_OK;
    std::vector<float> ms((size_t)reps);
    for (int j = 0; j <= s->M && rc == SGS_OK; j++) {
        cache_pin(net, j < s->M ? j : -1);
        for (int i = 0; i < s->N && rc == SGS_OK; i++) {
            // one untimed run builds the plan and brings the SubNet's weights in under the hints of column j
            rc = run_query(net, &s->subnets[i], d_input, batch, res, d_logits, st, false, 0, nullptr);
            for (int r = 0; r < reps && rc == SGS_OK; r++) {
                if (flush_bytes && cudaMemsetAsync(s->flush, r & 1, flush_bytes, st) != cudaSuccess) rc = fail(net, SGS_ECUDA, "flush failed");
                if (rc == SGS_OK && cudaEventRecord(ev[2 * r], st) != cudaSuccess) rc = fail(net, SGS_ECUDA, "event record failed");
                if (rc == SGS_OK) rc = run_query(net, &s->subnets[i], d_input, batch, res, d_logits, st, false, 0, nullptr);
                if (rc == SGS_OK && cudaEventRecord(ev[2 * r + 1], st) != cudaSuccess) rc = fail(net, SGS_ECUDA, "event record failed");
            }
            if (rc != SGS_OK) break;
            if (cudaStreamSynchronize(st) != cudaSuccess) { rc = fail(net, SGS_ECUDA, "stream synchronise failed"); break; }
            for (int r = 0; r < reps; r++) cudaEventElapsedTime(&ms[r], ev[2 * r], ev[2 * r + 1]);
            std::vector<float> sorted = ms;
            std::sort(sorted.begin(), sorted.end());
            s->table[(size_t)i * (s->M + 1) + j] = reps & 1 ? sorted[reps / 2] : 0.5 * ((double)sorted[reps / 2 - 1] + sorted[reps / 2]);
        }
    }
    cudaStreamSynchronize(st);
    for (auto &e : ev) cudaEventDestroy(e);
    cache_pin(net, s->state < s->M ? s->state : -1);
    if (rc == SGS_OK && tc_conv_status()) return fail(net, SGS_ETIMEOUT, "a bounded wait ran out in a tensor-core kernel");
    return rc;
}

sgs_status_t sgs_sched_step(sgs_sched_t *s, int n, const int *policy, const double *a_t, const double *l_t, int *subnet,
                            int *cache_state) {
    if (!s) return SGS_EINVAL;
    if (n < 0 || (n && (!policy || !a_t || !l_t || !subnet))) return fail(s->net, SGS_EINVAL, "bad argument");
    if ((int)s->net->cache.cand.size() != s->M) return fail(s->net, SGS_EINVAL, "the candidate set changed under the scheduler");
    for (int t = 0; t < n; t++)
        if (policy[t] != SGS_STRICT_ACCURACY && policy[t] != SGS_STRICT_LATENCY) return fail(s->net, SGS_EINVAL, "unknown query policy");
    const int before = s->state;
    for (int t = 0; t < n; t++) {
        const int i = sched_select(s, policy[t], a_t[t], l_t[t]);
        subnet[t] = i;
        if (cache_state) cache_state[t] = s->state;
        s->window.push_back(s->encs[i]);
        while ((int)s->window.size() > s->q) s->window.pop_front();
        if (++s->since >= s->q) {
            s->since = 0;
            s->state = nearest_candidate(s->window, s->net->cache.cand);
        }
    }
    if (s->state != before || s->net->cache.policy != 2) cache_pin(s->net, s->state < s->M ? s->state : -1);
    return SGS_OK;
}

sgs_status_t sgs_sched_subnet(const sgs_sched_t *s, int i, sgs_subnet_cfg_t *out) {
    if (!s || !out || i < 0 || i >= s->N) return SGS_EINVAL;
    *out = s->subnets[i];
    return SGS_OK;
}

sgs_status_t sgs_cache_stats(const sgs_supernet_t *net, sgs_cache_stats_t *out) {
    if (!net || !out) return SGS_EINVAL;
    std::memset(out, 0, sizeof(*out));
    out->enabled = net->cache.enabled;
    out->window_q = net->cache.window_q;
    out->budget_bytes = net->cache.budget;
    out->l2_bytes = net->l2_bytes;
    out->persisting_l2_max = net->persist_max;
    out->access_window_max = net->window_max;
    out->cached_subgraph_bytes = net->cache.G_bytes;
    out->supernet_bytes = net->weight_arena_bytes;
    out->device_bytes_allocated = net->device_bytes;
    out->policy = net->cache.policy;
    out->n_candidates = (int)net->cache.cand_raw.size();
    out->decisions = net->cache.decisions;
    out->last_choice = net->cache.last_choice;
    return SGS_OK;
}

sgs_status_t sgs_profile_read(sgs_supernet_t *net, int kernel_class, long long *launches, double *total_ms,
                              double *alg_bytes, double *flops) {
    if (!net || kernel_class < 0 || kernel_class > 3) return SGS_EINVAL;
    DeviceGuard guard(net->device);
    fold_profile(net);
    if (launches) *launches = net->prof_launches[kernel_class];
    if (total_ms) *total_ms = net->prof_ms[kernel_class];
    if (alg_bytes) *alg_bytes = net->prof_bytes[kernel_class];
    if (flops) *flops = net->prof_flops[kernel_class];
    return SGS_OK;
}

int sgs_profile_trace(sgs_supernet_t *net, sgs_launch_record_t *out, int cap) {
    if (!net || cap < 0 || (cap && !out)) return -1;
    const int n = (int)std::min<size_t>(net->prof_trace.size(), (size_t)cap);
    if (n) std::memcpy(out, net->prof_trace.data(), (size_t)n * sizeof(sgs_launch_record_t));
    return (int)net->prof_trace.size();
}

int sgs_layer_name(const sgs_supernet_t *net, int layer, char *out, int cap) {
    if (!net || layer < 0 || layer >= (int)net->layers.size() || !out || cap < 1) return -1;
    std::snprintf(out, (size_t)cap, "%s", net->layers[(size_t)layer].name.c_str());
    return (int)net->layers[(size_t)layer].name.size();
}

sgs_status_t sgs_set_option(sgs_supernet_t *net, const char *name, long long value) {
    if (!net || !name) return SGS_EINVAL;
    std::string n(name);
    if (n == "conv_impl" || n == "pad_channels") {
        if (n == "conv_impl") net->force_plain = value == 1;
        else net->pad_channels = value != 0;
        DeviceGuard guard(net->device);
        cudaDeviceSynchronize();
        fold_profile(net);
        for (auto &kv : net->plans) destroy_plan_resources(kv.second.get());
        net->plans.clear();
        return SGS_OK;
    }
    if (n == "profile") {
        DeviceGuard guard(net->device);
        fold_profile(net);
        net->profile = value != 0;
        if (value == 2 || value == 0) {
            for (int i = 0; i < 4; i++) { net->prof_ms[i] = net->prof_bytes[i] = net->prof_flops[i] = 0; net->prof_launches[i] = 0; }
            net->prof_trace.clear();
        }
        return SGS_OK;
    }
    if (n == "persistent_held_kb") {
        if (value < 0 || (size_t)value * 1024 > subnet_kernel_held_max()) return fail(net, SGS_EINVAL, "persistent_held_kb out of range");
        net->persistent_held_kb = (int)value;
        return SGS_OK;
    }
    if (n == "nvtx") {
        net->nvtx = value != 0;
        return SGS_OK;
    }
    if (n == "fail_alloc_after") {
        net->fail_alloc_after = value < 0 ? -1 : value;
        return SGS_OK;
    }
    if (n == "cache_mechanism") {
        if (value < 0 || value > 2) return fail(net, SGS_EINVAL, "cache_mechanism");
        net->cache_mech = (int)value;
        return SGS_OK;
    }
    if (n == "drop_plans") {  // forget every plan (and its graphs): the next use of a config pays for planning again
        DeviceGuard guard(net->device);
        cudaDeviceSynchronize();
        fold_profile(net);
        for (auto &kv : net->plans) destroy_plan_resources(kv.second.get());
        net->plans.clear();
        return SGS_OK;
    }
    if (n == "dw_walk") {  // tuning aid (process-wide)
        dw_set_walk((int)value);
        return SGS_OK;
    }
    if (n == "stage_group") {  // tuning aid: stages per barrier pair of the grouped convolution kernel (0 = default)
        if (value < 0 || value > 4) return fail(net, SGS_EINVAL, "stage_group");
        tc_group_set_stage_group((int)value);
        return SGS_OK;
    }
    return fail(net, SGS_EINVAL, "unknown option " + n);
}

long long sgs_get_counter(const sgs_supernet_t *net, const char *name) {
    if (!net || !name) return -1;
    std::string n(name);
    if (n == "kernel_launches") return net->kernel_launches;
    if (n == "plan_hits") return net->plan_hits;
    if (n == "plan_misses") return net->plan_misses;
    if (n == "device_bytes") return (long long)net->device_bytes;
    if (n == "host_us_graph") return (long long)net->host_us_graph;
    if (n == "host_us_direct") return (long long)net->host_us_direct;
    if (n == "host_us_stream") return (long long)net->host_us_stream;
    if (n == "host_us_query") return (long long)net->host_us_query;
    if (n == "host_us_table") return (long long)net->host_us_table;
    if (n == "tc_convs") {
        long long c = 0;
        for (auto &kv : net->plans)
            for (const Op &op : kv.second->ops) c += op.impl == 1;
        return c;
    }
    return -1;
}

const char *sgs_last_error(const sgs_supernet_t *net) { return net ? net->err.c_str() : "null handle"; }

// Stand-alone sliced convolution.  The split-K scratch of the tensor-core kernel is one buffer per
// device, grown on demand and shared by all calls of this function.
sgs_status_t sgs_conv2d_sliced(const sgs_conv_desc_t *d, const void *d_x, const void *d_w, const float *d_scale,
                               const float *d_shift, const void *d_res, void *d_y, void *cuda_stream) {
    if (!d || !d_x || !d_w || !d_scale || !d_shift || !d_y) return SGS_EINVAL;
    if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->C <= 0 || d->K <= 0 || d->k <= 0 || (d->k & 1) == 0 || d->k > d->R ||
        ((d->R - d->k) & 1) || d->K > d->Kmax || (!d->depthwise && d->C > d->Cmax) || (d->stride != 1 && d->stride != 2) ||
        (d->dtype != SGS_F32 && d->dtype != SGS_BF16) || d->act < 0 || d->act > 2 || d->impl < 0 || d->impl > 2)
        return SGS_EINVAL;
    ConvArgs a;
    a.x = d_x; a.w = d_w; a.scale = d_scale; a.shift = d_shift; a.res = d_res; a.y = d_y;
    a.N = d->N; a.H = d->H; a.W = d->W; a.C = d->depthwise ? d->K : d->C; a.K = d->K;
    a.Kmax = d->Kmax; a.Cmax = d->depthwise ? 1 : d->Cmax; a.R = d->R; a.k = d->k; a.stride = d->stride; a.act = d->act;
    const int p = (d->k - 1) / 2;
    a.Ho = (d->H + 2 * p - d->k) / d->stride + 1;
    a.Wo = (d->W + 2 * p - d->k) / d->stride + 1;
    a.cacheK = d->cache_k; a.cacheC = d->cache_c; a.weight_policy = d->weight_policy;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    cudaError_t e;
    if (d->depthwise) {
        if (d->impl == 2) return SGS_EUNSUPPORTED;
        e = d->dtype == SGS_BF16 ? launch_dw<__nv_bfloat16>(a, st) : launch_dw<float>(a, st);
        return e == cudaSuccess ? SGS_OK : SGS_ECUDA;
    }
    if (d->impl != 1 && d->dtype == SGS_BF16 && tc_available()) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SGS_ECUDA;
        std::string why;
        std::shared_ptr<TcConvPlan> plan = tc_conv_prepare(a, dev, &why);
        if (plan) {
            static float *ws[64] = {};
            static size_t ws_elems[64] = {};
            const size_t need = d->split_k_off ? 0 : tc_conv_ws_elems(*plan);
            if (need > ws_elems[dev]) {
                cudaFree(ws[dev]);
                ws[dev] = nullptr; ws_elems[dev] = 0;
                if (cudaMalloc((void **)&ws[dev], need * 4) != cudaSuccess) return SGS_ENOMEM;
                ws_elems[dev] = need;
            }
            if (!d->split_k_off) { a.ws = ws[dev]; a.ws_elems = ws_elems[dev]; }
            int n = 0;
            e = tc_conv_launch(*plan, a, st, &n);
            return e == cudaSuccess ? SGS_OK : SGS_ECUDA;
        }
    }
    if (d->impl == 2) return SGS_EUNSUPPORTED;
    e = d->dtype == SGS_BF16 ? launch_conv_plain<__nv_bfloat16>(a, st) : launch_conv_plain<float>(a, st);
    return e == cudaSuccess ? SGS_OK : SGS_ECUDA;
}

// One sliced convolution layer with 8-bit operands on the tensor cores (see sgs.h).
sgs_status_t sgs_conv2d_sliced_i8(const sgs_conv_i8_desc_t *d, const void *d_x, const void *d_w, const int32_t *d_mult,
                                  const int32_t *d_shift, const int32_t *d_bias, const void *d_res, void *d_y, void *cuda_stream) {
    if (!d || !d_x || !d_w || !d_mult || !d_shift || !d_bias || !d_y) return SGS_EINVAL;
    if (d->N <= 0 || d->H <= 0 || d->W <= 0 || d->C <= 0 || d->K <= 0 || d->k <= 0 || (d->k & 1) == 0 || d->k > d->R ||
        ((d->R - d->k) & 1) || d->K > d->Kmax || d->C > d->Cmax || (d->stride != 1 && d->stride != 2) || d->res_shift < 0 || d->res_shift > 31)
        return SGS_EINVAL;
    if (d->zx != 0 || !tc_available()) return SGS_EUNSUPPORTED;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return SGS_ECUDA;
    ConvArgs a;
    a.x = d_x; a.w = d_w; a.res = d_res; a.y = d_y;
    a.N = d->N; a.H = d->H; a.W = d->W; a.C = d->C; a.K = d->K;
    a.Kmax = d->Kmax; a.Cmax = d->Cmax; a.R = d->R; a.k = d->k; a.stride = d->stride;
    const int p = (d->k - 1) / 2;
    a.Ho = (d->H + 2 * p - d->k) / d->stride + 1;
    a.Wo = (d->W + 2 * p - d->k) / d->stride + 1;
    a.i8 = 1;
    if (d->ldx < 0 || d->ldy < 0 || (d->ldx && d->ldx < d->C) || (d->ldy && d->ldy < d->K)) return SGS_EINVAL;
    a.ldx = d->ldx; a.ldy = d->ldy;
    a.q_mult = d_mult; a.q_shift = d_shift; a.q_bias = d_bias;
    a.q_zy = d->zy; a.q_zr = d->zr; a.q_res_mult = d->res_mult; a.q_res_shift = d->res_shift;
    a.q_flags = (d->x_signed ? 1 : 0) | (d->y_signed ? 2 : 0) | (d->res_signed ? 4 : 0) | (d->relu ? 8 : 0);
    std::string why;
    std::shared_ptr<TcConvPlan> plan = tc_conv_prepare(a, dev, &why);
    if (!plan) return SGS_EUNSUPPORTED;
    int n = 0;
    return tc_conv_launch(*plan, a, (cudaStream_t)cuda_stream, &n) == cudaSuccess ? SGS_OK : SGS_ECUDA;
}

// Non-convolution layers on caller tensors (see sgs.h).  Mirrors the dispatch of launch_op / wave_impl.
sgs_status_t sgs_aux_op(int n, const sgs_aux_desc_t *desc, const sgs_aux_args_t *args, int grouped, void *cuda_stream) {
    if (n <= 0 || n > 65535 || !desc || !args) return SGS_EINVAL;
    cudaStream_t st = (cudaStream_t)cuda_stream;
    std::vector<SmallEntry> es((size_t)n);
    int kind0 = -1;
    for (int m = 0; m < n; m++) {
        const sgs_aux_desc_t &d = desc[m];
        const sgs_aux_args_t &a = args[m];
        if (d.kind < SGS_AUX_MAXPOOL || d.kind > SGS_AUX_SE_SCALE || (d.dtype != SGS_F32 && d.dtype != SGS_BF16)) return SGS_EINVAL;
        if (!a.x || !a.y || d.N <= 0 || d.H <= 0 || d.W <= 0 || d.C <= 0 || d.act < 0 || d.act > 2) return SGS_EINVAL;
        const bool fc = d.kind == SGS_AUX_LINEAR || d.kind == SGS_AUX_SE_GATE;
        if (fc && (!a.w || !a.bias || d.K <= 0 || d.ld < d.C)) return SGS_EINVAL;
        if (d.kind == SGS_AUX_SE_GATE && (!a.w2 || !a.bias2 || d.ld2 < d.K)) return SGS_EINVAL;
        if (d.kind == SGS_AUX_SE_SCALE && !a.w) return SGS_EINVAL;
        SmallEntry &e = es[(size_t)m];
        std::memset(&e, 0, sizeof e);
        e.x = a.x; e.y = a.y; e.w = a.w; e.bias = a.bias; e.w2 = a.w2; e.bias2 = a.bias2;
        e.N = d.N; e.H = d.H; e.W = d.W; e.C = d.C; e.K = d.K; e.ld = d.ld; e.ld2 = d.ld2; e.act = d.act;
        e.Ho = (d.H - 1) / 2 + 1; e.Wo = (d.W - 1) / 2 + 1;
        static const int kinds[5] = {OP_MAXPOOL, OP_GAP, OP_LINEAR, OP_SE_GATE, OP_SCALE};
        const int kind = kinds[d.kind];
        if (m == 0) kind0 = kind;
        if (grouped && (kind != kind0 || d.dtype != SGS_BF16 || d.dtype != desc[0].dtype || !small_supported(kind, e))) return SGS_EUNSUPPORTED;
    }
    if (grouped) {
        SmallEntry *d_tbl = nullptr;
        if (cudaMalloc((void **)&d_tbl, (size_t)n * sizeof(SmallEntry)) != cudaSuccess) return SGS_ENOMEM;
        cudaError_t e = cudaMemcpyAsync(d_tbl, es.data(), (size_t)n * sizeof(SmallEntry), cudaMemcpyHostToDevice, st);
        if (e == cudaSuccess) e = launch_small(kind0, es.data(), d_tbl, n, st);
        const cudaError_t e2 = cudaStreamSynchronize(st);
        cudaFree(d_tbl);
        return (e == cudaSuccess && e2 == cudaSuccess) ? SGS_OK : SGS_ECUDA;
    }
    for (int m = 0; m < n; m++) {
        const sgs_aux_desc_t &d = desc[m];
        const SmallEntry &e = es[(size_t)m];
        const bool bf = d.dtype == SGS_BF16;
        cudaError_t ce = cudaSuccess;
        using B = __nv_bfloat16;
        switch (d.kind) {
        case SGS_AUX_MAXPOOL:
            ce = bf ? launch_maxpool3s2<B>((const B *)e.x, (B *)e.y, d.N, d.H, d.W, d.C, st) : launch_maxpool3s2<float>((const float *)e.x, (float *)e.y, d.N, d.H, d.W, d.C, st);
            break;
        case SGS_AUX_AVGPOOL:
            ce = bf ? launch_gap<B>((const B *)e.x, (float *)e.y, d.N, d.H * d.W, d.C, st) : launch_gap<float>((const float *)e.x, (float *)e.y, d.N, d.H * d.W, d.C, st);
            break;
        case SGS_AUX_LINEAR:
            ce = bf ? launch_linear<B>((const float *)e.x, (const B *)e.w, e.bias, (float *)e.y, d.N, d.C, d.K, d.ld, d.act, st)
                    : launch_linear<float>((const float *)e.x, (const float *)e.w, e.bias, (float *)e.y, d.N, d.C, d.K, d.ld, d.act, st);
            break;
        case SGS_AUX_SE_GATE:
            ce = bf ? launch_se_gate<B>((const float *)e.x, (const B *)e.w, e.bias, (const B *)e.w2, e.bias2, (float *)e.y, d.N, d.C, d.K, d.ld, d.ld2, st)
                    : launch_se_gate<float>((const float *)e.x, (const float *)e.w, e.bias, (const float *)e.w2, e.bias2, (float *)e.y, d.N, d.C, d.K, d.ld, d.ld2, st);
            break;
        default:
            ce = bf ? launch_scale<B>((const B *)e.x, (const float *)e.w, (B *)e.y, d.N, d.H * d.W, d.C, st)
                    : launch_scale<float>((const float *)e.x, (const float *)e.w, (float *)e.y, d.N, d.H * d.W, d.C, st);
            break;
        }
        if (ce != cudaSuccess) return SGS_ECUDA;
    }
    return SGS_OK;
}

int sgs_device_status(void) { return tc_conv_status(); }

sgs_status_t sgs_device_status_clear(void) { return tc_conv_status_clear() == cudaSuccess ? SGS_OK : SGS_ECUDA; }

sgs_status_t sgs_measure_fma_peak(double *tflops, void *cuda_stream) {
    if (!tflops) return SGS_EINVAL;
    return measure_fma_rate(tflops, (cudaStream_t)cuda_stream) == cudaSuccess ? SGS_OK : SGS_ECUDA;
}

sgs_status_t sgs_debug_expire_wait(unsigned limit_us, void *cuda_stream) {
    if (limit_us == 0 || limit_us > 1000000u) return SGS_EINVAL;
    return tc_expire_wait(limit_us, (cudaStream_t)cuda_stream) == cudaSuccess ? SGS_OK : SGS_ECUDA;
}

}  // extern "C"
