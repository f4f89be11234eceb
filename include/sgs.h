/*
 * sgs.h - C interface of the SubGraph-Stationary SubNet inference library for NVIDIA B200.
 *
 * The library executes a stream of inference queries, each activating a different SubNet of one
 * weight-shared SuperNet (paper: "SubGraph Stationary Hardware-Software Inference Co-design",
 * Sections 2.1, 2.2 and 3.1).  A SubNet is never copied out of the SuperNet: elastic width and
 * expand ratio select the first K' filters / first C' channels of a stored layer, elastic kernel
 * selects the centre k x k window of the stored kernel, elastic depth keeps the first d blocks of
 * a stage.  The weights shared by recent queries (their common SubGraph) are kept on chip instead
 * of being fetched again from HBM (Section 2.2, Section 4.2 "Persistent Buffer", Section 4.3.1).
 *
 * Conventions
 *   - Every function returns an sgs_status_t (SGS_OK == 0); none throws or aborts.  A text for the
 *     last failure of a handle is available from sgs_last_error().
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA device memory on the
 *     device the SuperNet was loaded on (for example torch.Tensor.data_ptr()).
 *   - Activations are NHWC.  In SGS_BF16 mode inputs are bfloat16 and arithmetic is bf16 x bf16
 *     with fp32 accumulation; every layer output is rounded to bf16 when it is stored.  In
 *     SGS_F32 mode everything is fp32.  Logits are always fp32, [batch][n_classes].
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the default stream).
 *   - A handle is not re-entrant: use it from one host thread / one stream at a time.
 *   - The library needs a CUDA device of compute capability 10.0 and fails with SGS_EUNSUPPORTED
 *     or SGS_ECUDA otherwise; there is no CPU fallback.
 */
#ifndef SGS_H_
#define SGS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SGS_MAX_STAGES 8
#define SGS_MAX_BLOCKS 8

typedef struct sgs_supernet sgs_supernet_t; /* opaque; owns all device weight memory */

typedef enum {
    SGS_OK = 0,
    SGS_EINVAL = 1,      /* NULL pointer, bad size, bad enum */
    SGS_ECONFIG = 2,     /* SubNet config outside the SuperNet's elastic sets */
    SGS_ENOMEM = 3,      /* host or device allocation failed */
    SGS_ECUDA = 4,       /* a CUDA call failed */
    SGS_ETIMEOUT = 5,    /* a bounded device-side wait ran out (kernel returned cleanly) */
    SGS_EUNSUPPORTED = 6 /* shape / device not supported */
} sgs_status_t;

typedef enum { SGS_F32 = 0, SGS_BF16 = 1 } sgs_dtype_t;
typedef enum { SGS_TINY = 0, SGS_RESNET = 1, SGS_MBV3 = 2 } sgs_family_t;

/* SuperNet family and maxima.  Only `family` selects behaviour; the other fields are checked
 * against the family's built-in definition (0 = do not check). */
typedef struct {
    int family; /* sgs_family_t */
    int n_stages;
    int max_depth[SGS_MAX_STAGES];
    int base_width[SGS_MAX_STAGES];
    int stem_width;
    int n_classes;
    int max_kernel;
} sgs_arch_desc_t;

/* Elastic choices of one SubNet (paper Section 2.1).
 *   depth[s]      blocks kept in stage s: the first depth[s] blocks
 *   width[0]      stem width multiplier; width[1+s] width multiplier of stage s
 *   expand[s][b]  expand ratio of block b of stage s
 *   kernel[s][b]  depthwise kernel size of block b of stage s (MobileNetV3-shaped family)
 * Fields a family does not use are ignored. */
typedef struct {
    int depth[SGS_MAX_STAGES];
    float width[SGS_MAX_STAGES + 1];
    float expand[SGS_MAX_STAGES][SGS_MAX_BLOCKS];
    int kernel[SGS_MAX_STAGES][SGS_MAX_BLOCKS];
} sgs_subnet_cfg_t;

enum { SGS_POLICY_INTERSECTION = 0, SGS_POLICY_AVGNET = 1 };

/* Options of sgs_stream_run. */
typedef struct {
    int cache_enabled;  /* 1: keep the SubGraph shared by recent queries resident in L2 */
    int window_q;       /* the cached SubGraph is re-chosen every window_q queries from the last
                           window_q SubNets (paper Section 3.3 and Appendix A.1); >= 1 */
    size_t cache_budget_bytes; /* 0 = the device's persisting-L2 maximum */
    int use_graphs;     /* 1: replay one captured CUDA graph per distinct (config, batch, res);
                           ignored on the legacy default stream, which cannot be captured */
    int record_latency; /* 1: bracket every query with events and fill the latency statistics */
    int weights_evict_first; /* with the cache off: 1 marks weight loads evict-first, which removes
                                the reuse the hardware L2 replacement gives for free */
    int concurrency;    /* queries of the stream in flight at once (they are independent; each gets its
                           own workspaces and CUDA stream, query t uses slot t % concurrency; the
                           caching decisions still follow the stream order).  0 or 1 = one at a time;
                           at most 16.  From 12 up the convolutions pick tiles for aggregate throughput
                           instead of single-launch latency.  More than 8 only overlap if the process
                           raised CUDA_DEVICE_MAX_CONNECTIONS before its CUDA context was created.
                           Results are bit-identical for a given tile choice (i.e. for <12 and for >=12). */
    int wave;           /* 0 = off.  G > 0 (at most 64, bf16 handles only): G consecutive queries form a
                           wave that advances through the layers together; at every layer the tensor-core
                           convolutions of all members whose SubNet has that layer are ONE grouped launch
                           (each member with its own slice of the shared weights), so a launch fills the
                           GPU although a single batch-1 SubNet cannot.  `concurrency` then counts waves
                           in flight (0 = 2, at most 8) and use_graphs is ignored.  Every query of a wave
                           starts and ends with its wave (that is its recorded latency).  The cached
                           SubGraph is still re-chosen in stream order, and every member's weight loads carry
                           the choice in force when ITS query is served (a wave of 32 with window_q = 4 sees
                           eight choices). */
    int policy;         /* how the cached SubGraph is chosen every window_q queries:
                           SGS_POLICY_INTERSECTION (0): the SubGraph common to the last window_q SubNets;
                           SGS_POLICY_AVGNET (1): Algorithm 1 - the candidate SubGraph (sgs_cache_set_candidates)
                           nearest to the running average of the last window_q SubNets' encodings */
    int persistent;     /* 1 (bf16 handles of the MobileNetV3-shaped family, one image per query): the whole stream
                           is ONE launch of a persistent kernel; every SM takes the next unserved query and runs all
                           layers of its SubNet by itself out of a private scratch area, pointwise convolutions on the
                           tensor cores (Section 3.1: one query per pass of the accelerator; Section 4.2: what is needed
                           again stays on chip).  wave, concurrency and use_graphs are ignored; every query starts and
                           ends with the launch (its recorded latency).  With the cache enabled one SubGraph is chosen for the launch,
                           from the call's first window_q queries, and every SM keeps its first pointwise layers in shared
                           memory for all the queries it serves; hit_ratio and hbm_weight_bytes are then against what is
                           held on chip.  Other handles: SGS_EUNSUPPORTED. */
} sgs_stream_opts_t;

/* Results of sgs_stream_run (all host-side; filled after the stream has been synchronised). */
typedef struct {
    int n_queries;
    double total_ms;        /* device time of the whole stream (events on the given stream) */
    double queries_per_s;   /* n_queries / total time */
    double images_per_s;    /* queries_per_s * batch_per_query */
    double p50_ms, p99_ms, mean_ms; /* per query; 0 unless record_latency */
    double useful_flops;    /* 2*M*K'*C'*k*k summed over the sliced layers of all queries */
    double weight_bytes;    /* stored-weight bytes the SubNets touch, summed over queries */
    double hbm_weight_bytes;/* analytic: bytes of SN_t not inside the cached SubGraph G_t */
    double hit_ratio;       /* mean over t of ||SN_t ∩ G_t||_2 / ||SN_t||_2 (paper Appendix A.4) */
    double byte_hit_ratio;  /* 1 - hbm_weight_bytes / weight_bytes */
    long long kernel_launches;
    int plan_hits, plan_misses;
    int cache_updates;      /* how many times the cached SubGraph changed */
} sgs_stream_stats_t;

/* State of the SubGraph cache. */
typedef struct {
    int enabled;
    int window_q;
    size_t budget_bytes;           /* after clamping to what the device offers */
    size_t l2_bytes;               /* cudaDevAttrL2CacheSize */
    size_t persisting_l2_max;      /* cudaDevAttrMaxPersistingL2CacheSize */
    size_t access_window_max;      /* cudaDevAttrMaxAccessPolicyWindowSize */
    size_t cached_subgraph_bytes;  /* weight bytes of the SubGraph currently marked resident */
    size_t supernet_bytes;         /* device bytes of all stored weights */
    size_t device_bytes_allocated; /* every device byte the handle owns (weights + workspaces) */
    int policy;                    /* SGS_POLICY_* in force; 2 while a scheduler object pins the cache */
    int n_candidates;              /* size of the candidate set S */
    int decisions;                 /* caching decisions taken since the cache was last reset */
    int last_choice;               /* index into S of the last AvgNet decision; -1 = none yet */
} sgs_cache_stats_t;

/*
 * sgs_supernet_load - build a SuperNet on `device` from a host blob (Section 2.1: one stored set of
 * weights contains every SubNet).
 *   arch       family (and optional maxima to cross-check)
 *   host_blob  host pointer, `nbytes` bytes, in the self-describing record format written by the
 *              workload generator: header of 8 uint32 (magic 'SGSB', version 1, family, n_records,
 *              seed, 0, 0, 0); per stored layer a record header of 8 uint32 (kind 0 conv / 1 depthwise
 *              / 2 linear, K_max, C_max, R, S, has_bn, has_bias, 0) followed by fp32
 *              weight[K_max][C_max][R][S], then gamma, beta, mean, var [K_max] if has_bn, then
 *              bias[K_max] if has_bias.  The blob is copied; the caller keeps ownership.
 *   compute_dtype  SGS_BF16 (weights re-laid out as bf16 [K][R][S][C]) or SGS_F32
 *   out        receives the handle; free with sgs_supernet_free
 * Batch norm is folded into a per-filter scale and shift at load.
 * Errors: SGS_EINVAL (NULL, bad header, blob does not match the family), SGS_ENOMEM, SGS_ECUDA,
 * SGS_EUNSUPPORTED (no sm_100 device).
 */
sgs_status_t sgs_supernet_load(const sgs_arch_desc_t *arch, const void *host_blob, size_t nbytes,
                               sgs_dtype_t compute_dtype, int device, sgs_supernet_t **out);

/* Check a config against the SuperNet's elastic sets (Section 2.1).  SGS_OK or SGS_ECONFIG. */
sgs_status_t sgs_subnet_validate(const sgs_supernet_t *net, const sgs_subnet_cfg_t *cfg);

/*
 * sgs_subnet_run - one query: inference of the SubNet `cfg` on `batch` images (Section 3.1: the
 * accelerator performs inference of the query using the selected SubNet).
 *   d_input   device pointer, [batch][res][res][3] NHWC, compute dtype, caller-owned, read only
 *   d_logits  device pointer, [batch][n_classes] fp32, caller-owned, written
 * Asynchronous on `cuda_stream`.  Invalid config -> SGS_ECONFIG before anything is launched.
 * No sliced copy of any weight is made; the only device memory that may grow is the activation
 * workspace (and the split-reduction scratch) on the first use of a larger (batch, res).
 */
sgs_status_t sgs_subnet_run(sgs_supernet_t *net, const sgs_subnet_cfg_t *cfg, const void *d_input, int batch,
                            int res, void *d_logits, void *cuda_stream);

/*
 * sgs_stream_run - a stream of queries (Sections 2.1 and 3.1), query t using cfgs[t] on
 * inputs[t] = d_inputs + t*batch_per_query*res*res*3 elements, writing logits[t] =
 * d_logits + t*batch_per_query*n_classes floats.  With the cache enabled the SubGraph shared by the
 * last window_q queries (element-wise minimum of their layer encodings = their exact intersection,
 * Section 2.2, Appendix A.4) is marked resident for the following queries.
 * Synchronises the stream before filling `stats` (may be NULL).  `opts` NULL = cache on, window 4,
 * graphs on, latency recorded, one query at a time.  Per-query latency is measured from the moment
 * the query's first operation starts on its slot's stream to its last operation's end.
 */
sgs_status_t sgs_stream_run(sgs_supernet_t *net, int n_queries, const sgs_subnet_cfg_t *cfgs,
                            const void *d_inputs, int batch_per_query, int res, void *d_logits,
                            const sgs_stream_opts_t *opts, sgs_stream_stats_t *stats, void *cuda_stream);

/*
 * sgs_stream_run_host - the same stream with HOST buffers: each query's input is copied host->device
 * and its logits device->host inside the call (inputs in the compute dtype, logits fp32).  Host
 * memory may be pageable or pinned; pinned memory overlaps better.
 */
sgs_status_t sgs_stream_run_host(sgs_supernet_t *net, int n_queries, const sgs_subnet_cfg_t *cfgs,
                                 const void *h_inputs, int batch_per_query, int res, void *h_logits,
                                 const sgs_stream_opts_t *opts, sgs_stream_stats_t *stats, void *cuda_stream);

/* sgs_cache_configure - the SubGraph cache used by sgs_subnet_run (sgs_stream_run takes its own options).
 * budget_bytes plays the part of the Persistent Buffer's capacity (Section 4.2: the buffer that holds the cached
 * SubGraph across queries); 0 = the most the device lets a process keep resident in L2.  window_q >= 1 is the
 * number of queries a caching decision is amortised over (Section 3.3 "Amortizing Caching Choices", Appendix A.1:
 * the cached SubGraph is re-chosen every Q queries from the last Q SubNets).  Errors: SGS_EINVAL.
 * sgs_cache_stats - state of that cache: what the device offers, the budget in force, the bytes of the SubGraph
 * currently marked resident (Section 4.3.1: the part of a query's weights that is not fetched again), and the
 * policy's counters.  `out` is a host struct.  Errors: SGS_EINVAL. */
sgs_status_t sgs_cache_configure(sgs_supernet_t *net, int enabled, size_t budget_bytes, int window_q);
sgs_status_t sgs_cache_stats(const sgs_supernet_t *net, sgs_cache_stats_t *out);

/*
 * sgs_cache_set_candidates - the set S of cacheable SubGraphs the scheduler chooses from (Section 3.2;
 * Algorithm 1's G_j).  cfgs: host array of n SubNet configs; candidate j is the vector encoding
 * (Section 3.3) of cfgs[j], with layers dropped, in network order, once the byte budget of the cache
 * is used up (re-applied whenever the budget changes).  The configs are copied.  n = 0 removes the set
 * and returns to SGS_POLICY_INTERSECTION.  Host-only; takes effect at the next caching decision.
 * Errors: SGS_EINVAL, SGS_ECONFIG (a config outside the elastic sets; the old set is kept).
 *
 * sgs_cache_set_policy - policy of the cache used by sgs_subnet_run (sgs_stream_run takes it from its
 * options).  SGS_POLICY_AVGNET: after every window_q queries, AvgNet = element-wise mean of the last
 * window_q encodings and the cached SubGraph becomes argmin_j Dist(G_j, AvgNet), Dist = Euclidean
 * distance over the (K_i, C_i) entries, compared exactly, ties to the lowest j.  SGS_EINVAL without a
 * candidate set.
 */
sgs_status_t sgs_cache_set_candidates(sgs_supernet_t *net, const sgs_subnet_cfg_t *cfgs, int n);
sgs_status_t sgs_cache_set_policy(sgs_supernet_t *net, int policy);

/*
 * Scheduler object: Algorithm 1 (Section 3.3) over a latency table with SubNets as rows and cacheable
 * SubGraphs as columns (Section 3.2).  Host-side state only, apart from sgs_sched_measure.
 *
 * sgs_sched_create - rows = `subnets` (host array of n_subnets configs, copied) with their `accuracy`
 *   (host array of n_subnets doubles, copied; any monotone proxy will do), columns = the candidate set
 *   installed with sgs_cache_set_candidates at this moment (M of them) plus column M = nothing cached.
 *   window_q >= 1 = Algorithm 1's Q.  The table starts as zeros; the cache of `net` is emptied and from
 *   now on moves only when the scheduler decides (sgs_subnet_run no longer re-chooses it; a later
 *   sgs_stream_run takes the cache back).  `net` must outlive the scheduler; do not change the candidate
 *   set or the cache budget while it lives.  Errors: SGS_EINVAL (no candidate set, bad argument),
 *   SGS_ECONFIG, SGS_ENOMEM.
 * sgs_sched_dims - n_subnets and n_columns (= M + 1); either pointer may be NULL.
 * sgs_sched_set_table / sgs_sched_get_table - latency[i * n_columns + j], host doubles, any unit.
 * sgs_sched_measure - fills the table on the device: for every column j the cache is pinned to SubGraph j
 *   and every SubNet i runs once untimed and then `reps` (1..1000) times on `cuda_stream` between two
 *   events; entry = median in milliseconds.  Before each timed run `flush_bytes` bytes of scratch owned by
 *   the scheduler are overwritten (0 = no flush): this stands for the other traffic of a serving system
 *   that pushes unprotected weights out of L2 between two queries.  d_input [batch][res][res][3] in the
 *   compute dtype and d_logits [batch][n_classes] fp32 are caller-owned device buffers.  Synchronises
 *   the stream.  Afterwards the cache is pinned to the scheduler's current state again.
 * sgs_sched_step - n queries in order.  Query t = (policy[t], a_t[t], l_t[t]) with policy
 *   SGS_STRICT_ACCURACY (serve the fastest SubNet among those with accuracy >= a_t) or SGS_STRICT_LATENCY
 *   (serve the most accurate SubNet among those with latency <= l_t), latency taken from the column of the
 *   current cache state.  An empty feasible set falls back to the most accurate / the fastest SubNet; ties
 *   are broken by the other quantity, then by the lowest row.  subnet[t] receives the row served,
 *   cache_state[t] (may be NULL) the column it was served under.  After every window_q-th query the cache
 *   state becomes the candidate nearest to the mean encoding of the last window_q served SubNets (as
 *   SGS_POLICY_AVGNET) and is enacted on `net` when the call returns.  All arrays are host arrays.
 * sgs_sched_subnet - copies row i's config to *out (to pass to sgs_subnet_run).
 */
typedef struct sgs_sched sgs_sched_t;
enum { SGS_STRICT_ACCURACY = 0, SGS_STRICT_LATENCY = 1 };
sgs_status_t sgs_sched_create(sgs_supernet_t *net, const sgs_subnet_cfg_t *subnets, const double *accuracy, int n_subnets,
                              int window_q, sgs_sched_t **out);
void sgs_sched_free(sgs_sched_t *sched);
sgs_status_t sgs_sched_dims(const sgs_sched_t *sched, int *n_subnets, int *n_columns);
sgs_status_t sgs_sched_set_table(sgs_sched_t *sched, const double *latency);
sgs_status_t sgs_sched_get_table(const sgs_sched_t *sched, double *latency);
sgs_status_t sgs_sched_measure(sgs_sched_t *sched, const void *d_input, int batch, int res, void *d_logits, int reps,
                               size_t flush_bytes, void *cuda_stream);
sgs_status_t sgs_sched_step(sgs_sched_t *sched, int n, const int *policy, const double *a_t, const double *l_t,
                            int *subnet, int *cache_state);
sgs_status_t sgs_sched_subnet(const sgs_sched_t *sched, int i, sgs_subnet_cfg_t *out);

/*
 * Vector encoding of a SubNet (Section 3.3): for every stored layer i, out[3i] = K_i (filters),
 * out[3i+1] = C_i (channels), out[3i+2] = k_i (kernel size); zeros for layers the SubNet does not
 * use.  `out` is a host array of 3*sgs_num_layers() ints.
 */
int sgs_num_layers(const sgs_supernet_t *net);
sgs_status_t sgs_subnet_encode(const sgs_supernet_t *net, const sgs_subnet_cfg_t *cfg, int *out);

/* sgs_subnet_cost - what one query of SubNet `cfg` costs, from its slices alone (Section 2.1: the elastic choices
 * fix which weights take part; Section 2.2 / Figure on arithmetic intensity: FLOPs against bytes moved decides
 * whether a SubNet is memory bound): useful FLOPs (2*M*K'*C'*k*k over the sliced layers), the stored-weight bytes
 * the SubNet touches, and the activation bytes its layers read and write.  Host pointers, any may be NULL.
 * Errors: SGS_EINVAL, SGS_ECONFIG. */
sgs_status_t sgs_subnet_cost(const sgs_supernet_t *net, const sgs_subnet_cfg_t *cfg, int batch, int res,
                             double *flops, double *weight_bytes, double *activation_bytes);

/*
 * sgs_conv2d_sliced - one sliced convolution layer with its fused epilogue, on caller-owned device
 * tensors (paper Section 2.1: the layer uses the first K filters and first C channels of the stored
 * tensor and the centre k x k window of its stored R x R kernel; Section 4.2 "Output Buffer": only
 * final outputs leave the chip):
 *   y[n][ho][wo][f] = act( scale[f] * sum_{r,s<k} sum_{c<C} x[n][ho*stride+r-p][wo*stride+s-p][c]
 *                          * w[f][o+r][o+s][c] + shift[f] + res[n][ho][wo][f] ),   p = (k-1)/2, o = (R-k)/2
 *   d_x     [N][H][W][C] NHWC, dtype elements            d_y, d_res  [N][Ho][Wo][K] (d_res may be NULL)
 *   d_w     stored weights, [Kmax][R][R][Cmax] (depthwise: [R][R][Kmax]), dtype elements
 *   d_scale, d_shift  [>= K] fp32
 * impl 0 = automatic (tensor cores when dtype is bf16, C, K, Cmax are multiples of 8, pointers are
 * 16-byte aligned and stride-2 inputs have even sizes), 1 = CUDA-core kernel, 2 = tensor cores or
 * SGS_EUNSUPPORTED.  weight_policy 0 = no L2 hint, 1 = evict-last for weight tiles with filter <
 * cache_k and channel < cache_c (default replacement for the rest), 2 = all weights evict-first.
 * Asynchronous on `cuda_stream`.  The tensor-core path may split the reduction over several CTAs
 * using a per-device scratch buffer that this function allocates on demand (cudaMalloc) and keeps;
 * calls that overlap on the same device must therefore not run concurrently.
 */
typedef struct {
    int N, H, W, C, K;      /* input dims, sliced channels C, sliced filters K */
    int Kmax, Cmax, R;      /* stored tensor dims */
    int k, stride, act;     /* kernel size, stride (1 or 2), activation 0 none / 1 ReLU / 2 h-swish */
    int dtype;              /* sgs_dtype_t */
    int impl;
    int depthwise;
    int cache_k, cache_c, weight_policy;
    int split_k_off;        /* 1: never split the reduction */
} sgs_conv_desc_t;
sgs_status_t sgs_conv2d_sliced(const sgs_conv_desc_t *desc, const void *d_x, const void *d_w, const float *d_scale,
                               const float *d_shift, const void *d_res, void *d_y, void *cuda_stream);

/*
 * sgs_conv2d_sliced_static - sgs_conv2d_sliced for callers that may not allocate device memory.
 * (The paper has no counterpart to this call; it exists for the way the library is deployed.)
 *
 * Who needs it: serving processes that gave all device memory to their own pool at start-up (a cudaMalloc
 * from a library then simply fails), and latency-critical loops that cannot afford the device-wide
 * synchronisation cudaMalloc and cudaFree imply.  sgs_conv2d_sliced may call cudaMalloc to
 * grow its split-reduction scratch; this variant never does.  Its scratch is a fixed array of
 * SGS_STATIC_SCRATCH_BYTES that is part of the library image, so every GPU that loads the library
 * holds that much memory until the process exits.
 *
 * Same arguments, layouts and result as sgs_conv2d_sliced, with these limits:
 *   - tensor-core path only: dtype SGS_BF16, not depthwise, impl 0 or 2; otherwise SGS_EUNSUPPORTED
 *     (also for shapes the tensor-core kernel does not take).
 *   - a layer whose split reduction needs more than SGS_STATIC_SCRATCH_BYTES of partial tiles is
 *     rejected with SGS_ENOMEM and nothing is launched.  (Partial tiles take
 *     splits * N*Ho*Wo*K * 4 bytes with splits <= 8; layers large enough to fill the GPU are not split
 *     and need no scratch at all.  Set split_k_off = 1 to run any shape without scratch.)
 *   - no cudaMalloc, cudaFree or other allocating device call is made, on any call.
 * The first call on each device looks up the device address of the array and sets the kernels'
 * shared-memory limit; make that first call outside any stream capture.  Later calls only enqueue
 * kernels on `cuda_stream` (nothing in the array has to start at zero: what the second step of a
 * split reduction reads was written by the first step of the same call).
 * All calls on a device share the one array and it keeps whatever the last call left in it: two calls
 * whose kernels may overlap on the GPU (different streams, or concurrent host threads) race on it and
 * give wrong results.  Issue them on one stream, or order them with events.
 */
#define SGS_STATIC_SCRATCH_BYTES (8u << 20)
sgs_status_t sgs_conv2d_sliced_static(const sgs_conv_desc_t *desc, const void *d_x, const void *d_w, const float *d_scale,
                                      const float *d_shift, const void *d_res, void *d_y, void *cuda_stream);

/*
 * sgs_conv2d_sliced_i8 - one sliced convolution layer in the paper's own numeric format (Section 5.1, workload
 * footnote: weights, activations and zero points are 8-bit integers, the scale a 32-bit integer; Section 4.2
 * "Zero Point/Scale Buffer": the per-filter parameters the accelerator applies to its accumulators), on the 8-bit
 * tensor cores with int32 accumulation.  Slicing is the same as in sgs_conv2d_sliced (first K filters, first C
 * channels, centre k x k window).  All arithmetic is exact integer arithmetic:
 *   acc[n][ho][wo][f] = sum_{r,s<k} sum_{c<C} (x[n][ho*stride+r-p][wo*stride+s-p][c] - zx) * w[f][o+r][o+s][c]
 *                       (positions outside the image count as the real value 0, i.e. as zx)
 *   t = rsr(acc * mult[f], 31 + shift[f]) + bias[f]  [+ rsr((res[n][ho][wo][f] - zr) * res_mult, 31 + res_shift)]  + zy
 *   y = saturate(relu ? max(t, zy) : t)      with rsr(v, s) = floor((v + 2^(s-1)) / 2^s) in 64-bit arithmetic
 * so that a real-valued layer y_r = act(scale_f * conv(x_r, w_r) + shift_f + res_r) with x_r = sx (x - zx),
 * w_r = sw_f w, y_r = sy (y - zy) is represented by mult[f] * 2^-(31 + shift[f]) ~ sx * sw_f * scale_f / sy and
 * bias[f] ~ shift_f / sy.
 *   d_x    [N][H][W][C] bytes (unsigned, or signed if x_signed)     d_y, d_res  [N][Ho][Wo][K] bytes
 *   d_w    stored weights [Kmax][R][R][Cmax] signed bytes            d_mult, d_shift, d_bias  [>= K] int32
 * Limits of this entry point: pixels of x in multiples of 16 bytes (C a multiple of 16, or of 8 with ldx), Cmax a
 * multiple of 16, K a multiple of 8, 16-byte aligned pointers, stride-2
 * inputs of even size, 0 <= shift[f] <= 31, and zx == 0 (an input zero point other than 0 would need the sum of the
 * sliced weights under every window position, which changes with the slice and at image borders; post-ReLU tensors
 * and symmetric signed tensors have zx = 0).  Other values: SGS_EUNSUPPORTED.  Asynchronous on `cuda_stream`.
 */
typedef struct {
    int N, H, W, C, K;       /* input dims, sliced channels C, sliced filters K */
    int Kmax, Cmax, R;       /* stored tensor dims */
    int k, stride;           /* kernel size, stride (1 or 2) */
    int relu;                /* 1: y = max(t, zy) */
    int x_signed, y_signed, res_signed; /* 0: bytes are 0..255, 1: -128..127 */
    int zx, zy, zr;          /* zero points of x, y, res */
    int res_mult, res_shift; /* residual rescaling (ignored without d_res) */
    int ldx, ldy;            /* bytes per pixel of x, and of y and res; 0 = dense (C resp. K).  Padded pixels: multiples of 16 with
                                ZEROS beyond the slice in x; the layer writes the zeros of y (ldy - K < 16) */
} sgs_conv_i8_desc_t;
sgs_status_t sgs_conv2d_sliced_i8(const sgs_conv_i8_desc_t *desc, const void *d_x, const void *d_w, const int32_t *d_mult,
                                  const int32_t *d_shift, const int32_t *d_bias, const void *d_res, void *d_y, void *cuda_stream);

/*
 * sgs_aux_op - the layers of a SubNet that are not convolutions, one at a time on caller-owned device tensors
 * (the paper's SuperNets are the OFA ResNet50 / MobileNetV3 families of Section 5.1: max pool after the stem,
 * global average pool before the classifier and inside squeeze-excite blocks, fully connected layers sliced by
 * prefix like every other stored layer, Section 2.1).  For layer-level tests and microbenchmarks.
 *   SGS_AUX_MAXPOOL   y[n][ho][wo][c] = max over the 3x3 window at stride 2, padding 1 (padding never wins);
 *                     x [N][H][W][C] -> y [N][(H-1)/2+1][(W-1)/2+1][C], dtype elements
 *   SGS_AUX_AVGPOOL   y[n][c] = mean over H*W pixels (fixed summation order); x [N][H][W][C] dtype -> y [N][C] fp32
 *   SGS_AUX_LINEAR    y[n][j] = act(sum_{c<C} w[j][c] x[n][c] + bias[j]), j < K; x [N][C] fp32, w [>=K][ld] dtype
 *                     (ld = stored input width >= C), bias [>=K] fp32, y [N][K] fp32
 *   SGS_AUX_SE_GATE   y[n][c] = hsigmoid(b2[c] + sum_{j<K} w2[c][j] relu(b1[j] + sum_{i<C} w[j][i] x[n][i])), c < C;
 *                     x [N][C] fp32 pooled vectors, w [>=K][ld], w2 [>=C][ld2] dtype, y [N][C] fp32
 *   SGS_AUX_SE_SCALE  y[n][h][w][c] = x[n][h][w][c] * g[n][c]; x, y [N][H][W][C] dtype, g = `w` [N][C] fp32
 * n_members >= 1 independent problems desc[m] / args[m].  grouped = 0: each runs in the kernel a single query
 * uses; grouped = 1: all of them (same kind and dtype SGS_BF16) run in ONE launch of the kernel a wave uses, whose
 * per-member records this call uploads to a temporary device table (it allocates and synchronises the stream).
 * Shapes the vectorised kernels do not take (channel counts that are not multiples of 8, unaligned pointers) fall back
 * to scalar kernels when grouped = 0 and are SGS_EUNSUPPORTED when grouped = 1.
 * Errors: SGS_EINVAL (NULL, non-positive size, K > ld ...), SGS_EUNSUPPORTED, SGS_ENOMEM, SGS_ECUDA.
 */
typedef enum { SGS_AUX_MAXPOOL = 0, SGS_AUX_AVGPOOL = 1, SGS_AUX_LINEAR = 2, SGS_AUX_SE_GATE = 3, SGS_AUX_SE_SCALE = 4 } sgs_aux_kind_t;
typedef struct {
    int kind;         /* sgs_aux_kind_t */
    int dtype;        /* sgs_dtype_t of tensors and weights */
    int N, H, W, C;   /* images, map size (1 x 1 for vectors), channels / input features */
    int K;            /* linear: outputs; SE gate: squeeze width */
    int ld, ld2;      /* row pitch (elements) of w and of w2 */
    int act;          /* linear: 0 none / 1 ReLU / 2 h-swish */
} sgs_aux_desc_t;
typedef struct {
    const void *x;
    void *y;
    const void *w;
    const float *bias;
    const void *w2;
    const float *bias2;
} sgs_aux_args_t;
sgs_status_t sgs_aux_op(int n_members, const sgs_aux_desc_t *desc, const sgs_aux_args_t *args, int grouped, void *cuda_stream);

/* Nonzero once a kernel of this process has reported that one of its bounded waits ran out (the paper has no
 * counterpart: every device-side wait of the kernels carries a time limit, after which the kernel records the fact
 * in a status word of its device, lets its copies land, frees its tensor memory and returns; calls that follow
 * report SGS_ETIMEOUT).  Reads the status words of the current device (sgs_conv2d_sliced_static keeps its own);
 * the answer is sticky until sgs_device_status_clear. */
int sgs_device_status(void);

/* Synchronises the current device, zeroes its status words and forgets earlier time-outs. */
sgs_status_t sgs_device_status_clear(void);

/* Measurement aid: the fp32 fused-multiply-add rate of the device's CUDA cores in TFLOP/s (2 FLOP per FMA), from a
 * kernel of independent register-only FMA chains, best of four timed launches on `cuda_stream`.  It is the ceiling
 * for the depthwise kernels with 5x5 and 7x7 windows, whose arithmetic intensity exceeds what the CUDA cores
 * sustain per byte of HBM traffic (paper Section 4.4: depthwise layers have the least reuse).  Allocates a small
 * scratch buffer and synchronises. */
sgs_status_t sgs_measure_fma_peak(double *tflops, void *cuda_stream);

/* Test aid for the time-out path: enqueues a one-block kernel on `cuda_stream` whose only wait can never be
 * satisfied, with a limit of limit_us microseconds (1 .. 1000000).  The kernel gives up after the limit, sets the
 * device status word exactly as the convolution kernels do, and returns normally; nothing faults or hangs. */
sgs_status_t sgs_debug_expire_wait(unsigned limit_us, void *cuda_stream);

/* Library options by name (debug and measurement aids): "conv_impl" 0 = automatic, 1 = force the
 * CUDA-core kernels; "pad_channels" 1 (default) = waves of the ResNet-shaped family keep their activation tensors
 * at 16-channel pixels (zeros beyond the slice), 0 = dense pixels; "cache_mechanism" how grouped launches keep the cached SubGraph in L2: 0 (default) = an evict-last
 * hint on every weight tile inside the SubGraph's box, 1 = an access-policy window on the launch (the cached filter
 * prefix of the launch's stored layer, persisting; the persisting-L2 carve-out of the process is sized to the cache
 * budget), 2 = both; "dw_walk" N = stride-1 depthwise launches of at least N million output
 * elements take the walking kernel (default 48; 0 never, negative always; process-wide); "persistent_held_kb" n = shared memory per SM that persistent
 * execution spends on the cached SubGraph's first pointwise layers (default 16, 0 = none); "nvtx" 1 = an NVTX range named after the stored layer around
 * every launch (for timeline tools); "fail_alloc_after" n = the handle's device allocations fail from
 * the (n+1)-th on with SGS_ENOMEM (fault injection on the host, -1 = off); "drop_plans" forgets every cached plan (measuring what a never-seen config costs); "profile" see
 * sgs_profile_read; "stage_group" 0 = default, 1..4 = pipeline stages that
 * share one barrier pair in the grouped convolution kernel (process-wide, a tuning aid).  Unknown name -> SGS_EINVAL. */
sgs_status_t sgs_set_option(sgs_supernet_t *net, const char *name, long long value);

/*
 * Per-kernel-class timing.  After sgs_set_option(net, "profile", 2) (2 = on and reset, 1 = on, 0 = off)
 * every kernel the handle launches is bracketed by CUDA events on the launching stream (graphs are
 * bypassed and queries run one at a time meanwhile; a short sleeping kernel ahead of every 8 queries
 * lets the host queue their launches first, so the intervals hold device time, not launch latency).  kernel_class: 0 tensor-core convolution, 1 CUDA-core convolution,
 * 2 depthwise convolution, 3 everything else.  Returns the launches, their summed device time, their
 * summed algorithmic bytes (sliced weights + input + output + residual of each launch) and useful
 * FLOPs since the last reset.  Synchronises the device.
 */
sgs_status_t sgs_profile_read(sgs_supernet_t *net, int kernel_class, long long *launches, double *total_ms,
                              double *alg_bytes, double *flops);

/*
 * Per-launch timing of waves.  While the profile is on, every launch of a wave (sgs_stream_opts_t.wave > 0)
 * also leaves one record, in issue order, until the next reset (at most 65536 are kept): its kernel class,
 * the stored layer it ran (index as in sgs_subnet_encode; the first of two for a launch that merges two
 * layers; -1 for operations without weights: pools, padding, SE scale), how many wave members it served, its
 * tiles (tensor-core convolutions, else 0), its device time and its algorithmic bytes and useful FLOPs.
 * sgs_profile_trace copies up to `cap` records to the host array `out` and returns how many exist (-1 on a
 * bad argument).  sgs_layer_name copies the name of a stored layer (NUL-terminated, truncated to cap - 1
 * characters) and returns its full length, -1 for a bad argument.
 */
typedef struct {
    int kernel_class, layer, members, tiles;
    double ms, alg_bytes, flops;
} sgs_launch_record_t;
int sgs_profile_trace(sgs_supernet_t *net, sgs_launch_record_t *out, int cap);
int sgs_layer_name(const sgs_supernet_t *net, int layer, char *out, int cap);

/* Counters by name ("kernel_launches", "plan_hits", "plan_misses", "device_bytes", "tc_convs";
 * diagnostics: "host_us_stream", "host_us_query", "host_us_table", "host_us_graph", "host_us_direct" =
 * accumulated host microseconds spent issuing streams / queries / cache-table updates / graph
 * launches / direct launches). */
long long sgs_get_counter(const sgs_supernet_t *net, const char *name);

/* Text of the last failure reported by a call on `net` (owned by the handle, valid until its next call); "null
 * handle" for NULL.  Library housekeeping: the paper has no counterpart. */
const char *sgs_last_error(const sgs_supernet_t *net);
/* Releases the SuperNet (Section 2.1: the one stored set of weights) with every device and host resource the handle
 * owns: weights, workspaces, plans, graphs, streams.  Synchronises the device first.  NULL is ignored. */
void sgs_supernet_free(sgs_supernet_t *net);

#ifdef __cplusplus
}
#endif
#endif /* SGS_H_ */
