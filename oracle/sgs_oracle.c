/*
 * CPU checker for SubNet inference on a weight-shared SuperNet.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the GPU library
 * must compute.  It shares no code, header, table or helper with the CUDA path and must never be
 * called from it.  fp32 arithmetic, direct nested loops, no BLAS, no im2col, no tiling.
 *
 * What it follows (paper = "SubGraph Stationary Hardware-Software Inference Co-design"):
 *   - Section 2.1: a SuperNet is a collection of stages, each a run of repeating blocks, each a
 *     few convolution layers; a SubNet is obtained by *selecting* weights of the SuperNet through
 *     its elastic dimensions (depth = the first d blocks of a stage; width / expand ratio = the
 *     first K' filters and first C' channels of a layer; kernel size).  The paper names the kernel
 *     dimension without giving its rule; the centre k x k window of the stored kernel is used.
 *   - Section 1: SubNets are activated without being extracted into separately stored models.
 *     The sliced forward below therefore indexes the stored tensors directly; a second, separate
 *     code path (orc_forward_extracted) copies the slices out first and runs dense loops, so the
 *     two can be compared.
 *   - Section 3.3 ("Encoding SubGraph NN Architecture"): a net is the vector [K_1, C_1, ...,
 *     K_N, C_N] of kernel and channel counts per layer.
 *   - Appendix A.4: cache hit ratio = || SN ∩ G ||_2 / || SN ||_2 on those vectors.
 *
 * Parity with outputs printed by the paper: unpinned (the paper prints no inference outputs and
 * its trained weights are not available).  Everything else is pinned by the CPU tests against
 * brute force, library convolutions and the nesting invariants of Section 2.1.
 *
 * Layout: activations NHWC float.  Stored weights [K][C][R][S] float as in the blob.  For speed
 * the sliced path also keeps a transposed copy [R][S][C][K] so that the innermost loop runs over
 * output filters; every output element still sums its terms in (r, s, c) order, exactly as the
 * definition is written.
 */
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#define ORC_MAX_STAGES 8
#define ORC_MAX_BLOCKS 8
#define ORC_MAX_LAYERS 256
#define ORC_BN_EPS 1e-5f

enum { ORC_TINY = 0, ORC_RESNET = 1, ORC_MBV3 = 2 };
enum { ORC_CONV = 0, ORC_DW = 1, ORC_LINEAR = 2 };
enum { ACT_NONE = 0, ACT_RELU = 1, ACT_HSWISH = 2 };
enum { ORC_FP32 = 0, ORC_BF16_STORE = 1 };

typedef struct {
    int depth[ORC_MAX_STAGES];
    float width[ORC_MAX_STAGES + 1];
    float expand[ORC_MAX_STAGES][ORC_MAX_BLOCKS];
    int kernel[ORC_MAX_STAGES][ORC_MAX_BLOCKS];
} orc_cfg;

typedef struct {
    int kind, K, C, R, S, has_bn, has_bias;
    float *w;  /* [K][C][R][S] */
    float *wt; /* [R][S][C][K] */
    float *gamma, *beta, *mean, *var, *bias;
} orc_layer;

typedef struct orc_net {
    int family;
    int n_layers;
    orc_layer L[ORC_MAX_LAYERS];
    /* layer indices by role */
    int stem, fc;
    int first_dw, first_pw, head_conv, head_mix;
    int l1[ORC_MAX_STAGES][ORC_MAX_BLOCKS]; /* conv1 / expand */
    int l2[ORC_MAX_STAGES][ORC_MAX_BLOCKS]; /* conv2 / depthwise */
    int l3[ORC_MAX_STAGES][ORC_MAX_BLOCKS]; /* conv3 / project (Tiny: unused) */
    int lp[ORC_MAX_STAGES][ORC_MAX_BLOCKS]; /* projection shortcut or -1 */
    int se1[ORC_MAX_STAGES][ORC_MAX_BLOCKS], se2[ORC_MAX_STAGES][ORC_MAX_BLOCKS];
    int n_stages, max_depth[ORC_MAX_STAGES];
} orc_net;

/* ------------------------------------------------------------------------------------------ */
/* The three synthetic SuperNets (topology constants)                                          */
/* ------------------------------------------------------------------------------------------ */
static const int TINY_W[3] = {16, 32, 64};
static const int TINY_STRIDE[3] = {1, 2, 2};
static const int RES_BASE[4] = {256, 512, 1024, 2048};
static const int RES_BASE_DEPTH[4] = {2, 2, 4, 2};
static const int RES_STRIDE[4] = {1, 2, 2, 2};
static const int RES_STEM = 64;
static const int MB_OUT[5] = {24, 40, 80, 112, 160};
static const int MB_STRIDE[5] = {2, 2, 2, 1, 2};
static const int MB_ACT[5] = {ACT_RELU, ACT_RELU, ACT_HSWISH, ACT_HSWISH, ACT_HSWISH};
static const int MB_SE[5] = {0, 1, 0, 1, 1};
static const int MB_STEM = 16;

/* nearest multiple of 8 to base*permille/1000, ties up, at least 8 */
static int r8_permille(int base, int permille) {
    long v = ((long)base * permille + 4000) / 8000;
    int r = (int)(8 * v);
    return r < 8 ? 8 : r;
}
/* SE squeeze width: nearest multiple of 8 to mid/4, at least 8 */
static int se_squeeze(int mid) {
    int r = 8 * ((mid + 16) / 32);
    return r < 8 ? 8 : r;
}
static int permille(float f) { return (int)lroundf(f * 1000.0f); }

static float bf16_round(float x) {
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) return x; /* inf / nan unchanged */
    u = (u + 0x7fffu + ((u >> 16) & 1u)) & 0xffff0000u;
    memcpy(&x, &u, 4);
    return x;
}
static void store_round(float *x, size_t n, int mode) {
    if (mode != ORC_BF16_STORE) return;
    for (size_t i = 0; i < n; i++) x[i] = bf16_round(x[i]);
}
static float act_apply(float v, int act) {
    if (act == ACT_RELU) return v > 0.f ? v : 0.f;
    if (act == ACT_HSWISH) {
        float t = v + 3.f;
        t = t < 0.f ? 0.f : (t > 6.f ? 6.f : t);
        return v * t / 6.f;
    }
    return v;
}
static float hsigmoid(float v) {
    float t = v + 3.f;
    t = t < 0.f ? 0.f : (t > 6.f ? 6.f : t);
    return t / 6.f;
}

/* ------------------------------------------------------------------------------------------ */
/* Loading                                                                                      */
/* ------------------------------------------------------------------------------------------ */
static int seterr(char *err, int errlen, const char *msg) {
    if (err && errlen > 0) snprintf(err, (size_t)errlen, "%s", msg);
    return -1;
}

typedef struct {
    const uint32_t *p;
    size_t left; /* words */
} rd_t;

static int expect_layer(orc_net *net, rd_t *rd, int kind, int K, int C, int R, int S, int bn, int bias) {
    if (net->n_layers >= ORC_MAX_LAYERS || rd->left < 8) return -1;
    const uint32_t *h = rd->p;
    if ((int)h[0] != kind || (int)h[1] != K || (int)h[2] != C || (int)h[3] != R || (int)h[4] != S ||
        (int)h[5] != bn || (int)h[6] != bias)
        return -1;
    size_t nw = (size_t)K * C * R * S, need = nw + (bn ? 4u * K : 0u) + (bias ? (size_t)K : 0u);
    if (rd->left < 8 + need) return -1;
    orc_layer *L = &net->L[net->n_layers];
    memset(L, 0, sizeof(*L));
    L->kind = kind; L->K = K; L->C = C; L->R = R; L->S = S; L->has_bn = bn; L->has_bias = bias;
    float *own = (float *)malloc(need * sizeof(float));
    if (!own) return -1;
    memcpy(own, h + 8, need * sizeof(float));
    L->w = own;
    float *q = own + nw;
    if (bn) { L->gamma = q; L->beta = q + K; L->mean = q + 2 * K; L->var = q + 3 * K; q += 4 * K; }
    if (bias) { L->bias = q; }
    L->wt = (float *)malloc(nw * sizeof(float));
    if (!L->wt) return -1;
    for (int k = 0; k < K; k++)
        for (int c = 0; c < C; c++)
            for (int r = 0; r < R; r++)
                for (int s = 0; s < S; s++)
                    L->wt[(((size_t)r * S + s) * C + c) * K + k] = L->w[(((size_t)k * C + c) * R + r) * S + s];
    rd->p += 8 + need;
    rd->left -= 8 + need;
    return net->n_layers++;
}

void orc_free(orc_net *net) {
    if (!net) return;
    for (int i = 0; i < net->n_layers; i++) { free(net->L[i].w); free(net->L[i].wt); }
    free(net);
}

#define EXPECT(dst, ...) do { int id_ = expect_layer(net, &rd, __VA_ARGS__); \
    if (id_ < 0) { orc_free(net); seterr(err, errlen, "blob does not match the architecture"); return NULL; } \
    dst = id_; } while (0)

orc_net *orc_load(int family, const void *blob, size_t nbytes, char *err, int errlen) {
    if (!blob || nbytes < 32 || nbytes % 4) { seterr(err, errlen, "bad blob size"); return NULL; }
    const uint32_t *hdr = (const uint32_t *)blob;
    if (hdr[0] != 0x42534753u || hdr[1] != 1u || (int)hdr[2] != family) {
        seterr(err, errlen, "bad blob header"); return NULL;
    }
    orc_net *net = (orc_net *)calloc(1, sizeof(orc_net));
    if (!net) { seterr(err, errlen, "out of memory"); return NULL; }
    net->family = family;
    rd_t rd = {hdr + 8, nbytes / 4 - 8};
    memset(net->lp, -1, sizeof(net->lp));
    memset(net->se1, -1, sizeof(net->se1));
    memset(net->se2, -1, sizeof(net->se2));
    if (family == ORC_TINY) {
        net->n_stages = 3;
        EXPECT(net->stem, ORC_CONV, TINY_W[0], 3, 3, 3, 1, 0);
        int prev = TINY_W[0];
        for (int s = 0; s < 3; s++) {
            net->max_depth[s] = 3;
            for (int b = 0; b < 3; b++) {
                int cin = b == 0 ? prev : TINY_W[s];
                EXPECT(net->l1[s][b], ORC_CONV, TINY_W[s], cin, 3, 3, 1, 0);
                EXPECT(net->l2[s][b], ORC_CONV, TINY_W[s], TINY_W[s], 3, 3, 1, 0);
                if (b == 0 && s > 0) EXPECT(net->lp[s][b], ORC_CONV, TINY_W[s], cin, 1, 1, 1, 0);
            }
            prev = TINY_W[s];
        }
        EXPECT(net->fc, ORC_LINEAR, 10, TINY_W[2], 1, 1, 0, 1);
    } else if (family == ORC_RESNET) {
        net->n_stages = 4;
        EXPECT(net->stem, ORC_CONV, RES_STEM, 3, 7, 7, 1, 0);
        int prev = RES_STEM;
        for (int s = 0; s < 4; s++) {
            int mid = r8_permille(RES_BASE[s], 350);
            net->max_depth[s] = RES_BASE_DEPTH[s] + 2;
            for (int b = 0; b < net->max_depth[s]; b++) {
                int cin = b == 0 ? prev : RES_BASE[s];
                EXPECT(net->l1[s][b], ORC_CONV, mid, cin, 1, 1, 1, 0);
                EXPECT(net->l2[s][b], ORC_CONV, mid, mid, 3, 3, 1, 0);
                EXPECT(net->l3[s][b], ORC_CONV, RES_BASE[s], mid, 1, 1, 1, 0);
                if (b == 0) EXPECT(net->lp[s][b], ORC_CONV, RES_BASE[s], cin, 1, 1, 1, 0);
            }
            prev = RES_BASE[s];
        }
        EXPECT(net->fc, ORC_LINEAR, 1000, RES_BASE[3], 1, 1, 0, 1);
    } else if (family == ORC_MBV3) {
        net->n_stages = 5;
        EXPECT(net->stem, ORC_CONV, MB_STEM, 3, 3, 3, 1, 0);
        EXPECT(net->first_dw, ORC_DW, MB_STEM, 1, 3, 3, 1, 0);
        EXPECT(net->first_pw, ORC_CONV, MB_STEM, MB_STEM, 1, 1, 1, 0);
        int prev = MB_STEM;
        for (int s = 0; s < 5; s++) {
            net->max_depth[s] = 4;
            for (int b = 0; b < 4; b++) {
                int cin = b == 0 ? prev : MB_OUT[s];
                int mid = cin * 6;
                EXPECT(net->l1[s][b], ORC_CONV, mid, cin, 1, 1, 1, 0);
                EXPECT(net->l2[s][b], ORC_DW, mid, 1, 7, 7, 1, 0);
                if (MB_SE[s]) {
                    int sq = se_squeeze(mid);
                    EXPECT(net->se1[s][b], ORC_LINEAR, sq, mid, 1, 1, 0, 1);
                    EXPECT(net->se2[s][b], ORC_LINEAR, mid, sq, 1, 1, 0, 1);
                }
                EXPECT(net->l3[s][b], ORC_CONV, MB_OUT[s], mid, 1, 1, 1, 0);
            }
            prev = MB_OUT[s];
        }
        EXPECT(net->head_conv, ORC_CONV, 960, MB_OUT[4], 1, 1, 1, 0);
        EXPECT(net->head_mix, ORC_LINEAR, 1280, 960, 1, 1, 0, 1);
        EXPECT(net->fc, ORC_LINEAR, 1000, 1280, 1, 1, 0, 1);
    } else {
        orc_free(net); seterr(err, errlen, "unknown family"); return NULL;
    }
    if (rd.left != 0 || (int)hdr[3] != net->n_layers) {
        orc_free(net); seterr(err, errlen, "blob has trailing or missing records"); return NULL;
    }
    return net;
}

int orc_num_layers(const orc_net *net) { return net->n_layers; }

/* ------------------------------------------------------------------------------------------ */
/* Config validation and the per-layer slice (K', C', k) of a SubNet                            */
/* ------------------------------------------------------------------------------------------ */
typedef struct { int active, K, C, k; } orc_slice;

static int in_set_i(int v, const int *set, int n) { for (int i = 0; i < n; i++) if (set[i] == v) return 1; return 0; }

int orc_validate(const orc_net *net, const orc_cfg *cfg) {
    static const int tw[3] = {500, 750, 1000}, td[3] = {1, 2, 3};
    static const int rw[3] = {650, 800, 1000}, re[3] = {200, 250, 350};
    static const int me[3] = {3000, 4000, 6000}, mk[3] = {3, 5, 7}, md[3] = {2, 3, 4};
    if (net->family == ORC_TINY) {
        for (int s = 0; s < 3; s++) {
            if (!in_set_i(cfg->depth[s], td, 3)) return -1;
            if (!in_set_i(permille(cfg->width[s + 1]), tw, 3)) return -1;
        }
    } else if (net->family == ORC_RESNET) {
        if (!in_set_i(permille(cfg->width[0]), rw, 3)) return -1;
        for (int s = 0; s < 4; s++) {
            int extra = cfg->depth[s] - RES_BASE_DEPTH[s];
            if (extra < 0 || extra > 2) return -1;
            if (!in_set_i(permille(cfg->width[s + 1]), rw, 3)) return -1;
            for (int b = 0; b < cfg->depth[s]; b++)
                if (!in_set_i(permille(cfg->expand[s][b]), re, 3)) return -1;
        }
    } else {
        for (int s = 0; s < 5; s++) {
            if (!in_set_i(cfg->depth[s], md, 3)) return -1;
            for (int b = 0; b < cfg->depth[s]; b++) {
                if (!in_set_i(permille(cfg->expand[s][b]), me, 3)) return -1;
                if (!in_set_i(cfg->kernel[s][b], mk, 3)) return -1;
            }
        }
    }
    return 0;
}

/* Fill sl[layer] for every stored layer: which prefix of filters / channels and which kernel
 * window the SubNet uses (Section 2.1), or active = 0 when the block is beyond the stage depth. */
static void slices_of(const orc_net *net, const orc_cfg *cfg, orc_slice *sl) {
    for (int i = 0; i < net->n_layers; i++) { sl[i].active = 0; sl[i].K = sl[i].C = sl[i].k = 0; }
#define SET(id, Kp, Cp, kk) do { sl[id].active = 1; sl[id].K = (Kp); sl[id].C = (Cp); sl[id].k = (kk); } while (0)
    if (net->family == ORC_TINY) {
        int w[3];
        for (int s = 0; s < 3; s++) w[s] = TINY_W[s] * permille(cfg->width[s + 1]) / 1000;
        SET(net->stem, w[0], 3, 3);
        int prev = w[0];
        for (int s = 0; s < 3; s++) {
            for (int b = 0; b < cfg->depth[s]; b++) {
                int cin = b == 0 ? prev : w[s];
                SET(net->l1[s][b], w[s], cin, 3);
                SET(net->l2[s][b], w[s], w[s], 3);
                if (net->lp[s][b] >= 0) SET(net->lp[s][b], w[s], cin, 1);
            }
            prev = w[s];
        }
        SET(net->fc, 10, w[2], 1);
    } else if (net->family == ORC_RESNET) {
        int stem = r8_permille(RES_STEM, permille(cfg->width[0]));
        SET(net->stem, stem, 3, 7);
        int prev = stem;
        for (int s = 0; s < 4; s++) {
            int out = r8_permille(RES_BASE[s], permille(cfg->width[s + 1]));
            for (int b = 0; b < cfg->depth[s]; b++) {
                int cin = b == 0 ? prev : out;
                int mid = r8_permille(out, permille(cfg->expand[s][b]));
                SET(net->l1[s][b], mid, cin, 1);
                SET(net->l2[s][b], mid, mid, 3);
                SET(net->l3[s][b], out, mid, 1);
                if (b == 0) SET(net->lp[s][b], out, cin, 1);
            }
            prev = out;
        }
        SET(net->fc, 1000, prev, 1);
    } else {
        SET(net->stem, MB_STEM, 3, 3);
        SET(net->first_dw, MB_STEM, 1, 3);
        SET(net->first_pw, MB_STEM, MB_STEM, 1);
        int prev = MB_STEM;
        for (int s = 0; s < 5; s++) {
            for (int b = 0; b < cfg->depth[s]; b++) {
                int cin = b == 0 ? prev : MB_OUT[s];
                int mid = r8_permille(cin, permille(cfg->expand[s][b]));
                SET(net->l1[s][b], mid, cin, 1);
                SET(net->l2[s][b], mid, 1, cfg->kernel[s][b]);
                if (MB_SE[s]) {
                    int sq = se_squeeze(mid);
                    SET(net->se1[s][b], sq, mid, 1);
                    SET(net->se2[s][b], mid, sq, 1);
                }
                SET(net->l3[s][b], MB_OUT[s], mid, 1);
            }
            prev = MB_OUT[s];
        }
        SET(net->head_conv, 960, MB_OUT[4], 1);
        SET(net->head_mix, 1280, 960, 1);
        SET(net->fc, 1000, 1280, 1);
    }
#undef SET
}

/* Vector encoding of Section 3.3 extended by the kernel size: out[3*i..] = K_i, C_i, k_i
 * (all zero for a layer the SubNet does not use).  Returns the number of stored layers. */
int orc_encode(const orc_net *net, const orc_cfg *cfg, int *out) {
    orc_slice sl[ORC_MAX_LAYERS];
    if (orc_validate(net, cfg)) return -1;
    slices_of(net, cfg, sl);
    for (int i = 0; i < net->n_layers; i++) { out[3 * i] = sl[i].K; out[3 * i + 1] = sl[i].C; out[3 * i + 2] = sl[i].k; }
    return net->n_layers;
}

/* Number of stored weight elements a (K, C, k) encoding selects, summed over layers. */
long long orc_encoding_weights(const int *enc, int n_layers) {
    long long t = 0;
    for (int i = 0; i < n_layers; i++) t += (long long)enc[3 * i] * enc[3 * i + 1] * enc[3 * i + 2] * enc[3 * i + 2];
    return t;
}

/* Intersection of two nets given as encodings: slices are prefixes (and centred windows), so the
 * common weights of a layer are the prefix box with the smaller K, C and k (Section 2.2). */
void orc_intersect(const int *a, const int *b, int n_layers, int *out) {
    for (int i = 0; i < 3 * n_layers; i++) out[i] = a[i] < b[i] ? a[i] : b[i];
}

/* Cache hit ratio of Appendix A.4 on the (K, C) entries of two encodings. */
double orc_hit_ratio(const int *sn, const int *g, int n_layers) {
    double num = 0, den = 0;
    for (int i = 0; i < n_layers; i++)
        for (int j = 0; j < 2; j++) {
            double a = sn[3 * i + j], m = a < g[3 * i + j] ? a : g[3 * i + j];
            num += m * m;
            den += a * a;
        }
    return den > 0 ? sqrt(num) / sqrt(den) : 0.0;
}

/* ------------------------------------------------------------------------------------------ */
/* Layer arithmetic on slices of the stored tensors                                            */
/* ------------------------------------------------------------------------------------------ */

/* Sliced convolution (cross-correlation, zero padding p = (k-1)/2, centre window offset
 * o = (R-k)/2 of the stored kernel):
 *   y[n,ho,wo,f] = sum_{r<k} sum_{s<k} sum_{c<Cp} x[n, ho*st + r - p, wo*st + s - p, c] * W[f][c][o+r][o+s]
 * for f < Kp.  Ho = (H + 2p - k)/st + 1. */
void orc_conv_sliced(const orc_layer *L, const float *x, int N, int H, int W, int Cp, int Kp, int k, int st,
                     float *y) {
    const int p = (k - 1) / 2, o = (L->R - k) / 2;
    const int Ho = (H + 2 * p - k) / st + 1, Wo = (W + 2 * p - k) / st + 1;
#pragma omp parallel for collapse(2) schedule(static) if (N * Ho >= 4)
    for (int n = 0; n < N; n++)
        for (int ho = 0; ho < Ho; ho++) {
            for (int wo = 0; wo < Wo; wo++) {
                float *acc = y + (((size_t)n * Ho + ho) * Wo + wo) * Kp;
                for (int f = 0; f < Kp; f++) acc[f] = 0.f;
                for (int r = 0; r < k; r++) {
                    int hi = ho * st + r - p;
                    if (hi < 0 || hi >= H) continue;
                    for (int s = 0; s < k; s++) {
                        int wi = wo * st + s - p;
                        if (wi < 0 || wi >= W) continue;
                        const float *xp = x + (((size_t)n * H + hi) * W + wi) * Cp;
                        const float *wp = L->wt + ((size_t)(o + r) * L->S + (o + s)) * L->C * L->K;
                        for (int c = 0; c < Cp; c++) {
                            const float xv = xp[c];
                            const float *wr = wp + (size_t)c * L->K;
                            for (int f = 0; f < Kp; f++) acc[f] += xv * wr[f];
                        }
                    }
                }
            }
        }
}

/* Sliced depthwise convolution: channel f < Kp uses W[f][0][o+r][o+s]. */
void orc_dw_sliced(const orc_layer *L, const float *x, int N, int H, int W, int Kp, int k, int st, float *y) {
    const int p = (k - 1) / 2, o = (L->R - k) / 2;
    const int Ho = (H + 2 * p - k) / st + 1, Wo = (W + 2 * p - k) / st + 1;
#pragma omp parallel for collapse(2) schedule(static) if (N * Ho >= 4)
    for (int n = 0; n < N; n++)
        for (int ho = 0; ho < Ho; ho++)
            for (int wo = 0; wo < Wo; wo++) {
                float *acc = y + (((size_t)n * Ho + ho) * Wo + wo) * Kp;
                for (int f = 0; f < Kp; f++) acc[f] = 0.f;
                for (int r = 0; r < k; r++) {
                    int hi = ho * st + r - p;
                    if (hi < 0 || hi >= H) continue;
                    for (int s = 0; s < k; s++) {
                        int wi = wo * st + s - p;
                        if (wi < 0 || wi >= W) continue;
                        const float *xp = x + (((size_t)n * H + hi) * W + wi) * Kp;
                        const float *wr = L->wt + ((size_t)(o + r) * L->S + (o + s)) * L->K; /* C == 1 */
                        for (int f = 0; f < Kp; f++) acc[f] += xp[f] * wr[f];
                    }
                }
            }
}

/* Inference batch norm on the first Kp channels, then activation, optional residual, storage
 * rounding:  y = act( (y - mean)/sqrt(var + eps) * gamma + beta  [+ res] ). */
static void bn_act(const orc_layer *L, float *y, size_t npix, int Kp, int act, const float *res, int mode) {
    for (size_t i = 0; i < npix; i++)
        for (int f = 0; f < Kp; f++) {
            float v = y[i * Kp + f];
            if (L->has_bn) v = (v - L->mean[f]) / sqrtf(L->var[f] + ORC_BN_EPS) * L->gamma[f] + L->beta[f];
            if (L->has_bias) v += L->bias[f];
            if (res) v += res[i * Kp + f];
            v = act_apply(v, act);
            y[i * Kp + f] = mode == ORC_BF16_STORE ? bf16_round(v) : v;
        }
}

/* 3x3 stride-2 max pooling, padding 1 (padding never wins: only in-image taps are compared). */
static void maxpool3s2(const float *x, int N, int H, int W, int C, float *y) {
    int Ho = (H + 2 - 3) / 2 + 1, Wo = (W + 2 - 3) / 2 + 1;
    for (int n = 0; n < N; n++)
        for (int ho = 0; ho < Ho; ho++)
            for (int wo = 0; wo < Wo; wo++)
                for (int c = 0; c < C; c++) {
                    float m = -INFINITY;
                    for (int r = 0; r < 3; r++)
                        for (int s = 0; s < 3; s++) {
                            int hi = 2 * ho + r - 1, wi = 2 * wo + s - 1;
                            if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;
                            float v = x[(((size_t)n * H + hi) * W + wi) * C + c];
                            if (v > m) m = v;
                        }
                    y[(((size_t)n * Ho + ho) * Wo + wo) * C + c] = m;
                }
}

/* Global average pool: g[n][c] = mean over h, w (kept in fp32, never rounded). */
static void gap(const float *x, int N, int HW, int C, float *g) {
    for (int n = 0; n < N; n++)
        for (int c = 0; c < C; c++) {
            float s = 0.f;
            for (int i = 0; i < HW; i++) s += x[((size_t)n * HW + i) * C + c];
            g[(size_t)n * C + c] = s / (float)HW;
        }
}

/* Sliced fully connected layer: y[n][j] = sum_{c<Cp} W[j][c] v[n][c] + bias[j], j < Kp. */
static void linear_sliced(const orc_layer *L, const float *v, int N, int Cp, int Kp, float *y) {
    for (int n = 0; n < N; n++)
        for (int j = 0; j < Kp; j++) {
            float s = 0.f;
            for (int c = 0; c < Cp; c++) s += L->w[(size_t)j * L->C + c] * v[(size_t)n * Cp + c];
            y[(size_t)n * Kp + j] = s + (L->has_bias ? L->bias[j] : 0.f);
        }
}

/* Squeeze-excite gate from the pooled vector g[n][mid] (config text: SE with squeeze width sq, FCs with bias):
 * gate[n][c] = hsigmoid(FC2(relu(FC1(g[n]))))[c].  tmp holds N * sq floats. */
static void se_gate(const orc_layer *fc1, const orc_layer *fc2, const float *g, int N, int mid, int sq, float *tmp, float *gate) {
    linear_sliced(fc1, g, N, mid, sq, tmp);
    for (int i = 0; i < N * sq; i++) tmp[i] = act_apply(tmp[i], ACT_RELU);
    linear_sliced(fc2, tmp, N, sq, mid, gate);
    for (int i = 0; i < N * mid; i++) gate[i] = hsigmoid(gate[i]);
}
/* x[n][i][c] *= gate[n][c], then storage rounding. */
static void se_scale(float *x, const float *gate, int N, int HW, int C, int mode) {
    for (int n = 0; n < N; n++)
        for (int i = 0; i < HW; i++)
            for (int c = 0; c < C; c++) {
                size_t idx = ((size_t)n * HW + i) * C + c;
                x[idx] = x[idx] * gate[(size_t)n * C + c];
            }
    store_round(x, (size_t)N * HW * C, mode);
}

/* ------------------------------------------------------------------------------------------ */
/* Optional tap: copy the activation a given stored layer produced (debug aid for the tests)    */
/* ------------------------------------------------------------------------------------------ */
static int g_tap_layer = -1;
static float *g_tap_buf = NULL;
static size_t g_tap_cap = 0;
static int g_tap_dims[4];
void orc_set_tap(int layer, float *buf, size_t cap) { g_tap_layer = layer; g_tap_buf = buf; g_tap_cap = cap; g_tap_dims[0] = 0; }
void orc_get_tap_dims(int *d) { memcpy(d, g_tap_dims, sizeof(g_tap_dims)); }
static void tap(int layer, const float *y, int N, int H, int W, int C) {
    if (layer != g_tap_layer || !g_tap_buf) return;
    size_t n = (size_t)N * H * W * C;
    if (n > g_tap_cap) return;
    memcpy(g_tap_buf, y, n * sizeof(float));
    g_tap_dims[0] = N; g_tap_dims[1] = H; g_tap_dims[2] = W; g_tap_dims[3] = C;
}

/* ------------------------------------------------------------------------------------------ */
/* Sliced forward pass                                                                          */
/* ------------------------------------------------------------------------------------------ */
static size_t max_act_elems(const orc_net *net, int N, int res) {
    /* generous bound: the largest activation of any of the three nets at this resolution */
    size_t r = (size_t)res;
    if (net->family == ORC_TINY) return (size_t)N * r * r * 64;
    if (net->family == ORC_RESNET) return (size_t)N * (r / 2) * (r / 2) * 64 * 4 + 1024;
    return (size_t)N * (r / 2) * (r / 2) * 16 * 6 + 1024;
}

static int conv_bn(const orc_net *net, int id, const orc_slice *sl, const float *x, int N, int H, int W, int st,
                   int act, const float *res, int mode, float *y, int *Ho, int *Wo) {
    const orc_layer *L = &net->L[id];
    int k = sl[id].k, p = (k - 1) / 2;
    *Ho = (H + 2 * p - k) / st + 1;
    *Wo = (W + 2 * p - k) / st + 1;
    if (L->kind == ORC_DW) orc_dw_sliced(L, x, N, H, W, sl[id].K, k, st, y);
    else orc_conv_sliced(L, x, N, H, W, sl[id].C, sl[id].K, k, st, y);
    bn_act(L, y, (size_t)N * *Ho * *Wo, sl[id].K, act, res, mode);
    tap(id, y, N, *Ho, *Wo, sl[id].K);
    return 0;
}

/* logits[batch][classes].  input NHWC [batch][res][res][3].  mode: ORC_FP32 keeps every tensor in
 * fp32; ORC_BF16_STORE rounds each stored activation tensor (every layer output, pooled map and
 * SE-scaled map) to bfloat16, the points at which the bf16 GPU path writes to memory. */
int orc_forward(const orc_net *net, const orc_cfg *cfg, const float *input, int N, int res, int mode,
                float *logits) {
    if (orc_validate(net, cfg)) return -1;
    orc_slice sl[ORC_MAX_LAYERS];
    slices_of(net, cfg, sl);
    size_t cap = max_act_elems(net, N, res);
    float *A = (float *)malloc(cap * sizeof(float)), *B = (float *)malloc(cap * sizeof(float));
    float *Cb = (float *)malloc(cap * sizeof(float)), *D = (float *)malloc(cap * sizeof(float));
    float *vec = (float *)malloc((size_t)N * 4096 * sizeof(float)), *vec2 = (float *)malloc((size_t)N * 4096 * sizeof(float));
    float *vec3 = (float *)malloc((size_t)N * 4096 * sizeof(float));
    if (!A || !B || !Cb || !D || !vec || !vec2 || !vec3) { free(A); free(B); free(Cb); free(D); free(vec); free(vec2); free(vec3); return -2; }
    int H = res, W = res, Ho, Wo;
    float *x = A, *t1 = B, *t2 = Cb, *sc = D, *tmp;
    int C;

    if (net->family == ORC_TINY) {
        conv_bn(net, net->stem, sl, input, N, H, W, 1, ACT_RELU, NULL, mode, x, &Ho, &Wo);
        C = sl[net->stem].K;
        for (int s = 0; s < 3; s++)
            for (int b = 0; b < cfg->depth[s]; b++) {
                int st = b == 0 ? TINY_STRIDE[s] : 1, H1, W1, H2, W2;
                const float *shortcut = x;
                if (net->lp[s][b] >= 0) {
                    conv_bn(net, net->lp[s][b], sl, x, N, H, W, st, ACT_NONE, NULL, mode, sc, &H1, &W1);
                    shortcut = sc;
                }
                conv_bn(net, net->l1[s][b], sl, x, N, H, W, st, ACT_RELU, NULL, mode, t1, &H1, &W1);
                conv_bn(net, net->l2[s][b], sl, t1, N, H1, W1, 1, ACT_RELU, shortcut, mode, t2, &H2, &W2);
                tmp = x; x = t2; t2 = tmp;
                H = H2; W = W2; C = sl[net->l2[s][b]].K;
            }
        gap(x, N, H * W, C, vec);
        linear_sliced(&net->L[net->fc], vec, N, C, 10, logits);
    } else if (net->family == ORC_RESNET) {
        conv_bn(net, net->stem, sl, input, N, H, W, 2, ACT_RELU, NULL, mode, t1, &Ho, &Wo);
        C = sl[net->stem].K;
        maxpool3s2(t1, N, Ho, Wo, C, x);
        H = (Ho + 2 - 3) / 2 + 1; W = (Wo + 2 - 3) / 2 + 1;
        store_round(x, (size_t)N * H * W * C, mode);
        for (int s = 0; s < 4; s++)
            for (int b = 0; b < cfg->depth[s]; b++) {
                int st = b == 0 ? RES_STRIDE[s] : 1, H1, W1, H2, W2, H3, W3;
                const float *shortcut = x;
                if (b == 0) {
                    conv_bn(net, net->lp[s][b], sl, x, N, H, W, st, ACT_NONE, NULL, mode, sc, &H1, &W1);
                    shortcut = sc;
                }
                conv_bn(net, net->l1[s][b], sl, x, N, H, W, 1, ACT_RELU, NULL, mode, t1, &H1, &W1);
                conv_bn(net, net->l2[s][b], sl, t1, N, H1, W1, st, ACT_RELU, NULL, mode, t2, &H2, &W2);
                conv_bn(net, net->l3[s][b], sl, t2, N, H2, W2, 1, ACT_RELU, shortcut, mode, t1, &H3, &W3);
                tmp = x; x = t1; t1 = tmp;
                H = H3; W = W3; C = sl[net->l3[s][b]].K;
            }
        gap(x, N, H * W, C, vec);
        linear_sliced(&net->L[net->fc], vec, N, C, 1000, logits);
    } else {
        conv_bn(net, net->stem, sl, input, N, H, W, 2, ACT_HSWISH, NULL, mode, x, &Ho, &Wo);
        H = Ho; W = Wo; C = MB_STEM;
        conv_bn(net, net->first_dw, sl, x, N, H, W, 1, ACT_RELU, NULL, mode, t1, &Ho, &Wo);
        conv_bn(net, net->first_pw, sl, t1, N, H, W, 1, ACT_NONE, x, mode, t2, &Ho, &Wo);
        tmp = x; x = t2; t2 = tmp;
        for (int s = 0; s < 5; s++)
            for (int b = 0; b < cfg->depth[s]; b++) {
                int st = b == 0 ? MB_STRIDE[s] : 1, H1, W1, H2, W2, H3, W3;
                int mid = sl[net->l1[s][b]].K, out = MB_OUT[s];
                conv_bn(net, net->l1[s][b], sl, x, N, H, W, 1, MB_ACT[s], NULL, mode, t1, &H1, &W1);
                conv_bn(net, net->l2[s][b], sl, t1, N, H1, W1, st, MB_ACT[s], NULL, mode, t2, &H2, &W2);
                if (MB_SE[s]) {
                    /* squeeze-excite: gate[c] = hsigmoid(FC2(relu(FC1(mean_hw t2)))), t2 *= gate */
                    int sq = sl[net->se1[s][b]].K;
                    gap(t2, N, H2 * W2, mid, vec);
                    se_gate(&net->L[net->se1[s][b]], &net->L[net->se2[s][b]], vec, N, mid, sq, vec2, vec3);
                    se_scale(t2, vec3, N, H2 * W2, mid, mode);
                    tap(net->se2[s][b], t2, N, H2, W2, mid);
                }
                const float *resid = (st == 1 && C == out) ? x : NULL;
                conv_bn(net, net->l3[s][b], sl, t2, N, H2, W2, 1, ACT_NONE, resid, mode, t1, &H3, &W3);
                tmp = x; x = t1; t1 = tmp;
                H = H3; W = W3; C = out;
            }
        conv_bn(net, net->head_conv, sl, x, N, H, W, 1, ACT_HSWISH, NULL, mode, t1, &Ho, &Wo);
        gap(t1, N, H * W, 960, vec);
        linear_sliced(&net->L[net->head_mix], vec, N, 960, 1280, vec2);
        for (int i = 0; i < N * 1280; i++) vec2[i] = act_apply(vec2[i], ACT_HSWISH);
        linear_sliced(&net->L[net->fc], vec2, N, 1280, 1000, logits);
    }
    free(A); free(B); free(Cb); free(D); free(vec); free(vec2); free(vec3);
    return 0;
}

/* ------------------------------------------------------------------------------------------ */
/* Second, separate path: standalone dense nets.                                                */
/* A dense net owns exact-size tensors [K][C][k][k] and is run by loops that know nothing about  */
/* slicing.  orc_forward_extracted builds it by copying the SubNet's slices out of the SuperNet; */
/* orc_forward_unsliced builds it from the whole stored tensors (the largest SubNet).           */
/* ------------------------------------------------------------------------------------------ */
typedef struct {
    int present, kind, K, C, k;
    float *w; /* [K][C][k][k] */
    float *gamma, *beta, *mean, *var, *bias;
    int has_bn, has_bias;
} dense_layer;

static void dense_free(dense_layer *d, int n) {
    for (int i = 0; i < n; i++) { free(d[i].w); free(d[i].gamma); free(d[i].beta); free(d[i].mean); free(d[i].var); free(d[i].bias); }
}
static float *dup_prefix(const float *src, int n) {
    float *p = (float *)malloc((size_t)n * sizeof(float));
    memcpy(p, src, (size_t)n * sizeof(float));
    return p;
}
/* copy filters < Kp, channels < Cp and the centred k x k window */
static void extract_layer(const orc_layer *L, int Kp, int Cp, int k, dense_layer *d) {
    memset(d, 0, sizeof(*d));
    d->present = 1; d->kind = L->kind; d->K = Kp; d->C = Cp; d->k = k;
    d->has_bn = L->has_bn; d->has_bias = L->has_bias;
    int o = (L->R - k) / 2;
    d->w = (float *)malloc((size_t)Kp * Cp * k * k * sizeof(float));
    for (int f = 0; f < Kp; f++)
        for (int c = 0; c < Cp; c++)
            for (int r = 0; r < k; r++)
                for (int s = 0; s < k; s++)
                    d->w[(((size_t)f * Cp + c) * k + r) * k + s] = L->w[(((size_t)f * L->C + c) * L->R + o + r) * L->S + o + s];
    if (L->has_bn) { d->gamma = dup_prefix(L->gamma, Kp); d->beta = dup_prefix(L->beta, Kp); d->mean = dup_prefix(L->mean, Kp); d->var = dup_prefix(L->var, Kp); }
    if (L->has_bias) d->bias = dup_prefix(L->bias, Kp);
}

/* dense conv + BN + residual + act on a standalone layer; naive [K][C][k][k] indexing */
static void dense_conv(const dense_layer *d, const float *x, int N, int H, int W, int st, int act, const float *res,
                       int mode, float *y, int *Ho_, int *Wo_) {
    int k = d->k, p = (k - 1) / 2, Ho = (H + 2 * p - k) / st + 1, Wo = (W + 2 * p - k) / st + 1;
    *Ho_ = Ho; *Wo_ = Wo;
#pragma omp parallel for collapse(2) schedule(static) if (N * Ho >= 4)
    for (int n = 0; n < N; n++)
        for (int ho = 0; ho < Ho; ho++)
            for (int wo = 0; wo < Wo; wo++)
                for (int f = 0; f < d->K; f++) {
                    float acc = 0.f;
                    for (int r = 0; r < k; r++)
                        for (int s = 0; s < k; s++) {
                            int hi = ho * st + r - p, wi = wo * st + s - p;
                            if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;
                            if (d->kind == ORC_DW) {
                                acc += x[(((size_t)n * H + hi) * W + wi) * d->K + f] * d->w[((size_t)f * k + r) * k + s];
                            } else {
                                for (int c = 0; c < d->C; c++)
                                    acc += x[(((size_t)n * H + hi) * W + wi) * d->C + c] * d->w[(((size_t)f * d->C + c) * k + r) * k + s];
                            }
                        }
                    float v = acc;
                    if (d->has_bn) v = (v - d->mean[f]) / sqrtf(d->var[f] + ORC_BN_EPS) * d->gamma[f] + d->beta[f];
                    if (d->has_bias) v += d->bias[f];
                    size_t oi = (((size_t)n * Ho + ho) * Wo + wo) * d->K + f;
                    if (res) v += res[oi];
                    v = act_apply(v, act);
                    y[oi] = mode == ORC_BF16_STORE ? bf16_round(v) : v;
                }
}
static void dense_linear(const dense_layer *d, const float *v, int N, float *y) {
    for (int n = 0; n < N; n++)
        for (int j = 0; j < d->K; j++) {
            float s = 0.f;
            for (int c = 0; c < d->C; c++) s += d->w[(size_t)j * d->C + c] * v[(size_t)n * d->C + c];
            y[(size_t)n * d->K + j] = s + (d->has_bias ? d->bias[j] : 0.f);
        }
}

/* Runs a dense net.  Widths come from the dense layers themselves; only the depth per stage (how
 * many blocks are present) is read from the layer table. */
static int dense_forward(const orc_net *net, const dense_layer *d, const int *depth, const float *input, int N,
                         int res, int mode, float *logits) {
    size_t cap = max_act_elems(net, N, res);
    float *A = (float *)malloc(cap * sizeof(float)), *B = (float *)malloc(cap * sizeof(float));
    float *Cb = (float *)malloc(cap * sizeof(float)), *D = (float *)malloc(cap * sizeof(float));
    float *vec = (float *)malloc((size_t)N * 4096 * sizeof(float)), *vec2 = (float *)malloc((size_t)N * 4096 * sizeof(float));
    if (!A || !B || !Cb || !D || !vec || !vec2) { free(A); free(B); free(Cb); free(D); free(vec); free(vec2); return -2; }
    float *x = A, *t1 = B, *t2 = Cb, *sc = D, *tmp;
    int H = res, W = res, C, Ho, Wo;
    if (net->family == ORC_TINY) {
        dense_conv(&d[net->stem], input, N, H, W, 1, ACT_RELU, NULL, mode, x, &Ho, &Wo);
        C = d[net->stem].K;
        for (int s = 0; s < 3; s++)
            for (int b = 0; b < depth[s]; b++) {
                int st = b == 0 ? TINY_STRIDE[s] : 1, H1, W1, H2, W2;
                const float *shortcut = x;
                if (net->lp[s][b] >= 0) { dense_conv(&d[net->lp[s][b]], x, N, H, W, st, ACT_NONE, NULL, mode, sc, &H1, &W1); shortcut = sc; }
                dense_conv(&d[net->l1[s][b]], x, N, H, W, st, ACT_RELU, NULL, mode, t1, &H1, &W1);
                dense_conv(&d[net->l2[s][b]], t1, N, H1, W1, 1, ACT_RELU, shortcut, mode, t2, &H2, &W2);
                tmp = x; x = t2; t2 = tmp; H = H2; W = W2; C = d[net->l2[s][b]].K;
            }
        gap(x, N, H * W, C, vec);
        dense_linear(&d[net->fc], vec, N, logits);
    } else if (net->family == ORC_RESNET) {
        dense_conv(&d[net->stem], input, N, H, W, 2, ACT_RELU, NULL, mode, t1, &Ho, &Wo);
        C = d[net->stem].K;
        maxpool3s2(t1, N, Ho, Wo, C, x);
        H = (Ho + 2 - 3) / 2 + 1; W = (Wo + 2 - 3) / 2 + 1;
        store_round(x, (size_t)N * H * W * C, mode);
        for (int s = 0; s < 4; s++)
            for (int b = 0; b < depth[s]; b++) {
                int st = b == 0 ? RES_STRIDE[s] : 1, H1, W1, H2, W2, H3, W3;
                const float *shortcut = x;
                if (b == 0) { dense_conv(&d[net->lp[s][b]], x, N, H, W, st, ACT_NONE, NULL, mode, sc, &H1, &W1); shortcut = sc; }
                dense_conv(&d[net->l1[s][b]], x, N, H, W, 1, ACT_RELU, NULL, mode, t1, &H1, &W1);
                dense_conv(&d[net->l2[s][b]], t1, N, H1, W1, st, ACT_RELU, NULL, mode, t2, &H2, &W2);
                dense_conv(&d[net->l3[s][b]], t2, N, H2, W2, 1, ACT_RELU, shortcut, mode, t1, &H3, &W3);
                tmp = x; x = t1; t1 = tmp; H = H3; W = W3; C = d[net->l3[s][b]].K;
            }
        gap(x, N, H * W, C, vec);
        dense_linear(&d[net->fc], vec, N, logits);
    } else {
        dense_conv(&d[net->stem], input, N, H, W, 2, ACT_HSWISH, NULL, mode, x, &Ho, &Wo);
        H = Ho; W = Wo; C = d[net->stem].K;
        dense_conv(&d[net->first_dw], x, N, H, W, 1, ACT_RELU, NULL, mode, t1, &Ho, &Wo);
        dense_conv(&d[net->first_pw], t1, N, H, W, 1, ACT_NONE, x, mode, t2, &Ho, &Wo);
        tmp = x; x = t2; t2 = tmp;
        for (int s = 0; s < 5; s++)
            for (int b = 0; b < depth[s]; b++) {
                int st = b == 0 ? MB_STRIDE[s] : 1, H1, W1, H2, W2, H3, W3;
                const dense_layer *ex = &d[net->l1[s][b]], *pr = &d[net->l3[s][b]];
                int mid = ex->K;
                dense_conv(ex, x, N, H, W, 1, MB_ACT[s], NULL, mode, t1, &H1, &W1);
                dense_conv(&d[net->l2[s][b]], t1, N, H1, W1, st, MB_ACT[s], NULL, mode, t2, &H2, &W2);
                if (MB_SE[s]) {
                    const dense_layer *f1 = &d[net->se1[s][b]], *f2 = &d[net->se2[s][b]];
                    gap(t2, N, H2 * W2, mid, vec);
                    dense_linear(f1, vec, N, vec2);
                    for (int i = 0; i < N * f1->K; i++) vec2[i] = act_apply(vec2[i], ACT_RELU);
                    dense_linear(f2, vec2, N, vec);
                    for (int n = 0; n < N; n++)
                        for (int i = 0; i < H2 * W2; i++)
                            for (int c = 0; c < mid; c++) {
                                size_t idx = ((size_t)n * H2 * W2 + i) * mid + c;
                                t2[idx] = t2[idx] * hsigmoid(vec[(size_t)n * mid + c]);
                            }
                    store_round(t2, (size_t)N * H2 * W2 * mid, mode);
                }
                const float *resid = (st == 1 && ex->C == pr->K) ? x : NULL;
                dense_conv(pr, t2, N, H2, W2, 1, ACT_NONE, resid, mode, t1, &H3, &W3);
                tmp = x; x = t1; t1 = tmp; H = H3; W = W3; C = pr->K;
            }
        dense_conv(&d[net->head_conv], x, N, H, W, 1, ACT_HSWISH, NULL, mode, t1, &Ho, &Wo);
        gap(t1, N, H * W, d[net->head_conv].K, vec);
        dense_linear(&d[net->head_mix], vec, N, vec2);
        for (int i = 0; i < N * d[net->head_mix].K; i++) vec2[i] = act_apply(vec2[i], ACT_HSWISH);
        dense_linear(&d[net->fc], vec2, N, logits);
    }
    (void)C;
    free(A); free(B); free(Cb); free(D); free(vec); free(vec2);
    return 0;
}

/* SubNet = standalone net built from explicitly copied slices, then run densely. */
int orc_forward_extracted(const orc_net *net, const orc_cfg *cfg, const float *input, int N, int res, int mode,
                          float *logits) {
    if (orc_validate(net, cfg)) return -1;
    orc_slice sl[ORC_MAX_LAYERS];
    slices_of(net, cfg, sl);
    dense_layer *d = (dense_layer *)calloc((size_t)net->n_layers, sizeof(dense_layer));
    for (int i = 0; i < net->n_layers; i++)
        if (sl[i].active) extract_layer(&net->L[i], sl[i].K, sl[i].C, sl[i].k, &d[i]);
    int rc = dense_forward(net, d, cfg->depth, input, N, res, mode, logits);
    dense_free(d, net->n_layers);
    free(d);
    return rc;
}

/* The whole SuperNet run on its full stored tensors, no config involved. */
int orc_forward_unsliced(const orc_net *net, const float *input, int N, int res, int mode, float *logits) {
    dense_layer *d = (dense_layer *)calloc((size_t)net->n_layers, sizeof(dense_layer));
    for (int i = 0; i < net->n_layers; i++) {
        const orc_layer *L = &net->L[i];
        extract_layer(L, L->K, L->C, L->R, &d[i]);
    }
    int rc = dense_forward(net, d, net->max_depth, input, N, res, mode, logits);
    dense_free(d, net->n_layers);
    free(d);
    return rc;
}

/* ------------------------------------------------------------------------------------------ */
/* Single-layer entry points for the tests (raw tensors in, no net needed)                      */
/* ------------------------------------------------------------------------------------------ */

/* Sliced conv on a raw stored tensor w[Kmax][Cmax][R][R]; depthwise when dw != 0 (Cmax == 1). */
int orc_layer_conv(const float *w, int Kmax, int Cmax, int R, int dw, const float *x, int N, int H, int W, int Cp,
                   int Kp, int k, int st, float *y) {
    orc_layer L;
    memset(&L, 0, sizeof(L));
    L.kind = dw ? ORC_DW : ORC_CONV; L.K = Kmax; L.C = Cmax; L.R = R; L.S = R;
    L.w = (float *)w;
    size_t nw = (size_t)Kmax * Cmax * R * R;
    L.wt = (float *)malloc(nw * sizeof(float));
    if (!L.wt) return -2;
    for (int f = 0; f < Kmax; f++)
        for (int c = 0; c < Cmax; c++)
            for (int r = 0; r < R; r++)
                for (int s = 0; s < R; s++)
                    L.wt[(((size_t)r * R + s) * Cmax + c) * Kmax + f] = w[(((size_t)f * Cmax + c) * R + r) * R + s];
    if (dw) orc_dw_sliced(&L, x, N, H, W, Kp, k, st, y);
    else orc_conv_sliced(&L, x, N, H, W, Cp, Kp, k, st, y);
    free(L.wt);
    return 0;
}

/* y = act(bn(y) + res) with storage rounding, on raw parameter vectors (any may be NULL). */
void orc_layer_epilogue(float *y, size_t npix, int Kp, const float *gamma, const float *beta, const float *mean,
                        const float *var, const float *bias, const float *res, int act, int mode) {
    orc_layer L;
    memset(&L, 0, sizeof(L));
    L.has_bn = gamma != NULL; L.has_bias = bias != NULL;
    L.gamma = (float *)gamma; L.beta = (float *)beta; L.mean = (float *)mean; L.var = (float *)var; L.bias = (float *)bias;
    bn_act(&L, y, npix, Kp, act, res, mode);
}

void orc_layer_maxpool(const float *x, int N, int H, int W, int C, float *y) { maxpool3s2(x, N, H, W, C, y); }
void orc_layer_gap(const float *x, int N, int HW, int C, float *g) { gap(x, N, HW, C, g); }

static orc_layer raw_linear(const float *w, int ld, const float *bias) {
    orc_layer L;
    memset(&L, 0, sizeof(L));
    L.kind = ORC_LINEAR; L.C = ld; L.w = (float *)w; L.has_bias = bias != NULL; L.bias = (float *)bias;
    return L;
}
/* Sliced fully connected layer on a raw stored matrix w[Kmax][ld]: y[n][j] = act(sum_{c<Cp} w[j][c] v[n][c] + bias[j]), j < Kp. */
void orc_layer_linear(const float *w, int ld, const float *bias, const float *v, int N, int Cp, int Kp, int act, float *y) {
    orc_layer L = raw_linear(w, ld, bias);
    linear_sliced(&L, v, N, Cp, Kp, y);
    for (int i = 0; i < N * Kp; i++) y[i] = act_apply(y[i], act);
}
/* Squeeze-excite gate on raw stored matrices w1[.][ld1] (first FC, sq outputs of mid inputs) and w2[.][ld2]. */
int orc_layer_se_gate(const float *w1, int ld1, const float *b1, const float *w2, int ld2, const float *b2, const float *g,
                      int N, int mid, int sq, float *gate) {
    orc_layer L1 = raw_linear(w1, ld1, b1), L2 = raw_linear(w2, ld2, b2);
    float *tmp = (float *)malloc((size_t)N * sq * sizeof(float));
    if (!tmp) return -2;
    se_gate(&L1, &L2, g, N, mid, sq, tmp, gate);
    free(tmp);
    return 0;
}
/* In place: x[n][i][c] *= gate[n][c], with the storage rounding of `mode`. */
void orc_layer_se_scale(float *x, const float *gate, int N, int HW, int C, int mode) { se_scale(x, gate, N, HW, C, mode); }
/* ------------------------------------------------------------------------------------------ */
/* 8-bit sliced convolution layer (the paper's numeric format: Section 5.1, workload footnote:   */
/* int8 weights, activations and zero points, int32 scale; Section 4.2 Zero Point/Scale Buffer). */
/* Exact integer arithmetic, direct loops.  w[Kmax][Cmax][R][R] signed bytes; x, res, y one byte */
/* per element, read as 0..255 or (signed flag) -128..127.                                       */
/*   acc = sum over in-image taps and c < Cp of (x - zx) * w      (outside the image: real 0)    */
/*   t   = rsr(acc * mult[f], 31 + shift[f]) + bias[f] + rsr((res - zr) * res_mult, 31 + res_shift) + zy */
/*   y   = saturate(relu ? max(t, zy) : t),   rsr(v, s) = floor((v + 2^(s-1)) / 2^s)             */
/* ------------------------------------------------------------------------------------------ */
static long long rsr64(long long v, int s) {
    long long q = v + ((long long)1 << (s - 1));
    /* floor division by 2^s written without relying on the shift of a negative number */
    long long d = (long long)1 << s, r = q / d;
    if (q % d != 0 && q < 0) r -= 1;
    return r;
}
static int byte_value(const unsigned char *p, size_t i, int is_signed) { return is_signed ? (int)(signed char)p[i] : (int)p[i]; }

int orc_layer_conv_i8(const signed char *w, int Kmax, int Cmax, int R, const unsigned char *x, int x_signed, int zx, int N,
                      int H, int W, int Cp, int Kp, int k, int st, const int *mult, const int *shift, const int *bias,
                      const unsigned char *res, int res_signed, int zr, int res_mult, int res_shift, int zy, int relu,
                      int y_signed, unsigned char *y) {
    const int p = (k - 1) / 2, o = (R - k) / 2;
    const int Ho = (H + 2 * p - k) / st + 1, Wo = (W + 2 * p - k) / st + 1;
    (void)Kmax;
    for (int n = 0; n < N; n++)
        for (int ho = 0; ho < Ho; ho++)
            for (int wo = 0; wo < Wo; wo++)
                for (int f = 0; f < Kp; f++) {
                    long long acc = 0;
                    for (int r = 0; r < k; r++) {
                        int hi = ho * st + r - p;
                        if (hi < 0 || hi >= H) continue;
                        for (int s = 0; s < k; s++) {
                            int wi = wo * st + s - p;
                            if (wi < 0 || wi >= W) continue;
                            for (int c = 0; c < Cp; c++) {
                                int xv = byte_value(x, (((size_t)n * H + hi) * W + wi) * Cp + c, x_signed) - zx;
                                int wv = (int)w[(((size_t)f * Cmax + c) * R + (o + r)) * R + (o + s)];
                                acc += (long long)xv * wv;
                            }
                        }
                    }
                    if (acc > 2147483647ll || acc < -2147483648ll) return -3; /* the format's accumulator is 32 bits */
                    int sh = shift[f] < 0 ? 0 : (shift[f] > 31 ? 31 : shift[f]);
                    size_t oi = (((size_t)n * Ho + ho) * Wo + wo) * Kp + f;
                    long long t = rsr64(acc * (long long)mult[f], 31 + sh) + bias[f];
                    if (res) t += rsr64((long long)(byte_value(res, oi, res_signed) - zr) * (long long)res_mult, 31 + res_shift);
                    t += zy;
                    if (relu && t < zy) t = zy;
                    long long lo = y_signed ? -128 : 0, hi2 = y_signed ? 127 : 255;
                    if (t < lo) t = lo;
                    if (t > hi2) t = hi2;
                    y[oi] = (unsigned char)(t & 0xff);
                }
    return 0;
}

float orc_bf16_round(float x) { return bf16_round(x); }

#ifdef _OPENMP
#include <omp.h>
int orc_num_threads(void) { return omp_get_max_threads(); }
#else
int orc_num_threads(void) { return 1; }
#endif
