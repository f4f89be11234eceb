"""Seeded synthetic workloads: SuperNet weight blobs, query inputs and SubNet config streams.

This module is the one piece shared by the CUDA library's callers and by the CPU checker.
It holds no inference arithmetic and no slicing rule: it only knows the *stored* (maximum)
shape of every SuperNet tensor, the elastic choice sets a config may draw from, and the
random recipes.  The paper evaluates on weight-shared ResNet50 / MobileNetV3 SuperNets with
trained weights (Section 5.1, "Workload"); those weights are not available, so the blobs
here are random tensors of the same organisation (stages -> blocks -> conv layers,
Section 2.1).

Blob format (little endian, all words 4 bytes):
    header   : 8 x uint32  = magic 'SGSB', version, family, n_records, seed, 0, 0, 0
    record i : 8 x uint32  = kind, K_max, C_max, R, S, has_bn, has_bias, 0
               float32 weight[K_max][C_max][R][S]        (depthwise: C_max == 1)
               if has_bn  : gamma[K_max], beta[K_max], mean[K_max], var[K_max]
               if has_bias: bias[K_max]
Records come in network order (see ``supernet_records``).
"""
from __future__ import annotations

import ctypes
import dataclasses
from typing import List, Sequence

import numpy as np

MAGIC = 0x42534753  # 'SGSB'
VERSION = 1

TINY, RESNET, MBV3 = 0, 1, 2
KIND_CONV, KIND_DW, KIND_LINEAR = 0, 1, 2

MAX_STAGES = 8
MAX_BLOCKS = 8


class SubnetCfg(ctypes.Structure):
    """Elastic choices of one SubNet (Section 2.1: depth, width / expand ratio, kernel).

    depth[s]      blocks kept in stage s (the first depth[s] blocks)
    width[0]      stem width multiplier, width[1+s] stage s width multiplier
    expand[s][b]  expand ratio of block b of stage s
    kernel[s][b]  depthwise kernel size of block b of stage s (MobileNetV3-shaped nets)
    """

    _fields_ = [
        ("depth", ctypes.c_int * MAX_STAGES),
        ("width", ctypes.c_float * (MAX_STAGES + 1)),
        ("expand", (ctypes.c_float * MAX_BLOCKS) * MAX_STAGES),
        ("kernel", (ctypes.c_int * MAX_BLOCKS) * MAX_STAGES),
    ]

    def key(self):
        return bytes(self)


class ArchDesc(ctypes.Structure):
    """SuperNet family and maxima, mirrored by both loaders."""

    _fields_ = [
        ("family", ctypes.c_int),
        ("n_stages", ctypes.c_int),
        ("max_depth", ctypes.c_int * MAX_STAGES),
        ("base_width", ctypes.c_int * MAX_STAGES),
        ("stem_width", ctypes.c_int),
        ("n_classes", ctypes.c_int),
        ("max_kernel", ctypes.c_int),
    ]


# ----------------------------------------------------------------------------------------------
# Stored shapes of the three synthetic SuperNets
# ----------------------------------------------------------------------------------------------

TINY_WIDTHS = (16, 32, 64)
TINY_MAX_DEPTH = (3, 3, 3)
TINY_WIDTH_SET = (0.5, 0.75, 1.0)
TINY_DEPTH_SET = (1, 2, 3)

RESNET_BASE = (256, 512, 1024, 2048)
RESNET_BASE_DEPTH = (2, 2, 4, 2)
RESNET_STEM = 64
RESNET_WIDTH_SET = (0.65, 0.8, 1.0)
RESNET_EXPAND_SET = (0.2, 0.25, 0.35)
RESNET_EXTRA_DEPTH_SET = (0, 1, 2)

MBV3_OUT = (24, 40, 80, 112, 160)
MBV3_SE = (0, 1, 0, 1, 1)
MBV3_STEM = 16
MBV3_DEPTH_SET = (2, 3, 4)
MBV3_EXPAND_SET = (3.0, 4.0, 6.0)
MBV3_KERNEL_SET = (3, 5, 7)
MBV3_HEAD = (960, 1280)


def arch_desc(family: int) -> ArchDesc:
    a = ArchDesc()
    a.family = family
    if family == TINY:
        a.n_stages = 3
        for s in range(3):
            a.max_depth[s] = TINY_MAX_DEPTH[s]
            a.base_width[s] = TINY_WIDTHS[s]
        a.stem_width = TINY_WIDTHS[0]
        a.n_classes = 10
        a.max_kernel = 3
    elif family == RESNET:
        a.n_stages = 4
        for s in range(4):
            a.max_depth[s] = RESNET_BASE_DEPTH[s] + 2
            a.base_width[s] = RESNET_BASE[s]
        a.stem_width = RESNET_STEM
        a.n_classes = 1000
        a.max_kernel = 7
    elif family == MBV3:
        a.n_stages = 5
        for s in range(5):
            a.max_depth[s] = 4
            a.base_width[s] = MBV3_OUT[s]
        a.stem_width = MBV3_STEM
        a.n_classes = 1000
        a.max_kernel = 7
    else:
        raise ValueError("unknown family")
    return a


@dataclasses.dataclass
class Record:
    name: str
    kind: int
    K: int
    C: int
    R: int
    S: int
    has_bn: bool
    has_bias: bool
    small_gamma: bool = False  # last BN of a residual branch: gamma ~ U(0.1, 0.3)

    @property
    def n_weights(self) -> int:
        return self.K * self.C * self.R * self.S

    @property
    def n_floats(self) -> int:
        return self.n_weights + (4 * self.K if self.has_bn else 0) + (self.K if self.has_bias else 0)


def _mult8_nearest(num: int, den: int) -> int:
    """Nearest multiple of 8 to num/den, ties up, at least 8 (stored widths only)."""
    return max(8, 8 * ((2 * num + 8 * den) // (16 * den)))


def supernet_records(family: int) -> List[Record]:
    """Stored tensors of a SuperNet in network (= blob) order."""
    rec: List[Record] = []
    if family == TINY:
        rec.append(Record("stem", KIND_CONV, TINY_WIDTHS[0], 3, 3, 3, True, False))
        prev = TINY_WIDTHS[0]
        for s, w in enumerate(TINY_WIDTHS):
            for b in range(TINY_MAX_DEPTH[s]):
                cin = prev if b == 0 else w
                rec.append(Record(f"s{s}b{b}.conv1", KIND_CONV, w, cin, 3, 3, True, False))
                rec.append(Record(f"s{s}b{b}.conv2", KIND_CONV, w, w, 3, 3, True, False, True))
                if b == 0 and s > 0:
                    rec.append(Record(f"s{s}b{b}.proj", KIND_CONV, w, cin, 1, 1, True, False))
            prev = w
        rec.append(Record("fc", KIND_LINEAR, 10, TINY_WIDTHS[-1], 1, 1, False, True))
    elif family == RESNET:
        rec.append(Record("stem", KIND_CONV, RESNET_STEM, 3, 7, 7, True, False))
        prev = RESNET_STEM
        for s, base in enumerate(RESNET_BASE):
            mid = _mult8_nearest(base * 35, 100)
            for b in range(RESNET_BASE_DEPTH[s] + 2):
                cin = prev if b == 0 else base
                rec.append(Record(f"s{s}b{b}.conv1", KIND_CONV, mid, cin, 1, 1, True, False))
                rec.append(Record(f"s{s}b{b}.conv2", KIND_CONV, mid, mid, 3, 3, True, False))
                rec.append(Record(f"s{s}b{b}.conv3", KIND_CONV, base, mid, 1, 1, True, False, True))
                if b == 0:
                    rec.append(Record(f"s{s}b{b}.proj", KIND_CONV, base, cin, 1, 1, True, False))
            prev = base
        rec.append(Record("fc", KIND_LINEAR, 1000, RESNET_BASE[-1], 1, 1, False, True))
    elif family == MBV3:
        rec.append(Record("stem", KIND_CONV, MBV3_STEM, 3, 3, 3, True, False))
        rec.append(Record("first.dw", KIND_DW, MBV3_STEM, 1, 3, 3, True, False))
        rec.append(Record("first.pw", KIND_CONV, MBV3_STEM, MBV3_STEM, 1, 1, True, False, True))
        prev = MBV3_STEM
        for s, out in enumerate(MBV3_OUT):
            for b in range(4):
                cin = prev if b == 0 else out
                mid = cin * 6
                rec.append(Record(f"s{s}b{b}.expand", KIND_CONV, mid, cin, 1, 1, True, False))
                rec.append(Record(f"s{s}b{b}.dw", KIND_DW, mid, 1, 7, 7, True, False))
                if MBV3_SE[s]:
                    sq = _mult8_nearest(mid, 4)
                    rec.append(Record(f"s{s}b{b}.se1", KIND_LINEAR, sq, mid, 1, 1, False, True))
                    rec.append(Record(f"s{s}b{b}.se2", KIND_LINEAR, mid, sq, 1, 1, False, True))
                rec.append(Record(f"s{s}b{b}.project", KIND_CONV, out, mid, 1, 1, True, False, True))
            prev = out
        rec.append(Record("head.conv", KIND_CONV, MBV3_HEAD[0], MBV3_OUT[-1], 1, 1, True, False))
        rec.append(Record("head.mix", KIND_LINEAR, MBV3_HEAD[1], MBV3_HEAD[0], 1, 1, False, True))
        rec.append(Record("fc", KIND_LINEAR, 1000, MBV3_HEAD[1], 1, 1, False, True))
    else:
        raise ValueError("unknown family")
    return rec


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even), returned as float32."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def make_blob(family: int, seed: int = 0, bf16_weights: bool = False) -> np.ndarray:
    """Random SuperNet blob (uint8 array).

    Conv / linear weights are He-normal with the fan-in of the *stored* tensor,
    std = sqrt(2 / (C_max R S)); BN gamma ~ U(0.5, 1.5) (U(0.1, 0.3) on the last BN of a
    residual branch so that deep SubNets stay in range), beta, mean ~ N(0, 0.1^2),
    var ~ U(0.5, 1.5); biases ~ N(0, 0.1^2).  With ``bf16_weights`` the conv / linear weights are
    rounded to bfloat16-representable values (still stored as float32).
    """
    rng = np.random.default_rng(seed)
    recs = supernet_records(family)
    total = 8 + sum(8 + r.n_floats for r in recs)
    out = np.empty(total, dtype=np.uint32)
    out[:8] = [MAGIC, VERSION, family, len(recs), seed & 0xFFFFFFFF, 0, 0, 0]
    pos = 8
    for r in recs:
        out[pos:pos + 8] = [r.kind, r.K, r.C, r.R, r.S, int(r.has_bn), int(r.has_bias), 0]
        pos += 8
        std = np.sqrt(2.0 / (r.C * r.R * r.S))
        w = (rng.standard_normal(r.n_weights, dtype=np.float32) * np.float32(std)).astype(np.float32)
        if bf16_weights:
            w = round_to_bf16(w)
        out[pos:pos + r.n_weights] = w.view(np.uint32)
        pos += r.n_weights
        if r.has_bn:
            lo, hi = (0.1, 0.3) if r.small_gamma else (0.5, 1.5)
            gamma = rng.uniform(lo, hi, r.K).astype(np.float32)
            beta = (rng.standard_normal(r.K) * 0.1).astype(np.float32)
            mean = (rng.standard_normal(r.K) * 0.1).astype(np.float32)
            var = rng.uniform(0.5, 1.5, r.K).astype(np.float32)
            for v in (gamma, beta, mean, var):
                out[pos:pos + r.K] = v.view(np.uint32)
                pos += r.K
        if r.has_bias:
            bias = (rng.standard_normal(r.K) * 0.1).astype(np.float32)
            out[pos:pos + r.K] = bias.view(np.uint32)
            pos += r.K
    assert pos == total
    return out.view(np.uint8)


def make_inputs(n: int, batch: int, res: int, seed: int = 1, bf16: bool = False) -> np.ndarray:
    """n queries of ``batch`` images each, NHWC, N(0, 1): shape (n, batch, res, res, 3) float32."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((n, batch, res, res, 3), dtype=np.float32)
    return round_to_bf16(x) if bf16 else x


# ----------------------------------------------------------------------------------------------
# SubNet config streams
# ----------------------------------------------------------------------------------------------

def _pick(rng, choices):
    return choices[int(rng.integers(len(choices)))]


def _fill_defaults(cfg: SubnetCfg) -> None:
    for s in range(MAX_STAGES):
        for b in range(MAX_BLOCKS):
            cfg.expand[s][b] = 1.0
            cfg.kernel[s][b] = 3
        cfg.width[s + 1] = 1.0
    cfg.width[0] = 1.0


def sample_cfg(family: int, rng) -> SubnetCfg:
    """One SubNet drawn uniformly from the elastic sets of the family."""
    cfg = SubnetCfg()
    _fill_defaults(cfg)
    if family == TINY:
        for s in range(3):
            cfg.depth[s] = _pick(rng, TINY_DEPTH_SET)
        for s in range(3):
            cfg.width[s + 1] = _pick(rng, TINY_WIDTH_SET)
        cfg.width[0] = cfg.width[1]
    elif family == RESNET:
        cfg.width[0] = _pick(rng, RESNET_WIDTH_SET)
        for s in range(4):
            cfg.width[s + 1] = _pick(rng, RESNET_WIDTH_SET)
        for s in range(4):
            cfg.depth[s] = RESNET_BASE_DEPTH[s] + _pick(rng, RESNET_EXTRA_DEPTH_SET)
        for s in range(4):
            for b in range(RESNET_BASE_DEPTH[s] + 2):
                cfg.expand[s][b] = _pick(rng, RESNET_EXPAND_SET)
    elif family == MBV3:
        for s in range(5):
            cfg.depth[s] = _pick(rng, MBV3_DEPTH_SET)
        for s in range(5):
            for b in range(4):
                cfg.expand[s][b] = _pick(rng, MBV3_EXPAND_SET)
                cfg.kernel[s][b] = _pick(rng, MBV3_KERNEL_SET)
    else:
        raise ValueError("unknown family")
    return cfg


def extreme_cfg(family: int, largest: bool) -> SubnetCfg:
    """The largest (= whole SuperNet) or smallest (shared by every SubNet) config."""
    cfg = SubnetCfg()
    _fill_defaults(cfg)
    sel = (lambda t: max(t)) if largest else (lambda t: min(t))
    if family == TINY:
        for s in range(3):
            cfg.depth[s] = sel(TINY_DEPTH_SET)
            cfg.width[s + 1] = sel(TINY_WIDTH_SET)
        cfg.width[0] = cfg.width[1]
    elif family == RESNET:
        cfg.width[0] = sel(RESNET_WIDTH_SET)
        for s in range(4):
            cfg.width[s + 1] = sel(RESNET_WIDTH_SET)
            cfg.depth[s] = RESNET_BASE_DEPTH[s] + sel(RESNET_EXTRA_DEPTH_SET)
            for b in range(RESNET_BASE_DEPTH[s] + 2):
                cfg.expand[s][b] = sel(RESNET_EXPAND_SET)
    elif family == MBV3:
        for s in range(5):
            cfg.depth[s] = sel(MBV3_DEPTH_SET)
            for b in range(4):
                cfg.expand[s][b] = sel(MBV3_EXPAND_SET)
                cfg.kernel[s][b] = sel(MBV3_KERNEL_SET)
    return cfg


def uniform_stream(family: int, n: int, seed: int) -> List[SubnetCfg]:
    rng = np.random.default_rng(seed)
    return [sample_cfg(family, rng) for _ in range(n)]


def candidate_cfgs(family: int, n: int, seed: int) -> List[SubnetCfg]:
    """A set of n SubNet configs whose encodings serve as the scheduler's cacheable SubGraphs (Section 3.2):
    the smallest and the largest SubNet, then seeded uniform draws."""
    rng = np.random.default_rng(seed)
    out = [extreme_cfg(family, False), extreme_cfg(family, True)][:n]
    while len(out) < n:
        out.append(sample_cfg(family, rng))
    return out


def proxy_accuracy(flops: Sequence[float], lo: float = 0.70, hi: float = 0.80) -> np.ndarray:
    """Stand-in for the trained SubNets' accuracies (inputs of the scheduler): monotone in the SubNet's FLOPs,
    spread linearly in log-FLOPs over [lo, hi]."""
    f = np.log(np.asarray(flops, dtype=np.float64))
    span = float(f.max() - f.min())
    return lo + (hi - lo) * ((f - f.min()) / span if span > 0 else np.zeros_like(f))


def sched_queries(n: int, seed: int, accuracy: Sequence[float], latency: Sequence[float], p_accuracy: float = 0.5):
    """n scheduler queries (policy, A_t, L_t): policy 0 (accuracy is the hard constraint) with probability
    p_accuracy, else 1 (latency is); targets drawn uniformly from a range slightly wider than the SubNets'
    own accuracies and latencies, so that some queries have an empty feasible set."""
    rng = np.random.default_rng(seed)
    acc = np.asarray(accuracy, dtype=np.float64)
    lat = np.asarray(latency, dtype=np.float64)
    da, dl = float(acc.max() - acc.min()), float(lat.max() - lat.min())
    policy = (rng.random(n) >= p_accuracy).astype(np.int32)
    a_t = rng.uniform(acc.min() - 0.1 * da, acc.max() + 0.1 * da, n)
    l_t = rng.uniform(lat.min() - 0.1 * dl, lat.max() + 0.1 * dl, n)
    return policy, a_t, l_t


def copy_cfg(c: SubnetCfg) -> SubnetCfg:
    d = SubnetCfg()
    ctypes.memmove(ctypes.byref(d), ctypes.byref(c), ctypes.sizeof(SubnetCfg))
    return d


def markov_stream(n: int, seed: int = 4, p_local: float = 0.9, family: int = RESNET) -> List[SubnetCfg]:
    """Locality stream on the ResNet-50-shaped (default) or MobileNetV3-shaped SuperNet.

    With probability ``p_local`` the next config differs from the previous one in one place (ResNet: one
    stage's depth or width; MobileNetV3: one stage's depth, or one block's expansion ratio or kernel size),
    redrawn possibly to the same value; otherwise the whole config is redrawn uniformly.  This gives
    consecutive queries a large shared SubGraph, the temporal locality the paper's SubGraph-Stationary reuse
    exploits (Section 2.2).
    """
    if family not in (RESNET, MBV3):
        raise ValueError("locality streams exist for the ResNet- and MobileNetV3-shaped families")
    rng = np.random.default_rng(seed)
    cur = sample_cfg(family, rng)
    out = [cur]
    for _ in range(n - 1):
        nxt = copy_cfg(cur)
        if rng.random() >= p_local:
            nxt = sample_cfg(family, rng)
        elif family == RESNET:
            s = int(rng.integers(4))
            if int(rng.integers(2)) == 0:
                nxt.depth[s] = RESNET_BASE_DEPTH[s] + _pick(rng, RESNET_EXTRA_DEPTH_SET)
            else:
                nxt.width[s + 1] = _pick(rng, RESNET_WIDTH_SET)
        else:
            s, what = int(rng.integers(5)), int(rng.integers(3))
            if what == 0:
                nxt.depth[s] = _pick(rng, MBV3_DEPTH_SET)
            elif what == 1:
                nxt.expand[s][int(rng.integers(4))] = _pick(rng, MBV3_EXPAND_SET)
            else:
                nxt.kernel[s][int(rng.integers(4))] = _pick(rng, MBV3_KERNEL_SET)
        out.append(nxt)
        cur = nxt
    return out


def cfg_array(cfgs: Sequence[SubnetCfg]):
    arr = (SubnetCfg * len(cfgs))()
    for i, c in enumerate(cfgs):
        ctypes.memmove(ctypes.byref(arr, i * ctypes.sizeof(SubnetCfg)), ctypes.byref(c),
                       ctypes.sizeof(SubnetCfg))
    return arr
