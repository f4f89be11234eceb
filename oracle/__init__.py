"""ctypes front end of the CPU checker (oracle/sgs_oracle.c).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU-baseline leg of
the benchmark.  Nothing in the product package may import it.  The C file is compiled on the
machine that runs it (``-march=native``), into ``oracle/_build``.
"""
from __future__ import annotations

import ctypes
import hashlib
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sgs_oracle.c")
FP32, BF16_STORE = 0, 1
ACT_NONE, ACT_RELU, ACT_HSWISH = 0, 1, 2

_lib = None


def _cpu_tag() -> str:
    flags = ""
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    flags = line
                    break
    except OSError:
        pass
    with open(_SRC, "rb") as f:
        src = f.read()
    return hashlib.sha1(flags.encode() + src).hexdigest()[:12]


def build(force: bool = False) -> str:
    """Compile the checker for this machine and return the path of the shared object."""
    out_dir = os.path.join(_HERE, "_build")
    os.makedirs(out_dir, exist_ok=True)
    so = os.path.join(out_dir, f"liboracle_{_cpu_tag()}.so")
    if force or not os.path.exists(so):
        tmp = so + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, so)
    return so


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.orc_load.restype = ctypes.c_void_p
        L.orc_load.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_char_p, ctypes.c_int]
        L.orc_free.argtypes = [ctypes.c_void_p]
        L.orc_num_layers.argtypes = [ctypes.c_void_p]
        L.orc_validate.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        L.orc_encode.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.orc_encoding_weights.restype = ctypes.c_longlong
        L.orc_encoding_weights.argtypes = [ctypes.c_void_p, ctypes.c_int]
        L.orc_intersect.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
        L.orc_hit_ratio.restype = ctypes.c_double
        L.orc_hit_ratio.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int]
        fw = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        L.orc_forward.argtypes = fw
        L.orc_forward_extracted.argtypes = fw
        L.orc_forward_unsliced.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        L.orc_layer_conv.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 4 + [ctypes.c_void_p] + [ctypes.c_int] * 7 + [ctypes.c_void_p]
        L.orc_layer_epilogue.argtypes = [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int] + [ctypes.c_void_p] * 6 + [ctypes.c_int, ctypes.c_int]
        L.orc_layer_maxpool.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 4 + [ctypes.c_void_p]
        L.orc_layer_gap.argtypes = [ctypes.c_void_p] + [ctypes.c_int] * 3 + [ctypes.c_void_p]
        L.orc_layer_linear.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 4 + [ctypes.c_void_p]
        L.orc_layer_se_gate.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 3 + [ctypes.c_void_p]
        L.orc_layer_se_scale.argtypes = [ctypes.c_void_p, ctypes.c_void_p] + [ctypes.c_int] * 4
        L.orc_layer_conv_i8.argtypes = ([ctypes.c_void_p] + [ctypes.c_int] * 3 + [ctypes.c_void_p] + [ctypes.c_int] * 9 + [ctypes.c_void_p] * 4
                                        + [ctypes.c_int] * 7 + [ctypes.c_void_p])
        L.orc_bf16_round.restype = ctypes.c_float
        L.orc_bf16_round.argtypes = [ctypes.c_float]
        L.orc_set_tap.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t]
        L.orc_get_tap_dims.argtypes = [ctypes.c_void_p]
        L.orc_num_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def num_threads() -> int:
    return int(lib().orc_num_threads())


class Net:
    """A loaded SuperNet blob."""

    def __init__(self, family: int, blob: np.ndarray):
        blob = np.ascontiguousarray(blob, dtype=np.uint8)
        err = ctypes.create_string_buffer(256)
        self._h = lib().orc_load(family, _ptr(blob), blob.nbytes, err, 256)
        if not self._h:
            raise ValueError(err.value.decode())
        self.family = family
        self.n_layers = lib().orc_num_layers(self._h)

    def __del__(self):
        if getattr(self, "_h", None):
            lib().orc_free(self._h)
            self._h = None

    def validate(self, cfg) -> bool:
        return lib().orc_validate(self._h, ctypes.byref(cfg)) == 0

    def encode(self, cfg) -> np.ndarray:
        """(n_layers, 3) int array of K_i, C_i, k_i per stored layer (zeros if unused)."""
        out = np.zeros((self.n_layers, 3), dtype=np.int32)
        if lib().orc_encode(self._h, ctypes.byref(cfg), _ptr(out)) < 0:
            raise ValueError("config outside the elastic sets")
        return out

    def _n_classes(self) -> int:
        return 10 if self.family == 0 else 1000

    def forward(self, cfg, x, mode: int = FP32, path: str = "sliced") -> np.ndarray:
        x = _f32(x)
        n, res = x.shape[0], x.shape[1]
        out = np.empty((n, self._n_classes()), dtype=np.float32)
        if path == "sliced":
            rc = lib().orc_forward(self._h, ctypes.byref(cfg), _ptr(x), n, res, mode, _ptr(out))
        elif path == "extracted":
            rc = lib().orc_forward_extracted(self._h, ctypes.byref(cfg), _ptr(x), n, res, mode, _ptr(out))
        elif path == "unsliced":
            rc = lib().orc_forward_unsliced(self._h, _ptr(x), n, res, mode, _ptr(out))
        else:
            raise ValueError(path)
        if rc:
            raise ValueError(f"oracle forward failed ({rc})")
        return out

    def forward_tap(self, cfg, x, layer: int, mode: int = FP32):
        """Run the sliced forward and also return the activation stored layer ``layer`` produced."""
        x = _f32(x)
        buf = np.zeros(x.shape[0] * x.shape[1] * x.shape[2] * 128, dtype=np.float32)
        lib().orc_set_tap(layer, _ptr(buf), buf.size)
        try:
            logits = self.forward(cfg, x, mode)
            d = (ctypes.c_int * 4)()
            lib().orc_get_tap_dims(d)
        finally:
            lib().orc_set_tap(-1, None, 0)
        dims = tuple(int(v) for v in d)
        if dims[0] == 0:
            return logits, None
        return logits, buf[: int(np.prod(dims))].reshape(dims).copy()


def encoding_weights(enc: np.ndarray) -> int:
    enc = np.ascontiguousarray(enc, dtype=np.int32)
    return int(lib().orc_encoding_weights(_ptr(enc), enc.shape[0]))


def intersect(a: np.ndarray, b: np.ndarray) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.int32)
    b = np.ascontiguousarray(b, dtype=np.int32)
    out = np.empty_like(a)
    lib().orc_intersect(_ptr(a), _ptr(b), a.shape[0], _ptr(out))
    return out


def hit_ratio(sn: np.ndarray, g: np.ndarray) -> float:
    sn = np.ascontiguousarray(sn, dtype=np.int32)
    g = np.ascontiguousarray(g, dtype=np.int32)
    return float(lib().orc_hit_ratio(_ptr(sn), _ptr(g), sn.shape[0]))


def layer_conv(w, x, Cp: int, Kp: int, k: int, stride: int, depthwise: bool = False) -> np.ndarray:
    """Sliced convolution of NHWC ``x`` with the stored tensor ``w`` [Kmax][Cmax][R][R]."""
    w = _f32(w)
    x = _f32(x)
    Kmax, Cmax, R, _ = w.shape
    N, H, W, _ = x.shape
    p = (k - 1) // 2
    Ho, Wo = (H + 2 * p - k) // stride + 1, (W + 2 * p - k) // stride + 1
    y = np.empty((N, Ho, Wo, Kp), dtype=np.float32)
    rc = lib().orc_layer_conv(_ptr(w), Kmax, Cmax, R, int(depthwise), _ptr(x), N, H, W, Cp, Kp, k, stride, _ptr(y))
    if rc:
        raise MemoryError
    return y


def layer_epilogue(y, gamma=None, beta=None, mean=None, var=None, bias=None, res=None, act=ACT_NONE,
                   mode=FP32) -> np.ndarray:
    y = _f32(y).copy()
    Kp = y.shape[-1]
    arrs = [None if a is None else _f32(a) for a in (gamma, beta, mean, var, bias, res)]
    lib().orc_layer_epilogue(_ptr(y), y.size // Kp, Kp, *[_ptr(a) for a in arrs], act, mode)
    return y


def layer_maxpool(x) -> np.ndarray:
    x = _f32(x)
    N, H, W, C = x.shape
    y = np.empty((N, (H - 1) // 2 + 1, (W - 1) // 2 + 1, C), dtype=np.float32)
    lib().orc_layer_maxpool(_ptr(x), N, H, W, C, _ptr(y))
    return y


def layer_gap(x) -> np.ndarray:
    x = _f32(x)
    N, H, W, C = x.shape
    g = np.empty((N, C), dtype=np.float32)
    lib().orc_layer_gap(_ptr(x), N, H * W, C, _ptr(g))
    return g


def layer_linear(w, bias, v, Cp: int, Kp: int, act: int = ACT_NONE) -> np.ndarray:
    """Sliced fully connected layer on the stored matrix ``w`` [Kmax][Cmax]: first Kp outputs of the first Cp inputs."""
    w, v = _f32(w), _f32(v)
    bias = None if bias is None else _f32(bias)
    y = np.empty((v.shape[0], Kp), dtype=np.float32)
    lib().orc_layer_linear(_ptr(w), w.shape[1], _ptr(bias), _ptr(v), v.shape[0], Cp, Kp, act, _ptr(y))
    return y


def layer_se_gate(w1, b1, w2, b2, g, sq: int) -> np.ndarray:
    """Squeeze-excite gate of the pooled vectors ``g`` [N][mid]: hsigmoid(FC2(relu(FC1(g)))), FC1 = first sq rows of
    ``w1`` [.][>=mid], FC2 = first mid rows of ``w2`` [.][>=sq]."""
    w1, w2, g = _f32(w1), _f32(w2), _f32(g)
    b1, b2 = _f32(b1), _f32(b2)
    gate = np.empty_like(g)
    if lib().orc_layer_se_gate(_ptr(w1), w1.shape[1], _ptr(b1), _ptr(w2), w2.shape[1], _ptr(b2), _ptr(g), g.shape[0], g.shape[1], sq, _ptr(gate)):
        raise MemoryError
    return gate


def layer_se_scale(x, gate, mode: int = FP32) -> np.ndarray:
    """x[n][h][w][c] * gate[n][c] with the storage rounding of ``mode``."""
    y = _f32(x).copy()
    gate = _f32(gate)
    N, H, W, C = y.shape
    lib().orc_layer_se_scale(_ptr(y), _ptr(gate), N, H * W, C, mode)
    return y


def layer_conv_i8(w, x, Cp: int, Kp: int, k: int, stride: int, mult, shift, bias, zx: int = 0, zy: int = 0, relu: bool = False,
                  res=None, zr: int = 0, res_mult: int = 0, res_shift: int = 0, y_signed: bool = False) -> np.ndarray:
    """8-bit sliced convolution layer in exact integer arithmetic (see the C function).  ``w`` int8 [Kmax][Cmax][R][R];
    ``x`` (and ``res``) uint8 or int8 NHWC, their dtype says how the bytes are read; returns uint8, or int8 if y_signed."""
    w = np.ascontiguousarray(w, dtype=np.int8)
    x = np.ascontiguousarray(x)
    assert x.dtype in (np.uint8, np.int8)
    Kmax, Cmax, R, _ = w.shape
    N, H, W, _ = x.shape
    p = (k - 1) // 2
    Ho, Wo = (H + 2 * p - k) // stride + 1, (W + 2 * p - k) // stride + 1
    mult, shift, bias = (np.ascontiguousarray(a, dtype=np.int32) for a in (mult, shift, bias))
    if res is not None:
        res = np.ascontiguousarray(res)
        assert res.dtype in (np.uint8, np.int8) and res.shape == (N, Ho, Wo, Kp)
    y = np.empty((N, Ho, Wo, Kp), dtype=np.int8 if y_signed else np.uint8)
    rc = lib().orc_layer_conv_i8(_ptr(w), Kmax, Cmax, R, _ptr(x), int(x.dtype == np.int8), zx, N, H, W, Cp, Kp, k, stride,
                                 _ptr(mult), _ptr(shift), _ptr(bias), _ptr(res), int(res is not None and res.dtype == np.int8), zr,
                                 res_mult, res_shift, zy, int(relu), int(y_signed), _ptr(y))
    if rc:
        raise OverflowError("accumulator beyond 32 bits" if rc == -3 else f"orc_layer_conv_i8 failed ({rc})")
    return y


def bf16_round(v: float) -> float:
    return float(lib().orc_bf16_round(v))


# ------------------------------------------------------------------------------------------------
# Scheduler's caching decision (paper Section 3.3 "Amortizing Caching Choices", "Predicting the Next
# SubGraph", Algorithm 1's cache branch, Section 3.2 for the candidate set S).  Plain loops on the
# (K, C, k) encodings; test infrastructure only.
# ------------------------------------------------------------------------------------------------
def layer_weights(enc: np.ndarray) -> np.ndarray:
    """Weights of every layer of an encoding: K * C * k * k."""
    e = np.asarray(enc, dtype=np.int64).reshape(-1, 3)
    return e[:, 0] * e[:, 1] * e[:, 2] * e[:, 2]


def clip_to_budget(enc: np.ndarray, budget_weights: int) -> np.ndarray:
    """A cacheable SubGraph of at most `budget_weights` weights (Section 3.2: SubGraphs in S have about the
    cache's size): walking the layers in network order, a layer's box is kept if it still fits beside the
    boxes kept so far, else the layer is left out."""
    e = np.array(enc, dtype=np.int32).reshape(-1, 3).copy()
    used = 0
    for i, w in enumerate(layer_weights(e)):
        if used + int(w) > budget_weights:
            e[i, :] = 0
        else:
            used += int(w)
    return e.reshape(np.asarray(enc).shape)


def nearest_candidate(window, candidates) -> int:
    """Index j of the candidate SubGraph closest to the running average of the SubNets in `window`
    (Algorithm 1: CacheState = argmin_j Dist(G_j, AvgNet); Dist = Euclidean distance on the (K_i, C_i)
    vector encoding of Section 3.3).  With Q = len(window) and S = the element-wise sum over the window,
    Dist^2 * Q^2 = sum_i (Q * G_ji - S_i)^2: compared exactly in integers.  Ties go to the lowest index."""
    q = len(window)
    s = np.zeros_like(np.asarray(window[0], dtype=np.int64).reshape(-1, 3))
    for e in window:
        s = s + np.asarray(e, dtype=np.int64).reshape(-1, 3)
    best, best_d = -1, None
    for j, g in enumerate(candidates):
        g3 = np.asarray(g, dtype=np.int64).reshape(-1, 3)
        d = 0
        for i in range(g3.shape[0]):
            for c in range(2):  # K and C entries
                t = q * int(g3[i, c]) - int(s[i, c])
                d += t * t
        if best_d is None or d < best_d:
            best, best_d = j, d
    return best


def sched_stream(encs, candidates, q: int):
    """Serve the SubNets `encs` in order; after every q-th query the cached SubGraph becomes the candidate
    nearest to the average of the last q served SubNets (Algorithm 1).  Query t is accounted against the
    SubGraph cached before it is served (none before the first decision).  Returns per-query hit ratios
    (Appendix A.4), missed weights, and the list of choices (one per decision)."""
    hits, missed, choices = [], [], []
    window, g, since = [], None, 0
    candidates = [np.ascontiguousarray(c, dtype=np.int32).reshape(-1, 3) for c in candidates]
    for e in encs:
        e = np.ascontiguousarray(e, dtype=np.int32).reshape(-1, 3)
        if g is None:
            hits.append(0.0)
            missed.append(encoding_weights(e))
        else:
            hits.append(hit_ratio(e, g))
            missed.append(encoding_weights(e) - encoding_weights(intersect(e, g)))
        window.append(e)
        if len(window) > q:
            window.pop(0)
        since += 1
        if since >= q:
            since = 0
            j = nearest_candidate(window, candidates)
            choices.append(j)
            g = candidates[j]
    return hits, missed, choices


STRICT_ACCURACY, STRICT_LATENCY = 0, 1


def select_subnet(policy: int, a_t: float, l_t: float, accuracy, latency_col) -> int:
    """Per-query SubNet selection of Algorithm 1 (Section 3.3) for the cache state whose latency column is
    `latency_col`.  STRICT_ACCURACY: the fastest SubNet among those with accuracy >= A_t.  STRICT_LATENCY: the
    most accurate SubNet among those with latency <= L_t.  Where the paper is silent: an empty feasible set
    falls back to the most accurate SubNet (STRICT_ACCURACY) or the fastest one (STRICT_LATENCY); ties are
    broken by the other quantity (higher accuracy / lower latency), then by the lowest index."""
    n = len(accuracy)
    by_latency = lambda i: (latency_col[i], -accuracy[i], i)
    by_accuracy = lambda i: (-accuracy[i], latency_col[i], i)
    if policy == STRICT_ACCURACY:
        feasible = [i for i in range(n) if accuracy[i] >= a_t]
        return min(feasible, key=by_latency) if feasible else min(range(n), key=by_accuracy)
    feasible = [i for i in range(n) if latency_col[i] <= l_t]
    return min(feasible, key=by_accuracy) if feasible else min(range(n), key=by_latency)


def sushi_sched(queries, accuracy, table, subnet_encs, cand_encs, q: int):
    """Algorithm 1 as a whole.  queries: (policy, A_t, L_t) per query; table[i][j]: latency of SubNet i with
    candidate SubGraph j cached, column M = len(cand_encs) for an empty cache (the state before the first
    caching decision).  Every query is served with the SubNet selected for the current cache state; after
    every q-th query the cache state becomes the candidate nearest to the average of the last q served
    SubNets.  Returns (served SubNet index per query, cache state each query was served under)."""
    m = len(cand_encs)
    state, window, since = m, [], 0
    served, states = [], []
    for policy, a_t, l_t in queries:
        col = [row[state] for row in table]
        i = select_subnet(policy, a_t, l_t, accuracy, col)
        served.append(i)
        states.append(state)
        window.append(subnet_encs[i])
        if len(window) > q:
            window.pop(0)
        since += 1
        if since >= q:
            since = 0
            state = nearest_candidate(window, cand_encs)
    return served, states
