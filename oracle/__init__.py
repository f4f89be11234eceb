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


def bf16_round(v: float) -> float:
    return float(lib().orc_bf16_round(v))
