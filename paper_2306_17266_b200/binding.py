"""Thin ctypes binding of libsgs.so: argument marshalling only, same names as include/sgs.h.

Device buffers are passed as integer addresses (for example ``tensor.data_ptr()``), streams as the
integer ``cudaStream_t`` (``torch.cuda.current_stream().cuda_stream``).  There is no CPU fallback:
importing works without the library, every call raises if it cannot be loaded.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

from .workload import ArchDesc, SubnetCfg, arch_desc, cfg_array

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("SGS_LIB") or os.path.join(_HERE, "libsgs.so")  # SGS_LIB: use another build of the library

SGS_OK, SGS_EINVAL, SGS_ECONFIG, SGS_ENOMEM, SGS_ECUDA, SGS_ETIMEOUT, SGS_EUNSUPPORTED = range(7)
SGS_POLICY_INTERSECTION, SGS_POLICY_AVGNET = 0, 1
SGS_STRICT_ACCURACY, SGS_STRICT_LATENCY = 0, 1
SGS_F32, SGS_BF16 = 0, 1
STATUS_NAMES = ["SGS_OK", "SGS_EINVAL", "SGS_ECONFIG", "SGS_ENOMEM", "SGS_ECUDA", "SGS_ETIMEOUT", "SGS_EUNSUPPORTED"]

EXPORTS = [
    "sgs_supernet_load", "sgs_subnet_validate", "sgs_subnet_run", "sgs_stream_run", "sgs_stream_run_host",
    "sgs_cache_configure", "sgs_cache_stats", "sgs_num_layers", "sgs_subnet_encode", "sgs_subnet_cost",
    "sgs_set_option", "sgs_get_counter", "sgs_last_error", "sgs_supernet_free", "sgs_conv2d_sliced", "sgs_device_status",
    "sgs_profile_read", "sgs_conv2d_sliced_static", "sgs_cache_set_candidates", "sgs_cache_set_policy",
    "sgs_sched_create", "sgs_sched_free", "sgs_sched_dims", "sgs_sched_set_table", "sgs_sched_get_table", "sgs_sched_measure",
    "sgs_sched_step", "sgs_sched_subnet", "sgs_profile_trace", "sgs_layer_name", "sgs_aux_op", "sgs_device_status_clear", "sgs_debug_expire_wait", "sgs_measure_fma_peak", "sgs_conv2d_sliced_i8",
]


class ConvDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("N", "H", "W", "C", "K", "Kmax", "Cmax", "R", "k", "stride", "act", "dtype",
                                             "impl", "depthwise", "cache_k", "cache_c", "weight_policy", "split_k_off")]


class ConvI8Desc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("N", "H", "W", "C", "K", "Kmax", "Cmax", "R", "k", "stride", "relu", "x_signed", "y_signed",
                                             "res_signed", "zx", "zy", "zr", "res_mult", "res_shift", "ldx", "ldy")]


SGS_AUX_MAXPOOL, SGS_AUX_AVGPOOL, SGS_AUX_LINEAR, SGS_AUX_SE_GATE, SGS_AUX_SE_SCALE = range(5)


class AuxDesc(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("kind", "dtype", "N", "H", "W", "C", "K", "ld", "ld2", "act")]


class AuxArgs(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("x", "y", "w", "bias", "w2", "bias2")]


class StreamOpts(ctypes.Structure):
    _fields_ = [("cache_enabled", ctypes.c_int), ("window_q", ctypes.c_int), ("cache_budget_bytes", ctypes.c_size_t),
                ("use_graphs", ctypes.c_int), ("record_latency", ctypes.c_int), ("weights_evict_first", ctypes.c_int),
                ("concurrency", ctypes.c_int), ("wave", ctypes.c_int), ("policy", ctypes.c_int), ("persistent", ctypes.c_int)]


class StreamStats(ctypes.Structure):
    _fields_ = [("n_queries", ctypes.c_int), ("total_ms", ctypes.c_double), ("queries_per_s", ctypes.c_double),
                ("images_per_s", ctypes.c_double), ("p50_ms", ctypes.c_double), ("p99_ms", ctypes.c_double),
                ("mean_ms", ctypes.c_double), ("useful_flops", ctypes.c_double), ("weight_bytes", ctypes.c_double),
                ("hbm_weight_bytes", ctypes.c_double), ("hit_ratio", ctypes.c_double), ("byte_hit_ratio", ctypes.c_double),
                ("kernel_launches", ctypes.c_longlong), ("plan_hits", ctypes.c_int), ("plan_misses", ctypes.c_int),
                ("cache_updates", ctypes.c_int)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class CacheStats(ctypes.Structure):
    _fields_ = [("enabled", ctypes.c_int), ("window_q", ctypes.c_int), ("budget_bytes", ctypes.c_size_t),
                ("l2_bytes", ctypes.c_size_t), ("persisting_l2_max", ctypes.c_size_t), ("access_window_max", ctypes.c_size_t),
                ("cached_subgraph_bytes", ctypes.c_size_t), ("supernet_bytes", ctypes.c_size_t),
                ("device_bytes_allocated", ctypes.c_size_t), ("policy", ctypes.c_int), ("n_candidates", ctypes.c_int),
                ("decisions", ctypes.c_int), ("last_choice", ctypes.c_int)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class LaunchRecord(ctypes.Structure):
    _fields_ = [("kernel_class", ctypes.c_int), ("layer", ctypes.c_int), ("members", ctypes.c_int), ("tiles", ctypes.c_int),
                ("ms", ctypes.c_double), ("alg_bytes", ctypes.c_double), ("flops", ctypes.c_double)]


class Scheduler:
    """sgs_sched_*: Algorithm 1 over a latency table (rows = SubNets, columns = the SuperNet's candidate SubGraphs
    plus one for an empty cache).  Argument marshalling only."""

    def __init__(self, net: "SuperNet", subnets: Sequence, accuracy: Sequence[float], window_q: int):
        import numpy as np
        self.net = net
        arr = subnets if isinstance(subnets, ctypes.Array) else cfg_array(subnets)
        acc = np.ascontiguousarray(accuracy, dtype=np.float64)
        if acc.shape != (len(arr),):
            raise ValueError("one accuracy per SubNet")
        self._h = ctypes.c_void_p()
        net._check(lib().sgs_sched_create(net._h, ctypes.addressof(arr), acc.ctypes.data, len(arr), window_q, ctypes.byref(self._h)))
        n, m = ctypes.c_int(), ctypes.c_int()
        net._check(lib().sgs_sched_dims(self._h, ctypes.addressof(n), ctypes.addressof(m)))
        self.n_subnets, self.n_columns = n.value, m.value

    def close(self):
        if self._h:
            lib().sgs_sched_free(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_table(self, table):
        import numpy as np
        tb = np.ascontiguousarray(table, dtype=np.float64)
        if tb.shape != (self.n_subnets, self.n_columns):
            raise ValueError("table must be [n_subnets][n_columns]")
        self.net._check(lib().sgs_sched_set_table(self._h, tb.ctypes.data))

    def get_table(self):
        import numpy as np
        tb = np.zeros((self.n_subnets, self.n_columns), dtype=np.float64)
        self.net._check(lib().sgs_sched_get_table(self._h, tb.ctypes.data))
        return tb

    def measure(self, d_input: int, batch: int, res: int, d_logits: int, reps: int = 5, flush_bytes: int = 0, stream: int = 0):
        self.net._check(lib().sgs_sched_measure(self._h, d_input, batch, res, d_logits, reps, flush_bytes, stream))

    def step(self, policy, a_t, l_t):
        """Arrays (or scalars) of query policies, accuracy and latency targets -> (served rows, cache-state columns)."""
        import numpy as np
        pol = np.ascontiguousarray(np.atleast_1d(policy), dtype=np.int32)
        a = np.ascontiguousarray(np.atleast_1d(a_t), dtype=np.float64)
        l = np.ascontiguousarray(np.atleast_1d(l_t), dtype=np.float64)
        if not (pol.shape == a.shape == l.shape) or pol.ndim != 1:
            raise ValueError("policy, a_t and l_t must be 1-d and of one length")
        sub = np.zeros(len(pol), dtype=np.int32)
        state = np.zeros(len(pol), dtype=np.int32)
        self.net._check(lib().sgs_sched_step(self._h, len(pol), pol.ctypes.data, a.ctypes.data, l.ctypes.data, sub.ctypes.data, state.ctypes.data))
        return sub, state

    def subnet(self, i: int) -> SubnetCfg:
        c = SubnetCfg()
        self.net._check(lib().sgs_sched_subnet(self._h, i, ctypes.byref(c)))
        return c


class SgsError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}: {text}")
        self.status = status


_lib = None


def lib():
    """Load libsgs.so (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2306_17266_b200.build` first")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci, cs = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.sgs_supernet_load.argtypes = [vp, vp, cs, ci, ci, ctypes.POINTER(vp)]
        L.sgs_subnet_validate.argtypes = [vp, vp]
        L.sgs_subnet_run.argtypes = [vp, vp, vp, ci, ci, vp, vp]
        L.sgs_stream_run.argtypes = [vp, ci, vp, vp, ci, ci, vp, vp, vp, vp]
        L.sgs_stream_run_host.argtypes = [vp, ci, vp, vp, ci, ci, vp, vp, vp, vp]
        L.sgs_cache_configure.argtypes = [vp, ci, cs, ci]
        L.sgs_cache_stats.argtypes = [vp, vp]
        L.sgs_cache_set_candidates.argtypes = [vp, vp, ci]
        L.sgs_cache_set_policy.argtypes = [vp, ci]
        L.sgs_sched_create.argtypes = [vp, vp, vp, ci, ci, ctypes.POINTER(vp)]
        L.sgs_sched_free.argtypes = [vp]
        L.sgs_sched_free.restype = None
        L.sgs_sched_dims.argtypes = [vp, vp, vp]
        L.sgs_sched_set_table.argtypes = [vp, vp]
        L.sgs_sched_get_table.argtypes = [vp, vp]
        L.sgs_sched_measure.argtypes = [vp, vp, ci, ci, vp, ci, cs, vp]
        L.sgs_sched_step.argtypes = [vp, ci, vp, vp, vp, vp, vp]
        L.sgs_sched_subnet.argtypes = [vp, ci, vp]
        L.sgs_profile_trace.argtypes = [vp, vp, ci]
        L.sgs_layer_name.argtypes = [vp, ci, ctypes.c_char_p, ci]
        L.sgs_num_layers.argtypes = [vp]
        L.sgs_subnet_encode.argtypes = [vp, vp, vp]
        L.sgs_subnet_cost.argtypes = [vp, vp, ci, ci, vp, vp, vp]
        L.sgs_set_option.argtypes = [vp, ctypes.c_char_p, ctypes.c_longlong]
        L.sgs_get_counter.argtypes = [vp, ctypes.c_char_p]
        L.sgs_get_counter.restype = ctypes.c_longlong
        L.sgs_last_error.argtypes = [vp]
        L.sgs_last_error.restype = ctypes.c_char_p
        L.sgs_supernet_free.argtypes = [vp]
        L.sgs_supernet_free.restype = None
        L.sgs_conv2d_sliced.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
        L.sgs_conv2d_sliced_static.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp]
        L.sgs_device_status.argtypes = []
        L.sgs_aux_op.argtypes = [ci, vp, vp, ci, vp]
        L.sgs_device_status_clear.argtypes = []
        L.sgs_debug_expire_wait.argtypes = [ctypes.c_uint, vp]
        L.sgs_measure_fma_peak.argtypes = [vp, vp]
        L.sgs_conv2d_sliced_i8.argtypes = [vp] * 9
        L.sgs_profile_read.argtypes = [vp, ci, vp, vp, vp, vp]
        _lib = L
    return _lib


def _addr(buf) -> int:
    """Integer address of a host buffer (numpy array / ctypes object) or pass an int through."""
    if buf is None:
        return 0
    if isinstance(buf, int):
        return buf
    if hasattr(buf, "ctypes"):
        return buf.ctypes.data
    return ctypes.addressof(buf)


def conv2d_sliced(desc: ConvDesc, d_x: int, d_w: int, d_scale: int, d_shift: int, d_res: int, d_y: int, stream: int = 0):
    st = lib().sgs_conv2d_sliced(ctypes.byref(desc), d_x, d_w, d_scale, d_shift, d_res or None, d_y, stream)
    if st != SGS_OK:
        raise SgsError(st, "sgs_conv2d_sliced")


def conv2d_sliced_static(desc: ConvDesc, d_x: int, d_w: int, d_scale: int, d_shift: int, d_res: int, d_y: int,
                         stream: int = 0):
    """The sliced convolution without any device allocation (fixed scratch inside the library)."""
    st = lib().sgs_conv2d_sliced_static(ctypes.byref(desc), d_x, d_w, d_scale, d_shift, d_res or None, d_y, stream)
    if st != SGS_OK:
        raise SgsError(st, "sgs_conv2d_sliced_static")


def conv2d_sliced_i8(desc: ConvI8Desc, d_x: int, d_w: int, d_mult: int, d_shift: int, d_bias: int, d_res: int, d_y: int, stream: int = 0):
    st = lib().sgs_conv2d_sliced_i8(ctypes.byref(desc), d_x, d_w, d_mult, d_shift, d_bias, d_res or None, d_y, stream)
    if st != SGS_OK:
        raise SgsError(st, "sgs_conv2d_sliced_i8")


def device_status_clear():
    st = lib().sgs_device_status_clear()
    if st != SGS_OK:
        raise SgsError(st, "sgs_device_status_clear")


def debug_expire_wait(limit_us: int, stream: int = 0):
    st = lib().sgs_debug_expire_wait(limit_us, ctypes.c_void_p(stream))
    if st != SGS_OK:
        raise SgsError(st, "sgs_debug_expire_wait")


def measure_fma_peak(stream: int = 0) -> float:
    v = ctypes.c_double()
    st = lib().sgs_measure_fma_peak(ctypes.addressof(v), ctypes.c_void_p(stream))
    if st != SGS_OK:
        raise SgsError(st, "sgs_measure_fma_peak")
    return v.value


def aux_op(descs: Sequence[AuxDesc], args: Sequence[AuxArgs], grouped: bool = False, stream: int = 0):
    """sgs_aux_op on len(descs) members (device addresses in ``args``)."""
    n = len(descs)
    d = (AuxDesc * n)(*descs)
    a = (AuxArgs * n)(*args)
    st = lib().sgs_aux_op(n, d, a, int(grouped), ctypes.c_void_p(stream))
    if st != SGS_OK:
        raise SgsError(st, "sgs_aux_op")


def device_status() -> int:
    return int(lib().sgs_device_status())


class SuperNet:
    """Owner of one loaded SuperNet handle."""

    def __init__(self, family: int, host_blob, dtype: int = SGS_BF16, device: int = 0, arch: Optional[ArchDesc] = None):
        self._h = ctypes.c_void_p()
        self.family, self.dtype, self.device = family, dtype, device
        a = arch if arch is not None else arch_desc(family)
        nbytes = host_blob.nbytes if hasattr(host_blob, "nbytes") else len(host_blob)
        st = lib().sgs_supernet_load(ctypes.byref(a), _addr(host_blob), nbytes, dtype, device, ctypes.byref(self._h))
        if st != SGS_OK:
            self._h = ctypes.c_void_p()
            raise SgsError(st, "sgs_supernet_load failed")
        self.n_classes = a.n_classes
        self.n_layers = lib().sgs_num_layers(self._h)

    def _check(self, st: int):
        if st != SGS_OK:
            raise SgsError(st, lib().sgs_last_error(self._h).decode())

    def close(self):
        if self._h:
            lib().sgs_supernet_free(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def subnet_validate(self, cfg: SubnetCfg) -> int:
        return lib().sgs_subnet_validate(self._h, ctypes.byref(cfg))

    def subnet_run(self, cfg: SubnetCfg, d_input: int, batch: int, res: int, d_logits: int, stream: int = 0):
        self._check(lib().sgs_subnet_run(self._h, ctypes.byref(cfg), d_input, batch, res, d_logits, stream))

    def stream_run(self, cfgs: Sequence[SubnetCfg], d_inputs, batch: int, res: int, d_logits,
                   opts: Optional[StreamOpts] = None, stream: int = 0, host: bool = False) -> StreamStats:
        arr = cfgs if isinstance(cfgs, ctypes.Array) else cfg_array(cfgs)
        stats = StreamStats()
        fn = lib().sgs_stream_run_host if host else lib().sgs_stream_run
        self._check(fn(self._h, len(arr), ctypes.addressof(arr), _addr(d_inputs), batch, res, _addr(d_logits),
                       ctypes.addressof(opts) if opts is not None else None, ctypes.addressof(stats), stream))
        return stats

    def cache_configure(self, enabled: bool, budget_bytes: int = 0, window_q: int = 4):
        self._check(lib().sgs_cache_configure(self._h, int(enabled), budget_bytes, window_q))

    def cache_set_candidates(self, cfgs: Sequence[SubnetCfg]):
        arr = cfgs if isinstance(cfgs, ctypes.Array) else (cfg_array(cfgs) if len(cfgs) else None)
        self._check(lib().sgs_cache_set_candidates(self._h, ctypes.addressof(arr) if arr is not None else None,
                                                   len(arr) if arr is not None else 0))

    def cache_set_policy(self, policy: int):
        self._check(lib().sgs_cache_set_policy(self._h, policy))

    def cache_stats(self) -> CacheStats:
        s = CacheStats()
        self._check(lib().sgs_cache_stats(self._h, ctypes.addressof(s)))
        return s

    def subnet_encode(self, cfg: SubnetCfg):
        import numpy as np
        out = np.zeros((self.n_layers, 3), dtype=np.int32)
        self._check(lib().sgs_subnet_encode(self._h, ctypes.byref(cfg), out.ctypes.data))
        return out

    def subnet_cost(self, cfg: SubnetCfg, batch: int, res: int):
        f, w, a = ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
        self._check(lib().sgs_subnet_cost(self._h, ctypes.byref(cfg), batch, res, ctypes.addressof(f), ctypes.addressof(w),
                                          ctypes.addressof(a)))
        return f.value, w.value, a.value

    def profile_trace(self):
        """Per-launch records of the profiled waves: list of dicts with the stored layer's name."""
        n = lib().sgs_profile_trace(self._h, None, 0)
        if n < 0:
            raise SgsError(SGS_EINVAL, "sgs_profile_trace")
        arr = (LaunchRecord * max(n, 1))()
        n = min(n, lib().sgs_profile_trace(self._h, ctypes.addressof(arr), n))
        out, buf = [], ctypes.create_string_buffer(128)
        for r in arr[:n]:
            name = buf.value.decode() if r.layer >= 0 and lib().sgs_layer_name(self._h, r.layer, buf, 128) >= 0 else ""
            out.append({"kernel_class": r.kernel_class, "layer": r.layer, "name": name, "members": r.members, "tiles": r.tiles,
                        "ms": r.ms, "alg_bytes": r.alg_bytes, "flops": r.flops})
        return out

    def profile_read(self, kernel_class: int):
        n, ms, b, f = ctypes.c_longlong(), ctypes.c_double(), ctypes.c_double(), ctypes.c_double()
        self._check(lib().sgs_profile_read(self._h, kernel_class, ctypes.addressof(n), ctypes.addressof(ms),
                                           ctypes.addressof(b), ctypes.addressof(f)))
        return {"launches": n.value, "total_ms": ms.value, "alg_bytes": b.value, "flops": f.value}

    def set_option(self, name: str, value: int):
        self._check(lib().sgs_set_option(self._h, name.encode(), value))

    def get_counter(self, name: str) -> int:
        return int(lib().sgs_get_counter(self._h, name.encode()))
