"""SubGraph-Stationary SubNet inference on B200: ctypes binding of the CUDA library plus the
seeded workload generators.  The CUDA library is loaded on first use, never at import."""
from . import workload  # noqa: F401
from .binding import (SGS_BF16, SGS_F32, SGS_POLICY_AVGNET, SGS_POLICY_INTERSECTION, SGS_STRICT_ACCURACY, SGS_STRICT_LATENCY, AuxArgs, AuxDesc, CacheStats, ConvDesc, ConvI8Desc, Scheduler, SgsError, StreamOpts, StreamStats, SuperNet,  # noqa: F401
                      aux_op, conv2d_sliced, conv2d_sliced_i8, conv2d_sliced_static, debug_expire_wait, device_status, device_status_clear, lib, measure_fma_peak)
