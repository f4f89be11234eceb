"""CPU-side checks of the C interface: the library loads and exports what include/sgs.h declares."""
import ctypes
import os
import re

import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl
from paper_2306_17266_b200.binding import EXPORTS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "sgs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sgs_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = sgs.lib()
    names = declared_functions()
    assert len(names) >= 17
    for n in names:
        assert hasattr(L, n), n
    assert sorted(EXPORTS) == names


def test_struct_sizes_match_the_header():
    # sizes implied by the header's field lists (LP64)
    assert ctypes.sizeof(wl.SubnetCfg) == 4 * (8 + 9 + 64 + 64)
    assert ctypes.sizeof(wl.ArchDesc) == 4 * (2 + 8 + 8 + 3)
    assert ctypes.sizeof(sgs.StreamOpts) == 48  # 2 ints, size_t, 7 ints (padded to 8 bytes)
    assert ctypes.sizeof(sgs.StreamStats) == 8 + 11 * 8 + 8 + 16
    assert ctypes.sizeof(sgs.ConvDesc) == 18 * 4
    assert ctypes.sizeof(sgs.CacheStats) == 8 + 7 * 8 + 4 * 4


def test_null_arguments_are_rejected_without_a_gpu():
    L = sgs.lib()
    assert L.sgs_supernet_load(None, None, 0, 1, 0, None) == sgs.binding.SGS_EINVAL
    assert L.sgs_subnet_validate(None, None) == sgs.binding.SGS_EINVAL
    assert L.sgs_num_layers(None) == 0
    assert L.sgs_last_error(None) == b"null handle"
    assert L.sgs_conv2d_sliced(None, None, None, None, None, None, None, None) == sgs.binding.SGS_EINVAL
