"""The allocation-free sliced convolution (sgs_conv2d_sliced_static) against sgs_conv2d_sliced.

Some callers of the library cannot allocate device memory when they call it: they own all device
memory through a pool of their own, or they cannot afford the device-wide synchronisation an
allocation implies.  For them the library offers a variant whose
split-reduction scratch is a fixed array inside the library image.  This file checks, through the C
interface, that the variant returns what the ordinary entry point returns (within the layer tests'
tolerance, 1e-2 * max|ref|), on two calls in a row, that free device memory does not change across
its calls, and that it refuses work beyond its fixed scratch.

Collected last on purpose (file name), so a run that stops at the first failure has already run every
other test.  It needs nothing from the other tests and passes in a fresh process as well.
"""
import numpy as np
import pytest
import torch

import paper_2306_17266_b200 as sgs
from tests.test_gpu_conv_layer import make_case

pytestmark = pytest.mark.gpu

# N, H, W, Cmax, C, Kmax, K, R, k, stride, act, residual
SPLIT_CASE = (1, 7, 7, 720, 720, 720, 720, 3, 3, 1, 1, True)    # reduction split over several CTAs: uses the scratch
PLAIN_CASE = (16, 14, 14, 360, 256, 1024, 824, 1, 1, 1, 1, True)  # fills the GPU unsplit: no scratch


def _desc(case):
    N, H, W, Cmax, C, Kmax, K, R, k, stride, act, _ = case
    return sgs.ConvDesc(N=N, H=H, W=W, C=C, K=K, Kmax=Kmax, Cmax=Cmax, R=R, k=k, stride=stride, act=act, dtype=sgs.SGS_BF16,
                        impl=2, depthwise=0, cache_k=0, cache_c=0, weight_policy=0, split_k_off=0)


@pytest.mark.parametrize("case", [SPLIT_CASE, PLAIN_CASE])
def test_static_variant_matches_the_allocating_entry_point_twice(case):
    ref, dev = make_case(*case, seed=11)
    desc = _desc(case)
    stream = torch.cuda.current_stream().cuda_stream
    args = (dev["x"].data_ptr(), dev["w"].data_ptr(), dev["scale"].data_ptr(), dev["shift"].data_ptr(),
            dev["res"].data_ptr() if dev["res"] is not None else 0)
    want = torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    sgs.conv2d_sliced(desc, *args, want.data_ptr(), stream)
    torch.cuda.synchronize()
    want = want.float().cpu().numpy()
    tol = 1e-2 * np.abs(ref).max()
    assert np.abs(want - ref).max() <= tol
    outs = [torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(3)]
    sgs.conv2d_sliced_static(desc, *args, outs[0].data_ptr(), stream)  # the first call on a device does the one-time set-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for i in (1, 2):  # the second call meets the array as the first one left it
        sgs.conv2d_sliced_static(desc, *args, outs[i].data_ptr(), stream)
        torch.cuda.synchronize()
        # no device memory was taken (the outputs were allocated before the measurement started)
        assert torch.cuda.mem_get_info()[0] == free_before
        got = outs[i].float().cpu().numpy()
        assert sgs.device_status() == 0  # also reads the status word that lives inside the fixed array
        assert np.all(np.isfinite(got))
        assert np.abs(got - want).max() <= tol
        assert np.abs(got - ref).max() <= tol


def test_static_variant_rejects_what_it_cannot_hold():
    # 128 pixels x 9216 filters split three ways: 13.5 MiB of fp32 partial sums, more than the fixed
    # 8 MiB: refused, nothing launched
    big = (2, 8, 8, 128, 128, 9216, 9216, 3, 3, 1, 0, False)
    N, H, W, Cmax, C, Kmax, K, R, k, stride, act, _ = big
    x = torch.zeros((N, H, W, C), dtype=torch.bfloat16, device="cuda")
    w = torch.zeros((Kmax, R, R, Cmax), dtype=torch.bfloat16, device="cuda")
    sc = torch.ones(Kmax, device="cuda")
    sh = torch.zeros(Kmax, device="cuda")
    y = torch.full((N, H, W, K), 7.0, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(sgs.SgsError) as e:
        sgs.conv2d_sliced_static(_desc(big), x.data_ptr(), w.data_ptr(), sc.data_ptr(), sh.data_ptr(), 0, y.data_ptr())
    assert e.value.status == sgs.binding.SGS_ENOMEM
    torch.cuda.synchronize()
    assert float(y.float().min()) == 7.0  # untouched
    # other refusals: fp32 and depthwise have no tensor-core path
    d = _desc(SPLIT_CASE)
    d.dtype = sgs.SGS_F32
    with pytest.raises(sgs.SgsError) as e:
        sgs.conv2d_sliced_static(d, x.data_ptr(), w.data_ptr(), sc.data_ptr(), sh.data_ptr(), 0, y.data_ptr())
    assert e.value.status == sgs.binding.SGS_EUNSUPPORTED
    d = _desc(SPLIT_CASE)
    d.impl = 7
    with pytest.raises(sgs.SgsError) as e:
        sgs.conv2d_sliced_static(d, x.data_ptr(), w.data_ptr(), sc.data_ptr(), sh.data_ptr(), 0, y.data_ptr())
    assert e.value.status == sgs.binding.SGS_EINVAL
