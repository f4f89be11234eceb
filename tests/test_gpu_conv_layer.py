"""Layer-level GPU parity of the sliced convolution (tensor-core and CUDA-core kernels) against the
CPU checker's single-layer functions, through the C entry point sgs_conv2d_sliced.

Tolerance (bf16 operands, fp32 accumulation, bf16 store): max|err| <= 1e-2 * max|ref| over the
tensor; the only differences are the fp32 summation order and the folded batch norm, i.e. at most a
bf16 rounding flip (2^-8 relative) on top of ~1e-6 accumulation noise.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl

pytestmark = pytest.mark.gpu


def make_case(N, H, W, Cmax, C, Kmax, K, R, k, stride, act, use_res, seed=0, depthwise=False):
    """Seeded layer inputs, the checker's result, and the device tensors in the library's layouts."""
    rng = np.random.default_rng(seed)
    cin = K if depthwise else C
    x = wl.round_to_bf16(rng.standard_normal((N, H, W, cin)).astype(np.float32))
    fan = (1 if depthwise else cin) * k * k
    w = wl.round_to_bf16((rng.standard_normal((Kmax, 1 if depthwise else Cmax, R, R)) * np.sqrt(2.0 / fan)).astype(np.float32))
    gamma = rng.uniform(0.5, 1.5, Kmax).astype(np.float32)
    beta = (rng.standard_normal(Kmax) * 0.1).astype(np.float32)
    mean = (rng.standard_normal(Kmax) * 0.1).astype(np.float32)
    var = rng.uniform(0.5, 1.5, Kmax).astype(np.float32)
    y = oracle.layer_conv(w, x, C, K, k, stride, depthwise=depthwise)
    res = wl.round_to_bf16(rng.standard_normal(y.shape).astype(np.float32)) if use_res else None
    ref = oracle.layer_epilogue(y, gamma[:K], beta[:K], mean[:K], var[:K], None, res, act, oracle.BF16_STORE)
    scale = gamma / np.sqrt(var + np.float32(1e-5))
    shift = beta - mean * scale
    dev = {"x": torch.from_numpy(x).cuda().to(torch.bfloat16)}
    if depthwise:
        dev["w"] = torch.from_numpy(np.ascontiguousarray(w[:, 0].transpose(1, 2, 0))).cuda().to(torch.bfloat16)  # [R][R][Kmax]
    else:
        dev["w"] = torch.from_numpy(np.ascontiguousarray(w.transpose(0, 2, 3, 1))).cuda().to(torch.bfloat16)  # [Kmax][R][R][Cmax]
    dev["scale"], dev["shift"] = torch.from_numpy(scale).cuda(), torch.from_numpy(shift).cuda()
    dev["res"] = torch.from_numpy(res).cuda().to(torch.bfloat16) if use_res else None
    return ref, dev


def run_case(N, H, W, Cmax, C, Kmax, K, R, k, stride, act, use_res, impl, seed=0, split_off=0, depthwise=False, policy=0):
    ref, dev = make_case(N, H, W, Cmax, C, Kmax, K, R, k, stride, act, use_res, seed, depthwise)
    dy = torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    desc = sgs.ConvDesc(N=N, H=H, W=W, C=C, K=K, Kmax=Kmax, Cmax=Cmax, R=R, k=k, stride=stride, act=act, dtype=sgs.SGS_BF16,
                        impl=impl, depthwise=int(depthwise), cache_k=K // 2, cache_c=C // 2, weight_policy=policy,
                        split_k_off=split_off)
    outs = []
    for _ in range(2):  # twice: the split-K counters must come back clean, and the result must repeat
        sgs.conv2d_sliced(desc, dev["x"].data_ptr(), dev["w"].data_ptr(), dev["scale"].data_ptr(), dev["shift"].data_ptr(),
                          dev["res"].data_ptr() if use_res else 0, dy.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        got = dy.float().cpu().numpy()
        assert sgs.device_status() == 0
        assert np.all(np.isfinite(got))
        err = np.abs(got - ref).max()
        assert err <= 1e-2 * max(np.abs(ref).max(), 1e-6), (err, np.abs(ref).max())
        outs.append(got)
    np.testing.assert_array_equal(outs[0], outs[1])


CASES = [
    # N, H, W, Cmax, C, Kmax, K, R, k, stride, act, res
    (1, 56, 56, 64, 64, 88, 72, 1, 1, 1, 1, False),       # 1x1, flat M = 3136 (24.5 tiles), K tail
    (2, 28, 28, 512, 336, 176, 104, 1, 1, 1, 0, True),    # channel chunks 5.25, residual
    (1, 7, 7, 720, 464, 2048, 1328, 1, 1, 1, 1, True),    # small M, many filters
    (3, 56, 56, 88, 56, 88, 56, 3, 3, 1, 1, False),       # 3x3 stride 1, C and K below one chunk
    (1, 28, 28, 176, 176, 176, 128, 3, 3, 1, 2, False),   # h-swish
    (2, 14, 14, 360, 208, 360, 256, 3, 3, 1, 1, False),
    (1, 7, 7, 720, 720, 720, 720, 3, 3, 1, 1, False),     # split K
    (5, 9, 9, 64, 40, 64, 48, 3, 3, 1, 0, True),          # odd sizes, ragged boxes over batch
    (1, 56, 56, 88, 88, 88, 64, 3, 3, 2, 1, False),       # 3x3 stride 2 (parity views)
    (2, 28, 28, 176, 104, 176, 168, 3, 3, 2, 1, False),
    (1, 56, 56, 256, 168, 512, 408, 1, 1, 2, 0, False),   # 1x1 stride 2 projection
    (3, 14, 14, 1024, 664, 2048, 1640, 1, 1, 2, 0, False),
    (1, 20, 20, 64, 64, 64, 64, 7, 5, 1, 1, False),       # centre 5x5 window of a stored 7x7 kernel
    (1, 16, 16, 24, 16, 32, 24, 7, 7, 2, 1, True),        # 7x7 stride 2
    (16, 14, 14, 360, 256, 1024, 824, 1, 1, 1, 1, True),  # batch 16
]


@pytest.mark.parametrize("case", CASES)
def test_tensor_core_conv(case):
    run_case(*case, impl=2, seed=1)


@pytest.mark.parametrize("case", [CASES[1], CASES[6], CASES[8], CASES[12]])
def test_tensor_core_conv_without_split_and_with_cache_hints(case):
    run_case(*case, impl=2, seed=2, split_off=1, policy=1)
    run_case(*case, impl=2, seed=3, split_off=0, policy=2)


@pytest.mark.parametrize("case", [CASES[0], CASES[3], CASES[8], CASES[10], CASES[13]])
def test_cuda_core_conv(case):
    run_case(*case, impl=1, seed=4)


def test_shapes_the_tensor_core_kernel_refuses():
    # 12 channels: rows of 24 bytes cannot be a TMA stride; impl 2 must say so, impl 0 must fall back
    with pytest.raises(sgs.SgsError) as e:
        run_case(1, 8, 8, 16, 12, 16, 12, 3, 3, 1, 1, False, impl=2)
    assert e.value.status == sgs.binding.SGS_EUNSUPPORTED
    run_case(1, 8, 8, 16, 12, 16, 12, 3, 3, 1, 1, False, impl=0)
    run_case(1, 9, 9, 16, 16, 16, 16, 3, 3, 2, 1, False, impl=0)  # odd input, stride 2 -> falls back


@pytest.mark.parametrize("k,stride", [(3, 1), (5, 1), (7, 1), (3, 2), (5, 2), (7, 2)])
def test_depthwise(k, stride):
    run_case(2, 28, 28, 1, 1, 144, 120, 7, k, stride, 2, False, impl=0, seed=5, depthwise=True)
    run_case(1, 15, 13, 1, 1, 96, 72, 7, k, stride, 1, False, impl=0, seed=6, depthwise=True)


@pytest.mark.parametrize("k", [3, 5, 7])
def test_depthwise_walking_kernel(k):
    # stride-1 launches of 48 M outputs and more walk down the image behind a shared-memory ring of input rows; the
    # library option makes every stride-1 shape take that kernel: ragged column tiles, maps shorter than the ring, more
    # rows than a 56-row segment (two segments with their halo rows), channel counts off the 128-channel block
    from tests import gpu_util as gu
    from paper_2306_17266_b200 import workload as wl
    _, _, net = gu.nets(wl.TINY, True)
    net.set_option("dw_walk", -1)
    try:
        run_case(2, 28, 28, 1, 1, 144, 120, 7, k, 1, 2, False, impl=0, seed=5, depthwise=True)
        run_case(1, 15, 13, 1, 1, 96, 72, 7, k, 1, 1, False, impl=0, seed=6, depthwise=True)
        run_case(1, 61, 37, 1, 1, 264, 264, 7, k, 1, 0, False, impl=0, seed=7, depthwise=True)
        run_case(1, 4, 5, 1, 1, 16, 8, 7, k, 1, 2, False, impl=0, seed=8, depthwise=True)
    finally:
        net.set_option("dw_walk", 48)
