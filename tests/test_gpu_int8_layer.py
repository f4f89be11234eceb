"""GPU parity of the 8-bit sliced convolution layer (sgs_conv2d_sliced_i8: the paper's numeric format on the 8-bit
tensor cores) against the CPU checker's exact integer layer.  Integer work: the comparison is bit exact."""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_17266_b200 as sgs

pytestmark = pytest.mark.gpu

# N, H, W, Cmax, C, Kmax, K, R, k, stride, x_signed, relu, y_signed, residual
CASES = [
    (1, 56, 56, 64, 64, 96, 72, 1, 1, 1, False, True, False, False),      # 1x1, K tail inside a 128-filter tile
    (2, 28, 28, 512, 336, 176, 104, 1, 1, 1, False, False, True, True),   # 2.6 channel chunks of 128, residual, signed output
    (1, 7, 7, 720, 464, 2048, 1328, 1, 1, 1, False, True, False, True),   # small M, many filter tiles
    (3, 56, 56, 96, 48, 96, 56, 3, 3, 1, False, True, False, False),      # 3x3, less than one chunk
    (2, 14, 14, 368, 208, 360, 256, 3, 3, 1, True, True, False, False),   # signed activations (symmetric, zero point 0)
    (5, 9, 9, 64, 48, 64, 48, 3, 3, 1, False, False, False, True),        # odd sizes, ragged boxes over the batch
    (1, 56, 56, 96, 80, 96, 64, 3, 3, 2, False, True, False, False),      # stride 2 (parity views)
    (1, 20, 20, 64, 64, 64, 64, 7, 5, 1, False, True, False, False),      # centre 5x5 window of a stored 7x7 kernel
    (16, 14, 14, 368, 256, 1024, 824, 1, 1, 1, False, True, False, True), # batch 16
]


def make(case, seed):
    N, H, W, Cmax, C, Kmax, K, R, k, stride, x_signed, relu, y_signed, use_res = case
    rng = np.random.default_rng(seed)
    w = rng.integers(-127, 128, (Kmax, Cmax, R, R)).astype(np.int8)
    x = (rng.integers(-128, 128, (N, H, W, C)).astype(np.int8) if x_signed else rng.integers(0, 256, (N, H, W, C)).astype(np.uint8))
    # multipliers that bring the accumulator (up to ~ 255 * 127 * C * k * k / 3) into the byte range
    scale = 96.0 / (128 * 64 * np.sqrt(C * k * k))
    real = scale * rng.uniform(0.5, 1.5, Kmax)
    shift = np.clip(np.floor(-np.log2(real)).astype(np.int64), 0, 31)
    mult = np.minimum(np.round(real * 2.0 ** (31 + shift)), 2 ** 31 - 1).astype(np.int32)
    bias = rng.integers(-30, 30, Kmax).astype(np.int32)
    p = (k - 1) // 2
    Ho, Wo = (H + 2 * p - k) // stride + 1, (W + 2 * p - k) // stride + 1
    res = rng.integers(0, 256, (N, Ho, Wo, K)).astype(np.uint8) if use_res else None
    zy = -3 if y_signed else 7
    kw = dict(zx=0, zy=zy, relu=relu, res=res, zr=11, res_mult=1932735283, res_shift=1, y_signed=y_signed)  # residual x 0.45
    ref = oracle.layer_conv_i8(w, x, C, K, k, stride, mult, shift.astype(np.int32), bias, **kw)
    return w, x, mult, shift.astype(np.int32), bias, res, zy, ref


@pytest.mark.parametrize("case", CASES)
def test_int8_layer_is_bit_exact(case):
    N, H, W, Cmax, C, Kmax, K, R, k, stride, x_signed, relu, y_signed, use_res = case
    w, x, mult, shift, bias, res, zy, ref = make(case, seed=3)
    assert 0.02 < np.mean((ref != ref.min()) & (ref != ref.max())) , "the case must not be all saturated"
    dw = torch.from_numpy(np.ascontiguousarray(w.transpose(0, 2, 3, 1))).cuda()   # [Kmax][R][R][Cmax]
    dx = torch.from_numpy(x).cuda()
    dm, ds, db = (torch.from_numpy(a).cuda() for a in (mult, shift, bias))
    dr = torch.from_numpy(res).cuda() if use_res else None
    dy = torch.full(ref.shape, 77, dtype=torch.int8 if y_signed else torch.uint8, device="cuda")
    desc = sgs.ConvI8Desc(N=N, H=H, W=W, C=C, K=K, Kmax=Kmax, Cmax=Cmax, R=R, k=k, stride=stride, relu=int(relu), x_signed=int(x_signed),
                          y_signed=int(y_signed), res_signed=0, zx=0, zy=zy, zr=11, res_mult=1932735283, res_shift=1)
    for _ in range(2):
        sgs.conv2d_sliced_i8(desc, dx.data_ptr(), dw.data_ptr(), dm.data_ptr(), ds.data_ptr(), db.data_ptr(), dr.data_ptr() if use_res else 0,
                             dy.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        assert sgs.device_status() == 0
        np.testing.assert_array_equal(dy.cpu().numpy(), ref)


# N, H, W, Cmax, C, Kmax, K, R, k, stride, x_signed, relu, y_signed, residual: channel counts that are multiples of 8 only
PADDED_CASES = [
    (2, 28, 28, 96, 72, 128, 88, 1, 1, 1, False, True, False, True),      # 72 -> 80 bytes per input pixel, 88 -> 96 per output pixel
    (1, 14, 14, 368, 328, 368, 328, 3, 3, 1, False, True, False, False),  # 3x3 over padded pixels, last chunk ragged
    (3, 56, 56, 64, 56, 256, 168, 1, 1, 2, False, False, True, True),     # strided 1x1 (projection shortcut), signed output
    (1, 30, 30, 32, 24, 64, 40, 3, 3, 2, False, True, False, False),      # stride-2 3x3, 24 -> 32 bytes, K = 40 -> 48
]


@pytest.mark.parametrize("case", PADDED_CASES)
def test_int8_layer_on_padded_pixels_is_bit_exact(case):
    # Pixels of 16-byte multiples with zeros beyond the slice (what a network of such layers keeps between them): the
    # layer reads x at pitch ldx, writes y at pitch ldy with zeros in the padding, reads the residual at pitch ldy.
    N, H, W, Cmax, C, Kmax, K, R, k, stride, x_signed, relu, y_signed, use_res = case
    w, x, mult, shift, bias, res, zy, ref = make(case, seed=5)
    ldx, ldy = (C + 15) // 16 * 16, (K + 15) // 16 * 16
    xp = np.zeros(x.shape[:3] + (ldx,), dtype=x.dtype); xp[..., :C] = x
    rp = None
    if use_res:
        rp = np.zeros(res.shape[:3] + (ldy,), dtype=res.dtype); rp[..., :K] = res
    dw = torch.from_numpy(np.ascontiguousarray(w.transpose(0, 2, 3, 1))).cuda()
    dx = torch.from_numpy(xp).cuda()
    dm, ds, db = (torch.from_numpy(a).cuda() for a in (mult, shift, bias))
    dr = torch.from_numpy(rp).cuda() if use_res else None
    dy = torch.full(ref.shape[:3] + (ldy,), 77, dtype=torch.int8 if y_signed else torch.uint8, device="cuda")
    desc = sgs.ConvI8Desc(N=N, H=H, W=W, C=C, K=K, Kmax=Kmax, Cmax=Cmax, R=R, k=k, stride=stride, relu=int(relu), x_signed=int(x_signed),
                          y_signed=int(y_signed), res_signed=0, zx=0, zy=zy, zr=11, res_mult=1932735283, res_shift=1, ldx=ldx, ldy=ldy)
    sgs.conv2d_sliced_i8(desc, dx.data_ptr(), dw.data_ptr(), dm.data_ptr(), ds.data_ptr(), db.data_ptr(), dr.data_ptr() if use_res else 0,
                         dy.data_ptr(), torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    assert sgs.device_status() == 0
    got = dy.cpu().numpy()
    np.testing.assert_array_equal(got[..., :K], ref)
    assert not got[..., K:].any()


def test_int8_layer_refuses_what_it_does_not_take():
    x = torch.zeros((1, 8, 8, 16), dtype=torch.uint8, device="cuda")
    w = torch.zeros((16, 3, 3, 16), dtype=torch.int8, device="cuda")
    v = torch.zeros(16, dtype=torch.int32, device="cuda")
    y = torch.zeros((1, 8, 8, 16), dtype=torch.uint8, device="cuda")
    d = sgs.ConvI8Desc(N=1, H=8, W=8, C=16, K=16, Kmax=16, Cmax=16, R=3, k=3, stride=1, zx=4)   # input zero point
    with pytest.raises(sgs.SgsError) as e:
        sgs.conv2d_sliced_i8(d, x.data_ptr(), w.data_ptr(), v.data_ptr(), v.data_ptr(), v.data_ptr(), 0, y.data_ptr())
    assert e.value.status == sgs.binding.SGS_EUNSUPPORTED
    d = sgs.ConvI8Desc(N=1, H=8, W=8, C=8, K=16, Kmax=16, Cmax=16, R=3, k=3, stride=1)          # 8 channels: 8-byte rows
    with pytest.raises(sgs.SgsError) as e:
        sgs.conv2d_sliced_i8(d, x.data_ptr(), w.data_ptr(), v.data_ptr(), v.data_ptr(), v.data_ptr(), 0, y.data_ptr())
    assert e.value.status == sgs.binding.SGS_EUNSUPPORTED
