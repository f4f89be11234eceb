"""The paper's 8-bit format through a whole SubNet trunk: every bottleneck block of a ResNet-shaped SubNet (projection
shortcut, 1x1, 3x3 with the stage's stride, 1x1 + residual + ReLU) as a chain of sgs_conv2d_sliced_i8 calls on padded
pixels, against the same chain of the CPU checker's exact integer layer.  Integer work: bit exact, layer after layer.

The 8-bit SuperNet is synthetic: seeded int8 weights in the stored shapes of the family, per-filter multipliers from the
layer's shape alone (no data-dependent calibration: the paper gives no rule), post-ReLU tensors unsigned with zero point
0, shortcuts signed.  The slices come from the checker's encoding of the config, so slicing by prefix is exercised on
every layer.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl

pytestmark = pytest.mark.gpu

STAGE_STRIDE = (1, 2, 2, 2)   # of the ResNet-shaped family
RES_MULT, RES_SHIFT = 1 << 30, 0   # shortcut x 0.5


def layer_params(rec, seed):
    """int8 weights [K][C][R][R] and per-filter requantisation (mult, shift, bias) of one stored layer."""
    rng = np.random.default_rng(seed)
    w = rng.integers(-127, 128, (rec.K, rec.C, rec.R, rec.S)).astype(np.int8)
    n = 0.8 * rec.C * rec.R * rec.S                     # terms of a typical slice
    real = 40.0 / (73.0 * 60.0 * np.sqrt(n)) * rng.uniform(0.8, 1.2, rec.K)
    shift = np.clip(np.floor(-np.log2(real)).astype(np.int64), 0, 31)
    mult = np.minimum(np.round(real * 2.0 ** (31 + shift)), 2 ** 31 - 1).astype(np.int32)
    bias = rng.integers(-20, 21, rec.K).astype(np.int32)
    return w, mult, shift.astype(np.int32), bias


def pad16(a):
    """NHWC bytes -> pixels of a 16-byte multiple, zeros beyond the channels."""
    c = a.shape[-1]
    ld = (c + 15) // 16 * 16
    out = np.zeros(a.shape[:-1] + (ld,), dtype=a.dtype)
    out[..., :c] = a
    return out


class GpuLayer:
    """One stored layer on the device ([K][R][R][Cp16] int8 + int32 vectors) and its call through the C ABI."""

    def __init__(self, rec, params):
        w, mult, shift, bias = params
        self.rec = rec
        self.Cp = (rec.C + 15) // 16 * 16
        wp = np.zeros((rec.K, rec.R, rec.S, self.Cp), dtype=np.int8)
        wp[..., :rec.C] = w.transpose(0, 2, 3, 1)
        self.w = torch.from_numpy(wp).cuda()
        self.mult, self.shift, self.bias = (torch.from_numpy(a).cuda() for a in (mult, shift, bias))

    def run(self, x, C, K, k, stride, relu, y_signed, res=None, res_signed=False):
        # x: [N][H][W][ld] device bytes with zeros beyond C; returns [N][Ho][Wo][ldy]
        N, H, W, ldx = x.shape
        p = (k - 1) // 2
        Ho, Wo = (H + 2 * p - k) // stride + 1, (W + 2 * p - k) // stride + 1
        ldy = (K + 15) // 16 * 16
        y = torch.full((N, Ho, Wo, ldy), 55, dtype=torch.int8 if y_signed else torch.uint8, device="cuda")
        d = sgs.ConvI8Desc(N=N, H=H, W=W, C=C, K=K, Kmax=self.rec.K, Cmax=self.Cp, R=self.rec.R, k=k, stride=stride, relu=int(relu),
                           x_signed=int(x.dtype == torch.int8), y_signed=int(y_signed), res_signed=int(res_signed), zx=0, zy=0, zr=0,
                           res_mult=RES_MULT, res_shift=RES_SHIFT, ldx=ldx, ldy=ldy)
        sgs.conv2d_sliced_i8(d, x.data_ptr(), self.w.data_ptr(), self.mult.data_ptr(), self.shift.data_ptr(), self.bias.data_ptr(),
                             res.data_ptr() if res is not None else 0, y.data_ptr(), torch.cuda.current_stream().cuda_stream)
        return y


@pytest.mark.parametrize("which,res_in,batch", [("uniform", 16, 2), ("smallest", 24, 1), ("largest", 16, 1)])
def test_int8_trunk_of_a_subnet_is_bit_exact(which, res_in, batch):
    # res_in: size of the trunk's input map (the tensor after the stem's pool; 56 for a 224x224 image)
    fam = wl.RESNET
    cfg = wl.uniform_stream(fam, 3, seed=17)[2] if which == "uniform" else wl.extreme_cfg(fam, which == "largest")
    recs = wl.supernet_records(fam)
    idx = {r.name: i for i, r in enumerate(recs)}
    enc = oracle.Net(fam, wl.make_blob(fam, seed=0)).encode(cfg)      # (K, C, k) per stored layer
    params = {r.name: layer_params(r, 1000 + i) for i, r in enumerate(recs) if r.kind == wl.KIND_CONV and r.name != "stem"}
    gpu = {name: GpuLayer(recs[idx[name]], p) for name, p in params.items()}
    C0 = int(enc[idx["stem"]][0])
    rng = np.random.default_rng(5)
    x_ref = rng.integers(0, 120, (batch, res_in, res_in, C0)).astype(np.uint8)
    x_gpu = torch.from_numpy(pad16(x_ref)).cuda()

    def both(name, xr, xg, stride, relu, y_signed, res_r=None, res_g=None):
        K, C, k = (int(v) for v in enc[idx[name]])
        assert K > 0 and C == xr.shape[-1]
        w, mult, shift, bias = params[name]
        yr = oracle.layer_conv_i8(w, xr, C, K, k, stride, mult, shift, bias, zx=0, zy=0, relu=relu, res=res_r, zr=0,
                                  res_mult=RES_MULT, res_shift=RES_SHIFT, y_signed=y_signed)
        yg = gpu[name].run(xg, C, K, k, stride, relu, y_signed, res_g, res_g is not None and res_g.dtype == torch.int8)
        got = yg.cpu().numpy()
        np.testing.assert_array_equal(got[..., :K], yr, err_msg=name)
        assert not got[..., K:].any(), name
        return yr, yg

    layers = 0
    for s in range(4):
        for b in range(int(cfg.depth[s])):
            st = STAGE_STRIDE[s] if b == 0 else 1
            sc_r, sc_g = x_ref, x_gpu
            if b == 0:
                sc_r, sc_g = both(f"s{s}b{b}.proj", x_ref, x_gpu, st, False, True)
                layers += 1
            t1r, t1g = both(f"s{s}b{b}.conv1", x_ref, x_gpu, 1, True, False)
            t2r, t2g = both(f"s{s}b{b}.conv2", t1r, t1g, st, True, False)
            x_ref, x_gpu = both(f"s{s}b{b}.conv3", t2r, t2g, 1, True, False, sc_r, sc_g)
            layers += 3
            assert 0.05 < np.mean((x_ref > 0) & (x_ref < 255)), "the chain must not saturate away"
    torch.cuda.synchronize()
    assert sgs.device_status() == 0 and layers >= 28
