"""Layer-level GPU parity of the layers that are not convolutions (max pool, global average pool, sliced fully
connected layer, squeeze-excite gate and scale) against the CPU checker's single-layer functions, through the C
entry point sgs_aux_op: the kernel a single query uses (grouped = 0) and the kernel a wave uses (grouped = 1), on odd
map sizes, ragged member mixes and channel counts at and off the kernels' 8-element vector width.

Tolerances: max pool is exact (a maximum of bf16 values); sums are fp32 in a different order than the checker's
(<= 2e-5 relative to the largest value); SE scale rounds one product to bf16 (one flip of 2^-8 relative at most).
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl
from paper_2306_17266_b200.binding import (SGS_AUX_AVGPOOL, SGS_AUX_LINEAR, SGS_AUX_MAXPOOL, SGS_AUX_SE_GATE, SGS_AUX_SE_SCALE,
                                           SGS_EUNSUPPORTED)

pytestmark = pytest.mark.gpu


def dev(a, bf16):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16).contiguous() if bf16 else t.contiguous()


def run(descs, args, grouped):
    sgs.aux_op(descs, args, grouped, torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()


# member shapes: (N, H, W, C)
MAPS_VEC = [(1, 7, 7, 64), (3, 9, 5, 8), (2, 14, 14, 168), (1, 1, 1, 24), (16, 7, 7, 2048)]
MAPS_ODD = [(2, 9, 5, 12), (1, 7, 7, 20), (1, 3, 3, 3)]


@pytest.mark.parametrize("bf16", [True, False])
@pytest.mark.parametrize("kind", [SGS_AUX_MAXPOOL, SGS_AUX_AVGPOOL, SGS_AUX_SE_SCALE])
def test_pools_and_se_scale(kind, bf16):
    rng = np.random.default_rng(10 + kind)
    dt = sgs.SGS_BF16 if bf16 else sgs.SGS_F32
    for grouped in (False, True):
        shapes = MAPS_VEC if grouped else MAPS_VEC + MAPS_ODD
        if grouped and not bf16:
            continue
        keep, descs, args, refs, outs = [], [], [], [], []
        for (N, H, W, C) in shapes:
            x = rng.standard_normal((N, H, W, C)).astype(np.float32)
            x = wl.round_to_bf16(x) if bf16 else x
            dx = dev(x, bf16)
            if kind == SGS_AUX_MAXPOOL:
                ref = oracle.layer_maxpool(x)
                dy = torch.full(ref.shape, float("nan"), dtype=dx.dtype, device="cuda")
                a = sgs.AuxArgs(x=dx.data_ptr(), y=dy.data_ptr())
            elif kind == SGS_AUX_AVGPOOL:
                ref = oracle.layer_gap(x)
                dy = torch.full(ref.shape, float("nan"), dtype=torch.float32, device="cuda")
                a = sgs.AuxArgs(x=dx.data_ptr(), y=dy.data_ptr())
            else:
                gate = rng.uniform(0, 1, (N, C)).astype(np.float32)
                ref = oracle.layer_se_scale(x, gate, oracle.BF16_STORE if bf16 else oracle.FP32)
                dg = dev(gate, False)
                dy = torch.full(ref.shape, float("nan"), dtype=dx.dtype, device="cuda")
                a = sgs.AuxArgs(x=dx.data_ptr(), y=dy.data_ptr(), w=dg.data_ptr())
                keep.append(dg)
            keep.append(dx)
            descs.append(sgs.AuxDesc(kind=kind, dtype=dt, N=N, H=H, W=W, C=C))
            args.append(a); refs.append(ref); outs.append(dy)
        run(descs, args, grouped)
        for shape, ref, dy in zip(shapes, refs, outs):
            got = dy.float().cpu().numpy()
            if kind == SGS_AUX_MAXPOOL:
                np.testing.assert_array_equal(got, ref, err_msg=str(shape))
            else:
                tol = 2e-5 if kind == SGS_AUX_AVGPOOL or not bf16 else 2.0 ** -8
                assert np.abs(got - ref).max() <= tol * max(np.abs(ref).max(), 1e-6), (shape, grouped)


# (N, C inputs, K outputs, stored row pitch, activation)
LINEAR_VEC = [(1, 2048, 1000, 2048, 0), (3, 1328, 1000, 2048, 0), (2, 960, 1280, 960, 2), (4, 24, 8, 40, 1)]
LINEAR_ODD = [(2, 12, 10, 20, 0), (1, 64, 10, 64, 1), (3, 20, 7, 36, 2)]


@pytest.mark.parametrize("bf16", [True, False])
def test_sliced_linear(bf16):
    rng = np.random.default_rng(3)
    dt = sgs.SGS_BF16 if bf16 else sgs.SGS_F32
    for grouped, shared in ((False, False), (True, False), (True, True)):
        if grouped and not bf16:
            continue
        # shared: every member slices the SAME stored layer with the same (N, K) -> the kernel that loads a weight row
        # once for several members
        shapes = [(2, c, 1000, 2048, 0) for c in (1328, 1640, 2048, 1328, 1640, 1328, 2048, 1328, 1640)] if shared else \
            (LINEAR_VEC if grouped else LINEAR_VEC + LINEAR_ODD)
        w_shared = rng.standard_normal((1000, 2048)).astype(np.float32) * 0.05
        w_shared = wl.round_to_bf16(w_shared) if bf16 else w_shared
        b_shared = rng.standard_normal(1000).astype(np.float32)
        dws, dbs = dev(w_shared, bf16), dev(b_shared, False)
        keep, descs, args, refs, outs = [], [], [], [], []
        for (N, C, K, ld, act) in shapes:
            v = rng.standard_normal((N, C)).astype(np.float32)
            if shared:
                w, b, dw, db = w_shared, b_shared, dws, dbs
            else:
                w = rng.standard_normal((K + 3, ld)).astype(np.float32) * 0.05
                w = wl.round_to_bf16(w) if bf16 else w
                b = rng.standard_normal(K + 3).astype(np.float32)
                dw, db = dev(w, bf16), dev(b, False)
            dv = dev(v, False)
            dy = torch.full((N, K), float("nan"), dtype=torch.float32, device="cuda")
            keep += [dw, db, dv]
            descs.append(sgs.AuxDesc(kind=SGS_AUX_LINEAR, dtype=dt, N=N, H=1, W=1, C=C, K=K, ld=ld, act=act))
            args.append(sgs.AuxArgs(x=dv.data_ptr(), y=dy.data_ptr(), w=dw.data_ptr(), bias=db.data_ptr()))
            refs.append(oracle.layer_linear(w, b, v, C, K, act)); outs.append(dy)
        run(descs, args, grouped)
        for shape, ref, dy in zip(shapes, refs, outs):
            got = dy.cpu().numpy()
            assert np.abs(got - ref).max() <= 2e-5 * max(np.abs(ref).max(), 1.0), (shape, grouped, shared)


# (N, mid, squeeze)
SE_CASES = [(1, 72, 16), (2, 240, 64), (3, 960, 240), (1, 120, 32), (16, 480, 120), (2, 24, 8)]


@pytest.mark.parametrize("bf16", [True, False])
def test_squeeze_excite_gate(bf16):
    rng = np.random.default_rng(4)
    dt = sgs.SGS_BF16 if bf16 else sgs.SGS_F32
    for grouped in (False, True):
        if grouped and not bf16:
            continue
        keep, descs, args, refs, outs = [], [], [], [], []
        for (N, mid, sq) in SE_CASES:
            mid_max, sq_max = mid + 24, sq + 8                      # stored layers are larger than the slice
            w1 = rng.standard_normal((sq_max, mid_max)).astype(np.float32) * 0.1
            w2 = rng.standard_normal((mid_max, sq_max)).astype(np.float32) * 0.2
            w1, w2 = (wl.round_to_bf16(w1), wl.round_to_bf16(w2)) if bf16 else (w1, w2)
            b1, b2 = rng.standard_normal(sq_max).astype(np.float32) * 0.1, rng.standard_normal(mid_max).astype(np.float32)
            g = rng.standard_normal((N, mid)).astype(np.float32)
            t = [dev(w1, bf16), dev(b1, False), dev(w2, bf16), dev(b2, False), dev(g, False)]
            dy = torch.full((N, mid), float("nan"), dtype=torch.float32, device="cuda")
            keep += t
            descs.append(sgs.AuxDesc(kind=SGS_AUX_SE_GATE, dtype=dt, N=N, H=1, W=1, C=mid, K=sq, ld=mid_max, ld2=sq_max))
            args.append(sgs.AuxArgs(x=t[4].data_ptr(), y=dy.data_ptr(), w=t[0].data_ptr(), bias=t[1].data_ptr(), w2=t[2].data_ptr(), bias2=t[3].data_ptr()))
            refs.append(oracle.layer_se_gate(w1, b1, w2, b2, g, sq)); outs.append(dy)
        run(descs, args, grouped)
        for shape, ref, dy in zip(SE_CASES, refs, outs):
            assert np.abs(dy.cpu().numpy() - ref).max() <= 2e-5, (shape, grouped)


def test_grouped_form_refuses_what_its_kernels_do_not_take():
    x = torch.zeros((1, 5, 5, 12), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((1, 3, 3, 12), dtype=torch.bfloat16, device="cuda")
    d = sgs.AuxDesc(kind=SGS_AUX_MAXPOOL, dtype=sgs.SGS_BF16, N=1, H=5, W=5, C=12)
    with pytest.raises(sgs.SgsError) as e:
        sgs.aux_op([d], [sgs.AuxArgs(x=x.data_ptr(), y=y.data_ptr())], True)
    assert e.value.status == SGS_EUNSUPPORTED
