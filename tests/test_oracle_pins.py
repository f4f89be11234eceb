"""Pins for the CPU checker: what the paper and plain mathematics fix, independent of the checker.

Paper facts used (Section 2.1): a SubNet is a selection of SuperNet weights; the largest SubNet is
the whole SuperNet and the smallest is contained in all others; a SubNet predicts without being
extracted.  Section 2.2: the shared SubGraph of two SubNets is the intersection of their graphs.
Appendix A.4: hit ratio formula, equal to 1 when the cached SubGraph is the served SubNet.
"""
import ctypes
import itertools
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2306_17266_b200 import workload as wl
from tests import torch_ref

RES = {wl.TINY: 32, wl.RESNET: 32, wl.MBV3: 32}


@pytest.fixture(scope="module")
def nets():
    out = {}
    for fam in (wl.TINY, wl.RESNET, wl.MBV3):
        blob = wl.make_blob(fam, seed=0)
        out[fam] = (blob, oracle.Net(fam, blob))
    return out


# ---------------------------------------------------------------- layer level: brute force & library

def brute_conv(x, w, Cp, Kp, k, st):
    """Seven nested Python loops straight from the definition (cross-correlation, zero padding)."""
    N, H, W, _ = x.shape
    R = w.shape[2]
    o, p = (R - k) // 2, (k - 1) // 2
    Ho, Wo = (H + 2 * p - k) // st + 1, (W + 2 * p - k) // st + 1
    y = np.zeros((N, Ho, Wo, Kp), dtype=np.float64)
    for n in range(N):
        for ho in range(Ho):
            for wo in range(Wo):
                for f in range(Kp):
                    acc = 0.0
                    for r in range(k):
                        for s in range(k):
                            hi, wi = ho * st + r - p, wo * st + s - p
                            if not (0 <= hi < H and 0 <= wi < W):
                                continue
                            for c in range(Cp):
                                acc += float(x[n, hi, wi, c]) * float(w[f, c, o + r, o + s])
                    y[n, ho, wo, f] = acc
    return y


@pytest.mark.parametrize("k,st,R", [(1, 1, 1), (3, 1, 3), (3, 2, 3), (3, 1, 7), (5, 2, 7), (7, 1, 7), (1, 2, 1)])
def test_conv_against_brute_force(k, st, R):
    rng = np.random.default_rng(10 * k + st)
    x = rng.standard_normal((2, 6, 5, 4)).astype(np.float32)
    w = rng.standard_normal((5, 4, R, R)).astype(np.float32)
    y = oracle.layer_conv(w, x[..., :3], Cp=3, Kp=2, k=k, stride=st)
    ref = brute_conv(x[..., :3], w, 3, 2, k, st)
    assert y.shape == ref.shape
    np.testing.assert_allclose(y, ref, rtol=1e-5, atol=1e-5)


def test_all_ones_weights_give_window_sums():
    x = np.arange(1, 1 + 4 * 4, dtype=np.float32).reshape(1, 4, 4, 1)
    w = np.ones((1, 1, 3, 3), dtype=np.float32)
    y = oracle.layer_conv(w, x, 1, 1, 3, 1)[0, :, :, 0]
    # hand-computed: corner = 1+2+5+6, centre (1,1) = sum of the 3x3 block starting at 1
    assert y[0, 0] == 14 and y[1, 1] == 54 and y[3, 3] == 11 + 12 + 15 + 16 and y[0, 1] == 1 + 2 + 3 + 5 + 6 + 7


def test_impulse_returns_unflipped_kernel():
    # an impulse at (2,2) must place w[r][s] at output (2 - (r-p), 2 - (s-p)): cross-correlation
    x = np.zeros((1, 5, 5, 1), dtype=np.float32)
    x[0, 2, 2, 0] = 1
    w = np.arange(9, dtype=np.float32).reshape(1, 1, 3, 3)
    y = oracle.layer_conv(w, x, 1, 1, 3, 1)[0, :, :, 0]
    for r in range(3):
        for s in range(3):
            assert y[2 - (r - 1), 2 - (s - 1)] == w[0, 0, r, s]
    # stride 2 keeps even output positions of the stride-1 result (pins the stride phase)
    y2 = oracle.layer_conv(w, x, 1, 1, 3, 2)[0, :, :, 0]
    np.testing.assert_array_equal(y2, y[::2, ::2])


@pytest.mark.parametrize("k,st", [(1, 1), (1, 2), (3, 1), (3, 2), (7, 2)])
def test_conv_matches_library(k, st):
    rng = np.random.default_rng(k + st)
    Kmax, Cmax, Kp, Cp = 24, 16, 16, 8
    x = rng.standard_normal((2, 12, 10, Cp)).astype(np.float32)
    w = rng.standard_normal((Kmax, Cmax, k, k)).astype(np.float32)
    y = oracle.layer_conv(w, x, Cp, Kp, k, st)
    ref = F.conv2d(torch.tensor(x, dtype=torch.float64).permute(0, 3, 1, 2), torch.tensor(w[:Kp, :Cp], dtype=torch.float64),
                   stride=st, padding=(k - 1) // 2).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-4, atol=1e-4)
    if k == 1 and st == 1:  # 1x1 conv is a matrix product
        np.testing.assert_allclose(y.reshape(-1, Kp), x.reshape(-1, Cp).astype(np.float64) @ w[:Kp, :Cp, 0, 0].T.astype(np.float64), rtol=1e-4, atol=1e-4)


@pytest.mark.parametrize("k,st", [(3, 1), (5, 1), (7, 2), (3, 2)])
def test_depthwise_matches_grouped_library_conv(k, st):
    rng = np.random.default_rng(100 + k + st)
    Kmax, Kp = 12, 8
    x = rng.standard_normal((2, 9, 11, Kp)).astype(np.float32)
    w = rng.standard_normal((Kmax, 1, 7, 7)).astype(np.float32)
    y = oracle.layer_conv(w, x, 1, Kp, k, st, depthwise=True)
    o = (7 - k) // 2
    ref = F.conv2d(torch.tensor(x, dtype=torch.float64).permute(0, 3, 1, 2),
                   torch.tensor(w[:Kp, :, o:o + k, o:o + k], dtype=torch.float64), stride=st, padding=(k - 1) // 2,
                   groups=Kp).permute(0, 2, 3, 1).numpy()
    np.testing.assert_allclose(y, ref, rtol=1e-4, atol=1e-4)


def test_zero_ring_makes_kernel_sizes_agree():
    # a stored 7x7 depthwise kernel whose outer rings are zero gives the same output at k = 7, 5, 3:
    # pins the crop offset (7-k)/2 together with the padding (k-1)/2
    rng = np.random.default_rng(5)
    w = np.zeros((8, 1, 7, 7), dtype=np.float32)
    w[:, :, 2:5, 2:5] = rng.standard_normal((8, 1, 3, 3))
    x = rng.standard_normal((1, 9, 9, 8)).astype(np.float32)
    y7 = oracle.layer_conv(w, x, 1, 8, 7, 1, depthwise=True)
    y5 = oracle.layer_conv(w, x, 1, 8, 5, 1, depthwise=True)
    y3 = oracle.layer_conv(w, x, 1, 8, 3, 1, depthwise=True)
    np.testing.assert_allclose(y5, y7, rtol=0, atol=1e-6)
    np.testing.assert_allclose(y3, y7, rtol=0, atol=1e-6)
    w[:, :, 1, 1] = 1.0  # ring 5 now non-zero: k=3 must differ from k=5
    assert np.abs(oracle.layer_conv(w, x, 1, 8, 5, 1, depthwise=True) - oracle.layer_conv(w, x, 1, 8, 3, 1, depthwise=True)).max() > 1e-3


def test_zeroed_complement_equals_slice_layer():
    # weights outside the prefix box set to zero, run at full width == sliced run (extra input
    # channels may hold anything)
    rng = np.random.default_rng(6)
    Kmax, Cmax, Kp, Cp = 16, 12, 8, 5
    w = rng.standard_normal((Kmax, Cmax, 3, 3)).astype(np.float32)
    x = rng.standard_normal((1, 7, 7, Cmax)).astype(np.float32)
    ys = oracle.layer_conv(w, np.ascontiguousarray(x[..., :Cp]), Cp, Kp, 3, 1)
    wz = np.zeros_like(w)
    wz[:Kp, :Cp] = w[:Kp, :Cp]
    yf = oracle.layer_conv(wz, x, Cmax, Kmax, 3, 1)
    np.testing.assert_allclose(yf[..., :Kp], ys, rtol=0, atol=1e-5)
    assert np.all(yf[..., Kp:] == 0)


def test_epilogue_maxpool_gap_bf16_against_library():
    rng = np.random.default_rng(7)
    y = rng.standard_normal((2, 5, 6, 8)).astype(np.float32) * 3
    g, b, m, v = (rng.uniform(0.5, 1.5, 8).astype(np.float32), rng.standard_normal(8).astype(np.float32),
                  rng.standard_normal(8).astype(np.float32), rng.uniform(0.5, 1.5, 8).astype(np.float32))
    res = rng.standard_normal(y.shape).astype(np.float32)
    t = torch.tensor(y, dtype=torch.float64).permute(0, 3, 1, 2)
    bn = F.batch_norm(t, torch.tensor(m, dtype=torch.float64), torch.tensor(v, dtype=torch.float64),
                      torch.tensor(g, dtype=torch.float64), torch.tensor(b, dtype=torch.float64), False, 0.0, 1e-5)
    bn = bn + torch.tensor(res, dtype=torch.float64).permute(0, 3, 1, 2)
    for act, fn in ((oracle.ACT_NONE, lambda z: z), (oracle.ACT_RELU, F.relu), (oracle.ACT_HSWISH, F.hardswish)):
        out = oracle.layer_epilogue(y, g, b, m, v, None, res, act)
        np.testing.assert_allclose(out, fn(bn).permute(0, 2, 3, 1).numpy(), rtol=1e-5, atol=1e-5)
    # bf16 storage rounding equals torch's round-to-nearest-even conversion
    out = oracle.layer_epilogue(y, g, b, m, v, None, res, oracle.ACT_NONE, oracle.BF16_STORE)
    f32 = oracle.layer_epilogue(y, g, b, m, v, None, res, oracle.ACT_NONE, oracle.FP32)
    np.testing.assert_array_equal(out, torch.tensor(f32).to(torch.bfloat16).to(torch.float32).numpy())
    np.testing.assert_array_equal(wl.round_to_bf16(f32), out)
    for val in (1.0, 1.00390625, 1.01171875, -3.0e-5, 65504.0):
        assert oracle.bf16_round(val) == float(torch.tensor(val, dtype=torch.float32).to(torch.bfloat16))
    # pooling
    x = rng.standard_normal((2, 9, 8, 4)).astype(np.float32)
    mp = F.max_pool2d(torch.tensor(x).permute(0, 3, 1, 2), 3, 2, 1).permute(0, 2, 3, 1).numpy()
    np.testing.assert_array_equal(oracle.layer_maxpool(x), mp)
    np.testing.assert_allclose(oracle.layer_gap(x), x.astype(np.float64).mean(axis=(1, 2)), rtol=1e-5, atol=1e-6)


# ---------------------------------------------------------------- network level

@pytest.mark.parametrize("fam", [wl.TINY, wl.RESNET, wl.MBV3])
def test_largest_subnet_is_the_supernet(nets, fam):
    blob, net = nets[fam]
    x = wl.make_inputs(1, 2, RES[fam], seed=1)[0]
    big = wl.extreme_cfg(fam, True)
    np.testing.assert_array_equal(net.forward(big, x), net.forward(big, x, path="unsliced"))


@pytest.mark.parametrize("fam", [wl.TINY, wl.RESNET, wl.MBV3])
def test_sliced_equals_extracted_copy(nets, fam):
    blob, net = nets[fam]
    x = wl.make_inputs(1, 1, RES[fam], seed=1)[0]
    cfgs = wl.uniform_stream(fam, 4, seed=2) + [wl.extreme_cfg(fam, False)]
    for mode in (oracle.FP32, oracle.BF16_STORE):
        for c in cfgs:
            np.testing.assert_array_equal(net.forward(c, x, mode), net.forward(c, x, mode, path="extracted"))


@pytest.mark.parametrize("fam", [wl.TINY, wl.RESNET, wl.MBV3])
def test_network_matches_library_restatement(nets, fam):
    blob, net = nets[fam]
    P = torch_ref.parse_blob(fam, blob)
    x = wl.make_inputs(1, 2, RES[fam], seed=3)[0]
    for c in wl.uniform_stream(fam, 3, seed=11) + [wl.extreme_cfg(fam, False), wl.extreme_cfg(fam, True)]:
        ref = torch_ref.forward(fam, P, c, x)
        got = net.forward(c, x)
        assert np.abs(got - ref).max() <= 2e-4 * max(1.0, np.abs(ref).max())


def _bf16_representable(a):
    return bool(np.all((np.ascontiguousarray(a, dtype=np.float32).view(np.uint32) & 0xFFFF) == 0))


def _stored_tensors(net, fam, cfg, x, mode):
    """Every tensor the checker stores on the way (one tapped run per stored layer the SubNet uses) and its logits."""
    names = [r.name for r in wl.supernet_records(fam)]
    out, logits = {}, None
    for i, name in enumerate(names):
        logits, t = net.forward_tap(cfg, x, i, mode)
        if t is not None:
            out[name] = t
    return out, logits


@pytest.mark.parametrize("fam,res", [(wl.TINY, 32), (wl.RESNET, 64), (wl.MBV3, 64)])
def test_bf16_store_mode_rounds_exactly_the_stored_tensors(fam, res):
    """Pins where the bf16-store mode rounds.  Layer by layer, each layer fed with the checker's own stored inputs:
    a tensor the mode stores (layer outputs, SE-scaled maps) holds only bf16 values and equals the fp64 library
    restatement rounded once, up to a few one-step flips from the order of additions; what is not stored (pooled and
    SE vectors, the head's mixing vector, logits) is not rounded, so the logits computed from the last stored tensor
    agree to fp32 accuracy.  (The max-pooled map is stored too, but the maximum of bf16 values is one of them: rounding
    it changes nothing and cannot be pinned.)"""
    blob = wl.make_blob(fam, seed=0, bf16_weights=True)
    net = oracle.Net(fam, blob)
    P = torch_ref.parse_blob(fam, blob)
    x = wl.make_inputs(1, 2, res, seed=3, bf16=True)[0]
    for c in wl.uniform_stream(fam, 2, seed=11) + [wl.extreme_cfg(fam, True)]:
        taught, logits = _stored_tensors(net, fam, c, x, oracle.BF16_STORE)
        assert len(taught) >= 5
        store = torch_ref.Store(True, teacher=taught)
        ref_logits = torch_ref.forward(fam, P, c, x, store)
        assert set(store.report) == set(taught)  # every tapped tensor was met on the way
        for name, t in taught.items():
            rep = store.report[name]
            assert _bf16_representable(t), name
            assert rep["beyond_one_step"] == 0, (name, rep)
            assert rep["unequal"] <= max(2, 0.005 * rep["n"]), (name, rep)
        assert np.abs(logits - ref_logits).max() <= 2e-5 * max(1.0, np.abs(ref_logits).max())
        # a checker that forgot to round (its fp32 mode) is caught by the same checks
        plain, _ = _stored_tensors(net, fam, c, x, oracle.FP32)
        assert not any(_bf16_representable(t) for t in plain.values())


@pytest.mark.parametrize("fam,res", [(wl.TINY, 32), (wl.MBV3, 64)])
def test_bf16_store_network_matches_library_restatement(fam, res):
    """Whole network, no teacher: on the shallow family, and on MobileNetV3-shaped SubNets of minimum depth, the two
    implementations stay within a few flips of each other end to end, and leaving out the rounding of the layer
    outputs (or, with squeeze-excite blocks, of the SE-scaled map) moves the logits visibly further away."""
    blob = wl.make_blob(fam, seed=0, bf16_weights=True)
    net = oracle.Net(fam, blob)
    P = torch_ref.parse_blob(fam, blob)
    x = wl.make_inputs(1, 2, res, seed=3, bf16=True)[0]
    c = wl.extreme_cfg(fam, False)
    got = net.forward(c, x, oracle.BF16_STORE)

    def dist(skip):
        ref = torch_ref.forward(fam, P, c, x, torch_ref.Store(True, skip))
        return np.abs(got - ref).max() / np.abs(ref).max()

    base = dist(())
    assert base <= 2e-5
    assert dist(("layer",)) > 20 * max(base, 1e-6)
    if fam == wl.MBV3:
        assert dist(("se_scale",)) > 20 * max(base, 1e-6)


def _record_offsets(fam):
    """word offset of each record's float payload in the blob"""
    pos, out = 8, {}
    for r in wl.supernet_records(fam):
        pos += 8
        out[r.name] = (pos, r)
        pos += r.n_floats
    return out


def test_zeroed_complement_equals_slice_network(nets):
    # zero every stored weight outside a config's prefixes, then run the widest config of the same
    # depth: the logits equal the config's own
    fam = wl.TINY
    blob, net = nets[fam]
    cfg = wl.uniform_stream(fam, 6, seed=21)[3]
    enc = net.encode(cfg)
    words = np.frombuffer(blob.copy(), dtype=np.uint32).copy()
    for i, (name, (pos, r)) in enumerate(_record_offsets(fam).items()):
        w = words[pos:pos + r.n_weights].view(np.float32).reshape(r.K, r.C, r.R, r.S)
        keep = np.zeros_like(w)
        Kp, Cp = enc[i, 0], enc[i, 1]
        keep[:Kp, :Cp] = w[:Kp, :Cp]
        w[...] = keep
    wide = wl.copy_cfg(cfg)
    for s in range(3):
        wide.width[s + 1] = 1.0
    x = wl.make_inputs(1, 1, 32, seed=4)[0]
    ref = net.forward(cfg, x)
    got = oracle.Net(fam, words.view(np.uint8)).forward(wide, x)
    np.testing.assert_allclose(got, ref, rtol=0, atol=1e-5)


@pytest.mark.parametrize("fam,stage", [(wl.TINY, 1), (wl.RESNET, 2), (wl.MBV3, 3)])
def test_dead_last_block_equals_shallower_stage(nets, fam, stage):
    # block d of a stage made a no-op (gamma = beta = 0 on its last BN): depth d+1 equals depth d.
    # Pins "the first d blocks" and the residual wiring.
    blob, net = nets[fam]
    base = wl.extreme_cfg(fam, False)
    d = base.depth[stage]
    last = {wl.TINY: "conv2", wl.RESNET: "conv3", wl.MBV3: "project"}[fam]
    pos, r = _record_offsets(fam)[f"s{stage}b{d}.{last}"]
    words = np.frombuffer(blob.copy(), dtype=np.uint32).copy()
    f = words[pos:pos + r.n_floats].view(np.float32)
    f[r.n_weights:r.n_weights + 2 * r.K] = 0  # gamma, beta
    net2 = oracle.Net(fam, words.view(np.uint8))
    deeper = wl.copy_cfg(base)
    deeper.depth[stage] = d + 1
    x = wl.make_inputs(1, 1, RES[fam], seed=5)[0]
    np.testing.assert_allclose(net2.forward(deeper, x), net2.forward(base, x), rtol=0, atol=1e-6)
    assert np.abs(net.forward(deeper, x) - net.forward(base, x)).max() > 1e-4


# ---------------------------------------------------------------- slice arithmetic, encoding, hit ratio

def test_channel_counts_of_the_named_configs(nets):
    # widths the workload definitions state in words: Tiny 16/32/64 x {0.5, 0.75, 1};
    # ResNet-shaped stem 64 x {0.65, 0.8, 1} -> 40/48/64 and mid = nearest multiple of 8
    _, tiny = nets[wl.TINY]
    c = wl.extreme_cfg(wl.TINY, False)
    c.width[2] = 0.75
    e = tiny.encode(c)
    assert e[0].tolist() == [8, 3, 3]            # stem: 16*0.5
    names = [r.name for r in wl.supernet_records(wl.TINY)]
    assert e[names.index("s1b0.conv1")].tolist() == [24, 8, 3]
    assert e[names.index("s1b0.proj")].tolist() == [24, 8, 1]
    assert e[names.index("s1b1.conv1")].tolist() == [0, 0, 0]  # depth 1: block 1 unused
    assert e[names.index("s2b0.conv1")].tolist() == [32, 24, 3]
    assert e[names.index("fc")].tolist() == [10, 32, 1]
    _, rn = nets[wl.RESNET]
    names = [r.name for r in wl.supernet_records(wl.RESNET)]
    for w, stem in ((0.65, 40), (0.8, 48), (1.0, 64)):
        c = wl.extreme_cfg(wl.RESNET, True)
        c.width[0] = w
        assert rn.encode(c)[0].tolist() == [stem, 3, 7]
    c = wl.extreme_cfg(wl.RESNET, True)
    e = rn.encode(c)
    assert e[names.index("s3b0.conv2")].tolist() == [720, 720, 3]   # 2048*0.35 = 716.8 -> 720
    assert e[names.index("s0b0.conv1")].tolist() == [88, 64, 1]     # 256*0.35 = 89.6 -> 88
    c.width[4] = 0.65
    e = rn.encode(c)
    assert e[names.index("s3b1.conv1")].tolist() == [464, 1328, 1]  # 2048*.65 -> 1328; *.35 -> 464
    assert e[names.index("fc")].tolist() == [1000, 1328, 1]
    _, mb = nets[wl.MBV3]
    names = [r.name for r in wl.supernet_records(wl.MBV3)]
    c = wl.extreme_cfg(wl.MBV3, False)
    e = mb.encode(c)
    assert e[names.index("s1b0.expand")].tolist() == [72, 24, 1]
    assert e[names.index("s1b0.dw")].tolist() == [72, 1, 3]
    assert e[names.index("s1b0.se1")].tolist() == [16, 72, 1]      # 72/4 = 18 -> 16
    assert e[names.index("s1b2.dw")].tolist() == [0, 0, 0]


def test_invalid_configs_are_rejected(nets):
    _, rn = nets[wl.RESNET]
    c = wl.extreme_cfg(wl.RESNET, True)
    assert rn.validate(c)
    c.width[2] = 0.7
    assert not rn.validate(c)
    c = wl.extreme_cfg(wl.RESNET, True)
    c.depth[1] = 5
    assert not rn.validate(c)
    _, mb = nets[wl.MBV3]
    c = wl.extreme_cfg(wl.MBV3, True)
    c.kernel[0][0] = 4
    assert not mb.validate(c)


def _index_set(enc_row, R):
    K, C, k = (int(v) for v in enc_row)
    o = (R - k) // 2
    return {(f, c, r, s) for f in range(K) for c in range(C) for r in range(o, o + k) for s in range(o, o + k)}


def test_intersection_is_elementwise_min(nets):
    # the shared SubGraph of two SubNets, found by enumerating stored weight indices, is the net
    # whose encoding is the element-wise minimum
    _, net = nets[wl.TINY]
    recs = wl.supernet_records(wl.TINY)
    cfgs = wl.uniform_stream(wl.TINY, 6, seed=9)
    for a, b in itertools.combinations(cfgs, 2):
        ea, eb = net.encode(a), net.encode(b)
        g = oracle.intersect(ea, eb)
        np.testing.assert_array_equal(g, np.minimum(ea, eb))
        total = 0
        for i, r in enumerate(recs):
            common = _index_set(ea[i], r.R) & _index_set(eb[i], r.R)
            assert common == _index_set(g[i], r.R)
            total += len(common)
        assert total == oracle.encoding_weights(g)
    _, mb = nets[wl.MBV3]
    a, b = wl.uniform_stream(wl.MBV3, 2, seed=1)
    recs = wl.supernet_records(wl.MBV3)
    ea, eb = mb.encode(a), mb.encode(b)
    g = oracle.intersect(ea, eb)
    i = [r.name for r in recs].index("s0b0.dw")
    assert _index_set(ea[i], 7) & _index_set(eb[i], 7) == _index_set(g[i], 7)


def test_nesting_and_sizes(nets):
    # smallest SubNet inside every SubNet, every SubNet inside the largest (Section 2.1)
    for fam in (wl.TINY, wl.RESNET, wl.MBV3):
        _, net = nets[fam]
        lo, hi = net.encode(wl.extreme_cfg(fam, False)), net.encode(wl.extreme_cfg(fam, True))
        recs = wl.supernet_records(fam)
        assert hi[:, 0].tolist() == [r.K for r in recs] and hi[:, 1].tolist() == [r.C for r in recs]
        assert oracle.encoding_weights(hi) == sum(r.n_weights for r in recs)
        for c in wl.uniform_stream(fam, 20, seed=13):
            e = net.encode(c)
            assert np.all(lo <= e) and np.all(e <= hi)


def test_hit_ratio_formula(nets):
    sn = np.array([[3, 4, 1], [6, 8, 3]], dtype=np.int32)
    g = np.array([[3, 2, 1], [0, 0, 0]], dtype=np.int32)
    # || (3,2,0,0) || / || (3,4,6,8) ||
    assert abs(oracle.hit_ratio(sn, g) - np.sqrt(13.0) / np.sqrt(125.0)) < 1e-12
    assert oracle.hit_ratio(sn, sn) == 1.0           # same SubNet cached: reuse probability 1
    big = np.array([[9, 9, 3], [9, 9, 3]], dtype=np.int32)
    assert oracle.hit_ratio(sn, big) == 1.0          # cache contains the SubNet
    assert oracle.hit_ratio(sn, np.zeros_like(sn)) == 0.0


def test_linear_and_squeeze_excite_layers_against_plain_formulas():
    # sliced fully connected layer = a matrix product on the prefix block; SE gate = hsigmoid(FC2(relu(FC1(g)))) with
    # hsigmoid(x) = min(max(x + 3, 0), 6) / 6; SE scale multiplies every pixel's channels by the gate of its image.
    # fp64 numpy on Python slices; a transposed operand, a wrong prefix or a missing bias fails.
    rng = np.random.default_rng(5)
    w = rng.standard_normal((40, 56)).astype(np.float32)
    b = rng.standard_normal(40).astype(np.float32)
    v = rng.standard_normal((3, 48)).astype(np.float32)
    for Cp, Kp in ((48, 40), (24, 17), (1, 1)):
        want = v[:, :Cp].astype(np.float64) @ w[:Kp, :Cp].astype(np.float64).T + b[:Kp]
        np.testing.assert_allclose(oracle.layer_linear(w, b, v[:, :Cp], Cp, Kp), want, rtol=0, atol=2e-5)
        np.testing.assert_allclose(oracle.layer_linear(w, None, v[:, :Cp], Cp, Kp, oracle.ACT_RELU), np.maximum(want - b[:Kp], 0), rtol=0, atol=2e-5)
    mid, sq = 24, 8
    w1 = rng.standard_normal((16, 40)).astype(np.float32)   # stored [sq_max][mid_max]
    w2 = rng.standard_normal((40, 16)).astype(np.float32)   # stored [mid_max][sq_max]
    b1, b2 = rng.standard_normal(16).astype(np.float32), rng.standard_normal(40).astype(np.float32)
    g = rng.standard_normal((2, mid)).astype(np.float32)
    h = np.maximum(g.astype(np.float64) @ w1[:sq, :mid].astype(np.float64).T + b1[:sq], 0)
    gate = np.clip(h @ w2[:mid, :sq].astype(np.float64).T + b2[:mid] + 3, 0, 6) / 6
    got = oracle.layer_se_gate(w1, b1, w2, b2, g, sq)
    np.testing.assert_allclose(got, gate, rtol=0, atol=2e-6)
    x = rng.standard_normal((2, 3, 5, mid)).astype(np.float32)
    np.testing.assert_allclose(oracle.layer_se_scale(x, got), x.astype(np.float64) * got[:, None, None, :], rtol=1e-6, atol=0)
    np.testing.assert_array_equal(oracle.layer_se_scale(x, got, oracle.BF16_STORE), wl.round_to_bf16(oracle.layer_se_scale(x, got)))


def _i8_case(rng, N, H, W, Cmax, C, Kmax, K, R, x_signed):
    w = rng.integers(-127, 128, (Kmax, Cmax, R, R), dtype=np.int64).astype(np.int8)
    x = (rng.integers(-128, 128, (N, H, W, C)) if x_signed else rng.integers(0, 256, (N, H, W, C)))
    x = x.astype(np.int8 if x_signed else np.uint8)
    mult = rng.integers(1 << 29, (1 << 31) - 1, Kmax, dtype=np.int64).astype(np.int32)
    shift = rng.integers(6, 12, Kmax).astype(np.int32)
    bias = rng.integers(-40, 40, Kmax).astype(np.int32)
    return w, x, mult, shift, bias


def test_int8_layer_against_big_integer_arithmetic():
    # the 8-bit layer of the paper's numeric format, restated with numpy int64 sums on Python slices and Python's
    # unbounded integers for the requantisation (floor division, so the rounding rule is explicit): zero padding
    # counts as the real value 0 (= the zero point), slices are prefixes / centre windows, ties of the rounding
    # shift go up, ReLU is a maximum with the output zero point, results saturate
    rng = np.random.default_rng(8)
    for (N, H, W, Cmax, C, Kmax, K, R, k, st, xs, zx, zy, relu, ys, use_res) in [
            (1, 5, 6, 16, 16, 8, 8, 3, 3, 1, False, 0, 0, True, False, False),
            (2, 7, 5, 32, 16, 16, 8, 7, 5, 2, False, 3, 10, False, False, True),
            (1, 6, 6, 16, 16, 16, 16, 3, 1, 1, True, -5, -7, True, True, True),
            (1, 4, 4, 48, 32, 24, 16, 3, 3, 2, True, 0, 4, False, True, False)]:
        w, x, mult, shift, bias = _i8_case(rng, N, H, W, Cmax, C, Kmax, K, R, xs)
        p, o = (k - 1) // 2, (R - k) // 2
        Ho, Wo = (H + 2 * p - k) // st + 1, (W + 2 * p - k) // st + 1
        res = None
        zr, rm, rs = 2, 1518500250, 1   # about 0.354
        if use_res:
            res = rng.integers(0, 256, (N, Ho, Wo, K)).astype(np.uint8)
        got = oracle.layer_conv_i8(w, x, C, K, k, st, mult, shift, bias, zx=zx, zy=zy, relu=relu, res=res, zr=zr, res_mult=rm, res_shift=rs, y_signed=ys)
        xp = np.zeros((N, H + 2 * p, W + 2 * p, C), dtype=np.int64)
        xp[:, p:p + H, p:p + W, :] = x.astype(np.int64) - zx
        wk = w[:K, :C, o:o + k, o:o + k].astype(np.int64)
        for n in range(N):
            for ho in range(Ho):
                for wo in range(Wo):
                    win = xp[n, ho * st:ho * st + k, wo * st:wo * st + k, :]          # [k][k][C]
                    acc = np.einsum("rsc,fcrs->f", win, wk)
                    for f in range(K):
                        s = 31 + int(shift[f])
                        t = (int(acc[f]) * int(mult[f]) + (1 << (s - 1))) // (1 << s) + int(bias[f])
                        if use_res:
                            t += ((int(res[n, ho, wo, f]) - zr) * rm + (1 << (31 + rs - 1))) // (1 << (31 + rs))
                        t += zy
                        if relu:
                            t = max(t, zy)
                        t = min(max(t, -128 if ys else 0), 127 if ys else 255)
                        assert int(got[n, ho, wo, f]) == t, (n, ho, wo, f)


def test_int8_layer_invariants():
    rng = np.random.default_rng(9)
    w, x, mult, shift, bias = _i8_case(rng, 1, 6, 6, 32, 32, 16, 16, 3, False)
    x = (x // 2).astype(np.uint8)          # 0..127, so that a shifted copy still fits a byte
    base = oracle.layer_conv_i8(w, x, 32, 16, 3, 1, mult, shift, bias, zx=0, zy=5)
    # a tensor and its zero point moved together describe the same real values, also next to the zero padding
    moved = oracle.layer_conv_i8(w, (x + 100).astype(np.uint8), 32, 16, 3, 1, mult, shift, bias, zx=100, zy=5)
    np.testing.assert_array_equal(moved, base)
    # the same numbers read as signed bytes give the same result
    np.testing.assert_array_equal(oracle.layer_conv_i8(w, x.astype(np.int8), 32, 16, 3, 1, mult, shift, bias, zx=0, zy=5), base)
    # multiplier 2^30 with shift s is a division by 2^(s+1), ties up: checked on a 1x1 layer with unit weights
    w1 = np.zeros((8, 16, 1, 1), dtype=np.int8)
    w1[np.arange(8), np.arange(8)] = 1
    xv = np.zeros((1, 1, 8, 16), dtype=np.int8)
    xv[0, 0, :, :8] = np.array([[-5, -3, -2, -1, 1, 2, 3, 5]] * 8, dtype=np.int8)
    y = oracle.layer_conv_i8(w1, xv, 16, 8, 1, 1, np.full(8, 1 << 30), np.zeros(8), np.zeros(8), y_signed=True)
    np.testing.assert_array_equal(y[0, 0, 0], np.array([-2, -1, -1, 0, 1, 1, 2, 3], dtype=np.int8))  # floor(v / 2 + 1 / 2)
