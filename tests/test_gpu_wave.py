"""GPU parity of the wave execution (grouped launches over many queries in flight) against the CPU checker.

Same tolerance as the other bf16 parity tests: max|err| <= 2e-2 * max|ref| per output row against the
checker run with the same storage rounding points.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def _run(gnet, cfgs, d_in, batch, res, n_classes, wave, conc, host=False, latency=0):
    n = len(cfgs)
    stream = torch.cuda.Stream()
    opts = sgs.StreamOpts(cache_enabled=1, window_q=4, cache_budget_bytes=0, use_graphs=1, record_latency=latency,
                          concurrency=conc, wave=wave)
    if host:
        h_out = np.zeros((n * batch, n_classes), dtype=np.float32)
        h_in = d_in.cpu().view(torch.int16).numpy()
        st = gnet.stream_run(cfgs, h_in, batch, res, h_out, opts, stream.cuda_stream, host=True)
        return h_out, st
    d_out = torch.zeros((n * batch, n_classes), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    st = gnet.stream_run(cfgs, d_in.data_ptr(), batch, res, d_out.data_ptr(), opts, stream.cuda_stream)
    return d_out.cpu().numpy(), st


def test_resnet_wave_matches_checker_and_is_deterministic():
    # 21 queries in waves of 8 (a ragged last wave of 5), two waves in flight, 64x64 inputs
    _, onet, gnet = gu.nets(wl.RESNET, True)
    n, res = 21, 64
    cfgs = wl.uniform_stream(wl.RESNET, n - 2, seed=11) + [wl.extreme_cfg(wl.RESNET, False), wl.extreme_cfg(wl.RESNET, True)]
    xs = wl.make_inputs(n, 1, res, seed=5, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    got, st = _run(gnet, cfgs, d_in, 1, res, 1000, wave=8, conc=2, latency=1)
    assert st.p50_ms > 0 and st.kernel_launches > 0
    for t in range(n):
        ref = onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)
        assert gu.rel_err(got[t:t + 1], ref) <= TOL_BF16, t
    again, _ = _run(gnet, cfgs, d_in, 1, res, 1000, wave=8, conc=2)
    np.testing.assert_array_equal(again, got)
    # other wave sizes and the host-buffer variant give the same bits (a tile never depends on its neighbours)
    for wave, conc in ((1, 1), (5, 3), (64, 1)):
        other, _ = _run(gnet, cfgs, d_in, 1, res, 1000, wave=wave, conc=conc)
        np.testing.assert_array_equal(other, got)
    hosted, _ = _run(gnet, cfgs, d_in, 1, res, 1000, wave=8, conc=2, host=True)
    np.testing.assert_array_equal(hosted, got)


def test_resnet_wave_accounting_equals_the_sequential_stream():
    # the cache policy and its byte accounting follow the stream order whatever the execution mode
    _, _, gnet = gu.nets(wl.RESNET, True)
    n, res = 16, 64
    cfgs = wl.markov_stream(n, seed=9)
    d_in = gu.to_device(wl.make_inputs(n, 1, res, seed=2, bf16=True).reshape(n, res, res, 3), True)
    _, seq = _run(gnet, cfgs, d_in, 1, res, 1000, wave=0, conc=1)
    _, wav = _run(gnet, cfgs, d_in, 1, res, 1000, wave=8, conc=2)
    assert wav.hit_ratio == seq.hit_ratio and wav.hbm_weight_bytes == seq.hbm_weight_bytes
    assert wav.weight_bytes == seq.weight_bytes and wav.useful_flops == seq.useful_flops
    assert wav.kernel_launches < seq.kernel_launches


def test_resnet_wave_batched_members_224():
    # members with several images each (4 configs x 4 images), full resolution: sampled against the checker
    _, onet, gnet = gu.nets(wl.RESNET, True)
    groups, batch, res = 4, 4, 224
    cfgs = wl.uniform_stream(wl.RESNET, groups, seed=5)
    xs = wl.make_inputs(groups, batch, res, seed=3, bf16=True)
    d_in = gu.to_device(xs.reshape(groups * batch, res, res, 3), True)
    got, _ = _run(gnet, cfgs, d_in, batch, res, 1000, wave=4, conc=1)
    assert np.all(np.isfinite(got))
    for g in (0, 3):
        ref = onet.forward(cfgs[g], xs[g], oracle.BF16_STORE)
        assert gu.rel_err(got[g * batch:(g + 1) * batch], ref) <= TOL_BF16, g


def test_wave_mode_on_the_other_families():
    # MobileNetV3-shaped (depthwise and SE layers grouped by kernel size) and Tiny SuperNets (CUDA-core
    # convolutions run per member)
    for fam, res, ncls, n in ((wl.MBV3, 64, 1000, 6), (wl.MBV3, 96, 1000, 11), (wl.TINY, 32, 10, 6)):
        _, onet, gnet = gu.nets(fam, True)
        cfgs = wl.uniform_stream(fam, n, seed=7)
        xs = wl.make_inputs(n, 1, res, seed=8, bf16=True)
        d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
        got, _ = _run(gnet, cfgs, d_in, 1, res, ncls, wave=4, conc=2)
        for t in range(n):
            ref = onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)
            assert gu.rel_err(got[t:t + 1], ref) <= TOL_BF16, (fam, t)


def test_bench_wave_configuration_sampled_against_checker():
    # the benchmark's launch configuration (224x224, batch 1, waves of 32, 4 waves in flight, cache on) on the
    # first 160 queries of its stream: sampled queries recomputed by the checker, every logit finite, the
    # stream reproduces itself bit for bit, and the top-1 class of the sampled queries agrees
    _, onet, gnet = gu.nets(wl.RESNET, True)
    n, res = 160, 224
    cfgs = wl.uniform_stream(wl.RESNET, 1000, seed=2)[:n]
    xs = wl.make_inputs(n, 1, res, seed=1, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    first, st = _run(gnet, cfgs, d_in, 1, res, 1000, wave=32, conc=4, latency=1)
    again, _ = _run(gnet, cfgs, d_in, 1, res, 1000, wave=32, conc=4)
    np.testing.assert_array_equal(again, first)
    assert np.all(np.isfinite(first)) and st.p50_ms > 0
    sample = list(range(0, n, 7))
    strict = 0
    worst = 0.0
    for t in sample:
        ref = onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)
        worst = max(worst, gu.rel_err(first[t:t + 1], ref))
        strict += int(first[t].argmax() == ref[0].argmax())
    print(f"wave configuration: worst rel err {worst:.2e}, top-1 agreement {strict}/{len(sample)}")
    assert worst <= TOL_BF16
    assert strict >= len(sample) - 1


def test_profile_trace_lists_every_launch_of_a_wave():
    _, onet, gnet = gu.nets(wl.RESNET, True)
    n, res, G = 8, 64, 4
    cfgs = wl.uniform_stream(wl.RESNET, n, seed=12)
    d_in = gu.to_device(wl.make_inputs(n, 1, res, seed=2, bf16=True).reshape(n, res, res, 3), True)
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    opts = sgs.StreamOpts(cache_enabled=1, window_q=2, record_latency=0, concurrency=1, wave=G)
    plain = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
    ref = d_out.cpu().numpy().copy()
    gnet.set_option("profile", 2)
    try:
        st = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
        trace = gnet.profile_trace()
        by_class = [gnet.profile_read(c) for c in range(4)]
    finally:
        gnet.set_option("profile", 0)
    np.testing.assert_array_equal(d_out.cpu().numpy(), ref)            # profiling does not change results
    assert len(trace) == st.kernel_launches == plain.kernel_launches   # one record per launch, in issue order
    for c in range(4):
        rows = [r for r in trace if r["kernel_class"] == c]
        assert len(rows) == by_class[c]["launches"]
        assert abs(sum(r["ms"] for r in rows) - by_class[c]["total_ms"]) < 1e-6 * max(1.0, by_class[c]["total_ms"])
        assert abs(sum(r["flops"] for r in rows) - by_class[c]["flops"]) <= 1e-9 * max(1.0, by_class[c]["flops"])
    conv = [r for r in trace if r["kernel_class"] == 0]
    assert conv and all(r["ms"] > 0 and 1 <= r["members"] <= 2 * G and 2 * r["tiles"] >= r["members"] and r["name"] for r in conv)   # (two small members may share a tile)
    assert conv[0]["name"] == "stem" and trace[-1]["name"] == "fc"
    # useful FLOPs of the trace = those of the stream
    assert abs(sum(r["flops"] for r in trace) - st.useful_flops) <= 1e-6 * st.useful_flops
    gnet.set_option("profile", 2)                                      # reset empties the trace
    gnet.set_option("profile", 0)
    assert gnet.profile_trace() == []


@pytest.mark.parametrize("family,res", [(wl.RESNET, 224), (wl.MBV3, 224), (wl.RESNET, 192)])
def test_members_sharing_a_tile_at_7x7_maps(family, res):
    # at 224x224 the last stage works on 7x7 maps: two members of a wave then share the 128 rows of a tile
    # (the one with the larger slice owns the weight copies).  Results must not depend on who shares with whom.
    _, onet, gnet = gu.nets(family, True)
    n = 7                                       # (192x192: 6x6 maps, 36 rows per member)
    cfgs = wl.uniform_stream(family, n, seed=31)
    cfgs[2] = wl.extreme_cfg(family, True)      # the largest and the smallest SubNet side by side
    cfgs[3] = wl.extreme_cfg(family, False)
    x = wl.make_inputs(n, 1, res, seed=4, bf16=True).reshape(n, res, res, 3)
    d_in = gu.to_device(x, True)
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = []
    for G in (1, 7, 2):
        d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
        opts = sgs.StreamOpts(cache_enabled=1, window_q=2, record_latency=0, concurrency=2, wave=G)
        gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
        outs.append(d_out.cpu().numpy())
    np.testing.assert_array_equal(outs[1], outs[0])     # waves of 7 (pairs) against waves of 1 (no pairs)
    np.testing.assert_array_equal(outs[2], outs[0])
    for t in (2, 3, 5):
        ref = onet.forward(cfgs[t], x[t:t + 1], oracle.BF16_STORE)
        assert gu.rel_err(outs[1][t:t + 1], ref) < 2e-2


@pytest.mark.parametrize("res", [160, 192, 224])
def test_sweep_launch_shape_16_images_per_member(res):
    # the throughput sweep's launch shape: waves of 4 SubNet configs x 16 images each (one batch of 64 per grouped
    # launch), two waves in flight; two members per resolution are recomputed by the checker (both modes), and the
    # result must be the bits of the same queries run one member per wave
    _, onet, gnet = gu.nets(wl.RESNET, True)
    groups, batch = 8, 16
    cfgs = wl.uniform_stream(wl.RESNET, groups, seed=5)
    cfgs[5] = wl.extreme_cfg(wl.RESNET, True)
    xs = wl.make_inputs(groups, batch, res, seed=3, bf16=True)
    d_in = gu.to_device(xs.reshape(groups * batch, res, res, 3), True)
    got, _ = _run(gnet, cfgs, d_in, batch, res, 1000, wave=4, conc=2)
    assert np.all(np.isfinite(got))
    single, _ = _run(gnet, cfgs, d_in, batch, res, 1000, wave=1, conc=1)
    np.testing.assert_array_equal(single, got)
    for g in (1, 5):
        rows = got[g * batch:(g + 1) * batch]
        assert gu.rel_err(rows, onet.forward(cfgs[g], xs[g], oracle.BF16_STORE)) <= TOL_BF16, g
        assert gu.rel_err(rows, onet.forward(cfgs[g], xs[g], oracle.FP32)) <= TOL_BF16, g


def test_mbv3_bench_wave_configuration_sampled_against_checker():
    # the MobileNetV3-shaped stream as the benchmark runs it: 224x224, waves of 32, 4 in flight, the first 128 queries
    # of its stream (depthwise kernels of 3, 5 and 7 mixed inside every wave, so one depthwise launch dispatches all
    # three bodies); sampled queries against the checker, bit-identical to waves of 5
    _, onet, gnet = gu.nets(wl.MBV3, True)
    n, res = 128, 224
    cfgs = wl.uniform_stream(wl.MBV3, 1000, seed=3)[:n]
    kernels = {int(c.kernel[s][b]) for c in cfgs[:32] for s in range(5) for b in range(c.depth[s])}
    assert kernels == {3, 5, 7}
    xs = wl.make_inputs(n, 1, res, seed=1, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    first, _ = _run(gnet, cfgs, d_in, 1, res, 1000, wave=32, conc=4)
    other, _ = _run(gnet, cfgs, d_in, 1, res, 1000, wave=5, conc=2)
    np.testing.assert_array_equal(other, first)
    assert np.all(np.isfinite(first))
    for t in range(0, n, 9):
        assert gu.rel_err(first[t:t + 1], onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)) <= TOL_BF16, t
        assert gu.rel_err(first[t:t + 1], onet.forward(cfgs[t], xs[t], oracle.FP32)) <= TOL_BF16, t


@pytest.mark.parametrize("fam", [wl.RESNET, wl.MBV3])
def test_fp32_mode_at_full_resolution(fam):
    # fp32 handles at 224x224 (CUDA-core kernels throughout): max|err| <= 1e-4 * max|ref| against the fp32 checker
    _, onet, gnet = gu.nets(fam, False)
    c = wl.uniform_stream(fam, 2, seed=17)[1]
    x = wl.make_inputs(1, 2, 224, seed=6)[0]
    got = gu.gpu_forward(gnet, c, x, False)
    ref = onet.forward(c, x, oracle.FP32)
    assert gu.rel_err(got, ref) <= 1e-4
    np.testing.assert_array_equal(got.argmax(-1), ref.argmax(-1))
