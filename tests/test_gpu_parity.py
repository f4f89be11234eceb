"""GPU parity: libsgs (through the C interface) against the CPU checker on the same seeded inputs.

Tolerances: fp32 mode max|err| <= 1e-4 * max|ref| per output row; bf16 mode (fp32 accumulation, every
stored tensor rounded to bf16) max|err| <= 2e-2 * max|ref| against the checker run with the same
storage rounding points.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu

TOL_F32 = 1e-4
TOL_BF16 = 2e-2


def test_library_reports_bad_arguments():
    blob = wl.make_blob(wl.TINY, 0)
    _, _, g = gu.nets(wl.TINY, False)
    bad = wl.extreme_cfg(wl.TINY, True)
    bad.width[2] = 0.6
    assert g.subnet_validate(bad) == sgs.binding.SGS_ECONFIG
    x = torch.zeros((1, 32, 32, 3), device="cuda")
    out = torch.zeros((1, 10), device="cuda")
    before = g.get_counter("kernel_launches")
    with pytest.raises(sgs.SgsError) as e:
        g.subnet_run(bad, x.data_ptr(), 1, 32, out.data_ptr())
    assert e.value.status == sgs.binding.SGS_ECONFIG
    assert g.get_counter("kernel_launches") == before  # nothing launched
    with pytest.raises(sgs.SgsError):
        sgs.SuperNet(wl.RESNET, blob)  # blob of another family
    with pytest.raises(sgs.SgsError):
        sgs.SuperNet(wl.TINY, blob[:-4])


def test_tiny_fp32_all_queries():
    _, onet, gnet = gu.nets(wl.TINY, False)
    xs = wl.make_inputs(8, 1, 32, seed=1)
    cfgs = wl.uniform_stream(wl.TINY, 8, seed=2)
    for x, c in zip(xs, cfgs):
        ref = onet.forward(c, x, oracle.FP32)
        got = gu.gpu_forward(gnet, c, x, False)
        assert gu.rel_err(got, ref) <= TOL_F32
        np.testing.assert_array_equal(got.argmax(-1), ref.argmax(-1))


def test_tiny_bf16_all_queries():
    _, onet, gnet = gu.nets(wl.TINY, True)
    xs = wl.make_inputs(8, 1, 32, seed=1, bf16=True)
    cfgs = wl.uniform_stream(wl.TINY, 8, seed=2)
    for x, c in zip(xs, cfgs):
        ref = onet.forward(c, x, oracle.BF16_STORE)
        got = gu.gpu_forward(gnet, c, x, True)
        assert gu.rel_err(got, ref) <= TOL_BF16


@pytest.mark.parametrize("fam", [wl.RESNET, wl.MBV3])
@pytest.mark.parametrize("bf16", [False, True])
def test_small_resolution_configs(fam, bf16):
    # 64x64 inputs keep the checker fast while every layer type, stride and elastic choice runs;
    # batch 3 and an odd feature-map size (res 72 -> 9, 5, 3 in the last stages) give ragged tiles
    _, onet, gnet = gu.nets(fam, bf16)
    cfgs = wl.uniform_stream(fam, 4, seed=7) + [wl.extreme_cfg(fam, False), wl.extreme_cfg(fam, True)]
    for i, c in enumerate(cfgs):
        res, batch = (64, 3) if i % 2 == 0 else (72, 2)
        x = wl.make_inputs(1, batch, res, seed=20 + i, bf16=bf16)[0]
        ref = onet.forward(c, x, oracle.BF16_STORE if bf16 else oracle.FP32)
        got = gu.gpu_forward(gnet, c, x, bf16)
        assert np.all(np.isfinite(got))
        assert gu.rel_err(got, ref) <= (TOL_BF16 if bf16 else TOL_F32), (fam, bf16, i)
    if bf16 and fam == wl.RESNET:
        assert gnet.get_counter("tc_convs") > 0  # the tensor-core kernel is the path that ran


@pytest.mark.parametrize("fam", [wl.RESNET, wl.MBV3])
def test_full_resolution_bf16(fam):
    _, onet, gnet = gu.nets(fam, True)
    cfgs = wl.uniform_stream(fam, 3, seed=2 if fam == wl.RESNET else 3)
    xs = wl.make_inputs(3, 1, 224, seed=1, bf16=True)
    for x, c in zip(xs, cfgs):
        ref = onet.forward(c, x, oracle.BF16_STORE)
        got = gu.gpu_forward(gnet, c, x, True)
        assert gu.rel_err(got, ref) <= TOL_BF16


def test_no_sliced_weight_copy_is_made():
    # device memory owned by the handle does not change across configs once the workspace for the
    # largest shape exists
    _, _, gnet = gu.nets(wl.RESNET, True)
    x = wl.make_inputs(1, 1, 64, seed=1, bf16=True)[0]
    gu.gpu_forward(gnet, wl.extreme_cfg(wl.RESNET, True), x, True)
    for c in wl.uniform_stream(wl.RESNET, 5, seed=31):
        gu.gpu_forward(gnet, c, x, True)
    base = gnet.get_counter("device_bytes")
    for c in wl.uniform_stream(wl.RESNET, 8, seed=32):
        gu.gpu_forward(gnet, c, x, True)
    # only the split-reduction scratch may have grown, never by as much as the smallest sliced layer set
    assert gnet.get_counter("device_bytes") - base < 4 << 20


def test_stream_run_matches_single_queries_and_counts_bytes():
    _, onet, gnet = gu.nets(wl.RESNET, True)
    n, res = 12, 64
    cfgs = wl.markov_stream(n, seed=4)
    xs = wl.make_inputs(n, 1, res, seed=1, bf16=True)
    singles = np.stack([gu.gpu_forward(gnet, c, x, True)[0] for c, x in zip(cfgs, xs)])
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()  # graphs cannot be captured on the legacy default stream
    torch.cuda.synchronize()
    for graphs in (0, 1):
        for cache in (0, 1):
            d_out.zero_()
            torch.cuda.synchronize()
            opts = sgs.StreamOpts(cache_enabled=cache, window_q=4, cache_budget_bytes=0, use_graphs=graphs, record_latency=1)
            st = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
            np.testing.assert_array_equal(d_out.cpu().numpy(), singles)  # deterministic, bit for bit
            assert st.n_queries == n and st.kernel_launches > 0 and st.p50_ms > 0
            encs = [onet.encode(c) for c in cfgs]
            wbytes = sum(oracle.encoding_weights(e) for e in encs) * 2
            assert abs(st.weight_bytes - wbytes) < 1
            if cache:
                assert 0 < st.hbm_weight_bytes < st.weight_bytes and 0 < st.hit_ratio <= 1
            else:
                assert st.hbm_weight_bytes == st.weight_bytes and st.hit_ratio == 0
    # several queries in flight: same bits
    for conc in (2, 3):
        d_out.zero_()
        torch.cuda.synchronize()
        opts = sgs.StreamOpts(cache_enabled=1, window_q=4, cache_budget_bytes=0, use_graphs=1, record_latency=1, concurrency=conc)
        st = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
        np.testing.assert_array_equal(d_out.cpu().numpy(), singles)
        assert st.p50_ms > 0
    # host-buffer variant
    h_out = np.zeros((n, 1000), dtype=np.float32)
    h_in = d_in.cpu().view(torch.int16).numpy()
    gnet.stream_run(cfgs, h_in, 1, res, h_out, None, stream.cuda_stream, host=True)
    np.testing.assert_array_equal(h_out, singles)
    h_out[:] = 0
    opts = sgs.StreamOpts(cache_enabled=1, window_q=4, cache_budget_bytes=0, use_graphs=1, record_latency=0, concurrency=4)
    gnet.stream_run(cfgs, h_in, 1, res, h_out, opts, stream.cuda_stream, host=True)
    np.testing.assert_array_equal(h_out, singles)


def test_cache_accounting_matches_checker_formulas():
    # hit ratio and missed bytes of a stream, recomputed from the checker's encodings and formulas
    _, onet, gnet = gu.nets(wl.RESNET, True)
    n, res, q = 16, 64, 4
    cfgs = wl.markov_stream(n, seed=9)
    d_in = gu.to_device(wl.make_inputs(n, 1, res, seed=2, bf16=True).reshape(n, res, res, 3), True)
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    opts = sgs.StreamOpts(cache_enabled=1, window_q=q, cache_budget_bytes=0, use_graphs=0, record_latency=0)
    st = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
    encs = [onet.encode(c) for c in cfgs]
    G, hits, missed = None, [], 0
    for t, e in enumerate(encs):
        if G is None:
            hits.append(0.0)
            missed += oracle.encoding_weights(e) * 2
        else:
            hits.append(oracle.hit_ratio(e, G))
            missed += (oracle.encoding_weights(e) - oracle.encoding_weights(oracle.intersect(e, G))) * 2
        if (t + 1) % q == 0:  # every q queries: G = intersection of the last q SubNets
            G = encs[t - q + 1]
            for f in encs[t - q + 2:t + 1]:
                G = oracle.intersect(G, f)
    assert abs(st.hit_ratio - np.mean(hits)) < 1e-9
    assert abs(st.hbm_weight_bytes - missed) < 1


def test_encoding_matches_checker():
    for fam in (wl.TINY, wl.RESNET, wl.MBV3):
        _, onet, gnet = gu.nets(fam, True)
        for c in wl.uniform_stream(fam, 5, seed=3) + [wl.extreme_cfg(fam, False), wl.extreme_cfg(fam, True)]:
            np.testing.assert_array_equal(gnet.subnet_encode(c), onet.encode(c))


def test_bench_launch_configuration_sampled_against_checker():
    # the benchmark's configuration (224x224, batch 1, graphs, cache on, 16 queries in flight) on the
    # first 48 queries of its stream; four sampled queries are recomputed by the checker, all logits
    # must be finite, and the stream must reproduce itself bit for bit
    _, onet, gnet = gu.nets(wl.RESNET, True)
    n, res = 48, 224
    cfgs = wl.uniform_stream(wl.RESNET, 1000, seed=2)[:n]
    xs = wl.make_inputs(n, 1, res, seed=1, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    opts = sgs.StreamOpts(cache_enabled=1, window_q=4, cache_budget_bytes=0, use_graphs=1, record_latency=0, concurrency=16)
    gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
    first = d_out.cpu().numpy().copy()
    d_out.zero_()
    torch.cuda.synchronize()
    gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
    np.testing.assert_array_equal(d_out.cpu().numpy(), first)
    assert np.all(np.isfinite(first))
    agree = []
    for t in (0, 13, 30, 47):
        ref = onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)
        assert gu.rel_err(first[t:t + 1], ref) <= TOL_BF16, t
        agree.append(int(first[t].argmax() == ref[0].argmax()))
    assert sum(agree) >= 3


def _three_argmax_figures(got, ref_store, ref_f32):
    """strict agreement with the bf16-store checker, strict and tie-aware agreement with the plain fp32 checker.
    Tie-aware: the GPU's class counts as agreeing when the checker's own logit at that class is within the error
    bound (2e-2 * max|ref|) of the checker's maximum."""
    g = got.argmax(-1)
    strict_store = float(np.mean(g == ref_store.argmax(-1)))
    strict_f32 = float(np.mean(g == ref_f32.argmax(-1)))
    at_g = np.take_along_axis(ref_f32, g[:, None], axis=1)[:, 0]
    tie_f32 = float(np.mean(ref_f32.max(-1) - at_g <= 2e-2 * np.abs(ref_f32).max(-1)))
    return strict_store, strict_f32, tie_f32


@pytest.mark.parametrize("fam,n", [(wl.RESNET, 200), (wl.MBV3, 120)])
def test_stream_against_plain_fp32_checker_and_argmax(fam, n):
    # The first queries of the benchmark streams, executed as the benchmark does (waves of 32, 4 in flight), against
    # BOTH checker modes: the plain fp32 forward pass on the same bf16-valued weights and inputs (the bar of
    # max|err| <= 2e-2 * max|ref| is meant against this one: it knows nothing about where the GPU rounds), and the
    # forward pass that rounds every stored tensor to bf16.  Top-1: strict agreement with the bf16-store checker and
    # tie-aware agreement with the fp32 checker must reach 99.5 %; strict agreement with the fp32 checker is reported
    # and held to the same bar: with random weights a few top-2 margins are below one bf16 step, if it misses the
    # test says so.
    _, onet, gnet = gu.nets(fam, True)
    res = 224
    cfgs = wl.uniform_stream(fam, 1000, seed=2 if fam == wl.RESNET else 3)[:n]
    xs = wl.make_inputs(n, 1, res, seed=1, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    opts = sgs.StreamOpts(cache_enabled=1, window_q=4, cache_budget_bytes=0, use_graphs=1, record_latency=0, concurrency=4, wave=32)
    gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
    got = d_out.cpu().numpy()
    ref_store = np.stack([onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)[0] for t in range(n)])
    ref_f32 = np.stack([onet.forward(cfgs[t], xs[t], oracle.FP32)[0] for t in range(n)])
    worst_store, worst_f32 = gu.rel_err(got, ref_store), gu.rel_err(got, ref_f32)
    strict_store, strict_f32, tie_f32 = _three_argmax_figures(got, ref_store, ref_f32)
    print(f"family {fam}: worst rel err vs bf16-store checker {worst_store:.2e}, vs fp32 checker {worst_f32:.2e}; "
          f"argmax strict vs bf16-store {strict_store:.3f}, strict vs fp32 {strict_f32:.3f}, tie-aware vs fp32 {tie_f32:.3f}")
    assert worst_f32 <= TOL_BF16
    assert worst_store <= TOL_BF16
    assert strict_store >= 0.995
    assert tie_f32 >= 0.995
    assert strict_f32 >= 0.995, "strict top-1 agreement with the plain fp32 checker is below 99.5 %"


@pytest.mark.parametrize("fam", [wl.RESNET, wl.MBV3])
def test_extreme_configs_against_plain_fp32_checker(fam):
    # smallest and largest SubNet at full resolution, batch 2, one query at a time
    _, onet, gnet = gu.nets(fam, True)
    for i, c in enumerate((wl.extreme_cfg(fam, False), wl.extreme_cfg(fam, True))):
        x = wl.make_inputs(1, 2, 224, seed=40 + i, bf16=True)[0]
        got = gu.gpu_forward(gnet, c, x, True)
        assert gu.rel_err(got, onet.forward(c, x, oracle.FP32)) <= TOL_BF16
        assert gu.rel_err(got, onet.forward(c, x, oracle.BF16_STORE)) <= TOL_BF16
