"""GPU parity of persistent execution (the whole stream as one launch of the SubNet kernel) against the CPU checker.

Same tolerance as the other bf16 parity tests: max|err| <= 2e-2 * max|ref| per output row, against the checker run
with the same storage rounding points and against the plain fp32 checker.
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


def _run(gnet, cfgs, d_in, res, host=False, cache=1, window_q=4):
    n = len(cfgs)
    stream = torch.cuda.Stream()
    opts = sgs.StreamOpts(cache_enabled=cache, window_q=window_q, cache_budget_bytes=0, use_graphs=0, record_latency=0,
                          concurrency=1, wave=0, policy=0, persistent=1)
    if host:
        h_out = np.zeros((n, 1000), dtype=np.float32)
        h_in = d_in.cpu().view(torch.int16).numpy()
        st = gnet.stream_run(cfgs, h_in, 1, res, h_out, opts, stream.cuda_stream, host=True)
        return h_out, st
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    st = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
    return d_out.cpu().numpy(), st


@pytest.mark.parametrize("res,n", [(64, 9), (96, 7)])
def test_persistent_stream_matches_checker(res, n):
    # uniform configs plus the smallest and the largest SubNet; fewer queries than SMs, so every block serves at most one
    _, onet, gnet = gu.nets(wl.MBV3, True)
    cfgs = wl.uniform_stream(wl.MBV3, n - 2, seed=21) + [wl.extreme_cfg(wl.MBV3, False), wl.extreme_cfg(wl.MBV3, True)]
    xs = wl.make_inputs(n, 1, res, seed=6, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    got, st = _run(gnet, cfgs, d_in, res)
    assert st.kernel_launches == 1 and st.n_queries == n
    assert np.all(np.isfinite(got))
    for t in range(n):
        ref = onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)
        assert gu.rel_err(got[t:t + 1], ref) <= TOL_BF16, t
        plain = onet.forward(cfgs[t], xs[t], oracle.FP32)
        assert gu.rel_err(got[t:t + 1], plain) <= TOL_BF16, t
    again, _ = _run(gnet, cfgs, d_in, res)
    np.testing.assert_array_equal(again, got)          # which block serves a query does not change its bits
    hosted, _ = _run(gnet, cfgs, d_in, res, host=True)
    np.testing.assert_array_equal(hosted, got)


def test_persistent_stream_many_queries_per_block_equals_the_wave_path():
    # 400 queries on 148 blocks: every block serves several queries out of the same scratch area.  The layer-by-layer
    # wave path (itself checked against the checker elsewhere) computes the same layers with other kernels: the two
    # agree within the parity bound on every query, and sampled queries are compared with the checker directly.
    _, onet, gnet = gu.nets(wl.MBV3, True)
    n, res = 400, 64
    cfgs = wl.uniform_stream(wl.MBV3, n, seed=33)
    xs = wl.make_inputs(n, 1, res, seed=8, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    got, st = _run(gnet, cfgs, d_in, res)
    assert st.kernel_launches == 1
    stream = torch.cuda.Stream()
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    wopts = sgs.StreamOpts(cache_enabled=1, window_q=4, cache_budget_bytes=0, use_graphs=0, record_latency=0,
                           concurrency=2, wave=32)
    wst = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), wopts, stream.cuda_stream)
    waves = d_out.cpu().numpy()
    for t in range(n):
        assert gu.rel_err(got[t:t + 1], waves[t:t + 1]) <= TOL_BF16, t
    for t in (0, 147, 148, 313, 399):
        ref = onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)
        assert gu.rel_err(got[t:t + 1], ref) <= TOL_BF16, t
    assert st.useful_flops == wst.useful_flops and st.weight_bytes == wst.weight_bytes


def test_weight_buffer_in_shared_memory_changes_no_bit():
    # With the cache on, every block keeps the chosen SubGraph's first pointwise layers in shared memory and multiplies
    # them in place; filters and channels of a query beyond the box still come through the ring.  The arithmetic of an
    # output column does not depend on where its filter came from, so logits are bit-identical with the buffer off,
    # small (a box that ends inside a layer's neighbours) and at its largest; the accounting is against what is held.
    _, _, gnet = gu.nets(wl.MBV3, True)
    n, res = 200, 96
    cfgs = wl.markov_stream(n, seed=12, family=wl.MBV3)
    d_in = gu.to_device(wl.make_inputs(n, 1, res, seed=13, bf16=True).reshape(n, res, res, 3), True)
    off, st_off = _run(gnet, cfgs, d_in, res, cache=0)
    assert st_off.hit_ratio == 0 and st_off.hbm_weight_bytes == st_off.weight_bytes
    try:
        for kb in (8, 40, 56):
            gnet.set_option("persistent_held_kb", kb)
            for q in (1, 4):
                on, st_on = _run(gnet, cfgs, d_in, res, cache=1, window_q=q)
                np.testing.assert_array_equal(on, off)
                assert 0 < st_on.hit_ratio < 1 and st_on.hbm_weight_bytes < st_on.weight_bytes
                assert st_on.cache_updates == 1
        gnet.set_option("persistent_held_kb", 0)
        none, st_none = _run(gnet, cfgs, d_in, res, cache=1)
        np.testing.assert_array_equal(none, off)
        assert st_none.hbm_weight_bytes == st_none.weight_bytes
        with pytest.raises(sgs.SgsError):
            gnet.set_option("persistent_held_kb", 4096)
    finally:
        gnet.set_option("persistent_held_kb", 16)


def test_persistent_stream_full_resolution_sampled():
    _, onet, gnet = gu.nets(wl.MBV3, True)
    n, res = 160, 224
    cfgs = wl.uniform_stream(wl.MBV3, n, seed=3)
    xs = wl.make_inputs(n, 1, res, seed=4, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    got, _ = _run(gnet, cfgs, d_in, res)
    assert np.all(np.isfinite(got))
    for t in (0, 150, 159):
        ref = onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)
        assert gu.rel_err(got[t:t + 1], ref) <= TOL_BF16, t


def test_persistent_refusals():
    _, _, rnet = gu.nets(wl.RESNET, True)
    cfgs = wl.uniform_stream(wl.RESNET, 2, seed=1)
    d_in = gu.to_device(wl.make_inputs(2, 1, 64, seed=1, bf16=True).reshape(2, 64, 64, 3), True)
    with pytest.raises(sgs.SgsError) as e:
        _run(rnet, cfgs, d_in, 64)
    assert e.value.status == sgs.binding.SGS_EUNSUPPORTED
    _, _, gnet = gu.nets(wl.MBV3, True)
    mcfgs = wl.uniform_stream(wl.MBV3, 2, seed=1)
    d_out = torch.zeros((4, 1000), dtype=torch.float32, device="cuda")
    d_in2 = gu.to_device(wl.make_inputs(2, 2, 64, seed=1, bf16=True).reshape(4, 64, 64, 3), True)
    opts = sgs.StreamOpts(cache_enabled=0, window_q=1, persistent=1)
    with pytest.raises(sgs.SgsError) as e:
        gnet.stream_run(mcfgs, d_in2.data_ptr(), 2, 64, d_out.data_ptr(), opts, 0)
    assert e.value.status == sgs.binding.SGS_EINVAL
    # an empty stream is fine
    st = gnet.stream_run(mcfgs[:0], d_in2.data_ptr(), 1, 64, d_out.data_ptr(), opts, 0)
    assert st.n_queries == 0
