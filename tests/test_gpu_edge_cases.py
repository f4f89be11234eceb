"""Edge cases of the GPU path: empty streams, smallest and odd resolutions, largest config at full
size on sampled outputs, repeated configs (plan reuse), and argument errors that must not launch."""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def test_empty_stream_and_bad_options():
    _, _, gnet = gu.nets(wl.RESNET, True)
    stream = torch.cuda.Stream()
    x = torch.zeros((1, 64, 64, 3), dtype=torch.bfloat16, device="cuda")
    out = torch.zeros((1, 1000), device="cuda")
    st = gnet.stream_run([], x.data_ptr(), 1, 64, out.data_ptr(), None, stream.cuda_stream)
    assert st.n_queries == 0 and st.kernel_launches == 0
    cfg = [wl.extreme_cfg(wl.RESNET, False)]
    for bad in (sgs.StreamOpts(cache_enabled=1, window_q=0, use_graphs=1), sgs.StreamOpts(cache_enabled=1, window_q=4, concurrency=99)):
        with pytest.raises(sgs.SgsError) as e:
            gnet.stream_run(cfg, x.data_ptr(), 1, 64, out.data_ptr(), bad, stream.cuda_stream)
        assert e.value.status == sgs.binding.SGS_EINVAL
    with pytest.raises(sgs.SgsError):
        gnet.subnet_run(cfg[0], x.data_ptr(), 0, 64, out.data_ptr())  # batch 0
    with pytest.raises(sgs.SgsError):
        gnet.subnet_run(cfg[0], x.data_ptr(), 1, 4, out.data_ptr())   # resolution too small


@pytest.mark.parametrize("fam,res", [(wl.TINY, 8), (wl.TINY, 33), (wl.RESNET, 32), (wl.RESNET, 80), (wl.MBV3, 32), (wl.MBV3, 96)])
def test_small_and_odd_resolutions(fam, res):
    # 32x32 leaves 1x1 feature maps in the last stage; 33 / 80 / 96 give odd maps (3, 5 ...) and tiles
    # that straddle image borders in every layer
    _, onet, gnet = gu.nets(fam, True)
    for i, c in enumerate([wl.extreme_cfg(fam, False), wl.extreme_cfg(fam, True)] + wl.uniform_stream(fam, 2, seed=41)):
        x = wl.make_inputs(1, 2, res, seed=50 + i, bf16=True)[0]
        ref = onet.forward(c, x, oracle.BF16_STORE)
        got = gu.gpu_forward(gnet, c, x, True)
        assert np.all(np.isfinite(got))
        assert gu.rel_err(got, ref) <= 2e-2, (fam, res, i)


def test_largest_and_smallest_config_full_size():
    # the two extreme SubNets at the benchmark's resolution and at batch 16 (the launch configuration of
    # the batch-16 suites); the checker computes the first two images of the batch
    _, onet, gnet = gu.nets(wl.RESNET, True)
    for largest in (False, True):
        c = wl.extreme_cfg(wl.RESNET, largest)
        x = wl.make_inputs(1, 16, 224, seed=7, bf16=True)[0]
        got = gu.gpu_forward(gnet, c, x, True)
        ref = onet.forward(c, x[:2], oracle.BF16_STORE)
        assert gu.rel_err(got[:2], ref) <= 2e-2
        # every image of the batch went through the same kernels: a permuted batch gives permuted logits
        perm = np.array([5, 0, 15, 3, 1, 2, 4, 6, 7, 8, 9, 10, 11, 12, 13, 14])
        got_p = gu.gpu_forward(gnet, c, x[perm], True)
        np.testing.assert_array_equal(got_p, got[perm])


def test_repeated_configs_reuse_plans_and_agree():
    _, _, gnet = gu.nets(wl.RESNET, True)
    c = wl.uniform_stream(wl.RESNET, 1, seed=77)[0]
    n, res = 9, 64
    cfgs = [c] * n
    xs = wl.make_inputs(1, 1, res, seed=3, bf16=True)
    x_all = np.repeat(xs, n, axis=0).reshape(n, res, res, 3)
    d_in = gu.to_device(x_all, True)
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    opts = sgs.StreamOpts(cache_enabled=1, window_q=4, use_graphs=1, record_latency=0, concurrency=3)
    st = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
    got = d_out.cpu().numpy()
    for i in range(1, n):
        np.testing.assert_array_equal(got[i], got[0])
    assert st.plan_misses <= 3                      # one plan per slot at most
    assert st.hit_ratio > 0.5                       # same SubNet over and over: after the first window the
    assert st.hbm_weight_bytes < 0.6 * st.weight_bytes  # cached SubGraph is the SubNet itself (paper App. A.4)


def test_a_wait_that_runs_out_is_reported_and_leaves_the_device_usable():
    # Every device-side wait of the kernels carries a time limit.  A one-block test kernel of the library waits on a
    # barrier nothing arrives at (limit 1 ms): it must return by itself, the status word must say so, the next stream
    # call must report SGS_ETIMEOUT, and after clearing the status the same stream must pass parity again.
    _, onet, gnet = gu.nets(wl.RESNET, True)
    n, res = 4, 64
    cfgs = wl.uniform_stream(wl.RESNET, n, seed=61)
    xs = wl.make_inputs(n, 1, res, seed=9, bf16=True)
    d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
    d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    opts = sgs.StreamOpts(cache_enabled=1, window_q=2, record_latency=0, concurrency=1, wave=4)
    torch.cuda.synchronize()
    assert sgs.device_status() == 0
    try:
        sgs.debug_expire_wait(1000, stream.cuda_stream)
        torch.cuda.synchronize()               # returns: the kernel ended on its own
        assert sgs.device_status() != 0
        with pytest.raises(sgs.SgsError) as e:
            gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
        assert e.value.status == sgs.binding.SGS_ETIMEOUT
    finally:
        sgs.device_status_clear()
    assert sgs.device_status() == 0
    gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
    got = d_out.cpu().numpy()
    for t in range(n):
        assert gu.rel_err(got[t:t + 1], onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)) <= 2e-2


def test_device_allocation_failure_is_reported_and_survivable():
    # fault injection on the host: the handle's device allocations are made to fail while its workspaces have to grow
    # (a larger resolution, more wave slots).  The call must come back with SGS_ENOMEM, nothing may be left half
    # grown, and with allocations working again the same handle must serve the same stream correctly.
    blob = wl.make_blob(wl.RESNET, seed=0, bf16_weights=True)
    onet = oracle.Net(wl.RESNET, blob)
    gnet = sgs.SuperNet(wl.RESNET, blob, sgs.SGS_BF16)
    n = 6
    cfgs = wl.uniform_stream(wl.RESNET, n, seed=71)
    stream = torch.cuda.Stream()
    out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")

    def run(res, wave, conc):
        xs = wl.make_inputs(n, 1, res, seed=10, bf16=True)
        d_in = gu.to_device(xs.reshape(n, res, res, 3), True)
        opts = sgs.StreamOpts(cache_enabled=1, window_q=2, record_latency=0, concurrency=conc, wave=wave)
        gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, out.data_ptr(), opts, stream.cuda_stream)
        return xs, out.cpu().numpy().copy()

    run(32, 2, 1)                                   # small workspaces exist
    for after in (0, 3, 9):                         # fail at once, and in the middle of growing several slots
        gnet.set_option("fail_alloc_after", after)
        with pytest.raises(sgs.SgsError) as e:
            run(96, 3, 2)                           # larger maps and more slots: everything has to grow
        assert e.value.status == sgs.binding.SGS_ENOMEM
        gnet.set_option("fail_alloc_after", -1)
        xs, got = run(64, 2, 1)                     # the handle still works ...
        assert gu.rel_err(got[:1], onet.forward(cfgs[0], xs[0], oracle.BF16_STORE)) <= 2e-2
    xs, got = run(96, 3, 2)                         # ... and can grow once memory is there
    for t in (0, 5):
        assert gu.rel_err(got[t:t + 1], onet.forward(cfgs[t], xs[t], oracle.BF16_STORE)) <= 2e-2
    assert sgs.device_status() == 0
    gnet.close()
