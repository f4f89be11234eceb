"""AvgNet cache policy (Algorithm 1's caching decision) through the C ABI against the checker's scheduler:
the choices, the hit ratio of Appendix A.4 and the missed weight bytes must agree exactly."""
import numpy as np
import pytest
import torch

import oracle
import paper_2306_17266_b200 as sgs
from paper_2306_17266_b200 import workload as wl
from tests import gpu_util as gu

pytestmark = pytest.mark.gpu


def _expected(onet, cfgs, cands, q, budget_bytes):
    encs = [onet.encode(c) for c in cfgs]
    cand_encs = [oracle.clip_to_budget(onet.encode(c), budget_bytes // 2) for c in cands]  # bf16 weights
    hits, missed, choices = oracle.sched_stream(encs, cand_encs, q)
    updates, prev = 0, None
    for j in choices:
        if prev is None or not np.array_equal(cand_encs[j], prev):
            updates += 1
        prev = cand_encs[j]
    return float(np.mean(hits)), 2.0 * float(sum(missed)), choices, updates


@pytest.mark.parametrize("q,budget,wave", [(4, 0, 0), (1, 48 << 20, 0), (3, 24 << 20, 8), (8, 2 << 20, 4)])
def test_avgnet_policy_matches_checker(q, budget, wave):
    _, onet, gnet = gu.nets(wl.RESNET, True)
    n, res = 26, 64
    cfgs = wl.markov_stream(n, seed=21 + q)
    cands = wl.candidate_cfgs(wl.RESNET, 12, seed=5)
    d_in = gu.to_device(wl.make_inputs(n, 1, res, seed=2, bf16=True).reshape(n, res, res, 3), True)
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    outs = {}
    try:
        gnet.cache_set_candidates(cands)
        for policy in (sgs.SGS_POLICY_AVGNET, sgs.SGS_POLICY_INTERSECTION):
            d_out = torch.zeros((n, 1000), dtype=torch.float32, device="cuda")
            opts = sgs.StreamOpts(cache_enabled=1, window_q=q, cache_budget_bytes=budget, use_graphs=0, record_latency=0,
                                  concurrency=2, wave=wave, policy=policy)
            st = gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, stream.cuda_stream)
            outs[policy] = (st, d_out.cpu().numpy(), gnet.cache_stats())
    finally:
        gnet.cache_set_candidates([])
    st, logits, cs = outs[sgs.SGS_POLICY_AVGNET]
    assert cs.policy == sgs.SGS_POLICY_AVGNET and cs.n_candidates == len(cands)
    hit, missed, choices, updates = _expected(onet, cfgs, cands, q, cs.budget_bytes)
    assert abs(st.hit_ratio - hit) < 1e-12
    assert st.hbm_weight_bytes == missed
    assert cs.decisions == len(choices) == n // q and cs.last_choice == choices[-1]
    assert st.cache_updates == updates
    assert len(set(choices)) > 1 or q >= 8   # the stream really moves the choice (a tiny budget leaves one winner)
    # the policy only moves L2 hints: the logits do not depend on it
    np.testing.assert_array_equal(logits, outs[sgs.SGS_POLICY_INTERSECTION][1])
    assert gnet.cache_stats().n_candidates == 0


def test_avgnet_policy_needs_candidates_and_valid_configs():
    _, _, gnet = gu.nets(wl.TINY, True)
    n, res = 2, 32
    cfgs = wl.uniform_stream(wl.TINY, n, seed=1)
    d_in = gu.to_device(wl.make_inputs(n, 1, res, seed=2, bf16=True).reshape(n, res, res, 3), True)
    d_out = torch.zeros((n, 10), dtype=torch.float32, device="cuda")
    opts = sgs.StreamOpts(cache_enabled=1, window_q=1, policy=sgs.SGS_POLICY_AVGNET)
    with pytest.raises(sgs.SgsError, match="EINVAL"):
        gnet.stream_run(cfgs, d_in.data_ptr(), 1, res, d_out.data_ptr(), opts, torch.cuda.current_stream().cuda_stream)
    with pytest.raises(sgs.SgsError, match="EINVAL"):
        gnet.cache_set_policy(sgs.SGS_POLICY_AVGNET)
    bad = wl.copy_cfg(cfgs[0])
    bad.depth[0] = 99
    with pytest.raises(sgs.SgsError, match="ECONFIG"):
        gnet.cache_set_candidates([cfgs[0], bad])
    assert gnet.cache_stats().n_candidates == 0
    # sgs_subnet_run follows the configured policy too
    gnet.cache_set_candidates(cfgs)
    try:
        gnet.cache_configure(True, 0, 1)
        gnet.cache_set_policy(sgs.SGS_POLICY_AVGNET)
        gnet.subnet_run(cfgs[1], d_in.data_ptr(), 1, res, d_out.data_ptr(), torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        cs = gnet.cache_stats()
        assert cs.decisions == 1 and cs.last_choice == 1
    finally:
        gnet.cache_set_candidates([])
        gnet.cache_configure(False, 0, 4)
