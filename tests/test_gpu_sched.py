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


@pytest.mark.parametrize("family,q,budget,wave", [(wl.RESNET, 4, 0, 0), (wl.RESNET, 1, 48 << 20, 0), (wl.RESNET, 3, 24 << 20, 8),
                                                  (wl.RESNET, 8, 2 << 20, 4), (wl.MBV3, 2, 0, 0), (wl.MBV3, 3, 6 << 20, 8)])
def test_avgnet_policy_matches_checker(family, q, budget, wave):
    _, onet, gnet = gu.nets(family, True)
    n, res = 26, 64
    cfgs = wl.markov_stream(n, seed=21 + q, family=family)
    cands = wl.candidate_cfgs(family, 12, seed=5)
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


def _sched_case(q, budget, measured):
    _, onet, gnet = gu.nets(wl.RESNET, True)
    res = 64
    subnets = wl.candidate_cfgs(wl.RESNET, 8, seed=11)
    cands = wl.candidate_cfgs(wl.RESNET, 6, seed=5)
    acc = wl.proxy_accuracy([gnet.subnet_cost(c, 1, res)[0] for c in subnets])
    d_in = gu.to_device(wl.make_inputs(1, 1, res, seed=2, bf16=True).reshape(1, res, res, 3), True)
    d_out = torch.zeros((1, 1000), dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    gnet.cache_set_candidates(cands)
    sched = None
    try:
        gnet.cache_configure(True, budget, q)
        budget_bytes = gnet.cache_stats().budget_bytes
        sched = sgs.Scheduler(gnet, subnets, acc, q)
        assert (sched.n_subnets, sched.n_columns) == (8, 7)
        assert gnet.cache_stats().policy == 2 and gnet.cache_stats().cached_subgraph_bytes == 0
        if measured:
            sched.measure(d_in.data_ptr(), 1, res, d_out.data_ptr(), reps=3, flush_bytes=160 << 20, stream=stream.cuda_stream)
            table = sched.get_table()
            assert table.shape == (8, 7) and np.all(table > 0) and np.all(table < 50)   # milliseconds of a batch-1 query
            assert table[1].mean() > table[0].mean()                                    # the largest SubNet is slower than the smallest
        else:
            # a synthetic table: latency grows with the SubNet, shrinks with the weights the column's SubGraph shares with it
            rng = np.random.default_rng(3)
            encs_ = [onet.encode(c) for c in subnets]
            cand_ = [oracle.clip_to_budget(onet.encode(c), budget_bytes // 2) for c in cands] + [np.zeros_like(encs_[0])]
            table = np.array([[1e-6 * oracle.encoding_weights(e) * (1.0 - 0.5 * oracle.encoding_weights(oracle.intersect(e, g)) / oracle.encoding_weights(e))
                               for g in cand_] for e in encs_]) + rng.uniform(0, 0.01, (8, 7))
            sched.set_table(table)
            np.testing.assert_array_equal(sched.get_table(), table)
        n = 90
        policy, a_t, l_t = wl.sched_queries(n, seed=17 + q, accuracy=acc, latency=table.reshape(-1))
        got_sub, got_state = [], []
        for lo, hi in ((0, 1), (1, 31), (31, 31), (31, n)):     # state carries over calls of any length
            s, c = sched.step(policy[lo:hi], a_t[lo:hi], l_t[lo:hi])
            got_sub += list(s)
            got_state += list(c)
        encs = [onet.encode(c) for c in subnets]
        cand_encs = [oracle.clip_to_budget(onet.encode(c), budget_bytes // 2) for c in cands]
        served, states = oracle.sushi_sched(list(zip(policy.tolist(), a_t.tolist(), l_t.tolist())), acc.tolist(), table.tolist(), encs, cand_encs, q)
        assert got_sub == served and got_state == states
        assert len(set(served)) >= 3 and len(set(states)) >= 2      # the queries and the table really move both decisions
        # the scheduler's last decision is what the device cache holds, and running queries does not move it
        final = oracle.nearest_candidate([encs[i] for i in served[-q:]], cand_encs) if n % q == 0 else None
        cs = gnet.cache_stats()
        if final is not None:
            assert cs.last_choice == final
        assert cs.policy == 2 and cs.cached_subgraph_bytes == 2 * oracle.encoding_weights(cand_encs[cs.last_choice])
        for i in served[-3:]:
            cfg = sched.subnet(i)
            gnet.subnet_run(cfg, d_in.data_ptr(), 1, res, d_out.data_ptr(), stream.cuda_stream)
            stream.synchronize()
            ref = onet.forward(cfg, wl.make_inputs(1, 1, res, seed=2, bf16=True).reshape(1, res, res, 3), oracle.BF16_STORE)
            assert gu.rel_err(d_out.cpu().numpy(), ref) < 2e-2
        assert gnet.cache_stats().last_choice == cs.last_choice
    finally:
        if sched is not None:
            sched.close()
        gnet.cache_set_candidates([])
        gnet.cache_configure(False, 0, 4)
    assert gnet.cache_stats().policy == 0 and gnet.cache_stats().enabled == 0


def test_scheduler_on_a_synthetic_table_matches_checker():
    _sched_case(q=3, budget=24 << 20, measured=False)
    _sched_case(q=1, budget=0, measured=False)


def test_scheduler_on_its_measured_table_matches_checker():
    _sched_case(q=5, budget=32 << 20, measured=True)


def test_scheduler_argument_errors():
    _, _, gnet = gu.nets(wl.TINY, True)
    cfgs = wl.uniform_stream(wl.TINY, 3, seed=1)
    with pytest.raises(sgs.SgsError, match="EINVAL"):       # no candidate set
        sgs.Scheduler(gnet, cfgs, [0.1, 0.2, 0.3], 2)
    gnet.cache_set_candidates(cfgs[:2])
    try:
        with pytest.raises(sgs.SgsError, match="EINVAL"):
            sgs.Scheduler(gnet, cfgs, [0.1, 0.2, 0.3], 0)
        s = sgs.Scheduler(gnet, cfgs, [0.1, 0.2, 0.3], 2)
        with pytest.raises(sgs.SgsError, match="EINVAL"):
            s.step([7], [0.0], [0.0])
        with pytest.raises(ValueError):
            s.set_table(np.zeros((2, 2)))
        sub, state = s.step([], [], [])
        assert len(sub) == 0
        gnet.cache_set_candidates(cfgs)                      # another set under a live scheduler: refused, not followed
        with pytest.raises(sgs.SgsError, match="EINVAL"):
            s.step([0], [0.0], [0.0])
        gnet.cache_set_candidates(cfgs[:2])
        sub, _ = s.step([0], [0.0], [0.0])
        assert len(sub) == 1
        s.close()
    finally:
        gnet.cache_set_candidates([])
        gnet.cache_configure(False, 0, 4)
