"""CPU pins of the checker's scheduler functions (Algorithm 1's caching decision, Section 3.3): hand-computed
vectors, closed forms and special cases that fix the running average, the distance, tie handling, the
budget clipping and the timing of the decisions."""
import numpy as np

import oracle


def enc(*kc):
    """Encoding from (K, C) pairs with 1x1 kernels."""
    return np.array([v for k, c in kc for v in (k, c, 1)], dtype=np.int32).reshape(-1, 3)


def test_nearest_candidate_on_hand_computed_vectors():
    # window mean = ((4+8)/2, 2) = (6, 2); distances^2: (8,2) -> 4, (6,2) -> 0, (5,4) -> 1 + 4 = 5
    window = [enc((4, 2)), enc((8, 2))]
    cands = [enc((8, 2)), enc((6, 2)), enc((5, 4))]
    assert oracle.nearest_candidate(window, cands) == 1
    # a single-query window: the nearest candidate to the SubNet itself
    assert oracle.nearest_candidate([enc((5, 3))], cands) == 2  # (5,4): 1; (6,2): 1+1 = 2; (8,2): 9+1 = 10
    # ties go to the lowest index; the kernel-size entry takes no part in the distance
    a, b = enc((7, 2)), enc((5, 2))
    assert oracle.nearest_candidate([enc((6, 2))], [a, b]) == 0
    assert oracle.nearest_candidate([enc((6, 2))], [b, a]) == 0
    g3 = np.array([[6, 2, 3]], dtype=np.int32)  # same (K, C), other kernel size
    assert oracle.nearest_candidate([enc((6, 2))], [a, g3]) == 1


def test_average_keeps_what_intersection_loses():
    # Section 3.3: a filter count used by most (not all) SubNets of the window still pulls the choice.
    # Window: three SubNets with K = 8 and one with K = 2: intersection has K = 2, the mean K = 6.5
    window = [enc((8, 4))] * 3 + [enc((2, 4))]
    cands = [enc((2, 4)), enc((6, 4)), enc((8, 4))]
    assert oracle.nearest_candidate(window, cands) == 1  # |6-6.5| < |8-6.5| < |2-6.5|
    inter = window[0]
    for e in window[1:]:
        inter = oracle.intersect(inter, e)
    assert list(inter[0, :2]) == [2, 4]


def test_identical_subnets_choose_themselves():
    e = enc((16, 8), (32, 16), (10, 32))
    others = [enc((8, 8), (16, 8), (10, 16)), enc((16, 16), (32, 32), (10, 64))]
    for pos in range(3):
        cands = others[:pos] + [e] + others[pos:]
        hits, missed, choices = oracle.sched_stream([e] * 6, cands, 2)
        assert choices == [pos] * 3
        assert hits[:2] == [0.0, 0.0] and missed[:2] == [oracle.encoding_weights(e)] * 2  # nothing cached before the first decision
        assert hits[2:] == [1.0] * 4 and missed[2:] == [0] * 4


def test_clip_to_budget_rule():
    e = np.array([5, 2, 1, 5, 4, 1, 5, 1, 1], dtype=np.int32)  # layer weights 10, 20, 5
    assert list(oracle.layer_weights(e)) == [10, 20, 5]
    assert list(oracle.clip_to_budget(e, 100)) == list(e)
    assert list(oracle.clip_to_budget(e, 16)) == [5, 2, 1, 0, 0, 0, 5, 1, 1]   # 10 kept, 20 does not fit, 5 fits
    assert list(oracle.clip_to_budget(e, 9)) == [0, 0, 0, 0, 0, 0, 5, 1, 1]
    assert list(oracle.clip_to_budget(e, 30)) == [5, 2, 1, 5, 4, 1, 0, 0, 0]
    k3 = np.array([2, 2, 3], dtype=np.int32)  # 3x3 kernel: 2*2*9 = 36 weights
    assert list(oracle.layer_weights(k3)) == [36] and list(oracle.clip_to_budget(k3, 35)) == [0, 0, 0]


def test_decisions_every_q_queries_use_the_last_q_subnets():
    small, big = enc((4, 4)), enc((16, 4))
    cands = [small, big]
    stream = [small, small, big, big, big, small]
    hits, missed, choices = oracle.sched_stream(stream, cands, 2)
    # decisions after queries 1, 3, 5 from windows (s,s), (b,b), (b,s): means K = 4, 16, 10 -> small, big, tie -> lowest index
    assert choices == [0, 1, 0]
    # query 2 (big) is served with `small` cached: shared K = 4 of 16, C = 4 of 4
    assert abs(hits[2] - np.sqrt(4 * 4 + 4 * 4) / np.sqrt(16 * 16 + 4 * 4)) < 1e-12
    assert missed[2] == 16 * 4 - 4 * 4
    # queries 4 (big) and 5 (small) with `big` cached: everything shared
    assert hits[4] == 1.0 and hits[5] == 1.0 and missed[4] == 0 and missed[5] == 0
    # q = 1: the cache follows the previous query
    _, _, ch1 = oracle.sched_stream(stream, cands, 1)
    assert ch1 == [0, 0, 1, 1, 1, 0]


# ---- per-query SubNet selection and Algorithm 1 as a whole ------------------------------------------------
ACC = [0.70, 0.74, 0.78, 0.80]
LAT = [1.0, 1.5, 2.5, 2.0]  # SubNet 3 is both faster and more accurate than SubNet 2


def test_select_subnet_strict_accuracy():
    A, L = oracle.STRICT_ACCURACY, oracle.STRICT_LATENCY
    assert oracle.select_subnet(A, 0.60, 0.0, ACC, LAT) == 0      # everything feasible: the fastest
    assert oracle.select_subnet(A, 0.74, 0.0, ACC, LAT) == 1      # accuracy bound is inclusive
    assert oracle.select_subnet(A, 0.75, 0.0, ACC, LAT) == 3      # {2, 3} feasible: 3 is faster
    assert oracle.select_subnet(A, 0.90, 0.0, ACC, LAT) == 3      # nothing feasible: the most accurate
    # the latency bound plays no part under STRICT_ACCURACY (the served latency may exceed it)
    assert oracle.select_subnet(A, 0.75, 0.1, ACC, LAT) == 3
    # ties on latency: the more accurate one, then the lowest index
    assert oracle.select_subnet(A, 0.0, 0.0, [0.7, 0.8, 0.8], [1.0, 1.0, 1.0]) == 1
    assert oracle.select_subnet(L, 0.0, 5.0, [0.8, 0.8], [2.0, 1.0]) == 1   # ties on accuracy: the faster one


def test_select_subnet_strict_latency():
    L = oracle.STRICT_LATENCY
    assert oracle.select_subnet(L, 0.0, 3.0, ACC, LAT) == 3       # everything feasible: the most accurate
    assert oracle.select_subnet(L, 0.0, 1.5, ACC, LAT) == 1       # latency bound is inclusive
    assert oracle.select_subnet(L, 0.0, 1.9, ACC, LAT) == 1
    assert oracle.select_subnet(L, 0.0, 2.0, ACC, LAT) == 3
    assert oracle.select_subnet(L, 0.0, 0.5, ACC, LAT) == 0       # nothing feasible: the fastest
    assert oracle.select_subnet(L, 0.99, 1.2, ACC, LAT) == 0      # the accuracy bound plays no part


def test_selection_depends_on_the_cache_state_column():
    # the same query picks another SubNet once the cached SubGraph makes that SubNet fast enough
    table = [[1.0, 1.0, 1.2], [1.4, 2.0, 2.2]]          # columns: G_0, G_1, empty cache
    acc = [0.70, 0.80]
    L = oracle.STRICT_LATENCY
    assert oracle.select_subnet(L, 0.0, 1.5, acc, [r[0] for r in table]) == 1
    assert oracle.select_subnet(L, 0.0, 1.5, acc, [r[1] for r in table]) == 0
    assert oracle.select_subnet(L, 0.0, 1.5, acc, [r[2] for r in table]) == 0


def test_algorithm_1_hand_run():
    # two SubNets (small, big), two candidates equal to them; q = 2
    small, big = enc((4, 4)), enc((16, 4))
    table = [[1.0, 1.1, 1.2],      # small: G_0 = small cached, G_1 = big cached, nothing cached
             [2.0, 1.4, 2.4]]      # big is fast only while the big SubGraph is cached
    acc = [0.70, 0.80]
    A, L = oracle.STRICT_ACCURACY, oracle.STRICT_LATENCY
    queries = [(L, 0.0, 2.0),      # empty cache: big takes 2.4 > 2.0 -> small
               (A, 0.75, 0.0),     # accuracy forces big; window (small, big): mean K = 10, tie -> G_0
               (L, 0.0, 2.0),      # G_0 cached: big takes 2.0 <= 2.0 -> big
               (L, 0.0, 1.5),      # G_0: big 2.0 > 1.5 -> small; window (big, small): tie -> G_0 again
               (A, 0.75, 0.0),     # big
               (A, 0.75, 0.0),     # big; window (big, big) -> G_1
               (L, 0.0, 1.5),      # G_1: big takes 1.4 -> big
               (L, 0.0, 1.05)]     # G_1: small 1.1, big 1.4, none feasible -> the fastest = small
    served, states = oracle.sushi_sched(queries, acc, table, [small, big], [small, big], 2)
    assert served == [0, 1, 1, 0, 1, 1, 1, 0]
    assert states == [2, 2, 0, 0, 0, 0, 1, 1]
