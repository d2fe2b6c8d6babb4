"""The retrieval-aware admission / eviction rule (Sec. 5.2) on hand-worked traces."""
import numpy as np

from paper_2609_32999_b200 import residency as rs
from paper_2609_32999_b200 import workloads as wl


def test_scores_and_first_retrieval_is_not_admitted():
    c = rs.ReuseScoreCache(capacity_blocks=10, window=3)
    assert c.request([("a", 4)]) == [False]
    assert abs(c.score("a") - 1.05) < 1e-12 and "a" not in c.resident          # s = 1*1 + 0.05*1 < theta
    assert c.request([("a", 4)]) == [False]                                     # second retrieval: s = 2.1 >= 2
    assert abs(c.score("a") - 2.1) < 1e-12 and c.resident == {"a": 4}
    assert c.request([("a", 4), ("b", 4)]) == [True, False]
    assert abs(c.score("a") - 3.15) < 1e-12


def test_window_forgets_and_cumulative_count_stays():
    c = rs.ReuseScoreCache(capacity_blocks=10, window=2)
    for _ in range(3):
        c.request([("a", 1)])
    assert c.recent["a"] == 2 and c.total["a"] == 3                             # f_W capped by the window
    c.request([("x", 1)]); c.request([("y", 1)])
    assert c.recent.get("a", 0) == 0 and abs(c.score("a") - 0.15) < 1e-12       # only the cumulative part is left


def test_eviction_takes_strictly_lower_scores_only_and_whole_units():
    c = rs.ReuseScoreCache(capacity_blocks=8, window=100)
    for _ in range(3):
        c.request([("hot", 4)])
    for _ in range(2):
        c.request([("warm", 4)])
    assert c.resident == {"hot": 4, "warm": 4} and c.used == 8
    # a candidate with the same score as the weakest resident is refused ...
    for _ in range(2):
        c.request([("cand", 4)])
    assert abs(c.score("cand") - c.score("warm")) < 1e-12 and "cand" not in c.resident
    # ... one more retrieval makes it strictly better: the weakest resident goes, as a whole
    c.request([("cand", 4)])
    assert set(c.resident) == {"hot", "cand"} and c.used == 8
    # a unit larger than what lower-scored residents can free is not admitted and evicts nothing
    for _ in range(3):
        c.request([("big", 9)])
    assert set(c.resident) == {"hot", "cand"}


def test_capacity_is_never_exceeded_and_policy_beats_lru_on_skewed_trace():
    rng = np.random.default_rng(0)
    trace = []
    for _ in range(1500):
        ranks = wl.zipf_ranks(rng, 5, 2000, 1.0, distinct=True)
        trace.append([(k, 8) for k in ranks])
    cap = 8 * 150
    pol = rs.ReuseScoreCache(cap, rs.ReuseScoreCache.window_for(cap, 40))
    lru, lfu = rs.LRUCache(cap), rs.LFUCache(cap)
    hp = 0
    n = 0
    for req in trace:
        r = pol.request(req)
        assert pol.used <= cap and pol.used == sum(pol.resident.values())
        hp += sum(r); n += len(r)
    h_lru, h_lfu = rs.hit_ratio(lru, trace), rs.hit_ratio(lfu, trace)
    assert lru.used <= cap and lfu.used <= cap
    assert hp / n > h_lru                    # one-time retrievals do not churn the cache
    assert 0.2 < hp / n < 0.9 and 0.1 < h_lfu < 0.9


def test_workloads_with_policy_are_valid_and_miss_some_units():
    from oracle import tessera_oracle as orc
    base = wl.config(3, requests_override=3)
    w = wl.config(3, requests_override=3, policy="reuse")
    assert orc.placement(w)[0] == 0
    n_cached = sum(1 for u in range(len(w.unit_len)) if w.unit_page_off[u + 1] > w.unit_page_off[u])
    assert 0 < n_cached < len(w.unit_len)            # some hits, some misses
    assert w.n_q > base.n_q                          # missed units are recomputed in full
    assert wl.config(3, requests_override=3).n_q == base.n_q     # default residency unchanged
