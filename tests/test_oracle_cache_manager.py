"""Pins for the cache-manager oracle (Eq. 2, PreferDegree, Algorithms 1 and 2): numbers worked by hand
from the paper's formulas, telescoping and threshold properties the text states."""
import math

import pytest

from oracle import cache_manager as cm

PURE_ATTENTION = (0.0, 0.0, 0.0, 0.0, 1.0)       # E_C = W / C


def test_prefill_time_by_hand():
    # Eq. 2 with d=1, a=2, b=3, c=4, alpha=5 at R=10, P=20, C=2: W = 200 + 55 = 255
    assert cm.remaining_workload(10, 20) == 255
    assert cm.prefill_time((1, 2, 3, 4, 5), 10, 20, 2) == 1 + 20 + 60 + (40 + 5 * 255) / 2


def test_prefer_degree_by_hand():
    # L = 100, E_C = W/C.  Worker 0: degree 1 with 60 cached tokens: W(40,60) = 2400 + 820 = 3220.
    # Worker 1: degree 4 without cache: W(100,0) = 5050 -> 1262.5.  C_min = 1.
    workers = [(1, 60), (4, 0)]
    # lambda = 0: pure service time, the degree-4 worker wins
    assert cm.prefer_degree(PURE_ATTENTION, 100, workers, 1.0, 0.0) == (1, 4)
    # lambda = 1: worker 1 pays 4 * 1262.5 - 1 * 5050 = 0 extra (perfect scaling), still wins
    assert cm.prefer_degree(PURE_ATTENTION, 100, workers, 1.0, 1.0) == (1, 4)
    # with a per-token cost that does not scale (a = 100): s0 = 4000 + 3220 = 7220, s1 = 10000 + 1262.5;
    # occupying 4 GPUs costs 4 * 11262.5 - 15050 = 30000 more -> the degree-1 worker wins at lambda = 1
    model = (0.0, 100.0, 0.0, 0.0, 1.0)
    assert cm.prefer_degree(model, 100, workers, 1.0, 0.0) == (0, 1)
    assert cm.prefer_degree(model, 100, workers, 1.0, 1.0) == (0, 1)
    # ties go to the first worker
    assert cm.prefer_degree(PURE_ATTENTION, 100, [(2, 0), (2, 0)], 1.0, 0.5) == (0, 2)


def _two_worker_trie():
    t = cm.Trie([1, 4], block_tokens=64)
    t.set_worker(10, 1)
    t.set_worker(20, 4)
    return t


def test_paths_and_replica_count():
    t = _two_worker_trie()
    z3 = t.add_replica([7, 8, 9], 10)
    t.add_replica([7, 8], 20)
    t.add_replica([7, 5], 20)
    assert t.prefix_length(z3) == 192
    assert t.matched_path([7, 8, 9, 1]) == [1, 2, 3]                 # the fourth block is unknown
    assert t.matched_path([6]) == []
    assert t.reused_path([7, 8, 9], 20) == [1, 2] and t.reused_path([7, 8, 9], 10) == [1, 2, 3]
    assert [t.replica_count(z, 4) for z in (1, 2, 3, 4)] == [1, 1, 0, 1]
    assert [t.replica_count(z, 1) for z in (1, 2, 3, 4)] == [1, 1, 1, 0]
    assert not t.drop_replica(2, 10)                                  # worker 10 still retains the child 3
    assert t.drop_replica(3, 10) and t.drop_replica(2, 10) and t.replica_count(2, 1) == 0
    t.set_worker(20, 0)                                               # the worker leaves: all its records go
    assert [t.replica_count(z, 4) for z in (1, 2, 4)] == [0, 0, 0]


def test_algorithm1_by_hand():
    # Request of L = 256 tokens matching three blocks; worker 10 (degree 1) holds all three, no degree-4
    # worker holds any.  Preferred degree 4, E_C = W / C.
    t = _two_worker_trie()
    t.add_replica([7, 8, 9], 10)
    t.update([7, 8, 9, 2], 256, 10, 4, PURE_ATTENTION)
    assert [t.access[z][1] for z in (1, 2, 3)] == [1.0, 1.0, 1.0] and t.access[1][4] == 0.0
    # W(256,0)=32896, W(192,64)=30816, W(128,128)=24640, W(64,192)=14368
    assert [t.missed[z][4] for z in (1, 2, 3)] == [(32896 - 30816) / 4, (30816 - 24640) / 4, (24640 - 14368) / 4]
    assert all(t.missed[z][1] == 0.0 for z in (1, 2, 3))
    # nodes that do have a replica at the preferred degree lose nothing
    t.add_replica([7], 20)
    t.update([7, 8, 9], 256, 20, 4, PURE_ATTENTION)
    assert t.missed[1][4] == (32896 - 30816) / 4 and t.missed[2][4] == 2 * (30816 - 24640) / 4
    assert t.access[1][4] == 1.0 and t.access[2][4] == 0.0            # worker 20 reused one block only


@pytest.mark.parametrize("model", [PURE_ATTENTION, (3e-4, 2e-7, 5e-8, 1e-6, 4e-11)])
def test_missed_benefits_telescope(model):
    # each node adds the benefit of extending its parent's prefix by one block, so along an unreplicated
    # path the sum is E(L, 0) - E(L - P, P): longer prefixes are not counted twice
    t = _two_worker_trie()
    blocks = list(range(100, 120))
    t.add_replica(blocks, 10)
    L = 20 * 64 + 17
    t.update(blocks, L, 10, 4, model)
    total = sum(t.missed[z][4] for z in range(1, 21))
    want = cm.prefill_time(model, L, 0, 4) - cm.prefill_time(model, L - 1280, 1280, 4)
    assert math.isclose(total, want, rel_tol=1e-12)
    assert all(t.missed[z][4] > 0 for z in range(1, 21))              # caching one more block always helps


def test_algorithm2_thresholds_and_decay():
    t = cm.Trie([1, 4], 64)
    for w, c in ((10, 1), (11, 1), (20, 4), (21, 4)):
        t.set_worker(w, c)
    a = t.add_replica([1], 10)            # node 1: one degree-1 replica
    t.add_replica([1], 11)                # ... now two
    b = t.add_replica([2], 10)            # node 2: one degree-1 replica
    c = t.add_replica([1, 3], 20)         # node 3 under node 1: one degree-4 replica (20 also holds node 1)
    t.access[a][1] = 8.0                  # r = 2: 8 > 2*3 -> intra;   exactly 6 would not be
    t.access[b][1] = 0.5                  # r = 1: 0.5 < 1*1 -> reclaim
    t.access[c][4] = 3.0                  # r = 1: neither (1 <= 3 <= 3)
    t.access[a][4] = 1.0                  # r = 1 (worker 20): exactly the reclaim threshold -> not reclaimed
    t.missed[b][4] = 5.0                  # r = 0 at degree 4: 5 > 4 -> inter
    t.missed[c][1] = 4.0                  # r = 0 at degree 1: exactly the threshold -> not listed
    inter, intra, reclaim, totals = t.scan(4.0, 3.0, 1.0, 0.5, 8)
    assert totals == (1, 1, 1)
    assert inter == [(b, 4, 0, 1, 5.0)]           # one block to copy to either degree-4 worker
    assert intra == [(a, 1, 2, 0, 4.0)]           # access per replica 8/2; no degree-1 worker lacks node 1
    assert reclaim == [(b, 1, 1, 0, 0.5)]
    # decay after the lists are made, on both statistics, everywhere
    assert t.access[a][1] == 4.0 and t.access[b][1] == 0.25 and t.missed[b][4] == 2.5 and t.missed[c][1] == 2.0
    # hysteresis (theta_reclaim < theta_intra): no (node, degree) is in both lists
    assert not set(x[:2] for x in intra) & set(x[:2] for x in reclaim)


def test_scan_ranking_and_bound():
    t = cm.Trie([2], 64)
    for w in range(4):
        t.set_worker(w, 2)
    z = [t.add_replica([k], 0) for k in range(5)]          # five one-block prefixes on worker 0
    t.add_replica([0, 9], 1)                               # worker 1 holds block 0 and a child
    for i, n in enumerate(z):
        t.access[n][2] = 10.0 + i
    t.access[z[0]][2] = 30.0                               # r = 2 there: per replica 15, the highest
    inter, intra, reclaim, totals = t.scan(1e9, 1.0, 0.5, 1.0, 3)
    assert totals[1] == 5 and [x[0] for x in intra] == [z[0], z[4], z[3]]     # descending access per replica, top 3
    assert intra[0][2] == 2 and intra[0][4] == 15.0
    t.access[6][2] = 0.0                                   # the child [0, 9]: reclaimable
    _, _, reclaim, _ = t.scan(1e9, 1e9, 0.5, 1.0, 3)
    assert [x[0] for x in reclaim] == [6]
