"""Library cp_trie_* / cp_prefer_degree / cp_prefill_time against the oracle: the hand-worked scenarios
again through the C ABI, then a seeded request stream driving both sides through placement, Algorithm 1,
periodic scans (Algorithm 2) and the execution of the chosen replications and reclamations, with the
whole state compared after every scan."""
import math

import numpy as np
import pytest

from oracle import cache_manager as cm
from paper_2609_04774_b200 import binding, build, cache_manager as lib, workloads as wl

MODEL = (3e-4, 2e-7, 5e-8, 1e-6, 4e-11)
PURE_ATTENTION = (0.0, 0.0, 0.0, 0.0, 1.0)


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def test_prefill_time_and_prefer_degree_match_oracle():
    rng = np.random.default_rng(5)
    for _ in range(200):
        R, P, C = int(rng.integers(1, 200000)), int(rng.integers(0, 200000)), int(rng.choice([1, 2, 4, 8]))
        assert lib.cp_prefill_time(MODEL, R, P, C) == cm.prefill_time(MODEL, R, P, C)
    assert lib.cp_prefill_time((1, 2, 3, 4, 5), 10, 20, 2) == 1 + 20 + 60 + (40 + 5 * 255) / 2
    assert math.isnan(lib.cp_prefill_time(MODEL, 10, 0, 0))
    for _ in range(200):
        n = int(rng.integers(1, 7))
        L = int(rng.integers(64, 100000))
        deg = rng.choice([1, 2, 4, 8], size=n)
        reused = (rng.integers(0, L // 64 + 1, size=n) * 64).clip(0, L)
        beta, lam = float(rng.uniform(1, 3)), float(rng.choice([0.0, 0.3, 1.0]))
        want = cm.prefer_degree(MODEL, L, list(zip(deg.tolist(), reused.tolist())), beta, lam)
        assert lib.cp_prefer_degree(MODEL, L, deg, reused, beta, lam) == want
    assert lib.cp_prefer_degree(PURE_ATTENTION, 100, [1, 4], [60, 0], 1.0, 0.0) == (1, 4)
    assert lib.cp_prefer_degree((0.0, 100.0, 0.0, 0.0, 1.0), 100, [1, 4], [60, 0], 1.0, 1.0) == (0, 1)
    with pytest.raises(binding.CpError):
        lib.cp_prefer_degree(MODEL, 100, [1, 0], [0, 0])
    with pytest.raises(binding.CpError):
        lib.cp_prefer_degree(MODEL, 100, [1], [101])


def test_hand_worked_update_and_scan_through_the_library():
    t = lib.Trie([1, 4], 64)
    t.set_worker(10, 1)
    t.set_worker(20, 4)
    assert t.add_replica([7, 8, 9], 10) == 3
    t.update([7, 8, 9, 2], 256, 10, 4, PURE_ATTENTION)
    assert [t.stats(z, 1)[0] for z in (1, 2, 3)] == [1.0, 1.0, 1.0]
    assert [t.stats(z, 4)[1] for z in (1, 2, 3)] == [(32896 - 30816) / 4, (30816 - 24640) / 4, (24640 - 14368) / 4]
    assert t.match([7, 8, 9, 1]) == [1, 2, 3] and t.match([6]) == [] and t.reused([7, 8, 9], 20) == 0
    with pytest.raises(binding.CpError):
        t.drop_replica(2, 10)                         # child 3 still retained
    with pytest.raises(binding.CpError):
        t.update([7, 8, 9], 100, 10, 4, PURE_ATTENTION)   # request shorter than its matched prefix
    with pytest.raises(binding.CpError):
        t.update([7], 256, 10, 2, PURE_ATTENTION)     # unsupported degree
    with pytest.raises(binding.CpError):
        t.add_replica([1], 99)                        # unknown worker
    inter, intra, reclaim, totals = t.scan(1000.0, 0.5, 0.25, 0.5, 4)
    # missed: 520, 1544, 2568 at degree 4 (r = 0) -> two above 1000; access 1 > 0.5 at degree 1 -> intra x3
    assert totals == (2, 3, 0)
    assert [c[0] for c in inter] == [3, 2] and inter[0][3:] == (3, 2568.0 / 3) and inter[1][3:] == (2, 1544.0 / 2)
    assert t.stats(3, 4) == (0.0, 1284.0) and t.stats(1, 1) == (0.5, 0.0)
    t.close()


def _same_candidates(a, b):
    assert len(a) == len(b)
    for x, y in zip(a, b):
        assert x[:4] == y[:4] and math.isclose(x[4], y[4], rel_tol=1e-12, abs_tol=1e-300), (x, y)


@pytest.mark.parametrize("seed", [1, 2])
def test_request_stream_matches_oracle(seed):
    degrees = [1, 2, 4, 8]
    workers = {w: degrees[w % 4] for w in range(12)}
    a, b = cm.Trie(degrees, 64), lib.Trie(degrees, 64)
    for w, c in workers.items():
        a.set_worker(w, c)
        b.set_worker(w, c)
    stream = wl.prefix_stream(seed, 600)
    u = wl.counter_uniform(seed, wl.TID_STREAM, 1 << 20, len(stream))
    ids = sorted(workers)
    seen = [0, 0, 0]
    for i, (blocks, L) in enumerate(stream):
        # PreferDegree from every worker's reusable prefix; the request itself lands on a pseudo-random
        # worker (queueing pressure), which then caches the whole prompt
        reused_a = [len(a.reused_path(blocks, w)) * 64 for w in ids]
        reused_b = [b.reused(blocks, w) * 64 for w in ids]
        assert reused_a == reused_b == (b.reused_all(blocks, ids) * 64).tolist()
        assert a.matched_path(blocks) == b.match(blocks)
        _, pref = cm.prefer_degree(MODEL, L, [(workers[w], p) for w, p in zip(ids, reused_a)], 1.2, 0.2)
        assert lib.cp_prefer_degree(MODEL, L, [workers[w] for w in ids], reused_b, 1.2, 0.2)[1] == pref
        w = ids[int(u[i] * len(ids))]
        a.update(blocks, L, w, pref, MODEL)
        b.update(blocks, L, w, pref, MODEL)
        assert a.add_replica(blocks, w) == b.add_replica(blocks, w)
        if i % 97 == 96:                                  # a worker is reconfigured to another degree
            workers[w] = degrees[(degrees.index(workers[w]) + 1) % 4]
            a.set_worker(w, workers[w])
            b.set_worker(w, workers[w])
        if i % 50 == 49:
            ra, rb = a.scan(1e-5, 3.0, 0.4, 0.8, 6), b.scan(1e-5, 3.0, 0.4, 0.8, 6)
            for k in range(3):
                _same_candidates(ra[k], rb[k])
            assert ra[3] == rb[3]
            seen = [x + y for x, y in zip(seen, ra[3])]
            # execute: replicate inter / intra candidates onto the first worker of that degree lacking the
            # node, reclaim from the first holder that retains no child
            for z, C, r, fp, score in ra[0] + ra[1]:
                path = []
                y = z
                while y > 0:
                    path.append(y)
                    y = a.parent[y]
                key_of = {c: k for p in path for k, c in a.children[a.parent[p]].items()}
                keys = [key_of[p] for p in reversed(path)]
                dst = [x for x in ids if workers[x] == C and x not in a.holders[z]]
                if dst:
                    assert a.add_replica(keys, dst[0]) == b.add_replica(keys, dst[0]) == z
            for z, C, r, fp, score in ra[2]:
                for x in sorted(a.holders[z]):
                    if workers[x] == C and a.drop_replica(z, x):
                        b.drop_replica(z, x)
                        break
    assert len(a.parent) == b.size() > 1000 and min(seen) > 20        # all three lists were exercised
    for z in range(1, len(a.parent), 7):
        for C in degrees:
            assert a.replica_count(z, C) == b.replica_count(z, C)
            sa, sb = (a.access[z][C], a.missed[z][C]), b.stats(z, C)
            assert math.isclose(sa[0], sb[0], rel_tol=1e-12, abs_tol=1e-300)
            assert math.isclose(sa[1], sb[1], rel_tol=1e-12, abs_tol=1e-300)
    b.set_worker(0, 0)
    a.set_worker(0, 0)
    assert all(a.replica_count(z, C) == b.replica_count(z, C) for z in range(1, len(a.parent), 11) for C in degrees)
    b.close()


def test_stream_generator_has_reuse_structure():
    stream = wl.prefix_stream(3, 400)
    t = cm.Trie([1], 64)
    t.set_worker(0, 1)
    hits = 0
    for blocks, L in stream:
        assert len(blocks) * 64 <= L < (len(blocks) + 1) * 64 and len(set(blocks)) == len(blocks)
        hits += len(t.matched_path(blocks)) > 0
        t.add_replica(blocks, 0)
    assert 0.5 < hits / len(stream) < 0.95            # most requests reuse a prefix, some start fresh
