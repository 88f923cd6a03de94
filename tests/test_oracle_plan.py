"""Pins for the oracle's zigzag planner and workload count (no GPU)."""
import itertools
import os

import pytest

from oracle import reference as orc


def _read(path):
    rows = []
    with open(path) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([int(x) for x in line.split()])
    return rows


def test_chunk_map_matches_paper_text(golden_dir):
    # Section 2.1: rank k receives the k-th and (2C-1-k)-th of 2C equal contiguous chunks.
    for C, k, c0, c1 in _read(os.path.join(golden_dir, "zigzag_chunk_map.txt")):
        cl = 8
        R = 2 * C * cl
        sh = orc.plan(R, 0, C)[k]
        assert sh["q_begin"] == [c0 * cl, c1 * cl]
        assert sh["q_end"] == [(c0 + 1) * cl, (c1 + 1) * cl]


def test_workload_matches_eq1_golden(golden_dir):
    for R, P, C, W, Wps in _read(os.path.join(golden_dir, "remaining_workload.txt")):
        assert orc.remaining_workload(R, P) == W
        shards = orc.plan(R, P, C)
        assert sum(s["pairs"] for s in shards) == W
        assert all(s["pairs"] == Wps for s in shards)      # zigzag balances exactly when 2C | R


@pytest.mark.parametrize("C", [1, 2, 3, 4, 5, 8])
def test_bruteforce_pairs_and_tiling(C):
    for R, P in itertools.product(list(range(1, 41)) + [64], [0, 1, 5, 8]):
        shards = orc.plan(R, P, C)
        assert len(shards) == C
        owned = []
        total = 0
        for s in shards:
            cnt = 0
            for b, e, kve in zip(s["q_begin"], s["q_end"], s["kv_end"]):
                assert 0 <= b <= e <= R and kve == P + e
                for r in range(b, e):
                    owned.append(r)
                    # enumerate the (query, key) pairs allowed by the causal mask M_ij = 0 for j <= i
                    cnt += sum(1 for j in range(P + R) if j <= P + r)
            assert cnt == s["pairs"]
            total += cnt
        assert sorted(owned) == list(range(R))             # chunks tile [0,R): no gap, no overlap
        assert total == R * P + R * (R + 1) // 2           # Eq. (1)


def test_padding_rule_short_and_empty_chunks():
    # R=5, C=4: chunk length ceil(5/8)=1 -> chunks 0..4 hold one token, 5..7 are empty.
    shards = orc.plan(5, 0, 4)
    assert [s["q_begin"] for s in shards] == [[0, 5], [1, 5], [2, 5], [3, 4]]
    assert [s["q_end"] for s in shards] == [[1, 5], [2, 5], [3, 5], [4, 5]]
    # R=10, C=2: chunk length 3 -> [0,3) [3,6) [6,9) [9,10)
    shards = orc.plan(10, 7, 2)
    assert shards[0]["q_begin"] == [0, 9] and shards[0]["q_end"] == [3, 10]
    assert shards[1]["q_begin"] == [3, 6] and shards[1]["q_end"] == [6, 9]
    assert shards[0]["kv_end"] == [10, 17]


def test_c1_owns_everything():
    s = orc.plan(37, 11, 1)
    assert len(s) == 1 and s[0]["q_begin"][0] == 0 and s[0]["q_end"][1] == 37
    assert s[0]["q_end"][0] == s[0]["q_begin"][1]
    assert s[0]["pairs"] == orc.remaining_workload(37, 11)
