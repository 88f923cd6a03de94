"""Randomised host-side properties (hypothesis): the C planner equals the oracle planner, and the varlen
tile schedule covers every (query tile, head unit, KV tile) step exactly once for arbitrary batches."""
import numpy as np
from hypothesis import given, settings, strategies as st

from oracle import reference as orc
from paper_2609_04774_b200 import binding, build
from paper_2609_04774_b200 import workloads as wl
from tests.test_schedule_host import check

build.build()


@settings(max_examples=200, deadline=None)
@given(R=st.integers(1, 5000), P=st.integers(0, 100000), C=st.integers(1, 16))
def test_cp_plan_equals_oracle(R, P, C):
    got = binding.cp_plan(R, P, C)
    assert got == orc.plan(R, P, C)
    assert sum(s["pairs"] for s in got) == orc.remaining_workload(R, P)


requests = st.lists(st.tuples(st.integers(1, 3000), st.integers(0, 40000), st.sampled_from([1, 2, 3, 4, 8])),
                    min_size=1, max_size=12)


@settings(max_examples=60, deadline=None)
@given(reqs=requests, heads=st.sampled_from([(8, 2), (4, 4), (6, 2), (32, 8)]), sms=st.sampled_from([1, 5, 132, 148]))
def test_schedule_covers_everything_once(reqs, heads, sms):
    w = wl.Workload("hyp", 0, heads[0], heads[1], [wl.Request(r, p, c) for r, p, c in reqs])
    info, loads = check(w, sms)
    share = -(-info["total"] // info["grid"])
    longest = max(-(-(r.prefix_len + r.new_len) // 128) for r in w.requests)
    # nobody carries more than its share plus one short remainder (or one unit that is too short to cut)
    assert info["max_load"] <= max(1.3 * share + 8, min(longest, 8) + 8), (info, share)
