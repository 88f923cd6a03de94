"""Host-side checks of the varlen tile schedule (no GPU): every (query tile, head pair, KV tile) step is
covered exactly once, per-CTA loads are balanced, split units have consistent partial slots."""
import numpy as np
import pytest

from paper_2609_04774_b200 import binding, build
from paper_2609_04774_b200 import workloads as wl


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build()


def check(w, num_sms=148):
    cu_new = w.cu_new
    prefix = [r.prefix_len for r in w.requests]
    Cs = [r.C for r in w.requests]
    info, pieces, items = binding.cp_schedule_inspect(cu_new, prefix, Cs, w.Hq, w.Hkv, num_sms)
    even = (w.Hq // w.Hkv) % 2 == 0
    HP = w.Hq // (2 if even else 1)
    TR = 128 if even else 256          # single-head units (odd group size) take two consecutive 128-row tiles
    # tiles: rows tile [0, total_new) exactly and never straddle a request; in a launch over all shards a tile
    # may span the boundary of adjacent zigzag chunks (the per-row causal limit does not care), so every tile
    # but a request's last has the full 128 rows
    rows = np.zeros(w.total_new, dtype=np.int32)
    for q0, n, kv0, nt in items:
        assert 1 <= n <= TR and nt == -(-(kv0 + n - 1) // 128)
        rows[q0:q0 + n] += 1
        b = int(np.searchsorted(cu_new, q0, side="right") - 1)
        r = w.requests[b]
        r0 = q0 - cu_new[b]
        assert r0 + n <= r.new_len and kv0 == r.prefix_len + r0 + 1
        assert r0 % TR == 0 and (n == TR or r0 + n == r.new_len)
    assert (rows == 1).all()
    # pieces: per unit the KV tile ranges tile [0, n_kv_tiles) exactly; slots only on split units
    cover = {}
    loads = np.zeros(info["grid"], dtype=np.int64)
    slots = set()
    for cta, item, pair, t0, t1, slot in pieces:
        assert 0 <= cta < info["grid"] and 0 <= pair < HP and 0 <= t0 < t1 <= items[item][3]
        cover.setdefault((item, pair), []).append((t0, t1, slot))
        loads[cta] += t1 - t0
        if slot >= 0:
            assert slot not in slots
            slots.add(slot)
    assert len(cover) == len(items) * HP
    n_split = 0
    for (item, pair), segs in cover.items():
        segs.sort()
        assert segs[0][0] == 0 and segs[-1][1] == items[item][3]
        for a, b2 in zip(segs, segs[1:]):
            assert a[1] == b2[0]
        if len(segs) == 1:
            assert segs[0][2] == -1
        else:
            n_split += 1
            assert all(s[2] >= 0 for s in segs)
    assert n_split == info["split_units"] and len(slots) == info["slots"] <= 2 * 192 + 32
    assert loads.sum() == info["total"] == sum(int(it[3]) for it in items) * HP
    assert loads.max() == info["max_load"] and loads.min() == info["min_load"]
    return info, loads


def test_schedule_covers_and_balances_all_configs():
    for cfg in (1, 2, 4, 5, 3):
        w = wl.CONFIGS[cfg]()
        info, loads = check(w)
        if info["pieces"] == info["grid"] <= 148 and info["max_load"] <= 8:
            # no more units than SMs, all short: one CTA per unit, nothing is cut (no partials, no merge launch)
            assert cfg == 1 and info["split_units"] == 0 and info["grid"] == 32
            continue
        share = -(-info["total"] // info["grid"])
        assert info["max_load"] <= 1.01 * share + 4, (cfg, info)   # at most one short remainder above the share
        assert loads.mean() >= 0.97 * info["max_load"] - 1, (cfg, info)   # the slowest CTA is within 3 % of the mean


def test_schedule_balances_short_no_prefix_requests():
    # many short units (no prefix): nothing may pile up on one CTA when the shares are rounded
    for R in (1024, 2048, 4096, 8192):
        for C in (1, 2, 8):
            info, loads = check(wl.Workload("noprefix", 1, 32, 8, [wl.Request(R, 0, C)]))
            share = -(-info["total"] // info["grid"])
            assert info["max_load"] <= max(1.25 * share, share + 8), (R, C, info)


def test_schedule_counts_a_fixed_cost_per_piece_for_small_kv():
    # small K/V (one group): the slowest CTA's estimated cost -- its KV tile steps plus two per piece of work -- stays
    # within 6 % (+2) of the mean cost for mid-size requests without a prefix; coverage is checked as everywhere
    for R, bound in ((1536, 14), (2048, 20), (3072, 42), (4096, 66), (6144, 140)):
        w = wl.Workload("mid", 1, 32, 8, [wl.Request(R, 0, 1)])
        info, loads = check(w)
        _, pieces, _ = binding.cp_schedule_inspect(w.cu_new, [0], [1], w.Hq, w.Hkv, 148)
        cnt = np.bincount(pieces[:, 0], minlength=info["grid"])
        cost = loads + 2 * cnt
        assert cost.max() <= bound, (R, cost.max())
        assert cost.max() <= 1.06 * cost.mean() + 4, (R, cost.max(), cost.mean())
        # these batches of many short units are dealt whole: nothing is cut, so the call is one launch
        assert info["split_units"] == 0 and info["launches"] == 1, info


def test_schedule_is_a_pure_function_of_its_inputs():
    # the same arguments give the same lists, whichever of the three schemes wins (ties in the least-loaded-first
    # dealing go to the lowest CTA index): a remembered schedule can stand in for a rebuilt one
    for w in (wl.Workload("p1", 1, 32, 8, [wl.Request(4096, 0, 1)]), wl.Workload("p2", 1, 32, 8, [wl.Request(2048, 4096, 2)]),
              wl.small_mixed(), wl.config2()):
        a = (w.cu_new, [r.prefix_len for r in w.requests], [r.C for r in w.requests], w.Hq, w.Hkv, 148)
        i1, p1, t1 = binding.cp_schedule_inspect(*a)
        i2, p2, t2 = binding.cp_schedule_inspect(*a)
        assert i1 == i2 and np.array_equal(p1, p2) and np.array_equal(t1, t2)


def test_schedule_small_and_odd_shapes():
    for w in (wl.small_mixed(), wl.Workload("one_row", 1, 4, 2, [wl.Request(1, 0, 1)]),
              wl.Workload("long_prefix", 2, 8, 2, [wl.Request(7, 100000, 2)]),
              wl.Workload("many_small", 3, 8, 2, [wl.Request(3 + i, 64 * (i % 3), 1 + i % 4) for i in range(40)]),
              wl.Workload("odd_group", 4, 6, 2, [wl.Request(300, 128, 2)]),
              wl.Workload("mha", 5, 4, 4, [wl.Request(513, 0, 3)])):
        for sms in (1, 7, 148):
            check(w, sms)


def test_large_kv_is_scheduled_kv_head_by_kv_head():
    # K/V beyond a quarter of L2: every CTA takes its whole units KV head by KV head (all CTAs then read one
    # head's K/V at a time); a small batch keeps the plain longest-first order
    def unit_sequences(w):
        info, pieces, items = binding.cp_schedule_inspect(w.cu_new, [r.prefix_len for r in w.requests],
                                                          [r.C for r in w.requests], w.Hq, w.Hkv, 148)
        per_cta = {}
        for cta, item, pair, t0, t1, slot in pieces:
            if slot < 0:
                per_cta.setdefault(int(cta), []).append((int(pair), int(items[item][3])))
        return per_cta
    big = wl.Workload("big", 1, 32, 8, [wl.Request(32768, 0, 4)])            # 134 MB of K/V
    pairs_per_kv = (big.Hq // big.Hkv) // 2
    for cta, seq in unit_sequences(big).items():
        heads = [p // pairs_per_kv for p, _ in seq]
        # (a whole unit placed by the tail pass may follow at the end of a list: at most one step back)
        assert sum(1 for a, b in zip(heads, heads[1:]) if b < a) <= 1, cta
        assert len(set(heads)) >= 4                                           # every CTA sees most of the heads
    small = wl.Workload("small", 1, 32, 8, [wl.Request(2048, 0, 4)])          # 8 MB of K/V
    for cta, seq in unit_sequences(small).items():
        lens = [n for _, n in seq]
        assert lens == sorted(lens, reverse=True)
