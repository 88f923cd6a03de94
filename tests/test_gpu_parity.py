"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded
inputs.  Planner and page indexing bit-exact; attention within max-abs 2e-2 / mean-abs 2e-3 and LSE
within 1e-3; merge within fp32 round-off."""
import os

import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_2609_04774_b200 import binding
from paper_2609_04774_b200 import workloads as wl
from tests.gpu_util import DeviceWorkload, bf16_to_f64, bits_to_bf16, compare

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


def oracle_request(mat, b, rows=None):
    w = mat.wl
    r = w.requests[b]
    q = mat.q[w.cu_new[b]:w.cu_new[b + 1]]
    pt = mat.page_table[w.cu_pages[b]:w.cu_pages[b + 1]]
    if rows is None:
        return orc.attn_full(q, mat.k_pages, mat.v_pages, pt, r.prefix_len, w.Hkv, w.scale)
    return orc.attn_rows(q, mat.k_pages, mat.v_pages, pt, r.prefix_len, w.Hkv, w.scale, rows)


def check_batch(ctx, w, pair_budget=3e8, seed_rows=123, cmp=compare):
    """Run the whole batch in one launch; compare every request (all rows when cheap, otherwise the
    rows around every tile / chunk boundary plus seeded random rows)."""
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    out, lse = dev.run_batch(ctx)
    stats = []
    for b, r in enumerate(w.requests):
        lo, hi = int(w.cu_new[b]), int(w.cu_new[b + 1])
        if r.new_len * (r.prefix_len + r.new_len / 2) * w.Hq <= pair_budget:
            rows = np.arange(r.new_len)
        else:
            n = max(16, int(pair_budget / (w.Hq * (r.prefix_len + r.new_len / 2))))
            cl = -(-r.new_len // (2 * r.C))
            edges = [x for j in range(2 * r.C + 1) for x in (j * cl - 1, j * cl, j * cl + 127, j * cl + 128)]
            rnd = wl.sample_rows(seed_rows + b, 1, r.new_len, n)[0]
            rows = np.unique(np.clip(np.concatenate([edges, rnd, [0, r.new_len - 1]]), 0, r.new_len - 1))
        ref_o, ref_l = oracle_request(mat, b, rows)
        stats.append(cmp(out[lo:hi][rows], lse[:, lo:hi][:, rows], ref_o, ref_l, "%s req %d" % (w.name, b)))
    return dev, out, lse, stats


def test_plan_matches_oracle_on_device_box():
    for R, P, C in [(1024, 0, 2), (4096, 12288, 4), (131072, 0, 8), (32768, 32768, 8), (333, 192, 3)]:
        assert binding.cp_plan(R, P, C) == orc.plan(R, P, C)


def test_merge_parity(ctx):
    for (N, T, H, dt) in [(2, 100, 5, torch.float32), (4, 37, 64, torch.bfloat16), (8, 64, 7, torch.float32),
                          (3, 9, 1, torch.bfloat16), (1, 20, 4, torch.float32), (16, 33, 3, torch.float32)]:
        parts, lses = wl.merge_inputs(6, N, T, H, 128, neg_inf_frac=5)
        if N > 2:
            lses[:, H - 1, 3] = -np.inf        # a row that is dead in every partial
            parts[2, 5, 0] = np.nan            # junk behind a -inf lse must be ignored
            lses[2, 0, 5] = -np.inf
        ref_o, ref_l = orc.merge(parts, lses)
        out = torch.empty((T, H, 128), dtype=dt, device="cuda")
        lse_out = torch.empty((H, T), dtype=torch.float32, device="cuda")
        binding.cp_merge(ctx, torch.from_numpy(parts).cuda(), torch.from_numpy(lses).cuda(), out, lse_out)
        torch.cuda.synchronize()
        o = out.float().cpu().numpy().astype(np.float64)
        tol = 1e-5 if dt == torch.float32 else 2.0 ** -8
        assert np.abs(o - ref_o).max() <= tol * max(1.0, np.abs(ref_o).max()), (N, T, H)
        l = lse_out.cpu().numpy().astype(np.float64)
        assert np.array_equal(np.isneginf(l), np.isneginf(ref_l))
        fin = np.isfinite(ref_l)
        assert np.abs(l[fin] - ref_l[fin]).max() <= 1e-5 * np.abs(ref_l[fin]).max()


def test_merge_many_tokens_one_head(ctx):
    # more than 65535 token blocks: block indices beyond a grid's y range; last rows compared with the oracle
    N, T, H = 2, 8 * 70000 + 3, 1
    g = torch.Generator(device="cuda").manual_seed(9)
    parts = torch.randn((N, T, H, 128), device="cuda", generator=g)
    lses = 8 + 2 * torch.randn((N, H, T), device="cuda", generator=g)
    out = torch.empty((T, H, 128), dtype=torch.float32, device="cuda")
    lse_out = torch.empty((H, T), dtype=torch.float32, device="cuda")
    binding.cp_merge(ctx, parts, lses, out, lse_out)
    torch.cuda.synchronize()
    for lo, hi in ((0, 64), (8 * 65535 - 32, 8 * 65535 + 32), (T - 64, T)):
        ref_o, ref_l = orc.merge(parts[:, lo:hi].cpu().numpy().astype(np.float64), lses[:, :, lo:hi].cpu().numpy().astype(np.float64))
        assert np.abs(out[lo:hi].cpu().numpy() - ref_o).max() <= 1e-5 * np.abs(ref_o).max()
        assert np.abs(lse_out[:, lo:hi].cpu().numpy() - ref_l).max() <= 1e-5 * np.abs(ref_l).max()


def test_kv_gather_append_bit_exact(ctx):
    w = wl.small_mixed()
    mat = wl.materialize(w)
    k = bits_to_bf16(mat.k_pages)
    v = bits_to_bf16(mat.v_pages)
    cache = binding.make_cache(k, v)
    b = 0
    r = w.requests[b]
    pt_host = mat.page_table[w.cu_pages[b]:w.cu_pages[b + 1]]
    pt = torch.from_numpy(pt_host.copy()).cuda()
    t0, n = 37, r.total_len - 37
    kr = torch.zeros((n, w.Hkv, w.D), dtype=torch.bfloat16, device="cuda")
    vr = torch.zeros_like(kr)
    binding.cp_kv_gather(ctx, cache, pt, t0, n, kr, vr)
    torch.cuda.synchronize()
    assert np.array_equal(kr.view(torch.int16).cpu().numpy().view(np.uint16), orc.kv_gather(mat.k_pages, pt_host, t0, t0 + n))
    assert np.array_equal(vr.view(torch.int16).cpu().numpy().view(np.uint16), orc.kv_gather(mat.v_pages, pt_host, t0, t0 + n))
    # append new rows and compare the whole pool with the oracle's append
    newk = wl.normal_bf16(5, wl.TID_K, (n, w.Hkv, w.D))
    newv = wl.normal_bf16(5, wl.TID_V, (n, w.Hkv, w.D))
    binding.cp_kv_append(ctx, cache, pt, t0, n, bits_to_bf16(newk), bits_to_bf16(newv))
    torch.cuda.synchronize()
    kp, vp = mat.k_pages.copy(), mat.v_pages.copy()
    orc.kv_append(kp, pt_host, t0, newk)
    orc.kv_append(vp, pt_host, t0, newv)
    assert np.array_equal(k.view(torch.int16).cpu().numpy().view(np.uint16), kp)
    assert np.array_equal(v.view(torch.int16).cpu().numpy().view(np.uint16), vp)


def test_kv_append_segments_bit_exact(ctx):
    # several runs of rows in one launch, in scrambled order, with an empty segment and gaps left untouched
    w = wl.Workload("segments", 48, 8, 2, [wl.Request(900, 448, 1)])
    mat = wl.materialize(w)
    k, v = bits_to_bf16(mat.k_pages), bits_to_bf16(mat.v_pages)
    cache = binding.make_cache(k, v)
    pt = torch.from_numpy(mat.page_table).cuda()
    rows_k = wl.normal_bf16(49, wl.TID_K, (700, w.Hkv, w.D))
    rows_v = wl.normal_bf16(49, wl.TID_V, (700, w.Hkv, w.D))
    segs = [(1000, 130, 0), (5, 59, 500), (64, 0, 3), (448, 333, 150), (200, 1, 699)]
    binding.cp_kv_append_segments(ctx, cache, pt, segs, bits_to_bf16(rows_k), bits_to_bf16(rows_v))
    torch.cuda.synchronize()
    ctx.poll_status()
    kp, vp = mat.k_pages.copy(), mat.v_pages.copy()
    for t0, n, r0 in segs:
        orc.kv_append(kp, mat.page_table, t0, rows_k[r0:r0 + n])
        orc.kv_append(vp, mat.page_table, t0, rows_v[r0:r0 + n])
    assert np.array_equal(k.view(torch.int16).cpu().numpy().view(np.uint16), kp)
    assert np.array_equal(v.view(torch.int16).cpu().numpy().view(np.uint16), vp)
    with pytest.raises(binding.CpError) as e:
        binding.cp_kv_append_segments(ctx, cache, pt, [(0, 1, 0)] * 65, bits_to_bf16(rows_k), bits_to_bf16(rows_v))
    assert e.value.code == binding.CP_ERR_UNSUPPORTED


@pytest.mark.parametrize("Hkv,page", [(1, 16), (3, 128), (16, 32), (8, 64)])
def test_kv_copies_other_head_counts_and_page_sizes(ctx, Hkv, page):
    # one warp copies one token: rows of 16 vectors (one KV head) up to 256 (sixteen heads, two passes of the warp),
    # a count that is no multiple of 32, every page size; the cache is a strided view; gather, append and the
    # segment form against the oracle, bit for bit
    w = wl.Workload("copies", 52, Hkv, Hkv, [wl.Request(333, 5 * page, 1)], page=page)
    mat = wl.materialize(w, need_q=False)
    npg = mat.k_pages.shape[0]
    big_k = torch.zeros((npg, page + 1, Hkv + 1, w.D), dtype=torch.bfloat16, device="cuda")
    big_v = torch.zeros_like(big_k)
    k, v = big_k[:, :page, :Hkv], big_v[:, :page, :Hkv]
    k.copy_(bits_to_bf16(mat.k_pages))
    v.copy_(bits_to_bf16(mat.v_pages))
    cache = binding.make_cache(k, v)
    pt = torch.from_numpy(mat.page_table).cuda()
    L = w.requests[0].total_len
    t0, n = 7, L - 7
    kr = torch.zeros((n, Hkv, w.D), dtype=torch.bfloat16, device="cuda")
    vr = torch.zeros_like(kr)
    binding.cp_kv_gather(ctx, cache, pt, t0, n, kr, vr)
    torch.cuda.synchronize()
    ctx.poll_status()
    bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    assert np.array_equal(bits(kr), orc.kv_gather(mat.k_pages, mat.page_table, t0, t0 + n))
    assert np.array_equal(bits(vr), orc.kv_gather(mat.v_pages, mat.page_table, t0, t0 + n))
    newk, newv = wl.normal_bf16(53, wl.TID_K, (n, Hkv, w.D)), wl.normal_bf16(53, wl.TID_V, (n, Hkv, w.D))
    kp, vp = mat.k_pages.copy(), mat.v_pages.copy()
    binding.cp_kv_append(ctx, cache, pt, t0, 100, bits_to_bf16(newk), bits_to_bf16(newv))
    orc.kv_append(kp, mat.page_table, t0, newk[:100])
    orc.kv_append(vp, mat.page_table, t0, newv[:100])
    segs = [(200, 57, 120), (130, 33, 300), (L - 9, 9, 0)]
    binding.cp_kv_append_segments(ctx, cache, pt, segs, bits_to_bf16(newk), bits_to_bf16(newv))
    for s0, sn, r0 in segs:
        orc.kv_append(kp, mat.page_table, s0, newk[r0:r0 + sn])
        orc.kv_append(vp, mat.page_table, s0, newv[r0:r0 + sn])
    torch.cuda.synchronize()
    ctx.poll_status()
    assert np.array_equal(bits(k), kp) and np.array_equal(bits(v), vp)
    assert not bool(big_k[:, page].any()) and not bool(big_k[:, :, Hkv].any())      # nothing outside the view was touched


def test_kv_copies_skip_page_ids_outside_the_pool(ctx):
    # the copies compare every page id with the pool size before they use it: tokens behind a bad entry are left alone
    # (rows keep their fill on a gather, the pool is untouched on an append) and the first bad entry is reported
    w = wl.Workload("bad_pages", 54, 4, 2, [wl.Request(200, 256, 1)])
    mat = wl.materialize(w, need_q=False)
    k, v = bits_to_bf16(mat.k_pages), bits_to_bf16(mat.v_pages)
    cache = binding.make_cache(k, v)
    pt_host = mat.page_table.copy()
    pt_host[2], pt_host[5] = k.shape[0], -1                    # one beyond the pool, one negative
    pt = torch.from_numpy(pt_host).cuda()
    L = w.requests[0].total_len
    bad = np.zeros(L, dtype=bool)
    bad[2 * wl.PAGE:3 * wl.PAGE] = bad[5 * wl.PAGE:6 * wl.PAGE] = True
    kr = torch.full((L, w.Hkv, w.D), 7.0, dtype=torch.bfloat16, device="cuda")
    vr = torch.full_like(kr, 7.0)
    binding.cp_kv_gather(ctx, cache, pt, 0, L, kr, vr)
    torch.cuda.synchronize()
    with pytest.raises(binding.CpError) as e:
        ctx.poll_status()
    assert e.value.code == binding.CP_ERR_BOUNDS
    bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    ref = orc.kv_gather(mat.k_pages, mat.page_table, 0, L)
    assert np.array_equal(bits(kr)[~bad], ref[~bad]) and bool((kr[torch.from_numpy(bad).cuda()] == 7.0).all())
    before_k, before_v = k.clone(), v.clone()
    rows = bits_to_bf16(wl.normal_bf16(55, wl.TID_K, (L, w.Hkv, w.D)))
    binding.cp_kv_append(ctx, cache, pt, 0, L, rows, rows)
    binding.cp_kv_append_segments(ctx, cache, pt, [(2 * wl.PAGE, wl.PAGE, 0)], rows, rows)      # entirely behind the bad entry
    torch.cuda.synchronize()
    with pytest.raises(binding.CpError) as e:
        ctx.poll_status()
    assert e.value.code == binding.CP_ERR_BOUNDS
    good = torch.from_numpy(mat.page_table[[i for i in range(len(pt_host)) if i not in (2, 5)]].astype(np.int64)).cuda()
    touched = torch.zeros(k.shape[0], dtype=torch.bool, device="cuda")
    touched[good] = True
    assert torch.equal(k[~touched], before_k[~touched]) and torch.equal(v[~touched], before_v[~touched])
    got = orc.kv_gather(bits(k), mat.page_table, 0, L)
    assert np.array_equal(got[~bad], bits(rows)[~bad])
    ctx.poll_status()                                          # cleared; the context is usable
    check_batch(ctx, wl.Workload("after_bad_pages", 56, 8, 2, [wl.Request(150, 64, 2)]))


def test_page_table_check_reports_bad_entries(ctx):
    # the checker only reads the table: a good table passes, an entry beyond the pool (or negative) is reported with
    # its index and value, and the context computes on afterwards
    pt = torch.arange(1000, dtype=torch.int32, device="cuda")
    binding.cp_check_page_table(ctx, pt, 1000)
    torch.cuda.synchronize()
    ctx.poll_status()
    pt[617] = 1000
    binding.cp_check_page_table(ctx, pt, 1000)
    torch.cuda.synchronize()
    with pytest.raises(binding.CpError) as e:
        ctx.poll_status()
    assert e.value.code == binding.CP_ERR_BOUNDS and "entry 617 holds page id 1000" in str(e.value)
    pt[617] = -3
    binding.cp_check_page_table(ctx, pt, 1000)
    torch.cuda.synchronize()
    with pytest.raises(binding.CpError) as e:
        ctx.poll_status()
    assert e.value.code == binding.CP_ERR_BOUNDS and "page id -3" in str(e.value)
    ctx.poll_status()                                    # cleared
    check_batch(ctx, wl.Workload("after_bounds", 51, 8, 2, [wl.Request(200, 64, 2)]))


def test_attention_small_mixed_batch(ctx):
    dev, out, lse, _ = check_batch(ctx, wl.small_mixed())
    # run-to-run bitwise determinism
    o1 = dev.out.clone()
    l1 = dev.lse.clone()
    dev.run_batch(ctx)
    assert torch.equal(o1.view(torch.int16), dev.out.view(torch.int16)) and torch.equal(l1, dev.lse)


@pytest.mark.parametrize("page", [16, 32, 128])
def test_attention_other_page_sizes(ctx, page):
    # cache pages of 16, 32 and 128 tokens: 8, 4 and 1 page boxes per 128-key tile; prefixes that are and are
    # not page multiples; KV-split units; the paged copies with the same page size, bit for bit
    reqs = [wl.Request(333, 192, 3), wl.Request(5, 0, 4), wl.Request(700, 1000, 2), wl.Request(64, 20000, 1)]
    w = wl.Workload("page_%d" % page, 45, 8, 2, reqs, page=page)
    dev, out, lse, _ = check_batch(ctx, w, pair_budget=3e7)
    assert dev.cache.page_size == page
    mat = dev.mat
    pt_host = mat.page_table[w.cu_pages[2]:w.cu_pages[3]]
    pt = dev.page_table[int(w.cu_pages[2]):int(w.cu_pages[3])].contiguous()
    t0, n = 37, 1500
    kr = torch.empty((n, w.Hkv, w.D), dtype=torch.bfloat16, device="cuda")
    vr = torch.empty_like(kr)
    binding.cp_kv_gather(ctx, dev.cache, pt, t0, n, kr, vr)
    torch.cuda.synchronize()
    assert np.array_equal(kr.view(torch.int16).cpu().numpy().view(np.uint16), orc.kv_gather(mat.k_pages, pt_host, t0, t0 + n))
    assert np.array_equal(vr.view(torch.int16).cpu().numpy().view(np.uint16), orc.kv_gather(mat.v_pages, pt_host, t0, t0 + n))


def test_attention_odd_group_sizes(ctx):
    # Hq / Hkv = 3 and plain multi-head attention (Hq == Hkv): one query head per work unit
    check_batch(ctx, wl.Workload("odd_group", 41, 6, 2, [wl.Request(333, 192, 3), wl.Request(129, 0, 2)]))
    check_batch(ctx, wl.Workload("mha", 42, 4, 4, [wl.Request(700, 64, 4)]))


def test_attention_tile_pair_edges(ctx):
    # single-head units (three heads per KV head; plain multi-head) over pairs of query tiles: requests of exactly
    # one tile, one row more, two tiles, two tiles and a row, a single row; long prefixes so that the units are cut
    # along KV (a piece may lie wholly behind the earlier tile's causal limit); unaligned prefixes
    reqs = [wl.Request(128, 40000, 1), wl.Request(129, 5003, 2), wl.Request(256, 0, 1), wl.Request(257, 64, 3),
            wl.Request(1, 70001, 1), wl.Request(385, 20000, 4)]
    for name, heads in (("pair_g3", (6, 2)), ("pair_mha", (4, 4))):
        w = wl.Workload(name, 49, heads[0], heads[1], reqs)
        info, _, _ = binding.cp_schedule_inspect(w.cu_new, [r.prefix_len for r in reqs], [r.C for r in reqs], w.Hq, w.Hkv,
                                                 torch.cuda.get_device_properties(0).multi_processor_count, want_lists=False)
        assert info["split_units"] > 0
        dev, out, lse, _ = check_batch(ctx, w, pair_budget=4e7)
        o1, l1 = dev.out.clone(), dev.lse.clone()
        dev.run_batch(ctx)
        assert torch.equal(o1.view(torch.int16), dev.out.view(torch.int16)) and torch.equal(l1, dev.lse)


def test_attention_many_small_requests(ctx):
    # forty requests of 3 to 42 new tokens behind 0, 64 or 128 cached ones: every tile is ragged, most units one KV tile
    reqs = [wl.Request(3 + i, 64 * (i % 3), 1 + i % 4) for i in range(40)]
    check_batch(ctx, wl.Workload("many_small", 50, 8, 2, reqs))
    check_batch(ctx, wl.Workload("many_small_mha", 50, 2, 2, reqs))


def test_attention_kv_split_units(ctx):
    # few query rows, long prefixes: every unit is cut along KV over many CTAs and merged by the fix-up
    # kernel; prefix lengths that are not page multiples; a request whose rows see no key of some piece
    w = wl.Workload("kv_split", 43, 8, 2, [wl.Request(130, 40000, 2), wl.Request(7, 100003, 1), wl.Request(64, 64, 1)])
    info, _, _ = binding.cp_schedule_inspect(w.cu_new, [r.prefix_len for r in w.requests], [r.C for r in w.requests],
                                             w.Hq, w.Hkv, torch.cuda.get_device_properties(0).multi_processor_count,
                                             want_lists=False)
    assert info["split_units"] >= 8 and info["slots"] > 2 * info["split_units"]
    dev, out, lse, _ = check_batch(ctx, w, pair_budget=1e10)
    o1, l1 = dev.out.clone(), dev.lse.clone()
    dev.run_batch(ctx)                                   # the merge order is fixed: bitwise reproducible
    assert torch.equal(o1.view(torch.int16), dev.out.view(torch.int16)) and torch.equal(l1, dev.lse)


def test_attention_one_unit_cut_over_all_sms(ctx):
    # a single work unit (one query tile, one pair of heads) behind a quarter of a million cached tokens: the planner
    # cuts it into one piece per SM, so the fix-up merges far more than 32 partials per row (it walks them in groups
    # of 32)
    w = wl.Workload("one_unit", 45, 2, 1, [wl.Request(100, 250000, 1)])
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    info, _, _ = binding.cp_schedule_inspect(w.cu_new, [250000], [1], w.Hq, w.Hkv, sms, want_lists=False)
    assert info["split_units"] == 1 and info["slots"] > 64, info
    check_batch(ctx, w, pair_budget=1e10)
    # the same with an odd group (a tile-pair unit of one head): 200 rows, two tiles
    w1 = wl.Workload("one_unit_mha", 46, 1, 1, [wl.Request(200, 180000, 1)])
    info, _, _ = binding.cp_schedule_inspect(w1.cu_new, [180000], [1], w1.Hq, w1.Hkv, sms, want_lists=False)
    assert info["split_units"] == 1 and info["slots"] > 64, info
    check_batch(ctx, w1, pair_budget=1e10)


def test_attention_reads_zeros_behind_page_ids_outside_the_pool(ctx):
    # a page id outside [0, num_pages) is a tensor-map coordinate outside the tensor: the copy engine fills zeros, the
    # same mechanism that serves the unused tail of every request's last key tile.  Reference: the oracle with those
    # table entries pointed at a page of zeros.
    w = wl.Workload("oob_pages", 58, 8, 2, [wl.Request(300, 640, 2)])
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    used = set(int(x) for x in mat.page_table)
    spare = [i for i in range(mat.k_pages.shape[0]) if i not in used][0]
    k_ref, v_ref = mat.k_pages.copy(), mat.v_pages.copy()
    k_ref[spare] = 0
    v_ref[spare] = 0
    pt_ref = mat.page_table.copy()
    pt_dev = mat.page_table.copy()
    for idx, bad in ((3, mat.k_pages.shape[0] + 7), (9, -2), (12, 2 ** 31 - 1)):
        pt_ref[idx] = spare
        pt_dev[idx] = bad
    dev.page_table = torch.from_numpy(pt_dev).cuda()
    out, lse = dev.run_batch(ctx)
    r = w.requests[0]
    ref_o, ref_l = orc.attn_full(mat.q, k_ref, v_ref, pt_ref, r.prefix_len, w.Hkv, w.scale)
    compare(out, lse, ref_o, ref_l, "oob pages")


def test_attention_strided_cache_view(ctx):
    # the cache is a view into a wider allocation (one unused head slot per token, an unused token row
    # per page): only the three strides say where things are
    w = wl.Workload("strided", 44, 8, 2, [wl.Request(300, 200, 2), wl.Request(90, 0, 1)])
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    npg = mat.k_pages.shape[0]
    big_k = torch.full((npg, wl.PAGE + 1, w.Hkv + 1, w.D), 3.0e38, dtype=torch.bfloat16, device="cuda")
    big_v = torch.full_like(big_k, -3.0e38)
    big_k[:, :wl.PAGE, :w.Hkv] = dev.k
    big_v[:, :wl.PAGE, :w.Hkv] = dev.v
    dev.k, dev.v = big_k[:, :wl.PAGE, :w.Hkv], big_v[:, :wl.PAGE, :w.Hkv]
    dev.cache = binding.make_cache(dev.k, dev.v)
    assert dev.cache.stride_tok == (w.Hkv + 1) * w.D and dev.cache.stride_page == (wl.PAGE + 1) * (w.Hkv + 1) * w.D
    out, lse = dev.run_batch(ctx)
    for b, r in enumerate(w.requests):
        lo, hi = int(w.cu_new[b]), int(w.cu_new[b + 1])
        ref_o, ref_l = oracle_request(mat, b)
        compare(out[lo:hi], lse[:, lo:hi], ref_o, ref_l, "strided req %d" % b)
    # gather through the same view is bit-exact too
    r = w.requests[0]
    kr = torch.zeros((r.total_len, w.Hkv, w.D), dtype=torch.bfloat16, device="cuda")
    vr = torch.zeros_like(kr)
    pt = dev.page_table[:r.n_pages]
    binding.cp_kv_gather(ctx, dev.cache, pt, 0, r.total_len, kr, vr)
    torch.cuda.synchronize()
    pth = mat.page_table[:r.n_pages]
    assert np.array_equal(kr.view(torch.int16).cpu().numpy().view(np.uint16), orc.kv_gather(mat.k_pages, pth, 0, r.total_len))
    assert np.array_equal(vr.view(torch.int16).cpu().numpy().view(np.uint16), orc.kv_gather(mat.v_pages, pth, 0, r.total_len))


@pytest.mark.parametrize("scale", [0.5, 2.0])
def test_attention_peaked_scores_exercise_the_rescale_path(ctx, scale):
    # with 1/sqrt(D) and N(0,1) inputs the running row max hardly moves after the first key tile, so the lazy
    # rescale of O (taken when the max grows by more than 2^8) would never run; a large scale makes the scores
    # N(0, (scale * 11.3)^2): new maxima far above the old ones arrive in later tiles of most rows
    # (the outputs are then close to single V rows, up to 4-5 in magnitude: the bf16 rounding of such an output alone is
    # 2^-9 of it, so the absolute bars of the benchmark spec are applied relative to max(1, |reference|) here)
    def cmp(out, lse, ref_o, ref_l, what):
        assert np.isfinite(out).all() and np.isfinite(lse).all(), what
        d = np.abs(out - ref_o) / np.maximum(1.0, np.abs(ref_o))
        assert d.max() <= 2e-2 and d.mean() <= 2e-3, (what, d.max(), d.mean())
        le = np.abs(lse - ref_l) / np.maximum(1.0, np.abs(ref_l))
        assert le.max() <= 1e-3, (what, "lse", le.max())
        return d.max(), d.mean(), le.max()

    w = wl.Workload("peaked_%g" % scale, 77, 8, 2, [wl.Request(700, 1280, 2), wl.Request(300, 0, 1), wl.Request(130, 4096, 3)],
                    meta={"scale": scale})
    check_batch(ctx, w, cmp=cmp)
    w1 = wl.Workload("peaked_mha_%g" % scale, 78, 3, 3, [wl.Request(400, 896, 2)], meta={"scale": scale})
    check_batch(ctx, w1, cmp=cmp)


def test_attention_config1(ctx):
    check_batch(ctx, wl.config1())


def test_single_request_entry_point_and_c_invariance(ctx):
    w = wl.Workload("one", 21, 8, 2, [wl.Request(517, 320, 1)])
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    ref_o, ref_l = oracle_request(mat, 0)
    ws = torch.zeros(binding.cp_workspace_bytes([517], [8], w.Hq), dtype=torch.uint8, device="cuda")
    outs = []
    for C in (1, 2, 3, 8):
        dev.out.fill_(float("nan"))
        binding.cp_prefill_attn(ctx, dev.q, dev.cache, dev.page_table, 320, 517, C, w.Hq, w.scale, dev.out, dev.lse, ws)
        torch.cuda.synchronize()
        ctx.poll_status()
        compare(bf16_to_f64(dev.out), dev.lse.cpu().numpy().astype(np.float64), ref_o, ref_l, "C=%d" % C)
        outs.append((dev.out.clone(), dev.lse.clone()))
    # a launch over all shards walks the rows as one run whatever C is: the results are the same bits
    for o, l in outs[1:]:
        assert torch.equal(o.view(torch.int16), outs[0][0].view(torch.int16)) and torch.equal(l, outs[0][1])


def test_shard_partials_merge_to_full(ctx):
    w = wl.Workload("shards", 22, 8, 2, [wl.Request(700, 192, 3)])
    r = w.requests[0]
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    out_full, lse_full = dev.run_batch(ctx)
    C = r.C
    parts = torch.full((C, r.new_len, w.Hq, w.D), float("nan"), dtype=torch.float32, device="cuda")
    lses = torch.full((C, w.Hq, r.new_len), float("nan"), dtype=torch.float32, device="cuda")
    plan = orc.plan(r.new_len, r.prefix_len, C)
    for k in range(C):
        binding.cp_prefill_attn_shard(ctx, dev.q, dev.cache, dev.page_table, r.prefix_len, r.new_len, C, k, w.Hq,
                                      w.scale, parts[k], lses[k], dev.ws)
    torch.cuda.synchronize()
    ctx.poll_status()
    for k in range(C):
        own = np.zeros(r.new_len, dtype=bool)
        own[orc.shard_rows(plan[k])] = True
        lk = lses[k].cpu().numpy()
        assert np.isfinite(lk[:, own]).all() and np.isneginf(lk[:, ~own]).all()
        assert (parts[k].cpu().numpy()[~own] == 0).all()
    merged = torch.empty((r.new_len, w.Hq, w.D), dtype=torch.bfloat16, device="cuda")
    mlse = torch.empty((w.Hq, r.new_len), dtype=torch.float32, device="cuda")
    binding.cp_merge(ctx, parts, lses, merged, mlse)
    torch.cuda.synchronize()
    ref_o, ref_l = oracle_request(mat, 0)
    compare(bf16_to_f64(merged), mlse.cpu().numpy().astype(np.float64), ref_o, ref_l, "merged shards")
    assert np.abs(bf16_to_f64(merged) - out_full).max() <= 2.0 ** -7 * max(1.0, np.abs(out_full).max())


def test_key_range_partials_match_oracle_and_merge_to_full(ctx):
    # the keys of a request cut into disjoint absolute ranges with unaligned edges (inside the prefix, across
    # the prefix / suffix border, inside the suffix, an empty one): every partial against the oracle restricted
    # to the same keys; all of them through cp_merge against full attention
    w = wl.Workload("kvrange", 46, 8, 2, [wl.Request(700, 1000, 1)])
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    r = w.requests[0]
    R, P, L = r.new_len, r.prefix_len, r.total_len
    edges = [0, 130, 640, 1000, 1000, 1217, 1536, L]
    parts = torch.empty((len(edges) - 1, R, w.Hq, w.D), dtype=torch.float32, device="cuda")
    lses = torch.empty((len(edges) - 1, w.Hq, R), dtype=torch.float32, device="cuda")
    rows = np.unique(np.concatenate([np.arange(0, 40), np.arange(200, 240), np.arange(R - 40, R), [217, 218, 535, 536]]))
    for n, (lo, hi) in enumerate(zip(edges, edges[1:])):
        parts[n].fill_(float("nan"))
        lses[n].fill_(float("nan"))
        binding.cp_prefill_attn_kvrange(ctx, dev.q, dev.cache, dev.page_table, P, R, lo, hi, w.Hq, w.scale, parts[n],
                                        lses[n], dev.ws)
        torch.cuda.synchronize()
        ctx.poll_status()
        assert not bool(torch.isnan(parts[n]).any()) and not bool(torch.isnan(lses[n]).any())
        ref_o, ref_l = orc.attn_rows(mat.q, mat.k_pages, mat.v_pages, mat.page_table, P, w.Hkv, w.scale, rows,
                                     key_ranges=[(lo, hi)])
        o = parts[n][rows].cpu().numpy().astype(np.float64)
        l = lses[n][:, rows].cpu().numpy().astype(np.float64)
        seen = np.isfinite(ref_l)                         # rows (per head) that see a key of the range
        assert np.array_equal(np.isneginf(l), ~seen), (lo, hi)
        assert (o[~seen.T] == 0).all()
        if seen.any():
            assert np.abs(o - np.nan_to_num(ref_o)).max() <= 2e-2, (lo, hi)
            assert (np.abs(l[seen] - ref_l[seen]) / np.maximum(1.0, np.abs(ref_l[seen]))).max() <= 1e-3, (lo, hi)
    out = torch.empty((R, w.Hq, w.D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.Hq, R), dtype=torch.float32, device="cuda")
    binding.cp_merge(ctx, parts, lses, out, lse)
    torch.cuda.synchronize()
    ref_o, ref_l = oracle_request(mat, 0)
    compare(bf16_to_f64(out), lse.cpu().numpy().astype(np.float64), ref_o, ref_l, "merged key ranges")
    with pytest.raises(binding.CpError):
        binding.cp_prefill_attn_kvrange(ctx, dev.q, dev.cache, dev.page_table, P, R, 10, 5, w.Hq, w.scale, parts[0],
                                        lses[0], dev.ws)


@pytest.mark.parametrize("seed", range(2000, 2008))
def test_random_key_ranges_merge_to_full(ctx, seed):
    # a random request, its keys cut at random positions into 2..6 ranges, other page sizes included: the range
    # partials merged by cp_merge against the oracle
    u = wl.counter_uniform(seed, wl.TID_LEN, 0, 16)
    R = 1 + int(u[0] * 1500)
    P = int(u[1] * 6000) if u[2] < 0.8 else 0
    page = [16, 32, 64, 128][int(u[3] * 4)]
    heads = [(8, 2), (4, 4), (16, 2)][int(u[4] * 3)]
    w = wl.Workload("kvr_%d" % seed, seed, heads[0], heads[1], [wl.Request(R, P, 1)], page=page)
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    L = R + P
    n_cuts = 1 + int(u[5] * 5)
    edges = sorted({0, L} | {int(x * L) for x in u[6:6 + n_cuts]})
    parts = torch.empty((len(edges) - 1, R, w.Hq, w.D), dtype=torch.float32, device="cuda")
    lses = torch.empty((len(edges) - 1, w.Hq, R), dtype=torch.float32, device="cuda")
    for n, (lo, hi) in enumerate(zip(edges, edges[1:])):
        binding.cp_prefill_attn_kvrange(ctx, dev.q, dev.cache, dev.page_table, P, R, lo, hi, w.Hq, w.scale, parts[n],
                                        lses[n], dev.ws)
    out = torch.empty((R, w.Hq, w.D), dtype=torch.bfloat16, device="cuda")
    lse = torch.empty((w.Hq, R), dtype=torch.float32, device="cuda")
    binding.cp_merge(ctx, parts, lses, out, lse)
    torch.cuda.synchronize()
    ctx.poll_status()
    ref_o, ref_l = oracle_request(mat, 0)
    compare(bf16_to_f64(out), lse.cpu().numpy().astype(np.float64), ref_o, ref_l, "random key ranges %s" % edges)


def test_argument_validation_launches_nothing(ctx):
    w = wl.Workload("val", 23, 8, 2, [wl.Request(64, 0, 1)])
    dev = DeviceWorkload(wl.materialize(w))
    small = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(binding.CpError) as e:
        binding.cp_prefill_attn(ctx, dev.q, dev.cache, dev.page_table, 0, 64, 1, w.Hq, w.scale, dev.out, dev.lse, small)
    assert e.value.code == binding.CP_ERR_WORKSPACE
    with pytest.raises(binding.CpError) as e:
        binding.cp_prefill_attn(ctx, dev.q, dev.cache, dev.page_table, 0, 64, 1, 7, w.scale, dev.out, dev.lse, dev.ws)
    assert e.value.code == binding.CP_ERR_INVALID_ARG      # Hq = 7 is not a multiple of Hkv = 2
    with pytest.raises(binding.CpError) as e:
        binding.cp_prefill_attn(ctx, dev.q, dev.cache, dev.page_table, 0, 0, 1, w.Hq, w.scale, dev.out, dev.lse, dev.ws)
    assert e.value.code == binding.CP_ERR_INVALID_ARG
    bad = binding.make_cache(dev.k, dev.v)
    bad.page_size = 48                                      # pages of 16, 32, 64 or 128 tokens only
    with pytest.raises(binding.CpError) as e:
        binding.cp_prefill_attn(ctx, dev.q, bad, dev.page_table, 0, 64, 1, w.Hq, w.scale, dev.out, dev.lse, dev.ws)
    assert e.value.code == binding.CP_ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert torch.isnan(dev.out.float()).all()               # nothing was written


def test_schedule_reuse_gives_identical_results(ctx):
    # the same batch three times with schedule reuse on (new q and cache contents in between), then another
    # shape and the first one again: bit-identical to the results without reuse
    w1, w2 = wl.small_mixed(), wl.Workload("other", 47, 8, 2, [wl.Request(500, 256, 2), wl.Request(90, 0, 1)])
    d1, d2 = DeviceWorkload(wl.materialize(w1)), DeviceWorkload(wl.materialize(w2))
    ref1 = [t.clone() for t in (d1.run_batch(ctx) and (d1.out, d1.lse))]
    ref2 = [t.clone() for t in (d2.run_batch(ctx) and (d2.out, d2.lse))]
    ctx.cache_schedule(True)
    try:
        for dev, ref in ((d1, ref1), (d1, ref1), (d1, ref1), (d2, ref2), (d1, ref1), (d2, ref2), (d2, ref2)):
            dev.out.fill_(float("nan"))
            dev.lse.fill_(float("nan"))
            dev.run_batch(ctx)
            assert torch.equal(dev.out.view(torch.int16), ref[0].view(torch.int16)) and torch.equal(dev.lse, ref[1])
        # same shape, other data: the remembered work lists serve a new q
        q_old = d1.q.clone()
        d1.q.copy_(torch.flip(q_old, dims=[2]))
        d1.run_batch(ctx)
        flipped = d1.out.clone()
        ctx.cache_schedule(False)
        d1.run_batch(ctx)
        assert torch.equal(flipped.view(torch.int16), d1.out.view(torch.int16))
        assert not torch.equal(flipped.view(torch.int16), ref1[0].view(torch.int16))
    finally:
        ctx.cache_schedule(False)


def test_expired_wait_is_reported_and_context_survives(ctx):
    # a block waits (about a millisecond) on a barrier nothing arrives at: the kernel returns, the status word
    # carries the time-out, polling clears it, and the same context computes correct attention afterwards
    ctx.selftest_wait_expiry()
    torch.cuda.synchronize()
    with pytest.raises(binding.CpError) as e:
        ctx.poll_status()
    assert e.value.code == binding.CP_ERR_TIMEOUT and "barrier 0, block 0, iteration 7" in str(e.value)
    ctx.poll_status()                                                       # cleared
    check_batch(ctx, wl.Workload("after_timeout", 44, 8, 2, [wl.Request(300, 128, 2)]))


def test_attention_config2_full(ctx):
    check_batch(ctx, wl.config2(), pair_budget=1e11)


def test_attention_config4_varlen(ctx):
    check_batch(ctx, wl.config4(), pair_budget=1.5e8)


def test_attention_variant_gqa8_and_chunked_prefill(ctx):
    # eight query heads per KV head; a short chunk behind a long cached prefix (all units KV-split)
    check_batch(ctx, wl.variant_gqa8(), pair_budget=2e8)
    w = wl.variant_chunked_prefill()
    info, _, _ = binding.cp_schedule_inspect(w.cu_new, [65536], [2], w.Hq, w.Hkv,
                                             torch.cuda.get_device_properties(0).multi_processor_count, want_lists=False)
    assert info["split_units"] == 64 and info["max_load"] * info["grid"] <= 1.02 * info["total"]
    check_batch(ctx, w, pair_budget=2e8)


def _random_workload(seed):
    u = wl.counter_uniform(seed, wl.TID_LEN, 0, 64)
    heads = [(8, 2), (4, 4), (6, 2), (16, 2), (32, 4), (8, 8), (2, 1)][int(u[0] * 7)]
    B = 1 + int(u[1] * 6)
    reqs = []
    for b in range(B):
        scale = float(os.environ.get("CPATTN_FUZZ_SCALE", "1"))            # > 1: longer requests, more KV splits
        R = max(1, int(round(scale * 2.0 ** (u[2 + 4 * b] * 11.5))))         # 1 .. ~2900, log-uniform
        kind = u[3 + 4 * b]
        P = 0 if kind < 0.25 else int(u[4 + 4 * b] * 8192 * scale)
        if kind < 0.75:
            P = P // 64 * 64                                                 # mostly page-aligned prefixes
        C = [1, 2, 3, 4, 5, 8][int(u[5 + 4 * b] * 6)]
        reqs.append(wl.Request(R, P, C))
    return wl.Workload("random_%d" % seed, seed, heads[0], heads[1], reqs)


@pytest.mark.parametrize("seed", range(1000, 1000 + int(os.environ.get("CPATTN_FUZZ_CASES", "48"))))
def test_attention_random_batches(ctx, seed):
    # seeded random batches: head shapes with even, odd and unit group sizes, ragged lengths from one token
    # up, prefixes that are absent, page-aligned or not, every supported kind of C
    check_batch(ctx, _random_workload(seed), pair_budget=6e6, seed_rows=seed)


def test_attention_config5_sampled(ctx):
    check_batch(ctx, wl.config5(), pair_budget=1.2e9)


def test_attention_config3_sampled(ctx):
    # 512 seeded random rows for every head, compared exactly, plus chunk-boundary rows for all heads.
    w = wl.config3()
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    out, lse = dev.run_batch(ctx)
    r = w.requests[0]
    rows = wl.sample_rows(w.seed, w.Hq, r.new_len, 512)                       # [Hq, 512]
    heads = np.repeat(np.arange(w.Hq, dtype=np.int32), 512)
    ro, rl = orc.attn_pairs(mat.q, mat.k_pages, mat.v_pages, mat.page_table, 0, w.Hkv, w.scale, rows.reshape(-1), heads)
    got_o = out[rows.reshape(-1), heads]
    got_l = lse[heads, rows.reshape(-1)]
    compare(got_o, got_l, ro, rl, "cfg3 sampled")
    cl = r.new_len // (2 * r.C)
    edge = np.unique(np.clip([x for j in range(2 * r.C + 1) for x in (j * cl - 1, j * cl)], 0, r.new_len - 1))
    eo, el = orc.attn_rows(mat.q, mat.k_pages, mat.v_pages, mat.page_table, 0, w.Hkv, w.scale, edge[::3])
    compare(out[edge[::3]], lse[:, edge[::3]], eo, el, "cfg3 chunk edges")
    assert np.isfinite(lse).all() and np.isfinite(out).all()
    # the LSE-merge invariant over ALL rows at full size: the C shard partials, each computed on its own,
    # merge into the one-launch result (every row is owned by exactly one shard)
    del out, lse
    R = r.new_len
    parts = torch.empty((r.C, R, w.Hq, w.D), dtype=torch.float32, device="cuda")
    lses = torch.empty((r.C, w.Hq, R), dtype=torch.float32, device="cuda")
    for k in range(r.C):
        binding.cp_prefill_attn_shard(ctx, dev.q, dev.cache, dev.page_table, 0, R, r.C, k, w.Hq, w.scale, parts[k],
                                      lses[k], dev.ws)
    torch.cuda.synchronize()
    ctx.poll_status()
    assert bool((torch.isfinite(lses).sum(0) == 1).all())
    merged = torch.empty((R, w.Hq, w.D), dtype=torch.bfloat16, device="cuda")
    mlse = torch.empty((w.Hq, R), dtype=torch.float32, device="cuda")
    binding.cp_merge(ctx, parts, lses, merged, mlse)
    torch.cuda.synchronize()
    del parts
    diff = (merged.float() - dev.out.float()).abs()
    assert float(diff.max()) <= 2e-2 and float(diff.mean()) <= 1e-4
    assert float(((mlse - dev.lse).abs() / dev.lse.abs().clamp(min=1.0)).max()) <= 1e-3
