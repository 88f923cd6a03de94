"""The multi-rank CP worker on CPU: layout arithmetic against the oracle's planner, the whole exchange +
attention orchestration with four in-process ranks, and with two gloo ranks over real collectives.
The device steps are stood in for by the oracle (tests/cp_rank_util.py); what is checked here is the
data movement: which rows a rank sends, where gathered rows land in its paged cache, which keys each
chunk call may rely on."""
import os
import socket
import sys
import threading

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import reference as orc
from paper_2609_04774_b200 import workloads as wl
from paper_2609_04774_b200.cp_rank import CpRankWorker, RankLayout, TorchComm

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("R,P,C", [(333, 192, 3), (5, 0, 4), (4096, 12288, 4), (700, 64, 2), (1, 64, 1), (129, 448, 8)])
def test_layout_matches_oracle_plan(R, P, C):
    shards = orc.plan(R, P, C)
    covered = np.zeros(P, dtype=np.int32)
    for k in range(C):
        lay = RankLayout(R, P, C, k)
        assert [lay.chunk(lay.early), lay.chunk(lay.late)] == [tuple(c) for c in zip(shards[k]["q_begin"], shards[k]["q_end"])]
        assert lay.late_chunk_of(k) == lay.late
        b, e = lay.prefix_block(k)
        assert b % 64 == 0 and e % 64 == 0 and e - b <= lay.block_pages * 64
        covered[b:e] += 1
    assert (covered == 1).all()                      # prefix blocks tile [0, P) exactly once
    assert lay.C * lay.cl * 2 >= R


def test_layout_rejects_bad_arguments():
    with pytest.raises(ValueError):
        RankLayout(10, 30, 2, 0)                     # prefix not page aligned
    with pytest.raises(ValueError):
        RankLayout(10, 0, 2, 2)


def _run_rank(w, mat, lay, comm, seed, result, pass_q=False):
    from cp_rank_util import OracleOps, rank_inputs
    k_pages, v_pages, page_table, rows = rank_inputs(mat, lay, seed)
    ops = OracleOps(k_pages, v_pages, page_table, w.Hq, w.scale)
    t = {k: torch.from_numpy(np.ascontiguousarray(v).view(np.int16)) for k, v in rows.items()}
    worker = CpRankWorker(lay, comm, ops)
    run = worker.prefill_pass_q if pass_q else worker.prefill
    out_e, lse_e, out_l, lse_l = run(t["q_early"], t["q_late"], t["k_early"], t["v_early"], t["k_late"], t["v_late"])
    as_np = lambda x: x.numpy() if isinstance(x, torch.Tensor) else x
    result[lay.rank] = (as_np(out_e), as_np(lse_e), as_np(out_l), as_np(lse_l), k_pages, v_pages, page_table)


def _check_rank(w, mat, lay, res, pass_q=False):
    out_e, lse_e, out_l, lse_l, k_pages, v_pages, page_table = res
    r = w.requests[0]
    ref_o, ref_l = orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, r.prefix_len, w.Hkv, w.scale)
    for j, o, l in ((lay.early, out_e, lse_e), (lay.late, out_l, lse_l)):
        b, e = lay.chunk(j)
        assert o.shape[0] == e - b
        if e > b:
            assert np.abs(o - ref_o[b:e]).max() < 1e-12 and np.abs(l - ref_l[:, b:e]).max() < 1e-12
    if pass_q:
        # K/V stayed sharded: the rank's cache holds its prefix block and its own chunks, nothing else
        own = np.zeros(r.prefix_len + r.new_len, dtype=bool)
        pb, pe = lay.prefix_block(lay.rank)
        own[pb:pe] = True
        for j in (lay.early, lay.late):
            b, e = lay.chunk(j)
            own[r.prefix_len + b:r.prefix_len + e] = True
        got = orc.kv_gather(k_pages, page_table, 0, own.size)
        ref = orc.kv_gather(mat.k_pages, mat.page_table, 0, own.size)
        assert np.array_equal(got[own], ref[own]) and not got[~own].any()
        return
    # after the exchange the rank's own cache holds every token of the request, bit for bit
    L = r.prefix_len + r.new_len
    assert np.array_equal(orc.kv_gather(k_pages, page_table, 0, L), orc.kv_gather(mat.k_pages, mat.page_table, 0, L))
    assert np.array_equal(orc.kv_gather(v_pages, page_table, 0, L), orc.kv_gather(mat.v_pages, mat.page_table, 0, L))


@pytest.mark.parametrize("pass_q", [False, True])
@pytest.mark.parametrize("R,P,C", [(333, 192, 4), (5, 0, 4), (200, 320, 3)])
def test_four_ranks_in_process(R, P, C, pass_q):
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from cp_rank_util import ThreadFabric
    w = wl.Workload("cp_rank", 51, 4, 2, [wl.Request(R, P, C)])
    mat = wl.materialize(w)
    fabric = ThreadFabric(C)
    result, errors = {}, []

    def body(k):
        try:
            _run_rank(w, mat, RankLayout(R, P, C, k), fabric.comm(k), 51, result, pass_q)
        except Exception as e:               # a failing rank must not leave the others at the barrier
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=body, args=(k,)) for k in range(C)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    for k in range(C):
        _check_rank(w, mat, RankLayout(R, P, C, k), result[k], pass_q)


@pytest.mark.parametrize("R,P,C", [(512, 256, 4), (509, 192, 4), (128, 0, 1), (254, 640, 2), (1536, 64, 3), (333, 192, 4)])
def test_landing_table_reads_the_gathers_in_token_order(R, P, C):
    # emulate the three all-gathers (rank r's contribution lands at slot r of each arena part) with token ids as
    # payload, then read every logical token through the landing page table
    from paper_2609_04774_b200.cp_rank import landing_pages, landing_rows, landing_table
    lay = RankLayout(R, P, C, 0)
    table = landing_table(lay, 1000)
    if lay.cl % lay.page:
        assert table is None
        return
    n_blk, cl = lay.block_pages * lay.page, lay.cl
    arena = np.full(landing_pages(lay) * lay.page, -1, dtype=np.int64)
    assert arena.size == C * (n_blk + 2 * cl)
    for r in range(C):
        b, e = lay.prefix_block(r)
        arena[r * n_blk:r * n_blk + (e - b)] = np.arange(b, e)
        for part, j in ((0, r), (1, lay.late_chunk_of(r))):
            b, e = lay.chunk(j)
            row0 = C * n_blk + part * C * cl + r * cl
            arena[row0:row0 + (e - b)] = P + np.arange(b, e)
    assert len(table) == -(-(P + R) // lay.page)
    t = np.arange(P + R)
    rows = (np.asarray(table)[t // lay.page] - 1000) * lay.page + t % lay.page
    assert np.array_equal(arena[rows], t)
    # the runs cover [0, P + R) exactly once, in token order
    runs = landing_rows(lay)
    assert runs[0][0] == 0 and all(a[0] + a[1] == b[0] for a, b in zip(runs, runs[1:])) and runs[-1][0] + runs[-1][1] == P + R


@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("R,P,C", [(512, 256, 4), (509, 192, 4), (254, 0, 2)])
def test_ranks_in_process_landing_mode(R, P, C, fp8):
    # the gathers land in pages of the rank's own pool and a page table reads them in token order: no appends at all,
    # results equal the oracle's, and the pool read through that table holds the whole request bit for bit
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from cp_rank_util import OracleOps, OracleOps8, ThreadFabric, rank_inputs, rank_inputs8
    from oracle import fp8 as o8
    from paper_2609_04774_b200.cp_rank import landing_pages
    w = wl.Workload("cp_rank_land", 57, 4, 2, [wl.Request(R, P, C)])
    mat = wl.materialize(w)
    m8 = wl.materialize_fp8(w) if fp8 else None
    fabric = ThreadFabric(C)
    result, errors = {}, []

    def body(k):
        try:
            lay = RankLayout(R, P, C, k)
            k_pages, v_pages, page_table, rows = rank_inputs8(m8, mat, lay, 57) if fp8 else rank_inputs(mat, lay, 57)
            a0 = k_pages.shape[0]
            extra = np.zeros((landing_pages(lay),) + k_pages.shape[1:], dtype=k_pages.dtype)
            k_pages, v_pages = np.concatenate([k_pages, extra]), np.concatenate([v_pages, extra])
            ops = (OracleOps8(k_pages, v_pages, m8.k_scale, m8.v_scale, page_table, w.Hq, w.scale, arena_page0=a0) if fp8
                   else OracleOps(k_pages, v_pages, page_table, w.Hq, w.scale, arena_page0=a0))
            ops.kv_append_segments = None            # landing mode must not append anything
            t = {n: torch.from_numpy(np.ascontiguousarray(v).view(np.int16)) for n, v in rows.items()}
            out = CpRankWorker(lay, fabric.comm(k), ops).prefill(t["q_early"], t["q_late"], t["k_early"], t["v_early"],
                                                                   t["k_late"], t["v_late"])
            result[k] = tuple(x.numpy() if isinstance(x, torch.Tensor) else x for x in out) + (k_pages, v_pages, ops.landing(lay)[2])
        except Exception as e:
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=body, args=(k,)) for k in range(C)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    L = P + R
    if fp8:
        ref_o, ref_l, _ = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv,
                                           w.scale, np.arange(R))
        ref_k, ref_v = orc.kv_gather(m8.k8_pages, m8.page_table, 0, L), orc.kv_gather(m8.v8_pages, m8.page_table, 0, L)
    else:
        ref_o, ref_l = orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, P, w.Hkv, w.scale)
        ref_k, ref_v = orc.kv_gather(mat.k_pages, mat.page_table, 0, L), orc.kv_gather(mat.v_pages, mat.page_table, 0, L)
    for k in range(C):
        lay = RankLayout(R, P, C, k)
        out_e, lse_e, out_l, lse_l, k_pages, v_pages, table = result[k]
        for j, o, l in ((lay.early, out_e, lse_e), (lay.late, out_l, lse_l)):
            b, e = lay.chunk(j)
            assert o.shape[0] == e - b and e > b
            assert np.abs(o - ref_o[b:e]).max() < 1e-12 and np.abs(l - ref_l[:, b:e]).max() < 1e-12
        got_k, got_v = orc.kv_gather(k_pages, table, 0, L), orc.kv_gather(v_pages, table, 0, L)
        if fp8:      # codes of +0 and -0 may differ between a rank's quantiser and the reference's: compare values
            assert np.array_equal(o8.e4m3_decode(got_k), o8.e4m3_decode(ref_k)) and np.array_equal(o8.e4m3_decode(got_v), o8.e4m3_decode(ref_v))
        else:
            assert np.array_equal(got_k, ref_k) and np.array_equal(got_v, ref_v)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _gloo_rank(rank, world, port, q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        R, P = 333, 192
        w = wl.Workload("cp_rank", 52, 4, 2, [wl.Request(R, P, world)])
        mat = wl.materialize(w)
        lay = RankLayout(R, P, world, rank)
        result = {}
        _run_rank(w, mat, lay, TorchComm(), 52, result)
        _check_rank(w, mat, lay, result[rank])
        result = {}
        _run_rank(w, mat, lay, TorchComm(), 52, result, pass_q=True)
        _check_rank(w, mat, lay, result[rank], pass_q=True)
        q.put((rank, "ok"))
    except Exception as e:
        q.put((rank, repr(e)))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_gloo_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=240) for _ in procs)
    for p in procs:
        p.join(timeout=60)
    assert got == [(0, "ok"), (1, "ok")]


@pytest.mark.parametrize("R,P,C", [(333, 192, 4), (5, 0, 4), (200, 320, 3)])
def test_four_ranks_in_process_fp8_cache(R, P, C):
    # the same exchange with FP8 caches: stored bytes travel, every rank's cache ends up holding the whole request's
    # bytes, and each chunk's result is the FP8 oracle's on those bytes
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from cp_rank_util import OracleOps8, ThreadFabric, rank_inputs8
    from oracle import fp8 as o8
    w = wl.Workload("cp_rank8", 53, 4, 2, [wl.Request(R, P, C)])
    m8, mat = wl.materialize_fp8(w), wl.materialize(w)
    fabric = ThreadFabric(C)
    result, errors = {}, []

    def body(k):
        try:
            lay = RankLayout(R, P, C, k)
            k_pages, v_pages, page_table, rows = rank_inputs8(m8, mat, lay, 53)
            ops = OracleOps8(k_pages, v_pages, m8.k_scale, m8.v_scale, page_table, w.Hq, w.scale)
            t = {n: torch.from_numpy(np.ascontiguousarray(v).view(np.int16)) for n, v in rows.items()}
            out = CpRankWorker(lay, fabric.comm(k), ops).prefill(t["q_early"], t["q_late"], t["k_early"], t["v_early"],
                                                                   t["k_late"], t["v_late"])
            result[k] = out + (k_pages, v_pages, page_table)
        except Exception as e:
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=body, args=(k,)) for k in range(C)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=300)
    assert not errors, errors
    ref_o, ref_l, _ = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv, w.scale,
                                       np.arange(R))
    L = P + R
    for k in range(C):
        lay = RankLayout(R, P, C, k)
        out_e, lse_e, out_l, lse_l, k_pages, v_pages, page_table = result[k]
        for j, o, l in ((lay.early, out_e, lse_e), (lay.late, out_l, lse_l)):
            b, e = lay.chunk(j)
            if e > b:
                assert np.abs(o - ref_o[b:e]).max() < 1e-12 and np.abs(l - ref_l[:, b:e]).max() < 1e-12
        for got, ref in ((k_pages, m8.k8_pages), (v_pages, m8.v8_pages)):
            a = o8.e4m3_decode(orc.kv_gather(got, page_table, 0, L))
            assert np.array_equal(a, o8.e4m3_decode(orc.kv_gather(ref, m8.page_table, 0, L)))
