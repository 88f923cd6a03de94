"""The multi-rank CP worker on one GPU: C ranks run as host threads, each with its own paged cache, its
own context and the library's kernels; rows are exchanged through an in-process communicator (a host
barrier, no kernel waits on another).  Plus the chunk entry point on its own, and the NCCL communicator
at world size 1 in a child process."""
import os
import socket
import sys
import threading

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

from oracle import reference as orc
from paper_2609_04774_b200 import workloads as wl

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _dev(bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def _f64(t):
    return t.float().cpu().numpy().astype(np.float64)


def _compare(o, l, ref_o, ref_l, what):
    err = np.abs(_f64(o) - ref_o)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (what, err.max(), err.mean())
    lerr = np.abs(_f64(l) - ref_l) / np.maximum(1.0, np.abs(ref_l))
    assert lerr.max() <= 1e-3, (what, lerr.max())


@pytest.mark.parametrize("page", [64, 16])
def test_chunk_entry_point_matches_oracle_rows(page):
    from paper_2609_04774_b200 import binding
    w = wl.Workload("chunk_call", 61, 8, 2, [wl.Request(1000, 320, 3)], page=page)
    mat = wl.materialize(w)
    r = w.requests[0]
    ctx = binding.Context(0)
    k, v = _dev(mat.k_pages), _dev(mat.v_pages)
    cache = binding.make_cache(k, v)
    pt = torch.from_numpy(mat.page_table).cuda()
    ws = torch.empty(binding.cp_workspace_bytes([r.new_len], [r.C], w.Hq), dtype=torch.uint8, device="cuda")
    plan = orc.plan(r.new_len, r.prefix_len, r.C)
    ref_o, ref_l = orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, r.prefix_len, w.Hkv, w.scale)
    for j in range(2 * r.C):
        shard = j if j < r.C else 2 * r.C - 1 - j
        half = 0 if j < r.C else 1
        b, e = plan[shard]["q_begin"][half], plan[shard]["q_end"][half]
        n = e - b
        q = _dev(mat.q[b:e])
        out = torch.full((n, w.Hq, w.D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((w.Hq, n), float("nan"), dtype=torch.float32, device="cuda")
        binding.cp_prefill_attn_chunk(ctx, q, cache, pt, r.prefix_len, r.new_len, r.C, j, w.Hq, w.scale, out, lse, ws)
        torch.cuda.synchronize()
        ctx.poll_status()
        _compare(out, lse, ref_o[b:e], ref_l[:, b:e], "chunk %d" % j)
    with pytest.raises(binding.CpError):
        binding.cp_prefill_attn_chunk(ctx, q, cache, pt, r.prefix_len, r.new_len, r.C, 2 * r.C, w.Hq, w.scale, out, lse, ws)


def _rank_on_gpu(w, mat, lay, comm, seed, result, pass_q=False):
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from cp_rank_util import rank_inputs
    from paper_2609_04774_b200 import binding
    from paper_2609_04774_b200.cp_rank import CpRankWorker, LibraryOps
    torch.cuda.set_device(0)
    k_pages, v_pages, page_table, rows = rank_inputs(mat, lay, seed)
    ops = LibraryOps(binding.Context(0), _dev(k_pages), _dev(v_pages), torch.from_numpy(page_table).cuda(), w.Hq, w.scale)
    t = {k: _dev(x) for k, x in rows.items()}
    worker = CpRankWorker(lay, comm, ops)
    run = worker.prefill_pass_q if pass_q else worker.prefill
    out = run(t["q_early"], t["q_late"], t["k_early"], t["v_early"], t["k_late"], t["v_late"])
    torch.cuda.synchronize()
    ops.ctx.poll_status()
    result[lay.rank] = out + (ops.k_pages, ops.v_pages, page_table)


def _check_rank_on_gpu(w, mat, lay, res, ref, pass_q=False):
    out_e, lse_e, out_l, lse_l, k_pages, v_pages, page_table = res
    r = w.requests[0]
    for j, o, l in ((lay.early, out_e, lse_e), (lay.late, out_l, lse_l)):
        b, e = lay.chunk(j)
        assert o.shape[0] == e - b
        if e > b:
            _compare(o, l, ref[0][b:e], ref[1][:, b:e], "rank %d chunk %d" % (lay.rank, j))
    if pass_q:
        return                                   # K/V stays sharded in this mode: nothing more to find in the cache
    L = r.prefix_len + r.new_len
    for dev_pages, ref_pages in ((k_pages, mat.k_pages), (v_pages, mat.v_pages)):
        got = dev_pages.view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(orc.kv_gather(got, page_table, 0, L), orc.kv_gather(ref_pages, mat.page_table, 0, L))


@pytest.mark.parametrize("pass_q", [False, True])
@pytest.mark.parametrize("R,P,C", [(1500, 640, 4), (333, 192, 3), (5, 0, 4)])
def test_ranks_as_threads_on_one_gpu(R, P, C, pass_q):
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from cp_rank_util import ThreadFabric
    from paper_2609_04774_b200.cp_rank import RankLayout
    w = wl.Workload("cp_rank_gpu", 62, 8, 2, [wl.Request(R, P, C)])
    mat = wl.materialize(w)
    ref = orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, P, w.Hkv, w.scale)
    fabric = ThreadFabric(C)
    result, errors = {}, []

    def body(k):
        try:
            _rank_on_gpu(w, mat, RankLayout(R, P, C, k), fabric.comm(k), 62, result, pass_q)
        except Exception as e:
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=body, args=(k,)) for k in range(C)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=600)
    assert not errors, errors
    for k in range(C):
        _check_rank_on_gpu(w, mat, RankLayout(R, P, C, k), result[k], ref, pass_q)


def _nccl_single_rank(port, q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    try:
        torch.cuda.set_device(0)
        dist.init_process_group("nccl", rank=0, world_size=1)
        from paper_2609_04774_b200.cp_rank import RankLayout, TorchComm
        R, P = 700, 256
        w = wl.Workload("cp_rank_nccl", 63, 8, 2, [wl.Request(R, P, 1)])
        mat = wl.materialize(w)
        ref = orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, P, w.Hkv, w.scale)
        lay = RankLayout(R, P, 1, 0)
        result = {}
        _rank_on_gpu(w, mat, lay, TorchComm(), 63, result)
        _check_rank_on_gpu(w, mat, lay, result[0], ref)
        result = {}
        _rank_on_gpu(w, mat, lay, TorchComm(), 63, result, pass_q=True)          # NCCL all-to-all at world size 1
        _check_rank_on_gpu(w, mat, lay, result[0], ref, pass_q=True)
        q.put("ok")
    except Exception as e:
        q.put(repr(e))
    finally:
        if dist.is_initialized():
            dist.destroy_process_group()


def test_nccl_communicator_world_size_one():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    p = ctx.Process(target=_nccl_single_rank, args=(port, q))
    p.start()
    got = q.get(timeout=600)
    p.join(timeout=120)
    assert got == "ok"


def test_rank_step_replays_from_a_cuda_graph():
    # a rank step whose chunk calls carry their work lists in the launch parameters reads no host memory after the
    # calls return, so the whole step (gathers, segment appends, both chunk attention calls) can be captured once and
    # replayed per layer: the replay must reproduce the eager results bit for bit, also after the inputs have changed
    # in place
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from cp_rank_util import ThreadFabric, rank_inputs
    from paper_2609_04774_b200 import binding
    from paper_2609_04774_b200.cp_rank import CpRankWorker, LibraryOps, RankLayout
    R, P, C = 1000, 640, 1
    w = wl.Workload("cp_rank_graph", 64, 8, 2, [wl.Request(R, P, C)])
    mat = wl.materialize(w)
    lay = RankLayout(R, P, C, 0)
    for j in (lay.early, lay.late):
        b, e = lay.chunk(j)
        info, _, _ = binding.cp_schedule_inspect([0, e - b], [P + b], [1], w.Hq, w.Hkv,
                                                 torch.cuda.get_device_properties(0).multi_processor_count, want_lists=False)
        assert info["inline"] == 1
    k_pages, v_pages, page_table, rows = rank_inputs(mat, lay, 64)
    ops = LibraryOps(binding.Context(0), _dev(k_pages), _dev(v_pages), torch.from_numpy(page_table).cuda(), w.Hq, w.scale)
    t = {k: _dev(x) for k, x in rows.items()}
    worker = CpRankWorker(lay, ThreadFabric(1).comm(0), ops)
    run = lambda: worker.prefill(t["q_early"], t["q_late"], t["k_early"], t["v_early"], t["k_late"], t["v_late"])
    eager = [x.clone() for x in run()]
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run()                                               # warm-up on a side stream, as graph capture wants
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        captured = run()
    graph.replay()
    torch.cuda.synchronize()
    ops.ctx.poll_status()
    for a, b in zip(eager, captured):
        assert torch.equal(a.view(torch.int16) if a.dtype == torch.bfloat16 else a, b.view(torch.int16) if b.dtype == torch.bfloat16 else b)
    ref = orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, P, w.Hkv, w.scale)
    _check_rank_on_gpu(w, mat, lay, tuple(captured) + (ops.k_pages, ops.v_pages, page_table), ref)
    # new queries in the same buffers: the replay computes on them
    t["q_early"].copy_(torch.flip(t["q_early"], dims=[2]))
    graph.replay()
    torch.cuda.synchronize()
    replayed = [x.clone() for x in captured]
    again = [x.clone() for x in run()]
    torch.cuda.synchronize()
    assert torch.equal(replayed[0].view(torch.int16), again[0].view(torch.int16)) and torch.equal(replayed[1], again[1])
    assert not torch.equal(replayed[0].view(torch.int16), eager[0].view(torch.int16))


def test_large_schedule_refuses_capture():
    # a call whose work lists do not fit the launch parameters stages them through pinned buffers; on a capturing
    # stream it must refuse (nothing enqueued) instead of recording a copy that would replay stale lists
    from paper_2609_04774_b200 import binding
    R = 40000
    w = wl.Workload("big_sched", 65, 8, 2, [wl.Request(R, 0, 1)])
    info, _, _ = binding.cp_schedule_inspect([0, R], [0], [1], w.Hq, w.Hkv,
                                             torch.cuda.get_device_properties(0).multi_processor_count, want_lists=False)
    assert info["inline"] == 0
    ctx = binding.Context(0)
    pages = -(-R // 64)
    k = torch.zeros((pages, 64, w.Hkv, 128), dtype=torch.bfloat16, device="cuda")
    cache = binding.make_cache(k, k)
    pt = torch.arange(pages, dtype=torch.int32, device="cuda")
    q = torch.zeros((R, w.Hq, 128), dtype=torch.bfloat16, device="cuda")
    out = torch.full_like(q, float("nan"))
    lse = torch.empty((w.Hq, R), dtype=torch.float32, device="cuda")
    ws = torch.zeros(binding.cp_workspace_bytes([R], [1], w.Hq), dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with pytest.raises(binding.CpError) as e:
        with torch.cuda.graph(graph):
            binding.cp_prefill_attn(ctx, q, cache, pt, 0, R, 1, w.Hq, w.scale, out, lse, ws)
    assert e.value.code == binding.CP_ERR_UNSUPPORTED and "captured" in str(e.value)
    torch.cuda.synchronize()
    assert bool(torch.isnan(out.float()).all())             # nothing ran
    binding.cp_prefill_attn(ctx, q, cache, pt, 0, R, 1, w.Hq, w.scale, out, lse, ws)      # outside capture it runs
    torch.cuda.synchronize()
    ctx.poll_status()
    assert not bool(torch.isnan(out.float()).any())
    ctx.close()


@pytest.mark.parametrize("R,P,C", [(1500, 640, 4), (333, 192, 3), (5, 0, 4)])
def test_ranks_as_threads_on_one_gpu_fp8_cache(R, P, C):
    # the rank worker on FP8 caches with the library's kernels: quantising append of the own rows, raw byte gathers,
    # raw segment appends, FP8 chunk attention; results within the FP8 variant's bound of the oracle on the stored
    # bytes, and every rank's cache holds the whole request's bytes afterwards
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from cp_rank_util import ThreadFabric, rank_inputs8
    from oracle import fp8 as o8
    from paper_2609_04774_b200 import binding
    from paper_2609_04774_b200.cp_rank import CpRankWorker, LibraryOps8, RankLayout
    from tests.test_gpu_fp8 import compare8
    w = wl.Workload("cp_rank_gpu8", 66, 8, 2, [wl.Request(R, P, C)])
    m8, mat = wl.materialize_fp8(w), wl.materialize(w)
    ro, rl, ra = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv, w.scale,
                                  np.arange(R))
    fabric = ThreadFabric(C)
    result, errors = {}, []

    def body(k):
        try:
            torch.cuda.set_device(0)
            lay = RankLayout(R, P, C, k)
            k_pages, v_pages, page_table, rows = rank_inputs8(m8, mat, lay, 66)
            ops = LibraryOps8(binding.Context(0), torch.from_numpy(k_pages).cuda(), torch.from_numpy(v_pages).cuda(),
                              torch.from_numpy(m8.k_scale).cuda(), torch.from_numpy(m8.v_scale).cuda(),
                              torch.from_numpy(page_table).cuda(), w.Hq, w.scale)
            t = {n: _dev(x) for n, x in rows.items()}
            out = CpRankWorker(lay, fabric.comm(k), ops).prefill(t["q_early"], t["q_late"], t["k_early"], t["v_early"],
                                                                   t["k_late"], t["v_late"])
            torch.cuda.synchronize()
            ops.ctx.poll_status()
            result[k] = tuple(x.clone() for x in out) + (ops.k_pages.cpu().numpy(), ops.v_pages.cpu().numpy(), page_table)
        except Exception as e:
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=body, args=(k,)) for k in range(C)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=600)
    assert not errors, errors
    L = P + R
    for k in range(C):
        lay = RankLayout(R, P, C, k)
        out_e, lse_e, out_l, lse_l, k_pages, v_pages, page_table = result[k]
        for j, o, l in ((lay.early, out_e, lse_e), (lay.late, out_l, lse_l)):
            b, e = lay.chunk(j)
            assert o.shape[0] == e - b
            if e > b:
                compare8(_f64(o), _f64(l), ro[b:e], rl[:, b:e], ra[b:e], "fp8 rank %d chunk %d" % (k, j))
        for got, ref in ((k_pages, m8.k8_pages), (v_pages, m8.v8_pages)):
            assert np.array_equal(o8.e4m3_decode(orc.kv_gather(got, page_table, 0, L)),
                                  o8.e4m3_decode(orc.kv_gather(ref, m8.page_table, 0, L)))


@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("R,P,C", [(2048, 1024, 4), (509, 192, 4), (1533, 0, 3)])
def test_ranks_on_one_gpu_landing_mode(R, P, C, fp8):
    # landing mode: the gathers write into pages of the rank's own pool, a page table reads them in token order, no
    # append runs (the method is taken away); results against the oracle, and the pool read through the landing table
    # holds the whole request bit for bit.  The step is run twice on the same worker (layer after layer).
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from cp_rank_util import ThreadFabric, rank_inputs, rank_inputs8
    from oracle import fp8 as o8
    from paper_2609_04774_b200 import binding
    from paper_2609_04774_b200.cp_rank import CpRankWorker, LibraryOps, LibraryOps8, RankLayout, landing_pages
    from tests.test_gpu_fp8 import compare8
    w = wl.Workload("cp_rank_land_gpu", 68, 8, 2, [wl.Request(R, P, C)])
    mat = wl.materialize(w)
    L = P + R
    if fp8:
        m8 = wl.materialize_fp8(w)
        ro, rl, ra = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv, w.scale,
                                      np.arange(R))
        ref_k, ref_v = orc.kv_gather(m8.k8_pages, m8.page_table, 0, L), orc.kv_gather(m8.v8_pages, m8.page_table, 0, L)
    else:
        ro, rl = orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, P, w.Hkv, w.scale)
        ref_k, ref_v = orc.kv_gather(mat.k_pages, mat.page_table, 0, L), orc.kv_gather(mat.v_pages, mat.page_table, 0, L)
    fabric = ThreadFabric(C)
    result, errors = {}, []

    def body(k):
        try:
            torch.cuda.set_device(0)
            lay = RankLayout(R, P, C, k)
            assert lay.cl % lay.page == 0
            k_pages, v_pages, page_table, rows = rank_inputs8(m8, mat, lay, 68) if fp8 else rank_inputs(mat, lay, 68)
            a0 = k_pages.shape[0]
            extra = np.zeros((landing_pages(lay),) + k_pages.shape[1:], dtype=k_pages.dtype)
            k_pages, v_pages = np.concatenate([k_pages, extra]), np.concatenate([v_pages, extra])
            pt = torch.from_numpy(page_table).cuda()
            if fp8:
                ops = LibraryOps8(binding.Context(0), torch.from_numpy(k_pages).cuda(), torch.from_numpy(v_pages).cuda(),
                                  torch.from_numpy(m8.k_scale).cuda(), torch.from_numpy(m8.v_scale).cuda(), pt, w.Hq, w.scale,
                                  arena_page0=a0)
            else:
                ops = LibraryOps(binding.Context(0), _dev(k_pages), _dev(v_pages), pt, w.Hq, w.scale, arena_page0=a0)
            assert ops.landing(lay) is not None
            ops.kv_append_segments = None
            t = {n: _dev(x) for n, x in rows.items()}
            worker = CpRankWorker(lay, fabric.comm(k), ops)
            for _ in range(2):
                out = worker.prefill(t["q_early"], t["q_late"], t["k_early"], t["v_early"], t["k_late"], t["v_late"])
            torch.cuda.synchronize()
            ops.ctx.poll_status()
            pool = lambda p: p.cpu().numpy() if fp8 else p.view(torch.int16).cpu().numpy().view(np.uint16)
            result[k] = tuple(x.clone() for x in out) + (pool(ops.k_pages), pool(ops.v_pages), ops.landing(lay)[2].cpu().numpy())
        except Exception as e:
            errors.append(e)
            fabric.barrier.abort()

    threads = [threading.Thread(target=body, args=(k,)) for k in range(C)]
    for t in threads:
        t.start()
    for t in threads:
        t.join(timeout=600)
    assert not errors, errors
    for k in range(C):
        lay = RankLayout(R, P, C, k)
        out_e, lse_e, out_l, lse_l, k_pages, v_pages, table = result[k]
        for j, o, l in ((lay.early, out_e, lse_e), (lay.late, out_l, lse_l)):
            b, e = lay.chunk(j)
            assert o.shape[0] == e - b and e > b
            if fp8:
                compare8(_f64(o), _f64(l), ro[b:e], rl[:, b:e], ra[b:e], "landing fp8 rank %d chunk %d" % (k, j))
            else:
                _compare(o, l, ro[b:e], rl[:, b:e], "landing rank %d chunk %d" % (k, j))
        got_k, got_v = orc.kv_gather(k_pages, table, 0, L), orc.kv_gather(v_pages, table, 0, L)
        if fp8:
            assert np.array_equal(o8.e4m3_decode(got_k), o8.e4m3_decode(ref_k)) and np.array_equal(o8.e4m3_decode(got_v), o8.e4m3_decode(ref_v))
        else:
            assert np.array_equal(got_k, ref_k) and np.array_equal(got_v, ref_v)
