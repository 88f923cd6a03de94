"""One rank of a degree-C context-parallel prefill worker, built on the library's single-GPU calls.

Section 2.1 of the paper: rank k of C holds zigzag chunks k and 2C-1-k of the uncached suffix, computes
Q/K/V for them, all-gathers K and V, attends its local queries to every causally visible key and the
outputs go back to their original order.  Section 2.2: on a prefix hit the cached KV is partitioned
across the worker's ranks, so it is gathered as well (the b*P term of Eq. 2).

What runs where.  The exchange is three all-gathers of K and of V (prefix blocks, early chunks, late
chunks) issued back to back on the communicator; the attention over the early chunk needs only the first
two, so it runs while the third is still in flight (early chunk first).  Every gather writes straight into
its part of one pre-allocated arena per tensor (prefix blocks | early chunks | late chunks); two
cp_kv_append_segments launches move the arena's rows into this rank's own paged cache (prefix blocks and early
chunks together, then the late chunks), and attention reads that cache through cp_prefill_attn_chunk.  A rank
step is five library launches (own prefix block read out, two appends, two attention calls) plus the merge of
KV-split units where the schedule cuts any.  Remote data is always copied into local HBM before a kernel reads
it.  The module holds no arithmetic of the method: it moves rows and calls the library.

Landing mode (LibraryOps(..., arena_page0=n)): when the chunks are whole pages (cl a multiple of the page size) and
the caller sets aside a run of pages of the cache pool, the arenas ARE those pages: every gather writes into the
pool, a page table built once per layout maps each logical token to the page its row landed in (prefix block r and
early chunk r at rank r's slot, late chunk 2C-1-r at rank r's slot, i.e. in reverse token order), and the two append
launches disappear: a rank step is the read-out of the own prefix block plus the two attention calls.

A second mode, prefill_pass_q, keeps the K/V sharded (a rank holds its prefix block and the K/V of its own
two chunks) and lets the queries travel: all-gather of Q, cp_prefill_attn_kvrange over each of the rank's key
ranges, a local cp_merge of those partials, an all-to-all that returns every row's partials to the rank that
owns the row, and a final cp_merge over the C partials.  It moves R*Hq*D query bytes plus fp32 partials
instead of (P+R)*Hkv*D*2 key/value bytes, which pays when the cached prefix is much longer than the suffix.

With an FP8 cache (LibraryOps8) the exchange carries the stored E4M3 bytes: a rank first writes its own new K/V
into its cache through the quantising append, reads the bytes back as its contribution, and appends the other ranks'
bytes as they are (all ranks share the per-head scales), so the link carries half of what bf16 rows cost.

Readings (the paper fixes none of these): prefix pages are owned in contiguous blocks of
ceil(n_prefix_pages / C) pages, block r on rank r; the prefix length is a multiple of the page size
(block-granular reuse, Section 7.1); chunks are padded to cl = ceil(R / 2C) rows for the collective.
"""
from __future__ import annotations

from dataclasses import dataclass
from functools import cached_property


@dataclass(frozen=True)
class RankLayout:
    """Integer layout of one rank's share of a request (R new tokens behind P cached ones)."""
    R: int
    P: int
    C: int
    rank: int
    page: int = 64

    def __post_init__(self):
        if self.R < 1 or self.P < 0 or self.C < 1 or not 0 <= self.rank < self.C:
            raise ValueError("bad layout R=%d P=%d C=%d rank=%d" % (self.R, self.P, self.C, self.rank))
        if self.P % self.page:
            raise ValueError("prefix length %d is not a multiple of the page size %d" % (self.P, self.page))

    @cached_property
    def _plan(self):
        """The library's shard plan of the request (cp_plan): the one place the chunk arithmetic lives."""
        from . import binding
        return binding.cp_plan(self.R, self.P, self.C)

    @property
    def cl(self) -> int:
        """Rows of a full chunk (chunk 0 is never short): what every chunk is padded to for the collectives."""
        s0 = self._plan[0]
        return s0["q_end"][0] - s0["q_begin"][0]

    def chunk(self, j: int):
        """Rows [begin, end) of zigzag chunk j: shard min(j, 2C-1-j) of the plan holds it as its early or late chunk."""
        s, half = (self._plan[j], 0) if j < self.C else (self._plan[2 * self.C - 1 - j], 1)
        return s["q_begin"][half], s["q_end"][half]

    @property
    def early(self) -> int:
        return self.rank

    @property
    def late(self) -> int:
        return 2 * self.C - 1 - self.rank

    def late_chunk_of(self, r: int) -> int:
        return 2 * self.C - 1 - r

    @property
    def prefix_pages(self) -> int:
        return self.P // self.page

    @property
    def block_pages(self) -> int:
        """Prefix pages per rank (the last blocks may be short or empty)."""
        return -(-self.prefix_pages // self.C) if self.prefix_pages else 0

    def prefix_block(self, r: int):
        """Token range [begin, end) of the prefix block owned by rank r."""
        b = min(r * self.block_pages, self.prefix_pages) * self.page
        e = min((r + 1) * self.block_pages, self.prefix_pages) * self.page
        return b, e


def landing_rows(lay: RankLayout):
    """Arena row of every logical token of the request when the gathers land in the layout
    prefix blocks (C x n_blk rows) | early chunks (C x cl) | late chunks (C x cl), rank r's contribution at slot r:
    a list of (token_begin, n_tokens, arena_row) runs covering [0, P + R), in token order."""
    C, cl, n_blk = lay.C, lay.cl, lay.block_pages * lay.page
    runs = []
    if lay.P:
        runs.append((0, lay.P, 0))                    # block r starts at token r * n_blk and at arena row r * n_blk
    for j in range(2 * C):
        b, e = lay.chunk(j)
        if e > b:
            slot = j if j < C else 2 * C - 1 - j      # early chunk j came from rank j, late chunk j from rank 2C-1-j
            runs.append((lay.P + b, e - b, C * n_blk + (0 if j < C else C * cl) + slot * cl))
    return runs


def landing_table(lay: RankLayout, arena_page0: int):
    """Page ids (one per page of [0, P + R)) that read the landed rows back in token order, or None when a chunk
    does not start on a page boundary (cl not a multiple of the page size)."""
    if lay.cl % lay.page:
        return None
    table = []
    for t0, n, a0 in landing_rows(lay):
        assert t0 % lay.page == 0 and a0 % lay.page == 0 and len(table) == t0 // lay.page
        table += [arena_page0 + a0 // lay.page + i for i in range(-(-n // lay.page))]
    return table


def landing_pages(lay: RankLayout) -> int:
    """Pages the landing arena takes in the pool."""
    return lay.C * lay.block_pages + 2 * lay.C * (-(-lay.cl // lay.page))


class TorchComm:
    """All-gather of equally sized row blocks over a torch.distributed group (NCCL on GPUs, gloo on CPU)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist = dist
        self.group = group
        self.size = dist.get_world_size(group)
        self.rank = dist.get_rank(group)

    def all_gather(self, block):
        """block [n, ...] -> (out [size, n, ...], handle); handle.wait() orders the caller's stream behind it."""
        import torch
        out = torch.empty((self.size,) + tuple(block.shape), dtype=block.dtype, device=block.device)
        # rows travel as bytes: every backend moves uint8, whatever the row type is
        src = block.contiguous().view(torch.uint8).reshape(-1)
        dst = out.view(torch.uint8).reshape(self.size, -1)
        work = self.dist.all_gather(list(dst.unbind(0)), src, group=self.group, async_op=True)
        return out, work


    def all_gather_into(self, out, block):
        """Gathers block [n, ...] of every rank into out [size * n, ...] (a contiguous view, e.g. a slice of an
        arena); returns a handle."""
        import torch
        src = block.contiguous().view(torch.uint8).reshape(-1)
        dst = out.view(torch.uint8).reshape(-1)
        return self.dist.all_gather_into_tensor(dst, src, group=self.group, async_op=True)

    def all_to_all(self, blocks):
        """blocks [size, n, ...]: block d goes to rank d.  -> (out [size, n, ...] with out[s] = the block rank s
        sent here, handle)."""
        import torch
        if self.dist.get_backend(self.group) == "gloo":
            # gloo has no all-to-all: gather everything and keep this rank's blocks (CPU test path only)
            gathered, work = self.all_gather(blocks)
            work.wait()

            class _Done:
                def wait(self):
                    return True
            return gathered[:, self.rank].contiguous(), _Done()
        out = torch.empty_like(blocks)
        src = blocks.contiguous().view(torch.uint8).reshape(self.size, -1)
        dst = out.view(torch.uint8).reshape(self.size, -1)
        work = self.dist.all_to_all(list(dst.unbind(0)), list(src.unbind(0)), group=self.group, async_op=True)
        return out, work


class LibraryOps:
    """The three device steps of a rank, on this rank's paged cache, through the C-ABI library."""

    def __init__(self, ctx, k_pages, v_pages, page_table, Hq, scale, arena_page0=None):
        import torch
        from . import binding
        self.b, self.ctx, self.torch = binding, ctx, torch
        self.arena_page0, self._landing = arena_page0, {}
        self.cache = binding.make_cache(k_pages, v_pages)
        self.k_pages, self.v_pages, self.page_table = k_pages, v_pages, page_table
        self.Hq, self.scale = Hq, scale
        self.Hkv, self.D = k_pages.shape[2], k_pages.shape[3]
        self.device = k_pages.device
        self._ws = None
        self._buffers = {}

    def empty_rows(self, n, heads):
        return self.torch.zeros((n, heads, self.D), dtype=self.torch.bfloat16, device=self.device)

    def buffer(self, name, shape, dtype=None):
        """A device buffer that lives as long as this object (allocated and zeroed on first use): the staging
        arenas, send buffers and outputs of a rank step are reused from layer to layer.  Default type: that of the
        rows on the wire."""
        dtype = dtype or self.wire_dtype
        key = (name, tuple(shape), dtype)
        if key not in self._buffers:
            self._buffers[key] = self.torch.zeros(tuple(shape), dtype=dtype, device=self.device)
        return self._buffers[key]

    @property
    def wire_dtype(self):
        """Element type of K/V rows as they travel between ranks and sit in the arenas."""
        return self.torch.bfloat16

    def landing(self, lay: RankLayout):
        """Landing mode for this layout: (k_rows, v_rows, page_table) -- the arena as row views
        [C * (n_blk + 2 cl), Hkv, D] of the pools' pages from arena_page0 on, and the device page table that reads
        the landed rows in token order -- or None (no pages set aside, chunks not whole pages, pool not contiguous
        or too small)."""
        key = (lay.R, lay.P, lay.C, lay.rank, lay.page)
        if key not in self._landing:
            land = None
            table = landing_table(lay, self.arena_page0) if self.arena_page0 is not None else None
            n_pg = landing_pages(lay)
            if (table is not None and lay.page == self.k_pages.shape[1] and self.k_pages.is_contiguous()
                    and self.v_pages.is_contiguous() and self.arena_page0 + n_pg <= self.k_pages.shape[0]):
                rows = n_pg * lay.page
                kr = self.k_pages[self.arena_page0:self.arena_page0 + n_pg].view(rows, self.Hkv, self.D)
                vr = self.v_pages[self.arena_page0:self.arena_page0 + n_pg].view(rows, self.Hkv, self.D)
                land = (kr, vr, self.torch.tensor(table, dtype=self.torch.int32, device=self.device))
            self._landing[key] = land
        return self._landing[key]

    def to_wire(self, name, t_begin, k_rows, v_rows, page_table=None):
        """This rank's new K/V rows (bf16, logical tokens t_begin..) in the form they travel in: as they are."""
        return k_rows, v_rows

    def kv_append_segments(self, segments, k_rows, v_rows):
        segments = [s for s in segments if s[1] > 0]
        if segments:
            self.b.cp_kv_append_segments(self.ctx, self.cache, self.page_table, segments, k_rows, v_rows)

    def kv_gather(self, t_begin, n, k_rows, v_rows):
        if n > 0:
            self.b.cp_kv_gather(self.ctx, self.cache, self.page_table, t_begin, n, k_rows, v_rows)

    def kv_append(self, t_begin, n, k_rows, v_rows):
        if n > 0:
            self.b.cp_kv_append(self.ctx, self.cache, self.page_table, t_begin, n, k_rows, v_rows)

    def attn_chunk(self, lay: RankLayout, chunk, q_chunk, page_table=None):
        n = q_chunk.shape[0]
        out = self.buffer("out_%d" % chunk, (n, self.Hq, self.D), self.torch.bfloat16)
        lse = self.buffer("lse_%d" % chunk, (self.Hq, n), self.torch.float32)
        if n == 0:
            return out, lse
        if self._ws is None:
            nbytes = self.b.cp_workspace_bytes([lay.R], [lay.C], self.Hq)
            self._ws = self.torch.empty(nbytes, dtype=self.torch.uint8, device=self.device)
        self.b.cp_prefill_attn_chunk(self.ctx, q_chunk, self.cache, self.page_table if page_table is None else page_table,
                                     lay.P, lay.R, lay.C, chunk, self.Hq, self.scale, out, lse, self._ws)
        return out, lse


class LibraryOps8(LibraryOps):
    """The device steps of a rank on an FP8 K/V cache (E4M3 pages, one fp32 scale per KV head shared by all ranks)."""

    def __init__(self, ctx, k8_pages, v8_pages, k_scale, v_scale, page_table, Hq, scale, arena_page0=None):
        import torch
        from . import binding
        self.b, self.ctx, self.torch = binding, ctx, torch
        self.arena_page0, self._landing = arena_page0, {}
        self.cache = binding.make_cache_fp8(k8_pages, v8_pages, k_scale, v_scale)
        self.k_pages, self.v_pages, self.page_table = k8_pages, v8_pages, page_table
        self.k_scale, self.v_scale = k_scale, v_scale
        self.Hq, self.scale = Hq, scale
        self.Hkv, self.D = k8_pages.shape[2], k8_pages.shape[3]
        self.device = k8_pages.device
        self._ws = None
        self._buffers = {}

    @property
    def wire_dtype(self):
        return self.torch.uint8

    def empty_rows(self, n, heads):
        return self.torch.zeros((n, heads, self.D), dtype=self.torch.uint8, device=self.device)

    def to_wire(self, name, t_begin, k_rows, v_rows, page_table=None):
        """Quantise the rank's own new rows into its cache (they belong there anyway) and read the stored bytes
        back: what the other ranks receive is exactly what this rank attends to."""
        n = k_rows.shape[0]
        pt = self.page_table if page_table is None else page_table
        kb, vb = self.buffer("wire_k_" + name, (n, self.Hkv, self.D)), self.buffer("wire_v_" + name, (n, self.Hkv, self.D))
        if n > 0:
            self.b.cp_kv_append_fp8(self.ctx, self.cache, pt, t_begin, n, k_rows, v_rows)
            self.b.cp_kv_gather_fp8(self.ctx, self.cache, pt, t_begin, n, kb, vb)
        return kb, vb

    def kv_gather(self, t_begin, n, k_rows, v_rows):
        if n > 0:
            self.b.cp_kv_gather_fp8(self.ctx, self.cache, self.page_table, t_begin, n, k_rows, v_rows)

    def kv_append_segments(self, segments, k_rows, v_rows):
        segments = [s for s in segments if s[1] > 0]
        if segments:
            self.b.cp_kv_append_segments_fp8(self.ctx, self.cache, self.page_table, segments, k_rows, v_rows)

    def attn_chunk(self, lay: RankLayout, chunk, q_chunk, page_table=None):
        n = q_chunk.shape[0]
        out = self.buffer("out_%d" % chunk, (n, self.Hq, self.D), self.torch.bfloat16)
        lse = self.buffer("lse_%d" % chunk, (self.Hq, n), self.torch.float32)
        if n == 0:
            return out, lse
        if self._ws is None:
            nbytes = self.b.cp_workspace_bytes_fp8([lay.R], [lay.C], self.Hq)
            self._ws = self.torch.empty(nbytes, dtype=self.torch.uint8, device=self.device)
        self.b.cp_prefill_attn_fp8_chunk(self.ctx, q_chunk, self.cache, self.page_table if page_table is None else page_table,
                                         lay.P, lay.R, lay.C, chunk, self.Hq, self.scale, out, lse, self._ws)
        return out, lse


def _library_extras():
    """Methods of LibraryOps used by the pass-Q mode (kept together; bound below)."""

    def attn_kvrange(self, lay, q_full, lo, hi):
        torch = self.torch
        R = lay.R
        part = torch.empty((R, self.Hq, self.D), dtype=torch.float32, device=self.device)
        lse = torch.empty((self.Hq, R), dtype=torch.float32, device=self.device)
        if self._ws is None:
            nbytes = self.b.cp_workspace_bytes([lay.R], [lay.C], self.Hq)
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.b.cp_prefill_attn_kvrange(self.ctx, q_full, self.cache, self.page_table, lay.P, R, lo, hi, self.Hq,
                                       self.scale, part, lse, self._ws)
        return part, lse

    def attn_kvranges(self, lay, q_full, ranges):
        """All R queries against each of the key ranges: partials written straight into one stacked, persistent
        buffer (parts [n, R, Hq, D] fp32, lses [n, Hq, R]), ready for cp_merge."""
        torch = self.torch
        R, n = lay.R, len(ranges)
        parts = self.buffer("kvr_parts", (n, R, self.Hq, self.D), torch.float32)
        lses = self.buffer("kvr_lses", (n, self.Hq, R), torch.float32)
        if self._ws is None:
            nbytes = self.b.cp_workspace_bytes([lay.R], [lay.C], self.Hq)
            self._ws = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        for i, (lo, hi) in enumerate(ranges):
            self.b.cp_prefill_attn_kvrange(self.ctx, q_full, self.cache, self.page_table, lay.P, R, lo, hi, self.Hq,
                                           self.scale, parts[i], lses[i], self._ws)
        return parts, lses

    def merge(self, parts, lses, final):
        """parts [N, T, Hq, D] fp32, lses [N, Hq, T] -> (out [T, Hq, D] bf16 if final else fp32, lse [Hq, T])."""
        torch = self.torch
        T = parts.shape[1]
        out = torch.empty((T, self.Hq, self.D), dtype=torch.bfloat16 if final else torch.float32, device=self.device)
        lse = torch.empty((self.Hq, T), dtype=torch.float32, device=self.device)
        if T:
            self.b.cp_merge(self.ctx, parts.contiguous(), lses.contiguous(), out, lse)
        return out, lse

    def empty_f32(self, shape):
        return self.torch.zeros(tuple(shape), dtype=self.torch.float32, device=self.device)

    LibraryOps.attn_kvrange, LibraryOps.merge, LibraryOps.empty_f32 = attn_kvrange, merge, empty_f32
    LibraryOps.attn_kvranges = attn_kvranges


_library_extras()


def _padded(ops, rows, n, name=None):
    """rows [m, H, D] -> [n, H, D] with zero rows behind (collectives need equal sizes).  A full chunk is sent as
    it is; a short one goes through a send buffer (a persistent one when the ops object keeps buffers)."""
    if rows.shape[0] == n:
        return rows
    buf = ops.buffer(name, (n,) + tuple(rows.shape[1:])) if name and hasattr(ops, "buffer") else ops.empty_rows(n, rows.shape[1])
    buf[:rows.shape[0]] = rows
    return buf


class CpRankWorker:
    """Runs one layer's attention for this rank's two chunks.

    comm: an object with .size, .rank and all_gather(block) -> (out, handle), e.g. TorchComm.
    ops: the device steps; LibraryOps is the only implementation in the package.
    """

    def __init__(self, layout: RankLayout, comm, ops):
        if comm.size != layout.C or comm.rank != layout.rank:
            raise ValueError("communicator (%d of %d) does not match the layout (%d of %d)" %
                             (comm.rank, comm.size, layout.rank, layout.C))
        self.lay, self.comm, self.ops = layout, comm, ops

    def prefill(self, q_early, q_late, k_early, v_early, k_late, v_late):
        """q_*: this rank's query rows [n, Hq, D]; k_*/v_*: its new K/V rows [n, Hkv, D] (n = chunk rows).
        The rank's prefix block must already be in its cache.  Returns (out_early, lse_early, out_late, lse_late)."""
        lay, ops, comm = self.lay, self.ops, self.comm
        (eb, ee), (lb, le) = lay.chunk(lay.early), lay.chunk(lay.late)
        assert q_early.shape[0] == ee - eb == k_early.shape[0] and q_late.shape[0] == le - lb == k_late.shape[0]

        C, cl = lay.C, lay.cl
        n_blk = lay.block_pages * lay.page
        # one arena per tensor: gathered prefix blocks | gathered early chunks | gathered late chunks (rows).
        # Landing mode: the arena is a run of pages of the cache pool itself and `table` reads it in token order.
        off_e, off_l = C * n_blk, C * (n_blk + cl)
        land = ops.landing(lay) if hasattr(ops, "landing") else None
        if land is not None:
            ak, av, table = land
            kw = {"page_table": table}
        else:
            ak = ops.buffer("arena_k", (C * (n_blk + 2 * cl), ops.Hkv, ops.D))
            av = ops.buffer("arena_v", (C * (n_blk + 2 * cl), ops.Hkv, ops.D))
            kw = {}

        # 1. contributions: own prefix block read out of the cache, own chunks (padded to cl rows when short);
        #    every gather lands in its part of the arena
        pb, pe = lay.prefix_block(lay.rank)
        hp = None
        if n_blk:
            sk, sv = ops.buffer("send_prefix_k", (n_blk, ops.Hkv, ops.D)), ops.buffer("send_prefix_v", (n_blk, ops.Hkv, ops.D))
            ops.kv_gather(pb, pe - pb, sk, sv)
            hp = (comm.all_gather_into(ak[:off_e], sk), comm.all_gather_into(av[:off_e], sv))
        if hasattr(ops, "to_wire"):       # an FP8 cache sends stored bytes; a bf16 cache the rows as they are
            k_early, v_early = ops.to_wire("early", lay.P + eb, k_early, v_early, **kw)
            k_late, v_late = ops.to_wire("late", lay.P + lb, k_late, v_late, **kw)
        he = (comm.all_gather_into(ak[off_e:off_l], _padded(ops, k_early, cl, "send_early_k")),
              comm.all_gather_into(av[off_e:off_l], _padded(ops, v_early, cl, "send_early_v")))
        hl = (comm.all_gather_into(ak[off_l:], _padded(ops, k_late, cl, "send_late_k")),
              comm.all_gather_into(av[off_l:], _padded(ops, v_late, cl, "send_late_v")))

        # 2. prefix blocks and early chunks into the own cache, one launch: block r and chunk r came from rank r
        segs = []
        if hp is not None:
            hp[0].wait()
            hp[1].wait()
            for r in range(C):
                b, e = lay.prefix_block(r)
                segs.append((b, e - b, r * n_blk))
        he[0].wait()
        he[1].wait()
        for r in range(C):
            b, e = lay.chunk(r)
            segs.append((lay.P + b, e - b, off_e + r * cl))
        if land is None:
            ops.kv_append_segments(segs, ak, av)

        # 3. early chunk: its keys are all here; the late all-gather is still in flight
        out_e, lse_e = ops.attn_chunk(lay, lay.early, q_early, **kw)

        # 4. late chunks (rank r sent chunk 2C-1-r), one launch, then the late chunk's attention
        hl[0].wait()
        hl[1].wait()
        segs = []
        for r in range(C):
            b, e = lay.chunk(lay.late_chunk_of(r))
            segs.append((lay.P + b, e - b, off_l + r * cl))
        if land is None:
            ops.kv_append_segments(segs, ak, av)
        out_l, lse_l = ops.attn_chunk(lay, lay.late, q_late, **kw)
        return out_e, lse_e, out_l, lse_l

    def _return_index(self, like):
        """The send-buffer row index as a tensor on the device of `like` (built once per worker)."""
        import torch
        if getattr(self, "_ret_idx", None) is None:
            idx, pad = _return_index_of(self.lay)
            self._ret_idx = torch.tensor(idx, dtype=torch.long, device=like.device)
            self._ret_pad = torch.tensor(pad, dtype=torch.bool, device=like.device) if any(pad) else None
        return self._ret_idx, self._ret_pad

    def prefill_pass_q(self, q_early, q_late, k_early, v_early, k_late, v_late):
        """Same inputs and outputs as prefill(), but the K/V never leaves its rank: the rank's cache must hold
        its prefix block; its own chunks' K/V are appended here, nothing else is ever read from the cache."""
        lay, ops, comm = self.lay, self.ops, self.comm
        (eb, ee), (lb, le) = lay.chunk(lay.early), lay.chunk(lay.late)
        assert q_early.shape[0] == ee - eb == k_early.shape[0] and q_late.shape[0] == le - lb == k_late.shape[0]
        Hq = q_early.shape[1]

        # 1. queries travel: both chunks of every rank, padded to cl rows
        (ge, he), (gl, hl) = comm.all_gather(_padded(ops, q_early, lay.cl)), comm.all_gather(_padded(ops, q_late, lay.cl))
        # 2. meanwhile the own new K/V goes into the own cache
        ops.kv_append(lay.P + eb, ee - eb, k_early, v_early)
        ops.kv_append(lay.P + lb, le - lb, k_late, v_late)
        he.wait()
        hl.wait()
        # rank order is token order for the early chunks; the late chunks arrive in reverse (rank r sent chunk 2C-1-r)
        q_full = ops.empty_rows(lay.R, Hq)
        n_first = min(lay.R, lay.C * lay.cl)
        q_full[:n_first] = ge.reshape((-1,) + tuple(ge.shape[2:]))[:n_first]
        if lay.R > n_first:
            late = gl.flip(0).reshape((-1,) + tuple(gl.shape[2:]))      # chunks C, C+1, ... in order, cl rows each
            q_full[n_first:] = late[:lay.R - n_first]

        # 3. partial attention of all queries over each of the rank's key ranges, merged locally
        pb, pe = lay.prefix_block(lay.rank)
        ranges = [(lo, hi) for lo, hi in ((pb, pe), (lay.P + eb, lay.P + ee), (lay.P + lb, lay.P + le)) if hi > lo]
        if ranges and hasattr(ops, "attn_kvranges"):
            po, pl = ops.attn_kvranges(lay, q_full, ranges)             # stacked by the ops, no copies
            mine_o, mine_l = (po[0], pl[0]) if len(ranges) == 1 else ops.merge(po, pl, final=False)
        elif ranges:
            parts = [ops.attn_kvrange(lay, q_full, lo, hi) for lo, hi in ranges]
            mine_o, mine_l = parts[0] if len(parts) == 1 else \
                ops.merge(_stack([p for p, _ in parts]), _stack([l for _, l in parts]), final=False)
        else:                                   # the rank holds no key at all (more ranks than blocks and chunks)
            mine_o = ops.empty_f32((lay.R, Hq, ops.D))
            mine_l = ops.empty_f32((Hq, lay.R)) - float("inf")

        # 4. every row's partial goes back to the rank that owns the row: block d = chunk d, then chunk 2C-1-d
        #    (one gather by row index per tensor; rows of the padding take row 0's values and lse = -inf)
        idx, pad = self._return_index(mine_l)
        send_o = mine_o.index_select(0, idx).reshape((lay.C, 2 * lay.cl, Hq, ops.D))
        send_l = mine_l.index_select(1, idx)
        if pad is not None:
            send_l = send_l.masked_fill(pad, float("-inf"))
        send_l = send_l.reshape((Hq, lay.C, 2 * lay.cl)).transpose(0, 1).contiguous()
        (ro, ho), (rl, hl2) = comm.all_to_all(send_o), comm.all_to_all(send_l)
        ho.wait()
        hl2.wait()

        # 5. the C partials of the own rows (each over a disjoint part of the keys) merge into the result
        out, lse = ops.merge(ro, rl, final=True)
        n_e, n_l = ee - eb, le - lb
        return out[:n_e], lse[:, :n_e], out[lay.cl:lay.cl + n_l], lse[:, lay.cl:lay.cl + n_l]


def _return_index_of(lay):
    """Row index of the all-to-all's send buffer: block d holds chunk d, then chunk 2C-1-d, cl rows each; rows of the
    padding point at row 0 and are flagged."""
    idx, pad = [], []
    for d in range(lay.C):
        for j in (d, lay.late_chunk_of(d)):
            b, e = lay.chunk(j)
            idx += list(range(b, e)) + [0] * (lay.cl - (e - b))
            pad += [False] * (e - b) + [True] * (lay.cl - (e - b))
    return idx, pad


def _stack(tensors):
    """Stack along a new first axis (torch.stack for tensors, the same for the test doubles' arrays)."""
    import torch
    return torch.stack(list(tensors), 0)
