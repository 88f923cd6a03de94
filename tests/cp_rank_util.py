"""Test doubles for the CP rank worker: an in-process communicator for ranks run as threads, and the
device steps restated on the oracle (numpy pools of bf16 bit patterns) for the CPU tests."""
import threading

import numpy as np
import torch

from oracle import reference as orc
from paper_2609_04774_b200 import workloads as wl


class _Done:
    def wait(self):
        return True


class ThreadFabric:
    """Shared state of C in-process ranks: the n-th all_gather of every rank meets the others'."""

    def __init__(self, size):
        self.size = size
        self.barrier = threading.Barrier(size)
        self.slots = {}
        self.lock = threading.Lock()

    def comm(self, rank):
        return ThreadComm(self, rank)


class ThreadComm:
    def __init__(self, fabric, rank):
        self.fabric, self.rank, self.size = fabric, rank, fabric.size
        self.calls = 0

    def all_to_all(self, blocks):
        # every rank's [size, n, ...] blocks meet; rank r takes block r of each
        gathered, done = self.all_gather(blocks)
        return gathered[:, self.rank].contiguous(), done

    def all_gather_into(self, out, block):
        gathered, done = self.all_gather(block)
        out.copy_(gathered.reshape(out.shape))
        return done

    def all_gather(self, block):
        f, n = self.fabric, self.calls
        self.calls += 1
        with f.lock:
            f.slots.setdefault(n, [None] * f.size)[self.rank] = block
        f.barrier.wait(timeout=120)
        out = torch.stack([b.to(block.device) for b in f.slots[n]], 0)
        f.barrier.wait(timeout=120)
        return out, _Done()


class OracleOps:
    """kv_gather / kv_append / attn_chunk of one rank on numpy page pools, through the oracle."""

    def __init__(self, k_pages, v_pages, page_table, Hq, scale, arena_page0=None):
        self.k_pages, self.v_pages, self.page_table = k_pages, v_pages, np.asarray(page_table)
        self.Hq, self.scale = Hq, scale
        self.Hkv, self.D = k_pages.shape[2], k_pages.shape[3]
        self.arena_page0 = arena_page0

    def landing(self, lay):
        """Landing mode on the numpy pools: torch views of the arena pages (shared memory) and the page table."""
        from paper_2609_04774_b200 import cp_rank
        table = cp_rank.landing_table(lay, self.arena_page0) if self.arena_page0 is not None else None
        if table is None:
            return None
        n_pg, a0 = cp_rank.landing_pages(lay), self.arena_page0
        assert a0 + n_pg <= self.k_pages.shape[0]
        dt = np.int16 if self.k_pages.dtype == np.uint16 else self.k_pages.dtype
        kr = torch.from_numpy(self.k_pages.view(dt))[a0:a0 + n_pg].view(n_pg * lay.page, self.Hkv, self.D)
        vr = torch.from_numpy(self.v_pages.view(dt))[a0:a0 + n_pg].view(n_pg * lay.page, self.Hkv, self.D)
        return kr, vr, np.asarray(table)

    def empty_rows(self, n, heads):
        return torch.zeros((n, heads, self.D), dtype=torch.int16)

    def buffer(self, name, shape, dtype=None):
        self._buffers = getattr(self, "_buffers", {})
        key = (name, tuple(shape))
        if key not in self._buffers:
            self._buffers[key] = torch.zeros(tuple(shape), dtype=torch.int16)
        return self._buffers[key]

    def kv_append_segments(self, segments, k_rows, v_rows):
        for t_begin, n, row0 in segments:
            self.kv_append(t_begin, n, k_rows[row0:row0 + n], v_rows[row0:row0 + n])

    @staticmethod
    def _bits(t):
        return t.contiguous().numpy().view(np.uint16)

    def kv_gather(self, t_begin, n, k_rows, v_rows):
        if n > 0:
            k_rows[:n] = torch.from_numpy(orc.kv_gather(self.k_pages, self.page_table, t_begin, t_begin + n).view(np.int16))
            v_rows[:n] = torch.from_numpy(orc.kv_gather(self.v_pages, self.page_table, t_begin, t_begin + n).view(np.int16))

    def kv_append(self, t_begin, n, k_rows, v_rows):
        if n > 0:
            orc.kv_append(self.k_pages, self.page_table, t_begin, self._bits(k_rows)[:n])
            orc.kv_append(self.v_pages, self.page_table, t_begin, self._bits(v_rows)[:n])

    def attn_chunk(self, lay, chunk, q_chunk, page_table=None):
        b, e = lay.chunk(chunk)
        q = np.zeros((lay.R, self.Hq, self.D), dtype=np.uint16)
        q[b:e] = self._bits(q_chunk)
        if e == b:
            return np.zeros((0, self.Hq, self.D)), np.zeros((self.Hq, 0))
        pt = self.page_table if page_table is None else page_table
        return orc.attn_rows(q, self.k_pages, self.v_pages, pt, lay.P, self.Hkv, self.scale, np.arange(b, e))


    # ---- pass-Q mode: partial attention over a key range, LSE merge (fp64 torch tensors) ----
    def attn_kvrange(self, lay, q_full, lo, hi):
        o, l = orc.attn_rows(self._bits(q_full), self.k_pages, self.v_pages, self.page_table, lay.P, self.Hkv, self.scale,
                             np.arange(lay.R), key_ranges=[(lo, hi)])
        dead = ~np.isfinite(l)                                   # [Hq, R]: rows that see no key of the range
        o = np.where(dead.T[:, :, None], 0.0, o)
        return torch.from_numpy(o), torch.from_numpy(np.where(dead, -np.inf, l))

    def merge(self, parts, lses, final):
        if parts.shape[1] == 0:
            return torch.zeros(parts.shape[1:], dtype=torch.float64), torch.zeros(lses.shape[1:], dtype=torch.float64)
        o, l = orc.merge(parts.numpy(), lses.numpy())
        return torch.from_numpy(o), torch.from_numpy(l)

    def empty_f32(self, shape):
        return torch.zeros(tuple(shape), dtype=torch.float64)


class OracleOps8(OracleOps):
    """The same steps on E4M3 byte pools with per-head scales, through the FP8 oracle."""

    def __init__(self, k8_pages, v8_pages, k_scale, v_scale, page_table, Hq, scale, arena_page0=None):
        super().__init__(k8_pages, v8_pages, page_table, Hq, scale, arena_page0)
        self.k_scale, self.v_scale = k_scale, v_scale

    def empty_rows(self, n, heads):
        return torch.zeros((n, heads, self.D), dtype=torch.uint8)

    def buffer(self, name, shape, dtype=None):
        self._buffers = getattr(self, "_buffers", {})
        key = (name, tuple(shape))
        if key not in self._buffers:
            self._buffers[key] = torch.zeros(tuple(shape), dtype=torch.uint8)
        return self._buffers[key]

    @staticmethod
    def _bits(t):
        return t.contiguous().numpy()

    def to_wire(self, name, t_begin, k_rows, v_rows, page_table=None):
        from oracle import fp8 as o8
        pt = self.page_table if page_table is None else page_table
        kc = o8.quantize_kv(k_rows.contiguous().numpy().view(np.uint16), self.k_scale)
        vc = o8.quantize_kv(v_rows.contiguous().numpy().view(np.uint16), self.v_scale)
        if kc.shape[0]:
            orc.kv_append(self.k_pages, pt, t_begin, kc)
            orc.kv_append(self.v_pages, pt, t_begin, vc)
        return torch.from_numpy(kc), torch.from_numpy(vc)

    def kv_gather(self, t_begin, n, k_rows, v_rows):
        if n > 0:
            k_rows[:n] = torch.from_numpy(orc.kv_gather(self.k_pages, self.page_table, t_begin, t_begin + n))
            v_rows[:n] = torch.from_numpy(orc.kv_gather(self.v_pages, self.page_table, t_begin, t_begin + n))

    def attn_chunk(self, lay, chunk, q_chunk, page_table=None):
        from oracle import fp8 as o8
        b, e = lay.chunk(chunk)
        q = np.zeros((lay.R, self.Hq, self.D), dtype=np.uint16)
        q[b:e] = q_chunk.contiguous().numpy().view(np.uint16)
        if e == b:
            return np.zeros((0, self.Hq, self.D)), np.zeros((self.Hq, 0))
        o, l, _ = o8.attn_fp8_rows(q, self.k_pages, self.v_pages, self.k_scale, self.v_scale,
                                   self.page_table if page_table is None else page_table, lay.P, self.Hkv,
                                   self.scale, np.arange(b, e))
        return o, l


def rank_inputs8(m8, mat, lay, seed):
    """FP8 form of rank_inputs: the rank's own byte pool holds only its prefix block (the stored bytes of the seeded
    request); its q / k / v rows are the bf16 rows the bytes were made from."""
    pt_ref = m8.page_table
    n_pages = len(pt_ref)
    page_table = wl.permutation(seed + 100 * (lay.rank + 1), wl.TID_PERM, n_pages + 2)[:n_pages].astype(np.int32)
    k_pages = np.zeros((n_pages + 2,) + m8.k8_pages.shape[1:], dtype=np.uint8)
    v_pages = np.zeros_like(k_pages)
    pb, pe = lay.prefix_block(lay.rank)
    if pe > pb:
        orc.kv_append(k_pages, page_table, pb, orc.kv_gather(m8.k8_pages, pt_ref, pb, pe))
        orc.kv_append(v_pages, page_table, pb, orc.kv_gather(m8.v8_pages, pt_ref, pb, pe))
    rows = {}
    for name, j in (("early", lay.early), ("late", lay.late)):
        b, e = lay.chunk(j)
        rows["q_" + name] = mat.q[b:e]
        rows["k_" + name] = orc.kv_gather(mat.k_pages, mat.page_table, lay.P + b, lay.P + e)
        rows["v_" + name] = orc.kv_gather(mat.v_pages, mat.page_table, lay.P + b, lay.P + e)
    return k_pages, v_pages, page_table, rows


def rank_inputs(mat, lay, seed):
    """What rank `lay.rank` starts with, cut from the seeded full request: an empty page pool of its own
    (its own page permutation) holding only the rank's prefix block, and the rank's q/k/v rows."""
    w = mat.wl
    pt_ref = mat.page_table
    n_pages = len(pt_ref)
    page_table = wl.permutation(seed + 100 * (lay.rank + 1), wl.TID_PERM, n_pages + 2)[:n_pages].astype(np.int32)
    k_pages = np.zeros((n_pages + 2,) + mat.k_pages.shape[1:], dtype=np.uint16)
    v_pages = np.zeros_like(k_pages)
    pb, pe = lay.prefix_block(lay.rank)
    if pe > pb:
        orc.kv_append(k_pages, page_table, pb, orc.kv_gather(mat.k_pages, pt_ref, pb, pe))
        orc.kv_append(v_pages, page_table, pb, orc.kv_gather(mat.v_pages, pt_ref, pb, pe))
    rows = {}
    for name, j in (("early", lay.early), ("late", lay.late)):
        b, e = lay.chunk(j)
        rows["q_" + name] = mat.q[b:e]
        rows["k_" + name] = orc.kv_gather(mat.k_pages, pt_ref, lay.P + b, lay.P + e)
        rows["v_" + name] = orc.kv_gather(mat.v_pages, pt_ref, lay.P + b, lay.P + e)
    return k_pages, v_pages, page_table, rows
