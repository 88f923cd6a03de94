"""CPU oracle for zigzag-CP cache-aware causal prefill attention.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
module; the product path never does, and nothing here shares code with the CUDA library.
Everything is fp64 and written the way the definition reads:

  * ``plan``            the zigzag shard plan (paper Section 2.1: pad to a multiple of 2C, 2C equal
                        contiguous chunks, rank k takes chunks k and 2C-1-k), applied to the
                        uncached suffix (Section 2.2)
  * ``remaining_workload``  W(R,P) = R*P + R(R+1)/2, Eq. (1)
  * ``attn_definition`` F1: the masked L x L score matrix and a textbook row softmax (tiny sizes)
  * ``attn_pairs``      F2: row-streaming evaluation of chosen (row, head) pairs through the page
                        table (compiled C, ``cp_oracle.c``)
  * ``attn_sharded``    F3: every shard of the plan computes only its own rows; rows are put back
                        at their original positions (Section 2.1, last step)
  * ``merge``           N-way log-sum-exp combination of partial results over the same rows
  * ``page_offset`` / ``kv_gather`` / ``kv_append``  page-table indexing

Parity pins for each function live in ``tests/test_oracle_*.py``; the measured prefill-time
table has no counterpart in the paper to compare with: parity unpinned for that table.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``cp_oracle.c`` into ``liboracle.so`` next to it (gcc, OpenMP)."""
    src = os.path.join(_HERE, "cp_oracle.c")
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", _LIB_PATH, src, "-lm"])
    return _LIB_PATH


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB_PATH)
        _lib.oracle_attn_pairs.restype = ctypes.c_int
    return _lib


def host_threads() -> int:
    return os.cpu_count() or 1


# ------------------------------------------------------------------------------------------
# Shard plan (Section 2.1) and remaining workload (Eq. 1)
# ------------------------------------------------------------------------------------------

def remaining_workload(R: int, P: int) -> int:
    """Eq. (1): attention workload left after a prefix hit, W(R,P) = R*P + R(R+1)/2."""
    return R * P + R * (R + 1) // 2


def plan(R: int, P: int, C: int):
    """Zigzag plan of the R uncached tokens over C shards.

    The suffix is padded on the right to a multiple of 2C, i.e. chunk length cl = ceil(R / 2C);
    chunk j is [j*cl, (j+1)*cl) clipped to R (trailing chunks may be short or empty); shard k owns
    chunks k and 2C-1-k.  A query at new-token index r sees absolute keys [0, P+r], so a chunk
    ending at q_end needs keys [0, P+q_end) (reported for empty chunks too).  ``pairs`` counts the visible (query, key) pairs.
    """
    assert R >= 1 and P >= 0 and C >= 1
    cl = -(-R // (2 * C))
    shards = []
    for k in range(C):
        qb, qe, kve, pairs = [], [], [], 0
        for j in (k, 2 * C - 1 - k):
            b, e = min(j * cl, R), min((j + 1) * cl, R)
            qb.append(b)
            qe.append(e)
            kve.append(P + e)
            pairs += sum(P + r + 1 for r in range(b, e))     # row r sees keys 0 .. P+r
        shards.append({"q_begin": qb, "q_end": qe, "kv_end": kve, "pairs": pairs})
    return shards


def shard_rows(shard) -> np.ndarray:
    """New-token indices owned by one shard of ``plan``."""
    return np.concatenate([np.arange(b, e, dtype=np.int64) for b, e in zip(shard["q_begin"], shard["q_end"])])


# ------------------------------------------------------------------------------------------
# Page-table indexing
# ------------------------------------------------------------------------------------------

def page_offset(page_table, t, g, page_size, stride_page, stride_tok, stride_head):
    """Element offset of logical token t, KV head g: page_table[t // ps]*stride_page + (t % ps)*stride_tok + g*stride_head."""
    t = np.asarray(t, dtype=np.int64)
    return np.asarray(page_table, dtype=np.int64)[t // page_size] * stride_page + (t % page_size) * stride_tok \
        + g * stride_head


def kv_gather(pages: np.ndarray, page_table, t_begin: int, t_end: int) -> np.ndarray:
    """Paged [num_pages, ps, Hkv, D] -> contiguous [t_end - t_begin, Hkv, D], one token at a time."""
    ps = pages.shape[1]
    out = np.empty((t_end - t_begin,) + pages.shape[2:], dtype=pages.dtype)
    for t in range(t_begin, t_end):
        out[t - t_begin] = pages[page_table[t // ps], t % ps]
    return out


def kv_append(pages: np.ndarray, page_table, t_begin: int, rows: np.ndarray) -> None:
    """Contiguous rows [n, Hkv, D] -> logical tokens t_begin.. of a paged cache (in place)."""
    ps = pages.shape[1]
    for n in range(rows.shape[0]):
        t = t_begin + n
        pages[page_table[t // ps], t % ps] = rows[n]


# ------------------------------------------------------------------------------------------
# Attention
# ------------------------------------------------------------------------------------------

def _bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32) \
        .astype(np.float64)


def attn_definition(q_bits, k_bits, v_bits, P: int, scale: float):
    """F1.  q [R,Hq,D], k/v [L,Hkv,D] contiguous bf16 bits, L = P+R.

    Builds, per head, the full L x L matrix QK^T * scale + M with M_ij = 0 for j <= i and -inf
    otherwise (queries of the cached positions are zero rows that are discarded), applies a
    row softmax and multiplies by V; returns rows [P, L): O [R,Hq,D] and LSE [Hq,R] in fp64.
    """
    q, k, v = _bf16_to_f64(q_bits), _bf16_to_f64(k_bits), _bf16_to_f64(v_bits)
    R, Hq, D = q.shape
    L, Hkv, _ = k.shape
    assert L == P + R
    G = Hq // Hkv
    O = np.zeros((R, Hq, D))
    LSE = np.zeros((Hq, R))
    i = np.arange(L)[:, None]
    j = np.arange(L)[None, :]
    M = np.where(j <= i, 0.0, -np.inf)
    for h in range(Hq):
        g = h // G
        Qfull = np.zeros((L, D))
        Qfull[P:] = q[:, h]
        S = Qfull @ k[:, g].T * scale + M
        m = S.max(axis=1, keepdims=True)
        E = np.exp(S - m)
        l = E.sum(axis=1, keepdims=True)
        A = E / l
        O[:, h] = (A @ v[:, g])[P:]
        LSE[h] = (m + np.log(l))[P:, 0]
    return O, LSE


def attn_pairs(q_bits, k_pages, v_pages, page_table, P: int, Hkv: int, scale: float, rows, heads,
               key_ranges=None, n_threads: int | None = None):
    """F2.  Evaluate the given (row, head) pairs of one request through its page table.

    q_bits [R,Hq,D]; k_pages/v_pages [num_pages, page_size, Hkv, D] (any strides, dim stride 1);
    returns O [n, D] and LSE [n] in fp64.  ``key_ranges`` optionally restricts the attended keys
    to a union of half-open absolute ranges (for KV-split partials).
    """
    lib = _load()
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    R, Hq, D = q_bits.shape
    assert k_pages.dtype == np.uint16 and v_pages.dtype == np.uint16 and k_pages.strides == v_pages.strides
    assert k_pages.strides[3] == 2
    sp, st, sh = (s // 2 for s in k_pages.strides[:3])
    page_size = k_pages.shape[1]
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    heads = np.ascontiguousarray(heads, dtype=np.int32)
    n = rows.size
    pt = np.ascontiguousarray(page_table, dtype=np.int32)
    assert pt.size >= -(-(P + R) // page_size)
    out = np.empty((n, D), dtype=np.float64)
    lse = np.empty(n, dtype=np.float64)
    if key_ranges is None:
        kr_p, n_kr = None, 0
    else:
        kr = np.ascontiguousarray(key_ranges, dtype=np.int64).reshape(-1, 2)
        kr_p, n_kr = kr.ctypes.data_as(ctypes.c_void_p), kr.shape[0]
    rc = lib.oracle_attn_pairs(
        q_bits.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(R), ctypes.c_int32(Hq), ctypes.c_int32(Hkv),
        ctypes.c_int32(D), ctypes.c_void_p(k_pages.ctypes.data), ctypes.c_void_p(v_pages.ctypes.data),
        ctypes.c_int32(page_size), ctypes.c_int64(sp), ctypes.c_int64(st), ctypes.c_int64(sh),
        pt.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(P), ctypes.c_double(scale),
        rows.ctypes.data_as(ctypes.c_void_p), heads.ctypes.data_as(ctypes.c_void_p), ctypes.c_int64(n),
        kr_p, ctypes.c_int32(n_kr),
        out.ctypes.data_as(ctypes.c_void_p), lse.ctypes.data_as(ctypes.c_void_p),
        ctypes.c_int32(n_threads or host_threads()))
    if rc != 0:
        raise ValueError("oracle_attn_pairs: bad argument")
    return out, lse


def attn_rows(q_bits, k_pages, v_pages, page_table, P, Hkv, scale, rows, key_ranges=None, n_threads=None):
    """F2 for whole rows: all heads of the given new-token rows.  O [len(rows),Hq,D], LSE [Hq,len(rows)]."""
    R, Hq, D = q_bits.shape
    rows = np.asarray(rows, dtype=np.int64)
    rr = np.repeat(rows, Hq)
    hh = np.tile(np.arange(Hq, dtype=np.int32), rows.size)
    o, l = attn_pairs(q_bits, k_pages, v_pages, page_table, P, Hkv, scale, rr, hh, key_ranges, n_threads)
    return o.reshape(rows.size, Hq, D), l.reshape(rows.size, Hq).T.copy()


def attn_full(q_bits, k_pages, v_pages, page_table, P, Hkv, scale, n_threads=None):
    """F2 over every new token of one request: O [R,Hq,D], LSE [Hq,R]."""
    return attn_rows(q_bits, k_pages, v_pages, page_table, P, Hkv, scale, np.arange(q_bits.shape[0]),
                     n_threads=n_threads)


def attn_sharded(q_bits, k_pages, v_pages, page_table, P, Hkv, scale, C, n_threads=None):
    """F3.  Each shard of ``plan(R,P,C)`` evaluates only its own rows against keys [0, kv_end) of the
    chunk the row lies in; the shard outputs are restored to the original order.  Also returns the
    per-shard partials (zeros / -inf on rows a shard does not own), ready for ``merge``."""
    R, Hq, D = q_bits.shape
    O = np.full((R, Hq, D), np.nan)
    LSE = np.full((Hq, R), np.nan)
    partial_o = np.zeros((C, R, Hq, D))
    partial_lse = np.full((C, Hq, R), -np.inf)
    for k, sh in enumerate(plan(R, P, C)):
        for b, e, kve in zip(sh["q_begin"], sh["q_end"], sh["kv_end"]):
            if e <= b:
                continue
            rows = np.arange(b, e)
            o, l = attn_rows(q_bits, k_pages, v_pages, page_table, P, Hkv, scale, rows,
                             key_ranges=[[0, kve]], n_threads=n_threads)
            O[b:e], LSE[:, b:e] = o, l
            partial_o[k, b:e], partial_lse[k][:, b:e] = o, l
    return O, LSE, partial_o, partial_lse


# ------------------------------------------------------------------------------------------
# LSE merge
# ------------------------------------------------------------------------------------------

def merge(partials, lses):
    """Combine N partial results over the same rows.

    partials [N,T,H,D], lses [N,H,T] (natural-log sum-exp of the scaled scores each partial saw).
    m = max_n lse_n; where m = -inf the row has no contribution: O = 0, lse = -inf.  Otherwise
    w_n = exp(lse_n - m), O = sum_n w_n O_n / sum_n w_n, lse = m + ln sum_n w_n.  fp64.
    """
    partials = np.asarray(partials, dtype=np.float64)
    lses = np.asarray(lses, dtype=np.float64)
    N, T, H, D = partials.shape
    assert lses.shape == (N, H, T)
    m = lses.max(axis=0)                                   # [H,T]
    dead = np.isneginf(m)
    m_safe = np.where(dead, 0.0, m)
    w = np.exp(lses - m_safe[None])                        # exp(-inf) = 0 for absent partials
    w = np.where(dead[None], 0.0, w)
    wsum = w.sum(axis=0)                                   # [H,T]
    num = np.zeros((T, H, D))
    for n in range(N):
        wn = w[n].T[:, :, None]                            # [T,H,1]
        num += np.where(wn > 0, wn * partials[n], 0.0)     # a zero weight hides whatever the partial holds
    den = np.where(dead, 1.0, wsum).T[:, :, None]
    out = num / den
    with np.errstate(divide="ignore"):
        lse = np.where(dead, -np.inf, m_safe + np.log(np.where(dead, 1.0, wsum)))
    return out, lse
