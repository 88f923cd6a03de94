"""Seeded synthetic inputs for cache-aware causal prefill attention under zigzag CP.

This module only manufactures bytes: tensors of i.i.d. N(0,1) values rounded to
bf16, page tables, request-length draws.  It contains none of the method's
arithmetic (no planner, no attention, no merge) so that the CPU oracle and the
CUDA path can both be fed from it without sharing any code of the method.

Every value is a pure function ``value(seed, tensor_id, flat_index)`` of a
counter-based generator (a splitmix64-style mixer followed by Box-Muller), so a
tensor can be produced in chunks, in any order, on any number of threads, and
is reproducible across runs.

The workloads stand in for the shapes of the paper's evaluation traces
(Table 1: mean / P99 input lengths of 7K-14K / 62K-82K tokens, 25-80 % prefix
reuse; Section 2.3: 35-55 % token-level hit rate); none of the traces' items are
reproduced here.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

PAGE = 64          # tokens per KV-cache page (cache block)
HEAD_DIM = 128

_GOLD = np.uint64(0x9E3779B97F4A7C15)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)

# tensor ids (second argument of the counter-based generator)
TID_Q, TID_K, TID_V, TID_PERM, TID_LEN, TID_FRAC, TID_C, TID_PART, TID_LSE, TID_ROWS, TID_STREAM = range(11)


def _mix64(x: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser on a uint64 array (wrap-around arithmetic)."""
    x = x.copy()
    x ^= x >> np.uint64(30)
    x *= _C1
    x ^= x >> np.uint64(27)
    x *= _C2
    x ^= x >> np.uint64(31)
    return x


def _stream_key(seed: int, tensor_id: int) -> np.uint64:
    with np.errstate(over="ignore"):
        k = np.array([(seed * 0x9E3779B97F4A7C15 + tensor_id * 0xD1B54A32D192ED03 + 0x1234567) % (1 << 64)],
                     dtype=np.uint64)
        return _mix64(_mix64(k))[0]


def counter_u64(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """64 random bits for counters ``start .. start+count-1`` of one stream."""
    with np.errstate(over="ignore"):
        idx = np.arange(start, start + count, dtype=np.uint64)
        return _mix64((idx + _stream_key(seed, tensor_id)) * _GOLD)


def counter_uniform(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """Uniform doubles in (0,1), one per counter."""
    bits = counter_u64(seed, tensor_id, start, count)
    return ((bits >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / (1 << 53))


def _normal_block(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """float32 N(0,1) for flat indices start..start+count-1 (start must be even).

    Counter c yields the Box-Muller pair (flat indices 2c and 2c+1).
    """
    assert start % 2 == 0
    npair = (count + 1) // 2
    bits = counter_u64(seed, tensor_id, start // 2, npair)
    u1 = ((bits >> np.uint64(40)).astype(np.float32) + np.float32(0.5)) * np.float32(1.0 / (1 << 24))
    u2 = ((bits & np.uint64(0xFFFFFF)).astype(np.float32) + np.float32(0.5)) * np.float32(1.0 / (1 << 24))
    rad = np.sqrt(np.float32(-2.0) * np.log(u1))
    ang = np.float32(2.0 * math.pi) * u2
    out = np.empty(2 * npair, dtype=np.float32)
    out[0::2] = rad * np.cos(ang)
    out[1::2] = rad * np.sin(ang)
    return out[:count]


def _threads() -> int:
    return max(1, min(16, os.cpu_count() or 1))


def normal_f32(seed: int, tensor_id: int, count: int, start: int = 0) -> np.ndarray:
    """i.i.d. N(0,1) float32 values for flat indices start..start+count-1."""
    out = np.empty(count, dtype=np.float32)
    chunk = 1 << 18
    first = start - (start % 2)

    def work(lo: int) -> None:
        hi = min(lo + chunk, start + count)
        blk = _normal_block(seed, tensor_id, lo, hi - lo)
        a = max(lo, start)
        out[a - start:hi - start] = blk[a - lo:]

    los = list(range(first, start + count, chunk))
    if len(los) == 1:
        work(los[0])
    else:
        with ThreadPoolExecutor(_threads()) as ex:
            list(ex.map(work, los))
    return out


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (round-to-nearest-even), returned as uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(bits).astype(np.float64)


def normal_bf16(seed: int, tensor_id: int, shape, start: int = 0) -> np.ndarray:
    """N(0,1) rounded to bf16; uint16 bit patterns of the given shape."""
    count = int(np.prod(shape))
    out = np.empty(count, dtype=np.uint16)
    chunk = 1 << 24
    for lo in range(0, count, chunk):
        hi = min(lo + chunk, count)
        out[lo:hi] = f32_to_bf16_bits(normal_f32(seed, tensor_id, hi - lo, start + lo))
    return out.reshape(shape)


def permutation(seed: int, tensor_id: int, n: int) -> np.ndarray:
    """Seeded Fisher-Yates permutation of 0..n-1 (int32)."""
    u = counter_uniform(seed, tensor_id, 0, max(n, 1))
    p = np.arange(n, dtype=np.int32)
    for i in range(n - 1, 0, -1):
        j = int(u[i] * (i + 1))
        p[i], p[j] = p[j], p[i]
    return p


# --------------------------------------------------------------------------------------
# Request / batch descriptions
# --------------------------------------------------------------------------------------

@dataclass
class Request:
    new_len: int      # R: uncached suffix length (the queries)
    prefix_len: int   # P: cached prefix length
    C: int            # CP degree

    @property
    def total_len(self) -> int:
        return self.new_len + self.prefix_len

    @property
    def n_pages(self) -> int:
        return (self.total_len + PAGE - 1) // PAGE


@dataclass
class Workload:
    """A batch of requests sharing one paged KV pool."""
    name: str
    seed: int
    Hq: int
    Hkv: int
    requests: list
    D: int = HEAD_DIM
    spare_pages: int = 3          # physical pages never referenced by any page table
    shuffle_pages: bool = True
    page: int = PAGE              # tokens per cache page
    meta: dict = field(default_factory=dict)

    @property
    def scale(self) -> float:
        """Softmax scale passed to the calls: 1/sqrt(D) unless ``meta["scale"]`` overrides it (tests use large scales to
        make the row maxima jump between key tiles)."""
        return float(self.meta.get("scale", 1.0 / math.sqrt(self.D)))

    @property
    def total_new(self) -> int:
        return sum(r.new_len for r in self.requests)

    @property
    def cu_new(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum([r.new_len for r in self.requests])]).astype(np.int64)

    @property
    def cu_pages(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum([-(-r.total_len // self.page) for r in self.requests])]).astype(np.int64)

    @property
    def num_pages(self) -> int:
        return int(self.cu_pages[-1]) + self.spare_pages


GARBAGE_POS = 0x7F61   # bf16 bits of about +2.99e38 (finite)
GARBAGE_NEG = 0xFF61


@dataclass
class Materialized:
    wl: Workload
    q: np.ndarray            # [sum R, Hq, D] bf16 bits (uint16), requests packed in order
    k_pages: np.ndarray      # [num_pages, PAGE, Hkv, D] bf16 bits
    v_pages: np.ndarray
    page_table: np.ndarray   # int32 [sum n_pages], packed per request (cu_pages)


def materialize(wl: Workload, need_q: bool = True) -> Materialized:
    """Build Q, the paged K/V pool and the page tables for a workload.

    Logical K/V token ``t`` of request ``b`` is the flat-index block
    ``(cu_tok[b] + t) * Hkv * D`` of streams TID_K / TID_V, so the logical content
    does not depend on the page permutation.  Slots of the pool that no request
    owns (tail of a last page, spare pages) are filled with large finite garbage
    of alternating sign: a correct implementation never lets them influence a
    result.
    """
    Hq, Hkv, D = wl.Hq, wl.Hkv, wl.D
    q = normal_bf16(wl.seed, TID_Q, (wl.total_new, Hq, D)) if need_q else None
    npg = wl.num_pages
    perm = permutation(wl.seed, TID_PERM, npg) if wl.shuffle_pages else np.arange(npg, dtype=np.int32)
    n_logical = int(wl.cu_pages[-1])
    page_table = perm[:n_logical].astype(np.int32).copy()

    ps = wl.page
    k_pages = np.empty((npg, ps, Hkv, D), dtype=np.uint16)
    v_pages = np.empty((npg, ps, Hkv, D), dtype=np.uint16)
    garb = np.where((np.arange(ps * Hkv * D) % 2) == 0, GARBAGE_POS, GARBAGE_NEG).astype(np.uint16)
    garb = garb.reshape(ps, Hkv, D)
    for p in perm[n_logical:]:
        k_pages[p] = garb
        v_pages[p] = garb[::-1]

    tok0 = 0
    row_elems = Hkv * D
    for b, r in enumerate(wl.requests):
        L = r.total_len
        kb = normal_bf16(wl.seed, TID_K, (L, Hkv, D), start=tok0 * row_elems)
        vb = normal_bf16(wl.seed, TID_V, (L, Hkv, D), start=tok0 * row_elems)
        pt = page_table[wl.cu_pages[b]:wl.cu_pages[b + 1]]
        full = L // ps
        if full:
            k_pages[pt[:full]] = kb[:full * ps].reshape(full, ps, Hkv, D)
            v_pages[pt[:full]] = vb[:full * ps].reshape(full, ps, Hkv, D)
        rem = L - full * ps
        if rem:
            k_pages[pt[full], :rem] = kb[full * ps:]
            v_pages[pt[full], :rem] = vb[full * ps:]
            k_pages[pt[full], rem:] = garb[rem:]
            v_pages[pt[full], rem:] = garb[::-1][rem:]
        tok0 += L
    return Materialized(wl, q, k_pages, v_pages, page_table)


@dataclass
class MaterializedFp8:
    wl: Workload
    q: np.ndarray            # [sum R, Hq, D] bf16 bits, as in Materialized
    k8_pages: np.ndarray     # [num_pages, PAGE, Hkv, D] uint8: E4M3 bytes
    v8_pages: np.ndarray
    k_scale: np.ndarray      # fp32 [Hkv]: value of a stored byte = scale[g] * e4m3(byte)
    v_scale: np.ndarray
    page_table: np.ndarray


def materialize_fp8(wl: Workload) -> MaterializedFp8:
    """The same logical N(0,1) K/V content as ``materialize``, stored as E4M3 bytes with one fp32 scale per
    KV head.  The scales differ from head to head (a wrong head-to-scale mapping changes the result) and put
    6 standard deviations at the format's largest value; the bytes are made by PyTorch's own float8 conversion
    (round to nearest even) after clipping to +-448, so the unused slots' large garbage becomes +-448."""
    import torch
    mat = materialize(wl)
    g = np.arange(wl.Hkv, dtype=np.float32)
    k_scale = ((6.0 / 448.0) * (1.0 + g / 8.0)).astype(np.float32)
    v_scale = ((6.0 / 448.0) * (1.5 - g / 16.0)).astype(np.float32)

    def to_e4m3(pages_bits, scale):
        out = np.empty(pages_bits.shape, dtype=np.uint8)
        step = max(1, (1 << 24) // int(np.prod(pages_bits.shape[1:])))
        for lo in range(0, pages_bits.shape[0], step):
            with np.errstate(over="ignore"):              # the unused slots' garbage overflows to inf and is clipped
                x = bf16_bits_to_f32(pages_bits[lo:lo + step]) / scale[None, None, :, None]
            t = torch.from_numpy(np.clip(x, -448.0, 448.0).astype(np.float32)).to(torch.float8_e4m3fn)
            out[lo:lo + step] = t.view(torch.uint8).numpy()
        return out

    return MaterializedFp8(wl, mat.q, to_e4m3(mat.k_pages, k_scale), to_e4m3(mat.v_pages, v_scale), k_scale, v_scale,
                           mat.page_table)


# --------------------------------------------------------------------------------------
# The five benchmark configurations
# --------------------------------------------------------------------------------------

def config1() -> Workload:
    """Single request, no prefix: R=1024, Hq=8, Hkv=2, C=2 (4 chunks of 256), seed 0."""
    return Workload("cfg1_R1024_P0_C2", 0, 8, 2, [Request(1024, 0, 2)])


def config2() -> Workload:
    """Llama-3-8B-shaped layer with a prefix hit: P=12288 (paged, shuffled), R=4096, C=4, seed 2."""
    return Workload("cfg2_R4096_P12288_C4", 2, 32, 8, [Request(4096, 12288, 4)])


def config3() -> Workload:
    """Long-context prefill, no prefix: R=131072, C=8 (16 chunks of 8192), seed 3."""
    return Workload("cfg3_R131072_P0_C8", 3, 32, 8, [Request(131072, 0, 8)])


def config4(seed: int = 4, B: int = 32, sigma: float = 1.0) -> Workload:
    """Heterogeneous varlen batch: log-normal total lengths (median 2048, clipped to [128, 65536]),
    cached fraction U[0, 0.9] rounded down to whole pages, C drawn from {1,2,4,8}."""
    u = counter_uniform(seed, TID_LEN, 0, 2 * B)
    z = np.sqrt(-2.0 * np.log(u[0::2])) * np.cos(2.0 * math.pi * u[1::2])
    L = np.clip(np.rint(np.exp(math.log(2048.0) + sigma * z)), 128, 65536).astype(np.int64)
    f = 0.9 * counter_uniform(seed, TID_FRAC, 0, B)
    P = (np.floor(f * L / PAGE) * PAGE).astype(np.int64)
    cs = np.array([1, 2, 4, 8])[(counter_uniform(seed, TID_C, 0, B) * 4).astype(np.int64)]
    reqs = [Request(int(L[i] - P[i]), int(P[i]), int(cs[i])) for i in range(B)]
    return Workload("cfg4_varlen_B%d" % B, seed, 32, 8, reqs)


def config5() -> Workload:
    """Qwen-72B-shaped layer: P=32768 (paged), R=32768, Hq=64, Hkv=8, C=8, seed 5."""
    return Workload("cfg5_R32768_P32768_C8", 5, 64, 8, [Request(32768, 32768, 8)])


def small_mixed(seed: int = 11) -> Workload:
    """A small ragged batch for element-by-element parity: spans several 128-row tiles, ragged
    tails, C that does not divide R, an empty trailing chunk, page-unaligned totals."""
    reqs = [Request(333, 192, 3), Request(5, 0, 4), Request(1, 64, 1), Request(700, 0, 2),
            Request(129, 448, 8), Request(256, 1024, 4)]
    return Workload("small_mixed", seed, 8, 2, reqs)


def variant_gqa8() -> Workload:
    """Config 2's lengths with the head shape of a 32/4 grouped-query model (eight query heads per KV
    head, the second model family of the paper's evaluation), seed 7."""
    return Workload("var_gqa8_R4096_P12288_C4", 7, 32, 4, [Request(4096, 12288, 4)])


def variant_chunked_prefill() -> Workload:
    """One 512-token chunk of a chunked prefill behind a 64K-token cached prefix (R << P): every work
    unit is cut along KV and merged by LSE, seed 8."""
    return Workload("var_chunk_R512_P65536_C2", 8, 32, 8, [Request(512, 65536, 2)])


def variant_mha() -> Workload:
    """Config 2's lengths with plain multi-head attention (16 query heads on 16 KV heads: every work unit is a
    single head, no K/V tile is shared), seed 9."""
    return Workload("var_mha_R4096_P12288_C4", 9, 16, 16, [Request(4096, 12288, 4)])


CONFIGS = {1: config1, 2: config2, 3: config3, 4: config4, 5: config5}
VARIANTS = {6: variant_gqa8, 7: variant_chunked_prefill, 8: variant_mha}


# --------------------------------------------------------------------------------------
# Merge-sweep inputs
# --------------------------------------------------------------------------------------

def merge_inputs(seed: int, N: int, T: int, H: int, D: int = HEAD_DIM, neg_inf_frac: int = 16):
    """Partials [N,T,H,D] fp32 ~ N(0,1), lses [N,H,T] fp32 ~ N(8, 2^2); in partial 0 every
    ``neg_inf_frac``-th (token, head) row has lse = -inf (a row that partial does not own)."""
    parts = normal_f32(seed, TID_PART, N * T * H * D).reshape(N, T, H, D)
    lses = (8.0 + 2.0 * normal_f32(seed, TID_LSE, N * H * T)).astype(np.float32).reshape(N, H, T)
    if neg_inf_frac and N > 1:
        flat = lses[0].reshape(-1)
        flat[::neg_inf_frac] = -np.inf
    return parts, lses


def sample_rows(seed: int, Hq: int, R: int, per_head: int) -> np.ndarray:
    """``per_head`` seeded random query rows for every head: int64 [Hq, per_head]."""
    u = counter_uniform(seed, TID_ROWS, 0, Hq * per_head).reshape(Hq, per_head)
    return np.minimum((u * R).astype(np.int64), R - 1)


# --------------------------------------------------------------------------------------
# Synthetic prefix streams for the cache-manager tests
# --------------------------------------------------------------------------------------

def prefix_stream(seed: int, n_requests: int, block_tokens: int = PAGE, max_new_blocks: int = 12):
    """Requests as (block keys, total length L) with the reuse structure of multi-turn and shared-prompt
    traffic: half of the requests extend an earlier request (next turn), three in ten branch off an earlier
    request's prefix at a random depth (shared system prompt, different question), the rest start a new
    prefix.  Block keys are distinct 64-bit integers; L = whole blocks plus a ragged tail."""
    u = counter_uniform(seed, TID_STREAM, 0, 4 * n_requests)
    keys = counter_u64(seed, TID_STREAM, 1 << 40, n_requests * max_new_blocks)
    history, out, used = [], [], 0
    for i in range(n_requests):
        kind, pick, depth, grow = u[4 * i], u[4 * i + 1], u[4 * i + 2], u[4 * i + 3]
        n_new = 1 + int(grow * max_new_blocks) % max_new_blocks
        if history and kind < 0.5:
            base = list(history[int(pick * len(history))])
        elif history and kind < 0.8:
            src = history[int(pick * len(history))]
            base = list(src[:1 + int(depth * len(src)) % len(src)])
        else:
            base = []
        blocks = base + [int(k) for k in keys[used:used + n_new]]
        used += n_new
        history.append(blocks)
        out.append((blocks, len(blocks) * block_tokens + int(depth * block_tokens) % block_tokens))
    return out
