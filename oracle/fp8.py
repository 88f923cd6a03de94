"""CPU oracle of the FP8 K/V variant of cache-aware causal prefill attention.  TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this module; it shares no
code with the CUDA library.  The paper's main model is an FP8 model (Section 9.1) but the paper gives no
recipe for an FP8 attention path, so the storage format is a reading (stated in full in the design notes):

  * K and V pages hold OCP E4M3 bytes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits; no infinities,
    S.1111.111 is NaN, largest finite value 448); the value of a stored byte b of KV head g is
    ``scale[g] * e4m3(b)`` with one fp32 scale per KV head for K and one for V.
  * A query row (one token, one head; 128 bf16 values) is quantised to E4M3 with its own scale:
    ``amax = max |q|``; ``q_scale = amax / 448`` and ``inv = 448 / amax`` (both IEEE fp32 divisions);
    ``code = e4m3_rne_satfinite(q * inv)`` with the product rounded to fp32 first.  A row of zeros has
    scale 0 and codes 0.  Because a quantised code is an integer decision, this module takes it in fp32
    exactly as stated, so that the library's codes can be compared bit for bit.
  * With ``q^ = q_scale * e4m3(code)``, ``k_j = k_scale[g] * e4m3(K8[j])``, ``v_j = v_scale[g] * e4m3(V8[j])``
    widened exactly to fp64, the result is the Section 2.1 formula on these values, in fp64: scores
    ``S_j = s * q^ . k_j`` for ``j <= P + r`` (Section 2.2: prefix plus preceding new tokens), softmax over them,
    ``O = sum_j p_j v_j``, ``LSE = m + ln sum_j exp(S_j - m)``.  Nothing else is rounded.

Functions: ``e4m3_decode`` / ``e4m3_encode`` (the format), ``quantize_q``, ``quantize_kv`` (what a writer of
such a cache does: ``e4m3_rne_satfinite(x / scale[g])`` with the quotient rounded to fp32), ``attn_fp8_pairs``
/ ``attn_fp8_rows`` (the attention itself, also returning the absolute-value weighted mean
``A = sum_j p_j |v_j|`` that bounds the effect of rounding the weights p).  Pins: ``tests/test_oracle_fp8.py``.
"""
from __future__ import annotations

import numpy as np


# ------------------------------------------------------------------------------------------
# The E4M3 format
# ------------------------------------------------------------------------------------------

def _decode_table() -> np.ndarray:
    t = np.empty(256, dtype=np.float64)
    for b in range(256):
        sign = -1.0 if b & 0x80 else 1.0
        e, m = (b >> 3) & 0xF, b & 0x7
        if e == 0xF and m == 0x7:
            t[b] = np.nan
        elif e == 0:
            t[b] = sign * m * 2.0 ** -9                  # subnormal: m/8 * 2^(1-7)
        else:
            t[b] = sign * (1.0 + m / 8.0) * 2.0 ** (e - 7)
    return t


_DECODE = _decode_table()
E4M3_MAX = 448.0


def e4m3_decode(codes) -> np.ndarray:
    """uint8 codes -> fp64 values (exact)."""
    return _DECODE[np.asarray(codes, dtype=np.uint8)]


def e4m3_encode(x) -> np.ndarray:
    """fp32 values -> uint8 codes: round to the nearest representable value, ties to the even code,
    magnitudes beyond 448 (infinities included) saturate to +-448, NaN -> 0x7F."""
    x = np.asarray(x, dtype=np.float32)
    mag = np.abs(x).astype(np.float64)
    grid = _DECODE[:0x7F]                                 # the 127 finite non-negative values, ascending with the code
    hi = np.searchsorted(grid, mag, side="left")          # first code whose value is >= mag
    hi = np.clip(hi, 0, 0x7E)
    lo = np.clip(hi - 1, 0, 0x7E)
    d_lo, d_hi = mag - grid[lo], grid[hi] - mag
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    code = np.where(pick_hi, hi, lo)
    code = np.where(mag >= E4M3_MAX, 0x7E, code)          # satfinite
    code = np.where(mag <= 0.0, 0, code).astype(np.uint8)
    code = code | np.where(np.signbit(x), 0x80, 0).astype(np.uint8)
    return np.where(np.isnan(x), np.uint8(0x7F), code).astype(np.uint8)


def _bf16_bits_to_f32(bits) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def quantize_q(q_bits):
    """q [R, Hq, D] bf16 bits -> (codes uint8 [R, Hq, D], q_scale fp32 [R, Hq]); fp32 decisions as stated above."""
    q = _bf16_bits_to_f32(q_bits)
    amax = np.abs(q).max(axis=-1)                                       # exact: a max of bf16 values
    live = amax > 0
    safe = np.where(live, amax, np.float32(1.0)).astype(np.float32)
    q_scale = np.where(live, safe / np.float32(448.0), np.float32(0.0)).astype(np.float32)
    inv = np.where(live, np.float32(448.0) / safe, np.float32(0.0)).astype(np.float32)
    y = (q * inv[..., None]).astype(np.float32)
    return e4m3_encode(y), q_scale


def quantize_kv(rows_bits, scale):
    """rows [n, Hkv, D] bf16 bits, scale fp32 [Hkv] (positive) -> uint8 codes: e4m3_rne_satfinite(x / scale[g]),
    the quotient rounded to fp32 (IEEE division)."""
    x = _bf16_bits_to_f32(rows_bits)
    s = np.asarray(scale, dtype=np.float32)[None, :, None]
    with np.errstate(over="ignore"):                      # a quotient beyond fp32 is +-inf, which saturates like any large value
        return e4m3_encode((x / s).astype(np.float32))


# ------------------------------------------------------------------------------------------
# Attention on the stored bytes (Section 2.1 formula, Section 2.2 prefix rule), fp64
# ------------------------------------------------------------------------------------------

def _gather_head(pages8, page_table, n_tokens, g):
    """Logical tokens [0, n_tokens) of KV head g through the page table: token t is slot t % page_size of page
    page_table[t // page_size].  -> uint8 [n_tokens, D]"""
    ps = pages8.shape[1]
    t = np.arange(n_tokens)
    return pages8[np.asarray(page_table, dtype=np.int64)[t // ps], t % ps, g]


def attn_fp8_pairs(q_bits, k8_pages, v8_pages, k_scale, v_scale, page_table, P: int, Hkv: int, scale: float, rows, heads):
    """Evaluate chosen (row, head) pairs of one request.

    q_bits [R, Hq, D] bf16 bits; k8_pages / v8_pages [num_pages, page_size, Hkv, D] uint8 (E4M3);
    k_scale / v_scale fp32 [Hkv]; rows / heads: equally long index arrays.
    Returns O [n, D], LSE [n] and A [n, D] = sum_j p_j |v_j| (p normalised), all fp64.
    """
    R, Hq, D = q_bits.shape
    G = Hq // Hkv
    rows = np.asarray(rows, dtype=np.int64)
    heads = np.asarray(heads, dtype=np.int64)
    codes, q_scale = quantize_q(q_bits)
    L = P + R
    O = np.zeros((rows.size, D))
    A = np.zeros((rows.size, D))
    LSE = np.zeros(rows.size)
    for g in range(Hkv):
        sel = np.nonzero(heads // G == g)[0]
        if sel.size == 0:
            continue
        n_need = int(P + rows[sel].max() + 1)
        assert n_need <= L
        K = float(np.float32(k_scale[g])) * e4m3_decode(_gather_head(k8_pages, page_table, n_need, g))
        V = float(np.float32(v_scale[g])) * e4m3_decode(_gather_head(v8_pages, page_table, n_need, g))
        for i in sel:
            r, h = int(rows[i]), int(heads[i])
            n = P + r + 1                                             # keys 0 .. P + r, diagonal included
            qv = float(q_scale[r, h]) * e4m3_decode(codes[r, h])
            s = scale * (K[:n] @ qv)
            m = s.max()
            p = np.exp(s - m)
            l = p.sum()
            O[i] = (p @ V[:n]) / l
            A[i] = (p @ np.abs(V[:n])) / l
            LSE[i] = m + np.log(l)
    return O, LSE, A


def attn_fp8_rows(q_bits, k8_pages, v8_pages, k_scale, v_scale, page_table, P, Hkv, scale, rows):
    """All heads of the given new-token rows: O [len(rows), Hq, D], LSE [Hq, len(rows)], A like O."""
    R, Hq, D = q_bits.shape
    rows = np.asarray(rows, dtype=np.int64)
    rr = np.repeat(rows, Hq)
    hh = np.tile(np.arange(Hq), rows.size)
    o, l, a = attn_fp8_pairs(q_bits, k8_pages, v8_pages, k_scale, v_scale, page_table, P, Hkv, scale, rr, hh)
    return o.reshape(rows.size, Hq, D), l.reshape(rows.size, Hq).T.copy(), a.reshape(rows.size, Hq, D)
