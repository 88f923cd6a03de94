"""Pins for the attention oracle: closed forms, brute force, library routines, invariances (no GPU)."""
import math

import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_2609_04774_b200 import workloads as wl

PAGE = 16


def _tiny(seed, R, P, Hq, Hkv, D, shuffle=True, extra_pages=2):
    """Contiguous K/V plus the same content scattered into a paged pool."""
    L = P + R
    q = wl.normal_bf16(seed, wl.TID_Q, (R, Hq, D))
    k = wl.normal_bf16(seed, wl.TID_K, (L, Hkv, D))
    v = wl.normal_bf16(seed, wl.TID_V, (L, Hkv, D))
    npg = -(-L // PAGE)
    pool = npg + extra_pages
    perm = wl.permutation(seed, wl.TID_PERM, pool) if shuffle else np.arange(pool, dtype=np.int32)
    pt = perm[:npg].copy()
    kp = np.full((pool, PAGE, Hkv, D), wl.GARBAGE_POS, dtype=np.uint16)
    vp = np.full((pool, PAGE, Hkv, D), wl.GARBAGE_NEG, dtype=np.uint16)
    for t in range(L):
        kp[pt[t // PAGE], t % PAGE] = k[t]
        vp[pt[t // PAGE], t % PAGE] = v[t]
    return q, k, v, kp, vp, pt


def _f64(bits):
    return wl.bf16_bits_to_f64(bits)


def test_streaming_equals_definition_form():
    R, P, Hq, Hkv, D = 37, 27, 4, 2, 16
    scale = 1 / math.sqrt(D)
    q, k, v, kp, vp, pt = _tiny(1, R, P, Hq, Hkv, D)
    O1, L1 = orc.attn_definition(q, k, v, P, scale)
    O2, L2 = orc.attn_full(q, kp, vp, pt, P, Hkv, scale)
    assert np.abs(O1 - O2).max() < 1e-12 and np.abs(L1 - L2).max() < 1e-12
    for C in (1, 2, 3, 4, 8):
        O3, L3, po, pl = orc.attn_sharded(q, kp, vp, pt, P, Hkv, scale, C)
        assert np.abs(O1 - O3).max() < 1e-12 and np.abs(L1 - L3).max() < 1e-12   # CP == single rank
        Om, Lm = orc.merge(po, pl)                                                # row-disjoint partials
        assert np.abs(O1 - Om).max() < 1e-12 and np.abs(L1 - Lm).max() < 1e-12


def test_against_torch_sdpa_fp64():
    # An independent library routine: PyTorch's scaled_dot_product_attention on CPU in fp64 with an
    # explicit boolean mask (key j visible to new token r iff j <= P + r) and grouped KV heads.
    R, P, Hq, Hkv, D = 45, 19, 6, 2, 32
    scale = 0.37
    q, k, v, kp, vp, pt = _tiny(2, R, P, Hq, Hkv, D)
    G = Hq // Hkv
    tq = torch.from_numpy(_f64(q)).permute(1, 0, 2)[None]                       # [1,Hq,R,D]
    tk = torch.from_numpy(_f64(k)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    tv = torch.from_numpy(_f64(v)).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    mask = torch.arange(P + R)[None, :] <= (P + torch.arange(R))[:, None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask, scale=scale)
    ref = ref[0].permute(1, 0, 2).numpy()
    lse_ref = torch.logsumexp((tq @ tk.transpose(-1, -2) * scale).masked_fill(~mask, -math.inf), -1)[0].numpy()
    O, LSE = orc.attn_full(q, kp, vp, pt, P, Hkv, scale)
    assert np.abs(O - ref).max() < 1e-12
    assert np.abs(LSE - lse_ref).max() < 1e-12


def test_zero_queries_give_running_mean_and_log_count():
    R, P, Hq, Hkv, D = 21, 13, 2, 1, 8
    q, k, v, kp, vp, pt = _tiny(3, R, P, Hq, Hkv, D)
    q[:] = 0
    O, LSE = orc.attn_full(q, kp, vp, pt, P, Hkv, 1.0)
    vf = _f64(v)
    for r in range(R):
        n = P + r + 1
        assert np.allclose(LSE[:, r], math.log(n), atol=1e-13)
        assert np.allclose(O[r, 0], vf[:n, 0].mean(axis=0), atol=1e-13)


def test_equal_values_row_zero_and_dominant_key():
    R, P, Hq, Hkv, D = 9, 0, 2, 2, 8
    scale = 0.5
    q, k, v, kp, vp, pt = _tiny(4, R, P, Hq, Hkv, D, shuffle=False)
    # row 0 with no prefix sees only key 0
    O, LSE = orc.attn_full(q, kp, vp, pt, P, Hkv, scale)
    assert np.allclose(O[0], _f64(v)[0], atol=0)
    assert np.allclose(LSE[:, 0], scale * (_f64(q)[0] * _f64(k)[0]).sum(-1), atol=1e-14)
    # all values equal -> output equals that value whatever the scores
    vp2 = vp.copy()
    vp2[:] = wl.f32_to_bf16_bits(np.array([1.5], dtype=np.float32))[0]
    O2, _ = orc.attn_full(q, kp, vp2, pt, P, Hkv, scale)
    assert np.allclose(O2, 1.5, atol=1e-14)
    # one key with a dominating score: q = e0 * 64, key 3 = e0 * 64 (score 2048 * scale), others ~N(0,1)
    q3 = q.copy()
    k3 = kp.copy()
    big = wl.f32_to_bf16_bits(np.array([64.0], dtype=np.float32))[0]
    q3[:] = 0
    q3[:, :, 0] = big
    k3[pt[3 // PAGE], 3 % PAGE, :, :] = 0
    k3[pt[3 // PAGE], 3 % PAGE, :, 0] = big
    O3, L3 = orc.attn_full(q3, k3, vp, pt, P, Hkv, scale)
    for r in range(3, R):
        assert np.allclose(O3[r], _f64(v)[3], atol=1e-9)
        assert abs(L3[0, r] - 4096 * scale) < 1e-9


def test_prefix_equivalence_and_page_permutation():
    # Section 2.2: with a cached prefix only the R new tokens are computed, and they attend to the
    # prefix plus the preceding new tokens -> rows [P, L) of plain causal attention over L tokens.
    R, P, Hq, Hkv, D = 23, 32, 4, 2, 16
    scale = 1 / math.sqrt(D)
    q, k, v, kp, vp, pt = _tiny(5, R, P, Hq, Hkv, D)
    L = P + R
    qfull = wl.normal_bf16(99, wl.TID_Q, (L, Hq, D))
    qfull[P:] = q
    Ofull, Lfull = orc.attn_full(qfull, kp, vp, pt, 0, Hkv, scale)
    O, LSE = orc.attn_full(q, kp, vp, pt, P, Hkv, scale)
    assert np.array_equal(O, Ofull[P:]) and np.array_equal(LSE, Lfull[:, P:])
    # any permutation of physical pages leaves the result bit-identical
    perm2 = wl.permutation(77, wl.TID_PERM, kp.shape[0])
    kp2, vp2 = np.empty_like(kp), np.empty_like(vp)
    kp2[perm2] = kp
    vp2[perm2] = vp
    O2, LSE2 = orc.attn_full(q, kp2, vp2, perm2[pt], P, Hkv, scale)
    assert np.array_equal(O, O2) and np.array_equal(LSE, LSE2)
    # strided cache view (extra padding between heads) addresses the same elements
    kpad = np.zeros(kp.shape[:2] + (Hkv + 1, D), dtype=np.uint16)
    vpad = np.zeros_like(kpad)
    kpad[:, :, :Hkv], vpad[:, :, :Hkv] = kp, vp
    O3, LSE3 = orc.attn_full(q, kpad[:, :, :Hkv], vpad[:, :, :Hkv], pt, P, Hkv, scale)
    assert np.array_equal(O, O3) and np.array_equal(LSE, LSE3)


def test_softmax_rows_sum_to_one_via_unit_values():
    # With V = 1 in one dim and a second dim holding the key index, O[...,0] is the sum of the softmax
    # weights (must be 1) and O[...,1] is a convex combination of visible indices (must lie in [0, P+r]).
    R, P, Hq, Hkv, D = 17, 8, 2, 1, 4
    q, k, v, kp, vp, pt = _tiny(6, R, P, Hq, Hkv, D)
    one = wl.f32_to_bf16_bits(np.array([1.0], dtype=np.float32))[0]
    for t in range(P + R):
        vp[pt[t // PAGE], t % PAGE, :, 0] = one
        vp[pt[t // PAGE], t % PAGE, :, 1] = wl.f32_to_bf16_bits(np.array([t], dtype=np.float32))[0]
    O, _ = orc.attn_full(q, kp, vp, pt, P, Hkv, 0.3)
    assert np.allclose(O[..., 0], 1.0, atol=1e-14)
    for r in range(R):
        assert (O[r, :, 1] >= 0).all() and (O[r, :, 1] <= P + r + 1e-12).all()


def test_kv_split_partials_merge_to_full():
    # Keys split by zigzag chunk ownership (KV-disjoint partials over the same rows) merge exactly.
    R, P, Hq, Hkv, D = 40, 16, 4, 2, 16
    scale = 1 / math.sqrt(D)
    q, k, v, kp, vp, pt = _tiny(7, R, P, Hq, Hkv, D)
    O, LSE = orc.attn_full(q, kp, vp, pt, P, Hkv, scale)
    C = 4
    parts, lses = [], []
    for kk, sh in enumerate(orc.plan(R, P, C)):
        ranges = [[P + b, P + e] for b, e in zip(sh["q_begin"], sh["q_end"])]
        if kk == 0:
            ranges.append([0, P])                                   # shard 0 also holds the prefix keys
        o, l = orc.attn_rows(q, kp, vp, pt, P, Hkv, scale, np.arange(R), key_ranges=ranges)
        parts.append(o)
        lses.append(l)
    assert any(np.isneginf(l).any() for l in lses)                  # early rows see none of a late shard's keys
    Om, Lm = orc.merge(np.stack(parts), np.stack(lses))
    assert np.abs(Om - O).max() < 1e-12 and np.abs(Lm - LSE).max() < 1e-12


def test_bad_arguments_raise():
    q, k, v, kp, vp, pt = _tiny(8, 4, 0, 2, 1, 8)
    with pytest.raises(ValueError):
        orc.attn_pairs(q, kp, vp, pt, 0, 1, 1.0, [4], [0])
