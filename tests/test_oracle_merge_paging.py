"""Pins for the merge oracle and the page-index oracle (no GPU)."""
import math

import numpy as np

from oracle import reference as orc
from paper_2609_04774_b200 import workloads as wl


def test_merge_worked_example():
    # Two partials over one row: lse = ln 1 and ln 3 -> weights 1/4 and 3/4, lse = ln 4.
    a = np.array([1.0, -2.0, 0.5, 8.0])
    b = np.array([3.0, 2.0, -0.5, 0.0])
    parts = np.stack([a, b]).reshape(2, 1, 1, 4)
    lses = np.array([math.log(1.0), math.log(3.0)]).reshape(2, 1, 1)
    out, lse = orc.merge(parts, lses)
    assert np.allclose(out[0, 0], 0.25 * a + 0.75 * b, atol=1e-15)
    assert abs(lse[0, 0] - math.log(4.0)) < 1e-15


def test_merge_identity_copy_and_dead_rows():
    parts, lses = wl.merge_inputs(6, 3, 40, 4, 8, neg_inf_frac=5)
    out, lse = orc.merge(parts, lses)
    # N = 1 is a copy
    o1, l1 = orc.merge(parts[:1], np.where(np.isneginf(lses[:1]), 0.0, lses[:1]))
    assert np.array_equal(o1, parts[0].astype(np.float64))
    # a partial with lse = -inf is the identity element, whatever (even non-finite) values it holds
    extra = np.full((1,) + parts.shape[1:], np.nan)
    o2, l2 = orc.merge(np.concatenate([parts, extra]), np.concatenate([lses, np.full((1,) + lses.shape[1:], -np.inf)]))
    assert np.array_equal(o2, out) and np.array_equal(l2, lse)
    # a row dead in every partial -> zeros and -inf
    dl = lses.copy()
    dl[:, 2, 7] = -np.inf
    o3, l3 = orc.merge(parts, dl)
    assert np.all(o3[7, 2] == 0) and np.isneginf(l3[2, 7])
    assert np.isfinite(o3).all()


def test_merge_commutative_associative():
    parts, lses = wl.merge_inputs(7, 4, 33, 3, 8, neg_inf_frac=4)
    out, lse = orc.merge(parts, lses)
    perm = [2, 0, 3, 1]
    o2, l2 = orc.merge(parts[perm], lses[perm])
    assert np.abs(o2 - out).max() < 1e-13 and np.abs(l2 - lse).max() < 1e-13
    oa, la = orc.merge(parts[:2], lses[:2])
    ob, lb = orc.merge(parts[2:], lses[2:])
    o3, l3 = orc.merge(np.stack([oa, ob]), np.stack([la, lb]))
    assert np.abs(o3 - out).max() < 1e-13 and np.abs(l3 - lse).max() < 1e-13


def test_merge_matches_logsumexp_and_softmax_weights():
    from scipy.special import logsumexp, softmax
    parts, lses = wl.merge_inputs(8, 5, 20, 2, 4, neg_inf_frac=0)
    out, lse = orc.merge(parts, lses)
    assert np.allclose(lse, logsumexp(lses.astype(np.float64), axis=0), atol=1e-13)
    w = softmax(lses.astype(np.float64), axis=0)                         # [N,H,T]
    ref = np.einsum("nht,nthd->thd", w, parts.astype(np.float64))
    assert np.allclose(out, ref, atol=1e-13)


def test_page_offset_closed_form_and_roundtrip():
    ps, Hkv, D = 64, 2, 8
    pool = 9
    sp, st, sh = ps * Hkv * D, Hkv * D, D
    pt = wl.permutation(3, wl.TID_PERM, pool)[:6]
    for t in (0, 1, 63, 64, 65, 200, 383):
        for g in range(Hkv):
            assert orc.page_offset(pt, t, g, ps, sp, st, sh) == int(pt[t // 64]) * sp + (t % 64) * st + g * sh
    ident = np.arange(6, dtype=np.int32)
    assert orc.page_offset(ident, 130, 1, ps, sp, st, sh) == 130 * st + sh    # identity table == contiguous
    pages = wl.normal_bf16(3, wl.TID_K, (pool, ps, Hkv, D))
    before = pages.copy()
    rows = wl.normal_bf16(4, wl.TID_V, (150, Hkv, D))
    orc.kv_append(pages, pt, 70, rows)
    assert np.array_equal(orc.kv_gather(pages, pt, 70, 220), rows)            # gather o append = identity
    untouched = orc.kv_gather(before, pt, 0, 70)
    assert np.array_equal(orc.kv_gather(pages, pt, 0, 70), untouched)
    flat = pages.reshape(-1)
    offs = orc.page_offset(pt, np.arange(70, 220), 1, ps, sp, st, sh)
    assert np.array_equal(flat[offs], rows[:, 1, 0])
