"""Pins of the FP8 K/V oracle (no GPU): the E4M3 format against hand values and PyTorch's float8 type, the
quantisers against exactly representable inputs, and the attention function against the bf16 oracle on values
that both formats hold exactly, closed forms and scale identities."""
import numpy as np
import pytest
import torch

from oracle import fp8 as o8
from oracle import reference as orc
from paper_2609_04774_b200 import workloads as wl


def f32_to_bf16_bits_exact(x):
    """fp32 values that are exactly representable in bf16 -> their bf16 bits."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    assert (b & 0xFFFF == 0).all()
    return (b >> 16).astype(np.uint16)


def test_e4m3_decode_hand_values_and_torch():
    hand = {0x00: 0.0, 0x01: 2.0 ** -9, 0x07: 7 * 2.0 ** -9, 0x08: 2.0 ** -6, 0x38: 1.0, 0x39: 1.125, 0x40: 2.0,
            0x7E: 448.0, 0xB8: -1.0, 0xFE: -448.0, 0x77: 240.0, 0x30: 0.5}
    for code, val in hand.items():
        assert o8.e4m3_decode(np.uint8(code)) == val, hex(code)
    assert np.isnan(o8.e4m3_decode(np.uint8(0x7F))) and np.isnan(o8.e4m3_decode(np.uint8(0xFF)))
    codes = np.arange(256, dtype=np.uint8)
    ref = torch.from_numpy(codes).view(torch.float8_e4m3fn).to(torch.float32).numpy().astype(np.float64)
    got = o8.e4m3_decode(codes)
    fin = np.isfinite(ref)
    assert np.array_equal(np.isnan(got), ~fin) and np.array_equal(got[fin], ref[fin])


def test_e4m3_encode_round_trip_ties_saturation_and_torch():
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F and c != 0x80], dtype=np.uint8)
    assert np.array_equal(o8.e4m3_encode(o8.e4m3_decode(codes).astype(np.float32)), codes)       # every finite value
    # ties go to the even code: 1.0625 lies midway between 1.0 (0x38) and 1.125 (0x39); 1.1875 between 0x39 and 0x3A
    assert o8.e4m3_encode(np.float32(1.0625)) == 0x38 and o8.e4m3_encode(np.float32(1.1875)) == 0x3A
    assert o8.e4m3_encode(np.float32(-1.0625)) == 0xB8
    # subnormal spacing 2^-9: 1.5 * 2^-9 ties to 2 * 2^-9 (even), 0.5 * 2^-9 ties to zero, 0.51 * 2^-9 rounds up
    assert o8.e4m3_encode(np.float32(1.5 * 2.0 ** -9)) == 0x02 and o8.e4m3_encode(np.float32(0.5 * 2.0 ** -9)) == 0x00
    assert o8.e4m3_encode(np.float32(0.51 * 2.0 ** -9)) == 0x01
    # saturation: anything beyond 448 (also what would round past it, and infinity) is +-448; NaN is 0x7F
    for v, c in ((448.0, 0x7E), (463.9, 0x7E), (464.0, 0x7E), (1e30, 0x7E), (np.inf, 0x7E), (-5000.0, 0xFE)):
        assert o8.e4m3_encode(np.float32(v)) == c, v
    assert o8.e4m3_encode(np.float32(np.nan)) == 0x7F
    # PyTorch's conversion (round to nearest even) on in-range values
    x = (wl.normal_f32(77, wl.TID_Q, 200000) * np.float32(60.0)).astype(np.float32)
    x = np.concatenate([x, x * np.float32(1e-3), x * np.float32(1e-5)])
    x = x[np.abs(x) <= 448.0]
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = o8.e4m3_encode(x)
    same_value = o8.e4m3_decode(got) == o8.e4m3_decode(ref)          # -0 and +0 codes both stand for zero
    assert same_value.all()


def test_quantize_q_on_representable_rows():
    rng = np.random.default_rng(5)
    R, Hq, D = 7, 3, 128
    codes = rng.integers(0, 0x7F, size=(R, Hq, D)).astype(np.uint8) | (rng.integers(0, 2, size=(R, Hq, D)) << 7).astype(np.uint8)
    codes[..., 0] = 0x7E                                    # every row's largest magnitude is 448 * 2^j
    shift = rng.integers(-6, 4, size=(R, Hq))
    vals = o8.e4m3_decode(codes) * 2.0 ** shift[..., None]
    got_codes, got_scale = o8.quantize_q(f32_to_bf16_bits_exact(vals.astype(np.float32)))
    assert np.array_equal(got_scale, (2.0 ** shift).astype(np.float32))
    assert np.array_equal(o8.e4m3_decode(got_codes), o8.e4m3_decode(codes))
    # a row of zeros: scale 0, codes 0; a general row: its largest element maps to +-448 and nothing decodes beyond it
    z_codes, z_scale = o8.quantize_q(np.zeros((1, 1, D), dtype=np.uint16))
    assert z_scale[0, 0] == 0 and not z_codes.any()
    q = wl.normal_bf16(3, wl.TID_Q, (5, 2, D))
    c, s = o8.quantize_q(q)
    back = o8.e4m3_decode(c) * s[..., None].astype(np.float64)
    qf = wl.bf16_bits_to_f64(q)
    assert (np.abs(o8.e4m3_decode(c)).max(-1) == 448.0).all()
    assert (np.abs(back - qf) <= 2.0 ** -4 * np.abs(qf) + s[..., None] * 2.0 ** -10).all()      # half an ulp, or half a subnormal step


def test_quantize_kv_divides_by_the_heads_scale():
    rows = wl.normal_bf16(4, wl.TID_K, (9, 2, 128))
    scale = np.array([0.25, 2.0 ** -5], dtype=np.float32)
    c = o8.quantize_kv(rows, scale)
    x = wl.bf16_bits_to_f64(rows)
    for g in range(2):
        ref = torch.from_numpy(np.clip(x[:, g] / float(scale[g]), -448, 448).astype(np.float32)).to(torch.float8_e4m3fn)
        assert np.array_equal(o8.e4m3_decode(c[:, g]), ref.to(torch.float32).numpy().astype(np.float64))


def _grid_case(seed, R, P, Hq, Hkv, page=64):
    """Inputs that E4M3 (with power-of-two scales) and bf16 both hold exactly."""
    rng = np.random.default_rng(seed)
    D, L = 128, P + R
    n_pages = -(-L // page) + 2
    pt = rng.permutation(n_pages)[:-(-L // page)].astype(np.int32)
    small = np.array([c for c in range(0x20, 0x48)], dtype=np.uint8)          # magnitudes 2^-3 .. 3.75
    def codes(shape):
        return small[rng.integers(0, small.size, size=shape)] | (rng.integers(0, 2, size=shape) << 7).astype(np.uint8)
    k8, v8 = codes((n_pages, page, Hkv, D)), codes((n_pages, page, Hkv, D))
    k_scale = (2.0 ** rng.integers(-3, 2, size=Hkv)).astype(np.float32)
    v_scale = (2.0 ** rng.integers(-2, 3, size=Hkv)).astype(np.float32)
    qc = codes((R, Hq, D))
    qc[..., 5] = 0x7E
    q_vals = o8.e4m3_decode(qc) * 2.0 ** rng.integers(-9, -5, size=(R, Hq, 1))
    q_bits = f32_to_bf16_bits_exact(q_vals.astype(np.float32))
    k_bits = f32_to_bf16_bits_exact((o8.e4m3_decode(k8) * k_scale[None, None, :, None]).astype(np.float32))
    v_bits = f32_to_bf16_bits_exact((o8.e4m3_decode(v8) * v_scale[None, None, :, None]).astype(np.float32))
    return q_bits, k8, v8, k_scale, v_scale, pt, k_bits, v_bits


@pytest.mark.parametrize("shape", [(37, 0, 4, 2, 64), (20, 150, 6, 2, 16), (9, 64, 8, 8, 32), (130, 70, 2, 1, 128)])
def test_fp8_attention_equals_bf16_oracle_on_values_both_formats_hold(shape):
    R, P, Hq, Hkv, page = shape
    q_bits, k8, v8, ks, vs, pt, k_bits, v_bits = _grid_case(sum(shape), R, P, Hq, Hkv, page)
    rows = np.arange(R)
    o, l, a = o8.attn_fp8_rows(q_bits, k8, v8, ks, vs, pt, P, Hkv, 0.11, rows)
    ro, rl = orc.attn_rows(q_bits, k_bits, v_bits, pt, P, Hkv, 0.11, rows)
    assert np.abs(o - ro).max() <= 1e-12 * max(1.0, np.abs(ro).max())
    assert np.abs(l - rl).max() <= 1e-12 * max(1.0, np.abs(rl).max())
    assert (a >= np.abs(o) - 1e-12).all()                                     # |sum p v| <= sum p |v|
    # with the sign bits of V cleared the weighted mean of |v| is the output itself
    o2, _, a2 = o8.attn_fp8_rows(q_bits, k8, v8 & 0x7F, ks, vs, pt, P, Hkv, 0.11, rows)
    assert np.abs(o2 - a2).max() <= 1e-13 * max(1.0, a2.max()) and np.abs(a2 - a).max() <= 1e-13 * max(1.0, a.max())


def test_fp8_attention_closed_forms_and_scale_identities():
    m8 = wl.materialize_fp8(wl.Workload("fp8_pin", 12, 4, 2, [wl.Request(40, 64, 1)]))
    w = m8.wl
    P, R = 64, 40
    rows = np.array([0, 1, 17, 39])
    # zero queries: uniform weights -> LSE = ln(number of visible keys), O = mean of the dequantised values
    zq = np.zeros_like(m8.q)
    o, l, _ = o8.attn_fp8_rows(zq, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv, w.scale, rows)
    for i, r in enumerate(rows):
        n = P + r + 1
        assert np.allclose(l[:, i], np.log(n), rtol=0, atol=1e-12)
        for h in range(w.Hq):
            g = h // (w.Hq // w.Hkv)
            t = np.arange(n)
            v = float(m8.v_scale[g]) * o8.e4m3_decode(m8.v8_pages[m8.page_table[t // 64], t % 64, g])
            assert np.allclose(o[i, h], v.mean(0), rtol=0, atol=1e-12)
    # doubling v_scale doubles O and leaves LSE; doubling k_scale equals doubling the softmax scale
    base = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv, w.scale, rows)
    v2 = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, 2 * m8.v_scale, m8.page_table, P, w.Hkv, w.scale, rows)
    assert np.allclose(v2[0], 2 * base[0], rtol=1e-13, atol=0) and np.allclose(v2[1], base[1], rtol=0, atol=1e-12)
    k2 = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, 2 * m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv, w.scale, rows)
    s2 = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv, 2 * w.scale, rows)
    assert np.allclose(k2[0], s2[0], rtol=1e-12, atol=1e-13) and np.allclose(k2[1], s2[1], rtol=1e-12, atol=1e-12)
    # the stored bytes are close to the bf16 content they were made from, so the result is close to the bf16 oracle's
    mat = wl.materialize(w)
    ro, rl = orc.attn_rows(mat.q, mat.k_pages, mat.v_pages, mat.page_table, P, w.Hkv, w.scale, rows)
    assert np.abs(base[0] - ro).max() <= 0.12 and np.abs(base[1] - rl).max() <= 0.1


def test_fp8_inputs_keep_the_logical_content():
    w = wl.small_mixed()
    m8, mat = wl.materialize_fp8(w), wl.materialize(w)
    assert np.array_equal(m8.page_table, mat.page_table) and np.array_equal(m8.q, mat.q)
    x = wl.bf16_bits_to_f64(mat.k_pages)
    back = o8.e4m3_decode(m8.k8_pages) * m8.k_scale[None, None, :, None]
    real = np.abs(x) < 10                                   # slots holding logical content (the rest is large garbage)
    assert np.abs(back - x)[real].max() <= 2.0 ** -4 * 6.0 + 1e-6
    assert (np.abs(o8.e4m3_decode(m8.k8_pages)[~real]) == 448.0).all()
