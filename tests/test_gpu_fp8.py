"""GPU parity of the FP8 K/V variant, through the C ABI, against the fp64 oracle on the same stored bytes.

Bit-exact: the query codes and scales the library's pre-pass leaves in the workspace, and the bytes written by
cp_kv_append_fp8.  Attention: LSE as in the bf16 path; O element by element within the bound the format gives
for rounding the softmax weights to E4M3 (round to nearest: at most 2^-4 of each weight), 2^-4 * A with
A = sum_j p_j |v_j| (the oracle returns it), plus 2^-8 * A for the bf16 rounding of the output (|O| <= A, half an
ulp is 2^-9 of the value) and 1e-3 for the fp32 accumulation; per-row relative L2 error at most 2^-4 (expected
2^-4 / sqrt(3) * 0.75 = 0.027 for independent rounding errors)."""
import numpy as np
import pytest
import torch

from oracle import fp8 as o8
from paper_2609_04774_b200 import binding
from paper_2609_04774_b200 import workloads as wl
from tests.gpu_util import Guarded, bf16_to_f64, bits_to_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = binding.Context(0)
    yield c
    c.close()


class Device8:
    def __init__(self, m8):
        w = m8.wl
        self.w, self.m8 = w, m8
        self.q = bits_to_bf16(m8.q)
        self.k8 = torch.from_numpy(m8.k8_pages).cuda()
        self.v8 = torch.from_numpy(m8.v8_pages).cuda()
        self.ks = torch.from_numpy(m8.k_scale).cuda()
        self.vs = torch.from_numpy(m8.v_scale).cuda()
        self.page_table = torch.from_numpy(m8.page_table).cuda()
        self.cache = binding.make_cache_fp8(self.k8, self.v8, self.ks, self.vs)
        self._g_out = Guarded((w.total_new, w.Hq, w.D), torch.bfloat16, float("nan"))
        self._g_lse = Guarded((w.Hq, w.total_new), torch.float32, float("nan"))
        nl, cs = [r.new_len for r in w.requests], [r.C for r in w.requests]
        self.base_ws = binding.cp_workspace_bytes(nl, cs, w.Hq)
        self._g_ws = Guarded((binding.cp_workspace_bytes_fp8(nl, cs, w.Hq),), torch.uint8, 0)
        self.out, self.lse, self.ws = self._g_out.tensor, self._g_lse.tensor, self._g_ws.tensor

    def run(self, ctx):
        w = self.w
        binding.cp_prefill_attn_fp8_batch(ctx, self.q, self.cache, self.page_table, w.cu_new,
                                          [r.prefix_len for r in w.requests], [r.C for r in w.requests], w.cu_pages,
                                          w.Hq, w.scale, self.out, self.lse, self.ws)
        torch.cuda.synchronize()
        ctx.poll_status()
        for g, what in ((self._g_out, "out"), (self._g_lse, "lse"), (self._g_ws, "workspace")):
            g.check(what)
        assert not bool(torch.isnan(self.out).any()) and not bool(torch.isnan(self.lse).any()), "a row was not written"
        return bf16_to_f64(self.out), self.lse.cpu().numpy().astype(np.float64)

    def query_codes(self):
        """What the quantising pre-pass left behind the schedule space: codes [rows, Hq, 128], scales [rows, Hq]."""
        w = self.w
        n = w.total_new * w.Hq
        codes = self.ws[self.base_ws:self.base_ws + n * 128].cpu().numpy().reshape(w.total_new, w.Hq, 128)
        scales = self.ws[self.base_ws + n * 128:self.base_ws + n * 132].view(torch.float32).cpu().numpy().reshape(w.total_new, w.Hq)
        return codes, scales


def compare8(out, lse, ref_o, ref_l, ref_a, what):
    assert np.isfinite(out).all() and np.isfinite(lse).all(), what
    le = np.abs(lse - ref_l) / np.maximum(1.0, np.abs(ref_l))
    assert le.max() <= 1e-3, (what, "lse", le.max())
    excess = np.abs(out - ref_o) - ((2.0 ** -4 + 2.0 ** -8) * ref_a + 1e-3)
    assert excess.max() <= 0, (what, "element bound exceeded by", excess.max())
    num = np.sqrt(((out - ref_o) ** 2).sum(-1))
    den = np.sqrt((ref_o ** 2).sum(-1)) + 1e-30
    assert (num / den).max() <= 2.0 ** -4, (what, "row rel-L2", (num / den).max())
    return np.abs(out - ref_o).max(), np.abs(out - ref_o).mean(), (num / den).mean()


def check_batch8(ctx, w, rows_per_request=None, seed=7):
    m8 = wl.materialize_fp8(w)
    dev = Device8(m8)
    out, lse = dev.run(ctx)
    codes, scales = dev.query_codes()
    ref_codes, ref_scales = o8.quantize_q(m8.q)
    assert np.array_equal(scales, ref_scales), "query scales differ from the oracle's"
    assert np.array_equal(o8.e4m3_decode(codes), o8.e4m3_decode(ref_codes)), "query codes differ from the oracle's"
    stats = []
    for b, r in enumerate(w.requests):
        lo, hi = int(w.cu_new[b]), int(w.cu_new[b + 1])
        if rows_per_request is None or rows_per_request >= r.new_len:
            rows = np.arange(r.new_len)
        else:
            edges = [0, 127, 128, r.new_len - 1]
            rows = np.unique(np.clip(np.concatenate([wl.sample_rows(seed + b, 1, r.new_len, rows_per_request)[0], edges]), 0, r.new_len - 1))
        pt = m8.page_table[w.cu_pages[b]:w.cu_pages[b + 1]]
        ro, rl, ra = o8.attn_fp8_rows(m8.q[lo:hi], m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, pt, r.prefix_len,
                                      w.Hkv, w.scale, rows)
        stats.append(compare8(out[lo:hi][rows], lse[:, lo:hi][:, rows], ro, rl, ra, "%s req %d" % (w.name, b)))
    return dev, stats


@pytest.mark.parametrize("Hkv,page", [(2, 64), (1, 16), (3, 128), (16, 32)])
def test_fp8_append_matches_oracle_bit_for_bit(ctx, Hkv, page):
    w = wl.Workload("fp8_append", 51, 4 * Hkv, Hkv, [wl.Request(300, 3 * page, 1)], page=page)
    m8 = wl.materialize_fp8(w)
    dev = Device8(m8)
    r = w.requests[0]
    t0, n = 37, r.total_len - 37
    newk = wl.normal_bf16(52, wl.TID_K, (n, w.Hkv, w.D))
    newv = wl.normal_bf16(52, wl.TID_V, (n, w.Hkv, w.D))
    newk[3, 0, :8] = wl.f32_to_bf16_bits(np.array([1e4, -1e4, 0.0, 448 * m8.k_scale[0], 1e-6, -1e-6, 3e38, -3e38], dtype=np.float32))
    binding.cp_kv_append_fp8(ctx, dev.cache, dev.page_table, t0, n, bits_to_bf16(newk), bits_to_bf16(newv))
    torch.cuda.synchronize()
    ctx.poll_status()
    kc, vc = o8.quantize_kv(newk, m8.k_scale), o8.quantize_kv(newv, m8.v_scale)
    kp, vp = m8.k8_pages.copy(), m8.v8_pages.copy()
    t = np.arange(t0, t0 + n)
    kp[m8.page_table[t // page], t % page] = kc
    vp[m8.page_table[t // page], t % page] = vc
    got_k, got_v = dev.k8.cpu().numpy(), dev.v8.cpu().numpy()
    assert np.array_equal(o8.e4m3_decode(got_k), o8.e4m3_decode(kp))          # (+0 and -0 codes both stand for zero)
    assert np.array_equal(o8.e4m3_decode(got_v), o8.e4m3_decode(vp))
    assert np.array_equal(got_k & 0x7F, kp & 0x7F) and np.array_equal(got_v & 0x7F, vp & 0x7F)
    # the raw byte copies: read the stored bytes out, write them back at other tokens in two runs
    kb = torch.zeros((n, Hkv, w.D), dtype=torch.uint8, device="cuda")
    vb = torch.zeros_like(kb)
    binding.cp_kv_gather_fp8(ctx, dev.cache, dev.page_table, t0, n, kb, vb)
    torch.cuda.synchronize()
    assert np.array_equal(kb.cpu().numpy(), got_k[m8.page_table[t // page], t % page])
    assert np.array_equal(vb.cpu().numpy(), got_v[m8.page_table[t // page], t % page])
    segs = [(0, 30, 100), (t0 + 50, 41, 7)]
    binding.cp_kv_append_segments_fp8(ctx, dev.cache, dev.page_table, segs, kb, vb)
    torch.cuda.synchronize()
    ctx.poll_status()
    exp_k, exp_v = got_k.copy(), got_v.copy()
    for s0, sn, r0 in segs:
        ts = np.arange(s0, s0 + sn)
        exp_k[m8.page_table[ts // page], ts % page] = kb.cpu().numpy()[r0:r0 + sn]
        exp_v[m8.page_table[ts // page], ts % page] = vb.cpu().numpy()[r0:r0 + sn]
    assert np.array_equal(dev.k8.cpu().numpy(), exp_k) and np.array_equal(dev.v8.cpu().numpy(), exp_v)


def test_fp8_attention_small_mixed_batch(ctx):
    w = wl.Workload("fp8_small_mixed", 53, 8, 2, [wl.Request(333, 192, 3), wl.Request(5, 0, 4), wl.Request(1, 64, 1),
                                                  wl.Request(700, 0, 2), wl.Request(129, 448, 8), wl.Request(256, 1024, 4)])
    dev, stats = check_batch8(ctx, w)
    o1, l1 = dev.out.clone(), dev.lse.clone()
    dev.run(ctx)                                                               # run-to-run bitwise determinism
    assert torch.equal(o1.view(torch.int16), dev.out.view(torch.int16)) and torch.equal(l1, dev.lse)


@pytest.mark.parametrize("page", [16, 32, 128])
def test_fp8_attention_other_page_sizes_and_kv_split(ctx, page):
    reqs = [wl.Request(333, 200, 3), wl.Request(130, 30000, 2), wl.Request(64, 20000, 1)]
    check_batch8(ctx, wl.Workload("fp8_page_%d" % page, 54, 8, 2, reqs, page=page), rows_per_request=48)


def test_fp8_single_request_entry_and_validation(ctx):
    w = wl.Workload("fp8_one", 55, 16, 2, [wl.Request(517, 320, 2)])
    m8 = wl.materialize_fp8(w)
    dev = Device8(m8)
    binding.cp_prefill_attn_fp8(ctx, dev.q, dev.cache, dev.page_table, 320, 517, 2, w.Hq, w.scale, dev.out, dev.lse, dev.ws)
    torch.cuda.synchronize()
    ctx.poll_status()
    ro, rl, ra = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, 320, w.Hkv, w.scale,
                                  np.arange(517))
    compare8(bf16_to_f64(dev.out), dev.lse.cpu().numpy().astype(np.float64), ro, rl, ra, "fp8 single")
    before = dev.out.clone()
    small = torch.zeros(dev.base_ws, dtype=torch.uint8, device="cuda")      # the bf16 path's workspace is too small
    with pytest.raises(binding.CpError) as e:
        binding.cp_prefill_attn_fp8(ctx, dev.q, dev.cache, dev.page_table, 320, 517, 2, w.Hq, w.scale, dev.out, dev.lse, small)
    assert e.value.code == binding.CP_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert torch.equal(before.view(torch.int16), dev.out.view(torch.int16))


def test_fp8_attention_odd_group_sizes(ctx):
    # three query heads per KV head and plain multi-head attention: single-head units over pairs of query tiles
    check_batch8(ctx, wl.Workload("fp8_odd_group", 56, 6, 2, [wl.Request(333, 192, 3), wl.Request(129, 0, 2), wl.Request(700, 64, 1)]))
    check_batch8(ctx, wl.Workload("fp8_mha", 57, 4, 4, [wl.Request(700, 64, 4), wl.Request(90, 3000, 1)]))


def test_fp8_strided_cache_view_and_tile_pair_splits(ctx):
    # the FP8 cache as a view into a wider allocation (an unused head slot per token, an unused token row per page);
    # then single-head units with prefixes long enough for KV cuts
    w = wl.Workload("fp8_strided", 59, 8, 2, [wl.Request(300, 200, 2), wl.Request(90, 0, 1)])
    m8 = wl.materialize_fp8(w)
    dev = Device8(m8)
    npg = m8.k8_pages.shape[0]
    big_k = torch.full((npg, wl.PAGE + 1, w.Hkv + 1, w.D), 0x7E, dtype=torch.uint8, device="cuda")
    big_v = torch.full_like(big_k, 0xFE)
    big_k[:, :wl.PAGE, :w.Hkv] = dev.k8
    big_v[:, :wl.PAGE, :w.Hkv] = dev.v8
    dev.k8, dev.v8 = big_k[:, :wl.PAGE, :w.Hkv], big_v[:, :wl.PAGE, :w.Hkv]
    dev.cache = binding.make_cache_fp8(dev.k8, dev.v8, dev.ks, dev.vs)
    assert dev.cache.stride_tok == (w.Hkv + 1) * w.D and dev.cache.stride_page == (wl.PAGE + 1) * (w.Hkv + 1) * w.D
    out, lse = dev.run(ctx)
    for b, r in enumerate(w.requests):
        lo, hi = int(w.cu_new[b]), int(w.cu_new[b + 1])
        pt = m8.page_table[w.cu_pages[b]:w.cu_pages[b + 1]]
        ro, rl, ra = o8.attn_fp8_rows(m8.q[lo:hi], m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, pt, r.prefix_len, w.Hkv,
                                      w.scale, np.arange(r.new_len))
        compare8(out[lo:hi], lse[:, lo:hi], ro, rl, ra, "fp8 strided req %d" % b)
    # quantising append through the same view
    newk = wl.normal_bf16(60, wl.TID_K, (64, w.Hkv, w.D))
    binding.cp_kv_append_fp8(ctx, dev.cache, dev.page_table, 10, 64, bits_to_bf16(newk), None)
    torch.cuda.synchronize()
    ctx.poll_status()
    kc = o8.quantize_kv(newk, m8.k_scale)
    t = np.arange(10, 74)
    got = dev.k8.cpu().numpy()[m8.page_table[t // wl.PAGE], t % wl.PAGE]
    assert np.array_equal(o8.e4m3_decode(got), o8.e4m3_decode(kc))
    assert bool((big_k[:, wl.PAGE] == 0x7E).all()) and bool((big_k[:, :, w.Hkv] == 0x7E).all())     # nothing outside the view
    reqs = [wl.Request(128, 30000, 1), wl.Request(257, 5003, 3), wl.Request(1, 40001, 1)]
    check_batch8(ctx, wl.Workload("fp8_pair_split", 61, 6, 2, reqs), rows_per_request=40)


def test_fp8_shard_chunk_and_key_range_calls(ctx):
    # one request through the three partial forms of the variant: the C shard partials and a set of key-range
    # partials each merge (cp_merge) into the oracle's full result; every chunk call reproduces its rows
    from oracle import reference as orc
    w = wl.Workload("fp8_partials", 58, 8, 2, [wl.Request(700, 320, 3)])
    m8 = wl.materialize_fp8(w)
    dev = Device8(m8)
    r = w.requests[0]
    R, P, C = r.new_len, r.prefix_len, r.C
    ro, rl, ra = o8.attn_fp8_rows(m8.q, m8.k8_pages, m8.v8_pages, m8.k_scale, m8.v_scale, m8.page_table, P, w.Hkv, w.scale,
                                  np.arange(R))
    plan = orc.plan(R, P, C)
    parts = torch.full((C, R, w.Hq, w.D), float("nan"), dtype=torch.float32, device="cuda")
    lses = torch.full((C, w.Hq, R), float("nan"), dtype=torch.float32, device="cuda")
    for k in range(C):
        binding.cp_prefill_attn_fp8_shard(ctx, dev.q, dev.cache, dev.page_table, P, R, C, k, w.Hq, w.scale, parts[k], lses[k], dev.ws)
    torch.cuda.synchronize()
    ctx.poll_status()
    for k in range(C):
        own = np.zeros(R, dtype=bool)
        own[orc.shard_rows(plan[k])] = True
        lk = lses[k].cpu().numpy()
        assert np.isfinite(lk[:, own]).all() and np.isneginf(lk[:, ~own]).all() and (parts[k].cpu().numpy()[~own] == 0).all()
    merged = torch.empty((R, w.Hq, w.D), dtype=torch.float32, device="cuda")
    mlse = torch.empty((w.Hq, R), dtype=torch.float32, device="cuda")
    binding.cp_merge(ctx, parts, lses, merged, mlse)
    torch.cuda.synchronize()
    compare8(merged.cpu().numpy().astype(np.float64), mlse.cpu().numpy().astype(np.float64), ro, rl, ra, "fp8 merged shards")
    edges = [0, 130, 320, 577, P + R]
    kparts = torch.empty((len(edges) - 1, R, w.Hq, w.D), dtype=torch.float32, device="cuda")
    klses = torch.empty((len(edges) - 1, w.Hq, R), dtype=torch.float32, device="cuda")
    for n, (lo, hi) in enumerate(zip(edges, edges[1:])):
        binding.cp_prefill_attn_fp8_kvrange(ctx, dev.q, dev.cache, dev.page_table, P, R, lo, hi, w.Hq, w.scale, kparts[n], klses[n], dev.ws)
    binding.cp_merge(ctx, kparts, klses, merged, mlse)
    torch.cuda.synchronize()
    ctx.poll_status()
    compare8(merged.cpu().numpy().astype(np.float64), mlse.cpu().numpy().astype(np.float64), ro, rl, ra, "fp8 merged key ranges")
    for j in range(2 * C):
        b, e = (plan[j]["q_begin"][0], plan[j]["q_end"][0]) if j < C else (plan[2 * C - 1 - j]["q_begin"][1], plan[2 * C - 1 - j]["q_end"][1])
        out = torch.full((e - b, w.Hq, w.D), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((w.Hq, e - b), float("nan"), dtype=torch.float32, device="cuda")
        binding.cp_prefill_attn_fp8_chunk(ctx, dev.q[b:e].contiguous(), dev.cache, dev.page_table, P, R, C, j, w.Hq, w.scale, out, lse, dev.ws)
        torch.cuda.synchronize()
        ctx.poll_status()
        compare8(bf16_to_f64(out), lse.cpu().numpy().astype(np.float64), ro[b:e], rl[:, b:e], ra[b:e], "fp8 chunk %d" % j)


def _random_workload8(seed):
    u = wl.counter_uniform(seed, wl.TID_LEN, 0, 64)
    heads = [(8, 2), (4, 4), (6, 2), (16, 2), (32, 4), (8, 8), (2, 1)][int(u[0] * 7)]
    page = [16, 32, 64, 128][int(u[1] * 4)]
    reqs = []
    for b in range(1 + int(u[2] * 5)):
        R = max(1, int(round(2.0 ** (u[3 + 4 * b] * 10.5))))                  # 1 .. ~1450, log-uniform
        kind = u[4 + 4 * b]
        P = 0 if kind < 0.25 else int(u[5 + 4 * b] * 6000)
        if kind < 0.75:
            P = P // page * page
        reqs.append(wl.Request(R, P, [1, 2, 3, 4, 5, 8][int(u[6 + 4 * b] * 6)]))
    return wl.Workload("fp8_random_%d" % seed, seed, heads[0], heads[1], reqs, page=page)


@pytest.mark.parametrize("seed", range(3000, 3008))
def test_fp8_attention_random_batches(ctx, seed):
    # seeded random batches: even, odd and unit group sizes, all page sizes, ragged lengths from one token up
    check_batch8(ctx, _random_workload8(seed), rows_per_request=64, seed=seed)


def test_fp8_attention_config2_shape_sampled(ctx):
    check_batch8(ctx, wl.config2(), rows_per_request=96)


def test_fp8_attention_config5_shape_sampled(ctx):
    check_batch8(ctx, wl.config5(), rows_per_request=24)


@pytest.mark.parametrize("scale", [0.5, 2.0])
def test_fp8_attention_peaked_scores_exercise_the_rescale_path(ctx, scale):
    # a large softmax scale makes new row maxima arrive in later key tiles, so the rescale of O and of the running sum
    # (threshold 2^4 in this variant, weights scaled by 16 and saturating at 448) really runs
    w = wl.Workload("fp8_peaked_%g" % scale, 79, 8, 2, [wl.Request(600, 1280, 2), wl.Request(260, 0, 1)], meta={"scale": scale})
    check_batch8(ctx, w)
