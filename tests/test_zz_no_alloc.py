"""The allocation-free entry point (collected last on purpose).

Some callers of this library cannot allocate device memory at the time they need attention: an
inference engine that has already given all of HBM to its KV-cache pool, or a serving loop that must
not hit an allocating (device-synchronising) call.  `cp_prefill_attn_static` serves them from a fixed
scratch array inside the library.  Here it is called twice in a row through the C ABI, on different
shapes (the second smaller, so stale scratch contents from the first call are still there), and each
result is compared with the regular entry point's on the same inputs AND with the fp64 oracle, within the
tolerances the parity tests use; a request whose K/V is large enough for the KV-head-by-KV-head walk of the
implicit schedule is checked against the oracle on its own; then an oversized request must be refused before
anything is launched."""
import numpy as np
import pytest
import torch

from oracle import reference as orc
from paper_2609_04774_b200 import binding
from paper_2609_04774_b200 import workloads as wl
from tests.gpu_util import DeviceWorkload, bf16_to_f64, compare

pytestmark = pytest.mark.gpu


def _both(ctx, w):
    r = w.requests[0]
    dev = DeviceWorkload(wl.materialize(w))
    binding.cp_prefill_attn(ctx, dev.q, dev.cache, dev.page_table, r.prefix_len, r.new_len, r.C, w.Hq, w.scale,
                            dev.out, dev.lse, dev.ws)
    torch.cuda.synchronize()
    ctx.poll_status()
    ref_o, ref_l = dev.out.clone(), dev.lse.clone()
    out = torch.full_like(dev.out, float("nan"))
    lse = torch.full_like(dev.lse, float("nan"))
    binding.cp_prefill_attn_static(dev.q, dev.cache, dev.page_table, r.prefix_len, r.new_len, r.C, w.Hq, w.scale,
                                   out, lse)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all()), "a row was not written"
    mat = dev.mat
    oo, ol = orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, r.prefix_len, w.Hkv, w.scale)
    compare(bf16_to_f64(out), lse.cpu().numpy().astype(np.float64), oo, ol, w.name + " static vs oracle")
    return bf16_to_f64(out), lse.cpu().numpy().astype(np.float64), bf16_to_f64(ref_o), ref_l.cpu().numpy().astype(np.float64)


def test_static_entry_point_matches_regular_one_twice():
    ctx = binding.Context(0)
    try:
        for w in (wl.Workload("static_a", 31, 8, 2, [wl.Request(1500, 448, 4)]),
                  wl.Workload("static_b", 32, 8, 2, [wl.Request(200, 64, 3)]),
                  wl.Workload("static_mha", 34, 4, 4, [wl.Request(900, 320, 2)])):      # single-head units
            o, l, ro, rl = _both(ctx, w)
            assert np.isfinite(o).all() and np.isfinite(l).all()
            assert np.abs(o - ro).max() <= 2e-2 and np.abs(o - ro).mean() <= 2e-3
            assert (np.abs(l - rl) / np.maximum(1.0, np.abs(rl))).max() <= 1e-3
    finally:
        ctx.close()


@pytest.mark.parametrize("heads", [(32, 8), (24, 8)])
def test_static_entry_point_large_kv_walks_kv_head_by_kv_head(heads):
    # 8192 + 512 tokens x 8 KV heads = 35.7 MB of K/V, above the 32 MB switch: the implicit schedule then walks
    # the units KV head by KV head (even group: two heads per unit; group of 3: single-head units)
    w = wl.Workload("static_big_%d" % heads[0], 35, heads[0], heads[1], [wl.Request(512, 8192, 2)])
    mat = wl.materialize(w)
    dev = DeviceWorkload(mat)
    r = w.requests[0]
    assert r.total_len * w.Hkv * 128 * 4 > 32 << 20
    out = torch.full_like(dev.out, float("nan"))
    lse = torch.full_like(dev.lse, float("nan"))
    binding.cp_prefill_attn_static(dev.q, dev.cache, dev.page_table, r.prefix_len, r.new_len, r.C, w.Hq, w.scale, out, lse)
    torch.cuda.synchronize()
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all()), "a row was not written"
    rows = np.unique(np.concatenate([wl.sample_rows(35, 1, r.new_len, 96)[0], [0, 127, 128, 255, 256, 511]]))
    ro, rl = orc.attn_rows(mat.q, mat.k_pages, mat.v_pages, mat.page_table, r.prefix_len, w.Hkv, w.scale, rows)
    compare(bf16_to_f64(out)[rows], lse.cpu().numpy().astype(np.float64)[:, rows], ro, rl, w.name)


def test_static_entry_point_rejects_oversized_requests():
    w = wl.Workload("static_c", 33, 8, 2, [wl.Request(64, 0, 1)])
    dev = DeviceWorkload(wl.materialize(w))
    before = dev.out.clone()
    with pytest.raises(binding.CpError) as e:
        # one token more than the 2048 query tiles of the built-in tile list; refused before any launch
        binding.cp_prefill_attn_static(dev.q, dev.cache, dev.page_table, 0, 2048 * 128 + 1, 8, w.Hq, w.scale, dev.out, dev.lse)
    assert e.value.code == binding.CP_ERR_WORKSPACE
    assert "2048" in str(e.value)
    torch.cuda.synchronize()
    assert torch.equal(before.view(torch.int16), dev.out.view(torch.int16))
