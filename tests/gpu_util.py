"""Helpers shared by the GPU parity tests: move a materialised workload to the device and run it
through the C ABI."""
import numpy as np
import torch

from paper_2609_04774_b200 import binding, build


def bits_to_bf16(a: np.ndarray, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


class DeviceWorkload:
    def __init__(self, mat):
        build.build()
        wl = mat.wl
        self.wl = wl
        self.q = bits_to_bf16(mat.q)
        self.k = bits_to_bf16(mat.k_pages)
        self.v = bits_to_bf16(mat.v_pages)
        self.page_table = torch.from_numpy(mat.page_table).cuda()
        self.cache = binding.make_cache(self.k, self.v)
        self.out = torch.full((wl.total_new, wl.Hq, wl.D), float("nan"), dtype=torch.bfloat16, device="cuda")
        self.lse = torch.full((wl.Hq, wl.total_new), float("nan"), dtype=torch.float32, device="cuda")
        nl = [r.new_len for r in wl.requests]
        cs = [r.C for r in wl.requests]
        self.ws = torch.zeros(binding.cp_workspace_bytes(nl, cs, wl.Hq), dtype=torch.uint8, device="cuda")

    def run_batch(self, ctx):
        wl = self.wl
        binding.cp_prefill_attn_batch(ctx, self.q, self.cache, self.page_table, wl.cu_new,
                                      [r.prefix_len for r in wl.requests], [r.C for r in wl.requests], wl.cu_pages,
                                      wl.Hq, wl.scale, self.out, self.lse, self.ws)
        torch.cuda.synchronize()
        ctx.poll_status()
        return bf16_to_f64(self.out), self.lse.cpu().numpy().astype(np.float64)


def compare(out, lse, ref_o, ref_lse, what=""):
    """spec tolerances: max-abs 2e-2, mean-abs 2e-3 on O; LSE within 1e-3 (relative to max(1,|ref|));
    plus a per-row relative L2 bar so that long rows with tiny outputs are really checked."""
    assert np.isfinite(out).all() and np.isfinite(lse).all(), what
    d = np.abs(out - ref_o)
    assert d.max() <= 2e-2, (what, "max-abs", d.max())
    assert d.mean() <= 2e-3, (what, "mean-abs", d.mean())
    le = np.abs(lse - ref_lse) / np.maximum(1.0, np.abs(ref_lse))
    assert le.max() <= 1e-3, (what, "lse", le.max())
    num = np.sqrt(((out - ref_o) ** 2).sum(-1))
    den = np.sqrt((ref_o ** 2).sum(-1)) + 1e-30
    assert (num / den).max() <= 2e-2, (what, "row rel-L2", (num / den).max())
    return d.max(), d.mean(), le.max(), (num / den).max()
