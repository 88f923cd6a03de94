"""Helpers shared by the GPU parity tests: move a materialised workload to the device and run it
through the C ABI."""
import numpy as np
import torch

from paper_2609_04774_b200 import binding, build


def bits_to_bf16(a: np.ndarray, device="cuda"):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(device).view(torch.bfloat16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.float().cpu().numpy().astype(np.float64)


GUARD_BYTES = 4096
GUARD_PATTERN = 0xA5


class Guarded:
    """A device tensor placed between two guard regions of a known byte pattern; check() fails if a
    kernel wrote outside the tensor."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % 256
        self.raw = torch.full((GUARD_BYTES + n + pad + GUARD_BYTES,), GUARD_PATTERN, dtype=torch.uint8, device="cuda")
        self.n = n
        self.tensor = self.raw[GUARD_BYTES:GUARD_BYTES + n].view(dtype).view(shape)
        if fill is not None:
            self.tensor.fill_(fill)

    def check(self, what):
        head, tail = self.raw[:GUARD_BYTES], self.raw[GUARD_BYTES + self.n:]
        assert bool((head == GUARD_PATTERN).all()) and bool((tail == GUARD_PATTERN).all()), "write outside " + what


class DeviceWorkload:
    def __init__(self, mat):
        build.build()
        wl = mat.wl
        self.wl = wl
        self.mat = mat
        self.q = bits_to_bf16(mat.q)
        self.k = bits_to_bf16(mat.k_pages)
        self.v = bits_to_bf16(mat.v_pages)
        self.page_table = torch.from_numpy(mat.page_table).cuda()
        self.cache = binding.make_cache(self.k, self.v)
        # outputs start as NaN (every row must be written) and sit between guard regions, as does the workspace
        self._g_out = Guarded((wl.total_new, wl.Hq, wl.D), torch.bfloat16, float("nan"))
        self._g_lse = Guarded((wl.Hq, wl.total_new), torch.float32, float("nan"))
        nl = [r.new_len for r in wl.requests]
        cs = [r.C for r in wl.requests]
        self._g_ws = Guarded((binding.cp_workspace_bytes(nl, cs, wl.Hq),), torch.uint8, 0)
        self.out, self.lse, self.ws = self._g_out.tensor, self._g_lse.tensor, self._g_ws.tensor

    def run_batch(self, ctx):
        wl = self.wl
        binding.cp_prefill_attn_batch(ctx, self.q, self.cache, self.page_table, wl.cu_new,
                                      [r.prefix_len for r in wl.requests], [r.C for r in wl.requests], wl.cu_pages,
                                      wl.Hq, wl.scale, self.out, self.lse, self.ws)
        torch.cuda.synchronize()
        ctx.poll_status()
        for g, what in ((self._g_out, "out"), (self._g_lse, "lse"), (self._g_ws, "workspace")):
            g.check(what)
        assert not bool(torch.isnan(self.out).any()) and not bool(torch.isnan(self.lse).any()), "a row was not written"
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
