#!/usr/bin/env python
"""Benchmark of libcpattn's hot path: cache-aware causal prefill attention under zigzag CP.

Default mode prints ONE JSON line.  Its headline (`value`, `roofline`, `e2e`) is configuration 2
(Llama-3-8B-shaped layer, 12288 cached + 4096 new tokens, C=4, paged KV).  A step is one pass of the hot
path over the batch: cp_plan (host) -> varlen tile schedule (host; small work lists ride in the launch
parameters, large ones are uploaded by a copy kernel) -> one persistent attention launch over all C shards
reading K/V through the page table and storing rows at their original positions -> LSE merge of the units
whose KV range was split across CTAs.  `value` is measured with inputs resident in HBM; `e2e` goes through
the same C-ABI calls from pinned HOST buffers (q, the new tokens' K/V rows appended into the paged cache,
page table up; out and lse down).  At one GPU the same line also carries: `sustained` (the headline
workload repeated for at least two seconds of GPU time, clocks sampled), `configs` (configurations 1-5,
each with its own clocks), `merge` (cp_merge bandwidth points), `kvcopy` (paged copy bandwidth), `cp_rank` (local
time of the slowest rank of a degree-4 worker on configuration 2, call by call and from a CUDA graph) and the
`cpu_baseline` legs (the fp64 oracle on the host cores), plus `prefill_time_table`, a corner of the measured
t(new_len, prefix_len, C) table (the whole table: `--mode table`).

Other modes (`--mode merge|table|configs|kvcopy|cprank|cachemgr|cpu`) write the cp_merge sweep, the measured
prefill-time table over (new_len, prefix_len, C), the per-config numbers, the paged KV copy bandwidth, one CP rank's
local time, the cache-manager throughput and the oracle's full passes over whole configurations as JSON lines to
`--out`.

`--impl reference` times the CPU fp64 oracle (host cores) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2609_04774_b200 import workloads as wl  # noqa: E402

METRIC = "causal_effective_prefill_attention_tflops"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
# Secondary roofline of softmax attention at D = 128: one exponential per visible (query, key) pair and head, i.e.
# per 512 causal-effective flops.  The MUFU pipe delivers 16 ex2 results per clock per SM (measured: fp32 and packed
# 16-bit forms alike), so at the 1965 MHz maximum clock 148 SMs sustain at most 148 * 16 * 512 * 1.965e9 flop/s
# worth of attention, whatever the operand precision of the two matrix products.
MUFU_ROOFLINE_TFLOPS = 148 * 16 * 512 * 1.965e9 / 1e12
# dram__bytes_read.sum + dram__bytes_write.sum of one cp_attn_kernel launch, from the ncu captures
# summarised in profiles/ (per workload name; a workload without a capture reports null)
ATTN_TRAFFIC_BYTES = {"cfg2_R4096_P12288_C4": 121_965_056, "cfg3_R131072_P0_C8": 7_200_575_488}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def get_workload(cfg: int) -> wl.Workload:
    return (wl.CONFIGS.get(cfg) or wl.VARIANTS[cfg])()


def pairs_of(w: wl.Workload) -> int:
    """Visible (query, key) pairs: the remaining attention workload W(R,P) = R*P + R(R+1)/2 of Eq. (1), summed over
    the requests of the batch."""
    return sum(r.new_len * r.prefix_len + r.new_len * (r.new_len + 1) // 2 for r in w.requests)


def flops_of(w: wl.Workload) -> int:
    """Causal-effective flops: 4*D per visible pair per query head (masked halves of diagonal tiles do not count)."""
    return 4 * w.D * w.Hq * pairs_of(w)


def algorithmic_bytes(w: wl.Workload) -> int:
    """Q and O once, K and V once, LSE (bf16 tensors, fp32 LSE)."""
    return 2 * w.total_new * w.Hq * w.D * 2 + 2 * sum(r.total_len for r in w.requests) * w.Hkv * w.D * 2 + 4 * w.Hq * w.total_new


# ----------------------------------------------------------------------------------------------
# clocks sampling during the timed region
# ----------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "power_w_median": None, "power_w_max": None}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    smax.append(float(f[2]))
                except ValueError:
                    continue
                try:
                    power.append(float(f[3]))
                except ValueError:
                    pass
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm))
        if power:
            out.update(power_w_median=statistics.median(power), power_w_max=max(power))
        return out


# ----------------------------------------------------------------------------------------------
# device-side runner
# ----------------------------------------------------------------------------------------------
class Runner:
    """Holds device copies of one workload and runs steps through the C ABI."""

    def __init__(self, w: wl.Workload, device: int, need_host: bool = False, fp8: bool = False):
        import torch
        from paper_2609_04774_b200 import binding, build
        build.build()
        self.torch, self.binding, self.w, self.fp8 = torch, binding, w, fp8
        torch.cuda.set_device(device)
        self.ctx = binding.Context(device)
        mat = wl.materialize_fp8(w) if fp8 else wl.materialize(w)
        self.mat = mat

        def dev(bits):
            return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

        self.q = dev(mat.q)
        self.page_table = torch.from_numpy(mat.page_table).cuda()
        if fp8:      # E4M3 pages with one fp32 scale per KV head
            self.k, self.v = torch.from_numpy(mat.k8_pages).cuda(), torch.from_numpy(mat.v8_pages).cuda()
            self.k_scale, self.v_scale = torch.from_numpy(mat.k_scale).cuda(), torch.from_numpy(mat.v_scale).cuda()
            self.cache = binding.make_cache_fp8(self.k, self.v, self.k_scale, self.v_scale)
        else:
            self.k, self.v = dev(mat.k_pages), dev(mat.v_pages)
            self.cache = binding.make_cache(self.k, self.v)
        self.out = torch.empty((w.total_new, w.Hq, w.D), dtype=torch.bfloat16, device="cuda")
        self.lse = torch.empty((w.Hq, w.total_new), dtype=torch.float32, device="cuda")
        self.new_len = [r.new_len for r in w.requests]
        self.prefix = np.array([r.prefix_len for r in w.requests], dtype=np.int64)
        self.Cs = np.array([r.C for r in w.requests], dtype=np.int32)
        ws_bytes = (binding.cp_workspace_bytes_fp8 if fp8 else binding.cp_workspace_bytes)(self.new_len, self.Cs, w.Hq)
        self.ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
        self.cu_new, self.cu_pages = w.cu_new, w.cu_pages
        if need_host:
            self._host_buffers()

    def _host_buffers(self):
        """Pinned host copies of one step's inputs: q, the new tokens' K/V rows, the page table."""
        torch, w, mat = self.torch, self.w, self.mat
        self.h_q = torch.from_numpy(mat.q.view(np.int16)).view(torch.bfloat16).pin_memory()
        newk, newv = [], []
        for b, r in enumerate(w.requests):
            pt = mat.page_table[w.cu_pages[b]:w.cu_pages[b + 1]]
            idx = np.arange(r.prefix_len, r.total_len)
            newk.append(mat.k_pages[pt[idx // wl.PAGE], idx % wl.PAGE])
            newv.append(mat.v_pages[pt[idx // wl.PAGE], idx % wl.PAGE])
        self.h_newk = torch.from_numpy(np.concatenate(newk).view(np.int16)).view(torch.bfloat16).pin_memory()
        self.h_newv = torch.from_numpy(np.concatenate(newv).view(np.int16)).view(torch.bfloat16).pin_memory()
        self.h_pt = torch.from_numpy(mat.page_table).pin_memory()
        self.d_newk = torch.empty_like(self.h_newk, device="cuda")
        self.d_newv = torch.empty_like(self.h_newv, device="cuda")
        self.h_out = torch.empty(self.out.shape, dtype=torch.bfloat16).pin_memory()
        self.h_lse = torch.empty(self.lse.shape, dtype=torch.float32).pin_memory()
        self.h2d_bytes = sum(t.numel() * t.element_size() for t in (self.h_q, self.h_newk, self.h_newv, self.h_pt))
        self.d2h_bytes = sum(t.numel() * t.element_size() for t in (self.h_out, self.h_lse))
        # one pinned block per direction (256-byte aligned parts): a step's inputs go up in ONE copy, its results
        # come down in ONE copy, instead of four and two
        def packed(tensors):
            offs, total = [], 0
            for t in tensors:
                offs.append(total)
                total += -(-t.numel() * t.element_size() // 256) * 256
            return offs, total
        self.in_offs, in_total = packed((self.h_q, self.h_newk, self.h_newv, self.h_pt))
        self.h_in = torch.empty(in_total, dtype=torch.uint8).pin_memory()
        for off, t in zip(self.in_offs, (self.h_q, self.h_newk, self.h_newv, self.h_pt)):
            self.h_in[off:off + t.numel() * t.element_size()].copy_(t.contiguous().view(-1).view(torch.uint8))
        self.out_offs, out_total = packed((self.h_out, self.h_lse))
        self.h_outbuf = torch.empty(out_total, dtype=torch.uint8).pin_memory()

    def step(self):
        """One pass of the hot path with device-resident inputs: plan + schedule + attention launch."""
        b, w = self.binding, self.w
        for r in w.requests:
            b.cp_plan(r.new_len, r.prefix_len, r.C)
        call = b.cp_prefill_attn_fp8_batch if self.fp8 else b.cp_prefill_attn_batch
        call(self.ctx, self.q, self.cache, self.page_table, self.cu_new, self.prefix, self.Cs, self.cu_pages, w.Hq, w.scale,
             self.out, self.lse, self.ws)

    def _e2e_setup(self):
        """Streams and double-buffered device staging for the end-to-end leg."""
        torch = self.torch
        self.s_in, self.s_c, self.s_out = (torch.cuda.Stream() for _ in range(3))
        def view(buf, off, like):
            n = like.numel() * like.element_size()
            return buf[off:off + n].view(like.dtype).view(like.shape)
        self.e_in = [torch.empty(self.h_in.numel(), dtype=torch.uint8, device="cuda") for _ in range(2)]
        self.e_q = [view(b, self.in_offs[0], self.h_q) for b in self.e_in]
        self.e_k = [view(b, self.in_offs[1], self.h_newk) for b in self.e_in]
        self.e_v = [view(b, self.in_offs[2], self.h_newv) for b in self.e_in]
        self.e_pt = [view(b, self.in_offs[3], self.h_pt) for b in self.e_in]
        self.e_outbuf = [torch.empty(self.h_outbuf.numel(), dtype=torch.uint8, device="cuda") for _ in range(2)]
        self.e_out = [view(b, self.out_offs[0], self.h_out) for b in self.e_outbuf]
        self.e_lse = [view(b, self.out_offs[1], self.h_lse) for b in self.e_outbuf]
        self.ev_in = [torch.cuda.Event() for _ in range(2)]
        self.ev_c = [torch.cuda.Event() for _ in range(2)]
        self.ev_out = [torch.cuda.Event() for _ in range(2)]
        self.e2e_k = 0
        for e in self.ev_c + self.ev_out:
            e.record()

    def step_e2e(self):
        """The same pass from pinned host buffers through the public calls, pipelined over three streams the way
        a serving loop would: step k's inputs (q, the new tokens' K/V rows, the page table) go up while step k-1
        computes (cp_kv_append through the page table, then attention) and step k-2's out / lse come down.
        Every step moves all of its own bytes inside the timed region."""
        torch, b, w = self.torch, self.binding, self.w
        if not hasattr(self, "s_in"):
            self._e2e_setup()
        i = self.e2e_k % 2
        self.e2e_k += 1
        with torch.cuda.stream(self.s_in):
            self.s_in.wait_event(self.ev_c[i])                 # staging buffers i were last read by step k-2
            self.e_in[i].copy_(self.h_in, non_blocking=True)       # q, new K rows, new V rows, page table
            self.ev_in[i].record()
        with torch.cuda.stream(self.s_c):
            self.s_c.wait_event(self.ev_in[i])
            self.s_c.wait_event(self.ev_out[i])                # out / lse buffers i were copied out by step k-2
            row0 = 0
            for j, r in enumerate(w.requests):
                b.cp_plan(r.new_len, r.prefix_len, r.C)
                pt = self.e_pt[i][int(self.cu_pages[j]):int(self.cu_pages[j + 1])]
                b.cp_kv_append(self.ctx, self.cache, pt, r.prefix_len, r.new_len, self.e_k[i][row0:row0 + r.new_len],
                               self.e_v[i][row0:row0 + r.new_len], stream=self.s_c)
                row0 += r.new_len
            b.cp_prefill_attn_batch(self.ctx, self.e_q[i], self.cache, self.e_pt[i], self.cu_new, self.prefix, self.Cs,
                                    self.cu_pages, w.Hq, w.scale, self.e_out[i], self.e_lse[i], self.ws, stream=self.s_c)
            self.ev_c[i].record()
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_c[i])
            self.h_outbuf.copy_(self.e_outbuf[i], non_blocking=True)     # out and lse
            self.ev_out[i].record()
        torch.cuda.current_stream().wait_event(self.ev_out[i])   # the timing events sit on the current stream

    def launches_per_step(self, e2e=False):
        """Kernels of this library per step, as the library's own schedule reports them: list copy (unless the
        work lists ride in the launch parameters) + attention + LSE fix-up when units were split."""
        info, _, _ = self.binding.cp_schedule_inspect(self.cu_new, self.prefix, self.Cs, self.w.Hq, self.w.Hkv,
                                                      self.torch.cuda.get_device_properties(0).multi_processor_count,
                                                      want_lists=False)
        self.schedule = info
        return info["launches"] + (len(self.w.requests) if e2e else 0) + (1 if self.fp8 else 0)   # + the query quantiser

    def close(self):
        self.ctx.close()


def max_over_ranks(torch, dist, values, device):
    """MAX all-reduce of a list of per-rank timings (no-op without a process group)."""
    if dist is None:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def whole_job_value(world, flops_per_rank, ms_per_step):
    """Aggregate over all ranks: every rank runs its own replica of the workload (weak scaling), the job
    is as slow as its slowest rank."""
    return world * flops_per_rank / (ms_per_step * 1e-3) / 1e12


def timed_loop(torch, fn, steps, warmup, dist=None, stride=1):
    """W warm-up steps, then exactly `steps` steps between CUDA events; returns total ms and the list of per-step ms
    (an event after every `stride` steps: for steps of a few tens of microseconds an event per step would be a
    visible share of what is measured)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        torch.cuda.synchronize()
    marks = list(range(0, steps, stride)) + [steps]
    evs = [torch.cuda.Event(enable_timing=True) for _ in marks]
    evs[0].record()
    k = 1
    for i in range(steps):
        fn()
        if i + 1 == marks[k]:
            evs[k].record()
            k += 1
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
        torch.cuda.synchronize()
    per = [evs[i].elapsed_time(evs[i + 1]) / (marks[i + 1] - marks[i]) for i in range(len(marks) - 1)]
    return evs[0].elapsed_time(evs[-1]), per


def kernel_only_ms(torch, runner, steps):
    """Average duration of one step's launches: events recorded directly around each call on the launching
    stream, after the loop above has warmed everything up."""
    w, b = runner.w, runner.binding
    ds = []
    for _ in range(steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        b.cp_prefill_attn_batch(runner.ctx, runner.q, runner.cache, runner.page_table, runner.cu_new, runner.prefix,
                                runner.Cs, runner.cu_pages, w.Hq, w.scale, runner.out, runner.lse, runner.ws)
        e1.record()
        ds.append((e0, e1))
    torch.cuda.synchronize()
    return statistics.mean(a.elapsed_time(c) for a, c in ds)


def fractions(tflops, peaks):
    return {"of_nominal_2250": tflops / NOMINAL_BF16_TFLOPS, "of_measured_burst": tflops / peaks["bf16_tflops"],
            "of_measured_sustained": tflops / peaks["bf16_tflops_sustained"]}


def sustained_leg(torch, runner, peaks, device, seconds=2.2):
    """The headline workload back to back for at least `seconds` of GPU time (long enough for the board to reach
    its power-capped clocks), with the clocks sampled during the loop."""
    for _ in range(5):
        runner.step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(20):
        runner.step()
    e1.record()
    torch.cuda.synchronize()
    steps = max(50, int(seconds * 1e3 / max(e0.elapsed_time(e1) / 20, 1e-3)) + 1)
    sampler = ClockSampler(device)
    sampler.start()
    time.sleep(0.3)                     # the sampler's first sample
    total_ms, _ = timed_loop(torch, runner.step, steps, 3)
    clocks = sampler.stop()
    ms = total_ms / steps
    tf = flops_of(runner.w) / (ms * 1e-3) / 1e12
    return {"workload": runner.w.name, "steps": steps, "gpu_seconds": total_ms * 1e-3, "ms_per_step": ms, "tflops": tf,
            "sm_mhz_median": clocks["sm_mhz"], "ms_x_mhz": ms * clocks["sm_mhz"] if clocks["sm_mhz"] else None,
            "power_w_median": clocks["power_w_median"],
            "frac": fractions(tf, peaks), "clocks": clocks}


def config_leg(torch, cfg, peaks, device, budget_ms=1200.0, fp8=False, page=None):
    """One configuration: 3 warm-up steps, then steps for about `budget_ms` of GPU time (at least 5), clocks sampled.
    fp8: the same lengths and heads with E4M3 K/V pages (queries quantised per step by the library's pre-pass)."""
    w = get_workload(cfg)
    if page:
        w.page = page                   # tokens per cache page (16, 32, 64 or 128) instead of the configurations' 64
    runner = Runner(w, device, fp8=fp8)
    sampler = ClockSampler(device)
    sampler.start()
    for _ in range(3):
        runner.step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    runner.step()
    e1.record()
    torch.cuda.synchronize()
    one = max(e0.elapsed_time(e1), 1e-3)
    steps = int(max(5, min(2000, budget_ms / one)))
    total_ms, per = timed_loop(torch, runner.step, steps, 0, stride=16 if one < 0.2 else 1)
    clocks = sampler.stop()
    runner.ctx.poll_status()
    ms = total_ms / steps
    tf = flops_of(w) / (ms * 1e-3) / 1e12
    entry = {"config": cfg, "workload": w.name, "page_tokens": w.page, "steps": steps, "ms": ms, "ms_best": min(per), "tflops": tf,
             "tokens_per_s": w.total_new / (ms * 1e-3), "frac": fractions(tf, peaks), "pairs": pairs_of(w),
             "launches_per_step": runner.launches_per_step(), "gpu_seconds": total_ms * 1e-3, "clocks": clocks,
             "traffic": ATTN_TRAFFIC_BYTES.get(w.name), "algorithmic_bytes": algorithmic_bytes(w),
             "frac_of_mufu_roofline_%d" % round(MUFU_ROOFLINE_TFLOPS): tf / MUFU_ROOFLINE_TFLOPS}
    if fp8:
        # tensor roofline of one-byte operands: the measured bf16 rates times the nominal fp8 / bf16 ratio of 2
        entry.update(dtype="fp8_e4m3 K/V and P, bf16 q/out", traffic=None,
                     algorithmic_bytes=2 * w.total_new * w.Hq * w.D * 2 + 2 * sum(r.total_len for r in w.requests) * w.Hkv * w.D + 4 * w.Hq * w.total_new,
                     frac={"of_nominal_4500": tf / (2 * NOMINAL_BF16_TFLOPS), "of_2x_measured_bf16_burst": tf / (2 * peaks["bf16_tflops"]),
                           "of_2x_measured_bf16_sustained": tf / (2 * peaks["bf16_tflops_sustained"]),
                           "of_nominal_bf16_2250": tf / NOMINAL_BF16_TFLOPS},
                     roofline={"bound": "alu", "achieved": tf, "peak": MUFU_ROOFLINE_TFLOPS, "unit": "TFLOP/s",
                               "frac": tf / MUFU_ROOFLINE_TFLOPS,
                               "note": "with one-byte operands the tensor pipe is 38 % busy and the exponentials bound the loop: "
                                       "16 ex2/clk/SM x 148 SMs x 1965 MHz x 512 flops per exponential"})
    runner.close()
    del runner
    torch.cuda.empty_cache()
    return entry


def merge_points(torch, peaks, points, reps=10):
    """cp_merge bandwidth at (T, N, out dtype) points: H = 64, D = 128, partials N(0,1), lses N(8, 2^2) with every
    16th row of partial 0 at -inf; L2 flushed between repetitions when the operands are small."""
    from paper_2609_04774_b200 import binding
    ctx = binding.Context(torch.cuda.current_device())
    H, D = 64, 128
    g = torch.Generator(device="cuda").manual_seed(6)
    out = []
    # one allocation for all points (views per point): freeing and re-allocating multi-GB operands between points
    # leaves the first launches on fresh mappings up to 25 % slower, which is the allocator's doing, not the kernel's
    big_parts = torch.randn(max(N * T for T, N, _ in points) * H * D, dtype=torch.float32, device="cuda", generator=g)
    big_lses = 8 + 2 * torch.randn(max(N * T for T, N, _ in points) * H, dtype=torch.float32, device="cuda", generator=g)
    big_out = torch.empty(max(T for T, _, _ in points) * H * D, dtype=torch.float32, device="cuda")
    big_lo = torch.empty(max(T for T, _, _ in points) * H, dtype=torch.float32, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for T, N, dt in points:
        in_bytes = N * T * H * (D * 4 + 4)
        out_bytes = T * H * (D * dt.itemsize) + 4 * T * H
        parts = big_parts[:N * T * H * D].view(N, T, H, D)
        lses = big_lses[:N * H * T].view(N, H, T)
        lses[0].view(-1)[::16] = float("-inf")
        o = (big_out.view(torch.bfloat16) if dt == torch.bfloat16 else big_out)[:T * H * D].view(T, H, D)
        lo = big_lo[:H * T].view(H, T)
        do_flush = in_bytes < 512e6
        ds = []
        for i in range(3 + reps):
            if do_flush:
                flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            binding.cp_merge(ctx, parts, lses, o, lo)
            e1.record()
            if i >= 3:
                ds.append((e0, e1))
        torch.cuda.synchronize()
        ms = [a.elapsed_time(b) for a, b in ds]
        med = statistics.median(ms)
        gbs = (in_bytes + out_bytes) / (med * 1e-3) / 1e9
        out.append({"T": T, "N": N, "H": H, "out": str(dt).split(".")[-1], "bytes": in_bytes + out_bytes, "ms_median": med,
                    "ms_best": min(ms), "GBps": gbs, "frac_nominal_8000": gbs / NOMINAL_HBM_GBS,
                    "frac_measured_copy": gbs / peaks["hbm_gbs"], "l2_flush": do_flush})
    del big_parts, big_lses, big_out, big_lo, flush
    torch.cuda.empty_cache()
    ctx.close()
    return out


def kvcopy_points(torch, peaks, tokens=(1048576,)):
    """cp_kv_gather / cp_kv_append bandwidth: n tokens x 8 KV heads x 128 dims, K and V, shuffled pages."""
    from paper_2609_04774_b200 import binding
    ctx = binding.Context(torch.cuda.current_device())
    Hkv, D = 8, 128
    out = []
    for n in tokens:
        pages = n // wl.PAGE
        k = torch.randn((pages, wl.PAGE, Hkv, D), device="cuda").to(torch.bfloat16)
        v = torch.randn((pages, wl.PAGE, Hkv, D), device="cuda").to(torch.bfloat16)
        pt = torch.from_numpy(wl.permutation(9, wl.TID_PERM, pages)).cuda()
        cache = binding.make_cache(k, v)
        kr = torch.empty((n, Hkv, D), dtype=torch.bfloat16, device="cuda")
        vr = torch.empty_like(kr)
        moved = 2 * 2 * n * Hkv * D * 2 + 4 * pages          # K and V, read + written, plus the table
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda") if moved < 512e6 else None
        for name, fn in (("gather", lambda: binding.cp_kv_gather(ctx, cache, pt, 0, n, kr, vr)),
                         ("append", lambda: binding.cp_kv_append(ctx, cache, pt, 0, n, kr, vr))):
            ds = []
            for i in range(13):
                if flush is not None:
                    flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                if i >= 3:
                    ds.append((e0, e1))
            torch.cuda.synchronize()
            ctx.poll_status()
            ms = statistics.median(a.elapsed_time(b) for a, b in ds)
            gbs = moved / (ms * 1e-3) / 1e9
            out.append({"op": name, "tokens": n, "bytes": moved, "ms_median": ms, "GBps": gbs,
                        "frac_nominal_8000": gbs / NOMINAL_HBM_GBS, "frac_measured_copy": gbs / peaks["hbm_gbs"],
                        "l2_flush": flush is not None})
        del k, v, kr, vr, flush
        torch.cuda.empty_cache()
    ctx.close()
    return out


# ----------------------------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------------------------
def oracle_sample(w: wl.Workload, mat, rows_per_request: int, seed: int, threads=None):
    """Time the oracle on `rows_per_request` seeded rows (all heads) of every request; returns
    (seconds, visible pairs evaluated per query head summed over heads, threads used)."""
    from oracle import reference as orc
    threads = threads or orc.host_threads()
    pairs = 0
    t0 = time.perf_counter()
    for b, r in enumerate(w.requests):
        n = min(rows_per_request, r.new_len)
        rows = np.unique(wl.sample_rows(seed + b, 1, r.new_len, n)[0])
        q = mat.q[w.cu_new[b]:w.cu_new[b + 1]]
        pt = mat.page_table[w.cu_pages[b]:w.cu_pages[b + 1]]
        orc.attn_rows(q, mat.k_pages, mat.v_pages, pt, r.prefix_len, w.Hkv, w.scale, rows, n_threads=threads)
        pairs += int((r.prefix_len + rows + 1).sum()) * w.Hq
    return time.perf_counter() - t0, pairs, threads


def cpu_model():
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def cpu_baseline_legs(headline, headline_mat, args):
    """The oracle as it stands on the host cores, bounded to about half a minute in total: the headline
    configuration on a seeded row sample (the `value` of the object), configuration 1 in full with one thread and
    with all cores, the other configurations on small row samples with the full-workload time extrapolated by
    pairs (labelled), and the merge oracle on small T scaled linearly in T."""
    from oracle import reference as orc
    orc.build()
    t, pairs, threads = oracle_sample(headline, headline_mat, args.cpu_rows, 4242)
    tf = 4 * headline.D * pairs / t / 1e12
    base = {"value": tf, "unit": UNIT, "cores": threads, "kind": "oracle",
            "sample": "%s: %d seeded rows x %d heads (%.1f s); full pass extrapolated by pairs: %.0f s" %
                      (headline.name, args.cpu_rows, headline.Hq, t, flops_of(headline) / (tf * 1e12)),
            "cpu_model": cpu_model(), "nproc": os.cpu_count(), "threads": threads}
    per = []
    rows_for = {1: None, 2: None, 3: 48, 4: 6, 5: 40}
    for cfg in (1, 3, 4, 5):
        w = get_workload(cfg)
        mat = wl.materialize(w)
        if cfg == 1:
            entry = {"config": cfg, "workload": w.name, "mode": "full"}
            for label, th in (("threads_1", 1), ("threads_all", threads)):
                r = w.requests[0]
                t0 = time.perf_counter()
                orc.attn_full(mat.q, mat.k_pages, mat.v_pages, mat.page_table, r.prefix_len, w.Hkv, w.scale, n_threads=th)
                dt = time.perf_counter() - t0
                entry[label] = {"seconds": dt, "gflops_equivalent": flops_of(w) / dt / 1e9, "tokens_per_s": w.total_new / dt}
        else:
            t, pairs, _ = oracle_sample(w, mat, rows_for[cfg], 4300 + cfg)
            rate = 4 * w.D * pairs / t
            entry = {"config": cfg, "workload": w.name, "mode": "sampled", "rows_per_request": rows_for[cfg],
                     "sample_seconds": t, "pairs_per_s": pairs / t, "gflops_equivalent": rate / 1e9,
                     "full_seconds_extrapolated": flops_of(w) / rate, "tokens_per_s_extrapolated": w.total_new * rate / flops_of(w)}
        per.append(entry)
        del mat
    base["per_config"] = per
    merges = []
    for N, T in ((2, 2048), (4, 1024), (8, 512)):
        parts, lses = wl.merge_inputs(6, N, T, 64)
        t0 = time.perf_counter()
        orc.merge(parts, lses)
        dt = time.perf_counter() - t0
        nbytes = N * T * 64 * 516 + T * 64 * 260
        merges.append({"N": N, "T_timed": T, "seconds": dt, "GBps_equivalent": nbytes / dt / 1e9,
                       "seconds_at_T4096_scaled": dt * 4096 / T})
    base["merge_oracle"] = merges
    return base


def run_cpu_full(args, out):
    """The oracle as it stands over WHOLE configurations (every row, every head) on the host cores: what the bounded
    `cpu_baseline` legs extrapolate to.  Minutes of CPU time for the larger configurations; no GPU is used."""
    from oracle import reference as orc
    orc.build()
    threads = orc.host_threads()
    for cfg in args.configs:
        w = get_workload(cfg)
        mat = wl.materialize(w)
        t0 = time.perf_counter()
        for b, r in enumerate(w.requests):
            q = mat.q[w.cu_new[b]:w.cu_new[b + 1]]
            pt = mat.page_table[w.cu_pages[b]:w.cu_pages[b + 1]]
            orc.attn_full(q, mat.k_pages, mat.v_pages, pt, r.prefix_len, w.Hkv, w.scale, n_threads=threads)
        dt = time.perf_counter() - t0
        out.write(json.dumps({"mode": "cpu_full", "config": cfg, "workload": w.name, "threads": threads, "nproc": os.cpu_count(),
                              "cpu_model": cpu_model(), "seconds": dt, "gflops_equivalent": flops_of(w) / dt / 1e9,
                              "tokens_per_s": w.total_new / dt, "pairs": pairs_of(w)}) + "\n")
        out.flush()


def run_reference(args):
    """`--impl reference`: the CPU oracle as it stands, one bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import reference as orc
    orc.build()
    w = get_workload(args.config)
    mat = wl.materialize(w)
    rows = args.ref_rows
    for i in range(args.warmup):
        oracle_sample(w, mat, rows, 1000 + i)
    tot_t, tot_pairs, threads = 0.0, 0, orc.host_threads()
    for i in range(args.steps):
        t, p, threads = oracle_sample(w, mat, rows, 2000 + i)
        tot_t += t
        tot_pairs += p
    value = 4 * w.D * tot_pairs / tot_t / 1e12
    sample = "%d seeded rows x %d heads per request per step (%d steps)" % (rows, w.Hq, args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / max(args.steps, 1), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "Hq": w.Hq, "Hkv": w.Hkv, "D": w.D, "seed": w.seed},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------
# main (ours)
# ----------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(local)
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist = dist_mod
        # one rank compiles (if the library is stale at all), the others wait and then only load it
        from paper_2609_04774_b200 import build
        if rank == 0:
            build.build()
        dist.barrier()
    peaks = load_peaks()
    w = get_workload(args.config)
    runner = Runner(w, local, need_host=True)
    flops = flops_of(w)

    # headline: exactly K steps between events, clocks sampled from the warm-up on
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    total_ms, per = timed_loop(torch, runner.step, args.steps, args.warmup, dist)
    kern_steps = max(20, min(args.steps, 50))
    kern_ms = kernel_only_ms(torch, runner, kern_steps)
    clocks = sampler.stop() if rank == 0 else None
    e2e_steps = max(50, args.steps)
    e2e_ms, _ = timed_loop(torch, runner.step_e2e, e2e_steps, 3, dist)
    runner.ctx.poll_status()

    total_ms, e2e_ms = max_over_ranks(torch, dist, [total_ms, e2e_ms], "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    value = whole_job_value(world, flops, ms_per_step)
    e2e_value = whole_job_value(world, flops, e2e_ms / e2e_steps)
    achieved = flops / (kern_ms * 1e-3) / 1e12
    peak = peaks["bf16_tflops"]
    launches = runner.launches_per_step()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "requests": len(w.requests), "new_tokens": w.total_new, "Hq": w.Hq,
                   "Hkv": w.Hkv, "D": w.D, "page_size": wl.PAGE, "seed": w.seed, "pairs": pairs_of(w),
                   "l2": "inputs (q+kv+out = %.0f MB) exceed the 126 MB L2; no flush between steps" % (algorithmic_bytes(w) / 1e6),
                   "multi_gpu": "independent replicas of the workload per rank, no collective"},
        "tokens_per_s": world * w.total_new / (ms_per_step * 1e-3),
        # the K timed steps are a burst (tens of milliseconds at full clocks): fractions of the burst figures only;
        # the power-capped regime is the `sustained` leg's
        "frac": {k: v for k, v in fractions(value / world, peaks).items() if k != "of_measured_sustained"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": runner.h2d_bytes,
                "d2h_bytes_per_step": runner.d2h_bytes, "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps,
                "pipelining": "3 streams (copy in / compute / copy out), 2 staging buffers, one packed copy per direction; every step's bytes move inside the timed region"},
        "gpu_launches": args.steps * launches,
        "launches_per_step": launches,
        "schedule": runner.schedule,
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "traffic": ATTN_TRAFFIC_BYTES.get(w.name),
                     "algorithmic_bytes": algorithmic_bytes(w), "kernel": "cp_attn_kernel",
                     "kernel_ms": kern_ms, "kernel_launches_timed": kern_steps,
                     "kernel_ms_covers": "the launches of one step (list copy if any + cp_attn_kernel + LSE fix-up)",
                     "peak_source": "%s burst bf16 (of %s): the timed launches are short and run at burst clocks" % (peaks["_source"], peaks["_source"]),
                     "frac_of_nominal_2250": achieved / NOMINAL_BF16_TFLOPS},
        "clocks": clocks,
    }
    if world == 1 and not args.headline_only:
        sus = sustained_leg(torch, runner, peaks, local)
        line["sustained"] = sus
        # the fraction of the power-capped peak comes from the power-capped leg only
        line["roofline"]["frac_of_sustained"] = sus["tflops"] / peaks["bf16_tflops_sustained"]
        line["roofline"]["frac_of_sustained_source"] = "sustained leg (%.1f s of GPU time) over the measured sustained bf16 rate" % sus["gpu_seconds"]
        mat_headline = runner.mat
        runner.close()
        del runner
        torch.cuda.empty_cache()
        line["configs"] = [config_leg(torch, c, peaks, local) for c in (1, 2, 3, 4, 5)]
        line["configs_fp8"] = [config_leg(torch, c, peaks, local, fp8=True) for c in (2, 5)]
        bf, f32 = torch.bfloat16, torch.float32
        line["merge"] = merge_points(torch, peaks, [(T, N, bf) for T in (4096, 16384, 65536) for N in (2, 4, 8)] +
                                     [(16384, N, f32) for N in (2, 4, 8)])
        line["kvcopy"] = kvcopy_points(torch, peaks)
        line["cp_rank"] = cp_rank_leg(args)
        line["prefill_time_table"] = table_leg(torch)
        targets = {c["workload"]: c["ms"] for c in line["configs"]}
        line["targets"] = {
            "cfg2_ms_le_0.855": targets.get("cfg2_R4096_P12288_C4"), "cfg3_ms_le_125.1": targets.get("cfg3_R131072_P0_C8"),
            "merge_points_below_5600_GBps": [(m["T"], m["N"], m["out"], round(m["GBps"])) for m in line["merge"] if m["GBps"] < 5600.0],
            "cp_rank_graph_ms_le_0.30": line["cp_rank"]["slowest_rank_ms_graph_replay"]}
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline_legs(w, mat_headline, args)
    elif not args.no_cpu_baseline and world == 1:
        from oracle import reference as orc
        orc.build()
        t, pairs, threads = oracle_sample(w, runner.mat, args.cpu_rows, 4242)
        line["cpu_baseline"] = {"value": 4 * w.D * pairs / t / 1e12, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": "%d seeded rows x %d heads per request (%.1f s)" % (args.cpu_rows, w.Hq, t)}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------------
# extra modes: per-config numbers, merge sweep, prefill-time table
# ----------------------------------------------------------------------------------------------
def run_configs(args, out):
    import torch
    peaks = load_peaks()
    for cfg in args.configs:
        out.write(json.dumps(dict(mode="config", **config_leg(torch, cfg, peaks, 0, budget_ms=args.config_ms, fp8=args.fp8, page=args.page))) + "\n")
        out.flush()


def run_merge_sweep(args, out):
    import torch
    from paper_2609_04774_b200 import build
    build.build()
    peaks = load_peaks()
    points = [(T, N, dt) for T in args.merge_T for N in (2, 4, 8) for dt in (torch.bfloat16, torch.float32)
              if N * T * 64 * 516 <= 100e9]
    for m in merge_points(torch, peaks, points, reps=args.merge_reps):
        out.write(json.dumps(dict(mode="merge", **m)) + "\n")
    out.flush()


def run_kvcopy(args, out):
    import torch
    from paper_2609_04774_b200 import build
    build.build()
    for m in kvcopy_points(torch, load_peaks(), tuple(args.kv_tokens)):
        out.write(json.dumps(dict(mode="kvcopy", **m)) + "\n")
    out.flush()


def _time_call(torch, fn):
    """Best of three batch means of one call; a batch runs for about 10 ms (2 to 50 launches)."""
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    fn()
    e1.record()
    torch.cuda.synchronize()
    reps = int(max(2, min(50, 10.0 / max(e0.elapsed_time(e1), 1e-3))))
    best = float("inf")
    for _ in range(3):
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1) / reps)
    return best


def table_leg(torch):
    """A corner of the prefill-time table for the default line: (new_len, prefix_len) in {4096, 16384} x hit ratio
    {0, 0.75}, C in {1, 2, 4, 8}: time of all shards in one launch and of the slowest / fastest single shard (what one
    CP rank computes), with W(R, P) of Eq. 1.  Random K/V made on the device (the values do not matter for the time)."""
    from paper_2609_04774_b200 import binding
    ctx = binding.Context(torch.cuda.current_device())
    Hq, Hkv, D = 32, 8, 128
    scale = D ** -0.5
    rows = []
    for R in (4096, 16384):
        for hit in (0.0, 0.75):
            P = (int(round(R / (1 - hit))) - R) // wl.PAGE * wl.PAGE
            pages = (P + R + wl.PAGE - 1) // wl.PAGE
            q = torch.randn((R, Hq, D), device="cuda").to(torch.bfloat16)
            k = torch.randn((pages, wl.PAGE, Hkv, D), device="cuda").to(torch.bfloat16)
            v = torch.randn((pages, wl.PAGE, Hkv, D), device="cuda").to(torch.bfloat16)
            pt = torch.from_numpy(wl.permutation(11, wl.TID_PERM, pages)).cuda()
            cache = binding.make_cache(k, v)
            o = torch.empty((R, Hq, D), dtype=torch.bfloat16, device="cuda")
            lse = torch.empty((Hq, R), dtype=torch.float32, device="cuda")
            po = torch.empty((R, Hq, D), dtype=torch.float32, device="cuda")
            ws = torch.zeros(binding.cp_workspace_bytes([R], [8], Hq), dtype=torch.uint8, device="cuda")
            W = R * P + R * (R + 1) // 2
            for C in (1, 2, 4, 8):
                t_all = _time_call(torch, lambda: binding.cp_prefill_attn(ctx, q, cache, pt, P, R, C, Hq, scale, o, lse, ws))
                ts = [_time_call(torch, lambda: binding.cp_prefill_attn_shard(ctx, q, cache, pt, P, R, C, s, Hq, scale, po, lse, ws))
                      for s in range(C)]
                rows.append({"R": R, "P": P, "C": C, "W": W, "t_all_ms": t_all, "t_shard_max_ms": max(ts), "t_shard_min_ms": min(ts)})
            ctx.poll_status()
            del q, k, v, o, po, lse, ws
            torch.cuda.empty_cache()
    ctx.close()
    base = {(r["R"], r["P"]): r["t_shard_max_ms"] for r in rows if r["C"] == 1}
    for r in rows:
        r["speedup_vs_C1"] = base[(r["R"], r["P"])] / r["t_shard_max_ms"]
    return rows


def run_table(args, out):
    """Measured prefill-time table over (new_len, prefix_len, C): all-shard time and the slowest /
    fastest single shard (what one CP rank would compute), with W(R,P) of Eq. (1) -- the inputs of the
    paper's cache-aware prefill-time model (Eq. 2)."""
    import torch
    from paper_2609_04774_b200 import binding, build
    build.build()
    ctx = binding.Context(0)
    Hq, Hkv, D = 32, 8, 128
    out.write("R,P,C,W,W_over_C,t_all_ms,t_shard_max_ms,t_shard_min_ms\n")
    rows = []
    for R in args.table_R:
        for hit in (0.0, 0.25, 0.5, 0.75, 0.9):
            L = int(round(R / (1 - hit)))
            P = (L - R) // wl.PAGE * wl.PAGE
            w0 = wl.Workload("table", 7, Hq, Hkv, [wl.Request(R, P, 1)])
            mat = wl.materialize(w0)
            dev = lambda bits: torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)
            q, k, v = dev(mat.q), dev(mat.k_pages), dev(mat.v_pages)
            pt = torch.from_numpy(mat.page_table).cuda()
            cache = binding.make_cache(k, v)
            o = torch.empty((R, Hq, D), dtype=torch.bfloat16, device="cuda")
            lse = torch.empty((Hq, R), dtype=torch.float32, device="cuda")
            po = torch.empty((R, Hq, D), dtype=torch.float32, device="cuda")
            ws = torch.zeros(binding.cp_workspace_bytes([R], [8], Hq), dtype=torch.uint8, device="cuda")

            timeit = lambda fn: _time_call(torch, fn)

            W = R * P + R * (R + 1) // 2
            for C in (1, 2, 4, 8):
                t_all = timeit(lambda: binding.cp_prefill_attn(ctx, q, cache, pt, P, R, C, Hq, w0.scale, o, lse, ws))
                ts = [timeit(lambda: binding.cp_prefill_attn_shard(ctx, q, cache, pt, P, R, C, s, Hq, w0.scale, po, lse, ws))
                      for s in range(C)]
                out.write("%d,%d,%d,%d,%.1f,%.4f,%.4f,%.4f\n" % (R, P, C, W, W / C, t_all, max(ts), min(ts)))
                out.flush()
                rows.append((R, P, C, max(ts) * 1e-3))
            ctx.poll_status()
            del q, k, v, o, po, lse
            torch.cuda.empty_cache()
    # Eq. (2) fitted to the slowest shard of every (R, P, C): what one CP rank of degree C would take
    from paper_2609_04774_b200 import prefill_model as pm
    Rs, Ps, Cs, ts = (np.array(x, dtype=np.float64) for x in zip(*rows))
    m = pm.fit(Rs, Ps, Cs, ts)
    rel = np.abs(m.predict(Rs, Ps, Cs) / ts - 1)
    out.write("# fit of Eq. 2 to t_shard_max (seconds): d=%.3e a=%.3e b=%.3e c=%.3e alpha=%.3e ; relative error median %.3f "
              "p90 %.3f max %.3f\n" % (m.d, m.a, m.b, m.c, m.alpha, np.median(rel), np.quantile(rel, 0.9), rel.max()))
    out.flush()


class _LoopbackComm:
    """Stands in for the C-rank all-gather on one GPU: every peer's block is a device copy of this
    rank's own block.  The bytes written to local HBM equal a real gather's; the values do not, so
    this is for timing one rank's local work only."""

    class _Done:
        def wait(self):
            return True

    def __init__(self, size, rank):
        self.size, self.rank = size, rank

    def all_gather(self, block):
        return block.unsqueeze(0).expand((self.size,) + tuple(block.shape)).contiguous(), self._Done()

    def all_gather_into(self, out, block):
        out.view((self.size,) + tuple(block.shape)).copy_(block.unsqueeze(0).expand((self.size,) + tuple(block.shape)))
        return self._Done()

    def all_to_all(self, blocks):
        return blocks.clone(), self._Done()


def cp_rank_leg(args):
    """The rank worker's local time on the headline configuration for the default line: slowest rank, issued call by
    call and replayed from a CUDA graph (bf16 cache, all-gather-KV exchange, landing mode)."""
    import copy
    import io
    a = copy.copy(args)
    a.configs, a.fp8, a.pass_q, a.no_landing = [2], False, False, False
    buf = io.StringIO()
    run_cprank(a, buf)
    d = json.loads(buf.getvalue().strip().splitlines()[-1])
    g = [x for x in d["rank_local_ms_graph_replay"] if x]
    return {"workload": d["workload"], "C": d["C"], "exchange": d["exchange"], "landing": d["landing"],
            "slowest_rank_ms": d["slowest_rank_ms"], "slowest_rank_ms_graph_replay": max(g) if g else None,
            "nvlink_bytes_received_per_rank": d["nvlink_bytes_received_per_rank"],
            "nvlink_ms_modelled_at_770GBps": d["nvlink_ms_modelled_at_770GBps"],
            "note": "one GPU: local work of each rank measured with loopback gathers; the link time is modelled, not measured"}


def run_cprank(args, out):
    """Local time of every rank of a degree-C CP worker (early-chunk-first order): own prefix block read
    out, gathered rows appended to the rank's paged cache, the two chunk attention calls.  The NVLink
    transfer itself cannot be run on one GPU; its size and a modelled time at the measured peer-copy
    bandwidth are printed beside the measured local time."""
    import torch
    from paper_2609_04774_b200 import binding, build
    from paper_2609_04774_b200.cp_rank import CpRankWorker, LibraryOps, LibraryOps8, RankLayout, landing_pages
    build.build()
    D = 128
    for cfg in args.configs:
        w = get_workload(cfg)
        if len(w.requests) != 1:
            continue
        r = w.requests[0]
        R, P, C = r.new_len, r.prefix_len, r.C
        n_pages = r.n_pages
        pt = torch.from_numpy(wl.permutation(w.seed, wl.TID_PERM, n_pages)).cuda()
        # landing mode (the default here when the chunks are whole pages): the gathers write into a run of pages behind
        # the request's own pages and no append runs; --no-landing times the arena + append path
        land_pages = landing_pages(RankLayout(R, P, C, 0))
        a0 = None if args.no_landing else n_pages
        pool = n_pages + land_pages
        if args.fp8:      # E4M3 pages (finite codes), per-head scales shared by all ranks; stored bytes travel
            k = (torch.randn((pool, wl.PAGE, w.Hkv, D), device="cuda") * 70).to(torch.float8_e4m3fn).view(torch.uint8)
            v = (torch.randn((pool, wl.PAGE, w.Hkv, D), device="cuda") * 70).to(torch.float8_e4m3fn).view(torch.uint8)
            sc = torch.full((w.Hkv,), 6.0 / 448.0, dtype=torch.float32, device="cuda")
            ops = LibraryOps8(binding.Context(0), k, v, sc, sc.clone(), pt, w.Hq, w.scale, arena_page0=a0)
        else:
            k = torch.randn((pool, wl.PAGE, w.Hkv, D), device="cuda").to(torch.bfloat16)
            v = torch.randn((pool, wl.PAGE, w.Hkv, D), device="cuda").to(torch.bfloat16)
            ops = LibraryOps(binding.Context(0), k, v, pt, w.Hq, w.scale, arena_page0=a0)
        landed = ops.landing(RankLayout(R, P, C, 0)) is not None
        per_rank, per_rank_graph = [], []
        for rank in range(C):
            lay = RankLayout(R, P, C, rank)
            rows = {}
            for name, j in (("early", lay.early), ("late", lay.late)):
                b, e = lay.chunk(j)
                rows["q_" + name] = torch.randn((e - b, w.Hq, D), device="cuda").to(torch.bfloat16)
                rows["k_" + name] = torch.randn((e - b, w.Hkv, D), device="cuda").to(torch.bfloat16)
                rows["v_" + name] = torch.randn((e - b, w.Hkv, D), device="cuda").to(torch.bfloat16)
            worker = CpRankWorker(lay, _LoopbackComm(C, rank), ops)
            run = worker.prefill_pass_q if args.pass_q else worker.prefill
            fn = lambda: run(rows["q_early"], rows["q_late"], rows["k_early"], rows["v_early"], rows["k_late"], rows["v_late"])
            ms = []
            for i in range(2 + args.rank_reps):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                fn()
                e1.record()
                torch.cuda.synchronize()
                if i >= 2:
                    ms.append(e0.elapsed_time(e1))
            ops.ctx.poll_status()
            per_rank.append(statistics.median(ms))
            # the same step replayed from a CUDA graph (one launch per layer instead of ~20 calls from Python): only when
            # both chunk calls carry their work lists in the launch parameters, so that a replay reads no host staging
            g_ms = None
            small = all(binding.cp_schedule_inspect([0, e - b], [P + b], [1], w.Hq, w.Hkv, want_lists=False)[0]["inline"]
                        for b, e in (lay.chunk(lay.early), lay.chunk(lay.late)) if e > b)
            if small and not args.pass_q:
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    fn()
                torch.cuda.current_stream().wait_stream(side)
                torch.cuda.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph):
                    fn()
                ts = []
                for i in range(2 + args.rank_reps):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    graph.replay()
                    e1.record()
                    torch.cuda.synchronize()
                    if i >= 2:
                        ts.append(e0.elapsed_time(e1))
                ops.ctx.poll_status()
                g_ms = statistics.median(ts)
                del graph
            per_rank_graph.append(g_ms)
        lay0 = RankLayout(R, P, C, 0)
        if args.pass_q:   # queries in (bf16), partials of the own rows back (fp32 + lse)
            recv = (C - 1) * 2 * lay0.cl * w.Hq * (D * 2 + D * 4 + 4)
        else:             # K and V of the other ranks' prefix blocks and chunks
            recv = (C - 1) * 2 * (1 if args.fp8 else 2) * w.Hkv * D * (lay0.block_pages * wl.PAGE + 2 * lay0.cl)
        out.write(json.dumps({"mode": "cprank", "exchange": "pass-q" if args.pass_q else ("all-gather-kv, fp8 bytes" if args.fp8 else "all-gather-kv"),
                              "landing": bool(landed and not args.pass_q), "config": cfg, "workload": w.name, "R": R, "P": P, "C": C,
                              "rank_local_ms": per_rank, "slowest_rank_ms": max(per_rank),
                              "rank_local_ms_graph_replay": per_rank_graph,
                              "tflops_per_gpu_slowest_rank": flops_of(w) / C / (max(per_rank) * 1e-3) / 1e12,
                              "nvlink_bytes_received_per_rank": recv,
                              "nvlink_ms_modelled_at_770GBps": recv / 770e9 * 1e3,
                              "note": "local work measured with loopback gathers; link time modelled, not measured"}) + "\n")
        out.flush()
        del k, v, ops
        torch.cuda.empty_cache()


def run_cachemgr(args, out):
    """Host throughput of the prefix-cache bookkeeping on a seeded request stream: per request one
    match per worker (ReusedPath), PreferDegree, Algorithm 1 and the new replica; a scan (Algorithm 2)
    every 1000 requests.  The oracle runs the first tenth of the same stream for scale."""
    from paper_2609_04774_b200 import build, cache_manager as cmgr
    build.build()
    model = (3e-4, 2e-7, 5e-8, 1e-6, 4e-11)
    degrees = [1, 2, 4, 8]
    workers = {w: degrees[w % 4] for w in range(16)}
    ids = sorted(workers)
    stream = wl.prefix_stream(21, args.cache_requests)
    pick = wl.counter_uniform(21, wl.TID_STREAM, 1 << 20, len(stream))

    def drive(trie, reused_fn, prefer_fn, n, wrap=lambda b: b):
        t0 = time.perf_counter()
        scans = 0
        for i, (blocks, L) in enumerate(stream[:n]):
            blocks = wrap(blocks)
            reused = reused_fn(trie, blocks)
            pref = prefer_fn(L, reused)
            w = ids[int(pick[i] * len(ids))]
            trie.update(blocks, L, w, pref, model)
            trie.add_replica(blocks, w)
            if i % 1000 == 999:
                trie.scan(1e-5, 3.0, 0.4, 0.8, 16)
                scans += 1
        return time.perf_counter() - t0, scans

    t = cmgr.Trie(degrees, 64)
    for w, c in workers.items():
        t.set_worker(w, c)
    ids_arr, deg_arr = np.array(ids, dtype=np.int32), np.array([workers[w] for w in ids], dtype=np.int32)
    dt, scans = drive(t, lambda tr, b: tr.reused_all(b, ids_arr).astype(np.int64) * 64,
                      lambda L, reused: cmgr.cp_prefer_degree(model, L, deg_arr, reused, 1.2, 0.2)[1],
                      len(stream), cmgr.Keys)
    nodes = t.size()
    # cpu_baseline leg: the oracle on the first tenth of the stream
    sys.path.insert(0, ROOT)
    from oracle import cache_manager as ocm
    o = ocm.Trie(degrees, 64)
    for w, c in workers.items():
        o.set_worker(w, c)
    n_o = max(1, len(stream) // 10)
    dto, _ = drive(o, lambda tr, b: [len(tr.reused_path(b, w)) * 64 for w in ids],
                   lambda L, reused: ocm.prefer_degree(model, L, [(workers[w], p) for w, p in zip(ids, reused)], 1.2, 0.2)[1], n_o)
    out.write(json.dumps({"mode": "cachemgr", "requests": len(stream), "workers": len(ids), "nodes": nodes, "scans": scans,
                          "library_requests_per_s": len(stream) / dt,
                          "cpu_baseline": {"value": n_o / dto, "unit": "requests/s", "cores": 1, "kind": "oracle",
                                           "sample": "first %d requests of the same stream" % n_o},
                          "note": "driven from Python through ctypes"}) + "\n")
    out.flush()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="number of the configuration used as the headline workload")
    ap.add_argument("--mode", default="bench", choices=["bench", "configs", "merge", "table", "kvcopy", "cprank", "cachemgr", "cpu"])
    ap.add_argument("--configs", type=int, nargs="*", default=[1, 2, 3, 4, 5],
                    help="1-5: the benchmark configurations; 6: 32/4 grouped-query head shape; 7: chunked prefill, R << P; 8: multi-head (16/16)")
    ap.add_argument("--config-ms", type=float, default=1200.0, help="configs mode: GPU time per configuration")
    ap.add_argument("--fp8", action="store_true", help="configs / cprank modes: the FP8 K/V variant")
    ap.add_argument("--page", type=int, default=None, help="configs mode: tokens per cache page (16, 32, 64, 128)")
    ap.add_argument("--rank-reps", type=int, default=5)
    ap.add_argument("--pass-q", action="store_true", help="cprank mode: K/V stays sharded, queries travel")
    ap.add_argument("--kv-tokens", type=int, nargs="*", default=[16384, 131072, 1048576], help="kvcopy mode: tokens per point")
    ap.add_argument("--no-landing", action="store_true",
                    help="cprank mode: gather into separate arenas and append into the cache instead of landing in pool pages")
    ap.add_argument("--cache-requests", type=int, default=20000)
    ap.add_argument("--merge-T", type=int, nargs="*", default=[4096, 16384, 65536, 262144])
    ap.add_argument("--merge-reps", type=int, default=20)
    ap.add_argument("--table-R", type=int, nargs="*", default=[1024, 2048, 4096, 8192, 16384, 32768, 65536, 131072])
    ap.add_argument("--out", default=None)
    ap.add_argument("--cpu-rows", type=int, default=512, help="rows per request of the cpu_baseline sample")
    ap.add_argument("--ref-rows", type=int, default=96, help="rows per request per step of --impl reference")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true",
                    help="bench mode: only the headline workload (no sustained / configs / merge / kvcopy legs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    if args.mode == "bench":
        return run_ours(args)
    out = open(args.out, "w") if args.out else sys.stdout
    {"configs": run_configs, "merge": run_merge_sweep, "table": run_table, "kvcopy": run_kvcopy, "cprank": run_cprank, "cachemgr": run_cachemgr, "cpu": run_cpu_full}[args.mode](args, out)


if __name__ == "__main__":
    main()
