"""Benchmark of the OCS hot path on B200: split -> clip search -> quantize -> int8 GEMM/conv.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload fc6|fc6-fused|fc6-small|fc|conv|resnet50|lstm|act-ocs|exact-mse] [--impl reference]

One step is one pass of the whole path over one batch of synthetic input:
  fc6   (default) the VGG-16-fc6-shaped sweep: W [4096, 25088], 5 expand ratios x 4 weight bit
        widths = 20 points; every point runs ocs_split, ocs_quantize with the MSE clip search,
        the activation quantization and ocs_qlinear (nothing is cached between points).
  fc6-fused  the same sweep through ocs_split_quantize, which never writes the fp32 W'.
  fc6-small  the same recipe on W [256, 6272] (quick checks).
  fc    the small fully-connected layer [256, 512], batch 64, r = 0.05, 8-bit, no clipping.
  conv / resnet50 / lstm   the single 3x3 convolution, the ResNet-50 stack at batch 128 and the LSTM
        language model: a step prepares every layer (split, quantize, pack) and runs the forward pass;
        these report integer TOP/s of the quantized layers instead of bytes per second.
  act-ocs  per-batch activation OCS (Eq. 4) on a ResNet-50 stage-1 1x1 convolution at batch 128: channel
        extrema, split plan, expanded 6-bit activation codes, duplicated weight columns, integer layer.
The reported value is algorithmic bytes per second: the bytes the method must move (listed in
`algorithmic_bytes` below) divided by the step time.  Rank 0 prints one JSON line.

With N > 1 (launched by torch.distributed.run) every rank runs the same step on its own GPU; the
path has no exchange step, so there is no collective on the data path (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from ocs_inputs import configs, prng  # noqa: E402

N_BINS, N_CAND = 2048, 128
INT8_OVER_BF16 = 2.0          # nominal dense int8 rate / nominal dense bf16 rate of the part (fallback only)


# ----------------------------------------------------------------------------------------------
# algorithmic bytes / ops of each kernel (what the method has to move; padding not counted)
def algorithmic_bytes(kernel: str, *, N=0, n=0, M=0, C=0, S=0, Nout=0, R=1, rows=0):
    """N = weight elements before the split, n = elements of the tensor a quantize pass reads,
    GEMM: M x Nout outputs over K' = (C+S)*R."""
    if kernel == "col_minmax_kernel":
        return 4 * N
    if kernel in ("split_rows_kernel", "split_scatter_kernel"):   # row-staged form / plain-load fallback
        return 4 * N + 4 * n
    if kernel in ("hist_kernel", "maxabs_kernel"):
        return 4 * n
    if kernel == "split_hist_kernel":          # fused path: W is read, the expanded rows live in shared memory
        return 4 * N
    if kernel == "split_quantize_kernel":
        return 4 * N + n
    if kernel == "quantize_kernel":
        return 4 * n + n
    if kernel.startswith("ocs_gemm_kernel"):
        return rows * C + Nout * (C + S) * R + 4 * M * Nout + 4 * (C + S)
    if kernel == "pack_conv_kernel":
        return 2 * n
    if kernel == "transpose_codes_kernel":
        return 2 * n
    return 0


class Ledger:
    """Sums algorithmic bytes and integer ops per kernel name over one step."""

    def __init__(self):
        self.bytes = {}
        self.ops = 0

    def add(self, kernel, **kw):
        self.bytes[kernel] = self.bytes.get(kernel, 0) + algorithmic_bytes(kernel, **kw)

    @property
    def total(self):
        return sum(self.bytes.values())


def reduce_max(value: float, world: int, device) -> float:
    """Max over ranks of a per-rank timing (the multi-GPU step time is the slowest rank's)."""
    if world == 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_gbs(bytes_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput: every rank moves the same bytes per step (replicas, weak scaling)."""
    return bytes_per_rank_step * world / (ms_per_step * 1e-3) / 1e9


# DRAM traffic of the dominant kernel from one ncu capture (profiles/split_rows_kernel_fc6.md): the launch
# at r = 0.1 moved 810.3 MB for 863.2 MB of algorithmic bytes.  The figure is only reported while the
# kernel's source text is the one that was profiled.
NCU_TRAFFIC = {"split_rows_kernel": dict(fingerprint="f3a092c5bcf7b39a", dram_bytes=810.3e6, algorithmic_bytes=863.2e6)}


def kernel_fingerprint(kernel: str):
    if kernel != "split_rows_kernel":
        return None
    import hashlib
    try:
        src = open(os.path.join(ROOT, "paper_1901_09504_b200", "csrc", "split.cu")).read()
        a, b = src.index("// K3, bulk-copy form."), src.index("struct SplitWs {")
    except (OSError, ValueError):
        return None
    return hashlib.sha256(src[a:b].encode()).hexdigest()[:16]


def ncu_traffic(kernel: str, algorithmic_bytes_per_launch: float):
    """Per-launch DRAM bytes, scaled from the captured launch by algorithmic bytes (traffic is
    proportional to the rows moved); None when the kernel has changed since the capture."""
    rec = NCU_TRAFFIC.get(kernel)
    if not rec or kernel_fingerprint(kernel) != rec["fingerprint"]:
        return None
    return rec["dram_bytes"] / rec["algorithmic_bytes"] * algorithmic_bytes_per_launch


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=float(p["hbm_gbs"]), bf16_burst=float(p["bf16_tflops"]),
                    bf16_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ----------------------------------------------------------------------------------------------
# The tensor half of the metric on shapes the tensor pipe bounds.  (1) The int8 peak of this GPU, measured in
# the same run: the library int8 GEMM (torch._int_mm, cuBLASLt) on 8192^3, best of 10, CUDA events -- a library
# measurement, used as the denominator.  (2) ocs_qlinear on the same shape without and with 2 % duplicated
# channels.  (3) The 3x3 convolutions of ResNet-50's stages 3 and 4 at batch 128 (configs[3]'s heavy layers)
# through ocs_qconv, ops-weighted.  Inputs are random codes made on the device: these are timings of the
# contraction alone, reported beside the headline, not in it.
def _time_best(torch, fn, reps=10, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    best = float("inf")
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        best = min(best, e0.elapsed_time(e1))
    return best


def tensor_probe(ocs, torch, dev):
    out = {}
    g = torch.Generator(device=dev)
    g.manual_seed(7)
    n = 8192
    ops = 2.0 * n * n * n
    a8 = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=dev, generator=g)
    b8 = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=dev, generator=g)
    try:
        ms = _time_best(torch, lambda: torch._int_mm(a8, b8))
        out["int8_peak_tops"] = ops / (ms * 1e-3) / 1e12
        out["int8_peak_note"] = "measured in this run: torch._int_mm (library int8 GEMM) 8192^3, best of 10, CUDA events"
    except Exception as e:      # the library routine is missing: fall back to the nominal ratio
        out["int8_peak_tops"] = None
        out["int8_peak_note"] = f"torch._int_mm unavailable ({type(e).__name__})"
    del b8
    st = ocs.new_status(dev)
    a_scale = torch.full((1,), 0.01, dtype=torch.float32, device=dev)
    w_scale = torch.full((1,), 0.001, dtype=torch.float32, device=dev)
    Au = a8.view(torch.uint8)
    Y = torch.empty((n, n), dtype=torch.float32, device=dev)
    ws = torch.empty(int(ocs.lib().ocs_qlinear_workspace_bytes(n, n, n, 164)) + 256, dtype=torch.uint8, device=dev)
    for S, key in ((0, "qlinear_8192_tops"), (164, "qlinear_8192_dup2pct_tops")):
        ldw = ocs.round_up(n + S, 16)
        Wc = torch.randint(-127, 128, (n, ldw), dtype=torch.int8, device=dev, generator=g)
        idx = torch.cat([torch.arange(n, dtype=torch.int32, device=dev),
                         torch.randint(0, n, (S,), dtype=torch.int32, device=dev, generator=g)]).contiguous()
        AT = ocs.ocs_transpose_codes(Au) if S else None      # channel-major copy: the duplicated channels arrive by TMA
        ms = _time_best(torch, lambda: ocs.ocs_qlinear(Au, a_scale, Wc, w_scale, idx, n, S, out=Y, ws=ws, dev_status=st,
                                                       A_codes_T=AT))
        out[key] = 2.0 * n * n * (n + S) / (ms * 1e-3) / 1e12
        del Wc
    del a8, Au, Y
    # ResNet-50 stages 3-4, 3x3 convolutions at batch 128: (C = O, H_in, stride, how many such layers)
    tot_ops, tot_ms = 0.0, 0.0
    for Cn, H, stride, count in ((256, 28, 2, 1), (256, 14, 1, 5), (512, 14, 2, 1), (512, 7, 1, 2)):
        S = configs_num_splits(Cn, 0.01)
        Ho = (H + 2 - 3) // stride + 1
        X = torch.randint(0, 256, (128, H, H, Cn), dtype=torch.uint8, device=dev, generator=g)
        Kp = ocs.ocs_conv_packed_k(Cn, S, 3, 3)
        Wp = torch.randint(-127, 128, (Cn, ocs.round_up(Kp, 16)), dtype=torch.int8, device=dev, generator=g)
        idx = torch.cat([torch.arange(Cn, dtype=torch.int32, device=dev),
                         torch.randint(0, Cn, (S,), dtype=torch.int32, device=dev, generator=g)]).contiguous()
        Yc = torch.empty((128, Ho, Ho, Cn), dtype=torch.float32, device=dev)
        wsc = torch.empty(int(ocs.lib().ocs_qconv_workspace_bytes(128, H, H, Cn, Cn, S, 3, 3, stride, 1)) + 256,
                          dtype=torch.uint8, device=dev)
        ms = _time_best(torch, lambda: ocs.ocs_qconv(X, a_scale, Wp, w_scale, idx, S, 3, 3, stride, 1, out=Yc, ws=wsc,
                                                     dev_status=st), reps=5)
        tot_ops += count * 2.0 * 128 * Ho * Ho * Cn * (Cn + S) * 9
        tot_ms += count * ms
    out["resnet50_3x3_stage34_tops"] = tot_ops / (tot_ms * 1e-3) / 1e12
    assert ocs.ocs_poll_status(st) == 0, "device status word set during the tensor probe"
    return out


# ----------------------------------------------------------------------------------------------
class Fc6Sweep:
    name = "fc6"
    LANES = 3      # sweep points in flight (measured on the fc6 sweep: 9.44 / 8.62 / 8.40 / 8.45 ms with 1 / 2 / 3 / 4)

    def __init__(self, small=False):
        self.O, self.C, self.M = (256, 6272, 128) if small else (4096, 25088, 128)
        if small:
            self.name = "fc6-small"
        self.desc = (f"configs[2]: fc6-shaped W [{self.O}, {self.C}] fp32, sweep of 5 expand ratios x 4 weight bit "
                     f"widths (20 points), MSE clip search ({N_CAND} candidates, {N_BINS} bins), int8 containers, "
                     f"activations [{self.M}, {self.C}] 8-bit unsigned; seed 2")
        self.points = [(r, b) for r in configs.CONFIG3_RATIOS for b in configs.CONFIG3_BITS]

    def host_inputs(self):
        c = configs.config3(O=self.O, C=self.C, M=self.M)
        return dict(W=c["W"], A=c["A"])

    def setup(self, ocs, torch, dev, host):
        self.ocs, self.torch = ocs, torch
        O, C, M = self.O, self.C, self.M
        Smax = max(ocs.ocs_num_splits(C, r) for r, _ in self.points)
        self.W = torch.empty((O, C), dtype=torch.float32, device=dev)
        self.A = torch.empty((M, C), dtype=torch.float32, device=dev)
        self.ld_out = ocs.round_up(C + Smax, 16)
        self.W_out = torch.empty((O, self.ld_out), dtype=torch.float32, device=dev)
        self.idx_map = torch.empty(C + Smax, dtype=torch.int32, device=dev)
        self.max_abs = torch.zeros(3, dtype=torch.float32, device=dev)
        self.codes = torch.empty((O, self.ld_out), dtype=torch.int8, device=dev)
        self.a_codes = torch.empty((M, ocs.round_up(C, 16)), dtype=torch.uint8, device=dev)
        self.a_codes_T = torch.empty((C, ocs.round_up(M, 16)), dtype=torch.uint8, device=dev)   # channel-major copy
        self.scal = torch.zeros(4, dtype=torch.float32, device=dev)      # w_scale, alpha, a_scale, a_alpha
        self.Y = [torch.empty((M, O), dtype=torch.float32, device=dev) for _ in self.points]
        L = ocs.lib()
        nws = max(L.ocs_split_workspace_bytes(O, C, 1, Smax), L.ocs_quantize_workspace_bytes(N_BINS, N_CAND),
                  max(L.ocs_qlinear_workspace_bytes(M, O, C, ocs.ocs_num_splits(C, r)) for r, _ in self.points))
        self.ws = torch.empty(int(nws) + 256, dtype=torch.uint8, device=dev)
        self.status = ocs.new_status(dev)
        self.W.copy_(host["W"])
        self.A.copy_(host["A"])
        # Sweep points are independent: they run in two lanes (two streams, each with its own working buffers), so
        # that the latency-bound kernels of one point (the single-CTA split plan, the candidate scores, the short
        # GEMM) overlap the streaming kernels of the other.
        self.lanes = min(self.LANES, len(self.points))
        self.lane_bufs = [dict(W_out=self.W_out, idx_map=self.idx_map, max_abs=self.max_abs, codes=self.codes,
                               a_codes=self.a_codes, a_codes_T=self.a_codes_T, scal=self.scal, ws=self.ws)]
        for _ in range(1, self.lanes):
            self.lane_bufs.append({k: torch.zeros_like(v) if k in ("scal", "max_abs") else torch.empty_like(v)
                                   for k, v in self.lane_bufs[0].items()})
        self.lane_streams = [torch.cuda.Stream() for _ in range(self.lanes)] if self.lanes > 1 else []

    def release(self):
        """Drops the big device buffers (called after the last timed region)."""
        self.lane_bufs = None
        for k in ("W", "A", "W_out", "codes", "a_codes_T", "Wd", "Ad", "Yd", "Y", "slot_graphs", "graph_obj", "ws"):
            if hasattr(self, k):
                setattr(self, k, None)
        self.torch.cuda.empty_cache()

    def ledger(self):
        led = Ledger()
        O, C, M = self.O, self.C, self.M
        N = O * C
        for r, _ in self.points:
            S = configs_num_splits(C, r)
            n = O * (C + S)
            led.add("col_minmax_kernel", N=N)
            led.add("split_rows_kernel", N=N, n=n)
            led.add("hist_kernel", n=n)
            led.add("quantize_kernel", n=n)
            led.add("maxabs_kernel", n=M * C)
            led.add("quantize_kernel", n=M * C)
            if S > 0:
                led.add("transpose_codes_kernel", n=M * C)
            led.add("ocs_gemm_kernel(linear)", rows=M, M=M, C=C, S=S, Nout=O)
            led.ops += 2 * M * O * (C + S)
        return led

    def gemm(self, i, S, b):
        """Activation codes -> layer output of sweep point i: with duplicated channels the layer gathers them as
        whole rows of a channel-major copy of the codes (made here, every point: nothing is cached)."""
        ocs, C = self.ocs, self.C
        at = None
        if S > 0:
            at = ocs.ocs_transpose_codes(b["a_codes"], cols=C, out=b["a_codes_T"])
        ocs.ocs_qlinear(b["a_codes"], b["scal"][2:3], b["codes"], b["scal"][0:1], b["idx_map"], C, S,
                        out=self.Y[i], ws=b["ws"], dev_status=self.status, A_codes_T=at)

    def point(self, i, b):
        ocs, C = self.ocs, self.C
        r, bits = self.points[i]
        S = ocs.ocs_num_splits(C, r)
        ocs.ocs_split(self.W, S, out=(b["W_out"], b["idx_map"], None, b["max_abs"]), ws=b["ws"],
                      dev_status=self.status)
        ocs.ocs_quantize(b["W_out"], bits, True, ocs.CLIP_MSE, N_CAND, N_BINS, cols=C + S,
                         max_abs_in=b["max_abs"][1:2], out=(b["codes"], b["scal"][0:1], b["scal"][1:2]),
                         ws=b["ws"], dev_status=self.status)
        ocs.ocs_quantize(self.A, 8, False, ocs.CLIP_NONE, out=(b["a_codes"], b["scal"][2:3], b["scal"][3:4]),
                         ws=b["ws"], dev_status=self.status)
        self.gemm(i, S, b)

    def step(self):
        torch = self.torch
        if self.lanes <= 1:
            for i in range(len(self.points)):
                self.point(i, self.lane_bufs[0])
            return
        main = torch.cuda.current_stream()
        for k, st in enumerate(self.lane_streams):
            st.wait_stream(main)
            with torch.cuda.stream(st):
                for i in range(k, len(self.points), self.lanes):
                    self.point(i, self.lane_bufs[k])
        for st in self.lane_streams:
            main.wait_stream(st)

    # The step is a fixed chain of stream-ordered, allocation-free library calls on preallocated buffers: it is
    # captured once in a CUDA graph (after an eager warm-up) and replayed, which removes the host work between
    # the ~200 launches of a step.
    graph = True
    graph_obj = None

    def _capture(self):
        torch = self.torch
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            self.step()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        n0 = self.ocs.ocs_kernel_launches()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, capture_error_mode="thread_local"):
            self.step()
        self.graph_launches = int(self.ocs.ocs_kernel_launches() - n0)
        return g

    def make_graph(self):
        self.graph_obj = self._capture()

    def step_graph(self):
        self.graph_obj.replay()

    def e2e_buffers(self, host):
        """End-to-end steps: every step's inputs travel from pinned host memory and its outputs travel
        back.  The copy of step i+1's inputs runs on a second stream into a second pair of device
        buffers while step i computes (one host-to-device copy of W and A per step); step i's outputs travel
        back on a third stream while step i+1 computes."""
        torch = self.torch
        self.hW = torch.from_numpy(host["W"]).pin_memory()
        self.hA = torch.from_numpy(host["A"]).pin_memory()
        self.hY = [torch.empty(y.shape, dtype=torch.float32).pin_memory() for y in self.Y]
        self.copy_stream = torch.cuda.Stream()
        self.Wd = [self.W, torch.empty_like(self.W)]
        self.Ad = [self.A, torch.empty_like(self.A)]
        self.ready = [torch.cuda.Event(), torch.cuda.Event()]
        self.consumed = [torch.cuda.Event(), torch.cuda.Event()]
        # the outputs are double-buffered too: step i's device-to-host copy runs on a third stream while step
        # i+1 computes into the other set
        self.out_stream = torch.cuda.Stream()
        self.Yd = [self.Y, [torch.empty_like(y) for y in self.Y]]
        self.done = [torch.cuda.Event(), torch.cuda.Event()]
        self.copied = [torch.cuda.Event(), torch.cuda.Event()]
        self.k = 0
        self.slot_graphs = {} if self.graph_obj is None else {0: self.graph_obj}
        torch.cuda.current_stream().synchronize()
        for e in self.consumed + self.copied:
            e.record()
        self._prefetch(0)
        return self.hW.numel() * 4 + self.hA.numel() * 4, sum(y.numel() * 4 for y in self.hY)

    def _prefetch(self, slot):
        torch = self.torch
        with torch.cuda.stream(self.copy_stream):
            self.copy_stream.wait_event(self.consumed[slot])      # the step that last read this slot is done
            self.Wd[slot].copy_(self.hW, non_blocking=True)
            self.Ad[slot].copy_(self.hA, non_blocking=True)
            self.ready[slot].record(self.copy_stream)

    def step_e2e(self):
        torch = self.torch
        cur = self.k % 2
        self._prefetch(1 - cur)                                   # next step's inputs, overlapping this step
        main = torch.cuda.current_stream()
        main.wait_event(self.ready[cur])
        main.wait_event(self.copied[cur])                          # this slot's outputs of two steps ago are home
        self.W, self.A, self.Y = self.Wd[cur], self.Ad[cur], self.Yd[cur]
        if self.graph_obj is None:
            self.step()
        else:
            if cur not in self.slot_graphs:      # one graph per input slot (the graph holds the buffers' addresses)
                self.slot_graphs[cur] = self._capture()
            self.slot_graphs[cur].replay()
        self.consumed[cur].record(main)
        self.done[cur].record(main)
        with torch.cuda.stream(self.out_stream):
            self.out_stream.wait_event(self.done[cur])
            for h, y in zip(self.hY, self.Yd[cur]):
                h.copy_(y, non_blocking=True)
            self.copied[cur].record(self.out_stream)
        self.k += 1

    # the CPU checker on a bounded sample of the same step
    oracle_sample_desc = "3 of the 20 sweep points on the full tensors: (r, bits) = (0.01, 4), (0.05, 6), (0.1, 8)"

    def oracle_sample(self, orc, host):
        W, A = host["W"], host["A"]
        led = Ledger()
        O, C, M = W.shape[0], W.shape[1], A.shape[0]
        t0 = time.perf_counter()
        for r, bits in ((0.01, 4), (0.05, 6), (0.1, 8)):
            S = orc.num_splits(C, r)
            Wp, idx, _, _ = orc.split(W, S, 0.0)
            alpha = orc.clip_mse(Wp, bits, True, N_BINS, N_CAND)["alpha"]
            wc, wsc = orc.quantize(Wp, bits, True, alpha)
            ac, asc = orc.quantize(A, 8, False, orc.maxabs(A))
            orc.qlinear(ac, False, asc, wc, wsc, idx)
            n = O * (C + S)
            for k, kw in (("col_minmax_kernel", dict(N=O * C)), ("split_rows_kernel", dict(N=O * C, n=n)),
                          ("hist_kernel", dict(n=n)), ("quantize_kernel", dict(n=n)), ("maxabs_kernel", dict(n=M * C)),
                          ("quantize_kernel", dict(n=M * C)),
                          ("ocs_gemm_kernel(linear)", dict(rows=M, M=M, C=C, S=S, Nout=O))):
                led.add(k, **kw)
        return time.perf_counter() - t0, led.total


def configs_num_splits(C, r):
    import math
    return 0 if r <= 0 else int(math.ceil(r * C - 1e-9))


class Fc6Fused(Fc6Sweep):
    """The same sweep through ocs_split_quantize (no fp32 W'): fewer bytes per point."""
    name = "fc6-fused"

    def __init__(self):
        super().__init__()
        self.desc = self.desc.replace("configs[2]:", "configs[2] through the fused ocs_split_quantize call:")

    def setup(self, ocs, torch, dev, host):
        super().setup(ocs, torch, dev, host)
        nws = ocs.lib().ocs_split_quantize_workspace_bytes(self.O, self.C, 1, self.idx_map.numel() - self.C, N_BINS, N_CAND)
        self.W_out = None      # never written
        for b in self.lane_bufs:
            b["W_out"] = None
            if nws + 256 > b["ws"].numel():
                b["ws"] = torch.empty(int(nws) + 256, dtype=torch.uint8, device=dev)
        self.ws = self.lane_bufs[0]["ws"]

    def ledger(self):
        led = Ledger()
        O, C, M = self.O, self.C, self.M
        N = O * C
        for r, _ in self.points:
            S = configs_num_splits(C, r)
            n = O * (C + S)
            led.add("col_minmax_kernel", N=N)
            led.add("split_hist_kernel", N=N)
            led.add("split_quantize_kernel", N=N, n=n)
            led.add("maxabs_kernel", n=M * C)
            led.add("quantize_kernel", n=M * C)
            if S > 0:
                led.add("transpose_codes_kernel", n=M * C)
            led.add("ocs_gemm_kernel(linear)", rows=M, M=M, C=C, S=S, Nout=O)
            led.ops += 2 * M * O * (C + S)
        return led

    def point(self, i, b):
        ocs, C = self.ocs, self.C
        r, bits = self.points[i]
        S = ocs.ocs_num_splits(C, r)
        ocs.ocs_split_quantize(self.W, S, bits, ocs.CLIP_MSE, n_candidates=N_CAND, n_bins=N_BINS,
                               out=(b["codes"], b["scal"][0:1], b["scal"][1:2], b["idx_map"], None, b["max_abs"]),
                               ws=b["ws"], dev_status=self.status)
        ocs.ocs_quantize(self.A, 8, False, ocs.CLIP_NONE, out=(b["a_codes"], b["scal"][2:3], b["scal"][3:4]),
                         ws=b["ws"], dev_status=self.status)
        self.gemm(i, S, b)


class ActOcs(Fc6Sweep):
    """Per-batch activation OCS (Eq. 4, Section 5.3) on a ResNet-50 stage-1 1x1 convolution at batch 128."""
    name = "act-ocs"
    l2_note = "activations larger than L2 (no flush)"

    def __init__(self):
        self.Nb, self.H, self.C, self.O, self.S, self.bits = 128, 56, 256, 64, 6, 6
        self.rows = self.Nb * self.H * self.H
        self.desc = (f"per-batch activation OCS with Table 4's settings (r = 0.02 -> {self.S} splits, {self.bits} activation "
                     f"bits, batch {self.Nb}) on a ResNet-50 stage-1 1x1 convolution: activations NHWC [{self.Nb}, {self.H}, "
                     f"{self.H}, {self.C}] fp32 half-normal, weights [{self.O}, {self.C}] as 8-bit codes; a step = channel "
                     "extrema + split plan + expanded unsigned codes (ocs_split_quantize), ocs_dup_weight_columns and the "
                     "integer layer (ocs_qlinear over the pixels); seed 5")
        self.oracle_sample_desc = "the same layer on 8 of the 128 images (its own batch: 25088 pixels)"

    def host_inputs(self):
        X = prng.normal(5, 0, (self.rows, self.C), 1.0, absolute=True)
        W = prng.laplace(5, 1, (self.O, self.C), 0.02)
        return dict(X=X, W=W)

    def setup(self, ocs, torch, dev, host):
        self.ocs, self.torch = ocs, torch
        rows, C, O, S = self.rows, self.C, self.O, self.S
        self.ld = ocs.round_up(C + S, 16)
        self.X = host["X"].to(dev)
        self.status = ocs.new_status(dev)
        Wd = host["W"].to(dev)
        self.w_codes, self.w_scale, _ = ocs.ocs_quantize(Wd, 8, True, ocs.CLIP_NONE, ld_codes=self.ld)
        self.w_codes[:, C:] = 0
        self.codes = torch.empty((rows, self.ld), dtype=torch.uint8, device=dev)
        self.idx_map = torch.empty(C + S, dtype=torch.int32, device=dev)
        self.ident = torch.arange(C + S, dtype=torch.int32, device=dev)
        self.max_abs = torch.zeros(3, dtype=torch.float32, device=dev)
        self.scal = torch.zeros(2, dtype=torch.float32, device=dev)
        self.Y = torch.empty((rows, O), dtype=torch.float32, device=dev)
        L = ocs.lib()
        nws = max(L.ocs_split_quantize_workspace_bytes(rows, C, 1, S, N_BINS, N_CAND),
                  L.ocs_qlinear_workspace_bytes(rows, O, C + S, 0))
        self.ws = torch.empty(int(nws) + 256, dtype=torch.uint8, device=dev)

    def ledger(self):
        led = Ledger()
        rows, C, O, S = self.rows, self.C, self.O, self.S
        led.add("col_minmax_kernel", N=rows * C)
        led.add("split_quantize_kernel", N=rows * C, n=rows * (C + S))
        led.add("ocs_gemm_kernel(linear)", rows=rows, M=rows, C=C + S, S=0, Nout=O)
        led.ops = 2 * rows * O * (C + S)
        return led

    def step(self):
        ocs, C, S = self.ocs, self.C, self.S
        ocs.ocs_split_quantize(self.X, S, self.bits, ocs.CLIP_NONE, is_signed=False,
                               out=(self.codes, self.scal[0:1], self.scal[1:2], self.idx_map, None, self.max_abs),
                               ws=self.ws, dev_status=self.status)
        ocs.ocs_dup_weight_columns(self.w_codes, C, S, self.idx_map, dev_status=self.status)
        ocs.ocs_qlinear(self.codes, self.scal[0:1], self.w_codes, self.w_scale, self.ident, C + S, 0, out=self.Y,
                        ws=self.ws, dev_status=self.status)

    def e2e_buffers(self, host):
        self.hX = self.torch.from_numpy(host["X"]).pin_memory()
        self.hY = self.torch.empty(self.Y.shape, dtype=self.torch.float32).pin_memory()
        return self.hX.numel() * 4, self.hY.numel() * 4

    def step_e2e(self):
        self.X.copy_(self.hX, non_blocking=True)
        if self.graph_obj is None:
            self.step()
        else:
            self.graph_obj.replay()
        self.hY.copy_(self.Y, non_blocking=True)

    def oracle_sample(self, orc, host):
        rows = 8 * self.H * self.H
        X, W = host["X"][:rows], host["W"]
        t0 = time.perf_counter()
        wc, ws = orc.quantize(W, 8, True, orc.maxabs(W))
        orc.act_ocs_linear(X, self.S, self.bits, False, wc, ws, None)
        sec = time.perf_counter() - t0
        led = Ledger()
        led.add("col_minmax_kernel", N=rows * self.C)
        led.add("split_quantize_kernel", N=rows * self.C, n=rows * (self.C + self.S))
        led.add("ocs_gemm_kernel(linear)", rows=rows, M=rows, C=self.C + self.S, S=0, Nout=self.O)
        return sec, led.total


class ExactMse(Fc6Sweep):
    l2_note = "input larger than L2 (103 MB, no flush)"
    """The element-wise MSE scorer (no histogram): every candidate threshold scored on every element in double.
    Bound by fp64 arithmetic, not by memory: reported against an fp64 instruction rate, not against HBM."""
    name = "exact-mse"
    graph = False
    N_INSTR = 8          # fp64 instructions per element and candidate: div, rint, min, max, mul, sub, mul, add

    def __init__(self):
        self.O, self.C, self.M = 1024, 25088, 128
        self.bits = 4
        self.desc = (f"Section 4.1's MSE on the elements themselves (OCS_CLIP_MSE_EXACT): W [{self.O}, {self.C}] fp32 (a quarter "
                     f"of the fc6-shaped tensor of configs[2]), {N_CAND} candidates, {self.bits}-bit codes; a step = max |W|, the "
                     "scorer, the combine and the quantization; seed 2")
        self.points = [(0.0, self.bits)]
        self.oracle_sample_desc = "the same search on the first 64 rows (1.6 M elements)"

    def setup(self, ocs, torch, dev, host):
        self.ocs, self.torch = ocs, torch
        self.W = host["W"].to(dev)
        self.codes = torch.empty((self.O, ocs.round_up(self.C, 16)), dtype=torch.int8, device=dev)
        self.scal = torch.zeros(2, dtype=torch.float32, device=dev)
        self.ws = torch.empty(int(ocs.lib().ocs_quantize_workspace_bytes(0, N_CAND)) + 256, dtype=torch.uint8, device=dev)
        self.status = ocs.new_status(dev)

    def host_inputs(self):
        c = configs.config3(O=self.O, C=self.C, M=self.M)
        return dict(W=c["W"])

    def ledger(self):
        led = Ledger()
        n = self.O * self.C
        led.add("maxabs_kernel", n=n)
        led.bytes["exact_score_kernel"] = 4 * n
        led.add("quantize_kernel", n=n)
        led.ops = n * N_CAND * self.N_INSTR
        return led

    def step(self):
        ocs = self.ocs
        ocs.ocs_quantize(self.W, self.bits, True, ocs.CLIP_MSE_EXACT, N_CAND, out=(self.codes, self.scal[0:1], self.scal[1:2]),
                         ws=self.ws, dev_status=self.status)

    def e2e_buffers(self, host):
        torch = self.torch
        self.hW = torch.from_numpy(host["W"]).pin_memory()
        self.hC = torch.empty(self.codes.shape, dtype=torch.int8).pin_memory()
        return self.hW.numel() * 4, self.hC.numel()

    def step_e2e(self):
        self.W.copy_(self.hW, non_blocking=True)
        self.step()
        self.hC.copy_(self.codes, non_blocking=True)

    def oracle_sample(self, orc, host):
        W = host["W"][:64]
        t0 = time.perf_counter()
        a = orc.clip_mse_exact(W, self.bits, True, N_CAND)["alpha"]
        orc.quantize(W, self.bits, True, a)
        return time.perf_counter() - t0, 13 * W.size

    def fp64_peak(self, torch, dev):
        """fp64 instruction rate of this GPU, measured: the library's double-precision matrix product (4096^3, best
        of 5) issues one fused multiply-add per two counted operations, so instructions/s = flop/s / 2."""
        a = torch.randn((4096, 4096), dtype=torch.float64, device=dev)
        ms = _time_best(torch, lambda: torch.matmul(a, a), reps=5)
        return 2.0 * 4096 ** 3 / (ms * 1e-3) / 2.0


class SmallFc(Fc6Sweep):
    """configs[0]: one fully-connected layer, no clip search."""
    name = "fc"

    def __init__(self):
        self.O, self.C, self.M = 256, 512, 64
        self.desc = ("configs[0]: fc W [256, 512] fp32, r = 0.05 (26 splits), 8-bit weights no clipping, activations "
                     "[64, 512] 8-bit unsigned; seed 0 (fits in L2: launch-bound)")
        self.points = [(0.05, 8)]

    def host_inputs(self):
        c = configs.config1()
        return dict(W=c["W"], A=c["A"])

    def step(self):
        ocs, C = self.ocs, self.C
        S = ocs.ocs_num_splits(C, 0.05)
        ocs.ocs_split(self.W, S, out=(self.W_out, self.idx_map, None, self.max_abs), ws=self.ws, dev_status=self.status)
        ocs.ocs_quantize(self.W_out, 8, True, ocs.CLIP_NONE, cols=C + S, max_abs_in=self.max_abs[1:2],
                         out=(self.codes, self.scal[0:1], self.scal[1:2]), ws=self.ws, dev_status=self.status)
        ocs.ocs_quantize(self.A, 8, False, ocs.CLIP_NONE, out=(self.a_codes, self.scal[2:3], self.scal[3:4]),
                         ws=self.ws, dev_status=self.status)
        self.gemm(0, S, self.lane_bufs[0])

    def ledger(self):
        led = Ledger()
        O, C, M = self.O, self.C, self.M
        S = configs_num_splits(C, 0.05)
        n = O * (C + S)
        led.add("col_minmax_kernel", N=O * C)
        led.add("split_rows_kernel", N=O * C, n=n)
        led.add("quantize_kernel", n=n)
        led.add("maxabs_kernel", n=M * C)
        led.add("quantize_kernel", n=M * C)
        led.add("transpose_codes_kernel", n=M * C)
        led.add("ocs_gemm_kernel(linear)", rows=M, M=M, C=C, S=S, Nout=O)
        led.ops = 2 * M * O * (C + S)
        return led

    oracle_sample_desc = "the whole step, repeated 200 times"

    def oracle_sample(self, orc, host):
        W, A = host["W"], host["A"]
        t0 = time.perf_counter()
        reps = 200
        for _ in range(reps):
            Wp, idx, _, _ = orc.split(W, 26, 0.0)
            wc, wsc = orc.quantize(Wp, 8, True, orc.maxabs(Wp))
            ac, asc = orc.quantize(A, 8, False, orc.maxabs(A))
            orc.qlinear(ac, False, asc, wc, wsc, idx)
        return (time.perf_counter() - t0) / reps, self.ledger().total


# ----------------------------------------------------------------------------------------------
# Whole-network workloads (configs[3], configs[4]) and the single convolution (configs[1]): reported
# in integer TOP/s of the quantized layers, the unit of the GEMM/conv half of the metric.
class NetWorkload:
    kind = "net"
    l2_note = "activations and weights of most layers fit in L2; nothing is flushed between steps"

    def setup(self, ocs, torch, dev, host):
        self.ocs, self.torch, self.dev = ocs, torch, dev
        from paper_1901_09504_b200 import nets
        self.nets = nets
        self.status = ocs.new_status(dev)
        self.dev_in = {k: torch.from_numpy(v).to(dev) for k, v in self.host_arrays().items()}

    def e2e_buffers(self, host):
        torch = self.torch
        self.pinned = {k: torch.from_numpy(v).pin_memory() for k, v in self.host_arrays().items()}
        out = self.step()
        self.h_out = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        return sum(v.numel() * v.element_size() for v in self.pinned.values()), out.numel() * out.element_size()

    def step_e2e(self):
        for k, v in self.pinned.items():
            self.dev_in[k].copy_(v, non_blocking=True)
        self.h_out.copy_(self.step_graph() if self.graph_obj is not None else self.step(), non_blocking=True)

    # Launch-bound workloads replay their step from a CUDA graph: every library call is stream-ordered and
    # allocation-free, so the whole chain of launches is captured once (after an eager warm-up, which also
    # finishes the library's one-time set-up) and replayed without per-launch host work.
    graph = False
    graph_obj = None

    def make_graph(self):
        torch = self.torch
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(2):
                self.step()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        n0 = self.ocs.ocs_kernel_launches()
        self.graph_obj = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_obj, capture_error_mode="thread_local"):
            self.graph_out = self.step()
        self.graph_launches = int(self.ocs.ocs_kernel_launches() - n0)

    def step_graph(self):
        self.graph_obj.replay()
        return self.graph_out


class ResNet50(NetWorkload):
    name = "resnet50"
    graph = True

    def __init__(self, batch=128, image=224):
        self.batch, self.image = batch, image
        self.desc = (f"configs[3]: ResNet-50 conv/fc stack at random init (folded BN), batch {batch}, input "
                     f"[{batch}, 3, {image}, {image}] fp32, OCS r = 0.01 on every layer, 8-bit weights and activations; "
                     "a step splits, quantizes and packs all 54 layers, then runs the forward pass; seed 3")
        self.oracle_sample_desc = "all 54 layers prepared + forward of 1 image at 64x64"

    def host_inputs(self):
        self.cfg = configs.config4(batch=self.batch, image=self.image)
        return {}

    def host_arrays(self):
        return {"X": self.cfg["X"]}

    def setup(self, ocs, torch, dev, host):
        super().setup(ocs, torch, dev, host)
        # the fp32 weights live on the device; preparing them (split, quantize, pack) is part of every step
        self.Wd = {}
        for spec in self.cfg["layers"] + [self.cfg["fc"]]:
            W, b = self.cfg["params"][spec.name]
            self.Wd[spec.name] = (torch.from_numpy(W).to(dev), torch.from_numpy(b).to(dev))
        self.ops = 0
        for spec in self.cfg["layers"]:
            S = configs_num_splits(spec.C, self.cfg["ratio"])
            self.ops += 2 * self.batch * spec.H_out ** 2 * spec.O * (spec.C + S) * spec.k ** 2
        fc = self.cfg["fc"]
        self.ops += 2 * self.batch * fc.O * (fc.C + configs_num_splits(fc.C, self.cfg["ratio"]))
        self.prep_streams = [torch.cuda.Stream() for _ in range(8)]
        self.ev_start = torch.cuda.Event()
        self.ev_done = [torch.cuda.Event() for _ in self.prep_streams]

    batched = True

    def step(self):
        """Preparation of the 54 layers, then the forward pass.  Batched (default): every layer but the first goes
        through ocs_split_quantize_batch -- five launches for 53 layers -- and the weight reordering of the
        convolutions follows layer by layer.  Otherwise the layers are prepared one by one, spread over a few
        streams so that their small, latency-bound kernels run side by side."""
        nets, cfg, torch = self.nets, self.cfg, self.torch
        if self.batched:
            layers = nets.prepare_resnet50(cfg, self.dev, dev_status=self.status, batched=True, weights=self.Wd)
            return nets.resnet50_forward(cfg, layers, self.dev_in["X"], dev_status=self.status)
        main = torch.cuda.current_stream()
        self.ev_start.record(main)
        layers = {}
        for i, spec in enumerate(cfg["layers"] + [cfg["fc"]]):
            W, b = self.Wd[spec.name]
            side = self.prep_streams[i % len(self.prep_streams)]
            with torch.cuda.stream(side):
                if i < len(self.prep_streams):
                    side.wait_event(self.ev_start)      # after everything the caller's stream has queued so far
                if spec.name == "fc":
                    layers["fc"] = nets.prepare_layer(W.reshape(spec.O, spec.C), b, cfg["ratio"], cfg["w_bits"],
                                                      dev_status=self.status)
                else:
                    layers[spec.name] = nets.prepare_layer(W, b, cfg["ratio"], cfg["w_bits"], conv=True,
                                                           stride=spec.stride, pad=spec.pad, dev_status=self.status)
        for side, ev in zip(self.prep_streams, self.ev_done):
            ev.record(side)
            main.wait_event(ev)
        return nets.resnet50_forward(cfg, layers, self.dev_in["X"], dev_status=self.status)

    def oracle_sample(self, orc, host):
        from oracle import net_oracle
        small = configs.config4(batch=1, image=64)
        t0 = time.perf_counter()
        net_oracle.resnet50(small)
        sec = time.perf_counter() - t0
        ops = sum(2 * s.H_out ** 2 * s.O * (s.C + configs_num_splits(s.C, 0.01)) * s.k ** 2 for s in small["layers"])
        return sec, ops


class Lstm(NetWorkload):
    name = "lstm"
    graph = True
    fold = False

    def __init__(self):
        self.desc = ("configs[4]: 2-layer LSTM language model, hidden 650, vocabulary 33278, batch 20, sequence 35, "
                     "OCS r = 0.02 on W_ih, W_hh and the decoder, 6-bit weights, signed 8-bit activations, per-timestep "
                     "quantized GEMMs; a step prepares the five weight matrices and runs the 35 time steps and the "
                     "decoder; seed 4")
        self.oracle_sample_desc = "the same model with vocabulary 3000, batch 4, 6 time steps"

    def host_inputs(self):
        self.cfg = configs.config5()
        return {}

    def host_arrays(self):
        return {"tokens": self.cfg["tokens"]}

    def setup(self, ocs, torch, dev, host):
        super().setup(ocs, torch, dev, host)
        self.Pd = {k: torch.from_numpy(v).to(dev) for k, v in self.cfg["params"].items()}
        h, V = self.cfg["hidden"], self.cfg["vocab"]
        seq, batch = self.cfg["tokens"].shape
        S = configs_num_splits(h, self.cfg["ratio"])
        self.ops = 2 * (h + S) * (seq * batch * 4 * h * 4 + seq * batch * V)
        self.prep_streams = [torch.cuda.Stream() for _ in range(5)]
        self.ev_start = torch.cuda.Event()
        self.ev_done = [torch.cuda.Event() for _ in self.prep_streams]

    def step(self):
        """The five weight matrices are prepared side by side on their own streams; the decoder's (the largest)
        keeps going beside the time steps and is waited for right before the decoder layer."""
        nets, cfg, P, torch = self.nets, self.cfg, self.Pd, self.torch
        main = torch.cuda.current_stream()
        self.ev_start.record(main)
        layers = {"emb": P["emb"]}
        names = [(f"{nm}{l}", f"{bn}{l}") for l in range(2) for nm, bn in (("W_ih", "b_ih"), ("W_hh", "b_hh"))]
        names.append(("W_dec", "b_dec"))
        for i, (wn, bname) in enumerate(names):
            side = self.prep_streams[i]
            with torch.cuda.stream(side):
                side.wait_event(self.ev_start)
                layers[wn] = nets.prepare_layer(P[wn], P[bname], cfg["ratio"], cfg["w_bits"], dev_status=self.status,
                                                fold=self.fold)
                self.ev_done[i].record(side)
        for i in range(4):
            main.wait_event(self.ev_done[i])
        return nets.lstm_forward(cfg, layers, self.dev_in["tokens"], dev_status=self.status,
                                 before_decoder=lambda: main.wait_event(self.ev_done[4]))

    def oracle_sample(self, orc, host):
        from oracle import net_oracle
        small = configs.config5(vocab=3000, batch=4, seq=6)
        t0 = time.perf_counter()
        net_oracle.lstm(small)
        sec = time.perf_counter() - t0
        h = small["hidden"]
        S = configs_num_splits(h, 0.02)
        return sec, 2 * (h + S) * (6 * 4 * 4 * h * 4 + 6 * 4 * 3000)


class ResNet50PerLayer(ResNet50):
    """The same step with every layer prepared by its own calls (eight streams), for comparison."""
    name = "resnet50-per-layer"
    batched = False


class LstmFolded(Lstm):
    """The same model with the duplicated weight codes folded back into their source channels (6-bit codes:
    the sums fit int8): no gather in any GEMM, identical outputs."""
    name = "lstm-folded"
    fold = True

    def __init__(self):
        super().__init__()
        self.desc = self.desc.replace("configs[4]:", "configs[4] with ocs_fold_duplicates after the quantization:")


class Conv3x3(NetWorkload):
    name = "conv"
    graph = True
    l2_note = "everything fits in L2 (launch-bound); nothing is flushed between steps"

    def __init__(self):
        self.desc = ("configs[1]: conv 3x3 s1 p1, W [256, 256, 3, 3] fp32 (Student-t), input [32, 256, 14, 14], r = 0.02 "
                     f"(6 splits), 6-bit weights with the MSE clip search ({N_CAND} candidates), 8-bit unsigned activations; "
                     "a step splits, searches, quantizes, packs, converts the input layout and runs the convolution; seed 1")
        self.oracle_sample_desc = "the same layer on 4 of the 32 images"

    def host_inputs(self):
        self.cfg = configs.config2()
        return {}

    def host_arrays(self):
        return {"X": self.cfg["X"]}

    def setup(self, ocs, torch, dev, host):
        super().setup(ocs, torch, dev, host)
        self.W = torch.from_numpy(self.cfg["W"]).to(dev)
        self.ops = 2 * 32 * 14 * 14 * 256 * (256 + 6) * 9

    def step(self):
        nets, ocs = self.nets, self.ocs
        L = nets.prepare_layer(self.W, None, 0.02, 6, ocs.CLIP_MSE, conv=True, stride=1, pad=1, dev_status=self.status)
        x = ocs.ocs_nchw_to_nhwc(self.dev_in["X"])
        return nets.conv_forward(L, x, a_signed=False, dev_status=self.status)

    def oracle_sample(self, orc, host):
        c = configs.config2(batch=4)
        t0 = time.perf_counter()
        Wp, idx, _, _ = orc.split(c["W"], 6)
        alpha = orc.clip_mse(Wp, 6, True, N_BINS, N_CAND)["alpha"]
        wc, ws = orc.quantize(Wp, 6, True, alpha)
        xh = orc.nchw_to_nhwc(c["X"])
        xc, xs = orc.quantize(xh, 8, False, orc.maxabs(xh))
        orc.qconv(xc, False, xs, wc, ws, idx, 1, 1)
        return time.perf_counter() - t0, 2 * 4 * 14 * 14 * 256 * (256 + 6) * 9


NET_METRIC = "OCS quantized layers int8 TOP/s (whole step: split + quantize + pack of every layer, then the forward pass)"


# ----------------------------------------------------------------------------------------------
def sample_clocks_start():
    q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")
    try:
        return subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "100"],
                                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
    except OSError:
        return None


def sample_clocks_stop(proc, gpu_index):
    if proc is None:
        return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
    time.sleep(0.15)
    proc.terminate()
    try:
        out = proc.communicate(timeout=5)[0]
    except subprocess.TimeoutExpired:
        proc.kill()
        out = ""
    sm, mx, reasons = [], [], set()
    for line in out.splitlines():
        f = [x.strip() for x in line.split(",")]
        if len(f) < 9 or not f[0].isdigit() or int(f[0]) != gpu_index:
            continue
        try:
            sm.append(float(f[1]))
            mx.append(float(f[2]))
        except ValueError:
            continue
        for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
            if val.lower().startswith("active"):
                reasons.add(name)
    return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                reasons=sorted(reasons), samples=len(sm))


def run_reference(args, wl):
    """The CPU checker, as it stands, on a bounded sample of the same workload (host cores only)."""
    from oracle import oracle as orc
    orc.build()
    host = wl.host_inputs()
    for _ in range(min(args.warmup, 1)):
        wl.oracle_sample(orc, host)
    times, nbytes = [], 0
    for _ in range(args.steps):
        t, nbytes = wl.oracle_sample(orc, host)
        times.append(t)
    sec = sum(times) / len(times)
    net = getattr(wl, "kind", "") == "net"
    val = nbytes / sec / (1e12 if net else 1e9)       # network workloads count integer ops, the others bytes
    unit = "TOPS" if net else "GB/s"
    line = dict(impl="reference", metric=NET_METRIC if net else METRIC, value=val, unit=unit, n_gpus=args.gpus,
                steps=args.steps,
                warmup=min(args.warmup, 1), ms_per_step=sec * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f32 (split, clip search, quantize) + int8 x int8 -> int32 (GEMM)", data="synthetic",
                config=dict(workload=wl.desc, sample=wl.oracle_sample_desc),
                cpu_baseline=dict(value=val, unit=unit, cores=orc.threads(), kind="oracle",
                                  sample=wl.oracle_sample_desc),
                e2e=dict(value=val, unit=unit, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


METRIC = "OCS hot path (split + clip search + quantize + int8 GEMM with idx_map gather) algorithmic HBM GB/s"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="fc6", choices=["fc6", "fc6-fused", "fc6-small", "fc", "conv", "resnet50", "lstm", "lstm-folded", "act-ocs", "exact-mse", "resnet50-per-layer"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-tensor-probe", action="store_true")
    ap.add_argument("--lanes", type=int, default=0,
                    help="sweep points in flight in the fc6 sweeps (0: the workload's default; 1 gives the launch "
                         "order the ncu summaries under profiles/ index into)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    wl = {"fc6": Fc6Sweep, "fc6-fused": Fc6Fused, "fc6-small": lambda: Fc6Sweep(small=True), "fc": SmallFc, "conv": Conv3x3,
          "resnet50": ResNet50, "resnet50-per-layer": ResNet50PerLayer, "lstm": Lstm, "lstm-folded": LstmFolded, "act-ocs": ActOcs, "exact-mse": ExactMse}[args.workload]()
    net = getattr(wl, "kind", "") == "net"
    if args.lanes > 0 and hasattr(wl, "LANES"):
        wl.LANES = args.lanes

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, wl)
        return

    host = wl.host_inputs()

    # the CPU checker first, before the first GPU call (rank 0, one GPU only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import oracle as orc
        orc.build()
        sec, nbytes = wl.oracle_sample(orc, host)
        cpu = dict(value=nbytes / sec / (1e12 if net else 1e9), unit="TOPS" if net else "GB/s", cores=orc.threads(),
                   kind="oracle", sample=wl.oracle_sample_desc, seconds=sec)

    import torch
    import torch.distributed as dist

    import paper_1901_09504_b200 as ocs
    from paper_1901_09504_b200 import build as ocs_build

    ocs_build.build()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    wl.setup(ocs, torch, dev, {k: torch.from_numpy(v) for k, v in host.items()})
    led = Ledger() if net else wl.ledger()
    if net:
        led.ops = wl.ops
    pk = peaks()

    def timed(fn, steps, warmup):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n0 = ocs.ocs_kernel_launches()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        ms = reduce_max(e0.elapsed_time(e1), world, dev)
        return ms / steps, (ocs.ocs_kernel_launches() - n0) // steps

    use_graph = bool(getattr(wl, "graph", False))
    if use_graph:
        try:
            wl.make_graph()
        except RuntimeError as e:      # capture refused (another thread's CUDA call, an old driver): eager launches
            print(f"bench: CUDA graph capture failed ({e}); timing eager launches", file=sys.stderr)
            torch.cuda.synchronize()
            wl.graph_obj = None
            use_graph = False
    clk = sample_clocks_start() if rank == 0 else None
    ms_step, launches = timed(wl.step_graph if use_graph else wl.step, args.steps, args.warmup)
    if use_graph:
        launches = wl.graph_launches      # the library's counter advances at capture, not at replay
    clocks = sample_clocks_stop(clk, local_rank) if rank == 0 else None
    assert ocs.ocs_poll_status(wl.status) == 0, "device status word set during the timed steps"

    # second pass over the same K steps with per-kernel CUDA events (the launches are identical)
    barrier()
    ocs.ocs_trace_start(launches * args.steps + 16)
    lanes = getattr(wl, "lanes", 1)
    if lanes > 1:
        wl.lanes = 1          # one kernel at a time: a launch's duration is then its own
    for _ in range(args.steps):
        wl.step()
    if lanes > 1:
        wl.lanes = lanes
    trace = ocs.ocs_trace_stop()
    barrier()

    # end to end: inputs start in pinned host memory, results end there
    h2d, d2h = wl.e2e_buffers(host)
    ms_e2e, _ = timed(wl.step_e2e, args.steps, 3)

    # the tensor-bound half of the metric (rank 0, one GPU, default workload): measured int8 peak and three
    # contraction timings
    probe = None
    if rank == 0 and world == 1 and wl.name == "fc6" and not args.no_tensor_probe:
        wl.release()
        probe = tensor_probe(ocs, torch, dev)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    kernels = {}
    for name, (cnt, ms) in sorted(trace.items(), key=lambda kv: -kv[1][1]):
        nb = led.bytes.get(name, 0) * args.steps
        kernels[name] = dict(launches_per_step=cnt // args.steps, ms_per_step=ms / args.steps,
                             share=ms / max(sum(t for _, t in trace.values()), 1e-12),
                             algorithmic_gbs=(nb / (ms * 1e-3) / 1e9) if ms > 0 and nb else None)
    top = next(iter(kernels))
    top_cnt, top_ms = trace[top]
    if probe and probe.get("int8_peak_tops"):
        int8_peak, int8_note = probe["int8_peak_tops"], probe["int8_peak_note"]
    else:
        int8_peak = pk["bf16_burst"] * INT8_OVER_BF16
        int8_note = f"{pk['source']} bf16 burst x {INT8_OVER_BF16:g} (nominal int8:bf16 ratio; no int8 measurement in this run)"
    gemm_name = "ocs_gemm_kernel(linear)"
    gemm_ms = sum(trace.get(k, (0, 0.0))[1] for k in ("ocs_gemm_kernel(linear)", "ocs_gemm_kernel(conv)"))
    gemm_tops = (led.ops * args.steps / (gemm_ms * 1e-3) / 1e12) if gemm_ms > 0 else None
    sq_names = ("col_minmax_kernel", "split_rows_kernel", "split_scatter_kernel", "hist_kernel", "quantize_kernel", "maxabs_kernel",
                "split_hist_kernel", "split_quantize_kernel", "transpose_codes_kernel")
    sq_ms = sum(trace[k][1] for k in sq_names if k in trace) + sum(
        trace[k][1] for k in ("split_plan_kernel", "score_kernel", "pick_kernel") if k in trace)
    sq_bytes = sum(led.bytes.get(k, 0) for k in sq_names) * args.steps
    sq_gbs = sq_bytes / (sq_ms * 1e-3) / 1e9 if sq_ms > 0 else None
    top_bytes = led.bytes.get(top, 0)
    if net and top.startswith("ocs_gemm_kernel"):
        # the contraction: integer ops of the step over the kernel's traced time, against the int8 peak
        ach = led.ops * args.steps / (top_ms * 1e-3) / 1e12
        roofline = dict(kernel=top, bound="tensor", achieved=ach, peak=int8_peak, unit="TOP/s", frac=ach / int8_peak,
                        traffic=None, peak_source=int8_note,
                        avg_launch_ms=top_ms / top_cnt, note="ops of every quantized layer of the step (linear and conv "
                        "launches share one kernel); layers with few channels are bound by their output traffic, not by "
                        "the tensor pipe",
                        timed="second pass over the same steps with CUDA events around every kernel launch")
    elif top == "exact_score_kernel":
        # bound by fp64 arithmetic: counted fp64 instructions of the scorer over its traced time, against the fp64
        # instruction rate measured in this run
        peak_i = wl.fp64_peak(torch, dev) / 1e12
        ach = led.ops * args.steps / (top_ms * 1e-3) / 1e12
        roofline = dict(kernel=top, bound="alu", achieved=ach, peak=peak_i, unit="T fp64 instr/s", frac=ach / peak_i,
                        traffic=None, peak_source="measured in this run: fp64 matrix product 4096^3 (library), flop/s / 2",
                        avg_launch_ms=top_ms / top_cnt,
                        note=f"{wl.N_INSTR} counted instructions per element and candidate (the division alone expands to "
                        "a dozen machine instructions, so the fraction understates the pipe's load)",
                        timed="second pass over the same steps with CUDA events around every kernel launch")
    elif top_bytes:
        roof_achieved = top_bytes * args.steps / (top_ms * 1e-3) / 1e9
        roofline = dict(kernel=top, bound="hbm", achieved=roof_achieved, peak=pk["hbm"], unit="GB/s",
                        frac=roof_achieved / pk["hbm"], traffic=ncu_traffic(top, top_bytes * args.steps / top_cnt),
                        traffic_unit="bytes per launch (ncu dram read + write, scaled from the r = 0.1 launch)",
                        peak_source=f"of {pk['source']}",
                        avg_launch_ms=top_ms / top_cnt,
                        timed="second pass over the same steps with CUDA events around every kernel launch")
    else:   # a dependent-step kernel (greedy plan, scoring): no bytes to speak of
        roofline = dict(kernel=top, bound="latency", achieved=None, peak=None, unit="GB/s", frac=None, traffic=None,
                        avg_launch_ms=top_ms / top_cnt,
                        timed="second pass over the same steps with CUDA events around every kernel launch")

    if net:
        scale = lambda ms: led.ops * world / (ms * 1e-3) / 1e12      # whole-job integer TOP/s
        unit, metric = "TOPS", NET_METRIC
    else:
        scale = lambda ms: aggregate_gbs(led.total, world, ms)
        unit, metric = "GB/s", METRIC
    value = scale(ms_step)
    line = dict(
        metric=metric, value=value, unit=unit, n_gpus=world, steps=args.steps, warmup=args.warmup,
        ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None,
        dtype="f32 (split, clip search, quantize) + int8 x int8 -> int32 (GEMM)", data="synthetic",
        config=dict(workload=wl.desc, l2=getattr(wl, "l2_note", None) or (
            "inputs larger than L2 (no flush)" if wl.name.startswith("fc6") else "inputs fit in L2; nothing is flushed between steps"),
                    bytes_per_step=led.total, int_ops_per_step=led.ops,
                    launch=("the step's kernel launches are captured once in a CUDA graph and replayed"
                            if use_graph else "eager launches"),
                    **({"lanes": f"{wl.lanes} sweep points in flight on {wl.lanes} streams (independent points; the "
                                 "per-kernel timings are taken one kernel at a time)"} if getattr(wl, "lanes", 1) > 1 else {})),
        parts=dict(split_quantize_gbs=sq_gbs, split_quantize_frac_of_hbm=(sq_gbs / pk["hbm"]) if sq_gbs else None,
                   gemm_tops=gemm_tops, gemm_frac_of_int8_peak=(gemm_tops / int8_peak) if gemm_tops else None,
                   int8_peak_tops=int8_peak, int8_peak_note=int8_note,
                   gemm_algorithmic_gbs=kernels.get(gemm_name, {}).get("algorithmic_gbs"),
                   gemm_frac_of_hbm=(kernels.get(gemm_name, {}).get("algorithmic_gbs") or 0) / pk["hbm"] or None,
                   **({k: v for k, v in probe.items() if k.endswith("_tops") and k != "int8_peak_tops"} if probe else {}),
                   **({k.replace("_tops", "_frac_of_int8_peak"): v / int8_peak for k, v in probe.items()
                       if k.endswith("_tops") and k != "int8_peak_tops" and v} if probe else {})),
        roofline=roofline,
        kernels=kernels,
        cpu_baseline=cpu,
        e2e=dict(value=scale(ms_e2e), unit=unit, ms_per_step=ms_e2e,
                 h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h),
        gpu_launches=int(launches) * args.steps,
        clocks=clocks,
    )
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
