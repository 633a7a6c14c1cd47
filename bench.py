#!/usr/bin/env python
"""Benchmark of the SNIP mixed-precision linear hot path on B200.

A step = one transformer block of the Llama-7B-shaped workload (tokens 16384; fused QKV, O,
gate, up, down): for every linear the quantization of X, W and dY (each read once, both quantized
copies written: the tile kind of each of the two GEMMs that consume the tensor, with fused error-norm
statistics per copy) and the forward, input-gradient and weight-gradient GEMMs, run once with every
GEMM in FP4 E2M1 and once with every GEMM in FP8 E4M3.  `--quantizer single` runs one quantizer call
per GEMM operand instead (six reads per linear).

Prints ONE JSON line (rank 0).  `value` is GEMM TFLOP/s (2*M*N*K per GEMM) over the whole step,
quantizers and statistics included, with inputs resident in HBM.  `roofline` describes the
dominant kernel family (the GEMM kernels of the slower format), timed with CUDA events around
each launch inside the timed region.  `e2e` repeats the step through the snip_linear_* calls with
the inputs starting in pinned host memory: every step copies all of them to the device (on a copy
stream, into one of two input sets, so that the copy of one step overlaps the kernels of the
previous one) and reads the statistics back.  `cpu_baseline` times the CPU oracle on a bounded
sample on this machine's host cores.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload 7b|1b|small|3b|70b]
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

FMT_BF16, FMT_FP8, FMT_FP4 = 0, 1, 2
FMT_NAME = {0: "bf16", 1: "fp8_e4m3", 2: "fp4_e2m1"}
NOMINAL_RATIO = {0: 1.0, 1: 2.0, 2: 4.0}   # dense tensor peak relative to bf16
# DRAM bytes (read + write) of one GEMM launch on the fused-QKV forward shape 16384 x 12288 x 4096, from the
# ncu captures summarised in profiles/gemm_kernel_gemm_<fmt>_fwd_16384x12288x4096.md (algorithmic: 519 MB FP8,
# 461 MB FP4).  Reported as `traffic` of the roofline object together with the shape it belongs to.
NCU_TRAFFIC = {1: 823.5e6, 2: 493.9e6}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "25", "-i", str(self.gpu)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        for ln in self.lines:
            f = [v.strip() for v in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        busy = [c for c, p in zip(sm, power) if p > 300] or sm
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------

WORKLOADS = {
    # name: (config index in paper_2602_01410_b200.workloads.CONFIGS, tokens override)
    "7b": (3, None),
    "1b": (1, None),
    "small": (0, None),
    # table-driven precision mix: every GEMM takes the tag the configuration's seeded table gives it
    "3b": (2, None),
    "70b": (4, None),
}
TAGGED_LAYERS = 4   # layers of a table-driven workload kept resident and run per step


def make_device_inputs(cfg, torch, device, seed):
    """bf16 tensors of one block, drawn on the device with the recipe of workloads.py (normal X
    with outlier channels, N(0,0.02) W, row-scaled dY).  The bench needs the distribution, not
    the exact bytes; parity tests use the host generators."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    M = cfg.M
    lin = []
    for li, L in enumerate(cfg.linears):
        x = torch.randn(M, L.K, generator=g, device=device, dtype=torch.float32)
        n_out = max(1, int(-(-cfg.outlier_frac * L.K // 1)))
        cols = torch.randperm(L.K, generator=g, device=device)[:n_out]
        x[:, cols] *= cfg.outlier_scale
        w = torch.randn(L.N, L.K, generator=g, device=device, dtype=torch.float32) * 0.02
        dy = torch.randn(M, L.N, generator=g, device=device, dtype=torch.float32) * 1e-3
        dy *= torch.exp(torch.randn(M, 1, generator=g, device=device, dtype=torch.float32))
        lin.append((x.to(torch.bfloat16), w.to(torch.bfloat16), dy.to(torch.bfloat16)))
        del x, w, dy
    return lin


class Step:
    """Device buffers and the call sequence of one step."""

    def __init__(self, api, torch, cfg, device, formats, dual=True):
        self.api, self.torch, self.cfg, self.formats, self.dual = api, torch, cfg, formats, dual
        self.inputs = make_device_inputs(cfg, torch, device, 260201410)
        M = cfg.M
        self.out = []
        ws_bytes = 0
        for L in cfg.linears:
            self.out.append((torch.empty(M, L.N, dtype=torch.bfloat16, device=device),
                             torch.empty(M, L.K, dtype=torch.bfloat16, device=device),
                             torch.empty(L.N, L.K, dtype=torch.bfloat16, device=device)))
            for op in (api.OP_FWD, api.OP_DGRAD, api.OP_WGRAD):
                for f in formats:
                    ws_bytes = max(ws_bytes, api.snip_workspace_size(op, M, L.N, L.K, f, f)[1])
            for f in formats:
                for pow2 in (False, True):
                    ws_bytes = max(ws_bytes, api.snip_linear_fwd_bwd_workspace(M, L.N, L.K, f, f, f, pow2))
        self.ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=device)
        n_gemm = len(cfg.linears) * 3 * len(formats)
        self.stats = torch.zeros(n_gemm * 2, 32, dtype=torch.uint8, device=device)  # one 16-byte-aligned snip_stats_t per row
        self.stats6 = torch.zeros(len(cfg.linears) * len(formats), 6 * 24, dtype=torch.uint8, device=device)
        self.flops = sum(2.0 * M * L.N * L.K * 3 for L in cfg.linears) * len(formats)
        # per GEMM: dual = 1 quantizer + 1 statistics reduction + 1 GEMM; single = 2 + 2 + 1
        self.launches_per_step = n_gemm * (3 if dual else 5)

    # -- the step through the snip_linear_* entry points (what a user calls) -------------
    def run_linear_calls(self, mx=False, inputs=None, before=None):
        """One step through the per-layer entry points.  `inputs` replaces the resident input tensors;
        `before(j)` runs ahead of the first call that reads linear j's inputs (end-to-end leg: wait for their copy)."""
        api = self.api
        i = 0
        inputs = self.inputs if inputs is None else inputs
        if self.dual:
            lib, p, st = api._lib, api._p, api._stream()
            for fi, f in enumerate(self.formats):
                for j, ((x, w, dy), (y, dx, dw)) in enumerate(zip(inputs, self.out)):
                    if before is not None and fi == 0:
                        before(j)
                    M, K = x.shape
                    N = w.shape[0]
                    api._check("snip_linear_fwd_bwd", lib.snip_linear_fwd_bwd(p(x), p(w), p(dy), p(y), p(dx), p(dw), M, N, K, f, f, f, api.OUT_BF16,
                                                                              int(mx), 0, 0, p(self.stats6[i]), p(self.ws), self.ws.numel(), st))
                    i += 1
            return
        for fi, f in enumerate(self.formats):
            for j, ((x, w, dy), (y, dx, dw)) in enumerate(zip(inputs, self.out)):
                if before is not None and fi == 0:
                    before(j)
                M, K = x.shape
                N = w.shape[0]
                lib, p, st = api._lib, api._p, api._stream()
                sa, sb = self.stats[2 * i], self.stats[2 * i + 1]
                api._check("snip_linear_fwd", lib.snip_linear_fwd(p(x), p(w), p(y), M, N, K, f, f, api.OUT_BF16, p(sa), p(sb), p(self.ws), self.ws.numel(), st)); i += 1
                sa, sb = self.stats[2 * i], self.stats[2 * i + 1]
                api._check("snip_linear_dgrad", lib.snip_linear_dgrad(p(dy), p(w), p(dx), M, N, K, f, f, api.OUT_BF16, p(sa), p(sb), p(self.ws), self.ws.numel(), st)); i += 1
                sa, sb = self.stats[2 * i], self.stats[2 * i + 1]
                api._check("snip_linear_wgrad", lib.snip_linear_wgrad(p(dy), p(x), p(dw), M, N, K, f, f, api.OUT_BF16, 0, p(sa), p(sb), p(self.ws), self.ws.numel(), st)); i += 1

    # -- the same device work as separate quantize / GEMM calls, so that CUDA events can bracket
    #    every GEMM launch inside the timed region ------------------------------------------------
    def _alloc_decomposed(self):
        api, torch = self.api, self.torch
        cb = sb = wb = 0
        M = self.cfg.M
        for L in self.cfg.linears:
            for (r, c) in ((M, L.K), (L.N, L.K), (M, L.N)):
                for blk in (api.BLOCK_ROW, api.BLOCK_COL, api.BLOCK_BLK):
                    a, b, w = api.snip_quantize_sizes(r, c, FMT_FP8, blk, api.Q_STATS)
                    cb, sb, wb = max(cb, a), max(sb, b), max(wb, w)
        dev = self.ws.device
        nbuf = 6 if self.dual else 2
        self.codes = [torch.empty(cb, dtype=torch.uint8, device=dev) for _ in range(nbuf)]
        self.scales = [torch.empty(sb, dtype=torch.float32, device=dev) for _ in range(nbuf)]   # room for the 32-long tile kinds (4 x the scales)
        self.qws = torch.empty(2 * wb, dtype=torch.uint8, device=dev)
        self.sf = [torch.empty(cb // 32 + 4096, dtype=torch.uint8, device=dev) for _ in range(nbuf)]   # UE8M0 atoms (power-of-two option)
        # GEMM workspace: the size the library reports for a weight-gradient product (room for its contraction slices)
        self.gws = torch.zeros(max(1024, api.snip_workspace_size(api.OP_WGRAD, 16384, 4096, 4096, api.FMT_FP8_E4M3, api.FMT_FP8_E4M3)[0]), dtype=torch.uint8, device=dev)

    def run_decomposed(self, events=None, mx=False, qevents=None):
        api, torch = self.api, self.torch
        if not hasattr(self, "codes"):
            self._alloc_decomposed()
        lib, p, st = api._lib, api._p, api._stream()
        T = api.Q_TRANSPOSED
        i = 0

        def quant(x, fmt, block, flags, slot, stats):
            r, c = x.shape
            if mx:
                api._check("snip_quantize_mx", lib.snip_quantize_mx(p(x), r, c, c, fmt, block, flags | api.Q_STATS, p(self.codes[slot]), p(self.scales[slot]),
                                                                    p(self.sf[slot]), p(stats), p(self.qws), self.qws.numel(), st))
            else:
                api._check("snip_quantize", lib.snip_quantize(p(x), r, c, c, fmt, block, flags | api.Q_STATS, p(self.codes[slot]), p(self.scales[slot]),
                                                              p(stats), None, p(self.qws), self.qws.numel(), st))

        def dual(x, fmt, kind, slot, stats_row):
            r, c = x.shape
            outs = [api.QOut(fmt, 0, p(self.codes[slot + j]), p(self.scales[slot + j]), p(self.sf[slot + j]) if mx else None,
                             p(stats_row[24 * j:24 * j + 24]), 0) for j in range(2)]
            if qevents is not None:
                q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                q0.record()
            api._check("snip_quantize_dual", lib.snip_quantize_dual(p(x), r, c, c, kind, 1 if mx else 0, outs[0], outs[1], p(self.qws), self.qws.numel(), st))
            if qevents is not None:
                q1.record()
                # algorithmic bytes: one bf16 read, two code + scale outputs
                qevents.append((fmt, (2.0 + 2.0 * ((1.0 if fmt == FMT_FP8 else 0.5) + 4.0 / 128.0)) * r * c, q0, q1))

        def gemm(op, fmt, ra, ca, blka, ta, rb, cb_, blkb, tb, out, flops, sa=0, sb_=1):
            a = api.make_qtensor(self.codes[sa], self.scales[sa], ra, ca, fmt, blka, ta)
            b = api.make_qtensor(self.codes[sb_], self.scales[sb_], rb, cb_, fmt, blkb, tb)
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            if mx:
                api._check("snip_gemm_mx", lib.snip_gemm_mx(op, a, p(self.sf[sa]), b, p(self.sf[sb_]), p(out), api.OUT_BF16, p(self.gws), self.gws.numel(), st))
            else:
                api._check("snip_gemm_quantized", lib.snip_gemm_quantized(op, a, b, p(out), api.OUT_BF16, 0, p(self.gws), self.gws.numel(), st))
            if events is not None:
                e1.record()
                events.append((fmt, op, flops, e0, e1))

        for f in self.formats:
            for (x, w, dy), (y, dx, dw) in zip(self.inputs, self.out):
                M, K = x.shape
                N = w.shape[0]
                fl = 2.0 * M * N * K
                # mx == 2: power-of-two scales on 32-long tiles (1x32 as stored, 32x1 transposed, for W as well)
                R, C, B = (api.BLOCK_ROW32, api.BLOCK_COL32, None) if mx == 2 else (api.BLOCK_ROW, api.BLOCK_COL, api.BLOCK_BLK)
                if self.dual and mx == 2:
                    srow = self.stats6[i // 3].view(-1)
                    i += 3
                    k32 = api.DUAL_ROW32_COL32T
                    dual(x, f, k32, 0, srow[0:48]); dual(w, f, k32, 2, srow[48:96])
                    gemm(api.OP_FWD, f, M, K, R, 0, N, K, R, 0, y, fl, 0, 2)
                    dual(dy, f, k32, 4, srow[96:144])
                    gemm(api.OP_DGRAD, f, M, N, R, 0, N, K, C, 1, dx, fl, 4, 3)
                    gemm(api.OP_WGRAD, f, M, N, C, 1, M, K, C, 1, dw, fl, 5, 1)
                    continue
                if mx == 2:
                    quant(x, f, R, 0, 0, self.stats[2 * i]); quant(w, f, R, 0, 1, self.stats[2 * i + 1]); i += 1
                    gemm(api.OP_FWD, f, M, K, R, 0, N, K, R, 0, y, fl)
                    quant(dy, f, R, 0, 0, self.stats[2 * i]); quant(w, f, C, T, 1, self.stats[2 * i + 1]); i += 1
                    gemm(api.OP_DGRAD, f, M, N, R, 0, N, K, C, 1, dx, fl)
                    quant(dy, f, C, T, 0, self.stats[2 * i]); quant(x, f, C, T, 1, self.stats[2 * i + 1]); i += 1
                    gemm(api.OP_WGRAD, f, M, N, C, 1, M, K, C, 1, dw, fl)
                    continue
                if self.dual:
                    # slots: 0 X/ROW, 1 X/COL^T, 2 W/BLK, 3 W/BLK^T, 4 dY/ROW, 5 dY/COL^T
                    srow = self.stats6[i // 3].view(-1)
                    i += 3
                    dual(x, f, api.DUAL_ROW_COLT, 0, srow[0:48]); dual(w, f, api.DUAL_BLK_BLKT, 2, srow[48:96])
                    gemm(api.OP_FWD, f, M, K, api.BLOCK_ROW, 0, N, K, api.BLOCK_BLK, 0, y, fl, 0, 2)
                    dual(dy, f, api.DUAL_ROW_COLT, 4, srow[96:144])
                    gemm(api.OP_DGRAD, f, M, N, api.BLOCK_ROW, 0, N, K, api.BLOCK_BLK, 1, dx, fl, 4, 3)
                    gemm(api.OP_WGRAD, f, M, N, api.BLOCK_COL, 1, M, K, api.BLOCK_COL, 1, dw, fl, 5, 1)
                    continue
                quant(x, f, api.BLOCK_ROW, 0, 0, self.stats[2 * i]); quant(w, f, api.BLOCK_BLK, 0, 1, self.stats[2 * i + 1]); i += 1
                gemm(api.OP_FWD, f, M, K, api.BLOCK_ROW, 0, N, K, api.BLOCK_BLK, 0, y, fl)
                quant(dy, f, api.BLOCK_ROW, 0, 0, self.stats[2 * i]); quant(w, f, api.BLOCK_BLK, T, 1, self.stats[2 * i + 1]); i += 1
                gemm(api.OP_DGRAD, f, M, N, api.BLOCK_ROW, 0, N, K, api.BLOCK_BLK, 1, dx, fl)
                quant(dy, f, api.BLOCK_COL, T, 0, self.stats[2 * i]); quant(x, f, api.BLOCK_COL, T, 1, self.stats[2 * i + 1]); i += 1
                gemm(api.OP_WGRAD, f, M, N, api.BLOCK_COL, 1, M, K, api.BLOCK_COL, 1, dw, fl)


def run_two_level(step, events=None, qevents=None):
    """The FP4 half of the step under the two-level (NVFP4-style) option: per linear three one-read two-output
    quantizer calls (statistics on) and the three block-scaled GEMMs; the per-tensor bounds are the tensors' maxima,
    computed once outside the timed region (a training loop would carry them over from the previous step)."""
    api, torch = step.api, step.torch
    if not hasattr(step, "codes"):
        step._alloc_decomposed()
    if not hasattr(step, "nv_bounds"):
        step.nv_bounds = [tuple(t.float().abs().max().reshape(1).contiguous() for t in trip) for trip in step.inputs]
        step.nv_sf = [torch.empty(api.snip_quantize_nvfp4_sizes(step.cfg.M, max(max(L.N, L.K) for L in step.cfg.linears))[1] + 4096, dtype=torch.uint8,
                                  device=step.ws.device) for _ in range(6)]
    lib, p, st = api._lib, api._p, api._stream()
    F4 = api.FMT_FP4_E2M1
    R, C = api.BLOCK_ROW16, api.BLOCK_COL16

    def dual(x, bound, slot, stats_row):
        r, c = x.shape
        if qevents is not None:
            q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            q0.record()
        api._check("snip_quantize_nvfp4_dual", lib.snip_quantize_nvfp4_dual(p(x), r, c, c, p(bound), p(step.codes[slot]), p(step.nv_sf[slot]), p(stats_row[0:24]),
                                                                         p(step.codes[slot + 1]), p(step.nv_sf[slot + 1]), p(stats_row[24:48]),
                                                                         0, 0, p(step.qws), step.qws.numel(), st))
        if qevents is not None:
            q1.record()
            qevents.append((F4, (2.0 + 2.0 * (0.5 + 1.0 / 16.0)) * r * c, q0, q1))   # one bf16 read, two code + scale-byte outputs

    def gemm(op, ra, ca, blka, ta, sa, ba, rb, cb_, blkb, tb, sb_, bb, out, flops):
        a = api.make_qtensor(step.codes[sa], None, ra, ca, F4, blka, ta)
        b = api.make_qtensor(step.codes[sb_], None, rb, cb_, F4, blkb, tb)
        if events is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
        api._check("snip_gemm_nvfp4", lib.snip_gemm_nvfp4(op, a, p(step.nv_sf[sa]), p(ba), b, p(step.nv_sf[sb_]), p(bb), p(out), api.OUT_BF16,
                                                       p(step.gws), step.gws.numel(), st))
        if events is not None:
            e1.record()
            events.append((F4, op, flops, e0, e1))

    for i, (((x, w, dy), (y, dx, dw)), (bx, bw, bdy)) in enumerate(zip(zip(step.inputs, step.out), step.nv_bounds)):
        M, K = x.shape
        N = w.shape[0]
        fl = 2.0 * M * N * K
        srow = step.stats6[i].view(-1)
        # slots: 0 X/1x16, 1 X/16x1^T, 2 W/1x16, 3 W/16x1^T, 4 dY/1x16, 5 dY/16x1^T
        dual(x, bx, 0, srow[0:48]); dual(w, bw, 2, srow[48:96])
        gemm(api.OP_FWD, M, K, R, 0, 0, bx, N, K, R, 0, 2, bw, y, fl)
        dual(dy, bdy, 4, srow[96:144])
        gemm(api.OP_DGRAD, M, N, R, 0, 4, bdy, N, K, C, 1, 3, bw, dx, fl)
        gemm(api.OP_WGRAD, M, N, C, 1, 5, bdy, M, K, C, 1, 1, bx, dw, fl)


class TaggedStep:
    """A table-driven workload (3B: each GEMM drawn FP4 / FP8 / BF16; 70B slice: at least 80 % of the linear-layer
    FLOPs in FP4, the rest FP8): `layers` layers resident, every linear's forward, input-gradient and weight-gradient
    GEMM with the tag of that GEMM on both operands, statistics on.  A linear whose three tags are all quantized formats
    goes through snip_linear_fwd_bwd (each tensor read once, both of its copies and their statistics written); one with a
    BF16 tag through snip_linear_fwd / dgrad / wgrad."""

    def __init__(self, api, torch, cfg, device, layers):
        from paper_2602_01410_b200 import workloads as wl
        self.api, self.torch, self.cfg, self.layers = api, torch, cfg, layers
        self.tags = wl.precision_tags(cfg)[:layers]
        self.inputs = [make_device_inputs(cfg, torch, device, 260201410 + 17 * l) for l in range(layers)]
        M = cfg.M
        self.out = [(torch.empty(M, L.N, dtype=torch.bfloat16, device=device), torch.empty(M, L.K, dtype=torch.bfloat16, device=device),
                     torch.empty(L.N, L.K, dtype=torch.bfloat16, device=device)) for L in cfg.linears]
        ws_bytes = 0
        for L in cfg.linears:
            for op in (api.OP_FWD, api.OP_DGRAD, api.OP_WGRAD):
                for f in (FMT_BF16, FMT_FP8, FMT_FP4):
                    ws_bytes = max(ws_bytes, api.snip_workspace_size(op, M, L.N, L.K, f, f)[1])
        for L in cfg.linears:
            ws_bytes = max(ws_bytes, api.snip_linear_fwd_bwd_workspace(M, L.N, L.K, FMT_FP8, FMT_FP8, FMT_FP8, 0))
        self.ws = torch.zeros(ws_bytes, dtype=torch.uint8, device=device)
        n_gemm = layers * len(cfg.linears) * 3
        self.stats = torch.zeros(n_gemm * 2, 32, dtype=torch.uint8, device=device)
        self.stats6 = torch.zeros(layers * len(cfg.linears), 6 * 24, dtype=torch.uint8, device=device)
        self.flops = layers * sum(2.0 * M * L.N * L.K * 3 for L in cfg.linears)
        self.flops_by_fmt = {}
        for l in range(layers):
            for j, L in enumerate(cfg.linears):
                for gi in range(3):
                    f = int(self.tags[l, j, gi])
                    self.flops_by_fmt[f] = self.flops_by_fmt.get(f, 0.0) + 2.0 * M * L.N * L.K
        # a linear through snip_linear_fwd_bwd: 3 two-output quantizers + 3 reductions + 3 GEMMs; through the three separate calls, per GEMM:
        # 2 quantizers (BF16 tags: statistics kernels, transposes) + 2 reductions + 1 GEMM
        n_fused = sum(1 for l in range(layers) for j in range(len(cfg.linears)) if FMT_BF16 not in [int(t) for t in self.tags[l, j]])
        self.launches_per_step = n_fused * 9 + (layers * len(cfg.linears) - n_fused) * 15

    def run(self, events=None, inputs=None, before=None):
        api, torch = self.api, self.torch
        lib, p, st = api._lib, api._p, api._stream()
        inputs = self.inputs if inputs is None else inputs
        i = 0
        for l in range(self.layers):
            for j, ((x, w, dy), (y, dx, dw)) in enumerate(zip(inputs[l], self.out)):
                if before is not None:
                    before(l, j)
                M, K = x.shape
                N = w.shape[0]
                t3 = [int(self.tags[l, j, gi]) for gi in range(3)]
                if FMT_BF16 not in t3:
                    if events is not None:
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                    api._check("snip_linear_fwd_bwd", lib.snip_linear_fwd_bwd(p(x), p(w), p(dy), p(y), p(dx), p(dw), M, N, K, t3[0], t3[1], t3[2], api.OUT_BF16,
                                                                              0, 0, 0, p(self.stats6[l * len(self.out) + j]), p(self.ws), self.ws.numel(), st))
                    if events is not None:
                        e1.record()
                        for f in t3:   # one call, three GEMMs of equal size: a third of its time to each tag
                            events.append((f, 2.0 * M * N * K, e0, e1, 1.0 / 3.0))
                    i += 3
                    continue
                calls = (("snip_linear_fwd", lambda f, sa, sb: lib.snip_linear_fwd(p(x), p(w), p(y), M, N, K, f, f, api.OUT_BF16, p(sa), p(sb), p(self.ws), self.ws.numel(), st)),
                         ("snip_linear_dgrad", lambda f, sa, sb: lib.snip_linear_dgrad(p(dy), p(w), p(dx), M, N, K, f, f, api.OUT_BF16, p(sa), p(sb), p(self.ws), self.ws.numel(), st)),
                         ("snip_linear_wgrad", lambda f, sa, sb: lib.snip_linear_wgrad(p(dy), p(x), p(dw), M, N, K, f, f, api.OUT_BF16, 0, p(sa), p(sb), p(self.ws), self.ws.numel(), st)))
                for gi, (name, call) in enumerate(calls):
                    f = int(self.tags[l, j, gi])
                    if events is not None:
                        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        e0.record()
                    api._check(name, call(f, self.stats[2 * i], self.stats[2 * i + 1]))
                    if events is not None:
                        e1.record()
                        events.append((f, 2.0 * M * N * K, e0, e1))
                    i += 1


class KernelTimer:
    """Times one kernel family alone (pre-quantized operands), CUDA events around each launch,
    rotating over operand sets so that L2 cannot serve the inputs."""

    def __init__(self, api, torch, cfg, device):
        self.api, self.torch, self.cfg, self.device = api, torch, cfg, device

    def gemm(self, fmt, op, lin_index, iters=20, warmup=3, mx=False):
        api, torch = self.api, self.torch
        L = self.cfg.linears[lin_index]
        M, N, K = self.cfg.M, L.N, L.K
        g = torch.Generator(device=self.device); g.manual_seed(1)
        def rnd(r, c, s=1.0):
            return (torch.randn(r, c, generator=g, device=self.device, dtype=torch.float32) * s).to(torch.bfloat16)
        quant = (lambda t, f, blk, fl=0: api.snip_quantize_mx(t, f, blk, fl)) if mx else (lambda t, f, blk, fl=0: api.snip_quantize(t, f, blk, fl))
        if op == api.OP_FWD:
            A, B, out_shape = rnd(M, K), rnd(N, K, 0.02), (M, N)
            qa = quant(A, fmt, api.BLOCK_ROW); qb = quant(B, fmt, api.BLOCK_BLK)
            a = api.make_qtensor(qa[0], qa[1], M, K, fmt, api.BLOCK_ROW); b = api.make_qtensor(qb[0], qb[1], N, K, fmt, api.BLOCK_BLK)
        elif op == api.OP_DGRAD:
            A, B, out_shape = rnd(M, N, 1e-3), rnd(N, K, 0.02), (M, K)
            qa = quant(A, fmt, api.BLOCK_ROW); qb = quant(B, fmt, api.BLOCK_BLK, api.Q_TRANSPOSED)
            a = api.make_qtensor(qa[0], qa[1], M, N, fmt, api.BLOCK_ROW); b = api.make_qtensor(qb[0], qb[1], N, K, fmt, api.BLOCK_BLK, True)
        else:
            A, B, out_shape = rnd(M, N, 1e-3), rnd(M, K), (N, K)
            qa = quant(A, fmt, api.BLOCK_COL, api.Q_TRANSPOSED); qb = quant(B, fmt, api.BLOCK_COL, api.Q_TRANSPOSED)
            a = api.make_qtensor(qa[0], qa[1], M, N, fmt, api.BLOCK_COL, True); b = api.make_qtensor(qb[0], qb[1], M, K, fmt, api.BLOCK_COL, True)
        out = torch.empty(out_shape, dtype=torch.bfloat16, device=self.device)
        ws = torch.zeros(max(1024, api.snip_workspace_size(op, M, N, K, fmt, fmt)[0]), dtype=torch.uint8, device=self.device)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=self.device)
        times = []
        for i in range(warmup + iters):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            if mx:
                api.snip_gemm_mx(op, a, qa[2], b, qb[2], out_shape, api.OUT_BF16, out=out, ws=ws)
            else:
                api.snip_gemm_quantized(op, a, b, out_shape, api.OUT_BF16, out=out, ws=ws)
            e1.record()
            torch.cuda.synchronize()
            if i >= warmup:
                times.append(e0.elapsed_time(e1))
        assert api.snip_poll_status(ws) == 0
        return 2.0 * M * N * K, times

    def quantizer(self, fmt, block, transposed, rows, cols, iters=20, warmup=3, stats=True):
        api, torch = self.api, self.torch
        g = torch.Generator(device=self.device); g.manual_seed(2)
        xs = [torch.randn(rows, cols, generator=g, device=self.device, dtype=torch.float32).to(torch.bfloat16) for _ in range(3)]
        flags = (api.Q_STATS if stats else 0) | (api.Q_TRANSPOSED if transposed else 0)
        codes, scales, stats, _ = api.snip_quantize(xs[0], fmt, block, flags)
        _, _, wb = api.snip_quantize_sizes(rows, cols, fmt, block, flags)
        ws = torch.empty(wb, dtype=torch.uint8, device=self.device)
        # batches of back-to-back calls on rotating inputs (each input exceeds L2), one event pair per
        # batch: host launch latency overlaps the previous call, as it does inside a training step
        times = []
        batch = 6
        for i in range(warmup + iters):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for j in range(batch):
                api.snip_quantize(xs[j % 3], fmt, block, flags, codes=codes, scales=scales, stats=stats, ws=ws)
            e1.record()
            torch.cuda.synchronize()
            if i >= warmup:
                times.append(e0.elapsed_time(e1) / batch)
        bytes_per_elt = 2.0 + (1.0 if fmt == FMT_FP8 else 0.5) + 4.0 / 128.0
        return bytes_per_elt * rows * cols, times


    def quantizer_dual(self, fmt, kind, rows, cols, iters=20, warmup=3, stats=True):
        """snip_quantize_dual (with statistics unless stats=False), timed like quantizer(); bytes = one read + two outputs."""
        api, torch = self.api, self.torch
        g = torch.Generator(device=self.device); g.manual_seed(2)
        xs = [torch.randn(rows, cols, generator=g, device=self.device, dtype=torch.float32).to(torch.bfloat16) for _ in range(3)]
        b32 = kind == api.DUAL_ROW32_COL32T    # power-of-two scales per 32-long tile, with the scale-factor atoms
        bufs = api.snip_quantize_dual(xs[0], kind, fmt, fmt, want_stats=stats, pow2_scale=b32, want_sf=b32)
        ws = torch.empty(api.snip_quantize_dual_workspace(rows, cols), dtype=torch.uint8, device=self.device)
        times = []
        batch = 6
        for i in range(warmup + iters):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for j in range(batch):
                api.snip_quantize_dual(xs[j % 3], kind, fmt, fmt, bufs=bufs, ws=ws, pow2_scale=b32)
            e1.record()
            torch.cuda.synchronize()
            if i >= warmup:
                times.append(e0.elapsed_time(e1) / batch)
        bytes_per_elt = 2.0 + 2.0 * ((1.0 if fmt == FMT_FP8 else 0.5) + (5.0 / 32.0 if b32 else 4.0 / 128.0))   # FP32 scale (+ 1 atom byte) per tile
        return bytes_per_elt * rows * cols, times


def cpu_baseline_sample(cfg, tokens=4096):
    """The CPU oracle, as it stands, on a bounded sample: `tokens` rows of the O projection
    (K -> K) through quantize + fwd + dgrad + wgrad in FP8.  Returns (TFLOP/s, cores, text)."""
    from oracle import snip_oracle as orc
    from paper_2602_01410_b200 import workloads as wl
    li = 1 if len(cfg.linears) > 1 else 0
    L = cfg.linears[li]
    x, w, dy = wl.linear_inputs(cfg, 0, li, M=tokens)
    t0 = time.perf_counter()
    orc.linear_fwd(x, w, FMT_FP8, FMT_FP8)
    orc.linear_dgrad(dy, w, FMT_FP8, FMT_FP8)
    orc.linear_wgrad(dy, x, FMT_FP8, FMT_FP8)
    dt = time.perf_counter() - t0
    flops = 3 * 2.0 * tokens * L.N * L.K
    return flops / dt / 1e12, orc.num_threads(), (f"{tokens} tokens of linear '{L.name}' ({L.K}->{L.N}), FP8: 3 quantize pairs + "
                                                   f"fwd/dgrad/wgrad float64 GEMMs, {dt:.2f} s")


def run_profile_case(name):
    """A few launches of one kernel on a small case (inputs above L2 size, well under a GB)."""
    import torch
    from paper_2602_01410_b200 import api, workloads as wl
    from dataclasses import replace
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    parts = name.split("_")
    if len(parts) > 1 and parts[1] == "nvfp4":
        # two-level (NVFP4-style) option: quantize_nvfp4_dual | gemm_nvfp4_<fwd|dgrad|wgrad> on the 7B QKV shape
        M, K, N = 16384, 4096, 12288
        g = torch.Generator(device=device); g.manual_seed(3)
        rnd = lambda r, c, sc: (torch.randn(r, c, generator=g, device=device, dtype=torch.float32) * sc).to(torch.bfloat16)
        bound = lambda t: t.float().abs().max().reshape(1).contiguous()
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
        times = []
        if parts[0] == "quantize":
            xs = [rnd(M, K, 1.0) for _ in range(3)]
            bs = [bound(t) for t in xs]
            bufs = api.snip_quantize_nvfp4_dual(xs[0], bs[0])
            ws = torch.empty(api.snip_quantize_dual_workspace(M, K), dtype=torch.uint8, device=device)
            for i in range(4):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for j in range(6):
                    api.snip_quantize_nvfp4_dual(xs[j % 3], bs[j % 3], bufs=bufs, ws=ws)
                e1.record(); torch.cuda.synchronize()
                if i >= 1: times.append(e0.elapsed_time(e1) / 6)
            by = (2.0 + 2.0 * (0.5 + 1.0 / 16.0)) * M * K
            print(f"{name}: {by / (min(times) * 1e-3) / 1e9:.0f} GB/s best of {len(times)}")
            return
        op = {"fwd": api.OP_FWD, "dgrad": api.OP_DGRAD, "wgrad": api.OP_WGRAD}[parts[2]]
        R, C, F4 = api.BLOCK_ROW16, api.BLOCK_COL16, api.FMT_FP4_E2M1
        if op == api.OP_FWD:
            A, B, oshape = rnd(M, K, 1.0), rnd(N, K, 0.02), (M, N)
            (qa, _), (qb, _) = api.snip_quantize_nvfp4_dual(A, bound(A), want_stats=False), api.snip_quantize_nvfp4_dual(B, bound(B), want_stats=False)
            a, b = api.make_qtensor(qa["codes"], None, M, K, F4, R), api.make_qtensor(qb["codes"], None, N, K, F4, R)
        elif op == api.OP_DGRAD:
            A, B, oshape = rnd(M, N, 1e-3), rnd(N, K, 0.02), (M, K)
            (qa, _), (_, qb) = api.snip_quantize_nvfp4_dual(A, bound(A), want_stats=False), api.snip_quantize_nvfp4_dual(B, bound(B), want_stats=False)
            a, b = api.make_qtensor(qa["codes"], None, M, N, F4, R), api.make_qtensor(qb["codes"], None, N, K, F4, C, True)
        else:
            A, B, oshape = rnd(M, N, 1e-3), rnd(M, K, 1.0), (N, K)
            (_, qa), (_, qb) = api.snip_quantize_nvfp4_dual(A, bound(A), want_stats=False), api.snip_quantize_nvfp4_dual(B, bound(B), want_stats=False)
            a, b = api.make_qtensor(qa["codes"], None, M, N, F4, C, True), api.make_qtensor(qb["codes"], None, M, K, F4, C, True)
        out = torch.empty(oshape, dtype=torch.bfloat16, device=device)
        ws = torch.zeros(1024, dtype=torch.uint8, device=device)
        ba, bb = bound(A), bound(B)
        for i in range(4):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            api.snip_gemm_nvfp4(op, a, qa["sf"], ba, b, qb["sf"], bb, oshape, api.OUT_BF16, out=out, ws=ws)
            e1.record(); torch.cuda.synchronize()
            if i >= 1: times.append(e0.elapsed_time(e1))
        print(f"{name}: {2.0 * M * N * K / (min(times) * 1e-3) / 1e12:.0f} TFLOP/s best of {len(times)}")
        return
    if name.startswith("adamw"):
        n = 12288 * 4096
        ms_ = [torch.randn(n, device=device) * 1e-3 for _ in range(2)]
        vs_ = [torch.rand(n, device=device) * 1e-6 + 1e-12 for _ in range(2)]
        gs_ = [(torch.randn(n, device=device) * 1e-3).to(torch.bfloat16) for _ in range(2)]
        out = torch.zeros(1, dtype=torch.float64, device=device)
        ws = torch.empty(1 << 16, dtype=torch.uint8, device=device)
        times = []
        for i in range(6):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            api.snip_adamw_sensitivity(ms_[i % 2], vs_[i % 2], gs_[i % 2], 0.9, 0.95, 1e-8, out=out, ws=ws)
            e1.record(); torch.cuda.synchronize()
            if i >= 2: times.append(e0.elapsed_time(e1))
        by = 10.0 * n
        print(f"adamw_sensitivity 12288x4096 (m, v fp32, g bf16): {min(times) * 1e3:.1f} us, {by / (min(times) * 1e-3) / 1e9:.0f} GB/s")
        return
    if name.startswith("layer_stats"):
        return run_layer_stats_case(api, torch, device, parts[2] if len(parts) > 2 else "x")
    mx = parts[1].startswith("mx")
    if parts[1].startswith("pair"):
        # the CTA-pair form of the paper-rule GEMM (an alternative kept for comparison; see include/snip.h, snip_debug_set)
        api.snip_debug_set(api.DEBUG_GEMM_KERNEL, api.GEMM_KERNEL_PAIR)
        parts[1] = parts[1][4:]
    fmt = {"bf16": FMT_BF16, "fp8": FMT_FP8, "fp4": FMT_FP4, "mxfp8": FMT_FP8, "mxfp4": FMT_FP4}[parts[1]]
    nostats = parts[-1] == "nostats"
    if nostats:
        parts = parts[:-1]
    if parts[0] == "quantize" and parts[2] == "dual":
        kt = KernelTimer(api, torch, wl.CONFIGS[3], device)
        kind = api.DUAL_BLK_BLKT if parts[-1] == "blk" else api.DUAL_ROW32_COL32T if parts[-1] == "b32" else api.DUAL_ROW_COLT
        by, times = kt.quantizer_dual(fmt, kind, 16384, 4096, iters=3, warmup=1, stats=not nostats)
        print(f"{name}: {by / (min(times) * 1e-3) / 1e9:.0f} GB/s best of {len(times)}")
    elif parts[0] == "quantize" and parts[2] == "sr":
        # stochastic rounding (FP4): quantize_fp4_sr_row | quantize_fp4_sr_col_t
        block, flags = (api.BLOCK_ROW, api.Q_STATS) if parts[3] == "row" else (api.BLOCK_COL, api.Q_STATS | api.Q_TRANSPOSED)
        xs = [torch.randn(16384, 4096, device=device, dtype=torch.bfloat16) for _ in range(3)]
        cb, sb, wb = api.snip_quantize_sizes(16384, 4096, FMT_FP4, block, flags)
        codes = torch.empty(cb, dtype=torch.uint8, device=device); scales = torch.empty(sb // 4, dtype=torch.float32, device=device)
        stats = torch.empty(32, dtype=torch.uint8, device=device); ws = torch.empty(wb, dtype=torch.uint8, device=device)
        times = []
        for i in range(4):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for j in range(6):
                x = xs[j % 3]
                api._check("snip_quantize_sr", api._lib.snip_quantize_sr(api._p(x), 16384, 4096, 4096, block, flags, 17 + j, 0, api._p(codes), api._p(scales),
                                                                         None, api._p(stats), api._p(ws), ws.numel(), api._stream()))
            e1.record(); torch.cuda.synchronize()
            if i: times.append(e0.elapsed_time(e1) / 6)
        by = 2.531 * 16384 * 4096
        print(f"{name}: {by / (min(times) * 1e-3) / 1e9:.0f} GB/s best of {len(times)} ({min(times) * 1e3:.1f} us per call)")
    elif parts[0] == "quantize":
        kind = "_".join(parts[2:])
        block, tr = {"row": (api.BLOCK_ROW, False), "col_t": (api.BLOCK_COL, True), "blk_t": (api.BLOCK_BLK, True),
                     "blk": (api.BLOCK_BLK, False), "col": (api.BLOCK_COL, False)}[kind]
        kt = KernelTimer(api, torch, wl.CONFIGS[3], device)
        by, times = kt.quantizer(fmt, block, tr, 16384, 4096, iters=3, warmup=1, stats=not nostats)
        print(f"{name}: {by / (min(times) * 1e-3) / 1e9:.0f} GB/s best of {len(times)}")
    else:
        op = {"fwd": api.OP_FWD, "dgrad": api.OP_DGRAD, "wgrad": api.OP_WGRAD}[parts[2]]
        M, N, K = (int(v) for v in parts[3].split("x")) if len(parts) > 3 else (4096, 4096, 4096)
        cfg = replace(wl.CONFIGS[3], M=M, linears=(wl.Linear("case", K, N),))
        kt = KernelTimer(api, torch, cfg, device)
        if fmt == FMT_BF16:
            raise SystemExit("bf16 GEMM cases run through snip_linear_*; use fp8/fp4 here")
        fl, times = kt.gemm(fmt, op, 0, iters=3, warmup=1, mx=mx)
        print(f"{name}: {fl / (min(times) * 1e-3) / 1e12:.0f} TFLOP/s best of {len(times)}")


def run_layer_stats_case(api, torch, device, which, rows=16384, cols=4096, copies=4, iters=5):
    """snip_layer_stats on one 7B-sized tensor (x: all four options of an activation; w: both options of a
    weight; plain: norm only), rotating over `copies` buffers so that L2 cannot serve the reads."""
    xs = [torch.randn(rows, cols, device=device, dtype=torch.bfloat16) for _ in range(copies)]
    ws = torch.empty(api.snip_layer_stats_workspace(rows, cols, cols), dtype=torch.uint8, device=device)
    out = torch.zeros(24, dtype=torch.float64, device=device)
    times = []
    for i in range(iters + 2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        x = xs[i % copies]
        e0.record()
        if which == "x":
            api.snip_layer_stats(X=x, M=rows, N=cols, K=cols, out=out, ws=ws)
        elif which == "w":
            api.snip_layer_stats(dX=None, W=x, M=cols, N=rows, K=cols, out=out, ws=ws)
        else:
            api.snip_layer_stats(dX=x, M=rows, N=cols, K=cols, out=out, ws=ws)
        e1.record()
        torch.cuda.synchronize()
        if i >= 2:
            times.append(e0.elapsed_time(e1))
    by = 2.0 * rows * cols
    print(f"layer_stats_{which}: {min(times) * 1e3:.1f} us best of {len(times)} (memset + kernel + reduction), "
          f"{by / (min(times) * 1e-3) / 1e9:.0f} GB/s of tensor read")


def run_reference(args):
    """--impl reference: the CPU oracle on a bounded sample per step (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2602_01410_b200 import workloads as wl
    cfg = wl.CONFIGS[WORKLOADS[args.workload][0]]
    tokens = 512
    vals = []
    for i in range(args.warmup + args.steps):
        v, cores, sample = cpu_baseline_sample(cfg, tokens)
        if i >= args.warmup:
            vals.append(v)
    v = sum(vals) / len(vals)
    L = cfg.linears[1 if len(cfg.linears) > 1 else 0]
    ms = 3 * 2.0 * tokens * L.N * L.K / (v * 1e12) * 1e3
    line = {"impl": "reference", "metric": "mixed-precision linear fwd+dgrad+wgrad TFLOP/s", "value": v, "unit": "TFLOP/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{cfg.name}: sample of {sample}"},
            "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_tagged(args, api, torch, dist, wl, cfg, device, world, rank, local_rank, barrier, peaks):
    """Contract line of a table-driven workload (--workload 3b | 70b)."""
    from paper_2602_01410_b200.replicas import combine_replicas
    layers = min(cfg.layers, TAGGED_LAYERS)
    step = TaggedStep(api, torch, cfg, device, layers)
    for _ in range(max(args.warmup, 3)):
        step.run()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    events = []
    e0.record()
    for _ in range(args.steps):
        step.run(events)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    ms_total, flops_job = combine_replicas(ms_total, step.flops, dist if world > 1 else None, device)
    assert api.snip_poll_status(step.ws) == 0, "device-side timeout reported"
    ms_per_step = ms_total / args.steps
    value = flops_job / (ms_per_step * 1e-3) / 1e12
    # per operand format: the linear calls (quantizers + GEMM) of the timed region against the GEMM's tensor peak
    per_format = {}
    for ev in events:
        f, fl, a, b = ev[:4]
        d = per_format.setdefault(f, {"flops": 0.0, "ms": 0.0, "calls": 0})
        d["flops"] += fl; d["ms"] += a.elapsed_time(b) * (ev[4] if len(ev) > 4 else 1.0); d["calls"] += 1
    pf = {}
    for f, d in per_format.items():
        ach = d["flops"] / (d["ms"] * 1e-3) / 1e12
        pk = peaks["bf16_tflops_sustained"] * NOMINAL_RATIO[f]
        pf[FMT_NAME[f]] = {"achieved": ach, "peak": pk, "frac": ach / pk, "calls": d["calls"], "share_of_step": d["ms"] / ms_total,
                           "share_of_flops": step.flops_by_fmt.get(f, 0.0) / step.flops}
    worst = min(pf, key=lambda k: pf[k]["frac"])
    roofline = {"kernel": f"snip_linear_fwd_bwd / snip_linear_fwd/dgrad/wgrad calls (quantizer passes with statistics + GEMMs), headline = {worst} tags",
                "bound": "tensor", "achieved": pf[worst]["achieved"], "peak": pf[worst]["peak"], "unit": "TFLOP/s", "frac": pf[worst]["frac"],
                "traffic": None, "per_format": pf,
                "peak_source": f"{peaks['source']} cuBLAS bf16 sustained x nominal format ratio (x1 bf16, x2 fp8, x4 fp4)"}
    # end to end: every step copies the layers' inputs from pinned host memory and reads the statistics back
    host = [[tuple(t.cpu().pin_memory() for t in trip) for trip in layer] for layer in step.inputs]
    h2d = sum(t.numel() * 2 for layer in host for trip in layer for t in trip)
    stats_host = torch.empty_like(step.stats, device="cpu").pin_memory()
    copy_stream = torch.cuda.Stream(device=device)
    main_stream = torch.cuda.current_stream(device)
    state = {"free": None}

    def e2e_step():
        ready = {}
        with torch.cuda.stream(copy_stream):
            if state["free"] is not None:
                copy_stream.wait_event(state["free"])
            for l, layer in enumerate(host):
                for j, trip_h in enumerate(layer):
                    for d_, h_ in zip(step.inputs[l][j], trip_h):
                        d_.copy_(h_, non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(copy_stream)
                    ready[(l, j)] = ev
        step.run(before=lambda l, j: main_stream.wait_event(ready[(l, j)]))
        stats_host.copy_(step.stats, non_blocking=True)
        state["free"] = torch.cuda.Event()
        state["free"].record(main_stream)
    e2e_step(); barrier()
    n_e2e = max(2, min(args.steps, 5))
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s0.record()
    copy_stream.wait_event(s0)
    for _ in range(n_e2e):
        e2e_step()
    s1.record()
    barrier()
    ms_e2e, flops_e2e = combine_replicas(s0.elapsed_time(s1) / n_e2e, step.flops, dist if world > 1 else None, device)
    e2e = {"value": flops_e2e / (ms_e2e * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms_e2e, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": stats_host.numel(), "steps": n_e2e, "overlap": "copies on a second stream, one input set"}
    if rank != 0:
        return
    cpu = None
    if not args.no_cpu_baseline:
        v, cores, sample = cpu_baseline_sample(cfg, tokens=2048)
        cpu = {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample}
    input_bytes = layers * sum(2 * (cfg.M * L.K + L.N * L.K + cfg.M * L.N) for L in cfg.linears)
    mix = ", ".join(f"{FMT_NAME[f]} {100.0 * v / step.flops:.0f} % of FLOPs" for f, v in sorted(step.flops_by_fmt.items()))
    line = {"metric": "mixed-precision linear fwd+dgrad+wgrad TFLOP/s", "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "seeded mix of bf16 / fp8_e4m3 / fp4_e2m1 per GEMM (fp32 accumulate)", "data": "synthetic",
            "config": {"workload": f"{cfg.name}: {layers} of {cfg.layers} layers x ({','.join(L.name for L in cfg.linears)}) x (fwd,dgrad,wgrad), tokens {cfg.M}, "
                                   f"per-GEMM precision tags of the seeded table '{cfg.tag_rule}' ({mix}), quantize+stats of both operands of every GEMM",
                       "l2": f"inputs ({input_bytes / 1e6:.0f} MB) larger than L2", "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": step.launches_per_step * args.steps, "roofline": roofline, "cpu_baseline": cpu}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="snip")
    ap.add_argument("--workload", default="7b", choices=sorted(WORKLOADS))
    ap.add_argument("--quantizer", default="dual", choices=("dual", "single"),
                    help="dual: X, W, dY each read once, both quantized copies written; single: one quantizer call per GEMM operand")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-legs", action="store_true")
    ap.add_argument("--profile-case", default=None,
                    help="run one small kernel case a few times and exit (for ncu): quantize_<fp8|fp4>_<row|col_t|blk_t|dual_rowcol|dual_blk|dual_b32> "
                         "or gemm_<fp8|fp4|mxfp8|mxfp4|pairfp8|pairfp4>_<fwd|dgrad|wgrad>[_MxNxK] or layer_stats_<x|w|plain>")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.profile_case:
        return run_profile_case(args.profile_case)

    import torch
    import torch.distributed as dist
    from paper_2602_01410_b200 import api, workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl")

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    cfg = wl.CONFIGS[WORKLOADS[args.workload][0]]
    if args.workload in ("3b", "70b"):
        run_tagged(args, api, torch, dist, wl, cfg, device, world, rank, local_rank, barrier, load_peaks())
        if world > 1:
            dist.destroy_process_group()
        return
    formats = (FMT_FP4, FMT_FP8)
    step = Step(api, torch, cfg, device, formats, dual=(args.quantizer == "dual"))
    peaks = load_peaks()

    # ---- timed region: K steps, inputs resident in HBM ------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step.run_decomposed()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    events, qevents = [], []
    e0.record()
    for _ in range(args.steps):
        step.run_decomposed(events, qevents=qevents if step.dual else None)
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop() if rank == 0 else None
    from paper_2602_01410_b200.replicas import combine_replicas
    ms_total, flops_job = combine_replicas(ms_total, step.flops, dist if world > 1 else None, device)
    assert api.snip_poll_status(step.gws) == 0, "device-side timeout reported"
    # GEMM launches inside the timed region, per format: total flops / total event time
    in_region = {}
    for fmt, op, fl, a, b in events:
        d = in_region.setdefault(fmt, {"flops": 0.0, "ms": 0.0, "launches": 0})
        d["flops"] += fl; d["ms"] += a.elapsed_time(b); d["launches"] += 1
    ms_per_step = ms_total / args.steps
    value = flops_job / (ms_per_step * 1e-3) / 1e12

    # ---- the same step under the power-of-two scale option (hardware-applied scales) ----------------
    for _ in range(3):
        step.run_decomposed(mx=True)
    barrier()
    mx_events = []
    m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    m0.record()
    for _ in range(args.steps):
        step.run_decomposed(mx_events, mx=True)
    m1.record()
    barrier()
    ms_mx, flops_mx = combine_replicas(m0.elapsed_time(m1), step.flops, dist if world > 1 else None, device)
    assert api.snip_poll_status(step.gws) == 0, "device-side timeout reported"
    mx_region = {}
    for fmt, op, fl, a, b in mx_events:
        d = mx_region.setdefault(fmt, {"flops": 0.0, "ms": 0.0})
        d["flops"] += fl; d["ms"] += a.elapsed_time(b)
    pow2_option = {"value": flops_mx / (ms_mx / args.steps * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms_mx / args.steps,
                   "note": "same step with S = 2^e scales applied by the tensor core (snip_quantize_mx + snip_gemm_mx); an added quantization option, not the paper's rule",
                   "gemm": {FMT_NAME[f]: {"tflops": d["flops"] / (d["ms"] * 1e-3) / 1e12,
                                          "frac_of_sustained_peak": d["flops"] / (d["ms"] * 1e-3) / 1e12 / (peaks["bf16_tflops_sustained"] * NOMINAL_RATIO[f]),
                                          "frac_of_burst_peak": d["flops"] / (d["ms"] * 1e-3) / 1e12 / (peaks["bf16_tflops"] * NOMINAL_RATIO[f])}
                            for f, d in mx_region.items()}}

    # ---- ... and with those scales on 32-long tiles (the tile length of the microscaling formats) ----
    for _ in range(3):
        step.run_decomposed(mx=2)
    barrier()
    mx32_events = []
    m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    m0.record()
    for _ in range(args.steps):
        step.run_decomposed(mx32_events, mx=2)
    m1.record()
    barrier()
    ms_mx32, flops_mx32 = combine_replicas(m0.elapsed_time(m1), step.flops, dist if world > 1 else None, device)
    assert api.snip_poll_status(step.gws) == 0, "device-side timeout reported"
    mx32_region = {}
    for fmt, op, fl, a, b in mx32_events:
        d = mx32_region.setdefault(fmt, {"flops": 0.0, "ms": 0.0})
        d["flops"] += fl; d["ms"] += a.elapsed_time(b)
    pow2_option["block32"] = {"value": flops_mx32 / (ms_mx32 / args.steps * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms_mx32 / args.steps,
                              "note": "power-of-two scales per 1x32 / 32x1 tile (W included), same hardware-scaled GEMM kernels",
                              "gemm": {FMT_NAME[f]: {"tflops": d["flops"] / (d["ms"] * 1e-3) / 1e12,
                                                     "frac_of_sustained_peak": d["flops"] / (d["ms"] * 1e-3) / 1e12 / (peaks["bf16_tflops_sustained"] * NOMINAL_RATIO[f])}
                                       for f, d in mx32_region.items()}}

    # ---- the FP4 half of the step under the two-level (NVFP4-style) option ------------------------
    for _ in range(3):
        run_two_level(step)
    barrier()
    nv_events, nv_q = [], []
    m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    m0.record()
    for _ in range(args.steps):
        run_two_level(step, nv_events, nv_q)
    m1.record()
    barrier()
    flops_half = step.flops / len(step.formats)
    ms_nv, flops_nv = combine_replicas(m0.elapsed_time(m1), flops_half, dist if world > 1 else None, device)
    assert api.snip_poll_status(step.gws) == 0, "device-side timeout reported"
    nv_g = sum(fl for _, _, fl, _, _ in nv_events) / (sum(a.elapsed_time(b) for _, _, _, a, b in nv_events) * 1e-3) / 1e12
    nv_qgbs = sum(by for _, by, _, _ in nv_q) / (sum(a.elapsed_time(b) for _, _, a, b in nv_q) * 1e-3) / 1e9
    pow2_option["two_level_fp4"] = {"value": flops_nv / (ms_nv / args.steps * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms_nv / args.steps,
                                    "note": "the FP4 half of the step (15 GEMMs) with E2M1 codes in 16-long tiles, E4M3 scale bytes and a per-tensor bound "
                                            "(snip_quantize_nvfp4_dual + snip_gemm_nvfp4, kind::mxf4nvf4); an added option",
                                    "gemm": {"tflops": nv_g, "frac_of_sustained_peak": nv_g / (peaks["bf16_tflops_sustained"] * NOMINAL_RATIO[FMT_FP4])},
                                    "quantizer": {"gbs": nv_qgbs, "frac_of_hbm": nv_qgbs / peaks["hbm_gbs"]}}

    # ---- end to end: inputs start in pinned host memory, statistics come back -------------------
    e2e = None
    if rank == 0 or world > 1:
        host = [tuple(t.cpu().pin_memory() for t in trip) for trip in step.inputs]
        h2d = sum(t.numel() * 2 for trip in host for t in trip)
        stats_dev = step.stats6 if step.dual else step.stats
        stats_host = torch.empty_like(stats_dev, device="cpu").pin_memory()
        # Two device copies of the inputs: while one step computes from one set, the copy engine fills the other
        # from pinned host memory on its own stream.  Every linear waits only for its own three tensors, and a set
        # is overwritten only after the last kernel that reads it has finished.
        sets = [step.inputs, [tuple(torch.empty_like(t) for t in trip) for trip in step.inputs]]
        copy_stream = torch.cuda.Stream(device=device)
        main_stream = torch.cuda.current_stream(device)
        set_free = [None, None]
        def e2e_step(k):
            dev_in = sets[k % 2]
            ready = []
            with torch.cuda.stream(copy_stream):
                if set_free[k % 2] is not None:
                    copy_stream.wait_event(set_free[k % 2])
                for trip_d, trip_h in zip(dev_in, host):
                    for d, h in zip(trip_d, trip_h):
                        d.copy_(h, non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(copy_stream)
                    ready.append(ev)
            step.run_linear_calls(inputs=dev_in, before=lambda i: main_stream.wait_event(ready[i]))
            stats_host.copy_(stats_dev, non_blocking=True)
            set_free[k % 2] = torch.cuda.Event()
            set_free[k % 2].record(main_stream)
        e2e_step(0); e2e_step(1); barrier()
        n_e2e = max(2, min(args.steps, 10))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s0.record()
        copy_stream.wait_event(s0)   # no copy of a timed step starts before the clock does
        for k in range(n_e2e):
            e2e_step(k)
        s1.record()
        barrier()
        ms_e2e = s0.elapsed_time(s1) / n_e2e
        ms_e2e, flops_e2e = combine_replicas(ms_e2e, step.flops, dist if world > 1 else None, device)
        e2e = {"value": flops_e2e / (ms_e2e * 1e-3) / 1e12, "unit": "TFLOP/s", "ms_per_step": ms_e2e,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": stats_host.numel(), "steps": n_e2e,
               "overlap": "copies on a second stream into alternating input sets"}
        del host, sets

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- kernel legs: the GEMM and quantizer kernels alone, events around each launch ---------------
    roofline, kernels = None, {}
    if not args.no_kernel_legs:
        del step.inputs, step.out, step.codes, step.scales, step.sf
        torch.cuda.empty_cache()
        kt = KernelTimer(api, torch, cfg, device)
        qkv = 0
        fam = {}
        for f in formats:
            per_op = {}
            tot_fl, tot_ms = 0.0, 0.0
            for op, name in ((api.OP_FWD, "fwd"), (api.OP_DGRAD, "dgrad"), (api.OP_WGRAD, "wgrad")):
                fl, times = kt.gemm(f, op, qkv)
                avg = sum(times) / len(times)
                per_op[name] = {"tflops": fl / (avg * 1e-3) / 1e12, "ms": avg}
                tot_fl += fl; tot_ms += avg
            peak = peaks["bf16_tflops"] * NOMINAL_RATIO[f]
            fam[f] = {"achieved": tot_fl / (tot_ms * 1e-3) / 1e12, "peak": peak, "per_op": per_op, "ms": tot_ms}
            kernels[f"gemm_{FMT_NAME[f]}"] = {"tflops": fam[f]["achieved"], "frac_of_peak": fam[f]["achieved"] / peak,
                                              "peak_tflops": peak, "per_op": per_op}
    # One roofline object for the step's two kernel families.  GEMMs (tensor-bound): every launch of the timed region,
    # per operand format, against the measured sustained cuBLAS bf16 rate x the nominal format ratio; the headline
    # `frac` is the LOWER of the two formats.  Quantizers (HBM-bound): the two-output calls with statistics that the
    # step runs, algorithmic bytes / event time against the measured copy bandwidth.
    per_format = {}
    for f, d in in_region.items():
        ach = d["flops"] / (d["ms"] * 1e-3) / 1e12
        pk = peaks["bf16_tflops_sustained"] * NOMINAL_RATIO[f]
        per_format[FMT_NAME[f]] = {"achieved": ach, "peak": pk, "frac": ach / pk, "launches": d["launches"], "share_of_step": d["ms"] / ms_total,
                                   "nominal_dense_peak": 2250.0 * NOMINAL_RATIO[f], "frac_of_nominal": ach / (2250.0 * NOMINAL_RATIO[f]),
                                   "traffic": NCU_TRAFFIC.get(f)}
    worst = min(per_format, key=lambda k: per_format[k]["frac"])
    qleg = None
    if qevents:
        qfmt = {}
        for fmt, by, a_, b_ in qevents:
            q = qfmt.setdefault(fmt, {"bytes": 0.0, "ms": 0.0, "calls": 0})
            q["bytes"] += by; q["ms"] += a_.elapsed_time(b_); q["calls"] += 1
        qleg = {"kernel": "quantize_dual_kernel + stats_reduce_kernel (two outputs with statistics, every call of the timed region)",
                "bound": "hbm", "unit": "GB/s", "peak": peaks["hbm_gbs"],
                "per_format": {FMT_NAME[f]: {"achieved": q["bytes"] / (q["ms"] * 1e-3) / 1e9, "frac": q["bytes"] / (q["ms"] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                             "calls": q["calls"], "share_of_step": q["ms"] / ms_total} for f, q in qfmt.items()}}
        qleg["achieved"] = min(v["achieved"] for v in qleg["per_format"].values())
        qleg["frac"] = min(v["frac"] for v in qleg["per_format"].values())
        qleg["traffic"] = "DRAM bytes of one call equal the algorithmic bytes within 1 % (ncu, profiles/quantize_dual_kernel_*)"
    roofline = {"kernel": f"gemm_kernel (tcgen05, per-chunk FP32 promotion), headline = {worst} operands: the lower fraction of the two formats",
                "bound": "tensor", "achieved": per_format[worst]["achieved"], "peak": per_format[worst]["peak"], "unit": "TFLOP/s",
                "frac": per_format[worst]["frac"], "traffic": per_format[worst]["traffic"],
                "traffic_case": "one launch, fwd 16384x12288x4096 (ncu, profiles/)",
                "per_format": per_format, "quantizer": qleg,
                "peak_source": f"{peaks['source']} cuBLAS bf16 sustained x nominal format ratio (x2 fp8, x4 fp4); nominal dense peaks printed beside"}
    for f, d in in_region.items():
        kernels[f"gemm_{FMT_NAME[f]}_in_step"] = {"tflops": d["flops"] / (d["ms"] * 1e-3) / 1e12, "ms_per_step": d["ms"] / args.steps,
                                                   "frac_of_sustained_peak": d["flops"] / (d["ms"] * 1e-3) / 1e12 / (peaks["bf16_tflops_sustained"] * NOMINAL_RATIO[f])}
    if not args.no_kernel_legs:
        for f in formats:
            for block, tr, name in ((api.BLOCK_ROW, False, "row"), (api.BLOCK_COL, True, "col_t"), (api.BLOCK_BLK, True, "blk_t")):
                by, times = kt.quantizer(f, block, tr, cfg.M, 4096)
                avg = sum(times) / len(times)
                kernels[f"quantize_{FMT_NAME[f]}_{name}"] = {"gbs": by / (avg * 1e-3) / 1e9, "frac_of_hbm": by / (avg * 1e-3) / 1e9 / peaks["hbm_gbs"], "ms": avg}
            for kind, name in ((api.DUAL_ROW_COLT, "row+col_t"), (api.DUAL_BLK_BLKT, "blk+blk_t"), (api.DUAL_ROW32_COL32T, "row32+col32_t_pow2")):
                by, times = kt.quantizer_dual(f, kind, cfg.M, 4096)
                avg = sum(times) / len(times)
                kernels[f"quantize_dual_{FMT_NAME[f]}_{name}"] = {"gbs": by / (avg * 1e-3) / 1e9, "frac_of_hbm": by / (avg * 1e-3) / 1e9 / peaks["hbm_gbs"], "ms": avg}
            # the same quantizers without the fused statistics (the paper collects them at intervals, Sec. 3.1)
            by, times = kt.quantizer(f, api.BLOCK_ROW, False, cfg.M, 4096, stats=False)
            avg = sum(times) / len(times)
            kernels[f"quantize_{FMT_NAME[f]}_row_nostats"] = {"gbs": by / (avg * 1e-3) / 1e9, "frac_of_hbm": by / (avg * 1e-3) / 1e9 / peaks["hbm_gbs"], "ms": avg}
            by, times = kt.quantizer_dual(f, api.DUAL_ROW_COLT, cfg.M, 4096, stats=False)
            avg = sum(times) / len(times)
            kernels[f"quantize_dual_{FMT_NAME[f]}_row+col_t_nostats"] = {"gbs": by / (avg * 1e-3) / 1e9, "frac_of_hbm": by / (avg * 1e-3) / 1e9 / peaks["hbm_gbs"], "ms": avg}

    cpu = None
    if not args.no_cpu_baseline:
        v, cores, sample = cpu_baseline_sample(cfg)
        cpu = {"value": v, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample}
        # the same oracle on one core, on an eighth of the sample
        from oracle import snip_oracle as orc
        orc.set_num_threads(1)
        v1, _, sample1 = cpu_baseline_sample(cfg, tokens=512)
        orc.set_num_threads(cores)
        cpu["one_core"] = {"value": v1, "unit": "TFLOP/s", "cores": 1, "sample": sample1}

    input_bytes = sum(2 * (cfg.M * L.K + L.N * L.K + cfg.M * L.N) for L in cfg.linears)   # bf16 X, W, dY of every linear
    line = {"metric": "mixed-precision linear fwd+dgrad+wgrad TFLOP/s", "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp4_e2m1+fp8_e4m3 (fp32 accumulate)", "data": "synthetic",
            "config": {"workload": f"{cfg.name}: one block ({','.join(L.name for L in cfg.linears)}) x (fwd,dgrad,wgrad) all-FP4 then all-FP8, tokens {cfg.M}, quantize+stats of both operands of every GEMM "
                                   + ("(X, W, dY read once each, two quantized copies per read)" if step.dual else "(one quantizer call per operand)"),
                       "l2": (f"inputs ({input_bytes / 1e6:.0f} MB) larger than L2" if input_bytes > 126e6
                              else f"inputs ({input_bytes / 1e6:.1f} MB) fit in L2: a test workload, not a measurement"),
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks, "e2e": e2e, "gpu_launches": step.launches_per_step * args.steps,
            "roofline": roofline, "kernels": kernels, "pow2_option": pow2_option, "cpu_baseline": cpu}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
