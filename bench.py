#!/usr/bin/env python
"""Benchmark of the LBA contraction on B200: emulated GMAC/s and fraction of the ALU roofline.

Headline workload (N = 1 GPU): ONE LBA GEMM, M = N = K = 8192, Gaussian operands quantised to E4M3 with
per-tensor scales, M7E4 product and accumulator formats (the 12-bit accumulator), chunk-16 accumulation (the
paper's order), floor rounding -- the largest single-GPU case of the five benchmark configurations.  A step is
one launch through lba_gemm with both operands resident in HBM.  With N > 1 every rank runs the same step on
its own row block (rows of the output are independent chains; no collective on the data path): weak scaling.

After the headline, rank 0 of a single-GPU run also times the other configurations (single small GEMM,
ResNet-18 and ResNet-50 convolution stacks, BERT-base linears in both orders, the 42-point accumulator-format
sweep on the 8192^3 GEMM) and reports them under "configs", each with its GMAC/s and its fraction of the ALU
roofline of the kernel variant it ran.

One JSON line is printed by rank 0.  `--impl reference` times the CPU oracle instead (rank 0 only).
`--gpus N` without a launcher environment starts N ranks itself (one process per GPU).
"""
import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "emulated_lba_gmacs"
UNIT = "GMAC/s"
HEADLINE = "gemm:8192x8192x8192:chunk"

# ---------------------------------------------------------------------------------------------------------
# ALU roofline for sm_100.  Per SM and clock 4 schedulers issue one warp instruction each (128 lanes); the
# FP32 pipe retires 128 lane-operations per clock (a packed f32x2 instruction holds it for two clocks), the
# integer/logic pipe 64 (every instruction holds it for two clocks).  A kernel variant is described by the
# minimal instruction mix of one emulated MAC: (issue slots, logic-pipe instructions, packed FP32 instructions,
# scalar FP32 instructions); its bound in clocks per warp-MAC per scheduler is the largest of
#   issue slots,  2 x logic-pipe instructions,  2 x packed + 1 x scalar FP32 instructions.
# The chunked order adds one fold T <- Q_acc(C + T) per output per chunk.
LANES_PER_SM_CLK = 128
MIX = {
    # mode: (issue, logic, packed_fp, scalar_fp, text)
    "floor": (2.0, 1.0, 1.0, 0.0, "0.5 FMUL2 + 0.5 FFMA2 + 1 LOP3"),
    "floor_cut": (3.0, 2.0, 1.0, 0.0, "0.5 FMUL2 + 1 LOP3 (product mask) + 0.5 FFMA2 + 1 LOP3"),
    "floor_cut_sat": (4.0, 3.0, 1.0, 0.0, "0.5 FMUL2 + 1 LOP3 + 1 FMNMX (product) + 0.5 FFMA2 + 1 LOP3"),
    "floor_fused": (1.5, 1.0, 0.5, 0.0, "0.5 FFMA2 (product and sum in one instruction) + 1 LOP3"),
    "rne": (4.0, 2.0, 2.0, 0.0, "0.5 FMUL2 + 0.5 FFMA2 + 1 LOP3 + 1 FFMA2 (rounding on the FP32 pipe) + 1 FMNMX"),
    "rne_cut": (6.0, 3.0, 3.0, 0.0, "as rne, plus 1 LOP3 + 1 FFMA2 for the product's rounding"),
    "rne_cut_sat": (7.0, 4.0, 3.0, 0.0, "as rne_cut, plus 1 FMNMX for the product's saturation"),
    "rne_fused": (3.5, 2.0, 1.5, 0.0, "0.5 FFMA2 (product and sum) + 1 LOP3 + 1 FFMA2 (rounding) + 1 FMNMX"),
    "rne_wide": (1.0, 0.0, 0.0, 1.0, "1 FFMA (24-bit accumulator: one IEEE FMA per MAC)"),
    "generic": (6.0, 4.0, 0.0, 2.0, "scalar FMUL + FFMA + mask + clamp (+ product steps): the generic kernel"),
    "fixed": (6.0, 4.0, 0.0, 2.0, "2 SHF + 2 add-min/max on the logic pipe; IMAD + IADD beside them"),
    "ste_diff": (7.0, 3.0, 3.0, 1.0, "0.5 each of FMUL2, FFMA2 (chain), FMUL2, FFMA2 (distance), FFMA2, FMUL2 (threshold) "
                                     "+ LOP3 + FMNMX + FADD (thr - |d|) + SHF (its sign into the mask)"),
}
FOLD = {  # per output per chunk: (issue, logic, packed_fp, scalar_fp)
    "floor": (2.5, 2.0, 0.5, 0.0), "rne": (3.5, 2.0, 1.5, 0.0), "rne_wide": (1.0, 0.0, 0.0, 1.0), "generic": (4.0, 2.0, 0.0, 1.0),
    "fixed": (4.0, 4.0, 0.0, 0.0),
}


def clocks_per_warp_mac(mode: str, chunk: int):
    """(clocks per warp-MAC per scheduler, which limit binds) of the minimal mix of `mode`; chunk = 0: sequential."""
    issue, logic, packed, scalar, _ = MIX[mode]
    if chunk:
        base = "rne" if mode.startswith("rne") and mode != "rne_wide" else ("floor" if mode.startswith("floor") else mode)
        f = FOLD.get(base, FOLD["generic"])
        issue, logic, packed, scalar = (issue + f[0] / chunk, logic + f[1] / chunk, packed + f[2] / chunk,
                                        scalar + f[3] / chunk)
    limits = {"issue": issue, "logic pipe": 2.0 * logic, "fp32 pipe": 2.0 * packed + scalar}
    which = max(limits, key=limits.get)
    return limits[which], which


def min_issue_slots(mode: str, chunk: int) -> float:
    """Issue slots per emulated MAC of the minimal mix (the figure executed instructions per MAC compare with)."""
    base = "rne" if mode.startswith("rne") and mode != "rne_wide" else ("floor" if mode.startswith("floor") else mode)
    return MIX[mode][0] + (FOLD.get(base, FOLD["generic"])[0] / chunk if chunk else 0.0)


def mode_of(desc: str, ste=None, fixed=False) -> str:
    """Mix name of the kernel variant a plan description names."""
    if fixed:
        return "fixed"
    if ste == "diff":
        return "ste_diff"
    f = dict(p.split("=", 1) for p in desc.split() if "=" in p)
    q, pq = f.get("q", ""), f.get("pq", "none")
    suffix = {"none": "", "cut": "_cut", "cut_sat": "_cut_sat", "fused": "_fused"}.get(pq, "")
    if f.get("kernel") == "generic" and q != "rne_wide":
        return "generic"
    if q.startswith("floor"):
        return "floor" + suffix
    if q == "rne_wide":
        return "rne_wide"
    return "rne" + suffix


def peak_gmacs(mode, chunk, sm_count, mhz):
    """(ALU-issue roofline in GMAC/s, issue slots per MAC of the minimal mix, tighter pipe limit or None).

    The roofline every fraction is quoted against is the issue roofline: lanes issued per clock x clock / issue slots
    per emulated MAC of the minimal mix.  Where one pipe alone needs more clocks than the issue slots (the logic pipe
    holds every instruction for two clocks), that tighter limit is reported beside it, not used as the denominator."""
    slots = min_issue_slots(mode, chunk)
    clk, which = clocks_per_warp_mac(mode, chunk)
    pipe = None if which == "issue" or clk <= slots else {"limit": which, "clocks_per_warp_mac": clk,
                                                           "peak": sm_count * LANES_PER_SM_CLK * mhz * 1e6 / clk / 1e9}
    return sm_count * LANES_PER_SM_CLK * mhz * 1e6 / slots / 1e9, slots, pipe


# DRAM bytes (read + write) of ONE launch of the dominant kernel, from the ncu captures summarised under profiles/
# (workload, kernel description) -> (bytes, what was captured, executed instructions per emulated MAC).
_K_FLOOR = "tile=128x128x16 micro=8x8 q=floor_fast pq=none kernel=packed order=chunk16 load=gemm_vec"
_CAP = "profiles/packed_floor_kernel_gemm_8192x8192x1024_chunk.txt"
NCU = {
    # the headline launch is too long for a multi-pass capture (52 ms, 39 passes): the K = 1024 case of the same kernel was
    # captured; its reads grow in proportion to K (x 8), its writes (the output) do not grow with K
    ("single_lba_gemm_8192x8192x8192_m7e4_chunk16", _K_FLOOR):
        (8 * 17673984 + 214364672, "scaled from the 8192x8192x1024 capture (" + _CAP + "): 8 x 17.7 MB read + 214.4 MB written; "
         "algorithmic 128 MB + 256 MB (part of the output is still in L2 when the kernel ends)", 2.453),
    ("single_lba_gemm_8192x8192x1024_m7e4_chunk16", _K_FLOOR):
        (17673984 + 214364672, "17.7 MB read + 214.4 MB written (" + _CAP + "); algorithmic 272 MB", 2.453),
    ("single_lba_gemm_8192x8192x1024_m7e4_sequential", "tile=128x128x16 micro=8x8 q=floor_fast pq=none kernel=packed order=seq load=gemm_vec"):
        (18133504 + 212325376, "18.1 MB read + 212.3 MB written (profiles/packed_floor_kernel_gemm_8192x8192x1024_seq.txt)", 2.323),
    ("single_lba_gemm_8192x8192x1024_m7e4_rne_chunk16", "tile=64x64x16 micro=4x8 q=rne_full pq=none kernel=packed order=chunk16 load=gemm_vec"):
        (17937920 + 212977664, "17.9 MB read + 213.0 MB written (profiles/packed_nearest_even_kernel_gemm_8192x8192x1024_chunk.txt)", 4.921),
    ("single_lba_gemm_8192x8192x1024_m8e6_chunk16", "tile=128x128x16 micro=8x8 q=floor_fast pq=fused kernel=packed order=chunk16 load=gemm_vec"):
        (17225472 + 213304832, "17.2 MB read + 213.3 MB written (profiles/packed_floor_kernel_fused_gemm_8192x8192x1024_chunk.txt)", 1.946),
}


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE,
                    help="gemm:MxNxK[:seq|chunk] (default gemm:8192x8192x8192:chunk, the headline), resnet18, resnet50, "
                         "bgemm:ZxMxNxK[:seq|chunk] (one batched call), ste:MxNxK[:of|diff][:seq|chunk] (STE mask "
                         "re-computation of one GEMM), fixed:MxNxK[:seq|chunk][:wrap] (12-bit fixed-point accumulation, Eq. 1); "
                         "append :rne or :mMeE (e.g. :m4e5) to a gemm workload for another accumulator format")
    ap.add_argument("--configs", default="auto", choices=["auto", "all", "none"],
                    help="time the other benchmark configurations too (auto: only with the headline workload on one GPU)")
    ap.add_argument("--cpu-baseline-macs", type=float, default=2.0e9,
                    help="size of the oracle sample timed for cpu_baseline (emulated MACs)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-streams", type=int, default=12,
                    help="network workloads: streams (each with its own device workspace) the end-to-end calls are spread over")
    ap.add_argument("--e2e-row-blocks", type=int, default=2,
                    help="single-GEMM workloads: the end-to-end step is issued as this many row blocks (rows of the output are "
                         "independent chains), one lba_gemm_host call each, over up to three streams, so that one block's copies "
                         "overlap another block's kernel; 1 = one call")
    ap.add_argument("--force-dist", action="store_true",
                    help="initialise torch.distributed (NCCL) even for a single rank: exercises the multi-GPU plumbing "
                         "(barrier, max over ranks) on one GPU")
    return ap.parse_args(argv)


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only queries) while the timed region runs."""

    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
               "hw_power_brake_slowdown": 0x80}

    def __init__(self, index):
        self.index = index
        self.samples = []
        self.power = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None
        self._handle = None

    def _open(self):
        import pynvml
        pynvml.nvmlInit()
        self._nvml = pynvml
        # NVML numbers devices by PCI order, CUDA possibly by a CUDA_VISIBLE_DEVICES subset: go through the UUID
        uuid = torch.cuda.get_device_properties(self.index).uuid
        try:
            self._handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
        except Exception:
            self._handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
        self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM))

    def _run(self):
        n = self._nvml
        while not self._stop.is_set():
            try:
                self.samples.append(float(n.nvmlDeviceGetClockInfo(self._handle, n.NVML_CLOCK_SM)))
                self.power.append(n.nvmlDeviceGetPowerUsage(self._handle) / 1000.0)
                mask = n.nvmlDeviceGetCurrentClocksEventReasons(self._handle) if hasattr(
                    n, "nvmlDeviceGetCurrentClocksEventReasons") else n.nvmlDeviceGetCurrentClocksThrottleReasons(self._handle)
                for name, bit in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(0.002)

    def start(self):
        try:
            self._open()
        except Exception:
            self._nvml = None
            return
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread:
            self._thread.join(timeout=10)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_min_mhz": min(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "power_w_max": max(self.power) if self.power else None,
                "samples": len(self.samples), "source": "nvml"}


# ---------------------------------------------------------------------------------------------------------
# workloads
class Workload:
    """What one step runs: a list of LbaCall with the formats, the order and the kind of pass."""

    def __init__(self, name, prod, acc, order, chunk=16, ste=None, fixed=None, batch=None):
        self.name, self.prod, self.acc, self.order, self.chunk = name, prod, acc, order, chunk
        self.ste, self.fixed, self.batch = ste, fixed, batch
        self.calls = []
        self.ste_eps = (2.0 ** -20, 0.25)

    def run_call(self, c, stream=None):
        from paper_2401_14110_b200 import binding as lba
        if c.kind == "conv":
            lba.lba_conv2d(c.x, c.w, c.sx, c.sw, None, c.stride, c.pad, self.prod, self.acc, self.order, self.chunk,
                           out=c.out_nhwc, stream=stream)
        elif c.kind == "bgemm":
            lba.lba_gemm_batched(c.x, c.w, c.sx, c.sw, None, self.prod, self.acc, self.order, self.chunk, out=c.out)
        elif c.kind == "ste":
            lba.lba_gemm_ste_mask(c.x, c.w, self.prod, self.acc, self.order, self.chunk,
                                  lba.STE_DIFF if self.ste == "diff" else lba.STE_OF, self.ste_eps[0], self.ste_eps[1],
                                  mask1=c.mask1, mask2=c.mask2)
        else:
            lba.lba_gemm(c.x, c.w, c.sx, c.sw, None, self.prod, self.acc, self.order, self.chunk, out=c.out, stream=stream)

    def run_step(self, events=None, streams=None):
        for i, c in enumerate(self.calls):
            if events is not None:
                events[i][0].record()
            self.run_call(c, None if streams is None else streams[i % len(streams)])
            if events is not None:
                events[i][1].record()

    def describe(self, c):
        from paper_2401_14110_b200 import binding as lba
        m, n, k = c.gemm_shape
        if c.kind == "ste":
            return "ste_mask=%s tile=64x64x16 micro=%s q=floor order=%s" % (
                self.ste, "4x8 packed" if self.ste == "of" else "4x4 scalar", "chunk16" if self.order else "seq")
        vec = (c.x.shape[-1] % 16 == 0) if c.kind == "conv" else (k % 16 == 0)
        return lba.describe_plan(m, n, k, self.prod, self.acc, self.order, self.chunk, is_conv=c.kind == "conv", vec_ok=vec,
                                 batch=c.x.shape[0] if c.kind == "bgemm" else 1)

    @property
    def macs(self):
        return sum(c.macs for c in self.calls)

    def finish(self, device):
        from paper_2401_14110_b200 import binding as lba
        for c in self.calls:
            m, n, _ = c.gemm_shape
            if c.out is None:
                c.out = torch.empty((m, n), dtype=torch.float32, device=device)
            if c.kind == "conv":
                b, h, w, _ = c.x.shape
                ho, wo = lba.conv_out_hw(h, w, c.w.shape[1], c.w.shape[2], c.stride, c.pad)
                c.out_nhwc = c.out.view(b, ho, wo, c.w.shape[0])
        return self


def parse_format_tokens(tokens, default=(7, 4, 0)):
    """(M, E, rounding) from workload tokens such as 'm4e5' and 'rne'."""
    m, e, rnd = default
    for t in tokens:
        if t == "rne":
            rnd = 1
        elif t.startswith("m") and "e" in t[1:]:
            a, b = t[1:].split("e")
            m, e = int(a), int(b)
    return m, e, rnd


def gemm_operands(m, n, k, device, config=5, outliers=False, weight_std=1.0):
    from paper_2401_14110_b200 import synth
    a, sa, b, sb = synth.gemm_case(m, n, k, config=config, outliers=outliers, weight_std=weight_std)
    return a.to(device), sa.to(device), b.to(device), sb.to(device)


def build_workload(spec: str, device):
    """A Workload from a --workload string."""
    from paper_2401_14110_b200 import (binding as lba, synth, workloads, code_domain_formats, fixed_point_format,
                                       m4e3_input_formats, ORDER_CHUNKED, ORDER_SEQUENTIAL)
    parts = spec.lower().split(":")
    kind = parts[0]
    m4e3 = "wa=m4e3" in parts[1:]   # operands in the paper's own weight/activation byte format (Sec. 3.1) instead of OCP E4M3
    if kind in ("resnet18", "resnet50"):
        prod, acc = m4e3_input_formats(7, 4) if m4e3 else code_domain_formats(7, 4)
        batch, config = (32, 2) if kind == "resnet18" else (64, 3)
        wl = Workload(f"{kind}_fwd_conv_stack_b{batch}_224_{'wa_m4e3_' if m4e3 else ''}m7e4_chunk16", prod, acc, ORDER_CHUNKED,
                      batch=batch)

        def conv_fn(x, w, sx, sw, stride, pad):
            return lba.lba_conv2d(x, w, sx, sw, None, stride, pad, prod, acc, ORDER_CHUNKED, 16)

        def gemm_fn(a, b, sa, sb):
            return lba.lba_gemm(a, b, sa, sb, None, prod, acc, ORDER_CHUNKED, 16)

        wl.calls, _ = workloads.build_resnet_calls(kind, batch, config, device, conv_fn, gemm_fn,
                                                   wa_format="m4e3" if m4e3 else "e4m3")
        return wl.finish(device)
    if kind == "bert":
        seq = "seq" in parts[1:]
        prod, acc = code_domain_formats(7, 4)
        wl = Workload("bert_base_linears_4096tok_m7e4_%s" % ("sequential" if seq else "chunk16"), prod, acc,
                      ORDER_SEQUENTIAL if seq else ORDER_CHUNKED)
        wl.calls = workloads.build_bert_calls(4096, 4, device)
        return wl.finish(device)
    dims = tuple(int(v) for v in parts[1].split("x"))
    order = ORDER_SEQUENTIAL if "seq" in parts[2:] else ORDER_CHUNKED
    oname = "sequential" if order == ORDER_SEQUENTIAL else "chunk16"
    if kind == "bgemm":
        if len(dims) != 4:
            raise SystemExit("--workload bgemm:ZxMxNxK")
        z, m, n, k = dims
        prod, acc = code_domain_formats(7, 4)
        wl = Workload("batched_lba_gemm_%dx%dx%dx%d_m7e4_%s" % (dims + (oname,)), prod, acc, order)
        a = synth.e4m3_encode(synth.gaussian((z, m, k), synth.seed_for(5, 0)) * 100.0)
        b = synth.e4m3_encode(synth.gaussian((z, n, k), synth.seed_for(5, 1)) * 100.0)
        one = torch.ones(1, device=device)
        c = workloads.LbaCall("bgemm", "bgemm", a.to(device), b.to(device), one, one)
        c.out = torch.empty((z, m, n), dtype=torch.float32, device=device)
        wl.calls = [c]
        return wl
    if len(dims) != 3:
        raise SystemExit("--workload %s:MxNxK" % kind)
    m, n, k = dims
    a, sa, b, sb = gemm_operands(m, n, k, device)
    if kind == "gemm":
        M_, E_, rnd = parse_format_tokens(parts[2:])
        prod, acc = (m4e3_input_formats if m4e3 else code_domain_formats)(M_, E_, rnd)
        if m4e3:   # the same Gaussian operands, quantised per tensor to the paper's byte format
            ga, gb = synth.gaussian((m, k), synth.seed_for(5, 0)), synth.gaussian((n, k), synth.seed_for(5, 1))
            (a, sa), (b, sb) = synth.quantise_m4e3_per_tensor(ga), synth.quantise_m4e3_per_tensor(gb)
            a, sa, b, sb = a.to(device), sa.to(device), b.to(device), sb.to(device)
        wl = Workload("single_lba_gemm_%dx%dx%d_%sm%de%d%s_%s" % (m, n, k, "wa_m4e3_" if m4e3 else "", M_, E_,
                                                                  "_rne" if rnd else "", oname), prod, acc, order)
        wl.calls = [workloads.LbaCall("gemm", "gemm", a, b, sa, sb)]
    elif kind == "fixed":
        wrap = "wrap" in parts[2:]
        # 12-bit fixed-point formats with the ranges of the 12-bit floating ones: products up to 2^7 * 2047 >= 448^2,
        # sums up to 2^9 * 2047 (R_OF of the M7E4 accumulator is 1044480)
        prod, acc = fixed_point_format(12, -7, wrap), fixed_point_format(12, -9, wrap)
        wl = Workload("fixed12_%s_gemm_%dx%dx%d_%s" % ("wrap" if wrap else "sat", m, n, k, oname), prod, acc, order,
                      fixed="wrap" if wrap else "sat")
        wl.calls = [workloads.LbaCall("gemm", "gemm", a, b, sa, sb)]
    elif kind == "ste":
        ste = "diff" if "diff" in parts[2:] else "of"
        prod, acc = code_domain_formats(7, 4)
        wl = Workload("ste_%s_mask_%dx%dx%d_m7e4_%s" % (ste, m, n, k, oname), prod, acc, order, ste=ste)
        c = workloads.LbaCall("gemm", "ste", a, b, sa, sb)
        c.mask1 = torch.empty((m, (k + 31) // 32, n), dtype=torch.int32, device=device)
        c.mask2 = torch.empty((m, ((k + 15) // 16 + 31) // 32, n), dtype=torch.int32, device=device) if order else None
        wl.calls = [c]
    else:
        raise SystemExit("unknown --workload")
    return wl.finish(device)


def time_workload(wl, steps, warmup, barrier=None):
    """(ms per step over the whole bracket, mean ms of every call) with CUDA events on the launching stream."""
    for _ in range(warmup):
        wl.run_step()
    (barrier or torch.cuda.synchronize)()
    events = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in wl.calls]
              for _ in range(steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for s in range(steps):
        wl.run_step(events[s])
    stop.record()
    (barrier or torch.cuda.synchronize)()
    per_call = [statistics.mean(events[s][i][0].elapsed_time(events[s][i][1]) for s in range(steps))
                for i in range(len(wl.calls))]
    return start.elapsed_time(stop) / steps, per_call


def kernel_table(wl, per_call_ms, sm_count, max_mhz):
    """Per kernel variant: time, launches, MACs, GMAC/s, roofline peak and fraction."""
    table = {}
    for c, ms in zip(wl.calls, per_call_ms):
        d = wl.describe(c)
        key = " ".join(p for p in d.split() if not p.startswith("grid="))
        e = table.setdefault(key, {"ms": 0.0, "macs": 0, "launches": 0})
        e["ms"] += ms
        e["macs"] += c.macs
        e["launches"] += 1
    for key, e in table.items():
        mode = mode_of(key, ste=wl.ste if wl.ste == "diff" else None, fixed=wl.fixed is not None)
        peak, slots, pipe = peak_gmacs(mode, wl.chunk if wl.order == 1 else 0, sm_count, max_mhz)
        e.update(gmacs=e["macs"] / (e["ms"] * 1e-3) / 1e9, mode=mode, peak=peak, slots=slots, pipe=pipe)
        e["frac"] = e["gmacs"] / peak
    return table


def summary_entry(wl, ms_per_step, per_call_ms, sm_count, max_mhz):
    """One line of the "configs" object."""
    table = kernel_table(wl, per_call_ms, sm_count, max_mhz)
    dom_key, dom = max(table.items(), key=lambda kv: kv[1]["ms"])
    # the step's own roofline: every call at the peak of the variant it runs
    ideal_ms = sum(e["macs"] / (e["peak"] * 1e9) * 1e3 for e in table.values())
    return {"workload": wl.name, "lba_calls": len(wl.calls), "macs": wl.macs, "ms": ms_per_step,
            "gmacs": wl.macs / (ms_per_step * 1e-3) / 1e9, "frac": ideal_ms / sum(per_call_ms),
            "dominant_kernel": dom_key, "dominant_kernel_gmacs": dom["gmacs"], "dominant_kernel_frac": dom["frac"],
            "dominant_kernel_share": dom["ms"] / sum(per_call_ms)}


def other_configs(device, sm_count, max_mhz, headline_wl):
    """GMAC/s and roofline fraction of the benchmark configurations the headline does not cover."""
    from paper_2401_14110_b200 import binding as lba, workloads, code_domain_formats, ORDER_CHUNKED, ORDER_SEQUENTIAL
    out = {}
    # config 1: one small GEMM in sequential order (latency-bound: 4096 chains of 576 dependent steps; for information)
    wl = build_workload("gemm:64x64x576:seq", device)
    wl.calls[0].x, wl.calls[0].sx, wl.calls[0].w, wl.calls[0].sw = gemm_operands(64, 64, 576, device, config=1)
    ms, per = time_workload(wl, 200, 20)
    e = summary_entry(wl, ms, per, sm_count, max_mhz)
    e["us_per_launch"] = per[0] * 1e3
    # the same launch replayed from a CUDA graph (32 per replay): the device time without the host's launch path
    side = torch.cuda.Stream(device=device)
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        wl.run_step()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(32):
            wl.run_step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        graph.replay()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(10):
        graph.replay()
    t1.record()
    torch.cuda.synchronize()
    e["us_per_launch_in_graph"] = t0.elapsed_time(t1) * 1e3 / 320
    e["gmacs_in_graph"] = wl.macs / (e["us_per_launch_in_graph"] * 1e-6) / 1e9
    e["note"] = "latency-bound by construction: 4096 outputs, 576 dependent steps each"
    out["config1_gemm_64x64x576_sequential"] = e
    # configs 2 and 3: the convolution stacks
    for name, steps in (("resnet18", 10), ("resnet50", 5)):
        wl = build_workload(name, device)
        ms, per = time_workload(wl, steps, 3)
        e = summary_entry(wl, ms, per, sm_count, max_mhz)
        table = kernel_table(wl, per, sm_count, max_mhz)
        e["kernels"] = {k: {"ms": v["ms"], "launches": v["launches"], "gmacs": v["gmacs"], "frac": v["frac"]}
                        for k, v in table.items()}
        out["config%d_%s" % (2 if name == "resnet18" else 3, wl.name)] = e
        del wl
        torch.cuda.empty_cache()
    # config 4: the six linear layers of a BERT-base encoder layer, both orders
    for order in ("chunk", "seq"):
        wl = build_workload("bert:" + order, device)
        ms, per = time_workload(wl, 10, 3)
        e = summary_entry(wl, ms, per, sm_count, max_mhz)
        e["layers"] = {c.name: {"shape": list(c.gemm_shape), "ms": t, "gmacs": c.macs / (t * 1e-3) / 1e9}
                       for c, t in zip(wl.calls, per)}
        out["config4_" + wl.name] = e
    # config 5: accumulator-format sweep on the headline's operands (mantissa 4..10 x exponent 4..6 x two roundings)
    c0 = headline_wl.calls[0]
    points, by_mode = {}, {}
    for rnd in (0, 1):
        for E_ in (4, 5, 6):
            for M_ in range(4, 11):
                prod, acc = code_domain_formats(M_, E_, rnd)
                wl = Workload("m%de%d_%s" % (M_, E_, "rne" if rnd else "floor"), prod, acc, ORDER_CHUNKED)
                wl.calls = [workloads.LbaCall("gemm", "gemm", c0.x, c0.w, c0.sx, c0.sw, out=c0.out)]
                ms, per = time_workload(wl, 2, 1)
                table = kernel_table(wl, per, sm_count, max_mhz)
                (key, e), = table.items()
                points[wl.name] = {"ms": per[0], "gmacs": e["gmacs"], "mode": e["mode"], "frac": e["frac"]}
                by_mode.setdefault(e["mode"], []).append((e["gmacs"], e["frac"], e["peak"], key, e["pipe"]))
    modes = {m: {"points": len(v), "gmacs_min": min(x[0] for x in v), "gmacs_median": statistics.median(x[0] for x in v),
                 "gmacs_max": max(x[0] for x in v), "frac_median": statistics.median(x[1] for x in v), "peak": v[0][2],
                 "mix": MIX[m][4], "kernel": v[0][3], "pipe_limit": v[0][4]} for m, v in by_mode.items()}
    out["config5_format_sweep_gemm_8192x8192x8192_chunk16"] = {
        "points": points, "modes": modes, "note": "one warm-up and two timed launches per point; biases by the flex-bias rule "
        "applied to products (b_prod = 2^E - 18, b_acc = b_prod - 2)"}
    return out


# ---------------------------------------------------------------------------------------------------------
def cpu_baseline(wl, target_macs):
    """Time the oracle, as it stands, on a bounded sample: seeded 16x16 output tiles of the workload's calls."""
    from oracle import lba_oracle as orc
    from paper_2401_14110_b200 import synth
    calls = wl.calls
    picks = ([c for c in calls if c.kind == "conv"][1::4] + [calls[0]]) if len(calls) > 1 else calls
    per_layer = target_macs / len(picks)
    jobs = []
    for i, c in enumerate(picks):
        m, n, k = c.gemm_shape
        tiles = max(1, int(per_layer / (256 * k)))
        ms, ns = synth.sample_tiles(m, n, tiles, 16, 777 + i)
        jobs.append((c, c.x.cpu().numpy(), c.w.cpu().numpy(), c.sx.cpu().numpy(), c.sw.cpu().numpy(), ms, ns, k))
    cores = orc.default_threads()
    orc.lib()
    t0 = time.perf_counter()
    macs = 0
    for c, x, w, sx, sw, ms, ns, k in jobs:
        if c.kind == "conv":
            orc.conv2d_points(x, w, sx, sw, None, c.stride, c.pad, wl.prod.as_tuple(), wl.acc.as_tuple(), wl.order, wl.chunk,
                              ms, ns, nthreads=cores)
        else:
            orc.gemm_points(x, w, sx, sw, None, wl.prod.as_tuple(), wl.acc.as_tuple(), wl.order, wl.chunk, ms, ns,
                            nthreads=cores)
        macs += len(ms) * k
    dt = time.perf_counter() - t0
    return {"value": macs / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(jobs)} call(s) x seeded 16x16 output tiles, {macs:.3g} MACs in {dt:.1f} s",
            "macs": macs, "seconds": dt}


def reference_arm(args):
    """The oracle timed on the host cores; each step is a bounded sample (seeded 16x16 output tiles) of the headline GEMM."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import lba_oracle as orc
    from paper_2401_14110_b200 import synth, code_domain_formats, ORDER_CHUNKED
    prod, acc = code_domain_formats(7, 4)
    m = n = k = 8192
    a, sa, b, sb = synth.gemm_case(m, n, k, config=5)
    a, sa, b, sb = a.numpy(), sa.numpy(), b.numpy(), sb.numpy()
    cores = orc.default_threads()
    tiles = 24
    ms_, ns_ = synth.sample_tiles(m, n, tiles, 16, 900)
    step_macs = len(ms_) * k

    def step():
        orc.gemm_points(a, b, sa, sb, None, prod.as_tuple(), acc.as_tuple(), ORDER_CHUNKED, 16, ms_, ns_, nthreads=cores)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = step_macs * args.steps / dt / 1e9
    sample = f"per step: {tiles} seeded 16x16 output tiles of the 8192x8192x8192 GEMM, {step_macs:.3g} MACs"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int128", "data": "synthetic",
        "config": {"workload": "single_lba_gemm_8192x8192x8192_m7e4_chunk16", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def end_to_end(wl, args, device, world, dist, barrier):
    """The same step through the host-buffer C entry points: pinned host operands in, pinned host result out."""
    from paper_2401_14110_b200 import binding as lba, sharding
    host, ws_bytes, h2d, d2h = [], 0, 0, 0
    for c in wl.calls:
        hx, hw_, hsx, hsw = (t.cpu().pin_memory() for t in (c.x, c.w, c.sx, c.sw))
        hout = torch.empty(c.out.shape if c.kind == "gemm" else c.out_nhwc.shape, dtype=torch.float32).pin_memory()
        if c.kind == "conv":
            b, h, w, cin = c.x.shape
            cout, kh, kw, _ = c.w.shape
            need = lba.conv2d_host_workspace_bytes(b, h, w, cin, cout, kh, kw, c.stride, c.pad, 1, cout, False)
        else:
            m, n, k = c.gemm_shape
            need = lba.gemm_host_workspace_bytes(m, n, k, hsx.numel(), hsw.numel(), False)
        ws_bytes = max(ws_bytes, need)
        h2d += hx.numel() + hw_.numel() + 4 * (hsx.numel() + hsw.numel())
        d2h += 4 * hout.numel()
        host.append((c, hx, hw_, hsx, hsw, hout))
    whole = [(c, hout) for c, _, _, _, _, hout in host]
    # independent calls of a step are spread round-robin over a few streams, each with its own workspace: one call's
    # copies overlap another call's kernel.  A single GEMM is issued as row blocks for the same reason: the rows of the
    # output are independent chains, so each block is a complete lba_gemm_host call on its own rows (B travels with
    # every block, which the byte counts include)
    blocks = 1
    if len(host) == 1 and host[0][0].kind == "gemm" and host[0][3].numel() == 1 and args.e2e_row_blocks > 1:
        c, hx, hw_, hsx, hsw, hout = host[0]
        m, n, k = c.gemm_shape
        blocks = min(args.e2e_row_blocks, m)
        spans = [sharding.shard_rows(m, blocks, r) for r in range(blocks)]
        host = [(c, hx[a:b], hw_, hsx, hsw, hout[a:b]) for a, b in spans]
        ws_bytes = max(lba.gemm_host_workspace_bytes(b - a, n, k, 1, hsw.numel(), False) for a, b in spans)
        h2d = hx.numel() + blocks * (hw_.numel() + 4 * hsw.numel() + 4)
    n_streams = max(1, min(args.e2e_streams, len(host), 3 if blocks > 1 else len(host)))
    streams = [torch.cuda.Stream(device=device) for _ in range(n_streams)]
    wss = [torch.empty(ws_bytes, dtype=torch.uint8, device=device) for _ in range(n_streams)]
    torch.cuda.synchronize()

    def step():
        for i, (c, hx, hw_, hsx, hsw, hout) in enumerate(host):
            st, ws = streams[i % n_streams], wss[i % n_streams]
            if c.kind == "conv":
                lba.lba_conv2d_host(hx, hw_, hsx, hsw, None, c.stride, c.pad, wl.prod, wl.acc, wl.order, wl.chunk, hout, ws,
                                    stream=st)
            else:
                lba.lba_gemm_host(hx, hw_, hsx, hsw, None, wl.prod, wl.acc, wl.order, wl.chunk, hout, ws, stream=st)
    steps = max(2, min(args.steps, 10))
    step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    barrier()
    ms = sharding.max_over_ranks((time.perf_counter() - t0) * 1e3 / steps, dist, device)
    # the host results are the device-resident step's results, bit for bit
    wl.run_step()
    torch.cuda.synchronize()
    same = all(torch.equal(hout, (c.out if c.kind == "gemm" else c.out_nhwc).cpu()) for c, hout in whole)
    return {"value": sharding.whole_job_rate(wl.macs, world, ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": ms, "steps": steps, "equals_device_step": same,
            "api": "lba_gemm_host / lba_conv2d_host (pinned host buffers, caller-owned device workspaces, "
                   f"{len(host)} call(s) over {n_streams} stream(s)" + (f": {blocks} row blocks of one GEMM" if blocks > 1 else "") + ")"}


def main(argv=None):
    args = parse_args(argv)
    if args.impl == "reference":
        reference_arm(args)
        return 0
    from paper_2401_14110_b200 import launcher
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        # no launcher environment: start the ranks here, one process per GPU
        return launcher.spawn_ranks(args.gpus, [os.path.abspath(__file__)] + (sys.argv[1:] if argv is None else list(argv)),
                                    devices=torch.cuda.device_count())
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the LBA library has no CPU path")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1 or args.force_dist:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29511")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=device)

    from paper_2401_14110_b200 import binding as lba, sharding
    lba.load_library()
    wl = build_workload(args.workload, device)
    step_macs = wl.macs

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        wl.run_step()
    barrier()

    # ---- timed region: K steps, per-launch CUDA events on the launching stream
    events = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in wl.calls]
              for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    for s in range(args.steps):
        wl.run_step(events[s])
    stop.record()
    barrier()
    clocks = sampler.stop()
    total_ms = sharding.max_over_ranks(start.elapsed_time(stop), dist, device)
    ms_per_step = total_ms / args.steps
    value = sharding.whole_job_rate(step_macs, world, ms_per_step * 1e-3) / 1e9

    # ---- per-kernel accounting from the per-launch events
    per_call_ms = [statistics.mean(events[s][i][0].elapsed_time(events[s][i][1]) for s in range(args.steps))
                   for i in range(len(wl.calls))]
    sm_count = torch.cuda.get_device_properties(device).multi_processor_count
    max_mhz = clocks["sm_max_mhz"] or 1965.0
    mhz = clocks["sm_mhz"] or max_mhz
    table = kernel_table(wl, per_call_ms, sm_count, max_mhz)
    dom_key, dom = max(table.items(), key=lambda kv: kv[1]["ms"])
    ncu = NCU.get((wl.name, dom_key))
    ideal_ms = sum(e["macs"] / (e["peak"] * 1e9) * 1e3 for e in table.values())
    roofline = {
        "bound": "alu", "achieved": dom["gmacs"], "peak": dom["peak"], "unit": UNIT, "frac": dom["frac"],
        "traffic": ncu[0] if ncu else None,
        "traffic_note": ncu[1] if ncu else "no ncu capture of this kernel on this workload",
        "instr_per_mac": ncu[2] if ncu else None,
        "instr_per_mac_minimum": min_issue_slots(dom["mode"], wl.chunk if wl.order == 1 else 0),
        "kernel": dom_key, "kernel_launches_per_step": dom["launches"], "kernel_ms_per_step": dom["ms"],
        "kernel_share_of_step": dom["ms"] / sum(per_call_ms),
        "peak_derivation": f"{sm_count} SMs x {LANES_PER_SM_CLK} lanes issued per clock x {max_mhz:.0f} MHz (clocks.max.sm) / "
                           f"{dom['slots']:g} issue slots per emulated MAC of the minimal mix ({MIX[dom['mode']][4]}"
                           + (f", plus {FOLD.get('rne' if dom['mode'].startswith('rne') else 'floor', FOLD['generic'])[0]:g} per output "
                              f"per chunk of {wl.chunk}" if wl.order == 1 else "") + ")",
        "pipe_limit": dom["pipe"],
        "frac_at_sampled_clock": dom["gmacs"] / (dom["peak"] * mhz / max_mhz),
        "whole_step_frac_of_peak": ideal_ms / sum(per_call_ms),
    }
    if wl.ste is not None:   # one bit per step: the masks are the bulk of the algorithmic bytes
        mask_bytes = sum(c.mask1.numel() * 4 + (c.mask2.numel() * 4 if c.mask2 is not None else 0) for c in wl.calls)
        roofline["mask_bytes_per_launch"] = mask_bytes
        roofline["mask_write_gbs"] = mask_bytes / (dom["ms"] * 1e-3) / 1e9

    # ---- network workloads: the same device-resident step with its (independent) calls spread over several streams
    concurrent = None
    if len(wl.calls) > 1 and args.e2e_streams > 1:
        cstreams = [torch.cuda.Stream(device=device) for _ in range(args.e2e_streams)]
        barrier()
        wl.run_step(streams=cstreams)
        barrier()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for st in cstreams:
            st.wait_event(c0)
        for _ in range(args.steps):
            wl.run_step(streams=cstreams)
        for st in cstreams:
            torch.cuda.current_stream().wait_stream(st)
        c1.record()
        barrier()
        cms = sharding.max_over_ranks(c0.elapsed_time(c1), dist, device) / args.steps
        concurrent = {"value": sharding.whole_job_rate(step_macs, world, cms * 1e-3) / 1e9, "unit": UNIT,
                      "ms_per_step": cms, "streams": args.e2e_streams}

    kernel_only = wl.ste is not None or wl.fixed is not None or wl.calls[0].kind == "bgemm"
    e2e = None if (args.no_e2e or kernel_only) else end_to_end(wl, args, device, world, dist, barrier)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not kernel_only:
        cpu = cpu_baseline(wl, args.cpu_baseline_macs)
    configs = None
    want_configs = args.configs == "all" or (args.configs == "auto" and args.workload == HEADLINE)
    if rank == 0 and world == 1 and want_configs:
        configs = other_configs(device, sm_count, max_mhz, wl)

    if rank == 0:
        working_set = sum(c.x.numel() + c.w.numel() + 4 * c.out.numel() for c in wl.calls)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": wl.name, "lba_calls_per_step": len(wl.calls),
                       "macs_per_step_per_gpu": step_macs, "prod_fmt": list(wl.prod.as_tuple()),
                       "acc_fmt": list(wl.acc.as_tuple()), "order": "chunked" if wl.order == 1 else "sequential",
                       "chunk": wl.chunk,
                       "l2": f"no flush: each step streams {working_set / 1e6:.0f} MB of distinct operands and "
                             f"outputs, larger than the 126 MB L2",
                       "parallelism": f"dp{world} (rows sharded, weights replicated, no collective)"},
            "clocks": clocks, "gpu_launches": len(wl.calls) * args.steps,
            "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu, "concurrent": concurrent,
            "kernels": {k: {"ms_per_step": v["ms"], "launches_per_step": v["launches"], "gmacs": v["gmacs"],
                            "frac": v["frac"]} for k, v in table.items()},
            "configs": configs,
        }
        if wl.batch:
            line["config"]["batch_per_gpu"] = wl.batch
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
