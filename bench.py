#!/usr/bin/env python
"""Benchmark of the LBA contraction on B200: emulated GMAC/s and fraction of the ALU roofline.

Workload (N = 1 GPU): the ResNet-18 forward convolution stack as implicit LBA GEMMs, batch 32,
synthetic 224x224x3 N(0,1) images, He-normal weights quantised to E4M3 per output channel, activations
re-quantised per tensor, M7E4 product and accumulator formats (12-bit accumulator), chunk-16 accumulation
(the paper's order), floor rounding.  A step is one pass over all 20 convolutions and the final linear
layer through lba_conv2d / lba_gemm; operands are produced once by a real forward pass (PyTorch glue
between layers) and stay resident in HBM.  With N > 1 every rank runs the same step on its own batch
(rows of the implicit GEMM are independent; no collective on the data path): weak scaling.

One JSON line is printed by rank 0.  `--impl reference` times the CPU oracle instead (rank 0 only).
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
WORKLOAD = "resnet18_fwd_conv_stack_b32_224_m7e4_chunk16"
BATCH = 32
CONFIG_ID = 2
RUN_ORDER = 1        # ORDER_CHUNKED, the paper's order; a single-GEMM workload may ask for the sequential order
GEMM_CASE = None     # (M, N, K) when --workload gemm:MxNxK[:seq|chunk] replaces the network
STE_KIND = None      # "of" / "diff" when --workload ste:... times the mask re-computation pass
STE_EPS = (2.0 ** -20, 0.25)
FIXED_POINT = None   # "sat" / "wrap" when --workload fixed:... times the fixed-point accumulator (Eq. 1)

# ALU roofline for sm_100.  Per SM and clock 4 schedulers issue one warp instruction each (128 lanes), the
# FP32 pipe retires 128 lanes and the integer/logic pipe 64.  The packed floor path needs, per emulated MAC,
# half an FMUL2 and half an FFMA2 (one FP32 lane-op each) and one LOP3 (the mantissa mask), i.e. 2 issue
# slots, 2 FP32 lane-ops and 1 logic lane-op: all three limits coincide at 2 clocks per warp-MAC per
# scheduler.  The chunked order adds, per chunk of `chunk` MACs, one packed add, two masks and two clamps
# per output pair: (0.5 + 1 + 1) issue slots per output.
ISSUE_LANES_PER_SM_CLK = 128
ISSUE_SLOTS_PER_MAC_LEVEL1 = 2.0
ISSUE_SLOTS_PER_CHUNK_CLOSE = 2.5


# DRAM bytes (read + write) of ONE launch of the dominant kernel, from the ncu captures summarised under profiles/
# (workload, kernel description) -> (bytes, what was captured).  A kernel that is not listed reports null.
NCU_DRAM_TRAFFIC = {
    ("resnet18_fwd_conv_stack_b32_224_m7e4_chunk16", "tile=64x64x16 micro=4x8 q=floor_fast order=chunk16 load=conv_vec"):
        (3425280, "one of the 14 launches (layer2.0.conv2, M=25088 N=128 K=1152): 3.4 MB read, 0 written while the kernel "
                  "ran (its 12.8 MB output was still in L2); algorithmic 16.2 MB"),
    ("single_lba_gemm_8192x8192x1024_m7e4_chunk16", "tile=64x64x16 micro=4x8 q=floor_fast order=chunk16 load=gemm_vec"):
        (230966784, "17.2 MB read + 213.7 MB written; algorithmic 272 MB (part of the output still in L2)"),
    ("single_lba_gemm_8192x8192x1024_m7e4_sequential", "tile=128x128x16 micro=8x8 q=floor_fast order=seq load=gemm_vec"):
        (230249216, "18.0 MB read + 212.3 MB written; algorithmic 272 MB (part of the output still in L2)"),
}


def issue_slots_per_mac(order_chunked: bool, chunk: int) -> float:
    return ISSUE_SLOTS_PER_MAC_LEVEL1 + (ISSUE_SLOTS_PER_CHUNK_CLOSE / chunk if order_chunked else 0.0)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18",
                    help="resnet18 (default, the benchmark), gemm:MxNxK[:seq|chunk] (one LBA GEMM on Gaussian "
                         "operands, used for kernel profiles), bgemm:ZxMxNxK[:seq|chunk] (one batched call) or "
                         "ste:MxNxK[:of|diff][:seq|chunk] (STE mask re-computation of one GEMM) or "
                         "fixed:MxNxK[:seq|chunk][:wrap] (one GEMM with 12-bit fixed-point accumulation, Eq. 1)")
    ap.add_argument("--cpu-baseline-macs", type=float, default=1.5e9,
                    help="size of the oracle sample timed for cpu_baseline (emulated MACs)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-streams", type=int, default=12,
                    help="streams (each with its own device workspace) the end-to-end calls are spread over")
    ap.add_argument("--force-dist", action="store_true",
                    help="initialise torch.distributed (NCCL) even for a single rank: exercises the multi-GPU plumbing "
                         "(barrier, max over ranks) on one GPU")
    return ap.parse_args()


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


def formats():
    from paper_2401_14110_b200 import code_domain_formats, fixed_point_format
    if FIXED_POINT is not None:
        # 12-bit fixed-point formats with the ranges of the 12-bit floating ones: products up to 2^7 * 2047 >= 448^2,
        # sums up to 2^9 * 2047 (R_OF of the M7E4 accumulator is 1044480)
        wrap = FIXED_POINT == "wrap"
        return fixed_point_format(12, -7, wrap), fixed_point_format(12, -9, wrap)
    return code_domain_formats(7, 4)


def build_calls(device):
    from paper_2401_14110_b200 import binding as lba, synth, workloads, ORDER_CHUNKED
    prod, acc = formats()
    if GEMM_CASE is not None and len(GEMM_CASE) == 4:      # batched: Z problems of M x N x K (attention matmuls)
        z, m, n, k = GEMM_CASE
        a = synth.e4m3_encode(synth.gaussian((z, m, k), synth.seed_for(5, 0)) * 100.0)
        b = synth.e4m3_encode(synth.gaussian((z, n, k), synth.seed_for(5, 1)) * 100.0)
        one = torch.ones(1, device=device)
        c = workloads.LbaCall("bgemm", "bgemm", a.to(device), b.to(device), one, one)
        c.out = torch.empty((z, m, n), dtype=torch.float32, device=device)
        return [c]
    if GEMM_CASE is not None:
        m, n, k = GEMM_CASE
        a, sa, b, sb = synth.gemm_case(m, n, k, config=5)
        c = workloads.LbaCall("gemm", "gemm", a.to(device), b.to(device), sa.to(device), sb.to(device))
        c.out = torch.empty((m, n), dtype=torch.float32, device=device)
        if STE_KIND is not None:
            c.kind = "ste"
            c.mask1 = torch.empty((m, (k + 31) // 32, n), dtype=torch.int32, device=device)
            c.mask2 = torch.empty((m, ((k + 15) // 16 + 31) // 32, n), dtype=torch.int32, device=device) if RUN_ORDER else None
        return [c]

    def conv_fn(x, w, sx, sw, stride, pad):
        return lba.lba_conv2d(x, w, sx, sw, None, stride, pad, prod, acc, ORDER_CHUNKED, 16)

    def gemm_fn(a, b, sa, sb):
        return lba.lba_gemm(a, b, sa, sb, None, prod, acc, ORDER_CHUNKED, 16)

    calls, _ = workloads.build_resnet_calls("resnet18", BATCH, CONFIG_ID, device, conv_fn, gemm_fn)
    for c in calls:
        m, n, _ = c.gemm_shape
        c.out = torch.empty((m, n), dtype=torch.float32, device=device)
    return calls


def run_step(calls, events=None, streams=None):
    from paper_2401_14110_b200 import binding as lba
    ORDER_CHUNKED = RUN_ORDER
    prod, acc = formats()
    for i, c in enumerate(calls):
        if events is not None:
            events[i][0].record()
        st = None if streams is None else streams[i % len(streams)]
        if c.kind == "conv":
            lba.lba_conv2d(c.x, c.w, c.sx, c.sw, None, c.stride, c.pad, prod, acc, ORDER_CHUNKED, 16, out=c.out_nhwc,
                           stream=st)
        elif c.kind == "bgemm":
            lba.lba_gemm_batched(c.x, c.w, c.sx, c.sw, None, prod, acc, ORDER_CHUNKED, 16, out=c.out)
        elif c.kind == "ste":
            lba.lba_gemm_ste_mask(c.x, c.w, prod, acc, ORDER_CHUNKED, 16, lba.STE_DIFF if STE_KIND == "diff" else lba.STE_OF,
                                  STE_EPS[0], STE_EPS[1], mask1=c.mask1, mask2=c.mask2)
        else:
            lba.lba_gemm(c.x, c.w, c.sx, c.sw, None, prod, acc, ORDER_CHUNKED, 16, out=c.out, stream=st)
        if events is not None:
            events[i][1].record()


def describe(c):
    from paper_2401_14110_b200 import binding as lba
    ORDER_CHUNKED = RUN_ORDER
    prod, acc = formats()
    m, n, k = c.gemm_shape
    if c.kind == "ste":
        return "ste_mask=%s tile=64x64x16 micro=%s q=floor order=%s" % (
            STE_KIND, "4x8 packed" if STE_KIND == "of" else "4x4 scalar", "chunk16" if RUN_ORDER else "seq")
    vec = (c.x.shape[-1] % 16 == 0) if c.kind == "conv" else (k % 16 == 0)
    return lba.describe_plan(m, n, k, prod, acc, ORDER_CHUNKED, 16, is_conv=c.kind == "conv", vec_ok=vec)


def cpu_baseline(calls, target_macs):
    """Time the oracle, as it stands, on a bounded sample: seeded 16x16 output tiles of several layers."""
    from oracle import lba_oracle as orc
    from paper_2401_14110_b200 import synth
    ORDER_CHUNKED = RUN_ORDER
    prod, acc = formats()
    picks = ([c for c in calls if c.kind == "conv"][1::4] + [calls[0]]) if GEMM_CASE is None else calls
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
            orc.conv2d_points(x, w, sx, sw, None, c.stride, c.pad, prod.as_tuple(), acc.as_tuple(), ORDER_CHUNKED, 16,
                              ms, ns, nthreads=cores)
        else:
            orc.gemm_points(x, w, sx, sw, None, prod.as_tuple(), acc.as_tuple(), ORDER_CHUNKED, 16, ms, ns,
                            nthreads=cores)
        macs += len(ms) * k
    dt = time.perf_counter() - t0
    return {"value": macs / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(jobs)} layers x seeded 16x16 output tiles, {macs:.3g} MACs in {dt:.1f} s",
            "macs": macs, "seconds": dt}


def reference_arm(args):
    """The oracle timed on the host cores; each step is a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import lba_oracle as orc
    from paper_2401_14110_b200 import synth, workloads, ORDER_CHUNKED
    prod, acc = formats()
    specs = workloads.resnet18_convs()
    picks = [specs[1], specs[6], specs[11], specs[16]]       # one 3x3 convolution from each stage
    cores = orc.default_threads()
    jobs = []
    for i, s in enumerate(picks):
        hw = s.h_in
        x, sx = synth.quantise_per_tensor(synth.gaussian((2, hw, hw, s.c_in), synth.seed_for(CONFIG_ID, 500 + i)).relu())
        w, sw = synth.quantise_per_channel(synth.he_normal((s.c_out, s.k, s.k, s.c_in), s.k * s.k * s.c_in,
                                                           synth.seed_for(CONFIG_ID, 600 + i)))
        m, n, k = 2 * s.h_out * s.h_out, s.c_out, s.k * s.k * s.c_in
        tiles = max(1, int(5e7 / (256 * k)))
        ms, ns = synth.sample_tiles(m, n, tiles, 16, 900 + i)
        jobs.append((s, x.numpy(), w.numpy(), sx.numpy(), sw.numpy(), ms, ns, k))
    step_macs = sum(len(j[5]) * j[7] for j in jobs)

    def step():
        for s, x, w, sx, sw, ms, ns, k in jobs:
            orc.conv2d_points(x, w, sx, sw, None, (s.stride, s.stride), (s.pad, s.pad), prod.as_tuple(),
                              acc.as_tuple(), ORDER_CHUNKED, 16, ms, ns, nthreads=cores)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = step_macs * args.steps / dt / 1e9
    sample = f"per step: seeded 16x16 output tiles of 4 ResNet-18 3x3 convolutions, {step_macs:.3g} MACs"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int128", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    global WORKLOAD, RUN_ORDER, GEMM_CASE, STE_KIND, FIXED_POINT
    args = parse_args()
    if args.workload.startswith("bgemm:"):
        parts = args.workload.split(":")
        GEMM_CASE = tuple(int(v) for v in parts[1].lower().split("x"))
        if len(GEMM_CASE) != 4:
            raise SystemExit("--workload bgemm:ZxMxNxK")
        RUN_ORDER = 0 if (len(parts) > 2 and parts[2].startswith("seq")) else 1
        WORKLOAD = "batched_lba_gemm_%dx%dx%dx%d_m7e4_%s" % (GEMM_CASE + ("sequential" if RUN_ORDER == 0 else "chunk16",))
        args.no_e2e = args.no_cpu_baseline = True      # kernel timing only for this workload
    elif args.workload.startswith("gemm:"):
        parts = args.workload.split(":")
        GEMM_CASE = tuple(int(v) for v in parts[1].lower().split("x"))
        RUN_ORDER = 0 if (len(parts) > 2 and parts[2].startswith("seq")) else 1
        WORKLOAD = "single_lba_gemm_%dx%dx%d_m7e4_%s" % (GEMM_CASE + ("sequential" if RUN_ORDER == 0 else "chunk16",))
    elif args.workload.startswith("fixed:"):
        # fixed:MxNxK[:seq|chunk][:wrap]: one GEMM with 12-bit fixed-point product and accumulator formats
        parts = args.workload.split(":")
        GEMM_CASE = tuple(int(v) for v in parts[1].lower().split("x"))
        FIXED_POINT = "wrap" if "wrap" in parts[2:] else "sat"
        RUN_ORDER = 0 if "seq" in parts[2:] else 1
        WORKLOAD = "fixed12_%s_gemm_%dx%dx%d_%s" % ((FIXED_POINT,) + GEMM_CASE + ("sequential" if RUN_ORDER == 0 else "chunk16",))
        args.no_e2e = args.no_cpu_baseline = True      # kernel timing only for this workload
    elif args.workload.startswith("ste:"):
        # ste:MxNxK[:of|diff][:seq|chunk]: the mask re-computation pass of the straight-through estimators
        parts = args.workload.split(":")
        GEMM_CASE = tuple(int(v) for v in parts[1].lower().split("x"))
        STE_KIND = "diff" if "diff" in parts[2:] else "of"
        RUN_ORDER = 0 if "seq" in parts[2:] else 1
        WORKLOAD = "ste_%s_mask_%dx%dx%d_m7e4_%s" % ((STE_KIND,) + GEMM_CASE + ("sequential" if RUN_ORDER == 0 else "chunk16",))
        args.no_e2e = args.no_cpu_baseline = True      # kernel timing only for this workload
    elif args.workload != "resnet18":
        raise SystemExit("unknown --workload")
    if args.impl == "reference":
        reference_arm(args)
        return
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

    from paper_2401_14110_b200 import binding as lba
    ORDER_CHUNKED = RUN_ORDER
    lba.load_library()
    prod, acc = formats()
    calls = build_calls(device)
    for c in calls:
        if c.kind == "conv":
            b, h, w, _ = c.x.shape
            ho, wo = lba.conv_out_hw(h, w, c.w.shape[1], c.w.shape[2], c.stride, c.pad)
            c.out_nhwc = c.out.view(b, ho, wo, c.w.shape[0])
    step_macs = sum(c.macs for c in calls)
    launches_per_step = len(calls)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        run_step(calls)
    barrier()

    # ---- timed region: K steps, per-launch CUDA events on the launching stream
    events = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in calls]
              for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    sampler.start()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    for s in range(args.steps):
        run_step(calls, events[s])
    stop.record()
    barrier()
    clocks = sampler.stop()
    from paper_2401_14110_b200 import sharding
    total_ms = sharding.max_over_ranks(start.elapsed_time(stop), dist, device)
    ms_per_step = total_ms / args.steps
    value = sharding.whole_job_rate(step_macs, world, ms_per_step * 1e-3) / 1e9

    # ---- per-kernel accounting from the per-launch events
    per_call_ms = [statistics.mean(events[s][i][0].elapsed_time(events[s][i][1]) for s in range(args.steps))
                   for i in range(len(calls))]
    by_kernel = {}
    for c, ms in zip(calls, per_call_ms):
        d = describe(c)
        key = " ".join(p for p in d.split() if not p.startswith("grid="))
        e = by_kernel.setdefault(key, {"ms": 0.0, "macs": 0, "launches": 0})
        e["ms"] += ms
        e["macs"] += c.macs
        e["launches"] += 1
    dom_key, dom = max(by_kernel.items(), key=lambda kv: kv[1]["ms"])
    sm_count = torch.cuda.get_device_properties(device).multi_processor_count
    max_mhz = clocks["sm_max_mhz"] or 1965.0
    mhz = clocks["sm_mhz"] or max_mhz
    slots = issue_slots_per_mac(RUN_ORDER == 1, 16)
    mix = "0.5 FMUL2 + 0.5 FFMA2 + 1 LOP3, plus 2.5 per output per chunk of 16"
    if STE_KIND == "of":
        # the packed kernel: slabs proved free of overflow cost what the forward pass costs, the mask words are constants
        mix += "; the overflow mask of a slab that provably cannot overflow needs no per-step work"
    elif FIXED_POINT is not None:
        # integer kernel, bound by the logic pipe (2 clocks per warp instruction): the floor (one shift), the
        # change of grid (one shift) and the add with its hold (two add-min/max) = 4 logic-pipe instructions per
        # step; the multiply and the shift count run beside them on the FP32/integer-multiply pipe.  These
        # formats hold every product, so Q_prod needs no saturation.
        slots = 8.0 + (4.0 / 16 if RUN_ORDER == 1 else 0.0)
        mix = "2 SHF + 2 VIADDMNMX on the logic pipe at 2 clocks each; IMAD + IADD beside them; plus the chunk folds"
    elif STE_KIND == "diff":
        # scalar tracking kernel: multiply, add (toward zero), mantissa mask, clamp, the rescaled sum, the subtraction,
        # |x w|, + eps1, * eps2, compare, bit insert
        slots = 11.0 + (slots - ISSUE_SLOTS_PER_MAC_LEVEL1)
        mix = "FMUL + FFMA + LOP3 + FMNMX + 3 FMUL + 2 FADD + FSETP + bit insert, scalar, plus the chunk folds"
    peak = sm_count * ISSUE_LANES_PER_SM_CLK * max_mhz * 1e6 / slots / 1e9
    achieved = dom["macs"] / (dom["ms"] * 1e-3) / 1e9
    roofline = {
        "bound": "alu", "achieved": achieved, "peak": peak, "unit": UNIT, "frac": achieved / peak,
        "traffic": NCU_DRAM_TRAFFIC.get((WORKLOAD, dom_key), (None, None))[0],
        "traffic_note": NCU_DRAM_TRAFFIC.get((WORKLOAD, dom_key), (None, "no ncu capture of this kernel on this workload"))[1],
        "kernel": dom_key, "kernel_launches_per_step": dom["launches"], "kernel_ms_per_step": dom["ms"],
        "kernel_share_of_step": dom["ms"] / sum(per_call_ms),
        "peak_derivation": f"{sm_count} SMs x {ISSUE_LANES_PER_SM_CLK} lanes issued per clock x {max_mhz:.0f} MHz "
                           f"(clocks.max.sm) / {slots:g} issue slots per emulated MAC ({mix})"
                           + ("; the FP32 and logic pipes give the same limit" if STE_KIND is None else ""),
        "frac_at_sampled_clock": achieved / (peak * mhz / max_mhz),
        "whole_step_frac_of_peak": (step_macs / (sum(per_call_ms) * 1e-3) / 1e9) / peak,
    }
    if STE_KIND is not None:   # one bit per step: the masks are the bulk of the algorithmic bytes
        mask_bytes = sum(c.mask1.numel() * 4 + (c.mask2.numel() * 4 if c.mask2 is not None else 0) for c in calls)
        roofline["mask_bytes_per_launch"] = mask_bytes
        roofline["mask_write_gbs"] = mask_bytes / (dom["ms"] * 1e-3) / 1e9

    # ---- the same device-resident step with its (independent) calls spread over several streams: kernels of
    # different calls share the SMs, which fills the tail waves a serial sequence leaves idle.  Reported beside
    # `value`, which stays the serial figure a layer-by-layer forward pass would see.
    concurrent = None
    if GEMM_CASE is None and args.e2e_streams > 1:
        cstreams = [torch.cuda.Stream(device=device) for _ in range(args.e2e_streams)]
        barrier()
        run_step(calls, streams=cstreams)
        barrier()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for st in cstreams:
            st.wait_event(c0)
        for _ in range(args.steps):
            run_step(calls, streams=cstreams)
        for st in cstreams:
            torch.cuda.current_stream().wait_stream(st)
        c1.record()
        barrier()
        cms = sharding.max_over_ranks(c0.elapsed_time(c1), dist, device) / args.steps
        concurrent = {"value": sharding.whole_job_rate(step_macs, world, cms * 1e-3) / 1e9, "unit": UNIT,
                      "ms_per_step": cms, "streams": args.e2e_streams}

    # ---- end to end through the host-buffer C entry points
    e2e = None
    if not args.no_e2e:
        host = []
        ws_bytes = 0
        h2d = d2h = 0
        for c in calls:
            hx, hw_, hsx, hsw = (t.cpu().pin_memory() for t in (c.x, c.w, c.sx, c.sw))
            hout = torch.empty(c.out.shape if c.kind == "gemm" else c.out_nhwc.shape, dtype=torch.float32).pin_memory()
            if c.kind == "conv":
                b, h, w, cin = c.x.shape
                cout, kh, kw, _ = c.w.shape
                need = lba.conv2d_host_workspace_bytes(b, h, w, cin, cout, kh, kw, c.stride, c.pad, 1, cout, False)
            else:
                m, n, k = c.gemm_shape
                need = lba.gemm_host_workspace_bytes(m, n, k, 1, n, False)
            ws_bytes = max(ws_bytes, need)
            h2d += hx.numel() + hw_.numel() + 4 * (hsx.numel() + hsw.numel())
            d2h += 4 * hout.numel()
            host.append((c, hx, hw_, hsx, hsw, hout))
        # the calls of a step are independent here (operands recorded beforehand), so they are spread round-robin
        # over a few streams, each with its own workspace: one call's copies overlap another call's kernel
        n_streams = max(1, args.e2e_streams)
        streams = [torch.cuda.Stream(device=device) for _ in range(n_streams)]
        wss = [torch.empty(ws_bytes, dtype=torch.uint8, device=device) for _ in range(n_streams)]
        torch.cuda.synchronize()

        def e2e_step():
            for i, (c, hx, hw_, hsx, hsw, hout) in enumerate(host):
                st, ws = streams[i % n_streams], wss[i % n_streams]
                if c.kind == "conv":
                    lba.lba_conv2d_host(hx, hw_, hsx, hsw, None, c.stride, c.pad, prod, acc, ORDER_CHUNKED, 16, hout, ws,
                                        stream=st)
                else:
                    lba.lba_gemm_host(hx, hw_, hsx, hsw, None, prod, acc, ORDER_CHUNKED, 16, hout, ws, stream=st)
        e2e_steps = max(2, min(args.steps, 10))
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            e2e_step()
        barrier()
        e2e_ms = (time.perf_counter() - t0) * 1e3 / e2e_steps
        e2e_ms = sharding.max_over_ranks(e2e_ms, dist, device)
        e2e = {"value": sharding.whole_job_rate(step_macs, world, e2e_ms * 1e-3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": e2e_steps,
               "api": "lba_conv2d_host / lba_gemm_host (pinned host buffers, caller-owned device workspaces, "
                      f"{n_streams} streams round-robin)"}
        del wss, host

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(calls, args.cpu_baseline_macs)

    if rank == 0:
        working_set = sum(c.x.numel() + c.w.numel() + 4 * c.out.numel() for c in calls)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32",
            "data": "synthetic",
            "config": {"workload": WORKLOAD, "batch_per_gpu": BATCH, "lba_calls_per_step": launches_per_step,
                       "macs_per_step_per_gpu": step_macs, "prod_fmt": list(prod.as_tuple()),
                       "acc_fmt": list(acc.as_tuple()), "order": "chunked" if RUN_ORDER == 1 else "sequential", "chunk": 16,
                       "l2": f"no flush: each step streams {working_set / 1e6:.0f} MB of distinct operands and "
                             f"outputs, larger than the 126 MB L2",
                       "parallelism": f"dp{world} (batch sharded, weights replicated, no collective)"},
            "clocks": clocks, "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "e2e": e2e, "cpu_baseline": cpu, "concurrent": concurrent,
            "kernels": {k: {"ms_per_step": v["ms"], "launches_per_step": v["launches"],
                            "gmacs": v["macs"] / (v["ms"] * 1e-3) / 1e9} for k, v in by_kernel.items()},
        }
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
