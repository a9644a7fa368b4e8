#!/usr/bin/env python
"""Benchmark of the GEMM hot path on B200.

One "step" is one pass over every problem of a workload (default: the square fp32 sweep
m=n=k in {1024, 2048, 4096, 8192}, alpha=1.5, beta=0.5), each problem one call of the C-ABI `gemm`.
Prints ONE JSON line: whole-job TFLOP/s with operands resident in HBM (`value`), the same metric
through `gemm_host` with pinned host buffers (`e2e`), the roofline of the dominant kernel, the CPU
oracle timed on the host cores on a bounded sample (`cpu_baseline`), and the SM clocks seen.

`--impl reference` times the CPU oracle (as it stands) on the host cores instead.
With N > 1 (torchrun) every rank runs an independent replica of the step on its own GPU: GEMM calls
do not communicate, so there is no collective on the data path ("replicas only").
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from workloads import (DTYPE_BF16, DTYPE_F16, DTYPE_F32, DTYPE_NAMES, config_problems, conv_layer_problems,  # noqa: E402
                       im2row_problems)

SM_COUNT = 148
FP32_LANES_PER_SM = 128
WORKLOADS = {
    "cfg2_fp32_squares": lambda: config_problems(2),
    "cfg1_fp32_512": lambda: config_problems(1),
    # config 2 through GEMM_F32_TC: fp32 data on the tensor cores as three bfloat16 pieces per entry (not IEEE fp32 arithmetic)
    "cfg2_fp32_tc": lambda: [__import__("dataclasses").replace(p, name=p.name + "_tc", tc3=True) for p in config_problems(2)],
    "cfg3_fp32_im2row": lambda: config_problems(3),
    "cfg4_fp32_nonsquarish": lambda: config_problems(4),
    "cfg5_f16": lambda: config_problems(5, dtype=DTYPE_F16),
    "cfg5_bf16": lambda: config_problems(5, dtype=DTYPE_BF16),
    "cfg5_f16_squares": lambda: config_problems(5, dtype=DTYPE_F16)[:3],
    "cfg5_bf16_squares": lambda: config_problems(5, dtype=DTYPE_BF16)[:3],
    # the same squares with A stored transposed (both operands contiguous along k), for information
    "cfg5_bf16_squares_tn": lambda: [__import__("dataclasses").replace(p, name=p.name + "_tn", transA="T")
                                     for p in config_problems(5, dtype=DTYPE_BF16)[:3]],
    # config 5 with the result in the operands' 16-bit type as well (the library's GEMM_BF16_C16)
    "cfg5_bf16_c16": lambda: config_problems(5, dtype=DTYPE_BF16, c16=True),
    # the paper's f16 arithmetic: binary16 operands, accumulator and result (GEMM_F16_ACC16)
    "cfg5_f16_acc16": lambda: [__import__("dataclasses").replace(p, name=p.name + "_acc16", acc16=True)
                               for p in config_problems(5, dtype=DTYPE_F16, c16=True)],
    # second workload (VGG16, batch 32) and the paper's own orientation (m = batch*pixels, n = channels)
    "vgg16_fp32": lambda: im2row_problems("vgg16"),
    "vgg16_bf16": lambda: im2row_problems("vgg16", dtype=DTYPE_BF16),
    "vgg16_fp32_paper_orientation": lambda: im2row_problems("vgg16", weights_as_A=False),
    "resnet50_fp32_paper_orientation": lambda: im2row_problems("resnet50", weights_as_A=False),
    "resnet50_bf16_paper_orientation": lambda: im2row_problems("resnet50", weights_as_A=False, dtype=DTYPE_BF16),
}
# the convolution layers themselves (NHWC activations in, NHWC result out): lowering fused into the GEMM kernels,
# timed beside the explicit route (im2row pass + gemm) and beside the GEMM alone on an already lowered matrix
CONV_WORKLOADS = {
    "resnet50_conv_fp32": lambda: conv_layer_problems("resnet50"),
    "resnet50_conv_bf16": lambda: conv_layer_problems("resnet50", dtype=DTYPE_BF16),
    "vgg16_conv_fp32": lambda: conv_layer_problems("vgg16"),
    "vgg16_conv_bf16": lambda: conv_layer_problems("vgg16", dtype=DTYPE_BF16),
    # the same layers with the result in bf16 as well: a layer's output is the next layer's input type
    "resnet50_conv_bf16_c16": lambda: conv_layer_problems("resnet50", dtype=DTYPE_BF16, c16=True),
    "vgg16_conv_bf16_c16": lambda: conv_layer_problems("vgg16", dtype=DTYPE_BF16, c16=True),
}


# DRAM traffic per launch (dram__bytes_read.sum + dram__bytes_write.sum from one ncu capture, see profiles/), keyed by
# kernel and problem, with the hash of the kernel's source file at capture time: a changed kernel reports null.
TRAFFIC = {
    ("simt_fast_kernel", "8192x8192x8192", "f32"): {
        "bytes": 3575662080 + 273164288, "source": "paper_2310_17408_b200/csrc/simt_fast.cu",
        "sha256": "9804c708bee85f95cd74403ad6bf228cfae6c0ec4a7f5c2cc2a687e997c259e9"},
    ("tc_gemm_pair_kernel", "8192x8192x8192", "bf16"): {
        "bytes": 1102845440 + 261591296, "source": "paper_2310_17408_b200/csrc/tc_gemm_pair.cu",
        "sha256": "685014adedc009c9b779c6688ae86bec26bc19f5f047537ceaf5adfa1302e6b9"},
    ("tc_gemm_pair_kernel", "16384x16384x16384", "bf16"): {
        "bytes": 17754797056 + 1102154240, "source": "paper_2310_17408_b200/csrc/tc_gemm_pair.cu",
        "sha256": "685014adedc009c9b779c6688ae86bec26bc19f5f047537ceaf5adfa1302e6b9"},
    ("tc_gemm_pair_kernel", "16384x16384x16384", "f16"): {
        "bytes": 22216240384 + 1103545344, "source": "paper_2310_17408_b200/csrc/tc_gemm_pair.cu",
        "sha256": "685014adedc009c9b779c6688ae86bec26bc19f5f047537ceaf5adfa1302e6b9"},
}


def recorded_traffic(kernel, p):
    import hashlib
    rec = TRAFFIC.get((kernel, f"{p.m}x{p.n}x{p.k}", DTYPE_NAMES[p.dtype]))
    if not rec:
        return None
    try:
        with open(os.path.join(ROOT, rec["source"]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != rec["sha256"]:
                return None
    except OSError:
        return None
    return rec["bytes"]


def load_peaks():
    """Roofline denominators: the measured copy bandwidth and library GEMM throughput of MEASURED_PEAKS.json when that file
    exists, otherwise the fallback figures stated below."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return dict(hbm_gbs=float(d["hbm_gbs"]), tensor_tflops=float(d["bf16_tflops"]),
                    tensor_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    sm_max_mhz=float(d.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, tensor_tflops=1590.0, tensor_tflops_sustained=1400.0, sm_max_mhz=1965.0,
                source="fallback")


def fp32_alu_peak_tflops(sm_mhz: float) -> float:
    # 148 SMs x 128 fp32 lanes x 2 flops per FMA x clock
    return SM_COUNT * FP32_LANES_PER_SM * 2 * sm_mhz * 1e6 / 1e12


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons (read-only queries).  It is started well before the timed
    region, because nvidia-smi takes a moment to produce its first line; only samples whose timestamp falls
    inside the timed window are used."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t_begin=None, t_end=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for seen, line in self.lines:
            # a sample is attributed to the moment its line arrived (nvidia-smi prints as it samples)
            if t_begin is not None and not (t_begin <= seen <= t_end + 0.05):
                continue
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx.append(float(parts[2])); power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples inside the timed region"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_median": statistics.median(power), "power_w_max": max(power)}


def rank_info():
    """(rank, world size, local rank) from the launcher's environment (torchrun); a plain run is rank 0 of 1."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (a job is as slow as its slowest replica).
    Needs an initialised process group when the world size is above 1; returns the list unchanged otherwise."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return list(values)
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def aggregate_throughput(flops_per_rank_step, step_ms_max, world):
    """Whole-job TFLOP/s of `world` independent replicas that each did flops_per_rank_step in step_ms_max."""
    return world * flops_per_rank_step / (step_ms_max * 1e-3) / 1e12


def roofline_class(p, peaks):
    """(bound, peak, unit, algorithmic amount) of one problem: the slower of compute and HBM time decides."""
    t_hbm = p.algorithmic_bytes() / (peaks["hbm_gbs"] * 1e9)
    if getattr(p, "tc3", False):
        # six bfloat16 products per fp32 product: the tensor peak counts a sixth in fp32-equivalent flops
        peak_c = peaks["tensor_tflops"] / 6.0
        if p.flops / (peak_c * 1e12) >= t_hbm:
            return "tensor", peak_c, "TFLOP/s", p.flops / 1e12
    elif p.dtype == DTYPE_F32:
        peak_c = fp32_alu_peak_tflops(peaks["sm_max_mhz"])
        t_cmp = p.flops / (peak_c * 1e12)
        if t_cmp >= t_hbm:
            return "alu", peak_c, "TFLOP/s", p.flops / 1e12
    else:
        peak_c = peaks["tensor_tflops"]
        t_cmp = p.flops / (peak_c * 1e12)
        if t_cmp >= t_hbm:
            return "tensor", peak_c, "TFLOP/s", p.flops / 1e12
    return "hbm", peaks["hbm_gbs"], "GB/s", p.algorithmic_bytes() / 1e9


# ------------------------------------------------------------------------------------------ reference arm (CPU oracle)

def reference_sample(problems):
    """Bounded sample of the workload for the CPU oracle: its members with at most ~2e10 flops each."""
    small = [p for p in problems if p.flops <= 2.0e10]
    return small or [min(problems, key=lambda p: p.flops)]


def oracle_call(oracle, p, ops):
    A, B, C0 = ops
    acc = oracle.ACC_F32 if p.dtype == DTYPE_F32 else oracle.ACC_F64
    return oracle.gemm_l1(p.dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, A.buf, A.ld, B.buf, B.ld, p.beta,
                          C0.buf, C0.ld, acc=acc)


def run_reference(args, problems, workload_name):
    rank, _, _ = rank_info()
    if rank != 0:          # under torchrun only rank 0 runs the CPU oracle; the others leave quietly
        return 0
    import oracle
    sample = reference_sample(problems)
    ops = [p.operands() for p in sample]
    flops = sum(p.flops for p in sample)
    for _ in range(args.warmup):
        for p, o in zip(sample, ops):
            oracle_call(oracle, p, o)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        for p, o in zip(sample, ops):
            oracle_call(oracle, p, o)
    dt = time.perf_counter() - t0
    val = flops * args.steps / dt / 1e12
    desc = "oracle L1 (blocked, packed, 8x12 micro-kernel, OpenMP) on " + ", ".join(p.name for p in sample)
    line = {"impl": "reference", "metric": "gemm_tflops", "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": DTYPE_NAMES[problems[0].dtype], "data": "synthetic",
            "config": {"workload": workload_name, "sample": [p.name for p in sample]},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def cpu_baseline(problems, operands, budget_s=30.0):
    """The oracle as it stands, on the host cores: one call each of the workload's members, smallest first,
    for as long as the next one is predicted (from the rate just measured) to fit the time budget."""
    import oracle
    order = sorted(range(len(problems)), key=lambda i: problems[i].flops)
    oracle_call(oracle, problems[order[0]], operands[order[0]])      # builds / loads the library, warms the threads
    chosen, flops, secs, rate = [], 0.0, 0.0, None
    for i in order:
        p = problems[i]
        if rate is not None and secs + p.flops / rate > budget_s:
            break
        t0 = time.perf_counter()
        oracle_call(oracle, p, operands[i])
        dt = time.perf_counter() - t0
        chosen.append(p)
        flops += p.flops
        secs += dt
        rate = p.flops / max(dt, 1e-9)
    blk = oracle.DEFAULT_BLOCKING
    return {"value": flops / secs / 1e12, "unit": "TFLOP/s", "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"one call each of {', '.join(p.name for p in chosen)} ({flops / 1e9:.1f} GFLOP, {secs:.1f} s); "
                      f"blocked packed GEMM, micro-kernel {blk['mr']}x{blk['nr']}, mc/kc/nc={blk['mc']}/{blk['kc']}/{blk['nc']}"}


# ------------------------------------------------------------------------------------------ CUDA arm

def run_probes(g, torch, stream, peaks):
    """The library's own peak-confirmation probes on this device: HBM copy, fp32 FMA loops (register-only chains and the SIMT micro-kernel fed from shared memory) and
    tcgen05.mma on shared-memory-resident operands.  Each is run a few times; best and median are reported."""
    out = {}

    def series(call, reps=5):
        vals = []
        for _ in range(reps):
            rc, rate, ms = call()
            if rc != 0:
                raise RuntimeError(f"probe failed: {g.gemm_status_string(rc)}")
            vals.append(rate)
        return {"best": max(vals), "median": statistics.median(vals)}

    nbytes = 1 << 30
    src = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    dst = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    src.zero_()
    out["hbm_copy_gbs"] = series(lambda: g.gemm_probe_copy(dst.data_ptr(), src.data_ptr(), nbytes, stream))
    del src, dst
    out["fp32_ffma_tflops"] = {
        "independent_chains": series(lambda: g.gemm_probe_ffma(0, 4096, stream)),
        "block_8x8": series(lambda: g.gemm_probe_ffma(1, 4096, stream)),
        "block_8x8_packed_f32x2": series(lambda: g.gemm_probe_ffma(2, 4096, stream)),
    }
    out["tensor_umma_tflops"] = {
        "bf16_128x256x16": series(lambda: g.gemm_probe_umma(DTYPE_BF16, 0, 60000, stream)),
        "bf16_pair_256x256x16": series(lambda: g.gemm_probe_umma(DTYPE_BF16, 1, 60000, stream)),
        "f16_pair_256x256x16": series(lambda: g.gemm_probe_umma(DTYPE_F16, 1, 60000, stream)),
    }
    if g.gemm_poll_status() != 0:
        raise RuntimeError(f"device status {hex(g.gemm_status_detail())} after the probes")
    out["note"] = ("measured by this library's probe kernels in this run (5 runs each); the roofline fractions divide by "
                   f"the {peaks['source']} peaks, 'frac_of_probe' by these")
    return out


def run_cuda(args, problems, workload_name):
    import torch
    import paper_2310_17408_b200 as g

    rank, world, local_rank = rank_info()
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    peaks = load_peaks()
    stream = torch.cuda.current_stream().cuda_stream

    # the CPU baseline runs first (rank 0, N = 1 only), before the GPU is busy
    base = None
    operands = [p.operands(need_c0=p.beta != 0.0) for p in problems]
    if world == 1 and not args.no_cpu_baseline:
        base = cpu_baseline(problems, operands, args.cpu_budget)
    probes = None
    if not args.no_probes:
        probes = run_probes(g, torch, stream, peaks)
        peaks["probes"] = probes
    ctx = dict(torch=torch, g=g, rank=rank, world=world, local_rank=local_rank, peaks=peaks, stream=stream, args=args)
    main = measure_workload(ctx, problems, operands, workload_name)
    del operands
    tensor = None
    if args.tensor_leg and workload_name == "cfg2_fp32_squares":
        # the tensor-core half of the metric in the same run: config 5's squares in both 16-bit input types
        tprobs = WORKLOADS["cfg5_bf16_squares"]() + WORKLOADS["cfg5_f16_squares"]()
        if args.only_tensor:
            names = set(args.only_tensor.split(","))
            tprobs = [p for p in tprobs if p.name in names]
        tops = [p.operands(need_c0=False) for p in tprobs]
        tensor = measure_workload(ctx, tprobs, tops, "cfg5_bf16_squares+cfg5_f16_squares", e2e_steps=2,
                                  steps=max(3, args.steps // 2))
        del tops
    if rank == 0:
        line = main
        if tensor is not None:
            tensor["dtype"] = "bf16+f16"
            line["tensor"] = tensor
            line["gpu_launches_tensor"] = tensor["gpu_launches"]
        if probes is not None:
            line["peaks_confirmed"] = probes
        if base:
            line["cpu_baseline"] = base
        print(json.dumps(line))
        if args.table:
            with open(args.table, "w") as f:
                json.dump(line, f, indent=1)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    return 0


def measure_workload(ctx, problems, operands, workload_name, e2e_steps=None, steps=None):
    """Times one workload (a list of problems with their host operands): `value` with operands resident, per-shape
    cold-cache numbers, the end-to-end leg through gemm_host, clocks, roofline.  Returns the report dict (on every
    rank; times are the maximum over ranks)."""
    torch, g, args = ctx["torch"], ctx["g"], ctx["args"]
    rank, world, local_rank, peaks, stream = ctx["rank"], ctx["world"], ctx["local_rank"], ctx["peaks"], ctx["stream"]
    n_steps = steps or args.steps
    if world > 1:
        import torch.distributed as dist

    # pinned host copies for the end-to-end leg, resident device copies for `value`
    host, dev = [], []
    ws_need = 0
    for p, (A, B, C0) in zip(problems, operands):
        view = (lambda x: x.view(np.int16)) if p.dtype != DTYPE_F32 else (lambda x: x)
        hA, hB, hC = (torch.from_numpy(view(A.buf)).pin_memory(), torch.from_numpy(view(B.buf)).pin_memory(),
                      torch.from_numpy(view(C0.buf) if C0.buf.dtype == np.uint16 else C0.buf).pin_memory())
        host.append((hA, hB, hC, A.ld, B.ld, C0.ld))
        dev.append((hA.cuda(), hB.cuda(), hC.cuda(), hC.cuda()))      # A, B, C0 (pristine), C (working)
        ws_need = max(ws_need, g.gemm_workspace_bytes(p.api_dtype, p.transA, p.transB, p.m, p.n, p.k))
    ws = torch.empty(max(ws_need, 1 << 20), dtype=torch.uint8, device="cuda")
    assert g.gemm_set_workspace(ws.data_ptr(), ws.numel(), 0) == 0

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    launches = 0

    def one_step(events=None):
        nonlocal launches
        for i, p in enumerate(problems):
            dA, dB, dC0, dC = dev[i]
            _, _, _, lda, ldb, ldc = host[i]
            if events is not None:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
            rc = g.gemm(p.api_dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, dA.data_ptr(), lda, dB.data_ptr(), ldb,
                        p.beta, dC.data_ptr(), ldc, stream)
            if rc != 0:
                raise RuntimeError(f"gemm failed: {g.gemm_status_string(rc)} (cuda error {g.gemm_last_cuda_error()})")
            if events is not None:
                e1.record()
                events[i].append((e0, e1))
            launches += g.gemm_last_config()["launches"]

    # ---- device-resident timing
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(max(args.warmup, 3)):
        one_step()
    barrier()
    events = [[] for _ in problems]
    launches = 0
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    wall_begin = time.time()
    t_begin.record()
    for _ in range(n_steps):
        one_step(events)
    t_end.record()
    barrier()
    wall_end = time.time()
    total_ms = t_begin.elapsed_time(t_end)
    if wall_end - wall_begin >= 0.4:
        clocks = sampler.stop(wall_begin, wall_end)
    else:
        # a timed region this short sees no nvidia-smi sample: keep running the same steps for 0.6 s and sample there
        w0 = time.time()
        while time.time() - w0 < 0.6:
            one_step()
        torch.cuda.synchronize()
        clocks = sampler.stop(w0, time.time())
        clocks["window"] = "0.6 s of the same steps run right after the (shorter) timed region"
    timed_launches = launches
    if g.gemm_poll_status() != 0:
        raise RuntimeError(f"device status {hex(g.gemm_status_detail())}")
    configs = []
    for p in problems:   # what the selector chose (one untimed call each)
        i = problems.index(p)
        dA, dB, dC0, dC = dev[i]
        g.gemm(p.api_dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, dA.data_ptr(), host[i][3], dB.data_ptr(), host[i][4],
               p.beta, dC.data_ptr(), host[i][5], stream)
        configs.append(g.gemm_last_config())
    torch.cuda.synchronize()

    # ---- per-shape numbers: back-to-back calls (launch latency hidden behind the previous call), cycling through
    # enough distinct copies of A, B, C that every call finds its operands in HBM, not in L2
    def measure_shape(i, p, step_ms_est):
        dA, dB, dC0, dC = dev[i]
        _, _, _, lda, ldb, ldc = host[i]
        nsets = int(min(32, max(1, -(-2 * 126e6 // p.algorithmic_bytes()))))
        sets = [(dA, dB, dC)] + [(dA.clone(), dB.clone(), dC.clone()) for _ in range(nsets - 1)]
        reps = int(min(400, max(20, 0.05 / max(step_ms_est * 1e-3, 1e-6))))

        def call(r):
            a, b, c = sets[r % nsets]
            rc = g.gemm(p.api_dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, a.data_ptr(), lda, b.data_ptr(), ldb,
                        p.beta, c.data_ptr(), ldc, stream)
            if rc != 0:
                raise RuntimeError(g.gemm_status_string(rc))
        for r in range(3):
            call(r)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record()
        for r in range(reps):
            call(r)
        e1.record()
        host_us = (time.perf_counter() - t0) / reps * 1e6
        torch.cuda.synchronize()
        stream_ms = e0.elapsed_time(e1) / reps
        # the same calls captured once into a CUDA graph and replayed: no per-call host work between the kernels
        graph_ms = None
        if stream_ms < 1.0:
            try:
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(side):
                    cap = torch.cuda.current_stream().cuda_stream
                    with torch.cuda.graph(graph, stream=side):
                        for r in range(reps):
                            a, b, c = sets[r % nsets]
                            rc = g.gemm(p.api_dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, a.data_ptr(), lda,
                                        b.data_ptr(), ldb, p.beta, c.data_ptr(), ldc, cap)
                            if rc != 0:
                                raise RuntimeError(g.gemm_status_string(rc))
                    graph.replay()
                    side.synchronize()
                    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    g0.record(side)
                    graph.replay()
                    g1.record(side)
                    side.synchronize()
                    graph_ms = g0.elapsed_time(g1) / reps
                torch.cuda.current_stream().wait_stream(side)
            except Exception as exc:          # graph capture is a measurement convenience, not part of the contract
                sys.stderr.write(f"graph timing skipped for {p.name}: {exc}\n")
                graph_ms = None
        # twenty calls timed one by one (an event pair around each; the pair itself costs a few microseconds, which shows
        # on the shortest calls): median and best
        singles = []
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for r, (a0, a1) in enumerate(pairs):
            a0.record()
            call(r)
            a1.record()
        torch.cuda.synchronize()
        singles = sorted(a0.elapsed_time(a1) for a0, a1 in pairs)
        one_by_one = {"median": statistics.median(singles), "best": singles[0]}
        return stream_ms, host_us, nsets, reps, graph_ms, one_by_one

    b2b = []
    for i, p in enumerate(problems):
        est = sum(a.elapsed_time(b) for a, b in events[i]) / len(events[i])
        b2b.append(measure_shape(i, p, est))

    # ---- end to end: pinned host buffers through gemm_host, copies inside the timed region
    e2e = None
    if not args.no_e2e:
        def host_step():
            for i, p in enumerate(problems):
                hA, hB, hC, lda, ldb, ldc = host[i]
                rc = g.gemm_host(p.api_dtype, p.transA, p.transB, p.m, p.n, p.k, p.alpha, hA.data_ptr(), lda, hB.data_ptr(),
                                 ldb, p.beta, hC.data_ptr(), ldc, stream)
                if rc != 0:
                    raise RuntimeError(f"gemm_host failed: {g.gemm_status_string(rc)}")
        host_c0 = [h[2].clone() for h in host]
        for _ in range(2):
            host_step()
        for h, c0 in zip(host, host_c0):
            h[2].copy_(c0)
        barrier()
        t0 = time.perf_counter()
        e2e_steps = max(1, min(n_steps, e2e_steps or args.e2e_steps))
        for _ in range(e2e_steps):
            host_step()
        barrier()
        e2e_s = time.perf_counter() - t0
        h2d = sum(h[0].numel() * h[0].element_size() + h[1].numel() * h[1].element_size() +
                  (h[2].numel() * h[2].element_size() if p.beta != 0.0 else 0) for h, p in zip(host, problems))   # C goes in only when beta != 0
        d2h = sum(h[2].numel() * h[2].element_size() for h in host)
        e2e = (e2e_s / e2e_steps, h2d, d2h, e2e_steps)

    # ---- reduce over ranks (max time), report on rank 0
    step_ms = total_ms / n_steps
    e2e_ms = e2e[0] * 1e3 if e2e else 0.0
    step_ms, e2e_ms = max_over_ranks([step_ms, e2e_ms], device="cuda")
    flops_step = sum(p.flops for p in problems)
    value = aggregate_throughput(flops_step, step_ms, world)

    shapes, dominant, dom_ms = [], None, -1.0
    for i, p in enumerate(problems):
        ms = [a.elapsed_time(b) for a, b in events[i]]
        avg = sum(ms) / len(ms)
        bound, peak, unit, amount = roofline_class(p, peaks)
        achieved = amount / (avg * 1e-3)
        cold_ms, host_us, nsets, reps, graph_ms, one_by_one = b2b[i]
        shapes.append({"name": p.name, "m": p.m, "n": p.n, "k": p.k, "ms_in_step": avg, "ms": cold_ms,
                       "tflops": p.flops / (cold_ms * 1e-3) / 1e12, "gbs": p.algorithmic_bytes() / (cold_ms * 1e-3) / 1e9,
                       "bound": bound, "frac": amount / (cold_ms * 1e-3) / peak, "frac_in_step": achieved / peak,
                       "ms_single_median": one_by_one["median"], "ms_single_best": one_by_one["best"],
                       "ms_graph": graph_ms, "frac_graph": (amount / (graph_ms * 1e-3) / peak) if graph_ms else None,
                       "host_us_per_call": host_us, "operand_sets": nsets, "calls": reps, "kernel": configs[i]["kernel"],
                       "tile": [configs[i]["tile_m"], configs[i]["tile_n"]], "split_k": configs[i]["split_k"], "tail_split": configs[i].get("tail_split", 0),
                       "launches": configs[i]["launches"]})
        if avg > dom_ms:
            dom_ms, dominant = avg, (p, bound, peak, unit, achieved, configs[i])
    p, bound, peak, unit, achieved, cfg = dominant
    kernel_names = {1: "simt_generic_kernel", 2: "simt_fast_kernel", 3: "tc_gemm_kernel", 6: "scale_kernel"}
    kname = kernel_names.get(cfg["kernel"], "?")
    if cfg["kernel"] == 3 and cfg["tile_m"] == 256:
        kname = "tc_gemm_pair_kernel"          # 256 x 256 tiles on CTA pairs
    roof = {"bound": bound, "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
            "traffic": recorded_traffic(kname, p),
            "kernel": kname, "problem": p.name,
            "peak_source": (f"{SM_COUNT} SMs x {FP32_LANES_PER_SM} lanes x 2 x {peaks['sm_max_mhz']:.0f} MHz (max SM clock)"
                            if bound == "alu" else f"{peaks['source']} ({'MEASURED_PEAKS.json' if peaks['source'] == 'measured' else 'fallback figures'})")}
    if bound == "alu" and clocks.get("sm_mhz"):
        roof["frac_at_sampled_clock"] = achieved / fp32_alu_peak_tflops(clocks["sm_mhz"])
    if bound == "tensor":
        # a kernel timed inside a step that runs for a long time sits at the power-capped clock: the sustained figure
        roof["peak_sustained"] = peaks["tensor_tflops_sustained"]
        roof["frac_of_sustained"] = achieved / peaks["tensor_tflops_sustained"]
        roof["frac_of_nominal_2250"] = achieved / 2250.0
    probes = peaks.get("probes")
    if probes:      # the same achieved rate against what this library's own probe kernels reached in this run
        own = {"alu": probes["fp32_ffma_tflops"]["independent_chains"]["best"],
               "tensor": probes["tensor_umma_tflops"]["bf16_pair_256x256x16"]["best"],
               "hbm": probes["hbm_copy_gbs"]["best"]}[bound]
        roof["peak_probe"] = own
        roof["frac_of_probe"] = achieved / own if own else None
    line = {"metric": "gemm_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": n_steps,
            "warmup": max(args.warmup, 3), "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": DTYPE_NAMES[problems[0].dtype], "data": "synthetic",
            "config": {"workload": workload_name, "problems": [f"{q.m}x{q.n}x{q.k}" for q in problems],
                       "alpha": problems[0].alpha, "beta": problems[0].beta, "layout": f"column-major {problems[0].transA},{problems[0].transB}",
                       "l2": "inputs larger than L2: one step touches more than 126 MB of operands"
                             if sum(q.algorithmic_bytes() for q in problems) > 126e6 else
                             "working set smaller than L2 (warm-cache number)",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "roofline": roof, "clocks": clocks, "gpu_launches": timed_launches, "shapes": shapes}
    if e2e:
        line["e2e"] = {"value": aggregate_throughput(flops_step, e2e_ms, world), "unit": "TFLOP/s",
                       "h2d_bytes_per_step": e2e[1], "d2h_bytes_per_step": e2e[2], "steps": e2e[3],
                       # average rates over the whole step (the wire is idle while the last panels are multiplied)
                       "h2d_gbs": e2e[1] / (e2e_ms * 1e-3) / 1e9, "d2h_gbs": e2e[2] / (e2e_ms * 1e-3) / 1e9,
                       "ms_per_step": e2e_ms,
                       "api": "gemm_host (pinned host buffers, copies inside the timed region)"}
    g.gemm_set_workspace(0, 0, 0)
    del dev, host, ws
    torch.cuda.empty_cache()
    return line


# ------------------------------------------------------------------------------------------ convolution layers

def run_conv_layers(args, layers, workload_name):
    """One step = every layer of the network once through conv2d_im2row (the selector's route).  Per layer it also
    times the explicit route (im2row pass + gemm) and gemm alone on a lowered matrix that is already in memory
    (what the paper's experiment measures), all cold-cache: calls cycle through enough operand sets to exceed L2."""
    import torch
    import paper_2310_17408_b200 as g

    torch.cuda.set_device(0)
    peaks = load_peaks()
    stream = torch.cuda.current_stream().cuda_stream
    shapes = [g.conv_shape(p.batch, p.h, p.w, p.c_in, p.c_out, p.kh, p.kw, p.stride, p.stride, p.pad, p.pad) for p in layers]
    g.conv2d_force_lowering(g.CONV_LOWERING_EXPLICIT)
    ws_need = max(g.conv2d_workspace_bytes(p.api_dtype, s) for p, s in zip(layers, shapes))
    g.conv2d_force_lowering(0)
    ws = torch.empty(ws_need + (64 << 20), dtype=torch.uint8, device="cuda")
    assert g.gemm_set_workspace(ws.data_ptr(), ws.numel(), 0) == 0
    rows, step_ms, step_flops, launches = [], 0.0, 0.0, 0
    sampler = ClockSampler(0)
    sampler.start()
    wall_begin = time.time()
    for p, shp in zip(layers, shapes):
        X, W, Y0 = p.operands()
        view = (lambda x: x.view(np.int16)) if p.dtype != DTYPE_F32 else (lambda x: x)
        m, n, k = p.gemm_mnk
        es = 4 if p.dtype == DTYPE_F32 else 2
        nsets = int(min(16, max(1, -(-2 * 126e6 // p.algorithmic_bytes()))))
        dX = [torch.from_numpy(view(X.buf)).cuda() for _ in range(nsets)]
        dW = [torch.from_numpy(view(W.buf)).cuda() for _ in range(nsets)]
        dY = [torch.from_numpy(view(Y0.buf) if Y0.buf.dtype == np.uint16 else Y0.buf).cuda() for _ in range(nsets)]

        def timed(call, reps):
            for r in range(3):
                call(r)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for r in range(reps):
                call(r)
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1) / reps

        def conv_call(r):
            i = r % nsets
            rc = g.conv2d_im2row(p.api_dtype, shp, p.alpha, dX[i].data_ptr(), dW[i].data_ptr(), W.ld, p.beta, dY[i].data_ptr(), Y0.ld, stream)
            if rc != 0:
                raise RuntimeError(f"conv2d_im2row failed on {p.name}: {g.gemm_status_string(rc)}")

        reps = max(args.steps, 10)
        ms_auto = timed(conv_call, reps)
        cfg = g.gemm_last_config()
        launches += reps * (cfg["launches"] + (1 if cfg["lowering"] == g.CONV_LOWERING_EXPLICIT else 0))
        g.conv2d_force_lowering(g.CONV_LOWERING_EXPLICIT)
        ms_explicit = timed(conv_call, reps)
        g.conv2d_force_lowering(0)
        # gemm alone on a lowered matrix that already exists (one copy: k x pixels can be hundreds of MB)
        ld = -(-k // 8) * 8
        low = torch.empty(ld * n, dtype=dX[0].dtype, device="cuda")
        assert g.im2row(p.dtype, shp, dX[0].data_ptr(), low.data_ptr(), ld, stream) == 0

        def gemm_call(r):
            i = r % nsets
            rc = g.gemm(p.api_dtype, "N", "N", m, n, k, p.alpha, dW[i].data_ptr(), W.ld, low.data_ptr(), ld, p.beta, dY[i].data_ptr(), Y0.ld, stream)
            if rc != 0:
                raise RuntimeError(g.gemm_status_string(rc))
        ms_gemm = timed(gemm_call, reps)
        del low
        bound, peak, unit, amount = roofline_class(p, peaks)
        rows.append({"name": p.name, "layer": f"{p.c_in}->{p.c_out} {p.kh}x{p.kw}/{p.stride} on {p.h}x{p.w}", "m": m, "n": n, "k": k,
                     "lowering": {1: "fused", 2: "explicit", 3: "identity"}.get(cfg["lowering"], "?"),
                     "kernel": cfg["kernel"], "tile": [cfg["tile_m"], cfg["tile_n"]], "split_k": cfg["split_k"],
                     "ms": ms_auto, "ms_explicit_route": ms_explicit, "ms_gemm_on_lowered": ms_gemm,
                     "tflops": p.flops / (ms_auto * 1e-3) / 1e12, "gbs": p.algorithmic_bytes() / (ms_auto * 1e-3) / 1e9,
                     "lowered_matrix_mb": ld * n * es / 1e6, "bound": bound, "frac": amount / (ms_auto * 1e-3) / peak})
        step_ms += ms_auto
        step_flops += p.flops
        del dX, dW, dY
        torch.cuda.empty_cache()
    clocks = sampler.stop(wall_begin, time.time())
    if g.gemm_poll_status() != 0:
        raise RuntimeError(f"device status {hex(g.gemm_status_detail())}")
    dom = max(rows, key=lambda r: r["ms"])
    line = {"metric": "gemm_tflops", "value": step_flops / (step_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "n_gpus": 1,
            "steps": max(args.steps, 10), "warmup": 3, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": DTYPE_NAMES[layers[0].dtype], "data": "synthetic",
            "config": {"workload": workload_name, "batch": layers[0].batch, "layout": "NHWC activations, C_out x k filters",
                       "l2": "calls cycle through operand sets larger than L2", "parallelism": "single GPU",
                       "step": "sum over the layers of the per-layer cold-cache time"},
            "roofline": {"bound": dom["bound"], "achieved": dom["tflops"] if dom["bound"] != "hbm" else dom["gbs"],
                         "peak": roofline_class(layers[rows.index(dom)], peaks)[1],
                         "unit": "GB/s" if dom["bound"] == "hbm" else "TFLOP/s", "frac": dom["frac"], "traffic": None,
                         "kernel": "conv2d_im2row (" + dom["lowering"] + ")", "problem": dom["name"]},
            "clocks": clocks, "gpu_launches": launches, "shapes": rows}
    print(json.dumps(line))
    if args.table:
        with open(args.table, "w") as f:
            json.dump(line, f, indent=1)
    return 0


# ------------------------------------------------------------------------------------------ strided batches of small problems

BATCHED_WORKLOADS = {
    # (m, n, k, batch): many small fp32 problems in one call of gemm_strided_batched
    "batched_fp32_small": [(64, 64, 64, 4096), (32, 32, 32, 16384), (16, 16, 16, 65535), (128, 128, 128, 1024),
                           (96, 96, 200, 2048), (256, 256, 256, 128)],
    # the same through the tensor cores: bf16 operands, fp32 results, one launch per call (problem index = third
    # coordinate of the operand maps)
    "batched_bf16_small": [(64, 64, 64, 4096), (128, 128, 128, 1024), (96, 96, 200, 2048), (256, 256, 256, 128),
                           (512, 512, 512, 32), (128, 128, 64, 8192)],
}


def run_batched(args, cases, workload_name):
    """One step = every case once through gemm_strided_batched.  Operands are seeded uniform[-1, 1) values generated on
    the host for one problem and tiled over the batch with a per-problem sign flip (cheap and still distinct); calls
    cycle through enough operand sets to exceed L2.  Roofline per case: the slower of 2*m*n*k*batch flops at the fp32
    ALU peak and 4*(m*k + k*n + m*n)*batch bytes at the HBM peak."""
    import torch
    import paper_2310_17408_b200 as g
    from workloads import make_matrix

    torch.cuda.set_device(0)
    peaks = load_peaks()
    stream = torch.cuda.current_stream().cuda_stream
    half = "bf16" in workload_name
    api_dtype, es, tdt = (DTYPE_BF16, 2, torch.bfloat16) if half else (DTYPE_F32, 4, torch.float32)
    rows, step_ms, step_flops, launches = [], 0.0, 0.0, 0
    sampler = ClockSampler(0)
    sampler.start()
    wall_begin = time.time()
    for idx, (m, n, k, batch) in enumerate(cases):
        A1 = torch.from_numpy(make_matrix(m, k, kind="uniform", seed=7000 + idx, matrix_id=0).buf).cuda()
        B1 = torch.from_numpy(make_matrix(k, n, kind="uniform", seed=7000 + idx, matrix_id=1).buf).cuda()
        sign = (1.0 - 2.0 * (torch.arange(batch, device="cuda") % 2)).float()[:, None]
        bytes_call = (es * (m * k + k * n) + 4.0 * m * n) * batch
        flops = 2.0 * m * n * k * batch
        nsets = int(min(16, max(1, -(-2 * 126e6 // bytes_call))))
        sets = [((A1[None, :] * sign).to(tdt).contiguous(), (B1[None, :] * sign).to(tdt).contiguous(), torch.empty(batch * m * n, device="cuda"))
                for _ in range(nsets)]

        def call(r):
            a, b, c = sets[r % nsets]
            rc = g.gemm_strided_batched(api_dtype, "N", "N", m, n, k, 1.0, a.data_ptr(), m, m * k, b.data_ptr(), k, k * n, 0.0,
                                        c.data_ptr(), m, m * n, batch, stream)
            if rc != 0:
                raise RuntimeError(f"gemm_strided_batched failed: {rc}")
        reps = max(args.steps, 10)
        for r in range(3):
            call(r)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for r in range(reps):
            call(r)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        cfg = g.gemm_last_config()
        launches += reps * cfg["launches"]
        cmp_peak = peaks["tensor_tflops"] if half else fp32_alu_peak_tflops(peaks["sm_max_mhz"])
        t_cmp = flops / (cmp_peak * 1e12)
        t_hbm = bytes_call / (peaks["hbm_gbs"] * 1e9)
        bound = ("tensor" if half else "alu") if t_cmp >= t_hbm else "hbm"
        rows.append({"name": f"{m}x{n}x{k}x{batch}", "m": m, "n": n, "k": k, "batch": batch, "ms": ms,
                     "tflops": flops / (ms * 1e-3) / 1e12, "gbs": bytes_call / (ms * 1e-3) / 1e9, "bound": bound,
                     "frac": max(t_cmp, t_hbm) / (ms * 1e-3), "kernel": cfg["kernel"], "tile": [cfg["tile_m"], cfg["tile_n"]],
                     "launches": cfg["launches"], "operand_sets": nsets})
        step_ms += ms
        step_flops += flops
        del sets
        torch.cuda.empty_cache()
    clocks = sampler.stop(wall_begin, time.time())
    if g.gemm_poll_status() != 0:
        raise RuntimeError(f"device status {hex(g.gemm_status_detail())}")
    dom = max(rows, key=lambda r: r["ms"])
    line = {"metric": "gemm_tflops", "value": step_flops / (step_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "n_gpus": 1,
            "steps": max(args.steps, 10), "warmup": 3, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16" if half else "f32", "data": "synthetic",
            "config": {"workload": workload_name, "api": "gemm_strided_batched", "layout": "column-major N,N, dense strides",
                       "l2": "calls cycle through operand sets larger than L2", "parallelism": "single GPU"},
            "roofline": {"bound": dom["bound"], "achieved": dom["gbs"] if dom["bound"] == "hbm" else dom["tflops"],
                         "peak": peaks["hbm_gbs"] if dom["bound"] == "hbm" else
                                 (peaks["tensor_tflops"] if half else fp32_alu_peak_tflops(peaks["sm_max_mhz"])),
                         "unit": "GB/s" if dom["bound"] == "hbm" else "TFLOP/s", "frac": dom["frac"], "traffic": None,
                         "kernel": {2: "simt_batched_kernel", 4: "simt_direct_kernel", 1: "simt_generic_kernel",
                                    3: "tc_gemm_kernel"}.get(dom["kernel"], "?"),
                         "problem": dom["name"]},
            "clocks": clocks, "gpu_launches": launches, "shapes": rows}
    print(json.dumps(line))
    if args.table:
        with open(args.table, "w") as f:
            json.dump(line, f, indent=1)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="cfg2_fp32_squares", choices=sorted(WORKLOADS) + sorted(CONV_WORKLOADS) + sorted(BATCHED_WORKLOADS))
    ap.add_argument("--shape", default=None, help="M,N,K: time this single problem instead of a workload (alpha=1, beta=0)")
    ap.add_argument("--dtype", default="f32", choices=["f32", "f32tc", "f16", "bf16"],
                    help="operand type for --shape (f32tc: fp32 data through GEMM_F32_TC)")
    ap.add_argument("--kind", default=None, choices=["uniform", "normal", "int"],
                    help="value distribution for --shape (default: uniform for f32, normal for 16-bit inputs; int = integers in [-4, 4])")
    ap.add_argument("--alpha", type=float, default=1.0, help="alpha for --shape")
    ap.add_argument("--beta", type=float, default=0.0, help="beta for --shape")
    ap.add_argument("--only", default=None, help="comma-separated problem names: keep only these members of the workload")
    ap.add_argument("--table", default=None, help="also write the JSON (indented, with per-shape rows) to this file")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-probes", action="store_true", help="skip the peak-confirmation probes")
    ap.add_argument("--no-tensor-leg", dest="tensor_leg", action="store_false",
                    help="default workload only: skip config 5's 16-bit squares (the `tensor` key)")
    ap.add_argument("--only-tensor", default=None, help="comma-separated problem names: members of the tensor leg to keep")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-budget", type=float, default=30.0)
    args = ap.parse_args()
    def keep(items):
        if not args.only:
            return items
        names = set(args.only.split(","))
        kept = [p for p in items if p.name in names]
        if not kept:
            raise SystemExit(f"--only {args.only}: no such problem in {args.workload} ({', '.join(p.name for p in items)})")
        return kept
    if args.workload in BATCHED_WORKLOADS:
        return run_batched(args, BATCHED_WORKLOADS[args.workload], args.workload)
    if args.workload in CONV_WORKLOADS:
        return run_conv_layers(args, keep(CONV_WORKLOADS[args.workload]()), args.workload)
    problems = keep(WORKLOADS[args.workload]())
    if args.shape:
        from workloads import Problem
        m, n, k = (int(t) for t in args.shape.split(","))
        dt = {"f32": DTYPE_F32, "f32tc": DTYPE_F32, "f16": DTYPE_F16, "bf16": DTYPE_BF16}[args.dtype]
        kind = args.kind or ("uniform" if dt == DTYPE_F32 else "normal")
        problems = [Problem(f"{args.dtype}_{m}x{n}x{k}", dt, m, n, k, args.alpha, args.beta, kindA=kind, kindB=kind, seed=0,
                            tc3=args.dtype == "f32tc")]
        args.workload = f"single:{args.dtype}:{m}x{n}x{k}"
    if args.impl == "reference":
        return run_reference(args, problems, args.workload)
    return run_cuda(args, problems, args.workload)


if __name__ == "__main__":
    sys.exit(main())
