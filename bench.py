#!/usr/bin/env python
"""Benchmark of the GWQ mixed-precision linear layer on B200.

One "step" is one pass of gwq_linear over the Llama-7B-shaped decode layer set
(7 projections, each packed to 4 and to 3 bits, group 128, 1 % outliers) at
M = 1, 4 and 16 tokens: 42 products in 24 calls (sibling projections share a call),
replayed as one CUDA graph.  The headline
value is the HBM rate over the algorithmic bytes of that step.  Beside it the
line reports per-layer decode times, the tensor-core prefill cases, the encode
kernels, a dense fp16 GEMM (torch.matmul, a library call) on the unquantized
weights, the end-to-end rate through the host-buffer entry point, and the CPU
checker timed on the host cores.

  python bench.py --gpus 1 --steps 20 --warmup 3
  python bench.py --impl reference ...      (times the CPU checker instead)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2411_00850_b200 import synth

METRIC = "GWQ W4/W3 linear: decode µs & HBM GB/s (% roofline); prefill TFLOP/s"
WORKLOAD = "llama7b_decode_layer_set_w4_w3_g128_1pct_M1_4_16"
DECODE_MS = (1, 4, 16)
BIT_WIDTHS = (4, 3)
GROUP = 128
FRAC = 0.01
CONFIG_INDEX = 1
# layers of the set (by index) in decoder-block data-flow order: q|k|v read the same x, then o, gate|up, down
STAGES = ((0, 1, 2), (3,), (4, 5), (6,))
PREFILL_SHAPES = ((11008, 4096), (4096, 11008))
PREFILL_MS = (512, 2048, 8192)


def measured_peaks():
    """(hbm GB/s, bf16 TFLOP/s burst, sustained, source) from the pool's measured file, else the fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        d = json.load(open(path))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), float(d["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 6650.0, 1590.0, 1400.0, "fallback"


def algorithmic_bytes(N: int, K: int, bits: int, group: int, nnz: int, M: int, col_bytes: int = 2) -> int:
    """Bytes one decode launch has to move: codes, scales, zero-points, the CSR (row
    pointers, columns as the kernel reads them, fp16 values), x and y."""
    codes = N * K * bits // 8
    meta = N * (K // group) * 3
    csr = (N + 1) * 4 + nnz * (col_bytes + 2)
    return codes + meta + csr + M * K * 2 + M * N * 2


def kernels_per_linear(M: int, K: int) -> int:
    """Kernels one gwq_linear call launches on the decode path: the product itself, plus the
    token-major copy of x when M > 1 and the activations are not staged up front (M > 8, or
    M K too large for 72 KB of staging)."""
    nchunks = (K // 128 + 7) // 8
    staged = M <= 8 and nchunks * M * 148 * 16 <= 72 * 1024   # (80 KB for small grids: no case of this step)
    return 1 if (staged or M == 1) else 2


def dominant_kernel_traffic():
    """(dram bytes / algorithmic bytes) of the decode kernel from the committed ncu capture, or None when
    the kernel source has changed since the capture was taken."""
    import hashlib
    try:
        rec = json.load(open(os.path.join(ROOT, "profiles", "decode_kernel_traffic.json")))
        src = open(os.path.join(ROOT, "paper_2411_00850_b200", "csrc", "decode_kernel.cuh"), "rb").read()
        if hashlib.sha1(src).hexdigest() != rec["kernel_source_sha1"]:
            return None
        return float(rec["dram_bytes_per_launch"]) / float(rec["algorithmic_bytes_per_launch"])
    except Exception:
        return None


def linear_flops(N: int, K: int, nnz: int, M: int) -> int:
    return 2 * M * (N * K + nnz)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while a region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(smax)), "power_w_max": float(max(power)),
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(ms_local: float, device=None) -> float:
    """Slowest rank's time: the whole job is as slow as its slowest replica.  Works on any backend
    (NCCL on the GPUs, gloo in the CPU test); a single process returns its own time."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local)
    t = torch.tensor([float(ms_local)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_gbs(step_bytes: int, ms_step_max: float, world: int) -> float:
    """Replicas only: every rank runs the same step on its own copy of the layer set, nothing is
    exchanged; the job moved world * step_bytes in the time of the slowest rank."""
    return world * step_bytes / (ms_step_max * 1e-3) / 1e9


# ----------------------------------------------------------------------------- the CUDA arm
def build_layer_set(torch, gwq, dev, replicas: int, keep_dense: bool):
    """Generate the 7 seeded layers, encode each to 4 and 3 bits on the GPU.
    Returns (layers, encode_stats); layers[i] = dict(name, N, K, packed={bits: [Packed]*replicas}, W=dense)."""
    layers, enc = [], {"select_ms": 0.0, "pack_ms": 0.0, "select_bytes": 0, "pack_bytes": 0}
    for li, (name, N, K) in enumerate(synth.LLAMA7B_LAYER_SET):
        W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(CONFIG_INDEX, li))
        Wd, Gd = torch.from_numpy(W).to(dev), torch.from_numpy(G).to(dev)
        entry = dict(name=name, N=N, K=K, packed={}, W=Wd if keep_dense else None, G=Gd if keep_dense else None)
        for bits in BIT_WIDTHS:
            reps = []
            for r in range(replicas):
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record()
                S = gwq.gwq_select_outliers(Wd, Gd, FRAC)
                e1.record()
                P = gwq.gwq_pack(Wd, S, bits, GROUP)
                e2.record()
                torch.cuda.synchronize()
                if r == replicas - 1:   # the last copy: one-time costs (module load, attributes) are behind
                    enc["select_ms"] += e0.elapsed_time(e1)
                    enc["pack_ms"] += e1.elapsed_time(e2)
                    enc["select_bytes"] += N * K * 4
                    enc["pack_bytes"] += N * K * 2 + N * K * bits // 8
                reps.append(P)
            entry["packed"][bits] = reps
        layers.append(entry)
        if not keep_dense:
            del Gd
    return layers, enc


def decode_cases(layers):
    """(layer index, bits, M) for every launch of one step, in launch order."""
    return [(li, bits, M) for M in DECODE_MS for bits in BIT_WIDTHS for li in range(len(layers))]


def time_region(torch, fn, iters: int) -> float:
    """Milliseconds per call of fn(i), CUDA events on the current stream, synchronised on both sides."""
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(iters):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters

class ReadProbe:
    """The read-only launch that gives the per-layer floor: the benchmark's own small CUDA library
    (paper_2411_00850_b200/bench_aid), loaded here and given the public arrays of a packed layer."""

    def __init__(self, torch):
        import ctypes
        path = os.path.join(ROOT, "paper_2411_00850_b200", "bench_aid", "libbench_read_probe.so")
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2411_00850_b200.build`")
        self.C = ctypes
        self.lib = ctypes.CDLL(path)
        self.lib.bench_read_probe.restype = ctypes.c_longlong
        self.lib.bench_read_probe.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_ulonglong),
                                              ctypes.c_int, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
        self.torch = torch
        self.sink = torch.zeros(4, dtype=torch.int32, device="cuda")
        self.blocks = 4 * torch.cuda.get_device_properties(0).multi_processor_count

    def arrays(self, P):
        """(pointer, bytes) of what a one-token product reads of P: codes, scales, zero-points, row pointers and
        4 bytes per outlier (the column indices stand for the 4-byte entries the kernels stream)."""
        h = P._h.contents
        S = h.S.contents
        groups = h.N * (h.K // h.group)
        return [(h.codes, h.N * (h.K // 32) * h.bits * 4), (h.scales, groups * 2), (h.zeros, groups),
                (S.row_ptr, (h.N + 1) * 4), (S.col_idx, S.nnz * 4)]

    def launch(self, P):
        arr = [(p, b) for (p, b) in self.arrays(P) if p and b >= 16]
        base = (self.C.c_void_p * len(arr))(*[p for p, _ in arr])
        size = (self.C.c_ulonglong * len(arr))(*[b for _, b in arr])
        n = self.lib.bench_read_probe(base, size, len(arr), self.sink.data_ptr(), self.blocks,
                                      self.torch.cuda.current_stream().cuda_stream)
        if n < 0:
            raise RuntimeError("bench_read_probe failed")
        return int(n)


def capture(torch, fn):
    """Capture fn() into a CUDA graph (after one eager run) and return a replay callable."""
    fn()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        fn()
    return g.replay


def run_cuda_arm(args):
    import torch
    import torch.distributed as dist

    from paper_2411_00850_b200 import binding as gwq
    from paper_2411_00850_b200 import build as gbuild

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        gbuild.build()
    if world > 1:
        dist.barrier()
    gwq.load_library()
    hbm_peak, tf_burst, tf_sust, peak_src = measured_peaks()

    replicas = 2   # two copies of every packed layer: ~420 MB touched between reuses (L2 is 126 MB)
    layers, enc = build_layer_set(torch, gwq, dev, replicas, keep_dense=True)
    cases = decode_cases(layers)
    xs = {}
    for li, L in enumerate(layers):
        for M in DECODE_MS:
            bits16, _ = synth.make_activations(M, L["K"], seed=synth.layer_seed(CONFIG_INDEX, li), dtype="f16")
            xs[(li, M)] = torch.from_numpy(bits16.view(np.int16).copy()).to(dev).view(torch.float16)
    ys = {(li, bits, M): torch.empty((M, layers[li]["N"]), dtype=torch.float16, device=dev)
          for (li, bits, M) in cases}

    side = [torch.cuda.Stream(device=dev) for _ in range(2)]
    fuse = not args.no_fuse
    # kernel launches of one step: one call per stage when the siblings are fused, else one per layer
    calls = [(lis if not fuse else lis[:1], M) for M in DECODE_MS for _b in BIT_WIDTHS for lis in STAGES]
    launches_per_step = sum(kernels_per_linear(M, layers[li]["K"]) for (lis, M) in calls for li in lis)
    calls_per_step = sum(len(lis) for (lis, M) in calls)

    def step_fn(rep):
        """The 7 linears of a decoder block in their data-flow order: q, k, v side by side, then o,
        then gate and up side by side, then down; the six (M, bits) passes follow one another."""
        def run():
            main = torch.cuda.current_stream()

            def stage(lis, bits, M):
                if len(lis) > 1 and fuse:   # sibling projections read the same activations: one call, one launch
                    gwq.gwq_linear_multi([layers[li]["packed"][bits][rep] for li in lis], xs[(lis[0], M)],
                                         outs=[ys[(li, bits, M)] for li in lis])
                    return
                if len(lis) > 1:
                    for s_ in side[:len(lis) - 1]:
                        s_.wait_stream(main)
                for k, li in enumerate(lis):
                    with torch.cuda.stream(main if k == 0 else side[k - 1]):
                        gwq.gwq_linear(layers[li]["packed"][bits][rep], xs[(lis[0], M)], out=ys[(li, bits, M)])
                if len(lis) > 1:
                    for s_ in side[:len(lis) - 1]:
                        main.wait_stream(s_)
            for M in DECODE_MS:
                for bits in BIT_WIDTHS:
                    for lis in STAGES:
                        stage(lis, bits, M)
        return run

    graphs = [capture(torch, step_fn(r)) for r in range(replicas)]
    step_bytes = sum(algorithmic_bytes(layers[li]["N"], layers[li]["K"], bits, GROUP,
                                       layers[li]["packed"][bits][0].nnz, M) for (li, bits, M) in cases)

    # ---- headline: W warm-up steps, then exactly K timed steps, barrier + synchronize on both sides
    for i in range(args.warmup):
        graphs[i % replicas]()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # the timed block of exactly `steps` steps is repeated at least `repeats` times and for at least `min_seconds` (each
    # block bracketed by a synchronisation on both sides); the headline is the median block, the fastest one is beside it
    blocks_ms, t_wall = [], time.perf_counter()
    while len(blocks_ms) < max(1, args.repeats) or (time.perf_counter() - t_wall < args.min_seconds and len(blocks_ms) < 2000):
        blocks_ms.append(time_region(torch, lambda i: graphs[i % replicas](), args.steps))
    ms_step, ms_step_min = float(np.median(blocks_ms)), float(min(blocks_ms))
    if world > 1:
        ms_step = max_over_ranks(ms_step, dev)
        ms_step_min = max_over_ranks(ms_step_min, dev)
        dist.barrier()
    clocks = sampler.stop() if rank == 0 else {}
    value = whole_job_gbs(step_bytes, ms_step, world)

    out = {
        "metric": METRIC, "value": round(value, 1), "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_step, 4), "ms_per_step_min": round(ms_step_min, 4),
        "timed_blocks": len(blocks_ms), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f16 x int4/int3 -> f32 accumulate", "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": [f"{n}:{N}x{K}" for n, N, K in synth.LLAMA7B_LAYER_SET],
                   "bits": list(BIT_WIDTHS), "group": GROUP, "outlier_frac": FRAC, "M": list(DECODE_MS),
                   "products_per_step": len(cases), "calls_per_step": calls_per_step,
                   "kernel_launches_per_step": launches_per_step, "step_bytes": step_bytes, "fused_siblings": fuse,
                   "launch_order": ("per (M, bits): q|k|v as one gwq_linear_multi launch, o, gate|up as one launch, down "
                                    "(decoder-block data flow)") if fuse else
                                   "per (M, bits): q|k|v concurrently, o, gate|up concurrently, down (decoder-block data flow)",
                   "l2": f"{replicas} rotating copies of the packed set ({replicas * step_bytes // 3 / 1e6:.0f} MB) "
                         "exceed the 126 MB L2 between reuses; one CUDA graph per copy"},
        "gpu_launches": args.steps * launches_per_step * len(blocks_ms),
        "clocks": clocks,
    }
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return None

    # ---- everything below: rank 0 only, N = 1 detail
    detail_iters = max(5, min(args.steps, 20))
    out["roofline"] = {
        "bound": "hbm", "kernel": f"gwq decode linear (all {calls_per_step} calls = {len(cases)} products of the step)",
        "achieved": round(step_bytes / (ms_step * 1e-3) / 1e9, 1), "peak": hbm_peak, "unit": "GB/s",
        "frac": round(step_bytes / (ms_step * 1e-3) / 1e9 / hbm_peak, 4), "peak_source": peak_src,
        "frac_of_nominal_8TBs": round(step_bytes / (ms_step * 1e-3) / 1e9 / 8000.0, 4),
        "avg_launch_us": round(ms_step * 1e3 / calls_per_step, 3), "traffic": None,
    }
    ratio = dominant_kernel_traffic()
    if ratio is not None:   # DRAM bytes per launch, averaged like `achieved` (traffic scales with the bytes streamed)
        out["roofline"]["traffic"] = round(ratio * step_bytes / calls_per_step)
        out["roofline"]["traffic_source"] = "profiles/decode_kernel_traffic.json (ncu, 11008x4096 W4 M=1), scaled by algorithmic bytes"
    if world == 1 and not args.headline_only:
        out["decode_cases"] = bench_decode_detail(torch, gwq, layers, xs, ys, detail_iters, hbm_peak)
        out["cublas_fp16"] = bench_dense_library(torch, layers, xs, detail_iters, step_bytes, ms_step)
        out["e2e"] = bench_e2e(torch, gwq, layers, cases, detail_iters, step_bytes)
        out["encode"] = {"select_ms": round(enc["select_ms"], 3), "pack_ms": round(enc["pack_ms"], 3),
                         "select_gbs_per_pass_of_G": round(enc["select_bytes"] / (enc["select_ms"] * 1e-3) / 1e9, 1),
                         "pack_gbs": round(enc["pack_bytes"] / (enc["pack_ms"] * 1e-3) / 1e9, 1),
                         "note": "14 encodes of the layer set (7 layers x 2 bit widths), last copy; call times: allocation of the outputs, "
                                 "9 + 3 dependent kernels and the read-back of the status word included"}
        out["decode_step_7b"] = bench_decode_step_7b(torch, gwq, layers, dev, detail_iters, hbm_peak)
        for L in layers:
            L["W"] = None
            L["G"] = None
        out["config0_single_layer"] = bench_config0(torch, gwq, dev, detail_iters, hbm_peak)
        if not args.skip_70b:
            out["llama70b_cases"] = bench_config4(torch, gwq, dev, 3, hbm_peak, tf_burst, args.prefill_iters)
        out["other_widths"] = bench_other_widths(args)
        out["prefill"] = bench_prefill(torch, gwq, dev, args, tf_burst, tf_sust)
        best = max(out["prefill"], key=lambda r: r["tflops"])
        out["prefill_roofline"] = {"bound": "tensor", "kernel": "gwq prefill linear (tcgen05)",
                                   "case": f"{best['N']}x{best['K']} W4 g128 1% M={best['M']} bf16 in",
                                   "achieved": best["tflops"], "peak": tf_burst, "unit": "TFLOP/s",
                                   "frac": round(best["tflops"] / tf_burst, 4), "peak_source": peak_src,
                                   "frac_of_sustained": round(best["tflops"] / tf_sust, 4),
                                   "frac_of_nominal_2250": round(best["tflops"] / 2250.0, 4)}
        out["cpu_baseline"] = cpu_baseline(sample_seconds=args.cpu_seconds)
        # compact copy of every per-case figure inside `roofline` ([N, K, bits, group, outlier %, M, us, fraction of the
        # measured peak]: HBM for M <= 32, tensor burst for the rest), so that one record carries them all
        cases = [[r["N"], r["K"], r["bits"], GROUP, 1.0, r["M"], r["us"], r["frac_measured_peak"]] for r in out["decode_cases"]]
        c0 = out["config0_single_layer"]
        cases.append([c0["N"], c0["K"], 4, GROUP, 1.0, 1, c0["us"], c0["frac_measured_peak"]])
        for r in out.get("llama70b_cases", []):
            cases.append([r["N"], r["K"], r["bits"], r["group"], round(100 * r["frac"], 1), r["M"], r["us"],
                          r.get("frac_measured_peak", r.get("frac_measured_burst"))])
        for r in out["other_widths"]:
            cases.append([r["N"], r["K"], r["bits"], r["group"], 1.0, r["M"], r["us"],
                          r["frac_measured_peak"] if r["M"] <= 32 else round(r["tflops"] / tf_burst, 4)])
        for r in out["prefill"]:
            cases.append([r["N"], r["K"], 4, GROUP, 1.0, r["M"], r["us"], r["frac_measured_burst"]])
        out["roofline"]["cases"] = cases
        out["roofline"]["cases_columns"] = "N, K, bits, group, outlier %, M, us per call, fraction of measured peak (HBM copy rate for M <= 32, bf16 tensor burst above)"
        out["roofline"]["decode_step_7b"] = [{"M": r["M"], "us": r["us_per_step"], "frac": r["frac_measured_peak"],
                                               "x_library_fp16": r["speedup_over_library_fp16"]}
                                              for r in out["decode_step_7b"]["cases"]]
    else:
        out["e2e"] = bench_e2e(torch, gwq, layers, cases, detail_iters, step_bytes, world)
    if world > 1:
        dist.destroy_process_group()
    return out


def bench_decode_detail(torch, gwq, layers, xs, ys, iters, hbm_peak):
    """Per (shape, bits, M): microseconds per launch with a cold L2 (the launches of one graph
    cycle through the layers of equal shape in both copies and a 256 MB read-only scrub precedes every timing).
    `read_only_launch_us` is the same loop with a kernel that only reads the layer's packed arrays: the
    floor of a one-launch-per-layer product (launch, ramp-up and drain included)."""
    rows = []
    # L2 scrub: READ 256 MB, so that the cache is left full of clean lines (a written scrub would leave dirty
    # lines whose write-back competes with the timed reads)
    scrub = torch.zeros(64 * 1024 * 1024, dtype=torch.int32, device=xs[(0, 1)].device)
    read_probe = ReadProbe(torch)

    def scrub_l2():
        return int(scrub.sum().item())
    shapes = {}
    for li, L in enumerate(layers):
        shapes.setdefault((L["N"], L["K"]), []).append(li)
    for (N, K), lis in shapes.items():
        for bits in BIT_WIDTHS:
            members = [(li, r) for r in range(len(layers[lis[0]]["packed"][bits])) for li in lis]

            def probe():
                for (li, r) in members:
                    read_probe.launch(layers[li]["packed"][bits][r])
            replay_probe = capture(torch, probe)
            floor_ms = None
            for _ in range(iters):
                scrub_l2()
                ms = time_region(torch, lambda i: replay_probe(), 1)
                floor_ms = ms if floor_ms is None else min(floor_ms, ms)
            floor_us = floor_ms * 1e3 / len(members)
            for M in DECODE_MS:

                def run():
                    for (li, r) in members:
                        gwq.gwq_linear(layers[li]["packed"][bits][r], xs[(li, M)], out=ys[(li, bits, M)])
                replay = capture(torch, run)
                best = None
                for _ in range(iters):
                    scrub_l2()
                    ms = time_region(torch, lambda i: replay(), 1)
                    best = ms if best is None else min(best, ms)
                us = best * 1e3 / len(members)
                nnz = layers[lis[0]]["packed"][bits][0].nnz
                b = algorithmic_bytes(N, K, bits, GROUP, nnz, M)
                rows.append({"N": N, "K": K, "bits": bits, "M": M, "us": round(us, 3), "bytes": b,
                             "gbs": round(b / us / 1e3, 1), "frac_measured_peak": round(b / us / 1e3 / hbm_peak, 4),
                             "frac_8TBs": round(b / us / 1e3 / 8000.0, 4), "launches_in_graph": len(members),
                             "read_only_launch_us": round(floor_us, 3), "x_read_only": round(us / floor_us, 2)})
    del scrub
    return rows


def bench_config4(torch, gwq, dev, iters, hbm_peak, tf_burst, prefill_iters):
    """Llama-70B-shaped layers (8192 x 8192, 28672 x 8192, 8192 x 28672) as the configuration states them: 4 and 3
    bits, groups of 64 and 128, 0.5 / 1 / 2 % outliers, M = 1, 8, 32 (fp16 activations; microseconds per launch with
    a cold L2, as in `bench_decode_detail`) and M = 2048 (bf16 activations with 8 heavy channels; TFLOP/s, the bf16
    library product on the unquantised weights beside it).  A layer is 31 to 137 MB of packed data, so the fixed
    cost of a launch weighs little here and the figures show what the kernels themselves sustain."""
    rows = []
    scrub = torch.zeros(64 * 1024 * 1024, dtype=torch.int32, device=dev)
    for si, (N, K) in enumerate(synth.LLAMA70B_SHAPES):
        W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(4, si))
        Wd, Gd = torch.from_numpy(W).to(dev), torch.from_numpy(G).to(dev)
        del W, G
        xs = {}
        for M in (1, 8, 32):
            bits16, _ = synth.make_activations(M, K, seed=synth.layer_seed(4, si), dtype="f16")
            xs[M] = torch.from_numpy(bits16.view(np.int16).copy()).to(dev).view(torch.float16)
        bits16, _ = synth.make_activations(2048, K, seed=synth.layer_seed(4, si), dtype="bf16", heavy_channels=8)
        xp = torch.from_numpy(bits16.view(np.int16).copy()).to(dev).view(torch.bfloat16)
        Wb = Wd.to(torch.bfloat16)
        for _ in range(2):
            torch.matmul(xp, Wb.t())
        lib_ms = time_region(torch, lambda i: torch.matmul(xp, Wb.t()), max(3, prefill_iters // 2))
        del Wb
        copies = 4 if N * K < 100_000_000 else 2     # more than the 126 MB L2 between reuses
        for frac in (0.005, 0.01, 0.02):
            S_list = [gwq.gwq_select_outliers(Wd, Gd, frac) for _ in range(copies * 4)]
            for bits in BIT_WIDTHS:
                for group in (64, 128):
                    packed = [gwq.gwq_pack(Wd, S_list.pop(), bits, group) for _ in range(copies)]
                    nnz = packed[0].nnz
                    for M in (1, 8, 32):
                        y = torch.empty((M, N), dtype=torch.float16, device=dev)
                        need = max(int(gwq.load_library().gwq_linear_workspace_bytes(P._h, gwq.GWQ_F16, M)) for P in packed)
                        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)

                        def run():
                            for P in packed:
                                gwq.gwq_linear(P, xs[M], out=y, workspace=ws if need else None)
                        replay = capture(torch, run)
                        best = None
                        for _ in range(iters):
                            int(scrub.sum().item())
                            ms = time_region(torch, lambda i: replay(), 1)
                            best = ms if best is None else min(best, ms)
                        us = best * 1e3 / copies
                        b = algorithmic_bytes(N, K, bits, group, nnz, M)
                        rows.append({"N": N, "K": K, "bits": bits, "group": group, "frac": frac, "M": M, "us": round(us, 2),
                                     "gbs": round(b / us / 1e3, 1), "frac_measured_peak": round(b / us / 1e3 / hbm_peak, 4)})
                    # M = 2048 on the tensor-core path (one packed copy; weights and activations exceed L2 together)
                    P = packed[0]
                    yp = torch.empty((2048, N), dtype=torch.bfloat16, device=dev)
                    need = int(gwq.load_library().gwq_linear_workspace_bytes(P._h, gwq.GWQ_BF16, 2048))
                    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)
                    for _ in range(2):
                        gwq.gwq_linear(P, xp, out=yp, workspace=ws)
                    ms = time_region(torch, lambda i: gwq.gwq_linear(P, xp, out=yp, workspace=ws), max(3, prefill_iters // 2))
                    tf = linear_flops(N, K, nnz, 2048) / (ms * 1e-3) / 1e12
                    rows.append({"N": N, "K": K, "bits": bits, "group": group, "frac": frac, "M": 2048, "us": round(ms * 1e3, 1),
                                 "tflops": round(tf, 1), "frac_measured_burst": round(tf / tf_burst, 4),
                                 "library_bf16_us": round(lib_ms * 1e3, 1)})
                    del packed, P, ws, yp
            del S_list
        del Wd, Gd, xp
        torch.cuda.empty_cache()
    del scrub
    return rows


def bench_config0(torch, gwq, dev, iters, hbm_peak):
    """The single-layer configuration as written: 4096 x 4096, seed 0, 4 bits, groups of 128, 1 % outliers, fp16
    activations, one token.  32 packed copies (300 MB) are cycled through in one CUDA graph, cold L2."""
    N = K = 4096
    W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(0, 0))
    Wd, Gd = torch.from_numpy(W).to(dev), torch.from_numpy(G).to(dev)
    packed = [gwq.gwq_pack(Wd, gwq.gwq_select_outliers(Wd, Gd, FRAC), 4, GROUP) for _ in range(32)]
    bits16, _ = synth.make_activations(1, K, seed=synth.layer_seed(0, 0), dtype="f16")
    x = torch.from_numpy(bits16.view(np.int16).copy()).to(dev).view(torch.float16)
    y = torch.empty((1, N), dtype=torch.float16, device=dev)

    def run():
        for P in packed:
            gwq.gwq_linear(P, x, out=y)
    replay = capture(torch, run)
    scrub = torch.zeros(64 * 1024 * 1024, dtype=torch.int32, device=dev)
    times = []
    for _ in range(iters):
        int(scrub.sum().item())
        times.append(time_region(torch, lambda i: replay(), 1) * 1e3 / len(packed))
    b = algorithmic_bytes(N, K, 4, GROUP, packed[0].nnz, 1)
    us = min(times)
    return {"N": N, "K": K, "bits": 4, "group": GROUP, "frac": FRAC, "M": 1, "seed": 0, "nnz": packed[0].nnz,
            "us": round(us, 3), "us_median": round(float(np.median(times)), 3), "bytes": b, "gbs": round(b / us / 1e3, 1),
            "frac_measured_peak": round(b / us / 1e3 / hbm_peak, 4), "launches_in_graph": len(packed)}


def bench_dense_library(torch, layers, xs, iters, step_bytes, ms_step):
    """torch.matmul (cuBLAS) fp16 on the unquantized weights: same layers, same M, one graph, two
    passes per replay so that each weight matrix (404 MB in total) is cold when it is read again."""
    ws = [L["W"] for L in layers]

    def run():
        for M in DECODE_MS:
            for _ in BIT_WIDTHS:          # the GWQ step visits every layer twice per M (W4 and W3)
                for li, W in enumerate(ws):
                    torch.matmul(xs[(li, M)], W.t())
    replay = capture(torch, run)
    for _ in range(3):
        replay()
    ms = time_region(torch, lambda i: replay(), iters)
    dense_bytes = sum(W.numel() * 2 for W in ws) * len(DECODE_MS) * len(BIT_WIDTHS)
    return {"ms_per_step": round(ms, 4), "dense_bytes_per_step": dense_bytes,
            "gbs_on_dense_bytes": round(dense_bytes / (ms * 1e-3) / 1e9, 1),
            "gwq_speedup_over_library": round(ms / ms_step, 3),
            "note": "library call (torch.matmul fp16), same 42 (layer, M) products, CUDA graph"}


def bench_decode_step_7b(torch, gwq, layers, dev, iters, hbm_peak, blocks: int = 32, bits: int = 4):
    """Linear time of one whole decode step of a Llama-2-7B-shaped model: `blocks` decoder blocks x 7 projections,
    every one its own packed copy (distinct addresses, ~3.8 GB at 4 bits: cold by construction), in data-flow
    order with the sibling projections fused, one CUDA graph; the dense fp16 library product on as many
    distinct dense copies beside it."""
    packed = []
    for b in range(blocks):
        row = []
        for L in layers:
            S = gwq.gwq_select_outliers(L["W"], L["G"], FRAC)
            row.append(gwq.gwq_pack(L["W"], S, bits, GROUP))
        packed.append(row)
    dense = [[L["W"].clone() for L in layers] for _ in range(blocks)]
    torch.cuda.synchronize()
    rows = []
    for M in (1, 8):
        xk = {}
        for K in sorted({L["K"] for L in layers}):
            bits16, _ = synth.make_activations(M, K, seed=synth.layer_seed(3, K % 97), dtype="f16")
            xk[K] = torch.from_numpy(bits16.view(np.int16).copy()).to(dev).view(torch.float16)
        ys = [torch.empty((M, L["N"]), dtype=torch.float16, device=dev) for L in layers]

        def run_gwq():
            for b in range(blocks):
                for lis in STAGES:
                    x = xk[layers[lis[0]]["K"]]
                    if len(lis) > 1:
                        gwq.gwq_linear_multi([packed[b][li] for li in lis], x, outs=[ys[li] for li in lis])
                    else:
                        gwq.gwq_linear(packed[b][lis[0]], x, out=ys[lis[0]])

        def run_dense():
            for b in range(blocks):
                for li, L in enumerate(layers):
                    torch.matmul(xk[L["K"]], dense[b][li].t())
        t = {}
        for name, fn in (("gwq", run_gwq), ("dense", run_dense)):
            replay = capture(torch, fn)
            for _ in range(2):
                replay()
            t[name] = time_region(torch, lambda i: replay(), iters)
        step_bytes = blocks * sum(algorithmic_bytes(L["N"], L["K"], bits, GROUP, packed[0][li].nnz, M)
                                  for li, L in enumerate(layers))
        rows.append({"M": M, "us_per_step": round(t["gwq"] * 1e3, 1), "tokens_per_s": round(M / (t["gwq"] * 1e-3), 1),
                     "step_bytes": step_bytes, "gbs": round(step_bytes / (t["gwq"] * 1e-3) / 1e9, 1),
                     "frac_measured_peak": round(step_bytes / (t["gwq"] * 1e-3) / 1e9 / hbm_peak, 4),
                     "library_fp16_us_per_step": round(t["dense"] * 1e3, 1),
                     "speedup_over_library_fp16": round(t["dense"] / t["gwq"], 3)})
    out = {"blocks": blocks, "bits": bits, "linears": blocks * len(layers),
           "calls_per_step": blocks * len(STAGES), "cases": rows,
           "note": f"{blocks} packed copies of the 7 synthetic layers at distinct addresses; q|k|v and gate|up fused; "
                   "linear layers only (no attention, norms or sampling)"}
    for row in packed:
        for P in row:
            P.free()
    del dense
    torch.cuda.empty_cache()
    return out


def bench_e2e(torch, gwq, layers, cases, iters, step_bytes, world=1):
    """The same step through gwq_linear_host: pinned host x in, pinned host y out, copies and the
    synchronisation inside the timed region."""
    xh, yh = {}, {}
    for li, L in enumerate(layers):
        for M in DECODE_MS:
            bits16, _ = synth.make_activations(M, L["K"], seed=synth.layer_seed(CONFIG_INDEX, li), dtype="f16")
            xh[(li, M)] = torch.from_numpy(bits16.view(np.int16).copy()).view(torch.float16).pin_memory()
    for (li, bits, M) in cases:
        yh[(li, bits, M)] = torch.empty((M, layers[li]["N"]), dtype=torch.float16).pin_memory()
    h2d = sum(xh[(li, M)].numel() * 2 for (li, bits, M) in cases)
    d2h = sum(yh[c].numel() * 2 for c in cases)

    def timed(call, sync_each_step):
        def step(i):
            r = i % 2
            for (li, bits, M) in cases:
                call(layers[li]["packed"][bits][r], xh[(li, M)], yh[(li, bits, M)])
            if sync_each_step:
                torch.cuda.synchronize()   # the step's results are on the host from here on
        for i in range(2):
            step(i)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for i in range(iters):
            step(i)
        torch.cuda.synchronize()
        return (time.perf_counter() - t0) / iters
    sec = timed(gwq.gwq_linear_host_async, True)
    sec_sync = timed(gwq.gwq_linear_host, False)
    return {"value": round(world * step_bytes / sec / 1e9, 1), "unit": "GB/s", "ms_per_step": round(sec * 1e3, 4),
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "note": "42 gwq_linear_host_async calls per step (pinned x copied in, product, y copied out), one "
                    "synchronisation per step after which every y is on the host",
            "synchronous_calls": {"value": round(world * step_bytes / sec_sync / 1e9, 1),
                                  "ms_per_step": round(sec_sync * 1e3, 4),
                                  "note": "the same with gwq_linear_host, which synchronises inside every call"}}


def bench_prefill(torch, gwq, dev, args, tf_burst, tf_sust):
    """4-bit, group 128, 1 % outliers, bf16 activations with 8 heavy channels; TFLOP/s on 2 M (N K + nnz)."""
    rows = []
    for si, (N, K) in enumerate(PREFILL_SHAPES):
        W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(2, si))
        Wd, Gd = torch.from_numpy(W).to(dev), torch.from_numpy(G).to(dev)
        P = gwq.gwq_pack(Wd, gwq.gwq_select_outliers(Wd, Gd, FRAC), 4, GROUP)
        del Gd
        Wb = Wd.to(torch.bfloat16)
        for M in PREFILL_MS:
            bits16, _ = synth.make_activations(M, K, seed=synth.layer_seed(2, si), dtype="bf16", heavy_channels=8)
            x = torch.from_numpy(bits16.view(np.int16).copy()).to(dev).view(torch.bfloat16)
            y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            need = int(gwq.load_library().gwq_linear_workspace_bytes(P._h, gwq.GWQ_BF16, M))
            ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)   # scratch of the call (caller-supplied)
            for _ in range(2):
                gwq.gwq_linear(P, x, out=y, workspace=ws)
            ms = time_region(torch, lambda i: gwq.gwq_linear(P, x, out=y, workspace=ws), args.prefill_iters)
            for _ in range(2):
                torch.matmul(x, Wb.t())
            ms_lib = time_region(torch, lambda i: torch.matmul(x, Wb.t()), args.prefill_iters)
            fl = linear_flops(N, K, P.nnz, M)
            tf = fl / (ms * 1e-3) / 1e12
            rows.append({"N": N, "K": K, "M": M, "us": round(ms * 1e3, 2), "tflops": round(tf, 2),
                         "frac_measured_burst": round(tf / tf_burst, 4), "frac_measured_sustained": round(tf / tf_sust, 4),
                         "frac_nominal_2250": round(tf / 2250.0, 4), "library_bf16_us": round(ms_lib * 1e3, 2),
                         "library_bf16_tflops": round(2 * M * N * K / (ms_lib * 1e-3) / 1e12, 2),
                         "workspace_bytes": need})
            del x, y, ws
        P.free()
        del Wd, Wb
    return rows


# ----------------------------------------------------------------------------- single cases (profiling, sweeps)
def bench_other_widths(args):
    """2- and 8-bit codes (the widths beside the paper's 3 and 4) on two layer shapes: one and sixteen tokens on the
    streaming kernel, 2048 tokens on the tensor-core path; the same protocol as --case (CUDA graph, cold L2).  The
    streaming kernel executes the same instructions per weight whatever the width, so these rows show how its time
    follows the instruction count rather than the bytes."""
    specs = []
    for bits in (8, 2):
        specs += [f"28672,8192,{bits},128,1,f16", f"11008,4096,{bits},128,1,f16", f"11008,4096,{bits},128,16,f16",
                  f"11008,4096,{bits},128,2048,bf16"]
    sub = argparse.Namespace(case=specs, case_copies=0, case_iters=max(3, args.prefill_iters // 4), case_stream=False)
    return run_cases(sub, quiet=True)["cases"]


def run_cases(args, quiet: bool = False):
    """--case N,K,bits,group,M,dtype[,frac] (repeatable): one synthetic layer per case, `copies` packed copies
    cycled through so that a launch does not find its weights in L2 (at least 256 MB between reuses unless
    --case-copies says otherwise).  Per case: microseconds per gwq_linear call, cold L2, replayed from a CUDA
    graph (min and median over --case-iters replays, a 256 MB read-only scrub before each), or in plain stream
    order with --case-stream (the form the profiler captures are taken on: few launches, no graph)."""
    import torch

    from paper_2411_00850_b200 import binding as gwq
    from paper_2411_00850_b200 import build as gbuild
    gbuild.build()
    gwq.load_library()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    hbm_peak, tf_burst, _tf_sust, peak_src = measured_peaks()
    scrub = torch.zeros(64 * 1024 * 1024, dtype=torch.int32, device=dev)
    rows, cache = [], {}
    for spec in args.case:
        f = spec.split(",")
        N, K, bits, group, M = (int(v) for v in f[:5])
        dtype = f[5] if len(f) > 5 else "f16"
        frac = float(f[6]) if len(f) > 6 else FRAC
        key = (N, K, bits, group, frac)
        if key not in cache:
            cache.clear()
            W, G = synth.make_weight_and_grad(N, K, 1)
            Wd, Gd = torch.from_numpy(W).to(dev), torch.from_numpy(G).to(dev)
            per_copy = N * K * bits // 8
            copies = args.case_copies or max(2, min(32, -(-256 * 1024 * 1024 // per_copy)))
            cache[key] = [gwq.gwq_pack(Wd, gwq.gwq_select_outliers(Wd, Gd, frac), bits, group) for _ in range(copies)]
            del Wd, Gd
        packed = cache[key]
        bits16, _ = synth.make_activations(M, K, 1, dtype=dtype, heavy_channels=8 if M > 32 else 0)
        x = torch.from_numpy(bits16.view(np.int16).copy()).to(dev).view(torch.float16 if dtype == "f16" else torch.bfloat16)
        y = torch.empty((M, N), dtype=x.dtype, device=dev)
        need = max(int(gwq.load_library().gwq_linear_workspace_bytes(P._h, gwq._dtype_code(x.dtype), M)) for P in packed)
        ws = torch.empty(max(need, 256), dtype=torch.uint8, device=dev)

        def run():
            for P in packed:
                gwq.gwq_linear(P, x, out=y, workspace=ws if need else None)
        for _ in range(2):
            run()
        torch.cuda.synchronize()
        times = []
        if args.case_stream:
            for _ in range(args.case_iters):
                times.append(time_region(torch, lambda i: run(), 1))
        else:
            replay = capture(torch, run)
            for _ in range(args.case_iters):
                int(scrub.sum().item())
                times.append(time_region(torch, lambda i: replay(), 1))
        us_min, us_med = min(times) * 1e3 / len(packed), float(np.median(times)) * 1e3 / len(packed)
        nnz = packed[0].nnz
        b = algorithmic_bytes(N, K, bits, group, nnz, M)
        fl = linear_flops(N, K, nnz, M)
        rows.append({"N": N, "K": K, "bits": bits, "group": group, "M": M, "dtype": dtype, "frac": frac,
                     "copies": len(packed), "us": round(us_min, 3), "us_median": round(us_med, 3), "bytes": b,
                     "gbs": round(b / us_min / 1e3, 1), "frac_measured_peak": round(b / us_min / 1e3 / hbm_peak, 4),
                     "tflops": round(fl / us_min / 1e6, 2), "status": gwq.gwq_device_status(packed[0])})
        if not quiet:
            print(json.dumps(rows[-1]), file=sys.stderr, flush=True)
    return {"mode": "cases", "order": "stream" if args.case_stream else "cuda graph, cold L2", "peak_source": peak_src,
            "hbm_peak_gbs": hbm_peak, "cases": rows}


# ----------------------------------------------------------------------------- the CPU checker, timed
def cpu_baseline(sample_seconds: float = 20.0) -> dict:
    """Times the CPU checker's forward product (reconstruction + float64 product) as it stands, on a
    bounded sample of the same workload: the first 4096x4096 layer of the set, 4 and 3 bits,
    M = 1, 4, 16, repeated until about `sample_seconds` have passed."""
    from oracle import gwq_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        blas_threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        blas_threads = 1
    name, N, K = synth.LLAMA7B_LAYER_SET[0]
    W, G = synth.make_weight_and_grad(N, K, synth.layer_seed(CONFIG_INDEX, 0))
    t_enc = time.perf_counter()
    enc = {bits: orc.quantize_layer(W, G, FRAC, bits, GROUP) for bits in BIT_WIDTHS}
    t_enc = time.perf_counter() - t_enc
    xs = {M: synth.make_activations(M, K, seed=synth.layer_seed(CONFIG_INDEX, 0), dtype="f16")[1] for M in DECODE_MS}
    done_bytes, passes = 0, 0
    t0 = time.perf_counter()
    while True:
        for bits in BIT_WIDTHS:
            L = enc[bits]
            for M in DECODE_MS:
                w_hat = orc.dequantize(L["codes"], L["scales"], L["zeros"], GROUP, L["row_ptr"], L["col_idx"], L["val"])
                orc.linear(xs[M], w_hat)
                done_bytes += algorithmic_bytes(N, K, bits, GROUP, int(L["row_ptr"][-1]), M)
        passes += 1
        if time.perf_counter() - t0 >= sample_seconds or passes >= 50:
            break
    sec = time.perf_counter() - t0
    return {"value": round(done_bytes / sec / 1e9, 4), "unit": "GB/s", "cores": int(blas_threads),
            "host_cores_available": len(os.sched_getaffinity(0)), "kind": "oracle",
            "sample": f"{passes} passes over q_proj 4096x4096 (W4 and W3, g128, 1% outliers) x M in (1,4,16): "
                      f"reconstruction + float64 product per call, {sec:.1f} s; encode on the CPU took {t_enc:.1f} s (untimed)",
            "seconds": round(sec, 2)}


def run_reference_arm(args):
    """--impl reference: the CPU checker on the host cores, same metric and unit."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    per_step = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    vals = []
    for i in range(args.warmup + args.steps):
        r = cpu_baseline(sample_seconds=per_step)
        if i >= args.warmup:
            vals.append(r)
    value = float(np.mean([v["value"] for v in vals]))
    ms = float(np.mean([v["seconds"] for v in vals])) * 1e3
    return {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": "GB/s",
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": round(ms, 2), "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD + " (sampled: q_proj 4096x4096 only)", "sampled": vals[-1]["sample"]},
            "cpu_baseline": {"value": round(value, 4), "unit": "GB/s", "cores": vals[-1]["cores"], "kind": "oracle",
                             "sample": vals[-1]["sample"]},
            "e2e": {"value": round(value, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--repeats", type=int, default=10, help="timed blocks of `steps` steps, at least (median reported)")
    ap.add_argument("--min-seconds", type=float, default=2.0,
                    help="keep timing blocks until this much time has passed, so that the clock sampler sees the load")
    ap.add_argument("--prefill-iters", type=int, default=20)
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--headline-only", action="store_true", help="skip the per-case detail sections")
    ap.add_argument("--skip-70b", action="store_true", help="skip the Llama-70B-shaped decode cases")
    ap.add_argument("--no-fuse", action="store_true",
                    help="launch sibling projections as separate concurrent calls instead of one gwq_linear_multi")
    ap.add_argument("--case", action="append", default=[], metavar="N,K,bits,group,M,dtype[,frac]",
                    help="time gwq_linear on one synthetic layer instead of the benchmark (repeatable)")
    ap.add_argument("--case-copies", type=int, default=0, help="packed copies cycled through (default: 256 MB worth)")
    ap.add_argument("--case-iters", type=int, default=10)
    ap.add_argument("--case-stream", action="store_true", help="plain stream order instead of a CUDA graph, no L2 scrub")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.case:
        print(json.dumps(run_cases(args), ensure_ascii=False))
        return
    out = run_reference_arm(args) if args.impl == "reference" else run_cuda_arm(args)
    if out is not None:
        print(json.dumps(out, ensure_ascii=False))


if __name__ == "__main__":
    main()
