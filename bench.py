#!/usr/bin/env python
"""Benchmark of the MeteoRA linear forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--tokens T]

Workload (N = 1 and every rank of N > 1): the LLaMA3-8B q_proj-shaped MeteoRA linear, d_in = d_out = 4096,
28 adapters of rank 8, top-2, bf16 with fp32 accumulation, a decode batch of T = 128 tokens.  One STEP is one
pass of the whole layer (gate, top-k, softmax, shrink, base product, expand, store) over `--modules` = 16
independent MeteoRA modules (own weights, own gate, own tokens), the way consecutive projections of a decoder
are visited during decoding; their weights total ~0.6 GB, far beyond the 126 MB L2, so every step streams its
weights from HBM.  value = (modules x T x K x ranks) tokens through a MeteoRA linear per second.

The step is captured once into a CUDA graph (the library's launches are capturable: no allocation, no
synchronisation) and replayed K times; `--launch stream` issues the same calls directly instead.
One JSON line is printed by rank 0.  `--impl reference` times the CPU oracle instead.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "MeteoRA-linear tokens/s at LLaMA3-8B shapes (N=28, r=8, k=2)"
D_IN = D_OUT = 4096
N_ADAPTERS, RANK, TOPK = 28, 8, 2
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0          # the figure quoted for the part (7.7 - 8 TB/s); context beside the measured peak
NOMINAL_BF16_TFLOPS = 2250.0      # dense bf16, nominal

# DRAM traffic of one launch of the dominant kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum), keyed by tokens; valid only for the kernel source it was taken from.
NCU_TRAFFIC = {"kernel_sha": "977a04827624e8b9", "bytes_per_launch": {"128": 38597803 + 27563, "1": 37557589 + 0}}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--tokens", type=int, default=128, help="decode batch T per module")
    ap.add_argument("--repeats", type=int, default=5,
                    help="the timed region of --steps steps is run this many times; the line reports the median region "
                         "(value, ms_per_step) and the spread")
    ap.add_argument("--no-prefill-line", action="store_true", help="skip the prefill_roofline measurement")
    ap.add_argument("--prefill-only", action="store_true",
                    help="run only the prefill_roofline measurement (config 2 gate/up, T = 2048) and print it")
    ap.add_argument("--modules", type=int, default=16, help="independent MeteoRA modules visited per step")
    ap.add_argument("--launch", choices=["graph", "stream"], default="graph")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="target length of the cpu_baseline sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-streams", type=int, default=4,
                    help="streams the end-to-end step spreads its independent modules over")
    ap.add_argument("--sweep", action="store_true",
                    help="time every (shape, T) of configs 1-3 instead of the headline step; one JSON line each")
    ap.add_argument("--variants", action="store_true",
                    help="time the variants of the method at 4096 -> 4096 (top-k, rank, adapter count, temperature), "
                         "the axes of the paper's synthetic sweep (App. A.7); one JSON line each")
    ap.add_argument("--knob", action="append", default=[], metavar="NAME=VALUE",
                    help="set a measurement knob of the library (meteora_set_tuning) before timing; repeatable")
    ap.add_argument("--gate-backward", action="store_true",
                    help="meteora_gate_backward / _bt at 1 - 8192 tokens (4096 -> 4096), per call from a CUDA graph")
    ap.add_argument("--standalone", action="store_true",
                    help="time the standalone entry points (gate + top-k, bucketing, LoRA term by segments) beside the fused "
                         "forward's stacked shrink + selection; also part of --sweep")
    ap.add_argument("--layer", action="store_true",
                    help="time a LLaMA3-8B decoder layer whose seven linears are MeteoRA linears fed by the real upstream "
                         "activations (64 sequences at context 2048, and one 4096-token prefill); also part of --sweep")
    ap.add_argument("--decode-loop", action="store_true",
                    help="time one autoregressive decode step over the 224 MeteoRA linears of a LLaMA3-8B-shaped "
                         "stack (ms per generated token, the unit of App. A.7); also part of --sweep")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peak():
    """Sustained dense bf16 TFLOP/s (the kernels here are timed inside long loops)."""
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            return float(json.load(fh)["bf16_tflops_sustained"]), "measured"
    except Exception:
        return 1400.0, "fallback"


def kernel_sha():
    """Hash of the code of the kernels the ncu traffic figure was taken on: their sources with comments and
    white space removed, so that an edit of a comment does not void the figure and an edit of the code does."""
    import re
    h = hashlib.sha256()
    for name in ("wgemm_tcgen05.cu", "decode_fused.cuh", "decode_stream.cuh", "decode_cluster.cuh", "wgemm_pair.cuh",
                 "select.cuh"):
        with open(os.path.join(ROOT, "paper_2405_13053_b200", "csrc", name), "r") as fh:
            text = fh.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update(re.sub(r"\s+", "", text).encode())
    return h.hexdigest()[:16]


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in out.splitlines():
            f = [c.strip() for c in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------------- reference arm
def run_reference(args):
    """The CPU oracle, as it stands, on this machine's host cores: each step is one module's T tokens."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2405_13053_b200 import workloads

    T = args.tokens
    w = workloads.config1(T)
    cores = oracle.num_threads()
    steps, warmup = args.steps, args.warmup
    # bound the run: the oracle needs ~21 ms of one core per token at this shape
    budget_steps = max(1, int(60.0 / max(0.021 * T / cores, 1e-3)))
    steps = min(steps, budget_steps)
    warmup = min(warmup, max(1, budget_steps // 10))
    for _ in range(warmup):
        oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], w.k)
    t0 = time.perf_counter()
    for _ in range(steps):
        oracle.linear_forward(w["x"], w["W0"], w["A"], w["B"], w["Wg"], w.k)
    dt = time.perf_counter() - t0
    value = T * steps / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": 1e3 * dt / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"config1: 4096->4096 MeteoRA linear, N=28 r=8 k=2, bf16-valued inputs, T={T}",
                       "sample": f"one module, {T} tokens per step"},
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": f"{steps} steps of {T} tokens of one module"},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------- rank plumbing
def rank_info():
    """(world size, rank, local rank) of this process as torchrun exports them; (1, 0, 0) when launched alone."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def module_seed(i, rank):
    """Seed of module i on a rank: every rank works on modules of its own (token / module shards, no exchange)."""
    return 1000 + 100 * i + 17 * rank


def max_over_ranks(ms, world, device):
    """The slowest rank's elapsed time: the job is as fast as its slowest shard."""
    import torch
    import torch.distributed as dist

    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(modules, tokens, world, steps, ms_total):
    """Tokens through a MeteoRA linear per second, summed over all ranks."""
    return modules * tokens * world * steps / (ms_total * 1e-3)


def prefill_line(mb, lib, tc_peak, tc_kind, hbm_peak):
    """One prefill figure for the default line (the headline workload is a decode batch and HBM-bound): config 2's
    gate/up shape, 4096 -> 14336 with 2048 tokens from 4 clusters, the whole MeteoRA linear per call (three or four launches:
    stacked shrink, selection, base product with the expand) against the sustained bf16 tensor peak, and the
    base-product kernel alone from event pairs around its launches."""
    import ctypes

    import torch

    from paper_2405_13053_b200 import workloads

    d_in, d_out, T = workloads.CONFIG2_SHAPES["gate_up"][0], workloads.CONFIG2_SHAPES["gate_up"][1], 2048
    dt = torch.bfloat16
    g = torch.Generator(device="cuda").manual_seed(29)
    x = torch.from_numpy(workloads.make_x(T, d_in, "clusters", 2001, "bf16")).to(dt).cuda()
    W0 = (0.02 * torch.randn(d_out, d_in, device="cuda", generator=g)).to(dt)
    A = ((torch.rand(N_ADAPTERS, RANK, d_in, device="cuda", generator=g) * 2 - 1) / d_in ** 0.5).to(dt)
    B = (0.01 * torch.randn(N_ADAPTERS, d_out, RANK, device="cuda", generator=g)).to(dt)
    Wg = (torch.randn(N_ADAPTERS, d_in, device="cuda", generator=g) / d_in ** 0.5).to(dt)
    y = torch.empty(T, d_out, device="cuda", dtype=dt)
    shape = mb.make_shape(T, d_in, d_out, N_ADAPTERS, RANK, TOPK, dt)
    ws = mb.alloc_workspace(shape)

    def call():
        rc = lib.meteora_linear_forward(x.data_ptr(), W0.data_ptr(), A.data_ptr(), B.data_ptr(), Wg.data_ptr(),
                                        ctypes.byref(shape), y.data_ptr(), ws.data_ptr(), ws.numel(),
                                        torch.cuda.current_stream().cuda_stream)
        if rc != 0:
            raise mb.MeteoraError(rc, "meteora_linear_forward")

    for _ in range(3):
        call()
    torch.cuda.synchronize()
    regions = []
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(20):
            call()
        e1.record()
        torch.cuda.synchronize()
        regions.append(e0.elapsed_time(e1) * 1e3 / 20)
    us_call = float(np.median(regions))
    mb.meteora_profile_begin(20)
    for _ in range(20):
        call()
    ms, n = mb.meteora_profile_end()
    if mb.meteora_workspace_status(ws) != 0:
        raise mb.MeteoraError(-6, "device status after the prefill region")
    us_base = ms * 1e3 / max(n, 1)
    flops = 2.0 * T * d_in * d_out + 2.0 * T * N_ADAPTERS * d_in + 2.0 * T * TOPK * RANK * (d_in + d_out)
    flops_base = 2.0 * T * d_in * d_out + 2.0 * T * TOPK * RANK * d_out
    plan = mb.meteora_describe_plan(shape).split(" fused_refused")[0]
    return {"workload": f"config2 gate_up: 4096->14336 MeteoRA linear, N=28 r=8 k=2, bf16, prefill batch T={T} (4 clusters)",
            "bound": "tensor", "unit": "TFLOP/s", "peak": tc_peak, "peak_kind": f"of {tc_kind} (sustained dense bf16)",
            "us_per_call": us_call, "us_per_call_min": min(regions), "us_per_call_max": max(regions),
            "algorithmic_flops_per_call": flops, "achieved": flops / us_call / 1e6, "frac": flops / us_call / 1e6 / tc_peak,
            "frac_of_nominal": flops / us_call / 1e6 / NOMINAL_BF16_TFLOPS,
            "base_product_kernel": {"us_per_launch": us_base, "achieved": flops_base / us_base / 1e6,
                                    "frac": flops_base / us_base / 1e6 / tc_peak, "launches_timed": n},
            "launches_per_call": int(plan.split("launches=")[1].split()[0]) if "launches=" in plan else 3, "plan": plan}


# --------------------------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2405_13053_b200 import binding as mb
    from paper_2405_13053_b200 import build as lib_build
    from paper_2405_13053_b200 import workloads

    world, rank, local = rank_info()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        lib_build.build_library()
    if world > 1:
        dist.barrier()
    lib = mb.load_library()
    import ctypes

    T, R, K, W = args.tokens, args.modules, args.steps, max(args.warmup, 3)
    dt = torch.bfloat16
    shape = mb.make_shape(T, D_IN, D_OUT, N_ADAPTERS, RANK, TOPK, dt)
    es = 2

    # ---- inputs: R independent modules (seeded), resident in HBM; pinned host copies of x / y for e2e
    mods = []
    host_w0 = None
    for i in range(R):
        w = workloads.make_workload(f"config1/T{T}/module{i}", T=T, d_in=D_IN, d_out=D_OUT, N=N_ADAPTERS, r=RANK,
                                    k=TOPK, dtype="bf16", x_kind="rms", seed=module_seed(i, rank))
        if i == 0:
            host_w0 = w
        m = {n: torch.from_numpy(w[n]).to(dt).cuda() for n in ("x", "W0", "A", "B", "Wg")}
        m["y"] = torch.empty((T, D_OUT), dtype=dt, device="cuda")
        m["x_host"] = torch.from_numpy(w["x"]).to(dt).pin_memory()
        m["y_host"] = torch.empty((T, D_OUT), dtype=dt).pin_memory()
        mods.append(m)
    # Scratch: the calls of the device-resident step are ordered on one stream and share ONE workspace, the way a
    # decoder passes the same scratch buffer to every layer; the end-to-end step spreads its modules over several
    # streams, so there every stream has its own (calls that may overlap in time must not share one).
    n_e2e = max(1, args.e2e_streams)
    ws_dev = mb.alloc_workspace(shape)
    ws_e2e = [mb.alloc_workspace(shape) for _ in range(n_e2e)]
    for i, m in enumerate(mods):
        m["ws"] = ws_dev
        m["ws_host"] = ws_e2e[i % n_e2e]
    torch.cuda.synchronize()

    def call_device(m):
        rc = lib.meteora_linear_forward(m["x"].data_ptr(), m["W0"].data_ptr(), m["A"].data_ptr(), m["B"].data_ptr(),
                                        m["Wg"].data_ptr(), ctypes.byref(shape), m["y"].data_ptr(),
                                        m["ws"].data_ptr(), m["ws"].numel(), torch.cuda.current_stream().cuda_stream)
        if rc != 0:
            raise mb.MeteoraError(rc, "meteora_linear_forward")

    def call_host(m):
        rc = lib.meteora_linear_forward_host(m["x_host"].data_ptr(), m["W0"].data_ptr(), m["A"].data_ptr(),
                                             m["B"].data_ptr(), m["Wg"].data_ptr(), ctypes.byref(shape),
                                             m["y_host"].data_ptr(), m["ws_host"].data_ptr(), m["ws_host"].numel(),
                                             torch.cuda.current_stream().cuda_stream)
        if rc != 0:
            raise mb.MeteoraError(rc, "meteora_linear_forward_host")

    def step_device():
        for m in mods:
            call_device(m)

    # End-to-end step: the modules are independent, so their calls go round-robin onto a few streams and the
    # host-to-device copy of one module, the kernel of another and the device-to-host copy of a third overlap
    # (the two copy engines and the SMs); every stream is joined before the step ends.
    e2e_streams = [torch.cuda.Stream() for _ in range(n_e2e)]

    def step_host():
        cur = torch.cuda.current_stream()
        for st in e2e_streams:
            st.wait_stream(cur)
        for i, m in enumerate(mods):
            with torch.cuda.stream(e2e_streams[i % len(e2e_streams)]):
                call_host(m)
        for st in e2e_streams:
            cur.wait_stream(st)

    def make_runner(step_fn):
        """Capture one step into a CUDA graph; fall back to direct launches if capture is refused."""
        if args.launch == "graph":
            try:
                side = torch.cuda.Stream()
                side.wait_stream(torch.cuda.current_stream())
                with torch.cuda.stream(side):
                    step_fn()                                  # tensor maps get encoded outside the capture
                torch.cuda.current_stream().wait_stream(side)
                torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    step_fn()
                return g.replay, "graph"
            except Exception as e:                             # noqa: BLE001
                sys.stderr.write(f"[bench] graph capture failed ({e}); using direct launches\n")
                torch.cuda.synchronize()
        return step_fn, "stream"

    def timed(run, steps, warmup):
        for _ in range(warmup):
            run()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            run()
        e1.record()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        return max_over_ranks(e0.elapsed_time(e1), world, "cuda")

    def check_status():
        for ws in [ws_dev] + ws_e2e:
            st = mb.meteora_workspace_status(ws)
            if st != 0:
                raise mb.MeteoraError(st, "device status after the timed region")

    # ---- device-resident timing (the headline value)
    run_dev, mode = make_runner(step_device)
    uuid = str(torch.cuda.get_device_properties(local).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    sampler = ClockSampler(uuid)
    reps = max(1, args.repeats)
    regions = [timed(run_dev, K, W if i == 0 else 0) for i in range(reps)]     # every region: exactly K steps
    ms_total = float(np.median(regions))
    # keep the GPU under the same load a little longer if the regions were too short for a clock sample
    t_extra = time.time()
    while time.time() - t_extra < 0.7:
        run_dev()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    check_status()
    value = whole_job_value(R, T, world, K, ms_total)

    # ---- end to end: x from pinned host memory, y back to host, every step, through the host entry point
    run_e2e, mode_e2e = make_runner(step_host)

    def e2e_step():
        run_e2e()
        torch.cuda.current_stream().synchronize()          # the step's result is read on the host

    e2e_regions = [timed(e2e_step, K, W if i == 0 else 0) for i in range(reps)]
    ms_e2e = float(np.median(e2e_regions))
    check_status()
    e2e_value = whole_job_value(R, T, world, K, ms_e2e)

    # ---- dominant kernel.  Which kernels a call launches depends on the shape (meteora_describe_plan):
    #   single-launch decode kernel: one launch is the whole call, so its average duration over the timed region
    #     is the graph-replayed region itself divided by the launches (idle gaps between launches included);
    #   three-launch chain: event pairs around the base-product launch of every call, in a second region of the
    #     same launches issued behind a long blocker kernel so that the host is never the bottleneck.
    plan = mb.meteora_describe_plan(shape)
    single_launch = "path=fused_decode" in plan or "path=stream_decode" in plan
    launches_per_call = 1 if single_launch else 3
    if single_launch:
        kernel_name = ("k_decode_stream" if "path=stream_decode" in plan else "k_decode_fused") + \
            " (base product + stacked shrink + selection + LoRA expand, one launch per call)"
        kernel_ms, kernel_launches = ms_total, K * R
    else:
        kernel_name = ("k_wgemm_pair (base product + LoRA expand on pairs of SMs)" if "pairs_of_ctas" in plan
                       else "k_wgemm (base product + LoRA expand)")
        prof_steps = min(K, 8)
        step_device()
        torch.cuda.synchronize()
        blocker = torch.empty((8192, 8192), dtype=dt, device="cuda")
        for _ in range(6):
            torch.matmul(blocker, blocker)                      # ~6 ms of queued work ahead of the timed launches
        mb.meteora_profile_begin(prof_steps * R)
        for _ in range(prof_steps):
            step_device()
        kernel_ms, kernel_launches = mb.meteora_profile_end()
        del blocker
    check_status()

    # ---- algorithmic bytes (adapters actually selected, from the realised routing of module 0)
    step_device()                                              # the shared workspace holds the last module's routing
    torch.cuda.synchronize()
    idx0, _ = mb.meteora_workspace_routing(shape, ws_dev)
    touched = int(torch.unique(idx0).numel())
    bytes_base = (D_IN * D_OUT + touched * D_OUT * RANK + T * (D_IN + D_OUT)) * es
    bytes_path = bytes_base + (N_ADAPTERS * D_IN + touched * RANK * D_IN) * es
    bytes_kernel = bytes_path if single_launch else bytes_base
    peak, peak_kind = measured_peaks()
    tc_peak, tc_kind = measured_tensor_peak()
    per_launch_s = kernel_ms * 1e-3 / max(kernel_launches, 1)
    flops_base = 2.0 * T * D_IN * D_OUT + 2.0 * T * TOPK * RANK * D_OUT
    flops_path = flops_base + 2.0 * T * N_ADAPTERS * D_IN + 2.0 * T * TOPK * RANK * D_IN
    flops_kernel = flops_path if single_launch else flops_base
    # the bound of the kernel: whichever of its algorithmic bytes / HBM and flops / tensor peak takes longer
    tensor_bound = flops_kernel / (tc_peak * 1e12) > bytes_kernel / (peak * 1e9)
    achieved = bytes_kernel / per_launch_s / 1e9
    traffic = None
    if NCU_TRAFFIC["kernel_sha"] == kernel_sha() and single_launch:
        traffic = NCU_TRAFFIC["bytes_per_launch"].get(str(T))
    per_call_s = ms_total * 1e-3 / (K * R)

    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_total / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "repeats": {"regions": reps, "steps_per_region": K, "statistic": "median",
                    "ms_per_step_min": min(regions) / K, "ms_per_step_median": ms_total / K,
                    "ms_per_step_max": max(regions) / K,
                    "value_best": whole_job_value(R, T, world, K, min(regions)),
                    "value_worst": whole_job_value(R, T, world, K, max(regions))},
        "config": {"workload": f"config1: LLaMA3-8B q_proj MeteoRA linear 4096->4096, N=28 r=8 k=2, bf16, "
                               f"{'decode' if T <= 256 else 'prefill'} batch T={T}; step = {R} independent modules",
                   "tokens_per_module": T, "modules_per_step": R, "launch": mode, "e2e_launch": mode_e2e, "e2e_streams": len(e2e_streams),
                   "l2": f"weights of the {R} modules total {R * bytes_path / 1e6:.0f} MB > 126 MB L2, "
                         "so no weight is L2-resident between visits",
                   "workspace": "one scratch buffer shared by the step's stream-ordered calls (one per stream end to end)",
                   "parallelism": f"token-sharded replicas x{world}, no collective", "plan": plan},
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": R * T * D_IN * es,
                "d2h_bytes_per_step": R * T * D_OUT * es, "ms_per_step": ms_e2e / K,
                "ms_per_step_min": min(e2e_regions) / K, "ms_per_step_max": max(e2e_regions) / K},
        "gpu_launches": launches_per_call * R * K,
        "clocks": clocks,
        "roofline": ({"bound": "tensor", "kernel": kernel_name, "achieved": flops_kernel / per_launch_s / 1e12,
                      "peak": tc_peak, "peak_kind": f"of {tc_kind} (sustained dense bf16)", "unit": "TFLOP/s",
                      "frac": flops_kernel / per_launch_s / 1e12 / tc_peak, "traffic": None,
                      "frac_of_nominal": flops_kernel / per_launch_s / 1e12 / NOMINAL_BF16_TFLOPS,
                      "nominal_peak": NOMINAL_BF16_TFLOPS,
                      "algorithmic_flops_per_launch": flops_kernel, "us_per_launch": per_launch_s * 1e6,
                      "launches_timed": kernel_launches} if tensor_bound else
                     {"bound": "hbm", "kernel": kernel_name, "achieved": achieved,
                      "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                      "frac_of_nominal": achieved / NOMINAL_HBM_GBS, "nominal_peak": NOMINAL_HBM_GBS,
                      "traffic": traffic, "algorithmic_bytes_per_launch": bytes_kernel,
                      "us_per_launch": per_launch_s * 1e6, "launches_timed": kernel_launches}),
        "path_roofline": ({"bound": "tensor", "algorithmic_flops_per_call": flops_path, "us_per_call": per_call_s * 1e6,
                           "achieved": flops_path / per_call_s / 1e12, "peak": tc_peak, "unit": "TFLOP/s",
                           "frac": flops_path / per_call_s / 1e12 / tc_peak, "adapters_touched": touched}
                          if flops_path / (tc_peak * 1e12) > bytes_path / (peak * 1e9) else
                          {"bound": "hbm", "algorithmic_bytes_per_call": bytes_path, "us_per_call": per_call_s * 1e6,
                           "achieved": bytes_path / per_call_s / 1e9, "peak": peak, "unit": "GB/s",
                           "frac": bytes_path / per_call_s / 1e9 / peak, "adapters_touched": touched}),
    }

    if world == 1 and not args.no_prefill_line:
        line["prefill_roofline"] = prefill_line(mb, lib, tc_peak, tc_kind, peak)

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        cores = oracle.num_threads()
        w = host_w0
        n_tok, t_cpu, chunk = 0, 0.0, min(T, 32)
        while t_cpu < args.cpu_seconds and n_tok < 16384:
            sl = slice(n_tok % T, n_tok % T + chunk) if n_tok % T + chunk <= T else slice(0, chunk)
            t0 = time.perf_counter()
            oracle.linear_forward(w["x"][sl], w["W0"], w["A"], w["B"], w["Wg"], w.k)
            t_cpu += time.perf_counter() - t0
            n_tok += chunk
        # the same oracle on one core (a short sample: ~3 s)
        oracle.set_threads(1)
        n1, t1 = 0, 0.0
        while t1 < 3.0 and n1 < 4096:
            t0 = time.perf_counter()
            oracle.linear_forward(w["x"][:1], w["W0"], w["A"], w["B"], w["Wg"], w.k)
            t1 += time.perf_counter() - t0
            n1 += 1
        oracle.set_threads(cores)
        line["cpu_baseline"] = {"value": n_tok / t_cpu, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                                "sample": f"{n_tok} tokens of module 0 in chunks of {chunk} ({t_cpu:.1f} s)",
                                "value_1core": n1 / t1, "sample_1core": f"{n1} tokens one at a time ({t1:.1f} s)",
                                "note": "the oracle as it stands: plain C, fp64 accumulation, -O2 -ffp-contract=off, "
                                        "OpenMP over tokens; never tuned"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------- sweep
def run_sweep(args):
    """Per-call time of meteora_linear_forward for every shape of configs 1-3 (device-resident inputs, graph
    replay over enough independent modules that HBM-bound shapes never find their weights in L2)."""
    import ctypes

    import torch

    from paper_2405_13053_b200 import binding as mb
    from paper_2405_13053_b200 import build as lib_build
    from paper_2405_13053_b200 import workloads

    lib_build.build_library()
    lib = mb.load_library()
    torch.cuda.set_device(0)
    hbm, _ = measured_peaks()
    tc, _ = measured_tensor_peak()
    dt, es = torch.bfloat16, 2
    cases = [("config1", "q_proj", 4096, 4096, T, "rms") for T in workloads.CONFIG1_T]
    for name, (di, do) in workloads.CONFIG2_SHAPES.items():
        cases += [("config2", name, di, do, T, "clusters") for T in workloads.CONFIG2_T]
    for name, (di, do) in workloads.CONFIG3_SHAPES.items():
        cases += [("config3", name, di, do, T, "normal") for T in workloads.CONFIG3_T]
    for cfg, name, d_in, d_out, T, x_kind in cases:
        w_bytes = d_in * d_out * es
        R = max(1, min(16, int(600e6 // w_bytes))) if T <= 256 else 1
        shape = mb.make_shape(T, d_in, d_out, N_ADAPTERS, RANK, TOPK, dt)
        g = torch.Generator(device="cuda").manual_seed(7)
        x_np = workloads.make_x(T, d_in, x_kind, 5, "bf16")          # token statistics of the config; weights on device
        mods = []
        ws_shared = mb.alloc_workspace(shape)                        # stream-ordered calls share one scratch buffer
        for i in range(R):
            m = {"x": torch.from_numpy(x_np).to(dt).cuda(),
                 "W0": (0.02 * torch.randn(d_out, d_in, device="cuda", generator=g)).to(dt),
                 "A": ((torch.rand(N_ADAPTERS, RANK, d_in, device="cuda", generator=g) * 2 - 1) / d_in ** 0.5).to(dt),
                 "B": (0.01 * torch.randn(N_ADAPTERS, d_out, RANK, device="cuda", generator=g)).to(dt),
                 "Wg": (torch.randn(N_ADAPTERS, d_in, device="cuda", generator=g) / d_in ** 0.5).to(dt),
                 "y": torch.empty(T, d_out, device="cuda", dtype=dt), "ws": ws_shared}
            mods.append(m)

        def step():
            for m in mods:
                rc = lib.meteora_linear_forward(m["x"].data_ptr(), m["W0"].data_ptr(), m["A"].data_ptr(),
                                                m["B"].data_ptr(), m["Wg"].data_ptr(), ctypes.byref(shape),
                                                m["y"].data_ptr(), m["ws"].data_ptr(), m["ws"].numel(),
                                                torch.cuda.current_stream().cuda_stream)
                if rc != 0:
                    raise mb.MeteoraError(rc, "meteora_linear_forward")

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        iters = 100 if T <= 256 else 20
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        for m in mods:
            st = mb.meteora_workspace_status(m["ws"])
            if st != 0:
                raise mb.MeteoraError(st, "device status")
        us = e0.elapsed_time(e1) * 1e3 / (iters * R)
        idx0, _ = mb.meteora_workspace_routing(shape, mods[0]["ws"])
        touched = int(torch.unique(idx0).numel())
        counts = torch.bincount(idx0.flatten().long(), minlength=N_ADAPTERS).tolist()
        nbytes = (d_in * d_out + N_ADAPTERS * d_in + touched * RANK * (d_in + d_out) + T * (d_in + d_out)) * es
        flops = 2.0 * T * d_in * d_out + 2.0 * T * N_ADAPTERS * d_in + 2.0 * T * TOPK * RANK * (d_in + d_out)
        t_mem, t_tc = nbytes / hbm / 1e3, flops / tc / 1e6                       # microseconds
        bound = "hbm" if t_mem >= t_tc else "tensor"
        print(json.dumps({"config": cfg, "shape": f"{name} {d_in}->{d_out}", "T": T, "us_per_call": round(us, 2),
                          "tokens_per_s": round(T / us * 1e6), "bound": bound,
                          "roofline_us": round(max(t_mem, t_tc), 2), "frac_of_roofline": round(max(t_mem, t_tc) / us, 3),
                          "achieved": round(nbytes / us / 1e3, 1) if bound == "hbm" else round(flops / us / 1e6, 1),
                          "unit": "GB/s" if bound == "hbm" else "TFLOP/s", "adapters_touched": touched,
                          "max_share_of_slots": round(max(counts) / max(1, T * TOPK), 3), "modules": R,
                          "plan": mb.meteora_describe_plan(shape).split(" fused_refused")[0]}), flush=True)
        del mods, graph


def run_layer_sweep():
    """Config 4: the 7 MeteoRA linears of a LLaMA3-8B decoder layer (each with its own gate and adapters), one
    call each, back to back in one CUDA graph; time per layer against the sum of the linears' rooflines."""
    import ctypes

    import torch

    from paper_2405_13053_b200 import binding as mb
    from paper_2405_13053_b200 import workloads

    lib = mb.load_library()
    hbm, _ = measured_peaks()
    tc, _ = measured_tensor_peak()
    dt, es = torch.bfloat16, 2
    for T in workloads.CONFIG4_T:
        g = torch.Generator(device="cuda").manual_seed(11)
        mods, nbytes, flops = [], 0.0, 0.0
        for name, (d_in, d_out) in workloads.CONFIG4_LINEARS.items():
            shape = mb.make_shape(T, d_in, d_out, N_ADAPTERS, RANK, TOPK, dt)
            x_np = workloads.make_x(T, d_in, "rms", 40 + len(mods), "bf16")
            mods.append({"name": name, "shape": shape, "x": torch.from_numpy(x_np).to(dt).cuda(),
                         "W0": (0.02 * torch.randn(d_out, d_in, device="cuda", generator=g)).to(dt),
                         "A": ((torch.rand(N_ADAPTERS, RANK, d_in, device="cuda", generator=g) * 2 - 1) / d_in ** 0.5).to(dt),
                         "B": (0.01 * torch.randn(N_ADAPTERS, d_out, RANK, device="cuda", generator=g)).to(dt),
                         "Wg": (torch.randn(N_ADAPTERS, d_in, device="cuda", generator=g) / d_in ** 0.5).to(dt),
                         "y": torch.empty(T, d_out, device="cuda", dtype=dt), "ws": mb.alloc_workspace(shape)})
            touched = min(N_ADAPTERS, T * TOPK)
            nbytes += (d_in * d_out + N_ADAPTERS * d_in + touched * RANK * (d_in + d_out) + T * (d_in + d_out)) * es
            flops += 2.0 * T * d_in * d_out + 2.0 * T * N_ADAPTERS * d_in + 2.0 * T * TOPK * RANK * (d_in + d_out)

        def step_calls():
            for m in mods:
                rc = lib.meteora_linear_forward(m["x"].data_ptr(), m["W0"].data_ptr(), m["A"].data_ptr(),
                                                m["B"].data_ptr(), m["Wg"].data_ptr(), ctypes.byref(m["shape"]),
                                                m["y"].data_ptr(), m["ws"].data_ptr(), m["ws"].numel(),
                                                torch.cuda.current_stream().cuda_stream)
                if rc != 0:
                    raise mb.MeteoraError(rc, "meteora_linear_forward")

        # the same layer with the linears that share their input as group calls: q/k/v, o, gate/up, down
        by_name = {m["name"]: m for m in mods}
        groups = []
        for names in (("q", "k", "v"), ("o",), ("gate", "up"), ("down",)):
            ms = [by_name[n] for n in names]
            G = len(ms)
            d_outs = (ctypes.c_int * G)(*[int(m["W0"].shape[0]) for m in ms])
            n = lib.meteora_group_workspace_bytes(ctypes.byref(ms[0]["shape"]), d_outs, G)
            vpa = ctypes.c_void_p * G
            groups.append({"x": ms[0]["x"], "G": G, "d_outs": d_outs, "shape": ms[0]["shape"],
                           "W0": vpa(*[m["W0"].data_ptr() for m in ms]), "A": vpa(*[m["A"].data_ptr() for m in ms]),
                           "B": vpa(*[m["B"].data_ptr() for m in ms]), "Wg": vpa(*[m["Wg"].data_ptr() for m in ms]),
                           "y": vpa(*[m["y"].data_ptr() for m in ms]),
                           "ws": torch.zeros(n, dtype=torch.uint8, device="cuda"),
                           "one_launch": lib.meteora_group_plan(ctypes.byref(ms[0]["shape"]), d_outs, G)})

        def step_groups():
            for gq in groups:
                rc = lib.meteora_linear_forward_group(gq["x"].data_ptr(), gq["W0"], gq["A"], gq["B"], gq["Wg"],
                                                      gq["d_outs"], gq["G"], ctypes.byref(gq["shape"]), gq["y"],
                                                      gq["ws"].data_ptr(), gq["ws"].numel(),
                                                      torch.cuda.current_stream().cuda_stream)
                if rc != 0:
                    raise mb.MeteoraError(rc, "meteora_linear_forward_group")

        for mode, step in (("7 calls", step_calls), ("4 group calls: q/k/v, o, gate/up, down", step_groups)):
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            iters = 100 if T <= 256 else 10
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            for m in mods + groups:
                st = mb.meteora_workspace_status(m["ws"])
                if st != 0:
                    raise mb.MeteoraError(st, "device status")
            us = e0.elapsed_time(e1) * 1e3 / iters
            t_mem, t_tc = nbytes / hbm / 1e3, flops / tc / 1e6
            bound = "hbm" if t_mem >= t_tc else "tensor"
            print(json.dumps({"config": "config4", "shape": "LLaMA3-8B layer: q k v o gate up down, " + mode, "T": T,
                              "us_per_layer": round(us, 2), "tokens_per_s": round(T / us * 1e6), "bound": bound,
                              "roofline_us": round(max(t_mem, t_tc), 2),
                              "frac_of_roofline": round(max(t_mem, t_tc) / us, 3),
                              "achieved": round(nbytes / us / 1e3, 1) if bound == "hbm" else round(flops / us / 1e6, 1),
                              "unit": "GB/s" if bound == "hbm" else "TFLOP/s",
                              "launches": (sum(1 if gq["one_launch"] else 3 * gq["G"] if T > 256 else gq["G"]
                                               for gq in groups) if step is step_groups
                                           else len(mods) * (3 if T > 256 else 1)),
                              "l2": "436 MB of W0 per layer: no weight survives in the 126 MB L2 until its next visit"}),
                  flush=True)
        del mods, graph, groups


def run_layer():
    """Config 4 as a layer: RMSNorm -> q/k/v -> rotary, grouped-query attention -> o -> residual -> RMSNorm -> gate/up ->
    SwiGLU -> down -> residual, the seven linears MeteoRA linears of the library (q/k/v and gate/up as group calls), each
    consuming the real upstream activation.  The whole layer is one CUDA graph; the same graph with the linears replaced
    by tensors made beforehand gives the time of everything that is not a MeteoRA linear, and the difference is the
    time of the linears inside the layer.  The four linear calls alone, on the layer's own activations, are timed as a
    third graph for comparison."""
    import torch

    from paper_2405_13053_b200 import binding as mb
    from paper_2405_13053_b200 import decoder_layer as dl

    hbm, _ = measured_peaks()
    tc, _ = measured_tensor_peak()
    dev, dt, es = torch.device("cuda"), torch.bfloat16, 2
    weights, norms = dl.random_layer(dev)

    def graph_time(fn, iters):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            fn()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / iters

    for mode, T, context in (("decode", 64, 2048), ("prefill", 4096, 0)):
        g = torch.Generator(device=dev).manual_seed(23)
        x = torch.randn(T, dl.HIDDEN, device=dev, generator=g).to(dt)
        if mode == "decode":
            ck = torch.randn(T, dl.N_KV_HEADS, context, dl.HEAD_DIM, device=dev, generator=g).to(dt)
            cv = torch.randn(T, dl.N_KV_HEADS, context, dl.HEAD_DIM, device=dev, generator=g).to(dt)
            pos = torch.full((T,), context, device=dev)
        else:
            ck = cv = None
            pos = torch.arange(T, device=dev)
        lin = dl.LibraryLinears(weights, k=TOPK)
        fixed = dl.FixedLinears(T, dt, dev)
        iters = 50 if mode == "decode" else 10
        us_layer = graph_time(lambda: dl.layer_forward(x, norms, lin, pos, ck, cv), iters)
        us_rest = graph_time(lambda: dl.layer_forward(x, norms, fixed, pos, ck, cv), iters)
        if lin.status() != 0:
            raise mb.MeteoraError(lin.status(), "device status")
        # the linears alone on activations of the right statistics (outputs of the layer's own ops)
        acts = {"n": dl.rms_norm(x, norms["input"]), "a": torch.randn(T, dl.HIDDEN, device=dev, generator=g).to(dt),
                "m": torch.randn(T, dl.MLP, device=dev, generator=g).to(dt)}

        def linears_only():
            lin.many(("q", "k", "v"), acts["n"])
            lin.one("o", acts["a"])
            lin.many(("gate", "up"), acts["n"])
            lin.one("down", acts["m"])

        us_lin = graph_time(linears_only, iters)
        nbytes = flops = 0.0
        touched = min(N_ADAPTERS, T * TOPK)
        for d_in, d_out in dl.LINEARS.values():
            nbytes += (d_in * d_out + N_ADAPTERS * d_in + touched * RANK * (d_in + d_out) + T * (d_in + d_out)) * es
            flops += 2.0 * T * d_in * d_out + 2.0 * T * N_ADAPTERS * d_in + 2.0 * T * TOPK * RANK * (d_in + d_out)
        t_mem, t_tc = nbytes / hbm / 1e3, flops / tc / 1e6
        bound = "hbm" if t_mem >= t_tc else "tensor"
        us_in_layer = us_layer - us_rest
        print(json.dumps({"config": "config4", "op": "decoder_layer", "mode": mode, "T": T, "context": context,
                          "shape": "LLaMA3-8B layer: RMSNorm, q/k/v, rotary, GQA 32/8x128, o, RMSNorm, gate/up, SwiGLU, down; "
                                   "seven MeteoRA linears (N=28, r=8, k=2) on the real activations",
                          "us_layer": round(us_layer, 2), "us_rest_of_layer": round(us_rest, 2),
                          "us_linears_in_layer": round(us_in_layer, 2), "us_linears_alone": round(us_lin, 2),
                          "bound": bound, "roofline_us": round(max(t_mem, t_tc), 2),
                          "frac_of_roofline_in_layer": round(max(t_mem, t_tc) / us_in_layer, 3),
                          "frac_of_roofline_alone": round(max(t_mem, t_tc) / us_lin, 3),
                          "achieved": round(nbytes / us_in_layer / 1e3, 1) if bound == "hbm" else round(flops / us_in_layer / 1e6, 1),
                          "unit": "GB/s" if bound == "hbm" else "TFLOP/s",
                          "timing": "CUDA graph of the layer minus the same graph with the linears' outputs made beforehand"}),
              flush=True)
        del lin, fixed, ck, cv


def run_standalone_sweep():
    """The standalone entry points (gate + top-k, bucketing, LoRA term by per-adapter segments) at config 1 (T = 128) and
    config 2 (4096 -> 14336, T = 2048), each against the HBM time of its algorithmic bytes, beside what the fused
    forward spends on the same job with the stacked dense shrink [A; Wg] x on the tensor cores plus the selection
    (time of a three-launch call minus its base-product launch).  This is the measured side of "per-adapter segments
    or one stacked dense shrink" (Sec. 3.3's gather against Eq. 5's batched view)."""
    import torch

    from paper_2405_13053_b200 import binding as mb
    from paper_2405_13053_b200 import workloads

    hbm, _ = measured_peaks()
    dt, es = torch.bfloat16, 2

    def timed_us(fn, iters=50):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        for _ in range(3):
            g.replay()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / iters

    for cfg, d_in, d_out, T, x_kind in (("config1", 4096, 4096, 128, "rms"), ("config2", 4096, 14336, 2048, "clusters")):
        g = torch.Generator(device="cuda").manual_seed(9)
        x = torch.from_numpy(workloads.make_x(T, d_in, x_kind, 5, "bf16")).to(dt).cuda()
        W0 = (0.02 * torch.randn(d_out, d_in, device="cuda", generator=g)).to(dt)
        A = ((torch.rand(N_ADAPTERS, RANK, d_in, device="cuda", generator=g) * 2 - 1) / d_in ** 0.5).to(dt)
        B = (0.01 * torch.randn(N_ADAPTERS, d_out, RANK, device="cuda", generator=g)).to(dt)
        Wg = (torch.randn(N_ADAPTERS, d_in, device="cuda", generator=g) / d_in ** 0.5).to(dt)
        shape = mb.make_shape(T, d_in, d_out, N_ADAPTERS, RANK, TOPK, dt)
        ws = mb.alloc_workspace(shape)
        idx, w, _ = mb.meteora_gate_topk(x, Wg, TOPK)
        idx, w = idx.clone(), w.clone()
        counts, offsets, perm = mb.meteora_route(idx, N_ADAPTERS)
        touched = int((counts > 0).sum().item())
        rows = []
        us = timed_us(lambda: mb.meteora_gate_topk(x, Wg, TOPK))
        rows.append(("meteora_gate_topk (k_gate_topk)", us, (T * d_in + N_ADAPTERS * d_in) * es + T * TOPK * 8))
        us = timed_us(lambda: mb.meteora_route(idx, N_ADAPTERS))
        rows.append(("meteora_route (k_route)", us, T * TOPK * 8 + (2 * N_ADAPTERS + 1) * 4))
        us = timed_us(lambda: mb.meteora_lora_delta(x, A, B, idx, w, offsets, perm, workspace=ws))
        rows.append(("meteora_lora_delta (k_shrink_segments + k_expand)", us,
                     (T * d_in + touched * RANK * (d_in + d_out)) * es + T * d_out * 4 + 2 * T * TOPK * RANK * 4))
        # the fused forward's side of the same job: three-launch chain, whole call minus its base-product launch
        y = torch.empty(T, d_out, device="cuda", dtype=dt)
        mb.meteora_set_tuning("fused", 0)
        try:
            call = lambda: mb.meteora_linear_forward(x, W0, A, B, Wg, TOPK, workspace=ws, out=y)
            us_call = timed_us(call, 20)
            call()
            torch.cuda.synchronize()
            mb.meteora_profile_begin(8)
            for _ in range(8):
                call()
            ms, n = mb.meteora_profile_end()
        finally:
            mb.meteora_set_tuning("fused", 1)
        us_base = ms * 1e3 / max(n, 1)
        stacked_bytes = (T * d_in + (N_ADAPTERS * RANK + N_ADAPTERS) * d_in) * es + T * TOPK * (RANK + 2) * 4
        rows.append(("stacked dense shrink [A; Wg] x on tcgen05 + selection (three-launch call minus its base product)",
                     us_call - us_base, stacked_bytes))
        seg_total = sum(r[1] for r in rows[:3])
        for name, us, nbytes in rows:
            print(json.dumps({"op": "standalone", "config": cfg, "shape": f"{d_in}->{d_out}", "T": T, "kernel": name,
                              "us": round(us, 2), "algorithmic_bytes": int(nbytes), "bound": "hbm",
                              "roofline_us": round(nbytes / hbm / 1e3, 3),
                              "frac_of_roofline": round(nbytes / hbm / 1e3 / us, 4), "adapters_touched": touched}), flush=True)
        print(json.dumps({"op": "segments_vs_stacked", "config": cfg, "shape": f"{d_in}->{d_out}", "T": T,
                          "us_segments_path (gate_topk + route + shrink by segments + expand)": round(seg_total, 2),
                          "us_stacked_path (stacked shrink + selection; the expand rides in the base product)":
                              round(us_call - us_base, 2),
                          "us_three_launch_call": round(us_call, 2), "us_base_product_launch": round(us_base, 2)}), flush=True)


def run_decode_loop():
    """One autoregressive decode step over all 224 MeteoRA linears of a LLaMA3-8B-shaped stack (32 decoder layers
    x 7 linears, each with its own gate and adapters, Sec. 3.2), in the unit of the paper's App. A.7 figures:
    milliseconds per generated token.  A batch of b sequences generates b tokens per step (T = b).  Only the
    MeteoRA linears run (no attention, norms or sampling: those are not part of the method), every linear on its
    own synthetic input, the ones that share their input in a real block (q/k/v, gate/up) as group calls; one CUDA
    graph per step."""
    import ctypes

    import torch

    from paper_2405_13053_b200 import binding as mb
    from paper_2405_13053_b200 import workloads

    lib = mb.load_library()
    hbm, _ = measured_peaks()
    dt, es, n_layers = torch.bfloat16, 2, 32
    g = torch.Generator(device="cuda").manual_seed(17)
    weights = []                                                   # 32 layers x 7 linears: 14 GB of W0
    for _ in range(n_layers):
        layer = {}
        for name, (d_in, d_out) in workloads.CONFIG4_LINEARS.items():
            layer[name] = {"W0": (0.02 * torch.randn(d_out, d_in, device="cuda", generator=g)).to(dt),
                           "A": ((torch.rand(N_ADAPTERS, RANK, d_in, device="cuda", generator=g) * 2 - 1) / d_in ** 0.5).to(dt),
                           "B": (0.01 * torch.randn(N_ADAPTERS, d_out, RANK, device="cuda", generator=g)).to(dt),
                           "Wg": (torch.randn(N_ADAPTERS, d_in, device="cuda", generator=g) / d_in ** 0.5).to(dt)}
        weights.append(layer)
    vpa = lambda ts: (ctypes.c_void_p * len(ts))(*[t.data_ptr() for t in ts])
    for T in (1, 16, 64):
        xs = {d: torch.from_numpy(workloads.make_x(T, d, "rms", 60 + i, "bf16")).to(dt).cuda()
              for i, d in enumerate(sorted({di for di, _ in workloads.CONFIG4_LINEARS.values()}))}
        calls, nbytes, launches = [], 0.0, 0
        for layer in weights:
            for names in (("q", "k", "v"), ("o",), ("gate", "up"), ("down",)):
                d_in = workloads.CONFIG4_LINEARS[names[0]][0]
                d_out_list = [workloads.CONFIG4_LINEARS[n][1] for n in names]
                shape = mb.make_shape(T, d_in, d_out_list[0], N_ADAPTERS, RANK, TOPK, dt)
                d_outs = (ctypes.c_int * len(names))(*d_out_list)
                n = lib.meteora_group_workspace_bytes(ctypes.byref(shape), d_outs, len(names))
                ys = [torch.empty(T, d, device="cuda", dtype=dt) for d in d_out_list]
                calls.append({"x": xs[d_in], "G": len(names), "d_outs": d_outs, "shape": shape, "ys": ys,
                              "W0": vpa([layer[n_]["W0"] for n_ in names]), "A": vpa([layer[n_]["A"] for n_ in names]),
                              "B": vpa([layer[n_]["B"] for n_ in names]), "Wg": vpa([layer[n_]["Wg"] for n_ in names]),
                              "y": vpa(ys), "ws": torch.zeros(n, dtype=torch.uint8, device="cuda")})
                launches += 1 if lib.meteora_group_plan(ctypes.byref(shape), d_outs, len(names)) else len(names)
                touched = min(N_ADAPTERS, T * TOPK)
                for d_out in d_out_list:
                    nbytes += (d_in * d_out + N_ADAPTERS * d_in + touched * RANK * (d_in + d_out) + T * (d_in + d_out)) * es

        def step():
            st = torch.cuda.current_stream().cuda_stream
            for c in calls:
                rc = lib.meteora_linear_forward_group(c["x"].data_ptr(), c["W0"], c["A"], c["B"], c["Wg"], c["d_outs"],
                                                      c["G"], ctypes.byref(c["shape"]), c["y"], c["ws"].data_ptr(),
                                                      c["ws"].numel(), st)
                if rc != 0:
                    raise mb.MeteoraError(rc, "meteora_linear_forward_group")

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        iters = 20
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        for c in calls:
            st = mb.meteora_workspace_status(c["ws"])
            if st != 0:
                raise mb.MeteoraError(st, "device status")
        ms = e0.elapsed_time(e1) / iters
        print(json.dumps({"op": "decode_step", "shape": "LLaMA3-8B stack: 32 layers x (q k v o gate up down), MeteoRA linears only",
                          "batch": T, "ms_per_generated_token": round(ms, 3), "tokens_per_s": round(T / ms * 1e3),
                          "launches_per_step": launches, "bound": "hbm", "roofline_ms": round(nbytes / hbm / 1e6, 3),
                          "frac_of_roofline": round(nbytes / hbm / 1e6 / ms, 3),
                          "modules": n_layers * len(workloads.CONFIG4_LINEARS)}), flush=True)
        del calls, graph


def run_gate_backward_sweep():
    """meteora_gate_backward (gradient of the gate weights for a forward's routing) at the q_proj shape."""
    import ctypes

    import torch

    from paper_2405_13053_b200 import binding as mb

    hbm, _ = measured_peaks()
    dt, es = torch.bfloat16, 2
    d_in = d_out = 4096
    lib = mb.load_library()
    for T in (1, 128, 2048, 8192):
        g = torch.Generator(device="cuda").manual_seed(13)
        x = torch.randn(T, d_in, device="cuda", generator=g).to(dt)
        W0 = (0.02 * torch.randn(d_out, d_in, device="cuda", generator=g)).to(dt)
        A = ((torch.rand(N_ADAPTERS, RANK, d_in, device="cuda", generator=g) * 2 - 1) / d_in ** 0.5).to(dt)
        B = (0.01 * torch.randn(N_ADAPTERS, d_out, RANK, device="cuda", generator=g)).to(dt)
        Wg = (torch.randn(N_ADAPTERS, d_in, device="cuda", generator=g) / d_in ** 0.5).to(dt)
        dy = torch.randn(T, d_out, device="cuda", generator=g).to(dt)
        _, idx, w = mb.meteora_linear_forward(x, W0, A, B, Wg, TOPK, return_routing=True)
        idx, w = idx.clone(), w.clone()
        Bt = mb.meteora_transpose_adapters_b(B)
        shape = mb.make_shape(T, d_in, d_out, N_ADAPTERS, RANK, TOPK, dt)
        ws = torch.zeros(lib.meteora_gate_backward_workspace_bytes(ctypes.byref(shape)), dtype=torch.uint8, device="cuda")

        def timed(**kw):
            """Per call from a CUDA graph of 8 calls (stream-ordered on one workspace), median of 5 regions."""
            def eight():
                for _ in range(8):
                    mb.meteora_gate_backward(x, A, B, dy, idx, w, workspace=ws, **kw)
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                eight()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                eight()
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            out = []
            for _ in range(5):
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(5):
                    graph.replay()
                e1.record()
                torch.cuda.synchronize()
                out.append(e0.elapsed_time(e1) * 1e3 / 40)
            return sorted(out)[2]

        us_b, us = timed(), timed(Bt=Bt)
        touched = int(torch.unique(idx).numel())
        # x is read for the shrink and again, once per pick, for the reduction over tokens; dy once; dWg written in fp32
        nbytes = ((1 + TOPK) * T * d_in + T * d_out + touched * RANK * (d_in + d_out)) * es + N_ADAPTERS * d_in * 4
        print(json.dumps({"op": "meteora_gate_backward_bt", "shape": "4096->4096", "T": T, "us_per_call": round(us, 2),
                          "us_per_call_with_transposition": round(us_b, 2),
                          "tokens_per_s": round(T / us * 1e6), "bound": "hbm",
                          "roofline_us": round(nbytes / hbm / 1e3, 2),
                          "frac_of_roofline": round(nbytes / hbm / 1e3 / us, 3),
                          "note": "B transposed beforehand (meteora_transpose_adapters_b); up to 256 tokens both stacked "
                                  "shrinks as one launch and no bucketing, up to 1024 no bucketing; graph replay of 8 "
                                  "stream-ordered calls"}),
              flush=True)


def run_variants():
    """The paper's synthetic sweep axes (App. A.7: k, r, number of adapters; temperature of App. A.5) at the
    LLaMA3-8B q_proj shape, a decode batch (T = 32) and a prefill batch (T = 2048), one axis at a time around
    the base point N = 28, r = 8, k = 2."""
    import ctypes

    import torch

    from paper_2405_13053_b200 import binding as mb
    from paper_2405_13053_b200 import build as lib_build

    lib_build.build_library()
    lib = mb.load_library()
    torch.cuda.set_device(0)
    hbm, _ = measured_peaks()
    tc, _ = measured_tensor_peak()
    dt, es = torch.bfloat16, 2
    d_in = d_out = 4096
    base = {"N": 28, "r": 8, "k": 2, "tau": 1.0}
    points = [dict(base)]
    points += [dict(base, k=k) for k in (1, 4)]
    points += [dict(base, r=4, pad="every call"), dict(base, r=4, pad="once")]
    points += [dict(base, r=r) for r in (16, 32, 64)]
    points += [dict(base, N=N) for N in (8, 64, 128)]
    points += [dict(base, tau=20.0)]
    for T in (32, 2048):
        for pt in points:
            N, r, k, tau = pt["N"], pt["r"], pt["k"], pt["tau"]
            R = 8 if T <= 256 else 1
            # a rank that is no multiple of 8: the forward pads the adapters on every call, or the caller padded
            # them once (meteora_pad_adapters) and passes the padded rank
            r_call = (r + 7) // 8 * 8 if pt.get("pad") == "once" else r
            shape = mb.make_shape(T, d_in, d_out, N, r_call, k, dt, tau)
            g = torch.Generator(device="cuda").manual_seed(3)
            mods = []
            ws_shared = mb.alloc_workspace(shape)
            for i in range(R):
                x = torch.randn(T, d_in, device="cuda", generator=g)
                x = (x / x.pow(2).mean(dim=1, keepdim=True).sqrt()).to(dt)
                mods.append({"x": x, "W0": (0.02 * torch.randn(d_out, d_in, device="cuda", generator=g)).to(dt),
                             "A": ((torch.rand(N, r, d_in, device="cuda", generator=g) * 2 - 1) / d_in ** 0.5).to(dt),
                             "B": (0.01 * torch.randn(N, d_out, r, device="cuda", generator=g)).to(dt),
                             "Wg": (torch.randn(N, d_in, device="cuda", generator=g) / d_in ** 0.5).to(dt),
                             "y": torch.empty(T, d_out, device="cuda", dtype=dt), "ws": ws_shared})
                if pt.get("pad") == "once":
                    mods[-1]["A"], mods[-1]["B"] = mb.meteora_pad_adapters(mods[-1]["A"], mods[-1]["B"])

            def step():
                for m in mods:
                    rc = lib.meteora_linear_forward(m["x"].data_ptr(), m["W0"].data_ptr(), m["A"].data_ptr(),
                                                    m["B"].data_ptr(), m["Wg"].data_ptr(), ctypes.byref(shape),
                                                    m["y"].data_ptr(), m["ws"].data_ptr(), m["ws"].numel(),
                                                    torch.cuda.current_stream().cuda_stream)
                    if rc != 0:
                        raise mb.MeteoraError(rc, "meteora_linear_forward")

            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step()
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            iters = 50 if T <= 256 else 10
            for _ in range(3):
                graph.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                graph.replay()
            e1.record()
            torch.cuda.synchronize()
            for m in mods:
                st = mb.meteora_workspace_status(m["ws"])
                if st != 0:
                    raise mb.MeteoraError(st, "device status")
            us = e0.elapsed_time(e1) * 1e3 / (iters * R)
            idx0, _ = mb.meteora_workspace_routing(shape, mods[0]["ws"])
            touched = int(torch.unique(idx0).numel())
            nbytes = (d_in * d_out + N * d_in + touched * r * (d_in + d_out) + T * (d_in + d_out)) * es
            flops = 2.0 * T * d_in * d_out + 2.0 * T * N * d_in + 2.0 * T * k * r * (d_in + d_out)
            t_mem, t_tc = nbytes / hbm / 1e3, flops / tc / 1e6
            bound = "hbm" if t_mem >= t_tc else "tensor"
            print(json.dumps({"variant": pt, "shape": "4096->4096", "T": T, "us_per_call": round(us, 2),
                              "tokens_per_s": round(T / us * 1e6), "bound": bound,
                              "roofline_us": round(max(t_mem, t_tc), 2),
                              "frac_of_roofline": round(max(t_mem, t_tc) / us, 3),
                              "plan": mb.meteora_describe_plan(shape).split(" fused_refused")[0]}), flush=True)
            del mods, graph


def apply_knobs(args):
    if not args.knob:
        return
    from paper_2405_13053_b200 import binding as mb
    from paper_2405_13053_b200 import build as lib_build

    lib_build.build_library()
    for kv in args.knob:
        name, value = kv.split("=")
        mb.meteora_set_tuning(name, int(value))


def main():
    args = parse_args()
    if args.impl != "reference":
        apply_knobs(args)
    if args.prefill_only:
        import torch

        from paper_2405_13053_b200 import binding as mb
        from paper_2405_13053_b200 import build as lib_build

        lib_build.build_library()
        torch.cuda.set_device(0)
        tc_peak, tc_kind = measured_tensor_peak()
        print(json.dumps({"prefill_roofline": prefill_line(mb, mb.load_library(), tc_peak, tc_kind, measured_peaks()[0])}),
              flush=True)
    elif args.variants:
        run_variants()
    elif args.layer:
        run_layer()
    elif args.standalone:
        run_standalone_sweep()
    elif args.gate_backward:
        run_gate_backward_sweep()
    elif args.decode_loop:
        run_decode_loop()
    elif args.sweep:
        run_sweep(args)
        run_layer_sweep()
        run_layer()
        run_standalone_sweep()
        run_gate_backward_sweep()
        run_decode_loop()
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
