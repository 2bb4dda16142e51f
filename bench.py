#!/usr/bin/env python
"""Benchmark of the BitLinear forward hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One step = one BitLinear forward (LN + absmax quantisation, 1-bit x 8-bit matmul, rescale; Eq. 11)
over the prefill batch: x bf16 [8192, 4096], W [4096, 4096] binarised and packed beforehand,
per-tensor gamma, y bf16.  The headline value is the layer's integer throughput, 2*M*N*K / step
time.  The same JSON line also carries the other rows of the path, each measured on its own
workload: the batch-1 decode GEMV (K = 4096, N = 16384, 1000 calls in one CUDA graph rotating
over 64 packed weight buffers), the LN+quant kernels and the binarise+pack kernels.

Every rank runs the same replica on its own GPU (the layer has no exchange step); the job's
value is the sum over ranks divided by the slowest rank's time.
"""
import argparse
import hashlib
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "BitLinear prefill int8 TOPS + decode GEMV GB/s, % of B200 roofline"
PREFILL = dict(M=8192, K=4096, N=4096, G=1)          # batch 4 x seq 2048, 6.7B-shaped projection
DECODE = dict(K=4096, N=16384, calls=1000, buffers=64)
ROTATE = 3                                           # distinct input/output sets per workload
NOMINAL_INT8_TOPS = 4500.0
NOMINAL_HBM_GBS = 8000.0
INT8_TO_BF16 = 2.0                                   # nominal dense int8 : bf16 tensor rate
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the summaries under
# profiles/, taken with ncu on these same workloads.  A figure is valid only while its kernel is the
# one that was profiled: set it to None when the kernel changes, until the capture is redone.
NCU_TRAFFIC = {
    "gemm_tc2_kernel": 70.6e6,                       # 37.1 MB read + 33.5 MB written (half of y still in L2)
    "rows_tensor_fused": 70.9e6,                     # 67.2 MB read + 3.7 MB written (second pass from smem and L2)
    "gemv_decode_fast_kernel": 8.43e6,
    "reduce_partials + sign_pack_rows": 70.1e6,      # first pass 66.3 MB read, second pass served from L2
                                                     # (capture without cache flushes between the launches)
}


def load_peaks():
    """Measured denominators (copy bandwidth, bf16 GEMM) or the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index, period_s=0.0002):
        self.index, self.period, self.samples, self.reasons = index, period_s, [], set()
        self.max_mhz, self._stop, self._thread, self._h, self._nv = None, threading.Event(), None, None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            uuid = torch.cuda.get_device_properties(index).uuid
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _names(self, mask):
        nv = self._nv
        table = [("hw_slowdown", "nvmlClocksEventReasonHwSlowdown", 0x8),
                 ("hw_thermal_slowdown", "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
                 ("sw_thermal_slowdown", "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
                 ("sw_power_cap", "nvmlClocksEventReasonSwPowerCap", 0x4),
                 ("hw_power_brake", "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80)]
        return {name for name, attr, default in table if mask & getattr(nv, attr, default)}

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                self.reasons |= self._names(mask)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return self._smi_once()
        return dict(sm_mhz=statistics.median(self.samples), sm_max_mhz=self.max_mhz,
                    reasons=sorted(self.reasons), samples=len(self.samples), source="nvml")

    def _smi_once(self):
        try:
            out = subprocess.check_output(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=clocks.sm,clocks.max.sm",
                 "--format=csv,noheader,nounits"], timeout=10).decode().split(",")
            return dict(sm_mhz=float(out[0]), sm_max_mhz=float(out[1]), reasons=[], samples=1,
                        source="nvidia-smi after the run")
        except Exception:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0, source="unavailable")


def job_throughput(units_local, ms_local, dist=None, device=None):
    """Whole-job rate of replicas that each processed `units_local` units in `ms_local` ms: the sum
    of the units over the ranks divided by the slowest rank's time.  Returns (units per second,
    max ms).  `dist` is torch.distributed (any backend) or None for one process."""
    if dist is None:
        return units_local / (ms_local * 1e-3), ms_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(u.item()) / (float(t.item()) * 1e-3), float(t.item())


def sha256_of(t):
    """SHA-256 of a host tensor's bytes (inputs are logged by hash so that a run can be reproduced)."""
    return hashlib.sha256(t.contiguous().view(torch.uint8).numpy().tobytes()).hexdigest()


def library_int8_tops(M, K, N, dev, reps=20):
    """In-job calibration of the box: the library int8 GEMM (torch._int_mm, int32 output) on the bench
    shape, timed alone with CUDA events.  None when the routine is unavailable."""
    try:
        a = torch.randint(-127, 128, (M, K), dtype=torch.int8, device=dev)
        b = torch.randint(-1, 2, (K, N), dtype=torch.int8, device=dev)
        for _ in range(3):
            torch._int_mm(a, b)
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        t0.record()
        for _ in range(reps):
            torch._int_mm(a, b)
        t1.record()
        torch.cuda.synchronize()
        return 2.0 * M * N * K / (t0.elapsed_time(t1) / reps * 1e-3) / 1e12
    except Exception:
        return None


def measured_copy_gbs(dev, nbytes=1 << 30, reps=5):
    """In-job device-to-device copy rate (read + write bytes), the same kind of figure as the measured peak."""
    a = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    b = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    b.copy_(a)
    best = None
    for _ in range(reps):
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record()
        b.copy_(a)
        t1.record()
        torch.cuda.synchronize()
        ms = t0.elapsed_time(t1)
        best = ms if best is None else min(best, ms)
    return 2.0 * nbytes / (best * 1e-3) / 1e9


# --------------------------------------------------------------------------------------- own arm

def run_b200(args):
    from paper_2310_11453_b200 import binding as B
    from paper_2310_11453_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the BitLinear library has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    B.lib()                                           # fail here, loudly, if the library is missing
    peaks = load_peaks()
    run_clocks = ClockSampler(local, period_s=0.01)   # across every part of the run
    run_clocks.__enter__()
    K_steps, W_steps = args.steps, max(args.warmup, 3)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- prefill workload: inputs resident in HBM, ROTATE distinct sets (> L2 in total) ----------
    M, K, N, G = PREFILL["M"], PREFILL["K"], PREFILL["N"], PREFILL["G"]
    xs_host = [synth.make_x(M, K, torch.bfloat16, seed=2 + 101 * r + 7919 * rank, outliers=True).pin_memory()
               for r in range(ROTATE)]
    xs = [x.to(dev) for x in xs_host]
    W_host = synth.make_w(N, K, torch.float32, seed=2)
    hashes = {f"x[{r}] bf16 [{M},{K}]": sha256_of(x) for r, x in enumerate(xs_host)}
    hashes[f"W fp32 [{N},{K}]"] = sha256_of(W_host)
    W = W_host.to(dev)
    w = B.binarize_pack(W, G=G, layout=B.PREFILL)
    ys = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _ in range(ROTATE)]
    qs = [dict(x_q=torch.empty((M, K), dtype=torch.int8, device=dev),
               gamma=torch.empty(G, dtype=torch.float32, device=dev),
               eta=torch.zeros(G, dtype=torch.float32, device=dev)) for _ in range(ROTATE)]
    ws_q = torch.empty(B.workspace_bytes(B.OP_QUANT_ACT, M, 1, K, G), dtype=torch.uint8, device=dev)
    ws_g = torch.empty(B.workspace_bytes(B.OP_MATMUL_DEQUANT, M, N, K, G), dtype=torch.uint8, device=dev)
    ws_f = torch.empty(B.workspace_bytes(B.OP_FORWARD, M, N, K, G), dtype=torch.uint8, device=dev)

    def step(i, ev=None):
        r = i % ROTATE
        if ev is not None:
            ev[0].record()
        B.quant_act(xs[r], G=G, mode=B.ABSMAX, gran=B.PER_TENSOR, out=qs[r], ws=ws_q)
        if ev is not None:
            ev[1].record()
        B.matmul_dequant(qs[r]["x_q"], qs[r]["gamma"], w["W_packed"], w["beta"], N, G=G, gran=B.PER_TENSOR,
                         layout=B.PREFILL, y=ys[r], ws=ws_g)
        if ev is not None:
            ev[2].record()

    for i in range(W_steps):
        step(i)
    assert B.ws_status(ws_g) == B.OK, "tensor-core GEMM reported a device-side timeout"
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K_steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    # The stream must not run dry at the start of the timed region: after the barrier the GPU is
    # idle and the first steps would be timed with the host's launch latency inside them.  A fill
    # of a buffer larger than L2 (which also leaves L2 cold) keeps the GPU busy while the host
    # queues the first steps; t0 is recorded behind it.
    head_start = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    with ClockSampler(local) as clocks:
        head_start.zero_()
        head_start.zero_()
        t0.record()
        for i in range(K_steps):
            step(i, evs[i])
        t1.record()
        barrier()
    ops_per_step = 2.0 * M * N * K
    job_ops_per_s, total_ms = job_throughput(ops_per_step * K_steps, t0.elapsed_time(t1), dist, dev)
    assert B.ws_status(ws_g) == B.OK
    ms_per_step = total_ms / K_steps
    value = job_ops_per_s / 1e12
    gemm_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in evs)
    quant_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in evs)
    gemm_tops = ops_per_step / (gemm_ms * 1e-3) / 1e12
    tensor_peak = INT8_TO_BF16 * peaks["bf16_tflops"]
    quant_bytes = 2.0 * M * K * 2 + M * K                      # per-tensor: x read twice, codes written
    quant_gbs = quant_bytes / (quant_ms * 1e-3) / 1e9

    # ---- end to end through the public call, host buffers, copies inside the timed region -------
    # Every step copies its x from pinned host memory and its y back to pinned host memory.  Serial:
    # copy in, forward, copy out on one stream.  Pipelined (the reported value): two buffer sets and
    # three streams, so the copy-in of step i+1 and the copy-out of step i-1 run beside the forward of
    # step i, each step still moving all of its own bytes.
    x_dev = [torch.empty((M, K), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    y_dev = [torch.empty((M, N), dtype=torch.bfloat16, device=dev) for _ in range(2)]
    y_host = [torch.empty((M, N), dtype=torch.bfloat16).pin_memory() for _ in range(2)]

    def fwd(b):
        B.forward(x_dev[b], w["W_packed"], w["beta"], N, G=G, mode=B.ABSMAX, gran=B.PER_TENSOR,
                  layout=B.PREFILL, y=y_dev[b], ws=ws_f)

    def e2e_serial(i):
        x_dev[0].copy_(xs_host[i % ROTATE], non_blocking=True)
        fwd(0)
        y_host[0].copy_(y_dev[0], non_blocking=True)

    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
    in_done = [torch.cuda.Event() for _ in range(2)]
    fwd_done = [torch.cuda.Event() for _ in range(2)]
    out_done = [torch.cuda.Event() for _ in range(2)]

    def e2e_pipelined(i):
        b = i & 1
        with torch.cuda.stream(s_in):
            s_in.wait_event(fwd_done[b])                 # x_dev[b] was last read by step i-2
            x_dev[b].copy_(xs_host[i % ROTATE], non_blocking=True)
            in_done[b].record(s_in)
        main.wait_event(in_done[b])
        main.wait_event(out_done[b])                     # y_dev[b] was last copied out by step i-2
        fwd(b)
        fwd_done[b].record(main)
        with torch.cuda.stream(s_out):
            s_out.wait_event(fwd_done[b])
            y_host[b].copy_(y_dev[b], non_blocking=True)
            out_done[b].record(s_out)

    def join():
        for st in (s_in, s_out):
            e = torch.cuda.Event()
            e.record(st)
            main.wait_event(e)

    e2e_steps = min(K_steps, 100)

    def run_e2e(step_fn):
        for i in range(4):
            step_fn(i)
        join()
        barrier()
        t0.record()
        for i in range(e2e_steps):
            step_fn(i)
        join()
        t1.record()
        barrier()
        return job_throughput(ops_per_step * e2e_steps, t0.elapsed_time(t1), dist, dev)

    _, serial_total = run_e2e(e2e_serial)
    e2e_ops_per_s, e2e_total = run_e2e(e2e_pipelined)
    assert B.ws_status(ws_f) == B.OK
    e2e_ms = e2e_total / e2e_steps
    e2e = dict(value=e2e_ops_per_s / 1e12, unit="TOPS", ms_per_step=e2e_ms,
               serial_ms_per_step=serial_total / e2e_steps,
               h2d_bytes_per_step=M * K * 2, d2h_bytes_per_step=M * N * 2,
               call="bitlinear_forward on device copies of pinned host x; y copied back to pinned host; "
                    "copy-in of step i+1 and copy-out of step i-1 overlap the forward of step i "
                    "(serial_ms_per_step: the three in sequence on one stream)")

    line = {
        "metric": METRIC, "value": value, "unit": "TOPS", "n_gpus": world, "steps": K_steps,
        "warmup": W_steps, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8 x 1-bit -> int32, fp32 rescale", "data": "synthetic",
        "config": {"workload": "prefill BitLinear forward: x bf16 [8192,4096] N(0,1) + 0.1% x20 outliers, "
                               "W [4096,4096] N(0,0.02) binarised+packed beforehand, b=8, per-tensor gamma, "
                               "y bf16",
                   "M": M, "K": K, "N": N, "G": G, "parallelism": "replicas only" if world > 1 else "1 GPU",
                   "l2": f"rotating over {ROTATE} input/output sets, {ROTATE * (M * K * 3 + M * N * 2) >> 20} MiB "
                         "in total, larger than L2"},
        "clocks": None,
        "inputs_sha256": hashes,
        "e2e": e2e,
        "gpu_launches": 2 * K_steps,
        "kernels_per_step": ["rows_tensor_fused", "gemm_tc2_kernel"],
        "roofline": {"bound": "tensor", "kernel": "gemm_tc2_kernel", "achieved": gemm_tops, "peak": tensor_peak,
                     "unit": "TFLOP/s", "frac": gemm_tops / tensor_peak, "traffic": NCU_TRAFFIC["gemm_tc2_kernel"],
                     "op_kind": "int8 (s8 x s8 -> s32), 2 ops per multiply-accumulate",
                     "peak_source": f"{peaks['source']} bf16 burst {peaks['bf16_tflops']} x {INT8_TO_BF16} "
                                    "(nominal int8:bf16 ratio)",
                     "frac_of_nominal": gemm_tops / NOMINAL_INT8_TOPS, "avg_launch_ms": gemm_ms},
        "roofline_quant": {"bound": "hbm", "kernel": "rows_tensor_fused", "achieved": quant_gbs,
                           "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": quant_gbs / peaks["hbm_gbs"],
                           "traffic": NCU_TRAFFIC["rows_tensor_fused"], "avg_ms": quant_ms, "peak_source": peaks["source"] + " copy"},
    }

    parts = set(args.parts.split(","))
    lib_tops = library_int8_tops(M, K, N, dev) if rank == 0 and "calib" in parts else None
    if lib_tops:
        line["roofline"]["library_int8_tops"] = lib_tops
        line["roofline"]["frac_of_library_int8"] = gemm_tops / lib_tops
        line["roofline"]["library_int8"] = "torch._int_mm on the same shape, int32 output, timed in this job"
    if rank == 0 and "calib" in parts:
        line["copy_gbs_in_job"] = measured_copy_gbs(dev)
    if rank == 0 and world == 1:
        if "decode" in parts:
            line["decode"] = bench_decode(B, synth, dev, peaks)
        if "pack" in parts:
            line["pack"] = bench_pack(B, synth, dev, peaks)
        if "block" in parts:
            line["block"] = bench_block(B, synth, dev, peaks)
        if "grouped" in parts:
            line["grouped"] = bench_grouped(B, synth, dev, peaks)
        if "small" in parts:
            line["small"] = bench_small(B, synth, dev)
        if "cpu" in parts:
            line["cpu_baseline"] = cpu_baseline_prefill(xs_host[0], W.cpu())
            line["cpu_baseline_decode"] = cpu_baseline_decode()
            line["cpu_baseline_grouped"] = cpu_baseline_grouped()
    line["clocks"] = clocks.summary()
    run_clocks.__exit__()
    line["clocks_whole_run"] = run_clocks.summary()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def bench_decode(B, synth, dev, peaks):
    """Batch-1 decode: 1000 GEMV calls in one CUDA graph, rotating over 64 packed weight buffers
    (512 MiB, so every call streams its weights from HBM) with a fresh x per call."""
    K, N, calls, nbuf = DECODE["K"], DECODE["N"], DECODE["calls"], DECODE["buffers"]
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    packs = []
    for _ in range(nbuf):
        Wd = torch.randn((N, K), generator=gen, device=dev, dtype=torch.float32) * synth.W_STD
        packs.append(B.binarize_pack(Wd, layout=B.DECODE, want_rowsum=False))
        del Wd
    torch.cuda.synchronize()                             # decode reads its weights ahead of stream order
    x = synth.make_x(calls, K, torch.float16, seed=1, outliers=False).to(dev)
    y = torch.empty((calls, N), dtype=torch.float16, device=dev)

    side = [torch.cuda.Stream(device=dev) for _ in range(3)]

    def issue(n_bufs, n_streams=1):
        """Issues the 1000 calls; with n_streams > 1 call i goes to stream i % n_streams, so calls on
        different streams are independent of one another (each stream keeps its own order)."""
        main = torch.cuda.current_stream()
        lanes = [main] + side[:n_streams - 1]
        if n_streams > 1:
            fork = torch.cuda.Event()
            fork.record(main)
            for st in lanes[1:]:
                st.wait_event(fork)
        for i in range(calls):
            p = packs[i % n_bufs]
            with torch.cuda.stream(lanes[i % n_streams]):
                B.gemv_decode(x[i], p["W_packed"], p["beta"], N, y=y[i])
        for st in lanes[1:]:
            join = torch.cuda.Event()
            join.record(st)
            main.wait_event(join)

    issue(nbuf)
    torch.cuda.synchronize()
    out = {}
    for name, n_bufs, n_streams in (("hbm", nbuf, 1), ("hbm_2streams", nbuf, 2), ("hbm_4streams", nbuf, 4),
                                    ("l2_hot", 1, 1)):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            issue(n_bufs, n_streams)
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        times = []
        for _ in range(10):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            graph.replay()
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        out[name] = statistics.median(times) / calls * 1e3       # us per call
        del graph
    bytes_per_call = N * K / 8 + 2 * K + 2 * N
    gbs = bytes_per_call / (out["hbm"] * 1e-6) / 1e9

    # small batches through bitlinear_gemv_decode_batch: M tokens share one pass over the weights
    batch, batch_ws = {}, {}
    bcalls = 400
    yb = torch.empty((32, N), dtype=torch.float16, device=dev)
    wsb = torch.empty(B.workspace_bytes(B.OP_GEMV_DECODE_BATCH, 32, N, K, 1), dtype=torch.uint8, device=dev)
    for Mb, with_ws in ((1, False), (2, False), (4, False), (8, False), (16, False),
                        (2, True), (4, True), (8, True), (16, True), (32, True)):
        def issue_batch():
            for i in range(bcalls):
                p = packs[i % nbuf]
                r0 = (i * Mb) % (calls - Mb)
                if with_ws:
                    B.gemv_decode_batch_ws(x[r0:r0 + Mb], p["W_packed"], p["beta"], N, y=yb[:Mb], ws=wsb)
                else:
                    B.gemv_decode_batch(x[r0:r0 + Mb], p["W_packed"], p["beta"], N, y=yb[:Mb])
        issue_batch()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            issue_batch()
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        times = []
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            graph.replay()
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        us = statistics.median(times) / bcalls * 1e3
        (batch_ws if with_ws else batch)[f"M{Mb}"] = {"us_per_call": us, "us_per_token": us / Mb,
                                                      "weight_gbs": (N * K / 8 + Mb * 2 * (K + N)) / (us * 1e-6) / 1e9}
        del graph
    if B.ws_status(wsb) != B.OK:
        raise RuntimeError("a bounded wait of the tensor-core decode kernel ran out during the bench")

    # the same call on projection shapes of the larger models of the paper's Table 1 sizes
    del packs, y, yb
    other = {}
    ocalls = 200
    for label, Ko, No in (("6.7B FFN down", 16384, 4096), ("13B FFN up", 5120, 20480), ("30B attention", 7168, 7168)):
        obufs = -(-(256 << 20) // (No * Ko // 8))            # 256 MiB of packed weights in rotation
        opacks = []
        for _ in range(obufs):
            Wd = torch.randn((No, Ko), generator=gen, device=dev, dtype=torch.float32) * synth.W_STD
            opacks.append(B.binarize_pack(Wd, layout=B.DECODE, want_rowsum=False))
            del Wd
        torch.cuda.synchronize()
        xo = synth.make_x(ocalls, Ko, torch.float16, seed=3, outliers=False).to(dev)
        yo = torch.empty((ocalls, No), dtype=torch.float16, device=dev)

        def issue_other():
            for i in range(ocalls):
                p = opacks[i % obufs]
                B.gemv_decode(xo[i], p["W_packed"], p["beta"], No, y=yo[i])
        issue_other()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            issue_other()
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        times = []
        for _ in range(5):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            graph.replay()
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        us = statistics.median(times) / ocalls * 1e3
        ob = No * Ko / 8 + 2 * Ko + 2 * No
        other[label] = {"K": Ko, "N": No, "us_per_call": us, "gbs": ob / (us * 1e-6) / 1e9,
                        "frac": ob / (us * 1e-6) / 1e9 / peaks["hbm_gbs"]}
        del graph, opacks, xo, yo
    fallbacks = B.debug_decode_fallbacks()

    def rate(us):
        return bytes_per_call / (us * 1e-6) / 1e9

    return {"workload": "decode GEMV: x fp16 [1,4096], packed 1-bit W K=4096 N=16384, y fp16; 1000 calls in one "
                        "CUDA graph over 64 weight buffers (512 MiB > L2), fresh x per call, one stream "
                        "(every call ordered after the one before it)",
            "us_per_call": out["hbm"], "us_per_call_l2_hot": out["l2_hot"], "bytes_per_call": bytes_per_call,
            "gpu_launches": calls,
            "other_shapes": {"note": "one stream, 200 calls in one CUDA graph rotating over 256 MiB of weight buffers", **other},
            "waits_run_out": fallbacks,
            "small_batch": {"note": "bitlinear_gemv_decode_batch, M tokens per call (one launch per 8 tokens), "
                                    "400 calls in one CUDA graph over the same 64 weight buffers, one stream",
                            **batch},
            "small_batch_ws": {"note": "bitlinear_gemv_decode_batch_ws (workspace; a quantising kernel, then one tcgen05 "
                                       "product kernel per 16 tokens), same graph and buffers",
                               **batch_ws},
            "independent_streams": {
                "note": "same 1000 calls spread round-robin over 2 / 4 streams inside the graph: calls on "
                        "different streams do not wait for one another",
                "us_per_call_2": out["hbm_2streams"], "us_per_call_4": out["hbm_4streams"],
                "gbs_2": rate(out["hbm_2streams"]), "gbs_4": rate(out["hbm_4streams"]),
                "frac_2": rate(out["hbm_2streams"]) / peaks["hbm_gbs"],
                "frac_4": rate(out["hbm_4streams"]) / peaks["hbm_gbs"]},
            "roofline": {"bound": "hbm", "kernel": "gemv_decode_fast_kernel", "achieved": gbs, "peak": peaks["hbm_gbs"],
                         "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"], "traffic": NCU_TRAFFIC["gemv_decode_fast_kernel"],
                         "frac_of_nominal": gbs / NOMINAL_HBM_GBS, "peak_source": peaks["source"] + " copy"}}


def bench_pack(B, synth, dev, peaks):
    """Binarise+pack of the prefill weight matrix (fp32 [4096,4096]), rotating over 3 copies."""
    N, K = PREFILL["N"], PREFILL["K"]
    Ws = [synth.make_w(N, K, torch.float32, seed=2 + r).to(dev) for r in range(ROTATE)]
    outs = [B.binarize_pack(Wr, layout=B.PREFILL) for Wr in Ws]
    ws = torch.empty(B.workspace_bytes(B.OP_BINARIZE_PACK, 1, N, K, 1), dtype=torch.uint8, device=dev)
    reps = 30
    for i in range(3):
        B.binarize_pack(Ws[i % ROTATE], layout=B.PREFILL, out=outs[i % ROTATE], ws=ws)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record()
    for i in range(reps):
        B.binarize_pack(Ws[i % ROTATE], layout=B.PREFILL, out=outs[i % ROTATE], ws=ws)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / reps
    nbytes = 2.0 * N * K * 4 + N * K / 8
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"workload": "binarize+pack W fp32 [4096,4096] -> 1 bit/weight (PREFILL layout), alpha, beta, rowsum",
            "ms": ms, "gpu_launches": 2 * reps,
            "roofline": {"bound": "hbm", "kernel": "reduce_partials + sign_pack_rows", "achieved": gbs,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                         "traffic": NCU_TRAFFIC["reduce_partials + sign_pack_rows"],
                         "peak_source": peaks["source"] + " copy"}}


def bench_grouped(B, synth, dev, peaks):
    """Config 5: 30B-shaped FFN down-projection with group quantization, G = 8 along K.  Binarize+pack,
    LN+quant (eta form, per-group scalars over all tokens) and the full forward, each timed alone."""
    M, K, N, G = 4096, 28672, 7168, 8
    W = synth.make_w(N, K, torch.float32, seed=4).to(dev)
    x = synth.make_x(M, K, torch.bfloat16, seed=4, outliers=False, relu=True).to(dev)
    w = B.binarize_pack(W, G=G, layout=B.PREFILL)
    ws_p = torch.empty(B.workspace_bytes(B.OP_BINARIZE_PACK, 1, N, K, G), dtype=torch.uint8, device=dev)
    ws_q = torch.empty(B.workspace_bytes(B.OP_QUANT_ACT, M, 1, K, G), dtype=torch.uint8, device=dev)
    ws_f = torch.empty(B.workspace_bytes(B.OP_FORWARD, M, N, K, G), dtype=torch.uint8, device=dev)
    q = dict(x_q=torch.empty((M, K), dtype=torch.int8, device=dev),
             gamma=torch.empty(G, dtype=torch.float32, device=dev), eta=torch.empty(G, dtype=torch.float32, device=dev))
    y = torch.empty((M, N), dtype=torch.bfloat16, device=dev)

    def timed(fn, reps):
        for _ in range(2):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    t_pack = timed(lambda: B.binarize_pack(W, G=G, layout=B.PREFILL, out=w, ws=ws_p), 5)
    t_quant = timed(lambda: B.quant_act(x, G=G, mode=B.ETA, gran=B.PER_TENSOR, out=q, ws=ws_q), 5)
    t_gemm = timed(lambda: B.matmul_dequant(q["x_q"], q["gamma"], w["W_packed"], w["beta"], N, G=G,
                                            gran=B.PER_TENSOR, layout=B.PREFILL, y=y, ws=ws_f), 5)
    t_fwd = timed(lambda: B.forward(x, w["W_packed"], w["beta"], N, G=G, mode=B.ETA, gran=B.PER_TENSOR,
                                    layout=B.PREFILL, y=y, ws=ws_f), 5)
    assert B.ws_status(ws_f) == B.OK
    pack_bytes = 2.0 * N * K * 4 + N * K / 8
    quant_bytes = 2.0 * M * K * 2 + M * K
    ops = 2.0 * M * N * K
    tensor_peak = INT8_TO_BF16 * peaks["bf16_tflops"]
    return {"workload": "30B-shaped FFN down-projection, G = 8 groups along K: W fp32 [7168,28672], x bf16 "
                        "[4096,28672] = ReLU(N(0,1)), eta form, per-group alpha/beta/gamma/eta, y bf16; working "
                        "sets exceed L2",
            "pack_ms": t_pack, "pack_gbs": pack_bytes / t_pack / 1e6, "pack_frac": pack_bytes / t_pack / 1e6 / peaks["hbm_gbs"],
            "quant_ms": t_quant, "quant_gbs": quant_bytes / t_quant / 1e6,
            "quant_frac": quant_bytes / t_quant / 1e6 / peaks["hbm_gbs"],
            "gemm_ms": t_gemm, "gemm_tops": ops / t_gemm / 1e9, "gemm_frac": ops / t_gemm / 1e9 / tensor_peak,
            "forward_ms": t_fwd, "forward_tops": ops / t_fwd / 1e9}


def bench_block(B, synth, dev, peaks):
    """Config 4: one BitNet decoder block forward, d = 2048, 16 heads, FFN 8192, batch 4 x seq 2048,
    fp16 activations, per-token quantisation; whole block and the attention core alone."""
    batch, seq, heads, ffn = 4, 2048, 16, 8192
    d, T = heads * 128, batch * seq
    x = synth.make_x(T, d, torch.float16, seed=3, outliers=False).to(dev)
    shapes = dict(q=(d, d), k=(d, d), v=(d, d), o=(d, d), up=(ffn, d), down=(d, ffn))
    w = {n: B.binarize_pack(synth.make_w(N, K, torch.float32, seed=3 + 17 * i).to(dev), layout=B.PREFILL)
         for i, (n, (N, K)) in enumerate(shapes.items())}
    w = B.fuse_qkv_weights(w)                        # Q, K, V back to back: one [3d, d] GEMM
    ws = torch.empty(B.workspace_bytes(B.OP_BLOCK_FORWARD, T, ffn, d, 1), dtype=torch.uint8, device=dev)
    out = B.block_forward(x, w, batch, seq, heads, ffn, ws=ws, fused_qkv=True)

    def timed(fn, reps):
        for _ in range(2):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    t_block = timed(lambda: B.block_forward(x, w, batch, seq, heads, ffn, ws=ws, fused_qkv=True), 10)
    t_attn = timed(lambda: B.attention_causal(out["q"], out["k"], out["v"], batch, seq, heads, o=out["a"]), 10)
    assert B.ws_status(ws) == B.OK
    lin_ops = 2.0 * T * (4 * d * d + 2 * d * ffn)
    attn_flops = 4.0 * batch * heads * (seq * (seq + 1) / 2) * 128
    return {"workload": "BitNet decoder block forward: d 2048, 16 heads, FFN 8192 (ReLU, eta form on the down "
                        "input), batch 4 x seq 2048, fp16 activations, per-token quantisation, six BitLinear "
                        "layers (Q, K, V as one GEMM; ReLU and residual adds in the GEMM epilogues) + causal "
                        "fp16 attention: 4 LN+quant, 4 GEMM and 1 attention launch",
            "block_ms": t_block, "attention_ms": t_attn, "bitlinear_ops": lin_ops,
            "bitlinear_tops_of_block_time": lin_ops / t_block / 1e9,
            "attention_tflops": attn_flops / t_attn / 1e9,
            "gpu_launches": 10 * 9}


def bench_small(B, synth, dev):
    """Config 1: one 125M-shaped layer, x fp32 [64, 768], W fp32 [3072, 768], per-tensor absmax, y fp32.
    0.3 GOP: a latency case, reported in microseconds per call (each entry point timed alone, calls
    back to back on one stream)."""
    M, K, N = 64, 768, 3072
    x = synth.make_x(M, K, torch.float32, seed=0, outliers=True).to(dev)
    W = synth.make_w(N, K, torch.float32, seed=0).to(dev)
    w = B.binarize_pack(W, layout=B.PREFILL)
    ws_p = torch.empty(B.workspace_bytes(B.OP_BINARIZE_PACK, 1, N, K, 1), dtype=torch.uint8, device=dev)
    ws_q = torch.empty(B.workspace_bytes(B.OP_QUANT_ACT, M, 1, K, 1), dtype=torch.uint8, device=dev)
    ws_f = torch.empty(B.workspace_bytes(B.OP_FORWARD, M, N, K, 1), dtype=torch.uint8, device=dev)
    q = dict(x_q=torch.empty((M, K), dtype=torch.int8, device=dev), gamma=torch.empty(1, device=dev),
             eta=torch.zeros(1, device=dev))
    y = torch.empty((M, N), dtype=torch.float32, device=dev)

    def timed(fn, reps=200):
        for _ in range(5):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(reps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps * 1e3

    out = {"workload": "single BitLinear layer: x fp32 [64,768] N(0,1) + 0.1% x20 outliers, W fp32 [3072,768] "
                       "N(0,0.02), per-tensor absmax, y fp32, seed 0 (latency case: microseconds per call)",
           "pack_us": timed(lambda: B.binarize_pack(W, layout=B.PREFILL, out=w, ws=ws_p)),
           "quant_us": timed(lambda: B.quant_act(x, gran=B.PER_TENSOR, out=q, ws=ws_q)),
           "forward_us": timed(lambda: B.forward(x, w["W_packed"], w["beta"], N, gran=B.PER_TENSOR, layout=B.PREFILL,
                                                 y=y, ws=ws_f))}
    assert B.ws_status(ws_f) == B.OK
    return out


# --------------------------------------------------------------------------- the CPU oracle, timed

def cpu_baseline_decode(reps=20):
    """The oracle on config 2 (one token, K 4096, N 16384): full size, a few repetitions."""
    from oracle import oracle as O
    from paper_2310_11453_b200 import synth
    K, N = DECODE["K"], DECODE["N"]
    W = synth.make_w(N, K, torch.float32, seed=1)
    wb = O.binarize(W.numpy())
    x = synth.make_x(reps, K, torch.float16, seed=1, outliers=False).to(torch.float32).numpy()
    t = time.perf_counter()
    for i in range(reps):
        O.forward(x[i:i + 1], wb["bits"], wb["beta"], gran=O.PER_TOKEN, ln_eps=1e-5)
    dt = (time.perf_counter() - t) / reps
    nbytes = N * K / 8 + 2 * K + 2 * N
    return {"value": nbytes / dt / 1e9, "unit": "GB/s of packed weights", "us_per_call": dt * 1e6, "cores": O.num_threads(),
            "kind": "oracle", "sample": f"oracle forward, one token, full W [16384,4096], mean of {reps} calls"}


def cpu_baseline_grouped(tokens=16):
    """The oracle on config 5 (G = 8): binarisation of the full weight matrix, and the forward on a
    token sample against the full matrix."""
    from oracle import oracle as O
    from paper_2310_11453_b200 import synth
    M, K, N, G = 4096, 28672, 7168, 8
    W = synth.make_w(N, K, torch.float32, seed=4)
    t = time.perf_counter()
    wb = O.binarize(W.numpy(), G=G)
    t_bin = time.perf_counter() - t
    del W
    x = synth.make_x(tokens, K, torch.bfloat16, seed=4, outliers=False, relu=True).to(torch.float32).numpy()
    t = time.perf_counter()
    O.forward(x, wb["bits"], wb["beta"], G=G, mode=O.ETA, gran=O.PER_TENSOR, ln_eps=1e-5)
    dt = time.perf_counter() - t
    return {"value": 2.0 * tokens * N * K / dt / 1e12, "unit": "TOPS", "cores": O.num_threads(), "kind": "oracle",
            "binarize_s": t_bin, "binarize_gbs": (2.0 * N * K * 4 + N * K / 8) / t_bin / 1e9,
            "sample": f"oracle forward on {tokens} of {M} tokens against the full W [7168,28672], G = 8, eta form "
                      f"({dt:.2f} s); binarisation of the full matrix {t_bin:.2f} s"}


def oracle_prefill_sample(x_host, W_host, tokens, reps=1):
    """Times the CPU oracle's forward (LN+quant, matmul, rescale) on the first `tokens` tokens of the
    prefill batch against the full weight matrix.  Returns (seconds per call, threads)."""
    from oracle import oracle as O
    xs = x_host[:tokens].to(torch.float32).numpy()
    wb = O.binarize(W_host.numpy())
    best = None
    for _ in range(reps):
        t = time.perf_counter()
        O.forward(xs, wb["bits"], wb["beta"], G=1, mode=O.ABSMAX, gran=O.PER_TENSOR, ln_eps=1e-5)
        dt = time.perf_counter() - t
        best = dt if best is None else min(best, dt)
    return best, O.num_threads()


def cpu_baseline_prefill(x_host, W_host, target_s=15.0):
    # two probes separate the fixed cost (unpacking W) from the per-token cost
    d1, _ = oracle_prefill_sample(x_host, W_host, 64)
    d2, _ = oracle_prefill_sample(x_host, W_host, 512)
    per_token = max((d2 - d1) / 448.0, 1e-7)
    tokens = int(min(PREFILL["M"], max(512, (target_s - d1) / per_token)))
    tokens -= tokens % 64
    dt, cores = oracle_prefill_sample(x_host, W_host, tokens)
    ops = 2.0 * tokens * PREFILL["N"] * PREFILL["K"]
    return {"value": ops / dt / 1e12, "unit": "TOPS", "cores": cores, "kind": "oracle",
            "sample": f"oracle forward on the first {tokens} of {PREFILL['M']} tokens of the prefill batch, "
                      f"full W [4096,4096]; {dt:.2f} s"}


def run_reference(args):
    """The reference arm: the CPU oracle as it stands, on the host cores, same metric and config.
    Each step is the oracle's forward on a token sample of the prefill batch (16 to 1024 tokens,
    sized so that the run ends in about a minute)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2310_11453_b200 import synth
    M, K, N = PREFILL["M"], PREFILL["K"], PREFILL["N"]
    from oracle import oracle as O
    x_all = synth.make_x(1024, K, torch.bfloat16, seed=2, outliers=True)
    W = synth.make_w(N, K, torch.float32, seed=2)
    wb = O.binarize(W.numpy())
    # size the per-step token sample so that the whole run takes about a minute
    probe = x_all[:16].to(torch.float32).numpy()
    t = time.perf_counter()
    O.forward(probe, wb["bits"], wb["beta"], G=1, mode=O.ABSMAX, gran=O.PER_TENSOR, ln_eps=1e-5)
    per_token = (time.perf_counter() - t) / 16
    budget = 60.0 / (args.steps + max(args.warmup, 1))
    tokens = int(max(16, min(1024, budget / max(per_token, 1e-9))))
    tokens -= tokens % 16
    xs = x_all[:tokens].to(torch.float32).numpy()

    def step():
        O.forward(xs, wb["bits"], wb["beta"], G=1, mode=O.ABSMAX, gran=O.PER_TENSOR, ln_eps=1e-5)

    for _ in range(max(args.warmup, 1)):
        step()
    t = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t) / args.steps
    value = 2.0 * tokens * N * K / dt / 1e12
    sample = f"oracle forward on {tokens} of {M} tokens of the prefill batch per step, full W [4096,4096]"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TOPS",
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64 and exact integers (CPU oracle)", "data": "synthetic",
            "config": {"workload": "prefill BitLinear forward (CPU oracle on a token sample)", "M": M, "K": K,
                       "N": N, "G": 1, "sample_tokens": tokens},
            "cpu_baseline": {"value": value, "unit": "TOPS", "cores": O.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--parts", default="calib,decode,pack,grouped,block,small,cpu",
                    help="extra measurements beside the prefill step (comma list of calib, decode, pack, grouped, block, small, cpu; "
                         "'none' for the prefill step alone, e.g. under a profiler)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand with --gpus N: run the N replicas (one process per GPU) under torchrun
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_b200(args)


if __name__ == "__main__":
    main()
