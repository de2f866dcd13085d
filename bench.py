#!/usr/bin/env python
"""Benchmark of the W4A8 linear hot path (activation FP8 quantize -> fused INT4->FP8 GEMM ->
scaled BF16) on the decode sweep: M in {1,4,16}, K=4096, N=14336 (Llama-3-8B MLP up-projection).

One step = one pass of the whole path over the sweep: for each M, the Eq. 13 activation
quantization and the W4A8 linear, run as three problems of a w4a8_linear_chain launch (one
persistent kernel; --steps-per-launch consecutive steps share a launch, as a decode launch holds
the layers of a forward pass).  The metric is the weight stream rate: bytes of INT4 codes + group
scales the method must read per step, divided by the step time.  Weights rotate over several
distinct copies whose total size exceeds twice the L2, so every pass streams them from HBM.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 runs one independent replica per GPU (the path has no exchange step): under torchrun when
the launcher set WORLD_SIZE, else bench.py starts the N ranks itself.
--impl reference times the CPU oracle on the host cores on a bounded sample of the same
workload.  Prints one JSON line on rank 0.
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

SWEEP_M = (1, 4, 16)
K, N = 4096, 14336
GROUP = 128
SIGMA, OUTLIER_FRAC, OUTLIER_MULT = 0.02, 0.01, 20.0
WEIGHT_COPIES = 10          # 10 x 30.3 MB = 303 MB > 2 x 126 MB L2
METRIC = "w4a8_decode_weight_stream_rate"
UNIT = "GB/s"
WORKLOAD = ("c2 decode sweep: W4A8 linear, M in {1,4,16}, K=4096, N=14336, INT4 group-128 symmetric "
            "weights from N(0,0.02), BF16 N(0,1) activations with 1% outlier channels x20, "
            "per-token FP8 E4M3 scales, BF16 output")

# DRAM bytes per problem of the dominant kernel from an ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum of one launch divided by its problems); see profiles/.  None until a capture
# exists for the current kernel.
NCU_TRAFFIC_BYTES_PER_PROBLEM = 30.65e6  # profiles/linear_chain_decode_c2.md: (727.65 + 8.1) MB per 24-problem launch


def weight_bytes(n=N, k=K):
    """Bytes of the stored weight format one linear must read: codes + BF16 group scales."""
    return n * k // 2 + n * (k // GROUP) * 2


def linear_algorithmic_bytes(m, n=N, k=K):
    """Everything one linear launch must move: weights, FP8 activations + scales, the weight scale,
    BF16 output."""
    return weight_bytes(n, k) + m * k + 4 * m + 4 + 2 * m * n


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.lines = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._pump, daemon=True)
        self.thread.start()

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power = [], [], []
        reasons = set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
                power.append(float(parts[3]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(smax), "samples": len(sm),
                "power_w_max": max(power), "reasons": sorted(reasons)}


# --------------------------------------------------------------------------------------------
# CPU oracle legs
# --------------------------------------------------------------------------------------------

def oracle_sample_pass(rows, x_bits_by_m, w_sample):
    """One pass of the sweep through the oracle as it stands on `rows` output channels."""
    import oracle
    codes, gscale, gzero, s_w = w_sample
    t0 = time.perf_counter()
    for m in SWEEP_M:
        x8, s_x = oracle.quantize_act(x_bits_by_m[m])
        w8 = oracle.dequant_weight(codes, gscale, gzero)
        oracle.linear(x8, s_x, w8, s_w, want=("ybf16",))
    return time.perf_counter() - t0


def make_oracle_sample(rows, seed=0):
    import oracle
    from paper_2505_14638_b200 import inputs
    W = inputs.make_weight(rows, K, SIGMA, seed)
    return oracle.quantize_weight_rtn(W, symmetric=True)


def make_x_bits(seed=0):
    from paper_2505_14638_b200 import inputs
    return {m: inputs.make_activation(m, K, seed + m, OUTLIER_FRAC, OUTLIER_MULT) for m in SWEEP_M}


def cpu_baseline(budget_s=12.0):
    """The oracle timed on the host cores on a bounded sample (a slab of output channels)."""
    import oracle
    oracle.build()
    x_bits = make_x_bits()
    rows = 512
    t = oracle_sample_pass(rows, x_bits, make_oracle_sample(rows))
    rows_fit = int(min(N, max(512, rows * budget_s / max(t, 1e-6))))
    rows_fit -= rows_fit % 16
    if rows_fit > rows:
        rows = rows_fit
        t = oracle_sample_pass(rows, x_bits, make_oracle_sample(rows))
    value = len(SWEEP_M) * weight_bytes(rows, K) / t / 1e9
    return {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": "one pass of the sweep M in {1,4,16} on the first %d of %d output channels "
                      "(act quant + Eq. 10 dequant + exact matmul), %.2f s" % (rows, N, t)}


def run_reference(args, rank):
    if rank != 0:
        return
    import oracle
    oracle.build()
    total_budget = 150.0
    per_step = total_budget / max(1, args.steps + args.warmup)
    x_bits = make_x_bits()
    rows = 256
    t = oracle_sample_pass(rows, x_bits, make_oracle_sample(rows))
    rows_fit = int(min(N, max(128, rows * per_step / max(t, 1e-6))))
    rows_fit -= rows_fit % 16
    rows = max(16, rows_fit)
    sample = make_oracle_sample(rows)
    for _ in range(args.warmup):
        oracle_sample_pass(rows, x_bits, sample)
    times = [oracle_sample_pass(rows, x_bits, sample) for _ in range(args.steps)]
    total = sum(times)
    value = args.steps * len(SWEEP_M) * weight_bytes(rows, K) / total / 1e9
    desc = ("each step = one pass of the sweep M in {1,4,16} on %d of %d output channels" % (rows, N))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": WORKLOAD, "sample": desc},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------

def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings (the job is as slow as its slowest replica)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_rate(world, steps, ms_total):
    """Whole-job weight stream rate in GB/s: every replica streams the sweep's weights each step."""
    return world * steps * len(SWEEP_M) * weight_bytes() / (ms_total * 1e-3) / 1e9


def chain_algorithmic_bytes(ms, n=N, k=K):
    """Everything one chain launch over the token counts `ms` must move: per problem the stored
    weights (codes + group scales), the BF16 activations in, the weight scale and the BF16 output."""
    return sum(weight_bytes(n, k) + 2 * m * k + 4 + 2 * m * n for m in ms)


def run_ours(args, rank, world, local_rank):
    import torch
    from paper_2505_14638_b200 import binding, inputs
    from paper_2505_14638_b200 import build as _build

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the W4A8 path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    if rank == 0:
        _build.build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist.barrier()
    binding.lib()
    dev = torch.device("cuda", local_rank)

    # ---- inputs: seeded synthetic, quantized and tiled offline, resident in HBM ----
    weights = []
    for c in range(WEIGHT_COPIES):
        W = torch.from_numpy(inputs.make_weight(N, K, SIGMA, seed=1000 * rank + c)).to(dev)
        wq = binding.quantize_weight_rtn(W, symmetric=True)
        weights.append(binding.prepack_weight(*wq))
        del W, wq
    torch.cuda.synchronize()
    if binding.query_device_status() != 0:
        raise RuntimeError("prepack reported an unrepresentable code")
    xs, ys, x_host, y_host = {}, {}, {}, {}
    for m in SWEEP_M:
        xb = inputs.make_activation(m, K, 1000 * rank + m, OUTLIER_FRAC, OUTLIER_MULT)
        t = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16)
        x_host[m] = t
        xs[m] = t.to(dev)
        ys[m] = torch.empty((m, N), dtype=torch.bfloat16, device=dev)
        y_host[m] = [torch.empty((m, N), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    torch.cuda.synchronize()

    # ---- the step: one pass of the whole path (Eq. 13 quantization, Eq. 10 expansion, FP8 MMAs,
    # Eq. 4 / Eq. 11 epilogue) over the sweep, as problems of ONE persistent launch
    # (w4a8_linear_chain).  A launch carries `spl` consecutive steps, as a decode launch carries the
    # layers of a forward pass; every problem reads the next weight copy of the rotation.
    spl = max(1, min(args.steps_per_launch, binding.CHAIN_MAX_PROBLEMS // len(SWEEP_M)))
    workspace = [None]

    def make_launch(first_step, nsteps, host_buffers=None):
        probs = []
        for s_ in range(nsteps):
            for i, m in enumerate(SWEEP_M):
                c = ((first_step + s_) * len(SWEEP_M) + i) % WEIGHT_COPIES
                if host_buffers is None:
                    x_, y_ = xs[m], ys[m]
                else:
                    # this step's rows of the staging buffer that the call's one host-to-device copy fills;
                    # the results go straight to pinned host memory
                    x_ = x_stage[host_buffers][s_, row0[m]:row0[m] + m]
                    y_ = y_host[m][host_buffers]
                probs.append(dict(x=x_, weight=weights[c], y=y_))
        ch = binding.LinearChain(probs, workspace=workspace[0])
        if workspace[0] is None or ch.ws.numel() > workspace[0].numel():
            workspace[0] = ch.ws
        return ch

    probe = make_launch(0, spl)                     # sizes the shared workspace
    n_full, n_tail = args.steps // spl, args.steps % spl
    period = WEIGHT_COPIES                          # the weight rotation repeats after this many launches
    full = [make_launch(g * spl, spl) for g in range(min(period, max(n_full, 1)))]
    tail = make_launch(n_full * spl, n_tail) if n_tail else None
    del probe

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for g in range(max(3, (max(args.warmup, 3) + spl - 1) // spl)):
        full[g % len(full)]()
    if tail is not None:
        tail()
    barrier()
    if binding.query_device_status() != 0:
        raise RuntimeError("device status word set by the first steps (a bounded wait gave up)")

    # ---- timed region 1: K steps, device timed ----
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for g in range(n_full):
        full[g % len(full)]()
    if tail is not None:
        tail()
    e1.record()
    barrier()
    launches = n_full + (1 if tail is not None else 0)
    ms_total = e0.elapsed_time(e1)

    # ---- timed region 2: the dominant kernel alone -- full launches back to back, bracketed by events ----
    reps = max(10, n_full)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for g in range(reps):
        full[g % len(full)]()
    b.record()
    torch.cuda.synchronize()
    launch_ms = a.elapsed_time(b) / reps
    clocks = sampler.stop() if rank == 0 else None
    if binding.query_device_status() != 0:
        raise RuntimeError("device status word set during the timed region")

    # ---- end to end: host buffers in and out.  Every step's activations sit in pinned host memory
    # and are brought to the device inside the timed region, one asynchronous copy per call (all
    # the steps of the call) on a copy stream; every step's result is written to pinned host memory
    # by the kernel itself, over the bus.  Two sets of buffers: the copy for call i + 1 runs while
    # call i computes, and the caller waits for call i's event (and reads its results) after it
    # has issued call i + 1.  (A kernel that reads its activations from host memory directly takes
    # 60-75 us longer per call: loads issued by SMs fetch 1.4 MB over the bus far more slowly than
    # the copy engine does; stores to host memory cost nothing measurable.)  Also measured: a full
    # stop after every call. ----
    rows_per_step = sum(SWEEP_M)
    row0, acc = {}, 0
    for m in SWEEP_M:
        row0[m] = acc
        acc += m
    x_pin, x_stage = [], []
    for par in range(2):
        hp = torch.empty((spl, rows_per_step, K), dtype=torch.bfloat16).pin_memory()
        for m in SWEEP_M:
            hp[:, row0[m]:row0[m] + m] = x_host[m]
        x_pin.append(hp)
        x_stage.append(torch.empty((spl, rows_per_step, K), dtype=torch.bfloat16, device=dev))
    e2e_calls = [make_launch(g * spl, spl, host_buffers=g % 2) for g in range(min(2, max(n_full, 1)))]
    e2e_tail = make_launch(n_full * spl, n_tail, host_buffers=n_full % 2) if n_tail else None
    seq = [(e2e_calls[g % len(e2e_calls)], g % 2, spl) for g in range(n_full)]
    if e2e_tail is not None:
        seq.append((e2e_tail, n_full % 2, n_tail))
    copy_stream = torch.cuda.Stream(device=dev)
    copied = [torch.cuda.Event() for _ in seq]
    done = [torch.cuda.Event() for _ in seq]

    def e2e_pass(overlap):
        main = torch.cuda.current_stream()
        for i, (call, par, nsteps) in enumerate(seq):
            with torch.cuda.stream(copy_stream):
                if i >= 2:
                    copy_stream.wait_event(done[i - 2])      # the call that read this staging buffer last
                x_stage[par][:nsteps].copy_(x_pin[par][:nsteps], non_blocking=True)
                copied[i].record()
            main.wait_event(copied[i])
            call()
            done[i].record()
            if not overlap:
                done[i].synchronize()           # the caller reads this call's results
            elif i > 0:
                done[i - 1].synchronize()       # the caller reads the previous call's results
        done[-1].synchronize()

    # Every pass is K steps; three passes per mode, the median reported (a single pass of a few hundred
    # microseconds that goes through the host scatters by several percent from one run to the next), all
    # three kept in the line.
    ms_e2e_by_mode, e2e_passes = {}, {}
    for overlap in (False, True):
        e2e_pass(True)
        got = []
        for _ in range(3):
            barrier()
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record()
            e2e_pass(overlap)
            g1.record()
            barrier()
            got.append(g0.elapsed_time(g1))
        e2e_passes[overlap] = got
        ms_e2e_by_mode[overlap] = sorted(got)[1]
    ms_e2e, ms_e2e_stop = ms_e2e_by_mode[True], ms_e2e_by_mode[False]
    if binding.query_device_status() != 0:
        raise RuntimeError("device status word set during the end-to-end region")

    ms_total, ms_e2e, ms_e2e_stop, launch_ms = max_over_ranks([ms_total, ms_e2e, ms_e2e_stop, launch_ms], dist, dev)

    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    value = aggregate_rate(world, args.steps, ms_total)
    e2e_value = aggregate_rate(world, args.steps, ms_e2e)
    alg_bytes = chain_algorithmic_bytes(SWEEP_M * spl)
    achieved = alg_bytes / (launch_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3", "data": "synthetic",
        "config": {"workload": WORKLOAD, "parallelism": "replicas x%d (no collective)" % world,
                   "l2": "weights rotate over %d distinct copies (%.0f MB > 2 x 126 MB L2)"
                         % (WEIGHT_COPIES, WEIGHT_COPIES * weight_bytes() / 1e6),
                   "step": "for M in (1,4,16): Eq. 13 activation quantization + W4A8 linear on tiled sign-magnitude "
                           "weights, as three problems of a w4a8_linear_chain launch",
                   "launch": "one persistent launch per %d steps (%d problems), eager, back to back; "
                             "%d launch(es) in the timed region" % (spl, spl * len(SWEEP_M), launches)},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": sum(m * K * 2 for m in SWEEP_M),
                "d2h_bytes_per_step": sum(m * N * 2 for m in SWEEP_M),
                "ms_per_step": ms_e2e / args.steps,
                "passes_ms_per_step": [t / args.steps for t in e2e_passes[True]], "statistic": "median of three passes of K steps",
                "ms_per_step_full_stop_after_every_call": ms_e2e_stop / args.steps,
                "how": "per call of %d steps: one asynchronous copy of the steps' activations from pinned host memory "
                       "(copy stream), w4a8_linear_chain writing every step's result to pinned host memory over the "
                       "bus; two sets of buffers, the caller waits for a call's event after issuing the next call" % spl},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "linear_chain_kernel (w4a8_linear_chain), %d problems per launch: "
                               "M in {1,4,16} x %d" % (spl * len(SWEEP_M), spl),
                     "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "peak_source": peaks["source"],
                     "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_us": launch_ms * 1e3,
                     "us_per_problem": launch_ms * 1e3 / (spl * len(SWEEP_M)),
                     "traffic": NCU_TRAFFIC_BYTES_PER_PROBLEM * spl * len(SWEEP_M)
                     if NCU_TRAFFIC_BYTES_PER_PROBLEM else None},
    }
    if not args.no_extras:
        line["decode_detail"] = decode_detail(torch, binding, weights, xs, ys, peaks)
        line["act_quant"] = act_quant_extra(torch, binding, inputs, dev, peaks)
        line["prefill"] = prefill_extra(torch, binding, inputs, dev, peaks)
        line["prefill_c4"] = prefill_c4_extra(torch, binding, inputs, dev, peaks)
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline()
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def _time_loop(torch, fn, iters, warm=3):
    for _ in range(warm):
        fn()
    torch.cuda.synchronize()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(iters):
        fn()
    b.record()
    torch.cuda.synchronize()
    return a.elapsed_time(b) * 1e-3 / iters


def decode_detail(torch, binding, weights, xs, ys, peaks):
    """Per M: time per problem of a chain launch that carries one problem per weight copy, next to
    the per-launch path (w4a8_quantize_act + w4a8_linear replayed from a CUDA graph) and cuBLAS BF16."""
    out = {}
    dev = ys[1].device
    wb = [torch.randn((N, K), dtype=torch.bfloat16, device=dev) for _ in range(4)]
    side = torch.cuda.Stream()
    x8s = {m: torch.empty((m, K), dtype=torch.uint8, device=dev) for m in SWEEP_M}
    sxs = {m: torch.empty((m,), dtype=torch.float32, device=dev) for m in SWEEP_M}
    workspace = binding.new_workspace(max(SWEEP_M), N, K, weights[0].fmt, dev)
    for m in SWEEP_M:
        chain = binding.LinearChain([dict(x=xs[m], weight=weights[c], y=ys[m]) for c in range(WEIGHT_COPIES)])
        t = _time_loop(torch, chain, 20) / WEIGHT_COPIES
        one = [binding.LinearChain([dict(x=xs[m], weight=weights[c], y=ys[m])], workspace=chain.ws)
               for c in range(WEIGHT_COPIES)]
        j1 = [0]

        def single():
            j1[0] += 1
            one[j1[0] % WEIGHT_COPIES]()
        t1 = _time_loop(torch, single, 40)
        side.wait_stream(torch.cuda.current_stream())
        g3 = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g3, stream=side):
                for c in range(WEIGHT_COPIES):
                    binding.quantize_act(xs[m], out=(x8s[m], sxs[m]))
                    binding.linear_tiled(x8s[m], sxs[m], weights[c], out=ys[m], workspace=workspace)
        torch.cuda.current_stream().wait_stream(side)
        t2 = _time_loop(torch, g3.replay, 20) / WEIGHT_COPIES
        xb = torch.randn((m, K), dtype=torch.bfloat16, device=dev)
        j = [0]

        def f():
            j[0] += 1
            torch.matmul(xb, wb[j[0] % 4].t())
        tb = _time_loop(torch, f, 40)
        alg = chain_algorithmic_bytes((m,))
        out["M=%d" % m] = {"chain_us_per_problem": t * 1e6, "chain_weight_GBps": weight_bytes() / t / 1e9,
                           "chain_frac_hbm_measured": alg / t / 1e9 / peaks["hbm_gbs"],
                           "chain_single_problem_launch_us": t1 * 1e6,
                           "per_launch_quantize_then_linear_us": t2 * 1e6,
                           "per_launch_frac_hbm_measured": alg / t2 / 1e9 / peaks["hbm_gbs"],
                           "cublas_bf16_us": tb * 1e6}
    return out


def act_quant_extra(torch, binding, inputs, dev, peaks):
    """w4a8_quantize_act alone (Eq. 13: 2 bytes read + 1 byte written per element, plus one scale per
    token) at the prefill sizes of c3 and c4, against the measured HBM copy rate."""
    out = {}
    for name, m, k in (("c3", 2048, 4096), ("c4", 8192, 8192)):
        copies = max(2, int(2.2 * 126e6 / (3 * m * k)) + 1)
        xs_ = []
        for c in range(copies):
            xb = inputs.make_activation(m, k, 300 + c, OUTLIER_FRAC, OUTLIER_MULT)
            xs_.append(torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev))
        x8 = torch.empty((m, k), dtype=torch.uint8, device=dev)
        s_x = torch.empty((m,), dtype=torch.float32, device=dev)
        # a graph of back-to-back launches over the distinct copies: the kernel, not the host's launch rate
        # (issued eagerly through the binding the c3 launch is host-bound at 9.7 us)
        side = torch.cuda.Stream()
        for c in range(2):
            binding.quantize_act(xs_[c], out=(x8, s_x))
        side.wait_stream(torch.cuda.current_stream())
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(gr, stream=side):
                for c in range(copies):
                    binding.quantize_act(xs_[c], out=(x8, s_x))
        torch.cuda.current_stream().wait_stream(side)
        t = _time_loop(torch, gr.replay, 10, warm=3) / copies
        b = 3.0 * m * k + 4.0 * m
        out[name] = {"M": m, "K": k, "us": t * 1e6, "algorithmic_bytes": b, "GBps": b / t / 1e9,
                     "frac_hbm_measured": b / t / 1e9 / peaks["hbm_gbs"],
                     "l2": "inputs rotate over %d copies" % copies}
        del xs_
    return out


def prefill_c4_extra(torch, binding, inputs, dev, peaks):
    """Config c4 (M=8192, K=8192, N=28672): w4a8_linear on quantized activations, a few repeats of the
    1.9 ms launch, against 2 x the SUSTAINED BF16 figure (a long tensor-bound launch runs under the
    power cap) and against the burst figure."""
    M4, K4, N4 = 8192, 8192, 28672
    W = torch.from_numpy(inputs.make_weight(N4, K4, 0.015, seed=77)).to(dev)
    tw = binding.prepack_weight(*binding.quantize_weight_rtn(W, symmetric=True))
    del W
    xb = inputs.make_activation(M4, K4, 78, 0.005, 30.0)
    x = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev)
    x8, s_x = binding.quantize_act(x)
    y = torch.empty((M4, N4), dtype=torch.bfloat16, device=dev)
    ws = binding.new_workspace(M4, N4, K4, tw.fmt, dev)
    t = _time_loop(torch, lambda: binding.linear_tiled(x8, s_x, tw, out=y, workspace=ws), 5, warm=3)
    flops = 2.0 * M4 * N4 * K4
    sus = 2.0 * peaks["bf16_tflops_sustained"]
    res = {"workload": "c4 prefill M=8192 K=8192 N=28672 (weights + activations 0.36 GB > L2)", "us": t * 1e6,
           "tflops": flops / t / 1e12, "fp8_peak_sustained_tflops": sus,
           "frac_of_fp8_peak_sustained": flops / t / 1e12 / sus,
           "frac_of_fp8_peak_burst": flops / t / 1e12 / (2.0 * peaks["bf16_tflops"]),
           "frac_of_nominal_4500": flops / t / 1e12 / 4500.0, "peak_source": peaks["source"]}
    del tw, x, x8, y, ws
    torch.cuda.empty_cache()
    return res


def library_fp8_gemm_tflops(torch, dev, n=8192):
    """Empirical dense-FP8 reference on this machine: the library's FP8 GEMM (torch._scaled_mm, E4M3 x
    E4M3 -> BF16, per-tensor scales) at n^3, best of a few short loops.  None when unavailable."""
    try:
        a = torch.randn((n, n), device=dev).to(torch.float8_e4m3fn)
        b = torch.randn((n, n), device=dev).to(torch.float8_e4m3fn).t()  # column-major second operand
        one = torch.ones((), device=dev, dtype=torch.float32)
        f = lambda: torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)  # noqa: E731
        f()
        best = min(_time_loop(torch, f, 5, warm=1) for _ in range(3))
        return 2.0 * n ** 3 / best / 1e12
    except Exception:  # the call's signature and availability differ between torch builds
        return None


def prefill_extra(torch, binding, inputs, dev, peaks):
    """Config c3 (M=2048, K=4096, N=4096): FP8 tensor-pipe rate of w4a8_linear next to cuBLAS BF16."""
    M3, K3, N3 = 2048, 4096, 4096
    copies = 8
    sets = []
    for c in range(copies):
        W = torch.from_numpy(inputs.make_weight(N3, K3, SIGMA, seed=50 + c)).to(dev)
        tw = binding.prepack_weight(*binding.quantize_weight_rtn(W, symmetric=True))
        xb = inputs.make_activation(M3, K3, 50 + c, OUTLIER_FRAC, OUTLIER_MULT)
        x = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev)
        x8, s_x = binding.quantize_act(x)
        sets.append((tw, x8, s_x, x))
    y = torch.empty((M3, N3), dtype=torch.bfloat16, device=dev)
    ws = binding.new_workspace(M3, N3, K3, sets[0][0].fmt, dev)
    i = [0]

    # a graph of back-to-back launches over the distinct copies: the kernel, not the launch path
    side = torch.cuda.Stream()
    for tw, x8, s_x, _ in sets[:2]:
        binding.linear_tiled(x8, s_x, tw, out=y, workspace=ws)
    side.wait_stream(torch.cuda.current_stream())
    gr = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(gr, stream=side):
            for tw, x8, s_x, _ in sets:
                binding.linear_tiled(x8, s_x, tw, out=y, workspace=ws)
    torch.cuda.current_stream().wait_stream(side)
    t = _time_loop(torch, gr.replay, 10, warm=3) / copies
    wb = torch.randn((N3, K3), dtype=torch.bfloat16, device=dev)

    def g():
        _, _, _, x = sets[i[0] % copies]
        i[0] += 1
        torch.matmul(x, wb.t())
    tb = _time_loop(torch, g, 40, warm=5)
    flops = 2.0 * M3 * N3 * K3
    fp8_peak = 2.0 * peaks["bf16_tflops"]
    lib_fp8 = library_fp8_gemm_tflops(torch, dev)
    return {"workload": "c3 prefill M=2048 K=4096 N=4096", "us": t * 1e6, "tflops": flops / t / 1e12,
            "library_fp8_gemm_8192_tflops": lib_fp8,
            "fp8_peak_tflops": fp8_peak, "peak_note": "2 x bf16 burst peak (%s)" % peaks["source"],
            "frac_of_fp8_peak": flops / t / 1e12 / fp8_peak, "frac_of_nominal_4500": flops / t / 1e12 / 4500.0,
            "cublas_bf16_us": tb * 1e6, "cublas_bf16_tflops": flops / tb / 1e12}


C5_LAYERS = (("qkv", 4096, 6144), ("o", 4096, 4096), ("gate_up", 4096, 28672), ("down", 14336, 4096))
C5_M = (1, 8, 32, 128, 512, 4096)


def layer_sweep(torch, binding, inputs, dev, peaks, layers=C5_LAYERS, ms=C5_M, with_cublas=True):
    """Config c5: the four Llama-3-8B linears x M.  Per case: time of quantize_act + linear and of the
    linear alone (for M <= 16 also per problem of a w4a8_linear_chain launch), from CUDA graphs of
    back-to-back launches that rotate over enough weight copies to exceed twice the L2; the
    roofline time is the larger of bytes / HBM peak and flops / (2 x BF16 burst peak)."""
    out = []
    fp8_peak = 2.0 * peaks["bf16_tflops"] * 1e12
    hbm = peaks["hbm_gbs"] * 1e9
    side = torch.cuda.Stream()

    def graph_time(fn, reps):
        fn(0)
        torch.cuda.synchronize()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for c in range(reps):
                    fn(c)
        torch.cuda.current_stream().wait_stream(side)
        return _time_loop(torch, g.replay, 5, warm=2) / reps

    for name, k, n in layers:
        wbytes = weight_bytes(n, k)
        copies = max(2, min(32, int(2.2 * 126e6 / wbytes) + 1))
        tws = []
        for c in range(copies):
            W = torch.from_numpy(inputs.make_weight(n, k, SIGMA, seed=7000 + c)).to(dev)
            tws.append(binding.prepack_weight(*binding.quantize_weight_rtn(W, symmetric=True)))
            del W
        wb = torch.randn((n, k), dtype=torch.bfloat16, device=dev) if with_cublas else None
        w8b = wb.to(torch.float8_e4m3fn) if with_cublas else None
        for m in ms:
            xb = inputs.make_activation(m, k, 7000 + m, OUTLIER_FRAC, OUTLIER_MULT)
            x = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev)
            x8, s_x = binding.quantize_act(x)
            y = torch.empty((m, n), dtype=torch.bfloat16, device=dev)
            ws = binding.new_workspace(m, n, k, tws[0].fmt, dev)
            reps = copies if m <= 512 else max(2, copies // 4)

            def lin(c):
                binding.linear_tiled(x8, s_x, tws[c % copies], out=y, workspace=ws)

            def whole(c):
                binding.quantize_act(x, out=(x8, s_x))
                lin(c)
            t_lin = graph_time(lin, reps)
            t_all = graph_time(whole, reps)
            t_chain = None
            if m <= binding.CHAIN_MAX_M:
                # the same layer as problems of one persistent launch (quantization included)
                nprob = min(binding.CHAIN_MAX_PROBLEMS, max(copies, 8))
                chain = binding.LinearChain([dict(x=x, weight=tws[c % copies], y=y) for c in range(nprob)])
                t_chain = _time_loop(torch, chain, 10, warm=3) / nprob
                del chain
            flops = 2.0 * m * n * k
            t_roof = max(linear_algorithmic_bytes(m, n, k) / hbm, flops / fp8_peak)
            row = {"layer": name, "K": k, "N": n, "M": m, "linear_us": t_lin * 1e6, "quant_plus_linear_us": t_all * 1e6,
                   "tflops": flops / t_lin / 1e12, "weight_GBps": wbytes / t_lin / 1e9,
                   "roofline_us": t_roof * 1e6, "frac_of_roofline": t_roof / t_lin,
                   "bound": "hbm" if linear_algorithmic_bytes(m, n, k) / hbm > flops / fp8_peak else "tensor"}
            if t_chain is not None:
                row["chain_us_per_problem"] = t_chain * 1e6
                row["chain_frac_of_roofline"] = chain_algorithmic_bytes((m,), n, k) / hbm / t_chain
            if with_cublas:
                row["cublas_bf16_us"] = graph_time(lambda c: torch.matmul(x, wb.t()), 4) * 1e6
                # W8A8 with the library's FP8 GEMM (FP8 weights read as they are: twice the bytes, no
                # expansion): the same-box counterpart of the paper's W8A8 comparison
                try:
                    a8 = x.to(torch.float8_e4m3fn)
                    one = torch.ones((), device=dev, dtype=torch.float32)
                    row["library_w8a8_fp8_us"] = graph_time(
                        lambda c: torch._scaled_mm(a8, w8b.t(), scale_a=one, scale_b=one,
                                                   out_dtype=torch.bfloat16), 4) * 1e6
                except Exception:
                    row["library_w8a8_fp8_us"] = None
            out.append(row)
            del x, x8, s_x, y, ws
        del tws, wb, w8b
        torch.cuda.empty_cache()
    if binding.query_device_status() != 0:
        raise RuntimeError("device status word set during the sweep")
    return out


def mlp_sweep(torch, binding, inputs, dev, peaks):
    """The MLP block of a Llama-3-8B decoder layer at decode sizes, all on the W4A8 path:
    quantize_act(x) -> stacked gate/up projection (K = 4096 -> N = 2 x 14336) -> silu(gate) * up fused
    with the activation quantization of the next layer (w4a8_silu_mul_quantize) -> down projection
    (K = 14336 -> N = 4096).  Per token count: the block as two dependent problems of a w4a8_linear_chain
    launch (eight blocks per launch), the block time of the per-launch kernels from CUDA graphs of
    consecutive blocks on rotating weight copies (more than twice the L2), the same with the activation
    written as BF16 and quantized by a separate launch, and the BF16 library block (two torch.matmul +
    silu * mul)."""
    H, F = 4096, 14336
    out = []
    side = torch.cuda.Stream()

    def graph_time(fn, reps):
        fn(0)
        torch.cuda.synchronize()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for c in range(reps):
                    fn(c)
        torch.cuda.current_stream().wait_stream(side)
        return _time_loop(torch, g.replay, 5, warm=2) / reps

    copies = 4   # 4 x (60.6 + 30.3) MB of packed weights > 2 x 126 MB
    gus, downs = [], []
    for c in range(copies):
        W = torch.from_numpy(inputs.make_weight(2 * F, H, SIGMA, seed=9100 + c)).to(dev)
        gus.append(binding.prepack_weight(*binding.quantize_weight_rtn(W, symmetric=True)))
        del W
        W = torch.from_numpy(inputs.make_weight(H, F, SIGMA, seed=9200 + c)).to(dev)
        downs.append(binding.prepack_weight(*binding.quantize_weight_rtn(W, symmetric=True)))
        del W
    wbytes = (2 * F * H + H * F) * (0.5 + 2.0 / GROUP)
    wg_bf = torch.randn((2 * F, H), dtype=torch.bfloat16, device=dev) * SIGMA
    wd_bf = torch.randn((H, F), dtype=torch.bfloat16, device=dev) * SIGMA
    for m in (1, 4, 16):
        x = torch.from_numpy(inputs.make_activation(m, H, 77 + m, OUTLIER_FRAC, OUTLIER_MULT)).to(dev).view(torch.bfloat16)
        x8, s_x = binding.quantize_act(x)
        gu = torch.empty((m, 2 * F), dtype=torch.bfloat16, device=dev)
        h8 = torch.empty((m, F), dtype=torch.uint8, device=dev)
        s_h = torch.empty((m,), dtype=torch.float32, device=dev)
        hbf = torch.empty((m, F), dtype=torch.bfloat16, device=dev)
        y = torch.empty((m, H), dtype=torch.bfloat16, device=dev)
        ws1 = binding.new_workspace(m, 2 * F, H, gus[0].fmt, dev)
        ws2 = binding.new_workspace(m, H, F, downs[0].fmt, dev)

        def block(c):
            binding.quantize_act(x, out=(x8, s_x))
            binding.linear_tiled(x8, s_x, gus[c % copies], out=gu, workspace=ws1)
            binding.silu_mul_quantize(gu, out=(h8, s_h))
            binding.linear_tiled(h8, s_h, downs[c % copies], out=y, workspace=ws2)

        def block_unfused(c):
            binding.quantize_act(x, out=(x8, s_x))
            binding.linear_tiled(x8, s_x, gus[c % copies], out=gu, workspace=ws1)
            torch.mul(torch.nn.functional.silu(gu[:, :F]), gu[:, F:], out=hbf)
            binding.quantize_act(hbf, out=(h8, s_h))
            binding.linear_tiled(h8, s_h, downs[c % copies], out=y, workspace=ws2)

        def block_bf16(c):
            g2 = torch.matmul(x, wg_bf.t())
            torch.matmul(torch.nn.functional.silu(g2[:, :F]) * g2[:, F:], wd_bf.t())

        # The same blocks as ONE w4a8_linear_chain launch: per block a gate/up problem and a down
        # problem of the gated kind that depends on it (Eq. 13 of silu(gate) * up inside the kernel);
        # every block of the launch has its own gate/up buffer, because a CTA that is ahead may write
        # the next block's while another still reads this one's.
        nblk = 2 * copies
        gus_out = [torch.empty((m, 2 * F), dtype=torch.bfloat16, device=dev) for _ in range(nblk)]
        probs = []
        for b in range(nblk):
            probs.append(dict(x=x, weight=gus[b % copies], y=gus_out[b]))
            probs.append(dict(x=gus_out[b], weight=downs[b % copies], y=y, kind=binding.CHAIN_INPUT_SILU_MUL,
                              depends_on=2 * b))
        chain = binding.LinearChain(probs)
        t_c = _time_loop(torch, chain, 10, warm=3) / nblk

        t = graph_time(block, 2 * copies)
        t_u = graph_time(block_unfused, 2 * copies)
        t_b = graph_time(block_bf16, 4)
        if binding.query_device_status() != 0:
            raise RuntimeError("device status word set")
        out.append({"M": m, "block_chain_us": t_c * 1e6, "block_per_launch_us": t * 1e6,
                    "block_unfused_activation_us": t_u * 1e6,
                    "chain_weight_GBps": wbytes / t_c / 1e9, "chain_frac_hbm_measured": wbytes / t_c / 1e9 / peaks["hbm_gbs"],
                    "per_launch_frac_hbm_measured": wbytes / t / 1e9 / peaks["hbm_gbs"],
                    "library_bf16_block_us": t_b * 1e6})
    return out


def tp_sweep(torch, binding, inputs, dev, peaks, rank, world):
    """The tensor-parallel MLP block of Llama-3-8B (H = 4096, F = 14336) at decode sizes.
    One process: for TP degrees 1, 2, 4, 8 the time one rank spends on its shard (column-parallel
    gate/up, fused activation + quantization, row-parallel down; no exchange), from CUDA graphs that
    rotate over the shards of all ranks of several full layers (more than twice the L2 in total).
    Several processes (one per GPU): TP degree = world size, the whole block with its NCCL
    all-reduce of the BF16 partial outputs, max over ranks."""
    from paper_2505_14638_b200 import tp
    H, F = 4096, 14336
    layers = 3      # 3 x 90.8 MB of packed weights > 2 x 126 MB
    full = []
    for c in range(layers):
        W = torch.from_numpy(inputs.make_weight(2 * F, H, SIGMA, seed=9300 + c)).to(dev)
        gu = tp.Weights(*binding.quantize_weight_rtn(W, symmetric=True))
        del W
        W = torch.from_numpy(inputs.make_weight(H, F, SIGMA, seed=9400 + c)).to(dev)
        down = tp.Weights(*binding.quantize_weight_rtn(W, symmetric=True))
        del W
        full.append((gu, down))
    ops = tp.CudaOps()
    side = torch.cuda.Stream()
    out = []
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    degrees = (world,) if world > 1 else (1, 2, 4, 8)
    for t in degrees:
        ex = tp.Exchange(world=t)
        ranks = (rank,) if world > 1 else tuple(range(t))
        blocks = [tp.TPMlpBlock(gu, down, r, t, ops=ops, exchange=ex) for gu, down in full for r in ranks]
        shard_bytes = (2 * F * H + H * F) * (0.5 + 2.0 / GROUP) / t
        for m in (1, 4, 16):
            x = torch.from_numpy(inputs.make_activation(m, H, 88 + m, OUTLIER_FRAC, OUTLIER_MULT)).to(dev).view(torch.bfloat16)
            fn = (lambda b: b.forward(x)) if world > 1 else (lambda b: b.partial(x))
            for b in blocks:
                fn(b)
            torch.cuda.synchronize()
            side.wait_stream(torch.cuda.current_stream())
            g = torch.cuda.CUDAGraph()
            reps = 2 * len(blocks) if world == 1 else 8 * len(blocks)
            with torch.cuda.stream(side):
                with torch.cuda.graph(g, stream=side):
                    for i in range(reps):
                        fn(blocks[i % len(blocks)])
            torch.cuda.current_stream().wait_stream(side)
            if dist is not None:
                dist.barrier()
            sec = _time_loop(torch, g.replay, 5, warm=2) / reps
            sec = max_over_ranks([sec], dist, dev)[0]
            row = {"tp": t, "M": m, "rank_shard_MB": shard_bytes / 1e6, "weight_GBps_per_rank": shard_bytes / sec / 1e9,
                   "frac_hbm_measured": shard_bytes / sec / 1e9 / peaks["hbm_gbs"]}
            row["block_with_allreduce_us" if world > 1 else "rank_compute_us"] = sec * 1e6
            out.append(row)
    if binding.query_device_status() != 0:
        raise RuntimeError("device status word set during the sweep")
    if dist is not None:
        dist.destroy_process_group()
    return out


def scheme_sweep(torch, binding, inputs, dev):
    """Same-box counterpart of the paper's scheme comparison (Sec. 4.3, Fig. 4, Table 3): per layer
    and token count the time of W4A8 as built here (group-aware order: groups are runs of columns),
    of W8A8 (FP8 weights, own kernel and the library's FP8 GEMM), of W4A16 (own kernel) and of W4A8 quantized in an
    unconstrained activation order (per-column group index), both as two launches (the FP8 weights
    materialised by w4a8_dequant_weight_gidx, then a W8A8 GEMM) and as one kernel with the look-up
    inside (w4a8_linear_gidx), next to the same tile kernel on the group-aware order.  CUDA graphs,
    rotating weights."""
    out = []
    side = torch.cuda.Stream()

    def graph_time(fn, reps):
        fn(0)
        torch.cuda.synchronize()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for c in range(reps):
                    fn(c)
        torch.cuda.current_stream().wait_stream(side)
        return _time_loop(torch, g.replay, 5, warm=2) / reps

    for name, k, n in C5_LAYERS:
        copies = max(2, min(16, int(2.2 * 126e6 / (n * k)) + 1))     # FP8 copies: 1 byte per weight
        tws, w8s, raw, tw8s = [], [], [], []
        for c in range(copies):
            W = torch.from_numpy(inputs.make_weight(n, k, SIGMA, seed=8000 + c)).to(dev)
            q = binding.quantize_weight_rtn(W, symmetric=True)
            tws.append(binding.prepack_weight(*q))
            w8s.append(binding.dequant_weight(*q[:3]))
            tw8s.append(binding.prepack_fp8(w8s[-1], q[3]))
            raw.append(q)
            del W
        g_idx = (torch.randperm(k, device=dev) // GROUP).to(torch.int32)   # an unconstrained column order
        w8_tmp = torch.empty((n, k), dtype=torch.uint8, device=dev)
        one = torch.ones((), device=dev, dtype=torch.float32)
        for m in (1, 16, 128, 2048):
            xb = inputs.make_activation(m, k, 8000 + m, OUTLIER_FRAC, OUTLIER_MULT)
            x = torch.from_numpy(xb.view(np.int16)).view(torch.bfloat16).to(dev)
            x8, s_x = binding.quantize_act(x)
            a8 = x8.view(torch.float8_e4m3fn)
            y = torch.empty((m, n), dtype=torch.bfloat16, device=dev)
            ws = binding.new_workspace(m, n, k, tws[0].fmt, dev)
            reps = copies if m <= 128 else max(2, copies // 2)
            t_w4 = graph_time(lambda c: binding.linear_tiled(x8, s_x, tws[c % copies], out=y, workspace=ws), reps)
            t_w8 = graph_time(lambda c: binding.linear_w8a8(x8, s_x, w8s[c % copies], raw[0][3], out=y), reps)

            def act_order(c):
                cq = raw[c % copies]
                binding.dequant_weight_gidx(cq[0], cq[1], None, g_idx, out=w8_tmp)
                binding.linear_w8a8(x8, s_x, w8_tmp, cq[3], out=y)
            t_ao = graph_time(act_order, reps)
            # the same scheme in ONE kernel: per-weight scale look-up inside the canonical-layout tile kernel,
            # next to that kernel on the group-aware (consecutive) order of the same layer
            t_aof = graph_time(lambda c: binding.linear_gidx(x8, s_x, raw[c % copies][0], raw[c % copies][1], None,
                                                             g_idx, raw[c % copies][3], out=y), reps)
            t_tile = graph_time(lambda c: binding.linear(x8, s_x, raw[c % copies][0], raw[c % copies][1], None,
                                                         raw[c % copies][3], algo=binding.ALGO_UMMA, out=y), reps)
            t_lib = graph_time(lambda c: torch._scaled_mm(a8, w8s[c % copies].view(torch.float8_e4m3fn).t(),
                                                          scale_a=one, scale_b=one, out_dtype=torch.bfloat16), reps)

            ws16 = torch.empty((max(binding.lib().w4a8_linear_w4a16_workspace_bytes(m, n, k), 16),),
                               dtype=torch.uint8, device=dev)

            def w4a16(c):
                cq = raw[c % copies]
                binding.linear_w4a16(x, cq[0], cq[1], None, cq[3], out=y, workspace=ws16)
            t_16 = graph_time(w4a16, reps)
            # the same scheme on the persistent prefill kernel of the W4A8 path (prepacked weights, whole tiles):
            # the like-for-like partner of the W4A8 column at prefill sizes
            t_16p = None
            if m >= 128:
                t_16p = graph_time(lambda c: binding.linear_w4a16_tiled(x, tws[c % copies], out=y), reps)
            # decode sizes: both schemes as problems of a w4a8_linear_chain launch (same kernel, partition and
            # MMAs; the FP8 weights are copied to tensor memory where the INT4 codes are expanded)
            t_c4 = t_c8 = None
            if m <= binding.CHAIN_MAX_M:
                nprob = 12
                yc = torch.empty((m, n), dtype=torch.bfloat16, device=dev)
                c4 = binding.LinearChain([dict(x=x, weight=tws[j % copies], y=yc) for j in range(nprob)])
                c8 = binding.LinearChain([dict(x=x, weight=tw8s[j % copies], y=yc) for j in range(nprob)])
                t_c4 = _time_loop(torch, c4, 10, warm=3) / nprob
                t_c8 = _time_loop(torch, c8, 10, warm=3) / nprob
                del c4, c8
            out.append({"layer": name, "K": k, "N": n, "M": m, "w4a8_us": t_w4 * 1e6, "w8a8_own_kernel_us": t_w8 * 1e6,
                        "w8a8_library_us": t_lib * 1e6, "w4a8_act_order_dequant_plus_w8a8_us": t_ao * 1e6,
                        "w4a8_act_order_one_kernel_us": t_aof * 1e6, "w4a8_same_tile_kernel_group_order_us": t_tile * 1e6,
                        "w4a16_own_kernel_us": t_16 * 1e6,
                        "w4a16_persistent_kernel_us": None if t_16p is None else t_16p * 1e6,
                        "w4a8_chain_us_per_problem": None if t_c4 is None else t_c4 * 1e6,
                        "w8a8_chain_us_per_problem": None if t_c8 is None else t_c8 * 1e6})
            del x, x8, s_x, y, ws
        del tws, w8s, raw, w8_tmp, tw8s
        torch.cuda.empty_cache()
    if binding.query_device_status() != 0:
        raise RuntimeError("device status word set during the sweep")
    return out


def _inverse_factor(Hp):
    """Upper Cholesky factor of the inverse of the prepared Hessian (the output of w4a8_hessian_prepare;
    Sec. 3.3, as in GPTQ), with torch.linalg in float64: the library step between the Hessian and
    w4a8_dpq_quantize, which is the caller's."""
    import torch
    Hinv = torch.cholesky_inverse(torch.linalg.cholesky(Hp.to(torch.float64)))
    Hinv = 0.5 * (Hinv + Hinv.T)
    return torch.linalg.cholesky(Hinv, upper=True).to(torch.float32).contiguous()


def dpq_sweep(torch, binding, inputs, dev):
    """Offline DPQ quantizer (Algorithm 1 with Group-Aware Reordering and an 6-step scale search)
    on Llama-3-8B layer shapes: device time of w4a8_dpq_quantize against the plain-ALU roofline of
    its N K^2 / 2 dependent fused multiply-adds (Eq. 12), the oracle timed on a slab of rows."""
    import oracle
    rows = []
    fma_peak = 148 * 128 * 1.965e9      # FP32 FMA lanes x SMs x max SM clock
    for name, k, n in (("o", 4096, 4096), ("gate_up", 4096, 28672), ("down", 14336, 4096)):
        W = torch.from_numpy(inputs.make_weight(n, k, SIGMA, seed=9000)).to(dev)
        xb = inputs.make_activation(1024, k, 9001, OUTLIER_FRAC, OUTLIER_MULT)
        X = torch.from_numpy(inputs.bf16_bits_to_f32(xb)).to(dev)
        X = (X + 0.5 * torch.randn((1024, 1), dtype=torch.float32, device=dev)).to(torch.bfloat16)   # calibration tokens
        binding.hessian_accumulate(X)             # warm-up
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        H = binding.hessian_accumulate(X)         # H = X^T X (Sec. 3.1)
        perm = binding.gar_permutation(torch.diagonal(H).contiguous())
        Hp = binding.hessian_prepare(H, perm, damp=0.01)     # processing order, dead features, dampening (Sec. 3.3)
        torch.cuda.synchronize()
        t_hess = time.perf_counter() - t0
        U = _inverse_factor(Hp)   # the caller's library step: the factor is an input of the quantizer
        torch.cuda.synchronize()
        t_prep = time.perf_counter() - t0
        binding.dpq_quantize(W, U, perm, symmetric=False, mse_steps=6)   # warm-up
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        q = binding.dpq_quantize(W, U, perm, symmetric=False, mse_steps=6)
        b.record()
        torch.cuda.synchronize()
        t = a.elapsed_time(b) * 1e-3
        fmas = n * k * (k - 128) / 2.0 + n * k * 64.0      # trailing updates + updates inside the blocks
        # the oracle on a slab of rows (rows are independent), same U and order
        # (the slab holds the row with the tensor's absolute maximum, so that Eq. 6 gives both the same s_w)
        top = int(torch.argmax(W.abs().amax(dim=1)))
        ridx = torch.unique(torch.cat([torch.arange(63, device=dev), torch.tensor([top], device=dev)]))
        slab = int(ridx.numel())
        Wh, Uh, ph = W[ridx].cpu().numpy(), U.cpu().numpy(), perm.cpu().numpy()
        c0 = time.perf_counter()
        ref = oracle.dpq_quantize(Wh, Uh, ph, symmetric=False, mse_steps=6)
        t_cpu = time.perf_counter() - c0
        same = bool(np.array_equal(q[0][ridx].cpu().numpy(), ref[0]))
        rows.append({"layer": name, "K": k, "N": n, "dpq_ms": t * 1e3, "fma_per_s": fmas / t,
                     "frac_of_fp32_fma_peak": fmas / t / fma_peak, "hessian_and_factor_s": t_prep, "hessian_kernels_s": t_hess,
                     "oracle_slab_rows": slab, "oracle_slab_s": t_cpu, "oracle_full_layer_s_extrapolated":
                         t_cpu * n / slab, "oracle_cores": oracle.num_threads(), "slab_codes_equal": same})
        del W, X, H, U, q
        torch.cuda.empty_cache()
    return rows


def spawn_ranks(n):
    """`bench.py --gpus N` started without a launcher: re-run this command line under
    torch.distributed.run with one rank per GPU of this node (rendezvous on 127.0.0.1) and return its
    exit code.  Fails loudly when the node has fewer GPUs than asked for."""
    import socket
    import torch
    have = torch.cuda.device_count()
    if have < n:
        raise SystemExit("--gpus %d asked for, but this node has %d CUDA device(s)" % (n, have))
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        port = so.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the prefill / per-M detail sections")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip timing the CPU oracle")
    ap.add_argument("--steps-per-launch", type=int, default=8,
                    help="consecutive steps carried by one w4a8_linear_chain launch (3 problems per step, at most 24 "
                         "problems per launch; steps left over run in one shorter launch; default 8)")
    ap.add_argument("--prefill-only", action="store_true",
                    help="run only the c3 prefill section (small enough for a profiler capture) and print it")
    ap.add_argument("--sweep", default=None, choices=["c5", "c4", "dpq", "schemes", "mlp", "tp"],
                    help="instead of the bench line, print the per-layer table of config c5 (four Llama-3-8B "
                         "linears x M) or the single c4 case (M=8192, K=8192, N=28672)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.sweep:
        import torch
        from paper_2505_14638_b200 import binding, inputs
        from paper_2505_14638_b200 import build as _build
        _build.build()
        torch.cuda.set_device(local_rank)
        dev = torch.device("cuda", local_rank)
        if args.sweep == "dpq":
            rows = dpq_sweep(torch, binding, inputs, dev)
        elif args.sweep == "schemes":
            rows = scheme_sweep(torch, binding, inputs, dev)
        elif args.sweep == "mlp":
            rows = mlp_sweep(torch, binding, inputs, dev, load_peaks())
        elif args.sweep == "tp":
            rows = tp_sweep(torch, binding, inputs, dev, load_peaks(), rank, world)
            if rank != 0:
                return
        elif args.sweep == "c5":
            rows = layer_sweep(torch, binding, inputs, dev, load_peaks())
        else:
            rows = layer_sweep(torch, binding, inputs, dev, load_peaks(), layers=(("c4", 8192, 28672),), ms=(8192,))
        print(json.dumps({"sweep": args.sweep, "rows": rows}), flush=True)
        return
    if args.prefill_only:
        import torch
        from paper_2505_14638_b200 import binding, inputs
        from paper_2505_14638_b200 import build as _build
        _build.build()
        torch.cuda.set_device(local_rank)
        print(json.dumps({"prefill": prefill_extra(torch, binding, inputs, torch.device("cuda", local_rank),
                                                   load_peaks())}), flush=True)
        return
    if "WORLD_SIZE" in os.environ:
        if world != args.gpus:
            raise SystemExit("--gpus %d does not match WORLD_SIZE %d" % (args.gpus, world))
    elif args.gpus > 1:
        raise SystemExit(spawn_ranks(args.gpus))   # no launcher: start the N ranks ourselves
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
