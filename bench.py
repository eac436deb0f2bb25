#!/usr/bin/env python
"""Benchmark of the IKBO hot path on B200.

One step = one pass of the retrieval-MLP workload (configuration 2: R = 256 requests x 512
candidates, 768 -> 1024 -> 1024 -> 256, first layer split 512 | 256 between request and candidate
features): segment plan, request half, candidate half with the in-kernel broadcast, and the two
plain layers.  `value` is candidates scored per second over all ranks with inputs resident in HBM;
`e2e` is the same step from pinned host buffers (inputs copied in, scores copied out every step).
`roofline` describes the IKBO layer of that step (layer 1: request half + candidate half);
`dominant_launch` the launch with the largest share of the step.  Extra keys report every layer against
its own roofline and the other IKBO kernels on their own workloads (attention: configuration 3,
n_q = 32 / 64 query tokens; interaction, projected FM, group norm: configuration 4 / 2 shapes;
configuration 5: all three calls), each with a materialised-broadcast GPU comparator and with the cost
of a fresh segment plan; `summary`, the last key, repeats the headline figures in compact form.

With --gpus N > 1 and no torchrun environment the script starts itself under torch.distributed.run.
The global batch is N copies of the configuration's requests, split by request over the ranks with
`sharding.shard_batch` (weights replicated, no collective on the data path, NCCL only for the timing
barrier and the max over ranks): weak scaling.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl rocs|reference]

`--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2607_27744_b200 import sharding, workloads as wl  # noqa: E402

METRIC = "candidates scored/sec per IKBO layer (bf16, 1 B200) and % of roofline"
UNIT = "candidates/s"
WORKLOAD = "config 2: retrieval MLP bf16, R=256 x 512 candidates (N=131072), 768->1024->1024->256, layer 1 split 512|256"
N_SETS = 4  # rotating input/output sets: 4 x (67 MB in + 600 MB activations) >> 126 MB L2
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under
# profiles/ (bytes; the request half of layer 1 adds 1.3 MB).  Below the algorithmic bytes where the
# tail of the output is still in L2 when the kernel ends.
NCU_TRAFFIC = {"L1": 278.8e6 + 1.3e6, "L2": 500.8e6, "L3": 315.5e6}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=p["hbm_gbs"], tflops_burst=p["bf16_tflops"],
                    tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows, self.proc, self.index = [], None, index

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=5)

    def summary(self, t0=None, t1=None):
        """Median SM clock and the throttle reasons seen between host times t0 and t1 (all samples if None)."""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ts, r in self.rows:
            if t0 is not None and not (t0 <= ts <= t1):
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


# --------------------------------------------------------------------------------------------
# reference arm / cpu baseline: the oracle on a bounded sample
# --------------------------------------------------------------------------------------------
def oracle_mlp_rate(n_sample: int, data=None):
    """Times the oracle's three-layer MLP on `n_sample` candidates of configuration 2.
    Returns (candidates per second, threads used, seconds)."""
    from oracle import rocs_ref as ref
    cfg = wl.CONFIGS[2]
    if data is None:
        data = host_inputs(cfg)
    co, lin, ws = data["co"], data["lin"], data["ws"]
    N = int(co[-1])
    sample = np.unique(np.linspace(0, N - 1, n_sample).astype(np.int64))
    t0 = time.perf_counter()
    h = ref.ikbo_linear(co, lin["XR"], lin["XC"], lin["W"], relu=True, sample=sample)
    one = wl.offsets_from_counts([h.shape[0]])
    h = ref.ikbo_linear(one, None, h, wl.to_f64(ws[0]), relu=True)
    ref.ikbo_linear(one, None, h, wl.to_f64(ws[1]))
    dt = time.perf_counter() - t0
    return sample.size / dt, ref.num_threads(), dt


def host_inputs(cfg):
    co = wl.cand_offsets(cfg)
    return dict(co=co, lin=wl.linear_inputs(cfg, co), ws=wl.mlp_weights(cfg))


def sized_oracle_run(data, target_s: float = 12.0):
    rate, threads, dt = oracle_mlp_rate(64, data)
    n = int(max(64, min(int(data["co"][-1]), rate * target_s)))
    rate, threads, dt = oracle_mlp_rate(n, data)
    return rate, threads, dt, n


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    data = host_inputs(wl.CONFIGS[2])
    probe_rate, threads, _ = oracle_mlp_rate(64, data)
    seconds_per_step = min(8.0, 120.0 / max(1, args.steps + args.warmup))   # whole run within a few minutes
    per_step = int(max(8, min(4096, probe_rate * seconds_per_step)))
    for _ in range(args.warmup):
        oracle_mlp_rate(per_step, data)
    t0 = time.perf_counter()
    done = 0
    for _ in range(args.steps):
        oracle_mlp_rate(per_step, data)
        done += per_step
    dt = time.perf_counter() - t0
    value = done / dt
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample_per_step": per_step},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": f"{per_step} evenly spaced candidates of the workload per step, all three layers"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# --------------------------------------------------------------------------------------------
# CUDA arm
# --------------------------------------------------------------------------------------------
def relaunch_under_torchrun(args):
    """`python bench.py --gpus N` without a torchrun environment: start N ranks of this script."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    os.execv(sys.executable, cmd)


def run_rocs(args):
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        relaunch_under_torchrun(args)
    import torch
    from paper_2607_27744_b200 import binding as rocs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    rocs.lib()  # fail loudly if the CUDA library is missing
    peaks = measured_peaks()
    cfg = wl.CONFIGS[2]
    data = host_inputs(cfg)
    # Requests are independent units (Eq. 1 / Eq. 11).  The global batch is `world` copies of the
    # configuration's requests; every rank scores the shard sharding.shard_batch gives it (equal-cost
    # requests: each shard has the single-GPU size), no collective on the data path (weak scaling).
    co_one = data["co"]
    shard = sharding.shard_batch(sharding.replicate_offsets(co_one, world), world, rank)
    co = shard.cand_offsets
    N = int(co[-1])
    xr_host = data["lin"]["XR"][shard.requests % cfg.R]
    xc_host = data["lin"]["XC"][shard.cand_rows % int(co_one[-1])]

    def dev(a):
        t = torch.from_numpy(np.ascontiguousarray(a))
        return (t.view(torch.bfloat16) if a.dtype == np.uint16 else t).cuda()

    def pinned(a):
        t = torch.from_numpy(np.ascontiguousarray(a))
        return (t.view(torch.bfloat16) if a.dtype == np.uint16 else t).pin_memory()

    W1 = dev(data["lin"]["W"])
    W2, W3 = (dev(w) for w in data["ws"])
    W1_cr, W1_cc = W1[:, :cfg.d_req], W1[:, cfg.d_req:]
    co_dev = dev(co)
    XR_sets = [dev(xr_host) for _ in range(N_SETS)]
    XC_sets = [dev(xc_host) for _ in range(N_SETS)]
    h1 = [torch.empty((N, 1024), dtype=torch.bfloat16, device="cuda") for _ in range(N_SETS)]
    h2 = [torch.empty((N, 1024), dtype=torch.bfloat16, device="cuda") for _ in range(N_SETS)]
    y = [torch.empty((N, 256), dtype=torch.bfloat16, device="cuda") for _ in range(N_SETS)]
    workspace = torch.empty(rocs.ikbo_linear_workspace(rocs.plan_create(co_dev, co), 1024), dtype=torch.uint8, device="cuda")
    launches_per_step = 5  # fill_row2req, request half, candidate half, layer 2, layer 3

    def step(i, XR=None, XC=None, co_d=None, marks=None):
        s = i % N_SETS
        if marks is not None:
            marks[0].record()
        plan = rocs.plan_create(co_dev if co_d is None else co_d, co)
        if marks is not None:
            marks[1].record()
        rocs.ikbo_linear(plan, XR_sets[s] if XR is None else XR, XC_sets[s] if XC is None else XC, W1_cr, W1_cc,
                         relu=True, out=h1[s], workspace=workspace)
        if marks is not None:
            marks[2].record()
        rocs.linear(h1[s], W2, relu=True, out=h2[s])
        if marks is not None:
            marks[3].record()
        rocs.linear(h2[s], W3, out=y[s])
        if marks is not None:
            marks[4].record()
        plan.close()
        return y[s]

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        if dist is None:
            return ms
        t = torch.tensor([ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    # ---- device-resident timing -------------------------------------------------------------
    for i in range(args.warmup):
        step(i)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # events between the calls of every 4th timed step: per-layer durations measured INSIDE the timed
    # region, on the stream the kernels run on.  Not on every step: an event between two launches costs
    # about a microsecond and keeps the second kernel from setting itself up while the first one ends
    # (the layers are launched as programmatic dependents of one another).
    mark_every = 4 if args.steps >= 8 else 1
    marks = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(0, args.steps, mark_every)]
    with ClockSampler(local) as clocks:
        time.sleep(0.06)                   # one sample of the idle GPU in front of the region
        t_host0 = time.time()
        e0.record()
        for i in range(args.steps):
            step(i, marks=marks[i // mark_every] if i % mark_every == 0 else None)
        e1.record()
        barrier()
        t_host1 = time.time()
        clock_summary = clocks.summary(t_host0, t_host1)
        clock_summary["sampled"] = "during the timed steps"
        if clock_summary["samples"] < 3:
            # A region of a few milliseconds ends before nvidia-smi reports once: the same step keeps
            # running for 0.7 s and the clocks are read there (load and clocks of the timed steps,
            # sampled right behind them).
            t_pad0 = time.time()
            k = 0
            while time.time() < t_pad0 + 0.7:
                step(k)
                k += 1
            torch.cuda.synchronize()
            clock_summary = clocks.summary(t_pad0, time.time())
            clock_summary["sampled"] = "the timed region is too short to sample: same step repeated for 0.7 s right after it"
    ms = max_over_ranks(e0.elapsed_time(e1))
    rocs.last_device_status()
    ms_per_step = ms / args.steps
    value = world * N / (ms_per_step * 1e-3)
    # A kernel timed in a region of under a second runs at burst clocks: its tensor roof is the burst
    # measurement; only a seconds-long region is held against the sustained (power-capped) one.
    sustained_region = ms >= 1000.0
    tensor_peak = peaks["tflops_sustained"] if sustained_region else peaks["tflops_burst"]
    tensor_peak_name = ("sustained" if sustained_region else "burst") + f" (timed region {ms:.0f} ms)"

    # ---- per-layer durations inside the timed region ------------------------------------------
    def span(a, b):
        return float(np.mean([m[a].elapsed_time(m[b]) for m in marks])) * 1e-3

    t_plan_in, t_l1, t_l2, t_l3 = span(0, 1), span(1, 2), span(2, 3), span(3, 4)

    def span_median(ms_, a, b):
        return float(np.median([m[a].elapsed_time(m[b]) for m in ms_])) * 1e-3

    medians = [span_median(marks, a, a + 1) for a in (1, 2, 3)]
    # the same step on ONE buffer set (inputs and weights stay in L2 as far as they fit): "warm" figures
    warm_marks = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(30)]
    for i in range(3):
        step(0)
    for wm in warm_marks:
        step(0, marks=wm)
    torch.cuda.synchronize()
    warm = [span_median(warm_marks, a, a + 1) for a in (1, 2, 3)]

    # The HBM roof under the same conditions: a plain device copy of one activation (read + write,
    # larger than L2), timed (i) back to back after a pause, as the measured peak was, and (ii) between
    # the steps of a long run, where the power cap has lowered the clocks.  Reported beside the roofline;
    # the roofline's denominator stays the measured peak.
    def copy_gbs(in_step, reps):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for i, (a_, b_) in enumerate(ev):
            if in_step:
                step(i)
            a_.record()
            h2[(i + 1) % N_SETS].copy_(h1[i % N_SETS])
            b_.record()
        torch.cuda.synchronize()
        t_ = float(np.median([a_.elapsed_time(b_) for a_, b_ in ev])) * 1e-3
        return 2.0 * h1[0].numel() * 2 / t_ / 1e9
    time.sleep(0.5)
    copy_alone = copy_gbs(False, 10)
    copy_in_step = copy_gbs(True, min(args.steps, 400))
    hbm_copy = {"alone_gbs": copy_alone, "between_steps_gbs": copy_in_step, "bytes": 2 * h1[0].numel() * 2,

                "note": "torch copy_ of one 131072 x 1024 bf16 activation (read + write); between_steps: median over "
                        "copies placed between the steps of a run of up to 400 steps"}

    def time_call(fn, reps=20, warm=3):
        for i in range(warm):
            fn(i)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(reps):
            fn(i)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps * 1e-3

    t_plan = time_call(lambda i: rocs.plan_create(co_dev, co).close())

    def layer(name, t, flops, nbytes, traffic):
        t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
        t_tc = flops / (tensor_peak * 1e12)
        bound = "hbm" if t_hbm >= t_tc else "tensor"
        ach = nbytes / t / 1e9 if bound == "hbm" else flops / t / 1e12
        peak = peaks["hbm_gbs"] if bound == "hbm" else tensor_peak
        return {"layer": name, "us": t * 1e6, "cand_per_s": N / t, "bound": bound, "achieved": ach, "peak": peak,
                "unit": "GB/s" if bound == "hbm" else "TFLOP/s", "frac": ach / peak,
                "tflops": flops / t / 1e12, "gbs": nbytes / t / 1e9,
                "frac_of_burst_tensor_peak": flops / t / 1e12 / peaks["tflops_burst"],
                "frac_of_sustained_tensor_peak": flops / t / 1e12 / peaks["tflops_sustained"],
                "algorithmic_bytes": nbytes, "traffic": traffic}

    bf = 2
    layers = [
        layer("cfg2.L1 ikbo_linear 512|256->1024 (request half + candidate half)", t_l1,
              2.0 * N * 256 * 1024 + 2.0 * 256 * 512 * 1024,
              N * 256 * bf + N * 1024 * bf + 256 * 512 * bf + 1024 * 768 * bf, NCU_TRAFFIC["L1"]),
        layer("cfg2.L2 linear 1024->1024", t_l2, 2.0 * N * 1024 * 1024, N * 1024 * bf * 2 + 1024 * 1024 * bf,
              NCU_TRAFFIC["L2"]),
        layer("cfg2.L3 linear 1024->256", t_l3, 2.0 * N * 1024 * 256, N * 1024 * bf + N * 256 * bf + 256 * 1024 * bf,
              NCU_TRAFFIC["L3"]),
    ]

    def roofline_of(lay):
        return {"kernel": lay["layer"], "bound": lay["bound"], "achieved": lay["achieved"], "peak": lay["peak"],
                "unit": lay["unit"], "frac": lay["frac"], "traffic": lay["traffic"], "us": lay["us"],
                "peak_source": "of " + peaks["source"] + (", tensor peak: " + tensor_peak_name if lay["bound"] == "tensor" else ""),
                "timed": "CUDA events between the calls of every 4th timed step"}

    roofline = roofline_of(layers[0])                          # the IKBO layer of the metric
    dominant = roofline_of(max(layers, key=lambda l: l["us"]))  # the launch with the largest share of the step

    # ---- materialised-broadcast GPU path for the IKBO layer (reference point) ------------------
    counts_dev = dev(np.diff(co).astype(np.int64))
    t_mat = time_call(lambda i: materialised_linear(torch, XR_sets[i % N_SETS], XC_sets[i % N_SETS], W1, counts_dev), reps=10)
    layers[0]["materialised_broadcast_gpu_us"] = t_mat * 1e6
    layers[0]["speedup_vs_materialised"] = t_mat / t_l1
    # library GEMM (torch.matmul -> cuBLAS) on the plain layers, same buffers: a reference point
    t_lib2 = time_call(lambda i: torch.relu_(torch.matmul(h1[i % N_SETS], W2.t())), reps=10)
    t_lib3 = time_call(lambda i: torch.matmul(h2[i % N_SETS], W3.t()), reps=10)
    layers[1]["library_gemm_relu_us"] = t_lib2 * 1e6
    layers[2]["library_gemm_us"] = t_lib3 * 1e6
    # this library's kernels in the SAME harness as the library GEMMs above (10 back-to-back calls on
    # rotating buffers, burst clocks): the like-for-like figure beside library_gemm_*_us; the "us"
    # of a layer is measured inside the long timed region, at the clocks the power cap leaves
    plan_alone = rocs.plan_create(co_dev, co)
    t_own1 = time_call(lambda i: rocs.ikbo_linear(plan_alone, XR_sets[i % N_SETS], XC_sets[i % N_SETS], W1_cr, W1_cc,
                                                  relu=True, out=h1[i % N_SETS], workspace=workspace), reps=10)
    t_own2 = time_call(lambda i: rocs.linear(h1[i % N_SETS], W2, relu=True, out=h2[i % N_SETS]), reps=10)
    t_own3 = time_call(lambda i: rocs.linear(h2[i % N_SETS], W3, out=y[i % N_SETS]), reps=10)
    plan_alone.close()
    for lay, t_own in zip(layers, (t_own1, t_own2, t_own3)):
        lay["us_alone_burst"] = t_own * 1e6
    # the IKBO layer's fraction when it is not slowed by the power cap of the long run (same bytes, same peak)
    roofline["us_alone_burst"] = layers[0]["us_alone_burst"]
    roofline["frac_alone_burst"] = layers[0]["algorithmic_bytes"] / t_own1 / 1e9 / peaks["hbm_gbs"]
    for lay, med, w in zip(layers, medians, warm):
        lay["us_median"] = med * 1e6            # median over the timed steps (rotating sets: cold L2)
        lay["us_warm_l2"] = w * 1e6             # median of 30 steps on one buffer set

    # ---- end to end from pinned host buffers ------------------------------------------------
    # Every step copies its inputs from pinned host memory and reads its scores back.  The three
    # phases of consecutive steps are pipelined on three streams (copy-in of step i+1 and copy-out of
    # step i-1 run beside the kernels of step i), with two sets of device input buffers and of host
    # output buffers; every step still moves all of its bytes inside the timed region.
    XR_h, XC_h, co_h = pinned(xr_host), pinned(xc_host), pinned(co)
    y_h = [torch.empty((N, 256), dtype=torch.bfloat16).pin_memory() for _ in range(2)]
    in_d = [(torch.empty_like(XR_sets[0]), torch.empty_like(XC_sets[0]), torch.empty_like(co_dev)) for _ in range(2)]
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_run(n_steps):
        in_done = [None, None]
        cmp_done = [None, None]     # kernels of the step that last used input set / output y[s]
        out_done = [None, None]
        for i in range(n_steps):
            b = i % 2
            with torch.cuda.stream(s_in):
                if cmp_done[b] is not None:
                    s_in.wait_event(cmp_done[b])          # input set b is free again
                in_d[b][0].copy_(XR_h, non_blocking=True)
                in_d[b][1].copy_(XC_h, non_blocking=True)
                in_d[b][2].copy_(co_h, non_blocking=True)
                in_done[b] = torch.cuda.Event()
                in_done[b].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(in_done[b])
                if out_done[b] is not None:
                    s_cmp.wait_event(out_done[b])        # y[s] of this parity has been read back
                out = step(b, in_d[b][0], in_d[b][1], in_d[b][2])
                cmp_done[b] = torch.cuda.Event()
                cmp_done[b].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(cmp_done[b])
                y_h[b].copy_(out, non_blocking=True)
                out_done[b] = torch.cuda.Event()
                out_done[b].record(s_out)
        for st in (s_in, s_cmp, s_out):
            torch.cuda.current_stream().wait_stream(st)

    e2e_run(args.warmup)
    barrier()
    e0.record()
    e2e_run(args.steps)
    e1.record()
    barrier()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1)) / args.steps
    h2d = XR_h.numel() * 2 + XC_h.numel() * 2 + co_h.numel() * 4
    d2h = y_h[0].numel() * 2
    # the step's copies alone, both directions at once: what the PCIe link allows for these bytes
    def copies_only(n):
        for i in range(n):
            with torch.cuda.stream(s_in):
                in_d[i % 2][1].copy_(XC_h, non_blocking=True)
                in_d[i % 2][0].copy_(XR_h, non_blocking=True)
            with torch.cuda.stream(s_out):
                y_h[i % 2].copy_(y[i % N_SETS], non_blocking=True)
    copies_only(3)
    torch.cuda.synchronize()
    t_c0 = time.perf_counter()
    copies_only(20)
    torch.cuda.synchronize()
    copies_ms = (time.perf_counter() - t_c0) / 20 * 1e3
    del XR_sets, XC_sets, h1, h2, y, in_d, y_h, XR_h, XC_h
    torch.cuda.empty_cache()

    # ---- the other IKBO kernels on their own workloads (rank 0; the data path has no collective) ----
    extra = []
    if not args.skip_extra and rank == 0:
        extra = bench_other_ops(torch, rocs, peaks, dev, time_call, args.extra.split(","))
    barrier()
    if dist is not None:
        dist.destroy_process_group()
    if rank != 0:
        return
    cpu = None
    if world == 1 and not args.skip_cpu:
        rate, threads, dt, n = sized_oracle_run(data)
        cpu = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": f"{n} evenly spaced candidates of the workload, all three layers, {dt:.1f} s"}

    def brief(l):
        out = {"us": round(l["us"], 1)}
        for k_in, k_out in (("us_alone_burst", "alone"), ("library_gemm_relu_us", "lib"), ("library_gemm_us", "lib"),
                            ("frac", "frac"), ("frac_hbm", "f_hbm"), ("frac_tensor", "f_tc"),
                            ("frac_of_exp_unit_peak_at_max_clock", "f_exp"),
                            ("speedup_vs_materialised", "x_mat"), ("us_with_fresh_plan", "fresh"),
                            ("unfused_us", "unfused")):
            if k_in in l and l[k_in] is not None:
                out[k_out] = round(l[k_in], 3 if k_out.startswith("f") and k_out != "fresh" else 1)
        return out

    legend = ("us: microseconds per call inside the timed region (cfg2.*) or over 20 back-to-back calls (others); "
              "alone: same kernel, 10 back-to-back calls at burst clocks; lib: torch.matmul the same way; "
              "frac / f_hbm / f_tc / f_exp: fraction of the measured HBM, burst tensor and exp-unit roofs; "
              "x_mat: speed-up over the materialised-broadcast GPU path; fresh: us with a new plan per call")
    summary = {"cfg2.L1": brief(layers[0]) | {"bound": layers[0]["bound"]},
               "cfg2.L2": brief(layers[1]) | {"bound": layers[1]["bound"]},
               "cfg2.L3": brief(layers[2]) | {"bound": layers[2]["bound"]}}
    for l in extra:
        summary[l["key"]] = brief(l)
    print(json.dumps({
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "l2": f"{N_SETS} rotating input/activation sets, larger than L2",
                   "step": "plan + request half + candidate half (in-kernel broadcast) + 2 plain layers",
                   "sharding": f"global batch = {world} x the workload's requests, split by request "
                               f"(sharding.shard_batch), {shard.requests.size} requests / {N} candidates per rank"},
        "clocks": clock_summary,
        "e2e": {"value": world * N / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
                "copies_only_ms_per_step": copies_ms, "frac_of_copies_only": copies_ms / e2e_ms,
                "note": "copies_only: the step's host-to-device and device-to-host copies alone, both directions "
                        "at once, no kernels (host clock over 20 steps): the PCIe floor of this step"},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": roofline,
        "dominant_launch": dominant,
        "hbm_copy": hbm_copy,
        "cpu_baseline": cpu,
        "layers": layers,
        "plan_us": t_plan * 1e6, "plan_us_in_step": t_plan_in * 1e6,
        "other_ikbo_layers": extra,
        "summary_legend": legend, "summary": summary,
    }))


def bench_other_ops(torch, rocs, peaks, dev, time_call, which):
    """The other IKBO kernels, one layer each, on their own workloads."""
    out = []
    if "dca" in which:
        out.append(bench_dca(torch, rocs, peaks, dev, time_call))
    if "dh128" in which:
        out.append(bench_dca(torch, rocs, peaks, dev, time_call, dh=128))
    if "dh32" in which:
        out.append(bench_dca(torch, rocs, peaks, dev, time_call, dh=32))
    if "nq" in which:
        out.append(bench_dca_nq(torch, rocs, peaks, dev, time_call, 32))
    if "nq64" in which:
        out.append(bench_dca_nq(torch, rocs, peaks, dev, time_call, 64))
    if "glm" in which:
        out.append(bench_glm(torch, rocs, peaks, dev, time_call))
    if "fm" in which:
        out.append(bench_fm(torch, rocs, peaks, dev, time_call))
    if "norm" in which:
        out.append(bench_norm(torch, rocs, peaks, dev, time_call))
    if "normfused" in which:
        out.append(bench_norm_fused(torch, rocs, peaks, dev, time_call))
    if "cfg5" in which:
        out.extend(bench_cfg5(torch, rocs, peaks, dev, time_call))
    return out


def materialised_linear(torch, XR, XC, W, counts_dev, relu=True):
    """The dense path the paper starts from (Section 4, first paragraph): replicate the request rows
    per candidate, concatenate, one full GEMM.  torch library kernels; a reference point only."""
    u = torch.cat([XR.repeat_interleave(counts_dev, dim=0), XC], dim=1)
    y = u @ W.t()
    return torch.relu_(y) if relu else y


def materialised_linear_chunked(torch, XR, XC, W, row2req, chunk=1 << 18):
    """The same in candidate chunks, for batches whose materialised input does not fit at once."""
    for a in range(0, XC.shape[0], chunk):
        b = min(XC.shape[0], a + chunk)
        u = torch.cat([XR[row2req[a:b]], XC[a:b]], dim=1)
        y = u @ W.t()
    return y


def materialised_dca(torch, Q, K, V, co, so, chunk_bytes=4 << 30, requests=None):
    """Candidate-batched copies of K/V, then library attention (Section 4.3, second paragraph),
    request by request in chunks so the copies fit in memory; `requests` restricts it to a sample."""
    N, n_q, H, dh = Q.shape
    O = torch.empty_like(Q)
    for r in (range(len(co) - 1) if requests is None else requests):
        c0, c1, s0, s1 = int(co[r]), int(co[r + 1]), int(so[r]), int(so[r + 1])
        if c1 == c0 or s1 == s0:
            continue
        per_cand = 2 * (s1 - s0) * H * dh * 2
        step = max(1, int(chunk_bytes // per_cand))
        k = K[s0:s1].permute(1, 0, 2)  # [H, L, dh]
        v = V[s0:s1].permute(1, 0, 2)
        for a in range(c0, c1, step):
            b = min(c1, a + step)
            kk = k.unsqueeze(0).expand(b - a, -1, -1, -1).contiguous()   # the materialised broadcast
            vv = v.unsqueeze(0).expand(b - a, -1, -1, -1).contiguous()
            q = Q[a:b].permute(0, 2, 1, 3)
            O[a:b] = torch.nn.functional.scaled_dot_product_attention(q, kk, vv).permute(0, 2, 1, 3)
    return O


def materialised_glm(torch, XR, XC, W, counts_dev, n_r, n_ro):
    """X = [X^R[m_i]; X^C[i]] per candidate, G = X X^T, block mask, O = W~ G (Eq. 9-10, Eq. 5-6)."""
    X = torch.cat([XR.repeat_interleave(counts_dev, dim=0), XC], dim=1)
    G = torch.bmm(X, X.transpose(1, 2))
    G[:, :n_r, n_r:] = 0
    Wm = W.clone()
    Wm[:n_ro, n_r:] = 0
    return torch.matmul(Wm, G)


def materialised_glm_rows_chunked(torch, XR, XC, row2req, chunk=1 << 17):
    """Candidate rows of the masked interaction from the materialised X, in candidate chunks."""
    for a in range(0, XC.shape[0], chunk):
        b = min(XC.shape[0], a + chunk)
        X = torch.cat([XR[row2req[a:b]], XC[a:b]], dim=1)
        G = torch.bmm(XC[a:b], X.transpose(1, 2))
    return G


def with_fresh_plan(rocs, time_call, co_dev, co, call, reps=5):
    """The same call when the batch is new: segment plan (request ids, work list) built in front of it."""
    def once(i):
        plan = rocs.plan_create(co_dev, co)
        call(plan)
        plan.close()
    return time_call(once, reps=reps)


def dca_record(key, name, cfg, N, co, so, t, t_fresh, t_mat, peaks, rows_per_cand=1, mat_note=None):
    pairs = float(np.sum(np.diff(co).astype(np.float64) * np.diff(so))) * rows_per_cand
    flops = 4.0 * pairs * cfg.H * cfg.dh
    rec = {"key": key, "layer": name, "N": N, "us": t * 1e6, "us_with_fresh_plan": t_fresh * 1e6,
           "cand_per_s": N / t, "tflops": flops / t / 1e12,
           "frac_tensor": flops / t / 1e12 / peaks["tflops_burst"],
           "frac_tensor_sustained": flops / t / 1e12 / peaks["tflops_sustained"],
           "exps_per_s": pairs * cfg.H / t,
           "frac_of_exp_unit_peak_at_max_clock": pairs * cfg.H / t / (148 * 16 * 1.965e9),
           "bound": "tensor (nominal: 4 L H dh flop per candidate against the burst bf16 peak); at dh = 64 the "
                    "exponential unit (16 ex2/clk/SM, one per 256 tensor flops) is the tighter ceiling"}
    if t_mat is not None:
        rec["materialised_broadcast_gpu_us"] = t_mat * 1e6
        rec["speedup_vs_materialised"] = t_mat / t
        if mat_note:
            rec["materialised_note"] = mat_note
    return rec


def bench_dca(torch, rocs, peaks, dev, time_call, dh=64):
    # configuration 3: one DCA layer (dh = 128 / 32: the same width as 4 heads of 128 / 16 of 32, same flops)
    cfg = wl.CONFIGS[3] if dh == 64 else wl.CONFIGS[3].with_(H=8 * 64 // dh, dh=dh)
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    N = int(co[-1])
    d = wl.dca_inputs(cfg, co, so)
    co_dev = dev(co)
    plan = rocs.plan_create(co_dev, co)
    Q, K, V, sod = dev(d["Q"]), dev(d["K"]), dev(d["V"]), dev(so)
    O = torch.empty_like(Q)
    t = time_call(lambda i: rocs.dca_attention(plan, Q, K, V, sod, out=O), reps=10)
    t_fresh = with_fresh_plan(rocs, time_call, co_dev, co, lambda pl: rocs.dca_attention(pl, Q, K, V, sod, out=O), reps=10)
    if dh != 64:
        return dca_record(f"cfg3.dca_dh{dh}", f"cfg3 dca_attention with {cfg.H} heads of {dh} (R=64, L=2048)", cfg, N, co,
                          so, t, t_fresh, None, peaks)
    t_mat = time_call(lambda i: materialised_dca(torch, Q, K, V, co, so), reps=1, warm=1)
    return dca_record("cfg3.dca", "cfg3 dca_attention (R=64, L=2048, 8x64)", cfg, N, co, so, t, t_fresh, t_mat, peaks)


def bench_dca_nq(torch, rocs, peaks, dev, time_call, n_q=32):
    """Multi-token candidate queries (Section 4.3.2): configuration 3 with n_q query tokens per
    candidate and 1/n_q as many candidates per request, so the query rows and flops stay put."""
    base = wl.CONFIGS[3]
    cfg = base.with_(n_q=n_q)
    counts = np.maximum(1, np.diff(wl.cand_offsets(base)) // n_q)
    co, so = wl.offsets_from_counts(counts.tolist()), wl.seq_offsets(base)
    N = int(co[-1])
    d = wl.dca_inputs(cfg, co, so)
    co_dev = dev(co)
    plan = rocs.plan_create(co_dev, co)
    Q, K, V, sod = dev(d["Q"]), dev(d["K"]), dev(d["V"]), dev(so)
    O = torch.empty_like(Q)
    t = time_call(lambda i: rocs.dca_attention(plan, Q, K, V, sod, out=O), reps=10)
    t_fresh = with_fresh_plan(rocs, time_call, co_dev, co, lambda pl: rocs.dca_attention(pl, Q, K, V, sod, out=O), reps=10)
    rec = dca_record(f"cfg3.dca_nq{n_q}", f"cfg3 dca_attention with n_q={n_q} query tokens per candidate (R=64, L=2048, 8x64)",
                     cfg, N, co, so, t, t_fresh, None, peaks, rows_per_cand=n_q)
    rec["query_rows_per_s"] = N * n_q / t
    return rec


def bench_glm(torch, rocs, peaks, dev, time_call):
    # configuration 4: GLM interaction + compression
    cfg = wl.CONFIGS[4]
    co = wl.cand_offsets(cfg)
    N = int(co[-1])
    d = wl.glm_inputs(cfg, co)
    co_dev = dev(co)
    plan4 = rocs.plan_create(co_dev, co)
    XR, XC, W = dev(d["XR"]), dev(d["XC"]), dev(d["W"])
    n = cfg.n_r + cfg.n_c
    outs = {"OC": torch.empty((N, cfg.n_co, n), dtype=torch.bfloat16, device="cuda"),
            "OR": torch.empty((cfg.R, cfg.n_ro, n), dtype=torch.bfloat16, device="cuda")}
    ws = torch.empty(rocs.glm_interaction_workspace(plan4, cfg.n_r, cfg.n_c, cfg.n_co), dtype=torch.uint8, device="cuda")
    call = lambda pl: rocs.glm_interaction(pl, XR, XC, W, cfg.n_ro, cfg.n_co, want_raw=False, workspace=ws, outs=outs)
    t = time_call(lambda i: call(plan4), reps=10)
    t_fresh = with_fresh_plan(rocs, time_call, co_dev, co, call, reps=10)
    nbytes = XC.numel() * 2 + outs["OC"].numel() * 2 + XR.numel() * 2
    flops = N * (2.0 * cfg.n_c * n * cfg.d_emb + 2.0 * cfg.n_co * cfg.n_c * n)
    counts_dev = dev(np.diff(co).astype(np.int64))
    t_mat = time_call(lambda i: materialised_glm(torch, XR, XC, W, counts_dev, cfg.n_r, cfg.n_ro), reps=3)
    return {"key": "cfg4.glm", "layer": "cfg4 glm_interaction 32+16 x128, 48->16 compression (OC only)", "N": N,
            "us": t * 1e6, "us_with_fresh_plan": t_fresh * 1e6,
            "materialised_broadcast_gpu_us": t_mat * 1e6, "speedup_vs_materialised": t_mat / t,
            "cand_per_s": N / t, "gbs": nbytes / t / 1e9, "frac_hbm": nbytes / t / 1e9 / peaks["hbm_gbs"],
            "tflops": flops / t / 1e12, "bound": "hbm",
            "note": "input (537 MB) is larger than L2; same buffers every iteration"}


def materialised_fm(torch, XR, XC, P, counts_dev, n_r):
    """X = [X^R[m_i]; X^C[i]] per candidate, G = X X^T, block mask, F = G P (candidate rows)."""
    X = torch.cat([XR.repeat_interleave(counts_dev, dim=0), XC], dim=1)
    G = torch.bmm(X[:, n_r:], X.transpose(1, 2))
    return torch.matmul(G, P)


def bench_fm(torch, rocs, peaks, dev, time_call):
    # configuration 4 shapes: projected factorization machine, k = 16
    cfg = wl.CONFIGS[4]
    k = 16
    co = wl.cand_offsets(cfg)
    N = int(co[-1])
    d = wl.glm_inputs(cfg, co)
    co_dev = dev(co)
    plan4 = rocs.plan_create(co_dev, co)
    XR, XC, P = dev(d["XR"]), dev(d["XC"]), dev(wl.fm_projection_weight(cfg, k))
    outs = {"FC": torch.empty((N, cfg.n_c, k), dtype=torch.bfloat16, device="cuda"),
            "FR": torch.empty((cfg.R, cfg.n_r, k), dtype=torch.bfloat16, device="cuda")}
    ws = torch.empty(rocs.glm_fm_projection_workspace(plan4, cfg.d_emb, k), dtype=torch.uint8, device="cuda")
    call = lambda pl: rocs.glm_fm_projection(pl, XR, XC, P, workspace=ws, outs=outs)
    t = time_call(lambda i: call(plan4), reps=10)
    t_fresh = with_fresh_plan(rocs, time_call, co_dev, co, call, reps=10)
    nbytes = XC.numel() * 2 + outs["FC"].numel() * 2 + XR.numel() * 2
    flops = N * 4.0 * cfg.n_c * cfg.d_emb * k
    counts_dev = dev(np.diff(co).astype(np.int64))
    t_mat = time_call(lambda i: materialised_fm(torch, XR, XC, P, counts_dev, cfg.n_r), reps=3)
    return {"key": "cfg4.fm", "layer": "cfg4 shapes glm_fm_projection 32+16 x128 -> k=16", "N": N, "us": t * 1e6,
            "us_with_fresh_plan": t_fresh * 1e6,
            "materialised_broadcast_gpu_us": t_mat * 1e6, "speedup_vs_materialised": t_mat / t,
            "cand_per_s": N / t, "gbs": nbytes / t / 1e9, "frac_hbm": nbytes / t / 1e9 / peaks["hbm_gbs"],
            "tflops": flops / t / 1e12, "bound": "hbm",
            "note": "input (537 MB) is larger than L2; same buffers every iteration"}


def bench_norm(torch, rocs, peaks, dev, time_call):
    # group-local RMSNorm (Eq. 7) of the candidate-side activations of configuration 2: 131072 x 1024
    cfg = wl.CONFIGS[2]
    N = cfg.R * cfg.count_const
    g = torch.Generator(device="cuda").manual_seed(7)
    X = torch.randn(N, cfg.d_out, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    gamma = torch.ones(cfg.d_out, dtype=torch.bfloat16, device="cuda")
    Y = torch.empty_like(X)
    t = time_call(lambda i: rocs.group_norm(X, gamma, None, 1e-6, rocs.NORM_RMS, out=Y), reps=20)
    nbytes = 2 * X.numel() * 2
    t_lib = time_call(lambda i: torch.nn.functional.rms_norm(X, (cfg.d_out,), gamma, eps=1e-6), reps=20)
    return {"key": "cfg2.norm", "layer": "cfg2 activations group_norm (RMSNorm, 131072 x 1024)", "N": N, "us": t * 1e6,
            "cand_per_s": N / t, "gbs": nbytes / t / 1e9, "frac_hbm": nbytes / t / 1e9 / peaks["hbm_gbs"],
            "torch_rms_norm_us": t_lib * 1e6, "bound": "hbm",
            "note": "input and output (537 MB) are larger than L2"}


def bench_norm_fused(torch, rocs, peaks, dev, time_call):
    """Configuration 2 with an RMSNorm between layers 1 and 2 (Eq. 7): folded into the two layers (layer 1
    leaves the row sums, layer 2 scales its accumulators) against layer 1, the stand-alone normalisation
    kernel and layer 2."""
    cfg = wl.CONFIGS[2]
    co = wl.cand_offsets(cfg)
    N = int(co[-1])
    lin, ws = wl.linear_inputs(cfg, co), wl.mlp_weights(cfg)
    co_dev = dev(co)
    plan = rocs.plan_create(co_dev, co)
    XR, XC, W1, W2 = dev(lin["XR"]), dev(lin["XC"]), dev(lin["W"]), dev(ws[0])
    W1_cr, W1_cc = W1[:, :cfg.d_req], W1[:, cfg.d_req:]
    gamma = torch.ones(cfg.d_out, dtype=torch.bfloat16, device="cuda")
    h1 = torch.empty((N, cfg.d_out), dtype=torch.bfloat16, device="cuda")
    hn = torch.empty_like(h1)
    h2 = torch.empty((N, 1024), dtype=torch.bfloat16, device="cuda")
    stats = torch.empty((N, 2), dtype=torch.float32, device="cuda")
    wsp = torch.empty(int(rocs.lib().rocs_ikbo_linear_stats_workspace(plan.handle, cfg.d_out)), dtype=torch.uint8, device="cuda")

    def fused(i):
        rocs.ikbo_linear_stats(plan, XR, XC, W1_cr, W1_cc, relu=True, out=h1, row_stats=stats, workspace=wsp)
        rocs.linear_normed(h1, stats, W2, None, None, 1e-6, rocs.NORM_RMS, relu=True, out=h2)

    def unfused(i):
        rocs.ikbo_linear(plan, XR, XC, W1_cr, W1_cc, relu=True, out=h1, workspace=wsp)
        rocs.group_norm(h1, gamma, None, 1e-6, rocs.NORM_RMS, out=hn)
        rocs.linear(hn, W2, relu=True, out=h2)

    t_f, t_u = time_call(fused, reps=20), time_call(unfused, reps=20)
    return {"key": "cfg2.norm_fused", "layer": "cfg2 layers 1-2 with an RMSNorm between them, folded into both layers",
            "N": N, "us": t_f * 1e6, "cand_per_s": N / t_f, "unfused_us": t_u * 1e6, "speedup_vs_unfused": t_u / t_f,
            "note": "unfused = split layer, stand-alone group-norm kernel (reads and writes the 268 MB activation), plain layer"}


def bench_cfg5(torch, rocs, peaks, dev, time_call):
    """Configuration 5 (skewed, Zipf candidate counts): the three calls timed independently, each
    against a materialised-broadcast GPU path."""
    cfg = wl.CONFIGS[5]
    co, so = wl.cand_offsets(cfg), wl.seq_offsets(cfg)
    N = int(co[-1])
    co_dev = dev(co)
    plan = rocs.plan_create(co_dev, co)
    out = []
    g = torch.Generator(device="cuda").manual_seed(5)
    rnd = lambda *shape: torch.randn(*shape, generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    row2req = torch.repeat_interleave(torch.arange(cfg.R, device="cuda"), dev(np.diff(co).astype(np.int64)))
    # linear 768|256 -> 1024
    XR, XC = rnd(cfg.R, cfg.d_req), rnd(N, cfg.d_cand)
    W = (rnd(cfg.d_out, cfg.d_req + cfg.d_cand).float() / 32).to(torch.bfloat16)
    Y = torch.empty((N, cfg.d_out), dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(rocs.ikbo_linear_workspace(plan, cfg.d_out), dtype=torch.uint8, device="cuda")
    call = lambda pl: rocs.ikbo_linear(pl, XR, XC, W[:, :cfg.d_req], W[:, cfg.d_req:], out=Y, workspace=ws)
    t = time_call(lambda i: call(plan), reps=5)
    t_fresh = with_fresh_plan(rocs, time_call, co_dev, co, call)
    nbytes = (XC.numel() + Y.numel() + XR.numel() + W.numel()) * 2
    t_mat = time_call(lambda i: materialised_linear_chunked(torch, XR, XC, W, row2req), reps=2, warm=1)
    out.append({"key": "cfg5.linear", "layer": "cfg5 ikbo_linear 768|256->1024 (Zipf segments)", "N": N, "us": t * 1e6,
                "us_with_fresh_plan": t_fresh * 1e6, "cand_per_s": N / t, "bound": "hbm",
                "gbs": nbytes / t / 1e9, "frac_hbm": nbytes / t / 1e9 / peaks["hbm_gbs"],
                "materialised_broadcast_gpu_us": t_mat * 1e6, "speedup_vs_materialised": t_mat / t})
    del XC, Y
    # attention, L in [256, 1024]
    T = int(so[-1])
    Q, K, V = rnd(N, 1, cfg.H, cfg.dh), rnd(T, cfg.H, cfg.dh), rnd(T, cfg.H, cfg.dh)
    O = torch.empty_like(Q)
    sod = dev(so)
    call = lambda pl: rocs.dca_attention(pl, Q, K, V, sod, out=O)
    t = time_call(lambda i: call(plan), reps=3)
    t_fresh = with_fresh_plan(rocs, time_call, co_dev, co, call, reps=3)
    # the materialised path copies K and V once per candidate (about 2 TB here): timed on every 16th
    # request and scaled by key-candidate pairs
    pairs_r = np.diff(co).astype(np.float64) * np.diff(so)
    sample = list(range(3, cfg.R, 16))
    t_mat_s = time_call(lambda i: materialised_dca(torch, Q, K, V, co, so, requests=sample), reps=1, warm=0)
    t_mat = t_mat_s * float(pairs_r.sum() / max(1.0, pairs_r[sample].sum()))
    out.append(dca_record("cfg5.dca", "cfg5 dca_attention (Zipf segments, L in [256,1024], 8x64)", cfg, N, co, so, t,
                          t_fresh, t_mat, peaks,
                          mat_note="measured on every 16th request, scaled by key-candidate pairs"))
    del Q, K, V, O
    # interaction 24 + 8, no compression
    GR, GC = rnd(cfg.R, cfg.n_r, cfg.d_emb), rnd(N, cfg.n_c, cfg.d_emb)
    n = cfg.n_r + cfg.n_c
    outs = {"YC": torch.empty((N, cfg.n_c, n), dtype=torch.bfloat16, device="cuda"),
            "YR": torch.empty((cfg.R, cfg.n_r, n), dtype=torch.bfloat16, device="cuda")}
    call = lambda pl: rocs.glm_interaction(pl, GR, GC, None, 0, 0, want_raw=True, outs=outs)
    t = time_call(lambda i: call(plan), reps=5)
    t_fresh = with_fresh_plan(rocs, time_call, co_dev, co, call)
    nbytes = (GC.numel() + outs["YC"].numel()) * 2
    t_mat = time_call(lambda i: materialised_glm_rows_chunked(torch, GR, GC, row2req), reps=2, warm=1)
    out.append({"key": "cfg5.glm", "layer": "cfg5 glm_interaction 24+8 x128 (raw YC)", "N": N, "us": t * 1e6,
                "us_with_fresh_plan": t_fresh * 1e6, "cand_per_s": N / t, "bound": "hbm",
                "gbs": nbytes / t / 1e9, "frac_hbm": nbytes / t / 1e9 / peaks["hbm_gbs"],
                "materialised_broadcast_gpu_us": t_mat * 1e6, "speedup_vs_materialised": t_mat / t})
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="rocs", choices=["rocs", "reference"])
    ap.add_argument("--skip-extra", action="store_true", help="skip the attention / interaction side measurements")
    ap.add_argument("--extra", default="dca,dh128,dh32,nq,nq64,glm,fm,norm,normfused,cfg5",
                    help="side measurements to run: dca, dh128, dh32, nq, nq64, glm, fm, norm, normfused, cfg5")
    ap.add_argument("--skip-cpu", action="store_true", help="skip the cpu_baseline leg")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "rocs" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    else:
        run_rocs(args)


if __name__ == "__main__":
    main()
