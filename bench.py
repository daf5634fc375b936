#!/usr/bin/env python
"""Benchmark of the SCAP sparse-FC decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--detail]

Workload (N = 1): the Llama-2-7B-shaped FFN down projection, bf16, batch 1 - W[K=11008, N=4096] ~ N(0, 0.02^2),
inputs silu(g)*u with g, u ~ N(0,1), mode and tau calibrated on 1024 tokens at sparsity targets 50 / 65 / 80 %.
One step = one sparse FC call (one fused kernel: threshold + compaction + gather-GEMV + reduction) per sparsity target on
each of R device copies of W, R chosen so that even the sparsest call pattern touches at least four times the L2 size
per cycle: no call finds its weight rows in L2.
The metric is effective HBM GB/s on the bytes a call must touch (kept rows + activations + mode + bias + output),
summed over the step; the JSON line also carries us/call per sparsity, the library's own dense GEMV on the same
rotation, the speedup over it, the roofline fraction against the measured copy bandwidth, an end-to-end number
through the host-buffer entry point, and the CPU oracle timed on the host cores.

With --gpus N > 1 (launched by torchrun) every rank runs an independent replica of the same work (the path has no
cross-GPU step); the value is the sum over ranks divided by the slowest rank's time.
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

import scap_inputs as si  # noqa: E402

K, N = 11008, 4096
SPARSITIES = (0.5, 0.65, 0.8)
N_INPUTS = 64
NBINS = 2048
T_CALIB = 1024


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


def touched_bytes(nnz: int, B: int = 1) -> int:
    """Algorithmic bytes of one sparse FC call: kept weight rows + x + m + tau + b_fused + y."""
    return nnz * N * 2 + B * K * 2 + 4 * K + 4 + 4 * N + 4 * B * N


def dense_bytes(B: int = 1) -> int:
    return K * N * 2 + B * K * 2 + 4 * N + 4 * B * N


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [c.strip() for c in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for name, col in (("hw_slowdown", 5), ("hw_thermal_slowdown", 6), ("sw_thermal_slowdown", 7), ("sw_power_cap", 8)):
                if f[col].lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_step(d, cal, x_rows, threads: int):
    """One bounded CPU sample: the oracle's sparse FC once per sparsity target (one weight copy)."""
    import oracle
    nbytes = 0
    t0 = time.perf_counter()
    for i, s in enumerate(SPARSITIES):
        m, tau, bf = cal[s]
        xf = si.to_f32(x_rows[i:i + 1], si.BF16)
        oracle.sparse_fc(xf, d["W"], si.BF16, m, tau, bf, threads=threads)
        nbytes += touched_bytes(int(oracle.mask(xf, m, tau)[2].size))
    return time.perf_counter() - t0, nbytes


def oracle_calibration(d):
    import oracle
    xc = si.to_f32(d["x_calib"], si.BF16)
    m = oracle.mode(xc, NBINS)
    cal = {}
    for s in SPARSITIES:
        tau = oracle.tau(xc, m, s)
        cal[s] = (m, tau, oracle.fold_bias(d["W"], si.BF16, m, None).astype(np.float32))
    return cal


def run_reference(args, rank):
    """CPU oracle arm: the same metric on a bounded sample per step, on the host cores."""
    if rank != 0:
        return
    d = si.config1(B=N_INPUTS)
    cal = oracle_calibration(d)
    cores = os.cpu_count() or 1
    for _ in range(args.warmup):
        oracle_step(d, cal, d["x"], cores)
    tot_t, tot_b = 0.0, 0
    for k in range(args.steps):
        t, b = oracle_step(d, cal, d["x"][3 * (k % 20):], cores)
        tot_t += t
        tot_b += b
    val = tot_b / tot_t / 1e9
    line = {
        "impl": "reference", "metric": "sparse_fc_effective_hbm_gbs", "value": val, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama2_7b_down_proj_bf16_b1 (K=11008,N=4096), sparsity 50/65/80%",
                   "sample": "one oracle sparse-FC call per sparsity target per step (3 calls)"},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": cores, "kind": "oracle",
                         "sample": "3 calls per step x %d steps" % args.steps},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--detail", action="store_true", help="also print a per-sparsity table to stderr")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--copies", type=int, default=0,
                    help="number of weight copies to rotate (default: enough for the cold-HBM rule); a small value keeps "
                         "device memory low for a profiler capture and is recorded in config.l2_policy")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    import paper_2412_07174_b200 as scap

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    scap.lib()
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ------------------------------------------------------------------ inputs (seeded, synthetic)
    d = si.config1(B=N_INPUTS)
    dt = si.BF16
    # Cold-HBM rule: every call of a replay must miss L2, also at the highest sparsity, where a call touches only
    # (1 - s) of its weight copy.  So the copies are sized on the smallest touched footprint: R * (1 - s_max) * |W| >= 4 * L2.
    l2 = torch.cuda.get_device_properties(local_rank).L2_cache_size
    R = max(2, int(np.ceil(4 * l2 / ((1.0 - max(SPARSITIES)) * K * N * 2))))
    if args.copies > 0:
        R = args.copies
    W0 = si.as_torch(d["W"], dt).cuda()
    Ws = [W0] + [W0.clone() for _ in range(R - 1)]
    xs = si.as_torch(d["x"], dt).cuda()
    x_calib = si.as_torch(d["x_calib"], dt).cuda()

    # ------------------------------------------------------------------ calibration + bias folding (product path, untimed setup)
    cal_ws = torch.empty(scap.scap_calibrate_workspace(T_CALIB, K, NBINS), dtype=torch.uint8, device="cuda")
    fold_ws = torch.empty(scap.scap_fold_bias_workspace(K, N), dtype=torch.uint8, device="cuda")
    cal = {}
    cal_ms = {}
    for s in SPARSITIES:
        m = torch.empty(K, dtype=torch.float32, device="cuda")
        tau = torch.empty(1, dtype=torch.float32, device="cuda")
        bf = torch.empty(N, dtype=torch.float32, device="cuda")
        scap.scap_calibrate(x_calib, s, NBINS, m, tau, cal_ws)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        scap.scap_calibrate(x_calib, s, NBINS, m, tau, cal_ws)
        e1.record()
        torch.cuda.synchronize()
        cal_ms[s] = e0.elapsed_time(e1)
        scap.scap_fold_bias(W0, m, None, bf, fold_ws)
        cal[s] = (m, tau, bf)
    torch.cuda.synchronize()

    ws = torch.empty(scap.scap_fc_workspace(1, K, N), dtype=torch.uint8, device="cuda")
    y = torch.empty((1, N), dtype=torch.float32, device="cuda")
    nnz_buf = torch.zeros(1, dtype=torch.int32, device="cuda")

    # kept-channel counts of every (sparsity, input) pair: fixes the algorithmic bytes of each call
    nnz = {}
    for s in SPARSITIES:
        m, tau, bf = cal[s]
        cnt = []
        for i in range(N_INPUTS):
            scap.scap_sparse_fc(xs[i:i + 1], Ws[0], m, tau, bf, y, ws, nnz_out=nnz_buf)
            cnt.append(int(nnz_buf.item()))
        nnz[s] = cnt

    stream = torch.cuda.Stream()

    def sparse_calls(s_list, counter):
        nb = 0
        for s in s_list:
            m, tau, bf = cal[s]
            for r in range(R):
                i = counter[0] % N_INPUTS
                counter[0] += 1
                scap.scap_sparse_fc(xs[i:i + 1], Ws[r], m, tau, bf, y, ws)
                nb += touched_bytes(nnz[s][i])
        return nb

    def dense_calls(counter):
        for r in range(R):
            i = counter[0] % N_INPUTS
            counter[0] += 1
            scap.scap_dense_fc(xs[i:i + 1], Ws[r], None, y, ws)
        return R * dense_bytes()

    def capture(fn):
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(stream):
            fn()  # warm outside capture
            stream.synchronize()
            with torch.cuda.graph(g, stream=stream):
                nb = fn()
        return g, nb

    def time_graph(g, reps, warm):
        with torch.cuda.stream(stream):
            for _ in range(warm):
                g.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            stream.synchronize()
            e0.record(stream)
            for _ in range(reps):
                g.replay()
            e1.record(stream)
            stream.synchronize()
        return e0.elapsed_time(e1) / reps  # ms per replay

    g_step, step_bytes = capture(lambda: sparse_calls(SPARSITIES, [0]))
    calls_per_step = len(SPARSITIES) * R
    launches_per_step = calls_per_step  # one fused kernel per call

    # ------------------------------------------------------------------ timed region: K steps, device time, max over ranks
    with torch.cuda.stream(stream):
        for _ in range(args.warmup):
            g_step.replay()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(args.steps):
            g_step.replay()
        e1.record(stream)
    barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    ms_per_step = ms / args.steps
    value = world * step_bytes / (ms_per_step * 1e-3) / 1e9

    # ------------------------------------------------------------------ per-sparsity and dense detail (rank 0 reports)
    detail = {}
    reps = max(20, args.steps // 4)
    for s in SPARSITIES:
        g, nb = capture(lambda s=s: sparse_calls([s], [0]))
        t_ms = time_graph(g, reps, 5)
        detail[s] = {"us_per_call": 1e3 * t_ms / R, "gbs": nb / (t_ms * 1e-3) / 1e9, "bytes_per_call": nb / R,
                     "kept_fraction": float(np.mean(nnz[s][:R])) / K}
    g_dense, nb_dense = capture(lambda: dense_calls([0]))
    t_dense = time_graph(g_dense, reps, 5)
    dense_us = 1e3 * t_dense / R
    dense_gbs = nb_dense / (t_dense * 1e-3) / 1e9

    # ------------------------------------------------------------------ end to end through the host-buffer entry point
    hws = torch.empty(scap.scap_fc_host_workspace(1, K, N), dtype=torch.uint8, device="cuda")
    x_host = si.as_torch(d["x"], dt).pin_memory()
    y_host = torch.zeros((1, N), dtype=torch.float32).pin_memory()

    def host_step(counter):
        for s in SPARSITIES:
            m, tau, bf = cal[s]
            for r in range(R):
                i = counter[0] % N_INPUTS
                counter[0] += 1
                scap.scap_sparse_fc_host(x_host[i:i + 1], Ws[r], m, tau, bf, y_host, hws, stream=stream)
        stream.synchronize()  # the step's result is read on the host

    e2e_steps = max(5, min(args.steps, 50))
    for _ in range(3):
        host_step([0])
    barrier()
    t0 = time.perf_counter()
    ctr = [0]
    for _ in range(e2e_steps):
        host_step(ctr)
    barrier()
    e2e_s = time.perf_counter() - t0
    if world > 1:
        t = torch.tensor([e2e_s], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_s = float(t.item())
    e2e_value = world * step_bytes * e2e_steps / e2e_s / 1e9

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    per_call_s = ms_per_step * 1e-3 / calls_per_step
    achieved = step_bytes / calls_per_step / per_call_s / 1e9
    line = {
        "metric": "sparse_fc_effective_hbm_gbs", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {
            "workload": "llama2_7b_down_proj_bf16_b1 (K=11008,N=4096), sparsity targets 50/65/80%",
            "weights": "bf16", "accumulate": "f32", "batch": 1, "calls_per_step": calls_per_step,
            "l2_policy": "inputs larger than L2: %d weight copies (%.0f MB) rotated so that even the sparsest call pattern touches >= 4x L2 per cycle, %d input vectors" % (R, R * K * N * 2 / 1e6, N_INPUTS),
            "launch": "CUDA graph replay of one step", "parallelism": "replicas only" if world > 1 else "single GPU",
        },
        "us_per_call": {("%d%%" % round(100 * s)): round(detail[s]["us_per_call"], 3) for s in SPARSITIES},
        "gbs_per_sparsity": {("%d%%" % round(100 * s)): round(detail[s]["gbs"], 1) for s in SPARSITIES},
        "kept_fraction": {("%d%%" % round(100 * s)): round(detail[s]["kept_fraction"], 4) for s in SPARSITIES},
        "dense": {"us_per_call": round(dense_us, 3), "gbs": round(dense_gbs, 1)},
        "speedup_vs_dense": {("%d%%" % round(100 * s)): round(dense_us / detail[s]["us_per_call"], 3) for s in SPARSITIES},
        "calibrate_ms": {("%d%%" % round(100 * s)): round(cal_ms[s], 3) for s in SPARSITIES},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "peak_kind": peak_kind, "frac_of_nominal_8000": achieved / 8000.0,
                     "kernel": "fc_kernel (fused threshold + compaction + gather-GEMV + cluster reduction), one launch per call"},
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": calls_per_step * K * 2,
                "d2h_bytes_per_step": calls_per_step * N * 4, "steps": e2e_steps},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
    }

    if not args.no_cpu_baseline and world == 1:
        cores = os.cpu_count() or 1
        cal_o = {s: (cal[s][0].cpu().numpy(), float(cal[s][1].item()), cal[s][2].cpu().numpy()) for s in SPARSITIES}
        tot_t, tot_b, n = 0.0, 0, 0
        while tot_t < 10.0 and n < 2000:
            t, b = oracle_step(d, cal_o, d["x"][3 * (n % 20):], cores)
            tot_t += t
            tot_b += b
            n += 1
        line["cpu_baseline"] = {"value": tot_b / tot_t / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
                                "sample": "%d oracle sparse-FC calls (one per sparsity target, %d rounds), %.1f s" % (3 * n, n, tot_t)}
    if args.detail:
        for s in SPARSITIES:
            print("sparsity %.0f%%: %.2f us/call  %.0f GB/s  kept %.3f" % (100 * s, detail[s]["us_per_call"], detail[s]["gbs"],
                                                                           detail[s]["kept_fraction"]), file=sys.stderr)
        print("dense: %.2f us/call  %.0f GB/s" % (dense_us, dense_gbs), file=sys.stderr)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
