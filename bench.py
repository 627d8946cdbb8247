#!/usr/bin/env python
"""Benchmark of the CSB-RNN hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: one
csb_lstm_forward call over the full sequence of the largest recurrent workload
(two stacked LSTM layers, 8192x4096 CSB weights with 64x64 blocks at ~10x pruning,
512 steps, batch 1).  The headline value is microseconds per timestep.  Beside it
the JSON line carries the roofline of the time-loop kernel, the bare CSB-SpMV sweep
against the HBM roofline, microseconds per timestep of the other workloads, an
end-to-end figure with host buffers, and the float64 oracle timed on the host.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
    torchrun ... bench.py --gpus N ...     (N > 1: independent replicas, no collective)
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
sys.path.insert(0, ROOT)

import workloads  # noqa: E402

METRIC = "us_per_timestep_batch1"
UNIT = "us/timestep"
WORKLOAD = "cfg5: 2-layer LSTM, I=H=2048, 8192x4096 CSB weights, 64x64 blocks, ~10x pruning, T=512, B=1, fp16 values / fp32 accumulate"


def dram_counters():
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernels, taken with ncu
    and kept beside the profile summaries; an entry is null once its kernel has changed."""
    p = os.path.join(ROOT, "profiles", "dram_bytes_per_launch.json")
    try:
        with open(p) as f:
            return json.load(f)
    except Exception:
        return {}


def peaks():
    """Measured HBM copy bandwidth of this machine's B200 (generated file), else the fallback."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


SM_COUNT = 148
SMEM_BYTES_PER_CLK_PER_SM = 128


def three_rooflines(alg_bytes, us, hbm, l2, sm_mhz):
    """The same algorithmic bytes against three denominators.  The time loop keeps its weights in
    shared memory, so what bounds its stream is the shared-memory read rate (derived: 148 SMs x
    128 B per clock at the SM clock sampled during the run), then the L2 read rate measured in this
    run (what a kernel that re-read the weights from L2 every step could get), and, for context only,
    the HBM copy rate."""
    gbs = alg_bytes / us / 1e3
    smem_peak = SM_COUNT * SMEM_BYTES_PER_CLK_PER_SM * (sm_mhz or 1965.0) * 1e6 / 1e9
    return {"GBps": round(gbs, 1),
            "frac_smem_derived": round(gbs / smem_peak, 4), "smem_peak_GBps_derived": round(smem_peak, 0),
            "frac_l2_measured": round(gbs / l2, 4) if l2 else None,
            "frac_hbm_equivalent": round(gbs / hbm, 4)}


def layer_tuples(w):
    return [(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype) for m in w.layers]


# ----------------------------------------------------------------------------------------
# CPU oracle arm
# ----------------------------------------------------------------------------------------
def oracle_us_per_step(w, t_short=2, t_long=10):
    """Per-step cost of the oracle recurrence as it stands: the slope between two calls of
    different length, so that building the masked dense matrix (done once per call) drops out."""
    from oracle import rnn_oracle as R
    fn = R.lstm_forward if w.cell == "lstm" else R.gru_forward
    args = (layer_tuples(w), w.bias)

    def run(n):
        t0 = time.perf_counter()
        if w.cell == "lstm":
            fn(*args, w.x[:n], w.h0, w.c0)
        else:
            fn(*args, w.x[:n], w.h0)
        return time.perf_counter() - t0

    a, b = run(t_short), run(t_long)
    return max(b - a, 1e-9) / (t_long - t_short) * 1e6


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return len(os.sched_getaffinity(0))


REF_T = (2, 62)      # sequence lengths the reference arm runs per step (the slope between them is the value)


def reference_arm(args):
    """The float64 oracle as it stands on the host cores.  One step = two oracle calls on the
    benchmark's workload cut to REF_T[0] and REF_T[1] timesteps; value = the slope between them per
    timestep (the one-off build of the masked dense matrices drops out); ms_per_step = what those
    two calls took."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import rnn_oracle as R
    w = workloads.CONFIGS["cfg5"](T=REF_T[1])
    lay = layer_tuples(w)

    def step():
        # the short call twice (the faster one counts: most of a call is the one-off build of the masked
        # dense matrices, whose time varies more than the few timesteps cost), the long call once
        t0 = time.perf_counter()
        R.lstm_forward(lay, w.bias, w.x[:REF_T[0]])
        t1 = time.perf_counter()
        R.lstm_forward(lay, w.bias, w.x[:REF_T[0]])
        t2 = time.perf_counter()
        R.lstm_forward(lay, w.bias, w.x[:REF_T[1]])
        t3 = time.perf_counter()
        return (t3 - t0) * 1e3, max((t3 - t2) - min(t1 - t0, t2 - t1), 1e-9) / (REF_T[1] - REF_T[0]) * 1e6

    for _ in range(min(args.warmup, 1)):
        step()
    steps = max(1, min(args.steps, 5))              # each step is several seconds of host work
    res = [step() for _ in range(steps)]
    v = float(np.mean([r[1] for r in res]))
    ms = float(np.mean([r[0] for r in res]))
    sample = ("%d steps; a step = the oracle recurrence on cfg5 cut to %d (twice) and to %d timesteps (numpy BLAS), value = slope per timestep"
              % (steps, REF_T[0], REF_T[1]))
    line = {"impl": "reference", "metric": METRIC, "value": round(v, 1), "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": min(args.warmup, 1), "ms_per_step": round(ms, 1), "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "seq_len_run": list(REF_T), "batch": 1},
            "cpu_baseline": {"value": round(v, 1), "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": round(v, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


# ----------------------------------------------------------------------------------------
# GPU arm
# ----------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.lines, self.proc = [], None
        try:
            cmd = ["nvidia-smi", "--query-gpu=" + self.Q, "--format=csv,noheader,nounits", "-lms", "200"]
            if uuid:
                cmd += ["-i", uuid]
            self.proc = subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _pump(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def rnn_alg_bytes_per_step(w, infos):
    """Bytes the method itself must move per timestep: packed values, index lists and 6-byte block
    headers of every layer, the input and state vectors read, the states written, the bias."""
    B, H = w.B, w.hidden_size
    total = 0
    for l, info in enumerate(infos):
        in_l = w.input_size if l == 0 else H
        total += info["algorithmic_bytes"] + (in_l + H) * B * 4 + 4 * H * B * 4
        if w.bias[l] is not None:
            total += 4 * H * 4
    return total


def encode_layers(binding, w, dev):
    return [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, dev) for m in w.layers]


def make_runner(binding, torch, w, mats, host_io=False, sync=False):
    """Returns a zero-argument callable that performs one forward call, plus its I/O byte counts."""
    L, B, H, T = len(w.layers), w.B, w.hidden_size, w.T
    if host_io:
        x = torch.from_numpy(w.x).pin_memory()
        y = torch.empty((T, B, H), dtype=torch.float32).pin_memory()
        hT = torch.empty((L, B, H), dtype=torch.float32).pin_memory()
        cT = torch.empty((L, B, H), dtype=torch.float32).pin_memory()
        flags = binding.CSB_FLAG_HOST_IO
    else:
        x = torch.from_numpy(w.x).cuda()
        y = torch.empty((T, B, H), device="cuda")
        hT = torch.empty((L, B, H), device="cuda")
        cT = torch.empty((L, B, H), device="cuda")
        flags = 0 if sync else binding.CSB_FLAG_ASYNC
    if w.cell == "lstm":
        fn = lambda: binding.csb_lstm_forward(mats, None, x, None, None, y, hT, cT, flags)
        d2h = (y.numel() + hT.numel() + cT.numel()) * 4
    else:
        fn = lambda: binding.csb_gru_forward(mats, None, x, None, y, hT, flags)
        d2h = (y.numel() + hT.numel()) * 4
    return fn, x.numel() * 4, d2h, (x, y, hT, cT)


def checked_call(binding, torch, w, mats):
    """One synchronous call (the library waits for the kernel's status word and raises on a bounded
    wait that expired) before anything is timed; returns its outputs for the error figures."""
    fn, _, _, keep = make_runner(binding, torch, w, mats, sync=True)
    fn()
    torch.cuda.synchronize()
    return keep[1].cpu().numpy()


def time_calls(torch, fn, steps, warmup, flush):
    """Milliseconds of each of `steps` calls, CUDA events on the current stream around each call,
    an L2 flush (untimed) before each."""
    for _ in range(warmup):
        flush()
        fn()
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        flush()
        a.record()
        fn()
        b.record()
    torch.cuda.synchronize()
    return [a.elapsed_time(b) for a, b in ev]


def l2_read_roofline(torch, mbytes=48, reps=20):
    """Read bandwidth of a buffer that stays in L2 (48 MiB, summed repeatedly inside one CUDA graph):
    the denominator for products whose matrix is re-read from L2.  Measured here, nothing assumed."""
    x = torch.ones(mbytes << 18, dtype=torch.float32, device="cuda")
    out = torch.empty((), dtype=torch.float32, device="cuda")
    for _ in range(3):
        torch.sum(x, dim=0, out=out)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            for _ in range(reps):
                torch.sum(x, dim=0, out=out)
    g.replay()
    torch.cuda.synchronize()
    best = 1e9
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); g.replay(); b.record()
        torch.cuda.synchronize()
        best = min(best, a.elapsed_time(b) / reps)
    return x.numel() * 4 / (best * 1e-3) / 1e9


def cpu_csb_loops(m, x, reps=3):
    """The plain C loop nest over the CSB arrays (the oracle's second form) on the host cores."""
    from oracle import csb_oracle
    from oracle.csb_loops import CsbLoops
    stored = csb_oracle.round_to_storage(m.dense, m.val_dtype).astype(np.float32)
    L = CsbLoops(stored, m.block_r, m.block_c, m.row_keep, m.col_keep)
    cores = len(os.sched_getaffinity(0))
    return {"us_1_thread": round(L.seconds_per_spmv(x, 1, reps) * 1e6, 1),
            "us_all_cores": round(L.seconds_per_spmv(x, cores, reps) * 1e6, 1), "cores": cores, "kind": "oracle (C loop nest)"}


def product_error(m, X, Y):
    """Raw maximum relative error of a product against the float64 oracle over the outputs above the
    tolerance floor (1e-2 of the row's sum of |w||x|)."""
    from oracle import csb_oracle
    args = (m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype)
    want, scale = csb_oracle.spmm(*args, X), csb_oracle.abs_scale(*args, X)
    big = np.abs(want) > 1e-2 * scale
    return float(np.max(np.abs(Y.astype(np.float64) - want)[big] / np.abs(want)[big])) if big.any() else 0.0


def graph_us(torch, run, n, reps):
    """Microseconds per launch of `n` launches captured in one CUDA graph, median of `reps` replays."""
    g = torch.cuda.CUDAGraph()
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            run(n)
    g.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); g.replay(); b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b) / n * 1e3)
    del g
    return float(np.median(ts))


def spmv_sweep(binding, torch, dev, rates, batch, l2, reps=10, with_cpu=False, counters=None):
    """Bare CSB-SpMV / SpMM on the 8192x8192 / 64x64 matrix, cold: at least 200 launches in one CUDA
    graph rotate through enough encoded copies of the matrix to exceed L2, timed with events.  The
    panel kernel (batch 1) is timed twice: launched with programmatic stream serialization, as a
    stream of products runs in use (a launch's start-up overlaps the end of the one in front), and
    with ordinary launches, one product entirely after the other."""
    hbm, _ = peaks()
    out = []
    launches = 0
    for rate in rates:
        w = workloads.CONFIGS["cfg4"](rate=rate, B=batch)
        m = w.matrix
        A0 = binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, dev)
        info = A0.info()
        panel = batch == 1 and info["panel_ctas"] > 0      # which kernel serves this batch size
        stream_bytes = info["panel_stream_bytes"] if panel else info["device_stream_bytes"]
        ncopy = max(2, int(160e6 // max(info["algorithmic_bytes"], 1)) + 1)
        As = [A0] + [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, dev)
                     for _ in range(ncopy - 1)]
        X = torch.from_numpy(w.X).cuda()
        Y = torch.full((batch, m.rows), float("nan"), device="cuda")

        def run(n):
            for i in range(n):
                if batch == 1:
                    binding.csb_spmv(As[i % ncopy], X[0], Y[0])
                else:
                    binding.csb_spmm(As[i % ncopy], X, Y)
        run(ncopy)
        torch.cuda.synchronize()
        err = product_error(m, w.X, Y.cpu().numpy()) if with_cpu else None
        n = ncopy * -(-200 // ncopy)
        us = graph_us(torch, run, n, reps)
        launches += n * (reps + 1)
        us_serial = None
        if panel:
            os.environ["CSB_PANEL_PDL"] = "0"
            try:
                us_serial = graph_us(torch, run, n, reps)
            finally:
                del os.environ["CSB_PANEL_PDL"]
            launches += n * (reps + 1)
        # warm: the same matrix again and again (it fits L2), against the measured L2 read rate
        As_keep, ncopy_keep = As, ncopy
        As, ncopy = [A0], 1
        us_warm = graph_us(torch, run, 40, reps)
        launches += 40 * (reps + 1)
        As, ncopy = As_keep, ncopy_keep
        alg = info["algorithmic_bytes"] + (m.cols + m.rows) * 4 * batch
        e = {"rate": rate, "batch": batch, "nnz": info["nnz"], "us": round(us, 3), "algorithmic_bytes": alg,
             "GBps": round(alg / us / 1e3, 1), "frac_hbm_measured": round(alg / us / 1e3 / hbm, 4),
             "frac_hbm_8TBps": round(alg / us / 1e3 / 8000.0, 4), "GFLOPs": round(2 * info["nnz"] * batch / us / 1e3, 1),
             "us_warm_l2": round(us_warm, 3), "GBps_warm_l2": round(alg / us_warm / 1e3, 1),
             "frac_l2_warm": round(alg / us_warm / 1e3 / l2, 4) if l2 else None,
             "balance": round(info["panel_balance"] if panel else info["balance"], 3), "copies": ncopy, "launches_per_graph": n,
             "kernel": "csb_panel_kernel" if panel else ("csb_product_kernel" if batch < 8 else "csb_pack_x_kernel + csb_spmm_tile_kernel"),
             "streamed_bytes": stream_bytes if batch < 8 else None, "max_rel_err": err}
        if us_serial is not None:
            e["launch"] = "programmatic stream serialization (start-up overlaps the launch in front)"
            e["us_ordinary_launches"] = round(us_serial, 3)
            e["frac_hbm_measured_ordinary_launches"] = round(alg / us_serial / 1e3 / hbm, 4)
            e["frac_hbm_8TBps_ordinary_launches"] = round(alg / us_serial / 1e3 / 8000.0, 4)
        if with_cpu and rate == rates[0] and batch == 1:
            e["cpu_csb_loops"] = cpu_csb_loops(m, w.X[0])
        out.append(e)
        for a in As:
            a.free()
    return out, launches


def project_bench(binding, torch, reps=20):
    """Projection onto the CSB pattern (RowPrune / ColumnPrune of Algorithm 1) of an 8192x8192 dense
    weight, 64x64 blocks, 4x: two passes over the matrix plus two selections, device-resident input.
    Launches rotate over two matrices (2 x 268 MB > L2)."""
    hbm, _ = peaks()
    R = C = 8192
    g = torch.Generator(device="cuda").manual_seed(0)
    Ws = [torch.randn((R, C), device="cuda", generator=g) * 0.05 for _ in range(2)]
    rk, ck, ws = binding.csb_project(Ws[0], 64, 64, 0.75)
    for i in range(3):
        binding.csb_project(Ws[i % 2], 64, 64, 0.75, rk, ck, ws)
    torch.cuda.synchronize()
    ts = []
    for i in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); binding.csb_project(Ws[i % 2], 64, 64, 0.75, rk, ck, ws); b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b) * 1e3)
    us = float(np.median(ts))
    nbr = nbc = 128
    kept_rows = float(rk.float().mean())
    # W once in full, once without the pruned row segments; norms written and read; masks written, row flags read
    alg = int(R * C * 4 * (1.0 + kept_rows)) + 2 * (nbc * R + nbr * C) * 8 + 3 * nbr * nbc * 64
    kept = kept_rows * float(ck.float().mean())
    return {"workload": "8192x8192 fp32, 64x64 blocks, prune_fraction 0.75", "us": round(us, 1), "algorithmic_bytes": alg,
            "GBps": round(alg / us / 1e3, 1), "frac_hbm_measured": round(alg / us / 1e3 / hbm, 4), "kept_rows_x_cols": round(kept, 4),
            "launches_per_call": 4}


def slowest_rank_ms(local_ms, dist=None, device="cpu"):
    """Replicas only: every rank runs its own sequences with no data-path collective; the job's
    time for a step is the slowest rank's (max over ranks of the device-timed mean)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms)
    import torch
    t = torch.tensor([float(local_ms)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_us_per_timestep(ms_slowest, seq_len, world):
    """All replicas' timesteps over the slowest replica's time (aggregate, weak scaling)."""
    return ms_slowest * 1e3 / (seq_len * world)


def stepwise(w, nnz):
    """Whether the library runs this workload step by step on tensor cores (its own rule, restated)."""
    rows = 2 * w.B if w.cell == "gru" else w.B
    return (w.B >= 16 or (w.B >= 8 and nnz >= 100000)) and rows >= 8 and w.layers[0].val_dtype == "f16"


def oracle_sample(w, y_gpu, t_short, t_long):
    """The cpu_baseline leg of one recurrent workload: the float64 oracle as it stands on the first
    t_long timesteps (and on t_short, for the slope that drops the one-off mask build), timed, and
    the library's outputs of those timesteps compared with it (raw maximum relative error over the
    outputs above the tolerance floor of 1e-2 rms)."""
    from oracle import rnn_oracle as R
    lay = layer_tuples(w)
    fn = (lambda n: R.lstm_forward(lay, w.bias, w.x[:n])) if w.cell == "lstm" else (lambda n: R.gru_forward(lay, w.bias, w.x[:n]))
    t0 = time.perf_counter()
    fn(t_short)
    t1 = time.perf_counter()
    want = np.asarray(fn(t_long)[0])
    t2 = time.perf_counter()
    us = max((t2 - t1) - (t1 - t0), 1e-9) / (t_long - t_short) * 1e6
    got = y_gpu[:t_long].astype(np.float64)
    floor = 1e-2 * float(np.sqrt(np.mean(want ** 2)))
    big = np.abs(want) > floor
    err = float(np.max(np.abs(got - want)[big] / np.abs(want)[big])) if big.any() else 0.0
    return us, err


def layer_cpu_loops(w):
    """The plain CSB loop nest (C, double accumulation) over every layer's matrix with a vector of
    the layer's width: the method's own work on the host, one thread and all cores, summed over layers."""
    one = allc = 0.0
    cores = len(os.sched_getaffinity(0))
    for m in w.layers:
        r = cpu_csb_loops(m, np.ones(m.cols, np.float64), reps=3)
        one += r["us_1_thread"]
        allc += r["us_all_cores"]
    return {"us_per_step_1_thread": round(one, 1), "us_per_step_all_cores": round(allc, 1), "cores": cores, "kind": "oracle (C loop nest, one product per layer and step, batch column 0 only)"}


def config_entry(binding, torch, dev, flush, w, steps, hbm, l2, sm_mhz, with_cpu, t_sample):
    mats = encode_layers(binding, w, dev)
    infos = [m.info() for m in mats]
    nnz = sum(i["nnz"] for i in infos)
    y = checked_call(binding, torch, w, mats)
    fn, _, _, keep = make_runner(binding, torch, w, mats)
    ms = time_calls(torch, fn, steps, 3, flush)
    us = float(np.median(ms)) * 1e3 / w.T
    alg = rnn_alg_bytes_per_step(w, infos)
    sw = stepwise(w, nnz)
    e = {"us_per_timestep": round(us, 3), "T": w.T, "B": w.B, "algorithmic_bytes_per_step": alg,
         "GFLOPs": round(2 * nnz * w.B / us / 1e3, 1),
         "path": "per-step launches, products on tensor cores" if sw else "persistent time-loop kernel",
         "bound": "l2" if sw else "smem", "roofline": three_rooflines(alg, us, hbm, l2, sm_mhz)}
    launches = (steps + 4) * (1 if not sw else w.T * len(w.layers) * 3)
    if with_cpu:
        ts, tl = t_sample
        o_us, err = oracle_sample(w, y, ts, tl)
        e["cpu_baseline"] = {"value": round(o_us, 1), "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                             "sample": "slope of the float64 oracle recurrence between %d and %d timesteps" % (ts, tl)}
        e["max_rel_err"] = err
        e["max_rel_err_sample"] = "first %d timesteps of y against the oracle, outputs above 1e-2 rms" % tl
        e["cpu_csb_loops"] = layer_cpu_loops(w)
    for m in mats:
        m.free()
    return e, launches


def cells_bench(binding, torch, dev, flush, hbm, l2, sm_mhz, with_cpu):
    """The cell variants on the layer sizes of the paper's Table 1 (synthetic masks and weights; the
    paper's own latencies for these models, on its FPGA, are quoted as context): microseconds per
    timestep at batch 1, the float64 oracle beside them."""
    from oracle import rnn_oracle as R
    cases = [("lstmp_SR1", "lstmp", dict(I=153, H=1024, L=2, proj_size=512, lo=0.2, hi=0.35), "6.58 us per frame (Table 3, SR1, ZCU102 FPGA, int16)"),
             ("ligru_SR3", "ligru", dict(I=39, H=512, L=2, lo=0.3, hi=0.45), None),
             ("gru_reset_before_SR2", "gru_rb", dict(I=39, H=1024, L=2, lo=0.15, hi=0.3), "5.18 us per frame (Table 3, SR2, GRU, ZCU102 FPGA, int16)")]
    out, launches = {}, 0
    for name, cell, kw, ctx in cases:
        extra = dict(proj_size=kw["proj_size"]) if cell == "lstmp" else {}
        w = workloads.make_rnn_workload(0, cell, kw["I"], kw["H"], kw["L"], 32, 32, "uniform", lo=kw["lo"], hi=kw["hi"], T=100, B=1, w_std=0.05, **extra)
        mats = encode_layers(binding, w, dev)
        proj = [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, dev) for m in w.proj] if cell == "lstmp" else []
        S = w.proj_size if cell == "lstmp" else w.hidden_size
        x = torch.from_numpy(w.x).cuda()
        y = torch.empty((w.T, 1, S), device="cuda")
        hT = torch.empty((kw["L"], 1, S), device="cuda")
        cT = torch.empty((kw["L"], 1, w.hidden_size), device="cuda")

        def fn(flags=binding.CSB_FLAG_ASYNC):
            if cell == "lstmp":
                binding.csb_lstmp_forward(mats, proj, None, x, None, None, y, hT, cT, flags)
            elif cell == "ligru":
                binding.csb_ligru_forward(mats, None, x, None, y, hT, flags)
            else:
                binding.csb_gru_reset_before_forward(mats, None, x, None, y, hT, flags)
        fn(0)                                              # synchronous: raises if a device-side wait gave up
        torch.cuda.synchronize()
        y0 = y.cpu().numpy()
        ms = time_calls(torch, fn, 10, 3, flush)
        us = float(np.median(ms)) * 1e3 / w.T
        infos = [m.info() for m in mats + proj]
        alg = sum(i["algorithmic_bytes"] for i in infos) + sum((m.cols + m.rows) * 4 for m in w.layers + (w.proj or []))
        per_step_launches = {"lstmp": 4, "ligru": 2, "gru_rb": 4}[cell] * kw["L"]
        launches += 14 * w.T * per_step_launches
        e = {"us_per_timestep": round(us, 3), "T": w.T, "B": 1, "layers": kw["L"], "nnz": sum(i["nnz"] for i in infos),
             "algorithmic_bytes_per_step": alg, "launches_per_step": per_step_launches, "bound": "latency of %d dependent launches per step" % per_step_launches,
             "roofline": three_rooflines(alg, us, hbm, l2, sm_mhz), "paper_context": ctx}
        if with_cpu:
            lay = layer_tuples(w)
            prj = [(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype) for m in (w.proj or [])]
            run = {"lstmp": lambda n: R.lstmp_forward(lay, prj, w.bias, w.x[:n]), "ligru": lambda n: R.ligru_forward(lay, w.bias, w.x[:n]),
                   "gru_rb": lambda n: R.gru_reset_before_forward(lay, w.bias, w.x[:n])}[cell]
            t0 = time.perf_counter(); run(2); t1 = time.perf_counter(); want = np.asarray(run(42)[0]); t2 = time.perf_counter()
            floor = 1e-2 * float(np.sqrt(np.mean(want ** 2)))
            big = np.abs(want) > floor
            e["cpu_baseline"] = {"value": round(max((t2 - t1) - (t1 - t0), 1e-9) / 40 * 1e6, 1), "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                 "sample": "slope of the float64 oracle recurrence between 2 and 42 timesteps"}
            e["max_rel_err"] = float(np.max(np.abs(y0[:42] - want)[big] / np.abs(want)[big]))
        out[name] = e
        for m in mats + proj:
            m.free()
    return out, launches


def fixed_bench(binding, torch, dev, hbm, with_cpu, reps=10):
    """The 16-bit fixed-point product on the sweep's matrices, cold (rotating copies > L2 in one CUDA
    graph); integer work, so the check against the oracle is equality."""
    from oracle import fixed_oracle as F
    out, launches = [], 0
    for rate, batch in ((4.0, 1), (4.0, 4), (25.0, 1)):
        w = workloads.CONFIGS["cfg4"](rate=rate, B=batch)
        m = w.matrix
        A0 = binding.csb_encode_q16(m.dense, 64, 64, m.row_keep, m.col_keep, 16, dev)
        ncopy = max(2, int(160e6 // max(A0.info()["algorithmic_bytes"], 1)) + 1)      # rotating copies larger than L2
        As = [A0] + [binding.csb_encode_q16(m.dense, 64, 64, m.row_keep, m.col_keep, 16, dev) for _ in range(ncopy - 1)]
        Xq = torch.from_numpy(F.quantize(w.X, 12).astype(np.int16)).cuda()
        acc = torch.zeros((batch, m.rows), dtype=torch.int64, device="cuda")

        def run(n):
            for i in range(n):
                binding.csb_spmm_q16(As[i % ncopy], Xq, acc)
        run(ncopy)
        torch.cuda.synchronize()
        exact = None
        if with_cpu:
            exact = bool(np.array_equal(acc.cpu().numpy(), F.spmm_q16(m.dense, 64, 64, m.row_keep, m.col_keep, 16, Xq.cpu().numpy())))
        n = ncopy * -(-200 // ncopy)
        us = graph_us(torch, run, n, reps)
        launches += n * (reps + 1)
        v = As[0].view()
        alg = v["nnz"] * 2 + len(v["row_idx"]) + len(v["col_idx"]) + 6 * len(v["m"]) + m.cols * 2 * batch + m.rows * 8 * batch
        out.append({"rate": rate, "batch": batch, "nnz": int(v["nnz"]), "us": round(us, 3), "algorithmic_bytes": int(alg), "GBps": round(alg / us / 1e3, 1),
                    "frac_hbm_measured": round(alg / us / 1e3 / hbm, 4), "GMACs": round(v["nnz"] * batch / us / 1e3, 1), "equals_oracle": exact,
                    "kernel": "csb_q16_kernel", "copies": ncopy})
        for a in As:
            a.free()
    return out, launches


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--sections", default="rnn,e2e,spmv,spmm,project,configs,cells,fixed,cpu",
                    help="comma list of: rnn (always), e2e, spmv, spmm, project, configs, cells, fixed, cpu")
    ap.add_argument("--seq-len", type=int, default=512)
    ap.add_argument("--spmv-rates", default="4,8,16,25", help="pruning rates of the bare SpMV sweep")
    ap.add_argument("--spmv-reps", type=int, default=10)
    ap.add_argument("--spmm-batches", default="8,32,64", help="batch sizes of the SpMM sweep (section spmm)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return reference_arm(args)

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the library")
    from paper_2005_05758_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    sections = set(args.sections.split(",")) | {"rnn"}
    if rank != 0:
        sections &= {"rnn", "e2e"}
    hbm, peak_kind = peaks()
    counters = dram_counters()

    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    flush = lambda: flush_buf.zero_()

    w = workloads.CONFIGS["cfg5"](T=args.seq_len)
    mats = encode_layers(binding, w, local)
    infos = [m.info() for m in mats]
    y_checked = checked_call(binding, torch, w, mats)      # synchronous: a device-side give-up would raise here
    fn, _, _, keep = make_runner(binding, torch, w, mats)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    uuid = str(torch.cuda.get_device_properties(local).uuid)
    uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
    for _ in range(args.warmup):
        flush(); fn()
    barrier()
    sampler = ClockSampler(uuid) if rank == 0 else None
    wall0 = time.perf_counter()
    ms = time_calls(torch, fn, args.steps, 0, flush)
    barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop() if sampler else None
    sm_mhz = clocks.get("sm_mhz") if clocks else None
    mean_ms = slowest_rank_ms(float(np.mean(ms)), dist, "cuda")
    us_step = job_us_per_timestep(mean_ms, w.T, world)
    l2 = l2_read_roofline(torch) if rank == 0 else None
    launches = args.steps                              # one time-loop kernel per timed call

    line = {"metric": METRIC, "value": round(us_step, 4), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": round(mean_ms, 4), "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "seq_len": w.T, "batch": 1, "replicas": world,
                       "l2": "flushed (256 MiB written) before every timed call; weights then stay on chip for the sequence",
                       "paper_context": "0.79-6.58 us per frame on the paper's FPGA (other models, int16): not comparable"},
            "clocks": clocks, "wall_s_timed_region": round(wall, 3)}
    if l2:
        line["l2_read_GBps_measured"] = round(l2, 1)
    alg_step = rnn_alg_bytes_per_step(w, infos)
    three = three_rooflines(alg_step, mean_ms * 1e3 / w.T, hbm, l2, sm_mhz)
    line["roofline"] = {"kernel": "csb_rnn_kernel<half,1>", "bound": "smem", "achieved": three["GBps"],
                        "peak": three["smem_peak_GBps_derived"], "peak_kind": "derived: 148 SMs x 128 B/clk x sampled SM clock",
                        "unit": "GB/s", "frac": three["frac_smem_derived"],
                        "frac_l2_measured": three["frac_l2_measured"], "frac_hbm_equivalent": three["frac_hbm_equivalent"],
                        "hbm_peak": hbm, "hbm_peak_kind": peak_kind,
                        "traffic": counters.get("csb_rnn_kernel cfg5 T=512 B=1") if (w.T == 512 and world == 1) else None,
                        "algorithmic_bytes_per_launch": alg_step * w.T,
                        "note": "the compressed weights are read from HBM once per call and then stay in shared memory, so the "
                                "stream of a timestep is bounded by the shared-memory read rate (derived peak), not by DRAM (traffic "
                                "is far below the algorithmic bytes); frac_l2_measured compares with a kernel that re-read them from "
                                "L2 every step, frac_hbm_equivalent with what HBM could stream"}
    if "e2e" in sections:
        fn_h, h2d, d2h, keep_h = make_runner(binding, torch, w, mats, host_io=True)
        for _ in range(3):
            fn_h()
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            fn_h()                                     # synchronous: copies in, kernel, copies out
        barrier()
        e2e_ms = slowest_rank_ms((time.perf_counter() - t0) / args.steps * 1e3, dist, "cuda")
        line["e2e"] = {"value": round(job_us_per_timestep(e2e_ms, w.T, world), 4), "unit": UNIT, "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": d2h, "ms_per_step": round(e2e_ms, 4)}
    with_cpu = rank == 0 and "cpu" in sections
    if with_cpu:
        ts_, tl_ = 2, min(26, w.T)
        v, err = oracle_sample(w, y_checked, ts_, tl_)
        line["cpu_baseline"] = {"value": round(v, 1), "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                "sample": "slope of the float64 oracle recurrence between %d and %d timesteps of cfg5 (numpy BLAS)" % (ts_, tl_)}
        line["max_rel_err"] = err
        line["max_rel_err_sample"] = "first %d timesteps of y against the oracle, outputs above 1e-2 rms" % tl_
        line["cpu_csb_loops"] = layer_cpu_loops(w)
    for m in mats:
        m.free()
    if rank == 0 and "spmv" in sections:
        rates = [float(r) for r in args.spmv_rates.split(",")]
        line["spmv"], n_l = spmv_sweep(binding, torch, local, rates, 1, l2, reps=args.spmv_reps, with_cpu=with_cpu)
        launches += n_l
        best = max(line["spmv"], key=lambda r: r["frac_hbm_measured"])
        line["roofline_spmv"] = {"kernel": best["kernel"], "bound": "hbm", "achieved": best["GBps"], "peak": hbm,
                                 "peak_kind": peak_kind, "unit": "GB/s", "frac": best["frac_hbm_measured"],
                                 "frac_ordinary_launches": best.get("frac_hbm_measured_ordinary_launches"),
                                 "traffic": counters.get("csb_panel_kernel cfg4 4x B=1") if best["rate"] == 4.0 else None,
                                 "workload": "cfg4 8192x8192, 64x64 blocks, rate %gx, batch 1, cold (rotating copies > L2)" % best["rate"],
                                 "launch": "%d back-to-back launches in one CUDA graph; `frac` with programmatic stream serialization (a "
                                           "launch's start-up overlaps the end of the one in front), `frac_ordinary_launches` with one "
                                           "product entirely after the other" % best["launches_per_graph"]}
    if rank == 0 and "spmm" in sections:
        line["spmm"] = []
        rates = [float(r) for r in args.spmv_rates.split(",")]
        for bsz in [int(b) for b in args.spmm_batches.split(",")]:
            res, n_l = spmv_sweep(binding, torch, local, rates, bsz, l2, reps=args.spmv_reps, with_cpu=with_cpu)
            line["spmm"] += res
            launches += 2 * -(-bsz // 32) * n_l          # per pass of 32 batch columns: the pack kernel and the product kernel
        best = max(line["spmm"], key=lambda r: r["frac_hbm_measured"])
        line["roofline_spmm"] = {"kernel": "csb_spmm_tile_kernel", "bound": "hbm", "achieved": best["GBps"], "peak": hbm, "peak_kind": peak_kind,
                                 "unit": "GB/s", "frac": best["frac_hbm_measured"],
                                 "traffic": counters.get("csb_spmm_tile_kernel cfg4 4x B=64") if (best["rate"] == 4.0 and best["batch"] == 64) else None,
                                 "traffic_per_pass_4x_batch64": counters.get("csb_spmm_tile_kernel cfg4 4x B=64"),
                                 "workload": "cfg4 8192x8192, 64x64 blocks, rate %gx, batch %d, cold" % (best["rate"], best["batch"])}
    if rank == 0 and "project" in sections:
        line["project"] = project_bench(binding, torch)
        launches += 4 * 24
    if rank == 0 and "configs" in sections:
        line["configs"] = {}
        cases = [("cfg1", dict(), (2, 16)), ("cfg2", dict(), (2, 42)), ("cfg3", dict(B=1), (2, 42)), ("cfg3", dict(B=8), (2, 22)),
                 ("cfg5", dict(B=32, T=128), (2, 8))]
        for name, kw, tsamp in cases:
            wc = workloads.CONFIGS[name](**kw)
            e, n_l = config_entry(binding, torch, local, flush, wc, 10, hbm, l2, sm_mhz, with_cpu, tsamp)
            line["configs"]["%s_B%d" % (name, wc.B)] = e
            launches += n_l
    if rank == 0 and "cells" in sections:
        line["cells"], n_l = cells_bench(binding, torch, local, flush, hbm, l2, sm_mhz, with_cpu)
        launches += n_l
    if rank == 0 and "fixed" in sections:
        line["fixed_point"], n_l = fixed_bench(binding, torch, local, hbm, with_cpu)
        launches += n_l
    line["gpu_launches"] = launches
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
