"""In-kernel phase timing of the two batch-1 kernels, from an instrumented build of the library.

    python -m paper_2005_05758_b200.phase_clocks rnn   [cfg1 cfg2 cfg3 cfg5]
    python -m paper_2005_05758_b200.phase_clocks panel [4 8 16 25]
    python -m paper_2005_05758_b200.phase_clocks loop  [cfgN:batch ...]      (default cfg5:32 cfg3:8: the one-launch time loop at batch)
    python -m paper_2005_05758_b200.phase_clocks spmm  [rate:batch | cfgN:batch ...]   (default 4:8 4:32 25:8; cfgN = first layer of that config)

Builds libcsb_clocks.so beside the normal library with -DCSB_PHASE_CLOCKS -DCSB_PANEL_CLOCKS (see
build.py), loads it instead of libcsb.so and prints
  rnn:   cycles per timestep and phase of csb_rnn_kernel, summed by thread 0 of every CTA
         (mean / min / max over the CTAs);
  panel: wall-clock stamps of csb_panel_kernel per CTA, in microseconds from the earliest CTA start;
  spmm:  cycles per phase of csb_spmm_tile_kernel, summed per warp (mean / max over the warps, and the
         same for the slowest CTA, and the warp that finishes its items last).
The instrumented kernels are slower than the product ones (thread 0 reads the clock between phases),
so these figures say where the time goes, never how long a call takes.
"""
from __future__ import annotations

import ctypes as C
import os
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

RNN_PHASES = ["stage input half", "walk items (both halves)", "sync after accumulator sums", "gates + publish",
              "wait for h of the other CTAs", "activations (thread 0)", "slot-reuse guard", "loads + adds + shuffles of the sums"]
PANEL_STAMPS = ["CTA start", "barriers set, first copies out", "bookkeeping + x landed", "inputs gathered", "bundles done",
                "y stored", "-", "-"]


def _load():
    from paper_2005_05758_b200 import build
    lib = build.build(defines=build.INSTRUMENT_DEFINES, out=os.path.join(HERE, "libcsb_clocks.so"))
    os.environ["CSB_LIBRARY"] = lib
    import torch
    from paper_2005_05758_b200 import binding
    return torch, binding


def rnn(names):
    import workloads
    torch, binding = _load()
    for name in names:
        w = workloads.CONFIGS[name](**({"T": 128} if name == "cfg5" else {}))
        mats = [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, 0) for m in w.layers]
        L, B, H, T = len(w.layers), w.B, w.hidden_size, w.T
        x = torch.from_numpy(w.x).cuda()
        y = torch.empty((T, B, H), device="cuda")
        hT = torch.empty((L, B, H), device="cuda")
        cT = torch.empty((L, B, H), device="cuda")
        for _ in range(3):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if w.cell == "lstm":
                binding.csb_lstm_forward(mats, None, x, None, None, y, hT, cT, 0)
            else:
                binding.csb_gru_forward(mats, None, x, None, y, hT, 0)
            b.record()
            torch.cuda.synchronize()
        ck = np.zeros((256, 8), np.int64)
        n = binding.lib.csb_debug_rnn_clocks(C.c_void_p(ck.ctypes.data), 256)
        ck = ck[:n] / T
        print("%s: T=%d, %d CTAs, %.2f us per step (instrumented)" % (name, T, n, a.elapsed_time(b) * 1e3 / T))
        for i, nm in enumerate(RNN_PHASES):
            print("   %-38s cycles/step mean %7.0f  min %7.0f  max %7.0f" % (nm, ck[:, i].mean(), ck[:, i].min(), ck[:, i].max()))
        for m in mats:
            m.free()


def panel(rates):
    import workloads
    torch, binding = _load()
    for rate in rates:
        w = workloads.CONFIGS["cfg4"](rate=float(rate), B=1)
        m = w.matrix
        A = binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, 0)
        n = A.info()["panel_ctas"]
        # cold the way a stream of different products is cold: rotate through encoded copies whose
        # total exceeds L2 (a flush by writing would leave HBM busy with write-backs), the stamped
        # launch last and alone
        ncopy = max(2, int(200e6 // max(A.info()["algorithmic_bytes"], 1)) + 1)
        others = [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, 0) for _ in range(ncopy - 1)]
        x = torch.from_numpy(w.X).cuda()
        y = torch.empty(m.rows, device="cuda")
        for _ in range(3):
            for o in others:
                binding.csb_spmv(o, x[0], y)
            torch.cuda.synchronize()
            binding.csb_spmv(A, x[0], y)
            torch.cuda.synchronize()
        ck = np.zeros((n, 8), np.uint64)
        binding.lib.csb_debug_panel_clocks(C.c_void_p(ck.ctypes.data), n)
        t = (ck.astype(np.float64) - float(ck[:, 0].min())) / 1e3
        print("cfg4 rate %sx: %d CTAs, stamps in us from the earliest CTA start (cold L2)" % (rate, n))
        for i, nm in enumerate(PANEL_STAMPS[:6]):
            print("   %-34s mean %6.2f  min %6.2f  max %6.2f" % (nm, t[:, i].mean(), t[:, i].min(), t[:, i].max()))
        for o in others + [A]:
            o.free()


SPMM_PHASES = ["set-up, first copies, wait for the work in front", "waiting for weights", "passing tiles, waiting for the item's tile",
               "row map, operand loads, tensor instructions", "ring bookkeeping, item headers", "tiles behind the last item",
               "waiting for the CTA's other warps", "accumulators to shared memory", "sums over the warps of a block-row",
               "waiting for the cluster's other CTAs", "sums over the ranges, store", "until the cluster's CTAs have read",
               "(time loop) grid barrier behind the product pass", "(time loop) gate arithmetic", "(time loop) grid barrier behind the gates",
               "(time loop) next pass's first weights out"]


def spmm(cases):
    import workloads
    torch, binding = _load()
    for case in cases:
        rate, B = case.split(":")
        if rate.startswith("cfg"):                 # first layer of a recurrent config, e.g. cfg5:32
            m = workloads.CONFIGS[rate](T=1).layers[0]
            X = np.random.default_rng(1).standard_normal((int(B), m.cols)).astype(np.float32)
        else:
            w = workloads.CONFIGS["cfg4"](rate=float(rate), B=int(B))
            m, X = w.matrix, w.X
        As = [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, 0) for _ in range(3)]
        X = torch.from_numpy(X).cuda()
        Y = torch.empty((int(B), m.rows), device="cuda")
        for i in range(6):
            binding.csb_spmm(As[i % 3], X, Y)
            torch.cuda.synchronize()
        ck = np.zeros((1 << 16, 16), np.int64)
        n = binding.lib.csb_debug_spmm_clocks(C.c_void_p(ck.ctypes.data), 1 << 16)
        ck = ck[:n].astype(np.float64)
        wpc = 32 if int(B) <= 8 else 16
        per_cta = ck.reshape(-1, wpc, 16)
        slow = per_cta[np.argmax(per_cta.sum(axis=2).max(axis=1))]
        last = ck[np.argmax(ck[:, :6].sum(axis=1))]      # the warp that reaches the end of its items last
        print("%s batch %s: %d warps (%d per CTA); cycles per phase, last pass of 32 batch columns"
              % (rate if rate.startswith("cfg") else "cfg4 rate %sx" % rate, B, n, wpc))
        for i, nm in enumerate(SPMM_PHASES):
            print("   %-52s mean %8.0f  min %8.0f  max %8.0f   slowest CTA: mean %8.0f  max %8.0f   last warp %8.0f"
                  % (nm, ck[:, i].mean(), ck[:, i].min(), ck[:, i].max(), slow[:, i].mean(), slow[:, i].max(), last[i]))
        print("   %-52s mean %8.0f  max %8.0f" % ("all phases", ck.sum(axis=1).mean(), ck.sum(axis=1).max()))
        for a in As:
            a.free()


def loop(names):
    """The one-launch time loop of the batched recurrent path: cycles per phase and pass (layer and step)."""
    import workloads
    os.environ["CSB_RNN_STEP_LOOP"] = "1"          # the loop is not the default path
    torch, binding = _load()
    for case in names:
        name, B = case.split(":")
        w = workloads.CONFIGS[name](B=int(B), T=32)
        mats = [binding.csb_encode(m.dense, m.block_r, m.block_c, m.row_keep, m.col_keep, m.val_dtype, 0) for m in w.layers]
        L, B, H, T = len(w.layers), w.B, w.hidden_size, w.T
        x = torch.from_numpy(w.x).cuda()
        y = torch.empty((T, B, H), device="cuda")
        hT = torch.empty((L, B, H), device="cuda")
        cT = torch.empty((L, B, H), device="cuda")
        for _ in range(3):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if w.cell == "lstm":
                binding.csb_lstm_forward(mats, None, x, None, None, y, hT, cT, 0)
            else:
                binding.csb_gru_forward(mats, None, x, None, y, hT, 0)
            b.record()
            torch.cuda.synchronize()
        ck = np.zeros((1 << 16, 16), np.int64)
        n = binding.lib.csb_debug_spmm_clocks(C.c_void_p(ck.ctypes.data), 1 << 16)
        ck = ck[:n].astype(np.float64) / (T * L)
        print("%s batch %d: T=%d, %d warps, %.2f us per step (instrumented); cycles per phase and pass" % (name, B, T, n, a.elapsed_time(b) * 1e3 / T))
        for i, nm in enumerate(SPMM_PHASES):
            print("   %-52s mean %8.0f  min %8.0f  max %8.0f" % (nm, ck[:, i].mean(), ck[:, i].min(), ck[:, i].max()))
        print("   %-52s mean %8.0f" % ("all phases", ck.sum(axis=1).mean()))
        for m in mats:
            m.free()


if __name__ == "__main__":
    what = sys.argv[1] if len(sys.argv) > 1 else "rnn"
    rest = sys.argv[2:]
    if what == "rnn":
        rnn(rest or ["cfg1", "cfg2", "cfg3", "cfg5"])
    elif what == "panel":
        panel(rest or ["4", "25"])
    elif what == "spmm":
        spmm(rest or ["4:8", "4:32", "25:8"])
    elif what == "loop":
        loop(rest or ["cfg5:32", "cfg3:8"])
    else:
        raise SystemExit(__doc__)
