"""Build libcsb.so in-tree with nvcc for sm_100a (cross-compiles without a GPU)."""
from __future__ import annotations

import os
import subprocess
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
CSRC = os.path.join(HERE, "csrc")
LIB = os.path.join(HERE, "libcsb.so")
SOURCES = ["csb_api.cpp", "csb_encode.cpp", "csb_plan.cpp", "csb_schedule.cpp", "csb_spmm_plan.cpp", "csb_panel_plan.cpp", "csb_product.cu", "csb_panel.cu", "csb_spmm_mma.cu", "csb_rnn.cu", "csb_rnn_step.cu", "csb_cells.cu", "csb_fixed.cu", "csb_project.cu"]
HEADERS = ["csb_internal.hpp", "csb_device.cuh", os.path.join("..", "..", "include", "csb.h")]


def _stale() -> bool:
    if not os.path.exists(LIB):
        return True
    t = os.path.getmtime(LIB)
    deps = [os.path.join(CSRC, f) for f in SOURCES + HEADERS]
    return any(os.path.getmtime(d) > t for d in deps if os.path.exists(d))


#: Instrumented variants (never the default build).  CSB_PHASE_CLOCKS makes the time-loop kernel sum
#: clock64() cycles per phase and CTA (read back with csb_debug_rnn_clocks); CSB_PANEL_CLOCKS makes
#: the SpMV panel kernel record wall-clock stamps per phase and CTA (csb_debug_panel_clocks);
#: CSB_SPMM_CLOCKS makes the batched tensor-core kernel sum cycles per phase and warp (csb_debug_spmm_clocks).
#: paper_2005_05758_b200/phase_clocks.py builds such a library beside the normal one and prints the figures.
INSTRUMENT_DEFINES = ("CSB_PHASE_CLOCKS", "CSB_PANEL_CLOCKS", "CSB_SPMM_CLOCKS")


def build(force: bool = False, verbose: bool = False, defines=(), out: str = None) -> str:
    """Compile the library if it is missing or older than its sources; return its path.
    `defines` adds -D switches (see INSTRUMENT_DEFINES) and then needs `out`, the path of the
    instrumented library, so that the normal libcsb.so is never replaced by one."""
    if defines and not out:
        raise ValueError("an instrumented build needs its own output path")
    if not defines and not force and not _stale():
        return LIB
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-Xcompiler", "-fPIC", "-shared", "-o", out or LIB] + ["-D" + d for d in defines] + [os.path.join(CSRC, s) for s in SOURCES]
    if verbose:
        cmd.insert(1, "-Xptxas")
        cmd.insert(2, "-v")
    res = subprocess.run(cmd, capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError("nvcc failed:\n" + res.stdout + res.stderr)
    if verbose:
        sys.stderr.write(res.stderr)
    return out or LIB


if __name__ == "__main__":
    print(build(force="--force" in sys.argv, verbose="-v" in sys.argv))
