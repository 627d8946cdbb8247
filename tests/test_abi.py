"""The shared library loads and exports every symbol that include/csb.h declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_every_declared_symbol_is_exported():
    hdr = open(os.path.join(ROOT, "include", "csb.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(csb_[a-z_0-9]+)\s*\(", hdr))
    assert {"csb_encode", "csb_spmv", "csb_spmm", "csb_lstm_forward", "csb_gru_forward"} <= names
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2005_05758_b200", "libcsb.so"))
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_oracle_and_library_do_not_import_each_other():
    for d, banned in (("oracle", "paper_2005_05758_b200"), ("paper_2005_05758_b200", "oracle")):
        for dirpath, _, files in os.walk(os.path.join(ROOT, d)):
            for f in files:
                if f.endswith((".py", ".cu", ".cpp", ".hpp", ".cuh", ".h", ".c")):
                    src = open(os.path.join(dirpath, f)).read()
                    assert not re.search(r"^\s*(from|import)\s+" + banned, src, flags=re.M), (d, f)
                    assert ("#include \"../" + banned) not in src


def test_project_argument_checks_need_no_gpu():
    # csb_project validates sizes, fraction, workspace and the selection kernel's limit before it
    # touches the device, so the refusals can be checked with made-up (never dereferenced) pointers
    lib = ctypes.CDLL(os.path.join(ROOT, "paper_2005_05758_b200", "libcsb.so"))
    lib.csb_project_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int]
    lib.csb_project_workspace_bytes.restype = ctypes.c_int64
    lib.csb_project.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                ctypes.c_double, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
    lib.csb_last_error.restype = ctypes.c_char_p
    # 8 bytes per row segment and per column segment: (nbc * rows + nbr * cols) * 8
    assert lib.csb_project_workspace_bytes(300, 1177, 32, 32) == (37 * 300 + 10 * 1177) * 8
    assert lib.csb_project_workspace_bytes(0, 5, 2, 2) == 0
    fake = ctypes.c_void_p(4096)
    big = 1 << 40
    assert lib.csb_project(None, 8, 8, 8, 4, 4, 0.5, fake, fake, fake, big, None) == -1
    assert lib.csb_project(fake, 8, 8, 4, 4, 4, 0.5, fake, fake, fake, big, None) == -1          # ld < cols
    assert lib.csb_project(fake, 8, 8, 8, 4, 300, 0.5, fake, fake, fake, big, None) == -1        # block size
    assert lib.csb_project(fake, 8, 8, 8, 4, 4, 1.5, fake, fake, fake, big, None) == -1          # fraction
    assert lib.csb_project(fake, 8, 8, 8, 4, 4, float("nan"), fake, fake, fake, big, None) == -1
    assert lib.csb_project(fake, 8, 8, 8, 4, 4, 0.5, fake, fake, fake, 16, None) == -1 and b"workspace" in lib.csb_last_error()
    assert lib.csb_project(fake, 30000, 64, 64, 32, 32, 0.5, fake, fake, fake, big, None) == -8 and b"20480" in lib.csb_last_error()


def test_plan_opts_out_of_range_are_refused():
    # checked before anything is planned, so a host-only handle (device = -1) shows it without a GPU
    import numpy as np
    import pytest
    from paper_2005_05758_b200 import binding
    W = np.ones((8, 8), np.float32)
    rk = ck = np.ones(8 * 2, np.uint8)
    ok = binding.csb_encode(W, 4, 4, rk, ck, "f16", -1, dict(ctas=3, warps_per_cta=16, stage_bytes=16384, stages=8))
    ok.free()
    for bad in (dict(stages=9), dict(stage_bytes=512), dict(stage_bytes=1 << 20), dict(warps_per_cta=17), dict(ctas=-1)):
        opts = dict(ctas=0, warps_per_cta=0, stage_bytes=0, stages=0)
        opts.update(bad)
        with pytest.raises(binding.CsbError) as e:
            binding.csb_encode(W, 4, 4, rk, ck, "f16", -1, opts)
        assert e.value.status == -1 and "csb_plan_opts" in str(e.value)
