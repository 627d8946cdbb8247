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
