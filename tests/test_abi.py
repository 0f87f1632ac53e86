"""The C-ABI library loads without a GPU and exports every function include/dcp.h declares."""
import ctypes
import os
import re

from paper_2608_07524_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    with open(os.path.join(ROOT, "include", "dcp.h")) as f:
        text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
    return sorted(set(re.findall(r"\b(dcp_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    names = declared_functions()
    assert {"dcp_plan", "dcp_varlen_attn_fwd", "dcp_varlen_attn_bwd", "dcp_varlen_attn_workspace",
            "dcp_query_status", "dcp_last_error"} <= set(names)
    lib = ctypes.CDLL(B.LIB_PATH)
    for name in names:
        assert hasattr(lib, name), name


def test_workspace_sizes():
    fwd, bwd = B.dcp_varlen_attn_workspace(1000, 7, 4, 128)
    assert fwd % 256 == 0 and bwd % 256 == 0
    assert fwd >= 256 + 4 * 7 + 4 * 8
    assert bwd >= fwd + 4 * 1000 * 4 + 4 * 1000 * 4 * 128


def test_source_names_no_closed_cuda_calls():
    # the batched-memcpy entry points of the CUDA runtime and driver are not to be used (they have
    # faulted GPUs of this class); nothing in the source tree may even name them
    bad = re.compile("Memcpy" + "Batch|Memcpy3D" + "Batch")
    roots = [os.path.join(ROOT, d) for d in ("include", "oracle", "paper_2608_07524_b200", "tests")]
    paths = [os.path.join(ROOT, f) for f in ("bench.py", "__graft_entry__.py")]
    for root in roots:
        for dirpath, _, files in os.walk(root):
            paths += [os.path.join(dirpath, fn) for fn in files if fn.endswith((".cu", ".cuh", ".h", ".cpp", ".c", ".py"))]
    assert len(paths) > 20
    for path in paths:
        with open(path, errors="replace") as f:
            assert not bad.search(f.read()), path
