"""The C-ABI library builds for sm_100a, loads without a GPU, and exports every symbol that
include/grand.h declares (no compute is attempted here)."""
import ctypes
import os
import re

from paper_2608_21163_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "grand.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(grand_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    path = build.build()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    syms = declared_symbols()
    assert len(syms) >= 20
    for s in syms:
        assert hasattr(lib, s), f"{s} declared in grand.h but not exported"
    assert set(binding.EXPORTS) == set(syms)


def test_strerror_and_argument_checks_need_no_gpu():
    lib = binding.load()
    assert lib.grand_strerror(0) == b"ok"
    assert b"duplicate" in lib.grand_strerror(-3)
    h = ctypes.c_void_p()
    # Vamana mode + inner product is rejected before any CUDA call
    rc = lib.grand_create(ctypes.c_uint32(8), ctypes.c_uint32(0), ctypes.c_uint32(1), ctypes.c_uint32(8),
                          ctypes.c_uint32(16), ctypes.c_float(1.2), ctypes.byref(h))
    assert rc == -6
    rc = lib.grand_create(ctypes.c_uint32(8), ctypes.c_uint32(0), ctypes.c_uint32(0), ctypes.c_uint32(1000),
                          ctypes.c_uint32(16), ctypes.c_float(1.2), ctypes.byref(h))
    assert rc == -1


def test_options_struct_layout_matches_header():
    # 2 x u64, 9 x 32-bit fields (+4 padding), u64, one 32-bit field (+4 padding), 3 pointers
    assert ctypes.sizeof(binding.GrandOptions) == 16 + 40 + 8 + 8 + 24
    # 11 counters, 7 phase times, 5 launch counts, 2 per-kernel pair counters
    assert ctypes.sizeof(binding.GrandStats) == 11 * 8 + 7 * 8 + 5 * 8 + 2 * 8
    # field order as in the header: the 64-bit edge bound sits between the two 32-bit switches
    names = [n for n, _ in binding.GrandOptions._fields_]
    assert names.index("visited_set_delete") < names.index("max_delete_edges") < names.index("snapshot_search")


def test_workspace_bounds_are_checked_before_any_allocation():
    """The update workspace is sized from max_batch and max_delete_edges when the index is created; bounds that cannot
    be indexed with 32 bits are refused up front (no GPU is needed to be told so)."""
    lib = binding.load()
    h = ctypes.c_void_p()
    o = binding.GrandOptions(capacity=1 << 20, max_batch=1 << 10, max_delete_edges=1 << 33)
    rc = lib.grand_create_ex(ctypes.c_uint32(8), ctypes.c_uint32(0), ctypes.c_uint32(0), ctypes.c_uint32(8),
                             ctypes.c_uint32(16), ctypes.c_float(1.2), ctypes.byref(o), ctypes.byref(h))
    assert rc == -1 and not h.value
    assert b"capacity" in lib.grand_strerror(-2) and lib.grand_strerror(-8) == b"unknown status"
