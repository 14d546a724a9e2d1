"""The C-ABI library loads (no GPU needed) and exports every symbol include/gkv.h declares."""
import ctypes
import os
import re

from paper_2608_23599_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    B.build()
    header = open(os.path.join(ROOT, "include", "gkv.h")).read()
    declared = re.findall(r"GKV_API\s+[\w\s\*]*?\b(gkv_\w+)\s*\(", header)
    assert len(declared) >= 10
    lib = ctypes.CDLL(B.lib_path())
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in gkv.h but not exported"
    assert sorted(declared) == sorted(B.EXPORTS)


def test_config_struct_matches_header_size_and_validation():
    lib = B.load()
    cfg = B.make_config(1, 1, 8, 2, 128, 128, 4096)
    n = B.gkv_query_arena_bytes(cfg)
    assert n > 4096 * 2 * 512
    assert B.strerror(0) == "ok" and "arena" in B.strerror(-2)
    bad = B.make_config(1, 1, 8, 3, 128, 128, 4096)            # heads do not divide
    out = ctypes.c_size_t(0)
    assert lib.gkv_query_arena_bytes(ctypes.byref(bad), ctypes.byref(out)) == -1
    bad = B.make_config(1, 1, 8, 2, 64, 64, 4096)               # head dim not compiled
    assert lib.gkv_query_arena_bytes(ctypes.byref(bad), ctypes.byref(out)) == -5
    bad = B.make_config(1, 1, 8, 2, 128, 128, 4096)
    bad.abi_version = 99
    assert lib.gkv_query_arena_bytes(ctypes.byref(bad), ctypes.byref(out)) == -1
    # the staircase arena bound grows with the exact rung
    small = B.gkv_query_arena_bytes(B.make_config(1, 1, 8, 2, 128, 128, 4096, stair_tokens=(64, 64, 64, 64)))
    large = B.gkv_query_arena_bytes(B.make_config(1, 1, 8, 2, 128, 128, 4096, stair_tokens=(-1, 0, 0, 0)))
    assert small < large


def test_every_export_has_declared_argument_types():
    """Without argtypes ctypes passes Python ints as 32-bit C ints, which truncates device pointers."""
    lib = B.load()
    for name in B.EXPORTS:
        assert getattr(lib, name).argtypes is not None, f"{name}: argtypes not declared in binding.load()"
