"""The C-ABI library builds, loads, and exports every symbol include/recache.h
declares, and the binding's signatures cover exactly those.  No compute calls."""
import ctypes
import os
import re

import paper_2608_19662_b200 as pkg
from paper_2608_19662_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "recache.h")).read()
    return sorted(set(re.findall(r"RECACHE_API\s+[\w\s\*]+?\b(recache_\w+)\s*\(", text)))


def test_header_declares_the_four_hot_path_calls():
    syms = declared_symbols()
    for name in ("recache_encode_resources", "recache_compact_routes", "recache_attend_prefill",
                 "recache_attend_decode", "recache_create", "recache_destroy", "recache_poll_status"):
        assert name in syms


def test_library_builds_and_exports_every_declared_symbol():
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    for name in declared_symbols():
        assert hasattr(lib, name), name


def test_binding_covers_header():
    assert sorted(binding.SIGNATURES) == declared_symbols()


def test_null_and_bad_arguments_are_rejected_without_a_gpu():
    lib = binding.load_library()
    assert lib.recache_create(None, None, 0) == 1                      # EINVAL
    h = ctypes.c_void_p()
    bad = binding.Desc(6, 4, 128, 1, 1024, 64, 1e6)                    # 6 % 4 != 0
    assert lib.recache_create(ctypes.byref(h), ctypes.byref(bad), 0) == 2 and not h.value
    bad = binding.Desc(8, 4, 96, 1, 1024, 64, 1e6)                     # head_dim 96
    assert lib.recache_create(ctypes.byref(h), ctypes.byref(bad), 0) == 2
    assert lib.recache_encode_workspace_bytes(None, 1, 1, 1) == -1
    assert lib.recache_last_error(None) == b"null context"


def test_package_has_no_cpu_path():
    import torch
    if not torch.cuda.is_available():
        import pytest
        with pytest.raises(RuntimeError):
            pkg.ReCache(4, 2, 64, 1e4, "f32")
