"""The two checking builds of the library that only the tests load, each a shared object of its own
beside this file (never the product library):

  hooks   -DBT_TEST_HOOKS: the product's kernels plus bt_test_set_wait_ns(), which sets the bound of the
          compress kernels' waits so that a test can let a wait run out by itself;
  bounds  -DBT_BOUNDS_CHECK: every global store of every kernel is tested against the extent of its
          buffer, skipped and counted when it falls outside (bt_test_bounds_violations()); relocatable
          device code, because all kernels share the one counter.

Both are compiled for sm_100a from the same sources as the product; nvcc cross-compiles without a GPU.
"""
from __future__ import annotations

import ctypes
import os

from paper_2110_15362_b200 import binding as B
from paper_2110_15362_b200 import build as _build

LIB_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib")
HOOKS_PATH = os.path.join(LIB_DIR, "libbittrain_hooks.so")
BOUNDS_PATH = os.path.join(LIB_DIR, "libbittrain_bounds.so")
_FLAGS = {HOOKS_PATH: ["-DBT_TEST_HOOKS"], BOUNDS_PATH: ["-DBT_BOUNDS_CHECK", "-rdc=true"]}
_loaded = {}


def build_all(force: bool = False) -> None:
    for path, flags in _FLAGS.items():
        _build.build_library(force=force, out=path, extra_flags=flags)


def _load(path: str) -> ctypes.CDLL:
    if path not in _loaded:
        try:
            _build.build_library(out=path, extra_flags=_FLAGS[path])      # a no-op when the library is up to date
        except Exception:
            if not os.path.exists(path):                                   # no compiler here and nothing built: give up
                raise
        _loaded[path] = B.load_library(path)
    return _loaded[path]


def hooks_lib() -> ctypes.CDLL:
    L = _load(HOOKS_PATH)
    L.bt_test_set_wait_ns.restype = ctypes.c_uint64
    L.bt_test_set_wait_ns.argtypes = [ctypes.c_uint64]
    return L


def bounds_lib() -> ctypes.CDLL:
    L = _load(BOUNDS_PATH)
    L.bt_test_bounds_violations.restype = ctypes.c_longlong
    L.bt_test_bounds_violations.argtypes = [ctypes.c_int]
    return L
