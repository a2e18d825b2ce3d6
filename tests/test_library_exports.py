"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

import paper_2511_12500_b200 as iris
from paper_2511_12500_b200 import build as iris_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _header_functions():
    text = open(os.path.join(ROOT, "include", "iris_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    text = re.sub(r"typedef struct iris_gemm_args \{.*?\} iris_gemm_args;", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b([a-z_0-9]+)\s*\(", text)) - {"defined"})


@pytest.fixture(scope="module")
def library():
    iris_build.build()
    return ctypes.CDLL(iris.LIB_PATH)


def test_header_and_binding_list_agree():
    assert _header_functions() == sorted(iris.EXPORTS)


def test_every_declared_symbol_is_exported(library):
    for name in _header_functions():
        assert hasattr(library, name), name


def test_host_only_calls_work_without_a_gpu(library):
    L = iris.lib()
    assert b"sm_100a" in L.iris_version()
    assert L.iris_num_tiles(256, 256, 2) == 4
    assert L.iris_num_tiles(130, 544, 4) == 2 * 4 * 2
    assert L.iris_num_tiles(0, 256, 2) == 0
    assert L.iris_num_tiles(256, 255, 2) < 0
    assert L.iris_gemm_heap_bytes(256, 256, 2) == 256 * 256 * 2 + 256 + 256 + 256
    # bad handles are rejected before any CUDA call
    assert L.iris_heap_world(None) == iris.IRIS_ERR_STATE
    assert L.iris_heap_destroy(None) == iris.IRIS_ERR_STATE
    assert b"bad" in L.iris_last_error()


def test_no_cpu_fallback_when_library_is_missing(monkeypatch):
    import paper_2511_12500_b200.binding as b
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", "/nonexistent/libiris_b200.so")
    with pytest.raises(ImportError):
        b.lib()
