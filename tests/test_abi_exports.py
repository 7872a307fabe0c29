"""The C-ABI library builds, loads without a GPU and exports every symbol include/wide.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2607_28418_b200 import build
    return build.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "wide.h")).read()
    return re.findall(r"WIDE_API\s+[\w\s\*]+?\b(wide_\w+)\s*\(", text)


def test_header_declares_the_five_hot_path_calls():
    names = set(_declared())
    assert {"wide_route", "wide_reorder", "wide_ffn", "wide_oproj", "wide_unpermute"} <= names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in _declared():
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols(lib_path):
    from paper_2607_28418_b200 import binding
    assert set(binding.EXPORTS) <= set(_declared())
    assert set(n for n in _declared() if not n.endswith("_static")) <= set(binding.EXPORTS) | {
        n for n in _declared() if n not in binding.EXPORTS and hasattr(binding, n)}
    header = open(os.path.join(ROOT, "include", "wide.h")).read()
    assert binding.version() == int(re.search(r"#define\s+WIDE_VERSION\s+(\d+)", header).group(1))
    assert binding.strerror(0) == "ok" and "workspace" in binding.strerror(binding.ERR_WORKSPACE)


def test_host_only_calls_without_gpu(lib_path):
    from paper_2607_28418_b200 import binding
    # workspace sizing is pure host arithmetic
    n = binding.workspace_bytes(binding.OP_FFN, binding.BF16, 2048, 4096, 11008, 128, 86)
    assert n >= 2048 * 11008 * 2
    assert binding.workspace_bytes(binding.OP_ROUTE, binding.BF16, 2048, 4096, 0, 0, 86) >= 2048 * 86 * 8
    assert binding.workspace_bytes(binding.OP_FFN, binding.BF16, 8, 4096, 14336, 128, 112) > 0
    # argument validation happens before any CUDA call
    lib = binding.load_library()
    assert lib.wide_route(None, None, None, 0, 1, 8, None, None, 0, 4, 0, 1, None, None, None, None, 0, 0) == \
        binding.ERR_INVALID_ARG
    assert lib.wide_destroy(None) == binding.ERR_INVALID_ARG
