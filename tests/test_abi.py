"""The C-ABI library loads without a GPU and exports every symbol the header declares;
host-side argument handling that needs no device is exercised too."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib_path():
    from paper_2603_10846_b200 import build
    return build.build()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "evk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(evk_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_four_hot_calls():
    names = declared_functions()
    for need in ("evk_mem_create", "evk_mem_insert", "evk_retrieve", "evk_q_update"):
        assert need in names


def test_library_exports_every_declared_symbol(lib_path):
    lib = ctypes.CDLL(lib_path)
    for name in declared_functions():
        assert hasattr(lib, name), name


def test_binding_covers_the_header(lib_path):
    from paper_2603_10846_b200 import evk
    assert sorted(evk.EXPORTS) == declared_functions()
    for name in evk.EXPORTS:
        assert hasattr(evk._lib, name)


def test_sizes_and_messages_without_a_device(lib_path):
    from paper_2603_10846_b200 import evk
    n = evk.evk_mem_bytes_required(1024, 1 << 20, 2)
    assert n >= (1 << 20) * 1024 * 2 + 2 * (1 << 20) * 4 and n % 256 == 0
    for bad in ((12, 100, 2), (0, 100, 2), (4096, 100, 2), (64, 0, 2), (64, 1 << 31, 2), (64, 100, 0), (64, 100, 9)):
        with pytest.raises(evk.EvkError):
            evk.evk_mem_bytes_required(*bad)
    assert evk.strerror(0) == "ok"
    codes = [evk.EVK_ERR_INVALID, evk.EVK_ERR_CAPACITY, evk.EVK_ERR_WORKSPACE, evk.EVK_ERR_RANGE,
             evk.EVK_ERR_NONFINITE, evk.EVK_ERR_DEVICE_TIMEOUT, evk.EVK_ERR_CUDA, evk.EVK_ERR_UNSUPPORTED,
             evk.EVK_ERR_INCOMPLETE]
    assert len({evk.strerror(c) for c in codes}) == len(codes)
    # null handles are refused, not dereferenced
    assert evk._lib.evk_mem_size(None) == 0
    assert evk._lib.evk_mem_insert(None, None, 0, 0, 0, None, None, None) == evk.EVK_ERR_INVALID
    assert evk._lib.evk_retrieve(None, None, 0, 1, 0, 8, 2, 0.5, None, None, None, None, None, 0, None) == evk.EVK_ERR_INVALID
    assert evk._lib.evk_q_update(None, None, 1, 0, None, 0.5, None, 0, None) == evk.EVK_ERR_INVALID
    out = ctypes.c_void_p()
    assert evk._lib.evk_mem_create(None, ctypes.byref(out)) == evk.EVK_ERR_INVALID


def test_product_code_never_touches_the_oracle():
    # the package, the headers and the kernels must not import, read or link the oracle
    pkg = os.path.join(ROOT, "paper_2603_10846_b200")
    for base, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h", ".cpp")):
                text = open(os.path.join(base, f)).read()
                assert "oracle" not in text.lower(), os.path.join(base, f)
