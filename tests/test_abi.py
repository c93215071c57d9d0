"""Host-only checks of the C-ABI boundary: the library loads without a GPU and exports every symbol
that include/disco.h declares; the Python binding names the same entry points."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2405_04304_b200 import build, binding
    build.build()
    return binding.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "disco.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(disco_[a-z_0-9]+)\s*\(", text)))


def test_header_declares_the_named_entry_points():
    names = declared_functions()
    for must in ("disco_draft_step", "disco_verify", "disco_verify_ragged", "disco_create", "disco_destroy"):
        assert must in names


def test_library_exports_every_declared_symbol(lib):
    for name in declared_functions():
        assert hasattr(lib, name), f"libdisco.so does not export {name}"


def test_binding_lists_the_same_names(lib):
    from paper_2405_04304_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_strerror_and_argument_checks_need_no_gpu(lib):
    from paper_2405_04304_b200 import binding
    assert binding.strerror(0) == "ok"
    for code in (-1, -2, -3, -4, -5):
        assert binding.strerror(code) and "unknown" not in binding.strerror(code)
    h = ctypes.c_void_p()
    assert lib.disco_create(None, 100, 8, 8, 1, 2, 10, 8) == binding.ERR_INVALID_ARG
    assert lib.disco_create(ctypes.byref(h), 100, 7, 8, 1, 2, 10, 8) == binding.ERR_INVALID_ARG     # d % 8
    assert lib.disco_create(ctypes.byref(h), 100, 8, 8, 1, 2, 9, 8) == binding.ERR_INVALID_ARG      # k != 10
    assert lib.disco_create(ctypes.byref(h), 100, 8, 8, 1, 2, 10, 1000) == binding.ERR_INVALID_ARG  # H too large
    assert lib.disco_create(ctypes.byref(h), 100, 8, 1 << 20, 1, 2, 10, 8) == binding.ERR_UNSUPPORTED_SHAPE
    assert lib.disco_destroy(None) == binding.ERR_INVALID_ARG
    assert h.value is None
    # every per-step entry point refuses a null context before it touches the GPU
    z = ctypes.c_void_p(None)
    assert lib.disco_draft_step(None, z, z, 1, z, z, z, None, 0.5, 1, z, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_draft_step_ppl(None, z, z, 1, z, z, z, 1.0, 1, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_draft_step_sample(None, z, z, 1, z, z, z, None, 0.5, 1, z, z, z, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_verify_ragged(None, z, z, z, z, 1, 1, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_verify_sample_ragged(None, z, z, z, z, z, 1, 1, z, z, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_extract_features(None, z, z, z, z, z, 1, z, z, z, z, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_draft_loop(None, z, 0, z, 1, z, None, 0.5, 1, z, z, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_verify_sl(None, z, z, z, 1, 1, z, 1, 1, z, z, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_iteration(None, z, 0, z, z, z, 1, z, None, 0.5, 1, z, z, z, z, z, z, z, z, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_iteration_host(None, z, 0, z, z, z, 1, z, None, 0.5, 1, z, z, z, z, z, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_draft_step_host(None, z, z, 1, z, z, z, None, 0.5, 1, z, z, z, z, z) == binding.ERR_INVALID_ARG
    assert lib.disco_verify_ragged_host(None, z, z, z, z, 1, 1, z, z, z, z) == binding.ERR_INVALID_ARG


def test_oracle_and_library_share_no_code():
    """Neither side imports or includes the other."""
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2405_04304_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), f"{f} mentions the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".cpp", ".h")):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2405_04304_b200" not in src and "disco.h" not in src and "libdisco" not in src
