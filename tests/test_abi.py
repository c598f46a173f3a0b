"""The C-ABI library loads and exports every symbol include/tpq.h declares; the
context-free entry points agree with the oracle's closed forms.  No GPU needed."""
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2411_07942_b200 import build, binding

    build.build()
    return binding.lib()


def _declared():
    text = open(os.path.join(ROOT, "include", "tpq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tpq_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    from paper_2411_07942_b200 import binding

    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in tpq.h but not exported"
        assert n in binding.SIGNATURES, f"{n} has no ctypes signature"
    assert sorted(binding.SIGNATURES) == names


def test_status_strings_and_version(lib):
    assert lib.tpq_status_string(0) == b"ok"
    seen = {lib.tpq_status_string(i) for i in range(8)}
    assert len(seen) == 8
    assert b"sm_100a" in lib.tpq_version()


@pytest.mark.parametrize("T,E,k", [(1, 8, 0), (3, 65, 1), (16, 256, 4), (2048, 5120, 80), (64, 4608, 72),
                                   (8192, 8192, 128), (7, 253, 9), (5, 33, 33)])
def test_payload_bytes_closed_form(lib, corc, T, E, k):
    assert lib.tpq_payload_bytes_for(T, E, k) == corc.payload_bytes(T, E, k)


def test_payload_bytes_degenerate(lib):
    assert lib.tpq_payload_bytes_for(0, 8, 0) == 0
    assert lib.tpq_payload_bytes_for(4, 8, 9) == 0
    assert lib.tpq_payload_bytes(None, 16) == 0


def test_null_context_is_rejected_not_crashed(lib):
    assert lib.tpq_destroy(None) == 0
    assert lib.tpq_quantize_pack(None, 0, None, 1, 8, None, 0, None) == 1
    assert lib.tpq_dequant_reduce(None, None, 0, 1, None, 0, 8, None) == 1
    assert lib.tpq_calibrate_ranges(None, 0, None, 1, 1, 8, None) == 1
    assert lib.tpq_select_features(None, -1, None, None) == 1
    assert lib.tpq_last_error(None) == b""
    assert lib.tpq_num_selected(None) == -1


def test_create_validates_before_touching_cuda(lib):
    import ctypes

    h = ctypes.c_void_p()
    for args in [(0, 8, 4, 0.01), (2, 0, 4, 0.01), (2, 8, 9, 0.01), (2, 8, 1, 0.01), (2, 8, 4, -0.5), (2, 8, 4, 1.5), (65, 8, 4, 0.01)]:
        assert lib.tpq_create(ctypes.byref(h), *args) == 1
        assert not h.value
    assert lib.tpq_create(None, 2, 8, 4, 0.01) == 1


def test_product_never_imports_the_oracle():
    """The product path shares nothing with the oracle: no file of the package names it."""
    pkg = os.path.join(ROOT, "paper_2411_07942_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "tpqo_" not in src, f
