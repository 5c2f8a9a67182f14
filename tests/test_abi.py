"""The C-ABI library loads and exports every symbol include/embedpart.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "embedpart.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ep_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_01000_b200 import build, binding
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    names = _declared()
    assert {"ep_kmeans", "ep_partition_quality", "ep_reorder", "ep_create", "ep_destroy"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_binding_lists_the_same_symbols():
    from paper_2604_01000_b200 import binding
    assert sorted(binding.EXPORTED_SYMBOLS) == _declared()


def test_status_strings(lib):
    assert lib.ep_status_string(0) == b"ok"
    seen = {lib.ep_status_string(i) for i in range(7)}
    assert len(seen) == 7
    assert lib.ep_status_string(99) == b"unknown status"


def test_null_arguments_are_rejected_without_a_device(lib):
    assert lib.ep_create(None, 0) == 1
    assert lib.ep_destroy(None) == 1
    assert lib.ep_poll_status(None) == 1
    assert lib.ep_kmeans_workspace_bytes(None, 10, 8, 2) == 0
    assert lib.ep_kmeans(None, None, 10, 8, 2, 1, None, None, None, None, None, 0, None) == 1
    assert lib.ep_reorder(None, None, 10, 2, None, None, None, 0, None) == 1


def test_product_has_no_cpu_fallback_and_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2604_01000_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), f
