"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_02047_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "goose.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(goose_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    from paper_2604_02047_b200 import binding
    names = _declared()
    assert len(names) >= 10 and "goose_tree_attn" in names and "goose_kv_compact" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTS) == names


def test_strerror_and_null_context(lib):
    assert lib.goose_strerror(0) == b"ok"
    assert b"invalid" in lib.goose_strerror(-1)
    # argument errors are caught on the host before any CUDA call
    assert lib.goose_set_attn_impl(None, 0) == -1
    assert lib.goose_destroy(None) == -1
    assert lib.goose_node_topk(None, None, 0, 0, ctypes.c_int64(0), 0, None, 0, None, None, None, None) == -1
    out = ctypes.c_void_p()
    assert lib.goose_create(ctypes.byref(out), 0, 0, 128, 32, 128) == -1      # max_S < 1
    assert lib.goose_create(ctypes.byref(out), 0, 1, 129, 32, 128) == -1      # max_B > 128
    assert lib.goose_create(ctypes.byref(out), 0, 1, 128, 32, 64) == -1       # head_dim != 128


def test_product_path_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2604_02047_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in text and "from oracle" not in text and "goose_oracle" not in text, f
    assert "paper_2604_02047_b200" not in open(os.path.join(ROOT, "oracle", "__init__.py")).read()
    assert "goose.h" not in open(os.path.join(ROOT, "oracle", "goose_oracle.c")).read()
