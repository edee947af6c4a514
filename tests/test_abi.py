"""CPU-side checks of the boundary: the shared library builds, loads without a GPU, exports every symbol
the header declares, and rejects bad arguments before touching a device."""
import ctypes
import os
import re

import pytest

import paper_2602_02159_b200 as focus
from paper_2602_02159_b200 import binding as fb
from paper_2602_02159_b200 import build as fbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    fbuild.build()
    return fb.load_library()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "focus.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(focus_[a-z_]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = declared_symbols()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} declared in focus.h but not exported"
    assert set(names) == set(fb._SIGS), "binding and header disagree on the entry points"


def test_status_strings(lib):
    assert fb.status_string(fb.OK) == "ok"
    assert "invalid" in fb.status_string(fb.ERR_INVALID_ARG)
    assert "unknown" in fb.status_string(99)


def test_argument_errors_need_no_device(lib):
    null = None
    assert lib.focus_create(None, 0, 0) == fb.ERR_INVALID_ARG
    assert lib.focus_destroy(None) == fb.ERR_INVALID_ARG
    sh = fb.make_shape(1024, 896, 8, 8, 64, 64, fb.F32)
    out = ctypes.c_size_t(0)
    assert lib.focus_workspace_bytes(ctypes.byref(sh), 128, 4, 8, ctypes.byref(out)) == fb.OK and out.value > 0
    bad = fb.make_shape(1024, 2000, 8, 8, 64, 64, fb.F32)           # M > L
    assert lib.focus_workspace_bytes(ctypes.byref(bad), 128, 4, 8, ctypes.byref(out)) == fb.ERR_INVALID_ARG
    bad = fb.make_shape(1024, 896, 8, 3, 64, 64, fb.F32)            # H % Hkv != 0
    assert lib.focus_workspace_bytes(ctypes.byref(bad), 128, 4, 8, ctypes.byref(out)) == fb.ERR_INVALID_ARG
    # null context / null buffers are rejected on the host
    assert lib.focus_select_queries(null, null, null, 10, 0, 10, 2, 2, 0, 10, null, null, null, null, null) == fb.ERR_INVALID_ARG
    assert lib.focus_pool_keys(null, ctypes.byref(sh), null, null, null) == fb.ERR_INVALID_ARG
    assert lib.focus_dense_attn(null, ctypes.byref(sh), null, 0, 0, null, null, 0, null, null, null, null, null) == fb.ERR_INVALID_ARG


def test_stream_read_rejects_bad_arguments_on_the_host(lib):
    assert lib.focus_stream_read(None, None, 0, None, None) == fb.ERR_INVALID_ARG            # no context


def test_no_device_means_loud_failure(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(focus.FocusError):
        focus.Context(0)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2602_02159_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", src, flags=re.M), f"{f} imports the oracle"
                assert "focus_oracle" not in src, f"{f} names the oracle module"
    src = open(os.path.join(ROOT, "oracle", "focus_oracle.py")).read()
    assert "import paper_2602_02159_b200" not in src and "from paper_2602_02159_b200" not in src


def test_layer_schedule_matches_the_paper():
    """Sparse layers start after the cut-off layer; Dream keeps its final four layers dense (appendix
    'Details of Focus-dLLM')."""
    from paper_2602_02159_b200.step import layer_schedule
    s = layer_schedule(32, 16)
    assert s[:16] == ["dense"] * 16 and s[16] == "probe" and s[17:] == ["sparse"] * 15
    d = layer_schedule(28, 5, final_dense=4)                 # paper: l_dense = 6 (1-indexed) -> probe layer 5
    assert d[:5] == ["dense"] * 5 and d[5] == "probe" and d[6:24] == ["sparse"] * 18 and d[24:] == ["dense"] * 4
    assert layer_schedule(4, 3, final_dense=4) == ["dense", "dense", "dense", "probe"]
