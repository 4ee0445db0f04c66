"""CPU-side checks of the C-ABI library: it builds, loads, and exports every
symbol the header declares.  No compute call is made without a GPU."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2601_07667_b200 import build
    build.build()
    from paper_2601_07667_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "asl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(asl_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert {"asl_score_layer", "asl_rank_stat", "asl_select_topk", "asl_compact_kv"} <= set(names)
    handle = lib.library()
    for name in names:
        assert hasattr(handle, name), f"{name} declared in asl.h but not exported"
    assert set(lib.EXPORTS) <= set(names)


def test_struct_sizes_match_the_header(lib):
    assert ctypes.sizeof(lib.AslStat) == 64
    assert ctypes.sizeof(lib.AslParams) == 4 * 10 + 8 + 8 * 2 + 8 * 7 + 4 * 2 + 8      # ..., k_dtype, reserved0, k_scale


def test_strerror_and_null_handling(lib):
    assert lib.asl_strerror(0) == "ok"
    assert "workspace" in lib.asl_strerror(lib.ASL_ERR_WORKSPACE)
    assert "sm_100" in lib.asl_strerror(lib.ASL_ERR_ARCH)
    assert lib.library().asl_destroy(None) == lib.ASL_ERR_INVALID
    assert lib.library().asl_plan(None, None, None) == lib.ASL_ERR_INVALID


def test_create_fails_loudly_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(lib.AslError):
        lib.asl_create(0)
