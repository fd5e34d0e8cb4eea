"""CPU-side checks: the shared library loads without a GPU and exports every
symbol the public header declares; host-side validation needs no device."""
import ctypes as C
import os
import re

import pytest

import paper_2511_04063_b200 as dq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2511_04063_b200 import build
    build.build()
    return dq.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dartquant.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dq_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(dq.EXPORTED_SYMBOLS)


def test_version_and_status_strings(lib):
    assert "sm_100a" in dq.dq_version()
    seen = {dq.status_string(s) for s in range(9)}
    assert len(seen) == 9


def test_null_arguments_fail_before_any_cuda_call(lib):
    h = C.c_void_p(0)
    assert lib.dq_calib_init(C.byref(h), None, None, None, None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_calib_step(None, 1, None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_calib_get_rotation(None, None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_rotate_apply(None, 0, 1, 1, 1, None, None, 1, None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_calib_status(None) == dq.DQ_ERR_INVALID_ARG
    assert lib.dq_calib_launch_count(None) == 0
    lib.dq_calib_destroy(None)


def test_config_struct_layout_matches_header():
    # int32 d | (pad) | int64 n_tokens | int32 x4 | float lr | (pad) | int64 ldx
    assert C.sizeof(dq.dq_calib_config) == 48
    assert dq.dq_calib_config.n_tokens.offset == 8
    assert dq.dq_calib_config.lr.offset == 36
    assert dq.dq_calib_config.ldx.offset == 40
