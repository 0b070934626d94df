"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2511_03586_b200 import build
    return ctypes.CDLL(build.build())


def _declared():
    text = open(os.path.join(ROOT, "include", "pd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pd_[a-z0-9_]+)\s*\(", text)))


def test_header_declares_the_boundary():
    names = _declared()
    for required in ("pd_softmax", "pd_layernorm", "pd_bias_gelu_residual", "pd_gemm_bf16", "pd_encoder_layer_fwd",
                     "pd_encoder_layer_workspace_bytes", "pd_status_string"):
        assert required in names


def test_every_declared_symbol_is_exported(lib):
    for name in _declared():
        assert hasattr(lib, name), f"{name} is declared in pd.h but not exported by libpd.so"


def test_binding_lists_the_same_entry_points():
    src = open(os.path.join(ROOT, "paper_2511_03586_b200", "api.py")).read()
    for name in _declared():
        assert f'"{name}"' in src or f"_lib.{name}" in src, f"api.py has no binding for {name}"


def test_host_only_calls(lib):
    lib.pd_status_string.restype = ctypes.c_char_p
    assert lib.pd_status_string(0) == b"PD_OK"
    assert lib.pd_status_string(7) == b"PD_ERR_DEVICE_TIMEOUT"
    assert lib.pd_status_string(99) == b"PD_ERR_UNKNOWN"

    class Desc(ctypes.Structure):
        _fields_ = [("batch", ctypes.c_int32), ("seq", ctypes.c_int32), ("hidden", ctypes.c_int32),
                    ("heads", ctypes.c_int32), ("ffn", ctypes.c_int32), ("ln_eps", ctypes.c_float)]
    lib.pd_encoder_layer_workspace_bytes.restype = ctypes.c_size_t
    lib.pd_encoder_layer_workspace_bytes.argtypes = [ctypes.POINTER(Desc)]
    big = lib.pd_encoder_layer_workspace_bytes(ctypes.byref(Desc(32, 512, 1024, 16, 4096, 1e-5)))
    small = lib.pd_encoder_layer_workspace_bytes(ctypes.byref(Desc(1, 512, 1024, 16, 4096, 1e-5)))
    assert 0 < small < big
    assert lib.pd_encoder_layer_workspace_bytes(ctypes.byref(Desc(1, 512, 1000, 16, 4096, 1e-5))) == 0
    assert lib.pd_encoder_layer_workspace_bytes(None) == 0


def test_argument_errors_need_no_device(lib):
    i64 = ctypes.c_int64
    lib.pd_softmax.argtypes = [ctypes.c_void_p, ctypes.c_void_p, i64, i64, ctypes.c_void_p]
    assert lib.pd_softmax(None, None, 4, 4, None) == 1          # PD_ERR_NULL_POINTER
    assert lib.pd_softmax(16, 32, 4, 0, None) == 2              # PD_ERR_BAD_SHAPE
    assert lib.pd_softmax(16, 32, 0, 4, None) == 0              # empty: PD_OK, nothing launched
    assert lib.pd_softmax(18, 32, 4, 4, None) == 4              # PD_ERR_ALIGNMENT
