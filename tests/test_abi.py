"""The C ABI on a machine without a GPU: the library builds, loads, exports every function that
include/fastcot.h declares, and its host-only entry points (sizes, status strings, argument checks) behave."""
import ctypes as C
import os
import re

import pytest

from paper_2311_08263_b200 import build, lib

HEADER = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "include", "fastcot.h")


def _declared_functions():
    text = open(HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)          # comments mention names too
    names = set(re.findall(r"\b(fc_[a-z0-9_]+)\s*\(", text))
    assert len(names) >= 20
    return sorted(names)


@pytest.fixture(scope="module")
def cdll():
    path = build.build()
    return C.CDLL(path)


def test_library_exports_every_declared_function(cdll):
    missing = [n for n in _declared_functions() if not hasattr(cdll, n)]
    assert not missing, missing


def test_binding_names_match_the_header():
    l = lib.load()
    for n in _declared_functions():
        assert hasattr(l, n), n


def test_status_strings(cdll):
    cdll.fc_strerror.restype = C.c_char_p
    seen = set()
    for code in (lib.FC_OK, lib.FC_ERR_ARG, lib.FC_ERR_SHAPE, lib.FC_ERR_CAPACITY, lib.FC_ERR_TOKEN_RANGE, lib.FC_ERR_STATE,
                 lib.FC_ERR_BAD_WINDOW, lib.FC_ERR_DEVICE_TIMEOUT, lib.FC_ERR_CUDA):
        s = cdll.fc_strerror(code)
        assert s and s not in seen
        seen.add(s)
    assert cdll.fc_strerror(-12345) == b"unknown status"


def _shape(**kw):
    s = lib.fc_model_shape()
    vals = dict(n_layers=2, d_model=128, n_heads=4, n_kv_heads=4, head_dim=32, d_ffn=512, vocab=512, dtype=lib.FC_F32,
                rms_eps=1e-5, rope_theta=1e4, max_batch=1, max_c=8, max_seq=64, bias_beta=0.0, flags=0)
    vals.update(kw)
    for k, v in vals.items():
        setattr(s, k, v)
    return s


def test_sizes_are_host_arithmetic(cdll):
    cdll.fc_kv_bytes.restype = C.c_size_t
    cdll.fc_workspace_bytes.restype = C.c_size_t
    s = _shape()
    # [layer][K|V][batch][kv_head][max_seq][head_dim] fp32
    assert cdll.fc_kv_bytes(C.byref(s)) == 2 * 2 * 1 * 4 * 64 * 32 * 4
    assert cdll.fc_kv_bytes(C.byref(_shape(dtype=lib.FC_BF16))) == 2 * 2 * 1 * 4 * 64 * 32 * 2
    ws = cdll.fc_workspace_bytes(C.byref(s))
    assert ws > 0 and ws % 256 == 0
    assert cdll.fc_workspace_bytes(C.byref(_shape(max_batch=4))) > ws
    # shapes the library refuses report size 0
    for bad in (dict(head_dim=48), dict(n_heads=3, n_kv_heads=2), dict(max_c=65), dict(d_model=100), dict(dtype=7),
                dict(max_seq=8)):
        assert cdll.fc_kv_bytes(C.byref(_shape(**bad))) == 0
        assert cdll.fc_workspace_bytes(C.byref(_shape(**bad))) == 0


def test_init_rejects_bad_arguments_before_touching_the_device(cdll):
    ctx = C.c_void_p()
    s = _shape()
    w = lib.fc_weights()
    assert cdll.fc_init(C.byref(ctx), None, C.byref(w), None, 0, None, 0, None) == lib.FC_ERR_ARG
    assert cdll.fc_init(C.byref(ctx), C.byref(s), C.byref(w), None, 0, None, 0, None) == lib.FC_ERR_ARG
    assert ctx.value is None
    cdll.fc_destroy(None)                                          # destroying nothing is allowed
    cdll.fc_last_launch_count.restype = C.c_int64
    assert cdll.fc_last_launch_count(None) == 0
