"""Host-only checks of the C ABI: the library loads, exports every declared symbol, and rejects
bad arguments before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2501_06589_b200 import binding as B
from paper_2501_06589_b200 import build as builder
from paper_2501_06589_b200.synth import SHAPES

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    builder.build()
    return B.lib()


def test_every_declared_symbol_is_exported(L):
    header = open(os.path.join(ROOT, "include", "ladder.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ladder_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in ladder.h but not exported"
    assert declared == set(B.EXPORTS)


def test_status_strings(L):
    assert L.ladder_status_string(0) == b"ok"
    for s in range(1, 6):
        assert L.ladder_status_string(s) not in (b"ok", b"unknown status")
    assert L.ladder_status_string(99) == b"unknown status"


def test_kv_cache_bytes(L):
    s = SHAPES["70b"]
    cfg = B.make_config(s, 4, 1536)
    assert L.ladder_kv_cache_bytes(C.byref(cfg)) == 80 * 4 * 8 * 1536 * 128 * 2
    assert L.ladder_kv_cache_bytes(None) == 0


def test_create_rejects_bad_arguments_before_any_device_work(L):
    s = SHAPES["tiny"]
    h = C.c_void_p()
    w = B.ladder_weights_t()
    assert L.ladder_model_create(None, C.byref(w), C.byref(h)) == 1
    cfg = B.make_config(s, 1, 32)
    cfg.struct_size = 7
    assert L.ladder_model_create(C.byref(cfg), C.byref(w), C.byref(h)) == 1
    cfg = B.make_config(s, 1, 32)
    cfg.head_dim = 96
    assert L.ladder_model_create(C.byref(cfg), C.byref(w), C.byref(h)) == 2
    assert b"head_dim" in L.ladder_last_error(None)
    cfg = B.make_config(s, 65, 32)
    assert L.ladder_model_create(C.byref(cfg), C.byref(w), C.byref(h)) == 2
    cfg = B.make_config(s, 1, 32)
    assert L.ladder_model_create(C.byref(cfg), C.byref(w), C.byref(h)) == 1      # NULL weights
    assert h.value is None


def test_null_model_calls_are_rejected(L):
    assert L.ladder_destroy(None) == 0
    assert L.ladder_set_position(None, 0) == 1
    assert L.ladder_model_set_schedule(None, 2, 1, 1) == 1
    assert L.ladder_kernel_launches(None) == 0
    assert L.ladder_decode_step(None, None, None, 1, None, None) == 1
    assert L.ladder_prefill(None, None, None, 1, 1, None, None) == 1


def test_op_entry_points_validate_arguments(L):
    assert L.ladder_op_smallm_gemm(None, 8, 8, None, 0, None, 0.0, 1, 0, None, None, None) == 1
    assert L.ladder_op_decode_attention(None, None, None, None, 1, 8, 8, 128, 16, None, None, None) == 1
    assert L.ladder_op_prefill_gemm(None, None, None, 1, 8, 8, 0, None, None, None, None) == 1
    assert L.ladder_op_prefill_attention(None, None, None, None, 1, 1, 8, 8, 128, 16, None, None, None) == 1
    assert L.ladder_decode_attention_scratch_bytes(0, 8, 128, 16) == 0
    assert L.ladder_decode_attention_scratch_bytes(4, 64, 128, 1536) > 0
