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
    header = re.sub(r"typedef[^;{]*\(\*[^;]*;", "", header)          # function-pointer types are not entry points
    declared = set(re.findall(r"\b(ladder_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations parsed"
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} declared in ladder.h but not exported"
    assert declared == set(B.EXPORTS)


def test_status_strings(L):
    assert L.ladder_status_string(0) == b"ok"
    for s in range(1, 7):
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


def test_misaligned_and_overlong_attention_arguments_are_rejected_on_the_host(L):
    """Argument errors instead of device faults: the decode attention reads its operands with 16-byte loads, and
    its merge step handles at most 1024 splits of 64 keys.  Pointers here are made-up addresses: every call is
    rejected before anything is launched."""
    ok = 0x7F0000001000
    for entry, extra in ((L.ladder_op_decode_attention, (ok,)), (L.ladder_op_decode_attention_noalloc, ())):
        for bad_slot in range(3):                      # q, k, v in turn, 8 bytes off
            ptrs = [ok, ok, ok]
            ptrs[bad_slot] += 8
            assert entry(*ptrs, ok, 1, 8, 8, 128, 64, *extra, ok, None) == 1
        assert entry(ok, ok, ok, ok, 1, 8, 8, 128, 64, *extra, ok + 4, None) == 1          # o
        assert entry(ok, ok, ok, ok, 1, 8, 8, 128, 65537, *extra, ok, None) == 2           # too many splits
    s = SHAPES["tiny"]
    h = C.c_void_p()
    w = B.ladder_weights_t()
    cfg = B.make_config(s, 1, 65537)
    assert L.ladder_model_create(C.byref(cfg), C.byref(w), C.byref(h)) == 2
    assert b"max_seq_len" in L.ladder_last_error(None)


def test_config_struct_versions_and_layer_modes(L):
    """The configuration struct grew by two optional tables: the earlier size is still accepted (the tables are
    then absent), any other size is rejected, and a layer mode outside the defined values is an argument error."""
    from paper_2501_06589_b200.synth import replace
    s = SHAPES["tiny"]
    h = C.c_void_p()
    w = B.ladder_weights_t()
    old_size = B.ladder_config_t.layer_mode.offset
    cfg = B.make_config(s, 1, 32)
    cfg.struct_size = old_size
    assert L.ladder_model_create(C.byref(cfg), C.byref(w), C.byref(h)) == 1      # gets as far as the NULL weights
    assert b"NULL" in L.ladder_last_error(None)
    cfg.struct_size = old_size + 4
    assert L.ladder_model_create(C.byref(cfg), C.byref(w), C.byref(h)) == 1
    assert b"struct_size" in L.ladder_last_error(None)
    cfg = B.make_config(replace(s, layer_mode=("standard", "parallel", "ladder", "upper_bound")), 1, 32)
    assert [cfg.layer_mode[i] for i in range(4)] == [0, 2, 1, 3]
    cfg.layer_mode[1] = 9
    plan = (C.c_int32 * 4096)()
    assert L.ladder_stack_plan(C.byref(cfg), 1, 148, plan, 4096) == -1
