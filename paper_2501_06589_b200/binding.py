"""ctypes binding of libladder.so: argument marshalling only.

Every function here forwards to the C entry point of the same name declared in
``include/ladder.h``; tensors are torch CUDA tensors used purely as device
memory, and the CUDA stream is torch's current stream.  There is no fallback:
if the library is missing, importing :func:`lib` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

from .synth import AbiWeights, ModelShape

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libladder.so")

EXPORTS = [
    "ladder_kv_cache_bytes", "ladder_model_create", "ladder_model_set_schedule", "ladder_model_set_sm_split", "ladder_model_set_persistent", "ladder_model_persistent_active", "ladder_stack_plan", "ladder_debug_stall_last_phase",
    "ladder_prefill", "ladder_prefill_append", "ladder_prefill_ragged", "ladder_stage_prefill", "ladder_stage_decode_step",
    "ladder_decode_step", "ladder_decode_step_host", "ladder_prefill_host", "ladder_set_position",
    "ladder_device_status", "ladder_kernel_launches", "ladder_destroy", "ladder_status_string",
    "ladder_last_error", "ladder_op_smallm_gemm", "ladder_decode_attention_scratch_bytes",
    "ladder_op_decode_attention", "ladder_op_prefill_gemm", "ladder_op_prefill_attention", "ladder_op_prefill_attention_at",
    "ladder_op_decode_attention_noalloc", "ladder_set_prefill_gemm_impl", "ladder_set_decode_wide_impl", "ladder_set_decode_attention_impl",
    "ladder_op_prefill_gemm_f16", "ladder_op_convert_bf16_f16",
    "ladder_model_set_exchange", "ladder_model_set_tensor_parallel", "ladder_comm_unique_id", "ladder_comm_create",
    "ladder_comm_destroy", "ladder_comm_world", "ladder_comm_rank", "ladder_comm_all_reduce_sum",
    "ladder_peer_create", "ladder_peer_export", "ladder_peer_local_base", "ladder_peer_connect", "ladder_peer_connected",
    "ladder_peer_world", "ladder_peer_rank", "ladder_peer_max_floats", "ladder_peer_ctas_per_exchange",
    "ladder_peer_destroy", "ladder_peer_all_reduce_sum", "ladder_peer_probe_write", "ladder_peer_probe_read",
    "ladder_peer_slot", "ladder_peer_counter", "ladder_model_set_tensor_parallel_peer", "ladder_model_set_peer",
    "ladder_debug_set_peer_hook", "ladder_model_set_peer_max_bytes",
]
PEER_HOOK_FN = C.CFUNCTYPE(None, C.c_void_p, C.c_int32, C.c_void_p)                # ladder_peer_hook_fn
PEER_HANDLE_BYTES = 64                                                           # LADDER_PEER_HANDLE_BYTES

COMM_ID_BYTES = 128                                                              # LADDER_COMM_ID_BYTES
EXCHANGE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p)   # ladder_exchange_fn


class LadderError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(f"libladder status {status}: {msg}")
        self.status = status


class ladder_config_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("d_model", C.c_int32), ("n_layers", C.c_int32),
                ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("d_ff", C.c_int32), ("vocab_size", C.c_int32), ("rms_eps", C.c_float),
                ("rope_theta", C.c_float), ("max_batch", C.c_int32), ("max_seq_len", C.c_int32),
                ("max_prefill_tokens", C.c_int32), ("layer_is_ladder", C.POINTER(C.c_uint8)),
                ("layer_mode", C.POINTER(C.c_uint8)), ("module_stale", C.POINTER(C.c_uint8))]


LAYER_MODES = {"standard": 0, "ladder": 1, "parallel": 2, "upper_bound": 3}      # LADDER_LAYER_*


class ladder_weights_t(C.Structure):
    _fields_ = [("tok_embedding", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
                ("attn_norm", C.POINTER(C.c_void_p)), ("w_qkv", C.POINTER(C.c_void_p)),
                ("w_o", C.POINTER(C.c_void_p)), ("mlp_norm", C.POINTER(C.c_void_p)),
                ("w_gate_up", C.POINTER(C.c_void_p)), ("w_down", C.POINTER(C.c_void_p))]


class ladder_kv_cache_t(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("seq_lens", C.c_void_p)]


class ladder_stream_state_t(C.Structure):
    _fields_ = [("newest", C.c_void_p), ("older", C.c_void_p)]


class ladder_outputs_t(C.Structure):
    _fields_ = [("next_tokens", C.c_void_p), ("final_hidden", C.c_void_p), ("logits", C.c_void_p),
                ("all_hidden", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Load libladder.so (built in-tree by paper_2501_06589_b200.build); fails loudly if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(f"{LIB_PATH} not built: run `python -m paper_2501_06589_b200.build`")
        L = C.CDLL(LIB_PATH)
        L.ladder_kv_cache_bytes.restype = C.c_size_t
        L.ladder_kv_cache_bytes.argtypes = [C.POINTER(ladder_config_t)]
        L.ladder_model_create.argtypes = [C.POINTER(ladder_config_t), C.POINTER(ladder_weights_t),
                                          C.POINTER(C.c_void_p)]
        L.ladder_model_set_schedule.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32]
        L.ladder_model_set_sm_split.argtypes = [C.c_void_p, C.c_int32]
        L.ladder_model_set_persistent.argtypes = [C.c_void_p, C.c_int32]
        L.ladder_model_persistent_active.argtypes = [C.c_void_p]
        L.ladder_model_persistent_active.restype = C.c_int32
        L.ladder_debug_stall_last_phase.argtypes = [C.c_void_p, C.c_int32]
        L.ladder_stack_plan.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32]
        L.ladder_stack_plan.restype = C.c_int32
        L.ladder_prefill.argtypes = [C.c_void_p, C.POINTER(ladder_kv_cache_t), C.c_void_p, C.c_int32, C.c_int32,
                                     C.POINTER(ladder_outputs_t), C.c_void_p]
        L.ladder_prefill_append.argtypes = [C.c_void_p, C.POINTER(ladder_kv_cache_t), C.c_void_p, C.c_int32, C.c_int32,
                                     C.POINTER(ladder_outputs_t), C.c_void_p]
        L.ladder_prefill_ragged.argtypes = [C.c_void_p, C.POINTER(ladder_kv_cache_t), C.c_void_p, C.c_void_p, C.c_int32,
                                            C.c_int32, C.POINTER(ladder_outputs_t), C.c_void_p]
        L.ladder_stage_prefill.argtypes = [C.c_void_p, C.POINTER(ladder_kv_cache_t), C.c_void_p,
                                           C.POINTER(ladder_stream_state_t), C.c_int32, C.c_int32,
                                           C.POINTER(ladder_stream_state_t), C.POINTER(ladder_outputs_t), C.c_void_p]
        L.ladder_stage_decode_step.argtypes = [C.c_void_p, C.POINTER(ladder_kv_cache_t), C.c_void_p,
                                               C.POINTER(ladder_stream_state_t), C.c_int32,
                                               C.POINTER(ladder_stream_state_t), C.POINTER(ladder_outputs_t), C.c_void_p]
        L.ladder_decode_step.argtypes = [C.c_void_p, C.POINTER(ladder_kv_cache_t), C.c_void_p, C.c_int32,
                                         C.POINTER(ladder_outputs_t), C.c_void_p]
        L.ladder_decode_step_host.argtypes = [C.c_void_p, C.POINTER(ladder_kv_cache_t), C.c_void_p, C.c_int32,
                                              C.c_void_p, C.c_void_p]
        L.ladder_prefill_host.argtypes = [C.c_void_p, C.POINTER(ladder_kv_cache_t), C.c_void_p, C.c_int32,
                                          C.c_int32, C.c_void_p, C.c_void_p]
        L.ladder_set_position.argtypes = [C.c_void_p, C.c_int32]
        L.ladder_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.c_void_p]
        L.ladder_kernel_launches.restype = C.c_int64
        L.ladder_kernel_launches.argtypes = [C.c_void_p]
        L.ladder_destroy.argtypes = [C.c_void_p]
        L.ladder_status_string.restype = C.c_char_p
        L.ladder_status_string.argtypes = [C.c_int]
        L.ladder_last_error.restype = C.c_char_p
        L.ladder_last_error.argtypes = [C.c_void_p]
        L.ladder_op_smallm_gemm.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p,
                                            C.c_float, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ladder_decode_attention_scratch_bytes.restype = C.c_size_t
        L.ladder_decode_attention_scratch_bytes.argtypes = [C.c_int32] * 4
        L.ladder_op_decode_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                                 C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                                 C.c_void_p, C.c_void_p]
        L.ladder_op_decode_attention_noalloc.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                                         C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p,
                                                         C.c_void_p]
        L.ladder_set_prefill_gemm_impl.restype = None
        L.ladder_set_prefill_gemm_impl.argtypes = [C.c_int32]
        L.ladder_set_decode_wide_impl.restype = None
        L.ladder_set_decode_wide_impl.argtypes = [C.c_int32]
        L.ladder_set_decode_attention_impl.restype = None
        L.ladder_set_decode_attention_impl.argtypes = [C.c_int32]
        L.ladder_op_prefill_gemm.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                             C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.ladder_op_prefill_gemm_f16.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                 C.c_void_p, C.c_void_p, C.c_void_p]
        L.ladder_op_convert_bf16_f16.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.ladder_op_prefill_attention.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                                  C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                  C.c_void_p, C.c_void_p, C.c_void_p]
        L.ladder_op_prefill_attention_at.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32,
                                                     C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                                     C.c_int32, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                                     C.c_void_p]
        L.ladder_model_set_exchange.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32]
        L.ladder_model_set_tensor_parallel.argtypes = [C.c_void_p, C.c_void_p]
        L.ladder_comm_unique_id.argtypes = [C.c_void_p]
        L.ladder_comm_create.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.POINTER(C.c_void_p)]
        L.ladder_comm_destroy.argtypes = [C.c_void_p]
        L.ladder_comm_world.argtypes = [C.c_void_p]
        L.ladder_comm_world.restype = C.c_int32
        L.ladder_comm_rank.argtypes = [C.c_void_p]
        L.ladder_comm_rank.restype = C.c_int32
        L.ladder_comm_all_reduce_sum.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.ladder_peer_create.argtypes = [C.c_int32, C.c_int32, C.c_int64, C.POINTER(C.c_void_p)]
        L.ladder_peer_export.argtypes = [C.c_void_p, C.c_void_p]
        L.ladder_peer_local_base.argtypes = [C.c_void_p]
        L.ladder_peer_local_base.restype = C.c_void_p
        L.ladder_peer_connect.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        for f in (L.ladder_peer_connected, L.ladder_peer_world, L.ladder_peer_rank):
            f.argtypes, f.restype = [C.c_void_p], C.c_int32
        L.ladder_peer_max_floats.argtypes, L.ladder_peer_max_floats.restype = [C.c_void_p], C.c_int64
        L.ladder_peer_ctas_per_exchange.argtypes, L.ladder_peer_ctas_per_exchange.restype = [], C.c_int32
        L.ladder_peer_destroy.argtypes = [C.c_void_p]
        L.ladder_peer_all_reduce_sum.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
        L.ladder_peer_probe_write.argtypes = [C.c_void_p, C.c_int32, C.c_uint32]
        L.ladder_peer_probe_read.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_uint32)]
        L.ladder_peer_slot.argtypes, L.ladder_peer_slot.restype = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32], C.c_void_p
        L.ladder_peer_counter.argtypes, L.ladder_peer_counter.restype = [C.c_void_p, C.c_int32, C.c_int32], C.c_void_p
        L.ladder_model_set_tensor_parallel_peer.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.ladder_model_set_peer.argtypes = [C.c_void_p, C.c_void_p]
        L.ladder_model_set_peer_max_bytes.argtypes = [C.c_void_p, C.c_int64]
        L.ladder_debug_set_peer_hook.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous()
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, model=None):
    if status != 0:
        L = lib()
        msg = L.ladder_status_string(status).decode()
        detail = L.ladder_last_error(model).decode() if True else ""
        raise LadderError(status, f"{msg}: {detail}")


def make_config(shape: ModelShape, max_batch: int, max_seq_len: int, max_prefill_tokens: int = 0):
    mask = (C.c_uint8 * shape.n_layers)(*shape.ladder_mask())
    modes = flags = None
    if shape.layer_mode is not None:
        modes = (C.c_uint8 * shape.n_layers)(*[LAYER_MODES[m] for m in shape.layer_mode])
    if shape.module_stale is not None:
        flags = (C.c_uint8 * (2 * shape.n_layers))(*[int(bool(f)) for f in shape.module_stale])
    u8p = C.POINTER(C.c_uint8)
    cfg = ladder_config_t(C.sizeof(ladder_config_t), shape.d_model, shape.n_layers, shape.n_q_heads,
                          shape.n_kv_heads, shape.head_dim, shape.d_ff, shape.vocab_size, shape.rms_eps,
                          shape.rope_theta, max_batch, max_seq_len, max_prefill_tokens,
                          C.cast(mask, u8p), C.cast(modes, u8p) if modes is not None else None,
                          C.cast(flags, u8p) if flags is not None else None)
    cfg._keep = (mask, modes, flags)
    return cfg


def stack_plan(shape: ModelShape, batch: int, max_seq_len: int, sm_count: int = 148):
    """Phase list of the persistent decode kernel for this configuration (host only, no GPU needed)."""
    cfg = make_config(shape, batch, max_seq_len)
    cap = 8 + 56 * (4 * shape.n_layers + 1) + 29 * shape.n_layers
    buf = (C.c_int32 * cap)()
    n = lib().ladder_stack_plan(C.byref(cfg), batch, sm_count, buf, cap)
    if n < 0:
        raise RuntimeError(f"ladder_stack_plan failed ({n})")
    w = list(buf[:n])
    n_ph, n_at, n_ctr, begin, ok = w[:5]
    pos, phases, attn = 5, [], []
    for _ in range(n_ph):
        r = w[pos:pos + 56]
        pos += 56
        phases.append(dict(kind=r[0], layer=r[1], N=r[2], K=r[3], n_units=r[4], n_static=r[5], n_claims=r[6],
                           work=r[7], done=r[8], rounds=list(zip(r[10:10 + r[9]], r[20:20 + r[9]])),
                           act_deps=list(zip(r[31:31 + r[30]], r[37:37 + r[30]])),
                           epi_deps=list(zip(r[44:44 + r[43]], r[50:50 + r[43]]))))
    for _ in range(n_at):
        r = w[pos:pos + 29]
        pos += 29
        attn.append(dict(layer=r[0], split=r[1], merge=r[2], deps=list(zip(r[4:4 + r[3]], r[10:10 + r[3]])),
                         merge_deps=list(zip(r[17:17 + r[16]], r[23:23 + r[16]]))))
    assert pos == n
    return dict(phases=phases, attn=attn, n_counters=n_ctr, first_layer=begin, ok=bool(ok))


class KVCache:
    """Caller-owned cache buffers (torch device memory) for one model configuration."""

    def __init__(self, shape: ModelShape, max_batch: int, max_seq_len: int, device="cuda", fill: Optional[int] = None):
        n = shape.n_layers * max_batch * shape.n_kv_heads * max_seq_len * shape.head_dim
        self.k = torch.empty(n, dtype=torch.float16, device=device)     # binary16: see ladder_kv_cache_t
        self.v = torch.empty(n, dtype=torch.float16, device=device)
        if fill is not None:       # canary pattern for indexing tests
            self.k.view(torch.int16).fill_(fill)
            self.v.view(torch.int16).fill_(fill)
        self.seq_lens = torch.zeros(max_batch, dtype=torch.int32, device=device)
        self.dims = (shape.n_layers, max_batch, shape.n_kv_heads, max_seq_len, shape.head_dim)
        self.c = ladder_kv_cache_t(self.k.data_ptr(), self.v.data_ptr(), self.seq_lens.data_ptr())

    def slot(self, b: int) -> "KVCache":
        """The same buffers seen from sequence b on (its rows of every layer come first, its length first in
        seq_lens): a prompt pass with batch 1 on it fills sequence b alone, so sequences of different lengths can
        be filled one by one and then decoded together."""
        view = object.__new__(KVCache)
        _, mb, hkv, ms, dh = self.dims
        off = b * hkv * ms * dh
        view.k, view.v, view.seq_lens, view.dims = self.k[off:], self.v[off:], self.seq_lens[b:], self.dims
        view.c = ladder_kv_cache_t(view.k.data_ptr(), view.v.data_ptr(), view.seq_lens.data_ptr())
        return view

    def k5(self) -> torch.Tensor:
        return self.k.view(*self.dims)

    def v5(self) -> torch.Tensor:
        return self.v.view(*self.dims)


class Comm:
    """Owns a ladder_comm_t (one NCCL communicator of this process's current CUDA device)."""

    def __init__(self, world: int, rank: int, unique_id: bytes):
        assert len(unique_id) == COMM_ID_BYTES
        h = C.c_void_p()
        buf = C.create_string_buffer(unique_id, COMM_ID_BYTES)
        _check(lib().ladder_comm_create(world, rank, buf, C.byref(h)))
        self.h, self.world, self.rank = h, world, rank

    @staticmethod
    def unique_id() -> bytes:
        buf = C.create_string_buffer(COMM_ID_BYTES)
        _check(lib().ladder_comm_unique_id(buf))
        return buf.raw

    def all_reduce_sum(self, t: torch.Tensor):
        assert t.dtype == torch.float32 and t.is_cuda and t.is_contiguous()
        _check(lib().ladder_comm_all_reduce_sum(self.h, t.data_ptr(), t.numel(), _stream()))

    def close(self):
        if getattr(self, "h", None):
            lib().ladder_comm_destroy(self.h)
            self.h = None


class Peer:
    """Owns a ladder_peer_t: this rank's receive slots for the exchange over peer memory, and the peers' addresses."""

    def __init__(self, world: int, rank: int, max_floats: int):
        h = C.c_void_p()
        _check(lib().ladder_peer_create(world, rank, max_floats, C.byref(h)))
        self.h, self.world, self.rank, self.max_floats = h, world, rank, max_floats

    def export(self) -> bytes:
        buf = C.create_string_buffer(PEER_HANDLE_BYTES)
        _check(lib().ladder_peer_export(self.h, buf))
        return buf.raw

    def local_base(self) -> int:
        return lib().ladder_peer_local_base(self.h)

    def connect(self, r: int, ipc_handle: Optional[bytes] = None, same_process_base: Optional[int] = None):
        buf = C.create_string_buffer(ipc_handle, PEER_HANDLE_BYTES) if ipc_handle is not None else None
        _check(lib().ladder_peer_connect(self.h, r, buf, same_process_base))

    def connected(self) -> bool:
        return bool(lib().ladder_peer_connected(self.h))

    @staticmethod
    def ctas_per_exchange() -> int:
        return lib().ladder_peer_ctas_per_exchange()

    def all_reduce_sum(self, channel: int, ptr: int, count: int, status_ptr: Optional[int] = None, stream: Optional[int] = None):
        _check(lib().ladder_peer_all_reduce_sum(self.h, channel, ptr, count, status_ptr,
                                                _stream() if stream is None else stream))

    def probe_write(self, r: int, value: int):
        _check(lib().ladder_peer_probe_write(self.h, r, value))

    def probe_read(self, frm: int) -> int:
        v = C.c_uint32(0)
        _check(lib().ladder_peer_probe_read(self.h, frm, C.byref(v)))
        return v.value

    def slot_ptr(self, channel: int, parity: int, frm: int) -> int:
        return lib().ladder_peer_slot(self.h, channel, parity, frm)

    def counter_ptr(self, channel: int, frm: int) -> int:
        return lib().ladder_peer_counter(self.h, channel, frm)

    def close(self):
        if getattr(self, "h", None):
            lib().ladder_peer_destroy(self.h)
            self.h = None


class Model:
    """Owns a ladder_model_t; keeps the borrowed weight tensors alive."""

    def __init__(self, weights: AbiWeights, max_batch: int, max_seq_len: int, max_prefill_tokens: int = 0):
        L = lib()
        s = weights.shape
        self.shape, self.weights = s, weights
        self.max_batch, self.max_seq_len = max_batch, max_seq_len
        self._cfg = make_config(s, max_batch, max_seq_len, max_prefill_tokens)

        def arr(ts: Sequence[torch.Tensor]):
            return (C.c_void_p * len(ts))(*[t.data_ptr() for t in ts])

        self._arrs = [arr(weights.attn_norm), arr(weights.w_qkv), arr(weights.w_o), arr(weights.mlp_norm),
                      arr(weights.w_gate_up), arr(weights.w_down)]
        w = ladder_weights_t(weights.tok_embedding.data_ptr(), weights.final_norm.data_ptr(),
                             weights.lm_head.data_ptr(), *[C.cast(a, C.POINTER(C.c_void_p)) for a in self._arrs])
        h = C.c_void_p()
        _check(L.ladder_model_create(C.byref(self._cfg), C.byref(w), C.byref(h)))
        self.h = h

    def close(self):
        if getattr(self, "h", None):
            lib().ladder_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_schedule(self, n_streams: int = 2, use_graph: bool = True, use_pdl: bool = True):
        _check(lib().ladder_model_set_schedule(self.h, n_streams, int(use_graph), int(use_pdl)), self.h)

    def set_persistent(self, on=True):
        """False / 0: one kernel per GEMM; True / 1: the default split; 2: every layer in the persistent kernel."""
        _check(lib().ladder_model_set_persistent(self.h, int(on)), self.h)

    def debug_stall_last_phase(self, on: bool):
        _check(lib().ladder_debug_stall_last_phase(self.h, int(on)), self.h)

    def persistent_active(self) -> bool:
        return bool(lib().ladder_model_persistent_active(self.h))

    def set_sm_split(self, sms_attention_stream: int = 0):
        _check(lib().ladder_model_set_sm_split(self.h, sms_attention_stream), self.h)

    def set_exchange(self, fn=None, capturable: bool = False):
        """Tensor parallelism with a caller-supplied sum over the ranks: fn(partial_ptr, count, cuda_stream) -> 0
        enqueues the in-place sum of `count` fp32 values at device address `partial_ptr` on `cuda_stream`
        (ladder_model_set_exchange).  None switches it off."""
        if fn is None:
            self._exchange_cb = None
            _check(lib().ladder_model_set_exchange(self.h, None, None, 0), self.h)
            return

        def thunk(_ctx, ptr, count, stream):
            try:
                return int(fn(ptr, count, stream) or 0)
            except Exception:                      # an exception must not cross the C frames
                import traceback
                traceback.print_exc()
                return 1

        cb = EXCHANGE_FN(thunk)
        _check(lib().ladder_model_set_exchange(self.h, C.cast(cb, C.c_void_p), None, int(capturable)), self.h)
        self._exchange_cb = cb                     # keep the thunk alive as long as the model may call it

    def set_tensor_parallel(self, comm: Optional["Comm"]):
        """This model is one rank's slice; partial sums are all-reduced over `comm` (ladder_model_set_tensor_parallel)."""
        _check(lib().ladder_model_set_tensor_parallel(self.h, comm.h if comm is not None else None), self.h)
        self._comm = comm

    def set_tensor_parallel_peer(self, comm: "Comm", peer: "Peer"):
        """Decode-step exchanges over peer memory, the prompt pass over NCCL (ladder_model_set_tensor_parallel_peer)."""
        _check(lib().ladder_model_set_tensor_parallel_peer(self.h, comm.h, peer.h), self.h)
        self._comm, self._peer = comm, peer

    def set_peer(self, peer: Optional["Peer"]):
        """Decode-step exchanges fused into the GEMM epilogues over `peer` (ladder_model_set_peer)."""
        _check(lib().ladder_model_set_peer(self.h, peer.h if peer is not None else None), self.h)
        self._peer = peer

    def set_peer_max_bytes(self, n: int):
        """Largest (world - 1) x batch x d_model x 8 for which a decode step uses the fused exchange (negative: never)."""
        _check(lib().ladder_model_set_peer_max_bytes(self.h, n), self.h)

    def debug_set_peer_hook(self, fn=None):
        """fn(channel, cuda_stream), called after each decode-step output GEMM has been enqueued (tests)."""
        if fn is None:
            _check(lib().ladder_debug_set_peer_hook(self.h, None, None), self.h)
            self._peer_hook = None
            return

        def thunk(_ctx, channel, stream):
            try:
                fn(channel, stream)
            except Exception:
                import traceback
                traceback.print_exc()

        cb = PEER_HOOK_FN(thunk)
        _check(lib().ladder_debug_set_peer_hook(self.h, C.cast(cb, C.c_void_p), None), self.h)
        self._peer_hook = cb

    def set_position(self, length: int):
        _check(lib().ladder_set_position(self.h, length), self.h)

    def device_status(self) -> int:
        """The LADDER_DEV_* bits, read and cleared.  A timeout bit comes back as a value, not as an exception
        (the C call returns LADDER_ERR_TIMEOUT with the word filled in); the steps after it raise."""
        f = C.c_int32(0)
        st = lib().ladder_device_status(self.h, C.byref(f), _stream())
        if st != 6:
            _check(st, self.h)
        return f.value

    def kernel_launches(self) -> int:
        return int(lib().ladder_kernel_launches(self.h))

    @staticmethod
    def _outs(next_tokens=None, final_hidden=None, logits=None, all_hidden=None):
        return ladder_outputs_t(_ptr(next_tokens), _ptr(final_hidden), _ptr(logits), _ptr(all_hidden))

    def prefill(self, cache: KVCache, tokens: torch.Tensor, next_tokens=None, final_hidden=None, logits=None,
                all_hidden=None):
        assert tokens.dtype == torch.int32 and tokens.is_cuda and tokens.dim() == 2
        o = self._outs(next_tokens, final_hidden, logits, all_hidden)
        _check(lib().ladder_prefill(self.h, C.byref(cache.c), _ptr(tokens), tokens.shape[0], tokens.shape[1],
                                    C.byref(o), _stream()), self.h)

    def prefill_ragged(self, cache: KVCache, tokens: torch.Tensor, lens: Sequence[int], next_tokens=None,
                       final_hidden=None, logits=None, all_hidden=None):
        """Prompts of different lengths in one call: tokens [batch, padded length], lens the true lengths."""
        assert tokens.dtype == torch.int32 and tokens.is_cuda and tokens.dim() == 2 and len(lens) == tokens.shape[0]
        o = self._outs(next_tokens, final_hidden, logits, all_hidden)
        h_lens = (C.c_int32 * len(lens))(*[int(v) for v in lens])
        _check(lib().ladder_prefill_ragged(self.h, C.byref(cache.c), _ptr(tokens), h_lens, tokens.shape[0],
                                           tokens.shape[1], C.byref(o), _stream()), self.h)

    @staticmethod
    def _state(pair):
        if pair is None:
            return None
        newest, older = pair
        return C.byref(ladder_stream_state_t(_ptr(newest), _ptr(older)))

    def stage_prefill(self, cache: KVCache, tokens, batch: int, seq_len: int, state_in=None, state_out=None, **outs):
        """Prompt pass of one pipeline stage.  state_in / state_out: (newest, older) fp32 tensors [batch*seq_len, d]
        or None (first stage: tokens; last stage: head outputs as keyword arguments)."""
        o = self._outs(**outs)
        _check(lib().ladder_stage_prefill(self.h, C.byref(cache.c), _ptr(tokens), self._state(state_in), batch, seq_len,
                                          self._state(state_out), C.byref(o), _stream()), self.h)

    def stage_decode_step(self, cache: KVCache, tokens, batch: int, state_in=None, state_out=None, **outs):
        o = self._outs(**outs)
        _check(lib().ladder_stage_decode_step(self.h, C.byref(cache.c), _ptr(tokens), self._state(state_in), batch,
                                              self._state(state_out), C.byref(o), _stream()), self.h)

    def prefill_append(self, cache: KVCache, tokens: torch.Tensor, next_tokens=None, final_hidden=None, logits=None,
                       all_hidden=None):
        """Continues the prompt: tokens [batch, chunk] follow the positions already cached."""
        assert tokens.dtype == torch.int32 and tokens.is_cuda and tokens.dim() == 2
        o = self._outs(next_tokens, final_hidden, logits, all_hidden)
        _check(lib().ladder_prefill_append(self.h, C.byref(cache.c), _ptr(tokens), tokens.shape[0], tokens.shape[1],
                                           C.byref(o), _stream()), self.h)

    def decode_step(self, cache: KVCache, tokens: torch.Tensor, next_tokens=None, final_hidden=None, logits=None):
        assert tokens.dtype == torch.int32 and tokens.is_cuda
        o = self._outs(next_tokens, final_hidden, logits)
        _check(lib().ladder_decode_step(self.h, C.byref(cache.c), _ptr(tokens), tokens.numel(), C.byref(o),
                                        _stream()), self.h)

    def decode_step_host(self, cache: KVCache, h_tokens: torch.Tensor, h_next: torch.Tensor):
        assert not h_tokens.is_cuda and not h_next.is_cuda and h_tokens.dtype == torch.int32
        _check(lib().ladder_decode_step_host(self.h, C.byref(cache.c), h_tokens.data_ptr(), h_tokens.numel(),
                                             h_next.data_ptr(), _stream()), self.h)

    def prefill_host(self, cache: KVCache, h_tokens: torch.Tensor, h_next: torch.Tensor):
        assert not h_tokens.is_cuda and h_tokens.dtype == torch.int32 and h_tokens.dim() == 2
        _check(lib().ladder_prefill_host(self.h, C.byref(cache.c), h_tokens.data_ptr(), h_tokens.shape[0],
                                         h_tokens.shape[1], h_next.data_ptr(), _stream()), self.h)


# ----------------------------------------------------------------------------- single-kernel entry points
def op_smallm_gemm(W: torch.Tensor, act: torch.Tensor, act_mode: int, epi_mode: int, out: torch.Tensor,
                   gain: Optional[torch.Tensor] = None, eps: float = 1e-5, addend: Optional[torch.Tensor] = None):
    N, K = W.shape
    _check(lib().ladder_op_smallm_gemm(_ptr(W), N, K, _ptr(act), act_mode, _ptr(gain), eps, act.shape[0], epi_mode,
                                       _ptr(addend), _ptr(out), _stream()))


def decode_attention_scratch_bytes(batch: int, n_q_heads: int, head_dim: int, max_seq_len: int) -> int:
    return int(lib().ladder_decode_attention_scratch_bytes(batch, n_q_heads, head_dim, max_seq_len))


def op_decode_attention(q, k, v, kv_len, n_q_heads, n_kv_heads, head_dim, max_seq_len, scratch, o):
    _check(lib().ladder_op_decode_attention(_ptr(q), _ptr(k), _ptr(v), _ptr(kv_len), q.shape[0], n_q_heads,
                                            n_kv_heads, head_dim, max_seq_len, _ptr(scratch), _ptr(o), _stream()))


def op_decode_attention_noalloc(q, k, v, kv_len, n_q_heads, n_kv_heads, head_dim, max_seq_len, o):
    """Decode attention whose scratch lives inside the library image: for callers that cannot
    allocate device memory.  Raises LadderError(status 2) when the shape needs more than 8 MiB."""
    _check(lib().ladder_op_decode_attention_noalloc(_ptr(q), _ptr(k), _ptr(v), _ptr(kv_len), q.shape[0], n_q_heads,
                                                    n_kv_heads, head_dim, max_seq_len, _ptr(o), _stream()))


def set_prefill_gemm_impl(impl: int):
    """Test switch (process-wide).  0 = default (tcgen05, binary16 operands for calls of >= 256 tokens, else bf16
    pairs); 2 = tcgen05, one bf16 value per activation; 3 = tcgen05, bf16 hi + lo pairs at every size; 4 = as 0 with
    one CTA per tile everywhere (no CTA pairs)."""
    lib().ladder_set_prefill_gemm_impl(impl)


def set_decode_wide_impl(impl: int):
    """Decode GEMM: 0 = tcgen05 kernel for batch 5..64 (default), 2 = tcgen05 kernel for every batch."""
    lib().ladder_set_decode_wide_impl(impl)


def set_decode_attention_impl(impl: int):
    """Decode attention for batch > 8: 0 = TMA / tcgen05 kernel where there are >= 2048 tiles of 128 keys (default),
    1 = the register-fragment kernel always, 2 = the TMA / tcgen05 kernel always."""
    lib().ladder_set_decode_attention_impl(impl)


def op_prefill_gemm(A, W, epi_mode: int, out, addend=None, A_lo=None, out_lo=None):
    M, K = A.shape
    N = W.shape[0]
    _check(lib().ladder_op_prefill_gemm(_ptr(A), _ptr(A_lo), _ptr(W), M, N, K, epi_mode, _ptr(addend), _ptr(out),
                                        _ptr(out_lo), _stream()))


def op_prefill_gemm_f16(A, W, epi_mode: int, out, addend=None):
    """A binary16 [M, K], W binary16 [N, K]; outputs of modes 1 and 3 are binary16."""
    M, K = A.shape
    N = W.shape[0]
    _check(lib().ladder_op_prefill_gemm_f16(_ptr(A), _ptr(W), M, N, K, epi_mode, _ptr(addend), _ptr(out), _stream()))


def op_convert_bf16_f16(src, dst):
    _check(lib().ladder_op_convert_bf16_f16(_ptr(src), _ptr(dst), src.numel(), _stream()))


def op_prefill_attention(q, k, v, batch, seq_len, n_q_heads, n_kv_heads, head_dim, max_seq_len, o, q_lo=None,
                         o_lo=None, pos0=None, lens=None, out_binary16=False):
    """Prompt-pass attention of one layer.  With pos0 / lens / out_binary16 it goes through the entry point that
    takes a starting position, per-sequence lengths and a binary16 output."""
    if pos0 is None and lens is None and not out_binary16:
        _check(lib().ladder_op_prefill_attention(_ptr(q), _ptr(q_lo), _ptr(k), _ptr(v), batch, seq_len, n_q_heads,
                                                 n_kv_heads, head_dim, max_seq_len, _ptr(o), _ptr(o_lo), _stream()))
        return
    _check(lib().ladder_op_prefill_attention_at(_ptr(q), _ptr(q_lo), _ptr(k), _ptr(v), batch, seq_len, n_q_heads,
                                                n_kv_heads, head_dim, max_seq_len, int(pos0 or 0), _ptr(lens),
                                                1 if out_binary16 else 0, _ptr(o), _ptr(o_lo), _stream()))
