"""Seeded synthetic inputs (model shapes, weights, tokens) shared by tests and bench.

This module only *generates and re-arranges data*.  It contains none of the
method's arithmetic: no norm, no projection, no attention, no residual rule.
Weights are produced once, directly in the layout the C library consumes
(bf16, packed QKV rows, interleaved gate/up rows); the CPU checker receives the
very same bytes through :func:`logical_provider`, which only slices and widens.

Workloads stand in for the Llama-shaped models the paper benchmarks (Sec. 3.3.1:
prompt 1024, 512 generated tokens, batch 1..64): same shapes, N(0, 0.02) weights
rounded to bf16, unit RMSNorm gains, i.i.d. uniform token ids.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional

import numpy as np
import torch


@dataclass(frozen=True)
class ModelShape:
    name: str
    d_model: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab_size: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    layer_is_ladder: Optional[tuple] = None     # None = all ladder
    # workload attached to the shape
    batch: int = 1
    prompt_len: int = 16
    decode_steps: int = 16
    seed: int = 0
    # Per-layer architecture ("standard" | "ladder" | "parallel" | "upper_bound"), overriding layer_is_ladder,
    # and an explicit per-module rule (2 * n_layers flags: module reads one module back); see include/ladder.h.
    layer_mode: Optional[tuple] = None
    module_stale: Optional[tuple] = None

    @property
    def qkv_rows(self) -> int:
        return (self.n_q_heads + 2 * self.n_kv_heads) * self.head_dim

    @property
    def max_seq_len(self) -> int:
        return self.prompt_len + self.decode_steps

    def ladder_mask(self) -> List[int]:
        if self.layer_is_ladder is None:
            return [1] * self.n_layers
        return [int(bool(v)) for v in self.layer_is_ladder]

    def with_layers(self, n: int) -> "ModelShape":
        mask = None if self.layer_is_ladder is None else tuple(self.layer_is_ladder[:n])
        modes = None if self.layer_mode is None else tuple(self.layer_mode[:n])
        flags = None if self.module_stale is None else tuple(self.module_stale[:2 * n])
        return replace(self, n_layers=n, layer_is_ladder=mask, layer_mode=modes, module_stale=flags)

    def as_standard(self) -> "ModelShape":
        return replace(self, layer_is_ladder=tuple([0] * self.n_layers), layer_mode=None, module_stale=None)

    def as_mode(self, mode: str) -> "ModelShape":
        """Every layer in one architecture: "standard", "ladder", "parallel" or "upper_bound"."""
        return replace(self, layer_is_ladder=None, layer_mode=tuple([mode] * self.n_layers), module_stale=None)

    def param_count(self) -> int:
        d, F = self.d_model, self.d_ff
        per_layer = self.qkv_rows * d + d * self.n_q_heads * self.head_dim + 3 * F * d + 2 * d
        return self.n_layers * per_layer + 2 * self.vocab_size * d + d

    def layer_weight_bytes(self) -> int:
        d, F = self.d_model, self.d_ff
        return 2 * (self.qkv_rows * d + d * self.n_q_heads * self.head_dim + 3 * F * d + 2 * d)

    def kv_bytes_per_token(self) -> int:
        """Bytes of K plus V one sequence holds per cached position, all layers."""
        return 2 * 2 * self.n_layers * self.n_kv_heads * self.head_dim

    def decode_step_bytes(self, kv_len: float, batch: Optional[int] = None) -> float:
        """Algorithmic bytes one decode step must read: every layer weight once,
        the LM head once, the final norm, the live KV prefix, B embedding rows."""
        b = self.batch if batch is None else batch
        d = self.d_model
        return (self.n_layers * self.layer_weight_bytes() + 2 * self.vocab_size * d + 2 * d
                + b * kv_len * self.kv_bytes_per_token() + b * d * 2)


SHAPES: Dict[str, ModelShape] = {
    # configs of the benchmark description, in order
    "tiny": ModelShape("tiny", 256, 4, 4, 4, 64, 688, 1024, 1e-5, 10000.0, None, 1, 16, 16, 0),
    "1p2b": ModelShape("1p2b", 2048, 24, 16, 16, 128, 5504, 32000, 1e-5, 10000.0, None, 1, 512, 128, 1),
    "8b_hybrid": ModelShape("8b_hybrid", 4096, 32, 32, 8, 128, 14336, 128256, 1e-5, 500000.0,
                            tuple([0] * 16 + [1] * 16), 4, 1024, 256, 2),
    "70b": ModelShape("70b", 8192, 80, 64, 8, 128, 28672, 128256, 1e-5, 500000.0, None, 4, 1024, 512, 3),
    # one tensor-parallel rank's slice of the 70B shape at world size 8 (vocab slice 128256/8)
    "tp_slice": ModelShape("tp_slice", 8192, 80, 8, 1, 128, 3584, 16032, 1e-5, 500000.0, None, 4, 2048, 8, 4),
}

_TENSOR_IDS = {"tok_embedding": 1, "final_norm": 2, "lm_head": 3, "attn_norm": 4, "w_qkv": 5,
               "w_o": 6, "mlp_norm": 7, "w_gate_up": 8, "w_down": 9}


def _gen(device, seed: int, name: str, layer: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + _TENSOR_IDS[name] * 100003 + (layer + 1) * 7919) & 0x7FFFFFFFFFFF)
    return g


def _normal(shape, device, seed, name, layer, std) -> torch.Tensor:
    t = torch.empty(shape, dtype=torch.bfloat16, device=device)
    g = _gen(device, seed, name, layer)
    flat = t.view(-1)
    step = 1 << 27                               # bounded temporaries for the 70B tensors
    for s in range(0, flat.numel(), step):
        flat[s:s + step].normal_(0.0, std, generator=g)
    return t


def _gain(d, device, seed, name, layer, gains: str) -> torch.Tensor:
    if gains == "ones":
        return torch.ones(d, dtype=torch.bfloat16, device=device)
    g = _gen(device, seed, name, layer)           # U(0.5, 1.5): a dropped gain cannot hide
    return (torch.rand(d, generator=g, device=device) + 0.5).to(torch.bfloat16)


@dataclass
class AbiWeights:
    """bf16 tensors in the library's layout (see include/ladder.h)."""
    shape: ModelShape
    tok_embedding: torch.Tensor                   # [V, d]
    final_norm: torch.Tensor                      # [d]
    lm_head: torch.Tensor                         # [V, d]
    attn_norm: List[torch.Tensor] = field(default_factory=list)    # [d]
    w_qkv: List[torch.Tensor] = field(default_factory=list)        # [(Hq+2Hkv)Dh, d]
    w_o: List[torch.Tensor] = field(default_factory=list)          # [d, Hq*Dh]
    mlp_norm: List[torch.Tensor] = field(default_factory=list)     # [d]
    w_gate_up: List[torch.Tensor] = field(default_factory=list)    # [2F, d], row 2j gate_j, 2j+1 up_j
    w_down: List[torch.Tensor] = field(default_factory=list)       # [d, F]

    def nbytes(self) -> int:
        n = self.tok_embedding.numel() + self.final_norm.numel() + self.lm_head.numel()
        for lst in (self.attn_norm, self.w_qkv, self.w_o, self.mlp_norm, self.w_gate_up, self.w_down):
            n += sum(t.numel() for t in lst)
        return 2 * n


def make_weights(shape: ModelShape, device="cpu", std: float = 0.02, gains: str = "ones",
                 seed: Optional[int] = None) -> AbiWeights:
    """N(0, std) bf16 weights in ABI layout; each tensor has its own seed, so a
    model truncated to its first n layers has the same leading layers."""
    seed = shape.seed if seed is None else seed
    d, V, F = shape.d_model, shape.vocab_size, shape.d_ff
    w = AbiWeights(shape,
                   _normal((V, d), device, seed, "tok_embedding", -1, std),
                   _gain(d, device, seed, "final_norm", -1, gains),
                   _normal((V, d), device, seed, "lm_head", -1, std))
    for l in range(shape.n_layers):
        w.attn_norm.append(_gain(d, device, seed, "attn_norm", l, gains))
        w.w_qkv.append(_normal((shape.qkv_rows, d), device, seed, "w_qkv", l, std))
        w.w_o.append(_normal((d, shape.n_q_heads * shape.head_dim), device, seed, "w_o", l, std))
        w.mlp_norm.append(_gain(d, device, seed, "mlp_norm", l, gains))
        w.w_gate_up.append(_normal((2 * F, d), device, seed, "w_gate_up", l, std))
        w.w_down.append(_normal((d, F), device, seed, "w_down", l, std))
    return w


def make_tokens(shape: ModelShape, batch: Optional[int] = None, length: Optional[int] = None,
                seed: Optional[int] = None) -> np.ndarray:
    """i.i.d. uniform token ids [batch, length] (int32), independent per sequence."""
    b = shape.batch if batch is None else batch
    n = shape.prompt_len if length is None else length
    rng = np.random.default_rng(1000 + (shape.seed if seed is None else seed))
    return rng.integers(0, shape.vocab_size, size=(b, n), dtype=np.int64).astype(np.int32)


def _np(t: torch.Tensor, dtype) -> np.ndarray:
    return t.detach().to(torch.float32).cpu().numpy().astype(dtype, copy=False)


def logical_provider(w: AbiWeights, dtype=np.float32, keep: bool = True):
    """Callable (name, layer) -> ndarray giving the *logical* tensors
    (wq, wk, wv, wo, w_gate, w_up, w_down, norms, embedding, head) as slices of the
    packed bf16 data widened to ``dtype``.  Pure indexing and widening; tensors
    that live on a GPU are downloaded one at a time.  With ``keep`` the widened
    copies are remembered (host memory = model size in ``dtype``); without it
    every request converts again, which lets models larger than host memory stream."""
    s = w.shape
    nq = s.n_q_heads * s.head_dim
    nkv = s.n_kv_heads * s.head_dim
    memo: Dict = {}

    def get(name: str, layer: Optional[int] = None) -> np.ndarray:
        if not keep:
            return fetch(name, layer)
        key = (name, layer)
        if key not in memo:
            memo[key] = fetch(name, layer)
        return memo[key]

    def fetch(name: str, layer: Optional[int] = None) -> np.ndarray:
        if name == "tok_embedding":
            return _np(w.tok_embedding, dtype)
        if name == "final_norm":
            return _np(w.final_norm, dtype)
        if name == "lm_head":
            return _np(w.lm_head, dtype)
        if name == "attn_norm":
            return _np(w.attn_norm[layer], dtype)
        if name == "mlp_norm":
            return _np(w.mlp_norm[layer], dtype)
        if name == "wq":
            return _np(w.w_qkv[layer][:nq], dtype)
        if name == "wk":
            return _np(w.w_qkv[layer][nq:nq + nkv], dtype)
        if name == "wv":
            return _np(w.w_qkv[layer][nq + nkv:], dtype)
        if name == "wo":
            return _np(w.w_o[layer], dtype)
        if name == "w_gate":
            return _np(w.w_gate_up[layer][0::2], dtype)
        if name == "w_up":
            return _np(w.w_gate_up[layer][1::2], dtype)
        if name == "w_down":
            return _np(w.w_down[layer], dtype)
        raise KeyError(name)

    return get
