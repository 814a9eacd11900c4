"""CPU oracle for the Ladder-Residual / standard-residual transformer forward.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition the CUDA
library is checked against.  Nothing in the product path may import it; only
the tests, the smoke check and the CPU-baseline leg of the benchmark do.  It
shares no code with the CUDA path and never receives a value computed there.

What it follows
---------------
The model is a chain of 2N modules (attention, MLP, attention, ...) acting on a
residual stream x_0, x_1, ..., x_2N.  Every module adds its output to the newest
stream value; what differs between the architectures is only WHICH stream value
a module reads:
* Standard residual   x_m = x_{m-1} + h_m(x_{m-1})                  (Sec. 2, Eq. 1)
* Ladder residual     x_m = x_{m-1} + h_m(x_{m-2})                  (Sec. 3.1, Eq. 2)
* Parallel attention and MLP (Sec. 3.3.1): both modules of a layer read the
  layer's input through ONE norm, and both outputs are added.
* Communication-free upper bound (Sec. 3.3.1): the standard model with the
  all-reduce deleted; on a single device, where the all-reduce is the
  identity, it IS the standard model (``upper_bound`` is an alias).
``run_layers`` is that chain written once, with a per-module flag "reads one
module back".  Algorithm 1 (a layer routine that carries the two not-yet-added
module outputs from layer to layer, with the asynchronous all-reduce and its
handle being the identity on one device) computes the same thing; the tests
write Algorithm 1 out and pin this oracle to it.
Tensor parallelism (Sec. 2, Eq. 1 with AllReduce): ``tp_world > 1`` splits each
module over ranks by heads / MLP columns and sums the ranks' partial outputs --
the all-reduce -- before the residual add.
"Llama-3's model architecture" (Sec. 3.3.1): pre-norm RMSNorm, rotary position
embedding on interleaved pairs, grouped-query causal attention, SwiGLU MLP,
final RMSNorm, untied LM head, no biases.

Readings taken where the paper is silent (both sides of every parity test use
the same ones):
* initial pending outputs of Algorithm 1 are zero, so modules 1 and 2 both read x_0;
* the two outputs still pending after the last layer are added before the
  final norm (Eq. 2 adds every h_i into the stream);
* hybrid models: the attention module of a ladder layer that follows a standard
  (or parallel) layer reads the complete stream, and the MLP of that layer is
  the first module that reads one module back (in Algorithm 1's terms: a
  standard layer adds whatever is pending and leaves nothing pending) --
  PARITY UNPINNED by the paper for this hybrid boundary rule; ``module_stale``
  states any other rule explicitly, module by module;
* a parallel layer normalises once, with the layer's attention-norm gain; its
  MLP-norm gain is unused -- PARITY UNPINNED by the paper (it names the PaLM
  formulation and prints no equations);
* greedy argmax takes the lowest index among equal maxima.

Arithmetic: every array is ``dtype`` (float64 by default, float32 for the large
workloads); rotary angles, cos and sin are always formed in float64.

Storage precision switches (the definition is both off):
* ``bf16_kv`` rounds K (after rotation) and V where they enter the cache / the
  attention: ``True`` to bf16, ``"f16"`` to IEEE binary16 (the storage type of the
  CUDA library's cache).  A printed diagnostic in the parity tests: it separates
  what the cache's precision costs from everything else.  Assertions use the
  exact oracle.
* ``bf16_storage=True`` additionally rounds normalised activations, q, the
  attention output and the SwiGLU output: a diagnostic that separates bf16
  noise from bugs.

Pins (tests/test_oracle_pins.py): single-module ladder == standard, cached
decode == recomputation, softmax rows, brute-force attention, module chain ==
Algorithm 1 written out in the test, parallel layer == its recurrence written
out, upper bound == standard, tensor-parallel partial sums == the unsplit
module and == a model built from one rank's weight slice, pipeline stages
chained == the whole model, staleness, telescoping sum, single live module,
closed forms
for zeroed projections, RoPE relative-position property, RMSNorm textbook
formula, GQA == MHA with repeated heads, causality, batch independence,
linear layers vs float64 matmul written out in the test.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------- config
@dataclass
class OracleConfig:
    d_model: int
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    d_ff: int
    vocab_size: int
    rms_eps: float = 1e-5
    rope_theta: float = 10000.0
    layer_is_ladder: Optional[Sequence[bool]] = None  # None = every layer ladder
    # Per-layer architecture, overriding layer_is_ladder when given: "standard" (Eq. 1), "ladder" (Eq. 2),
    # "parallel" (Sec. 3.3.1, parallel attention and MLP), "upper_bound" (Sec. 3.3.1: standard without
    # communication = standard on one device).
    layer_mode: Optional[Sequence[str]] = None
    # Explicit per-module rule, overriding what the layer modes imply: entry m-1 is True when module m
    # (1-based; odd = attention, even = MLP) reads x_{m-2} instead of x_{m-1}.
    module_stale: Optional[Sequence[bool]] = None
    tp_world: int = 1     # tensor-parallel ranks the modules are split over (partials summed = all-reduce)

    def ladder(self, layer: int) -> bool:
        return self.mode(layer) == "ladder"

    def mode(self, layer: int) -> str:
        if self.layer_mode is not None:
            m = self.layer_mode[layer]
            return "standard" if m == "upper_bound" else m
        if self.layer_is_ladder is None:
            return "ladder"
        return "ladder" if self.layer_is_ladder[layer] else "standard"


@dataclass
class ModuleSpec:
    """Module m of the chain: what it is, and which stream value it reads."""
    kind: str            # "attention" | "mlp"
    layer: int
    stale: bool          # True: reads x_{m-2} (Eq. 2); False: reads x_{m-1} (Eq. 1)
    norm: str            # name of the RMSNorm gain applied to its input


def module_chain(cfg: OracleConfig) -> List[ModuleSpec]:
    """The 2N modules in order, each with the stream value it reads.

    standard layer : both modules read the newest value (Eq. 1).
    ladder layer   : both modules read one module back (Eq. 2), except an attention module that directly
                     follows a non-ladder layer, which reads the newest value (hybrid boundary reading).
    parallel layer : attention reads the newest value x_{m-1}; the MLP reads that same x_{m-1} -- one module
                     back from where it stands -- through the same (attention) norm, so that
                     x_{m+1} = x_{m-1} + Attn(n) + MLP(n) with n = Norm(x_{m-1}).
    """
    chain: List[ModuleSpec] = []
    for l in range(cfg.n_layers):
        mode = cfg.mode(l)
        if mode == "standard":
            flags, mlp_norm = (False, False), "mlp_norm"
        elif mode == "ladder":
            after_ladder = l > 0 and cfg.mode(l - 1) == "ladder"
            flags, mlp_norm = (after_ladder or l == 0, True), "mlp_norm"
        elif mode == "parallel":
            flags, mlp_norm = (False, True), "attn_norm"
        else:
            raise ValueError(mode)
        chain.append(ModuleSpec("attention", l, flags[0], "attn_norm"))
        chain.append(ModuleSpec("mlp", l, flags[1], mlp_norm))
    if cfg.module_stale is not None:
        assert len(cfg.module_stale) == len(chain)
        for spec, st in zip(chain, cfg.module_stale):
            spec.stale = bool(st)
    return chain


class OracleWeights:
    """Logical (unpacked) weights.  ``get(name, layer)`` returns a float array.

    names: tok_embedding [V,d], final_norm [d], lm_head [V,d] (layer=None) and per
    layer attn_norm [d], wq [Hq*Dh,d], wk [Hkv*Dh,d], wv [Hkv*Dh,d], wo [d,Hq*Dh],
    mlp_norm [d], w_gate [F,d], w_up [F,d], w_down [d,F].  A provider callback lets
    a caller stream one layer at a time for models larger than host memory.
    """

    def __init__(self, tensors: Optional[Dict] = None,
                 provider: Optional[Callable[[str, Optional[int]], np.ndarray]] = None):
        self._t = tensors or {}
        self._p = provider

    def get(self, name: str, layer: Optional[int] = None) -> np.ndarray:
        key = (name, layer)
        if key in self._t:
            return self._t[key]
        if self._p is None:
            raise KeyError(key)
        return self._p(name, layer)


# --------------------------------------------------------------------------- helpers
def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to bfloat16 precision, returned in a's dtype."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(a.dtype)


def f16_round(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even to IEEE binary16 precision (numpy's own conversion), returned in a's dtype."""
    return a.astype(np.float16).astype(a.dtype)


def _store(a: np.ndarray, bf16_storage: bool) -> np.ndarray:
    return bf16_round(a) if bf16_storage else a


def _store_kv(a: np.ndarray, mode) -> np.ndarray:
    """Cache storage precision: False = exact, True = bf16, "f16" = binary16."""
    if mode == "f16":
        return f16_round(a)
    return bf16_round(a) if mode else a


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """y_i = x_i / sqrt(mean_j x_j^2 + eps) * g_i over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + x.dtype.type(eps)) * g.astype(x.dtype, copy=False)


def rope_angles(positions: np.ndarray, head_dim: int, theta: float):
    """cos/sin [T, Dh/2] in float64: angle = p * theta^(-2j/Dh)."""
    j = np.arange(head_dim // 2, dtype=np.float64)
    inv_freq = np.float64(theta) ** (-2.0 * j / head_dim)
    ang = positions.astype(np.float64)[:, None] * inv_freq[None, :]
    return np.cos(ang), np.sin(ang)


def rope(u: np.ndarray, positions: np.ndarray, theta: float) -> np.ndarray:
    """Rotate interleaved pairs (u_{2j}, u_{2j+1}) of u[..., T, H, Dh] by position."""
    dh = u.shape[-1]
    cos, sin = rope_angles(positions, dh, theta)          # [T, Dh/2]
    cos = cos[:, None, :].astype(u.dtype)
    sin = sin[:, None, :].astype(u.dtype)
    ue, uo = u[..., 0::2], u[..., 1::2]
    out = np.empty_like(u)
    out[..., 0::2] = ue * cos - uo * sin
    out[..., 1::2] = ue * sin + uo * cos
    return out


def softmax_rows(s: np.ndarray) -> np.ndarray:
    """Softmax over the last axis with max subtraction; -inf entries give exactly 0."""
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def causal_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, q_pos0: int,
                     return_probs: bool = False):
    """Grouped-query causal attention for one sequence.

    q [T, Hq, Dh] holds queries at absolute positions q_pos0 .. q_pos0+T-1;
    k, v [L, Hkv, Dh] hold keys/values at absolute positions 0 .. L-1.
    Query head h uses kv head h // (Hq // Hkv).  Query at position p attends to
    keys t <= p.  Returns o [T, Hq, Dh] (and the probabilities [Hq, T, L]).
    """
    T, Hq, Dh = q.shape
    L, Hkv, _ = k.shape
    group = Hq // Hkv
    scale = q.dtype.type(1.0 / np.sqrt(Dh))
    o = np.empty_like(q)
    probs = np.empty((Hq, T, L), dtype=q.dtype) if return_probs else None
    p_idx = q_pos0 + np.arange(T)[:, None]
    t_idx = np.arange(L)[None, :]
    masked = t_idx > p_idx                                   # [T, L]
    for h in range(Hq):
        kh = h // group
        s = (q[:, h, :] @ k[:, kh, :].T) * scale             # [T, L]
        s = np.where(masked, -np.inf, s)
        pr = softmax_rows(s)
        o[:, h, :] = pr @ v[:, kh, :]
        if return_probs:
            probs[h] = pr
    return (o, probs) if return_probs else o


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


# --------------------------------------------------------------------------- cache
class OracleCache:
    """K (post-RoPE) and V for every layer: [n_layers][B][max_seq][Hkv][Dh]."""

    def __init__(self, cfg: OracleConfig, batch: int, max_seq_len: int, dtype=np.float64):
        shp = (cfg.n_layers, batch, max_seq_len, cfg.n_kv_heads, cfg.head_dim)
        self.k = np.zeros(shp, dtype=dtype)
        self.v = np.zeros(shp, dtype=dtype)
        self.seq_len = 0
        self.max_seq_len = max_seq_len


# --------------------------------------------------------------------------- modules
def _tp_slices(width: int, world: int) -> List[slice]:
    """Contiguous equal slices of an inner dimension, one per tensor-parallel rank."""
    assert width % world == 0
    step = width // world
    return [slice(r * step, (r + 1) * step) for r in range(world)]


def attention_module(cfg: OracleConfig, W: OracleWeights, layer: int, n: np.ndarray,
                     pos0: int, cache: Optional[OracleCache], bf16_storage: bool = False,
                     bf16_kv: bool = False, tp_rank: Optional[int] = None, parts_out: Optional[list] = None):
    """h(n) for the attention module of ``layer``.

    n [B, T, d] is the normalised input at absolute positions pos0..pos0+T-1.
    With a cache, the new K/V rows are appended at those positions first and
    attention then runs over positions 0..pos0+T-1 (append, then attend).
    With ``tp_rank`` the result is that rank's partial sum x* (before the all-reduce) only.
    ``parts_out`` (a list) receives every rank's partial sum, for tests that play one rank against the others.
    """
    B, T, d = n.shape
    Hq, Hkv, Dh = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
    dt = n.dtype
    wq = W.get("wq", layer).astype(dt, copy=False)
    wk = W.get("wk", layer).astype(dt, copy=False)
    wv = W.get("wv", layer).astype(dt, copy=False)
    wo = W.get("wo", layer).astype(dt, copy=False)
    positions = pos0 + np.arange(T)
    q = (n @ wq.T).reshape(B, T, Hq, Dh)
    k = (n @ wk.T).reshape(B, T, Hkv, Dh)
    v = (n @ wv.T).reshape(B, T, Hkv, Dh)
    q = _store(rope(q, positions, cfg.rope_theta), bf16_storage)
    k = _store_kv(rope(k, positions, cfg.rope_theta), bf16_storage or bf16_kv)
    v = _store_kv(v, bf16_storage or bf16_kv)
    o = np.empty((B, T, Hq, Dh), dtype=dt)
    for b in range(B):
        if cache is not None:
            cache.k[layer, b, pos0:pos0 + T] = k[b]
            cache.v[layer, b, pos0:pos0 + T] = v[b]
            kk = cache.k[layer, b, :pos0 + T].astype(dt, copy=False)
            vv = cache.v[layer, b, :pos0 + T].astype(dt, copy=False)
        else:
            assert pos0 == 0
            kk, vv = k[b], v[b]
        o[b] = causal_attention(q[b], kk, vv, pos0)
    o = _store(o.reshape(B, T, Hq * Dh), bf16_storage)
    # Output projection.  Under tensor parallelism rank r owns the query heads [r Hq/P, (r+1) Hq/P) (and their
    # kv heads), so everything up to here is rank-local; it multiplies its heads' slice of o with the matching
    # columns of W_o, and the partial products are summed over the ranks (the all-reduce of Sec. 2, Eq. 1).
    parts = [o[..., c] @ wo[:, c].T for c in _tp_slices(Hq * Dh, cfg.tp_world)]
    if parts_out is not None:
        parts_out.extend(parts)
    if tp_rank is not None:
        return parts[tp_rank]
    return parts[0] if len(parts) == 1 else np.sum(parts, axis=0)


def mlp_module(cfg: OracleConfig, W: OracleWeights, layer: int, n: np.ndarray,
               bf16_storage: bool = False, tp_rank: Optional[int] = None, parts_out: Optional[list] = None):
    """h(n) = W_down ( silu(W_gate n) * (W_up n) ).

    Under tensor parallelism rank r owns the hidden columns [r F/P, (r+1) F/P): W_gate and W_up split by
    output, W_down by input, partial products summed over the ranks (Sec. 2).  ``tp_rank``: that rank's partial."""
    dt = n.dtype
    wg = W.get("w_gate", layer).astype(dt, copy=False)
    wu = W.get("w_up", layer).astype(dt, copy=False)
    wd = W.get("w_down", layer).astype(dt, copy=False)
    h = _store(silu(n @ wg.T) * (n @ wu.T), bf16_storage)
    parts = [h[..., c] @ wd[:, c].T for c in _tp_slices(cfg.d_ff, cfg.tp_world)]
    if parts_out is not None:
        parts_out.extend(parts)
    if tp_rank is not None:
        return parts[tp_rank]
    return parts[0] if len(parts) == 1 else np.sum(parts, axis=0)


# --------------------------------------------------------------------------- forward
@dataclass
class ForwardResult:
    x_final: np.ndarray                 # [B, T, d]   residual stream after the last add
    hidden: np.ndarray                  # [B, T, d]   after the final RMSNorm
    logits: Optional[np.ndarray]        # [B, T', V]  (T' = T, or 1 when last_only)
    next_tokens: Optional[np.ndarray]   # [B, T']
    module_inputs: List[np.ndarray] = field(default_factory=list)   # residual each module read
    module_outputs: List[np.ndarray] = field(default_factory=list)  # h_m(.)
    module_partials: List[List[np.ndarray]] = field(default_factory=list)  # per module: every rank's partial sum


def greedy(logits: np.ndarray) -> np.ndarray:
    """argmax over the last axis; numpy returns the first (lowest) index on ties."""
    return np.argmax(logits, axis=-1).astype(np.int64)


def run_layers(cfg: OracleConfig, W: OracleWeights, x: np.ndarray, pos0: int,
               cache: Optional[OracleCache], bf16_storage: bool = False,
               record: Optional[ForwardResult] = None, n_layers: Optional[int] = None,
               bf16_kv: bool = False, first_layer: int = 0, older: Optional[np.ndarray] = None,
               return_state: bool = False):
    """The module chain x_m = x_{m-1} + h_m(x_{m-1} or x_{m-2}) (Eq. 1 / Eq. 2).  x [B,T,d] is x_0.

    Only the last two stream values are kept.  Module 1 has no x_{-1}: it reads x_0 whatever its flag.

    Pipeline stages (Sec. 5.1): a stage runs layers first_layer .. n_layers-1 starting from the stream state
    (older, x) = (x_{m-2}, x_{m-1}) it was handed and, with ``return_state``, hands on the same pair.  In
    Algorithm 1's variables the pair is (residual + attn_out, residual + attn_out + mlp_out): the three
    tensors the paper forwards carry exactly these two sums.
    """
    chain = module_chain(cfg)
    last = cfg.n_layers if n_layers is None else n_layers
    chain = chain[2 * first_layer:2 * last]
    newest = x                              # x_{m-1}; ``older`` is x_{m-2} (None before module 1)
    for spec in chain:
        src = older if (spec.stale and older is not None) else newest
        n = _store(rmsnorm(src, W.get(spec.norm, spec.layer), cfg.rms_eps), bf16_storage)
        parts = [] if record is not None else None
        if spec.kind == "attention":
            out = attention_module(cfg, W, spec.layer, n, pos0, cache, bf16_storage, bf16_kv, parts_out=parts)
        else:
            out = mlp_module(cfg, W, spec.layer, n, bf16_storage, parts_out=parts)
        if record is not None:
            record.module_inputs.append(src.copy())
            record.module_outputs.append(out.copy())
            record.module_partials.append(parts)
        older, newest = newest, newest + out
    return (older, newest) if return_state else newest


def embed(W: OracleWeights, tokens: np.ndarray, dtype) -> np.ndarray:
    E = W.get("tok_embedding")
    return E[np.asarray(tokens, dtype=np.int64)].astype(dtype)


def head(cfg: OracleConfig, W: OracleWeights, x: np.ndarray, bf16_storage: bool = False):
    hidden = rmsnorm(x, W.get("final_norm"), cfg.rms_eps)
    logits = _store(hidden, bf16_storage) @ W.get("lm_head").astype(x.dtype, copy=False).T
    return hidden, logits


def forward(cfg: OracleConfig, W: OracleWeights, tokens: np.ndarray, dtype=np.float64,
            cache: Optional[OracleCache] = None, pos0: int = 0, last_only: bool = False,
            bf16_storage: bool = False, record: bool = False,
            with_logits: bool = True, n_layers: Optional[int] = None,
            bf16_kv: bool = False) -> ForwardResult:
    """Full forward over tokens [B, T] at positions pos0..pos0+T-1.

    Without a cache pos0 must be 0 and the whole sequence is recomputed.  With a
    cache the new rows are appended and ``cache.seq_len`` advances by T.
    """
    tokens = np.asarray(tokens)
    res = ForwardResult(None, None, None, None)
    x = embed(W, tokens, dtype)
    x = run_layers(cfg, W, x, pos0, cache, bf16_storage, res if record else None, n_layers, bf16_kv)
    if cache is not None:
        assert cache.seq_len == pos0
        cache.seq_len = pos0 + tokens.shape[1]
    res.x_final = x
    xs = x[:, -1:, :] if last_only else x
    if with_logits:
        hidden, logits = head(cfg, W, xs, bf16_storage)
        res.logits = logits
        res.next_tokens = greedy(logits)
    else:
        hidden = rmsnorm(xs, W.get("final_norm"), cfg.rms_eps)
    res.hidden = hidden
    return res


def prefill(cfg, W, tokens, cache: OracleCache, dtype=np.float64, bf16_storage=False,
            n_layers=None, bf16_kv=False) -> ForwardResult:
    """Prompt pass: fills cache rows 0..S-1, returns hidden/logits at position S-1."""
    assert cache.seq_len == 0
    return forward(cfg, W, tokens, dtype, cache, 0, last_only=True,
                   bf16_storage=bf16_storage, n_layers=n_layers, bf16_kv=bf16_kv)


def decode_step(cfg, W, tokens, cache: OracleCache, dtype=np.float64, bf16_storage=False,
                n_layers=None, bf16_kv=False) -> ForwardResult:
    """One token per sequence at position cache.seq_len (append, then attend)."""
    tokens = np.asarray(tokens).reshape(-1, 1)
    return forward(cfg, W, tokens, dtype, cache, cache.seq_len, last_only=True,
                   bf16_storage=bf16_storage, n_layers=n_layers, bf16_kv=bf16_kv)


def generate(cfg, W, prompt: np.ndarray, n_steps: int, max_seq_len: int, dtype=np.float64,
             forced: Optional[np.ndarray] = None, bf16_storage=False, bf16_kv=False,
             return_logits: bool = False):
    """prefill + n_steps decode steps.

    Returns (tokens [B, n_steps+1], hiddens [B, n_steps+1, d]): entry 0 comes from
    the prefill (token at position S), entry j+1 from decode step j.  With
    ``forced`` [B, n_steps+1] the fed-back tokens are taken from it instead of the
    oracle's own argmax (teacher forcing), while the returned tokens stay the
    oracle's own choices.  ``return_logits`` adds the logits [B, n_steps+1, V].
    """
    prompt = np.asarray(prompt)
    B, S = prompt.shape
    cache = OracleCache(cfg, B, max_seq_len, dtype)
    r = prefill(cfg, W, prompt, cache, dtype, bf16_storage, bf16_kv=bf16_kv)
    toks = [r.next_tokens[:, 0]]
    hids = [r.hidden[:, 0]]
    logs = [r.logits[:, 0]]
    for j in range(n_steps):
        feed = toks[-1] if forced is None else np.asarray(forced)[:, j]
        r = decode_step(cfg, W, feed, cache, dtype, bf16_storage, bf16_kv=bf16_kv)
        toks.append(r.next_tokens[:, 0])
        hids.append(r.hidden[:, 0])
        logs.append(r.logits[:, 0])
    if return_logits:
        return np.stack(toks, axis=1), np.stack(hids, axis=1), np.stack(logs, axis=1)
    return np.stack(toks, axis=1), np.stack(hids, axis=1)
