"""Small helpers shared by the tests (no method arithmetic that a test relies on)."""
from __future__ import annotations

import numpy as np

from oracle.ladder_oracle import OracleConfig, OracleWeights


def small_cfg(n_layers=3, d=32, hq=4, hkv=2, dh=8, f=48, v=64, ladder=None, theta=10000.0):
    return OracleConfig(d_model=d, n_layers=n_layers, n_q_heads=hq, n_kv_heads=hkv, head_dim=dh,
                        d_ff=f, vocab_size=v, rms_eps=1e-5, rope_theta=theta, layer_is_ladder=ladder)


def rand_weights(cfg: OracleConfig, seed=0, std=0.2, dtype=np.float64):
    """Random logical weights (larger std than the benchmark's so every path matters)."""
    rng = np.random.default_rng(seed)
    d, F, V = cfg.d_model, cfg.d_ff, cfg.vocab_size
    nq, nkv = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    t = {("tok_embedding", None): rng.normal(0, 1.0, (V, d)).astype(dtype),
         ("final_norm", None): rng.uniform(0.5, 1.5, d).astype(dtype),
         ("lm_head", None): rng.normal(0, std, (V, d)).astype(dtype)}
    for l in range(cfg.n_layers):
        t[("attn_norm", l)] = rng.uniform(0.5, 1.5, d).astype(dtype)
        t[("mlp_norm", l)] = rng.uniform(0.5, 1.5, d).astype(dtype)
        t[("wq", l)] = rng.normal(0, std, (nq, d)).astype(dtype)
        t[("wk", l)] = rng.normal(0, std, (nkv, d)).astype(dtype)
        t[("wv", l)] = rng.normal(0, std, (nkv, d)).astype(dtype)
        t[("wo", l)] = rng.normal(0, std, (d, nq)).astype(dtype)
        t[("w_gate", l)] = rng.normal(0, std, (F, d)).astype(dtype)
        t[("w_up", l)] = rng.normal(0, std, (F, d)).astype(dtype)
        t[("w_down", l)] = rng.normal(0, std, (d, F)).astype(dtype)
    return t


def W(tensors) -> OracleWeights:
    return OracleWeights(dict(tensors))


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max_i |g_i - o_i| / max_i |o_i| over the last axis, maximised over rows."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    num = np.max(np.abs(got - ref), axis=-1)
    den = np.max(np.abs(ref), axis=-1) + 1e-30
    return float(np.max(num / den))
