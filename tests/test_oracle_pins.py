"""Pins for the CPU oracle: every check compares it with something other than itself --
a closed form, a textbook formula written out here, brute force in scalar loops, or an
invariant the paper fixes (Sec. 2 Eq. 1, Sec. 3.1 Eq. 2, Algorithm 1)."""
import math

import numpy as np
import pytest
import torch

from oracle import ladder_oracle as O
from tests.helpers import W, rand_weights, small_cfg

TOK = np.array([[3, 17, 5, 9, 60, 1], [8, 8, 2, 33, 4, 50]])


def _x0(t, tokens):
    return t[("tok_embedding", None)][tokens]


# ---------------------------------------------------------------- elementary operations
def test_rmsnorm_textbook_formula():
    rng = np.random.default_rng(1)
    x = rng.normal(size=(3, 10))
    g = rng.uniform(0.5, 1.5, 10)
    y = O.rmsnorm(x, g, 1e-5)
    for r in range(3):
        ms = sum(float(v) ** 2 for v in x[r]) / 10
        for i in range(10):
            assert abs(y[r, i] - x[r, i] / math.sqrt(ms + 1e-5) * g[i]) < 1e-12
    # scale invariance and unit rms for g = 1, eps -> 0
    y1 = O.rmsnorm(x, np.ones(10), 0.0)
    assert np.allclose(np.sqrt(np.mean(y1 ** 2, -1)), 1.0, atol=1e-12)
    assert np.allclose(O.rmsnorm(7.5 * x, g, 0.0), O.rmsnorm(x, g, 0.0), atol=1e-12)


def test_rope_is_complex_rotation_of_interleaved_pairs():
    rng = np.random.default_rng(2)
    T, H, Dh, theta = 5, 2, 8, 10000.0
    u = rng.normal(size=(T, H, Dh))
    pos = np.array([0, 1, 2, 7, 100])
    out = O.rope(u, pos, theta)
    for t in range(T):
        for h in range(H):
            for j in range(Dh // 2):
                z = complex(u[t, h, 2 * j], u[t, h, 2 * j + 1])
                ang = pos[t] * theta ** (-2.0 * j / Dh)
                zr = z * complex(math.cos(ang), math.sin(ang))
                assert abs(out[t, h, 2 * j] - zr.real) < 1e-12
                assert abs(out[t, h, 2 * j + 1] - zr.imag) < 1e-12
    assert np.array_equal(out[0], u[0])                                # position 0 is the identity
    assert np.allclose(np.linalg.norm(out, axis=-1), np.linalg.norm(u, axis=-1), atol=1e-12)


def test_rope_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(3)
    q = rng.normal(size=(1, 1, 16))
    k = rng.normal(size=(1, 1, 16))
    def score(p, t):
        return float(np.sum(O.rope(q, np.array([p]), 500000.0) * O.rope(k, np.array([t]), 500000.0)))
    assert abs(score(9, 4) - score(9 + 37, 4 + 37)) < 1e-10
    assert abs(score(9, 4) - score(8, 4)) > 1e-6


def test_silu_and_swiglu_scalar_formula():
    rng = np.random.default_rng(4)
    cfg = small_cfg(n_layers=1)
    t = rand_weights(cfg, 4)
    n = rng.normal(size=(1, 2, cfg.d_model))
    out = O.mlp_module(cfg, W(t), 0, n)
    wg, wu, wd = t[("w_gate", 0)], t[("w_up", 0)], t[("w_down", 0)]
    for p in range(2):
        h = []
        for j in range(cfg.d_ff):
            zg = sum(wg[j, i] * n[0, p, i] for i in range(cfg.d_model))
            zu = sum(wu[j, i] * n[0, p, i] for i in range(cfg.d_model))
            h.append(zg / (1.0 + math.exp(-zg)) * zu)
        for i in range(cfg.d_model):
            ref = sum(wd[i, j] * h[j] for j in range(cfg.d_ff))
            assert abs(out[0, p, i] - ref) < 1e-10


def test_bf16_round_matches_library_conversion():
    rng = np.random.default_rng(5)
    a = np.concatenate([rng.normal(size=1000), [0.0, 1.0, -1.0, 1.00390625, 3.0e-5, 65504.0]]).astype(np.float32)
    ref = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(O.bf16_round(a), ref)


# ---------------------------------------------------------------- attention
def _brute_attention(q, k, v, pos0):
    """Scalar loops, explicit K/V replication per query head, explicit mask."""
    T, Hq, Dh = q.shape
    L, Hkv, _ = k.shape
    rep = Hq // Hkv
    k_rep = [[k[t][h // rep] for h in range(Hq)] for t in range(L)]
    v_rep = [[v[t][h // rep] for h in range(Hq)] for t in range(L)]
    out = np.zeros((T, Hq, Dh))
    for p in range(T):
        for h in range(Hq):
            s = []
            for t in range(L):
                if t <= pos0 + p:
                    s.append(sum(q[p, h, i] * k_rep[t][h][i] for i in range(Dh)) / math.sqrt(Dh))
            m = max(s)
            e = [math.exp(v_ - m) for v_ in s]
            z = sum(e)
            for t in range(len(s)):
                for i in range(Dh):
                    out[p, h, i] += e[t] / z * v_rep[t][h][i]
    return out


@pytest.mark.parametrize("hq,hkv,pos0,T", [(4, 2, 0, 5), (4, 4, 0, 4), (6, 1, 3, 2), (2, 2, 6, 1)])
def test_attention_brute_force(hq, hkv, pos0, T):
    rng = np.random.default_rng(6)
    Dh, L = 4, pos0 + T
    q = rng.normal(size=(T, hq, Dh))
    k = rng.normal(size=(L, hkv, Dh))
    v = rng.normal(size=(L, hkv, Dh))
    assert np.allclose(O.causal_attention(q, k, v, pos0), _brute_attention(q, k, v, pos0), atol=1e-12)


def test_softmax_rows_sum_to_one_and_mask_is_exact():
    rng = np.random.default_rng(7)
    q = rng.normal(size=(6, 4, 8)) * 3
    k = rng.normal(size=(6, 2, 8)) * 3
    v = rng.normal(size=(6, 2, 8))
    _, p = O.causal_attention(q, k, v, 0, return_probs=True)
    assert np.all(p >= 0)
    assert np.allclose(p.sum(-1), 1.0, atol=1e-12)
    for a in range(6):
        assert np.all(p[:, a, a + 1:] == 0.0)
        assert np.all(p[:, a, :a + 1] > 0.0)


def test_zero_query_gives_causal_running_mean_of_values():
    cfg = small_cfg(n_layers=1)
    t = rand_weights(cfg, 8)
    t[("wq", 0)] = np.zeros_like(t[("wq", 0)])
    rng = np.random.default_rng(8)
    n = rng.normal(size=(1, 5, cfg.d_model))
    out = O.attention_module(cfg, W(t), 0, n, 0, None)
    v = (n[0] @ t[("wv", 0)].T).reshape(5, cfg.n_kv_heads, cfg.head_dim)
    run = np.cumsum(v, axis=0) / np.arange(1, 6)[:, None, None]
    rep = cfg.n_q_heads // cfg.n_kv_heads
    o = np.repeat(run, rep, axis=1).reshape(5, -1)
    assert np.allclose(out[0], o @ t[("wo", 0)].T, atol=1e-12)


def test_gqa_equals_mha_with_repeated_kv_heads():
    cfg_g = small_cfg(n_layers=2, hq=4, hkv=2)
    cfg_m = small_cfg(n_layers=2, hq=4, hkv=4)
    t = rand_weights(cfg_g, 9)
    tm = dict(t)
    for l in range(2):
        for nm in ("wk", "wv"):
            w = t[(nm, l)].reshape(2, cfg_g.head_dim, -1)
            tm[(nm, l)] = np.repeat(w, 2, axis=0).reshape(4 * cfg_g.head_dim, -1)
    a = O.forward(cfg_g, W(t), TOK)
    b = O.forward(cfg_m, W(tm), TOK)
    assert np.allclose(a.hidden, b.hidden, atol=1e-12)


def test_linear_layers_match_float64_matmul_written_here():
    cfg = small_cfg(n_layers=1, hq=2, hkv=2)
    t = rand_weights(cfg, 10)
    rng = np.random.default_rng(10)
    n = rng.normal(size=(1, 1, cfg.d_model))
    out = O.attention_module(cfg, W(t), 0, n, 0, None)
    # one token at position 0: RoPE is the identity, softmax over one key is 1, so out = Wo Wv n
    v = np.array([sum(t[("wv", 0)][r, i] * n[0, 0, i] for i in range(cfg.d_model))
                  for r in range(cfg.n_kv_heads * cfg.head_dim)])
    ref = np.array([sum(t[("wo", 0)][r, c] * v[c] for c in range(v.size)) for r in range(cfg.d_model)])
    assert np.allclose(out[0, 0], ref, atol=1e-12)


# ---------------------------------------------------------------- routing (Eq. 1, Eq. 2, Algorithm 1)
def _modules(cfg, t):
    """h_m for m = 1..2N acting on a residual value, built from the oracle's module functions."""
    Wt = W(t)
    mods = []
    for l in range(cfg.n_layers):
        mods.append(lambda x, l=l: O.attention_module(
            cfg, Wt, l, O.rmsnorm(x, t[("attn_norm", l)], cfg.rms_eps), 0, None))
        mods.append(lambda x, l=l: O.mlp_module(
            cfg, Wt, l, O.rmsnorm(x, t[("mlp_norm", l)], cfg.rms_eps)))
    return mods


def _algorithm1(cfg, t, x0, masks):
    """Algorithm 1 written out here: a layer routine that carries the stream `residual` and the two module
    outputs that have not been added yet from layer to layer (the all-reduce and its handle are the identity
    on one device).  masks[l] true: ladder layer; false: a standard layer, which first adds what is pending."""
    mods = _modules(cfg, t)
    residual = x0
    attn_out = np.zeros_like(x0)
    mlp_out = np.zeros_like(x0)
    states = []
    for l in range(cfg.n_layers):
        attn, mlp = mods[2 * l], mods[2 * l + 1]
        if masks[l]:
            residual = residual + attn_out
            attn_out = attn(residual)
            residual = residual + mlp_out
            mlp_out = mlp(residual)
        else:
            residual = residual + attn_out + mlp_out
            residual = residual + attn(residual)
            residual = residual + mlp(residual)
            attn_out = np.zeros_like(x0)
            mlp_out = np.zeros_like(x0)
        states.append((residual, attn_out, mlp_out))
    return residual + attn_out + mlp_out, states


@pytest.mark.parametrize("masks", [[1, 1, 1], [0, 1, 1], [1, 0, 1], [1, 1, 0], [0, 0, 0]])
def test_module_chain_equals_algorithm1_written_here(masks):
    cfg = small_cfg(n_layers=3, ladder=masks)
    t = rand_weights(cfg, 11)
    want, _ = _algorithm1(cfg, t, _x0(t, TOK), masks)
    r = O.forward(cfg, W(t), TOK, record=True)
    assert np.allclose(r.x_final, want, atol=1e-11)


def test_all_ladder_chain_reads_two_back():
    cfg = small_cfg(n_layers=3)
    t = rand_weights(cfg, 11)
    mods = _modules(cfg, t)
    xs = [_x0(t, TOK)]
    for m in range(1, 2 * cfg.n_layers + 1):
        xs.append(xs[m - 1] + mods[m - 1](xs[max(m - 2, 0)]))           # Eq. 2
    r = O.forward(cfg, W(t), TOK, record=True)
    assert np.allclose(r.x_final, xs[-1], atol=1e-11)
    for m in range(1, 2 * cfg.n_layers + 1):
        assert np.allclose(r.module_inputs[m - 1], xs[max(m - 2, 0)], atol=1e-11)


def test_parallel_layers_recurrence_written_here():
    """Parallel attention and MLP (Sec. 3.3.1): x_l = x_{l-1} + Attn(n) + MLP(n), n = Norm(x_{l-1}) with one
    norm (the attention gain); the MLP gain must not matter; and the result differs from the standard model."""
    cfg = small_cfg(n_layers=3)
    cfg.layer_mode = ["parallel"] * 3
    t = rand_weights(cfg, 31)
    Wt = W(t)
    x = _x0(t, TOK)
    for l in range(3):
        n = O.rmsnorm(x, t[("attn_norm", l)], cfg.rms_eps)
        x = x + O.attention_module(cfg, Wt, l, n, 0, None) + O.mlp_module(cfg, Wt, l, n)
    r = O.forward(cfg, Wt, TOK)
    assert np.allclose(r.x_final, x, atol=1e-11)
    t2 = dict(t)
    for l in range(3):
        t2[("mlp_norm", l)] = t[("mlp_norm", l)] * 3.0
    assert np.array_equal(O.forward(cfg, W(t2), TOK).x_final, r.x_final)
    std = O.forward(small_cfg(n_layers=3, ladder=[0, 0, 0]), Wt, TOK)
    assert not np.allclose(std.x_final, x, atol=1e-3)


def test_parallel_layer_mixed_with_ladder_and_standard():
    cfg = small_cfg(n_layers=4)
    cfg.layer_mode = ["standard", "parallel", "ladder", "parallel"]
    t = rand_weights(cfg, 32)
    mods = _modules(cfg, t)
    Wt = W(t)
    par_mlp = lambda x, l: O.mlp_module(cfg, Wt, l, O.rmsnorm(x, t[("attn_norm", l)], cfg.rms_eps))
    x0 = _x0(t, TOK)
    x1 = x0 + mods[0](x0)
    x2 = x1 + mods[1](x1)                 # standard layer
    x3 = x2 + mods[2](x2)
    x4 = x3 + par_mlp(x2, 1)              # parallel layer: both read x2
    x5 = x4 + mods[4](x4)                 # ladder attention after a non-ladder layer: complete stream
    x6 = x5 + mods[5](x4)                 # its MLP reads one module back
    x7 = x6 + mods[6](x6)                 # parallel layer after a ladder layer: complete stream
    x8 = x7 + par_mlp(x6, 3)
    assert np.allclose(O.forward(cfg, Wt, TOK).x_final, x8, atol=1e-11)


def test_upper_bound_is_the_standard_model_on_one_device():
    cfg_u = small_cfg(n_layers=3)
    cfg_u.layer_mode = ["upper_bound"] * 3
    cfg_s = small_cfg(n_layers=3, ladder=[0, 0, 0])
    t = rand_weights(cfg_u, 33)
    assert np.array_equal(O.forward(cfg_u, W(t), TOK).hidden, O.forward(cfg_s, W(t), TOK).hidden)


def test_explicit_module_flags_give_the_other_hybrid_boundary_reading():
    """module_stale states the rule module by module: here the first ladder attention after a standard layer
    also reads one module back (x_1, skipping the standard layer's MLP output)."""
    cfg = small_cfg(n_layers=2, ladder=[0, 1])
    cfg.module_stale = [0, 0, 1, 1]
    t = rand_weights(cfg, 34)
    mods = _modules(cfg, t)
    x0 = _x0(t, TOK)
    x1 = x0 + mods[0](x0)
    x2 = x1 + mods[1](x1)
    x3 = x2 + mods[2](x1)
    x4 = x3 + mods[3](x2)
    assert np.allclose(O.forward(cfg, W(t), TOK).x_final, x4, atol=1e-11)
    cfg.module_stale = None
    assert not np.allclose(O.forward(cfg, W(t), TOK).x_final, x4, atol=1e-6)


def _rank_slice(cfg, t, r, world):
    """Weights of the model one tensor-parallel rank holds: its query heads with their kv heads, its MLP columns."""
    dh = cfg.head_dim
    hq, hkv, f = cfg.n_q_heads // world, cfg.n_kv_heads // world, cfg.d_ff // world
    cfg_r = small_cfg(n_layers=cfg.n_layers, d=cfg.d_model, hq=hq, hkv=hkv, dh=dh, f=f, v=cfg.vocab_size,
                      ladder=cfg.layer_is_ladder)
    tr = dict(t)
    for l in range(cfg.n_layers):
        tr[("wq", l)] = t[("wq", l)][r * hq * dh:(r + 1) * hq * dh]
        tr[("wk", l)] = t[("wk", l)][r * hkv * dh:(r + 1) * hkv * dh]
        tr[("wv", l)] = t[("wv", l)][r * hkv * dh:(r + 1) * hkv * dh]
        tr[("wo", l)] = t[("wo", l)][:, r * hq * dh:(r + 1) * hq * dh]
        tr[("w_gate", l)] = t[("w_gate", l)][r * f:(r + 1) * f]
        tr[("w_up", l)] = t[("w_up", l)][r * f:(r + 1) * f]
        tr[("w_down", l)] = t[("w_down", l)][:, r * f:(r + 1) * f]
    return cfg_r, tr


def test_tensor_parallel_partials_sum_to_the_unsplit_module():
    """(XA)B = sum_r (X A_r) B_r (Sec. 2): a rank's partial equals the module of the model built from that rank's
    weight slice (what the one-rank benchmark configuration runs), and the partials sum to the unsplit module."""
    cfg = small_cfg(n_layers=1, hq=4, hkv=2, f=48)
    t = rand_weights(cfg, 35)
    rng = np.random.default_rng(35)
    n = rng.normal(size=(2, 5, cfg.d_model))
    whole_a = O.attention_module(cfg, W(t), 0, n, 0, None)
    whole_m = O.mlp_module(cfg, W(t), 0, n)
    cfg.tp_world = 2
    parts_a, parts_m = [], []
    for r in range(2):
        cfg_r, tr = _rank_slice(cfg, t, r, 2)
        pa = O.attention_module(cfg, W(t), 0, n, 0, None, tp_rank=r)
        pm = O.mlp_module(cfg, W(t), 0, n, tp_rank=r)
        assert np.allclose(pa, O.attention_module(cfg_r, W(tr), 0, n, 0, None), atol=1e-12)
        assert np.allclose(pm, O.mlp_module(cfg_r, W(tr), 0, n), atol=1e-12)
        parts_a.append(pa)
        parts_m.append(pm)
    assert np.allclose(sum(parts_a), whole_a, atol=1e-12) and not np.allclose(parts_a[0], whole_a, atol=1e-3)
    assert np.allclose(sum(parts_m), whole_m, atol=1e-12)
    assert np.allclose(O.attention_module(cfg, W(t), 0, n, 0, None), whole_a, atol=1e-12)
    # a whole model under tensor parallelism computes what the unsplit model computes, ladder or not
    for ladder in (None, [0, 0]):
        c1 = small_cfg(n_layers=2, hq=4, hkv=2, ladder=ladder)
        c2 = small_cfg(n_layers=2, hq=4, hkv=2, ladder=ladder)
        c2.tp_world = 2
        t2 = rand_weights(c1, 36)
        assert np.allclose(O.forward(c1, W(t2), TOK).hidden, O.forward(c2, W(t2), TOK).hidden, atol=1e-11)


def test_recorded_partials_are_the_ranks_partial_sums():
    """The per-rank partial sums a recorded forward pass keeps (what a test hands to a GPU rank in place of its
    absent peers) are the tp_rank partials of the recorded module inputs, and add up to the recorded outputs."""
    cfg = small_cfg(n_layers=2, hq=4, hkv=2, f=48, ladder=[1, 0])
    cfg.tp_world = 2
    t = rand_weights(cfg, 38)
    r = O.forward(cfg, W(t), TOK, record=True)
    assert len(r.module_partials) == 4 and all(len(p) == 2 for p in r.module_partials)
    for m, (parts, out, src) in enumerate(zip(r.module_partials, r.module_outputs, r.module_inputs)):
        assert np.allclose(parts[0] + parts[1], out, atol=1e-12)
        layer, norm = m // 2, ("attn_norm" if m % 2 == 0 else "mlp_norm")
        n = O.rmsnorm(src, W(t).get(norm, layer), cfg.rms_eps)
        for rank in range(2):
            ref = (O.attention_module(cfg, W(t), layer, n, 0, None, tp_rank=rank) if m % 2 == 0
                   else O.mlp_module(cfg, W(t), layer, n, tp_rank=rank))
            assert np.allclose(parts[rank], ref, atol=1e-12)
    assert O.forward(cfg, W(t), TOK).module_partials == []          # nothing is kept unless asked for


@pytest.mark.parametrize("masks", [[1, 1, 1, 1], [0, 0, 1, 1], [1, 0, 1, 0]])
def test_pipeline_stages_chained_equal_the_whole_model(masks):
    """Sec. 5.1: at a stage boundary the stream state is handed on.  Two stages chained give the whole model,
    and the pair handed on is (residual + attn_out, residual + attn_out + mlp_out) of Algorithm 1's three tensors."""
    cfg = small_cfg(n_layers=4, ladder=masks)
    t = rand_weights(cfg, 37)
    x0 = _x0(t, TOK)
    whole = O.run_layers(cfg, W(t), x0, 0, None)
    older, newest = O.run_layers(cfg, W(t), x0, 0, None, n_layers=2, return_state=True)
    rest = O.run_layers(cfg, W(t), newest, 0, None, first_layer=2, older=older)
    assert np.allclose(rest, whole, atol=1e-11)
    _, states = _algorithm1(cfg, t, x0, masks)
    residual, attn_out, mlp_out = states[1]
    assert np.allclose(newest, residual + attn_out + mlp_out, atol=1e-11)
    if masks[1]:
        assert np.allclose(older, residual + attn_out, atol=1e-11)


def test_standard_mask_equals_equation1():
    cfg = small_cfg(n_layers=3, ladder=[0, 0, 0])
    t = rand_weights(cfg, 12)
    mods = _modules(cfg, t)
    x = _x0(t, TOK)
    for h in mods:
        x = x + h(x)                                                     # Eq. 1
    r = O.forward(cfg, W(t), TOK)
    assert np.allclose(r.x_final, x, atol=1e-11)
    lad = O.forward(small_cfg(n_layers=3), W(t), TOK)
    assert not np.allclose(lad.x_final, x, atol=1e-3)                    # the two really differ


def test_hybrid_boundary_reading():
    # layers: standard, ladder, ladder, standard.  Inputs each module must read (x_k = stream after k adds):
    cfg = small_cfg(n_layers=4, ladder=[0, 1, 1, 0])
    t = rand_weights(cfg, 13)
    mods = _modules(cfg, t)
    reads = [0, 1, 2, 2, 3, 4, 6, 7]        # m=3 reads the complete stream, m=4..6 are stale, m=7,8 complete
    xs = [_x0(t, TOK)]
    for m in range(1, 9):
        xs.append(xs[m - 1] + mods[m - 1](xs[reads[m - 1]]))
    r = O.forward(cfg, W(t), TOK, record=True)
    assert np.allclose(r.x_final, xs[-1], atol=1e-11)


def test_single_live_module_ladder_equals_standard_bitwise():
    for dead in ("w_down", "wo"):
        cfg_l = small_cfg(n_layers=1)
        cfg_s = small_cfg(n_layers=1, ladder=[0])
        t = rand_weights(cfg_l, 14)
        t[(dead, 0)] = np.zeros_like(t[(dead, 0)])
        a = O.forward(cfg_l, W(t), TOK)
        b = O.forward(cfg_s, W(t), TOK)
        assert np.array_equal(a.hidden, b.hidden)
        assert np.array_equal(a.logits, b.logits)


def test_only_module_k_live_gives_x0_plus_hk_x0():
    cfg = small_cfg(n_layers=3)
    base = rand_weights(cfg, 15)
    for k in range(1, 7):
        t = dict(base)
        for l in range(3):
            if 2 * l + 1 != k:
                t[("wo", l)] = np.zeros_like(base[("wo", l)])
            if 2 * l + 2 != k:
                t[("w_down", l)] = np.zeros_like(base[("w_down", l)])
        x0 = _x0(t, TOK)
        want = x0 + _modules(cfg, t)[k - 1](x0)
        for ladder in (None, [0, 0, 0]):
            cfg.layer_is_ladder = ladder
            assert np.allclose(O.forward(cfg, W(t), TOK).x_final, want, atol=1e-11)
        cfg.layer_is_ladder = None


def test_telescoping_sum_of_module_outputs():
    for ladder in (None, [0, 0, 0], [0, 1, 1]):
        cfg = small_cfg(n_layers=3, ladder=ladder)
        t = rand_weights(cfg, 16)
        r = O.forward(cfg, W(t), TOK, record=True)
        assert len(r.module_outputs) == 6
        assert np.allclose(r.x_final, _x0(t, TOK) + sum(r.module_outputs), atol=1e-11)


def test_staleness_is_one_module():
    cfg = small_cfg(n_layers=3)
    t = rand_weights(cfg, 17)
    t2 = dict(t)
    t2[("wo", 1)] = rand_weights(cfg, 99)[("wo", 1)]     # module 3 = attention of layer 1
    for ladder, same_next in ((None, True), ([0, 0, 0], False)):
        cfg.layer_is_ladder = ladder
        a = O.forward(cfg, W(t), TOK, record=True).module_inputs
        b = O.forward(cfg, W(t2), TOK, record=True).module_inputs
        assert np.array_equal(a[2], b[2])                  # module 3 itself reads nothing it wrote
        assert np.array_equal(a[3], b[3]) == same_next     # module 4: unchanged only under ladder
        assert not np.array_equal(a[4], b[4])              # module 5 sees it in both
    cfg.layer_is_ladder = None


def test_zeroed_output_projections_closed_form():
    cfg = small_cfg(n_layers=2)
    t = rand_weights(cfg, 18)
    for l in range(2):
        t[("wo", l)] = np.zeros_like(t[("wo", l)])
        t[("w_down", l)] = np.zeros_like(t[("w_down", l)])
    r = O.forward(cfg, W(t), TOK)
    x0 = _x0(t, TOK)
    hid = x0 / np.sqrt((x0 ** 2).mean(-1, keepdims=True) + 1e-5) * t[("final_norm", None)]
    assert np.allclose(r.hidden, hid, atol=1e-12)
    logits = np.einsum("btd,vd->btv", hid, t[("lm_head", None)])
    assert np.allclose(r.logits, logits, atol=1e-11)
    assert np.array_equal(r.next_tokens, logits.argmax(-1))


def test_greedy_lowest_index_on_ties():
    assert O.greedy(np.array([[0.5, 2.0, 2.0, -1.0, 2.0]]))[0] == 1


# ---------------------------------------------------------------- cache, causality, batching
@pytest.mark.parametrize("ladder", [None, [0, 0, 0], [0, 1, 1]])
def test_cached_decode_equals_full_recomputation(ladder):
    cfg = small_cfg(n_layers=3, ladder=ladder)
    t = rand_weights(cfg, 19)
    S, steps = 4, 5
    rng = np.random.default_rng(19)
    seq = rng.integers(0, cfg.vocab_size, size=(2, S + steps))
    cache = O.OracleCache(cfg, 2, S + steps)
    r = O.prefill(cfg, W(t), seq[:, :S], cache)
    full = O.forward(cfg, W(t), seq)
    assert np.allclose(r.hidden[:, 0], full.hidden[:, S - 1], atol=1e-10)
    for j in range(steps):
        r = O.decode_step(cfg, W(t), seq[:, S + j], cache)
        assert cache.seq_len == S + j + 1
        assert np.allclose(r.hidden[:, 0], full.hidden[:, S + j], atol=1e-10)
        assert np.allclose(r.logits[:, 0], full.logits[:, S + j], atol=1e-10)


def test_generate_is_consistent_with_recomputation_and_teacher_forcing():
    cfg = small_cfg(n_layers=2)
    t = rand_weights(cfg, 20)
    prompt = TOK[:, :4]
    toks, hid = O.generate(cfg, W(t), prompt, 5, 16)
    seq = np.concatenate([prompt, toks[:, :-1]], axis=1)
    full = O.forward(cfg, W(t), seq)
    assert np.array_equal(full.next_tokens[:, 3:], toks)
    assert np.allclose(full.hidden[:, 3:], hid, atol=1e-10)
    forced = np.array(toks)
    forced[:, 2] = (forced[:, 2] + 1) % cfg.vocab_size
    toks_f, _ = O.generate(cfg, W(t), prompt, 5, 16, forced=forced)
    assert np.array_equal(toks_f[:, :3], toks[:, :3])      # history identical up to the forced change
    seq_f = np.concatenate([prompt, forced[:, :-1]], axis=1)
    assert np.array_equal(O.forward(cfg, W(t), seq_f).next_tokens[:, 3:], toks_f)


def test_causality_bitwise():
    cfg = small_cfg(n_layers=2)
    t = rand_weights(cfg, 21)
    a = O.forward(cfg, W(t), TOK)
    tok2 = TOK.copy()
    tok2[:, 4] = (tok2[:, 4] + 7) % cfg.vocab_size
    b = O.forward(cfg, W(t), tok2)
    assert np.array_equal(a.hidden[:, :4], b.hidden[:, :4])
    assert not np.allclose(a.hidden[:, 4:], b.hidden[:, 4:])


def test_batch_rows_are_independent():
    cfg = small_cfg(n_layers=2)
    t = rand_weights(cfg, 22)
    both = O.forward(cfg, W(t), TOK)
    for b in range(2):
        one = O.forward(cfg, W(t), TOK[b:b + 1])
        assert np.allclose(both.hidden[b], one.hidden[0], atol=1e-12)


def test_float32_mode_tracks_float64():
    cfg = small_cfg(n_layers=3)
    t = rand_weights(cfg, 23)
    a = O.forward(cfg, W(t), TOK, dtype=np.float64)
    b = O.forward(cfg, W(t), TOK, dtype=np.float32)
    assert b.hidden.dtype == np.float32
    assert np.max(np.abs(a.hidden - b.hidden)) < 1e-4


def test_bf16_kv_switch_rounds_exactly_the_cache():
    cfg = small_cfg(n_layers=2)
    t = rand_weights(cfg, 24)
    exact, rounded = O.OracleCache(cfg, 2, 8), O.OracleCache(cfg, 2, 8)
    a = O.prefill(cfg, W(t), TOK, exact)
    b = O.prefill(cfg, W(t), TOK, rounded, bf16_kv=True)
    # layer 0 sees identical inputs, so its cache is the bf16 rounding of the exact one (library conversion)
    for src, dst in ((exact.k, rounded.k), (exact.v, rounded.v)):
        ref = torch.from_numpy(src[0, :, :6].astype(np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
        assert np.array_equal(dst[0, :, :6], ref)
    assert np.array_equal(O.bf16_round(rounded.k), rounded.k)          # every cached value is a bf16 value
    assert 0 < np.max(np.abs(a.hidden - b.hidden)) < 0.05              # close to, but not, the exact result
    # cached decode still equals recomputation under the switch
    full = O.forward(cfg, W(t), np.concatenate([TOK, TOK[:, :1]], 1), bf16_kv=True)
    step = O.decode_step(cfg, W(t), TOK[:, 0], rounded, bf16_kv=True)
    assert np.allclose(step.hidden[:, 0], full.hidden[:, 6], atol=1e-10)


def test_f16_kv_switch_rounds_to_binary16_as_the_library_conversion_does():
    cfg = small_cfg(n_layers=1)
    t = rand_weights(cfg, 25)
    c = O.OracleCache(cfg, 2, 8)
    e = O.OracleCache(cfg, 2, 8)
    O.prefill(cfg, W(t), TOK, e)
    O.prefill(cfg, W(t), TOK, c, bf16_kv="f16")
    ref = torch.from_numpy(e.k[0, :, :6].astype(np.float32)).to(torch.float16).to(torch.float64).numpy()
    assert np.array_equal(c.k[0, :, :6], ref)
    x = np.array([1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, 70000.0, 1e-8])     # ties to even; overflow; underflow
    assert np.array_equal(O.f16_round(x), np.array([1.0, 1.0 + 2.0 ** -9, np.inf, 0.0]))


# ---------------------------------------------------------------- the paper's own arithmetic (Tab. 2)
def test_table2_reading_latency_reduction_vs_throughput_gain():
    import os
    path = os.path.join(os.path.dirname(__file__), "golden", "table2_improvements.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert len(rows) == 6
    for name, prefill, decode, toks in rows:
        gain = 100.0 * (1.0 / (1.0 - float(decode) / 100.0) - 1.0)
        # tokens/s gain is dominated by the decode latency reduction r: about 1/(1-r) - 1
        assert abs(gain - float(toks)) < 1.0, (name, gain, toks)
