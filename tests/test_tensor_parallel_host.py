"""Tensor parallelism, host side (no GPU): the rank slices of the library's weight layout against the oracle's
partial sums (Sec. 2: (XA)B = sum_r (X A_r) B_r), alone and summed over two gloo ranks."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import ladder_oracle as O                                        # noqa: E402
from paper_2501_06589_b200 import synth                                      # noqa: E402
from paper_2501_06589_b200 import tensor_parallel as TP                      # noqa: E402

SHAPE = synth.ModelShape("tiny_tp", 64, 2, 8, 2, 16, 96, 128, 1e-5, 10000.0, None, 2, 8, 4, 7)


def _cfg(s, world=1):
    c = O.OracleConfig(s.d_model, s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.vocab_size,
                       s.rms_eps, s.rope_theta, None)
    c.tp_world = world
    return c


def _weights(w):
    return O.OracleWeights(provider=synth.logical_provider(w, np.float64))


def _n(seed=3):
    return np.random.default_rng(seed).normal(0, 1, (2, 5, SHAPE.d_model))


@pytest.mark.parametrize("world", [2, 4, 8])
def test_rank_slices_give_the_oracles_partial_sums(world):
    """world 2: one kv head per rank; world 4 and 8: more ranks than kv heads, each kv head replicated."""
    w = synth.make_weights(SHAPE, std=0.2)
    n = _n()
    full = _cfg(SHAPE, world)
    for rank in range(world):
        rw = TP.rank_weights(w, rank, world)
        rs = rw.shape
        assert (rs.n_q_heads, rs.n_kv_heads, rs.d_ff) == (8 // world, max(2 // world, 1), 96 // world)
        assert rw.w_qkv[0].shape == (rs.qkv_rows, 64) and rw.w_o[0].shape == (64, rs.n_q_heads * 16)
        assert rw.w_gate_up[0].shape == (2 * rs.d_ff, 64) and rw.w_down[0].shape == (64, rs.d_ff)
        for layer in range(SHAPE.n_layers):
            mine_a = O.attention_module(_cfg(rs), _weights(rw), layer, n, 0, None)
            mine_m = O.mlp_module(_cfg(rs), _weights(rw), layer, n)
            ref_a = O.attention_module(full, _weights(w), layer, n, 0, None, tp_rank=rank)
            ref_m = O.mlp_module(full, _weights(w), layer, n, tp_rank=rank)
            np.testing.assert_allclose(mine_a, ref_a, rtol=0, atol=1e-12)
            np.testing.assert_allclose(mine_m, ref_m, rtol=0, atol=1e-12)


def test_rank_shape_rejects_what_does_not_divide():
    with pytest.raises(ValueError):
        TP.rank_shape(SHAPE, 3)
    with pytest.raises(ValueError):
        TP.rank_weights(synth.make_weights(SHAPE), 2, 2)
    assert TP.rank_shape(SHAPE, 1).d_ff == SHAPE.d_ff


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = synth.make_weights(SHAPE, std=0.2)
    rw = TP.rank_weights(w, rank, world)
    n = _n()
    part = torch.from_numpy(np.stack([O.attention_module(_cfg(rw.shape), _weights(rw), 1, n, 0, None),
                                      O.mlp_module(_cfg(rw.shape), _weights(rw), 1, n)]))
    dist.all_reduce(part)                         # the exchange of Sec. 2, Eq. 1
    whole = np.stack([O.attention_module(_cfg(SHAPE), _weights(w), 1, n, 0, None), O.mlp_module(_cfg(SHAPE), _weights(w), 1, n)])
    out[rank] = float(np.max(np.abs(part.numpy() - whole)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_sum_to_the_unsplit_modules():
    world, port = 2, 31500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        for r in range(world):
            assert out[r] < 1e-11, out[r]


def test_comm_entry_points_reject_bad_arguments_without_a_gpu():
    from paper_2501_06589_b200 import binding as B, build
    build.build()
    L = B.lib()
    import ctypes as C
    h = C.c_void_p()
    ident = C.create_string_buffer(B.COMM_ID_BYTES)
    assert L.ladder_comm_unique_id(None) == 1
    assert L.ladder_comm_create(0, 0, ident, C.byref(h)) == 1
    assert L.ladder_comm_create(2, 2, ident, C.byref(h)) == 1
    assert L.ladder_comm_create(2, 0, None, C.byref(h)) == 1
    assert L.ladder_comm_all_reduce_sum(None, None, 4, None) == 1
    assert L.ladder_comm_destroy(None) == 0 and L.ladder_comm_world(None) == 0 and L.ladder_comm_rank(None) == -1
    assert L.ladder_model_set_exchange(None, None, None, 0) == 1
    assert L.ladder_model_set_tensor_parallel(None, None) == 1
