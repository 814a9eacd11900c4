"""Tensor parallelism (paper Sec. 2, Eq. 1; Sec. 3.1, Algorithm 1): the host side.

One process per GPU.  Each rank builds its slice of the model (:func:`rank_shape`, :func:`rank_weights`: pure
indexing of the library's weight layout), creates a communicator (:func:`make_comm`) and installs it with
``Model.set_tensor_parallel``; every module's partial output is then summed over the ranks inside
``ladder_prefill`` / ``ladder_decode_step`` (see ``ladder_model_set_exchange`` in include/ladder.h for the schedule).

The split follows Sec. 2: rank r owns the query heads [r Hq/P, (r+1) Hq/P) with their key/value heads (replicated
when there are fewer kv heads than ranks) and the MLP hidden units [r F/P, (r+1) F/P); the projections into them are
split by output row, the projections out of them (W_o, W_down) by input column, so each rank's module output is a
partial sum.  Norm gains, embedding and LM head are whole on every rank.
"""
from __future__ import annotations

from dataclasses import replace
from typing import Optional

import torch

from .binding import Comm, Peer
from .synth import AbiWeights, ModelShape


def rank_shape(shape: ModelShape, world: int) -> ModelShape:
    """The shape of one rank's slice (the same for every rank)."""
    if world < 1 or shape.n_q_heads % world or shape.d_ff % world:
        raise ValueError("query heads and MLP hidden units must divide by the world size")
    if shape.n_kv_heads % world and world % shape.n_kv_heads:
        raise ValueError("kv heads must divide by the world size, or the world size by the kv heads")
    return replace(shape, name=f"{shape.name}_tp{world}", n_q_heads=shape.n_q_heads // world,
                   n_kv_heads=max(shape.n_kv_heads // world, 1), d_ff=shape.d_ff // world)


def rank_weights(w: AbiWeights, rank: int, world: int) -> AbiWeights:
    """Rank ``rank``'s slice of whole-model weights, in the library's layout (contiguous copies on w's device)."""
    s = w.shape
    rs = rank_shape(s, world)
    if not 0 <= rank < world:
        raise ValueError("rank outside the world")
    Dh = s.head_dim
    q0 = rank * rs.n_q_heads                                   # first query head
    kv0 = q0 // (s.n_q_heads // s.n_kv_heads)                  # the kv head its group reads
    k_base, v_base = s.n_q_heads * Dh, (s.n_q_heads + s.n_kv_heads) * Dh
    F0, F1 = rank * rs.d_ff, (rank + 1) * rs.d_ff
    out = AbiWeights(rs, w.tok_embedding, w.final_norm, w.lm_head)
    for l in range(s.n_layers):
        qkv = w.w_qkv[l]
        out.attn_norm.append(w.attn_norm[l])
        out.w_qkv.append(torch.cat([qkv[q0 * Dh:(q0 + rs.n_q_heads) * Dh],
                                    qkv[k_base + kv0 * Dh:k_base + (kv0 + rs.n_kv_heads) * Dh],
                                    qkv[v_base + kv0 * Dh:v_base + (kv0 + rs.n_kv_heads) * Dh]]).contiguous())
        out.w_o.append(w.w_o[l][:, q0 * Dh:(q0 + rs.n_q_heads) * Dh].contiguous())
        out.mlp_norm.append(w.mlp_norm[l])
        out.w_gate_up.append(w.w_gate_up[l][2 * F0:2 * F1].contiguous())       # rows 2j (gate_j), 2j + 1 (up_j)
        out.w_down.append(w.w_down[l][:, F0:F1].contiguous())
    return out


def make_comm(group=None) -> Comm:
    """A communicator over the ranks of a torch.distributed process group (the default group; a world of one when
    torch.distributed is not initialised).  Collective: every rank of the group calls it; each rank's current CUDA
    device must be the GPU it computes on.  Only the 128-byte id travels through torch.distributed."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return Comm(1, 0, Comm.unique_id())
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    box = [Comm.unique_id() if rank == 0 else None]
    dist.broadcast_object_list(box, src=dist.get_global_rank(group, 0) if group is not None else 0, group=group)
    return Comm(world, rank, box[0])


def make_peer(max_floats: int, group=None) -> Peer:
    """This rank's object for the exchange over peer memory, connected to every other rank of the group (one process
    per GPU: the CUDA IPC handles travel through torch.distributed).  max_floats >= max_batch x d_model, a multiple
    of 4.  Collective; ends with a barrier, so every rank is connected when it returns."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return Peer(1, 0, max_floats)
    world, rank = dist.get_world_size(group), dist.get_rank(group)
    peer = Peer(world, rank, max_floats)
    handles = [None] * world
    dist.all_gather_object(handles, peer.export(), group=group)
    for r in range(world):
        if r != rank:
            peer.connect(r, ipc_handle=handles[r])
    dist.barrier(group=group)
    return peer
