"""Tensor parallelism on ONE GPU (paper Sec. 2, Eq. 1; Sec. 3.1, Algorithm 1).

No second GPU is available to these tests, so the other ranks are played by the oracle: it runs the whole model
split over the ranks and records every rank's partial sum of every module; the GPU runs rank 0's weight slice and
its exchange callback adds the recorded partials of the other ranks where an all-reduce would.  What comes out must
be the unsplit model.  A second set runs the NCCL exchange itself in a world of one rank (the collective is then
the identity, but it is enqueued, captured into the decode graph and replayed like any other)."""
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from oracle import ladder_oracle as O                                        # noqa: E402
from paper_2501_06589_b200 import synth                                      # noqa: E402
from tests.helpers import rel_err                                            # noqa: E402

pytestmark = pytest.mark.gpu
HIDDEN_TOL = 2e-2
BASE = synth.ModelShape("tiny_tp", 256, 4, 4, 2, 64, 704, 1024, 1e-5, 10000.0, None, 2, 12, 6, 11)
VARIANTS = {"ladder": None, "standard": (0, 0, 0, 0), "hybrid": (0, 0, 1, 1)}


@pytest.fixture(scope="module")
def B():
    from paper_2501_06589_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def oracle_cfg(s, world):
    c = O.OracleConfig(s.d_model, s.n_layers, s.n_q_heads, s.n_kv_heads, s.head_dim, s.d_ff, s.vocab_size,
                       s.rms_eps, s.rope_theta, None if s.layer_is_ladder is None else list(s.layer_is_ladder),
                       layer_mode=None if s.layer_mode is None else list(s.layer_mode),
                       module_stale=None if s.module_stale is None else list(s.module_stale))
    c.tp_world = world
    return c


def exchanged(parts, variant):
    """The oracle's per-module partial sums, grouped the way the library exchanges them: one by one, except that a
    parallel attention + MLP layer (Sec. 3.3.1) sums its two outputs before its ONE exchange."""
    if variant != "parallel":
        return list(parts)
    return [parts[i] + parts[i + 1] for i in range(0, len(parts), 2)]


class _DeviceFloats:
    """`count` fp32 values at a raw device address, for torch.as_tensor (no copy)."""

    def __init__(self, ptr, count):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": "<f4", "data": (ptr, False), "version": 2}


def shape_of(variant):
    from dataclasses import replace
    if variant == "parallel":                    # attention and MLP of a layer read the same input (Sec. 3.3.1)
        return BASE.as_mode("parallel")
    if variant == "flags":                       # an arbitrary per-module rule: every kind of neighbour pair occurs
        return replace(BASE, layer_mode=tuple(["standard"] * BASE.n_layers), module_stale=(0, 1, 1, 0, 0, 0, 1, 1))
    return replace(BASE, layer_is_ladder=VARIANTS[variant])


CASES = [(v, b, st, 12) for v in ("ladder", "standard", "hybrid") for b in (2, 6) for st in (2, 1)]
CASES += [("ladder", 4, 2, 80), ("standard", 4, 2, 80)]     # 320 prompt tokens: the binary16 prompt-pass GEMMs
CASES += [(v, b, st, 12) for v in ("parallel", "flags") for b in (3, 9) for st in (2, 1)]


@pytest.mark.parametrize("variant,batch,streams,S", CASES)
def test_rank_0_with_the_oracle_as_rank_1(B, variant, batch, streams, S):
    from paper_2501_06589_b200 import tensor_parallel as TP
    s = shape_of(variant)
    world, steps = 2, 6
    w = synth.make_weights(s, device="cuda", gains="uniform")
    prompt = synth.make_tokens(s, batch, S)

    # the oracle: the model split over two ranks, every rank's partial sums recorded call by call
    cfg = oracle_cfg(s, world)
    OW = O.OracleWeights(provider=synth.logical_provider(w, np.float64))
    cache_o = O.OracleCache(cfg, batch, S + steps + 1, np.float64)
    calls, o_toks, o_hids = [], [], []
    r = O.forward(cfg, OW, prompt, np.float64, cache_o, 0, last_only=True, record=True)
    for j in range(steps + 1):
        calls.append(exchanged([parts[1] for parts in r.module_partials], variant))
        o_toks.append(r.next_tokens[:, 0])
        o_hids.append(r.hidden[:, 0])
        if j < steps:
            r = O.forward(cfg, OW, o_toks[-1].reshape(-1, 1), np.float64, cache_o, cache_o.seq_len, last_only=True,
                          record=True)
    unsplit = O.generate(oracle_cfg(s, 1), OW, prompt, steps, S + steps + 1, dtype=np.float64,
                         forced=np.stack(o_toks, 1))
    assert rel_err(np.stack(o_hids, 1), unsplit[1]) < 1e-9            # the split oracle is the unsplit one

    # the GPU: rank 0's slice; the exchange adds rank 1's recorded partial of the same module
    rw = TP.rank_weights(w, 0, world)
    model = B.Model(rw, batch, S + steps + 1, batch * S)
    model.set_schedule(streams, True, True)
    queue, seen = [], []

    def exchange(ptr, count, stream):
        peer = queue.pop(0)
        assert peer.numel() == count, (peer.numel(), count)
        view = torch.as_tensor(_DeviceFloats(ptr, count), device="cuda")
        with torch.cuda.stream(torch.cuda.ExternalStream(stream or 0)):
            view.add_(peer)
        seen.append(count)
        return 0

    model.set_exchange(exchange, capturable=False)
    cache = B.KVCache(rw.shape, batch, S + steps + 1)
    nxt = torch.zeros(batch, dtype=torch.int32, device="cuda")
    hid = torch.zeros(batch, s.d_model, device="cuda")
    toks, hids = [], []
    for j in range(steps + 1):
        queue[:] = [torch.from_numpy(np.ascontiguousarray(p, dtype=np.float32).reshape(-1)).cuda() for p in calls[j]]
        if j == 0:
            model.prefill(cache, torch.from_numpy(prompt).cuda(), next_tokens=nxt, final_hidden=hid)
        else:                                                   # teacher forcing: the recorded partials belong to these tokens
            feed = torch.from_numpy(o_toks[j - 1].astype(np.int32)).cuda()
            model.decode_step(cache, feed, next_tokens=nxt, final_hidden=hid)
        torch.cuda.synchronize()
        assert not queue, "an exchange was skipped"
        toks.append(nxt.cpu().numpy().copy())
        hids.append(hid.cpu().numpy().copy())
    assert model.device_status() == 0
    per_pass = s.n_layers if variant == "parallel" else 2 * s.n_layers
    assert seen == [batch * S * s.d_model] * per_pass + [batch * s.d_model] * (per_pass * steps)
    err = rel_err(np.stack(hids, 1), np.stack(o_hids, 1))
    agree = float(np.mean(np.stack(toks, 1) == np.stack(o_toks, 1)))
    print(f"[tp rank 0 / oracle rank 1, {variant}, batch {batch}, {streams} stream(s)] hidden max-rel-err {err:.3e}, "
          f"greedy agreement {agree:.3f} over {batch * (steps + 1)}")
    assert err < HIDDEN_TOL, err
    assert agree >= 0.9, agree
    model.close()


@pytest.mark.parametrize("variant,batch", [("ladder", 3), ("standard", 3), ("ladder", 12), ("hybrid", 12)])
def test_world_of_one_over_nccl(B, variant, batch):
    """The NCCL exchange in a world of one: the steps run in the pending-output form with an all-reduce after every
    module, inside the captured decode graph.  Bit-identical to the same form with a do-nothing callback enqueued
    step by step, and to the ordinary schedule with the residual added in the GEMM epilogues, every GEMM on all SMs
    (batch > 4: the same kernels on the same grids, so the same bits)."""
    from paper_2501_06589_b200 import tensor_parallel as TP
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from tests.test_gpu_model import gpu_generate, oracle_teacher_forced
    s = shape_of(variant)
    w = synth.make_weights(s, device="cuda", gains="uniform")
    S, steps = 10, 12
    prompt = synth.make_tokens(s, batch, S)
    comm = TP.make_comm()
    assert (comm.world, comm.rank) == (1, 0)
    probe = torch.arange(8, dtype=torch.float32, device="cuda")
    comm.all_reduce_sum(probe)
    assert torch.equal(probe.cpu(), torch.arange(8, dtype=torch.float32))

    def run(mode):
        model = B.Model(w, batch, S + steps + 2, batch * S)
        if mode == "nccl":
            model.set_tensor_parallel(comm)
        elif mode == "callback":
            model.set_exchange(lambda ptr, count, stream: 0, capturable=False)
        else:
            model.set_sm_split(-2)
        cache = B.KVCache(s, batch, S + steps + 2)
        toks, hids = gpu_generate(B, model, cache, prompt, steps)
        assert model.device_status() == 0
        model.close()
        return toks, hids

    t_nccl, h_nccl = run("nccl")
    t_cb, h_cb = run("callback")
    assert np.array_equal(t_nccl, t_cb) and np.array_equal(h_nccl, h_cb)
    if batch > 4:
        t_def, h_def = run("default")
        assert np.array_equal(t_nccl, t_def) and np.array_equal(h_nccl, h_def)
    o_toks, o_hids, _ = oracle_teacher_forced(s, w, prompt, t_nccl, np.float64)
    err = rel_err(h_nccl, o_hids)
    print(f"[nccl world 1, {variant}, batch {batch}] hidden max-rel-err {err:.3e}, greedy agreement "
          f"{float(np.mean(t_nccl == o_toks)):.3f}")
    assert err < HIDDEN_TOL, err
    comm.close()


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("mask,cut,bsz", [((1, 1, 1, 1), 2, 3), ((0, 1, 1, 0), 2, 6), ((1, 1, 0, 1), 1, 3)])
def test_pipeline_stages_under_tensor_parallelism(B, mask, cut, bsz, fused):
    """Tensor parallelism inside every pipeline stage (Sec. 5.1), in a world of one: two stage models chained through
    the handed-on pair reproduce the whole tensor-parallel model bit for bit, prompt pass and decode steps, with the
    exchange over NCCL and fused over peer memory (one peer object per model)."""
    from paper_2501_06589_b200 import tensor_parallel as TP
    from tests.test_gpu_model import gpu_generate, _whole_model_flags
    s = synth.replace(BASE, layer_is_ladder=mask)
    w = synth.make_weights(s, device="cuda", gains="uniform")
    S, steps = 20, 6
    max_seq = S + steps + 2
    prompt = synth.make_tokens(s, bsz, S)
    tok = torch.from_numpy(prompt).cuda()
    flags = _whole_model_flags(s)
    comm = TP.make_comm()
    peers = []

    def parallel(model):
        if fused:
            peers.append(TP.make_peer(bsz * s.d_model))
            model.set_tensor_parallel_peer(comm, peers[-1])
        else:
            model.set_tensor_parallel(comm)
        return model

    whole = parallel(B.Model(w, bsz, max_seq, bsz * S))
    ref_toks, ref_hids = gpu_generate(B, whole, B.KVCache(s, bsz, max_seq), prompt, steps)
    whole.close()

    def stage(lo, hi):
        sh = synth.replace(s, n_layers=hi - lo, layer_is_ladder=tuple(mask[lo:hi]), module_stale=tuple(flags[2 * lo:2 * hi]))
        ws = synth.AbiWeights(sh, w.tok_embedding, w.final_norm, w.lm_head, w.attn_norm[lo:hi], w.w_qkv[lo:hi],
                              w.w_o[lo:hi], w.mlp_norm[lo:hi], w.w_gate_up[lo:hi], w.w_down[lo:hi])
        return parallel(B.Model(ws, bsz, max_seq, bsz * S)), B.KVCache(sh, bsz, max_seq)

    (m0, c0), (m1, c1) = stage(0, cut), stage(cut, 4)
    d = s.d_model
    big = (torch.zeros(bsz * S, d, device="cuda"), torch.zeros(bsz * S, d, device="cuda"))
    small = (torch.zeros(bsz, d, device="cuda"), torch.zeros(bsz, d, device="cuda"))
    nxt = torch.zeros(bsz, dtype=torch.int32, device="cuda")
    hid = torch.zeros(bsz, d, device="cuda")
    m0.stage_prefill(c0, tok, bsz, S, state_out=big)
    m1.stage_prefill(c1, None, bsz, S, state_in=big, next_tokens=nxt, final_hidden=hid)
    toks, hids = [nxt.clone()], [hid.clone()]
    for _ in range(steps):
        m0.stage_decode_step(c0, nxt, bsz, state_out=small)
        m1.stage_decode_step(c1, None, bsz, state_in=small, next_tokens=nxt, final_hidden=hid)
        toks.append(nxt.clone())
        hids.append(hid.clone())
    torch.cuda.synchronize()
    assert m0.device_status() == 0 and m1.device_status() == 0
    assert np.array_equal(torch.stack(toks, 1).cpu().numpy(), ref_toks)
    assert np.array_equal(torch.stack(hids, 1).cpu().numpy(), ref_hids)
    assert c0.seq_lens.cpu().tolist() == [S + steps] * bsz and c1.seq_lens.cpu().tolist() == [S + steps] * bsz
    m0.close()
    m1.close()
    for p in peers:
        p.close()
    comm.close()


@pytest.mark.parametrize("variant,batch", [("ladder", 3), ("hybrid", 12)])
def test_decode_exchange_over_peer_memory_in_a_world_of_one(B, variant, batch):
    """Decode steps exchange through the peer-memory kernel (inside the captured graph), the prompt pass through
    NCCL: bit-identical to NCCL for both."""
    from paper_2501_06589_b200 import tensor_parallel as TP
    from tests.test_gpu_model import gpu_generate
    s = shape_of(variant)
    w = synth.make_weights(s, device="cuda", gains="uniform")
    S, steps = 10, 12
    prompt = synth.make_tokens(s, batch, S)
    comm = TP.make_comm()
    peer = TP.make_peer(batch * s.d_model)
    runs = []
    for use_peer in (False, True):
        model = B.Model(w, batch, S + steps + 2, batch * S)
        if use_peer:
            model.set_tensor_parallel_peer(comm, peer)
        else:
            model.set_tensor_parallel(comm)
        cache = B.KVCache(s, batch, S + steps + 2)
        runs.append(gpu_generate(B, model, cache, prompt, steps))
        assert model.device_status() == 0
        model.close()
    assert np.array_equal(runs[0][0], runs[1][0]) and np.array_equal(runs[0][1], runs[1][1])
    # above the size limit the decode steps leave the exchange to NCCL: same results, nothing lands in the slots
    fresh = TP.make_peer(batch * s.d_model)
    model = B.Model(w, batch, S + steps + 2, batch * S)
    model.set_tensor_parallel_peer(comm, fresh)
    model.set_peer_max_bytes(-1)
    t3, h3 = gpu_generate(B, model, B.KVCache(s, batch, S + steps + 2), prompt, steps)
    assert np.array_equal(runs[0][0], t3) and np.array_equal(runs[0][1], h3)
    slot = torch.as_tensor(_DeviceFloats(fresh.slot_ptr(0, 0, 0), 2 * batch * s.d_model), device="cuda")
    assert float(slot.abs().max()) == 0.0
    used = torch.as_tensor(_DeviceFloats(peer.slot_ptr(0, 0, 0), 2 * batch * s.d_model), device="cuda")
    assert float(used.abs().max()) > 0.0
    model.close()
    fresh.close()
    small = B.Peer(1, 0, 64)
    model = B.Model(w, batch, 32, 32)
    with pytest.raises(B.LadderError):
        model.set_tensor_parallel_peer(comm, small)        # slots smaller than batch x d_model
    model.close()
    small.close()
    peer.close()
    comm.close()


@pytest.mark.parametrize("streams", [2, 1])
@pytest.mark.parametrize("variant,batch,world", [("ladder", 6, 2), ("standard", 6, 2), ("hybrid", 3, 2), ("ladder", 40, 2),
                                                 ("parallel", 6, 2), ("flags", 5, 2), ("ladder", 9, 4), ("standard", 2, 4)])
def test_rank_0_over_peer_memory_with_the_oracle_as_rank_1(B, variant, batch, world, streams):
    """As test_rank_0_with_the_oracle_as_rank_1, but the decode-step exchange is the fused one: rank 0's output GEMMs
    push their partial sums into the receive slots (rank 0's own and, on the same GPU, those of a second object that
    stands for rank 1's memory) as (value, sequence number) pairs, and the staging launches poll the pairs and add
    the slots.  Rank 1's stores - the oracle's rank-1 partial, numbered like rank 0's - are enqueued by the test right
    behind each output GEMM, so every poll succeeds at once."""
    from paper_2501_06589_b200 import tensor_parallel as TP
    s = shape_of(variant)
    S, steps = 12, 6                                          # world 4: more ranks than kv heads (each kv head on two ranks)
    w = synth.make_weights(s, device="cuda", gains="uniform")
    prompt = synth.make_tokens(s, batch, S)
    cfg = oracle_cfg(s, world)
    OW = O.OracleWeights(provider=synth.logical_provider(w, np.float64))
    cache_o = O.OracleCache(cfg, batch, S + steps + 1, np.float64)
    calls, o_toks, o_hids = [], [], []
    r = O.forward(cfg, OW, prompt, np.float64, cache_o, 0, last_only=True, record=True)
    for j in range(steps + 1):
        calls.append([exchanged([parts[k] for parts in r.module_partials], variant) for k in range(1, world)])
        o_toks.append(r.next_tokens[:, 0])
        o_hids.append(r.hidden[:, 0])
        if j < steps:
            r = O.forward(cfg, OW, o_toks[-1].reshape(-1, 1), np.float64, cache_o, cache_o.seq_len, last_only=True,
                          record=True)

    n = batch * s.d_model
    p0 = B.Peer(world, 0, n)
    others = [B.Peer(world, k, n) for k in range(1, world)]   # memory that stands for the other ranks'
    for k, pk in enumerate(others, start=1):
        p0.connect(k, same_process_base=pk.local_base())
    p1 = others[0]
    rw = TP.rank_weights(w, 0, world)
    model = B.Model(rw, batch, S + steps + 1, batch * S)
    model.set_schedule(streams, True, True)
    queue, turns = [], [0, 0]

    class _Words:
        def __init__(self, ptr, count):
            self.__cuda_array_interface__ = {"shape": (count,), "typestr": "<i4", "data": (ptr, False), "version": 2}

    def words(ptr, count):
        return torch.as_tensor(_Words(ptr, count), device="cuda")

    def prompt_exchange(ptr, count, stream):                 # the prompt pass: NCCL's place
        with torch.cuda.stream(torch.cuda.ExternalStream(stream or 0)):
            for part in queue.pop(0):
                torch.as_tensor(_DeviceFloats(ptr, count), device="cuda").add_(part)
        return 0

    def rank_1_arrives(channel, stream):                     # a decode-step output GEMM of rank 0 has been enqueued
        for k, part in enumerate(queue.pop(0), start=1):      # the other ranks' stores into rank 0's receive slots
            pairs = torch.empty(n, 2, dtype=torch.int32, device="cuda")   # (value, sequence number of the exchange)
            pairs[:, 0] = part.view(torch.int32)
            pairs[:, 1] = turns[channel] + 1
            with torch.cuda.stream(torch.cuda.ExternalStream(stream or 0)):
                words(p0.slot_ptr(channel, turns[channel] & 1, k), 2 * n).copy_(pairs.view(-1))
        turns[channel] += 1

    model.set_exchange(prompt_exchange, capturable=False)
    model.set_peer(p0)
    model.debug_set_peer_hook(rank_1_arrives)
    cache = B.KVCache(rw.shape, batch, S + steps + 1)
    nxt = torch.zeros(batch, dtype=torch.int32, device="cuda")
    hid = torch.zeros(batch, s.d_model, device="cuda")
    hids = []
    for j in range(steps + 1):
        up = lambda p: torch.from_numpy(np.ascontiguousarray(p, dtype=np.float32).reshape(-1)).cuda()
        queue[:] = [[up(calls[j][k][i]) for k in range(world - 1)] for i in range(len(calls[j][0]))]
        if j == 0:
            model.prefill(cache, torch.from_numpy(prompt).cuda(), next_tokens=nxt, final_hidden=hid)
        else:
            model.decode_step(cache, torch.from_numpy(o_toks[j - 1].astype(np.int32)).cuda(), next_tokens=nxt,
                              final_hidden=hid)
        torch.cuda.synchronize()
        assert not queue
        hids.append(hid.cpu().numpy().copy())
    assert model.device_status() == 0
    assert turns == ([0, s.n_layers * steps] if variant == "parallel" else [s.n_layers * steps] * 2)
    # rank 0's partial of the last exchange of a channel has landed in "rank 1's" memory too, numbered like its own copy
    ch = 1 if variant == "parallel" else 0
    last = turns[ch] - 1
    mine = words(p0.slot_ptr(ch, last & 1, 0), 2 * n).view(n, 2)
    theirs = words(p1.slot_ptr(ch, last & 1, 0), 2 * n).view(n, 2)
    assert torch.equal(mine, theirs) and bool((mine[:, 1] == last + 1).all()) and int(mine[:, 0].abs().max()) > 0
    err = rel_err(np.stack(hids, 1), np.stack(o_hids, 1))
    print(f"[tp rank 0, fused exchange over peer memory / oracle rank 1, {variant}, batch {batch}, {streams} stream(s)] "
          f"hidden max-rel-err {err:.3e}")
    assert err < HIDDEN_TOL, err
    model.close()
    p0.close()
    for pk in others:
        pk.close()


def test_fused_exchange_gives_up_cleanly_when_a_rank_never_stores(B):
    """Rank 1 of a world of two never shows up: the first staging launch that needs its pairs polls for its limit
    (about 0.3 s), sets LADDER_DEV_TIMEOUT, and from then on nothing waits any more; nothing hangs or faults, the status word says so, the
    model refuses further steps, and the device keeps working."""
    import time
    from paper_2501_06589_b200 import tensor_parallel as TP
    s = shape_of("ladder")
    batch, S = 2, 8
    w = synth.make_weights(s, device="cuda", gains="uniform")
    rw = TP.rank_weights(w, 0, 2)
    n = batch * s.d_model
    p0, p1 = B.Peer(2, 0, n), B.Peer(2, 1, n)
    p0.connect(1, same_process_base=p1.local_base())
    model = B.Model(rw, batch, 32, batch * S)
    model.set_exchange(lambda ptr, count, stream: 0, capturable=True)     # the prompt pass: rank 1 contributes nothing
    model.set_peer(p0)
    cache = B.KVCache(rw.shape, batch, 32)
    nxt = torch.zeros(batch, dtype=torch.int32, device="cuda")
    model.prefill(cache, torch.from_numpy(synth.make_tokens(s, batch, S)).cuda(), next_tokens=nxt)
    torch.cuda.synchronize()
    t0 = time.time()
    model.decode_step(cache, nxt, next_tokens=nxt)
    torch.cuda.synchronize()
    took = time.time() - t0
    assert model.device_status() == 4                     # LADDER_DEV_TIMEOUT
    assert 0.2 < took < 5.0, took                         # one wait of ~0.3 s; the launches behind it do not wait again
    with pytest.raises(B.LadderError):
        model.decode_step(cache, nxt, next_tokens=nxt)    # refused until the caller has dealt with it
    x = torch.arange(1024, device="cuda", dtype=torch.float32)
    assert float((x * 2).sum()) == 2 * 1023 * 1024 / 2    # the context is intact
    model.close()
    p0.close()
    p1.close()
