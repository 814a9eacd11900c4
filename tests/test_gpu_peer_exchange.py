"""The exchange over peer memory on ONE GPU: a world of one; a world of two in which the test makes the absent
rank's stores (always BEFORE the kernel that waits for them, on the same stream, so nothing ever spins on another
launch); the bounded wait running out; the IPC hand-shake between two processes by host copies only."""
import os
import sys

import numpy as np
import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2501_06589_b200 import binding, build
    build.build()
    binding.lib()
    return binding


class _Dev:
    def __init__(self, ptr, count, typestr):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": typestr, "data": (ptr, False), "version": 2}


def floats_at(ptr, count):
    return torch.as_tensor(_Dev(ptr, count, "<f4"), device="cuda")


def counter_at(ptr):
    return torch.as_tensor(_Dev(ptr, 1, "<i4"), device="cuda")


def test_world_of_one_is_the_identity_on_both_channels(B):
    n = 6 * 1024
    peer = B.Peer(1, 0, n)
    assert peer.connected()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    for t in range(5):                       # both slot parities, several turns
        for ch in (0, 1):
            x = torch.randn(n - 4 * t, device="cuda")
            y = x.clone()
            peer.all_reduce_sum(ch, y.data_ptr(), y.numel(), status.data_ptr())
            assert torch.equal(x, y)
            assert counter_at(peer.counter_ptr(ch, 0)).item() == (t + 1) * B.Peer.ctas_per_exchange()
    assert status.item() == 0
    with pytest.raises(B.LadderError):
        peer.all_reduce_sum(0, y.data_ptr(), n + 4, status.data_ptr())      # larger than the slots
    with pytest.raises(B.LadderError):
        peer.all_reduce_sum(2, y.data_ptr(), 4, status.data_ptr())
    peer.close()


def two_ranks_in_one_process(B, n):
    p0, p1 = B.Peer(2, 0, n), B.Peer(2, 1, n)
    assert not p0.connected()
    p0.connect(1, same_process_base=p1.local_base())
    p1.connect(0, same_process_base=p0.local_base())
    assert p0.connected() and p1.connected()
    return p0, p1


def test_world_of_two_with_the_other_ranks_stores_made_by_the_test(B):
    """Rank 0 runs the kernel; what rank 1 would have stored into rank 0's memory (its partial and its 16 arrivals)
    is written beforehand.  Rank 0's sum is x0 + x1 in that order, and rank 0's own partial and arrivals have landed
    in rank 1's memory."""
    n = 4096
    p0, p1 = two_ranks_in_one_process(B, n)
    g = B.Peer.ctas_per_exchange()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    turns = [0, 0]
    for step in range(7):
        ch = step % 2 if step < 4 else 1
        t = turns[ch]
        count = n - 8 * step
        x0, x1 = torch.randn(count, device="cuda"), torch.randn(count, device="cuda")
        floats_at(p0.slot_ptr(ch, t & 1, 1), count).copy_(x1)
        counter_at(p0.counter_ptr(ch, 1)).add_(g)
        y = x0.clone()
        p0.all_reduce_sum(ch, y.data_ptr(), count, status.data_ptr())
        assert torch.equal(y, x0 + x1)
        assert torch.equal(floats_at(p1.slot_ptr(ch, t & 1, 0), count), x0)
        assert counter_at(p1.counter_ptr(ch, 0)).item() == (t + 1) * g
        turns[ch] += 1
    assert status.item() == 0
    p0.close()
    p1.close()


def test_the_wait_runs_out_cleanly_when_a_rank_never_arrives(B):
    """Nothing sets rank 1's counter: the kernel gives up after its limit, reports LADDER_DEV_TIMEOUT (4), leaves the
    partial alone, and the context stays usable; the next exchange (with rank 1 present) works."""
    n = 1024
    p0, p1 = two_ranks_in_one_process(B, n)
    g = B.Peer.ctas_per_exchange()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    x0 = torch.randn(n, device="cuda")
    y = x0.clone()
    p0.all_reduce_sum(0, y.data_ptr(), n, status.data_ptr())
    torch.cuda.synchronize()
    assert status.item() == 4 and torch.equal(y, x0)
    status.zero_()
    counter_at(p0.counter_ptr(0, 1)).add_(g)          # rank 1's late arrival for the turn that was given up
    x1 = torch.randn(n, device="cuda")
    floats_at(p0.slot_ptr(0, 1, 1), n).copy_(x1)       # turn 1: the other slot
    counter_at(p0.counter_ptr(0, 1)).add_(g)
    p0.all_reduce_sum(0, y.data_ptr(), n, status.data_ptr())
    assert status.item() == 0 and torch.equal(y, x0 + x1)
    p0.close()
    p1.close()


def _ipc_worker(rank, world, port, out):
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from paper_2501_06589_b200 import binding as Bm, tensor_parallel as TP
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    torch.cuda.set_device(0)                       # both ranks on the one GPU: host copies only, no kernel waits
    peer = TP.make_peer(256)
    other = 1 - rank
    peer.probe_write(other, 1000 + rank)
    dist.barrier()
    out[rank] = (peer.connected(), peer.probe_read(other))
    dist.barrier()
    peer.close()
    dist.destroy_process_group()


def test_ipc_handles_connect_two_processes(B):
    import torch.multiprocessing as mp
    world, port = 2, 33500 + os.getpid() % 2000
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_ipc_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == (True, 1001) and out[1] == (True, 1000)
