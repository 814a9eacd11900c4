"""The allocation-free decode-attention entry point against the regular one.

Who needs it: callers that are not allowed to allocate device memory while running -- a server
whose own pool allocator owns the whole GPU, a memory-capped container slice, a framework that
forbids cudaMalloc after start-up.  Its scratch is a fixed array inside the library image.  The
test calls it through the C ABI twice in a row (the array keeps the first call's partials, which
must not leak into the second) and checks both results against ladder_op_decode_attention and
against the CPU oracle's attention.
Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from oracle import ladder_oracle as O
from tests.helpers import rel_err

pytestmark = pytest.mark.gpu


def _case(B, batch, Hq, Hkv, Dh, max_seq, lens, seed):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(batch, Hq * Dh, generator=g).cuda()
    k = torch.randn(batch, Hkv, max_seq, Dh, generator=g).to(torch.float16).cuda()
    v = torch.randn(batch, Hkv, max_seq, Dh, generator=g).to(torch.float16).cuda()
    kv_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scratch = torch.empty(B.decode_attention_scratch_bytes(batch, Hq, Dh, max_seq) // 4, device="cuda")
    want = torch.full((batch, Hq * Dh), float("nan"), device="cuda")
    B.op_decode_attention(q, k, v, kv_len, Hq, Hkv, Dh, max_seq, scratch, want)
    got = torch.full_like(want, float("nan"))
    B.op_decode_attention_noalloc(q, k, v, kv_len, Hq, Hkv, Dh, max_seq, got)
    torch.cuda.synchronize()
    # and directly against the CPU oracle's attention, one sequence at a time (the tolerance of the regular
    # entry point's own test: fp32 accumulation against float64)
    f64 = lambda t: t.detach().float().cpu().numpy().astype(np.float64)
    for b, L in enumerate(lens):
        ref = O.causal_attention(f64(q[b]).reshape(1, Hq, Dh), f64(k[b, :, :L]).transpose(1, 0, 2),
                                 f64(v[b, :, :L]).transpose(1, 0, 2), L - 1)[0]
        assert rel_err(f64(got[b]).reshape(Hq, Dh), ref) < 1e-3, b
    return got, want


def test_noalloc_decode_attention_matches_regular_entry_point_twice():
    from paper_2501_06589_b200 import binding as B, build
    build.build()
    B.lib()
    # first call: a long context; second call right after it: a different, shorter problem that
    # reuses the front of the same scratch array
    got, want = _case(B, 4, 64, 8, 128, 1536, [1025, 1300, 1536, 1], seed=1)
    assert torch.allclose(got, want, rtol=0.0, atol=1e-6)
    got, want = _case(B, 2, 16, 16, 128, 640, [513, 77], seed=2)
    assert torch.allclose(got, want, rtol=0.0, atol=1e-6)


def test_noalloc_rejects_shapes_beyond_its_fixed_scratch():
    from paper_2501_06589_b200 import binding as B, build
    build.build()
    q = torch.zeros(64, 64 * 128, device="cuda")
    k = torch.zeros(8, dtype=torch.float16, device="cuda")
    lens = torch.zeros(64, dtype=torch.int32, device="cuda")
    o = torch.zeros_like(q)
    with pytest.raises(B.LadderError) as e:                      # 64 x 64 x 128 splits x 130 floats >> 8 MiB
        B.op_decode_attention_noalloc(q, k, k, lens, 64, 8, 128, 8192, o)
    assert e.value.status == 2
