"""The allocation-free decode-attention entry point against the regular one.

Who needs it: callers that are not allowed to allocate device memory while running -- a server
whose own pool allocator owns the whole GPU, a memory-capped container slice, a framework that
forbids cudaMalloc after start-up.  Its scratch is a fixed array inside the library image.  The
test calls it through the C ABI twice in a row (the array keeps the first call's partials, which
must not leak into the second) and checks both results against ladder_op_decode_attention.
Collected last on purpose: a run that stops at the first failure has then run everything else.
"""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(B, batch, Hq, Hkv, Dh, max_seq, lens, seed):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(batch, Hq * Dh, generator=g).cuda()
    k = torch.randn(batch, Hkv, max_seq, Dh, generator=g).to(torch.bfloat16).cuda()
    v = torch.randn(batch, Hkv, max_seq, Dh, generator=g).to(torch.bfloat16).cuda()
    kv_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scratch = torch.empty(B.decode_attention_scratch_bytes(batch, Hq, Dh, max_seq) // 4, device="cuda")
    want = torch.full((batch, Hq * Dh), float("nan"), device="cuda")
    B.op_decode_attention(q, k, v, kv_len, Hq, Hkv, Dh, max_seq, scratch, want)
    got = torch.full_like(want, float("nan"))
    B.op_decode_attention_noalloc(q, k, v, kv_len, Hq, Hkv, Dh, max_seq, got)
    torch.cuda.synchronize()
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
    k = torch.zeros(1, dtype=torch.bfloat16, device="cuda")
    lens = torch.zeros(64, dtype=torch.int32, device="cuda")
    o = torch.zeros_like(q)
    with pytest.raises(B.LadderError) as e:                      # 64 x 64 x 128 splits x 130 floats >> 8 MiB
        B.op_decode_attention_noalloc(q, k, k, lens, 64, 8, 128, 8192, o)
    assert e.value.status == 2
