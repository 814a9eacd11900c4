"""Per-kernel parity: each CUDA kernel, called through the C ABI, against the oracle's
operation on the same seeded inputs, at shapes that span several tiles and a ragged tail
and at the true 70B decode shapes."""
import numpy as np
import pytest
import torch

from oracle import ladder_oracle as O
from tests.helpers import rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2501_06589_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def _bf16(shape, seed, std=1.0, device="cuda"):
    g = torch.Generator(device="cpu").manual_seed(seed)
    return (torch.randn(shape, generator=g) * std).to(torch.bfloat16).to(device)


def _f16(shape, seed, std=1.0, device="cuda"):
    g = torch.Generator(device="cpu").manual_seed(seed)
    return (torch.randn(shape, generator=g) * std).to(torch.float16).to(device)


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


# Decode GEMMs feed the activation as a bf16 hi+lo pair for batch <= 4 (packed into one MMA tile)
# and for batch 9..64 (tcgen05 kernel: hi and lo are separate MMA columns): what is left is fp32
# accumulation error, ~1e-5 of the row maximum.  Batches 5..8 use a single bf16 (2^-9 relative rounding
# per element, random sign), ~1e-3 of the maximum.
def tol_gemm(batch):
    return 2e-4 if (batch <= 4 or batch >= 9) else 1e-2


@pytest.mark.parametrize("N,K,batch", [(256, 256, 1), (1376, 256, 4), (256, 688, 3), (1024, 2048, 8),
                                       (10240, 8192, 4), (4104, 1024, 16), (2048, 1280, 33), (1000, 520, 64)])
def test_smallm_gemm_norm_plain(B, N, K, batch):
    W = _bf16((N, K), 1, 0.02)
    x = torch.randn(batch, K, generator=torch.Generator().manual_seed(2)).cuda() * 3.0
    g = (torch.rand(K, generator=torch.Generator().manual_seed(3)) + 0.5).to(torch.bfloat16).cuda()
    out = torch.full((batch, N), float("nan"), device="cuda")
    B.op_smallm_gemm(W, x, 1, 2, out, gain=g, eps=1e-5)
    torch.cuda.synchronize()
    ref = O.rmsnorm(_f64(x), _f64(g), 1e-5) @ _f64(W).T
    assert rel_err(out.cpu().numpy(), ref) < tol_gemm(batch)


@pytest.mark.parametrize("N,K,batch", [(256, 688, 1), (8192, 8192, 4), (8192, 28672, 4), (512, 1032, 7), (776, 3584, 16)])
def test_smallm_gemm_bf16_residual(B, N, K, batch):
    W = _bf16((N, K), 4, 0.02)
    a = torch.randn(batch, K, generator=torch.Generator().manual_seed(5)).cuda()
    addend = torch.randn(batch, N, generator=torch.Generator().manual_seed(6)).cuda()
    out = torch.empty_like(addend)
    B.op_smallm_gemm(W, a, 0, 0, out, addend=addend)
    torch.cuda.synchronize()
    ref = _f64(addend) + _f64(a) @ _f64(W).T
    assert rel_err(out.cpu().numpy(), ref) < tol_gemm(batch)
    # in place (standard-residual layers): destination == addend
    inplace = addend.clone()
    B.op_smallm_gemm(W, a, 0, 0, inplace, addend=inplace)
    torch.cuda.synchronize()
    assert torch.equal(inplace, out)


@pytest.mark.parametrize("F,K,batch", [(688, 256, 1), (28672 // 8, 8192, 4), (1004, 520, 5)])
def test_smallm_gemm_swiglu(B, F, K, batch):
    W = _bf16((2 * F, K), 7, 0.05)
    x = torch.randn(batch, K, generator=torch.Generator().manual_seed(8)).cuda()
    g = torch.ones(K, dtype=torch.bfloat16, device="cuda")
    out = torch.empty(batch, F, device="cuda")
    B.op_smallm_gemm(W, x, 1, 1, out, gain=g, eps=1e-5)
    torch.cuda.synchronize()
    n = O.rmsnorm(_f64(x), _f64(g), 1e-5)
    w = _f64(W)
    ref = O.silu(n @ w[0::2].T) * (n @ w[1::2].T)
    assert rel_err(_f64(out), ref) < (5e-4 if batch <= 4 else 2e-2)


@pytest.mark.parametrize("impl", [0, 2])          # 0 = tcgen05 kernel for batch > 4, 2 = tcgen05 kernel for any batch
@pytest.mark.parametrize("N,K,batch,mode", [
    (1024, 8192, 16, "resid"),      # 8 row tiles over 148 CTAs: every tile is shared by ~18 CTAs (fix-up path)
    (1000, 520, 64, "plain"),       # ragged last tile, K not a multiple of 64
    (7168, 1024, 33, "swiglu"),     # padded batch 64, whole and shared tiles mixed
    (8192, 3584, 9, "resid"),       # TP-rank slice down projection
    (57344 // 4, 8192, 64, "swiglu"),
    (2048, 28672, 24, "plain"),
    (1280, 8192, 4, "plain"),       # batch <= 8 through the tcgen05 kernel (impl 2 only; otherwise the usual kernel)
    (3584, 2048, 7, "swiglu"),
])
def test_smallm_gemm_wide_batches(B, N, K, batch, mode, impl):
    B.set_decode_wide_impl(impl)
    try:
        W = _bf16((N, K), 21, 0.02)
        x = torch.randn(batch, K, generator=torch.Generator().manual_seed(22)).cuda()
        g = (torch.rand(K, generator=torch.Generator().manual_seed(23)) + 0.5).to(torch.bfloat16).cuda()
        w = _f64(W)
        if mode == "resid":
            addend = torch.randn(batch, N, generator=torch.Generator().manual_seed(24)).cuda()
            out = torch.full((batch, N), float("nan"), device="cuda")
            run = lambda o: B.op_smallm_gemm(W, x, 0, 0, o, addend=addend)
            ref = _f64(addend) + _f64(x) @ w.T
        elif mode == "plain":
            out = torch.full((batch, N), float("nan"), device="cuda")
            run = lambda o: B.op_smallm_gemm(W, x, 1, 2, o, gain=g, eps=1e-5)
            ref = O.rmsnorm(_f64(x), _f64(g), 1e-5) @ w.T
        else:
            out = torch.full((batch, N // 2), float("nan"), device="cuda")
            run = lambda o: B.op_smallm_gemm(W, x, 1, 1, o, gain=g, eps=1e-5)
            n = O.rmsnorm(_f64(x), _f64(g), 1e-5)
            ref = O.silu(n @ w[0::2].T) * (n @ w[1::2].T)
        run(out)
        again = torch.empty_like(out)
        run(again)
        torch.cuda.synchronize()
        tol = 2e-4
        if mode == "swiglu":
            tol *= 2.5
        assert rel_err(_f64(out), ref) < tol
        assert torch.equal(out, again)               # shared tiles are summed in a fixed order
    finally:
        B.set_decode_wide_impl(0)


def test_smallm_gemm_is_deterministic_and_batch_invariant(B):
    N, K = 2048, 4096
    W = _bf16((N, K), 9, 0.02)
    x = torch.randn(4, K, generator=torch.Generator().manual_seed(10)).cuda()
    g = torch.ones(K, dtype=torch.bfloat16, device="cuda")
    o1 = torch.empty(4, N, device="cuda")
    o2 = torch.empty(4, N, device="cuda")
    B.op_smallm_gemm(W, x, 1, 2, o1, gain=g)
    B.op_smallm_gemm(W, x, 1, 2, o2, gain=g)
    o3 = torch.empty(1, N, device="cuda")
    B.op_smallm_gemm(W, x[2:3].contiguous(), 1, 2, o3, gain=g)
    torch.cuda.synchronize()
    assert torch.equal(o1, o2)
    assert torch.equal(o1[2:3], o3)          # row b of a batch == the same row run alone


@pytest.mark.parametrize("batch,Hq,Hkv,Dh,max_seq,lens", [
    (1, 4, 4, 64, 32, [17]),
    (2, 16, 16, 128, 640, [513, 640]),
    (4, 64, 8, 128, 1536, [1025, 1300, 1536, 1]),
    (3, 32, 8, 128, 300, [0, 299, 37]),
    (2, 8, 1, 128, 2048, [2048, 2047]),
    (2, 6, 3, 64, 100, [100, 31]),
    # batch > 8: the probabilities-times-values product runs on the tensor cores (binary16 hi + lo probabilities)
    (12, 16, 2, 128, 300, [300, 1, 64, 65, 17, 128, 299, 0, 200, 77, 16, 255]),
    (9, 4, 4, 64, 130, [130, 129, 1, 64, 63, 65, 100, 2, 33]),
    (16, 8, 1, 128, 2048, [2048, 2047, 1025, 7] * 4),
    (10, 12, 3, 64, 96, [96, 95, 80, 64, 48, 32, 16, 8, 4, 1]),
])
def test_decode_attention(B, batch, Hq, Hkv, Dh, max_seq, lens):
    q = torch.randn(batch, Hq * Dh, generator=torch.Generator().manual_seed(11)).cuda()
    k = _f16((batch, Hkv, max_seq, Dh), 12, 1.0)          # the cache holds binary16 keys and values
    v = _f16((batch, Hkv, max_seq, Dh), 13, 1.0)
    kv_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scratch = torch.empty(B.decode_attention_scratch_bytes(batch, Hq, Dh, max_seq) // 4, device="cuda")
    o = torch.full((batch, Hq * Dh), float("nan"), device="cuda")
    for _ in range(2):                       # twice: the ticket counters must clean themselves up
        B.op_decode_attention(q, k, v, kv_len, Hq, Hkv, Dh, max_seq, scratch, o)
    torch.cuda.synchronize()
    got = _f64(o).reshape(batch, Hq, Dh)
    qb = _f64(q).reshape(batch, 1, Hq, Dh)
    for b in range(batch):
        L = lens[b]
        if L == 0:
            assert np.all(got[b] == 0.0)
            continue
        kk = _f64(k[b, :, :L]).transpose(1, 0, 2)
        vv = _f64(v[b, :, :L]).transpose(1, 0, 2)
        ref = O.causal_attention(qb[b], kk, vv, L - 1)[0]
        assert rel_err(got[b], ref) < 1e-3, b


@pytest.mark.parametrize("impl", [2, 1])          # 2 = TMA / tcgen05 kernel, 1 = register-fragment kernel
@pytest.mark.parametrize("batch,Hq,Hkv,Dh,max_seq,lens", [
    (16, 8, 1, 128, 2200, [2048, 2047, 1025, 7, 129, 128, 127, 1, 2200, 640, 0, 300, 1999, 64, 65, 256]),  # TP-rank slice
    (9, 32, 8, 128, 700, [700, 1, 129, 500, 0, 384, 385, 699, 256]),              # groups of 4 heads (8B shape)
    (10, 16, 16, 128, 300, [300, 299, 128, 1, 0, 257, 17, 200, 64, 130]),         # one query head per kv head
    (12, 32, 2, 128, 260, [260, 259, 131, 5, 128, 256, 1, 77, 190, 33, 12, 250]), # groups of 16 heads
    (64, 8, 1, 128, 1100, None),                                                  # more work items than SMs (a ring per CTA)
    (33, 64, 8, 128, 400, None),
    (64, 64, 8, 128, 1300, [1300 - (i % 3) for i in range(64)]),   # 70B shape: 35 tiles and four (sequence, kv head) groups per CTA
])
def test_decode_attention_wide_batches(B, batch, Hq, Hkv, Dh, max_seq, lens, impl):
    """Batch > 8 against the oracle, sequence by sequence: lengths that end inside, at the edge of and one past a
    128-key tile, empty sequences, cache rows beyond a sequence's length holding NaN (they must leave no trace)."""
    if lens is None:
        lens = [int(x) for x in np.random.default_rng(batch).integers(1, max_seq + 1, batch)]
        lens[0], lens[-1] = max_seq, 1
    q = torch.randn(batch, Hq * Dh, generator=torch.Generator().manual_seed(31)).cuda()
    k = _f16((batch, Hkv, max_seq, Dh), 32, 1.0)
    v = _f16((batch, Hkv, max_seq, Dh), 33, 1.0)
    for b in range(batch):
        k[b, :, lens[b]:] = float("nan")
        v[b, :, lens[b]:] = float("nan")
    kv_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scratch = torch.full((B.decode_attention_scratch_bytes(batch, Hq, Dh, max_seq) // 4,), float("nan"), device="cuda")
    o = torch.full((batch, Hq * Dh), float("nan"), device="cuda")
    B.set_decode_attention_impl(impl)
    try:
        B.op_decode_attention(q, k, v, kv_len, Hq, Hkv, Dh, max_seq, scratch, o)
        first = o.clone()
        B.op_decode_attention(q, k, v, kv_len, Hq, Hkv, Dh, max_seq, scratch, o)
        torch.cuda.synchronize()
    finally:
        B.set_decode_attention_impl(0)
    assert torch.equal(first, o)                     # partials are merged in a fixed order
    got = _f64(o).reshape(batch, Hq, Dh)
    qb = _f64(q).reshape(batch, 1, Hq, Dh)
    for b in range(batch):
        L = lens[b]
        if L == 0:
            assert np.all(got[b] == 0.0)
            continue
        ref = O.causal_attention(qb[b], _f64(k[b, :, :L]).transpose(1, 0, 2), _f64(v[b, :, :L]).transpose(1, 0, 2), L - 1)[0]
        assert rel_err(got[b], ref) < 1e-3, b


def _split(shape, seed, std=1.0, dtype=torch.bfloat16):
    """fp32 values and their 16-bit hi / lo parts (value ~ hi + lo)."""
    f = torch.randn(shape, generator=torch.Generator().manual_seed(seed)) * std
    hi = f.to(dtype)
    lo = (f - hi.float()).to(dtype)
    return f.cuda(), hi.cuda(), lo.cuda()


@pytest.mark.parametrize("split", [False, True])
@pytest.mark.parametrize("M,N,K,mode", [(16, 768, 256, 3), (300, 1376, 256, 1), (512, 256, 688, 0),
                                        (1000, 520, 264, 2), (4096, 1024, 1024, 0), (384, 2056, 8192, 2),
                                        # enough 128 x 256 tiles for every SM (wide tiles); the others use 128 x 128
                                        (2048, 2560, 512, 1), (2500, 2312, 320, 0)])
def test_prefill_gemm(B, M, N, K, mode, split):
    Af, A, A_lo = _split((M, K), 14)
    W = _bf16((N, K), 15, 0.05)
    acc = (_f64(Af) if split else _f64(A)) @ _f64(W).T
    lo_in = A_lo if split else None
    out_lo = None
    if mode == 0:
        addend = torch.randn(M, N, generator=torch.Generator().manual_seed(16)).cuda()
        out = torch.empty_like(addend)
        B.op_prefill_gemm(A, W, 0, out, addend=addend, A_lo=lo_in)
        ref = _f64(addend) + acc
    elif mode == 1:
        out = torch.empty(M, N // 2, dtype=torch.bfloat16, device="cuda")
        out_lo = torch.empty_like(out) if split else None
        B.op_prefill_gemm(A, W, 1, out, A_lo=lo_in, out_lo=out_lo)
        ref = O.silu(acc[:, 0::2]) * acc[:, 1::2]
    elif mode == 2:
        out = torch.empty(M, N, device="cuda")
        B.op_prefill_gemm(A, W, 2, out, A_lo=lo_in)
        ref = acc
    else:
        out = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
        out_lo = torch.empty_like(out) if split else None
        B.op_prefill_gemm(A, W, 3, out, A_lo=lo_in, out_lo=out_lo)
        ref = acc
    torch.cuda.synchronize()
    got = _f64(out) + (_f64(out_lo) if out_lo is not None else 0.0)
    # fp32 outputs / hi+lo outputs carry only accumulation error; a single bf16 output rounds at 2^-9
    tol = 2e-4 if (mode in (0, 2) or out_lo is not None) else 1e-2
    assert rel_err(got, ref) < tol


@pytest.mark.parametrize("impl", [0, 4])       # 0 = CTA pairs where tiles are plenty, 4 = one CTA per tile everywhere
@pytest.mark.parametrize("M,N,K,mode", [(16, 768, 256, 3), (300, 1376, 256, 1), (512, 256, 688, 0),
                                        (1000, 520, 264, 2), (4096, 1024, 1024, 0), (384, 2056, 8192, 2),
                                        (2048, 2560, 512, 1), (2500, 2312, 320, 0),
                                        # at least 74 tiles of 256 x 256: the CTA-pair kernel.  Ragged M and N (a pair's
                                        # second CTA partly or wholly outside), K not a multiple of 64, more tiles
                                        # than pairs (two accumulators in flight), a deep K (ring wraps many times)
                                        (4100, 4608, 200, 3), (2304, 2304 * 2, 4096, 1), (130 * 128, 1280, 576, 0),
                                        (1024, 19 * 256 + 8, 1024, 2)])
def test_prefill_gemm_binary16(B, M, N, K, mode, impl):
    """The prompt pass's default GEMM: binary16 activations (one value each) against bf16 weights converted to
    binary16 by the library's own conversion (exact but for magnitudes below 2^-14, which move by at most 2^-25)."""
    B.set_prefill_gemm_impl(impl)
    try:
        _prefill_gemm_binary16(B, M, N, K, mode)
    finally:
        B.set_prefill_gemm_impl(0)


def _prefill_gemm_binary16(B, M, N, K, mode):
    A = _f16((M, K), 24, 1.0)
    Wb = _bf16((N, K), 25, 0.05)
    W = torch.empty(N, K, dtype=torch.float16, device="cuda")
    B.op_convert_bf16_f16(Wb, W)
    torch.cuda.synchronize()
    assert torch.equal(W.view(torch.int16), Wb.float().to(torch.float16).view(torch.int16))   # round to nearest even
    assert float((W.float() - Wb.float()).abs().max()) <= 2.0 ** -25      # exact except below 2^-14 (subnormal grid)
    acc = _f64(A) @ _f64(Wb).T
    if mode == 0:
        addend = torch.randn(M, N, generator=torch.Generator().manual_seed(26)).cuda()
        out = torch.empty_like(addend)
        B.op_prefill_gemm_f16(A, W, 0, out, addend=addend)
        ref = _f64(addend) + acc
    elif mode == 1:
        out = torch.empty(M, N // 2, dtype=torch.float16, device="cuda")
        B.op_prefill_gemm_f16(A, W, 1, out)
        ref = O.silu(acc[:, 0::2]) * acc[:, 1::2]
    elif mode == 2:
        out = torch.empty(M, N, device="cuda")
        B.op_prefill_gemm_f16(A, W, 2, out)
        ref = acc
    else:
        out = torch.empty(M, N, dtype=torch.float16, device="cuda")
        B.op_prefill_gemm_f16(A, W, 3, out)
        ref = acc
    torch.cuda.synchronize()
    # fp32 outputs carry only accumulation error; a binary16 output rounds at 2^-12
    assert rel_err(_f64(out), ref) < (2e-4 if mode in (0, 2) else 1.5e-3)


def test_convert_bf16_to_binary16_small_magnitudes(B):
    """Below 2^-14 binary16 is subnormal: the conversion rounds to its 2^-24 grid (at most 2^-25 away), signed
    zeros and everything at or above 2^-14 pass unchanged."""
    vals = torch.tensor([0.0, -0.0, 2.0 ** -14, -(2.0 ** -14), 2.0 ** -15, 3 * 2.0 ** -20, 1.2345e-6, -7.7e-8, 1e-9,
                         0.02, -1.5, 255.0, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -25, 1.0], dtype=torch.float32)
    src = vals.to(torch.bfloat16).cuda()
    dst = torch.empty(16, dtype=torch.float16, device="cuda")
    B.op_convert_bf16_f16(src, dst)
    torch.cuda.synchronize()
    want = src.float().to(torch.float16)                         # the library conversion: round to nearest even
    assert torch.equal(dst.view(torch.int16), want.view(torch.int16))
    assert float((dst.float() - src.float()).abs().max()) <= 2.0 ** -25


@pytest.mark.parametrize("split", [False, True])
@pytest.mark.parametrize("batch,S,Hq,Hkv,Dh,max_seq", [(1, 16, 4, 4, 64, 32), (2, 200, 8, 2, 128, 256),
                                                       (1, 1024, 8, 1, 128, 1536), (2, 65, 6, 3, 64, 70),
                                                       (1, 128, 2, 1, 128, 128), (3, 385, 4, 2, 128, 385),
                                                       # more work items than SMs: a CTA walks several items, their
                                                       # key tiles forming one pipelined sequence
                                                       (4, 640, 32, 4, 128, 700), (2, 300, 80, 80, 64, 300)])
def test_prefill_attention(B, batch, S, Hq, Hkv, Dh, max_seq, split):
    qf, q, q_lo = _split((batch, S, Hq * Dh), 17, dtype=torch.float16)    # query, keys, values: binary16
    k = _f16((batch, Hkv, max_seq, Dh), 18, 1.0)
    v = _f16((batch, Hkv, max_seq, Dh), 19, 1.0)
    o = torch.full((batch, S, Hq * Dh), float("nan"), dtype=torch.bfloat16, device="cuda")
    o_lo = torch.zeros_like(o) if split else None
    B.op_prefill_attention(q, k, v, batch, S, Hq, Hkv, Dh, max_seq, o, q_lo=q_lo if split else None, o_lo=o_lo)
    torch.cuda.synchronize()
    got = _f64(o) + (_f64(o_lo) if split else 0.0)
    for b in range(batch):
        ref = O.causal_attention(_f64(qf[b] if split else q[b]).reshape(S, Hq, Dh),
                                 _f64(k[b, :, :S]).transpose(1, 0, 2), _f64(v[b, :, :S]).transpose(1, 0, 2), 0)
        # the probabilities enter the P.V MMA as single binary16 values (2^-12 relative each, averaged over keys);
        # without the lo parts the query (2^-12) and the single-bf16 output (2^-9) round as well
        assert rel_err(got[b].reshape(S, Hq, Dh), ref) < (1e-3 if split else 1e-2), b


@pytest.mark.parametrize("batch,S,Hq,Hkv,Dh,max_seq,pos0,lens", [
    (2, 96, 4, 2, 128, 512, 200, None),            # a chunk in the middle of a prompt; queries straddle key tiles
    (1, 300, 8, 8, 64, 1024, 724, None),           # the last chunk: the cache fills to its end
    (3, 260, 4, 1, 128, 300, 0, [260, 1, 129]),    # prompts of different lengths, padded to 260 rows
    (2, 130, 2, 2, 64, 400, 128, [5, 130]),        # both at once
])
def test_prefill_attention_offset_and_lengths(B, batch, S, Hq, Hkv, Dh, max_seq, pos0, lens):
    """Queries at positions pos0.. attend the pos0 rows already cached plus their own; padding rows are neither read
    nor written, and stale cache rows behind a sequence's own (here: NaN) leave no trace.  The output is the single
    binary16 value the binary16 output projection reads."""
    qf, q, q_lo = _split((batch, S, Hq * Dh), 27, dtype=torch.float16)
    k = _f16((batch, Hkv, max_seq, Dh), 28, 1.0)
    v = _f16((batch, Hkv, max_seq, Dh), 29, 1.0)
    lens_l = lens if lens is not None else [S] * batch
    for b in range(batch):                         # rows no sequence owns hold NaN
        k[b, :, pos0 + lens_l[b]:] = float("nan")
        v[b, :, pos0 + lens_l[b]:] = float("nan")
    canary = 777.0
    o = torch.full((batch, S, Hq * Dh), canary, dtype=torch.float16, device="cuda")
    d_lens = torch.tensor(lens, dtype=torch.int32, device="cuda") if lens is not None else None
    B.op_prefill_attention(q, k, v, batch, S, Hq, Hkv, Dh, max_seq, o, q_lo=q_lo, pos0=pos0, lens=d_lens,
                           out_binary16=True)
    torch.cuda.synchronize()
    got = _f64(o)
    for b in range(batch):
        n = lens_l[b]
        ref = O.causal_attention(_f64(qf[b, :n]).reshape(n, Hq, Dh), _f64(k[b, :, :pos0 + n]).transpose(1, 0, 2),
                                 _f64(v[b, :, :pos0 + n]).transpose(1, 0, 2), pos0)
        assert rel_err(got[b, :n].reshape(n, Hq, Dh), ref) < 2e-3, b      # binary16 output: 2^-12 per element
        assert np.all(got[b, n:] == canary), b                              # padding rows untouched


def _repeat_bitwise(torch_mod, launch, out, reps):
    """Launches `launch` `reps` times, every other time beside a copy kernel on a second stream, and counts the runs
    whose output differs from the first run's: the role pipelines of the tcgen05 kernels hand tiles over through
    mbarriers, and a protocol slip (a barrier phase arrived on twice, a ring slot rewritten early) shows up as a rare
    wrong tile rather than as a wrong formula."""
    side = torch_mod.cuda.Stream()
    big = torch_mod.randn(16 << 20, device="cuda")
    big2 = torch_mod.empty_like(big)
    launch()
    torch_mod.cuda.synchronize()
    ref = out.clone()
    assert not bool(torch_mod.isnan(ref.float()).any())
    bad = 0
    for rep in range(reps):
        out.fill_(float("nan"))
        if rep & 1:
            with torch_mod.cuda.stream(side):
                big2.copy_(big)
        launch()
        bad += 0 if torch_mod.equal(out, ref) else 1
    torch_mod.cuda.synchronize()
    return bad


def test_prefill_attention_many_launches_bitwise(B):
    """70B-shaped prompt-pass attention (2048 work items, 14 per CTA), 400 launches: all bit-identical."""
    bsz, S, Hq, Hkv, Dh, ms = 4, 1024, 64, 8, 128, 1100
    _, q, q_lo = _split((bsz, S, Hq * Dh), 41, dtype=torch.float16)
    k = _f16((bsz, Hkv, ms, Dh), 42, 1.0)
    v = _f16((bsz, Hkv, ms, Dh), 43, 1.0)
    k[:, :, S:] = float("nan")
    v[:, :, S:] = float("nan")
    o = torch.empty(bsz, S, Hq * Dh, dtype=torch.float16, device="cuda")
    launch = lambda: B.op_prefill_attention(q, k, v, bsz, S, Hq, Hkv, Dh, ms, o, q_lo=q_lo, out_binary16=True)
    assert _repeat_bitwise(torch, launch, o, 400) == 0


def test_decode_attention_tc_many_launches_bitwise(B):
    """Wide-batch decode attention on the TMA / tcgen05 kernel (35 tiles and four groups per CTA), 600 launches."""
    bsz, Hq, Hkv, Dh, ms = 64, 64, 8, 128, 1536
    q = torch.randn(bsz, Hq * Dh, generator=torch.Generator().manual_seed(51)).cuda()
    k = _f16((bsz, Hkv, ms, Dh), 52, 1.0)
    v = _f16((bsz, Hkv, ms, Dh), 53, 1.0)
    lens = [1280 - 7 * (i % 5) for i in range(bsz)]
    for b in range(bsz):
        k[b, :, lens[b]:] = float("nan")
        v[b, :, lens[b]:] = float("nan")
    kv_len = torch.tensor(lens, dtype=torch.int32, device="cuda")
    scratch = torch.empty(B.decode_attention_scratch_bytes(bsz, Hq, Dh, ms) // 4, device="cuda")
    o = torch.empty(bsz, Hq * Dh, device="cuda")
    B.set_decode_attention_impl(2)
    try:
        launch = lambda: B.op_decode_attention(q, k, v, kv_len, Hq, Hkv, Dh, ms, scratch, o)
        assert _repeat_bitwise(torch, launch, o, 600) == 0
    finally:
        B.set_decode_attention_impl(0)


def test_prefill_gemm_pairs_many_launches_bitwise(B):
    """The CTA-pair prompt-pass GEMM (cluster of two, 160 tiles over 74 pairs), 300 launches."""
    M, N, K = 2560, 4096, 1024
    A = _f16((M, K), 61, 1.0)
    W = _f16((N, K), 62, 0.05)
    addend = torch.randn(M, N, generator=torch.Generator().manual_seed(63)).cuda()
    out = torch.empty(M, N, device="cuda")
    launch = lambda: B.op_prefill_gemm_f16(A, W, 0, out, addend=addend)
    assert _repeat_bitwise(torch, launch, out, 300) == 0
