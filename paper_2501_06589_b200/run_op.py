"""Run ONE kernel of the decode path at a model's true shape, a few launches in a row -- the
small, self-ending workload to put under `ncu` (or to time with CUDA events).

    python -m paper_2501_06589_b200.run_op gate_up --config 70b --layers 2 --iters 2

ops: qkv, wo, gate_up, down, lm_head (weight-streaming GEMMs), attn (split-KV decode attention),
     prefill_gemm, prefill_attn, stack (whole decode steps of a model cut to --layers layers: the
     persistent layer-stack kernel, or with --multi-kernel the per-GEMM schedule).  Each launch uses a different layer's weights, so nothing is
     served from L2.  Prints one line with the mean time per launch and the achieved GB/s or TFLOP/s.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as B
from . import build, synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("op")
    ap.add_argument("--config", default="70b")
    ap.add_argument("--layers", type=int, default=2, help="distinct weight sets to allocate")
    ap.add_argument("--iters", type=int, default=2, help="passes over the layers")
    ap.add_argument("--batch", type=int, default=None)
    ap.add_argument("--kv-len", type=int, default=None)
    ap.add_argument("--tokens", type=int, default=4096, help="M of the prefill GEMM")
    ap.add_argument("--multi-kernel", action="store_true", help="stack: use the per-GEMM schedule")
    ap.add_argument("--wide-impl", type=int, default=0,
                    help="decode GEMM: 0 = default, 2 = tcgen05 kernel for every batch")
    ap.add_argument("--persistent-all", action="store_true", help="stack: standard layers in the persistent kernel too")
    ap.add_argument("--standard", action="store_true", help="stack: standard residuals in every layer")
    ap.add_argument("--which", default="gate_up", choices=["qkv", "wo", "gate_up", "down"],
                    help="prefill_gemm: which projection's shape and epilogue")
    ap.add_argument("--pairs", action="store_true",
                    help="prefill_gemm: bf16 hi + lo activation pairs instead of the default binary16 operands")
    ap.add_argument("--prefill-impl", type=int, default=0,
                    help="prefill_gemm: 4 = one CTA per tile everywhere (no CTA pairs)")
    ap.add_argument("--attn-impl", type=int, default=0,
                    help="attn, stack: 1 = the register-fragment decode attention kernel at every batch, 2 = the TMA / tcgen05 kernel for every batch > 8")
    ap.add_argument("--sm-split", type=int, default=-1,
                    help="stack (one kernel per GEMM): SMs for the attention module's GEMMs, the rest for the MLP's (0 = by bytes)")
    ap.add_argument("--tp", action="store_true",
                    help="stack: as the one rank of a tensor-parallel world (pending-output form, fused exchange)")
    ap.add_argument("--no-lo", action="store_true", help="prefill_attn: queries and outputs without their lo parts")
    ap.add_argument("--seq", type=int, default=None, help="prefill_attn: tokens per sequence")
    a = ap.parse_args()
    build.build()
    B.lib()
    B.set_decode_wide_impl(a.wide_impl)
    B.set_prefill_gemm_impl(a.prefill_impl)
    B.set_decode_attention_impl(a.attn_impl)
    s = synth.SHAPES[a.config]
    bsz = a.batch or s.batch
    d, F, Hq, Hkv, Dh, V = s.d_model, s.d_ff, s.n_q_heads, s.n_kv_heads, s.head_dim, s.vocab_size
    L = a.layers
    dev = "cuda"

    if a.op == "stack":
        return run_stack(a, s, bsz)

    def w(rows, cols):
        return [(torch.randn(rows, cols, device=dev) * 0.02).to(torch.bfloat16) for _ in range(L)]

    x = torch.randn(bsz, d, device=dev)
    gain = torch.ones(d, dtype=torch.bfloat16, device=dev)
    if a.op == "qkv":
        W, out = w(s.qkv_rows, d), torch.empty(bsz, s.qkv_rows, device=dev)
        fn, nbytes, flops = (lambda l: B.op_smallm_gemm(W[l], x, 1, 2, out, gain=gain)), 2 * s.qkv_rows * d, 0
    elif a.op == "wo":
        W, xin, add, out = w(d, Hq * Dh), torch.randn(bsz, Hq * Dh, device=dev), torch.randn(bsz, d, device=dev), torch.empty(bsz, d, device=dev)
        fn, nbytes, flops = (lambda l: B.op_smallm_gemm(W[l], xin, 0, 0, out, addend=add)), 2 * d * Hq * Dh, 0
    elif a.op == "gate_up":
        W, out = w(2 * F, d), torch.empty(bsz, F, device=dev)
        fn, nbytes, flops = (lambda l: B.op_smallm_gemm(W[l], x, 1, 1, out, gain=gain)), 4 * F * d, 0
    elif a.op == "down":
        W, xin, add, out = w(d, F), torch.randn(bsz, F, device=dev), torch.randn(bsz, d, device=dev), torch.empty(bsz, d, device=dev)
        fn, nbytes, flops = (lambda l: B.op_smallm_gemm(W[l], xin, 0, 0, out, addend=add)), 2 * d * F, 0
    elif a.op == "lm_head":
        W, out = w(V, d), torch.empty(bsz, V, device=dev)
        fn, nbytes, flops = (lambda l: B.op_smallm_gemm(W[l], x, 1, 2, out, gain=gain)), 2 * V * d, 0
    elif a.op == "attn":
        max_seq = s.prompt_len + s.decode_steps
        kv = a.kv_len or (s.prompt_len + s.decode_steps // 2)
        q = torch.randn(bsz, Hq * Dh, device=dev)
        k = [torch.randn(bsz, Hkv, max_seq, Dh, device=dev).to(torch.float16) for _ in range(L)]
        v = [torch.randn(bsz, Hkv, max_seq, Dh, device=dev).to(torch.float16) for _ in range(L)]
        lens = torch.full((bsz,), kv, dtype=torch.int32, device=dev)
        scr = torch.empty(B.decode_attention_scratch_bytes(bsz, Hq, Dh, max_seq) // 4, device=dev)
        o = torch.empty(bsz, Hq * Dh, device=dev)
        fn = lambda l: B.op_decode_attention(q, k[l], v[l], lens, Hq, Hkv, Dh, max_seq, scr, o)
        nbytes, flops = 2 * 2 * bsz * Hkv * kv * Dh, 0
    elif a.op == "convert":          # one layer's gate/up weights bf16 -> binary16 (what the prompt pass does per layer)
        W = w(2 * F, d)
        dst = torch.empty(2 * F, d, dtype=torch.float16, device=dev)
        fn = lambda l: B.op_convert_bf16_f16(W[l], dst)
        nbytes, flops = 2 * 2 * 2 * F * d, 0
    elif a.op == "prefill_gemm" and not a.pairs:
        M = a.tokens
        N, K, mode = {"gate_up": (2 * F, d, 1), "qkv": (s.qkv_rows, d, 3), "wo": (d, Hq * Dh, 0), "down": (d, F, 0)}[a.which]
        A = torch.randn(M, K, device=dev).to(torch.float16)
        W = [t.to(torch.float16) for t in w(N, K)]
        add = torch.randn(M, N, device=dev) if mode == 0 else None
        out = torch.empty(M, N, device=dev) if mode == 0 else \
            torch.empty(M, N // 2 if mode == 1 else N, dtype=torch.float16, device=dev)
        fn = lambda l: B.op_prefill_gemm_f16(A, W[l], mode, out, addend=add)
        nbytes, flops = 0, 2.0 * M * N * K
    elif a.op == "prefill_gemm":
        M = a.tokens
        A = (torch.randn(M, d, device=dev)).to(torch.bfloat16)
        A_lo = (torch.randn(M, d, device=dev) * 1e-3).to(torch.bfloat16)
        W, out = w(2 * F, d), torch.empty(M, F, dtype=torch.bfloat16, device=dev)
        out_lo = torch.empty_like(out)
        fn = lambda l: B.op_prefill_gemm(A, W[l], 1, out, A_lo=A_lo, out_lo=out_lo)
        nbytes, flops = 0, 2.0 * M * 2 * F * d
        if a.which != "gate_up":     # QKV without its rotary / cache epilogue (plain bf16 store); Wo and down add a residual
            N, K, mode = {"qkv": (s.qkv_rows, d, 3), "wo": (d, Hq * Dh, 0), "down": (d, F, 0)}[a.which]
            A = torch.randn(M, K, device=dev).to(torch.bfloat16)
            A_lo = (torch.randn(M, K, device=dev) * 1e-3).to(torch.bfloat16)
            W = w(N, K)
            add = torch.randn(M, N, device=dev)
            out = torch.empty(M, N, device=dev) if mode == 0 else torch.empty(M, N, dtype=torch.bfloat16, device=dev)
            out_lo = None if mode == 0 else torch.empty_like(out)
            fn = lambda l: B.op_prefill_gemm(A, W[l], mode, out, addend=add if mode == 0 else None, A_lo=A_lo, out_lo=out_lo)
            flops = 2.0 * M * N * K
    elif a.op == "prefill_attn":
        S = a.seq or s.prompt_len
        q = torch.randn(bsz, S, Hq * Dh, device=dev).to(torch.float16)
        q_lo = (torch.randn(bsz, S, Hq * Dh, device=dev) * 1e-3).to(torch.float16)
        k = [torch.randn(bsz, Hkv, S, Dh, device=dev).to(torch.float16) for _ in range(L)]
        v = [torch.randn(bsz, Hkv, S, Dh, device=dev).to(torch.float16) for _ in range(L)]
        o = torch.empty_like(q)
        o_lo = torch.empty_like(q)
        if a.no_lo:
            q_lo = o_lo = None
        fn = lambda l: B.op_prefill_attention(q, k[l], v[l], bsz, S, Hq, Hkv, Dh, S, o, q_lo=q_lo, o_lo=o_lo)
        nbytes, flops = 0, 4.0 * bsz * Hq * Dh * S * (S + 1) / 2
    else:
        raise SystemExit(f"unknown op {a.op}")

    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for l in range(L):          # warm-up pass
        fn(l)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(a.iters):
        for l in range(L):
            fn(l)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / (a.iters * L)
    rate = f"{nbytes / ms / 1e6:.0f} GB/s" if nbytes else f"{flops / ms / 1e9:.1f} TFLOP/s"
    print(f"{a.op} [{a.config}, batch {bsz}]: {ms * 1e3:.2f} us per launch, {rate}")


def run_stack(a, s, bsz):
    """Decode steps of the model cut to a.layers layers, KV length from the configuration."""
    s = synth.replace(s, n_layers=a.layers, layer_is_ladder=None if s.layer_is_ladder is None
                      else tuple(s.layer_is_ladder[:a.layers]))
    if a.standard:
        s = s.as_standard()
    w = synth.make_weights(s, device="cuda")
    S = a.kv_len or s.prompt_len
    steps = a.iters + 3
    model = B.Model(w, bsz, S + steps + 1, bsz * min(S, 256))
    if a.multi_kernel:
        model.set_persistent(False)
    if a.persistent_all:
        model.set_persistent(2)
    if a.sm_split != -1:
        model.set_sm_split(a.sm_split)
    if a.tp:      # the one rank of a tensor-parallel world: exchange fused over peer memory (with nobody)
        from . import tensor_parallel as TP
        comm, peer = TP.make_comm(), TP.make_peer(bsz * s.d_model)
        model.set_tensor_parallel_peer(comm, peer)
    persistent = model.persistent_active() and bsz <= 8 and not a.tp
    cache = B.KVCache(s, bsz, S + steps + 1)
    cache.k.normal_()                                 # a synthetic prefix instead of a prompt pass
    cache.v.normal_()
    cache.seq_lens.fill_(S)
    model.set_position(S)
    nxt = torch.from_numpy(synth.make_tokens(s, bsz, 1)[:, 0].copy()).cuda()
    for _ in range(3):
        model.decode_step(cache, nxt, next_tokens=nxt)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        model.decode_step(cache, nxt, next_tokens=nxt)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    nbytes = s.decode_step_bytes(S + 3 + a.iters // 2, bsz)
    print(f"stack [{a.config}, {a.layers} layers, batch {bsz}, kv {S}, "
          f"{'persistent' if persistent else 'one kernel per GEMM'}]: {ms * 1e3:.1f} us per step, "
          f"{nbytes / ms / 1e6:.0f} GB/s, status {model.device_status()}")
    model.close()


if __name__ == "__main__":
    main()
