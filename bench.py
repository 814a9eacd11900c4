#!/usr/bin/env python
"""Benchmark of the Ladder-Residual decode path on B200: decode tokens/s and the fraction of
the HBM roofline, 70B shape, batch 4, 1024-token prompts, 512 decode steps (paper Sec. 3.3.1
workload; seeded synthetic weights and tokens).

A *step* is one autoregressive decode step of the whole model over the batch (embedding,
80 x [RMSNorm+QKV+RoPE+KV append, split-KV attention, output projection + ladder add,
RMSNorm+gate/up+SwiGLU, down projection + ladder add], final norm, LM head, argmax), replayed
as one CUDA graph with the token fed back on the device.  The prompt pass runs before the
timed region and is reported separately as `prefill`.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 70b] [--impl reference]

N > 1 runs N independent replicas (one process per GPU under torch.distributed; no data-path
collective: the path does not shard) and reports the aggregate.  Started without a launcher,
`--gpus N` starts the N ranks itself.  The K-step loop is timed `--repeats` times (default 3)
and the median is reported with every repeat's time and sampled SM clock.  At N = 1 the line also
carries short runs of the other benchmark configurations and of the paper's comparison
architectures (`other_configs`).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return float(j["hbm_gbs"]), float(j.get("bf16_tflops_sustained", j["bf16_tflops"])), "measured"
    return FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                pass
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}


def oracle_decode_sample(shape, weights, kv_len, n_layers_sample, dtype_name="float32"):
    """Time the CPU oracle on a bounded sample of one decode step: `n_layers_sample` layers of
    the stack at KV length `kv_len` plus the LM head; returns (seconds for the sample's layers,
    seconds for the head, threads).  The cache content is seeded noise (timing only)."""
    import numpy as np
    from oracle import ladder_oracle as O
    from paper_2501_06589_b200 import synth
    dt = getattr(np, dtype_name)
    sub = shape.with_layers(n_layers_sample)
    cfg = O.OracleConfig(sub.d_model, sub.n_layers, sub.n_q_heads, sub.n_kv_heads, sub.head_dim, sub.d_ff,
                         sub.vocab_size, sub.rms_eps, sub.rope_theta,
                         None if sub.layer_is_ladder is None else list(sub.layer_is_ladder),
                         layer_mode=None if sub.layer_mode is None else list(sub.layer_mode))
    prov = synth.logical_provider(weights, dt)
    W = O.OracleWeights(provider=prov)
    for l in range(n_layers_sample):                       # widen the sample's weights outside the timed part
        for nm in ("attn_norm", "mlp_norm", "wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down"):
            W.get(nm, l)
    for nm in ("tok_embedding", "final_norm", "lm_head"):
        W.get(nm)
    B = shape.batch
    cache = O.OracleCache(cfg, B, kv_len + 1, dt)
    rng = np.random.default_rng(7)
    cache.k[:, :, :kv_len] = rng.standard_normal(cache.k[:, :, :kv_len].shape, dtype=np.float32).astype(dt)
    cache.v[:, :, :kv_len] = rng.standard_normal(cache.v[:, :, :kv_len].shape, dtype=np.float32).astype(dt)
    cache.seq_len = kv_len
    toks = synth.make_tokens(shape, B, 1)[:, 0]
    t0 = time.perf_counter()
    x = O.embed(W, toks.reshape(-1, 1), dt)
    x = O.run_layers(cfg, W, x, kv_len, cache)
    t1 = time.perf_counter()
    O.head(cfg, W, x)
    t2 = time.perf_counter()
    try:
        from threadpoolctl import threadpool_info
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    return t1 - t0, t2 - t1, threads


def cpu_baseline(shape, weights, kv_len):
    n_sample = min(2, shape.n_layers)
    t_layers, t_head, threads = oracle_decode_sample(shape, weights, kv_len, n_sample)
    t_step = t_layers * (shape.n_layers / n_sample) + t_head
    return {"value": shape.batch / t_step, "unit": "tokens/s", "cores": threads, "kind": "oracle",
            "sample": (f"one decode step at KV length {kv_len}, batch {shape.batch}: {n_sample} of {shape.n_layers} "
                       f"layers ({t_layers:.2f} s) + LM head ({t_head:.2f} s) in float32, layer time extrapolated "
                       f"x{shape.n_layers / n_sample:g}")}


def run_reference(args):
    """--impl reference: the CPU oracle as it stands, timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import torch
    from paper_2501_06589_b200 import synth
    shape = shape_for(args, synth)
    n_sample = min(2, shape.n_layers)
    w = synth.make_weights(shape.with_layers(n_sample), device="cpu")
    kv_len = shape.prompt_len
    times = []
    t_start = time.perf_counter()
    for i in range(args.warmup + args.steps):
        t_layers, t_head, threads = oracle_decode_sample(shape, w, kv_len, n_sample)
        if i >= args.warmup:
            times.append(t_layers * (shape.n_layers / n_sample) + t_head)
        if times and time.perf_counter() - t_start > 60.0:      # keep the whole run within a few minutes
            break
    t = statistics.mean(times)
    sample = (f"per step: one decode step at KV length {kv_len}, batch {shape.batch}, {n_sample} of {shape.n_layers} "
              f"layers + LM head in float32, layer time extrapolated x{shape.n_layers / n_sample:g}; "
              f"{len(times)} of {args.steps} steps sampled (60 s cap)")
    val = shape.batch / t
    line = {"impl": "reference", "metric": "decode_tokens_per_s", "value": val, "unit": "tokens/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": workload_config(shape, args),
            "cpu_baseline": {"value": val, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))
    return 0


def residual_rule(shape):
    if shape.layer_mode is not None:
        kinds = sorted(set(shape.layer_mode))
        return f"all {kinds[0]}" if len(kinds) == 1 else "mixed " + "/".join(kinds)
    if shape.layer_is_ladder is None:
        return "all ladder"
    return "all standard" if not any(shape.layer_is_ladder) else "hybrid mask"


def workload_config(shape, args):
    return {"workload": f"{shape.name}: d_model {shape.d_model}, {shape.n_layers} layers "
                        f"({residual_rule(shape)}), "
                        f"{shape.n_q_heads}q/{shape.n_kv_heads}kv heads x {shape.head_dim}, ffn {shape.d_ff}, "
                        f"vocab {shape.vocab_size}",
            "batch": shape.batch, "prompt_len": shape.prompt_len, "decode_steps": args.steps,
            "prefill_chunk": getattr(args, "prefill_chunk", 0) or shape.prompt_len,
            "l2": "inputs larger than L2 (every step streams all weights, far above 126 MB)",
            "parallelism": (f"tensor parallel x{args.gpus} (this line's shape is one rank's slice)" if getattr(args, "tp", False)
                            else f"replicas x{args.gpus}" if args.gpus > 1 else "single GPU")}


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=512)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--repeats", type=int, default=3,
                    help="the K-step timed loop is run this many times; the median is reported")
    ap.add_argument("--config", default="70b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--streams", type=int, default=None)
    ap.add_argument("--graph", type=int, default=None)
    ap.add_argument("--pdl", type=int, default=None)
    ap.add_argument("--batch", type=int, default=None, help="sequences decoded together (default: the configuration's)")
    ap.add_argument("--wide-impl", type=int, default=0,
                    help="decode GEMM kernels: 0 = default, 2 = tcgen05 for every batch")
    ap.add_argument("--standard", action="store_true", help="the same shape with standard residuals (Eq. 1) in every layer")
    ap.add_argument("--mode", default=None, choices=["ladder", "standard", "parallel", "upper_bound"],
                    help="every layer in this architecture (paper Sec. 3.3.1) instead of the configuration's own")
    ap.add_argument("--multi-kernel", action="store_true",
                    help="one kernel per GEMM (two streams, CUDA graph, PDL) instead of the persistent decode kernel")
    ap.add_argument("--sm-split", type=int, default=None,
                    help="one kernel per GEMM: SMs for the attention module's GEMMs, the rest for the MLP's "
                         "(-2 = every GEMM on all SMs, -1 = the library's choice, 0 = by bytes)")
    ap.add_argument("--tp", action="store_true",
                    help="tensor parallelism over the --gpus ranks (Sec. 2, Eq. 1): every rank holds its slice of the "
                         "configuration and the modules' partial sums are all-reduced over NCCL; one model, so the "
                         "value is batch x steps / time (strong scaling).  With one GPU: a world of one")
    ap.add_argument("--tp-nccl", action="store_true",
                    help="with --tp: NCCL for the decode-step exchanges too (default: the library's own kernel over "
                         "peer memory for decode steps, NCCL for the prompt pass)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-prefill-timing", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short runs of the other benchmark configurations appended to the line at N = 1")
    ap.add_argument("--prefill-chunk", type=int, default=0,
                    help="feed the prompt in chunks of this many tokens per sequence (ladder_prefill_append): the prompt-pass "
                         "workspace then holds one chunk, which is what lets batch 64 of the 70B shape fit beside 141 GB of weights")
    ap.add_argument("--prefill-impl", type=int, default=0,
                    help="prompt-pass GEMMs: 0 = default; 2 = one bf16 per activation (not the precision the parity "
                         "bound is stated for); 3 = bf16 hi + lo pairs at every size")
    ap.add_argument("--selftest-cpu", action="store_true", help=argparse.SUPPRESS)
    return ap.parse_args(argv)


def spawn_ranks(args, argv):
    """`python bench.py --gpus N` outside a launcher: start N ranks (one per GPU) of this same script under
    torch.distributed.run on 127.0.0.1 and pass rank 0's JSON line through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.run(cmd).returncode


def selftest_cpu(args, rank, world):
    """Plumbing check without a GPU (tests only): gloo ranks, made-up per-rank timings, the real reduction."""
    import torch.distributed as dist
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = max_over_ranks([100.0 * (rank + 1)], dist, "cpu")[0]
    dist.barrier()
    if rank == 0:
        print(json.dumps({"selftest": True, "n_gpus": world, "ms": ms,
                          "value": aggregate_rate(world, 4, args.steps, ms)}))
    dist.destroy_process_group()
    return 0


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    args = parse_args(argv)
    world_env = os.environ.get("WORLD_SIZE")
    if args.gpus > 1 and world_env is None:
        return spawn_ranks(args, argv)
    rank = int(os.environ.get("RANK", "0"))
    world = int(world_env or "1")
    if world != args.gpus and rank == 0:      # the ranks that actually run are what the line reports as n_gpus
        sys.stderr.write(f"bench.py: --gpus {args.gpus} but the launcher started {world} ranks; reporting {world}\n")
    if args.selftest_cpu:
        return selftest_cpu(args, rank, world)
    if args.impl == "reference":
        return run_reference(args)
    return run_rank(args, rank, world)


def shape_for(args, synth):
    shape = synth.SHAPES[args.config]
    if args.batch:
        shape = synth.replace(shape, batch=args.batch)
    if args.standard:
        shape = shape.as_standard()
    if args.mode:
        shape = shape.as_mode(args.mode)
    return shape


class DecodeRun:
    """One model + cache ready to decode from a fixed position; times K-step loops on the device."""

    def __init__(self, B, torch, synth, shape, weights, steps, warm, args, dist, local, noise_kv=False):
        self.B, self.torch, self.shape, self.dist, self.local = B, torch, shape, dist, local
        self.steps, self.warm = steps, warm
        S, bsz = shape.prompt_len, shape.batch
        self.S, self.bsz = S, bsz
        max_seq = S + max(steps, warm) + 1
        chunk = args.prefill_chunk if 0 < args.prefill_chunk < S else S
        if noise_kv:
            chunk = 16
        self.chunk = chunk
        w = weights if weights.shape is shape else synth.replace(weights, shape=shape)
        self.model = B.Model(w, bsz, max_seq, bsz * chunk)
        if args.multi_kernel:
            self.model.set_persistent(False)
        if getattr(args, "sm_split", None) is not None:
            self.model.set_sm_split(args.sm_split)
        self.persistent = self.model.persistent_active() and bsz <= 8
        if args.streams is not None or args.graph is not None or args.pdl is not None:
            self.model.set_schedule(2 if args.streams is None else args.streams, 1 if args.graph is None else args.graph,
                                    1 if args.pdl is None else args.pdl)
        self.cache = B.KVCache(shape, bsz, max_seq)
        self.prompt = torch.from_numpy(synth.make_tokens(shape, bsz, S)).cuda()
        self.nxt = torch.zeros(bsz, dtype=torch.int32, device="cuda")
        self.first = torch.zeros(bsz, dtype=torch.int32, device="cuda")
        self.noise_kv = noise_kv
        if noise_kv:     # timing only: a cache of seeded noise instead of a prompt pass over S tokens
            g = torch.Generator(device="cuda")
            g.manual_seed(11)
            for t in (self.cache.k, self.cache.v):
                for s0 in range(0, t.numel(), 1 << 27):
                    t[s0:s0 + (1 << 27)].normal_(0.0, 0.5, generator=g)
            self.first.copy_(self.prompt[:, 0])

    def sync_all(self):
        self.torch.cuda.synchronize()
        if self.dist:
            self.dist.barrier()
            self.torch.cuda.synchronize()

    def prefill(self):
        m, c = self.model, self.chunk
        m.prefill(self.cache, self.prompt[:, :c].contiguous(), next_tokens=self.first)
        for p0 in range(c, self.S, c):
            m.prefill_append(self.cache, self.prompt[:, p0:min(self.S, p0 + c)].contiguous(), next_tokens=self.first)

    def rewind(self):
        self.cache.seq_lens.fill_(self.S)
        self.model.set_position(self.S)
        self.nxt.copy_(self.first)

    def timed_loop(self):
        """K decode steps, device-timed with events on the launching stream; returns (ms, clock summary, launches)."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        self.rewind()
        self.sync_all()
        l0 = self.model.kernel_launches()
        with ClockSampler(self.local) as clocks:
            e0.record()
            for _ in range(self.steps):
                self.model.decode_step(self.cache, self.nxt, next_tokens=self.nxt)
            e1.record()
            self.sync_all()
        return e0.elapsed_time(e1), clocks.summary(), self.model.kernel_launches() - l0

    def warm_up(self):
        self.rewind()
        for _ in range(self.warm):
            self.model.decode_step(self.cache, self.nxt, next_tokens=self.nxt)

    def close(self):
        self.model.close()


def median_loop(run, repeats):
    """Runs the timed loop `repeats` times; returns (median ms over ranks' maxima, per-repeat records, launches)."""
    recs, launches = [], 0
    for _ in range(max(1, repeats)):
        ms, clk, launches = run.timed_loop()
        ms = max_over_ranks([ms], run.dist, "cuda")[0]
        recs.append({"ms": ms, "sm_mhz": clk["sm_mhz"], "reasons": clk["reasons"], "samples": clk["samples"]})
    return statistics.median(r["ms"] for r in recs), recs, launches


def merged_clocks(recs):
    mhz = [r["sm_mhz"] for r in recs if r["sm_mhz"] is not None]
    reasons = sorted({x for r in recs for x in r["reasons"]})
    return mhz, reasons


def short_run(B, torch, synth, shape, weights, args, local, steps=32, repeats=3, noise_kv=False, tp=None):
    """One of the other configurations: ms/step (median of `repeats` loops) and roofline fractions.
    tp = (comm, peer): the model as the one rank of a tensor-parallel world of one (exchange fused over peer memory)."""
    hbm_peak, _, _ = measured_peaks()
    run = DecodeRun(B, torch, synth, shape, weights, steps, 3, args, None, local, noise_kv=noise_kv)
    if tp is not None:
        run.model.set_tensor_parallel_peer(*tp)
        run.persistent = False
    if not noise_kv:
        run.prefill()
    run.warm_up()
    ms, recs, launches = median_loop(run, repeats)
    status = run.model.device_status()
    run.close()
    per = ms / steps
    step_bytes = shape.decode_step_bytes(shape.prompt_len + (steps + 1) / 2.0)
    gbs = step_bytes / (per * 1e-3) / 1e9
    mhz, reasons = merged_clocks(recs)
    return {"ms_per_step": round(per, 4), "tokens_per_s": round(shape.batch * steps / (ms * 1e-3), 1),
            "gb_per_step": round(step_bytes / 1e9, 3), "frac_of_8tbs": round(gbs / NOMINAL_HBM_GBS, 4),
            "frac_of_measured_copy_peak": round(gbs / hbm_peak, 4), "steps": steps,
            "repeat_ms": [round(r["ms"], 3) for r in recs], "sm_mhz": mhz, "reasons": reasons,
            "persistent": run.persistent, "launches_per_step": launches / steps, "device_status": status,
            "kv": "seeded noise" if noise_kv else "prompt pass"}


def other_configs(B, torch, synth, args, local, w70=None, shape70=None):
    """Short decode runs of the other benchmark configurations and of the comparison architectures of the
    paper's Sec. 3.3.1 (standard / parallel / ladder), so that one line carries them all."""
    out = {}
    if w70 is not None:      # the same 70B weights under the two other residual rules
        for mode in ("standard", "parallel"):
            out[f"70b_b{shape70.batch}_{mode}"] = short_run(B, torch, synth, shape70.as_mode(mode), w70, args, local)
        # the batch sweep of the paper's Sec. 3.3.1 at the full shape (decode steps from a 1024-token cache of seeded
        # noise: the prompt-pass workspace for 64 x 1024 tokens would not fit beside 141 GB of weights)
        for b in (1, 16, 32, 64):
            out[f"70b_b{b}_ladder"] = short_run(B, torch, synth, synth.replace(shape70, batch=b), w70, args, local,
                                                noise_kv=True)
    return out


def other_configs_small(B, torch, synth, args, local):
    out = {}
    for name in ("1p2b", "8b_hybrid"):
        shape = synth.SHAPES[name]
        w = synth.make_weights(shape, device="cuda")
        out[name] = short_run(B, torch, synth, shape, w, args, local)
        if name == "8b_hybrid":
            for mode in ("standard", "ladder", "parallel"):
                out[f"{name}_all_{mode}"] = short_run(B, torch, synth, shape.as_mode(mode), w, args, local)
        del w
        torch.cuda.empty_cache()
    base = synth.SHAPES["tp_slice"]
    w = synth.make_weights(base, device="cuda")
    for mode in ("ladder", "standard", "parallel"):
        for b in (1, 4, 16, 64):
            shape = synth.replace(base.as_mode(mode), batch=b)
            out[f"tp_slice_b{b}_{mode}"] = short_run(B, torch, synth, shape, w, args, local, noise_kv=True)
    # the same slice as the ONE rank of a tensor-parallel world (Sec. 2, Eq. 1; Algorithm 1): every module's output is
    # stored, exchanged (here with nobody: what the schedule and the fused exchange cost by themselves) and added by
    # the next reader
    try:      # (an extra: a machine without an NCCL library must not cost the rest of the line)
        from paper_2501_06589_b200 import tensor_parallel as TP
        comm = TP.make_comm()
        for mode in ("ladder", "standard", "parallel"):
            shape = synth.replace(base.as_mode(mode), batch=16)
            peer = TP.make_peer(16 * base.d_model)
            out[f"tp_slice_b16_{mode}_tensor_parallel_world1"] = short_run(B, torch, synth, shape, w, args, local,
                                                                          noise_kv=True, tp=(comm, peer))
            peer.close()
        comm.close()
    except Exception as e:      # noqa: BLE001
        out["tensor_parallel_world1_skipped"] = repr(e)[:200]
    del w
    torch.cuda.empty_cache()
    return out


def run_rank(args, rank, world):
    import numpy as np  # noqa: F401
    import torch
    from paper_2501_06589_b200 import binding as B
    from paper_2501_06589_b200 import build, synth

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if dist:
        dist.barrier()
    B.lib()

    shape = shape_for(args, synth)
    comm = None
    if args.tp:       # this rank's slice; timing only, so the slice is generated directly (same shapes, own seeds)
        from paper_2501_06589_b200 import tensor_parallel as TP
        shape = TP.rank_shape(shape, world)
        comm = TP.make_comm()
        peer = None if args.tp_nccl else TP.make_peer(shape.batch * shape.d_model)
    steps, warm = args.steps, max(args.warmup, 0)
    S, bsz = shape.prompt_len, shape.batch
    hbm_peak, bf16_peak, peak_src = measured_peaks()

    t0 = time.time()
    w = synth.make_weights(shape, device="cuda")
    torch.cuda.synchronize()
    t_gen = time.time() - t0
    B.set_decode_wide_impl(args.wide_impl)
    B.set_prefill_gemm_impl(args.prefill_impl)
    run = DecodeRun(B, torch, synth, shape, w, steps, warm, args, dist, local)
    model, cache = run.model, run.cache
    if comm is not None:
        if peer is not None:
            model.set_tensor_parallel_peer(comm, peer)
        else:
            model.set_tensor_parallel(comm)
        run.persistent = False
    persistent = run.persistent

    # ---- prefill: once untimed (warm-up), once timed
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    run.prefill()
    torch.cuda.synchronize()
    prefill_ms = None
    if not args.no_prefill_timing:
        ev[0].record()
        run.prefill()
        ev[1].record()
        torch.cuda.synchronize()
        prefill_ms = ev[0].elapsed_time(ev[1])

    # ---- decode: warm-up, then K timed steps (token fed back on the device, no host sync inside), `repeats` times
    run.warm_up()
    dev_ms, dev_recs, launches = median_loop(run, args.repeats)
    status = model.device_status()

    # ---- end to end: host token buffers in, host tokens out, every step (pinned memory); same number of repeats
    h_in = run.first.cpu().pin_memory()
    h_out = torch.zeros(bsz, dtype=torch.int32).pin_memory()
    run.rewind()
    model.decode_step_host(cache, h_in, h_out)      # untimed: captures the graph for the staging buffers
    e2e_recs = []
    for _ in range(max(1, args.repeats)):
        run.rewind()
        h_in.copy_(run.first.cpu())
        run.sync_all()
        t0 = time.perf_counter()
        for _ in range(steps):
            model.decode_step_host(cache, h_in, h_out)
            h_in.copy_(h_out)
        torch.cuda.synchronize()
        e2e_recs.append(max_over_ranks([(time.perf_counter() - t0) * 1e3], dist, "cuda")[0])
    e2e_ms = statistics.median(e2e_recs)

    # ---- dominant kernel alone: the gate/up weight-streaming GEMM over every layer's weights, with the kernel the
    # steps above used for it (batch > 4, tensor parallelism, and slice-like all-ladder models at any batch: tcgen05)
    all_ladder = shape.layer_mode is None and shape.module_stale is None and all(shape.ladder_mask())
    slice_like = all_ladder and shape.layer_weight_bytes() < 300e6 and 4 * shape.n_q_heads * shape.head_dim <= shape.d_model
    step_used_tcgen05 = bsz > 4 or args.wide_impl == 2 or args.tp or (
        not persistent and slice_like and args.sm_split is None and args.streams in (None, 2))
    if step_used_tcgen05:
        B.set_decode_wide_impl(2)
    x_act = torch.randn(bsz, shape.d_model, device="cuda")
    h_out_buf = torch.empty(bsz, shape.d_ff, device="cuda")
    n_l = shape.n_layers
    for l in range(min(3, n_l)):
        B.op_smallm_gemm(w.w_gate_up[l], x_act, 1, 1, h_out_buf, gain=w.mlp_norm[l], eps=shape.rms_eps)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for l in range(n_l):
        B.op_smallm_gemm(w.w_gate_up[l], x_act, 1, 1, h_out_buf, gain=w.mlp_norm[l], eps=shape.rms_eps)
    e1.record()
    torch.cuda.synchronize()
    B.set_decode_wide_impl(args.wide_impl)
    k_ms = e0.elapsed_time(e1) / n_l
    k_bytes = 2.0 * 2 * shape.d_ff * shape.d_model
    k_gbs = k_bytes / (k_ms * 1e-3) / 1e9

    prefill_ms_max = max_over_ranks([prefill_ms or 0.0], dist, "cuda")[0]
    ms_per_step = dev_ms / steps
    jobs = 1 if args.tp else world          # tensor parallelism: ONE model over all ranks
    value = aggregate_rate(jobs, bsz, steps, dev_ms)
    e2e_value = aggregate_rate(jobs, bsz, steps, e2e_ms)
    mean_kv = S + (steps + 1) / 2.0
    step_bytes = shape.decode_step_bytes(mean_kv)
    step_gbs = step_bytes / (ms_per_step * 1e-3) / 1e9
    mhz, reasons = merged_clocks(dev_recs)
    sm_max = None
    with ClockSampler(local) as probe:      # the clock limit itself (idle sample)
        time.sleep(0.5)
    sm_max = probe.summary()["sm_max_mhz"]

    traffic = ncu_traffic()
    line = {
        "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": steps,
        "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if args.tp else "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": workload_config(shape, args),
        "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": 4 * bsz, "d2h_bytes_per_step": 4 * bsz,
                "repeat_ms": [round(x, 3) for x in e2e_recs]},
        "gpu_launches": int(launches),
        "repeats": {"n": len(dev_recs), "statistic": "median", "ms": [round(r["ms"], 3) for r in dev_recs],
                    "sm_mhz": [r["sm_mhz"] for r in dev_recs]},
        "roofline": {"bound": "hbm", "kernel": ("decode_gemm_wide_tc (tcgen05; " if step_used_tcgen05 else "smallm_gemm (") +
                               "RMSNorm + gate/up projection + SwiGLU)",
                     "achieved": k_gbs, "peak": hbm_peak, "peak_source": peak_src, "unit": "GB/s",
                     "frac": k_gbs / hbm_peak, "bytes_per_launch": k_bytes, "ms_per_launch": k_ms,
                     "traffic": traffic.get((shape.name, bsz, "decode_gemm_gate_up_bytes"))},
        "step_roofline": {"bytes_per_step": step_bytes, "achieved_gbs": step_gbs,
                          "frac_of_measured_copy_peak": step_gbs / hbm_peak,
                          "frac_of_nominal_8tbs": step_gbs / NOMINAL_HBM_GBS, "mean_kv_len": mean_kv},
        "clocks": {"sm_mhz": statistics.median(mhz) if mhz else None, "sm_max_mhz": sm_max, "reasons": reasons,
                   "samples": sum(r["samples"] for r in dev_recs)},
        "device_status": status,
        "schedule": {"persistent": persistent, "streams": args.streams, "graph": args.graph, "pdl": args.pdl},
        "weights_gb": w.nbytes() / 1e9, "weight_gen_s": t_gen,
    }
    if args.tp:
        line["tensor_parallel"] = {"world": world,
                                   "exchange": "all-reduce of fp32 [rows, d_model] partial sums, one per module, on the "
                                               "producing module's stream (decode) / a stream of its own (prompt pass)",
                                   "decode": "NCCL" if peer is None else "fused into the GEMM epilogues and the staging launches over peer memory",
                                   "prompt_pass": "NCCL"}
    if prefill_ms_max:
        flops = prefill_flops(shape, bsz, S)
        line["prefill"] = {"tokens_per_s": jobs * bsz * S / (prefill_ms_max * 1e-3), "ms": prefill_ms_max,
                           "tflops": flops / (prefill_ms_max * 1e-3) / 1e12,
                           "frac_of_bf16_peak": flops / (prefill_ms_max * 1e-3) / 1e12 / bf16_peak,
                           "impl": args.prefill_impl,
                           "peak_tflops": bf16_peak, "peak_source": peak_src}
    if persistent:
        # One launch of the persistent kernel IS the decode step (the embedding gather, the counter reset
        # and the argmax around it take ~10 us), so the step's device time is its launch duration.
        line["gemm_kernel"] = line["roofline"]
        ratio = traffic.get((shape.name, bsz, "decode_stack_traffic_ratio"))
        line["roofline"] = {
            "bound": "hbm", "kernel": "decode_stack_kernel (every GEMM and the attention of a decode step, one launch)",
            "achieved": step_gbs, "peak": hbm_peak, "peak_source": peak_src, "unit": "GB/s",
            "frac": step_gbs / hbm_peak, "bytes_per_launch": step_bytes, "ms_per_launch": ms_per_step,
            "traffic": None if ratio is None else step_bytes * ratio}
    solo = rank == 0 and world == 1
    if solo and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(shape, w, S)
    run.close()
    del run, model, cache
    if comm is not None:
        if peer is not None:
            peer.close()
        comm.close()
    if solo and not args.no_other_configs and args.config == "70b" and args.mode is None and not args.standard and not args.tp:
        t0 = time.time()
        others = {}
        try:      # the headline above is measured already: a failure here must not lose it
            others.update(other_configs(B, torch, synth, args, local, w, shape))
            del w
            torch.cuda.empty_cache()
            others.update(other_configs_small(B, torch, synth, args, local))
        except Exception as e:      # noqa: BLE001
            line["other_configs_error"] = repr(e)[:300]
        line["other_configs"] = others
        line["other_configs_s"] = round(time.time() - t0, 1)
    if rank == 0:
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()
    return 0


def ncu_traffic():
    """DRAM traffic figures taken from ncu captures (dram__bytes_read.sum + dram__bytes_write.sum), kept as data
    beside the capture summaries: lines of `config batch key value`."""
    out = {}
    path = os.path.join(ROOT, "profiles", "ncu_traffic.txt")
    if os.path.exists(path):
        for ln in open(path):
            f = ln.split()
            if len(f) == 4 and not ln.startswith("#"):
                out[(f[0], int(f[1]), f[2])] = float(f[3])
    return out


def max_over_ranks(values, dist, device):
    """Element-wise maximum of per-rank timings over the process group (replicas: no data-path collective)."""
    import torch
    t = torch.tensor(values, device=device, dtype=torch.float64)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def aggregate_rate(world, batch, steps, ms_max):
    """Whole-job tokens/s of `world` independent replicas, each doing batch x steps tokens in ms_max."""
    return world * batch * steps / (ms_max * 1e-3)


def prefill_flops(shape, bsz, S):
    d, F = shape.d_model, shape.d_ff
    per_tok_layer = 2 * (shape.qkv_rows * d + d * shape.n_q_heads * shape.head_dim + 3 * F * d)
    attn = 2 * 2 * shape.n_q_heads * shape.head_dim * (S * (S + 1) / 2)       # QK^T and PV, causal
    return shape.n_layers * (bsz * S * per_tok_layer + bsz * attn) + 2 * bsz * shape.vocab_size * d


if __name__ == "__main__":
    sys.exit(main())
