"""Host logic of the persistent decode kernel, checked without a GPU: the phase list the library builds
(ladder_stack_plan) against an independent model of which buffer every GEMM / attention node reads and
writes.  Every read-after-write, write-after-read and write-after-write pair between nodes of one launch
must be ordered by the dependency counters (directly or transitively), every dependency must point at a
node that comes earlier in the common phase order (so CTAs that walk the phases in order cannot deadlock),
and every phase's batch schedule must cover its 8-row units exactly once."""
import pytest

from paper_2501_06589_b200 import synth

QKV, GU, WO, DN, HEAD = 0, 1, 2, 3, 4


@pytest.fixture(scope="module")
def B():
    from paper_2501_06589_b200 import binding, build
    build.build()
    binding.lib()
    return binding


def module_flags(shape):
    """Per module (1-based m -> index m-1): does it read x_{m-2} instead of x_{m-1}?  From the layer modes as
    include/ladder.h states them, or the explicit table."""
    if shape.module_stale is not None:
        return [bool(f) for f in shape.module_stale]
    modes = list(shape.layer_mode) if shape.layer_mode is not None else \
        ["ladder" if v else "standard" for v in shape.ladder_mask()]
    flags = []
    for l, mode in enumerate(modes):
        if mode == "ladder":
            flags += [l == 0 or modes[l - 1] == "ladder", True]
        elif mode == "parallel":
            flags += [False, True]
        else:
            flags += [False, False]
    return flags


def routes(flags):
    """Which of the two residual buffers every module reads, adds onto and writes, from value liveness: the
    buffers hold stream values x_k; module m must find x_{m-1} (to add onto) and the value it reads, and x_m may
    only replace a value nobody needs any more -- x_{m-1} itself when module m read it and module m+1 will not,
    otherwise the other buffer (which holds x_{m-2} or nothing)."""
    holds = {0: 0, 1: None}
    out = []
    n = len(flags)
    for m in range(1, n + 1):
        newest = next(b for b, v in holds.items() if v == m - 1)
        want = m - 2 if (flags[m - 1] and m >= 2) else m - 1
        src = next(b for b, v in holds.items() if v == want)      # StopIteration = the value was destroyed
        next_reads_newest = m < n and flags[m]                    # module m+1 reads x_{m-1}
        dst = newest if (src == newest and not next_reads_newest) else newest ^ 1
        out.append((src, newest, dst))
        holds[dst] = m
    final = next(b for b, v in holds.items() if v == n)
    return [out[2 * l:2 * l + 2] for l in range(n // 2)], final


def expected_nodes(shape, first_layer):
    """Emission order of the launch with (name, act reads, epilogue reads, writes) per node."""
    flags = module_flags(shape)
    rt, final = routes(flags)
    nodes = []
    for l in range(first_layer, shape.n_layers):
        (a_in, a_add, a_dst), (m_in, m_add, m_dst) = rt[l]
        qkv = (("gemm", QKV, l), {f"R{a_in}"}, set(), {"q", f"K{l}", f"V{l}"})
        att = (("attn", l), {"q", f"K{l}", f"V{l}"}, set(), {"o"})
        wo = (("gemm", WO, l), {"o"}, {f"R{a_add}"}, {f"R{a_dst}"})
        gu = (("gemm", GU, l), {f"R{m_in}"}, set(), {"h"})
        dn = (("gemm", DN, l), {"h"}, {f"R{m_add}"}, {f"R{m_dst}"})
        independent = flags[2 * l + 1] and m_in != a_dst       # the MLP's input does not come from this layer's attention
        nodes += [qkv, att] + ([gu, wo] if independent else [wo, gu]) + [dn]
    nodes.append((("gemm", HEAD, shape.n_layers), {f"R{final}"}, set(), {"logits"}))
    return nodes


CASES = {
    "tiny_ladder": (synth.SHAPES["tiny"], 4),
    "tiny_hybrid_top": (synth.replace(synth.SHAPES["tiny"], layer_is_ladder=(0, 0, 1, 1)), 4),
    "tiny_mixed": (synth.replace(synth.SHAPES["tiny"], layer_is_ladder=(1, 1, 0, 1)), 3),
    "tiny_after_standard": (synth.replace(synth.SHAPES["tiny"], layer_is_ladder=(0, 1, 1, 1)), 2),
    "70b": (synth.SHAPES["70b"], 4),
    "8b_hybrid": (synth.SHAPES["8b_hybrid"], 4),
    "1p2b": (synth.SHAPES["1p2b"], 1),
    "tiny_parallel": (synth.SHAPES["tiny"].as_mode("parallel"), 4),
    "tiny_parallel_mixed": (synth.replace(synth.SHAPES["tiny"], layer_mode=("standard", "parallel", "ladder", "parallel")), 2),
    "tiny_explicit_flags": (synth.replace(synth.SHAPES["tiny"], layer_is_ladder=(0, 1, 1, 0),
                                          module_stale=(0, 0, 1, 1, 1, 1, 0, 0)), 3),
    "70b_parallel": (synth.SHAPES["70b"].as_mode("parallel"), 4),
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_plan_orders_every_hazard(B, case):
    shape, batch = CASES[case]
    plan = B.stack_plan(shape, batch, 256)
    assert plan["ok"]
    mask = shape.ladder_mask() if shape.layer_mode is None else [m == "ladder" for m in shape.layer_mode]
    first = shape.n_layers
    while first > 0 and mask[first - 1]:
        first -= 1
    if shape.layer_weight_bytes() < 300e6:       # small layers: standard ones run inside the launch too
        first = 0
    assert plan["first_layer"] == first
    if first == shape.n_layers:
        return                                   # top layer is standard: the launch is not used
    want = expected_nodes(shape, first)
    # ---- the library's nodes in emission order: attention node right after its layer's QKV phase
    got, attn_by_layer = [], {a["layer"]: a for a in plan["attn"]}
    for ph in plan["phases"]:
        got.append((("gemm", ph["kind"], ph["layer"]), ph))
        if ph["kind"] == QKV:
            got.append((("attn", ph["layer"]), attn_by_layer[ph["layer"]]))
    assert [g[0] for g in got] == [w[0] for w in want]
    # ---- counters: completion counter -> node index and the value that means "complete"
    done, total = {}, {}
    for i, (key, d) in enumerate(got):
        if key[0] == "gemm":
            done[d["done"]], total[d["done"]] = i, d["n_units"]
            assert d["n_units"] * 8 == d["N"]
        else:
            done[d["merge"]], total[d["merge"]] = i, batch * shape.n_q_heads
    early, late = [], []                         # per node: nodes it waits for before reading / before writing
    for i, (key, d) in enumerate(got):
        a = d["act_deps"] if key[0] == "gemm" else d["deps"]
        e = d["epi_deps"] if key[0] == "gemm" else d["merge_deps"]
        for ctr, need in a + e:
            assert ctr in done, f"{key}: waits on a counter that is not a completion counter"
            assert done[ctr] < i, f"{key}: waits on a later node (deadlock)"
            assert need == total[ctr], f"{key}: waits for {need}, producer completes at {total[ctr]}"
        early.append({done[c] for c, _ in a})
        late.append({done[c] for c, _ in a + e})
    # transitive closure: a node that is complete has itself waited for everything in late[]
    reach_early, reach_late = [], []
    closure = []
    for i in range(len(got)):
        def expand(seed):
            out = set()
            for j in seed:
                out |= {j} | closure[j]
            return out
        reach_early.append(expand(early[i]))
        reach_late.append(expand(late[i]))
        closure.append(reach_late[i])
    # ---- every hazard pair is ordered
    for j, (kj, act_r, epi_r, wr) in enumerate(want):
        for i in range(j):
            ki, act_i, epi_i, wr_i = want[i]
            if wr_i & act_r:
                assert i in reach_early[j], f"read-after-write {ki} -> {kj} (activation input) not ordered"
            if wr_i & epi_r:
                assert i in reach_late[j], f"read-after-write {ki} -> {kj} (epilogue input) not ordered"
            if (act_i | epi_i | wr_i) & wr:
                assert i in reach_late[j], f"write-after-read/write {ki} -> {kj} not ordered"


@pytest.mark.parametrize("case", ["70b", "8b_hybrid", "tiny_ladder", "1p2b"])
@pytest.mark.parametrize("grid", [148, 132, 7])
def test_schedule_covers_every_unit_once(B, case, grid):
    shape, batch = CASES[case]
    plan = B.stack_plan(shape, batch, 256, sm_count=grid)
    for ph in plan["phases"][:5] + plan["phases"][-1:]:
        n_units, rounds = ph["n_units"], ph["rounds"]
        assert ph["n_claims"] == sum(c for c, _ in rounds) and 0 <= ph["n_static"] <= ph["n_claims"]
        assert ph["n_static"] % grid == 0 or ph["n_static"] == ph["n_claims"]      # whole rounds of one claim per CTA
        covered, base = [], 0
        for count, size in rounds:
            assert 1 <= size <= 10               # a batch holds at most 5 MMA row groups of accumulators
            for ci in range(count):
                u0 = base + ci * size
                covered.append((u0, min(size, n_units - u0)))
            base += count * size
        units = [u for u0, nu in covered for u in range(u0, u0 + max(nu, 0))]
        assert units == list(range(n_units)), f"{case} kind {ph['kind']}: units not covered exactly once"
