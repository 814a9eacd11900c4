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


def routes(mask):
    """Residual routing of Eq. 1 / Eq. 2 on two buffers, re-derived here: per module (in, add, dst)."""
    cur, stale, out = 0, -1, []
    for lad in mask:
        per_layer = []
        for _ in range(2):                      # attention module, MLP module
            if lad and stale >= 0:              # x_m = x_{m-1} + h(x_{m-2}), overwriting x_{m-2}
                r = (stale, cur, stale)
                cur, stale = stale, cur
            elif lad:                           # first ladder module after a standard one
                r = (cur, cur, cur ^ 1)
                stale, cur = cur, cur ^ 1
            else:                               # x_m = x_{m-1} + h(x_{m-1}) in place
                r = (cur, cur, cur)
                stale = -1
            per_layer.append(r)
        out.append(per_layer)
    return out, cur


def expected_nodes(shape, first_layer):
    """Emission order of the launch with (name, act reads, epilogue reads, writes) per node."""
    mask = shape.ladder_mask()
    rt, final = routes(mask)
    nodes = []
    for l in range(first_layer, shape.n_layers):
        (a_in, a_add, a_dst), (m_in, m_add, m_dst) = rt[l]
        qkv = (("gemm", QKV, l), {f"R{a_in}"}, set(), {"q", f"K{l}", f"V{l}"})
        att = (("attn", l), {"q", f"K{l}", f"V{l}"}, set(), {"o"})
        wo = (("gemm", WO, l), {"o"}, {f"R{a_add}"}, {f"R{a_dst}"})
        gu = (("gemm", GU, l), {f"R{m_in}"}, set(), {"h"})
        dn = (("gemm", DN, l), {"h"}, {f"R{m_add}"}, {f"R{m_dst}"})
        independent = bool(mask[l]) and m_in != a_dst
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
}


@pytest.mark.parametrize("case", sorted(CASES))
def test_plan_orders_every_hazard(B, case):
    shape, batch = CASES[case]
    plan = B.stack_plan(shape, batch, 256)
    assert plan["ok"]
    mask = shape.ladder_mask()
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
