"""Host-side tests of the C-ABI library (no GPU): exports, error paths, and bit-exact agreement of
the planner (Algorithms 1-4) with the oracle's step-by-step versions."""
import ctypes

import numpy as np
import pytest

from oracle import arena as OA
from oracle import planner as OP
from paper_2411_09242_b200 import fluid, synth
from tests.helpers import ensure_lib, header_symbols, plan_records, random_dag, table_eval


@pytest.fixture(scope="module", autouse=True)
def _lib():
    return ensure_lib()


def test_library_exports_every_declared_symbol():
    L = fluid.lib()
    names = header_symbols()
    assert len(names) >= 24 and "fluid_plan" in names and "fluid_run" in names
    for n in names:
        assert hasattr(L, n), n
    assert set(names) == set(fluid._SIGNATURES)


def test_graph_error_paths():
    g = fluid.fluid_graph_create()
    with pytest.raises(fluid.FluidError) as e:
        fluid.fluid_graph_add_tensor(g, 7, [4, 4], synth.ACT)
    assert e.value.code == fluid.FLUID_EINVAL
    with pytest.raises(fluid.FluidError):
        fluid.fluid_graph_add_tensor(g, synth.F32, [4, 0], synth.ACT)
    a = fluid.fluid_graph_add_tensor(g, synth.F32, [4, 8], synth.INPUT)
    w = fluid.fluid_graph_add_tensor(g, synth.F32, [7, 3], synth.CONST)
    y = fluid.fluid_graph_add_tensor(g, synth.F32, [4, 3], synth.OUTPUT)
    with pytest.raises(fluid.FluidError):                   # K mismatch
        fluid.fluid_graph_add_op(g, synth.LINEAR, [a, w], [y], {"contract": 1})
    with pytest.raises(fluid.FluidError):                   # bad tensor id
        fluid.fluid_graph_add_op(g, synth.GELU, [99], [y])
    with pytest.raises(fluid.FluidError):                   # writing an input
        fluid.fluid_graph_add_op(g, synth.GELU, [y], [a])
    with pytest.raises(fluid.FluidError):                   # empty graph
        fluid.fluid_plan(g)
    fluid.fluid_graph_destroy(g)


def test_bad_candidates_are_rejected():
    d = random_dag(0, 3)
    g = fluid.graph_from_desc(d)
    c = synth.canonical_candidates(d)
    c[1] = [(1, 0)]                                          # first candidate must be the identity
    with pytest.raises(fluid.FluidError):
        fluid.fluid_plan(g, c)
    c[1] = [(0, 1), (1, 1)]                                  # not a permutation
    with pytest.raises(fluid.FluidError):
        fluid.fluid_plan(g, c)
    fluid.fluid_graph_destroy(g)


def _oracle_inputs(d, cands):
    ops = [{"ins": o["ins"], "outs": o["outs"]} for o in d.ops]
    ncand = {}
    for t, td in enumerate(d.tensors):
        pinned = td["kind"] in (synth.INPUT, synth.OUTPUT)
        ncand[t] = 1 if pinned else len(cands[t])
    consts = {t for t, td in enumerate(d.tensors) if td["kind"] == synth.CONST}
    return ops, ncand, consts


@pytest.mark.parametrize("seed", range(12))
def test_sequences_and_layouts_match_the_oracle_bit_for_bit(seed):
    d = random_dag(seed, n_ops=6 + seed % 7)
    cands = synth.default_candidates(d)
    ops, ncand, consts = _oracle_inputs(d, cands)
    ev = table_eval(seed)

    def c_eval(user, node, n, tids, lidx):
        return ev(node, {tids[i]: lidx[i] for i in range(n)})

    plan = fluid.Plan(d, cands, eval=fluid.EVAL_FN(c_eval))
    want, cost, seqs = OP.plan_layouts(ops, ncand, ev, consts)
    assert plan.sequences() == seqs
    got = {t: plan.tensor_info(t).layout_index for t in range(len(d.tensors))}
    assert got == want
    assert plan.cost == cost
    assert plan.canonical_cost == OP.total_cost(ops, {t: 0 for t in ncand}, ev)
    plan.close()


@pytest.mark.parametrize("name", ["tiny", "bert_base", "gpt2_small", "llama"])
def test_model_graph_sequences_match_oracle(name):
    m = synth.build_model(synth.scaled(synth.CONFIGS[name], L=2), materialize=False)
    d = m.graph
    plan = fluid.Plan(d, synth.canonical_candidates(d), fusion=0)
    ops, _, consts = _oracle_inputs(d, synth.canonical_candidates(d))
    seqs = OP.split(OP.Flow(ops, consts))
    assert plan.sequences() == seqs
    assert sorted(o for s in seqs for o in s) == list(range(len(d.ops)))
    plan.close()


@pytest.mark.parametrize("name", ["tiny", "bert_base", "gpt2_small", "llama"])
@pytest.mark.parametrize("policy", [0, 1])
def test_arena_matches_greedy_by_size_oracle(name, policy):
    cfg = synth.CONFIGS[name]
    m = synth.build_model(synth.scaled(cfg, L=min(cfg.L, 3)), materialize=False)
    plan = fluid.Plan(m.graph, synth.default_candidates(m.graph), arena_policy=policy, split_k=policy)
    recs, offs = plan_records(plan)
    assert len(recs) > 5
    want, peak = OA.greedy_by_size(recs, policy="best" if policy else "first")
    assert offs == want and plan.arena_bytes == peak
    assert OA.check_arena(recs, offs, plan.arena_bytes) == []
    assert plan.live_bound_bytes == OA.live_set_bound(recs)
    assert plan.naive_bytes == OA.naive_sum(recs)
    assert plan.live_bound_bytes <= plan.arena_bytes <= plan.naive_bytes
    # lifetimes recomputed independently from the step list
    steps = plan.steps()
    nt = len(m.graph.tensors)
    for rid, _, first, last in recs:
        if rid >= 3 * nt:
            # the scratch of a split RMS normalisation: from the GEMM step that fills it to the next step, which
            # lists the normalisation among its ops and reads the scratch instead of the normalised tensor
            assert (first, last) in ((rid - 3 * nt, rid - 3 * nt + 1), (rid - 3 * nt - len(steps), rid - 3 * nt - len(steps) + 1))
            assert steps[first]["kernel_name"] == steps[last]["kernel_name"] == "GEMM_TC"
            assert any(m.graph.ops[o]["kind"] == synth.RMSNORM for o in steps[last]["ops"])
            continue
        if rid >= 2 * nt:
            assert first == last == rid - 2 * nt      # per-step scratch lives during its step only
            continue
        tid = rid % nt
        group = [t for t in range(nt) if plan.tensor_info(t).alias_of == tid]
        touched = [i for i, s in enumerate(steps) if set(group) & set(s["ins"] + s["outs"])]
        assert (first, last) == (min(touched), max(touched))
    plan.close()


@pytest.mark.parametrize("name", ["tiny", "bert_base", "gpt2_small", "llama"])
def test_arena_over_several_orders_is_valid_and_never_larger(name):
    """arena_policy 2 (not in the paper): Algorithm 4's placement over several record orders, the smallest arena kept.
    Checked with the independent validity checker; never above first or best fit in the paper's order; on the four
    model shapes it meets the largest live set."""
    cfg = synth.CONFIGS[name]
    m = synth.build_model(cfg, materialize=False)
    cands = synth.default_candidates(m.graph)
    sizes = {}
    for policy in (0, 1, 2):
        plan = fluid.Plan(m.graph, cands, arena_policy=policy)
        recs, offs = plan_records(plan)
        assert OA.check_arena(recs, offs, plan.arena_bytes) == []
        sizes[policy] = (plan.arena_bytes, plan.live_bound_bytes)
        plan.close()
    assert sizes[2][0] <= min(sizes[0][0], sizes[1][0])
    if name == "llama":
        # with the RMS normalisations split across their neighbouring GEMM steps the 16 MB operand of the readers
        # lives one step longer than the normalised tensor did; the packing that meets the largest live set then
        # alternates from layer to layer (found by placing the 43 MB products from the bottom and the top in turn):
        # 96.5 MB against 96.25 MB (no_norm_split = 1: 96 = 96)
        assert sizes[2][0] <= 1.005 * sizes[2][1]
        plan = fluid.Plan(m.graph, cands, arena_policy=2, no_norm_split=1)
        assert plan.arena_bytes == plan.live_bound_bytes
        plan.close()
    else:
        assert sizes[2][0] == sizes[2][1]


@pytest.mark.parametrize("seed", range(12))
def test_arena_over_several_orders_on_records_of_mixed_sizes(seed):
    """Random layered graphs whose tensors have a common width and a few odd, larger ones (what sets off the padded,
    alternating-ends placement of arena_policy 2): every policy's placement passes the independent checker, and the
    several-orders policy is never larger than first or best fit."""
    rng = np.random.default_rng(100 + seed)
    g = synth.GraphDesc()
    M, common = 64, 64
    x = g.tensor("in", synth.F32, [M, common], synth.INPUT)
    avail = [(x, common)]
    n_ops = 14 + seed % 5
    for i in range(n_ops):
        last = i == n_ops - 1
        kind = synth.OUTPUT if last else synth.ACT
        a, wa = avail[int(rng.integers(max(0, len(avail) - 4), len(avail)))]
        r = rng.random()
        same = [t for t in avail if t[1] == wa and t[0] != a]
        if r < 0.45:
            wb = common if rng.random() < 0.6 else int(rng.choice([112, 176, 200, 328]))
            w = g.tensor(f"w{i}", synth.F32, [wa, wb], synth.CONST)
            out = g.tensor(f"t{i}", synth.F32, [M, wb], kind)
            g.op(synth.LINEAR, [a, w], [out], contract=1)
            avail.append((out, wb))
        elif r < 0.75 and same:
            b, _ = same[int(rng.integers(len(same)))]
            out = g.tensor(f"t{i}", synth.F32, [M, wa], kind)
            g.op(synth.ADD, [a, b], [out])
            avail.append((out, wa))
        else:
            out = g.tensor(f"t{i}", synth.F32, [M, wa], kind)
            g.op(synth.GELU, [a], [out])
            avail.append((out, wa))
    sizes = {}
    for policy in (0, 1, 2):
        for extra in ({}, {"fusion": 0}):
            plan = fluid.Plan(g, None, arena_policy=policy, **extra)
            recs, offs = plan_records(plan)
            assert OA.check_arena(recs, offs, plan.arena_bytes) == []
            assert plan.live_bound_bytes <= plan.arena_bytes <= plan.naive_bytes
            sizes[(policy, bool(extra))] = plan.arena_bytes
            plan.close()
    for unfused in (False, True):
        assert sizes[(2, unfused)] <= min(sizes[(0, unfused)], sizes[(1, unfused)])


def test_no_reuse_plan_is_the_naive_sum():
    m = synth.build_model(synth.CONFIGS["tiny"], materialize=False)
    plan = fluid.Plan(m.graph, None, no_reuse=1)
    recs, offs = plan_records(plan)
    assert plan.arena_bytes == plan.naive_bytes == OA.naive_sum(recs)
    spans = sorted((offs[r[0]], offs[r[0]] + r[1]) for r in recs)
    assert all(a[1] <= b[0] for a, b in zip(spans, spans[1:]))
    plan.close()


@pytest.mark.parametrize("name", ["tiny", "bert_base", "gpt2_small", "llama"])
def test_planned_layouts_elide_every_transpose(name):
    cfg = synth.CONFIGS[name]
    m = synth.build_model(synth.scaled(cfg, L=2), materialize=False)
    d = m.graph
    cands = synth.default_candidates(d)
    plan = fluid.Plan(d, cands)
    canon = fluid.Plan(d, None)
    assert plan.cost <= plan.canonical_cost == pytest.approx(canon.cost)
    kinds = [s["kernel_name"] for s in plan.steps()]
    assert "PERMUTE" not in kinds
    assert [s["kernel_name"] for s in canon.steps()].count("PERMUTE") == 4 * 2 + (0 if name != "gpt2_small" else 1)
    for t in range(len(d.tensors)):
        info = plan.tensor_info(t)
        assert info.perm in [tuple(c) for c in cands[t]]
        if d.tensors[t]["kind"] in (synth.INPUT, synth.OUTPUT):
            assert info.layout_index == 0
    # every op of the graph is covered by exactly one step or is an elided transpose
    covered = sorted(o for s in plan.steps() for o in s["ops"])
    elided = [i for i, o in enumerate(d.ops) if o["kind"] == synth.TRANSPOSE]
    assert sorted(covered + elided) == list(range(len(d.ops)))
    # layout planning optimises time; it must not cost memory beyond what keeping head tensors alive as views needs
    assert plan.arena_bytes <= 1.15 * canon.arena_bytes
    plan.close(); canon.close()


def test_fusion_folds_epilogues():
    m = synth.build_model(synth.scaled(synth.CONFIGS["bert_base"], L=1), materialize=False)
    fused = fluid.Plan(m.graph, None)
    plain = fluid.Plan(m.graph, None, fusion=0)
    assert fluid.fluid_plan_num_steps(plain.handle) == len(m.graph.ops)
    names = lambda p: [s["kernel_name"] for s in p.steps()]
    assert names(plain).count("ELTWISE") == 3 and names(fused).count("ELTWISE") == 0
    gelu_steps = [s for s in fused.steps() if len(s["ops"]) == 3]        # LINEAR + GELU? no: LINEAR+ADD pairs
    assert all(len(s["ops"]) <= 3 for s in fused.steps())
    assert fused.arena_bytes <= plain.arena_bytes
    fused.close(); plain.close()


def test_sibling_projections_share_one_launch():
    m = synth.build_model(synth.scaled(synth.CONFIGS["bert_base"], L=1), materialize=False)
    plan = fluid.Plan(m.graph, synth.default_candidates(m.graph))
    grouped = [s for s in plan.steps() if s["kernel_name"] == "GEMM_TC" and ((s["variant"] >> 20) & 15) == 3]
    assert len(grouped) == 1 and len(grouped[0]["outs"]) == 3 and len(grouped[0]["ops"]) == 3
    names = {m.graph.tensors[t]["name"] for t in grouped[0]["outs"]}
    assert names == {"l0.q", "l0.k", "l0.v"}
    # the three outputs are alive from that step on and keep separate slices
    offs = {plan.tensor_info(t).offset for t in grouped[0]["outs"]}
    assert len(offs) == 3 and all(o >= fluid.ARENA_HEADER for o in offs)
    ll = synth.build_model(synth.scaled(synth.CONFIGS["llama"], L=1), materialize=False)
    lp = fluid.Plan(ll.graph, synth.default_candidates(ll.graph))
    groups = sorted(((s["variant"] >> 20) & 15) for s in lp.steps() if s["kernel_name"] == "GEMM_TC" and ((s["variant"] >> 20) & 15))
    assert groups == [2, 3]                      # gate/up and q/k/v
    # the gate/up launch also applies SiLU(gate) * up and runs the second half of the RMS normalisation in front of
    # it (the o-proj step did the first half): five graph ops, one output, no slice for the normalised tensor, gate or up
    fused = [s for s in lp.steps() if s["kernel_name"] == "GEMM_TC" and any(ll.graph.ops[o]["kind"] == synth.SILU for o in s["ops"])]
    assert len(fused) == 1 and len(fused[0]["outs"]) == 1 and len(fused[0]["ops"]) == 5
    kinds = sorted(ll.graph.ops[o]["kind"] for o in fused[0]["ops"])
    assert kinds == sorted([synth.RMSNORM, synth.LINEAR, synth.LINEAR, synth.SILU, synth.MUL])
    assert ll.graph.ops[fused[0]["ops"][0]]["kind"] == synth.RMSNORM     # listed first: the GEMMs read its result
    apart = fluid.Plan(ll.graph, synth.default_candidates(ll.graph), no_norm_split=1)
    four = [s for s in apart.steps() if s["kernel_name"] == "GEMM_TC" and any(ll.graph.ops[o]["kind"] == synth.SILU for o in s["ops"])]
    assert len(four) == 1 and len(four[0]["ops"]) == 4 and len(apart.steps()) == len(lp.steps()) + 1
    apart.close()
    unfused = fluid.Plan(ll.graph, synth.default_candidates(ll.graph), fusion=0)
    assert all(((s["variant"] >> 20) & 15) == 0 for s in unfused.steps())
    plan.close(); lp.close(); unfused.close()


def test_residual_stream_is_held_in_fp32():
    m = synth.build_model(synth.scaled(synth.CONFIGS["gpt2_small"], L=2), materialize=False)
    d = m.graph
    plan = fluid.Plan(d, synth.default_candidates(d))
    holder = {r["tensor"]: r for r in plan.records() if not r["twin"]}
    by_name = {td["name"]: holder.get(plan.tensor_info(t).alias_of) for t, td in enumerate(d.tensors)}
    assert by_name["embed"]["dtype"] == synth.F32 and by_name["l0.res1"]["dtype"] == synth.F32
    assert by_name["l0.ln1.out"]["dtype"] == synth.BF16          # feeds GEMMs only
    assert not any(r["twin"] for r in plan.records())            # pre-LN: no tensor needs both
    narrow = fluid.Plan(d, synth.default_candidates(d), narrow_stream=1)
    assert all(r["dtype"] == synth.BF16 for r in narrow.records())
    enc = synth.build_model(synth.scaled(synth.CONFIGS["bert_base"], L=1), materialize=False)
    ep = fluid.Plan(enc.graph, synth.default_candidates(enc.graph))
    twins = {enc.graph.tensors[r["tensor"]]["name"] for r in ep.records() if r["twin"]}
    assert "emb_ln.out" in twins and "l0.ln1.out" in twins       # post-LN: stream value also feeds GEMMs
    plan.close(); narrow.close(); ep.close()


def test_attention_chain_becomes_one_step_and_frees_the_score_tensors():
    for name, arena_cap_mb in [("gpt2_small", 60), ("llama", 200)]:
        m = synth.build_model(synth.CONFIGS[name], materialize=False)
        d = m.graph
        fused = fluid.Plan(d, synth.default_candidates(d))
        unfused = fluid.Plan(d, synth.default_candidates(d), unfused_attention=1)
        attn = [s for s in fused.steps() if s["kernel_name"] == "ATTN"]
        assert len(attn) == m.cfg.L and all(len(s["ops"]) == 3 for s in attn)
        assert [d.ops[o]["kind"] for o in attn[0]["ops"]] == [synth.BMM_QK, synth.SOFTMAX, synth.BMM_PV]
        assert "SOFTMAX" not in [s["kernel_name"] for s in fused.steps()]
        assert "ATTN" not in [s["kernel_name"] for s in unfused.steps()]
        # scores and probabilities no longer exist as arena slices
        names = {d.tensors[r["tensor"]]["name"] for r in fused.records()}
        assert not any(n.endswith("scores") or n.endswith("probs") for n in names)
        assert fused.arena_bytes < arena_cap_mb * 2 ** 20 < unfused.arena_bytes
        recs, offs = plan_records(fused)
        assert OA.check_arena(recs, offs, fused.arena_bytes) == []
        fused.close(); unfused.close()
    # head dims the tensor-core attention kernel does not take stay unfused
    t = synth.build_model(synth.scaled(synth.CONFIGS["bert_base"], L=1, H=96, nh=2), materialize=False)   # D = 48
    p = fluid.Plan(t.graph, synth.default_candidates(t.graph))
    assert "ATTN" not in [s["kernel_name"] for s in p.steps()] and "SOFTMAX" in [s["kernel_name"] for s in p.steps()]
    p.close()


def test_split_k_takes_a_step_lifetime_scratch_slice():
    m = synth.build_model(synth.scaled(synth.CONFIGS["bert_base"], L=1), materialize=False)
    d = m.graph
    off = fluid.Plan(d, synth.default_candidates(d))
    on = fluid.Plan(d, synth.default_candidates(d), split_k=1)
    assert not any(r["tensor"] < 0 for r in off.records())
    scratch = [r for r in on.records() if r["tensor"] < 0]
    # bit 28 marks a cut that runs inside a thread-block cluster: it needs no scratch
    split_steps = [i for i, s in enumerate(on.steps())
                   if s["kernel_name"] == "GEMM_TC" and ((s["variant"] >> 24) & 15) > 1 and not (s["variant"] >> 28) & 1]
    assert len(scratch) == len(split_steps) >= 1
    assert any((s["variant"] >> 28) & 1 for s in off.steps())
    never = fluid.Plan(d, synth.default_candidates(d), split_k=-1)
    assert all((s["variant"] >> 24) == 0 for s in never.steps() if s["kernel_name"] == "GEMM_TC")
    never.close()
    assert sorted(r["first"] for r in scratch) == split_steps and all(r["first"] == r["last"] for r in scratch)
    recs, offs = plan_records(on)
    assert OA.check_arena(recs, offs, on.arena_bytes) == []
    assert on.arena_bytes >= off.arena_bytes
    off.close(); on.close()


def test_a_cost_function_that_picks_unrunnable_layouts_gives_a_plan_that_refuses_to_run():
    """The caller's eval may rate as cheap a combination no kernel can run (here: a softmax whose input and
    output sit in different, non-row-contiguous layouts). The plan is still returned, for inspection, and
    fluid_run refuses it before any device work."""
    ensure_lib()
    g = synth.GraphDesc()
    BF = synth.BF16
    x = g.tensor("x", BF, [2, 3, 16, 16], synth.INPUT)
    a = g.tensor("a", BF, [2, 3, 16, 16])
    b = g.tensor("b", BF, [2, 3, 16, 16])
    y = g.tensor("y", BF, [2, 3, 16, 16], synth.OUTPUT)
    g.op(synth.TRANSPOSE, [x], [a], perm=[0, 1, 2, 3])
    sm = g.op(synth.SOFTMAX, [a], [b], causal=0, scale=1.0)
    g.op(synth.TRANSPOSE, [b], [y], perm=[0, 1, 2, 3])
    cands = synth.default_candidates(g)
    assert len(cands[a]) == 6

    def ev(user, node, n, tids, lidx):
        if node != sm:
            return 1.0
        want = {a: 5, b: 2}
        return 0.0 if all(lidx[i] == want[tids[i]] for i in range(n)) else 100.0

    plan = fluid.Plan(g, cands, eval=fluid.EVAL_FN(ev))
    assert plan.tensor_info(a).layout_index == 5 and plan.tensor_info(b).layout_index == 2
    assert len(plan.steps()) >= 1 and plan.arena_bytes > 0
    with pytest.raises(fluid.FluidError) as e:
        fluid.fluid_run(plan.handle, 0x10000, [0x20000], [0x30000])
    assert e.value.code == fluid.FLUID_EUNSUPPORTED and "no kernel runs" in str(e.value)
    plan.close()


def test_decoding_graph_plans_without_a_gpu():
    """Host logic of the decoding workload: state tensors stay outside the arena and among the inputs, the rotary ops
    and SwiGLU fold into their consumers, every LINEAR of a few rows takes the weight-streaming kernel."""
    cfg = synth.scaled(synth.CONFIGS["llama"], S=1, L=2, B=4)
    dec = synth.build_decode_model(cfg, 2048, materialize=False)
    g = dec.graph
    plan = fluid.Plan(g, synth.default_candidates(g))
    names = [s["kernel_name"] for s in plan.steps()]
    # per layer: RMSNorm + Q/K/V, attention (+ rotary), O + residual, RMSNorm + gate/up + SwiGLU, down + residual
    assert names == ["EMBED"] + ["GEMM_ROWS", "ATTN_DECODE", "GEMM_ROWS", "GEMM_ROWS", "GEMM_ROWS"] * 2 + ["NORM", "GEMM_ROWS"]
    normed = [s for s in plan.steps() if s["kernel_name"] == "GEMM_ROWS" and (s["variant"] >> 30) & 1]
    assert len(normed) == 4 and all(synth.RMSNORM in [g.ops[o]["kind"] for o in s["ops"]] for s in normed)
    att = [s for s in plan.steps() if s["kernel_name"] == "ATTN_DECODE"]
    assert all(len(s["ops"]) == 3 and (s["variant"] >> 16) & 1 for s in att)            # attention + two ROPE ops
    fused = [s for s in plan.steps() if s["kernel_name"] == "GEMM_ROWS" and len(s["ops"]) == 5]
    assert len(fused) == 2 and all(len(s["outs"]) == 1 for s in fused)                   # RMSNorm, gate, up, SiLU, MUL
    for kc, vc in dec.caches:
        for t in (kc, vc):
            info = plan.tensor_info(t)
            assert info.offset < 0 and info.layout_index == 0
    assert g.inputs == [dec.ids, dec.pos] + [t for pair in dec.caches for t in pair]
    assert plan.arena_bytes < 2 ** 20                                                     # a few [B,1,.] rows
    unfused = fluid.Plan(g, synth.default_candidates(g), fusion=0)
    un = [s["kernel_name"] for s in unfused.steps()]
    assert un.count("ROPE") == 4 and un.count("ATTN_DECODE") == 2
    simt = fluid.Plan(g, synth.default_candidates(g), gemm_path=1)
    assert "GEMM_ROWS" not in [s["kernel_name"] for s in simt.steps()]
    for p in (plan, unfused, simt):
        p.close()
    # the GPT-family step: LayerNorm folds into the few-row GEMMs as well (its bias as one more activation row)
    gcfg = synth.scaled(synth.CONFIGS["gpt2_small"], S=1, L=2, B=4)
    gdec = synth.build_decode_model(gcfg, 1024, materialize=False)
    gplan = fluid.Plan(gdec.graph, synth.default_candidates(gdec.graph))
    gnames = [s["kernel_name"] for s in gplan.steps()]
    assert gnames[0] == "EMBED" and gnames[1:11] == ["GEMM_ROWS", "ATTN_DECODE", "GEMM_ROWS", "GEMM_ROWS", "GEMM_ROWS"] * 2
    assert sum((s["variant"] >> 30) & 1 for s in gplan.steps() if s["kernel_name"] == "GEMM_ROWS") == 4
    gplan.close()


def test_state_tensors_and_cached_attention_are_checked():
    def base():
        g = synth.GraphDesc()
        q = g.tensor("q", synth.BF16, [2, 1, 4, 64], synth.INPUT)
        k = g.tensor("k", synth.BF16, [2, 1, 2, 64], synth.INPUT)
        v = g.tensor("v", synth.BF16, [2, 1, 2, 64], synth.INPUT)
        kc = g.tensor("kc", synth.BF16, [2, 16, 2, 64], synth.STATE)
        vc = g.tensor("vc", synth.BF16, [2, 16, 2, 64], synth.STATE)
        pos = g.tensor("pos", synth.I32, [1], synth.INPUT)
        out = g.tensor("o", synth.BF16, [2, 1, 4, 64], synth.OUTPUT)
        return g, [q, k, v, kc, vc, pos], out
    g, ins, out = base()
    g.op(synth.CACHED_ATTENTION, ins, [out], scale=0.125)
    fluid.Plan(g, None).close()
    # the same cache twice, a cache that is a plain input, a state tensor read by another op, a query of two rows
    g, ins, out = base()
    g.op(synth.CACHED_ATTENTION, ins[:4] + [ins[3], ins[5]], [out], scale=0.125)
    with pytest.raises(fluid.FluidError):
        fluid.Plan(g, None)
    g, ins, out = base()
    g.tensors[ins[3]]["kind"] = synth.INPUT
    g.op(synth.CACHED_ATTENTION, ins, [out], scale=0.125)
    with pytest.raises(fluid.FluidError):
        fluid.Plan(g, None)
    g, ins, out = base()
    y = g.tensor("y", synth.BF16, [2, 16, 2, 64], synth.OUTPUT)
    g.op(synth.GELU, [ins[3]], [y])
    with pytest.raises(fluid.FluidError):
        fluid.Plan(g, None)
    g, ins, out = base()
    g.tensors[ins[0]]["dims"] = [2, 2, 4, 64]
    g.tensors[out]["dims"] = [2, 2, 4, 64]
    g.op(synth.CACHED_ATTENTION, ins, [out], scale=0.125)
    with pytest.raises(fluid.FluidError):
        fluid.Plan(g, None)


# ---- implementation variants: the dynamic programme sees the best variant's cost, the step runs it --------------
def _mlp_graph(M=256, H=512, F=1024):
    """x -> LINEAR(+bias) -> GELU -> LINEAR(+bias): two tensor-core GEMM nodes on one chain (bf16)."""
    g = synth.GraphDesc()
    x = g.tensor("x", synth.BF16, [M, H], synth.INPUT)
    w1 = g.tensor("w1", synth.BF16, [H, F], synth.CONST)
    w2 = g.tensor("w2", synth.BF16, [F, H], synth.CONST)
    h = g.tensor("h", synth.BF16, [M, F], synth.ACT)
    a = g.tensor("a", synth.BF16, [M, F], synth.ACT)
    y = g.tensor("y", synth.BF16, [M, H], synth.OUTPUT)
    g.op(synth.LINEAR, [x, w1], [h], contract=1)
    g.op(synth.GELU, [h], [a])
    g.op(synth.LINEAR, [a, w2], [y], contract=1)
    return g


def _decode(code):
    return code & 15, code >> 4


def test_every_gemm_step_lists_its_variants_and_runs_the_rated_best():
    d = _mlp_graph()
    plan = fluid.Plan(d, synth.default_candidates(d))
    steps = [s for s in plan.steps() if s["kernel_name"] == "GEMM_TC"]
    assert len(steps) == 2
    for s in steps:
        codes, chosen = plan.gemm_variants(s["ops"][0])
        assert len(codes) >= 3 and chosen in codes and len(set(codes)) == len(codes)
        form, bn = _decode(chosen)
        assert bn == (s["variant"] >> 8) & 0xfff
        assert form == (3 if (s["variant"] >> 28) & 1 else 2 if (s["variant"] >> 29) & 1 else 1)
    assert plan.gemm_variants(1) == ([], 0)                # the GELU op anchors no GEMM step
    plan.close()


def test_a_requested_variant_is_the_one_that_runs():
    d = _mlp_graph()
    base = fluid.Plan(d, synth.default_candidates(d))
    codes, chosen = base.gemm_variants(0)
    base.close()
    for code in codes:
        plan = fluid.Plan(d, synth.default_candidates(d), op_variant={0: code})
        assert plan.gemm_variants(0)[1] == code
        plan.close()
    # a code the shape cannot take (a CTA pair over 100 rows) is ignored
    g = _mlp_graph(M=100)
    plan = fluid.Plan(g, synth.default_candidates(g), op_variant={0: fluid.gemm_variant_code(fluid.GV_PAIR, 256)})
    assert _decode(plan.gemm_variants(0)[1])[0] != fluid.GV_PAIR
    plan.close()


@pytest.mark.parametrize("cheap_form", [fluid.GV_SINGLE, fluid.GV_PAIR])
def test_variant_costs_from_the_caller_decide_layouts_and_variant_with_the_oracle(cheap_form):
    """eval_variant(node, layouts, variant) = base(node, layouts) + bump(variant). The node cost the dynamic programme
    must see is the minimum over the node's variants (paper, Sec. "Design", "Loop Reordering"), so the oracle planner,
    handed eval(node, layouts) = base + min over that node's variant list of bump, must arrive at the same layouts and
    the same total cost; and the step must run the arg-min variant. Making another form cheap flips the variant."""
    d = _mlp_graph()
    cands = synth.default_candidates(d)
    probe = fluid.Plan(d, cands, fusion=0)
    variants = {op: probe.gemm_variants(op)[0] for op in range(len(d.ops))}
    probe.close()
    assert all(len(variants[op]) >= 3 for op in (0, 2)) and variants[1] == []
    base = table_eval(3)

    def bump(code):
        form, bn = _decode(code)
        return 0.0 if code == 0 else (1.0 if form == cheap_form else 5.0) + {64: 0.75, 128: 0.25, 192: 0.625, 256: 0.5}[bn]

    asked, offered = set(), {}     # offered: which variants the library listed for (node, layouts): kernel knowledge

    def c_eval(user, node, n, tids, lidx, variant):
        asked.add((node, variant))
        lay = {tids[i]: lidx[i] for i in range(n)}
        offered.setdefault((node, tuple(sorted(lay.items()))), set()).add(variant)
        return base(node, lay) + bump(variant)

    def o_eval(op, lay):
        listed = offered.get((op, tuple(sorted(lay.items()))), variants[op])
        return base(op, lay) + min((bump(v) for v in listed), default=0.0)

    plan = fluid.Plan(d, cands, eval_variant=fluid.EVAL_VARIANT_FN(c_eval))
    ops, ncand, consts = _oracle_inputs(d, cands)
    want, cost, seqs = OP.plan_layouts(ops, ncand, o_eval, consts)
    assert {t: plan.tensor_info(t).layout_index for t in range(len(d.tensors))} == want
    assert plan.cost == cost and plan.sequences() == seqs
    for op in (0, 2):
        assert {v for (n, v) in asked if n == op} >= set(variants[op])      # every variant was rated
        codes, chosen = plan.gemm_variants(op)
        assert chosen == min(codes, key=bump) and _decode(chosen)[0] == cheap_form
    assert {v for (n, v) in asked if n == 1} == {0}                          # a node without variants is asked once
    plan.close()


def test_in_place_results_share_the_record_of_their_dying_operand():
    """Residual epilogues and rotary embeddings write over the operand that dies with them: one record, union
    lifetime, a smaller arena, and still a valid one (independent checker). no_inplace = 1 gives every result its own."""
    m = synth.build_model(synth.CONFIGS["llama"], materialize=False)
    d = m.graph
    cands = synth.default_candidates(d)
    plan = fluid.Plan(d, cands)
    apart = fluid.Plan(d, cands, no_inplace=1)
    name = {td["name"]: t for t, td in enumerate(d.tensors)}
    root = lambda n: plan.tensor_info(name[n]).alias_of
    # the fp32 residual stream of a pre-norm model is one buffer from the embedding to the last layer
    assert root("l0.res1") == root("l0.res2") == root("l3.res2") == root("embed") == name["embed"]
    assert root("l0.ln1.out") == name["l0.ln1.out"]
    # (at this head width the rotary embedding runs in the projection's epilogue; with 64-wide heads it is a step of its
    # own and writes over the projection it rotates)
    assert "ROPE" not in [s["kernel_name"] for s in plan.steps()] and plan.tensor_info(name["l0.q"]).offset < 0
    m64 = synth.build_model(synth.scaled(synth.CONFIGS["llama"], nh=64, L=2), materialize=False)
    p64 = fluid.Plan(m64.graph, synth.default_candidates(m64.graph))
    n64 = {td["name"]: t for t, td in enumerate(m64.graph.tensors)}
    r64 = lambda n: p64.tensor_info(n64[n]).alias_of
    assert r64("l0.q_rope") == r64("l0.q") == n64["l0.q"] and r64("l1.k_rope") == r64("l1.k") and r64("l0.q") != r64("l0.k")
    p64.close()
    assert apart.tensor_info(name["l0.res1"]).alias_of == name["l0.res1"]
    recs, offs = plan_records(plan)
    assert OA.check_arena(recs, offs, plan.arena_bytes) == []
    assert len(recs) < len(apart.records()) and plan.arena_bytes < apart.arena_bytes
    assert plan.live_bound_bytes < apart.live_bound_bytes
    # the holder's lifetime covers every tensor that lives in it
    steps = plan.steps()
    first, last = next((f, l) for rid, _, f, l in recs if rid == name["embed"])
    group = [t for t in range(len(d.tensors)) if plan.tensor_info(t).alias_of == name["embed"]]
    touched = [i for i, s in enumerate(steps) if set(group) & set(s["ins"] + s["outs"])]
    assert (first, last) == (min(touched), max(touched)) and last > len(steps) // 2
    plan.close(); apart.close()
