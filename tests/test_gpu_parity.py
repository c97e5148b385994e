"""Parity of the CUDA path (through the C-ABI) against the fp64 oracle, element by element."""
import math

import numpy as np
import pytest

from paper_2411_09242_b200 import fluid, synth
from tests.helpers import assert_close, check_steps_sampled, rand_feed, run_gpu, run_oracle, single_op_graph, tol_for

pytestmark = pytest.mark.gpu

DT = [synth.F32, synth.BF16]


def model_feeds(m):
    feeds = dict(m.consts)
    feeds[m.graph.inputs[0]] = m.ids
    return feeds


SMALL = {
    "encoder": synth.scaled(synth.CONFIGS["bert_base"], L=2, H=256, nh=4, F=512, S=160, B=2, V=1000),
    "gpt": synth.scaled(synth.CONFIGS["gpt2_small"], L=2, H=256, nh=4, F=512, S=192, B=2, V=1003),
    "llama": synth.scaled(synth.CONFIGS["llama"], L=2, H=512, nh=4, F=1408, S=256, B=1, V=2000),
}


def test_tiny_fp32_config_end_to_end():
    m = synth.build_model(synth.CONFIGS["tiny"])
    ref = run_oracle(m.graph, model_feeds(m))
    for cands in (None, synth.default_candidates(m.graph)):
        got, plan, _ = run_gpu(m.graph, model_feeds(m), cands)
        for t in m.graph.outputs:
            assert_close(got[t], ref[t], synth.F32, "tiny")
        plan.close()


@pytest.mark.parametrize("family", ["encoder", "gpt", "llama"])
@pytest.mark.parametrize("dtype", DT)
def test_small_models_planned_and_canonical(family, dtype):
    cfg = synth.scaled(SMALL[family], dtype=dtype)
    m = synth.build_model(cfg)
    feeds = model_feeds(m)
    ref = run_oracle(m.graph, feeds)
    results = {}
    for label, cands, opts in [("planned", synth.default_candidates(m.graph), {}),
                               ("canonical", None, {}),
                               ("unfused", synth.default_candidates(m.graph), {"fusion": 0}),
                               ("simt", synth.default_candidates(m.graph), {"gemm_path": 1}),
                               ("unfused_attention", synth.default_candidates(m.graph), {"unfused_attention": 1}),
                               ("no_reuse", synth.default_candidates(m.graph), {"no_reuse": 1}),
                               ("best_fit", synth.default_candidates(m.graph), {"arena_policy": 1}),
                               ("several_orders", synth.default_candidates(m.graph), {"arena_policy": 2})]:
        got, plan, _ = run_gpu(m.graph, feeds, cands, **opts)
        for t in m.graph.outputs:
            assert_close(got[t], ref[t], dtype, f"{family}/{label}")
        results[label] = got
        plan.close()
    # same kernels, different arena offsets: bit-identical outputs
    for t in m.graph.outputs:
        assert np.array_equal(results["planned"][t], results["no_reuse"][t])


def test_rms_norm_split_across_gemm_steps():
    """A pre-norm decoder wide enough for the CTA-pair GEMMs (hidden 1024, FFN 4096, 1024 tokens): the RMS
    normalisations between o-proj and gate / up and between down and the next layer's q / k / v have no launch of their
    own (the first GEMM writes bf16(x * gain) and per-slab sums of squares, the readers scale their rows by 1 / rms).
    Whole outputs against the oracle, with the split and with no_norm_split = 1; every launch of the split plan on
    sampled rows; a planned arena (the scratch slices among the reused ones) against one slice per tensor, bit for bit."""
    cfg = synth.scaled(synth.CONFIGS["llama"], L=2, H=1024, nh=8, F=4096, S=1024, B=1, V=2000)
    m = synth.build_model(cfg)
    feeds = model_feeds(m)
    ref = run_oracle(m.graph, feeds)
    cands = synth.default_candidates(m.graph)
    got, plan, runner = run_gpu(m.graph, feeds, cands, arena_policy=2)
    split_steps = [s for s in plan.steps() if s["kernel_name"] == "GEMM_TC"
                   and any(m.graph.ops[o]["kind"] == synth.RMSNORM for o in s["ops"])]
    assert len(split_steps) == 3                                   # layer 0: gate / up; layer 1: q / k / v and gate / up
    assert [s["kernel_name"] for s in plan.steps()].count("NORM") == 2   # the first and the last one stay
    assert runner.status() == 0
    for t in m.graph.outputs:
        assert_close(got[t], ref[t], synth.BF16, "split RMS normalisation")
    apart, plan_apart, _ = run_gpu(m.graph, feeds, cands, arena_policy=2, no_norm_split=1)
    assert [s["kernel_name"] for s in plan_apart.steps()].count("NORM") == 5
    for t in m.graph.outputs:
        assert_close(apart[t], ref[t], synth.BF16, "RMS normalisation as its own step")
    alone, plan_alone, runner_alone = run_gpu(m.graph, feeds, cands, no_reuse=1)
    for t in m.graph.outputs:
        assert np.array_equal(alone[t], got[t])
    assert check_steps_sampled(m.graph, plan_alone, runner_alone, feeds) >= len(plan_alone.steps())
    plan.close(); plan_apart.close(); plan_alone.close()


@pytest.mark.parametrize("family", ["gpt", "llama"])
def test_per_step_parity_localises_drift(family):
    """Each step's output vs the oracle op applied to the GPU's own inputs of that step."""
    cfg = synth.scaled(SMALL[family], dtype=synth.BF16, L=1)
    m = synth.build_model(cfg)
    feeds = model_feeds(m)
    got, plan, runner = run_gpu(m.graph, feeds, synth.default_candidates(m.graph), fusion=0, no_reuse=1)
    from oracle import graph_exec
    d = m.graph
    const_derived = run_oracle(d, feeds, keep_all=True)
    for s in plan.steps():
        op = d.ops[s["ops"][0]]
        ins = []
        for t in op["ins"]:
            k = d.tensors[t]["kind"]
            root_kind = d.tensors[plan.tensor_info(t).alias_of]["kind"]
            if k in (synth.CONST, synth.INPUT):
                ins.append(feeds[t])
            elif root_kind == synth.CONST:          # a zero-copy view of a constant
                ins.append(const_derived[t])
            else:
                ins.append(runner.read_tensor(t))
        want = graph_exec.run_op(op["kind"], [np.asarray(a) if np.asarray(a).dtype.kind in "iu" else np.asarray(a, np.float64) for a in ins], op["attrs"])[0]
        have = runner.read_tensor(op["outs"][0])
        if op["kind"] == synth.BMM_QK:          # strictly-upper entries are never read downstream
            S = want.shape[-1]
            mask = np.tril(np.ones((S, S), bool))
            want, have = want * mask, np.where(mask, have, 0.0)
        assert_close(have, want, synth.BF16, f"{family} step {s['kernel_name']} op {s['ops'][0]}", tol=2 ** -7)
    plan.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("M,N,K", [(64, 64, 64), (130, 70, 50), (1, 33, 200), (257, 129, 72), (128, 256, 1024)])
def test_linear_shapes_with_ragged_tails(dtype, M, N, K):
    g = single_op_graph(synth.LINEAR, [[M, K], [K, N], [N]], [M, N], dtype, {"contract": 1},
                        in_kinds={1: synth.CONST, 2: synth.CONST})
    feeds = {0: rand_feed([M, K], dtype, 1), 1: rand_feed([K, N], dtype, 2), 2: rand_feed([N], dtype, 3)}
    ref = run_oracle(g, feeds)
    for cands in (None, synth.default_candidates(g)):
        got, plan, _ = run_gpu(g, feeds, cands)
        assert_close(got[3], ref[3], dtype, f"linear {M}x{N}x{K}")
        plan.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("a_major", ["row", "col"])
@pytest.mark.parametrize("b_major", ["row", "col"])
@pytest.mark.parametrize("n", [96, 256])
def test_gemm_operand_majors(dtype, a_major, b_major, n):
    g, arrs = synth.gemm_case(n, n + 64, n + 128, a_major, b_major, dtype=dtype)
    ref = run_oracle(g, arrs)
    got, plan, _ = run_gpu(g, arrs, synth.default_candidates(g))
    assert "PERMUTE" not in [s["kernel_name"] for s in plan.steps()]     # operands read in place
    assert_close(got[g.outputs[0]], ref[g.outputs[0]], dtype, f"gemm {a_major}/{b_major}")
    got_c, plan_c, _ = run_gpu(g, arrs, None)                            # canonical: real transposes
    assert_close(got_c[g.outputs[0]], ref[g.outputs[0]], dtype, "gemm canonical")
    plan.close(); plan_c.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("causal,n", [(0, n) for n in (1, 7, 128, 200, 1024, 2048, 4100)] +
                         [(1, n) for n in (1, 7, 128, 200, 1024)])     # the square causal cases are kept small
def test_softmax_rows(dtype, causal, n):
    rows = 3 if not causal else n
    shape = [2, rows, n]
    g = single_op_graph(synth.SOFTMAX, [shape], shape, dtype, {"causal": causal, "scale": 0.5})
    feeds = {0: rand_feed(shape, dtype, 4, -8.0, 8.0)}
    ref = run_oracle(g, feeds)[1]
    got, plan, _ = run_gpu(g, feeds)
    assert_close(got[1], ref, dtype, f"softmax n={n}")
    np.testing.assert_allclose(got[1].sum(-1), 1.0, atol=2e-2 if dtype == synth.BF16 else 1e-5)
    if causal:
        iu = np.triu_indices(n, 1)
        assert np.all(got[1][:, iu[0], iu[1]] == 0.0)
    plan.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("rows,width", [(5, 128), (33, 768), (4, 4096), (3, 100), (2, 8192)])
@pytest.mark.parametrize("rms", [0, 1])
def test_norm_rows(dtype, rows, width, rms):
    kind = synth.RMSNORM if rms else synth.LAYERNORM
    shapes = [[1, rows, width], [width]] + ([] if rms else [[width]])
    g = single_op_graph(kind, shapes, [1, rows, width], dtype, {"eps": 1e-5},
                        in_kinds={1: synth.CONST, 2: synth.CONST})
    feeds = {0: rand_feed([1, rows, width], dtype, 5, -3.0, 5.0), 1: rand_feed([width], dtype, 6, 0.5, 1.5)}
    if not rms:
        feeds[2] = rand_feed([width], dtype, 7)
    out = len(shapes)
    ref = run_oracle(g, feeds)[out]
    got, plan, _ = run_gpu(g, feeds)
    assert_close(got[out], ref, dtype, "norm")
    plan.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("kind,attrs,nin", [(synth.ADD, {}, 2), (synth.MUL, {}, 2), (synth.GELU, {"gelu_tanh": 0}, 1),
                                            (synth.GELU, {"gelu_tanh": 1}, 1), (synth.SILU, {}, 1)])
@pytest.mark.parametrize("shape", [[3, 5, 7], [2, 64, 256]])
def test_elementwise(dtype, kind, attrs, nin, shape):
    g = single_op_graph(kind, [shape] * nin, shape, dtype, attrs)
    feeds = {i: rand_feed(shape, dtype, 8 + i, -4.0, 4.0) for i in range(nin)}
    ref = run_oracle(g, feeds)[nin]
    got, plan, _ = run_gpu(g, feeds)
    assert_close(got[nin], ref, dtype, "eltwise")
    plan.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("interleaved", [0, 1])
def test_rope_in_every_head_layout(dtype, interleaved):
    B, S, nh, D = 2, 70, 3, 64
    d = synth.GraphDesc()
    x = d.tensor("x", dtype, [B, S, nh, D], synth.INPUT)
    for perm in [(0, 1, 2, 3), (0, 2, 1, 3), (0, 2, 3, 1)]:
        # force the layout: transpose into it, rope there, transpose back
        d = synth.GraphDesc()
        x = d.tensor("x", dtype, [B, S, nh, D], synth.INPUT)
        a = d.tensor("a", dtype, [B, S, nh, D], synth.ACT)
        d.op(synth.GELU, [x], [a])          # a producer whose output layout is free
        r = d.tensor("r", dtype, [B, S, nh, D], synth.ACT)
        d.op(synth.ROPE, [a], [r], rope_base=10000.0, rope_interleaved=interleaved)
        y = d.tensor("y", dtype, [B, S, nh, D], synth.OUTPUT)
        d.op(synth.ADD, [r, r], [y])
        feeds = {x: rand_feed([B, S, nh, D], dtype, 9)}
        ref = run_oracle(d, feeds)[y]
        cands = synth.canonical_candidates(d)
        got, plan, _ = run_gpu(d, feeds, cands)
        assert_close(got[y], ref, dtype, "rope canonical")
        plan.close()
    # rope directly on tensors held in non-canonical layouts, via a planned attention block
    cfg = synth.scaled(SMALL["llama"], dtype=dtype, L=1, S=64)
    m = synth.build_model(cfg)
    got, plan, _ = run_gpu(m.graph, model_feeds(m), synth.default_candidates(m.graph))
    ref = run_oracle(m.graph, model_feeds(m))
    for t in m.graph.outputs:
        assert_close(got[t], ref[t], dtype, "rope in planned model")
    plan.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("case", [dict(B=1, S=128, nh=12, D=64), dict(B=2, S=100, nh=3, D=40), dict(B=3, S=257, nh=2, D=128),
                                  dict(B=2, S=37, nh=5, D=64), dict(B=1, S=20, nh=33, D=256), dict(B=2, S=9, nh=17, D=128)])
@pytest.mark.parametrize("target", ["BHSD", "BHDS"])
def test_layout_transforms_bit_exact(dtype, case, target):
    g, a = synth.permute_case(target=target, dtype=dtype, **case)
    got, plan, _ = run_gpu(g, {0: a})
    ref = run_oracle(g, {0: a})[1]
    assert np.array_equal(got[1], ref)            # pure data movement: bit exact
    assert [s["kernel_name"] for s in plan.steps()] == ["PERMUTE"]
    plan.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("case", [dict(B=2, S=1000, nh=5, D=72), dict(B=1, S=4104, nh=3, D=136), dict(B=3, S=520, nh=7, D=64),
                                  dict(B=1, S=1001, nh=9, D=128), dict(B=2, S=264, nh=40, D=200)])
@pytest.mark.parametrize("target", ["BHSD", "BHDS"])
def test_large_ragged_layout_transforms_bit_exact(dtype, case, target):
    """Transforms above a megabyte take the bulk-tensor (TMA) forms when their strides allow it: extents that are not
    multiples of the 64-wide tile or of the box rows, 16- and 32-bit elements, and one case (S = 1001) whose output
    stride is not 16-byte aligned and therefore stays on the register kernels."""
    g, a = synth.permute_case(target=target, dtype=dtype, **case)
    got, plan, r = run_gpu(g, {0: a})
    ref = run_oracle(g, {0: a})[1]
    assert np.array_equal(got[1], ref)
    assert r.status() == 0
    plan.close()


@pytest.mark.parametrize("dtype", DT)
@pytest.mark.parametrize("dims,perm", [([6, 40, 24, 136], [2, 0, 1, 3]), ([6, 40, 24, 136], [1, 2, 0, 3]), ([6, 40, 24, 136], [0, 3, 2, 1]),
                                       ([6, 40, 24, 136], [3, 1, 0, 2]), ([2, 3, 40, 24, 72], [0, 3, 1, 2, 4]),
                                       ([2, 3, 40, 24, 72], [2, 1, 4, 0, 3]), ([1100, 520], [1, 0]), ([3, 520, 1096], [0, 2, 1])])
def test_general_permutations_above_a_megabyte(dtype, dims, perm):
    """Permutations other than the two head transposes, of rank 2 to 5, large enough for the bulk-tensor forms: the same
    fastest dim on both sides (rows form, any order of the outer dims), a new fastest dim (tiles form: 16-bit elements
    only, the others stay on the register kernels), extents that are no multiples of the 64-wide tile."""
    g = synth.GraphDesc()
    x = g.tensor("x", dtype, dims, synth.INPUT)
    y = g.tensor("y", dtype, [dims[q] for q in perm], synth.OUTPUT)
    g.op(synth.TRANSPOSE, [x], [y], perm=perm)
    a = rand_feed(dims, dtype, 77)
    got, plan, r = run_gpu(g, {x: a})
    ref = run_oracle(g, {x: a})[y]
    assert np.array_equal(got[y], ref)
    assert r.status() == 0
    plan.close()


@pytest.mark.parametrize("dtype", DT)
def test_embed_and_select_last(dtype):
    g = synth.GraphDesc()
    ids = g.tensor("ids", synth.I32, [3, 17], synth.INPUT)
    tok = g.tensor("tok", dtype, [50, 96], synth.CONST)
    pos = g.tensor("pos", dtype, [17, 96], synth.CONST)
    x = g.tensor("x", dtype, [3, 17, 96], synth.OUTPUT)
    g.op(synth.EMBED, [ids, tok, pos], [x])
    last = g.tensor("last", dtype, [3, 96], synth.OUTPUT)
    g.op(synth.SELECT_LAST_TOKEN, [x], [last])
    feeds = {ids: synth.token_ids(3, 0, [3, 17], 50), tok: rand_feed([50, 96], dtype, 10), pos: rand_feed([17, 96], dtype, 11)}
    ref = run_oracle(g, feeds)
    got, plan, _ = run_gpu(g, feeds)
    assert_close(got[x], ref[x], dtype, "embed")
    assert np.array_equal(got[last], got[x][:, -1, :])
    plan.close()


def test_run_allocates_nothing_and_rejects_bad_pointers():
    import torch
    m = synth.build_model(synth.CONFIGS["tiny"])
    plan = fluid.Plan(m.graph, synth.default_candidates(m.graph))
    r = fluid.Runner(plan, m.consts)
    r.set_inputs([m.ids])
    r.run(); torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    before = fluid.fluid_launch_count()
    for _ in range(5):
        r.run()
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0                                   # no device allocation inside fluid_run
    assert fluid.fluid_launch_count() - before == 5 * len(plan.steps())
    with pytest.raises(fluid.FluidError) as e:              # misaligned arena
        fluid.fluid_run(plan.handle, r.arena.data_ptr() + 8, [b.data_ptr() for b in r.inputs],
                        [b.data_ptr() for b in r.outputs])
    assert e.value.code == fluid.FLUID_EALIGN
    plan2 = fluid.Plan(m.graph, None)                       # constants not bound
    with pytest.raises(fluid.FluidError):
        fluid.fluid_run(plan2.handle, r.arena.data_ptr(), [b.data_ptr() for b in r.inputs],
                        [b.data_ptr() for b in r.outputs])
    plan.close(); plan2.close()


def _attention_graph(B, S, nh, D, causal, k_layout, v_layout, dtype=synth.BF16):
    """q, k, v arrive as graph inputs in [B,S,nh,D]; k and v are first copied into a chosen physical
    layout (a GELU-free pass-through would change values, so a TRANSPOSE pair pins the layout)."""
    g = synth.GraphDesc()
    q = g.tensor("q", dtype, [B, S, nh, D], synth.INPUT)
    k = g.tensor("k", dtype, [B, S, nh, D], synth.INPUT)
    v = g.tensor("v", dtype, [B, S, nh, D], synth.INPUT)
    qh = g.tensor("qh", dtype, [B, nh, S, D]); g.op(synth.TRANSPOSE, [q], [qh], perm=[0, 2, 1, 3])
    kT = g.tensor("kT", dtype, [B, nh, D, S]); g.op(synth.TRANSPOSE, [k], [kT], perm=[0, 2, 3, 1])
    vh = g.tensor("vh", dtype, [B, nh, S, D]); g.op(synth.TRANSPOSE, [v], [vh], perm=[0, 2, 1, 3])
    sc = g.tensor("sc", dtype, [B, nh, S, S]); g.op(synth.BMM_QK, [qh, kT], [sc], scale=1.0 / math.sqrt(D))
    pr = g.tensor("pr", dtype, [B, nh, S, S]); g.op(synth.SOFTMAX, [sc], [pr], causal=int(causal), scale=1.0)
    ch = g.tensor("ch", dtype, [B, nh, S, D]); g.op(synth.BMM_PV, [pr, vh], [ch])
    out = g.tensor("out", dtype, [B, nh, S, D], synth.OUTPUT)
    g.op(synth.ADD, [ch, ch], [out])
    cands = synth.canonical_candidates(g)
    cands[kT] = [(0, 1, 2, 3), k_layout] if k_layout != (0, 1, 2, 3) else [(0, 1, 2, 3)]
    cands[vh] = [(0, 1, 2, 3), v_layout] if v_layout != (0, 1, 2, 3) else [(0, 1, 2, 3)]
    return g, cands, (kT, vh)


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("causal", [0, 1])
@pytest.mark.parametrize("S", [8, 104, 128, 328])
def test_fused_attention_shapes_and_operand_majors(D, causal, S):
    """Ragged sequence lengths (one tile, partial tiles, several tiles) and both majors of K and V: the
    canonical kT [B,nh,D,S] is sequence-contiguous, its aliasing layout is head-dim-contiguous."""
    B, nh = 2, 3
    for k_layout, v_layout in [((0, 1, 2, 3), (0, 1, 2, 3)), ((0, 3, 1, 2), (0, 2, 1, 3)), ((0, 1, 2, 3), (0, 1, 3, 2))]:
        g, cands, _ = _attention_graph(B, S, nh, D, causal, k_layout, v_layout)
        feeds = {t: rand_feed([B, S, nh, D], synth.BF16, 20 + t, -2.0, 2.0) for t in g.inputs}
        ref = run_oracle(g, feeds)[g.outputs[0]]
        opts = {"force_canonical": 1} if k_layout == (0, 1, 2, 3) and v_layout == (0, 1, 2, 3) else {}
        got, plan, _ = run_gpu(g, feeds, cands, **opts)
        assert "ATTN" in [s["kernel_name"] for s in plan.steps()]
        assert_close(got[g.outputs[0]], ref, synth.BF16, f"attention D={D} S={S} causal={causal} k={k_layout} v={v_layout}")
        plan.close()


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("causal", [0, 1])
def test_short_sequence_attention_in_registers(D, causal):
    """Sequences of at most 128 positions whose K and V have the head dim contiguous run on the register form (16
    query rows per CTA, four warps that split the keys and then the head dim): lengths that end inside a warp's 32
    keys, inside a 16-key step and inside a 16-row block, one key only, and the full 128; K and V rows strided
    ([B,S,nh,D]) or dense per head ([B,nh,S,D])."""
    B, nh = 2, 5
    for S in (8, 16, 24, 40, 72, 120, 128):
        for k_layout, v_layout in [((0, 3, 1, 2), (0, 2, 1, 3)), ((0, 1, 3, 2), (0, 1, 2, 3))]:
            g, cands, _ = _attention_graph(B, S, nh, D, causal, k_layout, v_layout)
            feeds = {t: rand_feed([B, S, nh, D], synth.BF16, 60 + t + S, -2.0, 2.0) for t in g.inputs}
            ref = run_oracle(g, feeds)[g.outputs[0]]
            got, plan, runner = run_gpu(g, feeds, cands)
            assert "ATTN" in [s["kernel_name"] for s in plan.steps()]
            assert runner.status() == 0
            assert_close(got[g.outputs[0]], ref, synth.BF16, f"short attention D={D} S={S} causal={causal} k={k_layout}")
            plan.close()


@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("causal", [0, 1])
def test_fused_attention_more_work_items_than_sms(D, causal):
    """The persistent form deals its work items (a head's pair of query tiles) to one CTA per SM: with 4 x 40 heads and
    two items per head (the second one a partial tile pair: 328 = 256 + 72 rows) every CTA walks two or three items of
    different heads and lengths, so the barrier phases, the K / V ring and the tensor-memory tiles are carried across
    item boundaries, including from a two-tile item to a one-tile one."""
    B, nh, S = 4, 40, 328
    for k_layout, v_layout in [((0, 1, 2, 3), (0, 1, 2, 3)), ((0, 3, 1, 2), (0, 2, 1, 3))]:
        g, cands, _ = _attention_graph(B, S, nh, D, causal, k_layout, v_layout)
        feeds = {t: rand_feed([B, S, nh, D], synth.BF16, 40 + t, -2.0, 2.0) for t in g.inputs}
        ref = run_oracle(g, feeds)[g.outputs[0]]
        opts = {"force_canonical": 1} if k_layout == (0, 1, 2, 3) else {}
        got, plan, runner = run_gpu(g, feeds, cands, **opts)
        assert "ATTN" in [s["kernel_name"] for s in plan.steps()]
        assert runner.status() == 0
        assert_close(got[g.outputs[0]], ref, synth.BF16, f"attention over many items D={D} causal={causal} k={k_layout}")
        plan.close()


@pytest.mark.parametrize("M,N,K", [(1024, 2552, 136), (512, 5120, 72), (768, 4096, 200)])
def test_cta_pair_gemm_ragged_shapes(M, N, K):
    """Enough 256-wide tiles for the CTA-pair kernel (two CTAs per 256 x 256 tile), with a ragged last column
    tile, a k range that is not a multiple of the stage depth and, in the last case, an odd number of row tiles
    (which must fall back to the single-CTA kernel)."""
    g = single_op_graph(synth.LINEAR, [[M, K], [K, N], [N]], [M, N], synth.BF16, {"contract": 1},
                        in_kinds={1: synth.CONST, 2: synth.CONST})
    feeds = {0: rand_feed([M, K], synth.BF16, 1), 1: rand_feed([K, N], synth.BF16, 2), 2: rand_feed([N], synth.BF16, 3)}
    ref = run_oracle(g, feeds)[3]
    # (with so short a k range the planner's rating prefers narrow tiles: the pair form is asked for by name)
    want = fluid.gemm_variant_code(fluid.GV_PAIR if M % 256 == 0 else fluid.GV_SINGLE, 256)
    got, plan, runner = run_gpu(g, feeds, synth.default_candidates(g), op_variant={0: want})
    v = plan.steps()[0]["variant"]
    assert ((v >> 8) & 0xfff) == 256 and bool((v >> 29) & 1) == (M % 256 == 0)
    assert_close(got[3], ref, synth.BF16, f"pair GEMM {M}x{N}x{K}")
    runner.run()
    assert np.array_equal(runner.outputs_host()[0], got[3])
    plan.close()


def test_gelu_erf_over_a_wide_range():
    """The kernels evaluate erf as a clamped polynomial: check it element by element well beyond the clamp."""
    shape = [4, 4096]
    g = single_op_graph(synth.GELU, [shape], shape, synth.BF16, {"gelu_tanh": 0})
    x = rand_feed(shape, synth.BF16, 77, -9.0, 9.0)
    ref = run_oracle(g, {0: x})[1]
    got, plan, _ = run_gpu(g, {0: x})
    err = np.abs(got[1].astype(np.float64) - ref)
    assert np.all(err <= 3e-4 + 2.0 ** -8 * np.abs(ref))      # polynomial error + bf16 rounding of the output
    plan.close()


@pytest.mark.parametrize("M,N,K", [(128, 768, 3072), (100, 256, 2048), (64, 1536, 1024)])
def test_split_k_gemm_matches_oracle_and_unsplit(M, N, K):
    g = single_op_graph(synth.LINEAR, [[M, K], [K, N], [N]], [M, N], synth.BF16, {"contract": 1},
                        in_kinds={1: synth.CONST, 2: synth.CONST})
    feeds = {0: rand_feed([M, K], synth.BF16, 1), 1: rand_feed([K, N], synth.BF16, 2), 2: rand_feed([N], synth.BF16, 3)}
    ref = run_oracle(g, feeds)[3]
    split, plan, runner = run_gpu(g, feeds, synth.default_candidates(g), split_k=1)
    assert (plan.steps()[0]["variant"] >> 24) > 1 and any(r["tensor"] < 0 for r in plan.records())
    assert_close(split[3], ref, synth.BF16, "split-K")
    runner.run()                                   # counters are left at zero: a second run works the same
    assert np.array_equal(runner.outputs_host()[0], split[3])
    whole, plan2, _ = run_gpu(g, feeds, synth.default_candidates(g), split_k=-1)
    assert (plan2.steps()[0]["variant"] >> 24) == 0
    assert_close(split[3], whole[3], synth.BF16, "split vs unsplit", tol=2 ** -7)
    # default options: the cut runs inside one thread-block cluster per output tile, no scratch record
    clus, plan3, runner3 = run_gpu(g, feeds, synth.default_candidates(g))
    v = plan3.steps()[0]["variant"]
    assert (v >> 28) & 1 and ((v >> 24) & 15) in (2, 4, 8) and not any(r["tensor"] < 0 for r in plan3.records())
    assert_close(clus[3], ref, synth.BF16, "cluster split-K")
    assert_close(clus[3], whole[3], synth.BF16, "cluster split vs unsplit", tol=2 ** -7)
    runner3.run()                                  # the summation order is fixed: bit-identical reruns
    assert np.array_equal(runner3.outputs_host()[0], clus[3])
    plan.close(); plan2.close(); plan3.close()


def test_split_k_inside_a_model():
    cfg = synth.scaled(SMALL["encoder"], dtype=synth.BF16, F=2048)
    m = synth.build_model(cfg)
    ref = run_oracle(m.graph, model_feeds(m))
    got, plan, _ = run_gpu(m.graph, model_feeds(m), synth.default_candidates(m.graph), split_k=1)
    assert any((s["variant"] >> 24) > 1 for s in plan.steps())
    for t in m.graph.outputs:
        assert_close(got[t], ref[t], synth.BF16, "encoder with split-K")
    plan.close()


@pytest.mark.parametrize("family,dtype", [("encoder", synth.F32), ("gpt", synth.BF16), ("llama", synth.BF16)])
def test_plan_from_measured_costs(family, dtype):
    """The paper's eval: every (operator, layouts) cost the dynamic programme asks for is measured on the GPU
    (one operator alone, its tensors forced into those layouts). The plan that comes out is a valid plan:
    same results as the oracle, a cost that is the sum of measured times, not above the all-canonical cost."""
    from paper_2411_09242_b200.measure import MeasuredEval
    cfg = synth.scaled(SMALL[family], dtype=dtype, L=1)
    m = synth.build_model(cfg)
    cands = synth.default_candidates(m.graph)
    ev = MeasuredEval(m.graph, cands, reps=3, warmup=1)
    plan = fluid.Plan(m.graph, cands, eval=ev.callback)
    assert ev.measured > len({o["kind"] for o in m.graph.ops}) and 0 < plan.cost <= plan.canonical_cost < 1.0
    ref = run_oracle(m.graph, model_feeds(m))
    runner = fluid.Runner(plan, m.consts)
    runner.set_inputs([m.ids])
    runner.run()
    assert runner.status() == 0
    for tid, got in zip(m.graph.outputs, runner.outputs_host()):
        assert_close(got, ref[tid], dtype, f"measured-cost plan {family} output {tid}")
    # asking again costs nothing: the table answers
    before = ev.measured
    plan2 = fluid.Plan(m.graph, cands, eval=ev.callback)
    assert ev.measured == before and plan2.cost == plan.cost
    plan.close(); plan2.close()


@pytest.mark.parametrize("kind,dtype,rows,width", [
    (synth.LAYERNORM, synth.BF16, 20001, 768),
    (synth.RMSNORM, synth.BF16, 19000, 1024),
    (synth.LAYERNORM, synth.BF16, 19500, 200),
    (synth.LAYERNORM, synth.F32, 19001, 256),
    (synth.RMSNORM, synth.F32, 19000, 500),
    (synth.RMSNORM, synth.BF16, 5001, 4096),      # a row shared by four warps
    (synth.LAYERNORM, synth.BF16, 9999, 2048),    # by two
    (synth.LAYERNORM, synth.F32, 5000, 2048),     # fp32: by four
    (synth.RMSNORM, synth.BF16, 2501, 8192),      # by eight
])
def test_norm_over_many_rows(kind, dtype, rows, width):
    """Inputs with many more rows than resident warps take the persistent kernel (rows walked with the grid's stride,
    pieces prefetched through a per-lane ring); ragged row counts and widths that leave lanes idle included."""
    shapes = [[1, rows, width], [width]] + ([[width]] if kind == synth.LAYERNORM else [])
    g = single_op_graph(kind, shapes, [1, rows, width], dtype, {"eps": 1e-5})
    feeds = {0: rand_feed(shapes[0], dtype, 1, -3, 3), 1: rand_feed([width], dtype, 2, 0.5, 1.5)}
    if kind == synth.LAYERNORM:
        feeds[2] = rand_feed([width], dtype, 3)
    got, plan, _ = run_gpu(g, feeds)
    out = g.outputs[0]
    assert_close(got[out], run_oracle(g, feeds)[out], dtype, "norm, many rows")
    plan.close()


def test_norm_over_many_rows_reading_the_fp32_stream():
    """EMBED -> LAYERNORM over 20480 tokens: the embedding is held in fp32 (it feeds a normalisation only), so the
    persistent kernel reads 32-byte chunks through its ring."""
    g = synth.GraphDesc()
    ids = g.tensor("ids", synth.I32, [10, 2048], synth.INPUT)
    tok = g.tensor("tok", synth.BF16, [1000, 768], synth.CONST)
    x = g.tensor("x", synth.BF16, [10, 2048, 768], synth.ACT)
    gam = g.tensor("gamma", synth.BF16, [768], synth.CONST)
    bet = g.tensor("beta", synth.BF16, [768], synth.CONST)
    y = g.tensor("y", synth.BF16, [10, 2048, 768], synth.OUTPUT)
    g.op(synth.EMBED, [ids, tok], [x])
    g.op(synth.LAYERNORM, [x, gam, bet], [y], eps=1e-5)
    feeds = {ids: synth.token_ids(4, 0, [10, 2048], 1000), tok: rand_feed([1000, 768], synth.BF16, 5, -2, 2),
             gam: rand_feed([768], synth.BF16, 6, 0.5, 1.5), bet: rand_feed([768], synth.BF16, 7)}
    got, plan, _ = run_gpu(g, feeds)
    assert plan.tensor_info(x).bytes >= 10 * 2048 * 768 * 4     # held in fp32
    assert_close(got[y], run_oracle(g, feeds)[y], synth.BF16, "embed -> layernorm")
    plan.close()


# ---- implementation variants of the tensor-core GEMM (the paper's "Loop Reordering": speed changes, numbers do not) ----
@pytest.mark.parametrize("M,N,K", [(512, 768, 1024), (128, 2304, 768), (1024, 512, 256)])
def test_every_gemm_variant_gives_the_same_numbers(M, N, K):
    g = single_op_graph(synth.LINEAR, [[M, K], [K, N], [N]], [M, N], synth.BF16, {"contract": 1},
                        in_kinds={1: synth.CONST, 2: synth.CONST})
    feeds = {0: rand_feed([M, K], synth.BF16, 3), 1: rand_feed([K, N], synth.BF16, 4), 2: rand_feed([N], synth.BF16, 5)}
    ref = run_oracle(g, feeds)[g.outputs[0]]
    base = fluid.Plan(g, synth.default_candidates(g))
    codes, chosen = base.gemm_variants(0)
    base.close()
    assert len(codes) >= 3 and chosen in codes
    outs = {}
    for code in codes:
        got, plan, _ = run_gpu(g, feeds, synth.default_candidates(g), op_variant={0: code})
        assert plan.gemm_variants(0)[1] == code
        assert_close(got[g.outputs[0]], ref, synth.BF16, f"variant {code & 15}/{code >> 4}", tol=2 ** -7)
        outs[code] = got[g.outputs[0]]
        plan.close()
    # forms that do not split k add up in the same order: bit-identical
    whole = [outs[c] for c in codes if (c & 15) != fluid.GV_CLUSTER]
    assert all(np.array_equal(whole[0], w) for w in whole[1:])


def test_plan_from_measured_variant_costs():
    """eval_variant answered by measurement: every (operator, layouts, variant) the dynamic programme asks about is
    timed on the GPU; the node cost it sees is the fastest variant's time and that variant runs."""
    from paper_2411_09242_b200.measure import MeasuredEval
    cfg = synth.scaled(SMALL["gpt"], dtype=synth.BF16, L=1, H=256, F=512, S=256)
    m = synth.build_model(cfg)
    cands = synth.default_candidates(m.graph)
    ev = MeasuredEval(m.graph, cands, reps=3, warmup=1, variants=True)
    plan = fluid.Plan(m.graph, cands, eval_variant=ev.callback_variant)
    rated = {k[2] for k in ev.table}
    assert len(rated - {0}) >= 2 and 0 < plan.cost <= plan.canonical_cost < 1.0
    for s in plan.steps():
        if s["kernel_name"] == "GEMM_TC":
            codes, chosen = plan.gemm_variants(s["ops"][0])
            assert chosen in codes
    ref = run_oracle(m.graph, model_feeds(m))
    runner = fluid.Runner(plan, m.consts)
    runner.set_inputs([m.ids])
    runner.run()
    assert runner.status() == 0
    for tid, got in zip(m.graph.outputs, runner.outputs_host()):
        assert_close(got, ref[tid], synth.BF16, f"measured-variant plan output {tid}")
    plan.close()


def test_step_variants_tuned_in_place():
    """The fused steps a model really runs, each timed inside the whole plan with every variant its shape admits; the
    fastest per step goes back into the plan. Results stay those of the oracle."""
    from paper_2411_09242_b200.measure import tune_step_variants
    cfg = synth.scaled(SMALL["gpt"], dtype=synth.BF16, L=2, H=256, F=1024, S=512, B=2)
    m = synth.build_model(cfg)
    cands = synth.default_candidates(m.graph)
    op_variant, table = tune_step_variants(m.graph, cands, m.consts, [m.ids], reps=3, warmup=1)
    assert op_variant and all(len(t) >= 2 and min(t, key=t.get) == op_variant[op] for op, t in table.items())
    got, plan, _ = run_gpu(m.graph, model_feeds(m), cands, op_variant=op_variant)
    for s in plan.steps():
        if s["kernel_name"] == "GEMM_TC" and s["ops"][0] in op_variant:
            assert plan.gemm_variants(s["ops"][0])[1] == op_variant[s["ops"][0]]
    ref = run_oracle(m.graph, model_feeds(m))
    for tid in m.graph.outputs:
        assert_close(got[tid], ref[tid], synth.BF16, f"tuned-variant plan output {tid}")
    plan.close()


# ---- substitutes for a memory checker ------------------------------------------------------------------------------
@pytest.mark.parametrize("family,dtype", [("encoder", synth.F32), ("gpt", synth.BF16), ("llama", synth.BF16)])
def test_no_kernel_writes_past_its_slice(family, dtype):
    """Red zones: a plan with one disjoint slice per activation, each followed by 512 bytes no kernel may touch, run
    from an arena filled with 0xFF. Every zone still holds the pattern afterwards, the outputs are the oracle's, and
    they equal, bit for bit, those of the planned (shared-slice, in-place) arena."""
    cfg = synth.scaled(SMALL[family], dtype=dtype)
    m = synth.build_model(cfg)
    cands = synth.default_candidates(m.graph)
    got, plan, runner = run_gpu(m.graph, model_feeds(m), cands, no_reuse=1, redzone_bytes=512)
    assert runner.redzone_violations(512) == []
    assert all(r["bytes"] % 256 == 0 and r["bytes"] >= 768 for r in plan.records() if r["tensor"] >= 0)
    ref = run_oracle(m.graph, model_feeds(m))
    shared, plan2, _ = run_gpu(m.graph, model_feeds(m), cands)
    for tid in m.graph.outputs:
        assert_close(got[tid], ref[tid], dtype, f"{family} with red zones")
        assert np.array_equal(got[tid], shared[tid])
    # the check itself works: a byte scribbled into a zone is found
    rec = next(r for r in plan.records() if r["tensor"] >= 0)
    runner.arena[rec["offset"] + rec["bytes"] - 1] = 0
    assert runner.redzone_violations(512) == [rec["id"]]
    plan.close(); plan2.close()


def test_status_word_in_the_arena_header_is_reported():
    """The read-back path of the bounded waits, exercised from the host: a non-zero status word written into the arena
    header (as a kernel whose wait ran out would leave it) makes fluid_status answer FLUID_ETIMEOUT with the code;
    the next run clears it. No kernel waits on anything here."""
    import ctypes
    import torch
    m = synth.build_model(synth.CONFIGS["tiny"])
    plan = fluid.Plan(m.graph, synth.default_candidates(m.graph))
    r = fluid.Runner(plan, m.consts)
    r.set_inputs([m.ids])
    r.run()
    assert r.status() == 0
    r.arena[:4].copy_(torch.tensor([0x04, 0x01, 0, 0], dtype=torch.uint8, device="cuda"))   # word 0x104
    st = ctypes.c_int()
    rc = fluid.lib().fluid_status(plan.handle, ctypes.c_void_p(r.arena.data_ptr()), None, ctypes.byref(st))
    assert rc == fluid.FLUID_ETIMEOUT and st.value == 0x104
    assert b"0x104" in fluid.lib().fluid_last_error()
    r.arena[:4].copy_(torch.tensor([0x10, 0, 0, 0], dtype=torch.uint8, device="cuda"))      # position outside the cache
    rc = fluid.lib().fluid_status(plan.handle, ctypes.c_void_p(r.arena.data_ptr()), None, ctypes.byref(st))
    assert rc == fluid.FLUID_EINVAL and st.value == 0x10
    r.run()                                       # the header is zeroed at the start of every run
    assert r.status() == 0
    plan.close()
