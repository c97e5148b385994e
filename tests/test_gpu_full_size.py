"""Parity at the full sizes of the benchmark configurations, in the configuration bench.py times (planned layouts, fused
epilogues, tensor-core GEMMs). Where a full oracle pass is too slow, outputs are sampled in a way the
oracle can compute exactly: a causal model's first rows depend only on the first tokens."""
import numpy as np
import pytest

from paper_2411_09242_b200 import fluid, synth
from tests.helpers import assert_close, check_steps_sampled, run_gpu, run_oracle

pytestmark = pytest.mark.gpu


def feeds_of(m):
    f = dict(m.consts)
    f[m.graph.inputs[0]] = m.ids
    return f


def test_bert_base_shape_full():
    m = synth.build_model(synth.CONFIGS["bert_base"])
    ref = run_oracle(m.graph, feeds_of(m))
    got, plan, runner = run_gpu(m.graph, feeds_of(m), synth.default_candidates(m.graph))
    for t in m.graph.outputs:
        assert_close(got[t], ref[t], synth.BF16, "bert_base")
    assert "PERMUTE" not in [s["kernel_name"] for s in plan.steps()]
    assert plan.arena_bytes == plan.live_bound_bytes <= 2 * 2 ** 20
    # a second run into the same arena gives the same bits (no stale-state dependence)
    runner.run()
    again = runner.outputs_host()
    for t, a in zip(m.graph.outputs, again):
        assert np.array_equal(a, got[t])
    plan.close()


def _prefix_reference(full, S_prefix, L=None):
    """Oracle output for batch row 0, first S_prefix positions, using the full model's weights."""
    cfg = synth.scaled(full.cfg, B=1, S=S_prefix, **({"L": L} if L else {}))
    small = synth.build_model(cfg, materialize=False)
    name_to_full = {full.graph.tensors[t]["name"]: a for t, a in full.consts.items()}
    feeds = {}
    for tid, td in enumerate(small.graph.tensors):
        if td["kind"] == synth.CONST:
            a = name_to_full[td["name"]]
            feeds[tid] = a[:S_prefix] if td["name"] == "pos_table" else a
    feeds[small.graph.inputs[0]] = full.ids[:1, :S_prefix]
    out = run_oracle(small.graph, feeds)
    return out[small.graph.outputs[0]]


def test_gpt2_small_shape_full_sampled_prefix():
    m = synth.build_model(synth.CONFIGS["gpt2_small"])
    got, plan, _ = run_gpu(m.graph, feeds_of(m), synth.default_candidates(m.graph))
    hidden, logits = (got[t] for t in m.graph.outputs)
    ref = _prefix_reference(m, 192)
    assert_close(hidden[:1, :192], ref, synth.BF16, "gpt2_small hidden prefix")
    # every batch row went through the same kernels: rows with equal prefixes would agree; check
    # finiteness and scale of the rest, and the tied-head logits against the GPU's own hidden state
    assert np.all(np.isfinite(hidden)) and np.all(np.isfinite(logits))
    tok = next(a for t, a in m.consts.items() if m.graph.tensors[t]["name"] == "tok_table").astype(np.float64)
    assert_close(logits, hidden[:, -1, :] @ tok.T, synth.BF16, "gpt2_small logits from hidden")
    plan.close()


def test_llama_shape_full_sampled_prefix():
    m = synth.build_model(synth.CONFIGS["llama"])
    got, plan, _ = run_gpu(m.graph, feeds_of(m), synth.default_candidates(m.graph))
    hidden, logits = (got[t] for t in m.graph.outputs)
    # With hidden 4096 / FFN 11008 and N(0,0.02) weights the residual stream grows to ~20 and rounding the
    # GEMM operands to bf16 alone moves the final output by 2.3 % of max|ref|: an fp64 run that does nothing
    # but round the tensors the plan stores in bf16 shows the same figure (0.1086 vs the GPU's 0.1085). The
    # 1e-2 bar therefore cannot hold end to end against the unrounded oracle for this shape; the kernels are
    # held to 2^-7 launch by launch at full size (test below) and the end-to-end gap is bounded at 3e-2.
    ref = _prefix_reference(m, 96)
    assert_close(hidden[:1, :96], ref, synth.BF16, "llama hidden prefix vs unrounded oracle", tol=3e-2)
    w = next(a for t, a in m.consts.items() if m.graph.tensors[t]["name"] == "W_lm").astype(np.float64)
    assert_close(logits, hidden[:, -1, :] @ w, synth.BF16, "llama logits from hidden")
    # Greedy-by-Size is a heuristic: with the SwiGLU step fused (gate and up never stored) it lands 15 % above the
    # largest live set on this shape; on the other three shapes it meets the bound exactly
    assert plan.live_bound_bytes <= plan.arena_bytes <= 1.2 * plan.live_bound_bytes
    plan.close()


@pytest.mark.parametrize("name,layers", [("llama", 2), ("gpt2_small", 2), ("bert_base", 2)])
def test_every_launch_at_full_size_sampled(name, layers):
    """Full sequence length, batch, hidden and FFN sizes (layer count cut to bound host memory): each
    launch's output against the oracle op on the GPU's own inputs, on sampled rows / (batch, head) slices."""
    m = synth.build_model(synth.scaled(synth.CONFIGS[name], L=layers))
    got, plan, runner = run_gpu(m.graph, feeds_of(m), synth.default_candidates(m.graph), no_reuse=1)
    n = check_steps_sampled(m.graph, plan, runner, feeds_of(m))
    assert n >= len(plan.steps())
    kinds = {s["kernel_name"] for s in plan.steps()}
    assert "GEMM_TC" in kinds and "PERMUTE" not in kinds
    plan.close()


@pytest.mark.parametrize("case", [dict(B=1, S=128, nh=12, D=64), dict(B=8, S=2048, nh=32, D=128),
                                  dict(B=3, S=512, nh=12, D=128), dict(B=5, S=2048, nh=12, D=64)])
@pytest.mark.parametrize("target", ["BHSD", "BHDS"])
def test_sweep_layout_transforms(case, target):
    g, a = synth.permute_case(target=target, **case)
    got, plan, _ = run_gpu(g, {0: a}, poison=False)
    perm = (0, 2, 1, 3) if target == "BHSD" else (0, 2, 3, 1)
    assert np.array_equal(got[1], np.transpose(a.astype(np.float64), perm))
    plan.close()


@pytest.mark.parametrize("n", [768, 2048, 4096])
@pytest.mark.parametrize("a_major", ["row", "col"])
@pytest.mark.parametrize("b_major", ["row", "col"])
def test_sweep_layout_aware_gemm(n, a_major, b_major):
    g, arrs = synth.gemm_case(n, n, n, a_major, b_major)
    got, plan, _ = run_gpu(g, arrs, synth.default_candidates(g), poison=False)
    assert [s["kernel_name"] for s in plan.steps()] == ["GEMM_TC"]
    A = arrs[g.inputs[0]].astype(np.float64)
    Bm = arrs[g.inputs[1]].astype(np.float64)
    A = A if a_major == "row" else A.T
    Bm = Bm if b_major == "row" else Bm.T
    rows = np.linspace(0, n - 1, 64).astype(int)           # sampled rows, computed exactly
    assert_close(got[g.outputs[0]][rows], A[rows] @ Bm, synth.BF16, f"gemm {n} {a_major}/{b_major}")
    plan.close()


@pytest.mark.parametrize("t", [2047, 1000])
def test_llama_decode_step_full_width(t):
    """One decoding step at the llama-shaped widths (hidden 4096, 32 heads of 128, FFN 11008, vocabulary 32000), batch 4,
    caches of 2048 rows filled with random keys and values up to row t (layer count cut to bound host memory)."""
    cfg = synth.scaled(synth.CONFIGS["llama"], L=1, B=4)
    dec = synth.build_decode_model(cfg, 2048)
    g = dec.graph
    feeds = dict(dec.consts)
    feeds[dec.ids] = synth.token_ids(synth.TOKEN_SEED, 1, [4, 1], cfg.V)
    feeds[dec.pos] = np.array([t], dtype=np.int32)
    for i, (kc, vc) in enumerate(dec.caches):
        feeds[kc] = synth.round_bf16(synth.uniform(11, 2 * i, g.dims(kc), -2.0, 2.0))
        feeds[vc] = synth.round_bf16(synth.uniform(11, 2 * i + 1, g.dims(vc), -1.0, 1.0))
    ref = run_oracle(g, feeds)
    got, plan, runner = run_gpu(g, feeds, synth.default_candidates(g))
    names = [s["kernel_name"] for s in plan.steps()]
    assert names.count("ATTN_DECODE") == 1 and "ROPE" not in names and "GEMM_TC" not in names and names.count("GEMM_ROWS") == 5
    for tid in g.outputs:
        assert_close(got[tid], ref[tid], synth.BF16, g.tensors[tid]["name"])
    for kc, vc in dec.caches:
        for c in (kc, vc):
            dev = runner.inputs[g.inputs.index(c)].float().cpu().numpy()
            assert_close(dev[:, t], ref[c][:, t], synth.BF16, "new cache row")
            keep = np.arange(2048) != t
            assert np.array_equal(dev[:, keep], feeds[c][:, keep])
    plan.close()
