"""Parity at the full sizes of the benchmark configurations, in the configuration bench.py times (planned layouts, fused
epilogues, tensor-core GEMMs): whole outputs against full passes of the fp64 oracle (minutes of host time for the two
largest shapes), and every launch on its own against the oracle op on sampled rows."""
import numpy as np
import pytest

from paper_2411_09242_b200 import fluid, synth
from tests.helpers import assert_close, check_steps_sampled, run_gpu, run_oracle, storage_hooks

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


def test_gpt2_small_shape_full():
    """Every element of the hidden state [4, 1024, 768] and of the last-token logits [4, 50257] against one full
    pass of the fp64 oracle, at the stated bf16 tolerance."""
    m = synth.build_model(synth.CONFIGS["gpt2_small"])
    ref = run_oracle(m.graph, feeds_of(m))
    got, plan, _ = run_gpu(m.graph, feeds_of(m), synth.default_candidates(m.graph))
    for t in m.graph.outputs:
        assert_close(got[t], ref[t], synth.BF16, f"gpt2_small {m.graph.tensors[t]['name']} (whole tensor)")
    assert "PERMUTE" not in [s["kernel_name"] for s in plan.steps()]
    plan.close()


def test_llama_shape_full():
    """The Llama-shaped config, whole outputs, against two full oracle passes.

    With hidden 4096 / FFN 11008 and N(0, 0.02) weights this four-layer network amplifies a relative perturbation
    of a stored activation several times over on its way to the output. (i) An fp64 run that does nothing but round
    each tensor to the dtype the plan stores it in (read from the plan: bf16 GEMM operands, fp32 residual stream,
    nothing for tensors fused away) already lands about 1.8 % of max|ref| from the unrounded oracle: the stated 1e-2
    cannot be met by any executor that keeps bf16 activations for this shape. (ii) Against that storage-rounded
    oracle the GPU differs only by arithmetic (fp32 accumulation order in the tensor core, ex2.approx) and by which
    way borderline values round; those flips (0.3 % of the first projection's elements, see the cascade test below)
    grow through the same amplification, so the two agree to about 1 %, not to a rounding unit: bounded at 1.5e-2.
    (iii) The distance to the unrounded oracle is bounded at 2.5e-2 (measured 1.86 %, the floor itself being 1.82 %)."""
    m = synth.build_model(synth.CONFIGS["llama"])
    g = m.graph
    got, plan, _ = run_gpu(g, feeds_of(m), synth.default_candidates(g))
    store, load = storage_hooks(g, plan)
    ref = run_oracle(g, feeds_of(m))
    ref_stored = run_oracle(g, feeds_of(m), store=store, load=load)
    for t in g.outputs:
        name = g.tensors[t]["name"]
        scale = float(np.max(np.abs(ref[t])))
        floor = float(np.max(np.abs(ref_stored[t] - ref[t]))) / scale
        gap = float(np.max(np.abs(got[t] - ref[t]))) / scale
        arith = float(np.max(np.abs(got[t] - ref_stored[t]))) / scale
        print(f"llama {name}: storage floor {floor:.4%}, GPU vs plain oracle {gap:.4%}, GPU vs storage-rounded oracle {arith:.4%}")
        if g.tensors[t]["dims"][-1] == m.cfg.H:
            assert floor > 1e-2, "the storage floor moved under the stated tolerance: tighten this test to 1e-2"
        assert_close(got[t], ref_stored[t], synth.BF16, f"llama {name} vs storage-rounded oracle", tol=1.5e-2)
        assert_close(got[t], ref[t], synth.BF16, f"llama {name} vs plain oracle", tol=2.5e-2)
    # Greedy-by-Size is a heuristic: with the SwiGLU step fused (gate and up never stored) it lands 15 % above the
    # largest live set on this shape; on the other three shapes it meets the bound exactly
    assert plan.live_bound_bytes <= plan.arena_bytes <= 1.2 * plan.live_bound_bytes
    plan.close()


def test_llama_first_layer_rounding_cascade():
    """Why the Llama shape agrees with the storage-rounded oracle to a per cent and not to a rounding unit. One layer
    at full widths, every tensor kept (no arena reuse), each stored tensor compared with the storage-rounded oracle's:
    the first projections differ in well under 1 % of their elements (a bf16 rounding that went the other way,
    because the tensor core's fp32 accumulation and the oracle's fp64 differ by ~1e-5 relative) and by ~2e-4 rms;
    after attention, whose output mixes thousands of such inputs, an order of magnitude more elements differ; by the
    end of the layer the difference is a few times 1e-3 rms, and the next layer starts from there. Every stored
    tensor of the layer still agrees within one bf16 unit of max|ref| (2^-7)."""
    m = synth.build_model(synth.scaled(synth.CONFIGS["llama"], L=1))
    g = m.graph
    got, plan, runner = run_gpu(g, feeds_of(m), synth.default_candidates(g), no_reuse=1)
    store, load = storage_hooks(g, plan)
    stored = run_oracle(g, feeds_of(m), keep_all=True, store=store, load=load)
    frac, rms = {}, {}
    for s in plan.steps():
        for t in s["outs"]:
            have = got[t] if g.tensors[t]["kind"] == synth.OUTPUT else runner.read_tensor(t)
            name = g.tensors[t]["name"]
            d = np.abs(have - stored[t])
            frac[name] = float(np.mean(d > 0))
            rms[name] = float(np.sqrt(np.mean(d ** 2)) / np.sqrt(np.mean(stored[t] ** 2)))
            print(f"{s['kernel_name']:10s} {name:16s} differing {frac[name]:.4f}  rms {rms[name]:.2e}  max {d.max() / np.abs(stored[t]).max():.2e}")
            assert_close(have, stored[t], synth.BF16, f"one layer, {name} vs storage-rounded oracle", tol=2 ** -7)
    assert frac["l0.v"] < 0.01 and rms["l0.v"] < 5e-4 and frac["l0.q_rope"] < 0.01
    assert frac["l0.ctx_h"] > 5 * frac["l0.v"]
    assert rms["final_norm.out"] > 5 * rms["l0.v"]
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
