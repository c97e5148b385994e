"""The oracle's storage-rounding mode (graph_exec.run_graph(store=, load=)) and the hooks that derive it from a plan.

The parity reference never rounds. This mode exists to separate two things a device run mixes: the rounding of
what a plan *stores* (bf16 operands, fp32 residual stream) and arithmetic error proper. Host-only: the planner runs
on the CPU, nothing here launches a kernel."""
import numpy as np

from paper_2411_09242_b200 import fluid, synth
from tests.helpers import ensure_lib, run_oracle, storage_hooks


def _feeds(m):
    f = dict(m.consts)
    f[m.graph.inputs[0]] = m.ids
    return f


def _is_bf16(a):
    return np.array_equal(synth.round_bf16(np.asarray(a, np.float32)).astype(np.float64), a)


def _is_f32(a):
    return np.array_equal(np.asarray(a, np.float32).astype(np.float64), a)


def test_hooks_round_exactly_what_the_plan_stores():
    ensure_lib()
    cfg = synth.scaled(synth.CONFIGS["llama"], L=2, H=256, nh=4, F=512, S=128, V=512)
    m = synth.build_model(cfg)
    g = m.graph
    plan = fluid.Plan(g, synth.default_candidates(g))
    store, load = storage_hooks(g, plan)
    plain = run_oracle(g, _feeds(m), keep_all=True)
    stored = run_oracle(g, _feeds(m), keep_all=True, store=store, load=load)
    recs = {r["tensor"]: r["dtype"] for r in plan.records() if r["tensor"] >= 0 and not r["twin"]}
    step_outs = {t for s in plan.steps() for t in s["outs"]}
    n_bf16 = n_wide = n_folded = 0
    wide_only = False                           # some wide tensor really carries more than bf16 precision
    for t, td in enumerate(g.tensors):
        if td["kind"] != synth.ACT:
            continue
        dt = recs.get(plan.tensor_info(t).alias_of)
        if dt == synth.BF16:
            assert _is_bf16(stored[t]), td["name"]
            n_bf16 += 1
        elif dt == synth.F32:
            assert _is_f32(stored[t]), td["name"]
            wide_only |= not _is_bf16(stored[t])
            n_wide += 1
        else:                                   # folded into a fused step: never stored, never rounded
            assert t not in step_outs and not _is_f32(stored[t]), td["name"]
            n_folded += 1
    assert n_bf16 and n_wide and n_folded and wide_only
    for t in g.outputs:
        assert _is_bf16(stored[t])
        floor = np.max(np.abs(stored[t] - plain[t])) / np.max(np.abs(plain[t]))
        assert 0 < floor < 1e-2                 # two narrow layers: rounding is visible and small
    # without hooks the executor is the plain definition, bit for bit
    again = run_oracle(g, _feeds(m), keep_all=True)
    assert all(np.array_equal(again[t], plain[t]) for t in plain)
    plan.close()


def test_twin_tensors_are_read_narrow_by_gemms_and_wide_by_the_stream():
    ensure_lib()
    m = synth.build_model(synth.scaled(synth.CONFIGS["bert_base"], L=1, S=32, V=256))   # post-LN: LN output feeds a GEMM and a residual add
    g = m.graph
    plan = fluid.Plan(g, synth.default_candidates(g))
    twins = {r["tensor"] for r in plan.records() if r["twin"]}
    assert twins
    _, load = storage_hooks(g, plan)
    t = next(iter(twins))
    x = np.full(g.tensors[t]["dims"], 1.0 + 2.0 ** -12)               # fp32-exact, not bf16-exact
    gemm = next(i for i, o in enumerate(g.ops) if o["kind"] == synth.LINEAR and t in o["ins"])
    other = next(i for i, o in enumerate(g.ops) if o["kind"] != synth.LINEAR and t in o["ins"])
    assert np.all(load(gemm, t, x) == 1.0) and np.array_equal(load(other, t, x), x)
    plan.close()


def test_llama_width_storage_floor_exceeds_the_stated_tolerance():
    """The Llama-shaped config at its full widths (hidden 4096, FFN 11008, 32 heads of 128, 4 layers), first 64
    positions (causal: exactly the first 64 rows of the full sequence). Exact fp64 arithmetic with the plan's
    storage dtypes misses the unrounded oracle by more than the stated 1e-2 of max|ref|: the bar is out of reach
    for this shape whatever the kernels do. (About a minute of host time, most of it generating 2 GB of weights.)"""
    ensure_lib()
    m = synth.build_model(synth.scaled(synth.CONFIGS["llama"], S=64))
    g = m.graph
    plan = fluid.Plan(g, synth.default_candidates(g))
    store, load = storage_hooks(g, plan)
    plain = run_oracle(g, _feeds(m))
    stored = run_oracle(g, _feeds(m), store=store, load=load)
    hidden = g.outputs[0]
    floor = np.max(np.abs(stored[hidden] - plain[hidden])) / np.max(np.abs(plain[hidden]))
    print(f"llama widths, 64 positions: storage floor {floor:.4%} of max|ref|")
    assert 1e-2 < floor < 3e-2
    plan.close()
