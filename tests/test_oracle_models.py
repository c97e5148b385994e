"""Pins for the graph interpreter and the synthetic graph wiring: the direct per-family formulas
must give the same numbers, and whole-model invariants must hold."""
import numpy as np
import pytest

from oracle import graph_exec, models
from paper_2411_09242_b200 import synth

SMALL = {
    "encoder": synth.scaled(synth.CONFIGS["tiny"], L=2, H=32, nh=2, F=64, S=8, B=2, V=50),
    "gpt": synth.scaled(synth.CONFIGS["gpt2_small"], L=2, H=32, nh=4, F=64, S=8, B=2, V=50, dtype=synth.F32),
    "llama": synth.scaled(synth.CONFIGS["llama"], L=2, H=32, nh=2, F=48, S=8, B=2, V=50, dtype=synth.F32),
}


def run(model, ids=None, consts=None):
    g = model.graph
    feeds = dict(consts if consts is not None else model.consts)
    feeds[g.inputs[0]] = model.ids if ids is None else ids
    out = graph_exec.run_graph(g.tensors, g.ops, feeds)
    return [out[t] for t in g.outputs]


def named(model):
    return {model.graph.tensors[t]["name"]: a for t, a in model.consts.items()}


@pytest.mark.parametrize("family", ["encoder", "gpt", "llama"])
def test_graph_matches_direct_formula(family):
    m = synth.build_model(SMALL[family])
    outs = run(m)
    h, logits = models.forward(family, m.cfg.L, named(m), m.ids)
    np.testing.assert_allclose(outs[0], h, rtol=1e-10, atol=1e-12)
    if logits is not None:
        np.testing.assert_allclose(outs[1], logits, rtol=1e-10, atol=1e-12)
    assert np.all(np.isfinite(outs[0])) and outs[0].std() > 0.1


@pytest.mark.parametrize("family", ["gpt", "llama"])
def test_causality(family):
    m = synth.build_model(SMALL[family])
    ids2 = m.ids.copy()
    ids2[:, 5:] = (ids2[:, 5:] + 7) % m.cfg.V
    a, b = run(m)[0], run(m, ids=ids2)[0]
    assert np.array_equal(a[:, :5], b[:, :5])
    assert not np.allclose(a[:, 5:], b[:, 5:])


@pytest.mark.parametrize("family", ["encoder", "gpt", "llama"])
def test_batch_independence(family):
    m = synth.build_model(SMALL[family])
    full = run(m)[0]
    one = synth.build_model(synth.scaled(SMALL[family], B=1))
    for t in one.consts:                   # same tensor ids -> same seeded weights
        assert np.array_equal(one.consts[t], m.consts[t])
    for b in range(2):
        np.testing.assert_allclose(run(one, ids=m.ids[b:b + 1])[0][0], full[b], rtol=1e-12, atol=1e-13)


def test_encoder_permutation_equivariant_without_positions():
    m = synth.build_model(SMALL["encoder"])
    consts = dict(m.consts)
    pos_id = next(t for t, d in enumerate(m.graph.tensors) if d["name"] == "pos_table")
    consts[pos_id] = np.zeros_like(consts[pos_id])
    perm = np.random.default_rng(0).permutation(m.cfg.S)
    a = run(m, consts=consts)[0]
    b = run(m, ids=m.ids[:, perm], consts=consts)[0]
    np.testing.assert_allclose(b, a[:, perm], rtol=1e-11, atol=1e-12)


def test_torch_float64_second_opinion_on_tiny():
    torch = pytest.importorskip("torch")
    m = synth.build_model(synth.CONFIGS["tiny"])
    w = {k: torch.tensor(v, dtype=torch.float64) for k, v in named(m).items()}
    cfg = m.cfg
    x = w["tok_table"][torch.tensor(m.ids, dtype=torch.long)] + w["pos_table"][None]
    F = torch.nn.functional
    x = F.layer_norm(x, (cfg.H,), w["emb_ln.gamma"], w["emb_ln.beta"], 1e-5)
    for l in range(cfg.L):
        p = f"l{l}"
        q, k, v = (torch.einsum("bsk,khd->bhsd", x, w[f"{p}.W{n}"]) + w[f"{p}.b{n}"][None, :, None, :] for n in "qkv")
        c = F.scaled_dot_product_attention(q, k, v).permute(0, 2, 1, 3)
        o = torch.einsum("bshd,hdn->bsn", c, w[f"{p}.Wo"]) + w[f"{p}.bo"]
        x = F.layer_norm(x + o, (cfg.H,), w[f"{p}.ln1.gamma"], w[f"{p}.ln1.beta"], 1e-5)
        o = F.gelu(x @ w[f"{p}.W1"] + w[f"{p}.b1"]) @ w[f"{p}.W2"] + w[f"{p}.b2"]
        x = F.layer_norm(x + o, (cfg.H,), w[f"{p}.ln2.gamma"], w[f"{p}.ln2.beta"], 1e-5)
    np.testing.assert_allclose(run(m)[0], x.numpy(), rtol=1e-10, atol=1e-11)


def test_synth_is_seeded_and_bf16_representable():
    a = synth.build_model(SMALL["encoder"]); b = synth.build_model(SMALL["encoder"])
    assert all(np.array_equal(a.consts[t], b.consts[t]) for t in a.consts) and np.array_equal(a.ids, b.ids)
    m = synth.build_model(synth.scaled(SMALL["encoder"], dtype=synth.BF16))
    for t, arr in m.consts.items():
        assert np.array_equal(synth.round_bf16(arr), arr)
    x = np.array([1.0, 1.00390625, 1.005859375, -3.1415927, 65504.0, 1e-30], dtype=np.float32)
    torch = pytest.importorskip("torch")
    ref = torch.tensor(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(synth.round_bf16(x), ref)
    gam = next(arr for t, arr in a.consts.items() if a.graph.tensors[t]["name"].endswith("ln1.gamma"))
    assert abs(gam.mean() - 1.0) < 0.02
    assert a.ids.min() >= 0 and a.ids.max() < a.cfg.V


def test_sweep_graphs():
    g, a = synth.permute_case(2, 4, 3, 8, "BHDS", dtype=synth.F32)
    out = graph_exec.run_graph(g.tensors, g.ops, {g.inputs[0]: a})
    assert np.array_equal(out[g.outputs[0]], np.transpose(a, (0, 2, 3, 1)))
    for am in ("row", "col"):
        for bm in ("row", "col"):
            g, arrs = synth.gemm_case(6, 5, 4, am, bm, dtype=synth.F32)
            out = graph_exec.run_graph(g.tensors, g.ops, arrs)[g.outputs[0]]
            g0, arr0 = synth.gemm_case(6, 5, 4, "row", "row", dtype=synth.F32)
            ref = graph_exec.run_graph(g0.tensors, g0.ops, arr0)[g0.outputs[0]]
            assert np.array_equal(out, ref)
    assert len(list(synth.permute_sweep_cases())) == 192
