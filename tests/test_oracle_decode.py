"""Pins of the oracle's decoding step (key/value cache): everything here runs on the CPU.

The cached step has a plain definition through something that is pinned elsewhere: decoding token t with
the keys and values of tokens 0..t-1 cached must give the row for position t of causal attention over the
whole prefix. So a run of decoding steps through the graph interpreter is compared with the direct
whole-sequence model formulas (oracle/models.py, itself pinned against the graph interpreter and by
invariants), and the operator alone with brute-force loops.
"""
import math

import numpy as np
import pytest

from oracle import graph_exec, models, ops
from paper_2411_09242_b200 import synth


def _brute_cached(q, k, v, kc, vc, t, scale):
    B, _, nh, D = q.shape
    nkv = kc.shape[2]
    kc, vc = kc.copy(), vc.copy()
    out = np.zeros_like(q)
    for b in range(B):
        for g in range(nkv):
            for d in range(D):
                kc[b, t, g, d] = k[b, 0, g, d]
                vc[b, t, g, d] = v[b, 0, g, d]
        for h in range(nh):
            g = h // (nh // nkv)
            sc = []
            for j in range(t + 1):
                acc = 0.0
                for d in range(D):
                    acc += q[b, 0, h, d] * kc[b, j, g, d]
                sc.append(acc * scale)
            m = max(sc)
            e = [math.exp(x - m) for x in sc]
            z = sum(e)
            for d in range(D):
                out[b, 0, h, d] = sum(e[j] / z * vc[b, j, g, d] for j in range(t + 1))
    return out, kc, vc


@pytest.mark.parametrize("nh,nkv,t", [(4, 4, 0), (4, 4, 5), (6, 2, 3), (4, 1, 6)])
def test_cached_attention_against_loops(nh, nkv, t):
    rng = np.random.default_rng(nh * 100 + nkv * 10 + t)
    B, D, Tmax = 2, 8, 7
    q = rng.standard_normal((B, 1, nh, D))
    k = rng.standard_normal((B, 1, nkv, D))
    v = rng.standard_normal((B, 1, nkv, D))
    kc = rng.standard_normal((B, Tmax, nkv, D))
    vc = rng.standard_normal((B, Tmax, nkv, D))
    got = ops.cached_attention(q, k, v, kc, vc, np.array([t]), scale=0.37)
    ref = _brute_cached(q, k, v, kc, vc, t, 0.37)
    for a, b in zip(got, ref):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-12)
    # rows other than t are untouched, rows after t play no part
    assert np.array_equal(got[1][:, :t], kc[:, :t]) and np.array_equal(got[1][:, t + 1:], kc[:, t + 1:])
    kc2, vc2 = kc.copy(), vc.copy()
    kc2[:, t + 1:] = 1e30
    vc2[:, t + 1:] = -1e30
    again = ops.cached_attention(q, k, v, kc2, vc2, np.array([t]), scale=0.37)
    assert np.array_equal(again[0], got[0])


def test_cached_attention_is_the_last_row_of_causal_attention():
    rng = np.random.default_rng(3)
    B, T, nh, D = 2, 9, 3, 16
    q = rng.standard_normal((B, T, nh, D))
    k = rng.standard_normal((B, T, nh, D))
    v = rng.standard_normal((B, T, nh, D))
    s = np.einsum("bihd,bjhd->bhij", q, k) / math.sqrt(D)
    full = np.einsum("bhij,bjhd->bihd", ops.softmax(s, causal=True), v)
    kc = np.zeros((B, T, nh, D))
    vc = np.zeros((B, T, nh, D))
    for t in range(T):
        ctx, kc, vc = ops.cached_attention(q[:, t:t + 1], k[:, t:t + 1], v[:, t:t + 1], kc, vc, [t], scale=1 / math.sqrt(D))
        np.testing.assert_allclose(ctx[:, 0], full[:, t], rtol=1e-12, atol=1e-13)
    assert np.array_equal(kc, k) and np.array_equal(vc, v)


def test_rope_with_an_offset_is_a_slice_of_the_whole_sequence():
    rng = np.random.default_rng(4)
    x = rng.standard_normal((2, 11, 3, 8))
    for inter in (False, True):
        whole = ops.rope(x, base=500.0, interleaved=inter)
        for p0 in (0, 1, 7):
            part = ops.rope(x[:, p0:p0 + 3], base=500.0, interleaved=inter, pos0=p0)
            np.testing.assert_allclose(part, whole[:, p0:p0 + 3], rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("family", ["llama", "gpt2_small"])
def test_decoding_steps_reproduce_the_whole_sequence_model(family):
    """S decoding steps from empty caches give, at step t, the logits of the whole-sequence model run on the
    first t+1 tokens; the caches end up holding the (rotated) keys and the values of the whole sequence."""
    cfg = synth.scaled(synth.CONFIGS[family], dtype=synth.F32, L=2, H=32, nh=4, F=48, S=6, B=2, V=50)
    whole = synth.build_model(cfg)
    dec = synth.build_decode_model(cfg, t_max=8, like=whole)
    g = dec.graph
    names = {whole.graph.tensors[t]["name"]: a for t, a in whole.consts.items()}
    state = {t: np.full(g.dims(t), np.nan) for pair in dec.caches for t in pair}   # unwritten rows must not matter
    for t in range(cfg.S):
        feeds = dict(dec.consts)
        feeds[dec.ids] = whole.ids[:, t:t + 1]
        feeds[dec.pos] = np.array([t], dtype=np.int32)
        # rows >= t are unspecified on entry: hand over garbage there, not NaN (0 * NaN would leak)
        for tid, a in state.items():
            a = a.copy()
            a[:, t:] = 7.0
            feeds[tid] = a
        out = graph_exec.run_graph(g.tensors, g.ops, feeds)
        for tid in state:
            state[tid] = out[tid]
        logits = out[g.outputs[1]]
        _, ref_logits = models.forward(cfg.family, cfg.L, names, whole.ids[:, :t + 1])
        np.testing.assert_allclose(logits[:, 0], ref_logits, rtol=1e-9, atol=1e-12)
    vals = graph_exec.run_graph(whole.graph.tensors, whole.graph.ops, {**whole.consts, whole.graph.inputs[0]: whole.ids}, keep_all=True)
    by_name = {td["name"]: vals[t] for t, td in enumerate(whole.graph.tensors) if t in vals}
    for l, (kc, vc) in enumerate(dec.caches):
        np.testing.assert_allclose(state[kc][:, :cfg.S], by_name[f"l{l}.k_rope" if cfg.family == "llama" else f"l{l}.k"], rtol=1e-9, atol=1e-12)
        np.testing.assert_allclose(state[vc][:, :cfg.S], by_name[f"l{l}.v"], rtol=1e-9, atol=1e-12)


def test_positions_per_sequence_equal_each_sequence_alone():
    rng = np.random.default_rng(9)
    B, nh, D, Tmax = 3, 2, 8, 10
    q = rng.standard_normal((B, 1, nh, D)); k = rng.standard_normal((B, 1, nh, D)); v = rng.standard_normal((B, 1, nh, D))
    kc = rng.standard_normal((B, Tmax, nh, D)); vc = rng.standard_normal((B, Tmax, nh, D))
    pos = np.array([0, 9, 4])
    ctx, kc2, vc2 = ops.cached_attention(q, k, v, kc, vc, pos, scale=0.5)
    for b in range(B):
        one = ops.cached_attention(q[b:b + 1], k[b:b + 1], v[b:b + 1], kc[b:b + 1], vc[b:b + 1], [pos[b]], scale=0.5)
        assert np.array_equal(ctx[b:b + 1], one[0]) and np.array_equal(kc2[b:b + 1], one[1]) and np.array_equal(vc2[b:b + 1], one[2])
    x = rng.standard_normal((B, 2, nh, D))
    r = ops.rope(x, base=100.0, pos0=pos)
    for b in range(B):
        np.testing.assert_allclose(r[b:b + 1], ops.rope(x[b:b + 1], base=100.0, pos0=int(pos[b])), rtol=1e-14, atol=1e-14)


def test_embedding_with_a_position_offset_is_a_slice_of_the_whole_sequence():
    rng = np.random.default_rng(6)
    tok, pos = rng.standard_normal((20, 8)), rng.standard_normal((12, 8))
    ids = rng.integers(0, 20, size=(2, 12))
    whole = ops.embed(ids, tok, pos)
    for p0 in (0, 3, 9):
        np.testing.assert_array_equal(ops.embed(ids[:, p0:p0 + 2], tok, pos, pos0=p0), whole[:, p0:p0 + 2])
    both = ops.embed(np.stack([ids[0, 3:5], ids[1, 7:9]]), tok, pos, pos0=[3, 7])
    np.testing.assert_array_equal(both, np.stack([whole[0, 3:5], whole[1, 7:9]]))
