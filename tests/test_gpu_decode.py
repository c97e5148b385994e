"""Parity of the decoding path (key/value cache) on the GPU against the CPU oracle, through the C-ABI."""
import math

import numpy as np
import pytest

from paper_2411_09242_b200 import fluid, synth
from tests import helpers

pytestmark = pytest.mark.gpu


def _cached_graph(B, nh, nkv, D, Tmax, dtype):
    g = synth.GraphDesc()
    q = g.tensor("q", dtype, [B, 1, nh, D], synth.INPUT)
    k = g.tensor("k", dtype, [B, 1, nkv, D], synth.INPUT)
    v = g.tensor("v", dtype, [B, 1, nkv, D], synth.INPUT)
    kc = g.tensor("kc", dtype, [B, Tmax, nkv, D], synth.STATE)
    vc = g.tensor("vc", dtype, [B, Tmax, nkv, D], synth.STATE)
    pos = g.tensor("pos", synth.I32, [1], synth.INPUT)
    out = g.tensor("ctx", dtype, [B, 1, nh, D], synth.OUTPUT)
    g.op(synth.CACHED_ATTENTION, [q, k, v, kc, vc, pos], [out], scale=1.0 / math.sqrt(D))
    return g, (q, k, v, kc, vc, pos, out)


@pytest.mark.parametrize("B,nh,nkv,D,Tmax,dtype,ts", [
    (2, 8, 8, 128, 700, synth.BF16, (0, 1, 5, 127, 128, 255, 256, 699)),
    (3, 8, 2, 128, 300, synth.BF16, (0, 17, 299)),
    (2, 12, 12, 64, 1100, synth.BF16, (0, 63, 64, 1023, 1099)),
    (1, 6, 3, 32, 90, synth.F32, (0, 7, 89)),
    (2, 4, 4, 8, 40, synth.F32, (0, 3, 39)),
    (1, 2, 1, 128, 50, synth.F32, (0, 33, 49)),
])
def test_cached_attention_step(B, nh, nkv, D, Tmax, dtype, ts):
    g, (q, k, v, kc, vc, pos, out) = _cached_graph(B, nh, nkv, D, Tmax, dtype)
    helpers.ensure_lib()
    plan = fluid.Plan(g, synth.default_candidates(g))
    assert [s["kernel_name"] for s in plan.steps()] == ["ATTN_DECODE"]
    runner = fluid.Runner(plan, {}, poison=True)
    for t in ts:
        feeds = {q: helpers.rand_feed([B, 1, nh, D], dtype, 10 + t, -2, 2), k: helpers.rand_feed([B, 1, nkv, D], dtype, 20 + t, -2, 2),
                 v: helpers.rand_feed([B, 1, nkv, D], dtype, 30 + t), kc: helpers.rand_feed([B, Tmax, nkv, D], dtype, 40 + t, -2, 2),
                 vc: helpers.rand_feed([B, Tmax, nkv, D], dtype, 50 + t), pos: np.array([t], dtype=np.int32)}
        # rows past t are unspecified: huge values there would wreck the result if they were read
        dev = {x: a.copy() for x, a in feeds.items()}
        dev[kc][:, t + 1:] = 32768.0
        dev[vc][:, t + 1:] = -32768.0
        runner.set_inputs([dev[x] for x in g.inputs])
        runner.run()
        got = runner.outputs_host()[0]
        assert runner.status() == 0
        ref = helpers.run_oracle(g, feeds)
        helpers.assert_close(got, ref[out], dtype, f"ctx t={t}")
        # caches: row t is the new key / value bit for bit, every other row is untouched
        kc_dev = runner.inputs[g.inputs.index(kc)].float().cpu().numpy()
        vc_dev = runner.inputs[g.inputs.index(vc)].float().cpu().numpy()
        assert np.array_equal(kc_dev[:, t], feeds[k][:, 0]) and np.array_equal(vc_dev[:, t], feeds[v][:, 0])
        keep = np.ones(Tmax, bool)
        keep[t] = False
        assert np.array_equal(kc_dev[:, keep], dev[kc][:, keep]) and np.array_equal(vc_dev[:, keep], dev[vc][:, keep])
    plan.close()


@pytest.mark.parametrize("B,nh", [(25, 8), (10, 12), (10, 10), (10, 8), (7, 10), (6, 10), (37, 16)])
def test_cached_attention_every_cluster_size(B, nh):
    """The number of CTAs that share a head's rows follows the head count (1 to 8, powers of two or not)."""
    D, Tmax, t = 64, 131, 130
    g, (q, k, v, kc, vc, pos, out) = _cached_graph(B, nh, nh, D, Tmax, synth.BF16)
    feeds = {q: helpers.rand_feed([B, 1, nh, D], synth.BF16, 1, -2, 2), k: helpers.rand_feed([B, 1, nh, D], synth.BF16, 2, -2, 2),
             v: helpers.rand_feed([B, 1, nh, D], synth.BF16, 3), kc: helpers.rand_feed([B, Tmax, nh, D], synth.BF16, 4, -2, 2),
             vc: helpers.rand_feed([B, Tmax, nh, D], synth.BF16, 5), pos: np.array([t], dtype=np.int32)}
    got, plan, _ = helpers.run_gpu(g, feeds, synth.default_candidates(g))
    helpers.assert_close(got[out], helpers.run_oracle(g, feeds)[out], synth.BF16, f"{B}x{nh}")
    plan.close()


def test_position_outside_the_cache_is_reported_and_nothing_is_written():
    g, (q, k, v, kc, vc, pos, out) = _cached_graph(1, 4, 4, 64, 32, synth.BF16)
    helpers.ensure_lib()
    plan = fluid.Plan(g, synth.default_candidates(g))
    runner = fluid.Runner(plan, {})
    for bad in (-1, 32, 1000):
        feeds = [np.zeros(g.dims(t), np.float32) for t in g.inputs]
        feeds[g.inputs.index(pos)] = np.array([bad], dtype=np.int32)
        feeds[g.inputs.index(kc)] += 1.0
        runner.set_inputs(feeds)
        runner.run()
        with pytest.raises(fluid.FluidError):
            runner.status()
        assert float(runner.inputs[g.inputs.index(kc)].float().min()) == 1.0
    plan.close()


@pytest.mark.parametrize("dtype,D", [(synth.BF16, 128), (synth.BF16, 64), (synth.F32, 16)])
def test_rope_with_a_position_read_on_the_device(dtype, D):
    g = synth.GraphDesc()
    x = g.tensor("x", dtype, [2, 3, 4, D], synth.INPUT)
    pos = g.tensor("pos", synth.I32, [1], synth.INPUT)
    y = g.tensor("y", dtype, [2, 3, 4, D], synth.OUTPUT)
    g.op(synth.ROPE, [x, pos], [y], rope_base=10000.0, rope_interleaved=0)
    for p0 in (0, 5, 2047):
        feeds = {x: helpers.rand_feed([2, 3, 4, D], dtype, 3), pos: np.array([p0], dtype=np.int32)}
        got, plan, _ = helpers.run_gpu(g, feeds)
        helpers.assert_close(got[y], helpers.run_oracle(g, feeds)[y], dtype, f"rope pos {p0}")
        plan.close()


@pytest.mark.parametrize("family,dtype,kw", [
    ("llama", synth.F32, dict(L=2, H=64, nh=4, F=96, B=2, V=100)),
    ("llama", synth.BF16, dict(L=2, H=256, nh=4, F=384, B=3, V=500)),
    ("llama", synth.BF16, dict(L=1, H=512, nh=4, F=1024, B=1, V=1000)),
    ("gpt2_small", synth.F32, dict(L=2, H=64, nh=4, F=96, B=2, V=100)),
    ("gpt2_small", synth.BF16, dict(L=2, H=256, nh=4, F=512, B=3, V=501)),
])
def test_decoding_steps_of_a_small_model(family, dtype, kw):
    """Several decoding steps in a row on one plan: the caches the device carries forward are its own; every
    step's logits are compared with the oracle run on the oracle's own caches."""
    cfg = synth.scaled(synth.CONFIGS[family], dtype=dtype, S=1, **kw)
    t_max = 24
    dec = synth.build_decode_model(cfg, t_max)
    g = dec.graph
    helpers.ensure_lib()
    plan = fluid.Plan(g, synth.default_candidates(g))
    names = [s["kernel_name"] for s in plan.steps()]
    assert names.count("ATTN_DECODE") == cfg.L
    runner = fluid.Runner(plan, dec.consts, poison=True)
    rng = np.random.default_rng(1)
    state_ids = [t for pair in dec.caches for t in pair]
    oracle_state = {t: np.zeros(g.dims(t)) for t in state_ids}
    for t in state_ids:   # the device's unwritten rows hold NaN patterns
        runner.inputs[g.inputs.index(t)].fill_(float("nan"))
    for step in range(7):
        ids = rng.integers(0, cfg.V, size=(cfg.B, 1)).astype(np.int32)
        feeds = dict(dec.consts)
        feeds[dec.ids] = ids
        feeds[dec.pos] = np.array([step], dtype=np.int32)
        feeds.update(oracle_state)
        ref = helpers.run_oracle(g, feeds)
        for t in state_ids:
            oracle_state[t] = ref[t]
        runner.inputs[g.inputs.index(dec.ids)].copy_(fluid.to_device(ids, synth.I32, "cuda"))
        runner.inputs[g.inputs.index(dec.pos)].copy_(fluid.to_device(feeds[dec.pos], synth.I32, "cuda"))
        runner.run()
        outs = runner.outputs_host()
        assert runner.status() == 0
        for tid, got in zip(g.outputs, outs):
            helpers.assert_close(got, ref[tid], dtype, f"step {step} {g.tensors[tid]['name']}")
        for t in state_ids:
            dev = runner.inputs[g.inputs.index(t)].float().cpu().numpy()[:, :step + 1]
            helpers.assert_close(dev, oracle_state[t][:, :step + 1], dtype, f"step {step} cache")
    plan.close()


@pytest.mark.parametrize("M,N,K,bias,act,res", [
    (1, 4096, 4096, False, False, False),
    (4, 1000, 136, True, True, True),
    (8, 50, 8, True, False, True),
    (3, 2304, 768, True, False, False),
    (5, 97, 1032, False, True, False),
    (8, 11008, 4096, False, False, True),
    (2, 16400, 4096, True, False, True),      # above 128 MiB of weights: the bulk-tensor form by default
])
def test_few_row_linear_streams_its_weight(M, N, K, bias, act, res):
    """LINEAR with at most 8 rows: the weight-streaming kernel, with the fused bias / GELU / residual epilogue."""
    g = synth.GraphDesc()
    x = g.tensor("x", synth.BF16, [M, K], synth.INPUT)
    w = g.tensor("w", synth.BF16, [K, N], synth.CONST)
    ins = [x, w]
    feeds = {x: helpers.rand_feed([M, K], synth.BF16, 1), w: synth.round_bf16(synth.normal(7, 1, [K, N], 0.05))}
    if bias:
        b = g.tensor("b", synth.BF16, [N], synth.CONST)
        ins.append(b)
        feeds[b] = helpers.rand_feed([N], synth.BF16, 2)
    last = not (act or res)
    y = g.tensor("y", synth.BF16, [M, N], synth.OUTPUT if last else synth.ACT)
    g.op(synth.LINEAR, ins, [y], contract=1)
    if act:
        a = g.tensor("a", synth.BF16, [M, N], synth.ACT if res else synth.OUTPUT)
        g.op(synth.GELU, [y], [a], gelu_tanh=0)
        y = a
    if res:
        r = g.tensor("r", synth.BF16, [M, N], synth.INPUT)
        feeds[r] = helpers.rand_feed([M, N], synth.BF16, 3)
        o = g.tensor("o", synth.BF16, [M, N], synth.OUTPUT)
        g.op(synth.ADD, [y, r], [o])
        y = o
    got, plan, _ = helpers.run_gpu(g, feeds, synth.default_candidates(g))
    names = [s["kernel_name"] for s in plan.steps()]
    assert names[0] == "GEMM_ROWS", names
    helpers.assert_close(got[y], helpers.run_oracle(g, feeds)[y], synth.BF16, f"{M}x{N}x{K}")
    plan.close()


def test_one_captured_graph_serves_every_step_of_a_generation_loop():
    """The position is read on the device, so a single CUDA-graph capture of fluid_run is replayed for every step while
    the caller only rewrites the ids and the position buffers: results equal the step-by-step oracle."""
    import torch
    cfg = synth.scaled(synth.CONFIGS["llama"], dtype=synth.BF16, S=1, L=2, H=256, nh=4, F=512, B=2, V=300)
    dec = synth.build_decode_model(cfg, 16)
    g = dec.graph
    helpers.ensure_lib()
    plan = fluid.Plan(g, synth.default_candidates(g))
    runner = fluid.Runner(plan, dec.consts)
    state_ids = [t for pair in dec.caches for t in pair]
    for t in state_ids:
        runner.inputs[g.inputs.index(t)].zero_()
    oracle_state = {t: np.zeros(g.dims(t)) for t in state_ids}
    ids_buf, pos_buf = runner.inputs[g.inputs.index(dec.ids)], runner.inputs[g.inputs.index(dec.pos)]
    stream = torch.cuda.Stream()
    rng = np.random.default_rng(5)
    with torch.cuda.stream(stream):
        ids_buf.zero_(); pos_buf.zero_()
        runner.run(stream)                       # warm-up outside the capture (tensor maps, function attributes)
        for t in state_ids:
            runner.inputs[g.inputs.index(t)].zero_()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            runner.run(torch.cuda.current_stream())
        for t in state_ids:                      # the capture itself ran nothing, but start clean all the same
            runner.inputs[g.inputs.index(t)].zero_()
        for step in range(10):
            ids = rng.integers(0, cfg.V, size=(cfg.B, 1)).astype(np.int32)
            ids_buf.copy_(torch.from_numpy(ids)); pos_buf.fill_(step)
            graph.replay()
            stream.synchronize()
            feeds = dict(dec.consts)
            feeds[dec.ids], feeds[dec.pos] = ids, np.array([step], dtype=np.int32)
            feeds.update(oracle_state)
            ref = helpers.run_oracle(g, feeds)
            for t in state_ids:
                oracle_state[t] = ref[t]
            logits = runner.outputs[1].float().cpu().numpy()
            helpers.assert_close(logits, ref[g.outputs[1]], synth.BF16, f"replayed step {step}")
    assert runner.status() == 0
    plan.close()


def test_positions_per_sequence():
    """pos of shape [B]: every sequence appends at, and attends up to, its own position; a sequence whose position lies
    outside the cache is left alone and reported, the others are served."""
    B, nh, nkv, D, Tmax = 5, 8, 4, 128, 300
    g = synth.GraphDesc()
    q = g.tensor("q", synth.BF16, [B, 1, nh, D], synth.INPUT)
    k = g.tensor("k", synth.BF16, [B, 1, nkv, D], synth.INPUT)
    v = g.tensor("v", synth.BF16, [B, 1, nkv, D], synth.INPUT)
    kc = g.tensor("kc", synth.BF16, [B, Tmax, nkv, D], synth.STATE)
    vc = g.tensor("vc", synth.BF16, [B, Tmax, nkv, D], synth.STATE)
    pos = g.tensor("pos", synth.I32, [B], synth.INPUT)
    out = g.tensor("ctx", synth.BF16, [B, 1, nh, D], synth.OUTPUT)
    g.op(synth.CACHED_ATTENTION, [q, k, v, kc, vc, pos], [out], scale=1.0 / math.sqrt(D))
    helpers.ensure_lib()
    plan = fluid.Plan(g, synth.default_candidates(g))
    runner = fluid.Runner(plan, {}, poison=True)
    feeds = {q: helpers.rand_feed([B, 1, nh, D], synth.BF16, 1, -2, 2), k: helpers.rand_feed([B, 1, nkv, D], synth.BF16, 2, -2, 2),
             v: helpers.rand_feed([B, 1, nkv, D], synth.BF16, 3), kc: helpers.rand_feed([B, Tmax, nkv, D], synth.BF16, 4, -2, 2),
             vc: helpers.rand_feed([B, Tmax, nkv, D], synth.BF16, 5), pos: np.array([0, 299, 17, 128, 255], dtype=np.int32)}
    runner.set_inputs([feeds[t] for t in g.inputs])
    runner.run()
    got = runner.outputs_host()[0]
    assert runner.status() == 0
    ref = helpers.run_oracle(g, feeds)
    helpers.assert_close(got, ref[out], synth.BF16, "ragged positions")
    kc_dev = runner.inputs[g.inputs.index(kc)].float().cpu().numpy()
    assert np.array_equal(kc_dev, ref[kc])
    # sequence 2 out of range: its context row and caches keep what they held, the others are computed
    bad = dict(feeds)
    bad[pos] = np.array([3, 4, 300, 5, 6], dtype=np.int32)
    runner.set_inputs([bad[t] for t in g.inputs])
    runner.outputs[0].fill_(7.0)
    runner.run()
    with pytest.raises(fluid.FluidError):
        runner.status()
    got = runner.outputs[0].float().cpu().numpy()
    ok_rows = [0, 1, 3, 4]
    good = {t: (a[ok_rows] if a.shape[0] == B else a) for t, a in bad.items()}
    good[pos] = bad[pos][ok_rows]
    g4 = synth.GraphDesc()
    ids4 = [g4.tensor(g.tensors[t]["name"], g.tensors[t]["dtype"], [4] + g.dims(t)[1:] if t != pos else [4], g.tensors[t]["kind"]) for t in (q, k, v, kc, vc, pos)]
    o4 = g4.tensor("ctx", synth.BF16, [4, 1, nh, D], synth.OUTPUT)
    g4.op(synth.CACHED_ATTENTION, ids4, [o4], scale=1.0 / math.sqrt(D))
    ref4 = helpers.run_oracle(g4, {i4: good[t] for i4, t in zip(ids4, (q, k, v, kc, vc, pos))})
    helpers.assert_close(got[ok_rows], ref4[o4], synth.BF16, "served sequences")
    assert np.all(got[2] == 7.0)
    plan.close()


def test_decoding_with_ragged_lengths():
    """A batch whose sequences are at different lengths: positions per sequence through the whole model (rotary offset,
    cache append and attention span all per sequence), several steps in a row."""
    cfg = synth.scaled(synth.CONFIGS["llama"], dtype=synth.BF16, S=1, L=2, H=256, nh=4, F=384, B=3, V=400)
    t_max = 40
    dec = synth.build_decode_model(cfg, t_max, per_sequence_pos=True)
    g = dec.graph
    helpers.ensure_lib()
    plan = fluid.Plan(g, synth.default_candidates(g))
    runner = fluid.Runner(plan, dec.consts)
    rng = np.random.default_rng(2)
    start = np.array([0, 11, 30], dtype=np.int32)
    state_ids = [t for pair in dec.caches for t in pair]
    oracle_state = {t: synth.round_bf16(synth.uniform(8, t, g.dims(t))).astype(np.float64) for t in state_ids}
    for t in state_ids:
        runner.inputs[g.inputs.index(t)].copy_(fluid.to_device(oracle_state[t].astype(np.float32), synth.BF16, "cuda"))
    for step in range(6):
        ids = rng.integers(0, cfg.V, size=(cfg.B, 1)).astype(np.int32)
        feeds = dict(dec.consts)
        feeds[dec.ids], feeds[dec.pos] = ids, start + step
        feeds.update(oracle_state)
        ref = helpers.run_oracle(g, feeds)
        for t in state_ids:
            oracle_state[t] = ref[t]
        runner.inputs[g.inputs.index(dec.ids)].copy_(fluid.to_device(ids, synth.I32, "cuda"))
        runner.inputs[g.inputs.index(dec.pos)].copy_(fluid.to_device(feeds[dec.pos], synth.I32, "cuda"))
        runner.run()
        outs = runner.outputs_host()
        assert runner.status() == 0
        for tid, got in zip(g.outputs, outs):
            helpers.assert_close(got, ref[tid], synth.BF16, f"ragged step {step} {g.tensors[tid]['name']}")
    plan.close()


@pytest.mark.parametrize("dtype", [synth.BF16, synth.F32])
def test_embedding_with_a_position_read_on_the_device(dtype):
    g = synth.GraphDesc()
    ids = g.tensor("ids", synth.I32, [3, 2], synth.INPUT)
    tok = g.tensor("tok", dtype, [50, 64], synth.CONST)
    ptab = g.tensor("ptab", dtype, [40, 64], synth.CONST)
    off = g.tensor("off", synth.I32, [3], synth.INPUT)
    y = g.tensor("y", dtype, [3, 2, 64], synth.OUTPUT)
    g.op(synth.EMBED, [ids, tok, ptab, off], [y])
    feeds = {ids: synth.token_ids(1, 0, [3, 2], 50), tok: helpers.rand_feed([50, 64], dtype, 2), ptab: helpers.rand_feed([40, 64], dtype, 3),
             off: np.array([0, 17, 38], dtype=np.int32)}
    got, plan, _ = helpers.run_gpu(g, feeds)
    helpers.assert_close(got[y], helpers.run_oracle(g, feeds)[y], dtype, "embed with offsets")
    plan.close()


@pytest.mark.parametrize("family", ["llama", "gpt2_small"])
def test_prefill_then_decode_continues_the_sequence(family):
    """A prompt goes through the whole-sequence graph, whose keys and values are graph outputs; they are copied into the
    caches and the next tokens are decoded one by one. Every step's logits are compared with the oracle's direct
    whole-sequence formulas on the prefix so far."""
    import torch
    from oracle import models
    S0, S1, t_max = 12, 16, 20
    base = synth.scaled(synth.CONFIGS[family], dtype=synth.BF16, L=2, H=256, nh=4, F=512, B=2, V=300)
    whole = synth.build_model(synth.scaled(base, S=S1))                  # weights and tokens of the full sequence
    by_name = {whole.graph.tensors[t]["name"]: a for t, a in whole.consts.items()}
    pre = synth.build_model(synth.scaled(base, S=S0), materialize=False, emit_kv=True)
    pre_consts = {t: (by_name[td["name"]][:S0] if td["name"] == "pos_table" else by_name[td["name"]])
                  for t, td in enumerate(pre.graph.tensors) if td["kind"] == synth.CONST}
    helpers.ensure_lib()
    pplan = fluid.Plan(pre.graph, synth.default_candidates(pre.graph))
    prun = fluid.Runner(pplan, pre_consts, poison=True)
    prun.set_inputs([whole.ids[:, :S0]])
    prun.run()
    assert prun.status() == 0
    outs = dict(zip(pre.graph.outputs, prun.outputs))
    names = {pre.graph.tensors[t]["name"]: t for t in pre.graph.outputs}
    _, ref_logits = models.forward(base.family, base.L, by_name, whole.ids[:, :S0])
    helpers.assert_close(outs[names["logits"]].float().cpu().numpy(), ref_logits, synth.BF16, "prompt logits")

    dec = synth.build_decode_model(synth.scaled(base, S=S1), t_max, like=whole)
    g = dec.graph
    dplan = fluid.Plan(g, synth.default_candidates(g))
    drun = fluid.Runner(dplan, dec.consts, poison=True)
    for l, (kc, vc) in enumerate(dec.caches):
        kname = f"l{l}.k_rope" if base.family == "llama" else f"l{l}.k"
        for cache, name in ((kc, kname), (vc, f"l{l}.v")):
            buf = drun.inputs[g.inputs.index(cache)]
            buf.fill_(float("nan"))
            buf[:, :S0].copy_(outs[names[name]])
    for t in range(S0, S1):
        drun.inputs[g.inputs.index(dec.ids)].copy_(torch.from_numpy(np.ascontiguousarray(whole.ids[:, t:t + 1])))
        drun.inputs[g.inputs.index(dec.pos)].fill_(t)
        drun.run()
        logits = drun.outputs[1].float().cpu().numpy()
        assert drun.status() == 0
        _, ref_logits = models.forward(base.family, base.L, by_name, whole.ids[:, :t + 1])
        helpers.assert_close(logits[:, 0], ref_logits, synth.BF16, f"decoded token {t}")
    pplan.close()
    dplan.close()


def test_cached_attention_random_shapes():
    """Seeded random sweep: head dims, grouped heads, batch sizes (hence cluster sizes), cache lengths, positions shared
    or per sequence, both dtypes."""
    rng = np.random.default_rng(20241125)
    helpers.ensure_lib()
    for it in range(24):
        dtype = synth.BF16 if rng.random() < 0.7 else synth.F32
        vec = 8 if dtype == synth.BF16 else 4
        D = min(128, int(vec * rng.choice([1, 2, 4, 8, 16])))
        nkv = int(rng.choice([1, 2, 3, 4, 8]))
        nh = nkv * int(rng.choice([1, 2, 4]))
        B, Tmax, per_seq = int(rng.integers(1, 40)), int(rng.integers(1, 700)), bool(rng.random() < 0.5)
        g = synth.GraphDesc()
        q = g.tensor("q", dtype, [B, 1, nh, D], synth.INPUT)
        k = g.tensor("k", dtype, [B, 1, nkv, D], synth.INPUT)
        v = g.tensor("v", dtype, [B, 1, nkv, D], synth.INPUT)
        kc = g.tensor("kc", dtype, [B, Tmax, nkv, D], synth.STATE)
        vc = g.tensor("vc", dtype, [B, Tmax, nkv, D], synth.STATE)
        pos = g.tensor("pos", synth.I32, [B if per_seq else 1], synth.INPUT)
        out = g.tensor("o", dtype, [B, 1, nh, D], synth.OUTPUT)
        g.op(synth.CACHED_ATTENTION, [q, k, v, kc, vc, pos], [out], scale=1 / math.sqrt(D))
        feeds = {q: helpers.rand_feed([B, 1, nh, D], dtype, it, -2, 2), k: helpers.rand_feed([B, 1, nkv, D], dtype, it + 1000, -2, 2),
                 v: helpers.rand_feed([B, 1, nkv, D], dtype, it + 2000), kc: helpers.rand_feed([B, Tmax, nkv, D], dtype, it + 3000, -2, 2),
                 vc: helpers.rand_feed([B, Tmax, nkv, D], dtype, it + 4000),
                 pos: rng.integers(0, Tmax, size=(B if per_seq else 1)).astype(np.int32)}
        got, plan, runner = helpers.run_gpu(g, feeds, synth.default_candidates(g))
        ref = helpers.run_oracle(g, feeds)
        what = f"case {it}: D {D} nh {nh} nkv {nkv} B {B} Tmax {Tmax} per_seq {per_seq}"
        helpers.assert_close(got[out], ref[out], dtype, what)
        assert np.array_equal(runner.inputs[g.inputs.index(kc)].float().cpu().numpy(), ref[kc]), what
        assert np.array_equal(runner.inputs[g.inputs.index(vc)].float().cpu().numpy(), ref[vc]), what
        plan.close()


@pytest.mark.parametrize("form", ["0", "1", "1,2,1", "1,4,4", "2,2,8", "4,1,2", "2,3,16"])
def test_few_row_linear_both_weight_paths(form, monkeypatch):
    """The few-row GEMM brings its weights in either by per-lane asynchronous copies (form "0") or by bulk-tensor
    boxes ("1": its own choice of boxes per stage, stages, warps per tile; else those three): every form against the oracle, on ragged N and K, 1 to 16 rows,
    the epilogues, and one decoding step of a small Llama-shaped model (sibling projections behind a folded
    normalisation, SwiGLU)."""
    monkeypatch.setenv("FLUID_ROWS_TMA", form)
    for it, (M, N, K, bias, act, res) in enumerate([(4, 1000, 136, True, True, True), (8, 4112, 4096, False, False, True),
                                                    (13, 520, 2056, True, False, False), (16, 300, 1024, False, True, False),
                                                    (1, 33, 8, True, False, False), (5, 2304, 768, True, False, True)]):
        g = synth.GraphDesc()
        x = g.tensor("x", synth.BF16, [M, K], synth.INPUT)
        w = g.tensor("w", synth.BF16, [K, N], synth.CONST)
        ins = [x, w]
        feeds = {x: helpers.rand_feed([M, K], synth.BF16, 10 + it), w: synth.round_bf16(synth.normal(7, 20 + it, [K, N], 0.05))}
        if bias:
            b = g.tensor("b", synth.BF16, [N], synth.CONST)
            ins.append(b)
            feeds[b] = helpers.rand_feed([N], synth.BF16, 30 + it)
        y = g.tensor("y", synth.BF16, [M, N], synth.ACT if (act or res) else synth.OUTPUT)
        g.op(synth.LINEAR, ins, [y], contract=1)
        if act:
            a = g.tensor("a", synth.BF16, [M, N], synth.ACT if res else synth.OUTPUT)
            g.op(synth.GELU, [y], [a], gelu_tanh=0)
            y = a
        if res:
            r = g.tensor("r", synth.BF16, [M, N], synth.INPUT)
            feeds[r] = helpers.rand_feed([M, N], synth.BF16, 40 + it)
            o = g.tensor("o", synth.BF16, [M, N], synth.OUTPUT)
            g.op(synth.ADD, [y, r], [o])
            y = o
        got, plan, _ = helpers.run_gpu(g, feeds, synth.default_candidates(g))
        assert "GEMM_ROWS" in [s["kernel_name"] for s in plan.steps()]
        helpers.assert_close(got[y], helpers.run_oracle(g, feeds)[y], synth.BF16, f"form {form}: {M}x{N}x{K}")
        plan.close()
    for family in ("llama", "gpt2_small"):
        cfg = synth.scaled(synth.CONFIGS[family], dtype=synth.BF16, S=1, L=1, H=256, nh=4, F=640, B=3, V=777)
        dec = synth.build_decode_model(cfg, 16)
        g = dec.graph
        feeds = dict(dec.consts)
        feeds[dec.ids] = synth.token_ids(synth.TOKEN_SEED, 1, [cfg.B, 1], cfg.V)
        feeds[dec.pos] = np.array([9], dtype=np.int32)
        for i, pair in enumerate(dec.caches):
            for j, t in enumerate(pair):
                feeds[t] = synth.round_bf16(synth.uniform(3, 2 * i + j, g.dims(t)))
        ref = helpers.run_oracle(g, feeds)
        plan = fluid.Plan(g, synth.default_candidates(g))
        assert [s["kernel_name"] for s in plan.steps()].count("GEMM_ROWS") >= 4
        runner = fluid.Runner(plan, dec.consts, poison=True)
        runner.set_inputs([feeds[t] for t in g.inputs])
        runner.run()
        outs = runner.outputs_host()
        assert runner.status() == 0
        for tid, got in zip(g.outputs, outs):
            helpers.assert_close(got, ref[tid], synth.BF16, f"form {form} {family} {g.tensors[tid]['name']}")
        plan.close()


def test_few_row_linear_random_shapes():
    """Seeded random sweep of LINEAR with 1 to 16 rows: ragged N and K, bias / GELU / residual epilogues, and the RMS
    normalisation folded in."""
    rng = np.random.default_rng(2411)
    helpers.ensure_lib()
    for it in range(40):
        M, N, K = int(rng.integers(1, 17)), int(rng.integers(1, 5000)), 8 * int(rng.integers(1, 600))
        bias, act, res, rms = (bool(rng.random() < p) for p in (0.5, 0.3, 0.5, 0.6))
        layer = rms and M <= 15 and bool(rng.random() < 0.5)     # LayerNorm instead of RMSNorm
        g = synth.GraphDesc()
        x = g.tensor("x", synth.BF16, [M, K], synth.INPUT)
        feeds = {x: helpers.rand_feed([M, K], synth.BF16, it, -1.0, 3.0)}   # a mean well away from zero
        a = x
        if rms:
            gam = g.tensor("gam", synth.BF16, [K], synth.CONST)
            feeds[gam] = helpers.rand_feed([K], synth.BF16, it + 50, 0.5, 1.5)
            a = g.tensor("n", synth.BF16, [M, K], synth.ACT)
            if layer:
                bet = g.tensor("bet", synth.BF16, [K], synth.CONST)
                feeds[bet] = helpers.rand_feed([K], synth.BF16, it + 60)
                g.op(synth.LAYERNORM, [x, gam, bet], [a], eps=1e-5)
            else:
                g.op(synth.RMSNORM, [x, gam], [a], eps=1e-5)
        w = g.tensor("w", synth.BF16, [K, N], synth.CONST)
        feeds[w] = synth.round_bf16(synth.normal(7, it, [K, N], 0.05))
        ins = [a, w]
        if bias:
            b = g.tensor("b", synth.BF16, [N], synth.CONST)
            ins.append(b)
            feeds[b] = helpers.rand_feed([N], synth.BF16, it + 100)
        y = g.tensor("y", synth.BF16, [M, N], synth.ACT if (act or res) else synth.OUTPUT)
        g.op(synth.LINEAR, ins, [y], contract=1)
        if act:
            a2 = g.tensor("a2", synth.BF16, [M, N], synth.ACT if res else synth.OUTPUT)
            g.op(synth.GELU, [y], [a2], gelu_tanh=0)
            y = a2
        if res:
            r = g.tensor("r", synth.BF16, [M, N], synth.INPUT)
            feeds[r] = helpers.rand_feed([M, N], synth.BF16, it + 200)
            o = g.tensor("o", synth.BF16, [M, N], synth.OUTPUT)
            g.op(synth.ADD, [y, r], [o])
            y = o
        got, plan, _ = helpers.run_gpu(g, feeds, synth.default_candidates(g))
        steps = plan.steps()
        # the staged activation rows (and the bias row of a LayerNorm) must fit the SM next to the rings (five stages
        # deep, seven beyond 8 rows)
        def fits(rows):
            return rows * (2 * K + 64) + 128 + 16 * 1024 * (7 if rows > 8 else 5) <= 226 * 1024
        assert ("GEMM_ROWS" in [s["kernel_name"] for s in steps]) == fits(M)
        if rms and fits(M) and (not layer or fits(M + 1)):
            assert len(steps) == 1 and (steps[0]["variant"] >> 30) & 1      # one launch: norm, GEMM and epilogue
        helpers.assert_close(got[y], helpers.run_oracle(g, feeds)[y], synth.BF16, f"case {it}: {M}x{N}x{K} bias {bias} act {act} res {res} norm {rms} layer {layer}")
        plan.close()


def test_plan_of_a_decoding_step_from_measured_costs():
    """The measured cost function handles the decoding operators too (state tensors, device-side positions): the plan
    built from measured per-operator times gives the oracle's results."""
    from paper_2411_09242_b200.measure import MeasuredEval
    cfg = synth.scaled(synth.CONFIGS["llama"], dtype=synth.BF16, S=1, L=1, H=256, nh=4, F=384, B=3, V=300)
    dec = synth.build_decode_model(cfg, 24)
    g = dec.graph
    helpers.ensure_lib()
    cands = synth.default_candidates(g)
    ev = MeasuredEval(g, cands, reps=3, warmup=1)
    plan = fluid.Plan(g, cands, eval=ev.callback)
    assert ev.measured >= 8 and 0 < plan.cost <= plan.canonical_cost < 1.0
    kinds = [s["kernel_name"] for s in plan.steps()]
    assert "ATTN_DECODE" in kinds and "GEMM_ROWS" in kinds
    feeds = dict(dec.consts)
    feeds[dec.ids] = synth.token_ids(3, 0, [cfg.B, 1], cfg.V)
    feeds[dec.pos] = np.array([9], dtype=np.int32)
    for i, pair in enumerate(dec.caches):
        for j, t in enumerate(pair):
            feeds[t] = synth.round_bf16(synth.uniform(5, 2 * i + j, g.dims(t)))
    runner = fluid.Runner(plan, dec.consts)
    runner.set_inputs([feeds[t] for t in g.inputs])
    runner.run()
    assert runner.status() == 0
    ref = helpers.run_oracle(g, feeds)
    for tid, got in zip(g.outputs, runner.outputs_host()):
        helpers.assert_close(got, ref[tid], synth.BF16, f"measured-cost decoding plan output {tid}")
    plan.close()
