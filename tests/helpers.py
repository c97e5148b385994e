"""Shared test helpers: build the CUDA library once, random DAGs, plan records."""
import os
import re

import numpy as np

from paper_2411_09242_b200 import build as _build
from paper_2411_09242_b200 import fluid, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def ensure_lib():
    _build.build()
    return fluid.lib()


def header_symbols():
    text = open(os.path.join(ROOT, "include", "fluid.h")).read()
    return re.findall(r"FLUID_API[^;(]*?\b(fluid_\w+)\s*\(", text)


def random_dag(seed, n_ops=10, dims=(4, 8)):
    """A random DAG of unary (GELU) and binary (ADD) ops over small matrices."""
    rng = np.random.default_rng(seed)
    g = synth.GraphDesc()
    avail = [g.tensor("in0", synth.F32, dims, synth.INPUT)]
    for i in range(n_ops):
        last = i == n_ops - 1
        out = g.tensor(f"t{i}", synth.F32, dims, synth.OUTPUT if last else synth.ACT)
        if len(avail) >= 2 and rng.random() < 0.45:
            a, b = rng.choice(len(avail), size=2, replace=False)
            g.op(synth.ADD, [avail[a], avail[b]], [out])
        else:
            a = int(rng.integers(max(0, len(avail) - 3), len(avail)))
            g.op(synth.GELU, [avail[a]], [out])
        avail.append(out)
    return g


def plan_records(plan):
    """(id, bytes, first, last) per arena-resident root tensor, and {id: offset}."""
    recs, offs = [], {}
    for r in plan.records():
        recs.append((r["id"], r["bytes"], r["first"], r["last"]))
        offs[r["id"]] = r["offset"]
    return recs, offs


def table_eval(seed, hi=20):
    def ev(op, lay):
        key = (seed, op) + tuple(sorted(lay.items()))
        return float(np.random.default_rng(abs(hash(key)) % (2 ** 32)).integers(1, hi))
    return ev


# ---- GPU-side helpers (imported lazily by the gpu tests) ---------------------------------------
def run_gpu(desc, feeds, candidates=None, poison=True, **opts):
    """Plan + run a graph on the GPU through the C-ABI; returns ({output tid: fp64 array}, plan, runner)."""
    ensure_lib()
    plan = fluid.Plan(desc, candidates, **opts)
    consts = {t: a for t, a in feeds.items() if desc.tensors[t]["kind"] == synth.CONST}
    runner = fluid.Runner(plan, consts, poison=poison)
    runner.set_inputs([feeds[t] for t in desc.inputs])
    runner.run()
    outs = runner.outputs_host()
    assert runner.status() == 0
    return dict(zip(desc.outputs, outs)), plan, runner


def run_oracle(desc, feeds, keep_all=False, store=None, load=None):
    from oracle import graph_exec
    return graph_exec.run_graph(desc.tensors, desc.ops, feeds, keep_all=keep_all, store=store, load=load)


def tol_for(dtype):
    """max|err| <= tol * max|ref|: 1e-2 on bf16 paths, 1e-4 on fp32 paths."""
    return 1e-2 if dtype == synth.BF16 else 1e-4


def assert_close(got, ref, dtype, what="", tol=None):
    tol = tol_for(dtype) if tol is None else tol
    scale = float(np.max(np.abs(ref))) or 1.0
    err = float(np.max(np.abs(got - ref)))
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    assert err <= tol * scale, f"{what}: max|err| {err:.3e} > {tol:g} * max|ref| {scale:.3e}"


def storage_hooks(desc, plan):
    """(store, load) for run_oracle that round each tensor the way `plan` keeps it, read from the plan itself:
      * an op output that owns an arena record (or aliases one) is rounded to that record's dtype: bf16, or
        fp32 for the residual-stream tensors the planner keeps wide;
      * a graph output is rounded to its declared dtype;
      * an op output with no record (folded into a fused step: scores, gate, up, pre-activation sums) is not
        rounded at all: it only ever exists in fp32 accumulators;
      * a tensor with a bf16 twin record is read rounded to bf16 by the tensor-core ops (LINEAR, BMM) and wide
        by everything else;
      * inside a fused-attention step the probabilities are a tensor-core operand: BMM_PV reads the bf16 rounding
        of the exponentials 2^(t - n) (n a whole number per row) over the sum of the unrounded exponentials,
        which is how the fused kernel forms P.
    With these hooks the oracle is still exact fp64 arithmetic; only what is *stored* is rounded. The distance
    between this run and the plain oracle is the floor no executor that stores these dtypes can get under."""
    T = desc.tensors
    recs = {}
    twins = set()
    for r in plan.records():
        if r["tensor"] < 0:
            continue
        if r["twin"]:
            twins.add(r["tensor"])
        else:
            recs[r["tensor"]] = r["dtype"]
    fused_p = {}              # (op index, probabilities) read inside a fused-attention step -> its SOFTMAX op
    for s in plan.steps():
        if s["kernel_name"] == "ATTN":
            for o in s["ops"]:
                if desc.ops[o]["kind"] == synth.BMM_PV:
                    probs = desc.ops[o]["ins"][0]
                    fused_p[(o, probs)] = next(d for d in desc.ops if probs in d["outs"] and d["kind"] == synth.SOFTMAX)
    scores_of = {sm["ins"][0]: None for sm in fused_p.values()}     # score tensors to hold on to until P is formed
    # an RMS normalisation split across two tensor-core steps has no record of its own, but what its readers take as
    # their operand is bf16(x * gain), scaled by 1 / rms afterwards: a bf16 rounding of the normalised value up to that
    # row-wise factor, i.e. of the same relative size
    split_norm = {desc.ops[o]["outs"][0] for s in plan.steps() if s["kernel_name"] == "GEMM_TC"
                  for o in s["ops"] if desc.ops[o]["kind"] == synth.RMSNORM}

    def rb(a):
        return synth.round_bf16(np.asarray(a, dtype=np.float32)).astype(np.float64)

    def fused_probabilities(sm):
        """What the fused kernel feeds the tensor core as P: the exponentials relative to a whole-number reference
        point in the base-2 domain, rounded to bf16, over the sum of the unrounded exponentials."""
        sc = scores_of[sm["ins"][0]] * (sm["attrs"].get("scale", 1.0) * np.log2(np.e))
        scores_of[sm["ins"][0]] = None
        if sm["attrs"].get("causal"):
            allowed = np.arange(sc.shape[-1])[None, :] <= np.arange(sc.shape[-2])[:, None]
            sc = np.where(allowed, sc, -np.inf)
        e = np.exp2(sc - np.ceil(np.max(sc, axis=-1, keepdims=True)))
        return rb(e) / np.sum(e, axis=-1, keepdims=True)

    def store(tid, a):
        if tid in scores_of:
            scores_of[tid] = a
        if tid in split_norm:
            return rb(a)
        if T[tid]["kind"] == synth.OUTPUT:
            dt = T[tid]["dtype"]
        else:
            dt = recs.get(plan.tensor_info(tid).alias_of)
        if dt == synth.BF16:
            return rb(a)
        if dt == synth.F32:
            return np.asarray(a, dtype=np.float32).astype(np.float64)
        return a

    def load(op_index, tid, a):
        kind = desc.ops[op_index]["kind"]
        if (op_index, tid) in fused_p:
            return fused_probabilities(fused_p[(op_index, tid)])
        if kind in (synth.LINEAR, synth.BMM_QK, synth.BMM_PV) and T[tid]["kind"] == synth.ACT \
                and plan.tensor_info(tid).alias_of in twins:
            return rb(a)
        return a

    return store, load


def single_op_graph(kind, in_shapes, out_shape, dtype, attrs=None, in_kinds=None):
    g = synth.GraphDesc()
    ins = []
    for i, shp in enumerate(in_shapes):
        k = (in_kinds or {}).get(i, synth.INPUT)
        dt = synth.I32 if k == "ids" else dtype
        ins.append(g.tensor(f"in{i}", dt, shp, synth.INPUT if k == "ids" else k))
    out = g.tensor("out", dtype, out_shape, synth.OUTPUT)
    g.op(kind, ins, [out], **(attrs or {}))
    return g


def rand_feed(shape, dtype, seed, lo=-1.0, hi=1.0):
    a = synth.uniform(seed, 0, shape, lo, hi)
    return synth.round_bf16(a) if dtype == synth.BF16 else a


# ---- sampled per-step parity at full size -----------------------------------------------------------
ROWWISE = (synth.LINEAR, synth.ADD, synth.MUL, synth.GELU, synth.SILU, synth.LAYERNORM, synth.RMSNORM, synth.EMBED)


def check_steps_sampled(desc, plan, runner, feeds, n_rows=48, tol=2 ** -7, seed=0):
    """Per-step parity on samples: for every executed step, the oracle op(s) of that step are fed the GPU's
    own inputs restricted to sampled rows (row-wise ops) or to one sampled (batch, head) slice (attention
    products, softmax, RoPE), and the GPU's output is compared there. Localises any error to one kernel
    launch and is affordable at full model sizes. The plan must keep every tensor alive (no_reuse=1).
    Returns the number of outputs compared."""
    from oracle import graph_exec
    rng = np.random.default_rng(seed)
    T = desc.tensors
    consts = {}

    def const_like(t):
        return T[t]["kind"] in (synth.CONST, synth.INPUT) or T[plan.tensor_info(t).alias_of]["kind"] == synth.CONST

    def const_value(t):
        if t not in consts:
            if t in feeds:
                consts[t] = np.asarray(feeds[t])
            else:                              # a zero-copy view of a constant: replay its producer
                op = next(o for o in desc.ops if t in o["outs"])
                consts[t] = graph_exec.run_op(op["kind"], [np.asarray(const_value(i), np.float64) for i in op["ins"]],
                                              op["attrs"])[0]
        return consts[t]

    compared = 0
    for s in plan.steps():
        ops = [desc.ops[o] for o in s["ops"]]
        first = ops[0]
        od = T[first["outs"][0]]["dims"]
        if first["kind"] in (synth.BMM_QK, synth.BMM_PV, synth.SOFTMAX) and len(od) == 4:
            b, h = int(rng.integers(od[0])), int(rng.integers(od[1]))
            index = (slice(b, b + 1), slice(h, h + 1))
        elif first["kind"] == synth.ROPE:
            h = int(rng.integers(od[2]))
            index = (slice(None), slice(None), slice(h, h + 1))
        elif first["kind"] in ROWWISE:
            x_dims = T[first["ins"][0]]["dims"]
            nlead = len(x_dims) - (first["attrs"].get("contract", 1) if first["kind"] == synth.LINEAR else 1)
            if first["kind"] == synth.EMBED:
                nlead = 2
            lead = (T[first["ins"][0]]["dims"] if first["kind"] != synth.EMBED else od)[:nlead]
            total = int(np.prod(lead))
            rows = np.sort(rng.choice(total, size=min(n_rows, total), replace=False))
            index = tuple(list(int(v) for v in ix) for ix in np.unravel_index(rows, lead))
        else:
            index = None                        # small tensors (SELECT_LAST_TOKEN): whole tensor
        local = {}

        def value(t, sampled=True):
            if t in local:
                return local[t]
            if const_like(t):
                v = np.asarray(const_value(t))
                return v[index] if (sampled and index is not None and v.ndim == len(T[t]["dims"]) and T[t]["kind"] == synth.INPUT) else v
            return runner.read_tensor(t, index if sampled else None)

        for op in ops:
            kind, out = op["kind"], op["outs"][0]
            if kind == synth.EMBED:
                ids = np.asarray(feeds[op["ins"][0]])[index]
                want = np.asarray(const_value(op["ins"][1]), np.float64)[ids]
                if len(op["ins"]) > 2:
                    want = want + np.asarray(const_value(op["ins"][2]), np.float64)[np.asarray(index[1])]
            elif kind == synth.LINEAR:
                x = value(op["ins"][0])
                w_t = op["ins"][1]
                w = np.asarray(const_value(w_t), np.float64) if const_like(w_t) else runner.read_tensor(w_t)
                c = op["attrs"].get("contract", 1)
                K = int(np.prod(w.shape[:c]))
                want = x.reshape(x.shape[0], K) @ w.reshape(K, -1)
                if len(op["ins"]) > 2:
                    want = want + np.asarray(const_value(op["ins"][2]), np.float64).reshape(1, -1)
                want = want.reshape((x.shape[0],) + tuple(T[out]["dims"][len(index):]))
            elif kind in (synth.LAYERNORM, synth.RMSNORM):
                want = graph_exec.run_op(kind, [value(op["ins"][0])] + [np.asarray(const_value(t), np.float64) for t in op["ins"][1:]],
                                         op["attrs"])[0]
            elif kind == synth.ROPE and first["kind"] in (synth.LINEAR, synth.RMSNORM):
                # a rotary embedding folded into the projection's step: the sampled rows are (batch, position) pairs,
                # each rotated by its own position
                x = np.asarray(value(op["ins"][0]), np.float64)
                pos = np.asarray(index[1], dtype=np.int64)
                want = graph_exec.run_op(kind, [x[:, None], pos], op["attrs"])[0][:, 0]
            elif kind == synth.SELECT_LAST_TOKEN:
                want = runner.read_tensor(op["ins"][0])[:, -1, :]
            else:
                ins = [np.asarray(value(t), np.float64) for t in op["ins"]]
                if kind == synth.BMM_PV:        # causal probabilities are zero above the diagonal by definition;
                    prod = next((d for d in desc.ops if op["ins"][0] in d["outs"]), None)   # the device need not store them
                    if prod is not None and prod["kind"] == synth.SOFTMAX and prod["attrs"].get("causal"):
                        ins[0] = np.where(np.tril(np.ones(ins[0].shape[-2:], bool)), ins[0], 0.0)
                want = graph_exec.run_op(kind, ins, op["attrs"])[0]
            local[out] = want
            if out not in s["outs"]:
                continue                       # folded into the fused step: never stored
            have = runner.read_tensor(out, index)
            if kind in (synth.BMM_QK, synth.SOFTMAX):
                causal = op["attrs"].get("causal") or any(
                    d["kind"] == synth.SOFTMAX and d["attrs"].get("causal") and out in d["ins"] for d in desc.ops)
                if causal:                      # entries above the diagonal are never read downstream
                    S = want.shape[-1]
                    mask = np.tril(np.ones((S, S), bool))
                    want, have = np.where(mask, want, 0.0), np.where(mask, have, 0.0)
            assert_close(have.reshape(want.shape), want, synth.BF16,
                         f"step {s['kernel_name']} ops {s['ops']} -> {T[out]['name']}", tol=tol)
            compared += 1
    return compared
