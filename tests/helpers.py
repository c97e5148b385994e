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


def run_oracle(desc, feeds, keep_all=False):
    from oracle import graph_exec
    return graph_exec.run_graph(desc.tensors, desc.ops, feeds, keep_all=keep_all)


def tol_for(dtype):
    """max|err| <= tol * max|ref|: 1e-2 on bf16 paths, 1e-4 on fp32 paths."""
    return 1e-2 if dtype == synth.BF16 else 1e-4


def assert_close(got, ref, dtype, what="", tol=None):
    tol = tol_for(dtype) if tol is None else tol
    scale = float(np.max(np.abs(ref))) or 1.0
    err = float(np.max(np.abs(got - ref)))
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    assert err <= tol * scale, f"{what}: max|err| {err:.3e} > {tol:g} * max|ref| {scale:.3e}"


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
