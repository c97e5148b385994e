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
    for tid, t in enumerate(plan.desc.tensors):
        info = plan.tensor_info(tid)
        if info.offset >= 0 and info.alias_of == tid:
            recs.append((tid, info.bytes, info.first_step, info.last_step))
            offs[tid] = info.offset
    return recs, offs


def table_eval(seed, hi=20):
    def ev(op, lay):
        key = (seed, op) + tuple(sorted(lay.items()))
        return float(np.random.default_rng(abs(hash(key)) % (2 ** 32)).integers(1, hi))
    return ev
