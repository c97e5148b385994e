"""CPU fp64 oracle: run an operator graph node by node. TEST INFRASTRUCTURE ONLY.

The graph is the plain-data description the planner receives (tensors = the paper's "edges",
ops = its "nodes"; Sec. "Design"). The oracle ignores every layout and every arena offset: each
tensor is one fresh canonical fp64 array, ops run in declaration order (which is a topological
order of the flow), exactly the unoptimised blueprint the method must stay equal to.

Pinned by tests/test_oracle_models.py against the direct model formulas in oracle/models.py
and by whole-model invariants (causality, batch independence, permutation equivariance).
"""
from __future__ import annotations

import numpy as np

from . import ops

# operator codes of the graph description (the C header's fluid_op_kind values)
(EMBED, LINEAR, ADD, MUL, GELU, SILU, SOFTMAX, LAYERNORM, RMSNORM, ROPE, TRANSPOSE, BMM_QK,
 BMM_PV, SELECT_LAST_TOKEN, CACHED_ATTENTION) = range(15)
STATE = 4   # tensor kind: a caller-owned buffer an op reads and updates (a key/value cache)


def run_op(kind, ins, attrs):
    """Apply one node to canonical fp64 inputs; returns the list of outputs."""
    if kind == EMBED:
        return [ops.embed(ins[0], ins[1], ins[2] if len(ins) > 2 else None,
                          pos0=np.asarray(ins[3]).reshape(-1) if len(ins) > 3 else 0)]
    if kind == LINEAR:
        return [ops.linear(ins[0], ins[1], ins[2] if len(ins) > 2 else None,
                           contract=attrs.get("contract", 1))]
    if kind == ADD:
        return [ops.add(ins[0], ins[1])]
    if kind == MUL:
        return [ops.mul(ins[0], ins[1])]
    if kind == GELU:
        return [ops.gelu(ins[0], tanh_form=bool(attrs.get("gelu_tanh", 0)))]
    if kind == SILU:
        return [ops.silu(ins[0])]
    if kind == SOFTMAX:
        return [ops.softmax(ins[0], causal=bool(attrs.get("causal", 0)),
                            scale=attrs.get("scale", 1.0))]
    if kind == LAYERNORM:
        return [ops.layernorm(ins[0], ins[1], ins[2], eps=attrs.get("eps", 1e-5))]
    if kind == RMSNORM:
        return [ops.rmsnorm(ins[0], ins[1], eps=attrs.get("eps", 1e-5))]
    if kind == ROPE:
        pos0 = np.asarray(ins[1]).reshape(-1) if len(ins) > 1 else 0
        return [ops.rope(ins[0], base=attrs.get("rope_base", 10000.0),
                         interleaved=bool(attrs.get("rope_interleaved", 0)), pos0=pos0)]
    if kind == TRANSPOSE:
        return [ops.transpose(ins[0], attrs["perm"])]
    if kind == BMM_QK:
        return [ops.bmm_qk(ins[0], ins[1], scale=attrs.get("scale", 1.0))]
    if kind == BMM_PV:
        return [ops.bmm_pv(ins[0], ins[1])]
    if kind == SELECT_LAST_TOKEN:
        return [ops.select_last_token(ins[0])]
    raise ValueError(f"unknown op kind {kind}")


def run_graph(tensors, op_list, feeds, keep_all=False, store=None, load=None):
    """Execute the graph.

    store: optional callable (tensor id, fp64 array) -> fp64 array applied to every op output
    before it is handed on. load: optional callable (op index, tensor id, fp64 array) -> fp64 array
    applied to each input as an op reads it. The parity reference uses neither (no intermediate
    rounding). They are a diagnostic mode: a test may pass functions that round each tensor the way
    a device plan stores it (bf16, fp32, or not at all for tensors fused away; `load` for a tensor
    the plan keeps in two precisions, one per kind of reader), to tell storage rounding apart from
    arithmetic errors.

    tensors : list of dicts with "dims" (and "kind"); op_list : list of dicts with "kind",
    "ins", "outs", "attrs"; feeds : {tensor id: array} for every graph input and constant.
    Returns {tensor id: fp64 array} for every tensor (keep_all) or only those no op consumes
    plus anything marked as a graph output (kind == 1) and the final contents of every state
    tensor (kind == 4); in that case an intermediate array is dropped after its last reader.
    """
    vals = {}
    for tid, a in feeds.items():
        a = np.asarray(a)
        vals[tid] = a if a.dtype.kind in "iu" else a.astype(np.float64)
    last_reader = {}
    for n, op in enumerate(op_list):
        for i in op["ins"]:
            last_reader[i] = n
    consumed = set()
    for n, op in enumerate(op_list):
        ins = [vals[i] for i in op["ins"]]
        if load is not None:
            ins = [a if a.dtype.kind in "iu" else np.asarray(load(n, i, a), dtype=np.float64)
                   for i, a in zip(op["ins"], ins)]
        if op["kind"] == CACHED_ATTENTION:
            # the one op with a side effect: rows `pos` of its two state tensors are replaced
            ctx, kc, vc = ops.cached_attention(*ins, scale=op.get("attrs", {}).get("scale", 1.0))
            vals[op["ins"][3]], vals[op["ins"][4]] = kc, vc
            outs = [ctx]
        else:
            outs = run_op(op["kind"], ins, op.get("attrs", {}))
        for tid, o in zip(op["outs"], outs):
            assert list(o.shape) == list(tensors[tid]["dims"]), (
                tensors[tid].get("name"), o.shape, tensors[tid]["dims"])
            vals[tid] = o if store is None else np.asarray(store(tid, o), dtype=np.float64)
        consumed.update(op["ins"])
        if not keep_all:
            for i in set(op["ins"]):
                if last_reader[i] == n and i not in feeds and tensors[i].get("kind") not in (1, STATE):
                    del vals[i]
    if keep_all:
        return vals
    return {tid: v for tid, v in vals.items()
            if tensors[tid].get("kind") in (1, STATE) or (tid not in consumed and tid not in feeds)}
