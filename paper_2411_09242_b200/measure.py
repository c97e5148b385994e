"""The paper's external cost function, measured: eval(node, layouts) = the time of that operator, alone,
with its tensors in those layouts, on the GPU at hand (Algorithm 3's `eval`; Sec. "Implementation": the
compiler tries a layout and the runtime times it).

`MeasuredEval(graph, candidates)` is a callable for `fluid.Plan(..., eval=...)`. Every time the planner's
dynamic programme asks for the cost of (operator, layout per tensor), the answer comes from a table keyed
by the operator's signature (kind, attributes, tensor shapes and dtypes) and the layouts; a missing entry is
measured on the spot: a two-operator graph (the operator, then a copy to the caller's buffer) is planned
with a cost function that forces exactly those layouts, bound to random constants, run a few times with one
CUDA event pair per step, and the operator's own step time is recorded. Combinations the kernels cannot
run are recorded as +infinity. Operators repeat across layers, so a model needs a few hundred measurements.

Implementation variants (the paper's "Loop Reordering": several implementations of a matrix-multiply-like operator
are tried and the fastest is the operator's cost and the one that runs). `MeasuredEval(..., variants=True)` offers
`callback_variant` for `fluid.Plan(..., eval_variant=...)`: the planner then asks once per (operator, layouts,
variant) and every answer is a measurement of that operator run with that variant. `tune_step_variants` does the
same for the fused steps of a finished plan, which is what a model actually runs: every tensor-core GEMM step is
timed in place (inside the whole plan, epilogue fusions and sibling grouping included) with each variant its shape
admits, and the fastest per step is returned as an `op_variant` table for the final plan.

Only marshalling and bookkeeping live here; the planning and the timed kernels are the library's.
"""
from __future__ import annotations

import math

import numpy as np

from . import fluid, synth

FORBIDDEN = 1e9   # cost of a layout combination other than the forced one, inside a measuring plan


class MeasuredEval:
    def __init__(self, desc: synth.GraphDesc, candidates: dict, reps: int = 5, warmup: int = 2, seed: int = 7,
                 variants: bool = False):
        import torch
        self.torch = torch
        self.desc, self.cands, self.reps, self.warmup, self.seed = desc, candidates, reps, warmup, seed
        self.table = {}        # (signature, layouts[, variant]) -> seconds
        self.measured = 0      # GPU measurements taken (table misses)
        self._c = fluid.EVAL_FN(self._call)
        self._cv = fluid.EVAL_VARIANT_FN(self._call_variant) if variants else None

    @property
    def callback_variant(self):
        """The C function pointer for `fluid.Plan(..., eval_variant=...)` (needs variants=True)."""
        return self._cv

    def _call_variant(self, user, node, n, tids, lidx, variant):
        try:
            return self.cost(int(node), {int(tids[i]): int(lidx[i]) for i in range(n)}, int(variant))
        except Exception:
            return math.inf

    @property
    def callback(self):
        """The C function pointer for `fluid.Plan(..., eval=...)` (keep this object alive while planning)."""
        return self._c

    # ---- the planner's side ----
    def _call(self, user, node, n, tids, lidx):
        try:
            return self.cost(int(node), {int(tids[i]): int(lidx[i]) for i in range(n)})
        except Exception:   # never let an exception cross the C boundary: unknown means unusable
            return math.inf

    def cost(self, op_id: int, layout_index: dict, variant: int = 0) -> float:
        op = self.desc.ops[op_id]
        tids = list(op["ins"]) + list(op["outs"])
        perms = tuple(tuple(self.cands.get(t, [synth.identity_perm(len(self.desc.dims(t)))])[layout_index.get(t, 0)])
                      for t in tids)
        attrs = tuple(sorted((k, tuple(v) if isinstance(v, (list, tuple)) else v) for k, v in op["attrs"].items()))
        sig = (op["kind"], attrs,
               tuple((self.desc.tensors[t]["dtype"], tuple(self.desc.dims(t))) for t in tids))
        key = (sig, perms, variant)
        if key not in self.table:
            self.table[key] = self._measure(op, tids, perms, variant)
            self.measured += 1
        return self.table[key]

    # ---- one measurement ----
    def _measure(self, op, tids, perms, variant=0) -> float:
        torch = self.torch
        d = self.desc
        g = synth.GraphDesc()
        local, cands, consts, fed = {}, {}, {}, {}     # fed: local input / state tensor -> array handed to the runner
        for slot, (t, perm) in enumerate(zip(op["ins"], perms)):
            src = d.tensors[t]
            if t in local:                                 # the same tensor in two roles (the position of a decoding step)
                continue
            if src["dtype"] == synth.I32:
                lt = g.tensor(f"in{t}", synth.I32, src["dims"], synth.INPUT)
                if op["kind"] == synth.EMBED and slot == 0:     # ids index the first dim of the table they look up
                    fed[lt] = np.asarray(synth.token_ids(self.seed, 0, src["dims"], d.dims(op["ins"][1])[0]), dtype=np.int32)
                else:                                           # a position: the start of the sequence
                    fed[lt] = np.zeros(src["dims"], dtype=np.int32)
            elif src["kind"] == synth.STATE:
                # a caller-owned cache: canonical, read and updated in place by the timed step
                lt = g.tensor(f"in{t}", src["dtype"], src["dims"], synth.STATE)
                fed[lt] = np.zeros(src["dims"], dtype=np.float32)
            else:
                # a constant may sit in any candidate layout and is packed outside the timed path
                lt = g.tensor(f"in{t}", src["dtype"], src["dims"], synth.CONST)
                a = synth.uniform(self.seed, lt, src["dims"], -1.0, 1.0)
                consts[lt] = synth.round_bf16(a) if src["dtype"] == synth.BF16 else a
            local[t] = lt
            ident = synth.identity_perm(len(src["dims"]))
            cands[lt] = [ident] if tuple(perm) == ident else [ident, tuple(perm)]
        (t_out,), perm_out = op["outs"], perms[len(op["ins"])]
        src = d.tensors[t_out]
        y = g.tensor("y", src["dtype"], src["dims"], synth.ACT)
        z = g.tensor("z", src["dtype"], src["dims"], synth.OUTPUT)
        ident = synth.identity_perm(len(src["dims"]))
        cands[y] = [ident] if tuple(perm_out) == ident else [ident, tuple(perm_out)]
        cands[z] = [ident]
        g.op(op["kind"], [local[t] for t in op["ins"]], [y], **op["attrs"])
        g.op(synth.TRANSPOSE, [y], [z], perm=list(ident))
        want = {lt: len(c) - 1 for lt, c in cands.items()}   # index of the forced layout of each local tensor

        def forcing(user, node, n, ltids, lidx):
            if node != 0:
                return 0.0
            return 0.0 if all(lidx[i] == want[ltids[i]] for i in range(n)) else FORBIDDEN

        cb = fluid.EVAL_FN(forcing)
        try:
            plan = fluid.Plan(g, cands, eval=cb, **({"op_variant": {0: variant}} if variant else {}))
        except fluid.FluidError:
            return math.inf
        try:
            got = {lt: plan.tensor_info(lt).layout_index for lt in want}
            if got != want:
                return math.inf   # the planner could not honour the combination (its guard fell back to canonical)
            if variant and plan.gemm_variants(0)[1] != variant:
                return math.inf   # the step cannot run with this variant under these layouts
            runner = fluid.Runner(plan, consts)
            if fed:
                runner.set_inputs([fed[lt] for lt in g.inputs])
            steps = plan.steps()
            mine = [i for i, s in enumerate(steps) if 0 in s["ops"]]
            if len(mine) != 1:
                return math.inf
            stream = torch.cuda.current_stream().cuda_stream
            args = (plan.handle, runner.arena.data_ptr(), [b.data_ptr() for b in runner.inputs],
                    [b.data_ptr() for b in runner.outputs], stream)
            for _ in range(self.warmup):
                fluid.fluid_run(*args)
            ms = [fluid.fluid_run_profiled(*args)[mine[0]] for _ in range(self.reps)]
            torch.cuda.synchronize()
            if runner.status() != 0:
                return math.inf
            return float(np.median(ms)) * 1e-3
        except fluid.FluidError:
            return math.inf
        finally:
            plan.close()


def tune_step_variants(desc: synth.GraphDesc, candidates: dict, consts: dict, inputs: list, reps: int = 5, warmup: int = 2,
                       **options):
    """Times every tensor-core GEMM step of the plan for `desc` with each implementation variant its shape admits, in
    place: the whole plan runs (fused epilogues, grouped sibling projections, the real producers and consumers around
    the step) with one CUDA event pair per step, once per variant rank. Returns (op_variant, table): op_variant maps
    the anchor op of each step to its fastest variant, ready for `fluid.Plan(..., op_variant=...)`; table maps anchor
    op -> {variant code: seconds}. Steps with the same shapes and variant list (the layers of a model) share one
    set of measurements."""
    import torch
    base = fluid.Plan(desc, candidates, **options)
    try:
        gemm_steps = [(i, s) for i, s in enumerate(base.steps()) if s["kernel_name"] == "GEMM_TC"]
        avail = {s["ops"][0]: base.gemm_variants(s["ops"][0])[0] for _, s in gemm_steps}

        def signature(s):
            return (tuple(tuple(desc.dims(t)) for t in s["ins"] + s["outs"]), len(s["ops"]), tuple(avail[s["ops"][0]]))

        groups = {}
        for i, s in gemm_steps:
            groups.setdefault(signature(s), []).append((i, s["ops"][0]))
        n_ranks = max((len(v) for v in avail.values()), default=0)
    finally:
        base.close()
    times = {}      # (signature, code) -> seconds
    for rank in range(n_ranks):
        # one plan per rank: the first step of every group runs its rank-th variant
        force = {ops[0][1]: avail[ops[0][1]][rank] for ops in groups.values() if rank < len(avail[ops[0][1]])}
        plan = fluid.Plan(desc, candidates, op_variant=force, **options)
        try:
            runner = fluid.Runner(plan, consts)
            runner.set_inputs(inputs)
            for _ in range(warmup):
                runner.run()
            ms = np.median(np.array([runner.run_profiled() for _ in range(reps)]), axis=0)
            torch.cuda.synchronize()
            if runner.status() != 0:
                continue
            steps = plan.steps()
            for sig, ops in groups.items():
                idx, op = ops[0]
                if op in force and idx < len(steps) and steps[idx]["ops"][0] == op and plan.gemm_variants(op)[1] == force[op]:
                    times[(sig, force[op])] = float(ms[idx]) * 1e-3
            del runner
        finally:
            plan.close()
    op_variant, table = {}, {}
    for sig, ops in groups.items():
        mine = {code: t for (g, code), t in times.items() if g == sig}
        if not mine:
            continue
        best = min(mine, key=mine.get)
        for _, op in ops:
            op_variant[op] = best
            table[op] = dict(mine)
    return op_variant, table
