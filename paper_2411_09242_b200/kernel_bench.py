"""Single-kernel measurements: each case is a one-operator graph planned and run through the C-ABI, timed with
CUDA events over a CUDA-graph replay of several runs (so launch overhead is amortised), reported as algorithmic
bytes (or flops) per second. The cases are the memory-bound kernels at sizes well beyond L2 and the GEMM / layout
sweep shapes. (The replay re-reads the same operands: a case whose operands fit the 126 MB L2, such as the few-row
GEMMs below 100 MB, is served from L2 and reads optimistic; the decoding workload of bench.py is the honest figure.)

    python -m paper_2411_09242_b200.kernel_bench [substring ...]

Synthetic inputs (uniform values, random token ids); nothing here checks results (the parity tests do).
"""
from __future__ import annotations

import sys

from . import build, fluid, synth

BF = synth.BF16


def _one_op(kind, in_shapes, out_shape, attrs=None):
    g = synth.GraphDesc()
    ins = [g.tensor(f"in{i}", BF, shp, synth.INPUT) for i, shp in enumerate(in_shapes)]
    out = g.tensor("out", BF, out_shape, synth.OUTPUT)
    g.op(kind, ins, [out], **(attrs or {}))
    return g


def cases():
    """(name, graph, bytes(n_out_elements) or None, flops or None)"""
    out = []
    out.append(("softmax dense 32x2048x2048", _one_op(synth.SOFTMAX, [[1, 32, 2048, 2048]], [1, 32, 2048, 2048], {"causal": 0, "scale": 1.0}),
                lambda n: 2 * n * 2, None))
    out.append(("softmax causal 32x2048x2048", _one_op(synth.SOFTMAX, [[1, 32, 2048, 2048]], [1, 32, 2048, 2048], {"causal": 1, "scale": 1.0}),
                lambda n: 2 * n * 0.5 * 2, None))
    out.append(("layernorm 65536x768", _one_op(synth.LAYERNORM, [[1, 65536, 768], [768], [768]], [1, 65536, 768], {"eps": 1e-5}),
                lambda n: 2 * n * 2, None))
    out.append(("rmsnorm 16384x4096", _one_op(synth.RMSNORM, [[1, 16384, 4096], [4096]], [1, 16384, 4096], {"eps": 1e-5}),
                lambda n: 2 * n * 2, None))
    out.append(("rope 4x2048x32x128", _one_op(synth.ROPE, [[4, 2048, 32, 128]], [4, 2048, 32, 128], {"rope_base": 10000.0}),
                lambda n: 2 * n * 2, None))
    out.append(("add 8192x11008", _one_op(synth.ADD, [[1, 8192, 11008]] * 2, [1, 8192, 11008]), lambda n: 3 * n * 2, None))
    out.append(("gelu 8192x11008", _one_op(synth.GELU, [[1, 8192, 11008]], [1, 8192, 11008]), lambda n: 2 * n * 2, None))
    g = synth.GraphDesc()
    a = g.tensor("a", BF, [1, 8192, 11008], synth.INPUT)
    b = g.tensor("b", BF, [1, 8192, 11008], synth.INPUT)
    s_ = g.tensor("s", BF, [1, 8192, 11008], synth.ACT)
    o = g.tensor("o", BF, [1, 8192, 11008], synth.OUTPUT)
    g.op(synth.SILU, [a], [s_])
    g.op(synth.MUL, [s_, b], [o])
    out.append(("silu*mul 8192x11008", g, lambda n: 3 * n * 2, None))
    for tgt in ("BHSD", "BHDS"):
        for (B, S, nh, D) in ((8, 2048, 32, 128), (8, 2048, 12, 64)):
            gg, _ = synth.permute_case(B, S, nh, D, tgt)
            out.append((f"permute {tgt} {B}x{S}x{nh}x{D}", gg, lambda n: 2 * n * 2, None))
    g = synth.GraphDesc()
    ids = g.tensor("ids", synth.I32, [16, 2048], synth.INPUT)
    tok = g.tensor("tok", BF, [32000, 4096], synth.INPUT)
    x = g.tensor("x", BF, [16, 2048, 4096], synth.OUTPUT)
    g.op(synth.EMBED, [ids, tok], [x])
    out.append(("embed 32768x4096", g, lambda n: 2 * n * 2, None))
    # (128, 1, 128, 2048) moves the same bytes as (4, 32, 128, 2048) with every head's rows contiguous in memory
    for (B_, nh, D, T) in ((4, 32, 128, 2048), (128, 1, 128, 2048), (16, 32, 128, 4096), (4, 12, 64, 2048)):
        g = synth.GraphDesc()
        q = g.tensor("q", BF, [B_, 1, nh, D], synth.INPUT)
        k = g.tensor("k", BF, [B_, 1, nh, D], synth.INPUT)
        v = g.tensor("v", BF, [B_, 1, nh, D], synth.INPUT)
        kc = g.tensor("kc", BF, [B_, T, nh, D], synth.STATE)
        vc = g.tensor("vc", BF, [B_, T, nh, D], synth.STATE)
        pos = g.tensor("pos", synth.I32, [1], synth.INPUT)
        o = g.tensor("ctx", BF, [B_, 1, nh, D], synth.OUTPUT)
        g.op(synth.CACHED_ATTENTION, [q, k, v, kc, vc, pos], [o], scale=D ** -0.5)
        out.append((f"decode attention {B_}x{nh}x{D} cache {T}", g, lambda n, b=2.0 * 2 * B_ * T * nh * D: b, None))
    for (M, N, K) in ((768, 768, 768), (2048, 2048, 2048), (4096, 4096, 4096), (8192, 8192, 8192), (4096, 2304, 768), (4096, 3072, 768),
                      (2048, 11008, 4096), (128, 768, 3072), (128, 3072, 768), (4, 50257, 768),
                      (4, 4096, 4096), (4, 11008, 4096), (4, 4096, 11008), (4, 32000, 4096)):
        for majors in (("row", "col"), ("col", "row")) if M == N == K and M <= 4096 else (("row", "col"),):
            gg, _ = synth.gemm_case(M, N, K, *majors, materialize=False)
            # few rows: the step streams the weight once, so bytes are the figure; otherwise flops
            out.append((f"gemm {M}x{N}x{K} A {majors[0]} B {majors[1]}", gg,
                        (lambda n, b=2.0 * (M * K + K * N + M * N): b) if M <= 16 else None, 2.0 * M * N * K))
    return out


def main(argv):
    import torch
    build.build()
    only = [a for a in argv if not a.startswith("-")]
    reps = 10
    for name, g, fbytes, flops in cases():
        if only and not any(o in name for o in only):
            continue
        plan = fluid.Plan(g, synth.default_candidates(g))
        r = fluid.Runner(plan, {})
        for b_ in r.inputs:
            if b_.dtype == torch.int32 and b_.numel() == 1:
                b_.fill_(g.dims(g.inputs[3])[1] - 1 if len(g.inputs) > 3 else 0)   # a decoding position: the last cache row
            elif b_.dtype == torch.int32:
                b_.random_(0, 32000)
            else:
                b_.uniform_(-2, 2)
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            for _ in range(3):
                r.run(st)
            st.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=st):
                for _ in range(reps):
                    r.run(torch.cuda.current_stream())
            graph.replay()
            st.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            graph.replay()
            e1.record(st)
            st.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / reps
        n = 1
        for d in g.tensors[g.outputs[0]]["dims"]:
            n *= d
        steps = "+".join(s["kernel_name"] for s in plan.steps())
        if flops is not None and fbytes is None:
            print(f"{name:44s} {steps:10s} {us:9.1f} us  {flops / us / 1e6:8.1f} TFLOP/s  status {r.status()}")
        else:
            by = fbytes(n)
            print(f"{name:44s} {steps:10s} {us:9.1f} us  {by / us / 1e3:8.1f} GB/s algorithmic ({by / 1e6:.0f} MB)  status {r.status()}")
        plan.close()
        del r
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main(sys.argv[1:])
