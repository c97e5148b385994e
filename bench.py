#!/usr/bin/env python
"""Benchmark of the planned-arena transformer executor on B200.

One "step" = one whole planned inference (every kernel step of the plan) of one synthetic batch.
Headline workload: the Llama-shaped prefill (4 layers, hidden 4096, 32 heads, FFN 11008, seq 2048, batch 1,
bf16), the largest single-GPU configuration. Prints ONE JSON line: end-to-end latency (ms), peak arena MB, the
roofline of the dominant kernel, parity of the timed configuration against the fp64 oracle, the oracle's CPU time
beside it, and a summary (latency, arena, per-kernel rooflines, parity, clocks) of the other model workloads, the
decoding step and the layout-transform / layout-aware GEMM sweep.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With N > 1 (torchrun) every rank runs an independent replica: the path has no exchange step.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2411_09242_b200 import synth  # noqa: E402

METRIC = "end_to_end_inference_latency_ms"
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index=0):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            parts = [p.strip() for p in s.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0])); mx = float(parts[1])
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a short list of floats over all ranks (identity without a process group)."""
    import torch
    t = torch.tensor(values, device=device, dtype=torch.float64)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def feeds_of(m):
    f = dict(m.consts)
    f[m.graph.inputs[0]] = m.ids
    return f


def oracle_forward(m):
    from oracle import graph_exec
    t0 = time.perf_counter()
    out = graph_exec.run_graph(m.graph.tensors, m.graph.ops, feeds_of(m))
    return out, time.perf_counter() - t0


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def oracle_sample_config(cfg):
    """A bounded sample of the workload for the CPU oracle (a few seconds of CPU work per pass), the same in both
    arms. Returns (sample config, description, whole-workload tokens / sample tokens)."""
    if cfg.name in ("tiny", "bert_base"):
        return cfg, "the whole workload (one full forward pass)", 1.0
    if cfg.name == "gpt2_small":
        s = synth.scaled(cfg, B=1, S=min(cfg.S, 256))
        return s, f"batch row 0, first {s.S} positions, all {cfg.L} layers (causal prefix); time scaled by tokens", \
            cfg.B * cfg.S / (s.B * s.S)
    s = synth.scaled(cfg, S=min(cfg.S, 256))
    return s, f"first {s.S} positions, all {cfg.L} layers (causal prefix); time scaled by tokens", cfg.S / s.S


def sample_model(full, scfg):
    """The sample's graph bound to the full model's weights (nothing is generated twice)."""
    if scfg == full.cfg:
        return full
    small = synth.build_model(scfg, materialize=False)
    by_name = {full.graph.tensors[t]["name"]: a for t, a in full.consts.items()}
    consts = {}
    for tid, td in enumerate(small.graph.tensors):
        if td["kind"] == synth.CONST:
            a = by_name[td["name"]]
            consts[tid] = a[:scfg.S] if td["name"] == "pos_table" else a
    return synth.Model(scfg, small.graph, consts, full.ids[:scfg.B, :scfg.S])


def time_oracle_sample(m, warmup, steps, budget_s=None):
    """warmup untimed passes, then `steps` timed ones (fewer if budget_s runs out): seconds per pass."""
    times = []
    for i in range(warmup + steps):
        _, dt = oracle_forward(m)
        if i >= warmup:
            times.append(dt)
        if budget_s is not None and i >= warmup and sum(times) > budget_s:
            break
    return times


class L2Flush:
    """Called between timed iterations, outside the event pair: writes a buffer larger than L2 (nothing of the
    workload stays cached), then reads a second one, so that the dirty lines the write leaves behind (up to the
    L2's 126 MB) are written back here and not inside the timed region. (Measured on a read-only streaming kernel:
    after a written flush alone, ~19 us of write-back fell into the launch that followed.)"""

    def __init__(self, torch, mib=256):
        self.written = torch.empty(mib << 20, dtype=torch.uint8, device="cuda")
        self.read = torch.zeros(mib << 20, dtype=torch.uint8, device="cuda")

    def __call__(self):
        self.written.fill_(1)
        self.read.max()


def config_of(cfg, world):
    return {"workload": cfg.name, "layers": cfg.L, "hidden": cfg.H, "heads": cfg.nh, "ffn": cfg.F,
            "seq_len": cfg.S, "batch": cfg.B, "vocab": cfg.V, "replicas": world,
            "launch": "CUDA graph replay of one fluid_run",
            "l2": "flushed between timed steps (256 MiB written, then 256 MiB of a second buffer read, outside the event pair)"}


def time_decode(steps, warmup, torch, fluid, peaks, batch=4, t_max=2048):
    """The second workload: one decoding step of the llama-shaped model (one new token per sequence) against
    key/value caches holding t_max - 1 earlier tokens (the longest, most expensive step). The step is bound by
    reading every weight and every cached row once: bytes streamed / time is reported against the copy peak."""
    cfg = synth.scaled(synth.CONFIGS["llama"], S=1, B=batch)
    dec = synth.build_decode_model(cfg, t_max)
    g = dec.graph
    plan = fluid.Plan(g, synth.default_candidates(g))
    runner = fluid.Runner(plan, dec.consts)
    for t in g.inputs:
        buf = runner.inputs[g.inputs.index(t)]
        if t == dec.pos:
            buf.fill_(t_max - 1)
        elif t == dec.ids:
            buf.copy_(torch.from_numpy(synth.token_ids(synth.TOKEN_SEED, 1, [batch, 1], cfg.V)))
        else:
            buf.uniform_(-1, 1)      # cache contents: values only matter to the parity tests
    stream = torch.cuda.Stream()
    flush = L2Flush(torch)
    with torch.cuda.stream(stream):
        for _ in range(max(3, warmup)):
            runner.run(stream)
        stream.synchronize()
        assert runner.status() == 0
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            runner.run(torch.cuda.current_stream())
        ts = []
        for _ in range(steps):
            flush()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); graph.replay(); b.record(stream)
            b.synchronize()
            ts.append(a.elapsed_time(b))
    es = synth.DTYPE_BYTES[cfg.dtype]
    # every constant but the embedding table (gathered: batch rows of it) is read once, and so are the cached rows
    w_bytes = sum(a.size for t, a in dec.consts.items() if g.tensors[t]["name"] != "tok_table") * es + batch * cfg.H * es
    c_bytes = 2 * cfg.L * batch * t_max * cfg.H * es
    ms = float(np.mean(ts))
    info = plan.steps()
    res = {"workload": "llama_decode", "batch": batch, "cache_rows": t_max, "position": t_max - 1, "layers": cfg.L,
           "latency_ms": ms, "latency_min_ms": float(np.min(ts)), "tokens_per_s": batch / (ms * 1e-3),
           "kernel_steps": len(info), "kernels": sorted({s["kernel_name"] for s in info}),
           "weight_mb": w_bytes / 2 ** 20, "cache_mb": c_bytes / 2 ** 20, "arena_mb": plan.arena_bytes / 2 ** 20,
           "streamed_gbs": (w_bytes + c_bytes) / (ms * 1e-3) / 1e9,
           "frac_measured_hbm": (w_bytes + c_bytes) / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    plan.close()
    return res


def run_reference(args, rank):
    """The reference arm: the CPU oracle as it stands, timed on this machine's host cores: W untimed passes over the
    bounded sample, then K timed ones; the value is the mean pass scaled to the whole workload by tokens."""
    if rank != 0:
        return
    cfg = synth.CONFIGS[args.workload]
    scfg, sample, scale = oracle_sample_config(cfg)
    m = synth.build_model(scfg)
    times = time_oracle_sample(m, args.warmup, args.steps)
    ms = 1e3 * float(np.mean(times)) * scale
    line = {"impl": "reference", "metric": METRIC, "value": ms, "unit": "ms", "n_gpus": args.gpus,
            "steps": len(times), "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(cfg, max(1, args.gpus)),
            "cpu_baseline": {"value": ms, "unit": "ms", "cores": cpu_threads(), "kind": "oracle", "sample": sample,
                             "sample_pass_ms": 1e3 * float(np.mean(times)), "scaled_by": scale},
            "e2e": {"value": ms, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel, per launch, from the ncu capture
# summarised in the named file under profiles/ (null where no capture of that workload was taken)
NCU_TRAFFIC = {
    "llama": {"kernel": "GEMM_TC", "bytes_per_launch": 181800000,
              "source": "profiles/launch_list_llama.md (34 GEMM_TC launches, dram read + write)"},
    "bert_base": {"kernel": "GEMM_TC", "bytes_per_launch": 4122080,
                  "source": "profiles/dram_traffic_bert_base.md (the four GEMM steps of two layers, dram read + write)"},
}


def roofline_of(kernels, peaks, step_ms=None):
    """Roofline entry for the kernel with the largest share of the step.

    `achieved` uses the kernel's launch durations from one event pair per step (launches serialised by the events: no
    overlap of a step's prologue with its predecessor's tail). A tensor-bound kernel is set against the measured
    BURST bf16 rate (`frac`), the stricter of the two measured peaks; the timed steps run back to back for seconds and
    the clocks sampled beside them usually show the power cap active, which is the regime of the SUSTAINED figure:
    `frac_of_sustained` stands beside it, and so does `frac_of_nominal`. `in_step` is an estimate, not a measurement: the timed step (graph
    replay, where programmatic dependent launch overlaps neighbours) times this kernel's share of the per-step
    event times."""
    name = max(kernels, key=lambda k: kernels[k]["ms"])
    dom = kernels[name]
    if dom["bound"] == "tensor":
        roof = {"bound": "tensor", "achieved": dom["tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                "frac_of_sustained": dom["tflops"] / peaks["bf16_tflops_sustained"],
                "peak_kind": "burst (cuBLAS bf16 8192^3, best of 10)"}
    else:
        roof = {"bound": "hbm", "achieved": dom["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s"}
    roof.update({"frac": roof["achieved"] / roof["peak"], "traffic": None, "kernel": name,
                 "launches_per_step": dom["launches"], "avg_launch_us": dom["ms"] / dom["launches"] * 1e3,
                 "share_of_step": dom["share"], "peak_source": peaks["source"], "frac_of_nominal": dom["frac_nominal"],
                 "algorithmic_per_launch": (dom["flops"] if dom["bound"] == "tensor" else dom["bytes"]) / dom["launches"]})
    if step_ms:
        us = step_ms * dom["share"] / dom["launches"] * 1e3
        ach = roof["algorithmic_per_launch"] / (us * 1e-6) / (1e12 if dom["bound"] == "tensor" else 1e9)
        roof["in_step"] = {"avg_launch_us": us, "achieved": ach, "frac": ach / roof["peak"],
                           "how": "estimate: timed step (graph replay) x this kernel's share of the per-step event times / launches"}
    return roof


def parity_of(m, plan, outs, fluid_mod, storage=True):
    """Whole outputs of the timed configuration against one full pass of the fp64 oracle. Where a bf16 workload
    misses the stated tolerance, a second pass rounds every tensor to the dtype the plan stores it in (exact fp64
    arithmetic otherwise): its distance from the plain pass is the floor no executor with this storage gets under."""
    ref, dt = oracle_forward(m)
    tol = 1e-2 if m.cfg.dtype == synth.BF16 else 1e-4
    errs = [float(np.max(np.abs(got - ref[tid])) / np.max(np.abs(ref[tid]))) for tid, got in zip(m.graph.outputs, outs)]
    par = {"max_err_over_max_ref": max(errs), "tolerance": tol, "ok": bool(max(errs) <= tol),
           "compared": "every element of every output", "oracle_full_pass_s": dt}
    if not par["ok"] and storage and m.cfg.dtype == synth.BF16:
        from oracle import graph_exec
        from tests.helpers import storage_hooks
        store, load = storage_hooks(m.graph, plan)
        rs = graph_exec.run_graph(m.graph.tensors, m.graph.ops, feeds_of(m), store=store, load=load)
        par["storage_floor"] = max(float(np.max(np.abs(rs[t] - ref[t])) / np.max(np.abs(ref[t]))) for t in m.graph.outputs)
        par["vs_storage_rounded_oracle"] = max(float(np.max(np.abs(got - rs[t])) / np.max(np.abs(ref[t])))
                                               for t, got in zip(m.graph.outputs, outs))
        par["note"] = ("storage_floor: fp64 arithmetic with the plan's storage dtypes (bf16 operands, fp32 residual "
                       "stream) vs the unrounded oracle; the stated tolerance is below it for this shape")
    return par, dt


def time_workload(name, steps, warmup, torch, fluid, peaks, full=True, sampler=None, overrides=None, plan_opts=None,
                  parity=False):
    """Plan, bind and time one model workload; returns a dict of measurements."""
    cfg = synth.CONFIGS[name]
    if overrides:
        cfg = synth.scaled(cfg, **overrides)
    m = synth.build_model(cfg)
    cands = synth.default_candidates(m.graph)
    # the plan that runs places the arena with Algorithm 4 over several record orders (arena_policy 2, the smallest
    # kept); the sizes the algorithm gives as printed (first fit) and by its prose (best fit) are reported beside it
    plan_opts = dict({"arena_policy": 2}, **(plan_opts or {}))
    t0 = time.perf_counter()
    plan = fluid.Plan(m.graph, cands, **plan_opts)
    plan_ms = 1e3 * (time.perf_counter() - t0)
    canon = fluid.Plan(m.graph, None)
    sizes = {}
    for label, extra in (("first_fit", {"arena_policy": 0}), ("best_fit", {"arena_policy": 1}),
                         ("no_inplace", {"arena_policy": 2, "no_inplace": 1})):
        q = fluid.Plan(m.graph, cands, **dict(plan_opts, **extra))
        sizes[label] = q.arena_bytes / 2 ** 20
        q.close()
    runner = fluid.Runner(plan, m.consts)
    runner.set_inputs([m.ids])
    stream = torch.cuda.Stream()
    flush = L2Flush(torch)
    steps_info = plan.steps()
    n_steps = len(steps_info)
    res = {"workload": name, "arena_mb": plan.arena_bytes / 2 ** 20, "arena_naive_mb": plan.naive_bytes / 2 ** 20,
           "arena_live_bound_mb": plan.live_bound_bytes / 2 ** 20, "arena_canonical_plan_mb": canon.arena_bytes / 2 ** 20,
           "arena_policy": "Algorithm 4 over several record orders, smallest kept; in-place results share their operand's slice",
           "arena_first_fit_mb": sizes["first_fit"], "arena_best_fit_mb": sizes["best_fit"],
           "arena_without_inplace_mb": sizes["no_inplace"],
           "weights_mb": sum(a.size for a in m.consts.values()) * synth.DTYPE_BYTES[cfg.dtype] / 2 ** 20,
           "kernel_steps": n_steps, "plan_ms": plan_ms, "tokens": cfg.B * cfg.S,
           "planned_cost_ms": plan.cost * 1e3, "canonical_cost_ms": plan.canonical_cost * 1e3}
    with torch.cuda.stream(stream):
        for _ in range(max(3, warmup)):
            runner.run(stream)
        stream.synchronize()
        assert runner.status() == 0
        # CUDA graph of one fluid_run: the launches are captured once and replayed per step
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            runner.run(torch.cuda.current_stream())
        for _ in range(2):
            graph.replay()
        stream.synchronize()

        def timed(fn, k):
            ts = []
            for _ in range(k):
                flush()          # evict L2 between timed iterations (outside the event pair)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream); fn(); b.record(stream)
                b.synchronize()
                ts.append(a.elapsed_time(b))
            return ts

        if sampler:
            sampler.start()
        launches0 = fluid.fluid_launch_count()
        t_graph = timed(graph.replay, steps)
        t_eager = timed(lambda: runner.run(stream), steps)
        res["clocks"] = sampler.stop() if sampler else None
        res["eager_launches_counted"] = int(fluid.fluid_launch_count() - launches0)
        res["latency_ms"] = float(np.mean(t_graph))
        res["latency_min_ms"] = float(np.min(t_graph))
        res["latency_median_ms"] = float(np.median(t_graph))
        res["latency_eager_ms"] = float(np.mean(t_eager))
        # end to end through the public API with host buffers: H2D ids, run, D2H outputs
        ids_host = torch.from_numpy(m.ids).pin_memory()
        outs_host = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in runner.outputs]

        def e2e_step():
            runner.inputs[0].copy_(ids_host, non_blocking=True)
            graph.replay()
            for h, d in zip(outs_host, runner.outputs):
                h.copy_(d, non_blocking=True)

        t_e2e = timed(e2e_step, steps)
        res["e2e_ms"] = float(np.mean(t_e2e))
        res["h2d_bytes"] = int(ids_host.numel() * 4)
        res["d2h_bytes"] = int(sum(o.numel() * o.element_size() for o in outs_host))
        # per-kernel profile (event pair per step), eager
        prof = np.zeros(n_steps)
        reps = 3
        for _ in range(reps):
            flush()
            prof += np.array(fluid.fluid_run_profiled(plan.handle, runner.arena.data_ptr(),
                                                      [b.data_ptr() for b in runner.inputs],
                                                      [b.data_ptr() for b in runner.outputs], stream.cuda_stream))
        prof /= reps
    kernels = {}
    for info, ms in zip(steps_info, prof):
        k = kernels.setdefault(info["kernel_name"], {"launches": 0, "ms": 0.0, "flops": 0.0, "bytes": 0.0})
        k["launches"] += 1; k["ms"] += float(ms); k["flops"] += info["flops"]; k["bytes"] += info["bytes"]
    total = sum(k["ms"] for k in kernels.values()) or 1.0
    ridge = peaks["bf16_tflops"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    for name_k, k in kernels.items():
        k["share"] = k["ms"] / total
        k["gbs"] = k["bytes"] / (k["ms"] * 1e-3) / 1e9 if k["ms"] > 0 else 0.0
        k["tflops"] = k["flops"] / (k["ms"] * 1e-3) / 1e12 if k["ms"] > 0 else 0.0
        k["bound"] = "tensor" if (k["flops"] / max(k["bytes"], 1.0)) > ridge and name_k in ("GEMM_TC", "ATTN") else "hbm"
        if k["bound"] == "tensor":
            k["frac_measured"] = k["tflops"] / peaks["bf16_tflops"]            # of the measured burst rate
            k["frac_sustained"] = k["tflops"] / peaks["bf16_tflops_sustained"]
            k["frac_nominal"] = k["tflops"] / NOMINAL["bf16_tflops"]
        else:
            k["frac_measured"] = k["gbs"] / peaks["hbm_gbs"]
            k["frac_nominal"] = k["gbs"] / NOMINAL["hbm_gbs"]
    res["kernels"] = kernels
    res["roofline"] = roofline_of(kernels, peaks, step_ms=res["latency_ms"])
    res["profile_total_ms"] = float(total)
    if parity:
        res["parity"], res["oracle_full_pass_s"] = parity_of(m, plan, runner.outputs_host(), fluid)
    if full:
        res["_model"], res["_runner"], res["_plan"] = m, runner, plan
    else:
        plan.close()
    canon.close()
    return res


def time_sweep(torch, fluid, peaks, reps=5):
    """The layout-transform and layout-aware GEMM sweep: all 192 permute cases ([B,S,nh,D] -> [B,nh,S,D] and
    [B,nh,D,S]; B 1..8, S 128/512/2048, nh 12/32, D 64/128) and the 12 GEMM cases (M=N=K 768/2048/4096, A and B each
    row- or column-major), each planned and run through the C-ABI alone, timed with an event pair around one launch
    with the L2 flushed before it. Parity inline: every permute output bit for bit against the oracle's transpose
    (whole tensor up to 64 MiB of traffic, else batch row 0 and the last one); 64 sampled rows of every GEMM
    against the oracle's linear. Cases whose traffic fits the 126 MB L2 have their output absorbed by it (and at
    under ~10 MB are launch-bound): they are counted apart."""
    from oracle import ops as oracle_ops
    flush = L2Flush(torch)
    stream = torch.cuda.current_stream()

    def run_case(g, feeds, cands=None):
        plan = fluid.Plan(g, cands)
        runner = fluid.Runner(plan, {})
        runner.set_inputs([feeds[t] for t in g.inputs])
        for _ in range(2):
            runner.run()
        ts = []
        for _ in range(reps):
            flush()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); runner.run(); b.record(stream)
            b.synchronize()
            ts.append(a.elapsed_time(b))
        assert runner.status() == 0
        kernels = [s["kernel_name"] for s in plan.steps()]
        return float(np.median(ts)), runner, plan, kernels

    perm_rows = []
    base = {}
    bit_exact = True
    for c in synth.permute_sweep_cases():
        key = (c["S"], c["nh"], c["D"])
        if key not in base:     # one seeded batch-8 tensor per (S, nh, D); smaller batches are its leading rows
            base[key] = synth.round_bf16(synth.uniform(5, len(base), [8, c["S"], c["nh"], c["D"]]))
        a = base[key][: c["B"]]
        perm = {"BHSD": [0, 2, 1, 3], "BHDS": [0, 2, 3, 1]}[c["target"]]
        g = synth.GraphDesc()
        x = g.tensor("x", synth.BF16, list(a.shape), synth.INPUT)
        y = g.tensor("y", synth.BF16, [a.shape[i] for i in perm], synth.OUTPUT)
        g.op(synth.TRANSPOSE, [x], [y], perm=perm)
        ms, runner, plan, kernels = run_case(g, {x: a})
        traffic = 2.0 * a.size * 2
        out = runner.outputs[0]
        rows = list(range(c["B"])) if traffic <= 64 * 2 ** 20 else sorted({0, c["B"] - 1})
        got = out[rows].float().cpu().numpy().astype(np.float64)
        want = oracle_ops.transpose(a[rows], perm)
        ok = bool(np.array_equal(got, want))
        bit_exact &= ok
        perm_rows.append({"case": c, "us": ms * 1e3, "gbs": traffic / (ms * 1e-3) / 1e9, "traffic_mb": traffic / 2 ** 20,
                          "bit_exact": ok, "kernel": kernels[0]})
        plan.close()
        del runner

    def summary(rows):
        if not rows:
            return None
        v = np.array([r["gbs"] for r in rows])
        return {"cases": len(rows), "min_gbs": float(v.min()), "median_gbs": float(np.median(v)), "max_gbs": float(v.max()),
                "median_frac_measured_hbm": float(np.median(v)) / peaks["hbm_gbs"],
                "median_frac_nominal_hbm": float(np.median(v)) / NOMINAL["hbm_gbs"]}

    L2_MB = 126.0
    perm_summary = {}
    for tgt in ("BHSD", "BHDS"):
        rows = [r for r in perm_rows if r["case"]["target"] == tgt]
        perm_summary[tgt] = {"beyond_l2": summary([r for r in rows if r["traffic_mb"] > L2_MB]),
                             "l2_resident": summary([r for r in rows if r["traffic_mb"] <= L2_MB]),
                             "largest": max(rows, key=lambda r: r["traffic_mb"])}
    gemm_rows = []
    gemm_ok = True
    for n in (768, 2048, 4096):
        for a_major in ("row", "col"):
            for b_major in ("row", "col"):
                g, arrs = synth.gemm_case(n, n, n, a_major, b_major)
                ms, runner, plan, kernels = run_case(g, arrs, synth.default_candidates(g))
                A = arrs[g.inputs[0]].astype(np.float64)
                Bm = arrs[g.inputs[1]].astype(np.float64)
                A = A if a_major == "row" else A.T
                Bm = Bm if b_major == "row" else Bm.T
                rows = np.linspace(0, n - 1, 64).astype(int)
                want = oracle_ops.linear(A[rows], Bm)
                got = runner.outputs[0][torch.from_numpy(rows).cuda()].float().cpu().numpy().astype(np.float64)
                err = float(np.max(np.abs(got - want)) / np.max(np.abs(want)))
                gemm_ok &= err <= 1e-2
                tf = 2.0 * n ** 3 / (ms * 1e-3) / 1e12
                gemm_rows.append({"n": n, "a": a_major, "b": b_major, "us": ms * 1e3, "tflops": tf,
                                  "frac_measured_burst": tf / peaks["bf16_tflops"], "frac_nominal": tf / NOMINAL["bf16_tflops"],
                                  "max_err_over_max_ref": err, "kernels": kernels,
                                  "note": "launch-bound by shape (36 tiles)" if n == 768 else None})
                plan.close()
                del runner
    return {"workload": "sweep", "timing": "event pair around one launch, L2 flushed before it, median of %d" % reps,
            "permute": perm_summary, "permute_cases": len(perm_rows), "permute_bit_exact": bit_exact,
            "gemm": gemm_rows, "gemm_parity_ok": gemm_ok,
            "gemm_tflops_min_median_max": [float(np.min([r["tflops"] for r in gemm_rows])),
                                           float(np.median([r["tflops"] for r in gemm_rows])),
                                           float(np.max([r["tflops"] for r in gemm_rows]))]}


def single_cases():
    """One-operator graphs for the captures under profiles/: the memory-bound kernels at sizes well beyond L2, the
    decoding kernels, a few GEMM shapes. name -> (graph, algorithmic bytes or None, flops or None)."""
    BF = synth.BF16

    def one_op(kind, in_shapes, out_shape, attrs=None):
        g = synth.GraphDesc()
        ins = [g.tensor(f"in{i}", BF, shp, synth.INPUT) for i, shp in enumerate(in_shapes)]
        out = g.tensor("out", BF, out_shape, synth.OUTPUT)
        g.op(kind, ins, [out], **(attrs or {}))
        return g

    n_big = 8192 * 11008
    out = {
        "softmax_dense": (one_op(synth.SOFTMAX, [[1, 32, 2048, 2048]], [1, 32, 2048, 2048], {"causal": 0, "scale": 1.0}), 2.0 * 32 * 2048 * 2048 * 2, None),
        "softmax_causal": (one_op(synth.SOFTMAX, [[1, 32, 2048, 2048]], [1, 32, 2048, 2048], {"causal": 1, "scale": 1.0}), 1.0 * 32 * 2048 * 2048 * 2, None),
        "layernorm_65536x768": (one_op(synth.LAYERNORM, [[1, 65536, 768], [768], [768]], [1, 65536, 768], {"eps": 1e-5}), 2.0 * 65536 * 768 * 2, None),
        "rmsnorm_16384x4096": (one_op(synth.RMSNORM, [[1, 16384, 4096], [4096]], [1, 16384, 4096], {"eps": 1e-5}), 2.0 * 16384 * 4096 * 2, None),
        "rope_4x2048x32x128": (one_op(synth.ROPE, [[4, 2048, 32, 128]], [4, 2048, 32, 128], {"rope_base": 10000.0}), 2.0 * 4 * 2048 * 32 * 128 * 2, None),
        "add_8192x11008": (one_op(synth.ADD, [[1, 8192, 11008]] * 2, [1, 8192, 11008]), 3.0 * n_big * 2, None),
        "gelu_8192x11008": (one_op(synth.GELU, [[1, 8192, 11008]], [1, 8192, 11008]), 2.0 * n_big * 2, None),
    }
    for tgt in ("BHSD", "BHDS"):
        for (B, S, nh, D) in ((8, 2048, 32, 128), (32, 2048, 32, 128), (8, 2048, 12, 64)):
            g, _ = synth.permute_case(B, S, nh, D, tgt)
            out[f"permute_{tgt}_{B}x{S}x{nh}x{D}"] = (g, 2.0 * B * S * nh * D * 2, None)
    g = synth.GraphDesc()
    ids = g.tensor("ids", synth.I32, [16, 2048], synth.INPUT)
    tok = g.tensor("tok", BF, [32000, 4096], synth.INPUT)
    x = g.tensor("x", BF, [16, 2048, 4096], synth.OUTPUT)
    g.op(synth.EMBED, [ids, tok], [x])
    out["embed_32768x4096"] = (g, 2.0 * 32768 * 4096 * 2, None)
    for (B_, nh, D, T) in ((4, 32, 128, 2048), (16, 32, 128, 4096)):
        g = synth.GraphDesc()
        q = g.tensor("q", BF, [B_, 1, nh, D], synth.INPUT)
        k = g.tensor("k", BF, [B_, 1, nh, D], synth.INPUT)
        v = g.tensor("v", BF, [B_, 1, nh, D], synth.INPUT)
        kc = g.tensor("kc", BF, [B_, T, nh, D], synth.STATE)
        vc = g.tensor("vc", BF, [B_, T, nh, D], synth.STATE)
        pos = g.tensor("pos", synth.I32, [1], synth.INPUT)
        o = g.tensor("ctx", BF, [B_, 1, nh, D], synth.OUTPUT)
        g.op(synth.CACHED_ATTENTION, [q, k, v, kc, vc, pos], [o], scale=D ** -0.5)
        out[f"decode_attention_{B_}x{nh}x{D}_cache{T}"] = (g, 2.0 * 2 * B_ * T * nh * D, None)
    for (M, N, K) in ((8192, 8192, 8192), (4096, 2304, 768), (2048, 11008, 4096), (128, 768, 3072), (4, 32000, 4096), (4, 4096, 11008),
                      (4, 128256, 4096), (4, 4096, 4096), (4, 12288, 4096), (4, 22016, 4096), (4, 50257, 768)):
        g, _ = synth.gemm_case(M, N, K, "row", "col", materialize=False)
        out[f"gemm_{M}x{N}x{K}"] = (g, 2.0 * (M * K + K * N + M * N) if M <= 16 else None, 2.0 * M * N * K)
    return out


def run_single(name, torch, fluid, peaks, reps=10):
    """One single-operator case: planned and run through the C-ABI, timed with an event pair around `reps` back-to-back
    runs. Operands of a few hundred MB defeat L2; the small GEMM shapes here are L2-resident and say so."""
    cases = single_cases()
    if name not in cases:
        raise SystemExit("unknown case; one of: " + ", ".join(cases))
    g, by, fl = cases[name]
    plan = fluid.Plan(g, synth.default_candidates(g))
    r = fluid.Runner(plan, {})
    for b_ in r.inputs:
        if b_.dtype == torch.int32 and b_.numel() == 1:
            b_.fill_(g.dims(g.inputs[3])[1] - 1 if len(g.inputs) > 3 else 0)   # a decoding position: the last cache row
        elif b_.dtype == torch.int32:
            b_.random_(0, 32000)
        else:
            b_.uniform_(-2, 2)
    for _ in range(3):
        r.run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        r.run()
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / reps
    line = {"single": name, "kernels": [s["kernel_name"] for s in plan.steps()], "us_per_run": us, "status": r.status()}
    if by is not None:
        line.update({"algorithmic_mb": by / 1e6, "gbs": by / us / 1e3, "frac_measured_hbm": by / us / 1e3 / peaks["hbm_gbs"]})
    else:
        line.update({"gflop": fl / 1e9, "tflops": fl / us / 1e6, "frac_measured_burst": fl / us / 1e6 / peaks["bf16_tflops"]})
    print(json.dumps(line), flush=True)
    plan.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--workload", default="llama", choices=list(synth.CONFIGS))
    ap.add_argument("--others", default="tiny,bert_base,gpt2_small,decode,sweep",
                    help="comma list of extra workloads to summarise (model names, decode, sweep)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--split-k", type=int, default=0, help="allow split-K GEMM steps (costs arena scratch)")
    ap.add_argument("--decode-batch", type=int, default=4, help="sequences of the decoding workload")
    ap.add_argument("--decode-cache-rows", type=int, default=2048, help="rows of its key/value caches (the step times the last)")
    ap.add_argument("--tune-variants", action="store_true",
                    help="time every tensor-core GEMM step of the headline plan with each implementation variant, in place, "
                         "and run the plan with the fastest per step (reported beside the rated plan's latency)")
    ap.add_argument("--single", default="", help="run one single-operator case (for the captures under profiles/) and exit; "
                                                 "'list' prints the names")
    ap.add_argument("--layers", type=int, default=0, help="reduced copy of the workload (profiling captures only)")
    ap.add_argument("--seq", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0)
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2411_09242_b200 import build as b
    from paper_2411_09242_b200 import fluid
    if rank == 0:
        b.build()
    if dist:
        dist.barrier()
    fluid.lib()
    peaks = load_peaks()
    args.warmup = max(3, args.warmup)
    if args.single:
        if rank == 0:
            if args.single == "list":
                print("\n".join(single_cases()))
            else:
                run_single(args.single, torch, fluid, peaks)
        return

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    overrides = {k: v for k, v in (("L", args.layers), ("S", args.seq), ("B", args.batch)) if v}
    plan_opts = {"split_k": args.split_k} if args.split_k else {}
    main_res = time_workload(args.workload, args.steps, args.warmup, torch, fluid, peaks, full=True, sampler=sampler,
                             overrides=overrides, plan_opts=plan_opts)
    tuned = None
    if args.tune_variants:
        # the paper's loop reordering with the runtime in the loop: each GEMM step's variants timed inside the plan
        from paper_2411_09242_b200 import measure
        m = main_res["_model"]
        op_variant, table = measure.tune_step_variants(m.graph, synth.default_candidates(m.graph), m.consts, [m.ids], **plan_opts)
        rated = {op: main_res["_plan"].gemm_variants(op)[1] for op in op_variant}
        changed = sorted(op for op in op_variant if op_variant[op] != rated[op])
        tuned = {"rated_latency_ms": main_res["latency_ms"], "steps_tuned": len(op_variant), "steps_changed": len(changed),
                 "changes": {str(op): {"rated": rated[op], "measured_best": op_variant[op],
                                       "us": {str(c): round(t * 1e6, 2) for c, t in table[op].items()}} for op in changed[:8]}}
        if changed:
            main_res["_runner"] = main_res["_plan"] = None
            torch.cuda.empty_cache()
            main_res = time_workload(args.workload, args.steps, args.warmup, torch, fluid, peaks, full=True,
                                     sampler=ClockSampler(local_rank) if rank == 0 else None, overrides=overrides,
                                     plan_opts=dict(plan_opts, op_variant=op_variant))
        tuned["tuned_latency_ms"] = main_res["latency_ms"]
    barrier()
    latency_ms, e2e_ms = max_over_ranks([main_res["latency_ms"], main_res["e2e_ms"]], dist, torch.device("cuda"))
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return
    cfg = synth.CONFIGS[args.workload]
    if overrides:
        cfg = synth.scaled(cfg, **overrides)
    kernels = main_res["kernels"]
    roof = roofline_of(kernels, peaks, step_ms=latency_ms)
    if args.workload in NCU_TRAFFIC and not overrides and roof["kernel"] == NCU_TRAFFIC[args.workload]["kernel"]:
        roof["traffic"] = NCU_TRAFFIC[args.workload]["bytes_per_launch"]
        roof["traffic_source"] = NCU_TRAFFIC[args.workload]["source"]
    # parity of the timed configuration against the oracle (whole outputs), and the oracle's own time on a bounded
    # sample, taken the way the reference arm takes it (one untimed pass, then timed ones)
    cpu = None
    parity = None
    if not args.no_cpu_baseline:
        m = main_res["_model"]
        parity, _ = parity_of(m, main_res["_plan"], main_res["_runner"].outputs_host(), fluid)
        scfg, sample, scale = oracle_sample_config(cfg)
        times = time_oracle_sample(sample_model(m, scfg), 1, 3, budget_s=20.0)
        cpu = {"value": 1e3 * float(np.mean(times)) * scale, "unit": "ms", "cores": cpu_threads(), "kind": "oracle",
               "sample": sample, "sample_pass_ms": 1e3 * float(np.mean(times)), "scaled_by": scale, "passes": len(times)}
    main_res["_runner"] = main_res["_plan"] = main_res["_model"] = None
    torch.cuda.empty_cache()
    others = []
    names = [n for n in args.others.split(",") if n and n != args.workload]
    for name in [n for n in names if n in synth.CONFIGS]:
        try:
            r = time_workload(name, max(5, args.steps // 3), args.warmup, torch, fluid, peaks, full=False,
                              sampler=ClockSampler(local_rank), parity=not args.no_cpu_baseline)
            others.append({k: v for k, v in r.items() if not k.startswith("_")})
        except Exception as e:  # a failed extra workload must not hide the headline number
            others.append({"workload": name, "error": repr(e)[:300]})
        torch.cuda.empty_cache()
    if "decode" in names:
        try:
            others.append(time_decode(max(5, args.steps // 3), args.warmup, torch, fluid, peaks, batch=args.decode_batch,
                                      t_max=args.decode_cache_rows))
        except Exception as e:
            others.append({"workload": "llama_decode", "error": repr(e)[:300]})
        torch.cuda.empty_cache()
    if "sweep" in names:
        try:
            others.append(time_sweep(torch, fluid, peaks))
        except Exception as e:
            others.append({"workload": "sweep", "error": repr(e)[:300]})
        torch.cuda.empty_cache()
    line = {
        "metric": METRIC, "value": latency_ms, "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": latency_ms, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if cfg.dtype == synth.BF16 else "f32", "data": "synthetic",
        "config": config_of(cfg, world),
        "peak_arena_mb": main_res["arena_mb"], "arena_naive_mb": main_res["arena_naive_mb"],
        "arena_live_bound_mb": main_res["arena_live_bound_mb"], "arena_canonical_plan_mb": main_res["arena_canonical_plan_mb"],
        "arena_first_fit_mb": main_res["arena_first_fit_mb"], "arena_best_fit_mb": main_res["arena_best_fit_mb"],
        "arena_without_inplace_mb": main_res["arena_without_inplace_mb"], "arena_policy": main_res["arena_policy"],
        "weights_mb": main_res["weights_mb"],
        "tokens_per_s": world * main_res["tokens"] / (latency_ms * 1e-3),
        "latency_eager_ms": main_res["latency_eager_ms"], "latency_min_ms": main_res["latency_min_ms"],
        "latency_median_ms": main_res["latency_median_ms"],
        "e2e": {"value": e2e_ms, "unit": "ms", "h2d_bytes_per_step": main_res["h2d_bytes"],
                "d2h_bytes_per_step": main_res["d2h_bytes"]},
        "gpu_launches": main_res["kernel_steps"] * args.steps,
        "gpu_launches_note": "kernel steps per inference x timed graph replays (the eager and host-buffer legs launch as many again each)",
        "kernel_steps_per_inference": main_res["kernel_steps"],
        "clocks": main_res["clocks"], "roofline": roof, "kernels": kernels, "cpu_baseline": cpu, "parity": parity,
        "variant_tuning": tuned,
        "other_workloads": others,
    }
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
