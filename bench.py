#!/usr/bin/env python
"""Benchmark of the planned-arena transformer executor on B200.

One "step" = one whole planned inference (every kernel step of the plan) of one synthetic batch.
Headline workload: the BERT-base-shaped encoder (12 layers, hidden 768, seq 128, batch 1, bf16).
Prints ONE JSON line: end-to-end latency (ms), peak arena MB, the roofline of the dominant
kernel, the oracle's CPU time beside it, and a short summary for the other model workloads.

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
    """A bounded sample of the workload for the CPU oracle (about 10-30 s of CPU work)."""
    if cfg.name in ("tiny", "bert_base"):
        return cfg, "the whole workload (one full forward pass)"
    if cfg.name == "gpt2_small":
        return synth.scaled(cfg, B=1, S=256), "batch row 0, first 256 positions, all 12 layers (causal prefix)"
    return synth.scaled(cfg, S=128, L=2), "first 128 positions, 2 of 4 layers"


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
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
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
            flush.fill_(1)
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
    """The reference arm: the CPU oracle as it stands, timed on this machine's host cores."""
    if rank != 0:
        return
    cfg = synth.CONFIGS[args.workload]
    scfg, sample = oracle_sample_config(cfg)
    m = synth.build_model(scfg)
    times = []
    for i in range(args.warmup + args.steps):
        _, dt = oracle_forward(m)
        if i >= args.warmup:
            times.append(dt)
        if sum(times) > 120:
            break
    ms = 1e3 * float(np.mean(times))
    line = {"impl": "reference", "metric": METRIC, "value": ms, "unit": "ms", "n_gpus": args.gpus,
            "steps": len(times), "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "sample": sample},
            "cpu_baseline": {"value": ms, "unit": "ms", "cores": cpu_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": ms, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel, per launch, from the ncu capture
# summarised in the named file under profiles/ (null where no capture of that workload was taken)
NCU_TRAFFIC = {
    "bert_base": {"kernel": "GEMM_TC", "bytes_per_launch": 4121931,
                  "source": "profiles/dram_traffic_bert_base.md (48 launches of one inference, dram read + write)"},
}


def roofline_of(kernels, peaks, step_ms=None):
    """Roofline entry for the kernel with the largest share of the step.

    `achieved` and `frac` use the kernel's launch durations from one event pair per step (launches serialised by the
    events: no overlap of a step's prologue with its predecessor's tail). When the timed step's duration (the CUDA-graph
    replay, where programmatic dependent launch overlaps neighbours) is given, `in_step` adds the same figures with the
    kernel charged its share of that step instead."""
    name = max(kernels, key=lambda k: kernels[k]["ms"])
    dom = kernels[name]
    if dom["bound"] == "tensor":
        roof = {"bound": "tensor", "achieved": dom["tflops"], "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s"}
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
                           "how": "timed step (graph replay) x this kernel's share of the per-step event times / launches"}
    return roof


def time_workload(name, steps, warmup, torch, fluid, peaks, full=True, sampler=None, overrides=None, plan_opts=None):
    """Plan, bind and time one model workload; returns a dict of measurements."""
    cfg = synth.CONFIGS[name]
    if overrides:
        cfg = synth.scaled(cfg, **overrides)
    m = synth.build_model(cfg)
    cands = synth.default_candidates(m.graph)
    t0 = time.perf_counter()
    plan = fluid.Plan(m.graph, cands, **(plan_opts or {}))
    plan_ms = 1e3 * (time.perf_counter() - t0)
    canon = fluid.Plan(m.graph, None)
    runner = fluid.Runner(plan, m.consts)
    runner.set_inputs([m.ids])
    stream = torch.cuda.Stream()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    steps_info = plan.steps()
    n_steps = len(steps_info)
    res = {"workload": name, "arena_mb": plan.arena_bytes / 2 ** 20, "arena_naive_mb": plan.naive_bytes / 2 ** 20,
           "arena_live_bound_mb": plan.live_bound_bytes / 2 ** 20, "arena_canonical_plan_mb": canon.arena_bytes / 2 ** 20,
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
                flush.fill_(1)          # evict L2 between timed iterations (outside the event pair)
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
            flush.fill_(1)
            prof += np.array(fluid.fluid_run_profiled(plan.handle, runner.arena.data_ptr(),
                                                      [b.data_ptr() for b in runner.inputs],
                                                      [b.data_ptr() for b in runner.outputs], stream.cuda_stream))
        prof /= reps
    kernels = {}
    for info, ms in zip(steps_info, prof):
        k = kernels.setdefault(info["kernel_name"], {"launches": 0, "ms": 0.0, "flops": 0.0, "bytes": 0.0})
        k["launches"] += 1; k["ms"] += float(ms); k["flops"] += info["flops"]; k["bytes"] += info["bytes"]
    total = sum(k["ms"] for k in kernels.values()) or 1.0
    ridge = peaks["bf16_tflops_sustained"] * 1e12 / (peaks["hbm_gbs"] * 1e9)
    for name_k, k in kernels.items():
        k["share"] = k["ms"] / total
        k["gbs"] = k["bytes"] / (k["ms"] * 1e-3) / 1e9 if k["ms"] > 0 else 0.0
        k["tflops"] = k["flops"] / (k["ms"] * 1e-3) / 1e12 if k["ms"] > 0 else 0.0
        k["bound"] = "tensor" if (k["flops"] / max(k["bytes"], 1.0)) > ridge and name_k in ("GEMM_TC", "ATTN") else "hbm"
        k["frac_measured"] = (k["tflops"] / peaks["bf16_tflops_sustained"]) if k["bound"] == "tensor" else (k["gbs"] / peaks["hbm_gbs"])
        k["frac_nominal"] = (k["tflops"] / NOMINAL["bf16_tflops"]) if k["bound"] == "tensor" else (k["gbs"] / NOMINAL["hbm_gbs"])
    res["kernels"] = kernels
    res["roofline"] = roofline_of(kernels, peaks, step_ms=res["latency_ms"])
    res["profile_total_ms"] = float(total)
    if full:
        res["_model"], res["_runner"], res["_plan"] = m, runner, plan
    else:
        plan.close()
    canon.close()
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--workload", default="bert_base", choices=list(synth.CONFIGS))
    ap.add_argument("--others", default="tiny,gpt2_small,llama", help="comma list of extra workloads to summarise")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--split-k", type=int, default=0, help="allow split-K GEMM steps (costs arena scratch)")
    ap.add_argument("--decode-batch", type=int, default=4, help="sequences of the decoding workload")
    ap.add_argument("--decode-cache-rows", type=int, default=2048, help="rows of its key/value caches (the step times the last)")
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

    def barrier():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    overrides = {k: v for k, v in (("L", args.layers), ("S", args.seq), ("B", args.batch)) if v}
    main_res = time_workload(args.workload, args.steps, args.warmup, torch, fluid, peaks, full=True, sampler=sampler,
                             overrides=overrides, plan_opts={"split_k": args.split_k} if args.split_k else None)
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
    # parity of the timed configuration against the oracle, and the oracle's own time
    cpu = None
    parity = None
    if not args.no_cpu_baseline:
        scfg, sample = oracle_sample_config(cfg)
        m = main_res["_model"]
        if scfg is cfg and not overrides:
            ref, dt = oracle_forward(m)
            outs = main_res["_runner"].outputs_host()
            errs = []
            for tid, got in zip(m.graph.outputs, outs):
                errs.append(float(np.max(np.abs(got - ref[tid])) / np.max(np.abs(ref[tid]))))
            parity = {"max_err_over_max_ref": max(errs), "tolerance": 1e-2 if cfg.dtype == synth.BF16 else 1e-4,
                      "ok": bool(max(errs) <= (1e-2 if cfg.dtype == synth.BF16 else 1e-4))}
        else:
            _, dt = oracle_forward(synth.build_model(scfg))
        cpu = {"value": dt * 1e3, "unit": "ms", "cores": cpu_threads(), "kind": "oracle", "sample": sample}
    others = []
    for name in [n for n in args.others.split(",") if n and n != args.workload]:
        try:
            r = time_workload(name, max(5, args.steps // 3), args.warmup, torch, fluid, peaks, full=False)
            others.append({k: v for k, v in r.items() if not k.startswith("_")})
        except Exception as e:  # a failed extra workload must not hide the headline number
            others.append({"workload": name, "error": repr(e)[:300]})
        torch.cuda.empty_cache()
    if "llama" in args.others.split(","):
        try:
            others.append(time_decode(max(5, args.steps // 3), args.warmup, torch, fluid, peaks, batch=args.decode_batch,
                                      t_max=args.decode_cache_rows))
        except Exception as e:
            others.append({"workload": "llama_decode", "error": repr(e)[:300]})
        torch.cuda.empty_cache()
    line = {
        "metric": METRIC, "value": latency_ms, "unit": "ms", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": latency_ms, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if cfg.dtype == synth.BF16 else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "layers": cfg.L, "hidden": cfg.H, "heads": cfg.nh, "ffn": cfg.F,
                   "seq_len": cfg.S, "batch": cfg.B, "vocab": cfg.V, "replicas": world,
                   "launch": "CUDA graph replay of one fluid_run", "l2": "flushed between timed steps (256 MiB fill outside the event pair)"},
        "peak_arena_mb": main_res["arena_mb"], "arena_naive_mb": main_res["arena_naive_mb"],
        "arena_live_bound_mb": main_res["arena_live_bound_mb"], "weights_mb": main_res["weights_mb"],
        "tokens_per_s": world * main_res["tokens"] / (latency_ms * 1e-3),
        "latency_eager_ms": main_res["latency_eager_ms"], "latency_min_ms": main_res["latency_min_ms"],
        "latency_median_ms": main_res["latency_median_ms"],
        "e2e": {"value": e2e_ms, "unit": "ms", "h2d_bytes_per_step": main_res["h2d_bytes"],
                "d2h_bytes_per_step": main_res["d2h_bytes"]},
        "gpu_launches": main_res["kernel_steps"] * args.steps * 3,
        "kernel_steps_per_inference": main_res["kernel_steps"],
        "clocks": main_res["clocks"], "roofline": roof, "kernels": kernels, "cpu_baseline": cpu, "parity": parity,
        "other_workloads": others,
    }
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
