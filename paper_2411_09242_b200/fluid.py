"""ctypes binding of the C-ABI in include/fluid.h: same names, argument marshalling only.

Every step of the hot path (planning, arena placement, kernels) runs inside libfluid.so; this
module converts Python values to C arguments and keeps device buffers alive. There is no CPU
fallback: if the library is missing, loading raises.

Besides the one-to-one wrappers (fluid_graph_create ... fluid_status) there is `Runner`, a
convenience that owns the torch-allocated device memory (arena, constants, inputs, outputs) for
one plan. torch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import numpy as np

from . import synth

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfluid.so")

FLUID_OK = 0
FLUID_EINVAL, FLUID_EUNSUPPORTED, FLUID_EALIGN, FLUID_ECUDA, FLUID_ENOMEM, FLUID_ETIMEOUT = -1, -2, -3, -4, -5, -6
ARENA_ALIGN, ARENA_HEADER, SLOT_ALIGN = 1024, 256, 256
KERNEL_NAMES = ["EMBED", "NORM", "GEMM_SIMT", "GEMM_TC", "SOFTMAX", "ROPE", "ELTWISE", "PERMUTE", "SELECT_LAST", "ATTN", "ATTN_DECODE", "GEMM_ROWS"]


class FluidError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"fluid error {code}: {msg}")
        self.code = code


class OpAttrs(C.Structure):
    _fields_ = [("contract", C.c_int32), ("causal", C.c_int32), ("gelu_tanh", C.c_int32),
                ("rope_interleaved", C.c_int32), ("perm", C.c_int32 * 8), ("scale", C.c_double),
                ("eps", C.c_double), ("rope_base", C.c_double)]


class LayoutCandidates(C.Structure):
    _fields_ = [("n_tensors", C.c_int32), ("n_cands", C.POINTER(C.c_int32)), ("perms", C.POINTER(C.c_int32))]


EVAL_FN = C.CFUNCTYPE(C.c_double, C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32))
EVAL_VARIANT_FN = C.CFUNCTYPE(C.c_double, C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.c_int32)
GV_SINGLE, GV_PAIR, GV_CLUSTER = 1, 2, 3


def gemm_variant_code(form, tile_n):
    return form | (tile_n << 4)


class PlanOptions(C.Structure):
    _fields_ = [("fusion", C.c_int32), ("arena_policy", C.c_int32), ("no_reuse", C.c_int32),
                ("force_canonical", C.c_int32), ("gemm_path", C.c_int32), ("narrow_stream", C.c_int32),
                ("unfused_attention", C.c_int32), ("split_k", C.c_int32),
                ("eval", EVAL_FN), ("eval_user", C.c_void_p), ("eval_variant", EVAL_VARIANT_FN),
                ("op_variant", C.POINTER(C.c_int32)), ("n_op_variant", C.c_int32), ("no_inplace", C.c_int32),
                ("redzone_bytes", C.c_int32), ("no_norm_split", C.c_int32)]


class StepInfo(C.Structure):
    _fields_ = [("kernel", C.c_int32), ("variant", C.c_int32), ("n_ops", C.c_int32), ("ops", C.c_int32 * 8),
                ("n_in", C.c_int32), ("n_out", C.c_int32), ("in_ids", C.c_int32 * 8), ("out_ids", C.c_int32 * 4),
                ("cost", C.c_double), ("flops", C.c_double), ("bytes", C.c_double)]


_lib = None

_SIGNATURES = {
    "fluid_graph_create": (C.c_int, [C.POINTER(C.c_void_p)]),
    "fluid_graph_destroy": (None, [C.c_void_p]),
    "fluid_graph_add_tensor": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int64), C.c_int, C.POINTER(C.c_int)]),
    "fluid_graph_add_op": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_int),
                                      C.POINTER(OpAttrs), C.POINTER(C.c_int)]),
    "fluid_plan": (C.c_int, [C.c_void_p, C.POINTER(LayoutCandidates), C.POINTER(PlanOptions), C.POINTER(C.c_void_p)]),
    "fluid_plan_destroy": (None, [C.c_void_p]),
    "fluid_plan_default_options": (None, [C.POINTER(PlanOptions)]),
    "fluid_plan_arena_bytes": (C.c_size_t, [C.c_void_p]),
    "fluid_plan_arena_naive_bytes": (C.c_size_t, [C.c_void_p]),
    "fluid_plan_arena_live_bound_bytes": (C.c_size_t, [C.c_void_p]),
    "fluid_plan_cost": (C.c_double, [C.c_void_p]),
    "fluid_plan_canonical_cost": (C.c_double, [C.c_void_p]),
    "fluid_plan_tensor_info": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int64),
                                          C.POINTER(C.c_int64), C.POINTER(C.c_int), C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "fluid_plan_num_records": (C.c_int, [C.c_void_p]),
    "fluid_plan_record_info": (C.c_int, [C.c_void_p, C.c_int] + [C.POINTER(C.c_int)] * 4 + [C.POINTER(C.c_int64)] * 2 +
                               [C.POINTER(C.c_int)] * 2),
    "fluid_plan_gemm_variants": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "fluid_plan_num_steps": (C.c_int, [C.c_void_p]),
    "fluid_plan_step_info": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(StepInfo)]),
    "fluid_plan_num_sequences": (C.c_int, [C.c_void_p]),
    "fluid_plan_sequence": (C.c_int, [C.c_void_p, C.c_int, C.POINTER(C.c_int), C.c_int, C.POINTER(C.c_int)]),
    "fluid_plan_bind_constant": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p]),
    "fluid_pack_constant": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]),
    "fluid_run": (C.c_int, [C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_void_p]),
    "fluid_run_profiled": (C.c_int, [C.c_void_p, C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_void_p,
                                      C.POINTER(C.c_float)]),
    "fluid_status": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(C.c_int)]),
    "fluid_gemm_bf16_static_scratch": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                                  C.c_void_p]),
    "fluid_static_scratch_status": (C.c_int, [C.c_void_p, C.POINTER(C.c_int)]),
    "fluid_last_error": (C.c_char_p, []),
    "fluid_launch_count": (C.c_int64, []),
}


def lib():
    """The loaded CUDA library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2411_09242_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def _check(rc):
    if rc != FLUID_OK:
        raise FluidError(rc, lib().fluid_last_error().decode())
    return rc


# ---- one-to-one wrappers ---------------------------------------------------------------------
def fluid_graph_create():
    h = C.c_void_p()
    _check(lib().fluid_graph_create(C.byref(h)))
    return h


def fluid_graph_destroy(g):
    lib().fluid_graph_destroy(g)


def fluid_graph_add_tensor(g, dtype, dims, kind):
    arr = (C.c_int64 * len(dims))(*dims)
    tid = C.c_int()
    _check(lib().fluid_graph_add_tensor(g, dtype, len(dims), arr, kind, C.byref(tid)))
    return tid.value


def make_attrs(attrs: dict) -> OpAttrs:
    a = OpAttrs()
    for k, v in attrs.items():
        if k == "perm":
            for i, p in enumerate(v):
                a.perm[i] = p
        else:
            setattr(a, k, v)
    return a


def fluid_graph_add_op(g, kind, ins, outs, attrs=None):
    a = make_attrs(attrs or {})
    i_arr = (C.c_int * len(ins))(*ins)
    o_arr = (C.c_int * len(outs))(*outs)
    oid = C.c_int()
    _check(lib().fluid_graph_add_op(g, kind, len(ins), i_arr, len(outs), o_arr, C.byref(a), C.byref(oid)))
    return oid.value


def fluid_plan_default_options() -> PlanOptions:
    o = PlanOptions()
    lib().fluid_plan_default_options(C.byref(o))
    return o


def fluid_plan(g, candidates=None, options: PlanOptions | None = None):
    """candidates: {tensor id: [perm, ...]} or None; returns the plan handle."""
    cand_struct = None
    keep = []
    if candidates is not None:
        n = max(candidates) + 1 if candidates else 0
        counts = (C.c_int32 * n)()
        flat = []
        for t in range(n):
            opts = candidates.get(t, [])
            counts[t] = len(opts)
            for perm in opts:
                flat.extend(int(v) for v in perm)
        perms = (C.c_int32 * max(1, len(flat)))(*flat)
        cand_struct = LayoutCandidates(n, counts, perms)
        keep = [counts, perms]
    h = C.c_void_p()
    _check(lib().fluid_plan(g, C.byref(cand_struct) if cand_struct is not None else None,
                            C.byref(options) if options is not None else None, C.byref(h)))
    del keep
    return h


def fluid_plan_destroy(p):
    lib().fluid_plan_destroy(p)


def fluid_plan_arena_bytes(p):
    return lib().fluid_plan_arena_bytes(p)


def fluid_plan_arena_naive_bytes(p):
    return lib().fluid_plan_arena_naive_bytes(p)


def fluid_plan_arena_live_bound_bytes(p):
    return lib().fluid_plan_arena_live_bound_bytes(p)


def fluid_plan_cost(p):
    return lib().fluid_plan_cost(p)


def fluid_plan_canonical_cost(p):
    return lib().fluid_plan_canonical_cost(p)


@dataclass
class TensorInfo:
    layout_index: int
    perm: tuple
    offset: int
    bytes: int
    first_step: int
    last_step: int
    alias_of: int


def fluid_plan_tensor_info(p, tid, rank) -> TensorInfo:
    li, off, by, fs, ls, al = C.c_int(), C.c_int64(), C.c_int64(), C.c_int(), C.c_int(), C.c_int()
    perm = (C.c_int * 8)()
    _check(lib().fluid_plan_tensor_info(p, tid, C.byref(li), perm, C.byref(off), C.byref(by), C.byref(fs),
                                        C.byref(ls), C.byref(al)))
    return TensorInfo(li.value, tuple(perm[:rank]), off.value, by.value, fs.value, ls.value, al.value)


def fluid_plan_num_records(p):
    return lib().fluid_plan_num_records(p)


def fluid_plan_record_info(p, index) -> dict:
    rid, tid, tw, dt, fs, ls = (C.c_int() for _ in range(6))
    off, by = C.c_int64(), C.c_int64()
    _check(lib().fluid_plan_record_info(p, index, C.byref(rid), C.byref(tid), C.byref(tw), C.byref(dt),
                                        C.byref(off), C.byref(by), C.byref(fs), C.byref(ls)))
    return {"id": rid.value, "tensor": tid.value, "twin": tw.value, "dtype": dt.value, "offset": off.value,
            "bytes": by.value, "first": fs.value, "last": ls.value}


def fluid_plan_num_steps(p):
    return lib().fluid_plan_num_steps(p)


def fluid_plan_step_info(p, step) -> dict:
    s = StepInfo()
    _check(lib().fluid_plan_step_info(p, step, C.byref(s)))
    return {"kernel": s.kernel, "kernel_name": KERNEL_NAMES[s.kernel], "variant": s.variant,
            "ops": list(s.ops[: s.n_ops]), "ins": list(s.in_ids[: s.n_in]), "outs": list(s.out_ids[: s.n_out]),
            "cost": s.cost, "flops": s.flops, "bytes": s.bytes}


def fluid_plan_gemm_variants(p, op_id):
    """(variant codes the GEMM step anchored at graph op `op_id` can run with, the one the plan runs)."""
    n, chosen = C.c_int(), C.c_int()
    _check(lib().fluid_plan_gemm_variants(p, op_id, None, 0, C.byref(n), C.byref(chosen)))
    buf = (C.c_int * max(1, n.value))()
    _check(lib().fluid_plan_gemm_variants(p, op_id, buf, n.value, C.byref(n), C.byref(chosen)))
    return list(buf[: n.value]), chosen.value


def fluid_plan_num_sequences(p):
    return lib().fluid_plan_num_sequences(p)


def fluid_plan_sequence(p, index):
    n = C.c_int()
    _check(lib().fluid_plan_sequence(p, index, None, 0, C.byref(n)))
    buf = (C.c_int * max(1, n.value))()
    _check(lib().fluid_plan_sequence(p, index, buf, n.value, C.byref(n)))
    return list(buf[: n.value])


def fluid_plan_bind_constant(p, tid, dev_ptr):
    _check(lib().fluid_plan_bind_constant(p, tid, C.c_void_p(dev_ptr)))


def fluid_pack_constant(p, tid, dev_src, dev_dst, stream=0):
    _check(lib().fluid_pack_constant(p, tid, C.c_void_p(dev_src), C.c_void_p(dev_dst), C.c_void_p(stream)))


def _ptr_array(ptrs):
    return (C.c_void_p * max(1, len(ptrs)))(*ptrs)


def fluid_run(p, arena_ptr, inputs, outputs, stream=0):
    _check(lib().fluid_run(p, C.c_void_p(arena_ptr), _ptr_array(inputs), _ptr_array(outputs), C.c_void_p(stream)))


def fluid_run_profiled(p, arena_ptr, inputs, outputs, stream=0):
    n = fluid_plan_num_steps(p)
    ms = (C.c_float * max(1, n))()
    _check(lib().fluid_run_profiled(p, C.c_void_p(arena_ptr), _ptr_array(inputs), _ptr_array(outputs),
                                    C.c_void_p(stream), ms))
    return list(ms[:n])


def fluid_status(p, arena_ptr, stream=0):
    st = C.c_int()
    rc = lib().fluid_status(p, C.c_void_p(arena_ptr), C.c_void_p(stream), C.byref(st))
    if rc not in (FLUID_OK, FLUID_ETIMEOUT):
        _check(rc)
    return st.value


def fluid_gemm_bf16_static_scratch(dev_a, dev_b, dev_bias, dev_c, m, n, k, stream=0):
    """C[m,n] = A[m,k] . B[n,k]^T (+ bias) on device pointers, with the split-K scratch in the library's
    own fixed device array: for callers that have no arena and may not allocate one."""
    _check(lib().fluid_gemm_bf16_static_scratch(C.c_void_p(dev_a), C.c_void_p(dev_b), C.c_void_p(dev_bias or None),
                                                C.c_void_p(dev_c), m, n, k, C.c_void_p(stream)))


def fluid_static_scratch_status(stream=0):
    """Status word of the last static-scratch GEMM on the current device (0 = every wait completed); synchronises."""
    st = C.c_int()
    rc = lib().fluid_static_scratch_status(C.c_void_p(stream), C.byref(st))
    if rc not in (FLUID_OK, FLUID_ETIMEOUT):
        _check(rc)
    return st.value


def fluid_launch_count():
    return lib().fluid_launch_count()


# ---- helpers built on the wrappers --------------------------------------------------------------
def graph_from_desc(desc: synth.GraphDesc):
    g = fluid_graph_create()
    for t in desc.tensors:
        fluid_graph_add_tensor(g, t["dtype"], t["dims"], t["kind"])
    for op in desc.ops:
        fluid_graph_add_op(g, op["kind"], op["ins"], op["outs"], op["attrs"])
    return g


def make_options(**kw) -> PlanOptions:
    """Plan options from keywords. op_variant: {graph op id: variant code} (marshalled to the C array)."""
    o = fluid_plan_default_options()
    ev = kw.pop("eval", None)
    evv = kw.pop("eval_variant", None)
    opv = kw.pop("op_variant", None)
    for k, v in kw.items():
        setattr(o, k, v)
    if ev is not None:
        o.eval = ev
    if evv is not None:
        o.eval_variant = evv
    if opv:
        n = max(opv) + 1
        arr = (C.c_int32 * n)()
        for k, v in opv.items():
            arr[k] = v
        o.op_variant, o.n_op_variant = arr, n
        o._keep = arr        # alive until fluid_plan has copied it
    return o


class Plan:
    """A graph handle plus its plan handle, destroyed together."""

    def __init__(self, desc: synth.GraphDesc, candidates=None, **options):
        self.desc = desc
        self._eval_keepalive = (options.get("eval"), options.get("eval_variant"))
        self.graph = graph_from_desc(desc)
        try:
            self.handle = fluid_plan(self.graph, candidates, make_options(**options))
        except Exception:
            fluid_graph_destroy(self.graph)
            raise

    def close(self):
        if getattr(self, "handle", None):
            fluid_plan_destroy(self.handle)
            self.handle = None
        if getattr(self, "graph", None):
            fluid_graph_destroy(self.graph)
            self.graph = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # introspection
    @property
    def arena_bytes(self):
        return fluid_plan_arena_bytes(self.handle)

    @property
    def naive_bytes(self):
        return fluid_plan_arena_naive_bytes(self.handle)

    @property
    def live_bound_bytes(self):
        return fluid_plan_arena_live_bound_bytes(self.handle)

    @property
    def cost(self):
        return fluid_plan_cost(self.handle)

    @property
    def canonical_cost(self):
        return fluid_plan_canonical_cost(self.handle)

    def tensor_info(self, tid) -> TensorInfo:
        return fluid_plan_tensor_info(self.handle, tid, len(self.desc.tensors[tid]["dims"]))

    def records(self):
        return [fluid_plan_record_info(self.handle, i) for i in range(fluid_plan_num_records(self.handle))]

    def steps(self):
        return [fluid_plan_step_info(self.handle, i) for i in range(fluid_plan_num_steps(self.handle))]

    def sequences(self):
        return [fluid_plan_sequence(self.handle, i) for i in range(fluid_plan_num_sequences(self.handle))]

    def gemm_variants(self, op_id):
        return fluid_plan_gemm_variants(self.handle, op_id)


_TORCH_DTYPE = None


def _torch():
    import torch
    global _TORCH_DTYPE
    if _TORCH_DTYPE is None:
        _TORCH_DTYPE = {synth.F32: torch.float32, synth.BF16: torch.bfloat16, synth.I32: torch.int32}
    return torch


def to_device(arr: np.ndarray, dtype: int, device="cuda"):
    """Host array -> device tensor of the graph dtype (bf16 values must already be representable)."""
    torch = _torch()
    if dtype == synth.I32:
        return torch.from_numpy(np.ascontiguousarray(arr, dtype=np.int32)).to(device)
    t = torch.from_numpy(np.ascontiguousarray(arr, dtype=np.float32))
    if dtype == synth.BF16:
        t = t.to(torch.bfloat16)   # exact: the values are bf16-representable
    return t.to(device)


class Runner:
    """Device memory for one plan: the arena (one allocation), packed constants, I/O buffers."""

    def __init__(self, plan: Plan, consts: dict, device="cuda", poison=False):
        torch = _torch()
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (there is no CPU fallback)")
        self.plan, self.device = plan, device
        desc = plan.desc
        nbytes = plan.arena_bytes
        raw = torch.empty(nbytes + ARENA_ALIGN, dtype=torch.uint8, device=device)
        shift = (-raw.data_ptr()) % ARENA_ALIGN
        self._arena_raw = raw
        self.arena = raw[shift: shift + nbytes]
        if poison:
            self.arena.fill_(0xFF)     # bf16/fp32 NaN patterns: reads of stale memory show up
        self.consts = {}
        for tid, arr in consts.items():
            t = desc.tensors[tid]
            src = to_device(arr, t["dtype"], device)
            info = plan.tensor_info(tid)
            if info.layout_index != 0:
                dst = torch.empty_like(src)
                fluid_pack_constant(plan.handle, tid, src.data_ptr(), dst.data_ptr(),
                                    torch.cuda.current_stream().cuda_stream)
                torch.cuda.current_stream().synchronize()
                src = dst
            self.consts[tid] = src
            fluid_plan_bind_constant(plan.handle, tid, src.data_ptr())
        self.inputs = [torch.empty(desc.tensors[t]["dims"], dtype=_TORCH_DTYPE[desc.tensors[t]["dtype"]], device=device)
                       for t in desc.inputs]
        self.outputs = [torch.empty(desc.tensors[t]["dims"], dtype=_TORCH_DTYPE[desc.tensors[t]["dtype"]], device=device)
                        for t in desc.outputs]

    def set_inputs(self, arrays):
        for buf, tid, arr in zip(self.inputs, self.plan.desc.inputs, arrays):
            buf.copy_(to_device(arr, self.plan.desc.tensors[tid]["dtype"], self.device))

    def run(self, stream=None):
        torch = _torch()
        s = (stream or torch.cuda.current_stream()).cuda_stream
        fluid_run(self.plan.handle, self.arena.data_ptr(), [b.data_ptr() for b in self.inputs],
                  [b.data_ptr() for b in self.outputs], s)

    def run_profiled(self):
        torch = _torch()
        s = torch.cuda.current_stream().cuda_stream
        return fluid_run_profiled(self.plan.handle, self.arena.data_ptr(), [b.data_ptr() for b in self.inputs],
                                  [b.data_ptr() for b in self.outputs], s)

    def status(self):
        torch = _torch()
        return fluid_status(self.plan.handle, self.arena.data_ptr(), torch.cuda.current_stream().cuda_stream)

    def redzone_violations(self, zone_bytes):
        """For a plan made with no_reuse = 1 and redzone_bytes = zone_bytes, run from a poisoned arena (every byte
        0xFF): the ids of the arena records whose trailing zone no longer holds the pattern (some kernel stored
        past the end of that slice). Empty = clean."""
        torch = _torch()
        torch.cuda.synchronize()
        zone = (zone_bytes + SLOT_ALIGN - 1) // SLOT_ALIGN * SLOT_ALIGN
        bad = []
        for r in self.plan.records():
            if r["tensor"] < 0:
                continue          # per-step scratch has no zone
            tail = self.arena[r["offset"] + r["bytes"] - zone: r["offset"] + r["bytes"]]
            if not bool((tail == 0xFF).all()):
                bad.append(r["id"])
        return bad

    def outputs_host(self):
        torch = _torch()
        torch.cuda.synchronize()
        return [o.float().cpu().numpy().astype(np.float64) for o in self.outputs]

    def read_tensor(self, tid, index=None):
        """Copy one arena-resident (or output) tensor back in canonical order, for per-op checks.
        index: optional tuple of slices / index lists applied on the device before the copy."""
        torch = _torch()
        torch.cuda.synchronize()
        desc = self.plan.desc
        t = desc.tensors[tid]
        info = self.plan.tensor_info(tid)
        if t["kind"] == synth.OUTPUT:
            view = self.outputs[desc.outputs.index(tid)]
        else:
            if info.offset < 0:
                raise ValueError(f"tensor {tid} is not arena-resident")
            rec = next(r for r in self.plan.records() if r["tensor"] == info.alias_of and not r["twin"])
            n = int(np.prod(t["dims"]))
            es = synth.DTYPE_BYTES[rec["dtype"]]
            raw = self.arena[info.offset: info.offset + n * es]
            pd = [t["dims"][p] for p in info.perm]
            inv = [int(i) for i in np.argsort(info.perm)]
            view = raw.view(_TORCH_DTYPE[rec["dtype"]]).view(pd).permute(inv)
        if index is not None:
            view = view[index]
        return view.float().cpu().numpy().astype(np.float64)
