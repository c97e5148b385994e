"""Seeded synthetic inputs: operator graphs, layout-candidate lists, weights and token ids.

Everything here is *input* to the method: the transformer inference graph whose execution
blueprint a layout-and-memory planner rewrites (paper, Sec. "Design": a flow of operator nodes
joined by tensor edges, each edge with a few layout options), plus the numbers fed through it.
This module holds none of the method's arithmetic: no operator maths, no planning, no kernels.
Both the CPU oracle's tests and the CUDA path's tests/bench call it, so that both sides see the
very same arrays and the very same graph description (plain dicts, lists and numpy arrays).

Workload recipe (the paper evaluates language models such as BERT and GPT-NeoX, Sec.
"Evaluation"; their files are not available, so shape-alike random models stand in):
  * matrices, embedding tables and linear biases ~ N(0, 0.02); norm gains 1 + N(0, 0.02),
    norm biases ~ N(0, 0.02); token ids uniform in [0, vocab);
  * bf16 workloads round every generated value to bf16 (round-to-nearest-even) on the host
    before either side sees it;
  * random numbers are counter-based (Philox keyed by (seed, tensor index)), so a tensor's
    values do not depend on generation order.
"""
from __future__ import annotations

import itertools
import math
from dataclasses import dataclass, field

import numpy as np

# ---- enumerations shared by the graph description (mirrored by include/fluid.h) -------------
F32, BF16, I32 = 0, 1, 2
INPUT, OUTPUT, CONST, ACT, STATE = 0, 1, 2, 3, 4
(EMBED, LINEAR, ADD, MUL, GELU, SILU, SOFTMAX, LAYERNORM, RMSNORM, ROPE, TRANSPOSE, BMM_QK,
 BMM_PV, SELECT_LAST_TOKEN, CACHED_ATTENTION) = range(15)
OP_NAMES = ["EMBED", "LINEAR", "ADD", "MUL", "GELU", "SILU", "SOFTMAX", "LAYERNORM", "RMSNORM",
            "ROPE", "TRANSPOSE", "BMM_QK", "BMM_PV", "SELECT_LAST_TOKEN", "CACHED_ATTENTION"]
DTYPE_BYTES = {F32: 4, BF16: 2, I32: 4}

WEIGHT_SEED = 2411
TOKEN_SEED = 9242


# ---- counter-based random numbers -----------------------------------------------------------
def _gen(seed: int, index: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[np.uint64(seed), np.uint64(index)]))


def normal(seed: int, index: int, shape, std: float = 0.02, mean: float = 0.0) -> np.ndarray:
    g = _gen(seed, index)
    a = g.standard_normal(size=tuple(shape), dtype=np.float32)
    a *= np.float32(std)
    if mean != 0.0:
        a += np.float32(mean)
    return a


def uniform(seed: int, index: int, shape, lo: float = -1.0, hi: float = 1.0) -> np.ndarray:
    g = _gen(seed, index)
    a = g.random(size=tuple(shape), dtype=np.float32)
    a *= np.float32(hi - lo)
    a += np.float32(lo)
    return a


def token_ids(seed: int, index: int, shape, vocab: int) -> np.ndarray:
    g = _gen(seed, index)
    return g.integers(0, vocab, size=tuple(shape), dtype=np.int32)


# ---- bf16 storage helpers (input preparation only) ------------------------------------------
def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 array -> uint16 bf16 bit patterns, round-to-nearest-even."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (u + (((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_bf16(a: np.ndarray) -> np.ndarray:
    """float32 array -> float32 array holding bf16-representable values."""
    return bf16_bits_to_f32(bf16_bits(a)).reshape(a.shape)


# ---- graph description ----------------------------------------------------------------------
@dataclass
class GraphDesc:
    """A plain-data operator graph: tensors (edges) and ops (nodes) in declaration order."""
    tensors: list = field(default_factory=list)   # dicts: name, dtype, dims, kind
    ops: list = field(default_factory=list)       # dicts: kind, ins, outs, attrs
    inputs: list = field(default_factory=list)    # tensor ids, declaration order (INPUT and STATE kinds)
    outputs: list = field(default_factory=list)

    def tensor(self, name, dtype, dims, kind=ACT) -> int:
        tid = len(self.tensors)
        self.tensors.append({"name": name, "dtype": dtype, "dims": [int(d) for d in dims],
                             "kind": kind})
        if kind in (INPUT, STATE):
            self.inputs.append(tid)
        elif kind == OUTPUT:
            self.outputs.append(tid)
        return tid

    def op(self, kind, ins, outs, **attrs) -> int:
        oid = len(self.ops)
        self.ops.append({"kind": kind, "ins": [int(i) for i in ins],
                         "outs": [int(o) for o in outs], "attrs": dict(attrs)})
        return oid

    def dims(self, tid):
        return self.tensors[tid]["dims"]


def identity_perm(rank):
    return tuple(range(rank))


def default_candidates(g: GraphDesc) -> dict:
    """Layout options per tensor id: permutations of the logical dims, slowest to fastest.

    The first entry is always the canonical row-major order. Graph inputs and outputs stay
    canonical (they are the caller's buffers). Rank-4 activations (head tensors) may take any
    order that keeps the batch dim outermost; weight matrices may be stored with either their
    contraction dims or their output dims fastest ("row-" or "column-major"); rank-2 activations
    (plain matrices) may be row- or column-major. Everything else is canonical only.
    """
    cands = {}
    w_roles = {}
    for op in g.ops:
        if op["kind"] == LINEAR:
            w_roles[op["ins"][1]] = op["attrs"].get("contract", 1)
    for tid, t in enumerate(g.tensors):
        rank = len(t["dims"])
        ident = identity_perm(rank)
        opts = [ident]
        if t["kind"] == ACT:
            if rank == 4:
                opts += [(0,) + p for p in itertools.permutations((1, 2, 3)) if (0,) + p != ident]
            elif rank == 2:
                opts.append((1, 0))
        elif t["kind"] == CONST and tid in w_roles and rank >= 2:
            c = w_roles[tid]
            swapped = tuple(range(c, rank)) + tuple(range(c))
            if swapped != ident:
                opts.append(swapped)
        cands[tid] = opts
    return cands


def canonical_candidates(g: GraphDesc) -> dict:
    return {tid: [identity_perm(len(t["dims"]))] for tid, t in enumerate(g.tensors)}


# ---- model configurations ---------------------------------------------------------------------
@dataclass(frozen=True)
class ModelConfig:
    name: str
    family: str            # "encoder" (post-LN), "gpt" (pre-LN causal), "llama"
    dtype: int
    L: int
    H: int
    nh: int
    F: int
    S: int
    B: int
    V: int

    @property
    def D(self):
        return self.H // self.nh


CONFIGS = {
    "tiny": ModelConfig("tiny", "encoder", F32, 2, 128, 2, 512, 32, 1, 1000),
    "bert_base": ModelConfig("bert_base", "encoder", BF16, 12, 768, 12, 3072, 128, 1, 30522),
    "gpt2_small": ModelConfig("gpt2_small", "gpt", BF16, 12, 768, 12, 3072, 1024, 4, 50257),
    "llama": ModelConfig("llama", "llama", BF16, 4, 4096, 32, 11008, 2048, 1, 32000),
}


def scaled(cfg: ModelConfig, **kw) -> ModelConfig:
    """A smaller or otherwise altered copy of a configuration (tests use reduced sizes)."""
    d = dict(name=cfg.name, family=cfg.family, dtype=cfg.dtype, L=cfg.L, H=cfg.H, nh=cfg.nh,
             F=cfg.F, S=cfg.S, B=cfg.B, V=cfg.V)
    d.update(kw)
    return ModelConfig(**d)


@dataclass
class Model:
    cfg: ModelConfig
    graph: GraphDesc
    consts: dict           # tensor id -> float32 ndarray (bf16-representable for BF16 models)
    ids: np.ndarray        # int32 [B, S]


class _Builder:
    def __init__(self, cfg: ModelConfig, weight_seed: int, materialize: bool):
        self.cfg = cfg
        self.g = GraphDesc()
        self.consts = {}
        self.seed = weight_seed
        self.materialize = materialize

    def const(self, name, dims, std=0.02, mean=0.0):
        tid = self.g.tensor(name, self.cfg.dtype, dims, CONST)
        if self.materialize:
            a = normal(self.seed, tid, dims, std, mean)
            if self.cfg.dtype == BF16:
                a = round_bf16(a)
            self.consts[tid] = a
        return tid

    def act(self, name, dims, kind=ACT):
        return self.g.tensor(name, self.cfg.dtype, dims, kind)


def _attention(b: _Builder, x, pfx, causal, bias, rope, emit_kv=False):
    cfg, g = b.cfg, b.g
    B, S, H, nh, D = cfg.B, cfg.S, cfg.H, cfg.nh, cfg.D
    heads = {}
    for nm in ("q", "k", "v"):
        w = b.const(f"{pfx}.W{nm}", [H, nh, D])
        ins = [x, w]
        if bias:
            ins.append(b.const(f"{pfx}.b{nm}", [nh, D]))
        # emit_kv: the keys (after the rotary embedding, if any) and the values are graph outputs, in the layout of a
        # key/value cache, so that decoding steps can continue from them
        kv_out = emit_kv and nm in ("k", "v")
        t = b.act(f"{pfx}.{nm}", [B, S, nh, D], OUTPUT if kv_out and not (rope and nm == "k") else ACT)
        g.op(LINEAR, ins, [t], contract=1)
        if rope and nm in ("q", "k"):
            r = b.act(f"{pfx}.{nm}_rope", [B, S, nh, D], OUTPUT if kv_out else ACT)
            g.op(ROPE, [t], [r], rope_base=10000.0, rope_interleaved=0)
            t = r
        heads[nm] = t
    qh = b.act(f"{pfx}.qh", [B, nh, S, D])
    g.op(TRANSPOSE, [heads["q"]], [qh], perm=[0, 2, 1, 3])
    kT = b.act(f"{pfx}.kT", [B, nh, D, S])
    g.op(TRANSPOSE, [heads["k"]], [kT], perm=[0, 2, 3, 1])
    vh = b.act(f"{pfx}.vh", [B, nh, S, D])
    g.op(TRANSPOSE, [heads["v"]], [vh], perm=[0, 2, 1, 3])
    sc = b.act(f"{pfx}.scores", [B, nh, S, S])
    g.op(BMM_QK, [qh, kT], [sc], scale=1.0 / math.sqrt(D))
    p = b.act(f"{pfx}.probs", [B, nh, S, S])
    g.op(SOFTMAX, [sc], [p], causal=int(causal), scale=1.0)
    ch = b.act(f"{pfx}.ctx_h", [B, nh, S, D])
    g.op(BMM_PV, [p, vh], [ch])
    c = b.act(f"{pfx}.ctx", [B, S, nh, D])
    g.op(TRANSPOSE, [ch], [c], perm=[0, 2, 1, 3])
    wo = b.const(f"{pfx}.Wo", [nh, D, H])
    ins = [c, wo]
    if bias:
        ins.append(b.const(f"{pfx}.bo", [H]))
    o = b.act(f"{pfx}.attn_out", [B, S, H])
    g.op(LINEAR, ins, [o], contract=2)
    return o


def _norm(b: _Builder, x, name, rms, out_kind=ACT):
    cfg, g = b.cfg, b.g
    gamma = b.const(f"{name}.gamma", [cfg.H], 0.02, 1.0)
    y = b.act(f"{name}.out", [cfg.B, cfg.S, cfg.H], out_kind)
    if rms:
        g.op(RMSNORM, [x, gamma], [y], eps=1e-5)
    else:
        beta = b.const(f"{name}.beta", [cfg.H])
        g.op(LAYERNORM, [x, gamma, beta], [y], eps=1e-5)
    return y


def _mlp_gelu(b: _Builder, x, pfx):
    cfg, g = b.cfg, b.g
    B, S, H, F = cfg.B, cfg.S, cfg.H, cfg.F
    w1 = b.const(f"{pfx}.W1", [H, F]); b1 = b.const(f"{pfx}.b1", [F])
    f = b.act(f"{pfx}.ffn1", [B, S, F]); g.op(LINEAR, [x, w1, b1], [f], contract=1)
    a = b.act(f"{pfx}.gelu", [B, S, F]); g.op(GELU, [f], [a], gelu_tanh=0)
    w2 = b.const(f"{pfx}.W2", [F, H]); b2 = b.const(f"{pfx}.b2", [H])
    o = b.act(f"{pfx}.ffn2", [B, S, H]); g.op(LINEAR, [a, w2, b2], [o], contract=1)
    return o


def _mlp_swiglu(b: _Builder, x, pfx):
    cfg, g = b.cfg, b.g
    B, S, H, F = cfg.B, cfg.S, cfg.H, cfg.F
    wg = b.const(f"{pfx}.Wg", [H, F]); wu = b.const(f"{pfx}.Wu", [H, F])
    gt = b.act(f"{pfx}.gate", [B, S, F]); g.op(LINEAR, [x, wg], [gt], contract=1)
    up = b.act(f"{pfx}.up", [B, S, F]); g.op(LINEAR, [x, wu], [up], contract=1)
    s = b.act(f"{pfx}.silu", [B, S, F]); g.op(SILU, [gt], [s])
    m = b.act(f"{pfx}.swiglu", [B, S, F]); g.op(MUL, [s, up], [m])
    wd = b.const(f"{pfx}.Wd", [F, H])
    o = b.act(f"{pfx}.down", [B, S, H]); g.op(LINEAR, [m, wd], [o], contract=1)
    return o


def build_model(cfg: ModelConfig, weight_seed: int = WEIGHT_SEED, token_seed: int = TOKEN_SEED,
                materialize: bool = True, emit_kv: bool = False) -> Model:
    """Graph + seeded weights + token ids for one configuration.

    Wiring (generic public architecture families):
      encoder: x0 = LN(embed); per layer x = LN(x + attn(x)); x = LN(x + ffn(x)); output x.
      gpt    : x0 = embed; per layer x += attn(LN(x)); x += ffn(LN(x)); h = LN(x);
               outputs h and last-token logits against the tied token table.
      llama  : as gpt with RMSNorm, rotary q/k, bias-free linears, SwiGLU, separate LM head.
    emit_kv (causal families): every layer's keys and values [B,S,nh,D] are extra graph outputs (declared before the
    hidden state and the logits), the prompt's contribution to a key/value cache.
    Attention is written the way exported graphs spell it: per-head tensors are produced by
    explicit TRANSPOSE ops, which the planner may turn into zero-copy views.
    """
    b = _Builder(cfg, weight_seed, materialize)
    g = b.g
    B, S, H, V = cfg.B, cfg.S, cfg.H, cfg.V
    ids = g.tensor("ids", I32, [B, S], INPUT)
    tok = b.const("tok_table", [V, H])
    x = b.act("embed", [B, S, H])
    if cfg.family == "llama":
        g.op(EMBED, [ids, tok], [x])
    else:
        pos = b.const("pos_table", [S, H])
        g.op(EMBED, [ids, tok, pos], [x])

    if cfg.family == "encoder":
        x = _norm(b, x, "emb_ln", rms=False)
        for l in range(cfg.L):
            pfx = f"l{l}"
            o = _attention(b, x, pfx, causal=False, bias=True, rope=False)
            a = b.act(f"{pfx}.res1", [B, S, H]); g.op(ADD, [x, o], [a])
            x = _norm(b, a, f"{pfx}.ln1", rms=False)
            o = _mlp_gelu(b, x, pfx)
            a = b.act(f"{pfx}.res2", [B, S, H]); g.op(ADD, [x, o], [a])
            last = l == cfg.L - 1
            x = _norm(b, a, f"{pfx}.ln2", rms=False, out_kind=OUTPUT if last else ACT)
    else:
        rms = cfg.family == "llama"
        for l in range(cfg.L):
            pfx = f"l{l}"
            n = _norm(b, x, f"{pfx}.ln1", rms)
            o = _attention(b, n, pfx, causal=True, bias=not rms, rope=rms, emit_kv=emit_kv)
            a = b.act(f"{pfx}.res1", [B, S, H]); g.op(ADD, [x, o], [a])
            n = _norm(b, a, f"{pfx}.ln2", rms)
            o = _mlp_swiglu(b, n, pfx) if rms else _mlp_gelu(b, n, pfx)
            x = b.act(f"{pfx}.res2", [B, S, H]); g.op(ADD, [a, o], [x])
        h = _norm(b, x, "final_norm", rms, out_kind=OUTPUT)
        hl = b.act("last_hidden", [B, H])
        g.op(SELECT_LAST_TOKEN, [h], [hl])
        if cfg.family == "llama":
            wlm = b.const("W_lm", [H, V])
        else:
            wlm = b.act("tok_table_T", [H, V])
            g.op(TRANSPOSE, [tok], [wlm], perm=[1, 0])
        logits = b.act("logits", [B, V], OUTPUT)
        g.op(LINEAR, [hl, wlm], [logits], contract=1)

    tok_ids = token_ids(token_seed, 0, [B, S], V)
    return Model(cfg, g, b.consts, tok_ids)


# ---- single-token decoding against a key/value cache ---------------------------------------------
@dataclass
class DecodeModel:
    cfg: ModelConfig       # S == 1: one new token per sequence and step
    t_max: int             # rows of every cache
    graph: GraphDesc
    consts: dict
    ids: int               # tensor ids of the step's inputs
    pos: int
    caches: list           # [(k_cache tensor id, v_cache tensor id)] per layer


def build_decode_model(cfg: ModelConfig, t_max: int, like: Model = None, weight_seed: int = WEIGHT_SEED,
                       materialize: bool = True, per_sequence_pos: bool = False) -> DecodeModel:
    """The graph of ONE decoding step of a causal family ("llama": RMSNorm, rotary q/k, SwiGLU; "gpt": LayerNorm,
    learned positions, biases, GELU, tied head): B sequences, one new token each, the keys and values of the
    earlier tokens in per-layer caches [B, t_max, nh, D] that the caller owns and the step extends (STATE
    tensors). `pos` (int32 [1], or [B] with per_sequence_pos; on the device at run time) is the number of tokens
    already cached, for all sequences or per sequence. Outputs: the final hidden state [B,1,H] and the logits
    [B,1,V].

    like: a whole-sequence model of the same family and widths; its weights are taken over by name, so that a run
    of decoding steps can be compared with that model on the same tokens.
    """
    assert cfg.family in ("llama", "gpt"), "decoding graphs are built for the causal families"
    rms = cfg.family == "llama"
    pos_rows = like.cfg.S if like is not None else t_max    # rows of the learned position table (gpt)
    cfg = scaled(cfg, S=1)
    b = _Builder(cfg, weight_seed, materialize and like is None)
    g = b.g
    B, H, V, nh, D = cfg.B, cfg.H, cfg.V, cfg.nh, cfg.D
    ids = g.tensor("ids", I32, [B, 1], INPUT)
    pos = g.tensor("pos", I32, [B if per_sequence_pos else 1], INPUT)
    tok = b.const("tok_table", [V, H])
    x = b.act("embed", [B, 1, H])
    if rms:
        g.op(EMBED, [ids, tok], [x])
    else:
        ptab = b.const("pos_table", [pos_rows, H])
        g.op(EMBED, [ids, tok, ptab, pos], [x])
    caches = []
    for l in range(cfg.L):
        pfx = f"l{l}"
        n = _norm(b, x, f"{pfx}.ln1", rms)
        heads = {}
        for nm in ("q", "k", "v"):
            w = b.const(f"{pfx}.W{nm}", [H, nh, D])
            ins = [n, w]
            if not rms:
                ins.append(b.const(f"{pfx}.b{nm}", [nh, D]))
            t = b.act(f"{pfx}.{nm}", [B, 1, nh, D])
            g.op(LINEAR, ins, [t], contract=1)
            if rms and nm != "v":
                r = b.act(f"{pfx}.{nm}_rope", [B, 1, nh, D])
                g.op(ROPE, [t, pos], [r], rope_base=10000.0, rope_interleaved=0)
                t = r
            heads[nm] = t
        kc = g.tensor(f"{pfx}.k_cache", cfg.dtype, [B, t_max, nh, D], STATE)
        vc = g.tensor(f"{pfx}.v_cache", cfg.dtype, [B, t_max, nh, D], STATE)
        caches.append((kc, vc))
        c = b.act(f"{pfx}.ctx", [B, 1, nh, D])
        g.op(CACHED_ATTENTION, [heads["q"], heads["k"], heads["v"], kc, vc, pos], [c], scale=1.0 / math.sqrt(D))
        wo = b.const(f"{pfx}.Wo", [nh, D, H])
        ins = [c, wo]
        if not rms:
            ins.append(b.const(f"{pfx}.bo", [H]))
        o = b.act(f"{pfx}.attn_out", [B, 1, H])
        g.op(LINEAR, ins, [o], contract=2)
        a = b.act(f"{pfx}.res1", [B, 1, H]); g.op(ADD, [x, o], [a])
        n = _norm(b, a, f"{pfx}.ln2", rms)
        o = _mlp_swiglu(b, n, pfx) if rms else _mlp_gelu(b, n, pfx)
        x = b.act(f"{pfx}.res2", [B, 1, H]); g.op(ADD, [a, o], [x])
    h = _norm(b, x, "final_norm", rms, out_kind=OUTPUT)
    if rms:
        wlm = b.const("W_lm", [H, V])
    else:
        wlm = b.act("tok_table_T", [H, V])
        g.op(TRANSPOSE, [tok], [wlm], perm=[1, 0])
    logits = b.act("logits", [B, 1, V], OUTPUT)
    g.op(LINEAR, [h, wlm], [logits], contract=1)
    consts = b.consts
    if like is not None:
        by_name = {like.graph.tensors[t]["name"]: a for t, a in like.consts.items()}
        consts = {t: by_name[td["name"]] for t, td in enumerate(g.tensors) if td["kind"] == CONST}
    return DecodeModel(cfg, t_max, g, consts, ids, pos, caches)


# ---- the layout-transform / layout-aware GEMM sweep ---------------------------------------------
def permute_case(B, S, nh, D, target, dtype=BF16, seed=5):
    """[B,S,nh,D] -> [B,nh,S,D] (target "BHSD") or [B,nh,D,S] (target "BHDS")."""
    perm = {"BHSD": [0, 2, 1, 3], "BHDS": [0, 2, 3, 1]}[target]
    g = GraphDesc()
    x = g.tensor("x", dtype, [B, S, nh, D], INPUT)
    od = [[B, S, nh, D][p] for p in perm]
    y = g.tensor("y", dtype, od, OUTPUT)
    g.op(TRANSPOSE, [x], [y], perm=perm)
    a = uniform(seed, 0, [B, S, nh, D])
    if dtype == BF16:
        a = round_bf16(a)
    return g, a


def permute_sweep_cases():
    for B in range(1, 9):
        for S in (128, 512, 2048):
            for nh in (12, 32):
                for D in (64, 128):
                    for target in ("BHSD", "BHDS"):
                        yield dict(B=B, S=S, nh=nh, D=D, target=target)


def gemm_case(M, N, K, a_major="row", b_major="row", dtype=BF16, seed=5, materialize=True):
    """Y[M,N] = A[M,K] . Bm[K,N] with A and Bm each held row- or column-major.

    A column-major operand is declared as the caller's transposed buffer followed by a
    TRANSPOSE op, which a planner can resolve to a zero-copy view.
    """
    g = GraphDesc()
    if a_major == "row":
        a = g.tensor("A", dtype, [M, K], INPUT)
        a_in = a
    else:
        a_in = g.tensor("A_T", dtype, [K, M], INPUT)
        a = g.tensor("A", dtype, [M, K], ACT)
        g.op(TRANSPOSE, [a_in], [a], perm=[1, 0])
    if b_major == "row":
        bm = g.tensor("Bm", dtype, [K, N], INPUT)
        b_in = bm
    else:
        b_in = g.tensor("Bm_T", dtype, [N, K], INPUT)
        bm = g.tensor("Bm", dtype, [K, N], ACT)
        g.op(TRANSPOSE, [b_in], [bm], perm=[1, 0])
    y = g.tensor("Y", dtype, [M, N], OUTPUT)
    g.op(LINEAR, [a, bm], [y], contract=1)
    arrays = None
    if materialize:
        A = uniform(seed, 0, [M, K]); Bv = uniform(seed, 1, [K, N])
        if dtype == BF16:
            A, Bv = round_bf16(A), round_bf16(Bv)
        arrays = {a_in: A if a_major == "row" else np.ascontiguousarray(A.T),
                  b_in: Bv if b_major == "row" else np.ascontiguousarray(Bv.T)}
    return g, arrays
