"""CPU fp64 oracle: whole-model formulas written directly. TEST INFRASTRUCTURE ONLY.

A second, independent statement of what the three model families compute, straight from the
per-family equations (no graph, no TRANSPOSE ops, attention written per head with einsum). It
exists to pin the graph interpreter and the graph wiring: both must give the same numbers.

  encoder (post-LN): x0 = LN(tok[ids] + pos); x <- LN(x + Attn(x) Wo + bo);
                     x <- LN(x + GELU(x W1 + b1) W2 + b2).
  gpt (pre-LN, causal): x0 = tok[ids] + pos; x <- x + Attn(LN(x)) Wo + bo;
                     x <- x + GELU(LN(x) W1 + b1) W2 + b2; h = LN(x); logits = h[:, -1] tok^T.
  llama: x0 = tok[ids]; n = RMS(x); q, k = RoPE(n Wq), RoPE(n Wk); x <- x + Attn(q,k,v) Wo;
                     n = RMS(x); x <- x + (SiLU(n Wg) * (n Wu)) Wd; h = RMS(x); logits = h[-1] Wlm.
  Attn: softmax_j(q_i . k_j / sqrt(D)) v_j per head (j <= i when causal).

`w` maps tensor names to arrays (the names the synthetic workloads use).
"""
from __future__ import annotations

import math

import numpy as np

from . import ops


def _f(a):
    return np.asarray(a, dtype=np.float64)


def _attn(q, k, v, causal):
    # q, k, v: [B, S, nh, D]
    D = q.shape[-1]
    s = np.einsum("bihd,bjhd->bhij", q, k) / math.sqrt(D)
    p = ops.softmax(s, causal=causal)
    return np.einsum("bhij,bjhd->bihd", p, v)


def _proj_heads(x, W, b=None):
    y = np.einsum("bsk,khd->bshd", x, _f(W))
    return y if b is None else y + _f(b)[None, None]


def forward(family, L, w, ids):
    """Returns (hidden [B,S,H], logits [B,V] or None)."""
    ids = np.asarray(ids)
    x = _f(w["tok_table"])[ids]
    if family != "llama":
        x = x + _f(w["pos_table"])[None, : ids.shape[1]]
    if family == "encoder":
        x = ops.layernorm(x, w["emb_ln.gamma"], w["emb_ln.beta"])
        for l in range(L):
            p = f"l{l}"
            q = _proj_heads(x, w[f"{p}.Wq"], w[f"{p}.bq"])
            k = _proj_heads(x, w[f"{p}.Wk"], w[f"{p}.bk"])
            v = _proj_heads(x, w[f"{p}.Wv"], w[f"{p}.bv"])
            c = _attn(q, k, v, causal=False)
            o = np.einsum("bshd,hdn->bsn", c, _f(w[f"{p}.Wo"])) + _f(w[f"{p}.bo"])
            x = ops.layernorm(x + o, w[f"{p}.ln1.gamma"], w[f"{p}.ln1.beta"])
            f = ops.gelu(x @ _f(w[f"{p}.W1"]) + _f(w[f"{p}.b1"]))
            o = f @ _f(w[f"{p}.W2"]) + _f(w[f"{p}.b2"])
            x = ops.layernorm(x + o, w[f"{p}.ln2.gamma"], w[f"{p}.ln2.beta"])
        return x, None
    if family == "gpt":
        for l in range(L):
            p = f"l{l}"
            n = ops.layernorm(x, w[f"{p}.ln1.gamma"], w[f"{p}.ln1.beta"])
            q = _proj_heads(n, w[f"{p}.Wq"], w[f"{p}.bq"])
            k = _proj_heads(n, w[f"{p}.Wk"], w[f"{p}.bk"])
            v = _proj_heads(n, w[f"{p}.Wv"], w[f"{p}.bv"])
            c = _attn(q, k, v, causal=True)
            x = x + np.einsum("bshd,hdn->bsn", c, _f(w[f"{p}.Wo"])) + _f(w[f"{p}.bo"])
            n = ops.layernorm(x, w[f"{p}.ln2.gamma"], w[f"{p}.ln2.beta"])
            f = ops.gelu(n @ _f(w[f"{p}.W1"]) + _f(w[f"{p}.b1"]))
            x = x + f @ _f(w[f"{p}.W2"]) + _f(w[f"{p}.b2"])
        h = ops.layernorm(x, w["final_norm.gamma"], w["final_norm.beta"])
        return h, h[:, -1, :] @ _f(w["tok_table"]).T
    if family == "llama":
        for l in range(L):
            p = f"l{l}"
            n = ops.rmsnorm(x, w[f"{p}.ln1.gamma"])
            q = ops.rope(_proj_heads(n, w[f"{p}.Wq"]))
            k = ops.rope(_proj_heads(n, w[f"{p}.Wk"]))
            v = _proj_heads(n, w[f"{p}.Wv"])
            c = _attn(q, k, v, causal=True)
            x = x + np.einsum("bshd,hdn->bsn", c, _f(w[f"{p}.Wo"]))
            n = ops.rmsnorm(x, w[f"{p}.ln2.gamma"])
            m = ops.silu(n @ _f(w[f"{p}.Wg"])) * (n @ _f(w[f"{p}.Wu"]))
            x = x + m @ _f(w[f"{p}.Wd"])
        h = ops.rmsnorm(x, w["final_norm.gamma"])
        return h, h[:, -1, :] @ _f(w["W_lm"])
    raise ValueError(family)
