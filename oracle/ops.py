"""CPU fp64 oracle: operator definitions. TEST INFRASTRUCTURE ONLY.

Only tests, the smoke entry and the bench's cpu-baseline leg may import this package; the product
(the CUDA library and its binding) never does, and shares no code with it.

The method under test moves data between layouts and arena offsets without changing values
(paper, Sec. "Design", paragraphs "Loop Reordering" and "Memory Allocation and Management": loop
order and layout affect speed only; tensors with disjoint lifetimes may share memory). Its result
therefore has a plain definition: run every operator of the graph on canonical row-major arrays,
one fresh array per tensor, in double precision. Each function below is that definition.

GEMM is the one operator the paper defines (Sec. "Background", "Memory Layout in Kernel
Implementation": left input (i,k), right input (k,j), output (i,j)). The remaining operators are
the standard textbook definitions of the operators the paper lists by name (Softmax, LayerNorm,
GELU, Add, Transpose, Gather; Sec. "Implementation", "Compiler").

Pins (tests/test_oracle_ops.py, tests/test_oracle_decode.py): brute-force loops on tiny shapes, closed
forms and invariants; the cached decoding step against whole-sequence causal attention.
No function here is "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

try:  # library routine for erf; math.erf element by element if scipy is absent
    from scipy.special import erf as _erf
except Exception:  # pragma: no cover
    _erf = np.vectorize(math.erf, otypes=[np.float64])


def embed(ids, tok, pos=None, pos0=0):
    """x[b,s,:] = tok[ids[b,s],:] (+ pos[pos0 + s,:]) — a gather plus an optional add of the position rows; pos0 is
    the number of tokens that came before (0 for a whole sequence; one number for the batch or one per sequence)."""
    x = np.asarray(tok, dtype=np.float64)[np.asarray(ids, dtype=np.int64)]
    if pos is not None:
        B, S = x.shape[0], x.shape[1]
        p0 = np.asarray(pos0, dtype=np.int64).reshape(-1)
        assert p0.size in (1, B)
        rows = np.broadcast_to(p0, (B,))[:, None] + np.arange(S)[None, :]
        assert rows.min() >= 0 and rows.max() < np.asarray(pos).shape[0]
        x = x + np.asarray(pos, dtype=np.float64)[rows]
    return x


def linear(x, w, bias=None, contract=1):
    """Contract the last `contract` dims of x with the first `contract` dims of w (GEMM).

    y[m, n] = sum_k x[m, k] * w[k, n] (+ bias[n]) with m, k, n the flattened index groups.
    """
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    kd = x.shape[x.ndim - contract:]
    assert tuple(kd) == tuple(w.shape[:contract]), (x.shape, w.shape, contract)
    K = int(np.prod(kd))
    lead = x.shape[: x.ndim - contract]
    nd = w.shape[contract:]
    y = x.reshape(-1, K) @ w.reshape(K, -1)
    if bias is not None:
        y = y + np.asarray(bias, dtype=np.float64).reshape(1, -1)
    return y.reshape(tuple(lead) + tuple(nd))


def bmm_qk(qh, kT, scale=1.0):
    """s[b,h,i,j] = scale * sum_d qh[b,h,i,d] * kT[b,h,d,j]."""
    return np.matmul(np.asarray(qh, np.float64), np.asarray(kT, np.float64)) * float(scale)


def bmm_pv(p, vh):
    """c[b,h,i,d] = sum_j p[b,h,i,j] * vh[b,h,j,d]."""
    return np.matmul(np.asarray(p, np.float64), np.asarray(vh, np.float64))


def softmax(s, causal=False, scale=1.0):
    """Row-wise over the last dim: exp(s-max)/sum over the allowed j (j <= i when causal).

    Disallowed entries are exactly 0 and take no part in max or sum.
    """
    s = np.asarray(s, dtype=np.float64) * float(scale)
    if causal:
        n_i, n_j = s.shape[-2], s.shape[-1]
        allowed = np.arange(n_j)[None, :] <= np.arange(n_i)[:, None]
        s = np.where(allowed, s, -np.inf)
    m = np.max(s, axis=-1, keepdims=True)
    e = np.exp(s - m)
    return e / np.sum(e, axis=-1, keepdims=True)


def layernorm(x, gamma, beta, eps=1e-5):
    """(x - mean) / sqrt(var + eps) * gamma + beta over the last dim; population variance."""
    x = np.asarray(x, dtype=np.float64)
    mu = np.mean(x, axis=-1, keepdims=True)
    var = np.mean((x - mu) ** 2, axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * np.asarray(gamma, np.float64) + np.asarray(beta, np.float64)


def rmsnorm(x, gamma, eps=1e-5):
    """x / sqrt(mean(x^2) + eps) * gamma over the last dim."""
    x = np.asarray(x, dtype=np.float64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * np.asarray(gamma, np.float64)


def gelu(x, tanh_form=False):
    """erf form x/2 (1 + erf(x/sqrt 2)), or the tanh approximation when asked."""
    x = np.asarray(x, dtype=np.float64)
    if tanh_form:
        return 0.5 * x * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)))
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def silu(x):
    """x / (1 + exp(-x))."""
    x = np.asarray(x, dtype=np.float64)
    return x / (1.0 + np.exp(-x))


def add(a, b):
    return np.asarray(a, np.float64) + np.asarray(b, np.float64)


def mul(a, b):
    return np.asarray(a, np.float64) * np.asarray(b, np.float64)


def rope(x, base=10000.0, interleaved=False, pos0=0):
    """Rotary embedding on x[b, s, h, d]; position p = pos0 + s (0-based; pos0 is the number of
    tokens that came before this call's first row, 0 for a whole sequence; one number for the whole
    batch or one per sequence).

    Rotate-half pairing (i, i + D/2) by angle p * base^(-2i/D); the interleaved form pairs
    (2i, 2i+1) with the same angles.
    """
    x = np.asarray(x, dtype=np.float64)
    B, S, nh, D = x.shape
    half = D // 2
    i = np.arange(half, dtype=np.float64)
    p0 = np.asarray(pos0, dtype=np.float64).reshape(-1)
    assert p0.size in (1, B)
    p0 = np.broadcast_to(p0, (B,))
    theta = (p0[:, None] + np.arange(S, dtype=np.float64)[None, :])[:, :, None] * base ** (-2.0 * i / D)[None, None, :]
    c = np.cos(theta)[:, :, None, :]
    s = np.sin(theta)[:, :, None, :]
    y = np.empty_like(x)
    if interleaved:
        a, b = x[..., 0::2], x[..., 1::2]
        y[..., 0::2] = a * c - b * s
        y[..., 1::2] = b * c + a * s
    else:
        a, b = x[..., :half], x[..., half:]
        y[..., :half] = a * c - b * s
        y[..., half:] = b * c + a * s
    return y


def cached_attention(q, k, v, k_cache, v_cache, pos, scale=1.0):
    """One decoding step of attention against a key/value cache.

    q[B,1,nh,D] is the query of the token at position t = pos (one position for the whole batch, or
    pos[b] per sequence); k, v[B,1,nkv,D] are its key and value; k_cache, v_cache[B,Tmax,nkv,D] hold
    the keys and values of positions 0..t-1 (rows from t on are unspecified). The step stores k, v as
    row t of the caches and returns
      ctx[b,0,h,:] = sum_{j<=t} softmax_j(scale * q[b,0,h,:] . K[b,j,g,:]) V[b,j,g,:],  g = h // (nh/nkv),
    that is, the row for query position t of causal attention over the t+1 tokens so far (query
    heads share key/value heads in groups when nkv < nh). Returns (ctx, k_cache', v_cache').
    """
    q = np.asarray(q, np.float64)
    kc = np.array(k_cache, dtype=np.float64)
    vc = np.array(v_cache, dtype=np.float64)
    B, one, nh, D = q.shape
    Tmax, nkv = kc.shape[1], kc.shape[2]
    ts = np.asarray(pos).reshape(-1)
    assert ts.size in (1, B) and one == 1 and nh % nkv == 0
    ts = [int(ts[b if ts.size == B else 0]) for b in range(B)]
    ctx = np.zeros((B, 1, nh, D))
    for b in range(B):
        t = ts[b]
        assert 0 <= t < Tmax
        kc[b, t] = np.asarray(k, np.float64)[b, 0]
        vc[b, t] = np.asarray(v, np.float64)[b, 0]
        for h in range(nh):
            g = h // (nh // nkv)
            s = (kc[b, : t + 1, g, :] @ q[b, 0, h, :]) * float(scale)
            e = np.exp(s - np.max(s))
            ctx[b, 0, h, :] = (e / np.sum(e)) @ vc[b, : t + 1, g, :]
    return ctx, kc, vc


def transpose(x, perm):
    """out[i0, i1, ...] = x[index with out dim j taken from x dim perm[j]] (numpy semantics)."""
    return np.ascontiguousarray(np.transpose(np.asarray(x, np.float64), perm))


def select_last_token(x):
    """[B, S, H] -> [B, H], the row of the final position."""
    return np.ascontiguousarray(np.asarray(x, np.float64)[:, -1, :])


# ---- layouts as index arithmetic (for the "every layout agrees with canonical" pin) ----------
def strides_for(dims, perm):
    """Element strides per logical dim of a dense tensor stored with dims ordered `perm`
    (slowest to fastest)."""
    st = [0] * len(dims)
    run = 1
    for d in reversed(perm):
        st[d] = run
        run *= dims[d]
    return st


def store_in_layout(x, perm):
    """Flat buffer holding x with logical dims ordered `perm` slowest->fastest."""
    return np.ascontiguousarray(np.transpose(x, perm)).reshape(-1)


def load_from_layout(buf, dims, perm):
    """Inverse of store_in_layout: rebuild the canonical array from a flat buffer."""
    pd = [dims[p] for p in perm]
    inv = np.argsort(perm)
    return np.ascontiguousarray(np.transpose(np.asarray(buf).reshape(pd), inv))
