"""Pins for the numeric oracle: brute force on tiny shapes, closed forms, invariants."""
import math

import numpy as np
import pytest

from oracle import ops

RNG = np.random.default_rng(7)


def brute_linear(x, w, b):
    M, K = x.shape
    N = w.shape[1]
    y = [[0.0] * N for _ in range(M)]
    for i in range(M):
        for j in range(N):
            acc = 0.0
            for k in range(K):
                acc += float(x[i, k]) * float(w[k, j])
            y[i][j] = acc + (float(b[j]) if b is not None else 0.0)
    return np.array(y)


@pytest.mark.parametrize("M,K,N", [(8, 8, 8), (5, 3, 7), (1, 4, 2)])
def test_linear_brute_force(M, K, N):
    x, w, b = RNG.normal(size=(M, K)), RNG.normal(size=(K, N)), RNG.normal(size=N)
    np.testing.assert_allclose(ops.linear(x, w, b), brute_linear(x, w, b), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(ops.linear(x, w), brute_linear(x, w, None), rtol=1e-13, atol=1e-13)


def test_linear_identity_linearity_ones_and_transposed_operand():
    x = RNG.normal(size=(4, 6))
    assert np.array_equal(ops.linear(x, np.eye(6)), x)
    w = RNG.normal(size=(6, 3))
    y = RNG.normal(size=(4, 6))
    np.testing.assert_allclose(ops.linear(2 * x - 3 * y, w), 2 * ops.linear(x, w) - 3 * ops.linear(y, w),
                               rtol=1e-12, atol=1e-12)
    assert np.array_equal(ops.linear(np.ones((2, 5)), np.ones((5, 3))), np.full((2, 3), 5.0))
    # a transposed operand must NOT give the same answer (guards against x.T / w.T mix-ups)
    sq = RNG.normal(size=(5, 5))
    assert not np.allclose(ops.linear(sq, sq.T @ sq), ops.linear(sq.T, sq.T @ sq))


def test_linear_multi_dim_contraction():
    x = RNG.normal(size=(2, 3, 4, 5))          # [B,S,nh,D]
    w = RNG.normal(size=(4, 5, 6))             # [nh,D,H]
    y = ops.linear(x, w, contract=2)
    ref = np.zeros((2, 3, 6))
    for b in range(2):
        for s in range(3):
            for n in range(6):
                ref[b, s, n] = sum(x[b, s, h, d] * w[h, d, n] for h in range(4) for d in range(5))
    np.testing.assert_allclose(y, ref, rtol=1e-13, atol=1e-13)
    w1 = RNG.normal(size=(5, 2, 3))            # [K, nh, D]
    y1 = ops.linear(x, w1, RNG.normal(size=(2, 3)) * 0, contract=1)
    assert y1.shape == (2, 3, 4, 2, 3)


def brute_attention(q, k, v, causal):
    B, S, nh, D = q.shape
    out = np.zeros_like(q)
    for b in range(B):
        for h in range(nh):
            for i in range(S):
                js = [j for j in range(S) if (j <= i or not causal)]
                logits = [sum(q[b, i, h, d] * k[b, j, h, d] for d in range(D)) / math.sqrt(D) for j in js]
                m = max(logits)
                e = [math.exp(l - m) for l in logits]
                z = sum(e)
                for d in range(D):
                    out[b, i, h, d] = sum(e[n] / z * v[b, j, h, d] for n, j in enumerate(js))
    return out


@pytest.mark.parametrize("causal", [False, True])
def test_attention_chain_brute_force(causal):
    B, S, nh, D = 2, 7, 2, 4
    q, k, v = (RNG.normal(size=(B, S, nh, D)) for _ in range(3))
    qh = ops.transpose(q, (0, 2, 1, 3)); kT = ops.transpose(k, (0, 2, 3, 1)); vh = ops.transpose(v, (0, 2, 1, 3))
    p = ops.softmax(ops.bmm_qk(qh, kT, scale=1 / math.sqrt(D)), causal=causal)
    c = ops.transpose(ops.bmm_pv(p, vh), (0, 2, 1, 3))
    np.testing.assert_allclose(c, brute_attention(q, k, v, causal), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("causal", [False, True])
def test_attention_zero_query_is_mean_of_allowed_values(causal):
    B, S, nh, D = 1, 6, 2, 4
    k, v = RNG.normal(size=(B, S, nh, D)), RNG.normal(size=(B, S, nh, D))
    qh = np.zeros((B, nh, S, D))
    p = ops.softmax(ops.bmm_qk(qh, ops.transpose(k, (0, 2, 3, 1))), causal=causal)
    c = ops.bmm_pv(p, ops.transpose(v, (0, 2, 1, 3)))
    vh = np.transpose(v, (0, 2, 1, 3))
    for i in range(S):
        ref = vh[:, :, : i + 1].mean(axis=2) if causal else vh.mean(axis=2)
        np.testing.assert_allclose(c[:, :, i], ref, rtol=1e-12, atol=1e-13)


def test_attention_one_dominant_key_selects_its_value():
    S, D = 5, 4
    k = RNG.normal(size=(1, 1, S, D)); v = RNG.normal(size=(1, 1, S, D))
    q = 1e4 * k[:, :, 3:4, :] / np.linalg.norm(k[0, 0, 3])
    p = ops.softmax(ops.bmm_qk(q, np.transpose(k, (0, 1, 3, 2))))
    # the matching key wins unless another key has a larger projection; construct so it does
    scores = (q @ np.transpose(k, (0, 1, 3, 2)))[0, 0, 0]
    j = int(np.argmax(scores))
    np.testing.assert_allclose(ops.bmm_pv(p, v)[0, 0, 0], v[0, 0, j], rtol=1e-9, atol=1e-9)


def test_softmax_invariants():
    s = RNG.normal(size=(2, 3, 6, 6)) * 4
    p = ops.softmax(s)
    np.testing.assert_allclose(p.sum(-1), 1.0, rtol=0, atol=1e-12)
    np.testing.assert_allclose(ops.softmax(s + 123.0), p, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(ops.softmax(np.array([[1.0, 1.0, 0.0]]))[0, 0],
                               ops.softmax(np.array([[1.0, 1.0, 0.0]]))[0, 1], rtol=0, atol=0)
    np.testing.assert_allclose(ops.softmax(np.array([[0.0, math.log(3.0)]])), [[0.25, 0.75]], rtol=1e-15)
    pc = ops.softmax(s, causal=True)
    assert np.all(pc[..., np.triu_indices(6, 1)[0], np.triu_indices(6, 1)[1]] == 0.0)
    assert np.array_equal(pc[..., 0, :], np.broadcast_to(np.eye(6)[0], pc[..., 0, :].shape))
    np.testing.assert_allclose(pc.sum(-1), 1.0, atol=1e-12)
    np.testing.assert_allclose(ops.softmax(s, scale=0.5), ops.softmax(0.5 * s), rtol=1e-14)


def test_layernorm_rmsnorm_invariants():
    x = RNG.normal(size=(5, 64)) * 3 + 1.5
    one, zero = np.ones(64), np.zeros(64)
    y = ops.layernorm(x, one, zero, eps=1e-5)
    np.testing.assert_allclose(y.mean(-1), 0.0, atol=1e-12)
    var = x.var(-1)                                 # population variance (ddof = 0)
    np.testing.assert_allclose(y.var(-1), var / (var + 1e-5), rtol=1e-12)
    np.testing.assert_allclose(ops.layernorm(3 * x + 7, one, zero, eps=0.0), ops.layernorm(x, one, zero, eps=0.0),
                               rtol=1e-10, atol=1e-12)
    g, b = RNG.normal(size=64), RNG.normal(size=64)
    np.testing.assert_allclose(ops.layernorm(x, g, b), y * g + b, rtol=1e-13, atol=1e-13)
    # a two-element row has the closed form (+-1) * sqrt(v/(v+eps)) with v = ((a-b)/2)^2
    r = ops.layernorm(np.array([[1.0, 3.0]]), np.ones(2), np.zeros(2), eps=1e-5)
    np.testing.assert_allclose(r, [[-1 / math.sqrt(1 + 1e-5), 1 / math.sqrt(1 + 1e-5)]], rtol=1e-14)
    z = ops.rmsnorm(x, one, eps=1e-5)
    ms = (x * x).mean(-1)
    np.testing.assert_allclose((z * z).mean(-1), ms / (ms + 1e-5), rtol=1e-12)
    np.testing.assert_allclose(ops.rmsnorm(np.array([[3.0, 4.0]]), np.array([2.0, 1.0]), eps=0.0),
                               [[2 * 3 / math.sqrt(12.5), 4 / math.sqrt(12.5)]], rtol=1e-14)


def test_gelu_silu_closed_forms():
    x = RNG.normal(size=100) * 3
    assert ops.gelu(np.zeros(3)).tolist() == [0, 0, 0]
    np.testing.assert_allclose(ops.gelu(x) - ops.gelu(-x), x, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(ops.silu(x) - ops.silu(-x), x, rtol=1e-13, atol=1e-14)
    np.testing.assert_allclose(ops.gelu(np.array([1.0])), [0.5 * (1 + math.erf(1 / math.sqrt(2)))], rtol=1e-15)
    np.testing.assert_allclose(ops.gelu(np.array([1.0]))[0], 0.8413447460685429, rtol=1e-13)  # Phi(1)
    np.testing.assert_allclose(ops.gelu(np.array([40.0, -40.0])), [40.0, 0.0], atol=1e-12)
    np.testing.assert_allclose(ops.silu(np.array([40.0, -40.0])), [40.0, 0.0], atol=1e-12)
    np.testing.assert_allclose(ops.silu(np.array([math.log(3.0)])), [math.log(3.0) * 0.75], rtol=1e-14)
    np.testing.assert_allclose(ops.gelu(x, tanh_form=True), ops.gelu(x), atol=2e-3)
    pts = np.linspace(-4, 4, 33)
    np.testing.assert_allclose(ops.gelu(pts), [0.5 * t * (1 + math.erf(t / math.sqrt(2))) for t in pts], rtol=1e-14, atol=1e-16)


@pytest.mark.parametrize("interleaved", [False, True])
def test_rope_invariants(interleaved):
    B, S, nh, D = 1, 9, 2, 8
    q, k = RNG.normal(size=(B, S, nh, D)), RNG.normal(size=(B, S, nh, D))
    rq, rk = ops.rope(q, interleaved=interleaved), ops.rope(k, interleaved=interleaved)
    assert np.array_equal(rq[:, 0], q[:, 0])                                   # position 0: identity
    np.testing.assert_allclose(np.linalg.norm(rq, axis=-1), np.linalg.norm(q, axis=-1), rtol=1e-13)
    # scores depend on p - p' only: same vectors placed 3 positions later give the same product
    q2 = np.zeros_like(q); k2 = np.zeros_like(k)
    q2[:, 3:] = q[:, :-3]; k2[:, 3:] = k[:, :-3]
    s1 = np.einsum("bihd,bjhd->bhij", rq, rk)[:, :, :-3, :-3]
    s2 = np.einsum("bihd,bjhd->bhij", ops.rope(q2, interleaved=interleaved), ops.rope(k2, interleaved=interleaved))[:, :, 3:, 3:]
    np.testing.assert_allclose(s1, s2, rtol=1e-11, atol=1e-12)


def test_rope_explicit_small_case():
    x = np.zeros((1, 2, 1, 4)); x[0, 1, 0] = [1.0, 2.0, 3.0, 4.0]
    y = ops.rope(x, base=100.0)
    # D=4: pairs (0,2) at angle 1*100^0 = 1, (1,3) at angle 1*100^(-1/2) = 0.1
    np.testing.assert_allclose(y[0, 1, 0], [math.cos(1) - 3 * math.sin(1), 2 * math.cos(.1) - 4 * math.sin(.1),
                                            3 * math.cos(1) + math.sin(1), 4 * math.cos(.1) + 2 * math.sin(.1)], rtol=1e-14)
    yi = ops.rope(x, base=100.0, interleaved=True)
    np.testing.assert_allclose(yi[0, 1, 0], [math.cos(1) - 2 * math.sin(1), 2 * math.cos(1) + math.sin(1),
                                             3 * math.cos(.1) - 4 * math.sin(.1), 4 * math.cos(.1) + 3 * math.sin(.1)], rtol=1e-14)


def test_transpose_and_layout_round_trip():
    x = RNG.normal(size=(2, 3, 4, 5))
    for perm in [(0, 2, 1, 3), (0, 2, 3, 1), (3, 1, 0, 2)]:
        y = ops.transpose(x, perm)
        for idx in np.ndindex(*y.shape):
            src = [0] * 4
            for j, p in enumerate(perm):
                src[p] = idx[j]
            assert y[idx] == x[tuple(src)]
        assert np.array_equal(ops.transpose(y, np.argsort(perm)), x)
        buf = ops.store_in_layout(x, perm)
        st = ops.strides_for(x.shape, perm)
        for idx in [(1, 2, 3, 4), (0, 0, 0, 0), (1, 0, 2, 1)]:
            assert buf[sum(i * s for i, s in zip(idx, st))] == x[idx]
        assert np.array_equal(ops.load_from_layout(buf, x.shape, perm), x)


def test_every_layout_agrees_with_canonical_gemm():
    """Operands stored row- or column-major, read back through index arithmetic, same GEMM."""
    A, Bm = RNG.normal(size=(5, 7)), RNG.normal(size=(7, 3))
    ref = ops.linear(A, Bm)
    for pa in [(0, 1), (1, 0)]:
        for pb in [(0, 1), (1, 0)]:
            a2 = ops.load_from_layout(ops.store_in_layout(A, pa), A.shape, pa)
            b2 = ops.load_from_layout(ops.store_in_layout(Bm, pb), Bm.shape, pb)
            assert np.array_equal(ops.linear(a2, b2), ref)


def test_embed_and_select():
    tok = RNG.normal(size=(10, 4)); pos = RNG.normal(size=(3, 4))
    ids = np.array([[1, 9, 0], [2, 2, 5]])
    x = ops.embed(ids, tok, pos)
    for b in range(2):
        for s in range(3):
            assert np.array_equal(x[b, s], tok[ids[b, s]] + pos[s])
    assert np.array_equal(ops.embed(ids, tok), tok[ids])
    assert np.array_equal(ops.select_last_token(x), x[:, 2, :])
