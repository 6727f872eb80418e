"""Pins for the oracle's primitives: closed forms, special cases and brute force."""
import math

import numpy as np
import pytest

from oracle import odb_oracle as O

RNG = np.random.default_rng(1234)


def test_bf16_round_known_values():
    # bf16 keeps 8 significant bits: spacing 2^-7 in [1,2)
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -(1.0 + 2 ** -8), 0.0,
                  1.0 + 2 ** -8 + 2 ** -20, 3.14159265])
    want = np.array([1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7, -1.0, 0.0, 1.0 + 2 ** -7, 3.140625])
    got = O.bf16_round(x)
    assert got.dtype == x.dtype
    assert (got == want).all()                      # ties go to the even mantissa
    y = RNG.normal(size=1000)
    r = O.bf16_round(y)
    assert (O.bf16_round(r) == r).all()             # idempotent
    assert (np.abs(r - y) <= np.abs(y) * 2 ** -8 * 1.0001).all()


def test_rmsnorm_closed_forms():
    x = RNG.normal(size=(5, 64)) * 7.0
    y = O.rmsnorm(x, np.ones(64), 0.0)
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0, atol=1e-12)
    # constant vector c -> c/|c| regardless of scale; gain multiplies elementwise
    g = RNG.normal(size=64)
    y2 = O.rmsnorm(np.full((1, 64), -3.0), g, 0.0)
    assert np.allclose(y2, -g[None, :], atol=1e-12)
    # eps enters under the root: x = 0 -> 0, and a single row of ones -> 1/sqrt(1+eps)
    assert (O.rmsnorm(np.zeros((1, 8)), np.ones(8), 1e-5) == 0).all()
    assert np.allclose(O.rmsnorm(np.ones((1, 8)), np.ones(8), 0.21), 1 / math.sqrt(1.21))


def test_normed_projection_is_rmsnorm_then_matmul():
    x = RNG.normal(size=(6, 32)) * 3.0
    g = RNG.normal(size=32)
    w1, w2 = RNG.normal(size=(5, 32)), RNG.normal(size=(7, 32))
    ident = lambda a: a
    y1, y2 = O.normed_projection(x, g, 1e-5, [w1, w2], ident)
    assert np.allclose(y1, O.rmsnorm(x, g, 1e-5) @ w1.T, rtol=1e-12) and np.allclose(y2, O.rmsnorm(x, g, 1e-5) @ w2.T, rtol=1e-12)
    # with rounding, the rounded operand is x * gain (scale invariant input: the row scalar is applied afterwards)
    y, = O.normed_projection(x, g, 0.0, [w1], O.bf16_round)
    yk, = O.normed_projection(64.0 * x, g, 0.0, [w1], O.bf16_round)     # power-of-two rescale: same bf16 mantissas
    assert np.allclose(y, yk, rtol=1e-12)
    assert np.abs(y - y1).max() <= 2 ** -7 * np.abs(O.rmsnorm(x, g, 0.0)) .max() * np.abs(w1).sum(1).max()


def test_rope_closed_forms():
    hd, H = 16, 3
    x = RNG.normal(size=(6, H, hd))
    pos = np.array([0, 1, 2, 5, 100, 2047])
    y = O.rope(x, pos, 500000.0)
    assert np.allclose(y[0], x[0], atol=0)                           # identity at position 0
    assert np.allclose((y * y).sum(-1), (x * x).sum(-1), rtol=1e-12)  # a rotation
    # first pair (i=0, i+hd/2) rotates by exactly pos radians
    p = 5.0
    want0 = x[3, :, 0] * math.cos(p) - x[3, :, hd // 2] * math.sin(p)
    want8 = x[3, :, hd // 2] * math.cos(p) + x[3, :, 0] * math.sin(p)
    assert np.allclose(y[3, :, 0], want0) and np.allclose(y[3, :, hd // 2], want8)
    # last pair rotates by pos * theta^(-(hd-2)/hd)
    a = 100.0 * 500000.0 ** (-(hd - 2) / hd)
    want = x[4, :, hd // 2 - 1] * math.cos(a) - x[4, :, hd - 1] * math.sin(a)
    assert np.allclose(y[4, :, hd // 2 - 1], want)
    # relative property: <rope(q,m), rope(k,n)> depends only on m-n
    q = RNG.normal(size=(1, 1, hd))
    k = RNG.normal(size=(1, 1, hd))
    def dot(m, n):
        return float((O.rope(q, np.array([m]), 1e4) * O.rope(k, np.array([n]), 1e4)).sum())
    assert abs(dot(7, 3) - dot(104, 100)) < 1e-9
    assert abs(dot(7, 3) - dot(3, 7)) > 1e-6


def test_silu():
    assert O.silu(np.array([0.0]))[0] == 0.0
    x = np.array([-3.0, 0.5, 4.0])
    assert np.allclose(O.silu(x), x * (1 / (1 + np.exp(-x))))
    assert np.allclose(O.silu(x) - O.silu(-x), x)                   # x*sig(x) - (-x)*sig(-x) = x


def _attention_loops(q, k, v, vis):
    """Per row, per head, per key Python loops: the definition with nothing vectorised."""
    M, H, hd = q.shape
    out = np.zeros_like(q)
    for r in range(M):
        for h in range(H):
            keys = [j for j in range(k.shape[0]) if vis[r, j]]
            sc = [sum(q[r, h, t] * k[j, h, t] for t in range(hd)) / math.sqrt(hd) for j in keys]
            mx = max(sc)
            w = [math.exp(s - mx) for s in sc]
            z = sum(w)
            for wj, j in zip(w, keys):
                for t in range(hd):
                    out[r, h, t] += wj / z * v[j, h, t]
    return out


def test_attention_brute_force_random_visibility():
    M, N, H, hd = 5, 9, 2, 8
    q = RNG.normal(size=(M, H, hd))
    k = RNG.normal(size=(N, H, hd))
    v = RNG.normal(size=(N, H, hd))
    vis = RNG.random((M, N)) < 0.6
    vis[:, 0] = True
    got = O.attention(q, k, v, vis)
    assert np.allclose(got, _attention_loops(q, k, v, vis), atol=1e-12)


def test_attention_special_cases():
    M, N, H, hd = 3, 4, 2, 8
    q = RNG.normal(size=(M, H, hd))
    k = RNG.normal(size=(N, H, hd))
    v = RNG.normal(size=(N, H, hd))
    one = np.zeros((M, N), dtype=bool)
    one[:, 2] = True
    assert np.allclose(O.attention(q, k, v, one), np.broadcast_to(v[2], (M, H, hd)))  # single key -> its V
    # identical keys -> uniform weights -> mean of V
    ksame = np.broadcast_to(k[:1], (N, H, hd)).copy()
    allv = np.ones((M, N), dtype=bool)
    assert np.allclose(O.attention(q, ksame, v, allv), np.broadcast_to(v.mean(0), (M, H, hd)))
    # a key far more aligned with q than the rest takes all the weight
    kbig = k.copy()
    kbig[1] = 1000.0 * q[0]
    assert np.allclose(O.attention(q[:1], kbig, v, allv[:1])[0], v[1], atol=1e-9)
    # value rows identical -> output equals that row whatever the scores (weights sum to 1)
    vsame = np.broadcast_to(v[:1], (N, H, hd)).copy()
    assert np.allclose(O.attention(q, k, vsame, allv), np.broadcast_to(v[0], (M, H, hd)))


def test_confidence_matches_softmax_and_rules():
    V, mask_id = 50, 49
    logits = RNG.normal(size=(7, V)) * 3
    conf, tok = O.confidence(logits, mask_id)
    l32 = logits.astype(np.float32).astype(np.float64)[:, :mask_id]
    p = np.exp(l32 - l32.max(1, keepdims=True))
    p /= p.sum(1, keepdims=True)
    assert np.allclose(p.sum(1), 1.0)
    assert (tok == p.argmax(1)).all()
    assert np.allclose(conf, p.max(1), rtol=1e-6)
    assert conf.dtype == np.float32 and tok.dtype == np.int32
    # [MASK] is never predicted even when its logit is the largest
    logits[:, mask_id] = 100.0
    conf2, tok2 = O.confidence(logits, mask_id)
    assert (tok2 == tok).all() and np.allclose(conf2, conf)
    # all-equal logits: V-1 candidates, lowest id wins
    c0, t0 = O.confidence(np.zeros((2, V)), mask_id)
    assert (t0 == 0).all() and np.allclose(c0, 1.0 / (V - 1))
    # exact tie between two ids -> lower id
    tie = np.zeros((1, V))
    tie[0, 7] = tie[0, 3] = 5.0
    assert O.confidence(tie, mask_id)[1][0] == 3
