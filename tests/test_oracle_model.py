"""Pins for the oracle's forward, refresh and block step."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import synth
from oracle import odb_oracle as O
from oracle.inputs import model_from_synth

SMALL = synth.ModelShape(n_layers=2, d_model=64, n_heads=4, head_dim=16, d_ffn=96, vocab=97,
                         mask_id=96, eos_id=95, rope_theta=10000.0)


@pytest.fixture(scope="module")
def small_model():
    return model_from_synth(SMALL, seed=3)


@pytest.fixture(scope="module")
def tiny_model():
    return model_from_synth(synth.TINY, seed=0)


def _torch_forward(model: O.Model, tok, T):
    """Full bidirectional forward restated with torch library routines (fp64, no rounding).
    RoPE is written with complex multiplication, a different formulation from the oracle's."""
    d, H, hd = model.d_model, model.n_heads, model.head_dim
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    h = t(model.embed)[torch.from_numpy(np.asarray(tok[:T], dtype=np.int64))]
    inv = model.rope_theta ** (-torch.arange(0, hd // 2, dtype=torch.float64) * 2 / hd)
    rot = torch.polar(torch.ones(T, hd // 2, dtype=torch.float64),
                      torch.arange(T, dtype=torch.float64)[:, None] * inv[None, :])   # e^{i pos theta_i}

    def rope(x):                                           # x [T][H][hd]
        z = torch.complex(x[..., : hd // 2], x[..., hd // 2:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    for l in range(model.n_layers):
        w = model.layer(l)
        a = F.rms_norm(h, (d,), t(w["g1"]), model.rms_eps)
        q = rope(F.linear(a, t(w["wq"])).view(T, H, hd)).transpose(0, 1)
        k = rope(F.linear(a, t(w["wk"])).view(T, H, hd)).transpose(0, 1)
        v = F.linear(a, t(w["wv"])).view(T, H, hd).transpose(0, 1)
        o = F.scaled_dot_product_attention(q, k, v).transpose(0, 1).reshape(T, d)
        h = h + F.linear(o, t(w["wo"]))
        b = F.rms_norm(h, (d,), t(w["g2"]), model.rms_eps)
        h = h + F.linear(F.silu(F.linear(b, t(w["wg"]))) * F.linear(b, t(w["wu"])), t(w["wd"]))
    n = F.rms_norm(h, (d,), t(model.final_gain), model.rms_eps)
    return F.linear(n, t(model.lm_head)).numpy()


def test_refresh_equals_torch_library_forward(small_model):
    m = small_model
    x = synth.sequence(1, 0, 10, 14, SMALL)
    x[12] = 5                                                         # a decoded token inside the response
    T, s = 24, 10
    _, conf, tok, logits = O.refresh_prefill(m, x, T, s, faithful=False, return_logits=True)
    ref = _torch_forward(m, x, T)[s:T]
    assert np.allclose(logits, ref, rtol=1e-9, atol=1e-11)
    p = torch.softmax(torch.from_numpy(np.delete(ref, SMALL.mask_id, axis=1).astype(np.float32)).double(), -1)
    assert np.allclose(conf, p.max(-1).values.numpy(), rtol=1e-5)
    assert (tok == np.delete(ref, SMALL.mask_id, axis=1).argmax(1)).all()


def test_cache_holds_post_rope_k_and_v(small_model):
    m = small_model
    x = synth.sequence(2, 0, 6, 6, SMALL)
    cache, _, _ = O.refresh_prefill(m, x, 12, 6, faithful=False)
    w = m.layer(0)
    a = O.rmsnorm(m.embed[x[:12]], w["g1"], m.rms_eps)
    k = O.rope((a @ w["wk"].T).reshape(12, 4, 16), np.arange(12), m.rope_theta)
    assert np.allclose(cache.k[0], k) and np.allclose(cache.v[0], (a @ w["wv"].T).reshape(12, 4, 16))
    assert cache.length == 12 and len(cache.k) == m.n_layers


@pytest.mark.parametrize("faithful", [False, True])
def test_step_right_after_refresh_equals_refresh(small_model, faithful):
    """A plain step issued right after a refresh, nothing committed in between, sees exactly
    the keys the refresh saw, so its logits on the block rows equal the refresh's."""
    m = small_model
    x = synth.sequence(4, 0, 9, 16, SMALL).astype(np.int64)
    T, s, e = 25, 13, 17                                             # second block of 4
    x[9:13] = [3, 1, 4, 1]
    cache, conf, tok, logits = O.refresh_prefill(m, x, T, 9, faithful=faithful, return_logits=True)
    c1, t1, lg, _, _ = O.block_decode_step(m, cache, x, T, s, e, [()], [], [], False,
                                           faithful=faithful, return_logits=True)
    tol = dict(rtol=1e-9, atol=1e-11) if not faithful else dict(rtol=0, atol=0)
    assert np.allclose(lg, logits[s - 9:e - 9], **tol)
    assert (t1[0] == tok[s - 9:e - 9]).all() and np.allclose(c1[0], conf[s - 9:e - 9], rtol=1e-6)


def test_step_uses_cached_outside_and_fresh_inside(small_model):
    m = small_model
    x = synth.sequence(5, 0, 8, 12, SMALL).astype(np.int64)
    T, s, e = 20, 8, 12
    cache, _, _ = O.refresh_prefill(m, x, T, s, faithful=False)
    base = O.block_decode_step(m, cache, x, T, s, e, [()], [], [], False, faithful=False, return_logits=True)[2]
    # negative control: a token outside the block changed after the refresh is not seen (stale cache)
    y = x.copy()
    y[2] = (y[2] + 1) % 90
    y[15] = 7
    out = O.block_decode_step(m, cache, y, T, s, e, [()], [], [], False, faithful=False, return_logits=True)[2]
    assert np.array_equal(out, base)
    # a token inside the block changed after the refresh is seen by every row of the block
    z = x.copy()
    z[9] = 11
    out2 = O.block_decode_step(m, cache, z, T, s, e, [()], [], [], False, faithful=False, return_logits=True)[2]
    assert (np.abs(out2 - base).max(axis=1) > 1e-6).all()
    # and equals a full forward of the changed sequence only if the outside K/V are recomputed:
    full = _torch_forward(m, z, T)[s:e]
    assert np.abs(out2 - full).max() > 1e-6
    # block covering the whole response with an unchanged prompt... first layer K/V of the prompt
    # do not depend on the response, deeper layers do: so equality holds for a 1-layer model
    m1 = model_from_synth(SMALL.with_layers(1), seed=3)
    cache1, _, _ = O.refresh_prefill(m1, x, T, s, faithful=False)
    zz = x.copy()
    zz[8:20] = np.arange(12) + 20
    st = O.block_decode_step(m1, cache1, zz, T, 8, 20, [()], [], [], False, faithful=False, return_logits=True)[2]
    assert np.allclose(st, _torch_forward(m1, zz, T)[8:20], rtol=1e-9, atol=1e-11)


def test_copies_are_mutually_invisible(small_model):
    m = small_model
    x = synth.sequence(6, 0, 8, 8, SMALL).astype(np.int64)
    T, s, e = 16, 8, 16
    cache, conf, tok = O.refresh_prefill(m, x, T, s, faithful=False)
    x[9] = tok[1]
    rank_pos, rank_tok = [11, 14], [int(tok[3]), int(tok[6])]
    subsets = O.copy_subsets(2, 4, False)
    assert subsets == [(), (1,), (2,), (1, 2)]
    conf4, tok4, lg4, r_copy, r_pos = O.block_decode_step(m, cache, x, T, s, e, subsets, rank_pos, rank_tok,
                                                          False, faithful=False, return_logits=True)
    assert lg4.shape[0] == 32
    for c, y in enumerate(subsets):
        xc = x.copy()
        for r in y:
            xc[rank_pos[r - 1]] = rank_tok[r - 1]
        alone = O.block_decode_step(m, cache, xc, T, s, e, [()], [], [], False, faithful=False, return_logits=True)[2]
        assert np.allclose(lg4[r_copy == c], alone, rtol=1e-10, atol=1e-12)
    assert np.abs(lg4[r_copy == 1] - lg4[r_copy == 0]).max() > 1e-6   # the fill does matter inside its copy


def test_stage2_layout_and_values(small_model):
    """Decoded-share: a speculative copy computes only the still-masked positions and reads the
    decoded positions' K/V from copy 0.  Checked against a run that feeds copy 0's K/V of the
    decoded rows in as extra *context* keys."""
    m = small_model
    x = synth.sequence(7, 0, 8, 8, SMALL).astype(np.int64)
    T, s, e = 16, 8, 16
    cache, conf, tok = O.refresh_prefill(m, x, T, s, faithful=False)
    for p in (8, 10, 11, 13, 15):
        x[p] = tok[p - s]
    rank_pos, rank_tok = [9, 12, 14], [int(tok[1]), int(tok[4]), int(tok[6])]
    subsets = O.copy_subsets(3, 8, True)
    assert subsets == [(), (1,), (2,), (1, 2), (3,), (1, 2, 3)]
    r_copy, r_pos, r_tok = O.build_rows(x, s, e, SMALL.mask_id, subsets, rank_pos, rank_tok, True)
    assert (r_copy == 0).sum() == 8 and all((r_copy == c).sum() == 3 for c in range(1, 6))
    assert sorted(r_pos[r_copy == 3]) == [9, 12, 14]
    conf8, tok8, lg8, _, _ = O.block_decode_step(m, cache, x, T, s, e, subsets, rank_pos, rank_tok, True,
                                                 faithful=False, return_logits=True)
    assert (conf8[1:, [0, 2, 3, 5, 7]] == -1).all() and (conf8[0] > 0).all() and (conf8[1:, [1, 4, 6]] > 0).all()
    # copy 0 alone
    ctx = np.r_[0:s, e:T]
    vis0 = np.ones((8, len(ctx) + 8), dtype=bool)
    lg0, k0, v0 = O.forward_rows(m, x[s:e], np.arange(s, e), [k[ctx] for k in cache.k], [v[ctx] for v in cache.v],
                                 vis0, faithful=False)
    assert np.allclose(lg8[r_copy == 0], lg0, rtol=1e-10, atol=1e-12)
    dec = np.array([0, 2, 3, 5, 7])
    for c, y in enumerate(subsets[1:], start=1):
        fills = {rank_pos[r - 1]: rank_tok[r - 1] for r in y}
        toks = np.array([fills.get(p, SMALL.mask_id) for p in (9, 12, 14)])
        ck = [np.concatenate([k[ctx], k0[l][dec]]) for l, k in enumerate(cache.k)]
        cv = [np.concatenate([v[ctx], v0[l][dec]]) for l, v in enumerate(cache.v)]
        visc = np.ones((3, len(ctx) + 5 + 3), dtype=bool)
        lgc, _, _ = O.forward_rows(m, toks, np.array([9, 12, 14]), ck, cv, visc, faithful=False)
        assert np.allclose(lg8[r_copy == c], lgc, rtol=1e-10, atol=1e-12)
    # with nothing decoded the shared layout is the full computation
    x2 = synth.sequence(7, 0, 8, 8, SMALL).astype(np.int64)
    a = O.block_decode_step(m, cache, x2, T, s, e, O.copy_subsets(2, 4, False), [9, 12], rank_tok[:2], False,
                            faithful=False, return_logits=True)[2]
    b = O.block_decode_step(m, cache, x2, T, s, e, O.copy_subsets(2, 4, True)[:4], [9, 12], rank_tok[:2], True,
                            faithful=False, return_logits=True)[2]
    assert np.array_equal(a, b)


def test_zero_lm_head_gives_uniform_confidence(small_model):
    m = small_model
    import dataclasses
    mz = dataclasses.replace(m, lm_head=np.zeros_like(m.lm_head))
    x = synth.sequence(8, 0, 4, 4, SMALL)
    _, conf, tok = O.refresh_prefill(mz, x, 8, 4)
    assert (tok == 0).all() and np.allclose(conf, 1.0 / (SMALL.vocab - 1))


def test_faithful_mode_is_close_to_exact(tiny_model):
    x = synth.sequence(0, 0, 64, 64, synth.TINY)
    _, c0, t0, l0 = O.refresh_prefill(tiny_model, x, 128, 64, faithful=False, return_logits=True)
    _, c1, t1, l1 = O.refresh_prefill(tiny_model, x, 128, 64, faithful=True, return_logits=True)
    rms = np.sqrt((l0 * l0).mean())
    assert np.abs(l1 - l0).max() < 2e-2 * rms
    _, c2, t2, l2 = O.refresh_prefill(tiny_model, x, 128, 64, faithful=True, dtype=np.float32, return_logits=True)
    assert np.abs(l2 - l1).max() < 2e-2 * rms          # bf16 rounding flips only
