"""Refresh prefill and block decode step of the CUDA path against the oracle, element by element."""
import dataclasses

import numpy as np
import pytest

import synth
from oracle import odb_oracle as O
from oracle.inputs import model_from_synth
from gpu_common import engine, requires_gpu, logits_close, bf16_bits_to_f64


def _setup(shape, P, L, *, max_copies=8, seed=0, with_lm_head=True, block=16):
    E = engine()
    om = model_from_synth(shape, seed=seed, with_lm_head=with_lm_head)
    gm = E.Model.from_synth(shape, seed=seed, with_lm_head=with_lm_head, max_batch=1, max_seq=P + L,
                            max_block=block, max_copies=max_copies)
    sess = E.Session(gm)
    x0 = synth.sequence(seed, 0, P, L, shape)
    sess.set_sequence(0, x0, P)
    return E, om, gm, sess, x0


@requires_gpu
@pytest.mark.parametrize("shape_name", ["TINY", "TINY_PEAKY"])
def test_refresh_logits_conf_tok(shape_name):
    shape = getattr(synth, shape_name)
    P, L = 64, 64
    E, om, gm, sess, x0 = _setup(shape, P, L)
    p = E.DecodeParams(block_len=16)
    sess.refresh_prefill(p, 0)
    logits = sess.debug_read("logits")
    conf, tok = sess.debug_read("conf"), sess.debug_read("tok")
    cache, oconf, otok, ologits = O.refresh_prefill(om, x0, P + L, P, return_logits=True)
    assert logits.shape == ologits.shape == (L, shape.vocab)
    ok, worst = logits_close(logits, ologits)
    assert ok, worst
    assert worst < 0.5                                   # in practice far inside the 2e-2 bound
    # decisions: same greedy token unless the oracle's own top-2 logit gap is below the logit error
    l32 = ologits.astype(np.float32).astype(np.float64)
    l32[:, shape.mask_id] = -np.inf
    top2 = np.sort(l32, axis=1)[:, -2:]
    gap = top2[:, 1] - top2[:, 0]
    err = np.abs(logits - ologits).max(axis=1)
    bad = (tok != otok) & (gap > 2 * err)
    assert not bad.any()
    assert np.allclose(conf, oconf, rtol=2e-2)
    # the fresh K/V of the last layer and the K/V cache rows agree with the oracle to one bf16 step
    k = bf16_bits_to_f64(sess.debug_read("k")).reshape(P + L, shape.n_heads, shape.head_dim)
    v = bf16_bits_to_f64(sess.debug_read("v")).reshape(P + L, shape.n_heads, shape.head_dim)
    for got, want in ((k, cache.k[-1]), (v, cache.v[-1])):
        d = np.abs(got - want)
        assert (d <= 2.0 ** -7 * np.maximum(np.abs(want), 1e-2)).all()
        assert (d == 0).mean() > 0.9
    sess.close(); gm.close()


@requires_gpu
def test_one_layer_intermediates():
    """One-layer model without LM head: K/V are exact functions of the embedding, so they must
    match the oracle bit for bit except where fp32-vs-fp64 accumulation flips a bf16 rounding."""
    shape = synth.TINY.with_layers(1)
    P, L = 40, 24
    E, om, gm, sess, x0 = _setup(shape, P, L, with_lm_head=False)
    sess.refresh_prefill(E.DecodeParams(block_len=16), 0)
    hid, fk, fv = O.forward_rows(om, x0.astype(np.int64), np.arange(P + L), None, None,
                                 np.ones((P + L, P + L), bool), return_hidden=True)
    k = bf16_bits_to_f64(sess.debug_read("k")).reshape(P + L, 4, 64)
    v = bf16_bits_to_f64(sess.debug_read("v")).reshape(P + L, 4, 64)
    assert (k == fk[0]).mean() > 0.99 and (v == fv[0]).mean() > 0.99
    assert np.abs(k - fk[0]).max() <= 2.0 ** -7 * np.abs(fk[0]).max()
    h = sess.debug_read("hidden")
    assert np.abs(h - hid).max() <= 2e-2 * np.sqrt((hid * hid).mean())
    sess.close(); gm.close()


@requires_gpu
@pytest.mark.parametrize("shape_name,n_copies", [("TINY", 1), ("TINY", 4), ("TINY_PEAKY", 4), ("TINY_PEAKY", 8)])
def test_step_matches_oracle(shape_name, n_copies):
    """refresh -> accept -> step on both sides; the step's rows, logits, conf and tok per copy."""
    shape = getattr(synth, shape_name)
    P, L, Bk = 64, 64, 16
    E, om, gm, sess, x0 = _setup(shape, P, L)
    gp = E.DecodeParams(block_len=Bk, n_copies=n_copies, stage2_min_decoded=2)
    op = O.DecodeParams(block_len=Bk, n_copies=n_copies, stage2_min_decoded=2)
    sess.refresh_prefill(gp, 0)
    res = sess.unmask_accept(gp, True)
    # oracle side, by hand
    x = x0.astype(np.int64).copy()
    cache, conf_r, tok_r = O.refresh_prefill(om, x, P + L, P)
    masked = x[P:P + Bk] == shape.mask_id
    acc = O.accept_set(conf_r[:Bk], masked, 0.9)
    for i in np.flatnonzero(acc):
        x[P + i] = tok_r[i]
    got_acc = sorted((res[0].accepted_pos[j], res[0].accepted_tok[j]) for j in range(res[0].n_accepted))
    assert got_acc == [(int(P + i), int(tok_r[i])) for i in np.flatnonzero(acc)]
    for _ in range(3):                                   # three consecutive steps
        masked = x[P:P + Bk] == shape.mask_id
        if not masked.any():
            break
        k_ranks = {1: 0, 4: 2, 8: 4}[n_copies]
        last_conf, last_tok = (conf_r[:Bk], tok_r[:Bk]) if _ == 0 else (conf[last], tok[last])
        ranks = O.rank_candidates(last_conf, masked, k_ranks)
        rank_tok = [int(last_tok[i]) for i in ranks]
        st2 = O.use_stage2(op, Bk, int((~masked).sum()))
        subsets = O.copy_subsets(len(ranks), 4 if (n_copies == 8 and not st2) else n_copies, st2)
        conf, tok, lg, r_copy, r_pos = O.block_decode_step(om, cache, x, P + L, P, P + Bk, subsets,
                                                           [P + i for i in ranks], rank_tok, st2, return_logits=True)
        sess.block_decode_step(gp)
        assert (sess.debug_read("row_pos") == r_pos).all() and (sess.debug_read("row_copy") == r_copy).all()
        glog = sess.debug_read("logits")
        ok, worst = logits_close(glog, lg)
        assert ok, worst
        gconf = sess.debug_read("conf")
        assert np.allclose(gconf, conf[r_copy, r_pos - P], rtol=2e-2)
        res = sess.unmask_accept(gp, False)
        new, chain, last = O.jump_walk(conf, tok, masked, subsets, ranks, rank_tok, 0.9)
        margin = min(O.decision_margin(conf[c], masked & (conf[c] >= 0), 0.9, k_ranks + 1) for c in chain)
        got = sorted((res[0].accepted_pos[j] - P, res[0].accepted_tok[j]) for j in range(res[0].n_accepted))
        if margin > 1e-3:
            assert got == sorted(new.items()) and [res[0].chain[j] for j in range(res[0].chain_len)] == chain
        for i, t in new.items():
            x[P + i] = t
        if got != sorted(new.items()):
            break                                        # near-tie: the two sides are on different paths now
    sess.close(); gm.close()
