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
    sess.set_logit_dump(True)
    return E, om, gm, sess, x0


@requires_gpu
@pytest.mark.parametrize("shape_name", ["TINY", "TINY_PEAKY", "TINY_HD128"])
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
    tol = 4e-2 if shape_name == "TINY_PEAKY" else 2e-2
    ok, worst = logits_close(logits, ologits, tol)
    assert ok, worst
    # and against the PLAIN definition (float64, nothing rounded to bf16 anywhere): parity does not rest on the
    # oracle mode that rounds where the kernels round.  The benchmark spec's 2e-2 on the N(0, 0.02) models; the
    # sharp-logit model's own bf16 mode is already 1.2 - 1.4 x 2e-2 away from its plain definition
    # (tests/test_oracle_self_distance.py), hence 4e-2 there.
    _, pconf, ptok, plogits = O.refresh_prefill(om, x0, P + L, P, return_logits=True, faithful=False)
    ok_p, worst_p = logits_close(logits, plogits, tol)
    print(f"\n{shape_name}: logits vs the bf16-faithful oracle {worst:.2f} x, vs the plain float64 definition {worst_p:.2f} x "
          f"the bound of {tol:g}")
    assert ok_p, worst_p
    # decisions: same greedy token unless the oracle's own top-2 logit gap is below the logit error
    l32 = ologits.astype(np.float32).astype(np.float64)
    l32[:, shape.mask_id] = -np.inf
    top2 = np.sort(l32, axis=1)[:, -2:]
    gap = top2[:, 1] - top2[:, 0]
    err = np.abs(logits - ologits).max(axis=1)
    bad = (tok != otok) & (gap > 2 * err)
    assert not bad.any()
    assert np.allclose(conf, oconf, rtol=0.15 if shape_name == "TINY_PEAKY" else 2e-2)   # sharp logits: d(conf) ~ d(logit)
    # the fresh K/V of the last layer and the K/V cache rows agree with the oracle to one bf16 step
    k = bf16_bits_to_f64(sess.debug_read("k")).reshape(P + L, shape.n_heads, shape.head_dim)
    v = bf16_bits_to_f64(sess.debug_read("v")).reshape(P + L, shape.n_heads, shape.head_dim)
    for got, want in ((k, cache.k[-1]), (v, cache.v[-1])):
        ok, worst = logits_close(got.reshape(P + L, -1), want.reshape(P + L, -1), 4e-2)
        assert ok, worst
        assert (got == want).mean() > 0.7                # most elements land on the same bf16 value
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
def test_fused_lm_head_confidence_equals_logit_dump():
    """The product path never writes logits: the LM-head GEMM's epilogue reduces every vocabulary tile
    to (max, sum of exp, argmax).  Same state, both modes: identical greedy tokens, confidences equal to
    fp32 rounding of a differently ordered sum; the logits buffer is refused when not dumped."""
    from paper_2511_21759_b200 import binding as B
    for shape in (synth.TINY, synth.TINY_PEAKY):
        P, L = 64, 64
        E, om, gm, sess, x0 = _setup(shape, P, L)
        p = E.DecodeParams(block_len=16)
        sess.set_logit_dump(True)
        sess.refresh_prefill(p, 0)
        conf_d, tok_d = sess.debug_read("conf"), sess.debug_read("tok")
        sess.unmask_accept(p, True)
        sess.set_sequence(0, x0, P)
        sess.set_logit_dump(False)
        sess.refresh_prefill(p, 0)
        conf_f, tok_f = sess.debug_read("conf"), sess.debug_read("tok")
        with pytest.raises(B.OdbError) as e:
            sess.debug_read("logits")
        assert e.value.status == B.ODB_ERR_STATE
        assert np.array_equal(tok_d, tok_f)
        assert np.allclose(conf_d, conf_f, rtol=2e-6, atol=0)
        sess.close(); gm.close()
