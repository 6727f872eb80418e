"""Tensor-parallel forward (weights divided over R ranks, partial sums and confidence statistics exchanged through
the projections' epilogues) against the oracle of the WHOLE model.  One GPU: all ranks of a group run in this
process on one stream, every forward issued segment by segment, so no kernel ever waits for a later launch; the
kernels, the stores into the other ranks' buffers, the flags and their sequence numbers are the ones a group of
R GPUs runs."""
import dataclasses

import numpy as np
import pytest

import synth
from oracle import odb_oracle as O
from oracle.inputs import model_from_synth
from gpu_common import engine, requires_gpu, lockstep_generate, assert_near_ties_only, logits_close, bf16_bits_to_f64

# shapes whose heads and FFN width divide over the ranks (d_ffn a multiple of 64 R)
TP_TINY = dataclasses.replace(synth.TINY, d_ffn=768)                       # 4 heads of 64: R = 2, 4
TP_PEAKY = dataclasses.replace(synth.TINY_PEAKY, d_ffn=768)
TP_HD128 = dataclasses.replace(synth.TINY_HD128, d_ffn=768)               # 2 heads of 128: R = 2
TP_WIDE = dataclasses.replace(synth.TINY, d_model=512, n_heads=8, d_ffn=1024)   # 8 heads: R = 8, two vocabulary tiles each
SHAPES = {"tiny": TP_TINY, "peaky": TP_PEAKY, "hd128": TP_HD128, "wide": TP_WIDE}

CASES = [
    # name          shape    R  P   L   block copies poison  conf bound
    ("r2_c1",       "tiny",  2, 64, 64, 16,   1,     False,  1e-2),
    ("r4_c4",       "tiny",  4, 37, 41, 16,   4,     True,   1e-2),    # ragged tail, odd prompt, NaN-filled buffers
    ("r2_peaky_c8", "peaky", 2, 51, 45, 16,   8,     False,  0.15),    # threshold accepts, jumps, decoded-share layout
    ("r2_hd128_c4", "hd128", 2, 150, 77, 16,  4,     False,  1e-2),    # tcgen05 refresh attention, one head per rank
    ("r8_c1",       "wide",  8, 40, 48, 16,   1,     False,  1e-2),
    ("r4_b64_c8",   "peaky", 4, 64, 128, 64,  8,     False,  0.15),    # 512 query rows per step: CTA-pair projections
]


def _group(E, shape, R, P, L, Bk, *, seed=3, poison=False):
    from paper_2511_21759_b200 import tp
    g = tp.TPGroupOneGPU(shape, seed, R, max_batch=1, max_seq=P + L, max_block=Bk, max_copies=8, poison=poison)
    x0 = synth.sequence(seed, 0, P, L, shape)
    g.set_sequence(0, x0, P)
    return g, x0


@requires_gpu
@pytest.mark.parametrize("name,shape_name,R,P,L,Bk,copies,poison,conf_bound", CASES, ids=[c[0] for c in CASES])
def test_tp_group_in_lockstep(name, shape_name, R, P, L, Bk, copies, poison, conf_bound):
    """Whole generation of the group in lock step with the oracle of the unsharded model: confidences within the
    bound every iteration, accept sets / chains / row tables bit-exact from the group's own confidences, the
    oracle's own decisions equal except at measured near-ties; every rank ends with the same tokens (the group
    object asserts rank-by-rank equality of confidences, tokens, row tables, results after every call)."""
    E = engine()
    shape = SHAPES[shape_name]
    om = model_from_synth(shape, seed=3)
    g, x0 = _group(E, shape, R, P, L, Bk, poison=poison)
    kw = dict(block_len=Bk, n_copies=copies)
    st = lockstep_generate(E, g, om, x0, P, E.DecodeParams(**kw), O.DecodeParams(**kw), check_logits=False)
    assert g.status() == [0] * R
    assert_near_ties_only(st)
    assert np.array_equal(g.get_tokens(0), st["tokens_final"])
    assert (st["tokens_final"][P:] != shape.mask_id).all() and st["tokens"] == L
    assert st["worst_conf"] < conf_bound, st["worst_conf"]
    print(f"\n{name}: {R} ranks, {st['iters']} iterations ({st['refreshes']} refreshes), worst conf rel err {st['worst_conf']:.2e}, "
          f"oracle-side decision diffs {st['oracle_decision_diff']}")
    g.close()


@requires_gpu
@pytest.mark.parametrize("shape_name,R", [("tiny", 2), ("tiny", 4), ("hd128", 2), ("wide", 8)])
def test_tp_refresh_shards_against_the_whole_model(shape_name, R):
    """After a refresh: every rank's K / V rows of the last layer are the oracle's columns of that rank's heads (to
    one bf16 step, most elements identical), the residual streams are bit-identical on all ranks, and the
    confidences / greedy tokens agree with the oracle as the single-GPU path's do."""
    E = engine()
    shape = SHAPES[shape_name]
    P, L = 64, 64
    om = model_from_synth(shape, seed=0)
    g, x0 = _group(E, shape, R, P, L, 16, seed=0)
    p = E.DecodeParams(block_len=16)
    g.refresh_prefill(p, 0)
    conf, tok = g.debug_read("conf"), g.debug_read("tok")          # asserts the ranks agree
    g.debug_read("hidden")
    cache, oconf, otok, ologits = O.refresh_prefill(om, x0, P + L, P, return_logits=True)
    hl = shape.n_heads // R
    for r, sess in enumerate(g.ranks):
        k = bf16_bits_to_f64(sess.debug_read("k")).reshape(P + L, hl, shape.head_dim)
        v = bf16_bits_to_f64(sess.debug_read("v")).reshape(P + L, hl, shape.head_dim)
        for got, want in ((k, cache.k[-1][:, r * hl:(r + 1) * hl]), (v, cache.v[-1][:, r * hl:(r + 1) * hl])):
            ok, worst = logits_close(got.reshape(P + L, -1), want.reshape(P + L, -1), 4e-2)
            assert ok, (r, worst)
            assert (got == want).mean() > 0.7
    assert np.allclose(conf, oconf, rtol=2e-2)
    l32 = ologits.astype(np.float32).astype(np.float64)
    l32[:, shape.mask_id] = -np.inf
    top2 = np.sort(l32, axis=1)[:, -2:]
    assert not ((tok != otok) & (top2[:, 1] - top2[:, 0] > 4e-2 * np.abs(l32[np.isfinite(l32)]).max())).any()
    g.close()


@requires_gpu
def test_tp_expired_flag_wait_is_reported_and_the_group_stays_usable():
    """A wait for a sequence number no rank has signalled runs into its (short) limit: the status word reports the
    timeout to the host, nothing faults, and the group decodes on afterwards."""
    from paper_2511_21759_b200 import binding as B
    E = engine()
    P, L = 32, 32
    g, x0 = _group(E, TP_TINY, 2, P, L, 16)
    p = E.DecodeParams(block_len=16)
    g.refresh_prefill(p, 0)
    g.unmask_accept(p, True)
    for kind in range(3):
        B.check(B.lib().odb_debug_tp_expire_wait(g.ranks[0].handle, kind, 2_000_000), "odb_debug_tp_expire_wait")
        assert g.ranks[0].status() == B.ODB_ERR_TIMEOUT
        assert g.ranks[0].status() == 0                            # read and cleared
    assert g.ranks[1].status() == 0
    g.block_decode_step(p)
    res = g.unmask_accept(p, False)
    assert res[0].n_accepted >= 1 and g.status() == [0, 0]
    g.close()


@requires_gpu
def test_tp_state_errors():
    """Unattached sessions, the logits test mode and the device-resident loop are refused; shard configurations the
    library cannot divide are refused at model creation."""
    import ctypes as C
    from paper_2511_21759_b200 import binding as B, tp
    E = engine()
    m = tp.model_shard_from_synth(TP_TINY, 0, 0, 2, max_batch=1, max_seq=64, max_block=16, max_copies=4)
    s = E.Session(m)
    s.set_sequence(0, synth.sequence(0, 0, 32, 32, TP_TINY), 32)
    p = E.DecodeParams(block_len=16)
    with pytest.raises(B.OdbError) as e:
        s.refresh_prefill(p, 0)
    assert e.value.status == B.ODB_ERR_STATE                      # not attached
    with pytest.raises(B.OdbError) as e:
        s.set_logit_dump(True)
    assert e.value.status == B.ODB_ERR_STATE
    assert B.lib().odb_debug_tp_segments(s.handle, 0, 99) == B.ODB_ERR_ARG
    assert B.lib().odb_debug_tp_expire_wait(s.handle, 0, 1000) == B.ODB_ERR_STATE
    s.close(); m.close()
    g, _ = _group(E, TP_TINY, 2, 32, 32, 16)
    g.refresh_prefill(p, 0)
    g.unmask_accept(p, True)
    with pytest.raises(B.OdbError) as e:
        g.ranks[0].decode_block_resident(p)
    assert e.value.status == B.ODB_ERR_STATE
    g.close()
    import torch
    assert B.lib().odb_tp_enable_peer_access(torch.cuda.current_device()) == B.ODB_OK      # itself: nothing to enable
    assert B.lib().odb_tp_enable_peer_access(torch.cuda.device_count()) == B.ODB_ERR_ARG   # no such device
    assert B.lib().odb_tp_enable_peer_access(-1) == B.ODB_ERR_ARG
    with pytest.raises(B.OdbError) as e:                          # 688 FFN features do not divide into 2 x 64
        tp.model_shard_from_synth(synth.TINY, 0, 0, 2, max_batch=1, max_seq=64, max_block=16, max_copies=4)
    assert e.value.status == B.ODB_ERR_SHAPE


@requires_gpu
@pytest.mark.parametrize("shape_name,R,copies", [("tiny", 2, 1), ("peaky", 4, 4), ("hd128", 2, 8)])
def test_tp_rank_alone_resident_loop_equals_call_by_call(shape_name, R, copies):
    """A tensor-parallel step inside the device-resident loop (its exchanges count their sequence numbers on the
    device, so the launches replay from a graph).  Ranks that wait for one another cannot share a GPU inside graphs,
    so ONE rank runs alone: attached to its own buffers, the absent ranks' flags raised locally, their partial sums
    zeros (zero-filled workspace).  The loop must reproduce the call-by-call run of the same rank bit for bit:
    tokens, every iteration's accept set and chain, and no wait may have expired."""
    from paper_2511_21759_b200 import tp
    E = engine()
    shape = SHAPES[shape_name]
    P, L, Bk = 48, 64, 16
    x0 = synth.sequence(5, 0, P, L, shape)
    p = E.DecodeParams(block_len=Bk, n_copies=copies)
    runs = []
    for resident in (False, True):
        gm = tp.model_shard_from_synth(shape, 5, R - 1, R, max_batch=1, max_seq=P + L, max_block=Bk, max_copies=8)
        sess = E.Session(gm, zero=True)
        tp.attach_alone(sess)
        sess.set_sequence(0, x0, P)
        toks, trace = E.generate(sess, p, resident=resident)
        assert sess.status() == 0
        runs.append((toks[0], trace))
        sess.close(); gm.close()
    assert np.array_equal(runs[0][0], runs[1][0])
    assert runs[0][1] == runs[1][1]
    assert (runs[0][0][P:] != shape.mask_id).all()


def _ipc_child(shared, offset, n, done):
    """Second process of the mapping test: opens the first process's buffer through the inter-process handle and
    writes a pattern through the mapping (no kernel of either process waits for the other)."""
    try:
        import torch
        from paper_2511_21759_b200 import tp
        view = tp.open_workspace(shared)
        view[offset:offset + n] = torch.arange(n, device=view.device, dtype=torch.int64).to(torch.uint8)
        torch.cuda.synchronize()
        done.put(("ok", int(view.data_ptr())))
    except Exception:                      # the parent reports it
        import traceback
        done.put(("error", traceback.format_exc()))


@requires_gpu
def test_tp_workspace_mapping_between_processes():
    """The multi-process attach maps a peer's workspace through torch's CUDA inter-process storage handles and
    addresses the peer's regions by offset.  Two processes on this one GPU: the second opens the first's buffer and
    stores a pattern at an offset; the first sees it at that offset of its own tensor.  (Only the mapping is exercised:
    ranks whose kernels wait for one another need a GPU each.)"""
    import types
    import torch
    import torch.multiprocessing as mp
    from paper_2511_21759_b200 import tp
    engine()
    ws = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    shared = tp.share_workspace(types.SimpleNamespace(ws=ws))
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    offset, n = 4096 + 256, 200
    p = ctx.Process(target=_ipc_child, args=(shared, offset, n, q))
    p.start()
    status, detail = q.get(timeout=90)
    p.join(timeout=60)
    assert status == "ok", detail
    assert p.exitcode == 0
    torch.cuda.synchronize()
    got = ws[offset:offset + n].cpu().numpy()
    assert np.array_equal(got, np.arange(n, dtype=np.uint8))
    assert int(ws[:offset].sum()) == 0 and int(ws[offset + n:].sum()) == 0


@requires_gpu
@pytest.mark.parametrize("R,copies", [(2, 4), (4, 8)])
def test_tp_ragged_batch_equals_independent_runs(R, copies):
    """Three sequences of different prompt / response lengths in one tensor-parallel group: each must come out exactly as
    when it runs alone through a group of the same size (sequences never see each other; the row tables, the
    attention work items and the exchanges cover all sequences of a forward at once).  Free-running engine.generate
    over the group object: refreshes of some sequences alternate with steps of the others."""
    from paper_2511_21759_b200 import tp
    E = engine()
    shape = TP_PEAKY
    lens = [(64, 64), (40, 48), (17, 30)]
    params = E.DecodeParams(block_len=16, n_copies=copies)
    xs = [synth.sequence(0, i, P, L, shape) for i, (P, L) in enumerate(lens)]
    g = tp.TPGroupOneGPU(shape, 0, R, max_batch=3, max_seq=128, max_block=16, max_copies=8)
    for i, (P, L) in enumerate(lens):
        g.set_sequence(i, xs[i], P)
    together, _ = E.generate(g, params)
    assert g.status() == [0] * R
    g.close()
    for i, (P, L) in enumerate(lens):
        g1 = tp.TPGroupOneGPU(shape, 0, R, max_batch=3, max_seq=128, max_block=16, max_copies=8)
        g1.set_sequence(0, xs[i], P)
        alone, _ = E.generate(g1, params)
        g1.close()
        assert np.array_equal(together[i], alone[0]), i
        assert (together[i][P:] != shape.mask_id).all()


@requires_gpu
def test_tp_group_with_the_stochastic_reverse_step():
    """The stochastic unmasking of Section 2.1, Eq. 1 as the accept rule under tensor parallelism: every rank gets the
    caller's uniform deviates, so all ranks unmask the same positions as the oracle in every iteration."""
    from paper_2511_21759_b200 import tp
    E = engine()
    shape, R = TP_TINY, 2
    P, L, Bk, n = 40, 48, 16, 6
    om = model_from_synth(shape, seed=4)
    x0 = synth.sequence(4, 0, P, L, shape)
    noise = lambda b, k: synth.uniform(9, 1000 * b + k, Bk)
    kw = dict(block_len=Bk, n_copies=1, alp=False, sampling=True, sample_steps=n)
    g = tp.TPGroupOneGPU(shape, 4, R, max_batch=1, max_seq=P + L, max_block=Bk, max_copies=4)
    g.set_sequence(0, x0, P)
    st = lockstep_generate(E, g, om, x0, P, E.DecodeParams(**kw), O.DecodeParams(**kw), noise=noise, check_logits=False)
    assert g.status() == [0] * R and st["tokens"] == L and st["refreshes"] == L // Bk
    _, otrace = O.generate(om, x0, P, O.DecodeParams(**kw), noise=noise)
    g.set_sequence(0, x0, P)
    gtok, gtrace = E.generate(g, E.DecodeParams(**kw), noise=lambda seq, b: np.stack([noise(b, k) for k in range(n)]))
    assert [[p_ for p_, _ in t["seqs"][0]["accepted"]] for t in gtrace] == [[p_ for p_, _ in t["accepted"]] for t in otrace]
    assert np.array_equal(gtok[0], st["tokens_final"])
    g.close()


@requires_gpu
def test_tp_one_layer_without_lm_head():
    """One-layer model without LM head over two ranks: each rank's K / V rows are exact functions of the embedding
    (bit-equal to the oracle's columns of its heads except where fp32-vs-fp64 accumulation flips a bf16 rounding),
    and the replicated residual stream after the last exchange matches the oracle's hidden state."""
    from paper_2511_21759_b200 import tp
    E = engine()
    shape = TP_TINY.with_layers(1)
    P, L, R = 40, 24, 2
    om = model_from_synth(shape, seed=0, with_lm_head=False)
    g = tp.TPGroupOneGPU(shape, 0, R, with_lm_head=False, max_batch=1, max_seq=P + L, max_block=16, max_copies=1)
    x0 = synth.sequence(0, 0, P, L, shape)
    g.set_sequence(0, x0, P)
    g.refresh_prefill(E.DecodeParams(block_len=16), 0)
    hid, fk, fv = O.forward_rows(om, x0.astype(np.int64), np.arange(P + L), None, None,
                                 np.ones((P + L, P + L), bool), return_hidden=True)
    hl = shape.n_heads // R
    for r, sess in enumerate(g.ranks):
        k = bf16_bits_to_f64(sess.debug_read("k")).reshape(P + L, hl, shape.head_dim)
        v = bf16_bits_to_f64(sess.debug_read("v")).reshape(P + L, hl, shape.head_dim)
        assert (k == fk[0][:, r * hl:(r + 1) * hl]).mean() > 0.99 and (v == fv[0][:, r * hl:(r + 1) * hl]).mean() > 0.99
    h = g.debug_read("hidden")                                   # asserts the ranks hold the same bits
    assert np.abs(h - hid).max() <= 2e-2 * np.sqrt((hid * hid).mean())
    assert g.status() == [0] * R
    g.close()
