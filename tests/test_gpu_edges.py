"""Edge cases of the decoding iteration through the C ABI, each in lock step with the oracle: ragged
tails (response not a multiple of the block, prompt not a multiple of any tile), the degenerate
shapes (no prompt, a one-position block, a one-position response), and the largest sizes the
library accepts (block 64 with 8 copies = 512 query rows; a 2048-position sequence)."""
import numpy as np
import pytest

import synth
from oracle import odb_oracle as O
from oracle.inputs import model_from_synth
from gpu_common import engine, requires_gpu, lockstep_generate, assert_near_ties_only

CASES = [
    # name              shape        P    L   block copies  max_iters
    ("ragged_tail",     "TINY",      37,  41, 16,   4,      None),   # last block has 9 positions; odd prompt
    ("ragged_peaky_c8", "TINY_PEAKY", 51, 45, 16,   8,      None),   # last block 13, stage-2 copies on a short block
    ("no_prompt",       "TINY",      0,   32, 16,   4,      None),   # the first refresh has no prefix at all
    ("block_of_one",    "TINY",      20,  5,  1,    1,      None),   # every iteration is a refresh
    ("response_of_one", "TINY",      33,  1,  16,   4,      None),   # one masked position in total
    ("block_3_c4",      "TINY_PEAKY", 17, 10, 3,    4,      None),   # fewer masked positions than candidate ranks
    ("block64_c8",      "TINY_PEAKY", 64, 128, 64,  8,      None),   # 512 query rows per step: the largest step
    ("long_2048",       "TINY",      1984, 64, 32,  4,      12),     # the longest sequence: 16 key splits in the step
    # head dim 128: the refresh attention runs on the tcgen05 tensor cores (128-row work items, 64-key tiles)
    ("hd128_ragged",    "TINY_HD128", 150, 77, 16,  4,      None),   # T = 227: second row tile 99 rows, last key tile 35 keys
    ("hd128_one_tile",  "TINY_HD128", 20,  30, 16,  1,      None),   # T = 50: a single ragged row tile and key tile
    ("hd128_long",      "TINY_HD128", 1000, 64, 32, 8,      6),      # T = 1064: 9 row tiles x 17 key tiles
    # decode steps with several copies on the tensor cores: cached key tiles for all rows, one fresh tile per copy
    ("hd128_c8_stage2", "TINY_HD128", 40,  48, 16,  8,      None),   # runs into the decoded-share layout in every block
    ("hd128_b64_c8",    "TINY_HD128", 70,  128, 64, 8,      None),   # 512 rows per step: several 128-row work items
    ("hd128_c4_noprompt", "TINY_HD128", 0, 64, 32,  4,      None),   # first block: no cached key at all (empty key splits)
]


@requires_gpu
@pytest.mark.parametrize("name,shape_name,P,L,Bk,copies,max_iters", CASES, ids=[c[0] for c in CASES])
def test_edge_case_in_lockstep(name, shape_name, P, L, Bk, copies, max_iters):
    E = engine()
    shape = getattr(synth, shape_name)
    om = model_from_synth(shape, seed=3)
    gm = E.Model.from_synth(shape, seed=3, max_batch=1, max_seq=P + L, max_block=Bk, max_copies=8)
    sess = E.Session(gm)
    x0 = synth.sequence(3, 0, P, L, shape)
    sess.set_sequence(0, x0, P)
    kw = dict(block_len=Bk, n_copies=copies)
    tol = 4e-2 if shape_name == "TINY_PEAKY" else 2e-2
    st = lockstep_generate(E, sess, om, x0, P, E.DecodeParams(**kw), O.DecodeParams(**kw), tol=tol,
                           max_iters=max_iters)
    assert sess.status() == 0
    assert_near_ties_only(st)
    if max_iters is None:
        assert np.array_equal(sess.get_tokens(0), st["tokens_final"])
        assert (st["tokens_final"][P:] != shape.mask_id).all() and st["tokens"] == L
        assert st["refreshes"] == -(-L // Bk)
    else:
        assert st["iters"] == max_iters and st["tokens"] >= max_iters
    print(f"\n{name}: {st['iters']} iterations ({st['refreshes']} refreshes), worst logit {st['worst_logit']:.2f} x bound, "
          f"oracle-side decision diffs {st['oracle_decision_diff']}")
    sess.close(); gm.close()


@requires_gpu
def test_step_attention_alternatives_for_head_dim_128():
    """Multi-copy decode steps with head dim 128 run on the tensor-core attention with key splits.  The two other
    configurations of that step are selected through environment variables read once per process, so the cases run
    in child processes: the tensor-core kernel without key splits (one CTA per work item over cached and fresh keys,
    final output: what batched steps with a work item for every CTA slot use), and the mma.sync multi-copy kernel
    (the path of head dim 64, here at head dim 128)."""
    import os, subprocess, sys
    engine()
    names = ["hd128_ragged", "hd128_c8_stage2", "hd128_b64_c8", "hd128_c4_noprompt"]
    code = ("import sys; sys.path.insert(0, 'tests'); import test_gpu_edges as t\n"
            f"for c in t.CASES:\n    if c[0] in {names!r}: t.test_edge_case_in_lockstep(*c)\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    for extra in ({"ODB_ATTN_KS": "1"}, {"ODB_ATTN_TC_STEP_MIN": "1000000"}):
        env = dict(os.environ, **extra)
        r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=900)
        assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
        assert r.stdout.count("iterations") == len(names), r.stdout[-2000:]


@requires_gpu
def test_fully_decoded_block_is_a_state_error_not_a_launch():
    """A step on a block with no masked position left has no rows: the call reports the state error
    and launches nothing (the degenerate empty input)."""
    E = engine()
    shape = synth.TINY
    gm = E.Model.from_synth(shape, seed=0, max_batch=1, max_seq=24, max_block=1, max_copies=1)
    sess = E.Session(gm)
    sess.set_sequence(0, synth.sequence(0, 0, 20, 4, shape), 20)
    gp = E.DecodeParams(block_len=1, n_copies=1)
    sess.refresh_prefill(gp, 0)
    res = sess.unmask_accept(gp, True)[0]
    assert res.n_accepted == 1 and res.masks_left == 0        # top-1 fallback filled the only position
    from paper_2511_21759_b200 import binding as B
    with pytest.raises(B.OdbError) as err:
        sess.block_decode_step(gp)
    assert err.value.status == B.ODB_ERR_STATE
    assert sess.status() == 0
    sess.refresh_prefill(gp, 1)                                # the session is still usable
    assert sess.unmask_accept(gp, True)[0].n_accepted == 1
    sess.close(); gm.close()


@requires_gpu
def test_an_expired_device_wait_is_reported_and_the_session_stays_usable():
    """Every device-side wait of the library is the same bounded wait.  Here one runs out by design (a barrier
    nothing arrives at, limit about a millisecond): the kernel returns normally, the status word carries the
    timeout to the host (through odb_session_status, or through the next accept), is cleared by the read, and
    the session goes on working.  Nothing faults or hangs."""
    import ctypes as C
    E = engine()
    from paper_2511_21759_b200 import binding as B
    shape = synth.TINY
    gm = E.Model.from_synth(shape, seed=0, max_batch=1, max_seq=48, max_block=16, max_copies=1)
    sess = E.Session(gm)
    sess.set_sequence(0, synth.sequence(0, 0, 16, 32, shape), 16)
    gp = E.DecodeParams(block_len=16, n_copies=1)
    lib = B.lib()
    assert lib.odb_debug_expire_wait(sess.handle, C.c_int64(0)) == B.ODB_ERR_ARG
    assert lib.odb_debug_expire_wait(sess.handle, C.c_int64(2_000_000)) == B.ODB_OK
    assert sess.status() == B.ODB_ERR_TIMEOUT
    assert sess.status() == 0                                   # reading clears it
    # reported by the accept that follows, whose own work is done all the same
    sess.refresh_prefill(gp, 0)
    assert lib.odb_debug_expire_wait(sess.handle, C.c_int64(2_000_000)) == B.ODB_OK
    with pytest.raises(B.OdbError) as err:
        sess.unmask_accept(gp, True)
    assert err.value.status == B.ODB_ERR_TIMEOUT
    assert sess.status() == 0
    sess.block_decode_step(gp)                                  # the accept had committed its token: the step has rows
    res = sess.unmask_accept(gp, False)[0]
    assert res.n_accepted >= 1 and res.masks_left <= 14
    # and by the device-resident loop, which stops after the iteration that saw it
    assert lib.odb_debug_expire_wait(sess.handle, C.c_int64(2_000_000)) == B.ODB_OK
    with pytest.raises(B.OdbError) as err:
        sess.decode_block_resident(gp)
    assert err.value.status == B.ODB_ERR_TIMEOUT
    assert sess.status() == 0
    log = sess.decode_block_resident(gp)
    assert log[-1][0].masks_left == 0
    sess.close(); gm.close()


@requires_gpu
@pytest.mark.parametrize("copies", [1, 4])
def test_resumed_session_continues_identically(copies):
    """Checkpoint / resume: the state of a sequence is its token ids (the K/V cache is recomputed by the next
    refresh).  A generation stopped at a block boundary, read out with get_tokens, handed to a NEW session with
    set_sequence and continued from the next block gives the same trace and the same final tokens as the
    uninterrupted generation."""
    E = engine()
    shape = synth.TINY_PEAKY
    P, L, Bk = 24, 48, 16
    gm = E.Model.from_synth(shape, seed=3, max_batch=1, max_seq=P + L, max_block=Bk, max_copies=4)
    gp = E.DecodeParams(block_len=Bk, n_copies=copies, alp=False)
    x0 = synth.sequence(3, 0, P, L, shape)
    s0 = E.Session(gm)
    s0.set_sequence(0, x0, P)
    full_tok, full_trace = E.generate(s0, gp)
    s0.close()
    # the iteration that closes block 0 of the uninterrupted run
    n0 = next(i for i, t in enumerate(full_trace) if t["seqs"][0]["masks_left"] == 0) + 1
    assert 0 < n0 < len(full_trace)
    s1 = E.Session(gm)
    s1.set_sequence(0, x0, P)
    _, head = E.generate(s1, gp, max_iters=n0)
    saved = s1.get_tokens(0)
    s1.close()
    assert head == full_trace[:n0]
    assert (saved[P:P + Bk] != shape.mask_id).all() and (saved[P + Bk:] == shape.mask_id).all()
    s2 = E.Session(gm)                               # nothing of the first session survives but the ids
    s2.set_sequence(0, saved, P)
    tok, tail = E.generate(s2, gp, start_block=1)
    assert s2.status() == 0
    s2.close(); gm.close()
    assert tail == full_trace[n0:]
    assert np.array_equal(tok[0], full_tok[0])


@requires_gpu
@pytest.mark.parametrize("shape_name,copies", [("TINY_PEAKY", 1), ("TINY_PEAKY", 8), ("TINY_HD128", 4)])
def test_poisoned_workspace_reads_nothing_unwritten(shape_name, copies):
    """The caller's workspace and K/V cache arrive filled with NaN patterns (0xFF bytes): the library initialises
    what it needs at session creation and every kernel reads only what an earlier kernel of the same call chain
    wrote.  A whole ragged generation in lock step (logits compared element by element) would turn any read of
    unwritten memory into NaN."""
    E = engine()
    shape = getattr(synth, shape_name)
    P, L, Bk = 37, 41, 16
    om = model_from_synth(shape, seed=6)
    gm = E.Model.from_synth(shape, seed=6, max_batch=2, max_seq=P + L + 11, max_block=Bk, max_copies=8)
    sess = E.Session(gm, poison=True)
    x0 = synth.sequence(6, 0, P, L, shape)
    sess.set_sequence(0, x0, P)
    kw = dict(block_len=Bk, n_copies=copies)
    st = lockstep_generate(E, sess, om, x0, P, E.DecodeParams(**kw), O.DecodeParams(**kw),
                           tol=4e-2 if shape_name == "TINY_PEAKY" else 2e-2)
    assert sess.status() == 0 and np.isfinite(st["worst_logit"]) and np.isfinite(st["worst_conf"])
    assert_near_ties_only(st)
    # the fused product path and the device-resident loop on the same poisoned buffers
    sess.set_sequence(0, x0, P)
    toks, trace = E.generate(sess, E.DecodeParams(**kw), resident=True)
    assert sess.status() == 0 and (toks[0][P:] != shape.mask_id).all()
    assert np.array_equal(toks[0], st["tokens_final"])
    sess.close(); gm.close()


@requires_gpu
def test_read_bandwidth_probes_are_sane_and_validate_their_arguments():
    """The two read-stream probes the benchmark quotes beside the copy bandwidth: both land between 3 and 9 TB/s on
    a buffer far larger than L2, the bulk-copy ring (the projections' weight path) is not slower than 90 % of the
    plain loads, and bad arguments are refused before any launch."""
    import ctypes as C
    import torch
    from paper_2511_21759_b200 import binding as B
    E = engine()
    ld = E.measure_read_bandwidth(1 << 30, 3)
    bulk = E.measure_read_bandwidth(1 << 30, 3, bulk=True)
    print(f"\nread probes: 16-byte loads {ld:.0f} GB/s, bulk-copy rings {bulk:.0f} GB/s")
    assert 3000 < ld < 9000 and 3000 < bulk < 9000
    assert bulk > 0.9 * ld
    buf = torch.empty(1 << 21, dtype=torch.uint8, device="cuda")
    out = C.c_double()
    for fn in (B.lib().odb_measure_read_bandwidth, B.lib().odb_measure_bulk_read_bandwidth):
        assert fn(buf.data_ptr() + 8, 1 << 20, 1, None, C.byref(out)) == B.ODB_ERR_ARG      # misaligned
        assert fn(buf.data_ptr(), 1 << 10, 1, None, C.byref(out)) == B.ODB_ERR_ARG          # too small
        assert fn(buf.data_ptr(), 1 << 20, 0, None, C.byref(out)) == B.ODB_ERR_ARG          # no passes
        assert fn(None, 1 << 20, 1, None, C.byref(out)) == B.ODB_ERR_ARG
