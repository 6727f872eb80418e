"""End-to-end generation through the C ABI against the oracle's generate loop.

Two regimes, tested apart:
  * separated workloads (tests/golden/separated_workloads.json): every decision of the oracle's own
    run is far from flipping, measured against the error of the kernels; token ids and the
    per-iteration accepted sets / jump chains must be IDENTICAL, free running, no exception;
  * random-weight workloads, where some decision is always closer than bf16 rounding noise: the
    first divergence, if any, must be a near-tie by the measured error at that very iteration
    (oracle margin <= max(1e-3, 4 x confidence error)); it is printed, and the test fails otherwise.
"""
import dataclasses
import json
import os

import numpy as np
import pytest

import synth
from oracle import odb_oracle as O
from oracle.inputs import model_from_synth
from gpu_common import engine, requires_gpu, compare_traces, lockstep_generate, assert_near_ties_only

with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "separated_workloads.json")) as _f:
    SEPARATED = json.load(_f)


def _run_both(wl_name, *, seed=0, schedule=None, params_kw=None, shape=None, x0=None, om=None, lm_head_bits=None,
              resident=False):
    E = engine()
    wl = synth.WORKLOADS[wl_name]
    shape = shape or wl.shape
    om = om or model_from_synth(shape, seed=seed)
    gm = E.Model.from_synth(shape, seed=seed, max_batch=1, max_seq=wl.prompt_len + wl.gen_len,
                            max_block=wl.block_len, max_copies=8, lm_head_bits=lm_head_bits)
    sess = E.Session(gm)
    x0 = x0 if x0 is not None else synth.sequence(seed, 0, wl.prompt_len, wl.gen_len, shape)
    sess.set_sequence(0, x0, wl.prompt_len)
    kw = dict(block_len=wl.block_len, n_copies=wl.n_copies, accept_threshold=wl.accept_threshold,
              truncate_threshold=wl.truncate_threshold)
    kw.update(params_kw or {})
    gsched = (lambda seq, b, L: schedule(b, L)) if schedule else None
    gtok, gtrace = E.generate(sess, E.DecodeParams(**kw), length_schedule=gsched, resident=resident)
    otok, otrace = O.generate(om, x0, wl.prompt_len, O.DecodeParams(**kw), length_schedule=schedule)
    assert sess.status() == 0
    # where the two runs part (if they do), the error is measured on that very state: the lock-step harness
    # replays the generation up to and including that iteration
    n, div = compare_traces(gtrace, otrace)
    measured = None
    if div is not None and div["gpu"] is not None:
        sess.set_sequence(0, x0, wl.prompt_len)
        # the replay takes the same kernels as the free run (LM head fused with the confidence reduction)
        st = lockstep_generate(E, sess, om, x0, wl.prompt_len, E.DecodeParams(**kw), O.DecodeParams(**kw),
                               schedule=schedule, tol=1.0, max_iters=div["iter"] + 1, check_logits=False)
        g, o = div["gpu"], div["oracle"]
        if [p_ for p_, _ in g["accepted"]] == [p_ for p_, _ in sorted(o["accepted"])] and g["chain"] == o["chain"]:
            # same positions, another greedy token: replayed once more with the logits materialised, which asserts
            # that every differing token sits on a top-2 logit gap below twice the logit error
            sess.set_sequence(0, x0, wl.prompt_len)
            st = lockstep_generate(E, sess, om, x0, wl.prompt_len, E.DecodeParams(**kw), O.DecodeParams(**kw),
                                   schedule=schedule, tol=1.0, max_iters=div["iter"] + 1)
        measured = st
    sess.close(); gm.close()
    return gtok[0], gtrace, otok, otrace, measured


def _assert_identical_or_near_tie(gtok, gtrace, otok, otrace, measured):
    """Passes when the free runs are identical, or when they part at a measured near-tie; fails otherwise."""
    n, div = compare_traces(gtrace, otrace)
    if div is None:
        assert np.array_equal(gtok, otok)
        print(f"\nfree run identical over {n} iterations")
        return
    assert measured is not None, f"traces differ in length after {n} equal iterations: {div}"
    g, o = div["gpu"], div["oracle"]
    if [p_ for p_, _ in g["accepted"]] == [p_ for p_, _ in sorted(o["accepted"])] and g["chain"] == o["chain"]:
        # same positions, another greedy token: the replay has already asserted that every differing token sits
        # on a top-2 logit gap below twice the logit error measured there
        print(f"\nfree runs part at iteration {div['iter']} after {n} identical ones on a greedy token whose top-2 "
              f"logit gap is below twice the measured logit error ({measured['tok_diff']} such rows): a near-tie")
        return
    ties = [t for t in measured["near_ties"] if t[0] == div["iter"]]
    assert ties, f"iteration {div['iter']}: the free runs part but the oracle decides like the kernels in lock step: {div}"
    assert_near_ties_only({"near_ties": ties})
    it, kind, margin, cerr = ties[0][:4]
    print(f"\nfree runs part at iteration {it} ({kind}) after {n} identical ones: oracle margin {margin:.2e}, "
          f"measured confidence error {cerr:.2e}: a near-tie")


def _separated(name):
    w = SEPARATED["workloads"][name]
    shape = dataclasses.replace(synth.TINY_PEAKY, w_std=w["w_std"], lm_std=w["lm_std"])
    x0 = synth.sequence(w["seed"], 0, w["prompt_len"], w["gen_len"], shape)
    kw = dict(block_len=w["block_len"], n_copies=w["n_copies"], accept_threshold=w["accept_threshold"], alp=False)
    return w, shape, x0, kw


@requires_gpu
@pytest.mark.parametrize("resident", [False, True])
@pytest.mark.parametrize("name", sorted(SEPARATED["workloads"]))
def test_free_run_identical_on_separated_workloads(name, resident):
    """Free-running generation (call by call, and through the device-resident loop) of a workload whose every
    decision is separated: final tokens and every iteration's accepted set and jump chain equal the stored
    oracle trace exactly.  There is no excuse path."""
    E = engine()
    w, shape, x0, kw = _separated(name)
    P = w["prompt_len"]
    gm = E.Model.from_synth(shape, seed=w["seed"], max_batch=1, max_seq=len(x0), max_block=w["block_len"], max_copies=8)
    sess = E.Session(gm)
    sess.set_sequence(0, x0, P)
    gtok, gtrace = E.generate(sess, E.DecodeParams(**kw), resident=resident)
    assert sess.status() == 0
    sess.close(); gm.close()
    assert len(gtrace) == len(w["trace"])
    for i, (g, o) in enumerate(zip(gtrace, w["trace"])):
        assert g["kind"] == o["kind"], i
        assert g["seqs"][0]["accepted"] == sorted(tuple(a) for a in o["accepted"]), (i, g["seqs"][0], o)
        assert g["seqs"][0]["chain"] == o["chain"], (i, g["seqs"][0], o)
    assert gtok[0].tolist() == w["tokens"]


@requires_gpu
@pytest.mark.parametrize("name", sorted(SEPARATED["workloads"]))
def test_separated_workloads_are_separated_by_the_measured_error(name):
    """Lock step on the same workloads: at every iteration the oracle's distance from flipping a decision is at
    least ten times the confidence error measured there (both in ln(c / (1 - c))), and every greedy token that
    is used has a top-2 logit gap of at least four times the largest logit error; the oracle never decides
    differently from the kernels."""
    E = engine()
    w, shape, x0, kw = _separated(name)
    P = w["prompt_len"]
    om = model_from_synth(shape, seed=w["seed"])
    gm = E.Model.from_synth(shape, seed=w["seed"], max_batch=1, max_seq=len(x0), max_block=w["block_len"], max_copies=8)
    sess = E.Session(gm)
    sess.set_sequence(0, x0, P)
    st = lockstep_generate(E, sess, om, x0, P, E.DecodeParams(**kw), O.DecodeParams(**kw), tol=4e-2)
    assert sess.status() == 0
    sess.close(); gm.close()
    assert st["oracle_decision_diff"] == 0 and st["tokens_final"].tolist() == w["tokens"]
    worst_c = min(e["sep"] / max(e["cl_err"], 1e-12) for e in st["log"])
    worst_t = min(e["tok_gap"] / max(e["logit_err"], 1e-12) for e in st["log"])
    print(f"\n{name}: {len(st['log'])} iterations; decision distance / confidence error >= {worst_c:.1f}, "
          f"top-2 gap / logit error >= {worst_t:.1f}")
    for i, (e, o) in enumerate(zip(st["log"], w["trace"])):
        assert e["sep"] == pytest.approx(o["sep"], rel=1e-6) and e["tok_gap"] == pytest.approx(o["tok_gap"], rel=1e-6), i
        assert e["sep"] >= 10 * e["cl_err"], (i, e)
        assert e["tok_gap"] >= 4 * e["logit_err"], (i, e)


@requires_gpu
@pytest.mark.parametrize("resident", [False, True])
@pytest.mark.parametrize("wl", ["cfg1_tiny", "cfg1_tiny_c4", "peaky_c1", "peaky_c4", "peaky_c8"])
def test_free_run_parts_only_at_a_measured_near_tie(wl, resident):
    """Random weights: the free runs are compared until they part; the iteration where they do is replayed in
    lock step, and the oracle's margin there must be within four times the confidence error measured there."""
    _assert_identical_or_near_tie(*_run_both(wl, resident=resident))


@requires_gpu
@pytest.mark.parametrize("copies", [1, 4, 8])
def test_resident_loop_equals_call_by_call(copies):
    """A ragged batch of three sequences, decoded call by call and through the device-resident loop: the
    traces (accepted sets, chains, masks left, block bounds, per iteration and sequence), the final tokens
    and the number of kernels launched are identical; the loop returns to the host once per change of the
    step's shape instead of once per iteration."""
    E = engine()
    shape = synth.TINY_PEAKY
    P, lens, Bk = 24, [48, 37, 16], 16
    gm = E.Model.from_synth(shape, seed=2, max_batch=3, max_seq=P + max(lens), max_block=Bk, max_copies=8)
    params = E.DecodeParams(block_len=Bk, n_copies=copies)
    runs = []
    for resident in (False, True):
        sess = E.Session(gm)
        for i, n in enumerate(lens):
            sess.set_sequence(i, synth.sequence(2, i, P, n, shape), P)
        calls = {"n": 0}
        inner = sess.decode_block_resident

        def counted(*a, _inner=inner, **k):
            calls["n"] += 1
            return _inner(*a, **k)
        sess.decode_block_resident = counted
        toks, trace = E.generate(sess, params, resident=resident)
        assert sess.status() == 0
        runs.append((toks, trace, sess.profile_read()[1], calls["n"]))
        sess.close()
    gm.close()
    (t0, tr0, l0, _), (t1, tr1, l1, n_loops) = runs
    assert tr0 == tr1
    for i in range(3):
        assert np.array_equal(t0[i], t1[i]) and (t0[i][P:] != shape.mask_id).all()
    steps = sum(t["kind"] == "step" for t in tr0)
    assert l0 == l1, (l0, l1)
    assert 0 < n_loops < steps or steps <= 1
    print(f"\n{copies} copies: {steps} step iterations in {n_loops} loop launches")


@requires_gpu
def test_resident_loop_respects_max_iters_and_state():
    E = engine()
    from paper_2511_21759_b200 import binding as B
    shape = synth.TINY
    P, L, Bk = 20, 32, 16
    gm = E.Model.from_synth(shape, seed=1, max_batch=1, max_seq=P + L, max_block=Bk, max_copies=4)
    sess = E.Session(gm)
    sess.set_sequence(0, synth.sequence(1, 0, P, L, shape), P)
    gp = E.DecodeParams(block_len=Bk, n_copies=1, accept_threshold=1.0)     # one token per iteration: 15 steps per block
    with pytest.raises(B.OdbError) as err:                                  # nothing refreshed yet
        sess.decode_block_resident(gp)
    assert err.value.status == B.ODB_ERR_STATE
    sess.refresh_prefill(gp, 0)
    assert sess.unmask_accept(gp, True)[0].masks_left == 15
    log = sess.decode_block_resident(gp, 4)
    assert len(log) == 4 and [it[0].masks_left for it in log] == [14, 13, 12, 11]
    log = sess.decode_block_resident(gp)                                     # runs the block to its end
    assert len(log) == 11 and log[-1][0].masks_left == 0
    with pytest.raises(B.OdbError) as err:                                  # the block is closed: no rows
        sess.decode_block_resident(gp)
    assert err.value.status == B.ODB_ERR_STATE
    sess.refresh_prefill(gp, 1)                                             # the session goes on normally
    assert sess.unmask_accept(gp, True)[0].masks_left == 15
    sess.block_decode_step(gp)                                              # mixing with the single calls
    assert sess.unmask_accept(gp, False)[0].masks_left == 14
    log = sess.decode_block_resident(gp)
    assert len(log) == 14 and log[-1][0].masks_left == 0
    assert sess.status() == 0
    sess.close(); gm.close()


@requires_gpu
@pytest.mark.parametrize("wl_name,tol,fused", [("cfg1_tiny", 2e-2, False), ("cfg1_tiny_c4", 2e-2, False),
                                               ("peaky_c1", 4e-2, False), ("peaky_c4", 4e-2, False),
                                               ("peaky_c8", 4e-2, False), ("cfg1_tiny_c4", 2e-2, True),
                                               ("peaky_c8", 4e-2, True)])
def test_lockstep_generate(wl_name, tol, fused):
    """Whole generation in lock step: numerics every iteration, control bit-exact on the GPU's own
    confidences, oracle-side decisions equal except at measured near-ties.  The sharp-logit model
    amplifies bf16 rounding (the oracle's own fp32 and fp64 runs differ by 0.8 of the 2e-2 bound
    there), hence its wider logit tolerance."""
    E = engine()
    wl = synth.WORKLOADS[wl_name]
    om = model_from_synth(wl.shape, seed=0)
    gm = E.Model.from_synth(wl.shape, seed=0, max_batch=1, max_seq=wl.prompt_len + wl.gen_len,
                            max_block=wl.block_len, max_copies=8)
    sess = E.Session(gm)
    x0 = synth.sequence(0, 0, wl.prompt_len, wl.gen_len, wl.shape)
    sess.set_sequence(0, x0, wl.prompt_len)
    kw = dict(block_len=wl.block_len, n_copies=wl.n_copies)
    # fused: the product path (LM head fused with the confidence reduction, no logits); otherwise the
    # test mode that also materialises the logits for the element-wise comparison
    st = lockstep_generate(E, sess, om, x0, wl.prompt_len, E.DecodeParams(**kw), O.DecodeParams(**kw), tol=tol,
                           check_logits=not fused)
    assert sess.status() == 0
    assert np.array_equal(sess.get_tokens(0), st["tokens_final"])
    assert (st["tokens_final"][wl.prompt_len:] != wl.shape.mask_id).all() and st["tokens"] == wl.gen_len
    assert_near_ties_only(st)
    print(f"\n{wl_name}: {st['iters']} iterations ({st['refreshes']} refreshes), worst logit {st['worst_logit']:.2f} x bound, "
          f"worst conf rel err {st['worst_conf']:.2e}, oracle-side decision diffs {st['oracle_decision_diff']}")
    sess.close(); gm.close()


@requires_gpu
@pytest.mark.parametrize("mode", ["vanilla", "fast_dllm", "odb", "spec_vanilla", "accept_jump", "decoded_share"])
def test_baseline_modes_in_lockstep(mode):
    """The three systems the paper's tables compare, as settings of the same calls: the cache-less
    baseline (every iteration a refresh prefill, one token each), DualCache block decoding without
    speculation or length prediction, and the full method; and the three speculation variants of the
    ablation (Section 5.3): one picked block, the jump chain over four copies, eight copies."""
    E = engine()
    shape = synth.TINY_PEAKY
    P, L, Bk = 40, 24, 8
    om = model_from_synth(shape, seed=2)
    gm = E.Model.from_synth(shape, seed=2, max_batch=1, max_seq=P + L, max_block=Bk, max_copies=8)
    sess = E.Session(gm)
    x0 = synth.sequence(2, 0, P, L, shape)
    sess.set_sequence(0, x0, P)
    gp, cache_g = E.mode_settings(mode, Bk)
    op, cache_o = O.mode_settings(mode, Bk)
    assert cache_g == cache_o and dataclasses.asdict(op) == {k: getattr(gp, k) for k in dataclasses.asdict(op)}
    st = lockstep_generate(E, sess, om, x0, P, gp, op, tol=4e-2, cache_blocks=cache_g)
    assert sess.status() == 0
    assert_near_ties_only(st)
    assert np.array_equal(sess.get_tokens(0), st["tokens_final"])
    if mode == "vanilla":
        assert st["iters"] == st["refreshes"] == L and st["steps"] == 0
    else:
        assert st["refreshes"] == L // Bk and st["iters"] <= L
    sess.close(); gm.close()


@requires_gpu
def test_pick_best_speculation_counters_and_resident_loop():
    """The compared speculation: every step's chain is the one adopted copy, so Eff_NFE equals NFE
    (Section 5.3); the device-resident loop gives the same trace as the call-by-call path."""
    E = engine()
    wl = synth.WORKLOADS["peaky_c4"]
    gm = E.Model.from_synth(wl.shape, seed=0, max_batch=1, max_seq=wl.prompt_len + wl.gen_len, max_block=wl.block_len,
                            max_copies=4)
    gp, cache_blocks = E.mode_settings("spec_vanilla", wl.block_len)
    traces = []
    for resident in (False, True):
        sess = E.Session(gm)
        sess.set_sequence(0, synth.sequence(0, 0, wl.prompt_len, wl.gen_len, wl.shape), wl.prompt_len)
        toks, tr = E.generate(sess, gp, cache_blocks=cache_blocks, resident=resident)
        assert sess.status() == 0 and (toks[0][wl.prompt_len:] != wl.shape.mask_id).all()
        traces.append(tr)
        sess.close()
    gm.close()
    assert traces[0] == traces[1]
    c = E.trace_counters(traces[0])
    assert c["tokens"] == wl.gen_len and c["eff_nfe"] == c["nfe"]
    assert all(len(t["seqs"][0]["chain"]) == 1 for t in traces[0])
    assert any(t["seqs"][0]["chain"] != [0] for t in traces[0]), "no speculative block was ever adopted"


@requires_gpu
def test_trace_counters_match_the_oracle_definition():
    E = engine()
    wl = synth.WORKLOADS["peaky_c4"]
    gm = E.Model.from_synth(wl.shape, seed=0, max_batch=1, max_seq=wl.prompt_len + wl.gen_len, max_block=wl.block_len,
                            max_copies=8)
    sess = E.Session(gm)
    sess.set_sequence(0, synth.sequence(0, 0, wl.prompt_len, wl.gen_len, wl.shape), wl.prompt_len)
    gp, cache_blocks = E.mode_settings("odb", wl.block_len)
    _, gtrace = E.generate(sess, gp, cache_blocks=cache_blocks)
    c = E.trace_counters(gtrace)
    # the same counters from the oracle's function on the GPU's trace, re-shaped to the oracle's records
    as_oracle = [{"kind": t["kind"], "accepted": t["seqs"][0]["accepted"], "chain": t["seqs"][0]["chain"]} for t in gtrace]
    assert c == O.trace_counters(as_oracle)
    assert c["tokens"] == wl.gen_len and c["eff_nfe"] >= c["nfe"] and c["refreshes"] == wl.gen_len // wl.block_len
    sess.close(); gm.close()


@requires_gpu
def test_generate_with_length_schedule():
    sched = lambda b, L: {0: 40, 1: 24}.get(b)
    gtok, gtrace, otok, otrace, measured = _run_both("peaky_c4", schedule=sched)
    assert [r["seqs"][0]["gen_len"] for r in gtrace if r["kind"] == "refresh"][:2] == [40, 24]
    _assert_identical_or_near_tie(gtok, gtrace, otok, otrace, measured)


@requires_gpu
def test_generate_alp_truncates():
    """[EOS] direction planted in the LM head (as in the oracle's ALP pin); threshold 0."""
    E = engine()
    shape = dataclasses.replace(synth.TINY_PEAKY, vocab=64, mask_id=63, eos_id=62)
    om = model_from_synth(shape, seed=5)
    x0 = synth.sequence(5, 0, 32, 64, shape)
    hid, _, _ = O.forward_rows(om, x0.astype(np.int64), np.arange(96), None, None, np.ones((96, 96), bool),
                               return_hidden=True)
    n = O.bf16_round(O.rmsnorm(hid, om.final_gain, om.rms_eps))[32:]
    row = O.bf16_round(30.0 * (n[40] - n.mean(0)))
    lm = om.lm_head.copy()
    lm[shape.eos_id] = row
    om = dataclasses.replace(om, lm_head=lm)
    bits = synth.lm_head_bits(shape, 5)
    bits[shape.eos_id] = (row.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)   # row is bf16-exact
    wl = dataclasses.replace(synth.WORKLOADS["peaky_c1"], prompt_len=32, gen_len=64)
    synth.WORKLOADS["_alp"] = wl
    try:
        gtok, gtrace, otok, otrace, measured = _run_both("_alp", seed=5, shape=shape, x0=x0, om=om, lm_head_bits=bits,
                                                         params_kw=dict(truncate_threshold=0.0))
    finally:
        del synth.WORKLOADS["_alp"]
    assert otrace[0]["T"] < 96 and gtrace[0]["seqs"][0]["gen_len"] == otrace[0]["T"] - 32
    _assert_identical_or_near_tie(gtok, gtrace, otok, otrace, measured)


@requires_gpu
def test_ragged_batch_equals_independent_runs():
    """Three sequences of different prompt / response lengths in one session: each must come out
    exactly as when it runs alone (sequences never see each other)."""
    E = engine()
    shape = synth.TINY_PEAKY
    lens = [(64, 64), (40, 48), (17, 30)]
    gm = E.Model.from_synth(shape, seed=0, max_batch=3, max_seq=128, max_block=16, max_copies=4)
    params = E.DecodeParams(block_len=16, n_copies=4)
    xs = [synth.sequence(0, i, P, L, shape) for i, (P, L) in enumerate(lens)]
    sess = E.Session(gm)
    for i, (P, L) in enumerate(lens):
        sess.set_sequence(i, xs[i], P)
    together, _ = E.generate(sess, params)
    sess.close()
    for i, (P, L) in enumerate(lens):
        s1 = E.Session(gm)
        s1.set_sequence(0, xs[i], P)
        alone, _ = E.generate(s1, params)
        s1.close()
        assert np.array_equal(together[i], alone[0]), i
    om = model_from_synth(shape, seed=0)
    otok, otrace = O.generate(om, xs[2], 17, O.DecodeParams(block_len=16, n_copies=4))
    if min(t["margin"] for t in otrace) > 0.5:          # only when no decision of the oracle's run is close
        assert np.array_equal(together[2], otok)
    gm.close()


@requires_gpu
def test_argument_validation_and_state_errors():
    E = engine()
    from paper_2511_21759_b200 import binding as B
    shape = synth.TINY
    gm = E.Model.from_synth(shape, seed=0, max_batch=1, max_seq=64, max_block=16, max_copies=4)
    sess = E.Session(gm)
    p = E.DecodeParams(block_len=16)
    with pytest.raises(B.OdbError) as e:
        sess.block_decode_step(p)                        # no refresh yet
    assert e.value.status == B.ODB_ERR_STATE
    with pytest.raises(B.OdbError) as e:
        sess.set_sequence(0, synth.sequence(0, 0, 40, 40, shape), 40)   # longer than max_seq
    assert e.value.status == B.ODB_ERR_SHAPE
    sess.set_sequence(0, synth.sequence(0, 0, 32, 32, shape), 32)
    with pytest.raises(B.OdbError) as e:
        sess.refresh_prefill(E.DecodeParams(block_len=32), 0)          # block beyond max_block
    assert e.value.status == B.ODB_ERR_SHAPE
    sess.refresh_prefill(p, 0)
    with pytest.raises(B.OdbError) as e:
        sess.unmask_accept(E.DecodeParams(block_len=16, n_copies=8), True)   # more copies than configured
    assert e.value.status == B.ODB_ERR_SHAPE
    with pytest.raises(B.OdbError) as e:
        sess.set_gen_len(0, 40)                          # may not grow
    assert e.value.status == B.ODB_ERR_ARG
    sess.set_gen_len(0, 20)
    res = sess.unmask_accept(p, True)
    assert res[0].gen_len == 20 and res[0].block_end == 48
    assert len(sess.get_tokens(0)) == 52
    # the device-resident loop validates the same way, and refuses to run while launches are being timed
    import ctypes as C
    lib, log, n = B.lib(), (B.odb_result * 4)(), C.c_int32()
    pc = p.c()
    assert lib.odb_decode_block_resident(sess.handle, C.byref(pc), 0, log, 0, C.byref(n)) == B.ODB_ERR_ARG      # no room in the log
    assert lib.odb_decode_block_resident(sess.handle, C.byref(pc), 0, None, 4, C.byref(n)) == B.ODB_ERR_ARG
    bad = E.DecodeParams(block_len=16, n_copies=8).c()
    assert lib.odb_decode_block_resident(sess.handle, C.byref(bad), 0, log, 4, C.byref(n)) == B.ODB_ERR_SHAPE
    sess.profile(True)
    assert lib.odb_decode_block_resident(sess.handle, C.byref(pc), 0, log, 4, C.byref(n)) == B.ODB_ERR_STATE
    sess.profile(False)
    assert lib.odb_decode_block_resident(sess.handle, C.byref(pc), 0, log, 4, C.byref(n)) == B.ODB_OK
    assert 1 <= n.value <= 4 and log[n.value - 1].masks_left < res[0].masks_left      # log_cap bounds the iterations
    assert sess.status() == 0
    sess.close(); gm.close()


@requires_gpu
@pytest.mark.parametrize("shape_name", ["TINY", "TINY_PEAKY"])
def test_stochastic_reverse_step_in_lockstep_and_free_running(shape_name):
    """The stochastic unmasking of Section 2.1, Eq. 1 as the accept rule (odb_decode_params.sampling): which
    positions an iteration unmasks depends on the caller's uniform deviates alone, so the accepted POSITIONS of every
    iteration must equal the oracle's exactly; the tokens are the greedy tokens of that iteration's forward.  Lock
    step first, then the same generation free running, call by call and through the device-resident loop."""
    E = engine()
    from paper_2511_21759_b200 import binding as B
    shape = getattr(synth, shape_name)
    P, L, Bk, n = 40, 48, 16, 6
    om = model_from_synth(shape, seed=4)
    gm = E.Model.from_synth(shape, seed=4, max_batch=1, max_seq=P + L, max_block=Bk, max_copies=4)
    x0 = synth.sequence(4, 0, P, L, shape)
    noise = lambda b, k: synth.uniform(9, 1000 * b + k, Bk)
    kw = dict(block_len=Bk, n_copies=1, alp=False, sampling=True, sample_steps=n)
    sess = E.Session(gm)
    sess.set_sequence(0, x0, P)
    st = lockstep_generate(E, sess, om, x0, P, E.DecodeParams(**kw), O.DecodeParams(**kw), noise=noise,
                           tol=4e-2 if shape_name == "TINY_PEAKY" else 2e-2)
    assert sess.status() == 0 and st["tokens"] == L and st["refreshes"] == L // Bk and st["iters"] <= n * (L // Bk)
    assert st["iters"] > L // Bk                      # some block needed more than its refresh
    locked = st["tokens_final"]
    # the oracle's own free run: identical positions per iteration; tokens identical unless a greedy token sits on
    # a top-2 logit gap below the logit error (counted by the harness)
    otok, otrace = O.generate(om, x0, P, O.DecodeParams(**kw), noise=noise)
    runs = []
    for resident in (False, True):
        sess.set_sequence(0, x0, P)
        gtok, gtrace = E.generate(sess, E.DecodeParams(**kw), noise=lambda seq, b: np.stack([noise(b, k) for k in range(n)]),
                                  resident=resident)
        assert sess.status() == 0
        runs.append((gtok[0], gtrace))
        assert [[p_ for p_, _ in t["seqs"][0]["accepted"]] for t in gtrace] == [[p_ for p_, _ in t["accepted"]] for t in otrace]
    assert np.array_equal(runs[0][0], runs[1][0]) and runs[0][1] == runs[1][1]
    assert np.array_equal(runs[0][0], locked)
    if st["tok_diff"] == 0:
        assert np.array_equal(runs[0][0], otok)
    # only with one copy, and with a step count the schedule can hold
    sess.set_sequence(0, x0, P)
    sess.refresh_prefill(E.DecodeParams(**kw), 0)
    for bad in (dict(kw, n_copies=4), dict(kw, sample_steps=0), dict(kw, sample_steps=65)):
        with pytest.raises(B.OdbError) as err:
            sess.unmask_accept(E.DecodeParams(**bad), True)
        assert err.value.status == B.ODB_ERR_ARG
    sess.close(); gm.close()
