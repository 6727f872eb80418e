"""Shared helpers of the GPU parity tests (no test functions here)."""
import numpy as np
import pytest
import torch

import synth
from oracle import odb_oracle as O
from oracle.inputs import model_from_synth

requires_gpu = pytest.mark.gpu


def engine():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2511_21759_b200 import engine as E
    return E


def logits_close(got, want, tol=2e-2):
    """|d| <= tol * max(|l_oracle|, rms(row)): 2e-2 relative, with the row's RMS as the floor
    that keeps the relative measure meaningful for logits near zero."""
    want = np.asarray(want, dtype=np.float64)
    rms = np.sqrt((want * want).mean(axis=-1, keepdims=True))
    bound = tol * np.maximum(np.abs(want), rms)
    err = np.abs(np.asarray(got, dtype=np.float64) - want)
    return bool((err <= bound).all()), float((err / bound).max())


def rel_l2(got, want):
    """Worst per-row relative L2 error: ||got - want|| / ||want|| over the last axis."""
    want = np.asarray(want, dtype=np.float64)
    d = np.asarray(got, dtype=np.float64) - want
    return float((np.sqrt((d * d).sum(-1)) / np.sqrt((want * want).sum(-1))).max())


def bf16_bits_to_f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def compare_traces(gpu_trace, oracle_trace, seq=0, near_tie=1e-3):
    """Walks both traces; returns (n_equal, divergence) where divergence is None or a dict with the
    iteration index, both records and the oracle's decision margin there."""
    n = min(len(gpu_trace), len(oracle_trace))
    for i in range(n):
        g = gpu_trace[i]["seqs"][seq]
        o = oracle_trace[i]
        same = (gpu_trace[i]["kind"] == o["kind"] and g["accepted"] == sorted(o["accepted"])
                and g["chain"] == o["chain"])
        if not same:
            return i, {"iter": i, "gpu": g, "oracle": o, "margin": o["margin"],
                       "near_tie": o["margin"] < near_tie}
    if len(gpu_trace) != len(oracle_trace):
        return n, {"iter": n, "gpu": None, "oracle": None, "margin": np.inf, "near_tie": False}
    return n, None


def lockstep_generate(E, sess, om, x0, P, gp, op, *, schedule=None, tol=2e-2, check_logits=True, max_iters=None,
                      seq=0, cache_blocks=True, dtype=np.float64, l2_tol=None, stop=None, noise=None):
    """Lock-step parity harness for one sequence.

    Every iteration both sides start from the same state.  (1) Numerics: the GPU's logits /
    confidences / greedy tokens are compared with the oracle's for that state.  (2) Control: the
    oracle's accept rule, jump walk, ranking and row-table code are run on the GPU's OWN fp32
    confidences and tokens and must reproduce the GPU's decision, chain and next row table bit
    for bit (same inputs, same precision => identical integers).  (3) Bit-exact tokens: the
    decision the oracle takes from ITS confidences is compared too; where it differs, the
    oracle's decision margin must be below the confidence error measured in that iteration (a
    near-tie); these are counted and returned, never hidden.  The GPU's decision then advances
    both sides.  cache_blocks=False runs the cache-less baseline (every iteration a refresh).
    noise(block, k) -> uniforms [block_len]: the deviates of the stochastic reverse step when op.sampling is set.
    dtype: the oracle's arithmetic (float32 for the 8B shape); l2_tol: also bound the worst per-row relative L2
    error of the logits; stop(stats) -> True ends the run after an iteration.  Returns a stats dict."""
    sess.set_logit_dump(check_logits)                   # logits are only materialised in the test mode
    shape_mask, eos = om.mask_id, om.eos_id
    Bk, tau = op.block_len, op.accept_threshold
    k_ranks = {1: 0, 4: 2, 8: 4}[op.n_copies]
    x = np.array(x0, dtype=np.int64)
    T = len(x)
    st = {"iters": 0, "refreshes": 0, "steps": 0, "tokens": 0, "oracle_decision_diff": 0, "near_ties": [],
          "worst_logit": 0.0, "worst_conf": 0.0, "tok_diff": 0, "log": [], "worst_l2": 0.0, "stage2_steps": 0, "tok_only_diff": 0}

    def record(kind, diag, rows, g_conf, o_conf, g_logits, o_logits):
        """Per iteration: the oracle's distance from flipping (walk_diagnostics) beside the errors measured on the
        rows at masked positions: |d conf_logit| and the largest |d logit|."""
        rows = np.flatnonzero(rows)
        e = {"kind": kind, **diag, "cl_err": 0.0, "logit_err": None}
        if len(rows):
            e["cl_err"] = float(np.abs(O.conf_logit(g_conf[rows].astype(np.float64)) - O.conf_logit(o_conf[rows].astype(np.float64))).max())
            if g_logits is not None:
                e["logit_err"] = float(np.abs(g_logits[rows] - o_logits[rows]).max())
        st["log"].append(e)

    def numerics(g_conf, g_tok, g_logits, o_conf, o_tok, o_logits):
        rel = np.abs(g_conf.astype(np.float64) - o_conf) / np.maximum(o_conf, 1e-30)
        st["worst_conf"] = max(st["worst_conf"], float(rel.max()))
        if g_logits is not None:
            ok, worst = logits_close(g_logits, o_logits, tol)
            st["worst_logit"] = max(st["worst_logit"], worst)
            l2 = rel_l2(g_logits, o_logits)
            st["worst_l2"] = max(st["worst_l2"], l2)
            assert ok, f"logits off by {worst:.2f} x bound at iteration {st['iters']} (per-row relative L2 error {l2:.3e})"
            if l2_tol is not None:
                assert l2 <= l2_tol, f"per-row relative L2 error {l2:.3e} at iteration {st['iters']}"
            l32 = o_logits.astype(np.float32).astype(np.float64)
            l32[:, shape_mask] = -np.inf
            top2 = np.partition(l32, -2, axis=1)[:, -2:]
            gap = np.abs(top2[:, 1] - top2[:, 0])
            err = np.abs(g_logits - o_logits).max(axis=1)
            diff = g_tok != o_tok
            assert not (diff & (gap > 2 * err)).any(), "greedy token differs beyond the logit error"
            st["tok_diff"] += int(diff.sum())
        return float(rel.max())

    def res_tuple(r):
        return (sorted((r.accepted_pos[j], r.accepted_tok[j]) for j in range(r.n_accepted)),
                [r.chain[j] for j in range(r.chain_len)])

    b = 0
    while True:
        s = P + b * Bk
        if s >= T or (max_iters is not None and st["iters"] >= max_iters):
            break
        if op.sampling:
            sess.set_sampling_noise(seq, np.stack([noise(b, k) for k in range(op.sample_steps)]))
        sess.refresh_prefill(gp, b)
        g_conf, g_tok = sess.debug_read("conf"), sess.debug_read("tok")
        g_logits = sess.debug_read("logits") if check_logits else None
        out = O.refresh_prefill(om, x, T, s, return_logits=True, dtype=dtype)
        cache, o_conf, o_tok, o_logits = out
        assert len(g_conf) == T - s
        cerr = numerics(g_conf, g_tok, g_logits, o_conf, o_tok, o_logits)
        newL = O.alp_scan(g_conf, g_tok, s, P, eos, op.truncate_threshold) if op.alp else None
        newL_o = O.alp_scan(o_conf, o_tok, s, P, eos, op.truncate_threshold) if op.alp else None
        if schedule is not None:
            cand = schedule(b, T - P)
            if cand is not None and s - P < cand < T - P:
                sess.set_gen_len(seq, cand)
                newL = cand if newL is None else min(newL, cand)
                newL_o = cand if newL_o is None else min(newL_o, cand)
        res = sess.unmask_accept(gp, True)[seq]
        if newL is not None and P + newL < T:
            T = P + newL
            x = x[:T]
        assert res.gen_len == T - P, (res.gen_len, T - P)
        e = min(s + Bk, T)
        B = e - s
        assert (res.block_start, res.block_end) == (s, e)
        masked = x[s:e] == shape_mask
        k_iter = 0
        unmask = (lambda c_, m_, k_: O.reverse_step_unmask(m_, noise(b, k_)[:B], k_, op.sample_steps)) if op.sampling else \
                 (lambda c_, m_, k_: O.accept_set(c_, m_, tau))
        acc = unmask(g_conf[:B], masked, 0)
        want = [(int(s + i), int(g_tok[i])) for i in np.flatnonzero(acc)]
        assert res_tuple(res) == (want, [0]), (res_tuple(res), want)
        acc_o = unmask(o_conf[:B], masked, 0)
        want_o = [(int(s + i), int(o_tok[i])) for i in np.flatnonzero(acc_o)]
        record("refresh", O.walk_diagnostics(o_conf[None, :B], O.top2_gap(o_logits[:B], shape_mask)[None, :], masked, [()], [], [0],
                                             {int(i): 0 for i in np.flatnonzero(acc_o)}, tau, k_ranks),
               masked, g_conf[:B], o_conf[:B], None if g_logits is None else g_logits[:B], o_logits[:B])
        if [p_ for p_, _ in want_o] != [p_ for p_, _ in want] or newL_o != newL:
            margin = O.decision_margin(o_conf[:B], masked, tau, 0)
            st["oracle_decision_diff"] += 1
            st["near_ties"].append((st["iters"], "refresh", margin, cerr, st["log"][-1]["tok_gap"], st["log"][-1]["logit_err"]))
        elif want_o != want:
            st["tok_only_diff"] += 1          # same positions, another greedy token (numerics() bounded its top-2 gap)
        for p_, t_ in want:
            x[p_] = t_
        st["iters"] += 1; st["refreshes"] += 1; st["tokens"] += len(want)
        assert res.masks_left == int((x[s:e] == shape_mask).sum())
        last_conf, last_tok = g_conf[:B], g_tok[:B]
        if not cache_blocks:                            # cache-less baseline: the next iteration is a refresh again
            if not (x[s:e] == shape_mask).any():
                b += 1
            continue
        while (x[s:e] == shape_mask).any():
            if max_iters is not None and st["iters"] >= max_iters:
                break
            masked = x[s:e] == shape_mask
            ranks = O.rank_candidates(last_conf, masked, k_ranks)
            rank_pos = [s + i for i in ranks]
            rank_tok = [int(last_tok[i]) for i in ranks]
            st2 = O.use_stage2(op, B, int((~masked).sum()))
            subsets = O.copy_subsets(len(ranks), 4 if (op.n_copies == 8 and not st2) else op.n_copies, st2)
            o_c, o_t, o_logits, r_copy, r_pos = O.block_decode_step(om, cache, x, T, s, e, subsets, rank_pos,
                                                                    rank_tok, st2, return_logits=True, dtype=dtype)
            st["stage2_steps"] += int(st2)
            _, _, r_tok = O.build_rows(x, s, e, shape_mask, subsets, rank_pos, rank_tok, st2)
            sess.block_decode_step(gp)
            assert np.array_equal(sess.debug_read("row_pos"), r_pos), "row positions"
            assert np.array_equal(sess.debug_read("row_copy"), r_copy), "row copies"
            assert np.array_equal(sess.debug_read("row_tok"), r_tok), "row tokens (ranking / fills)"
            g_cr, g_tr = sess.debug_read("conf"), sess.debug_read("tok")
            g_logits = sess.debug_read("logits") if check_logits else None
            cerr = numerics(g_cr, g_tr, g_logits, o_c[r_copy, r_pos - s], o_t[r_copy, r_pos - s], o_logits)
            C = len(subsets)
            g_c = np.full((C, B), -1.0, dtype=np.float32)
            g_t = np.full((C, B), -1, dtype=np.int32)
            g_c[r_copy, r_pos - s] = g_cr
            g_t[r_copy, r_pos - s] = g_tr
            res = sess.unmask_accept(gp, False)[seq]
            k_iter += 1
            if op.sampling:
                walk = lambda c_, t_, m_, *a_: ({int(i): int(t_[0][i]) for i in np.flatnonzero(unmask(c_[0], m_, k_iter))}, [0], 0)
            else:
                walk = O.pick_best_walk if op.pick_best else O.jump_walk
            new, chain, last = walk(g_c, g_t, masked, subsets, ranks, rank_tok, tau)
            want = sorted((int(s + i), int(t)) for i, t in new.items())
            assert res_tuple(res) == (want, [int(c) for c in chain]), (res_tuple(res), want, chain)
            new_o, chain_o, last_o = walk(o_c, o_t, masked, subsets, ranks, rank_tok, tau)
            o_gaps = np.full(o_c.shape, np.inf)
            o_gaps[r_copy, r_pos - s] = O.top2_gap(o_logits, shape_mask)
            visited = chain_o if not (op.pick_best and chain_o != [0]) else [0] + chain_o
            record("step", O.walk_diagnostics(o_c, o_gaps, masked, subsets, ranks, visited, new_o, tau, k_ranks),
                   masked[r_pos - s], g_cr, o_c[r_copy, r_pos - s], g_logits, o_logits)
            if set(new_o) != set(new) or chain_o != chain:
                margin = min(O.decision_margin(o_c[c], masked & (o_c[c] >= 0), tau, 0) for c in chain_o)
                st["oracle_decision_diff"] += 1
                st["near_ties"].append((st["iters"], "step", margin, cerr, st["log"][-1]["tok_gap"], st["log"][-1]["logit_err"]))
            elif new_o != new:
                st["tok_only_diff"] += 1
            for p_, t_ in want:
                x[p_] = t_
            st["iters"] += 1; st["steps"] += 1; st["tokens"] += len(want)
            assert res.masks_left == int((x[s:e] == shape_mask).sum())
            last_conf, last_tok = g_c[last], g_t[last]
            if stop is not None and stop(st):
                max_iters = st["iters"]
        b += 1
    st["tokens_final"] = x.astype(np.int32)
    return st


def assert_near_ties_only(st, floor=1e-3):
    """Every iteration where the oracle would have decided differently (other positions, another jump chain) must be a
    near-tie: its decision margin no larger than four times the confidence error measured there (floor 1e-3), or - a
    jump hangs on a greedy token matching its fill - a used greedy token whose top-2 logit gap is within twice the
    largest logit error measured there."""
    for it, kind, margin, cerr, *rest in st["near_ties"]:
        tok_gap, lerr = rest if rest else (None, None)
        by_conf = margin <= max(floor, 4 * cerr)
        by_token = lerr is not None and tok_gap is not None and tok_gap <= 2 * lerr
        assert by_conf or by_token, (f"iteration {it} ({kind}): margin {margin:.3e}, conf error {cerr:.3e}, "
                                     f"top-2 gap {tok_gap}, logit error {lerr}")


def anchored_bounds(layers, n_elements):
    """(per-row relative L2 bound, element-wise factor over the small-model bound) for a model of this depth, from
    the oracle's measured distance between its own float32 and float64 runs (tests/golden/oracle_self_distance.py)."""
    import importlib.util
    import os
    path = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "oracle_self_distance.py")
    spec = importlib.util.spec_from_file_location("oracle_self_distance", path)
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return mod.l2_bound(layers), mod.elementwise_factor(layers, n_elements)
