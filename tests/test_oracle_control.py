"""Pins for the oracle's control logic: accept rule, ranking, jump walk, ALP, generate."""
import dataclasses

import numpy as np
import pytest

import synth
from oracle import odb_oracle as O
from oracle.inputs import model_from_synth

f32 = lambda *a: np.array(a, dtype=np.float32)


# ----------------------------------------------------------------------------- accept / rank

def test_accept_set_rule():
    conf = f32(.95, .2, .93, .9, .5)
    masked = np.array([1, 1, 1, 1, 0], dtype=bool)
    assert O.accept_set(conf, masked, 0.9).tolist() == [True, False, True, False, False]   # strict ">"
    # nothing passes -> the single most confident masked position; ties -> lowest position
    assert O.accept_set(f32(.3, .7, .7, .99), np.array([1, 1, 1, 0], bool), 0.9).tolist() == [False, True, False, False]
    # unmasked positions never accepted even if confident
    assert O.accept_set(f32(.99, .1), np.array([0, 1], bool), 0.9).tolist() == [False, True]
    assert not O.accept_set(f32(.99, .1), np.array([0, 0], bool), 0.9).any()
    # the compare happens in fp32: 0.9 as fp32 is not > fp32(0.9)
    assert not (np.float32(0.9) > np.float32(0.9))
    assert O.accept_set(f32(0.9, 0.1), np.array([1, 1], bool), 0.9).tolist() == [True, False]  # by fallback only


def test_rank_candidates():
    conf = f32(.5, .8, .8, .1, .7)
    masked = np.array([1, 1, 1, 1, 0], bool)
    assert O.rank_candidates(conf, masked, 2) == [1, 2]
    assert O.rank_candidates(conf, masked, 4) == [1, 2, 0, 3]
    assert O.rank_candidates(conf, np.array([0, 0, 0, 1, 0], bool), 4) == [3]


def test_copy_subsets():
    assert O.copy_subsets(0, 1, False) == [()]
    assert O.copy_subsets(2, 4, False) == [(), (1,), (2,), (1, 2)]         # Section 4.2.1
    assert O.copy_subsets(1, 4, False) == [(), (1,)]
    assert O.copy_subsets(0, 4, False) == [()]
    assert O.copy_subsets(4, 8, True) == [(), (1,), (2,), (1, 2), (3,), (1, 2, 3), (4,), (1, 2, 3, 4)]  # Section 4.2.2
    assert O.copy_subsets(3, 8, True) == [(), (1,), (2,), (1, 2), (3,), (1, 2, 3)]


# ----------------------------------------------------------------------------- jump walk

def _walk(conf_rows, tok_rows, masked, subsets, rank_off, rank_tok, tau=0.9):
    conf = np.array(conf_rows, dtype=np.float32)
    tok = np.array(tok_rows, dtype=np.int32)
    return O.jump_walk(conf, tok, np.array(masked, bool), subsets, rank_off, rank_tok, tau)


S1 = [(), (1,), (2,), (1, 2)]


def test_jump_both_hit_goes_to_copy_3():
    # Section 4.2.1: B and D both unmasked in block 0 -> jump directly to block 3
    masked = [1, 1, 1, 1]
    conf = [[.95, .92, .1, .2], [0, .5, .1, .2], [.5, 0, .1, .2], [0, 0, .3, .6]]
    tok = [[7, 8, 1, 1], [7, 8, 1, 1], [7, 8, 1, 1], [7, 8, 5, 6]]
    new, chain, last = _walk(conf, tok, masked, S1, [0, 1], [7, 8])
    assert chain == [0, 3] and last == 3
    assert new == {0: 7, 1: 8, 3: 6}            # block 3's own decoding (fallback: its best position) is incorporated


def test_jump_one_hit_then_verify_other():
    masked = [1, 1, 1, 1]
    # only B (rank 1) unmasked in block 0 -> block 1; there D passes -> block 3
    conf = [[.95, .5, .1, .2], [0, .91, .1, .2], [.5, 0, .1, .2], [0, 0, .95, .6]]
    tok = [[7, 8, 1, 1], [7, 8, 1, 1], [7, 8, 1, 1], [7, 8, 5, 6]]
    new, chain, last = _walk(conf, tok, masked, S1, [0, 1], [7, 8])
    assert chain == [0, 1, 3] and new == {0: 7, 1: 8, 2: 5}
    # verification fails in block 1 -> adopt block 1's decoding
    conf[1] = [0, .3, .6, .2]
    new, chain, last = _walk(conf, tok, masked, S1, [0, 1], [7, 8])
    assert chain == [0, 1] and last == 1 and new == {0: 7, 2: 1}    # block 1's own decoding (its top-1) is adopted
    # an acceptance by the top-1 fallback verifies D just like one by threshold
    conf[1] = [0, .6, .3, .2]
    new, chain, last = _walk(conf, tok, masked, S1, [0, 1], [7, 8])
    assert chain == [0, 1, 3]
    # only D (rank 2) unmasked -> block 2
    conf[0] = [.5, .95, .1, .2]
    conf[2] = [.3, 0, .1, .2]
    new, chain, last = _walk(conf, tok, masked, S1, [0, 1], [7, 8])
    assert chain == [0, 2, 3]   # block 2's fallback accepts B's position (its top-1), which verifies B


def test_jump_needs_token_match_and_no_hit_stays():
    masked = [1, 1, 1, 1]
    conf = [[.95, .5, .1, .2], [0, .5, .1, .2], [.5, 0, .1, .2], [0, 0, .3, .6]]
    tok = [[9, 8, 1, 1], [7, 8, 1, 1], [7, 8, 1, 1], [7, 8, 5, 6]]      # block 0 now predicts 9, fill was 7
    new, chain, last = _walk(conf, tok, masked, S1, [0, 1], [7, 8])
    assert chain == [0] and new == {0: 9}
    # accepted position is not a candidate -> stay in block 0
    conf[0] = [.5, .4, .1, .97]
    new, chain, last = _walk(conf, tok, masked, S1, [0, 1], [7, 8])
    assert chain == [0] and new == {3: 1}


def test_jump_chain_union_keeps_earlier_link():
    masked = [1, 1, 1, 1]
    # block 0 accepts rank-1 position and position 3 (token 4); block 1 would predict 6 at position 3
    conf = [[.95, .5, .1, .93], [0, .5, .1, .99], [0, 0, 0, 0], [0, 0, 0, 0]]
    tok = [[7, 8, 1, 4], [7, 8, 1, 6], [0, 0, 0, 0], [0, 0, 0, 0]]
    new, chain, last = _walk(conf, tok, masked, S1, [0, 1], [7, 8])
    assert chain == [0, 1] and new == {0: 7, 3: 4}


def test_jump_walk_worked_example_six_positions():
    """Hand-worked case: tau .9, block of 6, fills match.  Block 0 accepts only r1; copy {r1}
    then accepts r2; copy {r1,r2} accepts one more position; three tokens from one forward."""
    masked = [0, 1, 0, 1, 1, 1]                 # p0, p2 already decoded; r1 = p1, r2 = p5
    n = -1.0
    conf = [[n, .92, n, .50, .20, .85],
            [n, n, n, .60, .25, .91],
            [n, .3, n, .1, .1, n],
            [n, n, n, .95, .30, n]]
    tok = [[0, 11, 0, 13, 14, 15]] * 4
    new, chain, last = _walk(conf, tok, masked, S1, [1, 5], [11, 15])
    assert chain == [0, 1, 3] and last == 3 and new == {1: 11, 5: 15, 3: 13}


def test_jump_walk_stage2_lattice():
    S2 = O.copy_subsets(4, 8, True)
    masked = [1] * 6
    rank_off, rank_tok = [0, 1, 2, 3], [10, 11, 12, 13]
    tok = [[10, 11, 12, 13, 14, 15]] * 8
    conf = np.zeros((8, 6), np.float32)
    conf[0, [0, 1, 2]] = .95                     # ranks 1,2,3 hit in block 0 -> largest available superset {1,2,3}
    conf[5, 3] = .95                             # there rank 4 hits -> {1,2,3,4}
    conf[7, 4] = .5
    new, chain, last = O.jump_walk(conf, np.array(tok, np.int32), np.array(masked, bool), S2, rank_off, rank_tok, .9)
    assert chain == [0, 5, 7] and new == {0: 10, 1: 11, 2: 12, 3: 13, 4: 14}
    conf[:] = 0
    conf[0, 2] = .95                             # only rank 3 hit -> copy {3} (index 4); no further superset of {3} exists
    conf[4, 5] = .2
    new, chain, last = O.jump_walk(conf, np.array(tok, np.int32), np.array(masked, bool), S2, rank_off, rank_tok, .9)
    assert chain == [0, 4] and new == {2: 12, 5: 15}


# ----------------------------------------------------------------------------- the compared "vanilla" speculation

def _pick(conf_rows, tok_rows, masked, subsets, rank_off, rank_tok, tau=0.9):
    return O.pick_best_walk(np.array(conf_rows, np.float32), np.array(tok_rows, np.int32), np.array(masked, bool),
                            subsets, rank_off, rank_tok, tau)


def test_pick_best_adopts_one_block_and_nothing_else():
    """Fig. 7(a) / Section 5.3: candidates are checked in the main block, one appended block is picked and
    its decoding replaces the main block's; one state change per step (chain of one link)."""
    masked = [1] * 6
    rank_off, rank_tok = [1, 5], [11, 15]
    tok = [[20, 11, 22, 23, 24, 15]] * 4
    # both candidates accepted in block 0, which also accepts position 0: the block filling both is adopted; its own
    # accept set is position 3; position 0 (output of the block that was not adopted) is NOT committed
    conf = [[.95, .95, .1, .1, .1, .95], [0] * 6, [0] * 6, [.5, 0, .1, .95, .1, 0]]
    new, chain, last = _pick(conf, tok, masked, S1, rank_off, rank_tok)
    assert (new, chain, last) == ({1: 11, 5: 15, 3: 23}, [3], 3)
    # the jump chain on the same numbers keeps position 0 as well and has two links
    new_j, chain_j, _ = _walk(conf, tok, masked, S1, rank_off, rank_tok)
    assert new_j == {0: 20, 1: 11, 5: 15, 3: 23} and chain_j == [0, 3]
    # only the first candidate is hit: its block is adopted; that block accepts the second candidate's position,
    # which is committed as that block's output, but no second block is entered (the jump chain would go on to {1,2})
    conf = [[.1, .95, .1, .1, .1, .3], [.1, 0, .1, .1, .1, .95], [0] * 6, [.1, 0, .95, .1, .1, 0]]
    new, chain, last = _pick(conf, tok, masked, S1, rank_off, rank_tok)
    assert (new, chain, last) == ({1: 11, 5: 15}, [1], 1)
    new_j, chain_j, _ = _walk(conf, tok, masked, S1, rank_off, rank_tok)
    assert chain_j == [0, 1, 3] and new_j == {1: 11, 5: 15, 2: 22}
    # a candidate accepted with ANOTHER token is not a hit; nothing hit: the main block's own result
    tok2 = [[20, 99, 22, 23, 24, 15]] + tok[1:]
    conf = [[.1, .95, .1, .1, .1, .3]] + [[.95] * 6] * 3
    new, chain, last = _pick(conf, tok2, masked, S1, rank_off, rank_tok)
    assert (new, chain, last) == ({1: 99}, [0], 0)
    # nothing above the threshold anywhere: top-1 fallback of the main block, which is a hit when it is the first
    # candidate with its token -> that candidate's block, whose own fallback commits one more position
    conf = [[.1, .6, .1, .1, .1, .3], [.1, 0, .1, .4, .1, .2], [0] * 6, [0] * 6]
    new, chain, last = _pick(conf, tok, masked, S1, rank_off, rank_tok)
    assert (new, chain, last) == ({1: 11, 3: 23}, [1], 1)
    # the adopted block has nothing left to decode: only its fills are committed
    new, chain, last = _pick([[.95, .95], [0, 0], [0, 0], [0, 0]], [[11, 15]] * 4, [1, 1], S1, [0, 1], [11, 15])
    assert (new, chain, last) == ({0: 11, 1: 15}, [3], 3)


def test_pick_best_generation_has_eff_nfe_equal_to_nfe(tiny_model):
    """Section 5.3: for the compared speculation Eff_NFE equals NFE; the run still fills every position, never
    needs more passes than plain block decoding needs in the worst case, and without a hit it IS plain block
    decoding (one block's accept set per pass)."""
    shape = synth.TINY
    P, L, Bk = 12, 32, 16
    x0 = synth.sequence(4, 0, P, L, shape)
    pv, cb = O.mode_settings("spec_vanilla", Bk)
    assert pv.pick_best and pv.n_copies == 4 and not pv.alp and cb
    xv, tv = O.generate(tiny_model, x0, P, pv)
    cv = O.trace_counters(tv)
    assert (xv[P:] != shape.mask_id).all() and cv["tokens"] == L
    assert cv["eff_nfe"] == cv["nfe"] <= L and all(len(t["chain"]) == 1 for t in tv)
    pj, _ = O.mode_settings("accept_jump", Bk)
    xj, tj = O.generate(tiny_model, x0, P, pj)
    cj = O.trace_counters(tj)
    assert not pj.pick_best and cj["tokens"] == L and cj["eff_nfe"] >= cj["nfe"]
    pd, _ = O.mode_settings("decoded_share", Bk)
    assert pd.n_copies == 8 and not pd.alp
    # every committed token of a picked block is either a verified fill or in that block's own accept set: replay
    for t in tv:
        assert len(t["accepted"]) >= 1


# ----------------------------------------------------------------------------- ALP

def test_alp_scan_cases():
    eos = 5
    conf = f32(.1, .95, .99, .4, .97)
    assert O.alp_scan(conf, np.array([1, 2, 3, 4, 6]), 20, 10, eos, 0.9) is None          # no EOS
    assert O.alp_scan(conf, np.array([5, 2, 3, 5, 6]), 20, 10, eos, 0.9) is None          # EOS below threshold
    assert O.alp_scan(conf, np.array([5, 5, 5, 4, 5]), 20, 10, eos, 0.9) == 12            # earliest passing EOS, slot kept
    assert O.alp_scan(conf, np.array([1, 2, 3, 4, 5]), 20, 10, eos, 0.9) == 15
    assert O.alp_scan(f32(.9), np.array([5]), 20, 10, eos, 0.9) is None                   # strict ">"


# ----------------------------------------------------------------------------- generate

@pytest.fixture(scope="module")
def tiny_model():
    return model_from_synth(synth.TINY, seed=0)


def test_generate_cfg1_one_token_per_iteration(tiny_model):
    x0 = synth.sequence(0, 0, 64, 64, synth.TINY)
    x, trace = O.generate(tiny_model, x0, 64, O.DecodeParams(block_len=16))
    assert (x[:64] == x0[:64]).all() and (x[64:] != synth.TINY.mask_id).all()
    assert all(len(t["accepted"]) >= 1 for t in trace)                # progress every iteration
    assert [t["kind"] for t in trace].count("refresh") == 4
    # random weights: no confidence gets near 0.9, every iteration accepts exactly one token
    assert len(trace) == 64 and all(len(t["accepted"]) == 1 for t in trace)
    for t in trace:
        (p, _), = t["accepted"]
        assert 64 + 16 * t["block"] <= p < 64 + 16 * (t["block"] + 1)  # unmasking restricted to the block


def test_generate_threshold_extremes(tiny_model):
    x0 = synth.sequence(0, 0, 64, 64, synth.TINY)
    # tau >= 1: never exceeded -> exactly one token per iteration, in descending confidence order
    x_hi, tr_hi = O.generate(tiny_model, x0, 64, O.DecodeParams(block_len=16, accept_threshold=1.0))
    assert len(tr_hi) == 64
    # tau < 0: everything exceeds -> a block fills in its refresh iteration: iterations == blocks
    x_lo, tr_lo = O.generate(tiny_model, x0, 64, O.DecodeParams(block_len=16, accept_threshold=-1.0))
    assert len(tr_lo) == 4 and all(t["kind"] == "refresh" and len(t["accepted"]) == 16 for t in tr_lo)
    # the first iteration of block 0 is the same prediction in both runs
    cache, conf, tok = O.refresh_prefill(tiny_model, x0, 128, 64)
    assert (x_lo[64:80] == tok[:16]).all()
    assert tr_hi[0]["accepted"] == [(64 + int(np.argmax(conf[:16])), int(tok[np.argmax(conf[:16])]))]


def test_jump_share_is_lossless_when_single_accepts(tiny_model):
    """When every accept set is a single position, copy {r1} is exactly the state plain decoding
    reaches next, so the jump walk reproduces plain decoding with fewer forwards."""
    x0 = synth.sequence(0, 0, 64, 64, synth.TINY)
    x1, tr1 = O.generate(tiny_model, x0, 64, O.DecodeParams(block_len=16, n_copies=1))
    x4, tr4 = O.generate(tiny_model, x0, 64, O.DecodeParams(block_len=16, n_copies=4))
    assert (x1 == x4).all()
    assert len(tr4) < len(tr1)
    assert [t["kind"] for t in tr4].count("refresh") == 4
    assert max(len(t["chain"]) for t in tr4) <= 3 and max(len(t["accepted"]) for t in tr4) <= 3
    # the order of commitment is the same sequence of (position, token) pairs
    flat = lambda tr: [a for t in tr for a in t["accepted"]]
    assert sorted(flat(tr1)) == sorted(flat(tr4))


def test_generate_stage2_runs_and_respects_row_budget(tiny_model):
    x0 = synth.sequence(0, 0, 64, 64, synth.TINY)
    p = O.DecodeParams(block_len=16, n_copies=8)
    x8, tr8 = O.generate(tiny_model, x0, 64, p)
    assert (x8[64:] != synth.TINY.mask_id).all()
    assert any(t.get("stage2") for t in tr8) and any(not t.get("stage2") for t in tr8 if t["kind"] == "step")
    assert O.use_stage2(p, 16, 9) is False and O.use_stage2(p, 16, 10) is True          # ceil(64/7) = 10
    assert 16 + 7 * (16 - 10) <= 4 * 16 < 16 + 7 * (16 - 9)
    assert O.use_stage2(p, 32, 18) is False and O.use_stage2(p, 32, 19) is True


def test_alp_truncates_and_generation_continues_shorter():
    """A sharp 64-word model with an [EOS] direction planted deep in the response: with truncate
    threshold 0 the first refresh must cut the response at the first predicted [EOS].  Lengths
    never grow afterwards."""
    shape = dataclasses.replace(synth.TINY_PEAKY, vocab=64, mask_id=63, eos_id=62)
    m = model_from_synth(shape, seed=5)
    x0 = synth.sequence(5, 0, 32, 64, shape)
    # plant an [EOS] direction: the LM-head row of [EOS] points along what is particular to the
    # final hidden state of response position 40 in the first refresh
    hid, _, _ = O.forward_rows(m, x0.astype(np.int64), np.arange(96), None, None, np.ones((96, 96), bool),
                               return_hidden=True)
    n = O.bf16_round(O.rmsnorm(hid, m.final_gain, m.rms_eps))[32:]
    lm = m.lm_head.copy()
    lm[shape.eos_id] = O.bf16_round(30.0 * (n[40] - n.mean(0)))
    m = dataclasses.replace(m, lm_head=lm)
    eos = shape.eos_id
    _, conf, tok = O.refresh_prefill(m, x0, 96, 32)
    first = int(np.flatnonzero(tok == eos)[0])
    assert 16 < first <= 40                                           # lands beyond the first block
    p = O.DecodeParams(block_len=16, truncate_threshold=0.0)
    x, tr = O.generate(m, x0, 32, p)
    lens = [t["T"] for t in tr]
    assert tr[0]["T"] == 32 + first + 1                               # cut at that position, slot kept
    assert all(a >= b for a, b in zip(lens, lens[1:])) and lens[-1] < 96
    assert len(x) == lens[-1] and (x[32:] != shape.mask_id).all()
    last_block = (len(x) - 32 - 1) // 16
    assert tr[-1]["block"] == last_block                              # a partial last block is still decoded
    # a high truncate threshold leaves the length alone unless the confidence passes it
    x_hi, tr_hi = O.generate(m, x0, 32, dataclasses.replace(p, truncate_threshold=float(conf[first]) + 1e-3), max_iters=1)
    assert tr_hi[0]["T"] == 96 or tr_hi[0]["T"] > tr[0]["T"]
    # ALP off: full length
    x_off, tr_off = O.generate(m, x0, 32, dataclasses.replace(p, alp=False))
    assert len(x_off) == 96
    # after the cut the run is that of a session that owns only the first T' tokens: replaying
    # block 1's refresh on the truncated sequence reproduces the traced decision
    T1 = tr[0]["T"]
    n0 = sum(1 for t in tr if t["block"] == 0)
    xa = x0[:T1].astype(np.int64)
    for t in tr[:n0]:
        for pos, tk in t["accepted"]:
            xa[pos] = tk
    _, conf_a, tok_a = O.refresh_prefill(m, xa, T1, 48)
    newL = O.alp_scan(conf_a, tok_a, 48, 32, eos, 0.0)
    T2 = T1 if newL is None else min(T1, 32 + newL)
    assert tr[n0]["kind"] == "refresh" and tr[n0]["block"] == 1 and tr[n0]["T"] == T2


def test_length_schedule_lever(tiny_model):
    x0 = synth.sequence(0, 0, 64, 64, synth.TINY)
    sched = lambda b, L: {0: 40, 1: 24}.get(b)
    x, tr = O.generate(tiny_model, x0, 64, O.DecodeParams(block_len=16), length_schedule=sched)
    assert len(x) == 64 + 24 and [t["T"] for t in tr if t["kind"] == "refresh"] == [104, 88]
    assert (x[64:] != synth.TINY.mask_id).all()


# ---- baseline modes and counters (Tables 2 and 3; Section 5.3) ----------------------------------

def test_cacheless_baseline_is_one_refresh_per_token():
    shape = synth.TINY
    om = model_from_synth(shape, seed=0)
    P, L, Bk = 24, 12, 4
    x0 = synth.sequence(0, 0, P, L, shape)
    params, cache_blocks = O.mode_settings("vanilla", Bk)
    assert not cache_blocks and params.n_copies == 1 and not params.alp
    x, trace = O.generate(om, x0, P, params, cache_blocks=cache_blocks)
    c = O.trace_counters(trace)
    # no confidence exceeds 1, so the fallback commits exactly one token per full forward
    assert c == {"nfe": L, "eff_nfe": L, "tokens": L, "refreshes": L, "tokens_per_nfe": 1.0}
    assert all(t["kind"] == "refresh" and len(t["accepted"]) == 1 for t in trace)
    assert [t["block"] for t in trace] == [i // Bk for i in range(L)]          # blocks in order, Bk iterations each
    assert (x[P:] != shape.mask_id).all()
    # every iteration sees the exact current state: each committed token is the argmax of an uncached
    # forward over the sequence as it stood, at the most confident masked position of the block
    xs = x0.astype(np.int64).copy()
    for t in trace:
        s = P + t["block"] * Bk
        _, conf, tok = O.refresh_prefill(om, xs, len(xs), s)
        masked = xs[s:s + Bk] == shape.mask_id
        i = int(np.argmax(np.where(masked, conf[:Bk], -1.0)))
        assert t["accepted"] == [(s + i, int(tok[i]))]
        xs[s + i] = tok[i]


def test_block_of_one_makes_cached_and_cacheless_decoding_identical():
    # with one position per block every iteration is a refresh in both systems
    shape = synth.TINY
    om = model_from_synth(shape, seed=1)
    P, L = 16, 6
    x0 = synth.sequence(1, 0, P, L, shape)
    p = O.DecodeParams(block_len=1, n_copies=1, alp=False)
    xa, ta = O.generate(om, x0, P, p, cache_blocks=True)
    xb, tb = O.generate(om, x0, P, p, cache_blocks=False)
    assert np.array_equal(xa, xb)
    assert [(t["kind"], t["accepted"]) for t in ta] == [(t["kind"], t["accepted"]) for t in tb]


def test_counters_of_the_three_systems():
    shape = synth.TINY_PEAKY
    om = model_from_synth(shape, seed=0)
    wl = synth.WORKLOADS["peaky_c4"]
    x0 = synth.sequence(0, 0, wl.prompt_len, wl.gen_len, shape)
    out = {}
    for mode in ("vanilla", "fast_dllm", "odb"):
        params, cache_blocks = O.mode_settings(mode, wl.block_len)
        x, trace = O.generate(om, x0, wl.prompt_len, params, cache_blocks=cache_blocks)
        out[mode] = (x, O.trace_counters(trace))
    L, nb = wl.gen_len, wl.gen_len // wl.block_len
    assert out["vanilla"][1]["nfe"] == L and out["vanilla"][1]["refreshes"] == L
    f, o = out["fast_dllm"][1], out["odb"][1]
    assert f["refreshes"] == nb and f["eff_nfe"] == f["nfe"] <= L              # no speculation: one state change per pass
    assert o["refreshes"] <= nb and o["nfe"] <= f["nfe"]                       # jumps only ever save passes
    assert o["eff_nfe"] >= o["nfe"]                                            # several state changes in one pass
    assert f["tokens"] == L and o["tokens"] == len(out["odb"][0]) - wl.prompt_len



# ----------------------------------------------------------------------------- diagnostics (decide nothing)

ALL4 = np.ones(4, bool)


def test_decision_margin_threshold_term_binds():
    # something passes tau: only the distances to the threshold count; .95 is the closest, (.95 - .9) / .9
    m = O.decision_margin(f32(.95, .5, .1), np.ones(3, bool), 0.9)
    assert m == pytest.approx(0.05 / 0.9, rel=1e-5)
    # a position just BELOW the threshold binds the same way
    assert O.decision_margin(f32(.99, .89, .1), np.ones(3, bool), 0.9) == pytest.approx(0.01 / 0.9, rel=1e-4)
    # positions that are not masked take no part, however close to tau they are
    assert O.decision_margin(f32(.9001, .5), np.array([0, 1], bool), 0.9) == pytest.approx(0.4 / 0.9, rel=1e-5)


def test_decision_margin_fallback_term_binds():
    # nothing passes: the best must beat the runner-up, (.5 - .45) / .5 = .1 < distance to tau .4 / .9
    assert O.decision_margin(f32(.5, .45, .1), np.ones(3, bool), 0.9) == pytest.approx(0.1, rel=1e-5)
    # as soon as one position passes, the top-2 gap decides nothing any more
    assert O.decision_margin(f32(.95, .949, .1), np.ones(3, bool), 0.9) == pytest.approx(0.049 / 0.9, rel=1e-4)
    # a single masked position has no runner-up
    assert O.decision_margin(f32(.5, .49), np.array([1, 0], bool), 0.9) == pytest.approx(0.4 / 0.9, rel=1e-5)


def test_decision_margin_ranking_term_binds():
    conf = f32(.95, .6, .57, .2)
    assert O.decision_margin(conf, ALL4, 0.9, 0) == pytest.approx(0.05 / 0.9, rel=1e-5)       # no ranking asked for
    # one candidate: .6 against the first one left out, (.6 - .57) / .6 = .05 < .0556
    assert O.decision_margin(conf, ALL4, 0.9, 1) == pytest.approx(0.05, rel=1e-5)
    # two candidates add (.57 - .2) / .57, which does not bind
    assert O.decision_margin(conf, ALL4, 0.9, 2) == pytest.approx(0.05, rel=1e-5)
    # more candidates than positions left: only the gaps that exist
    assert O.decision_margin(conf, ALL4, 0.9, 7) == pytest.approx(0.05, rel=1e-5)
    # the last candidate against the first one left out binds too
    assert O.decision_margin(f32(.95, .6, .3, .299), ALL4, 0.9, 2) == pytest.approx(0.001 / 0.3, rel=1e-3)
    assert O.decision_margin(f32(.95, .6, .3, .299), ALL4, 0.9, 1) == pytest.approx(0.05 / 0.9, rel=1e-5)


def test_decision_margin_ignores_order_among_accepted_positions():
    # .99 and .9899 are both accepted: their near-tie decides nothing; the fallback's winner is accepted too
    assert O.decision_margin(f32(.99, .9899, .3, .1), ALL4, 0.9, 2) == pytest.approx(0.0899 / 0.9, rel=1e-3)
    assert O.decision_margin(f32(.5, .3, .299, .1), ALL4, 0.9, 1) == pytest.approx(0.001 / 0.3, rel=1e-3)   # .5 taken by fallback
    assert O.decision_margin(f32(.5, .3, .299, .1), ALL4, 0.9, 0) == pytest.approx(0.4, rel=1e-5)          # (.5 - .3) / .5


def test_decision_margin_empty_and_overrides():
    assert O.decision_margin(f32(.5, .6), np.zeros(2, bool), 0.9, 2) == np.inf
    # still_masked: rank only what a jump chain left ({2, 3}), not everything this row did not accept
    conf = f32(.95, .6, .599, .2)
    assert O.decision_margin(conf, ALL4, 0.9, 1) == pytest.approx(0.001 / 0.6, rel=1e-3)
    assert O.decision_margin(conf, ALL4, 0.9, 1, np.array([0, 0, 1, 1], bool)) == pytest.approx(0.05 / 0.9, rel=1e-5)
    # plain differences instead of relative gaps
    assert O.decision_margin(f32(.5, .45, .1), np.ones(3, bool), 0.9, relative=False) == pytest.approx(0.05, rel=1e-5)
    assert O.decision_margin(conf, ALL4, 0.9, 1, relative=False) == pytest.approx(0.001, rel=1e-3)


def test_top2_gap_and_conf_logit():
    logits = np.array([[1.0, 3.0, 2.5, 9.0], [0.0, -1.0, 7.0, 9.0]])
    assert O.top2_gap(logits, 3).tolist() == [0.5, 7.0]                  # entry 3 is [MASK]: excluded
    assert O.top2_gap(logits, 0).tolist() == [6.0, 2.0]
    assert O.conf_logit(0.5) == pytest.approx(0.0, abs=1e-12)
    assert O.conf_logit(0.9) == pytest.approx(np.log(9.0))
    assert O.conf_logit(1.0) == pytest.approx(-O.conf_logit(0.0)) and np.isfinite(O.conf_logit(1.0))
    # the property it is used for: moving every logit by at most eps moves conf_logit by at most 2 eps
    rng = np.random.default_rng(0)
    l = rng.normal(0, 3, (50, 40))
    for eps in (1e-3, 0.1):
        c0, _ = O.confidence(l, 39)
        c1, _ = O.confidence(l + rng.uniform(-eps, eps, l.shape), 39)
        ok = O.top2_gap(l, 39) > 2 * eps                                   # same greedy token on both sides
        d = np.abs(O.conf_logit(c1.astype(np.float64)) - O.conf_logit(c0.astype(np.float64)))
        assert (d[ok] <= 2 * eps * (1 + 1e-3) + 1e-6).all()


def test_walk_diagnostics_on_the_worked_example():
    """The six-position example above: chain 0 -> {r1} -> {r1, r2}; p1, p5, p3 committed, p4 left."""
    n = -1.0
    masked = np.array([0, 1, 0, 1, 1, 1], bool)
    conf = np.array([[n, .92, n, .50, .20, .85],
                     [n, n, n, .60, .25, .91],
                     [n, .3, n, .1, .1, n],
                     [n, n, n, .95, .30, n]], np.float32)
    gaps = np.full((4, 6), 5.0)
    gaps[0, 1], gaps[1, 5], gaps[3, 3], gaps[3, 4], gaps[0, 3] = 1.0, 0.7, 2.0, 0.9, 0.01
    d = O.walk_diagnostics(conf, gaps, masked, S1, [1, 5], [0, 1, 3], {1: 11, 5: 15, 3: 13}, 0.9, 2)
    # closest confidence decision: .91 against tau in copy {r1} (its own fill p1 is not masked there)
    assert d["margin"] == pytest.approx(0.01 / 0.9, rel=1e-3)
    assert d["sep"] == pytest.approx(float(O.conf_logit(.91) - O.conf_logit(.9)), rel=1e-3)
    # tokens used: p1 in copy 0, p5 in copy {r1}, p3 in the last copy and the next candidate p4 there;
    # the near-tie of p3's token in copy 0 (gap .01) is not used: p3 is not accepted there
    assert d["tok_gap"] == 0.7
    # with only the main block visited the closest decision is .92 against tau, and p1's token the one used,
    # next candidates ranked from copy 0: p5 (.85), p3 (.50) -> p3's token there now counts
    d0 = O.walk_diagnostics(conf, gaps, masked, S1, [1, 5], [0], {1: 11}, 0.9, 2)
    assert d0["margin"] == pytest.approx(0.02 / 0.9, rel=1e-3) and d0["tok_gap"] == 0.01


# ----------------------------------------------------------------------------- stochastic reverse step (Eq. 1)

def test_reverse_step_keeps_unmasked_and_ends_unmasking_everything():
    masked = np.array([1, 0, 1, 1, 0, 1], bool)
    u = f32(.99, .99, .0, .5, .0, .74)
    acc = O.reverse_step_unmask(masked, u, 0, 4)            # stay with probability 3/4: unmask iff u >= .75
    assert acc.tolist() == [True, False, False, False, False, False]      # unmasked positions never change (first case)
    assert O.reverse_step_unmask(masked, u, 2, 4).tolist() == [True, False, False, True, False, True]   # stay 1/2
    # the boundary is "stay masked iff u < s / t", in fp32
    assert O.reverse_step_unmask(np.ones(2, bool), f32(0.75, np.nextafter(np.float32(0.75), np.float32(0))), 0, 4).tolist() == [True, False]
    # last iteration: s = 0, nothing stays masked, whatever the deviates
    assert O.reverse_step_unmask(masked, np.zeros(6, np.float32), 3, 4).tolist() == masked.tolist()
    assert O.reverse_step_unmask(masked, np.zeros(6, np.float32), 0, 1).tolist() == masked.tolist()


def test_reverse_step_stay_probability_and_linear_survival():
    """Second case of Eq. 1: a masked position stays masked with probability s / t.  With t falling linearly over
    the n iterations of a block, the probability of still being masked after iteration k is the product of the
    stay probabilities = (n - k - 1) / n: every position is unmasked at a uniformly distributed iteration."""
    n, N = 8, 200000
    alive = np.ones(N, bool)
    for k in range(n):
        u = synth.uniform(7, 100 + k, N)
        acc = O.reverse_step_unmask(alive, u, k, n)
        frac_stay = 1.0 - acc.sum() / alive.sum()
        want = (n - k - 1) / (n - k)
        assert abs(frac_stay - want) < 4 * np.sqrt(max(want * (1 - want), 1e-9) / alive.sum()) + 1e-12, (k, frac_stay, want)
        alive &= ~acc
        assert abs(alive.mean() - (n - k - 1) / n) < 4 * np.sqrt(0.25 / N), (k, alive.mean())
    assert not alive.any()


def test_generate_with_sampling(tiny_model):
    om, P = tiny_model, 64
    x0 = synth.sequence(0, 0, P, 64, synth.TINY)
    L, Bk, n = len(x0) - P, 16, 6
    noise = lambda b, k: synth.uniform(3, 1000 * b + k, Bk)
    p = O.DecodeParams(block_len=Bk, sampling=True, sample_steps=n, alp=False)
    x, tr = O.generate(om, x0, P, p, noise=noise)
    assert (x[P:] != om.mask_id).all() and sum(len(t["accepted"]) for t in tr) == L
    per_block = [sum(t["block"] == b for t in tr) for b in range(L // Bk)]
    assert all(1 <= c <= n for c in per_block) and max(per_block) > 1
    # what is committed at an iteration is the greedy token of THAT iteration's forward at the unmasked positions,
    # and which positions are unmasked depends on the deviates alone: replay the schedule without the model
    b, k, masked = -1, 0, None
    for t in tr:
        if t["kind"] == "refresh":
            b, k, masked = t["block"], 0, np.ones(Bk, bool)
        else:
            k += 1
        acc = O.reverse_step_unmask(masked, noise(b, k), k, n)
        assert [p_ - (P + b * Bk) for p_, _ in t["accepted"]] == np.flatnonzero(acc).tolist()
        masked &= ~acc
    # same deviates, same run; one iteration per block is the "accept everything at the refresh" regime
    x2, tr2 = O.generate(om, x0, P, p, noise=noise)
    assert np.array_equal(x, x2) and [t["accepted"] for t in tr] == [t["accepted"] for t in tr2]
    x1, tr1 = O.generate(om, x0, P, O.DecodeParams(block_len=Bk, sampling=True, sample_steps=1, alp=False), noise=noise)
    x0_, tr0 = O.generate(om, x0, P, O.DecodeParams(block_len=Bk, accept_threshold=-1.0, alp=False))
    assert np.array_equal(x1, x0_) and len(tr1) == len(tr0) == L // Bk
