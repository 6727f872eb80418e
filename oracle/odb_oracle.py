"""CPU oracle for the ODB-dLLM block-decoding path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, by-eye-checkable numpy implementation of what the hot path computes: the
refresh prefill, the block-decode step over the block copies, the vocab softmax-confidence,
the threshold accept rule, the jump-share walk and adaptive length prediction, plus the
generate loop that strings them together.  It shares no code with the CUDA path and neither
imports the other; only tests, the smoke check and the benchmark's CPU-baseline leg may call
it.  Inputs (weights, token ids) are handed in as arrays.

What the paper fixes and what it leaves open
  * Block-wise decoding with a cache of the K/V of every token outside the block, refreshed
    by a full forward when the block is full: Section 1 (Fast-dLLM description) and
    Section 2.1 ("DualCache": prefix prompt and suffix [MASK] tokens).
  * Confidence-threshold acceptance, others re-masked: Section 3, Observation 3.
  * Adaptive length prediction: Section 4.1.
  * Speculative copies of the block, mutually invisible, all seeing the cached context:
    Section 4.2; accept-jump rule: Section 4.2.1; decoded-share layout and the four extra
    candidates: Section 4.2.2 and the caption of Fig. 8.
  * The paper states no model internals, threshold values, temperature or tie-breaks; the
    readings taken here are listed beside each function.

Arithmetic: `dtype` (float64 by default; float32 for large shapes).  With `faithful=True`
activations are rounded to bf16 exactly where the CUDA path stores bf16 (the projection input
of each RMSNorm, q/k/v after RoPE, attention output, SwiGLU output); the residual stream,
softmax statistics and logits are never rounded to bf16.  RMSNorm feeds a projection, and its
per-row scalar 1/rms commutes with the projection: the value stored in bf16 is x * gain, and
the scalar multiplies the projection's fp32 output (`normed_projection`).  Decisions that turn floating point
into integers (argmax over the vocabulary, threshold compares, ranking) are taken on fp32
values, the precision the kernels decide in.

Pins (tests/test_oracle_*.py): closed forms for RMSNorm/RoPE/SiLU, brute-force per-row
attention loops, a torch-CPU restatement of the full forward, the step-after-refresh
invariant, copy invisibility, zero-weight confidence 1/(V-1), accept-rule extremes
(threshold >= 1: one token per iteration; < 0: one iteration per block), the lossless
single-accept regime of jump-share (tokens with 4 copies == tokens with 1 copy), ALP unit
cases and the truncated-refresh equivalence, batch == independent runs.
PARITY UNPINNED (the paper prints no trace that could confirm them): the committed state
after a multi-link jump (chain union), the stage-2 walk over eight copies, the stage switch
point, "truncate keeps the [EOS] slot, effective immediately", and the compared speculation
variant of Section 5.3 (pick_best_walk: the paper gives its properties, not its rule).
"""
from __future__ import annotations

import dataclasses
from typing import Callable, Optional, Sequence

import numpy as np


# ----------------------------------------------------------------------------- containers

@dataclasses.dataclass
class Model:
    """LLaDA-style bidirectional transformer: pre-norm, MHA, RoPE, SwiGLU, untied LM head.

    `layer(l)` returns a dict with wq, wk, wv, wo [d][d], wg, wu [F][d], wd [d][F] (each
    [out][in]) and RMSNorm gains g1, g2 [d].  Matrices hold bf16-representable values.
    """
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    mask_id: int
    eos_id: int
    rope_theta: float
    rms_eps: float
    embed: np.ndarray                       # [V][d]
    lm_head: Optional[np.ndarray]           # [V][d]; None for the single-layer microbench
    final_gain: np.ndarray                  # [d]
    layer: Callable[[int], dict]


@dataclasses.dataclass
class Cache:
    """Global K/V cache written by the refresh: per layer [T][H][hd], K after RoPE."""
    k: list
    v: list
    length: int


# ----------------------------------------------------------------------------- primitives

def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round to the nearest bf16 value (ties to even), by way of fp32 as the kernels do."""
    f = np.ascontiguousarray(x, dtype=np.float32)
    u = f.view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32).astype(np.asarray(x).dtype)


def rmsnorm(x: np.ndarray, gain: np.ndarray, eps: float) -> np.ndarray:
    """y = x / sqrt(mean(x^2) + eps) * gain, over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gain


def normed_projection(x: np.ndarray, gain: np.ndarray, eps: float, weights: Sequence[np.ndarray], rnd) -> list:
    """[rmsnorm(x, gain) @ W^T for W in weights], evaluated as ((rnd(x * gain)) @ W^T) / rms(x).

    Mathematically rmsnorm(x) @ W^T (the row scalar 1/sqrt(mean(x^2) + eps) commutes with the
    matrix product); the order matters only for where the bf16 rounding `rnd` falls: on x * gain,
    the operand the kernels hand to the tensor cores, with the scalar applied to the fp32 result."""
    inv = 1.0 / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps)
    a = rnd(x * gain)
    return [(a @ w.T) * inv for w in weights]


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, rotate-half pairing: element i pairs with i + hd/2.

    x: [rows][H][hd]; pos: [rows] absolute positions (index in the sequence, prompt first).
    angle(row, i) = pos[row] * theta^(-2 i / hd), evaluated in float64.
    """
    hd = x.shape[-1]
    half = hd // 2
    inv_freq = np.asarray(theta, dtype=np.float64) ** (-2.0 * np.arange(half, dtype=np.float64) / hd)
    ang = pos.astype(np.float64)[:, None] * inv_freq[None, :]          # [rows][half]
    c = np.cos(ang).astype(x.dtype)[:, None, :]
    s = np.sin(ang).astype(x.dtype)[:, None, :]
    lo, hi = x[..., :half], x[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, vis: np.ndarray) -> np.ndarray:
    """Masked bidirectional softmax attention, written as its definition.

    q: [M][H][hd]; k, v: [N][H][hd]; vis: bool [M][N], row r attends key j iff vis[r][j].
    o[r][h] = sum_j softmax_j(q[r][h] . k[j][h] / sqrt(hd)) v[j][h] over visible j.
    """
    M, H, hd = q.shape
    out = np.empty_like(q)
    scale = 1.0 / np.sqrt(np.asarray(hd, dtype=q.dtype))
    for h in range(H):
        s = (q[:, h, :] @ k[:, h, :].T) * scale                         # [M][N]
        s = np.where(vis, s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=1, keepdims=True)
        out[:, h, :] = p @ v[:, h, :]
    return out


# ----------------------------------------------------------------------------- forward

def forward_rows(model: Model, tok: np.ndarray, pos: np.ndarray,
                 ctx_k: Optional[Sequence[np.ndarray]], ctx_v: Optional[Sequence[np.ndarray]],
                 vis: np.ndarray, *, faithful: bool = True, dtype=np.float64,
                 logit_rows: Optional[np.ndarray] = None, return_hidden: bool = False):
    """One forward of the transformer over M query rows.

    Keys of every layer = the given context K/V (cached rows; may be empty) followed by the
    fresh K/V of the M rows themselves; `vis` [M][Nc + M] says which keys each row sees.
    Returns (logits [len(logit_rows)][V] or final hidden [M][d], fresh_k, fresh_v) where
    fresh_k/v are per-layer lists of [M][H][hd] (K after RoPE; bf16-rounded if faithful).
    """
    rnd = bf16_round if faithful else (lambda a: a)
    H, hd, d = model.n_heads, model.head_dim, model.d_model
    M = len(tok)
    h = model.embed[tok].astype(dtype)                                  # [M][d]
    fresh_k, fresh_v = [], []
    for l in range(model.n_layers):
        w = model.layer(l)
        q, k, v = normed_projection(h, w["g1"].astype(dtype), model.rms_eps,
                                    [w["wq"].astype(dtype), w["wk"].astype(dtype), w["wv"].astype(dtype)], rnd)
        q, k, v = q.reshape(M, H, hd), k.reshape(M, H, hd), v.reshape(M, H, hd)
        q = rnd(rope(q, pos, model.rope_theta))
        k = rnd(rope(k, pos, model.rope_theta))
        v = rnd(v)
        fresh_k.append(k)
        fresh_v.append(v)
        if ctx_k is not None and len(ctx_k[l]) > 0:
            k_all = np.concatenate([ctx_k[l].astype(dtype), k], axis=0)
            v_all = np.concatenate([ctx_v[l].astype(dtype), v], axis=0)
        else:
            k_all, v_all = k, v
        o = rnd(attention(q, k_all, v_all, vis)).reshape(M, d)
        h = h + o @ w["wo"].astype(dtype).T
        gate, up = normed_projection(h, w["g2"].astype(dtype), model.rms_eps,
                                     [w["wg"].astype(dtype), w["wu"].astype(dtype)], rnd)
        g = rnd(silu(gate) * up)
        h = h + g @ w["wd"].astype(dtype).T
    if return_hidden or model.lm_head is None:
        return h, fresh_k, fresh_v
    if logit_rows is not None:
        h = h[logit_rows]
    logits, = normed_projection(h, model.final_gain.astype(dtype), model.rms_eps, [model.lm_head.astype(dtype)], rnd)
    return logits, fresh_k, fresh_v


def confidence(logits: np.ndarray, mask_id: int):
    """Greedy token and its softmax probability per row (Section 3, Observation 3).

    Readings: temperature 0 (greedy); [MASK] can never be predicted (its logit is set to
    -inf, otherwise a committed [MASK] would never make progress); argmax ties go to the
    lowest id.  conf = 1 / sum_j exp(l_j - l_max).  Logits are taken at fp32, the precision
    the kernel decides in; the sum runs in float64 and the result is rounded to fp32.
    """
    l = logits.astype(np.float32).astype(np.float64)
    l[:, mask_id] = -np.inf
    tok = np.argmax(l, axis=1).astype(np.int32)
    m = l.max(axis=1, keepdims=True)
    conf = 1.0 / np.exp(l - m).sum(axis=1)
    return conf.astype(np.float32), tok


# ----------------------------------------------------------------------------- refresh / step

def refresh_prefill(model: Model, x: np.ndarray, T: int, s: int, *, faithful=True,
                    dtype=np.float64, return_logits=False):
    """Block-boundary refresh (Sections 1, 2.1, 4.1): an unmasked bidirectional forward over
    all T positions that rewrites the K/V cache of every position and layer and yields the
    prediction (conf, tok) of every response row from the block start s to T."""
    tok = np.asarray(x[:T], dtype=np.int64)
    pos = np.arange(T)
    vis = np.ones((T, T), dtype=bool)
    logits, fk, fv = forward_rows(model, tok, pos, None, None, vis, faithful=faithful,
                                  dtype=dtype, logit_rows=np.arange(s, T))
    cache = Cache(k=fk, v=fv, length=T)
    if model.lm_head is None:
        return cache, None, None
    conf, pred = confidence(logits, model.mask_id)
    if return_logits:
        return cache, conf, pred, logits
    return cache, conf, pred


def copy_subsets(n_ranks: int, n_copies: int, stage2: bool) -> list:
    """Rank subsets of the block copies, copy 0 (no speculative fill) first.

    Stage 1 (Section 4.2.1): {}, {1}, {2}, {1,2}.  Stage 2 (Section 4.2.2) adds {3}, {1,2,3},
    {4}, {1,2,3,4}.  Copies that need a rank that does not exist (fewer masked positions
    than candidates) are dropped."""
    if n_copies <= 1:
        return [()]
    subsets = [(), (1,), (2,), (1, 2)]
    if stage2:
        subsets += [(3,), (1, 2, 3), (4,), (1, 2, 3, 4)]
    return [y for y in subsets if all(r <= n_ranks for r in y)]


def build_rows(x: np.ndarray, s: int, e: int, mask_id: int, subsets: list, rank_pos: list,
               rank_tok: list, stage2: bool):
    """Row table of one step: for each copy the block positions it computes and their input
    ids.  Stage 1: every copy holds the whole block.  Stage 2 (caption of Fig. 8, Section
    4.2.2): copy 0 holds the whole block; a speculative copy holds only the positions still
    masked in the committed state.  Position ids are the true positions in every copy.
    Returns arrays (copy, pos, tok) over rows."""
    r_copy, r_pos, r_tok = [], [], []
    for c, y in enumerate(subsets):
        fills = {rank_pos[r - 1]: rank_tok[r - 1] for r in y}
        for p in range(s, e):
            if stage2 and c > 0 and x[p] != mask_id:
                continue
            r_copy.append(c)
            r_pos.append(p)
            r_tok.append(fills.get(p, x[p]))
    return np.array(r_copy), np.array(r_pos), np.array(r_tok, dtype=np.int64)


def step_visibility(x, s, e, T, mask_id, r_copy, r_pos, stage2):
    """Which keys each row of a step sees (Section 4.2: copies see the cached context and
    stay mutually invisible; Section 4.2.2: decoded tokens are computed once in copy 0 and
    their K/V shared with every speculative copy).  Keys: the cached positions outside the
    block, [0,s) then [e,T), followed by the step's own rows.  The block's stale cached rows
    are not visible: the fresh rows stand in for them."""
    n_ctx = s + (T - e)
    M = len(r_copy)
    vis = np.zeros((M, n_ctx + M), dtype=bool)
    vis[:, :n_ctx] = True
    same = r_copy[:, None] == r_copy[None, :]
    vis[:, n_ctx:] = same
    if stage2:
        decoded_key = (r_copy == 0) & (x[r_pos] != mask_id)            # copy-0 rows at decoded positions
        spec_row = r_copy > 0
        vis[:, n_ctx:] |= spec_row[:, None] & decoded_key[None, :]
    return vis


def block_decode_step(model: Model, cache: Cache, x: np.ndarray, T: int, s: int, e: int,
                      subsets: list, rank_pos: list, rank_tok: list, stage2: bool, *,
                      faithful=True, dtype=np.float64, return_logits=False):
    """One decoding iteration of block [s,e) over all its copies.

    Returns conf, tok of shape [n_copies][e-s]; entries of positions a copy does not compute
    (stage 2, decoded positions) are conf = -1, tok = -1."""
    r_copy, r_pos, r_tok = build_rows(x, s, e, model.mask_id, subsets, rank_pos, rank_tok, stage2)
    vis = step_visibility(x, s, e, T, model.mask_id, r_copy, r_pos, stage2)
    ctx = np.concatenate([np.arange(0, s), np.arange(e, T)]).astype(np.int64)
    ctx_k = [k[ctx] for k in cache.k]
    ctx_v = [v[ctx] for v in cache.v]
    out, _, _ = forward_rows(model, r_tok, r_pos, ctx_k, ctx_v, vis, faithful=faithful, dtype=dtype)
    if model.lm_head is None:
        return out, r_copy, r_pos
    conf_r, tok_r = confidence(out, model.mask_id)
    C, B = len(subsets), e - s
    conf = np.full((C, B), -1.0, dtype=np.float32)
    tok = np.full((C, B), -1, dtype=np.int32)
    conf[r_copy, r_pos - s] = conf_r
    tok[r_copy, r_pos - s] = tok_r
    if return_logits:
        return conf, tok, out, r_copy, r_pos
    return conf, tok


# ----------------------------------------------------------------------------- control

def accept_set(conf: np.ndarray, masked: np.ndarray, tau: float) -> np.ndarray:
    """Threshold accept rule (Section 3, Observation 3) over the positions masked in the
    copy's input: every position whose confidence exceeds tau (strict), and if none does,
    the single most confident one (lowest position on an exact tie), so an iteration always
    makes progress.  conf fp32 [B], masked bool [B] -> bool [B]."""
    acc = masked & (conf.astype(np.float32) > np.float32(tau))
    if not acc.any() and masked.any():
        c = np.where(masked, conf.astype(np.float32), np.float32(-np.inf))
        acc[int(np.argmax(c))] = True
    return acc


def reverse_step_unmask(masked: np.ndarray, u: np.ndarray, k: int, n_steps: int) -> np.ndarray:
    """The stochastic reverse step of the masked-diffusion process (Section 2.1, Eq. 1), as the unmask decision
    of iteration k = 0 .. n_steps-1 of a block decoded in n_steps iterations.

    Noise levels fall linearly over the block's iterations, t = 1 - k / n_steps to s = 1 - (k + 1) / n_steps.
    A position that is not masked keeps its token (first case of Eq. 1).  A masked position stays masked with
    probability s / t = (n_steps - k - 1) / (n_steps - k) (second case) and is otherwise given a token of the
    model's clean-token distribution (third case); u holds one uniform [0, 1) deviate per position, and a
    position is unmasked iff u >= s / t, compared in fp32.  The last iteration (s = 0) unmasks everything left.
    Reading: the token itself is taken greedily (the distribution sampled at temperature 0, as everywhere in this
    build); the paper's method replaces this stochastic schedule by the confidence threshold (Section 3).
    masked bool [B], u fp32 [B] -> bool [B]."""
    if k >= n_steps - 1:
        return masked.copy()
    stay = np.float32(n_steps - k - 1) / np.float32(n_steps - k)
    return masked & (np.asarray(u, dtype=np.float32) >= stay)


def decision_margin(conf: np.ndarray, masked: np.ndarray, tau: float, k_ranks: int = 0,
                    still_masked: Optional[np.ndarray] = None, relative: bool = True) -> float:
    """How close the decisions taken on this row of confidences are to flipping.  Diagnostic only
    (tells a near-tie from a real disagreement); decides nothing.

    The decisions are those of `accept_set` followed by `rank_candidates` on what stays masked:
      (a) threshold: every masked confidence against tau            -> |c - tau| / tau;
      (b) fallback, only when nothing exceeds tau: best against runner-up -> (c0 - c1) / c0;
      (c) ranking of the positions still masked AFTER the accept: the k_ranks most confident among
          them, each against the next one down (the last of them against the first one left out)
                                                                      -> (c_i - c_{i+1}) / c_i.
    Returns the smallest of these gaps (relative as written, or plain differences with
    relative=False); inf when no position is masked.  Positions that are accepted take no part in
    (c): their order among themselves decides nothing.  `still_masked` names the positions ranked
    in (c) when they are not simply `masked` minus this row's accept set (after a jump chain:
    minus everything the chain committed)."""
    idx = np.flatnonzero(masked)
    if len(idx) == 0:
        return np.inf
    c = conf[idx].astype(np.float32).astype(np.float64)
    over = (lambda v: max(abs(v), 1e-30)) if relative else (lambda v: 1.0)
    with np.errstate(invalid="ignore"):
        m = float(np.min(np.abs(c - tau))) / over(tau)
    acc = accept_set(conf, masked, tau)[idx]
    if not (c > np.float32(tau)).any() and len(c) > 1:
        top = np.sort(c)[::-1]
        m = min(m, float(top[0] - top[1]) / over(top[0]))
    if still_masked is None:
        rest = np.sort(c[~acc])[::-1]
    else:
        rest = np.sort(conf[np.flatnonzero(still_masked)].astype(np.float32).astype(np.float64))[::-1]
    for i in range(min(k_ranks, len(rest) - 1)):
        m = min(m, float(rest[i] - rest[i + 1]) / over(rest[i]))
    return m


def conf_logit(c):
    """ln(c / (1 - c)) of a confidence, clipped to +-16.  A perturbation of every logit of the row by
    at most eps moves this quantity by at most 2 eps (c is the softmax probability of the row's best
    entry), so distances between decisions are measured in it.  Diagnostic only."""
    c = np.clip(np.asarray(c, dtype=np.float64), 1e-7, 1.0 - 1e-7)
    return np.log(c) - np.log1p(-c)


def top2_gap(logits: np.ndarray, mask_id: int) -> np.ndarray:
    """Per row: best logit minus second-best logit, on the fp32 values the greedy token is decided
    on, [MASK] excluded.  Diagnostic only: the distance of each argmax from flipping."""
    l = logits.astype(np.float32).astype(np.float64)
    l[:, mask_id] = -np.inf
    top = np.partition(l, -2, axis=1)[:, -2:]
    return np.abs(top[:, 1] - top[:, 0])


def walk_diagnostics(conf: np.ndarray, gaps: np.ndarray, masked0: np.ndarray, subsets: list, rank_off: list,
                     visited: list, new: dict, tau: float, k_ranks: int) -> dict:
    """Distance of one iteration's decisions from flipping.  Diagnostic only.

    conf [copies][B] and gaps [copies][B] (top2_gap per row) are the iteration's outputs, `visited`
    the copies whose outputs decided something (the jump chain; the main block too when one block is
    picked), `new` what the iteration committed.  In every visited copy the accept decisions count
    over the positions masked in that copy's input; the last visited copy also ranks what is left
    for the next candidates.  Greedy tokens count where they are used: at accepted positions and at
    the next candidates.
    Returns margin (decision_margin, relative, in confidence), sep (the same gaps as plain
    differences of conf_logit) and tok_gap (smallest top-2 logit gap among the tokens used)."""
    left = masked0.copy()
    left[np.array(list(new.keys()), dtype=np.int64)] = False
    last = visited[-1]
    tau_l = float(conf_logit(tau)) if 0.0 < tau < 1.0 else (np.inf if tau >= 1.0 else -np.inf)
    out = {"margin": np.inf, "sep": np.inf, "tok_gap": np.inf}
    for c in visited:
        m_c = masked0.copy()
        m_c[np.array([rank_off[r - 1] for r in subsets[c]], dtype=np.int64)] = False   # its fills are not masked in its input
        if not m_c.any():
            continue
        kk, lm = (k_ranks, left) if c == last else (0, None)
        out["margin"] = min(out["margin"], decision_margin(conf[c], m_c, tau, kk, lm))
        out["sep"] = min(out["sep"], decision_margin(conf_logit(conf[c]), m_c, tau_l, kk, lm, relative=False))
        used = [int(i) for i in np.flatnonzero(accept_set(conf[c], m_c, tau))]
        if c == last:
            used += rank_candidates(conf[c], left, k_ranks)
        out["tok_gap"] = min(out["tok_gap"], float(gaps[c][used].min()))
    return out


def rank_candidates(conf: np.ndarray, masked: np.ndarray, k: int) -> list:
    """Speculative candidates (Section 4.2): the k most confident still-masked positions
    (all of them are below the accept threshold), descending, ties to the lower position."""
    idx = [int(i) for i in np.flatnonzero(masked)]
    idx.sort(key=lambda i: (-float(np.float32(conf[i])), i))
    return idx[:k]


def jump_walk(conf: np.ndarray, tok: np.ndarray, masked0: np.ndarray, subsets: list,
              rank_off: list, rank_tok: list, tau: float):
    """Accept-jump walk over the copies of one step (Section 4.2.1; extended to the eight
    copies of Section 4.2.2 by the same rule).

    Start in copy X = {} (the main block).  In copy X take its accept set over the positions
    masked in X's input; a rank r outside X is *hit* if its position was accepted and the
    copy's token there equals the speculative fill.  Jump to the available copy Y that
    strictly contains X with every added rank hit (largest first, then lowest ranks); stop
    when there is none.  With copies {}, {1}, {2}, {1,2} this is the printed rule: both hit
    -> copy {1,2}; one hit -> its copy, where the other is verified -> {1,2} or stay.

    Committed result (reading; the paper says "incorporate/adopt its decoding"): the union of
    the accept sets along the chain, an earlier link's token winning at a shared position.
    Returns (new_tokens dict offset->token, chain list of copy indices, last copy index).
    """
    B = conf.shape[1]
    cur = 0
    chain = [0]
    new = {}
    while True:
        X = subsets[cur]
        masked = masked0.copy()
        for r in X:
            masked[rank_off[r - 1]] = False
        if not masked.any():
            break
        acc = accept_set(conf[cur], masked, tau)
        for i in np.flatnonzero(acc):
            new.setdefault(int(i), int(tok[cur][i]))
        hit = {r for r in range(1, len(rank_off) + 1)
               if r not in X and acc[rank_off[r - 1]] and tok[cur][rank_off[r - 1]] == rank_tok[r - 1]}
        best = None
        for ci, Y in enumerate(subsets):
            if len(Y) > len(X) and set(X) < set(Y) and (set(Y) - set(X)) <= hit:
                key = (-len(Y), Y)
                if best is None or key < best[0]:
                    best = (key, ci)
        if best is None:
            break
        cur = best[1]
        chain.append(cur)
    return new, chain, cur


def pick_best_walk(conf: np.ndarray, tok: np.ndarray, masked0: np.ndarray, subsets: list,
                   rank_off: list, rank_tok: list, tau: float):
    """The speculation the paper compares against ("traditional dLLM speculative", Fig. 7(a); the
    "vanilla speculation" of Section 5.3): the same copies, but one of them is picked and its
    decoding replaces the main block's.  The candidates are verified in the main block only (hit =
    accepted there with the speculated token); the copy filling the largest set of hit candidates
    is adopted (lowest ranks on a tie, the main block if nothing is hit): its fills and its own
    accept set are committed, nothing else.  No candidate is verified inside a copy and no second
    jump is made, so every step is one state change: the chain has the adopted copy as its only
    link, which is why Section 5.3 can say that Eff_NFE equals NFE for this variant.
    Reading: the paper describes this variant only by that property and by "pick"-ing among the
    appended blocks; the main block's other accepted tokens are not carried over (they are the
    output of a block that was not adopted).
    Returns (new_tokens dict offset->token, chain [adopted copy], adopted copy index)."""
    acc0 = accept_set(conf[0], masked0, tau)
    hit = {r for r in range(1, len(rank_off) + 1)
           if acc0[rank_off[r - 1]] and tok[0][rank_off[r - 1]] == rank_tok[r - 1]}
    best = None
    for ci, Y in enumerate(subsets):
        if len(Y) > 0 and set(Y) <= hit:
            key = (-len(Y), Y)
            if best is None or key < best[0]:
                best = (key, ci)
    if best is None:
        return {int(i): int(tok[0][i]) for i in np.flatnonzero(acc0)}, [0], 0
    cur = best[1]
    new = {int(rank_off[r - 1]): int(rank_tok[r - 1]) for r in subsets[cur]}
    masked = masked0.copy()
    for r in subsets[cur]:
        masked[rank_off[r - 1]] = False
    if masked.any():
        acc = accept_set(conf[cur], masked, tau)
        for i in np.flatnonzero(acc):
            new[int(i)] = int(tok[cur][i])
    return new, [cur], cur


def alp_scan(conf: np.ndarray, tok: np.ndarray, s: int, P: int, eos_id: int, tau_trunc: float):
    """Adaptive length prediction (Section 4.1): scan the refresh's prediction of the whole
    response from the block start on; the first [EOS] whose confidence exceeds the truncate
    threshold cuts the response there (the [EOS] slot is kept).  conf/tok cover positions
    [s, T).  Returns the new response length, or None if unchanged."""
    for i in range(len(tok)):
        if tok[i] == eos_id and np.float32(conf[i]) > np.float32(tau_trunc):
            return (s + i) - P + 1
    return None


@dataclasses.dataclass
class DecodeParams:
    block_len: int
    n_copies: int = 1                 # 1: plain; 4: accept-jump; 8: + decoded-share stage
    accept_threshold: float = 0.9
    truncate_threshold: float = 0.9
    stage2_min_decoded: int = -1      # -1: ceil(4 B / 7), the point where 8 copies fit 4 B rows
    alp: bool = True
    pick_best: bool = False           # the compared "vanilla speculation": pick_best_walk instead of jump_walk
    sampling: bool = False            # Eq. 1's stochastic unmasking (reverse_step_unmask) instead of the threshold rule
    sample_steps: int = 0             # iterations a block is decoded in when sampling (<= 64)


def use_stage2(params: DecodeParams, B: int, n_decoded: int) -> bool:
    """Stage switch (Section 4.2.2 gives no number): decoded-share once the eight-copy layout
    needs no more rows than four full copies, B + 7 (B - n_dec) <= 4 B."""
    if params.n_copies < 8:
        return False
    thr = params.stage2_min_decoded if params.stage2_min_decoded >= 0 else -(-4 * B // 7)
    return n_decoded >= thr


def generate(model: Model, x0: np.ndarray, P: int, params: DecodeParams, *, faithful=True,
             dtype=np.float64, length_schedule: Optional[Callable[[int, int], Optional[int]]] = None,
             max_iters: Optional[int] = None, cache_blocks: bool = True,
             noise: Optional[Callable[[int, int], np.ndarray]] = None):
    """Whole-response generation: per block a refresh (itself a decoding iteration restricted
    to the block), adaptive length prediction, then block steps until the block is full.

    x0: prompt ids followed by [MASK]s.  `length_schedule(block_index, gen_len)` may return a
    shorter response length at a refresh (same lever as ALP; drives the ragged batch
    workload).  cache_blocks=False is the cache-less baseline of Section 1 (bidirectional
    attention without a KV cache: every iteration re-executes the whole prefill), i.e. every
    iteration of a block is a refresh and no block step is ever taken.
    With params.sampling the accept rule of every iteration is Eq. 1's stochastic unmasking
    (reverse_step_unmask; one copy only): noise(block_index, k) gives the uniforms [block_len] of
    iteration k of a block (k = 0 is the refresh); an iteration may unmask nothing.
    Returns (tokens [P + final length], trace list of per-iteration dicts).
    """
    assert not params.sampling or (params.n_copies == 1 and 1 <= params.sample_steps <= 64 and noise is not None)
    x = np.array(x0, dtype=np.int64)
    T = len(x)
    tau = params.accept_threshold
    k_ranks = {1: 0, 4: 2, 8: 4}[params.n_copies]
    trace = []
    b = 0
    while True:
        s = P + b * params.block_len
        if s >= T or (max_iters is not None and len(trace) >= max_iters):
            break
        cache, conf_r, tok_r, logits_r = refresh_prefill(model, x, T, s, faithful=faithful, dtype=dtype,
                                                         return_logits=True)
        newL = alp_scan(conf_r, tok_r, s, P, model.eos_id, params.truncate_threshold) if params.alp else None
        if length_schedule is not None:
            cand = length_schedule(b, T - P)
            if cand is not None and cand > s - P and (newL is None or cand < newL):
                newL = cand
        if newL is not None and P + newL < T:
            T = P + newL
            x = x[:T]
        e = min(s + params.block_len, T)
        B = e - s
        masked = x[s:e] == model.mask_id
        k_iter = 0                                                   # iteration of the block (sampling schedule)
        acc = (reverse_step_unmask(masked, noise(b, 0)[:B], 0, params.sample_steps) if params.sampling
               else accept_set(conf_r[:B], masked, tau))
        for i in np.flatnonzero(acc):
            x[s + i] = tok_r[i]
        if params.sampling:   # no confidence decides anything; the greedy tokens of the unmasked positions do
            g_ = top2_gap(logits_r[:B], model.mask_id)[acc]
            diag = {"margin": np.inf, "sep": np.inf, "tok_gap": float(g_.min()) if len(g_) else np.inf}
        else:
            diag = walk_diagnostics(conf_r[None, :B], top2_gap(logits_r[:B], model.mask_id)[None, :], masked, [()], [], [0],
                                    {int(i): 0 for i in np.flatnonzero(acc)}, tau, k_ranks)
        trace.append({"kind": "refresh", "block": b, "T": T,
                      "accepted": [(int(s + i), int(tok_r[i])) for i in np.flatnonzero(acc)], "chain": [0], **diag})
        last_conf, last_tok = conf_r[:B], tok_r[:B]
        if not cache_blocks:
            if not (x[s:e] == model.mask_id).any():
                b += 1
            continue
        while (x[s:e] == model.mask_id).any():
            if max_iters is not None and len(trace) >= max_iters:
                break
            masked = x[s:e] == model.mask_id
            ranks = rank_candidates(last_conf, masked, k_ranks)
            rank_pos = [s + i for i in ranks]
            rank_tok = [int(last_tok[i]) for i in ranks]
            st2 = use_stage2(params, B, int((~masked).sum()))
            subsets = copy_subsets(len(ranks), 4 if (params.n_copies == 8 and not st2) else params.n_copies, st2)
            conf, tok, logits, r_copy, r_pos = block_decode_step(model, cache, x, T, s, e, subsets, rank_pos, rank_tok,
                                                                 st2, faithful=faithful, dtype=dtype, return_logits=True)
            k_iter += 1
            if params.sampling:
                acc = reverse_step_unmask(masked, noise(b, k_iter)[:B], k_iter, params.sample_steps)
                new, chain, last = {int(i): int(tok[0][i]) for i in np.flatnonzero(acc)}, [0], 0
            else:
                walk = pick_best_walk if params.pick_best else jump_walk
                new, chain, last = walk(conf, tok, masked, subsets, ranks, rank_tok, tau)
            for i, t in new.items():
                x[s + i] = t
            gaps = np.full(conf.shape, np.inf)
            gaps[r_copy, r_pos - s] = top2_gap(logits, model.mask_id)
            visited = chain if not (params.pick_best and chain != [0]) else [0] + chain
            if params.sampling:
                g_ = gaps[0][np.array(list(new.keys()), dtype=np.int64)]
                diag = {"margin": np.inf, "sep": np.inf, "tok_gap": float(g_.min()) if len(g_) else np.inf}
            else:
                diag = walk_diagnostics(conf, gaps, masked, subsets, ranks, visited, new, tau, k_ranks)
            trace.append({"kind": "step", "block": b, "T": T, "stage2": st2,
                          "accepted": sorted((int(s + i), int(t)) for i, t in new.items()),
                          "chain": [int(c) for c in chain], **diag})
            last_conf, last_tok = conf[last], tok[last]
        b += 1
    return x.astype(np.int32), trace


# The three systems the paper compares (Tables 2 and 3), as settings of `generate`:
# the cache-less dLLM baseline (one token per full forward: no confidence passes a threshold of 1),
# Fast-dLLM (DualCache block decoding with threshold acceptance, fixed length, no speculation),
# and the paper's method (adaptive length prediction + jump-share speculation).
def mode_settings(mode: str, block_len: int, n_copies: int = 4, accept_threshold: float = 0.9):
    """Returns (DecodeParams, cache_blocks) for "vanilla", "fast_dllm" or "odb", and for the speculation
    variants of Section 5.3 (Fig. 11), each on block decoding without length prediction: "spec_vanilla"
    (pick one of four blocks), "accept_jump" (four copies, jump chain), "decoded_share" (eight copies)."""
    if mode in ("spec_vanilla", "accept_jump", "decoded_share"):
        return DecodeParams(block_len=block_len, n_copies=8 if mode == "decoded_share" else 4,
                            accept_threshold=accept_threshold, alp=False, pick_best=mode == "spec_vanilla"), True
    if mode == "vanilla":
        return DecodeParams(block_len=block_len, n_copies=1, accept_threshold=1.0, alp=False), False
    if mode == "fast_dllm":
        return DecodeParams(block_len=block_len, n_copies=1, accept_threshold=accept_threshold, alp=False), True
    if mode == "odb":
        return DecodeParams(block_len=block_len, n_copies=n_copies, accept_threshold=accept_threshold, alp=True), True
    raise ValueError(mode)


def trace_counters(trace) -> dict:
    """Counters of Section 5.3: NFE = forward passes (refreshes and block steps alike); Eff_NFE =
    effective state changes of the unmasking sequence = links of the jump chains (equal to NFE
    without speculation); tokens = positions committed."""
    nfe = len(trace)
    eff = sum(len(t["chain"]) for t in trace)
    tokens = sum(len(t["accepted"]) for t in trace)
    return {"nfe": nfe, "eff_nfe": eff, "tokens": tokens, "refreshes": sum(t["kind"] == "refresh" for t in trace),
            "tokens_per_nfe": tokens / nfe if nfe else 0.0}

