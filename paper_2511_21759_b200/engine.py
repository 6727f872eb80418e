"""Thin object layer over the C ABI: owns device buffers (torch tensors), marshals arguments.

`Model` and `Session` mirror odb_model / odb_session.  `generate` is the host control loop of
the method (refresh -> accept, with adaptive length prediction inside the accept and an optional
external length schedule through the same lever -> block steps until the block is full), written
only in terms of the exported calls.  No arithmetic of the method happens in this file.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
from typing import Callable, Optional

import numpy as np
import torch

from . import binding as B


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def bits_to_device(bits: np.ndarray, device) -> torch.Tensor:
    """bf16 bit patterns (numpy uint16) -> torch.bfloat16 tensor on `device` (a re-interpretation)."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device).view(torch.bfloat16)


def pack_weight(w: torch.Tensor) -> torch.Tensor:
    """Row-major bf16 [N][K] on the device -> the library's packed tile layout (odb_pack_weight)."""
    N, K = w.shape
    w = w.contiguous()
    out = torch.empty(B.lib().odb_packed_weight_bytes(N, K) // 2, dtype=torch.bfloat16, device=w.device)
    st = torch.cuda.current_stream(w.device)
    B.check(B.lib().odb_pack_weight(w.data_ptr(), out.data_ptr(), N, K, C.c_void_p(st.cuda_stream)), "odb_pack_weight")
    return out


def pack_gate_up(w: torch.Tensor) -> torch.Tensor:
    """Row-major bf16 [2F][K] (gate rows, then up rows) -> the gate/up packed layout (odb_pack_gate_up)."""
    F2, K = w.shape
    w = w.contiguous()
    out = torch.empty(B.lib().odb_packed_gate_up_bytes(F2 // 2, K) // 2, dtype=torch.bfloat16, device=w.device)
    st = torch.cuda.current_stream(w.device)
    B.check(B.lib().odb_pack_gate_up(w.data_ptr(), out.data_ptr(), F2 // 2, K, C.c_void_p(st.cuda_stream)),
            "odb_pack_gate_up")
    return out


@dataclasses.dataclass
class DecodeParams:
    block_len: int
    n_copies: int = 1
    accept_threshold: float = 0.9
    truncate_threshold: float = 0.9
    stage2_min_decoded: int = -1
    alp: bool = True
    pick_best: bool = False
    sampling: bool = False
    sample_steps: int = 0

    def c(self) -> B.odb_decode_params:
        return B.odb_decode_params(self.block_len, self.n_copies, self.accept_threshold, self.truncate_threshold,
                                   self.stage2_min_decoded, 1 if self.alp else 0, 1 if self.pick_best else 0,
                                   1 if self.sampling else 0, self.sample_steps)


class Model:
    """Device-resident weights + the library's model handle."""

    def __init__(self, shape, tensors: dict, *, max_batch=1, max_seq=2048, max_block=64, max_copies=8,
                 with_lm_head=True, tp=(0, 0)):
        """tensors: embed, lm_head (or None), final_norm, and lists norm1, wqkv, wo, norm2, wgu, wd.
        tp = (world, rank): the tensors are that tensor-parallel rank's shard (see odb.h); (0, 0): the whole model."""
        self.shape = shape
        self.t = tensors
        nl = shape.n_layers
        self.cfg = B.odb_config(nl, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                                shape.mask_id, shape.eos_id, shape.rope_theta, shape.rms_eps,
                                max_batch, max_seq, max_block, max_copies, 1 if with_lm_head else 0, tp[0], tp[1])
        arr = lambda name: (C.c_void_p * nl)(*[tensors[name][l].data_ptr() for l in range(nl)])
        self._arrays = {n: arr(n) for n in ("norm1", "wqkv", "wo", "norm2", "wgu", "wd")}
        w = B.odb_weights(_ptr(tensors["embed"]), _ptr(tensors.get("lm_head")) if with_lm_head else None,
                          _ptr(tensors["final_norm"]),
                          *[C.cast(self._arrays[n], C.POINTER(C.c_void_p))
                            for n in ("norm1", "wqkv", "wo", "norm2", "wgu", "wd")])
        self.handle = C.c_void_p()
        B.check(B.lib().odb_model_create(C.byref(self.cfg), C.byref(w), C.byref(self.handle)), "odb_model_create")

    @classmethod
    def from_synth(cls, shape, seed=0, device="cuda", *, with_lm_head=True, lm_head_bits=None, **kw) -> "Model":
        """Uploads the seeded synthetic weights of `shape` (data marshalling only).  lm_head_bits
        (bf16 bit patterns [V][d]) replaces the generated LM head when given."""
        import synth
        d = shape.d_model
        ones = lambda: torch.ones(d, dtype=torch.float32, device=device)
        t = {"embed": bits_to_device(synth.embed_bits(shape, seed), device),
             "lm_head": pack_weight(bits_to_device(lm_head_bits if lm_head_bits is not None
                                                   else synth.lm_head_bits(shape, seed), device)) if with_lm_head else None,
             "final_norm": ones(), "norm1": [], "wqkv": [], "wo": [], "norm2": [], "wgu": [], "wd": []}
        for l in range(shape.n_layers):
            w = synth.layer_bits(shape, l, seed)
            t["norm1"].append(ones())
            t["norm2"].append(ones())
            t["wqkv"].append(pack_weight(bits_to_device(np.concatenate([w["wq"], w["wk"], w["wv"]], axis=0), device)))
            t["wo"].append(pack_weight(bits_to_device(w["wo"], device)))
            t["wgu"].append(pack_gate_up(bits_to_device(np.concatenate([w["wg"], w["wu"]], axis=0), device)))
            t["wd"].append(pack_weight(bits_to_device(w["wd"], device)))
        return cls(shape, t, with_lm_head=with_lm_head, **kw)

    def close(self):
        if self.handle:
            B.lib().odb_model_destroy(self.handle)
            self.handle = C.c_void_p()

    def step_algorithmic_bytes(self, keys: int) -> float:
        return B.lib().odb_step_algorithmic_bytes(C.byref(self.cfg), keys)


class Session:
    def __init__(self, model: Model, stream: Optional[torch.cuda.Stream] = None, poison: bool = False, zero: bool = False):
        """poison: hand the library a workspace and a K/V cache filled with 0xFF bytes (NaN as fp32 and as bf16), so
        that a kernel reading memory nothing has written shows up as NaN in the results (tests).  zero: zero-filled
        buffers instead (a tensor-parallel rank run without its peers then adds zeros for their partial sums)."""
        self.model = model
        lib = B.lib()
        dev = model.t["embed"].device
        self.kv = torch.empty(lib.odb_kv_bytes(C.byref(model.cfg)), dtype=torch.uint8, device=dev)
        self.ws = torch.empty(lib.odb_workspace_bytes(C.byref(model.cfg)), dtype=torch.uint8, device=dev)
        if poison:
            self.kv.fill_(0xFF)
            self.ws.fill_(0xFF)
        elif zero:
            self.kv.zero_()
            self.ws.zero_()
        self.stream = stream if stream is not None else torch.cuda.current_stream(dev)
        self.handle = C.c_void_p()
        B.check(lib.odb_session_create(model.handle, self.kv.data_ptr(), self.kv.numel(), self.ws.data_ptr(),
                                       self.ws.numel(), C.c_void_p(self.stream.cuda_stream), C.byref(self.handle)),
                "odb_session_create")
        self.nb = model.cfg.max_batch
        self._results = (B.odb_result * self.nb)()
        self.gen_len = {}        # seq -> current response length (host copy, for the control loop)
        self.prompt_len = {}

    def close(self):
        if self.handle:
            B.lib().odb_session_destroy(self.handle)
            self.handle = C.c_void_p()

    def set_sequence(self, seq: int, ids: np.ndarray, prompt_len: int):
        ids = np.ascontiguousarray(ids, dtype=np.int32)
        B.check(B.lib().odb_session_set_sequence(self.handle, seq, ids.ctypes.data, prompt_len, len(ids) - prompt_len),
                "odb_session_set_sequence")
        self.gen_len[seq] = len(ids) - prompt_len
        self.prompt_len[seq] = prompt_len

    def set_gen_len(self, seq: int, new_len: int):
        B.check(B.lib().odb_session_set_gen_len(self.handle, seq, new_len), "odb_session_set_gen_len")
        self.gen_len[seq] = new_len

    def set_sampling_noise(self, seq: int, u: np.ndarray):
        """u [iterations][block_len]: the uniform deviates of the stochastic reverse step for the block the next
        refresh opens (data of the caller's; nothing is drawn here)."""
        u = np.ascontiguousarray(u, dtype=np.float32)
        B.check(B.lib().odb_session_set_sampling_noise(self.handle, seq, u.ctypes.data, u.shape[0], u.shape[1]),
                "odb_session_set_sampling_noise")

    def set_active(self, seq: int, active: bool):
        B.check(B.lib().odb_session_set_active(self.handle, seq, 1 if active else 0), "odb_session_set_active")

    def get_tokens(self, seq: int) -> np.ndarray:
        out = np.empty(self.model.cfg.max_seq, dtype=np.int32)
        n = C.c_int32()
        B.check(B.lib().odb_session_get_tokens(self.handle, seq, out.ctypes.data, len(out), C.byref(n)),
                "odb_session_get_tokens")
        return out[: n.value].copy()

    def status(self) -> int:
        return B.lib().odb_session_status(self.handle)

    def refresh_prefill(self, params: DecodeParams, block_index):
        bi = np.ascontiguousarray(np.broadcast_to(np.asarray(block_index, dtype=np.int32), (self.nb,)))
        p = params.c()
        B.check(B.lib().odb_refresh_prefill(self.handle, C.byref(p), bi.ctypes.data), "odb_refresh_prefill")

    def block_decode_step(self, params: DecodeParams):
        p = params.c()
        B.check(B.lib().odb_block_decode_step(self.handle, C.byref(p)), "odb_block_decode_step")

    def unmask_accept(self, params: DecodeParams, after_refresh: bool):
        p = params.c()
        B.check(B.lib().odb_unmask_accept(self.handle, C.byref(p), 1 if after_refresh else 0, self._results),
                "odb_unmask_accept")
        return self._results

    def decode_block_resident(self, params: DecodeParams, max_iters: int = 0):
        """The device-resident loop: steps and accepts of the open blocks until they close, the step's shape
        changes or max_iters iterations have run.  Returns a list with one entry per iteration, each the
        per-sequence results of that iteration's accept (copies: they stay valid)."""
        p = params.c()
        cap = 64 if max_iters <= 0 else min(max_iters, 64)
        log = (B.odb_result * (cap * self.nb))()
        n = C.c_int32()
        B.check(B.lib().odb_decode_block_resident(self.handle, C.byref(p), max_iters, log, cap, C.byref(n)),
                "odb_decode_block_resident")
        return [[log[i * self.nb + j] for j in range(self.nb)] for i in range(n.value)]

    def set_logit_dump(self, enable: bool):
        """Test mode: the LM head writes fp32 logits (debug_read("logits")) instead of fusing the reduction."""
        B.check(B.lib().odb_debug_set_logit_dump(self.handle, 1 if enable else 0), "odb_debug_set_logit_dump")

    def profile(self, enable: bool):
        B.check(B.lib().odb_session_profile(self.handle, 1 if enable else 0), "odb_session_profile")

    def profile_read(self):
        """({kind: ms}, {kind: launches}) since the last read."""
        ms = (C.c_double * len(B.KINDS))()
        n = (C.c_int64 * len(B.KINDS))()
        B.check(B.lib().odb_session_profile_read(self.handle, ms, n), "odb_session_profile_read")
        return dict(zip(B.KINDS, list(ms))), dict(zip(B.KINDS, list(n)))

    def persistent_barrier_times(self, n_ctas: int, n_barriers: int) -> np.ndarray:
        """[CTA][barrier][arrived, released] global-timer values (ns) of the last persistent step (needs
        ODB_PERSISTENT=1 and ODB_PERSISTENT_TIMING=1 in the environment when the library was loaded)."""
        buf = np.zeros(n_ctas * n_barriers * 2, dtype=np.uint64)
        rows = C.c_int32()
        B.check(B.lib().odb_debug_read(self.handle, 11, buf.ctypes.data, buf.nbytes, C.byref(rows)), "odb_debug_read")
        return buf.reshape(n_ctas, n_barriers, 2).astype(np.int64)

    _READ = {"logits": (0, np.float32), "conf": (1, np.float32), "tok": (2, np.int32), "hidden": (3, np.float32),
             "q": (4, np.uint16), "k": (5, np.uint16), "v": (6, np.uint16), "o": (7, np.uint16),
             "row_tok": (8, np.int32), "row_pos": (9, np.int32), "row_copy": (10, np.int32)}

    def debug_read(self, what: str) -> np.ndarray:
        which, dt = self._READ[what]
        cfg = self.model.cfg
        da = cfg.d_model // max(cfg.tp_world, 1)      # q / k / v / o rows hold this rank's heads
        width = {"logits": cfg.vocab, "hidden": cfg.d_model, "q": da, "k": da, "v": da, "o": da}.get(what, 1)
        cap_rows = self.ws.numel() // (width * np.dtype(dt).itemsize)
        cap_rows = min(cap_rows, cfg.max_batch * max(cfg.max_seq, cfg.max_copies * cfg.max_block))
        buf = np.empty(cap_rows * width, dtype=dt)
        rows = C.c_int32()
        B.check(B.lib().odb_debug_read(self.handle, which, buf.ctypes.data, buf.nbytes, C.byref(rows)), "odb_debug_read")
        out = buf[: rows.value * width]
        return out.reshape(rows.value, width).copy() if width > 1 else out.copy()


def debug_gemm(x: torch.Tensor, w: torch.Tensor, k_splits: int = 0) -> torch.Tensor:
    """out[M][N] fp32 = x[M][K] @ w[N][K]^T through the library's tcgen05 GEMM (w row-major here; it is
    packed with odb_pack_weight first)."""
    M, K = x.shape
    N = w.shape[0]
    w = pack_weight(w)
    out = torch.empty(M, N, dtype=torch.float32, device=x.device)
    scratch = torch.empty(max(k_splits, 16) * M * N * 4 + 1024, dtype=torch.uint8, device=x.device)
    st = torch.cuda.current_stream(x.device)
    B.check(B.lib().odb_debug_gemm(x.data_ptr(), w.data_ptr(), out.data_ptr(), scratch.data_ptr(), scratch.numel(),
                                   M, N, K, k_splits, C.c_void_p(st.cuda_stream)), "odb_debug_gemm")
    return out


def measure_read_bandwidth(n_bytes: int = 4 << 30, reps: int = 4, device="cuda", bulk: bool = False) -> float:
    """GB/s of a read-only stream over a buffer of n_bytes: 16-byte loads (odb_measure_read_bandwidth) or, with
    bulk=True, rings of bulk copies as the projections' weights are fetched (odb_measure_bulk_read_bandwidth)."""
    buf = torch.empty(n_bytes, dtype=torch.uint8, device=device)
    buf.fill_(1)
    st = torch.cuda.current_stream(buf.device)
    out = C.c_double()
    name = "odb_measure_bulk_read_bandwidth" if bulk else "odb_measure_read_bandwidth"
    B.check(getattr(B.lib(), name)(buf.data_ptr(), buf.numel(), reps, C.c_void_p(st.cuda_stream), C.byref(out)), name)
    return out.value


def gemm_static_scratch(x: torch.Tensor, w: torch.Tensor, k_splits: int = 0) -> torch.Tensor:
    """Same product as debug_gemm through odb_gemm_static_scratch: the library keeps the split-K
    partial sums in its own fixed device array, so the call itself allocates nothing (the tensors
    created here are the caller's inputs and output)."""
    M, K = x.shape
    N = w.shape[0]
    w = pack_weight(w)
    out = torch.empty(M, N, dtype=torch.float32, device=x.device)
    st = torch.cuda.current_stream(x.device)
    B.check(B.lib().odb_gemm_static_scratch(x.data_ptr(), w.data_ptr(), out.data_ptr(), M, N, K, k_splits,
                                            C.c_void_p(st.cuda_stream)), "odb_gemm_static_scratch")
    return out


def generate(sess: Session, params: DecodeParams, *,
             length_schedule: Optional[Callable[[int, int, int], Optional[int]]] = None,
             max_iters: Optional[int] = None, cache_blocks: bool = True, resident: bool = False,
             start_block: int = 0, noise: Optional[Callable[[int, int], np.ndarray]] = None):
    """Runs every sequence set on the session to completion.

    Per iteration: the sequences standing at a block boundary are refreshed and accepted
    together (the others wait); otherwise every sequence with an open block takes one block
    step and its accept.  length_schedule(seq, block_index, gen_len) may return a shorter
    response length, applied between the refresh and its accept (the lever adaptive length
    prediction also pulls).  Returns ({seq: tokens}, trace); trace is a list of per-call dicts
    {"kind", "seqs": {seq: {"accepted", "chain", "masks_left", "gen_len", "block"}}}.
    cache_blocks=False is the cache-less baseline (Section 1): every iteration of a block is a
    refresh prefill and no block step is taken.  resident=True runs the steps of a block through the
    device-resident loop (same trace, one host round trip per block instead of one per iteration).
    start_block: the block every sequence starts at (a resumed session: the blocks before it are already
    decoded in the ids given to set_sequence; the refresh of start_block recomputes the whole cache).
    noise(seq, block_index) -> [sample_steps][block_len] uniforms, handed to the session before the block's refresh
    when params.sampling is set."""
    seqs = sorted(sess.gen_len)
    block = {i: start_block for i in seqs}
    need_refresh = {i: True for i in seqs}
    done = {i: False for i in seqs}
    trace = []

    def record(res, kind, which):
        rec = {"kind": kind, "seqs": {}}
        for i in which:
            r = res[i]
            rec["seqs"][i] = {
                "accepted": sorted((r.accepted_pos[j], r.accepted_tok[j]) for j in range(min(r.n_accepted, 64))),
                "chain": [r.chain[j] for j in range(min(r.chain_len, B.ODB_MAX_CHAIN))],
                "masks_left": r.masks_left, "gen_len": r.gen_len, "block": (r.block_start, r.block_end)}
        trace.append(rec)

    while max_iters is None or len(trace) < max_iters:
        todo = [i for i in seqs if not done[i]]
        if not todo:
            break
        refresh = [i for i in todo if need_refresh[i]]
        if refresh:
            bi = [-1] * sess.nb
            for i in refresh:
                bi[i] = block[i]
            if params.sampling:
                for i in refresh:
                    sess.set_sampling_noise(i, noise(i, block[i]))
            sess.refresh_prefill(params, bi)
            if length_schedule is not None:
                for i in refresh:
                    new = length_schedule(i, block[i], sess.gen_len[i])
                    if new is not None and block[i] * params.block_len < new < sess.gen_len[i]:
                        sess.set_gen_len(i, new)
            res = sess.unmask_accept(params, True)
            record(res, "refresh", refresh)
            touched = refresh
        elif resident:
            left = 0 if max_iters is None else max_iters - len(trace)
            for res in sess.decode_block_resident(params, left):
                record(res, "step", todo)
            touched = todo
        else:
            sess.block_decode_step(params)
            res = sess.unmask_accept(params, False)
            record(res, "step", todo)
            touched = todo
        for i in touched:
            sess.gen_len[i] = res[i].gen_len
            need_refresh[i] = not cache_blocks
            if res[i].masks_left == 0:
                block[i] += 1
                if block[i] * params.block_len >= sess.gen_len[i]:
                    done[i] = True
                    sess.set_active(i, False)
                else:
                    need_refresh[i] = True
    return {i: sess.get_tokens(i) for i in seqs}, trace


def mode_settings(mode: str, block_len: int, n_copies: int = 4, accept_threshold: float = 0.9):
    """(DecodeParams, cache_blocks) of the three systems of Tables 2 and 3: "vanilla" (no cache, one
    token per full forward), "fast_dllm" (DualCache block decoding, threshold acceptance, fixed
    length) and "odb" (adaptive length prediction + jump-share speculation); and of the speculation
    variants of Section 5.3 (Fig. 11), each on block decoding without length prediction: "spec_vanilla"
    (one of four blocks is picked), "accept_jump" (four copies, jump chain), "decoded_share" (eight copies)."""
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


def trace_counters(trace, seq: int = 0) -> dict:
    """Section 5.3's counters for one sequence of a `generate` trace: NFE (forward passes), Eff_NFE
    (links of the jump chains = effective state changes), committed tokens."""
    recs = [t for t in trace if seq in t["seqs"]]
    nfe = len(recs)
    eff = sum(len(t["seqs"][seq]["chain"]) for t in recs)
    tokens = sum(len(t["seqs"][seq]["accepted"]) for t in recs)
    return {"nfe": nfe, "eff_nfe": eff, "tokens": tokens, "refreshes": sum(t["kind"] == "refresh" for t in recs),
            "tokens_per_nfe": tokens / nfe if nfe else 0.0}

