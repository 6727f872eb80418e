"""Tensor-parallel groups over the C ABI (argument marshalling only; every step runs in the library's kernels).

Two ways to form a group of R ranks of one model:

* `TPGroupOneGPU`: all R ranks in this process on ONE device and one stream - the test arrangement.  Ranks whose
  kernels wait for one another must not be separate launches on one GPU, so every forward is issued segment by
  segment (odb_debug_tp_segments): segment k of every rank before segment k+1 of any, which raises every flag
  before the kernel that waits for it starts.  It has the methods of `engine.Session`, so the host control loop
  (`engine.generate`) and the lock-step test harness drive it unchanged.
* `attach_process_group`: one process per GPU under torch.distributed.  Every rank shares its workspace storage
  through CUDA inter-process memory handles (torch's own storage sharing), gathers the peers' handles and offsets
  with all_gather_object, maps them and hands the pointers to odb_session_tp_attach.  From then on the ordinary
  Session calls run the tensor-parallel forward: the projections' epilogues store into the peers' buffers, flags
  order the exchange on the device.
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional

import numpy as np
import torch

from . import binding as B
from . import engine as E


def vocab_range(cfg: B.odb_config, rank: int):
    first, last = C.c_int32(), C.c_int32()
    B.check(B.lib().odb_tp_vocab_range(C.byref(cfg), rank, C.byref(first), C.byref(last)), "odb_tp_vocab_range")
    return first.value, last.value


def shard_layer(w: dict, shape, rank: int, world: int) -> dict:
    """Rows / columns of one layer's row-major bf16 bit matrices that rank `rank` of `world` holds (views)."""
    hd = shape.head_dim
    hl = shape.n_heads // world
    fl = shape.d_ffn // world
    a0, a1 = rank * hl * hd, (rank + 1) * hl * hd
    f0, f1 = rank * fl, (rank + 1) * fl
    return {"wq": w["wq"][a0:a1], "wk": w["wk"][a0:a1], "wv": w["wv"][a0:a1], "wo": w["wo"][:, a0:a1],
            "wg": w["wg"][f0:f1], "wu": w["wu"][f0:f1], "wd": w["wd"][:, f0:f1]}


def model_shards_from_synth(shape, seed, ranks: List[int], world: int, device="cuda", *, with_lm_head=True,
                            lm_head_bits=None, **kw) -> List[E.Model]:
    """The seeded synthetic model's shards of the given ranks (data marshalling: slicing, upload, packing); every
    layer is generated once and sliced for each rank."""
    import synth
    d = shape.d_model
    ones = lambda: torch.ones(d, dtype=torch.float32, device=device)
    embed = E.bits_to_device(synth.embed_bits(shape, seed), device)      # replicated: one device copy serves every rank here
    lm_bits = (lm_head_bits if lm_head_bits is not None else synth.lm_head_bits(shape, seed)) if with_lm_head else None
    ts = []
    for r in ranks:
        lm = None
        if with_lm_head:
            probe = B.odb_config(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                                 shape.mask_id, shape.eos_id, shape.rope_theta, shape.rms_eps, 1, 2, 1, 1, 1, world, r)
            v0, v1 = vocab_range(probe, r)
            lm = E.pack_weight(E.bits_to_device(lm_bits[v0:v1], device))
        ts.append({"embed": embed, "lm_head": lm, "final_norm": ones(), "norm1": [], "wqkv": [], "wo": [], "norm2": [],
                   "wgu": [], "wd": []})
    for l in range(shape.n_layers):
        full = synth.layer_bits(shape, l, seed)
        for t, r in zip(ts, ranks):
            w = shard_layer(full, shape, r, world)
            t["norm1"].append(ones())
            t["norm2"].append(ones())
            t["wqkv"].append(E.pack_weight(E.bits_to_device(np.concatenate([w["wq"], w["wk"], w["wv"]], axis=0), device)))
            t["wo"].append(E.pack_weight(E.bits_to_device(w["wo"], device)))
            t["wgu"].append(E.pack_gate_up(E.bits_to_device(np.concatenate([w["wg"], w["wu"]], axis=0), device)))
            t["wd"].append(E.pack_weight(E.bits_to_device(w["wd"], device)))
    return [E.Model(shape, t, with_lm_head=with_lm_head, tp=(world, r), **kw) for t, r in zip(ts, ranks)]


def model_shard_from_synth(shape, seed, rank: int, world: int, device="cuda", **kw) -> E.Model:
    """One rank's shard (what a process of a multi-process group uploads)."""
    return model_shards_from_synth(shape, seed, [rank], world, device, **kw)[0]


def tp_buffers(sess: E.Session):
    """(recv_ptr, recv_bytes, flags_ptr, flags_bytes, conf_ptr, conf_bytes) of the regions peers write into."""
    ptr = [C.c_void_p() for _ in range(3)]
    size = [C.c_size_t() for _ in range(3)]
    B.check(B.lib().odb_session_tp_buffers(sess.handle, C.byref(ptr[0]), C.byref(size[0]), C.byref(ptr[1]), C.byref(size[1]),
                                           C.byref(ptr[2]), C.byref(size[2])), "odb_session_tp_buffers")
    return tuple(v for pair in zip((p.value for p in ptr), (s.value for s in size)) for v in pair)


def tp_attach(sess: E.Session, recv: List[Optional[int]], flags: List[Optional[int]], conf: List[Optional[int]]):
    n = len(recv)
    arr = lambda xs: (C.c_void_p * n)(*[C.c_void_p(x) for x in xs])
    B.check(B.lib().odb_session_tp_attach(sess.handle, arr(recv), arr(flags), arr(conf)), "odb_session_tp_attach")


def attach_alone(sess: E.Session):
    """Measurement: the rank as its own peers (every rank's regions = its own) with all flags raised locally, so that
    its steps can be timed on one GPU without the other ranks (odb_debug_tp_alone); results are meaningless."""
    b = tp_buffers(sess)
    n = sess.model.cfg.tp_world
    tp_attach(sess, [b[0]] * n, [b[2]] * n, [b[4]] * n)
    B.check(B.lib().odb_debug_tp_alone(sess.handle, 1), "odb_debug_tp_alone")


def segment_count(cfg: B.odb_config) -> int:
    return B.lib().odb_tp_segment_count(C.byref(cfg))


class TPGroupOneGPU:
    """All ranks of a tensor-parallel group on one device and one stream, forwards issued segment by segment."""

    def __init__(self, shape, seed=0, world=2, device="cuda", *, with_lm_head=True, lm_head_bits=None, poison=False, **kw):
        self.world = world
        self.models = model_shards_from_synth(shape, seed, list(range(world)), world, device, with_lm_head=with_lm_head,
                                              lm_head_bits=lm_head_bits, **kw)
        self.ranks = [E.Session(m, poison=poison) for m in self.models]
        bufs = [tp_buffers(s) for s in self.ranks]
        for s in self.ranks:
            tp_attach(s, [b[0] for b in bufs], [b[2] for b in bufs], [b[4] for b in bufs])
        self.segments = segment_count(self.models[0].cfg)
        self.model = self.models[0]
        self.nb = self.ranks[0].nb
        self.gen_len = self.ranks[0].gen_len
        self.prompt_len = self.ranks[0].prompt_len

    def close(self):
        for s in self.ranks:
            s.close()
        for m in self.models:
            m.close()

    # ---- state: the same on every rank ----
    def set_sequence(self, seq, ids, prompt_len):
        for s in self.ranks:
            s.set_sequence(seq, ids, prompt_len)

    def set_gen_len(self, seq, new_len):
        for s in self.ranks:
            s.set_gen_len(seq, new_len)

    def set_sampling_noise(self, seq, u):
        for s in self.ranks:
            s.set_sampling_noise(seq, u)

    def set_active(self, seq, active):
        for s in self.ranks:
            s.set_active(seq, active)

    def set_logit_dump(self, enable):
        if enable:
            raise ValueError("a tensor-parallel rank holds a slice of the vocabulary: no logits test mode")

    def get_tokens(self, seq):
        toks = [s.get_tokens(seq) for s in self.ranks]
        for t in toks[1:]:
            assert np.array_equal(t, toks[0]), "ranks disagree on the sequence"
        return toks[0]

    def status(self):
        return [s.status() for s in self.ranks]

    # ---- forwards: segment k on every rank before segment k + 1 on any ----
    def _segmented(self, call):
        lib = B.lib()
        for k in range(self.segments):
            for s in self.ranks:
                B.check(lib.odb_debug_tp_segments(s.handle, k, k + 1), "odb_debug_tp_segments")
                call(s)

    def refresh_prefill(self, params, block_index):
        self._segmented(lambda s: s.refresh_prefill(params, block_index))

    def block_decode_step(self, params):
        self._segmented(lambda s: s.block_decode_step(params))

    def unmask_accept(self, params, after_refresh):
        res = [s.unmask_accept(params, after_refresh) for s in self.ranks]
        raw = [bytes(memoryview(r)) for r in res]
        for r in raw[1:]:
            assert r == raw[0], "ranks disagree on the accept"
        return res[0]

    def debug_read(self, what):
        """Rank 0's copy; confidences, tokens and the row table must be identical on every rank."""
        out = self.ranks[0].debug_read(what)
        if what in ("conf", "tok", "row_tok", "row_pos", "row_copy", "hidden"):
            for s in self.ranks[1:]:
                other = s.debug_read(what)
                assert other.tobytes() == out.tobytes(), f"ranks disagree on {what}"
        return out


# ---- one process per GPU ----

def share_workspace(sess: E.Session):
    """What a peer process needs to map this session's workspace: torch's inter-process handle of the storage the
    workspace tensor lives in, and the tensor's offset in it."""
    st = sess.ws.untyped_storage()
    return {"handle": st._share_cuda_(), "tensor_offset": sess.ws.storage_offset()}


def open_workspace(shared) -> torch.Tensor:
    """The peer's workspace as a uint8 tensor of this process (kept alive by the caller for the session's life)."""
    torch.cuda.init()                       # the handle is opened by the CUDA runtime: it must be up in this process
    st = torch.UntypedStorage._new_shared_cuda(*shared["handle"])
    return torch.empty(0, dtype=torch.uint8, device=st.device).set_(st)[shared["tensor_offset"]:]


def peer_pointers(my_rank: int, bufs: List[tuple], bases: List[Optional[int]], my_base: int):
    """Pointers to every rank's three regions in THIS process's address space.  bufs[r] = that rank's tp_buffers()
    in ITS address space together with its workspace base as the last element; bases[r] = where this process mapped
    rank r's workspace (None for itself)."""
    recv, flags, conf = [], [], []
    for r, b in enumerate(bufs):
        their_base = b[6]
        base = my_base if r == my_rank else bases[r]
        recv.append(base + (b[0] - their_base))
        flags.append(base + (b[2] - their_base))
        conf.append(base + (b[4] - their_base))
    return recv, flags, conf


def gather_descriptors(mine, group=None):
    """Every rank's descriptor (any picklable object), in rank order, on every rank."""
    import torch.distributed as dist
    everyone = [None] * dist.get_world_size(group)
    dist.all_gather_object(everyone, mine, group=group)
    return everyone


def attach_process_group(sess: E.Session, group=None):
    """Collective over the ranks of `group` (default group if None): exchanges workspace handles and attaches."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    cfg = sess.model.cfg
    if cfg.tp_world != world or cfg.tp_rank != rank:
        raise ValueError(f"model shard is rank {cfg.tp_rank} of {cfg.tp_world}, process is rank {rank} of {world}")
    device = sess.ws.device.index
    everyone = gather_descriptors({"shared": share_workspace(sess), "bufs": tp_buffers(sess) + (sess.ws.data_ptr(),),
                                   "device": device}, group)
    with torch.cuda.device(device):      # this rank's kernels store into every peer's memory
        for r in range(world):
            if r != rank:
                B.check(B.lib().odb_tp_enable_peer_access(everyone[r]["device"]), "odb_tp_enable_peer_access")
    mapped = [None if r == rank else open_workspace(everyone[r]["shared"]) for r in range(world)]
    recv, flags, conf = peer_pointers(rank, [e["bufs"] for e in everyone],
                                      [None if m is None else m.data_ptr() for m in mapped], sess.ws.data_ptr())
    tp_attach(sess, recv, flags, conf)
    sess._tp_peer_mappings = mapped    # the mappings live as long as the session
    dist.barrier(group=group)
    return mapped
