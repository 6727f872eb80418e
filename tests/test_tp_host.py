"""Host side of the tensor-parallel path, without a GPU: shard geometry the library reports, the slicing of the
weights, the pointer arithmetic of a multi-process attach, and the descriptor exchange between two gloo ranks."""
import ctypes as C
import os
import sys

import numpy as np
import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

import synth
from paper_2511_21759_b200 import binding as B
from paper_2511_21759_b200 import tp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _cfg(shape, world, rank, **kw):
    a = dict(max_batch=1, max_seq=768, max_block=32, max_copies=4, with_lm_head=1)
    a.update(kw)
    return B.odb_config(shape.n_layers, shape.d_model, shape.n_heads, shape.head_dim, shape.d_ffn, shape.vocab,
                        shape.mask_id, shape.eos_id, shape.rope_theta, shape.rms_eps, a["max_batch"], a["max_seq"],
                        a["max_block"], a["max_copies"], a["with_lm_head"], world, rank)


@pytest.mark.parametrize("world", [2, 4, 8])
def test_vocabulary_ranges_partition_the_vocabulary_in_whole_tiles(world):
    shape = synth.LLADA_8B                                      # 126464 ids = 988 tiles of 128
    spans = [tp.vocab_range(_cfg(shape, world, r), r) for r in range(world)]
    assert spans[0][0] == 0 and spans[-1][1] == shape.vocab
    for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
        assert a1 == b0 and a0 < a1                              # contiguous, none empty
    assert all(a0 % 128 == 0 for a0, _ in spans)
    per = -(-988 // world)
    assert [a1 - a0 for a0, a1 in spans[:-1]] == [per * 128] * (world - 1)


def test_shard_configurations_are_validated():
    lib = B.lib()
    ok = _cfg(synth.LLADA_8B, 4, 3)
    whole = _cfg(synth.LLADA_8B, 0, 0)
    assert lib.odb_workspace_bytes(C.byref(ok)) > lib.odb_workspace_bytes(C.byref(whole)) > 0   # + the receive slots
    assert lib.odb_kv_bytes(C.byref(ok)) * 4 == lib.odb_kv_bytes(C.byref(whole))                # a quarter of the heads
    assert lib.odb_tp_segment_count(C.byref(ok)) == 2 * 32 + 2 and lib.odb_tp_segment_count(C.byref(whole)) == 1
    first, last = C.c_int32(), C.c_int32()
    for bad, want in ((_cfg(synth.LLADA_8B, 3, 0), B.ODB_ERR_SHAPE),      # not 2, 4 or 8
                      (_cfg(synth.LLADA_8B, 4, 4), B.ODB_ERR_ARG),        # rank out of range
                      (_cfg(synth.LLADA_8B, 0, 1), B.ODB_ERR_ARG),        # a rank without a group
                      (_cfg(synth.TINY, 2, 0), B.ODB_ERR_SHAPE),          # 688 FFN features: not 2 x a multiple of 64
                      (_cfg(synth.TINY, 8, 0), B.ODB_ERR_SHAPE)):         # 4 heads over 8 ranks
        assert lib.odb_workspace_bytes(C.byref(bad)) == 0
        assert lib.odb_tp_vocab_range(C.byref(bad), 0, C.byref(first), C.byref(last)) == want
    assert lib.odb_tp_vocab_range(C.byref(ok), 4, C.byref(first), C.byref(last)) == B.ODB_ERR_ARG
    for fn in (lib.odb_session_tp_attach,):
        assert fn(None, None, None, None) == B.ODB_ERR_ARG
    assert lib.odb_debug_tp_segments(None, 0, 1) == B.ODB_ERR_ARG
    assert lib.odb_debug_tp_expire_wait(None, 0, 1000) == B.ODB_ERR_ARG


@pytest.mark.parametrize("world", [2, 4])
def test_layer_shards_reassemble_to_the_layer(world):
    import dataclasses
    shape = dataclasses.replace(synth.TINY, d_ffn=768)
    w = synth.layer_bits(shape, 1, 5)
    parts = [tp.shard_layer(w, shape, r, world) for r in range(world)]
    for name, axis in (("wq", 0), ("wk", 0), ("wv", 0), ("wg", 0), ("wu", 0), ("wo", 1), ("wd", 1)):
        assert np.array_equal(np.concatenate([p[name] for p in parts], axis=axis), w[name]), name
    hl = shape.n_heads // world
    assert parts[0]["wq"].shape == (hl * shape.head_dim, shape.d_model)
    assert parts[0]["wo"].shape == (shape.d_model, hl * shape.head_dim)
    assert parts[0]["wd"].shape == (shape.d_model, shape.d_ffn // world)


def test_peer_pointers_rebase_every_region_into_this_process():
    # rank r's workspace sits at 0x1000 * (r + 1) in ITS address space; regions at fixed offsets inside it
    off = (0x100, 0x400, 0x800)
    bufs = [(0x1000 * (r + 1) + off[0], 64, 0x1000 * (r + 1) + off[1], 96, 0x1000 * (r + 1) + off[2], 128, 0x1000 * (r + 1))
            for r in range(3)]
    mapped = [0x7000_0000, None, 0x9000_0000]                    # where rank 1 mapped ranks 0 and 2
    recv, flags, conf = tp.peer_pointers(1, bufs, mapped, my_base=0x2000)
    assert recv == [0x7000_0000 + off[0], 0x2000 + off[0], 0x9000_0000 + off[0]]
    assert flags == [0x7000_0000 + off[1], 0x2000 + off[1], 0x9000_0000 + off[1]]
    assert conf == [0x7000_0000 + off[2], 0x2000 + off[2], 0x9000_0000 + off[2]]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2511_21759_b200 import tp as tpm
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    base = 0x10_0000 * (rank + 1)
    mine = {"shared": {"handle": ("fake", rank), "tensor_offset": 16 * rank},
            "bufs": (base + 0x100, 64, base + 0x400, 96, base + 0x800, 128, base)}
    everyone = tpm.gather_descriptors(mine)
    # "map" a peer's workspace at an address derived from its handle, as the real opener would return a mapping
    mapped = [None if r == rank else 0x5000_0000 + 0x100_0000 * everyone[r]["shared"]["handle"][1] for r in range(world)]
    recv, flags, conf = tpm.peer_pointers(rank, [e["bufs"] for e in everyone], mapped, base)
    dist.barrier()
    out.put((rank, [e["shared"]["handle"] for e in everyone], recv, flags, conf))
    dist.destroy_process_group()


def test_two_gloo_ranks_exchange_descriptors_and_agree_on_the_layout():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, handles, recv, flags, conf in res:
        assert handles == [("fake", 0), ("fake", 1)]             # rank order, the same on both ranks
        own, peer = 0x10_0000 * (rank + 1), 0x5000_0000 + 0x100_0000 * (1 - rank)
        want = [own, peer] if rank == 0 else [peer, own]
        assert recv == [b + 0x100 for b in want] and flags == [b + 0x400 for b in want] and conf == [b + 0x800 for b in want]
