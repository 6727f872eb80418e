"""One generation of a tensor-parallel group, one process per GPU:

    python -m torch.distributed.run --nnodes=1 --nproc-per-node R --master-addr 127.0.0.1 --master-port P \
        -m paper_2511_21759_b200.tp_run --workload cfg3_8b_c1 [--copies 4] [--host-loop]

Every rank uploads its shard of the seeded synthetic model, creates a session on its GPU, maps the other ranks'
workspaces (tp.attach_process_group) and runs the ordinary host control loop (engine.generate); the projections'
epilogues store into the peers' buffers and flags order the exchange on the device.  Rank 0 prints one JSON line:
tokens/s of the whole response, timed with CUDA events, the maximum over the ranks.  The ranks must end with the same
tokens; that is checked.  NVLS is not used (plain peer stores); NCCL only carries the final checks.

This entry point composes pieces that are each tested on one GPU (shards, exchange kernels, flags as a group issued
segment by segment; the descriptor exchange between two gloo ranks; the inter-process mapping); it needs R GPUs to run.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch
import torch.distributed as dist


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg3_8b_c1")
    ap.add_argument("--copies", type=int, default=0, help="jump-share copies (default: the workload's)")
    ap.add_argument("--host-loop", action="store_true", help="one host round trip per iteration instead of the device loop")
    args = ap.parse_args()

    import synth
    from . import engine as E, tp
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    local = int(os.environ.get("LOCAL_RANK", rank))
    if world not in (2, 4, 8):
        raise SystemExit("a tensor-parallel group has 2, 4 or 8 ranks")
    torch.cuda.set_device(local)
    dist.init_process_group("nccl", rank=rank, world_size=world)
    host_group = dist.new_group(backend="gloo")          # descriptors travel as pickled objects

    wl = synth.WORKLOADS[args.workload]
    if wl.batch != 1:
        raise SystemExit("this runner takes the batch-1 workloads")
    copies = args.copies or wl.n_copies
    shape, T = wl.shape, wl.prompt_len + wl.gen_len
    gm = tp.model_shard_from_synth(shape, 0, rank, world, f"cuda:{local}", max_batch=1, max_seq=T, max_block=wl.block_len,
                                   max_copies=max(copies, 1))
    sess = E.Session(gm)
    tp.attach_process_group(sess, host_group)
    x0 = synth.sequence(0, 0, wl.prompt_len, wl.gen_len, shape)
    params = E.DecodeParams(block_len=wl.block_len, n_copies=copies)

    def run():
        sess.set_sequence(0, x0, wl.prompt_len)
        dist.barrier()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(sess.stream)
        toks, trace = E.generate(sess, params, resident=not args.host_loop)
        b.record(sess.stream)
        b.synchronize()
        return toks[0], trace, a.elapsed_time(b)

    run()                                                  # warm-up (records the loop graphs)
    toks, trace, ms = run()
    status = sess.status()
    t = torch.tensor([ms], dtype=torch.float64, device=f"cuda:{local}")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    mine = torch.from_numpy(np.ascontiguousarray(toks, dtype=np.int64)).to(f"cuda:{local}")
    ref = mine.clone()
    dist.broadcast(ref, src=0)
    same = torch.tensor([int(torch.equal(mine, ref)) and status == 0], device=f"cuda:{local}")
    dist.all_reduce(same, op=dist.ReduceOp.MIN)
    if rank == 0:
        print(json.dumps({"metric": "generated tokens/s, tensor-parallel group", "value": wl.gen_len / (float(t.item()) * 1e-3),
                          "unit": "tokens/s", "n_gpus": world, "ms": float(t.item()), "iterations": len(trace),
                          "ranks_agree_and_no_wait_expired": bool(same.item()), "scaling": "strong",
                          "config": {"workload": wl.name, "copies": copies, "parallelism": f"tp{world}",
                                     "block_loop": "host" if args.host_loop else "device-resident"}}))
    sess.close()
    gm.close()
    dist.barrier()
    dist.destroy_process_group()
    if not bool(same.item()):
        raise SystemExit(1)


if __name__ == "__main__":
    main()
