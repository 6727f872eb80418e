#!/usr/bin/env python
"""Benchmark of the block-decoding hot path (one line of JSON on stdout).

A "step" is one block cycle of the generation: refresh prefill + accept, then block decode
steps + accepts until the block is full, for the workload named in `config.workload`
(default: the 32-layer 8B-shaped model, batch 1, prompt 512, response 256, block 32).  The
headline value is generated tokens per second over the timed steps.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

--impl reference times the CPU oracle (as it stands) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "gen tokens/s (8B-shaped, bs1, block 32); decode-step % of HBM roofline"
UNIT = "tokens/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def recorded_layer_traffic():
    """DRAM bytes (read + written) of the GEMM launches of one decode step of ONE 8B-shaped layer with 32 rows, as
    the ncu capture summarised in profiles/ recorded them; None if the summary is not there."""
    import re
    path = os.path.join(ROOT, "profiles", "gemm_kernel_cfg2_layer_c1.md")
    try:
        m = re.search(r"dram_bytes_per_layer_step:\s*([0-9.eE+]+)", open(path).read())
        return float(m.group(1)) if m else None
    except OSError:
        return None


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=2)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self):
        sm, mx, reasons = [], 0.0, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = max(mx, float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ----------------------------------------------------------------------------- CPU oracle arm

def oracle_sample(wl, budget_layers=2):
    """Times the oracle, as it stands, on a bounded sample of the workload: one refresh and one
    block decode step of the first `budget_layers` layers (fp32), plus the LM head of the step
    rows; layer time is scaled to the full depth.  Returns tokens/s of a block cycle so estimated
    and a description of the sample."""
    import synth
    from oracle import odb_oracle as O
    from oracle.inputs import model_from_synth
    shape = wl.shape
    nl = min(budget_layers, shape.n_layers)
    T, P, Bk = wl.prompt_len + wl.gen_len, wl.prompt_len, wl.block_len
    small = shape.with_layers(nl)
    om = model_from_synth(small, seed=0, dtype=np.float32, with_lm_head=False)
    for l in range(nl):
        om.layer(l)                                   # weight synthesis is input preparation, not timed
    x0 = synth.sequence(0, 0, P, wl.gen_len, shape).astype(np.int64)
    t0 = time.perf_counter()
    cache, _, _ = O.refresh_prefill(om, x0, T, P, dtype=np.float32)
    t_refresh_layers = time.perf_counter() - t0
    subsets = O.copy_subsets(2, wl.n_copies, False)
    rank_pos, rank_tok = [P, P + 1][:2 if wl.n_copies > 1 else 0], [1, 2][:2 if wl.n_copies > 1 else 0]
    t0 = time.perf_counter()
    hid, _, _ = O.block_decode_step(om, cache, x0, T, P, P + Bk, subsets, rank_pos, rank_tok, False, dtype=np.float32)
    t_step_layers = time.perf_counter() - t0
    t_lm_step = t_lm_refresh = 0.0
    if wl.with_lm_head:
        lm = synth.bf16_bits_to_f32(synth.lm_head_bits(shape, 0))
        hid32 = hid.astype(np.float32)
        t0 = time.perf_counter()
        logits, = O.normed_projection(hid32, np.ones(shape.d_model, np.float32), shape.rms_eps, [lm], O.bf16_round)
        O.confidence(logits, shape.mask_id)
        t_lm_step = time.perf_counter() - t0
        t_lm_refresh = t_lm_step * (wl.gen_len / max(len(hid32), 1))
    scale = shape.n_layers / nl
    t_refresh = t_refresh_layers * scale + t_lm_refresh
    t_step = t_step_layers * scale + t_lm_step
    # random weights: one token per iteration, so a block of Bk tokens = 1 refresh + (Bk - 1) steps
    t_block = t_refresh + (Bk - 1) * t_step
    cores = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else os.cpu_count()
    return {"tokens_per_s": Bk / t_block, "t_step_s": t_step, "t_refresh_s": t_refresh, "cores": cores,
            "extrapolated": True, "measured_s": t_refresh_layers + t_step_layers + t_lm_step,
            "sample": f"{nl} of {shape.n_layers} layers of one refresh (T={T}) and one block step (M={len(subsets) * Bk}) "
                      f"in fp32 + LM head of the step rows, layer time scaled x{scale:g}; block cycle = 1 refresh + {Bk - 1} steps"}


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for i in range(args.warmup + args.steps):
        r = oracle_sample(wl)
        if i >= args.warmup:
            vals.append(r)
    v = float(np.mean([r["tokens_per_s"] for r in vals]))
    ms = float(np.mean([wl.block_len / r["tokens_per_s"] for r in vals])) * 1e3
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": config_of(wl),
            "cpu_baseline": {"value": v, "unit": UNIT, "cores": vals[-1]["cores"], "kind": "oracle",
                             "sample": vals[-1]["sample"], "extrapolated": True,
                             "measured_s_per_step": float(np.mean([r["measured_s"] for r in vals]))},
            "extrapolated": True,   # ms_per_step is the block cycle estimated from the sample, not a block cycle run in full
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def config_of(wl):
    return {"workload": wl.name, "batch": wl.batch, "prompt_len": wl.prompt_len, "gen_len": wl.gen_len,
            "block_len": wl.block_len, "n_copies": wl.n_copies, "layers": wl.shape.n_layers,
            "d_model": wl.shape.d_model, "vocab": wl.shape.vocab,
            "l2": "weights streamed per forward (15 GB) exceed L2 (126 MB); no flush needed",
            "step": "one block cycle: refresh prefill + accept, then block decode steps + accepts until the block is full"}


# ----------------------------------------------------------------------------- ranks

def max_over_ranks(ms: float, dist, device=None) -> float:
    """Replicas only: every rank runs the same workload on its own GPU, nothing is exchanged on the
    data path.  The job's time is the slowest rank's (all-reduce MAX of the device-timed interval)."""
    if dist is None:
        return ms
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, ms: float, world: int) -> float:
    """Whole-job throughput of `world` independent replicas: all units processed / the slowest rank's time."""
    return world * units_per_rank / (ms * 1e-3)


# ----------------------------------------------------------------------------- CUDA arm

def run_cuda(args, wl):
    import torch
    import synth
    from paper_2511_21759_b200 import engine as E
    import __graft_entry__ as G

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        G.build()
    if dist:
        dist.barrier()
    peaks = load_peaks()
    shape = wl.shape
    T = wl.prompt_len + wl.gen_len
    gm = E.Model.from_synth(shape, seed=0, device=f"cuda:{local}", with_lm_head=wl.with_lm_head, max_batch=wl.batch,
                            max_seq=T, max_block=wl.block_len, max_copies=8 if args.modes else max(wl.n_copies, 1))
    sess = E.Session(gm)
    params = E.DecodeParams(block_len=wl.block_len, n_copies=wl.n_copies, accept_threshold=wl.accept_threshold,
                            truncate_threshold=wl.truncate_threshold)
    n_blocks = wl.gen_len // wl.block_len
    seqs = [synth.sequence(0, rank * wl.batch + i, wl.prompt_len, wl.gen_len, shape) for i in range(wl.batch)]
    pinned = [torch.from_numpy(s.copy()).pin_memory() for s in seqs]

    state = {"block": 0}
    targets = synth.shrink_schedule(0, wl.batch, wl.gen_len) if wl.batch > 1 else None

    def reset():
        for i in range(wl.batch):
            sess.set_sequence(i, pinned[i].numpy(), wl.prompt_len)
        state["block"] = 0

    def block_cycle(e2e=False):
        """refresh + accept, then steps + accepts until the block is full; returns (tokens, iterations)."""
        if state["block"] >= n_blocks:
            reset()
        if e2e:   # inputs come from the host every step, the result goes back to the host
            toks = [sess.get_tokens(i) for i in range(wl.batch)] if state["block"] else [p.numpy() for p in pinned]
            blk = state["block"]
            for i in range(wl.batch):
                sess.set_sequence(i, toks[i], wl.prompt_len)
            state["block"] = blk
        b = state["block"]
        if all(b * wl.block_len >= sess.gen_len[i] for i in range(wl.batch)):
            reset()
            b = 0
        bi = [b if b * wl.block_len < sess.gen_len[i] else -1 for i in range(wl.batch)]
        sess.refresh_prefill(params, bi)
        if targets is not None:
            # ragged batch: every sequence gives up half of its remaining excess over its seeded target
            # length at each refresh (the lever adaptive length prediction pulls on a trained model)
            for i in range(wl.batch):
                cur = sess.gen_len[i]
                new = max(int(targets[i]), cur - (cur - int(targets[i]) + 1) // 2, (b + 1) * wl.block_len)
                if bi[i] >= 0 and b * wl.block_len < new < cur:
                    sess.set_gen_len(i, new)
        res = sess.unmask_accept(params, True)
        toks, iters = sum(res[i].n_accepted for i in range(wl.batch)), 1
        while any(res[i].masks_left > 0 for i in range(wl.batch)):
            if not args.host_loop:
                log = sess.decode_block_resident(params)
            else:
                sess.block_decode_step(params)
                log = [sess.unmask_accept(params, False)]
            for res in log:
                toks += sum(res[i].n_accepted for i in range(wl.batch))
                iters += 1
        state["block"] += 1
        if e2e:
            for i in range(wl.batch):
                sess.get_tokens(i)
        return toks, iters

    def timed(n, e2e=False):
        if dist:
            dist.barrier()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(sess.stream)
        toks = iters = 0
        for _ in range(n):
            t, it = block_cycle(e2e)
            toks += t; iters += it
        ev1.record(sess.stream)
        torch.cuda.synchronize()
        ms = max_over_ranks(ev0.elapsed_time(ev1), dist, "cuda")
        if dist:
            dist.barrier()
        return ms, toks, iters

    reset()
    timed(args.warmup)
    sess.profile_read()
    with ClockSampler(local) as clocks:
        ms, toks, iters = timed(args.steps)
    _, launches = sess.profile_read()
    clk = clocks.summary()
    value = job_throughput(toks, ms, world)

    # end to end: same steps, sequence pushed from pinned host memory and read back every step
    timed(1, e2e=True)
    ms_e, toks_e, _ = timed(args.steps, e2e=True)
    e2e_value = job_throughput(toks_e, ms_e, world)

    # per-kind device time of decode steps and refreshes, measured live with event pairs
    sess.profile(True)
    reset()
    sess.refresh_prefill(params, [0] * wl.batch)
    res = sess.unmask_accept(params, True)
    ms_refresh, n_refresh = sess.profile_read()
    n_prof = 0
    while any(res[i].masks_left > 0 for i in range(wl.batch)) and n_prof < 16:
        sess.block_decode_step(params)
        res = sess.unmask_accept(params, False)
        n_prof += 1
    ms_step, n_step = sess.profile_read()
    sess.profile(False)
    # whole decode step (enqueue to completion), events on the session's stream, profiling off
    state["block"] = n_blocks
    reset()
    sess.refresh_prefill(params, [0] * wl.batch)
    res = sess.unmask_accept(params, True)
    step_ms = []
    for _ in range(12):
        if not any(res[i].masks_left > 0 for i in range(wl.batch)):
            break
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(sess.stream)
        sess.block_decode_step(params)
        b_.record(sess.stream)
        res = sess.unmask_accept(params, False)
        step_ms.append(a.elapsed_time(b_))
    # the same iteration inside the device-resident loop (row table + step + accept, no host in between)
    loop_ms = None
    if not args.host_loop:
        reset()
        sess.refresh_prefill(params, [0] * wl.batch)
        sess.unmask_accept(params, True)
        sess.decode_block_resident(params, 2)                  # records the loop body on first use
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(sess.stream)
        n_loop = len(sess.decode_block_resident(params, 8))
        b_.record(sess.stream)
        torch.cuda.synchronize()
        loop_ms = a.elapsed_time(b_) / n_loop
    state["block"] = n_blocks

    keys = T - wl.block_len                                   # cached positions outside the block
    step_bytes = gm.step_algorithmic_bytes(keys) * 1.0
    d, F, V, nl = shape.d_model, shape.d_ffn, shape.vocab, shape.n_layers
    gemm_bytes = nl * (3 * d * d + d * d + 2 * F * d + d * F) * 2 + (V * d * 2 if wl.with_lm_head else 0)
    gemm_launches = max(n_step["gemm"], 1)
    gemm_ms = ms_step["gemm"] / max(n_prof, 1)                # per decode step
    gemm_gbs = gemm_bytes / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else None
    step_med = float(np.median(step_ms)) if step_ms else None
    step_gbs = step_bytes / (step_med * 1e-3) / 1e9 if step_med else None
    # the step is a READ stream; the measured peak is a read+write copy: a read-only probe in the same run
    # (16-byte loads), and the same through rings of bulk copies, the way the projections fetch their weights
    read_gbs = bulk_gbs = None
    if rank == 0:
        try:
            read_gbs = E.measure_read_bandwidth(4 << 30, 4, f"cuda:{local}")
            bulk_gbs = E.measure_read_bandwidth(4 << 30, 4, f"cuda:{local}", bulk=True)
        except Exception:
            pass
    layer_traffic = recorded_layer_traffic()
    rows = wl.batch * wl.block_len * wl.n_copies
    frac_of = lambda gbs, peak: (gbs / peak) if (gbs and peak) else None
    roofline = {"bound": "hbm",
                "kernel": "one decode step = every kernel of one odb_block_decode_step (weights once + visible K/V once)",
                "achieved": step_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": frac_of(step_gbs, peaks["hbm_gbs"]),
                "peak_source": peaks["source"],
                "definition": "algorithmic bytes of a step / median device time of a whole step (enqueue to completion, CUDA "
                              "events on the session's stream, nothing instrumented) / MEASURED_PEAKS.json hbm_gbs (a "
                              "read+write copy)",
                "algorithmic_bytes": step_bytes, "ms": step_med, "rows": rows,
                "frac_of_nominal_8tbs": frac_of(step_gbs, 8000.0),
                "hbm_read_gbs": read_gbs, "frac_of_read_probe": frac_of(step_gbs, read_gbs),
                "hbm_bulk_read_gbs": bulk_gbs, "frac_of_bulk_read_probe": frac_of(step_gbs, bulk_gbs),
                "ms_in_resident_loop": loop_ms,
                "frac_in_resident_loop": frac_of(step_bytes / (loop_ms * 1e-3) / 1e9 if loop_ms else None, peaks["hbm_gbs"]),
                # DRAM bytes of a step: the ncu capture of the single-layer case recorded under profiles/ (the full
                # model holds 33 GB on the device: too large to capture), x layers + the LM head's weight bytes
                "traffic": (nl * layer_traffic + (V * d * 2 if wl.with_lm_head else 0))
                if (layer_traffic and shape.d_model == 4096 and rows == 32) else None,
                "traffic_source": "recorded ncu capture (profiles/), scaled by the layer count; not a measurement of this run",
                "gemm_only": {"definition": "weight bytes of the GEMM launches of one step / their summed device time with an "
                                            "event pair around EVERY launch (serialises the launches: pessimistic)",
                              "achieved": gemm_gbs, "frac": frac_of(gemm_gbs, peaks["hbm_gbs"]), "bytes_per_step": gemm_bytes,
                              "launches_per_step": gemm_launches / max(n_prof, 1), "ms_per_step": gemm_ms},
                "ms_by_kind": {k: v / max(n_prof, 1) for k, v in ms_step.items()},
                "refresh": {"ms_by_kind": ms_refresh, "T": T}}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": dict(config_of(wl), block_loop="device-resident (odb_decode_block_resident)" if not args.host_loop
                           else "host (odb_block_decode_step + odb_unmask_accept per iteration)"),
            "tokens_per_step": toks / args.steps, "iterations_per_step": iters / args.steps,
            "clocks": clk,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 4 * T * wl.batch,
                    "d2h_bytes_per_step": 4 * T * wl.batch},
            "gpu_launches": int(sum(launches.values())),
            "roofline": roofline}
    if args.modes and world == 1 and wl.batch == 1:
        # the three systems of the paper's tables on this workload's shapes, whole response each:
        # cache-less baseline, DualCache block decoding, and the full method (speed relative to the first two);
        # then the speculation variants of the ablation (Section 5.3, Fig. 11), each on DualCache block decoding
        # without length prediction: one picked block, the jump chain over four copies, eight copies with
        # decoded-share (NFE and Eff_NFE relative to plain block decoding are the figure's other axis)
        modes = {}
        for mode in ("vanilla", "fast_dllm", "odb", "spec_vanilla", "accept_jump", "decoded_share"):
            mp, cache_blocks = E.mode_settings(mode, wl.block_len, n_copies=4, accept_threshold=wl.accept_threshold)
            if cache_blocks and not args.host_loop:
                # untimed first run: the device-resident loop records one graph per step shape on first use
                reset()
                E.generate(sess, mp, cache_blocks=cache_blocks, resident=True)
                sess.set_active(0, True)
            reset()
            torch.cuda.synchronize()
            m0, m1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            m0.record(sess.stream)
            _, mtrace = E.generate(sess, mp, cache_blocks=cache_blocks, resident=not args.host_loop)
            m1.record(sess.stream)
            torch.cuda.synchronize()
            sess.set_active(0, True)
            cnt = E.trace_counters(mtrace)
            mms = m0.elapsed_time(m1)
            modes[mode] = dict(cnt, ms=mms, tokens_per_s=cnt["tokens"] / (mms * 1e-3))
        for mode in modes:
            modes[mode]["speed_vs_vanilla"] = modes[mode]["tokens_per_s"] / modes["vanilla"]["tokens_per_s"]
            modes[mode]["speed_vs_fast_dllm"] = modes[mode]["tokens_per_s"] / modes["fast_dllm"]["tokens_per_s"]
            modes[mode]["nfe_vs_fast_dllm"] = modes[mode]["nfe"] / modes["fast_dllm"]["nfe"]
            modes[mode]["eff_nfe_vs_fast_dllm"] = modes[mode]["eff_nfe"] / modes["fast_dllm"]["eff_nfe"]
        line["modes"] = modes
    if rank == 0 and world == 1 and args.workload == "cfg3_8b_c1" and not args.no_secondary:
        try:
            line["secondary"] = secondary_measurements(E, synth, gm, peaks, args)
        except Exception as exc:      # the headline line must come out whatever happens to the extras
            line["secondary"] = {"error": f"{type(exc).__name__}: {exc}"}
        try:                          # the tensor-parallel path: one rank's step alone (a lower bound, no NVLink in it)
            line["secondary"]["tp_rank_alone"] = tp_rank_alone(wl, peaks, 10, 3)
        except Exception as exc:
            line["secondary"]["tp_rank_alone"] = {"error": f"{type(exc).__name__}: {exc}"}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            r = oracle_sample(wl)
            line["cpu_baseline"] = {"value": r["tokens_per_s"], "unit": UNIT, "cores": r["cores"], "kind": "oracle",
                                    "sample": r["sample"], "t_step_s": r["t_step_s"], "t_refresh_s": r["t_refresh_s"],
                                    "extrapolated": True, "measured_s": r["measured_s"]}
        print(json.dumps(line))
    sess.close()
    gm.close()
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def secondary_measurements(E, synth, gm, peaks, args):
    """The other configurations the metric names, in the same process after the headline: the 4-copy workload on the
    same weights (block cycle tokens/s and its 128-row decode step), and the single-layer decode step with 1 and 4
    copies (L2 flushed before every step)."""
    import torch
    out = {}
    # ---- 4 copies, prompt 512 + response 512, same weights, a session of its own ----
    wl4 = synth.WORKLOADS["cfg4_8b_c4"]
    T4 = wl4.prompt_len + wl4.gen_len
    gm4 = E.Model(wl4.shape, gm.t, max_batch=1, max_seq=T4, max_block=wl4.block_len, max_copies=4)
    s4 = E.Session(gm4)
    p4 = E.DecodeParams(block_len=wl4.block_len, n_copies=4)
    x4 = synth.sequence(0, 0, wl4.prompt_len, wl4.gen_len, wl4.shape)

    def cycle(block):
        s4.refresh_prefill(p4, block)
        res = s4.unmask_accept(p4, True)
        toks, its = res[0].n_accepted, 1
        while res[0].masks_left > 0:
            for res in (s4.decode_block_resident(p4) if not args.host_loop else [(s4.block_decode_step(p4), s4.unmask_accept(p4, False))[1]]):
                toks += res[0].n_accepted
                its += 1
        return toks, its

    s4.set_sequence(0, x4, wl4.prompt_len)
    cycle(0)                                                   # warm-up (records the loop graphs of the shapes met)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(s4.stream)
    toks = its = 0
    for blk in range(1, 4):
        t_, i_ = cycle(blk)
        toks += t_; its += i_
    b.record(s4.stream)
    torch.cuda.synchronize()
    ms4 = a.elapsed_time(b)
    # the 128-row step on its own
    s4.set_sequence(0, x4, wl4.prompt_len)
    s4.refresh_prefill(p4, 0)
    res = s4.unmask_accept(p4, True)
    steps = []
    for _ in range(8):
        if res[0].masks_left <= 0:
            break
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s4.stream)
        s4.block_decode_step(p4)
        e1.record(s4.stream)
        res = s4.unmask_accept(p4, False)
        steps.append(e0.elapsed_time(e1))
    bytes4 = gm4.step_algorithmic_bytes(T4 - wl4.block_len)
    st4 = float(np.median(steps)) if steps else None
    out["cfg4_8b_c4"] = {"tokens_per_s": toks / (ms4 * 1e-3), "block_cycles": 3, "iterations_per_block": its / 3,
                         "step_rows": 4 * wl4.block_len, "step_ms": st4, "step_algorithmic_bytes": bytes4,
                         "step_frac_of_measured": (bytes4 / (st4 * 1e-3) / 1e9 / peaks["hbm_gbs"]) if st4 else None}
    s4.close(); gm4.close()
    # ---- batch 16, prompt 1024, response 1024 shrunk per sequence, block 64, 4 copies: one block cycle ----
    wl5 = synth.WORKLOADS["cfg5_8b_b16"]
    T5 = wl5.prompt_len + wl5.gen_len
    gm5 = E.Model(wl5.shape, gm.t, max_batch=wl5.batch, max_seq=T5, max_block=wl5.block_len, max_copies=4)
    s5 = E.Session(gm5)
    p5 = E.DecodeParams(block_len=wl5.block_len, n_copies=4)
    targets = synth.shrink_schedule(0, wl5.batch, wl5.gen_len)
    for i in range(wl5.batch):
        s5.set_sequence(i, synth.sequence(0, i, wl5.prompt_len, wl5.gen_len, wl5.shape), wl5.prompt_len)

    def cycle5(block, timed_steps=None):
        bi = [block if block * wl5.block_len < s5.gen_len[i] else -1 for i in range(wl5.batch)]
        s5.refresh_prefill(p5, bi)
        for i in range(wl5.batch):       # every sequence gives up half of its excess over its seeded target length
            cur = s5.gen_len[i]
            new = max(int(targets[i]), cur - (cur - int(targets[i]) + 1) // 2, (block + 1) * wl5.block_len)
            if bi[i] >= 0 and block * wl5.block_len < new < cur:
                s5.set_gen_len(i, new)
        res = s5.unmask_accept(p5, True)
        toks = sum(res[i].n_accepted for i in range(wl5.batch))
        while any(res[i].masks_left > 0 for i in range(wl5.batch)):
            if timed_steps is not None and len(timed_steps) < 4:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(s5.stream)
                s5.block_decode_step(p5)
                e1.record(s5.stream)
                log = [s5.unmask_accept(p5, False)]
                timed_steps.append(e0.elapsed_time(e1))
            else:
                log = s5.decode_block_resident(p5) if not args.host_loop else [(s5.block_decode_step(p5), s5.unmask_accept(p5, False))[1]]
            for res in log:
                toks += sum(res[i].n_accepted for i in range(wl5.batch))
        for i in range(wl5.batch):
            s5.gen_len[i] = res[i].gen_len
        return toks

    cycle5(0)                                                  # warm-up block (graphs of the shapes met)
    steps5 = []
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(s5.stream)
    toks5 = cycle5(1, steps5)
    b.record(s5.stream)
    torch.cuda.synchronize()
    rows5 = wl5.batch * wl5.block_len * 4
    d_, F_, V_, nl_ = wl5.shape.d_model, wl5.shape.d_ffn, wl5.shape.vocab, wl5.shape.n_layers
    flops5 = 2.0 * rows5 * (nl_ * (4 * d_ * d_ + 3 * d_ * F_) + V_ * d_)      # projections of one full step (attention excluded)
    st5 = float(np.median(steps5)) if steps5 else None
    out["cfg5_8b_b16"] = {"tokens_per_s": toks5 / (a.elapsed_time(b) * 1e-3), "block_cycles": 1, "batch": wl5.batch,
                          "response_lengths_after_two_refreshes": [int(s5.gen_len[i]) for i in range(wl5.batch)],
                          "step_rows_at_block_start": rows5, "step_ms": st5, "bound": "tensor",
                          "step_tflops": flops5 / (st5 * 1e-3) / 1e12 if st5 else None,
                          "step_frac_of_sustained_bf16": (flops5 / (st5 * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]) if st5 else None}
    s5.close(); gm5.close()
    # ---- one 8B-shaped layer, context 512, block 32: the decode step with 1 and 4 copies ----
    shape1 = synth.LLADA_8B.with_layers(1)
    wl1 = synth.WORKLOADS["cfg2_layer_c1"]
    T1 = wl1.prompt_len + wl1.gen_len
    gm1 = E.Model.from_synth(shape1, seed=0, with_lm_head=False, max_batch=1, max_seq=T1, max_block=wl1.block_len, max_copies=4)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for name, copies in (("cfg2_layer_c1", 1), ("cfg2_layer_c4", 4)):
        s1 = E.Session(gm1)
        p1 = E.DecodeParams(block_len=wl1.block_len, n_copies=copies)
        s1.set_sequence(0, synth.sequence(0, 0, wl1.prompt_len, wl1.gen_len, shape1), wl1.prompt_len)
        s1.refresh_prefill(p1, 0)
        s1.unmask_accept(p1, True)
        times = []
        for i in range(3 + 12):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(s1.stream)
            s1.block_decode_step(p1)
            e1.record(s1.stream)
            s1.unmask_accept(p1, False)
            if i >= 3:
                times.append(e0.elapsed_time(e1))
        ms1 = float(np.median(times))
        b1 = gm1.step_algorithmic_bytes(T1 - wl1.block_len)
        out[name] = {"step_us": ms1 * 1e3, "rows": copies * wl1.block_len, "algorithmic_bytes": b1,
                     "frac_of_measured": b1 / (ms1 * 1e-3) / 1e9 / peaks["hbm_gbs"], "l2": "flushed before every step"}
        s1.close()
    gm1.close()
    return out


def run_persistent_phases(args, wl):
    """Where the time of the persistent decode-step kernel goes: mean duration of every phase between two grid
    barriers (from the release of the previous barrier to the last CTA's arrival at the next), and the barrier's
    own latency (last arrival to release), over the layers of one step.  Prints one JSON line."""
    os.environ["ODB_PERSISTENT"] = "1"
    os.environ["ODB_PERSISTENT_TIMING"] = "1"
    import torch
    import synth
    import __graft_entry__ as G
    from paper_2511_21759_b200 import engine as E
    G.build()
    shape, T = wl.shape, wl.prompt_len + wl.gen_len
    gm = E.Model.from_synth(shape, seed=0, max_batch=1, max_seq=T, max_block=wl.block_len, max_copies=max(wl.n_copies, 1))
    sess = E.Session(gm)
    sess.set_sequence(0, synth.sequence(0, 0, wl.prompt_len, wl.gen_len, shape), wl.prompt_len)
    gp = E.DecodeParams(block_len=wl.block_len, n_copies=wl.n_copies)
    sess.refresh_prefill(gp, 0)
    sess.unmask_accept(gp, True)
    step_ms = []
    for _ in range(args.warmup + args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(sess.stream)
        sess.block_decode_step(gp)
        b.record(sess.stream)
        sess.unmask_accept(gp, False)
        step_ms.append(a.elapsed_time(b))
    n_cta = torch.cuda.get_device_properties(0).multi_processor_count
    ks = max(1, min(8, n_cta // (wl.n_copies * shape.n_heads)))
    names = ["norm1", "qkv", "rope", "attention"] + (["merge"] if ks > 1 else []) + ["o", "norm2", "gate_up", "swiglu", "down"]
    nb = len(names)
    t = sess.persistent_barrier_times(n_cta, shape.n_layers * nb + 1)
    arr, rel = t[:, :, 0], t[:, :, 1]
    last_arr, last_rel = arr.max(0), rel.max(0)
    phases = {}
    for j, n in enumerate(names):
        ids = [l * nb + j for l in range(1, shape.n_layers)]
        phases[n] = {"us": float(np.mean([last_arr[i] - last_rel[i - 1] for i in ids])) / 1e3,
                     "barrier_us": float(np.mean([last_rel[i] - last_arr[i] for i in ids])) / 1e3}
    print(json.dumps({"kernel": "step_persistent_kernel", "workload": wl.name, "ctas": n_cta, "key_splits": ks,
                      "step_ms": float(np.median(step_ms[args.warmup:])),
                      "per_layer_us": float(sum(v["us"] + v["barrier_us"] for v in phases.values())), "phases": phases}))
    sess.close(); gm.close()


def run_layer_microbench(args, wl):
    """Single-layer block-decode-step microbenchmark (model without LM head): one refresh fills the
    cache, then every timed iteration is one odb_block_decode_step over block 0 with the workload's
    number of copies.  L2 is flushed (256 MB written) before every iteration; each iteration is
    timed on its own with CUDA events on the session's stream."""
    import torch
    import __graft_entry__ as G
    from paper_2511_21759_b200 import engine as E
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    G.build()
    peaks = load_peaks()
    shape, T = wl.shape, wl.prompt_len + wl.gen_len
    import synth
    gm = E.Model.from_synth(shape, seed=0, with_lm_head=False, max_batch=wl.batch, max_seq=T, max_block=wl.block_len,
                            max_copies=max(wl.n_copies, 1))
    sess = E.Session(gm)
    params = E.DecodeParams(block_len=wl.block_len, n_copies=wl.n_copies)
    # a batch is ragged the way the full benchmark's is: seeded response lengths between a quarter and a half of the allocation
    lens = [wl.gen_len] if wl.batch == 1 else [int(n) for n in synth.shrink_schedule(0, wl.batch, wl.gen_len)]
    for i in range(wl.batch):
        sess.set_sequence(i, synth.sequence(0, i, wl.prompt_len, lens[i], shape), wl.prompt_len)
    sess.refresh_prefill(params, 0)
    sess.unmask_accept(params, True)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    times = []
    with ClockSampler(0) as clocks:
        for i in range(args.warmup + args.steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(sess.stream)
            sess.block_decode_step(params)
            b.record(sess.stream)
            sess.unmask_accept(params, False)
            if i >= args.warmup:
                times.append(a.elapsed_time(b))
    _, launches = sess.profile_read()
    sess.profile(True)
    for _ in range(8):
        flush.zero_()
        sess.block_decode_step(params)
        sess.unmask_accept(params, False)
    ms_kind, n_kind = sess.profile_read()
    sess.profile(False)
    ms = float(np.median(times))
    keys = T - wl.block_len
    step_bytes = gm.step_algorithmic_bytes(keys)
    d, F = shape.d_model, shape.d_ffn
    gemm_bytes = (3 * d * d + d * d + 2 * F * d + d * F) * 2
    gemm_ms = ms_kind["gemm"] / 8
    line = {"metric": "single-layer block decode step latency", "value": ms * 1e3, "unit": "us", "n_gpus": 1,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": dict(config_of(wl), l2="flushed before every iteration (256 MB written)",
                           step="one odb_block_decode_step of the single layer"),
            "clocks": clocks.summary(), "gpu_launches": int(sum(launches.values())),
            "roofline": {"bound": "hbm", "kernel": "whole layer step (4 GEMMs + attention + elementwise)",
                         "achieved": step_bytes / (ms * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": step_bytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "peak_source": peaks["source"],
                         "traffic": None, "algorithmic_bytes": step_bytes,
                         "gemm": {"ms": gemm_ms, "achieved_gbs": gemm_bytes / (gemm_ms * 1e-3) / 1e9 if gemm_ms else None},
                         "ms_by_kind": {k: v / 8 for k, v in ms_kind.items()},
                         "p10_ms": float(np.percentile(times, 10)), "p90_ms": float(np.percentile(times, 90))}}
    print(json.dumps(line))
    sess.close()
    gm.close()


def tp_rank_alone(wl, peaks, steps, warmup, only=0):
    """Device time of ONE tensor-parallel rank's decode step, timed alone on this GPU, for groups of 2, 4 and 8: rank 0's
    shard of the workload's model, attached to its own buffers as if they were its peers', with the flags of the
    absent ranks raised locally (odb_debug_tp_alone).  Every kernel of the rank runs (its projections store their
    partial tiles R times, the flags are raised and waited for, the RMSNorm adds R blocks of partials); what is missing
    is the NVLink latency and bandwidth of the stores and flags, so this is a lower bound of a rank's step time, not a
    scaling measurement.  Results of the forward are meaningless (the peers' partial sums are absent)."""
    import torch
    from paper_2511_21759_b200 import engine as E, tp
    import synth
    shape, T = wl.shape, wl.prompt_len + wl.gen_len
    worlds = [r for r in (2, 4, 8) if shape.n_heads % r == 0 and shape.d_ffn % (64 * r) == 0 and only in (0, r)]
    d, F, nl = shape.d_model, shape.d_ffn, shape.n_layers
    keys = T - wl.block_len
    out = {"definition": "one rank of R timed alone on one GPU (own buffers as peers, absent ranks' flags raised locally): "
                         "lower bound of a rank's step time, no NVLink in it; not a scaling measurement"}
    params = E.DecodeParams(block_len=wl.block_len, n_copies=wl.n_copies, alp=False)
    for R in worlds:
        gm = tp.model_shard_from_synth(shape, 0, 0, R, max_batch=1, max_seq=T, max_block=wl.block_len,
                                       max_copies=max(wl.n_copies, 1))
        sess = E.Session(gm)
        tp.attach_alone(sess)

        def reopen():
            sess.set_sequence(0, synth.sequence(0, 0, wl.prompt_len, wl.gen_len, shape), wl.prompt_len)
            sess.refresh_prefill(params, 0)
            sess.unmask_accept(params, True)
        reopen()
        times, loop_times = [], []
        for i in range(warmup + steps):       # call by call: one launch sequence from the host per step
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(sess.stream)
            sess.block_decode_step(params)
            b.record(sess.stream)
            res = sess.unmask_accept(params, False)
            if i >= warmup:
                times.append(a.elapsed_time(b))
            if res[0].masks_left == 0:      # block full (garbage confidences may accept anything): open it again
                reopen()
        reopen()
        for i in range(warmup + steps):       # the device-resident loop: the same kernels replayed from a graph
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(sess.stream)
            its = sess.decode_block_resident(params, 4)
            b.record(sess.stream)
            b.synchronize()
            if i >= warmup:
                loop_times.append(a.elapsed_time(b) / len(its))
            if its[-1][0].masks_left == 0:
                reopen()
        ms, loop_ms = float(np.median(times)), float(np.median(loop_times))
        v0, v1 = tp.vocab_range(gm.cfg, 0)
        rank_bytes = nl * ((3 * d * d + d * d + 3 * F * d) * 2 / R + 2 * keys * d * 2 / R) + (v1 - v0) * d * 2
        out[f"ranks_{R}"] = {"ms_per_step_host_launched": ms, "ms_per_iteration_in_resident_loop": loop_ms,
                             "rank_algorithmic_bytes": rank_bytes, "achieved_gbs": rank_bytes / (loop_ms * 1e-3) / 1e9,
                             "frac_of_hbm_peak": rank_bytes / (loop_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], "status": sess.status()}
        sess.close(); gm.close()
        del sess, gm
        torch.cuda.empty_cache()
    return out


def run_tp_rank_step(args, wl):
    """bench.py --tp-rank-step: tp_rank_alone as one JSON line."""
    import torch
    import __graft_entry__ as G
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    G.build()
    peaks = load_peaks()
    out = tp_rank_alone(wl, peaks, args.steps, args.warmup, args.tp_ranks)
    print(json.dumps({"metric": "device time of one tensor-parallel rank's decode step, timed alone (no peers, no NVLink)",
                      "unit": "ms", "n_gpus": 1, "steps": args.steps, "warmup": args.warmup, "higher_is_better": False,
                      "dtype": "bf16", "data": "synthetic", "config": config_of(wl), "peak": peaks["hbm_gbs"],
                      "peak_source": peaks["source"], "tp": out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg3_8b_c1")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the secondary object (4-copy workload and single-layer steps measured after the headline)")
    ap.add_argument("--host-loop", action="store_true",
                    help="take every iteration of a block as odb_block_decode_step + odb_unmask_accept from the host instead "
                         "of odb_decode_block_resident (one host round trip per iteration instead of one per change of the "
                         "step's shape)")
    ap.add_argument("--persistent-phases", action="store_true",
                    help="run decode steps through the persistent step kernel and print the mean time of each of its phases")
    ap.add_argument("--tp-rank-step", action="store_true",
                    help="time one tensor-parallel rank's decode step alone on this GPU for groups of 2, 4 and 8 (lower bound "
                         "of a rank's step time: no peers, no NVLink latency)")
    ap.add_argument("--tp-ranks", type=int, default=0, help="with --tp-rank-step: only this group size (2, 4 or 8)")
    ap.add_argument("--modes", action="store_true",
                    help="also run the whole response as cache-less baseline / DualCache block decoding / full method")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not under a launcher: start the N local ranks (one process per GPU) and pass their output through
        import socket
        with socket.socket() as so:
            so.bind(("127.0.0.1", 0))
            port = so.getsockname()[1]
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    import synth
    wl = synth.WORKLOADS[args.workload]
    if args.persistent_phases:
        run_persistent_phases(args, wl)
    elif args.tp_rank_step:
        run_tp_rank_step(args, wl)
    elif args.impl == "reference":
        run_reference(args, wl)
    elif not wl.with_lm_head:
        run_layer_microbench(args, wl)
    else:
        run_cuda(args, wl)


if __name__ == "__main__":
    main()
