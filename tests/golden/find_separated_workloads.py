"""Searches small workloads on which EVERY decision of the oracle's own generation is far from
flipping, and stores their traces (separated_workloads.json).  Calls only `oracle/` and `synth/`.

With random weights a generation takes hundreds of decisions among continuous values (threshold
compares, the top-1 fallback, the candidate ranking, greedy tokens), and some of them are always
closer than a bf16 implementation's rounding noise: a free run of such a workload cannot be
compared token for token.  The workloads found here are the ones where it can: for every
iteration of the oracle's trace,
    sep     (smallest distance of a confidence decision from flipping, in ln(c / (1 - c)))  >= SEP_MIN
    tok_gap (smallest top-2 logit gap of a greedy token that is used)                        >= GAP_MIN
with both limits a multiple of the logit error a bf16 forward of this model shows (the GPU parity
test measures that error in lock step and checks the multiple).  Their free runs must then be
bit-identical on any correct implementation.

Usage:  python tests/golden/find_separated_workloads.py [--procs N] [--tries K] [--redo]
(families already in the file are kept unless --redo is given)
"""
import argparse
import dataclasses
import json
import multiprocessing as mp
import os
import sys

os.environ.setdefault("OMP_NUM_THREADS", "1")        # one thread per worker process: the pool is the parallelism
os.environ.setdefault("OPENBLAS_NUM_THREADS", "1")
os.environ.setdefault("MKL_NUM_THREADS", "1")

import numpy as np                              # noqa: E402

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth                                    # noqa: E402
from oracle import odb_oracle as O              # noqa: E402
from oracle.inputs import model_from_synth      # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "separated_workloads.json")

# the tiny shape with unit-gain layers and a sharp LM head (logit rms 8): logit error of a bf16
# forward about 0.05 (worst element), so ten and eight times that
SEP_MIN = 0.6
GAP_MIN = 0.4

# (name, copies, prompt, response, block, accept threshold): small on purpose, the number of
# decisions that must all be separated grows with the response.  A family stays here only if the workload found
# for it also passes the GPU parity test that measures the error on it (ten times / four times the measured
# error): one more family (prompt 30, block 10) was found with a top-2 gap of 0.47 and dropped at 3.6 times.
FAMILIES = [
    ("sep_c1_a", 1, 24, 12, 6, 0.9),
    ("sep_c1_b", 1, 17, 16, 8, 0.7),
    ("sep_c4_a", 4, 24, 8, 8, 0.9),
    ("sep_c8_a", 8, 24, 8, 8, 0.9),
]


def shape_of(lm_std):
    return dataclasses.replace(synth.TINY_PEAKY, lm_std=lm_std)


def run(args):
    name, C, P, L, B, tau, seed = args
    shape = shape_of(0.5)
    om = model_from_synth(shape, seed=seed)
    x0 = synth.sequence(seed, 0, P, L, shape)
    params = O.DecodeParams(block_len=B, n_copies=C, accept_threshold=tau, alp=False)
    tok, tr = O.generate(om, x0, P, params)
    sep = min(t["sep"] for t in tr)
    gap = min(t["tok_gap"] for t in tr)
    steps = [t for t in tr if t["kind"] == "step"]
    # the run must exercise what it is there for: steps, several tokens in one pass, and with
    # copies a jump chain (with eight copies also a step in the decoded-share layout)
    rich = len(steps) >= 2 and any(len(t["accepted"]) > 1 for t in tr)
    if C > 1:
        rich = rich and any(len(t["chain"]) > 1 for t in steps)
    if C == 8:
        rich = rich and any(t["stage2"] for t in steps)
    if not (rich and sep >= SEP_MIN and gap >= GAP_MIN):
        return None
    return {"name": name, "seed": seed, "w_std": shape.w_std, "lm_std": shape.lm_std, "prompt_len": P, "gen_len": L,
            "block_len": B, "n_copies": C, "accept_threshold": tau, "min_sep": sep, "min_tok_gap": gap,
            "tokens": [int(t) for t in tok],
            "trace": [{"kind": t["kind"], "T": t["T"], "accepted": [list(a) for a in t["accepted"]], "chain": t["chain"],
                       "sep": t["sep"], "tok_gap": t["tok_gap"]} for t in tr]}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--procs", type=int, default=max(1, (os.cpu_count() or 2) - 1))
    ap.add_argument("--tries", type=int, default=20000)
    ap.add_argument("--chunk", type=int, default=400)
    ap.add_argument("--redo", action="store_true")
    a = ap.parse_args()
    found = {}
    if os.path.exists(OUT) and not a.redo:
        with open(OUT) as f:
            found = json.load(f)["workloads"]
    with mp.Pool(a.procs) as pool:
        for fam in FAMILIES:
            if fam[0] in found:
                continue
            for s0 in range(0, a.tries, a.chunk):
                hits = [r for r in pool.imap(run, [fam + (s,) for s in range(s0, s0 + a.chunk)], chunksize=8) if r]
                if hits:
                    found[fam[0]] = max(hits, key=lambda r: min(r["min_sep"] / SEP_MIN, r["min_tok_gap"] / GAP_MIN))
                    print(fam[0], "seed", found[fam[0]]["seed"], "sep %.2f gap %.2f" % (found[fam[0]]["min_sep"],
                          found[fam[0]]["min_tok_gap"]), len(found[fam[0]]["trace"]), "iterations", flush=True)
                    break
            else:
                print(fam[0], "nothing found in", a.tries, "seeds", flush=True)
    with open(OUT, "w") as f:
        json.dump({"sep_min": SEP_MIN, "gap_min": GAP_MIN, "workloads": found}, f, indent=1)
    print("wrote", OUT, len(found), "workloads")


if __name__ == "__main__":
    main()
