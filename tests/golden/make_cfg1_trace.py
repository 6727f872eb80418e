"""Writes cfg1_trace.json: the oracle's own generation trace on the tiny end-to-end workload
(2 layers, d 256, vocab 2048, prompt 64, response 64, block 16, threshold 0.9; 1 and 4 copies) and on
the sharp-logit variant.  Calls only the oracle and the seeded input generator.

    python tests/golden/make_cfg1_trace.py
"""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

import synth  # noqa: E402
from oracle import odb_oracle as O  # noqa: E402
from oracle.inputs import model_from_synth  # noqa: E402


def main():
    out = {}
    for name in ("cfg1_tiny", "cfg1_tiny_c4", "peaky_c1", "peaky_c4", "peaky_c8"):
        wl = synth.WORKLOADS[name]
        om = model_from_synth(wl.shape, seed=0)
        x0 = synth.sequence(0, 0, wl.prompt_len, wl.gen_len, wl.shape)
        x, trace = O.generate(om, x0, wl.prompt_len, O.DecodeParams(block_len=wl.block_len, n_copies=wl.n_copies))
        out[name] = {"tokens": [int(t) for t in x[wl.prompt_len:]],
                     "iterations": [[t["kind"], t["block"], t["accepted"], t["chain"]] for t in trace]}
    with open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "cfg1_trace.json"), "w") as f:
        json.dump(out, f, separators=(",", ":"))


if __name__ == "__main__":
    main()
