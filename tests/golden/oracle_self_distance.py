"""How far two correct evaluations of the same bf16-faithful forward are from each other, by depth.

The oracle is run twice on the 8B shape (d 4096, 32 heads of 128, FFN 12288), once with float32 and once with
float64 arithmetic between the bf16 rounding points.  Both are "the oracle"; they differ only in the order and
precision of the sums, which is exactly how a correct GPU implementation differs from either.  A tiny difference
before a rounding point flips some bf16 roundings, the flips are re-amplified by the next projection, and the
distance performs a random walk over the layers: the per-row relative L2 distance of the K rows written by layer l
(l = 1 is the second layer: the first layer's K is an exact function of the embeddings) follows c * sqrt(l).

This file measures c (stored in oracle_self_distance.json) and states the two bounds the full-size GPU parity
test uses, as functions of that measurement instead of literals:
    l2_bound(layers)                 = 1.3 * c * sqrt(layers)
    elementwise_factor(layers, n)    = z(n) * c * sqrt(layers) / 2e-2,  z(n) = sqrt(2 ln n) + 1
(the 1.3: c is the worst of the 16 rows of a six-layer measurement, the bound is applied to the worst of several
hundred rows at 32 layers - the rows' own constants spread by +-6 %, which puts the worst of 256 rows 20 % above
their mean - and to kernels whose exp2 / rsqrt are approximations; measured on the GPU: 1.3e-2 ... 2.4e-2 against
c sqrt(32) = 1.99e-2;
the element bound is the largest of n roughly Gaussian errors of relative size c sqrt(layers), in units of the small-model element bound
2e-2 * max(|x|, rms(row)); the + 1 sigma is for the rows not being identically distributed: a row's own distance
ranges up to the bound while the typical row sits a quarter below it.  Measured on the GPU: 4.9 x at n = 3.2e7 and
6.1 x at n = 8.1e6, against 6.9 x and 6.6 x from this formula).  Calls only `oracle/` and `synth/`.

    python tests/golden/oracle_self_distance.py [--layers 6] [--rows 16]      (writes the JSON; minutes)
"""
import argparse
import json
import math
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth                                    # noqa: E402
from oracle import odb_oracle as O              # noqa: E402
from oracle.inputs import model_from_synth      # noqa: E402

OUT = os.path.join(os.path.dirname(os.path.abspath(__file__)), "oracle_self_distance.json")


def measure(n_layers: int, rows: int, seed: int = 0):
    """Per layer: worst per-row relative L2 distance and worst element distance (in units of
    2e-2 * max(|x|, rms(row))) between the float32 and the float64 run, on the K rows the layer writes."""
    shape = synth.LLADA_8B.with_layers(n_layers)
    x = synth.sequence(seed, 0, rows // 2, rows - rows // 2, shape).astype(np.int64)
    om = model_from_synth(shape, seed=seed, dtype=np.float32, with_lm_head=False)      # weights generated once, shared
    vis = np.ones((rows, rows), bool)
    runs = {}
    for dt in (np.float32, np.float64):
        _, fk, _ = O.forward_rows(om, x, np.arange(rows), None, None, vis, dtype=dt, return_hidden=True)
        runs[dt] = [k.reshape(rows, -1).astype(np.float64) for k in fk]
    out = []
    for l in range(n_layers):
        a, b = runs[np.float32][l], runs[np.float64][l]
        rms = np.sqrt((b * b).mean(-1, keepdims=True))
        out.append({"layer": l,
                    "rel_l2": float((np.sqrt(((a - b) ** 2).sum(-1)) / np.sqrt((b * b).sum(-1))).max()),
                    "elementwise": float((np.abs(a - b) / (2e-2 * np.maximum(np.abs(b), rms))).max())})
    return out


def fit_c(per_layer) -> float:
    """c of rel_l2(l) = c * sqrt(l), least squares over the layers l >= 1."""
    pts = [(math.sqrt(p["layer"]), p["rel_l2"]) for p in per_layer if p["layer"] >= 1]
    return sum(s * d for s, d in pts) / sum(s * s for s, _ in pts)


def stored_c() -> float:
    with open(OUT) as f:
        return json.load(f)["c"]


def l2_bound(layers: int) -> float:
    return 1.3 * stored_c() * math.sqrt(layers)


def elementwise_factor(layers: int, n_elements: int) -> float:
    return (math.sqrt(2.0 * math.log(n_elements)) + 1.0) * stored_c() * math.sqrt(layers) / 2e-2


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--layers", type=int, default=6)
    ap.add_argument("--rows", type=int, default=16)
    a = ap.parse_args()
    per_layer = measure(a.layers, a.rows)
    c = fit_c(per_layer)
    with open(OUT, "w") as f:
        json.dump({"shape": "LLADA_8B", "layers": a.layers, "rows": a.rows, "c": c, "per_layer": per_layer}, f, indent=1)
    for p in per_layer:
        print(p, "c*sqrt(l) = %.2e" % (c * math.sqrt(p["layer"])))
    print("c = %.3e; 32 layers: l2 bound %.2e" % (c, c * math.sqrt(32)))


if __name__ == "__main__":
    main()
