"""Shared helpers of the GPU parity tests (no test functions here)."""
import numpy as np
import pytest
import torch

import synth
from oracle import odb_oracle as O
from oracle.inputs import model_from_synth

requires_gpu = pytest.mark.gpu


def engine():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2511_21759_b200 import engine as E
    return E


def logits_close(got, want, tol=2e-2):
    """|d| <= tol * max(|l_oracle|, rms(row)): 2e-2 relative, with the row's RMS as the floor
    that keeps the relative measure meaningful for logits near zero."""
    want = np.asarray(want, dtype=np.float64)
    rms = np.sqrt((want * want).mean(axis=-1, keepdims=True))
    bound = tol * np.maximum(np.abs(want), rms)
    err = np.abs(np.asarray(got, dtype=np.float64) - want)
    return bool((err <= bound).all()), float((err / bound).max())


def bf16_bits_to_f64(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def compare_traces(gpu_trace, oracle_trace, seq=0, near_tie=1e-3):
    """Walks both traces; returns (n_equal, divergence) where divergence is None or a dict with the
    iteration index, both records and the oracle's decision margin there."""
    n = min(len(gpu_trace), len(oracle_trace))
    for i in range(n):
        g = gpu_trace[i]["seqs"][seq]
        o = oracle_trace[i]
        same = (gpu_trace[i]["kind"] == o["kind"] and g["accepted"] == sorted(o["accepted"])
                and g["chain"] == o["chain"])
        if not same:
            return i, {"iter": i, "gpu": g, "oracle": o, "margin": o["margin"],
                       "near_tie": o["margin"] < near_tie}
    if len(gpu_trace) != len(oracle_trace):
        return n, {"iter": n, "gpu": None, "oracle": None, "margin": np.inf, "near_tie": False}
    return n, None
