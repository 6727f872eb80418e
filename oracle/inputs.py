"""Builds the oracle's `Model` from the seeded synthetic generator.  TEST INFRASTRUCTURE ONLY.

Only data crosses here: bf16 bit patterns from `synth` are widened to the oracle's dtype.
"""
from __future__ import annotations

import numpy as np

import synth
from . import odb_oracle as O


def model_from_synth(shape: synth.ModelShape, seed: int = 0, dtype=np.float64, *,
                     with_lm_head: bool = True, cache_layers: bool = True) -> O.Model:
    """Random-weight model of the given shape; RMSNorm gains are 1.

    cache_layers=False regenerates a layer's matrices at every use (large shapes: keeps only
    one layer resident)."""
    d = shape.d_model
    ones = np.ones(d, dtype=dtype)
    store: dict = {}

    def layer(l: int) -> dict:
        if l in store:
            return store[l]
        bits = synth.layer_bits(shape, l, seed)
        w = {k: synth.bf16_bits_to_f32(v).astype(dtype) for k, v in bits.items()}
        w["g1"] = ones
        w["g2"] = ones
        if cache_layers:
            store[l] = w
        return w

    embed = synth.bf16_bits_to_f32(synth.embed_bits(shape, seed)).astype(dtype)
    lm = synth.bf16_bits_to_f32(synth.lm_head_bits(shape, seed)).astype(dtype) if with_lm_head else None
    return O.Model(n_layers=shape.n_layers, d_model=d, n_heads=shape.n_heads, head_dim=shape.head_dim,
                   d_ffn=shape.d_ffn, vocab=shape.vocab, mask_id=shape.mask_id, eos_id=shape.eos_id,
                   rope_theta=shape.rope_theta, rms_eps=shape.rms_eps, embed=embed, lm_head=lm,
                   final_gain=ones, layer=layer)
