"""Seeded synthetic inputs: model shapes, bf16 weights, token ids, length schedules.

This module produces *data only*.  It holds none of the method's arithmetic, so both the
CPU oracle's tests and the CUDA path's tests/bench may draw their inputs from it without
sharing any code of the computation itself.  The generator proper is `gen.c` (counter based,
transcendental free, bit reproducible); this file compiles it on first use and wraps it.

Weights are returned as numpy uint16 arrays holding bf16 bit patterns (numpy has no bf16).
"""
from __future__ import annotations

import ctypes
import dataclasses
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libodb_synth.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into libodb_synth.so next to it (gcc, OpenMP)."""
    src = os.path.join(_HERE, "gen.c")
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(src):
        subprocess.check_call(
            ["gcc", "-O3", "-fopenmp", "-shared", "-fPIC", src, "-o", _SO])
    return _SO


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_SO)
        u64 = ctypes.c_uint64
        lib.synth_normal_bf16.argtypes = [u64, u64, u64, u64, ctypes.c_float, ctypes.c_void_p]
        lib.synth_normal_bf16.restype = None
        lib.synth_tokens.argtypes = [u64, u64, u64, ctypes.c_int32, ctypes.c_int32,
                                     ctypes.c_int32, ctypes.c_void_p]
        lib.synth_tokens.restype = None
        lib.synth_uniform_f32.argtypes = [u64, u64, u64, ctypes.c_void_p]
        lib.synth_uniform_f32.restype = None
        _lib = lib
    return _lib


# ----------------------------------------------------------------------------- shapes

@dataclasses.dataclass(frozen=True)
class ModelShape:
    """Shape of the LLaDA-style bidirectional transformer (pre-norm, MHA, SwiGLU, RoPE)."""
    n_layers: int
    d_model: int
    n_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    mask_id: int
    eos_id: int
    rope_theta: float = 500000.0
    rms_eps: float = 1e-5
    w_std: float = 0.02          # standard deviation of every layer matrix and the embedding
    lm_std: float = 0.02         # standard deviation of the LM head

    def with_layers(self, n_layers: int) -> "ModelShape":
        return dataclasses.replace(self, n_layers=n_layers)


TINY = ModelShape(n_layers=2, d_model=256, n_heads=4, head_dim=64, d_ffn=688, vocab=2048,
                  mask_id=2047, eos_id=2046)
# same tiny shape with unit-gain layers and a sharp LM head: predictions depend on position and
# confidences straddle the accept threshold, so the threshold branch, multi-token accepts and
# jump-share misses all occur (they never do with N(0, 0.02) weights)
TINY_PEAKY = dataclasses.replace(TINY, w_std=0.0625, lm_std=0.5)
# the tiny model with the 8B shape's head dimension (2 heads of 128): exercises the kernels that exist
# for head dim 128 only, at a size the oracle finishes in seconds
TINY_HD128 = dataclasses.replace(TINY, n_heads=2, head_dim=128)
LLADA_8B = ModelShape(n_layers=32, d_model=4096, n_heads=32, head_dim=128, d_ffn=12288,
                      vocab=126464, mask_id=126336, eos_id=126081)

# tensor ids of the counter-based generator
TID_EMBED = 1
TID_LM_HEAD = 2
TID_LAYER0 = 16          # layer l: TID_LAYER0 + 8*l + {0: wq, 1: wk, 2: wv, 3: wo, 4: wg, 5: wu, 6: wd}
LAYER_TENSORS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd")
WEIGHT_STD = 0.02


def layer_tensor_shape(shape: ModelShape, name: str) -> tuple[int, int]:
    d, f = shape.d_model, shape.d_ffn
    return {"wq": (d, d), "wk": (d, d), "wv": (d, d), "wo": (d, d),
            "wg": (f, d), "wu": (f, d), "wd": (d, f)}[name]


def normal_bf16(seed: int, tensor_id: int, shape: tuple[int, ...], std: float = WEIGHT_STD,
                offset: int = 0) -> np.ndarray:
    """bf16 bit patterns (uint16) of N(0, std^2) deviates for elements [offset, offset+n)."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)
    _load().synth_normal_bf16(seed, tensor_id, offset, n, std, out.ctypes.data)
    return out.reshape(shape)


def embed_bits(shape: ModelShape, seed: int = 0) -> np.ndarray:
    return normal_bf16(seed, TID_EMBED, (shape.vocab, shape.d_model), shape.w_std)


def lm_head_bits(shape: ModelShape, seed: int = 0) -> np.ndarray:
    return normal_bf16(seed, TID_LM_HEAD, (shape.vocab, shape.d_model), shape.lm_std)


def layer_bits(shape: ModelShape, layer: int, seed: int = 0) -> dict[str, np.ndarray]:
    """All seven matrices of one layer, each [out_features][in_features] (K contiguous)."""
    return {name: normal_bf16(seed, TID_LAYER0 + 8 * layer + i, layer_tensor_shape(shape, name), shape.w_std)
            for i, name in enumerate(LAYER_TENSORS)}


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float32 (a re-interpretation, no arithmetic)."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def tokens(seed: int, stream: int, n: int, shape: ModelShape) -> np.ndarray:
    """n prompt ids uniform over the vocabulary without the [MASK] and [EOS] ids."""
    out = np.empty(n, dtype=np.int32)
    _load().synth_tokens(seed, stream, n, shape.vocab, shape.mask_id, shape.eos_id,
                         out.ctypes.data)
    return out


def uniform(seed: int, stream: int, n: int) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)
    _load().synth_uniform_f32(seed, stream, n, out.ctypes.data)
    return out


def sequence(seed: int, stream: int, prompt_len: int, gen_len: int, shape: ModelShape) -> np.ndarray:
    """Prompt ids followed by gen_len [MASK] ids."""
    x = np.full(prompt_len + gen_len, shape.mask_id, dtype=np.int32)
    x[:prompt_len] = tokens(seed, stream, prompt_len, shape)
    return x


def shrink_schedule(seed: int, n_seq: int, gen_len: int, lo_frac: float = 0.25,
                    hi_frac: float = 0.5) -> np.ndarray:
    """Per-sequence target response lengths, uniform in [lo_frac, hi_frac] of the allocation.

    Stands in for adaptive length prediction firing on a trained model: with random weights
    no [EOS] confidence ever passes the truncate threshold, so the batch-16 workload drives
    the same length lever with these seeded targets.
    """
    u = uniform(seed, 0x5C4ED, n_seq)
    return (gen_len * (lo_frac + (hi_frac - lo_frac) * u)).astype(np.int32)


# ----------------------------------------------------------------------------- workloads

@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    shape: ModelShape
    batch: int
    prompt_len: int
    gen_len: int
    block_len: int
    n_copies: int
    accept_threshold: float = 0.9
    truncate_threshold: float = 0.9
    with_lm_head: bool = True


WORKLOADS = {
    # tiny end-to-end case the oracle finishes in seconds
    "cfg1_tiny": Workload("cfg1_tiny", TINY, 1, 64, 64, 16, 1),
    "cfg1_tiny_c4": Workload("cfg1_tiny_c4", TINY, 1, 64, 64, 16, 4),
    "peaky_c1": Workload("peaky_c1", TINY_PEAKY, 1, 64, 64, 16, 1),
    "peaky_c4": Workload("peaky_c4", TINY_PEAKY, 1, 64, 64, 16, 4),
    "peaky_c8": Workload("peaky_c8", TINY_PEAKY, 1, 64, 64, 16, 8),
    # one 8B-shaped layer, context 512, block 32, 1 and 4 copies
    "cfg2_layer_c1": Workload("cfg2_layer_c1", LLADA_8B.with_layers(1), 1, 256, 256, 32, 1,
                              with_lm_head=False),
    "cfg2_layer_c4": Workload("cfg2_layer_c4", LLADA_8B.with_layers(1), 1, 256, 256, 32, 4,
                              with_lm_head=False),
    # one 8B-shaped layer, 16 ragged sequences, block 64, 4 copies: the batched step's kernels on a small footprint
    "cfg2_layer_b16_c4": Workload("cfg2_layer_b16_c4", LLADA_8B.with_layers(1), 16, 1024, 1024, 64, 4,
                                  with_lm_head=False),
    # full 8B shape
    "cfg3_8b_c1": Workload("cfg3_8b_c1", LLADA_8B, 1, 512, 256, 32, 1),
    "cfg4_8b_c4": Workload("cfg4_8b_c4", LLADA_8B, 1, 512, 512, 32, 4),
    "cfg5_8b_b16": Workload("cfg5_8b_b16", LLADA_8B, 16, 1024, 1024, 64, 4),
}
