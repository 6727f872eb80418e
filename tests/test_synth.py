"""The seeded generator: reproducible, chunk invariant, right distribution and exclusions."""
import numpy as np

import synth


def test_normal_is_counter_based_and_chunk_invariant():
    a = synth.normal_bf16(0, 7, (4096,))
    b = np.concatenate([synth.normal_bf16(0, 7, (1000,)), synth.normal_bf16(0, 7, (3096,), offset=1000)])
    assert (a == b).all()
    assert (a != synth.normal_bf16(1, 7, (4096,))).mean() > 0.9       # seed matters
    assert (a != synth.normal_bf16(0, 8, (4096,))).mean() > 0.9       # tensor id matters


def test_normal_distribution():
    f = synth.bf16_bits_to_f32(synth.normal_bf16(0, 3, (512, 512))).astype(np.float64)
    assert abs(f.mean()) < 2e-4
    assert abs(f.std() - 0.02) < 2e-4
    assert np.abs(f).max() <= 6 * 0.02 * 1.01
    # standard normal quantiles: 68.27 % within one sigma, 95.45 % within two
    assert abs((np.abs(f) < 0.02).mean() - 0.6827) < 1e-2
    assert abs((np.abs(f) < 0.04).mean() - 0.9545) < 1e-2


def test_bf16_bits_are_exact_bf16():
    bits = synth.normal_bf16(0, 3, (1000,))
    f = synth.bf16_bits_to_f32(bits)
    assert ((f.view(np.uint32) & 0xFFFF) == 0).all()
    assert ((f.view(np.uint32) >> 16).astype(np.uint16) == bits).all()


def test_tokens_exclude_mask_and_eos():
    for shape in (synth.TINY, synth.LLADA_8B):
        t = synth.tokens(0, 0, 20000, shape)
        assert t.min() >= 0 and t.max() < shape.vocab
        assert (t != shape.mask_id).all() and (t != shape.eos_id).all()
    t2 = synth.tokens(0, 1, 100, synth.TINY)
    assert (t2 != synth.tokens(0, 0, 100, synth.TINY)).any()
    x = synth.sequence(0, 0, 64, 64, synth.TINY)
    assert (x[64:] == synth.TINY.mask_id).all() and (x[:64] == synth.tokens(0, 0, 64, synth.TINY)).all()


def test_shrink_schedule_range():
    t = synth.shrink_schedule(0, 16, 1024)
    assert t.shape == (16,) and t.min() >= 256 and t.max() <= 512 and len(set(t.tolist())) > 8


def test_layer_shapes():
    w = synth.layer_bits(synth.TINY, 1)
    assert w["wq"].shape == (256, 256) and w["wg"].shape == (688, 256) and w["wd"].shape == (256, 688)
    assert (w["wq"] != w["wk"]).any()
