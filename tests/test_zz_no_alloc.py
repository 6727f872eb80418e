"""odb_gemm_static_scratch: the GEMM for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off the table: every byte of the GPU already
belongs to their own pool, or the allocator belongs to the host application they are a plug-in of,
or the path is too latency-critical for an allocation's device-wide synchronisation.  For them the
library offers one GEMM entry point whose split-K partial sums live in a fixed array inside the
library's device image instead of a caller-lent buffer.  This file checks that it gives the same
numbers as the ordinary entry point (odb_debug_gemm, which gets its scratch from the caller), twice
in a row with different inputs - the second call finds the first call's partial sums still in the
shared array and must not be disturbed by them - and with the product written out in float64, that it
refuses problems larger than the array without launching anything, and that a call leaves the amount of
free device memory exactly as it found it.

The file name sorts last on purpose: if this check ever fails, a run that stops at the first failure
has already been through every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import synth
from gpu_common import engine, requires_gpu


def _inputs(E, M, N, K, seed):
    x = E.bits_to_device(synth.normal_bf16(seed, 200, (M, K), 1.0), "cuda")
    w = E.bits_to_device(synth.normal_bf16(seed, 201, (N, K), 0.05), "cuda")
    return x, w


@requires_gpu
def test_static_scratch_gemm_matches_caller_scratch_gemm_twice():
    E = engine()
    # first call: three K splits of a 32 x 768 product leave 3 * 32 * 768 partial sums in the array
    x1, w1 = _inputs(E, 32, 768, 256, seed=11)
    ref1 = E.debug_gemm(x1, w1, 3)
    got1 = E.gemm_static_scratch(x1, w1, 3)
    # second call, right after it: other shape, other data, fewer splits (stale partials lie beyond)
    x2, w2 = _inputs(E, 48, 512, 688, seed=12)
    ref2 = E.debug_gemm(x2, w2, 2)
    got2 = E.gemm_static_scratch(x2, w2, 2)
    # third: more than 128 rows and an even number of weight tiles, the CTA-pair kernel (200 x 512 x 2 splits)
    x3, w3 = _inputs(E, 200, 512, 512, seed=14)
    ref3 = E.debug_gemm(x3, w3, 2)
    got3 = E.gemm_static_scratch(x3, w3, 2)
    torch.cuda.synchronize()
    for got, ref, x, w in ((got1, ref1, x1, w1), (got2, ref2, x2, w2), (got3, ref3, x3, w3)):
        got, ref = got.cpu().numpy().astype(np.float64), ref.cpu().numpy().astype(np.float64)
        xf, wf = x.float().cpu().numpy().astype(np.float64), w.float().cpu().numpy().astype(np.float64)
        scale = (np.abs(xf) @ np.abs(wf).T).max()
        assert np.abs(got - ref).max() <= 2e-6 * scale          # the tolerance of the GEMM tests
        assert np.array_equal(got, ref)                          # same kernel, same split order: identical
        assert np.abs(got - xf @ wf.T).max() <= 2e-6 * scale     # and against the product itself, in float64
    # and again the first problem: the array now holds the second call's partial sums
    assert torch.equal(E.gemm_static_scratch(x1, w1, 3), ref1)


@requires_gpu
def test_static_scratch_gemm_rejects_what_does_not_fit():
    E = engine()
    from paper_2511_21759_b200 import binding as B
    M, N, K = 64, 16384, 256                                      # 2 splits * 64 * 16384 * 4 B = 8 MiB: fits exactly
    x, w = _inputs(E, M, N, K, seed=13)
    assert torch.equal(E.gemm_static_scratch(x, w, 2), E.debug_gemm(x, w, 2))
    with pytest.raises(B.OdbError) as e:
        E.gemm_static_scratch(x, w, 4)                            # 16 MiB of partial sums: beyond the array
    assert e.value.status == B.ODB_ERR_WORKSPACE
    # a refused call launches nothing: an output buffer filled with a sentinel comes back untouched
    st = torch.cuda.current_stream()
    wp = E.pack_weight(w)
    out = torch.full((M, N), -7.25, dtype=torch.float32, device="cuda")
    assert B.lib().odb_gemm_static_scratch(x.data_ptr(), wp.data_ptr(), out.data_ptr(), M, N, K, 4,
                                           C.c_void_p(st.cuda_stream)) == B.ODB_ERR_WORKSPACE
    torch.cuda.synchronize()
    assert bool((out == -7.25).all())
    assert B.lib().odb_gemm_static_scratch(None, w.data_ptr(), x.data_ptr(), M, N, K, 1,
                                           C.c_void_p(st.cuda_stream)) == B.ODB_ERR_ARG


@requires_gpu
def test_static_scratch_gemm_allocates_nothing():
    """What the entry point is for: once the library is loaded and the array's address has been looked up (the
    first call), a call changes the device's free memory by not one byte.  Inputs and output are created
    before the measurement; they are the caller's."""
    E = engine()
    from paper_2511_21759_b200 import binding as B
    M, N, K = 32, 768, 256
    x, w = _inputs(E, M, N, K, seed=15)
    wp = E.pack_weight(w)
    out = torch.empty(M, N, dtype=torch.float32, device="cuda")
    st = torch.cuda.current_stream()
    call = lambda: B.lib().odb_gemm_static_scratch(x.data_ptr(), wp.data_ptr(), out.data_ptr(), M, N, K, 3,
                                                   C.c_void_p(st.cuda_stream))
    assert call() == B.ODB_OK                                     # warm-up: module load, address look-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        assert call() == B.ODB_OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.equal(out, E.debug_gemm(x, w, 3))
