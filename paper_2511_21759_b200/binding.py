"""ctypes binding of libodb.so: the same names as include/odb.h, argument marshalling only.

Every step of the path runs inside the library's kernels.  PyTorch appears here only as the
owner of device memory and streams.  Importing this module never needs a GPU; loading the
library does not either (so the exported symbols can be checked on a CPU-only machine), but
any compute call without the library or without a device fails loudly.
"""
from __future__ import annotations

import ctypes as C
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libodb.so")

ODB_OK, ODB_ERR_ARG, ODB_ERR_SHAPE, ODB_ERR_WORKSPACE, ODB_ERR_STATE, ODB_ERR_CUDA, ODB_ERR_TIMEOUT = 0, -1, -2, -3, -4, -5, -6
ODB_MAX_COPIES, ODB_MAX_RANKS, ODB_MAX_CHAIN = 8, 4, 5
ODB_STATIC_SCRATCH_BYTES = 8 << 20
KINDS = ("gemm", "attention", "elementwise", "confidence", "control")


class OdbError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().odb_status_string(status).decode()
        if status == ODB_ERR_CUDA:
            msg += ": " + lib().odb_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})")


class odb_config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "head_dim", "d_ffn", "vocab",
                                         "mask_id", "eos_id")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int32) for n in ("max_batch", "max_seq", "max_block", "max_copies", "with_lm_head",
                                         "tp_world", "tp_rank")]


class odb_weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("lm_head", C.c_void_p), ("final_norm", C.c_void_p),
                ("norm1", C.POINTER(C.c_void_p)), ("wqkv", C.POINTER(C.c_void_p)), ("wo", C.POINTER(C.c_void_p)),
                ("norm2", C.POINTER(C.c_void_p)), ("wgu", C.POINTER(C.c_void_p)), ("wd", C.POINTER(C.c_void_p))]


class odb_decode_params(C.Structure):
    _fields_ = [("block_len", C.c_int32), ("n_copies", C.c_int32), ("accept_threshold", C.c_float),
                ("truncate_threshold", C.c_float), ("stage2_min_decoded", C.c_int32), ("alp", C.c_int32),
                ("pick_best", C.c_int32), ("sampling", C.c_int32), ("sample_steps", C.c_int32)]


class odb_result(C.Structure):
    _fields_ = [("masks_left", C.c_int32), ("n_accepted", C.c_int32), ("chain_len", C.c_int32),
                ("chain", C.c_int32 * ODB_MAX_CHAIN), ("gen_len", C.c_int32), ("block_start", C.c_int32),
                ("block_end", C.c_int32), ("accepted_pos", C.c_int32 * 64), ("accepted_tok", C.c_int32 * 64)]


# name -> (restype, argtypes); the list the header declares
SIGNATURES = {
    "odb_status_string": (C.c_char_p, [C.c_int32]),
    "odb_last_cuda_error": (C.c_char_p, []),
    "odb_packed_weight_bytes": (C.c_size_t, [C.c_int32, C.c_int32]),
    "odb_pack_weight": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "odb_packed_gate_up_bytes": (C.c_size_t, [C.c_int32, C.c_int32]),
    "odb_pack_gate_up": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]),
    "odb_model_create": (C.c_int32, [C.POINTER(odb_config), C.POINTER(odb_weights), C.POINTER(C.c_void_p)]),
    "odb_model_destroy": (C.c_int32, [C.c_void_p]),
    "odb_kv_bytes": (C.c_size_t, [C.POINTER(odb_config)]),
    "odb_workspace_bytes": (C.c_size_t, [C.POINTER(odb_config)]),
    "odb_session_create": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p, C.c_size_t, C.c_void_p,
                                       C.POINTER(C.c_void_p)]),
    "odb_session_destroy": (C.c_int32, [C.c_void_p]),
    "odb_session_set_sequence": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_int32]),
    "odb_session_set_gen_len": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32]),
    "odb_session_get_tokens": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]),
    "odb_session_set_sampling_noise": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_int32, C.c_int32]),
    "odb_session_set_active": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32]),
    "odb_session_status": (C.c_int32, [C.c_void_p]),
    "odb_refresh_prefill": (C.c_int32, [C.c_void_p, C.POINTER(odb_decode_params), C.c_void_p]),
    "odb_block_decode_step": (C.c_int32, [C.c_void_p, C.POINTER(odb_decode_params)]),
    "odb_unmask_accept": (C.c_int32, [C.c_void_p, C.POINTER(odb_decode_params), C.c_int32, C.POINTER(odb_result)]),
    "odb_decode_block_resident": (C.c_int32, [C.c_void_p, C.POINTER(odb_decode_params), C.c_int32, C.POINTER(odb_result),
                                              C.c_int32, C.POINTER(C.c_int32)]),
    "odb_debug_set_logit_dump": (C.c_int32, [C.c_void_p, C.c_int32]),
    "odb_debug_expire_wait": (C.c_int32, [C.c_void_p, C.c_int64]),
    "odb_debug_read": (C.c_int32, [C.c_void_p, C.c_int32, C.c_void_p, C.c_size_t, C.POINTER(C.c_int32)]),
    "odb_debug_gemm": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_int32, C.c_int32,
                                   C.c_int32, C.c_int32, C.c_void_p]),
    "odb_gemm_static_scratch": (C.c_int32, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                            C.c_void_p]),
    "odb_session_profile": (C.c_int32, [C.c_void_p, C.c_int32]),
    "odb_session_profile_read": (C.c_int32, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "odb_session_tp_buffers": (C.c_int32, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_size_t), C.POINTER(C.c_void_p),
                                           C.POINTER(C.c_size_t), C.POINTER(C.c_void_p), C.POINTER(C.c_size_t)]),
    "odb_session_tp_attach": (C.c_int32, [C.c_void_p, C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.POINTER(C.c_void_p)]),
    "odb_tp_enable_peer_access": (C.c_int32, [C.c_int32]),
    "odb_tp_vocab_range": (C.c_int32, [C.POINTER(odb_config), C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]),
    "odb_tp_segment_count": (C.c_int32, [C.POINTER(odb_config)]),
    "odb_debug_tp_segments": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int32]),
    "odb_debug_tp_alone": (C.c_int32, [C.c_void_p, C.c_int32]),
    "odb_debug_tp_expire_wait": (C.c_int32, [C.c_void_p, C.c_int32, C.c_int64]),
    "odb_measure_read_bandwidth": (C.c_int32, [C.c_void_p, C.c_size_t, C.c_int32, C.c_void_p, C.POINTER(C.c_double)]),
    "odb_measure_bulk_read_bandwidth": (C.c_int32, [C.c_void_p, C.c_size_t, C.c_int32, C.c_void_p, C.POINTER(C.c_double)]),
    "odb_step_algorithmic_bytes": (C.c_double, [C.POINTER(odb_config), C.c_int32]),
}

_lib = None


def lib() -> C.CDLL:
    """Loads libodb.so (built in-tree by paper_2511_21759_b200.build); never falls back."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -c 'import __graft_entry__ as g; g.build()'` "
                               "(there is no CPU fallback)")
        l = C.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def check(status: int, where: str) -> None:
    if status != ODB_OK:
        raise OdbError(status, where)
