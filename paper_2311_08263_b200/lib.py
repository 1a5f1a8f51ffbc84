"""Thin ctypes binding of the C ABI in include/fastcot.h: argument marshalling only.

Every function here has the name of the C entry point it calls.  Nothing is computed in
Python, and there is no fallback: if the CUDA library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfastcot.so")

FC_F32, FC_BF16 = 0, 1
FC_REFILL_PROMPT_CYCLE, FC_REFILL_PAD = 0, 1
FC_FLAG_SIMT_GEMM, FC_FLAG_NO_PDL, FC_FLAG_NO_CHAIN, FC_FLAG_NO_FFN_SPLIT, FC_FLAG_NO_CTA_PAIRS = 1, 4, 8, 16, 32
FC_OK = 0
FC_NOALLOC_SCRATCH_BYTES = 8 << 20
FC_CLASSES = ["embed", "qkv", "rope", "attn", "oproj", "gateup", "down", "head", "accept", "chain"]
FC_ERR_ARG, FC_ERR_SHAPE, FC_ERR_CAPACITY, FC_ERR_TOKEN_RANGE = -1, -2, -3, -4
FC_ERR_STATE, FC_ERR_BAD_WINDOW, FC_ERR_DEVICE_TIMEOUT, FC_ERR_CUDA = -5, -6, -7, -8

EXPORTS = ["fc_kv_bytes", "fc_workspace_bytes", "fc_init", "fc_prefill", "fc_jacobi_step", "fc_generate",
           "fc_set_window", "fc_finish_with_trigger", "fc_debug_inject_timeout", "fc_debug_check_guards",
           "fc_debug_set_state", "fc_debug_logits", "fc_get_state", "fc_bench_steps", "fc_profile_step",
           "fc_last_launch_count", "fc_destroy", "fc_strerror", "fc_last_cuda_error",
           "fc_op_linear", "fc_op_accept", "fc_op_window_attention",
           "fc_op_window_attention_scratch_bytes", "fc_op_window_attention_noalloc",
           "fc_op_fused_window_attention", "fc_op_fused_window_attention_scratch_bytes"]


class fc_model_shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim",
                                         "d_ffn", "vocab", "dtype")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float),
                ("max_batch", C.c_int32), ("max_c", C.c_int32), ("max_seq", C.c_int32),
                ("bias_beta", C.c_float), ("flags", C.c_int32)]


_PP = C.POINTER(C.c_void_p)


class fc_weights(C.Structure):
    _fields_ = [("tok_emb", C.c_void_p)] + \
               [(n, _PP) for n in ("wq", "wk", "wv", "wo", "w_gate", "w_up", "w_down", "g_attn", "g_ffn")] + \
               [("g_final", C.c_void_p), ("lm_head", C.c_void_p), ("bias_perm", C.c_void_p)]


class fc_stats(C.Structure):
    _fields_ = [("steps", C.c_int64), ("tokens", C.c_int64), ("accept_hist", C.c_int32 * 65),
                ("ms_prefill", C.c_float), ("ms_steps", C.c_float)]


_lib = None


def load() -> C.CDLL:
    """Load libfastcot.so (build it first with `paper_2311_08263_b200.build.build()`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2311_08263_b200.build` "
                           "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i32p = C.c_void_p, C.c_int32, C.c_void_p
    lib.fc_kv_bytes.restype = C.c_size_t
    lib.fc_kv_bytes.argtypes = [C.POINTER(fc_model_shape)]
    lib.fc_workspace_bytes.restype = C.c_size_t
    lib.fc_workspace_bytes.argtypes = [C.POINTER(fc_model_shape)]
    lib.fc_init.argtypes = [C.POINTER(vp), C.POINTER(fc_model_shape), C.POINTER(fc_weights),
                            vp, C.c_size_t, vp, C.c_size_t, vp]
    lib.fc_prefill.argtypes = [vp, i32, i32p, i32, i32p, i32, i32, i32]
    lib.fc_jacobi_step.argtypes = [vp, i32p, i32p, i32p, i32p]
    lib.fc_generate.argtypes = [vp, i32, i32, i32, i32, i32p, i32p, C.POINTER(fc_stats)]
    lib.fc_set_window.argtypes = [vp, i32]
    lib.fc_finish_with_trigger.argtypes = [vp, i32p, i32, i32, i32, i32p, i32p]
    lib.fc_debug_inject_timeout.argtypes = [vp]
    lib.fc_debug_check_guards.argtypes = [vp, C.POINTER(C.c_int32)]
    lib.fc_debug_set_state.argtypes = [vp, i32, i32p, i32p, i32, i32]
    lib.fc_debug_logits.argtypes = [vp, vp]
    lib.fc_get_state.argtypes = [vp, i32p, i32p]
    lib.fc_bench_steps.argtypes = [vp, i32, i32, C.POINTER(C.c_float), C.POINTER(C.c_int64)]
    lib.fc_profile_step.argtypes = [vp, C.POINTER(C.c_float), C.POINTER(C.c_int32)]
    lib.fc_last_launch_count.restype = C.c_int64
    lib.fc_last_launch_count.argtypes = [vp]
    lib.fc_destroy.restype = None
    lib.fc_destroy.argtypes = [vp]
    lib.fc_strerror.restype = C.c_char_p
    lib.fc_strerror.argtypes = [C.c_int]
    lib.fc_last_cuda_error.restype = C.c_char_p
    lib.fc_last_cuda_error.argtypes = [vp]
    lib.fc_op_linear.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp]
    lib.fc_op_accept.argtypes = [vp] * 8 + [i32] * 5 + [vp]
    lib.fc_op_window_attention_scratch_bytes.restype = C.c_size_t
    lib.fc_op_window_attention_scratch_bytes.argtypes = [i32] * 7
    lib.fc_op_window_attention.argtypes = [vp] * 5 + [i32] * 8 + [vp, C.c_size_t, vp]
    lib.fc_op_window_attention_noalloc.argtypes = [vp] * 5 + [i32] * 8 + [vp]
    lib.fc_op_fused_window_attention_scratch_bytes.restype = C.c_size_t
    lib.fc_op_fused_window_attention_scratch_bytes.argtypes = [i32] * 7
    lib.fc_op_fused_window_attention.argtypes = [vp, vp, C.c_float, i32, C.c_float, vp, vp, vp, vp] + [i32] * 9 + \
                                                [vp, C.c_size_t, vp]
    _lib = lib
    return lib
