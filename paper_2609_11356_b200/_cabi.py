"""ctypes mirror of include/rg.h: structures, prototypes and the loader.

Argument marshalling only.  If the CUDA library has not been built the loader raises; there is
no fallback path of any kind.
"""
from __future__ import annotations

import ctypes as C
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "librg.so")

RG_OK = 0
STATUS_NAMES = {0: "RG_OK", 1: "RG_ERR_NULL", 2: "RG_ERR_INVALID_DESC", 3: "RG_ERR_UNSUPPORTED", 4: "RG_ERR_SHAPE",
                5: "RG_ERR_ALIGNMENT", 6: "RG_ERR_WORKSPACE", 7: "RG_ERR_CUDA", 8: "RG_ERR_TIMEOUT"}
RG_BF16, RG_F32, RG_F16, RG_F8E4M3 = 0, 1, 2, 3
RG_TREE_LEFT, RG_TREE_BALANCED = 0, 1
RG_ATOM_TC_BF16_K16, RG_ATOM_SCALAR, RG_ATOM_TC_F8_K32 = 0, 1, 2
RG_COLOP_SUM, RG_COLOP_DOT = 0, 1
RG_OP_SUM, RG_OP_RMSNORM, RG_OP_SOFTMAX_DENOM = 0, 1, 2
RG_MAX_CUTS = 63
RG_NOALLOC_WS_BYTES = 8 << 20
RG_SELFTEST_WAIT_CODE = 0xE00

# every symbol include/rg.h declares
EXPORTS = ["rg_desc_init", "rg_desc_validate", "rg_desc_class", "rg_gemm_workspace_bytes", "rg_gemm",
           "rg_reduce_rows", "rg_gemm_host_scratch_bytes", "rg_gemm_host", "rg_reduce_rows_host_scratch_bytes",
           "rg_reduce_rows_host", "rg_device_status", "rg_status_string", "rg_gemm_noalloc",
           "rg_reduce_cols_workspace_bytes", "rg_reduce_cols", "rg_attention", "rg_selftest_bounded_wait", "rg_selftest_exp"]


class rg_attn_desc_t(C.Structure):
    _fields_ = [("size", C.c_uint32), ("heads", C.c_uint32), ("block_n", C.c_uint32), ("block_m", C.c_uint32), ("scale", C.c_float),
                ("sum_tree", C.c_uint8), ("p_dtype", C.c_uint8), ("mask", C.c_uint8), ("div_place", C.c_uint8),
                ("exp_base", C.c_uint8), ("_pad", C.c_uint8 * 3)]


class rg_desc_t(C.Structure):
    _fields_ = [("size", C.c_uint32),
                ("BM", C.c_uint16), ("BN", C.c_uint16), ("BK", C.c_uint16),
                ("stages", C.c_uint8), ("cta_group", C.c_uint8), ("raster", C.c_uint8), ("split_merge", C.c_uint8),
                ("in_dtype", C.c_uint8), ("acc_dtype", C.c_uint8), ("partial_dtype", C.c_uint8), ("merge_dtype", C.c_uint8),
                ("atom", C.c_uint8), ("k_tail", C.c_uint8), ("fma", C.c_uint8), ("tree", C.c_uint8),
                ("n_cuts", C.c_uint32), ("cuts", C.c_uint32 * RG_MAX_CUTS), ("inner_span", C.c_uint32),
                ("gemv_layout", C.c_uint8), ("gemv_fold", C.c_uint8), ("sm_share", C.c_uint8), ("b_static", C.c_uint8)]


class rg_tensor_t(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("rows", C.c_int64), ("cols", C.c_int64), ("ld", C.c_int64)]


class rg_epilogue_t(C.Structure):
    _fields_ = [("bias", C.c_void_p), ("bias_dtype", C.c_int32), ("act", C.c_int32),
                ("residual", C.c_void_p), ("residual_dtype", C.c_int32), ("ldr", C.c_int64)]


class rg_reduce_args_t(C.Structure):
    _fields_ = [("weight", C.c_void_p), ("weight_dtype", C.c_int32), ("eps", C.c_float), ("aux_out", C.c_void_p)]


_lib = None


def load():
    """Load librg.so.  Raises if it is missing: the product has no other path."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build the CUDA library first "
            "(python -m paper_2609_11356_b200.build, or __graft_entry__.build()).")
    L = C.CDLL(LIB_PATH)
    D, T, E, A = C.POINTER(rg_desc_t), C.POINTER(rg_tensor_t), C.POINTER(rg_epilogue_t), C.POINTER(rg_reduce_args_t)
    i64, vp, sz = C.c_int64, C.c_void_p, C.c_size_t
    L.rg_desc_init.restype = None; L.rg_desc_init.argtypes = [D]
    L.rg_desc_validate.restype = C.c_int; L.rg_desc_validate.argtypes = [D, i64, i64, i64]
    L.rg_desc_class.restype = C.c_uint64; L.rg_desc_class.argtypes = [D]
    L.rg_gemm_workspace_bytes.restype = sz; L.rg_gemm_workspace_bytes.argtypes = [D, i64, i64]
    L.rg_gemm.restype = C.c_int; L.rg_gemm.argtypes = [D, T, T, T, E, vp, sz, vp]
    L.rg_reduce_rows.restype = C.c_int; L.rg_reduce_rows.argtypes = [D, C.c_int, T, T, A, vp]
    L.rg_gemm_host_scratch_bytes.restype = sz; L.rg_gemm_host_scratch_bytes.argtypes = [D, i64, i64, i64, C.c_int32, E]
    L.rg_gemm_host.restype = C.c_int; L.rg_gemm_host.argtypes = [D, T, T, T, E, vp, sz, vp]
    L.rg_reduce_rows_host_scratch_bytes.restype = sz; L.rg_reduce_rows_host_scratch_bytes.argtypes = [C.c_int, T, T]
    L.rg_reduce_rows_host.restype = C.c_int; L.rg_reduce_rows_host.argtypes = [D, C.c_int, T, T, A, vp, sz, vp]
    L.rg_reduce_cols_workspace_bytes.restype = sz; L.rg_reduce_cols_workspace_bytes.argtypes = [i64, i64]
    L.rg_reduce_cols.restype = C.c_int; L.rg_reduce_cols.argtypes = [D, C.c_int, T, T, T, vp, sz, vp]
    L.rg_attention.restype = C.c_int; L.rg_attention.argtypes = [C.POINTER(rg_attn_desc_t), T, T, T, T, vp]
    L.rg_gemm_noalloc.restype = C.c_int; L.rg_gemm_noalloc.argtypes = [D, T, T, T, E, vp]
    L.rg_selftest_bounded_wait.restype = C.c_int; L.rg_selftest_bounded_wait.argtypes = [C.c_uint64, vp, vp]
    L.rg_selftest_exp.restype = C.c_int; L.rg_selftest_exp.argtypes = [C.c_int32, vp, vp, C.c_int64, vp]
    L.rg_device_status.restype = C.c_int; L.rg_device_status.argtypes = [C.POINTER(C.c_uint32)]
    L.rg_status_string.restype = C.c_char_p; L.rg_status_string.argtypes = [C.c_int]
    _lib = L
    return L
