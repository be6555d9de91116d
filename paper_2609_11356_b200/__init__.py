"""rg — reduction-order-fixed GEMM and row reductions for B200 (sm_100a).

Thin Python binding over the C ABI of ``include/rg.h``; torch supplies device memory and
streams only.  Every arithmetic step runs in the CUDA library.
"""
from ._cabi import (RG_ATOM_SCALAR, RG_ATOM_TC_BF16_K16, RG_ATOM_TC_F8_K32, RG_BF16, RG_COLOP_DOT, RG_COLOP_SUM, RG_F16, RG_F32, RG_F8E4M3, RG_OP_RMSNORM, RG_OP_SOFTMAX_DENOM,
                    RG_OP_SUM, RG_TREE_BALANCED, RG_TREE_LEFT)
from .api import (RgError, rg_attention, rg_attn_desc, rg_desc, rg_desc_class, rg_desc_validate, rg_device_status, rg_gemm, rg_gemm_host, rg_gemm_noalloc,
                  rg_gemm_workspace_bytes, rg_reduce_cols, rg_reduce_cols_workspace_bytes, rg_reduce_rows, rg_reduce_rows_host, rg_status_string)

__all__ = [n for n in dir() if n.startswith(("rg_", "RG_", "Rg"))]
