"""Python names for the C entry points (same names, argument marshalling only)."""
from __future__ import annotations

import ctypes as C
from typing import Optional, Sequence

from . import _cabi as K


class RgError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = K.load().rg_status_string(status).decode()
        super().__init__(f"{where}: {K.STATUS_NAMES.get(status, status)} ({msg})")


def _check(status: int, where: str):
    if status != K.RG_OK:
        raise RgError(status, where)


def rg_desc(*, cuts: Sequence[int] = (), tree: int = K.RG_TREE_BALANCED, fma: int = 0, BM: int = 0, BN: int = 0,
            BK: int = 0, stages: int = 0, cta_group: int = 0, raster: int = 0, split_merge: int = 0, **order_fields) -> K.rg_desc_t:
    """A descriptor with the library defaults (rg_desc_init), then the given fields."""
    d = K.rg_desc_t()
    K.load().rg_desc_init(C.byref(d))
    d.BM, d.BN, d.BK, d.stages, d.cta_group, d.raster, d.split_merge = BM, BN, BK, stages, cta_group, raster, split_merge
    d.tree, d.fma = tree, fma
    for k, v in order_fields.items():
        setattr(d, k, v)
    if "in_dtype" not in order_fields:
        d.in_dtype = K.RG_BF16
    if d.in_dtype == K.RG_F8E4M3 and "atom" not in order_fields:
        d.atom = K.RG_ATOM_TC_F8_K32           # the 8-bit operand type and the 32-wide step go together
    cuts = list(cuts)
    if len(cuts) > K.RG_MAX_CUTS:
        raise RgError(2, "rg_desc")
    d.n_cuts = len(cuts)
    for i, c in enumerate(cuts):
        d.cuts[i] = int(c)
    return d


def rg_desc_validate(d: K.rg_desc_t, M: int, N: int, Kdim: int) -> int:
    return int(K.load().rg_desc_validate(C.byref(d), M, N, Kdim))


def rg_desc_class(d: K.rg_desc_t) -> int:
    return int(K.load().rg_desc_class(C.byref(d)))


def rg_gemm_workspace_bytes(d: K.rg_desc_t, M: int, N: int) -> int:
    return int(K.load().rg_gemm_workspace_bytes(C.byref(d), M, N))


def rg_status_string(status: int) -> str:
    return K.load().rg_status_string(status).decode()


def rg_device_status() -> int:
    """Read and clear the device health word (synchronises).  0 = healthy."""
    code = C.c_uint32(0)
    K.load().rg_device_status(C.byref(code))
    return int(code.value)


def rg_selftest_exp(form: int, x, y):
    """y[i] = FORM(x[i]) by the device functions the kernels use (forms: see include/rg.h).  x, y: float32 CUDA tensors."""
    st = K.load().rg_selftest_exp(int(form), x.data_ptr(), y.data_ptr(), int(x.numel()), _stream(x))
    _check(st, "rg_selftest_exp")
    return y


def rg_selftest_bounded_wait(limit_ns: int, counter):
    """Launch the bounded-wait self-test (see include/rg.h).  `counter`: a zeroed CUDA int32/uint32
    tensor of one element; it holds 2 afterwards (both warps abandoned their wait)."""
    st = K.load().rg_selftest_bounded_wait(int(limit_ns), counter.data_ptr(), _stream(counter))
    _check(st, "rg_selftest_bounded_wait")


# ---------------------------------------------------------------- marshalling
def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.bfloat16:
        return K.RG_BF16
    if t.dtype == torch.float32:
        return K.RG_F32
    if t.dtype == torch.float16:
        return K.RG_F16
    if t.dtype == torch.float8_e4m3fn:
        return K.RG_F8E4M3
    raise TypeError(f"rg tensors are bfloat16, float16, float32 or float8_e4m3fn, got {t.dtype}")


def _tensor(t) -> K.rg_tensor_t:
    if t.dim() == 1:
        return K.rg_tensor_t(t.data_ptr(), _dtype_code(t), t.shape[0], 1, max(int(t.stride(0)), 1))
    assert t.dim() == 2 and (t.shape[1] <= 1 or t.stride(1) == 1), "rows must be contiguous"
    ld = int(t.stride(0)) if t.shape[0] > 1 else max(int(t.stride(0)), int(t.shape[1]))
    return K.rg_tensor_t(t.data_ptr(), _dtype_code(t), t.shape[0], t.shape[1], max(ld, int(t.shape[1])))


def _epilogue(bias, act, residual) -> Optional[K.rg_epilogue_t]:
    if bias is None and residual is None and not act:
        return None
    e = K.rg_epilogue_t()
    e.act = int(act)
    if bias is not None:
        e.bias, e.bias_dtype = bias.data_ptr(), _dtype_code(bias)
    if residual is not None:
        e.residual, e.residual_dtype, e.ldr = residual.data_ptr(), _dtype_code(residual), int(residual.stride(0))
    return e


def _stream(t) -> int:
    import torch
    return torch.cuda.current_stream(t.device).cuda_stream if t.is_cuda else 0


def rg_gemm(d: K.rg_desc_t, A, B, C_out, *, bias=None, act: int = 0, residual=None, ws=None):
    """C_out[M,N] = epilogue(A[M,K] @ B[N,K]^T) with the bits the descriptor fixes.
    All tensors are CUDA tensors; `ws` is a CUDA byte/float tensor of at least
    rg_gemm_workspace_bytes(d, M, N) bytes when the descriptor has cuts."""
    L = K.load()
    a, b, c = _tensor(A), _tensor(B), _tensor(C_out)
    e = _epilogue(bias, act, residual)
    ws_ptr = ws.data_ptr() if ws is not None else None
    ws_bytes = ws.numel() * ws.element_size() if ws is not None else 0
    st = L.rg_gemm(C.byref(d), C.byref(a), C.byref(b), C.byref(c), C.byref(e) if e is not None else None,
                   ws_ptr, ws_bytes, _stream(A))
    _check(st, "rg_gemm")
    return C_out


def rg_gemm_noalloc(d: K.rg_desc_t, A, B, C_out, *, bias=None, act: int = 0, residual=None):
    """rg_gemm for callers that cannot allocate device memory: the split-K workspace is a fixed
    array inside the library (at most RG_NOALLOC_WS_BYTES; larger shapes raise RG_ERR_WORKSPACE).
    Calls on one device share that array, so do not let two of them overlap on the GPU."""
    L = K.load()
    a, b, c = _tensor(A), _tensor(B), _tensor(C_out)
    e = _epilogue(bias, act, residual)
    st = L.rg_gemm_noalloc(C.byref(d), C.byref(a), C.byref(b), C.byref(c), C.byref(e) if e is not None else None,
                           _stream(A))
    _check(st, "rg_gemm_noalloc")
    return C_out


def rg_reduce_rows(d: K.rg_desc_t, op: int, x, out, *, weight=None, eps: float = 0.0, aux_out=None):
    """Row reduction with the descriptor's tree (see include/rg.h for the three operations)."""
    L = K.load()
    xt, ot = _tensor(x), _tensor(out)
    args = K.rg_reduce_args_t()
    if weight is not None:
        args.weight, args.weight_dtype = weight.data_ptr(), _dtype_code(weight)
    args.eps = float(eps)
    if aux_out is not None:
        args.aux_out = aux_out.data_ptr()
    st = L.rg_reduce_rows(C.byref(d), int(op), C.byref(xt), C.byref(ot), C.byref(args), _stream(x))
    _check(st, "rg_reduce_rows")
    return out


def rg_attn_desc(*, block_n: int, scale: float, heads: int = 1, sum_tree: int = K.RG_TREE_BALANCED, p_dtype: int = K.RG_BF16,
                 mask: int = 0, div_place: int = 0, exp_base: int = 0, block_m: int = 0) -> K.rg_attn_desc_t:
    d = K.rg_attn_desc_t()
    d.size = C.sizeof(K.rg_attn_desc_t)
    d.heads, d.block_n, d.scale = heads, block_n, scale
    d.block_m = block_m if block_m else (128 if mask else 0)
    d.sum_tree, d.p_dtype, d.mask, d.div_place, d.exp_base = sum_tree, p_dtype, mask, div_place, exp_base
    return d


def rg_attention(d: K.rg_attn_desc_t, Q, Kt, Vt, O):
    """O = attention(Q, K, V) with the descriptor's key-block recurrence.  Q [heads*Nq, d],
    Kt [heads*Nk, d], Vt [heads*d, Nk] (V transposed), O [heads*Nq, d]: CUDA tensors."""
    L = K.load()
    q, k, v, o = _tensor(Q), _tensor(Kt), _tensor(Vt), _tensor(O)
    st = L.rg_attention(C.byref(d), C.byref(q), C.byref(k), C.byref(v), C.byref(o), _stream(Q))
    _check(st, "rg_attention")
    return O


def rg_reduce_cols_workspace_bytes(rows: int, cols: int) -> int:
    return int(K.load().rg_reduce_cols_workspace_bytes(rows, cols))


def rg_reduce_cols(d: K.rg_desc_t, op: int, x, out, *, y=None, ws=None):
    """Reduction along axis 0 with the descriptor's tree: out[c] = TREE_r x[r, c] (RG_COLOP_SUM) or
    TREE_r x[r, c] * y[r, c] (RG_COLOP_DOT).  `ws`: CUDA tensor of at least
    rg_reduce_cols_workspace_bytes(rows, cols) bytes when x has more than 256 rows."""
    L = K.load()
    xt, ot = _tensor(x), _tensor(out)
    yt = _tensor(y) if y is not None else None
    ws_ptr = ws.data_ptr() if ws is not None else None
    ws_bytes = ws.numel() * ws.element_size() if ws is not None else 0
    st = L.rg_reduce_cols(C.byref(d), int(op), C.byref(xt), C.byref(yt) if yt is not None else None, C.byref(ot),
                          ws_ptr, ws_bytes, _stream(x))
    _check(st, "rg_reduce_cols")
    return out


def rg_gemm_host(d: K.rg_desc_t, A, B, C_out, dev_scratch, *, bias=None, act: int = 0, residual=None):
    """Host-buffer form: A, B, C_out, bias, residual are CPU tensors (pinned for async copies);
    `dev_scratch` is a CUDA tensor.  Enqueues copies + kernels on the current stream."""
    L = K.load()
    a, b, c = _tensor(A), _tensor(B), _tensor(C_out)
    e = _epilogue(bias, act, residual)
    st = L.rg_gemm_host(C.byref(d), C.byref(a), C.byref(b), C.byref(c), C.byref(e) if e is not None else None,
                        dev_scratch.data_ptr(), dev_scratch.numel() * dev_scratch.element_size(), _stream(dev_scratch))
    _check(st, "rg_gemm_host")
    return C_out


def rg_gemm_host_scratch_bytes(d, M, N, Kdim, c_dtype, bias=None, act=0, residual=None) -> int:
    e = _epilogue(bias, act, residual)
    return int(K.load().rg_gemm_host_scratch_bytes(C.byref(d), M, N, Kdim, c_dtype, C.byref(e) if e is not None else None))


def rg_reduce_rows_host(d: K.rg_desc_t, op: int, x, out, dev_scratch, *, weight=None, eps: float = 0.0, aux_out=None):
    L = K.load()
    xt, ot = _tensor(x), _tensor(out)
    args = K.rg_reduce_args_t()
    if weight is not None:
        args.weight, args.weight_dtype = weight.data_ptr(), _dtype_code(weight)
    args.eps = float(eps)
    if aux_out is not None:
        args.aux_out = aux_out.data_ptr()
    st = L.rg_reduce_rows_host(C.byref(d), int(op), C.byref(xt), C.byref(ot), C.byref(args), dev_scratch.data_ptr(),
                               dev_scratch.numel() * dev_scratch.element_size(), _stream(dev_scratch))
    _check(st, "rg_reduce_rows_host")
    return out


def rg_reduce_rows_host_scratch_bytes(op, x, out) -> int:
    xt, ot = _tensor(x), _tensor(out)
    return int(K.load().rg_reduce_rows_host_scratch_bytes(int(op), C.byref(xt), C.byref(ot)))
