"""Helpers for the GPU parity tests: run the CUDA path through the C ABI on numpy inputs."""
import numpy as np
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth

DEV = "cuda"
HW = rgo.TCGEN05_BF16_B200   # the atom model the probes selected for this GPU
HW8 = rgo.TCGEN05_F8E4M3_B200   # and for the 32-wide e4m3 step


def gpu_gemm(A, B, *, out_dtype=rgo.BF16, bias=None, act=0, residual=None, poison=True, **desc_kw):
    """A, B: numpy uint16 (bf16 bits) or CUDA tensors.  Returns numpy (uint16 bits or float32)."""
    At = A if torch.is_tensor(A) else synth.to_torch(A, DEV)
    Bt = B if torch.is_tensor(B) else synth.to_torch(B, DEV)
    if At.dtype == torch.uint8:                                   # numpy uint8 = e4m3 bit patterns
        def rows16(t):                                            # rows start on 16-byte boundaries
            Kp = (t.shape[1] + 15) // 16 * 16
            buf = torch.full((t.shape[0], Kp), 0x7f, dtype=torch.uint8, device=DEV)   # padding is NaN: must never be read as data
            buf[:, :t.shape[1]] = t
            return buf.view(torch.float8_e4m3fn)[:, :t.shape[1]]
        At, Bt = rows16(At), rows16(Bt)
    M, N = At.shape[0], Bt.shape[0]
    if At.dtype == torch.float16:
        desc_kw.setdefault("in_dtype", rg.RG_F16)
    if At.dtype == torch.float8_e4m3fn:
        desc_kw.setdefault("in_dtype", rg.RG_F8E4M3)
    d = rg.rg_desc(**desc_kw)
    tdt = {rgo.BF16: torch.bfloat16, rgo.F32: torch.float32, rgo.F16: torch.float16}[out_dtype]
    Ct = torch.empty((M, N), dtype=tdt, device=DEV)
    if poison and Ct.numel():
        Ct.view(torch.int32 if out_dtype == rgo.F32 else torch.int16).fill_(-1)   # NaN pattern: unwritten elements show
    nb = rg.rg_gemm_workspace_bytes(d, M, N)
    ws = None
    if nb:
        ws = torch.empty(nb, dtype=torch.uint8, device=DEV)
        ws.fill_(0xFF)
        if d.split_merge == 3:
            # the tickets in front of the parts start at zero (the caller's promise); the parts stay poisoned
            d1 = rg.rg_desc(**{**desc_kw, "split_merge": 1})
            ws[:nb - rg.rg_gemm_workspace_bytes(d1, M, N)].zero_()
    bt = None if bias is None else (bias if torch.is_tensor(bias) else synth.to_torch(bias, DEV))
    rt = None if residual is None else (residual if torch.is_tensor(residual) else synth.to_torch(residual, DEV))
    rg.rg_gemm(d, At, Bt, Ct, bias=bt, act=act, residual=rt, ws=ws)
    torch.cuda.synchronize()
    return synth.from_torch(Ct)


def gpu_reduce(op, x, *, weight=None, eps=0.0, out_dtype=None, **desc_kw):
    xt = x if torch.is_tensor(x) else synth.to_torch(x, DEV)
    R, Cc = xt.shape
    d = rg.rg_desc(**desc_kw)
    aux = torch.full((R,), float("nan"), dtype=torch.float32, device=DEV)
    if op == rg.RG_OP_RMSNORM:
        out = torch.empty((R, Cc), dtype=xt.dtype if out_dtype is None else out_dtype, device=DEV)
    else:
        out = torch.full((R,), float("nan"), dtype=torch.float32, device=DEV)
    wt = None if weight is None else (weight if torch.is_tensor(weight) else synth.to_torch(weight, DEV))
    rg.rg_reduce_rows(d, op, xt, out, weight=wt, eps=eps, aux_out=aux)
    torch.cuda.synchronize()
    return synth.from_torch(out), aux.cpu().numpy()


def bits(a: np.ndarray) -> np.ndarray:
    return a.view(np.uint32) if a.dtype == np.float32 else a.view(np.uint16)   # uint16 and float16 alike


def assert_bits_equal(got, want, what=""):
    got, want = np.ascontiguousarray(got), np.ascontiguousarray(want)
    g, w = bits(got), bits(want)
    differ = g != w
    if differ.any() and got.dtype != np.uint16:
        differ &= ~(np.isnan(got) & np.isnan(want))          # NaN results compare as "both NaN"
    elif differ.any():
        differ &= ~(((g & 0x7fff) > 0x7f80) & ((w & 0x7fff) > 0x7f80))
    if differ.any():
        bad = np.argwhere(differ)
        raise AssertionError(f"{what}: {len(bad)} of {g.size} elements differ; first at {bad[0].tolist()}: "
                             f"got {got[tuple(bad[0])]!r} want {want[tuple(bad[0])]!r}")
