"""Host-side logic of the C boundary: the library loads without a GPU, exports every declared
symbol, validates descriptors and arguments before anything could launch, and hashes classes."""
import ctypes as C
import os
import re

import pytest

import paper_2609_11356_b200 as rg
from paper_2609_11356_b200 import _cabi as K

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    L = K.load()
    header = open(os.path.join(ROOT, "include", "rg.h")).read()
    declared = set(re.findall(r"\b(rg_[a-z_]+)\s*\(", header))
    assert declared == set(K.EXPORTS)
    for name in declared:
        assert hasattr(L, name), name


def test_struct_layout_matches_c():
    d = rg.rg_desc()
    assert d.size == C.sizeof(K.rg_desc_t)
    assert (d.in_dtype, d.acc_dtype, d.partial_dtype, d.merge_dtype) == (K.RG_BF16, K.RG_F32, K.RG_F32, K.RG_F32)
    assert d.tree == K.RG_TREE_BALANCED and d.n_cuts == 0 and d.BN == 0


def test_validate_rules():
    ok = rg.rg_desc(cuts=(256,))
    assert rg.rg_desc_validate(ok, 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(cuts=(256, 128)), 64, 256, 512) == 2      # not increasing
    assert rg.rg_desc_validate(rg.rg_desc(cuts=(512,)), 64, 256, 512) == 2          # cut at K
    assert rg.rg_desc_validate(rg.rg_desc(cuts=(0,)), 64, 256, 512) == 2
    assert rg.rg_desc_validate(rg.rg_desc(cuts=(40,)), 64, 256, 512) == 3           # splits a 16-wide step
    assert rg.rg_desc_validate(rg.rg_desc(atom=K.RG_ATOM_SCALAR), 64, 256, 512) == 0           # GEMV family
    assert rg.rg_desc_validate(rg.rg_desc(atom=K.RG_ATOM_SCALAR, cuts=(256,)), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(atom=K.RG_ATOM_SCALAR, tree=K.RG_TREE_LEFT), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(gemv_fold=1), 64, 256, 512) == 2                      # lane fields without the scalar atom
    assert rg.rg_desc_validate(rg.rg_desc(atom=K.RG_ATOM_SCALAR, gemv_layout=2), 64, 256, 512) == 2
    # 8-bit operands and the 32-wide step name each other; cuts fall on whole steps
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=K.RG_F8E4M3), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=K.RG_F8E4M3, atom=K.RG_ATOM_TC_BF16_K16), 64, 256, 512) == 2
    assert rg.rg_desc_validate(rg.rg_desc(atom=K.RG_ATOM_TC_F8_K32), 64, 256, 512) == 2
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=K.RG_F8E4M3, cuts=(48,)), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=K.RG_F8E4M3, cuts=(64,)), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=K.RG_F8E4M3, inner_span=48), 64, 256, 512) == 3     # not a whole number of 32-wide steps
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=K.RG_F8E4M3, inner_span=32), 64, 256, 512) == 0     # one step per accumulator
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=K.RG_F8E4M3, inner_span=128), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(inner_span=16), 64, 256, 512) == 0                            # the two-rounding plan
    assert rg.rg_desc_validate(rg.rg_desc(inner_span=8), 64, 256, 512) == 3                             # half a step
    assert rg.rg_desc_validate(rg.rg_desc(inner_span=16, BK=128), 64, 256, 512) == 3
    # speed knobs and promises that are not order fields
    assert rg.rg_desc_validate(rg.rg_desc(cuts=(256,), split_merge=2), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(split_merge=2), 64, 256, 512) == 3                            # nothing to merge
    assert rg.rg_desc_validate(rg.rg_desc(cuts=(256,), split_merge=3), 64, 256, 512) == 0                # the last-arriver merge
    assert rg.rg_desc_validate(rg.rg_desc(cuts=(256,), split_merge=3, cta_group=2), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(cuts=(256,), split_merge=4), 64, 256, 512) == 2
    # its tickets sit in front of the parts, 64 KiB for every shape
    assert rg.rg_gemm_workspace_bytes(rg.rg_desc(cuts=(256,), split_merge=3), 64, 256) == 2 * 64 * 256 * 4 + 65536
    assert rg.rg_gemm_workspace_bytes(rg.rg_desc(cuts=(256,), split_merge=3), 300, 4096) == 2 * 300 * 4096 * 4 + 65536
    assert rg.rg_desc_validate(rg.rg_desc(sm_share=2), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(sm_share=2, BN=256), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(b_static=1), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(b_static=2), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(b_static=3), 64, 256, 512) == 2
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=K.RG_F8E4M3, partial_dtype=K.RG_F8E4M3), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(in_dtype=4), 64, 256, 512) == 2
    assert rg.rg_desc_validate(rg.rg_desc(partial_dtype=K.RG_BF16), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(partial_dtype=K.RG_BF16, merge_dtype=K.RG_BF16), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(merge_dtype=K.RG_BF16), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(BN=100), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(BN=112, BK=256), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(BN=112, cta_group=2), 64, 256, 512) == 0     # a pair takes any width from 32 columns
    assert rg.rg_desc_validate(rg.rg_desc(BN=112, cta_group=2, inner_span=64), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(cta_group=2), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(cta_group=3), 64, 256, 512) == 2
    assert rg.rg_desc_validate(rg.rg_desc(cta_group=2, BN=64), 64, 256, 512) == 0
    assert rg.rg_desc_validate(rg.rg_desc(cta_group=2, BN=16), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(cta_group=1, BM=256), 64, 256, 512) == 3
    assert rg.rg_desc_validate(rg.rg_desc(tree=7), 64, 256, 512) == 2
    assert rg.rg_desc_validate(ok, 64, 256, 0) == 4
    bad = rg.rg_desc(); bad.size = 12
    assert rg.rg_desc_validate(bad, 1, 1, 16) == 2
    assert rg.rg_desc_validate(rg.rg_desc(cuts=tuple(16 * i for i in range(1, 64))), 4, 4, 2048) == 0


def test_class_key_holds_order_fields_only():
    base = rg.rg_desc(cuts=(1792, 3584))
    k = rg.rg_desc_class(base)
    assert k != 0
    # speed knobs do not move the class (Sec. 3.2.2)
    for kw in (dict(BN=64), dict(BN=256, BK=128), dict(stages=2), dict(raster=1), dict(BM=128), dict(BM=256), dict(cta_group=2),
               dict(split_merge=1), dict(split_merge=2), dict(split_merge=3), dict(sm_share=2), dict(b_static=1)):
        assert rg.rg_desc_class(rg.rg_desc(cuts=(1792, 3584), **kw)) == k
    # every order-deciding field does
    others = [rg.rg_desc(cuts=(1792,)), rg.rg_desc(cuts=(1792, 3600)), rg.rg_desc(),
              rg.rg_desc(cuts=(1792, 3584), tree=K.RG_TREE_LEFT), rg.rg_desc(cuts=(1792, 3584), fma=1),
              rg.rg_desc(cuts=(1792, 3584), partial_dtype=K.RG_BF16), rg.rg_desc(cuts=(1792, 3584), merge_dtype=K.RG_BF16),
              rg.rg_desc(cuts=(1792, 3584), atom=K.RG_ATOM_SCALAR), rg.rg_desc(cuts=(1792, 3584), k_tail=1),
              rg.rg_desc(cuts=(1792, 3584), inner_span=64), rg.rg_desc(cuts=(1792, 3584), atom=K.RG_ATOM_SCALAR, gemv_fold=1),
              rg.rg_desc(cuts=(1792, 3584), atom=K.RG_ATOM_SCALAR, gemv_layout=1), rg.rg_desc(cuts=(1792, 3584), in_dtype=K.RG_F16)]
    keys = [rg.rg_desc_class(o) for o in others]
    assert len(set(keys + [k])) == len(keys) + 1
    # stale entries beyond n_cuts are not part of the record
    d = rg.rg_desc(cuts=(1792, 3584)); d.cuts[5] = 999
    assert rg.rg_desc_class(d) == k
    assert rg.rg_desc_class(rg.rg_desc(cuts=(256, 128))) == 0


def test_workspace_bytes():
    assert rg.rg_gemm_workspace_bytes(rg.rg_desc(), 64, 256) == 0
    assert rg.rg_gemm_workspace_bytes(rg.rg_desc(cuts=(256,)), 64, 256) == 2 * 64 * 256 * 4
    assert rg.rg_gemm_workspace_bytes(rg.rg_desc(cuts=(16, 32, 48)), 3, 5) == 4 * 3 * 8 * 4
    assert rg.rg_gemm_workspace_bytes(rg.rg_desc(cuts=(16, 32, 48), partial_dtype=K.RG_BF16), 3, 5) == 4 * 3 * 8 * 2


def test_workspace_bytes_do_not_wrap():
    """Shapes at the dimension limit with many parts: the byte count is reported as unsatisfiable
    rather than wrapped around, so neither rg_gemm nor rg_gemm_noalloc can accept a short buffer."""
    L = K.load()
    big = (1 << 31) - 1024
    d = rg.rg_desc(cuts=tuple(16 * i for i in range(1, 64)))
    exact = 64 * big * big * 4                                   # = 2^70: does not fit 64 bits
    assert exact >= 1 << 64
    assert rg.rg_gemm_workspace_bytes(d, big, big) == (1 << 64) - 1
    assert rg.rg_gemm_workspace_bytes(rg.rg_desc(cuts=(16,)), big, 4096) == 2 * big * 4096 * 4   # large but representable
    A = _t(0x1000, K.RG_BF16, big, 2048); B = _t(0x2000, K.RG_BF16, big, 2048); Cm = _t(0x3000, K.RG_BF16, big, big)
    assert L.rg_gemm(C.byref(d), C.byref(A), C.byref(B), C.byref(Cm), None, 0x4000, 1 << 40, None) == 6
    assert L.rg_gemm_noalloc(C.byref(d), C.byref(A), C.byref(B), C.byref(Cm), None, None) == 6


def _align256(n):
    return (n + 255) // 256 * 256


@pytest.mark.parametrize("op", [K.RG_OP_SUM, K.RG_OP_RMSNORM, K.RG_OP_SOFTMAX_DENOM])
@pytest.mark.parametrize("xdt,odt", [(K.RG_F32, K.RG_F32), (K.RG_BF16, K.RG_BF16), (K.RG_BF16, K.RG_F32)])
def test_reduce_host_scratch_size_covers_every_slot(op, xdt, odt):
    """The scratch a host-buffer reduction asks for holds the row copy, the result, the RMSNorm weight and
    the auxiliary output, each on a 256-byte boundary, for every op; a weight handed to an op that does not
    read one is refused before any copy."""
    L = K.load()
    R, Cc = 37, 1001
    es = {K.RG_F32: 4, K.RG_BF16: 2}
    if op != K.RG_OP_RMSNORM:
        odt = K.RG_F32
    x = _t(0x10000, xdt, R, Cc); o = _t(0x20000, odt, R, Cc if op == K.RG_OP_RMSNORM else 1)
    ldx = (Cc + 7) // 8 * 8
    want = _align256(R * ldx * es[xdt])
    want += _align256(R * ldx * es[odt]) if op == K.RG_OP_RMSNORM else _align256(R * 4)
    want += _align256(Cc * 4) if op == K.RG_OP_RMSNORM else 0
    want += _align256(R * 4)
    need = L.rg_reduce_rows_host_scratch_bytes(op, C.byref(x), C.byref(o))
    assert need == want
    d = rg.rg_desc()
    args = K.rg_reduce_args_t(); args.weight = 0x30000; args.weight_dtype = K.RG_F32; args.aux_out = 0x40000
    short = L.rg_reduce_rows_host(C.byref(d), op, C.byref(x), C.byref(o), C.byref(args), 0x100000, need - 1, None)
    if op == K.RG_OP_RMSNORM:
        assert short == 6                                        # one byte short: refused
    else:
        assert short == 3                                        # a weight with SUM / SOFTMAX_DENOM
        args.weight = None
        assert L.rg_reduce_rows_host(C.byref(d), op, C.byref(x), C.byref(o), C.byref(args), 0x100000, need - 1, None) == 6


def test_selftest_arguments():
    L = K.load()
    assert L.rg_selftest_bounded_wait(1_000_000, None, None) == 1
    assert L.rg_selftest_bounded_wait(10, 0x1000, None) == 4              # below 1 us
    assert L.rg_selftest_bounded_wait(10**9, 0x1000, None) == 4           # above 100 ms: never a long stall
    assert L.rg_selftest_exp(8, 0x1000, 0x2000, 4, None) == 4             # no such form
    assert L.rg_selftest_exp(7, 0x1000, 0x2000, 33, None) == 4            # SiLU segments are 32 wide
    assert L.rg_selftest_exp(-1, 0x1000, 0x2000, 4, None) == 4
    assert L.rg_selftest_exp(0, 0x1000, 0x2000, -1, None) == 4
    assert L.rg_selftest_exp(0, None, 0x2000, 4, None) == 1
    assert L.rg_selftest_exp(3, None, None, 0, None) == 0                 # nothing to do, nothing launched


def _t(ptr, dtype, rows, cols, ld=None):
    return K.rg_tensor_t(ptr, dtype, rows, cols, cols if ld is None else ld)


def test_argument_errors_are_reported_before_any_launch():
    L = K.load()
    d = rg.rg_desc()
    A = _t(0x1000, K.RG_BF16, 4, 64); B = _t(0x2000, K.RG_BF16, 8, 64); Cm = _t(0x3000, K.RG_BF16, 4, 8)
    call = lambda d_, a, b, c, e=None, ws=None, wsb=0: L.rg_gemm(
        C.byref(d_) if d_ is not None else None, C.byref(a) if a is not None else None,
        C.byref(b) if b is not None else None, C.byref(c) if c is not None else None, e, ws, wsb, None)
    assert call(None, A, B, Cm) == 1
    assert call(d, None, B, Cm) == 1
    assert call(d, _t(None, K.RG_BF16, 4, 64), B, Cm) == 1
    assert call(d, A, _t(0x2000, K.RG_BF16, 8, 32), Cm) == 4                       # K disagrees
    assert call(d, A, B, _t(0x3000, K.RG_BF16, 4, 9)) == 4
    assert call(d, _t(0x1000, K.RG_F32, 4, 64), B, Cm) == 3                        # fp32 operands
    assert call(d, _t(0x1000, K.RG_F16, 4, 64), _t(0x2000, K.RG_F16, 8, 64), Cm) == 4   # fp16 operands, bf16 descriptor
    assert call(d, _t(0x1000, K.RG_F16, 4, 64), B, Cm) == 3                        # mixed operand types
    assert call(d, _t(0x1008, K.RG_BF16, 4, 64), B, Cm) == 5                       # 16-byte rule
    assert call(d, _t(0x1000, K.RG_BF16, 4, 60, 60), _t(0x2000, K.RG_BF16, 8, 60, 60), Cm) == 5   # ld % 8
    assert call(d, _t(0x1000, K.RG_BF16, 4, 0), _t(0x2000, K.RG_BF16, 8, 0), Cm) == 4            # K = 0
    d8 = rg.rg_desc(in_dtype=K.RG_F8E4M3)
    assert call(d8, _t(0x1000, K.RG_F8E4M3, 4, 63, 64), _t(0x2000, K.RG_F8E4M3, 8, 63, 64), Cm) == 4   # odd K: rows are whole byte pairs
    assert call(d8, _t(0x1000, K.RG_F8E4M3, 4, 64, 72), _t(0x2000, K.RG_F8E4M3, 8, 64, 72), Cm) == 5   # ld % 16
    assert call(d8, A, B, Cm) == 4                                                  # bf16 operands, e4m3 descriptor
    assert call(d8, _t(0x1000, K.RG_F8E4M3, 4, 64), _t(0x2000, K.RG_F8E4M3, 8, 64), _t(0x3000, K.RG_F8E4M3, 4, 8)) == 4   # e4m3 is an operand type only
    ds = rg.rg_desc(cuts=(32,))
    assert call(ds, A, B, Cm) == 6                                                  # workspace missing
    assert call(ds, A, B, Cm, None, 0x4000, 16) == 6                                # too small
    e = K.rg_epilogue_t(); e.act = 5
    assert call(d, A, B, Cm, C.byref(e)) == 3
    # empty problems are a no-op
    assert call(d, _t(None, K.RG_BF16, 0, 64), B, _t(None, K.RG_BF16, 0, 8)) == 0
    x = _t(0x1000, K.RG_F32, 4, 64); o = _t(0x2000, K.RG_F32, 4, 1)
    red = lambda d_, op, x_, o_: L.rg_reduce_rows(C.byref(d_), op, C.byref(x_), C.byref(o_), None, None)
    assert red(rg.rg_desc(tree=K.RG_TREE_LEFT), K.RG_OP_SUM, x, _t(0x2000, K.RG_F32, 5, 1)) == 4      # the left fold takes the same checks
    assert red(d, K.RG_OP_SUM, _t(0x1000, K.RG_F32, 4, 0), o) == 4
    assert red(d, K.RG_OP_SUM, x, _t(0x2000, K.RG_F32, 5, 1)) == 4
    assert red(d, K.RG_OP_RMSNORM, x, o) == 4
    assert red(d, 9, x, o) == 3
    assert red(d, K.RG_OP_SUM, _t(None, K.RG_F32, 0, 64), _t(None, K.RG_F32, 0, 1)) == 0
    col = lambda d_, op, x_, y_, o_, ws=None, wsb=0: L.rg_reduce_cols(C.byref(d_), op, C.byref(x_), C.byref(y_) if y_ is not None else None,
                                                                   C.byref(o_), ws, wsb, None)
    xc = _t(0x1000, K.RG_F32, 300, 64); oc = _t(0x2000, K.RG_F32, 64, 1)
    assert col(d, K.RG_COLOP_SUM, xc, None, oc) == 6                                # more than 256 rows need the workspace
    assert col(d, K.RG_COLOP_SUM, xc, None, oc, 0x4008, 1 << 20) == 5
    assert col(d, K.RG_COLOP_DOT, xc, None, oc, 0x4000, 1 << 20) == 1               # y missing
    assert col(d, K.RG_COLOP_DOT, xc, _t(0x5000, K.RG_BF16, 300, 64), oc, 0x4000, 1 << 20) == 4
    assert col(d, K.RG_COLOP_SUM, xc, None, _t(0x2000, K.RG_F32, 63, 1), 0x4000, 1 << 20) == 4
    assert col(d, K.RG_COLOP_SUM, _t(0x1000, K.RG_F32, 0, 64), None, oc) == 4       # no rows: nothing to fold
    assert col(d, K.RG_COLOP_SUM, _t(None, K.RG_F32, 5, 0), None, _t(None, K.RG_F32, 0, 1)) == 0
    assert col(rg.rg_desc(tree=K.RG_TREE_LEFT), K.RG_COLOP_SUM, xc, None, _t(0x2000, K.RG_F32, 63, 1)) == 4   # shape errors come first
    assert col(d, 7, xc, None, oc, 0x4000, 1 << 20) == 3
    assert L.rg_reduce_cols_workspace_bytes(256, 1000) == 0 and L.rg_reduce_cols_workspace_bytes(257, 1000) == 2 * 1000 * 4
    assert L.rg_reduce_cols_workspace_bytes(65537, 10) == (257 + 2) * 10 * 4


def test_status_strings():
    for s in range(9):
        assert len(rg.rg_status_string(s)) > 1
    with pytest.raises(rg.RgError):
        raise rg.RgError(3, "x")
