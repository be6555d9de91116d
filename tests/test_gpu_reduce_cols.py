"""GPU parity for reductions along the other axis: the CUDA path against the oracle, bit for bit."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth
from tests._gpu_util import DEV, assert_bits_equal

pytestmark = pytest.mark.gpu


def gpu_cols(op, x, y=None, *, poison=True, **desc_kw):
    xt = x if torch.is_tensor(x) else synth.to_torch(x, DEV)
    yt = None if y is None else (y if torch.is_tensor(y) else synth.to_torch(y, DEV))
    R, Cc = xt.shape
    out = torch.full((Cc,), float("nan"), dtype=torch.float32, device=DEV)
    nb = rg.rg_reduce_cols_workspace_bytes(R, Cc)
    ws = None
    if nb:
        ws = torch.empty(nb, dtype=torch.uint8, device=DEV)
        if poison:
            ws.fill_(0xFF)
    rg.rg_reduce_cols(rg.rg_desc(**desc_kw), op, xt, out, y=yt, ws=ws)
    torch.cuda.synchronize()
    return out.cpu().numpy()


SHAPES = [(1, 1), (1, 300), (2, 5), (7, 129), (8, 128), (31, 4), (32, 64), (33, 257), (255, 100), (256, 128), (257, 131),
          (1000, 77), (4096, 512), (5000, 260), (65536 + 3, 36), (70000, 130)]


@pytest.mark.parametrize("R,C", SHAPES)
def test_col_sum_fp32_bit_exact(R, C):
    x = synth.normal_f32((R, C), 100.0, 3 + R + C)
    assert_bits_equal(gpu_cols(rg.RG_COLOP_SUM, x), rgo.reduce_cols(0, x), f"col sum {R}x{C}")


@pytest.mark.parametrize("R,C", [(1, 9), (33, 257), (300, 128), (5000, 260), (66000, 40)])
def test_col_sum_bf16_and_integers(R, C):
    x = synth.normal_bf16((R, C), 1.0, 5 + R)
    assert_bits_equal(gpu_cols(rg.RG_COLOP_SUM, x), rgo.reduce_cols(0, x), f"bf16 col sum {R}x{C}")
    xi = np.random.default_rng(R).integers(-100, 101, (R, C)).astype(np.float32)
    assert_bits_equal(gpu_cols(rg.RG_COLOP_SUM, xi), xi.astype(np.int64).sum(0).astype(np.float32), "integer col sum")


@pytest.mark.parametrize("R,C", [(2, 5), (33, 257), (257, 131), (4096, 512), (70000, 130)])
@pytest.mark.parametrize("fma", [0, 1])
def test_col_dot_bit_exact(R, C, fma):
    x = synth.normal_f32((R, C), 1.0, 11 + R); y = synth.normal_f32((R, C), 1.0, 12 + C)
    assert_bits_equal(gpu_cols(rg.RG_COLOP_DOT, x, y, fma=fma), rgo.reduce_cols(1, x, y, fma=fma), f"col dot {R}x{C} fma={fma}")
    xb = synth.normal_bf16((R, C), 1.0, 13 + R); yb = synth.normal_bf16((R, C), 1.0, 14 + C)
    assert_bits_equal(gpu_cols(rg.RG_COLOP_DOT, xb, yb, fma=fma), rgo.reduce_cols(1, xb, yb, fma=fma), f"bf16 col dot {R}x{C} fma={fma}")


def test_cancellation_probe_and_strided_unaligned_inputs():
    # +L / -L / r along the rows of single columns: the tree, not just a sum
    L, r = np.float32(1024.0), np.float32(2.0 ** -15)
    x = np.zeros((600, 6), np.float32)
    x[0, 0] = r; x[2, 0] = L; x[3, 0] = -L             # (2,3) pair first: r survives
    x[0, 1] = r; x[1, 1] = L; x[2, 1] = -L             # (0,1) pair first: r absorbed
    x[255, 2] = L; x[256, 2] = -L; x[599, 2] = r       # the pair straddles two blocks of 256 rows
    x[511, 3] = r; x[512, 3] = L; x[513, 3] = -L
    got = gpu_cols(rg.RG_COLOP_SUM, x)
    assert_bits_equal(got, rgo.reduce_cols(0, x), "probe columns")
    assert got[0] == r and got[1] == 0 and got[3] == r
    # a view with an odd leading dimension and an unaligned start: scalar loads, same bits
    base = synth.normal_f32((700, 203), 10.0, 9)
    bt = synth.to_torch(base, DEV)
    view = bt[3:, 1:198]
    assert_bits_equal(gpu_cols(rg.RG_COLOP_SUM, view), rgo.reduce_cols(0, base[3:, 1:198]), "strided unaligned view")
    bb = synth.to_torch(synth.normal_bf16((300, 77), 1.0, 4), DEV)
    assert_bits_equal(gpu_cols(rg.RG_COLOP_SUM, bb[:, 1:70]), rgo.reduce_cols(0, synth.from_torch(bb)[:, 1:70]), "bf16 unaligned view")


def test_full_size_sampled_columns_and_repeatable():
    R, C = 65536, 8192
    x = synth.device_normal((R, C), 100.0, 13, torch.float32, DEV)
    a = gpu_cols(rg.RG_COLOP_SUM, x); b = gpu_cols(rg.RG_COLOP_SUM, x, poison=False)
    assert_bits_equal(a, b, "repeatable")
    cols = np.random.default_rng(1).integers(0, C, 24)
    sub = x[:, torch.from_numpy(cols).to(DEV)].cpu().numpy()
    assert_bits_equal(a[cols], rgo.reduce_cols(0, sub), "sampled columns at full size")


def test_argument_errors():
    x = torch.zeros((300, 8), dtype=torch.float32, device=DEV); out = torch.zeros(8, dtype=torch.float32, device=DEV)
    with pytest.raises(rg.RgError):
        rg.rg_reduce_cols(rg.rg_desc(), rg.RG_COLOP_SUM, x, out)                     # workspace missing (300 rows)
    with pytest.raises(rg.RgError):
        rg.rg_reduce_cols(rg.rg_desc(), rg.RG_COLOP_DOT, x[:200], out)               # y missing
    with pytest.raises(rg.RgError):
        rg.rg_reduce_cols(rg.rg_desc(), rg.RG_COLOP_SUM, x[:200], torch.zeros(9, dtype=torch.float32, device=DEV))


@pytest.mark.parametrize("R,C", [(1, 9), (2, 5), (33, 257), (300, 131), (5000, 260), (70000, 40)])
@pytest.mark.parametrize("in16", [False, True])
def test_left_fold_bit_exact(R, C, in16):
    """RG_TREE_LEFT: the chain over the rows in index order (Sec. 3.1), no workspace."""
    x = synth.normal_bf16((R, C), 1.0, 5 + R) if in16 else synth.add_cancellation_pairs(synth.normal_f32((R, C), 100.0, 3 + R + C).T.copy(), 7, pairs=min(2, R // 2)).T.copy()
    y = synth.normal_bf16((R, C), 1.0, 6 + R) if in16 else synth.normal_f32((R, C), 1.0, 4 + R)
    xt, yt = synth.to_torch(x, DEV), synth.to_torch(y, DEV)
    out = torch.full((C,), float("nan"), dtype=torch.float32, device=DEV)
    rg.rg_reduce_cols(rg.rg_desc(tree=rg.RG_TREE_LEFT), rg.RG_COLOP_SUM, xt, out)           # no workspace at any row count
    torch.cuda.synchronize()
    assert_bits_equal(out.cpu().numpy(), rgo.reduce_cols(0, x, tree=rgo.TREE_LEFT), f"left col sum {R}x{C}")
    for fma in (0, 1):
        rg.rg_reduce_cols(rg.rg_desc(tree=rg.RG_TREE_LEFT, fma=fma), rg.RG_COLOP_DOT, xt, out, y=yt)
        torch.cuda.synchronize()
        assert_bits_equal(out.cpu().numpy(), rgo.reduce_cols(1, x, y, tree=rgo.TREE_LEFT, fma=fma), f"left col dot {R}x{C} fma={fma}")
    if R >= 33 and not in16:                                      # and it is a different sum from the balanced tree
        assert not np.array_equal(rgo.reduce_cols(0, x, tree=rgo.TREE_LEFT), rgo.reduce_cols(0, x))
