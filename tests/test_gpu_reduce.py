"""GPU parity: row reductions through the C ABI against the CPU oracle, bit for bit."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth

from _gpu_util import DEV, assert_bits_equal, gpu_reduce

pytestmark = pytest.mark.gpu

SHAPES = [(64, 4096), (1, 1), (3, 1), (5, 7), (9, 127), (4, 128), (7, 1000), (33, 4097), (5, 33000), (2, 65536),
          (300, 257), (2, 131072 + 5)]


def _draw(shape, dtype, seed, spread):
    if dtype == "f32":
        x = synth.normal_f32(shape, 1.0, seed)
        return synth.spread_exponents_f32(x, seed + 100) if spread else x
    x = synth.normal_bf16(shape, 1.0, seed)
    return synth.spread_exponents_bf16(x, seed + 100) if spread else x


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("spread", [False, True])
def test_row_sum_bit_exact(shape, dtype, spread):
    x = _draw(shape, dtype, 0, spread)
    got, _ = gpu_reduce(rg.RG_OP_SUM, x)
    want, _ = rgo.reduce_rows(rgo.OP_SUM, x)
    assert_bits_equal(got, want, f"row sum {shape} {dtype}")


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_softmax_normaliser_bit_exact(shape, dtype):
    x = _draw(shape, dtype, 1, False)
    if dtype == "f32":
        x = x * np.float32(100.0)
    got, gmax = gpu_reduce(rg.RG_OP_SOFTMAX_DENOM, x)
    want, wmax = rgo.reduce_rows(rgo.OP_SOFTMAX_DENOM, x)
    assert_bits_equal(got, want, f"softmax normaliser {shape} {dtype}")
    assert_bits_equal(gmax, wmax, "row max")


@pytest.mark.parametrize("shape", [(64, 4096), (1, 1), (5, 7), (7, 1000), (33, 4097), (3, 33000), (100, 256)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("fma", [0, 1])
def test_rmsnorm_bit_exact(shape, dtype, fma):
    x = _draw(shape, dtype, 2, False)
    w = synth.normal_bf16((shape[1],), 0.05, 10, mean=1.0) if dtype == "bf16" else synth.normal_f32((shape[1],), 0.05, 10, mean=1.0)
    got, grinv = gpu_reduce(rg.RG_OP_RMSNORM, x, weight=w, eps=1e-5, fma=fma)
    want, wrinv = rgo.reduce_rows(rgo.OP_RMSNORM, x, weight=w, eps=1e-5, fma=fma)
    assert_bits_equal(got, want, f"rmsnorm {shape} {dtype}")
    assert_bits_equal(grinv, wrinv, "1/rms")


@pytest.mark.parametrize("shape", [(300, 8192), (200, 20000), (150, 32764), (160, 12292), (149, 32768), (700, 8196), (150, 49152)])
@pytest.mark.parametrize("spread", [False, True])
def test_softmax_normaliser_long_rows_bit_exact(shape, spread):
    """fp32 rows of 8192 to 49152 columns, at least one row per SM: several steps of the two-pass kernel per
    row; row lengths off the 16-byte and the warp-block grid, and exponent-spread draws included."""
    x = synth.normal_f32(shape, 100.0, 31)
    if spread:
        x = synth.spread_exponents_f32(synth.normal_f32(shape, 1.0, 32), 33, -6, 6)
    got, gmax = gpu_reduce(rg.RG_OP_SOFTMAX_DENOM, x)
    want, wmax = rgo.reduce_rows(rgo.OP_SOFTMAX_DENOM, x)
    assert_bits_equal(got, want, f"long-row softmax normaliser {shape}")
    assert_bits_equal(gmax, wmax, "row max")
    # the generic kernel gives the same bits
    other, _ = gpu_reduce(rg.RG_OP_SOFTMAX_DENOM, x, BN=256)
    assert_bits_equal(other, got, "staged vs CTA-per-row kernel")
    assert rg.rg_device_status() == 0


@pytest.mark.parametrize("shape", [(500, 4096), (77, 8192), (40, 2048), (9, 520), (300, 3000), (50, 1536), (20, 6144), (2500, 512)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_rmsnorm_register_resident_rows_match_generic_kernels(shape, dtype):
    x = _draw(shape, dtype, 41, True)
    w = synth.normal_bf16((shape[1],), 0.05, 42, mean=1.0) if dtype == "bf16" else synth.normal_f32((shape[1],), 0.05, 42, mean=1.0)
    got, gr = gpu_reduce(rg.RG_OP_RMSNORM, x, weight=w, eps=1e-5)
    want, wr = rgo.reduce_rows(rgo.OP_RMSNORM, x, weight=w, eps=1e-5)
    assert_bits_equal(got, want, f"rmsnorm {shape} {dtype}")
    assert_bits_equal(gr, wr, "1/rms")
    for threads in (32, 128):
        other, _ = gpu_reduce(rg.RG_OP_RMSNORM, x, weight=w, eps=1e-5, BN=threads)
        assert_bits_equal(other, got, f"generic kernel, threads={threads}")


def test_rmsnorm_mixed_types_and_no_weight():
    x = synth.normal_bf16((17, 520), 1.0, 3)
    got, _ = gpu_reduce(rg.RG_OP_RMSNORM, x, eps=1e-6, out_dtype=torch.float32)
    want, _ = rgo.reduce_rows(rgo.OP_RMSNORM, x, eps=1e-6, out_dtype=rgo.F32)
    assert_bits_equal(got, want, "bf16 in, fp32 out, no weight")
    w32 = synth.normal_f32((520,), 0.05, 4, mean=1.0)
    got, _ = gpu_reduce(rg.RG_OP_RMSNORM, x, weight=w32, eps=1e-6)
    want, _ = rgo.reduce_rows(rgo.OP_RMSNORM, x, weight=w32, eps=1e-6)
    assert_bits_equal(got, want, "fp32 weight on bf16 rows")


def test_unaligned_views_take_the_scalar_path_with_the_same_bits():
    base = synth.normal_f32((9, 1003), 1.0, 5)
    xt = synth.to_torch(base, DEV)
    view = xt[:, 1:1000]                      # ld = 1003, first element 4 bytes off a 16-byte boundary
    got, _ = gpu_reduce(rg.RG_OP_SUM, view)
    want, _ = rgo.reduce_rows(rgo.OP_SUM, np.ascontiguousarray(base[:, 1:1000]))
    assert_bits_equal(got, want, "unaligned view")
    b16 = synth.normal_bf16((6, 1001), 1.0, 6)
    got, _ = gpu_reduce(rg.RG_OP_RMSNORM, synth.to_torch(b16, DEV)[:, 3:900], eps=1e-5)
    want, _ = rgo.reduce_rows(rgo.OP_RMSNORM, np.ascontiguousarray(b16[:, 3:900]), eps=1e-5)
    assert_bits_equal(got, want, "unaligned bf16 rmsnorm")


@pytest.mark.parametrize("op", [rg.RG_OP_SUM, rg.RG_OP_SOFTMAX_DENOM, rg.RG_OP_RMSNORM])
def test_layout_knobs_do_not_move_a_bit(op):
    """Sec. 5.2: with the tree pinned, threads per row and loads in flight are free speed knobs."""
    x = synth.spread_exponents_f32(synth.normal_f32((6, 20000), 1.0, 7), 8, -10, 10)
    ref, _ = gpu_reduce(op, x, eps=1e-5)
    for threads in (32, 64, 128, 256, 512, 1024):
        for unroll in (1, 2, 4, 8):
            got, _ = gpu_reduce(op, x, eps=1e-5, BN=threads, stages=unroll)
            assert_bits_equal(got, ref, f"threads={threads} unroll={unroll}")


def test_cancellation_rows_and_closed_forms():
    x = synth.add_cancellation_pairs(synth.normal_f32((8, 32768), 100.0, 13), 14, pairs=64)
    got, gmax = gpu_reduce(rg.RG_OP_SOFTMAX_DENOM, x)
    assert got[0] == np.float32(64) and got[2] == np.float32(64) and gmax[0] == np.float32(1e8)
    want, _ = rgo.reduce_rows(rgo.OP_SOFTMAX_DENOM, x)
    assert_bits_equal(got, want, "softmax with +-1e8 pairs")
    gs, _ = gpu_reduce(rg.RG_OP_SUM, x)
    ws, _ = rgo.reduce_rows(rgo.OP_SUM, x)
    assert_bits_equal(gs, ws, "sum with +-1e8 pairs")
    ones = np.ones((2, 4096), np.float32)
    assert np.all(gpu_reduce(rg.RG_OP_SUM, ones)[0] == np.float32(4096))
    assert np.all(gpu_reduce(rg.RG_OP_SOFTMAX_DENOM, np.full((2, 4096), 3.25, np.float32))[0] == np.float32(4096))
    # signed zeros: a row of -0.0 sums to -0.0 (padding is the additive identity, not +0)
    nz = np.full((1, 100), -0.0, np.float32)
    assert np.signbit(gpu_reduce(rg.RG_OP_SUM, nz)[0][0]) and np.signbit(rgo.reduce_rows(rgo.OP_SUM, nz)[0][0])


def test_runs_are_bitwise_repeatable():
    x = synth.normal_f32((128, 8192), 1.0, 9)
    a, _ = gpu_reduce(rg.RG_OP_SUM, x)
    for _ in range(5):
        assert_bits_equal(gpu_reduce(rg.RG_OP_SUM, x)[0], a, "repeat")


def test_full_size_reductions_sampled_rows():
    """65536 x 32768 fp32 ~ N(0,100) with +-1e8 pairs on even rows, in the launch configuration
    the benchmark times; the oracle recomputes sampled rows from the same bytes."""
    R, Cc = 65536, 32768
    x = synth.device_normal((R, Cc), 100.0, 13, torch.float32, DEV)
    synth.device_add_cancellation_pairs(x, 14, pairs=64)
    rows = np.unique(np.concatenate([np.arange(8), np.random.default_rng(0).integers(0, R, 120), [R - 2, R - 1]]))
    xs = x[torch.from_numpy(rows).to(DEV)].cpu().numpy()
    gs, _ = gpu_reduce(rg.RG_OP_SUM, x)
    ws, _ = rgo.reduce_rows(rgo.OP_SUM, xs)
    assert_bits_equal(gs[rows], ws, "full-size row sum, sampled rows")
    gz, gm = gpu_reduce(rg.RG_OP_SOFTMAX_DENOM, x)
    wz, wm = rgo.reduce_rows(rgo.OP_SOFTMAX_DENOM, xs)
    assert_bits_equal(gz[rows], wz, "full-size softmax normaliser, sampled rows")
    assert_bits_equal(gm[rows], wm, "full-size row max")
    even = rows[rows % 2 == 0]
    assert np.all(gz[even] == np.float32(64))
    assert not np.isnan(gs).any() and not np.isnan(gz).any()
    del x
    # RMSNorm 8192 x 4096 bf16: the whole output against the oracle
    xr = synth.normal_bf16((8192, 4096), 1.0, 9); w = synth.normal_bf16((4096,), 0.05, 10, mean=1.0)
    gy, _ = gpu_reduce(rg.RG_OP_RMSNORM, xr, weight=w, eps=1e-5)
    wy, _ = rgo.reduce_rows(rgo.OP_RMSNORM, xr, weight=w, eps=1e-5)
    assert_bits_equal(gy, wy, "RMSNorm 8192x4096")


def test_host_buffer_form_matches_device_form():
    x = synth.normal_f32((50, 3000), 1.0, 21)
    d = rg.rg_desc()
    xh = torch.from_numpy(x).pin_memory()
    oh = torch.empty(50, dtype=torch.float32).pin_memory()
    from paper_2609_11356_b200.api import rg_reduce_rows_host, rg_reduce_rows_host_scratch_bytes
    scratch = torch.empty(rg_reduce_rows_host_scratch_bytes(rg.RG_OP_SUM, xh, oh) + 256, dtype=torch.uint8, device=DEV)
    rg_reduce_rows_host(d, rg.RG_OP_SUM, xh, oh, scratch)
    torch.cuda.synchronize()
    want, _ = rgo.reduce_rows(rgo.OP_SUM, x)
    assert_bits_equal(oh.numpy(), want, "host-buffer row sum")


@pytest.mark.parametrize("op", [rg.RG_OP_SUM, rg.RG_OP_RMSNORM, rg.RG_OP_SOFTMAX_DENOM])
@pytest.mark.parametrize("with_weight,with_aux", [(False, False), (True, True), (False, True), (True, False)])
def test_host_buffer_form_stays_inside_its_scratch(op, with_weight, with_aux):
    """Scratch of exactly the size the library asks for, with canary bytes right behind it: every op and
    every combination of optional arguments stays inside, and the results equal the oracle's."""
    from paper_2609_11356_b200.api import rg_reduce_rows_host, rg_reduce_rows_host_scratch_bytes
    R, Cc = 37, 1001
    x = synth.normal_f32((R, Cc), 1.0, 40 + op)
    w = synth.normal_f32((Cc,), 0.05, 41, mean=1.0)
    xh = torch.from_numpy(x).pin_memory()
    oh = (torch.empty((R, Cc), dtype=torch.float32) if op == rg.RG_OP_RMSNORM else torch.empty(R, dtype=torch.float32)).pin_memory()
    auxh = torch.empty(R, dtype=torch.float32).pin_memory() if with_aux else None
    need = rg_reduce_rows_host_scratch_bytes(op, xh, oh)
    buf = torch.full((need + 4096,), 0xA5, dtype=torch.uint8, device=DEV)
    kw = dict(aux_out=auxh)
    if with_weight:
        kw["weight"] = torch.from_numpy(w).pin_memory()
    if with_weight and op != rg.RG_OP_RMSNORM:
        with pytest.raises(rg.RgError) as ei:                    # only RMSNorm reads a weight
            rg_reduce_rows_host(rg.rg_desc(), op, xh, oh, buf[:need], eps=1e-5, **kw)
        assert ei.value.status == 3
        torch.cuda.synchronize()
        assert bool((buf == 0xA5).all())                         # refused before any copy
        return
    rg_reduce_rows_host(rg.rg_desc(), op, xh, oh, buf[:need], eps=1e-5, **kw)
    torch.cuda.synchronize()
    assert bool((buf[need:] == 0xA5).all()), "the call wrote past the scratch it asked for"
    want, waux = rgo.reduce_rows({rg.RG_OP_SUM: rgo.OP_SUM, rg.RG_OP_RMSNORM: rgo.OP_RMSNORM, rg.RG_OP_SOFTMAX_DENOM: rgo.OP_SOFTMAX_DENOM}[op],
                                 x, weight=w if with_weight else None, eps=1e-5)
    assert_bits_equal(oh.numpy(), want, f"host-buffer reduction {op}")
    if with_aux and op != rg.RG_OP_SUM:
        assert_bits_equal(auxh.numpy(), waux, f"host-buffer reduction {op} aux")


@pytest.mark.parametrize("shape", [(1, 1), (3, 7), (33, 31), (40, 32), (64, 4096), (300, 1001), (70, 20000)])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_left_fold_bit_exact(shape, dtype):
    """RG_TREE_LEFT (Sec. 3.1: the chain, the other end of the work/depth range): all three operations, both
    input types, with and without the fused square; a different class of bits from the balanced tree."""
    if dtype == "f32":
        x = synth.add_cancellation_pairs(synth.normal_f32(shape, 100.0, 51 + shape[1]), 52, pairs=min(4, shape[1] // 2)) if shape[1] > 1 else synth.normal_f32(shape, 100.0, 51)
        w = synth.normal_f32((shape[1],), 0.05, 53, mean=1.0)
    else:
        x = synth.normal_bf16(shape, 1.0, 54 + shape[1]); w = synth.normal_bf16((shape[1],), 0.05, 55, mean=1.0)
    got, _ = gpu_reduce(rg.RG_OP_SUM, x, tree=rg.RG_TREE_LEFT)
    assert_bits_equal(got, rgo.reduce_rows(rgo.OP_SUM, x, tree=rgo.TREE_LEFT)[0], f"left row sum {shape} {dtype}")
    got, gmax = gpu_reduce(rg.RG_OP_SOFTMAX_DENOM, x, tree=rg.RG_TREE_LEFT)
    want, wmax = rgo.reduce_rows(rgo.OP_SOFTMAX_DENOM, x, tree=rgo.TREE_LEFT)
    assert_bits_equal(got, want, f"left softmax normaliser {shape} {dtype}")
    assert_bits_equal(gmax, wmax, "row maxima")
    for fma in (0, 1):
        got, grinv = gpu_reduce(rg.RG_OP_RMSNORM, x, weight=w, eps=1e-5, tree=rg.RG_TREE_LEFT, fma=fma)
        want, wrinv = rgo.reduce_rows(rgo.OP_RMSNORM, x, weight=w, eps=1e-5, tree=rgo.TREE_LEFT, fma=fma)
        assert_bits_equal(got, want, f"left rmsnorm {shape} {dtype} fma={fma}")
        assert_bits_equal(grinv, wrinv, "1/rms")
    assert rg.rg_desc_class(rg.rg_desc(tree=rg.RG_TREE_LEFT)) != rg.rg_desc_class(rg.rg_desc())
