"""Split-K in one launch (App. E: "a single launch across the split-K slices"; Sec. 3.2.2 "Split-K"): the
parts of an output tile are walked by the CTAs of one thread-block cluster and merged over distributed
shared memory inside the GEMM kernel.  Where the parts are added is a speed knob (`split_merge`), so the
in-cluster path must return the oracle's bits and the bits of the two-kernel path through the workspace,
for every tree, part type, epilogue and tile width."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import synth
from tests._gpu_util import DEV, HW, HW8, assert_bits_equal, gpu_gemm

pytestmark = pytest.mark.gpu

IN_CLUSTER, TWO_KERNELS, LAST_ARRIVER = 2, 1, 3


def _inputs(M, N, K, seed, spread=True):
    A = synth.normal_bf16((M, K), 1.0, seed); B = synth.normal_bf16((N, K), 0.02, seed + 1)
    if spread:
        A = synth.spread_exponents_bf16(A, seed + 2, -8, 8)
    return A, B


def _even_cuts(K, parts, step=16):
    return tuple(sorted({max(step, (K * t // parts) // step * step) for t in range(1, parts)}))


@pytest.mark.parametrize("M", [1, 8, 32, 64, 65, 128])
@pytest.mark.parametrize("parts", [2, 3, 5, 8])
def test_in_cluster_merge_matches_oracle_and_two_kernel_path(M, parts):
    N, K = 520, 2304
    A, B = _inputs(M, N, K, 10 * M + parts)
    cuts = _even_cuts(K, parts)
    res = synth.normal_bf16((M, N), 1.0, 99)
    for tree in (rg.RG_TREE_LEFT, rg.RG_TREE_BALANCED):
        want = rgo.gemm(A, B, cuts=cuts, tree=tree, atom_model=HW, residual=res, out_dtype=rgo.BF16)
        got = gpu_gemm(A, B, cuts=cuts, tree=tree, residual=res, split_merge=IN_CLUSTER)
        assert_bits_equal(got, want, f"in-cluster M={M} parts={parts} tree={tree} vs oracle")
        assert_bits_equal(gpu_gemm(A, B, cuts=cuts, tree=tree, residual=res, split_merge=TWO_KERNELS), want,
                          f"two kernels M={M} parts={parts} tree={tree} vs oracle")
        assert_bits_equal(gpu_gemm(A, B, cuts=cuts, tree=tree, residual=res), want, f"default path M={M} parts={parts}")
        assert_bits_equal(gpu_gemm(A, B, cuts=cuts, tree=tree, residual=res, b_static=1), want, f"static weights M={M} parts={parts}")
        assert_bits_equal(gpu_gemm(A, B, cuts=cuts, tree=tree, residual=res, b_static=2), want, f"static operands M={M} parts={parts}")
        assert_bits_equal(gpu_gemm(A, B, cuts=cuts, tree=tree, residual=res, split_merge=LAST_ARRIVER), want, f"last-arriver merge M={M} parts={parts}")


@pytest.mark.parametrize("M,N,K,cuts", [(32, 4096, 14336, tuple(1792 * t for t in range(1, 8))),
                                        (8, 4096, 14336, tuple(1792 * t for t in range(1, 8))),
                                        (1, 4096, 14336, tuple(1792 * t for t in range(1, 8)))])
def test_decode_shape_every_element_for_small_m_sampled_for_32(M, N, K, cuts):
    A, B = _inputs(M, N, K, 4, spread=False)
    res = synth.normal_bf16((M, N), 1.0, 5)
    got = gpu_gemm(A, B, cuts=cuts, residual=res, split_merge=IN_CLUSTER)
    two = gpu_gemm(A, B, cuts=cuts, residual=res, split_merge=TWO_KERNELS)
    assert_bits_equal(got, two, f"decode M={M}: in-cluster vs two kernels")
    if M <= 8:
        want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, residual=res, out_dtype=rgo.BF16)
        assert_bits_equal(got, want, f"decode M={M} vs oracle")
    else:
        g = np.random.default_rng(0)
        si, sj = g.integers(0, M, 2048), g.integers(0, N, 2048)
        want = rgo.gemm_samples(A, B, si, sj, cuts=cuts, atom_model=HW, residual=res, out_dtype=rgo.BF16)
        assert_bits_equal(synth.bf16_bits_to_f32(got[si, sj]), want, f"decode M={M} sampled vs oracle")


@pytest.mark.parametrize("knobs", [dict(BN=32), dict(BN=48), dict(BN=64, BK=64), dict(BN=112), dict(BN=128, BK=64), dict(BN=128, stages=2),
                                   dict(BN=208, BK=64), dict(BN=256, BK=64), dict(BN=256, BK=128), dict(raster=1)])
def test_tile_widths_and_ragged_edges(knobs):
    """Tile widths that are not multiples of 32, N not a multiple of the tile or of 4, K with a short last
    step: the same bits from every width."""
    M, N, K = 37, 1003, 1000
    A, B = _inputs(M, N, K, 7)
    cuts = (256, 512, 768)
    bias = synth.uniform_bf16((N,), -0.1, 0.1, 8)
    want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, bias=bias, act=1, out_dtype=rgo.F32)
    assert_bits_equal(gpu_gemm(A, B, cuts=cuts, bias=bias, act=1, out_dtype=rgo.F32, split_merge=IN_CLUSTER, **knobs), want, f"{knobs}")


def test_part_and_merge_types_outputs_and_epilogues():
    M, N, K = 70, 200, 1024
    A, B = _inputs(M, N, K, 5)
    cuts = (256, 512, 768)
    bias = synth.uniform_bf16((N,), -0.1, 0.1, 2); res = synth.normal_bf16((M, N), 1.0, 3)
    for pd, md in ((rgo.F32, rgo.F32), (rgo.BF16, rgo.F32), (rgo.BF16, rgo.BF16), (rgo.F16, rgo.F32), (rgo.F16, rgo.F16)):
        for tree in (rg.RG_TREE_LEFT, rg.RG_TREE_BALANCED):
            for out in (rgo.BF16, rgo.F16, rgo.F32):
                got = gpu_gemm(A, B, cuts=cuts, tree=tree, partial_dtype=pd, merge_dtype=md, bias=bias, act=1, residual=res, out_dtype=out,
                               split_merge=IN_CLUSTER)
                want = rgo.gemm(A, B, cuts=cuts, tree=tree, atom_model=HW, partial_dtype=pd, merge_dtype=md, bias=bias, act=1,
                                residual=res, out_dtype=out)
                assert_bits_equal(got, want, f"in-cluster partial={pd} merge={md} tree={tree} out={out}")


def test_other_operand_types_and_more_than_one_tile_row():
    # fp16 operands
    g = np.random.default_rng(3)
    A16 = (g.standard_normal((40, 768)) * np.exp2(g.integers(-4, 5, (40, 768)))).astype(np.float16)
    B16 = g.standard_normal((130, 768)).astype(np.float16)
    assert_bits_equal(gpu_gemm(A16, B16, cuts=(256, 512), out_dtype=rgo.F32, split_merge=IN_CLUSTER),
                      rgo.gemm(A16, B16, cuts=(256, 512), atom_model=HW, out_dtype=rgo.F32), "fp16 in-cluster")
    # e4m3 operands (32-wide step)
    A8 = synth.f32_to_f8e4m3_bits(np.clip(g.standard_normal((33, 1024)) * np.exp2(g.integers(-5, 6, (33, 1024))), -448, 448).astype(np.float32))
    B8 = synth.f32_to_f8e4m3_bits(g.standard_normal((96, 1024)).astype(np.float32))
    assert_bits_equal(gpu_gemm(A8, B8, cuts=(256, 512, 768), out_dtype=rgo.F32, split_merge=IN_CLUSTER),
                      rgo.gemm(A8, B8, cuts=(256, 512, 768), atom_model=HW8, out_dtype=rgo.F32), "e4m3 in-cluster")
    # several tile rows and columns: asked for explicitly (the default keeps it to one tile row)
    A, B = _inputs(300, 520, 2048, 11)
    cuts = (512, 1024, 1536)
    want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, out_dtype=rgo.F32)
    assert_bits_equal(gpu_gemm(A, B, cuts=cuts, out_dtype=rgo.F32, split_merge=IN_CLUSTER), want, "300 rows in-cluster")
    assert_bits_equal(gpu_gemm(A, B, cuts=cuts, out_dtype=rgo.F32, split_merge=IN_CLUSTER, raster=1, BN=64), want, "300 rows in-cluster, row-major walk")


def test_needs_no_workspace_and_refuses_what_it_cannot_do():
    A, B = _inputs(16, 256, 1024, 21)
    At, Bt = synth.to_torch(A, DEV), synth.to_torch(B, DEV)
    out = torch.empty((16, 256), dtype=torch.float32, device=DEV)
    d = rg.rg_desc(cuts=(256, 512), split_merge=IN_CLUSTER)
    rg.rg_gemm(d, At, Bt, out)                                   # no workspace passed
    torch.cuda.synchronize()
    assert_bits_equal(out.cpu().numpy(), rgo.gemm(A, B, cuts=(256, 512), atom_model=HW, out_dtype=rgo.F32), "no workspace")
    assert rg.rg_desc_class(d) == rg.rg_desc_class(rg.rg_desc(cuts=(256, 512)))       # where the parts are added is not part of the class
    for bad in (dict(cuts=tuple(64 * t for t in range(1, 10))), dict(cuts=(256,), inner_span=64), dict(cuts=(256,), cta_group=2), dict()):
        with pytest.raises(rg.RgError) as ei:
            rg.rg_gemm(rg.rg_desc(split_merge=IN_CLUSTER, **bad), At, Bt, out)
        assert ei.value.status == 3
    with pytest.raises(rg.RgError):                              # the two-kernel path still wants its workspace
        rg.rg_gemm(rg.rg_desc(cuts=(256, 512), split_merge=TWO_KERNELS), At, Bt, out)
    assert rg.rg_device_status() == 0


def test_rows_keep_their_bits_across_m_and_paths():
    """Batch invariance through the in-cluster path: row i of C is the same for every M, and equals the row the
    two-kernel path and a larger problem (several tile rows, default path) give."""
    N, K = 512, 3584
    cuts = tuple(448 * t for t in range(1, 8))
    A, B = _inputs(200, N, K, 31)
    ref = gpu_gemm(A, B, cuts=cuts, out_dtype=rgo.F32)                       # 200 rows, the default path (two kernels)
    for M in (1, 2, 7, 16, 64, 100, 128):
        assert_bits_equal(gpu_gemm(A[:M], B, cuts=cuts, out_dtype=rgo.F32), ref[:M], f"M={M} default")
        assert_bits_equal(gpu_gemm(A[:M], B, cuts=cuts, out_dtype=rgo.F32, split_merge=IN_CLUSTER), ref[:M], f"M={M} in-cluster")


@pytest.mark.parametrize("M,N,K,cuts", [(32, 520, 2304, (768, 1536)), (8, 1003, 1000, (256, 512, 768)), (64, 300, 4096, tuple(512 * t for t in range(1, 8))),
                                        (200, 260, 1024, (512,)), (16, 512, 1024, ())])
def test_two_ctas_per_sm_form_is_the_same_class(M, N, K, cuts):
    """The one-CTA kernel with four epilogue warps and half an SM's shared and tensor memory (`sm_share = 2`):
    a schedule, not an order; same bits as the oracle and as the one-CTA-per-SM form, for every tile width it takes."""
    A, B = _inputs(M, N, K, 41 + M)
    bias = synth.uniform_bf16((N,), -0.1, 0.1, 8); res = synth.normal_bf16((M, N), 1.0, 9)
    want = rgo.gemm(A, B, cuts=cuts, atom_model=HW, bias=bias, act=1, residual=res, out_dtype=rgo.BF16)
    wide_stage = (dict(BN=128, BK=128, stages=2),) if M <= 64 else ()     # 128 rows of A and 128-wide stages: no two fit half an SM
    for knobs in (dict(), dict(BN=32), dict(BN=48, BK=64), dict(BN=112), dict(BN=128, BK=64)) + wide_stage:
        got = gpu_gemm(A, B, cuts=cuts, bias=bias, act=1, residual=res, sm_share=2, split_merge=TWO_KERNELS if cuts else 0, **knobs)
        assert_bits_equal(got, want, f"two CTAs per SM {M}x{N}x{K} {knobs}")
    assert_bits_equal(gpu_gemm(A, B, cuts=cuts, bias=bias, act=1, residual=res, sm_share=1, split_merge=TWO_KERNELS if cuts else 0), want, "one CTA per SM")
    for bad in (dict(BN=256), dict(cta_group=2), dict(BK=256)):
        with pytest.raises(rg.RgError):
            gpu_gemm(A, B, cuts=cuts, sm_share=2, **bad)


def test_last_arriver_merge_reuses_its_workspace_and_leaves_the_tickets_zero():
    """split_merge = 3: the parts go through the workspace and the CTA that stores a tile's last part merges it.  The
    tickets in front of the parts are zero before the first call (the caller's promise) and zero again after every
    call, so the same workspace serves call after call, for shapes and tilings that change from call to call."""
    cuts8 = tuple(1792 * t for t in range(1, 8))
    A, B = _inputs(32, 4096, 14336, 4, spread=False)
    res = synth.normal_bf16((32, 4096), 1.0, 5)
    d = rg.rg_desc(cuts=cuts8, split_merge=LAST_ARRIVER, b_static=1)
    nb = rg.rg_gemm_workspace_bytes(d, 32, 4096)
    tickets = nb - rg.rg_gemm_workspace_bytes(rg.rg_desc(cuts=cuts8), 32, 4096)
    assert tickets == 65536                                          # the same place for every shape
    ws = torch.zeros(nb, dtype=torch.uint8, device=DEV)              # zero-filled once
    At, Bt, Rt = synth.to_torch(A, DEV), synth.to_torch(B, DEV), synth.to_torch(res, DEV)
    two = gpu_gemm(A, B, cuts=cuts8, residual=res, split_merge=TWO_KERNELS)
    for call in range(4):
        out = torch.empty((32, 4096), dtype=torch.bfloat16, device=DEV); out.view(torch.int16).fill_(-1)
        rg.rg_gemm(d, At, Bt, out, residual=Rt, ws=ws)
        torch.cuda.synchronize()
        assert_bits_equal(synth.from_torch(out), two, f"decode shape, call {call}")
        assert int(ws[:tickets].max().item()) == 0, "tickets not back at zero"
    # the same problem on narrow tiles: 512 work items, more than one round, so nobody may wait for anybody and the
    # CTA that stores a tile's last part merges it alone (the default width above is one round: the tile's CTAs share it)
    d64 = rg.rg_desc(cuts=cuts8, split_merge=LAST_ARRIVER, BN=64)
    for call in range(2):
        out = torch.empty((32, 4096), dtype=torch.bfloat16, device=DEV); out.view(torch.int16).fill_(-1)
        rg.rg_gemm(d64, At, Bt, out, residual=Rt, ws=ws)
        torch.cuda.synchronize()
        assert_bits_equal(synth.from_torch(out), two, f"decode shape on 64-wide tiles, call {call}")
        assert int(ws[:tickets].max().item()) == 0, "tickets not back at zero"
    # other shapes, tilings and part counts on the same (never re-zeroed) workspace
    for M, N, K, cuts, knobs in ((8, 1003, 1000, (256, 512, 768), dict(BN=48)), (37, 520, 2304, (768, 1536), dict(BN=112, BK=64)),
                                 (128, 260, 1024, (512,), dict(BN=64)), (300, 200, 2048, (512, 1024, 1536), dict(BN=128)),
                                 (70, 2100, 1024, (256, 512, 768), dict(BN=32))):     # 264 work items: two rounds
        A2, B2 = _inputs(M, N, K, 60 + M)
        bias = synth.uniform_bf16((N,), -0.1, 0.1, 8)
        d2 = rg.rg_desc(cuts=cuts, split_merge=LAST_ARRIVER, **knobs)
        assert rg.rg_gemm_workspace_bytes(d2, M, N) <= nb
        out = torch.empty((M, N), dtype=torch.float32, device=DEV); out.view(torch.int32).fill_(-1)
        rg.rg_gemm(d2, synth.to_torch(A2, DEV), synth.to_torch(B2, DEV), out, bias=synth.to_torch(bias, DEV), act=1, ws=ws)
        torch.cuda.synchronize()
        assert_bits_equal(out.cpu().numpy(), rgo.gemm(A2, B2, cuts=cuts, atom_model=HW, bias=bias, act=1, out_dtype=rgo.F32), f"{M}x{N}x{K} {knobs}")
        assert int(ws[:tickets].max().item()) == 0
    for pd, md in ((rgo.BF16, rgo.F32), (rgo.F16, rgo.F16)):
        for tree in (rg.RG_TREE_LEFT, rg.RG_TREE_BALANCED):
            got = gpu_gemm(A[:, :2048], B[:300, :2048], cuts=(512, 1024, 1536), tree=tree, partial_dtype=pd, merge_dtype=md, split_merge=LAST_ARRIVER, out_dtype=rgo.F16)
            want = rgo.gemm(A[:, :2048], B[:300, :2048], cuts=(512, 1024, 1536), tree=tree, atom_model=HW, partial_dtype=pd, merge_dtype=md, out_dtype=rgo.F16)
            assert_bits_equal(got, want, f"last-arriver partial={pd} merge={md} tree={tree}")
    assert rg.rg_desc_class(d) == rg.rg_desc_class(rg.rg_desc(cuts=cuts8))
    with pytest.raises(rg.RgError):
        rg.rg_gemm(rg.rg_desc(cuts=tuple(64 * t for t in range(1, 10)), split_merge=LAST_ARRIVER), At, Bt, out, ws=ws)   # nine cuts: ten parts
    with pytest.raises(rg.RgError):
        rg.rg_gemm_noalloc(rg.rg_desc(cuts=cuts8, split_merge=LAST_ARRIVER), At, Bt, torch.empty((32, 4096), dtype=torch.bfloat16, device=DEV))
    assert rg.rg_device_status() == 0


def test_static_operands_in_a_run_of_independent_calls():
    """b_static = 2 (neither operand is written by work in flight): the loads of a call start while the merge of the
    call before it is still running; its stores wait.  A run of calls that share the workspace, back to back on one
    stream, with and without cuts and on both kernels, gives the bits of the same calls made one at a time."""
    cuts8 = tuple(1792 * t for t in range(1, 8))
    A, _ = _inputs(32, 8, 14336, 21, spread=False)
    At = synth.to_torch(A, DEV)
    Ws = [synth.device_normal((4096, 14336), 0.02, 30 + i, torch.bfloat16, DEV) for i in range(3)]
    res = synth.device_normal((32, 4096), 1.0, 40, torch.bfloat16, DEV)
    d = rg.rg_desc(cuts=cuts8, b_static=2)
    ws = torch.empty(rg.rg_gemm_workspace_bytes(d, 32, 4096), dtype=torch.uint8, device=DEV)
    alone = [gpu_gemm(At, W, cuts=cuts8, residual=res) for W in Ws]
    outs = [torch.empty((32, 4096), dtype=torch.bfloat16, device=DEV) for _ in range(12)]
    for o in outs: o.view(torch.int16).fill_(-1)
    torch.cuda.synchronize()
    for i, o in enumerate(outs):
        rg.rg_gemm(d, At, Ws[i % 3], o, residual=res, ws=ws)
    torch.cuda.synchronize()
    for i, o in enumerate(outs):
        assert_bits_equal(synth.from_torch(o), alone[i % 3], f"call {i} of the run")
    # large tiles without cuts (the two-SM kernel), alternating with the split-K calls above on the same stream
    X = synth.device_normal((600, 2048), 1.0, 50, torch.bfloat16, DEV); Wb = synth.device_normal((1500, 2048), 0.05, 51, torch.bfloat16, DEV)
    ref = gpu_gemm(X, Wb)
    d2 = rg.rg_desc(b_static=2)
    big = [torch.empty((600, 1500), dtype=torch.bfloat16, device=DEV) for _ in range(4)]
    for i, o in enumerate(big):
        rg.rg_gemm(d2, X, Wb, o)
        rg.rg_gemm(d, At, Ws[i % 3], outs[i], residual=res, ws=ws)
    torch.cuda.synchronize()
    for i, o in enumerate(big):
        assert_bits_equal(synth.from_torch(o), ref, f"two-SM call {i}")
        assert_bits_equal(synth.from_torch(outs[i]), alone[i % 3], f"split-K call {i} between them")
    # the GEMV family under the same promise: its loads do not wait either, its epilogue reads and stores do
    dv = rg.rg_desc(atom=rg.RG_ATOM_SCALAR, fma=1, b_static=2)
    alone_v = [gpu_gemm(At[:2], W, atom=rg.RG_ATOM_SCALAR, fma=1, residual=res[:2]) for W in Ws]
    outs_v = [torch.empty((2, 4096), dtype=torch.bfloat16, device=DEV) for _ in range(9)]
    for o in outs_v: o.view(torch.int16).fill_(-1)
    torch.cuda.synchronize()
    for i, o in enumerate(outs_v):
        rg.rg_gemm(dv, At[:2], Ws[i % 3], o, residual=res[:2])
    torch.cuda.synchronize()
    for i, o in enumerate(outs_v):
        assert_bits_equal(synth.from_torch(o), alone_v[i % 3], f"GEMV call {i} of the run")
    assert rg.rg_device_status() == 0
