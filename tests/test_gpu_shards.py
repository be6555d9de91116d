"""What every rank of a multi-GPU run computes: its own slice of the rows (Sec. 3.2.2: which tile owns an
output element does not move its chain, so a row shard returns the bits of the same rows of the
unsharded call).  One GPU runs every rank's slice in turn and the concatenation must equal the
unsharded result bit for bit; there is no exchange step to emulate."""
import numpy as np
import pytest
import torch

import paper_2609_11356_b200 as rg
from oracle import rgo
from paper_2609_11356_b200 import dist, synth
from tests._gpu_util import DEV, HW, assert_bits_equal, gpu_gemm, gpu_reduce
from tests.test_gpu_attention import gpu_attention

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("world", [2, 3, 8])
def test_gemm_row_shards_concatenate_to_the_unsharded_bits(world):
    M, N, K = 777, 520, 2048
    A = synth.spread_exponents_bf16(synth.normal_bf16((M, K), 1.0, 1), 2, -8, 8)
    B = synth.normal_bf16((N, K), 0.02, 3)
    bias = synth.uniform_bf16((N,), -0.1, 0.1, 4)
    res = synth.normal_bf16((M, N), 1.0, 5)
    for cuts in ((), (512, 1024, 1536)):
        whole = gpu_gemm(A, B, cuts=cuts, bias=bias, act=1, residual=res)
        parts = []
        for r in range(world):
            lo, hi = dist.shard_rows(M, r, world)
            parts.append(gpu_gemm(A[lo:hi], B, cuts=cuts, bias=bias, act=1, residual=res[lo:hi]))
        assert_bits_equal(np.concatenate(parts), whole, f"GEMM rows over {world} ranks, cuts={cuts}")
    # column shards of the weight matrix concatenate along N the same way
    whole = gpu_gemm(A[:130], B, out_dtype=rgo.F32)
    cols = [gpu_gemm(A[:130], B[slice(*dist.shard_rows(N, r, world))], out_dtype=rgo.F32) for r in range(world)]
    assert_bits_equal(np.concatenate(cols, axis=1), whole, f"GEMM columns over {world} ranks")


@pytest.mark.parametrize("world", [2, 3, 8])
def test_reduction_row_shards(world):
    x = synth.add_cancellation_pairs(synth.normal_f32((301, 5000), 100.0, 6), 7, pairs=8)
    w = synth.normal_f32((5000,), 0.05, 8, mean=1.0)
    for op, kw in ((rg.RG_OP_SUM, {}), (rg.RG_OP_SOFTMAX_DENOM, {}), (rg.RG_OP_RMSNORM, dict(weight=w, eps=1e-5))):
        whole, aux = gpu_reduce(op, x, **kw)
        outs, auxs = [], []
        for r in range(world):
            lo, hi = dist.shard_rows(x.shape[0], r, world)
            o, a = gpu_reduce(op, x[lo:hi], **kw)
            outs.append(o); auxs.append(a)
        assert_bits_equal(np.concatenate(outs), whole, f"reduction {op} over {world} ranks")
        if op != rg.RG_OP_SUM:
            assert_bits_equal(np.concatenate(auxs), aux, f"reduction {op} aux over {world} ranks")


@pytest.mark.parametrize("world", [2, 3, 8])
def test_attention_shards_by_head_and_by_query_rows(world):
    H, Nq, Nk, d = 8, 200, 330, 128
    g = np.random.default_rng(9)
    Q = synth.f32_to_bf16_bits(g.standard_normal((H * Nq, d)).astype(np.float32))
    Kk = synth.f32_to_bf16_bits(g.standard_normal((H * Nk, d)).astype(np.float32))
    V = synth.f32_to_bf16_bits(g.standard_normal((H * Nk, d)).astype(np.float32))
    scale = float(np.float32(d ** -0.5))
    whole = gpu_attention(Q, Kk, V, block_n=128, scale=scale, heads=H, out_dtype=rgo.F32)
    # heads are independent units: a rank takes a contiguous range of heads
    parts = []
    for r in range(world):
        lo, hi = dist.shard_rows(H, r, world)
        if hi > lo:
            parts.append(gpu_attention(Q[lo * Nq:hi * Nq], Kk[lo * Nk:hi * Nk], V[lo * Nk:hi * Nk], block_n=128, scale=scale,
                                       heads=hi - lo, out_dtype=rgo.F32))
    assert_bits_equal(np.concatenate(parts), whole, f"attention heads over {world} ranks")
    # and, without masking, so are the query rows of one head
    q0 = Q[:Nq]; k0 = Kk[:Nk]; v0 = V[:Nk]
    rows = []
    for r in range(world):
        lo, hi = dist.shard_rows(Nq, r, world)
        rows.append(gpu_attention(q0[lo:hi], k0, v0, block_n=128, scale=scale, out_dtype=rgo.F32))
    assert_bits_equal(np.concatenate(rows), whole[:Nq], f"attention query rows over {world} ranks")


def test_attention_at_the_benchmark_shape_on_sampled_rows():
    """32 heads x 4096 queries x 4096 keys x 128, the shape the benchmark times: 96 sampled query rows
    (three per head, tile edges included) against the oracle, bit for bit, in both exponential bases."""
    H, N, d = 32, 4096, 128
    bf = torch.bfloat16
    Q = synth.device_normal((H * N, d), 1.0, 41, bf, DEV); Kt = synth.device_normal((H * N, d), 1.0, 42, bf, DEV)
    Vt = synth.device_normal((H * d, N), 1.0, 43, bf, DEV)
    O = torch.empty((H * N, d), dtype=bf, device=DEV)
    g = np.random.default_rng(44)
    for base in (2, 0):
        scale = float(np.float32(d ** -0.5 * (np.log2(np.e) if base == 2 else 1.0)))
        O.view(torch.int16).fill_(-1)
        rg.rg_attention(rg.rg_attn_desc(block_n=128, scale=scale, heads=H, exp_base=base), Q, Kt, Vt, O)
        torch.cuda.synchronize()
        for h in range(H):
            rows = np.unique(np.concatenate([g.integers(0, N, 2), [[0, 127, 128, N - 1][h % 4]]]))
            q = synth.from_torch(Q[h * N + torch.from_numpy(rows).to(DEV)])
            k = synth.from_torch(Kt[h * N:(h + 1) * N])
            v = np.ascontiguousarray(synth.from_torch(Vt[h * d:(h + 1) * d]).T)
            want = rgo.attention(q, k, v, block_n=128, scale=scale, atom_model=HW, out_dtype=rgo.BF16, exp_base=base)
            got = synth.from_torch(O[h * N + torch.from_numpy(rows).to(DEV)])
            assert_bits_equal(got, want, f"attention bench shape, base {base}, head {h}")
    assert rg.rg_device_status() == 0
