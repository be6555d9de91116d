/* rg — reduction-order-fixed GEMM, reductions and attention for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every result's bits are decided by a reduction-order descriptor and by nothing
 * else: not by the tile shape, the batch size M, the launch, or the run.  The descriptor is
 * the frozen record of every order-deciding factor (paper Sec. 3.2.2 "GEMM computation
 * descriptor", Sec. 4: "two equal records owe each other the same bits"); tile sizes,
 * pipeline depth and warp roles are speed knobs that leave the dependence tree alone
 * (Sec. 3.1 "Pipeline depth leaves the tree alone", "Warp specialization leaves it alone";
 * Sec. 3.2.2 "What tiles the output stays out of all three").
 *
 * Conventions
 *   - Pointers named in rg_tensor_t / rg_epilogue_t / rg_reduce_args_t are DEVICE pointers
 *     unless a function says "host".  The caller owns every buffer.  No function here
 *     allocates or frees device memory, and none synchronises the device or the stream,
 *     except rg_device_status (which reads a word back) and entry points that say otherwise.
 *   - Matrices are row-major; `ld` is the distance between rows in ELEMENTS.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Every call validates all of its arguments before launching anything; a call that
 *     returns an error has launched nothing.  A well-formed request the kernels cannot honour
 *     returns RG_ERR_UNSUPPORTED rather than silently computing in a different order.
 *   - No exceptions cross this boundary and there is no global state that changes arithmetic.
 */
#ifndef RG_H_
#define RG_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RG_OK = 0,
  RG_ERR_NULL = 1,          /* a required pointer is NULL */
  RG_ERR_INVALID_DESC = 2,  /* descriptor malformed (size, enum range, cuts not increasing, ...) */
  RG_ERR_UNSUPPORTED = 3,   /* well-formed, but no kernel here realises it */
  RG_ERR_SHAPE = 4,         /* tensor shapes disagree or are out of range */
  RG_ERR_ALIGNMENT = 5,     /* pointer or leading dimension breaks a 16-byte rule */
  RG_ERR_WORKSPACE = 6,     /* workspace missing or too small */
  RG_ERR_CUDA = 7,          /* the CUDA runtime or driver reported an error */
  RG_ERR_TIMEOUT = 8        /* a bounded device-side wait gave up (see rg_device_status) */
} rg_status_t;

/* RG_F16 = IEEE binary16.  RG_F8E4M3 = 8-bit float, 1-4-3, bias 7, no infinities, NaN = S.1111.111
 * (the fp8 input type of Sec. 2); it is an operand type only (A and B of rg_gemm). */
typedef enum { RG_BF16 = 0, RG_F32 = 1, RG_F16 = 2, RG_F8E4M3 = 3 } rg_dtype_t;

/* The tree that combines values (split-K partials in rg_gemm, the leaves of a row in
 * rg_reduce_rows).  Sec. 3.1: a reduction order is a binary tree up to swapping an addition's
 * inputs.  LEFT = ((v0+v1)+v2)+...; BALANCED = neighbours pair first, level by level, an
 * unpaired last value moves up unchanged: the tree a count-up butterfly builds over the logical
 * element order (Sec. 5.1, Fig. 3), height ceil(log2 n). */
typedef enum { RG_TREE_LEFT = 0, RG_TREE_BALANCED = 1 } rg_tree_t;

/* Which instruction folds products into the accumulator and how many per rounding step
 * (`instruction_k`, Sec. 3.2.1/3.2.2).  TC_BF16_K16: one tcgen05.mma kind::f16 step of 16
 * bf16 products, accumulator fp32 in tensor memory, steps chained in ascending k (App. E).
 * With RG_F16 operands the same step runs on fp16 products.  SCALAR names the GEMV family: no matrix
 * instruction; the 32 lanes of a warp share one output element, each folding its k tiles with scalar
 * multiply-adds (fused when `fma` is set), then a shuffle butterfly over the lane totals (gemv_layout,
 * gemv_fold below).  It is a different class of bits from the tensor-core path and is meant for a
 * handful of rows (decode); it takes no cuts and no inner span.  TC_F8_K32: one tcgen05.mma
 * kind::f8f6f4 step of 32 e4m3 products (operands RG_F8E4M3, and only with them); cuts are multiples
 * of 32, K is even (rows of A and B are whole byte pairs) and the leading dimensions are multiples
 * of 16.  Its step has its own rounding behaviour (Sec. 3.2.1, footnote: fp8 steps differ between
 * instruction families), so it is a class of its own. */
typedef enum { RG_ATOM_TC_BF16_K16 = 0, RG_ATOM_SCALAR = 1, RG_ATOM_TC_F8_K32 = 2 } rg_atom_t;

#define RG_MAX_CUTS 63

typedef struct {
  uint32_t size;          /* = sizeof(rg_desc_t) */
  /* ---- speed knobs: validated, NOT part of the class key (Sec. 3.2.2) ---- */
  uint16_t BM, BN, BK;    /* output tile and K step per pipeline stage; 0 = library default */
  uint8_t stages;         /* shared-memory ring depth; 0 = as many as fit */
  uint8_t cta_group;      /* 1, or 2 (pair of SMs on one 256-row tile: BN from 32, BK 64 or 128; with inner_span BN 128 or 256); 0 = default */
  uint8_t raster;         /* tile walk: 0 = default grouped walk, 1 = row-major, n in 2..64 = groups of n tile rows */
  uint8_t split_merge;    /* where split-K parts are added (same tree, same bits): 0 = the library chooses (today: 1);
                             1 = by a second kernel, through the workspace; 2 = inside the GEMM kernel, by the CTAs
                             of a thread-block cluster over distributed shared memory (one launch, no workspace;
                             2..8 parts, one-CTA tiles; RG_ERR_UNSUPPORTED where it does not apply);
                             3 = inside the GEMM kernel, through the workspace, whose first bytes hold one ticket per
                             tile (2..8 parts, one-CTA tiles): by the tile's CTAs together when every part has a
                             resident CTA of its own (no more work items than SMs: they wait for each other, with the
                             library's bounded wait), else by the CTA that stores the tile's last part.  The caller's PROMISE with 3: the workspace was zero-filled once (e.g. a
                             cudaMemset when it was allocated) and only calls of this library with split_merge = 3
                             have written it since; every such call leaves the tickets zero again.  After an
                             RG_ERR_TIMEOUT from rg_device_status, zero it again */
  /* ---- order-deciding fields: these ARE the class key ---- */
  uint8_t in_dtype;       /* rg_dtype_t of A and B: RG_BF16, RG_F16, or RG_F8E4M3 (with atom = RG_ATOM_TC_F8_K32) */
  uint8_t acc_dtype;      /* accumulator: RG_F32 */
  uint8_t partial_dtype;  /* type a finished split-K part is written at: RG_F32, RG_BF16 or RG_F16 (Sec. 3.2.2);
                             without cuts no part is written and the field has no effect on the bits */
  uint8_t merge_dtype;    /* type the running sum of the parts is kept at: RG_F32, or the 16-bit type of the parts */
  uint8_t atom;           /* rg_atom_t */
  uint8_t k_tail;         /* 0 = the short K turn runs last, missing products are absent */
  uint8_t fma;            /* multiply-add fusion on scalar leaves (reductions: x*x feeding an add) */
  uint8_t tree;           /* rg_tree_t */
  uint32_t n_cuts;        /* split-K: number of interior cut points (0 = plain GEMM) */
  uint32_t cuts[RG_MAX_CUTS]; /* 0 < cuts[0] < ... < cuts[n_cuts-1] < K; part s = [cuts[s-1], cuts[s]) */
  uint32_t inner_span;    /* second level of the cut nest (Sec. 3.2.2; App. E per-group accumulation): 0 = none;
                             else, inside every part, an accumulator is closed every inner_span k (a multiple of the
                             step width: 16, or 32 with e4m3 operands) and the closed groups are added at fp32, in
                             ascending order, into the part's running sum.  inner_span = one step is the plan in
                             which an instruction's result reaches the running sum in a rounding of its own
                             (Sec. 3.2.2, `use_fast_accum` off; App. E, per-MMA accumulation).  Order-deciding:
                             part of the class key. */
  uint8_t gemv_layout;    /* RG_ATOM_SCALAR only: how the 32 lanes of a warp deal the 8-wide k tiles of one output
                             element (Sec. 3.2.2 "GEMV", `layout`): 0 = strided (lane l takes tiles l, l+32, ...),
                             1 = contiguous (lane l takes the l-th run of ceil(tiles/32) tiles) */
  uint8_t gemv_fold;      /* RG_ATOM_SCALAR only: the butterfly over the lane totals: 0 = offsets counted up
                             (balanced tree over the lanes), 1 = counted down (balanced tree over the lanes in
                             bit-reversed order: a different sum) */
  /* ---- two more speed knobs (not part of the class key) ---- */
  uint8_t sm_share;       /* one-CTA kernel: 0 = the library chooses (today: 1); 1 = a CTA takes a whole SM; 2 = a CTA takes
                             half an SM's shared and tensor memory (four epilogue warps, tiles up to 128 columns), so the
                             CTAs of the next launch become resident beside it while it finishes */
  uint8_t b_static;       /* 1 = the caller promises that no work still in flight on the stream when this call is
                             enqueued writes B (weights in an inference loop): the kernel may fetch its first B boxes
                             before the kernels ahead of it have finished (A is not read early).  2 = the same
                             promise for A and B (calls that share an input, or whose input was complete before the work
                             now in flight was enqueued): no load of the call waits for the kernels ahead; its stores to
                             C and to the workspace still do, and a split-K call leaves its merge a few SMs of its own so
                             that such calls follow each other at the weights' streaming rate.  Honoured by the
                             tensor-core kernels and the GEMV family.  0 = no promise */
} rg_desc_t;

/* A row-major matrix in device memory. */
typedef struct {
  void* ptr;
  int32_t dtype;          /* rg_dtype_t */
  int64_t rows, cols;
  int64_t ld;             /* elements between consecutive rows, >= cols */
} rg_tensor_t;

/* Fused epilogue, applied in this fixed order in fp32 with one rounding at the very end
 * (where the rounding to the output type falls is part of the order, Sec. 2):
 *   v = merged accumulator;  v += bias[j];  v = silu(v);  v += residual[i, j];  C = round(v). */
typedef struct {
  const void* bias;       /* [N], nullable */
  int32_t bias_dtype;
  int32_t act;            /* 0 none, 1 SiLU: v / (1 + exp(-v)), exp as fixed by this library */
  const void* residual;   /* [M, N], nullable */
  int32_t residual_dtype;
  int64_t ldr;
} rg_epilogue_t;

typedef enum { RG_OP_SUM = 0, RG_OP_RMSNORM = 1, RG_OP_SOFTMAX_DENOM = 2 } rg_reduce_op_t;

typedef struct {
  const void* weight;     /* RMSNorm: [cols], nullable (= all ones) */
  int32_t weight_dtype;
  float eps;              /* RMSNorm: added to the mean square inside the square root */
  void* aux_out;          /* SOFTMAX_DENOM: row maxima [rows] fp32; RMSNorm: 1/rms [rows] fp32; nullable */
} rg_reduce_args_t;

/* Fill *d with the library defaults: bf16 in, fp32 accumulate/partial/merge, tensor-core atom,
 * balanced tree, no cuts, all speed knobs 0. */
void rg_desc_init(rg_desc_t* d);

/* Check a descriptor against a GEMM shape (Sec. 3.2.2: cuts are contiguous parts of the
 * contracted axis).  Host only.  Cuts must be strictly increasing multiples of the step width (16; 32
 * with e4m3 operands) inside (0, K). */
rg_status_t rg_desc_validate(const rg_desc_t* d, int64_t M, int64_t N, int64_t K);

/* Equivalence-class key (Sec. 4: a descriptor holds every order-deciding factor "and nothing
 * else"; Sec. 6: configs that differ only in tiling form one class).  A 64-bit hash of the
 * canonical serialisation of the order-deciding fields; BM/BN/BK/stages/cta_group/raster and
 * the epilogue are excluded.  Returns 0 for a malformed descriptor.  Host only. */
uint64_t rg_desc_class(const rg_desc_t* d);

/* Bytes of workspace rg_gemm needs: 0 without cuts, else (n_cuts+1) * M * roundup(N,4) * sizeof(partial_dtype),
 * plus, with split_merge = 3, 64 KiB of tickets in front of the parts (the same place for every shape, so one
 * zero-filled workspace serves calls of different shapes; at most 16384 output tiles);
 * SIZE_MAX if that does not fit size_t (no buffer satisfies it, so the call is refused). */
size_t rg_gemm_workspace_bytes(const rg_desc_t* d, int64_t M, int64_t N);

/* C[M,N] = epilogue( merge_s( sum_{k in part s} A[i,k] * B[j,k] ) )   (C = A * B^T).
 *
 * Sec. 3.2.2 "Plain GEMM" and "Split-K"; Sec. 3.2.1 for the step; App. E for the chaining:
 * per output element and per part, the accumulator starts at zero and takes one tensor-core
 * step per 16 consecutive k, in ascending k; a finished part is an fp32 value; the parts are
 * added in the descriptor's tree; then the epilogue.  Without cuts one kernel does everything;
 * with cuts the parts go to `ws` as [part][M][roundup(N,4)] at partial_dtype and a second kernel
 * merges them, the running sum kept at merge_dtype (no atomics anywhere); or, on request and with 2..8
 * parts (App. E: a single launch across the split-K slices), the parts stay in the shared memory of
 * the CTAs of one thread-block cluster, which merge them in the same tree inside the GEMM kernel
 * (`split_merge = 2`).
 *
 *   A: [M,K], B: [N,K] (both K-contiguous) at d->in_dtype (bf16 or fp16); C: [M,N] bf16, fp16 or fp32;
 *   bias and residual likewise bf16, fp16 or fp32.
 *   A.ptr, B.ptr 16-byte aligned; A.ld, B.ld multiples of 8.  C, bias, residual: any alignment.
 *   epi: nullable.  ws: device, 16-byte aligned, >= rg_gemm_workspace_bytes; contents undefined
 *   afterwards (it may not be touched at all when the library merges in-cluster); may be NULL when
 *   there are no cuts or when the descriptor sets split_merge = 2.
 *   M == 0 or N == 0: returns RG_OK and launches nothing.  K == 0: RG_ERR_SHAPE.
 * Asynchronous on `cuda_stream`. */
rg_status_t rg_gemm(const rg_desc_t* d, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                    const rg_epilogue_t* epi, void* ws, size_t ws_bytes, void* cuda_stream);

/* Row reductions with a fixed tree over the columns (Sec. 3.1, Sec. 5.1; kernels named in
 * Sec. 7: row sums, softmax, rmsnorm).  `d->tree`, `d->acc_dtype` (fp32) and `d->fma` apply; the leaves
 * are the `x.cols` columns in index order.  RG_TREE_LEFT is the chain ((l0 + l1) + l2) + ... (Sec. 3.1:
 * the other end of the work/depth range; with `fma` the sum of squares is acc = fma(x, x, acc)): the
 * same class on every GPU as the balanced tree is, and far slower (C - 1 dependent adds per row).
 *   RG_OP_SUM:           out[r] = TREE(f32(x[r,:]));            out: rows x 1 fp32
 *   RG_OP_RMSNORM:       ss = TREE(x*x); rinv = 1/sqrt(ss/cols + eps);
 *                        y[r,c] = round((x*rinv)*w[c]);           out: rows x cols, bf16 or fp32
 *   RG_OP_SOFTMAX_DENOM: m = max_c x; out[r] = TREE(exp(x - m)); out: rows x 1 fp32;
 *                        args->aux_out (nullable) receives m.
 * x: bf16 or fp32.  rows == 0: RG_OK, nothing launched.  cols == 0: RG_ERR_SHAPE.
 * Asynchronous on `cuda_stream`. */
rg_status_t rg_reduce_rows(const rg_desc_t* d, rg_reduce_op_t op, const rg_tensor_t* x, const rg_tensor_t* out,
                           const rg_reduce_args_t* args, void* cuda_stream);

/* Reductions along the other axis: one tree per column over the rows in index order (Sec. 6:
 * "reductions on different dims/axes", the column sum a matrix-multiply epilogue emits, the
 * LayerNorm weight-gradient reduction; the tree is the one of Sec. 5.1, or the left fold when
 * `d->tree` is RG_TREE_LEFT, which needs no workspace).
 *   RG_COLOP_SUM: out[c] = TREE_r f32(x[r,c])
 *   RG_COLOP_DOT: out[c] = TREE_r f32(x[r,c]) * f32(y[r,c])   one rounding per product; with
 *                 `d->fma` the second product of each level-0 pair is fused into that pair's add
 * x (and y, same shape and type): bf16 or fp32, device pointers.  out: cols x 1 fp32.  More than
 * 256 rows go through partial rows in `ws` (device, 16-byte aligned, at least
 * rg_reduce_cols_workspace_bytes(rows, cols) bytes, caller-owned, contents arbitrary); the
 * partials are totals of aligned blocks of 256 rows, i.e. subtrees of the same tree, so the result
 * does not depend on the blocking.  cols == 0: RG_OK, nothing launched.  rows == 0: RG_ERR_SHAPE.
 * Asynchronous on `cuda_stream`. */
typedef enum { RG_COLOP_SUM = 0, RG_COLOP_DOT = 1 } rg_col_op_t;
size_t rg_reduce_cols_workspace_bytes(int64_t rows, int64_t cols);
rg_status_t rg_reduce_cols(const rg_desc_t* d, rg_col_op_t op, const rg_tensor_t* x, const rg_tensor_t* y,
                           const rg_tensor_t* out, void* ws, size_t ws_bytes, void* cuda_stream);

/* Attention of `heads` independent heads with a fixed reduction order (App. F).  Per query row the
 * keys are walked in blocks of `block_n`; with s_t = scale * (q . k_t), everything fp32:
 *   m_j = max(m_{j-1}, max_t s_t);  alpha = exp(m_{j-1} - m_j);  p_t = exp(s_t - m_j)
 *   l_j = alpha * l_{j-1} + TREE_t p_t          (the block's row sum, keys in index order, `sum_tree`)
 *   O_j = alpha * O_{j-1} + (P . V)_block       (P = p narrowed to `p_dtype`)
 * and the answer is O_B / l_B: one division at the end, one rounding to O's type.  Both products are
 * chains of tensor-core steps from a zero accumulator (RG_ATOM_TC_BF16_K16): over the head dimension
 * for the scores, over the block's keys for P . V.  exp is an exponential this library fixes from IEEE
 * operations: base e, or base two (`exp_base`), a cheaper polynomial and another class of bits.
 * Every block boundary is a rounding of O and l, so block_n is part of the class of bits.
 * mask = 1 is causal masking (query row i sees keys t <= i, Nq rows against the first keys): the walk of
 * the query tile [q0, q0 + block_m) stops at key q0 + block_m, and in the blocks from q0 on every score
 * takes an offset before the maximum, 0 where t <= i and -1e6 where t > i.  block_m must be 128 (the
 * kernel's query tile) and a multiple of block_n; it is 0 or 128 without masking.
 *
 * Q [heads*Nq, d], K [heads*Nk, d], Vt [heads*d, Nk] (V transposed: keys contiguous, what rg_gemm
 * writes for W_v . X^T) and O [heads*Nq, d]: device pointers, heads stacked along the rows.  Q, K,
 * Vt bf16, 16-byte aligned, leading dimensions multiples of 8; O bf16, fp16 or fp32.  d is 64 or 128,
 * block_n 64 or 128.  Asynchronous on `cuda_stream`; no workspace. */
typedef struct {
  uint32_t size;          /* = sizeof(rg_attn_desc_t) */
  uint32_t heads;         /* >= 1 */
  uint32_t block_n;       /* key block width: 64 or 128 */
  uint32_t block_m;       /* query tile height, part of the descriptor when mask = 1 (App. F): 128; else 0 or 128 */
  float scale;            /* scores are multiplied by this in fp32 */
  uint8_t sum_tree;       /* rg_tree_t of the row sum inside a block: RG_TREE_BALANCED */
  uint8_t p_dtype;        /* type the probabilities are narrowed to: RG_BF16 */
  uint8_t mask;           /* 0 = none, 1 = causal */
  uint8_t div_place;      /* 0 = once, at the end */
  uint8_t exp_base;       /* 0 = base e; 2 = base two (the caller folds log2 e into `scale`, App. F) */
  uint8_t _pad[3];
} rg_attn_desc_t;
rg_status_t rg_attention(const rg_attn_desc_t* d, const rg_tensor_t* Q, const rg_tensor_t* K, const rg_tensor_t* Vt,
                         const rg_tensor_t* O, void* cuda_stream);

/* Host-buffer forms of rg_gemm and rg_reduce_rows, for callers whose data lives in host memory.
 * Every tensor / epilogue / args pointer is a HOST pointer (pinned memory makes the copies
 * asynchronous).  `dev_scratch` is a caller-owned DEVICE buffer of at least
 * rg_*_host_scratch_bytes(...) bytes, 256-byte aligned, that the call uses for the device
 * copies of its operands, its result and the split-K workspace.  Each call enqueues the
 * host-to-device copies, the kernels and the device-to-host copy of the result on
 * `cuda_stream` and returns without synchronising. */
size_t rg_gemm_host_scratch_bytes(const rg_desc_t* d, int64_t M, int64_t N, int64_t K, int32_t c_dtype,
                                  const rg_epilogue_t* epi);
rg_status_t rg_gemm_host(const rg_desc_t* d, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                         const rg_epilogue_t* epi, void* dev_scratch, size_t dev_scratch_bytes, void* cuda_stream);
/* rg_reduce_rows_host: args->weight is read by RG_OP_RMSNORM only; with another op a non-null weight is
 * refused (RG_ERR_UNSUPPORTED) before anything is copied.  The scratch size covers the row copy, the
 * result, the RMSNorm weight and the auxiliary output, whether or not a call uses them. */
size_t rg_reduce_rows_host_scratch_bytes(rg_reduce_op_t op, const rg_tensor_t* x, const rg_tensor_t* out);
rg_status_t rg_reduce_rows_host(const rg_desc_t* d, rg_reduce_op_t op, const rg_tensor_t* x, const rg_tensor_t* out,
                                const rg_reduce_args_t* args, void* dev_scratch, size_t dev_scratch_bytes,
                                void* cuda_stream);

/* Split-K GEMM for callers that cannot allocate device memory (the paper has no counterpart:
 * this entry point exists for deployment, not for the method).  A serving loop whose memory
 * pool is frozen after start-up, a plugin whose host framework owns the allocator, or a decode
 * path that cannot afford the device-wide synchronisation of cudaMalloc still needs somewhere
 * to put the fp32 parts of a split-K GEMM.  This variant of rg_gemm keeps that workspace in a
 * fixed array of RG_NOALLOC_WS_BYTES inside the library image (each GPU that loads the library
 * holds it until the process exits), so the caller passes only inputs and the output.
 *   - Same arguments, results and bits as rg_gemm with the same descriptor.
 *   - It calls no cudaMalloc, cudaFree or allocating library routine.
 *   - A shape whose workspace, rg_gemm_workspace_bytes(d, M, N), exceeds RG_NOALLOC_WS_BYTES is
 *     refused with RG_ERR_WORKSPACE; nothing is launched.
 *   - The first call on each device looks up the array's device address (with that device
 *     current).  Make that first call before any stream capture begins.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left.
 *     Nothing needs clearing (every part that is read was written by the same call), but two
 *     calls that overlap on the GPU (different streams, no dependency) race on it: serialise
 *     them. */
#define RG_NOALLOC_WS_BYTES (8u << 20)
rg_status_t rg_gemm_noalloc(const rg_desc_t* d, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                            const rg_epilogue_t* epi, void* cuda_stream);

/* Self-test of the bounded device-side wait (the paper has no counterpart: this is the library's
 * failure-detection path, exercised on purpose).  Launches one small CTA that waits on a barrier
 * nothing arrives on: one warp with the limit `limit_ns` (1 us .. 100 ms, else RG_ERR_SHAPE), which
 * runs out, records RG_SELFTEST_WAIT_CODE in the health word and raises the CTA's abort flag; a second
 * warp with the library's ordinary long limit, which must leave as soon as it sees the flag.  Each
 * warp that abandoned its wait adds one to *dev_counter (a DEVICE pointer to 4 bytes the caller has
 * set to zero), so a caller reads 2 there afterwards.  The kernel returns normally: nothing hangs,
 * nothing faults and the context stays usable; rg_device_status then reports RG_ERR_TIMEOUT with
 * that code, once.  Asynchronous on `cuda_stream`. */
#define RG_SELFTEST_WAIT_CODE 0xE00u
rg_status_t rg_selftest_bounded_wait(uint64_t limit_ns, uint32_t* dev_counter, void* cuda_stream);

/* Self-test of the exponentials.  The paper's attention kernel calls the hardware's base-two exponential
 * (App. F), whose bits are not defined off the GPU; this library fixes exp and exp2 as sequences of IEEE
 * operations instead (rg_exp, rg_exp2), and its kernels use forms of them with the range selects removed where an
 * argument's range is known.  y[i] = FORM(x[i]), computed on the device by the very functions the kernels call,
 * so that every form can be compared with the CPU oracle directly rather than through a reduction:
 *   0 rg_exp            1 rg_exp2            2 the GEMM epilogue's form of rg_exp for |x| <= 87
 *   3 the attention kernel's packed (fp32x2) form of rg_exp for -87.33655 <= x <= 0
 *   4 the attention kernel's form of rg_exp2 for -126 <= x <= 0      5 its form of rg_exp2 for x <= 0 or NaN
 *   6 the softmax normaliser's form of rg_exp for x <= 0 or NaN
 *   7 the GEMM epilogue's SiLU, v / (1 + e^-v) with the specified exponential, applied as the kernels apply it: to segments of 32
 *     consecutive values, with the range-free exponential when no magnitude of a segment exceeds 87 (n % 32 == 0)
 * Outside a form's stated range its result is unspecified.  x, y: DEVICE pointers to n floats (n >= 0, may
 * alias).  RG_ERR_SHAPE for another form, n < 0, or form 7 with n not a multiple of 32.  Asynchronous on
 * `cuda_stream`. */
rg_status_t rg_selftest_exp(int32_t form, const float* x, float* y, int64_t n, void* cuda_stream);

/* Device-side health word of the current device.  Every wait inside the kernels is bounded; a
 * wait that gives up records a code here, lets the kernel drain and return, and leaves the
 * context usable.  Copies the word to *code (0 = healthy) and clears it.  Synchronises the
 * device.  Returns RG_ERR_TIMEOUT if the word was non-zero. */
rg_status_t rg_device_status(uint32_t* code);

const char* rg_status_string(rg_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* RG_H_ */
