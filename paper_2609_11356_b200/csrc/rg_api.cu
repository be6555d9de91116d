// The C boundary: argument validation, descriptor canonicalisation and class key, plan
// selection, and the host-buffer forms.  Nothing here does arithmetic on data.
#include <algorithm>
#include <string.h>

#include "rg_internal.h"

namespace {

constexpr int64_t DIM_LIMIT = (int64_t(1) << 31) - 1024;

bool dtype_ok(int32_t t) { return t == RG_BF16 || t == RG_F32 || t == RG_F16; }   // epilogue operands and outputs
size_t esize(int32_t t) { return t == RG_F32 ? 4 : t == RG_F8E4M3 ? 1 : 2; }
size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Structural checks that do not depend on a shape.
rg_status_t check_desc_fields(const rg_desc_t* d) {
  if (!d) return RG_ERR_NULL;
  if (d->size != sizeof(rg_desc_t)) return RG_ERR_INVALID_DESC;
  if (d->in_dtype > RG_F8E4M3 || d->acc_dtype > RG_F8E4M3 || d->partial_dtype > RG_F8E4M3 || d->merge_dtype > RG_F8E4M3)
    return RG_ERR_INVALID_DESC;
  // the 8-bit operand type and the 32-wide step name each other
  if ((d->in_dtype == RG_F8E4M3) != (d->atom == RG_ATOM_TC_F8_K32)) return RG_ERR_INVALID_DESC;
  if (d->atom > RG_ATOM_TC_F8_K32 || d->tree > RG_TREE_BALANCED || d->fma > 1 || d->k_tail > 1) return RG_ERR_INVALID_DESC;
  if (d->n_cuts > RG_MAX_CUTS) return RG_ERR_INVALID_DESC;
  if (d->gemv_layout > 1 || d->gemv_fold > 1) return RG_ERR_INVALID_DESC;
  for (uint32_t i = 0; i < d->n_cuts; ++i) {
    if (d->cuts[i] == 0) return RG_ERR_INVALID_DESC;
    if (i > 0 && d->cuts[i] <= d->cuts[i - 1]) return RG_ERR_INVALID_DESC;
  }
  return RG_OK;
}

// What the kernels of this library can honour.
rg_status_t check_desc_supported(const rg_desc_t* d) {
  if (d->in_dtype == RG_F32 || d->acc_dtype != RG_F32) return RG_ERR_UNSUPPORTED;
  if (d->partial_dtype == RG_F8E4M3 || d->merge_dtype == RG_F8E4M3) return RG_ERR_UNSUPPORTED;
  // parts at fp32 summed at fp32, parts at a 16-bit type summed at fp32, or both at that type (Sec. 3.2.2)
  if (d->merge_dtype != RG_F32 && d->merge_dtype != d->partial_dtype) return RG_ERR_UNSUPPORTED;
  if (d->k_tail != 0) return RG_ERR_UNSUPPORTED;
  if (d->atom == RG_ATOM_SCALAR) {
    // GEMV family: one chain per lane, a balanced lane fold, nothing to split
    if (d->n_cuts || d->inner_span || d->tree != RG_TREE_BALANCED) return RG_ERR_UNSUPPORTED;
    return RG_OK;
  }
  if (d->gemv_layout || d->gemv_fold) return RG_ERR_INVALID_DESC;   // lane fields belong to the scalar family
  if (d->BM != 0 && d->BM != 128 && d->BM != 256) return RG_ERR_UNSUPPORTED;
  if (d->BN != 0 && (d->BN % 16 != 0 || d->BN < 16 || d->BN > 256)) return RG_ERR_UNSUPPORTED;
  if (d->BK != 0 && d->BK != 64 && d->BK != 128 && d->BK != 256) return RG_ERR_UNSUPPORTED;

  if (d->cta_group > 2) return RG_ERR_INVALID_DESC;
  // a pair works on 256 rows and at least 32 columns; with a second cut level on 128 or 256 columns
  if (d->cta_group == 2 && (d->BM == 128 || (d->BN != 0 && (d->BN < 32 || (d->inner_span && d->BN != 128 && d->BN != 256))) || d->BK == 256))
    return RG_ERR_UNSUPPORTED;
  if (d->cta_group == 1 && d->BM == 256) return RG_ERR_UNSUPPORTED;
  if (d->raster > 64) return RG_ERR_INVALID_DESC;
  if (d->split_merge > 3 || d->sm_share > 2 || d->b_static > 2) return RG_ERR_INVALID_DESC;
  // the last-arriver merge: 2 to 8 parts, one-CTA tiles at a whole SM each, no second cut level
  if (d->split_merge == 3 && (d->n_cuts < 1 || d->n_cuts > 7 || d->inner_span || d->cta_group == 2 || d->BM == 256 || d->BK == 256 || d->sm_share == 2))
    return RG_ERR_UNSUPPORTED;
  // two CTAs per SM: the one-CTA kernel with four epilogue warps, tiles up to 128 columns, no second cut level
  if (d->sm_share == 2 && (d->cta_group == 2 || d->BM == 256 || d->BN > 128 || d->BK == 256 || d->inner_span || d->split_merge == 2))
    return RG_ERR_UNSUPPORTED;
  // the in-cluster merge: 2 to 8 parts (one CTA of a cluster per part), one-CTA tiles, no second cut level
  if (d->split_merge == 2 && (d->n_cuts < 1 || d->n_cuts > 7 || d->inner_span || d->cta_group == 2 || d->BM == 256 || d->BK == 256))
    return RG_ERR_UNSUPPORTED;
  const uint32_t step = d->atom == RG_ATOM_TC_F8_K32 ? 32 : 16;   // products per tensor-core step
  for (uint32_t i = 0; i < d->n_cuts; ++i)
    if (d->cuts[i] % step != 0) return RG_ERR_UNSUPPORTED;   // a cut may not split a step
  if (d->inner_span) {
    // a group is a whole number of steps, down to a single one (an accumulator closed after every instruction:
    // the two-rounding plan); the running sum lives in the epilogue warps' registers; 64-wide stages
    if (d->inner_span % step != 0) return RG_ERR_UNSUPPORTED;
    if (d->BK != 0 && d->BK != 64) return RG_ERR_UNSUPPORTED;
  }
  return RG_OK;
}

rg_status_t check_tensor(const rg_tensor_t* t, bool operand = false) {
  if (!t) return RG_ERR_NULL;
  if (!dtype_ok(t->dtype) && !(operand && t->dtype == RG_F8E4M3)) return RG_ERR_SHAPE;
  if (t->rows < 0 || t->cols < 0 || t->rows > DIM_LIMIT || t->cols > DIM_LIMIT) return RG_ERR_SHAPE;
  if (t->ld < t->cols) return RG_ERR_SHAPE;
  if (t->rows > 0 && t->cols > 0 && !t->ptr) return RG_ERR_NULL;
  return RG_OK;
}

rg_status_t check_epilogue(const rg_epilogue_t* e, int64_t N) {
  if (!e) return RG_OK;
  if (e->act != 0 && e->act != 1) return RG_ERR_UNSUPPORTED;
  if (e->bias && !dtype_ok(e->bias_dtype)) return RG_ERR_SHAPE;
  if (e->residual && (!dtype_ok(e->residual_dtype) || e->ldr < N)) return RG_ERR_SHAPE;
  return RG_OK;
}

rg_status_t check_gemm_shapes(const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C) {
  rg_status_t s;
  if ((s = check_tensor(A, true)) != RG_OK || (s = check_tensor(B, true)) != RG_OK || (s = check_tensor(C)) != RG_OK) return s;
  if (A->dtype == RG_F32 || B->dtype != A->dtype) return RG_ERR_UNSUPPORTED;
  if (A->cols != B->cols || C->rows != A->rows || C->cols != B->rows) return RG_ERR_SHAPE;
  return RG_OK;
}

int device_sms() { return rg::current_device().sms; }

// Split-K in one launch: the parts of an output tile go to the CTAs of one thread-block cluster, which merge
// them over distributed shared memory (no workspace, no second kernel).  Taken when the descriptor asks for it
// (`split_merge = 2`); the default stays the two-kernel path, which is faster on this GPU: a cluster of eight
// must sit in one GPC, so only 15 of them (120 of 148 SMs) stream at once, and the cluster-wide hand-over at the
// end of a tile costs more than the second launch it saves (decode shape: 27.7 us against 26.2 us).
// Returns false if it does not apply or fit.
bool plan_cluster_merge(const rg_desc_t* d, int64_t M, int64_t N, rg::GemmPlan* plan) {
  const int S = plan->n_parts;
  if (S < 2 || S > 8 || d->inner_span || d->cta_group == 2 || d->BM == 256 || d->BK == 256 || d->split_merge == 1) return false;
  if (d->split_merge != 2) return false;                    // on request only (see make_plan)
  const bool f8 = d->in_dtype == RG_F8E4M3;
  const int bk = d->BK ? d->BK : (M <= 64 ? 128 : 64);
  const int avail = rg::max_active_clusters(S, bk, f8);
  if (avail < 1) return false;
  const int64_t tiles_m = (M + 127) / 128;
  const int64_t rows = M < 128 ? M : 128;
  int best = 0; int64_t best_cost = -1;
  for (int bn = 32; bn <= 256; bn += 16) {
    if (d->BN && bn != d->BN) continue;
    const int smax = rg::max_stages_for(bn, bk, 1, M, true);
    if (smax < (d->stages ? d->stages : 2)) continue;
    // time ~ rounds of clusters x bytes a CTA streams per tile (its rows of A and its bn rows of B)
    const int64_t tiles = tiles_m * ((N + bn - 1) / bn);
    const int64_t cost = ((tiles + avail - 1) / avail) * (bn + rows);
    if (best_cost < 0 || cost < best_cost) { best = bn; best_cost = cost; }
  }
  if (!best) return false;
  plan->cluster_merge = 1;
  plan->BN = best; plan->BK = bk; plan->cta_group = 1;
  plan->stages = d->stages ? d->stages : rg::max_stages_for(best, bk, 1, M, true);
  plan->raster = d->raster == 1 ? 1 : 0;
  plan->group_m = d->raster >= 2 ? d->raster : 8;
  return true;
}

rg_status_t make_plan(const rg_desc_t* d, int64_t M, int64_t N, int64_t K, rg::GemmPlan* plan) {
  plan->n_parts = (int)d->n_cuts + 1;
  plan->cluster_merge = 0;
  plan->ticket_merge = d->split_merge == 3 ? 1 : 0;
  plan->reserve_sms = 0; plan->merge_small = 0;
  plan->half_sm = 0;
  plan->b_static = d->b_static;
  plan->tree = d->tree;
  plan->partial_dtype = d->partial_dtype;
  plan->merge_dtype = d->merge_dtype;
  plan->inner_span = (int)d->inner_span;
  for (int s = 0; s < plan->n_parts; ++s) {
    plan->part_begin[s] = s == 0 ? 0 : (int32_t)d->cuts[s - 1];
    plan->part_end[s] = s == plan->n_parts - 1 ? (int32_t)K : (int32_t)d->cuts[s];
  }
  if (plan_cluster_merge(d, M, N, plan)) return RG_OK;
  if (d->split_merge == 2) return RG_ERR_UNSUPPORTED;       // asked for, but it does not fit this shape or device
  const int sms = device_sms();
  const int64_t tiles_m = (M + 127) / 128;
  const bool skinny = M <= 64;     // weight-streaming regime: HBM bound, one partial tile row
  // On request (`sm_share = 2`) the one-CTA kernel runs at half an SM's shared and tensor memory, one CTA per SM:
  // the CTAs of the next launch in the stream then become resident beside this launch's, set themselves up and,
  // under `b_static`, fetch their first weight boxes before the kernels ahead have finished.  Not the default:
  // on the decode shape the half-depth ring streams 8 % slower, which costs more than the overlap returns while
  // the chain GEMM -> merge -> next GEMM (about 5 us of completion and launch hand-overs) paces a run of calls.
  const bool half_ok = !d->inner_span && d->cta_group != 2 && d->BM != 256 && d->BN <= 128 && d->BK != 256;
  const bool half = half_ok && d->sm_share == 2;
  if (d->sm_share == 2 && !half) return RG_ERR_UNSUPPORTED;
  // Calls that do not depend on each other (b_static = 2) with a split-K merge behind them: the merge's CTAs cannot
  // sit beside a GEMM CTA (registers), so they take SMs as the GEMM's CTAs leave, and the next call's CTAs on those SMs
  // start late.  Leaving the merge a few SMs of its own (128-thread CTAs of two units per thread, four to an SM) lets
  // the calls follow each other at the weights' streaming rate: decode shape, 1 / 8 / 32 rows: 26.5 / 23.7 / 22.7 us
  // per call without, 18.2 / 18.8 / about 20 with (117 MB in 18.2 us is 0.98 of the measured copy bandwidth).
  plan->reserve_sms = 0; plan->merge_small = 0;
  if (d->b_static == 2 && plan->n_parts > 1 && plan->n_parts <= 8 && skinny && d->split_merge <= 1 && d->sm_share != 2) {
    // the general merge kernel (256-thread CTAs, two to an SM) where that takes no more than an eighth of the SMs (it is
    // the faster of the two: 8 rows 18.8 against 20.5 us per call), else the 128-thread form (four to an SM) up to a quarter
    const int64_t merge_ctas = (M * ((N + 3) / 4) + 255) / 256;
    const int64_t need2 = (merge_ctas + 1) / 2, need4 = (merge_ctas + 3) / 4;
    if (need2 <= sms / 8) { plan->reserve_sms = (int)need2; plan->merge_small = 0; }
    else if (need4 <= sms / 4) { plan->reserve_sms = (int)need4; plan->merge_small = 1; }
  }
  const int slots = sms - plan->reserve_sms;
  if (d->BN) plan->BN = d->BN;
  else if (skinny) {
    // Weight streaming: time ~ (rounds of work items per SM) x (tile width).  Any multiple of 16 is a
    // legal tile width, so pick the one that wastes the least of the last round.
    int best = 128; int64_t best_cost = -1;
    // Without cuts a tile is one long chain of steps and narrow tiles keep every SM busy: down to 32 columns.
    // The merge by the tile's own CTAs (split_merge = 3) wants one round: every part of a tile on a resident CTA of its
    // own, so that the tile's CTAs can wait for each other and share the merge.  Widths that need a second round
    // are considered for it only if none fits one.
    for (int pass = plan->ticket_merge ? 0 : 1; pass < 2 && best_cost < 0; ++pass) {
      for (int bn = plan->n_parts == 1 ? 32 : 64; bn <= (half ? 128 : 256); bn += 16) {
        const int64_t items = ((N + bn - 1) / bn) * plan->n_parts;
        if (pass == 0 && items > slots) continue;
        const int64_t rounds = (items + slots - 1) / slots;
        // with SMs set aside for the merge a round costs about 24 columns' worth beside its width (4 rows: three rounds of
        // 80-wide tiles 22 us per call, one round of 256-wide tiles 19)
        const int64_t cost = rounds * (bn + (plan->reserve_sms ? 24 : 0));
        if (best_cost < 0 || cost < best_cost) { best = bn; best_cost = cost; }
      }
    }
    plan->BN = best;
  } else {
    plan->BN = 0;                                         // chosen together with the kernel below
  }
  // one CTA per 128-row tile, or a pair of CTAs (two SMs) per 256-row tile
  int want_group = 0;
  if (plan->ticket_merge) want_group = 1;
  else if (d->cta_group) want_group = d->cta_group;
  else if (d->BM == 256) want_group = 2;
  else if (d->BM == 128) want_group = 1;
  if (plan->BN == 0 || (want_group == 0 && !skinny)) {
    // Time per k of a round of work items, in operand rows pulled from L2 (2 bytes per row and k), is the largest of
    //   the round's CTAs x rows of one CTA / 121   L2 feeds the SMs about 15 TB/s in total, 121 SMs' worth of the next line
    //   rows of one CTA                            an SM takes in 64 bytes per clock
    //   1.3 x width (1.4 for a pair)               the arithmetic of a 128-row step, at the clock the power cap leaves
    // where a CTA of the one-CTA kernel pulls 128 rows of A and the tile's width of B, a CTA of a pair 128 and half
    // the width (charged 1.17 of that: the two CTAs' boxes meet on one barrier), and a pair's launch costs about
    // 1.4 us more (88000 row-k), which counts on short K.  Fitted on 4096- and 14336-column problems of 256-2048
    // rows (K = 512 ... 14336): 512 x 4096 x 4096 is one round of 256 x 128 pairs (19 us; 128 x 112 tiles 24),
    // 768 rows one round of 256 x 192 pairs, 384 rows 128 x 96 tiles.  Any multiple of 16 is a legal width; the
    // pair is offered multiples of 32 (a pair's step on an odd multiple of 16 measured 10-15 % slower than on its
    // neighbours).
    const int64_t tiles_m2 = (M + 255) / 256;
    const int64_t klen = plan->n_parts > 1 ? (K + plan->n_parts - 1) / plan->n_parts : K;
    int best_bn = 0, best_group = 0; double best_cost = -1;
    for (int group = 1; group <= 2; ++group) {
      if (want_group && group != want_group) continue;
      if (group == 2 && (M <= 128 || d->BK == 256)) continue;        // a pair's stage is 64 or 128 k
      // the second cut level keeps a running sum per thread: up to 128 columns it stays in registers, and the
      // one-CTA kernel's hand-over is the shorter one (8192^3, a group every 64 k: 539 TFLOP/s on 128 x 128 tiles,
      // 274 on two-SM 256 x 128, 171 on 256-wide tiles of either kernel)
      if (d->inner_span && !want_group && group == 2) continue;
      for (int bn = 256; bn >= 32; bn -= 16) {
        if (d->BN && bn != d->BN) continue;
        if (d->inner_span && !d->BN && bn > 128) continue;
        if (group == 2 && d->inner_span && bn != 256 && bn != 128) continue;
        if (group == 2 && !d->BN && bn % 32 != 0) continue;
        const int64_t items = (group == 2 ? tiles_m2 : tiles_m) * ((N + bn - 1) / bn) * plan->n_parts;
        const int64_t slots = group == 2 ? sms / 2 : sms;
        const double rows = group == 2 ? 128 + bn / 2 : 128 + bn;
        const double one_cta = std::max(rows * (group == 2 ? 1.17 : 1.0), (group == 2 ? 1.4 : 1.3) * bn);
        const int64_t last = items % slots;                               // work items of the last, partial round
        double cost = (double)(items / slots) * std::max((double)(slots * group) * rows / 121.0, one_cta);
        if (last) cost += std::max((double)(last * group) * rows / 121.0, one_cta);
        if (group == 2) cost += 88000.0 / (double)(klen > 0 ? klen : 1);
        if (group == 2 && bn != 256 && bn != 128) cost *= 1.03;       // 256 and 128 columns are compile-time forms of the pair kernel
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best_bn = bn; best_group = group; }
      }
    }
    if (best_bn) {
      if (plan->BN == 0) plan->BN = best_bn;
      if (want_group == 0) want_group = best_group;
    }
    if (plan->BN == 0) plan->BN = 64;
  }
  if (half && plan->BN > 128) plan->BN = 128;
  plan->cta_group = want_group ? want_group : 1;
  if (plan->cta_group == 2 && plan->BN < 32) plan->cta_group = 1;
  // the widest two-SM tile runs a seven-stage ring of 64-wide K steps: more slack per byte of shared memory than
  // three 128-wide stages, now that a whole turn of the ring is issued from precomputed descriptor words
  // skinny problems read long runs of each weight row per stage (DRAM likes 512-byte bursts)
  // tiles up to 128 columns (pairs up to 192) take 128-wide K steps as well (half the hand-overs; the stage still fits four times)
  plan->BK = d->BK ? d->BK : (!d->inner_span && (skinny || ((plan->BN <= 128 || (plan->cta_group == 2 && plan->BN <= 192)) && !half)) ? 128 : 64);
  // a skinny problem without cuts is bounded by the hand-overs along its one K chain: 256-wide stages halve them,
  // as long as four of them still fit
  if (!d->BK && skinny && plan->n_parts == 1 && !d->inner_span && plan->cta_group == 1 && !half &&
      rg::max_stages_for(plan->BN, 256, 1, M) >= 4)
    plan->BK = 256;
  if (plan->ticket_merge && plan->BK > 128) plan->BK = 128;
  if (plan->cta_group == 2 && ((d->inner_span && plan->BN != 128 && plan->BN != 256) || plan->BK == 256)) return RG_ERR_UNSUPPORTED;
  plan->half_sm = half && plan->cta_group == 1 && plan->BK <= 128 && rg::max_stages_for(plan->BN, plan->BK, 1, M, false, true) >= 2;
  if (d->sm_share == 2 && !plan->half_sm) return RG_ERR_UNSUPPORTED;
  const int smax = rg::max_stages_for(plan->BN, plan->BK, plan->cta_group, M, false, plan->half_sm != 0);
  plan->stages = d->stages ? d->stages : smax;
  if (plan->stages > smax) return RG_ERR_UNSUPPORTED;
  plan->raster = d->raster == 1 ? 1 : 0;
  // Tile walk: groups of group_m tile rows, column by column inside a group.  A B tile is then fetched once per group
  // (the group's tiles of that column run together) and the group's A rows are read again for every column, which
  // costs nothing while they stay in L2: the tallest group whose A rows take no more than about 56 MiB of it, as a
  // power of two from 4 to 32 (8192^3 and K = 14336: 8; K = 4096 or e4m3 operands at K = 8192: 16, +2 %; K = 2048: 32, +2 %).
  {
    const int64_t row_bytes = (int64_t)(plan->cta_group == 2 ? 256 : 128) * K * (d->in_dtype == RG_F8E4M3 ? 1 : 2);
    int g = 32;
    while (g > 4 && (int64_t)g * row_bytes > ((int64_t)56 << 20)) g >>= 1;
    plan->group_m = d->raster >= 2 ? d->raster : g;
  }
  return RG_OK;
}

}  // namespace

extern "C" {

void rg_desc_init(rg_desc_t* d) {
  if (!d) return;
  memset(d, 0, sizeof(*d));
  d->size = sizeof(rg_desc_t);
  d->in_dtype = RG_BF16; d->acc_dtype = RG_F32; d->partial_dtype = RG_F32; d->merge_dtype = RG_F32;
  d->atom = RG_ATOM_TC_BF16_K16; d->k_tail = 0; d->fma = 0; d->tree = RG_TREE_BALANCED;
}

rg_status_t rg_desc_validate(const rg_desc_t* d, int64_t M, int64_t N, int64_t K) {
  rg_status_t s = check_desc_fields(d);
  if (s != RG_OK) return s;
  if (M < 0 || N < 0 || K < 1 || M > DIM_LIMIT || N > DIM_LIMIT || K > DIM_LIMIT) return RG_ERR_SHAPE;
  if (d->n_cuts && (int64_t)d->cuts[d->n_cuts - 1] >= K) return RG_ERR_INVALID_DESC;
  return check_desc_supported(d);
}

uint64_t rg_desc_class(const rg_desc_t* d) {
  if (check_desc_fields(d) != RG_OK) return 0;
  // canonical serialisation of the order-deciding fields only; "no cuts" has one spelling
  uint8_t buf[20 + 4 * RG_MAX_CUTS];
  size_t n = 0;
  const uint8_t head[8] = {d->in_dtype, d->acc_dtype, d->partial_dtype, d->merge_dtype, d->atom, d->k_tail, d->fma, d->tree};
  memcpy(buf, head, 8); n = 8;
  const uint32_t nc = d->n_cuts;
  for (int b = 0; b < 4; ++b) buf[n++] = (uint8_t)(nc >> (8 * b));
  for (uint32_t i = 0; i < nc; ++i)
    for (int b = 0; b < 4; ++b) buf[n++] = (uint8_t)(d->cuts[i] >> (8 * b));
  for (int b = 0; b < 4; ++b) buf[n++] = (uint8_t)(d->inner_span >> (8 * b));
  buf[n++] = d->gemv_layout; buf[n++] = d->gemv_fold;
  uint64_t h = 0xcbf29ce484222325ull;                  // FNV-1a, 64 bit
  for (size_t i = 0; i < n; ++i) { h ^= buf[i]; h *= 0x100000001b3ull; }
  return h ? h : 1;
}

size_t rg_gemm_workspace_bytes(const rg_desc_t* d, int64_t M, int64_t N) {
  if (!d || d->n_cuts == 0 || d->n_cuts > RG_MAX_CUTS || M <= 0 || N <= 0) return 0;
  // a product that does not fit size_t is reported as SIZE_MAX, which no buffer satisfies
  if (N > INT64_MAX - 3) return SIZE_MAX;
  size_t b = (size_t)(d->n_cuts + 1);
  if (__builtin_mul_overflow(b, (size_t)M, &b) || __builtin_mul_overflow(b, (size_t)((N + 3) / 4 * 4), &b) ||
      __builtin_mul_overflow(b, (size_t)(d->partial_dtype == RG_F32 ? 4 : 2), &b))
    return SIZE_MAX;
  if (d->split_merge == 3 && __builtin_add_overflow(b, rg::ticket_bytes(), &b)) return SIZE_MAX;   // the tickets in front of the parts
  return b;
}

rg_status_t rg_gemm(const rg_desc_t* d, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                    const rg_epilogue_t* epi, void* ws, size_t ws_bytes, void* cuda_stream) {
  rg_status_t s = check_desc_fields(d);
  if (s != RG_OK) return s;
  if ((s = check_gemm_shapes(A, B, C)) != RG_OK) return s;
  const int64_t M = A->rows, K = A->cols, N = B->rows;
  if (K < 1) return RG_ERR_SHAPE;
  if ((s = rg_desc_validate(d, M, N, K)) != RG_OK) return s;
  if (A->dtype != d->in_dtype) return RG_ERR_SHAPE;          // operands must be of the descriptor's input type
  if ((s = check_epilogue(epi, N)) != RG_OK) return s;
  if (M == 0 || N == 0) return RG_OK;
  const int64_t ld_mult = 16 / (int64_t)esize(A->dtype);        // rows start on 16-byte boundaries
  if ((reinterpret_cast<uintptr_t>(A->ptr) & 15) || (reinterpret_cast<uintptr_t>(B->ptr) & 15) ||
      (A->ld % ld_mult) || (B->ld % ld_mult))
    return RG_ERR_ALIGNMENT;
  if (A->dtype == RG_F8E4M3 && (K & 1)) return RG_ERR_SHAPE;   // rows of 8-bit operands are whole byte pairs
  if (d->n_cuts && d->split_merge != 2) {                    // the in-cluster merge keeps the parts in shared memory
    if (!ws || ws_bytes < rg_gemm_workspace_bytes(d, M, N)) return RG_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 15) return RG_ERR_ALIGNMENT;
  }
  if (d->atom == RG_ATOM_SCALAR) return rg::launch_gemv(d, A, B, C, epi, static_cast<cudaStream_t>(cuda_stream));
  rg::GemmPlan plan;
  if ((s = make_plan(d, M, N, K, &plan)) != RG_OK) return s;
  return rg::launch_gemm(plan, A, B, C, epi, ws, static_cast<cudaStream_t>(cuda_stream));
}

static rg_status_t check_reduce(const rg_desc_t* d, rg_reduce_op_t op, const rg_tensor_t* x, const rg_tensor_t* out) {
  rg_status_t s = check_desc_fields(d);
  if (s != RG_OK) return s;
  if ((s = check_tensor(x)) != RG_OK || (s = check_tensor(out)) != RG_OK) return s;
  if (op != RG_OP_SUM && op != RG_OP_RMSNORM && op != RG_OP_SOFTMAX_DENOM) return RG_ERR_UNSUPPORTED;
  if (d->acc_dtype != RG_F32) return RG_ERR_UNSUPPORTED;
  if (x->dtype == RG_F16 || out->dtype == RG_F16) return RG_ERR_UNSUPPORTED;   // reductions read bf16 or fp32 rows
  if (x->cols < 1) return RG_ERR_SHAPE;
  if (out->rows != x->rows) return RG_ERR_SHAPE;
  if (op == RG_OP_RMSNORM) { if (out->cols != x->cols) return RG_ERR_SHAPE; }
  else if (out->cols != 1 || out->dtype != RG_F32) return RG_ERR_SHAPE;
  return RG_OK;
}

rg_status_t rg_reduce_rows(const rg_desc_t* d, rg_reduce_op_t op, const rg_tensor_t* x, const rg_tensor_t* out,
                           const rg_reduce_args_t* args, void* cuda_stream) {
  rg_status_t s = check_reduce(d, op, x, out);
  if (s != RG_OK) return s;
  if (args && args->weight && !dtype_ok(args->weight_dtype)) return RG_ERR_SHAPE;
  if (x->rows == 0) return RG_OK;
  // speed knobs reused for reductions: BN = threads per row, stages = warp-blocks per step
  return rg::launch_reduce_rows((int)op, d->tree, d->fma, x, out, args, d->BN, d->stages, static_cast<cudaStream_t>(cuda_stream));
}

size_t rg_reduce_cols_workspace_bytes(int64_t rows, int64_t cols) {
  if (rows <= 0 || cols <= 0) return 0;
  return rg::reduce_cols_workspace_bytes(rows, cols);
}

rg_status_t rg_reduce_cols(const rg_desc_t* d, rg_col_op_t op, const rg_tensor_t* x, const rg_tensor_t* y,
                           const rg_tensor_t* out, void* ws, size_t ws_bytes, void* cuda_stream) {
  rg_status_t s = check_desc_fields(d);
  if (s != RG_OK) return s;
  if ((s = check_tensor(x)) != RG_OK || (s = check_tensor(out)) != RG_OK) return s;
  if (op != RG_COLOP_SUM && op != RG_COLOP_DOT) return RG_ERR_UNSUPPORTED;
  if (d->acc_dtype != RG_F32) return RG_ERR_UNSUPPORTED;
  if (x->dtype == RG_F16) return RG_ERR_UNSUPPORTED;                       // leaves are bf16 or fp32
  if (op == RG_COLOP_DOT) {
    if ((s = check_tensor(y)) != RG_OK) return s;
    if (y->dtype != x->dtype || y->rows != x->rows || y->cols != x->cols) return RG_ERR_SHAPE;
  }
  if (x->rows < 1) return RG_ERR_SHAPE;
  if (out->rows != x->cols || out->cols != 1 || out->dtype != RG_F32) return RG_ERR_SHAPE;
  if (x->cols == 0) return RG_OK;
  const size_t need = d->tree == RG_TREE_LEFT ? 0 : rg_reduce_cols_workspace_bytes(x->rows, x->cols);   // a chain has no partial rows
  if (need) {
    if (!ws || ws_bytes < need) return RG_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(ws) & 15) return RG_ERR_ALIGNMENT;
  }
  return rg::launch_reduce_cols((int)op, d->tree, d->fma, x, op == RG_COLOP_DOT ? y : nullptr, out, ws, static_cast<cudaStream_t>(cuda_stream));
}

rg_status_t rg_attention(const rg_attn_desc_t* d, const rg_tensor_t* Q, const rg_tensor_t* K, const rg_tensor_t* Vt,
                         const rg_tensor_t* O, void* cuda_stream) {
  if (!d) return RG_ERR_NULL;
  if (d->size != sizeof(rg_attn_desc_t) || d->heads < 1 || d->sum_tree > RG_TREE_BALANCED || d->p_dtype > RG_F8E4M3)
    return RG_ERR_INVALID_DESC;
  rg_status_t s;
  if ((s = check_tensor(Q)) != RG_OK || (s = check_tensor(K)) != RG_OK || (s = check_tensor(Vt)) != RG_OK || (s = check_tensor(O)) != RG_OK)
    return s;
  if (d->mask > 1) return RG_ERR_INVALID_DESC;
  if (d->sum_tree != RG_TREE_BALANCED || d->p_dtype != RG_BF16 || d->div_place != 0) return RG_ERR_UNSUPPORTED;
  if (d->mask ? d->block_m != 128 : (d->block_m != 0 && d->block_m != 128)) return RG_ERR_UNSUPPORTED;
  if (d->block_n != 64 && d->block_n != 128) return RG_ERR_UNSUPPORTED;
  if (d->exp_base != 0 && d->exp_base != 2) return RG_ERR_INVALID_DESC;
  if (Q->dtype != RG_BF16 || K->dtype != RG_BF16 || Vt->dtype != RG_BF16) return RG_ERR_UNSUPPORTED;
  const int64_t hd = Q->cols, H = d->heads;
  if (hd != 64 && hd != 128) return RG_ERR_UNSUPPORTED;
  if (Q->rows % H || K->rows % H || K->cols != hd || Vt->rows != H * hd) return RG_ERR_SHAPE;
  const int64_t Nq = Q->rows / H, Nk = K->rows / H;
  if (Nk < 1 || Vt->cols != Nk || O->rows != Q->rows || O->cols != hd) return RG_ERR_SHAPE;
  if (Nq == 0) return RG_OK;
  if ((reinterpret_cast<uintptr_t>(Q->ptr) & 15) || (reinterpret_cast<uintptr_t>(K->ptr) & 15) ||
      (reinterpret_cast<uintptr_t>(Vt->ptr) & 15) || (reinterpret_cast<uintptr_t>(O->ptr) & 15) ||
      (Q->ld % 8) || (K->ld % 8) || (Vt->ld % 8) || (O->ld % 8))
    return RG_ERR_ALIGNMENT;
  return rg::launch_attention_fixed((int)d->block_n, (int)d->exp_base, (int)d->mask, d->scale, (int)H, Q, K, Vt, O, static_cast<cudaStream_t>(cuda_stream));
}

// ------------------------------------------------------------ host-buffer forms
size_t rg_gemm_host_scratch_bytes(const rg_desc_t* d, int64_t M, int64_t N, int64_t K, int32_t c_dtype,
                                  const rg_epilogue_t* epi) {
  if (M <= 0 || N <= 0 || K <= 0) return 0;
  const size_t ies = (d && d->in_dtype == RG_F8E4M3) ? 1 : 2;   // operand element size
  const int64_t per16 = 16 / (int64_t)ies;
  const int64_t ldk = (K + per16 - 1) / per16 * per16;
  size_t b = 0;
  b += align_up((size_t)M * ldk * ies, 256);
  b += align_up((size_t)N * ldk * ies, 256);
  b += align_up((size_t)M * N * esize(c_dtype), 256);
  if (epi && epi->bias) b += align_up((size_t)N * esize(epi->bias_dtype), 256);
  if (epi && epi->residual) b += align_up((size_t)M * N * esize(epi->residual_dtype), 256);
  b += align_up(rg_gemm_workspace_bytes(d, M, N), 256);
  return b;
}

rg_status_t rg_gemm_host(const rg_desc_t* d, const rg_tensor_t* A, const rg_tensor_t* B, const rg_tensor_t* C,
                         const rg_epilogue_t* epi, void* dev_scratch, size_t dev_scratch_bytes, void* cuda_stream) {
  rg_status_t s = check_desc_fields(d);
  if (s != RG_OK) return s;
  if ((s = check_gemm_shapes(A, B, C)) != RG_OK) return s;
  const int64_t M = A->rows, K = A->cols, N = B->rows;
  if (K < 1) return RG_ERR_SHAPE;
  if ((s = rg_desc_validate(d, M, N, K)) != RG_OK) return s;
  if ((s = check_epilogue(epi, N)) != RG_OK) return s;
  if (M == 0 || N == 0) return RG_OK;
  if (!dev_scratch || dev_scratch_bytes < rg_gemm_host_scratch_bytes(d, M, N, K, C->dtype, epi)) return RG_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(dev_scratch) & 255) return RG_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (A->dtype != d->in_dtype) return RG_ERR_SHAPE;
  const size_t ies = esize(A->dtype);
  const int64_t per16 = 16 / (int64_t)ies;
  const int64_t ldk = (K + per16 - 1) / per16 * per16;
  uint8_t* cur = static_cast<uint8_t*>(dev_scratch);
  auto take = [&](size_t bytes) { uint8_t* p = cur; cur += align_up(bytes, 256); return p; };
  rg_tensor_t dA{take((size_t)M * ldk * ies), A->dtype, M, K, ldk};
  rg_tensor_t dB{take((size_t)N * ldk * ies), B->dtype, N, K, ldk};
  rg_tensor_t dC{take((size_t)M * N * esize(C->dtype)), C->dtype, M, N, N};
  rg_epilogue_t de{};
  if (epi) de = *epi;
  bool ok = true;
  // rows that are already dense on both sides go as one flat copy
  auto h2d_rows = [&](void* dst, int64_t dst_ld, const void* src, int64_t src_ld, int64_t cols, int64_t rows, size_t es) {
    if (dst_ld == cols && src_ld == cols)
      return cudaMemcpyAsync(dst, src, (size_t)rows * cols * es, cudaMemcpyHostToDevice, st) == cudaSuccess;
    return cudaMemcpy2DAsync(dst, dst_ld * es, src, src_ld * es, cols * es, rows, cudaMemcpyHostToDevice, st) == cudaSuccess;
  };
  ok &= h2d_rows(dA.ptr, ldk, A->ptr, A->ld, K, M, ies);
  ok &= h2d_rows(dB.ptr, ldk, B->ptr, B->ld, K, N, ies);
  if (epi && epi->bias) {
    void* p = take((size_t)N * esize(epi->bias_dtype));
    ok &= cudaMemcpyAsync(p, epi->bias, (size_t)N * esize(epi->bias_dtype), cudaMemcpyHostToDevice, st) == cudaSuccess;
    de.bias = p;
  }
  if (epi && epi->residual) {
    const size_t es = esize(epi->residual_dtype);
    void* p = take((size_t)M * N * es);
    ok &= cudaMemcpy2DAsync(p, N * es, epi->residual, epi->ldr * es, N * es, M, cudaMemcpyHostToDevice, st) == cudaSuccess;
    de.residual = p; de.ldr = N;
  }
  if (!ok) return RG_ERR_CUDA;
  const size_t wsb = rg_gemm_workspace_bytes(d, M, N);
  void* ws = wsb ? take(wsb) : nullptr;
  if ((s = rg_gemm(d, &dA, &dB, &dC, epi ? &de : nullptr, ws, wsb, cuda_stream)) != RG_OK) return s;
  const size_t ces = esize(C->dtype);
  const cudaError_t ce = C->ld == N ? cudaMemcpyAsync(C->ptr, dC.ptr, (size_t)M * N * ces, cudaMemcpyDeviceToHost, st)
                                    : cudaMemcpy2DAsync(C->ptr, C->ld * ces, dC.ptr, N * ces, N * ces, M, cudaMemcpyDeviceToHost, st);
  if (ce != cudaSuccess) return RG_ERR_CUDA;
  return RG_OK;
}

// Where each piece of a host-buffer reduction lives in the caller's device scratch.  The size
// function and the call both go through this one routine, so they cannot disagree.  Every slot is
// reserved whether or not this call uses it (the size function does not see `args`): the row copy,
// the result, the RMSNorm weight (only that op reads one) and the per-row auxiliary output.
struct ReduceHostLayout { size_t x, out, weight, aux, total; int64_t ldx; };

static ReduceHostLayout reduce_host_layout(rg_reduce_op_t op, const rg_tensor_t* x, const rg_tensor_t* out) {
  ReduceHostLayout L{};
  L.ldx = (x->cols + 7) / 8 * 8;
  size_t cur = 0;
  auto take = [&](size_t bytes) { const size_t at = cur; cur += align_up(bytes, 256); return at; };
  L.x = take((size_t)x->rows * L.ldx * esize(x->dtype));
  L.out = take(op == RG_OP_RMSNORM ? (size_t)x->rows * L.ldx * esize(out->dtype) : (size_t)x->rows * 4);
  L.weight = take(op == RG_OP_RMSNORM ? (size_t)x->cols * 4 : 0);
  L.aux = take((size_t)x->rows * 4);
  L.total = cur;
  return L;
}

size_t rg_reduce_rows_host_scratch_bytes(rg_reduce_op_t op, const rg_tensor_t* x, const rg_tensor_t* out) {
  if (!x || !out || x->rows <= 0 || x->cols <= 0) return 0;
  return reduce_host_layout(op, x, out).total;
}

rg_status_t rg_reduce_rows_host(const rg_desc_t* d, rg_reduce_op_t op, const rg_tensor_t* x, const rg_tensor_t* out,
                                const rg_reduce_args_t* args, void* dev_scratch, size_t dev_scratch_bytes,
                                void* cuda_stream) {
  rg_status_t s = check_reduce(d, op, x, out);
  if (s != RG_OK) return s;
  if (args && args->weight && !dtype_ok(args->weight_dtype)) return RG_ERR_SHAPE;
  // only RMSNorm reads a weight; a weight handed to another op has no slot in the scratch layout
  if (args && args->weight && op != RG_OP_RMSNORM) return RG_ERR_UNSUPPORTED;
  if (x->rows == 0) return RG_OK;
  const ReduceHostLayout L = reduce_host_layout(op, x, out);
  if (!dev_scratch || dev_scratch_bytes < L.total) return RG_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(dev_scratch) & 255) return RG_ERR_ALIGNMENT;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const int64_t R = x->rows, Cc = x->cols, ldx = L.ldx;
  const size_t xes = esize(x->dtype), oes = esize(out->dtype);
  uint8_t* base = static_cast<uint8_t*>(dev_scratch);
  rg_tensor_t dx{base + L.x, x->dtype, R, Cc, ldx};
  rg_tensor_t dout;
  if (op == RG_OP_RMSNORM) dout = rg_tensor_t{base + L.out, out->dtype, R, Cc, ldx};
  else dout = rg_tensor_t{base + L.out, RG_F32, R, 1, 1};
  rg_reduce_args_t da{};
  if (args) da = *args;
  bool ok = cudaMemcpy2DAsync(dx.ptr, ldx * xes, x->ptr, x->ld * xes, Cc * xes, R, cudaMemcpyHostToDevice, st) == cudaSuccess;
  if (args && args->weight) {
    const size_t wes = esize(args->weight_dtype);
    void* p = base + L.weight;
    ok &= cudaMemcpyAsync(p, args->weight, (size_t)Cc * wes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    da.weight = p;
  }
  void* daux = (args && args->aux_out) ? base + L.aux : nullptr;
  da.aux_out = daux;
  if (!ok) return RG_ERR_CUDA;
  if ((s = rg_reduce_rows(d, op, &dx, &dout, &da, cuda_stream)) != RG_OK) return s;
  if (op == RG_OP_RMSNORM)
    ok = cudaMemcpy2DAsync(out->ptr, out->ld * oes, dout.ptr, ldx * oes, Cc * oes, R, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  else
    ok = cudaMemcpy2DAsync(out->ptr, out->ld * 4, dout.ptr, 4, 4, R, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  if (daux) ok &= cudaMemcpyAsync(args->aux_out, daux, (size_t)R * 4, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  return ok ? RG_OK : RG_ERR_CUDA;
}

rg_status_t rg_selftest_exp(int32_t form, const float* x, float* y, int64_t n, void* cuda_stream) {
  if (form < 0 || form > 7 || n < 0 || (form == 7 && n % 32 != 0)) return RG_ERR_SHAPE;
  if (n == 0) return RG_OK;
  if (!x || !y) return RG_ERR_NULL;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (form == 7) return rg::launch_silu_selftest(x, y, n, st);
  return (form >= 3 && form <= 5) ? rg::launch_exp_selftest_attention(form, x, y, n, st) : rg::launch_exp_selftest(form, x, y, n, st);
}

rg_status_t rg_selftest_bounded_wait(uint64_t limit_ns, uint32_t* dev_counter, void* cuda_stream) {
  if (!dev_counter) return RG_ERR_NULL;
  if (limit_ns < 1000ull || limit_ns > 100000000ull) return RG_ERR_SHAPE;     // 1 us .. 100 ms: never a long stall
  return rg::launch_wait_selftest(limit_ns, RG_SELFTEST_WAIT_CODE, dev_counter, static_cast<cudaStream_t>(cuda_stream));
}

rg_status_t rg_device_status(uint32_t* code) {
  uint32_t a = 0, b = 0, c = 0;
  const rg_status_t s1 = rg::read_and_clear_status(&a);          // synchronises the device
  if (s1 == RG_ERR_CUDA) return s1;
  const rg_status_t s2 = rg::read_and_clear_reduce_status(&b);
  if (s2 == RG_ERR_CUDA) return s2;
  const rg_status_t s3 = rg::read_and_clear_attn_status(&c);
  if (s3 == RG_ERR_CUDA) return s3;
  if (code) *code = a ? a : (b ? b : c);
  return (a || b || c) ? RG_ERR_TIMEOUT : RG_OK;
}

const char* rg_status_string(rg_status_t s) {
  switch (s) {
    case RG_OK: return "ok";
    case RG_ERR_NULL: return "a required pointer is null";
    case RG_ERR_INVALID_DESC: return "malformed descriptor";
    case RG_ERR_UNSUPPORTED: return "well-formed request that no kernel here realises";
    case RG_ERR_SHAPE: return "tensor shapes disagree or are out of range";
    case RG_ERR_ALIGNMENT: return "pointer or leading dimension breaks a 16-byte rule";
    case RG_ERR_WORKSPACE: return "workspace missing or too small";
    case RG_ERR_CUDA: return "CUDA runtime or driver error";
    case RG_ERR_TIMEOUT: return "a bounded device-side wait gave up";
  }
  return "unknown status";
}

}  // extern "C"
