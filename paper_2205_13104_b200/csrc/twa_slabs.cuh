// Row slabs of the per-column stepping calls (twa_api.cu, twa_project_batch.cu).
#pragma once

#include "twa_common.cuh"

namespace {

// A basis of more than TWA_MAX_LAUNCH_ROWS rows (or of more than TWA_TUNE_SLAB_ROWS, where that is set) is
// walked in slabs: the kernels index rows with 32-bit integers, the projection is a sum over row
// ranges and the lift is independent per row.  One launch takes up to TWA_MAX_LAUNCH_ROWS: the kernels
// round row numbers up to whole tiles (at most 4096 rows) in 32-bit integers, and the margin below
// 2^31 keeps those sums from wrapping.
constexpr long long TWA_SLAB_ROWS = 1LL << 30;
static_assert(TWA_MAX_ROWS == TWA_SLAB_ROWS * TWA_HOST_CHUNKS, "one slot of per-slab coefficients in ws per slab");

struct SlabPlan {
  long long rows;    // rows per slab: whole 512-byte segments at every storage width
  int count;         // 1: the whole basis in one launch
};

SlabPlan slab_plan(const twa_ctx* ctx, long long D) {
  const long long one = ctx->tune_slab_rows ? ctx->tune_slab_rows : TWA_MAX_LAUNCH_ROWS;
  if (D <= one) return {D, 1};
  const long long rows = ctx->tune_slab_rows ? ctx->tune_slab_rows : TWA_SLAB_ROWS;
  return {rows, static_cast<int>((D + rows - 1) / rows)};
}

// Rows [k * plan.rows, ...) of P as a basis of its own.
twa_basis slab_view(const twa_basis* P, const SlabPlan& plan, int k, long long* r0) {
  *r0 = static_cast<long long>(k) * plan.rows;
  twa_basis v = *P;
  v.data = static_cast<char*>(P->data) + (*r0 * P->bits) / 8;
  v.D = (*r0 + plan.rows < P->D) ? plan.rows : P->D - *r0;
  return v;
}

// twa_check_basis with the row limit of the slab-walking calls instead of the kernels' own.
int check_basis_slabbed(const twa_ctx* ctx, const twa_basis* P) {
  if (!P) return TWA_ERR_INVALID_ARG;
  if (P->D > TWA_MAX_ROWS) return TWA_ERR_INVALID_ARG;
  if (slab_plan(ctx, P->D).count > TWA_HOST_CHUNKS) return TWA_ERR_INVALID_ARG;
  if (P->D <= TWA_MAX_LAUNCH_ROWS) return twa_check_basis(P);
  twa_basis head = *P;
  head.D = TWA_SLAB_ROWS;
  int rc = twa_check_basis(&head);
  if (rc) return rc;
  return P->col_stride < (P->D * P->bits + 7) / 8 ? TWA_ERR_INVALID_ARG : TWA_OK;
}

}  // namespace
