// Entry points of the layer path: compress / decompress over the plan, layer forward and backward.
//
// Forward, per Algorithm 1 of the paper: gather + compress the boundary rows (step 2), put them in
// the receivers' halo slots decompressed (step 3), aggregate exact local rows and lossy remote
// rows, transform (Eq. (2)).  Backward mirrors it: transform gradients, transposed aggregation
// to local rows and halo slots, compress the slot gradients with the forward's key, return them
// to the owners and add (back-propagation across machines and through the compression routine,
// Algorithm 1, step 4).
#include <new>

#include "device_common.cuh"
#include "kernels.h"

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_matrix(const void *p, int64_t ld, int F, int V) {
  if (!p || !aligned16(p) || ld < F || (ld % V) != 0) return VARCO_INVALID_ARG;
  return VARCO_OK;
}

int check_desc(const varco_plan *pl, const varco_layer_desc_t *d) {
  if (!pl || !d) return VARCO_INVALID_ARG;
  if (d->dtype != VARCO_F32 && d->dtype != VARCO_BF16) return VARCO_INVALID_ARG;
  if ((int)d->conv != pl->conv) return VARCO_INVALID_ARG;
  if (d->F_in < 1 || d->F_out < 1) return VARCO_INVALID_ARG;
  if (d->F_in > 2048 || d->F_out > 2048) return VARCO_UNSUPPORTED;
  if (!pl->uploaded) return VARCO_NOT_UPLOADED;
  return VARCO_OK;
}

}  // namespace

size_t varco_gemm_scratch_bytes(int F_in, int F_out) {
  const size_t a = varco_simt_dw_scratch_bytes(F_in, F_out), b = varco_tc_scratch_bytes(F_in, F_out);
  return a > b ? a : b;
}

int varco_ws_arm_guards(char *ws, const varco_ws_layout &L, cudaStream_t st) {
#ifdef VARCO_DEBUG
  unsigned long long table[9] = {0};
  table[0] = (unsigned long long)L.num_guards;
  for (int g = 0; g < L.num_guards; ++g) {
    table[1 + g] = (unsigned long long)L.guard[g];
    VARCO_CUDA_CHECK(cudaMemsetAsync(ws + L.guard[g], 0xC5, 256, st));
  }
  // pageable source: the runtime stages the 72 bytes before the call returns
  VARCO_CUDA_CHECK(cudaMemcpyAsync(ws + 64, table, sizeof(table), cudaMemcpyHostToDevice, st));
#else
  (void)ws;
  (void)L;
  (void)st;
#endif
  return VARCO_OK;
}

static char *ws_base(void *workspace) {
  char *ws = static_cast<char *>(workspace);
  return ws + ((256 - (reinterpret_cast<uintptr_t>(ws) & 255u)) & 255u);
}

extern "C" {

int varco_compress(const varco_plan_t *plan, const void *X, int64_t ld, int32_t F, varco_dtype_t dtype,
                   varco_ratio_t c, varco_key_t key, void *packed, uint64_t *bytes, void *stream) {
  if (!plan || (dtype != VARCO_F32 && dtype != VARCO_BF16)) return VARCO_INVALID_ARG;
  const int V = dtype == VARCO_F32 ? 4 : 8;
  const int k = varco_kept_internal(F, c);
  if (k < 0) return VARCO_INVALID_ARG;
  if (F > 2048) return VARCO_UNSUPPORTED;
  if (check_matrix(X, ld, F, V) != VARCO_OK) return VARCO_INVALID_ARG;
  if (plan->H > 0 && k > 0 && !packed) return VARCO_INVALID_ARG;
  if (!plan->uploaded) return VARCO_NOT_UPLOADED;
  if (bytes) *bytes = (uint64_t)plan->H * (uint64_t)k * (dtype == VARCO_F32 ? 4u : 2u);
  if (k == 0) return VARCO_OK;   // no communication: nothing to pack
  StageTimer t(plan, VARCO_STAGE_COMPRESS, stream);
  return varco_launch_compress_rows(plan, X, ld, F, k, dtype, key, packed, k, 1, nullptr, 0, (cudaStream_t)stream);
}

int varco_decompress(const varco_plan_t *plan, const void *packed, int32_t F, varco_dtype_t dtype, varco_ratio_t c,
                     varco_key_t key, void *Xhalo, int64_t ld, void *stream) {
  if (!plan || (dtype != VARCO_F32 && dtype != VARCO_BF16)) return VARCO_INVALID_ARG;
  const int V = dtype == VARCO_F32 ? 4 : 8;
  const int k = varco_kept_internal(F, c);
  if (k < 0) return VARCO_INVALID_ARG;
  if (F > 2048) return VARCO_UNSUPPORTED;
  if (plan->H > 0 && ((k > 0 && !packed) || check_matrix(Xhalo, ld, F, V) != VARCO_OK)) return VARCO_INVALID_ARG;
  if (!plan->uploaded) return VARCO_NOT_UPLOADED;
  StageTimer t(plan, VARCO_STAGE_DECOMPRESS, stream);
  if (k == 0) {   // no communication: every halo row is the zero vector
    const size_t es = dtype == VARCO_F32 ? 4 : 2;
    if (plan->H > 0)
      VARCO_CUDA_CHECK(cudaMemset2DAsync(Xhalo, (size_t)ld * es, 0, (size_t)F * es, (size_t)plan->H, (cudaStream_t)stream));
    return VARCO_OK;
  }
  return varco_launch_decompress_slots(plan, packed, k, 1, F, k, dtype, key, Xhalo, ld, nullptr, 0,
                                       (cudaStream_t)stream);
}

int varco_layer_fwd(const varco_plan_t *plan, const varco_layer_desc_t *desc, const void *X, const void *W_self,
                    const void *W_neigh, const float *bias, void *Y, void *Agg_saved, varco_ratio_t c,
                    varco_key_t key, void *workspace, size_t ws_bytes, uint64_t *halo_bytes, void *stream) {
  int rc = check_desc(plan, desc);
  if (rc != VARCO_OK) return rc;
  const varco_dtype_t dt = desc->dtype;
  const int V = dt == VARCO_F32 ? 4 : 8;
  const size_t es = dt == VARCO_F32 ? 4 : 2;
  const int F_in = desc->F_in, F_out = desc->F_out;
  const int k = varco_kept_internal(F_in, c);
  if (k < 0) return VARCO_INVALID_ARG;
  if (check_matrix(X, desc->ld_in, F_in, V) || check_matrix(Agg_saved, desc->ld_in, F_in, V) ||
      check_matrix(Y, desc->ld_out, F_out, V))
    return VARCO_INVALID_ARG;
  if (!W_neigh || (desc->conv == VARCO_SAGE_MEAN && !W_self) || (desc->conv == VARCO_GCN && W_self))
    return VARCO_INVALID_ARG;
  if (!workspace || !aligned16(workspace)) return VARCO_INVALID_ARG;
  const varco_ws_layout L = varco_make_ws_layout(plan, F_in, F_out, dt);
  if (ws_bytes < L.total) return VARCO_WORKSPACE_TOO_SMALL;
  char *ws = ws_base(workspace);
  void *packed = ws + L.packed;
  void *Xhalo = ws + L.halo;
  // kept positions of this call's boundary rows: written by the sender-side kernel, read by the receivers
  uint16_t *wpos = reinterpret_cast<uint16_t *>(ws + L.wpos);
  int *status = reinterpret_cast<int *>(ws + L.status);
  cudaStream_t st = (cudaStream_t)stream;
  VARCO_CUDA_CHECK(cudaMemsetAsync(status, 0, 256, st));
  if (int grc = varco_ws_arm_guards(ws, L, st)) return grc;
  if (halo_bytes) *halo_bytes = (uint64_t)plan->H * (uint64_t)k * es;

  // Exchange.  The copy of a boundary row goes straight to the position of its halo slot at the
  // receiver, so "send buffer -> receive buffer" is folded into the write address.  At full
  // communication the row travels whole and in order: one gather-copy fills the halo slots.
  const int64_t kstride = round_up64(k, V);
  // rows of the position table are as long as this call's kept count needs (a multiple of 8 entries), not F_in:
  // at high ratios the table of all boundary rows then fits L2 and a 16-byte read of it costs one sector, not a line
  const int64_t wstride = round_up64(k > 0 ? k : 1, 8);
  // Compressed epochs with at most a quarter of a row kept: the receiver keeps (value, position)
  // pairs instead of rows that are mostly zeros, and the aggregation reads k pairs per remote
  // neighbour instead of F elements.
  const bool sparse = k > 0 && k < F_in && varco_spmm_sparse_supported(F_in, k, dt);
  if (k == 0) {
    // "no communication" (Section V): nothing is exchanged and every remote neighbour counts as the zero vector
  } else if (k == F_in) {
    StageTimer t(plan, VARCO_STAGE_COMPRESS, stream);
    rc = varco_launch_gather_copy(plan, X, desc->ld_in, F_in, dt, Xhalo, L.ld_in, st);
  } else {
    {
      StageTimer t(plan, VARCO_STAGE_COMPRESS, stream);
      rc = varco_launch_compress_rows(plan, X, desc->ld_in, F_in, k, dt, key, packed, kstride, 0, wpos, wstride, st);
    }
    if (rc != VARCO_OK) return rc;
    StageTimer t(plan, VARCO_STAGE_DECOMPRESS, stream);
    if (sparse)
      rc = varco_launch_expand_slots(plan, packed, kstride, k, dt, Xhalo, round_up64(k, 4), wpos, wstride, st);
    else
      rc = varco_launch_decompress_slots(plan, packed, kstride, 0, F_in, k, dt, key, Xhalo, L.ld_in, wpos, wstride,
                                         st);
  }
  if (rc != VARCO_OK) return rc;
  {
    StageTimer t(plan, VARCO_STAGE_SPMM, stream);
    if (k == 0)
      rc = varco_launch_spmm_fwd(plan, X, desc->ld_in, nullptr, 0, F_in, dt, Agg_saved, desc->ld_in, st);
    else if (sparse)
      rc = varco_launch_spmm_fwd_sparse(plan, X, desc->ld_in, Xhalo, round_up64(k, 4), k, F_in, dt, Agg_saved,
                                        desc->ld_in, st);
    else
      rc = varco_launch_spmm_fwd(plan, X, desc->ld_in, Xhalo, L.ld_in, F_in, dt, Agg_saved, desc->ld_in, st);
  }
  if (rc != VARCO_OK) return rc;
  {
    StageTimer t(plan, VARCO_STAGE_GEMM_FWD, stream);
    if (dt == VARCO_BF16 && F_out <= 256)
      rc = varco_tc_gemm_fwd((int)plan->n, F_in, F_out, X, desc->ld_in, Agg_saved, desc->ld_in, W_self, W_neigh, bias,
                             desc->relu, Y, desc->ld_out, ws + L.scratch, status, st);
    else
      rc = varco_simt_gemm_fwd((int)plan->n, F_in, F_out, dt, X, desc->ld_in, Agg_saved, desc->ld_in, W_self,
                               W_neigh, bias, desc->relu, Y, desc->ld_out, st);
  }
  return rc;
}

int varco_workspace_status(const void *workspace, void *stream, int *device_status) {
  if (!workspace || !device_status) return VARCO_INVALID_ARG;
  const char *ws = ws_base(const_cast<void *>(workspace));
  int v = 0;
  VARCO_CUDA_CHECK(cudaMemcpyAsync(&v, ws, sizeof(int), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
  VARCO_CUDA_CHECK(cudaStreamSynchronize((cudaStream_t)stream));
#ifdef VARCO_DEBUG
  // guard table of the last layer call: [count, offsets...] at byte 64 of the status block; a damaged guard
  // block (some kernel wrote past its segment) sets bit 30 of the status
  unsigned long long table[9] = {0};
  VARCO_CUDA_CHECK(cudaMemcpy(table, ws + 64, sizeof(table), cudaMemcpyDeviceToHost));
  for (unsigned long long g = 0; g < table[0] && g < 8; ++g) {
    unsigned char block[256];
    VARCO_CUDA_CHECK(cudaMemcpy(block, ws + table[1 + g], sizeof(block), cudaMemcpyDeviceToHost));
    for (unsigned char b : block)
      if (b != 0xC5) v |= 1 << 30;
  }
#endif
  *device_status = v;
  return VARCO_OK;
}


int varco_layer_bwd(const varco_plan_t *plan, const varco_layer_desc_t *desc, const void *X, const void *Y,
                    const void *Agg_saved, const void *W_self, const void *W_neigh, const void *dY, void *dX,
                    float *dW_self, float *dW_neigh, float *dbias, varco_ratio_t c, varco_key_t key, void *workspace,
                    size_t ws_bytes, uint64_t *halo_bytes, void *stream) {
  int rc = check_desc(plan, desc);
  if (rc != VARCO_OK) return rc;
  const varco_dtype_t dt = desc->dtype;
  const int V = dt == VARCO_F32 ? 4 : 8;
  const size_t es = dt == VARCO_F32 ? 4 : 2;
  const int F_in = desc->F_in, F_out = desc->F_out;
  const int n = (int)plan->n;
  const bool sage = desc->conv == VARCO_SAGE_MEAN;
  const int k = varco_kept_internal(F_in, c);
  if (k < 0) return VARCO_INVALID_ARG;
  if (check_matrix(X, desc->ld_in, F_in, V) || check_matrix(Agg_saved, desc->ld_in, F_in, V) ||
      check_matrix(dX, desc->ld_in, F_in, V) || check_matrix(dY, desc->ld_out, F_out, V))
    return VARCO_INVALID_ARG;
  if (desc->relu && check_matrix(Y, desc->ld_out, F_out, V)) return VARCO_INVALID_ARG;
  if (!W_neigh || !dW_neigh || (sage && (!W_self || !dW_self)) || (!sage && (W_self || dW_self)))
    return VARCO_INVALID_ARG;
  if (!workspace || !aligned16(workspace)) return VARCO_INVALID_ARG;
  const varco_ws_layout L = varco_make_ws_layout(plan, F_in, F_out, dt);
  if (ws_bytes < L.total) return VARCO_WORKSPACE_TOO_SMALL;
  char *ws = ws_base(workspace);
  int *status = reinterpret_cast<int *>(ws + L.status);
  VARCO_CUDA_CHECK(cudaMemsetAsync(status, 0, 256, (cudaStream_t)stream));
  if (int grc = varco_ws_arm_guards(ws, L, (cudaStream_t)stream)) return grc;
  const bool tc = dt == VARCO_BF16 && F_out <= 256 && (sage ? 2 : 1) * ((F_in + 127) / 128) <= 8;
  void *packed = ws + L.packed;
  void *Ghalo = ws + L.halo;
  void *dZbuf = ws + L.dZ;
  void *dAgg = ws + L.dAgg;
  float *scratch = reinterpret_cast<float *>(ws + L.scratch);
  cudaStream_t st = (cudaStream_t)stream;
  if (halo_bytes) *halo_bytes = (uint64_t)plan->H * (uint64_t)k * es;

  const void *dZ = dY;
  int64_t lddz = desc->ld_out;
  bool bias_done = false;
  if (desc->relu) {
    // the mask and, when asked for, the bias gradient (column sums of the masked rows) in one pass
    StageTimer t(plan, VARCO_STAGE_AUX, stream);
    if (dbias) {
      rc = varco_relu_mask_colsum(n, F_out, dt, Y, desc->ld_out, dY, desc->ld_out, dZbuf, L.ld_out, dbias, scratch, st);
      bias_done = true;
    } else {
      rc = varco_relu_mask(n, F_out, dt, Y, desc->ld_out, dY, desc->ld_out, dZbuf, L.ld_out, st);
    }
    if (rc != VARCO_OK) return rc;
    dZ = dZbuf;
    lddz = L.ld_out;
  }
  {
    StageTimer t(plan, VARCO_STAGE_GEMM_DW, stream);
    if (tc) {
      rc = varco_tc_gemm_dw(n, F_in, F_out, X, desc->ld_in, Agg_saved, desc->ld_in, dZ, lddz, dW_self, dW_neigh,
                            scratch, status, st);
    } else {
      rc = varco_simt_gemm_dw(n, F_in, F_out, dt, Agg_saved, desc->ld_in, dZ, lddz, dW_neigh, scratch, st);
      if (rc == VARCO_OK && sage)
        rc = varco_simt_gemm_dw(n, F_in, F_out, dt, X, desc->ld_in, dZ, lddz, dW_self, scratch, st);
    }
    if (rc == VARCO_OK && dbias && !bias_done) rc = varco_colsum(n, F_out, dt, dZ, lddz, dbias, scratch, st);
  }
  if (rc != VARCO_OK) return rc;
  // Narrow backward (F_out well below F_in, tensor-core path): aggregation and the weight product commute,
  // so the transposed aggregation runs on the F_out-wide dZ instead of the F_in-wide dZ W_neigh^T, and the
  // product with W_neigh^T is applied afterwards to the local sums and to the slot sums.  The slot gradient
  // rows come out of that product densely; with k < F their kept values are selected from them.
  const bool narrow = tc && 2 * L.ld_out <= F_in;
  uint16_t *wpos = reinterpret_cast<uint16_t *>(ws + L.wpos);
  const int64_t kstride = round_up64(k, V);
  // rows of the position table are as long as this call's kept count needs (a multiple of 8 entries), not F_in:
  // at high ratios the table of all boundary rows then fits L2 and a 16-byte read of it costs one sector, not a line
  const int64_t wstride = round_up64(k > 0 ? k : 1, 8);
  if (k > 0 && k < F_in) {
    // the kept positions of every unique boundary row are evaluated once, then used by the compression of
    // the slot gradients and by the owners' add
    StageTimer t(plan, VARCO_STAGE_COMPRESS_BWD, stream);
    rc = varco_launch_wire_positions(plan, F_in, k, key, wpos, wstride, st);
    if (rc != VARCO_OK) return rc;
  }
  if (narrow) {
    const bool kept_product = k > 0 && k < F_in && varco_slot_kept_product_supported(F_in, F_out, k, dt);
    void *Gl = dAgg;      // [n x ld_out] local sums of dZ
    void *Gh = k > 0 ? packed : nullptr;    // [H x ld_out] slot sums of dZ (dead once the slot rows exist)
    {
      StageTimer t(plan, VARCO_STAGE_SPMM_T, stream);
      rc = varco_launch_spmm_bwd(plan, dZ, lddz, F_out, dt, Gl, L.ld_out, 0, Gh, L.ld_out, nullptr, 0, 0, key, nullptr, 0,
                                 st);
    }
    if (rc != VARCO_OK) return rc;
    {
      StageTimer t(plan, VARCO_STAGE_GEMM_DX, stream);
      if (sage)
        rc = varco_tc_gemm_cat_t(n, F_in, F_out, dZ, lddz, Gl, L.ld_out, W_self, W_neigh, dX, desc->ld_in, scratch,
                                 status, st);
      else
        rc = varco_tc_gemm_cat_t(n, F_in, F_out, Gl, L.ld_out, nullptr, 0, W_neigh, nullptr, dX, desc->ld_in, scratch,
                                 status, st);
      if (rc == VARCO_OK && plan->H > 0 && k > 0 && !kept_product)
        rc = varco_tc_gemm_cat_t((int)plan->H, F_in, F_out, Gh, L.ld_out, nullptr, 0, W_neigh, nullptr, Ghalo, L.ld_in,
                                 scratch, status, st);
    }
    if (rc != VARCO_OK || k == 0) return rc;   // no communication: no gradient crosses a partition boundary
    if (kept_product) {
      // few kept entries: each one is a dot product with one row of W_neigh; the F_in-wide rows never exist
      {
        StageTimer t(plan, VARCO_STAGE_COMPRESS_BWD, stream);
        rc = varco_launch_slot_kept_product(plan, Gh, L.ld_out, F_out, W_neigh, F_in, k, Ghalo, kstride, wpos, wstride,
                                            st);
      }
      if (rc != VARCO_OK) return rc;
      StageTimer t(plan, VARCO_STAGE_SCATTER_ADD, stream);
      return varco_launch_scatter_add_rows(plan, Ghalo, kstride, F_in, k, dt, dX, desc->ld_in, wpos, wstride, st);
    }
    if (k == F_in) {
      StageTimer t(plan, VARCO_STAGE_SCATTER_ADD, stream);
      return varco_launch_add_dense_rows(plan, Ghalo, L.ld_in, F_in, dt, dX, desc->ld_in, st);
    }
    {
      StageTimer t(plan, VARCO_STAGE_COMPRESS_BWD, stream);
      rc = varco_launch_select_slots(plan, Ghalo, L.ld_in, F_in, k, dt, packed, kstride, wpos, wstride, st);
    }
    if (rc != VARCO_OK) return rc;
    StageTimer t(plan, VARCO_STAGE_SCATTER_ADD, stream);
    return varco_launch_scatter_add_rows(plan, packed, kstride, F_in, k, dt, dX, desc->ld_in, wpos, wstride, st);
  }
  {
    StageTimer t(plan, VARCO_STAGE_GEMM_DX, stream);
    if (tc) {
      rc = varco_tc_gemm_dx(n, F_in, F_out, dZ, lddz, W_self, W_neigh, dX, desc->ld_in, dAgg, L.ld_in, scratch, status,
                            st);
    } else {
      rc = varco_simt_gemm_dx(n, F_in, F_out, dt, dZ, lddz, W_neigh, dAgg, L.ld_in, st);
      if (rc == VARCO_OK && sage) rc = varco_simt_gemm_dx(n, F_in, F_out, dt, dZ, lddz, W_self, dX, desc->ld_in, st);
    }
  }
  if (rc != VARCO_OK) return rc;
  {
    StageTimer t(plan, VARCO_STAGE_SPMM_T, stream);
    // k < F: the slot gradients are compressed in the epilogue (no dense slot rows)
    rc = varco_launch_spmm_bwd(plan, dAgg, L.ld_in, F_in, dt, dX, desc->ld_in, sage ? 1 : 0, k > 0 ? Ghalo : nullptr,
                               L.ld_in, (k > 0 && k < F_in) ? packed : nullptr, kstride, k, key, wpos, wstride, st);
  }
  if (rc != VARCO_OK || k == 0) return rc;   // no communication: no gradient crosses a partition boundary
  // Return of the halo-slot gradients to the owners.  At full communication the slot rows are
  // the messages; otherwise they are compressed with the forward's key first.
  if (k == F_in) {
    StageTimer t(plan, VARCO_STAGE_SCATTER_ADD, stream);
    return varco_launch_add_dense_rows(plan, Ghalo, L.ld_in, F_in, dt, dX, desc->ld_in, st);
  }
  {
    StageTimer t(plan, VARCO_STAGE_SCATTER_ADD, stream);
    rc = varco_launch_scatter_add_rows(plan, packed, kstride, F_in, k, dt, dX, desc->ld_in, wpos, wstride, st);
  }
  return rc;
}

}  // extern "C"
