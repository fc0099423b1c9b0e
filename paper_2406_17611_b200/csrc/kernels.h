// Launchers of the kernels behind the C ABI (internal).
#ifndef VARCO_KERNELS_H_
#define VARCO_KERNELS_H_

#include <cuda_runtime.h>

#include "varco_internal.h"

// workspace carving shared by varco_workspace_bytes and the layer entry points
struct varco_ws_layout {
  int64_t ld_in = 0, ld_out = 0;  // leading dimensions of the internal buffers
  int64_t wstride = 0;            // row stride of the kept-position table (16-bit entries)
  size_t status = 0, packed = 0, halo = 0, wpos = 0, dZ = 0, dAgg = 0, scratch = 0, scratch_bytes = 0, total = 0;
  // debug build: offsets of the 256-byte guard blocks behind the segments (filled with a pattern by every layer
  // call, verified by varco_workspace_status)
  size_t guard[8] = {0, 0, 0, 0, 0, 0, 0, 0};
  int num_guards = 0;
};
// debug build: write the guard pattern / the guard table of a layer call (no-ops in a release build)
int varco_ws_arm_guards(char *ws_base, const varco_ws_layout &L, cudaStream_t st);
varco_ws_layout varco_make_ws_layout(const varco_plan *pl, int F_in, int F_out, varco_dtype_t dt);
size_t varco_gemm_scratch_bytes(int F_in, int F_out);

// halo.cu
int varco_launch_gather_copy(const varco_plan *pl, const void *X, int64_t ld, int F, varco_dtype_t dt, void *Xhalo,
                             int64_t ldh, cudaStream_t st);
int varco_launch_compress_rows(const varco_plan *pl, const void *X, int64_t ld, int F, int k, varco_dtype_t dt,
                               varco_key_t key, void *packed, int64_t kstride, int send_order, uint16_t *wpos,
                               int64_t wstride, cudaStream_t st);
int varco_launch_decompress_slots(const varco_plan *pl, const void *packed, int64_t kstride, int send_order, int F,
                                  int k, varco_dtype_t dt, varco_key_t key, void *Xhalo, int64_t ld, const uint16_t *wpos,
                                  int64_t wstride, cudaStream_t st);
int varco_launch_expand_slots(const varco_plan *pl, const void *packed, int64_t kstride, int k, varco_dtype_t dt,
                              void *pairs, int64_t pstride, const uint16_t *wpos, int64_t wstride, cudaStream_t st);
int varco_launch_scatter_add_rows(const varco_plan *pl, const void *packed, int64_t kstride, int F, int k,
                                  varco_dtype_t dt, void *dX, int64_t ld, const uint16_t *wpos, int64_t wstride,
                                  cudaStream_t st);
int varco_launch_wire_positions(const varco_plan *pl, int F, int k, varco_key_t key, uint16_t *wpos, int64_t wstride,
                                cudaStream_t st);
int varco_launch_select_slots(const varco_plan *pl, const void *Gh, int64_t ldg, int F, int k, varco_dtype_t dt,
                              void *packed, int64_t kstride, const uint16_t *wpos, int64_t wstride, cudaStream_t st);
bool varco_slot_kept_product_supported(int F_in, int F_out, int k, varco_dtype_t dt);
int varco_launch_slot_kept_product(const varco_plan *pl, const void *Gh, int64_t ldg, int F_out, const void *W_neigh,
                                   int F_in, int k, void *packed, int64_t kstride, const uint16_t *wpos,
                                   int64_t wstride, cudaStream_t st);
int varco_launch_add_dense_rows(const varco_plan *pl, const void *Gh, int64_t ldg, int F, varco_dtype_t dt, void *dX,
                                int64_t ld, cudaStream_t st);
// spmm.cu
int varco_debug_word_spmm();   // debug build: first failed index check of the aggregation kernels (else 0)
int varco_launch_spmm_fwd(const varco_plan *pl, const void *X, int64_t ldx, const void *Xhalo, int64_t ldh, int F,
                          varco_dtype_t dt, void *Agg, int64_t ldagg, cudaStream_t st);
int varco_launch_spmm_bwd(const varco_plan *pl, const void *dAgg, int64_t ldd, int F, varco_dtype_t dt, void *dX,
                          int64_t ldx, int accumulate, void *Ghalo, int64_t ldh, void *packed, int64_t kstride, int k,
                          varco_key_t key, const uint16_t *wpos, int64_t wstride, cudaStream_t st);
int varco_launch_spmm_fwd_sparse(const varco_plan *pl, const void *X, int64_t ldx, const void *pairs, int64_t pstride,
                                 int k, int F, varco_dtype_t dt, void *Agg, int64_t ldagg, cudaStream_t st);
bool varco_spmm_sparse_supported(int F, int k, varco_dtype_t dt);
// gemm_simt.cu
size_t varco_simt_dw_scratch_bytes(int F_in, int F_out);
int varco_simt_gemm_fwd(int n, int F_in, int F_out, varco_dtype_t dt, const void *X, int64_t ldx, const void *Agg,
                        int64_t lda, const void *Ws, const void *Wn, const float *bias, int relu, void *Y,
                        int64_t ldy, cudaStream_t st);
int varco_simt_gemm_dx(int n, int F_in, int F_out, varco_dtype_t dt, const void *dZ, int64_t lddz, const void *W,
                       void *out, int64_t ldo, cudaStream_t st);
int varco_simt_gemm_dw(int n, int F_in, int F_out, varco_dtype_t dt, const void *A, int64_t lda, const void *dZ,
                       int64_t lddz, float *dW, float *scratch, cudaStream_t st);
int varco_colsum(int n, int F_out, varco_dtype_t dt, const void *dZ, int64_t lddz, float *out, float *scratch,
                 cudaStream_t st);
int varco_relu_mask_colsum(int n, int F_out, varco_dtype_t dt, const void *Y, int64_t ldy, const void *dY, int64_t lddy,
                           void *dZ, int64_t lddz, float *out, float *scratch, cudaStream_t st);
int varco_relu_mask(int n, int F_out, varco_dtype_t dt, const void *Y, int64_t ldy, const void *dY, int64_t lddy,
                    void *dZ, int64_t lddz, cudaStream_t st);

// gemm_tc.cu (bf16, tcgen05)
size_t varco_tc_scratch_bytes(int F_in, int F_out);
int varco_tc_gemm_fwd(int n, int F_in, int F_out, const void *X, int64_t ldx, const void *Agg, int64_t lda,
                      const void *Ws, const void *Wn, const float *bias, int relu, void *Y, int64_t ldy,
                      void *scratch, int *err, cudaStream_t st);
int varco_tc_gemm_dx(int n, int F_in, int F_out, const void *dZ, int64_t lddz, const void *Ws, const void *Wn,
                     void *dXs, int64_t ldxs, void *dAgg, int64_t ldagg, void *scratch, int *err, cudaStream_t st);
int varco_tc_gemm_cat_t(int m, int F_in, int F_out, const void *A0, int64_t lda0, const void *A1, int64_t lda1,
                        const void *W0, const void *W1, void *out, int64_t ldo, void *scratch, int *err,
                        cudaStream_t st);
int varco_tc_gemm_dw(int n, int F_in, int F_out, const void *X, int64_t ldx, const void *Agg, int64_t lda,
                     const void *dZ, int64_t lddz, float *dWs, float *dWn, void *scratch, int *err, cudaStream_t st);

#endif  // VARCO_KERNELS_H_
