/*
 * varco.h -- C ABI of the VARCO partitioned graph-convolution layer for NVIDIA B200 (sm_100a).
 *
 * The method is the one of "Distributed Training of Large Graph Neural Networks with Variable
 * Communication Rates": a graph is split into P partitions (Section III); at every layer each
 * partition compresses the activations of its boundary ("halo") rows at the current compression
 * ratio, sends them to the partitions that aggregate from them, the receivers decompress and
 * aggregate exact local rows plus lossy remote rows (Algorithm 1, Definition 1, appendix
 * "Compression Mechanism"); the backward pass sends the halo-row gradients back through the same
 * compressor (Algorithm 1, Section III-A).  Here the P partitions live side by side in the memory
 * of ONE GPU: "communication" is a device-side gather into packed send buffers and a scatter into
 * receive buffers, and the bytes that would cross the network are counted exactly.
 *
 * Conventions
 *   - Every function returns an int status: 0 = VARCO_OK, negative = error (see below).  Nothing
 *     throws, aborts or traps.  varco_status_string() names a status.
 *   - "host" pointers are ordinary CPU memory; "device" pointers are CUDA global memory of the
 *     current device, allocated and owned by the caller.  The library allocates no device memory
 *     on the layer path: scratch comes from the caller-provided workspace.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Kernels are enqueued
 *     on it and the call returns without synchronising, unless stated otherwise.
 *   - Row-major matrices with a leading dimension `ld` counted in ELEMENTS.  Every activation
 *     matrix must have its base pointer 16-byte aligned and ld * element_size a multiple of 16
 *     (ld % 4 == 0 for fp32, ld % 8 == 0 for bf16), ld >= F.  Padding columns [F, ld) are never read
 *     as data and are never counted as communicated bytes; in outputs they are either left
 *     untouched or written as zero.
 *   - Rows of X, Y, Agg, dY, dX are in the plan's partition-contiguous order: all rows of
 *     partition 0 (ascending original id), then partition 1, ... (varco_partition_perm).
 *   - Outputs must not alias inputs.  Byte counters are host values computed exactly from the
 *     plan's counts; they need no synchronisation.
 */
#ifndef VARCO_H_
#define VARCO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  VARCO_OK = 0,
  VARCO_INVALID_ARG = -1,        /* NULL pointer, bad size, bad alignment, bad enum, ratio < 1 */
  VARCO_BAD_GRAPH = -2,          /* row_ptr not monotone from 0, column out of range, unsorted or
                                    duplicate columns in a row, or a diagonal entry */
  VARCO_BAD_PARTITION = -3,      /* a label outside [0, P) */
  VARCO_NOMEM = -4,              /* host allocation failed */
  VARCO_CUDA = -5,               /* a CUDA runtime call failed (no device, launch error, ...) */
  VARCO_WORKSPACE_TOO_SMALL = -6,
  VARCO_UNSUPPORTED = -7,        /* valid request outside what the kernels cover (e.g. F > 2048) */
  VARCO_NOT_UPLOADED = -8        /* a device entry point was called before varco_partition_upload */
};

typedef struct varco_plan varco_plan_t;
typedef enum { VARCO_F32 = 0, VARCO_BF16 = 1 } varco_dtype_t;
typedef enum { VARCO_GCN = 0, VARCO_SAGE_MEAN = 1 } varco_conv_t;

/* Compression ratio c = num/den >= 1 as an exact rational (the scheduler produces non-integers). */
typedef struct { uint32_t num, den; } varco_ratio_t;

/* The shared random key of the appendix "Compression Mechanism": encoder and decoder derive the
 * positions of the values that are sent from (seed, epoch, layer, global node id); no index is
 * ever transmitted. */
typedef struct { uint64_t seed; uint32_t epoch, layer; } varco_key_t;

const char *varco_status_string(int status);

/* ------------------------------------------------------------------------------------------
 * Plan: partition and halo structure (Section III: every worker holds the nodes of one partition;
 * the boundary nodes of that section are the halo rows).
 *
 * varco_partition_build
 *   n, row_ptr[n+1], col_idx[nnz]  host CSR adjacency: row i lists the nodes j that i aggregates
 *                                  from.  Columns strictly ascending inside a row, no diagonal
 *                                  entries (GCN adds its self-loop itself).  Need not be symmetric.
 *   part[n]                        host partition label of every node, in [0, P).
 *   conv                           VARCO_SAGE_MEAN: s_ij = 1/deg(i) (0 for an isolated node);
 *                                  VARCO_GCN: s_ij = 1/sqrt((deg(i)+1)(deg(j)+1)), self-loop
 *                                  included.  Degrees are those of the WHOLE graph.
 *   out                            receives a plan that owns only host memory; free it with
 *                                  varco_partition_destroy.
 *   Canonical orders: rows of a partition by ascending original id; the halo slots of partition q
 *   (rows it receives) by (owner partition p ascending, original id ascending); the send segments
 *   of partition p by (destination q ascending, original id ascending).
 *   halo(p->q) = { j owned by p : some i owned by q has an entry (i, j) }, p != q.
 *   Errors: INVALID_ARG, BAD_GRAPH, BAD_PARTITION, NOMEM, UNSUPPORTED (n or n + H_total beyond
 *   2^31 - 1: rows and halo slots share one 32-bit index space; the number of stored entries is
 *   not limited, entry offsets are 64-bit).
 *   Inputs of the layer entry points must be finite: the weighted aggregation kernels pad their
 *   gather batches with zero-weight copies of a real source row, and 0 * Inf is NaN.
 */
int varco_partition_build(int64_t n, const int64_t *row_ptr, const int32_t *col_idx,
                          const int32_t *part, int32_t P, varco_conv_t conv, varco_plan_t **out);
int varco_partition_destroy(varco_plan_t *plan);

/* Counters of the plan.  Any output pointer may be NULL.
 *   H_total        number of (row, destination partition) copies per exchange = sum |halo(p->q)|
 *   cross_entries  stored entries (i, j) with part(i) != part(j); self_entries the others. */
int varco_partition_info(const varco_plan_t *plan, int64_t *n, int64_t *nnz, int32_t *P,
                         int64_t *H_total, int64_t *cross_entries, int64_t *self_entries);
/* Number of distinct rows that are a halo row of at least one other partition. */
int varco_partition_boundary_rows(const varco_plan_t *plan, int64_t *count);
/* Tuning knob (no counterpart in the paper), off by default.  With bytes > 0 the forward aggregation splits the
 * feature row into panels so that the rows one partition gathers from (its own plus its halo slots) fit in
 * `bytes` of L2.  On B200 this did not pay on the measured workloads; results are unchanged either way. */
int varco_partition_set_l2_budget(varco_plan_t *plan, int64_t bytes);
/* Analysis aid (no counterpart in the paper): what the aggregation's row gathers cost under a simple cache model.
 * The aggregation of a partition reads one source row per stored entry, at random; a source used several times
 * inside the partition is read from memory once only if it stays cached in between.  The model keeps the
 * `resident_rows` most used sources of every partition cached (read once each) and reads every other source once
 * per use.  transposed = 0: forward structure (sources = the partition's rows and halo slots); 1: transposed
 * structure (sources = the partition's rows of the upstream gradient).  Outputs (any may be NULL), summed over
 * the partitions: entries = row gathers issued, sources = distinct rows gathered (the traffic of an unbounded
 * cache), rows_read = rows read from memory under the model.  Multiply by the row size for bytes. */
int varco_partition_gather_model(const varco_plan_t *plan, int32_t transposed, int64_t resident_rows,
                                 int64_t *entries, int64_t *sources, int64_t *rows_read);
/* PxP[p * P + q] = |halo(p->q)| (host array of P*P entries). */
int varco_partition_counts(const varco_plan_t *plan, int64_t *PxP);
/* Original ids of halo(p->q), ascending; the pointer stays valid until the plan is destroyed. */
int varco_partition_halo(const varco_plan_t *plan, int32_t p, int32_t q,
                         const int64_t **global_ids, int64_t *count);
/* new_to_old[r] = original id of row r of the partition-contiguous order (n entries, plan-owned). */
int varco_partition_perm(const varco_plan_t *plan, const int64_t **new_to_old);

/* Device image of the plan (index arrays only).  The caller allocates `bytes` of device memory
 * (256-byte aligned), keeps it alive as long as the plan is used, and frees it afterwards.
 * The copy is enqueued on `stream` from plan-owned host memory and the call synchronises that
 * stream before returning.  Errors: INVALID_ARG, WORKSPACE_TOO_SMALL, CUDA. */
int varco_partition_device_bytes(const varco_plan_t *plan, size_t *bytes);
int varco_partition_upload(varco_plan_t *plan, void *dev_buf, size_t bytes, void *stream);

/* Scratch bytes that varco_layer_fwd / varco_layer_bwd / varco_compress need for layers with
 * F_in <= F_in_max and F_out <= F_out_max of the given dtype. */
int varco_workspace_bytes(const varco_plan_t *plan, int32_t F_in_max, int32_t F_out_max,
                          varco_dtype_t dtype, size_t *bytes);

/* ------------------------------------------------------------------------------------------
 * Rate helpers (host, integer-exact).
 *
 * varco_kept: number of values of an F-vector that are sent at ratio c (Definition 1: the
 *   compressed signal has F/c entries; appendix "Compression Mechanism").  For non-integer F/c:
 *   k = ceil(F * den / num), clamped to [1, F].  INVALID_ARG if F < 1 or c < 1.
 * varco_schedule_linear: the scheduler of the appendix "Scheduler" (and r_lin of Section IV),
 *   c_e = max(c_max - a (c_max - c_min) e / K, c_min) for epoch e >= 0, returned as the exact
 *   rational {num = max(c_max K - a (c_max - c_min) e, c_min K), den = K}.  The printed formula
 *   clips with "min"; it is read as a lower clip at c_min, which is the only reading that starts
 *   at c_max and ends at full communication.  INVALID_ARG on K < 1, a < 1, c_min < 1,
 *   c_max < c_min, e < 0, or num beyond 32 bits.
 */
int varco_kept(int32_t F, varco_ratio_t c, int32_t *k);
int varco_schedule_linear(int32_t epoch, int32_t K, int32_t slope_a, int32_t c_max, int32_t c_min,
                          varco_ratio_t *c);

/* The other schedulers of the appendix "Scheduler".  There r_k is the communicated fraction ("compress rate",
 * raised while training) and the compressor is handed c_k = 1 / r_k.
 *   varco_schedule_rate_linear   r_k = (alpha k + r0) / den clipped at 1 (full communication); the fixed
 *                                increment r_{k+1} = r_k + R of the same appendix is this sequence with
 *                                alpha = R.  Returns c = den / (alpha k + r0) as the exact rational.
 *                                INVALID_ARG unless 0 < r0 <= den and epoch >= 0.
 *   varco_schedule_exponential   r_k = 1 / beta^(K - k + 1) for steps k = 1..K, epoch = k - 1, i.e.
 *                                c = beta^(K - epoch) (the last epoch still compresses by beta; epochs >= K
 *                                give 1); the power saturates at 2^32 - 1.  INVALID_ARG unless beta >= 2,
 *                                K >= 1, epoch >= 0.
 * The fixed ratios of Section V are the constant {c, 1}; its "no communication" setting is a ratio with
 * den = 0: varco_kept returns k = 0 for it, the layer entry points then send nothing (halo_bytes = 0) and
 * every remote neighbour contributes the zero vector, forward and backward. */
int varco_schedule_rate_linear(int32_t epoch, uint32_t r0, uint32_t alpha, uint32_t den, varco_ratio_t *c);
int varco_schedule_exponential(int32_t epoch, int32_t K, int32_t beta, varco_ratio_t *c);

/* ------------------------------------------------------------------------------------------
 * Compression over all halo copies of the plan (Algorithm 1, second step; Definition 1;
 * appendix "Compression Mechanism").
 *
 * varco_compress: for every owner p, destination q (ascending) and row j of halo(p->q)
 *   (ascending id):  packed[pos][m] = X[row(j)][pi_j(m)],  m < k,  pos running over that send order.
 *   pi_j is the keyed permutation of [0, F) derived from (key, original id of j); k = varco_kept.
 *   X       device, [n x ld] in plan order;   packed  device, H_total * k elements, contiguous.
 *   bytes   host, optional: H_total * k * element_size, the volume one exchange puts on the wire.
 * varco_decompress: the receiving side.  For every destination q, owner p, row j (receive order):
 *   Xhalo[slot][c] = packed[pos(slot)][m] if c == pi_j(m) for some m < k, else 0.
 *   Xhalo   device, [H_total x ld]; all F columns of every slot are written.
 * Values are copied bit for bit, never rescaled.  Both need an uploaded plan.
 * Errors: INVALID_ARG, NOT_UPLOADED, UNSUPPORTED (F > 2048), CUDA.
 */
int varco_compress(const varco_plan_t *plan, const void *X, int64_t ld, int32_t F, varco_dtype_t dtype,
                   varco_ratio_t c, varco_key_t key, void *packed, uint64_t *bytes, void *stream);
int varco_decompress(const varco_plan_t *plan, const void *packed, int32_t F, varco_dtype_t dtype,
                     varco_ratio_t c, varco_key_t key, void *Xhalo, int64_t ld, void *stream);

/* ------------------------------------------------------------------------------------------
 * Exchange round trip without any allocation.  The paper has no counterpart: this entry point
 * exists for callers that are not allowed to allocate device memory -- code running where
 * cudaMalloc is forbidden or would stall the device (a serving loop with a latency budget, a hook
 * called while another framework owns the memory pool, a process whose caching allocator already
 * holds all device memory).
 *
 * varco_exchange_noalloc computes Xhalo = varco_decompress(varco_compress(X)) -- every halo slot
 * receives the row of its owner with the k kept values in place and zeros elsewhere -- and keeps
 * the packed rows in between in a fixed array of VARCO_NOALLOC_SCRATCH_BYTES bytes that is part
 * of the library image (every GPU that loads the library holds that much until the process
 * exits).  It calls no cudaMalloc, cudaFree or other allocating routine.
 *   X [n x ld], Xhalo [H_total x ld_halo]  device, caller-owned, same rules as varco_compress /
 *                                           varco_decompress; bytes (host, optional) as there.
 *   Limit: H_total * round_up(k, 16 / element_size) * element_size <= VARCO_NOALLOC_SCRATCH_BYTES,
 *   otherwise VARCO_WORKSPACE_TOO_SMALL and nothing is launched.
 *   The first call on a device looks up the device address of the array (once per device, with
 *   that device current); make that first call outside any stream capture.
 *   All calls on a device share the one array, which keeps the last call's packed rows: two calls
 *   whose kernels may overlap on the GPU (different streams) race on it.  Calls on one stream are
 *   ordered and safe.  Nothing needs clearing between calls.
 *   Errors: INVALID_ARG, NOT_UPLOADED, UNSUPPORTED, WORKSPACE_TOO_SMALL, CUDA.
 */
#define VARCO_NOALLOC_SCRATCH_BYTES (32u << 20)
int varco_exchange_noalloc(const varco_plan_t *plan, const void *X, int64_t ld, int32_t F,
                           varco_dtype_t dtype, varco_ratio_t c, varco_key_t key, void *Xhalo,
                           int64_t ld_halo, uint64_t *bytes, void *stream);

/* ------------------------------------------------------------------------------------------
 * One layer over all partitions (Eq. (2) with two taps; Algorithm 1 steps 2-4).
 *
 *   relu    1: ReLU after the transform, 0: identity (last layer).
 *   dtype   element type of X, Y, Agg, dY, dX and of the weight matrices (fp32 accumulation
 *           everywhere; with VARCO_BF16 the feature transform runs on the tensor cores).
 *   bias, dW_*, dbias are always fp32.
 */
typedef struct {
  varco_conv_t conv;
  varco_dtype_t dtype;
  int32_t F_in, F_out;
  int32_t relu;
  int64_t ld_in;   /* leading dimension of X, Agg, dX */
  int64_t ld_out;  /* leading dimension of Y, dY */
} varco_layer_desc_t;

/* varco_layer_fwd
 *   For every partition q and row i it owns:
 *     agg_i = sum_{j in N(i)} s_ij u_j,  u_j = x_j if q owns j, else decompress(compress(x_j));
 *     SAGE: y_i = rho(x_i W_self + agg_i W_neigh + b);   GCN: y_i = rho(agg_i W_neigh + b).
 *   X [n x ld_in], W_self / W_neigh [F_in x F_out] dense row-major (W_self NULL for GCN),
 *   bias [F_out] fp32 or NULL, Y [n x ld_out] out, Agg_saved [n x ld_in] out (needed by the
 *   backward pass), all device.  halo_bytes (host, optional) = H_total * k * element_size.
 *   Errors: INVALID_ARG, NOT_UPLOADED, WORKSPACE_TOO_SMALL, UNSUPPORTED, CUDA.
 */
int varco_layer_fwd(const varco_plan_t *plan, const varco_layer_desc_t *desc, const void *X,
                    const void *W_self, const void *W_neigh, const float *bias, void *Y,
                    void *Agg_saved, varco_ratio_t c, varco_key_t key, void *workspace,
                    size_t ws_bytes, uint64_t *halo_bytes, void *stream);

/* varco_layer_bwd
 *   Given dY = dLoss/dY and the forward's X, Y, Agg_saved and the same (c, key):
 *     dZ = dY (.) 1[Y > 0] (relu) or dY;
 *     dW_self = sum_i x_i^T dZ_i,  dW_neigh = sum_i agg_i^T dZ_i,  dbias = sum_i dZ_i over the rows
 *     of ALL partitions (the weight-gradient sum of Section III-A, third round);
 *     dx_j = [SAGE] dZ_j W_self^T + sum over local users i of s_ij dagg_i
 *            + sum over remote partitions q of M_j (.) (sum_{i in q} s_ij dagg_i),   dagg_i = dZ_i W_neigh^T,
 *     M_j the 0/1 mask of the forward's kept positions: the halo-slot gradients are compressed with
 *     the same permutation and k, sent back to the owner and added there in ascending q order
 *     (deterministic, no atomics).
 *   dX [n x ld_in] out; dW_self (NULL for GCN), dW_neigh [F_in x F_out] fp32 out; dbias [F_out]
 *   fp32 out (may be NULL).  halo_bytes as in the forward pass.
 */
int varco_layer_bwd(const varco_plan_t *plan, const varco_layer_desc_t *desc, const void *X,
                    const void *Y, const void *Agg_saved, const void *W_self, const void *W_neigh,
                    const void *dY, void *dX, float *dW_self, float *dW_neigh, float *dbias,
                    varco_ratio_t c, varco_key_t key, void *workspace, size_t ws_bytes,
                    uint64_t *halo_bytes, void *stream);

/* Device-side status of the most recent varco_layer_fwd / varco_layer_bwd that used `workspace`:
 * 0 = every kernel ran to completion; non-zero = a tensor-core kernel gave up on a bounded wait
 * (its outputs are then invalid; the kernel released its resources and returned, the context stays
 * usable).  Copies one word back on `stream` and synchronises it.  No counterpart in the paper. */
int varco_workspace_status(const void *workspace, void *stream, int *device_status);

/* ------------------------------------------------------------------------------------------
 * Per-stage device timing (no counterpart in the paper; a measurement aid).
 * When enabled, every kernel stage of the entry points above is bracketed by CUDA events on the
 * stream it is launched on.  varco_profile_read synchronises those events and returns, per stage,
 * the number of timed stage executions and the summed milliseconds since the last reset.
 */
enum {
  VARCO_STAGE_COMPRESS = 0,      /* halo gather + compress (forward)            */
  VARCO_STAGE_DECOMPRESS = 1,    /* decompress into halo slots (dense rows, or
                                    (value, position) pairs when k <= F/8)      */
  VARCO_STAGE_SPMM = 2,          /* aggregation over local + halo rows          */
  VARCO_STAGE_GEMM_FWD = 3,      /* feature transform, bias, activation         */
  VARCO_STAGE_GEMM_DX = 4,       /* dZ W^T                                       */
  VARCO_STAGE_GEMM_DW = 5,       /* [X | Agg]^T dZ and dbias                     */
  VARCO_STAGE_SPMM_T = 6,        /* transposed aggregation (to rows and slots)   */
  VARCO_STAGE_COMPRESS_BWD = 7,  /* k < F: kept positions of the boundary rows for the
                                    backward; the gradient compression itself runs in the
                                    epilogue of the transposed aggregation (stage 6) */
  VARCO_STAGE_SCATTER_ADD = 8,   /* decompress + ordered add into owner rows     */
  VARCO_STAGE_AUX = 9,           /* small helpers: masks, casts, weight repacks  */
  VARCO_STAGE_COUNT = 10
};
int varco_profile_enable(varco_plan_t *plan, int on);
int varco_profile_reset(varco_plan_t *plan);
int varco_profile_read(varco_plan_t *plan, int64_t *launches /* [VARCO_STAGE_COUNT] */,
                       double *milliseconds /* [VARCO_STAGE_COUNT] */);
/* The individual timed executions of one stage since the last reset, in the order they were enqueued
 * (one per layer call that ran the stage): up to `capacity` durations in milliseconds are written to
 * `milliseconds`, `count` receives how many exist.  Synchronises the events it reads. */
int varco_profile_spans(varco_plan_t *plan, int32_t stage, double *milliseconds, int64_t capacity,
                        int64_t *count);
/* Debug build (no counterpart in the paper).  A library compiled with -DVARCO_DEBUG checks, on the device,
 * every source row, destination row and kept position its aggregation kernels index against the extent of the
 * array it addresses; a failed check records a code (11 source row, 12 destination row, 13 kept position) and
 * skips the access -- nothing traps.  The same build validates the plan's index arrays on the host at upload
 * (BAD_GRAPH), puts 256 guard bytes behind every workspace segment, and reports a damaged guard block as bit 30
 * of varco_workspace_status.  This call synchronises the device and returns the first recorded code (0 = none)
 * and clears it; in a release build is_debug_build = 0 and word = 0. */
int varco_debug_status(int32_t *is_debug_build, int32_t *word);
/* Random-row gather probe (no counterpart in the paper; a measurement aid).  Every output row is the
 * bitwise XOR of `per_out` rows of `table`, picked by `index`; nothing else is computed, so the time of the
 * launch is the time the memory system needs for out_rows * per_out random row reads.  The benchmark calls
 * it on a table that fits L2 and on one that does not: those two rates are what the aggregation stages,
 * which read one feature row per stored entry, are measured against.
 *   table  device, [table_rows x row_chunks * 16 bytes], 16-byte aligned; row_chunks in {8, 16, 32}
 *   index  device int32 [out_rows x per_out], 16-byte aligned, per_out a positive multiple of 4; values are
 *          clamped into [0, table_rows) by the kernel
 *   out    device, [out_rows x row_chunks * 16 bytes]
 * Enqueued on `stream`, no synchronisation.  INVALID_ARG / UNSUPPORTED on anything else. */
int varco_probe_gather(const void *table, int64_t table_rows, int32_t row_chunks, const int32_t *index,
                       int64_t out_rows, int32_t per_out, void *out, void *stream);
/* Number of CUDA kernels this library has launched in this process so far (all plans, all
 * streams).  Also a measurement aid without a counterpart in the paper. */
int varco_kernel_launches(int64_t *count);

#ifdef __cplusplus
}
#endif
#endif /* VARCO_H_ */
