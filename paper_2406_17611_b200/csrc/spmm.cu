// Aggregation kernels: CSR SpMM over local rows plus halo slots, and its transpose.
//
// Forward (Algorithm 1, third step; Eq. (2) with one AGGREGATE tap): for every row i of every
// partition, agg_i = sum_j s_ij u_j where u_j is the exact row of X when the owner of i also
// owns j and the decompressed halo-slot row otherwise.  Backward: the same kernels walk the
// transposed structure, sources being dAgg rows and destinations the local rows of dX and the
// halo-slot gradient rows.
//
// One group of G lanes per row (G = 4..32); every lane owns NCH 16-byte chunks of the feature
// row, gathers them with 128-bit loads and accumulates in fp32.  Column indices and weights of G
// entries are loaded cooperatively and broadcast with shuffles; several row gathers are kept in
// flight per lane.  Rows come in three classes by number of entries: hubs get a CTA each, short
// rows get narrow lane groups (several rows per warp), the rest a full-width group.
//
// Scheduling: the gathers are random 16..512-byte reads bounded by DRAM unless the gathered set
// stays in L2.  Work is issued partition by partition; the kernels can also split the feature
// row into panels (task = (partition, panel, row)) so that a partition's gathered set fits in L2,
// but on the measured workloads the extra passes cost more than the hits return, so the
// launchers use one panel.
#include <algorithm>

#include "device_common.cuh"
#include "kernels.h"

namespace {

struct RowClass {
  const int32_t *rows;   // row ids, partition-major
  const int32_t *start;  // [P + 1] first position of every partition in `rows`
  int count;
};

struct SpmmArgs {
  const int64_t *rp;
  const int32_t *col;
  const float *val;
  RowClass hubs, normal, shorts;
  int P;
  const void *A0;
  int64_t lda0;
  const void *A1;
  int64_t lda1;
  int src_split;
  void *O0;
  int64_t ldo0;
  void *O1;
  int64_t ldo1;
  int dst_split;
  int accumulate0;
  int nv;        // 16-byte chunks per row
  int panels;    // feature panels
  int nv_panel;  // chunks per panel
};

// task id -> (position in the class list, panel); tasks are ordered (partition, panel, row)
__device__ __forceinline__ void locate(const RowClass &rc, int P, int panels, int64_t task, int &pos, int &panel) {
  if (panels == 1) {
    pos = (int)task;
    panel = 0;
    return;
  }
  int lo = 0, hi = P;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if ((int64_t)__ldg(rc.start + mid) * panels <= task) lo = mid;
    else hi = mid;
  }
  const int s0 = __ldg(rc.start + lo), s1 = __ldg(rc.start + lo + 1);
  const int64_t local = task - (int64_t)s0 * panels;
  const int rows_q = s1 - s0;
  panel = (int)(local / rows_q);
  pos = s0 + (int)(local % rows_q);
}

// Where the gathers read from: sources below `split` are rows of A0, the others rows of A1.  The A1 base is
// stored pre-offset by -split rows, so that both cases are base + c * stride.
struct GatherSrc {
  const uint4 *b0, *b1s;   // in 16-byte units
  int ld0, ld1;            // row strides in 16-byte units
  int split;
};

// Accumulate `len` entries of one row: acc[i][:] += val[e] * chunk (ch_lo + gl + i G) of source col[e].
// FULL: the group covers exactly the row's chunks, no bounds test on the chunk index.
// Entries are taken G at a time; lanes beyond the last entry of a batch hold a valid column with weight
// zero, so that the inner loop needs no per-entry predicate.
template <typename T, int G, int NCH, int UNR, bool FULL>
__device__ __forceinline__ void accumulate_range(const int32_t *__restrict__ colp, const float *__restrict__ valp,
                                                 int len, const GatherSrc &gs, int ch_lo, int ch_hi, int gl,
                                                 unsigned gmask, float (&acc)[NCH][ElemTraits<T>::kVec]) {
  constexpr int V = ElemTraits<T>::kVec;
  for (int base = 0; base < len; base += G) {
    const int cnt = min(G, len - base);
    const int mine = base + min(gl, cnt - 1);
    const int myc = __ldg(colp + mine);
    const float myw = gl < cnt ? __ldg(valp + mine) : 0.f;
    for (int t = 0; t < cnt; t += UNR) {
      uint4 v[UNR][NCH];
      float w[UNR];
#pragma unroll
      for (int u = 0; u < UNR; ++u) {
        const int c = __shfl_sync(gmask, myc, t + u, G);
        w[u] = __shfl_sync(gmask, myw, t + u, G);
        const bool loc = c < gs.split;
        const uint4 *src = (loc ? gs.b0 : gs.b1s) + (int64_t)c * (loc ? gs.ld0 : gs.ld1) + (ch_lo + gl);
#pragma unroll
        for (int i = 0; i < NCH; ++i)
          v[u][i] = (FULL || ch_lo + gl + i * G < ch_hi) ? __ldg(src + i * G) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < UNR; ++u)
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
          float f[V];
          unpack16(v[u][i], f, T());
#pragma unroll
          for (int j = 0; j < V; ++j) acc[i][j] = fmaf(w[u], f[j], acc[i][j]);
        }
    }
  }
}

template <typename T>
__device__ __forceinline__ uint4 *dest_row(int r, T *O0, int64_t ldo0, T *O1, int64_t ldo1, int dst_split,
                                           int accumulate0, bool &add) {
  if (r < dst_split) {
    add = accumulate0 != 0;
    return reinterpret_cast<uint4 *>(O0 + (int64_t)r * ldo0);
  }
  add = false;
  return reinterpret_cast<uint4 *>(O1 + (int64_t)(r - dst_split) * ldo1);
}

template <typename T, int G, int NCH, int UNR, bool FULL>
__global__ void __launch_bounds__(256)
    spmm_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ col, const float *__restrict__ val,
                RowClass rc, int P, int panels, int nv_panel, GatherSrc gs, T *__restrict__ O0, int64_t ldo0,
                T *__restrict__ O1, int64_t ldo1, int dst_split, int accumulate0, int nv) {
  constexpr int V = ElemTraits<T>::kVec;
  const int64_t task = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int gl = threadIdx.x % G;
  if (task >= (int64_t)rc.count * panels) return;
  const unsigned lane = threadIdx.x % 32;
  const unsigned gmask = (G == 32) ? 0xFFFFFFFFu : (((1u << G) - 1u) << (lane & ~(unsigned)(G - 1)));
  int pos, panel;
  locate(rc, P, panels, task, pos, panel);
  const int r = __ldg(rc.rows + pos);
  const int ch_lo = panel * nv_panel;
  const int ch_hi = min(nv, ch_lo + nv_panel);

  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  const int64_t e0 = rp[r];
  accumulate_range<T, G, NCH, UNR, FULL>(col + e0, val + e0, (int)(rp[r + 1] - e0), gs, ch_lo, ch_hi, gl, gmask, acc);
  bool add;
  uint4 *dst = dest_row<T>(r, O0, ldo0, O1, ldo1, dst_split, accumulate0, add);
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int ch = ch_lo + gl + i * G;
    if (ch < ch_hi) {
      if (add) {
        float f[V];
        unpack16(dst[ch], f, T());
#pragma unroll
        for (int j = 0; j < V; ++j) acc[i][j] += f[j];
      }
      dst[ch] = pack16(acc[i], T());
    }
  }
}

// Long rows (hubs of a skewed degree distribution): one CTA per (row, panel), every warp takes a
// contiguous share of the entries, partial sums meet in shared memory and are added in warp order.
template <typename T, int NCH, int UNR, bool FULL>
__global__ void __launch_bounds__(256)
    spmm_hub_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ col, const float *__restrict__ val,
                    RowClass rc, int P, int panels, int nv_panel, GatherSrc gs, T *__restrict__ O0, int64_t ldo0,
                    T *__restrict__ O1, int64_t ldo1, int dst_split, int accumulate0, int nv) {
  extern __shared__ float hub_part[];
  constexpr int V = ElemTraits<T>::kVec;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int nwarps = blockDim.x / 32;
  int pos, panel;
  locate(rc, P, panels, blockIdx.x, pos, panel);
  const int r = __ldg(rc.rows + pos);
  const int ch_lo = panel * nv_panel;
  const int ch_hi = min(nv, ch_lo + nv_panel);
  const int64_t e0 = rp[r], e1 = rp[r + 1];
  const int64_t per = ((e1 - e0 + nwarps - 1) / nwarps + 31) / 32 * 32;
  const int64_t b0 = e0 + warp * per < e1 ? e0 + warp * per : e1;
  const int64_t b1 = b0 + per < e1 ? b0 + per : e1;
  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  if (b1 > b0)
    accumulate_range<T, 32, NCH, UNR, FULL>(col + b0, val + b0, (int)(b1 - b0), gs, ch_lo, ch_hi, lane, 0xFFFFFFFFu,
                                            acc);
  const int row_floats = nv_panel * V;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int c = lane + i * 32;
    if (c < nv_panel)
#pragma unroll
      for (int j = 0; j < V; ++j) hub_part[(size_t)warp * row_floats + c * V + j] = acc[i][j];
  }
  __syncthreads();
  bool add;
  uint4 *dst = dest_row<T>(r, O0, ldo0, O1, ldo1, dst_split, accumulate0, add);
  for (int c = threadIdx.x; c < ch_hi - ch_lo; c += blockDim.x) {
    float f[V];
#pragma unroll
    for (int j = 0; j < V; ++j) f[j] = 0.f;
    if (add) unpack16(dst[ch_lo + c], f, T());
    for (int w = 0; w < nwarps; ++w)
#pragma unroll
      for (int j = 0; j < V; ++j) f[j] += hub_part[(size_t)w * row_floats + c * V + j];
    dst[ch_lo + c] = pack16(f, T());
  }
}

template <typename T>
GatherSrc gather_src(const SpmmArgs &a) {
  constexpr int V = ElemTraits<T>::kVec;
  GatherSrc gs;
  gs.b0 = reinterpret_cast<const uint4 *>(a.A0);
  gs.ld0 = (int)(a.lda0 / V);
  gs.ld1 = (int)(a.lda1 / V);
  gs.b1s = reinterpret_cast<const uint4 *>(a.A1) - (int64_t)a.src_split * gs.ld1;
  gs.split = a.src_split;
  return gs;
}

template <typename T, int NCH, int UNR>
int launch_hubs(const SpmmArgs &a, cudaStream_t st) {
  if (a.hubs.count == 0) return VARCO_OK;
  constexpr int V = ElemTraits<T>::kVec;
  const size_t row_bytes = (size_t)a.nv_panel * V * sizeof(float);
  int warps = 8;
  while (warps > 1 && warps * row_bytes > 48 * 1024) warps /= 2;
  const dim3 grid((unsigned)(a.hubs.count * a.panels));
  if (a.panels == 1 && a.nv == 32 * NCH)
    spmm_hub_kernel<T, NCH, UNR, true><<<grid, warps * 32, warps * row_bytes, st>>>(
        a.rp, a.col, a.val, a.hubs, a.P, a.panels, a.nv_panel, gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1, a.ldo1,
        a.dst_split, a.accumulate0, a.nv);
  else
    spmm_hub_kernel<T, NCH, UNR, false><<<grid, warps * 32, warps * row_bytes, st>>>(
        a.rp, a.col, a.val, a.hubs, a.P, a.panels, a.nv_panel, gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1, a.ldo1,
        a.dst_split, a.accumulate0, a.nv);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

template <typename T, int G, int NCH, int UNR>
int launch_rows(const SpmmArgs &a, const RowClass &rc, cudaStream_t st) {
  if (rc.count == 0) return VARCO_OK;
  const int threads = 256;
  const int64_t total = (int64_t)rc.count * a.panels * G;
  dim3 grid((unsigned)((total + threads - 1) / threads));
  if (a.panels == 1 && a.nv == G * NCH)
    spmm_kernel<T, G, NCH, UNR, true><<<grid, threads, 0, st>>>(a.rp, a.col, a.val, rc, a.P, a.panels, a.nv_panel,
                                                                gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1, a.ldo1,
                                                                a.dst_split, a.accumulate0, a.nv);
  else
    spmm_kernel<T, G, NCH, UNR, false><<<grid, threads, 0, st>>>(a.rp, a.col, a.val, rc, a.P, a.panels, a.nv_panel,
                                                                 gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1,
                                                                 a.ldo1, a.dst_split, a.accumulate0, a.nv);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// G/NCH: lanes per row and 16-byte chunks per lane for ordinary rows; GS/NCHS: the same for rows of
// at most a handful of entries, where narrower groups keep more rows in flight per warp.
template <typename T, int G, int NCH, int UNR, int GS, int NCHS, int UNRS>
int launch(const SpmmArgs &a, cudaStream_t st) {
  if (int rc = launch_hubs<T, NCH, UNR>(a, st)) return rc;
  if (int rc = launch_rows<T, G, NCH, UNR>(a, a.normal, st)) return rc;
  return launch_rows<T, GS, NCHS, UNRS>(a, a.shorts, st);
}

template <typename T>
int dispatch(const SpmmArgs &a, cudaStream_t st) {
  const int w = a.nv_panel;  // chunks a group has to cover
  // short-row variants keep one gather per lane in flight: with few entries per row the
  // parallelism comes from the number of rows resident per SM, i.e. from a low register count
  if (w <= 4) return launch<T, 4, 1, 4, 4, 1, 2>(a, st);
  if (w <= 8) return launch<T, 8, 1, 4, 4, 2, 2>(a, st);
  if (w <= 16) return launch<T, 16, 1, 4, 4, 4, 1>(a, st);
  if (w <= 32) return launch<T, 32, 1, 4, 8, 4, 1>(a, st);
  if (w <= 64) return launch<T, 32, 2, 4, 16, 4, 1>(a, st);
  if (w <= 96) return launch<T, 32, 3, 4, 16, 6, 1>(a, st);
  if (w <= 128) return launch<T, 32, 4, 2, 32, 4, 1>(a, st);
  if (w <= 256) return launch<T, 32, 8, 2, 32, 8, 1>(a, st);
  return VARCO_UNSUPPORTED;
}

}  // namespace

// Forward aggregation: Agg[r] = sum_e val[e] * (col[e] < n ? X[col[e]] : Xhalo[col[e] - n]).
int varco_launch_spmm_fwd(const varco_plan *pl, const void *X, int64_t ldx, const void *Xhalo, int64_t ldh, int F,
                          varco_dtype_t dt, void *Agg, int64_t ldagg, cudaStream_t st) {
  const int V = dt == VARCO_F32 ? 4 : 8;
  const int nv = (F + V - 1) / V;
  SpmmArgs a{};
  a.rp = pl->d.rp;
  a.col = pl->d.col;
  a.val = pl->d.val;
  a.hubs = RowClass{pl->d.hub_f, pl->d.hub_f_start, (int)pl->hub_f.size()};
  a.normal = RowClass{pl->d.order_f, pl->d.order_f_start, (int)pl->order_f.size()};
  a.shorts = RowClass{pl->d.short_f, pl->d.short_f_start, (int)pl->short_f.size()};
  a.P = pl->P;
  a.A0 = X;
  a.lda0 = ldx;
  a.A1 = Xhalo;
  a.lda1 = ldh;
  a.src_split = (int)pl->n;
  a.O0 = Agg;
  a.ldo0 = ldagg;
  a.O1 = nullptr;
  a.ldo1 = 0;
  a.dst_split = (int)pl->n;
  a.accumulate0 = 0;
  a.nv = nv;
  a.panels = 1;
  a.nv_panel = nv;
  return dt == VARCO_F32 ? dispatch<float>(a, st) : dispatch<__nv_bfloat16>(a, st);
}

// Transposed aggregation: for a source u, g_u = sum over the rows i that use it of s_iu dAgg[i];
// u < n lands in dX[u] (added to what is there when `accumulate`), u >= n in Ghalo[u - n].
// Every source of partition q is used by rows of q only, so the gathered set of a partition is
// its own block of dAgg: panels are chosen so that this block stays in L2.
int varco_launch_spmm_bwd(const varco_plan *pl, const void *dAgg, int64_t ldd, int F, varco_dtype_t dt, void *dX,
                          int64_t ldx, int accumulate, void *Ghalo, int64_t ldh, cudaStream_t st) {
  const int V = dt == VARCO_F32 ? 4 : 8;
  const int nv = (F + V - 1) / V;
  SpmmArgs a{};
  a.rp = pl->d.rpT;
  a.col = pl->d.colT;
  a.val = pl->d.valT;
  a.hubs = RowClass{pl->d.hub_t, pl->d.hub_t_start, (int)pl->hub_t.size()};
  a.normal = RowClass{pl->d.order_t, pl->d.order_t_start, (int)pl->order_t.size()};
  a.shorts = RowClass{pl->d.short_t, pl->d.short_t_start, (int)pl->short_t.size()};
  a.P = pl->P;
  a.A0 = dAgg;
  a.lda0 = ldd;
  a.A1 = dAgg;
  a.lda1 = ldd;
  a.src_split = (int)pl->n;
  a.O0 = dX;
  a.ldo0 = ldx;
  a.O1 = Ghalo;
  a.ldo1 = ldh;
  a.dst_split = (int)pl->n;
  a.accumulate0 = accumulate;
  a.nv = nv;
  a.panels = 1;
  a.nv_panel = nv;
  return dt == VARCO_F32 ? dispatch<float>(a, st) : dispatch<__nv_bfloat16>(a, st);
}
