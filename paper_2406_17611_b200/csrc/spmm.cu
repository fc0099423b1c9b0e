// Aggregation kernels: CSR SpMM over local rows plus halo slots, and its transpose.
//
// Forward (Algorithm 1, third step; Eq. (2) with one AGGREGATE tap): for every row i of every
// partition, agg_i = sum_j s_ij u_j where u_j is the exact row of X when the owner of i also
// owns j and the decompressed halo-slot row otherwise.  Backward: the same kernel walks the
// transposed structure, sources being dAgg rows and destinations the local rows of dX and the
// halo-slot gradient rows.
//
// One group of G lanes per row (G = 4..32, a whole warp for rows of >= 32 x 16 bytes); every lane
// owns NCH 16-byte chunks of the feature row, gathers them with 128-bit loads and accumulates in
// fp32.  Column indices and weights of G entries are loaded cooperatively and broadcast with
// shuffles; four row gathers are kept in flight per lane.  Rows are taken longest-first.
#include "device_common.cuh"

namespace {

template <typename T, int G, int NCH, int UNR>
__global__ void __launch_bounds__(256)
    spmm_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ col, const float *__restrict__ val,
                const int32_t *__restrict__ order, int nrows, const T *__restrict__ A0, int64_t lda0,
                const T *__restrict__ A1, int64_t lda1, int src_split, T *__restrict__ O0, int64_t ldo0,
                T *__restrict__ O1, int64_t ldo1, int dst_split, int accumulate0, int nv) {
  constexpr int V = ElemTraits<T>::kVec;
  const int tid = blockIdx.x * blockDim.x + threadIdx.x;
  const int gid = tid / G;
  const int gl = threadIdx.x % G;
  if (gid >= nrows) return;
  const unsigned lane = threadIdx.x % 32;
  const unsigned gmask = (G == 32) ? 0xFFFFFFFFu : (((1u << G) - 1u) << (lane & ~(unsigned)(G - 1)));
  const int r = order[gid];
  const int64_t e0 = rp[r], e1 = rp[r + 1];

  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;

  for (int64_t base = e0; base < e1; base += G) {
    const int cnt = (int)((e1 - base) < (int64_t)G ? (e1 - base) : (int64_t)G);
    int myc = 0;
    float myw = 0.f;
    if (gl < cnt) {
      myc = __ldg(col + base + gl);
      myw = __ldg(val + base + gl);
    }
    for (int t = 0; t < cnt; t += UNR) {
      uint4 v[UNR][NCH];
      float w[UNR];
#pragma unroll
      for (int u = 0; u < UNR; ++u) {
        const int tt = t + u;
        const int c = __shfl_sync(gmask, myc, tt, G);
        w[u] = __shfl_sync(gmask, myw, tt, G);
        const bool live = tt < cnt;
        const uint4 *src = (c < src_split)
                               ? reinterpret_cast<const uint4 *>(A0 + (int64_t)c * lda0)
                               : reinterpret_cast<const uint4 *>(A1 + (int64_t)(c - src_split) * lda1);
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
          const int ch = gl + i * G;
          v[u][i] = (live && ch < nv) ? __ldg(src + ch) : make_uint4(0u, 0u, 0u, 0u);
        }
        if (!live) w[u] = 0.f;
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

  uint4 *dst;
  bool add = false;
  if (r < dst_split) {
    dst = reinterpret_cast<uint4 *>(O0 + (int64_t)r * ldo0);
    add = accumulate0 != 0;
  } else {
    dst = reinterpret_cast<uint4 *>(O1 + (int64_t)(r - dst_split) * ldo1);
  }
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int ch = gl + i * G;
    if (ch < nv) {
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

struct SpmmArgs {
  const int64_t *rp;
  const int32_t *col;
  const float *val;
  const int32_t *order;
  int nrows;
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
  int nv;
};

template <typename T, int G, int NCH, int UNR>
int launch(const SpmmArgs &a, cudaStream_t st) {
  const int threads = 256;
  const int64_t total = (int64_t)a.nrows * G;
  dim3 grid((unsigned)((total + threads - 1) / threads));
  spmm_kernel<T, G, NCH, UNR><<<grid, threads, 0, st>>>(a.rp, a.col, a.val, a.order, a.nrows, (const T *)a.A0, a.lda0,
                                                        (const T *)a.A1, a.lda1, a.src_split, (T *)a.O0, a.ldo0,
                                                        (T *)a.O1, a.ldo1, a.dst_split, a.accumulate0, a.nv);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

template <typename T>
int dispatch(const SpmmArgs &a, cudaStream_t st) {
  const int nv = a.nv;
  if (nv <= 4) return launch<T, 4, 1, 4>(a, st);
  if (nv <= 8) return launch<T, 8, 1, 4>(a, st);
  if (nv <= 16) return launch<T, 16, 1, 4>(a, st);
  if (nv <= 32) return launch<T, 32, 1, 4>(a, st);
  if (nv <= 64) return launch<T, 32, 2, 4>(a, st);
  if (nv <= 96) return launch<T, 32, 3, 4>(a, st);
  if (nv <= 128) return launch<T, 32, 4, 2>(a, st);
  if (nv <= 256) return launch<T, 32, 8, 2>(a, st);
  return VARCO_UNSUPPORTED;
}

}  // namespace

// Forward aggregation: Agg[r] = sum_e val[e] * (col[e] < n ? X[col[e]] : Xhalo[col[e] - n]).
int varco_launch_spmm_fwd(const varco_plan *pl, const void *X, int64_t ldx, const void *Xhalo, int64_t ldh, int F,
                          varco_dtype_t dt, void *Agg, int64_t ldagg, cudaStream_t st) {
  const int V = dt == VARCO_F32 ? 4 : 8;
  SpmmArgs a{pl->d.rp, pl->d.col, pl->d.val, pl->d.order_f, (int)pl->n, X, ldx, Xhalo, ldh, (int)pl->n,
             Agg,      ldagg,     nullptr,   0,             (int)pl->n, 0, (F + V - 1) / V};
  return dt == VARCO_F32 ? dispatch<float>(a, st) : dispatch<__nv_bfloat16>(a, st);
}

// Transposed aggregation: for a source u, g_u = sum over the rows i that use it of s_iu dAgg[i];
// u < n lands in dX[u] (added to what is there when `accumulate`), u >= n in Ghalo[u - n].
int varco_launch_spmm_bwd(const varco_plan *pl, const void *dAgg, int64_t ldd, int F, varco_dtype_t dt, void *dX,
                          int64_t ldx, int accumulate, void *Ghalo, int64_t ldh, cudaStream_t st) {
  const int V = dt == VARCO_F32 ? 4 : 8;
  SpmmArgs a{pl->d.rpT, pl->d.colT, pl->d.valT, pl->d.order_t, (int)(pl->n + pl->H), dAgg, ldd, dAgg, ldd,
             (int)pl->n, dX, ldx, Ghalo, ldh, (int)pl->n, accumulate, (F + V - 1) / V};
  return dt == VARCO_F32 ? dispatch<float>(a, st) : dispatch<__nv_bfloat16>(a, st);
}
