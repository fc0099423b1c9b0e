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
// launchers use one panel.  Measured and dropped: fetching every gathered row with one bulk asynchronous
// copy (cp.async.bulk into a per-warp shared-memory ring, mbarrier completion, two or four stages): at
// 512 bytes per copy the copy path sustained about one row per 25 SM cycles, 1.5x slower than the 128-bit
// loads used here.
#include <algorithm>

#include "device_common.cuh"
#include "kernels.h"

#ifndef VARCO_SHORT_UNR
#define VARCO_SHORT_UNR 2
#endif

namespace {

// Resident CTAs per SM the aggregation kernels are compiled for.  At full size the gathers wait on DRAM, and
// the bytes in flight per SM decide the rate: for rows of at most 512 bytes (one 16-byte chunk per lane of an
// ordinary or hub row, at most four per lane of a short row) one more resident CTA than the unconstrained
// register allocation gives (4 -> 5, short rows 3 -> 4, at the price of a few spilled registers) took 1.7 ms
// off the 57 ms epoch of the 2.45M-node workload; one more again spills into the inner loop and loses 10 ms.
// Wider rows keep their registers: forced to the same residency they spill and run at half speed.
constexpr int rows_blocks_per_sm(int nch) { return nch == 1 ? 5 : 1; }
constexpr int short_blocks_per_sm(int nch) { return nch <= 4 ? 4 : 1; }

struct RowClass {
  const int32_t *rows;   // row ids, partition-major
  const int32_t *start;  // [P + 1] first position of every partition in `rows`
  int count;
};

// Optional epilogue of the transposed pass: a halo-slot gradient row is not written out densely but
// compressed on the spot with the forward's key (k values at the kept positions, slot order).
struct HaloCompress {
  void *packed;          // nullptr: write dense rows
  int64_t kstride;       // elements per packed row
  int k, F, h;
  uint64_t lkey;
  const int32_t *slot_gid;
  const uint16_t *wpos;      // table of kept positions by source row (nullptr: evaluate the permutation here)
  int64_t wstride;
  const int32_t *slot_src;
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
  HaloCompress hc;
  const int32_t *short_col;   // 8-entry records of the short class (nullptr: walk the CSR)
  const float *short_val;
  int short_nlocal;           // leading rows of the short class whose result is a local row (the rest: halo slots)
  const int32_t *nloc_only;   // forward, no communication: per-row count of local entries (else nullptr)
  int row_limit;              // transposed, no communication: first row that is not computed (0: all rows)
  int nsrc, ndst;             // extents of the source / destination index spaces
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
  // "no communication" (k = 0): a forward row stops after its nloc[r] local entries (the halo entries would
  // add zero vectors), and the transposed pass leaves out the rows at or beyond row_limit (the halo slots,
  // whose gradients nobody receives)
  const int32_t *nloc_only;   // nullptr: rows are walked whole
  int row_limit;              // rows >= row_limit are not computed (INT_MAX: all)
  int nsrc, ndst;             // extents of the source and destination index spaces (checked in the debug build)
};

// acc[j] = w * f[j] + acc[j] for V values, two per instruction (packed fp32 FMA of sm_100; each half rounds
// like a scalar fmaf, so results are unchanged)
template <int V>
__device__ __forceinline__ void fma_row(float (&acc)[V], float w, const float (&f)[V]) {
#pragma unroll
  for (int j = 0; j < V; j += 2)
    asm("{\n\t.reg .b64 a, b, c, d;\n\tmov.b64 a, {%2, %3};\n\tmov.b64 b, {%4, %4};\n\tmov.b64 c, {%0, %1};\n\t"
        "fma.rn.f32x2 d, a, b, c;\n\tmov.b64 {%0, %1}, d;\n\t}"
        : "+f"(acc[j]), "+f"(acc[j + 1])
        : "f"(f[j]), "f"(f[j + 1]), "f"(w));
}

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
        const bool ok = VARCO_DBG_OK(c, gs.nsrc, 11);
        const uint4 *src = (loc ? gs.b0 : gs.b1s) + (int64_t)c * (loc ? gs.ld0 : gs.ld1) + (ch_lo + gl);
#pragma unroll
        for (int i = 0; i < NCH; ++i)
          v[u][i] = (ok && (FULL || ch_lo + gl + i * G < ch_hi)) ? __ldg(src + i * G) : make_uint4(0u, 0u, 0u, 0u);
      }
#pragma unroll
      for (int u = 0; u < UNR; ++u)
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
          float f[V];
          unpack16(v[u][i], f, T());
          fma_row<V>(acc[i], w[u], f);
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

// Packed row of one slot from its staged gradient row: z[m] = srow[pos[m]], m < k, zeros up to kstride.  Works in
// 16-byte chunks: a lane reads V positions of the table with one load, picks V elements from shared memory and
// writes them with one store (the table rows and the packed rows are 16-byte aligned, kstride a multiple of V).
template <int V>
__device__ __forceinline__ uint4 load_positions(const uint16_t *__restrict__ prow, int c) {
  if (V == 8) return __ldg(reinterpret_cast<const uint4 *>(prow + c * V));
  const uint2 pw = __ldg(reinterpret_cast<const uint2 *>(prow + c * V));
  return make_uint4(pw.x, pw.y, 0u, 0u);
}
template <typename E, int V>
__device__ __forceinline__ void pick_kept(const E *srow, const uint16_t *__restrict__ prow, E *__restrict__ z, int k,
                                          int kstride, int lane, int lanes) {
  uint4 *z4 = reinterpret_cast<uint4 *>(z);
  for (int c = lane; c * V < kstride; c += lanes) {
    const uint4 pw = load_positions<V>(prow, c);
    const uint32_t ps[4] = {pw.x, pw.y, pw.z, pw.w};
    E out[V];
#pragma unroll
    for (int i = 0; i < V; ++i) out[i] = c * V + i < k ? srow[(ps[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu] : (E)0;
    z4[c] = *reinterpret_cast<const uint4 *>(out);
  }
}

// Write one finished row: dense (optionally added to what is there), or -- for a halo-slot gradient row of
// the transposed pass when hc.packed is set -- compressed with the forward's key.
template <typename T, int G, int NCH, bool FULL>
__device__ __forceinline__ void finish_row(float (&acc)[NCH][ElemTraits<T>::kVec], int r, int gl, unsigned gmask,
                                           int ch_lo, int ch_hi, int nv, uint4 *stage_rows, T *__restrict__ O0,
                                           int64_t ldo0, T *__restrict__ O1, int64_t ldo1, int dst_split,
                                           int accumulate0, const HaloCompress &hc) {
  constexpr int V = ElemTraits<T>::kVec;
  if (hc.packed && r >= dst_split) {
    // stage the row in the element type, pick the kept positions, write k values
    typedef typename ElemBits<T>::type E;
    uint4 *srow4 = stage_rows + (size_t)(threadIdx.x / G) * nv;
#pragma unroll
    for (int i = 0; i < NCH; ++i) {
      const int ch = gl + i * G;
      if (FULL || ch < nv) srow4[ch] = pack16(acc[i], T());
    }
    const int slot = r - dst_split;
    const E *srow = reinterpret_cast<const E *>(srow4);
    E *z = reinterpret_cast<E *>(hc.packed) + (int64_t)slot * hc.kstride;
    if (hc.wpos) {
      const uint16_t *prow = hc.wpos + (int64_t)__ldg(hc.slot_src + slot) * hc.wstride;
      __syncwarp(gmask);
      pick_kept<E, V>(srow, prow, z, hc.k, (int)hc.kstride, gl, G);
      return;
    }
    vperm::RowPerm pm;
    if (G >= 8) init_perm<(G >= 8 ? G : 8)>(pm, hc.lkey, (uint32_t)__ldg(hc.slot_gid + slot), (uint32_t)hc.F, hc.h, gl, gmask);
    else pm.init(hc.lkey, (uint32_t)__ldg(hc.slot_gid + slot), (uint32_t)hc.F, hc.h);
    __syncwarp(gmask);
    for (int m = gl; m < (int)hc.kstride; m += G) z[m] = m < hc.k ? srow[pm.pi((uint32_t)m)] : (E)0;
    return;
  }
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

template <typename T, int G, int NCH, int UNR, bool FULL>
__global__ void __launch_bounds__(256, rows_blocks_per_sm(NCH))
    spmm_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ col, const float *__restrict__ val,
                RowClass rc, int P, int panels, int nv_panel, GatherSrc gs, T *__restrict__ O0, int64_t ldo0,
                T *__restrict__ O1, int64_t ldo1, int dst_split, int accumulate0, int nv, HaloCompress hc) {
  extern __shared__ uint4 stage_rows[];
  constexpr int V = ElemTraits<T>::kVec;
  const int64_t task = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int gl = threadIdx.x % G;
  if (task >= (int64_t)rc.count * panels) return;
  const unsigned lane = threadIdx.x % 32;
  const unsigned gmask = (G == 32) ? 0xFFFFFFFFu : (((1u << G) - 1u) << (lane & ~(unsigned)(G - 1)));
  int pos, panel;
  locate(rc, P, panels, task, pos, panel);
  const int r = __ldg(rc.rows + pos);
  if (r >= gs.row_limit || !VARCO_DBG_OK(r, gs.ndst, 12)) return;
  const int ch_lo = panel * nv_panel;
  const int ch_hi = min(nv, ch_lo + nv_panel);

  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  const int64_t e0 = rp[r];
  const int len = gs.nloc_only ? __ldg(gs.nloc_only + r) : (int)(rp[r + 1] - e0);
  accumulate_range<T, G, NCH, UNR, FULL>(col + e0, val + e0, len, gs, ch_lo, ch_hi, gl, gmask, acc);
  finish_row<T, G, NCH, FULL>(acc, r, gl, gmask, ch_lo, ch_hi, nv, stage_rows, O0, ldo0, O1, ldo1, dst_split, accumulate0,
                              hc);
}

// Short rows (at most 8 entries) from fixed-size records: sources and weights of a row sit at 8 * task, so
// the gathers start after a single dependent load.
template <typename T, int G, int NCH, int UNR, bool FULL>
__global__ void __launch_bounds__(256, short_blocks_per_sm(NCH))
    spmm_short_kernel(const int32_t *__restrict__ rec_col, const float *__restrict__ rec_val,
                      const int32_t *__restrict__ rows, int count, GatherSrc gs, T *__restrict__ O0, int64_t ldo0,
                      T *__restrict__ O1, int64_t ldo1, int dst_split, int accumulate0, int nv, HaloCompress hc) {
  extern __shared__ uint4 stage_rows[];
  constexpr int V = ElemTraits<T>::kVec;
  static_assert(G >= 8, "a record has 8 entries, one per lane");
  const int task = (blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int gl = threadIdx.x % G;
  if (task >= count) return;
  const unsigned lane = threadIdx.x % 32;
  const unsigned gmask = (G == 32) ? 0xFFFFFFFFu : (((1u << G) - 1u) << (lane & ~(unsigned)(G - 1)));
  int myc = -1;
  float myw = 0.f;
  if (gl < 8) {
    myc = __ldg(rec_col + (int64_t)task * 8 + gl);
    myw = __ldg(rec_val + (int64_t)task * 8 + gl);
  }
  const int r = __ldg(rows + task);
  if (!VARCO_DBG_OK(r, gs.ndst, 12)) return;
  if (gs.nloc_only && myc >= gs.split) myc = -1;   // no communication: halo entries add nothing
  const int cnt = __popc(__ballot_sync(gmask, myc >= 0) & gmask);
  const int c_first = __shfl_sync(gmask, myc, 0, G);
  if (myc < 0) {   // lanes past the row's length: a valid source with weight zero
    myc = c_first;
    myw = 0.f;
  }
  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  for (int t = 0; t < cnt; t += UNR) {
    uint4 v[UNR][NCH];
    float w[UNR];
#pragma unroll
    for (int u = 0; u < UNR; ++u) {
      const int c = __shfl_sync(gmask, myc, t + u, G);
      w[u] = __shfl_sync(gmask, myw, t + u, G);
      const bool loc = c < gs.split;
      const bool ok = VARCO_DBG_OK(c, gs.nsrc, 11);
      const uint4 *src = (loc ? gs.b0 : gs.b1s) + (int64_t)c * (loc ? gs.ld0 : gs.ld1) + gl;
#pragma unroll
      for (int i = 0; i < NCH; ++i)
        v[u][i] = (ok && (FULL || gl + i * G < nv)) ? __ldg(src + i * G) : make_uint4(0u, 0u, 0u, 0u);
    }
#pragma unroll
    for (int u = 0; u < UNR; ++u)
#pragma unroll
      for (int i = 0; i < NCH; ++i) {
        float f[V];
        unpack16(v[u][i], f, T());
        fma_row<V>(acc[i], w[u], f);
      }
  }
  finish_row<T, G, NCH, FULL>(acc, r, gl, gmask, 0, nv, nv, stage_rows, O0, ldo0, O1, ldo1, dst_split, accumulate0, hc);
}

// Halo-slot rows of the short class in compressed epochs.  Only the k kept positions of a slot's gradient row
// travel back to the owner, so only those columns of the gathered rows are read: KL lanes per slot, lane m
// owns kept position m (from the call's table) and adds up its column over the slot's entries in entry
// order -- the same fp32 operations the dense kernel performs for that column, hence the same bits.
template <typename T, int KL>
__global__ void __launch_bounds__(256)
    spmm_short_kept_kernel(const int32_t *__restrict__ rec_col, const float *__restrict__ rec_val,
                           const int32_t *__restrict__ rows, int count, const T *__restrict__ A, int64_t lda,
                           int dst_split, HaloCompress hc) {
  typedef typename ElemBits<T>::type E;
  static_assert(KL >= 8, "a record has 8 entries, one per lane");
  const int task = (blockIdx.x * blockDim.x + threadIdx.x) / KL;
  const int gl = threadIdx.x % KL;
  if (task >= count) return;
  const unsigned lane = threadIdx.x % 32;
  const unsigned gmask = (KL == 32) ? 0xFFFFFFFFu : (((1u << KL) - 1u) << (lane & ~(unsigned)(KL - 1)));
  int myc = -1;
  float myw = 0.f;
  if (gl < 8) {
    myc = __ldg(rec_col + (int64_t)task * 8 + gl);
    myw = __ldg(rec_val + (int64_t)task * 8 + gl);
  }
  const int slot = __ldg(rows + task) - dst_split;
  int pos = 0;
  if (gl < hc.k) pos = __ldg(hc.wpos + (int64_t)__ldg(hc.slot_src + slot) * hc.wstride + gl);
  const int cnt = __popc(__ballot_sync(gmask, myc >= 0) & gmask);
  const int c_first = __shfl_sync(gmask, myc, 0, KL);
  if (myc < 0) myc = c_first;   // lanes past the row's length: a valid source with weight zero
  const E *col_base = reinterpret_cast<const E *>(A) + pos;
  float acc = 0.f;
  for (int t = 0; t < cnt; t += 4) {
    E x[4];
    float w[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = __shfl_sync(gmask, myc, t + u, KL);
      w[u] = __shfl_sync(gmask, myw, t + u, KL);
      x[u] = VARCO_DBG_OK(c, dst_split, 11) ? __ldg(col_base + (int64_t)c * lda) : (E)0;
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      float f;
      if (sizeof(E) == 2) f = __uint_as_float((uint32_t)x[u] << 16);
      else f = __uint_as_float((uint32_t)x[u]);
      acc = fmaf(f, w[u], acc);
    }
  }
  if (gl < (int)hc.kstride) {
    E out = (E)0;
    if (gl < hc.k) {
      const T v = ElemTraits<T>::from_f(acc);
      out = *reinterpret_cast<const E *>(&v);
    }
    reinterpret_cast<E *>(hc.packed)[(int64_t)slot * hc.kstride + gl] = out;
  }
}

// Long rows (hubs of a skewed degree distribution): one CTA per (row, panel), every warp takes a
// contiguous share of the entries, partial sums meet in shared memory and are added in warp order.
template <typename T, int G, int NCH, int UNR, bool FULL>
__global__ void __launch_bounds__(256, rows_blocks_per_sm(NCH))
    spmm_hub_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ col, const float *__restrict__ val,
                    RowClass rc, int P, int panels, int nv_panel, GatherSrc gs, T *__restrict__ O0, int64_t ldo0,
                    T *__restrict__ O1, int64_t ldo1, int dst_split, int accumulate0, int nv, HaloCompress hc) {
  extern __shared__ float hub_part[];
  constexpr int V = ElemTraits<T>::kVec;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int nwarps = blockDim.x / 32;
  int pos, panel;
  locate(rc, P, panels, blockIdx.x, pos, panel);
  const int r = __ldg(rc.rows + pos);
  if (r >= gs.row_limit || !VARCO_DBG_OK(r, gs.ndst, 12)) return;
  const int ch_lo = panel * nv_panel;
  const int ch_hi = min(nv, ch_lo + nv_panel);
  const int64_t e0 = rp[r], e1 = gs.nloc_only ? e0 + __ldg(gs.nloc_only + r) : rp[r + 1];
  // the entries are shared out over the warps, and inside a warp over its 32 / G lane groups (narrow rows
  // need fewer than 32 lanes per gathered row); the groups' sums meet by a fixed shuffle tree
  constexpr int kGroups = 32 / G;
  const int gl = lane % G, gi = lane / G;
  const unsigned gmask = (G == 32) ? 0xFFFFFFFFu : (((1u << G) - 1u) << (lane & ~(unsigned)(G - 1)));
  const int64_t shares = (int64_t)nwarps * kGroups;
  const int64_t per = ((e1 - e0 + shares - 1) / shares + G - 1) / G * G;
  const int64_t mine = (int64_t)warp * kGroups + gi;
  const int64_t b0 = e0 + mine * per < e1 ? e0 + mine * per : e1;
  const int64_t b1 = b0 + per < e1 ? b0 + per : e1;
  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  if (b1 > b0)
    accumulate_range<T, G, NCH, UNR, FULL>(col + b0, val + b0, (int)(b1 - b0), gs, ch_lo, ch_hi, gl, gmask, acc);
#pragma unroll
  for (int off = G; off < 32; off <<= 1)
#pragma unroll
    for (int i = 0; i < NCH; ++i)
#pragma unroll
      for (int j = 0; j < V; ++j) acc[i][j] += __shfl_xor_sync(0xFFFFFFFFu, acc[i][j], off);
  const int row_floats = nv_panel * V;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int c = gl + i * G;
    if (gi == 0 && c < nv_panel)
#pragma unroll
      for (int j = 0; j < V; ++j) hub_part[(size_t)warp * row_floats + c * V + j] = acc[i][j];
  }
  __syncthreads();
  if (hc.packed && r >= dst_split) {
    // reduce into the first warp's row, convert in place to the element type, then compress
    typedef typename ElemBits<T>::type E;
    uint4 *srow4 = reinterpret_cast<uint4 *>(hub_part);
    uint4 mine[(NCH * 32 + 255) / 256 + 1];
    int cnt = 0;
    for (int c = threadIdx.x; c < nv; c += blockDim.x) {
      float f[V];
#pragma unroll
      for (int j = 0; j < V; ++j) f[j] = 0.f;
      for (int w = 0; w < nwarps; ++w)
#pragma unroll
        for (int j = 0; j < V; ++j) f[j] += hub_part[(size_t)w * row_floats + c * V + j];
      mine[cnt++] = pack16(f, T());
    }
    __syncthreads();
    cnt = 0;
    for (int c = threadIdx.x; c < nv; c += blockDim.x) srow4[c] = mine[cnt++];
    __syncthreads();
    const int slot = r - dst_split;
    const E *srow = reinterpret_cast<const E *>(srow4);
    E *z = reinterpret_cast<E *>(hc.packed) + (int64_t)slot * hc.kstride;
    if (hc.wpos) {
      const uint16_t *prow = hc.wpos + (int64_t)__ldg(hc.slot_src + slot) * hc.wstride;
      pick_kept<E, V>(srow, prow, z, hc.k, (int)hc.kstride, (int)threadIdx.x, (int)blockDim.x);
      return;
    }
    vperm::RowPerm pm;
    pm.init(hc.lkey, (uint32_t)__ldg(hc.slot_gid + slot), (uint32_t)hc.F, hc.h);
    for (int m = threadIdx.x; m < (int)hc.kstride; m += blockDim.x) z[m] = m < hc.k ? srow[pm.pi((uint32_t)m)] : (E)0;
    return;
  }
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
  gs.nloc_only = a.nloc_only;
  gs.row_limit = a.row_limit > 0 ? a.row_limit : 0x7FFFFFFF;
  gs.nsrc = a.nsrc;
  gs.ndst = a.ndst;
  return gs;
}

template <typename T, int G, int NCH, int UNR>
int launch_hubs(const SpmmArgs &a, cudaStream_t st) {
  if (a.hubs.count == 0) return VARCO_OK;
  constexpr int V = ElemTraits<T>::kVec;
  const size_t row_bytes = (size_t)a.nv_panel * V * sizeof(float);
  int warps = 8;
  while (warps > 1 && warps * row_bytes > 48 * 1024) warps /= 2;
  const dim3 grid((unsigned)(a.hubs.count * a.panels));
  if (a.panels == 1 && a.nv == G * NCH)
    spmm_hub_kernel<T, G, NCH, UNR, true><<<grid, warps * 32, warps * row_bytes, st>>>(
        a.rp, a.col, a.val, a.hubs, a.P, a.panels, a.nv_panel, gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1, a.ldo1,
        a.dst_split, a.accumulate0, a.nv, a.hc);
  else
    spmm_hub_kernel<T, G, NCH, UNR, false><<<grid, warps * 32, warps * row_bytes, st>>>(
        a.rp, a.col, a.val, a.hubs, a.P, a.panels, a.nv_panel, gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1, a.ldo1,
        a.dst_split, a.accumulate0, a.nv, a.hc);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

template <typename T, int G, int NCH, int UNR>
int launch_rows(const SpmmArgs &a, const RowClass &rc, cudaStream_t st) {
  if (rc.count == 0) return VARCO_OK;
  const int threads = 256;
  const int64_t total = (int64_t)rc.count * a.panels * G;
  dim3 grid((unsigned)((total + threads - 1) / threads));
  const size_t smem = a.hc.packed ? (size_t)(threads / G) * a.nv * 16 : 0;
  if (a.panels == 1 && a.nv == G * NCH)
    spmm_kernel<T, G, NCH, UNR, true><<<grid, threads, smem, st>>>(a.rp, a.col, a.val, rc, a.P, a.panels, a.nv_panel,
                                                                   gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1,
                                                                   a.ldo1, a.dst_split, a.accumulate0, a.nv, a.hc);
  else
    spmm_kernel<T, G, NCH, UNR, false><<<grid, threads, smem, st>>>(a.rp, a.col, a.val, rc, a.P, a.panels, a.nv_panel,
                                                                    gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1,
                                                                    a.ldo1, a.dst_split, a.accumulate0, a.nv, a.hc);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

template <typename T, int G, int NCH, int UNR>
int launch_short(const SpmmArgs &a, int first, int count, cudaStream_t st) {
  if (count == 0) return VARCO_OK;
  const int threads = 256;
  dim3 grid((unsigned)(((int64_t)count * G + threads - 1) / threads));
  const size_t smem = a.hc.packed ? (size_t)(threads / G) * a.nv * 16 : 0;
  const int32_t *rc = a.short_col + (int64_t)first * 8;
  const float *rv = a.short_val + (int64_t)first * 8;
  const int32_t *rows = a.shorts.rows + first;
  if (a.nv == G * NCH)
    spmm_short_kernel<T, G, NCH, UNR, true><<<grid, threads, smem, st>>>(
        rc, rv, rows, count, gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1, a.ldo1, a.dst_split, a.accumulate0, a.nv,
        a.hc);
  else
    spmm_short_kernel<T, G, NCH, UNR, false><<<grid, threads, smem, st>>>(
        rc, rv, rows, count, gather_src<T>(a), (T *)a.O0, a.ldo0, (T *)a.O1, a.ldo1, a.dst_split, a.accumulate0, a.nv,
        a.hc);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// Reading single columns pays while the k scattered 32-byte sectors of a gathered row are fewer than the
// sectors of the whole row.
#ifndef VARCO_KEPT_SECTOR_NUM
#define VARCO_KEPT_SECTOR_NUM 1
#define VARCO_KEPT_SECTOR_DEN 1
#endif
template <typename T>
bool kept_columns_pay(const SpmmArgs &a) {
  if (!a.hc.packed || !a.hc.wpos || a.hc.kstride > 32) return false;
  return (int64_t)a.hc.k * 32 * VARCO_KEPT_SECTOR_DEN <= (int64_t)a.nv * 16 * VARCO_KEPT_SECTOR_NUM;
}

template <typename T>
int launch_short_kept(const SpmmArgs &a, int first, int count, cudaStream_t st) {
  if (count == 0) return VARCO_OK;
  const int threads = 256;
  const int32_t *rc = a.short_col + (int64_t)first * 8;
  const float *rv = a.short_val + (int64_t)first * 8;
  const int32_t *rows = a.shorts.rows + first;
  const int KL = a.hc.kstride <= 8 ? 8 : (a.hc.kstride <= 16 ? 16 : 32);
  dim3 grid((unsigned)(((int64_t)count * KL + threads - 1) / threads));
  if (KL == 8)
    spmm_short_kept_kernel<T, 8><<<grid, threads, 0, st>>>(rc, rv, rows, count, (const T *)a.A0, a.lda0, a.dst_split, a.hc);
  else if (KL == 16)
    spmm_short_kept_kernel<T, 16><<<grid, threads, 0, st>>>(rc, rv, rows, count, (const T *)a.A0, a.lda0, a.dst_split, a.hc);
  else
    spmm_short_kept_kernel<T, 32><<<grid, threads, 0, st>>>(rc, rv, rows, count, (const T *)a.A0, a.lda0, a.dst_split, a.hc);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// G/NCH: lanes per row and 16-byte chunks per lane for ordinary rows; GS/NCHS: the same for rows of
// at most a handful of entries, where narrower groups keep more rows in flight per warp.
template <typename T, int G, int NCH, int UNR, int GS, int NCHS, int UNRS>
int launch(const SpmmArgs &a, cudaStream_t st) {
  if (int rc = launch_hubs<T, (G < 8 ? 8 : G), (G < 8 ? 1 : NCH), UNR>(a, st)) return rc;
  if (int rc = launch_rows<T, G, NCH, UNR>(a, a.normal, st)) return rc;
  if (a.panels == 1 && a.short_col) {
    constexpr int GR = GS < 8 ? 8 : GS, NR = GS < 8 ? (NCHS * GS + 7) / 8 : NCHS;
    const int nl = a.short_nlocal, ns = a.shorts.count - nl;
    if (a.row_limit > 0) return launch_short<T, GR, NR, VARCO_SHORT_UNR>(a, 0, nl, st);
    if (ns > 0 && kept_columns_pay<T>(a)) {
      if (int rc = launch_short<T, GR, NR, VARCO_SHORT_UNR>(a, 0, nl, st)) return rc;
      return launch_short_kept<T>(a, nl, ns, st);
    }
    return launch_short<T, GR, NR, VARCO_SHORT_UNR>(a, 0, a.shorts.count, st);
  }
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

// ------------------------------------------------------------------------------------------
// Forward mean aggregation as unweighted sums.  Every entry of row i carries the same weight 1 / deg(i), so the
// source rows are added as they are and the finished row is scaled once.  Per entry the inner loop is one index
// broadcast, one multiply-add for the address, one 16-byte load and one add per element; a bf16 element goes
// into its fp32 accumulator with the mixed-precision add of sm_100 (add.rn.f32.bf16: the bf16 operand is widened
// exactly and the sum rounded once, the result of widening first; measured against unpack + packed fp32 add it
// executes 17 % fewer instructions and the forward stage is 1.2 ms per epoch faster).  A row walks its local entries
// against X and its halo entries against the slot rows in two loops, so no entry needs a base select, and no
// lane ever multiplies a source by a padding weight of zero (a non-finite source row stays where it belongs).
__device__ __forceinline__ void add_chunk(float (&acc)[8], const uint4 &v, __nv_bfloat16) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int j = 0; j < 4; ++j)
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tadd.rn.f32.bf16 %0, lo, %0;\n\tadd.rn.f32.bf16 %1, hi, %1;\n\t}"
        : "+f"(acc[2 * j]), "+f"(acc[2 * j + 1])
        : "r"(w[j]));
}
__device__ __forceinline__ void add_chunk(float (&acc)[4], const uint4 &v, float) {
  asm("{\n\t.reg .b64 a, c, d;\n\tmov.b64 a, {%2, %3};\n\tmov.b64 c, {%0, %1};\n\tadd.rn.f32x2 d, a, c;\n\t"
      "mov.b64 {%0, %1}, d;\n\t}"
      : "+f"(acc[0]), "+f"(acc[1])
      : "r"(v.x), "r"(v.y));
  asm("{\n\t.reg .b64 a, c, d;\n\tmov.b64 a, {%2, %3};\n\tmov.b64 c, {%0, %1};\n\tadd.rn.f32x2 d, a, c;\n\t"
      "mov.b64 {%0, %1}, d;\n\t}"
      : "+f"(acc[2]), "+f"(acc[3])
      : "r"(v.z), "r"(v.w));
}

// acc[i][:] += chunk (gl + i G) of every source col[e], e < len; `base` is the lane's own chunk of row 0.
// The indices of the next G entries are fetched while the gathers of the current ones are in flight, and a
// ragged last batch issues all its loads before the first add (the loads of a batch must never wait on each
// other: a row is a handful of round trips to L2 or DRAM and nothing else).
template <typename T, int G, int NCH, int UNR, bool FULL>
__device__ __forceinline__ void sum_range(const int32_t *__restrict__ colp, int len, const uint4 *__restrict__ base,
                                          int ld, int nv, int gl, unsigned gmask,
                                          float (&acc)[NCH][ElemTraits<T>::kVec], int c_lo, int c_hi) {
  if (len <= 0) return;
  int myc = __ldg(colp + min(gl, len - 1));
  for (int b = 0; b < len; b += G) {
    const int cnt = min(G, len - b);
    const int cur = myc;
    if (b + G < len) myc = __ldg(colp + b + G + min(gl, len - b - G - 1));
    for (int t = 0; t < cnt; t += UNR) {
      uint4 v[UNR][NCH];
#pragma unroll
      for (int u = 0; u < UNR; ++u) {
        if (t + u < cnt) {   // the same for every lane of the group
          const int c = __shfl_sync(gmask, cur, t + u, G);
          const bool ok = VARCO_DBG_OK(c - c_lo, c_hi - c_lo, 11);
          const uint4 *src = base + (int64_t)c * ld;
#pragma unroll
          for (int i = 0; i < NCH; ++i)
            v[u][i] = (ok && (FULL || gl + i * G < nv)) ? __ldg(src + i * G) : make_uint4(0u, 0u, 0u, 0u);
        }
      }
#pragma unroll
      for (int u = 0; u < UNR; ++u)
        if (t + u < cnt) {
#pragma unroll
          for (int i = 0; i < NCH; ++i) add_chunk(acc[i], v[u][i], T());
        }
    }
  }
}

// the first nloc[r] entries of row r read rows of X, the others slot rows (base stored pre-offset by -n rows)
struct SumSrc {
  const uint4 *b0, *b1s;
  int ld0, ld1;
  const int32_t *nloc;
  const float *row_scale;   // 1 / deg(r)
  int n, nsrc;              // rows, rows + halo slots (checked in the debug build)
};

template <typename T, int NCH, bool FULL>
__device__ __forceinline__ void store_scaled(float (&acc)[NCH][ElemTraits<T>::kVec], float s, T *__restrict__ O,
                                             int64_t ldo, int r, int gl, int G, int nv) {
  constexpr int V = ElemTraits<T>::kVec;
  uint4 *dst = reinterpret_cast<uint4 *>(O + (int64_t)r * ldo);
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int ch = gl + i * G;
    if (FULL || ch < nv) {
#pragma unroll
      for (int j = 0; j < V; ++j) acc[i][j] *= s;
      dst[ch] = pack16(acc[i], T());
    }
  }
}

// residency of the sum kernels: eight gathers in flight per lane need 64 registers
constexpr int sum_blocks_per_sm(int nch, int unr) { return nch == 1 ? (unr <= 4 ? 5 : 4) : 1; }

template <typename T, int G, int NCH, int UNR, bool FULL>
__global__ void __launch_bounds__(256, sum_blocks_per_sm(NCH, UNR))
    spmm_sum_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ col, const int32_t *__restrict__ rows,
                    int count, SumSrc ss, T *__restrict__ O, int64_t ldo, int nv) {
  constexpr int V = ElemTraits<T>::kVec;
  const int task = (int)(((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G);
  const int gl = threadIdx.x % G;
  if (task >= count) return;
  const unsigned gmask = group_mask<G>();
  const int r = __ldg(rows + task);
  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  const int64_t e0 = rp[r];
  const int len = (int)(rp[r + 1] - e0);
  const int nl = __ldg(ss.nloc + r);
  if (!VARCO_DBG_OK(r, ss.n, 12)) return;
  sum_range<T, G, NCH, UNR, FULL>(col + e0, nl, ss.b0 + gl, ss.ld0, nv, gl, gmask, acc, 0, ss.n);
  if (len > nl && ss.b1s)   // no halo rows: "no communication", the remote entries add nothing
    sum_range<T, G, NCH, UNR, FULL>(col + e0 + nl, len - nl, ss.b1s + gl, ss.ld1, nv, gl, gmask, acc, ss.n, ss.nsrc);
  store_scaled<T, NCH, FULL>(acc, __ldg(ss.row_scale + r), O, ldo, r, gl, G, nv);
}

// Hubs: one CTA per row.  Every warp (and, for rows narrower than 512 bytes, every lane group of a warp) takes a
// contiguous share of the local and of the halo entries; the partial sums meet by a fixed shuffle tree and
// an ordered shared-memory reduction.
template <typename T, int G, int NCH, int UNR, bool FULL>
__global__ void __launch_bounds__(256, sum_blocks_per_sm(NCH, UNR))
    spmm_sum_hub_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ col,
                        const int32_t *__restrict__ rows, SumSrc ss, T *__restrict__ O, int64_t ldo, int nv) {
  extern __shared__ float hub_part[];
  constexpr int V = ElemTraits<T>::kVec;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int nwarps = blockDim.x / 32;
  const int r = __ldg(rows + blockIdx.x);
  const int64_t e0 = rp[r];
  const int len = (int)(rp[r + 1] - e0);
  const int nl = __ldg(ss.nloc + r);
  constexpr int kGroups = 32 / G;
  const int gl = lane % G, gi = lane / G;
  const unsigned gmask = group_mask<G>();
  const int shares = nwarps * kGroups;
  const int mine = warp * kGroups + gi;
  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  auto share = [&](int total, int &b0, int &b1) {
    const int per = ((total + shares - 1) / shares + G - 1) / G * G;
    b0 = min(total, mine * per);
    b1 = min(total, b0 + per);
  };
  int b0, b1;
  share(nl, b0, b1);
  if (b1 > b0) sum_range<T, G, NCH, UNR, FULL>(col + e0 + b0, b1 - b0, ss.b0 + gl, ss.ld0, nv, gl, gmask, acc, 0, ss.n);
  share(ss.b1s ? len - nl : 0, b0, b1);
  if (b1 > b0)
    sum_range<T, G, NCH, UNR, FULL>(col + e0 + nl + b0, b1 - b0, ss.b1s + gl, ss.ld1, nv, gl, gmask, acc, ss.n, ss.nsrc);
#pragma unroll
  for (int off = G; off < 32; off <<= 1)
#pragma unroll
    for (int i = 0; i < NCH; ++i)
#pragma unroll
      for (int j = 0; j < V; ++j) acc[i][j] += __shfl_xor_sync(0xFFFFFFFFu, acc[i][j], off);
  const int row_floats = nv * V;
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int c = gl + i * G;
    if (gi == 0 && c < nv)
#pragma unroll
      for (int j = 0; j < V; ++j) hub_part[(size_t)warp * row_floats + c * V + j] = acc[i][j];
  }
  __syncthreads();
  const float s = __ldg(ss.row_scale + r);
  uint4 *dst = reinterpret_cast<uint4 *>(O + (int64_t)r * ldo);
  for (int c = threadIdx.x; c < nv; c += blockDim.x) {
    float f[V];
#pragma unroll
    for (int j = 0; j < V; ++j) f[j] = 0.f;
    for (int w = 0; w < nwarps; ++w)
#pragma unroll
      for (int j = 0; j < V; ++j) f[j] += hub_part[(size_t)w * row_floats + c * V + j];
#pragma unroll
    for (int j = 0; j < V; ++j) f[j] *= s;
    dst[c] = pack16(f, T());
  }
}

struct SumArgs {
  const int64_t *rp;
  const int32_t *col;
  RowClass hubs, normal, shorts;
  SumSrc ss;
  void *O;
  int64_t ldo;
  int nv;
};

// G lanes x NCH chunks for hub and ordinary rows; the few rows of at most 8 entries take GS lanes x NCHS chunks
template <typename T, int G, int NCH, int UNR, int GS, int NCHS>
int launch_sum(const SumArgs &a, cudaStream_t st) {
  constexpr int V = ElemTraits<T>::kVec;
  const int threads = 256;
  if (a.hubs.count) {
    constexpr int GH = G < 8 ? 8 : G, NH = G < 8 ? 1 : NCH;
    const size_t row_bytes = (size_t)a.nv * V * sizeof(float);
    int warps = 8;
    while (warps > 1 && warps * row_bytes > 48 * 1024) warps /= 2;
    if (a.nv == GH * NH)
      spmm_sum_hub_kernel<T, GH, NH, UNR, true><<<a.hubs.count, warps * 32, warps * row_bytes, st>>>(
          a.rp, a.col, a.hubs.rows, a.ss, (T *)a.O, a.ldo, a.nv);
    else
      spmm_sum_hub_kernel<T, GH, NH, UNR, false><<<a.hubs.count, warps * 32, warps * row_bytes, st>>>(
          a.rp, a.col, a.hubs.rows, a.ss, (T *)a.O, a.ldo, a.nv);
    VARCO_KERNEL_LAUNCHED();
  }
  if (a.normal.count) {
    const unsigned grid = (unsigned)(((int64_t)a.normal.count * G + threads - 1) / threads);
    if (a.nv == G * NCH)
      spmm_sum_kernel<T, G, NCH, UNR, true><<<grid, threads, 0, st>>>(a.rp, a.col, a.normal.rows, a.normal.count, a.ss,
                                                                     (T *)a.O, a.ldo, a.nv);
    else
      spmm_sum_kernel<T, G, NCH, UNR, false><<<grid, threads, 0, st>>>(a.rp, a.col, a.normal.rows, a.normal.count, a.ss,
                                                                      (T *)a.O, a.ldo, a.nv);
    VARCO_KERNEL_LAUNCHED();
  }
  if (a.shorts.count) {
    const unsigned grid = (unsigned)(((int64_t)a.shorts.count * GS + threads - 1) / threads);
    if (a.nv == GS * NCHS)
      spmm_sum_kernel<T, GS, NCHS, 1, true><<<grid, threads, 0, st>>>(a.rp, a.col, a.shorts.rows, a.shorts.count, a.ss,
                                                                     (T *)a.O, a.ldo, a.nv);
    else
      spmm_sum_kernel<T, GS, NCHS, 1, false><<<grid, threads, 0, st>>>(a.rp, a.col, a.shorts.rows, a.shorts.count, a.ss,
                                                                      (T *)a.O, a.ldo, a.nv);
    VARCO_KERNEL_LAUNCHED();
  }
  return VARCO_OK;
}

template <typename T>
int dispatch_sum(const SumArgs &a, cudaStream_t st) {
  const int w = a.nv;
  if (w <= 4) return launch_sum<T, 4, 1, 4, 4, 1>(a, st);
  if (w <= 8) return launch_sum<T, 8, 1, 4, 4, 2>(a, st);
  if (w <= 16) return launch_sum<T, 16, 1, 8, 4, 4>(a, st);
  if (w <= 32) return launch_sum<T, 32, 1, 8, 8, 4>(a, st);
  if (w <= 64) return launch_sum<T, 32, 2, 4, 16, 4>(a, st);
  if (w <= 96) return launch_sum<T, 32, 3, 2, 16, 6>(a, st);
  if (w <= 128) return launch_sum<T, 32, 4, 2, 32, 4>(a, st);
  if (w <= 256) return launch_sum<T, 32, 8, 1, 32, 8>(a, st);
  return VARCO_UNSUPPORTED;
}

// ------------------------------------------------------------------------------------------
// Forward aggregation with SPARSE halo rows (compressed epochs).  A remote neighbour contributes
// only its k kept values, so its slot is stored as k (value, position) pairs and the row's
// remote part is accumulated by scattering those pairs into a shared-memory fp32 row; the local
// part goes through the dense register path above.  Entry order is unchanged (local entries
// first, then halo slots ascending).
template <typename T> struct SparsePair;
template <> struct SparsePair<float> {
  typedef uint2 type;
  __device__ static __forceinline__ float val(uint2 p) { return __uint_as_float(p.x); }
  __device__ static __forceinline__ int pos(uint2 p) { return (int)p.y; }
};
template <> struct SparsePair<__nv_bfloat16> {
  typedef uint32_t type;
  __device__ static __forceinline__ float val(uint32_t p) { return __uint_as_float(p << 16); }
  __device__ static __forceinline__ int pos(uint32_t p) { return (int)(p >> 16); }
};

// halo entries [0, len) of one row: sacc[pos] += w * value for the k pairs of every entry's slot
// (SUM: every weight is 1 and the weights are not read; the caller scales the finished row)
template <typename T, int G, bool SUM = false>
__device__ __forceinline__ void accumulate_sparse(const int32_t *__restrict__ colp, const float *__restrict__ valp,
                                                  int len, const typename SparsePair<T>::type *__restrict__ pairs,
                                                  int64_t pstride, int k, int split, float *sacc, int gl,
                                                  unsigned gmask, int nslots, int width) {
  typedef typename SparsePair<T>::type P;
  for (int base = 0; base < len; base += G) {
    const int cnt = min(G, len - base);
    const int mine = base + min(gl, cnt - 1);
    const int myc = __ldg(colp + mine);
    const float myw = SUM ? 1.f : (gl < cnt ? __ldg(valp + mine) : 0.f);
    if (k <= G) {
      // one pair per lane and entry: fetch kAhead entries ahead of the shared-memory updates
      constexpr int kAhead = G >= 8 ? 8 : 4;
      for (int t = 0; t < cnt; t += kAhead) {
        P p[kAhead];
        float w[kAhead];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
          const int slot = __shfl_sync(gmask, myc, t + u, G) - split;
          // past the end of a ragged batch the lane re-reads the last entry with weight 0
          w[u] = SUM ? (t + u < cnt ? 1.f : 0.f) : __shfl_sync(gmask, myw, t + u, G);
          p[u] = VARCO_DBG_OK(slot, nslots, 11) ? __ldg(pairs + (int64_t)slot * pstride + min(gl, k - 1)) : P();
        }
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
          if (gl < k && VARCO_DBG_OK(SparsePair<T>::pos(p[u]), width, 13)) {
            if (SUM) {
              if (w[u] != 0.f) sacc[SparsePair<T>::pos(p[u])] += SparsePair<T>::val(p[u]);
            } else {
              sacc[SparsePair<T>::pos(p[u])] += w[u] * SparsePair<T>::val(p[u]);
            }
          }
          __syncwarp(gmask);
        }
      }
    } else {
      for (int t = 0; t < cnt; ++t) {
        const int slot = __shfl_sync(gmask, myc, t, G) - split;
        const float w = SUM ? 1.f : __shfl_sync(gmask, myw, t, G);
        const P *pr = pairs + (int64_t)slot * pstride;
        if (VARCO_DBG_OK(slot, nslots, 11))
          for (int m = gl; m < k; m += G) {
            const P q = __ldg(pr + m);
            if (VARCO_DBG_OK(SparsePair<T>::pos(q), width, 13)) sacc[SparsePair<T>::pos(q)] += w * SparsePair<T>::val(q);
          }
        __syncwarp(gmask);
      }
    }
  }
}

// One group per row (normal and short classes).  Shared memory: F floats per group.
// SUM (mean aggregation): the local rows are added unweighted, the pairs likewise, and the finished row is
// scaled by 1 / deg once.
// The group is as narrow as the kept count allows (8 lanes for k <= 8, 16 for k <= 16): a pair update occupies k
// lanes of a group, so a 32-lane group at k = 4 would leave seven lanes in eight idle through the remote part,
// which is most of the entries on a 16-way partition.
// (eight pairs in flight per lane: the one-chunk kernels need a few registers more than five resident blocks leave)
constexpr int sparse_blocks_per_sm(int nch) { return nch == 1 ? 4 : (nch <= 4 ? 3 : 1); }

template <typename T, int G, int NCH, int UNR, bool FULL, bool SUM>
__global__ void __launch_bounds__(256, sparse_blocks_per_sm(NCH))
    spmm_sparse_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ nloc,
                       const int32_t *__restrict__ col, const float *__restrict__ val, RowClass rc, GatherSrc gs,
                       const typename SparsePair<T>::type *__restrict__ pairs, int64_t pstride, int k,
                       const float *__restrict__ row_scale, T *__restrict__ O, int64_t ldo, int nv) {
  extern __shared__ float sparse_acc[];
  constexpr int V = ElemTraits<T>::kVec;
  const int task = (blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int grp = threadIdx.x / G, gl = threadIdx.x % G;
  const unsigned gmask = group_mask<G>();
  float *sacc = sparse_acc + (size_t)grp * nv * V;
  if (task >= rc.count) return;
  for (int c = gl; c < nv * V; c += G) sacc[c] = 0.f;
  const int r = __ldg(rc.rows + task);
  const int64_t e0 = rp[r];
  const int len = (int)(rp[r + 1] - e0);
  const int nl = __ldg(nloc + r);
  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  __syncwarp(gmask);
  if (nl > 0) {
    if (SUM)
      sum_range<T, G, NCH, UNR, FULL>(col + e0, nl, gs.b0 + gl, gs.ld0, nv, gl, gmask, acc, 0, gs.split);
    else
      accumulate_range<T, G, NCH, UNR, FULL>(col + e0, val + e0, nl, gs, 0, nv, gl, gmask, acc);
  }
  if (len > nl)
    accumulate_sparse<T, G, SUM>(col + e0 + nl, val + e0 + nl, len - nl, pairs, pstride, k, gs.split, sacc, gl, gmask,
                                 gs.nsrc - gs.split, nv * V);
  const float scale = SUM ? __ldg(row_scale + r) : 1.f;
  uint4 *dst = reinterpret_cast<uint4 *>(O + (int64_t)r * ldo);
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int ch = gl + i * G;
    if (FULL || ch < nv) {
#pragma unroll
      for (int j = 0; j < V; ++j) {
        acc[i][j] += sacc[ch * V + j];
        if (SUM) acc[i][j] *= scale;
      }
      dst[ch] = pack16(acc[i], T());
    }
  }
}

// Hubs: one CTA per row; every warp takes a contiguous share of the local and of the halo entries and
// owns one shared-memory row; the rows are added in warp order.
template <typename T, int NCH, int GK, bool FULL>
__global__ void __launch_bounds__(256, sparse_blocks_per_sm(NCH))
    spmm_sparse_hub_kernel(const int64_t *__restrict__ rp, const int32_t *__restrict__ nloc,
                           const int32_t *__restrict__ col, const float *__restrict__ val, RowClass rc, GatherSrc gs,
                           const typename SparsePair<T>::type *__restrict__ pairs, int64_t pstride, int k,
                           T *__restrict__ O, int64_t ldo, int nv) {
  extern __shared__ float sparse_acc[];
  constexpr int V = ElemTraits<T>::kVec;
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  const int nwarps = blockDim.x / 32;
  const int rowf = nv * V;
  // the halo entries are walked by groups of GK lanes (GK >= k where k <= 32), every group with a row of its own
  constexpr int kSub = 32 / GK;
  const int gi = lane / GK, gl = lane % GK;
  float *wacc = sparse_acc + (size_t)warp * kSub * rowf;   // the warp's kSub rows; the first also takes the local sums
  float *sacc = wacc + (size_t)gi * rowf;
  for (int c = lane; c < kSub * rowf; c += 32) wacc[c] = 0.f;
  const int r = __ldg(rc.rows + blockIdx.x);
  const int64_t e0 = rp[r];
  const int len = (int)(rp[r + 1] - e0);
  const int nl = __ldg(nloc + r);
  float acc[NCH][V];
#pragma unroll
  for (int i = 0; i < NCH; ++i)
#pragma unroll
    for (int j = 0; j < V; ++j) acc[i][j] = 0.f;
  __syncwarp();
  auto share = [&](int total, int &b0, int &b1) {
    const int per = ((total + nwarps - 1) / nwarps + 31) / 32 * 32;
    b0 = min(total, warp * per);
    b1 = min(total, b0 + per);
  };
  int b0, b1;
  share(nl, b0, b1);
  if (b1 > b0) accumulate_range<T, 32, NCH, 4, FULL>(col + e0 + b0, val + e0 + b0, b1 - b0, gs, 0, nv, lane, 0xFFFFFFFFu, acc);
  {
    const int total = len - nl, shares = nwarps * kSub, mine = warp * kSub + gi;
    const int per = ((total + shares - 1) / shares + GK - 1) / GK * GK;
    b0 = min(total, mine * per);
    b1 = min(total, b0 + per);
  }
  if (b1 > b0)
    accumulate_sparse<T, GK>(col + e0 + nl + b0, val + e0 + nl + b0, b1 - b0, pairs, pstride, k, gs.split, sacc, gl,
                             group_mask<GK>(), gs.nsrc - gs.split, nv * V);
  __syncwarp();
#pragma unroll
  for (int i = 0; i < NCH; ++i) {
    const int ch = lane + i * 32;
    if (FULL || ch < nv)
#pragma unroll
      for (int j = 0; j < V; ++j) wacc[ch * V + j] += acc[i][j];
  }
  __syncthreads();
  uint4 *dst = reinterpret_cast<uint4 *>(O + (int64_t)r * ldo);
  for (int ch = threadIdx.x; ch < nv; ch += blockDim.x) {
    float f[V];
#pragma unroll
    for (int j = 0; j < V; ++j) f[j] = 0.f;
    for (int w = 0; w < nwarps * kSub; ++w)
#pragma unroll
      for (int j = 0; j < V; ++j) f[j] += sparse_acc[(size_t)w * rowf + ch * V + j];
    dst[ch] = pack16(f, T());
  }
}

template <typename T, int G, int NCH, int UNR>
int launch_sparse_rows(const SpmmArgs &a, const RowClass &rc, const int32_t *nloc, const void *pairs, int64_t pstride,
                       int k, const float *row_scale, cudaStream_t st) {
  if (rc.count == 0) return VARCO_OK;
  constexpr int V = ElemTraits<T>::kVec;
  typedef typename SparsePair<T>::type P;
  const int threads = 256;
  const size_t smem = (size_t)(threads / G) * a.nv * V * sizeof(float);
  dim3 grid((unsigned)(((int64_t)rc.count * G + threads - 1) / threads));
  const bool full = a.nv == G * NCH;
#define VARCO_SPARSE_LAUNCH(FULL, SUM)                                                                              \
  spmm_sparse_kernel<T, G, NCH, UNR, FULL, SUM><<<grid, threads, smem, st>>>(                                       \
      a.rp, nloc, a.col, a.val, rc, gather_src<T>(a), (const P *)pairs, pstride, k, row_scale, (T *)a.O0, a.ldo0, a.nv)
  if (row_scale) {
    if (full)
      VARCO_SPARSE_LAUNCH(true, true);
    else
      VARCO_SPARSE_LAUNCH(false, true);
  } else {
    if (full)
      VARCO_SPARSE_LAUNCH(true, false);
    else
      VARCO_SPARSE_LAUNCH(false, false);
  }
#undef VARCO_SPARSE_LAUNCH
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

template <typename T, int NCH, int GK>
int launch_sparse_hubs(const SpmmArgs &a, const int32_t *nloc, const void *pairs, int64_t pstride, int k,
                       cudaStream_t st) {
  if (a.hubs.count == 0) return VARCO_OK;
  constexpr int V = ElemTraits<T>::kVec;
  typedef typename SparsePair<T>::type P;
  const size_t row_bytes = (size_t)(32 / GK) * a.nv * V * sizeof(float);   // per warp: one row per group of GK lanes
  int warps = 8;
  while (warps > 1 && warps * row_bytes > 48 * 1024) warps /= 2;
  if (warps * row_bytes > 48 * 1024) return VARCO_UNSUPPORTED;
  if (a.nv == 32 * NCH)
    spmm_sparse_hub_kernel<T, NCH, GK, true><<<a.hubs.count, warps * 32, warps * row_bytes, st>>>(
        a.rp, nloc, a.col, a.val, a.hubs, gather_src<T>(a), (const P *)pairs, pstride, k, (T *)a.O0, a.ldo0, a.nv);
  else
    spmm_sparse_hub_kernel<T, NCH, GK, false><<<a.hubs.count, warps * 32, warps * row_bytes, st>>>(
        a.rp, nloc, a.col, a.val, a.hubs, gather_src<T>(a), (const P *)pairs, pstride, k, (T *)a.O0, a.ldo0, a.nv);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// Lanes per row for the ordinary class / the short class, by row width in chunks (nv <= 64 only) and by the
// kept count; UNR x NCH 16-byte gathers of the local part in flight per lane.  row_scale != nullptr: mean
// aggregation as unweighted sums (hub rows keep the weighted kernel: the same sums, scaled entry by entry).
template <typename T>
int dispatch_sparse(const SpmmArgs &a, const int32_t *nloc, const void *pairs, int64_t pstride, int k,
                    const float *row_scale, cudaStream_t st) {
  const int w = a.nv;
#define VARCO_SPARSE(G, NCH, UNR, GS, NCHS)                                                                     \
  do {                                                                                                          \
    if (int rc = launch_sparse_hubs<T, (NCH * G + 31) / 32, G>(a, nloc, pairs, pstride, k, st)) return rc;      \
    if (int rc = launch_sparse_rows<T, G, NCH, UNR>(a, a.normal, nloc, pairs, pstride, k, row_scale, st)) return rc; \
    return launch_sparse_rows<T, GS, NCHS, 2>(a, a.shorts, nloc, pairs, pstride, k, row_scale, st);             \
  } while (0)
  if (w <= 8) VARCO_SPARSE(8, 1, 4, 8, 1);
  if (w <= 16) {
    if (k <= 8) VARCO_SPARSE(8, 2, 4, 8, 2);
    VARCO_SPARSE(16, 1, 4, 8, 2);
  }
  if (w <= 32) {
    if (k <= 8) VARCO_SPARSE(8, 4, 2, 8, 4);
    if (k <= 16) VARCO_SPARSE(16, 2, 4, 8, 4);
    VARCO_SPARSE(32, 1, 4, 8, 4);
  }
  if (w <= 64) {
    if (k <= 16) VARCO_SPARSE(16, 4, 2, 16, 4);
    VARCO_SPARSE(32, 2, 4, 16, 4);
  }
#undef VARCO_SPARSE
  return VARCO_UNSUPPORTED;
}

}  // namespace

// Forward aggregation: Agg[r] = sum_e val[e] * (col[e] < n ? X[col[e]] : Xhalo[col[e] - n]).
// Xhalo == nullptr: nothing was communicated, the halo entries contribute zero vectors.
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
  a.nsrc = (int)(pl->n + pl->H);
  a.ndst = (int)pl->n;
  a.O0 = Agg;
  a.ldo0 = ldagg;
  a.O1 = nullptr;
  a.ldo1 = 0;
  a.dst_split = (int)pl->n;
  a.accumulate0 = 0;
  a.nv = nv;
  a.panels = 1;
  a.nv_panel = nv;
  // Optional feature panels (off unless an L2 budget is set on the plan): split the feature row so that what
  // one partition gathers from fits the budget.  Measured on this part it does not pay, neither on the
  // products-like graph (5 uses per source row) nor on the dense one (60 uses): the kernels are bound by
  // instruction issue at about 6-7 TB/s of gathered bytes, below what L2 could deliver, so the extra index
  // passes only add work.  Kept as a knob for other graphs and parts.
  const int64_t footprint = pl->max_part_sources * (int64_t)nv * 16;
  if (pl->l2_budget > 0 && footprint > pl->l2_budget && nv > 4) {
    int panels = (int)((footprint + pl->l2_budget - 1) / pl->l2_budget);
    int nvp = (nv + panels - 1) / panels;
    nvp = (nvp + 3) / 4 * 4;              // whole 64-byte units
    if (nvp < 4) nvp = 4;
    a.nv_panel = nvp;
    a.panels = (nv + nvp - 1) / nvp;
  }
  a.short_col = pl->d.short_f_col;
  a.short_val = pl->d.short_f_val;
  a.short_nlocal = (int)pl->short_f.size();
  if (!Xhalo) {   // no communication: local entries only
    a.A1 = X;
    a.lda1 = ldx;
    a.nloc_only = pl->d.nloc;
    a.panels = 1;
    a.nv_panel = nv;
    ldh = ldx;
  }
  if (a.panels == 1 && !pl->row_scale.empty() && (ldx % V) == 0 && (ldh % V) == 0) {
    // mean aggregation: unweighted sums, one scale per finished row
    SumArgs u{};
    u.rp = a.rp;
    u.col = a.col;
    u.hubs = a.hubs;
    u.normal = a.normal;
    u.shorts = a.shorts;
    u.ss.b0 = reinterpret_cast<const uint4 *>(X);
    u.ss.ld0 = (int)(ldx / V);
    u.ss.ld1 = (int)(ldh / V);
    u.ss.b1s = Xhalo ? reinterpret_cast<const uint4 *>(Xhalo) - (int64_t)pl->n * u.ss.ld1 : nullptr;
    u.ss.nloc = pl->d.nloc;
    u.ss.row_scale = pl->d.row_scale;
    u.ss.n = (int)pl->n;
    u.ss.nsrc = (int)(pl->n + pl->H);
    u.O = Agg;
    u.ldo = ldagg;
    u.nv = nv;
    return dt == VARCO_F32 ? dispatch_sum<float>(u, st) : dispatch_sum<__nv_bfloat16>(u, st);
  }
  return dt == VARCO_F32 ? dispatch<float>(a, st) : dispatch<__nv_bfloat16>(a, st);
}

bool varco_spmm_sparse_supported(int F, int k, varco_dtype_t dt) {
  const int V = dt == VARCO_F32 ? 4 : 8;
  const int nv = (F + V - 1) / V;
  // pays (measured) when a remote row shrinks to at most an eighth (at a quarter the shared-memory updates cost
  // more than the halved gathers save); positions must fit the pair format;
  // 32 groups of nv * V floats must fit the default shared-memory window
  return nv <= 64 && 8 * k <= F && F <= 65535 && (size_t)32 * nv * V * sizeof(float) <= 48 * 1024;
}

// Forward aggregation when the halo slots hold (value, position) pairs instead of dense rows.
int varco_launch_spmm_fwd_sparse(const varco_plan *pl, const void *X, int64_t ldx, const void *pairs, int64_t pstride,
                                 int k, int F, varco_dtype_t dt, void *Agg, int64_t ldagg, cudaStream_t st) {
  const int V = dt == VARCO_F32 ? 4 : 8;
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
  a.A1 = X;
  a.lda1 = ldx;
  a.src_split = (int)pl->n;
  a.nsrc = (int)(pl->n + pl->H);
  a.ndst = (int)pl->n;
  a.O0 = Agg;
  a.ldo0 = ldagg;
  a.dst_split = (int)pl->n;
  a.nv = (F + V - 1) / V;
  a.panels = 1;
  a.nv_panel = a.nv;
  const float *row_scale = (!pl->row_scale.empty() && ldx % V == 0) ? pl->d.row_scale : nullptr;
  return dt == VARCO_F32 ? dispatch_sparse<float>(a, pl->d.nloc, pairs, pstride, k, row_scale, st)
                         : dispatch_sparse<__nv_bfloat16>(a, pl->d.nloc, pairs, pstride, k, row_scale, st);
}

// Transposed aggregation: for a source u, g_u = sum over the rows i that use it of s_iu dAgg[i];
// u < n lands in dX[u] (added to what is there when `accumulate`), u >= n in Ghalo[u - n].
// Every source of partition q is used by rows of q only, so the gathered set of a partition is
// its own block of dAgg: panels are chosen so that this block stays in L2.
// With `packed` set (k < F) the halo-slot rows are compressed in the kernels' epilogue with the forward's
// key and only the k kept values of every slot are written (slot order, stride kstride).
int varco_launch_spmm_bwd(const varco_plan *pl, const void *dAgg, int64_t ldd, int F, varco_dtype_t dt, void *dX,
                          int64_t ldx, int accumulate, void *Ghalo, int64_t ldh, void *packed, int64_t kstride, int k,
                          varco_key_t key, const uint16_t *wpos, int64_t wstride, cudaStream_t st) {
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
  a.nsrc = (int)pl->n;
  a.ndst = (int)(pl->n + pl->H);
  a.O0 = dX;
  a.ldo0 = ldx;
  a.O1 = Ghalo;
  a.ldo1 = ldh;
  a.dst_split = (int)pl->n;
  a.accumulate0 = accumulate;
  a.nv = nv;
  a.panels = 1;
  a.nv_panel = nv;
  a.short_col = pl->d.short_t_col;
  a.short_val = pl->d.short_t_val;
  a.short_nlocal = (int)pl->short_t_nlocal;
  if (!Ghalo && !packed) a.row_limit = (int)pl->n;   // no communication: the halo-slot rows are not computed
  if (packed)
    a.hc = HaloCompress{packed, kstride, k, F, vperm::half_bits(F), vperm::layer_key(key), pl->d.slot_gid, wpos, wstride,
                        pl->d.slot_src};
  return dt == VARCO_F32 ? dispatch<float>(a, st) : dispatch<__nv_bfloat16>(a, st);
}

// debug build: this translation unit's word of failed index checks (0 in a release build)
VARCO_DEFINE_DEBUG_READER(varco_debug_word_spmm)
