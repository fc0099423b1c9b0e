// Halo exchange kernels: gather + compress, decompress + scatter, and their backward mirrors.
//
// Algorithm 1 of the paper, second and third step: every partition compresses the activations
// of its boundary rows and sends them to the adjacent partitions, which decompress them.  The
// compressor keeps k = ceil(F / c) values of a row at keyed pseudo-random positions and the
// decoder puts them back in place with zeros elsewhere (Definition 1; appendix "Compression
// Mechanism").  The backward pass returns the halo-row gradients through the same compressor.
// At full communication (k == F) nothing is dropped and rows travel in their natural order, so
// the exchange is a plain row copy.
//
// The kernels are data movement (bit-exact) plus the integer permutation.  A group of G lanes
// (8, 16 or 32, by row width) owns one row, so that a warp keeps several rows in flight; rows are
// staged in shared memory with 128-bit accesses and permuted there; packed rows are read and
// written with 128-bit accesses whenever their stride allows it.
//
// Packed buffers come in two orders.  The layer path writes a copy straight to the position of
// its halo slot at the receiver ("receive order": destination, owner, id), which folds the
// exchange step into the write address.  The stand-alone compress / decompress entry points use
// the sender's order (owner, destination, id) on the packed side.
#include "device_common.cuh"
#include "kernels.h"

namespace {

template <typename E> struct VecOf { static constexpr int kVec = 16 / (int)sizeof(E); };

__device__ __forceinline__ uint32_t wire_pos(const vperm::RowPerm &pm, int m, bool identity) {
  return identity ? (uint32_t)m : pm.pi((uint32_t)m);
}

// ------------------------------------------------------------------------------------------
// Full communication, sender side: copy every unique boundary row into the halo slot of every
// partition that uses it.  Works on 16-byte chunks, any element type.
template <int G>
__global__ void __launch_bounds__(256) gather_copy_kernel(const uint4 *__restrict__ X, int64_t ldx4, int nv,
                                                          const int32_t *__restrict__ brow,
                                                          const int32_t *__restrict__ brow_ptr,
                                                          const int32_t *__restrict__ brow_slot, int nb,
                                                          uint4 *__restrict__ Xhalo, int64_t ldh4) {
  const int b = (blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int gl = threadIdx.x % G;
  if (b >= nb) return;
  const int r = brow[b];
  const int s0 = brow_ptr[b], s1 = brow_ptr[b + 1];
  const uint4 *src = X + (int64_t)r * ldx4;
  for (int v0 = 0; v0 < nv; v0 += 4 * G) {
    uint4 val[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int v = v0 + u * G + gl;
      val[u] = v < nv ? __ldg(src + v) : make_uint4(0u, 0u, 0u, 0u);
    }
    for (int s = s0; s < s1; ++s) {
      uint4 *dst = Xhalo + (int64_t)brow_slot[s] * ldh4;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int v = v0 + u * G + gl;
        if (v < nv) dst[v] = val[u];
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Sender side, general k.  One group per unique boundary row: the row is read once, its k kept
// values are selected once and written to the copy of every destination partition.
template <typename E, int G>
__global__ void __launch_bounds__(256) compress_rows_kernel(const E *__restrict__ X, int64_t ld, int F, int k, int h,
                                                            uint64_t lkey, const int32_t *__restrict__ brow,
                                                            const int32_t *__restrict__ brow_ptr,
                                                            const int32_t *__restrict__ brow_slot,
                                                            const int32_t *__restrict__ slot_sendpos,
                                                            const int32_t *__restrict__ row_gid, int nb,
                                                            E *__restrict__ packed, int64_t kstride,
                                                            uint16_t *__restrict__ wpos, int64_t wstride) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = VecOf<E>::kVec;
  const int nv = (F + V - 1) / V;      // chunks of a row
  const int kv = (k + V - 1) / V;      // chunks of a packed row
  const int grp = threadIdx.x / G, gl = threadIdx.x % G;
  const int b = blockIdx.x * (blockDim.x / G) + grp;
  if (b >= nb) return;
  const unsigned gmask = group_mask<G>();
  uint4 *srow4 = smem_u4 + (size_t)grp * (nv + kv);
  uint4 *zrow4 = srow4 + nv;
  const E *srow = reinterpret_cast<const E *>(srow4);
  E *zrow = reinterpret_cast<E *>(zrow4);
  const int r = brow[b];
  const int s0 = brow_ptr[b], s1 = brow_ptr[b + 1];
  const uint4 *src = reinterpret_cast<const uint4 *>(X + (int64_t)r * ld);
  for (int v = gl; v < nv; v += G) srow4[v] = __ldg(src + v);
  vperm::RowPerm pm;
  init_perm<G>(pm, lkey, (uint32_t)row_gid[r], (uint32_t)F, h, gl, gmask);
  const bool identity = k == F;
  __syncwarp(gmask);
  for (int m = gl; m < kv * V; m += G) {
    E v = (E)0;
    if (m < k) {
      const uint32_t p = wire_pos(pm, m, identity);
      v = srow[p];
      if (wpos) wpos[(int64_t)r * wstride + m] = (uint16_t)p;   // kept for the receivers of this call
    }
    zrow[m] = v;
  }
  __syncwarp(gmask);
  const bool vec = ((kstride * (int64_t)sizeof(E)) & 15) == 0;
  for (int s = s0; s < s1; ++s) {
    const int slot = brow_slot[s];
    const int64_t pos = slot_sendpos ? (int64_t)slot_sendpos[slot] : (int64_t)slot;
    E *dst = packed + pos * kstride;
    if (vec) {
      uint4 *dst4 = reinterpret_cast<uint4 *>(dst);
      for (int v = gl; v < kv; v += G) dst4[v] = zrow4[v];
    } else {
      for (int m = gl; m < k; m += G) dst[m] = zrow[m];
    }
  }
}

// ------------------------------------------------------------------------------------------
// Receiver side.  One group per halo slot: the k received values are put back at their
// positions in a zeroed row, which is then written out densely.
template <typename E, int G>
__global__ void __launch_bounds__(256) decompress_slots_kernel(const E *__restrict__ packed, int64_t kstride, int F,
                                                               int k, int h, uint64_t lkey,
                                                               const int32_t *__restrict__ slot_gid,
                                                               const int32_t *__restrict__ slot_sendpos, int H,
                                                               E *__restrict__ Xhalo, int64_t ld,
                                                               const uint16_t *__restrict__ wpos, int64_t wstride,
                                                               const int32_t *__restrict__ slot_src) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = VecOf<E>::kVec;
  const int nv = (F + V - 1) / V;
  const int kv = (k + V - 1) / V;
  const int grp = threadIdx.x / G, gl = threadIdx.x % G;
  const int slot = blockIdx.x * (blockDim.x / G) + grp;
  if (slot >= H) return;
  const unsigned gmask = group_mask<G>();
  uint4 *srow4 = smem_u4 + (size_t)grp * (nv + kv);
  uint4 *zrow4 = srow4 + nv;
  E *srow = reinterpret_cast<E *>(srow4);
  E *zrow = reinterpret_cast<E *>(zrow4);
  const int64_t pos = slot_sendpos ? (int64_t)slot_sendpos[slot] : (int64_t)slot;
  const E *z = packed + pos * kstride;
  const bool vec = ((kstride * (int64_t)sizeof(E)) & 15) == 0;
  if (vec) {
    const uint4 *z4 = reinterpret_cast<const uint4 *>(z);
    for (int v = gl; v < kv; v += G) zrow4[v] = __ldg(z4 + v);
  } else {
    for (int m = gl; m < k; m += G) zrow[m] = z[m];
  }
  for (int v = gl; v < nv; v += G) srow4[v] = make_uint4(0u, 0u, 0u, 0u);
  if (wpos) {
    const uint16_t *prow = wpos + (int64_t)slot_src[slot] * wstride;
    __syncwarp(gmask);
    for (int m = gl; m < k; m += G) srow[__ldg(prow + m)] = zrow[m];
  } else {
    vperm::RowPerm pm;
    init_perm<G>(pm, lkey, (uint32_t)slot_gid[slot], (uint32_t)F, h, gl, gmask);
    const bool identity = k == F;
    __syncwarp(gmask);
    for (int m = gl; m < k; m += G) srow[wire_pos(pm, m, identity)] = zrow[m];
  }
  __syncwarp(gmask);
  uint4 *dst = reinterpret_cast<uint4 *>(Xhalo + (int64_t)slot * ld);
  for (int v = gl; v < nv; v += G) dst[v] = srow4[v];
}

// ------------------------------------------------------------------------------------------
// Receiver side of the layer path, walked by source row.  Every destination of one boundary row uses
// the same kept positions, so a group takes one unique boundary row: the staging row is zeroed once and
// the copy of every destination is put in place and written out in turn (each copy overwrites exactly
// the positions of the one before).  A lane owns KPL 16-byte chunks of the packed rows; it reads the
// positions of its values once per boundary row (16-byte reads of the call's table, kept in registers)
// and fetches its chunks of several destinations' copies before the first is used, so a copy costs
// V 16-bit shared-memory stores per chunk, the row's read-out and its stores to the slot.
template <typename E, int G, int KPL>
__global__ void __launch_bounds__(256) decompress_brows_kernel(const E *__restrict__ packed, int64_t kstride, int F,
                                                               int k, const int32_t *__restrict__ brow,
                                                               const int32_t *__restrict__ brow_ptr,
                                                               const int32_t *__restrict__ brow_slot, int nb,
                                                               E *__restrict__ Xhalo, int64_t ld,
                                                               const uint16_t *__restrict__ wpos, int64_t wstride) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = VecOf<E>::kVec;
  constexpr int kAhead = KPL == 1 ? 4 : 2;
  const int nv = (F + V - 1) / V;
  const int kv = (int)(kstride / V);     // <= G * KPL
  const int grp = threadIdx.x / G, gl = threadIdx.x % G;
  const int b = blockIdx.x * (blockDim.x / G) + grp;
  if (b >= nb) return;
  const unsigned gmask = group_mask<G>();
  uint4 *srow4 = smem_u4 + (size_t)grp * nv;
  E *srow = reinterpret_cast<E *>(srow4);
  const int r = brow[b];
  const int s0 = brow_ptr[b], s1 = brow_ptr[b + 1];
  const uint16_t *prow = wpos + (int64_t)r * wstride;
  const uint4 *packed4 = reinterpret_cast<const uint4 *>(packed);
  const int64_t kstride4 = kstride / V;
  // positions of this lane's values, two per word
  uint32_t ps[KPL][V / 2];
#pragma unroll
  for (int j = 0; j < KPL; ++j) {
    const int c = gl + j * G;
    if (V == 8) {
      const uint4 pw = c < kv ? __ldg(reinterpret_cast<const uint4 *>(prow + c * V)) : make_uint4(0u, 0u, 0u, 0u);
      ps[j][0] = pw.x, ps[j][1] = pw.y, ps[j][V / 2 - 2] = pw.z, ps[j][V / 2 - 1] = pw.w;
    } else {
      const uint2 pw = c < kv ? __ldg(reinterpret_cast<const uint2 *>(prow + c * V)) : make_uint2(0u, 0u);
      ps[j][0] = pw.x, ps[j][1] = pw.y;
    }
  }
  for (int v = gl; v < nv; v += G) srow4[v] = make_uint4(0u, 0u, 0u, 0u);
  __syncwarp(gmask);
  for (int s = s0; s < s1; s += kAhead) {
    int slot[kAhead];
    uint4 z[kAhead][KPL];
#pragma unroll
    for (int u = 0; u < kAhead; ++u) slot[u] = __ldg(brow_slot + min(s + u, s1 - 1));
#pragma unroll
    for (int u = 0; u < kAhead; ++u)
#pragma unroll
      for (int j = 0; j < KPL; ++j)
        z[u][j] = gl + j * G < kv ? __ldg(packed4 + (int64_t)slot[u] * kstride4 + gl + j * G) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int u = 0; u < kAhead; ++u) {
      if (s + u >= s1) break;
#pragma unroll
      for (int j = 0; j < KPL; ++j) {
        const uint32_t zw[4] = {z[u][j].x, z[u][j].y, z[u][j].z, z[u][j].w};
        const int m0 = (gl + j * G) * V;
#pragma unroll
        for (int i = 0; i < V; ++i) {
          const uint32_t pos = (ps[j][i >> 1] >> ((i & 1) * 16)) & 0xFFFFu;
          E val;
          if (sizeof(E) == 2) val = (E)((zw[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu);
          else val = (E)zw[i];
          if (m0 + i < k) srow[pos] = val;
        }
      }
      __syncwarp(gmask);
      uint4 *dst = reinterpret_cast<uint4 *>(Xhalo + (int64_t)slot[u] * ld);
      for (int v = gl; v < nv; v += G) dst[v] = srow4[v];
      __syncwarp(gmask);
    }
  }
}

// ------------------------------------------------------------------------------------------
// Receiver side, sparse form.  Instead of a dense row with F - k zeros, the slot keeps its k
// received values next to the positions they belong to: pair m = (value m, pi(m)).  The
// aggregation then reads k pairs per remote neighbour instead of F elements.  bf16: one 32-bit
// word per pair (value in the low half, position in the high half); fp32: two words.
template <typename E>
__global__ void __launch_bounds__(256) expand_slots_kernel(const E *__restrict__ packed, int64_t kstride, int k, int H,
                                                           uint32_t *__restrict__ pairs, int64_t pstride,
                                                           const uint16_t *__restrict__ wpos, int64_t wstride,
                                                           const int32_t *__restrict__ slot_src) {
  // one thread per 16-byte chunk of a packed row: V values and their V positions from the table
  constexpr int V = VecOf<E>::kVec;
  const int kv = (int)(kstride / V);
  const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int slot = (int)(t / kv), c = (int)(t % kv);
  if (slot >= H) return;
  const uint4 z = __ldg(reinterpret_cast<const uint4 *>(packed + (int64_t)slot * kstride) + c);
  const uint16_t *prow = wpos + (int64_t)__ldg(slot_src + slot) * wstride + c * V;
  const uint32_t zw[4] = {z.x, z.y, z.z, z.w};
  uint32_t out[8];
  if (sizeof(E) == 2) {
    const uint4 pw = __ldg(reinterpret_cast<const uint4 *>(prow));
    const uint32_t ps[4] = {pw.x, pw.y, pw.z, pw.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int m = c * 8 + i;
      const uint32_t v = (zw[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu;
      const uint32_t pos = (ps[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu;
      out[i] = m < k ? (v | (pos << 16)) : 0u;   // padding pairs: value 0 at position 0
    }
  } else {
    const uint2 pw = __ldg(reinterpret_cast<const uint2 *>(prow));
    const uint32_t ps[2] = {pw.x, pw.y};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int m = c * 4 + i;
      const uint32_t pos = (ps[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu;
      out[2 * i] = m < k ? zw[i] : 0u;
      out[2 * i + 1] = m < k ? pos : 0u;
    }
  }
  // 32 bytes of pairs per chunk; pstride is a multiple of 4 pairs, so a row may end after the first half
  constexpr int kPairWords = sizeof(E) == 2 ? 1 : 2;
  uint4 *dst = reinterpret_cast<uint4 *>(pairs + ((int64_t)slot * pstride + (int64_t)c * V) * kPairWords);
  constexpr int kHalf = V / 2;   // pairs per 16 bytes
  if (c * V < pstride) dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
  if (c * V + kHalf < pstride) dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
}

// ------------------------------------------------------------------------------------------
// Kept positions of every unique boundary row, evaluated once per call: entry m of table row r is
// pi_r(m), m < k.  The forward fills the table while compressing; the backward, which runs after
// other layers have reused the workspace, fills it again from the same key before the kernels
// that consult it (one evaluation per unique row instead of one per slot copy and per kernel).
template <int G>
__global__ void __launch_bounds__(256) wire_positions_kernel(int F, int k, int h, uint64_t lkey,
                                                             const int32_t *__restrict__ brow,
                                                             const int32_t *__restrict__ row_gid, int nb,
                                                             uint16_t *__restrict__ wpos, int64_t wstride) {
  const int b = (blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int gl = threadIdx.x % G;
  if (b >= nb) return;
  const unsigned gmask = group_mask<G>();
  const int r = brow[b];
  vperm::RowPerm pm;
  init_perm<G>(pm, lkey, (uint32_t)row_gid[r], (uint32_t)F, h, gl, gmask);
  for (int m = gl; m < k; m += G) wpos[(int64_t)r * wstride + m] = (uint16_t)pm.pi((uint32_t)m);
}

// ------------------------------------------------------------------------------------------
// Backward, receiver side, when the slot gradient rows exist densely (they came out of a GEMM):
// keep the k values at the forward's positions.  One group per slot; positions from the table.
template <typename E, int G>
__global__ void __launch_bounds__(256) select_slots_kernel(const E *__restrict__ Gh, int64_t ldg, int nv, int k,
                                                           int H, E *__restrict__ packed, int64_t kstride,
                                                           const uint16_t *__restrict__ wpos, int64_t wstride,
                                                           const int32_t *__restrict__ slot_src) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = VecOf<E>::kVec;
  const int kv = (int)(kstride / V);
  const int grp = threadIdx.x / G, gl = threadIdx.x % G;
  const int slot = blockIdx.x * (blockDim.x / G) + grp;
  if (slot >= H) return;
  const unsigned gmask = group_mask<G>();
  uint4 *srow4 = smem_u4 + (size_t)grp * nv;
  const E *srow = reinterpret_cast<const E *>(srow4);
  const uint4 *src = reinterpret_cast<const uint4 *>(Gh + (int64_t)slot * ldg);
  for (int v = gl; v < nv; v += G) srow4[v] = __ldg(src + v);
  const uint16_t *prow = wpos + (int64_t)__ldg(slot_src + slot) * wstride;
  __syncwarp(gmask);
  uint4 *dst = reinterpret_cast<uint4 *>(packed + (int64_t)slot * kstride);
  for (int c = gl; c < kv; c += G) {
    uint32_t ps[4];
    if (V == 8) {
      const uint4 pw = __ldg(reinterpret_cast<const uint4 *>(prow + c * V));
      ps[0] = pw.x, ps[1] = pw.y, ps[2] = pw.z, ps[3] = pw.w;
    } else {
      const uint2 pw = __ldg(reinterpret_cast<const uint2 *>(prow + c * V));
      ps[0] = pw.x, ps[1] = pw.y, ps[2] = 0u, ps[3] = 0u;
    }
    E z[V];
#pragma unroll
    for (int i = 0; i < V; ++i)
      z[i] = c * V + i < k ? srow[(ps[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu] : (E)0;
    dst[c] = *reinterpret_cast<const uint4 *>(z);
  }
}

// ------------------------------------------------------------------------------------------
// Backward, receiver side, narrow layers in compressed epochs with at most 16 kept entries (bf16).  The
// gradient row of a halo slot is (slot sum of dZ) W_neigh^T, F_in wide, but only its k kept entries are
// returned to the owner: entry m is the dot product of the slot's F_out-wide sum with row pi(m) of W_neigh.
// One thread per slot: the sum is read once into registers, the positions come eight at a time as 16-byte
// reads of the call's table, W_neigh sits in shared memory as F_in rows of bf16 pairs (16-byte aligned rows an
// odd number of 16-byte units apart, read with 16-byte loads: the lanes of a warp read different rows), and
// every 8 packed values of the slot leave as one 16-byte store.  fp32 accumulation, results rounded to bf16 as a
// GEMM epilogue would.  Against the dense product (H x F_in values written, read again and picked from: 10 GB
// each way on the 2.45M-node workload) this is k F_out multiply-adds and k F_out / 2 shared-memory words per
// slot.  NVO: 16-byte chunks of a row of sums; kv: 16-byte chunks of a packed row.
template <int NVO>
__global__ void __launch_bounds__(256) slot_kept_product_kernel(const uint4 *__restrict__ Gh4, int64_t ldg4, int F_out,
                                                                const __nv_bfloat16 *__restrict__ W, int F_in, int k,
                                                                int H, uint4 *__restrict__ packed4, int kv,
                                                                const uint16_t *__restrict__ wpos, int64_t wstride,
                                                                const int32_t *__restrict__ slot_src) {
  extern __shared__ __align__(16) uint32_t w_pairs[];
  constexpr int NW = NVO * 4;          // words (pairs) per row
  constexpr int kRowWords = NW + 4;    // rows 16-byte aligned, an odd number of 16-byte units apart
  const uint16_t *Wbits = reinterpret_cast<const uint16_t *>(W);
  for (int i = threadIdx.x; i < F_in * NW; i += blockDim.x) {
    const int f = i / NW, j = i % NW;
    const uint32_t lo = 2 * j < F_out ? Wbits[(int64_t)f * F_out + 2 * j] : 0u;
    const uint32_t hi = 2 * j + 1 < F_out ? Wbits[(int64_t)f * F_out + 2 * j + 1] : 0u;
    w_pairs[f * kRowWords + j] = lo | (hi << 16);
  }
  __syncthreads();
  for (int slot = blockIdx.x * blockDim.x + threadIdx.x; slot < H; slot += gridDim.x * blockDim.x) {
    const uint4 *prow = reinterpret_cast<const uint4 *>(wpos + (int64_t)__ldg(slot_src + slot) * wstride);
    float g[NVO * 8];
#pragma unroll
    for (int i = 0; i < NVO; ++i) {
      float f[8];
      unpack16(i * 8 < F_out ? __ldg(Gh4 + (int64_t)slot * ldg4 + i) : make_uint4(0u, 0u, 0u, 0u), f, __nv_bfloat16());
#pragma unroll
      for (int j = 0; j < 8; ++j) g[i * 8 + j] = i * 8 + j < F_out ? f[j] : 0.f;
    }
    for (int c = 0; c * 8 < k; ++c) {
      const uint4 pw = __ldg(prow + c);
      const uint32_t ps[4] = {pw.x, pw.y, pw.z, pw.w};
      float acc[8];
#pragma unroll
      for (int m = 0; m < 8; ++m) {
        acc[m] = 0.f;
        if (c * 8 + m < k) {   // table entries at or beyond k are not defined
          const uint4 *wr = reinterpret_cast<const uint4 *>(w_pairs + ((ps[m >> 1] >> ((m & 1) * 16)) & 0xFFFFu) * kRowWords);
#pragma unroll
          for (int jq = 0; jq < NVO; ++jq) {
            const uint4 wq = wr[jq];
            const uint32_t wj[4] = {wq.x, wq.y, wq.z, wq.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int j = jq * 4 + i;
              acc[m] = fmaf(g[2 * j], __uint_as_float(wj[i] << 16), acc[m]);
              acc[m] = fmaf(g[2 * j + 1], __uint_as_float(wj[i] & 0xFFFF0000u), acc[m]);
            }
          }
        }
      }
      packed4[(int64_t)slot * kv + c] = pack16(acc, __nv_bfloat16());
    }
  }
}

// ------------------------------------------------------------------------------------------
// Backward, owner side, k < F.  One group per unique boundary row: the packed gradients
// returned by every destination partition are summed in ascending destination order and added
// to the owner's gradient row at the kept positions.  No atomics: the result is reproducible.
template <typename T, int G>
__global__ void __launch_bounds__(256) scatter_add_rows_kernel(const T *__restrict__ packed, int64_t kstride, int F,
                                                               int k, const int32_t *__restrict__ brow,
                                                               const int32_t *__restrict__ brow_ptr,
                                                               const int32_t *__restrict__ brow_slot, int nb,
                                                               T *__restrict__ dX, int64_t ld,
                                                               const uint16_t *__restrict__ wpos, int64_t wstride) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = ElemTraits<T>::kVec;
  const int nv = (F + V - 1) / V;
  const int kv = (int)(kstride / V);
  const int grp = threadIdx.x / G, gl = threadIdx.x % G;
  const int b = blockIdx.x * (blockDim.x / G) + grp;
  if (b >= nb) return;
  const unsigned gmask = group_mask<G>();
  float *srow = reinterpret_cast<float *>(smem_u4) + (size_t)grp * nv * V;
  const int r = brow[b];
  const int s0 = brow_ptr[b], s1 = brow_ptr[b + 1];
  uint4 *row4 = reinterpret_cast<uint4 *>(dX + (int64_t)r * ld);
  for (int v = gl; v < nv; v += G) {
    float f[V];
    unpack16(row4[v], f, T());
#pragma unroll
    for (int i = 0; i < V; ++i) srow[v * V + i] = f[i];
  }
  __syncwarp(gmask);
  const uint16_t *prow = wpos + (int64_t)r * wstride;
  // a lane owns 16-byte chunks of the packed rows: V kept values per load, four slot copies in flight,
  // summed from zero in ascending slot order, then added at the kept positions (all distinct)
  for (int v = gl; v < kv; v += G) {
    float sum[V];
#pragma unroll
    for (int i = 0; i < V; ++i) sum[i] = 0.f;
    int s = s0;
    for (; s + 3 < s1; s += 4) {
      uint4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        q[u] = __ldg(reinterpret_cast<const uint4 *>(packed + (int64_t)brow_slot[s + u] * kstride) + v);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float f[V];
        unpack16(q[u], f, T());
#pragma unroll
        for (int i = 0; i < V; ++i) sum[i] += f[i];
      }
    }
    for (; s < s1; ++s) {
      float f[V];
      unpack16(__ldg(reinterpret_cast<const uint4 *>(packed + (int64_t)brow_slot[s] * kstride) + v), f, T());
#pragma unroll
      for (int i = 0; i < V; ++i) sum[i] += f[i];
    }
    uint32_t ps[4];
    if (V == 8) {
      const uint4 pw = __ldg(reinterpret_cast<const uint4 *>(prow + v * V));
      ps[0] = pw.x, ps[1] = pw.y, ps[2] = pw.z, ps[3] = pw.w;
    } else {
      const uint2 pw = __ldg(reinterpret_cast<const uint2 *>(prow + v * V));
      ps[0] = pw.x, ps[1] = pw.y, ps[2] = 0u, ps[3] = 0u;
    }
#pragma unroll
    for (int i = 0; i < V; ++i)
      if (v * V + i < k) srow[(ps[i >> 1] >> ((i & 1) * 16)) & 0xFFFFu] += sum[i];
  }
  __syncwarp(gmask);
  for (int v = gl; v < nv; v += G) {
    float f[V];
#pragma unroll
    for (int i = 0; i < V; ++i) f[i] = srow[v * V + i];
    row4[v] = pack16(f, T());
  }
}

// Backward, owner side, full communication: the slot gradient rows are dense; add them to the
// owner's row in ascending destination order.
template <typename T, int G>
__global__ void __launch_bounds__(256) add_dense_rows_kernel(const T *__restrict__ Gh, int64_t ldg, int nv,
                                                             const int32_t *__restrict__ brow,
                                                             const int32_t *__restrict__ brow_ptr,
                                                             const int32_t *__restrict__ brow_slot, int nb,
                                                             T *__restrict__ dX, int64_t ld) {
  constexpr int V = ElemTraits<T>::kVec;
  const int b = (blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int gl = threadIdx.x % G;
  if (b >= nb) return;
  const int r = brow[b];
  const int s0 = brow_ptr[b], s1 = brow_ptr[b + 1];
  uint4 *row4 = reinterpret_cast<uint4 *>(dX + (int64_t)r * ld);
  for (int v = gl; v < nv; v += G) {
    float acc[V];
    unpack16(row4[v], acc, T());
    int s = s0;
    for (; s + 3 < s1; s += 4) {   // four slot rows in flight, added in ascending slot order
      uint4 q[4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
        q[u] = __ldg(reinterpret_cast<const uint4 *>(Gh + (int64_t)brow_slot[s + u] * ldg) + v);
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        float f[V];
        unpack16(q[u], f, T());
#pragma unroll
        for (int i = 0; i < V; ++i) acc[i] += f[i];
      }
    }
    for (; s + 1 < s1; s += 2) {
      const uint4 a = __ldg(reinterpret_cast<const uint4 *>(Gh + (int64_t)brow_slot[s] * ldg) + v);
      const uint4 c = __ldg(reinterpret_cast<const uint4 *>(Gh + (int64_t)brow_slot[s + 1] * ldg) + v);
      float fa[V], fc[V];
      unpack16(a, fa, T());
      unpack16(c, fc, T());
#pragma unroll
      for (int i = 0; i < V; ++i) acc[i] = (acc[i] + fa[i]) + fc[i];
    }
    if (s < s1) {
      float fa[V];
      unpack16(__ldg(reinterpret_cast<const uint4 *>(Gh + (int64_t)brow_slot[s] * ldg) + v), fa, T());
#pragma unroll
      for (int i = 0; i < V; ++i) acc[i] += fa[i];
    }
    row4[v] = pack16(acc, T());
  }
}

int group_size(int nv) { return nv <= 32 ? 8 : (nv <= 64 ? 16 : 32); }

struct HaloLaunch {
  int G, threads;
  unsigned blocks;
  size_t smem;
};
// rows -> launch shape; `row_smem` bytes of shared memory per row
HaloLaunch shape(int64_t rows, int nv, size_t row_smem) {
  HaloLaunch L;
  L.G = group_size(nv);
  L.threads = 256;
  while (L.threads > L.G && (size_t)(L.threads / L.G) * row_smem > 48 * 1024) L.threads /= 2;
  const int per_block = L.threads / L.G;
  L.blocks = (unsigned)((rows + per_block - 1) / per_block);
  L.smem = (size_t)per_block * row_smem;
  return L;
}

#define VARCO_DISPATCH_G(L, CALL)   \
  do {                              \
    if ((L).G == 8) {               \
      constexpr int G = 8;          \
      CALL;                         \
    } else if ((L).G == 16) {       \
      constexpr int G = 16;         \
      CALL;                         \
    } else {                        \
      constexpr int G = 32;         \
      CALL;                         \
    }                               \
  } while (0)

}  // namespace

// ------------------------------------------------------------------------------------------ launchers
// Full-communication exchange of the layer path: X rows -> dense halo slots.
int varco_launch_gather_copy(const varco_plan *pl, const void *X, int64_t ld, int F, varco_dtype_t dt, void *Xhalo,
                             int64_t ldh, cudaStream_t st) {
  if (pl->nb == 0) return VARCO_OK;
  const int es = dt == VARCO_F32 ? 4 : 2, V = 16 / es;
  const int nv = (F + V - 1) / V;
  HaloLaunch L = shape(pl->nb, nv, 0);
  VARCO_DISPATCH_G(L, (gather_copy_kernel<G><<<L.blocks, L.threads, 0, st>>>(
                          (const uint4 *)X, ld / V, nv, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, (int)pl->nb,
                          (uint4 *)Xhalo, ldh / V)));
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// send_order != 0: packed rows at the sender's positions (stand-alone entry point), else at the slot
int varco_launch_compress_rows(const varco_plan *pl, const void *X, int64_t ld, int F, int k, varco_dtype_t dt,
                               varco_key_t key, void *packed, int64_t kstride, int send_order, uint16_t *wpos,
                               int64_t wstride, cudaStream_t st) {
  if (pl->nb == 0) return VARCO_OK;
  const int es = dt == VARCO_F32 ? 4 : 2, V = 16 / es;
  const int nv = (F + V - 1) / V, kv = (k + V - 1) / V;
  HaloLaunch L = shape(pl->nb, nv, (size_t)(nv + kv) * 16);
  const int h = vperm::half_bits(F);
  const uint64_t lkey = vperm::layer_key(key);
  const int32_t *sp = send_order ? pl->d.slot_sendpos : nullptr;
  if (dt == VARCO_F32)
    VARCO_DISPATCH_G(L, (compress_rows_kernel<uint32_t, G><<<L.blocks, L.threads, L.smem, st>>>(
                            (const uint32_t *)X, ld, F, k, h, lkey, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, sp,
                            pl->d.row_gid, (int)pl->nb, (uint32_t *)packed, kstride, wpos, wstride)));
  else
    VARCO_DISPATCH_G(L, (compress_rows_kernel<uint16_t, G><<<L.blocks, L.threads, L.smem, st>>>(
                            (const uint16_t *)X, ld, F, k, h, lkey, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, sp,
                            pl->d.row_gid, (int)pl->nb, (uint16_t *)packed, kstride, wpos, wstride)));
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

int varco_launch_decompress_slots(const varco_plan *pl, const void *packed, int64_t kstride, int send_order, int F,
                                  int k, varco_dtype_t dt, varco_key_t key, void *Xhalo, int64_t ld, const uint16_t *wpos,
                                  int64_t wstride, cudaStream_t st) {
  if (pl->H == 0) return VARCO_OK;
  const int es = dt == VARCO_F32 ? 4 : 2, V = 16 / es;
  const int nv = (F + V - 1) / V, kv = (k + V - 1) / V;
  if (wpos && !send_order && kstride % V == 0 && wstride % 8 == 0 && kstride / V <= 2 * group_size(nv)) {
    // layer path: slot order on the packed side and a table of positions -> walk by source row
    HaloLaunch B = shape(pl->nb, nv, (size_t)nv * 16);
    const bool one = kstride / V <= B.G;
#define VARCO_DBR(E, KPL)                                                                                        \
  VARCO_DISPATCH_G(B, (decompress_brows_kernel<E, G, KPL><<<B.blocks, B.threads, B.smem, st>>>(                  \
                          (const E *)packed, kstride, F, k, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, (int)pl->nb, \
                          (E *)Xhalo, ld, wpos, wstride)))
    if (dt == VARCO_F32) {
      if (one) VARCO_DBR(uint32_t, 1);
      else VARCO_DBR(uint32_t, 2);
    } else {
      if (one) VARCO_DBR(uint16_t, 1);
      else VARCO_DBR(uint16_t, 2);
    }
#undef VARCO_DBR
    VARCO_KERNEL_LAUNCHED();
    return VARCO_OK;
  }
  HaloLaunch L = shape(pl->H, nv, (size_t)(nv + kv) * 16);
  const int h = vperm::half_bits(F);
  const uint64_t lkey = vperm::layer_key(key);
  const int32_t *sp = send_order ? pl->d.slot_sendpos : nullptr;
  if (dt == VARCO_F32)
    VARCO_DISPATCH_G(L, (decompress_slots_kernel<uint32_t, G><<<L.blocks, L.threads, L.smem, st>>>(
                            (const uint32_t *)packed, kstride, F, k, h, lkey, pl->d.slot_gid, sp, (int)pl->H,
                            (uint32_t *)Xhalo, ld, wpos, wstride, pl->d.slot_src)));
  else
    VARCO_DISPATCH_G(L, (decompress_slots_kernel<uint16_t, G><<<L.blocks, L.threads, L.smem, st>>>(
                            (const uint16_t *)packed, kstride, F, k, h, lkey, pl->d.slot_gid, sp, (int)pl->H,
                            (uint16_t *)Xhalo, ld, wpos, wstride, pl->d.slot_src)));
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// packed rows (slot order, stride kstride) -> (value, position) pairs, pstride pairs per slot; the positions
// come from the call's table
int varco_launch_expand_slots(const varco_plan *pl, const void *packed, int64_t kstride, int k, varco_dtype_t dt,
                              void *pairs, int64_t pstride, const uint16_t *wpos, int64_t wstride, cudaStream_t st) {
  if (pl->H == 0) return VARCO_OK;
  if (!wpos) return VARCO_INVALID_ARG;
  const int V = dt == VARCO_F32 ? 4 : 8;
  const int threads = 256;
  const unsigned blocks = (unsigned)(((int64_t)pl->H * (kstride / V) + threads - 1) / threads);
  if (dt == VARCO_F32)
    expand_slots_kernel<uint32_t><<<blocks, threads, 0, st>>>((const uint32_t *)packed, kstride, k, (int)pl->H,
                                                              (uint32_t *)pairs, pstride, wpos, wstride, pl->d.slot_src);
  else
    expand_slots_kernel<uint16_t><<<blocks, threads, 0, st>>>((const uint16_t *)packed, kstride, k, (int)pl->H,
                                                              (uint32_t *)pairs, pstride, wpos, wstride, pl->d.slot_src);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

int varco_launch_scatter_add_rows(const varco_plan *pl, const void *packed, int64_t kstride, int F, int k,
                                  varco_dtype_t dt, void *dX, int64_t ld, const uint16_t *wpos, int64_t wstride,
                                  cudaStream_t st) {
  if (pl->nb == 0) return VARCO_OK;
  if (!wpos) return VARCO_INVALID_ARG;
  const int V = dt == VARCO_F32 ? 4 : 8;
  const int nv = (F + V - 1) / V;
  HaloLaunch L = shape(pl->nb, nv, (size_t)nv * V * sizeof(float));
  if (dt == VARCO_F32)
    VARCO_DISPATCH_G(L, (scatter_add_rows_kernel<float, G><<<L.blocks, L.threads, L.smem, st>>>(
                            (const float *)packed, kstride, F, k, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot,
                            (int)pl->nb, (float *)dX, ld, wpos, wstride)));
  else
    VARCO_DISPATCH_G(L, (scatter_add_rows_kernel<__nv_bfloat16, G><<<L.blocks, L.threads, L.smem, st>>>(
                            (const __nv_bfloat16 *)packed, kstride, F, k, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot,
                            (int)pl->nb, (__nv_bfloat16 *)dX, ld, wpos, wstride)));
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// Dense slot gradient rows -> their k kept values (slot order, stride kstride).
int varco_launch_select_slots(const varco_plan *pl, const void *Gh, int64_t ldg, int F, int k, varco_dtype_t dt,
                              void *packed, int64_t kstride, const uint16_t *wpos, int64_t wstride, cudaStream_t st) {
  if (pl->H == 0) return VARCO_OK;
  if (!wpos) return VARCO_INVALID_ARG;
  const int V = dt == VARCO_F32 ? 4 : 8;
  const int nv = (F + V - 1) / V;
  HaloLaunch L = shape(pl->H, nv, (size_t)nv * 16);
  if (dt == VARCO_F32)
    VARCO_DISPATCH_G(L, (select_slots_kernel<uint32_t, G><<<L.blocks, L.threads, L.smem, st>>>(
                            (const uint32_t *)Gh, ldg, nv, k, (int)pl->H, (uint32_t *)packed, kstride, wpos, wstride,
                            pl->d.slot_src)));
  else
    VARCO_DISPATCH_G(L, (select_slots_kernel<uint16_t, G><<<L.blocks, L.threads, L.smem, st>>>(
                            (const uint16_t *)Gh, ldg, nv, k, (int)pl->H, (uint16_t *)packed, kstride, wpos, wstride,
                            pl->d.slot_src)));
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// Kept entries of the slot gradient rows straight from the slot sums of a narrow layer (bf16, k <= 16; the
// lanes of a warp read different rows of W_neigh, so the shared-memory reads collide and at k = 32 the dense
// product followed by a pick is the faster way again):
// packed[slot][m] = Gh[slot] . W_neigh[pi(m)], m < k; packed rows of kstride (a multiple of 8) values.
bool varco_slot_kept_product_supported(int F_in, int F_out, int k, varco_dtype_t dt) {
  if (dt != VARCO_BF16 || F_out > 64 || k > 16) return false;
  const int nvo = ((F_out + 7) / 8 + 1) / 2 * 2;
  return (size_t)F_in * (nvo * 4 + 4) * 4 <= 48 * 1024;
}

int varco_launch_slot_kept_product(const varco_plan *pl, const void *Gh, int64_t ldg, int F_out, const void *W_neigh,
                                   int F_in, int k, void *packed, int64_t kstride, const uint16_t *wpos,
                                   int64_t wstride, cudaStream_t st) {
  if (pl->H == 0) return VARCO_OK;
  if (!wpos || !varco_slot_kept_product_supported(F_in, F_out, k, VARCO_BF16) || ldg % 8 != 0 || ldg < F_out ||
      kstride % 8 != 0 || kstride < k || wstride % 8 != 0)
    return VARCO_INVALID_ARG;
  const int nvo = ((F_out + 7) / 8 + 1) / 2 * 2;   // 2, 4, 6 or 8 chunks
  int dev = 0, sms = 148;
  VARCO_CUDA_CHECK(cudaGetDevice(&dev));
  VARCO_CUDA_CHECK(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const size_t smem = (size_t)F_in * (nvo * 4 + 4) * 4;
  const int64_t want = (pl->H + 255) / 256;
  const unsigned grid = (unsigned)(want < (int64_t)sms * 8 ? want : (int64_t)sms * 8);
#define VARCO_SKP(N)                                                                                               \
  slot_kept_product_kernel<N><<<grid, 256, smem, st>>>((const uint4 *)Gh, ldg / 8, F_out, (const __nv_bfloat16 *)W_neigh, \
                                                       F_in, k, (int)pl->H, (uint4 *)packed, (int)(kstride / 8),     \
                                                       wpos, wstride,                                                \
                                                       pl->d.slot_src)
  if (nvo == 2) VARCO_SKP(2);
  else if (nvo == 4) VARCO_SKP(4);
  else if (nvo == 6) VARCO_SKP(6);
  else VARCO_SKP(8);
#undef VARCO_SKP
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// Kept positions of every unique boundary row of this call (k < F) into the table.
int varco_launch_wire_positions(const varco_plan *pl, int F, int k, varco_key_t key, uint16_t *wpos, int64_t wstride,
                                cudaStream_t st) {
  if (pl->nb == 0) return VARCO_OK;
  HaloLaunch L;
  L.G = k <= 8 ? 8 : (k <= 16 ? 16 : 32);
  const int threads = 256;
  const unsigned blocks = (unsigned)(((int64_t)pl->nb * L.G + threads - 1) / threads);
  const int h = vperm::half_bits(F);
  const uint64_t lkey = vperm::layer_key(key);
  VARCO_DISPATCH_G(L, (wire_positions_kernel<G><<<blocks, threads, 0, st>>>(F, k, h, lkey, pl->d.brow, pl->d.row_gid,
                                                                           (int)pl->nb, wpos, wstride)));
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

int varco_launch_add_dense_rows(const varco_plan *pl, const void *Gh, int64_t ldg, int F, varco_dtype_t dt, void *dX,
                                int64_t ld, cudaStream_t st) {
  if (pl->nb == 0) return VARCO_OK;
  const int V = dt == VARCO_F32 ? 4 : 8;
  const int nv = (F + V - 1) / V;
  HaloLaunch L = shape(pl->nb, nv, 0);
  if (dt == VARCO_F32)
    VARCO_DISPATCH_G(L, (add_dense_rows_kernel<float, G><<<L.blocks, L.threads, 0, st>>>(
                            (const float *)Gh, ldg, nv, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, (int)pl->nb,
                            (float *)dX, ld)));
  else
    VARCO_DISPATCH_G(L, (add_dense_rows_kernel<__nv_bfloat16, G><<<L.blocks, L.threads, 0, st>>>(
                            (const __nv_bfloat16 *)Gh, ldg, nv, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot,
                            (int)pl->nb, (__nv_bfloat16 *)dX, ld)));
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}
