// Halo exchange kernels: gather + compress, decompress + scatter, and their backward mirrors.
//
// Algorithm 1 of the paper, second and third step: every partition compresses the activations
// of its boundary rows and sends them to the adjacent partitions, which decompress them.  The
// compressor keeps k = ceil(F / c) values of a row at keyed pseudo-random positions and the
// decoder puts them back in place with zeros elsewhere (Definition 1; appendix "Compression
// Mechanism").  The backward pass returns the halo-row gradients through the same compressor.
//
// All four kernels are pure data movement (bit-exact) plus the integer permutation, one warp per
// row: the row is staged in shared memory with 128-bit accesses, permuted there, and the packed
// side is written/read as contiguous k-element rows.
#include "device_common.cuh"

namespace {

constexpr int kWarp = 32;

template <typename E> struct VecOf { static constexpr int kVec = 16 / (int)sizeof(E); };

__device__ __forceinline__ uint4 ld_nc(const uint4 *p) { return __ldg(p); }

// ------------------------------------------------------------------------------------------
// Forward, sender side.  One warp per UNIQUE boundary row: the row is read once, its k kept
// values are selected once and written to the send segment of every destination partition.
template <typename E>
__global__ void __launch_bounds__(256) compress_rows_kernel(const E *__restrict__ X, int64_t ld, int F, int k, int h,
                                                            uint64_t lkey, const int32_t *__restrict__ brow,
                                                            const int32_t *__restrict__ brow_ptr,
                                                            const int32_t *__restrict__ brow_slot,
                                                            const int32_t *__restrict__ slot_sendpos,
                                                            const int32_t *__restrict__ row_gid, int nb,
                                                            E *__restrict__ packed) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = VecOf<E>::kVec;
  const int nv = (F + V - 1) / V;
  const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
  const int wpb = blockDim.x / kWarp;
  const int b = blockIdx.x * wpb + warp;
  if (b >= nb) return;
  uint4 *srow4 = smem_u4 + (size_t)warp * nv;
  const E *srow = reinterpret_cast<const E *>(srow4);
  const int r = brow[b];
  const uint4 *src = reinterpret_cast<const uint4 *>(X + (int64_t)r * ld);
  for (int v = lane; v < nv; v += kWarp) srow4[v] = ld_nc(src + v);
  vperm::RowPerm pm;
  pm.init(lkey, (uint32_t)row_gid[r], (uint32_t)F, h);
  const int s0 = brow_ptr[b], s1 = brow_ptr[b + 1];
  __syncwarp();
  for (int m = lane; m < k; m += kWarp) {
    const E v = srow[pm.pi((uint32_t)m)];
    for (int s = s0; s < s1; ++s) {
      const int64_t pos = slot_sendpos[brow_slot[s]];
      packed[pos * k + m] = v;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Forward, receiver side.  One warp per halo slot: the k received values are put back at
// their positions in a zeroed row, which is then written out densely.
template <typename E>
__global__ void __launch_bounds__(256) decompress_slots_kernel(const E *__restrict__ packed, int F, int k, int h,
                                                               uint64_t lkey, const int32_t *__restrict__ slot_gid,
                                                               const int32_t *__restrict__ slot_sendpos, int H,
                                                               E *__restrict__ Xhalo, int64_t ld) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = VecOf<E>::kVec;
  const int nv = (F + V - 1) / V;
  const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
  const int wpb = blockDim.x / kWarp;
  const int slot = blockIdx.x * wpb + warp;
  if (slot >= H) return;
  uint4 *srow4 = smem_u4 + (size_t)warp * nv;
  E *srow = reinterpret_cast<E *>(srow4);
  for (int v = lane; v < nv; v += kWarp) srow4[v] = make_uint4(0u, 0u, 0u, 0u);
  vperm::RowPerm pm;
  pm.init(lkey, (uint32_t)slot_gid[slot], (uint32_t)F, h);
  const E *z = packed + (int64_t)slot_sendpos[slot] * k;
  __syncwarp();
  for (int m = lane; m < k; m += kWarp) srow[pm.pi((uint32_t)m)] = z[m];
  __syncwarp();
  uint4 *dst = reinterpret_cast<uint4 *>(Xhalo + (int64_t)slot * ld);
  for (int v = lane; v < nv; v += kWarp) dst[v] = srow4[v];
}

// ------------------------------------------------------------------------------------------
// Backward, receiver side (now the sender of gradients).  One warp per halo slot: the slot's
// gradient row is compressed with the forward's permutation; packed rows are in slot order.
template <typename E>
__global__ void __launch_bounds__(256) compress_slots_kernel(const E *__restrict__ G, int64_t ld, int F, int k, int h,
                                                             uint64_t lkey, const int32_t *__restrict__ slot_gid,
                                                             int H, E *__restrict__ packed) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = VecOf<E>::kVec;
  const int nv = (F + V - 1) / V;
  const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
  const int wpb = blockDim.x / kWarp;
  const int slot = blockIdx.x * wpb + warp;
  if (slot >= H) return;
  uint4 *srow4 = smem_u4 + (size_t)warp * nv;
  const E *srow = reinterpret_cast<const E *>(srow4);
  const uint4 *src = reinterpret_cast<const uint4 *>(G + (int64_t)slot * ld);
  for (int v = lane; v < nv; v += kWarp) srow4[v] = ld_nc(src + v);
  vperm::RowPerm pm;
  pm.init(lkey, (uint32_t)slot_gid[slot], (uint32_t)F, h);
  E *z = packed + (int64_t)slot * k;
  __syncwarp();
  for (int m = lane; m < k; m += kWarp) z[m] = srow[pm.pi((uint32_t)m)];
}

// ------------------------------------------------------------------------------------------
// Backward, owner side.  One warp per unique boundary row: the packed gradients returned by
// every destination partition are summed in ascending destination order and added to the
// owner's gradient row at the kept positions.  No atomics: the result is reproducible.
template <typename T>
__global__ void __launch_bounds__(256) scatter_add_rows_kernel(const T *__restrict__ packed, int F, int k, int h,
                                                               uint64_t lkey, const int32_t *__restrict__ brow,
                                                               const int32_t *__restrict__ brow_ptr,
                                                               const int32_t *__restrict__ brow_slot,
                                                               const int32_t *__restrict__ row_gid, int nb,
                                                               T *__restrict__ dX, int64_t ld) {
  extern __shared__ uint4 smem_u4[];
  constexpr int V = ElemTraits<T>::kVec;
  const int nv = (F + V - 1) / V;
  const int warp = threadIdx.x / kWarp, lane = threadIdx.x % kWarp;
  const int wpb = blockDim.x / kWarp;
  const int b = blockIdx.x * wpb + warp;
  if (b >= nb) return;
  float *srow = reinterpret_cast<float *>(smem_u4) + (size_t)warp * nv * V;
  const int r = brow[b];
  uint4 *row4 = reinterpret_cast<uint4 *>(dX + (int64_t)r * ld);
  for (int v = lane; v < nv; v += kWarp) {
    float f[V];
    unpack16(row4[v], f, T());
#pragma unroll
    for (int i = 0; i < V; ++i) srow[v * V + i] = f[i];
  }
  vperm::RowPerm pm;
  pm.init(lkey, (uint32_t)row_gid[r], (uint32_t)F, h);
  const int s0 = brow_ptr[b], s1 = brow_ptr[b + 1];
  __syncwarp();
  for (int m = lane; m < k; m += kWarp) {
    float sum = 0.f;
    for (int s = s0; s < s1; ++s) sum += ElemTraits<T>::to_f(packed[(int64_t)brow_slot[s] * k + m]);
    srow[pm.pi((uint32_t)m)] += sum;
  }
  __syncwarp();
  for (int v = lane; v < nv; v += kWarp) {
    float f[V];
#pragma unroll
    for (int i = 0; i < V; ++i) f[i] = srow[v * V + i];
    row4[v] = pack16(f, T());
  }
}

int warps_per_block(size_t row_bytes) {
  int w = (int)(48 * 1024 / row_bytes);
  if (w >= 8) return 8;
  if (w >= 4) return 4;
  if (w >= 2) return 2;
  return 1;
}

}  // namespace

// ------------------------------------------------------------------------------------------ launchers
int varco_launch_compress_rows(const varco_plan *pl, const void *X, int64_t ld, int F, int k, varco_dtype_t dt,
                               varco_key_t key, void *packed, cudaStream_t st) {
  if (pl->nb == 0) return VARCO_OK;
  const int es = dt == VARCO_F32 ? 4 : 2;
  const int V = 16 / es;
  const size_t row_bytes = (size_t)((F + V - 1) / V) * 16;
  const int wpb = warps_per_block(row_bytes);
  const int h = vperm::half_bits(F);
  const uint64_t lkey = vperm::layer_key(key);
  dim3 grid((unsigned)((pl->nb + wpb - 1) / wpb)), block(wpb * 32);
  if (dt == VARCO_F32)
    compress_rows_kernel<uint32_t><<<grid, block, row_bytes * wpb, st>>>(
        (const uint32_t *)X, ld, F, k, h, lkey, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, pl->d.slot_sendpos,
        pl->d.row_gid, (int)pl->nb, (uint32_t *)packed);
  else
    compress_rows_kernel<uint16_t><<<grid, block, row_bytes * wpb, st>>>(
        (const uint16_t *)X, ld, F, k, h, lkey, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, pl->d.slot_sendpos,
        pl->d.row_gid, (int)pl->nb, (uint16_t *)packed);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

int varco_launch_decompress_slots(const varco_plan *pl, const void *packed, int F, int k, varco_dtype_t dt,
                                  varco_key_t key, void *Xhalo, int64_t ld, cudaStream_t st) {
  if (pl->H == 0) return VARCO_OK;
  const int es = dt == VARCO_F32 ? 4 : 2;
  const int V = 16 / es;
  const size_t row_bytes = (size_t)((F + V - 1) / V) * 16;
  const int wpb = warps_per_block(row_bytes);
  const int h = vperm::half_bits(F);
  const uint64_t lkey = vperm::layer_key(key);
  dim3 grid((unsigned)((pl->H + wpb - 1) / wpb)), block(wpb * 32);
  if (dt == VARCO_F32)
    decompress_slots_kernel<uint32_t><<<grid, block, row_bytes * wpb, st>>>(
        (const uint32_t *)packed, F, k, h, lkey, pl->d.slot_gid, pl->d.slot_sendpos, (int)pl->H, (uint32_t *)Xhalo,
        ld);
  else
    decompress_slots_kernel<uint16_t><<<grid, block, row_bytes * wpb, st>>>(
        (const uint16_t *)packed, F, k, h, lkey, pl->d.slot_gid, pl->d.slot_sendpos, (int)pl->H, (uint16_t *)Xhalo,
        ld);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

int varco_launch_compress_slots(const varco_plan *pl, const void *G, int64_t ld, int F, int k, varco_dtype_t dt,
                                varco_key_t key, void *packed, cudaStream_t st) {
  if (pl->H == 0) return VARCO_OK;
  const int es = dt == VARCO_F32 ? 4 : 2;
  const int V = 16 / es;
  const size_t row_bytes = (size_t)((F + V - 1) / V) * 16;
  const int wpb = warps_per_block(row_bytes);
  const int h = vperm::half_bits(F);
  const uint64_t lkey = vperm::layer_key(key);
  dim3 grid((unsigned)((pl->H + wpb - 1) / wpb)), block(wpb * 32);
  if (dt == VARCO_F32)
    compress_slots_kernel<uint32_t><<<grid, block, row_bytes * wpb, st>>>(
        (const uint32_t *)G, ld, F, k, h, lkey, pl->d.slot_gid, (int)pl->H, (uint32_t *)packed);
  else
    compress_slots_kernel<uint16_t><<<grid, block, row_bytes * wpb, st>>>(
        (const uint16_t *)G, ld, F, k, h, lkey, pl->d.slot_gid, (int)pl->H, (uint16_t *)packed);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

int varco_launch_scatter_add_rows(const varco_plan *pl, const void *packed, int F, int k, varco_dtype_t dt,
                                  varco_key_t key, void *dX, int64_t ld, cudaStream_t st) {
  if (pl->nb == 0) return VARCO_OK;
  const int V = dt == VARCO_F32 ? 4 : 8;
  const size_t row_bytes = (size_t)((F + V - 1) / V) * V * sizeof(float);
  const int wpb = warps_per_block(row_bytes);
  const int h = vperm::half_bits(F);
  const uint64_t lkey = vperm::layer_key(key);
  dim3 grid((unsigned)((pl->nb + wpb - 1) / wpb)), block(wpb * 32);
  if (dt == VARCO_F32)
    scatter_add_rows_kernel<float><<<grid, block, row_bytes * wpb, st>>>(
        (const float *)packed, F, k, h, lkey, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, pl->d.row_gid,
        (int)pl->nb, (float *)dX, ld);
  else
    scatter_add_rows_kernel<__nv_bfloat16><<<grid, block, row_bytes * wpb, st>>>(
        (const __nv_bfloat16 *)packed, F, k, h, lkey, pl->d.brow, pl->d.brow_ptr, pl->d.brow_slot, pl->d.row_gid,
        (int)pl->nb, (__nv_bfloat16 *)dX, ld);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}
