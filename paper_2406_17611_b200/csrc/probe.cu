// Measurement aid (no counterpart in the paper): the rate at which this GPU serves random row gathers.
//
// The aggregation kernels read one feature row per stored adjacency entry, at random.  What bounds them is
// therefore not the streaming bandwidth of HBM but the rate of random 16..512-byte row reads out of L2 (rows
// that are reused) or DRAM (rows that are not).  This kernel measures exactly that with nothing else in the
// way: every group of lanes sums `per_out` rows of a table, picked by an index list, and writes one row.
// The benchmark runs it on a table that stays in L2 and on one that does not and reports the aggregation
// stages against those two rates.
#include "device_common.cuh"
#include "kernels.h"

namespace {

template <int G>
__global__ void __launch_bounds__(256) probe_gather_kernel(const uint4 *__restrict__ table, int64_t table_rows, int ld,
                                                           const int4 *__restrict__ index, int64_t out_rows, int quads,
                                                           uint4 *__restrict__ out) {
  const int64_t row = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) / G;
  const int gl = threadIdx.x % G;
  if (row >= out_rows) return;
  const int4 *ip = index + row * quads;
  const uint4 *base = table + gl;
  const int last = (int)(table_rows - 1);
  uint32_t acc[4] = {0u, 0u, 0u, 0u};
  for (int t = 0; t < quads; t += 2) {
    int c[8];
    const int4 a = __ldg(ip + t);
    const int4 b = t + 1 < quads ? __ldg(ip + t + 1) : a;
    c[0] = a.x, c[1] = a.y, c[2] = a.z, c[3] = a.w, c[4] = b.x, c[5] = b.y, c[6] = b.z, c[7] = b.w;
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = __ldg(base + (int64_t)min(max(c[u], 0), last) * ld);   // never out of the table
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      acc[0] ^= v[u].x;
      acc[1] ^= v[u].y;
      acc[2] ^= v[u].z;
      acc[3] ^= v[u].w;
    }
  }
  out[row * G + gl] = make_uint4(acc[0], acc[1], acc[2], acc[3]);
}

}  // namespace

extern "C" int varco_probe_gather(const void *table, int64_t table_rows, int32_t row_chunks, const int32_t *index,
                                  int64_t out_rows, int32_t per_out, void *out, void *stream) {
  if (!table || !index || !out || table_rows < 1 || out_rows < 1 || per_out < 4 || (per_out % 4) != 0)
    return VARCO_INVALID_ARG;
  if (row_chunks != 8 && row_chunks != 16 && row_chunks != 32) return VARCO_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(table) & 15u) || (reinterpret_cast<uintptr_t>(index) & 15u) ||
      (reinterpret_cast<uintptr_t>(out) & 15u))
    return VARCO_INVALID_ARG;
  const int threads = 256;
  const unsigned grid = (unsigned)((out_rows * row_chunks + threads - 1) / threads);
  cudaStream_t st = (cudaStream_t)stream;
  const uint4 *t4 = reinterpret_cast<const uint4 *>(table);
  const int4 *i4 = reinterpret_cast<const int4 *>(index);
  uint4 *o4 = reinterpret_cast<uint4 *>(out);
  if (row_chunks == 8)
    probe_gather_kernel<8><<<grid, threads, 0, st>>>(t4, table_rows, 8, i4, out_rows, per_out / 4, o4);
  else if (row_chunks == 16)
    probe_gather_kernel<16><<<grid, threads, 0, st>>>(t4, table_rows, 16, i4, out_rows, per_out / 4, o4);
  else
    probe_gather_kernel<32><<<grid, threads, 0, st>>>(t4, table_rows, 32, i4, out_rows, per_out / 4, o4);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}
