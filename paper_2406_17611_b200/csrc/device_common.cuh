// Device-side helpers shared by the kernels of libvarco.
#ifndef VARCO_DEVICE_COMMON_CUH_
#define VARCO_DEVICE_COMMON_CUH_

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "varco_internal.h"

#define VARCO_CUDA_CHECK(expr)                   \
  do {                                           \
    cudaError_t e__ = (expr);                    \
    if (e__ != cudaSuccess) return VARCO_CUDA;   \
  } while (0)

// every kernel launch of the library goes through this: count it, then check the launch status
void varco_count_launch();
#define VARCO_KERNEL_LAUNCHED()                  \
  do {                                           \
    varco_count_launch();                        \
    VARCO_CUDA_CHECK(cudaGetLastError());        \
  } while (0)

// ------------------------------------------------------------------------------------------
// Debug build (-DVARCO_DEBUG): every index a kernel gathers from or scatters to is checked against the extent
// of the array it addresses.  A failed check records a code in the translation unit's debug word and the access
// is skipped; nothing traps, the context stays usable.  varco_debug_status() collects the words.
// Codes: 11 source row, 12 destination row, 13 kept position of the aggregation kernels.  The index arrays the
// halo kernels walk are fixed at plan build time; the debug build validates them on the host when the plan is
// uploaded (varco_partition_upload returns BAD_GRAPH on a damaged image).
#ifdef VARCO_DEBUG
#ifdef __CUDACC__
static __device__ int varco_dbg_word;
__device__ __forceinline__ bool varco_dbg_ok(long long idx, long long limit, int code) {
  if (idx >= 0 && idx < limit) return true;
  atomicCAS(&varco_dbg_word, 0, code);
  return false;
}
// host side of one translation unit: read and clear its word
#define VARCO_DEFINE_DEBUG_READER(name)                                              \
  int name() {                                                                        \
    int v = 0, zero = 0;                                                              \
    if (cudaMemcpyFromSymbol(&v, varco_dbg_word, sizeof(int)) != cudaSuccess) return -1; \
    cudaMemcpyToSymbol(varco_dbg_word, &zero, sizeof(int));                           \
    return v;                                                                         \
  }
#endif
#define VARCO_DBG_OK(idx, limit, code) varco_dbg_ok((long long)(idx), (long long)(limit), (code))
#else
#define VARCO_DBG_OK(idx, limit, code) (true)
#define VARCO_DEFINE_DEBUG_READER(name) \
  int name() { return 0; }
#endif

// ------------------------------------------------------------------------------------------
// Shared-key permutation of [0, F): which positions of a row are sent (appendix "Compression
// Mechanism": chosen at random at the encoder, known to the decoder through a shared key).
// A 6-round balanced Feistel network over the smallest even-bit domain covering [0, F),
// cycle-walked into [0, F); keyed per (seed, epoch, layer, original node id).
namespace vperm {

constexpr uint64_t kPhi64 = 0x9E3779B97F4A7C15ull;  // floor(2^64 / golden ratio)
constexpr uint64_t kMulA = 0x6A09E667F3BCC909ull;   // frac(sqrt 2) 2^64, odd
constexpr uint64_t kMulB = 0xBB67AE8584CAA73Bull;   // frac(sqrt 3) 2^64, odd
constexpr uint32_t kGold32 = 0x9E3779B9u;           // floor(2^32 / golden ratio)

__host__ __device__ inline uint64_t mix(uint64_t x) {
  x ^= x >> 32;
  x *= kMulA;
  x ^= x >> 29;
  x *= kMulB;
  x ^= x >> 32;
  return x;
}

// the part of the row key that does not depend on the node: computed once on the host
inline uint64_t layer_key(varco_key_t key) {
  uint64_t a = mix(key.seed ^ kPhi64);
  a = mix(a + key.epoch);
  a = mix(a + key.layer);
  return a;
}

inline int half_bits(int F) {
  int bits = 0;
  while ((1ll << bits) < (long long)F) ++bits;
  if (bits < 2) bits = 2;
  if (bits & 1) ++bits;
  return bits / 2;
}

struct RowPerm {
  uint32_t rkg[6];  // round key times the round multiplier: (R + rk) G == R G + rk G (mod 2^32)
  uint32_t F;
  int h;

  __device__ __forceinline__ void init(uint64_t layer_key, uint32_t node, uint32_t width, int half) {
    uint64_t a = mix(layer_key + (uint64_t)node);
#pragma unroll
    for (int i = 0; i < 6; ++i) rkg[i] = (uint32_t)(mix(a + (uint64_t)(i + 1) * kPhi64) >> 32) * kGold32;
    F = width;
    h = half;
  }
  __device__ __forceinline__ uint32_t enc(uint32_t x) const {
    const int sh = 32 - h;
    uint32_t L = x >> h, R = x & ((1u << h) - 1u);
#pragma unroll
    for (int i = 0; i < 6; i += 2) {
      L ^= (R * kGold32 + rkg[i]) >> sh;
      R ^= (L * kGold32 + rkg[i + 1]) >> sh;
    }
    return (L << h) | R;
  }
  // position of the m-th value that is sent
  __device__ __forceinline__ uint32_t pi(uint32_t m) const {
    uint32_t x = enc(m);
    while (x >= F) x = enc(x);
    return x;
  }
};

}  // namespace vperm

// ------------------------------------------------------------------------------------------
template <typename T> struct ElemTraits;
template <> struct ElemTraits<float> {
  static constexpr int kVec = 4;  // elements per 16 bytes
  __device__ static __forceinline__ float to_f(float v) { return v; }
  __device__ static __forceinline__ float from_f(float v) { return v; }
};
template <> struct ElemTraits<__nv_bfloat16> {
  static constexpr int kVec = 8;
  __device__ static __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
  __device__ static __forceinline__ __nv_bfloat16 from_f(float v) { return __float2bfloat16_rn(v); }
};

// raw element type of the same width, for bit-exact copies
template <typename T> struct ElemBits;
template <> struct ElemBits<float> { typedef uint32_t type; };
template <> struct ElemBits<__nv_bfloat16> { typedef uint16_t type; };

// unpack 16 bytes of T into floats
__device__ __forceinline__ void unpack16(const uint4 &v, float (&f)[4], float) {
  f[0] = __uint_as_float(v.x);
  f[1] = __uint_as_float(v.y);
  f[2] = __uint_as_float(v.z);
  f[3] = __uint_as_float(v.w);
}
__device__ __forceinline__ void unpack16(const uint4 &v, float (&f)[8], __nv_bfloat16) {
  f[0] = __uint_as_float(v.x << 16);
  f[1] = __uint_as_float(v.x & 0xFFFF0000u);
  f[2] = __uint_as_float(v.y << 16);
  f[3] = __uint_as_float(v.y & 0xFFFF0000u);
  f[4] = __uint_as_float(v.z << 16);
  f[5] = __uint_as_float(v.z & 0xFFFF0000u);
  f[6] = __uint_as_float(v.w << 16);
  f[7] = __uint_as_float(v.w & 0xFFFF0000u);
}
__device__ __forceinline__ uint4 pack16(const float (&f)[4], float) {
  return make_uint4(__float_as_uint(f[0]), __float_as_uint(f[1]), __float_as_uint(f[2]), __float_as_uint(f[3]));
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&p);
}
__device__ __forceinline__ uint4 pack16(const float (&f)[8], __nv_bfloat16) {
  return make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]), pack_bf16x2(f[4], f[5]),
                    pack_bf16x2(f[6], f[7]));
}

#ifdef __CUDACC__
// lanes of the G-lane group this thread belongs to (G a power of two, groups aligned inside the warp)
template <int G> __device__ __forceinline__ unsigned group_mask() {
  if (G == 32) return 0xFFFFFFFFu;
  const unsigned lane = threadIdx.x & 31u;
  return ((1u << (G & 31)) - 1u) << (lane & ~(unsigned)(G - 1));
}

// Round keys of one row, computed by six lanes of the group and shared by shuffle (G >= 8).
template <int G>
__device__ __forceinline__ void init_perm(vperm::RowPerm &pm, uint64_t lkey, uint32_t node, uint32_t F, int h, int gl,
                                          unsigned gmask) {
  const uint64_t a = vperm::mix(lkey + (uint64_t)node);
  uint32_t mine = 0;
  if (gl < 6) mine = (uint32_t)(vperm::mix(a + (uint64_t)(gl + 1) * vperm::kPhi64) >> 32) * vperm::kGold32;
#pragma unroll
  for (int i = 0; i < 6; ++i) pm.rkg[i] = __shfl_sync(gmask, mine, i, G);
  pm.F = F;
  pm.h = h;
}

#endif

static inline int64_t round_up64(int64_t a, int64_t b) { return (a + b - 1) / b * b; }

#endif  // VARCO_DEVICE_COMMON_CUH_
