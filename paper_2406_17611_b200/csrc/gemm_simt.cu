// Feature-transform GEMMs on the CUDA cores with fp32 accumulation.
//
// Eq. (2) of the paper with two taps: Y = rho(X W_self + Agg W_neigh + b) (SAGE) or
// Y = rho(Agg W + b) (GCN), and the matching backward products dZ W^T and [X | Agg]^T dZ.
// This path serves the fp32 configurations, whose 1e-5 tolerance rules out bf16 / tf32 tensor
// core inputs; the bf16 configurations use the tcgen05 kernels instead.
#include <algorithm>
#include <type_traits>

#include "device_common.cuh"

// SM count of the current device (sizes the split reductions)
static int simt_sms() {
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
      sms = 148;   // no device visible (a build host): the part this library targets
  }
  return sms;
}

namespace {

constexpr int BM = 64, BN = 64, BK = 16, TM = 4, TN = 4;

template <typename T> __device__ __forceinline__ float ldf(const T *p) { return ElemTraits<T>::to_f(*p); }

// One (A, B) operand pair of a concatenated-K product.
template <typename T> struct Operand {
  const T *A;
  int64_t lda;
  const T *B;
  int64_t ldb;
  int K;
};

// C[M x N] = epilogue( sum_pairs A_p op B_p ), with
//   A_T == false: A_p is [M x K_p] row-major;   A_T == true: A_p is [K_p x M] row-major (A^T product)
//   B_T == false: B_p is [K_p x N] row-major;   B_T == true: B_p is [N x K_p] row-major (B^T product)
// With A_T the K range [k_begin, k_end) of pair 0 is split over blockIdx.z and every z writes its
// own partial result (C + z * M * ldc); a second kernel sums the partials in order.
template <typename T, typename TC, bool A_T, bool B_T>
__global__ void __launch_bounds__(256) gemm_kernel(int M, int N, Operand<T> p0, Operand<T> p1, int npairs,
                                                   const float *__restrict__ bias, int relu, TC *__restrict__ C,
                                                   int64_t ldc, int k_chunk) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs[BK][BN + 4];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
  float acc[TM][TN];
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

  for (int pi = 0; pi < npairs; ++pi) {
    const Operand<T> p = pi == 0 ? p0 : p1;
    int kb = 0, ke = p.K;
    if (A_T) {
      kb = blockIdx.z * k_chunk;
      ke = min(p.K, kb + k_chunk);
    }
    for (int k0 = kb; k0 < ke; k0 += BK) {
      // A tile -> As[kk][m]
      for (int idx = threadIdx.x; idx < BM * BK; idx += 256) {
        int m, kk;
        if (A_T) {
          m = idx % BM;
          kk = idx / BM;
        } else {
          kk = idx % BK;
          m = idx / BK;
        }
        const int gm = m0 + m, gk = k0 + kk;
        float v = 0.f;
        if (gm < M && gk < ke) v = A_T ? ldf(p.A + (int64_t)gk * p.lda + gm) : ldf(p.A + (int64_t)gm * p.lda + gk);
        As[kk][m] = v;
      }
      // B tile -> Bs[kk][n]
      for (int idx = threadIdx.x; idx < BN * BK; idx += 256) {
        int nn, kk;
        if (B_T) {
          kk = idx % BK;
          nn = idx / BK;
        } else {
          nn = idx % BN;
          kk = idx / BN;
        }
        const int gn = n0 + nn, gk = k0 + kk;
        float v = 0.f;
        if (gn < N && gk < ke) v = B_T ? ldf(p.B + (int64_t)gn * p.ldb + gk) : ldf(p.B + (int64_t)gk * p.ldb + gn);
        Bs[kk][nn] = v;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < BK; ++kk) {
        float a[TM], b[TN];
#pragma unroll
        for (int i = 0; i < TM; ++i) a[i] = As[kk][ty * TM + i];
#pragma unroll
        for (int j = 0; j < TN; ++j) b[j] = Bs[kk][tx * TN + j];
#pragma unroll
        for (int i = 0; i < TM; ++i)
#pragma unroll
          for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
      }
      __syncthreads();
    }
  }
  TC *Cz = C;
  if (A_T) Cz += (int64_t)blockIdx.z * M * ldc;
#pragma unroll
  for (int i = 0; i < TM; ++i) {
    const int gm = m0 + ty * TM + i;
    if (gm >= M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int gn = n0 + tx * TN + j;
      if (gn >= N) continue;
      float v = acc[i][j];
      if (bias) v += bias[gn];
      if (relu) v = fmaxf(v, 0.f);
      Cz[(int64_t)gm * ldc + gn] = ElemTraits<TC>::from_f(v);
    }
  }
}

// fp32 products of the fp32 configurations: 128 x 64 x 16 tiles, 8 x 4 outputs per thread, 16-byte global loads
// and shared-memory reads, the next tile fetched into registers while the current one is multiplied (two
// shared-memory buffers, one barrier per step).  Same contract as gemm_kernel<float, float, A_T, B_T>.
constexpr int SM = 128, SN = 64, SK = 16;

__device__ __forceinline__ float4 ld4(const float *p, bool vec, int valid) {
  // 4 consecutive floats of which the first `valid` exist; one 16-byte load when the address allows it
  if (vec && valid >= 4) return __ldg(reinterpret_cast<const float4 *>(p));
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (valid > 0) v.x = __ldg(p);
  if (valid > 1) v.y = __ldg(p + 1);
  if (valid > 2) v.z = __ldg(p + 2);
  if (valid > 3) v.w = __ldg(p + 3);
  return v;
}

template <bool A_T, bool B_T>
__global__ void __launch_bounds__(256, 2) sgemm_kernel(int M, int N, Operand<float> p0, Operand<float> p1, int npairs,
                                                       const float *__restrict__ bias, int relu, float *__restrict__ C,
                                                       int64_t ldc, int k_chunk) {
  __shared__ __align__(16) float As[2][SK][SM + 4];
  __shared__ __align__(16) float Bs[2][SK][SN + 4];
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
  const int m0 = blockIdx.x * SM, n0 = blockIdx.y * SN;
  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  for (int pi = 0; pi < npairs; ++pi) {
    const Operand<float> p = pi == 0 ? p0 : p1;
    int kb = 0, ke = p.K;
    if (A_T) {
      kb = blockIdx.z * k_chunk;
      ke = min(p.K, kb + k_chunk);
    }
    if (ke <= kb) continue;
    const bool avec = (reinterpret_cast<uintptr_t>(p.A) & 15u) == 0 && (p.lda & 3) == 0 && (A_T || (kb & 3) == 0);
    const bool bvec = (reinterpret_cast<uintptr_t>(p.B) & 15u) == 0 && (p.ldb & 3) == 0 && (!B_T || (kb & 3) == 0);
    float4 ra[2], rb;
    auto fetch = [&](int k0) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int idx = tid + i * 256;
        if (A_T) {   // A is [K x M]: 16 rows of 128 consecutive outputs
          const int kk = idx / 32, m = m0 + (idx % 32) * 4;
          const int gk = k0 + kk;
          ra[i] = (gk < ke) ? ld4(p.A + (int64_t)gk * p.lda + m, avec, M - m) : make_float4(0.f, 0.f, 0.f, 0.f);
        } else {     // A is [M x K]: 128 rows of 16 consecutive k
          const int m = m0 + idx / 4, gk = k0 + (idx % 4) * 4;
          ra[i] = (m < M) ? ld4(p.A + (int64_t)m * p.lda + gk, avec, ke - gk) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
      }
      if (B_T) {     // B is [N x K]: 64 rows of 16 consecutive k
        const int nn = n0 + tid / 4, gk = k0 + (tid % 4) * 4;
        rb = (nn < N) ? ld4(p.B + (int64_t)nn * p.ldb + gk, bvec, ke - gk) : make_float4(0.f, 0.f, 0.f, 0.f);
      } else {       // B is [K x N]: 16 rows of 64 consecutive outputs
        const int gk = k0 + tid / 16, nn = n0 + (tid % 16) * 4;
        rb = (gk < ke) ? ld4(p.B + (int64_t)gk * p.ldb + nn, bvec, N - nn) : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    };
    auto stash = [&](int buf) {
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int idx = tid + i * 256;
        if (A_T) {
          *reinterpret_cast<float4 *>(&As[buf][idx / 32][(idx % 32) * 4]) = ra[i];
        } else {
          const int m = idx / 4, kk = (idx % 4) * 4;
          As[buf][kk][m] = ra[i].x;
          As[buf][kk + 1][m] = ra[i].y;
          As[buf][kk + 2][m] = ra[i].z;
          As[buf][kk + 3][m] = ra[i].w;
        }
      }
      if (B_T) {
        const int nn = tid / 4, kk = (tid % 4) * 4;
        Bs[buf][kk][nn] = rb.x;
        Bs[buf][kk + 1][nn] = rb.y;
        Bs[buf][kk + 2][nn] = rb.z;
        Bs[buf][kk + 3][nn] = rb.w;
      } else {
        *reinterpret_cast<float4 *>(&Bs[buf][tid / 16][(tid % 16) * 4]) = rb;
      }
    };
    const int steps = (ke - kb + SK - 1) / SK;
    __syncthreads();          // the buffers of the previous operand pair are no longer read
    fetch(kb);
    stash(0);
    __syncthreads();
    for (int s = 0; s < steps; ++s) {
      const int buf = s & 1;
      if (s + 1 < steps) fetch(kb + (s + 1) * SK);
#pragma unroll
      for (int kk = 0; kk < SK; ++kk) {
        const float4 a0 = *reinterpret_cast<const float4 *>(&As[buf][kk][ty * 8]);
        const float4 a1 = *reinterpret_cast<const float4 *>(&As[buf][kk][ty * 8 + 4]);
        const float4 b = *reinterpret_cast<const float4 *>(&Bs[buf][kk][tx * 4]);
        const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
        const float bb[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], bb[j], acc[i][j]);
      }
      if (s + 1 < steps) stash(buf ^ 1);
      __syncthreads();
    }
  }
  float *Cz = C;
  if (A_T) Cz += (int64_t)blockIdx.z * M * ldc;
  const int gn = n0 + tx * 4;
  const bool cvec = (reinterpret_cast<uintptr_t>(Cz) & 15u) == 0 && (ldc & 3) == 0 && gn + 3 < N;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int gm = m0 + ty * 8 + i;
    if (gm >= M) continue;
    float v[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      v[j] = acc[i][j];
      if (bias && gn + j < N) v[j] += bias[gn + j];
      if (relu) v[j] = fmaxf(v[j], 0.f);
    }
    if (cvec) {
      *reinterpret_cast<float4 *>(Cz + (int64_t)gm * ldc + gn) = make_float4(v[0], v[1], v[2], v[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
        if (gn + j < N) Cz[(int64_t)gm * ldc + gn + j] = v[j];
    }
  }
}

// out[i] = sum_z partial[z * count + i], z ascending (deterministic)
__global__ void reduce_partials_kernel(const float *__restrict__ partial, int64_t count, int splits,
                                       float *__restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= count) return;
  float s = 0.f;
#pragma unroll 16
  for (int z = 0; z < splits; ++z) s += partial[(int64_t)z * count + i];
  out[i] = s;
}

// partial[z][c] = sum over the rows of chunk z of dZ[row][c].  Block = 32 x 8 threads: x owns a 16-byte
// chunk of columns, y strides over the rows; the eight row-partials meet in shared memory in y order.
// With MASK the rows summed are dY where Y > 0 (else 0), and they are written to dZ on the way: the ReLU
// mask of the backward pass and the bias gradient in one pass over dY.
template <typename T, bool MASK>
__global__ void __launch_bounds__(256) colsum_kernel(const T *__restrict__ dZ, int64_t ld, int rows, int N, int nv,
                                                     int row_chunk, float *__restrict__ partial,
                                                     const T *__restrict__ Y, int64_t ldy, T *__restrict__ dZout,
                                                     int64_t ldout) {
  constexpr int V = ElemTraits<T>::kVec;
  __shared__ float red[8][32][V + 1];
  const int ch = blockIdx.x * 32 + threadIdx.x;
  const int r0 = blockIdx.y * row_chunk, r1 = min(rows, r0 + row_chunk);
  float s[V];
#pragma unroll
  for (int j = 0; j < V; ++j) s[j] = 0.f;
  if (ch < nv)
    for (int r = r0 + threadIdx.y; r < r1; r += 16) {
      // two rows in flight, added in row order
      const bool two = r + 8 < r1;
      const int rb = two ? r + 8 : r;
      const uint4 qa = __ldg(reinterpret_cast<const uint4 *>(dZ + (int64_t)r * ld) + ch);
      const uint4 qb = __ldg(reinterpret_cast<const uint4 *>(dZ + (int64_t)rb * ld) + ch);
      float fa[V], fb[V];
      unpack16(qa, fa, T());
      unpack16(qb, fb, T());
      if (MASK) {
        const uint4 ya4 = __ldg(reinterpret_cast<const uint4 *>(Y + (int64_t)r * ldy) + ch);
        const uint4 yb4 = __ldg(reinterpret_cast<const uint4 *>(Y + (int64_t)rb * ldy) + ch);
        float ya[V], yb[V];
        unpack16(ya4, ya, T());
        unpack16(yb4, yb, T());
#pragma unroll
        for (int j = 0; j < V; ++j) {
          fa[j] = ya[j] > 0.f ? fa[j] : 0.f;
          fb[j] = yb[j] > 0.f ? fb[j] : 0.f;
        }
        reinterpret_cast<uint4 *>(dZout + (int64_t)r * ldout)[ch] = pack16(fa, T());
        if (two) reinterpret_cast<uint4 *>(dZout + (int64_t)rb * ldout)[ch] = pack16(fb, T());
      }
#pragma unroll
      for (int j = 0; j < V; ++j) {
        s[j] += fa[j];
        if (two) s[j] += fb[j];
      }
    }
#pragma unroll
  for (int j = 0; j < V; ++j) red[threadIdx.y][threadIdx.x][j] = s[j];
  __syncthreads();
  if (threadIdx.y == 0 && ch < nv) {
#pragma unroll
    for (int j = 0; j < V; ++j) {
      float t = 0.f;
      for (int y = 0; y < 8; ++y) t += red[y][threadIdx.x][j];
      const int c = ch * V + j;
      if (c < N) partial[(int64_t)blockIdx.y * N + c] = t;
    }
  }
}

// dZ = dY where Y > 0, else 0; 16 bytes per thread
template <typename T>
__global__ void relu_mask_kernel(const T *__restrict__ Y, int64_t ldy, const T *__restrict__ dY, int64_t lddy,
                                 T *__restrict__ dZ, int64_t lddz, int rows, int nv) {
  constexpr int V = ElemTraits<T>::kVec;
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)rows * nv) return;
  const int64_t r = idx / nv;
  const int ch = (int)(idx % nv);
  float y[V], g[V];
  unpack16(reinterpret_cast<const uint4 *>(Y + r * ldy)[ch], y, T());
  unpack16(reinterpret_cast<const uint4 *>(dY + r * lddy)[ch], g, T());
#pragma unroll
  for (int i = 0; i < V; ++i) g[i] = y[i] > 0.f ? g[i] : 0.f;
  reinterpret_cast<uint4 *>(dZ + r * lddz)[ch] = pack16(g, T());
}

template <typename T>
int fwd_t(int n, int F_in, int F_out, const T *X, int64_t ldx, const T *Agg, int64_t lda, const T *Ws, const T *Wn,
          const float *bias, int relu, T *Y, int64_t ldy, cudaStream_t st) {
  Operand<T> pa{Agg, lda, Wn, F_out, F_in}, px{X, ldx, Ws, F_out, F_in};
  if constexpr (std::is_same<T, float>::value) {
    dim3 grid((n + SM - 1) / SM, (F_out + SN - 1) / SN, 1);
    sgemm_kernel<false, false><<<grid, 256, 0, st>>>(n, F_out, pa, px, Ws ? 2 : 1, bias, relu, Y, ldy, 0);
  } else {
    dim3 grid((n + BM - 1) / BM, (F_out + BN - 1) / BN, 1);
    gemm_kernel<T, T, false, false><<<grid, 256, 0, st>>>(n, F_out, pa, px, Ws ? 2 : 1, bias, relu, Y, ldy, 0);
  }
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

template <typename T>
int dx_t(int n, int F_in, int F_out, const T *dZ, int64_t lddz, const T *W, T *out, int64_t ldo, cudaStream_t st) {
  Operand<T> p{dZ, lddz, W, F_out, F_out};
  if constexpr (std::is_same<T, float>::value) {
    dim3 grid((n + SM - 1) / SM, (F_in + SN - 1) / SN, 1);
    sgemm_kernel<false, true><<<grid, 256, 0, st>>>(n, F_in, p, p, 1, nullptr, 0, out, ldo, 0);
  } else {
    dim3 grid((n + BM - 1) / BM, (F_in + BN - 1) / BN, 1);
    gemm_kernel<T, T, false, true><<<grid, 256, 0, st>>>(n, F_in, p, p, 1, nullptr, 0, out, ldo, 0);
  }
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

}  // namespace

// scratch floats needed by varco_simt_gemm_dw (split partials) and by varco_colsum
// splits of the node range of a weight-gradient product: about two CTAs per SM over all tiles
static int dw_splits(int tiles) {
  int splits = (2 * simt_sms() + tiles - 1) / tiles;
  return splits < 1 ? 1 : splits;
}

size_t varco_simt_dw_scratch_bytes(int F_in, int F_out) {
  // the larger of the two tilings' split counts (fp32 tiles are 128 x 64, the generic ones 64 x 64)
  const int t0 = ((F_in + BM - 1) / BM) * ((F_out + BN - 1) / BN), t1 = ((F_in + SM - 1) / SM) * ((F_out + SN - 1) / SN);
  const int splits = std::max(dw_splits(t0), dw_splits(t1)) + 1;
  size_t a = (size_t)splits * (size_t)F_in * F_out * sizeof(float);
  size_t b = (size_t)4 * simt_sms() * F_out * sizeof(float);   // column-sum partials
  return (a > b ? a : b) + 256;
}

int varco_simt_gemm_fwd(int n, int F_in, int F_out, varco_dtype_t dt, const void *X, int64_t ldx, const void *Agg,
                        int64_t lda, const void *Ws, const void *Wn, const float *bias, int relu, void *Y,
                        int64_t ldy, cudaStream_t st) {
  if (dt == VARCO_F32)
    return fwd_t<float>(n, F_in, F_out, (const float *)X, ldx, (const float *)Agg, lda, (const float *)Ws,
                        (const float *)Wn, bias, relu, (float *)Y, ldy, st);
  return fwd_t<__nv_bfloat16>(n, F_in, F_out, (const __nv_bfloat16 *)X, ldx, (const __nv_bfloat16 *)Agg, lda,
                              (const __nv_bfloat16 *)Ws, (const __nv_bfloat16 *)Wn, bias, relu, (__nv_bfloat16 *)Y,
                              ldy, st);
}

// out[n x F_in] = dZ[n x F_out] W^T, W being [F_in x F_out]
int varco_simt_gemm_dx(int n, int F_in, int F_out, varco_dtype_t dt, const void *dZ, int64_t lddz, const void *W,
                       void *out, int64_t ldo, cudaStream_t st) {
  if (dt == VARCO_F32)
    return dx_t<float>(n, F_in, F_out, (const float *)dZ, lddz, (const float *)W, (float *)out, ldo, st);
  return dx_t<__nv_bfloat16>(n, F_in, F_out, (const __nv_bfloat16 *)dZ, lddz, (const __nv_bfloat16 *)W,
                             (__nv_bfloat16 *)out, ldo, st);
}

// dW[F_in x F_out] = A[n x F_in]^T dZ[n x F_out] (fp32 out), split over n with ordered reduction.
template <typename T>
static int dw_t(int n, int F_in, int F_out, const T *A, int64_t lda, const T *dZ, int64_t lddz, float *dW,
                float *scratch, cudaStream_t st) {
  constexpr bool f32 = std::is_same<T, float>::value;
  const int tm = f32 ? SM : BM, tn = f32 ? SN : BN;
  const int tiles = ((F_in + tm - 1) / tm) * ((F_out + tn - 1) / tn);
  int splits = dw_splits(tiles);
  int chunk = (n + splits - 1) / splits;
  chunk = (chunk + BK - 1) / BK * BK;
  splits = (n + chunk - 1) / chunk;
  dim3 grid((F_in + tm - 1) / tm, (F_out + tn - 1) / tn, splits);
  Operand<T> p{A, lda, dZ, lddz, n};
  if constexpr (f32)
    sgemm_kernel<true, false><<<grid, 256, 0, st>>>(F_in, F_out, p, p, 1, nullptr, 0, scratch, F_out, chunk);
  else
    gemm_kernel<T, float, true, false><<<grid, 256, 0, st>>>(F_in, F_out, p, p, 1, nullptr, 0, scratch, F_out, chunk);
  VARCO_KERNEL_LAUNCHED();
  const int64_t count = (int64_t)F_in * F_out;
  reduce_partials_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(scratch, count, splits, dW);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

int varco_simt_gemm_dw(int n, int F_in, int F_out, varco_dtype_t dt, const void *A, int64_t lda, const void *dZ,
                       int64_t lddz, float *dW, float *scratch, cudaStream_t st) {
  if (dt == VARCO_F32) return dw_t<float>(n, F_in, F_out, (const float *)A, lda, (const float *)dZ, lddz, dW, scratch, st);
  return dw_t<__nv_bfloat16>(n, F_in, F_out, (const __nv_bfloat16 *)A, lda, (const __nv_bfloat16 *)dZ, lddz, dW,
                             scratch, st);
}

namespace {
template <typename T>
int colsum_t(int n, int F_out, const T *dZ, int64_t lddz, float *out, float *scratch, const T *Y, int64_t ldy,
             T *dZout, int64_t ldout, cudaStream_t st) {
  int splits = 4 * simt_sms();
  int chunk = (n + splits - 1) / splits;
  if (chunk < 1) chunk = 1;
  splits = (n + chunk - 1) / chunk;
  constexpr int V = ElemTraits<T>::kVec;
  const int nv = (F_out + V - 1) / V;
  dim3 grid((nv + 31) / 32, splits), block(32, 8);
  if (Y)
    colsum_kernel<T, true><<<grid, block, 0, st>>>(dZ, lddz, n, F_out, nv, chunk, scratch, Y, ldy, dZout, ldout);
  else
    colsum_kernel<T, false><<<grid, block, 0, st>>>(dZ, lddz, n, F_out, nv, chunk, scratch, nullptr, 0, nullptr, 0);
  VARCO_KERNEL_LAUNCHED();
  reduce_partials_kernel<<<(F_out + 255) / 256, 256, 0, st>>>(scratch, F_out, splits, out);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}
}  // namespace

int varco_colsum(int n, int F_out, varco_dtype_t dt, const void *dZ, int64_t lddz, float *out, float *scratch,
                 cudaStream_t st) {
  if (dt == VARCO_F32)
    return colsum_t<float>(n, F_out, (const float *)dZ, lddz, out, scratch, nullptr, 0, nullptr, 0, st);
  return colsum_t<__nv_bfloat16>(n, F_out, (const __nv_bfloat16 *)dZ, lddz, out, scratch, nullptr, 0, nullptr, 0, st);
}

// dZ = dY where Y > 0 (else 0) and out[c] = sum over the rows of dZ[.][c], in one pass over dY and Y
int varco_relu_mask_colsum(int n, int F_out, varco_dtype_t dt, const void *Y, int64_t ldy, const void *dY, int64_t lddy,
                           void *dZ, int64_t lddz, float *out, float *scratch, cudaStream_t st) {
  if (dt == VARCO_F32)
    return colsum_t<float>(n, F_out, (const float *)dY, lddy, out, scratch, (const float *)Y, ldy, (float *)dZ, lddz, st);
  return colsum_t<__nv_bfloat16>(n, F_out, (const __nv_bfloat16 *)dY, lddy, out, scratch, (const __nv_bfloat16 *)Y, ldy,
                                 (__nv_bfloat16 *)dZ, lddz, st);
}

int varco_relu_mask(int n, int F_out, varco_dtype_t dt, const void *Y, int64_t ldy, const void *dY, int64_t lddy,
                    void *dZ, int64_t lddz, cudaStream_t st) {
  const int V = dt == VARCO_F32 ? 4 : 8;
  const int nv = (F_out + V - 1) / V;
  const int64_t total = (int64_t)n * nv;
  dim3 grid((unsigned)((total + 255) / 256));
  if (dt == VARCO_F32)
    relu_mask_kernel<float><<<grid, 256, 0, st>>>((const float *)Y, ldy, (const float *)dY, lddy, (float *)dZ, lddz, n,
                                                  nv);
  else
    relu_mask_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16 *)Y, ldy, (const __nv_bfloat16 *)dY,
                                                          lddy, (__nv_bfloat16 *)dZ, lddz, n, nv);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}
