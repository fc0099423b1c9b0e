// Feature-transform GEMMs on the CUDA cores with fp32 accumulation.
//
// Eq. (2) of the paper with two taps: Y = rho(X W_self + Agg W_neigh + b) (SAGE) or
// Y = rho(Agg W + b) (GCN), and the matching backward products dZ W^T and [X | Agg]^T dZ.
// This path serves the fp32 configurations, whose 1e-5 tolerance rules out bf16 / tf32 tensor
// core inputs; the bf16 configurations use the tcgen05 kernels instead.
#include "device_common.cuh"

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
  dim3 grid((n + BM - 1) / BM, (F_out + BN - 1) / BN, 1);
  Operand<T> pa{Agg, lda, Wn, F_out, F_in}, px{X, ldx, Ws, F_out, F_in};
  gemm_kernel<T, T, false, false><<<grid, 256, 0, st>>>(n, F_out, pa, px, Ws ? 2 : 1, bias, relu, Y, ldy, 0);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

template <typename T>
int dx_t(int n, int F_in, int F_out, const T *dZ, int64_t lddz, const T *W, T *out, int64_t ldo, cudaStream_t st) {
  dim3 grid((n + BM - 1) / BM, (F_in + BN - 1) / BN, 1);
  Operand<T> p{dZ, lddz, W, F_out, F_out};
  gemm_kernel<T, T, false, true><<<grid, 256, 0, st>>>(n, F_in, p, p, 1, nullptr, 0, out, ldo, 0);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

}  // namespace

// scratch floats needed by varco_simt_gemm_dw (split partials) and by varco_colsum
size_t varco_simt_dw_scratch_bytes(int F_in, int F_out) {
  const int tiles = ((F_in + BM - 1) / BM) * ((F_out + BN - 1) / BN);
  int splits = (2 * 148 + tiles - 1) / tiles;
  if (splits < 1) splits = 1;
  size_t a = (size_t)splits * (size_t)F_in * F_out * sizeof(float);
  size_t b = (size_t)4 * 148 * F_out * sizeof(float);   // column-sum partials
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
  const int tiles = ((F_in + BM - 1) / BM) * ((F_out + BN - 1) / BN);
  int splits = (2 * 148 + tiles - 1) / tiles;
  int chunk = (n + splits - 1) / splits;
  chunk = (chunk + BK - 1) / BK * BK;
  splits = (n + chunk - 1) / chunk;
  dim3 grid((F_in + BM - 1) / BM, (F_out + BN - 1) / BN, splits);
  Operand<T> p{A, lda, dZ, lddz, n};
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
  int splits = 4 * 148;
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
