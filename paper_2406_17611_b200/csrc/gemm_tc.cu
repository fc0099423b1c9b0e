// Feature-transform GEMMs on the 5th-generation tensor cores (tcgen05 + TMEM), operands staged by TMA.
//
// Eq. (2) of the paper with two taps, for bf16 layers with fp32 accumulation:
//   forward   Y = rho([X | Agg] [W_self ; W_neigh] + b)         (concatenated K, bias/ReLU fused)
//   backward  [dX_self | dAgg] = dZ [W_self ; W_neigh]^T
//             [dW_self ; dW_neigh] = [X | Agg]^T dZ             (reduction over all nodes)
//
// Kernel 1 (rows_kernel): M = nodes.  A tiles [128 nodes x 64 features] are K-major straight from
// the activation matrices; B tiles come from a repacked, zero-padded K-major copy of the weights.
// One CTA per SM, persistent over (node tile, output tile) work items; warp 8 issues the TMA loads,
// warp 9 issues tcgen05.mma into one of two TMEM accumulators, warps 0-7 drain the other accumulator
// (tcgen05.ld, two warps per TMEM lane quarter), apply bias / ReLU, convert, stage 64-column slabs in
// swizzled shared-memory tiles and write them with TMA stores.
//
// Kernel 2 (dw_kernel): the reduction runs over nodes, so both operands are used MN-major: TMA
// boxes of [64 nodes x 64 features] land in shared memory exactly as loaded from the row-major
// activations and the instruction descriptor marks A and B as MN-major.  Each CTA owns up to two
// 128-feature tiles and a contiguous range of nodes; fp32 partial results go to scratch and are
// summed in a fixed order.
//
// Every mbarrier wait is bounded: on expiry the kernel raises an error flag in global memory,
// every role leaves its loop, TMEM is released and the kernel returns.
#include <cuda.h>

#include <cstring>

#include "device_common.cuh"
#include "kernels.h"

namespace {

constexpr int kStagesRows = 4;
constexpr int kStagesDw = 3;
constexpr int kBlockM = 128;     // UMMA M
constexpr int kBlockK = 64;      // bf16 elements per 128-byte swizzle span
constexpr int kUmmaK = 16;
constexpr uint32_t kTmemCols = 512;
constexpr int kThreads = 320;    // warps 0-7 epilogue (two per TMEM lane quarter), 8 TMA, 9 MMA
constexpr int kEpiWarps = 8;
constexpr int kTmaWarp = 8, kMmaWarp = 9;
constexpr int kThreadsDw = 192;  // dW kernel: warps 0-3 epilogue, 4 TMA, 5 MMA
constexpr uint32_t kSpinLimit = 1u << 24;
constexpr long long kSpinClocks = 2000000000ll;   // about one second of SM clocks

// ------------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the flags) when the limit is hit or another role gave up.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_smem, int *err, int code) {
  const long long t0 = clock64();
  for (uint32_t it = 0; it < kSpinLimit; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u) {
      if (*abort_smem) return false;
      if (clock64() - t0 > kSpinClocks) break;
    }
  }
  *abort_smem = 1;
  atomicCAS(err, 0, code);
  return false;
}

__device__ __forceinline__ void tma_load_2d(void *smem_dst, const CUtensorMap *tmap, int x, int y, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(smem_dst)),
      "l"(reinterpret_cast<uint64_t>(tmap)), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}

__device__ __forceinline__ void tmem_alloc(uint32_t *slot_smem, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot_smem)), "r"(cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
      "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the mbarrier once every tcgen05.mma issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint64_t *bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle, Blackwell descriptor version 1.
//   K-major operand : rows of 64 bf16 (128 B), 8-row groups 1024 B apart (SBO); LBO unused (1).
//   MN-major operand: rows are K indices holding 64 contiguous MN elements (128 B); 8-row K groups
//                     1024 B apart (SBO); successive 64-element MN chunks `lbo_bytes` apart (LBO).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= 1ull << 46;   // descriptor version
  d |= 2ull << 61;   // SWIZZLE_128B
  return d;
}
// Instruction descriptor of kind::f16 with bf16 inputs and fp32 accumulation.
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, int a_mn_major, int b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

// ------------------------------------------------------------------------------------------ kernel 1
struct RowsParams {
  CUtensorMap tmA[2];   // activations, box {64, 128}
  CUtensorMap tmB;      // packed weights [n_tiles * N_tile rows][(kb0 + kb1) * 64], box {64, N_tile}
  CUtensorMap tmOut[4]; // outputs of the n tiles: [M x valid columns], box {64, 32}, for the epilogue's stores
  int kblocks[2];
  int num_a;
  int M, m_tiles, n_tiles, N_tile;
  __nv_bfloat16 *out[4];
  int64_t ldo[4];
  int ncols[4];         // valid output columns of the tile
  int col0[4];          // first destination column
  const float *bias;    // length >= ncols of tile 0 (forward only) or nullptr
  int relu;
  int *err;
};

struct RowsSmem {
  uint64_t full[kStagesRows], empty[kStagesRows], tfull[2], tempty[2];
  uint32_t tmem_base;
  int abort_flag;
  float bias[256];
};

__global__ void __launch_bounds__(kThreads, 1) rows_kernel(const __grid_constant__ RowsParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t a_bytes = kBlockM * kBlockK * 2;
  const uint32_t b_bytes = (uint32_t)p.N_tile * kBlockK * 2;
  const uint32_t b_stride = 256 * kBlockK * 2;
  uint8_t *sA = base;
  uint8_t *sB = base + kStagesRows * a_bytes;
  uint8_t *stage_base = sB + kStagesRows * b_stride;   // 8 x 4 KB epilogue tiles (1024-byte aligned)
  RowsSmem *sh = reinterpret_cast<RowsSmem *>(stage_base + 8 * 4096);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  volatile int *abort_flag = &sh->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStagesRows; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(&sh->tfull[a], 1);
      mbar_init(&sh->tempty[a], kEpiWarps);
    }
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int i = threadIdx.x; i < 256; i += kThreads)
    sh->bias[i] = (p.bias && i < p.ncols[0]) ? p.bias[i] : 0.f;
  if (warp == kMmaWarp) tmem_alloc(&sh->tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  const int total_work = p.m_tiles * p.n_tiles;
  const int ksteps = p.kblocks[0] + (p.num_a > 1 ? p.kblocks[1] : 0);

  if (warp == kTmaWarp) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int w = blockIdx.x; ok && w < total_work; w += gridDim.x) {
        const int mt = w / p.n_tiles, nt = w % p.n_tiles;
        for (int ks = 0; ks < ksteps; ++ks) {
          const int a = ks < p.kblocks[0] ? 0 : 1;
          const int kb = a == 0 ? ks : ks - p.kblocks[0];
          if (!mbar_wait(&sh->empty[stage], phase ^ 1u, abort_flag, p.err, 1)) {
            ok = false;
            break;
          }
          mbar_expect_tx(&sh->full[stage], a_bytes + b_bytes);
          tma_load_2d(sA + stage * a_bytes, &p.tmA[a], kb * kBlockK, mt * kBlockM, &sh->full[stage]);
          tma_load_2d(sB + stage * b_stride, &p.tmB, ks * kBlockK, nt * p.N_tile, &sh->full[stage]);
          if (++stage == kStagesRows) {
            stage = 0;
            phase ^= 1u;
          }
        }
      }
      if (!ok) {
        // let loads that are still in flight land before the CTA retires
        for (int s = 0; s < kStagesRows; ++s)
          for (uint32_t it = 0; it < 4096u; ++it)
            if (mbar_try_wait(&sh->full[s], 0) || mbar_try_wait(&sh->full[s], 1)) break;
      }
    }
  } else if (warp == kMmaWarp) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kBlockM, p.N_tile, 0, 0);
      int stage = 0;
      uint32_t phase = 0;
      int local = 0;
      bool ok = true;
      for (int w = blockIdx.x; ok && w < total_work; w += gridDim.x, ++local) {
        const int acc = local & 1;
        const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
        if (!mbar_wait(&sh->tempty[acc], acc_phase ^ 1u, abort_flag, p.err, 2)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * 256u;
        for (int ks = 0; ks < ksteps; ++ks) {
          if (!mbar_wait(&sh->full[stage], phase, abort_flag, p.err, 3)) {
            ok = false;
            break;
          }
          tc_fence_after();
          const uint32_t a_addr = smem_u32(sA + stage * a_bytes);
          const uint32_t b_addr = smem_u32(sB + stage * b_stride);
#pragma unroll
          for (int kk = 0; kk < kBlockK / kUmmaK; ++kk) {
            const uint64_t adesc = smem_desc(a_addr + kk * kUmmaK * 2, 16, 1024);
            const uint64_t bdesc = smem_desc(b_addr + kk * kUmmaK * 2, 16, 1024);
            umma_bf16(d_tmem, adesc, bdesc, idesc, (ks | kk) != 0 ? 1u : 0u);
          }
          umma_commit(&sh->empty[stage]);
          if (++stage == kStagesRows) {
            stage = 0;
            phase ^= 1u;
          }
        }
        if (ok) umma_commit(&sh->tfull[acc]);
      }
    }
  } else {
    // epilogue warps: warp w reads TMEM lanes [32 (w % 4), + 32) = tile rows and takes every second
    // 64-column slab, starting with slab w / 4
    int local = 0;
    for (int w = blockIdx.x; w < total_work; w += gridDim.x, ++local) {
      const int mt = w / p.n_tiles, nt = w % p.n_tiles;
      const int acc = local & 1;
      const uint32_t acc_phase = (uint32_t)(local >> 1) & 1u;
      if (!mbar_wait(&sh->tfull[acc], acc_phase, abort_flag, p.err, 4)) break;
      tc_fence_after();
      const int quarter = warp & 3;
      const int row0 = mt * kBlockM + quarter * 32;          // first tile row of this warp
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * 256u;
      const int ncols = p.ncols[nt];
      // A thread holds one ROW of the accumulator, so storing from registers would touch 32 different lines
      // per instruction.  Instead every 64-column slab goes to a 128-byte-swizzled shared-memory tile
      // (32 rows x 128 B per warp) and leaves through one TMA store, which also clips the ragged edges.
      uint4 *stg = reinterpret_cast<uint4 *>(stage_base + (size_t)warp * 4096);   // one staging tile per warp
      for (int c64 = (warp >> 2) * 64; c64 < p.N_tile && c64 < ncols; c64 += 128) {
        uint32_t r[4][16];
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (c64 + q * 16 < p.N_tile) tmem_ld16(taddr + (uint32_t)(c64 + q * 16), r[q]);
        tmem_ld_wait();
        const bool plain = !p.bias && !p.relu && c64 + 64 <= ncols && c64 + 64 <= p.N_tile;
        // the previous store of this warp must have finished reading the tile
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const int c0 = c64 + q * 16;
          float f[16];
          if (plain) {   // no bias, no activation, slab fully inside the valid columns: convert only
#pragma unroll
            for (int j = 0; j < 16; ++j) f[j] = __uint_as_float(r[q][j]);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              float v = c0 < p.N_tile ? __uint_as_float(r[q][j]) : 0.f;
              if (p.bias) v += sh->bias[(c0 + j) & 255];
              if (p.relu) v = fmaxf(v, 0.f);
              f[j] = (c0 + j < ncols) ? v : 0.f;
            }
          }
          // 16-byte chunk j of row `lane` sits at chunk position j ^ (lane & 7)
          stg[lane * 8 + ((q * 2) ^ (lane & 7))] = make_uint4(pack_bf16x2(f[0], f[1]), pack_bf16x2(f[2], f[3]),
                                                              pack_bf16x2(f[4], f[5]), pack_bf16x2(f[6], f[7]));
          stg[lane * 8 + ((q * 2 + 1) ^ (lane & 7))] = make_uint4(pack_bf16x2(f[8], f[9]), pack_bf16x2(f[10], f[11]),
                                                                  pack_bf16x2(f[12], f[13]), pack_bf16x2(f[14], f[15]));
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        if (lane == 0) {
          asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%1, %2}], [%3];" ::"l"(
                           reinterpret_cast<uint64_t>(&p.tmOut[nt])),
                       "r"(p.col0[nt] + c64), "r"(row0), "r"(smem_u32(stg))
                       : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&sh->tempty[acc]);
    }
  }
  if (warp < kEpiWarps && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == kMmaWarp) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------------------------------ kernel 2
struct DwParams {
  CUtensorMap tmA[2];   // activation operands (X, Agg), box {64 features, 64 nodes}
  CUtensorMap tmB;      // dZ, box {64 outputs, 64 nodes}
  int tile_op[8];       // operand of every 128-feature tile
  int tile_f0[8];       // first feature of the tile
  int num_tiles;
  int n_chunks;         // 64-wide chunks of dZ columns that are loaded
  int N_pad;            // UMMA N (multiple of 16)
  int node_blocks;      // ceil(M / 64)
  int splits;           // gridDim.x
  float *partial;       // [group][split][2][128][N_pad]
  int *err;
};

struct DwSmem {
  uint64_t full[kStagesDw], empty[kStagesDw], done;
  uint32_t tmem_base;
  int abort_flag;
};

__global__ void __launch_bounds__(kThreadsDw, 1) dw_kernel(const __grid_constant__ DwParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t *base = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr uint32_t box_bytes = 64 * 64 * 2;             // 8 KB: 64 nodes x 128 B
  constexpr uint32_t stage_bytes = (4 + 4) * box_bytes;   // 2 tiles x 2 chunks of A, up to 4 chunks of B
  DwSmem *sh = reinterpret_cast<DwSmem *>(base + kStagesDw * stage_bytes);
  const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
  volatile int *abort_flag = &sh->abort_flag;
  const int group = blockIdx.y;
  const int tile0 = group * 2;
  const int ntile = min(2, p.num_tiles - tile0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStagesDw; ++s) {
      mbar_init(&sh->full[s], 1);
      mbar_init(&sh->empty[s], 1);
    }
    mbar_init(&sh->done, 1);
    sh->abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) tmem_alloc(&sh->tmem_base, kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;
  // contiguous range of 64-node blocks of this split
  const int per = (p.node_blocks + p.splits - 1) / p.splits;
  const int nb0 = blockIdx.x * per;
  const int nb1 = min(p.node_blocks, nb0 + per);
  const int steps = max(0, nb1 - nb0);
  const uint32_t tx_bytes = (uint32_t)(ntile * 2 + p.n_chunks) * box_bytes;

  if (warp == 4) {
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int s = 0; s < steps; ++s) {
        if (!mbar_wait(&sh->empty[stage], phase ^ 1u, abort_flag, p.err, 11)) {
          ok = false;
          break;
        }
        uint8_t *st = base + stage * stage_bytes;
        const int node = (nb0 + s) * 64;
        mbar_expect_tx(&sh->full[stage], tx_bytes);
        for (int t = 0; t < ntile; ++t)
          for (int c = 0; c < 2; ++c)
            tma_load_2d(st + (t * 2 + c) * box_bytes, &p.tmA[p.tile_op[tile0 + t]], p.tile_f0[tile0 + t] + c * 64, node,
                        &sh->full[stage]);
        for (int c = 0; c < p.n_chunks; ++c)
          tma_load_2d(st + (4 + c) * box_bytes, &p.tmB, c * 64, node, &sh->full[stage]);
        if (++stage == kStagesDw) {
          stage = 0;
          phase ^= 1u;
        }
      }
      if (!ok)
        for (int s = 0; s < kStagesDw; ++s)
          for (uint32_t it = 0; it < 4096u; ++it)
            if (mbar_try_wait(&sh->full[s], 0) || mbar_try_wait(&sh->full[s], 1)) break;
    }
  } else if (warp == 5) {
    if (lane == 0) {
      const uint32_t idesc = instr_desc(kBlockM, p.N_pad, 1, 1);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int s = 0; s < steps; ++s) {
        if (!mbar_wait(&sh->full[stage], phase, abort_flag, p.err, 12)) {
          ok = false;
          break;
        }
        tc_fence_after();
        const uint32_t st = smem_u32(base + stage * stage_bytes);
#pragma unroll
        for (int kk = 0; kk < 64 / kUmmaK; ++kk) {
          // 16 nodes further = 16 rows of 128 B
          const uint64_t bdesc = smem_desc(st + 4 * box_bytes + kk * kUmmaK * 128, box_bytes, 1024);
          for (int t = 0; t < ntile; ++t) {
            const uint64_t adesc = smem_desc(st + (t * 2) * box_bytes + kk * kUmmaK * 128, box_bytes, 1024);
            umma_bf16(tmem_base + (uint32_t)t * 256u, adesc, bdesc, idesc, (s | kk) != 0 ? 1u : 0u);
          }
        }
        umma_commit(&sh->empty[stage]);
        if (++stage == kStagesDw) {
          stage = 0;
          phase ^= 1u;
        }
      }
      if (ok) umma_commit(&sh->done);
    }
  } else {
    // epilogue: tile row = feature, 16 columns at a time, fp32 partials
    bool have = steps > 0;
    if (have) have = mbar_wait(&sh->done, 0, abort_flag, p.err, 13);
    tc_fence_after();
    const int frow = warp * 32 + lane;
    for (int t = 0; t < ntile; ++t) {
      float *dst = p.partial + ((((int64_t)group * p.splits + blockIdx.x) * 2 + t) * 128 + frow) * p.N_pad;
      const uint32_t taddr = tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)t * 256u;
      for (int c0 = 0; c0 < p.N_pad; c0 += 16) {
        uint32_t r[16];
        if (have) {
          tmem_ld16(taddr + (uint32_t)c0, r);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) r[j] = 0u;
        }
#pragma unroll
        for (int j = 0; j < 16; j += 4)
          *reinterpret_cast<uint4 *>(dst + c0 + j) = make_uint4(r[j], r[j + 1], r[j + 2], r[j + 3]);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 5) tmem_dealloc(tmem_base, kTmemCols);
}

// dW[f][o] = sum over splits (ascending) of the partial tiles; one thread per output element
__global__ void dw_reduce_kernel(const float *__restrict__ partial, int splits, int N_pad, int F_in, int F_out,
                                 int tiles_per_op, float *__restrict__ dW0, float *__restrict__ dW1, int num_ops) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t per_op = (int64_t)F_in * F_out;
  if (idx >= per_op * num_ops) return;
  const int op = (int)(idx / per_op);
  const int f = (int)((idx % per_op) / F_out), o = (int)(idx % F_out);
  const int tile = op * tiles_per_op + f / 128;
  const int group = tile / 2, t = tile % 2;
  float s = 0.f;
  for (int z = 0; z < splits; ++z)
    s += partial[((((int64_t)group * splits + z) * 2 + t) * 128 + (f % 128)) * N_pad + o];
  (op == 0 ? dW0 : dW1)[(int64_t)f * F_out + o] = s;
}

// Weight repack for kernel 1.
//  mode 0 (forward):  B[o][koff_a + c] = W_a[c][o]      rows = outputs, K = [X block | Agg block], zero padded
//  mode 1 (backward): B[t * N_tile + j][c] = W_t[j][c]  rows = input features of operand t, K = outputs
//  mode 2 (backward, concatenated K): B[j][a * koff1 + c] = W_a[j][c]  rows = input features, K = [op 0 | op 1]
__global__ void pack_weights_kernel(const __nv_bfloat16 *__restrict__ W0, const __nv_bfloat16 *__restrict__ W1,
                                    int F_in, int F_out, int mode, int rows, int kcols, int koff1, int N_tile,
                                    int tiles_per_op, __nv_bfloat16 *__restrict__ B) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (int64_t)rows * kcols) return;
  const int r = (int)(idx / kcols), c = (int)(idx % kcols);
  __nv_bfloat16 v = __float2bfloat16_rn(0.f);
  if (mode == 0) {
    const int a = (W1 && c >= koff1) ? 1 : 0;
    const int cc = a ? c - koff1 : c;
    const __nv_bfloat16 *W = a ? W1 : W0;
    if (r < F_out && cc < F_in) v = W[(int64_t)cc * F_out + r];
  } else if (mode == 2) {
    const int a = (W1 && c >= koff1) ? 1 : 0;
    const int cc = a ? c - koff1 : c;
    const __nv_bfloat16 *W = a ? W1 : W0;
    if (r < F_in && cc < F_out) v = W[(int64_t)r * F_out + cc];
  } else {
    const int tile = r / N_tile, j = r % N_tile;
    const int op = tile / tiles_per_op;
    const int f = (tile % tiles_per_op) * N_tile + j;
    const __nv_bfloat16 *W = op ? W1 : W0;
    if (W && f < F_in && c < F_out) v = W[(int64_t)f * F_out + c];
  }
  B[idx] = v;
}

// ------------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void *ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// 2-D bf16 tensor map over a row-major matrix: `cols` valid columns (reads beyond are zero filled),
// `rows` rows, leading dimension ld elements, box {64, box_rows}, 128-byte swizzle.
int make_map(CUtensorMap *m, const void *ptr, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return VARCO_CUDA;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(ptr), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? VARCO_OK : VARCO_CUDA;
}

int sm_count() {
  static int sms = 0;
  if (!sms) {
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (sms <= 0) sms = 148;   // no device visible (a build host): the part this library targets
  }
  return sms;
}

constexpr size_t rows_smem_bytes() {
  return 1024 + kStagesRows * (size_t)(kBlockM * kBlockK * 2 + 256 * kBlockK * 2) + 8 * 4096 + sizeof(RowsSmem) + 64;
}
constexpr size_t dw_smem_bytes() { return 1024 + kStagesDw * (size_t)(8 * 64 * 64 * 2) + sizeof(DwSmem) + 64; }

int ceil_div(int a, int b) { return (a + b - 1) / b; }

}  // namespace

// Scratch of the tensor-core path: repacked weights (bf16) and dW partial tiles (fp32).
struct TcScratch {
  __nv_bfloat16 *packed;
  float *partial;
};
static size_t packed_bytes(int F_in, int F_out) {
  const size_t kpad_in = (size_t)ceil_div(F_in, 64) * 64, kpad_out = (size_t)ceil_div(F_out, 64) * 64;
  size_t fwd = (size_t)256 * 2 * kpad_in * 2;                       // <= 256 rows x two K blocks
  const size_t bwd = (size_t)(2 * (F_in + 256)) * kpad_out * 2;     // two operands, tile padding
  if (bwd > fwd) fwd = bwd;
  return (fwd + 255) / 256 * 256;
}
size_t varco_tc_scratch_bytes(int F_in, int F_out) {
  const size_t partial = (size_t)sm_count() * 2 * 128 * 256 * 4;    // groups x splits <= one CTA per SM, 2 tiles each
  return packed_bytes(F_in, F_out) + partial + 256;
}
static TcScratch carve(void *scratch, int F_in, int F_out) {
  char *b = static_cast<char *>(scratch);
  TcScratch s;
  s.packed = reinterpret_cast<__nv_bfloat16 *>(b);
  s.partial = reinterpret_cast<float *>(b + packed_bytes(F_in, F_out));
  return s;
}

static int configure_once() {
  static int rc = -1;
  if (rc < 0) {
    cudaError_t e1 = cudaFuncSetAttribute(rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          (int)rows_smem_bytes());
    cudaError_t e2 = cudaFuncSetAttribute(dw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dw_smem_bytes());
    rc = (e1 == cudaSuccess && e2 == cudaSuccess) ? VARCO_OK : VARCO_CUDA;
  }
  return rc;
}

// tensor maps of the epilogue's stores: tile t writes columns [col0, col0 + ncols) of its destination
static int make_out_maps(RowsParams &p) {
  for (int t = 0; t < p.n_tiles; ++t)
    if (make_map(&p.tmOut[t], p.out[t], p.M, p.col0[t] + p.ncols[t], p.ldo[t], 32)) return VARCO_CUDA;
  return VARCO_OK;
}

// Y[n x F_out] = act([X | Agg] [Ws ; Wn] + bias); Ws == nullptr: Y = act(Agg Wn + bias)
int varco_tc_gemm_fwd(int n, int F_in, int F_out, const void *X, int64_t ldx, const void *Agg, int64_t lda,
                      const void *Ws, const void *Wn, const float *bias, int relu, void *Y, int64_t ldy,
                      void *scratch, int *err, cudaStream_t st) {
  if (F_out > 256) return VARCO_UNSUPPORTED;
  if (configure_once() != VARCO_OK) return VARCO_CUDA;
  TcScratch sc = carve(scratch, F_in, F_out);
  RowsParams p;
  memset(&p, 0, sizeof(p));
  const int kb = ceil_div(F_in, 64);
  const int N_tile = ceil_div(F_out, 16) * 16;
  p.num_a = Ws ? 2 : 1;
  p.kblocks[0] = kb;
  p.kblocks[1] = Ws ? kb : 0;
  const int kcols = (p.kblocks[0] + p.kblocks[1]) * 64;
  // operand 0 = X (if SAGE) else Agg; operand 1 = Agg
  const void *op0 = Ws ? X : Agg;
  const int64_t ld0 = Ws ? ldx : lda;
  if (make_map(&p.tmA[0], op0, n, F_in, ld0, 128)) return VARCO_CUDA;
  if (Ws && make_map(&p.tmA[1], Agg, n, F_in, lda, 128)) return VARCO_CUDA;
  if (make_map(&p.tmB, sc.packed, N_tile, kcols, kcols, N_tile)) return VARCO_CUDA;
  {
    const int64_t total = (int64_t)N_tile * kcols;
    pack_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
        (const __nv_bfloat16 *)(Ws ? Ws : Wn), (const __nv_bfloat16 *)(Ws ? Wn : nullptr), F_in, F_out, 0, N_tile,
        kcols, kb * 64, N_tile, 1, sc.packed);
    VARCO_KERNEL_LAUNCHED();
  }
  p.M = n;
  p.m_tiles = ceil_div(n, kBlockM);
  p.n_tiles = 1;
  p.N_tile = N_tile;
  p.out[0] = (__nv_bfloat16 *)Y;
  p.ldo[0] = ldy;
  p.ncols[0] = F_out;
  p.col0[0] = 0;
  p.bias = bias;
  p.relu = relu;
  p.err = err;
  const int grid = p.m_tiles < sm_count() ? p.m_tiles : sm_count();
  if (make_out_maps(p)) return VARCO_CUDA;
  rows_kernel<<<grid, kThreads, rows_smem_bytes(), st>>>(p);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// dXs[n x F_in] = dZ Ws^T (if Ws) and dAgg[n x F_in] = dZ Wn^T
int varco_tc_gemm_dx(int n, int F_in, int F_out, const void *dZ, int64_t lddz, const void *Ws, const void *Wn,
                     void *dXs, int64_t ldxs, void *dAgg, int64_t ldagg, void *scratch, int *err, cudaStream_t st) {
  if (configure_once() != VARCO_OK) return VARCO_CUDA;
  TcScratch sc = carve(scratch, F_in, F_out);
  RowsParams p;
  memset(&p, 0, sizeof(p));
  const int num_ops = Ws ? 2 : 1;
  // split every operand's F_in output columns into equal tiles of at most 256 (multiple of 16)
  const int tiles_per_op = ceil_div(F_in, 256);
  const int N_tile = ceil_div(ceil_div(F_in, tiles_per_op), 16) * 16;
  if (num_ops * tiles_per_op > 4) return VARCO_UNSUPPORTED;
  const int kb = ceil_div(F_out, 64);
  const int kcols = kb * 64;
  const int rows = num_ops * tiles_per_op * N_tile;
  p.num_a = 1;
  p.kblocks[0] = kb;
  if (make_map(&p.tmA[0], dZ, n, F_out, lddz, 128)) return VARCO_CUDA;
  if (make_map(&p.tmB, sc.packed, rows, kcols, kcols, N_tile)) return VARCO_CUDA;
  {
    const int64_t total = (int64_t)rows * kcols;
    pack_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
        (const __nv_bfloat16 *)(Ws ? Ws : Wn), (const __nv_bfloat16 *)(Ws ? Wn : nullptr), F_in, F_out, 1, rows, kcols,
        0, N_tile, tiles_per_op, sc.packed);
    VARCO_KERNEL_LAUNCHED();
  }
  p.M = n;
  p.m_tiles = ceil_div(n, kBlockM);
  p.n_tiles = num_ops * tiles_per_op;
  p.N_tile = N_tile;
  for (int t = 0; t < p.n_tiles; ++t) {
    const int op = t / tiles_per_op, sub = t % tiles_per_op;
    const bool self = Ws && op == 0;
    p.out[t] = (__nv_bfloat16 *)(self ? dXs : dAgg);
    p.ldo[t] = self ? ldxs : ldagg;
    p.col0[t] = sub * N_tile;
    int nc = F_in - sub * N_tile;
    p.ncols[t] = nc > N_tile ? N_tile : nc;
  }
  p.bias = nullptr;
  p.relu = 0;
  p.err = err;
  const int work = p.m_tiles * p.n_tiles;
  const int grid = work < sm_count() ? work : sm_count();
  if (make_out_maps(p)) return VARCO_CUDA;
  rows_kernel<<<grid, kThreads, rows_smem_bytes(), st>>>(p);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// out[m x F_in] = A0 W0^T (+ A1 W1^T), A_a being [m x F_out] and W_a [F_in x F_out]: the backward products
// with the K range concatenated over the two operands.
int varco_tc_gemm_cat_t(int m, int F_in, int F_out, const void *A0, int64_t lda0, const void *A1, int64_t lda1,
                        const void *W0, const void *W1, void *out, int64_t ldo, void *scratch, int *err,
                        cudaStream_t st) {
  if (configure_once() != VARCO_OK) return VARCO_CUDA;
  TcScratch sc = carve(scratch, F_in, F_out);
  RowsParams p;
  memset(&p, 0, sizeof(p));
  const int tiles = ceil_div(F_in, 256);
  const int N_tile = ceil_div(ceil_div(F_in, tiles), 16) * 16;
  if (tiles > 4) return VARCO_UNSUPPORTED;
  const int kb = ceil_div(F_out, 64);
  p.num_a = A1 ? 2 : 1;
  p.kblocks[0] = kb;
  p.kblocks[1] = A1 ? kb : 0;
  const int kcols = (p.kblocks[0] + p.kblocks[1]) * 64;
  const int rows = tiles * N_tile;
  if (make_map(&p.tmA[0], A0, m, F_out, lda0, 128)) return VARCO_CUDA;
  if (A1 && make_map(&p.tmA[1], A1, m, F_out, lda1, 128)) return VARCO_CUDA;
  if (make_map(&p.tmB, sc.packed, rows, kcols, kcols, N_tile)) return VARCO_CUDA;
  {
    const int64_t total = (int64_t)rows * kcols;
    pack_weights_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(
        (const __nv_bfloat16 *)W0, (const __nv_bfloat16 *)(A1 ? W1 : nullptr), F_in, F_out, 2, rows, kcols, kb * 64,
        N_tile, 1, sc.packed);
    VARCO_KERNEL_LAUNCHED();
  }
  p.M = m;
  p.m_tiles = ceil_div(m, kBlockM);
  p.n_tiles = tiles;
  p.N_tile = N_tile;
  for (int t = 0; t < tiles; ++t) {
    p.out[t] = (__nv_bfloat16 *)out;
    p.ldo[t] = ldo;
    p.col0[t] = t * N_tile;
    const int nc = F_in - t * N_tile;
    p.ncols[t] = nc > N_tile ? N_tile : nc;
  }
  p.err = err;
  const int64_t work = (int64_t)p.m_tiles * p.n_tiles;
  const int grid = work < sm_count() ? (int)work : sm_count();
  if (make_out_maps(p)) return VARCO_CUDA;
  rows_kernel<<<grid, kThreads, rows_smem_bytes(), st>>>(p);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

// dWs = X^T dZ (if dWs) and dWn = Agg^T dZ, fp32 [F_in x F_out]
int varco_tc_gemm_dw(int n, int F_in, int F_out, const void *X, int64_t ldx, const void *Agg, int64_t lda,
                     const void *dZ, int64_t lddz, float *dWs, float *dWn, void *scratch, int *err, cudaStream_t st) {
  if (F_out > 256) return VARCO_UNSUPPORTED;
  if (configure_once() != VARCO_OK) return VARCO_CUDA;
  TcScratch sc = carve(scratch, F_in, F_out);
  DwParams p;
  memset(&p, 0, sizeof(p));
  const int num_ops = dWs ? 2 : 1;
  const int tiles_per_op = ceil_div(F_in, 128);
  p.num_tiles = num_ops * tiles_per_op;
  if (p.num_tiles > 8) return VARCO_UNSUPPORTED;
  const void *op0 = dWs ? X : Agg;
  const int64_t ld0 = dWs ? ldx : lda;
  if (make_map(&p.tmA[0], op0, n, F_in, ld0, 64)) return VARCO_CUDA;
  if (dWs && make_map(&p.tmA[1], Agg, n, F_in, lda, 64)) return VARCO_CUDA;
  if (make_map(&p.tmB, dZ, n, F_out, lddz, 64)) return VARCO_CUDA;
  for (int t = 0; t < p.num_tiles; ++t) {
    p.tile_op[t] = t / tiles_per_op;
    p.tile_f0[t] = (t % tiles_per_op) * 128;
  }
  p.N_pad = ceil_div(F_out, 16) * 16;
  p.n_chunks = ceil_div(p.N_pad, 64);
  p.node_blocks = ceil_div(n, 64);
  const int groups = ceil_div(p.num_tiles, 2);
  int splits = sm_count() / groups;
  if (splits < 1) splits = 1;
  if (splits > p.node_blocks) splits = p.node_blocks;
  if (splits * groups > sm_count()) splits = sm_count() / groups > 0 ? sm_count() / groups : 1;
  p.splits = splits;
  p.partial = sc.partial;
  p.err = err;
  dim3 grid(splits, groups);
  dw_kernel<<<grid, kThreadsDw, dw_smem_bytes(), st>>>(p);
  VARCO_KERNEL_LAUNCHED();
  const int64_t total = (int64_t)num_ops * F_in * F_out;
  dw_reduce_kernel<<<(unsigned)((total + 255) / 256), 256, 0, st>>>(sc.partial, splits, p.N_pad, F_in, F_out,
                                                                   tiles_per_op, dWs ? dWs : dWn, dWn, num_ops);
  VARCO_KERNEL_LAUNCHED();
  return VARCO_OK;
}

