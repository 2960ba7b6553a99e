// Tensor-core kernels (sm_100a: tcgen05.mma, TMEM accumulator, TMA operand staging) for the steps of the
// path that are plain dense contractions: products of a bf16 tensor with a wide fp32 factor (16..64
// columns) in Algorithm 1 on token layers (B x N x D activations),
//   k_tc_lastmode      Y[q][j]     = sum_k X[q][k] U[k][j]          V_3 = A_(3)^T U_3, first core product
//   k_tc_expand        P[k][j]     = sum_q X[q][k] V[q][j]          P_3 = A_(3) V_3 (split-K partials)
//   k_tc_token         V[o][i][j]  = sum_k X[o][k][i] U[k][j]       V_2 = A_(2)^T U_2, one sample o per CTA row
//   k_tc_token_expand  P[k][j]     = sum_{o,i} X[o][k][i] V[o][i][j]  P_2 = A_(2) V_2 (split-K partials)
// X is exact in bf16; the fp32 factor (U or V) is split into three bf16 terms (24 mantissa bits), so one
// MMA of width 3 n per k-step (the three terms stacked as operand rows) yields three partial products in
// TMEM whose sum reproduces the fp32 product to fp32 rounding.
//
// k_tc_split writes the stacked operand [3 n][K] (bf16, K contiguous: hi rows, then mid, then lo) to
// scratch memory once per product; the GEMM kernel then streams both operands by TMA.  One CTA owns a
// 128-row tile of Y and walks K in chunks of 64, its warps in three roles that meet only through mbarriers:
//   * a producer thread keeps four stages in flight, each the X tile [128 x 64] and the operand tile
//     [3 n x 64] (cp.async.bulk.tensor, 128-byte swizzle);
//   * an issuer thread launches 4 k-steps of tcgen05.mma (M = 128, N = 3 n, K = 16) per chunk and commits
//     them to the mbarrier that frees the stage;
//   * eight warps then read the three accumulator groups with tcgen05.ld (lane = row), add them and store
//     fp32 rows.
// Every wait has a time limit; on expiry the kernel records ASI_ERR_TIMEOUT in the workspace's status word,
// frees its TMEM and returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "asi_internal.h"

namespace asi {

namespace {

constexpr int kTcWorkers = 8;       // epilogue warps
constexpr int kTcThreads = (kTcWorkers + 2) * 32;   // + the MMA issuer warp and the TMA producer warp
constexpr int kTcM = 128;          // rows of Y per CTA (= TMEM lanes)
constexpr int kTcKC = 64;          // k per chunk: 64 bf16 = one 128-byte swizzle row
constexpr int kTcStages = 4;       // X stages in flight
constexpr int kTcNMax = 64;
constexpr uint32_t kTileA = kTcM * kTcKC * 2;       // 16 KB
constexpr uint32_t kTileB = 3 * kTcNMax * kTcKC * 2;   // 24 KB: the three terms stacked

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
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
__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// waits for the phase with the given parity; gives up after ~1 s
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;       // the common case costs no timer read
  const uint64_t t0 = globaltimer_ns();
  for (uint32_t it = 0; it < (1u << 28); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 1023u) == 1023u && globaltimer_ns() - t0 > 1000000000ull) return false;
  }
  return false;
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
          smem_u32(dst)),
      "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
      : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(
          smem_u32(dst)),
      "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
      : "memory");
}
// shared-memory matrix descriptor of a 128-byte-swizzled operand (start address, leading and stride byte
// offsets in 16-byte units; descriptor version 1).  K-major: rows of 128 bytes along K, groups of 8 rows
// 1024 bytes apart (stride offset), the leading offset is unused.  MN-major: rows of 128 bytes along M/N
// (64 bf16), one row per K index, groups of 8 K-rows 1024 bytes apart (stride offset), the next 64 M/N
// elements `lbo` bytes further (leading offset).
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr, uint32_t lbo_bytes = 16) {
  uint64_t d = 0;
  d |= (uint64_t)((addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
  d |= (uint64_t)1 << 46;                 // version
  d |= (uint64_t)2 << 61;                 // 128-byte swizzle
  return d;
}
// instruction descriptor of kind::f16: fp32 accumulator, bf16 x bf16, B K-major, A K-major or MN-major
__device__ __forceinline__ uint32_t instr_desc_bf16(int M, int N, bool a_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn_major ? (1u << 15) : 0u) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(acc), "r"(0u)    // no output lane disabled
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, uint32_t (&v)[8]) {   // 8 columns of this thread's lane
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
               : "r"(taddr)
               : "memory");
}
struct TcArgs {
  float* Y;            // [M][ldy]; CTA (., s) writes Y + s * y_split
  int M, N, K, ldy;    // K: total extent of the contraction
  int k_per_split;     // multiple of 64; CTA (., s) contracts [s * k_per_split, min(K, (s + 1) * k_per_split))
  int64_t y_split;
  int inner;           // kTcTokenExpand: K enumerates (o, i) with i < inner (a multiple of 64)
  int* status;         // status word of the caller's workspace (may be null): ASI_ERR_TIMEOUT when a wait expires
  int nv;              // columns of Y that exist (a multiple of 4, N - 15 <= nv <= N): the factor is zero-padded to N
};

// Bt[(t*n + j) * ldb + k] = t-th bf16 term of U[k][j] (hi, mid, lo: U = hi + mid + lo to 24 bits)
__global__ void __launch_bounds__(256) k_tc_split(const float* __restrict__ U, int ldu, int K, int N, int nv,
                                                  __nv_bfloat16* __restrict__ Bt, int64_t ldb) {
  __shared__ float tile[32][33];
  const int k0 = blockIdx.x * 32, j0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  for (int r = ty; r < 32; r += 8) {
    const int k = k0 + r, j = j0 + tx;
    tile[r][tx] = (k < K && j < nv) ? U[(int64_t)k * ldu + j] : 0.f;     // columns nv..N-1 of the operand are zero
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    const int j = j0 + r, k = k0 + tx;
    if (j < N && k < K) {
      const float u = tile[tx][r];
      const __nv_bfloat16 h = __float2bfloat16_rn(u);
      const float r1 = u - __bfloat162float(h);
      const __nv_bfloat16 m = __float2bfloat16_rn(r1);
      const __nv_bfloat16 l = __float2bfloat16_rn(r1 - __bfloat162float(m));
      Bt[(int64_t)j * ldb + k] = h;
      Bt[(int64_t)(N + j) * ldb + k] = m;
      Bt[(int64_t)(2 * N + j) * ldb + k] = l;
    }
  }
}

// How the X operand of D[m][n] = sum_k A(m, k) B[n][k] is laid out in memory:
//   kTcLast        X[m][k], k contiguous: one box [128 m x 64 k] (K-major);            CTA (mt, split of K)
//   kTcLastExpand  X[k][m], m contiguous: two boxes [64 k x 64 m] (MN-major);          CTA (mt, split of K)
//   kTcToken       X[o][k][m], m contiguous, one o per CTA row: two boxes (MN-major);  CTA (mt, o)
//   kTcTokenExpand X[o][m][i], i contiguous, K = (o, i) flattened: one box (K-major);  CTA (mt, split of K)
// Rows of a box that fall outside the tensor are zero-filled by TMA.
enum TcMode { kTcLast = 0, kTcLastExpand = 1, kTcToken = 2, kTcTokenExpand = 3 };

template <int MODE>
__device__ __forceinline__ void tc_gemm_body(const CUtensorMap& mapX, const CUtensorMap& mapB, const TcArgs& p) {
  extern __shared__ __align__(1024) uint8_t tc_smem[];
  // carve-up: per stage the X tile and the operand tile, then barriers
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(tc_smem) + 1023) & ~(uintptr_t)1023);
  uint8_t* As = base;                                   // [stages][16 KB]
  uint8_t* Bs = As + kTcStages * kTileA;                // [stages][24 KB]
  uint64_t* full = reinterpret_cast<uint64_t*>(Bs + kTcStages * kTileB);   // [stages] both tiles landed
  uint64_t* s_free = full + kTcStages;                  // [stages] the MMAs that read the stage are done
  uint64_t* done = s_free + kTcStages;                  // all MMAs of the tile are done
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(done + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr bool A_MN = (MODE == kTcLastExpand || MODE == kTcToken);
  const int row0 = blockIdx.x * kTcM;
  const int k_begin = (MODE == kTcToken) ? 0 : blockIdx.y * p.k_per_split;
  const int k_end = (MODE == kTcToken || p.K - k_begin < p.k_per_split) ? p.K : k_begin + p.k_per_split;
  const int nchunk = (k_end - k_begin + kTcKC - 1) / kTcKC;   // a ragged last chunk is zero-filled by TMA
  const int N = p.N;
  float* Yout = p.Y + (int64_t)blockIdx.y * p.y_split;

  if (tid == 0) {
    for (int s = 0; s < kTcStages; ++s) { mbar_init(full + s, 1); mbar_init(s_free + s, 1); }
    mbar_init(done, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {                                      // TMEM: 256 fp32 columns x 128 lanes (3 N are used)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(256)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_d = *tmem_slot;

  // The three bf16 terms of the factor are stacked along the operand's rows: one MMA of width 3 N per
  // k-step reads the X tile once and leaves the three partial products in three column groups of TMEM.
  const uint32_t idesc = instr_desc_bf16(kTcM, 3 * N, A_MN);
  const uint32_t b_bytes = (uint32_t)(3 * N) * 128u;    // operand tile: 3 N rows of 64 bf16
  bool ok = true;                                       // this thread's waits so far
  if (warp == kTcWorkers) {
    // ---- MMA issuer (one thread): 4 k-steps per chunk, then the commit that frees the stage
    if (lane == 0) {
      const uint32_t a_base = smem_u32(As), b_base = smem_u32(Bs);
#pragma unroll 1
      for (int c = 0; c < nchunk && ok; ++c) {
        const int s = c % kTcStages;
        ok = mbar_wait(full + s, (c / kTcStages) & 1);
        if (!ok) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // a k-step is 16 bf16: 32 bytes inside the swizzle row of a K-major tile, 16 rows (2048 bytes) of
        // an MN-major tile (start-address field in 16-byte units)
        const uint64_t da0 = smem_desc_sw128(a_base + s * kTileA, A_MN ? kTileA / 2 : 16);
        const uint64_t db0 = smem_desc_sw128(b_base + s * kTileB);
#pragma unroll
        for (int ks = 0; ks < kTcKC / 16; ++ks)
          umma_bf16(tmem_d, da0 + (uint64_t)(ks * (A_MN ? 128 : 2)), db0 + (uint64_t)(ks * 2), idesc,
                    (c | ks) ? 1u : 0u);
        umma_commit(s_free + s);
      }
      umma_commit(done);
    }
  } else if (warp == kTcWorkers + 1) {
    // ---- TMA producer (one thread): keeps kTcStages stages in flight
    if (lane == 0) {
#pragma unroll 1
      for (int c = 0; c < nchunk && ok; ++c) {
        const int s = c % kTcStages;
        if (c >= kTcStages) ok = mbar_wait(s_free + s, ((c / kTcStages) - 1) & 1);
        if (!ok) break;
        mbar_expect_tx(full + s, kTileA + b_bytes);
        const int kc = k_begin + c * kTcKC;
        if (MODE == kTcLastExpand) {
          tma_load_2d(As + s * kTileA, &mapX, row0, kc, full + s);
          tma_load_2d(As + s * kTileA + kTileA / 2, &mapX, row0 + 64, kc, full + s);
        } else if (MODE == kTcToken) {
          tma_load_3d(As + s * kTileA, &mapX, row0, kc, blockIdx.y, full + s);
          tma_load_3d(As + s * kTileA + kTileA / 2, &mapX, row0 + 64, kc, blockIdx.y, full + s);
        } else if (MODE == kTcTokenExpand) {
          const int o = kc / p.inner;
          tma_load_3d(As + s * kTileA, &mapX, kc - o * p.inner, row0, o, full + s);
        } else {
          tma_load_2d(As + s * kTileA, &mapX, kc, row0, full + s);
        }
        tma_load_2d(Bs + s * kTileB, &mapB, kc, 0, full + s);
      }
    }
  } else {
    ok = mbar_wait(done, 0);                            // every reader of TMEM observes the completed phase
  }
  const bool fail = __syncthreads_or(ok ? 0 : 1) != 0;
  if (!fail) {
    if (warp < kTcWorkers) {
      // thread = row: warp w reads lanes 32 (w % 4) ..., warps 0-3 the columns [0, N/2), warps 4-7 the rest
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int half = N >> 1;                          // 8, 16, 24 or 32 columns per warp
      const int col0 = (warp >> 2) * half;
      const int row = row0 + (warp & 3) * 32 + lane;
      const uint32_t taddr = tmem_d + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)col0;
      for (int cc = 0; cc < half; cc += 8) {
        uint32_t h[8], m[8], l[8];
        tmem_ld8(taddr + (uint32_t)cc, h);
        tmem_ld8(taddr + (uint32_t)(N + cc), m);
        tmem_ld8(taddr + (uint32_t)(2 * N + cc), l);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (row < p.M) {
          float o[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)                   // small terms first
            o[i] = (__uint_as_float(l[i]) + __uint_as_float(m[i])) + __uint_as_float(h[i]);
          float* y = Yout + (int64_t)row * p.ldy + col0 + cc;
          if (col0 + cc < p.nv) *reinterpret_cast<float4*>(y) = make_float4(o[0], o[1], o[2], o[3]);
          if (col0 + cc + 4 < p.nv) *reinterpret_cast<float4*>(y + 4) = make_float4(o[4], o[5], o[6], o[7]);
        }
      }
    }
  } else if (tid == 0 && p.status) {
    atomicMax(p.status, (int)ASI_ERR_TIMEOUT);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(256) : "memory");
}

__global__ void __launch_bounds__(kTcThreads, 1) k_tc_lastmode(const __grid_constant__ CUtensorMap mapX,
                                                                const __grid_constant__ CUtensorMap mapB, TcArgs p) {
  tc_gemm_body<kTcLast>(mapX, mapB, p);
}
__global__ void __launch_bounds__(kTcThreads, 1) k_tc_expand(const __grid_constant__ CUtensorMap mapX,
                                                              const __grid_constant__ CUtensorMap mapB, TcArgs p) {
  tc_gemm_body<kTcLastExpand>(mapX, mapB, p);
}
__global__ void __launch_bounds__(kTcThreads, 1) k_tc_token(const __grid_constant__ CUtensorMap mapX,
                                                             const __grid_constant__ CUtensorMap mapB, TcArgs p) {
  tc_gemm_body<kTcToken>(mapX, mapB, p);
}
__global__ void __launch_bounds__(kTcThreads, 1) k_tc_token_expand(const __grid_constant__ CUtensorMap mapX,
                                                                    const __grid_constant__ CUtensorMap mapB, TcArgs p) {
  tc_gemm_body<kTcTokenExpand>(mapX, mapB, p);
}

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
  static EncodeFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeFn>(p);
  });
  return fn;
}

}  // namespace

size_t tc_scratch_bytes(int64_t K, int N) { return (size_t)3 * ((N + 15) / 16 * 16) * ((K + 63) / 64 * 64) * 2; }

namespace {
constexpr size_t kTcSmem = 1024 + kTcStages * (kTileA + kTileB) + (2 * kTcStages + 1) * 8 + 16;

bool encode_bf16_map(CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
                     const cuuint32_t* box) {
  EncodeFn enc = encode_fn();
  if (!enc) return false;
  const cuuint32_t estr[3] = {1, 1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims, strides, box,
             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// V[o][i][j] = sum_k X[o][k][i] U[k][j]: a middle mode of a bf16 token tensor (I = inner extent, a multiple of 64)
cudaError_t launch_tc_token(const ModeProdArgs& p, void* scratch, size_t scratch_bytes, cudaStream_t st) {
  const int nv = p.n_out, N = (nv + 15) / 16 * 16;       // the factor is zero-padded to a multiple of 16 columns
  const int64_t Kp = (p.a + 63) / 64 * 64;
  if (p.I < 64 || p.I % 64 != 0 || p.O < 1 || p.O >= 65536 || nv % 4 != 0 || nv < 16 || N > kTcNMax || p.a < 1 ||
      p.a >= (1ll << 31) || p.I >= (1ll << 31) || p.sj != 1 || p.si != nv || p.so != p.I * nv || p.ldb_j != 1 ||
      !scratch || scratch_bytes < tc_scratch_bytes(p.a, N) || (reinterpret_cast<uintptr_t>(scratch) & 15u) ||
      (reinterpret_cast<uintptr_t>(p.X) & 15u) || (reinterpret_cast<uintptr_t>(p.Y) & 15u))
    return cudaErrorNotSupported;
  CUtensorMap mapX, mapB;
  {
    const cuuint64_t dims[3] = {(cuuint64_t)p.I, (cuuint64_t)p.a, (cuuint64_t)p.O};
    const cuuint64_t strides[2] = {(cuuint64_t)p.I * 2, (cuuint64_t)p.a * p.I * 2};
    const cuuint32_t box[3] = {64, 64, 1};
    if (!encode_bf16_map(&mapX, p.X, 3, dims, strides, box)) return cudaErrorNotSupported;
  }
  {
    const cuuint64_t dims[2] = {(cuuint64_t)p.a, (cuuint64_t)(3 * N)};
    const cuuint64_t strides[1] = {(cuuint64_t)Kp * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTcKC, (cuuint32_t)(3 * N)};
    if (!encode_bf16_map(&mapB, scratch, 2, dims, strides, box)) return cudaErrorNotSupported;
  }
  const cudaError_t attr_err = opt_in_smem(reinterpret_cast<const void*>(k_tc_token), kTcSmem);
  if (attr_err != cudaSuccess) return attr_err;
  k_tc_split<<<dim3((unsigned)((p.a + 31) / 32), (unsigned)((N + 31) / 32)), 256, 0, st>>>(
      p.B, (int)p.ldb_k, (int)p.a, N, nv, static_cast<__nv_bfloat16*>(scratch), Kp);
  TcArgs a = {p.Y, (int)p.I, N, (int)p.a, nv, (int)Kp, p.so, 0, p.status, nv};
  dim3 grid((unsigned)((p.I + kTcM - 1) / kTcM), (unsigned)p.O);
  k_tc_token<<<grid, kTcThreads, kTcSmem, st>>>(mapX, mapB, a);
  return cudaGetLastError();
}

// Pp[s][k][j] = sum_{(o,i) in split s} X[o][k][i] V[o][i][j]: the expansion of a middle mode
cudaError_t launch_tc_token_expand(const ExpandArgs& e, void* scratch, size_t scratch_bytes, cudaStream_t st) {
  const int nv = e.r, N = (nv + 15) / 16 * 16;
  const int64_t Q = e.Q;
  if (e.I < 64 || e.I % 64 != 0 || e.O < 1 || e.O >= 65536 || nv % 4 != 0 || nv < 16 || N > kTcNMax || e.a < 1 ||
      e.a >= (1ll << 31) || Q >= (1ll << 31) || e.q_per_split % kTcKC != 0 || e.q_per_split >= (1ll << 31) ||
      e.nsplit < 1 || !scratch || scratch_bytes < tc_scratch_bytes(Q, N) ||
      (reinterpret_cast<uintptr_t>(scratch) & 15u) || (reinterpret_cast<uintptr_t>(e.X) & 15u) ||
      (reinterpret_cast<uintptr_t>(e.Pp) & 15u))
    return cudaErrorNotSupported;
  CUtensorMap mapX, mapB;
  {
    const cuuint64_t dims[3] = {(cuuint64_t)e.I, (cuuint64_t)e.a, (cuuint64_t)e.O};
    const cuuint64_t strides[2] = {(cuuint64_t)e.I * 2, (cuuint64_t)e.a * e.I * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)kTcM, 1};
    if (!encode_bf16_map(&mapX, e.X, 3, dims, strides, box)) return cudaErrorNotSupported;
  }
  {
    const cuuint64_t dims[2] = {(cuuint64_t)Q, (cuuint64_t)(3 * N)};
    const cuuint64_t strides[1] = {(cuuint64_t)Q * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTcKC, (cuuint32_t)(3 * N)};
    if (!encode_bf16_map(&mapB, scratch, 2, dims, strides, box)) return cudaErrorNotSupported;
  }
  const cudaError_t attr_err = opt_in_smem(reinterpret_cast<const void*>(k_tc_token_expand), kTcSmem);
  if (attr_err != cudaSuccess) return attr_err;
  k_tc_split<<<dim3((unsigned)((Q + 31) / 32), (unsigned)((N + 31) / 32)), 256, 0, st>>>(
      e.V, nv, (int)Q, N, nv, static_cast<__nv_bfloat16*>(scratch), Q);
  TcArgs a = {e.Pp, (int)e.a, N, (int)Q, nv, (int)e.q_per_split, e.a * nv, (int)e.I, e.status, nv};
  dim3 grid((unsigned)((e.a + kTcM - 1) / kTcM), (unsigned)e.nsplit);
  k_tc_token_expand<<<grid, kTcThreads, kTcSmem, st>>>(mapX, mapB, a);
  return cudaGetLastError();
}
}  // namespace


// Y[q][j] = sum_k X[q][k] U[k][j] on the tensor cores.  `scratch` (device, 16-byte aligned, at least
// tc_scratch_bytes(K, N)) receives the bf16 operand.  Returns cudaErrorNotSupported when the shape or the
// alignment does not fit (the caller then takes the SIMT kernel).
cudaError_t launch_tc_lastmode(const ModeProdArgs& p, void* scratch, size_t scratch_bytes, cudaStream_t st) {
  if (p.I != 1) return launch_tc_token(p, scratch, scratch_bytes, st);
  const int64_t M = p.Q, K = p.a;
  const int nv = p.n_out, N = (nv + 15) / 16 * 16;
  if (p.I != 1 || nv % 4 != 0 || nv < 16 || N > kTcNMax || K % kTcKC != 0 || K < kTcKC || M < kTcM ||
      M >= (1ll << 31) || K >= (1ll << 31) || p.sj != 1 || p.so % 4 != 0 || p.ldb_j != 1 || !scratch ||
      scratch_bytes < tc_scratch_bytes(K, N) || (reinterpret_cast<uintptr_t>(scratch) & 15u) ||
      (reinterpret_cast<uintptr_t>(p.X) & 15u) || (reinterpret_cast<uintptr_t>(p.Y) & 15u))
    return cudaErrorNotSupported;
  EncodeFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  CUtensorMap mapX, mapB;
  const cuuint32_t estr[2] = {1, 1};
  {
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)M};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTcKC, (cuuint32_t)kTcM};
    if (enc(&mapX, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(p.X), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorNotSupported;
  }
  {
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)(3 * N)};
    const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTcKC, (cuuint32_t)(3 * N)};
    if (enc(&mapB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, scratch, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorNotSupported;
  }
  const size_t smem = kTcSmem;
  const cudaError_t attr_err = opt_in_smem(reinterpret_cast<const void*>(k_tc_lastmode), smem);
  if (attr_err != cudaSuccess) return attr_err;
  k_tc_split<<<dim3((unsigned)((K + 31) / 32), (unsigned)((N + 31) / 32)), 256, 0, st>>>(
      p.B, (int)p.ldb_k, (int)K, N, nv, static_cast<__nv_bfloat16*>(scratch), K);
  TcArgs a = {p.Y, (int)M, N, (int)K, (int)p.so, (int)K, 0, 0, p.status, nv};
  const unsigned grid = (unsigned)((M + kTcM - 1) / kTcM);
  k_tc_lastmode<<<grid, kTcThreads, smem, st>>>(mapX, mapB, a);
  return cudaGetLastError();
}

// Pp[s][k][j] = sum_{q in split s} X[q][k] V[q][j] on the tensor cores (the expansion P = A_m V of the last
// mode, X bf16 [Q x a], V fp32 [Q x r]).  `scratch` as above, at least tc_scratch_bytes(Q, r).
cudaError_t launch_tc_expand(const ExpandArgs& e, void* scratch, size_t scratch_bytes, cudaStream_t st) {
  if (e.I != 1) return launch_tc_token_expand(e, scratch, scratch_bytes, st);
  const int64_t Q = e.Q, A = e.a;
  const int nv = e.r, N = (nv + 15) / 16 * 16;
  if (e.I != 1 || nv % 4 != 0 || nv < 16 || N > kTcNMax || A % 8 != 0 || A < kTcM || Q % 8 != 0 || Q < kTcKC ||
      Q >= (1ll << 31) || A >= (1ll << 31) || e.q_per_split % kTcKC != 0 || e.q_per_split >= (1ll << 31) ||
      e.nsplit < 1 || !scratch || scratch_bytes < tc_scratch_bytes(Q, N) ||
      (reinterpret_cast<uintptr_t>(scratch) & 15u) || (reinterpret_cast<uintptr_t>(e.X) & 15u) ||
      (reinterpret_cast<uintptr_t>(e.Pp) & 15u))
    return cudaErrorNotSupported;
  EncodeFn enc = encode_fn();
  if (!enc) return cudaErrorNotSupported;
  CUtensorMap mapX, mapB;
  const cuuint32_t estr[2] = {1, 1};
  {
    const cuuint64_t dims[2] = {(cuuint64_t)A, (cuuint64_t)Q};
    const cuuint64_t strides[1] = {(cuuint64_t)A * 2};
    const cuuint32_t box[2] = {64, 64};
    if (enc(&mapX, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(e.X), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorNotSupported;
  }
  {
    const cuuint64_t dims[2] = {(cuuint64_t)Q, (cuuint64_t)(3 * N)};
    const cuuint64_t strides[1] = {(cuuint64_t)Q * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kTcKC, (cuuint32_t)(3 * N)};
    if (enc(&mapB, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, scratch, dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
      return cudaErrorNotSupported;
  }
  const size_t smem = kTcSmem;
  const cudaError_t attr_err = opt_in_smem(reinterpret_cast<const void*>(k_tc_expand), smem);
  if (attr_err != cudaSuccess) return attr_err;
  k_tc_split<<<dim3((unsigned)((Q + 31) / 32), (unsigned)((N + 31) / 32)), 256, 0, st>>>(
      e.V, nv, (int)Q, N, nv, static_cast<__nv_bfloat16*>(scratch), Q);
  TcArgs a = {e.Pp, (int)A, N, (int)Q, nv, (int)e.q_per_split, A * nv, 0, e.status, nv};
  dim3 grid((unsigned)((A + kTcM - 1) / kTcM), (unsigned)e.nsplit);
  k_tc_expand<<<grid, kTcThreads, smem, st>>>(mapX, mapB, a);
  return cudaGetLastError();
}

}  // namespace asi
