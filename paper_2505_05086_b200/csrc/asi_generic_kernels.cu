// Shape-generic kernels of the ASI path (any number of modes, any sizes, ranks <= 64).
// They are the correctness baseline every layer shape can fall back on; shape-specialised
// kernels live in their own files.
//
//   k_modeprod : Y = X x_m B^T-like small contraction over one mode (Sec. 3.2, m-mode product)
//   k_expand   : P_m = A_m V_m, split over the columns of the unfolding (Algorithm 1)
//   k_qr_gram / k_qr_gsum / k_qr_solve : Orthogonalize(P) as Cholesky-QR with the Gram matrix and the
//                triangular solve in fp64 -- in exact arithmetic the Gram-Schmidt basis
//   k_conv_tail: terms 4 and 5 of C_ASI (appendix "Speedup")
#include <cuda_bf16.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <type_traits>
#include <utility>

#include "asi_internal.h"

namespace asi {

ProfState g_prof = {0, nullptr, 0, 0, 0.0};

cudaError_t opt_in_smem(const void* kernel, size_t need) {
  static std::mutex lock;
  static std::map<std::pair<int, const void*>, size_t> granted;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  std::lock_guard<std::mutex> guard(lock);
  size_t& have = granted[std::make_pair(dev, kernel)];
  if (need <= have) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
  if (e == cudaSuccess) have = need;
  return e;
}

__device__ __forceinline__ float ld_as_float(const float* p) { return *p; }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }
// four neighbouring values read once (streaming hint), as fp32
template <typename TX>
__device__ __forceinline__ float4 ld4_stream(const TX* p);
template <>
__device__ __forceinline__ float4 ld4_stream<float>(const float* p) {
  return __ldcs(reinterpret_cast<const float4*>(p));
}
template <>
__device__ __forceinline__ float4 ld4_stream<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(p));
  const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
  const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
  return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
}

// ---------------------------------------------------------------------------------------------
// Tile loader: Xs[kl][ql] = X(k0 + kl, q0 + ql), zero outside [0,a) x [q0, q_end).
// Fibers strided by I > 1 (or short fibers) are read column-wise: consecutive threads take
// consecutive columns.  Contiguous long fibers (I == 1, a >= 32) are read along k.
// ---------------------------------------------------------------------------------------------
template <int KC, int TQ, int NT, typename TX>
__device__ __forceinline__ void load_x_tile(float (*Xs)[TQ + 1], const TX* __restrict__ X, int64_t a,
                                            int64_t I, int64_t k0, int64_t q0, int64_t q_end) {
  const int tid = threadIdx.x;
  // All the loads of a thread are issued first, from clamped addresses where the tile hangs over
  // the edge, and selected when they are stored: a load under a condition, or next to the store of
  // the one before, waits for its predecessor, and a chunk then costs KC * TQ / NT round trips.
  static_assert((KC * TQ) % NT == 0 && NT % TQ == 0, "threads must tile the chunk");
  constexpr int PER = KC * TQ / NT;
  float v[PER];
  if (I == 1 && a >= 32) {
#pragma unroll
    for (int t = 0; t < PER; ++t) {
      const int idx = tid + t * NT;
      const int64_t k = k0 + idx % KC, q = q0 + idx / KC;
      const bool on = k < a && q < q_end;
      v[t] = ld_as_float(X + (on ? q * a + k : 0));
    }
#pragma unroll
    for (int t = 0; t < PER; ++t) {
      const int idx = tid + t * NT;
      const int kl = idx % KC, ql = idx / KC;
      Xs[kl][ql] = (k0 + kl < a && q0 + ql < q_end) ? v[t] : 0.f;
    }
  } else {
    const int ql = tid % TQ;
    const int64_t q = q0 + ql;
    const bool qok = q < q_end;
    int64_t base = 0;
    if (qok) {
      const int64_t o = q / I, i = q - o * I;
      base = o * a * I + i;
    }
#pragma unroll
    for (int t = 0; t < PER; ++t) {
      const int64_t k = k0 + tid / TQ + t * (NT / TQ);
      v[t] = ld_as_float(X + ((qok && k < a) ? base + k * I : 0));
    }
#pragma unroll
    for (int t = 0; t < PER; ++t) {
      const int kl = tid / TQ + t * (NT / TQ);
      Xs[kl][ql] = (qok && k0 + kl < a) ? v[t] : 0.f;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// k_modeprod: one thread per column q, R outputs per thread.
// ---------------------------------------------------------------------------------------------
template <int R, typename TX>
__global__ void __launch_bounds__(128) k_modeprod(ModeProdArgs p) {
  constexpr int KC = 32, TQ = 128, NT = 128;
  __shared__ float Xs[KC][TQ + 1];
  __shared__ __align__(16) float Bs[KC][R];
  const int tid = threadIdx.x;
  const int64_t q0 = (int64_t)blockIdx.x * TQ;
  const int j0 = blockIdx.y * R;
  const TX* X = reinterpret_cast<const TX*>(p.X);

  float acc[R];
#pragma unroll
  for (int j = 0; j < R; ++j) acc[j] = 0.f;

  for (int64_t k0 = 0; k0 < p.a; k0 += KC) {
    load_x_tile<KC, TQ, NT, TX>(Xs, X, p.a, p.I, k0, q0, p.Q);
    {
      // the factor's chunk, its loads issued together like the tile's
      static_assert((KC * R) % NT == 0, "threads must tile the factor chunk");
      constexpr int PB = KC * R / NT;
      float b[PB];
#pragma unroll
      for (int t = 0; t < PB; ++t) {
        const int idx = tid + t * NT;
        const int64_t k = k0 + idx / R;
        const int jj = j0 + idx % R;
        b[t] = p.B[(k < p.a && jj < p.n_out) ? k * p.ldb_k + jj * p.ldb_j : 0];
      }
#pragma unroll
      for (int t = 0; t < PB; ++t) {
        const int idx = tid + t * NT;
        const int kl = idx / R, j = idx % R;
        Bs[kl][j] = (k0 + kl < p.a && j0 + j < p.n_out) ? b[t] : 0.f;
      }
    }
    __syncthreads();
    const int kmax = (int)((p.a - k0 < KC) ? (p.a - k0) : KC);
    for (int kl = 0; kl < kmax; ++kl) {
      const float x = Xs[kl][tid];
#pragma unroll
      for (int j = 0; j < R; j += 4) {
        const float4 b = *reinterpret_cast<const float4*>(&Bs[kl][j]);
        acc[j + 0] = fmaf(x, b.x, acc[j + 0]);
        acc[j + 1] = fmaf(x, b.y, acc[j + 1]);
        acc[j + 2] = fmaf(x, b.z, acc[j + 2]);
        acc[j + 3] = fmaf(x, b.w, acc[j + 3]);
      }
    }
    __syncthreads();
  }
  const int64_t q = q0 + tid;
  if (q < p.Q) {
    const int64_t o = q / p.I, i = q - o * p.I;
    float* y = p.Y + o * p.so + i * p.si;
#pragma unroll
    for (int j = 0; j < R; ++j)
      if (j0 + j < p.n_out) y[(int64_t)(j0 + j) * p.sj] = acc[j];
  }
}

// ---------------------------------------------------------------------------------------------
// k_gemm: register-tiled fp32 GEMM C = op(A) B for the last mode of a tensor (contiguous fibers) at
// ranks >= 16, where the thread-per-column kernels above run out of parallelism:
//   AKMAJOR  : C[M x N] = A[M x K] B[K x N], A stored [M][lda]      (V = A_m^T U, core product)
//   !AKMAJOR : C[M x N] = A^T B,            A stored [K][lda]      (P = A_m V), K split over grid.y
// CTA tile 64 x BN, K chunks of 32, thread tile 4 x BN/16; B and C are row-major with N columns.
// ---------------------------------------------------------------------------------------------
struct GemmArgs {
  const void* A;
  const float* B;
  float* C;            // [nsplit][M][N]
  int M, N, K;
  int64_t lda;
  int k_per_split;
  int vec8;            // bf16 A rows may be read 16 bytes at a time (aligned base, lda % 8 == 0)
};

template <bool AKMAJOR, int BM, int BN, typename TX>
__global__ void __launch_bounds__(BM * 4) k_gemm(GemmArgs p) {
  constexpr int BK = 32, TN = BN / 16, NT = BM * 4;
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.x * BM;
  const int kb = blockIdx.y * p.k_per_split;
  const int ke = (kb + p.k_per_split < p.K) ? kb + p.k_per_split : p.K;
  const TX* __restrict__ A = reinterpret_cast<const TX*>(p.A);
  float acc[4][TN];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;
  for (int k0 = kb; k0 < ke; k0 += BK) {
    if (AKMAJOR) {
      if (sizeof(TX) == 2 && p.vec8 && k0 + BK <= ke) {
        // 8 bf16 (16 bytes) per load: thread -> row r, k-octet o
        for (int idx = tid; idx < BM * (BK / 8); idx += NT) {
          const int r = idx / (BK / 8), o = idx % (BK / 8);
          const int m = m0 + r;
          uint4 raw = make_uint4(0u, 0u, 0u, 0u);
          if (m < p.M) raw = *reinterpret_cast<const uint4*>(A + (int64_t)m * p.lda + k0 + 8 * o);
          const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            As[8 * o + 2 * e][r] = __uint_as_float(w[e] << 16);
            As[8 * o + 2 * e + 1][r] = __uint_as_float(w[e] & 0xffff0000u);
          }
        }
      } else {
        for (int idx = tid; idx < BM * BK; idx += NT) {
          const int r = idx / BK, kk = idx % BK;
          const int m = m0 + r, k = k0 + kk;
          As[kk][r] = (m < p.M && k < ke) ? ld_as_float(A + (int64_t)m * p.lda + k) : 0.f;
        }
      }
    } else {
      for (int idx = tid; idx < BM * BK; idx += NT) {
        const int kk = idx / BM, r = idx % BM;
        const int m = m0 + r, k = k0 + kk;
        As[kk][r] = (m < p.M && k < ke) ? ld_as_float(A + (int64_t)k * p.lda + m) : 0.f;
      }
    }
    for (int idx = tid; idx < BK * BN; idx += NT) {
      const int kk = idx / BN, n = idx % BN;
      const int k = k0 + kk;
      Bs[kk][n] = (k < ke && n < p.N) ? p.B[(int64_t)k * p.N + n] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w};
      float bv[TN];
      if constexpr (TN == 4) {
        const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
        bv[0] = b.x; bv[1] = b.y; bv[2] = b.z; bv[3] = b.w;
      } else {
        const float2 b = *reinterpret_cast<const float2*>(&Bs[kk][tx * 2]);
        bv[0] = b.x; bv[1] = b.y;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* C = p.C + (int64_t)blockIdx.y * p.M * p.N;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= p.M) continue;
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      const int n = tx * TN + j;
      if (n < p.N) C[(int64_t)m * p.N + n] = acc[i][j];
    }
  }
}

template <bool AKMAJOR, typename TX>
static cudaError_t launch_gemm_t(const GemmArgs& g, int nsplit, cudaStream_t st) {
  GemmArgs a = g;
  a.vec8 = (sizeof(TX) == 2 && g.lda % 8 == 0 && (reinterpret_cast<uintptr_t>(g.A) & 15u) == 0 &&
            g.k_per_split % 8 == 0) ? 1 : 0;
  if ((int64_t)((g.M + 63) / 64) * nsplit >= 148) {     // enough 64-row tiles to fill the machine
    dim3 grid((unsigned)((g.M + 63) / 64), (unsigned)nsplit);
    if (g.N <= 32) k_gemm<AKMAJOR, 64, 32, TX><<<grid, 256, 0, st>>>(a);
    else k_gemm<AKMAJOR, 64, 64, TX><<<grid, 256, 0, st>>>(a);
  } else {
    dim3 grid((unsigned)((g.M + 31) / 32), (unsigned)nsplit);
    if (g.N <= 32) k_gemm<AKMAJOR, 32, 32, TX><<<grid, 128, 0, st>>>(a);
    else k_gemm<AKMAJOR, 32, 64, TX><<<grid, 128, 0, st>>>(a);
  }
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// k_rowstream: the first-mode product Y[j][q] = sum_k B(k, j) X[k][q] (O = 1: row k of X is one
// contiguous slab of Q values) with n_out <= R <= 8.  Pure streaming: a thread owns four neighbouring
// columns and one of KS slices of the rows, and walks down its rows with UNR 16-byte loads in flight
// (a single thread walking all rows is bound by the latency of its own loads); the KS partial sums
// meet in shared memory in slice order.  The factor sits in shared memory.  X is read exactly once,
// coalesced; nothing else of size moves.
// ---------------------------------------------------------------------------------------------
template <int R, typename TX>
__global__ void __launch_bounds__(256) k_rowstream(ModeProdArgs p) {
  constexpr int NT = 256, CG = 64, KS = NT / CG, UNR = 8;
  extern __shared__ __align__(16) float rs_smem[];
  float* Bsm = rs_smem;                              // [a][R], zero-padded
  float* part = rs_smem + (((int)p.a * R + 3) & ~3); // [KS - 1][CG][4 R]
  const int tid = threadIdx.x;
  for (int idx = tid; idx < (int)p.a * R; idx += NT) {
    const int k = idx / R, j = idx % R;
    Bsm[idx] = (j < p.n_out) ? p.B[k * p.ldb_k + j * p.ldb_j] : 0.f;
  }
  __syncthreads();
  const int cg = tid & (CG - 1), ks = tid / CG;
  const int64_t q = ((int64_t)blockIdx.x * CG + cg) * 4;
  const bool live = q < p.Q;
  float acc[4][R];
#pragma unroll
  for (int c = 0; c < 4; ++c)
#pragma unroll
    for (int j = 0; j < R; ++j) acc[c][j] = 0.f;
  const int a = (int)p.a;
  const int kper = (a + KS - 1) / KS;
  int k0 = ks * kper;
  const int k1 = (k0 + kper < a) ? k0 + kper : a;
  if (live) {
    const TX* X = reinterpret_cast<const TX*>(p.X) + q;
    // batches of UNR rows, all loads of a batch issued before any is used; rows past the end of the
    // slice are read from the slice's last row and contribute zero
    for (; k0 < k1; k0 += UNR) {
      float4 x[UNR];
#pragma unroll
      for (int u = 0; u < UNR; ++u) x[u] = ld4_stream<TX>(X + (int64_t)((k0 + u < k1) ? (k0 + u) : (k1 - 1)) * p.Q);
#pragma unroll
      for (int u = 0; u < UNR; ++u) {
        const bool on = k0 + u < k1;
        const float xs[4] = {on ? x[u].x : 0.f, on ? x[u].y : 0.f, on ? x[u].z : 0.f, on ? x[u].w : 0.f};
        const int kr = on ? (k0 + u) : (k1 - 1);
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          const float4 b = *reinterpret_cast<const float4*>(Bsm + kr * R + j);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            acc[c][j] = fmaf(xs[c], b.x, acc[c][j]);
            acc[c][j + 1] = fmaf(xs[c], b.y, acc[c][j + 1]);
            acc[c][j + 2] = fmaf(xs[c], b.z, acc[c][j + 2]);
            acc[c][j + 3] = fmaf(xs[c], b.w, acc[c][j + 3]);
          }
        }
      }
    }
  }
  if (ks > 0) {
    float* dst = part + ((ks - 1) * CG + cg) * 4 * R;
#pragma unroll
    for (int c = 0; c < 4; ++c)
#pragma unroll
      for (int j = 0; j < R; j += 4)
        *reinterpret_cast<float4*>(dst + c * R + j) = make_float4(acc[c][j], acc[c][j + 1], acc[c][j + 2], acc[c][j + 3]);
  }
  __syncthreads();
  if (ks == 0 && live) {
#pragma unroll 1
    for (int s = 1; s < KS; ++s) {
      const float* src = part + ((s - 1) * CG + cg) * 4 * R;
#pragma unroll
      for (int c = 0; c < 4; ++c)
#pragma unroll
        for (int j = 0; j < R; ++j) acc[c][j] += src[c * R + j];
    }
#pragma unroll
    for (int j = 0; j < R; ++j)
      if (j < p.n_out)
        *reinterpret_cast<float4*>(p.Y + (int64_t)j * p.sj + q) = make_float4(acc[0][j], acc[1][j], acc[2][j], acc[3][j]);
  }
}

template <typename TX>
static cudaError_t launch_modeprod_t(const ModeProdArgs& p, cudaStream_t st) {
  if (p.Q <= 0 || p.n_out <= 0) return cudaSuccess;
  ProfScope prof(ASI_K_MODEPROD, st,
                 (double)p.Q * p.a * sizeof(TX) + 4.0 * ((double)p.a * p.n_out + (double)p.Q * p.n_out));
  if constexpr (std::is_same<TX, __nv_bfloat16>::value) {
    // a dense contraction with a wide factor: tensor cores (tcgen05), when the shape fits
    const cudaError_t e = launch_tc_lastmode(p, p.tc_scratch, p.tc_scratch_bytes, st);
    if (e != cudaErrorNotSupported) return e;
  }
  if (p.O == 1 && p.n_out <= 8 && p.si == 1 && p.Q % 4 == 0 && p.sj % 4 == 0 && p.Q >= (1 << 16) &&
      p.a <= 512 && p.a >= 8 && (reinterpret_cast<uintptr_t>(p.X) & 15u) == 0 &&
      (reinterpret_cast<uintptr_t>(p.Y) & 15u) == 0) {
    const unsigned grid = (unsigned)((p.Q / 4 + 63) / 64);
    const auto smem = [&](int R) { return (size_t)((((int)p.a * R + 3) & ~3) + 3 * 64 * 4 * R) * 4; };
    if (p.n_out <= 4) k_rowstream<4, TX><<<grid, 256, smem(4), st>>>(p);
    else k_rowstream<8, TX><<<grid, 256, smem(8), st>>>(p);
    return cudaGetLastError();
  }
  if (p.I == 1 && p.n_out >= 16 && p.n_out <= 64 && p.a >= 64 && p.Q >= 64 && p.sj == 1 && p.so == p.n_out &&
      p.ldb_k == p.n_out && p.ldb_j == 1 && p.Q < (1 << 30) && p.a < (1 << 30)) {
    GemmArgs g = {p.X, p.B, p.Y, (int)p.Q, p.n_out, (int)p.a, p.a, (int)p.a, 0};
    return launch_gemm_t<true, TX>(g, 1, st);
  }
  int R = 4;
  while (R < p.n_out && R < 64) R *= 2;
  dim3 grid((unsigned)((p.Q + 127) / 128), (unsigned)((p.n_out + R - 1) / R));
  switch (R) {
    case 4: k_modeprod<4, TX><<<grid, 128, 0, st>>>(p); break;
    case 8: k_modeprod<8, TX><<<grid, 128, 0, st>>>(p); break;
    case 16: k_modeprod<16, TX><<<grid, 128, 0, st>>>(p); break;
    case 32: k_modeprod<32, TX><<<grid, 128, 0, st>>>(p); break;
    default: k_modeprod<64, TX><<<grid, 128, 0, st>>>(p); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_modeprod(const ModeProdArgs& p, bool x_bf16, cudaStream_t st) {
  return x_bf16 ? launch_modeprod_t<__nv_bfloat16>(p, st) : launch_modeprod_t<float>(p, st);
}

// ---------------------------------------------------------------------------------------------
// k_expand: CTA (kc, s) owns rows [32 kc, 32 kc + 32) of P and the column split s.
// Thread (kl, jg) accumulates R/8 entries of its row.  Partials are summed later in a fixed
// order, so the result does not depend on scheduling.
// ---------------------------------------------------------------------------------------------
template <int R, typename TX>
__global__ void __launch_bounds__(256) k_expand(ExpandArgs p) {
  constexpr int KC = kExpandKC, TQ = 64, NT = 256, RJ = R / 8;
  __shared__ float Xs[KC][TQ + 1];
  __shared__ __align__(16) float Vs[TQ][R];
  const int tid = threadIdx.x;
  const int kl = tid / 8, jg = tid % 8;
  const int64_t k0 = (int64_t)blockIdx.x * KC;
  const int s = blockIdx.y;
  const int64_t qb = (int64_t)s * p.q_per_split;
  int64_t qe = qb + p.q_per_split;
  if (qe > p.Q) qe = p.Q;
  const TX* X = reinterpret_cast<const TX*>(p.X);

  float acc[RJ];
#pragma unroll
  for (int j = 0; j < RJ; ++j) acc[j] = 0.f;

  for (int64_t q0 = qb; q0 < qe; q0 += TQ) {
    load_x_tile<KC, TQ, NT, TX>(Xs, X, p.a, p.I, k0, q0, qe);
    for (int idx = tid; idx < TQ * R; idx += NT) {
      const int ql = idx / R, j = idx % R;
      const int64_t q = q0 + ql;
      Vs[ql][j] = (q < qe && j < p.r) ? p.V[q * p.r + j] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int ql = 0; ql < TQ; ++ql) {
      const float x = Xs[kl][ql];
#pragma unroll
      for (int j = 0; j < RJ; ++j) acc[j] = fmaf(x, Vs[ql][jg * RJ + j], acc[j]);
    }
    __syncthreads();
  }
  const int64_t k = k0 + kl;
  if (k < p.a) {
#pragma unroll
    for (int j = 0; j < RJ; ++j) {
      const int jj = jg * RJ + j;
      if (jj < p.r) p.Pp[((int64_t)s * p.a + k) * p.r + jj] = acc[j];
    }
  }
}

template <typename TX>
static cudaError_t launch_expand_t(const ExpandArgs& p, cudaStream_t st) {
  ProfScope prof(ASI_K_EXPAND, st,
                 (double)p.Q * p.a * sizeof(TX) + 4.0 * ((double)p.Q * p.r + (double)p.nsplit * p.a * p.r));
  if constexpr (std::is_same<TX, __nv_bfloat16>::value) {
    const cudaError_t e = launch_tc_expand(p, p.tc_scratch, p.tc_scratch_bytes, st);   // tensor cores when it fits
    if (e != cudaErrorNotSupported) return e;
  }
  if (p.I == 1 && p.r >= 16 && p.r <= 64 && p.a >= 64 && p.Q < (1 << 30) && p.a < (1 << 30)) {
    GemmArgs g = {p.X, p.V, p.Pp, (int)p.a, p.r, (int)p.Q, p.a, (int)p.q_per_split, 0};
    return launch_gemm_t<false, TX>(g, p.nsplit, st);
  }
  int R = 8;
  while (R < p.r) R *= 2;
  dim3 grid((unsigned)((p.a + kExpandKC - 1) / kExpandKC), (unsigned)p.nsplit);
  switch (R) {
    case 8: k_expand<8, TX><<<grid, 256, 0, st>>>(p); break;
    case 16: k_expand<16, TX><<<grid, 256, 0, st>>>(p); break;
    case 32: k_expand<32, TX><<<grid, 256, 0, st>>>(p); break;
    case 64: k_expand<64, TX><<<grid, 256, 0, st>>>(p); break;
    default: k_expand<128, TX><<<grid, 256, 0, st>>>(p); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_expand(const ExpandArgs& p, bool x_bf16, cudaStream_t st) {
  return x_bf16 ? launch_expand_t<__nv_bfloat16>(p, st) : launch_expand_t<float>(p, st);
}

// ---------------------------------------------------------------------------------------------
// k_fiber: P_m = A_m (A_m^T U_m) for one mode in ONE pass over the activation (Algorithm 1, both
// products of a mode).  A tile is TQ whole fibers of the mode: a rows of TQ contiguous values when the
// mode is not the last one, TQ contiguous fibers when it is.  Per tile, V[q,:] = sum_k X(k,q) U[k,:]
// stays in shared memory and P[k,:] += sum_q X(k,q) V[q,:] accumulates in registers across all tiles
// of the CTA, so V never reaches global memory and each CTA writes one partial of P.  fp32 tiles are
// double-buffered with cp.async.  Requires a <= 128, r <= R.
// ---------------------------------------------------------------------------------------------
constexpr int kFiberTQ = 64;

__device__ __forceinline__ unsigned smem_addr(const void* p) {
  return static_cast<unsigned>(__cvta_generic_to_shared(p));
}

template <int R, typename TX>
__global__ void __launch_bounds__(256) k_fiber(FiberArgs p) {
  constexpr int TQ = kFiberTQ, NT = 256, KS = NT / TQ;
  extern __shared__ __align__(16) float fsm[];
  const int tid = threadIdx.x, lane = tid & 31;
  const int a = (int)p.a, r = p.r;
  const bool last = p.I == 1;                       // fibers are contiguous
  // logical X(k, q) of a staged tile sits at k*SK + q*SQ
  const int PQ = TQ + 4;                            // row pitch, 16-byte aligned rows
  const int PA = a | 1;                             // fiber pitch (odd: conflict-free fiber-per-thread reads)
  const int SK = last ? 1 : PQ, SQ = last ? PA : 1;
  const int tile_floats = last ? TQ * PA : a * PQ;
  float* Xs0 = fsm;
  float* Xs1 = fsm + ((tile_floats + 3) & ~3);
  float* Us = Xs1 + ((tile_floats + 3) & ~3);      // [a][R]
  float* Vp = Us + a * R;                           // [KS][TQ][R]
  float* Vs = Vp + KS * TQ * R;                     // [TQ][R]
  for (int idx = tid; idx < a * R; idx += NT) {
    const int k = idx / R, j = idx % R;
    Us[idx] = (j < r) ? p.U[k * r + j] : 0.f;
  }
  const TX* __restrict__ X = reinterpret_cast<const TX*>(p.X);
  const int64_t tiles_per_o = last ? 0 : (p.I + TQ - 1) / TQ;

  auto stage = [&](float* dst, int64_t t, int& n_q) {
    if (last) {
      const int64_t q0 = t * TQ;
      n_q = (int)((p.O - q0 < TQ) ? (p.O - q0) : TQ);
      const TX* src = X + q0 * a;
      for (int idx = tid; idx < n_q * a; idx += NT) {
        const int q = idx / a, k = idx - q * a;
        if constexpr (sizeof(TX) == 4) {
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_addr(dst + q * PA + k)), "l"(src + idx) : "memory");
        } else {
          dst[q * PA + k] = ld_as_float(src + idx);
        }
      }
    } else {
      const int64_t o = t / tiles_per_o, i0 = (t - o * tiles_per_o) * TQ;
      n_q = (int)((p.I - i0 < TQ) ? (p.I - i0) : TQ);
      const TX* src = X + o * a * p.I + i0;
      if (sizeof(TX) == 4 && p.vec4) {
        const int n4 = n_q >> 2;                    // I and TQ are multiples of 4 here
        for (int idx = tid; idx < a * n4; idx += NT) {
          const int k = idx / n4, v = idx - k * n4;
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst + k * PQ + 4 * v)),
                       "l"(src + (int64_t)k * p.I + 4 * v)
                       : "memory");
        }
      } else {
        for (int idx = tid; idx < a * n_q; idx += NT) {
          const int k = idx / n_q, q = idx - k * n_q;
          if constexpr (sizeof(TX) == 4) {
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(smem_addr(dst + k * PQ + q)),
                         "l"(src + (int64_t)k * p.I + q)
                         : "memory");
          } else {
            dst[k * PQ + q] = ld_as_float(src + (int64_t)k * p.I + q);
          }
        }
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  // thread roles: projection (q, ks), expansion (k, qs)
  const int pq = tid % TQ, pks = tid / TQ;
  int QS = 32;
  while (QS * a > NT && QS > 1) QS >>= 1;           // largest power of two with QS * a <= 256
  const int ek = tid / QS, eqs = tid % QS;
  float acc2[R];
#pragma unroll
  for (int j = 0; j < R; ++j) acc2[j] = 0.f;

  int n_cur = 0, n_next = 0;
  int64_t t = blockIdx.x;
  if (t < p.n_tiles) stage(Xs0, t, n_cur);
  int buf = 0;
  for (; t < p.n_tiles; t += gridDim.x) {
    float* Xc = buf ? Xs1 : Xs0;
    float* Xn = buf ? Xs0 : Xs1;
    const int64_t tn = t + gridDim.x;
    if (tn < p.n_tiles) {
      stage(Xn, tn, n_next);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    // projection: V[q,:] = sum_k X(k,q) U[k,:]
    {
      float acc[R];
#pragma unroll
      for (int j = 0; j < R; ++j) acc[j] = 0.f;
      if (pq < n_cur) {
#pragma unroll 4
        for (int k = pks; k < a; k += KS) {
          const float x = Xc[k * SK + pq * SQ];
#pragma unroll
          for (int j = 0; j < R; j += 4) {
            const float4 u = *reinterpret_cast<const float4*>(Us + k * R + j);
            acc[j] = fmaf(x, u.x, acc[j]);
            acc[j + 1] = fmaf(x, u.y, acc[j + 1]);
            acc[j + 2] = fmaf(x, u.z, acc[j + 2]);
            acc[j + 3] = fmaf(x, u.w, acc[j + 3]);
          }
        }
      }
#pragma unroll
      for (int j = 0; j < R; j += 4)
        *reinterpret_cast<float4*>(Vp + (pks * TQ + pq) * R + j) = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
    }
    __syncthreads();
    for (int idx = tid; idx < TQ * R; idx += NT) {
      float v = 0.f;
#pragma unroll
      for (int ks = 0; ks < KS; ++ks) v += Vp[ks * TQ * R + idx];
      Vs[idx] = v;
    }
    __syncthreads();
    // expansion: P[k,:] += sum_q X(k,q) V[q,:]
    if (ek < a) {
#pragma unroll 4
      for (int q = eqs; q < n_cur; q += QS) {
        const float x = Xc[ek * SK + q * SQ];
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          const float4 v = *reinterpret_cast<const float4*>(Vs + q * R + j);
          acc2[j] = fmaf(x, v.x, acc2[j]);
          acc2[j + 1] = fmaf(x, v.y, acc2[j + 1]);
          acc2[j + 2] = fmaf(x, v.z, acc2[j + 2]);
          acc2[j + 3] = fmaf(x, v.w, acc2[j + 3]);
        }
      }
    }
    __syncthreads();
    n_cur = n_next;
    buf ^= 1;
  }
  // the QS threads of a row meet by shuffles (fixed order), one partial of P per CTA
#pragma unroll
  for (int j = 0; j < R; ++j)
    for (int off = 1; off < QS; off <<= 1) acc2[j] += __shfl_xor_sync(0xffffffffu, acc2[j], off);
  (void)lane;
  if (ek < a && eqs == 0) {
    float* dst = p.Pp + ((int64_t)blockIdx.x * a + ek) * r;
#pragma unroll
    for (int j = 0; j < R; ++j)
      if (j < r) dst[j] = acc2[j];
  }
}

// ---------------------------------------------------------------------------------------------
// k_plane: the two spatial modes of a conv activation in one pass.  A tile is NP = 256 / S whole
// planes X[h][w] (S x S, S a multiple of 4); thread (plane, i) owns column w = i and row h = i:
//   V3[w,:] = sum_h X[h][w] U3[h,:]   (column read)      V4[h,:] = sum_w X[h][w] U4[w,:]   (row read)
//   P3[h,:] += sum_w X[h][w] V3[w,:]  (row read)         P4[w,:] += sum_h X[h][w] V4[h,:]  (column read)
// i.e. P_m = A_m (A_m^T U_m) for m = 3, 4 (Algorithm 1).  Rows are read as float4 (conflict-free for the
// unpadded pitch S), columns as scalars.  P3 / P4 accumulate in registers across the CTA's tiles.
// ---------------------------------------------------------------------------------------------
template <int R, typename TX>
__global__ void __launch_bounds__(256) k_plane(PlaneArgs p) {
  constexpr int NT = 256;
  extern __shared__ __align__(16) float fsm[];
  const int tid = threadIdx.x;
  const int S = p.S, SS = S * S, NP = NT / S;
  float* Xs0 = fsm;
  float* Xs1 = Xs0 + NP * SS;
  float* U3s = Xs1 + NP * SS;                       // [S][R]
  float* U4s = U3s + S * R;                         // [S][R]
  float* V3s = U4s + S * R;                         // [NP][S][R]
  float* V4s = V3s + NP * S * R;                    // [NP][S][R]
  for (int idx = tid; idx < S * R; idx += NT) {
    const int k = idx / R, j = idx % R;
    U3s[idx] = (j < p.r3) ? p.U3[k * p.r3 + j] : 0.f;
    U4s[idx] = (j < p.r4) ? p.U4[k * p.r4 + j] : 0.f;
  }
  const TX* __restrict__ X = reinterpret_cast<const TX*>(p.X);
  const int pl = tid / S, i = tid - pl * S;
  const int64_t n_tiles = (p.n_planes + NP - 1) / NP;

  auto stage = [&](float* dst, int64_t t, int& np) {
    const int64_t p0 = t * NP;
    np = (int)((p.n_planes - p0 < NP) ? (p.n_planes - p0) : NP);
    const TX* src = X + p0 * SS;
    if (sizeof(TX) == 4 && p.vec4) {
      for (int idx = tid; idx < np * SS / 4; idx += NT)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_addr(dst + 4 * idx)), "l"(src + 4 * idx) : "memory");
    } else {
      for (int idx = tid; idx < np * SS; idx += NT) dst[idx] = ld_as_float(src + idx);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  float acc3[R], acc4[R];
#pragma unroll
  for (int j = 0; j < R; ++j) acc3[j] = acc4[j] = 0.f;
  int n_cur = 0, n_next = 0, buf = 0;
  int64_t t = blockIdx.x;
  if (t < n_tiles) stage(Xs0, t, n_cur);
  for (; t < n_tiles; t += gridDim.x) {
    float* Xc = buf ? Xs1 : Xs0;
    float* Xn = buf ? Xs0 : Xs1;
    const int64_t tn = t + gridDim.x;
    if (tn < n_tiles) {
      stage(Xn, tn, n_next);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const bool on = pl < n_cur;                     // pl < NP follows
    const float* Xp = Xc + pl * SS;
    if (on) {
      float v3[R], v4[R];
#pragma unroll
      for (int j = 0; j < R; ++j) v3[j] = v4[j] = 0.f;
#pragma unroll 4
      for (int h = 0; h < S; ++h) {                 // column i
        const float x = Xp[h * S + i];
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          const float4 u = *reinterpret_cast<const float4*>(U3s + h * R + j);
          v3[j] = fmaf(x, u.x, v3[j]); v3[j + 1] = fmaf(x, u.y, v3[j + 1]);
          v3[j + 2] = fmaf(x, u.z, v3[j + 2]); v3[j + 3] = fmaf(x, u.w, v3[j + 3]);
        }
      }
#pragma unroll 2
      for (int w = 0; w < S; w += 4) {              // row i
        const float4 x = *reinterpret_cast<const float4*>(Xp + i * S + w);
        const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
#pragma unroll
          for (int j = 0; j < R; j += 4) {
            const float4 u = *reinterpret_cast<const float4*>(U4s + (w + e) * R + j);
            v4[j] = fmaf(xs[e], u.x, v4[j]); v4[j + 1] = fmaf(xs[e], u.y, v4[j + 1]);
            v4[j + 2] = fmaf(xs[e], u.z, v4[j + 2]); v4[j + 3] = fmaf(xs[e], u.w, v4[j + 3]);
          }
      }
#pragma unroll
      for (int j = 0; j < R; j += 4) {
        *reinterpret_cast<float4*>(V3s + (pl * S + i) * R + j) = make_float4(v3[j], v3[j + 1], v3[j + 2], v3[j + 3]);
        *reinterpret_cast<float4*>(V4s + (pl * S + i) * R + j) = make_float4(v4[j], v4[j + 1], v4[j + 2], v4[j + 3]);
      }
    }
    __syncthreads();
    if (on) {
      const float* V3p = V3s + pl * S * R;
      const float* V4p = V4s + pl * S * R;
#pragma unroll 2
      for (int w = 0; w < S; w += 4) {              // row i: P3[i,:]
        const float4 x = *reinterpret_cast<const float4*>(Xp + i * S + w);
        const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
#pragma unroll
          for (int j = 0; j < R; j += 4) {
            const float4 v = *reinterpret_cast<const float4*>(V3p + (w + e) * R + j);
            acc3[j] = fmaf(xs[e], v.x, acc3[j]); acc3[j + 1] = fmaf(xs[e], v.y, acc3[j + 1]);
            acc3[j + 2] = fmaf(xs[e], v.z, acc3[j + 2]); acc3[j + 3] = fmaf(xs[e], v.w, acc3[j + 3]);
          }
      }
#pragma unroll 4
      for (int h = 0; h < S; ++h) {                 // column i: P4[i,:]
        const float x = Xp[h * S + i];
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          const float4 v = *reinterpret_cast<const float4*>(V4p + h * R + j);
          acc4[j] = fmaf(x, v.x, acc4[j]); acc4[j + 1] = fmaf(x, v.y, acc4[j + 1]);
          acc4[j + 2] = fmaf(x, v.z, acc4[j + 2]); acc4[j + 3] = fmaf(x, v.w, acc4[j + 3]);
        }
      }
    }
    __syncthreads();
    n_cur = n_next;
    buf ^= 1;
  }
  // the NP planes of the CTA meet in shared memory in plane order: one partial of P3 and P4 per CTA
  if (pl < NP) {
#pragma unroll
    for (int j = 0; j < R; ++j) {
      V3s[(pl * S + i) * R + j] = acc3[j];
      V4s[(pl * S + i) * R + j] = acc4[j];
    }
  }
  __syncthreads();
  for (int idx = tid; idx < S * R; idx += NT) {
    const int k = idx / R, j = idx % R;
    float s3 = 0.f, s4 = 0.f;
    for (int q = 0; q < NP; ++q) {
      s3 += V3s[q * S * R + idx];
      s4 += V4s[q * S * R + idx];
    }
    if (j < p.r3) p.Pp3[((int64_t)blockIdx.x * S + k) * p.r3 + j] = s3;
    if (j < p.r4) p.Pp4[((int64_t)blockIdx.x * S + k) * p.r4 + j] = s4;
  }
}

size_t plane_smem(int S) {
  const int NP = 256 / S;
  return 4 * ((size_t)2 * NP * S * S + 2 * S * 8 + 2 * NP * S * 8) + 64;
}

template <int R, typename TX>
static cudaError_t launch_plane_t(const PlaneArgs& p, int grid, cudaStream_t st) {
  const size_t smem = plane_smem(p.S);   // the default limit counts static shared memory too: always opt in
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_plane<R, TX>), smem);
  if (e != cudaSuccess) return e;
  k_plane<R, TX><<<grid, 256, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_plane(const PlaneArgs& p, int grid, bool x_bf16, cudaStream_t st) {
  ProfScope prof(ASI_K_EXPAND, st,
                 (double)p.n_planes * p.S * p.S * (x_bf16 ? 2 : 4) + 4.0 * p.S * (p.r3 + p.r4) * (grid + 1));
  const int r = p.r3 > p.r4 ? p.r3 : p.r4;
  if (r <= 4) return x_bf16 ? launch_plane_t<4, __nv_bfloat16>(p, grid, st) : launch_plane_t<4, float>(p, grid, st);
  return x_bf16 ? launch_plane_t<8, __nv_bfloat16>(p, grid, st) : launch_plane_t<8, float>(p, grid, st);
}

size_t fiber_smem(int a) {
  const int TQ = kFiberTQ, PQ = TQ + 4, PA = a | 1;
  const size_t tile = (size_t)std::max(TQ * PA, a * PQ);
  return 4 * (2 * ((tile + 3) & ~(size_t)3) + (size_t)a * 8 + 5 * TQ * 8) + 64;
}

int64_t fiber_tiles(int64_t O, int64_t a, int64_t I) {
  (void)a;
  return I == 1 ? (O + kFiberTQ - 1) / kFiberTQ : O * ((I + kFiberTQ - 1) / kFiberTQ);
}

template <int R, typename TX>
static cudaError_t launch_fiber_t(const FiberArgs& p, int grid, cudaStream_t st) {
  const size_t smem = fiber_smem((int)p.a);
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_fiber<R, TX>), smem);
  if (e != cudaSuccess) return e;
  k_fiber<R, TX><<<grid, 256, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_fiber(const FiberArgs& p, int grid, bool x_bf16, cudaStream_t st) {
  ProfScope prof(ASI_K_EXPAND, st,
                 (double)p.O * p.a * p.I * (x_bf16 ? 2 : 4) + 4.0 * ((double)p.a * p.r * (grid + 1)));
  if (p.r <= 4) return x_bf16 ? launch_fiber_t<4, __nv_bfloat16>(p, grid, st) : launch_fiber_t<4, float>(p, grid, st);
  return x_bf16 ? launch_fiber_t<8, __nv_bfloat16>(p, grid, st) : launch_fiber_t<8, float>(p, grid, st);
}

// ---------------------------------------------------------------------------------------------
// Orthogonalize.  Stage 1 (k_qr_gram): sum the column-split partials of P in fp64 in a fixed
// order, keep P in fp64, and form this row chunk's share of G = P^T P.  Stage 2 (k_qr_solve):
// G = R^T R by Cholesky (R upper, positive diagonal), U = P R^{-1} row by row.  That U is the
// Gram-Schmidt basis of the columns of P.  A pivot d_j with d_j <= 1e-12 * trace(G), i.e. a
// Gram-Schmidt residual below 1e-6 * ||P||_F, raises ASI_ERR_RANK_DEFICIENT in the status word.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_qr_gram(QRArgs args) {
  const QRMode M = args.m[blockIdx.y];
  const int c = blockIdx.x;
  if (c >= M.nchunk || M.r > kQRMaxRank) return;   // ranks above 64 take the k_qrb_* kernels
  __shared__ double Ps[kQRRows * kQRMaxRank];      // this chunk's rows of P, pitch r
  constexpr int kPer = 16;
  static_assert(kQRRows * kQRMaxRank == kPer * 256, "one thread holds 16 elements of a full chunk");
  const int tid = threadIdx.x;
  const int r = M.r;
  const int row0 = c * kQRRows;
  const int nrows = min(kQRRows, M.a - row0);
  const int nval = nrows * r;                        // the chunk is one contiguous run of P
  const int64_t base = (int64_t)row0 * r;
  // A thread has 16 accumulators: `ethr` elements (a power of two) times 16 / ethr lanes that take
  // every (16 / ethr)-th split, so 16 loads are in flight whatever the chunk's size; the lanes of
  // an element then fold pairwise.  The order of the sum is fixed by (nval, nsplit) alone.
  int ethr = 1, lg = 0;
  while (ethr * 256 < nval) { ethr <<= 1; ++lg; }
  const int ssub = 16 >> lg;
  const int64_t sstride = (int64_t)M.a * r;
  double acc[kPer];
#pragma unroll
  for (int q = 0; q < kPer; ++q) acc[q] = 0.0;
  // four batches of 16 loads are issued before the first is used: with many splits and a full chunk (one
  // split per batch) the loop is otherwise one memory round trip per split
  constexpr int kBatch = 4;
  for (int s0 = 0; s0 < M.nsplit; s0 += kBatch * ssub) {
    float t[kBatch][kPer];
#pragma unroll
    for (int b = 0; b < kBatch; ++b)
#pragma unroll
      for (int q = 0; q < kPer; ++q) {
        const int idx = tid + (q & (ethr - 1)) * 256;
        const int s = s0 + b * ssub + (q >> lg);
        const bool on = idx < nval && s < M.nsplit;
        // Every load is issued, from a clamped address when off, and nothing here touches its
        // result: a use or a condition next to a load makes the following loads wait for it.
        t[b][q] = __ldcg(M.Pp + (on ? s * sstride + base + idx : 0));
      }
#pragma unroll
    for (int b = 0; b < kBatch; ++b)
#pragma unroll
      for (int q = 0; q < kPer; ++q) {
        const bool on = tid + (q & (ethr - 1)) * 256 < nval && s0 + b * ssub + (q >> lg) < M.nsplit;
        acc[q] += on ? (double)t[b][q] : 0.0;
      }
  }
#pragma unroll
  for (int h = kPer / 2; h >= 1; h >>= 1)
    if (h >= ethr) {
#pragma unroll
      for (int q = 0; q < h; ++q) acc[q] += acc[q + h];
    }
#pragma unroll
  for (int q = 0; q < kPer; ++q) {
    const int idx = tid + q * 256;
    if (q < ethr && idx < nval) {
      M.Pred[base + idx] = acc[q];
      Ps[idx] = acc[q];
    }
  }
  __syncthreads();
  // Thread (ti, tj) owns G[ti + 16x][tj + 16y]: per row of P it reads 4 + 4 values for 16 products.
  const int ti = tid >> 4, tj = tid & 15;
  double g[4][4];
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) g[x][y] = 0.0;
  for (int rl = 0; rl < nrows; ++rl) {
    const double* prow = Ps + rl * r;
    double pi[4], pj[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      pi[t] = (ti + 16 * t < r) ? prow[ti + 16 * t] : 0.0;
      pj[t] = (tj + 16 * t < r) ? prow[tj + 16 * t] : 0.0;
    }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) g[x][y] = fma(pi[x], pj[y], g[x][y]);
  }
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int i = ti + 16 * x, j = tj + 16 * y;
      if (i < r && j < r && j >= i) M.Gp[((int64_t)c * r + i) * r + j] = g[x][y];
    }
}

// k_qr_gsum: G = sum of the row chunks' shares, chunk by chunk in order, left in the place of
// share 0, so that the solve kernel's CTAs read r*r numbers each instead of every share.  One
// thread per element of the upper triangle, eight loads in flight.
__global__ void __launch_bounds__(256) k_qr_gsum(QRArgs args) {
  const QRMode M = args.m[blockIdx.y];
  const int rr = M.r * M.r;
  const int e = blockIdx.x * 256 + threadIdx.x;
  if (M.r > kQRMaxRank || e >= rr || (e % M.r) < (e / M.r)) return;
  const double* G = M.Gp + e;
  double acc = 0.0;
#pragma unroll 16
  for (int cc = 0; cc < M.nchunk; ++cc) acc += __ldcg(G + (int64_t)cc * rr);
  M.Gp[e] = acc;
}

// k_qr_solve keeps the running Schur complement of the Cholesky factorisation and the rows it
// solves in registers; shared memory carries only what one step hands to the next (the pivot
// row, the next unknown of each row) and R^T for the row solve.
constexpr int kQRPitch = kQRMaxRank + 1;

__global__ void __launch_bounds__(256) k_qr_solve(QRArgs args) {
  static_assert(kQRMaxRank == 64 && kQRRows == 64, "4 x 4 slots of stride 16; four threads per row");
  const QRMode M = args.m[blockIdx.y];
  const int c = blockIdx.x;
  const int row0 = c * kQRRows;
  if (c >= M.nchunk || row0 >= M.a || M.r > kQRMaxRank) return;
  __shared__ double Rt[kQRMaxRank * kQRPitch];      // Rt[k][j] = R[j][k], k > j
  __shared__ double rowbuf[2][kQRMaxRank];          // pivot row of step j in rowbuf[j & 1]
  __shared__ double pub[2][kQRRows];                  // v_j of each row in pub[j & 1]
  __shared__ double Rinv[kQRMaxRank];               // 1 / R[j][j]
  __shared__ double s_trace;
  const int tid = threadIdx.x;
  const int r = M.r;
  const int ti = tid >> 4, tj = tid & 15;             // slot (x, y) of a thread is G[ti + 16x][tj + 16y]

  // The rows of P this CTA solves: four threads per row, thread ql holds columns ql, ql + 4, ...
  const int rowl = tid >> 2, ql = tid & 3;
  const int row = row0 + rowl;
  const bool live = row < M.a;                        // rows past the end are solved as zeros, unstored
  double v[kQRMaxRank / 4];
  {
    const double* prow = M.Pred + (int64_t)(live ? row : 0) * r;
#pragma unroll
    for (int t = 0; t < kQRMaxRank / 4; ++t) {
      const int k = ql + 4 * t;
      v[t] = __ldcg(prow + (k < r ? k : 0));         // unconditional, selected afterwards
    }
#pragma unroll
    for (int t = 0; t < kQRMaxRank / 4; ++t)
      if (!(live && ql + 4 * t < r)) v[t] = 0.0;
  }
  // G = sum of the row chunks' shares, chunk by chunk in order (upper triangle).
  double g[4][4];
#pragma unroll
  for (int x = 0; x < 4; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) g[x][y] = 0.0;
  const int nsum = args.gsum ? 1 : M.nchunk;          // share 0 already holds the total
  for (int cc = 0; cc < nsum; cc += 2) {              // two chunks' loads in flight, added in order
    const double* Gc = M.Gp + (int64_t)cc * r * r;
    const bool two = cc + 1 < nsum;
    double t0[4][4], t1[4][4];
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        const int i = ti + 16 * x, k = tj + 16 * y;
        const bool on = k < r && k >= i;
        const int o = on ? i * r + k : 0;
        t0[x][y] = __ldcg(Gc + o);                   // unconditional loads, selected afterwards
        t1[x][y] = __ldcg(Gc + (two ? r * r : 0) + o);
      }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        const int i = ti + 16 * x, k = tj + 16 * y;
        const bool on = k < r && k >= i;
        g[x][y] = (g[x][y] + (on ? t0[x][y] : 0.0)) + ((on && two) ? t1[x][y] : 0.0);
      }
  }
  // Diagonal -> trace; row 0 -> the first pivot row.
#pragma unroll
  for (int x = 0; x < 4; ++x)
    if (ti == tj && ti + 16 * x < r) Rinv[ti + 16 * x] = g[x][x];
  if (ti == 0) {
#pragma unroll
    for (int y = 0; y < 4; ++y)
      if (tj + 16 * y < r) rowbuf[0][tj + 16 * y] = g[0][y];
  }
  if (ql == 0) pub[0][rowl] = v[0];
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int i = 0; i < r; ++i) t += Rinv[i];
    s_trace = t;
  }
  __syncthreads();
  const double floor_d = 1e-12 * s_trace;
  // Right-looking Cholesky, one barrier per column.  Step j reads the pivot row (row j of the
  // Schur complement), updates the rows below it in registers, hands row j + 1 to the next step
  // and leaves R[j][k] = G[j][k] / R[j][j] in Rt.
  for (int j = 0; j < r; ++j) {
    const double* rb = rowbuf[j & 1];
    double* nb = rowbuf[(j + 1) & 1];
    double d = rb[j];
    if (!(d > floor_d)) {
      if (tid == 0 && c == 0) atomicMax(args.status, (int)ASI_ERR_RANK_DEFICIENT);
      d = (floor_d > 0.0) ? floor_d : 1.0;
    }
    const double inv = rsqrt(d);
    double ai[4], bk[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int i = ti + 16 * t, k = tj + 16 * t;
      ai[t] = (i > j && i < r) ? rb[i] * inv : 0.0;
      bk[t] = (k > j && k < r) ? rb[k] * inv : 0.0;
    }
#pragma unroll
    for (int x = 0; x < 4; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        const int i = ti + 16 * x, k = tj + 16 * y;
        g[x][y] = fma(-ai[x], bk[y], g[x][y]);       // ai, bk are 0 outside the trailing block
        if (i == j + 1 && k >= i && k < r) nb[k] = g[x][y];
      }
    if (tid > j && tid < r) Rt[tid * kQRPitch + j] = rb[tid] * inv;
    if (tid == 0) Rinv[j] = inv;
    __syncthreads();
  }
  // U = P R^{-1}, row by row: q_j = v_j / R[j][j], then v_k -= q_j R[j][k] for k > j.  The four
  // threads of a row sit in one warp; every lane takes every step (the warp barriers are
  // unconditional), and the thread that owns column j + 1 hands v_{j+1} to the next step.
  for (int j = 0; j < r; ++j) {
    double rt[kQRMaxRank / 4];
#pragma unroll
    for (int t = 0; t < kQRMaxRank / 4; ++t) {
      const int k = ql + 4 * t;
      rt[t] = (k > j && k < r) ? Rt[k * kQRPitch + j] : 0.0;
    }
    const double q = pub[j & 1][rowl] * Rinv[j];
    double* np = pub[(j + 1) & 1];
#pragma unroll
    for (int t = 0; t < kQRMaxRank / 4; ++t) {
      const int k = ql + 4 * t;
      v[t] = (k == j) ? q : fma(-q, rt[t], v[t]);     // rt = 0 leaves the solved and the unused columns alone
      if (k == j + 1 && k < r) np[rowl] = v[t];
    }
    __syncwarp();
  }
  if (live) {
    float* urow = M.Uout + (int64_t)row * r;
#pragma unroll
    for (int t = 0; t < kQRMaxRank / 4; ++t) {
      const int k = ql + 4 * t;
      if (k < r) urow[k] = (float)v[t];
    }
  }
}

cudaError_t launch_qr_solve(const QRArgs& p, int nd, int max_chunks, cudaStream_t st) {
  dim3 grid((unsigned)max_chunks, (unsigned)nd);
  k_qr_solve<<<grid, 256, 0, st>>>(p);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Orthogonalize for ranks 65..128: the same Cholesky-QR in fp64 in plain kernels (these ranks are rare
// and the matrices small: a x r with r <= 128).  k_qrb_reduce sums the column-split partials in split
// order, k_qrb_gram forms G = P^T P (one thread per entry of the upper triangle, rows in order),
// k_qrb_chol factors G = R^T R in one CTA (shared memory), k_qrb_solve solves u R = p one row per thread.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_qrb_reduce(QRArgs args) {
  const QRMode M = args.m[blockIdx.y];
  if (M.r <= kQRMaxRank) return;
  const int64_t n = (int64_t)M.a * M.r;
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < n; e += (int64_t)gridDim.x * 256) {
    double acc = 0.0;
    for (int s0 = 0; s0 < M.nsplit; s0 += 8) {
      float t[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) t[q] = __ldcg(M.Pp + (int64_t)((s0 + q < M.nsplit) ? (s0 + q) : 0) * n + e);
#pragma unroll
      for (int q = 0; q < 8; ++q) acc += (s0 + q < M.nsplit) ? (double)t[q] : 0.0;
    }
    M.Pred[e] = acc;
  }
}

__global__ void __launch_bounds__(256) k_qrb_gram(QRArgs args) {
  const QRMode M = args.m[blockIdx.y];
  const int r = M.r;
  if (r <= kQRMaxRank) return;
  const int e = blockIdx.x * 256 + threadIdx.x;
  if (e >= r * r) return;
  const int i = e / r, j = e - i * r;
  if (j < i) return;
  double g = 0.0;
#pragma unroll 4
  for (int k = 0; k < M.a; ++k) g = fma(__ldcg(M.Pred + (int64_t)k * r + i), __ldcg(M.Pred + (int64_t)k * r + j), g);
  M.Gp[e] = g;
}

__global__ void __launch_bounds__(1024) k_qrb_chol(QRArgs args) {
  extern __shared__ double qb_G[];                 // [r][r + 1]
  __shared__ double s_d;
  const QRMode M = args.m[blockIdx.x];
  const int r = M.r, tid = threadIdx.x, P = r + 1;
  if (r <= kQRMaxRank) return;
  for (int e = tid; e < r * r; e += 1024) {
    const int i = e / r, j = e - i * r;
    qb_G[i * P + j] = (j >= i) ? M.Gp[e] : 0.0;
  }
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int i = 0; i < r; ++i) t += qb_G[i * P + i];
    s_d = 1e-12 * t;
  }
  __syncthreads();
  const double floor_d = s_d;
  for (int j = 0; j < r; ++j) {
    double d = qb_G[j * P + j];
    if (!(d > floor_d)) {
      if (tid == 0) atomicMax(args.status, (int)ASI_ERR_RANK_DEFICIENT);
      d = (floor_d > 0.0) ? floor_d : 1.0;
    }
    const double inv = rsqrt(d);
    __syncthreads();
    for (int k = j + tid; k < r; k += 1024) qb_G[j * P + k] = (k == j) ? d * inv : qb_G[j * P + k] * inv;
    __syncthreads();
    const int nrem = r - j - 1;
    for (int e = tid; e < nrem * nrem; e += 1024) {
      const int i = j + 1 + e / nrem, k = j + 1 + e % nrem;
      if (k >= i) qb_G[i * P + k] -= qb_G[j * P + i] * qb_G[j * P + k];
    }
    __syncthreads();
  }
  for (int e = tid; e < r * r; e += 1024) {
    const int i = e / r, j = e - i * r;
    M.Gp[e] = (j >= i) ? qb_G[i * P + j] : 0.0;    // R, upper triangular
  }
}

__global__ void __launch_bounds__(128) k_qrb_solve(QRArgs args) {
  extern __shared__ double qb_R[];                 // [r][r]
  const QRMode M = args.m[blockIdx.y];
  const int r = M.r;
  if (r <= kQRMaxRank) return;
  for (int e = threadIdx.x; e < r * r; e += 128) qb_R[e] = M.Gp[e];
  __syncthreads();
  const int row = blockIdx.x * 128 + threadIdx.x;
  if (row >= M.a) return;
  double u[2 * kQRMaxRank];
  const double* prow = M.Pred + (int64_t)row * r;
  for (int j = 0; j < r; ++j) {
    double s = prow[j];
    for (int i = 0; i < j; ++i) s = fma(-u[i], qb_R[i * r + j], s);
    u[j] = s / qb_R[j * r + j];
  }
  float* urow = M.Uout + (int64_t)row * r;
  for (int j = 0; j < r; ++j) urow[j] = (float)u[j];
}

static cudaError_t launch_qr_big(const QRArgs& p, int nd, cudaStream_t st) {
  int amax = 1, rmax = 1;
  for (int m = 0; m < nd; ++m)
    if (p.m[m].r > kQRMaxRank) {
      amax = std::max(amax, p.m[m].a);
      rmax = std::max(rmax, p.m[m].r);
    }
  k_qrb_reduce<<<dim3(64, (unsigned)nd), 256, 0, st>>>(p);
  k_qrb_gram<<<dim3((unsigned)((rmax * rmax + 255) / 256), (unsigned)nd), 256, 0, st>>>(p);
  const size_t chol_smem = (size_t)rmax * (rmax + 1) * sizeof(double), solve_smem = (size_t)rmax * rmax * sizeof(double);
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_qrb_chol), chol_smem);
  if (e == cudaSuccess) e = opt_in_smem(reinterpret_cast<const void*>(k_qrb_solve), solve_smem);
  if (e != cudaSuccess) return e;
  k_qrb_chol<<<nd, 1024, chol_smem, st>>>(p);
  k_qrb_solve<<<dim3((unsigned)((amax + 127) / 128), (unsigned)nd), 128, solve_smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_qr(const QRArgs& p, int nd, int max_chunks, cudaStream_t st) {
  double qr_bytes = 0.0;
  for (int m = 0; m < nd; ++m)
    qr_bytes += 4.0 * p.m[m].a * p.m[m].r * (p.m[m].nsplit + 1);
  ProfScope prof(ASI_K_QR, st, qr_bytes);
  dim3 grid((unsigned)max_chunks, (unsigned)nd);
  k_qr_gram<<<grid, 256, 0, st>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  k_qr_gsum<<<dim3(kQRMaxRank * kQRMaxRank / 256, (unsigned)nd), 256, 0, st>>>(p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  QRArgs q = p;
  q.gsum = 1;
  k_qr_solve<<<grid, 256, 0, st>>>(q);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  for (int m = 0; m < nd; ++m)
    if (p.m[m].r > kQRMaxRank) return launch_qr_big(p, nd, st);
  return cudaSuccess;
}

// ---------------------------------------------------------------------------------------------
// k_conv_tail: one CTA per output channel c'.  Thread (o, s): output o = (j, kh, kw) of Z4 and
// split s of the reduction over (i, h'); partial sums meet in shared memory in a fixed order.
// Then dW[c', :, :, :] = Z4[c'] x_2 U2 over the channels of c''s group.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_conv_tail(ConvTailArgs p) {
  extern __shared__ float sm[];
  const int tid = threadIdx.x;
  const int co = blockIdx.x;
  const int kk = p.kh * p.kw;
  const int n_out = p.r2 * kk;
  float* Z4s = sm;                       // [n_out]
  float* red = sm + ((n_out + 31) / 32) * 32;   // [nsplit][n_out] when nsplit > 1

  int nsplit = (n_out <= 128) ? 256 / n_out : 1;
  const int n_items = p.r1 * p.Ho;
  if (nsplit > n_items) nsplit = n_items;
  if (nsplit < 1) nsplit = 1;

  if (nsplit > 1) {
    const int o = tid % n_out, s = tid / n_out;
    if (s < nsplit) {
      const int j = o / kk, t = o % kk, ky = t / p.kw, kx = t % p.kw;
      float acc = 0.f;
      for (int it = s; it < n_items; it += nsplit) {
        const int i = it / p.Ho, ho = it % p.Ho;
        const int h = ho * p.sh + ky - p.ph;
        if (h < 0 || h >= p.H) continue;
        const float* z1 = p.Z1 + (((int64_t)i * p.Cout + co) * p.Ho + ho) * p.Wo;
        const float* z3 = p.Z3 + (((int64_t)i * p.r2 + j) * p.H + h) * p.W;
        for (int wo = 0; wo < p.Wo; ++wo) {
          const int w = wo * p.sw + kx - p.pw;
          if (w >= 0 && w < p.W) acc = fmaf(z1[wo], z3[w], acc);
        }
      }
      red[s * n_out + o] = acc;
    }
    __syncthreads();
    if (tid < n_out) {
      float v = 0.f;
      for (int s = 0; s < nsplit; ++s) v += red[s * n_out + tid];
      Z4s[tid] = v;
    }
  } else {
    for (int o = tid; o < n_out; o += 256) {
      const int j = o / kk, t = o % kk, ky = t / p.kw, kx = t % p.kw;
      float acc = 0.f;
      for (int it = 0; it < n_items; ++it) {
        const int i = it / p.Ho, ho = it % p.Ho;
        const int h = ho * p.sh + ky - p.ph;
        if (h < 0 || h >= p.H) continue;
        const float* z1 = p.Z1 + (((int64_t)i * p.Cout + co) * p.Ho + ho) * p.Wo;
        const float* z3 = p.Z3 + (((int64_t)i * p.r2 + j) * p.H + h) * p.W;
        for (int wo = 0; wo < p.Wo; ++wo) {
          const int w = wo * p.sw + kx - p.pw;
          if (w >= 0 && w < p.W) acc = fmaf(z1[wo], z3[w], acc);
        }
      }
      Z4s[o] = acc;
    }
  }
  __syncthreads();
  const int cg = p.C / p.groups, og = p.Cout / p.groups;
  const int g = co / og;
  float* dw = p.dW + (int64_t)co * cg * kk;
  for (int idx = tid; idx < cg * kk; idx += 256) {
    const int cl = idx / kk, t = idx % kk;
    const float* u = p.U2 + (int64_t)(g * cg + cl) * p.r2;
    float v = 0.f;
    for (int j = 0; j < p.r2; ++j) v = fmaf(Z4s[j * kk + t], u[j], v);
    dw[idx] = v;
  }
}

// ---------------------------------------------------------------------------------------------
// Terms 4 and 5 for large output maps, in two launches so the long reduction over (i, h', w') is
// spread over Cout x nsp CTAs: k_conv_z4 writes nsp partial Z4 per output channel (CTA (c', sp)
// takes the pairs (i, h') == sp (mod nsp); thread (o, g) every G-th of those), k_conv_dw sums them in
// order and expands with U2.  Loop bounds are computed per tap, so the inner loops carry no branch.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_conv_z4(ConvTailArgs p, float* __restrict__ Z4p, int nsp) {
  extern __shared__ float sm[];
  const int tid = threadIdx.x;
  const int co = blockIdx.x, sp = blockIdx.y;
  const int kk = p.kh * p.kw;
  const int n_out = p.r2 * kk;
  const int G = (n_out <= 256) ? 256 / n_out : 1;
  float* red = sm;                                  // [G][n_out]
  const int n_items = p.r1 * p.Ho;
  for (int t = tid; t < n_out * G; t += 256) {
    const int o = t % n_out, g = t / n_out;
    const int j = o / kk, tt = o % kk, ky = tt / p.kw, kx = tt % p.kw;
    int wo_lo = (p.pw - kx > 0) ? (p.pw - kx + p.sw - 1) / p.sw : 0;
    int wo_hi = (p.W - 1 + p.pw - kx >= 0) ? (p.W - 1 + p.pw - kx) / p.sw + 1 : 0;
    if (wo_hi > p.Wo) wo_hi = p.Wo;
    float acc0 = 0.f, acc1 = 0.f;
    for (int it = sp + nsp * g; it < n_items; it += nsp * G) {
      const int i = it / p.Ho, ho = it - i * p.Ho;
      const int h = ho * p.sh + ky - p.ph;
      if (h < 0 || h >= p.H) continue;
      const float* z1 = p.Z1 + (((int64_t)i * p.Cout + co) * p.Ho + ho) * p.Wo;
      const float* z3 = p.Z3 + (((int64_t)i * p.r2 + j) * p.H + h) * p.W + kx - p.pw;
      int wo = wo_lo;
#pragma unroll 4
      for (; wo + 1 < wo_hi; wo += 2) {
        acc0 = fmaf(__ldg(z1 + wo), __ldg(z3 + wo * p.sw), acc0);
        acc1 = fmaf(__ldg(z1 + wo + 1), __ldg(z3 + (wo + 1) * p.sw), acc1);
      }
      if (wo < wo_hi) acc0 = fmaf(__ldg(z1 + wo), __ldg(z3 + wo * p.sw), acc0);
    }
    red[g * n_out + o] = acc0 + acc1;
  }
  __syncthreads();
  for (int o = tid; o < n_out; o += 256) {
    float v = 0.f;
    for (int g = 0; g < G; ++g) v += red[g * n_out + o];
    Z4p[((int64_t)sp * p.Cout + co) * n_out + o] = v;
  }
}

__global__ void __launch_bounds__(256) k_conv_dw(ConvTailArgs p, const float* __restrict__ Z4p, int nsp) {
  extern __shared__ float sm[];
  const int tid = threadIdx.x;
  const int co = blockIdx.x;
  const int kk = p.kh * p.kw;
  const int n_out = p.r2 * kk;
  float* Z4s = sm;
  for (int o = tid; o < n_out; o += 256) {
    float v = 0.f;
    for (int s = 0; s < nsp; ++s) v += Z4p[((int64_t)s * p.Cout + co) * n_out + o];
    Z4s[o] = v;
  }
  __syncthreads();
  const int cg = p.C / p.groups, og = p.Cout / p.groups;
  const int g = co / og;
  float* dw = p.dW + (int64_t)co * cg * kk;
  for (int idx = tid; idx < cg * kk; idx += 256) {
    const int cl = idx / kk, t = idx % kk;
    const float* u = p.U2 + (int64_t)(g * cg + cl) * p.r2;
    float v = 0.f;
    for (int j = 0; j < p.r2; ++j) v = fmaf(Z4s[j * kk + t], u[j], v);
    dw[idx] = v;
  }
}

cudaError_t launch_conv_tail_split(const ConvTailArgs& p, float* Z4p, int nsp, cudaStream_t st) {
  ProfScope prof(ASI_K_CONV_TAIL, st,
                 4.0 * ((double)p.r1 * p.Cout * p.Ho * p.Wo + (double)p.r1 * p.r2 * p.H * p.W +
                        (double)p.C * p.r2 + (double)p.Cout * (p.C / p.groups) * p.kh * p.kw));
  const int n_out = p.r2 * p.kh * p.kw;
  const int G = (n_out <= 256) ? 256 / n_out : 1;
  const size_t smem = (size_t)G * n_out * sizeof(float);
  cudaError_t e = cudaSuccess;
  if (smem > 40 * 1024) {
    e = opt_in_smem(reinterpret_cast<const void*>(k_conv_z4), smem);
    if (e == cudaSuccess) e = opt_in_smem(reinterpret_cast<const void*>(k_conv_dw), smem);
    if (e != cudaSuccess) return e;
  }
  k_conv_z4<<<dim3(p.Cout, nsp), 256, smem, st>>>(p, Z4p, nsp);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  k_conv_dw<<<p.Cout, 256, (size_t)n_out * sizeof(float), st>>>(p, Z4p, nsp);
  return cudaGetLastError();
}

size_t conv_tail_smem(int r2, int kh, int kw) {
  const int n_out = r2 * kh * kw;
  const int nsplit_max = (n_out <= 128) ? 256 / n_out : 1;
  const int G = (n_out <= 256) ? 256 / n_out : 1;            // k_conv_z4
  const size_t tail = (size_t)(((n_out + 31) / 32) * 32 + (size_t)nsplit_max * n_out) * sizeof(float);
  const size_t z4 = (size_t)G * n_out * sizeof(float);
  return tail > z4 ? tail : z4;
}

cudaError_t launch_conv_tail(const ConvTailArgs& p, cudaStream_t st) {
  ProfScope prof(ASI_K_CONV_TAIL, st,
                 4.0 * ((double)p.r1 * p.Cout * p.Ho * p.Wo + (double)p.r1 * p.r2 * p.H * p.W +
                        (double)p.C * p.r2 + (double)p.Cout * (p.C / p.groups) * p.kh * p.kw));
  const size_t smem = conv_tail_smem(p.r2, p.kh, p.kw);
  if (smem > 40 * 1024) {
    cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_conv_tail), smem);
    if (e != cudaSuccess) return e;
  }
  k_conv_tail<<<p.Cout, 256, smem, st>>>(p);
  return cudaGetLastError();
}

}  // namespace asi
