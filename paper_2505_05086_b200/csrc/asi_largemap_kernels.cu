// Streaming kernels for large feature maps and long token tensors (ranks <= 4 per mode): the two products
// of a mode, V_m = A_m^T U_m and P_m = A_m V_m (Algorithm 1), in one pass over the activation with
// register-tiled inner loops on packed fp32 pairs (fma.rn.f32x2: one instruction, two multiply-adds).
//
//   k_fiber2   : one mode with a_m <= 128 whose fibers are strided (not the last mode).  A tile is all a_m
//                rows of 128 neighbouring columns of the unfolding.  Warp w owns rows [w RW, w RW + RW), lane l
//                owns the four columns 4l..4l+3, in both products:
//                  projection   V[q][:]  = sum_k X[k][q] U[k][:]     partial over the warp's rows, the 16
//                                                                    partials meet in shared memory in order
//                  expansion    P[k][:] += sum_q X[k][q] V[q][:]     partial over the lane's columns, kept in
//                                                                    registers across all tiles of the CTA
//                With `project_only` the kernel stops after the projection and writes V: that is the mode
//                product Y = X x_m U^T of the first core step and of Z1 = dY x_1 U_1^T (C_ASI term 1).
//   k_plane2   : the two spatial modes of a conv activation with S x S planes, S = 28 or 56, in one pass over
//                whole planes: the column pass (contract h) gives V_3 and P_4, the row pass (contract w)
//                gives V_4 and P_3.
// Operand pairs are laid out so that no packing moves are needed: a 16-byte read of four neighbouring
// values of a row is two pairs; the factor they meet is stored either with every entry duplicated
// ((u,u): both halves of a pair take the same factor entry) or transposed ([j][q]: the pair holds the
// entries of the two columns, and the two halves of the accumulator are added at the end).
#include <cuda_bf16.h>

#include <algorithm>
#include <type_traits>

#include "asi_internal.h"

namespace asi {

namespace {

typedef unsigned long long f2;     // two packed fp32 values (lo, hi)

__device__ __forceinline__ f2 pack2(float lo, float hi) {
  f2 r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack2(f2 v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ float fold2(f2 v) {
  float lo, hi;
  unpack2(v, lo, hi);
  return lo + hi;
}
__device__ __forceinline__ f2 fadd2(f2 a, f2 b) {
  f2 r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ void ffma2(f2& d, f2 a, f2 b) {       // d += a * b on both halves
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d) : "l"(a), "l"(b));
}
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
// 16 bytes global -> shared, or 16 zero bytes when `on` is false
__device__ __forceinline__ void cp_async16(void* dst, const void* src, bool on) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(on ? 16 : 0)
               : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// four neighbouring values of a staged row as two packed pairs
template <typename TX>
__device__ __forceinline__ void ld_quad(const TX* p, f2& a, f2& b);
template <>
__device__ __forceinline__ void ld_quad<float>(const float* p, f2& a, f2& b) {
  const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(p);
  a = v.x;
  b = v.y;
}
template <>
__device__ __forceinline__ void ld_quad<__nv_bfloat16>(const __nv_bfloat16* p, f2& a, f2& b) {
  const uint2 w = *reinterpret_cast<const uint2*>(p);
  a = pack2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u));
  b = pack2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u));
}

constexpr int kF2Threads = 256, kF2Groups = 16, kF2TQ = 64;   // 16 half-warps: one row group each

}  // namespace

// ---------------------------------------------------------------------------------------------
// k_fiber2.  256 threads = 16 half-warps; half-warp g owns rows [g RW, g RW + RW) of the tile, its lane l the
// four columns 4l..4l+3 (a tile is 64 columns wide).  Two or three CTAs share an SM and every CTA keeps one
// further tile in flight (16-byte cp.async).
// ---------------------------------------------------------------------------------------------
template <int RW, int NJ, typename TX>
__global__ void __launch_bounds__(kF2Threads, (RW <= 4 && NJ == 4) ? 3 : 2) k_fiber2(Fiber2Args p) {
  constexpr int TQ = kF2TQ, NT = kF2Threads, NG = kF2Groups;
  constexpr int EPU = 16 / (int)sizeof(TX);          // elements per 16-byte unit
  constexpr int UPR = TQ / EPU;                      // units per staged row
  extern __shared__ __align__(128) unsigned char f2_smem[];
  const int tid = threadIdx.x, grp = tid >> 4, lane = tid & 15;
  const int a = p.a, r = p.r, nst = p.nstage;
  constexpr int AR = NG * RW;                        // staged rows: rows a..AR-1 stay zero, so no loop tests k < a
  constexpr size_t stage_bytes = (size_t)AR * TQ * sizeof(TX);
  unsigned char* stages = f2_smem;
  f2* Ud = reinterpret_cast<f2*>(f2_smem + (size_t)nst * stage_bytes);   // [AR][NJ]: (u, u)
  float* Vp = reinterpret_cast<float*>(Ud + (size_t)AR * NJ);            // [NG / 2][NJ][TQ]
  float* Vt = Vp + (NG / 2) * NJ * TQ;                                   // [NJ][TQ]
  for (int idx = tid; idx < AR * NJ; idx += NT) {
    const int k = idx / NJ, j = idx % NJ;
    const float u = (k < a && j < r) ? p.U[k * p.ldu + j] : 0.f;
    Ud[idx] = pack2(u, u);
  }
  if (a < AR) {
    for (int s = 0; s < nst; ++s) {
      uint32_t* z = reinterpret_cast<uint32_t*>(stages + (size_t)s * stage_bytes + (size_t)a * TQ * sizeof(TX));
      for (int idx = tid; idx < (int)((AR - a) * TQ * sizeof(TX) / 4); idx += NT) z[idx] = 0u;
    }
  }
  __syncthreads();
  const TX* __restrict__ X = reinterpret_cast<const TX*>(p.X);
  const int tpo = (int)((p.I + TQ - 1) / TQ);        // tiles per outer index (< 2^31: checked on the host)
  const int nt = (int)p.n_tiles, gs = (int)gridDim.x;

  // A thread copies the same 16-byte unit of every KSTEP-th row: unit u of rows k0, k0 + KSTEP, ...
  constexpr int KSTEP = NT / UPR;
  const int cu = tid % UPR, ck0 = tid / UPR;
  const int64_t src_row_step = (int64_t)KSTEP * p.I;
  auto issue = [&](int o, int ic, int st) {
    const int64_t i0 = (int64_t)ic * TQ;
    const int ncol = (int)((p.I - i0 < TQ) ? (p.I - i0) : TQ);
    const bool on = cu * EPU < ncol;
    const TX* src = X + ((int64_t)o * a + ck0) * p.I + i0 + (on ? cu * EPU : 0);
    TX* dst = reinterpret_cast<TX*>(stages + (size_t)st * stage_bytes) + ck0 * TQ + cu * EPU;
    for (int k = ck0; k < a; k += KSTEP) {
      cp_async16(dst, src, on);
      src += src_row_step;
      dst += KSTEP * TQ;
    }
  };
  // (o, ic) of a tile index advance by gs tiles at a time without divisions
  const int step_o = gs / tpo, step_i = gs - step_o * tpo;
  auto advance = [&](int& o, int& ic) {
    o += step_o;
    ic += step_i;
    if (ic >= tpo) {
      ic -= tpo;
      ++o;
    }
  };

  f2 accP[RW][NJ];
#pragma unroll
  for (int i = 0; i < RW; ++i)
#pragma unroll
    for (int j = 0; j < NJ; ++j) accP[i][j] = 0ull;

  // prologue: nst - 1 tiles in flight
  int t_issue = blockIdx.x;
  int io = (int)blockIdx.x / tpo, ii = (int)blockIdx.x - io * tpo;   // tile being issued
  int co = io, ci = ii;                                              // tile being computed
  for (int s = 0; s < nst - 1; ++s) {
    if (t_issue < nt) issue(io, ii, s);
    cp_commit();
    t_issue += gs;
    advance(io, ii);
  }
  int st = 0;
  for (int t = blockIdx.x; t < nt; t += gs) {
    // one group is committed per iteration, so all but the newest nst - 2 groups are complete
    // exactly when the tile about to be used has landed
    if (nst == 2) cp_wait<0>();
    else if (nst == 3) cp_wait<1>();
    else cp_wait<2>();
    __syncthreads();
    {
      // refill the stage freed by the previous iteration; its group is waited for nst - 1 iterations later
      int sf = st + nst - 1;
      if (sf >= nst) sf -= nst;
      if (t_issue < nt) issue(io, ii, sf);
      cp_commit();
      t_issue += gs;
      advance(io, ii);
    }
    const TX* Xs = reinterpret_cast<const TX*>(stages + (size_t)st * stage_bytes);
    // ---- projection: partial V over this half-warp's rows
    f2 accV[NJ][2];
#pragma unroll
    for (int j = 0; j < NJ; ++j) accV[j][0] = accV[j][1] = 0ull;
#pragma unroll
    for (int i = 0; i < RW; ++i) {
      const int k = grp * RW + i;
      f2 x01, x23;
      ld_quad<TX>(Xs + k * TQ + 4 * lane, x01, x23);
#pragma unroll
      for (int j = 0; j < NJ; j += 2) {
        const ulonglong2 u = *reinterpret_cast<const ulonglong2*>(Ud + k * NJ + j);
        ffma2(accV[j][0], x01, u.x); ffma2(accV[j][1], x23, u.x);
        ffma2(accV[j + 1][0], x01, u.y); ffma2(accV[j + 1][1], x23, u.y);
      }
    }
    // the two half-warps of a warp (same columns, neighbouring row groups) meet by one shuffle
#pragma unroll
    for (int j = 0; j < NJ; ++j)
#pragma unroll
      for (int h = 0; h < 2; ++h) accV[j][h] = fadd2(accV[j][h], __shfl_xor_sync(0xffffffffu, accV[j][h], 16));
    if ((tid & 16) == 0) {
#pragma unroll
      for (int j = 0; j < NJ; ++j)
        *reinterpret_cast<ulonglong2*>(Vp + ((grp >> 1) * NJ + j) * TQ + 4 * lane) = make_ulonglong2(accV[j][0], accV[j][1]);
    }
    __syncthreads();
    {
      // the eight partials meet in warp order: Vt[j][q]
#pragma unroll
      for (int e = tid; e < NJ * TQ; e += NT) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < NG / 2; ++w) s += Vp[w * NJ * TQ + e];
        Vt[e] = s;
      }
    }
    __syncthreads();
    if (p.project_only) {
      // Y[j][o, i0 + q] = V[q][j]
      const int64_t o = co, i0 = (int64_t)ci * TQ;
      const int ncol = (int)((p.I - i0 < TQ) ? (p.I - i0) : TQ);
      for (int idx = tid; idx < r * (TQ / 4); idx += NT) {
        const int j = idx / (TQ / 4), v = idx - j * (TQ / 4);
        if (4 * v < ncol)
          *reinterpret_cast<float4*>(p.Y + o * p.y_so + (int64_t)j * p.y_sj + i0 + 4 * v) =
              *reinterpret_cast<const float4*>(Vt + j * TQ + 4 * v);
      }
    } else {
      // ---- expansion: P[k][:] += sum over this lane's columns
      f2 vt[NJ][2];
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(Vt + j * TQ + 4 * lane);
        vt[j][0] = v.x;
        vt[j][1] = v.y;
      }
#pragma unroll
      for (int i = 0; i < RW; ++i) {
        const int k = grp * RW + i;
        f2 x01, x23;
        ld_quad<TX>(Xs + k * TQ + 4 * lane, x01, x23);
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
          ffma2(accP[i][j], x01, vt[j][0]);
          ffma2(accP[i][j], x23, vt[j][1]);
        }
      }
    }
    st = (st + 1 == nst) ? 0 : st + 1;
    advance(co, ci);
  }
  cp_wait<0>();
  if (p.project_only) return;
  // the 16 lanes of a row group meet by shuffles in a fixed order; one partial of P per CTA
#pragma unroll
  for (int i = 0; i < RW; ++i) {
    const int k = grp * RW + i;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      float v = fold2(accP[i][j]);
#pragma unroll
      for (int off = 8; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
      if (lane == 0 && k < a && j < r) p.Pp[((int64_t)blockIdx.x * a + k) * r + j] = v;
    }
  }
}

size_t fiber2_smem(int a, int rw, int nj, int nstage, bool bf16) {
  (void)a;
  return (size_t)nstage * kF2Groups * rw * kF2TQ * (bf16 ? 2 : 4) + (size_t)kF2Groups * rw * nj * 8 +
         (size_t)(kF2Groups / 2 + 1) * nj * kF2TQ * 4;
}

int fiber2_rows_per_group(int a) {
  const int rw = (a + kF2Groups - 1) / kF2Groups;
  return rw <= 1 ? 1 : (rw <= 2 ? 2 : (rw <= 4 ? 4 : 8));
}

// as many stages (2..4) as leave room for two CTAs per SM
// CTAs per SM the kernel is compiled for: three when the row accumulators are small (78 registers), else two
int fiber2_ctas_per_sm(int rw, int nj) { return (rw <= 4 && nj == 4) ? 3 : 2; }

// Two stages: one tile in flight per CTA while the other is used.  Deeper pipelines (3-4 stages) ran the kernel
// alone no faster, and their larger footprint kept other kernels of the same step off the SMs: the step of ten
// layers replayed as a graph was 2 % slower with them.
int fiber2_stages(int a, int nj, bool bf16) {
  (void)a; (void)nj; (void)bf16;
  return 2;
}

// ranks up to 4 for a <= 128, up to 8 for a <= 64 (the register budget of the row accumulators)
bool fiber2_supported(int64_t O, int64_t a, int64_t I, int r, bool bf16) {
  (void)O;
  return r <= 8 && a >= 2 && a <= (r <= 4 ? 128 : 64) && I >= kF2TQ && I % (bf16 ? 8 : 4) == 0 &&
         O * ((I + kF2TQ - 1) / kF2TQ) < (1ll << 30);
}

int64_t fiber2_tiles(int64_t O, int64_t I) { return O * ((I + kF2TQ - 1) / kF2TQ); }

// CTAs (= partials of P) of the kernel launch_fiber2 picks: the register kernel for short fibers
// share_sm: the variant that fills an SM's registers with two CTAs launches one per SM (other layers' kernels
// are expected beside it)
int fiber2_grid(int64_t O, int64_t a, int64_t I, int r, bool bf16, bool share_sm) {
  if (fiber_reg_supported(O, a, I, r, bf16)) return fiber_reg_grid(O, a, I, r, bf16);
  int per_sm = fiber2_ctas_per_sm(fiber2_rows_per_group((int)a), r <= 4 ? 4 : 8);
  if (share_sm && per_sm == 2) per_sm = 1;
  return (int)std::min<int64_t>(fiber2_tiles(O, I), 148 * per_sm);
}

template <int RW, int NJ, typename TX>
static cudaError_t launch_fiber2_t(const Fiber2Args& p, int grid, size_t smem, cudaStream_t st) {
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_fiber2<RW, NJ, TX>), smem);
  if (e != cudaSuccess) return e;
  k_fiber2<RW, NJ, TX><<<grid, kF2Threads, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_fiber2(const Fiber2Args& p0, int grid, bool bf16, cudaStream_t st) {
  Fiber2Args p = p0;
  if (fiber_reg_supported(p.O, p.a, p.I, p.r, bf16)) return launch_fiber_reg(p, grid, bf16, st);
  const int rw = fiber2_rows_per_group(p.a), nj = p.r <= 4 ? 4 : 8;
  p.nstage = fiber2_stages(p.a, nj, bf16);
  const size_t smem = fiber2_smem(p.a, rw, nj, p.nstage, bf16);
  const double xbytes = (double)p.O * p.a * p.I * (bf16 ? 2 : 4);
  ProfScope prof(p.project_only ? ASI_K_MODEPROD : ASI_K_EXPAND, st, xbytes);
#define ASI_F2(RW_, NJ_)                                                                        \
  return bf16 ? launch_fiber2_t<RW_, NJ_, __nv_bfloat16>(p, grid, smem, st) : launch_fiber2_t<RW_, NJ_, float>(p, grid, smem, st)
  if (nj == 4) {
    switch (rw) {
      case 1: ASI_F2(1, 4);
      case 2: ASI_F2(2, 4);
      case 4: ASI_F2(4, 4);
      default: ASI_F2(8, 4);
    }
  }
  switch (rw) {
    case 1: ASI_F2(1, 8);
    case 2: ASI_F2(2, 8);
    default: ASI_F2(4, 8);
  }
#undef ASI_F2
}

// ---------------------------------------------------------------------------------------------
// k_plane2<S>: G = 224 * 28 / S^2 whole planes per tile (2 for S = 56, 8 for S = 28), 224 threads.
//   column role  thread (quad, g, hs): columns 4 quad.. of plane g, rows 7 hs .. 7 hs + 6
//       pass A   V3 partial [w][j] = sum_h X[h][w] U3[h][j]           (pairs along w, U3 duplicated)
//       pass B   P4[w][j]        += sum_h X[h][w] V4[g,h][j]          (V4 duplicated)
//   row role     thread (row = g S + h, ws): the seven quads 7 ws .. 7 ws + 6 of that row
//       pass A   V4[g,h][j]  = sum_w X[h][w] U4[w][j]                 (U4 transposed, halves folded)
//       pass B   P3[h][j]   += sum_w X[h][w] V3[g][w][j]              (V3 transposed: as pass A of the columns left it)
// P3 and P4 accumulate in registers across the CTA's tiles.  Tiles are contiguous in memory and arrive
// through the bulk-copy engine (cp.async.bulk + mbarrier, bounded waits).
// ---------------------------------------------------------------------------------------------
namespace {
constexpr int kP2Threads = 224, kP2Stages = 2;   // a third stage bought nothing

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
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
// every thread waits for the phase; gives up after about one second
__device__ __forceinline__ bool mbar_wait_1s(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const uint64_t t0 = globaltimer_ns();
  for (uint32_t it = 0; it < (1u << 28); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u && globaltimer_ns() - t0 > 1000000000ull) return false;
  }
  return false;
}
}  // namespace

template <int S, typename TX>
__global__ void __launch_bounds__(kP2Threads, 2) k_plane2(PlaneArgs p) {
  constexpr int NT = kP2Threads, NST = kP2Stages;
  constexpr int QUADS = S / 4, HS = S / 7, WS = QUADS / 7, G = NT / (QUADS * HS);
  static_assert(S % 28 == 0 && QUADS * HS * G == NT && G * S * WS == NT, "S = 28 or 56");
  constexpr int SS = S * S;
  constexpr uint32_t kTileBytes = (uint32_t)(G * SS * sizeof(TX));
  extern __shared__ __align__(128) unsigned char p2_smem[];
  __shared__ __align__(8) uint64_t bars[NST];
  __shared__ int s_fail;
  TX* stages = reinterpret_cast<TX*>(p2_smem);                                   // [NST][G][S][S]
  f2* U3d = reinterpret_cast<f2*>(p2_smem + (size_t)NST * kTileBytes);           // [S][4]: (u, u)
  float* U4t = reinterpret_cast<float*>(U3d + S * 4);                            // [4][S]
  float* V3p = U4t + 4 * S;                                                      // [HS][G][4][S]
  float* V3t = V3p + HS * G * 4 * S;                                             // [G][4][S]
  f2* V4d = reinterpret_cast<f2*>(V3t + G * 4 * S);                              // [G S][4]: (v, v)
  const int tid = threadIdx.x;
  for (int idx = tid; idx < S * 4; idx += NT) {
    const int k = idx >> 2, j = idx & 3;
    const float u3 = (j < p.r3) ? p.U3[k * p.r3 + j] : 0.f;
    U3d[idx] = pack2(u3, u3);
    U4t[j * S + k] = (j < p.r4) ? p.U4[k * p.r4 + j] : 0.f;
  }
  if (tid == 0) {
    for (int s = 0; s < NST; ++s) mbar_init(bars + s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    s_fail = 0;
  }
  __syncthreads();
  const TX* __restrict__ X = reinterpret_cast<const TX*>(p.X);
  const int64_t n_tiles = p.n_planes / G;
  // thread 0 arms the stage's barrier and starts the copy (the plane count is a multiple of G: checked on the host)
  auto issue = [&](int64_t t, int st) {
    mbar_expect_tx(bars + st, kTileBytes);
    bulk_g2s(stages + (size_t)st * G * SS, X + t * G * SS, kTileBytes, bars + st);
  };
  int64_t t_issue = blockIdx.x;
  if (tid == 0) {
    for (int s = 0; s < NST - 1; ++s) {
      if (t_issue < n_tiles) issue(t_issue, s);
      t_issue += gridDim.x;
    }
  }
  // roles
  const int c_quad = tid % QUADS, c_g = (tid / QUADS) % G, c_hs = tid / (QUADS * G);
  const int r_row = tid / WS, r_ws = tid - r_row * WS;     // row = g S + h
  const int r_g = r_row / S;
  f2 accP3[4], accP4[4][2];
#pragma unroll
  for (int j = 0; j < 4; ++j) accP3[j] = accP4[j][0] = accP4[j][1] = 0ull;

  int st = 0;
  uint32_t phase_bits = 0;
  for (int64_t t = blockIdx.x; t < n_tiles; t += gridDim.x) {
    const bool ok = mbar_wait_1s(bars + st, (phase_bits >> st) & 1u);
    if (!ok) s_fail = 1;
    phase_bits ^= 1u << st;
    __syncthreads();                                 // everyone is past the previous tile: its stage is free
    if (s_fail) {
      if (tid == 0) atomicMax(p.status, (int)ASI_ERR_TIMEOUT);
      return;
    }
    if (tid == 0) {
      int sf = st + NST - 1;
      if (sf >= NST) sf -= NST;
      if (t_issue < n_tiles) issue(t_issue, sf);
      t_issue += gridDim.x;
    }
    const TX* Xs = stages + (size_t)st * G * SS;
    // the thread's values of the tile stay in registers for both passes: seven quads of its columns (rows
    // 7 hs ..) and the seven quads of its row
    f2 xc[7][2], xr[7][2];
    {
      const TX* xp = Xs + c_g * SS + (7 * c_hs) * S + 4 * c_quad;
#pragma unroll
      for (int i = 0; i < 7; ++i) ld_quad<TX>(xp + i * S, xc[i][0], xc[i][1]);
      const TX* xq = Xs + r_row * S + 28 * r_ws;
#pragma unroll
      for (int q = 0; q < 7; ++q) ld_quad<TX>(xq + 4 * q, xr[q][0], xr[q][1]);
    }
    // ---- pass A, column role: V3 partial over rows 7 hs ..
    {
      f2 acc[4][2];
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[j][0] = acc[j][1] = 0ull;
#pragma unroll
      for (int i = 0; i < 7; ++i) {
        const f2 x01 = xc[i][0], x23 = xc[i][1];
        const f2* ud = U3d + (7 * c_hs + i) * 4;
        const ulonglong2 ua = *reinterpret_cast<const ulonglong2*>(ud);
        const ulonglong2 ub = *reinterpret_cast<const ulonglong2*>(ud + 2);
        ffma2(acc[0][0], x01, ua.x); ffma2(acc[0][1], x23, ua.x);
        ffma2(acc[1][0], x01, ua.y); ffma2(acc[1][1], x23, ua.y);
        ffma2(acc[2][0], x01, ub.x); ffma2(acc[2][1], x23, ub.x);
        ffma2(acc[3][0], x01, ub.y); ffma2(acc[3][1], x23, ub.y);
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<ulonglong2*>(V3p + ((c_hs * G + c_g) * 4 + j) * S + 4 * c_quad) =
            make_ulonglong2(acc[j][0], acc[j][1]);
    }
    // ---- pass A, row role: V4 of this row
    {
      f2 acc[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[j] = 0ull;
#pragma unroll
      for (int q = 0; q < 7; ++q) {
        const f2 x01 = xr[q][0], x23 = xr[q][1];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const ulonglong2 u = *reinterpret_cast<const ulonglong2*>(U4t + j * S + 28 * r_ws + 4 * q);
          ffma2(acc[j], x01, u.x);
          ffma2(acc[j], x23, u.y);
        }
      }
      float v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        v[j] = fold2(acc[j]);
        if (WS == 2) v[j] += __shfl_xor_sync(0xffffffffu, v[j], 1);
      }
      if (r_ws == 0) {
        *reinterpret_cast<ulonglong2*>(V4d + r_row * 4) = make_ulonglong2(pack2(v[0], v[0]), pack2(v[1], v[1]));
        *reinterpret_cast<ulonglong2*>(V4d + r_row * 4 + 2) = make_ulonglong2(pack2(v[2], v[2]), pack2(v[3], v[3]));
      }
    }
    __syncthreads();
    // the HS partials of V3 meet in slice order
    for (int idx = tid; idx < G * 4 * S; idx += NT) {
      float s = 0.f;
#pragma unroll
      for (int h = 0; h < HS; ++h) s += V3p[h * G * 4 * S + idx];
      V3t[idx] = s;
    }
    __syncthreads();
    // ---- pass B, row role: P3[h] += sum_w X[h][w] V3[g][w]
    {
      const float* vp = V3t + r_g * 4 * S + 28 * r_ws;
#pragma unroll
      for (int q = 0; q < 7; ++q) {
        const f2 x01 = xr[q][0], x23 = xr[q][1];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const ulonglong2 v = *reinterpret_cast<const ulonglong2*>(vp + j * S + 4 * q);
          ffma2(accP3[j], x01, v.x);
          ffma2(accP3[j], x23, v.y);
        }
      }
    }
    // ---- pass B, column role: P4[w] += sum_h X[h][w] V4[g,h]
    {
#pragma unroll
      for (int i = 0; i < 7; ++i) {
        const f2 x01 = xc[i][0], x23 = xc[i][1];
        const f2* vd = V4d + (c_g * S + 7 * c_hs + i) * 4;
        const ulonglong2 va = *reinterpret_cast<const ulonglong2*>(vd);
        const ulonglong2 vb = *reinterpret_cast<const ulonglong2*>(vd + 2);
        ffma2(accP4[0][0], x01, va.x); ffma2(accP4[0][1], x23, va.x);
        ffma2(accP4[1][0], x01, va.y); ffma2(accP4[1][1], x23, va.y);
        ffma2(accP4[2][0], x01, vb.x); ffma2(accP4[2][1], x23, vb.x);
        ffma2(accP4[3][0], x01, vb.y); ffma2(accP4[3][1], x23, vb.y);
      }
    }
    st = (st + 1 == NST) ? 0 : st + 1;
  }
  // ---- one partial of P3 and P4 per CTA: the threads' sums meet in shared memory in thread order
  __syncthreads();
  float* red3 = V3p;                 // [NT][4]
  float* red4 = V3p + NT * 4;        // [NT][4 w][4 j]   (NT * 20 floats <= HS G 4 S + G 4 S + ..: checked on the host)
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    red3[tid * 4 + j] = fold2(accP3[j]);
    float a0, a1, b0, b1;
    unpack2(accP4[j][0], a0, a1);
    unpack2(accP4[j][1], b0, b1);
    red4[(tid * 4 + 0) * 4 + j] = a0;
    red4[(tid * 4 + 1) * 4 + j] = a1;
    red4[(tid * 4 + 2) * 4 + j] = b0;
    red4[(tid * 4 + 3) * 4 + j] = b1;
  }
  __syncthreads();
  for (int idx = tid; idx < S * 4; idx += NT) {
    const int k = idx >> 2, j = idx & 3;
    // P3[k][j]: rows g S + k of every plane slot g, both column halves
    float s3 = 0.f;
    for (int g = 0; g < G; ++g)
      for (int w = 0; w < WS; ++w) s3 += red3[((g * S + k) * WS + w) * 4 + j];
    // P4[k][j]: column k = 4 quad + e of every (g, hs)
    const int quad = k >> 2, e = k & 3;
    float s4 = 0.f;
    for (int h = 0; h < HS; ++h)
      for (int g = 0; g < G; ++g) s4 += red4[((((h * G + g) * QUADS + quad) * 4) + e) * 4 + j];
    if (j < p.r3) p.Pp3[((int64_t)blockIdx.x * S + k) * p.r3 + j] = s3;
    if (j < p.r4) p.Pp4[((int64_t)blockIdx.x * S + k) * p.r4 + j] = s4;
  }
}

size_t plane2_smem(int S, bool bf16) {
  const int QUADS = S / 4, HS = S / 7, G = kP2Threads / (QUADS * HS);
  const size_t tile = (size_t)G * S * S * (bf16 ? 2 : 4);
  size_t scratch = (size_t)(HS * G * 4 * S + G * 4 * S) * 4 + (size_t)G * S * 4 * 8;   // V3p, V3t, V4d (contiguous)
  const size_t red = (size_t)kP2Threads * 20 * 4;
  if (scratch < red) scratch = red;
  return kP2Stages * tile + (size_t)S * 4 * 8 + (size_t)4 * S * 4 + scratch;
}

int plane2_group(int S) { return kP2Threads / ((S / 4) * (S / 7)); }

bool plane2_supported(int S, int64_t n_planes, int r3, int r4) {
  return (S == 28 || S == 56) && r3 <= 4 && r4 <= 4 && n_planes % plane2_group(S) == 0;
}

template <int S, typename TX>
static cudaError_t launch_plane2_t(const PlaneArgs& p, int grid, cudaStream_t st) {
  const size_t smem = plane2_smem(S, sizeof(TX) == 2);
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_plane2<S, TX>), smem);
  if (e != cudaSuccess) return e;
  k_plane2<S, TX><<<grid, kP2Threads, smem, st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_plane2(const PlaneArgs& p, int grid, bool bf16, cudaStream_t st) {
  ProfScope prof(ASI_K_EXPAND, st, (double)p.n_planes * p.S * p.S * (bf16 ? 2 : 4));
  if (p.S == 56) return bf16 ? launch_plane2_t<56, __nv_bfloat16>(p, grid, st) : launch_plane2_t<56, float>(p, grid, st);
  return bf16 ? launch_plane2_t<28, __nv_bfloat16>(p, grid, st) : launch_plane2_t<28, float>(p, grid, st);
}

int plane2_grid(int S, int64_t n_planes, int max_ctas) {
  const int64_t tiles = n_planes / plane2_group(S);
  return (int)(tiles < max_ctas ? tiles : max_ctas);
}

// ---------------------------------------------------------------------------------------------
// k_core_tail: the core products that follow the first one on a conv activation, in one launch.
// T = A x_1 U_1^T is [r1][C][H][W]; CTA (chunk, i, cs) takes RH whole rows of the planes T[i][c], c in
// channel split cs:  Z[j][h,w] = sum_c U2[c][j] T[i][c][h][w]  (thread per position, coalesced),
// Y[j][h][l] = sum_w Z[j][h][w] U4[w][l],  part[j][k][l] = sum_h U3[h][k] Y[j][h][l]  over the chunk's rows.
// The last CTA to finish adds the partial cores in (chunk, split) order: core = T x_2 U_2^T x_3 U_3^T x_4 U_4^T.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_core_tail(CoreTailArgs p) {
  extern __shared__ __align__(16) float ct_smem[];
  __shared__ int s_last;
  const int tid = threadIdx.x;
  const int chunk = blockIdx.x, i = blockIdx.y, cs = blockIdx.z;
  const int r2 = p.r2, r3 = p.r3, r4 = p.r4, W = p.W, RH = p.RH;
  const int npos = RH * W;
  const int c0 = cs * p.cper, c1 = (c0 + p.cper < p.C) ? c0 + p.cper : p.C;
  float* Zs = ct_smem;                       // [r2][npos]
  float* Y1 = Zs + r2 * npos;                // [r2][RH][r4]
  float* U2s = Y1 + r2 * RH * r4;            // [cper][r2]
  float* U3s = U2s + p.cper * r2;            // [RH][r3]
  float* U4s = U3s + RH * r3;                // [W][r4]
  const int h0 = chunk * RH;
  for (int idx = tid; idx < (c1 - c0) * r2; idx += 256) U2s[idx] = p.U2[c0 * r2 + idx];
  for (int idx = tid; idx < RH * r3; idx += 256) U3s[idx] = (h0 + idx / r3 < p.H) ? p.U3[h0 * r3 + idx] : 0.f;
  for (int idx = tid; idx < W * r4; idx += 256) U4s[idx] = p.U4[idx];
  __syncthreads();
  for (int t = tid; t < npos; t += 256) {
    float acc[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[j] = 0.f;
    const bool on = h0 * W + t < p.H * W;
    const float* src = p.T + ((int64_t)i * p.C + c0) * p.H * W + (int64_t)h0 * W + t;
    if (on) {
#pragma unroll 4
      for (int c = 0; c < c1 - c0; ++c) {
        const float x = __ldg(src + (int64_t)c * p.H * W);
#pragma unroll
        for (int j = 0; j < 8; ++j)
          if (j < r2) acc[j] = fmaf(x, U2s[c * r2 + j], acc[j]);
      }
    }
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j < r2) Zs[j * npos + t] = acc[j];
  }
  __syncthreads();
  for (int idx = tid; idx < r2 * RH * r4; idx += 256) {
    const int l = idx % r4, jr = idx / r4;               // jr = j * RH + row
    const float* z = Zs + jr * W;                        // Zs[j][row][w]: npos = RH W
    float s = 0.f;
    for (int w = 0; w < W; ++w) s = fmaf(z[w], U4s[w * r4 + l], s);
    Y1[idx] = s;
  }
  __syncthreads();
  const int ce = r2 * r3 * r4;
  const int nparts = gridDim.x * gridDim.z;
  for (int idx = tid; idx < ce; idx += 256) {
    const int l = idx % r4, k = (idx / r4) % r3, j = idx / (r3 * r4);
    float s = 0.f;
    for (int row = 0; row < RH; ++row) s = fmaf(U3s[row * r3 + k], Y1[(j * RH + row) * r4 + l], s);
    p.part[((int64_t)i * nparts + chunk * gridDim.z + cs) * ce + idx] = s;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(p.counter, 1) == (int)(gridDim.x * gridDim.y * gridDim.z) - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int idx = tid; idx < p.r1 * ce; idx += 256) {
    const int ii = idx / ce, e = idx - ii * ce;
    const float* src = p.part + (int64_t)ii * nparts * ce + e;
    float s = 0.f;
    for (int q0 = 0; q0 < nparts; q0 += 8) {
      float v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = __ldcg(src + (int64_t)((q0 + q < nparts) ? (q0 + q) : 0) * ce);
#pragma unroll
      for (int q = 0; q < 8; ++q) s += (q0 + q < nparts) ? v[q] : 0.f;
    }
    p.core[idx] = s;
  }
  if (tid == 0) *p.counter = 0;
}

bool core_tail_supported(int r2, int r3, int r4, int H, int W) {
  return r2 <= 8 && r3 <= 8 && r4 <= 8 && W <= 128 && H * W >= 256;
}
void core_tail_shape(int C, int H, int W, int* RH, int* nchunk, int* csplit, int* cper) {
  int rh = 256 / W;
  if (rh < 1) rh = 1;
  *RH = rh;
  *nchunk = (H + rh - 1) / rh;
  int cs = 1;
  while (cs < 8 && C / (cs * 2) >= 16) cs *= 2;
  *cper = (C + cs - 1) / cs;
  *csplit = (C + *cper - 1) / *cper;
}
size_t core_tail_part_elems(int r1, int r2, int r3, int r4, int C, int H, int W) {
  int RH, nchunk, csplit, cper;
  core_tail_shape(C, H, W, &RH, &nchunk, &csplit, &cper);
  return (size_t)r1 * nchunk * csplit * r2 * r3 * r4;
}
cudaError_t launch_core_tail(const CoreTailArgs& p0, cudaStream_t st) {
  CoreTailArgs p = p0;
  int nchunk, csplit;
  core_tail_shape(p.C, p.H, p.W, &p.RH, &nchunk, &csplit, &p.cper);
  const size_t smem = 4 * ((size_t)p.r2 * p.RH * p.W + (size_t)p.r2 * p.RH * p.r4 + (size_t)p.cper * p.r2 +
                           (size_t)p.RH * p.r3 + (size_t)p.W * p.r4);
  ProfScope prof(ASI_K_MODEPROD, st, 4.0 * p.r1 * p.C * p.H * p.W);
  k_core_tail<<<dim3(nchunk, p.r1, csplit), 256, smem, st>>>(p);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// k_z3: Z3[ij][h][w] = sum_{k,l} core[ij][k][l] U3[h][k] U4[w][l]  (C_ASI terms 2 and 3 in one launch)
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_z3(const float* __restrict__ core, const float* __restrict__ U3,
                                            const float* __restrict__ U4, float* __restrict__ Z3, int r12, int r3,
                                            int r4, int H, int W) {
  extern __shared__ float z3_smem[];
  float* Ss = z3_smem;                 // [r3][r4] of this (i, j)
  float* U3s = Ss + r3 * r4;           // [H][r3]
  float* U4s = U3s + H * r3;           // [W][r4]
  const int ij = blockIdx.y, tid = threadIdx.x;
  for (int idx = tid; idx < r3 * r4; idx += 256) Ss[idx] = core[ij * r3 * r4 + idx];
  for (int idx = tid; idx < H * r3; idx += 256) U3s[idx] = U3[idx];
  for (int idx = tid; idx < W * r4; idx += 256) U4s[idx] = U4[idx];
  __syncthreads();
  for (int pos = blockIdx.x * 256 + tid; pos < H * W; pos += gridDim.x * 256) {
    const int h = pos / W, w = pos - h * W;
    float s = 0.f;
    for (int k = 0; k < r3; ++k) {
      float t = 0.f;
      for (int l = 0; l < r4; ++l) t = fmaf(Ss[k * r4 + l], U4s[w * r4 + l], t);
      s = fmaf(t, U3s[h * r3 + k], s);
    }
    Z3[(int64_t)ij * H * W + pos] = s;
  }
}

cudaError_t launch_z3(const float* core, const float* U3, const float* U4, float* Z3, int r12, int r3, int r4,
                      int H, int W, cudaStream_t st) {
  ProfScope prof(ASI_K_MODEPROD, st, 4.0 * r12 * H * W);
  int gx = (H * W + 255) / 256;
  if (gx > 16) gx = 16;
  const size_t smem = 4 * ((size_t)r3 * r4 + (size_t)H * r3 + (size_t)W * r4);
  k_z3<<<dim3(gx, r12), 256, smem, st>>>(core, U3, U4, Z3, r12, r3, r4, H, W);
  return cudaGetLastError();
}

}  // namespace asi
