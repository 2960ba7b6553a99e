// Fused kernels for conv layers with small square feature maps (S x S, S in {7, 14, 16}) and
// ranks <= 8 -- the shapes of the ResNet / MobileNet tails.  One compress call is three launches:
//
//   k_sm_pass1  : forms every P_m = A_m (A_m^T U_m^prev) (Algorithm 1) tile-locally, so no V_m ever
//                 reaches global memory.  CTAs of role B hold a tile [all B x J contiguous (c,h,w)]
//                 that contains whole mode-1/3/4 fibers (one half of the CTA iterates mode 1 while the
//                 other half does modes 3 and 4); CTAs of role C hold one sample [all C x HW] that
//                 contains whole mode-2 fibers.  fp32 tiles are staged in shared memory by the
//                 bulk-copy engine (cp.async.bulk + mbarrier), one row or chunk per copy; the
//                 activation comes from HBM once, the other role's traversal is served by L2.
//   k_sm_reduce : fixed-order fp64 reduction of the per-tile partials of every P_m and per-chunk
//                 shares of the Gram matrices G_m = P_m^T P_m;
//   k_sm_core   : every CTA finishes Orthogonalize for the factor rows it needs while its tile is in
//                 flight (Cholesky G_m = R^T R, U_m = P_m R^{-1}: the Gram-Schmidt basis), then
//                 contracts its tile [all B x J] with U_1..U_4; the last CTA sums the per-tile cores.
//
// and the whole compressed weight gradient is one kernel, k_sm_wgrad (terms 1-5 of C_ASI).
// Every wait on an mbarrier is bounded (about one second); on expiry the CTA records
// ASI_ERR_TIMEOUT in the status word and returns.
#include <cuda_bf16.h>

#include <type_traits>

#include "asi_internal.h"

namespace asi {

namespace {

constexpr int kNT = 512;             // threads per CTA of the tile kernels
constexpr int kNG = 256;             // threads of one half (warp-specialised phases)
constexpr int kRedNT = 256;          // threads per CTA of the partial-reduction kernel

__host__ __device__ constexpr int pitch4(int J) {      // >= J, multiple of 4, == 4 (mod 32)
  int p = (J + 3) / 4 * 4;
  while (p % 32 != 4) p += 4;
  return p;
}

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }

template <typename TX>
__device__ __forceinline__ float4 ld4(const TX* p);
template <>
__device__ __forceinline__ float4 ld4<float>(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}
template <>
__device__ __forceinline__ float4 ld4<__nv_bfloat16>(const __nv_bfloat16* p) {
  const uint2 raw = *reinterpret_cast<const uint2*>(p);
  const __nv_bfloat162 lo = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
  const __nv_bfloat162 hi = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
  return make_float4(__low2float(lo), __high2float(lo), __low2float(hi), __high2float(hi));
}

// ---- bulk-copy engine (TMA, untiled form) and mbarrier ------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
// dst and src 16-byte aligned, bytes a multiple of 16
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
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, uint64_t limit_ns) {
  const uint64_t t0 = globaltimer_ns();
  for (uint32_t it = 0; it < (1u << 28); ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 255u) == 255u && globaltimer_ns() - t0 > limit_ns) return false;
  }
  return false;
}
// Thread 0 waits for the staged tile with a time limit; every thread learns the outcome.  On expiry
// the status word gets ASI_ERR_TIMEOUT and thread 0 gives the copies in flight one more bounded
// wait before the CTA returns.
__device__ __forceinline__ bool cta_wait_tile(uint64_t* bar, int* s_flag, int* status, uint64_t limit_ns) {
  if (threadIdx.x == 0) {
    bool ok = mbar_wait_bounded(bar, 0, limit_ns);
    if (!ok) {
      atomicMax(status, (int)ASI_ERR_TIMEOUT);
      mbar_wait_bounded(bar, 0, limit_ns);
    }
    *s_flag = ok ? 1 : 0;
  }
  __syncthreads();
  const bool ok = *s_flag != 0;
  if (ok)
    for (int it = 0; it < 64 && !mbar_try_wait(bar, 0); ++it) {
    }
  return ok;
}

// Warp 0 stages one contiguous block in chunks of 16 KB.
__device__ __forceinline__ void stage_block(uint64_t* bar, char* dst, const char* src, uint32_t bytes, bool stall) {
  constexpr uint32_t kChunk = 16384;
  const int lane = threadIdx.x & 31;
  if ((threadIdx.x >> 5) != 0) return;
  if (lane == 0) {
    mbar_init(bar, 1);
    mbar_expect_tx(bar, bytes);
  }
  __syncwarp();
  const int nchunk = stall ? 0 : (int)((bytes + kChunk - 1) / kChunk);
  for (int i = lane; i < nchunk; i += 32) {
    const uint32_t off = (uint32_t)i * kChunk;
    const uint32_t n = (bytes - off < kChunk) ? bytes - off : kChunk;
    bulk_g2s(dst + off, src + off, n, bar);
  }
}

// Small read-only arrays a CTA keeps in shared memory (factors, the core).  fac_issue_*() start one
// 4-byte asynchronous copy (cp.async) per element -- short loops, no registers held -- and
// fac_wait() waits for this thread's copies; a __syncthreads() after it publishes them.  Whatever a
// kernel does in between overlaps the single round trip, and these small loads are ahead of its bulk
// traffic in the memory system.
__device__ __forceinline__ void cp_async4(float* dst, const float* src, int bytes /* 4, or 0 to store 0.f */) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(smem_u32(dst)), "l"(src), "r"(bytes) : "memory");
}
// dst[k*RD + j] = j < r ? src[k*r + j] : 0 for k < rows: a factor [rows x r] padded to RD columns
template <int RD>
__device__ __forceinline__ void fac_issue_padded(const float* __restrict__ src, float* dst, int rows, int r) {
#pragma unroll 1
  for (int idx = threadIdx.x; idx < rows * RD; idx += kNT) {
    const int k = idx / RD, j = idx % RD;
    cp_async4(dst + idx, src + (j < r ? k * r + j : 0), j < r ? 4 : 0);
  }
}
__device__ __forceinline__ void fac_issue_flat(const float* __restrict__ src, float* dst, int n) {
#pragma unroll 1
  for (int idx = threadIdx.x; idx < n; idx += kNT) cp_async4(dst + idx, src + idx, 4);
}
__device__ __forceinline__ void fac_wait() {
  asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
// waits until at most N of this thread's committed groups are still in flight
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// Starts the copy of `rows` fp32 rows of J values (J a multiple of 4, both sides 16-byte aligned): row i
// from src + i*src_stride to dst + i*PJ, 16 bytes per cp.async, one row per warp at a time.  (One bulk
// copy per row would leave the issuing warp busy for ~60 cycles per row: the tile of a 64-sample
// batch would arrive ~2 us later.)
__device__ __forceinline__ void stage_rows_async(float* dst, const float* __restrict__ src, int rows, int J,
                                                 int64_t src_stride, int PJ) {
  const int lane = threadIdx.x & 31, nv = J >> 2;
  for (int i = threadIdx.x >> 5; i < rows; i += kNT / 32) {
    const float* s = src + i * src_stride;
    float* d = dst + i * PJ;
    for (int v = lane; v < nv; v += 32)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(d + 4 * v)), "l"(s + 4 * v) : "memory");
  }
}

template <int R>
__device__ __forceinline__ void fma_row(float (&acc)[R], float x, const float* __restrict__ u) {
#pragma unroll
  for (int j = 0; j < R; j += 4) {
    const float4 v = *reinterpret_cast<const float4*>(u + j);
    acc[j] = fmaf(x, v.x, acc[j]);
    acc[j + 1] = fmaf(x, v.y, acc[j + 1]);
    acc[j + 2] = fmaf(x, v.z, acc[j + 2]);
    acc[j + 3] = fmaf(x, v.w, acc[j + 3]);
  }
}

// Programmatic dependent launch: the reduce and core kernels are launched with the
// programmatic-stream-serialization attribute, so their CTAs may start (and do whatever does not
// depend on the previous kernel, e.g. stage their activation tile) once every CTA of the previous
// kernel has passed pdl_launch_dependents(); pdl_wait() then blocks until that kernel has finished
// and its writes are visible.  Without the attribute both are no-ops.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Division of a small index (n < 2^21) by a run-time divisor through one reciprocal: the integer
// division sequence costs ~150 cycles of latency, which dominates the short index loops below.
struct FDiv {
  float inv;
  int d;
  __device__ __forceinline__ explicit FDiv(int d_) : inv(1.0f / (float)d_), d(d_) {}
  __device__ __forceinline__ int div(int n) const { return __float2int_rd(((float)n + 0.5f) * inv); }
  __device__ __forceinline__ void divmod(int n, int& q, int& r) const {
    q = div(n);
    r = n - q * d;
  }
};

__device__ __forceinline__ void bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Sum of N per-lane values over the 32 lanes of a warp by recursive halving: every step each lane
// hands half of its values to its partner, so the whole reduction costs N-N/32 shuffles.  On return
// v[i], i < N/32, is the total of element scatter_base<N>(lane) + i.  The order of additions is fixed.
template <int N, int OFF>
__device__ __forceinline__ void halving_step(float* v, int lane) {
  constexpr int n = N / 2;
  const bool up = (lane & OFF) != 0;
#pragma unroll
  for (int i = 0; i < n; ++i) {
    const float send = up ? v[i] : v[i + n];
    const float keep = up ? v[i + n] : v[i];
    v[i] = keep + __shfl_xor_sync(0xffffffffu, send, OFF);
  }
}
template <int N>
__device__ __forceinline__ void warp_reduce_scatter(float (&v)[N], int lane) {
  static_assert(N % 32 == 0, "pad the accumulator count to a multiple of 32");
  halving_step<N, 16>(v, lane);
  halving_step<N / 2, 8>(v, lane);
  halving_step<N / 4, 4>(v, lane);
  halving_step<N / 8, 2>(v, lane);
  halving_step<N / 16, 1>(v, lane);
}
template <int N>
__device__ __forceinline__ int scatter_base(int lane) {
  return ((lane >> 4) & 1) * (N / 2) + ((lane >> 3) & 1) * (N / 4) + ((lane >> 2) & 1) * (N / 8) +
         ((lane >> 1) & 1) * (N / 16) + (lane & 1) * (N / 32);
}

// Number of interleaved sample groups project_batch uses for a tile of J columns on nthr threads.
__host__ __device__ constexpr int batch_groups(int nthr, int J) {
  const int items = J / 2;
  int nh = nthr / items;
  return nh < 1 ? 1 : (nh > 4 ? 4 : nh);
}

// out[j][0..R) = sum_b Xs[b*PJ + j] * Us[b*R + ..] for j < J: the mode-1 contraction of a staged tile
// [B x J].  Runs on `nthr` threads (t = 0..nthr-1) that synchronise on named barrier `bar`.  A thread
// owns two neighbouring columns (one 8-byte shared load per sample) and the samples b == h (mod NH);
// the NH partial sums meet in `part` ([NH][J][R]) in a fixed order.
template <int R>
__device__ __forceinline__ void project_batch(const float* __restrict__ Xs, int PJ,
                                              const float* __restrict__ Us, int B, int J,
                                              float* __restrict__ part, float* __restrict__ out, int t,
                                              int nthr, int bar) {
  const int NH = batch_groups(nthr, J);
  const int J2 = J >> 1;                             // J is even
  const FDiv dJ2(J2);
#pragma unroll 1
  for (int it = t; it < NH * J2; it += nthr) {
    int h, jp;
    dJ2.divmod(it, h, jp);
    float a0[R], a1[R];
#pragma unroll
    for (int q = 0; q < R; ++q) a0[q] = a1[q] = 0.f;
#pragma unroll 4
    for (int b = h; b < B; b += NH) {
      const float2 x = *reinterpret_cast<const float2*>(Xs + b * PJ + 2 * jp);
      fma_row<R>(a0, x.x, Us + b * R);
      fma_row<R>(a1, x.y, Us + b * R);
    }
    float* dst = (NH > 1 ? part + h * J * R : out) + 2 * jp * R;
#pragma unroll
    for (int q = 0; q < R; q += 4) {
      *reinterpret_cast<float4*>(dst + q) = make_float4(a0[q], a0[q + 1], a0[q + 2], a0[q + 3]);
      *reinterpret_cast<float4*>(dst + R + q) = make_float4(a1[q], a1[q + 1], a1[q + 2], a1[q + 3]);
    }
  }
  if (NH > 1) {
    bar_sync(bar, nthr);
#pragma unroll 1
    for (int idx = t; idx < J * R; idx += nthr) {
      float s = 0.f;
      for (int h = 0; h < NH; ++h) s += part[h * J * R + idx];
      out[idx] = s;
    }
  }
  bar_sync(bar, nthr);
}

// V[hw][:] = sum_c Xs[c*PC + hw] * Us[c][:] for a staged block Xs [C][HWC] of one sample (the mode-2
// projection of HWC positions).  Thread (g, hw) sums the channels c = g (mod G); group 0 writes V
// itself, groups 1..G-1 write Vp ([G-1][HWC][R]; may alias Us: it is written only after every thread
// has finished reading Us) and the sums meet in a fixed order.  All kNT threads call it.
template <int HWC, int PC, int R>
__device__ __forceinline__ void project_channels(const float* __restrict__ Xs, const float* Us, float* Vp,
                                                 float* V, int C) {
  constexpr int G = kNT / HWC;
  const int tid = threadIdx.x;
  float acc[R];
#pragma unroll
  for (int j = 0; j < R; ++j) acc[j] = 0.f;
  const int g = tid / HWC, hw = tid - g * HWC;
  if (g < G) {
#pragma unroll 4
    for (int c = g; c < C; c += G) fma_row<R>(acc, Xs[c * PC + hw], Us + c * R);
  }
  if (G > 1) __syncthreads();
  if (g < G) {
    float* dst = (g == 0 ? V : Vp + (g - 1) * HWC * R) + hw * R;
#pragma unroll
    for (int j = 0; j < R; j += 4)
      *reinterpret_cast<float4*>(dst + j) = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
  }
  __syncthreads();
  if (G > 1) {
    for (int idx = tid; idx < HWC * R; idx += kNT) {
      float s = V[idx];
#pragma unroll
      for (int gg = 0; gg < G - 1; ++gg) s += Vp[gg * HWC * R + idx];
      V[idx] = s;
    }
    __syncthreads();
  }
}

// Stages one tile [B x J] (row b at src + b*sample_stride) as fp32 rows of pitch PJ.
template <typename TX>
__device__ __forceinline__ void stage_tile_begin(const TX* __restrict__ src, int64_t sample_stride, float* Xs,
                                                 int B, int J, int PJ) {
  if constexpr (std::is_same<TX, float>::value) {
    stage_rows_async(Xs, src, B, J, sample_stride, PJ);
  } else {
    const int J4 = J / 4;
    for (int idx = threadIdx.x; idx < B * J4; idx += kNT) {
      const int b = idx / J4, v = idx - b * J4;
      *reinterpret_cast<float4*>(Xs + b * PJ + 4 * v) = ld4<TX>(src + b * sample_stride + 4 * v);
    }
  }
}

// Role C of the first pass takes the positions of a sample in NQ parts.  S = 7: the whole map.  Larger
// maps: four parts that start on 16-byte boundaries -- 14 x 14 splits its 49 float4 per channel as
// 13 + 12 + 12 + 12 (parts 1..3 carry four zero columns), 16 x 16 as 4 x 16.
__host__ __device__ constexpr int role_c_hwc(int S) { return S == 7 ? 49 : (S == 14 ? 52 : S * S / 4); }
__host__ __device__ constexpr int role_c_pitch(int S) { return S == 7 ? 49 : pitch4(role_c_hwc(S)); }

__host__ __device__ constexpr int tri_index(int S, int k, int k2) {   // k <= k2 < S, row-major upper triangle
  return k * S - k * (k - 1) / 2 + (k2 - k);
}

// 14 x 14 Gram matrix G = A_m A_m^T of a tile [planes x 196] in 7 x 7 blocks.  With a = rows 0..6 and
// b = rows 7..13 of a fiber, warp role 0 accumulates the upper triangle of a a^T, role 1 that of
// b b^T, role 2 the block a b[0..3]^T and role 3 the block a b[4..6]^T (<= 28 accumulators each).
// A unit is a quarter of a plane (fibers == part mod 4), so the lanes of a warp hit 32 banks; this
// thread takes units u0, u0 + ustride, ...  es = step between the elements of a fiber, cs = step
// between neighbouring fibers (mode 3: 14, 1; mode 4: 1, 14).
template <int PJ>
__device__ __forceinline__ void gram14_accumulate(const float* __restrict__ Xs, int nunits, int u0, int ustride,
                                                  int role, int es, int cs, float (&acc)[32]) {
#pragma unroll
  for (int i = 0; i < 32; ++i) acc[i] = 0.f;
  for (int un = u0; un < nunits; un += ustride) {
    const float* base = Xs + (un >> 2) * PJ;
#pragma unroll 1
    for (int col = un & 3; col < 14; col += 4) {
      const float* colp = base + col * cs;
      if (role < 2) {
        const float* q = colp + role * 7 * es;
        float x[7];
#pragma unroll
        for (int k = 0; k < 7; ++k) x[k] = q[k * es];
#pragma unroll
        for (int k = 0; k < 7; ++k)
#pragma unroll
          for (int k2 = k; k2 < 7; ++k2) acc[tri_index(7, k, k2)] = fmaf(x[k], x[k2], acc[tri_index(7, k, k2)]);
      } else if (role == 2) {
        float xa[7], xb[4];
#pragma unroll
        for (int k = 0; k < 7; ++k) xa[k] = colp[k * es];
#pragma unroll
        for (int k = 0; k < 4; ++k) xb[k] = colp[(7 + k) * es];
#pragma unroll
        for (int k = 0; k < 7; ++k)
#pragma unroll
          for (int k2 = 0; k2 < 4; ++k2) acc[k * 4 + k2] = fmaf(xa[k], xb[k2], acc[k * 4 + k2]);
      } else {
        float xa[7], xb[3];
#pragma unroll
        for (int k = 0; k < 7; ++k) xa[k] = colp[k * es];
#pragma unroll
        for (int k = 0; k < 3; ++k) xb[k] = colp[(11 + k) * es];
#pragma unroll
        for (int k = 0; k < 7; ++k)
#pragma unroll
          for (int k2 = 0; k2 < 3; ++k2) acc[k * 3 + k2] = fmaf(xa[k], xb[k2], acc[k * 3 + k2]);
      }
    }
  }
}
// which role (rl) and accumulator (e) hold element o = k*14 + k2 of the symmetric 14 x 14 matrix
__device__ __forceinline__ void gram14_slot(int o, int& rl, int& e) {
  const int k = o / 14, k2 = o % 14;
  const int lo = k < k2 ? k : k2, hi = k < k2 ? k2 : k;
  if (hi < 7) { rl = 0; e = tri_index(7, lo, hi); }
  else if (lo >= 7) { rl = 1; e = tri_index(7, lo - 7, hi - 7); }
  else if (hi < 11) { rl = 2; e = lo * 4 + (hi - 7); }
  else { rl = 3; e = lo * 3 + (hi - 11); }
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// k_sm_pass1
// ---------------------------------------------------------------------------------------------
template <int S, int R, typename TX>
__device__ __forceinline__ void sm_pass1_cta(const SmPass1Args& p, const int bid) {
  constexpr bool kBulk = std::is_same<TX, float>::value;
  constexpr bool kGram = (S == 7);                   // modes 3, 4 as Gram matrices A_m A_m^T (7 x 7)
  constexpr bool kGram14 = (S == 14);                // ... as 14 x 14 Gram matrices in four 7 x 7 blocks
  constexpr int HW = S * S;
  constexpr int CC = (S == 7) ? 4 : 1;               // channels per role-B tile
  constexpr int J = CC * HW;                         // contiguous elements per sample in a tile
  constexpr int PJ = pitch4(J);                      // row pitch == 4 (mod 32): conflict-free (b, j) reads
  constexpr int NH1 = batch_groups(kNG, J);
  extern __shared__ __align__(128) float smem[];
  __shared__ __align__(8) uint64_t s_bar;
  __shared__ int s_flag;
  const int tid = threadIdx.x, lane = tid & 31;
  const TX* __restrict__ A = reinterpret_cast<const TX*>(p.act);
  const int B = p.B, C = p.C;

  if (bid == 0 && tid < 241) p.status[tid == 0 ? 0 : 15 + tid] = 0;  // status word, counters 16..255
  pdl_launch_dependents();

  constexpr int kNQ = (S == 7) ? 1 : 4;             // role-C CTAs per sample
  if (bid >= B * kNQ) {
    // ---------------- role B: modes 1, 3, 4 on tile [B x J] ----------------
    const int tile = bid - B * kNQ;
    float* Xs = smem;                                // [B][PJ]
    float* U1s = Xs + B * PJ;                        // [B][R]
    float* U3s = U1s + B * R;                        // [S][R]
    float* U4s = U3s + S * R;                        // [S][R]
    float* V1s = U4s + S * R;                        // [J][R]
    float* part = V1s + J * R;                       // [NH1][J][R] (NH1 > 1 only)
    float* red = part + (NH1 > 1 ? NH1 : 0) * J * R; // [8][32], S = 14: [8 + 16][32]
    fac_issue_padded<R>(p.U_prev + p.u_off[0], U1s, B, p.r[0]);
    if constexpr (!kGram && !kGram14) {
      fac_issue_padded<R>(p.U_prev + p.u_off[2], U3s, S, p.r[2]);
      fac_issue_padded<R>(p.U_prev + p.u_off[3], U4s, S, p.r[3]);
    }
    stage_tile_begin<TX>(A + (int64_t)tile * J, (int64_t)C * HW, Xs, B, J, PJ);
    fac_wait();
    __syncthreads();
    const int t = tid & (kNG - 1), wg = t >> 5;
    if (tid < kNG) {
      // ---- half 0: mode 1.  V[j,:] = sum_b X[b,j] U1[b,:], then P1[b,:] = sum_j X[b,j] V[j,:]
      project_batch<R>(Xs, PJ, U1s, B, J, part, V1s, t, kNG, 1);
      float* P1 = p.Pp[0] + (int64_t)tile * B * p.r[0];
      const int bl = lane >> 2, jl = lane & 3;       // a warp covers 8 samples x 4 column phases
      for (int b0 = wg * 8; b0 < B; b0 += 64) {
        const int b = b0 + bl;
        float acc[R];
#pragma unroll
        for (int q = 0; q < R; ++q) acc[q] = 0.f;
#pragma unroll 7
        for (int jj = jl; jj < J; jj += 4) fma_row<R>(acc, Xs[b * PJ + jj], V1s + jj * R);
#pragma unroll
        for (int q = 0; q < R; ++q) {
          acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], 1);
          acc[q] += __shfl_xor_sync(0xffffffffu, acc[q], 2);
        }
        if (jl == 0) {
#pragma unroll
          for (int q = 0; q < R; ++q)
            if (q < p.r[0]) P1[b * p.r[0] + q] = acc[q];
        }
      }
    } else if constexpr (kGram) {
      // ---- half 1, S = 7: G_m = A_m A_m^T for m = 3, 4, one plane (b, c) per thread at a time; the
      // 32 lanes of a warp touch 32 different banks.  P_m = G_m U_m^prev follows in k_sm_reduce.
      constexpr int NACC = 32;
      static_assert(S * (S + 1) / 2 <= NACC, "upper triangle of the Gram matrix");
      const int nplanes = B * CC;
#pragma unroll 1
      for (int mode = 2; mode <= 3; ++mode) {
        const int es = (mode == 2) ? S : 1;          // step between the elements of a fiber
        const int cs = (mode == 2) ? 1 : S;          // step between neighbouring fibers
        float* Gm = p.Pp[mode] + (int64_t)tile * HW;
        float acc[NACC];
#pragma unroll
        for (int i = 0; i < NACC; ++i) acc[i] = 0.f;
        for (int pl = t; pl < nplanes; pl += kNG) {
          const int b = pl / CC, cl = pl % CC;
          const float* base = Xs + b * PJ + cl * HW;
#pragma unroll 1
          for (int col = 0; col < S; ++col) {
            const float* colp = base + col * cs;
            float x[S];
#pragma unroll
            for (int k = 0; k < S; ++k) x[k] = colp[k * es];
#pragma unroll
            for (int k = 0; k < S; ++k)
#pragma unroll
              for (int k2 = k; k2 < S; ++k2) acc[tri_index(S, k, k2)] = fmaf(x[k], x[k2], acc[tri_index(S, k, k2)]);
          }
        }
        warp_reduce_scatter<NACC>(acc, lane);
        red[wg * 32 + scatter_base<NACC>(lane)] = acc[0];
        bar_sync(2, kNG);
        for (int o = t; o < HW; o += kNG) {
          const int k = o / S, k2 = o % S;
          const int e = (k <= k2) ? tri_index(S, k, k2) : tri_index(S, k2, k);
          float s = 0.f;
#pragma unroll
          for (int w = 0; w < 8; ++w) s += red[w * 32 + e];
          Gm[o] = s;
        }
        bar_sync(2, kNG);
      }
    } else if constexpr (kGram14) {
      // ---- half 1, S = 14: G_3 = A_3 A_3^T (see gram14_accumulate); G_4 follows on all sixteen warps
      const int role = wg & 3;
      float* Gm = p.Pp[2] + (int64_t)tile * HW;
      float acc[32];
      gram14_accumulate<PJ>(Xs, B * 4, (wg >> 2) * 32 + lane, 64, role, S, 1, acc);
      warp_reduce_scatter<32>(acc, lane);
      red[wg * 32 + scatter_base<32>(lane)] = acc[0];
      bar_sync(2, kNG);
      for (int o = t; o < HW; o += kNG) {
        int rl, e;
        gram14_slot(o, rl, e);
        Gm[o] = red[rl * 32 + e] + red[(rl + 4) * 32 + e];
      }
    } else {
      // ---- half 1, other sizes: P_m = A_m (A_m^T U_m^prev) for m = 3, 4.  A unit is a quarter of a plane
      // (columns == part mod 4); unit -> thread so that the 32 lanes of a warp touch 32 different
      // banks.  Each thread owns 2 columns of the factor; warp w serves column pair w mod JH.
      constexpr int TPP = 4, JT = 2, JH = R / JT, NACC = 32;
      static_assert(S * JT <= NACC, "accumulators of one thread");
      const int jh = wg % JH;
      const int u0 = (wg / JH) * 32 + lane;
      const int nunits = B * CC * TPP;
#pragma unroll 1
      for (int mode = 2; mode <= 3; ++mode) {
        const float* Us = ((mode == 2) ? U3s : U4s) + jh * JT;
        const int es = (mode == 2) ? S : 1;
        const int cs = (mode == 2) ? 1 : S;
        const int rm = p.r[mode];
        float* Pm = p.Pp[mode] + (int64_t)tile * S * rm;
        float acc[NACC];
#pragma unroll
        for (int i = 0; i < NACC; ++i) acc[i] = 0.f;
        for (int un = u0; un < nunits; un += kNG / JH) {
          const int pl = un / TPP, part_ = un % TPP;
          const int b = pl / CC, cl = pl % CC;
          const float* base = Xs + b * PJ + cl * HW;
#pragma unroll 1
          for (int col = part_; col < S; col += TPP) {
            const float* colp = base + col * cs;
            float x[S], v0 = 0.f, v1 = 0.f;
#pragma unroll
            for (int k = 0; k < S; ++k) {
              x[k] = colp[k * es];
              const float2 u = *reinterpret_cast<const float2*>(Us + k * R);
              v0 = fmaf(x[k], u.x, v0);
              v1 = fmaf(x[k], u.y, v1);
            }
#pragma unroll
            for (int k = 0; k < S; ++k) {
              acc[2 * k] = fmaf(x[k], v0, acc[2 * k]);
              acc[2 * k + 1] = fmaf(x[k], v1, acc[2 * k + 1]);
            }
          }
        }
        warp_reduce_scatter<NACC>(acc, lane);
        red[wg * 32 + scatter_base<NACC>(lane)] = acc[0];
        bar_sync(2, kNG);
        for (int o = t; o < S * R; o += kNG) {
          const int k = o / R, j = o % R;
          const int e = k * JT + (j % JT);
          float s = 0.f;
          for (int w = j / JT; w < 8; w += JH) s += red[w * 32 + e];
          if (j < rm) Pm[k * rm + j] = s;
        }
        bar_sync(2, kNG);
      }
    }
    if constexpr (kGram14) {
      // ---- S = 14, G_4 = A_4 A_4^T: each half joins as it finishes its first job (mode 1 or G_3)
      const int gw = tid >> 5, role = gw & 3;
      float* red4 = red + 8 * 32;                    // [16][32]
      float acc[32];
      gram14_accumulate<PJ>(Xs, B * 4, (gw >> 2) * 32 + lane, 128, role, 1, S, acc);
      warp_reduce_scatter<32>(acc, lane);
      red4[gw * 32 + scatter_base<32>(lane)] = acc[0];
      __syncthreads();
      float* Gm = p.Pp[3] + (int64_t)tile * HW;
      for (int o = tid; o < HW; o += kNT) {
        int rl, e;
        gram14_slot(o, rl, e);
        Gm[o] = ((red4[rl * 32 + e] + red4[(rl + 4) * 32 + e]) + red4[(rl + 8) * 32 + e]) + red4[(rl + 12) * 32 + e];
      }
    }
  } else {
    // ---------------- role C: mode 2 on block [C x HWC] of one sample ----------------
    // S = 7: the whole sample (contiguous, staged by the bulk-copy engine, odd row pitch for the
    // row-per-thread reads below); larger maps: one part of the positions, rows staged by 16-byte
    // cp.async at a pitch == 4 (mod 32), read back as float4.
    constexpr int NQ = (S == 7) ? 1 : 4;
    constexpr int HWC = role_c_hwc(S);
    constexpr int PC = role_c_pitch(S);
    constexpr int G = kNT / HWC;
    constexpr bool kBulkC = kBulk && NQ == 1;
    const int b = bid / NQ, q = bid % NQ;
    const int hw0 = (S == 14) ? (q == 0 ? 0 : 4 + 48 * q) : q * HWC;     // first position of this part
    const int nval = (S == 14 && q > 0) ? 48 : HWC;                      // positions it holds
    float* Xs = smem;                                // [C][PC]
    float* U2s = Xs + ((C * PC + 3) & ~3);           // [C][R]
    float* V2s = U2s + C * R;                        // [HWC][R]
    float* Vp = (C >= (G - 1) * HWC) ? U2s : V2s + HWC * R;   // [G-1][HWC][R]: on top of U2s when it fits
    const TX* Xb = A + (int64_t)b * C * HW + hw0;
    if constexpr (kBulkC)
      stage_block(&s_bar, reinterpret_cast<char*>(Xs), reinterpret_cast<const char*>(Xb), (uint32_t)C * HW * 4u,
                  p.stall_copy != 0);
    fac_issue_padded<R>(p.U_prev + p.u_off[1], U2s, C, p.r[1]);
    if constexpr (kBulkC) {
    } else if constexpr (NQ == 1) {
      const int n4 = C * HW / 4;
      for (int idx = tid; idx < n4; idx += kNT) *reinterpret_cast<float4*>(Xs + 4 * idx) = ld4<TX>(Xb + 4 * idx);
    } else {
      constexpr int NV = HWC / 4;
      const int n = C * NV;
#pragma unroll 1
      for (int idx = tid; idx < n; idx += kNT) {
        const int c = idx / NV, v = idx - c * NV;
        float* dst = Xs + c * PC + 4 * v;
        const TX* src = Xb + (int64_t)c * HW + 4 * v;
        if (4 * v >= nval) {
          *reinterpret_cast<float4*>(dst) = make_float4(0.f, 0.f, 0.f, 0.f);
        } else if constexpr (kBulk) {
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
        } else {
          *reinterpret_cast<float4*>(dst) = ld4<TX>(src);
        }
      }
    }
    fac_wait();
    if constexpr (kBulkC) {
      if (!cta_wait_tile(&s_bar, &s_flag, p.status, p.wait_ns)) return;
    } else {
      __syncthreads();
    }
    project_channels<HWC, PC, R>(Xs, U2s, Vp, V2s, C);
    // expansion: P2[c,:] = sum_hw X[c,hw] V2[hw,:], one channel row per thread
    float* P2 = p.Pp[1] + (int64_t)bid * C * p.r[1];
    for (int c = tid; c < C; c += kNT) {
      const float* row = Xs + c * PC;
      float acc[R];
#pragma unroll
      for (int j = 0; j < R; ++j) acc[j] = 0.f;
      if constexpr (NQ == 1) {
#pragma unroll 7
        for (int hw = 0; hw < HWC; ++hw) fma_row<R>(acc, row[hw], V2s + hw * R);
      } else {
#pragma unroll 2
        for (int hw = 0; hw < HWC; hw += 4) {
          const float4 x = *reinterpret_cast<const float4*>(row + hw);
          fma_row<R>(acc, x.x, V2s + hw * R);
          fma_row<R>(acc, x.y, V2s + (hw + 1) * R);
          fma_row<R>(acc, x.z, V2s + (hw + 2) * R);
          fma_row<R>(acc, x.w, V2s + (hw + 3) * R);
        }
      }
#pragma unroll
      for (int j = 0; j < R; ++j)
        if (j < p.r[1]) P2[c * p.r[1] + j] = acc[j];
    }
  }
}

// A launch over several layers at once: the CTAs of layer l are [first[l], first[l + 1]).
constexpr int kMaxBatch = 8;
template <typename Args>
struct SmBatch {
  Args a[kMaxBatch];
  int first[kMaxBatch + 1];
  int n;
};
template <typename Args>
__device__ __forceinline__ int batch_layer(const SmBatch<Args>& b, int bid) {
  int l = 0;
  while (l + 1 < b.n && bid >= b.first[l + 1]) ++l;
  return l;
}

template <int S, int R, typename TX>
__global__ void __launch_bounds__(kNT, 2) k_sm_pass1(const __grid_constant__ SmPass1Args p) {
  sm_pass1_cta<S, R, TX>(p, (int)blockIdx.x);
}
template <int S, int R, typename TX>
__global__ void __launch_bounds__(kNT, 2) k_sm_pass1_b(const __grid_constant__ SmBatch<SmPass1Args> b) {
  const int l = batch_layer(b, (int)blockIdx.x);
  sm_pass1_cta<S, R, TX>(b.a[l], (int)blockIdx.x - b.first[l]);
}

// ---------------------------------------------------------------------------------------------
// k_sm_reduce: CTA (c, m) sums rows [16 c, 16 c + 16) of the per-tile partials of P_m in fp64 in a
// fixed order (thread (e, sg) takes the partials s == sg (mod SG); the SG sums meet in shared memory
// in index order), stores them in fp64 and adds its share of P_m^T P_m.  A mode whose partials are
// Gram matrices A_m A_m^T (a <= 16) is summed the same way, a slice of the a x a elements per CTA.
// With args.factor the last CTA of a mode to finish then factors the mode once for all CTAs of the
// core kernel: it sums the shares of P_m^T P_m (a Gram mode: forms P_m = G_m U_m^prev first), and
// leaves the Cholesky factor R_m and 1 / diag(R_m) in args.Rf.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void sm_reduce_cta(const SmReduceArgs& args, const int c, const int mode) {
  constexpr int RM = 8, RPC = kRedRows;
  const SmReduceMode M = args.m[mode];   // a copy in registers: reading the fields through the parameter each time cost 9 % of a step
  pdl_launch_dependents();
  if (c >= M.nchunk) return;
  pdl_wait();                                      // the partials come from the previous kernel
  __shared__ double part[kRedNT];
  __shared__ double Ps[RPC][RM];
  const int tid = threadIdx.x;
  const int r = M.r, a = M.a;
  // a Gram mode: CTA c sums elements [c*per, c*per + per) of G_m = A_m A_m^T over the tiles;
  // otherwise rows [16 c, 16 c + 16) of P_m
  const int per = M.gram ? (a * a + M.nchunk - 1) / M.nchunk : 0;
  const int first = M.gram ? c * per : c * RPC * r;
  const int row0 = c * RPC;
  const int nrow = (a - row0 < RPC) ? (a - row0) : RPC;
  const int E = M.gram ? ((a * a - first < per) ? a * a - first : per) : nrow * r;   // <= 128
  const int64_t stride = M.gram ? (int64_t)a * a : (int64_t)a * r;
  int EP = 32;
  while (EP < E) EP <<= 1;
  const int SG = kRedNT / EP;
  {
    const int e = tid & (EP - 1), sg = tid >> (31 - __clz(EP));
    double acc = 0.0;
    if (e < E) {
      const float* ptr = M.Pp + first + e;
#pragma unroll 8
      for (int s = sg; s < M.nsplit; s += SG) acc += (double)__ldcg(ptr + s * stride);
    }
    part[tid] = acc;
  }
  for (int idx = tid; idx < RPC * RM; idx += kRedNT) Ps[idx / RM][idx % RM] = 0.0;
  __syncthreads();
  if (tid < E) {
    double v = 0.0;
    for (int sg = 0; sg < SG; ++sg) v += part[sg * EP + tid];
    M.Pred[first + tid] = v;                       // P_m rows, or G_m elements for a Gram mode
    if (!M.gram) {
      const FDiv dr(r);
      int k, j;
      dr.divmod(tid, k, j);
      Ps[k][j] = v;
    }
  }
  if (!M.gram) {
    __syncthreads();
    if (tid < r * r) {
      const FDiv dr(r);
      int i, j;
      dr.divmod(tid, i, j);
      double g = 0.0;
      if (j >= i) {
#pragma unroll 4
        for (int rl = 0; rl < RPC; ++rl) g = fma(Ps[rl][i], Ps[rl][j], g);
      }
      M.Gp[((int64_t)c * r + i) * r + j] = g;
    }
  }
  if (!args.factor) return;
  // ---- the last CTA of a mode to get here factors the mode once for every CTA of the core kernel:
  // G_m = P_m^T P_m = R_m^T R_m (Cholesky), stored as the rows of R_m and 1 / diag(R_m)
  __shared__ int s_last;
  __shared__ double Gq[8][RM * RM];
  __shared__ double Gs[RM][RM + 1];
  __shared__ double Dinv[RM];
  __shared__ double Gfull[16 * 16];
  __shared__ double Pm[16][RM];
  __shared__ float Ups[16 * RM];
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(args.counter + mode, 1) == M.nchunk - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const int lane = tid & 31, warp = tid >> 5;
  if (!M.gram) {
    // warp q sums the shares of the chunks == q (mod 8); the eight sums meet in index order
    for (int e = lane; e < r * r && warp < 8; e += 32) {
      double g = 0.0;
#pragma unroll 8
      for (int cc = warp; cc < M.nchunk; cc += 8) g += __ldcg(M.Gp + (int64_t)cc * r * r + e);
      Gq[warp][e] = g;
    }
    __syncthreads();
    if (tid < r * r) {
      double g = Gq[0][tid];
#pragma unroll
      for (int q = 1; q < 8; ++q) g += Gq[q][tid];
      const int i = tid / r, k = tid - i * r;
      Gs[i][k] = g;
    }
  } else {
    // Gram mode (a <= 16): P_m = G_m U_m^prev (Algorithm 1: A_m (A_m^T U)), kept in fp64 for the row
    // solves of the core kernel, then its Gram matrix
    for (int e = tid; e < a * a; e += kRedNT) Gfull[e] = __ldcg(M.Pred + e);
    for (int e = tid; e < a * r; e += kRedNT) Ups[e] = __ldg(M.U_prev + e);
    __syncthreads();
    if (tid < a * r) {
      const int k = tid / r, j = tid - k * r;
      double v = 0.0;
      for (int k2 = 0; k2 < a; ++k2) v = fma(Gfull[k * a + k2], (double)Ups[k2 * r + j], v);
      Pm[k][j] = v;
      M.Pg[tid] = v;
    }
    __syncthreads();
    if (tid < r * r) {
      const int i = tid / r, k = tid - i * r;
      double g = 0.0;
      if (k >= i)
        for (int kk = 0; kk < a; ++kk) g = fma(Pm[kk][i], Pm[kk][k], g);
      Gs[i][k] = g;
    }
  }
  __syncthreads();
  if (warp == 0) {
    // right-looking Cholesky G = R^T R on one warp; lane owns entries e0 = lane and e1 = lane + 32
    const int e0 = lane, e1 = lane + 32;
    const int i0 = e0 / r, k0 = e0 - i0 * r, i1 = e1 / r, k1 = e1 - i1 * r;
    const bool in0 = e0 < r * r, in1 = e1 < r * r;
    double trace = 0.0;
    for (int i = 0; i < r; ++i) trace += Gs[i][i];
    const double floor_d = 1e-12 * trace;
    for (int j = 0; j < r; ++j) {
      double d = Gs[j][j];
      if (!(d > floor_d)) {
        if (lane == 0) atomicMax(args.status, (int)ASI_ERR_RANK_DEFICIENT);
        d = (floor_d > 0.0) ? floor_d : 1.0;
      }
      const double inv = rsqrt(d);
      __syncwarp();
      if (lane == j) {
        Gs[j][j] = d * inv;
        Dinv[j] = inv;
      } else if (lane > j && lane < r) {
        Gs[j][lane] *= inv;
      }
      __syncwarp();
      if (in0 && i0 > j && k0 >= i0) Gs[i0][k0] -= Gs[j][i0] * Gs[j][k0];
      if (in1 && i1 > j && k1 >= i1) Gs[i1][k1] -= Gs[j][i1] * Gs[j][k1];
      __syncwarp();
    }
    double* Rf = args.Rf + mode * kRfStride;
    if (in0) Rf[i0 * RM + k0] = Gs[i0][k0];
    if (in1) Rf[i1 * RM + k1] = Gs[i1][k1];
    if (lane < r) Rf[RM * RM + lane] = Dinv[lane];
    if (lane == 0) args.counter[mode] = 0;
  }
}

__global__ void __launch_bounds__(kRedNT) k_sm_reduce(const __grid_constant__ SmReduceArgs args) {
  sm_reduce_cta(args, (int)blockIdx.x, (int)blockIdx.y);
}
__global__ void __launch_bounds__(kRedNT) k_sm_reduce_b(const __grid_constant__ SmBatch<SmReduceArgs> b) {
  const int l = batch_layer(b, (int)blockIdx.x);
  sm_reduce_cta(b.a[l], (int)blockIdx.x - b.first[l], (int)blockIdx.y);
}

// <<<>>> with the programmatic-stream-serialization attribute
template <typename Arg>
static cudaError_t launch_dependent(void (*kernel)(Arg), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    const Arg& arg) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, arg);
}

cudaError_t launch_sm_reduce(const SmReduceArgs& p, int nd, int max_chunks, cudaStream_t st) {
  double bytes = 0.0;
  for (int m = 0; m < nd; ++m)
    bytes += 4.0 * p.m[m].nsplit * p.m[m].a * (p.m[m].gram ? p.m[m].a : p.m[m].r) + 8.0 * p.m[m].a * p.m[m].r;
  ProfScope prof(ASI_K_QR, st, bytes);
  dim3 grid((unsigned)max_chunks, (unsigned)nd);
  return launch_dependent(k_sm_reduce, grid, dim3(kRedNT), 0, st, p);
}

// ---------------------------------------------------------------------------------------------
// k_sm_core.  Tile t = [all B x J] as in role B of the first pass.
//   prologue (while the tile is in flight): one thread per needed factor row fetches the fp64 row of
//     P_m and solves u = p R_m^{-1} with the Cholesky factor the reduction kernel left -- all of U_1,
//     the tile's own rows of U_2, all of U_3 and U_4 -- and the owners write them to U_new;
//   W[i][c,h,w] = sum_b U1[b,i] X[b][c,h,w];  Y[i,j][h,w] = sum_c U2[c,j] W[i][c,h,w];
//   T[i,j,k,l] = Y x_3 U3^T x_4 U4^T  -> per-tile partial core, summed in two ordered levels.
// ---------------------------------------------------------------------------------------------
template <int S, int R, typename TX>
__device__ __forceinline__ void sm_core_cta(const SmCoreArgs& p, const int bid) {
  constexpr int HW = S * S;
  constexpr int CC = (S == 7) ? 4 : 1;
  constexpr int J = CC * HW;
  constexpr int PJ = pitch4(J);
  constexpr int NH = batch_groups(kNT, J);
  extern __shared__ __align__(128) float smem[];
  __shared__ int s_last;
  __shared__ double Rs[4][kRfStride];   // per mode: rows of R_m (pitch 8), then 1 / diag(R_m) at [64..]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int B = p.B, C = p.C, tile = bid;
  const int r1 = p.r[0], r2 = p.r[1], r3 = p.r[2], r4 = p.r[3];
  float* Xs = smem;                     // [B][PJ]
  float* U1s = Xs + B * PJ;             // [B][R]
  float* U2s = U1s + B * R;             // [CC][R]
  float* U3s = U2s + CC * R;            // [S][R]
  float* U4s = U3s + S * R;             // [S][R]
  float* Ws = U4s + S * R;              // [J][R]
  float* part = Ws + J * R;             // [NH][J][R]
  float* Ysm = part + NH * J * R;       // [R R][HW]
  float* T3s = Ysm + R * R * HW;        // [R R][R][S]
  stage_tile_begin<TX>(reinterpret_cast<const TX*>(p.act) + (int64_t)tile * J, (int64_t)C * HW, Xs, B, J, PJ);
  cp_async_commit();
  pdl_wait();                           // P_m and the Gram shares come from the reduction kernel
  // ---- the factor row this thread will solve for: [U1: B rows][U2: CC rows][U3: S][U4: S]
  const int nrows = B + CC + 2 * S;     // <= kNT (checked when the plan picks this kernel)
  int rm = 0, rk = 0, rr = 0;
  float* rdst = nullptr;
  bool rowner = false;
  double prow[R];
#pragma unroll
  for (int j = 0; j < R; ++j) prow[j] = 0.0;
  if (tid < nrows) {
    if (tid < B) { rm = 0; rk = tid; rdst = U1s + rk * R; rowner = tile == 0; }
    else if (tid < B + CC) { rm = 1; rk = tile * CC + (tid - B); rdst = U2s + (tid - B) * R; rowner = true; }
    else if (tid < B + CC + S) { rm = 2; rk = tid - B - CC; rdst = U3s + rk * R; rowner = tile == 0; }
    else { rm = 3; rk = tid - B - CC - S; rdst = U4s + rk * R; rowner = tile == 0; }
    rr = p.r[rm];
    const double* src = p.Pred[rm] + (int64_t)rk * rr;
#pragma unroll
    for (int j = 0; j < R; ++j)
      if (j < rr) prow[j] = __ldcg(src + j);
  }
  // ---- the Cholesky factors of the four modes (computed once, by the reduction kernel)
  for (int e = tid; e < 4 * kRfStride; e += kNT) (&Rs[0][0])[e] = __ldcg(p.Rf + e);
  __syncthreads();
  if (tid < nrows) {
    float* gdst = p.U_new + p.u_off[rm] + (int64_t)rk * rr;
    double q[R];
#pragma unroll
    for (int j = 0; j < R; ++j) {
      float out = 0.f;
      if (j < rr) {
        double v = prow[j];
#pragma unroll
        for (int i = 0; i < R; ++i)
          if (i < j) v -= q[i] * Rs[rm][i * 8 + j];
        v *= Rs[rm][64 + j];
        q[j] = v;
        out = (float)v;
        if (rowner) gdst[j] = out;
      }
      rdst[j] = out;
    }
  }
  cp_async_wait<0>();
  __syncthreads();
  project_batch<R>(Xs, PJ, U1s, B, J, part, Ws, tid, kNT, 0);
  // Y[(i,j)][hw] = sum_cl U2[cl][j] W[cl*HW + hw][i]
  const int r12 = r1 * r2;
  const FDiv d_r2(r2), d_r3(r3), d_r4(r4);
  for (int idx = tid; idx < r12 * HW; idx += kNT) {
    const int hw = idx % HW, ij = idx / HW;
    int i, j;
    d_r2.divmod(ij, i, j);
    float s = 0.f;
#pragma unroll
    for (int cl = 0; cl < CC; ++cl) s = fmaf(U2s[cl * R + j], Ws[(cl * HW + hw) * R + i], s);
    Ysm[ij * HW + hw] = s;
  }
  __syncthreads();
  // T3[(i,j)][k][w] = sum_h Y[(i,j)][h,w] U3[h][k]
  for (int idx = tid; idx < r12 * r3 * S; idx += kNT) {
    const int w = idx % S;
    int ij, k;
    d_r3.divmod(idx / S, ij, k);
    float s = 0.f;
#pragma unroll
    for (int h = 0; h < S; ++h) s = fmaf(Ysm[ij * HW + h * S + w], U3s[h * R + k], s);
    T3s[(ij * R + k) * S + w] = s;
  }
  __syncthreads();
  // T[(i,j)][k][l] = sum_w T3[(i,j)][k][w] U4[w][l]
  const int ce = r12 * r3 * r4;
  for (int idx = tid; idx < ce; idx += kNT) {
    int t34, l, ij, k;
    d_r4.divmod(idx, t34, l);
    d_r3.divmod(t34, ij, k);
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < S; ++w) s = fmaf(T3s[(ij * R + k) * S + w], U4s[w * R + l], s);
    p.Tp[(int64_t)tile * ce + idx] = s;
  }
  // Two-level sum of the per-tile cores, both levels in index order: the last CTA of every group of
  // p.gs tiles sums that group, the last group to finish sums the groups.
  __threadfence();
  __syncthreads();
  const int grp = tile / p.gs, gfirst = grp * p.gs;
  const int gsize = (p.n_tiles - gfirst < p.gs) ? p.n_tiles - gfirst : p.gs;
  const int ngroups = (p.n_tiles + p.gs - 1) / p.gs;
  if (tid == 0) s_last = (atomicAdd(p.gcount + grp, 1) == gsize - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  for (int idx = tid; idx < ce; idx += kNT) {
    const float* src = p.Tp + (int64_t)gfirst * ce + idx;
    float s = 0.f;
    for (int t0 = 0; t0 < gsize; t0 += 8) {
      float v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = (t0 + k < gsize) ? __ldcg(src + (int64_t)(t0 + k) * ce) : 0.f;
#pragma unroll
      for (int k = 0; k < 8; ++k) s += v[k];
    }
    p.Tg[(int64_t)grp * ce + idx] = s;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    p.gcount[grp] = 0;
    s_last = (atomicAdd(p.counter, 1) == ngroups - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (ce * 2 <= kNT) {
    // few core elements: thread (e, q) sums the groups == q (mod nq) of element e, the nq sums meet
    // in index order (shared memory: the tile is no longer needed)
    int nq = kNT / ce;
    nq = nq > 8 ? 8 : nq;
    float* fold = smem;                              // [nq][ce]
    if (tid < nq * ce) {
      const int q = tid / ce, e = tid - q * ce;
      const float* src = p.Tg + e;
      float s = 0.f;
      for (int g0 = q; g0 < ngroups; g0 += 8 * nq) {
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) v[k] = (g0 + k * nq < ngroups) ? __ldcg(src + (int64_t)(g0 + k * nq) * ce) : 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) s += v[k];
      }
      fold[tid] = s;
    }
    __syncthreads();
    if (tid < ce) {
      float s = fold[tid];
      for (int q = 1; q < nq; ++q) s += fold[q * ce + tid];
      p.core[tid] = s;
    }
  } else {
    for (int idx = tid; idx < ce; idx += kNT) {
      const float* src = p.Tg + idx;
      float s = 0.f;
      for (int g0 = 0; g0 < ngroups; g0 += 16) {
        float v[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) v[k] = (g0 + k < ngroups) ? __ldcg(src + (int64_t)(g0 + k) * ce) : 0.f;
#pragma unroll
        for (int k = 0; k < 16; ++k) s += v[k];
      }
      p.core[idx] = s;
    }
  }
  if (tid == 0) *p.counter = 0;
}

template <int S, int R, typename TX>
__global__ void __launch_bounds__(kNT) k_sm_core(const __grid_constant__ SmCoreArgs p) {
  sm_core_cta<S, R, TX>(p, (int)blockIdx.x);
}
template <int S, int R, typename TX>
__global__ void __launch_bounds__(kNT) k_sm_core_b(const __grid_constant__ SmBatch<SmCoreArgs> b) {
  const int l = batch_layer(b, (int)blockIdx.x);
  sm_core_cta<S, R, TX>(b.a[l], (int)blockIdx.x - b.first[l]);
}

// ---------------------------------------------------------------------------------------------
// k_sm_wgrad: CTA owns cpb consecutive output channels, i.e. the dY tile [B x J], J = cpb*Ho*Wo
// contiguous values per sample (staged by 16-byte cp.async when fp32 and 16-byte aligned).
//   Z3 = core x_3 U3 x_4 U4 (recomputed per CTA while the tile is in flight);
//   Z1 = dY x_1 U1^T on the CTA's channels;
//   Z4[c',j,kh,kw] = sum_{i,h',w'} Z1[i,c',h',w'] Z3pad[i,j,h's+kh-p,w's+kw-p];  dW = Z4 x_2 U2.
// ---------------------------------------------------------------------------------------------
// Term 5: dW[c0+cl, c, t] = sum_j Z4[cl][t][j] U2[(g cg + c), j].  The rows of Z4 are the same for every
// thread, so each 16-byte shared-memory read of one costs a full warp-wide transfer; a thread therefore
// owns up to four input channels (their rows of U2 stay in registers) and every row of Z4 it reads feeds
// four dot products (fewer, busier threads: the shared-memory pipe is the limit).  p.ncl output channels
// are expanded per round, one thread group each, into a staging block [ncl][cg x kk] in shared memory
// that then leaves for global memory in one piece per channel -- by the bulk-copy engine
// (cp.async.bulk shared -> global) when a channel's block is 16-byte sized and aligned, else by
// coalesced stores.  With more than one round there are two staging blocks, so that a round's stores
// run under the next round's arithmetic: the write of dW by all CTAs at once is DRAM-bound.
template <int R>
__device__ __forceinline__ void wgrad_expand_rows(const SmWgradArgs& p, const float* __restrict__ Z4s,
                                                  const float* __restrict__ U2s, float* stage, int c0) {
  const int kk = p.kh * p.kw;
  const int cg = p.C / p.groups, og = p.Cout / p.groups;
  const int tid = threadIdx.x;
  const int nblk = cg * kk;
  const int lg = (p.ncl == 4) ? 2 : (p.ncl == 2 ? 1 : 0);
  const int TG = kNT >> lg;                          // threads per output channel
  const int grp = tid / TG, tg = tid - grp * TG;
  int ta = (((cg + 3) >> 2) + 31) & ~31;             // active threads of a group: four channels each
  if (ta > TG) ta = TG;
  const int rounds = p.cpb / p.ncl;
#pragma unroll 1
  for (int rd = 0; rd < rounds; ++rd) {
    const int cl = rd * p.ncl + grp;
    const int co = c0 + cl;
    const int g = co / og;
    float* dw = p.dW + (int64_t)(c0 + rd * p.ncl) * nblk;
    const float* u2 = U2s + (int64_t)g * cg * R;
    float* buf = stage + (rd & 1) * p.ncl * nblk;
    if (p.bulk_store && rd >= 2) {
      if (tid == 0) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
      __syncthreads();
    }
    float* out = buf + grp * nblk;
    const float* z = Z4s + cl * kk * R;
#pragma unroll 1
    for (int cb = tg; cb < cg && tg < ta; cb += 4 * ta) {
      float u[4][R];
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        const int c = cb + m * ta;
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
          if (c < cg) v = *reinterpret_cast<const float4*>(u2 + c * R + j);
          u[m][j] = v.x; u[m][j + 1] = v.y; u[m][j + 2] = v.z; u[m][j + 3] = v.w;
        }
      }
#pragma unroll 3
      for (int t = 0; t < kk; ++t) {
        float v[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          const float4 zz = *reinterpret_cast<const float4*>(z + t * R + j);
#pragma unroll
          for (int m = 0; m < 4; ++m) {
            v[m] = fmaf(zz.x, u[m][j], v[m]);
            v[m] = fmaf(zz.y, u[m][j + 1], v[m]);
            v[m] = fmaf(zz.z, u[m][j + 2], v[m]);
            v[m] = fmaf(zz.w, u[m][j + 3], v[m]);
          }
        }
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int c = cb + m * ta;
          if (c < cg) out[c * kk + t] = v[m];
        }
      }
    }
    if (p.bulk_store) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncthreads();
      if (tid == 0) {
        for (int q = 0; q < p.ncl; ++q)
          asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dw + (int64_t)q * nblk),
                       "r"(smem_u32(buf + q * nblk)), "r"((uint32_t)nblk * 4u)
                       : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
      }
    } else {
      __syncthreads();
      for (int idx = tid; idx < p.ncl * nblk; idx += kNT) dw[idx] = buf[idx];
    }
  }
  if (p.bulk_store && tid == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}

template <int R, typename TX>
__device__ __forceinline__ void sm_wgrad_cta(const SmWgradArgs& p, const int bid) {
  extern __shared__ __align__(128) float smem[];
  const int tid = threadIdx.x;
  const int r1 = p.r[0], r2 = p.r[1], r3 = p.r[2], r4 = p.r[3];
  const int H = p.H, W = p.W, HW = H * W, HoWo = p.Ho * p.Wo, kk = p.kh * p.kw;
  const int J = p.cpb * HoWo;                        // dY columns of this CTA, contiguous per sample
  const int PJ = p.pj;
  const int NH = batch_groups(kNT, J);
  const int c0 = bid * p.cpb;
  const int n_out = p.cpb * r2 * kk;
  // staging blocks of term 5 reuse the tile's space: ncl channels per round, doubled when rounds follow
  const int n_stage = (p.cpb > p.ncl ? 2 : 1) * p.ncl * (p.C / p.groups) * kk;
  float* Ys = smem;                                  // [B][PJ]
  float* U1s = Ys + ((p.B * PJ > n_stage ? p.B * PJ : n_stage) + 3) / 4 * 4;   // [B][R]
  float* U2s = U1s + p.B * R;                        // [C][R]
  float* Z1s = U2s + p.C * R;                        // [J][R]
  float* part = Z1s + J * R;                         // [NH][J][R] (NH > 1 only)
  float* Ss = part + (NH > 1 ? NH : 0) * J * R;      // [r1 r2][R (l)][R (k)]: core, modes 3 and 4 swapped, zero-padded
  float* U3s = Ss + r1 * r2 * R * R;                 // [H][R]
  float* U4s = U3s + H * R;                          // [W][R]
  float* Tm = U4s + W * R;                           // [r1 r2][H][R]
  const int Hp = H + 2 * p.ph, Wp = W + 2 * p.pw;    // Z3 is kept zero-padded: term 4 needs no bounds logic
  float* Z3s = Tm + r1 * r2 * H * R;                 // [r1 r2][Hp][Wp]
  float* Z4s = smem + ((Z3s + r1 * r2 * Hp * Wp) - smem + 3) / 4 * 4;   // [cpb][kk][R], 16-byte aligned (rank index fastest, zero-padded)
  float* red = Z4s + p.cpb * kk * R;                 // [G4][cpb][r2 kk]

  const TX* dY = reinterpret_cast<const TX*>(p.dY) + (int64_t)c0 * HoWo;
  const int64_t sstride = (int64_t)p.Cout * HoWo;
  const bool bulk = std::is_same<TX, float>::value && p.bulk;
  {
#pragma unroll 1
    for (int idx = tid; idx < r1 * r2 * R * R; idx += kNT) {      // Ss[ij][l][k] = core[ij][k][l]
      const int k = idx % R, l = (idx / R) % R, ij = idx / (R * R);
      const bool in = k < r3 && l < r4;
      cp_async4(Ss + idx, p.core + (in ? (ij * r3 + k) * r4 + l : 0), in ? 4 : 0);
    }
    fac_issue_padded<R>(p.U + p.u_off[2], U3s, H, r3);
    fac_issue_padded<R>(p.U + p.u_off[3], U4s, W, r4);
    fac_issue_padded<R>(p.U + p.u_off[0], U1s, p.B, r1);
    fac_issue_padded<R>(p.U + p.u_off[1], U2s, p.C, r2);
    cp_async_commit();                               // group 1: factors and core; group 0 (younger): the tile
    if constexpr (std::is_same<TX, float>::value) {
      if (bulk) stage_rows_async(Ys, reinterpret_cast<const float*>(dY), p.B, J, sstride, PJ);
    }
    if (!bulk) {
      for (int idx = tid; idx < p.B * J; idx += kNT) {
        const int b = idx / J, j = idx - b * J;
        Ys[b * PJ + j] = to_f(dY[b * sstride + j]);
      }
    }
    cp_async_commit();
    cp_async_wait<1>();
  }
  __syncthreads();
  // terms 2-3: Tm[ij][h][l] = sum_k S[ij][k][l] U3[h][k];  Z3[ij][h][w] = sum_l Tm[ij][h][l] U4[w][l]
  // (rank indices padded to R with zeros: every sum is a fixed-length dot product of 16-byte reads)
  const FDiv d_H(H), d_Wp(Wp), d_Hp(Hp), d_kk(kk), d_kw(p.kw);
  for (int idx = tid; idx < r1 * r2 * H * R; idx += kNT) {
    const int l = idx % R, t0 = idx / R;
    int ij, h;
    d_H.divmod(t0, ij, h);
    const float* sp = Ss + (ij * R + l) * R;
    const float* up = U3s + h * R;
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < R; k += 4) {
      const float4 a = *reinterpret_cast<const float4*>(sp + k), b = *reinterpret_cast<const float4*>(up + k);
      s = fmaf(a.x, b.x, s); s = fmaf(a.y, b.y, s); s = fmaf(a.z, b.z, s); s = fmaf(a.w, b.w, s);
    }
    Tm[idx] = s;
  }
  __syncthreads();
  for (int idx = tid; idx < r1 * r2 * Hp * Wp; idx += kNT) {
    int t0, wp, ij, hp;
    d_Wp.divmod(idx, t0, wp);
    d_Hp.divmod(t0, ij, hp);
    const int h = hp - p.ph, w = wp - p.pw;
    float s = 0.f;
    if (h >= 0 && h < H && w >= 0 && w < W) {
      const float* tp = Tm + (ij * H + h) * R;
      const float* up = U4s + w * R;
#pragma unroll
      for (int l = 0; l < R; l += 4) {
        const float4 a = *reinterpret_cast<const float4*>(tp + l), b = *reinterpret_cast<const float4*>(up + l);
        s = fmaf(a.x, b.x, s); s = fmaf(a.y, b.y, s); s = fmaf(a.z, b.z, s); s = fmaf(a.w, b.w, s);
      }
    }
    Z3s[idx] = s;
  }
  cp_async_wait<0>();
  __syncthreads();
  // term 1: Z1[j,:] = sum_b dY[b, c0*HoWo + j] U1[b,:]
  project_batch<R>(Ys, PJ, U1s, p.B, J, part, Z1s, tid, kNT, 0);
  // term 4: thread (n, g): outputs n = (j, kh, kw) of all cpb channels and every G-th pair (i, h') of
  // the reduction; one Z3 operand feeds cpb FMAs.  The G partial sums meet in order.
  const int N4 = r2 * kk;
  int G4 = (N4 <= kNT) ? kNT / N4 : 1;
  if (G4 > r1 * p.Ho) G4 = r1 * p.Ho;
  const FDiv d_Ho(p.Ho), d_N4(N4);
  for (int it = tid; it < N4 * G4; it += kNT) {
    int g, n, j, tt, ky, kx;
    d_N4.divmod(it, g, n);
    d_kk.divmod(n, j, tt);
    d_kw.divmod(tt, ky, kx);
    const float* z3 = Z3s + (j * Hp + ky) * Wp + kx;
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int q = g; q < r1 * p.Ho; q += G4) {
      int i, ho;
      d_Ho.divmod(q, i, ho);
      const float* z1r = Z1s + ho * p.Wo * R + i;
      const float* z3r = z3 + (i * r2 * Hp + ho * p.sh) * Wp;
#pragma unroll 7
      for (int wo = 0; wo < p.Wo; ++wo) {
        const float b = z3r[wo * p.sw];
#pragma unroll
        for (int cl = 0; cl < 4; ++cl)
          if (cl < p.cpb) acc[cl] = fmaf(z1r[(cl * HoWo + wo) * R], b, acc[cl]);
      }
    }
#pragma unroll
    for (int cl = 0; cl < 4; ++cl)
      if (cl < p.cpb) red[(g * p.cpb + cl) * N4 + n] = acc[cl];
  }
  __syncthreads();
  for (int o = tid; o < p.cpb * kk * R; o += kNT) {
    const int j = o % R, ct = o / R;                 // ct = cl*kk + t
    int cl, tt;
    d_kk.divmod(ct, cl, tt);
    float v = 0.f;
    if (j < r2)
      for (int g = 0; g < G4; ++g) v += red[(g * p.cpb + cl) * N4 + j * kk + tt];
    Z4s[o] = v;
  }
  __syncthreads();
  // term 5: dW[c0+cl, c, t] = sum_j Z4[cl][j][t] U2[(g cg + c), j]
  wgrad_expand_rows<R>(p, Z4s, U2s, Ys, c0);
}

template <int R, typename TX>
__global__ void __launch_bounds__(kNT) k_sm_wgrad(const __grid_constant__ SmWgradArgs p) {
  sm_wgrad_cta<R, TX>(p, (int)blockIdx.x);
}
template <int R, typename TX>
__global__ void __launch_bounds__(kNT) k_sm_wgrad_b(const __grid_constant__ SmBatch<SmWgradArgs> b) {
  const int l = batch_layer(b, (int)blockIdx.x);
  sm_wgrad_cta<R, TX>(b.a[l], (int)blockIdx.x - b.first[l]);
}

// ---------------------------------------------------------------------------------------------
// host-side launchers
// ---------------------------------------------------------------------------------------------
int sm_pass1_role_c_ctas(int S, int B) { return (S == 7) ? B : 4 * B; }

size_t sm_pass1_smem(int S, int R, int B, int C) {
  const int HW = S * S, CC = (S == 7) ? 4 : 1, J = CC * HW, PJ = pitch4(J);
  const int NH1 = batch_groups(kNG, J);
  const size_t role_b = (size_t)B * PJ + (size_t)B * R + 2 * S * R + (size_t)J * R +
                        (NH1 > 1 ? (size_t)NH1 * J * R : 0) + 24 * 32;
  const int HWC = role_c_hwc(S), PC = role_c_pitch(S);
  const int G = kNT / HWC;
  const size_t vp = (C >= (G - 1) * HWC) ? 0 : (size_t)(G - 1) * HWC * R;
  const size_t role_c = (size_t)((C * PC + 3) & ~3) + (size_t)C * R + (size_t)HWC * R + vp;
  return 4 * (role_b > role_c ? role_b : role_c);
}

size_t sm_core_smem(int S, int R, int B) {
  const int HW = S * S, CC = (S == 7) ? 4 : 1, J = CC * HW, PJ = pitch4(J);
  const int NH = batch_groups(kNT, J);
  return 4 * ((size_t)B * PJ + (size_t)B * R + (size_t)CC * R + 2 * S * R + (size_t)J * R + (size_t)NH * J * R +
              (size_t)R * R * HW + (size_t)R * R * R * S);
}

int sm_core_max_rows() { return kNT; }

int sm_wgrad_pitch(int J) { return pitch4(J); }

size_t sm_wgrad_smem(const SmWgradArgs& p, int R) {
  const int r1 = p.r[0], r2 = p.r[1];
  const int J = p.cpb * p.Ho * p.Wo, kk = p.kh * p.kw;
  const int N4 = r2 * kk;
  const int NH = batch_groups(kNT, J);
  const size_t tile = (size_t)p.B * pitch4(J),
               stage = (size_t)(p.cpb > p.ncl ? 2 : 1) * p.ncl * (p.C / p.groups) * kk;
  size_t n = ((tile > stage ? tile : stage) + 3) / 4 * 4 + (size_t)p.B * R + (size_t)p.C * R + (size_t)J * R +
             (NH > 1 ? (size_t)NH * J * R : 0) + (size_t)r1 * r2 * R * R + (size_t)p.H * R + (size_t)p.W * R +
             (size_t)r1 * r2 * p.H * R + ((size_t)r1 * r2 * (p.H + 2 * p.ph) * (p.W + 2 * p.pw) + 3) / 4 * 4 +
             (size_t)p.cpb * kk * R + (size_t)p.cpb * (N4 > kNT ? N4 : kNT);
  return 4 * n + 64;
}

template <int S, int R, typename TX>
static cudaError_t launch_pass1_t(const SmPass1Args& p, cudaStream_t st) {
  const size_t smem = sm_pass1_smem(S, R, p.B, p.C);   // the default limit counts static shared memory too: always opt in
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_sm_pass1<S, R, TX>), smem);
  if (e != cudaSuccess) return e;
  k_sm_pass1<S, R, TX><<<p.n_tiles_b + sm_pass1_role_c_ctas(S, p.B), kNT, smem, st>>>(p);
  return cudaGetLastError();
}

template <int S, int R, typename TX>
static cudaError_t launch_core_t(const SmCoreArgs& p, cudaStream_t st) {
  const size_t smem = sm_core_smem(S, R, p.B);
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_sm_core<S, R, TX>), smem);
  if (e != cudaSuccess) return e;
  return launch_dependent(k_sm_core<S, R, TX>, dim3(p.n_tiles), dim3(kNT), smem, st, p);
}

template <int R, typename TX>
static cudaError_t launch_wgrad_t(const SmWgradArgs& p, cudaStream_t st) {
  const size_t smem = sm_wgrad_smem(p, R);
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_sm_wgrad<R, TX>), smem);
  if (e != cudaSuccess) return e;
  k_sm_wgrad<R, TX><<<p.Cout / p.cpb, kNT, smem, st>>>(p);
  return cudaGetLastError();
}

#define ASI_DISPATCH_SR(FN, ARGS)                                              \
  do {                                                                         \
    if (S == 7) {                                                              \
      if (R == 4) return bf16 ? FN<7, 4, __nv_bfloat16>(ARGS, st) : FN<7, 4, float>(ARGS, st);   \
      return bf16 ? FN<7, 8, __nv_bfloat16>(ARGS, st) : FN<7, 8, float>(ARGS, st);               \
    }                                                                          \
    if (S == 14) {                                                             \
      if (R == 4) return bf16 ? FN<14, 4, __nv_bfloat16>(ARGS, st) : FN<14, 4, float>(ARGS, st); \
      return bf16 ? FN<14, 8, __nv_bfloat16>(ARGS, st) : FN<14, 8, float>(ARGS, st);             \
    }                                                                          \
    if (R == 4) return bf16 ? FN<16, 4, __nv_bfloat16>(ARGS, st) : FN<16, 4, float>(ARGS, st);   \
    return bf16 ? FN<16, 8, __nv_bfloat16>(ARGS, st) : FN<16, 8, float>(ARGS, st);               \
  } while (0)

cudaError_t launch_sm_pass1(const SmPass1Args& p, int S, int R, bool bf16, cudaStream_t st) {
  const size_t eb = bf16 ? 2 : 4;
  const double bytes = (double)p.B * p.C * S * S * eb;      // the activation, read once
  ProfScope prof(ASI_K_SM_PASS1, st, bytes);
  ASI_DISPATCH_SR(launch_pass1_t, p);
}

cudaError_t launch_sm_core(const SmCoreArgs& p, int S, int R, bool bf16, cudaStream_t st) {
  const size_t eb = bf16 ? 2 : 4;
  ProfScope prof(ASI_K_SM_CORE, st, (double)p.B * p.C * S * S * eb);
  ASI_DISPATCH_SR(launch_core_t, p);
}

cudaError_t launch_sm_wgrad(const SmWgradArgs& p, int R, bool bf16, cudaStream_t st) {
  const size_t eb = bf16 ? 2 : 4;
  ProfScope prof(ASI_K_SM_WGRAD, st,
                 (double)p.B * p.Cout * p.Ho * p.Wo * eb +
                     4.0 * (double)p.Cout * (p.C / p.groups) * p.kh * p.kw);
  if (R == 4) return bf16 ? launch_wgrad_t<4, __nv_bfloat16>(p, st) : launch_wgrad_t<4, float>(p, st);
  return bf16 ? launch_wgrad_t<8, __nv_bfloat16>(p, st) : launch_wgrad_t<8, float>(p, st);
}

// ---------------------------------------------------------------------------------------------
// Batched launches: the same kernels over the tiles of up to kMaxBatch layers of one variant (map size,
// rank bucket, input type) in one grid.  The per-layer argument blocks travel as a kernel parameter; a CTA
// finds its layer from the table of first CTA indices.
// ---------------------------------------------------------------------------------------------
int sm_max_batch() { return kMaxBatch; }

template <int S, int R, typename TX>
static cudaError_t launch_pass1_bt(const SmBatch<SmPass1Args>& b, size_t smem, cudaStream_t st) {
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_sm_pass1_b<S, R, TX>), smem);
  if (e != cudaSuccess) return e;
  k_sm_pass1_b<S, R, TX><<<b.first[b.n], kNT, smem, st>>>(b);
  return cudaGetLastError();
}
template <int S, int R, typename TX>
static cudaError_t launch_core_bt(const SmBatch<SmCoreArgs>& b, size_t smem, cudaStream_t st) {
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_sm_core_b<S, R, TX>), smem);
  if (e != cudaSuccess) return e;
  return launch_dependent(k_sm_core_b<S, R, TX>, dim3(b.first[b.n]), dim3(kNT), smem, st, b);
}
template <int R, typename TX>
static cudaError_t launch_wgrad_bt(const SmBatch<SmWgradArgs>& b, size_t smem, cudaStream_t st) {
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_sm_wgrad_b<R, TX>), smem);
  if (e != cudaSuccess) return e;
  k_sm_wgrad_b<R, TX><<<b.first[b.n], kNT, smem, st>>>(b);
  return cudaGetLastError();
}

#define ASI_DISPATCH_SRB(FN, ARGS, SMEM)                                       \
  do {                                                                         \
    if (S == 7) {                                                              \
      if (R == 4) return bf16 ? FN<7, 4, __nv_bfloat16>(ARGS, SMEM, st) : FN<7, 4, float>(ARGS, SMEM, st);   \
      return bf16 ? FN<7, 8, __nv_bfloat16>(ARGS, SMEM, st) : FN<7, 8, float>(ARGS, SMEM, st);               \
    }                                                                          \
    if (S == 14) {                                                             \
      if (R == 4) return bf16 ? FN<14, 4, __nv_bfloat16>(ARGS, SMEM, st) : FN<14, 4, float>(ARGS, SMEM, st); \
      return bf16 ? FN<14, 8, __nv_bfloat16>(ARGS, SMEM, st) : FN<14, 8, float>(ARGS, SMEM, st);             \
    }                                                                          \
    if (R == 4) return bf16 ? FN<16, 4, __nv_bfloat16>(ARGS, SMEM, st) : FN<16, 4, float>(ARGS, SMEM, st);   \
    return bf16 ? FN<16, 8, __nv_bfloat16>(ARGS, SMEM, st) : FN<16, 8, float>(ARGS, SMEM, st);               \
  } while (0)

cudaError_t launch_sm_pass1_batched(const SmPass1Args* a, int n, int S, int R, bool bf16, cudaStream_t st) {
  if (n < 1 || n > kMaxBatch) return cudaErrorInvalidValue;
  SmBatch<SmPass1Args> b;
  size_t smem = 0;
  double bytes = 0.0;
  b.n = n;
  b.first[0] = 0;
  for (int l = 0; l < n; ++l) {
    b.a[l] = a[l];
    b.first[l + 1] = b.first[l] + a[l].n_tiles_b + sm_pass1_role_c_ctas(S, a[l].B);
    const size_t need = sm_pass1_smem(S, R, a[l].B, a[l].C);
    if (need > smem) smem = need;
    bytes += (double)a[l].B * a[l].C * S * S * (bf16 ? 2 : 4);
  }
  ProfScope prof(ASI_K_SM_PASS1, st, bytes);
  ASI_DISPATCH_SRB(launch_pass1_bt, b, smem);
}

cudaError_t launch_sm_reduce_batched(const SmReduceArgs* a, const int* max_chunks, int n, cudaStream_t st) {
  if (n < 1 || n > kMaxBatch) return cudaErrorInvalidValue;
  SmBatch<SmReduceArgs> b;
  b.n = n;
  b.first[0] = 0;
  for (int l = 0; l < n; ++l) {
    b.a[l] = a[l];
    b.first[l + 1] = b.first[l] + max_chunks[l];
  }
  ProfScope prof(ASI_K_QR, st, 0.0);
  return launch_dependent(k_sm_reduce_b, dim3((unsigned)b.first[n], 4), dim3(kRedNT), 0, st, b);
}

cudaError_t launch_sm_core_batched(const SmCoreArgs* a, int n, int S, int R, bool bf16, cudaStream_t st) {
  if (n < 1 || n > kMaxBatch) return cudaErrorInvalidValue;
  SmBatch<SmCoreArgs> b;
  size_t smem = 0;
  double bytes = 0.0;
  b.n = n;
  b.first[0] = 0;
  for (int l = 0; l < n; ++l) {
    b.a[l] = a[l];
    b.first[l + 1] = b.first[l] + a[l].n_tiles;
    const size_t need = sm_core_smem(S, R, a[l].B);
    if (need > smem) smem = need;
    bytes += (double)a[l].B * a[l].C * S * S * (bf16 ? 2 : 4);
  }
  ProfScope prof(ASI_K_SM_CORE, st, bytes);
  ASI_DISPATCH_SRB(launch_core_bt, b, smem);
}

cudaError_t launch_sm_wgrad_batched(const SmWgradArgs* a, int n, int R, bool bf16, cudaStream_t st) {
  if (n < 1 || n > kMaxBatch) return cudaErrorInvalidValue;
  SmBatch<SmWgradArgs> b;
  size_t smem = 0;
  double bytes = 0.0;
  b.n = n;
  b.first[0] = 0;
  for (int l = 0; l < n; ++l) {
    b.a[l] = a[l];
    b.first[l + 1] = b.first[l] + a[l].Cout / a[l].cpb;
    const size_t need = sm_wgrad_smem(a[l], R);
    if (need > smem) smem = need;
    bytes += (double)a[l].B * a[l].Cout * a[l].Ho * a[l].Wo * (bf16 ? 2 : 4) +
             4.0 * (double)a[l].Cout * (a[l].C / a[l].groups) * a[l].kh * a[l].kw;
  }
  ProfScope prof(ASI_K_SM_WGRAD, st, bytes);
  if (R == 4) return bf16 ? launch_wgrad_bt<4, __nv_bfloat16>(b, smem, st) : launch_wgrad_bt<4, float>(b, smem, st);
  return bf16 ? launch_wgrad_bt<8, __nv_bfloat16>(b, smem, st) : launch_wgrad_bt<8, float>(b, smem, st);
}

}  // namespace asi
