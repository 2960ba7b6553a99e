// k_fiber_reg: the two products of one mode, V_m = A_m^T U_m and P_m = A_m V_m (Algorithm 1), or with
// project_only the mode product Y = X x_m U^T alone, streamed through REGISTERS: no tile is staged in shared
// memory, so the inner loops wait on no shared-memory read.
//
// The unfolding of the mode is X[o][k][i] (k the mode's index, i contiguous).  A lane owns CW neighbouring
// columns i and R rows k; the KS lanes of a warp that share a column group hold rows [R ks, R ks + R) and add
// their partial V with KS - 1 butterfly shuffles; every lane then expands its own rows,
//   P[k][:] += sum_c x[k][c] V[c][:],
// in registers across all columns the CTA visits.  The rows of the next column group are requested before the
// arithmetic of the current one.  P meets in shared memory once, at the end: one partial per CTA.
//
// Used with R = 8 rows and CW = 4 columns per lane (16-byte loads) for a_m <= 32, ranks up to 8: the batch mode
// of a token tensor.  For the long modes of large feature maps (a_m = 64, 128; R = 16, CW = 2) this kernel was
// measured SLOWER than the staged k_fiber2 (8 warps of 254 registers per SM keep 32 KB of loads in flight, too
// little for HBM): those modes stay on k_fiber2.
#include <cuda_bf16.h>

#include <algorithm>

#include "asi_internal.h"

namespace asi {

namespace {

template <typename TX, int CW> struct RawCols;
template <> struct RawCols<float, 4> {
  float4 v;
  __device__ __forceinline__ void load(const float* p) { v = __ldg(reinterpret_cast<const float4*>(p)); }
  __device__ __forceinline__ void get(float (&x)[4]) const { x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w; }
};
template <> struct RawCols<float, 2> {
  float2 v;
  __device__ __forceinline__ void load(const float* p) { v = __ldg(reinterpret_cast<const float2*>(p)); }
  __device__ __forceinline__ void get(float (&x)[2]) const { x[0] = v.x; x[1] = v.y; }
};
template <> struct RawCols<__nv_bfloat16, 4> {
  uint2 v;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = __ldg(reinterpret_cast<const uint2*>(p)); }
  __device__ __forceinline__ void get(float (&x)[4]) const {
    x[0] = __uint_as_float(v.x << 16); x[1] = __uint_as_float(v.x & 0xffff0000u);
    x[2] = __uint_as_float(v.y << 16); x[3] = __uint_as_float(v.y & 0xffff0000u);
  }
};

template <int CW> __device__ __forceinline__ void store_cols(float* dst, const float (&v)[CW]);
template <> __device__ __forceinline__ void store_cols<4>(float* dst, const float (&v)[4]) {
  *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void store_cols<2>(float* dst, const float (&v)[2]) {
  *reinterpret_cast<float2*>(dst) = make_float2(v[0], v[1]);
}

}  // namespace

template <int NJ, int KS, int R, int CW, int NT, typename TX>
__global__ void __launch_bounds__(NT, 1) k_fiber_reg(Fiber2Args p) {
  constexpr int QW = 32 / KS;                        // column groups per warp
  constexpr int NW = NT / 32;
  __shared__ __align__(16) float Us[R * KS * NJ];    // rows >= a and columns >= r are zero
  __shared__ float red[NW][R * KS * NJ];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int ks = lane / QW, cq = lane - ks * QW;
  const int a = p.a, r = p.r, r0 = R * ks;
  for (int e = tid; e < R * KS * NJ; e += NT) {
    const int k = e / NJ, j = e - k * NJ;
    Us[e] = (k < a && j < r) ? p.U[(int64_t)k * p.ldu + j] : 0.f;
  }
  __syncthreads();
  const int Iq = (int)(p.I / CW);
  const int total = (int)p.O * Iq;                   // column groups of the unfolding (< 2^30, checked by the host)
  const int stride = gridDim.x * NW * QW;
  // rows past the end of the mode re-read the last row (their factor row is zero)
  const int rfirst = (r0 < a) ? r0 : a - 1;
  const int nrow = (a - rfirst < R) ? a - rfirst : R;
  const TX* X = static_cast<const TX*>(p.X) + (int64_t)rfirst * p.I;
  const int64_t slab = (int64_t)a * p.I;
  float accP[R][NJ];
#pragma unroll
  for (int kk = 0; kk < R; ++kk)
#pragma unroll
    for (int j = 0; j < NJ; ++j) accP[kk][j] = 0.f;

  int gbase = (blockIdx.x * NW + warp) * QW;         // warp-uniform: the loop test is the same in every lane
  RawCols<TX, CW> cur[R], nxt[R];
  int o_c = 0, iq_c = 0;
  bool on_c = false;
  if (gbase < total) {
    const int g = gbase + cq;
    on_c = g < total;
    const int gl = on_c ? g : total - 1;
    o_c = gl / Iq; iq_c = gl - o_c * Iq;
    const TX* src = X + (int64_t)o_c * slab + CW * (int64_t)iq_c;
#pragma unroll
    for (int kk = 0; kk < R; ++kk) {
      cur[kk].load(src);
      if (kk + 1 < nrow) src += p.I;
    }
  }
  while (gbase < total) {
    // the next column group's rows are requested before this one's arithmetic (always from a valid address)
    const int gnb = gbase + stride;
    const int gn = gnb + cq;
    const bool on_n = gn < total;
    const int gl = on_n ? gn : total - 1;
    const int o_n = gl / Iq, iq_n = gl - o_n * Iq;
    {
      const TX* src = X + (int64_t)o_n * slab + CW * (int64_t)iq_n;
#pragma unroll
      for (int kk = 0; kk < R; ++kk) {
        nxt[kk].load(src);
        if (kk + 1 < nrow) src += p.I;
      }
    }
    float V[CW][NJ];
#pragma unroll
    for (int c = 0; c < CW; ++c)
#pragma unroll
      for (int j = 0; j < NJ; ++j) V[c][j] = 0.f;
#pragma unroll
    for (int kk = 0; kk < R; ++kk) {
      float x[CW];
      cur[kk].get(x);
#pragma unroll
      for (int j4 = 0; j4 < NJ; j4 += 4) {
        const float4 u = *reinterpret_cast<const float4*>(&Us[(r0 + kk) * NJ + j4]);
#pragma unroll
        for (int c = 0; c < CW; ++c) {
          V[c][j4 + 0] = fmaf(x[c], u.x, V[c][j4 + 0]);
          V[c][j4 + 1] = fmaf(x[c], u.y, V[c][j4 + 1]);
          V[c][j4 + 2] = fmaf(x[c], u.z, V[c][j4 + 2]);
          V[c][j4 + 3] = fmaf(x[c], u.w, V[c][j4 + 3]);
        }
      }
    }
#pragma unroll
    for (int s = QW; s < 32; s *= 2)                 // the KS row groups of a column group
#pragma unroll
      for (int c = 0; c < CW; ++c)
#pragma unroll
        for (int j = 0; j < NJ; ++j) V[c][j] += __shfl_xor_sync(0xffffffffu, V[c][j], s);
    if (p.project_only) {
      if (on_c) {
        float* dst = p.Y + (int64_t)o_c * p.y_so + CW * (int64_t)iq_c;
#pragma unroll
        for (int j = 0; j < NJ; ++j)
          if (j < r && (j % KS) == ks) {
            float v[CW];
#pragma unroll
            for (int c = 0; c < CW; ++c) v[c] = V[c][j];
            store_cols<CW>(dst + (int64_t)j * p.y_sj, v);
          }
      }
    } else {
      if (!on_c) {                                   // a lane past the end adds nothing
#pragma unroll
        for (int c = 0; c < CW; ++c)
#pragma unroll
          for (int j = 0; j < NJ; ++j) V[c][j] = 0.f;
      }
#pragma unroll
      for (int kk = 0; kk < R; ++kk) {
        float x[CW];
        cur[kk].get(x);
#pragma unroll
        for (int c = 0; c < CW; ++c)
#pragma unroll
          for (int j = 0; j < NJ; ++j) accP[kk][j] = fmaf(x[c], V[c][j], accP[kk][j]);
      }
    }
#pragma unroll
    for (int kk = 0; kk < R; ++kk) cur[kk] = nxt[kk];
    o_c = o_n; iq_c = iq_n; on_c = on_n;
    gbase = gnb;
  }
  if (p.project_only) return;
  // P of this CTA: over the lanes of a row group, then over the warps
#pragma unroll
  for (int kk = 0; kk < R; ++kk)
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      float v = accP[kk][j];
#pragma unroll
      for (int s = 1; s < QW; s *= 2) v += __shfl_xor_sync(0xffffffffu, v, s);
      if (cq == 0) red[warp][(r0 + kk) * NJ + j] = v;
    }
  __syncthreads();
  for (int e = tid; e < R * KS * NJ; e += NT) {
    const int k = e / NJ, j = e - k * NJ;
    if (k >= a || j >= r) continue;
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) v += red[w][e];
    p.Pp[((int64_t)blockIdx.x * a + k) * r + j] = v;
  }
}

namespace {

struct FrShape { int nj, ks, r, cw, nt; };

// the variant for (a, rank, element type); ks == 0 when none fits
FrShape fiber_reg_shape(int64_t a, int rank, bool bf16) {
  FrShape s = {0, 0, 0, 0, 0};
  if (rank < 1 || rank > 8 || a < 1) return s;
  (void)bf16;
  if (a <= 32) {
    s.nj = rank <= 4 ? 4 : 8; s.r = 8; s.cw = 4; s.nt = 256;
    s.ks = a <= 8 ? 1 : a <= 16 ? 2 : 4;
  }
  return s;
}

template <int NJ, int KS, int R, int CW, int NT, typename TX>
cudaError_t launch_fr(const Fiber2Args& p, int grid, cudaStream_t st) {
  k_fiber_reg<NJ, KS, R, CW, NT, TX><<<grid, NT, 0, st>>>(p);
  return cudaGetLastError();
}

template <int NJ, int R, int CW, int NT, typename TX>
cudaError_t launch_fr_ks(const Fiber2Args& p, int ks, int grid, cudaStream_t st) {
  switch (ks) {
    case 1: return launch_fr<NJ, 1, R, CW, NT, TX>(p, grid, st);
    case 2: return launch_fr<NJ, 2, R, CW, NT, TX>(p, grid, st);
    default: return launch_fr<NJ, 4, R, CW, NT, TX>(p, grid, st);
  }
}

}  // namespace

bool fiber_reg_supported(int64_t O, int64_t a, int64_t I, int r, bool bf16) {
  const FrShape s = fiber_reg_shape(a, r, bf16);
  return s.ks != 0 && I % s.cw == 0 && O * (I / s.cw) < (1ll << 30);
}

int fiber_reg_grid(int64_t O, int64_t a, int64_t I, int r, bool bf16) {
  const FrShape s = fiber_reg_shape(a, r, bf16);
  const int64_t per_cta = (int64_t)(s.nt / 32) * (32 / s.ks);
  return (int)std::min<int64_t>(148, (O * (I / s.cw) + per_cta - 1) / per_cta);
}

cudaError_t launch_fiber_reg(const Fiber2Args& p, int grid, bool bf16, cudaStream_t st) {
  const double xbytes = (double)p.O * p.a * p.I * (bf16 ? 2 : 4);
  ProfScope prof(p.project_only ? ASI_K_MODEPROD : ASI_K_EXPAND, st, xbytes);
  const FrShape s = fiber_reg_shape(p.a, p.r, bf16);
  if (s.nj == 4) {
    if (bf16) return launch_fr_ks<4, 8, 4, 256, __nv_bfloat16>(p, s.ks, grid, st);
    return launch_fr_ks<4, 8, 4, 256, float>(p, s.ks, grid, st);
  }
  if (bf16) return launch_fr_ks<8, 8, 4, 256, __nv_bfloat16>(p, s.ks, grid, st);
  return launch_fr_ks<8, 8, 4, 256, float>(p, s.ks, grid, st);
}

}  // namespace asi
