// Fused kernels for conv layers with small square feature maps (S x S, S in {7, 14, 16}) and
// ranks <= 8 -- the shapes of the ResNet / MobileNet tails.  One compress call is
//
//   k_sm_pass1  : streams the activation once and forms every P_m = A_m (A_m^T U_m^prev)
//                 (Algorithm 1) tile-locally: CTAs of role B hold tiles [all B x 196..256
//                 contiguous (c,h,w)] that contain whole mode-1/3/4 fibers, CTAs of role C hold
//                 one sample [all C x HW] that contains whole mode-2 fibers;
//   (generic)   : fixed-order fp64 reduction of the per-tile partials + Cholesky-QR;
//   k_sm_core   : second traversal (L2-resident): per-sample A[b] x_2 U_2^T x_3 U_3^T x_4 U_4^T,
//                 last CTA folds in U_1^T and writes the core.
//
// and the whole compressed weight gradient is one kernel, k_sm_wgrad (terms 1-5 of C_ASI).
#include <cuda_bf16.h>

#include "asi_internal.h"

namespace asi {

namespace {

// Opt-in dynamic shared memory ceiling of the fused kernels (plans only pick them when the
// layer needs less); leaves room for static shared memory under the 227 KB per-CTA limit.
constexpr int kMaxDynSmem = 200 * 1024;

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

// Loads a [rows x R] factor (row-major, r <= R real columns) into shared memory, zero-padded.
template <int R>
__device__ __forceinline__ void load_factor(float* dst, const float* __restrict__ U, int rows, int r) {
  for (int idx = threadIdx.x; idx < rows * R; idx += blockDim.x) {
    const int k = idx / R, j = idx % R;
    dst[idx] = (j < r) ? U[k * r + j] : 0.f;
  }
}

// Sum of `n` per-thread values over the CTA in a fixed order: warp shuffles, then warps in
// index order.  red: [8][n] floats of shared memory.  Threads tid < n return the total.
template <int N>
__device__ __forceinline__ void block_reduce_store(float (&v)[N], float* red, float* out_global, int n_keep_cols,
                                                   int R, int r) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int i = 0; i < N; ++i) {
    float x = v[i];
    x += __shfl_xor_sync(0xffffffffu, x, 16);
    x += __shfl_xor_sync(0xffffffffu, x, 8);
    x += __shfl_xor_sync(0xffffffffu, x, 4);
    x += __shfl_xor_sync(0xffffffffu, x, 2);
    x += __shfl_xor_sync(0xffffffffu, x, 1);
    if (lane == 0) red[warp * N + i] = x;
  }
  __syncthreads();
  const int nwarps = blockDim.x >> 5;
  for (int i = threadIdx.x; i < N; i += blockDim.x) {
    float s = 0.f;
    for (int w = 0; w < nwarps; ++w) s += red[w * N + i];
    const int k = i / R, j = i % R;      // value i is entry (k, j) of an [n_keep_cols.. x R] block
    if (j < r) out_global[k * r + j] = s;
  }
  __syncthreads();
  (void)n_keep_cols;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// k_sm_pass1
// ---------------------------------------------------------------------------------------------
template <int S, int R, typename TX>
__global__ void __launch_bounds__(256) k_sm_pass1(SmPass1Args p) {
  constexpr int HW = S * S;
  constexpr int CC = (S == 7) ? 4 : 1;               // channels per role-B tile
  constexpr int J = CC * HW;                         // contiguous elements per sample in a tile
  constexpr int PJ = (J % 32 == 4) ? J : J + 4;      // row pitch == 4 (mod 32): conflict-free b x j reads
  extern __shared__ __align__(16) float smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const TX* __restrict__ A = reinterpret_cast<const TX*>(p.act);
  const int B = p.B, C = p.C;

  if ((int)blockIdx.x < p.n_tiles_b) {
    // ---------------- role B: modes 1, 3, 4 on tile [B x J] ----------------
    const int tile = blockIdx.x;
    float* Xs = smem;                                // [B][PJ]
    float* U1s = Xs + B * PJ;                        // [B][R]
    float* U3s = U1s + B * R;                        // [S][R]
    float* U4s = U3s + S * R;                        // [S][R]
    float* Vs = U4s + S * R;                         // [J][R]
    float* red = Vs + J * R;                         // [8][S*R]
    const int64_t sample_stride = (int64_t)C * HW;
    const TX* src = A + (int64_t)tile * J;
    for (int idx = tid; idx < B * (J / 4); idx += 256) {
      const int b = idx / (J / 4), v = idx % (J / 4);
      const float4 x = ld4<TX>(src + b * sample_stride + 4 * v);
      *reinterpret_cast<float4*>(Xs + b * PJ + 4 * v) = x;
    }
    load_factor<R>(U1s, p.U_prev + p.u_off[0], B, p.r[0]);
    load_factor<R>(U3s, p.U_prev + p.u_off[2], S, p.r[2]);
    load_factor<R>(U4s, p.U_prev + p.u_off[3], S, p.r[3]);
    __syncthreads();

    // mode 1, projection: V[j,:] = sum_b X[b,j] U1[b,:]
    if (tid < J) {
      float acc[R];
#pragma unroll
      for (int j = 0; j < R; ++j) acc[j] = 0.f;
      for (int b = 0; b < B; ++b) {
        const float x = Xs[b * PJ + tid];
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          const float4 u = *reinterpret_cast<const float4*>(U1s + b * R + j);
          acc[j] = fmaf(x, u.x, acc[j]);
          acc[j + 1] = fmaf(x, u.y, acc[j + 1]);
          acc[j + 2] = fmaf(x, u.z, acc[j + 2]);
          acc[j + 3] = fmaf(x, u.w, acc[j + 3]);
        }
      }
#pragma unroll
      for (int j = 0; j < R; ++j) Vs[tid * R + j] = acc[j];
    }
    __syncthreads();
    // mode 1, expansion: P1[b,:] = sum_j X[b,j] V[j,:]; a warp covers 8 samples x 4 column phases
    {
      float* P1 = p.Pp[0] + (int64_t)tile * B * p.r[0];
      const int bl = lane >> 2, jl = lane & 3;
      for (int b0 = warp * 8; b0 < B; b0 += 64) {
        const int b = b0 + bl;
        float acc[R];
#pragma unroll
        for (int j = 0; j < R; ++j) acc[j] = 0.f;
        for (int jj = jl; jj < J; jj += 4) {
          const float x = Xs[b * PJ + jj];
#pragma unroll
          for (int j = 0; j < R; j += 4) {
            const float4 v = *reinterpret_cast<const float4*>(Vs + jj * R + j);
            acc[j] = fmaf(x, v.x, acc[j]);
            acc[j + 1] = fmaf(x, v.y, acc[j + 1]);
            acc[j + 2] = fmaf(x, v.z, acc[j + 2]);
            acc[j + 3] = fmaf(x, v.w, acc[j + 3]);
          }
        }
#pragma unroll
        for (int j = 0; j < R; ++j) {
          acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 1);
          acc[j] += __shfl_xor_sync(0xffffffffu, acc[j], 2);
        }
        if (jl == 0) {
#pragma unroll
          for (int j = 0; j < R; ++j)
            if (j < p.r[0]) P1[b * p.r[0] + j] = acc[j];
        }
      }
    }
    // modes 3 and 4: one column (fiber of S elements) per thread at a time
#pragma unroll 1
    for (int mode = 2; mode <= 3; ++mode) {
      const float* Us = (mode == 2) ? U3s : U4s;
      const int estride = (mode == 2) ? S : 1;       // step between fiber elements
      float acc[S * R];
#pragma unroll
      for (int i = 0; i < S * R; ++i) acc[i] = 0.f;
      const int ncols = B * CC * S;
      for (int q = tid; q < ncols; q += 256) {
        const int b = q / (CC * S), rem = q % (CC * S);
        const int cl = rem / S, o = rem % S;         // o = w for mode 3, h for mode 4
        const float* col = Xs + b * PJ + cl * HW + ((mode == 2) ? o : o * S);
        float x[S], v[R];
#pragma unroll
        for (int j = 0; j < R; ++j) v[j] = 0.f;
#pragma unroll
        for (int k = 0; k < S; ++k) {
          x[k] = col[k * estride];
#pragma unroll
          for (int j = 0; j < R; ++j) v[j] = fmaf(x[k], Us[k * R + j], v[j]);
        }
#pragma unroll
        for (int k = 0; k < S; ++k)
#pragma unroll
          for (int j = 0; j < R; ++j) acc[k * R + j] = fmaf(x[k], v[j], acc[k * R + j]);
      }
      block_reduce_store<S * R>(acc, red, p.Pp[mode] + (int64_t)tile * S * p.r[mode], S, R, p.r[mode]);
    }
  } else {
    // ---------------- role C: mode 2 on one sample [C x HW] ----------------
    constexpr int G = 256 / HW;                      // channel rows covered per sweep of the CTA
    constexpr int NACT = G * HW;                     // active threads in the projection
    const int b = blockIdx.x - p.n_tiles_b;
    float* U2s = smem;                               // [C][R]
    float* Vp = U2s + C * R;                         // [G][HW][R]
    float* V2s = Vp + G * HW * R;                    // [HW][R]
    load_factor<R>(U2s, p.U_prev + p.u_off[1], C, p.r[1]);
    __syncthreads();
    const TX* Xb = A + (int64_t)b * C * HW;
    if (tid < NACT) {
      // thread owns position hw = tid % HW and the channels c = tid / HW (mod G)
      float acc[R];
#pragma unroll
      for (int j = 0; j < R; ++j) acc[j] = 0.f;
      int c = tid / HW;
#pragma unroll 4
      for (int e = tid; e < C * HW; e += NACT, c += G) {
        const float x = to_f(Xb[e]);
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          const float4 u = *reinterpret_cast<const float4*>(U2s + c * R + j);
          acc[j] = fmaf(x, u.x, acc[j]);
          acc[j + 1] = fmaf(x, u.y, acc[j + 1]);
          acc[j + 2] = fmaf(x, u.z, acc[j + 2]);
          acc[j + 3] = fmaf(x, u.w, acc[j + 3]);
        }
      }
#pragma unroll
      for (int j = 0; j < R; ++j) Vp[tid * R + j] = acc[j];
    }
    __syncthreads();
    for (int idx = tid; idx < HW * R; idx += 256) {
      float s = 0.f;
#pragma unroll
      for (int g = 0; g < G; ++g) s += Vp[g * HW * R + idx];
      V2s[idx] = s;
    }
    __syncthreads();
    // expansion: P2[c,:] = sum_hw X[c,hw] V2[hw,:], one channel row per thread
    float* P2 = p.Pp[1] + (int64_t)b * C * p.r[1];
    for (int c = tid; c < C; c += 256) {
      const TX* row = Xb + (int64_t)c * HW;
      float acc[R];
#pragma unroll
      for (int j = 0; j < R; ++j) acc[j] = 0.f;
#pragma unroll 7
      for (int hw = 0; hw < HW; ++hw) {
        const float x = to_f(row[hw]);
#pragma unroll
        for (int j = 0; j < R; j += 4) {
          const float4 v = *reinterpret_cast<const float4*>(V2s + hw * R + j);
          acc[j] = fmaf(x, v.x, acc[j]);
          acc[j + 1] = fmaf(x, v.y, acc[j + 1]);
          acc[j + 2] = fmaf(x, v.z, acc[j + 2]);
          acc[j + 3] = fmaf(x, v.w, acc[j + 3]);
        }
      }
#pragma unroll
      for (int j = 0; j < R; ++j)
        if (j < p.r[1]) P2[c * p.r[1] + j] = acc[j];
    }
  }
}

// ---------------------------------------------------------------------------------------------
// k_sm_core: CTA b computes T[b] = A[b] x_2 U2^T x_3 U3^T x_4 U4^T ([r2,r3,r4]); the last CTA to
// finish sums core[i,:] = sum_b U1[b,i] T[b,:] in sample order.
// ---------------------------------------------------------------------------------------------
template <int S, int R, typename TX>
__global__ void __launch_bounds__(256) k_sm_core(SmCoreArgs p) {
  constexpr int HW = S * S;
  constexpr int G = 256 / HW;
  constexpr int NACT = G * HW;
  extern __shared__ __align__(16) float smem[];
  const int tid = threadIdx.x;
  const int b = blockIdx.x, C = p.C;
  const int r2 = p.r[1], r3 = p.r[2], r4 = p.r[3];
  float* U2s = smem;                    // [C][R]
  float* Vp = U2s + C * R;              // [G][HW][R]
  float* T2 = Vp + G * HW * R;          // [HW][R]      T2[(h,w)][j]
  float* U3s = T2 + HW * R;             // [S][R]
  float* U4s = U3s + S * R;             // [S][R]
  float* T3 = U4s + S * R;              // [R][R][S]    T3[j][k][w]
  __shared__ int s_last;
  load_factor<R>(U2s, p.U + p.u_off[1], C, r2);
  load_factor<R>(U3s, p.U + p.u_off[2], S, r3);
  load_factor<R>(U4s, p.U + p.u_off[3], S, r4);
  __syncthreads();
  const TX* Xb = reinterpret_cast<const TX*>(p.act) + (int64_t)b * C * HW;
  if (tid < NACT) {
    float acc[R];
#pragma unroll
    for (int j = 0; j < R; ++j) acc[j] = 0.f;
    int c = tid / HW;
#pragma unroll 4
    for (int e = tid; e < C * HW; e += NACT, c += G) {
      const float x = to_f(Xb[e]);
#pragma unroll
      for (int j = 0; j < R; j += 4) {
        const float4 u = *reinterpret_cast<const float4*>(U2s + c * R + j);
        acc[j] = fmaf(x, u.x, acc[j]);
        acc[j + 1] = fmaf(x, u.y, acc[j + 1]);
        acc[j + 2] = fmaf(x, u.z, acc[j + 2]);
        acc[j + 3] = fmaf(x, u.w, acc[j + 3]);
      }
    }
#pragma unroll
    for (int j = 0; j < R; ++j) Vp[tid * R + j] = acc[j];
  }
  __syncthreads();
  for (int idx = tid; idx < HW * R; idx += 256) {
    float s = 0.f;
#pragma unroll
    for (int g = 0; g < G; ++g) s += Vp[g * HW * R + idx];
    T2[idx] = s;
  }
  __syncthreads();
  // T3[j][k][w] = sum_h T2[(h,w)][j] U3[h][k]
  for (int idx = tid; idx < r2 * r3 * S; idx += 256) {
    const int w = idx % S, k = (idx / S) % r3, j = idx / (S * r3);
    float s = 0.f;
#pragma unroll
    for (int h = 0; h < S; ++h) s = fmaf(T2[(h * S + w) * R + j], U3s[h * R + k], s);
    T3[(j * R + k) * S + w] = s;
  }
  __syncthreads();
  // T[b][j][k][l] = sum_w T3[j][k][w] U4[w][l]
  const int n234 = r2 * r3 * r4;
  for (int idx = tid; idx < n234; idx += 256) {
    const int l = idx % r4, k = (idx / r4) % r3, j = idx / (r4 * r3);
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < S; ++w) s = fmaf(T3[(j * R + k) * S + w], U4s[w * R + l], s);
    p.Tb[(int64_t)b * n234 + idx] = s;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(p.counter, 1) == (int)gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const float* U1 = p.U + p.u_off[0];
  const int r1 = p.r[0];
  for (int idx = tid; idx < r1 * n234; idx += 256) {
    const int i = idx / n234, rest = idx % n234;
    float s = 0.f;
    for (int bb = 0; bb < p.B; ++bb) s = fmaf(U1[bb * r1 + i], __ldcg(p.Tb + (int64_t)bb * n234 + rest), s);
    p.core[idx] = s;
  }
  if (tid == 0) *p.counter = 0;
}

// ---------------------------------------------------------------------------------------------
// k_sm_wgrad: CTA owns CPB consecutive output channels.
//   Z3 = core x_3 U3 x_4 U4 (recomputed per CTA, tiny);  Z1 = dY x_1 U1^T on the CTA's channels;
//   Z4[c',j,kh,kw] = sum_{i,h',w'} Z1[i,c',h',w'] Z3pad[i,j,h's+kh-p,w's+kw-p];  dW = Z4 x_2 U2.
// ---------------------------------------------------------------------------------------------
template <int R, typename TX>
__global__ void __launch_bounds__(256) k_sm_wgrad(SmWgradArgs p) {
  extern __shared__ __align__(16) float smem[];
  const int tid = threadIdx.x;
  const int r1 = p.r[0], r2 = p.r[1], r3 = p.r[2], r4 = p.r[3];
  const int H = p.H, W = p.W, HW = H * W, HoWo = p.Ho * p.Wo, kk = p.kh * p.kw;
  const int J = p.cpb * HoWo;                        // dY columns of this CTA, contiguous per sample
  const int c0 = blockIdx.x * p.cpb;
  float* U1s = smem;                                 // [B][R]
  float* Ss = U1s + p.B * R;                         // [r1 r2 r3 r4]
  float* U3s = Ss + r1 * r2 * r3 * r4;               // [H][r3]
  float* U4s = U3s + H * r3;                         // [W][r4]
  float* Tm = U4s + W * r4;                          // [r1 r2][H][r4]
  float* Z3s = Tm + r1 * r2 * H * r4;                // [r1 r2][H][W]
  float* Z1s = Z3s + r1 * r2 * HW;                   // [J][R]
  float* Z4s = Z1s + J * R;                          // [cpb][r2][kk]
  float* red = Z4s + p.cpb * r2 * kk;                // [nsplit][cpb r2 kk]

  load_factor<R>(U1s, p.U + p.u_off[0], p.B, r1);
  for (int idx = tid; idx < r1 * r2 * r3 * r4; idx += 256) Ss[idx] = p.core[idx];
  for (int idx = tid; idx < H * r3; idx += 256) U3s[idx] = p.U[p.u_off[2] + idx];
  for (int idx = tid; idx < W * r4; idx += 256) U4s[idx] = p.U[p.u_off[3] + idx];
  __syncthreads();

  // term 1: Z1[j,:] = sum_b dY[b, c0*HoWo + j] U1[b,:]  (thread per column, coalesced per sample)
  const TX* dY = reinterpret_cast<const TX*>(p.dY) + (int64_t)c0 * HoWo;
  const int64_t sstride = (int64_t)p.Cout * HoWo;
  for (int j = tid; j < J; j += 256) {
    float acc[R];
#pragma unroll
    for (int q = 0; q < R; ++q) acc[q] = 0.f;
#pragma unroll 8
    for (int b = 0; b < p.B; ++b) {
      const float x = to_f(dY[b * sstride + j]);
#pragma unroll
      for (int q = 0; q < R; q += 4) {
        const float4 u = *reinterpret_cast<const float4*>(U1s + b * R + q);
        acc[q] = fmaf(x, u.x, acc[q]);
        acc[q + 1] = fmaf(x, u.y, acc[q + 1]);
        acc[q + 2] = fmaf(x, u.z, acc[q + 2]);
        acc[q + 3] = fmaf(x, u.w, acc[q + 3]);
      }
    }
#pragma unroll
    for (int q = 0; q < R; ++q) Z1s[j * R + q] = acc[q];
  }
  // terms 2-3: Tm[ij][h][l] = sum_k S[ij][k][l] U3[h][k];  Z3[ij][h][w] = sum_l Tm[ij][h][l] U4[w][l]
  for (int idx = tid; idx < r1 * r2 * H * r4; idx += 256) {
    const int l = idx % r4, h = (idx / r4) % H, ij = idx / (r4 * H);
    float s = 0.f;
    for (int k = 0; k < r3; ++k) s = fmaf(Ss[(ij * r3 + k) * r4 + l], U3s[h * r3 + k], s);
    Tm[idx] = s;
  }
  __syncthreads();
  for (int idx = tid; idx < r1 * r2 * HW; idx += 256) {
    const int w = idx % W, h = (idx / W) % H, ij = idx / HW;
    float s = 0.f;
    for (int l = 0; l < r4; ++l) s = fmaf(Tm[(ij * H + h) * r4 + l], U4s[w * r4 + l], s);
    Z3s[idx] = s;
  }
  __syncthreads();
  // term 4: thread (o, s): output o = (cl, j, kh, kw), split s of the (i, h') reduction
  const int n_out = p.cpb * r2 * kk;
  int nsplit = 256 / n_out;
  if (nsplit < 1) nsplit = 1;
  const int n_items = r1 * p.Ho;
  if (nsplit > n_items) nsplit = n_items;
  for (int t = tid; t < n_out * nsplit; t += 256) {
    const int o = t % n_out, s = t / n_out;
    const int cl = o / (r2 * kk), j = (o / kk) % r2, tt = o % kk, ky = tt / p.kw, kx = tt % p.kw;
    float acc = 0.f;
    for (int it = s; it < n_items; it += nsplit) {
      const int i = it / p.Ho, ho = it % p.Ho;
      const int h = ho * p.sh + ky - p.ph;
      if (h < 0 || h >= H) continue;
      const float* z1 = Z1s + (cl * HoWo + ho * p.Wo) * R + i;
      const float* z3 = Z3s + ((i * r2 + j) * H + h) * W;
      for (int wo = 0; wo < p.Wo; ++wo) {
        const int w = wo * p.sw + kx - p.pw;
        if (w >= 0 && w < W) acc = fmaf(z1[wo * R], z3[w], acc);
      }
    }
    red[s * n_out + o] = acc;
  }
  __syncthreads();
  for (int o = tid; o < n_out; o += 256) {
    float v = 0.f;
    for (int s = 0; s < nsplit; ++s) v += red[s * n_out + o];
    Z4s[o] = v;
  }
  __syncthreads();
  // term 5: dW[c0+cl, c, t] = sum_j Z4[cl][j][t] U2[(g cg + c), j]
  const int cg = p.C / p.groups, og = p.Cout / p.groups;
  const float* U2 = p.U + p.u_off[1];
  for (int cl = 0; cl < p.cpb; ++cl) {
    const int co = c0 + cl;
    const int g = co / og;
    float* dw = p.dW + (int64_t)co * cg * kk;
    const float* z4 = Z4s + cl * r2 * kk;
    for (int idx = tid; idx < cg * kk; idx += 256) {
      const int c = idx / kk, t = idx % kk;
      const float* u = U2 + (int64_t)(g * cg + c) * r2;
      float v = 0.f;
      for (int j = 0; j < r2; ++j) v = fmaf(z4[j * kk + t], __ldg(u + j), v);
      dw[idx] = v;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// host-side launchers
// ---------------------------------------------------------------------------------------------
size_t sm_pass1_smem(int S, int R, int B, int C) {
  const int HW = S * S, CC = (S == 7) ? 4 : 1, J = CC * HW, PJ = (J % 32 == 4) ? J : J + 4;
  const size_t role_b = (size_t)B * PJ + (size_t)B * R + 2 * S * R + (size_t)J * R + 8 * S * R;
  const int G = 256 / HW;
  const size_t role_c = (size_t)C * R + (size_t)G * HW * R + (size_t)HW * R;
  return 4 * (role_b > role_c ? role_b : role_c);
}

size_t sm_core_smem(int S, int R, int C) {
  const int HW = S * S, G = 256 / HW;
  return 4 * ((size_t)C * R + (size_t)G * HW * R + (size_t)HW * R + 2 * S * R + (size_t)R * R * S);
}

size_t sm_wgrad_smem(const SmWgradArgs& p, int R) {
  const int r1 = p.r[0], r2 = p.r[1], r3 = p.r[2], r4 = p.r[3];
  const int HW = p.H * p.W, J = p.cpb * p.Ho * p.Wo, kk = p.kh * p.kw;
  const int n_out = p.cpb * r2 * kk;
  int nsplit = 256 / n_out;
  if (nsplit < 1) nsplit = 1;
  size_t n = (size_t)p.B * R + (size_t)r1 * r2 * r3 * r4 + (size_t)p.H * r3 + (size_t)p.W * r4 +
             (size_t)r1 * r2 * p.H * r4 + (size_t)r1 * r2 * HW + (size_t)J * R + n_out +
             (size_t)nsplit * n_out;
  return 4 * n + 64;
}

template <int S, int R, typename TX>
static cudaError_t launch_pass1_t(const SmPass1Args& p, cudaStream_t st) {
  const size_t smem = sm_pass1_smem(S, R, p.B, p.C);
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_sm_pass1<S, R, TX>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kMaxDynSmem);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  k_sm_pass1<S, R, TX><<<p.n_tiles_b + p.B, 256, smem, st>>>(p);
  return cudaGetLastError();
}

template <int S, int R, typename TX>
static cudaError_t launch_core_t(const SmCoreArgs& p, cudaStream_t st) {
  const size_t smem = sm_core_smem(S, R, p.C);
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_sm_core<S, R, TX>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kMaxDynSmem);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  k_sm_core<S, R, TX><<<p.B, 256, smem, st>>>(p);
  return cudaGetLastError();
}

template <int R, typename TX>
static cudaError_t launch_wgrad_t(const SmWgradArgs& p, cudaStream_t st) {
  const size_t smem = sm_wgrad_smem(p, R);
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(k_sm_wgrad<R, TX>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kMaxDynSmem);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  k_sm_wgrad<R, TX><<<p.Cout / p.cpb, 256, smem, st>>>(p);
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
  double bytes = (double)p.B * p.C * S * S * eb;
  bytes += 4.0 * ((double)p.n_tiles_b * (p.B * p.r[0] + S * p.r[2] + S * p.r[3]) + (double)p.B * p.C * p.r[1]);
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

}  // namespace asi
