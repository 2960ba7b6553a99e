// Shape-generic kernels of the ASI path (any number of modes, any sizes, ranks <= 64).
// They are the correctness baseline every layer shape can fall back on; shape-specialised
// kernels live in their own files.
//
//   k_modeprod : Y = X x_m B^T-like small contraction over one mode (Sec. 3.2, m-mode product)
//   k_expand   : P_m = A_m V_m, split over the columns of the unfolding (Algorithm 1)
//   k_qr_gram / k_qr_solve : Orthogonalize(P) as Cholesky-QR with the Gram matrix and the
//                triangular solve in fp64 -- in exact arithmetic the Gram-Schmidt basis
//   k_conv_tail: terms 4 and 5 of C_ASI (appendix "Speedup")
#include <cuda_bf16.h>

#include "asi_internal.h"

namespace asi {

ProfState g_prof = {0, nullptr, 0, 0, 0.0};

__device__ __forceinline__ float ld_as_float(const float* p) { return *p; }
__device__ __forceinline__ float ld_as_float(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// ---------------------------------------------------------------------------------------------
// Tile loader: Xs[kl][ql] = X(k0 + kl, q0 + ql), zero outside [0,a) x [q0, q_end).
// Fibers strided by I > 1 (or short fibers) are read column-wise: consecutive threads take
// consecutive columns.  Contiguous long fibers (I == 1, a >= 32) are read along k.
// ---------------------------------------------------------------------------------------------
template <int KC, int TQ, int NT, typename TX>
__device__ __forceinline__ void load_x_tile(float (*Xs)[TQ + 1], const TX* __restrict__ X, int64_t a,
                                            int64_t I, int64_t k0, int64_t q0, int64_t q_end) {
  const int tid = threadIdx.x;
  if (I == 1 && a >= 32) {
    for (int idx = tid; idx < KC * TQ; idx += NT) {
      const int kl = idx % KC, ql = idx / KC;
      const int64_t k = k0 + kl, q = q0 + ql;
      float v = 0.f;
      if (k < a && q < q_end) v = ld_as_float(X + q * a + k);
      Xs[kl][ql] = v;
    }
  } else {
    static_assert(NT % TQ == 0, "threads must tile the columns");
    const int ql = tid % TQ;
    const int64_t q = q0 + ql;
    const bool qok = q < q_end;
    int64_t base = 0;
    if (qok) {
      const int64_t o = q / I, i = q - o * I;
      base = o * a * I + i;
    }
    for (int kl = tid / TQ; kl < KC; kl += NT / TQ) {
      const int64_t k = k0 + kl;
      float v = 0.f;
      if (qok && k < a) v = ld_as_float(X + base + k * I);
      Xs[kl][ql] = v;
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
    for (int idx = tid; idx < KC * R; idx += NT) {
      const int kl = idx / R, j = idx % R;
      const int64_t k = k0 + kl;
      const int jj = j0 + j;
      Bs[kl][j] = (k < p.a && jj < p.n_out) ? p.B[k * p.ldb_k + jj * p.ldb_j] : 0.f;
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

template <typename TX>
static cudaError_t launch_modeprod_t(const ModeProdArgs& p, cudaStream_t st) {
  if (p.Q <= 0 || p.n_out <= 0) return cudaSuccess;
  ProfScope prof(ASI_K_MODEPROD, st,
                 (double)p.Q * p.a * sizeof(TX) + 4.0 * ((double)p.a * p.n_out + (double)p.Q * p.n_out));
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
  int R = 8;
  while (R < p.r) R *= 2;
  dim3 grid((unsigned)((p.a + kExpandKC - 1) / kExpandKC), (unsigned)p.nsplit);
  switch (R) {
    case 8: k_expand<8, TX><<<grid, 256, 0, st>>>(p); break;
    case 16: k_expand<16, TX><<<grid, 256, 0, st>>>(p); break;
    case 32: k_expand<32, TX><<<grid, 256, 0, st>>>(p); break;
    default: k_expand<64, TX><<<grid, 256, 0, st>>>(p); break;
  }
  return cudaGetLastError();
}

cudaError_t launch_expand(const ExpandArgs& p, bool x_bf16, cudaStream_t st) {
  return x_bf16 ? launch_expand_t<__nv_bfloat16>(p, st) : launch_expand_t<float>(p, st);
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
  if (c >= M.nchunk) return;
  __shared__ double Ps[kQRRows][ASI_MAX_RANK];
  const int tid = threadIdx.x;
  const int r = M.r;
  const int row0 = c * kQRRows;
  for (int idx = tid; idx < kQRRows * r; idx += 256) {
    const int rl = idx / r, j = idx % r;
    const int row = row0 + rl;
    double v = 0.0;
    if (row < M.a) {
      for (int s = 0; s < M.nsplit; ++s) v += (double)M.Pp[((int64_t)s * M.a + row) * r + j];
      M.Pred[(int64_t)row * r + j] = v;
    }
    Ps[rl][j] = v;
  }
  __syncthreads();
  for (int idx = tid; idx < r * r; idx += 256) {
    const int i = idx / r, j = idx % r;
    if (j < i) continue;
    double g = 0.0;
#pragma unroll 8
    for (int rl = 0; rl < kQRRows; ++rl) g = fma(Ps[rl][i], Ps[rl][j], g);
    M.Gp[((int64_t)c * r + i) * r + j] = g;
  }
}

__global__ void __launch_bounds__(256) k_qr_solve(QRArgs args) {
  const QRMode M = args.m[blockIdx.y];
  const int c = blockIdx.x;
  if (c >= M.nchunk) return;
  __shared__ double G[ASI_MAX_RANK][ASI_MAX_RANK + 1];
  __shared__ double s_trace;
  const int tid = threadIdx.x;
  const int r = M.r;
  for (int idx = tid; idx < r * r; idx += 256) {
    const int i = idx / r, j = idx % r;
    double g = 0.0;
    if (j >= i)
      for (int cc = 0; cc < M.nchunk; ++cc) g += M.Gp[((int64_t)cc * r + i) * r + j];
    G[i][j] = g;
  }
  __syncthreads();
  if (tid == 0) {
    double t = 0.0;
    for (int i = 0; i < r; ++i) t += G[i][i];
    s_trace = t;
  }
  __syncthreads();
  const double floor_d = 1e-12 * s_trace;
  for (int j = 0; j < r; ++j) {
    double d = G[j][j];
    if (!(d > floor_d)) {
      if (tid == 0 && c == 0) atomicMax(args.status, (int)ASI_ERR_RANK_DEFICIENT);
      d = (floor_d > 0.0) ? floor_d : 1.0;
    }
    const double rjj = sqrt(d);
    __syncthreads();
    for (int k = j + 1 + tid; k < r; k += 256) G[j][k] /= rjj;
    if (tid == 0) G[j][j] = rjj;
    __syncthreads();
    const int n = r - j - 1;
    for (int idx = tid; idx < n * n; idx += 256) {
      const int i = j + 1 + idx / n, k = j + 1 + idx % n;
      if (k >= i) G[i][k] -= G[j][i] * G[j][k];
    }
    __syncthreads();
  }
  if (tid < kQRRows) {
    const int row = c * kQRRows + tid;
    if (row < M.a) {
      double q[ASI_MAX_RANK];
      const double* prow = M.Pred + (int64_t)row * r;
      for (int j = 0; j < r; ++j) {
        double v = prow[j];
        for (int i = 0; i < j; ++i) v -= q[i] * G[i][j];
        v /= G[j][j];
        q[j] = v;
        M.Uout[(int64_t)row * r + j] = (float)v;
      }
    }
  }
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
  k_qr_solve<<<grid, 256, 0, st>>>(p);
  return cudaGetLastError();
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

cudaError_t launch_conv_tail(const ConvTailArgs& p, cudaStream_t st) {
  ProfScope prof(ASI_K_CONV_TAIL, st,
                 4.0 * ((double)p.r1 * p.Cout * p.Ho * p.Wo + (double)p.r1 * p.r2 * p.H * p.W +
                        (double)p.C * p.r2 + (double)p.Cout * (p.C / p.groups) * p.kh * p.kw));
  const int n_out = p.r2 * p.kh * p.kw;
  const int nsplit_max = (n_out <= 128) ? 256 / n_out : 1;
  const size_t smem = (size_t)(((n_out + 31) / 32) * 32 + (size_t)nsplit_max * n_out) * sizeof(float);
  k_conv_tail<<<p.Cout, 256, smem, st>>>(p);
  return cudaGetLastError();
}

}  // namespace asi
