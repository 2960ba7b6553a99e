// Rank selection aids on the device (Sec. 3.2: HOSVD_eps truncates every mode at the smallest rank whose
// leading components hold a fraction eps of the mode's energy; Sec. 3.3: activation perplexity
// ||dW - dW~||_F).  Everything here runs once per layer before training, not per step: the kernels are
// plain and exact-minded (fp64 accumulation, fixed summation orders), not tuned.
//
//   k_gram / k_gram_sum : G_m = A_m A_m^T (a_m x a_m, fp64): 32 x 32 output blocks, the contraction split
//                         over CTAs, products and sums in fp64, the splits added in order
//   k_sub_* (a_m > 128) : block subspace iteration on G_m with 128 vectors -- Y = G X, Gram-Schmidt twice
//                         per column (one CTA), ten rounds -- then H = X^T G X, whose eigenvalues are the
//                         leading Ritz values of G_m
//   k_jacobi            : eigenvalues of a symmetric matrix of order <= 128 in one CTA: cyclic two-sided
//                         Jacobi with the round-robin ordering (n/2 disjoint rotations per step), fp64 in
//                         shared memory; sorted descending
//   k_pick_ranks        : smallest r with sum_{k<r} lambda_k >= (eps - 1e-15) trace, clipped to
//                         [1, min(r_max, a_m, b_m)]
//   k_sqdiff / k_sqdiff_sum : sqrt(sum (x - y)^2) in fp64, per-CTA partials added in order
#include <cuda_bf16.h>

#include <algorithm>

#include "asi_internal.h"

namespace asi {

namespace {

constexpr int kSpecK = ASI_SPECTRUM_MAX;      // eigenvalues kept per mode; order of the Jacobi problem
constexpr int kSubRounds = 10;

__device__ __forceinline__ float ldx(const float* p) { return *p; }
__device__ __forceinline__ float ldx(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// Gp[split][i][j] for the upper block triangle of G = A_m A_m^T; view X(o, k, i) at (o a + k) I + i, q = o I + i
template <typename TX>
__global__ void __launch_bounds__(256) k_gram(const TX* __restrict__ X, int64_t a, int64_t I, int64_t Q,
                                              int64_t q_per_split, double* __restrict__ Gp) {
  const int bi = blockIdx.x, bj = blockIdx.y;
  if (bj < bi) return;
  __shared__ float As[32][33], Bs[32][33];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int64_t q0 = (int64_t)blockIdx.z * q_per_split;
  const int64_t q1 = (q0 + q_per_split < Q) ? q0 + q_per_split : Q;
  double acc[2][2] = {{0.0, 0.0}, {0.0, 0.0}};
  for (int64_t qc = q0; qc < q1; qc += 32) {
    float va[4], vb[4];
#pragma unroll
    for (int t = 0; t < 4; ++t) {                       // all loads first, selected afterwards
      const int e = tid + t * 256, kl = e >> 5, ql = e & 31;
      const int64_t q = qc + ql;
      const bool qok = q < q1;
      const int64_t o = qok ? q / I : 0, i = qok ? q - o * I : 0;
      const int64_t ka = (int64_t)bi * 32 + kl, kb = (int64_t)bj * 32 + kl;
      va[t] = ldx(X + ((qok && ka < a) ? (o * a + ka) * I + i : 0));
      vb[t] = ldx(X + ((qok && kb < a) ? (o * a + kb) * I + i : 0));
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int e = tid + t * 256, kl = e >> 5, ql = e & 31;
      const bool qok = qc + ql < q1;
      As[kl][ql] = (qok && (int64_t)bi * 32 + kl < a) ? va[t] : 0.f;
      Bs[kl][ql] = (qok && (int64_t)bj * 32 + kl < a) ? vb[t] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int ql = 0; ql < 32; ++ql) {                 // fp64 products: the small eigenvalues need them
      const double a0 = As[ty][ql], a1 = As[ty + 16][ql], b0 = Bs[tx][ql], b1 = Bs[tx + 16][ql];
      acc[0][0] = fma(a0, b0, acc[0][0]); acc[0][1] = fma(a0, b1, acc[0][1]);
      acc[1][0] = fma(a1, b0, acc[1][0]); acc[1][1] = fma(a1, b1, acc[1][1]);
    }
    __syncthreads();
  }
  double* G = Gp + (int64_t)blockIdx.z * a * a;
#pragma unroll
  for (int x = 0; x < 2; ++x)
#pragma unroll
    for (int y = 0; y < 2; ++y) {
      const int64_t i = (int64_t)bi * 32 + ty + 16 * x, j = (int64_t)bj * 32 + tx + 16 * y;
      if (i < a && j < a) G[i * a + j] = acc[x][y];
    }
}

// G = sum of the splits (in order), mirrored to the lower triangle; trace[0] = sum of the diagonal
__global__ void __launch_bounds__(256) k_gram_sum(double* __restrict__ Gp, int64_t a, int nsplit, double* G) {
  const int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (e >= a * a) return;
  const int64_t i = e / a, j = e - i * a;
  const int64_t src = ((j / 32) >= (i / 32)) ? e : j * a + i;     // the block (i, j) was computed iff block_j >= block_i
  double s = 0.0;
  for (int sp = 0; sp < nsplit; ++sp) s += Gp[(int64_t)sp * a * a + src];
  G[e] = s;
}

__global__ void __launch_bounds__(256) k_trace(const double* __restrict__ G, int64_t a, double* out) {
  __shared__ double red[256];
  double s = 0.0;
  for (int64_t i = threadIdx.x; i < a; i += 256) s += G[i * a + i];
  red[threadIdx.x] = s;
  __syncthreads();
  for (int h = 128; h >= 1; h >>= 1) {
    if (threadIdx.x < h) red[threadIdx.x] += red[threadIdx.x + h];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[0] = red[0];
}

// ---- subspace iteration on G (n x n), basis X stored column-major Xc[K][n] -------------------------
// start: column j of X = column (j * n / K) of G (in the range of G, rich in the leading eigenvectors)
__global__ void __launch_bounds__(256) k_sub_init(const double* __restrict__ G, int64_t n, double* Xc) {
  const int j = blockIdx.y;
  const int64_t col = (int64_t)j * n / kSpecK;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256)
    Xc[(int64_t)j * n + i] = G[i * n + col];
}
// Yc[j][i] = sum_k G[i][k] Xc[j][k]
__global__ void __launch_bounds__(256) k_sub_matmul(const double* __restrict__ G, const double* __restrict__ Xc,
                                                    int64_t n, double* __restrict__ Yc) {
  __shared__ double Gs[16][17], Xs[16][17];
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int64_t i0 = (int64_t)blockIdx.x * 16;
  const int j0 = blockIdx.y * 16;
  double acc = 0.0;
  for (int64_t k0 = 0; k0 < n; k0 += 16) {
    Gs[ty][tx] = (i0 + ty < n && k0 + tx < n) ? G[(i0 + ty) * n + k0 + tx] : 0.0;
    Xs[ty][tx] = (k0 + tx < n) ? Xc[(int64_t)(j0 + ty) * n + k0 + tx] : 0.0;
    __syncthreads();
#pragma unroll
    for (int k = 0; k < 16; ++k) acc = fma(Gs[tx][k], Xs[ty][k], acc);
    __syncthreads();
  }
  if (i0 + tx < n) Yc[(int64_t)(j0 + ty) * n + i0 + tx] = acc;
}
// Gram-Schmidt on the K columns of Yc, twice per column, in one CTA (1024 threads): the columns of Yc become
// orthonormal.  A column that vanishes against its predecessors is replaced by zeros.
__global__ void __launch_bounds__(1024) k_sub_orth(double* __restrict__ Yc, int64_t n) {
  __shared__ double dots[kSpecK];
  __shared__ double red[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int j = 0; j < kSpecK; ++j) {
    double* yj = Yc + (int64_t)j * n;
    for (int pass = 0; pass < 2; ++pass) {
      for (int i = warp; i < j; i += 32) {
        const double* yi = Yc + (int64_t)i * n;
        double s = 0.0;
        for (int64_t k = lane; k < n; k += 32) s = fma(yi[k], yj[k], s);
        for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
        if (lane == 0) dots[i] = s;
      }
      __syncthreads();
      for (int64_t k = tid; k < n; k += 1024) {
        double v = yj[k];
        for (int i = 0; i < j; ++i) v = fma(-dots[i], Yc[(int64_t)i * n + k], v);
        yj[k] = v;
      }
      __syncthreads();
    }
    double s = 0.0;
    for (int64_t k = tid; k < n; k += 1024) s = fma(yj[k], yj[k], s);
    for (int off = 16; off >= 1; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    if (lane == 0) red[warp] = s;
    __syncthreads();
    if (tid == 0) {
      double t = 0.0;
      for (int w = 0; w < 32; ++w) t += red[w];
      red[0] = (t > 0.0) ? rsqrt(t) : 0.0;
    }
    __syncthreads();
    const double inv = red[0];
    for (int64_t k = tid; k < n; k += 1024) yj[k] *= inv;
    __syncthreads();
  }
}
// H[i][j] = sum_k Xc[i][k] Yc[j][k]   (K x K)
__global__ void __launch_bounds__(256) k_sub_ritz(const double* __restrict__ Xc, const double* __restrict__ Yc,
                                                  int64_t n, double* __restrict__ H) {
  __shared__ double red[256];
  const int i = blockIdx.x, j = blockIdx.y;
  double s = 0.0;
  for (int64_t k = threadIdx.x; k < n; k += 256) s = fma(Xc[(int64_t)i * n + k], Yc[(int64_t)j * n + k], s);
  red[threadIdx.x] = s;
  __syncthreads();
  for (int h = 128; h >= 1; h >>= 1) {
    if (threadIdx.x < h) red[threadIdx.x] += red[threadIdx.x + h];
    __syncthreads();
  }
  if (threadIdx.x == 0) H[i * kSpecK + j] = red[0];
}

// ---- Jacobi eigenvalues of a symmetric matrix of order n <= 128 ------------------------------------
__global__ void __launch_bounds__(1024) k_jacobi(const double* __restrict__ M, int n, int ldm, double* __restrict__ eig) {
  extern __shared__ double jac[];
  const int ne = (n + 1) & ~1, P = ne + 1, half = ne / 2;     // even order (a zero row/column is appended)
  double* A = jac;                                 // [ne][P]
  double* cs = A + ne * P;                         // [half][2]: rotation of pair t
  int* top = reinterpret_cast<int*>(cs + 2 * half);   // [half], bot [half]: the round-robin line-up
  int* bot = top + half;
  const int tid = threadIdx.x;
  for (int e = tid; e < ne * ne; e += 1024) {
    const int i = e / ne, j = e - i * ne;
    A[i * P + j] = (i < n && j < n) ? 0.5 * (M[(int64_t)i * ldm + j] + M[(int64_t)j * ldm + i]) : 0.0;
  }
  for (int t = tid; t < half; t += 1024) {
    top[t] = 2 * t;
    bot[t] = 2 * t + 1;
  }
  __syncthreads();
  for (int sweep = 0; sweep < 16; ++sweep) {
    for (int step = 0; step < ne - 1; ++step) {
      // rotation angles of the n/2 disjoint pairs
      for (int t = tid; t < half; t += 1024) {
        const int p = min(top[t], bot[t]), q = max(top[t], bot[t]);
        const double app = A[p * P + p], aqq = A[q * P + q], apq = A[p * P + q];
        double c = 1.0, s = 0.0;
        if (fabs(apq) > 1e-300 && fabs(apq) > 1e-22 * sqrt(fabs(app * aqq)) ) {
          const double tau = (aqq - app) / (2.0 * apq);
          const double tt = (tau >= 0.0 ? 1.0 : -1.0) / (fabs(tau) + sqrt(1.0 + tau * tau));
          c = rsqrt(1.0 + tt * tt);
          s = tt * c;
        }
        cs[2 * t] = c;
        cs[2 * t + 1] = s;
      }
      __syncthreads();
      // rows p, q of every pair: A <- J^T A
      for (int e = tid; e < half * ne; e += 1024) {
        const int t = e / ne, k = e - t * ne;
        const int p = min(top[t], bot[t]), q = max(top[t], bot[t]);
        const double c = cs[2 * t], s = cs[2 * t + 1];
        const double x = A[p * P + k], y = A[q * P + k];
        A[p * P + k] = c * x - s * y;
        A[q * P + k] = s * x + c * y;
      }
      __syncthreads();
      // columns p, q of every pair: A <- A J
      for (int e = tid; e < half * ne; e += 1024) {
        const int t = e / ne, k = e - t * ne;
        const int p = min(top[t], bot[t]), q = max(top[t], bot[t]);
        const double c = cs[2 * t], s = cs[2 * t + 1];
        const double x = A[k * P + p], y = A[k * P + q];
        A[k * P + p] = c * x - s * y;
        A[k * P + q] = s * x + c * y;
      }
      __syncthreads();
      // next line-up: player top[0] stays, the others move one seat round the table
      if (tid == 0) {
        const int last_top = top[half - 1], first_bot = bot[0];
        for (int t = half - 1; t >= 2; --t) top[t] = top[t - 1];
        if (half > 1) top[1] = first_bot;
        for (int t = 0; t + 1 < half; ++t) bot[t] = bot[t + 1];
        bot[half - 1] = (half > 1) ? last_top : first_bot;
      }
      __syncthreads();
    }
  }
  // descending order by counting; the appended zero of an odd order is dropped as the smallest entry
  double* d = cs;                                  // reuse: ne doubles fit in [half][2]
  for (int i = tid; i < ne; i += 1024) d[i] = A[i * P + i];
  __syncthreads();
  for (int i = tid; i < ne; i += 1024) {
    const double v = d[i];
    int rank = 0;
    for (int j = 0; j < ne; ++j) rank += (d[j] > v || (d[j] == v && j < i)) ? 1 : 0;
    if (rank < n && rank < kSpecK) eig[rank] = v > 0.0 ? v : 0.0;
  }
}

__global__ void k_pick_ranks(const double* __restrict__ eig, const double* __restrict__ energy, double eps,
                             int r_max, int nd, int64_t a0, int64_t a1, int64_t a2, int64_t a3, int64_t N,
                             int* __restrict__ ranks) {
  const int m = threadIdx.x;
  if (m >= nd) return;
  const int64_t a = (m == 0) ? a0 : (m == 1) ? a1 : (m == 2) ? a2 : a3;
  const double total = energy[m];
  const int nk = (int)((a < kSpecK) ? a : kSpecK);
  int r = nk;
  double cum = 0.0;
  for (int k = 0; k < nk; ++k) {
    cum += eig[m * kSpecK + k];
    if (cum / total >= eps - 1e-15) {
      r = k + 1;
      break;
    }
  }
  int64_t cap = r_max;
  if (a < cap) cap = a;
  if (N / a < cap) cap = N / a;
  if (r > cap) r = (int)cap;
  if (r < 1) r = 1;
  ranks[m] = r;
}

__global__ void __launch_bounds__(256) k_sqdiff(const float* __restrict__ x, const float* __restrict__ y, int64_t n,
                                                double* __restrict__ part) {
  __shared__ double red[256];
  double s = 0.0;
  for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256) {
    const double d = (double)x[i] - (double)y[i];
    s = fma(d, d, s);
  }
  red[threadIdx.x] = s;
  __syncthreads();
  for (int h = 128; h >= 1; h >>= 1) {
    if (threadIdx.x < h) red[threadIdx.x] += red[threadIdx.x + h];
    __syncthreads();
  }
  if (threadIdx.x == 0) part[blockIdx.x] = red[0];
}
__global__ void k_sqdiff_sum(const double* __restrict__ part, int n, double* out) {
  if (threadIdx.x != 0 || blockIdx.x != 0) return;
  double s = 0.0;
  for (int i = 0; i < n; ++i) s += part[i];
  out[0] = sqrt(s);
}

constexpr int kSqGrid = 296;

size_t jacobi_smem(int n) {
  const int ne = (n + 1) & ~1;
  return (size_t)ne * (ne + 1) * 8 + (size_t)ne * 8 + (size_t)ne * 4 + 64;
}

void gram_split(int64_t a, int64_t Q, int* nsplit, int64_t* qps) {
  const int64_t nb = (a + 31) / 32, blocks = nb * (nb + 1) / 2;
  int64_t ns = std::max<int64_t>(1, 592 / blocks);
  ns = std::min<int64_t>(ns, std::max<int64_t>(1, Q / 1024));
  while (ns > 1 && (double)ns * a * a * 8.0 > 256e6) --ns;
  int64_t q = (Q + ns - 1) / ns;
  q = (q + 31) / 32 * 32;
  *nsplit = (int)((Q + q - 1) / q);
  *qps = q;
}

}  // namespace

// workspace: per mode (one at a time): split partials of G, G itself, and for a > 128 the two bases and H
size_t spectrum_ws_bytes(const asi_plan* pl) {
  size_t need = 0;
  for (int m = 0; m < pl->nd; ++m) {
    const int64_t a = pl->mv[m].a;
    int ns;
    int64_t qps;
    gram_split(a, pl->mv[m].Q, &ns, &qps);
    size_t b = align_up((size_t)ns * a * a * 8, 256) + align_up((size_t)a * a * 8, 256);
    if (a > kSpecK) b += 2 * align_up((size_t)kSpecK * a * 8, 256) + align_up((size_t)kSpecK * kSpecK * 8, 256);
    need = std::max(need, b);
  }
  return need + 256;
}

cudaError_t launch_mode_spectrum(const asi_plan* pl, const void* act, double* eig, double* energy, char* w,
                                 cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(eig, 0, (size_t)pl->nd * kSpecK * sizeof(double), st);
  if (e != cudaSuccess) return e;
  e = opt_in_smem(reinterpret_cast<const void*>(k_jacobi), jacobi_smem(kSpecK));
  if (e != cudaSuccess) return e;
  for (int m = 0; m < pl->nd; ++m) {
    const ModeView& v = pl->mv[m];
    const int64_t a = v.a;
    int ns;
    int64_t qps;
    gram_split(a, v.Q, &ns, &qps);
    double* Gp = reinterpret_cast<double*>(w);
    double* G = reinterpret_cast<double*>(w + align_up((size_t)ns * a * a * 8, 256));
    const dim3 grid((unsigned)((a + 31) / 32), (unsigned)((a + 31) / 32), (unsigned)ns);
    if (pl->bf16)
      k_gram<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(act), a, v.I, v.Q, qps, Gp);
    else
      k_gram<float><<<grid, 256, 0, st>>>(static_cast<const float*>(act), a, v.I, v.Q, qps, Gp);
    k_gram_sum<<<(unsigned)((a * a + 255) / 256), 256, 0, st>>>(Gp, a, ns, G);
    k_trace<<<1, 256, 0, st>>>(G, a, energy + m);
    if (a <= kSpecK) {
      k_jacobi<<<1, 1024, jacobi_smem((int)a), st>>>(G, (int)a, (int)a, eig + m * kSpecK);
    } else {
      char* p = reinterpret_cast<char*>(G) + align_up((size_t)a * a * 8, 256);
      double* Xc = reinterpret_cast<double*>(p);
      double* Yc = reinterpret_cast<double*>(p + align_up((size_t)kSpecK * a * 8, 256));
      double* H = reinterpret_cast<double*>(p + 2 * align_up((size_t)kSpecK * a * 8, 256));
      const dim3 mm((unsigned)((a + 15) / 16), kSpecK / 16);
      k_sub_init<<<dim3(8, kSpecK), 256, 0, st>>>(G, a, Xc);
      k_sub_orth<<<1, 1024, 0, st>>>(Xc, a);
      for (int it = 0; it < kSubRounds; ++it) {
        k_sub_matmul<<<mm, 256, 0, st>>>(G, Xc, a, Yc);
        k_sub_orth<<<1, 1024, 0, st>>>(Yc, a);
        std::swap(Xc, Yc);
      }
      k_sub_matmul<<<mm, 256, 0, st>>>(G, Xc, a, Yc);
      k_sub_ritz<<<dim3(kSpecK, kSpecK), 256, 0, st>>>(Xc, Yc, a, H);
      k_jacobi<<<1, 1024, jacobi_smem(kSpecK), st>>>(H, kSpecK, kSpecK, eig + m * kSpecK);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_pick_ranks(const asi_plan* pl, const double* eig, const double* energy, double eps, int r_max,
                              int* ranks, cudaStream_t st) {
  int64_t a[4] = {1, 1, 1, 1};
  for (int m = 0; m < pl->nd; ++m) a[m] = pl->dims[m];
  k_pick_ranks<<<1, 32, 0, st>>>(eig, energy, eps, r_max, pl->nd, a[0], a[1], a[2], a[3], pl->N, ranks);
  return cudaGetLastError();
}

size_t perplexity_ws_bytes() { return (size_t)kSqGrid * sizeof(double); }

cudaError_t launch_perplexity(const float* x, const float* y, int64_t n, double* out, double* part, cudaStream_t st) {
  k_sqdiff<<<kSqGrid, 256, 0, st>>>(x, y, n, part);
  k_sqdiff_sum<<<1, 32, 0, st>>>(part, kSqGrid, out);
  return cudaGetLastError();
}

}  // namespace asi
