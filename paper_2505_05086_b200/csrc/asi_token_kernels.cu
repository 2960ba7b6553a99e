// Small dense kernels of the token (linear-layer) path.
//
//   k_modeprod_stage : a mode product Y(o, j, i) = sum_k X(o, k, i) B(k, j) whose tensor has FEW columns
//                      (O * I small) but a long contracted mode -- the later core products of a token layer
//                      (Algorithm 1, core update).  One thread per column leaves such a product on a handful
//                      of CTAs walking the mode serially; here a CTA stages X(o, :, i-chunk) and B in shared
//                      memory and its threads share the outputs (j, i).
//   k_lin_tail       : the end of the linear backward (Sec. 3.1 footnote, derived steps L2-L3) in one launch:
//                        Z4[o][k] = sum_{l1,l2} Z(l1, l2, o) core[l1][l2][k],   dW[o][d] = sum_k Z4[o][k] U[d][k].
//                      A CTA owns 64 output rows x 128 columns of dW: it forms its 64 rows of Z4 in shared
//                      memory (recomputed per column tile: the contraction is small next to the 4-byte
//                      write of every dW entry), then expands them in 8 x 4 register tiles with coalesced
//                      stores.  dW is written exactly once.
#include "asi_internal.h"

namespace asi {

namespace {
constexpr int kStageThreads = 256;
constexpr int kLtO = 64, kLtD = 128, kLtLead = 32;
}  // namespace

__global__ void __launch_bounds__(kStageThreads) k_modeprod_stage(ModeProdArgs p, int ichunk) {
  extern __shared__ __align__(16) float ms_smem[];
  const int a = (int)p.a, n = p.n_out;
  const int nic = (int)((p.I + ichunk - 1) / ichunk);
  const int64_t o = blockIdx.x / nic;
  const int i0 = (int)(blockIdx.x % nic) * ichunk;
  const int ni = (int)((p.I - i0 < ichunk) ? (p.I - i0) : ichunk);
  float* Xs = ms_smem;                       // [a][ichunk]
  float* Bs = Xs + (size_t)a * ichunk;       // [a][n]
  const float* X = reinterpret_cast<const float*>(p.X) + o * p.a * p.I + i0;
  const int tid = threadIdx.x;
  // all loads of a batch first, then the stores (a load next to the store of its value waits for it)
  for (int e0 = 0; e0 < a * ichunk; e0 += 8 * kStageThreads) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + tid + u * kStageThreads;
      const int k = e / ichunk, i = e - k * ichunk;
      v[u] = X[(e < a * ichunk && i < ni) ? (int64_t)k * p.I + i : 0];
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + tid + u * kStageThreads;
      if (e < a * ichunk) Xs[e] = (e % ichunk < ni) ? v[u] : 0.f;
    }
  }
  for (int e0 = 0; e0 < a * n; e0 += 8 * kStageThreads) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + tid + u * kStageThreads;
      const int k = e / n, j = e - k * n;
      v[u] = p.B[(e < a * n) ? (int64_t)k * p.ldb_k + (int64_t)j * p.ldb_j : 0];
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + tid + u * kStageThreads;
      if (e < a * n) Bs[e] = v[u];
    }
  }
  __syncthreads();
  for (int e = tid; e < n * ni; e += kStageThreads) {
    const int j = e / ni, i = e - j * ni;
    float s0 = 0.f, s1 = 0.f;
    int k = 0;
    for (; k + 1 < a; k += 2) {
      s0 = fmaf(Xs[k * ichunk + i], Bs[k * n + j], s0);
      s1 = fmaf(Xs[(k + 1) * ichunk + i], Bs[(k + 1) * n + j], s1);
    }
    if (k < a) s0 = fmaf(Xs[k * ichunk + i], Bs[k * n + j], s0);
    p.Y[o * p.so + (int64_t)j * p.sj + (int64_t)(i0 + i) * p.si] = s0 + s1;
  }
}

bool modeprod_stage_fits(const ModeProdArgs& p, int* ichunk, size_t* smem) {
  if (p.a < 64 || p.a > 8192 || p.O * p.I > 8192 || p.n_out > 128) return false;
  int ic = (int)(p.I < 64 ? p.I : 64);
  while (ic > 1 && (size_t)p.a * (ic + p.n_out) * 4 > 160 * 1024) ic = (ic + 1) / 2;
  const size_t need = (size_t)p.a * (ic + p.n_out) * 4;
  if (need > 160 * 1024) return false;
  *ichunk = ic;
  *smem = need;
  return true;
}

cudaError_t launch_modeprod_stage(const ModeProdArgs& p, int ichunk, size_t smem, cudaStream_t st) {
  ProfScope prof(ASI_K_MODEPROD, st, 4.0 * ((double)p.Q * p.a + (double)p.a * p.n_out + (double)p.Q * p.n_out));
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_modeprod_stage), smem);
  if (e != cudaSuccess) return e;
  const int64_t nic = (p.I + ichunk - 1) / ichunk;
  k_modeprod_stage<<<(unsigned)(p.O * nic), kStageThreads, smem, st>>>(p, ichunk);
  return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// k_lin_tail
// ---------------------------------------------------------------------------------------------
template <int NQ>      // a thread of phase 1 keeps NQ sums: ranks up to 4 NQ
__global__ void __launch_bounds__(256) k_lin_tail(LinTailArgs p) {
  extern __shared__ __align__(16) float lt_smem[];
  const int r = p.r, PR = r | 1;                     // odd pitch: conflict-free reads down a column of rows
  float* Z4s = lt_smem;                              // [64][PR]
  float* Us = Z4s + kLtO * PR;                       // [128][PR]
  float* Zc = Us + kLtD * PR;                        // [kLtLead][64 + 1]
  float* Sc = Zc + kLtLead * (kLtO + 1);             // [kLtLead][r]
  const int tid = threadIdx.x, lane = tid & 31;
  const int o0 = blockIdx.x * kLtO, d0 = blockIdx.y * kLtD;
  const int nlead = p.L1 * p.L2;
  // ---- phase 1: Z4s[o][k] = sum_lead Z(lead, o0 + o) core[lead][k]; thread (o, kg) keeps k = kg, kg + 4, ..
  const int po = tid & 63, kg = tid >> 6;
  float acc[NQ];
#pragma unroll
  for (int q = 0; q < NQ; ++q) acc[q] = 0.f;
  for (int l0 = 0; l0 < nlead; l0 += kLtLead) {
    const int nl = (nlead - l0 < kLtLead) ? nlead - l0 : kLtLead;
    {
      float v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {                  // 32 x 64 values, eight per thread, loads first
        const int e = tid + u * 256;
        int l, o;
        if (p.lead_fastest) { o = e / kLtLead; l = e - o * kLtLead; } else { l = e >> 6; o = e & 63; }
        const int lead = l0 + l, l1 = lead / p.L2, l2 = lead - l1 * p.L2;
        const bool on = l < nl && o0 + o < p.Dout;
        v[u] = p.Z[on ? (int64_t)l1 * p.s1 + (int64_t)l2 * p.s2 + (int64_t)(o0 + o) * p.so : 0];
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int e = tid + u * 256;
        int l, o;
        if (p.lead_fastest) { o = e / kLtLead; l = e - o * kLtLead; } else { l = e >> 6; o = e & 63; }
        Zc[l * (kLtO + 1) + o] = (l < nl && o0 + o < p.Dout) ? v[u] : 0.f;
      }
      for (int e = tid; e < kLtLead * r; e += 256) {
        const int l = e / r, k = e - l * r;
        Sc[e] = (l < nl) ? p.core[(int64_t)(l0 + l) * r + k] : 0.f;
      }
    }
    __syncthreads();
#pragma unroll 4
    for (int l = 0; l < kLtLead; ++l) {
      const float z = Zc[l * (kLtO + 1) + po];
#pragma unroll
      for (int q = 0; q < NQ; ++q)
        if (kg + 4 * q < r) acc[q] = fmaf(z, Sc[l * r + kg + 4 * q], acc[q]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int q = 0; q < NQ; ++q)
    if (kg + 4 * q < r) Z4s[po * PR + kg + 4 * q] = acc[q];
  // the factor rows of this column tile
  for (int e0 = 0; e0 < kLtD * r; e0 += 8 * 256) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + tid + u * 256, d = e / r;
      v[u] = p.U[(e < kLtD * r && d0 + d < p.Din) ? (int64_t)(d0 + d) * r + (e - d * r) : 0];
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + tid + u * 256, d = e / r;
      if (e < kLtD * r) Us[d * PR + (e - d * r)] = (d0 + d < p.Din) ? v[u] : 0.f;
    }
  }
  __syncthreads();
  // ---- phase 2: dW[o0 + o][d0 + d] for o = 8 to .. 8 to + 7, d = lane + 32 i
  const int to = tid >> 5;
  float out[8][4];
#pragma unroll
  for (int x = 0; x < 8; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) out[x][y] = 0.f;
  for (int k = 0; k < r; ++k) {
    float zz[8], uu[4];
#pragma unroll
    for (int x = 0; x < 8; ++x) zz[x] = Z4s[(8 * to + x) * PR + k];
#pragma unroll
    for (int y = 0; y < 4; ++y) uu[y] = Us[(lane + 32 * y) * PR + k];
#pragma unroll
    for (int x = 0; x < 8; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) out[x][y] = fmaf(zz[x], uu[y], out[x][y]);
  }
#pragma unroll
  for (int x = 0; x < 8; ++x) {
    const int o = o0 + 8 * to + x;
    if (o >= p.Dout) continue;
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int d = d0 + lane + 32 * y;
      if (d < p.Din) p.dW[(int64_t)o * p.Din + d] = out[x][y];
    }
  }
}

bool lin_tail_supported(int r) { return r >= 1 && r <= 128; }

cudaError_t launch_lin_tail(const LinTailArgs& p, cudaStream_t st) {
  const int PR = p.r | 1;
  const size_t smem = 4 * ((size_t)(kLtO + kLtD) * PR + (size_t)kLtLead * (kLtO + 1) + (size_t)kLtLead * p.r);
  ProfScope prof(ASI_K_MODEPROD, st, 4.0 * ((double)p.Dout * p.Din + (double)p.L1 * p.L2 * p.Dout));
  dim3 grid((unsigned)((p.Dout + kLtO - 1) / kLtO), (unsigned)((p.Din + kLtD - 1) / kLtD));
  cudaError_t e;
  if (p.r <= 32) {
    e = opt_in_smem(reinterpret_cast<const void*>(k_lin_tail<8>), smem);
    if (e != cudaSuccess) return e;
    k_lin_tail<8><<<grid, 256, smem, st>>>(p);
  } else if (p.r <= 64) {
    e = opt_in_smem(reinterpret_cast<const void*>(k_lin_tail<16>), smem);
    if (e != cudaSuccess) return e;
    k_lin_tail<16><<<grid, 256, smem, st>>>(p);
  } else {
    e = opt_in_smem(reinterpret_cast<const void*>(k_lin_tail<32>), smem);
    if (e != cudaSuccess) return e;
    k_lin_tail<32><<<grid, 256, smem, st>>>(p);
  }
  return cudaGetLastError();
}

}  // namespace asi
