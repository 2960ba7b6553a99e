// Small dense kernels of the token (linear-layer) path.
//
//   k_modeprod_stage : a mode product Y(o, j, i) = sum_k X(o, k, i) B(k, j) whose tensor has FEW columns
//                      (O * I small) but a long contracted mode -- the later core products of a token layer
//                      (Algorithm 1, core update).  One thread per column leaves such a product on a handful
//                      of CTAs walking the mode serially; here a cluster of up to eight CTAs owns X(o, :, i-chunk):
//                      each stages a slab of the mode's rows and of B in shared memory, its threads share the
//                      outputs (j, i), and the slabs' partial outputs meet in distributed shared memory.
//   k_lin_z4, k_lin_tail : the end of the linear backward (Sec. 3.1 footnote, derived steps L2-L3):
//                        Z4[o][k] = sum_{l1,l2} Z(l1, l2, o) core[l1][l2][k],   dW[o][d] = sum_k Z4[o][k] U[d][k].
//                      k_lin_z4 forms Z4 once (16 output rows per CTA, the leading indices shared between up to
//                      eight CTAs that each write their own share -- no atomics, the sum order is fixed);
//                      k_lin_tail adds the shares and expands 64 x 128 tiles of dW in 8 x 4 register tiles with
//                      coalesced stores.  dW is written exactly once.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include <algorithm>

#include "asi_internal.h"

namespace asi {

namespace {
constexpr int kStageThreads = 256;
constexpr int kLtO = 64, kLtD = 128;
constexpr int kLzO = 16, kLzLead = 64;
}  // namespace

// The CTAs of a cluster share one (o, i-chunk): CTA `rank` contracts the rows [rank * aslab, ..) of the mode and
// leaves its partial outputs in its own shared memory; rank 0 adds them in rank order through distributed shared
// memory and writes Y.  Both cluster barriers are reached by every thread of every CTA.
__global__ void __launch_bounds__(kStageThreads) k_modeprod_stage(ModeProdArgs p, int ichunk, int ksp, int aslab) {
  extern __shared__ __align__(16) float ms_smem[];
  namespace cg = cooperative_groups;
  cg::cluster_group cluster = cg::this_cluster();
  const int n = p.n_out;
  const int nic = (int)((p.I + ichunk - 1) / ichunk);
  const int rank = (int)(blockIdx.x % ksp);
  const int64_t tile = blockIdx.x / ksp;
  const int64_t o = tile / nic;
  const int i0 = (int)(tile % nic) * ichunk;
  const int ni = (int)((p.I - i0 < ichunk) ? (p.I - i0) : ichunk);
  const int k0 = rank * aslab;
  const int a = (int)((p.a - k0 < aslab) ? ((p.a > k0) ? p.a - k0 : 0) : aslab);   // rows of this CTA
  float* Xs = ms_smem;                            // [aslab][ichunk]
  float* Bs = Xs + (size_t)aslab * ichunk;        // [aslab][n]
  float* part = Bs + (size_t)aslab * n;           // [n][ichunk]
  const float* X = reinterpret_cast<const float*>(p.X) + (o * p.a + k0) * p.I + i0;
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
      v[u] = p.B[(e < a * n) ? (int64_t)(k0 + k) * p.ldb_k + (int64_t)j * p.ldb_j : 0];
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
    part[j * ichunk + i] = s0 + s1;
  }
  cluster.sync();
  if (rank == 0) {
    for (int e = tid; e < n * ni; e += kStageThreads) {
      const int j = e / ni, i = e - j * ni;
      float s = part[j * ichunk + i];
      for (int q = 1; q < ksp; ++q) s += cluster.map_shared_rank(part, q)[j * ichunk + i];
      p.Y[o * p.so + (int64_t)j * p.sj + (int64_t)(i0 + i) * p.si] = s;
    }
  }
  cluster.sync();                                 // the partials stay alive until rank 0 has read them
}

bool modeprod_stage_fits(const ModeProdArgs& p, int* ichunk, size_t* smem) {
  if (p.a < 64 || p.a > 8192 || p.O * p.I > 8192 || p.n_out > 128) return false;
  const int ksp = modeprod_stage_ksp(p.a);
  const int64_t aslab = (p.a + ksp - 1) / ksp;
  int ic = (int)(p.I < 64 ? p.I : 64);
  auto need_of = [&](int c) { return ((size_t)aslab * (c + p.n_out) + (size_t)p.n_out * c) * 4; };
  while (ic > 1 && need_of(ic) > 160 * 1024) ic = (ic + 1) / 2;
  if (need_of(ic) > 160 * 1024) return false;
  *ichunk = ic;
  *smem = need_of(ic);
  return true;
}

int modeprod_stage_ksp(int64_t a) {
  int k = 1;
  while (k < 8 && a / (2 * k) >= 32) k *= 2;      // at least 32 rows per CTA, at most the portable cluster size
  return k;
}

cudaError_t launch_modeprod_stage(const ModeProdArgs& p, int ichunk, size_t smem, cudaStream_t st) {
  ProfScope prof(ASI_K_MODEPROD, st, 4.0 * ((double)p.Q * p.a + (double)p.a * p.n_out + (double)p.Q * p.n_out));
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_modeprod_stage), smem);
  if (e != cudaSuccess) return e;
  const int64_t nic = (p.I + ichunk - 1) / ichunk;
  const int ksp = modeprod_stage_ksp(p.a);
  const int aslab = (int)((p.a + ksp - 1) / ksp);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(p.O * nic * ksp));
  cfg.blockDim = dim3(kStageThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)ksp;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_modeprod_stage, p, ichunk, ksp, aslab);
}

// ---------------------------------------------------------------------------------------------
// k_lin_z4 and k_lin_tail
// ---------------------------------------------------------------------------------------------
// Z4p[split][o][k] = sum over the split's leading indices of Z(lead, o) core[lead][k].  A CTA owns 16 output
// rows and one share of the leading indices; thread (o, kg) keeps the sums k = kg, kg + 16, ..
template <int NQ>
__global__ void __launch_bounds__(256) k_lin_z4(LinTailArgs p) {
  extern __shared__ __align__(16) float lt_smem[];
  const int r = p.r;
  float* Zc = lt_smem;                               // [kLzLead][16 + 1]
  float* Sc = Zc + kLzLead * (kLzO + 1);             // [kLzLead][r]
  const int tid = threadIdx.x;
  const int o0 = blockIdx.x * kLzO;
  const int nlead = p.L1 * p.L2;
  const int per = ((nlead + p.nsplit - 1) / p.nsplit + kLzLead - 1) / kLzLead * kLzLead;
  const int lbeg = blockIdx.y * per, lend = (lbeg + per < nlead) ? lbeg + per : nlead;
  const int po = tid & (kLzO - 1), kg = tid >> 4;
  constexpr int NS = 4 * NQ;                         // core values of a chunk per thread: 64 r / 256 <= 4 NQ
  float acc[NQ];
#pragma unroll
  for (int q = 0; q < NQ; ++q) acc[q] = 0.f;
  float vz[4], vs[NS];
  // the values of the chunk that starts at l0, into registers (loads only: nothing here uses them)
  auto fetch = [&](int l0) {
    const int nl = (lend - l0 < kLzLead) ? lend - l0 : kLzLead;
#pragma unroll
    for (int u = 0; u < 4; ++u) {                    // 64 x 16 values, four per thread
      const int e = tid + u * 256;
      int l, o;
      if (p.lead_fastest) { o = e / kLzLead; l = e - o * kLzLead; } else { l = e >> 4; o = e & (kLzO - 1); }
      const int lead = l0 + l, l1 = lead / p.L2, l2 = lead - l1 * p.L2;
      const bool on = l < nl && o0 + o < p.Dout;
      vz[u] = p.Z[on ? (int64_t)l1 * p.s1 + (int64_t)l2 * p.s2 + (int64_t)(o0 + o) * p.so : 0];
    }
#pragma unroll
    for (int u = 0; u < NS; ++u) {
      const int e = tid + u * 256;
      vs[u] = p.core[(e < nl * r) ? (int64_t)l0 * r + e : 0];
    }
  };
  if (lbeg < lend) fetch(lbeg);
  for (int l0 = lbeg; l0 < lend; l0 += kLzLead) {
    const int nl = (lend - l0 < kLzLead) ? lend - l0 : kLzLead;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = tid + u * 256;
      int l, o;
      if (p.lead_fastest) { o = e / kLzLead; l = e - o * kLzLead; } else { l = e >> 4; o = e & (kLzO - 1); }
      Zc[l * (kLzO + 1) + o] = (l < nl && o0 + o < p.Dout) ? vz[u] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < NS; ++u) {
      const int e = tid + u * 256;
      if (e < kLzLead * r) Sc[e] = (e < nl * r) ? vs[u] : 0.f;
    }
    __syncthreads();
    if (l0 + kLzLead < lend) fetch(l0 + kLzLead);    // the next chunk travels while this one is used
#pragma unroll 4
    for (int l = 0; l < kLzLead; ++l) {
      const float z = Zc[l * (kLzO + 1) + po];
#pragma unroll
      for (int q = 0; q < NQ; ++q)
        if (kg + 16 * q < r) acc[q] = fmaf(z, Sc[l * r + kg + 16 * q], acc[q]);
    }
    __syncthreads();
  }
  if (o0 + po < p.Dout) {
    float* dst = p.Z4p + ((int64_t)blockIdx.y * p.Dout + o0 + po) * r;
#pragma unroll
    for (int q = 0; q < NQ; ++q)
      if (kg + 16 * q < r) dst[kg + 16 * q] = acc[q];
  }
}

// dW[o][d] = sum_k Z4[o][k] U[d][k], Z4 = the sum of the nsplit shares: 64 x 128 tile per CTA, 8 x 4 per thread.
// Rows of Z4 and of U sit in shared memory with a pitch of 4 * (odd number) floats and zeros up to it, so the
// k loop reads four k at a time with 16-byte loads (the 8 Z4 rows of a warp are broadcasts; the 32 lanes' U
// rows fall in distinct banks): 12 loads per 128 multiply-adds.
__global__ void __launch_bounds__(256) k_lin_tail(LinTailArgs p, int PR) {
  extern __shared__ __align__(16) float lt_smem[];
  const int r = p.r;
  float* Z4s = lt_smem;                              // [64][PR]
  float* Us = Z4s + kLtO * PR;                       // [128][PR]
  const int tid = threadIdx.x, lane = tid & 31;
  const int o0 = blockIdx.x * kLtO, d0 = blockIdx.y * kLtD;
  const int no = (p.Dout - o0 < kLtO) ? p.Dout - o0 : kLtO;
  const int nd = (p.Din - d0 < kLtD) ? p.Din - d0 : kLtD;
  const float* zsrc = p.Z4p + (int64_t)o0 * r;
  const int64_t zstep = (int64_t)p.Dout * r;
  for (int e0 = 0; e0 < kLtO * PR; e0 += 4 * 256) {  // e = (o, k) over the padded pitch
    float v[4] = {0.f, 0.f, 0.f, 0.f};
    int src[4];
    bool on[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + tid + u * 256, o = e / PR, k = e - o * PR;
      on[u] = e < kLtO * PR && o < no && k < r;
      src[u] = on[u] ? o * r + k : 0;
    }
    for (int sp = 0; sp < p.nsplit; ++sp) {
      float t[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) t[u] = zsrc[sp * zstep + src[u]];
#pragma unroll
      for (int u = 0; u < 4; ++u) v[u] += t[u];
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + tid + u * 256;
      if (e < kLtO * PR) Z4s[e] = on[u] ? v[u] : 0.f;
    }
  }
  const float* usrc = p.U + (int64_t)d0 * r;
  for (int e0 = 0; e0 < kLtD * PR; e0 += 8 * 256) {
    float v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + tid + u * 256, d = e / PR, k = e - d * PR;
      v[u] = usrc[(e < kLtD * PR && d < nd && k < r) ? d * r + k : 0];
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + tid + u * 256, d = e / PR, k = e - d * PR;
      if (e < kLtD * PR) Us[e] = (d < nd && k < r) ? v[u] : 0.f;
    }
  }
  __syncthreads();
  // dW[o0 + o][d0 + d] for o = 8 to .. 8 to + 7, d = lane + 32 i
  const int to = tid >> 5;
  float out[8][4];
#pragma unroll
  for (int x = 0; x < 8; ++x)
#pragma unroll
    for (int y = 0; y < 4; ++y) out[x][y] = 0.f;
  const float* zrow = Z4s + 8 * to * PR;
  const float* urow = Us + lane * PR;
  for (int k = 0; k < PR; k += 4) {
    float4 zz[8], uu[4];
#pragma unroll
    for (int x = 0; x < 8; ++x) zz[x] = *reinterpret_cast<const float4*>(zrow + x * PR + k);
#pragma unroll
    for (int y = 0; y < 4; ++y) uu[y] = *reinterpret_cast<const float4*>(urow + 32 * y * PR + k);
#pragma unroll
    for (int x = 0; x < 8; ++x)
#pragma unroll
      for (int y = 0; y < 4; ++y) {
        out[x][y] = fmaf(zz[x].x, uu[y].x, out[x][y]);
        out[x][y] = fmaf(zz[x].y, uu[y].y, out[x][y]);
        out[x][y] = fmaf(zz[x].z, uu[y].z, out[x][y]);
        out[x][y] = fmaf(zz[x].w, uu[y].w, out[x][y]);
      }
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

int lin_tail_nsplit(int nlead, int64_t Dout) {
  const int64_t tiles = (Dout + kLzO - 1) / kLzO;
  int64_t ns = 592 / (tiles > 0 ? tiles : 1);       // about four CTAs per SM
  const int64_t cap = (nlead + kLzLead - 1) / kLzLead;      // at least one chunk of leads per share
  if (ns > cap) ns = cap;
  if (ns > 8) ns = 8;
  return (int)(ns < 1 ? 1 : ns);
}

cudaError_t launch_lin_tail(const LinTailArgs& p, cudaStream_t st) {
  int PR = (p.r + 3) / 4 * 4;                     // pitch: 4 * (odd number) floats
  if ((PR / 4) % 2 == 0) PR += 4;
  ProfScope prof(ASI_K_MODEPROD, st, 4.0 * ((double)p.Dout * p.Din + (double)p.L1 * p.L2 * p.Dout));
  {
    const size_t smem = 4 * ((size_t)kLzLead * (kLzO + 1) + (size_t)kLzLead * p.r);
    dim3 grid((unsigned)((p.Dout + kLzO - 1) / kLzO), (unsigned)p.nsplit);
    cudaError_t e;
    if (p.r <= 32) {
      e = opt_in_smem(reinterpret_cast<const void*>(k_lin_z4<2>), smem);
      if (e != cudaSuccess) return e;
      k_lin_z4<2><<<grid, 256, smem, st>>>(p);
    } else if (p.r <= 64) {
      e = opt_in_smem(reinterpret_cast<const void*>(k_lin_z4<4>), smem);
      if (e != cudaSuccess) return e;
      k_lin_z4<4><<<grid, 256, smem, st>>>(p);
    } else {
      e = opt_in_smem(reinterpret_cast<const void*>(k_lin_z4<8>), smem);
      if (e != cudaSuccess) return e;
      k_lin_z4<8><<<grid, 256, smem, st>>>(p);
    }
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  const size_t smem = 4 * (size_t)(kLtO + kLtD) * PR;
  dim3 grid((unsigned)((p.Dout + kLtO - 1) / kLtO), (unsigned)((p.Din + kLtD - 1) / kLtD));
  cudaError_t e = opt_in_smem(reinterpret_cast<const void*>(k_lin_tail), smem);
  if (e != cudaSuccess) return e;
  k_lin_tail<<<grid, 256, smem, st>>>(p, PR);
  return cudaGetLastError();
}

}  // namespace asi
