// Counter-based Gaussian test matrices for the cold start (Algorithm 1, t = 0: V ~ N(0, 1)).  The paper fixes no
// generator; this one is Philox4x32-10 (Salmon et al., SC'11): key = the 64-bit seed, counter = (group index low,
// group index high, stream, 0), four 32-bit words per group.  A word becomes a uniform with 24 significant bits,
// u = ((x >> 9) + 0.5) 2^-23, and the pairs (x0, x1), (x2, x3) go through Box-Muller in fp32.  Element e of a
// stream is value e mod 4 of group e div 4, so any part of a stream can be drawn by itself.
#include <algorithm>

#include "asi_internal.h"

namespace asi {

namespace {

struct Words { uint32_t w[4]; };

__device__ __forceinline__ Words philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                               uint32_t k1) {
  constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
    const uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += W0; k1 += W1;
  }
  Words r;
  r.w[0] = c0; r.w[1] = c1; r.w[2] = c2; r.w[3] = c3;
  return r;
}

__device__ __forceinline__ float unit(uint32_t x) { return ((float)(x >> 9) + 0.5f) * 1.1920928955078125e-7f; }

__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& z0, float& z1) {
  const float rad = sqrtf(-2.f * logf(unit(xa)));
  float s, c;
  sincospif(2.f * unit(xb), &s, &c);
  z0 = rad * c;
  z1 = rad * s;
}

__global__ void __launch_bounds__(256) k_philox_words(uint64_t seed, uint32_t stream, int64_t n_groups, uint32_t* out) {
  const int64_t g = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (g >= n_groups) return;
  const Words r = philox4x32_10((uint32_t)g, (uint32_t)((uint64_t)g >> 32), stream, 0u, (uint32_t)seed,
                                (uint32_t)(seed >> 32));
  *reinterpret_cast<uint4*>(out + 4 * g) = make_uint4(r.w[0], r.w[1], r.w[2], r.w[3]);
}

__global__ void __launch_bounds__(256) k_fill_gaussian(uint64_t seed, uint32_t stream, int64_t n, float* out) {
  const int64_t ng = (n + 3) / 4;
  for (int64_t g = (int64_t)blockIdx.x * 256 + threadIdx.x; g < ng; g += (int64_t)gridDim.x * 256) {
    const Words r = philox4x32_10((uint32_t)g, (uint32_t)((uint64_t)g >> 32), stream, 0u, (uint32_t)seed,
                                  (uint32_t)(seed >> 32));
    float z[4];
    box_muller(r.w[0], r.w[1], z[0], z[1]);
    box_muller(r.w[2], r.w[3], z[2], z[3]);
    if (4 * g + 3 < n && (reinterpret_cast<uintptr_t>(out) & 15u) == 0) {
      *reinterpret_cast<float4*>(out + 4 * g) = make_float4(z[0], z[1], z[2], z[3]);
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (4 * g + i < n) out[4 * g + i] = z[i];
    }
  }
}

}  // namespace

cudaError_t launch_philox_words(uint64_t seed, uint32_t stream, int64_t n_groups, uint32_t* out, cudaStream_t st) {
  if (n_groups <= 0) return cudaSuccess;
  k_philox_words<<<(unsigned)((n_groups + 255) / 256), 256, 0, st>>>(seed, stream, n_groups, out);
  return cudaGetLastError();
}

cudaError_t launch_fill_gaussian(uint64_t seed, uint32_t stream, int64_t n, float* out, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  const int64_t ng = (n + 3) / 4;
  const int64_t blocks = std::min<int64_t>((ng + 255) / 256, 148 * 8);
  k_fill_gaussian<<<(unsigned)blocks, 256, 0, st>>>(seed, stream, n, out);
  return cudaGetLastError();
}

}  // namespace asi
