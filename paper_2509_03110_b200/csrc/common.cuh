// common.cuh -- shared device helpers of the LSAM CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lsam {

typedef __nv_bfloat16 bf16;

// Device status word: kernels OR these bits in, the host maps them to error codes.
enum : int { STATUS_NONFINITE = 1, STATUS_TIMEOUT = 2, STATUS_BAD_INDEX = 4 };

// Programmatic dependent launch.  Every kernel of the library opens with this pair: `launch_dependents` lets the next
// kernel of the stream, if it was launched with programmatic stream serialization, make its blocks resident as soon as
// every block of this grid has started (so its launch latency and set-up overlap this grid's tail); `wait` then holds
// this block until the grids before it have completed and their writes are visible.  No global memory is touched before
// the wait, so a kernel never reads what a predecessor has yet to write nor overwrites what it still reads; the chain is
// transitive because a grid completes only after its own wait has returned.  Both are no-ops in a plain launch.
__device__ inline void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ inline void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ inline void grid_dep_sync() { grid_dep_launch(); grid_dep_wait(); }

__host__ __device__ inline int64_t round_up(int64_t a, int64_t b) { return (a + b - 1) / b * b; }
__host__ __device__ inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// ---- schedule hash (integer, bit-exact): SplitMix64 finaliser chained over (seed ^ tag, t, k * 2^20 + j)
__host__ __device__ inline uint64_t mix64(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xbf58476d1ce4e5b9ULL;
  z = (z ^ (z >> 27)) * 0x94d049bb133111ebULL;
  return z ^ (z >> 31);
}
constexpr uint64_t kTagIdx = 0x6c73616d5f696478ULL;    // "lsam_idx"
constexpr uint64_t kTagStale = 0x6c73616d5f73746cULL;  // "lsam_stl"
constexpr uint64_t kTagAct = 0x6c73616d5f616374ULL;    // "lsam_act"
constexpr uint64_t kTagOrd = 0x6c73616d5f6f7264ULL;    // "lsam_ord"
__host__ __device__ inline uint64_t schedule_hash(uint64_t seed, uint64_t tag, uint64_t t, uint64_t k, uint64_t j) {
  return mix64(mix64(mix64(seed ^ tag) + t) + ((k << 20) + j));
}

// ---- Langevin noise: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC 2011) + Box-Muller, four normals per block.
//   counter = (group low 32 bits, segment, worker, tick low 32 bits), key = (seed low ^ "lang", seed high ^ tick high)
//   u = ((r >> 8) + 0.5) 2^-24 (exact in binary32), (z0, z1) = sqrt(-2 ln u0) (cos 2 pi u1, sin 2 pi u1), (z2, z3) from (u2, u3)
__device__ inline void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1, uint32_t (&out)[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0, n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}
__device__ inline void langevin_noise4(uint64_t seed, uint64_t t, uint32_t k, uint32_t seg, uint64_t group, float (&z)[4]) {
  uint32_t r[4];
  philox4x32_10((uint32_t)group, seg, k, (uint32_t)t, (uint32_t)seed ^ 0x6c616e67u, (uint32_t)(seed >> 32) ^ (uint32_t)(t >> 32), r);
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const float u0 = ((float)(r[2 * h] >> 8) + 0.5f) * (1.0f / 16777216.0f);
    const float u1 = ((float)(r[2 * h + 1] >> 8) + 0.5f) * (1.0f / 16777216.0f);
    const float rad = sqrtf(-2.0f * logf(u0));
    float sn, cs;
    sincospif(2.0f * u1, &sn, &cs);
    z[2 * h] = rad * cs;
    z[2 * h + 1] = rad * sn;
  }
}

// ---- element conversion between the accumulator type (float) and a storage type
template <typename T> __device__ inline T from_float(float v);
template <> __device__ inline float from_float<float>(float v) { return v; }
template <> __device__ inline bf16 from_float<bf16>(float v) { return __float2bfloat16_rn(v); }
__device__ inline float to_float(float v) { return v; }
__device__ inline float to_float(bf16 v) { return __bfloat162float(v); }

// ---- fixed-order reductions: xor-shuffle tree inside a warp, then the warp totals are added in warp order
__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline int warp_sum(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
// Result valid in thread 0.  `smem` holds at least blockDim.x / 32 elements.
template <typename T>
__device__ inline T block_sum(T v, T* smem) {
  v = warp_sum(v);
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  if (lane == 0) smem[w] = v;
  __syncthreads();
  T total = T(0);
  if (threadIdx.x == 0)
    for (int i = 0; i < nw; ++i) total += smem[i];
  __syncthreads();
  return total;
}

}  // namespace lsam
