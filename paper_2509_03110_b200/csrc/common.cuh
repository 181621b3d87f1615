// common.cuh -- shared device helpers of the LSAM CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace lsam {

typedef __nv_bfloat16 bf16;

// Device status word: kernels OR these bits in, the host maps them to error codes.
enum : int { STATUS_NONFINITE = 1, STATUS_TIMEOUT = 2, STATUS_BAD_INDEX = 4 };

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
