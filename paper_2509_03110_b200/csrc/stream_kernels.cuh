// stream_kernels.cuh -- schedule, per-replica norm, perturbation, fused worker update, centre update.
// All of these are HBM-streaming kernels over the stacked [K, ld] state (ld = padded row length).
#pragma once

#include "common.cuh"

namespace lsam {

// ------------------------------------------------------------------------------------------------ S0 schedule
// hist.v[s] = centre version that was current when step t - s started (s = 0..15), clamped at step 0.
struct VerHist { int v[16]; };

// grid K, block 128.  idx [K, B]; stale, ver, slot [K].  slot = ring slot holding the version read.
// k_offset: global index of worker 0 (sharded contexts).  active (nullable) [K]: asynchronous progress (unsharded only).  Worker k is ready at this tick when H_act mod 256 < active_num; ready
// workers are served in the order of (H_ord, k) and only the first `budget` of them step (budget = n tau minus the
// iterations already counted since the last sync); active[k] = 1 for those.
__global__ void __launch_bounds__(128)
schedule_kernel(uint64_t seed, uint64_t t, int64_t n_samples, int B, int stale_max, VerHist hist, int ring,
                int32_t* __restrict__ idx, int32_t* __restrict__ stale, int32_t* __restrict__ ver, int32_t* __restrict__ slot,
                int K, int active_num, int64_t budget, int32_t* __restrict__ active, int k_offset) {
  grid_dep_sync();
  __shared__ int red[4];
  const uint64_t k = blockIdx.x;
  const uint64_t kg = k + (uint64_t)k_offset;  // global worker index: the key of the minibatch and staleness streams
  if (idx != nullptr)
    for (int j = threadIdx.x; j < B; j += blockDim.x)
      idx[k * B + j] = (int32_t)(schedule_hash(seed, kTagIdx, t, kg, (uint64_t)j) % (uint64_t)n_samples);
  if (threadIdx.x == 0) {
    const int s = (int)(schedule_hash(seed, kTagStale, t, kg, 0) % (uint64_t)(stale_max + 1));
    const int u = hist.v[s];
    if (stale) stale[k] = s;
    if (ver) ver[k] = u;
    if (slot) slot[k] = u >= 0 ? u % ring : 0;
  }
  if (active != nullptr) {
    const bool ready_k = (schedule_hash(seed, kTagAct, t, k, 0) % 256ULL) < (uint64_t)active_num;
    const uint64_t key_k = schedule_hash(seed, kTagOrd, t, k, 0);
    int cnt = 0;  // ready workers served before worker k
    for (int j = threadIdx.x; j < K; j += blockDim.x) {
      const bool ready_j = (schedule_hash(seed, kTagAct, t, (uint64_t)j, 0) % 256ULL) < (uint64_t)active_num;
      const uint64_t key_j = schedule_hash(seed, kTagOrd, t, (uint64_t)j, 0);
      cnt += (ready_j && (key_j < key_k || (key_j == key_k && (uint64_t)j < k))) ? 1 : 0;
    }
    const int rank = block_sum<int>(cnt, red);
    if (threadIdx.x == 0) active[k] = (ready_k && (int64_t)rank < budget) ? 1 : 0;
  }
}

// ------------------------------------------------------------------------------------------------ S3 norm
// Pass 1: partial[k][chunk] = sum of squares of one fixed chunk of g_k, in a fixed order:
// per thread ITER vectors in ascending address order, xor-shuffle tree, warps in ascending order.
constexpr int kNormThreads = 256;
constexpr int kNormIter = 8;
template <int VEC>
__host__ __device__ constexpr int64_t norm_chunk() { return (int64_t)kNormThreads * VEC * kNormIter; }

template <int VEC>
__global__ void __launch_bounds__(kNormThreads)
sumsq_partial_kernel(const float* __restrict__ g, int64_t ldg, int64_t n, float* __restrict__ partial, int64_t nchunks,
                     const int32_t* __restrict__ active) {
  grid_dep_sync();
  __shared__ float red[kNormThreads / 32];
  const int k = blockIdx.y;
  if (active != nullptr && !active[k]) return;  // a waiting worker (block-uniform)
  const int64_t base = (int64_t)blockIdx.x * norm_chunk<VEC>();
  const float* row = g + (int64_t)k * ldg;
  float s = 0.f;
  if (VEC == 4) {
    float4 r[kNormIter];
#pragma unroll
    for (int i = 0; i < kNormIter; ++i) {
      const int64_t j = base + ((int64_t)i * kNormThreads + threadIdx.x) * 4;
      r[i] = (j < n) ? __ldcs(reinterpret_cast<const float4*>(row + j)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int i = 0; i < kNormIter; ++i) s += (r[i].x * r[i].x + r[i].y * r[i].y) + (r[i].z * r[i].z + r[i].w * r[i].w);
  } else {
#pragma unroll
    for (int i = 0; i < kNormIter; ++i) {
      const int64_t j = base + (int64_t)i * kNormThreads + threadIdx.x;
      const float a = (j < n) ? row[j] : 0.f;
      s += a * a;
    }
  }
  const float tot = block_sum<float>(s, red);
  if (threadIdx.x == 0) partial[(int64_t)k * nchunks + blockIdx.x] = tot;
}

// Anchor gap (Lemma 5): partial sums of squares of x_k - y over fixed chunks of norm_chunk<4>() elements, same order as
// above; the rows are 16-byte aligned, the tail of a row whose length is not a multiple of 4 is masked.  grid (chunks, K).
// slot (nullable) [K]: replica k is measured against row slot[k] of y (the centre version it reads, row stride ldx) instead of row 0.
__global__ void __launch_bounds__(kNormThreads)
gap_sumsq_partial_kernel(const float* __restrict__ x, int64_t ldx, const float* __restrict__ y, int64_t n,
                         float* __restrict__ partial, int64_t nchunks, const int32_t* __restrict__ slot,
                         const int32_t* __restrict__ active) {
  grid_dep_sync();
  __shared__ float red[kNormThreads / 32];
  const int k = blockIdx.y;
  if (active != nullptr && !active[k]) return;
  const int64_t base = (int64_t)blockIdx.x * norm_chunk<4>();
  const float* row = x + (int64_t)k * ldx;
  if (slot != nullptr) y += (int64_t)slot[k] * ldx;
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < kNormIter; ++i) {
    const int64_t j = base + ((int64_t)i * kNormThreads + threadIdx.x) * 4;
    if (j >= n) continue;
    const float4 a = *reinterpret_cast<const float4*>(row + j);   // rows are padded to a multiple of 4 elements
    const float4 b = __ldg(reinterpret_cast<const float4*>(y + j));
    const float d0 = a.x - b.x, d1 = a.y - b.y, d2 = a.z - b.z, d3 = a.w - b.w;
    s += (d0 * d0 + (j + 1 < n ? d1 * d1 : 0.f)) + ((j + 2 < n ? d2 * d2 : 0.f) + (j + 3 < n ? d3 * d3 : 0.f));
  }
  const float tot = block_sum<float>(s, red);
  if (threadIdx.x == 0) partial[(int64_t)k * nchunks + blockIdx.x] = tot;
}

// Pass 2: norm[k] = sqrt(sum of partials) accumulated in double in a fixed order; scale[k] = rho / (norm + gamma).
// grid K, block 256; partial has row stride nchunks, of which the first nused are summed.  A non-finite norm raises STATUS_NONFINITE and leaves scale = 0 (no perturbation).
__global__ void __launch_bounds__(256)
norm_finalize_kernel(const float* __restrict__ partial, int64_t nchunks, int64_t nused, float rho, float gamma,
                     float* __restrict__ norm_out, float* __restrict__ scale_out, int* __restrict__ status,
                     const int32_t* __restrict__ active) {
  grid_dep_sync();
  __shared__ double red[8];
  const int k = blockIdx.x;
  if (active != nullptr && !active[k]) return;
  double s = 0.0;
  for (int64_t c = threadIdx.x; c < nused; c += blockDim.x) s += (double)partial[(int64_t)k * nchunks + c];
  const double tot = block_sum<double>(s, red);
  if (threadIdx.x == 0) {
    const float nrm = (float)sqrt(tot);
    norm_out[k] = nrm;
    if (scale_out) {
      if (isfinite(nrm)) {
        scale_out[k] = rho / (nrm + gamma);
      } else {
        scale_out[k] = 0.f;
        atomicOr(status, STATUS_NONFINITE);
      }
    }
  }
}

// Pull weight of a stationary kernel phi(x - y) (Corollary 8 and the remark after it): the worker's pull is
// grad phi(x - y) = w(r) (x - y) with r = ||x_k - y||.  partial holds the sums of squares of x_k - y per chunk (as above);
// weight[k] = w(r_k).  kind: 0 Gaussian w = lambda; 1 exponential-power phi = (lambda / a) r^a, w = lambda r^(a-2), w(0) = 0 for
// a < 2; 2 Cauchy phi = (lambda s^2 / 2) log(1 + r^2 / s^2), w = lambda / (1 + r^2 / s^2); 3 Matern-3/2, w = lambda / (1 + sqrt(lambda) r).
// grid K, block 256.
enum : int { KERNEL_GAUSSIAN = 0, KERNEL_EXP_POWER = 1, KERNEL_CAUCHY = 2, KERNEL_MATERN32 = 3 };
__global__ void __launch_bounds__(256)
pull_weight_kernel(const float* __restrict__ partial, int64_t nchunks, int64_t nused, int kind, float lambda, float param,
                   float* __restrict__ weight, const int32_t* __restrict__ active) {
  grid_dep_sync();
  __shared__ double red[8];
  const int k = blockIdx.x;
  if (active != nullptr && !active[k]) return;
  double s = 0.0;
  for (int64_t c = threadIdx.x; c < nused; c += blockDim.x) s += (double)partial[(int64_t)k * nchunks + c];
  const double tot = block_sum<double>(s, red);
  if (threadIdx.x == 0) {
    const float r = (float)sqrt(tot);
    float w = lambda;
    if (kind == KERNEL_EXP_POWER) w = (param == 2.f) ? lambda : (r > 0.f ? lambda * powf(r, param - 2.f) : 0.f);
    else if (kind == KERNEL_CAUCHY) w = lambda / (1.f + (r / param) * (r / param));
    else if (kind == KERNEL_MATERN32) w = lambda / (1.f + sqrtf(lambda) * r);
    weight[k] = w;
  }
}

// Synchronous data parallelism (the DP-SGD / DP-SAM baselines aggregate the workers' gradients at every iteration):
// out[j] = (1/K) sum_k g[k][j], k ascending, one thread per 4 consecutive columns (or per column when VEC == 1).
// TG = float or bf16 (gradient storage of the tensor-core path).  out may alias row 0 of an fp32 g.
template <int VEC, typename TG>
__global__ void __launch_bounds__(256)
mean_rows_kernel(const TG* g, int64_t ldg, int K, int64_t n, float* out) {
  grid_dep_sync();
  const int64_t j = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * VEC;
  if (j >= n) return;
  const float inv = 1.0f / (float)K;
  if (VEC == 4) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int k = 0; k < K; ++k) {
      if (sizeof(TG) == 4) {
        const float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g) + (int64_t)k * ldg + j);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
      } else {
        const uint2 raw = *reinterpret_cast<const uint2*>(reinterpret_cast<const bf16*>(g) + (int64_t)k * ldg + j);
        const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
        const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
        s.x += lo.x; s.y += lo.y; s.z += hi.x; s.w += hi.y;
      }
    }
    *reinterpret_cast<float4*>(out + j) = make_float4(s.x * inv, s.y * inv, s.z * inv, s.w * inv);
  } else {
    float s = 0.f;
    for (int k = 0; k < K; ++k) s += to_float(g[(int64_t)k * ldg + j]);
    out[j] = s * inv;
  }
}

// ------------------------------------------------------------------------------------------------ three bf16 planes of fp32 rows
// planes[p][k][j], p = 0, 1, 2:  p0 = bf16(a), p1 = bf16(a - p0), p2 = bf16(a - p0 - p1)  for a = src[k][j]  (the operand form of
// the fp32 GEMMs on the bf16 tensor cores; p0 + p1 + p2 = a exactly unless a part underflows).  n a multiple of 4.
// grid (ceil(n / 1024), K), block 256.
// four consecutive values -> plane 0 at dst, and (plane != 0) planes 1 and 2 at dst + plane, dst + 2 plane
__device__ inline void store_planes4(bf16* dst, int64_t plane, float a, float b, float c, float d) {
  float r[4] = {a, b, c, d};
  const int np = plane != 0 ? 3 : 1;
  for (int p = 0; p < np; ++p) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(r[0], r[1]), hi = __floats2bfloat162_rn(r[2], r[3]);
    const float2 flo = __bfloat1622float2(lo), fhi = __bfloat1622float2(hi);
    r[0] -= flo.x; r[1] -= flo.y; r[2] -= fhi.x; r[3] -= fhi.y;
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&lo);
    pk.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst + p * plane) = pk;
  }
}
__device__ inline void store_planes1(bf16* dst, int64_t plane, float a) {
  const int np = plane != 0 ? 3 : 1;
  for (int p = 0; p < np; ++p) {
    const bf16 h = __float2bfloat16_rn(a);
    dst[p * plane] = h;
    a -= __bfloat162float(h);
  }
}

__global__ void __launch_bounds__(256)
split3_rows_kernel(const float* __restrict__ src, int64_t ld_src, int64_t n, bf16* __restrict__ planes, int64_t ld, int64_t plane) {
  grid_dep_sync();
  const int k = blockIdx.y;
  const int64_t j = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 4;
  if (j >= n) return;
  const float4 a = *reinterpret_cast<const float4*>(src + (int64_t)k * ld_src + j);
  store_planes4(planes + (int64_t)k * ld + j, plane, a.x, a.y, a.z, a.w);
}

// ------------------------------------------------------------------------------------------------ S4 perturb
// xt[k][j] = x[k][j] + scale[k] * g[k][j]  (Eq. 3 with scale = rho / (||g|| + gamma)); the master x is not modified.
// TP = float (fp32 operand) or bf16 (tensor-core operand copy).  grid (chunks, K).
constexpr int kPertThreads = 256;
constexpr int kPertIter = 4;

// TG = type of the stored gradient: float, or bf16 where the tensor-core path stores its gradients in bf16 (packed rows of stride ldg).
// plane != 0 (TP = bf16): the perturbed point is written as three bf16 planes, `plane` elements apart (fp32 GEMMs on the tensor
// cores); xt32 != nullptr: an fp32 copy of it is kept as well (rows of stride ldt).
template <int VEC, typename TP, typename TG>
__global__ void __launch_bounds__(kPertThreads)
perturb_kernel(const float* __restrict__ x, int64_t ldx, const TG* __restrict__ g, int64_t ldg, int64_t n,
               const float* __restrict__ scale, TP* __restrict__ xt, int64_t ldt, const int32_t* __restrict__ active,
               int64_t plane = 0, float* __restrict__ xt32 = nullptr) {
  grid_dep_sync();
  const int k = blockIdx.y;
  if (active != nullptr && !active[k]) return;
  const float sc = scale[k];
  const int64_t base = (int64_t)blockIdx.x * ((int64_t)kPertThreads * VEC * kPertIter);
  const float* xr = x + (int64_t)k * ldx;
  const TG* gr = g + (int64_t)k * ldg;
  TP* tr = xt + (int64_t)k * ldt;
  if (VEC == 4) {
    float4 xv[kPertIter], gv[kPertIter];
#pragma unroll
    for (int i = 0; i < kPertIter; ++i) {
      const int64_t j = base + ((int64_t)i * kPertThreads + threadIdx.x) * 4;
      if (j < n) {
        xv[i] = *reinterpret_cast<const float4*>(xr + j);
        if (sizeof(TG) == 4) {
          gv[i] = __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(gr) + j));
        } else {
          const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(reinterpret_cast<const bf16*>(gr) + j));
          const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
          const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
          gv[i] = make_float4(lo.x, lo.y, hi.x, hi.y);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < kPertIter; ++i) {
      const int64_t j = base + ((int64_t)i * kPertThreads + threadIdx.x) * 4;
      if (j < n) {
        const float a = fmaf(sc, gv[i].x, xv[i].x), b = fmaf(sc, gv[i].y, xv[i].y);
        const float c = fmaf(sc, gv[i].z, xv[i].z), d = fmaf(sc, gv[i].w, xv[i].w);
        if (sizeof(TP) == 4) {
          *reinterpret_cast<float4*>(reinterpret_cast<float*>(tr) + j) = make_float4(a, b, c, d);
        } else {
          store_planes4(reinterpret_cast<bf16*>(tr) + j, plane, a, b, c, d);
          if (xt32 != nullptr) *reinterpret_cast<float4*>(xt32 + (int64_t)k * ldt + j) = make_float4(a, b, c, d);
        }
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < kPertIter; ++i) {
      const int64_t j = base + (int64_t)i * kPertThreads + threadIdx.x;
      if (j < n) {
        const float a = fmaf(sc, to_float(gr[j]), xr[j]);
        if (sizeof(TP) == 4) {
          reinterpret_cast<float*>(tr)[j] = a;
        } else {
          store_planes1(reinterpret_cast<bf16*>(tr) + j, plane, a);
          if (xt32 != nullptr) xt32[(int64_t)k * ldt + j] = a;
        }
      }
    }
  }
}

// Tensor-core path: gradient and operand are both bf16, so a thread takes 8 elements per access (two 128-bit loads of x,
// one of g, one 128-bit store).  Requires 16-byte aligned rows (ld multiples of 8).  grid (chunks, K).
constexpr int kPert8Iter = 2;
__global__ void __launch_bounds__(kPertThreads)
perturb8_kernel(const float* __restrict__ x, int64_t ldx, const bf16* __restrict__ g, int64_t ldg, int64_t n,
                const float* __restrict__ scale, bf16* __restrict__ xt, int64_t ldt, const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int k = blockIdx.y;
  if (active != nullptr && !active[k]) return;
  const float sc = scale[k];
  const int64_t base = (int64_t)blockIdx.x * ((int64_t)kPertThreads * 8 * kPert8Iter);
  const float* xr = x + (int64_t)k * ldx;
  const bf16* gr = g + (int64_t)k * ldg;
  bf16* tr = xt + (int64_t)k * ldt;
  float4 xa[kPert8Iter], xb[kPert8Iter];
  uint4 gv[kPert8Iter];
#pragma unroll
  for (int i = 0; i < kPert8Iter; ++i) {
    const int64_t j = base + ((int64_t)i * kPertThreads + threadIdx.x) * 8;
    if (j < n) {
      xa[i] = *reinterpret_cast<const float4*>(xr + j);
      xb[i] = *reinterpret_cast<const float4*>(xr + j + 4);
      gv[i] = __ldcs(reinterpret_cast<const uint4*>(gr + j));
    }
  }
#pragma unroll
  for (int i = 0; i < kPert8Iter; ++i) {
    const int64_t j = base + ((int64_t)i * kPertThreads + threadIdx.x) * 8;
    if (j < n) {
      const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gv[i].x));
      const float2 g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gv[i].y));
      const float2 g2 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gv[i].z));
      const float2 g3 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gv[i].w));
      __nv_bfloat162 o0 = __floats2bfloat162_rn(fmaf(sc, g0.x, xa[i].x), fmaf(sc, g0.y, xa[i].y));
      __nv_bfloat162 o1 = __floats2bfloat162_rn(fmaf(sc, g1.x, xa[i].z), fmaf(sc, g1.y, xa[i].w));
      __nv_bfloat162 o2 = __floats2bfloat162_rn(fmaf(sc, g2.x, xb[i].x), fmaf(sc, g2.y, xb[i].y));
      __nv_bfloat162 o3 = __floats2bfloat162_rn(fmaf(sc, g3.x, xb[i].z), fmaf(sc, g3.y, xb[i].w));
      uint4 pk;
      pk.x = *reinterpret_cast<uint32_t*>(&o0); pk.y = *reinterpret_cast<uint32_t*>(&o1);
      pk.z = *reinterpret_cast<uint32_t*>(&o2); pk.w = *reinterpret_cast<uint32_t*>(&o3);
      *reinterpret_cast<uint4*>(tr + j) = pk;
    }
  }
}

// ------------------------------------------------------------------------------------------------ S6 fused update
// One thread owns VEC consecutive columns for ALL replicas (k ascending), so that the centre versions are
// re-read from cache and the iterate accumulator is read and written once per column:
//   G = g2 + lambda (x - y_slot[k]);  v <- mu v + G;  x <- x - eta (G + mu v)  [Nesterov]  or  x - eta v;
//   acc += sum_k x_new;  optional operand copy xop = TP(x_new).
// NOISE: the Langevin term sqrt(2 eta T) N(0, I) is added to x_new before it is stored and accumulated; the normals are
// keyed by (tick, replica, segment, offset within the segment), so padding elements get none and stay zero.
// Parameter segments of a replica's row: seg i = {offset in the unpadded vector, offset in the padded row, length}.
struct SegMap { int n; int64_t src[18], dst[18], len[18]; };

struct UpdateArgs {
  float* x;            // [K, ld]
  float* v;            // [K, ld]
  const void* g;       // [K, ldg] descent gradient: fp32, or bf16 when g_mode == 2
  int g_mode;          // 0: fp32; 2: stored as bf16 (gradient storage format of the tensor-core path)
  const float* yring;  // [ring, ld]
  const int32_t* slot; // [K] ring slot of the centre version read by replica k
  const int32_t* active;  // nullable [K]: replicas with 0 wait this tick and are left untouched
  float* acc;          // [ld]
  void* xop;           // [K, ld] operand copy (or nullptr)
  int64_t xop_plane;   // != 0 (bf16 operand copy): three bf16 planes of x, this many elements apart (fp32 GEMMs on the tensor cores)
  int64_t ld, ldg, n;
  int K;
  int k_offset;        // global index of worker 0: the noise streams are keyed by the global worker index
  float eta, mu, lambda;
  const float* lam_k;  // nullable [K]: per-worker pull weight w(||x_k - y||) of a non-Gaussian stationary kernel, used instead of lambda
  // Langevin noise (NOISE variants): x_new += sigma * xi, xi from langevin_noise4(seed, tick, k, segment, offset / 4)
  float sigma;
  uint64_t seed, tick;
  SegMap seg;
};

constexpr int kUpdThreads = 256;

__device__ inline float4 update_load_g4(const void* g, int64_t idx, int mode) {
  if (mode == 2) {
    const uint2 raw = __ldcs(reinterpret_cast<const uint2*>(reinterpret_cast<const bf16*>(g) + idx));
    const float2 lo = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.x));
    const float2 hi = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&raw.y));
    return make_float4(lo.x, lo.y, hi.x, hi.y);
  }
  return __ldcs(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(g) + idx));
}
__device__ inline float update_load_g1(const void* g, int64_t idx, int mode) {
  if (mode == 2) return to_float(reinterpret_cast<const bf16*>(g)[idx]);
  return reinterpret_cast<const float*>(g)[idx];
}

template <int VEC, bool NESTEROV, typename TP, bool WRITE_OP, bool NOISE>
__global__ void __launch_bounds__(kUpdThreads) update_kernel(const UpdateArgs a) {
  grid_dep_sync();
  const int64_t j = ((int64_t)blockIdx.x * kUpdThreads + threadIdx.x) * VEC;
  if (j >= a.n) return;
  // segment of this thread's elements (segments ascend; all VEC elements lie in one segment: starts are multiples of 64)
  uint32_t nseg = 0;
  int64_t noff = 0, nlen = 0;
  if (NOISE) {
    for (int s = 1; s < a.seg.n; ++s)
      if (j >= a.seg.dst[s]) nseg = (uint32_t)s;
    noff = j - a.seg.dst[nseg];
    nlen = a.seg.len[nseg];
  }
  if (VEC == 4) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    // software pipeline over the replicas: the four loads of replica k + 1 are issued before the arithmetic and the
    // stores of replica k, so that twice as many bytes are in flight per thread
    int k = 0;
    if (a.active != nullptr)
      while (k < a.K && !a.active[k]) ++k;  // first replica that steps at this tick
    float4 gv = make_float4(0.f, 0.f, 0.f, 0.f), xv = gv, vv = gv, yv = gv;
    if (k < a.K) {
      gv = update_load_g4(a.g, (int64_t)k * a.ldg + j, a.g_mode);
      xv = *reinterpret_cast<const float4*>(a.x + (int64_t)k * a.ld + j);
      vv = *reinterpret_cast<const float4*>(a.v + (int64_t)k * a.ld + j);
      yv = __ldg(reinterpret_cast<const float4*>(a.yring + (int64_t)a.slot[k] * a.ld + j));
    }
    while (k < a.K) {
      const int64_t o = (int64_t)k * a.ld + j;
      int kn = k + 1;
      if (a.active != nullptr)
        while (kn < a.K && !a.active[kn]) ++kn;
      float4 gn = gv, xn = xv, vn = vv, yn = yv;
      if (kn < a.K) {
        const int64_t on = (int64_t)kn * a.ld + j;
        gn = update_load_g4(a.g, (int64_t)kn * a.ldg + j, a.g_mode);
        xn = *reinterpret_cast<const float4*>(a.x + on);
        vn = *reinterpret_cast<const float4*>(a.v + on);
        yn = __ldg(reinterpret_cast<const float4*>(a.yring + (int64_t)a.slot[kn] * a.ld + j));
      }
      float G;
      const float lam = a.lam_k != nullptr ? a.lam_k[k] : a.lambda;
#define LSAM_UPD(c)                                                         \
  G = fmaf(lam, xv.c - yv.c, gv.c);                                         \
  vv.c = fmaf(a.mu, vv.c, G);                                               \
  xv.c = NESTEROV ? xv.c - a.eta * fmaf(a.mu, vv.c, G) : xv.c - a.eta * vv.c;
      LSAM_UPD(x) LSAM_UPD(y) LSAM_UPD(z) LSAM_UPD(w)
#undef LSAM_UPD
      if (NOISE && noff < nlen) {
        float z[4];
        langevin_noise4(a.seed, a.tick, (uint32_t)(k + a.k_offset), nseg, (uint64_t)(noff >> 2), z);
        xv.x = fmaf(a.sigma, z[0], xv.x);
        if (noff + 1 < nlen) xv.y = fmaf(a.sigma, z[1], xv.y);
        if (noff + 2 < nlen) xv.z = fmaf(a.sigma, z[2], xv.z);
        if (noff + 3 < nlen) xv.w = fmaf(a.sigma, z[3], xv.w);
      }
      s.x += xv.x; s.y += xv.y; s.z += xv.z; s.w += xv.w;
      *reinterpret_cast<float4*>(a.x + o) = xv;
      __stcs(reinterpret_cast<float4*>(a.v + o), vv);
      if (WRITE_OP) {
        if (sizeof(TP) == 2) store_planes4(reinterpret_cast<bf16*>(a.xop) + o, a.xop_plane, xv.x, xv.y, xv.z, xv.w);
      }
      gv = gn; xv = xn; vv = vn; yv = yn;
      k = kn;
    }
    float4 av = *reinterpret_cast<const float4*>(a.acc + j);
    av.x += s.x; av.y += s.y; av.z += s.z; av.w += s.w;
    *reinterpret_cast<float4*>(a.acc + j) = av;
  } else {
    float s = 0.f;
    for (int k = 0; k < a.K; ++k) {
      if (a.active != nullptr && !a.active[k]) continue;
      const int64_t o = (int64_t)k * a.ld + j;
      const float gv = update_load_g1(a.g, (int64_t)k * a.ldg + j, a.g_mode);
      float xv = a.x[o], vv = a.v[o];
      const float yv = a.yring[(int64_t)a.slot[k] * a.ld + j];
      const float G = fmaf(a.lam_k != nullptr ? a.lam_k[k] : a.lambda, xv - yv, gv);
      vv = fmaf(a.mu, vv, G);
      xv = NESTEROV ? xv - a.eta * fmaf(a.mu, vv, G) : xv - a.eta * vv;
      if (NOISE && noff < nlen) {
        float z[4];
        langevin_noise4(a.seed, a.tick, (uint32_t)(k + a.k_offset), nseg, (uint64_t)(noff >> 2), z);
        xv = fmaf(a.sigma, z[noff & 3], xv);
      }
      s += xv;
      a.x[o] = xv;
      a.v[o] = vv;
      if (WRITE_OP) {
        if (sizeof(TP) == 2) store_planes1(reinterpret_cast<bf16*>(a.xop) + o, a.xop_plane, xv);
        else reinterpret_cast<TP*>(a.xop)[o] = from_float<TP>(xv);
      }
    }
    a.acc[j] += s;
  }
}

// Tensor-core path of the fused update: gradient and operand copy are bf16, so a thread takes 8 consecutive elements
// (one 128-bit load of g, two of x, v and the centre; one 128-bit store of the operand copy, two of x and v).
// Same arithmetic, order and noise keys as update_kernel<4, ...>.  Needs n % 8 == 0 and g_mode == 2.
template <bool NESTEROV, bool NOISE>
__global__ void __launch_bounds__(kUpdThreads, NOISE ? 1 : 3) update8_kernel(const UpdateArgs a) {
  grid_dep_sync();
  const int64_t j = ((int64_t)blockIdx.x * kUpdThreads + threadIdx.x) * 8;
  if (j >= a.n) return;
  uint32_t nseg = 0;
  int64_t noff = 0, nlen = 0;
  if (NOISE) {
    for (int s = 1; s < a.seg.n; ++s)
      if (j >= a.seg.dst[s]) nseg = (uint32_t)s;
    noff = j - a.seg.dst[nseg];
    nlen = a.seg.len[nseg];
  }
  const bf16* gb = reinterpret_cast<const bf16*>(a.g);
  float4 s[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
  int k = 0;
  if (a.active != nullptr)
    while (k < a.K && !a.active[k]) ++k;
  uint4 gr = make_uint4(0u, 0u, 0u, 0u);
  float4 xv[2], vv[2], yv[2];
  xv[0] = xv[1] = vv[0] = vv[1] = yv[0] = yv[1] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (k < a.K) {
    const int64_t o = (int64_t)k * a.ld + j;
    gr = __ldcs(reinterpret_cast<const uint4*>(gb + (int64_t)k * a.ldg + j));
    const float* yp = a.yring + (int64_t)a.slot[k] * a.ld + j;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      xv[h] = *reinterpret_cast<const float4*>(a.x + o + 4 * h);
      vv[h] = *reinterpret_cast<const float4*>(a.v + o + 4 * h);
      yv[h] = __ldg(reinterpret_cast<const float4*>(yp + 4 * h));
    }
  }
  while (k < a.K) {
    const int64_t o = (int64_t)k * a.ld + j;
    int kn = k + 1;
    if (a.active != nullptr)
      while (kn < a.K && !a.active[kn]) ++kn;
    uint4 gn = gr;
    float4 xn[2] = {xv[0], xv[1]}, vn[2] = {vv[0], vv[1]}, yn[2] = {yv[0], yv[1]};
    if (kn < a.K) {
      const int64_t on = (int64_t)kn * a.ld + j;
      gn = __ldcs(reinterpret_cast<const uint4*>(gb + (int64_t)kn * a.ldg + j));
      const float* yp = a.yring + (int64_t)a.slot[kn] * a.ld + j;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        xn[h] = *reinterpret_cast<const float4*>(a.x + on + 4 * h);
        vn[h] = *reinterpret_cast<const float4*>(a.v + on + 4 * h);
        yn[h] = __ldg(reinterpret_cast<const float4*>(yp + 4 * h));
      }
    }
    const uint32_t gw[4] = {gr.x, gr.y, gr.z, gr.w};
    uint32_t ow[4];
    const float lam = a.lam_k != nullptr ? a.lam_k[k] : a.lambda;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float2 ga = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw[2 * h]));
      const float2 gc = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&gw[2 * h + 1]));
      const float4 gv = make_float4(ga.x, ga.y, gc.x, gc.y);
      float G;
#define LSAM_UPD(c)                                                               \
  G = fmaf(lam, xv[h].c - yv[h].c, gv.c);                                         \
  vv[h].c = fmaf(a.mu, vv[h].c, G);                                               \
  xv[h].c = NESTEROV ? xv[h].c - a.eta * fmaf(a.mu, vv[h].c, G) : xv[h].c - a.eta * vv[h].c;
      LSAM_UPD(x) LSAM_UPD(y) LSAM_UPD(z) LSAM_UPD(w)
#undef LSAM_UPD
      const int64_t no = noff + 4 * h;
      if (NOISE && no < nlen) {
        float z[4];
        langevin_noise4(a.seed, a.tick, (uint32_t)(k + a.k_offset), nseg, (uint64_t)(no >> 2), z);
        xv[h].x = fmaf(a.sigma, z[0], xv[h].x);
        if (no + 1 < nlen) xv[h].y = fmaf(a.sigma, z[1], xv[h].y);
        if (no + 2 < nlen) xv[h].z = fmaf(a.sigma, z[2], xv[h].z);
        if (no + 3 < nlen) xv[h].w = fmaf(a.sigma, z[3], xv[h].w);
      }
      s[h].x += xv[h].x; s[h].y += xv[h].y; s[h].z += xv[h].z; s[h].w += xv[h].w;
      *reinterpret_cast<float4*>(a.x + o + 4 * h) = xv[h];
      __stcs(reinterpret_cast<float4*>(a.v + o + 4 * h), vv[h]);
      __nv_bfloat162 lo = __floats2bfloat162_rn(xv[h].x, xv[h].y), hi = __floats2bfloat162_rn(xv[h].z, xv[h].w);
      ow[2 * h] = *reinterpret_cast<uint32_t*>(&lo);
      ow[2 * h + 1] = *reinterpret_cast<uint32_t*>(&hi);
    }
    *reinterpret_cast<uint4*>(reinterpret_cast<bf16*>(a.xop) + o) = make_uint4(ow[0], ow[1], ow[2], ow[3]);
    gr = gn;
#pragma unroll
    for (int h = 0; h < 2; ++h) { xv[h] = xn[h]; vv[h] = vn[h]; yv[h] = yn[h]; }
    k = kn;
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float4 av = *reinterpret_cast<const float4*>(a.acc + j + 4 * h);
    av.x += s[h].x; av.y += s[h].y; av.z += s[h].z; av.w += s[h].w;
    *reinterpret_cast<float4*>(a.acc + j + 4 * h) = av;
  }
}

// fp32 counterpart of update8_kernel (gradient fp32 used as is, no operand copy): 8 consecutive elements per thread, i.e.
// two 128-bit accesses to each of g, x, v and the centre per replica, software-pipelined over the replicas.  Same arithmetic,
// order and noise keys as update_kernel<4, ...>.  Needs n % 8 == 0, 16-byte aligned rows and g_mode == 0.
// Compiled for three blocks per SM (80 registers): at 90 registers only two fit and the kernel streamed 5 % slower.
template <bool NESTEROV, bool NOISE>
__global__ void __launch_bounds__(kUpdThreads, NOISE ? 1 : 3) update8f_kernel(const UpdateArgs a) {
  grid_dep_sync();
  const int64_t j = ((int64_t)blockIdx.x * kUpdThreads + threadIdx.x) * 8;
  if (j >= a.n) return;
  uint32_t nseg = 0;
  int64_t noff = 0, nlen = 0;
  if (NOISE) {
    for (int s = 1; s < a.seg.n; ++s)
      if (j >= a.seg.dst[s]) nseg = (uint32_t)s;
    noff = j - a.seg.dst[nseg];
    nlen = a.seg.len[nseg];
  }
  const float* gf = reinterpret_cast<const float*>(a.g);
  float4 s[2] = {make_float4(0.f, 0.f, 0.f, 0.f), make_float4(0.f, 0.f, 0.f, 0.f)};
  int k = 0;
  if (a.active != nullptr)
    while (k < a.K && !a.active[k]) ++k;
  float4 gv[2], xv[2], vv[2], yv[2];
  gv[0] = gv[1] = xv[0] = xv[1] = vv[0] = vv[1] = yv[0] = yv[1] = make_float4(0.f, 0.f, 0.f, 0.f);
  if (k < a.K) {
    const int64_t o = (int64_t)k * a.ld + j;
    const float* yp = a.yring + (int64_t)a.slot[k] * a.ld + j;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      gv[h] = __ldcs(reinterpret_cast<const float4*>(gf + (int64_t)k * a.ldg + j + 4 * h));
      xv[h] = *reinterpret_cast<const float4*>(a.x + o + 4 * h);
      vv[h] = *reinterpret_cast<const float4*>(a.v + o + 4 * h);
      yv[h] = __ldg(reinterpret_cast<const float4*>(yp + 4 * h));
    }
  }
  while (k < a.K) {
    const int64_t o = (int64_t)k * a.ld + j;
    int kn = k + 1;
    if (a.active != nullptr)
      while (kn < a.K && !a.active[kn]) ++kn;
    float4 gn[2] = {gv[0], gv[1]}, xn[2] = {xv[0], xv[1]}, vn[2] = {vv[0], vv[1]}, yn[2] = {yv[0], yv[1]};
    if (kn < a.K) {
      const int64_t on = (int64_t)kn * a.ld + j;
      const float* yp = a.yring + (int64_t)a.slot[kn] * a.ld + j;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        gn[h] = __ldcs(reinterpret_cast<const float4*>(gf + (int64_t)kn * a.ldg + j + 4 * h));
        xn[h] = *reinterpret_cast<const float4*>(a.x + on + 4 * h);
        vn[h] = *reinterpret_cast<const float4*>(a.v + on + 4 * h);
        yn[h] = __ldg(reinterpret_cast<const float4*>(yp + 4 * h));
      }
    }
    const float lam = a.lam_k != nullptr ? a.lam_k[k] : a.lambda;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float G;
#define LSAM_UPD(c)                                                               \
  G = fmaf(lam, xv[h].c - yv[h].c, gv[h].c);                                      \
  vv[h].c = fmaf(a.mu, vv[h].c, G);                                               \
  xv[h].c = NESTEROV ? xv[h].c - a.eta * fmaf(a.mu, vv[h].c, G) : xv[h].c - a.eta * vv[h].c;
      LSAM_UPD(x) LSAM_UPD(y) LSAM_UPD(z) LSAM_UPD(w)
#undef LSAM_UPD
      const int64_t no = noff + 4 * h;
      if (NOISE && no < nlen) {
        float z[4];
        langevin_noise4(a.seed, a.tick, (uint32_t)(k + a.k_offset), nseg, (uint64_t)(no >> 2), z);
        xv[h].x = fmaf(a.sigma, z[0], xv[h].x);
        if (no + 1 < nlen) xv[h].y = fmaf(a.sigma, z[1], xv[h].y);
        if (no + 2 < nlen) xv[h].z = fmaf(a.sigma, z[2], xv[h].z);
        if (no + 3 < nlen) xv[h].w = fmaf(a.sigma, z[3], xv[h].w);
      }
      s[h].x += xv[h].x; s[h].y += xv[h].y; s[h].z += xv[h].z; s[h].w += xv[h].w;
      *reinterpret_cast<float4*>(a.x + o + 4 * h) = xv[h];
      __stcs(reinterpret_cast<float4*>(a.v + o + 4 * h), vv[h]);
    }
#pragma unroll
    for (int h = 0; h < 2; ++h) { gv[h] = gn[h]; xv[h] = xn[h]; vv[h] = vn[h]; yv[h] = yn[h]; }
    k = kn;
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    float4 av = *reinterpret_cast<const float4*>(a.acc + j + 4 * h);
    av.x += s[h].x; av.y += s[h].y; av.z += s[h].z; av.w += s[h].w;
    *reinterpret_cast<float4*>(a.acc + j + 4 * h) = av;
  }
}

// Iterate accumulation on its own (for the parameters whose update ran in a weight-gradient epilogue): acc[j] += sum over the
// replicas that stepped, k ascending, of x[k][j], j in [off, off + n); one thread per 4 consecutive columns.
__global__ void __launch_bounds__(256)
acc_add_kernel(const float* __restrict__ x, int64_t ld, int K, int64_t off, int64_t n, float* __restrict__ acc,
               const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int64_t j = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
  if (j >= n) return;
  float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int k = 0; k < K; ++k) {
    if (active != nullptr && !active[k]) continue;
    const float4 v = *reinterpret_cast<const float4*>(x + (int64_t)k * ld + off + j);
    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
  }
  float4 a = *reinterpret_cast<const float4*>(acc + off + j);
  a.x += s.x; a.y += s.y; a.z += s.z; a.w += s.w;
  *reinterpret_cast<float4*>(acc + off + j) = a;
}

// ------------------------------------------------------------------------------------------------ S7 centre update
//   g' = acc / (K tau) - y;  g = have_prev ? g' + beta (g' - g'_prev) : g';  y_new = y + eta' g;
//   g'_prev <- g';  acc <- 0.       (sync branch of Algorithm 2 with the look-ahead of Section 4.2)
__global__ void __launch_bounds__(256)
couple_kernel(float* __restrict__ acc, const float* __restrict__ y_cur, float* __restrict__ y_new,
              float* __restrict__ gprev, int64_t n, float inv_ktau, float beta, float eta_prime, int have_prev) {
  grid_dep_sync();
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  const float y = y_cur[j];
  const float gp = fmaf(acc[j], inv_ktau, -y);
  const float g = have_prev ? fmaf(beta, gp - gprev[j], gp) : gp;
  y_new[j] = fmaf(eta_prime, g, y);
  gprev[j] = gp;
  acc[j] = 0.f;
}

// ------------------------------------------------------------------------------------------------ small utilities
// dst[k][j] = TP(src[k][j]) over [K, n] with row strides.
template <typename TP>
__global__ void __launch_bounds__(256)
cast_rows_kernel(const float* __restrict__ src, int64_t lds, TP* __restrict__ dst, int64_t ldd, int64_t n) {
  grid_dep_sync();
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n) return;
  const int k = blockIdx.y;
  dst[(int64_t)k * ldd + j] = from_float<TP>(src[(int64_t)k * lds + j]);
}


template <bool TO_PADDED, typename TS, typename TD>
__global__ void __launch_bounds__(256)
seg_copy_kernel(const TS* __restrict__ src, int64_t lds, TD* __restrict__ dst, int64_t ldd, SegMap m) {
  grid_dep_sync();
  const int k = blockIdx.z, sgi = blockIdx.y;
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (sgi >= m.n || j >= m.len[sgi]) return;
  const int64_t so = TO_PADDED ? m.src[sgi] : m.dst[sgi];
  const int64_t dof = TO_PADDED ? m.dst[sgi] : m.src[sgi];
  dst[(int64_t)k * ldd + dof + j] = from_float<TD>(to_float(src[(int64_t)k * lds + so + j]));
}

}  // namespace lsam
