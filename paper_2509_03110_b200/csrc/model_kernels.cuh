// model_kernels.cuh -- minibatch gather, GEMM epilogues, softmax cross-entropy, bias gradient, least squares,
// and the SIMT batched GEMM used for fp32 models and for shapes the tensor-core path does not cover.
#pragma once

#include "common.cuh"

namespace lsam {

// ------------------------------------------------------------------------------------------------ S1 gather
// xb[k][b][:] = TA(X[idx[k][b]][:]) with row stride ld;  yb[k][b] = Y[idx[k][b]] (4-byte elements).  grid (K*B), block 128.
template <typename TA>
__global__ void __launch_bounds__(128)
gather_kernel(const float* __restrict__ X, const uint32_t* __restrict__ Y, const int32_t* __restrict__ idx,
              int64_t n_samples, int in, int ld, TA* __restrict__ xb, uint32_t* __restrict__ yb, int* __restrict__ status,
              int B, const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int64_t r = blockIdx.x;
  if (active != nullptr && !active[r / B]) return;
  int64_t s = idx[r];
  if (s < 0 || s >= n_samples) {
    if (threadIdx.x == 0) atomicOr(status, STATUS_BAD_INDEX);
    s = 0;
  }
  const float* src = X + s * in;
  TA* dst = xb + r * ld;
  for (int i = threadIdx.x; i < in; i += blockDim.x) dst[i] = from_float<TA>(src[i]);
  if (threadIdx.x == 0 && yb != nullptr) yb[r] = Y[s];
}

// Classifier inputs are stored FEATURE-MAJOR: xt[k][i][b] = TA(X[idx[k][b]][i]) with row stride ldb, so that the
// sample index is the contiguous one (see the layout note above the epilogues).  32 x 32 tiles go through shared
// memory: reads run along the features of a sample, writes along the samples of a feature.
// grid (ceil(in / 32), ceil(B / 32), K), block (32, 8).  idx == nullptr: rows come from the dense minibatch src [K, B, in].
// plane != 0 (TA = bf16): the value is stored as three bf16 planes p0 = bf16(v), p1 = bf16(v - p0), p2 = bf16(v - p0 - p1),
// `plane` elements apart (fp32 GEMMs on the bf16 tensor cores read their operands in this form).
template <typename TA>
__device__ inline void store_planes(TA* p, int64_t plane, float v) {
  const TA h = from_float<TA>(v);
  p[0] = h;
  if (sizeof(TA) == 2 && plane != 0) {
    float r = v - to_float(h);
    const TA m = from_float<TA>(r);
    p[plane] = m;
    r -= to_float(m);
    p[2 * plane] = from_float<TA>(r);
  }
}
template <typename TA>
__device__ inline float load_planes(const TA* p, int64_t plane) {
  float v = to_float(p[0]);
  if (sizeof(TA) == 2 && plane != 0) v = (v + to_float(p[plane])) + to_float(p[2 * plane]);  // exact for the planes of an fp32 value
  return v;
}

template <typename TA>
__global__ void __launch_bounds__(256)
gather_t_kernel(const float* __restrict__ X, const uint32_t* __restrict__ Y, const int32_t* __restrict__ idx, int64_t n_samples,
                int B, int in, int ldb, TA* __restrict__ xt, uint32_t* __restrict__ yb, int* __restrict__ status,
                const int32_t* __restrict__ active, int64_t plane = 0) {
  grid_dep_sync();
  __shared__ float tile[32][33];
  if (active != nullptr && !active[blockIdx.z]) return;
  const int k = blockIdx.z, i0 = blockIdx.x * 32, b0 = blockIdx.y * 32;
  for (int r = threadIdx.y; r < 32; r += 8) {
    const int b = b0 + r, i = i0 + threadIdx.x;
    float v = 0.f;
    if (b < B) {
      int64_t s = idx ? (int64_t)idx[(int64_t)k * B + b] : (int64_t)k * B + b;
      if (idx && (s < 0 || s >= n_samples)) {
        if (threadIdx.x == 0) atomicOr(status, STATUS_BAD_INDEX);
        s = 0;
      }
      if (i < in) v = X[s * in + i];
      if (idx && blockIdx.x == 0 && threadIdx.x == 0 && yb != nullptr) yb[(int64_t)k * B + b] = Y[s];
    }
    tile[r][threadIdx.x] = v;
  }
  __syncthreads();
  for (int r = threadIdx.y; r < 32; r += 8) {
    const int i = i0 + r, b = b0 + threadIdx.x;
    if (i < in && b < B) store_planes(xt + ((int64_t)k * in + i) * ldb + b, plane, tile[threadIdx.x][r]);
  }
}

// ------------------------------------------------------------------------------------------------ epilogues
// Every GEMM hands its accumulator to one of these functors in LOGICAL coordinates:
//   z = replica, b = sample in the minibatch, f = feature (output unit for forward, input unit for dgrad),
//   or (z, o, i) = (replica, output unit, input unit) for the weight gradient.
// Activation-like buffers (activations, ReLU masks, logits, backward signals) are FEATURE-MAJOR: [K, width, ldb]
// with the sample index contiguous (ldb >= B, a multiple of 16).  In the tensor-core epilogue a thread owns one
// feature and 32 consecutive samples, so this layout makes its accesses contiguous 16-byte vectors.
// TP = parameter operand type, TA = activation storage type.

// hidden layer: v = acc + bias[f]; r = relu(v); mask = v > 0; out = TA(skip + r)
template <typename TP, typename TA>
struct EpiFwdHidden {
  static constexpr bool kRowsContiguous = true;  // what it writes is contiguous along the GEMM's M index (the sample)
  const TP* bias;  int64_t ld_p;           // bias[z * ld_p + f]
  TA* out;  const TA* skip;  uint8_t* mask;  // [K, width, ldb]
  int width, ldb;
  __device__ inline void operator()(int z, int b, int f, float acc) const {
    const float v = acc + to_float(bias[(int64_t)z * ld_p + f]);
    const int64_t e = ((int64_t)z * width + f) * ldb + b;
    const float r = v > 0.f ? v : 0.f;
    mask[e] = v > 0.f;
    const float sk = skip ? to_float(skip[e]) : 0.f;
    out[e] = from_float<TA>(sk + r);
  }
};

// head: logits = acc + bias[f]  (fp32, not rounded)
template <typename TP>
struct EpiFwdHead {
  static constexpr bool kRowsContiguous = true;
  const TP* bias;  int64_t ld_p;
  float* logits;  // [K, width, ldb]
  int width, ldb;
  __device__ inline void operator()(int z, int b, int f, float acc) const {
    logits[((int64_t)z * width + f) * ldb + b] = acc + to_float(bias[(int64_t)z * ld_p + f]);
  }
};

// Forward of a narrow head (out <= kHeadMaxOut classes): logits[z][f][b] = bias[f] + sum_i W[z][f][i] a[z][i][b].
// A GEMM tile would be almost empty here and leave a handful of blocks to walk the whole contraction.  Instead the
// contraction is cut into chunks of kHeadChunkIn inputs, one block per (chunk, 128 samples, replica): the chunk's weights
// are staged in shared memory, a thread owns one sample, reads a[i][b] coalesced (all loads of the chunk in flight at once) and the weights as
// shared-memory broadcasts, and leaves its `out` partial sums in part[z][chunk][f][b]; softmax_ce_kernel adds the chunks
// in ascending order on top of the bias, so the result is deterministic.  a_plane / p_plane != 0: activations / parameters
// are stored as three bf16 planes (their sum is the fp32 value).  grid (chunks, ceil(B / 128), K), block 128.
constexpr int kHeadMaxOut = 16;
constexpr int kHeadChunkIn = 32;
template <typename T>
__global__ void __launch_bounds__(128)
head_chunk_kernel(const T* __restrict__ a, int64_t a_sz, int ldb, int64_t a_plane, const T* __restrict__ P, int64_t ld_p, int64_t w_off,
                  int64_t p_plane, int in, int out, int B, float* __restrict__ part, const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int z = blockIdx.z;
  if (active != nullptr && !active[z]) return;
  __shared__ __align__(16) float w[kHeadChunkIn][kHeadMaxOut];  // [input][class]: a thread reads the 16 weights of an input as four 128-bit broadcasts
  const int i0 = blockIdx.x * kHeadChunkIn;
  const int len = min(kHeadChunkIn, in - i0);
  const int b = blockIdx.y * 128 + threadIdx.x;
  const bool live = b < B;
  // every load of the chunk is issued before the first use: one round trip to memory per thread
  const T* az = a + (int64_t)z * a_sz + (int64_t)i0 * ldb + (live ? b : 0);
  float av[kHeadChunkIn];
#pragma unroll
  for (int u = 0; u < kHeadChunkIn; ++u) av[u] = (live && u < len) ? load_planes(az + (int64_t)u * ldb, a_plane) : 0.f;
  const T* W = P + (int64_t)z * ld_p + w_off;
  for (int e = threadIdx.x; e < kHeadMaxOut * kHeadChunkIn; e += 128) {
    const int f = e / kHeadChunkIn, ii = e % kHeadChunkIn;
    w[ii][f] = (f < out && ii < len) ? load_planes(W + (int64_t)f * in + i0 + ii, p_plane) : 0.f;
  }
  __syncthreads();
  if (!live) return;
  float acc[kHeadMaxOut];
#pragma unroll
  for (int f = 0; f < kHeadMaxOut; ++f) acc[f] = 0.f;
#pragma unroll
  for (int u = 0; u < kHeadChunkIn; ++u) {  // inputs past the end of the chunk have zero weights and zero activations
#pragma unroll
    for (int q = 0; q < kHeadMaxOut / 4; ++q) {
      const float4 wv = *reinterpret_cast<const float4*>(&w[u][4 * q]);
      acc[4 * q] = fmaf(wv.x, av[u], acc[4 * q]);
      acc[4 * q + 1] = fmaf(wv.y, av[u], acc[4 * q + 1]);
      acc[4 * q + 2] = fmaf(wv.z, av[u], acc[4 * q + 2]);
      acc[4 * q + 3] = fmaf(wv.w, av[u], acc[4 * q + 3]);
    }
  }
  float* dst = part + (((int64_t)z * gridDim.x + blockIdx.x) * kHeadMaxOut) * ldb + b;
#pragma unroll
  for (int f = 0; f < kHeadMaxOut; ++f)
    if (f < out) dst[(int64_t)f * ldb] = acc[f];
}

// Backward through a narrow head (out <= kHeadMaxOut classes) into the layer below, with that layer's bias gradient:
//   dh[i][b] = sum_c W[c][i] dz[c][b] (classes ascending);  dz_prev[i][b] = mask[i][b] ? T(dh) : 0;  dh_out = T(dh) (skip connections, nullable);
//   db[i] = sum_b dz_prev[i][b] as stored -> g[z][b_off + i];  sum of squares of the block's 8 db -> partial[z][slot0 + blockIdx.x] (nullable).
// A GEMM would contract over at most 16 classes.  Warp w owns input unit i = 8 blockIdx.x + w, its lanes stride the samples (coalesced).
// dz_plane / p_plane / out_plane != 0: backward signals / parameters / outputs are three bf16 planes.  grid (ceil(in / 8), K), block 256.
template <typename T>
__global__ void __launch_bounds__(256)
head_dgrad_kernel(const T* __restrict__ dz, int64_t dz_plane, const T* __restrict__ P, int64_t ld_p, int64_t w_off, int64_t p_plane, int in, int out,
                  int B, int ldb, const uint8_t* __restrict__ mask_prev, T* __restrict__ dz_prev, T* __restrict__ dh_out, int64_t out_plane,
                  float* __restrict__ g, int64_t ld_g, int64_t b_off, float* __restrict__ partial, int64_t ld_partial, int slot0,
                  const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int z = blockIdx.y;
  if (active != nullptr && !active[z]) return;
  __shared__ float wv[8][kHeadMaxOut];
  __shared__ float sq[8];
  __shared__ float dzs[kHeadMaxOut][256];  // the backward signal of 256 samples, planes already summed: read once per block, used by its 8 warps
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int i0 = blockIdx.x * 8, i = i0 + w;
  if (threadIdx.x < 8 * kHeadMaxOut) {
    const int u = threadIdx.x / kHeadMaxOut, c = threadIdx.x % kHeadMaxOut;
    wv[u][c] = (c < out && i0 + u < in) ? load_planes(P + (int64_t)z * ld_p + w_off + (int64_t)c * in + i0 + u, p_plane) : 0.f;
  }
  float bs = 0.f;
  for (int b0 = 0; b0 < B; b0 += 256) {
    __syncthreads();  // the weights are in place / the previous chunk has been used
    const int nb = min(256, B - b0);
    for (int c = 0; c < out; ++c) dzs[c][threadIdx.x] = (int)threadIdx.x < nb ? load_planes(dz + ((int64_t)z * out + c) * ldb + b0 + threadIdx.x, dz_plane) : 0.f;
    __syncthreads();
    if (i < in) {
      for (int bl = lane; bl < nb; bl += 32) {
        float s = 0.f;
        for (int c = 0; c < out; ++c) s = fmaf(wv[w][c], dzs[c][bl], s);
        const int64_t e = ((int64_t)z * in + i) * ldb + b0 + bl;
        if (dh_out != nullptr) store_planes(dh_out + e, out_plane, s);
        const float v = mask_prev[e] ? s : 0.f;
        store_planes(dz_prev + e, out_plane, v);
        bs += (sizeof(T) == 2 && out_plane == 0) ? to_float(from_float<T>(v)) : v;  // the value as stored (three planes hold it exactly)
      }
    }
  }
  bs = warp_sum(bs);
  if (lane == 0) {
    if (i < in) g[(int64_t)z * ld_g + b_off + i] = bs;
    sq[w] = i < in ? bs * bs : 0.f;
  }
  if (partial != nullptr) {
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
      for (int q = 0; q < 8; ++q) t += sq[q];
      partial[(int64_t)z * ld_partial + slot0 + blockIdx.x] = t;
    }
  }
}

// dgrad of layer l: dh = TA(acc + skip_grad);  dz_prev = mask_prev ? dh : 0;  optionally keep dh (residual nets)
template <typename TA>
struct EpiDgrad {
  static constexpr bool kRowsContiguous = true;
  const TA* dh_next;      // gradient w.r.t. the output of a residual layer (nullptr otherwise) [K, width, ldb]
  TA* dh_out;             // nullable
  TA* dz_prev;            // [K, width, ldb]
  const uint8_t* mask_prev;
  int width, ldb;
  __device__ inline void operator()(int z, int b, int f, float acc) const {
    const int64_t e = ((int64_t)z * width + f) * ldb + b;
    const float s = dh_next ? acc + to_float(dh_next[e]) : acc;
    const TA q = from_float<TA>(s);
    if (dh_out) dh_out[e] = q;
    dz_prev[e] = (mask_prev == nullptr || mask_prev[e]) ? q : from_float<TA>(0.f);  // no mask: the raw gradient (pooled layers apply theirs later)
  }
};

// wgrad: g[z][w_off + o * in + i] = acc
struct EpiWgrad {
  static constexpr bool kRowsContiguous = false;  // g[o][i]: contiguous along the GEMM's N index
  float* g;  int64_t ld_g, w_off;  int in;
  __device__ inline void operator()(int z, int o, int i, float acc) const {
    g[(int64_t)z * ld_g + w_off + (int64_t)o * in + i] = acc;
  }
};

// ------------------------------------------------------------------------------------------------ SIMT batched GEMM
// C(z, m, n) = sum_kk A(z, m, kk) * B(z, n, kk), accumulated in fp32 in ascending kk; arbitrary element strides.
// 128 x 64 tile, 16-deep slices, 256 threads, 8 x 4 outputs per thread.  The next slice is fetched from global memory
// into registers (128-bit loads along whichever direction of the operand is contiguous, when aligned) while the current
// one is multiplied out of shared memory.
struct GemmOperand { const void* p; int64_t sz, sr, sk; };  // element (z, r, kk) at p[z*sz + r*sr + kk*sk]

constexpr int kSimtBM = 128, kSimtBN = 64, kSimtBK = 16;

// Four consecutive elements of an operand tile, along the rows (ROWS_CONTIG) or along the contraction index.
// r, kk: first element; rmax, kmax: extents.  Out-of-range elements read as 0.
template <typename T, bool ROWS_CONTIG>
__device__ inline float4 simt_fetch4(const T* __restrict__ base, int64_t sr, int64_t sk, int r, int kk, int rmax, int kmax, bool vec_ok) {
  float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
  if (ROWS_CONTIG) {
    if (kk >= kmax || r >= rmax) return v;
    const T* p = base + (int64_t)r * sr + (int64_t)kk * sk;
    if (sizeof(T) == 4 && vec_ok && r + 3 < rmax) return *reinterpret_cast<const float4*>(p);
    v.x = to_float(p[0]);
    if (r + 1 < rmax) v.y = to_float(p[sr]);
    if (r + 2 < rmax) v.z = to_float(p[2 * sr]);
    if (r + 3 < rmax) v.w = to_float(p[3 * sr]);
  } else {
    if (r >= rmax || kk >= kmax) return v;
    const T* p = base + (int64_t)r * sr + (int64_t)kk * sk;
    if (sizeof(T) == 4 && vec_ok && kk + 3 < kmax) return *reinterpret_cast<const float4*>(p);
    v.x = to_float(p[0]);
    if (kk + 1 < kmax) v.y = to_float(p[sk]);
    if (kk + 2 < kmax) v.z = to_float(p[2 * sk]);
    if (kk + 3 < kmax) v.w = to_float(p[3 * sk]);
  }
  return v;
}

// SPLITK = 2: the block has two groups of 256 threads that walk alternate BK-slabs of the contraction with their own
// shared-memory tiles (twice the warps per SM for the GEMMs whose tile list is shorter than the machine); at the end group 1
// hands its accumulators to group 0 through shared memory and group 0 adds them in a fixed order (own + other) and runs the
// epilogue.  The groups synchronise on their own named barriers (their slab counts may differ by one).
// parts > 1: the contraction is also split over blocks, for products with a small output and a very long contraction (the weight
// gradient of a convolution: Cout x 9 Cin outputs, one term per image position and sample).  blockIdx.z = replica * parts + part;
// part s contracts kk in [s * chunk, (s + 1) * chunk) and hands its result to the epilogue under the index blockIdx.z, which stores
// the partial products for a second, fixed-order pass (EpiPartial / sum_parts_kernel).
template <typename TA_, typename TB_, bool A_MC, bool B_NC, class Epi, int SPLITK = 1>
__global__ void __launch_bounds__(256 * SPLITK)
gemm_simt_kernel(GemmOperand A, GemmOperand Bo, int M, int N, int Kd_all, Epi epi, const int32_t* __restrict__ active, int parts = 1, int chunk = 0) {
  grid_dep_sync();
  constexpr int BM = kSimtBM, BN = kSimtBN, BK = kSimtBK;
  const int z = parts > 1 ? (int)blockIdx.z / parts : (int)blockIdx.z;
  if (active != nullptr && !active[z]) return;  // a waiting replica
  const int k_begin = parts > 1 ? ((int)blockIdx.z % parts) * chunk : 0;
  const int Kd = parts > 1 ? min(Kd_all, k_begin + chunk) : Kd_all;  // end of this block's share of the contraction
  constexpr int A_FLOATS = BK * (BM + 4), B_FLOATS = BK * (BN + 4);
  __shared__ __align__(16) float smem[SPLITK * (A_FLOATS + B_FLOATS)];
  const int grp = SPLITK == 1 ? 0 : (int)threadIdx.x / 256;
  float (*As)[BM + 4] = reinterpret_cast<float (*)[BM + 4]>(smem + grp * (A_FLOATS + B_FLOATS));
  float (*Bs)[BN + 4] = reinterpret_cast<float (*)[BN + 4]>(smem + grp * (A_FLOATS + B_FLOATS) + A_FLOATS);
  auto group_sync = [&]() {
    if (SPLITK == 1) __syncthreads();
    else asm volatile("bar.sync %0, 256;" ::"r"(1 + grp) : "memory");
  };
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const TA_* Ap = reinterpret_cast<const TA_*>(A.p) + (int64_t)z * A.sz;
  const TB_* Bp = reinterpret_cast<const TB_*>(Bo.p) + (int64_t)z * Bo.sz;
  const int tid = threadIdx.x & 255;
  const int tx = tid & 15, ty = tid >> 4;
  // 128-bit loads need the contiguous stride to be 1 (guaranteed by the template flag), the other stride a multiple
  // of 4 elements and the replica's base 16-byte aligned
  const bool vecA = sizeof(TA_) == 4 && (reinterpret_cast<uintptr_t>(Ap) & 15) == 0 && ((A_MC ? A.sk : A.sr) % 4) == 0;
  const bool vecB = sizeof(TB_) == 4 && (reinterpret_cast<uintptr_t>(Bp) & 15) == 0 && ((B_NC ? Bo.sk : Bo.sr) % 4) == 0;
  // this thread's slots in the tiles: A has 2 groups of 4 elements, B has 1
  int a_r[2], a_k[2];
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int f = e * 256 + tid;
    if (A_MC) { a_k[e] = f >> 5; a_r[e] = (f & 31) * 4; } else { a_r[e] = f >> 2; a_k[e] = (f & 3) * 4; }
  }
  int b_r, b_k;
  if (B_NC) { b_k = tid >> 4; b_r = (tid & 15) * 4; } else { b_r = tid >> 2; b_k = (tid & 3) * 4; }

  float acc[8][4];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;

  float4 ra[2], rb;
  auto fetch = [&](int k0) {
#pragma unroll
    for (int e = 0; e < 2; ++e) ra[e] = simt_fetch4<TA_, A_MC>(Ap, A.sr, A.sk, m0 + a_r[e], k0 + a_k[e], M, Kd, vecA);
    rb = simt_fetch4<TB_, B_NC>(Bp, Bo.sr, Bo.sk, n0 + b_r, k0 + b_k, N, Kd, vecB);
  };
  auto stash = [&]() {
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      if (A_MC) {
        *reinterpret_cast<float4*>(&As[a_k[e]][a_r[e]]) = ra[e];
      } else {
        As[a_k[e]][a_r[e]] = ra[e].x; As[a_k[e] + 1][a_r[e]] = ra[e].y; As[a_k[e] + 2][a_r[e]] = ra[e].z; As[a_k[e] + 3][a_r[e]] = ra[e].w;
      }
    }
    if (B_NC) {
      *reinterpret_cast<float4*>(&Bs[b_k][b_r]) = rb;
    } else {
      Bs[b_k][b_r] = rb.x; Bs[b_k + 1][b_r] = rb.y; Bs[b_k + 2][b_r] = rb.z; Bs[b_k + 3][b_r] = rb.w;
    }
  };

  constexpr int KSTEP = SPLITK * BK;  // a group's slabs: k_begin + grp * BK, + KSTEP, ...
  if (k_begin + grp * BK < Kd) {
    fetch(k_begin + grp * BK);
    stash();
  }
  group_sync();
  for (int k0 = k_begin + grp * BK; k0 < Kd; k0 += KSTEP) {
    const bool more = k0 + KSTEP < Kd;
    if (more) fetch(k0 + KSTEP);
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[kk][ty * 8]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[kk][ty * 8 + 4]);
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float a_[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float b_[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a_[i], b_[j], acc[i][j]);
    }
    group_sync();
    if (more) {
      stash();
      group_sync();
    }
  }
  if (SPLITK == 2) {
    // group 1 -> group 0, in two halves of 4 accumulator rows (16 KB each, in the tile memory both groups are done with)
    float4* xch = reinterpret_cast<float4*>(smem);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      __syncthreads();
      if (grp == 1) {
#pragma unroll
        for (int i = 0; i < 4; ++i) xch[i * 256 + tid] = make_float4(acc[4 * h + i][0], acc[4 * h + i][1], acc[4 * h + i][2], acc[4 * h + i][3]);
      }
      __syncthreads();
      if (grp == 0) {
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float4 o = xch[i * 256 + tid];
          acc[4 * h + i][0] += o.x; acc[4 * h + i][1] += o.y; acc[4 * h + i][2] += o.z; acc[4 * h + i][3] += o.w;
        }
      }
    }
    if (grp == 1) return;
  }
  if constexpr (Epi::kRowsContiguous) {
    // the epilogue writes buffers that are contiguous along M (the sample index), while a thread holds 8 x 4 outputs with its
    // lanes spread along N: turn the tile through shared memory, 16 columns at a time, so that a warp hands the functor 32
    // consecutive rows of one column and every access it makes is coalesced
    constexpr int TC = 16;  // columns per turn
    float (*tr)[BM + 1] = reinterpret_cast<float (*)[BM + 1]>(smem);  // [TC][BM + 1] floats, in the tile memory the main loop is done with
    static_assert(TC * (BM + 1) <= A_FLOATS + B_FLOATS && BN % TC == 0 && TC % 4 == 0, "transpose buffer");
    const int warp = tid >> 5, lane = tid & 31;
#pragma unroll
    for (int h = 0; h < BN / TC; ++h) {
      group_sync();  // the main loop (or the previous turn) has been read
      if (tx / (TC / 4) == h) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) tr[(tx % (TC / 4)) * 4 + j][ty * 8 + i] = acc[i][j];
      }
      group_sync();
      for (int nl = warp; nl < TC; nl += 8) {
        const int gn = n0 + h * TC + nl;
        if (gn >= N) break;  // rows of a warp ascend: nothing further is inside
#pragma unroll
        for (int q = 0; q < BM / 32; ++q) {
          const int gm = m0 + q * 32 + lane;
          if (gm < M) epi((int)blockIdx.z, gm, gn, tr[nl][q * 32 + lane]);
        }
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int gm = m0 + ty * 8 + i;
      if (gm >= M) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int gn = n0 + tx * 4 + j;
        if (gn < N) epi((int)blockIdx.z, gm, gn, acc[i][j]);
      }
    }
  }
}

// partial products of a contraction split over blocks: part[zz][m][n], zz = replica * parts + part
struct EpiPartial {
  static constexpr bool kRowsContiguous = false;
  float* part;  int M, N;
  __device__ inline void operator()(int zz, int m, int n, float acc) const { part[((int64_t)zz * M + m) * N + n] = acc; }
};
// g[z][w_off + m * N + n] = sum over the parts, ascending, of part[z * parts + s][m][n].  grid (ceil(M N / 256), K).
__global__ void __launch_bounds__(256)
sum_parts_kernel(const float* __restrict__ part, int parts, int M, int N, float* __restrict__ g, int64_t ld_g, int64_t w_off,
                 const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int z = blockIdx.y;
  if (active != nullptr && !active[z]) return;
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (int64_t)M * N) return;
  float s = 0.f;
  for (int q = 0; q < parts; ++q) s += part[((int64_t)z * parts + q) * M * N + e];
  g[(int64_t)z * ld_g + w_off + e] = s;
}

// The same sum handed to an epilogue functor instead (a forward or dgrad product whose contraction was split over blocks):
// epi(z, m, n, sum over the parts, ascending).  Consecutive threads walk m (the sample index of the feature-major buffers).
// grid (ceil(M N / 256), K).
template <class Epi>
__global__ void __launch_bounds__(256)
sum_parts_epi_kernel(const float* __restrict__ part, int parts, int M, int N, Epi epi, const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int z = blockIdx.y;
  if (active != nullptr && !active[z]) return;
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (int64_t)M * N) return;
  const int n = (int)(e / M), m = (int)(e % M);
  float s = 0.f;
  for (int q = 0; q < parts; ++q) s += part[(((int64_t)z * parts + q) * M + m) * N + n];
  epi(z, m, n, s);
}

// ------------------------------------------------------------------------------------------------ softmax cross-entropy
// logits and dz are feature-major [K, C, ldb].  A block handles 32 consecutive samples (threadIdx.x, so every access is
// coalesced) with 8 class groups (threadIdx.y: classes cg, cg + 8, ...); the per-sample maximum and sum of exponentials
// are combined across the groups in group order.
//   rowloss[k][b] = logsumexp(l) - l[y];  dz[k][c][b] = TA((softmax(l)[c] - [c == y]) / B).
// grid (ceil(B / 32), K), block (32, 8).
template <typename TA>
__global__ void __launch_bounds__(256)
softmax_ce_kernel(float* logits, const int32_t* __restrict__ labels, int B, int C, int ldb,
                  TA* __restrict__ dz, float* __restrict__ rowloss, int* __restrict__ status, const int32_t* __restrict__ active,
                  int64_t plane = 0, const float* __restrict__ part = nullptr, int nparts = 0, const TA* __restrict__ bias = nullptr,
                  int64_t ld_p = 0, int64_t p_plane = 0) {
  grid_dep_sync();
  __shared__ float red[8][33];
  if (active != nullptr && !active[blockIdx.y]) return;
  const int b = blockIdx.x * 32 + threadIdx.x, cg = threadIdx.y, k = blockIdx.y;
  const bool live = b < B;
  if (part != nullptr) {
    // narrow head (head_chunk_kernel): the logits are the bias plus the partial sums of the input chunks, in ascending order
    if (live)
      for (int c = cg; c < C; c += 8) {
        float v = load_planes(bias + (int64_t)k * ld_p + c, p_plane);
        for (int p = 0; p < nparts; ++p) v += part[(((int64_t)k * nparts + p) * kHeadMaxOut + c) * ldb + b];
        logits[((int64_t)k * C + c) * ldb + b] = v;
      }
    __syncthreads();  // a sample's classes are spread over the eight thread rows of this block
  }
  const float* lg = logits + (int64_t)k * C * ldb + (live ? b : 0);
  float m = -INFINITY;
  if (live)
    for (int c = cg; c < C; c += 8) m = fmaxf(m, lg[(int64_t)c * ldb]);
  red[cg][threadIdx.x] = m;
  __syncthreads();
  m = red[0][threadIdx.x];
#pragma unroll
  for (int i = 1; i < 8; ++i) m = fmaxf(m, red[i][threadIdx.x]);
  __syncthreads();
  float se = 0.f;
  if (live)
    for (int c = cg; c < C; c += 8) se += expf(lg[(int64_t)c * ldb] - m);
  red[cg][threadIdx.x] = se;
  __syncthreads();
  se = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) se += red[i][threadIdx.x];
  if (!live) return;
  int y = labels[(int64_t)k * B + b];
  if (y < 0 || y >= C) {
    if (cg == 0) atomicOr(status, STATUS_BAD_INDEX);
    y = 0;
  }
  if (cg == 0) rowloss[(int64_t)k * B + b] = (m + logf(se)) - lg[(int64_t)y * ldb];
  const float inv = 1.f / se, invB = 1.f / (float)B;
  TA* out = dz + (int64_t)k * C * ldb + b;
  for (int c = cg; c < C; c += 8) {
    const float p = expf(lg[(int64_t)c * ldb] - m) * inv;
    store_planes(out + (int64_t)c * ldb, plane, (p - (c == y ? 1.f : 0.f)) * invB);
  }
}

// loss[k] = mean over the minibatch of rowloss[k][b], samples added in ascending order.  grid K, block 32.
__global__ void mean_loss_kernel(const float* __restrict__ rowloss, int B, float* __restrict__ loss, const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int k = blockIdx.x;
  if (active != nullptr && !active[k]) return;
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int b = 0; b < B; ++b) s += (double)rowloss[(int64_t)k * B + b];
    loss[k] = (float)(s / B);
  }
}

// ------------------------------------------------------------------------------------------------ bias gradient
// g[z][b_off + o] = sum_b dz[z][o][b]: one warp per (replica, unit); lane l adds samples l, l + 32, ... in ascending
// order, then the xor-shuffle tree (a fixed order).  grid (ceil(out / 8), K), block 256.
// If partial != nullptr the block also writes the sum of squares of its 8 bias gradients (warps in ascending order)
// to partial[z * ld_partial + slot0 + blockIdx.x], for the fused gradient norm.
// TG = float, or bf16 for the ascent pass of the tensor-core path (same packed bf16 view as its weight gradients).
template <typename TA, typename TG>
__global__ void __launch_bounds__(256)
bias_grad_kernel(const TA* __restrict__ dz, int B, int out, int ldb, TG* __restrict__ g, int64_t ld_g, int64_t b_off,
                 float* __restrict__ partial, int64_t ld_partial, int slot0, const int32_t* __restrict__ active, int64_t plane = 0) {
  grid_dep_sync();
  __shared__ float sq[8];
  if (active != nullptr && !active[blockIdx.y]) return;
  const int w = threadIdx.x >> 5, o = blockIdx.x * 8 + w;
  const int z = blockIdx.y, lane = threadIdx.x & 31;
  float s = 0.f;
  if (o < out) {
    const TA* p = dz + ((int64_t)z * out + o) * ldb;
    for (int b = lane; b < B; b += 32) s += load_planes(p + b, plane);
    s = warp_sum(s);
    if (lane == 0) g[(int64_t)z * ld_g + b_off + o] = from_float<TG>(s);
  }
  if (partial != nullptr) {
    if (lane == 0) sq[w] = s * s;
    __syncthreads();
    if (threadIdx.x == 0) {
      float t = 0.f;
      for (int i = 0; i < 8; ++i) t += sq[i];
      partial[(int64_t)z * ld_partial + slot0 + blockIdx.x] = t;
    }
  }
}

// The same for long rows (a convolution's bias gradient sums over every position and sample): one block per (replica, unit);
// thread t adds elements t, t + 256, ... in ascending order, then the xor-shuffle tree, then the eight warp sums in warp order.
// grid (out, K), block 256.
template <typename TA>
__global__ void __launch_bounds__(256)
bias_grad_long_kernel(const TA* __restrict__ dz, int64_t B, int out, int64_t ldb, float* __restrict__ g, int64_t ld_g, int64_t b_off,
                      const int32_t* __restrict__ active) {
  grid_dep_sync();
  __shared__ float ws[8];
  const int o = blockIdx.x, z = blockIdx.y;
  if (active != nullptr && !active[z]) return;
  const TA* p = dz + ((int64_t)z * out + o) * ldb;
  float s = 0.f;
  for (int64_t b = threadIdx.x; b < B; b += 256) s += to_float(p[b]);
  s = warp_sum(s);
  if ((threadIdx.x & 31) == 0) ws[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < 8; ++i) t += ws[i];
    g[(int64_t)z * ld_g + b_off + o] = t;
  }
}

// ------------------------------------------------------------------------------------------------ convolution layers
// A convolution layer (3x3, stride 1, zero padding 1, ReLU, 2x2 max-pooling) runs on the batched GEMMs through an explicit
// patch matrix.  Feature maps are feature-major like every activation buffer, [K, C, P] with the position index
// p = (y * W + x) * B + b (sample fastest), so that the gathered minibatch [K, C0 * H * W, B] already is the first layer's input and
// the pooled output of the last convolution already is the dense layers' input [K, C * H' * W', B].
//   col[z][ci * 9 + kh * 3 + kw][(y, x, b)] = a[z][ci][(y + kh - 1, x + kw - 1, b)]  (0 outside the image)
// The four helpers below give a thread FOUR consecutive positions p (the same pixel, four consecutive samples: B is a multiple of
// 16) moved as one 16- or 8-byte vector, with 32-bit index arithmetic (H W B < 2^31).
template <typename T>
struct alignas(sizeof(T) * 4) Vec4 { T v[4]; };
struct alignas(4) Byte4 { uint8_t v[4]; };

// One thread per four elements of col, consecutive threads along p.  grid (ceil(P / 1024), Cin * 9, K).
template <typename T>
__global__ void __launch_bounds__(256)
im2col_kernel(const T* __restrict__ a, int Cin, int H, int W, int B, T* __restrict__ col, const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int z = blockIdx.z;
  if (active != nullptr && !active[z]) return;
  const int P = H * W * B;
  const int p = ((int)blockIdx.x * (int)blockDim.x + (int)threadIdx.x) * 4;
  if (p >= P) return;
  const int r = blockIdx.y, ci = r / 9, kh = (r % 9) / 3, kw = r % 3;
  const int b = p % B, pix = p / B;
  const int x = pix % W, y = pix / W;
  const int yy = y + kh - 1, xx = x + kw - 1;
  Vec4<T> v;
#pragma unroll
  for (int i = 0; i < 4; ++i) v.v[i] = from_float<T>(0.f);
  if (yy >= 0 && yy < H && xx >= 0 && xx < W) v = *reinterpret_cast<const Vec4<T>*>(a + ((int64_t)z * Cin + ci) * P + (yy * W + xx) * B + b);
  *reinterpret_cast<Vec4<T>*>(col + ((int64_t)z * Cin * 9 + r) * P + p) = v;
}

// 2x2 max-pooling of the ReLU output r [K, C, (H, W, B)] -> pooled [K, C, (H/2, W/2, B)]; arg = which element of the window
// (dy * 2 + dx, the first maximum in that order).  One thread per four pooled elements.  grid (ceil(P4 / 1024), C, K).
template <typename T>
__global__ void __launch_bounds__(256)
maxpool_kernel(const T* __restrict__ r, int C, int H, int W, int B, T* __restrict__ pooled, uint8_t* __restrict__ arg,
               const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int z = blockIdx.z, c = blockIdx.y;
  if (active != nullptr && !active[z]) return;
  const int Ho = H / 2, Wo = W / 2;
  const int P4 = Ho * Wo * B;
  const int q = ((int)blockIdx.x * (int)blockDim.x + (int)threadIdx.x) * 4;
  if (q >= P4) return;
  const int b = q % B, pix = q / B;
  const int xo = pix % Wo, yo = pix / Wo;
  const T* src = r + ((int64_t)z * C + c) * (int64_t)H * W * B;
  float best[4] = {-1.f, -1.f, -1.f, -1.f};
  Byte4 a;
#pragma unroll
  for (int i = 0; i < 4; ++i) a.v[i] = 0;
#pragma unroll
  for (int dy = 0; dy < 2; ++dy)
#pragma unroll
    for (int dx = 0; dx < 2; ++dx) {
      const Vec4<T> v = *reinterpret_cast<const Vec4<T>*>(src + ((2 * yo + dy) * W + 2 * xo + dx) * B + b);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float f = to_float(v.v[i]);
        if (f > best[i]) { best[i] = f; a.v[i] = (uint8_t)(dy * 2 + dx); }
      }
    }
  Vec4<T> o;
#pragma unroll
  for (int i = 0; i < 4; ++i) o.v[i] = from_float<T>(best[i]);
  *reinterpret_cast<Vec4<T>*>(pooled + ((int64_t)z * C + c) * P4 + q) = o;
  *reinterpret_cast<Byte4*>(arg + ((int64_t)z * C + c) * P4 + q) = a;
}

// Backward of the pooling and the ReLU in one: dz[z][c][(y, x, b)] = dpool[z][c][(y/2, x/2, b)] if (y, x) was its window's
// maximum and the ReLU was active there, else 0.  One thread per four full-resolution elements.  grid (ceil(P / 1024), C, K).
template <typename T>
__global__ void __launch_bounds__(256)
unpool_kernel(const T* __restrict__ dpool, const uint8_t* __restrict__ arg, const uint8_t* __restrict__ mask, int C, int H, int W, int B,
              T* __restrict__ dz, const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int z = blockIdx.z, c = blockIdx.y;
  if (active != nullptr && !active[z]) return;
  const int P = H * W * B;
  const int p = ((int)blockIdx.x * (int)blockDim.x + (int)threadIdx.x) * 4;
  if (p >= P) return;
  const int b = p % B, pix = p / B;
  const int x = pix % W, y = pix / W;
  const int q = ((y / 2) * (W / 2) + x / 2) * B + b;
  const int64_t pc = ((int64_t)z * C + c);
  const Byte4 ar = *reinterpret_cast<const Byte4*>(arg + pc * (P / 4) + q);
  const Byte4 mk = *reinterpret_cast<const Byte4*>(mask + pc * P + p);
  const Vec4<T> dp = *reinterpret_cast<const Vec4<T>*>(dpool + pc * (P / 4) + q);
  const uint8_t me = (uint8_t)((y & 1) * 2 + (x & 1));
  Vec4<T> o;
#pragma unroll
  for (int i = 0; i < 4; ++i) o.v[i] = (ar.v[i] == me && mk.v[i] != 0) ? dp.v[i] : from_float<T>(0.f);
  *reinterpret_cast<Vec4<T>*>(dz + pc * P + p) = o;
}

// Gradient w.r.t. a convolution's input from the gradient of its patch matrix:
//   da[z][ci][(y, x, b)] = sum over (kh, kw) ascending of dcol[z][ci * 9 + kh * 3 + kw][(y - kh + 1, x - kw + 1, b)]  (terms outside the image dropped)
// summed in fp32, stored as T.  One thread per four elements.  grid (ceil(P / 1024), Cin, K).
template <typename T>
__global__ void __launch_bounds__(256)
col2im_kernel(const T* __restrict__ dcol, int Cin, int H, int W, int B, T* __restrict__ da, const int32_t* __restrict__ active) {
  grid_dep_sync();
  const int z = blockIdx.z, ci = blockIdx.y;
  if (active != nullptr && !active[z]) return;
  const int P = H * W * B;
  const int p = ((int)blockIdx.x * (int)blockDim.x + (int)threadIdx.x) * 4;
  if (p >= P) return;
  const int b = p % B, pix = p / B;
  const int x = pix % W, y = pix / W;
  float s[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int kh = 0; kh < 3; ++kh)
#pragma unroll
    for (int kw = 0; kw < 3; ++kw) {
      const int yy = y - kh + 1, xx = x - kw + 1;
      if (yy < 0 || yy >= H || xx < 0 || xx >= W) continue;
      const Vec4<T> v = *reinterpret_cast<const Vec4<T>*>(dcol + ((int64_t)z * Cin * 9 + ci * 9 + kh * 3 + kw) * P + (yy * W + xx) * B + b);
#pragma unroll
      for (int i = 0; i < 4; ++i) s[i] += to_float(v.v[i]);
    }
  Vec4<T> o;
#pragma unroll
  for (int i = 0; i < 4; ++i) o.v[i] = from_float<T>(s[i]);
  *reinterpret_cast<Vec4<T>*>(da + ((int64_t)z * Cin + ci) * P + p) = o;
}

// ------------------------------------------------------------------------------------------------ least squares
// One CTA per replica: r_b = a_b . w - y_b (one warp per sample), loss = sum r_b^2 / (2B),
// g[i] = (1/B) sum_b r_b a_b[i] (one thread per feature, samples in ascending order).
// xb [K, B, in] gathered minibatch, yb [K, B] targets, w = params (row stride ld_p).  Dynamic smem: B floats.
__global__ void __launch_bounds__(256)
lsq_grad_kernel(const float* __restrict__ xb, const float* __restrict__ yb, const float* __restrict__ params,
                int64_t ld_p, int B, int in, float* __restrict__ g, int64_t ld_g, float* __restrict__ loss,
                const int32_t* __restrict__ active) {
  grid_dep_sync();
  extern __shared__ float res[];
  const int k = blockIdx.x;
  if (active != nullptr && !active[k]) return;
  const float* w = params + (int64_t)k * ld_p;
  const float* a = xb + (int64_t)k * B * in;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int b = wid; b < B; b += nw) {
    float p = 0.f;
    for (int i = lane; i < in; i += 32) p = fmaf(a[(int64_t)b * in + i], w[i], p);
    p = warp_sum(p);
    if (lane == 0) res[b] = p - yb[(int64_t)k * B + b];
  }
  __syncthreads();
  if (threadIdx.x == 0 && loss != nullptr) {
    double s = 0.0;
    for (int b = 0; b < B; ++b) s += (double)res[b] * (double)res[b];
    loss[k] = (float)(s / (2.0 * B));
  }
  const float invB = 1.f / (float)B;
  for (int i = threadIdx.x; i < in; i += blockDim.x) {
    float s = 0.f;
    for (int b = 0; b < B; ++b) s = fmaf(res[b], a[(int64_t)b * in + i], s);
    g[(int64_t)k * ld_g + i] = s * invB;
  }
}

}  // namespace lsam
