// gemm_tcgen05.cuh -- batched-over-replicas bf16 GEMMs of the classifier path on the 5th-generation tensor cores:
// TMA (cp.async.bulk.tensor) stages 128B-swizzled operand tiles in shared memory, one elected thread issues
// tcgen05.mma with fp32 accumulators in tensor memory, eight warps (two per lane quadrant) drain the accumulators with
// tcgen05.ld and apply the fused epilogue.  One persistent CTA per SM walks the (replica, m-tile, n-tile) list; the accumulator is
// double-buffered in tensor memory so that the epilogue of a tile overlaps the main loop of the next one.
//
// Every GEMM is D(z, m, n) = sum_kd A(z, m, kd) * B(z, n, kd) with the 128-row M side on the weights:
//   forward   m = output unit, n = sample, kd = input unit   A = W   (kd contiguous)   B = activations (n contiguous)
//   dgrad     m = input unit,  n = sample, kd = output unit  A = W   (m contiguous)    B = dz          (n contiguous)
//   wgrad     m = output unit, n = input unit, kd = sample   A = dz  (kd contiguous)   B = activations (kd contiguous)
// so every weight is read from HBM exactly once per GEMM and the whole minibatch sits in one N tile.  Activations,
// masks, logits and backward signals are feature-major [Z, width, ldb] (sample index contiguous): the accumulator
// row a thread drains from tensor memory is then one feature x 32 consecutive samples, i.e. contiguous 16-byte
// vectors in every buffer the epilogue touches.
//
// PAIR form (cta_group::2): two CTAs of a cluster share one 256-row M tile.  Each CTA stages its own 128 rows of A and
// HALF of the N side of B; one thread of the leader CTA (cluster rank 0) issues tcgen05.mma.cta_group::2 with M = 256,
// which reads the two halves of B from both CTAs' shared memory and leaves rows 0-127 of the tile in the leader's tensor
// memory and rows 128-255 in the peer's.  A CTA so takes in a third fewer operand bytes per flop (the bound of the
// single-CTA form is the rate at which an SM can fill its shared memory).  Each CTA issues its own TMA loads, each into
// its own shared memory only; the loads of both CTAs complete on the leader's `full` barrier, the leader's tcgen05.commit arrives on the
// `empty` / `acc_full` barriers of both CTAs, and both CTAs' epilogue warps arrive on the leader's `acc_empty` barrier.
//
// All waits on mbarriers are bounded: when one expires the CTA raises STATUS_TIMEOUT, stops issuing work, lets the
// copies in flight land, frees its tensor memory and returns (the peer of a pair then runs into its own bounds).
#pragma once

#include <cuda.h>

#include <string>
#include <vector>

#include "common.cuh"
#include "lsam.h"

namespace lsam {

// ------------------------------------------------------------------------------------------------ PTX wrappers
namespace tc {

__device__ inline uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ inline void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ inline void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ inline bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait: false when the limit expires or another role has already given up.
constexpr uint32_t kSpinLimit = 1u << 22;
__device__ inline bool mbar_wait_limit(uint64_t* bar, uint32_t parity, volatile int* abort_flag, uint32_t limit) {
  for (uint32_t i = 0; i < limit; ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  return false;
}
__device__ inline bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  return mbar_wait_limit(bar, parity, abort_flag, kSpinLimit);
}

__device__ inline void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ inline void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 3-D tiled TMA load into this CTA's shared memory (each CTA loads its own tiles), completion counted on an mbarrier.
__device__ inline void tma_load_3d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(smem_u32(bar))
      : "memory");
}

// The same load issued by a CTA of a pair: data into this CTA's shared memory, completion counted on a barrier given by its
// shared::cluster address (the leader's `full` barrier, possibly in the peer CTA).  The data go to the issuing CTA alone.
__device__ inline void tma_load_3d_pair(void* dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(c2), "r"(bar_cluster_addr)
      : "memory");
}
// Bring a tensor map (a kernel parameter) into the descriptor cache before the first copy that uses it.
__device__ inline void prefetch_tensormap(const CUtensorMap* map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(map)) : "memory");
}
__device__ inline uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the location `local` (a shared::cta address of this CTA) in the CTA of rank `rank`
__device__ inline uint32_t map_to_cta(uint32_t local, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local), "r"(rank));
  return r;
}
// Arrive on a barrier of another CTA of the cluster.  Default semantics (release at CTA scope): what the barrier orders here are
// tensor-memory reads, which tcgen05.wait::ld and the tcgen05 fences have already completed.  A release at cluster scope would make the
// warp wait for every global store it has issued before (the outputs of the tile): measured 2000-3000 clocks per tile.
__device__ inline void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
// all threads of both CTAs of the cluster
__device__ inline void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// 3-D tiled TMA store from this CTA's shared memory (bulk async group); rows / columns outside the tensor are clipped.
__device__ inline void tma_store_3d(const CUtensorMap* map, const void* src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(src)), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ inline void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// wait until at most N of this thread's bulk groups are still READING shared memory / still pending at all
template <int N> __device__ inline void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N> __device__ inline void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }

__device__ inline void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ inline void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// pair form: the same warp of BOTH CTAs executes these; the columns are allocated in both CTAs' tensor memory
__device__ inline void tmem_alloc_pair(uint32_t* dst_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ inline void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc], bf16 inputs, fp32 accumulate.
__device__ inline void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrives when all tcgen05.mma issued so far by this thread have completed.
__device__ inline void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// pair form: M = 256 over the two CTAs (D rows 0-127 in the leader's tensor memory, 128-255 in the peer's; each CTA's shared
// memory holds its 128 rows of A and half of the N side of B at the same offsets).  Issued by one thread of the leader.
__device__ inline void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
      "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// the barrier at this offset in BOTH CTAs of the pair arrives when the pair's MMAs issued so far have completed
__device__ inline void umma_commit_pair(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(smem_u32(bar)), "h"((uint16_t)3) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns of tensor memory -> 32 registers per thread (thread = lane).
__device__ inline void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ inline void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  Fields (bits): start address >> 4 [0,14), leading-dimension
// byte offset >> 4 [16,30), stride-dimension byte offset >> 4 [32,46), descriptor version 1 [46,48), swizzle mode
// 2 = 128 B [61,64).
__device__ inline uint64_t smem_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor of kind::f16: D fp32 (bit 4), A and B bf16 (bits 7, 10), operand majors (bits 15, 16:
// 0 = contraction dimension contiguous, 1 = M / N contiguous), N >> 3 at [17,23), M >> 4 at [24,29).
__host__ __device__ constexpr uint32_t instr_desc(int M, int N, bool a_mn, bool b_mn) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn ? 1u : 0u) << 15) | ((b_mn ? 1u : 0u) << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

}  // namespace tc

// ------------------------------------------------------------------------------------------------ epilogue parameters
// TC_EPI_WGRAD_BF16: the weight gradient is stored rounded to bf16 (ascent pass: it only feeds the perturbation, whose
// result is rounded to bf16 anyway; its norm is still taken from the fp32 accumulators).
// TC_EPI_WGRAD_UPD: the descent-pass weight gradient with the worker update (S6) applied in the epilogue: the gradient block
// goes from tensor memory through the warp's staging buffer straight into G = g2 + lambda (x - y), v <- mu v + G,
// x <- x - eta (G + mu v) on the weights of the tile, and never reaches global memory.
enum : int { TC_EPI_FWD_HIDDEN = 0, TC_EPI_FWD_HEAD = 1, TC_EPI_DGRAD = 2, TC_EPI_WGRAD = 3, TC_EPI_WGRAD_BF16 = 4, TC_EPI_WGRAD_UPD = 5 };
__host__ __device__ constexpr bool tc_epi_is_wgrad(int e) { return e >= TC_EPI_WGRAD; }

struct TcEpi {
  // forward: bias (operand copy), out / skip / mask [Z, M, ldb]; head: logits fp32 [Z, M, ldb]
  const bf16* bias;  int64_t ld_p;
  bf16* out;  const bf16* skip;  uint8_t* mask;  float* logits;
  // dgrad: dh_next (skip gradient, nullable), dh_out (nullable), dz_prev, mask_prev  [Z, M, ldb]
  const bf16* dh_next;  bf16* dh_out;  bf16* dz_prev;  const uint8_t* mask_prev;
  // wgrad: g[z * ld_g + w_off + m * ldw + n]
  float* g;  int64_t ld_g, w_off;  int ldw;
  // wgrad: sum of squares of every 32-row block of the tile -> partial[z * ld_partial + slot0 + (mt * n_tiles + nt) * 8 + epilogue warp]
  float* partial;  int64_t ld_partial;  int slot0;
  int ldb;  // sample stride of the feature-major buffers (multiple of 16)
  int run_n;  // stationary weight gradient: consecutive n-tiles (B-stationary: m-tiles) per unit of the work list (>= 1)
  // TC_EPI_WGRAD_UPD: worker state rows (same addressing as g: [z * ld_g + w_off + m * ldw + n]), centre ring and the ring slot
  // each replica reads, the bf16 operand copy, and the step's scalars (lam_k nullable: per-replica pull weight instead of lambda)
  float* upd_x;  float* upd_v;  const float* upd_yring;  const int32_t* upd_slot;  bf16* upd_xop;  const float* upd_lam_k;
  float upd_eta, upd_mu, upd_lambda;  int upd_nesterov;
  // dgrad, optional (bias_g != nullptr; needs the whole minibatch in one N tile): the bias gradient of the layer below,
  // db[m] = sum_b dz_prev[m][b], written to bias_g[z * bias_ld + bias_off + m] (bf16 if bias_bf16, else fp32), and the sum
  // of squares of every 8 consecutive db to partial[z * ld_partial + bias_slot0 + m / 8]
  void* bias_g;  int bias_bf16;  int64_t bias_ld, bias_off;  int bias_slot0;
};

constexpr int kTcBlockM = 128;
constexpr int kTcBlockK = 64;
// warp 0: TMA producer, warp 1: MMA issuer + tensor-memory owner, warps 2-9: epilogue.  Two epilogue warps share each
// tensor-memory lane quadrant (warp % 4) and take alternate pairs of 32-column blocks, so that one drains while the other
// converts and stores.
constexpr int kTcThreads = 320;
constexpr int kTcEpiWarps = 8;

// PAIR: a CTA stages only BLOCK_N / 2 rows of B per k-block, so the ring is deeper
template <int BLOCK_N, bool PAIR = false>
__host__ __device__ constexpr int tc_stages() { return PAIR ? (BLOCK_N == 256 ? 6 : 8) : (BLOCK_N == 256 ? 4 : (BLOCK_N == 128 ? 6 : 8)); }
template <int BLOCK_N, bool PAIR = false>
__host__ __device__ constexpr int tc_stage_bytes() { return (kTcBlockM + (PAIR ? BLOCK_N / 2 : BLOCK_N)) * kTcBlockK * 2; }
constexpr int kTcStageOutBytes = 8 * 4096;  // wgrad epilogue staging: one 32-row x 128-byte block (128B-swizzled) per epilogue warp
// ASTAT (A-stationary, contraction of at most kTcAstatKBlocks k-blocks): the whole A block of a tile row stays in shared
// memory for a run of n-tiles, the ring holds B tiles only
constexpr int kTcAstatKBlocks = 4;
// PAIR: a CTA stages half the rows of a B tile, so the ring is twice as deep in the same space
template <int BLOCK_N, bool PAIR = false>
__host__ __device__ constexpr int tc_astat_stages() { return (BLOCK_N == 256 && !PAIR) ? 4 : 8; }
// SPLIT (fp32 operands as three bf16 planes each): a stage holds the three planes of the A tile and the three planes of
// the B tile of one k-block, and feeds six MMA groups (the plane pairs (i, j) with i + j <= 2)
constexpr int kTcSplitStages = 2;
constexpr int kTcSplitPairs = 6;
// BSTAT (B-stationary): the B block of a tile column (all k-blocks) stays in shared memory over a run of m-tiles, the ring holds A tiles
template <int BLOCK_N>
__host__ __device__ constexpr int tc_bstat_stages() { return BLOCK_N == 256 ? 4 : 8; }
template <int BLOCK_N, bool PAIR = false, bool ASTAT = false, bool SPLIT = false, bool BSTAT = false>
__host__ __device__ constexpr int tc_smem_bytes() {
  return (BSTAT ? kTcAstatKBlocks * BLOCK_N * kTcBlockK * 2 + tc_bstat_stages<BLOCK_N>() * kTcBlockM * kTcBlockK * 2
          : SPLIT ? kTcSplitStages * 3 * tc_stage_bytes<BLOCK_N, false>()
          : ASTAT ? kTcAstatKBlocks * kTcBlockM * kTcBlockK * 2 + tc_astat_stages<BLOCK_N, PAIR>() * (PAIR ? BLOCK_N / 2 : BLOCK_N) * kTcBlockK * 2
                  : tc_stages<BLOCK_N, PAIR>() * tc_stage_bytes<BLOCK_N, PAIR>()) + 1024 /*alignment slack*/ + 512 /*barriers*/ + kTcStageOutBytes;
}

// ------------------------------------------------------------------------------------------------ the kernel
// M, N, Kd: problem extents; Z replicas.  Operands are addressed through 3-D tensor maps (dim 2 = replica):
//   contraction-contiguous operand: map dims {Kd, rows, Z}, box {64, tile rows, 1}
//   M/N-contiguous operand:         map dims {rows, Kd, Z}, box {64, 64, 1} (one box per 64 rows of the tile)
//   PAIR: the B box has BLOCK_N / 2 rows (contraction-contiguous) resp. the CTA loads BLOCK_N / 128 boxes (N-contiguous);
//   the grid is a multiple of 2 and is launched with cluster dimension 2.
//   ASTAT (weight gradient, single CTA or pair, at most 4 k-blocks): the work list is made of runs of ep.run_n consecutive n-tiles of
//   one (replica, m-tile); the A block (dz rows, all k-blocks) is loaded once per run into its own slots and reused by every
//   tile of the run, so a tile takes in BLOCK_N x Kd instead of (128 + BLOCK_N) x Kd operand elements (the weight gradient is
//   bound by the rate at which TMA fills shared memory from L2).  A slot is handed back to the producer as soon as the last
//   tile of the run has used it, so the next run's A block streams in behind the current run's last tile.  In a pair each CTA keeps
//   the block of its own 128 rows and stages half of every B tile; the slot barriers work like the ring's (loads of both CTAs complete
//   on the leader's barrier, the leader's commit frees the slot in both).
//   SPLIT (fp32 GEMM on the bf16 tensor cores): every operand tensor is stored as three bf16 planes p0 = bf16(a),
//   p1 = bf16(a - p0), p2 = bf16(a - p0 - p1), plane p of replica z being "replica" z + p Z of the tensor map.  A stage
//   holds the three planes of both tiles; the product is the sum of the six plane pairs (i, j), i + j <= 2 (the pairs
//   left out are below 2^-24 of |a||b|), smallest terms first, all into the same fp32 accumulator.  The epilogues write
//   their bf16 outputs as three planes again (plane stride Z * M * ldb) and read the bias as the sum of its planes.
//   BSTAT (weight gradient, single CTA, at most 4 k-blocks): the mirror image of ASTAT.  The work list is made of runs of ep.run_n
//   consecutive m-tiles of one (replica, n-tile); the B block (activation rows of the tile column, all k-blocks) is loaded once per run
//   and the ring streams the A tiles (dz rows), so a tile takes in 128 x Kd instead of BLOCK_N x Kd operand elements: half the bytes of
//   the A-stationary form at BLOCK_N = 256.  (Measured per tile, stand-alone: the A-stationary main loop waits for its loads, 128 KB per
//   tile at about 30 B per clock and SM, while the epilogue is hidden.)
template <int BLOCK_N, bool A_MN, bool B_MN, int EPI, bool PAIR, bool ASTAT = false, bool SPLIT = false, bool BSTAT = false>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                    const __grid_constant__ CUtensorMap map_c, int M, int N, int Kd,
                    int Z, TcEpi ep, int* __restrict__ status, const int32_t* __restrict__ active) {
  static_assert(!PAIR || BLOCK_N >= 128, "the pair form needs 64 rows of B per CTA");
  static_assert(!ASTAT || (!A_MN && !B_MN), "A-stationary form: both operands contraction-contiguous");
  static_assert(!SPLIT || (!PAIR && !ASTAT && BLOCK_N <= 128 && EPI <= TC_EPI_WGRAD), "three-plane form: single CTAs, N tile of at most 128, fp32 gradient");
  static_assert(!BSTAT || (!PAIR && !ASTAT && !SPLIT && !A_MN && !B_MN), "B-stationary form: single CTA, both operands contraction-contiguous");
  constexpr bool STAT = ASTAT || BSTAT;  // one operand block stays in shared memory over a run of tiles
  constexpr int STAGES = BSTAT ? tc_bstat_stages<BLOCK_N>() : SPLIT ? kTcSplitStages : (ASTAT ? tc_astat_stages<BLOCK_N, PAIR>() : tc_stages<BLOCK_N, PAIR>());
  constexpr int NPL = SPLIT ? 3 : 1;  // planes per operand
  constexpr int A_BYTES = kTcBlockM * kTcBlockK * 2;
  constexpr int B_ROWS = PAIR ? BLOCK_N / 2 : BLOCK_N;  // rows of the N side staged by this CTA
  constexpr int B_BYTES = B_ROWS * kTcBlockK * 2;
  constexpr int TILE_M = PAIR ? 2 * kTcBlockM : kTcBlockM;  // rows of a tile of the work list
  // two accumulator stages (power of two >= 32).  SPLIT: a stage is two accumulators, [BLOCK_N columns: the product of the
  // leading planes][BLOCK_N columns: the five small plane pairs]; the epilogue adds them.  The tensor core aligns every
  // addend to the accumulator and drops the bits below its last place, so small terms added to a large running sum lose
  // their low bits one-sidedly (measured: 9e-6 relative error at a contraction of 784 against 6e-7 with the small terms kept apart).
  constexpr uint32_t ACC_COLS = SPLIT ? 2 * BLOCK_N : BLOCK_N;
  constexpr uint32_t TMEM_COLS = 2 * ACC_COLS;
  constexpr uint32_t IDESC = tc::instr_desc(TILE_M, BLOCK_N, A_MN, B_MN);

  extern __shared__ uint8_t smem_raw[];
  // round the tile area up to 1024 bytes by pointer arithmetic on the shared array itself (keeps the address space known)
  uint8_t* tiles = smem_raw + ((1024u - (tc::smem_u32(smem_raw) & 1023u)) & 1023u);
  // ASTAT: [A slots: kTcAstatKBlocks x A_BYTES][B ring: STAGES x B_BYTES]; BSTAT: [B slots: kTcAstatKBlocks x B_BYTES][A ring: STAGES x A_BYTES];
  // else a ring of STAGES x (A tile, B tile).  SPLIT: a stage is [A plane 0, 1, 2][B plane 0, 1, 2]
  constexpr int SLOT_BYTES = ASTAT ? A_BYTES : B_BYTES;  // a slot of the stationary block
  constexpr int RING_STRIDE = ASTAT ? B_BYTES : (BSTAT ? A_BYTES : NPL * (A_BYTES + B_BYTES));
  constexpr int RING_B_OFF = STAT ? 0 : NPL * A_BYTES;
  uint8_t* ring = tiles + (STAT ? kTcAstatKBlocks * SLOT_BYTES : 0);
  uint8_t* stage = ring + STAGES * RING_STRIDE;  // 1024-byte aligned: everything before it is a multiple of 1024
  uint64_t* bars = reinterpret_cast<uint64_t*>(stage + kTcStageOutBytes);
  uint64_t* full = bars;                     // [STAGES]  TMA -> MMA
  uint64_t* empty = bars + STAGES;           // [STAGES]  MMA -> TMA
  uint64_t* acc_full = bars + 2 * STAGES;    // [2]       MMA -> epilogue
  uint64_t* acc_empty = acc_full + 2;        // [2]       epilogue -> MMA
  uint64_t* bias_bar = acc_empty + 2;        // [4 quadrants][2]  dgrad: the two epilogue warps of a quadrant have left their partial bias sums
  uint64_t* a_full = bias_bar + 8;           // [4]  ASTAT / BSTAT: slot kb of the stationary block loaded        TMA -> MMA
  uint64_t* a_empty = a_full + 4;            // [4]  ASTAT / BSTAT: slot kb free again                            MMA -> TMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(a_empty + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (M + TILE_M - 1) / TILE_M;
  const int n_tiles = (N + BLOCK_N - 1) / BLOCK_N;
  const int k_blocks = (Kd + kTcBlockK - 1) / kTcBlockK;
  // work list: units of (replica, m-tile, run of n-tiles), B-stationary: (replica, n-tile, run of m-tiles); a run is one tile unless a block is stationary
  // a run walks `inner` (n-tiles; m-tiles in the B-stationary form) with the other tile index (`outer`) fixed
  const int run_n = STAT ? (ep.run_n > 0 ? ep.run_n : 1) : 1;
  const int inner_tiles = BSTAT ? m_tiles : n_tiles, outer_tiles = BSTAT ? n_tiles : m_tiles;
  const int runs = (inner_tiles + run_n - 1) / run_n;
  const int64_t total = (int64_t)Z * outer_tiles * runs;
  // a pair walks the work list together: unit = index of this CTA (or of its pair), units = how many walk the list
  const uint32_t rank = PAIR ? tc::cluster_ctarank() : 0u;
  const bool leader = rank == 0u;
  const int64_t unit = PAIR ? blockIdx.x / 2 : blockIdx.x, units = PAIR ? gridDim.x / 2 : gridDim.x;
  const int m_off = (int)rank * kTcBlockM;   // this CTA's rows inside a tile
  const int n_off = (int)rank * B_ROWS;      // this CTA's share of the N side of B

  // the next kernel's blocks may take the SMs this grid leaves free; this grid's own set-up (barriers, tensor memory, tensor
  // maps: nothing a predecessor writes) runs before it waits for the grids before it
  grid_dep_launch();
  if (threadIdx.x == 0) {
    tc::prefetch_tensormap(&map_a);
    tc::prefetch_tensormap(&map_b);
    if (tc_epi_is_wgrad(EPI)) tc::prefetch_tensormap(&map_c);
    for (int s = 0; s < STAGES; ++s) { tc::mbar_init(&full[s], 1); tc::mbar_init(&empty[s], 1); }
    for (int s = 0; s < 2; ++s) { tc::mbar_init(&acc_full[s], 1); tc::mbar_init(&acc_empty[s], PAIR ? 2 * kTcEpiWarps : kTcEpiWarps); }
    for (int s = 0; s < 8; ++s) tc::mbar_init(&bias_bar[s], 2);
    for (int s = 0; s < 4; ++s) { tc::mbar_init(&a_full[s], 1); tc::mbar_init(&a_empty[s], 1); }
    static_assert((2 * STAGES + 4 + 8 + 8) * 8 + 8 <= 512, "barrier area");
    *abort_flag = 0;
    tc::fence_barrier_init();
  }
  if (warp == 1) {
    if (PAIR) tc::tmem_alloc_pair(tmem_slot, TMEM_COLS);
    else tc::tmem_alloc(tmem_slot, TMEM_COLS);
  }
  tc::tc_fence_before();
  __syncthreads();
  if (PAIR) tc::cluster_sync_all();  // the peer's barriers exist before anything arrives on them
  tc::tc_fence_after();
  grid_dep_wait();  // every thread: from here on the roles read and write what earlier kernels produced
  const uint32_t tmem_base = *tmem_slot;
  if (PAIR) {
    // one MMA addresses the accumulator columns of both CTAs with the same number, so the two allocations must agree
    // (they do on SMs whose tensor memory was free); otherwise no role starts and the launch reports it
    uint32_t peer_base;
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(peer_base) : "r"(tc::map_to_cta(tc::smem_u32(tmem_slot), rank ^ 1u)) : "memory");
    if (peer_base != tmem_base) {
      if (threadIdx.x == 0) { *abort_flag = 1; atomicOr(status, STATUS_TIMEOUT); }
      __syncthreads();
    }
  }
  const bool run = !PAIR || (*abort_flag == 0);

  if (!run) {
    // nothing to do: fall through to the teardown
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      uint32_t run_ph = 0;  // phase of the barriers of the stationary slots, one flip per run
      for (int64_t t = unit; t < total && ok; t += units) {
        const int r = (int)(t % runs), fixed = (int)((t / runs) % outer_tiles), z = (int)(t / ((int64_t)runs * outer_tiles));
        if (active != nullptr && !active[z]) continue;  // waiting replica: all three roles skip the same tiles
        const int nt_begin = r * run_n, nt_end = (nt_begin + run_n < inner_tiles) ? nt_begin + run_n : inner_tiles;
        for (int it = nt_begin; it < nt_end && ok; ++it) {
        const int mt = BSTAT ? it : fixed, nt = BSTAT ? fixed : it;
        const int m0 = mt * TILE_M + m_off, n0 = nt * BLOCK_N + n_off;
        for (int kb = 0; kb < k_blocks; ++kb) {
          const int k0 = kb * kTcBlockK;
          if (BSTAT && it == nt_begin) {
            // first tile of a run: bring in B slot kb as soon as the previous run has released it
            if (!tc::mbar_wait(&a_empty[kb], run_ph ^ 1u, abort_flag)) { ok = false; break; }
            tc::mbar_expect_tx(&a_full[kb], B_BYTES);
            tc::tma_load_3d(tiles + kb * B_BYTES, &map_b, k0, n0, z, &a_full[kb]);
          }
          if (ASTAT && it == nt_begin) {
            // first tile of a run: bring in A slot kb as soon as the previous run has released it (pair form: each CTA its own
            // 128 rows into its own slot, both loads completing on the leader's barrier, which the leader arms with the bytes of both)
            if (!tc::mbar_wait(&a_empty[kb], run_ph ^ 1u, abort_flag)) { ok = false; break; }
            if (PAIR) {
              if (leader) tc::mbar_expect_tx(&a_full[kb], 2 * A_BYTES);
              tc::tma_load_3d_pair(tiles + kb * A_BYTES, &map_a, k0, m0, z, tc::map_to_cta(tc::smem_u32(&a_full[kb]), 0u));
            } else {
              tc::mbar_expect_tx(&a_full[kb], A_BYTES);
              tc::tma_load_3d(tiles + kb * A_BYTES, &map_a, k0, m0, z, &a_full[kb]);
            }
          }
          if (!tc::mbar_wait(&empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
          uint8_t* a_dst = ring + s * RING_STRIDE;
          uint8_t* b_dst = a_dst + RING_B_OFF;
          if (BSTAT) {
            tc::mbar_expect_tx(&full[s], A_BYTES);
            tc::tma_load_3d(a_dst, &map_a, k0, m0, z, &full[s]);
          } else if (ASTAT && PAIR) {
            if (leader) tc::mbar_expect_tx(&full[s], 2 * B_BYTES);
            tc::tma_load_3d_pair(b_dst, &map_b, k0, n0, z, tc::map_to_cta(tc::smem_u32(&full[s]), 0u));
          } else if (ASTAT) {
            tc::mbar_expect_tx(&full[s], B_BYTES);
            tc::tma_load_3d(b_dst, &map_b, k0, n0, z, &full[s]);
          } else if (PAIR) {
            // both CTAs' loads of this stage complete on the leader's barrier, which the leader arms with the bytes of both
            if (leader) tc::mbar_expect_tx(&full[s], 2 * (A_BYTES + B_BYTES));
            const uint32_t bar = tc::map_to_cta(tc::smem_u32(&full[s]), 0u);
            if (A_MN) {
#pragma unroll
              for (int i = 0; i < kTcBlockM / 64; ++i) tc::tma_load_3d_pair(a_dst + i * 8192, &map_a, m0 + 64 * i, k0, z, bar);
            } else {
              tc::tma_load_3d_pair(a_dst, &map_a, k0, m0, z, bar);
            }
            if (B_MN) {
#pragma unroll
              for (int i = 0; i < B_ROWS / 64; ++i) tc::tma_load_3d_pair(b_dst + i * 8192, &map_b, n0 + 64 * i, k0, z, bar);
            } else {
              tc::tma_load_3d_pair(b_dst, &map_b, k0, n0, z, bar);
            }
          } else {
            tc::mbar_expect_tx(&full[s], NPL * (A_BYTES + B_BYTES));
#pragma unroll
            for (int p = 0; p < NPL; ++p) {
              const int zp = z + p * Z;  // plane p of replica z
              uint8_t* a_p = a_dst + p * A_BYTES;
              uint8_t* b_p = b_dst + p * B_BYTES;
              if (A_MN) {
#pragma unroll
                for (int i = 0; i < kTcBlockM / 64; ++i) tc::tma_load_3d(a_p + i * 8192, &map_a, m0 + 64 * i, k0, zp, &full[s]);
              } else {
                tc::tma_load_3d(a_p, &map_a, k0, m0, zp, &full[s]);
              }
              if (B_MN) {
#pragma unroll
                for (int i = 0; i < BLOCK_N / 64; ++i) tc::tma_load_3d(b_p + i * 8192, &map_b, n0 + 64 * i, k0, zp, &full[s]);
              } else {
                tc::tma_load_3d(b_p, &map_b, k0, n0, zp, &full[s]);
              }
            }
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        }
        run_ph ^= 1u;
      }
      if (!ok) { *abort_flag = 1; atomicOr(status, STATUS_TIMEOUT); }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && leader) {  // pair form: the leader issues for both CTAs
      int s = 0;
      uint32_t ph = 0;
      int as = 0;
      uint32_t aph = 0;
      bool ok = true;
      uint32_t run_ph = 0;
      for (int64_t t = unit; t < total && ok; t += units) {
        if (active != nullptr && !active[(int)(t / ((int64_t)runs * outer_tiles))]) continue;
        const int nt_begin = (int)(t % runs) * run_n, nt_end = (nt_begin + run_n < inner_tiles) ? nt_begin + run_n : inner_tiles;
        for (int nt = nt_begin; nt < nt_end && ok; ++nt) {
        if (!tc::mbar_wait(&acc_empty[as], aph ^ 1u, abort_flag)) { ok = false; break; }
        tc::tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)as * ACC_COLS;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (STAT && nt == nt_begin && !tc::mbar_wait(&a_full[kb], run_ph, abort_flag)) { ok = false; break; }
          if (!tc::mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
          tc::tc_fence_after();
          const uint32_t a_addr = tc::smem_u32(ASTAT ? tiles + kb * A_BYTES : ring + s * RING_STRIDE);
          const uint32_t b_addr = tc::smem_u32(BSTAT ? tiles + kb * B_BYTES : ring + s * RING_STRIDE + RING_B_OFF);
#pragma unroll
          for (int pp = 0; pp < (SPLIT ? kTcSplitPairs : 1); ++pp) {
            // SPLIT: plane pairs (A plane, B plane) in the order (0,2) (1,1) (2,0) (0,1) (1,0) into the second accumulator,
            // then (0,0) into the first
            const int pa = SPLIT ? (pp < 3 ? pp : (pp < 5 ? pp - 3 : 0)) : 0;
            const int pb = SPLIT ? (pp < 3 ? 2 - pp : (pp < 5 ? 4 - pp : 0)) : 0;
            const uint32_t a_pl = a_addr + (uint32_t)(pa * A_BYTES), b_pl = b_addr + (uint32_t)(pb * B_BYTES);
            const uint32_t d_pp = (SPLIT && pp < 5) ? d_tmem + (uint32_t)BLOCK_N : d_tmem;
            const int first = (SPLIT && pp == 5) ? 0 : pp;  // 0: this pair opens its accumulator at the first k-block
#pragma unroll
            for (int k = 0; k < kTcBlockK / 16; ++k) {
              // contraction-contiguous tile: rows of 128 B, 8-row groups 1024 B apart, a K = 16 slice is 32 B further along the row;
              // M/N-contiguous tile: 64-element blocks 8192 B apart (leading offset), 8 contraction rows = 1024 B (stride offset),
              // a K = 16 slice is two such groups = 2048 B further.
              const uint64_t ad = A_MN ? tc::smem_desc(a_pl + k * 2048, 8192, 1024) : tc::smem_desc(a_pl + k * 32, 16, 1024);
              const uint64_t bd = B_MN ? tc::smem_desc(b_pl + k * 2048, 8192, 1024) : tc::smem_desc(b_pl + k * 32, 16, 1024);
              if (PAIR) tc::umma_bf16_pair(d_pp, ad, bd, IDESC, (kb | k | first) != 0 ? 1u : 0u);
              else tc::umma_bf16(d_pp, ad, bd, IDESC, (kb | k | first) != 0 ? 1u : 0u);
            }
          }
          // frees the stage (in both CTAs of a pair) when these MMAs have read it
          if (PAIR) tc::umma_commit_pair(&empty[s]);
          else tc::umma_commit(&empty[s]);
          if (STAT && nt == nt_end - 1) {  // last tile of the run: the slot (of both CTAs of a pair) is free once these MMAs are done
            if (PAIR) tc::umma_commit_pair(&a_empty[kb]);
            else tc::umma_commit(&a_empty[kb]);
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        if (PAIR) tc::umma_commit_pair(&acc_full[as]);
        else tc::umma_commit(&acc_full[as]);
        if (++as == 2) { as = 0; aph ^= 1u; }
        }
        run_ph ^= 1u;
      }
      if (!ok) { *abort_flag = 1; atomicOr(status, STATUS_TIMEOUT); }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (4 warps, one TMEM lane quadrant each)
    const int quad = warp & 3;
    const int ew = warp - 2;       // epilogue warp 0..7
    const int half = ew >> 2;      // which of the two warps of this quadrant
    uint8_t* sbuf_cur = stage;
    int as = 0;
    uint32_t aph = 0;
    bool ok = true;
    const uint32_t acc_empty_leader[2] = {PAIR ? tc::map_to_cta(tc::smem_u32(&acc_empty[0]), 0u) : 0u, PAIR ? tc::map_to_cta(tc::smem_u32(&acc_empty[1]), 0u) : 0u};
    for (int64_t t = unit; t < total && ok; t += units) {
      const int r_ = (int)(t % runs), fixed = (int)((t / runs) % outer_tiles), z = (int)(t / ((int64_t)runs * outer_tiles));
      if (active != nullptr && !active[z]) continue;
      const int nt_begin = r_ * run_n, nt_end = (nt_begin + run_n < inner_tiles) ? nt_begin + run_n : inner_tiles;
      for (int it = nt_begin; it < nt_end && ok; ++it) {
      const int mt = BSTAT ? it : fixed, nt = BSTAT ? fixed : it;
      const int m_base = mt * TILE_M + m_off;  // first row of the 128 rows this CTA drains
      const int m = m_base + quad * 32 + lane;
      const int n0 = nt * BLOCK_N;
      if (!tc::mbar_wait(&acc_full[as], aph, abort_flag)) { ok = false; break; }
      tc::tc_fence_after();
      const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)as * ACC_COLS;
      float bias = 0.f;
      float ssq4[4] = {0.f, 0.f, 0.f, 0.f};  // wgrad: sum of squares of this thread's row of the tile, four interleaved partial sums (column mod 4)
      float bsum = 0.f; // dgrad: this thread's share of the bias gradient of its row (samples of its chunks, ascending)
      if ((EPI == TC_EPI_FWD_HIDDEN || EPI == TC_EPI_FWD_HEAD) && m < M) {
        const bf16* bp = ep.bias + (int64_t)z * ep.ld_p + m;
        bias = to_float(bp[0]);
        if (SPLIT) bias = (bias + to_float(bp[(int64_t)Z * ep.ld_p])) + to_float(bp[2 * (int64_t)Z * ep.ld_p]);  // exact: the planes of an fp32 value
      }
#pragma unroll 1
      for (int c = 0; c < BLOCK_N / 32; ++c) {
        if (((c >> 1) & 1) != half) continue;  // pairs of blocks alternate between the two warps of a quadrant
        uint32_t r[32];
        tc::tmem_ld32(taddr + (uint32_t)(c * 32), r);
        tc::tmem_ld_wait();
        if (SPLIT) {
          uint32_t r2[32];
          tc::tmem_ld32(taddr + (uint32_t)(BLOCK_N + c * 32), r2);
          tc::tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r2[j]));
        }
        const int nb = n0 + c * 32;
        if (EPI == TC_EPI_WGRAD_UPD) {
          const int mrow0 = m_base + quad * 32;
          if (mrow0 < M && nb < N) {  // warp-uniform
#pragma unroll
            for (int j = 0; j < 32; ++j) ssq4[j & 3] = fmaf(__uint_as_float(r[j]), __uint_as_float(r[j]), ssq4[j & 3]);  // zero-filled edges add 0
            // transpose through the warp's staging buffer: written row = lane (swizzled 16-byte chunks), read back so that
            // 8 lanes cover the 128 contiguous bytes of a row and every global access below is coalesced
            uint8_t* sb = stage + ew * 4096;
            __syncwarp();  // the reads of the previous block are done
#pragma unroll
            for (int q = 0; q < 8; ++q)
              *reinterpret_cast<float4*>(sb + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                  make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
            __syncwarp();
            const int64_t base = (int64_t)z * ep.ld_g + ep.w_off;
            const float* yb = ep.upd_yring + (int64_t)ep.upd_slot[z] * ep.ld_g + ep.w_off;
            const float lam = ep.upd_lam_k != nullptr ? ep.upd_lam_k[z] : ep.upd_lambda;
            const int cq = lane & 7, rsub = lane >> 3;
#pragma unroll
            for (int pass = 0; pass < 2; ++pass) {
              float4 gv[4], xv[4], vv[4], yv[4];
              int64_t off[4];
              bool okv[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const int row = (pass * 4 + i) * 4 + rsub;
                const int mm = mrow0 + row, nn = nb + 4 * cq;
                okv[i] = mm < M && nn < N;  // rows are multiples of 8 elements long: a 4-element chunk is inside or outside as a whole
                off[i] = (int64_t)mm * ep.ldw + nn;
                gv[i] = *reinterpret_cast<const float4*>(sb + row * 128 + ((cq ^ (row & 7)) << 4));
                if (okv[i]) {
                  xv[i] = *reinterpret_cast<const float4*>(ep.upd_x + base + off[i]);
                  vv[i] = *reinterpret_cast<const float4*>(ep.upd_v + base + off[i]);
                  yv[i] = __ldg(reinterpret_cast<const float4*>(yb + off[i]));
                }
              }
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                if (!okv[i]) continue;
                float G;
#define LSAM_FUPD(c)                                                                  \
  G = fmaf(lam, xv[i].c - yv[i].c, gv[i].c);                                          \
  vv[i].c = fmaf(ep.upd_mu, vv[i].c, G);                                              \
  xv[i].c = ep.upd_nesterov ? xv[i].c - ep.upd_eta * fmaf(ep.upd_mu, vv[i].c, G) : xv[i].c - ep.upd_eta * vv[i].c;
                LSAM_FUPD(x) LSAM_FUPD(y) LSAM_FUPD(z) LSAM_FUPD(w)
#undef LSAM_FUPD
                *reinterpret_cast<float4*>(ep.upd_x + base + off[i]) = xv[i];
                __stcs(reinterpret_cast<float4*>(ep.upd_v + base + off[i]), vv[i]);
                __nv_bfloat162 lo = __floats2bfloat162_rn(xv[i].x, xv[i].y), hi = __floats2bfloat162_rn(xv[i].z, xv[i].w);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t*>(&lo);
                pk.y = *reinterpret_cast<uint32_t*>(&hi);
                *reinterpret_cast<uint2*>(ep.upd_xop + base + off[i]) = pk;
              }
            }
          }
        } else if (EPI == TC_EPI_WGRAD || EPI == TC_EPI_WGRAD_BF16) {
          // The warp's 32 x 32 fp32 block goes to shared memory in the 128-byte-swizzled layout of the output tensor
          // map (row = lane, 16-byte chunk q stored at position q ^ (row % 8)), then one TMA store writes it to the
          // gradient rows (clipped at the ragged edges).  Two buffers per warp: the store of a chunk overlaps the
          // staging of the next one.
          const int mrow0 = m_base + quad * 32;
          if (mrow0 < M && nb < N) {  // warp-uniform: blocks wholly outside the matrix are neither staged nor stored
#pragma unroll
            for (int j = 0; j < 32; ++j) ssq4[j & 3] = fmaf(__uint_as_float(r[j]), __uint_as_float(r[j]), ssq4[j & 3]);  // zero-filled edges add 0
            // fp32: one 32-column block per store.  bf16: two consecutive blocks share one buffer (rows of 64 bf16 = 128
            // bytes, the same swizzle) and are stored together after the second one, or after the last valid one.
            const bool first_half = (EPI == TC_EPI_WGRAD) || ((c & 1) == 0);
            const bool last_half = (EPI == TC_EPI_WGRAD) || ((c & 1) == 1) || (nb + 32 >= N);
            if (first_half) {
              sbuf_cur = stage + ew * 4096;
              // the previous store of this warp must have finished reading the buffer (the other warp of the quadrant
              // keeps the SM busy meanwhile)
              if (lane == 0) tc::bulk_wait_read<0>();
              __syncwarp();
            }
            if (EPI == TC_EPI_WGRAD) {
#pragma unroll
              for (int q = 0; q < 8; ++q)
                *reinterpret_cast<float4*>(sbuf_cur + lane * 128 + ((q ^ (lane & 7)) << 4)) =
                    make_float4(__uint_as_float(r[4 * q]), __uint_as_float(r[4 * q + 1]), __uint_as_float(r[4 * q + 2]), __uint_as_float(r[4 * q + 3]));
            } else {
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                uint4 pk;
                uint32_t* pw = reinterpret_cast<uint32_t*>(&pk);
#pragma unroll
                for (int h = 0; h < 4; ++h) {
                  __nv_bfloat162 two = __floats2bfloat162_rn(__uint_as_float(r[8 * q + 2 * h]), __uint_as_float(r[8 * q + 2 * h + 1]));
                  pw[h] = *reinterpret_cast<uint32_t*>(&two);
                }
                const int qq = (c & 1) * 4 + q;  // 16-byte chunk of the 128-byte row
                *reinterpret_cast<uint4*>(sbuf_cur + lane * 128 + ((qq ^ (lane & 7)) << 4)) = pk;
              }
            }
            if (last_half) {
              tc::fence_proxy_async();
              __syncwarp();
              if (lane == 0) {
                tc::tma_store_3d(&map_c, sbuf_cur, EPI == TC_EPI_WGRAD ? nb : nb - (c & 1) * 32, mrow0, z);
                tc::bulk_commit();
              }
            }
          }
        } else if (m < M && nb < N) {
          // element (unit m, sample nb + j) of the feature-major buffers: 32 consecutive samples per thread
          const int64_t t0 = ((int64_t)z * M + m) * ep.ldb + nb;
          const bool full = nb + 32 <= N;
          const int nvalid = full ? 32 : N - nb;
          if (SPLIT && EPI != TC_EPI_FWD_HEAD) {
            // three-plane outputs: forward  a = skip + relu(acc + bias) with its mask; dgrad  dh = acc + dh_next,  dz_prev = mask ? dh : 0
            uint4 ov[4], mv[2];
            bf16* ob = reinterpret_cast<bf16*>(ov);
            uint8_t* mb = reinterpret_cast<uint8_t*>(mv);
            const int64_t plane = (int64_t)Z * M * ep.ldb;
            float rr[32];
            // r[j] += the fp32 value held in the three planes at src: the planes are summed first (exact), so the accumulator
            // takes one fp32 addition of the stored value
            auto add_planes = [&](const bf16* src) {
#pragma unroll
              for (int p = 0; p < 3; ++p) {
                if (full) {
#pragma unroll
                  for (int q = 0; q < 4; ++q) ov[q] = *reinterpret_cast<const uint4*>(src + p * plane + t0 + q * 8);
                } else {
#pragma unroll
                  for (int j = 0; j < 32; ++j) ob[j] = j < nvalid ? src[p * plane + t0 + j] : __float2bfloat16_rn(0.f);
                }
#pragma unroll
                for (int j = 0; j < 32; ++j) rr[j] = p == 0 ? to_float(ob[j]) : rr[j] + to_float(ob[j]);
              }
#pragma unroll
              for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + rr[j]);
            };
            // the three planes of rr[j] -> dst (rr is used up)
            auto store_planes = [&](bf16* dst) {
#pragma unroll
              for (int p = 0; p < 3; ++p) {
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                  ob[j] = __float2bfloat16_rn(rr[j]);
                  rr[j] -= to_float(ob[j]);  // exact: the part the planes so far leave out
                }
                if (full) {
#pragma unroll
                  for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(dst + p * plane + t0 + q * 8) = ov[q];
                } else {
#pragma unroll
                  for (int j = 0; j < 32; ++j)
                    if (j < nvalid) dst[p * plane + t0 + j] = ob[j];
                }
              }
            };
            if (EPI == TC_EPI_FWD_HIDDEN) {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                const float v = __uint_as_float(r[j]) + bias;
                mb[j] = v > 0.f ? 1 : 0;
                r[j] = __float_as_uint(v > 0.f ? v : 0.f);
              }
              if (full) {
#pragma unroll
                for (int q = 0; q < 2; ++q) *reinterpret_cast<uint4*>(ep.mask + t0 + q * 16) = mv[q];
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j)
                  if (j < nvalid) ep.mask[t0 + j] = mb[j];
              }
              if (ep.skip != nullptr) add_planes(ep.skip);
#pragma unroll
              for (int j = 0; j < 32; ++j) rr[j] = __uint_as_float(r[j]);
              store_planes(ep.out);
            } else {
              if (ep.dh_next != nullptr) add_planes(ep.dh_next);
              if (ep.dh_out != nullptr) {
#pragma unroll
                for (int j = 0; j < 32; ++j) rr[j] = __uint_as_float(r[j]);
                store_planes(ep.dh_out);
              }
              if (full) {
#pragma unroll
                for (int q = 0; q < 2; ++q) mv[q] = *reinterpret_cast<const uint4*>(ep.mask_prev + t0 + q * 16);
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) mb[j] = j < nvalid ? ep.mask_prev[t0 + j] : 0;
              }
#pragma unroll
              for (int j = 0; j < 32; ++j) rr[j] = mb[j] ? __uint_as_float(r[j]) : 0.f;
              if (ep.bias_g != nullptr) {  // masked entries and entries past the minibatch are zero
#pragma unroll
                for (int j = 0; j < 32; ++j) bsum += rr[j];
              }
              store_planes(ep.dz_prev);
            }
          } else if (EPI == TC_EPI_FWD_HIDDEN) {
            uint4 skv[4], ov[4], mv[2];
            bf16* skb = reinterpret_cast<bf16*>(skv);
            bf16* ob = reinterpret_cast<bf16*>(ov);
            uint8_t* mb = reinterpret_cast<uint8_t*>(mv);
            if (ep.skip != nullptr) {
              if (full) {
#pragma unroll
                for (int q = 0; q < 4; ++q) skv[q] = *reinterpret_cast<const uint4*>(ep.skip + t0 + q * 8);
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) skb[j] = j < nvalid ? ep.skip[t0 + j] : __float2bfloat16_rn(0.f);
              }
            } else {
#pragma unroll
              for (int q = 0; q < 4; ++q) skv[q] = make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const float v = __uint_as_float(r[j]) + bias;
              mb[j] = v > 0.f ? 1 : 0;
              ob[j] = __float2bfloat16_rn(to_float(skb[j]) + (v > 0.f ? v : 0.f));
            }
            if (full) {
#pragma unroll
              for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(ep.out + t0 + q * 8) = ov[q];
#pragma unroll
              for (int q = 0; q < 2; ++q) *reinterpret_cast<uint4*>(ep.mask + t0 + q * 16) = mv[q];
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j < nvalid) { ep.out[t0 + j] = ob[j]; ep.mask[t0 + j] = mb[j]; }
            }
          } else if (EPI == TC_EPI_FWD_HEAD) {
            if (full) {
#pragma unroll
              for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4*>(ep.logits + t0 + j) = make_float4(__uint_as_float(r[j]) + bias, __uint_as_float(r[j + 1]) + bias,
                                                                             __uint_as_float(r[j + 2]) + bias, __uint_as_float(r[j + 3]) + bias);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j < nvalid) ep.logits[t0 + j] = __uint_as_float(r[j]) + bias;
            }
          } else {  // TC_EPI_DGRAD
            uint4 skv[4], qv[4], zv[4], mv[2];
            bf16* skb = reinterpret_cast<bf16*>(skv);
            bf16* qb = reinterpret_cast<bf16*>(qv);
            bf16* zb = reinterpret_cast<bf16*>(zv);
            uint8_t* mb = reinterpret_cast<uint8_t*>(mv);
            if (full) {
#pragma unroll
              for (int q = 0; q < 2; ++q) mv[q] = *reinterpret_cast<const uint4*>(ep.mask_prev + t0 + q * 16);
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) mb[j] = j < nvalid ? ep.mask_prev[t0 + j] : 0;
            }
            if (ep.dh_next != nullptr) {
              if (full) {
#pragma unroll
                for (int q = 0; q < 4; ++q) skv[q] = *reinterpret_cast<const uint4*>(ep.dh_next + t0 + q * 8);
              } else {
#pragma unroll
                for (int j = 0; j < 32; ++j) skb[j] = j < nvalid ? ep.dh_next[t0 + j] : __float2bfloat16_rn(0.f);
              }
            } else {
#pragma unroll
              for (int q = 0; q < 4; ++q) skv[q] = make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const bf16 qq = __float2bfloat16_rn(__uint_as_float(r[j]) + to_float(skb[j]));
              qb[j] = qq;
              zb[j] = mb[j] ? qq : __float2bfloat16_rn(0.f);
            }
            if (ep.bias_g != nullptr) {  // masked entries and entries past the minibatch are zero
#pragma unroll
              for (int j = 0; j < 32; ++j) bsum += to_float(zb[j]);
            }
            if (full) {
              if (ep.dh_out != nullptr) {
#pragma unroll
                for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(ep.dh_out + t0 + q * 8) = qv[q];
              }
#pragma unroll
              for (int q = 0; q < 4; ++q) *reinterpret_cast<uint4*>(ep.dz_prev + t0 + q * 8) = zv[q];
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j)
                if (j < nvalid) {
                  if (ep.dh_out != nullptr) ep.dh_out[t0 + j] = qb[j];
                  ep.dz_prev[t0 + j] = zb[j];
                }
            }
          }
        }
      }
      if (tc_epi_is_wgrad(EPI) && ep.partial != nullptr) {
        // fixed order: 32 columns x 8 chunks sequentially per thread, xor-shuffle tree over the 32 rows; the slots are
        // laid out by 128-row block of the output (a CTA of a pair whose rows lie wholly outside the matrix has none)
        const float tot = warp_sum((ssq4[0] + ssq4[1]) + (ssq4[2] + ssq4[3]));
        if (lane == 0 && m_base < M) ep.partial[(int64_t)z * ep.ld_partial + ep.slot0 + ((int64_t)(m_base / kTcBlockM) * n_tiles + nt) * kTcEpiWarps + ew] = tot;
      }
      if (EPI == TC_EPI_DGRAD && ep.bias_g != nullptr) {
        // the two warps of a quadrant hold the sums over their halves of the samples: exchange through shared memory (the
        // staging area is unused in this kernel), first warp adds them in a fixed order, stores db and the sum of squares
        // of each group of 8 (xor-shuffle tree over the 8 lanes)
        float* bsm = reinterpret_cast<float*>(stage) + as * 256;
        bsm[half * 128 + quad * 32 + lane] = bsum;
        __syncwarp();
        if (lane == 0) tc::mbar_arrive(&bias_bar[quad * 2 + as]);
        if (half == 0) {
          if (!tc::mbar_wait(&bias_bar[quad * 2 + as], aph, abort_flag)) { ok = false; break; }
          const float db = bsm[quad * 32 + lane] + bsm[128 + quad * 32 + lane];
          float sq = (m < M) ? db * db : 0.f;
          sq += __shfl_xor_sync(0xffffffffu, sq, 1);
          sq += __shfl_xor_sync(0xffffffffu, sq, 2);
          sq += __shfl_xor_sync(0xffffffffu, sq, 4);
          if (m < M) {
            const int64_t o = (int64_t)z * ep.bias_ld + ep.bias_off + m;
            if (ep.bias_bf16) reinterpret_cast<bf16*>(ep.bias_g)[o] = __float2bfloat16_rn(db);
            else reinterpret_cast<float*>(ep.bias_g)[o] = db;
            if ((lane & 7) == 0 && ep.partial != nullptr) ep.partial[(int64_t)z * ep.ld_partial + ep.bias_slot0 + (m >> 3)] = sq;
          }
        }
      }
      tc::tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) tc::mbar_arrive_cluster(acc_empty_leader[as]);  // the issuing thread lives in the leader CTA
        else tc::mbar_arrive(&acc_empty[as]);
      }
      if (++as == 2) { as = 0; aph ^= 1u; }
      }
    }
    if ((EPI == TC_EPI_WGRAD || EPI == TC_EPI_WGRAD_BF16) && lane == 0) tc::bulk_wait_all<0>();  // every gradient block has reached global memory
    if (!ok && lane == 0) { *abort_flag = 1; atomicOr(status, STATUS_TIMEOUT); }
  }

  // ---------------------------------------------------------------------- teardown
  tc::tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // something gave up: give copies that may still be in flight time to land before shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) { }
    __syncthreads();
  }
  // pair form: neither CTA may leave (or free its tensor memory) while the other can still read its shared memory, write
  // its barriers or has MMAs in flight that fill its tensor memory; every role of both CTAs has ended here (all waits are bounded)
  if (PAIR) tc::cluster_sync_all();
  if (warp == 1) {
    tc::tc_fence_after();
    if (PAIR) tc::tmem_dealloc_pair(tmem_base, TMEM_COLS);
    else tc::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// Self-test of the bounded wait: one thread waits, with the same routine the GEMM roles use, on a barrier that nothing
// will ever complete.  After `limit` polls it gives up, raises STATUS_TIMEOUT and the kernel ends normally.
__global__ void wait_selftest_kernel(uint32_t limit, int* __restrict__ status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  grid_dep_sync();
  if (threadIdx.x == 0) {
    abort_flag = 0;
    tc::mbar_init(&bar, 1);
    tc::fence_barrier_init();
    if (!tc::mbar_wait_limit(&bar, 0u, &abort_flag, limit)) atomicOr(status, STATUS_TIMEOUT);
  }
}

// ------------------------------------------------------------------------------------------------ host side
struct TcLayer { int in, out; int64_t w_pad, b_pad; bool residual; };
struct TcBuffers {
  bf16* xop; float* g; int64_t ld;
  bf16* act[9]; uint8_t* mask[9]; float* logits; bf16* dz[2]; bf16* dh[2]; int* status;
  int ldb;
  float* partial; int64_t ld_partial;  // per-replica slots for the fused sum of squares
  bf16* g1b;                           // [Z, ld] bf16 copy of the ascent gradient
  // fp32 GEMMs on three bf16 planes per operand: xop, act[], dz[] hold three planes each ([3][Z][...], plane-major), g is fp32
  bool split = false;
};

struct TcGemm {
  CUtensorMap map_a, map_b, map_c;  // map_c: fp32 output of wgrad (a copy of map_a elsewhere, unused)
  CUtensorMap map_c16;              // wgrad only: the same output rows in the bf16 ascent-gradient buffer
  int M = 0, N = 0, Kd = 0, block_n = 0;
  TcEpi ep{};
  bool valid = false;
  bool pair = false;  // run by pairs of CTAs (cta_group::2) on 256-row tiles
  bool astat = false; // weight gradient with the A block stationary over runs of n-tiles (ep.run_n)
  bool bstat = false; // weight gradient with the B block stationary over runs of m-tiles (ep.run_n); single CTAs
  bool split = false; // operands stored as three bf16 planes (fp32 GEMM); single CTAs, N tile of at most 128
};

struct TcPlan {
  const int32_t* active = nullptr;  // per-tick mask of the replicas that step (nullptr: all)
  int Z = 0, B = 0, n_layers = 0, sms = 148;
  int* status = nullptr;
  int64_t* launches = nullptr;
  std::vector<TcGemm> fwd, dgrad, wgrad;
  std::vector<int> bias_slot0;  // first partial slot of the bias-gradient blocks of each layer
  int n_slots = 0;              // partial slots used per replica
  bool allow_pair = true;       // false: every GEMM on the single-CTA kernels
  bool force_pair = false;      // true: CTA pairs wherever the kernel supports them (test coverage of every pair instantiation)
  bool allow_astat = true;      // false: the weight gradient walks single tiles
  int max_pairs = 0;            // CTA pairs that can be resident at once (0: not yet asked)
  bool pdl = false;             // launches carry the programmatic-stream-serialization attribute
};

typedef CUresult (*PFN_encodeTiled)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                    const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline PFN_encodeTiled tc_encode_fn() {
  static PFN_encodeTiled fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<PFN_encodeTiled>(p);
  }
  return fn;
}

// bf16 tensor [Z][rows][cols] with element strides (row_stride, z_stride); dim 0 = cols (contiguous).
template <typename T>
inline bool tc_make_map(CUtensorMap* m, const T* base, uint64_t cols, uint64_t rows, uint64_t Z, uint64_t row_stride,
                        uint64_t z_stride, uint32_t box_cols, uint32_t box_rows) {
  PFN_encodeTiled enc = tc_encode_fn();
  if (!enc) return false;
  constexpr uint64_t ES = sizeof(T);
  if ((reinterpret_cast<uintptr_t>(base) & 15) || (row_stride * ES) % 16 || (z_stride * ES) % 16 || box_cols * ES > 128) return false;
  cuuint64_t dims[3] = {cols, rows, Z};
  cuuint64_t strides[2] = {row_stride * ES, z_stride * ES};
  cuuint32_t box[3] = {box_cols, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  return enc(m, sizeof(T) == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<T*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline int tc_pick_block_n(int n, bool split = false) { return (n > 128 && !split) ? 256 : (n > 64 ? 128 : 64); }
// Where the pair form is used: forward and dgrad with a 256-wide minibatch tile (measured at the 4096-wide layers with
// B = 256: 985 -> 1100 and 945 -> 1030 TFLOP/s inside the step), and the weight gradient with 256-wide tiles and a minibatch of at
// most 256 samples, where the pair also keeps its dz blocks in shared memory (tc_plan; 850 -> 980).  It loses with 128-wide
// minibatch tiles (short kernels: 415 -> 405, 360 -> 335), which keep the single-CTA kernels; `force` (tests) pairs whatever can be.
inline bool tc_pick_pair(int M, int block_n, bool wgrad, bool force) { return M >= 256 && (force ? block_n >= 128 : (block_n == 256 && !wgrad)); }
// Partial-sum slots one replica needs when the sum of squares is fused into the weight-gradient epilogue:
// eight per output tile (one per epilogue warp) plus one per 8 bias units.
inline int64_t tc_norm_slots(const lsam_config& c, bool split = false) {
  int64_t n = 0;
  for (int l = 0; l < c.n_layers; ++l) {
    const int in = c.widths[l], out = c.widths[l + 1];
    n += ceil_div(out, kTcBlockM) * ceil_div(in, tc_pick_block_n(in, split)) * kTcEpiWarps + ceil_div(out, 8);
  }
  return n;
}

// The tensor-core path needs every layer's input width to be a multiple of 8 (16-byte row strides of W and of
// the activations); output widths are free (padded strides, TMA zero-fills the ragged edge).
inline bool tc_supported(const lsam_config& c) {
  if (c.n_layers < 1 || c.batch < 1) return false;
  for (int l = 0; l < c.n_layers; ++l)
    if (c.widths[l] % 8 != 0) return false;
  return true;
}

inline int tc_plan(TcPlan& P, const lsam_config& c, const std::vector<TcLayer>& layers, const TcBuffers& b, int64_t* launches,
                   std::string& why) {
  P.Z = c.K; P.B = c.batch; P.n_layers = (int)layers.size(); P.status = b.status; P.launches = launches;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&P.sms, cudaDevAttrMultiProcessorCount, dev);
  const int L = P.n_layers, B = c.batch, Z = c.K;
  const bool sp = b.split;
  const uint64_t ZM = sp ? 3 * (uint64_t)Z : (uint64_t)Z;  // "replicas" of an operand tensor map: plane p of replica z is z + p Z
  if (sp) { P.allow_pair = false; P.allow_astat = false; }
  P.fwd.assign(L, TcGemm()); P.dgrad.assign(L, TcGemm()); P.wgrad.assign(L, TcGemm());
  const uint64_t ldb = (uint64_t)b.ldb;
  P.bias_slot0.assign(L, 0);
  int slot = 0;
  for (int l = 0; l < L; ++l) {
    const TcLayer& ly = layers[l];
    const int cur = (L - 1 - l) & 1;  // dz buffer holding the pre-activation gradient of layer l
    const bf16* W = b.xop + ly.w_pad;
    const bool head = (l == L - 1);
    bool ok = true;
    {  // forward: A = W [out][in] (in contiguous), B = act_l [in][B] (samples contiguous)
      TcGemm& g = P.fwd[l];
      g.M = ly.out; g.N = B; g.Kd = ly.in; g.block_n = tc_pick_block_n(B, sp); g.split = sp;
      // three-plane form: a tile list shorter than the machine is cut into 64-sample tiles (twice as many CTAs, each taking in 3/4 of the bytes)
      if (sp && g.block_n == 128 && (int64_t)Z * ceil_div(g.M, kTcBlockM) * ceil_div(B, 128) < P.sms) g.block_n = 64;
      g.pair = P.allow_pair && tc_pick_pair(g.M, g.block_n, false, P.force_pair);
      ok &= tc_make_map(&g.map_a, W, ly.in, ly.out, ZM, ly.in, b.ld, 64, kTcBlockM);
      ok &= tc_make_map(&g.map_b, b.act[l], B, ly.in, ZM, ldb, (uint64_t)ly.in * ldb, 64, 64);
      g.ep.bias = b.xop + ly.b_pad; g.ep.ld_p = b.ld; g.ep.ldb = b.ldb;
      if (head) g.ep.logits = b.logits;
      else { g.ep.out = b.act[l + 1]; g.ep.skip = ly.residual ? b.act[l] : nullptr; g.ep.mask = b.mask[l]; }
      g.map_c = g.map_a;
      g.valid = ok;
    }
    {  // wgrad: A = dz_l [out][B] (samples contiguous = contraction), B = act_l [in][B]
      TcGemm& g = P.wgrad[l];
      g.M = ly.out; g.N = ly.in; g.Kd = B; g.block_n = tc_pick_block_n(ly.in, sp); g.split = sp;
      g.pair = P.allow_pair && tc_pick_pair(g.M, g.block_n, true, P.force_pair);
      // a minibatch of at most 256 samples (four k-blocks): the dz block stays in shared memory over a run of tiles; with 256-wide
      // tiles a pair of CTAs shares each activation tile on top of that (each CTA takes in half of it)
      const bool astat_ok = P.allow_astat && B <= kTcAstatKBlocks * kTcBlockK;
      if (P.allow_pair && astat_ok && g.M >= 256 && g.block_n == 256) g.pair = true;
      g.astat = astat_ok && (!g.pair || g.block_n >= 128);
      // single CTAs with 256-wide tiles: the activation block (256 rows) is the larger operand, so it is the one to keep in shared
      // memory: a tile then takes in 128 instead of 256 rows (measured inside the step at B = 256, 4096-wide layers: 783-798 -> 823-837
      // TFLOP/s; no gain with two k-blocks, B = 128, where the stores of the tile are what takes the time)
      g.bstat = g.astat && !g.pair && g.block_n == 256 && B > 2 * kTcBlockK;
      if (g.bstat) g.astat = false;
      ok &= tc_make_map(&g.map_a, b.dz[cur], B, ly.out, ZM, ldb, (uint64_t)ly.out * ldb, 64, kTcBlockM);
      ok &= tc_make_map(&g.map_b, b.act[l], B, ly.in, ZM, ldb, (uint64_t)ly.in * ldb, 64, g.pair ? g.block_n / 2 : g.block_n);  // a CTA of a pair loads half the rows
      ok &= tc_make_map(&g.map_c, b.g + ly.w_pad, ly.in, ly.out, Z, ly.in, b.ld, 32, 32);
      // the same rows of the bf16 gradient buffer
      if (!sp) ok &= tc_make_map(&g.map_c16, b.g1b + ly.w_pad, ly.in, ly.out, Z, ly.in, b.ld, 64, 32);
      g.ep.g = b.g; g.ep.ld_g = b.ld; g.ep.w_off = ly.w_pad; g.ep.ldw = ly.in; g.ep.ldb = b.ldb;
      g.ep.partial = b.partial; g.ep.ld_partial = b.ld_partial; g.ep.slot0 = slot;
      g.ep.run_n = 1;
      if (g.bstat) {
        const int64_t cols = (int64_t)Z * ceil_div(g.N, g.block_n), m_tiles = ceil_div(g.M, kTcBlockM);
        double best = 0.0;
        for (int rn = 1; rn <= m_tiles; ++rn) {
          const int64_t units = cols * ceil_div(m_tiles, (int64_t)rn);
          const double cost = (double)ceil_div(units, (int64_t)P.sms) * ((double)rn * kTcBlockM + g.block_n);
          if (rn == 1 || cost < best) { best = cost; g.ep.run_n = rn; }
        }
      }
      if (g.astat) {
        // run length: a unit of the list costs a CTA run_n B tiles (half tiles in a pair) plus one A block of 128 rows; the SMs (pairs of SMs)
        // work through ceil(units / SMs) rounds of units.  Pick the run length with the least bytes through the busiest SM.
        const int64_t rows = (int64_t)Z * ceil_div(g.M, g.pair ? 2 * kTcBlockM : kTcBlockM), n_tiles = ceil_div(g.N, g.block_n);
        const int64_t workers = g.pair ? P.sms / 2 : P.sms;
        const double b_rows = g.pair ? g.block_n / 2 : g.block_n;
        double best = 0.0;
        for (int rn = 1; rn <= n_tiles; ++rn) {
          const int64_t units = rows * ceil_div(n_tiles, (int64_t)rn);
          const double cost = (double)ceil_div(units, workers) * ((double)rn * b_rows + kTcBlockM);
          if (rn == 1 || cost < best) { best = cost; g.ep.run_n = rn; }
        }
      }
      slot += (int)(ceil_div(g.M, kTcBlockM) * ceil_div(g.N, g.block_n) * kTcEpiWarps);
      P.bias_slot0[l] = slot;
      slot += (int)ceil_div(ly.out, 8);
      g.valid = ok;
    }
    if (l > 0) {  // dgrad: A = W [out][in] read as (m = in contiguous, kd = out), B = dz_l [out][B] (samples contiguous)
      TcGemm& g = P.dgrad[l];
      g.M = ly.in; g.N = B; g.Kd = ly.out; g.block_n = tc_pick_block_n(B, sp); g.split = sp;
      g.pair = P.allow_pair && tc_pick_pair(g.M, g.block_n, false, P.force_pair);
      ok &= tc_make_map(&g.map_a, W, ly.in, ly.out, ZM, ly.in, b.ld, 64, 64);
      ok &= tc_make_map(&g.map_b, b.dz[cur], B, ly.out, ZM, ldb, (uint64_t)ly.out * ldb, 64, 64);
      g.ep.dh_next = ly.residual ? b.dh[(l + 1) & 1] : nullptr;
      g.ep.dh_out = layers[l - 1].residual ? b.dh[l & 1] : nullptr;
      g.ep.dz_prev = b.dz[cur ^ 1]; g.ep.mask_prev = b.mask[l - 1]; g.ep.ldb = b.ldb;
      g.ep.bias_g = nullptr; g.ep.bias_ld = b.ld; g.ep.bias_off = layers[l - 1].b_pad;
      g.ep.partial = b.partial; g.ep.ld_partial = b.ld_partial; g.ep.bias_slot0 = P.bias_slot0[l - 1];
      g.map_c = g.map_a;
      g.valid = ok;
    }
    if (!ok) { why = "tensor map creation failed"; return 1; }
  }
  P.n_slots = slot;
  return 0;
}

template <int BLOCK_N, bool A_MN, bool B_MN, int EPI, bool PAIR, bool ASTAT = false, bool SPLIT = false, bool BSTAT = false>
inline int tc_launch_one(TcPlan& P, const TcGemm& g, cudaStream_t stream) {
  auto kern = gemm_tcgen05_kernel<BLOCK_N, A_MN, B_MN, EPI, PAIR, ASTAT, SPLIT, BSTAT>;
  constexpr int smem = tc_smem_bytes<BLOCK_N, PAIR, ASTAT, SPLIT, BSTAT>();
  // the shared-memory limit of a kernel is a per-device attribute: remember it per device ordinal
  static bool attr_set[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
  if (!attr_set[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return 1;
    attr_set[dev] = true;
  }
  const int tile_m = PAIR ? 2 * kTcBlockM : kTcBlockM;
  const int64_t n_tiles = ceil_div(g.N, BLOCK_N);
  const int64_t rn = g.ep.run_n > 0 ? g.ep.run_n : 1;
  const int64_t tiles = BSTAT ? (int64_t)P.Z * n_tiles * ceil_div(ceil_div(g.M, tile_m), rn)
                              : (int64_t)P.Z * ceil_div(g.M, tile_m) * (ASTAT ? ceil_div(n_tiles, rn) : n_tiles);  // units of the work list
  // one persistent CTA per SM, or one persistent pair of CTAs (a cluster of two) per pair of SMs
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[2];
  unsigned na = 0;
  if (PAIR) {
    attr[na].id = cudaLaunchAttributeClusterDimension;
    attr[na].val.clusterDim.x = 2; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
    ++na;
  }
  cfg.blockDim = dim3(kTcThreads); cfg.dynamicSmemBytes = smem; cfg.stream = stream; cfg.attrs = attr; cfg.numAttrs = na;
  if (PAIR && P.max_pairs == 0) {
    cfg.gridDim = dim3((unsigned)(P.sms / 2 * 2));
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n < 1) return 1;
    P.max_pairs = n < P.sms / 2 ? n : P.sms / 2;
  }
  if (P.pdl) {
    attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[na].val.programmaticStreamSerializationAllowed = 1;
    cfg.numAttrs = ++na;
  }
  if (PAIR) {
    const int pairs = (int)(tiles < P.max_pairs ? tiles : P.max_pairs);
    cfg.gridDim = dim3((unsigned)(2 * pairs));
  } else {
    cfg.gridDim = dim3((unsigned)(tiles < P.sms ? tiles : P.sms));
  }
  int M = g.M, N = g.N, Kd = g.Kd, Z = P.Z;
  int* status = P.status;
  const int32_t* active = P.active;
  void* args[] = {(void*)&g.map_a, (void*)&g.map_b, (void*)&g.map_c, &M, &N, &Kd, &Z, (void*)&g.ep, &status, &active};
  return cudaLaunchKernelExC(&cfg, (const void*)kern, args) == cudaSuccess ? 0 : 1;
}

template <bool A_MN, bool B_MN, int EPI>
inline int tc_launch(TcPlan& P, const TcGemm& g, cudaStream_t stream) {
  if (!g.valid) return 1;
  if constexpr (EPI <= TC_EPI_WGRAD) {
    if (g.split) {
      if (g.block_n > 128 || g.pair || g.astat) return 1;
      return g.block_n == 128 ? tc_launch_one<128, A_MN, B_MN, EPI, false, false, true>(P, g, stream)
                              : tc_launch_one<64, A_MN, B_MN, EPI, false, false, true>(P, g, stream);
    }
  }
  if (g.split) return 1;
  if (g.pair) {
    if constexpr (tc_epi_is_wgrad(EPI) && !A_MN && !B_MN) {
      if (g.astat) {
        switch (g.block_n) {
          case 256: return tc_launch_one<256, A_MN, B_MN, EPI, true, true>(P, g, stream);
          default: return tc_launch_one<128, A_MN, B_MN, EPI, true, true>(P, g, stream);
        }
      }
    }
    switch (g.block_n) {
      case 256: return tc_launch_one<256, A_MN, B_MN, EPI, true>(P, g, stream);
      default: return tc_launch_one<128, A_MN, B_MN, EPI, true>(P, g, stream);
    }
  }
  if constexpr (tc_epi_is_wgrad(EPI) && !A_MN && !B_MN) {
    if (g.bstat && g.block_n == 256) return tc_launch_one<256, A_MN, B_MN, EPI, false, false, false, true>(P, g, stream);
    if (g.astat) {
      switch (g.block_n) {
        case 256: return tc_launch_one<256, A_MN, B_MN, EPI, false, true>(P, g, stream);
        case 128: return tc_launch_one<128, A_MN, B_MN, EPI, false, true>(P, g, stream);
        default: return tc_launch_one<64, A_MN, B_MN, EPI, false, true>(P, g, stream);
      }
    }
  }
  switch (g.block_n) {
    case 256: return tc_launch_one<256, A_MN, B_MN, EPI, false>(P, g, stream);
    case 128: return tc_launch_one<128, A_MN, B_MN, EPI, false>(P, g, stream);
    default: return tc_launch_one<64, A_MN, B_MN, EPI, false>(P, g, stream);
  }
}

inline int tc_forward(TcPlan& P, int l, cudaStream_t stream) {
  return (l == P.n_layers - 1) ? tc_launch<false, true, TC_EPI_FWD_HEAD>(P, P.fwd[l], stream)
                               : tc_launch<false, true, TC_EPI_FWD_HIDDEN>(P, P.fwd[l], stream);
}
inline int tc_wgrad(TcPlan& P, int l, cudaStream_t stream, bool out_bf16) {
  if (!out_bf16) return tc_launch<false, false, TC_EPI_WGRAD>(P, P.wgrad[l], stream);
  TcGemm g = P.wgrad[l];
  g.map_c = g.map_c16;
  return tc_launch<false, false, TC_EPI_WGRAD_BF16>(P, g, stream);
}
// Descent-pass weight gradient of layer l with the worker update applied to the layer's weights in the epilogue.
struct TcFusedUpdate {
  float* x; float* v; const float* yring; const int32_t* slot; bf16* xop; const float* lam_k;
  float eta, mu, lambda; int nesterov;
};
inline int tc_wgrad_update(TcPlan& P, int l, cudaStream_t stream, const TcFusedUpdate& u) {
  TcGemm g = P.wgrad[l];
  g.ep.upd_x = u.x; g.ep.upd_v = u.v; g.ep.upd_yring = u.yring; g.ep.upd_slot = u.slot; g.ep.upd_xop = u.xop; g.ep.upd_lam_k = u.lam_k;
  g.ep.upd_eta = u.eta; g.ep.upd_mu = u.mu; g.ep.upd_lambda = u.lambda; g.ep.upd_nesterov = u.nesterov;
  return tc_launch<false, false, TC_EPI_WGRAD_UPD>(P, g, stream);
}
// The dgrad of layer l can also deliver the bias gradient of layer l - 1 (row sums of the backward signal it writes) when the
// whole minibatch sits in one N tile; bias_g = destination buffer ([Z, ld] gradient rows, bf16 or fp32), nullptr = not fused.
inline bool tc_dgrad_can_fuse_bias(const TcPlan& P, int l) { return l > 0 && P.dgrad[l].valid && P.dgrad[l].N <= P.dgrad[l].block_n; }
inline int tc_dgrad(TcPlan& P, int l, cudaStream_t stream, void* bias_g = nullptr, bool bias_bf16 = false) {
  if (bias_g == nullptr) return tc_launch<true, true, TC_EPI_DGRAD>(P, P.dgrad[l], stream);
  TcGemm g = P.dgrad[l];
  g.ep.bias_g = bias_g; g.ep.bias_bf16 = bias_bf16 ? 1 : 0;
  return tc_launch<true, true, TC_EPI_DGRAD>(P, g, stream);
}

}  // namespace lsam
