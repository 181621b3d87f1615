// lsam_api.cu -- host side of the C ABI declared in include/lsam.h: configuration checks, workspace layout,
// and the launch sequence of one worker tick (schedule -> gather -> ascent gradient -> norm -> perturb ->
// descent gradient -> fused update) and of the centre update.  No device memory is allocated here: every
// buffer is carved from the caller's workspace.
#include "lsam.h"

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <string>
#include <utility>
#include <vector>

#include <nvtx3/nvToolsExt.h>

#include "common.cuh"
#include "model_kernels.cuh"
#include "stream_kernels.cuh"
#include "gemm_tcgen05.cuh"

using namespace lsam;

namespace {

struct LayerInfo {
  int in, out;           // shape of the weight matrix [out, in] (a convolution: [Cout, Cin * 9])
  int64_t w_unp, b_unp;  // offsets in the unpadded vector
  int64_t w_pad, b_pad;  // offsets in the padded row
  bool residual;
  // convolution layer (3x3, stride 1, padding 1, ReLU, 2x2 max-pooling) on H x W feature maps
  bool conv = false;
  int Cin = 0, Cout = 0, H = 0, W = 0;
  int wg_parts = 1, wg_chunk = 0;     // convolution: the weight gradient's contraction (one term per position and sample) is split over blocks
  int fw_parts = 1, fw_chunk = 0;     // dense layer of the convolutional model with few tiles and a long contraction: forward split over blocks
  int64_t feat_in = 0, feat_out = 0;  // features per sample entering / leaving the layer (dense: in / out)
};

struct Layout {
  bool ok = false;
  int64_t d = 0, ld = 0;
  std::vector<LayerInfo> layers;
  int ldb = 0;  // sample stride of the feature-major activation-like buffers [K, width, ldb] (multiple of 16)
  int in0 = 0;  // features of one minibatch row (widths[0]; convolutional model: C0 * H * W)
  SegMap seg{};
  int ring = 2;
  int64_t nchunks = 0;
  bool vec4 = true;
  // byte offsets into the workspace
  size_t x, v, g, g1b, g1keep, xpkeep, xop, acc, yring, gprev, tmp, idx, ylab, sched, partial, scalars, status, gbar1, gbar2;
  size_t act[9], mask[9], logits, rowloss, dz[2], dh[2], xstage, ystage, xstage2, ystage2;
  // fp32 GEMMs on the bf16 tensor cores (LSAM_GEMM_FP32 with LSAM_IMPL_TCGEN05): the parameters the next gradient pass reads,
  // activations and backward signals are stored as three bf16 planes each; xpl = planes of the parameters [3][K][ld]
  bool x3 = false;
  size_t xpl = 0;
  size_t hpart = 0;  // narrow head: partial logits [K, chunks, kHeadMaxOut, ldb]
  size_t col[9], parg[9], zout, dzc, dcol, wpart;  // convolutional model: patch matrices, pooling choices, pre-pooling output, its gradient, patch-matrix gradient
  size_t total = 0;
};

constexpr int64_t kSegAlign = 64;

bool plan(const lsam_config& c, Layout& L) {
  L = Layout();
  if (c.K < 1 || c.K > 4096 || c.tau < 1 || c.stale_max < 0 || c.stale_max > 15) return false;
  if (c.gemm_dtype != LSAM_GEMM_FP32 && c.gemm_dtype != LSAM_GEMM_BF16) return false;
  if (c.gemm_impl < LSAM_IMPL_AUTO || c.gemm_impl > LSAM_IMPL_TCGEN05_PAIRS) return false;
  if (!(c.gamma > 0.f)) return false;
  if (c.active_num < 0 || c.active_num > 256) return false;
  if (!(c.noise_temp >= 0.f)) return false;
  if (c.kernel_kind < KERNEL_GAUSSIAN || c.kernel_kind > KERNEL_MATERN32) return false;
  if (c.kernel_kind == KERNEL_EXP_POWER && !(c.kernel_param >= 1.f && c.kernel_param <= 2.f)) return false;
  if (c.kernel_kind == KERNEL_CAUCHY && !(c.kernel_param > 0.f)) return false;
  // synchronous gradient averaging: every worker steps at every tick, and all workers of the job live in this context
  if (c.dp_average != 0 && ((c.active_num != 0 && c.active_num != 256) || c.K_total != 0)) return false;
  if (c.K_total != 0) {  // a shard of a larger job: lock-step schedule only
    if (c.k_offset < 0 || c.K_total < c.K || c.k_offset > c.K_total - c.K) return false;
    if (c.active_num != 0 && c.active_num != 256) return false;
  } else if (c.k_offset != 0) {
    return false;
  }
  const bool bf = c.gemm_dtype == LSAM_GEMM_BF16;
  // fp32 MLP on the tensor cores (three bf16 planes per operand): on request, or by AUTO where the shapes are supported and a layer is
  // large enough for the tensor-core kernels to win (measured at 784-1024-10, K = 8, B = 128: 0.365 -> 0.238 ms per step)
  L.x3 = false;
  if (!bf && (c.model == LSAM_MODEL_MLP || c.model == LSAM_MODEL_RESMLP) && c.n_layers >= 1 && c.n_layers <= 8 && c.batch >= 1) {
    int64_t macs = 0;
    for (int l = 0; l < c.n_layers; ++l) macs = std::max<int64_t>(macs, (int64_t)c.K * c.batch * c.widths[l] * c.widths[l + 1]);
    L.x3 = c.gemm_impl == LSAM_IMPL_TCGEN05 || (c.gemm_impl == LSAM_IMPL_AUTO && tc_supported(c) && macs >= ((int64_t)1 << 27));
  }
  L.seg.n = 0;
  if (c.model == LSAM_MODEL_FLAT) {
    if (c.flat_d < 1 || bf) return false;
    L.d = c.flat_d;
    L.ld = round_up(L.d, 4);
    L.vec4 = (L.d % 4 == 0);
    L.seg.n = 1;
    L.seg.src[0] = 0; L.seg.dst[0] = 0; L.seg.len[0] = L.d;
  } else if (c.model == LSAM_MODEL_LSQ) {
    if (c.widths[0] < 1 || c.batch < 1 || c.n_samples < 1 || bf) return false;
    L.d = c.widths[0];
    L.in0 = c.widths[0];
    L.ld = round_up(L.d, kSegAlign);
    L.layers.push_back({c.widths[0], 1, 0, -1, 0, -1, false});
    L.seg.n = 1;
    L.seg.src[0] = 0; L.seg.dst[0] = 0; L.seg.len[0] = L.d;
  } else if (c.model == LSAM_MODEL_MLP || c.model == LSAM_MODEL_RESMLP || c.model == LSAM_MODEL_CNN) {
    if (c.n_layers < 1 || c.n_layers > 8 || c.batch < 1 || c.n_samples < 1) return false;
    const bool cnn = c.model == LSAM_MODEL_CNN;
    // convolutional model: positions are indexed (y, x, sample) with the sample fastest, so the minibatch must fill its stride
    if (cnn && (c.n_conv < 1 || c.n_conv >= c.n_layers || c.img_h < 1 || c.img_w < 1 || c.img_h % (1 << c.n_conv) || c.img_w % (1 << c.n_conv) || c.batch % 16)) return false;
    if (cnn && (int64_t)c.img_h * c.img_w * c.batch >= ((int64_t)1 << 31)) return false;  // the helper kernels index positions with 32 bits
    int64_t unp = 0, pad = 0;
    int H = c.img_h, W = c.img_w;
    for (int l = 0; l < c.n_layers; ++l) {
      LayerInfo li;
      if (c.widths[l] < 1 || c.widths[l + 1] < 1) return false;
      if (cnn && l < c.n_conv) {
        li.conv = true;
        li.Cin = c.widths[l]; li.Cout = c.widths[l + 1]; li.H = H; li.W = W;
        li.in = li.Cin * 9; li.out = li.Cout;
        li.feat_in = (int64_t)li.Cin * H * W;
        H /= 2; W /= 2;
        li.feat_out = (int64_t)li.Cout * H * W;
      } else {
        li.in = (cnn && l == c.n_conv) ? (int)L.layers.back().feat_out : c.widths[l];  // the first dense layer takes the flattened feature maps
        li.out = c.widths[l + 1];
        li.feat_in = li.in; li.feat_out = li.out;
      }
      li.w_unp = unp; unp += (int64_t)li.in * li.out;
      li.b_unp = unp; unp += li.out;
      li.w_pad = pad; pad = round_up(pad + (int64_t)li.in * li.out, kSegAlign);
      li.b_pad = pad; pad = round_up(pad + li.out, kSegAlign);
      li.residual = (c.model == LSAM_MODEL_RESMLP) && (l < c.n_layers - 1) && (li.in == li.out);
      L.layers.push_back(li);
      L.seg.src[L.seg.n] = li.w_unp; L.seg.dst[L.seg.n] = li.w_pad; L.seg.len[L.seg.n] = (int64_t)li.in * li.out; ++L.seg.n;
      L.seg.src[L.seg.n] = li.b_unp; L.seg.dst[L.seg.n] = li.b_pad; L.seg.len[L.seg.n] = li.out; ++L.seg.n;
    }
    L.in0 = (int)L.layers[0].feat_in;
    L.ldb = (int)round_up(c.batch, 16);
    L.d = unp;
    L.ld = pad;
  } else {
    return false;
  }
  L.ring = c.stale_max + 2;
  // partial-sum slots per replica; FLAT may fall back to scalar chunks when the caller's gradient buffers are misaligned
  L.nchunks = ceil_div(L.ld, (c.model == LSAM_MODEL_FLAT) ? norm_chunk<1>() : norm_chunk<4>());
  if (c.model == LSAM_MODEL_MLP || c.model == LSAM_MODEL_RESMLP) {  // room for the slots of the fused tensor-core norm (the convolutional model runs on the SIMT GEMMs)
    const int64_t slots = tc_norm_slots(c, L.x3);
    L.nchunks = slots > L.nchunks ? slots : L.nchunks;
  }

  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = (size_t)round_up((int64_t)(off + bytes), 256); return o; };
  const size_t K = c.K, ld = L.ld, B = c.batch > 0 ? c.batch : 1;
  const size_t esz = bf ? 2 : 4;
  const size_t asz = L.x3 ? 6 : esz;  // activation-like operands: three bf16 planes in the x3 form
  const bool flat = c.model == LSAM_MODEL_FLAT;
  L.status = take(256);
  L.scalars = take(sizeof(float) * 8 * K);  // norm1, norm2, scale, loss (4 x [K], padded)
  L.x = take(4 * K * ld);
  L.v = take(4 * K * ld);
  L.g = flat ? 0 : take(4 * K * ld);
  // tensor-core path: the ascent gradient is kept in bf16 (it only feeds the perturbation, itself rounded to bf16)
  L.g1b = (!flat && bf && c.model != LSAM_MODEL_LSQ) ? take(2 * K * ld) : 0;
  L.g1keep = (!flat && (c.flags & LSAM_FLAG_KEEP_G1)) ? take(4 * K * ld) : 0;
  L.xpkeep = (!flat && bf && (c.flags & LSAM_FLAG_KEEP_G1)) ? take(esz * K * ld) : 0;  // x~ survives the update
  L.xop = take(esz * K * ld);  // fp32: perturbed point x~;  bf16: operand copy of x, overwritten by x~
  L.xpl = L.x3 ? take(6 * K * ld) : 0;
  L.acc = take(4 * ld);
  L.yring = take(4 * (size_t)L.ring * ld);
  L.gprev = take(4 * ld);
  L.tmp = take(4 * ld);
  L.gbar1 = c.dp_average ? take(4 * ld) : 0;  // worker-averaged gradients of the two passes
  L.gbar2 = c.dp_average ? take(4 * ld) : 0;
  L.idx = take(4 * K * B * 2);     // step indices + scratch for lsam_read_schedule
  L.sched = take(4 * K * 8);       // stale, ver, slot + scratch copies
  L.partial = take(4 * K * (size_t)L.nchunks);
  L.ylab = take(4 * K * B);
  for (int i = 0; i < 9; ++i) L.act[i] = L.mask[i] = 0;
  L.logits = L.rowloss = L.dz[0] = L.dz[1] = L.dh[0] = L.dh[1] = L.xstage = L.ystage = L.xstage2 = L.ystage2 = 0;
  for (int i = 0; i < 9; ++i) L.col[i] = L.parg[i] = 0;
  L.zout = L.dzc = L.dcol = L.wpart = 0;
  if (!flat) {
    const size_t in0 = L.in0;
    const size_t ldb = L.ldb;
    // least squares keeps its minibatch sample-major [K, B, in]; the classifiers store everything feature-major [K, width, ldb]
    L.act[0] = (c.model == LSAM_MODEL_LSQ) ? take(4 * K * B * in0) : take(asz * K * in0 * ldb);
    L.xstage = take(4 * K * B * in0);
    L.ystage = take(4 * K * B);
    L.xstage2 = take(4 * K * B * in0);  // second slot of the prefetch queue (lsam_stage_batch)
    L.ystage2 = take(4 * K * B);
    if (c.model != LSAM_MODEL_LSQ) {
      size_t maxw = 0, max_full = 0, max_dcol = 0, max_part = 0;
      for (size_t l = 0; l < L.layers.size(); ++l) {
        LayerInfo& li = L.layers[l];
        const size_t w = (size_t)li.feat_out;
        maxw = w > maxw ? w : maxw;
        if (l + 1 < L.layers.size()) {
          L.act[l + 1] = take(asz * K * w * ldb);
          // ReLU mask: at the resolution before pooling for a convolution
          L.mask[l] = take(K * (li.conv ? (size_t)li.Cout * li.H * li.W : w) * ldb);
        }
        if (li.conv) {
          const size_t P = (size_t)li.H * li.W * ldb;
          L.col[l] = take(esz * K * (size_t)li.in * P);
          L.parg[l] = take(K * w * ldb);
          max_full = std::max(max_full, (size_t)li.Cout * P);
          if (l > 0) max_dcol = std::max(max_dcol, (size_t)li.in * P);
          // weight gradient [Cout, 9 Cin] with P terms per element: enough parts of the contraction for two blocks per SM,
          // each part at least 8 slabs long and a multiple of the slab
          const int64_t tiles = ceil_div(li.Cout, kSimtBM) * ceil_div(li.in, kSimtBN) * (int64_t)K;
          int64_t parts = std::max<int64_t>(1, std::min<int64_t>(ceil_div(2 * 148, tiles), (int64_t)P / (8 * kSimtBK)));
          const int64_t chunk = round_up(ceil_div((int64_t)P, parts), kSimtBK);
          parts = ceil_div((int64_t)P, chunk);
          li.wg_parts = (int)parts; li.wg_chunk = (int)chunk;
          if (parts > 1) max_part = std::max(max_part, (size_t)parts * li.Cout * li.in);
        } else if (c.model == LSAM_MODEL_CNN && l + 1 < L.layers.size()) {
          // dense hidden layer behind the convolutions (flattened feature maps in, a few hundred units out): a handful of tiles walking
          // thousands of inputs; split the inputs over blocks the same way
          const int64_t tiles = ceil_div((int64_t)B, kSimtBM) * ceil_div(li.out, kSimtBN) * (int64_t)K;
          int64_t parts = std::max<int64_t>(1, std::min<int64_t>(ceil_div(2 * 148, tiles), (int64_t)li.in / (8 * kSimtBK)));
          const int64_t chunk = round_up(ceil_div((int64_t)li.in, parts), kSimtBK);
          parts = ceil_div((int64_t)li.in, chunk);
          li.fw_parts = (int)parts; li.fw_chunk = (int)chunk;
          if (parts > 1) max_part = std::max(max_part, (size_t)parts * B * li.out);
        }
      }
      if (max_full) { L.zout = take(esz * K * max_full); L.dzc = take(esz * K * max_full); }
      if (max_dcol) L.dcol = take(esz * K * max_dcol);
      if (max_part) L.wpart = take(4 * K * max_part);
      L.logits = take(4 * K * (size_t)L.layers.back().out * ldb);
      if (L.layers.back().out <= kHeadMaxOut) L.hpart = take(4 * K * (size_t)ceil_div(L.layers.back().in, kHeadChunkIn) * kHeadMaxOut * ldb);
      L.rowloss = take(4 * K * B);
      for (int i = 0; i < 2; ++i) L.dz[i] = take(asz * K * maxw * ldb);
      for (int i = 0; i < 2; ++i) L.dh[i] = take(asz * K * maxw * ldb);
    }
  }
  L.total = off;
  L.ok = true;
  return true;
}

struct Profiler {
  bool on = false;
  std::vector<cudaEvent_t> pool;
  std::vector<int> cls;  // class of record i (events 2i, 2i+1)
  size_t used = 0;
};

}  // namespace

struct lsam_ctx {
  lsam_config cfg;
  Layout L;
  char* ws = nullptr;
  cudaStream_t stream = nullptr;
  const float* X = nullptr;
  const uint32_t* Y = nullptr;
  const float* eg1 = nullptr;
  const float* eg2 = nullptr;
  bool ext_vec4 = true;
  int64_t t = 0, t_y = 0;
  std::vector<int64_t> t_x;
  // centre version that was current when step s started, for the steps ver_lo <= s < ver_hi, kept in a ring keyed by
  // s mod kVerRing (a tick reads at most the last 16 of them)
  int ver_ring[32] = {};
  int64_t ver_lo = 0, ver_hi = 0;
  int device = 0;                     // ordinal of the GPU that holds the workspace
  bool grads_bf16 = false;            // tensor-core path with its gradients stored in bf16
  bool fused_update = false;          // LSAM_FLAG_FUSED_UPDATE: weights updated inside the descent-pass weight-gradient epilogue
  bool pdl = false;                   // LSAM_FLAG_PDL: kernels launched with programmatic stream serialization
  bool have_prev = false;
  bool use_tc = false;
  bool async_on = false;              // 0 < active_num < 256: unequal worker progress
  std::vector<int32_t> active_host;   // host mirror of the last tick's mask (drives the counters t_x)
  int64_t launches = 0;
  Profiler prof;
  // CUDA-graph replay of the step (LSAM_FLAG_CUDA_GRAPH): one executable graph per launch sequence
  struct GraphSlot {
    bool warm = false;
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    cudaGraphNode_t n_sched = nullptr, n_fin = nullptr, n_upd = nullptr;
    int64_t launches = 0;
  } graphs[4];
  void* upd_func = nullptr;  // the update_kernel instantiation this context launches
  // prefetch queue of caller-supplied minibatches (lsam_stage_batch / lsam_step_staged): two slots, own copy stream
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t staged_done[2] = {nullptr, nullptr}, slot_free[2] = {nullptr, nullptr};
  bool slot_used[2] = {false, false};
  int stage_head = 0, stage_count = 0;
  std::string err;
  TcPlan tc;

  template <typename T> T* at(size_t off) const { return reinterpret_cast<T*>(ws + off); }
  float* x() const { return at<float>(L.x); }
  float* v() const { return at<float>(L.v); }
  float* g() const { return at<float>(L.g); }
  float* norm1() const { return at<float>(L.scalars); }
  float* norm2() const { return at<float>(L.scalars) + cfg.K; }
  float* scale() const { return at<float>(L.scalars) + 2 * cfg.K; }
  float* loss() const { return at<float>(L.scalars) + 3 * cfg.K; }
  float* pull_weight() const { return at<float>(L.scalars) + 5 * cfg.K; }  // [K] w(||x_k - y||) of a non-Gaussian kernel
  int* status() const { return at<int>(L.status); }
  int32_t* idx() const { return at<int32_t>(L.idx); }
  int32_t* idx_scratch() const { return at<int32_t>(L.idx) + (size_t)cfg.K * (cfg.batch > 0 ? cfg.batch : 1); }
  int32_t* stale() const { return at<int32_t>(L.sched); }
  int32_t* ver() const { return at<int32_t>(L.sched) + cfg.K; }
  int32_t* slot() const { return at<int32_t>(L.sched) + 2 * cfg.K; }
  int32_t* active_buf() const { return at<int32_t>(L.sched) + 3 * cfg.K; }
  // per-tick mask of the workers that step; nullptr in lock-step mode (every worker steps every tick)
  const int32_t* act() const { return async_on ? active_buf() : nullptr; }
  int32_t* sched_scratch() const { return at<int32_t>(L.sched) + 4 * cfg.K; }
  // x3 form: distance between the planes of the gathered minibatch [K, in0, ldb]
  int64_t in_plane() const { return L.x3 ? (int64_t)cfg.K * L.in0 * L.ldb : 0; }
  float* yslot(int64_t version) const { return at<float>(L.yring) + (size_t)(version % L.ring) * L.ld; }

  int fail(int code, const std::string& m) { err = m; return code; }
  // version current when step s started, -1 when it is not (or no longer) on record
  int ver_of_step(int64_t s) const { return (s >= ver_lo && s < ver_hi) ? ver_ring[s & 31] : -1; }
  // the calls that touch the GPU want the context's device to be the current one
  int check_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return fail(LSAM_ERR_CUDA, "cudaGetDevice failed");
    if (dev != device) return fail(LSAM_ERR_INVALID, "the context lives on device " + std::to_string(device) + " but device " + std::to_string(dev) + " is current");
    return LSAM_OK;
  }
  int64_t budget() const {  // iterations still missing to n tau (Algorithm 2, sync trigger)
    int64_t done = 0;
    for (int64_t v : t_x) done += v;
    return (int64_t)cfg.K * cfg.tau - done;
  }
};

namespace {

#define LSAM_CUDA(ctx, call)                                                                          \
  do {                                                                                                \
    cudaError_t e__ = (call);                                                                         \
    if (e__ != cudaSuccess)                                                                           \
      return (ctx)->fail(LSAM_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e__));         \
  } while (0)

int prof_begin(lsam_ctx* c, int cls) {
  c->launches += 1;
  if (!c->prof.on) return LSAM_OK;
  Profiler& p = c->prof;
  while (p.pool.size() < 2 * (p.used + 1)) {
    cudaEvent_t e;
    LSAM_CUDA(c, cudaEventCreate(&e));
    p.pool.push_back(e);
  }
  if (p.cls.size() <= p.used) p.cls.resize(p.used + 1);
  p.cls[p.used] = cls;
  LSAM_CUDA(c, cudaEventRecord(p.pool[2 * p.used], c->stream));
  return LSAM_OK;
}
int prof_end(lsam_ctx* c) {
  LSAM_CUDA(c, cudaPeekAtLastError());
  if (!c->prof.on) return LSAM_OK;
  Profiler& p = c->prof;
  LSAM_CUDA(c, cudaEventRecord(p.pool[2 * p.used + 1], c->stream));
  p.used += 1;
  return LSAM_OK;
}
// LAUNCH(ctx, class, kernel<<<...>>>(...));
#define LAUNCH(ctx, cls, ...)                                  \
  do {                                                         \
    int rc__ = prof_begin((ctx), (cls));                       \
    if (rc__ != LSAM_OK) return rc__;                          \
    __VA_ARGS__;                                               \
    rc__ = prof_end((ctx));                                    \
    if (rc__ != LSAM_OK) return rc__;                          \
  } while (0)

// One kernel launch on the context's stream.  With LSAM_FLAG_PDL a launch may carry the programmatic-stream-serialization
// attribute: the blocks of the kernel may become resident while the kernel before it in the stream is still draining; every
// kernel of the library waits for its predecessors (grid_dep_sync) before its first global access, so the results are those
// of a plain in-order stream.  Which launches take it is a measured choice: the tensor-core GEMMs always (their set-up of
// barriers, tensor memory and tensor maps then overlaps the tail of the kernel before); the other kernels only in a context
// without tensor-core GEMMs and only with grids of at most kPdlMaxBlocks blocks (a least-squares tick of 26.5 us took 22.3 us),
// because beside tensor-core kernels they ran slower with it (perturb8_kernel at 58000 blocks took twice its time, the small
// kernels of a 784-1024-10 MLP cost 2-9 us more per tick).  A failed launch is picked up by prof_end (cudaPeekAtLastError).
constexpr int64_t kPdlMaxBlocks = 1024;
inline void launch_attrs(const lsam_ctx* c, cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, dim3 grid, dim3 block, size_t smem) {
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = c->stream;
  cfg.attrs = attr; cfg.numAttrs = (c->pdl && (int64_t)grid.x * grid.y * grid.z <= kPdlMaxBlocks) ? 1u : 0u;
}
template <typename... KArgs, typename... Args>
inline void launch_k(lsam_ctx* c, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  launch_attrs(c, cfg, attr, grid, block, smem);
  cudaLaunchKernelEx(&cfg, kern, std::forward<Args>(args)...);
}
// The same for a kernel whose arguments sit in a block of pointers (the kernels of a replayed graph whose arguments change per tick).
inline cudaError_t launch_p(lsam_ctx* c, const void* kern, dim3 grid, dim3 block, void** ptrs) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  launch_attrs(c, cfg, attr, grid, block, 0);
  return cudaLaunchKernelExC(&cfg, kern, ptrs);
}

// Argument blocks of the three kernels whose parameters change from step to step (tick, centre-version history,
// budget, rho, eta, noise scale).  They are launched through cudaLaunchKernel from these blocks, so that a captured
// graph can be replayed with cudaGraphExecKernelNodeSetParams on the same blocks.
struct SchedArgs {
  uint64_t seed, t; int64_t n_samples; int B, stale_max; VerHist hist; int ring;
  int32_t *idx, *stale, *ver, *slot; int K, active_num; int64_t budget; int32_t* active; int k_offset;
  void* ptrs[16];
  void bind() {
    void* p[16] = {&seed, &t, &n_samples, &B, &stale_max, &hist, &ring, &idx, &stale, &ver, &slot, &K, &active_num, &budget, &active, &k_offset};
    for (int i = 0; i < 16; ++i) ptrs[i] = p[i];
  }
};
struct FinArgs {
  const float* partial; int64_t nchunks, nused; float rho, gamma; float *norm_out, *scale_out; int* status; const int32_t* active;
  void* ptrs[9];
  void bind() {
    void* p[9] = {&partial, &nchunks, &nused, &rho, &gamma, &norm_out, &scale_out, &status, &active};
    for (int i = 0; i < 9; ++i) ptrs[i] = p[i];
  }
};

// ---- norm of [K, n] rows -> norm_out[K] (and scale[K] = rho / (norm + gamma) if scale_out)
// fused_ok = false: reduce the rows of g even on the tensor-core path (g is not what the weight-gradient epilogues just summed)
int launch_norm(lsam_ctx* c, const float* g, int64_t ldg, int64_t n, bool vec4, float rho, float* norm_out, float* scale_out, bool fused_ok = true) {
  float* partial = c->at<float>(c->L.partial);
  const int64_t nch = c->L.nchunks;
  if (c->use_tc && fused_ok) {
    // tensor-core path: the weight- and bias-gradient kernels of the pass just run have left the sums of squares of
    // all their blocks in the partial slots; only the fixed-order final sum remains
    FinArgs f{partial, nch, (int64_t)c->tc.n_slots, rho, c->cfg.gamma, norm_out, scale_out, c->status(), c->act(), {}};
    f.bind();
    LAUNCH(c, LSAM_PROF_NORM, launch_p(c, (const void*)norm_finalize_kernel, dim3(c->cfg.K), dim3(256), f.ptrs));
    return LSAM_OK;
  }
  dim3 grid((unsigned)ceil_div(n, vec4 ? norm_chunk<4>() : norm_chunk<1>()), c->cfg.K);
  if ((int64_t)grid.x > nch) return c->fail(LSAM_ERR_WORKSPACE, "norm: partial-sum buffer too small");
  if (vec4) LAUNCH(c, LSAM_PROF_NORM, launch_k(c, sumsq_partial_kernel<4>, grid, kNormThreads, 0, g, ldg, n, partial, nch, c->act()));
  else LAUNCH(c, LSAM_PROF_NORM, launch_k(c, sumsq_partial_kernel<1>, grid, kNormThreads, 0, g, ldg, n, partial, nch, c->act()));
  FinArgs f{partial, nch, (int64_t)grid.x, rho, c->cfg.gamma, norm_out, scale_out, c->status(), c->act(), {}};
  f.bind();
  LAUNCH(c, LSAM_PROF_NORM, launch_p(c, (const void*)norm_finalize_kernel, dim3(c->cfg.K), dim3(256), f.ptrs));
  return LSAM_OK;
}

template <typename TP, typename TG>
int launch_perturb(lsam_ctx* c, const TG* g, int64_t ldg, int64_t n, bool vec4) {
  // x3 form (TP = bf16): the perturbed point goes straight into the three planes the descent pass reads; an fp32 copy is kept
  // only where lsam_read_grads(3) can ask for it
  const bool x3 = c->L.x3;
  TP* xt = x3 ? c->at<TP>(c->L.xpl) : c->at<TP>(c->L.xop);
  const int64_t plane = x3 ? (int64_t)c->cfg.K * c->L.ld : 0;
  float* xt32 = (x3 && (c->cfg.flags & LSAM_FLAG_KEEP_G1)) ? c->at<float>(c->L.xop) : nullptr;
  const int64_t per = (int64_t)kPertThreads * kPertIter * (vec4 ? 4 : 1);
  dim3 grid((unsigned)ceil_div(n, per), c->cfg.K);
  if (vec4) LAUNCH(c, LSAM_PROF_PERTURB, launch_k(c, perturb_kernel<4, TP, TG>, grid, kPertThreads, 0, c->x(), c->L.ld, g, ldg, n, c->scale(), xt, c->L.ld, c->act(), plane, xt32));
  else LAUNCH(c, LSAM_PROF_PERTURB, launch_k(c, perturb_kernel<1, TP, TG>, grid, kPertThreads, 0, c->x(), c->L.ld, g, ldg, n, c->scale(), xt, c->L.ld, c->act(), plane, xt32));
  return LSAM_OK;
}

// out[j] = mean over the K workers of g[k][j] (fp32 rows, or the bf16 rows of the tensor-core path)
int launch_mean_rows(lsam_ctx* c, const void* g, bool g_is_bf16, int64_t ldg, int64_t n, bool vec4, float* out) {
  const int K = c->cfg.K;
  if (vec4) {
    const unsigned grid = (unsigned)ceil_div(n, (int64_t)256 * 4);
    if (g_is_bf16) LAUNCH(c, LSAM_PROF_NORM, launch_k(c, mean_rows_kernel<4, bf16>, grid, 256, 0, reinterpret_cast<const bf16*>(g), ldg, K, n, out));
    else LAUNCH(c, LSAM_PROF_NORM, launch_k(c, mean_rows_kernel<4, float>, grid, 256, 0, reinterpret_cast<const float*>(g), ldg, K, n, out));
  } else {
    const unsigned grid = (unsigned)ceil_div(n, (int64_t)256);
    if (g_is_bf16) LAUNCH(c, LSAM_PROF_NORM, launch_k(c, mean_rows_kernel<1, bf16>, grid, 256, 0, reinterpret_cast<const bf16*>(g), ldg, K, n, out));
    else LAUNCH(c, LSAM_PROF_NORM, launch_k(c, mean_rows_kernel<1, float>, grid, 256, 0, reinterpret_cast<const float*>(g), ldg, K, n, out));
  }
  return LSAM_OK;
}

// Non-Gaussian stationary kernel: weight[k] = w(||x_k - y_read(k)||) from one pass over x (fixed-order two-pass reduction)
int launch_pull_weights(lsam_ctx* c) {
  const Layout& L = c->L;
  const int K = c->cfg.K;
  const int64_t n = (c->cfg.model == LSAM_MODEL_FLAT) ? L.d : L.ld;  // padding elements are zero in x and in every centre version
  float* partial = c->at<float>(L.partial);
  dim3 grid((unsigned)ceil_div(n, norm_chunk<4>()), K);
  if ((int64_t)grid.x > L.nchunks) return c->fail(LSAM_ERR_WORKSPACE, "pull weights: partial-sum buffer too small");
  LAUNCH(c, LSAM_PROF_NORM, launch_k(c, gap_sumsq_partial_kernel, grid, kNormThreads, 0, c->x(), L.ld, c->at<float>(L.yring), n, partial, L.nchunks, c->slot(), c->act()));
  LAUNCH(c, LSAM_PROF_NORM, launch_k(c, pull_weight_kernel, K, 256, 0, partial, L.nchunks, (int64_t)grid.x, c->cfg.kernel_kind, c->cfg.lambda, c->cfg.kernel_param, c->pull_weight(), c->act()));
  return LSAM_OK;
}

UpdateArgs make_update_args(lsam_ctx* c, const void* g, int g_mode, int64_t ldg, int64_t n, float eta) {
  UpdateArgs a;
  a.g_mode = g_mode;
  a.active = c->act();
  a.x = c->x(); a.v = c->v(); a.g = g; a.yring = c->at<float>(c->L.yring); a.slot = c->slot();
  a.acc = c->at<float>(c->L.acc);
  a.xop = c->L.x3 ? c->at<void>(c->L.xpl) : c->at<void>(c->L.xop);
  a.xop_plane = c->L.x3 ? (int64_t)c->cfg.K * c->L.ld : 0;
  a.ld = c->L.ld; a.ldg = ldg; a.n = n; a.K = c->cfg.K; a.k_offset = c->cfg.k_offset; a.eta = eta; a.mu = c->cfg.mu; a.lambda = c->cfg.lambda;
  a.lam_k = c->cfg.kernel_kind != KERNEL_GAUSSIAN ? c->pull_weight() : nullptr;
  a.sigma = c->cfg.noise_temp > 0.f ? sqrtf(2.0f * eta * c->cfg.noise_temp) : 0.f;
  a.seed = c->cfg.seed; a.tick = (uint64_t)c->t; a.seg = c->L.seg;
  return a;
}

template <int V, bool N, typename T, bool W>
void* update_func(bool noise) {
  return noise ? (void*)update_kernel<V, N, T, W, true> : (void*)update_kernel<V, N, T, W, false>;
}

int launch_update(lsam_ctx* c, const void* g, int g_mode, int64_t ldg, int64_t n, bool vec4, float eta) {
  UpdateArgs a = make_update_args(c, g, g_mode, ldg, n, eta);
  const bool bf = c->cfg.gemm_dtype == LSAM_GEMM_BF16 || c->L.x3;  // a bf16 operand copy (x3: its three planes) is written with x
  const bool nes = c->cfg.nesterov != 0;
  const bool noise = c->cfg.noise_temp > 0.f;
  unsigned grid = (unsigned)ceil_div(n, (int64_t)kUpdThreads * (vec4 ? 4 : 1));
  void* f;
  if (g_mode == 2 && bf && vec4 && n % 8 == 0) {  // tensor-core path: 8 elements per thread
    grid = (unsigned)ceil_div(n, (int64_t)kUpdThreads * 8);
    if (nes) f = noise ? (void*)update8_kernel<true, true> : (void*)update8_kernel<true, false>;
    else     f = noise ? (void*)update8_kernel<false, true> : (void*)update8_kernel<false, false>;
  } else if (g_mode == 0 && !bf && vec4 && n % 8 == 0 && ldg % 4 == 0 && c->L.ld % 4 == 0 && n >= ((int64_t)1 << 22)) {
    // fp32 gradients, long rows: 8 elements per thread (short rows keep 4, for twice as many blocks)
    grid = (unsigned)ceil_div(n, (int64_t)kUpdThreads * 8);
    if (nes) f = noise ? (void*)update8f_kernel<true, true> : (void*)update8f_kernel<true, false>;
    else     f = noise ? (void*)update8f_kernel<false, true> : (void*)update8f_kernel<false, false>;
  } else if (vec4) {
    if (bf) f = nes ? update_func<4, true, bf16, true>(noise) : update_func<4, false, bf16, true>(noise);
    else    f = nes ? update_func<4, true, float, false>(noise) : update_func<4, false, float, false>(noise);
  } else {
    if (bf) f = nes ? update_func<1, true, bf16, true>(noise) : update_func<1, false, bf16, true>(noise);
    else    f = nes ? update_func<1, true, float, false>(noise) : update_func<1, false, float, false>(noise);
  }
  c->upd_func = f;
  void* ptrs[1] = {&a};
  LAUNCH(c, LSAM_PROF_UPDATE, launch_p(c, (const void*)f, dim3(grid), dim3(kUpdThreads), ptrs));
  return LSAM_OK;
}

// The fused update on the parameters [off, off + n) of every row only (off and n multiples of 64: one padded segment)
int launch_update_range(lsam_ctx* c, int64_t off, int64_t n, float eta) {
  const bool bfg = c->grads_bf16;
  const void* g = bfg ? (const void*)(c->at<bf16>(c->L.g1b) + off) : (const void*)(c->g() + off);
  UpdateArgs a = make_update_args(c, g, bfg ? 2 : 0, c->L.ld, n, eta);
  a.x += off; a.v += off; a.yring += off; a.acc += off;
  a.xop = c->cfg.gemm_dtype == LSAM_GEMM_BF16 ? (void*)(c->at<bf16>(c->L.xop) + off) : (void*)(c->at<float>(c->L.xop) + off);
  const bool nes = c->cfg.nesterov != 0;
  void* f;
  unsigned grid;
  if (bfg) {
    grid = (unsigned)ceil_div(n, (int64_t)kUpdThreads * 8);
    f = nes ? (void*)update8_kernel<true, false> : (void*)update8_kernel<false, false>;
  } else {
    grid = (unsigned)ceil_div(n, (int64_t)kUpdThreads * 4);
    f = nes ? update_func<4, true, bf16, true>(false) : update_func<4, false, bf16, true>(false);
  }
  void* ptrs[1] = {&a};
  LAUNCH(c, LSAM_PROF_UPDATE, launch_p(c, (const void*)f, dim3(grid), dim3(kUpdThreads), ptrs));
  return LSAM_OK;
}

SchedArgs make_sched_args(lsam_ctx* c, int64_t t, int32_t* idx, int32_t* stale, int32_t* ver, int32_t* slot, int64_t budget, int32_t* active) {
  SchedArgs a;
  for (int s = 0; s < 16; ++s) {
    const int64_t ts = t - s > 0 ? t - s : 0;
    a.hist.v[s] = c->ver_of_step(ts);
  }
  const bool flat = c->cfg.model == LSAM_MODEL_FLAT;
  a.seed = c->cfg.seed; a.t = (uint64_t)t; a.n_samples = flat ? 1 : c->cfg.n_samples; a.B = flat ? 0 : c->cfg.batch;
  a.stale_max = c->cfg.stale_max; a.ring = c->L.ring; a.idx = flat ? nullptr : idx; a.stale = stale; a.ver = ver; a.slot = slot;
  a.K = c->cfg.K; a.active_num = c->cfg.active_num; a.budget = budget; a.active = active; a.k_offset = c->cfg.k_offset;
  return a;
}

int launch_schedule(lsam_ctx* c, int64_t t, int32_t* idx, int32_t* stale, int32_t* ver, int32_t* slot, int64_t budget, int32_t* active) {
  SchedArgs a = make_sched_args(c, t, idx, stale, ver, slot, budget, active);
  a.bind();
  LAUNCH(c, LSAM_PROF_SCHEDULE, launch_p(c, (const void*)schedule_kernel, dim3(c->cfg.K), dim3(128), a.ptrs));
  return LSAM_OK;
}

// Host statement of the same rule as schedule_kernel: which workers step at tick t given the remaining budget.
void host_active_mask(const lsam_config& cfg, int64_t t, int64_t budget, std::vector<int32_t>& mask) {
  const int K = cfg.K;
  mask.assign(K, 0);
  std::vector<std::pair<uint64_t, int>> ready;
  for (int k = 0; k < K; ++k)
    if ((schedule_hash(cfg.seed, kTagAct, (uint64_t)t, (uint64_t)k, 0) % 256ULL) < (uint64_t)cfg.active_num)
      ready.push_back({schedule_hash(cfg.seed, kTagOrd, (uint64_t)t, (uint64_t)k, 0), k});
  std::sort(ready.begin(), ready.end());
  for (size_t r = 0; r < ready.size() && (int64_t)r < budget; ++r) mask[ready[r].second] = 1;
}

// ---- SIMT GEMM launches in logical coordinates
template <typename TA, typename TB, class Epi>
int launch_simt(lsam_ctx* c, int cls, GemmOperand A, GemmOperand B, int M, int N, int Kd, const Epi& epi, int parts = 1, int chunk = 0) {
  dim3 grid((unsigned)ceil_div(N, kSimtBN), (unsigned)ceil_div(M, kSimtBM), c->cfg.K * parts);
  // every operand of the classifier is contiguous either along its rows or along the contraction index
  const bool a_mc = (A.sr == 1), b_nc = (B.sr == 1);
  if (!a_mc && A.sk != 1) return c->fail(LSAM_ERR_INVALID, "SIMT GEMM: operand A has no unit stride");
  if (!b_nc && B.sk != 1) return c->fail(LSAM_ERR_INVALID, "SIMT GEMM: operand B has no unit stride");
  // a tile list shorter than two blocks per SM with a long contraction: two thread groups per block split the contraction
  const bool split = parts == 1 && (int64_t)grid.x * grid.y * grid.z < 2 * 148 && Kd >= 8 * kSimtBK;
#define LSAM_SIMT(AM, BN_)                                                                                                                        \
  do {                                                                                                                                            \
    if (split) LAUNCH(c, cls, launch_k(c, gemm_simt_kernel<TA, TB, AM, BN_, Epi, 2>, grid, 512, 0, A, B, M, N, Kd, epi, c->act(), 1, 0));              \
    else LAUNCH(c, cls, launch_k(c, gemm_simt_kernel<TA, TB, AM, BN_, Epi, 1>, grid, 256, 0, A, B, M, N, Kd, epi, c->act(), parts, chunk));       \
  } while (0)
  if (a_mc) { if (b_nc) LSAM_SIMT(true, true); else LSAM_SIMT(true, false); }
  else      { if (b_nc) LSAM_SIMT(false, true); else LSAM_SIMT(false, false); }
#undef LSAM_SIMT
  return LSAM_OK;
}

// One gradient pass of the classifier at the parameters P ([K, ld], type T); gradient -> g, loss -> loss_out (nullable).
// g_bf16 (tensor-core path only): store the gradient rounded to bf16 in the g1b buffer instead of fp32 in g.
// fu != nullptr (tensor-core path, descent pass): the weight gradient of every layer is consumed by the worker update in its own
// epilogue instead of being stored; the dgrad of a layer, which still reads the perturbed weights, then runs BEFORE that layer's wgrad.
template <typename T>
int mlp_pass(lsam_ctx* c, const T* P, float* loss_out, bool g_bf16, const TcFusedUpdate* fu = nullptr) {
  const Layout& L = c->L;
  const int K = c->cfg.K, B = c->cfg.batch;
  const int nl = (int)L.layers.size();
  const int64_t ld = L.ld;
  const int ldb = L.ldb;
  int rc;
  // a head of at most kHeadMaxOut classes: chunked forward + sum in the loss kernel (SIMT paths and the three-plane form; the
  // bf16 tensor-core path keeps its GEMM)
  const bool narrow = L.layers[nl - 1].out <= kHeadMaxOut && (!c->use_tc || L.x3);
  const int64_t p_plane = L.x3 ? (int64_t)K * ld : 0;
  // on the SIMT paths the same heads go backward through head_dgrad_kernel (the three-plane form keeps its GEMM, which measured the same)
  const bool head_bwd = narrow && nl >= 2 && !c->use_tc;
  // forward
  for (int l = 0; l < nl; ++l) {
    const LayerInfo& li = L.layers[l];
    const T* a_in = c->at<T>(L.act[l]);
    const bool head = (l == nl - 1);
    if (head && narrow) {
      dim3 hgrid((unsigned)ceil_div(li.in, kHeadChunkIn), (unsigned)ceil_div(B, 128), K);
      LAUNCH(c, LSAM_PROF_GEMM_FWD, launch_k(c, head_chunk_kernel<T>, hgrid, 128, 0, a_in, (int64_t)li.in * ldb, ldb, L.x3 ? (int64_t)K * li.in * ldb : 0, P, ld,
                                                                                     li.w_pad, p_plane, li.in, li.out, B, c->at<float>(L.hpart), c->act()));
      continue;
    }
    if (c->use_tc) {
      int trc = 0;
      LAUNCH(c, LSAM_PROF_GEMM_FWD, trc = tc_forward(c->tc, l, c->stream));
      if (trc != 0) return c->fail(LSAM_ERR_CUDA, "tcgen05 forward launch failed");
      continue;
    }
    GemmOperand A{a_in, (int64_t)li.in * ldb, 1, ldb};       // (z, b, i) in the feature-major buffer [z][i][b]
    GemmOperand W{P + li.w_pad, ld, li.in, 1};               // (z, o, i)
    if (head) {
      EpiFwdHead<T> e{P + li.b_pad, ld, c->at<float>(L.logits), li.out, ldb};
      rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_FWD, A, W, B, li.out, li.in, e);
    } else {
      EpiFwdHidden<T, T> e{P + li.b_pad, ld, c->at<T>(L.act[l + 1]), li.residual ? a_in : nullptr, c->at<uint8_t>(L.mask[l]), li.out, ldb};
      rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_FWD, A, W, B, li.out, li.in, e);
    }
    if (rc != LSAM_OK) return rc;
  }
  // loss and its gradient w.r.t. the logits
  const int C = L.layers[nl - 1].out;
  int cur = 0;
  // x3 form: backward signals are three planes, (K * width * ldb) elements apart
  LAUNCH(c, LSAM_PROF_LOSS, launch_k(c, softmax_ce_kernel<T>, dim3((unsigned)ceil_div(B, 32), K), dim3(32, 8), 0, 
      c->at<float>(L.logits), c->at<int32_t>(L.ylab), B, C, ldb, c->at<T>(L.dz[cur]), c->at<float>(L.rowloss), c->status(), c->act(),
      L.x3 ? (int64_t)K * C * ldb : 0, narrow ? c->at<float>(L.hpart) : nullptr, (int)ceil_div(L.layers[nl - 1].in, kHeadChunkIn),
      P + L.layers[nl - 1].b_pad, ld, p_plane));
  if (loss_out) LAUNCH(c, LSAM_PROF_LOSS, launch_k(c, mean_loss_kernel, K, 32, 0, c->at<float>(L.rowloss), B, loss_out, c->act()));
  // backward
  for (int l = nl - 1; l >= 0; --l) {
    const LayerInfo& li = L.layers[l];
    const T* dz = c->at<T>(L.dz[cur]);
    const int64_t dz_plane = L.x3 ? (int64_t)K * li.out * ldb : 0;
    const T* a_in = c->at<T>(L.act[l]);
    // tensor-core path: the dgrad of the layer above has already left this layer's bias gradient (and its sum of squares)
    // (and so has the backward kernel of a narrow head, on every path that uses it)
    const bool bias_done = (c->use_tc && l < nl - 1 && tc_dgrad_can_fuse_bias(c->tc, l + 1)) || (head_bwd && l == nl - 2);
    // backward through a narrow head into the layer below, with that layer's bias gradient
    auto head_dgrad = [&]() -> int {
      const LayerInfo& lp = L.layers[l - 1];
      const int64_t out_plane = L.x3 ? (int64_t)K * li.in * ldb : 0;
      LAUNCH(c, LSAM_PROF_GEMM_DGRAD, launch_k(c, head_dgrad_kernel<T>, dim3((unsigned)ceil_div(li.in, 8), K), 256, 0, 
          dz, dz_plane, P, ld, li.w_pad, p_plane, li.in, li.out, B, ldb, c->at<uint8_t>(L.mask[l - 1]), c->at<T>(L.dz[cur ^ 1]),
          lp.residual ? c->at<T>(L.dh[l & 1]) : nullptr, out_plane, c->g(), ld, lp.b_pad, c->use_tc ? c->at<float>(L.partial) : nullptr, L.nchunks,
          c->use_tc ? c->tc.bias_slot0[l - 1] : 0, c->act()));
      return LSAM_OK;
    };
    if (!bias_done) {
      float* part = c->use_tc ? c->at<float>(L.partial) : nullptr;
      const int slot0 = c->use_tc ? c->tc.bias_slot0[l] : 0;
      dim3 bgrid((unsigned)ceil_div(li.out, 8), K);
      if (g_bf16)
        LAUNCH(c, LSAM_PROF_BIAS_GRAD, launch_k(c, bias_grad_kernel<T, bf16>, bgrid, 256, 0, dz, B, li.out, ldb, c->at<bf16>(L.g1b), ld, li.b_pad, part, L.nchunks, slot0, c->act(), (int64_t)0));
      else
        LAUNCH(c, LSAM_PROF_BIAS_GRAD, launch_k(c, bias_grad_kernel<T, float>, bgrid, 256, 0, dz, B, li.out, ldb, c->g(), ld, li.b_pad, part, L.nchunks, slot0, c->act(), dz_plane));
    }
    if (c->use_tc) {
      int trc = 0;
      auto dgrad = [&]() -> int {
        if (l == 0) return LSAM_OK;
        if (head_bwd && l == nl - 1) return head_dgrad();
        void* bias_g = nullptr;
        if (tc_dgrad_can_fuse_bias(c->tc, l)) bias_g = g_bf16 ? (void*)c->at<bf16>(L.g1b) : (void*)c->g();
        LAUNCH(c, LSAM_PROF_GEMM_DGRAD, trc = tc_dgrad(c->tc, l, c->stream, bias_g, g_bf16));
        return LSAM_OK;
      };
      if (fu != nullptr) {
        if ((rc = dgrad()) != LSAM_OK) return rc;
        if (trc == 0) LAUNCH(c, LSAM_PROF_GEMM_WGRAD, trc = tc_wgrad_update(c->tc, l, c->stream, *fu));
      } else {
        LAUNCH(c, LSAM_PROF_GEMM_WGRAD, trc = tc_wgrad(c->tc, l, c->stream, g_bf16));
        if (trc == 0 && (rc = dgrad()) != LSAM_OK) return rc;
      }
      if (trc != 0) return c->fail(LSAM_ERR_CUDA, "tcgen05 backward launch failed");
      cur ^= 1;
      continue;
    }
    {
      GemmOperand A{dz, (int64_t)li.out * ldb, ldb, 1};      // (z, o, b)
      GemmOperand Bm{a_in, (int64_t)li.in * ldb, ldb, 1};    // (z, i, b)
      EpiWgrad e{c->g(), ld, li.w_pad, li.in};
      rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_WGRAD, A, Bm, li.out, li.in, B, e);
      if (rc != LSAM_OK) return rc;
    }
    if (l > 0 && head_bwd && l == nl - 1) {
      if ((rc = head_dgrad()) != LSAM_OK) return rc;
    } else if (l > 0) {
      GemmOperand A{dz, (int64_t)li.out * ldb, 1, ldb};      // (z, b, o)
      GemmOperand W{P + li.w_pad, ld, 1, li.in};             // (z, i, o)
      EpiDgrad<T> e{li.residual ? c->at<T>(L.dh[(l + 1) & 1]) : nullptr,
                    L.layers[l - 1].residual ? c->at<T>(L.dh[l & 1]) : nullptr,
                    c->at<T>(L.dz[cur ^ 1]), c->at<uint8_t>(L.mask[l - 1]), li.in, ldb};
      rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_DGRAD, A, W, B, li.in, li.out, e);
      if (rc != LSAM_OK) return rc;
    }
    cur ^= 1;
  }
  return LSAM_OK;
}

// One gradient pass of the convolutional model (SIMT GEMMs): convolution layers through an explicit patch matrix, then the
// dense layers exactly as in mlp_pass.  Feature maps are [K, C, (y, x, sample)] with the sample fastest (see im2col_kernel).
template <typename T>
int cnn_pass(lsam_ctx* c, const T* P, float* loss_out) {
  const Layout& L = c->L;
  const int K = c->cfg.K, B = c->cfg.batch;
  const int nl = (int)L.layers.size(), nconv = c->cfg.n_conv;
  const int64_t ld = L.ld;
  const int ldb = L.ldb;  // = B for this model
  const bool narrow = L.layers[nl - 1].out <= kHeadMaxOut;  // chunked head forward, summed by the loss kernel
  int rc;
  // forward
  for (int l = 0; l < nl; ++l) {
    const LayerInfo& li = L.layers[l];
    const T* a_in = c->at<T>(L.act[l]);
    const bool head = (l == nl - 1);
    if (li.conv) {
      const int64_t Pn = (int64_t)li.H * li.W * ldb;
      T* col = c->at<T>(L.col[l]);
      LAUNCH(c, LSAM_PROF_GATHER, launch_k(c, im2col_kernel<T>, dim3((unsigned)ceil_div(Pn, 1024), li.in, K), 256, 0, a_in, li.Cin, li.H, li.W, ldb, col, c->act()));
      GemmOperand A{col, (int64_t)li.in * Pn, 1, Pn};           // (z, position, patch element)
      GemmOperand W{P + li.w_pad, ld, li.in, 1};               // (z, output channel, patch element)
      EpiFwdHidden<T, T> e{P + li.b_pad, ld, c->at<T>(L.zout), nullptr, c->at<uint8_t>(L.mask[l]), li.Cout, (int)Pn};
      if ((rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_FWD, A, W, (int)Pn, li.Cout, li.in, e)) != LSAM_OK) return rc;
      LAUNCH(c, LSAM_PROF_GEMM_FWD, launch_k(c, maxpool_kernel<T>, dim3((unsigned)ceil_div(Pn / 4, 1024), li.Cout, K), 256, 0, 
          c->at<T>(L.zout), li.Cout, li.H, li.W, ldb, c->at<T>(L.act[l + 1]), c->at<uint8_t>(L.parg[l]), c->act()));
      continue;
    }
    GemmOperand A{a_in, (int64_t)li.in * ldb, 1, ldb};
    GemmOperand W{P + li.w_pad, ld, li.in, 1};
    if (head && narrow) {
      dim3 hgrid((unsigned)ceil_div(li.in, kHeadChunkIn), (unsigned)ceil_div(B, 128), K);
      LAUNCH(c, LSAM_PROF_GEMM_FWD, launch_k(c, head_chunk_kernel<T>, hgrid, 128, 0, a_in, (int64_t)li.in * ldb, ldb, 0, P, ld, li.w_pad, 0, li.in, li.out, B,
                                                                                     c->at<float>(L.hpart), c->act()));
      rc = LSAM_OK;
    } else if (head) {
      EpiFwdHead<T> e{P + li.b_pad, ld, c->at<float>(L.logits), li.out, ldb};
      rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_FWD, A, W, B, li.out, li.in, e);
    } else {
      EpiFwdHidden<T, T> e{P + li.b_pad, ld, c->at<T>(L.act[l + 1]), nullptr, c->at<uint8_t>(L.mask[l]), li.out, ldb};
      if (li.fw_parts > 1) {
        // partial products per share of the inputs, then their sum in a fixed order handed to the layer's epilogue
        EpiPartial ep{c->at<float>(L.wpart), B, li.out};
        if ((rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_FWD, A, W, B, li.out, li.in, ep, li.fw_parts, li.fw_chunk)) != LSAM_OK) return rc;
        LAUNCH(c, LSAM_PROF_GEMM_FWD, launch_k(c, sum_parts_epi_kernel<EpiFwdHidden<T, T>>, dim3((unsigned)ceil_div((int64_t)B * li.out, 256), K), 256, 0, 
            c->at<float>(L.wpart), li.fw_parts, B, li.out, e, c->act()));
        rc = LSAM_OK;
      } else {
        rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_FWD, A, W, B, li.out, li.in, e);
      }
    }
    if (rc != LSAM_OK) return rc;
  }
  const int C = L.layers[nl - 1].out;
  int cur = 0;
  LAUNCH(c, LSAM_PROF_LOSS, launch_k(c, softmax_ce_kernel<T>, dim3((unsigned)ceil_div(B, 32), K), dim3(32, 8), 0, 
      c->at<float>(L.logits), c->at<int32_t>(L.ylab), B, C, ldb, c->at<T>(L.dz[cur]), c->at<float>(L.rowloss), c->status(), c->act(),
      0, narrow ? c->at<float>(L.hpart) : nullptr, (int)ceil_div(L.layers[nl - 1].in, kHeadChunkIn), P + L.layers[nl - 1].b_pad, ld, 0));
  if (loss_out) LAUNCH(c, LSAM_PROF_LOSS, launch_k(c, mean_loss_kernel, K, 32, 0, c->at<float>(L.rowloss), B, loss_out, c->act()));
  // backward.  dz[cur] holds, for a dense layer, the gradient w.r.t. its pre-activation; for a convolution layer, the gradient
  // w.r.t. its POOLED output (the pooling and the ReLU are undone by unpool_kernel)
  for (int l = nl - 1; l >= 0; --l) {
    const LayerInfo& li = L.layers[l];
    const T* a_in = c->at<T>(L.act[l]);
    if (li.conv) {
      const int64_t Pn = (int64_t)li.H * li.W * ldb;
      T* dzc = c->at<T>(L.dzc);
      LAUNCH(c, LSAM_PROF_GEMM_DGRAD, launch_k(c, unpool_kernel<T>, dim3((unsigned)ceil_div(Pn, 1024), li.Cout, K), 256, 0, 
          c->at<T>(L.dz[cur]), c->at<uint8_t>(L.parg[l]), c->at<uint8_t>(L.mask[l]), li.Cout, li.H, li.W, ldb, dzc, c->act()));
      LAUNCH(c, LSAM_PROF_BIAS_GRAD, launch_k(c, bias_grad_long_kernel<T>, dim3((unsigned)li.Cout, K), 256, 0, dzc, Pn, li.Cout, Pn, c->g(), ld, li.b_pad, c->act()));
      {
        GemmOperand A{dzc, (int64_t)li.Cout * Pn, Pn, 1};                 // (z, output channel, position)
        GemmOperand Bm{c->at<T>(L.col[l]), (int64_t)li.in * Pn, Pn, 1};   // (z, patch element, position)
        if (li.wg_parts > 1) {
          // partial products per share of the positions, then their sum in a fixed order
          EpiPartial e{c->at<float>(L.wpart), li.Cout, li.in};
          if ((rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_WGRAD, A, Bm, li.Cout, li.in, (int)Pn, e, li.wg_parts, li.wg_chunk)) != LSAM_OK) return rc;
          LAUNCH(c, LSAM_PROF_GEMM_WGRAD, launch_k(c, sum_parts_kernel, dim3((unsigned)ceil_div((int64_t)li.Cout * li.in, 256), K), 256, 0, 
              c->at<float>(L.wpart), li.wg_parts, li.Cout, li.in, c->g(), ld, li.w_pad, c->act()));
        } else {
          EpiWgrad e{c->g(), ld, li.w_pad, li.in};
          if ((rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_WGRAD, A, Bm, li.Cout, li.in, (int)Pn, e)) != LSAM_OK) return rc;
        }
      }
      if (l > 0) {
        T* dcol = c->at<T>(L.dcol);
        GemmOperand A{dzc, (int64_t)li.Cout * Pn, 1, Pn};                  // (z, position, output channel)
        GemmOperand W{P + li.w_pad, ld, 1, li.in};                         // (z, patch element, output channel)
        EpiDgrad<T> e{nullptr, nullptr, dcol, nullptr, li.in, (int)Pn};    // the raw gradient of the patch matrix
        if ((rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_DGRAD, A, W, (int)Pn, li.in, li.Cout, e)) != LSAM_OK) return rc;
        LAUNCH(c, LSAM_PROF_GEMM_DGRAD, launch_k(c, col2im_kernel<T>, dim3((unsigned)ceil_div(Pn, 1024), li.Cin, K), 256, 0, 
            dcol, li.Cin, li.H, li.W, ldb, c->at<T>(L.dz[cur ^ 1]), c->act()));
      }
      cur ^= 1;
      continue;
    }
    const T* dz = c->at<T>(L.dz[cur]);
    LAUNCH(c, LSAM_PROF_BIAS_GRAD, launch_k(c, bias_grad_kernel<T, float>, dim3((unsigned)ceil_div(li.out, 8), K), 256, 0, 
        dz, B, li.out, ldb, c->g(), ld, li.b_pad, nullptr, L.nchunks, 0, c->act(), (int64_t)0));
    {
      GemmOperand A{dz, (int64_t)li.out * ldb, ldb, 1};
      GemmOperand Bm{a_in, (int64_t)li.in * ldb, ldb, 1};
      EpiWgrad e{c->g(), ld, li.w_pad, li.in};
      if ((rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_WGRAD, A, Bm, li.out, li.in, B, e)) != LSAM_OK) return rc;
    }
    {
      GemmOperand A{dz, (int64_t)li.out * ldb, 1, ldb};
      GemmOperand W{P + li.w_pad, ld, 1, li.in};
      // the layer below is dense (its ReLU mask applies here) or the last convolution (the raw gradient of its pooled output)
      const bool below_conv = (l - 1 < nconv);
      EpiDgrad<T> e{nullptr, nullptr, c->at<T>(L.dz[cur ^ 1]), below_conv ? nullptr : c->at<uint8_t>(L.mask[l - 1]), li.in, ldb};
      if ((rc = launch_simt<T, T>(c, LSAM_PROF_GEMM_DGRAD, A, W, B, li.in, li.out, e)) != LSAM_OK) return rc;
    }
    cur ^= 1;
  }
  return LSAM_OK;
}

// Gradient of the minibatch loss at the parameters held in `params` (x master, or the operand buffer).
int grad_pass(lsam_ctx* c, bool perturbed, float* loss_out, bool g_bf16 = false, const TcFusedUpdate* fu = nullptr) {
  const lsam_config& cfg = c->cfg;
  if (cfg.model == LSAM_MODEL_LSQ) {
    const float* P = perturbed ? c->at<float>(c->L.xop) : c->x();
    LAUNCH(c, LSAM_PROF_LSQ_GRAD, launch_k(c, lsq_grad_kernel, cfg.K, 256, sizeof(float) * cfg.batch, 
        c->at<float>(c->L.act[0]), c->at<float>(c->L.ylab), P, c->L.ld, cfg.batch, c->L.in0, c->g(), c->L.ld, loss_out, c->act()));
    return LSAM_OK;
  }
  if (cfg.model == LSAM_MODEL_CNN) {
    if (cfg.gemm_dtype == LSAM_GEMM_BF16) return cnn_pass<bf16>(c, c->at<bf16>(c->L.xop), loss_out);
    return cnn_pass<float>(c, perturbed ? c->at<float>(c->L.xop) : c->x(), loss_out);
  }
  if (cfg.gemm_dtype == LSAM_GEMM_BF16) return mlp_pass<bf16>(c, c->at<bf16>(c->L.xop), loss_out, g_bf16 && c->use_tc, c->use_tc ? fu : nullptr);
  if (c->L.x3) return mlp_pass<bf16>(c, c->at<bf16>(c->L.xpl), loss_out, false);  // the planes hold x or x~, whichever was split last
  return mlp_pass<float>(c, perturbed ? c->at<float>(c->L.xop) : c->x(), loss_out, false);
}

// x3 form: the three bf16 planes of src [K, ld] (x, or the perturbed point) -> xpl
int launch_split3(lsam_ctx* c, const float* src) {
  dim3 grid((unsigned)ceil_div(c->L.ld, 1024), c->cfg.K);
  LAUNCH(c, LSAM_PROF_COPY, launch_k(c, split3_rows_kernel, grid, 256, 0, src, c->L.ld, c->L.ld, c->at<bf16>(c->L.xpl), c->L.ld, (int64_t)c->cfg.K * c->L.ld));
  return LSAM_OK;
}

int refresh_operand_copy(lsam_ctx* c) {
  if (c->L.x3) return launch_split3(c, c->x());
  if (c->cfg.gemm_dtype != LSAM_GEMM_BF16) return LSAM_OK;
  dim3 grid((unsigned)ceil_div(c->L.ld, 256), c->cfg.K);
  LAUNCH(c, LSAM_PROF_COPY, launch_k(c, cast_rows_kernel<bf16>, grid, 256, 0, c->x(), c->L.ld, c->at<bf16>(c->L.xop), c->L.ld, c->L.ld));
  return LSAM_OK;
}

template <bool TO_PADDED>
int seg_copy(lsam_ctx* c, const float* src, int64_t lds, float* dst, int64_t ldd, int rows) {
  int64_t maxlen = 0;
  for (int i = 0; i < c->L.seg.n; ++i) maxlen = c->L.seg.len[i] > maxlen ? c->L.seg.len[i] : maxlen;
  dim3 grid((unsigned)ceil_div(maxlen, 256), c->L.seg.n, rows);
  LAUNCH(c, LSAM_PROF_COPY, launch_k(c, seg_copy_kernel<TO_PADDED, float, float>, grid, 256, 0, src, lds, dst, ldd, c->L.seg));
  return LSAM_OK;
}

// NVTX ranges around the phases of a tick, so that a profiler can filter or colour them (host-side markers only: a few
// tens of nanoseconds when no tool is attached).  next() closes the previous phase; the destructor closes the last one.
struct PhaseRange {
  bool open = false;
  void next(const char* name) {
    if (open) nvtxRangePop();
    nvtxRangePushA(name);
    open = true;
  }
  ~PhaseRange() {
    if (open) nvtxRangePop();
  }
};

// The launch sequence of one tick (no host state is changed here, so that it can also be recorded into a CUDA graph).
int step_enqueue(lsam_ctx* c, float eta, float rho, bool gather, int64_t budget) {
  PhaseRange phase;
  phase.next("lsam S0-S1 schedule, gather");
  const lsam_config& cfg = c->cfg;
  const Layout& L = c->L;
  const bool flat = cfg.model == LSAM_MODEL_FLAT;
  int rc;
  if ((rc = launch_schedule(c, c->t, c->idx(), c->stale(), c->ver(), c->slot(), budget, c->async_on ? c->active_buf() : nullptr)) != LSAM_OK) return rc;
  const int64_t rows = (int64_t)cfg.K * cfg.batch;
  if (!flat && gather) {
    if (cfg.model == LSAM_MODEL_LSQ) {
      LAUNCH(c, LSAM_PROF_GATHER, launch_k(c, gather_kernel<float>, (unsigned)rows, 128, 0, c->X, c->Y, c->idx(), cfg.n_samples, c->L.in0, c->L.in0, c->at<float>(L.act[0]), c->at<uint32_t>(L.ylab), c->status(), cfg.batch, c->act()));
    } else {
      dim3 grid((unsigned)ceil_div(c->L.in0, 32), (unsigned)ceil_div(cfg.batch, 32), cfg.K);
      if (cfg.gemm_dtype == LSAM_GEMM_BF16 || L.x3)
        LAUNCH(c, LSAM_PROF_GATHER, launch_k(c, gather_t_kernel<bf16>, grid, dim3(32, 8), 0, c->X, c->Y, c->idx(), cfg.n_samples, cfg.batch, c->L.in0, L.ldb, c->at<bf16>(L.act[0]), c->at<uint32_t>(L.ylab), c->status(), c->act(), c->in_plane()));
      else
        LAUNCH(c, LSAM_PROF_GATHER, launch_k(c, gather_t_kernel<float>, grid, dim3(32, 8), 0, c->X, c->Y, c->idx(), cfg.n_samples, cfg.batch, c->L.in0, L.ldb, c->at<float>(L.act[0]), c->at<uint32_t>(L.ylab), c->status(), c->act(), (int64_t)0));
    }
  }
  const bool vec4 = L.vec4 && (!flat || c->ext_vec4);
  const int64_t n = flat ? L.d : L.ld;
  const int64_t ldg = flat ? L.d : L.ld;
  // Gradient storage: the tensor-core path writes both gradients from the weight-gradient GEMM in bf16 into the g1b
  // buffer (a storage format: 2 instead of 4 bytes per element written and read back; the norms come from the fp32
  // accumulators) unless LSAM_FLAG_GRAD_FP32 asks for fp32; every other path keeps fp32 gradients and uses them as they are.
  const bool gb = c->grads_bf16;
  const int g_mode = gb ? 2 : 0;
  const void* gptr = gb ? (const void*)c->at<bf16>(L.g1b) : (flat ? (const void*)c->eg2 : (const void*)c->g());
  const bool dp = cfg.dp_average != 0;        // synchronous data parallelism: both gradients are averaged over the workers
  const bool other_kernel = cfg.kernel_kind != KERNEL_GAUSSIAN;
  float* gbar1 = c->at<float>(L.gbar1);
  float* gbar2 = c->at<float>(L.gbar2);
  // the fused update on the descent gradient: per-worker rows, or (dp) the one averaged row read by every worker (row stride 0)
  auto finish_tick = [&](const void* g2src) -> int {
    int rc2;
    if (dp) {
      if ((rc2 = launch_mean_rows(c, g2src, gb, ldg, n, vec4, gbar2)) != LSAM_OK) return rc2;
      if ((cfg.flags & LSAM_FLAG_STEP_INFO) && (rc2 = launch_norm(c, gbar2, 0, n, vec4, 0.f, c->norm2(), nullptr, false)) != LSAM_OK) return rc2;
    } else if (cfg.flags & LSAM_FLAG_STEP_INFO) {
      if ((rc2 = launch_norm(c, reinterpret_cast<const float*>(g2src), ldg, n, vec4, 0.f, c->norm2(), nullptr)) != LSAM_OK) return rc2;
    }
    if (other_kernel && (rc2 = launch_pull_weights(c)) != LSAM_OK) return rc2;
    if (dp) return launch_update(c, gbar2, 0, 0, n, vec4, eta);
    return launch_update(c, gptr, g_mode, ldg, n, vec4, eta);
  };
  // ascent gradient, its norm, perturbation
  if (rho == 0.f && !flat && !L.g1keep) {
    // rho = 0: the perturbed point is x itself, so the two gradients coincide (entropy-/elastic-averaging SGD, the
    // unperturbed case of Theorem 2; with dp_average: DP-SGD): one gradient pass, no norm, no perturbation
    phase.next("lsam S2 gradient (rho = 0: single pass)");
    if ((rc = grad_pass(c, false, c->loss(), gb)) != LSAM_OK) return rc;
    phase.next("lsam S6 update");
    if (cfg.flags & LSAM_FLAG_STEP_INFO) {
      if (dp) {
        if ((rc = launch_mean_rows(c, gptr, gb, ldg, n, vec4, gbar1)) != LSAM_OK) return rc;
        if ((rc = launch_norm(c, gbar1, 0, n, vec4, 0.f, c->norm1(), nullptr, false)) != LSAM_OK) return rc;
      } else if ((rc = launch_norm(c, c->g(), ldg, n, vec4, 0.f, c->norm1(), nullptr)) != LSAM_OK) return rc;
    }
    return finish_tick(gptr);
  }
  const float* g1 = flat ? c->eg1 : c->g();
  const bool g1_bf16 = gb;
  phase.next("lsam S2 ascent gradient");
  if (!flat && (rc = grad_pass(c, false, c->loss(), g1_bf16)) != LSAM_OK) return rc;
  if (!flat && L.g1keep && !dp) {
    if (g1_bf16) LSAM_CUDA(c, cudaMemcpyAsync(c->at<bf16>(L.g1keep), c->at<bf16>(L.g1b), sizeof(bf16) * cfg.K * L.ld, cudaMemcpyDeviceToDevice, c->stream));
    else LSAM_CUDA(c, cudaMemcpyAsync(c->at<float>(L.g1keep), c->g(), sizeof(float) * cfg.K * L.ld, cudaMemcpyDeviceToDevice, c->stream));
  }
  phase.next("lsam S3-S4 norm, perturbation");
  if (dp) {
    // the perturbation follows the averaged gradient and its norm (every worker's row of scale[] holds the same value)
    const void* g1src = g1_bf16 ? (const void*)c->at<bf16>(L.g1b) : (const void*)g1;
    if ((rc = launch_mean_rows(c, g1src, g1_bf16, ldg, n, vec4, gbar1)) != LSAM_OK) return rc;
    if ((rc = launch_norm(c, gbar1, 0, n, vec4, rho, c->norm1(), c->scale(), false)) != LSAM_OK) return rc;
    if (cfg.gemm_dtype == LSAM_GEMM_BF16 || L.x3) rc = launch_perturb<bf16, float>(c, gbar1, 0, n, vec4);
    else rc = launch_perturb<float, float>(c, gbar1, 0, n, vec4);
  } else {
    if ((rc = launch_norm(c, g1, ldg, n, vec4, rho, c->norm1(), c->scale())) != LSAM_OK) return rc;
    if (g1_bf16 && vec4 && n % 8 == 0) {
      dim3 pgrid((unsigned)ceil_div(n, (int64_t)kPertThreads * 8 * kPert8Iter), cfg.K);
      LAUNCH(c, LSAM_PROF_PERTURB, launch_k(c, perturb8_kernel, pgrid, kPertThreads, 0, c->x(), L.ld, c->at<bf16>(L.g1b), ldg, n, c->scale(), c->at<bf16>(L.xop), L.ld, c->act()));
      rc = LSAM_OK;
    } else if (g1_bf16) rc = launch_perturb<bf16, bf16>(c, c->at<bf16>(L.g1b), ldg, n, vec4);
    else if (cfg.gemm_dtype == LSAM_GEMM_BF16 || L.x3) rc = launch_perturb<bf16, float>(c, g1, ldg, n, vec4);
    else rc = launch_perturb<float, float>(c, g1, ldg, n, vec4);
  }
  if (rc != LSAM_OK) return rc;
  if (L.xpkeep) LSAM_CUDA(c, cudaMemcpyAsync(c->at<bf16>(L.xpkeep), c->at<bf16>(L.xop), sizeof(bf16) * cfg.K * L.ld, cudaMemcpyDeviceToDevice, c->stream));
  // descent gradient at the perturbed point, same minibatch
  phase.next("lsam S5 descent gradient");
  if (c->fused_update) {
    // weights: updated inside the weight-gradient epilogues of this pass; the pull weights of a non-Gaussian kernel are
    // distances of the iterates BEFORE the update, so they are taken first
    if (other_kernel && (rc = launch_pull_weights(c)) != LSAM_OK) return rc;
    TcFusedUpdate fu{c->x(), c->v(), c->at<float>(L.yring), c->slot(), c->at<bf16>(L.xop), other_kernel ? c->pull_weight() : nullptr,
                     eta, cfg.mu, cfg.lambda, cfg.nesterov != 0 ? 1 : 0};
    if ((rc = grad_pass(c, true, nullptr, gb, &fu)) != LSAM_OK) return rc;
    phase.next("lsam S6 update (biases, iterate sums)");
    if (cfg.flags & LSAM_FLAG_STEP_INFO)
      if ((rc = launch_norm(c, nullptr, ldg, n, vec4, 0.f, c->norm2(), nullptr)) != LSAM_OK) return rc;
    for (const LayerInfo& li : L.layers) {
      const int64_t wlen = round_up((int64_t)li.in * li.out, kSegAlign), blen = round_up((int64_t)li.out, kSegAlign);
      if ((rc = launch_update_range(c, li.b_pad, blen, eta)) != LSAM_OK) return rc;  // bias gradients were stored as usual
      LAUNCH(c, LSAM_PROF_UPDATE, launch_k(c, acc_add_kernel, (unsigned)ceil_div(wlen, 1024), 256, 0, c->x(), L.ld, cfg.K, li.w_pad, wlen, c->at<float>(L.acc), c->act()));
    }
    return LSAM_OK;
  }
  if (!flat && (rc = grad_pass(c, true, nullptr, gb)) != LSAM_OK) return rc;
  phase.next("lsam S6 update");
  return finish_tick(gptr);
}


// ---- CUDA-graph replay.  The sequence of a tick is recorded once per variant (gathered / supplied minibatch, rho = 0
// shortcut or not) after one eager run; afterwards a tick is one graph launch, with the arguments of the three kernels
// that change from tick to tick (schedule, norm finalisation, update) refreshed in the executable graph.
int graph_capture(lsam_ctx* c, lsam_ctx::GraphSlot& gs, float eta, float rho, bool gather, int64_t budget) {
  const int64_t l0 = c->launches;
  LSAM_CUDA(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
  const int rc = step_enqueue(c, eta, rho, gather, budget);
  cudaGraph_t graph = nullptr;
  const cudaError_t e = cudaStreamEndCapture(c->stream, &graph);
  if (rc != LSAM_OK || e != cudaSuccess || !graph) {
    if (graph) cudaGraphDestroy(graph);
    return rc != LSAM_OK ? rc : c->fail(LSAM_ERR_CUDA, std::string("cudaStreamEndCapture: ") + cudaGetErrorString(e));
  }
  gs.launches = c->launches - l0;
  LSAM_CUDA(c, cudaGraphInstantiate(&gs.exec, graph, 0));
  gs.graph = graph;
  size_t n = 0;
  LSAM_CUDA(c, cudaGraphGetNodes(graph, nullptr, &n));
  std::vector<cudaGraphNode_t> nodes(n);
  LSAM_CUDA(c, cudaGraphGetNodes(graph, nodes.data(), &n));
  for (cudaGraphNode_t nd : nodes) {
    cudaGraphNodeType ty;
    LSAM_CUDA(c, cudaGraphNodeGetType(nd, &ty));
    if (ty != cudaGraphNodeTypeKernel) continue;
    cudaKernelNodeParams kp;
    LSAM_CUDA(c, cudaGraphKernelNodeGetParams(nd, &kp));
    if (kp.func == (void*)schedule_kernel) gs.n_sched = nd;
    else if (kp.func == c->upd_func) gs.n_upd = nd;
    else if (kp.func == (void*)norm_finalize_kernel && *reinterpret_cast<float**>(kp.kernelParams[6]) != nullptr) gs.n_fin = nd;  // the one that takes rho
  }
  if (!gs.n_sched || !gs.n_upd) return c->fail(LSAM_ERR_CUDA, "graph capture: step kernels not found in the captured graph");
  LSAM_CUDA(c, cudaGraphLaunch(gs.exec, c->stream));  // the capture itself executed nothing: this is the tick
  return LSAM_OK;
}

int graph_replay(lsam_ctx* c, lsam_ctx::GraphSlot& gs, float eta, float rho, int64_t budget) {
  const lsam_config& cfg = c->cfg;
  cudaKernelNodeParams kp;
  SchedArgs sa = make_sched_args(c, c->t, c->idx(), c->stale(), c->ver(), c->slot(), budget, c->async_on ? c->active_buf() : nullptr);
  sa.bind();
  LSAM_CUDA(c, cudaGraphKernelNodeGetParams(gs.n_sched, &kp));
  kp.kernelParams = sa.ptrs; kp.extra = nullptr;
  LSAM_CUDA(c, cudaGraphExecKernelNodeSetParams(gs.exec, gs.n_sched, &kp));
  if (gs.n_fin) {
    LSAM_CUDA(c, cudaGraphKernelNodeGetParams(gs.n_fin, &kp));
    FinArgs f;
    f.partial = *reinterpret_cast<const float**>(kp.kernelParams[0]); f.nchunks = *reinterpret_cast<int64_t*>(kp.kernelParams[1]);
    f.nused = *reinterpret_cast<int64_t*>(kp.kernelParams[2]); f.rho = rho; f.gamma = cfg.gamma;
    f.norm_out = *reinterpret_cast<float**>(kp.kernelParams[5]); f.scale_out = *reinterpret_cast<float**>(kp.kernelParams[6]);
    f.status = c->status(); f.active = c->act();
    f.bind();
    kp.kernelParams = f.ptrs; kp.extra = nullptr;
    LSAM_CUDA(c, cudaGraphExecKernelNodeSetParams(gs.exec, gs.n_fin, &kp));
  }
  {
    LSAM_CUDA(c, cudaGraphKernelNodeGetParams(gs.n_upd, &kp));
    UpdateArgs old = *reinterpret_cast<UpdateArgs*>(kp.kernelParams[0]);
    UpdateArgs ua = make_update_args(c, old.g, old.g_mode, old.ldg, old.n, eta);
    void* ptrs[1] = {&ua};
    kp.kernelParams = ptrs; kp.extra = nullptr;
    LSAM_CUDA(c, cudaGraphExecKernelNodeSetParams(gs.exec, gs.n_upd, &kp));
  }
  LSAM_CUDA(c, cudaGraphLaunch(gs.exec, c->stream));
  c->launches += gs.launches;
  return LSAM_OK;
}

void graphs_reset(lsam_ctx* c) {
  for (auto& gs : c->graphs) {
    if (gs.exec) cudaGraphExecDestroy(gs.exec);
    if (gs.graph) cudaGraphDestroy(gs.graph);
    gs = lsam_ctx::GraphSlot();
  }
}

int step_common(lsam_ctx* c, float eta, float rho, bool gather) {
  const lsam_config& cfg = c->cfg;
  const Layout& L = c->L;
  const bool flat = cfg.model == LSAM_MODEL_FLAT;
  if (flat && (!c->eg1 || !c->eg2)) return c->fail(LSAM_ERR_STATE, "FLAT model: call lsam_set_external_grads first");
  const int64_t budget = c->budget();
  if (budget <= 0) return c->fail(LSAM_ERR_STATE, "the sync is due: call lsam_couple before the next lsam_step");
  // centre version current when this tick starts; the entry only counts once the tick has been enqueued (ver_hi below)
  c->ver_ring[c->t & 31] = (int)c->t_y;
  c->ver_hi = c->t + 1;
  if (c->ver_hi - c->ver_lo > 32) c->ver_lo = c->ver_hi - 32;
  if (c->async_on) host_active_mask(cfg, c->t, budget, c->active_host);
  int rc;
  const bool shortcut = rho == 0.f && !flat && !L.g1keep;
  if ((cfg.flags & LSAM_FLAG_CUDA_GRAPH) && !c->prof.on) {
    lsam_ctx::GraphSlot& gs = c->graphs[(gather ? 1 : 0) + (shortcut ? 2 : 0)];
    if (gs.exec) rc = graph_replay(c, gs, eta, rho, budget);
    else if (gs.warm) rc = graph_capture(c, gs, eta, rho, gather, budget);
    else { rc = step_enqueue(c, eta, rho, gather, budget); gs.warm = true; }
  } else {
    rc = step_enqueue(c, eta, rho, gather, budget);
  }
  if (rc != LSAM_OK) {
    c->ver_hi = c->t;  // the tick did not happen
    return rc;
  }
  for (int k = 0; k < cfg.K; ++k) c->t_x[k] += c->async_on ? c->active_host[k] : 1;
  c->t += 1;
  return LSAM_OK;
}

}  // namespace

// =================================================================================================== C ABI
extern "C" {

uint64_t lsam_schedule_hash(uint64_t seed, int tag, uint64_t t, uint64_t k, uint64_t j) {
  return schedule_hash(seed, tag == 0 ? kTagIdx : kTagStale, t, k, j);
}

int64_t lsam_param_count(const lsam_config* cfg) {
  Layout L;
  if (!cfg || !plan(*cfg, L)) return -1;
  return L.d;
}

size_t lsam_workspace_bytes(const lsam_config* cfg) {
  Layout L;
  if (!cfg || !plan(*cfg, L)) return 0;
  return L.total;
}

int lsam_init(lsam_ctx** out, const lsam_config* cfg, const void* d_X, const void* d_Y, const float* d_x0,
              const float* d_y0, void* d_workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!out) return LSAM_ERR_INVALID;
  *out = nullptr;
  if (!cfg || !d_x0 || !d_y0 || !d_workspace) return LSAM_ERR_INVALID;
  Layout L;
  if (!plan(*cfg, L)) return LSAM_ERR_INVALID;
  if (cfg->model != LSAM_MODEL_FLAT && (!d_X || !d_Y)) return LSAM_ERR_INVALID;
  if (workspace_bytes < L.total || (reinterpret_cast<uintptr_t>(d_workspace) & 255) != 0) return LSAM_ERR_WORKSPACE;
  if ((cfg->flags & LSAM_FLAG_CUDA_GRAPH) && cuda_stream == nullptr) return LSAM_ERR_INVALID;  // the default stream cannot be captured
  lsam_ctx* c = new lsam_ctx();
  c->cfg = *cfg;
  c->L = L;
  c->ws = reinterpret_cast<char*>(d_workspace);
  c->stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  c->X = reinterpret_cast<const float*>(d_X);
  c->Y = reinterpret_cast<const uint32_t*>(d_Y);
  c->t_x.assign(cfg->K, 0);
  c->async_on = cfg->active_num > 0 && cfg->active_num < 256;
  c->active_host.assign(cfg->K, 1);
  auto bail = [&](int code) { delete c; return code; };
  // tensor-core path: decided once per context
  const bool mlp = cfg->model == LSAM_MODEL_MLP || cfg->model == LSAM_MODEL_RESMLP;
  bool tc_ok = false;
  if (mlp && cfg->gemm_dtype == LSAM_GEMM_BF16 && cfg->gemm_impl != LSAM_IMPL_SIMT) tc_ok = tc_supported(*cfg);
  if (L.x3) tc_ok = tc_supported(*cfg);  // fp32 GEMMs as three bf16 planes per operand
  if (cfg->gemm_impl >= LSAM_IMPL_TCGEN05 && !tc_ok) return bail(LSAM_ERR_INVALID);
  c->use_tc = tc_ok;
  c->grads_bf16 = tc_ok && !L.x3 && !(cfg->flags & LSAM_FLAG_GRAD_FP32);
  c->pdl = (cfg->flags & LSAM_FLAG_PDL) != 0;
  if (cfg->flags & LSAM_FLAG_FUSED_UPDATE) {
    if (!tc_ok || L.x3 || cfg->noise_temp > 0.f || cfg->dp_average != 0 || (cfg->flags & LSAM_FLAG_CUDA_GRAPH)) return bail(LSAM_ERR_INVALID);
    c->fused_update = true;
  }
  {
    // the device that holds the workspace is the context's device; it has to be the current one here and in every later call
    cudaPointerAttributes pa;
    int cur = -1;
    if (cudaPointerGetAttributes(&pa, d_workspace) != cudaSuccess || cudaGetDevice(&cur) != cudaSuccess) return bail(LSAM_ERR_CUDA);
    if (pa.type != cudaMemoryTypeDevice && pa.type != cudaMemoryTypeManaged) return bail(LSAM_ERR_INVALID);
    if (pa.type == cudaMemoryTypeDevice && pa.device != cur) return bail(LSAM_ERR_INVALID);
    c->device = cur;
  }
  if (cudaMemsetAsync(c->ws, 0, L.total, c->stream) != cudaSuccess) return bail(LSAM_ERR_CUDA);
  int rc;
  if ((rc = seg_copy<true>(c, d_x0, L.d, c->x(), L.ld, cfg->K)) != LSAM_OK) return bail(rc);
  if ((rc = seg_copy<true>(c, d_y0, L.d, c->yslot(0), L.ld, 1)) != LSAM_OK) return bail(rc);
  if ((rc = refresh_operand_copy(c)) != LSAM_OK) return bail(rc);
  if (c->use_tc) {
    TcBuffers b;
    b.xop = L.x3 ? c->at<bf16>(L.xpl) : c->at<bf16>(L.xop); b.g = c->g(); b.ld = L.ld;
    b.split = L.x3;
    for (int i = 0; i < 9; ++i) { b.act[i] = c->at<bf16>(L.act[i]); b.mask[i] = c->at<uint8_t>(L.mask[i]); }
    b.logits = c->at<float>(L.logits);
    for (int i = 0; i < 2; ++i) { b.dz[i] = c->at<bf16>(L.dz[i]); b.dh[i] = c->at<bf16>(L.dh[i]); }
    b.status = c->status();
    b.ldb = L.ldb;
    b.partial = c->at<float>(L.partial); b.ld_partial = L.nchunks;
    b.g1b = c->at<bf16>(L.g1b);
    c->tc.active = c->act();
    c->tc.allow_pair = cfg->gemm_impl != LSAM_IMPL_TCGEN05_1CTA;
    c->tc.pdl = c->pdl;
    c->pdl = false;  // beside tensor-core GEMMs only the GEMMs take the attribute (see launch_k)
    c->tc.force_pair = cfg->gemm_impl == LSAM_IMPL_TCGEN05_PAIRS;
    c->tc.allow_astat = cfg->gemm_impl != LSAM_IMPL_TCGEN05_1CTA;  // the plain single-CTA kernels stay reachable (and tested) through this setting
    std::vector<TcLayer> tl;
    for (const LayerInfo& li : L.layers) tl.push_back({li.in, li.out, li.w_pad, li.b_pad, li.residual});
    std::string why;
    if (tc_plan(c->tc, *cfg, tl, b, &c->launches, why) != 0) { delete c; return LSAM_ERR_CUDA; }
  }
  *out = c;
  return LSAM_OK;
}

int lsam_step(lsam_ctx* c, float eta, float rho) {
  if (!c) return LSAM_ERR_INVALID;
  if (int rc = c->check_device()) return rc;
  return step_common(c, eta, rho, true);
}

int lsam_step_batch(lsam_ctx* c, float eta, float rho, const float* xb, const void* yb, int on_host, float* h_loss) {
  if (!c || !xb || !yb) return LSAM_ERR_INVALID;
  const lsam_config& cfg = c->cfg;
  if (cfg.model == LSAM_MODEL_FLAT) return c->fail(LSAM_ERR_INVALID, "lsam_step_batch: not available for FLAT");
  if (int rc = c->check_device()) return rc;
  // refused before anything is copied: while the sync is due the call does nothing
  if (c->budget() <= 0) return c->fail(LSAM_ERR_STATE, "the sync is due: call lsam_couple before the next lsam_step");
  const int64_t rows = (int64_t)cfg.K * cfg.batch;
  const int64_t nx = rows * c->L.in0;
  const cudaMemcpyKind kind = on_host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
  const bool lsq = cfg.model == LSAM_MODEL_LSQ;
  float* xdst = lsq ? c->at<float>(c->L.act[0]) : c->at<float>(c->L.xstage);  // classifiers: staged, then stored feature-major
  c->launches += 2;
  LSAM_CUDA(c, cudaMemcpyAsync(xdst, xb, sizeof(float) * nx, kind, c->stream));
  LSAM_CUDA(c, cudaMemcpyAsync(c->at<uint32_t>(c->L.ylab), yb, 4 * rows, kind, c->stream));
  if (!lsq) {
    dim3 grid((unsigned)ceil_div(c->L.in0, 32), (unsigned)ceil_div(cfg.batch, 32), cfg.K);
    if (cfg.gemm_dtype == LSAM_GEMM_BF16 || c->L.x3)
      LAUNCH(c, LSAM_PROF_GATHER, launch_k(c, gather_t_kernel<bf16>, grid, dim3(32, 8), 0, xdst, nullptr, nullptr, rows, cfg.batch, c->L.in0, c->L.ldb, c->at<bf16>(c->L.act[0]), nullptr, c->status(), nullptr, c->in_plane()));
    else
      LAUNCH(c, LSAM_PROF_GATHER, launch_k(c, gather_t_kernel<float>, grid, dim3(32, 8), 0, xdst, nullptr, nullptr, rows, cfg.batch, c->L.in0, c->L.ldb, c->at<float>(c->L.act[0]), nullptr, c->status(), nullptr, (int64_t)0));
  }
  int rc = step_common(c, eta, rho, false);
  if (rc != LSAM_OK) return rc;
  if (h_loss) {
    LSAM_CUDA(c, cudaMemcpyAsync(h_loss, c->loss(), sizeof(float) * cfg.K, cudaMemcpyDeviceToHost, c->stream));
    LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  }
  return LSAM_OK;
}

int lsam_stage_batch(lsam_ctx* c, const float* xb, const void* yb, int on_host) {
  if (!c || !xb || !yb) return LSAM_ERR_INVALID;
  const lsam_config& cfg = c->cfg;
  if (cfg.model == LSAM_MODEL_FLAT) return c->fail(LSAM_ERR_INVALID, "lsam_stage_batch: not available for FLAT");
  if (c->stage_count >= 2) return c->fail(LSAM_ERR_STATE, "lsam_stage_batch: both staging slots are full");
  if (int rc = c->check_device()) return rc;
  if (!c->copy_stream) {
    LSAM_CUDA(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i) {
      LSAM_CUDA(c, cudaEventCreateWithFlags(&c->staged_done[i], cudaEventDisableTiming));
      LSAM_CUDA(c, cudaEventCreateWithFlags(&c->slot_free[i], cudaEventDisableTiming));
    }
  }
  const int slot = (c->stage_head + c->stage_count) & 1;
  const int64_t rows = (int64_t)cfg.K * cfg.batch;
  const cudaMemcpyKind kind = on_host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
  // the slot may still be read by the tick that consumed it last
  if (c->slot_used[slot]) LSAM_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->slot_free[slot], 0));
  LSAM_CUDA(c, cudaMemcpyAsync(c->at<float>(slot ? c->L.xstage2 : c->L.xstage), xb, sizeof(float) * rows * c->L.in0, kind, c->copy_stream));
  LSAM_CUDA(c, cudaMemcpyAsync(c->at<uint32_t>(slot ? c->L.ystage2 : c->L.ystage), yb, 4 * rows, kind, c->copy_stream));
  LSAM_CUDA(c, cudaEventRecord(c->staged_done[slot], c->copy_stream));
  c->stage_count += 1;
  c->launches += 2;
  return LSAM_OK;
}

int lsam_step_staged(lsam_ctx* c, float eta, float rho, float* h_loss) {
  if (!c) return LSAM_ERR_INVALID;
  if (c->stage_count <= 0) return c->fail(LSAM_ERR_STATE, "lsam_step_staged: no staged minibatch (call lsam_stage_batch first)");
  if (int rc = c->check_device()) return rc;
  // refused before the staged minibatch is taken off the queue: it stays staged for the call after lsam_couple
  if (c->budget() <= 0) return c->fail(LSAM_ERR_STATE, "the sync is due: call lsam_couple before the next lsam_step");
  const lsam_config& cfg = c->cfg;
  const int slot = c->stage_head;
  const int64_t rows = (int64_t)cfg.K * cfg.batch;
  const float* xs = c->at<float>(slot ? c->L.xstage2 : c->L.xstage);
  LSAM_CUDA(c, cudaStreamWaitEvent(c->stream, c->staged_done[slot], 0));
  LSAM_CUDA(c, cudaMemcpyAsync(c->at<uint32_t>(c->L.ylab), c->at<uint32_t>(slot ? c->L.ystage2 : c->L.ystage), 4 * rows, cudaMemcpyDeviceToDevice, c->stream));
  if (cfg.model == LSAM_MODEL_LSQ) {
    LSAM_CUDA(c, cudaMemcpyAsync(c->at<float>(c->L.act[0]), xs, sizeof(float) * rows * c->L.in0, cudaMemcpyDeviceToDevice, c->stream));
  } else {
    dim3 grid((unsigned)ceil_div(c->L.in0, 32), (unsigned)ceil_div(cfg.batch, 32), cfg.K);
    if (cfg.gemm_dtype == LSAM_GEMM_BF16 || c->L.x3)
      LAUNCH(c, LSAM_PROF_GATHER, launch_k(c, gather_t_kernel<bf16>, grid, dim3(32, 8), 0, xs, nullptr, nullptr, rows, cfg.batch, c->L.in0, c->L.ldb, c->at<bf16>(c->L.act[0]), nullptr, c->status(), nullptr, c->in_plane()));
    else
      LAUNCH(c, LSAM_PROF_GATHER, launch_k(c, gather_t_kernel<float>, grid, dim3(32, 8), 0, xs, nullptr, nullptr, rows, cfg.batch, c->L.in0, c->L.ldb, c->at<float>(c->L.act[0]), nullptr, c->status(), nullptr, (int64_t)0));
  }
  LSAM_CUDA(c, cudaEventRecord(c->slot_free[slot], c->stream));
  c->slot_used[slot] = true;
  c->stage_head ^= 1;
  c->stage_count -= 1;
  int rc = step_common(c, eta, rho, false);
  if (rc != LSAM_OK) return rc;
  if (h_loss) {
    LSAM_CUDA(c, cudaMemcpyAsync(h_loss, c->loss(), sizeof(float) * cfg.K, cudaMemcpyDeviceToHost, c->stream));
    LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  }
  return LSAM_OK;
}

int lsam_should_couple(const lsam_ctx* c) {
  if (!c) return 0;
  int64_t s = 0;
  for (int64_t v : c->t_x) s += v;
  return (s > 0 && s % ((int64_t)c->cfg.K * c->cfg.tau) == 0) ? 1 : 0;
}

int lsam_couple(lsam_ctx* c) {
  if (!c) return LSAM_ERR_INVALID;
  if (!lsam_should_couple(c)) return c->fail(LSAM_ERR_STATE, "lsam_couple: sync trigger is false");
  if (int rc = c->check_device()) return rc;
  const Layout& L = c->L;
  PhaseRange phase;
  phase.next("lsam S7 couple");
  // divisor n tau of the sync branch: n counts the workers of the whole job (their accumulators have been summed into this one)
  const float inv = 1.0f / ((float)(c->cfg.K_total > 0 ? c->cfg.K_total : c->cfg.K) * (float)c->cfg.tau);
  LAUNCH(c, LSAM_PROF_COUPLE, launch_k(c, couple_kernel, (unsigned)ceil_div(L.ld, 256), 256, 0, 
      c->at<float>(L.acc), c->yslot(c->t_y), c->yslot(c->t_y + 1), c->at<float>(L.gprev), L.ld, inv, c->cfg.beta, c->cfg.eta_prime, c->have_prev ? 1 : 0));
  c->have_prev = true;
  c->t_y += 1;
  for (auto& tx : c->t_x) tx = 0;
  return LSAM_OK;
}

int lsam_acc_buffer(lsam_ctx* c, float** d_acc, int64_t* n) {
  if (!c || !d_acc || !n) return LSAM_ERR_INVALID;
  *d_acc = c->at<float>(c->L.acc);
  *n = c->L.ld;
  return LSAM_OK;
}

int lsam_read_params(lsam_ctx* c, int which, float* dst, int64_t n, int dst_on_device) {
  if (!c || !dst || which < -1 || which >= c->cfg.K) return LSAM_ERR_INVALID;
  if (n < c->L.d) return c->fail(LSAM_ERR_INVALID, "lsam_read_params: destination too small");
  if (int drc = c->check_device()) return drc;
  const float* src = which < 0 ? c->yslot(c->t_y) : c->x() + (size_t)which * c->L.ld;
  int rc;
  if (dst_on_device) return seg_copy<false>(c, src, c->L.ld, dst, c->L.d, 1);
  float* tmp = c->at<float>(c->L.tmp);
  if ((rc = seg_copy<false>(c, src, c->L.ld, tmp, c->L.d, 1)) != LSAM_OK) return rc;
  LSAM_CUDA(c, cudaMemcpyAsync(dst, tmp, sizeof(float) * c->L.d, cudaMemcpyDeviceToHost, c->stream));
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  return LSAM_OK;
}

int lsam_read_schedule(lsam_ctx* c, int64_t t, int32_t* h_idx, int32_t* h_stale, int32_t* h_ver) {
  if (!c || t < 0) return LSAM_ERR_INVALID;
  if (h_ver && t >= c->ver_hi) return c->fail(LSAM_ERR_STATE, "lsam_read_schedule: centre version of a future step");
  if (h_ver && (t > 15 ? t - 15 : 0) < c->ver_lo) return c->fail(LSAM_ERR_STATE, "lsam_read_schedule: the centre-version history of that step is no longer kept (last 16 steps only)");
  const int K = c->cfg.K;
  int32_t* s = c->sched_scratch();
  int rc = launch_schedule(c, t, c->idx_scratch(), s, s + K, s + 2 * K, 0, nullptr);
  if (rc != LSAM_OK) return rc;
  if (h_idx && c->cfg.model != LSAM_MODEL_FLAT)
    LSAM_CUDA(c, cudaMemcpyAsync(h_idx, c->idx_scratch(), 4 * (size_t)K * c->cfg.batch, cudaMemcpyDeviceToHost, c->stream));
  if (h_stale) LSAM_CUDA(c, cudaMemcpyAsync(h_stale, s, 4 * K, cudaMemcpyDeviceToHost, c->stream));
  if (h_ver) LSAM_CUDA(c, cudaMemcpyAsync(h_ver, s + K, 4 * K, cudaMemcpyDeviceToHost, c->stream));
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  return LSAM_OK;
}

int lsam_read_step_info(lsam_ctx* c, float* h_loss, float* h_gnorm1, float* h_gnorm2) {
  if (!c) return LSAM_ERR_INVALID;
  const size_t n = sizeof(float) * c->cfg.K;
  if (h_loss) LSAM_CUDA(c, cudaMemcpyAsync(h_loss, c->loss(), n, cudaMemcpyDeviceToHost, c->stream));
  if (h_gnorm1) LSAM_CUDA(c, cudaMemcpyAsync(h_gnorm1, c->norm1(), n, cudaMemcpyDeviceToHost, c->stream));
  if (h_gnorm2) LSAM_CUDA(c, cudaMemcpyAsync(h_gnorm2, c->norm2(), n, cudaMemcpyDeviceToHost, c->stream));
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  return LSAM_OK;
}

int lsam_read_anchor_gap(lsam_ctx* c, float* h_gap) {
  if (!c || !h_gap) return LSAM_ERR_INVALID;
  const Layout& L = c->L;
  const int K = c->cfg.K;
  const int64_t n = (c->cfg.model == LSAM_MODEL_FLAT) ? L.d : L.ld;  // padding elements are zero in x and in the centre
  float* partial = c->at<float>(L.partial);
  float* out = c->at<float>(L.scalars) + 4 * (size_t)K;
  dim3 grid((unsigned)ceil_div(n, norm_chunk<4>()), K);
  if ((int64_t)grid.x > L.nchunks) return c->fail(LSAM_ERR_WORKSPACE, "anchor gap: partial-sum buffer too small");
  LAUNCH(c, LSAM_PROF_NORM, launch_k(c, gap_sumsq_partial_kernel, grid, kNormThreads, 0, c->x(), L.ld, c->yslot(c->t_y), n, partial, L.nchunks, nullptr, nullptr));
  FinArgs f{partial, L.nchunks, (int64_t)grid.x, 0.f, c->cfg.gamma, out, nullptr, c->status(), nullptr, {}};
  f.bind();
  LAUNCH(c, LSAM_PROF_NORM, launch_p(c, (const void*)norm_finalize_kernel, dim3(K), dim3(256), f.ptrs));
  LSAM_CUDA(c, cudaMemcpyAsync(h_gap, out, sizeof(float) * K, cudaMemcpyDeviceToHost, c->stream));
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  return LSAM_OK;
}

static int read_grads_range(lsam_ctx* c, int pass, int k_begin, int k_end, float* h_dst) {
  if (!c || !h_dst || pass < 1 || pass > 3) return LSAM_ERR_INVALID;
  const Layout& L = c->L;
  const int K = c->cfg.K;
  const bool flat = c->cfg.model == LSAM_MODEL_FLAT;
  float* tmp = c->at<float>(L.tmp);
  (void)K;
  for (int k = k_begin; k < k_end; ++k) {
    int rc = LSAM_OK;
    if (pass == 3) {
      if (c->cfg.gemm_dtype == LSAM_GEMM_BF16) {
        if (!L.xpkeep) return c->fail(LSAM_ERR_STATE, "lsam_read_grads(3) in BF16 mode needs LSAM_FLAG_KEEP_G1");
        int64_t maxlen = 0;
        for (int i = 0; i < L.seg.n; ++i) maxlen = L.seg.len[i] > maxlen ? L.seg.len[i] : maxlen;
        dim3 grid((unsigned)ceil_div(maxlen, 256), L.seg.n, 1);
        LAUNCH(c, LSAM_PROF_COPY, launch_k(c, seg_copy_kernel<false, bf16, float>, grid, 256, 0, c->at<bf16>(L.xpkeep) + (size_t)k * L.ld, L.ld, tmp, L.d, L.seg));
      } else {
        // fp32 GEMMs on the tensor cores: the perturbed point lives in the three operand planes, which the update overwrites; an fp32 copy is kept on request
        if (L.x3 && !(c->cfg.flags & LSAM_FLAG_KEEP_G1)) return c->fail(LSAM_ERR_STATE, "lsam_read_grads(3) with fp32 GEMMs on the tensor cores needs LSAM_FLAG_KEEP_G1");
        rc = seg_copy<false>(c, c->at<float>(L.xop) + (size_t)k * L.ld, L.ld, tmp, L.d, 1);
      }
    } else if (c->cfg.dp_average) {
      // data-parallel mode: every worker used the gradient averaged over the workers
      rc = seg_copy<false>(c, c->at<float>(pass == 1 ? L.gbar1 : L.gbar2), L.ld, tmp, L.d, 1);
    } else if (flat) {
      const float* src = pass == 1 ? c->eg1 : c->eg2;
      if (!src) return c->fail(LSAM_ERR_STATE, "no external gradients set");
      LSAM_CUDA(c, cudaMemcpyAsync(tmp, src + (size_t)k * L.d, sizeof(float) * L.d, cudaMemcpyDeviceToDevice, c->stream));
    } else {
      if (pass == 1 && !L.g1keep) return c->fail(LSAM_ERR_STATE, "lsam_read_grads(1) needs LSAM_FLAG_KEEP_G1");
      if (pass == 2 && c->fused_update) return c->fail(LSAM_ERR_STATE, "lsam_read_grads(2): with LSAM_FLAG_FUSED_UPDATE the descent gradient of the weights is never stored");
      if (c->grads_bf16) {  // both gradients are stored as bf16
        const bf16* srcb = pass == 1 ? c->at<bf16>(L.g1keep) : c->at<bf16>(L.g1b);
        int64_t maxlen = 0;
        for (int i = 0; i < L.seg.n; ++i) maxlen = L.seg.len[i] > maxlen ? L.seg.len[i] : maxlen;
        dim3 grid((unsigned)ceil_div(maxlen, 256), L.seg.n, 1);
        LAUNCH(c, LSAM_PROF_COPY, launch_k(c, seg_copy_kernel<false, bf16, float>, grid, 256, 0, srcb + (size_t)k * L.ld, L.ld, tmp, L.d, L.seg));
      } else {
        const float* src = pass == 1 ? c->at<float>(L.g1keep) : c->g();
        rc = seg_copy<false>(c, src + (size_t)k * L.ld, L.ld, tmp, L.d, 1);
      }
    }
    if (rc != LSAM_OK) return rc;
    LSAM_CUDA(c, cudaMemcpyAsync(h_dst + (size_t)(k - k_begin) * L.d, tmp, sizeof(float) * L.d, cudaMemcpyDeviceToHost, c->stream));
    LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  }
  return LSAM_OK;
}

int lsam_read_grads(lsam_ctx* c, int pass, float* h_dst) {
  if (!c) return LSAM_ERR_INVALID;
  return read_grads_range(c, pass, 0, c->cfg.K, h_dst);
}

int lsam_read_grads_replica(lsam_ctx* c, int pass, int k, float* h_dst) {
  if (!c || k < 0 || k >= c->cfg.K) return LSAM_ERR_INVALID;
  return read_grads_range(c, pass, k, k + 1, h_dst);
}

int lsam_set_external_grads(lsam_ctx* c, const float* d_g1, const float* d_g2) {
  if (!c || !d_g1 || !d_g2) return LSAM_ERR_INVALID;
  if (c->cfg.model != LSAM_MODEL_FLAT) return c->fail(LSAM_ERR_INVALID, "external gradients are for the FLAT model only");
  if (c->eg1 != d_g1 || c->eg2 != d_g2) graphs_reset(c);  // recorded graphs point at the old buffers
  c->eg1 = d_g1;
  c->eg2 = d_g2;
  c->ext_vec4 = ((reinterpret_cast<uintptr_t>(d_g1) | reinterpret_cast<uintptr_t>(d_g2)) & 15) == 0;
  return LSAM_OK;
}

int lsam_write_state(lsam_ctx* c, const float* d_x, const float* d_v, const float* d_y) {
  if (!c) return LSAM_ERR_INVALID;
  int rc;
  if (d_x && (rc = seg_copy<true>(c, d_x, c->L.d, c->x(), c->L.ld, c->cfg.K)) != LSAM_OK) return rc;
  if (d_v && (rc = seg_copy<true>(c, d_v, c->L.d, c->v(), c->L.ld, c->cfg.K)) != LSAM_OK) return rc;
  if (d_y && (rc = seg_copy<true>(c, d_y, c->L.d, c->yslot(c->t_y), c->L.ld, 1)) != LSAM_OK) return rc;
  if (d_x) return refresh_operand_copy(c);
  return LSAM_OK;
}

int lsam_read_state(lsam_ctx* c, float* h_v, float* h_acc, float* h_gprev) {
  if (!c) return LSAM_ERR_INVALID;
  const Layout& L = c->L;
  float* tmp = c->at<float>(L.tmp);
  auto one = [&](const float* src, float* dst) -> int {
    int rc = seg_copy<false>(c, src, L.ld, tmp, L.d, 1);
    if (rc != LSAM_OK) return rc;
    LSAM_CUDA(c, cudaMemcpyAsync(dst, tmp, sizeof(float) * L.d, cudaMemcpyDeviceToHost, c->stream));
    LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
    return LSAM_OK;
  };
  int rc;
  if (h_v)
    for (int k = 0; k < c->cfg.K; ++k)
      if ((rc = one(c->v() + (size_t)k * L.ld, h_v + (size_t)k * L.d)) != LSAM_OK) return rc;
  if (h_acc && (rc = one(c->at<float>(L.acc), h_acc)) != LSAM_OK) return rc;
  if (h_gprev && (rc = one(c->at<float>(L.gprev), h_gprev)) != LSAM_OK) return rc;
  return LSAM_OK;
}

// ---- checkpoint: a host blob = header, per-worker counters, then the raw (padded) state buffers
namespace {
struct CkptHeader {
  char magic[8];
  int64_t d, ld, K, ring, t, t_y, have_prev;
  int32_t ver_hist[16];  // centre version current when step t - 1 - i started (-1: before step 0)
};
const char kCkptMagic[8] = {'L', 'S', 'A', 'M', 'C', 'K', 'P', '1'};
size_t ckpt_floats(const lsam_ctx* c) { return (size_t)c->L.ld * (2 * (size_t)c->cfg.K + 2 + (size_t)c->L.ring); }
}  // namespace

size_t lsam_checkpoint_bytes(const lsam_ctx* c) {
  return c ? sizeof(CkptHeader) + sizeof(int64_t) * (size_t)c->cfg.K + sizeof(float) * ckpt_floats(c) : 0;
}

int lsam_save_checkpoint(lsam_ctx* c, void* h_buf, size_t bytes) {
  if (!c || !h_buf) return LSAM_ERR_INVALID;
  if (bytes < lsam_checkpoint_bytes(c)) return c->fail(LSAM_ERR_INVALID, "lsam_save_checkpoint: buffer smaller than lsam_checkpoint_bytes()");
  if (int drc = c->check_device()) return drc;
  const Layout& L = c->L;
  const size_t K = (size_t)c->cfg.K, ld = (size_t)L.ld;
  CkptHeader h;
  std::memset(&h, 0, sizeof(h));
  std::memcpy(h.magic, kCkptMagic, 8);
  h.d = L.d; h.ld = L.ld; h.K = c->cfg.K; h.ring = L.ring; h.t = c->t; h.t_y = c->t_y; h.have_prev = c->have_prev ? 1 : 0;
  for (int i = 0; i < 16; ++i) {
    const int64_t st = c->t - 1 - i;
    h.ver_hist[i] = st >= 0 ? c->ver_of_step(st) : -1;
  }
  char* p = reinterpret_cast<char*>(h_buf);
  std::memcpy(p, &h, sizeof(h)); p += sizeof(h);
  std::memcpy(p, c->t_x.data(), sizeof(int64_t) * K); p += sizeof(int64_t) * K;
  const struct { const float* src; size_t n; } parts[5] = {
      {c->x(), K * ld}, {c->v(), K * ld}, {c->at<float>(L.acc), ld}, {c->at<float>(L.gprev), ld}, {c->at<float>(L.yring), (size_t)L.ring * ld}};
  for (const auto& q : parts) {
    LSAM_CUDA(c, cudaMemcpyAsync(p, q.src, sizeof(float) * q.n, cudaMemcpyDeviceToHost, c->stream));
    p += sizeof(float) * q.n;
  }
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  return LSAM_OK;
}

int lsam_load_checkpoint(lsam_ctx* c, const void* h_buf, size_t bytes) {
  if (!c || !h_buf) return LSAM_ERR_INVALID;
  if (bytes < lsam_checkpoint_bytes(c)) return c->fail(LSAM_ERR_INVALID, "lsam_load_checkpoint: blob smaller than this context's checkpoint");
  const Layout& L = c->L;
  const size_t K = (size_t)c->cfg.K, ld = (size_t)L.ld;
  CkptHeader h;
  const char* p = reinterpret_cast<const char*>(h_buf);
  std::memcpy(&h, p, sizeof(h)); p += sizeof(h);
  if (std::memcmp(h.magic, kCkptMagic, 8) != 0) return c->fail(LSAM_ERR_INVALID, "lsam_load_checkpoint: not a checkpoint blob");
  if (h.d != L.d || h.ld != L.ld || h.K != c->cfg.K || h.ring != L.ring || h.t < 0 || h.t_y < 0)
    return c->fail(LSAM_ERR_INVALID, "lsam_load_checkpoint: the blob was written by a context of another shape");
  // the blob's counters must describe a state the run can continue from
  std::vector<int64_t> tx(K);
  std::memcpy(tx.data(), p, sizeof(int64_t) * K); p += sizeof(int64_t) * K;
  int64_t done = 0;
  for (int64_t v : tx) {
    if (v < 0) return c->fail(LSAM_ERR_INVALID, "lsam_load_checkpoint: negative worker counter");
    done += v;
  }
  if (done > (int64_t)c->cfg.K * c->cfg.tau) return c->fail(LSAM_ERR_INVALID, "lsam_load_checkpoint: worker counters exceed K tau");
  for (int i = 0; i < 16; ++i) {
    const int64_t st = h.t - 1 - i;
    if (st >= 0 && (h.ver_hist[i] < 0 || h.ver_hist[i] > h.t_y)) return c->fail(LSAM_ERR_INVALID, "lsam_load_checkpoint: centre-version history out of range");
  }
  if (int drc = c->check_device()) return drc;
  // staged minibatches and recorded graphs belong to the run being replaced
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  if (c->copy_stream) LSAM_CUDA(c, cudaStreamSynchronize(c->copy_stream));
  graphs_reset(c);
  c->stage_head = 0; c->stage_count = 0; c->slot_used[0] = c->slot_used[1] = false;
  c->t = h.t; c->t_y = h.t_y; c->have_prev = h.have_prev != 0;
  c->t_x = tx;
  c->ver_hi = h.t;
  c->ver_lo = h.t > 16 ? h.t - 16 : 0;
  for (int i = 0; i < 16; ++i) {
    const int64_t st = h.t - 1 - i;
    if (st >= 0) c->ver_ring[st & 31] = h.ver_hist[i];
  }
  const struct { float* dst; size_t n; } parts[5] = {
      {c->x(), K * ld}, {c->v(), K * ld}, {c->at<float>(L.acc), ld}, {c->at<float>(L.gprev), ld}, {c->at<float>(L.yring), (size_t)L.ring * ld}};
  for (const auto& q : parts) {
    LSAM_CUDA(c, cudaMemcpyAsync(q.dst, p, sizeof(float) * q.n, cudaMemcpyHostToDevice, c->stream));
    p += sizeof(float) * q.n;
  }
  int rc = refresh_operand_copy(c);  // the bf16 operand copy is a function of x
  if (rc != LSAM_OK) return rc;
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));  // the blob may be freed on return
  return LSAM_OK;
}

int lsam_read_counters(const lsam_ctx* c, int64_t* t, int64_t* t_y, int64_t* h_t_x) {
  if (!c) return LSAM_ERR_INVALID;
  if (t) *t = c->t;
  if (t_y) *t_y = c->t_y;
  if (h_t_x) std::memcpy(h_t_x, c->t_x.data(), sizeof(int64_t) * c->t_x.size());
  return LSAM_OK;
}

int lsam_read_active(lsam_ctx* c, int32_t* h_active) {
  if (!c || !h_active) return LSAM_ERR_INVALID;
  if (!c->async_on) {
    for (int k = 0; k < c->cfg.K; ++k) h_active[k] = 1;
    return LSAM_OK;
  }
  LSAM_CUDA(c, cudaMemcpyAsync(h_active, c->active_buf(), sizeof(int32_t) * c->cfg.K, cudaMemcpyDeviceToHost, c->stream));
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  return LSAM_OK;
}

int lsam_status(lsam_ctx* c) {
  if (!c) return LSAM_ERR_INVALID;
  int h = 0;
  LSAM_CUDA(c, cudaMemcpyAsync(&h, c->status(), sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  if (h & STATUS_TIMEOUT) return c->fail(LSAM_ERR_TIMEOUT, "a bounded device-side wait expired");
  if (h & STATUS_NONFINITE) return c->fail(LSAM_ERR_NONFINITE, "a gradient norm was not finite");
  if (h & STATUS_BAD_INDEX) return c->fail(LSAM_ERR_INVALID, "a sample index or label was out of range");
  return LSAM_OK;
}

int lsam_selftest_bounded_wait(lsam_ctx* c, uint32_t polls) {
  if (!c || polls == 0 || polls > (1u << 20)) return LSAM_ERR_INVALID;
  LAUNCH(c, LSAM_PROF_COPY, launch_k(c, wait_selftest_kernel, 1, 32, 0, polls, c->status()));
  return LSAM_OK;
}

int lsam_profile_enable(lsam_ctx* c, int enable) {
  if (!c) return LSAM_ERR_INVALID;
  c->prof.on = enable != 0;
  return LSAM_OK;
}

int lsam_profile_read(lsam_ctx* c, double* h_ms, int64_t* h_launches) {
  if (!c) return LSAM_ERR_INVALID;
  LSAM_CUDA(c, cudaStreamSynchronize(c->stream));
  Profiler& p = c->prof;
  for (size_t i = 0; i < p.used; ++i) {
    float ms = 0.f;
    LSAM_CUDA(c, cudaEventElapsedTime(&ms, p.pool[2 * i], p.pool[2 * i + 1]));
    const int cl = p.cls[i];
    if (h_ms) h_ms[cl] += (double)ms;
    if (h_launches) h_launches[cl] += 1;
  }
  p.used = 0;
  return LSAM_OK;
}

int64_t lsam_launch_count(const lsam_ctx* c) { return c ? c->launches : 0; }
int lsam_uses_tcgen05(const lsam_ctx* c) { return (c && c->use_tc) ? 1 : 0; }
const char* lsam_last_error(const lsam_ctx* c) { return c ? c->err.c_str() : "null context"; }

void lsam_destroy(lsam_ctx* c) {
  if (!c) return;
  for (cudaEvent_t e : c->prof.pool) cudaEventDestroy(e);
  graphs_reset(c);
  for (int i = 0; i < 2; ++i) {
    if (c->staged_done[i]) cudaEventDestroy(c->staged_done[i]);
    if (c->slot_free[i]) cudaEventDestroy(c->slot_free[i]);
  }
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  delete c;
}

}  // extern "C"

// =================================================================================================== no-allocation entry point
// Scratch for lsam_row_norms_static(): per-chunk partial sums of squares.  It lives in the library image, so every
// GPU that loads the library carries this 1 MiB until the process exits, and all calls on a GPU share it.
// In host code this name is only a handle for cudaGetSymbolAddress(); it is NOT a device pointer.
static __device__ __align__(256) float lsam_static_norm_partials[LSAM_STATIC_NORM_MAX_PARTIALS];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_static_mu;
float* g_static_partials_addr[kMaxDevices] = {};  // device address of the array, looked up once per device

int static_fail(int code, const char* msg, char* h_err, size_t h_err_len) {
  if (h_err && h_err_len > 0) std::snprintf(h_err, h_err_len, "%s", msg);
  return code;
}
}  // namespace

extern "C" int lsam_row_norms_static(const float* d_g, int64_t ld, int64_t n, int32_t K, float* d_norm, void* cuda_stream,
                                     char* h_err, size_t h_err_len) {
  if (h_err && h_err_len > 0) h_err[0] = 0;
  if (!d_g || !d_norm || K < 1 || n < 1 || ld < n)
    return static_fail(LSAM_ERR_INVALID, "lsam_row_norms_static: need d_g, d_norm, K >= 1, n >= 1, ld >= n", h_err, h_err_len);
  // 128-bit loads only when every vector lies wholly inside the first n elements of its row
  const bool vec4 = (reinterpret_cast<uintptr_t>(d_g) & 15) == 0 && (ld % 4) == 0 && (n % 4) == 0;
  const int64_t chunk = vec4 ? norm_chunk<4>() : norm_chunk<1>();
  const int64_t nch = ceil_div(n, chunk);
  if (nch > LSAM_STATIC_NORM_MAX_PARTIALS || (int64_t)K * nch > LSAM_STATIC_NORM_MAX_PARTIALS || K > 65535) {
    char msg[256];
    std::snprintf(msg, sizeof msg,
                  "lsam_row_norms_static: K * ceil(n / %lld) = %lld partial sums exceed the built-in scratch of %d (use lsam_step with a workspace)",
                  (long long)chunk, (long long)K * (long long)nch, LSAM_STATIC_NORM_MAX_PARTIALS);
    return static_fail(LSAM_ERR_WORKSPACE, msg, h_err, h_err_len);
  }
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return static_fail(LSAM_ERR_CUDA, "lsam_row_norms_static: cudaGetDevice failed", h_err, h_err_len);
  float* partial = nullptr;
  {
    // set-up, once per device and with that device current: resolve the array's device address
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (!g_static_partials_addr[dev]) {
      void* p = nullptr;
      const cudaError_t e = cudaGetSymbolAddress(&p, lsam_static_norm_partials);
      if (e != cudaSuccess || !p) {
        char msg[256];
        std::snprintf(msg, sizeof msg, "lsam_row_norms_static: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        return static_fail(LSAM_ERR_CUDA, msg, h_err, h_err_len);
      }
      g_static_partials_addr[dev] = static_cast<float*>(p);
    }
    partial = g_static_partials_addr[dev];
  }
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  // Every slot the second pass reads (k * nch + c, c < nch) is written by the first pass of this same call,
  // so the previous call's contents never need clearing.
  dim3 grid((unsigned)nch, (unsigned)K);
  if (vec4) sumsq_partial_kernel<4><<<grid, kNormThreads, 0, stream>>>(d_g, ld, n, partial, nch, nullptr);
  else sumsq_partial_kernel<1><<<grid, kNormThreads, 0, stream>>>(d_g, ld, n, partial, nch, nullptr);
  norm_finalize_kernel<<<K, 256, 0, stream>>>(partial, nch, nch, 0.f, 1.f, d_norm, nullptr, nullptr, nullptr);
  const cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) {
    char msg[256];
    std::snprintf(msg, sizeof msg, "lsam_row_norms_static: launch failed: %s", cudaGetErrorString(e));
    return static_fail(LSAM_ERR_CUDA, msg, h_err, h_err_len);
  }
  return LSAM_OK;
}
