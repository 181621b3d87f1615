/*
 * lsam.h -- C ABI of the B200 (sm_100a) LSAM worker-step library.
 *
 * What it computes.  K worker replicas of a model are held as stacked parameter tensors on one GPU.
 * One lsam_step() is one tick of the sampling loop of Algorithm 2 ("Asynchronous Distributed LSAM")
 * for every replica k:
 *     g1_k = grad f(x_k; xi_k)                          minibatch gradient (ascent pass)
 *     x~_k = x_k + rho g1_k / (||g1_k|| + gamma)        look-back map, Eq. 3
 *     g2_k = grad f(x~_k; xi_k)                         same minibatch (Theorems 3 and 4)
 *     G    = g2_k + lambda (x_k - y_ver(k))             worker score, Gaussian kernel (Algorithm 1, first update)
 *     v_k <- mu v_k + G ;  x_k <- x_k - eta (G + mu v_k)  Nesterov momentum sampler (Section 4.3)
 *     Acc += x_k ;  t_x[k] += 1                         running sum of post-update iterates (Algorithm 2, sync branch)
 * and lsam_couple() is the sync branch of Algorithm 2:
 *     g' = Acc / (K tau) - y ;  g = g' + beta (g' - g'_prev) ;  y <- y + eta' g ;  Acc <- 0 ; t_x <- 0 ; t_y += 1.
 * The asynchrony of Algorithm 2 is replayed deterministically: replica k reads the centre version that was
 * current s_k steps ago, s_k drawn uniformly from [0, stale_max] by an integer hash of (seed, t, k); the
 * minibatch indices come from the same hash.
 *
 * Conventions.
 *  - Every entry point returns an int status (LSAM_OK = 0); nothing throws or aborts.  lsam_last_error()
 *    gives a message for the last failure of a context.
 *  - Pointers named d_* are DEVICE pointers, h_* are HOST pointers; others say which in their comment.
 *  - The caller owns all device memory (data, workspace) and the CUDA stream; the library owns only the
 *    host-side context.  All work is enqueued on the stream given to lsam_init(); calls are asynchronous
 *    unless they copy to host memory or say that they synchronise.
 *  - Parameter vector of one replica (what x0, y0, lsam_read_params use): the UNPADDED concatenation, layer by
 *    layer, of W_l stored [out, in] row-major then b_l [out].  LSQ: the weight vector w [in] only.  FLAT: flat_d
 *    values.  Inside the workspace each segment start is padded to a multiple of 64 elements.
 */
#ifndef LSAM_H
#define LSAM_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct lsam_ctx lsam_ctx;

enum {
  LSAM_OK = 0,
  LSAM_ERR_INVALID = 1,   /* bad argument or configuration                                          */
  LSAM_ERR_WORKSPACE = 2, /* workspace too small or misaligned                                      */
  LSAM_ERR_STATE = 3,     /* call not allowed in this state (e.g. lsam_couple while the trigger is false) */
  LSAM_ERR_CUDA = 4,      /* a CUDA runtime / driver call failed                                    */
  LSAM_ERR_NONFINITE = 5, /* a gradient norm was NaN or infinite (reported by lsam_status)          */
  LSAM_ERR_TIMEOUT = 6    /* a bounded device-side wait expired (reported by lsam_status)           */
};

enum { LSAM_MODEL_LSQ = 0, LSAM_MODEL_MLP = 1, LSAM_MODEL_RESMLP = 2, LSAM_MODEL_FLAT = 3, LSAM_MODEL_CNN = 4 };
enum { LSAM_GEMM_FP32 = 0, LSAM_GEMM_BF16 = 1 };
/* TCGEN05: tensor-core GEMMs; forward and dgrad with a minibatch tile of 256 samples are run by pairs of CTAs
 * (cta_group::2, 256-row tiles), everything else by single CTAs (128-row tiles); the weight gradient of a minibatch of at
 * most 256 samples keeps its dz block in shared memory over a run of tiles.  TCGEN05_1CTA: single CTAs walking single tiles only;
 * TCGEN05_PAIRS: pairs wherever the kernel supports them (at least 256 rows, minibatch tile of at least 128).
 * LSAM_GEMM_FP32 with LSAM_IMPL_TCGEN05 (LSAM_MODEL_MLP and LSAM_MODEL_RESMLP, every layer's input width a multiple of 8): the fp32 GEMMs
 * run on the bf16 tensor cores.
 * Every GEMM operand a is held as three bf16 planes bf16(a), bf16(a - p0), bf16(a - p0 - p1), whose sum is a, and a product is
 * the sum of the six plane pairs (i, j) with i + j <= 2 accumulated in fp32 (what is left out is below 2^-24 |a||b| per term):
 * fp32 results to within the fp32 tolerances of this library, parameters, gradients and optimiser state in fp32 as in the
 * SIMT path.  AUTO takes this form for an fp32 MLP whose widths allow it and whose largest layer has at least 2^27
 * multiply-adds per GEMM (K * batch * in * out), and the SIMT kernels otherwise. */
enum { LSAM_IMPL_AUTO = 0, LSAM_IMPL_SIMT = 1, LSAM_IMPL_TCGEN05 = 2, LSAM_IMPL_TCGEN05_1CTA = 3, LSAM_IMPL_TCGEN05_PAIRS = 4 };
/* Stationary kernels k(x, y) = phi(x - y) (Corollary 8 and the remark after it).  The worker's pull is
 * grad_x phi(x - y) = w(r) (x - y), r = ||x_k - y|| with y the centre version the worker reads; the centre update is
 * the one Algorithm 2 states (mean of the iterates minus the centre) for every kernel.
 *   GAUSSIAN   phi = (lambda / 2) r^2,                               w = lambda              (Algorithm 1)
 *   EXP_POWER  phi = (lambda / a) r^a, a = kernel_param in [1, 2],   w = lambda r^(a-2)      (w = 0 at r = 0 for a < 2)
 *   CAUCHY     phi = (lambda s^2 / 2) log(1 + r^2 / s^2), s = kernel_param > 0,  w = lambda / (1 + r^2 / s^2)
 *   MATERN32   exp(-phi) = (1 + c r) exp(-c r), c = sqrt(lambda),    w = lambda / (1 + c r)
 * A non-Gaussian kernel costs one more pass over x per tick (the distances r_k, fixed-order reduction).           */
enum { LSAM_KERNEL_GAUSSIAN = 0, LSAM_KERNEL_EXP_POWER = 1, LSAM_KERNEL_CAUCHY = 2, LSAM_KERNEL_MATERN32 = 3 };
enum {
  LSAM_FLAG_KEEP_G1 = 1,   /* keep copies of the ascent gradient and (BF16 mode, fp32 GEMMs on the tensor cores) of x~ for lsam_read_grads */
  LSAM_FLAG_STEP_INFO = 2, /* also reduce ||g2_k|| every step (one extra read of the gradient buffer)      */
  LSAM_FLAG_CUDA_GRAPH = 4, /* replay each tick as one CUDA graph launch (recorded at the second tick of each variant;
                              for launch-bound small models); needs a non-default stream (lsam_init fails with
                              LSAM_ERR_INVALID otherwise); ignored while profiling is enabled               */
  LSAM_FLAG_GRAD_FP32 = 8,  /* tensor-core path: store g1 and g2 in fp32 instead of bf16 (4 instead of 2 bytes per
                              element written by the weight-gradient GEMM and read back by perturbation and update) */
  LSAM_FLAG_FUSED_UPDATE = 16, /* tensor-core path: apply the worker update of the weights inside the epilogue of the descent-pass
                              weight-gradient GEMM, so that the descent gradient of the weights never reaches memory (biases keep
                              the streaming update kernel).  Needs the tensor-core path, noise_temp = 0, dp_average = 0 and no
                              LSAM_FLAG_CUDA_GRAPH (lsam_init: LSAM_ERR_INVALID otherwise); lsam_read_grads(2) is then unavailable */
  LSAM_FLAG_PDL = 32        /* programmatic dependent launch: kernels of a tick are launched with programmatic stream serialization, so
                              that a kernel's blocks may become resident, and run their set-up, while the kernel before it drains; each
                              kernel waits for all earlier ones before its first access to global memory, so results are those of
                              plain in-order launches, bit for bit.  Taken by the tensor-core GEMMs, and, in contexts without them,
                              by the kernels with small grids (where it was measured to pay); works with and without
                              LSAM_FLAG_CUDA_GRAPH (the edges are recorded into the graph); inert while profiling is enabled    */
};

/* Models.
 *  LSQ    f = (1/(2B)) sum_j (a_j . w - y_j)^2, widths[0] = number of features, no bias, fp32 only.
 *  MLP    h_{l+1} = relu(W_l h_l + b_l), linear head, softmax cross-entropy averaged over the minibatch.
 *  RESMLP as MLP, but every hidden layer with equal input and output width is h_{l+1} = h_l + relu(W_l h_l + b_l).
 *  FLAT   no model: the two gradients of a step are buffers supplied with lsam_set_external_grads().
 *  CNN    n_conv layers of 3x3 convolution (stride 1, zero padding 1) + ReLU + 2x2 max-pooling, then dense layers as in MLP (the paper's
 *         experiments train small convolutional nets, Section 5.1).  widths = channels C0 .. C_nconv, then the dense widths (hidden..., classes);
 *         a row of X is an img_h x img_w image with C0 channels, channel-major (feature = c H W + y W + x: the flattening every later layer uses
 *         too); img_h and img_w divisible by 2^n_conv, batch a multiple of 16.  Parameters: conv W_l [Cout][Cin * 9] (column = ci * 9 + kh * 3 + kw)
 *         then b_l [Cout]; dense layers as in MLP, the first one taking C_nconv (img_h / 2^n_conv) (img_w / 2^n_conv) inputs.  Runs on the SIMT
 *         GEMMs (fp32, or bf16 operands with fp32 accumulation) through an explicit patch matrix.
 * gemm_dtype BF16: matmul operands (weights, biases, inputs, stored activations and backward signals) are
 * rounded to bf16, products accumulate in fp32, all optimiser state (x, v, centre, accumulator) stays fp32.
 * Eq. 3 and the worker update are defined on the gradients as computed.  The SIMT path keeps g1 and g2 in fp32.  The
 * tensor-core path by default STORES them in bf16 (a storage format that saves 12 bytes of traffic per parameter and
 * step; it adds a relative rounding of at most 2^-8 per element, inside the bf16 tolerances; the norms ||g1||, ||g2|| are
 * taken from the fp32 accumulators before the rounding); LSAM_FLAG_GRAD_FP32 makes it store fp32 as well.   */
typedef struct {
  int32_t model;      /* LSAM_MODEL_*                                                               */
  int32_t n_layers;   /* weight matrices (MLP/RESMLP: 1..8; LSQ: 1; FLAT: 0)                        */
  int32_t widths[9];  /* in, hidden..., out: n_layers + 1 entries                                   */
  int32_t K;          /* worker replicas, the paper's n (Algorithm 2 inputs)                        */
  int32_t batch;      /* per-worker minibatch size B                                                */
  int32_t gemm_dtype; /* LSAM_GEMM_*                                                                */
  int32_t gemm_impl;  /* LSAM_IMPL_*: AUTO picks tcgen05 for bf16 shapes it supports, else SIMT; a TCGEN05* value
                         the configuration cannot run on (see above) makes lsam_init return LSAM_ERR_INVALID */
  int32_t nesterov;   /* 1: Nesterov form (Section 4.3); 0: heavy-ball x <- x - eta v               */
  int32_t tau;        /* sync period tau                                                            */
  int32_t stale_max;  /* staleness uniform in [0, stale_max], 0 = every worker reads the current centre; <= 15 */
  int32_t flags;      /* LSAM_FLAG_*                                                                */
  int64_t n_samples;  /* rows of the dataset                                                        */
  int64_t flat_d;     /* FLAT only: vector length                                                   */
  uint64_t seed;      /* schedule seed: indices and staleness are pure functions of (seed, t, k, j) */
  float mu;           /* worker momentum                                                            */
  float gamma;        /* stabiliser gamma > 0 of Eq. 3                                              */
  float lambda;       /* pull strength lambda (the rule lambda0/(eta tau) of Appendix D is the caller's) */
  float beta;         /* centre look-ahead factor beta (Section 4.2)                                */
  float eta_prime;    /* centre step size eta'                                                      */
  int32_t active_num; /* asynchronous progress: a worker is ready at a tick with probability active_num/256;
                         0 or 256 = every worker steps at every tick (lock-step)                     */
  float noise_temp;   /* Langevin temperature T >= 0 (Section 4.1): x += sqrt(2 eta T) N(0, I) after the step,
                         normals from Philox4x32-10 keyed by (seed, tick, worker, segment, offset); 0 = none */
  int32_t K_total;    /* workers of the whole job, n of Algorithm 2, when this context holds only a shard of them
                         (one context per GPU); 0 = K, a single context holding every worker                  */
  int32_t k_offset;   /* global index of this context's worker 0; workers k_offset .. k_offset + K - 1 live here */
  int32_t kernel_kind; /* LSAM_KERNEL_*: the stationary kernel k(x, y) = phi(x - y) that couples a worker to the centre       */
  float kernel_param;  /* EXP_POWER: exponent a in [1, 2]; CAUCHY: scale s > 0; others: unused                                */
  int32_t dp_average;  /* 1: synchronous data parallelism (the DP-SGD / DP-SAM baselines of Section 5.2): both gradients of a
                          tick are averaged over the K workers before they are used (perturbation along the averaged gradient
                          and its norm, update with the averaged descent gradient).  Workers that start equal stay equal;
                          lock-step schedule only, one context holds the whole job.  rho = 0 gives DP-SGD.                   */
  int32_t n_conv;      /* CNN: number of convolution layers (the first n_conv of the n_layers)                                */
  int32_t img_h, img_w; /* CNN: input image size                                                                              */
} lsam_config;

/* Unpadded parameter count d of one replica, or -1 if the configuration is invalid. */
int64_t lsam_param_count(const lsam_config* cfg);

/* Bytes of device workspace lsam_init() needs for this configuration (0 if invalid).  Host-only call. */
size_t lsam_workspace_bytes(const lsam_config* cfg);

/* Create a context (Algorithm 2, initialisation line: workers x0, centre y0, counters zero).
 *  d_X  [n_samples, widths[0]] fp32 row-major, device, BORROWED until lsam_destroy (NULL for FLAT).
 *  d_Y  device, borrowed: fp32 targets [n_samples] (LSQ) or int32 labels (MLP/RESMLP); NULL for FLAT.
 *  d_x0 [K, d] fp32 device, d_y0 [d] fp32 device: copied into the workspace.
 *  d_workspace: >= lsam_workspace_bytes() bytes, 256-byte aligned, owned by the caller, must outlive the context.
 *  cuda_stream: a cudaStream_t (NULL = default stream).
 * d_x0 and d_y0 are read, and d_X / d_Y are read by every later tick, ON cuda_stream: whatever produced them must be ordered before
 * this call on that stream (a non-blocking side stream does not wait for the default stream: synchronise or use an event first).
 * Errors: LSAM_ERR_INVALID, LSAM_ERR_WORKSPACE, LSAM_ERR_CUDA; *out is NULL on failure. */
int lsam_init(lsam_ctx** out, const lsam_config* cfg, const void* d_X, const void* d_Y, const float* d_x0,
              const float* d_y0, void* d_workspace, size_t workspace_bytes, void* cuda_stream);

/* One worker tick (sampling loop of Algorithm 2; Eq. 3; Algorithm 1, first update).  Every ready worker steps once,
 * but no more workers than are still missing to K tau iterations since the last sync: ready workers are served in the
 * order of a seeded key and the rest wait, as the workers of the paper block on the request queue while the servers run
 * the distributed step (Appendix C.1).  While a sync is due the call returns LSAM_ERR_STATE and does nothing.
 * The minibatch is drawn by the seeded schedule.  eta and rho are per call, so any schedule (eta0/sqrt(t+1),
 * rho0/sqrt(t+1), step decay) is the caller's.  Asynchronous on the context's stream. */
int lsam_step(lsam_ctx* ctx, float eta, float rho);

/* Same tick, but the minibatch is supplied by the caller instead of gathered from the resident dataset:
 *  xb [K, B, widths[0]] fp32, yb [K, B] (fp32 targets or int32 labels); both on the host (on_host = 1, copied
 *  with cudaMemcpyAsync on the stream; use pinned memory) or on the device (on_host = 0).
 *  h_loss (nullable, host [K]): receives the minibatch loss at x_k; if given, the call synchronises the stream.
 * The staleness part of the schedule is unchanged.  Not available for FLAT. */
int lsam_step_batch(lsam_ctx* ctx, float eta, float rho, const float* xb, const void* yb, int on_host, float* h_loss);

/* Prefetching variant of lsam_step_batch: lsam_stage_batch copies a minibatch (same layout) into one of two staging
 * slots on a copy stream owned by the context, so that the transfer overlaps the tick in flight; lsam_step_staged then
 * runs one tick on the oldest staged minibatch.  xb / yb must stay valid until the lsam_step_staged that consumes them
 * has returned with h_loss != NULL, or the stream has been synchronised; a device source must be complete before
 * lsam_stage_batch is called (the copy stream does not wait for the caller's streams).
 * LSAM_ERR_STATE: both slots full / none staged.
 * The copy stream and its events are host-side objects (no device memory is allocated). */
int lsam_stage_batch(lsam_ctx* ctx, const float* xb, const void* yb, int on_host);
int lsam_step_staged(lsam_ctx* ctx, float eta, float rho, float* h_loss);

/* Sync branch of Algorithm 2 (centre update with look-ahead, counters reset).  Returns LSAM_ERR_STATE and does
 * nothing when the trigger (sum_k t_x[k] > 0 and sum_k t_x[k] mod K tau == 0) is false. */
int lsam_couple(lsam_ctx* ctx);

/* Workers sharded over several contexts (K_total > K; Section 4 deploys one worker per GPU).  Between syncs the
 * workers are independent; the sync branch of Algorithm 2 needs one exchange, the sum over ALL workers of their
 * iterate accumulators.  Each context accumulates the iterates of its own workers; when the trigger holds the caller
 * sums the accumulators of all contexts element by element into every one of them (an all-reduce over the GPUs,
 * ordered with the context's stream) and then calls lsam_couple() on each: every context applies the same centre
 * update, dividing by K_total tau, so the centres stay identical without a broadcast.
 * The schedule (minibatch rows, staleness, noise keys) is keyed by the GLOBAL worker index k_offset + k, so a sharded
 * run reproduces the run of one context with K_total workers up to the order of the floating-point sum.
 * Lock-step schedule only (active_num 0 or 256): the serving order of unequal progress is a global decision.
 *  *d_acc  receives the device address of the accumulator, *n the number of floats to sum (the padded row length;
 *          padding elements are zero in every context).  The buffer lives in the caller's workspace. */
int lsam_acc_buffer(lsam_ctx* ctx, float** d_acc, int64_t* n);
/* 1 if the trigger of the sync branch holds, else 0.  Host-only. */
int lsam_should_couple(const lsam_ctx* ctx);

/* Copy the unpadded parameters of replica `which` (0..K-1) or of the current centre (which = -1) to dst [n >= d].
 * dst_on_device = 0: dst is host memory and the call synchronises the stream; 1: device memory, stream-ordered. */
int lsam_read_params(lsam_ctx* ctx, int which, float* dst, int64_t n, int dst_on_device);

/* ---- helpers (tests, checkpointing, measurement) ---- */
/* Schedule of step t: h_idx [K, B] minibatch rows, h_stale [K], h_ver [K] centre version read (any may be NULL).
 * idx and stale are defined for every t >= 0; ver only for the last 16 steps taken (else LSAM_ERR_STATE).
 * Computed by the device kernel the step itself uses; synchronises. */
int lsam_read_schedule(lsam_ctx* ctx, int64_t t, int32_t* h_idx, int32_t* h_stale, int32_t* h_ver);
/* Of the last step: minibatch loss at x_k, ||g1_k||, ||g2_k|| (host [K] each, nullable; ||g2|| needs
 * LSAM_FLAG_STEP_INFO, else it reads 0).  Synchronises. */
int lsam_read_step_info(lsam_ctx* ctx, float* h_loss, float* h_gnorm1, float* h_gnorm2);
/* Anchor gap of every worker, ||x_k - y|| with y the current centre (the quantity z_t = x_t - y_t that Lemma 5 bounds):
 * h_gap [K], host.  Two-pass fixed-order reduction over one read of x; synchronises.  A monitoring call, not part of a tick. */
int lsam_read_anchor_gap(lsam_ctx* ctx, float* h_gap);
/* Of the last step: pass = 1 ascent gradient (needs LSAM_FLAG_KEEP_G1), 2 descent gradient, 3 perturbed point x~
 * (as stored: rounded to bf16 in BF16 mode, where it also needs LSAM_FLAG_KEEP_G1 because the operand buffer
 * is reused by the update; the same holds for fp32 GEMMs on the tensor cores, whose operand planes are reused).
 * h_dst [K, d] unpadded, host; LSAM_ERR_STATE where the flag is missing.  Synchronises. */
int lsam_read_grads(lsam_ctx* ctx, int pass, float* h_dst);
/* Same for the single replica k: h_dst [d]. */
int lsam_read_grads_replica(lsam_ctx* ctx, int pass, int k, float* h_dst);
/* FLAT only: device buffers [K, d] fp32 (row stride d) holding g1 and g2 for the following steps; borrowed. */
int lsam_set_external_grads(lsam_ctx* ctx, const float* d_g1, const float* d_g2);
/* Overwrite worker iterates x [K, d], momentum v [K, d] and the CURRENT centre y [d] (device pointers, any may be
 * NULL) -- teacher forcing and resume.  Counters and the centre history are left as they are. */
int lsam_write_state(lsam_ctx* ctx, const float* d_x, const float* d_v, const float* d_y);
/* Read back momentum buffers and accumulator for checkpointing: h_v [K, d], h_acc [d], h_gprev [d] (nullable). Synchronises. */
int lsam_read_state(lsam_ctx* ctx, float* h_v, float* h_acc, float* h_gprev);
/* Checkpoint and resume.  lsam_save_checkpoint writes the whole state of the run -- worker iterates, momentum buffers, the
 * iterate accumulator, g'_prev, every centre version a stale read can still reach, the counters t, t_y, t_x and the
 * recent centre-version history -- into a host buffer of lsam_checkpoint_bytes() bytes (synchronises the stream).
 * lsam_load_checkpoint restores it into a context created with the same model, K and stale_max (x0 / y0 given to that
 * lsam_init are overwritten; hyper-parameters passed per call or held in the new configuration are the new context's).
 * Because minibatch rows, staleness, worker readiness and noise are pure functions of (seed, tick, worker, ...), the
 * resumed run continues bit for bit as the saved one would have, given the same seed and hyper-parameters.
 * The blob holds the library's padded layout and is meant for the same library build; a blob of another shape is refused
 * with LSAM_ERR_INVALID.  Minibatches staged with lsam_stage_batch are not part of the state.  (No counterpart in the paper.) */
size_t lsam_checkpoint_bytes(const lsam_ctx* ctx);
int lsam_save_checkpoint(lsam_ctx* ctx, void* h_buf, size_t bytes);
int lsam_load_checkpoint(lsam_ctx* ctx, const void* h_buf, size_t bytes);
/* Which workers stepped at the last tick: h_active [K], 1 = stepped (computed by the device schedule kernel).  Synchronises. */
int lsam_read_active(lsam_ctx* ctx, int32_t* h_active);
/* Counters: steps taken t, centre version t_y, per-worker t_x [K] (host, nullable). */
int lsam_read_counters(const lsam_ctx* ctx, int64_t* t, int64_t* t_y, int64_t* h_t_x);
/* Synchronise the stream and map the device status word to LSAM_OK / LSAM_ERR_NONFINITE / LSAM_ERR_TIMEOUT. */
int lsam_status(lsam_ctx* ctx);
/* Exercises the failure path of the device-side waits without a failure.  Every wait inside the tensor-core kernels (on a
 * TMA load, an MMA completion, a drained accumulator) polls its barrier a bounded number of times; when the bound is hit the
 * kernel sets a timeout bit in the status word and ends normally, and lsam_status() then returns LSAM_ERR_TIMEOUT.  This
 * call enqueues a one-thread kernel that runs that same wait, `polls` times (1 .. 2^20), on a barrier that nothing completes.
 * The status word is sticky: use a context you are about to destroy.  (No counterpart in the paper.) */
int lsam_selftest_bounded_wait(lsam_ctx* ctx, uint32_t polls);
/* Per-kernel-class device timing.  enable != 0: every launch of the following steps is bracketed by CUDA events
 * on the context's stream.  lsam_profile_read synchronises, adds the elapsed times to ms[c] and the launch counts
 * to launches[c] for c < LSAM_PROF_CLASSES (host arrays), and clears the record. */
enum {
  LSAM_PROF_SCHEDULE = 0, LSAM_PROF_GATHER, LSAM_PROF_GEMM_FWD, LSAM_PROF_GEMM_DGRAD, LSAM_PROF_GEMM_WGRAD,
  LSAM_PROF_LOSS, LSAM_PROF_BIAS_GRAD, LSAM_PROF_LSQ_GRAD, LSAM_PROF_NORM, LSAM_PROF_PERTURB, LSAM_PROF_UPDATE,
  LSAM_PROF_COUPLE, LSAM_PROF_COPY, LSAM_PROF_CLASSES
};
int lsam_profile_enable(lsam_ctx* ctx, int enable);
int lsam_profile_read(lsam_ctx* ctx, double* h_ms, int64_t* h_launches);
/* Kernels launched by this context since it was created. */
int64_t lsam_launch_count(const lsam_ctx* ctx);
/* 1 if the model GEMMs of this context run on the tcgen05 tensor-core path, 0 if on the SIMT path. */
int lsam_uses_tcgen05(const lsam_ctx* ctx);
const char* lsam_last_error(const lsam_ctx* ctx);
/* Frees the host context only; the caller frees the workspace. */
void lsam_destroy(lsam_ctx* ctx);

/* Host-side statement of the schedule hash, H(seed, tag, t, k, j) = mix(mix(mix(seed ^ tag) + t) + (k 2^20 + j))
 * with mix the SplitMix64 finaliser; tag 0 = minibatch index stream, 1 = staleness stream. */
uint64_t lsam_schedule_hash(uint64_t seed, int tag, uint64_t t, uint64_t k, uint64_t j);

/* Row norms without any allocation.  (The paper has no counterpart: this is a convenience of the library.)
 * For callers that must not allocate device memory -- code running inside a memory pool that has already handed
 * out the whole GPU, plug-ins that are only given their input and output buffers, latency-critical loops where a
 * cudaMalloc would synchronise the device -- this computes norm[k] = sqrt(sum_{j<n} g[k*ld + j]^2) for k < K with
 * the same two-pass, fixed-order reduction that lsam_step() uses for ||g1_k||, but keeps the per-chunk partial sums
 * in an array that is part of the library image instead of a caller workspace.
 *  d_g    device, [K, ld] fp32 rows of which the first n elements are reduced (ld >= n).
 *  d_norm device, [K] fp32 output.
 *  cuda_stream  a cudaStream_t (NULL = default stream); the call is asynchronous on it.
 *  h_err  nullable host buffer of h_err_len bytes that receives a message when the call fails.
 * Limit: K * ceil(n / C) <= LSAM_STATIC_NORM_MAX_PARTIALS, with C = 8192 elements when d_g is 16-byte aligned and
 * ld is a multiple of 4, else C = 2048.  Larger problems are refused with LSAM_ERR_WORKSPACE and nothing is launched.
 * The array (LSAM_STATIC_NORM_MAX_PARTIALS floats = 1 MiB) is held by every GPU that loads the library until the
 * process exits.  All calls on one GPU share it and it keeps the previous call's contents; every slot a call reads
 * it has written itself first, so nothing needs clearing, but two calls that overlap on the GPU (different streams,
 * or different host threads) race on it: serialise them.  The first call on each device looks up the array's device
 * address (with that device current); make that first call outside any stream capture.
 * No cudaMalloc, cudaFree or other allocating routine is called.  Errors: LSAM_ERR_INVALID, LSAM_ERR_WORKSPACE,
 * LSAM_ERR_CUDA. */
#define LSAM_STATIC_NORM_MAX_PARTIALS 262144
int lsam_row_norms_static(const float* d_g, int64_t ld, int64_t n, int32_t K, float* d_norm, void* cuda_stream,
                          char* h_err, size_t h_err_len);

#ifdef __cplusplus
}
#endif
#endif
