/*
 * lsam_oracle.h -- CPU oracle for the per-worker LSAM step and the worker/centre coupling.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, double-precision restatement of
 * Algorithm 2 (asynchronous distributed LSAM) with the SAM perturbation of Eq. 3 and the
 * Gaussian-kernel pull of Algorithm 1 (first update line); optionally the pull of another
 * stationary kernel (Corollary 8), or the synchronous gradient averaging of the DP baselines.  It shares no code with the CUDA
 * library and must never be reached from the product path: only the test-suite, the smoke
 * check and the benchmark's CPU-baseline leg may load it.
 *
 * Every function takes HOST pointers.  Parameters and optimiser state are double.
 * The parameter vector of one replica is the unpadded concatenation, layer by layer, of
 * W_l stored [out, in] row-major followed by b_l ([out]).  The least-squares model has a
 * single weight vector w [in] and no bias.  The FLAT model has no data: both gradients of a
 * step are supplied by the caller.
 *
 * Parity status of the pieces (what pins them independently of this file is listed in the
 * test-suite): schedule hash, gradients, perturbation, worker update, centre update are
 * pinned; free-running trajectories and the default hyper-parameters are "parity unpinned"
 * (the paper prints no worked numerical example).
 */
#ifndef LSAM_ORACLE_H
#define LSAM_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* CNN: n_conv layers of 3x3 convolution (stride 1, zero padding 1) + ReLU + 2x2 max-pooling, then dense layers as in MLP.
 * widths = channels C0 .. C_nconv, then the dense widths (hidden..., classes); the input is img_h x img_w with C0 channels,
 * a row of X holding it channel-major (feature = c * H * W + h * W + w, the flattening every later layer uses too).
 * Parameters: conv W_l [Cout][Cin * 9] (column = ci * 9 + kh * 3 + kw) then b_l [Cout]; dense layers as in MLP. */
enum { ORACLE_MODEL_LSQ = 0, ORACLE_MODEL_MLP = 1, ORACLE_MODEL_RESMLP = 2, ORACLE_MODEL_FLAT = 3, ORACLE_MODEL_CNN = 4 };
enum { ORACLE_GEMM_FP32 = 0, ORACLE_GEMM_BF16 = 1 };
/* Stationary kernels k(x, y) = phi(x - y) of Corollary 8 and the remark after it; see kernel_phi in the source. */
enum { ORACLE_KERNEL_GAUSSIAN = 0, ORACLE_KERNEL_EXP_POWER = 1, ORACLE_KERNEL_CAUCHY = 2, ORACLE_KERNEL_MATERN32 = 3 };

typedef struct {
  int32_t model;        /* ORACLE_MODEL_*                                                    */
  int32_t n_layers;     /* number of weight matrices (LSQ: 1; FLAT: 0)                       */
  int32_t widths[9];    /* in, hidden..., out : n_layers + 1 entries (LSQ: widths[0] = in)   */
  int32_t K;            /* number of worker replicas (the paper's n)                         */
  int32_t batch;        /* per-worker minibatch size                                         */
  int32_t gemm_dtype;   /* ORACLE_GEMM_*: BF16 rounds matmul operands, accumulates in double */
  int32_t nesterov;     /* 1: x <- x - eta (G + mu v); 0: x <- x - eta v                     */
  int32_t tau;          /* sync period of Algorithm 2                                        */
  int32_t stale_max;    /* staleness drawn uniformly from [0, stale_max]                     */
  int32_t active_num;   /* a worker is ready at a tick with probability active_num/256; 0 or 256: always  */
  int64_t n_samples;    /* rows of X                                                         */
  int64_t flat_d;       /* FLAT model only: length of a replica's vector                     */
  uint64_t seed;
  double mu;            /* worker momentum                                                   */
  double gamma;         /* stabiliser of Eq. 3                                               */
  double lambda;        /* pull strength of the Gaussian kernel                              */
  double beta;          /* centre look-ahead factor                                          */
  double eta_prime;     /* centre step size                                                  */
  double noise_temp;    /* Langevin temperature T: x += sqrt(2 eta T) N(0, I) after the step; 0 = none */
  int32_t kernel_kind;  /* ORACLE_KERNEL_*: the worker's pull is grad phi(x - y) = w(||x - y||) (x - y)           */
  int32_t dp_average;   /* 1: synchronous data parallelism (Section 5.2, DP-SGD / DP-SAM): both gradients of a tick
                           are averaged over the K workers before they are used; lock-step schedule only          */
  double kernel_param;  /* EXP_POWER: exponent a in [1, 2]; CAUCHY: scale s > 0; others: unused                   */
  int32_t n_conv;       /* CNN: number of convolution layers (the first n_conv of the n_layers)                    */
  int32_t img_h, img_w; /* CNN: input image size; both divisible by 2^n_conv                                       */
} oracle_config;

typedef struct oracle_ctx oracle_ctx;

/* Number of parameters of one replica (unpadded), or -1 for an invalid configuration. */
int64_t oracle_param_count(const oracle_config* cfg);

/* X [n_samples, widths[0]] fp32 row-major; Y: float targets [n_samples] for LSQ, int32 labels
 * for MLP/RESMLP, NULL for FLAT.  X and Y are borrowed.  x0 [K, d], y0 [d] are copied.
 * replica_ids (nullable, [K]): global worker ids fed to the schedule hash, so that a small
 * oracle can replay selected workers of a larger run; NULL means 0..K-1.                   */
oracle_ctx* oracle_create(const oracle_config* cfg, const float* X, const void* Y,
                          const double* x0, const double* y0, const int32_t* replica_ids);
void oracle_destroy(oracle_ctx*);

/* One tick of the sampling loop of Algorithm 2 (eta, rho per call): every ready worker steps once, but no more workers
 * than are missing to n tau iterations.  Returns 4 and does nothing while a sync is due (call oracle_couple first). */
int oracle_step(oracle_ctx*, double eta, double rho);
/* 1 when the sync condition of Algorithm 2 holds (and at least one iterate was collected). */
int oracle_should_couple(const oracle_ctx*);
/* The centre update of Algorithm 2; returns non-zero and does nothing if the trigger is false. */
int oracle_couple(oracle_ctx*);
/* The same update for a context that holds only K of the n_total workers of a job (Algorithm 2 runs one worker per
 * device): total_acc [d] is the element-wise sum of the iterate accumulators of ALL n_total workers (this context's
 * included; NULL = only those held here); the divisor is n_total * tau.  Lock-step schedule only (every shard reaches
 * its trigger at the same tick). */
int oracle_couple_sharded(oracle_ctx*, int32_t n_total, const double* total_acc);

/* which in [0,K): replica; which = -1: current centre. dst [d]. */
int oracle_read_params(const oracle_ctx*, int which, double* dst);
/* Any of the pointers may be NULL.  x, v, acc: [K, d]; y, gprev: [d].  acc is the per-replica
 * running sum of post-update iterates since the last sync.                                  */
int oracle_read_state(const oracle_ctx*, double* x, double* v, double* y, double* acc, double* gprev);
/* Overwrite worker iterates, momentum buffers and the CURRENT centre (any pointer may be NULL). */
int oracle_write_state(oracle_ctx*, const double* x, const double* v, const double* y);
/* Schedule of step t (any t >= 0 for idx and stale; ver needs t <= number of steps taken). */
int oracle_read_schedule(const oracle_ctx*, int64_t t, int32_t* idx, int32_t* stale, int32_t* ver);
/* Quantities of the LAST step: loss at x_k, ||g1_k||, ||g2_k||  ([K] each, nullable). */
int oracle_read_step_info(const oracle_ctx*, double* loss, double* gnorm1, double* gnorm2);
/* Gradients and perturbed point of the LAST step, [K, d] each, nullable. */
int oracle_read_grads(const oracle_ctx*, double* g1, double* g2, double* x_pert);
/* FLAT model: gradients used by the next steps, [K, d] fp32, borrowed. */
int oracle_set_external_grads(oracle_ctx*, const float* g1, const float* g2);
/* The kernel phi(r) and the weight w(r) = phi'(r) / r of its gradient, exposed so that they can be pinned against each other. */
double oracle_kernel_phi(int32_t kind, double lambda, double param, double r);
double oracle_kernel_weight(int32_t kind, double lambda, double param, double r);
/* Pull weights w(||x_k - y||) used at the LAST tick ([K]). */
int oracle_read_pull_weights(const oracle_ctx*, double* w);
/* Which workers stepped at the LAST tick ([K], 1 = stepped). */
int oracle_read_active(const oracle_ctx*, int32_t* active);
/* Counters: t (steps), t_y (centre version), t_x [K]. */
int oracle_read_counters(const oracle_ctx*, int64_t* t, int64_t* t_y, int64_t* t_x);

/* Stand-alone pieces, exposed so that they can be pinned one by one. */
/* Mean loss and its gradient at `params` on the minibatch idx[0..n_idx).  grad [d]. */
int oracle_loss_grad(const oracle_config* cfg, const float* X, const void* Y, const double* params,
                     const int32_t* idx, int32_t n_idx, double* loss, double* grad);
/* Logits (MLP/RESMLP: [n_idx, classes]) or predictions (LSQ: [n_idx]) at `params`. */
int oracle_forward(const oracle_config* cfg, const float* X, const double* params,
                   const int32_t* idx, int32_t n_idx, double* out);
/* Philox4x32-10 block (Salmon, Moraes, Dror, Shaw 2011): counter[4], key[2] -> out[4]. */
void oracle_philox4x32_10(const uint32_t* counter, const uint32_t* key, uint32_t* out);
/* The four standard normals of noise group `group` of parameter segment `seg` of worker k at tick t. */
void oracle_noise4(uint64_t seed, uint64_t t, uint64_t k, uint32_t seg, uint64_t group, double* out);
uint64_t oracle_mix64(uint64_t z);
uint64_t oracle_hash(uint64_t seed, uint64_t tag, uint64_t t, uint64_t k, uint64_t j);
uint64_t oracle_tag_idx(void);
uint64_t oracle_tag_stale(void);
uint64_t oracle_tag_active(void);
uint64_t oracle_tag_order(void);
float oracle_bf16_round(float v);
int oracle_num_threads(void);

#ifdef __cplusplus
}
#endif
#endif
