/*
 * cada.h -- C ABI of libcada: one full CADA iteration over M simulated workers on one GPU.
 *
 * Method: "CADA: Communication-Adaptive Distributed Adam" (arXiv 2012.15469).
 *   Problem      Eq. 1        min_theta (1/M) sum_m E[l(theta; xi_m)],  theta in R^p
 *   Main loop    Algorithm 1  broadcast, two minibatch gradients per worker on the SAME sample,
 *                             upload test, upload or skip, server update
 *   CADA1 rule   Eq. 6        skip iff || dtil_m^k - dtil_m^{k-tau} ||^2 <= RHS,
 *                             dtil_m^k = grad l(theta^k; xi_m^k) - grad l(theta~; xi_m^k),
 *                             theta~ a snapshot refreshed every D iterations
 *   CADA2 rule   Eq. 8        skip iff || grad l(theta^k; xi_m^k) - grad l(theta_m^{k-tau}; xi_m^k) ||^2 <= RHS
 *   RHS                       (c / d_max) * sum_{d=1..d_max} || theta^{k+1-d} - theta^{k-d} ||^2
 *   Stochastic LAG  Eq. 4     skip iff || grad l(theta^k; xi_m^k) - (gradient stored at the server) ||^2 <= RHS: one gradient
 *                             per worker-iteration, two iterates AND two samples (the paper's comparator, Section 2.1);
 *                             the paper pairs it with the SGD server theta <- theta - alpha * nabla (CADA_SERVER_SGD)
 *   Forced upload             tau_m^k >= D (Algorithm 1, Section 2.2)
 *   Server       Eqs. 2a-2c   h <- b1 h + (1-b1) nabla,  nabla = (1/M) sum_m (stored gradient of m)
 *                             v  = b2 vhat + (1-b2) nabla^2,  vhat <- max(v, vhat)
 *                             theta <- theta - alpha * h / sqrt(eps + vhat)
 *   Aggregate    Eq. 3        optionally nabla^k = nabla^{k-1} + (1/M) sum_{m uploads} (fresh gradient - last upload of m):
 *                             the server refines one p-vector instead of summing M stored gradients (CADA_AGG_RECURSIVE)
 *   Step size    Theorem 2    optionally alpha_k = alpha / (k + alpha_K0)  (the theorem's 2/mu is `alpha`)
 *
 * Conventions
 *   - "HOST" / "DEVICE" beside a pointer says which address space it must point into.
 *   - The library never allocates or frees device memory: all device state lives in the
 *     caller's `workspace`.  The caller owns X, y, workspace and the stream and keeps them
 *     alive (and unmodified, for X and y) until cada_destroy.
 *   - Every entry point returns a status code (CADA_OK = 0 or a negative CADA_ERR_*); none
 *     throws, aborts or exits.  cada_last_error gives a message for the last failure.
 *   - cada_step is asynchronous on the configured stream; cada_stats / cada_read /
 *     cada_step_host synchronise that stream.
 *   - Kernels of one cada_step call are launched with programmatic stream serialisation and may begin to fetch
 *     rows of X and y while earlier work on the stream still runs: X and y must be complete before cada_create
 *     returns and stay unchanged.  Everything else (indices passed to cada_set_indices, state written through
 *     cada_write) is read only after the preceding work on the stream has completed.
 *   - Calls on one handle must not overlap in time (no internal locking).
 *
 * Layout of theta (p floats, fp32):
 *   CADA_MODEL_LOGISTIC  [ w (n_features) | b (1, if has_bias) ]
 *   CADA_MODEL_SOFTMAX   [ W (n_features x n_classes, row-major) | b (n_classes, if has_bias) ]
 *   CADA_MODEL_MLP2      [ W1 (n_features x n_hidden) | b1 (n_hidden) | W2 (n_hidden x n_classes) | b2 (n_classes) ]
 * Losses (supplement, "Simulation details"): logistic loss with labels +-1, softmax
 * cross-entropy, each plus (lambda/2)||theta||^2 inside every worker's loss; minibatch
 * gradients are means over the `batch` sampled rows.  The MLP rounds the operands of each
 * dense product to bfloat16 (round-to-nearest-even) and accumulates in fp32.
 *
 * Minibatch sampling (Section 1: "a randomly selected ... minibatch"; Assumption 2): `batch`
 * rows drawn uniformly with replacement.  Row j of worker m at iteration k is
 *     SplitMix64(seed, n) mod n_samples[m],   n = (k*M + m)*batch + j,
 * where SplitMix64(seed, n) is the (n+1)-th output of that generator started at `seed`
 * (Steele, Lea, Flood, OOPSLA 2014).  cada_set_indices replaces the stream by explicit indices.
 */
#ifndef CADA_H_
#define CADA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CADA_ABI_VERSION 3u

typedef struct cada_handle cada_handle; /* opaque; created by cada_create, freed by cada_destroy */

enum {
  CADA_OK = 0,
  CADA_ERR_INVALID_ARG = -1, /* NULL pointer, non-positive size, inconsistent shape          */
  CADA_ERR_UNSUPPORTED = -2, /* valid request this build cannot run (shape limits)           */
  CADA_ERR_WORKSPACE = -3,   /* workspace too small or misaligned (256-byte alignment)       */
  CADA_ERR_CUDA = -4,        /* a CUDA runtime call failed; message in cada_last_error       */
  CADA_ERR_NONFINITE = -5,   /* a NaN/Inf reached the upload test (flag, see cada_stats)     */
  CADA_ERR_TIMEOUT = -6      /* a bounded device-side wait ran out                           */
};

enum { CADA_MODEL_LOGISTIC = 0, CADA_MODEL_SOFTMAX = 1, CADA_MODEL_MLP2 = 2 };
enum { CADA_RULE_CADA1 = 1, CADA_RULE_CADA2 = 2, CADA_RULE_LAG = 3 };
enum { CADA_SERVER_AMSGRAD = 0, CADA_SERVER_SGD = 1 };
enum { CADA_AGG_SLOTS = 0, CADA_AGG_RECURSIVE = 1 };
enum { CADA_X_F32 = 0, CADA_X_BF16 = 1 };

/* status_flags bits in cada_stats_t */
enum { CADA_FLAG_NONFINITE = 1, CADA_FLAG_BAD_INDEX = 2, CADA_FLAG_TIMEOUT = 4 };

/* cada_stats_t.path: how one iteration is laid out on the GPU for this configuration */
enum {
  CADA_PATH_THREE_KERNELS = 0,  /* gradient kernel(s), trigger kernel, update kernel              */
  CADA_PATH_ONE_LAUNCH_GRID = 1, /* small logistic: whole iterations in one cooperative launch, one CTA per worker */
  CADA_PATH_ONE_LAUNCH_CLUSTER = 2, /* small logistic, few workers: the same inside one thread-block cluster */
  CADA_PATH_SOFTMAX_CLUSTER = 3, /* softmax, <= 16 classes: a cluster per worker forms the gradient and decides; update kernel */
  CADA_PATH_MLP_CLUSTER = 4,    /* network: a cluster per worker (tensor cores, features split over the CTAs) forms both gradients and decides; update kernel */
  CADA_PATH_MLP_HIDDEN_SPLIT = 5 /* network, <= 128 rows x all features fit one CTA's shared memory: the same with the hidden layer split over the CTAs */
};

/* selectors for cada_read / cada_write (element type, element count) */
enum {
  CADA_BUF_THETA = 0,        /* float  [p]                                                   */
  CADA_BUF_H = 1,            /* float  [p]                                                   */
  CADA_BUF_VHAT = 2,         /* float  [p]                                                   */
  CADA_BUF_G = 3,            /* float  [M*p]   server copy of each worker's last upload      */
  CADA_BUF_THETA_HAT = 4,    /* float  [M*p]   CADA2: iterate at worker m's last upload      */
  CADA_BUF_DELTA_STORED = 5, /* float  [M*p]   CADA1: innovation stored at last upload       */
  CADA_BUF_THETA_TILDE = 6,  /* float  [p]     CADA1: snapshot                               */
  CADA_BUF_TAU = 7,          /* int32  [M]                                                   */
  CADA_BUF_RING = 8,         /* double [d_max] squared step norms, slot k mod d_max          */
  CADA_BUF_GRAD_FRESH = 9,   /* float  [M*p]   grad l(theta^k; xi_m^k) of the last iteration */
  CADA_BUF_INNOV_FRESH = 10, /* float  [M*p]   its difference to the gradient at the old iterate */
  CADA_BUF_LAST_LHS = 11,    /* double [M]     left-hand sides of the last iteration         */
  CADA_BUF_LAST_MASK = 12,   /* uint8  [M]     bit0 = uploaded, bit1 = forced (tau >= D)     */
  CADA_BUF_UPLOADS_PER_WORKER = 13, /* int64 [M]                                             */
  CADA_BUF_HIST_LHS = 14,    /* double [history_capacity*M]  slot (k mod capacity)           */
  CADA_BUF_HIST_RHS = 15,    /* double [history_capacity]                                    */
  CADA_BUF_HIST_MASK = 16,   /* uint8  [history_capacity*M]                                  */
  CADA_BUF_K = 17,           /* int64  [1]     iteration counter                             */
  CADA_BUF_MLP_Z1 = 18,      /* float  [M*2*batch*n_hidden]  MLP only: hidden pre-activations of the */
                             /* last iteration at (theta^k, old iterate), for tie diagnosis  */
  CADA_BUF_NABLA = 19,       /* float  [p]     CADA_AGG_RECURSIVE only: the aggregate nabla^{k-1} of Eq. 3 */
  CADA_BUF_MLP_DZ1 = 20,     /* float  [M*2*batch*n_hidden]   MLP only: gradients of the hidden pre-activations and  */
  CADA_BUF_MLP_DZ2 = 21      /* float  [M*2*batch*n_classes]  of the logits, (P - onehot)/batch, of the last iteration */
                             /* at (theta^k, old iterate), as fp32 BEFORE their rounding to bfloat16: with            */
                             /* CADA_BUF_MLP_Z1 these are the operands whose rounding a reference may need to compare  */
};

typedef struct cada_config {
  uint32_t struct_size;      /* sizeof(cada_config) of the caller                            */
  uint32_t abi_version;      /* CADA_ABI_VERSION                                             */
  int32_t model;             /* CADA_MODEL_*                                                 */
  int32_t rule;              /* CADA_RULE_*                                                  */
  int64_t p;                 /* dim of theta; must equal what the model shape implies        */
  int32_t M;                 /* workers (>= 1)                                               */
  int32_t batch;             /* minibatch rows per worker per iteration (>= 1)               */
  float alpha, beta1, beta2, eps; /* Eqs. 2a-2c; constant step size                          */
  float c;                   /* threshold of Eqs. 6/8; >= 0, +INF allowed (RHS = +INF)       */
  int32_t d_max;             /* window length of the RHS (>= 1)                              */
  int32_t D;                 /* maximum staleness and CADA1 snapshot period (>= 1)           */
  float lambda;              /* L2 coefficient                                               */
  int32_t n_features;        /* columns of X used by the model                               */
  int32_t n_classes;         /* softmax / MLP output width (1 for logistic)                  */
  int32_t n_hidden;          /* MLP hidden width (0 otherwise)                               */
  int32_t has_bias;          /* logistic/softmax: append a constant-1 feature; MLP: must be 1 */
  int32_t x_dtype;           /* CADA_X_F32 (logistic, softmax) or CADA_X_BF16 (MLP)          */
  int32_t history_capacity;  /* iterations of (LHS, RHS, mask) kept in a ring; 0 = none      */
  int32_t host_step_rows;    /* 0, or `batch`: reserve staging for cada_step_host            */
  int32_t server;            /* CADA_SERVER_AMSGRAD (Eqs. 2a-2c) or CADA_SERVER_SGD (Section 2.1)   */
  int64_t ldx;               /* row pitch of X in elements (>= n_features)                   */
  const void* const* X;      /* HOST array[M] of DEVICE pointers, row-major [n_samples[m] x ldx] */
  const void* const* y;      /* HOST array[M] of DEVICE pointers: float +-1 (logistic) or int32 class */
  const int64_t* n_samples;  /* HOST array[M], each >= 1                                     */
  const float* theta0;       /* DEVICE, p floats, copied during cada_create                  */
  const int32_t* tau0;       /* HOST array[M] of initial staleness, or NULL = all D (every   */
                             /* worker uploads at k = 0 through the tau >= D clause)         */
  uint64_t seed;             /* seed of the minibatch index stream                           */
  void* workspace;           /* DEVICE, 256-byte aligned, >= cada_workspace_bytes(cfg)       */
  size_t workspace_bytes;
  void* stream;              /* cudaStream_t all work is enqueued on (NULL = default stream) */
  int32_t aggregate;         /* CADA_AGG_SLOTS: nabla = (1/M) sum of the M stored gradients, in worker order (Eq. 2a); */
                             /* CADA_AGG_RECURSIVE: Eq. 3, only uploading workers' rows are read.  Equal in exact    */
                             /* arithmetic; in fp32 the recursive sum carries its rounding forward                    */
  float alpha_K0;            /* 0: constant alpha.  > 0: alpha_k = alpha / (k + alpha_K0), Theorem 2                  */
  const int32_t* batch_m;    /* HOST array[M] of per-worker minibatch sizes in [1, batch] (the supplement's fixed     */
                             /* batch RATIO with workers of different size), or NULL = all `batch`.  Worker m averages */
                             /* over the first batch_m[m] elements of its index stream; the stream's stride (and the   */
                             /* layouts of cada_set_indices / cada_step_host) stay `batch`.  Not for CADA_MODEL_MLP2   */
  /* Workers split over several handles (one per GPU): Algorithm 1's workers are independent until the server sums their */
  /* gradients (Eq. 2a / Eq. 3), so handle r may hold a subset of the M_total workers of the problem.  All zero (default): */
  /* this handle holds every worker.  Otherwise local worker i is worker m_first + i * m_stride of M_total: it samples    */
  /* the rows that worker samples in the one-handle run, and the server divides by M_total.  Such a handle is stepped     */
  /* with cada_step_local / cada_step_apply; the caller sums the p-vectors across handles in between.                      */
  int32_t M_total;
  int32_t m_first;
  int32_t m_stride;
  int32_t reserved0;
} cada_config;

typedef struct cada_stats_t {
  int64_t k;                 /* iterations completed                                         */
  int64_t uploads_total;     /* the paper's cost metric: number of worker uploads            */
  int64_t uploads_forced;    /* of which by tau >= D                                         */
  int64_t uploads_rule;      /* of which by a violated Eq. 6 / Eq. 8 alone                   */
  int64_t near_ties;         /* decisions with |LHS-RHS| <= 1e-4 * max(LHS, RHS)             */
  int64_t kernel_launches;   /* kernels this handle has launched so far                      */
  double last_rhs;           /* RHS used by the last iteration                               */
  double last_step_sqnorm;   /* ||theta^{k} - theta^{k-1}||^2 of the last iteration          */
  double grad_kernel_ms;     /* summed device time of the dominant kernel while profiling was */
  int64_t grad_kernel_launches; /* on (cada_profile), its launch count, and the iterations   */
  int64_t profiled_iterations;  /* those launches covered.  The dominant kernel is the       */
                             /* two-point gradient kernel, or the one-launch kernel that runs */
                             /* whole iterations of small logistic problems                   */
  int32_t status_flags;      /* CADA_FLAG_* accumulated since create                         */
  int32_t path;              /* CADA_PATH_*: which kernels run this handle's iterations       */
} cada_stats_t;

/* Device bytes the handle needs for this configuration (X, y, theta0, workspace and stream
 * fields are not inspected; batch_m, a HOST array, is read when it is non-NULL).  Returns 0 for
 * an invalid or unsupported configuration. */
size_t cada_workspace_bytes(const cada_config* cfg);

/* Algorithm 1, initialisation: validates cfg, carves the workspace and enqueues the state
 * initialisation (h = vhat = 0, stored gradients 0, theta_hat_m = theta~ = theta0, tau = tau0,
 * window = 0, k = 0).  Host arrays in cfg are copied; they may be freed after the call. */
int cada_create(const cada_config* cfg, cada_handle** out);

/* Algorithm 1, n_iters passes of the loop body (all steps of one iteration run on the
 * device, with no host decision in between).  Asynchronous on the stream. */
int cada_step(cada_handle* h, int32_t n_iters);

/* The iteration of Algorithm 1 in two halves, for workers split over several handles (cada_config.M_total).
 * cada_step_local: the worker side for this handle's workers (both gradients, Eq. 6 / Eq. 8 / Eq. 4, upload or skip, the
 * refresh of the uploaders' records) and the sum over ITS workers of the stored gradients (Eq. 2a; with
 * CADA_AGG_RECURSIVE the sum of its uploaders' innovations, Eq. 3) into dev_sum_out (DEVICE, p floats, caller-owned).
 * The caller then adds the vectors of all handles (one all-reduce of p floats per iteration is the only exchange; the
 * result must be in this GPU's memory) and hands the total to cada_step_apply, which divides by M_total and applies
 * Eqs. 2a-2c (or the SGD server), pushes the squared step norm into the window and advances k.  Every handle applies
 * the same total, so theta, h, vhat and the window stay identical replicas.  Both calls are asynchronous on the stream;
 * counters in cada_stats cover this handle's workers.  With M_total = 0 the pair is equivalent to cada_step(h, 1) up to
 * the order of the sum.  Not available on the one-launch paths (a handle created with M_total != 0 does not use them). */
int cada_step_local(cada_handle* h, float* dev_sum_out);
int cada_step_apply(cada_handle* h, const float* dev_sum);

/* One iteration whose minibatch is handed over from host memory (workers whose data arrive
 * per step): copies host_X ([M][batch][ldx], element type x_dtype) and host_y ([M][batch])
 * to the device, runs the iteration on exactly those rows in order, copies theta^{k+1}
 * (p floats) and the upload mask (M bytes, layout of CADA_BUF_LAST_MASK) back if the
 * pointers are non-NULL, and synchronises.  Needs host_step_rows == batch at create.
 * Pinned host buffers make the copies asynchronous with respect to the host. */
int cada_step_host(cada_handle* h, const void* host_X, const void* host_y, float* host_theta_out,
                   uint8_t* host_mask_out);

/* n iterations of the same kind in one call, for callers that stream their minibatches (Algorithm 1: the workers' data
 * arrive step by step): host_X is [n][M][batch][ldx], host_y [n][M][batch]; host_theta_out ([n][p]) and host_mask_out
 * ([n][M]) receive theta^{k+1} and the upload mask of every iteration if non-NULL.  The staging area has two halves:
 * the minibatch of iteration i+1 is copied in on a second stream (created by the first call; a host
 * resource) while iteration i computes, results go back as each iteration ends, and the call synchronises ONCE, at its
 * end.  Host buffers must be page-locked for the copies to overlap and stay valid until the call returns.  Where the
 * output buffers are page-locked memory the device can address (cudaHostAlloc / cudaHostRegister under unified
 * addressing), a small kernel stores the results into them directly, which keeps copy-engine operations out of the
 * compute stream; otherwise they are copied with cudaMemcpyAsync.
 * Small logistic problems on the one-cluster path (cada_stats_t.path == CADA_PATH_ONE_LAUNCH_CLUSTER) with ALL buffers of
 * the call in such page-locked memory skip the staging: ONE launch runs the n iterations, its fetching warps read the
 * minibatch of iteration i+1 from host_X / host_y over the bus while iteration i computes, and every iteration stores
 * its theta^{k+1} and mask into the output buffers.  Every byte of host_X and host_y still crosses the bus once per
 * call; the results are the same bits as with staged copies. */
int cada_step_host_n(cada_handle* h, int32_t n, const void* host_X, const void* host_y, float* host_theta_out,
                     uint8_t* host_mask_out);

/* Replaces the hashed index stream by explicit row indices for the next n_iters iterations:
 * dev_idx is DEVICE int32 [n_iters][M][batch], kept by reference until consumed.  Passing
 * NULL returns to the hashed stream.  An out-of-range index is clamped and raises
 * CADA_FLAG_BAD_INDEX. */
int cada_set_indices(cada_handle* h, const int32_t* dev_idx, int32_t n_iters);

/* Synchronises the stream and reports counters (uploads are the paper's cost metric, Section 4).  `out` is always
 * filled.  When the device has raised CADA_FLAG_TIMEOUT or CADA_FLAG_NONFINITE the call returns CADA_ERR_TIMEOUT /
 * CADA_ERR_NONFINITE (in that order of precedence) instead of CADA_OK, and from then on cada_step and cada_step_host on
 * this handle return the same code without enqueuing work: the paper's method has no recovery step for either
 * (Algorithm 1's only tolerance device is the maximum staleness D), and the state a timed-out launch leaves is
 * incomplete.  CADA_FLAG_BAD_INDEX is reported in status_flags only. */
int cada_stats(cada_handle* h, cada_stats_t* out);

/* No counterpart in the paper: every device-side wait of the library is bounded.  This sets the bound of the one wait
 * that depends on other CTAs making progress, the flag barrier of CADA_PATH_ONE_LAUNCH_GRID: `polls` reads of one
 * worker's flag (default 2^22, in [0, 2^32 - 1]) after which the CTA raises CADA_FLAG_TIMEOUT, waits for its own
 * outstanding copies and returns; the other CTAs then run into the same bound, so the launch always ends.  Waits on
 * the completion of a CTA's own asynchronous copies keep their built-in bounds.  Takes effect at the next cada_step. */
int cada_set_wait_limit(cada_handle* h, int64_t polls);

/* Section 4 plots loss and accuracy against iterations and uploads.  Evaluates, at the current iterate and over ALL rows
 * of every worker, the objective of Eq. 1, L = (1/M) sum_m [ mean loss of worker m's rows ] + (lambda/2)||theta||^2, and
 * the fraction of all rows classified correctly (sign of the logit / arg-max class).  The MLP is evaluated under the same
 * bf16 operand-rounding contract as its training pass.  Results go to HOST doubles; synchronises the stream.  Supports
 * up to 16 classes and 256 hidden units (CADA_ERR_UNSUPPORTED beyond). */
int cada_eval(cada_handle* h, double* host_loss, double* host_accuracy);

/* Synchronous copies of one state buffer to / from HOST memory; `bytes` must equal the
 * buffer's size.  cada_write of the full state resumes a run (checkpoint / restore). */
int cada_read(cada_handle* h, int32_t which, void* host_dst, size_t bytes);
int cada_write(cada_handle* h, int32_t which, const void* host_src, size_t bytes);

/* Turns per-launch timing of the dominant kernel on (1) or off (0): CUDA events are recorded on
 * the handle's stream around each launch and summed into cada_stats_t. */
int cada_profile(cada_handle* h, int32_t enable);

/* Largest vector length cada_server_update_noalloc accepts (its built-in scratch holds one
 * partial sum per 1024 coordinates: 32 KB + 256 bytes of device memory per GPU). */
#define CADA_NOALLOC_MAX_P (1u << 22)

/* The paper has no counterpart to this entry point; it exists for callers that are not allowed
 * to allocate device memory (a plug-in inside an application whose pool owns the GPU, a real-time
 * loop that may not block on the allocator, a sandboxed extension that only receives buffers)
 * and therefore cannot provide the workspace cada_create asks for.  It applies the server update
 * of Eqs. 2a-2c once, in place, to DEVICE vectors of p floats:
 *     h <- beta1 h + (1-beta1) nabla;  vhat <- max(beta2 vhat + (1-beta2) nabla^2, vhat);
 *     theta <- theta - alpha h / sqrt(eps + vhat);   *step_sqnorm_out (DEVICE double) <- ||delta theta||^2
 * The scratch it needs (block partial sums and a counter) is a fixed array inside the library's
 * device image, present on every GPU that loads the library until the process exits; nothing is
 * allocated or freed, by this call or by anything it calls.  p > CADA_NOALLOC_MAX_P returns
 * CADA_ERR_UNSUPPORTED; NULL pointers, p < 1 or hyper-parameters outside cada_config's ranges
 * return CADA_ERR_INVALID_ARG.  The first call on each device looks up the array's device address
 * with that device current; make that first call outside any stream capture.  All calls on a device
 * share the one array: the call clears the counter it relies on, but two calls whose kernels overlap
 * on the GPU (different streams) race on it -- serialise them.  Asynchronous on `stream`. */
int cada_server_update_noalloc(float* theta, float* h, float* vhat, const float* nabla, int64_t p, float alpha,
                               float beta1, float beta2, float eps, double* step_sqnorm_out, void* stream);

/* Releases host resources; NULL is accepted.  Device memory stays with the caller. */
int cada_destroy(cada_handle* h);

/* Message for the last error on this handle (or of the last failed cada_create when h is NULL). */
const char* cada_last_error(const cada_handle* h);

#ifdef __cplusplus
}
#endif
#endif /* CADA_H_ */
