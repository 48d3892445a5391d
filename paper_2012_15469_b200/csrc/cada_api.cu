// Host side of libcada: argument validation, workspace carving, kernel sequencing and the
// extern "C" entry points declared in include/cada.h.  No device memory is allocated here.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <utility>
#include <vector>

#include "../../include/cada.h"
#include "common.cuh"
#include "grad_generic.cuh"
#include "grad_stream.cuh"
#include "grad_softmax.cuh"
#include "fused_small.cuh"
#include "fused_cluster.cuh"
#include "grad_softmax_cluster.cuh"
#include "mlp.cuh"
#include "mlp_tc.cuh"
#include "mlp_cluster.cuh"
#include "mlp_hsplit.cuh"
#include "eval.cuh"
#include "trigger_update.cuh"

using namespace cada;

namespace {

thread_local char g_create_error[512] = "";

struct Region { size_t off = 0, bytes = 0; };

struct Layout {
  Region st, tickets, xtab, ytab, ntab, xtab_s, ytab_s, ntab_s, xtab_s2, ytab_s2;
  Region theta, h, vhat, theta_tilde, G, theta_hat, delta_stored, g_fresh, d_fresh, part;
  Region tau, mask, lhs, upw, ring, norm_part, step_part, hist_lhs, hist_rhs, hist_mask;
  Region stage_x, stage_y, stage_x2, stage_y2;    // two halves: step i+1 is copied in while step i computes
  Region G_alt, fused_flags;
  Region mlp_z1, mlp_dz1, mlp_dz2, mlp_w1img, mlp_dzimg, mlp_small;
  Region eval_part;
  Region btab, nabla, ustab;
  bool mlp_tc_ok = false;    // shape-eligible for the tensor-core products
  MlpTcGeom tg = {};
  Region mlp_ring, mlp_zpart, mlp_csmall, mlp_lhs;
  bool mlp_cluster_ok = false;   // ... and for the one-launch cluster form of the network's gradient
  MlpClusterGeom mcg = {};
  bool mlp_hsplit_ok = false;    // ... and for its hidden-split form (whole products per CTA)
  MlpHsplitGeom mhg = {};
  bool fused_ok = false;     // shape-eligible for the one-launch small-problem kernel
  FusedGeom fg = {};
  size_t total = 0;
  // geometry
  long long ldp = 0;
  int n_chunks = 0, rows_per_chunk = 0, trig_splits = 0, trig_cols = 0, upd_tx = 0, upd_ty = 0, upd_blocks = 0;
  size_t grad_smem = 0;
  // streaming gradient kernel (long-row logistic): shape-eligible?, its geometry and slot count
  bool softmax_fast = false; // the 8-row softmax kernel serves this configuration
  bool stream_ok = false;
  StreamGeom sg = {};
  int stream_slots = 0, stream_nch = 0;
};

constexpr int kStreamCtas = 148;   // one persistent CTA per SM of a B200

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

void carve(Layout& L, Region& r, size_t bytes) {
  r.off = L.total;
  r.bytes = bytes;
  L.total = align_up(L.total + bytes, 256);
}

long long model_dim(const cada_config& c) {
  const long long F = c.n_features, C = c.n_classes, H = c.n_hidden, b = c.has_bias ? 1 : 0;
  switch (c.model) {
    case CADA_MODEL_LOGISTIC: return F + b;
    case CADA_MODEL_SOFTMAX: return F * C + b * C;
    case CADA_MODEL_MLP2: return F * H + H + H * C + C;
  }
  return -1;
}

// Returns CADA_OK and fills L, or an error code with a message in msg.
int plan(const cada_config* c, Layout& L, char* msg, size_t msg_len) {
#define FAIL(code, ...) do { snprintf(msg, msg_len, __VA_ARGS__); return code; } while (0)
  if (!c) FAIL(CADA_ERR_INVALID_ARG, "cfg is NULL");
  if (c->struct_size != sizeof(cada_config)) FAIL(CADA_ERR_INVALID_ARG, "struct_size %u != %zu", c->struct_size, sizeof(cada_config));
  if (c->abi_version != CADA_ABI_VERSION) FAIL(CADA_ERR_INVALID_ARG, "abi_version %u != %u", c->abi_version, CADA_ABI_VERSION);
  if (c->model < 0 || c->model > CADA_MODEL_MLP2) FAIL(CADA_ERR_INVALID_ARG, "unknown model %d", c->model);
  if (c->rule < CADA_RULE_CADA1 || c->rule > CADA_RULE_LAG) FAIL(CADA_ERR_INVALID_ARG, "unknown rule %d", c->rule);
  if (c->server != CADA_SERVER_AMSGRAD && c->server != CADA_SERVER_SGD) FAIL(CADA_ERR_INVALID_ARG, "unknown server %d", c->server);
  if (c->aggregate != CADA_AGG_SLOTS && c->aggregate != CADA_AGG_RECURSIVE) FAIL(CADA_ERR_INVALID_ARG, "unknown aggregate %d", c->aggregate);
  if (!(c->alpha_K0 >= 0.f) || !isfinite(c->alpha_K0)) FAIL(CADA_ERR_INVALID_ARG, "alpha_K0 must be >= 0 and finite");
  if (c->M < 1 || c->batch < 1 || c->d_max < 1 || c->D < 1) FAIL(CADA_ERR_INVALID_ARG, "M, batch, d_max and D must be >= 1");
  if (c->n_features < 1 || c->ldx < c->n_features) FAIL(CADA_ERR_INVALID_ARG, "n_features >= 1 and ldx >= n_features required");
  if (c->model == CADA_MODEL_LOGISTIC && c->n_classes != 1) FAIL(CADA_ERR_INVALID_ARG, "logistic model needs n_classes == 1");
  if (c->model != CADA_MODEL_LOGISTIC && c->n_classes < 2) FAIL(CADA_ERR_INVALID_ARG, "n_classes >= 2 required");
  if (c->model == CADA_MODEL_MLP2 && (c->n_hidden < 1 || !c->has_bias)) FAIL(CADA_ERR_INVALID_ARG, "MLP needs n_hidden >= 1 and has_bias = 1");
  if (c->model != CADA_MODEL_MLP2 && c->n_hidden != 0) FAIL(CADA_ERR_INVALID_ARG, "n_hidden must be 0 for this model");
  if (c->p != model_dim(*c)) FAIL(CADA_ERR_INVALID_ARG, "p = %lld but the model shape implies %lld", (long long)c->p, model_dim(*c));
  if (!(c->alpha > 0.f) || !isfinite(c->alpha)) FAIL(CADA_ERR_INVALID_ARG, "alpha must be positive and finite");
  if (!(c->beta1 >= 0.f && c->beta1 < 1.f) || !(c->beta2 >= 0.f && c->beta2 < 1.f)) FAIL(CADA_ERR_INVALID_ARG, "beta1, beta2 must lie in [0,1)");
  if (!(c->eps >= 0.f) || !isfinite(c->eps)) FAIL(CADA_ERR_INVALID_ARG, "eps must be >= 0 and finite");
  if (!(c->c >= 0.f)) FAIL(CADA_ERR_INVALID_ARG, "c must be >= 0 (+INF allowed)");
  if (!(c->lambda >= 0.f) || !isfinite(c->lambda)) FAIL(CADA_ERR_INVALID_ARG, "lambda must be >= 0 and finite");
  if (c->history_capacity < 0) FAIL(CADA_ERR_INVALID_ARG, "history_capacity must be >= 0");
  if (c->host_step_rows != 0 && c->host_step_rows != c->batch) FAIL(CADA_ERR_INVALID_ARG, "host_step_rows must be 0 or batch");
  if (c->model == CADA_MODEL_MLP2) {
    if (c->x_dtype != CADA_X_BF16) FAIL(CADA_ERR_INVALID_ARG, "the MLP takes bf16 features");
    if (mlp_f2_smem(c->n_hidden, c->n_classes) > 200 * 1024) FAIL(CADA_ERR_UNSUPPORTED, "hidden layer too wide for this build");
  } else if (c->x_dtype != CADA_X_F32) {
    FAIL(CADA_ERR_INVALID_ARG, "logistic and softmax models take fp32 features");
  }
  if ((long long)c->M * c->batch > (1ll << 31) - 1) FAIL(CADA_ERR_UNSUPPORTED, "M*batch too large");
  if (c->M > 65535) FAIL(CADA_ERR_UNSUPPORTED, "M = %d: at most 65535 workers (the worker index is a grid y-coordinate)", c->M);
  if (c->M_total != 0 || c->m_first != 0 || c->m_stride != 0) {
    if (c->M_total < c->M || c->m_first < 0 || c->m_stride < 1 ||
        (long long)c->m_first + (long long)(c->M - 1) * c->m_stride >= c->M_total)
      FAIL(CADA_ERR_INVALID_ARG, "M_total, m_first, m_stride: the M local workers must be workers m_first + i * m_stride < M_total");
  }
  if (c->batch_m) {
    if (c->model == CADA_MODEL_MLP2) FAIL(CADA_ERR_UNSUPPORTED, "per-worker batch sizes are not available for the MLP");
    for (int m = 0; m < c->M; ++m)
      if (c->batch_m[m] < 1 || c->batch_m[m] > c->batch) FAIL(CADA_ERR_INVALID_ARG, "batch_m[%d] = %d outside [1, batch]", m, c->batch_m[m]);
  }

  const long long p = c->p, M = c->M;
  L = Layout();
  L.ldp = (long long)align_up((size_t)p, 32);
  // geometry of the generic gradient kernel
  long long rb = ((long long)c->batch * M + 295) / 296;
  rb = (rb + 7) / 8 * 8;
  if (rb < 8) rb = 8;
  if (rb > 64) rb = 64;
  while (rb > 8 && grad_generic_smem((int)rb, c->n_classes) > 96 * 1024) rb -= 8;
  L.rows_per_chunk = (int)rb;
  L.n_chunks = (c->batch + L.rows_per_chunk - 1) / L.rows_per_chunk;
  if (c->model == CADA_MODEL_MLP2) L.n_chunks = 1;
  if (c->model == CADA_MODEL_SOFTMAX && c->n_classes <= GSM_CMAX &&
      grad_softmax_smem(c->n_features, c->n_classes, c->has_bias ? 1 : 0, false) <= 160 * 1024) {
    L.softmax_fast = true;                                // 8 rows per CTA
    L.rows_per_chunk = GSM_ROWS;
    L.n_chunks = (c->batch + GSM_ROWS - 1) / GSM_ROWS;
  }      // one slot per worker: (gradient, gradient at the old iterate)
  L.grad_smem = grad_generic_smem(L.rows_per_chunk, c->n_classes);
  if (L.grad_smem > 200 * 1024) FAIL(CADA_ERR_UNSUPPORTED, "n_classes too large for the gradient kernel");
  // streaming kernel: binary logistic, rows of 1 KB .. 16 KB that start on 16-byte boundaries
  if (c->model == CADA_MODEL_LOGISTIC && c->n_features % 4 == 0 && c->ldx % 4 == 0 && c->n_features >= 256 &&
      c->n_features <= 4096) {
    StreamGeom g;
    g.row_bytes = (unsigned)c->n_features * 4u;
    g.stage_stride = (unsigned)align_up((size_t)GS_R * g.row_bytes, 128);
    g.n_stages = (int)((232448 - 1024) / g.stage_stride);
    if (g.n_stages > GS_MAX_STAGES) g.n_stages = GS_MAX_STAGES;
    g.units_per_worker = (c->batch + GS_R - 1) / GS_R;
    g.ustart = nullptr;
    // per-worker batch sizes: worker m owns ceil(B_m / R) units, so that CTAs get equal shares of the rows
    std::vector<long long> us((size_t)M + 1, 0);
    for (long long m = 0; m < M; ++m)
      us[m + 1] = us[m] + (c->batch_m ? (c->batch_m[m] + GS_R - 1) / GS_R : g.units_per_worker);
    g.n_units = us[M];
    int slots = 1;
    for (long long m = 0; m < M; ++m) {
      const int lo = stream_cta_of_unit(us[m], g.n_units, kStreamCtas);
      const int hi = stream_cta_of_unit(us[m + 1] - 1, g.n_units, kStreamCtas);
      if (hi - lo + 1 > slots) slots = hi - lo + 1;
    }
    L.stream_ok = g.n_stages >= 2;
    L.sg = g;
    L.stream_slots = slots;
    const int nq = c->n_features / 4;
    L.stream_nch = nq <= GS_CONSUMERS ? 1 : nq <= 2 * GS_CONSUMERS ? 2 : 4;
  }
  // one-launch kernel for small logistic problems: one CTA per worker, short rows
  if (c->model == CADA_MODEL_LOGISTIC && c->M <= kStreamCtas && c->n_features < 256 && c->ldx % 4 == 0 &&
      c->rule != CADA_RULE_LAG && c->server == CADA_SERVER_AMSGRAD && c->aggregate == CADA_AGG_SLOTS && c->M_total == 0)
    L.fused_ok = fused_plan(c->n_features, c->has_bias ? 1 : 0, c->batch, c->d_max, c->rule, c->M, L.fg);
  // trigger kernel
  long long S = (p + 2047) / 2048;                 // about two 128-bit columns per thread
  const long long smin = (296 + M - 1) / M, smax = (p + 1023) / 1024;
  if (S < smin) S = smin;
  if (S > smax) S = smax;
  if (S < 1) S = 1;
  long long cols = (p + S - 1) / S;
  cols = (cols + 3) / 4 * 4;
  L.trig_cols = (int)cols;
  L.trig_splits = (int)((p + cols - 1) / cols);
  // update kernel
  // worker lanes per 4-coordinate group: as many as it takes to put about two blocks' worth of threads on every SM (more lanes measured no faster), at
  // most one per worker and at most 32, rounded down to a power of two; with long iterates one lane walks all workers (no cross-lane sum, every thread
  // takes part in the optimiser step), with short ones the workers are spread over lanes
  const long long groups = (p + 3) / 4;
  long long want = ((long long)kStreamCtas * 2 * UPD_THREADS + groups - 1) / groups;
  if (want > 32) want = 32;
  if (want > M) want = M;
  int ty = 1;
  while (2 * ty <= want) ty *= 2;      // a power of two: the block then has exactly UPD_THREADS threads (whole warps)
  L.upd_ty = ty;
  L.upd_tx = UPD_THREADS / ty;
  L.upd_blocks = (int)((groups + L.upd_tx - 1) / L.upd_tx);

  const size_t vec = (size_t)L.ldp * sizeof(float), mat = vec * (size_t)M;
  carve(L, L.st, sizeof(DevState));
  carve(L, L.tickets, sizeof(unsigned) * (size_t)M);
  carve(L, L.xtab, sizeof(void*) * (size_t)M);
  carve(L, L.ytab, sizeof(void*) * (size_t)M);
  carve(L, L.ntab, sizeof(long long) * (size_t)M);
  carve(L, L.xtab_s, sizeof(void*) * (size_t)M);
  carve(L, L.ytab_s, sizeof(void*) * (size_t)M);
  carve(L, L.ntab_s, sizeof(long long) * (size_t)M);
  carve(L, L.xtab_s2, sizeof(void*) * (size_t)M);
  carve(L, L.ytab_s2, sizeof(void*) * (size_t)M);
  carve(L, L.theta, vec);
  carve(L, L.h, vec);
  carve(L, L.vhat, vec);
  if (c->rule == CADA_RULE_CADA1) carve(L, L.theta_tilde, vec);
  carve(L, L.G, mat);
  if (c->rule == CADA_RULE_CADA2) carve(L, L.theta_hat, mat);
  if (c->rule == CADA_RULE_CADA1) carve(L, L.delta_stored, mat);
  carve(L, L.g_fresh, mat);
  carve(L, L.d_fresh, mat);
  carve(L, L.part, mat * 2 * (size_t)(L.stream_ok && L.stream_slots > L.n_chunks ? L.stream_slots : L.n_chunks));
  carve(L, L.tau, sizeof(int) * (size_t)M);
  carve(L, L.mask, (size_t)M);
  carve(L, L.lhs, sizeof(double) * (size_t)M);
  carve(L, L.upw, sizeof(long long) * (size_t)M);
  carve(L, L.ring, sizeof(double) * (size_t)c->d_max);
  carve(L, L.norm_part, sizeof(double) * (size_t)M * L.trig_splits);
  carve(L, L.step_part, sizeof(double) * (size_t)L.upd_blocks);
  if (c->model == CADA_MODEL_MLP2) {
    const size_t act = sizeof(float) * (size_t)M * 2 * (size_t)c->batch * (size_t)c->n_hidden;
    carve(L, L.mlp_z1, act);
    carve(L, L.mlp_dz1, act);
    carve(L, L.mlp_dz2, sizeof(float) * (size_t)M * 2 * (size_t)c->batch * (size_t)c->n_classes);
    L.mlp_tc_ok = mlp_tc_plan(c->n_features, c->n_hidden, c->n_classes, c->batch, c->M, c->rule, c->ldx, L.tg);
    if (L.mlp_tc_ok) {
      carve(L, L.mlp_w1img, (size_t)L.tg.n_sets * L.tg.w_set_bytes);
      carve(L, L.mlp_dzimg, (size_t)M * 2 * L.tg.dz_bytes);
      carve(L, L.mlp_small, sizeof(float) * (size_t)M * 2 * L.tg.f2_blocks * L.tg.small);
      const bool cl = mlp_cluster_plan(c->n_features, c->n_hidden, c->n_classes, c->batch, c->M, c->rule, L.tg, L.mcg);
      const bool hs = mlp_hsplit_plan(c->n_features, c->n_hidden, c->n_classes, c->batch, c->rule, c->ldx, L.mhg);
      size_t set_bytes = cl ? L.tg.w_set_bytes : 0;
      if (hs && L.mhg.set_bytes > set_bytes) set_bytes = L.mhg.set_bytes;
      const size_t ring = ((size_t)c->D + 1) * set_bytes;              // one operand image per iteration a worker may still refer to
      if ((cl || hs) && ring <= ((size_t)1 << 30)) {
        L.mlp_cluster_ok = cl;
        L.mlp_hsplit_ok = hs;
        carve(L, L.mlp_ring, ring);
        if (cl) {
          carve(L, L.mlp_zpart, L.mcg.zpart_bytes);
          carve(L, L.mlp_csmall, L.mcg.small_bytes);
        }
        carve(L, L.mlp_lhs, sizeof(double) * (size_t)M * MC_MAX_SLICES);
      }
    }
  }
  if (L.fused_ok) {
    carve(L, L.G_alt, mat);
    carve(L, L.fused_flags, sizeof(unsigned) * 2 * (size_t)M);
  }
  carve(L, L.eval_part, sizeof(double) * 2 * (size_t)M * EV_CHUNKS);
  if (c->batch_m) carve(L, L.btab, sizeof(int) * (size_t)M);
  if (c->batch_m && L.stream_ok) carve(L, L.ustab, sizeof(long long) * ((size_t)M + 1));
  if (c->aggregate == CADA_AGG_RECURSIVE) carve(L, L.nabla, vec);
  if (c->history_capacity > 0) {
    carve(L, L.hist_lhs, sizeof(double) * (size_t)M * c->history_capacity);
    carve(L, L.hist_rhs, sizeof(double) * (size_t)c->history_capacity);
    carve(L, L.hist_mask, (size_t)M * c->history_capacity);
  }
  if (c->host_step_rows > 0) {
    const size_t elt = c->x_dtype == CADA_X_BF16 ? 2 : 4;
    carve(L, L.stage_x, (size_t)M * c->batch * (size_t)c->ldx * elt);
    carve(L, L.stage_y, (size_t)M * c->batch * 4);
    carve(L, L.stage_x2, (size_t)M * c->batch * (size_t)c->ldx * elt);
    carve(L, L.stage_y2, (size_t)M * c->batch * 4);
  }
  return CADA_OK;
#undef FAIL
}

struct EventPair { cudaEvent_t a, b; };

}  // namespace

struct cada_handle {
  cada_config cfg;
  Layout L;
  Params P;        // resident data, hashed or explicit indices
  Params Ph;       // staged minibatch (cada_step_host), identity indices
  Params Ph2;      // ... the second staging half (cada_step_host_n alternates between the two)
  cudaStream_t copy_stream;              // created by the first cada_step_host_n call
  cudaEvent_t ev_copied[2], ev_done[2], ev_start;
  bool copy_ready;
  bool half_done;            // cada_step_local has run, cada_step_apply has not yet
  cudaStream_t stream;
  char* ws;
  long long k_host;          // iterations enqueued so far
  long long idx_remaining;   // explicit-index iterations left
  long long launches;
  bool profile;
  bool use_stream;           // the streaming gradient kernel serves this configuration
  bool use_fused;            // whole iterations run in the one-launch kernel
  bool use_cluster;          // ... in its one-cluster form (exchange through distributed shared memory)
  bool stream_ok;            // ... whose streamed form (three minibatch buffers) fits as well: cada_step_host_n may use it
  ClusterGeom cg_stream;
  ClusterGeom cg;
  bool use_softmax_cluster;  // softmax: one cluster per worker forms the gradient and takes the upload decision
  SoftmaxClusterGeom scg;
  bool use_mlp_tc;           // the MLP's large products run on the tensor cores
  bool use_mlp_cluster;      // ... inside one cluster launch per iteration that also takes the upload decision
  bool use_mlp_hsplit;       // ... that launch being the hidden-split kernel (else the feature-split one)
  bool ring_dirty;           // iterates were written from the host: the operand-image ring must be rebuilt before the next step
  long long profiled_iters;
  std::vector<EventPair> pending, spare;
  std::vector<long long> n_samples;   // host copy (evaluation)
  double grad_ms;
  long long grad_launches;
  int device_error;          // CADA_ERR_TIMEOUT / CADA_ERR_NONFINITE once cada_stats has seen the device raise that flag
  unsigned wait_limit;       // polls a CTA of the grid-wide one-launch kernel spends on one flag of its barrier
  char err[512];
};

namespace {

int fail(cada_handle* h, int code, const char* what, cudaError_t e = cudaSuccess) {
  if (h) {
    if (e != cudaSuccess) snprintf(h->err, sizeof h->err, "%s: %s", what, cudaGetErrorString(e));
    else snprintf(h->err, sizeof h->err, "%s", what);
  }
  return code;
}

#define CUDA_TRY(h, call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return fail(h, CADA_ERR_CUDA, #call, e_); } while (0)

// Dynamic shared memory a kernel may be launched with.  The attribute belongs to the kernel, not to a handle: it is always
// raised to the device's limit (less the kernel's static shared memory), so that a handle created later with a smaller
// need does not lower it under an earlier one.
template <typename K>
cudaError_t raise_smem_limit(K kernel) {
  const void* fn = reinterpret_cast<const void*>(kernel);
  int dev = 0, optin = 0;
  cudaFuncAttributes fa;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e == cudaSuccess) e = cudaFuncGetAttributes(&fa, fn);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, optin - (int)fa.sharedSizeBytes);
  return e;
}

template <typename T>
T* at(cada_handle* h, const Region& r) { return r.bytes ? reinterpret_cast<T*>(h->ws + r.off) : nullptr; }

int drain_events(cada_handle* h) {
  for (EventPair& ep : h->pending) {
    float ms = 0.f;
    CUDA_TRY(h, cudaEventSynchronize(ep.b));
    CUDA_TRY(h, cudaEventElapsedTime(&ms, ep.a, ep.b));
    h->grad_ms += ms;
    h->grad_launches += 1;
    h->spare.push_back(ep);
  }
  h->pending.clear();
  return CADA_OK;
}

// Launch with programmatic stream serialisation: the kernel may be scheduled while its predecessor in the stream
// still runs; every kernel launched this way begins with pdl_wait(), which returns when the predecessor has completed.
template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t lc;
  memset(&lc, 0, sizeof lc);
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kernel, std::forward<Args>(args)...);
}

const void* softmax_cluster_kernel_for(int cgp) {
  switch (cgp) {
    case 1: case 2: return (const void*)grad_softmax_cluster_kernel<2>;
    case 3: case 4: return (const void*)grad_softmax_cluster_kernel<4>;
    case 5: return (const void*)grad_softmax_cluster_kernel<5>;
    case 6: return (const void*)grad_softmax_cluster_kernel<6>;
    default: return (const void*)grad_softmax_cluster_kernel<8>;
  }
}

void softmax_cluster_launch_config(const SoftmaxClusterGeom& g, int M, cudaStream_t stream, cudaLaunchConfig_t& lc,
                                   cudaLaunchAttribute* attr) {
  memset(&lc, 0, sizeof lc);
  lc.gridDim = dim3(g.nc, M);
  lc.blockDim = dim3(SC_THREADS);
  lc.dynamicSmemBytes = g.smem_bytes;
  lc.stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = g.nc;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start behind a running update kernel
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 2;
}

// CTAs per worker for the softmax cluster kernel: as many as keep all workers' clusters resident at once with two
// CTAs per SM, at most 8; the first count that plans and can be scheduled wins.
bool choose_softmax_cluster(const cada_config* c, cudaStream_t stream, SoftmaxClusterGeom& out) {
  int start = 296 / c->M;                  // two CTAs fit on an SM; measured on C3: 8 CTAs per worker (160 CTAs) beat 7 (140)
  if (start > SC_MAX_NC) start = SC_MAX_NC;
  if (start < 1) start = 1;
  for (int nc = start; nc >= 1; --nc) {
    SoftmaxClusterGeom g;
    if (!softmax_cluster_plan(c->n_features, c->n_classes, c->has_bias ? 1 : 0, c->batch, nc, g)) continue;
    const void* fn = softmax_cluster_kernel_for(g.cgp);
    if (raise_smem_limit(fn) != cudaSuccess) {
      cudaGetLastError();
      continue;
    }
    cudaLaunchConfig_t lc;
    cudaLaunchAttribute attr[2];
    softmax_cluster_launch_config(g, c->M, stream, lc, attr);
    int n_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&n_clusters, fn, &lc) != cudaSuccess) { cudaGetLastError(); continue; }
    if (n_clusters >= 1) { out = g; return true; }
  }
  return false;
}

void mlp_cluster_launch_config(int ns, unsigned smem_bytes, int M, cudaStream_t stream, cudaLaunchConfig_t& lc, cudaLaunchAttribute* attr) {
  memset(&lc, 0, sizeof lc);
  lc.gridDim = dim3(ns, M);
  lc.blockDim = dim3(MC_THREADS);
  lc.dynamicSmemBytes = smem_bytes;
  lc.stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = ns;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // may start behind a running update kernel
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 2;
}

int launch_grad(cada_handle* h, const Params& P) {
  EventPair ep{};
  if (h->profile) {
    if (h->pending.size() >= 2048) { int rc = drain_events(h); if (rc) return rc; }
    if (!h->spare.empty()) { ep = h->spare.back(); h->spare.pop_back(); }
    else { CUDA_TRY(h, cudaEventCreate(&ep.a)); CUDA_TRY(h, cudaEventCreate(&ep.b)); }
    CUDA_TRY(h, cudaEventRecord(ep.a, h->stream));
  }
  if (h->use_softmax_cluster) {
    Params Pk = P;
    SoftmaxClusterGeom g = h->scg;
    long long k_now = h->k_host;
    void* args[] = {&Pk, &g, &k_now};
    cudaLaunchConfig_t lc;
    cudaLaunchAttribute attr[2];
    softmax_cluster_launch_config(g, P.M, h->stream, lc, attr);
    CUDA_TRY(h, cudaLaunchKernelExC(&lc, softmax_cluster_kernel_for(g.cgp), args));
  } else if (h->use_mlp_cluster) {
    if (h->ring_dirty) {
      const long long groups = ((long long)P.F * P.H / 4 + 255) / 256;
      const int n_sets = P.rule == CADA_RULE_CADA2 ? 1 + P.M : P.rule == CADA_RULE_CADA1 ? 2 : 1;
      mlp_ring_rebuild_kernel<<<dim3((unsigned)groups, n_sets), 256, 0, h->stream>>>(P, h->k_host);
      h->launches += 1;
      h->ring_dirty = false;
    }
    Params Pk = P;
    MlpBufs mb{at<float>(h, h->L.mlp_z1), at<float>(h, h->L.mlp_dz1), at<float>(h, h->L.mlp_dz2)};
    if (h->use_mlp_hsplit) {
      MlpHsplitGeom hg = h->L.mhg;
      double* lhs_part = at<double>(h, h->L.mlp_lhs);
      long long k_now = h->k_host;
      void* args[] = {&Pk, &hg, &mb, &lhs_part, &k_now};
      cudaLaunchConfig_t lc;
      cudaLaunchAttribute attr[2];
      mlp_cluster_launch_config(hg.ns, hg.smem_bytes, P.M, h->stream, lc, attr);
      CUDA_TRY(h, cudaLaunchKernelExC(&lc, (const void*)mlp_hsplit_kernel, args));
    } else {
    MlpTcGeom g = h->L.tg;
    MlpClusterGeom cg = h->L.mcg;
    MlpTcBufs tb{nullptr, at<unsigned char>(h, h->L.mlp_dzimg), nullptr};
    MlpClusterBufs cb{at<float>(h, h->L.mlp_zpart), at<float>(h, h->L.mlp_csmall), at<double>(h, h->L.mlp_lhs)};
    long long k_now = h->k_host;
    void* args[] = {&Pk, &g, &cg, &mb, &tb, &cb, &k_now};
    cudaLaunchConfig_t lc;
    cudaLaunchAttribute attr[2];
    mlp_cluster_launch_config(cg.ns, cg.smem_bytes, P.M, h->stream, lc, attr);
    CUDA_TRY(h, cudaLaunchKernelExC(&lc, (const void*)mlp_cluster_kernel, args));
    }
  } else if (P.model == CADA_MODEL_MLP2 && h->use_mlp_tc) {
    MlpBufs mb{at<float>(h, h->L.mlp_z1), at<float>(h, h->L.mlp_dz1), at<float>(h, h->L.mlp_dz2)};
    MlpTcBufs tb{at<unsigned char>(h, h->L.mlp_w1img), at<unsigned char>(h, h->L.mlp_dzimg), at<float>(h, h->L.mlp_small)};
    const MlpTcGeom& g = h->L.tg;
    CUDA_TRY(h, launch_pdl(mlp_prep_kernel, dim3((P.F + 7) / 8, g.n_sets), dim3(256), 0, h->stream, P, g, tb));
    CUDA_TRY(h, launch_pdl(mlp_f1_tc_kernel, dim3(P.M, 2), dim3(TC_THREADS), mlp_f1_tc_smem(g), h->stream, P, g, mb, tb));
    CUDA_TRY(h, launch_pdl(mlp_f2_rows_kernel, dim3(g.f2_blocks, P.M, 2), dim3(MLP_THREADS), mlp_f2_rows_smem(P.H, P.C), h->stream,
                           P, g, mb, tb));
    CUDA_TRY(h, launch_pdl(mlp_b1_tc_kernel, dim3((P.F + TC_M - 1) / TC_M, P.M, 2), dim3(TC_THREADS), mlp_b1_tc_smem(g), h->stream,
                           P, g, mb, tb));
    h->launches += 3;
  } else if (P.model == CADA_MODEL_MLP2) {
    MlpBufs mb{at<float>(h, h->L.mlp_z1), at<float>(h, h->L.mlp_dz1), at<float>(h, h->L.mlp_dz2)};
    const int row_tiles = (P.B + MF1_ROWS - 1) / MF1_ROWS;
    CUDA_TRY(h, launch_pdl(mlp_f1_kernel, dim3((P.H + MF1_TN - 1) / MF1_TN, P.M * row_tiles, 2), dim3(MLP_THREADS), 0, h->stream, P, mb));
    CUDA_TRY(h, launch_pdl(mlp_f2_kernel, dim3(P.M, 2), dim3(MLP_THREADS), mlp_f2_smem(P.H, P.C), h->stream, P, mb));
    CUDA_TRY(h, launch_pdl(mlp_b1_kernel, dim3((P.H + MB1_T - 1) / MB1_T, (P.F + MB1_T - 1) / MB1_T, P.M * 2), dim3(MLP_THREADS), 0,
                           h->stream, P, mb));
    h->launches += 2;
  } else if (h->L.softmax_fast) {
    const bool wfit = grad_softmax_weights_fit(P.F, P.C, P.has_bias);
    const size_t smem = grad_softmax_smem(P.F, P.C, P.has_bias, wfit);
    const dim3 grid(h->L.n_chunks, P.M);
#define CADA_SOFTMAX_LAUNCH(CP_)                                                                  \
  if (wfit) CUDA_TRY(h, launch_pdl(grad_softmax_kernel<CP_, true>, grid, dim3(GSM_THREADS), smem, h->stream, P)); \
  else CUDA_TRY(h, launch_pdl(grad_softmax_kernel<CP_, false>, grid, dim3(GSM_THREADS), smem, h->stream, P))
    switch (grad_softmax_cp(P.C)) {
      case 4: CADA_SOFTMAX_LAUNCH(4); break;
      case 8: CADA_SOFTMAX_LAUNCH(8); break;
      case 10: CADA_SOFTMAX_LAUNCH(10); break;
      case 12: CADA_SOFTMAX_LAUNCH(12); break;
      default: CADA_SOFTMAX_LAUNCH(16); break;
    }
#undef CADA_SOFTMAX_LAUNCH
  } else if (h->use_stream) {
    const size_t smem = grad_stream_smem(h->L.sg);
    switch (h->L.stream_nch) {
      case 1: CUDA_TRY(h, launch_pdl(grad_stream_kernel<1>, dim3(kStreamCtas), dim3(GS_THREADS), smem, h->stream, P, h->L.sg, h->k_host)); break;
      case 2: CUDA_TRY(h, launch_pdl(grad_stream_kernel<2>, dim3(kStreamCtas), dim3(GS_THREADS), smem, h->stream, P, h->L.sg, h->k_host)); break;
      default: CUDA_TRY(h, launch_pdl(grad_stream_kernel<4>, dim3(kStreamCtas), dim3(GS_THREADS), smem, h->stream, P, h->L.sg, h->k_host)); break;
    }
  } else {
    dim3 grid(h->L.n_chunks, P.M);
    CUDA_TRY(h, launch_pdl(grad_generic_kernel, grid, dim3(GG_THREADS), h->L.grad_smem, h->stream, P));
  }
  h->launches += 1;
  if (h->profile) {
    CUDA_TRY(h, cudaEventRecord(ep.b, h->stream));
    h->pending.push_back(ep);
    h->profiled_iters += 1;
  }
  return CADA_OK;
}

// The server side (mode UPD_FULL), or one of its halves when the workers are split over several handles.
int launch_update(cada_handle* h, const Params& P, int mode, float* sum_io, bool finish = true) {
  const int fin = finish ? 1 : 0;
  const dim3 grid(h->L.upd_blocks), block(h->L.upd_tx, h->L.upd_ty);
  if (mode == UPD_APPLY) {
    const long long groups = (P.p + 3) / 4;
    CUDA_TRY(h, launch_pdl(update_kernel<false, UPD_APPLY>, dim3((unsigned)((groups + UPD_THREADS - 1) / UPD_THREADS)), dim3(UPD_THREADS, 1), 0,
                           h->stream, P, sum_io, h->k_host, fin));
  } else if (mode == UPD_LOCAL) {
    if (P.M > h->L.upd_ty) CUDA_TRY(h, launch_pdl(update_kernel<true, UPD_LOCAL>, grid, block, 0, h->stream, P, sum_io, h->k_host, fin));
    else CUDA_TRY(h, launch_pdl(update_kernel<false, UPD_LOCAL>, grid, block, 0, h->stream, P, sum_io, h->k_host, fin));
  } else {
    if (P.M > h->L.upd_ty) CUDA_TRY(h, launch_pdl(update_kernel<true, UPD_FULL>, grid, block, 0, h->stream, P, sum_io, h->k_host, fin));
    else CUDA_TRY(h, launch_pdl(update_kernel<false, UPD_FULL>, grid, block, 0, h->stream, P, sum_io, h->k_host, fin));
  }
  h->launches += 1;
  return CADA_OK;
}

// The worker side of one pass of Algorithm 1's loop body: gradients and upload decisions.
int enqueue_worker_side(cada_handle* h, const Params& P) {
  int rc = launch_grad(h, P);
  if (rc) return rc;
  if (!h->use_softmax_cluster && !h->use_stream && !h->use_mlp_cluster) {   // those gradient kernels take the decision themselves
    CUDA_TRY(h, launch_pdl(trigger_kernel, dim3(h->L.trig_splits, P.M), dim3(TRIG_THREADS), 0, h->stream, P));
    h->launches += 1;
  }
  return CADA_OK;
}

// One pass of the loop body of Algorithm 1, entirely on the device.
int enqueue_iteration(cada_handle* h, const Params& P, bool last_of_call = true) {
  int rc = enqueue_worker_side(h, P);
  if (rc) return rc;
  rc = launch_update(h, P, UPD_FULL, nullptr, last_of_call);
  if (rc) return rc;
  h->k_host += 1;
  CUDA_TRY(h, cudaGetLastError());
  return CADA_OK;
}

template <int W, int NCH>
const void* cluster_kernel_pick(bool streamed) {
  return streamed ? (const void*)fused_cluster_kernel<W, true, NCH> : (const void*)fused_cluster_kernel<W, false, NCH>;
}
// The one-cluster kernel for W workers per CTA, resident or streamed minibatches, and the worker phase the geometry names
// (nch = 0: two passes over the staged rows; 1: register-tiled).
const void* cluster_kernel_for(int W, bool streamed = false, int nch = 0) {
  if (W == 1) return nch == 1 ? cluster_kernel_pick<1, 1>(streamed) : cluster_kernel_pick<1, 0>(streamed);
  if (W == 2) return nch == 1 ? cluster_kernel_pick<2, 1>(streamed) : cluster_kernel_pick<2, 0>(streamed);
  return cluster_kernel_pick<4, 0>(streamed);
}

void cluster_launch_config(const ClusterGeom& cg, cudaStream_t stream, cudaLaunchConfig_t& lc, cudaLaunchAttribute* attr) {
  memset(&lc, 0, sizeof lc);
  lc.gridDim = dim3(cg.ncta);
  lc.blockDim = dim3((FC_GROUP + 32) * cg.W);
  lc.dynamicSmemBytes = cg.smem_bytes;
  lc.stream = stream;
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cg.ncta;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // consecutive launches overlap their set-up and write-back
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = attr;
  lc.numAttrs = 2;
}

// Picks the cluster shape for the one-cluster kernel: fewest workers per CTA first, the exact CTA count
// before one rounded up to a power of two; the first shape the device can co-schedule wins.
bool choose_cluster(const cada_config* c, cudaStream_t stream, ClusterGeom& out) {
  const int widths[3] = {1, 2, 4};
  for (int wi = 0; wi < 3; ++wi) {
    const int W = widths[wi], need = (c->M + W - 1) / W;
    if (need > FC_MAX_CTAS) continue;
    int pow2 = 1;
    while (pow2 < need) pow2 *= 2;
    const int shapes[2] = {need, pow2};
    for (int si = 0; si < (pow2 == need ? 1 : 2); ++si) {
      ClusterGeom g;
      if (!cluster_plan(c->n_features, c->has_bias ? 1 : 0, c->batch, c->d_max, c->rule, c->M, W, shapes[si], g)) continue;
      const void* fn = cluster_kernel_for(W, false, g.nch);
      if (raise_smem_limit(fn) != cudaSuccess ||
          (g.ncta > 8 && cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) != cudaSuccess)) {
        cudaGetLastError();
        continue;
      }
      cudaLaunchConfig_t lc;
      cudaLaunchAttribute attr[2];
      cluster_launch_config(g, stream, lc, attr);
      int n_clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&n_clusters, fn, &lc) != cudaSuccess) { cudaGetLastError(); continue; }
      if (n_clusters >= 1) { out = g; return true; }
    }
  }
  return false;
}

// n iterations in one launch of a single cluster (small logistic problems with few workers).
int enqueue_cluster(cada_handle* h, const Params& Pin, int n, const HostStream* stream_io = nullptr) {
  EventPair ep{};
  if (h->profile) {
    if (h->pending.size() >= 2048) { int rc = drain_events(h); if (rc) return rc; }
    if (!h->spare.empty()) { ep = h->spare.back(); h->spare.pop_back(); }
    else { CUDA_TRY(h, cudaEventCreate(&ep.a)); CUDA_TRY(h, cudaEventCreate(&ep.b)); }
    CUDA_TRY(h, cudaEventRecord(ep.a, h->stream));
  }
  Params P = Pin;
  ClusterGeom cg = stream_io ? h->cg_stream : h->cg;
  long long k_first = h->k_host;
  HostStream hs{nullptr, nullptr, nullptr, nullptr};
  if (stream_io) hs = *stream_io;
  void* args[] = {&P, &cg, &n, &k_first, &hs};
  cudaLaunchConfig_t lc;
  cudaLaunchAttribute attr[2];
  cluster_launch_config(cg, h->stream, lc, attr);
  CUDA_TRY(h, cudaLaunchKernelExC(&lc, cluster_kernel_for(cg.W, stream_io != nullptr, cg.nch), args));
  if (h->profile) {
    CUDA_TRY(h, cudaEventRecord(ep.b, h->stream));
    h->pending.push_back(ep);
    h->profiled_iters += n;
  }
  h->launches += 1;
  h->k_host += n;
  return CADA_OK;
}

// n iterations in one cooperative launch (small logistic problems).
int enqueue_fused(cada_handle* h, const Params& Pin, int n) {
  if (h->use_cluster) return enqueue_cluster(h, Pin, n);
  EventPair ep{};
  if (h->profile) {
    if (h->pending.size() >= 2048) { int rc = drain_events(h); if (rc) return rc; }
    if (!h->spare.empty()) { ep = h->spare.back(); h->spare.pop_back(); }
    else { CUDA_TRY(h, cudaEventCreate(&ep.a)); CUDA_TRY(h, cudaEventCreate(&ep.b)); }
  }
  unsigned* flags = at<unsigned>(h, h->L.fused_flags);
  CUDA_TRY(h, cudaMemsetAsync(flags, 0, h->L.fused_flags.bytes, h->stream));   // iteration tags restart at 1
  if (h->profile) CUDA_TRY(h, cudaEventRecord(ep.a, h->stream));
  Params P = Pin;
  FusedGeom fg = h->L.fg;
  float* g_alt = at<float>(h, h->L.G_alt);
  unsigned wait_limit = h->wait_limit;
  void* args[] = {&P, &fg, &n, &g_alt, &flags, &wait_limit};
  CUDA_TRY(h, cudaLaunchCooperativeKernel((const void*)fused_logistic_kernel, dim3(P.M), dim3(FS_THREADS), args,
                                          fg.smem_bytes, h->stream));
  if (h->profile) {
    CUDA_TRY(h, cudaEventRecord(ep.b, h->stream));
    h->pending.push_back(ep);
    h->profiled_iters += n;
  }
  h->launches += 1;
  h->k_host += n;
  return CADA_OK;
}

struct BufInfo { void* ptr; size_t elt; size_t rows; size_t cols; size_t pitch_elts; };

bool buffer_info(cada_handle* h, int which, BufInfo& b) {
  const Params& P = h->P;
  const size_t p = (size_t)P.p, M = (size_t)P.M, ldp = (size_t)P.ldp, cap = (size_t)h->cfg.history_capacity;
  switch (which) {
    case CADA_BUF_THETA: b = {P.theta, 4, 1, p, ldp}; return true;
    case CADA_BUF_H: b = {P.h, 4, 1, p, ldp}; return true;
    case CADA_BUF_VHAT: b = {P.vhat, 4, 1, p, ldp}; return true;
    case CADA_BUF_G: b = {P.G, 4, M, p, ldp}; return true;
    case CADA_BUF_THETA_HAT: b = {P.theta_hat, 4, M, p, ldp}; return P.theta_hat != nullptr;
    case CADA_BUF_DELTA_STORED: b = {P.delta_stored, 4, M, p, ldp}; return P.delta_stored != nullptr;
    case CADA_BUF_THETA_TILDE: b = {P.theta_tilde, 4, 1, p, ldp}; return P.theta_tilde != nullptr;
    case CADA_BUF_TAU: b = {P.tau, 4, 1, M, M}; return true;
    case CADA_BUF_RING: b = {P.ring, 8, 1, (size_t)P.d_max, (size_t)P.d_max}; return true;
    case CADA_BUF_GRAD_FRESH: b = {P.g_fresh, 4, M, p, ldp}; return true;
    case CADA_BUF_INNOV_FRESH: b = {P.d_fresh, 4, M, p, ldp}; return true;
    case CADA_BUF_LAST_LHS: b = {P.lhs, 8, 1, M, M}; return true;
    case CADA_BUF_LAST_MASK: b = {P.mask, 1, 1, M, M}; return true;
    case CADA_BUF_UPLOADS_PER_WORKER: b = {P.up_per_worker, 8, 1, M, M}; return true;
    case CADA_BUF_HIST_LHS: b = {P.hist_lhs, 8, 1, cap * M, cap * M}; return cap > 0;
    case CADA_BUF_HIST_RHS: b = {P.hist_rhs, 8, 1, cap, cap}; return cap > 0;
    case CADA_BUF_HIST_MASK: b = {P.hist_mask, 1, 1, cap * M, cap * M}; return cap > 0;
    case CADA_BUF_K: b = {&P.st->k, 8, 1, 1, 1}; return true;
    case CADA_BUF_MLP_Z1: {
      const size_t n = M * 2 * (size_t)P.B * (size_t)P.H;
      b = {at<float>(h, h->L.mlp_z1), 4, 1, n, n};
      return h->L.mlp_z1.bytes > 0;
    }
    case CADA_BUF_NABLA: b = {P.nabla, 4, 1, p, ldp}; return P.nabla != nullptr;
    case CADA_BUF_MLP_DZ1: {
      const size_t n = M * 2 * (size_t)P.B * (size_t)P.H;
      b = {at<float>(h, h->L.mlp_dz1), 4, 1, n, n};
      return h->L.mlp_dz1.bytes > 0;
    }
    case CADA_BUF_MLP_DZ2: {
      const size_t n = M * 2 * (size_t)P.B * (size_t)P.C;
      b = {at<float>(h, h->L.mlp_dz2), 4, 1, n, n};
      return h->L.mlp_dz2.bytes > 0;
    }
  }
  return false;
}

}  // namespace

extern "C" {
#pragma GCC visibility push(default)

size_t cada_workspace_bytes(const cada_config* cfg) {
  Layout L;
  char msg[256];
  if (plan(cfg, L, msg, sizeof msg) != CADA_OK) return 0;
  return L.total;
}

int cada_create(const cada_config* cfg, cada_handle** out) {
  if (!out) { snprintf(g_create_error, sizeof g_create_error, "out is NULL"); return CADA_ERR_INVALID_ARG; }
  *out = nullptr;
  Layout L;
  int rc = plan(cfg, L, g_create_error, sizeof g_create_error);
  if (rc != CADA_OK) return rc;
#define CFAIL(code, ...) do { snprintf(g_create_error, sizeof g_create_error, __VA_ARGS__); return code; } while (0)
  if (!cfg->X || !cfg->y || !cfg->n_samples || !cfg->theta0) CFAIL(CADA_ERR_INVALID_ARG, "X, y, n_samples and theta0 must be non-NULL");
  for (int m = 0; m < cfg->M; ++m) {
    if (!cfg->X[m] || !cfg->y[m]) CFAIL(CADA_ERR_INVALID_ARG, "X[%d] or y[%d] is NULL", m, m);
    if (cfg->n_samples[m] < 1) CFAIL(CADA_ERR_INVALID_ARG, "n_samples[%d] < 1", m);
    if (cfg->tau0 && cfg->tau0[m] < 0) CFAIL(CADA_ERR_INVALID_ARG, "tau0[%d] < 0", m);
  }
  if (!cfg->workspace) CFAIL(CADA_ERR_WORKSPACE, "workspace is NULL");
  if (reinterpret_cast<uintptr_t>(cfg->workspace) % 256 != 0) CFAIL(CADA_ERR_WORKSPACE, "workspace must be 256-byte aligned");
  if (cfg->workspace_bytes < L.total) CFAIL(CADA_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", cfg->workspace_bytes, L.total);

  cada_handle* h = new (std::nothrow) cada_handle();
  if (!h) CFAIL(CADA_ERR_INVALID_ARG, "out of host memory");
  h->cfg = *cfg;
  h->cfg.X = nullptr; h->cfg.y = nullptr; h->cfg.n_samples = nullptr; h->cfg.tau0 = nullptr; h->cfg.theta0 = nullptr;
  h->cfg.batch_m = nullptr;
  h->L = L;
  h->stream = static_cast<cudaStream_t>(cfg->stream);
  h->ws = static_cast<char*>(cfg->workspace);
  h->k_host = 0; h->idx_remaining = 0; h->launches = 0; h->profile = false; h->grad_ms = 0; h->grad_launches = 0;
  h->use_fused = false; h->use_cluster = false; h->stream_ok = false; h->use_softmax_cluster = false; h->profiled_iters = 0; h->use_mlp_tc = false;
  h->use_mlp_cluster = false; h->use_mlp_hsplit = false; h->ring_dirty = false; h->copy_ready = false; h->copy_stream = nullptr; h->half_done = false;
  h->err[0] = 0;
  h->device_error = CADA_OK;
  h->wait_limit = FS_SPIN_LIMIT;

  Params& P = h->P;
  memset(&P, 0, sizeof P);
  P.model = cfg->model; P.rule = cfg->rule; P.M = cfg->M; P.B = cfg->batch; P.F = cfg->n_features;
  P.C = cfg->n_classes; P.H = cfg->n_hidden; P.has_bias = cfg->has_bias ? 1 : 0; P.d_max = cfg->d_max; P.D = cfg->D;
  P.x_bf16 = cfg->x_dtype == CADA_X_BF16; P.server = cfg->server; P.aggregate = cfg->aggregate;
  P.Mg = cfg->M_total ? cfg->M_total : cfg->M; P.m0 = cfg->M_total ? cfg->m_first : 0; P.ms = cfg->M_total ? cfg->m_stride : 1;
  P.alpha_K0 = cfg->alpha_K0; P.batch_m = at<int>(h, L.btab); P.nabla = at<float>(h, L.nabla);
  P.p = cfg->p; P.ldp = L.ldp; P.ldx = cfg->ldx;
  P.alpha = cfg->alpha; P.beta1 = cfg->beta1; P.beta2 = cfg->beta2; P.eps = cfg->eps; P.c = cfg->c; P.lambda = cfg->lambda;
  P.seed = cfg->seed;
  P.X = at<const void*>(h, L.xtab); P.y = at<const void*>(h, L.ytab); P.n_samples = at<long long>(h, L.ntab);
  P.idx_mode = IDX_HASH; P.idx = nullptr; P.idx_k0 = 0;
  P.st = at<DevState>(h, L.st);
  P.theta = at<float>(h, L.theta); P.h = at<float>(h, L.h); P.vhat = at<float>(h, L.vhat);
  P.theta_tilde = at<float>(h, L.theta_tilde);
  P.G = at<float>(h, L.G); P.theta_hat = at<float>(h, L.theta_hat); P.delta_stored = at<float>(h, L.delta_stored);
  P.g_fresh = at<float>(h, L.g_fresh); P.d_fresh = at<float>(h, L.d_fresh); P.part = at<float>(h, L.part);
  P.tau = at<int>(h, L.tau); P.mask = at<unsigned char>(h, L.mask); P.lhs = at<double>(h, L.lhs);
  P.up_per_worker = at<long long>(h, L.upw); P.ring = at<double>(h, L.ring);
  P.norm_part = at<double>(h, L.norm_part); P.step_part = at<double>(h, L.step_part);
  P.worker_ticket = at<unsigned>(h, L.tickets);
  P.hist_lhs = at<double>(h, L.hist_lhs); P.hist_rhs = at<double>(h, L.hist_rhs); P.hist_mask = at<unsigned char>(h, L.hist_mask);
  P.hist_cap = cfg->history_capacity;
  P.n_chunks = L.n_chunks; P.rows_per_chunk = L.rows_per_chunk; P.trig_splits = L.trig_splits; P.trig_cols = L.trig_cols;
  P.upd_ty = L.upd_ty;

  auto bail = [&](int code, const char* what, cudaError_t e) {
    snprintf(g_create_error, sizeof g_create_error, "%s: %s", what, cudaGetErrorString(e));
    delete h;
    return code;
  };
#define CTRY(call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) return bail(CADA_ERR_CUDA, #call, e_); } while (0)
  if (L.grad_smem > 48 * 1024)
    CTRY(raise_smem_limit(grad_generic_kernel));
  if (cfg->model == CADA_MODEL_MLP2)
    CTRY(raise_smem_limit(mlp_f2_kernel));
  if (L.softmax_fast) {
    const int hb = cfg->has_bias ? 1 : 0;
    const bool wfit = grad_softmax_weights_fit(cfg->n_features, cfg->n_classes, hb);
    const int smem = (int)grad_softmax_smem(cfg->n_features, cfg->n_classes, hb, wfit);
#define CADA_SOFTMAX_ATTR(CP_)                                                                                         \
  if (wfit) CTRY(raise_smem_limit(grad_softmax_kernel<CP_, true>)); \
  else CTRY(raise_smem_limit(grad_softmax_kernel<CP_, false>))
    switch (grad_softmax_cp(cfg->n_classes)) {
      case 4: CADA_SOFTMAX_ATTR(4); break;
      case 8: CADA_SOFTMAX_ATTR(8); break;
      case 10: CADA_SOFTMAX_ATTR(10); break;
      case 12: CADA_SOFTMAX_ATTR(12); break;
      default: CADA_SOFTMAX_ATTR(16); break;
    }
#undef CADA_SOFTMAX_ATTR
  }
  if (cfg->model == CADA_MODEL_SOFTMAX && cfg->n_classes <= 16)
    h->use_softmax_cluster = choose_softmax_cluster(cfg, h->stream, h->scg);
  h->use_mlp_tc = L.mlp_tc_ok;
  for (int m = 0; m < cfg->M && h->use_mlp_tc; ++m)
    if (reinterpret_cast<uintptr_t>(cfg->X[m]) % 16 != 0) h->use_mlp_tc = false;     // 16-byte async copies of the rows
  if (h->use_mlp_tc) {
    CTRY(raise_smem_limit(mlp_f1_tc_kernel));
    CTRY(raise_smem_limit(mlp_f2_rows_kernel));
    CTRY(raise_smem_limit(mlp_b1_tc_kernel));
  }
  if (getenv("CADA_DEBUG")) fprintf(stderr, "mlp: tc=%d hs_ok=%d cl_ok=%d\n", (int)h->use_mlp_tc, (int)L.mlp_hsplit_ok, (int)L.mlp_cluster_ok);
  if (h->use_mlp_tc && L.mlp_hsplit_ok) {
    cudaLaunchConfig_t lc;
    cudaLaunchAttribute attr[2];
    mlp_cluster_launch_config(L.mhg.ns, L.mhg.smem_bytes, cfg->M, h->stream, lc, attr);
    int n_clusters = 0;
    if (getenv("CADA_DEBUG")) {
      cudaError_t e1 = raise_smem_limit(mlp_hsplit_kernel);
      cudaError_t e2 = cudaOccupancyMaxActiveClusters(&n_clusters, (const void*)mlp_hsplit_kernel, &lc);
      fprintf(stderr, "hsplit: ns=%d smem=%u e1=%d e2=%d (%s) n_clusters=%d\n", L.mhg.ns, L.mhg.smem_bytes, (int)e1, (int)e2, cudaGetErrorString(e2), n_clusters);
      cudaGetLastError();
    }
    if (raise_smem_limit(mlp_hsplit_kernel) == cudaSuccess &&
        cudaOccupancyMaxActiveClusters(&n_clusters, (const void*)mlp_hsplit_kernel, &lc) == cudaSuccess && n_clusters >= 1) {
      h->use_mlp_cluster = h->use_mlp_hsplit = true;
      P.w1_ring = at<unsigned char>(h, L.mlp_ring);
      P.w1_slots = cfg->D + 1;
      P.w1_nhc = 4;
      P.w1_set_bytes = L.mhg.set_bytes;
      P.w1_chunk_bytes = L.mhg.slice_bytes;
      P.w1_hsplit = 1;
    } else {
      cudaGetLastError();
    }
  }
  if (h->use_mlp_tc && L.mlp_cluster_ok && !h->use_mlp_hsplit) {
    cudaLaunchConfig_t lc;
    cudaLaunchAttribute attr[2];
    mlp_cluster_launch_config(L.mcg.ns, L.mcg.smem_bytes, cfg->M, h->stream, lc, attr);
    int n_clusters = 0;
    if (raise_smem_limit(mlp_cluster_kernel) == cudaSuccess &&
        cudaOccupancyMaxActiveClusters(&n_clusters, (const void*)mlp_cluster_kernel, &lc) == cudaSuccess && n_clusters >= 1) {
      h->use_mlp_cluster = true;
      P.w1_ring = at<unsigned char>(h, L.mlp_ring);
      P.w1_slots = cfg->D + 1;
      P.w1_nhc = L.tg.nhc;
      P.w1_set_bytes = L.tg.w_set_bytes;
      P.w1_chunk_bytes = L.tg.w_chunk_bytes;
    } else {
      cudaGetLastError();
    }
  }
  h->use_stream = L.stream_ok;
  for (int m = 0; m < cfg->M && h->use_stream; ++m)
    if (reinterpret_cast<uintptr_t>(cfg->X[m]) % 16 != 0) h->use_stream = false;   // bulk copies need 16-byte sources
  if (h->use_stream) {
    const int smem = (int)grad_stream_smem(L.sg);
    CTRY(raise_smem_limit(grad_stream_kernel<1>));
    CTRY(raise_smem_limit(grad_stream_kernel<2>));
    CTRY(raise_smem_limit(grad_stream_kernel<4>));
    P.n_chunks = L.stream_slots;
  }
  h->use_fused = L.fused_ok;
  for (int m = 0; m < cfg->M && h->use_fused; ++m)
    if (reinterpret_cast<uintptr_t>(cfg->X[m]) % 16 != 0) h->use_fused = false;     // 16-byte async copies of the rows
  if (h->use_fused) {
    int dev = 0, coop = 0, sms = 0, per_sm = 0;
    CTRY(cudaGetDevice(&dev));
    CTRY(cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev));
    CTRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CTRY(raise_smem_limit(fused_logistic_kernel));
    CTRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fused_logistic_kernel, FS_THREADS, L.fg.smem_bytes));
    if (!coop || (long long)per_sm * sms < cfg->M) h->use_fused = false;            // all CTAs must be resident at once
    // few workers: the same iteration with the exchange kept inside one thread-block cluster
    if (h->use_fused) h->use_cluster = choose_cluster(cfg, h->stream, h->cg);
    h->stream_ok = false;
    if (h->use_cluster && cfg->host_step_rows > 0) {
      // the streamed form keeps the cluster shape of the resident one and needs a third minibatch buffer per worker
      ClusterGeom g;
      const void* fn = nullptr;
      if (cluster_plan(cfg->n_features, cfg->has_bias ? 1 : 0, cfg->batch, cfg->d_max, cfg->rule, cfg->M, h->cg.W, h->cg.ncta, g, 3, cfg->ldx) &&
          (fn = cluster_kernel_for(h->cg.W, true, g.nch)) != nullptr && raise_smem_limit(fn) == cudaSuccess &&
          (g.ncta <= 8 || cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess)) {
        cudaLaunchConfig_t lc;
        cudaLaunchAttribute attr[2];
        cluster_launch_config(g, h->stream, lc, attr);
        int n_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&n_clusters, fn, &lc) == cudaSuccess && n_clusters >= 1) { h->cg_stream = g; h->stream_ok = true; }
      }
      cudaGetLastError();
    }
  }
  // zero everything except the staging area, then fill the tables and the iterates
  const size_t zero_bytes = L.stage_x.bytes ? L.stage_x.off : L.total;
  CTRY(cudaMemsetAsync(h->ws, 0, zero_bytes, h->stream));
  std::vector<long long> ns(cfg->M);
  std::vector<int> tau(cfg->M);
  for (int m = 0; m < cfg->M; ++m) { ns[m] = cfg->n_samples[m]; tau[m] = cfg->tau0 ? cfg->tau0[m] : cfg->D; }
  h->n_samples = ns;
  CTRY(cudaMemcpyAsync(h->ws + L.xtab.off, cfg->X, sizeof(void*) * cfg->M, cudaMemcpyHostToDevice, h->stream));
  CTRY(cudaMemcpyAsync(h->ws + L.ytab.off, cfg->y, sizeof(void*) * cfg->M, cudaMemcpyHostToDevice, h->stream));
  CTRY(cudaMemcpyAsync(h->ws + L.ntab.off, ns.data(), sizeof(long long) * cfg->M, cudaMemcpyHostToDevice, h->stream));
  CTRY(cudaMemcpyAsync(h->ws + L.tau.off, tau.data(), sizeof(int) * cfg->M, cudaMemcpyHostToDevice, h->stream));
  std::vector<int> bm(cfg->M, cfg->batch);
  if (cfg->batch_m) {
    for (int m = 0; m < cfg->M; ++m) bm[m] = cfg->batch_m[m];
    CTRY(cudaMemcpyAsync(h->ws + L.btab.off, bm.data(), sizeof(int) * cfg->M, cudaMemcpyHostToDevice, h->stream));
  }
  std::vector<long long> us((size_t)cfg->M + 1, 0);
  if (L.ustab.bytes) {
    for (int m = 0; m < cfg->M; ++m) us[m + 1] = us[m] + (bm[m] + GS_R - 1) / GS_R;
    CTRY(cudaMemcpyAsync(h->ws + L.ustab.off, us.data(), sizeof(long long) * ((size_t)cfg->M + 1), cudaMemcpyHostToDevice, h->stream));
    h->L.sg.ustart = at<long long>(h, L.ustab);
  }
  h->Ph = P;
  if (cfg->host_step_rows > 0) {
    const size_t elt = cfg->x_dtype == CADA_X_BF16 ? 2 : 4;
    std::vector<const void*> xs(cfg->M), ys(cfg->M);
    std::vector<long long> nb(cfg->M, cfg->batch);
    for (int m = 0; m < cfg->M; ++m) {
      xs[m] = h->ws + L.stage_x.off + (size_t)m * cfg->batch * (size_t)cfg->ldx * elt;
      ys[m] = h->ws + L.stage_y.off + (size_t)m * cfg->batch * 4;
    }
    CTRY(cudaMemcpyAsync(h->ws + L.xtab_s.off, xs.data(), sizeof(void*) * cfg->M, cudaMemcpyHostToDevice, h->stream));
    CTRY(cudaMemcpyAsync(h->ws + L.ytab_s.off, ys.data(), sizeof(void*) * cfg->M, cudaMemcpyHostToDevice, h->stream));
    CTRY(cudaMemcpyAsync(h->ws + L.ntab_s.off, nb.data(), sizeof(long long) * cfg->M, cudaMemcpyHostToDevice, h->stream));
    h->Ph.X = at<const void*>(h, L.xtab_s); h->Ph.y = at<const void*>(h, L.ytab_s); h->Ph.n_samples = at<long long>(h, L.ntab_s);
    h->Ph.idx_mode = IDX_IDENTITY;
    for (int m = 0; m < cfg->M; ++m) {
      xs[m] = h->ws + L.stage_x2.off + (size_t)m * cfg->batch * (size_t)cfg->ldx * elt;
      ys[m] = h->ws + L.stage_y2.off + (size_t)m * cfg->batch * 4;
    }
    CTRY(cudaMemcpyAsync(h->ws + L.xtab_s2.off, xs.data(), sizeof(void*) * cfg->M, cudaMemcpyHostToDevice, h->stream));
    CTRY(cudaMemcpyAsync(h->ws + L.ytab_s2.off, ys.data(), sizeof(void*) * cfg->M, cudaMemcpyHostToDevice, h->stream));
    h->Ph2 = h->Ph;
    h->Ph2.X = at<const void*>(h, L.xtab_s2); h->Ph2.y = at<const void*>(h, L.ytab_s2);
  }
  init_kernel<<<148, 256, 0, h->stream>>>(P, cfg->theta0);
  h->launches += 1;
  h->ring_dirty = h->use_mlp_cluster;       // the first step builds the image of theta^0
  CTRY(cudaGetLastError());
  CTRY(cudaStreamSynchronize(h->stream));   // host vectors above go out of scope
#undef CTRY
#undef CFAIL
  *out = h;
  return CADA_OK;
}

int cada_step(cada_handle* h, int32_t n_iters) {
  if (!h) return CADA_ERR_INVALID_ARG;
  if (n_iters < 0) return fail(h, CADA_ERR_INVALID_ARG, "n_iters < 0");
  if (h->device_error) return fail(h, h->device_error, "the device reported a problem earlier (see cada_stats); the run cannot continue");
  if (h->half_done) return fail(h, CADA_ERR_INVALID_ARG, "cada_step_apply must follow cada_step_local");
  if (h->P.Mg != h->P.M) return fail(h, CADA_ERR_INVALID_ARG, "this handle holds a subset of the workers: step it with cada_step_local / cada_step_apply");
  if (h->use_fused) {
    int left = n_iters;
    while (left > 0) {
      if (h->P.idx_mode == IDX_EXPLICIT && h->idx_remaining == 0) { h->P.idx_mode = IDX_HASH; h->P.idx = nullptr; }
      int chunk = left < (1 << 20) ? left : (1 << 20);
      if (h->P.idx_mode == IDX_EXPLICIT && h->idx_remaining < chunk) chunk = (int)h->idx_remaining;
      int rc = enqueue_fused(h, h->P, chunk);
      if (rc) return rc;
      if (h->P.idx_mode == IDX_EXPLICIT) h->idx_remaining -= chunk;
      left -= chunk;
    }
    return CADA_OK;
  }
  for (int it = 0; it < n_iters; ++it) {
    if (h->P.idx_mode == IDX_EXPLICIT && h->idx_remaining == 0) { h->P.idx_mode = IDX_HASH; h->P.idx = nullptr; }
    int rc = enqueue_iteration(h, h->P, it == n_iters - 1);
    if (rc) return rc;
    if (h->P.idx_mode == IDX_EXPLICIT) h->idx_remaining -= 1;
  }
  return CADA_OK;
}

int cada_step_local(cada_handle* h, float* dev_sum_out) {
  if (!h) return CADA_ERR_INVALID_ARG;
  if (!dev_sum_out || reinterpret_cast<uintptr_t>(dev_sum_out) % 16 != 0) return fail(h, CADA_ERR_INVALID_ARG, "dev_sum_out must be a 16-byte aligned device pointer");
  if (h->use_fused) return fail(h, CADA_ERR_UNSUPPORTED, "the one-launch paths cannot be stepped in halves: create the handle with M_total set");
  if (h->half_done) return fail(h, CADA_ERR_INVALID_ARG, "cada_step_apply must follow cada_step_local");
  if (h->device_error) return fail(h, h->device_error, "the device reported a problem earlier (see cada_stats); the run cannot continue");
  if (h->P.idx_mode == IDX_EXPLICIT && h->idx_remaining == 0) { h->P.idx_mode = IDX_HASH; h->P.idx = nullptr; }
  int rc = enqueue_worker_side(h, h->P);
  if (rc) return rc;
  rc = launch_update(h, h->P, UPD_LOCAL, dev_sum_out);
  if (rc) return rc;
  CUDA_TRY(h, cudaGetLastError());
  h->half_done = true;
  return CADA_OK;
}

int cada_step_apply(cada_handle* h, const float* dev_sum) {
  if (!h) return CADA_ERR_INVALID_ARG;
  if (!dev_sum || reinterpret_cast<uintptr_t>(dev_sum) % 16 != 0) return fail(h, CADA_ERR_INVALID_ARG, "dev_sum must be a 16-byte aligned device pointer");
  if (!h->half_done) return fail(h, CADA_ERR_INVALID_ARG, "cada_step_local must come first");
  int rc = launch_update(h, h->P, UPD_APPLY, const_cast<float*>(dev_sum));
  if (rc) return rc;
  CUDA_TRY(h, cudaGetLastError());
  h->half_done = false;
  h->k_host += 1;
  if (h->P.idx_mode == IDX_EXPLICIT) h->idx_remaining -= 1;
  return CADA_OK;
}

int cada_step_host(cada_handle* h, const void* host_X, const void* host_y, float* host_theta_out, uint8_t* host_mask_out) {
  if (!h) return CADA_ERR_INVALID_ARG;
  if (!host_X || !host_y) return fail(h, CADA_ERR_INVALID_ARG, "host_X and host_y must be non-NULL");
  if (!h->L.stage_x.bytes) return fail(h, CADA_ERR_INVALID_ARG, "handle was created without host_step_rows");
  if (h->device_error) return fail(h, h->device_error, "the device reported a problem earlier (see cada_stats); the run cannot continue");
  CUDA_TRY(h, cudaMemcpyAsync(h->ws + h->L.stage_x.off, host_X, h->L.stage_x.bytes, cudaMemcpyHostToDevice, h->stream));
  CUDA_TRY(h, cudaMemcpyAsync(h->ws + h->L.stage_y.off, host_y, h->L.stage_y.bytes, cudaMemcpyHostToDevice, h->stream));
  int rc = h->use_fused ? enqueue_fused(h, h->Ph, 1) : enqueue_iteration(h, h->Ph);
  if (rc) return rc;
  if (host_theta_out)
    CUDA_TRY(h, cudaMemcpyAsync(host_theta_out, h->P.theta, sizeof(float) * (size_t)h->P.p, cudaMemcpyDeviceToHost, h->stream));
  if (host_mask_out)
    CUDA_TRY(h, cudaMemcpyAsync(host_mask_out, h->P.mask, (size_t)h->P.M, cudaMemcpyDeviceToHost, h->stream));
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return CADA_OK;
}

int cada_step_host_n(cada_handle* h, int32_t n, const void* host_X, const void* host_y, float* host_theta_out,
                     uint8_t* host_mask_out) {
  if (!h) return CADA_ERR_INVALID_ARG;
  if (n < 0) return fail(h, CADA_ERR_INVALID_ARG, "n < 0");
  if (!host_X || !host_y) return fail(h, CADA_ERR_INVALID_ARG, "host_X and host_y must be non-NULL");
  if (!h->L.stage_x.bytes) return fail(h, CADA_ERR_INVALID_ARG, "handle was created without host_step_rows");
  if (h->device_error) return fail(h, h->device_error, "the device reported a problem earlier (see cada_stats); the run cannot continue");
  if (!h->copy_ready) {
    CUDA_TRY(h, cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
    for (int i = 0; i < 2; ++i) {
      CUDA_TRY(h, cudaEventCreateWithFlags(&h->ev_copied[i], cudaEventDisableTiming));
      CUDA_TRY(h, cudaEventCreateWithFlags(&h->ev_done[i], cudaEventDisableTiming));
    }
    CUDA_TRY(h, cudaEventCreateWithFlags(&h->ev_start, cudaEventDisableTiming));
    h->copy_ready = true;
  }
  const size_t xb = h->L.stage_x.bytes, yb = h->L.stage_y.bytes, p = (size_t)h->P.p, M = (size_t)h->P.M;
  // One-cluster path with every buffer in page-locked memory the device can address: ONE launch runs the n iterations;
  // its producer warps fetch the minibatch of iteration i+1 from the caller's buffers over the bus while iteration i
  // computes (the same double buffer that prefetches resident rows), and each iteration stores its theta and mask
  // straight into the caller's buffers.  No staging copy, no copy-engine operation, one synchronisation.
  if (h->use_fused && h->use_cluster && h->stream_ok) {
    auto mapped = [](const void* q) -> void* {
      cudaPointerAttributes a;
      if (cudaPointerGetAttributes(&a, q) != cudaSuccess) { cudaGetLastError(); return nullptr; }
      return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
    };
    HostStream hs{static_cast<const float*>(mapped(host_X)), static_cast<const float*>(mapped(host_y)),
                  host_theta_out ? static_cast<float*>(mapped(host_theta_out)) : nullptr,
                  host_mask_out ? static_cast<unsigned char*>(mapped(host_mask_out)) : nullptr};
    const bool ok = hs.x && hs.y && reinterpret_cast<uintptr_t>(hs.x) % 16 == 0 && reinterpret_cast<uintptr_t>(hs.y) % 4 == 0 &&
                    (!host_theta_out || hs.out_theta) && (!host_mask_out || hs.out_mask);
    if (ok) {
      int left = n;
      while (left > 0) {
        const int chunk = left < (1 << 20) ? left : (1 << 20);
        int rc = enqueue_cluster(h, h->P, chunk, &hs);
        if (rc) { cudaStreamSynchronize(h->stream); return rc; }
        hs.x += (size_t)chunk * (xb / sizeof(float)); hs.y += (size_t)chunk * (yb / sizeof(float));
        if (hs.out_theta) hs.out_theta += (size_t)chunk * p;
        if (hs.out_mask) hs.out_mask += (size_t)chunk * M;
        left -= chunk;
      }
      CUDA_TRY(h, cudaStreamSynchronize(h->stream));
      return CADA_OK;
    }
  }
  const Region* sx[2] = {&h->L.stage_x, &h->L.stage_x2};
  const Region* sy[2] = {&h->L.stage_y, &h->L.stage_y2};
  // Results: where the output buffers are page-locked host memory the device can address, a small kernel stores them
  // there directly; otherwise they are copied back with cudaMemcpyAsync on the caller's stream.
  float* map_theta = nullptr;
  uint8_t* map_mask = nullptr;
  {
    cudaPointerAttributes at_;
    if (host_theta_out && cudaPointerGetAttributes(&at_, host_theta_out) == cudaSuccess && at_.type == cudaMemoryTypeHost && at_.devicePointer)
      map_theta = static_cast<float*>(at_.devicePointer);
    if (host_mask_out && cudaPointerGetAttributes(&at_, host_mask_out) == cudaSuccess && at_.type == cudaMemoryTypeHost && at_.devicePointer)
      map_mask = static_cast<uint8_t*>(at_.devicePointer);
    cudaGetLastError();
  }
  // ... for small results only: stores over the bus from the SMs run at about 30 GB/s, a copy engine moves a long
  // iterate faster than that
  const bool direct = (!host_theta_out || map_theta) && (!host_mask_out || map_mask) && (host_theta_out || host_mask_out) &&
                      (host_theta_out ? p * sizeof(float) : 0) + M <= (size_t)128 * 1024;
  // earlier work on the caller's stream may still read the staging halves: the copy stream starts behind it
  CUDA_TRY(h, cudaEventRecord(h->ev_start, h->stream));
  CUDA_TRY(h, cudaStreamWaitEvent(h->copy_stream, h->ev_start, 0));
  for (int i = 0; i < n; ++i) {
    const int b = i & 1;
    // the host's calls per step bound the rate of small workloads: one copy stream, one event each way
    if (i >= 2) CUDA_TRY(h, cudaStreamWaitEvent(h->copy_stream, h->ev_done[b], 0));     // step i-2 has consumed this half
    CUDA_TRY(h, cudaMemcpyAsync(h->ws + sx[b]->off, static_cast<const char*>(host_X) + (size_t)i * xb, xb, cudaMemcpyHostToDevice, h->copy_stream));
    CUDA_TRY(h, cudaMemcpyAsync(h->ws + sy[b]->off, static_cast<const char*>(host_y) + (size_t)i * yb, yb, cudaMemcpyHostToDevice, h->copy_stream));
    CUDA_TRY(h, cudaEventRecord(h->ev_copied[b], h->copy_stream));
    CUDA_TRY(h, cudaStreamWaitEvent(h->stream, h->ev_copied[b], 0));
    const Params& Pb = b ? h->Ph2 : h->Ph;
    int rc = h->use_fused ? enqueue_fused(h, Pb, 1) : enqueue_iteration(h, Pb, i == n - 1);
    if (rc) { cudaStreamSynchronize(h->copy_stream); cudaStreamSynchronize(h->stream); return rc; }
    CUDA_TRY(h, cudaEventRecord(h->ev_done[b], h->stream));
    if (direct) {
      const long long work = (long long)(host_theta_out ? p : M);
      const unsigned blocks = (unsigned)((work + 1023) / 1024 < 1 ? 1 : (work + 1023) / 1024 > 592 ? 592 : (work + 1023) / 1024);
      CUDA_TRY(h, launch_pdl(export_kernel, dim3(blocks), dim3(256), 0, h->stream, (const float*)h->P.theta, (long long)p,
                             (const unsigned char*)h->P.mask, (int)M, map_theta ? map_theta + (size_t)i * p : (float*)nullptr,
                             map_mask ? map_mask + (size_t)i * M : (unsigned char*)nullptr));
      h->launches += 1;
    } else {
      if (host_theta_out)
        CUDA_TRY(h, cudaMemcpyAsync(host_theta_out + (size_t)i * p, h->P.theta, sizeof(float) * p, cudaMemcpyDeviceToHost, h->stream));
      if (host_mask_out)
        CUDA_TRY(h, cudaMemcpyAsync(host_mask_out + (size_t)i * M, h->P.mask, M, cudaMemcpyDeviceToHost, h->stream));
    }
  }
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return CADA_OK;
}

int cada_set_indices(cada_handle* h, const int32_t* dev_idx, int32_t n_iters) {
  if (!h) return CADA_ERR_INVALID_ARG;
  if (!dev_idx) { h->P.idx_mode = IDX_HASH; h->P.idx = nullptr; h->idx_remaining = 0; return CADA_OK; }
  if (n_iters < 1) return fail(h, CADA_ERR_INVALID_ARG, "n_iters < 1");
  h->P.idx_mode = IDX_EXPLICIT;
  h->P.idx = dev_idx;
  h->P.idx_k0 = h->k_host;
  h->idx_remaining = n_iters;
  return CADA_OK;
}

int cada_stats(cada_handle* h, cada_stats_t* out) {
  if (!h || !out) return h ? fail(h, CADA_ERR_INVALID_ARG, "out is NULL") : CADA_ERR_INVALID_ARG;
  DevState st;
  CUDA_TRY(h, cudaMemcpyAsync(&st, h->P.st, sizeof st, cudaMemcpyDeviceToHost, h->stream));
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  int rc = drain_events(h);
  if (rc) return rc;
  memset(out, 0, sizeof *out);
  out->k = st.k;
  out->uploads_total = st.uploads_total; out->uploads_forced = st.uploads_forced; out->uploads_rule = st.uploads_rule;
  out->near_ties = st.near_ties; out->kernel_launches = h->launches;
  out->last_rhs = st.last_rhs; out->last_step_sqnorm = st.last_step_sqnorm;
  out->grad_kernel_ms = h->grad_ms; out->grad_kernel_launches = h->grad_launches;
  out->profiled_iterations = h->profiled_iters;
  out->status_flags = st.status_flags;
  out->path = h->use_cluster ? CADA_PATH_ONE_LAUNCH_CLUSTER : h->use_fused ? CADA_PATH_ONE_LAUNCH_GRID
              : h->use_softmax_cluster ? CADA_PATH_SOFTMAX_CLUSTER : h->use_mlp_hsplit ? CADA_PATH_MLP_HIDDEN_SPLIT : h->use_mlp_cluster ? CADA_PATH_MLP_CLUSTER
              : CADA_PATH_THREE_KERNELS;
  // device-detected problems surface here (`out` is complete either way) and at every later cada_step
  if (st.status_flags & CADA_FLAG_TIMEOUT) {
    h->device_error = CADA_ERR_TIMEOUT;
    return fail(h, CADA_ERR_TIMEOUT, "a bounded device-side wait ran out; the state of this handle is incomplete");
  }
  if (st.status_flags & CADA_FLAG_NONFINITE) {
    h->device_error = CADA_ERR_NONFINITE;
    return fail(h, CADA_ERR_NONFINITE, "a NaN or Inf reached the upload test");
  }
  return CADA_OK;
}

int cada_set_wait_limit(cada_handle* h, int64_t polls) {
  if (!h) return CADA_ERR_INVALID_ARG;
  if (polls < 0 || polls > (int64_t)0xFFFFFFFFll) return fail(h, CADA_ERR_INVALID_ARG, "polls outside [0, 2^32 - 1]");
  h->wait_limit = (unsigned)polls;
  return CADA_OK;
}

int cada_eval(cada_handle* h, double* host_loss, double* host_accuracy) {
  if (!h || !host_loss || !host_accuracy) return h ? fail(h, CADA_ERR_INVALID_ARG, "output pointer is NULL") : CADA_ERR_INVALID_ARG;
  const Params& P = h->P;
  if (P.model != CADA_MODEL_LOGISTIC && P.C > EV_CMAX) return fail(h, CADA_ERR_UNSUPPORTED, "evaluation supports up to 16 classes");
  if (P.model == CADA_MODEL_MLP2 && P.H > 256) return fail(h, CADA_ERR_UNSUPPORTED, "evaluation supports up to 256 hidden units");
  double* part = at<double>(h, h->L.eval_part);
  if (P.model == CADA_MODEL_MLP2) eval_mlp_kernel<<<dim3(EV_CHUNKS, P.M), EV_THREADS, 0, h->stream>>>(P, part);
  else eval_linear_kernel<<<dim3(EV_CHUNKS, P.M), EV_THREADS, 0, h->stream>>>(P, part);
  h->launches += 1;
  CUDA_TRY(h, cudaGetLastError());
  std::vector<double> host((size_t)2 * P.M * EV_CHUNKS);
  std::vector<float> theta((size_t)P.p);
  CUDA_TRY(h, cudaMemcpyAsync(host.data(), part, host.size() * sizeof(double), cudaMemcpyDeviceToHost, h->stream));
  CUDA_TRY(h, cudaMemcpyAsync(theta.data(), P.theta, theta.size() * sizeof(float), cudaMemcpyDeviceToHost, h->stream));
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  double loss = 0.0, correct = 0.0, rows = 0.0;
  for (int m = 0; m < P.M; ++m) {                       // Eq. 1: the average over workers of each worker's mean loss
    double lm = 0.0;
    for (int c = 0; c < EV_CHUNKS; ++c) { lm += host[((size_t)m * EV_CHUNKS + c) * 2]; correct += host[((size_t)m * EV_CHUNKS + c) * 2 + 1]; }
    loss += lm / (double)h->n_samples[m];
    rows += (double)h->n_samples[m];
  }
  double sq = 0.0;
  for (float t : theta) sq += (double)t * (double)t;
  *host_loss = loss / P.M + 0.5 * (double)P.lambda * sq;
  *host_accuracy = correct / rows;
  return CADA_OK;
}

int cada_read(cada_handle* h, int32_t which, void* host_dst, size_t bytes) {
  if (!h || !host_dst) return h ? fail(h, CADA_ERR_INVALID_ARG, "host_dst is NULL") : CADA_ERR_INVALID_ARG;
  BufInfo b;
  if (!buffer_info(h, which, b)) return fail(h, CADA_ERR_INVALID_ARG, "buffer not present in this configuration");
  if (bytes != b.elt * b.rows * b.cols) return fail(h, CADA_ERR_INVALID_ARG, "byte count does not match the buffer");
  CUDA_TRY(h, cudaMemcpy2DAsync(host_dst, b.cols * b.elt, b.ptr, b.pitch_elts * b.elt, b.cols * b.elt, b.rows,
                                cudaMemcpyDeviceToHost, h->stream));
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  return CADA_OK;
}

int cada_write(cada_handle* h, int32_t which, const void* host_src, size_t bytes) {
  if (!h || !host_src) return h ? fail(h, CADA_ERR_INVALID_ARG, "host_src is NULL") : CADA_ERR_INVALID_ARG;
  BufInfo b;
  if (!buffer_info(h, which, b)) return fail(h, CADA_ERR_INVALID_ARG, "buffer not present in this configuration");
  if (bytes != b.elt * b.rows * b.cols) return fail(h, CADA_ERR_INVALID_ARG, "byte count does not match the buffer");
  CUDA_TRY(h, cudaMemcpy2DAsync(b.ptr, b.pitch_elts * b.elt, host_src, b.cols * b.elt, b.cols * b.elt, b.rows,
                                cudaMemcpyHostToDevice, h->stream));
  CUDA_TRY(h, cudaStreamSynchronize(h->stream));
  if (which == CADA_BUF_K) h->k_host = *static_cast<const long long*>(host_src);
  if (h->use_mlp_cluster && (which == CADA_BUF_K || which == CADA_BUF_THETA || which == CADA_BUF_THETA_HAT ||
                             which == CADA_BUF_THETA_TILDE || which == CADA_BUF_TAU))
    h->ring_dirty = true;
  return CADA_OK;
}

int cada_profile(cada_handle* h, int32_t enable) {
  if (!h) return CADA_ERR_INVALID_ARG;
  h->profile = enable != 0;
  return CADA_OK;
}

int cada_destroy(cada_handle* h) {
  if (!h) return CADA_OK;
  cudaStreamSynchronize(h->stream);
  for (EventPair& ep : h->pending) { cudaEventDestroy(ep.a); cudaEventDestroy(ep.b); }
  for (EventPair& ep : h->spare) { cudaEventDestroy(ep.a); cudaEventDestroy(ep.b); }
  if (h->copy_ready) {
    cudaStreamSynchronize(h->copy_stream);
    for (int i = 0; i < 2; ++i) { cudaEventDestroy(h->ev_copied[i]); cudaEventDestroy(h->ev_done[i]); }
    cudaEventDestroy(h->ev_start);
    cudaStreamDestroy(h->copy_stream);
  }
  delete h;
  return CADA_OK;
}

const char* cada_last_error(const cada_handle* h) { return h ? h->err : g_create_error; }

#pragma GCC visibility pop
}  // extern "C"
