// Shared device-side declarations of libcada: the parameter block every kernel receives, the
// device-resident scalar state, the minibatch sampler and small reduction helpers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace cada {

// Scalars that live in device memory so that a whole iteration (and any number of them)
// runs without a host round trip: kernels read k here and the update kernel advances it.
struct DevState {
  long long k;                // iteration counter of Algorithm 1
  long long uploads_total;    // the paper's cost metric
  long long uploads_forced;   // uploads caused by tau >= D
  long long uploads_rule;     // uploads caused by a violated Eq. 6 / Eq. 8 alone
  long long near_ties;        // |LHS-RHS| <= 1e-4 max(LHS,RHS)
  double last_rhs;
  double last_step_sqnorm;
  int status_flags;
  unsigned int update_ticket; // "last block done" counter of the update kernel
  unsigned int grad_ticket;   // spare
  unsigned int pad;
  // An update kernel that is not the last of its call leaves the newest window term as per-block partial sums in
  // Params::step_part and says here which iteration has to add them up before it takes decisions (0: none pending).
  long long step_part_for;
  int step_part_n;
  int pad2;
};

enum { IDX_HASH = 0, IDX_EXPLICIT = 1, IDX_IDENTITY = 2 };

struct Params {
  // problem shape (Eq. 1 and the model)
  int model, rule, M, B, F, C, H, has_bias, d_max, D, x_bf16, server, aggregate;
  int Mg, m0, ms;     // workers of the whole problem; local worker i is worker m0 + i * ms of them (Mg = M, 0, 1: one handle holds all)
  long long p;        // dim theta
  long long ldp;      // pitch (floats) of every p-vector and of each row of the [M x p] buffers
  long long ldx;      // pitch (elements) of X rows
  float alpha, beta1, beta2, eps, c, lambda;
  float alpha_K0;           // > 0: alpha_k = alpha / (k + alpha_K0) (Theorem 2)
  const int* batch_m;       // per-worker minibatch sizes (<= B), or nullptr: all B
  unsigned long long seed;
  // data: device arrays of per-worker pointers / sizes
  const void* const* X;
  const void* const* y;
  const long long* n_samples;
  int idx_mode;
  const int* idx;           // explicit indices [n][M][B] (IDX_EXPLICIT)
  long long idx_k0;         // iteration the explicit block starts at
  // state
  DevState* st;
  float* theta; float* h; float* vhat; float* theta_tilde;        // [ldp]
  float* G; float* theta_hat; float* delta_stored;                // [M x ldp]
  float* g_fresh; float* d_fresh;                                 // [M x ldp]
  float* nabla;             // [ldp] aggregate of the previous iteration (Eq. 3), recursive aggregation only
  float* part;              // partial gradient sums [slot][2][ldp]
  int* tau; unsigned char* mask; double* lhs; long long* up_per_worker;
  double* ring; double* norm_part; double* step_part;
  unsigned int* worker_ticket;
  double* hist_lhs; double* hist_rhs; unsigned char* hist_mask; int hist_cap;
  // launch geometry shared between kernels
  int n_chunks;             // partial slots per worker
  int rows_per_chunk;
  int trig_splits;          // CTAs per worker in the trigger kernel
  int trig_cols;            // floats of p handled by one trigger CTA (multiple of 4)
  int upd_ty;               // worker lanes of the update kernel's block
  // ring of bf16 operand images of the network's first-layer weights, one slot per iteration (null: not in use):
  // slot j mod w1_slots holds the image of theta^j; the update kernel writes the image of theta^{k+1}
  unsigned char* w1_ring;
  int w1_slots;             // D + 1
  int w1_nhc;               // hidden chunks of 8 per feature row of an image
  unsigned w1_set_bytes;    // bytes of one image
  unsigned w1_chunk_bytes;  // bytes of the 112-feature chunk of an image (w1_hsplit: of one 32-unit hidden slice)
  int w1_hsplit;            // 1: an image is laid out as contiguous 32-unit hidden slices (mlp_hsplit.cuh), 0: as 112-feature chunks
};

// SplitMix64 (Steele, Lea, Flood, OOPSLA 2014) as a counter-based generator: the (n+1)-th
// output of the stream started at `seed`.
__device__ __forceinline__ unsigned long long splitmix64_at(unsigned long long seed, unsigned long long n) {
  unsigned long long z = seed + (n + 1ull) * 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// x mod n for 64-bit x with a precomputed mu = floor((2^64 - 1) / n): one high multiply and at most two
// corrections instead of a 64-bit division; the result is exactly x % n.
__device__ __forceinline__ unsigned long long mod_by(unsigned long long x, unsigned long long n, unsigned long long mu) {
  unsigned long long r = x - __umul64hi(x, mu) * n;
  if (r >= n) r -= n;
  if (r >= n) r -= n;
  return r;
}

// Row of worker m's data used as element j of its minibatch at iteration k.
// `mu` = floor((2^64 - 1) / n_m) if the caller has it (0: divide).
__device__ __forceinline__ long long minibatch_row(const Params& P, long long k, int m, int j, long long n_m,
                                                   unsigned long long mu = 0) {
  if (P.idx_mode == IDX_HASH) {
    unsigned long long n = ((unsigned long long)k * (unsigned long long)P.Mg + (unsigned long long)(P.m0 + m * P.ms)) *
                               (unsigned long long)P.B + (unsigned long long)j;
    const unsigned long long x = splitmix64_at(P.seed, n);
    return (long long)(mu ? mod_by(x, (unsigned long long)n_m, mu) : x % (unsigned long long)n_m);
  }
  if (P.idx_mode == IDX_IDENTITY) return j;
  long long r = P.idx[((k - P.idx_k0) * P.M + m) * (long long)P.B + j];
  if (r < 0 || r >= n_m) {
    atomicOr(&P.st->status_flags, 2);
    r = r < 0 ? 0 : n_m - 1;
  }
  return r;
}

// Rows worker m averages over (the supplement's batch ratio gives workers of different size different counts).
__device__ __forceinline__ int worker_batch(const Params& P, int m) { return P.batch_m ? P.batch_m[m] : P.B; }

// Step size of iteration k: constant, or Theorem 2's alpha / (k + K0).
__device__ __forceinline__ float step_size(const Params& P, long long k) {
  return P.alpha_K0 > 0.f ? P.alpha / ((float)k + P.alpha_K0) : P.alpha;
}

// The iterate the second gradient is taken at: the snapshot (CADA1; it equals theta^k on
// iterations with k mod D == 0, when Algorithm 1 refreshes it before the gradients) or the
// iterate of worker m's last upload (CADA2).
__device__ __forceinline__ const float* old_iterate(const Params& P, long long k, int m) {
  if (P.rule == 1) return (k % P.D == 0) ? P.theta : P.theta_tilde;
  if (P.rule == 3) return P.theta;              // stochastic LAG takes one gradient: the difference is identically 0
  return P.theta_hat + (long long)m * P.ldp;
}

// Worker m's upload decision at iteration k (Algorithm 1: upload when Eq. 6 / Eq. 8 is violated or tau_m >= D), taken
// by ONE thread once the left-hand side is complete: right-hand side (c / d_max) * sum of the window of squared step
// norms (fp64, re-summed), staleness update, counters, near-tie count and the optional history ring.
__device__ __forceinline__ double window_rhs(const Params& P) {
  if (isinf(P.c)) return (double)INFINITY;
  double w = 0.0;
  for (int i = 0; i < P.d_max; ++i) w += P.ring[i];
  return ((double)P.c / (double)P.d_max) * w;
}
// `tau` is the worker's staleness: a caller that decides at the very end of its kernel loads it early (right after its wait for
// the preceding kernel), so that no load latency sits between the left-hand side and the kernel's end.
__device__ __forceinline__ void decide_upload_tau(const Params& P, long long k, int m, double lhs, double rhs /* window_rhs(P) */, int tau) {
  const bool forced = tau >= P.D;
  const bool violated = !(lhs <= rhs);
  const bool up = violated || forced;
  const unsigned char bits = (unsigned char)((up ? 1 : 0) | (forced ? 2 : 0));
  P.mask[m] = bits;
  P.lhs[m] = lhs;
  P.tau[m] = up ? 1 : tau + 1;
  if (up) {
    atomicAdd((unsigned long long*)&P.st->uploads_total, 1ull);
    atomicAdd((unsigned long long*)(forced ? &P.st->uploads_forced : &P.st->uploads_rule), 1ull);
    atomicAdd((unsigned long long*)&P.up_per_worker[m], 1ull);    // (one thread per worker: the atomic only spares the wait for a load)
  }
  if (!isfinite(lhs) || isnan(rhs)) atomicOr(&P.st->status_flags, 1);
  if (!isinf(rhs)) {
    const double big = fmax(lhs, rhs);
    if (fabs(lhs - rhs) <= 1e-4 * big && big > 0.0) atomicAdd((unsigned long long*)&P.st->near_ties, 1ull);
  }
  if (m == 0) P.st->last_rhs = rhs;
  if (P.hist_cap > 0) {
    const long long slot = k % P.hist_cap;
    P.hist_lhs[slot * P.M + m] = lhs;
    P.hist_mask[slot * P.M + m] = bits;
    if (m == 0) P.hist_rhs[slot] = rhs;
  }
}

__device__ __forceinline__ void decide_upload(const Params& P, long long k, int m, double lhs, double rhs /* window_rhs(P) */) {
  decide_upload_tau(P, k, m, lhs, rhs, P.tau[m]);
}

// Programmatic dependent launch: a kernel launched with the programmatic-serialisation attribute may start while
// its predecessor in the stream is still running.  pdl_wait() returns once the predecessor grid has completed and
// its writes are visible (everything that reads data the predecessor produces comes after it); pdl_trigger() lets
// the successor be scheduled from now on.  Both are no-ops for a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum over a block of up to 1024 threads in a fixed order; result valid in thread 0.
// The newest term of the window of Eq. 6 / Eq. 8, ||theta^k - theta^{k-1}||^2, as iteration k needs it for its decisions.
// The update kernel of iteration k-1 adds its blocks' partial sums itself only when it is the last kernel of a call
// (a ticket, a fence and a second pass: 2-3 us at the end of every iteration); otherwise it leaves the partials and
// whoever decides at iteration k calls this with ONE warp first, after its wait for that kernel and before a barrier
// that orders it ahead of decide_upload.  Fixed order (lane-strided, then the shuffle tree); every caller computes and
// stores the same value.
__device__ __forceinline__ void window_refresh(const Params& P, long long k, int lane) {
  if (P.st->step_part_for != k) return;
  const int n = P.st->step_part_n;
  double s = 0.0;
  for (int b = lane; b < n; b += 32) s += __ldcg(&P.step_part[b]);
  s = warp_sum(s);
  if (lane == 0) {
    P.ring[(k - 1) % P.d_max] = s;
    P.st->last_step_sqnorm = s;
  }
}

// The same, followed by the right-hand side of this iteration (lane 0 adds the window in index order; every lane gets it):
// taken early, the window's loads are off the end of the deciding kernel.
__device__ __forceinline__ double window_refresh_rhs(const Params& P, long long k, int lane) {
  window_refresh(P, k, lane);
  double rhs = 0.0;
  if (lane == 0) rhs = window_rhs(P);
  return __shfl_sync(0xffffffffu, rhs, 0);
}

__device__ __forceinline__ double block_sum(double v, double* scratch /* >= 32 doubles */) {
  const int nthreads = blockDim.x * blockDim.y;
  const int tid = threadIdx.y * blockDim.x + threadIdx.x;
  v = warp_sum(v);
  if ((tid & 31) == 0) scratch[tid >> 5] = v;
  __syncthreads();
  double total = 0.0;
  if (tid == 0) {
    const int nw = (nthreads + 31) >> 5;
    for (int w = 0; w < nw; ++w) total += scratch[w];
  }
  return total;
}

// sigma(z) and the accurate difference sigma(z) - sigma(z - dz).
__device__ __forceinline__ float sigmoidf_stable(float z) {
  float e = expf(-fabsf(z));
  return z >= 0.f ? 1.f / (1.f + e) : e / (1.f + e);
}
// sigma(a) - sigma(b) = sigma(a) * sigma(-b) * (1 - exp(-(a-b))): no cancellation for small a-b.
__device__ __forceinline__ float sigmoid_diff(float z, float dz) {
  if (fabsf(dz) > 20.f) return sigmoidf_stable(z) - sigmoidf_stable(z - dz);
  return sigmoidf_stable(z) * sigmoidf_stable(dz - z) * (-expm1f(-dz));
}

// Short-latency versions for the streaming kernel, whose consumers all wait on this result:
// sigma(z) - t and sigma(z) - sigma(z - dz) from ex2.approx-based exponentials, approximate
// reciprocals and a 6-term series for 1 - exp(-dz) at small |dz|.  Absolute error of either
// output is a few 1e-7 (|z| up to ~30), and the difference keeps ~1e-6 relative accuracy.
__device__ __forceinline__ void sigmoid_pair_fast(float z, float dz, float& sig, float& dsig) {
  const float e = __expf(-fabsf(z));
  sig = __fdividef(z >= 0.f ? 1.f : e, 1.f + e);
  const float w = dz - z;                       // -(z - dz)
  const float e2 = __expf(-fabsf(w));
  const float sigw = __fdividef(w >= 0.f ? 1.f : e2, 1.f + e2);       // sigma(-(z - dz))
  const float t = -dz;
  float em1;                                    // exp(-dz) - 1
  if (fabsf(t) < 0.125f) {
    em1 = t * (1.f + t * (0.5f + t * (1.f / 6.f + t * (1.f / 24.f + t * (1.f / 120.f + t * (1.f / 720.f))))));
  } else {
    em1 = __expf(t) - 1.f;
  }
  dsig = fabsf(dz) > 20.f ? sig - (1.f - sigw) : sig * sigw * (-em1);
}

}  // namespace cada
