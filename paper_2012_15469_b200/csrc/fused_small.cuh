// Whole CADA iterations in one launch for small binary-logistic problems (tens of workers, rows
// of up to ~2 KB): the case where three dependent launches per iteration cost far more than the
// arithmetic.  One CTA per worker, launched cooperatively so that all of them are resident; the
// kernel loops over n iterations with ONE grid-wide barrier per iteration.
//
// Per iteration k (Algorithm 1), CTA m:
//   top      start the copy (cp.async) of iteration k+1's minibatch rows into the other half of a
//            double buffer -- they do not depend on theta, so DRAM latency leaves the critical path
//   worker   forward: one thread per minibatch row, z = x.theta and dz = x.(theta - theta') from
//            shared memory; residuals; backward: threads own (feature, row group) pairs; g_m, d_m,
//            the left-hand side of Eq. 6 / Eq. 8 in fp64, the decision with the tau >= D clause.
//            An uploading worker writes its gradient into the slot buffer that is NOT current and
//            flips its selector; selector and decision go to a per-parity flag array.
//   barrier  every CTA publishes one flag word (iteration tag, selector, decision) with release
//            semantics and thread w of every CTA waits (bounded) for worker w's word: no atomics
//   server   every CTA redundantly sums the M current slots in worker order and applies
//            Eqs. 2a-2c to its own shared-memory copy of theta, h, vhat and of the window of
//            squared step norms, so no second barrier or broadcast is needed.
// Why one barrier is enough: a CTA that runs ahead into iteration k+1 can only write the slot
// buffer that the laggards (still in the server phase of k) are not reading, and it writes the
// flag array of the other parity; it cannot get two iterations ahead because of the barrier.
// Global state is read at kernel start and written back at the end (CTA 0: theta, h, vhat,
// window, k; each CTA: its worker's records), so cada_read / cada_write and the three-kernel
// path see the same layout.
#pragma once
#include "common.cuh"

namespace cada {

constexpr int FS_THREADS = 256;
constexpr unsigned FS_SPIN_LIMIT = 1u << 22;

struct FusedGeom {
  int pp;          // p rounded up to a multiple of 4
  int pitch;       // floats between staged rows in shared memory: multiple of 4 with pitch/4 odd
  int f4;          // 16-byte chunks per row (ceil(F / 4))
  int nqb;         // quads of theta (pp / 4): the backward pass's column groups
  int nrg;         // row groups of the backward pass (threads = nqb * nrg <= FS_THREADS)
  int wt;          // workers whose slots are staged per pass of the server phase
  size_t smem_bytes;
  // byte offsets into dynamic shared memory
  unsigned off_theta, off_h, off_vhat, off_old, off_dth, off_dstored, off_g, off_d, off_part, off_res, off_rows,
      off_y, off_x, off_ring, off_red, off_misc, off_flags, off_gst;
};

__host__ inline bool fused_plan(int F, int has_bias, int B, int d_max, int rule, int M, FusedGeom& g) {
  const int p = F + has_bias;
  if (F > 508 || B > 1024 || M > 160) return false;
  g.pp = (p + 3) / 4 * 4;
  g.f4 = (F + 3) / 4;
  g.pitch = (g.f4 | 1) * 4;              // odd number of 16-byte chunks: conflict-free row-per-thread float4 reads
  g.nqb = g.pp / 4;
  g.nrg = FS_THREADS / g.nqb;
  if (g.nrg < 1) g.nrg = 1;
  if (g.nrg > 32) g.nrg = 32;
  if (g.nrg > B) g.nrg = B;
  g.wt = 8192 / g.pp;                    // at most 32 KB of staged slots
  if (g.wt > M) g.wt = M;
  if (g.wt < 1) g.wt = 1;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = (o + bytes + 15) / 16 * 16; return (unsigned)at; };
  g.off_ring = take(sizeof(double) * (d_max + 2));            // window | rhs | spare
  g.off_red = take(sizeof(double) * 32);
  g.off_theta = take(4 * g.pp); g.off_h = take(4 * g.pp); g.off_vhat = take(4 * g.pp);
  g.off_old = take(4 * g.pp); g.off_dth = take(4 * g.pp);
  g.off_dstored = take(rule == 1 ? 4 * g.pp : 0);
  g.off_g = take(4 * g.pp); g.off_d = take(4 * g.pp);
  g.off_part = take((size_t)4 * g.nrg * 2 * g.pp);
  g.off_res = take((size_t)4 * 2 * B);
  g.off_rows = take((size_t)8 * 2 * B);
  g.off_y = take((size_t)4 * 2 * B);
  g.off_x = take((size_t)4 * 2 * B * g.pitch);
  g.off_misc = take(64);
  g.off_flags = take(4 * 160);
  g.off_gst = take((size_t)4 * g.wt * g.pp);
  g.smem_bytes = o;
  return o <= 200 * 1024;
}

__device__ __forceinline__ void cp_async16(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async4(void* smem_dst, const void* gsrc) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(smem_dst)), "l"(gsrc) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Fixed-order block sum of doubles (FS_THREADS threads); every thread gets the result.
__device__ __forceinline__ double fs_block_sum(double v, double* red) {
  v = warp_sum(v);
  __syncthreads();                       // protects `red` against readers of the previous use
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
  __syncthreads();
  double t = 0.0;
#pragma unroll
  for (int w = 0; w < FS_THREADS / 32; ++w) t += red[w];
  return t;
}

__global__ void __launch_bounds__(FS_THREADS, 1)
fused_logistic_kernel(const __grid_constant__ Params P, const __grid_constant__ FusedGeom fg, int n_iters,
                      float* __restrict__ G_alt, unsigned int* __restrict__ flags /* [2][M], zeroed before the launch */,
                      unsigned spin_limit /* polls spent on one flag before the launch is abandoned */) {
  extern __shared__ __align__(16) unsigned char sm[];
  double* s_ring = reinterpret_cast<double*>(sm + fg.off_ring);     // [d_max] window, [d_max] = RHS of the current iteration
  double* s_red = reinterpret_cast<double*>(sm + fg.off_red);
  float* s_theta = reinterpret_cast<float*>(sm + fg.off_theta);
  float* s_h = reinterpret_cast<float*>(sm + fg.off_h);
  float* s_vhat = reinterpret_cast<float*>(sm + fg.off_vhat);
  float* s_old = reinterpret_cast<float*>(sm + fg.off_old);        // theta' : theta_hat_m (CADA2) or the snapshot (CADA1)
  float* s_dth = reinterpret_cast<float*>(sm + fg.off_dth);        // theta - theta'
  float* s_dst = reinterpret_cast<float*>(sm + fg.off_dstored);    // CADA1: innovation stored at the last upload
  float* s_g = reinterpret_cast<float*>(sm + fg.off_g);
  float* s_d = reinterpret_cast<float*>(sm + fg.off_d);
  float* s_part = reinterpret_cast<float*>(sm + fg.off_part);      // [nrg][2][pp]
  float* s_res = reinterpret_cast<float*>(sm + fg.off_res);        // [2][B] : r | dr
  long long* s_rows = reinterpret_cast<long long*>(sm + fg.off_rows);  // [2][B]
  float* s_y = reinterpret_cast<float*>(sm + fg.off_y);            // [2][B]
  float* s_x = reinterpret_cast<float*>(sm + fg.off_x);            // [2][B][pitch]
  int* s_misc = reinterpret_cast<int*>(sm + fg.off_misc);          // [0] upload decision | selector, [1] abort
  unsigned* s_flags = reinterpret_cast<unsigned*>(sm + fg.off_flags);   // this iteration's flag word of every worker
  float* s_gst = reinterpret_cast<float*>(sm + fg.off_gst);        // [wt][pp] staged slots of the server phase

  const int tid = threadIdx.x, m = blockIdx.x, M = P.M, B = P.B, F = P.F, p = (int)P.p;
  const bool cada1 = P.rule == 1;
  const long long k0 = P.st->k;
  const float* __restrict__ Xm = static_cast<const float*>(P.X[m]);
  const float* __restrict__ ym = static_cast<const float*>(P.y[m]);
  const long long n_m = P.n_samples[m];
  const unsigned long long mu_m = ~0ull / (unsigned long long)n_m;
  const int Bm = worker_batch(P, m);                  // rows this worker averages over; buffers keep the stride B

  // ---- load state ------------------------------------------------------------------------------
  for (int j = tid; j < fg.pp; j += FS_THREADS) {
    const bool in = j < p;
    s_theta[j] = in ? P.theta[j] : 0.f;
    s_h[j] = in ? P.h[j] : 0.f;
    s_vhat[j] = in ? P.vhat[j] : 0.f;
    s_old[j] = in ? (cada1 ? P.theta_tilde[j] : P.theta_hat[(long long)m * P.ldp + j]) : 0.f;
    if (cada1) s_dst[j] = in ? P.delta_stored[(long long)m * P.ldp + j] : 0.f;
    s_g[j] = 0.f; s_d[j] = 0.f;
  }
  for (int j = tid; j < P.d_max; j += FS_THREADS) s_ring[j] = P.ring[j];
  if (tid == 0) { s_misc[0] = 0; s_misc[1] = 0; }
  int tau = P.tau[m];
  unsigned sel = 0;                                   // thread 0: which slot buffer holds worker m's current gradient
  long long n_up = 0, n_forced = 0, n_ties = 0;       // thread 0 only
  double last_lhs = 0.0, last_rhs = 0.0, last_step = 0.0;
  unsigned char last_bits = 0;

  // Minibatch staging, split so that nothing of it sits on the critical path: row indices and labels are
  // handled by the highest-numbered threads (idle while the low ones run the forward pass), the row copies
  // are issued by everyone after the forward pass's barrier.
  auto stage_indices = [&](long long k, int buf) {
    for (int j = FS_THREADS - 1 - tid; j < Bm; j += FS_THREADS) {
      const long long row = minibatch_row(P, k, m, j, n_m, mu_m);
      s_rows[buf * B + j] = row * P.ldx;               // element offset of the row
      cp_async4(&s_y[buf * B + j], ym + row);
    }
  };
  auto stage_copies = [&](int buf) {
    float* xb = s_x + (size_t)buf * B * fg.pitch;
    int j = tid / fg.f4, q = tid - j * fg.f4;
    const int dj = FS_THREADS / fg.f4, dq = FS_THREADS - dj * fg.f4;
    while (j < Bm) {
      cp_async16(xb + (size_t)j * fg.pitch + 4 * q, Xm + s_rows[buf * B + j] + 4 * q);
      j += dj; q += dq;
      if (q >= fg.f4) { q -= fg.f4; ++j; }
    }
    cp_async_commit();
  };

  // per-thread constants of the backward pass: quad q of theta, row group rg
  const int bw_rg = tid / fg.nqb, bw_q = tid - bw_rg * fg.nqb;
  const bool bw_active = bw_rg < fg.nrg;
  int bw_kind[4];                                     // 0: feature column, 1: the constant-1 column, 2: padding
#pragma unroll
  for (int e = 0; e < 4; ++e) { const int c = 4 * bw_q + e; bw_kind[e] = c < F ? 0 : (c == F && P.has_bias) ? 1 : 2; }

  stage_indices(k0, 0);
  __syncthreads();
  stage_copies(0);

  for (int it = 0; it < n_iters; ++it) {
    const long long k = k0 + it;
    const int buf = it & 1;
    const bool more = it + 1 < n_iters;
    // Algorithm 1, snapshot step (CADA1): theta~ <- theta^k before the gradients when k mod D == 0
    const bool snap = cada1 && (k % P.D == 0);
    for (int j = tid; j < fg.pp; j += FS_THREADS) {
      if (snap) s_old[j] = s_theta[j];
      s_dth[j] = s_theta[j] - s_old[j];
    }
    if (tid == FS_THREADS - 1) {                        // right-hand side of Eqs. 6 / 8 for this iteration
      double rhs;
      if (isinf(P.c)) rhs = (double)INFINITY;
      else { double w = 0.0; for (int i = 0; i < P.d_max; ++i) w += s_ring[i]; rhs = ((double)P.c / (double)P.d_max) * w; }
      s_ring[P.d_max] = rhs;
    }
    cp_async_wait<0>();
    __syncthreads();

    // ---- worker: forward, one thread per minibatch row ---------------------------------------
    if (more) stage_indices(k + 1, buf ^ 1);
    const float* xb = s_x + (size_t)buf * B * fg.pitch;
    const float invB = 1.0f / (float)Bm;
    for (int j = tid; j < Bm; j += FS_THREADS) {
      const float4* xr = reinterpret_cast<const float4*>(xb + (size_t)j * fg.pitch);
      float z = 0.f, dz = 0.f;
      const int qfull = F >> 2;                        // chunks whose four columns are all features
#pragma unroll 4
      for (int q = 0; q < qfull; ++q) {
        const float4 x = xr[q];
        const float4 t = reinterpret_cast<const float4*>(s_theta)[q];
        const float4 e = reinterpret_cast<const float4*>(s_dth)[q];
        z = fmaf(x.x, t.x, z); dz = fmaf(x.x, e.x, dz);
        z = fmaf(x.y, t.y, z); dz = fmaf(x.y, e.y, dz);
        z = fmaf(x.z, t.z, z); dz = fmaf(x.z, e.z, dz);
        z = fmaf(x.w, t.w, z); dz = fmaf(x.w, e.w, dz);
      }
      if (qfull < fg.f4) {                             // last chunk: columns beyond F are the caller's row padding
        const float4 x = xr[qfull];
        const int f = 4 * qfull;
        z = fmaf(x.x, s_theta[f], z); dz = fmaf(x.x, s_dth[f], dz);
        if (f + 1 < F) { z = fmaf(x.y, s_theta[f + 1], z); dz = fmaf(x.y, s_dth[f + 1], dz); }
        if (f + 2 < F) { z = fmaf(x.z, s_theta[f + 2], z); dz = fmaf(x.z, s_dth[f + 2], dz); }
      }
      if (P.has_bias) { z += s_theta[F]; dz += s_dth[F]; }
      float sig, dsig;
      sigmoid_pair_fast(z, dz, sig, dsig);
      s_res[j] = (sig - 0.5f * (s_y[buf * B + j] + 1.0f)) * invB;
      s_res[B + j] = dsig * invB;
    }
    __syncthreads();
    if (more) stage_copies(buf ^ 1);
    // ---- worker: backward, thread = (quad of columns, row group) -----------------------------
    if (bw_active) {
      float ag[4] = {0.f, 0.f, 0.f, 0.f}, ad[4] = {0.f, 0.f, 0.f, 0.f};
      const bool has_x = bw_q < fg.f4;
#pragma unroll 2
      for (int i = bw_rg; i < Bm; i += fg.nrg) {
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (has_x) x = *reinterpret_cast<const float4*>(xb + (size_t)i * fg.pitch + 4 * bw_q);
        const float xs[4] = {x.x, x.y, x.z, x.w};
        const float r = s_res[i], dr = s_res[B + i];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float xv = bw_kind[e] == 0 ? xs[e] : bw_kind[e] == 1 ? 1.f : 0.f;
          ag[e] = fmaf(r, xv, ag[e]);
          ad[e] = fmaf(dr, xv, ad[e]);
        }
      }
      *reinterpret_cast<float4*>(s_part + (bw_rg * 2 + 0) * fg.pp + 4 * bw_q) = make_float4(ag[0], ag[1], ag[2], ag[3]);
      *reinterpret_cast<float4*>(s_part + (bw_rg * 2 + 1) * fg.pp + 4 * bw_q) = make_float4(ad[0], ad[1], ad[2], ad[3]);
    }
    __syncthreads();
    double acc = 0.0;
    for (int j = tid; j < p; j += FS_THREADS) {
      float g = 0.f, d = 0.f;
#pragma unroll 6
      for (int r = 0; r < fg.nrg; ++r) { g += s_part[(r * 2 + 0) * fg.pp + j]; d += s_part[(r * 2 + 1) * fg.pp + j]; }
      g = fmaf(P.lambda, s_theta[j], g);
      d = fmaf(P.lambda, s_dth[j], d);
      s_g[j] = g; s_d[j] = d;
      const float e = cada1 ? d - s_dst[j] : d;
      acc = fma((double)e, (double)e, acc);
    }
    const double lhs = fs_block_sum(acc, s_red);          // left-hand side of Eq. 6 / Eq. 8
    if (tid == 0) {
      const double rhs = s_ring[P.d_max];
      const bool forced = tau >= P.D, violated = !(lhs <= rhs), up = violated || forced;
      last_bits = (unsigned char)((up ? 1 : 0) | (forced ? 2 : 0));
      last_lhs = lhs; last_rhs = rhs;
      tau = up ? 1 : tau + 1;
      if (up) { ++n_up; if (forced) ++n_forced; sel ^= 1u; }
      s_misc[0] = (up ? 1 : 0) | (int)(sel << 1);
    }
    __syncthreads();
    const bool up = s_misc[0] & 1;
    const unsigned my_sel = (unsigned)(s_misc[0] >> 1) & 1u;
    if (up) {                                             // upload: fresh gradient into the non-current slot buffer
      float* dst = (my_sel ? G_alt : P.G) + (long long)m * P.ldp;
      for (int q = tid; q < fg.nqb; q += FS_THREADS)
        reinterpret_cast<float4*>(dst)[q] = reinterpret_cast<const float4*>(s_g)[q];
      for (int j = tid; j < fg.pp; j += FS_THREADS) {
        if (cada1) s_dst[j] = s_d[j]; else s_old[j] = s_theta[j];
      }
    }
    __syncthreads();
    // ---- grid barrier: every worker publishes (iteration tag | selector | decision); all wait for all ----
    if (tid == 0) {
      // release at gpu scope: the slot written above (ordered by the barrier before) is visible before the flag
      const unsigned word = ((unsigned)(it + 1) << 8) | (my_sel << 2) | (unsigned)last_bits;
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(flags + (it & 1) * M + m), "r"(word) : "memory");
      // bookkeeping that nobody waits for
      const double lhs0 = last_lhs, rhs0 = last_rhs;
      if (!isfinite(lhs0) || isnan(rhs0)) atomicOr(&P.st->status_flags, 1);
      if (!isinf(rhs0)) { const double big = fmax(lhs0, rhs0); if (fabs(lhs0 - rhs0) <= 1e-4 * big && big > 0.0) ++n_ties; }
      if (P.hist_cap > 0) {
        const long long slot = k % P.hist_cap;
        P.hist_lhs[slot * M + m] = lhs0; P.hist_mask[slot * M + m] = last_bits;
        if (m == 0) P.hist_rhs[slot] = rhs0;
      }
    }
    if (tid >= 32 && tid < 32 + M) {                      // warps 1.. poll, one worker per thread (M <= 160)
      const int w = tid - 32;
      const unsigned* fp = flags + (it & 1) * M + w;
      unsigned v = 0, spins = 0;
      while (true) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(fp) : "memory");
        if ((v >> 8) == (unsigned)(it + 1)) break;
        if (++spins > spin_limit) { atomicOr(&P.st->status_flags, 4); s_misc[1] = 1; break; }
      }
      s_flags[w] = v;
    }
    __syncthreads();
    if (s_misc[1]) {                                      // a wait ran out: the launch is abandoned,
      cp_async_wait<0>();                                 // once this CTA's own prefetch of the next minibatch has landed
      return;
    }
    // ---- server: aggregate the current slots in worker order, Eqs. 2a-2c ---------------------
    float sum = 0.f;                                      // thread j < p owns coordinate j (p <= 2 * FS_THREADS)
    float sum2 = 0.f;
    for (int w0 = 0; w0 < M; w0 += fg.wt) {
      const int nw = min(fg.wt, M - w0);
      for (int c = tid; c < nw * fg.nqb; c += FS_THREADS) {
        const int wl = c / fg.nqb, q = c - wl * fg.nqb;
        const float* src = ((s_flags[w0 + wl] >> 2) & 1u) ? G_alt : P.G;
        const float4 v = __ldcg(reinterpret_cast<const float4*>(src + (long long)(w0 + wl) * P.ldp) + q);
        reinterpret_cast<float4*>(s_gst + (size_t)wl * fg.pp)[q] = v;
      }
      __syncthreads();
      for (int wl = 0; wl < nw; ++wl) {
        if (tid < p) sum += s_gst[(size_t)wl * fg.pp + tid];
        if (tid + FS_THREADS < p) sum2 += s_gst[(size_t)wl * fg.pp + tid + FS_THREADS];
      }
      if (w0 + fg.wt < M) __syncthreads();
    }
    double dsq = 0.0;
    const float invM = 1.0f / (float)M, alpha_k = step_size(P, k);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const int j = tid + half * FS_THREADS;
      if (j < p) {
        const float nab = (half ? sum2 : sum) * invM;
        const float hn = P.beta1 * s_h[j] + (1.0f - P.beta1) * nab;
        const float v = P.beta2 * s_vhat[j] + (1.0f - P.beta2) * nab * nab;
        const float vn = fmaxf(v, s_vhat[j]);
        const float t = s_theta[j];
        const float tn = t - alpha_k * hn / sqrtf(P.eps + vn);
        const double dl = (double)tn - (double)t;
        dsq = fma(dl, dl, dsq);
        s_h[j] = hn; s_vhat[j] = vn; s_theta[j] = tn;
      }
    }
    const double step = fs_block_sum(dsq, s_red);
    if (tid == 0) { s_ring[k % P.d_max] = step; last_step = step; }
    __syncthreads();
  }

  // ---- write the state back ----------------------------------------------------------------
  cp_async_wait<0>();
  const long long k_end = k0 + n_iters;
  const bool alt_is_current = n_iters > 0 && ((s_misc[0] >> 1) & 1);   // selector after the last iteration (thread 0 owns `sel`)
  for (int j = tid; j < p; j += FS_THREADS) {
    if (m == 0) {
      P.theta[j] = s_theta[j]; P.h[j] = s_h[j]; P.vhat[j] = s_vhat[j];
      if (cada1) P.theta_tilde[j] = s_old[j];
    }
    if (cada1) P.delta_stored[(long long)m * P.ldp + j] = s_dst[j];
    else P.theta_hat[(long long)m * P.ldp + j] = s_old[j];
    P.g_fresh[(long long)m * P.ldp + j] = s_g[j];
    P.d_fresh[(long long)m * P.ldp + j] = s_d[j];
    if (alt_is_current) P.G[(long long)m * P.ldp + j] = G_alt[(long long)m * P.ldp + j];   // make the primary buffer current again
  }
  if (m == 0) for (int j = tid; j < P.d_max; j += FS_THREADS) P.ring[j] = s_ring[j];
  if (tid == 0) {
    P.tau[m] = tau; P.mask[m] = last_bits; P.lhs[m] = last_lhs; P.up_per_worker[m] += n_up;
    atomicAdd((unsigned long long*)&P.st->uploads_total, (unsigned long long)n_up);
    atomicAdd((unsigned long long*)&P.st->uploads_forced, (unsigned long long)n_forced);
    atomicAdd((unsigned long long*)&P.st->uploads_rule, (unsigned long long)(n_up - n_forced));
    atomicAdd((unsigned long long*)&P.st->near_ties, (unsigned long long)n_ties);
    if (m == 0) { P.st->last_rhs = last_rhs; P.st->last_step_sqnorm = last_step; P.st->k = k_end; }
  }
}

}  // namespace cada
