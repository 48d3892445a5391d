// The two small kernels that finish a CADA iteration after the gradients.
//
// trigger_kernel (worker side of Algorithm 1): sums each worker's partial gradient slots in a
//   fixed order, adds the regulariser, keeps g_m and d_m for the server, and forms the
//   left-hand side of Eq. 6 (CADA1: ||d_m - stored d_m||^2) or Eq. 8 (CADA2: ||d_m||^2) in the
//   same pass.  The CTA that finishes a worker last compares with the right-hand side
//   (c/d_max) * sum of the window of squared step norms, applies the tau >= D clause, and
//   writes the decision, the new staleness and the counters.
//
// update_kernel (server side, Eqs. 2a-2c): for every coordinate, walks the workers in order;
//   an uploading worker's slot is overwritten by its fresh gradient (and its old-iterate /
//   stored-innovation record refreshed) with 128-bit stores while the same value enters the
//   aggregate (with the recursive aggregate of Eq. 3 only uploading workers are read: their
//   innovation against the last upload is added to the kept nabla^{k-1}); then h, vhat and
//   theta are updated and the squared step norm is reduced into the window slot k mod d_max.
//   The block that finishes last advances k.
#pragma once
#include <math.h>
#include "common.cuh"
#include "mlp_cluster.cuh"   // mlp_ring_store4

namespace cada {

constexpr int TRIG_THREADS = 256;
constexpr int UPD_THREADS = 256;

__global__ void __launch_bounds__(TRIG_THREADS, 6) trigger_kernel(const __grid_constant__ Params P) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  __shared__ double s_red[32];
  __shared__ unsigned int s_ticket;
  const int m = blockIdx.y, s = blockIdx.x, tid = threadIdx.x;
  const long long k = P.st->k;
  double rhs = 0.0;
  if (tid < 32) rhs = window_refresh_rhs(P, k, tid);     // the newest window term, if the preceding update kernel left it in parts; this iteration's right-hand side
  const long long c0 = (long long)s * P.trig_cols;
  const long long c1 = min(P.p, c0 + (long long)P.trig_cols);
  const float* __restrict__ tho = old_iterate(P, k, m);
  const float* __restrict__ part = P.part + (long long)m * P.n_chunks * 2 * P.ldp;
  float* __restrict__ gf = P.g_fresh + (long long)m * P.ldp;
  float* __restrict__ df = P.d_fresh + (long long)m * P.ldp;
  const float* ds = P.delta_stored ? P.delta_stored + (long long)m * P.ldp : nullptr;
  const bool cada1 = (P.rule == 1), lag = (P.rule == 3);
  if (lag) ds = P.G + (long long)m * P.ldp;        // Eq. 4 compares with the copy the server holds

  double acc = 0.0;
  const bool mlp = (P.model == 2);
  // rows of every [M x ldp] buffer start on 128-byte boundaries and c0 is a multiple of 4: 128-bit accesses
  for (long long o = c0 + 4 * (long long)tid; o < c1; o += 4 * TRIG_THREADS) {
    float4 g4 = make_float4(0.f, 0.f, 0.f, 0.f), d4 = g4;
    for (int ch = 0; ch < P.n_chunks; ++ch) {
      const float4 a = *reinterpret_cast<const float4*>(part + ((long long)ch * 2) * P.ldp + o);
      const float4 b = *reinterpret_cast<const float4*>(part + ((long long)ch * 2 + 1) * P.ldp + o);
      g4.x += a.x; g4.y += a.y; g4.z += a.z; g4.w += a.w;
      d4.x += b.x; d4.y += b.y; d4.z += b.z; d4.w += b.w;
    }
    const float4 t4 = *reinterpret_cast<const float4*>(P.theta + o);
    const float4 o4 = *reinterpret_cast<const float4*>(tho + o);
    float4 s4 = make_float4(0.f, 0.f, 0.f, 0.f);
    if (cada1 || lag) s4 = *reinterpret_cast<const float4*>(ds + o);
    float g[4] = {g4.x, g4.y, g4.z, g4.w}, d[4] = {d4.x, d4.y, d4.z, d4.w};
    const float t[4] = {t4.x, t4.y, t4.z, t4.w}, to[4] = {o4.x, o4.y, o4.z, o4.w}, st[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (o + e < P.p) {
        if (mlp) d[e] = g[e] - d[e];        // MLP: the second slot holds the gradient at the old iterate itself
        g[e] = fmaf(P.lambda, t[e], g[e]);
        d[e] = fmaf(P.lambda, t[e] - to[e], d[e]);
        const float e_ = cada1 ? d[e] - st[e] : lag ? g[e] - st[e] : d[e];
        acc = fma((double)e_, (double)e_, acc);
      } else {
        g[e] = 0.f; d[e] = 0.f;
      }
    }
    *reinterpret_cast<float4*>(gf + o) = make_float4(g[0], g[1], g[2], g[3]);
    *reinterpret_cast<float4*>(df + o) = make_float4(d[0], d[1], d[2], d[3]);
  }
  const double total = block_sum(acc, s_red);
  if (tid == 0) {
    P.norm_part[(long long)m * P.trig_splits + s] = total;
    __threadfence();
    s_ticket = atomicAdd(&P.worker_ticket[m], 1u);
  }
  __syncthreads();
  if (s_ticket != (unsigned)(P.trig_splits - 1) || tid >= 32) return;

  // last CTA of worker m: the decision (Algorithm 1, "if Eq. 6 / Eq. 8 is violated or tau >= D")
  __threadfence();
  double lhs = 0.0;                      // fixed order: lane-strided partial sums, then the shuffle tree
  for (int i = tid; i < P.trig_splits; i += 32) lhs += __ldcg(&P.norm_part[(long long)m * P.trig_splits + i]);
  lhs = warp_sum(lhs);
  if (tid != 0) return;
  decide_upload(P, k, m, lhs, rhs);
  P.worker_ticket[m] = 0;
}

// block = (tx, ty) with tx * ty = UPD_THREADS: tx column groups of 4 floats, ty worker lanes.
// BATCH (chosen when a lane walks more than one worker, M > ty): the loads of four workers are issued before the first
// store -- a store to one worker's record would otherwise hold back the next worker's load -- and the records are then
// refreshed and summed in the same worker order, so both forms produce the same bits.
// MODE 0: the whole server side.  MODE 1 (workers split over several handles): refresh of the uploaders' records and the
// sum over this handle's workers, written unscaled to sum_io; nothing else changes.  MODE 2: the rest of the server side
// from the total in sum_io (the caller has added the vectors of all handles); launched with one worker lane.
enum { UPD_FULL = 0, UPD_LOCAL = 1, UPD_APPLY = 2 };
template <bool BATCH, int MODE = UPD_FULL>
__global__ void __launch_bounds__(UPD_THREADS, BATCH ? 4 : 6) update_kernel(const __grid_constant__ Params P, float* sum_io, long long k /* iteration, as the host counts it */,
              int finish /* 1: the last update kernel of a call completes the window term itself */) {
  __shared__ float4 s_part[UPD_THREADS];
  __shared__ double s_red[32];
  __shared__ unsigned char s_mask[1024];
  __shared__ unsigned int s_ticket;
  const int TX = blockDim.x, TY = blockDim.y, tx = threadIdx.x, ty = threadIdx.y;
  const int tid = ty * TX + tx;
  pdl_trigger();                           // the next iteration's gradient kernel may start its data-independent part
  pdl_wait();                              // ... and this kernel reads what the kernels before it wrote
  const long long q = ((long long)blockIdx.x * TX + tx) * 4;   // first of this thread's 4 coordinates
  const bool live = q < P.p;
  const bool cada1 = (P.rule == 1), recursive = (P.aggregate == 1);
  const float alpha = step_size(P, k);

  float4 sum = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 th = make_float4(0.f, 0.f, 0.f, 0.f);
  float4 h4 = th, v4 = th;                 // loaded up front: they do not depend on the workers' sum
  if (live) th = *reinterpret_cast<const float4*>(P.theta + q);
  if (live && ty == 0 && MODE != UPD_LOCAL) {
    h4 = *reinterpret_cast<const float4*>(P.h + q);
    v4 = *reinterpret_cast<const float4*>(P.vhat + q);
  }
  for (int mb = 0; mb < (MODE == UPD_APPLY ? 0 : P.M); mb += 1024) {
    __syncthreads();
    for (int i = tid; i < min(1024, P.M - mb); i += TX * TY) s_mask[i] = P.mask[mb + i];
    __syncthreads();
    if (live) {
      const int mend = min(P.M, mb + 1024);
      if (!BATCH) {
        for (int m = mb + ty; m < mend; m += TY) {
          const long long off = (long long)m * P.ldp + q;
          float4 v;
          if (s_mask[m - mb] & 1) {          // uploaded: slot <- fresh gradient (masked 128-bit copy)
            v = *reinterpret_cast<const float4*>(P.g_fresh + off);
            if (recursive) {                 // Eq. 3: the innovation against the worker's last upload enters the sum
              const float4 old = *reinterpret_cast<const float4*>(P.G + off);
              *reinterpret_cast<float4*>(P.G + off) = v;
              v = make_float4(v.x - old.x, v.y - old.y, v.z - old.z, v.w - old.w);
            } else {
              *reinterpret_cast<float4*>(P.G + off) = v;
            }
            if (cada1) {
              *reinterpret_cast<float4*>(P.delta_stored + off) = *reinterpret_cast<const float4*>(P.d_fresh + off);
            } else if (P.rule == 2) {
              *reinterpret_cast<float4*>(P.theta_hat + off) = th;
            }
          } else if (recursive) {
            continue;                        // Eq. 3 never touches a skipping worker's record
          } else {
            v = *reinterpret_cast<const float4*>(P.G + off);
          }
          sum.x += v.x; sum.y += v.y; sum.z += v.z; sum.w += v.w;
        }
      } else {
        for (int m0 = mb + ty; m0 < mend; m0 += 4 * TY) {
          float4 v[4], aux[4];
          bool up[4];
  #pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int m = m0 + j * TY;
            v[j] = make_float4(0.f, 0.f, 0.f, 0.f); aux[j] = v[j]; up[j] = false;
            if (m < mend) {
              const long long off = (long long)m * P.ldp + q;
              up[j] = s_mask[m - mb] & 1;
              if (up[j]) {
                v[j] = *reinterpret_cast<const float4*>(P.g_fresh + off);
                if (recursive) aux[j] = *reinterpret_cast<const float4*>(P.G + off);
                else if (cada1) aux[j] = *reinterpret_cast<const float4*>(P.d_fresh + off);
              } else if (!recursive) {
                v[j] = *reinterpret_cast<const float4*>(P.G + off);
              }
            }
          }
  #pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int m = m0 + j * TY;
            if (m >= mend) continue;
            const long long off = (long long)m * P.ldp + q;
            if (up[j]) {                       // uploaded: slot <- fresh gradient (masked 128-bit copy)
              *reinterpret_cast<float4*>(P.G + off) = v[j];
              if (recursive) {                 // Eq. 3: the innovation against the worker's last upload enters the sum
                v[j] = make_float4(v[j].x - aux[j].x, v[j].y - aux[j].y, v[j].z - aux[j].z, v[j].w - aux[j].w);
                if (cada1) *reinterpret_cast<float4*>(P.delta_stored + off) = *reinterpret_cast<const float4*>(P.d_fresh + off);
              } else if (cada1) {
                *reinterpret_cast<float4*>(P.delta_stored + off) = aux[j];
              }
              if (P.rule == 2) *reinterpret_cast<float4*>(P.theta_hat + off) = th;
            } else if (recursive) {
              continue;                        // Eq. 3 never touches a skipping worker's record
            }
            sum.x += v[j].x; sum.y += v[j].y; sum.z += v[j].z; sum.w += v[j].w;
          }
        }
      }
    }
  }
  s_part[tid] = sum;
  __syncthreads();

  double dsq = 0.0;
  if (ty == 0 && live) {
    float4 a = s_part[tx];
    for (int y = 1; y < TY; ++y) {
      const float4 b = s_part[y * TX + tx];
      a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
    }
    if (MODE == UPD_LOCAL) {                                   // this handle's part of the sum of Eq. 2a / Eq. 3
      if (q + 0 >= P.p) a.x = 0.f;
      if (q + 1 >= P.p) a.y = 0.f;
      if (q + 2 >= P.p) a.z = 0.f;
      if (q + 3 >= P.p) a.w = 0.f;
      if (q + 3 < P.p) {
        *reinterpret_cast<float4*>(sum_io + q) = a;            // caller's vector of p floats: 16-byte aligned, no padding
      } else {
        const float av[4] = {a.x, a.y, a.z, a.w};
        for (int e = 0; e < 4; ++e) if (q + e < P.p) sum_io[q + e] = av[e];
      }
    }
    if (MODE == UPD_APPLY) {
      if (q + 3 < P.p) {
        a = *reinterpret_cast<const float4*>(sum_io + q);
      } else {
        float av[4] = {0.f, 0.f, 0.f, 0.f};
        for (int e = 0; e < 4; ++e) if (q + e < P.p) av[e] = sum_io[q + e];
        a = make_float4(av[0], av[1], av[2], av[3]);
      }
    }
    const float invM = 1.0f / (float)P.Mg;
    if (MODE != UPD_LOCAL) {
    float nab[4] = {a.x * invM, a.y * invM, a.z * invM, a.w * invM};       // Eq. 2a aggregate
    if (recursive) {                                                        // Eq. 3: nabla^k = nabla^{k-1} + (1/M) sum delta_m^k
      const float4 prev = *reinterpret_cast<const float4*>(P.nabla + q);
      nab[0] += prev.x; nab[1] += prev.y; nab[2] += prev.z; nab[3] += prev.w;
#pragma unroll
      for (int e = 0; e < 4; ++e) if (q + e >= P.p) nab[e] = 0.f;
      *reinterpret_cast<float4*>(P.nabla + q) = make_float4(nab[0], nab[1], nab[2], nab[3]);
    }
    float hh[4] = {h4.x, h4.y, h4.z, h4.w}, vv[4] = {v4.x, v4.y, v4.z, v4.w};
    float tt[4] = {th.x, th.y, th.z, th.w};
    float tn[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      if (q + e < P.p && P.server == 1) {                                     // SGD server (Section 2.1)
        tn[e] = tt[e] - alpha * nab[e];
        const double dlt = (double)tn[e] - (double)tt[e];
        dsq = fma(dlt, dlt, dsq);
      } else if (q + e < P.p) {
        hh[e] = P.beta1 * hh[e] + (1.0f - P.beta1) * nab[e];                 // Eq. 2a
        const float v = P.beta2 * vv[e] + (1.0f - P.beta2) * nab[e] * nab[e]; // Eq. 2b
        vv[e] = fmaxf(v, vv[e]);
        tn[e] = tt[e] - alpha * hh[e] / sqrtf(P.eps + vv[e]);              // Eq. 2c
        const double dlt = (double)tn[e] - (double)tt[e];
        dsq = fma(dlt, dlt, dsq);
      } else {
        tn[e] = tt[e];
      }
    }
    if (cada1 && (k % P.D == 0)) *reinterpret_cast<float4*>(P.theta_tilde + q) = th;   // snapshot = theta^k
    *reinterpret_cast<float4*>(P.h + q) = make_float4(hh[0], hh[1], hh[2], hh[3]);
    *reinterpret_cast<float4*>(P.vhat + q) = make_float4(vv[0], vv[1], vv[2], vv[3]);
    *reinterpret_cast<float4*>(P.theta + q) = make_float4(tn[0], tn[1], tn[2], tn[3]);
    // network path: the bf16 operand image of theta^{k+1}'s first-layer weights goes into its ring slot here, so that no
    // iterate is ever rounded twice (an uploading worker's old iterate IS this image from the next iteration on)
    if (P.w1_ring && q < (long long)P.F * P.H)
      mlp_ring_store4(P, (int)((k + 1) % P.w1_slots), q, make_float4(tn[0], tn[1], tn[2], tn[3]));
    }
  }
  if (MODE == UPD_LOCAL) return;                               // the window and k move in the second half
  const double total = block_sum(dsq, s_red);
  if (!finish) {                                               // the next iteration's deciders add the partials (window_refresh)
    if (tid == 0) {
      P.step_part[blockIdx.x] = total;
      if (blockIdx.x == 0) { P.st->step_part_for = k + 1; P.st->step_part_n = (int)gridDim.x; P.st->k = k + 1; }
    }
    return;
  }
  if (tid == 0) {
    P.step_part[blockIdx.x] = total;
    __threadfence();
    s_ticket = atomicAdd(&P.st->update_ticket, 1u);
  }
  __syncthreads();
  if (s_ticket != gridDim.x - 1) return;
  // last block: its first warp adds the block partials in the order window_refresh uses (lane-strided, then the shuffle
  // tree), so that a run gives the same bits however its iterations are divided into calls
  if (tid >= 32) return;
  __threadfence();
  double part = 0.0;
  for (unsigned b = tid; b < gridDim.x; b += 32u) part += __ldcg(&P.step_part[b]);
  const double s = warp_sum(part);
  if (tid == 0) {
    P.ring[k % P.d_max] = s;                    // newest window term ||theta^{k+1} - theta^k||^2
    P.st->last_step_sqnorm = s;
    P.st->update_ticket = 0;
    P.st->step_part_for = 0;
    P.st->k = k + 1;
  }
}

// Hands an iteration's results to the host without a copy-engine operation in the compute stream: theta^{k+1} and the
// upload mask are stored straight into page-locked host memory that the device can address (posted writes over the
// bus).  Launched with programmatic serialisation behind the iteration's last kernel.
__global__ void __launch_bounds__(256) export_kernel(const float* __restrict__ theta, long long p, const unsigned char* __restrict__ mask,
                                                     int M, float* host_theta, unsigned char* host_mask) {
  pdl_trigger();
  pdl_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (host_theta)
    for (long long o = i; o < p; o += (long long)gridDim.x * blockDim.x) host_theta[o] = theta[o];
  if (host_mask)
    for (long long o = i; o < M; o += (long long)gridDim.x * blockDim.x) host_mask[o] = mask[o];
}

// State initialisation of Algorithm 1 (theta_hat_m = theta~ = theta^0; everything else is
// zeroed by a memset of the workspace before this runs).
__global__ void init_kernel(const __grid_constant__ Params P, const float* __restrict__ theta0) {
  const long long n = P.p;
  for (long long o = blockIdx.x * (long long)blockDim.x + threadIdx.x; o < n; o += (long long)gridDim.x * blockDim.x) {
    const float t = theta0[o];
    P.theta[o] = t;
    if (P.theta_tilde) P.theta_tilde[o] = t;
    if (P.theta_hat)
      for (int m = 0; m < P.M; ++m) P.theta_hat[(long long)m * P.ldp + o] = t;
  }
}

}  // namespace cada
