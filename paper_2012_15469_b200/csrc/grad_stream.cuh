// Two-point minibatch gradient for the binary logistic model with long rows: the HBM-bound
// kernel.  Every sampled row of X crosses the memory system once and serves both iterates
// (Algorithm 1: both gradients are taken on the same minibatch).
//
// One persistent CTA per SM.  The M*ceil(B/R) "units" (R = 4 consecutive minibatch rows of one
// worker) are split evenly over the CTAs, so each CTA walks a contiguous run of units and, when
// the run crosses into the next worker, writes the finished worker's partial sums to its slot.
//
//   producer warp   per unit: arms the stage's mbarrier, issues one bulk copy (cp.async.bulk,
//                   global -> shared, completion counted on the mbarrier) per sampled row, and
//                   drops the rows' labels beside them; row indices and labels are prepared 8
//                   units at a time, one group ahead, by all 32 lanes
//   8 consumer warps  each thread owns 4*NCH float4 columns of the row: it keeps theta,
//                   theta - theta', and both gradient accumulators for them in registers, pulls
//                   the unit's rows into registers (the stage is released right away), forms
//                   partial logits z = x.theta and dz = x.(theta - theta'), reduces the 8 values
//                   over the CTA (shuffles + one named barrier), turns them into residuals
//                   r = (sigma(z) - t)/B, dr = (sigma(z) - sigma(z - dz))/B, and adds r*x, dr*x
// When a CTA's run leaves a worker it owns that worker's partial sums of g_m and of d_m = g_m - g'_m.  A worker whose
// units all lie in one CTA is finished from registers; otherwise each CTA stores its partial sums to the worker's slot
// and takes a ticket, and the CTA that arrives last adds the slots in slot order.  "Finishing" is the worker side of
// Algorithm 1 after the gradients: regulariser, g_m and d_m kept for the server, the left-hand side of Eq. 6 / Eq. 8
// (fp64) and the upload decision -- no trigger launch and no second pass over the gradients.
// All waits are bounded; on expiry the kernel raises CADA_FLAG_TIMEOUT, waits (bounded) for
// its copies in flight and returns.
#pragma once
#include "common.cuh"

namespace cada {

constexpr int GS_CONSUMERS = 256;                 // consumer threads (8 warps)
constexpr int GS_THREADS = GS_CONSUMERS + 32;     // + one producer warp
constexpr int GS_R = 4;                           // rows per unit / pipeline stage
constexpr int GS_MAX_STAGES = 8;
constexpr unsigned GS_SPIN_LIMIT = 1u << 24;

struct StreamGeom {
  int n_stages;
  unsigned row_bytes;      // F * 4
  unsigned stage_stride;   // bytes between stages (R rows, 128-byte aligned)
  int units_per_worker;    // ceil(B / R)
  long long n_units;       // all workers' units: M * units_per_worker, or the sum of ceil(B_m / R) with per-worker batch sizes
  const long long* ustart; // DEVICE [M + 1], per-worker batch sizes only: first unit of worker m (so that the even split of
                           // the units over the CTAs is an even split of the rows); nullptr: worker m starts at m * units_per_worker
};

__host__ __device__ inline size_t grad_stream_smem(const StreamGeom& g) {
  return (size_t)g.n_stages * g.stage_stride + 1024;   // + barriers, labels, reduction scratch
}

// CTA (of G) whose run [floor(c*U/G), floor((c+1)*U/G)) contains unit u.
__host__ __device__ inline int stream_cta_of_unit(long long u, long long U, int G) {
  long long c = ((u + 1) * G + U - 1) / U - 1;
  while (c > 0 && (c * U) / G > u) --c;
  while (c + 1 < G && ((c + 1) * U) / G <= u) ++c;
  return (int)c;
}

namespace ptx {
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity) {
  for (unsigned spin = 0; spin < GS_SPIN_LIMIT; ++spin)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void consumer_bar_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(GS_CONSUMERS) : "memory");
}
}  // namespace ptx

// Sums 8 per-thread values over the warp with 9 shuffles; lane l returns the total of value l>>2.
__device__ __forceinline__ float warp_reduce8(const float (&v)[8], int lane) {
  const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
  float w4[4], w2[2];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float send = b4 ? v[i] : v[i + 4], keep = b4 ? v[i + 4] : v[i];
    w4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const float send = b3 ? w4[i] : w4[i + 2], keep = b3 ? w4[i + 2] : w4[i];
    w2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
  }
  const float send = b2 ? w2[0] : w2[1], keep = b2 ? w2[1] : w2[0];
  float w = keep + __shfl_xor_sync(0xffffffffu, send, 4);
  w += __shfl_xor_sync(0xffffffffu, w, 2);
  w += __shfl_xor_sync(0xffffffffu, w, 1);
  return w;
}

template <int NCH>
__global__ void __launch_bounds__(GS_THREADS, 1)
grad_stream_kernel(const __grid_constant__ Params P, const __grid_constant__ StreamGeom geo,
                   long long k /* iteration, as the host counts it */) {
  // Launched with programmatic serialisation: this kernel may be scheduled while the update kernel of the previous
  // iteration still runs.  The sampled rows depend on k and on the caller's data only, so the producer warp starts
  // filling the ring at once; the consumers wait for the preceding kernels before they read the iterates.
  pdl_trigger();
  extern __shared__ __align__(128) unsigned char smem[];
  const int S = geo.n_stages;
  unsigned char* tail = smem + (size_t)S * geo.stage_stride;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(tail);            // full[S], empty[S]
  float* s_y = reinterpret_cast<float*>(tail + 2 * GS_MAX_STAGES * 8);                // [S][R]
  float* s_part = s_y + GS_MAX_STAGES * GS_R;                                         // [2][8 warps][8]
  double* s_red = reinterpret_cast<double*>(s_part + 128);                            // [8 warps] left-hand-side partials
  unsigned* s_ticket = reinterpret_cast<unsigned*>(s_red + GS_CONSUMERS / 32);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = gridDim.x, cta = blockIdx.x;
  const long long U = geo.n_units;
  const int UB = geo.units_per_worker;
  const long long* __restrict__ ustart = geo.ustart;
  auto first_unit = [&](int m) { return ustart ? ustart[m] : (long long)m * UB; };
  auto worker_of_unit = [&](long long u) {                 // worker whose run of units contains u (u < U)
    if (!ustart) return (int)(u / UB);
    int lo = 0, hi = P.M - 1;
    while (lo < hi) { const int mid = (lo + hi + 1) >> 1; if (ustart[mid] <= u) lo = mid; else hi = mid - 1; }
    return lo;
  };
  const long long u0 = ((long long)cta * U) / G, u1 = ((long long)(cta + 1) * U) / G;
  const int F = P.F;
  const uint32_t full0 = ptx::smem_u32(bars), empty0 = ptx::smem_u32(bars + GS_MAX_STAGES);

  if (tid == 0) {
    for (int s = 0; s < S; ++s) {
      ptx::mbar_init(full0 + 8 * s, 1);
      ptx::mbar_init(empty0 + 8 * s, GS_CONSUMERS / 32);
    }
    ptx::fence_barrier_init();
  }
  __syncthreads();

  if (warp == GS_CONSUMERS / 32) {
    // ------------------------------------------------------------------ producer warp
    // explicit row indices may have been produced on this stream just before the call: they are read only after
    // the kernels before this one have completed (X and y never change while the handle lives)
    if (P.idx_mode == IDX_EXPLICIT) pdl_wait();
    // Lane L looks after row L%4 of unit 8g + L/4 of the current group g of 8 units: it hashes the
    // row index and fetches the label one group ahead, so that neither latency sits between a
    // stage becoming free and its copies being issued.
    struct RowJob { const float* src; float y; int nrows; };
    auto prepare = [&](long long group) {
      RowJob j{nullptr, 0.f, 0};
      const long long u = u0 + group * 8 + (lane >> 2);
      if (u < u1) {
        const int m = worker_of_unit(u), b = (int)(u - first_unit(m)), r = lane & 3;
        j.nrows = max(0, min(GS_R, worker_batch(P, m) - b * GS_R));
        if (r < j.nrows) {
          const long long row = minibatch_row(P, k, m, b * GS_R + r, P.n_samples[m]);
          j.src = static_cast<const float*>(P.X[m]) + row * P.ldx;
          j.y = static_cast<const float*>(P.y[m])[row];
        }
      }
      return j;
    };
    const long long n_units = u1 - u0, n_groups = (n_units + 7) / 8;
    long long it = 0;
    int s = 0;
    uint32_t ephase = 1;      // parity of the "stage is free" phase; the first pass over the ring does not wait
    bool ok = true;
    RowJob nxt = prepare(0);
    for (long long g = 0; g < n_groups && ok; ++g) {
      const RowJob cur = nxt;
      if (g + 1 < n_groups) nxt = prepare(g + 1);
      const int in_group = (int)min(8ll, n_units - g * 8);
      for (int j = 0; j < in_group; ++j, ++it) {
        if (it >= S) {
          ok = ptx::mbar_wait_bounded(empty0 + 8 * s, ephase);
          ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
          if (!ok) break;
        }
        const int nrows = __shfl_sync(0xffffffffu, cur.nrows, 4 * j);
        if (lane == 0) ptx::mbar_expect_tx(full0 + 8 * s, (uint32_t)nrows * geo.row_bytes);
        __syncwarp();
        if ((lane >> 2) == j && cur.src != nullptr) {
          const int r = lane & 3;
          ptx::bulk_g2s(ptx::smem_u32(smem + (size_t)s * geo.stage_stride + (size_t)r * geo.row_bytes), cur.src,
                        geo.row_bytes, full0 + 8 * s);
          s_y[s * GS_R + r] = cur.y;
        }
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(full0 + 8 * s);
        if (++s == S) { s = 0; ephase ^= 1u; }
      }
    }
    if (!ok && lane == 0) atomicOr(&P.st->status_flags, 4);
    // copies still in flight belong to the last min(it, S) stages: wait for them (bounded)
    if (lane == 0) {
      const long long first = it > S ? it - S : 0;
      for (long long j = first; j < it; ++j)
        if (!ptx::mbar_wait_bounded(full0 + 8 * (int)(j % S), (uint32_t)((j / S) & 1))) atomicOr(&P.st->status_flags, 4);
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  pdl_wait();                                  // theta, the old iterates and the partial slots belong to earlier kernels until now
  double rhs = 0.0;                            // right-hand side of this iteration (thread 0 decides)
  if (tid < 32) rhs = window_refresh_rhs(P, k, tid);     // after the newest window term, if the update kernel left it in parts (any CTA may decide)
  const int nq = F >> 2;                       // float4 columns in a row
  float4 th[NCH], dth[NCH], ag[NCH], ad[NCH];
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
  for (int c = 0; c < NCH; ++c) {
    const int q = tid + c * GS_CONSUMERS;
    th[c] = q < nq ? reinterpret_cast<const float4*>(P.theta)[q] : zero4;
    dth[c] = zero4; ag[c] = zero4; ad[c] = zero4;
  }
  const float bias = P.has_bias ? P.theta[F] : 0.f;
  float dbias = 0.f, agb = 0.f, adb = 0.f;
  float invB = 0.f;
  int Bm = 0, cur_m = -1;
  // running unit coordinates (no divisions in the loop): worker, unit within worker, stage, phase
  int m = u0 < U ? worker_of_unit(u0) : 0, b = (int)(u0 - first_unit(m)), s = 0;
  int ub_m = ustart ? (int)(ustart[m + 1] - ustart[m]) : UB;       // units of the current worker
  uint32_t phase = 0;

  const bool cada1 = (P.rule == 1), lag = (P.rule == 3);
  // Leaves worker m: its partial sums go to the worker's slot unless this CTA holds all of its units; the CTA that
  // completes the worker (the only one, or the last to take a ticket) finishes it.  Called by all consumers at once.
  auto flush = [&](int m) {
    const long long um0 = first_unit(m), um1 = ustart ? ustart[m + 1] : um0 + UB;
    const int lo = stream_cta_of_unit(um0, U, G);
    const int hi = stream_cta_of_unit(um1 - 1, U, G);
    const int n_slots = hi - lo + 1;                 // slots the sum walks (slots of CTAs without units stay zero)
    const int n_owners = U >= G ? n_slots : (int)(um1 - um0);   // CTAs that hold units of m: with fewer units than CTAs, one each
    float* slot0 = P.part + ((long long)m * P.n_chunks * 2) * P.ldp;
    bool last = true;
    if (n_slots > 1) {
      float* og = slot0 + ((long long)(cta - lo) * 2) * P.ldp;
      float* od = og + P.ldp;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int q = tid + c * GS_CONSUMERS;
        if (q < nq) {
          reinterpret_cast<float4*>(og)[q] = ag[c];
          reinterpret_cast<float4*>(od)[q] = ad[c];
        }
      }
      if (P.has_bias && tid == 0) { og[F] = agb; od[F] = adb; }
      ptx::consumer_bar_sync();                      // every consumer's part of the slot is written
      if (tid == 0) {
        __threadfence();
        *s_ticket = atomicAdd(&P.worker_ticket[m], 1u);
      }
      ptx::consumer_bar_sync();
      last = *s_ticket == (unsigned)(n_owners - 1);
      if (last) __threadfence();
    }
    if (last) {
      float* gf = P.g_fresh + (long long)m * P.ldp;
      float* df = P.d_fresh + (long long)m * P.ldp;
      const float* ref = cada1 ? P.delta_stored + (long long)m * P.ldp : lag ? P.G + (long long)m * P.ldp : nullptr;
      double acc = 0.0;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int q = tid + c * GS_CONSUMERS;
        if (q < nq) {
          float4 g4 = ag[c], d4 = ad[c];
          if (n_slots > 1) {                          // slot order, whichever CTA does the sum
            g4 = zero4; d4 = zero4;
            for (int sl = 0; sl < n_slots; ++sl) {
              const float4 a = __ldcg(reinterpret_cast<const float4*>(slot0 + ((long long)sl * 2) * P.ldp) + q);
              const float4 b = __ldcg(reinterpret_cast<const float4*>(slot0 + ((long long)sl * 2 + 1) * P.ldp) + q);
              g4.x += a.x; g4.y += a.y; g4.z += a.z; g4.w += a.w;
              d4.x += b.x; d4.y += b.y; d4.z += b.z; d4.w += b.w;
            }
          }
          g4.x = fmaf(P.lambda, th[c].x, g4.x); g4.y = fmaf(P.lambda, th[c].y, g4.y);
          g4.z = fmaf(P.lambda, th[c].z, g4.z); g4.w = fmaf(P.lambda, th[c].w, g4.w);
          d4.x = fmaf(P.lambda, dth[c].x, d4.x); d4.y = fmaf(P.lambda, dth[c].y, d4.y);
          d4.z = fmaf(P.lambda, dth[c].z, d4.z); d4.w = fmaf(P.lambda, dth[c].w, d4.w);
          reinterpret_cast<float4*>(gf)[q] = g4;
          reinterpret_cast<float4*>(df)[q] = d4;
          float4 e4 = d4;                             // Eq. 8: d_m itself
          if (ref) {
            const float4 r4 = reinterpret_cast<const float4*>(ref)[q];
            if (cada1) e4 = make_float4(d4.x - r4.x, d4.y - r4.y, d4.z - r4.z, d4.w - r4.w);       // Eq. 6
            else e4 = make_float4(g4.x - r4.x, g4.y - r4.y, g4.z - r4.z, g4.w - r4.w);             // Eq. 4
          }
          acc = fma((double)e4.x, (double)e4.x, acc); acc = fma((double)e4.y, (double)e4.y, acc);
          acc = fma((double)e4.z, (double)e4.z, acc); acc = fma((double)e4.w, (double)e4.w, acc);
        }
      }
      if (P.has_bias && tid == 0) {                   // the constant-1 column
        float gb = agb, db = adb;
        if (n_slots > 1) {
          gb = 0.f; db = 0.f;
          for (int sl = 0; sl < n_slots; ++sl) {
            gb += __ldcg(slot0 + ((long long)sl * 2) * P.ldp + F);
            db += __ldcg(slot0 + ((long long)sl * 2 + 1) * P.ldp + F);
          }
        }
        gb = fmaf(P.lambda, bias, gb);
        db = fmaf(P.lambda, dbias, db);
        gf[F] = gb; df[F] = db;
        const float e = cada1 ? db - ref[F] : lag ? gb - ref[F] : db;
        acc = fma((double)e, (double)e, acc);
      }
      acc = warp_sum(acc);                            // fixed order: shuffle tree, then the warps in order
      if (lane == 0) s_red[warp] = acc;
      ptx::consumer_bar_sync();
      if (tid == 0) {
        double lhs = 0.0;
#pragma unroll
        for (int w8 = 0; w8 < GS_CONSUMERS / 32; ++w8) lhs += s_red[w8];
        decide_upload(P, k, m, lhs, rhs);
        if (n_slots > 1) P.worker_ticket[m] = 0;
      }
    }
#pragma unroll
    for (int c = 0; c < NCH; ++c) { ag[c] = zero4; ad[c] = zero4; }
    agb = 0.f; adb = 0.f;
  };

  const int n_mine = (int)(u1 - u0);
  for (int it = 0; it < n_mine; ++it) {
    if (m != cur_m) {
      if (cur_m >= 0) flush(cur_m);
      cur_m = m;
      Bm = worker_batch(P, m);
      invB = 1.0f / (float)Bm;
      const float* tho = old_iterate(P, k, m);
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int q = tid + c * GS_CONSUMERS;
        if (q < nq) {
          const float4 o = reinterpret_cast<const float4*>(tho)[q];
          dth[c] = make_float4(th[c].x - o.x, th[c].y - o.y, th[c].z - o.z, th[c].w - o.w);
        }
      }
      dbias = P.has_bias ? bias - tho[F] : 0.f;
    }
    const int nrows = max(0, min(GS_R, Bm - b * GS_R));     // 0: a unit past this worker's rows (no bytes were copied)
    if (!ptx::mbar_wait_bounded(full0 + 8 * s, phase)) {
      if (tid == 0) atomicOr(&P.st->status_flags, 4);
      return;        // every consumer waits on the same barrier, so all of them leave here
    }
    // pull the unit into registers and hand the stage back to the producer
    float4 x[GS_R][NCH];
    float yv[GS_R];
    const unsigned char* base = smem + (size_t)s * geo.stage_stride;
#pragma unroll
    for (int r = 0; r < GS_R; ++r) {
      yv[r] = r < nrows ? s_y[s * GS_R + r] : 0.f;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        const int q = tid + c * GS_CONSUMERS;
        x[r][c] = (r < nrows && q < nq) ? reinterpret_cast<const float4*>(base + (size_t)r * geo.row_bytes)[q] : zero4;
      }
    }
    __syncwarp();
    if (lane == 0) ptx::mbar_arrive(empty0 + 8 * s);

    // forward: partial logits for both iterates
    float v[2 * GS_R];
#pragma unroll
    for (int r = 0; r < GS_R; ++r) {
      float z = 0.f, dz = 0.f;
#pragma unroll
      for (int c = 0; c < NCH; ++c) {
        z = fmaf(x[r][c].x, th[c].x, z); z = fmaf(x[r][c].y, th[c].y, z);
        z = fmaf(x[r][c].z, th[c].z, z); z = fmaf(x[r][c].w, th[c].w, z);
        dz = fmaf(x[r][c].x, dth[c].x, dz); dz = fmaf(x[r][c].y, dth[c].y, dz);
        dz = fmaf(x[r][c].z, dth[c].z, dz); dz = fmaf(x[r][c].w, dth[c].w, dz);
      }
      v[2 * r] = z; v[2 * r + 1] = dz;
    }
    const float wsum = warp_reduce8(v, lane);          // lane l: value l>>2 summed over the warp
    float* sp = s_part + (it & 1) * 64;
    if ((lane & 3) == 0) sp[warp * 8 + (lane >> 2)] = wsum;
    ptx::consumer_bar_sync();
    float tot = sp[((lane & 3) * 2) * 8 + (lane >> 2)] + sp[((lane & 3) * 2 + 1) * 8 + (lane >> 2)];
    tot += __shfl_xor_sync(0xffffffffu, tot, 1);
    tot += __shfl_xor_sync(0xffffffffu, tot, 2);
    const float other = __shfl_xor_sync(0xffffffffu, tot, 4);
    const bool is_dz = (lane >> 2) & 1;
    const float z = (is_dz ? other : tot) + bias, dz = (is_dz ? tot : other) + dbias;
    const int myrow = lane >> 3;
    const float ylab = myrow == 0 ? yv[0] : myrow == 1 ? yv[1] : myrow == 2 ? yv[2] : yv[3];
    const bool valid = myrow < nrows;
    float sig, dsig;
    sigmoid_pair_fast(z, dz, sig, dsig);
    const float rv = valid ? (sig - 0.5f * (ylab + 1.0f)) * invB : 0.f;
    const float drv = valid ? dsig * invB : 0.f;
    float res[GS_R], dres[GS_R];
#pragma unroll
    for (int r = 0; r < GS_R; ++r) {
      res[r] = __shfl_sync(0xffffffffu, rv, 8 * r);
      dres[r] = __shfl_sync(0xffffffffu, drv, 8 * r);
      agb += res[r]; adb += dres[r];
    }
    // backward: rank-R update of both accumulators
#pragma unroll
    for (int c = 0; c < NCH; ++c) {
#pragma unroll
      for (int r = 0; r < GS_R; ++r) {
        ag[c].x = fmaf(res[r], x[r][c].x, ag[c].x); ag[c].y = fmaf(res[r], x[r][c].y, ag[c].y);
        ag[c].z = fmaf(res[r], x[r][c].z, ag[c].z); ag[c].w = fmaf(res[r], x[r][c].w, ag[c].w);
        ad[c].x = fmaf(dres[r], x[r][c].x, ad[c].x); ad[c].y = fmaf(dres[r], x[r][c].y, ad[c].y);
        ad[c].z = fmaf(dres[r], x[r][c].z, ad[c].z); ad[c].w = fmaf(dres[r], x[r][c].w, ad[c].w);
      }
    }
    if (++b == ub_m) {
      b = 0; ++m;
      if (ustart && m < P.M) ub_m = (int)(ustart[m + 1] - ustart[m]);
    }
    if (++s == S) { s = 0; phase ^= 1u; }
  }
  if (cur_m >= 0) flush(cur_m);
}

}  // namespace cada
