// Two-point minibatch gradient for softmax regression with up to 16 classes.
//
// One CTA (16 warps) per (worker, block of 8 minibatch rows); two warps share a row, each taking every other
// group of 32 features.
//   stage    the 8 rows are copied to shared memory once (read once from global memory); W and W - W' too when they fit
//   forward  lane l walks its features: for every NON-ZERO x it adds x * W[j][:] and x * (W - W')[j][:] to its CP logit
//            accumulators (sparse inputs skip most features); the 2C values are summed over the warp and the two
//            warps of a row are combined through shared memory
//   softmax  the first warp of each row forms P, P - onehot and the accurate difference
//            P_c - P'_c = P_c (T - e_c) / (1 + T), e_c = expm1(-dz_c), T = sum_j P_j e_j
//   backward thread (half, feature) accumulates r[i][:] * x (half 0) or dr[i][:] * x (half 1) over the 8 rows, again
//            skipping zeros; the results leave through a staging tile as contiguous runs
// Output: partial slot (worker, row block) of g_m and d_m = g_m - g'_m, without the regulariser.
// CP is the class count rounded up to one of {4, 8, 10, 12, 16}: it sizes the register arrays and unrolled loops.
#pragma once
#include "common.cuh"

namespace cada {

constexpr int GSM_THREADS = 512;
constexpr int GSM_ROWS = 8;          // rows per CTA
constexpr int GSM_CMAX = 16;
constexpr int GSM_STAGE_FEATS = 256; // features per coalesced store round (2 halves x 256 = 512 threads)

__host__ __device__ inline int grad_softmax_cp(int C) { return C <= 4 ? 4 : C <= 8 ? 8 : C <= 10 ? 10 : C <= 12 ? 12 : 16; }

// shared memory: the 8 rows, residuals, per-warp logit partials, an output staging tile, and (optionally) W and W - W'
__host__ __device__ inline size_t grad_softmax_smem(int F, int C, int has_bias, bool weights) {
  size_t n = (size_t)GSM_ROWS * (F + 4) + 2 * GSM_ROWS * GSM_CMAX + 2 * GSM_ROWS * 2 * GSM_CMAX +
             2 * (size_t)GSM_STAGE_FEATS * C;
  if (weights) n += 2 * ((size_t)(F + has_bias) * C + 4);
  return sizeof(float) * n + 64;
}
__host__ __device__ inline bool grad_softmax_weights_fit(int F, int C, int has_bias) {
  return grad_softmax_smem(F, C, has_bias, true) <= 110 * 1024;     // keeps two CTAs per SM
}

template <int CP, bool WSMEM>
__global__ void __launch_bounds__(GSM_THREADS) grad_softmax_kernel(const __grid_constant__ Params P) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  extern __shared__ __align__(16) float ssm[];
  const int F = P.F, C = P.C, xp = F + 4;
  float* s_x = ssm;                                   // [8][F + 4]
  float* s_r = s_x + (size_t)GSM_ROWS * xp;           // [8][CMAX]  (P - onehot)/B
  float* s_dr = s_r + GSM_ROWS * GSM_CMAX;            // [8][CMAX]  (P - P')/B
  float* s_zp = s_dr + GSM_ROWS * GSM_CMAX;           // [8 rows][2 warps][2 * CMAX] logit partials
  float* s_out = s_zp + 2 * GSM_ROWS * 2 * GSM_CMAX;  // [2][STAGE_FEATS * C] output staging
  float* s_w = s_out + 2 * (size_t)GSM_STAGE_FEATS * C;                       // [(F + bias) * C] W         (WSMEM)
  float* s_dw = s_w + ((size_t)(F + P.has_bias) * C + 3) / 4 * 4;             // [(F + bias) * C] W - W'    (WSMEM)
  const int m = blockIdx.y, chunk = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rowi = warp >> 1, wh = warp & 1;          // row of this warp, which half of the feature groups
  const long long k = P.st->k;
  const int i0 = chunk * GSM_ROWS;
  const int Bm = worker_batch(P, m);
  const int nrows = min(GSM_ROWS, Bm - i0);    // <= 0 for a block past this worker's rows: it writes zeros
  const float* __restrict__ X = static_cast<const float*>(P.X[m]);
  const long long n_m = P.n_samples[m];
  const float* __restrict__ th = P.theta;
  const float* __restrict__ tho = old_iterate(P, k, m);

  // stage: the two warps of a row copy alternate groups of 32 features
  long long row = -1;
  if (rowi < nrows) {
    row = minibatch_row(P, k, m, i0 + rowi, n_m);
    const float* __restrict__ x = X + row * P.ldx;
    for (int j = lane + 32 * wh; j < F; j += 64) s_x[rowi * xp + j] = x[j];
  }
  if (WSMEM) {            // the weights of both iterates, once per CTA, coalesced
    const int nw4 = ((F + P.has_bias) * C + 3) / 4;     // rows of the [M x p] buffers are padded, so the tail is readable
    for (int q = tid; q < nw4; q += GSM_THREADS) {
      const float4 a = reinterpret_cast<const float4*>(th)[q], b = reinterpret_cast<const float4*>(tho)[q];
      reinterpret_cast<float4*>(s_w)[q] = a;
      reinterpret_cast<float4*>(s_dw)[q] = make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w);
    }
  }
  __syncthreads();

  // forward: partial logits over this warp's features
  if (rowi < nrows) {
    float z[CP], dz[CP];
#pragma unroll
    for (int c = 0; c < CP; ++c) { z[c] = 0.f; dz[c] = 0.f; }
    for (int j = lane + 32 * wh; j < F; j += 64) {
      const float xv = s_x[rowi * xp + j];
      if (xv != 0.f) {
        if (WSMEM) {
#pragma unroll
          for (int c = 0; c < CP; ++c) {
            if (c < C) {
              z[c] = fmaf(xv, s_w[j * C + c], z[c]);
              dz[c] = fmaf(xv, s_dw[j * C + c], dz[c]);
            }
          }
        } else {
          const float* __restrict__ w = th + (long long)j * C;
          const float* __restrict__ wo = tho + (long long)j * C;
#pragma unroll
          for (int c = 0; c < CP; ++c) {
            if (c < C) {
              const float wv = w[c];
              z[c] = fmaf(xv, wv, z[c]);
              dz[c] = fmaf(xv, wv - wo[c], dz[c]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int c = 0; c < CP; ++c) {
      if (c < C) {
        const float a = warp_sum(z[c]), b = warp_sum(dz[c]);
        if (lane == 0) { s_zp[(rowi * 2 + wh) * 2 * GSM_CMAX + c] = a; s_zp[(rowi * 2 + wh) * 2 * GSM_CMAX + GSM_CMAX + c] = b; }
      }
    }
  }
  __syncthreads();

  // softmax: first warp of each row; every lane holds all logits, lane c writes class c
  if (rowi < nrows && wh == 0) {
    float z[CP], dz[CP];
    const float* p0 = s_zp + (rowi * 2) * 2 * GSM_CMAX;
    const float* p1 = p0 + 2 * GSM_CMAX;
#pragma unroll
    for (int c = 0; c < CP; ++c) {
      z[c] = 0.f; dz[c] = 0.f;
      if (c < C) {
        z[c] = p0[c] + p1[c];
        dz[c] = p0[GSM_CMAX + c] + p1[GSM_CMAX + c];
        if (P.has_bias) {
          const float b = th[(long long)F * C + c];
          z[c] += b;
          dz[c] += b - tho[(long long)F * C + c];
        }
      }
    }
    const int label = static_cast<const int*>(P.y[m])[row];
    float zmax = z[0], dzmax = fabsf(dz[0]);
#pragma unroll
    for (int c = 1; c < CP; ++c) if (c < C) { zmax = fmaxf(zmax, z[c]); dzmax = fmaxf(dzmax, fabsf(dz[c])); }
    float pc[CP], den = 0.f;
#pragma unroll
    for (int c = 0; c < CP; ++c) { pc[c] = c < C ? expf(z[c] - zmax) : 0.f; den += pc[c]; }
    const float inv = 1.f / den, invB = 1.0f / (float)Bm;
    float rr = 0.f, dd = 0.f;                 // values of class `lane`
    if (dzmax <= 20.f) {
      float T = 0.f, ec[CP];
#pragma unroll
      for (int c = 0; c < CP; ++c) { ec[c] = c < C ? expm1f(-dz[c]) : 0.f; T = fmaf(pc[c] * inv, ec[c], T); }
      const float invS = 1.f / (1.f + T);
#pragma unroll
      for (int c = 0; c < CP; ++c) {
        if (c == lane) {
          const float Pc = pc[c] * inv;
          rr = (Pc - (c == label ? 1.f : 0.f)) * invB;
          dd = Pc * (T - ec[c]) * invS * invB;
        }
      }
    } else {
      float zomax = z[0] - dz[0];
#pragma unroll
      for (int c = 1; c < CP; ++c) if (c < C) zomax = fmaxf(zomax, z[c] - dz[c]);
      float deno = 0.f;
#pragma unroll
      for (int c = 0; c < CP; ++c) if (c < C) deno += expf(z[c] - dz[c] - zomax);
#pragma unroll
      for (int c = 0; c < CP; ++c) {
        if (c == lane) {
          const float Pc = pc[c] * inv, Po = expf(z[c] - dz[c] - zomax) / deno;
          rr = (Pc - (c == label ? 1.f : 0.f)) * invB;
          dd = (Pc - Po) * invB;
        }
      }
    }
    if (lane < C) { s_r[rowi * GSM_CMAX + lane] = rr; s_dr[rowi * GSM_CMAX + lane] = dd; }
  }
  __syncthreads();

  // backward: rounds of STAGE_FEATS features; thread (half, f) accumulates g (half 0) or d (half 1) of feature f,
  // the round's 2 * STAGE_FEATS * C results go through shared memory and leave as contiguous runs
  float* __restrict__ out_g = P.part + ((long long)(m * P.n_chunks + chunk) * 2) * P.ldp;
  float* __restrict__ out_d = out_g + P.ldp;
  const int nfeat = F + (P.has_bias ? 1 : 0);
  const int half = tid / GSM_STAGE_FEATS, fl = tid - half * GSM_STAGE_FEATS;
  const float* __restrict__ s_res = half ? s_dr : s_r;
  for (int j0 = 0; j0 < nfeat; j0 += GSM_STAGE_FEATS) {
    const int j = j0 + fl;
    if (j < nfeat) {
      float acc[CP];
#pragma unroll
      for (int c = 0; c < CP; ++c) acc[c] = 0.f;
      for (int i = 0; i < nrows; ++i) {
        const float xv = j < F ? s_x[i * xp + j] : 1.f;
        if (xv != 0.f) {
#pragma unroll
          for (int c = 0; c < CP; ++c)
            if (c < C) acc[c] = fmaf(s_res[i * GSM_CMAX + c], xv, acc[c]);
        }
      }
#pragma unroll
      for (int c = 0; c < CP; ++c)
        if (c < C) s_out[(size_t)half * GSM_STAGE_FEATS * C + fl * C + c] = acc[c];
    }
    __syncthreads();
    const int nf = min(GSM_STAGE_FEATS, nfeat - j0), n = nf * C;
    for (int o = tid; o < 2 * n; o += GSM_THREADS) {
      const int hh = o >= n, oo = o - hh * n;
      (hh ? out_d : out_g)[(long long)j0 * C + oo] = s_out[(size_t)hh * GSM_STAGE_FEATS * C + oo];
    }
    __syncthreads();
  }
}

}  // namespace cada
