// Two-point minibatch gradient, shape-generic version (binary logistic and softmax regression).
//
// For worker m and a chunk of its minibatch rows, one CTA computes the partial sums of
//   g_m  = grad l(theta^k ; xi_m^k)                       (Algorithm 1, first gradient)
//   d_m  = g_m - grad l(theta' ; xi_m^k)                  (the same rows, old iterate theta')
// without the regulariser term, which the trigger kernel adds once per worker.  d_m is formed
// from the logit difference dz = x.(theta - theta') so that it keeps its relative accuracy when
// the two iterates are close (the upload test of Eqs. 6 / 8 compares ||d||^2 with a small RHS).
//
//   phase 1a  one warp per (row, class): logits z and dz, lanes strided over the features
//   phase 1b  one thread per row: residuals r = (P - onehot)/B and dr = (P - P')/B
//   phase 2   one thread per output (feature, class): sum_i r[i][c] * x[i][feature]
// The rows of the chunk are read from global memory in phase 1a and again (from L1/L2) in
// phase 2.  The streaming kernel in grad_stream.cuh replaces this one where rows are long.
#pragma once
#include "common.cuh"

namespace cada {

constexpr int GG_THREADS = 256;

// dynamic shared memory: int64 row[RB] | float z[RB][2C] | float r[RB][2C]
__host__ __device__ inline size_t grad_generic_smem(int rows_per_chunk, int C) {
  return (size_t)rows_per_chunk * (sizeof(long long) + 4 * (size_t)C * sizeof(float));
}

__global__ void __launch_bounds__(GG_THREADS) grad_generic_kernel(const __grid_constant__ Params P) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int RB = P.rows_per_chunk, C = P.C, F = P.F;
  long long* s_row = reinterpret_cast<long long*>(smem_raw);
  float* s_z = reinterpret_cast<float*>(s_row + RB);          // [RB][2C]: z | dz
  float* s_r = s_z + (size_t)RB * 2 * C;                      // [RB][2C]: r | dr

  const int m = blockIdx.y, chunk = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = GG_THREADS / 32;
  const long long k = P.st->k;
  const int i0 = chunk * RB;
  const int Bm = worker_batch(P, m);
  const int nrows = min(RB, Bm - i0);          // <= 0 for a chunk past this worker's rows: it writes zeros
  const float* __restrict__ X = static_cast<const float*>(P.X[m]);
  const long long n_m = P.n_samples[m];
  const float* __restrict__ th = P.theta;
  const float* __restrict__ tho = old_iterate(P, k, m);

  for (int i = tid; i < nrows; i += GG_THREADS) s_row[i] = minibatch_row(P, k, m, i0 + i, n_m);
  __syncthreads();

  // phase 1a
  for (int item = warp; item < nrows * C; item += nwarps) {
    const int i = item / C, c = item - i * C;
    const float* __restrict__ x = X + s_row[i] * P.ldx;
    float z = 0.f, dz = 0.f;
    for (int j = lane; j < F; j += 32) {
      const float xv = x[j];
      const float w = th[(long long)j * C + c];
      const float wo = tho[(long long)j * C + c];
      z = fmaf(xv, w, z);
      dz = fmaf(xv, w - wo, dz);
    }
    z = warp_sum(z);
    dz = warp_sum(dz);
    if (lane == 0) {
      if (P.has_bias) {
        const float b = th[(long long)F * C + c], bo = tho[(long long)F * C + c];
        z += b;
        dz += b - bo;
      }
      s_z[(size_t)i * 2 * C + c] = z;
      s_z[(size_t)i * 2 * C + C + c] = dz;
    }
  }
  __syncthreads();

  // phase 1b
  const float invB = 1.0f / (float)Bm;
  for (int i = tid; i < nrows; i += GG_THREADS) {
    const float* z = s_z + (size_t)i * 2 * C;
    const float* dz = z + C;
    float* r = s_r + (size_t)i * 2 * C;
    float* dr = r + C;
    if (P.model == 0) {
      const float yv = static_cast<const float*>(P.y[m])[s_row[i]];
      const float t = 0.5f * (yv + 1.0f);
      r[0] = (sigmoidf_stable(z[0]) - t) * invB;
      dr[0] = sigmoid_diff(z[0], dz[0]) * invB;
    } else {
      const int label = static_cast<const int*>(P.y[m])[s_row[i]];
      float zmax = z[0], dzmax = fabsf(dz[0]);
      for (int c = 1; c < C; ++c) { zmax = fmaxf(zmax, z[c]); dzmax = fmaxf(dzmax, fabsf(dz[c])); }
      float den = 0.f;
      for (int c = 0; c < C; ++c) den += expf(z[c] - zmax);
      const float inv = 1.f / den;
      if (dzmax <= 20.f) {
        // P_c - P'_c = P_c (T - e_c)/(1 + T),  e_c = expm1(-dz_c),  T = sum_j P_j e_j
        float T = 0.f;
        for (int c = 0; c < C; ++c) T += expf(z[c] - zmax) * inv * expm1f(-dz[c]);
        const float invS = 1.f / (1.f + T);
        for (int c = 0; c < C; ++c) {
          const float Pc = expf(z[c] - zmax) * inv;
          r[c] = (Pc - (c == label ? 1.f : 0.f)) * invB;
          dr[c] = Pc * (T - expm1f(-dz[c])) * invS * invB;
        }
      } else {
        float zomax = z[0] - dz[0];
        for (int c = 1; c < C; ++c) zomax = fmaxf(zomax, z[c] - dz[c]);
        float deno = 0.f;
        for (int c = 0; c < C; ++c) deno += expf(z[c] - dz[c] - zomax);
        for (int c = 0; c < C; ++c) {
          const float Pc = expf(z[c] - zmax) * inv;
          const float Po = expf(z[c] - dz[c] - zomax) / deno;
          r[c] = (Pc - (c == label ? 1.f : 0.f)) * invB;
          dr[c] = (Pc - Po) * invB;
        }
      }
    }
  }
  __syncthreads();

  // phase 2
  float* __restrict__ out_g = P.part + ((long long)(m * P.n_chunks + chunk) * 2) * P.ldp;
  float* __restrict__ out_d = out_g + P.ldp;
  for (long long o = tid; o < P.p; o += GG_THREADS) {
    const int j = (int)(o / C), c = (int)(o - (long long)j * C);
    float ag = 0.f, ad = 0.f;
    if (j < F) {
      for (int i = 0; i < nrows; ++i) {
        const float xv = X[s_row[i] * P.ldx + j];
        ag = fmaf(s_r[(size_t)i * 2 * C + c], xv, ag);
        ad = fmaf(s_r[(size_t)i * 2 * C + C + c], xv, ad);
      }
    } else {  // constant-1 feature
      for (int i = 0; i < nrows; ++i) {
        ag += s_r[(size_t)i * 2 * C + c];
        ad += s_r[(size_t)i * 2 * C + C + c];
      }
    }
    out_g[o] = ag;
    out_d[o] = ad;
  }
}

}  // namespace cada
