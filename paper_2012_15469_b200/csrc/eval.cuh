// Full-data evaluation at the current iterate: the loss of Eq. 1, L = (1/M) sum_m L_m(theta) with L_m the mean loss of
// worker m's rows plus (lambda/2)||theta||^2, and the fraction of all rows that are classified correctly -- the
// quantities the paper plots against iterations and uploads (Section 4).  Not on the iteration path.
//
// One warp per row (4 rows per warp for the MLP, so that W1 is re-read less often); per-CTA partial sums
// (loss in fp64, correct count) go to a scratch array that the host adds up in a fixed order.
#pragma once
#include <cuda_bf16.h>
#include "common.cuh"

namespace cada {

constexpr int EV_THREADS = 256;
constexpr int EV_CHUNKS = 64;        // CTAs per worker
constexpr int EV_CMAX = 16;

// scratch: [M][EV_CHUNKS][2] doubles: (sum of row losses, number of correct rows)
__global__ void __launch_bounds__(EV_THREADS) eval_linear_kernel(const __grid_constant__ Params P, double* __restrict__ out) {
  __shared__ double s_loss[EV_THREADS / 32], s_ok[EV_THREADS / 32];
  const int m = blockIdx.y, chunk = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int F = P.F, C = P.C;
  const long long n_m = P.n_samples[m];
  const float* __restrict__ X = static_cast<const float*>(P.X[m]);
  const float* __restrict__ th = P.theta;
  double loss = 0.0, okc = 0.0;
  for (long long row = (long long)chunk * (EV_THREADS / 32) + warp; row < n_m; row += (long long)EV_CHUNKS * (EV_THREADS / 32)) {
    const float* __restrict__ x = X + row * P.ldx;
    if (P.model == 0) {
      float z = 0.f;
      for (int j = lane; j < F; j += 32) z = fmaf(x[j], th[j], z);
      z = warp_sum(z);
      if (P.has_bias) z += th[F];
      const float y = static_cast<const float*>(P.y[m])[row];
      const float t = -y * z;                                   // log(1 + exp(-y z))
      loss += (double)(fmaxf(t, 0.f) + log1pf(expf(-fabsf(t))));
      okc += ((z >= 0.f) == (y > 0.f)) ? 1.0 : 0.0;
    } else {
      float z[EV_CMAX];
#pragma unroll
      for (int c = 0; c < EV_CMAX; ++c) z[c] = 0.f;
      for (int j = lane; j < F; j += 32) {
        const float xv = x[j];
        if (xv != 0.f) {
#pragma unroll
          for (int c = 0; c < EV_CMAX; ++c) if (c < C) z[c] = fmaf(xv, th[(long long)j * C + c], z[c]);
        }
      }
      float zmax = -INFINITY;
      int arg = 0;
#pragma unroll
      for (int c = 0; c < EV_CMAX; ++c) {
        if (c < C) {
          z[c] = warp_sum(z[c]);
          if (P.has_bias) z[c] += th[(long long)F * C + c];
          if (z[c] > zmax) { zmax = z[c]; arg = c; }
        }
      }
      const int label = static_cast<const int*>(P.y[m])[row];
      float den = 0.f, zl = 0.f;
#pragma unroll
      for (int c = 0; c < EV_CMAX; ++c) if (c < C) { den += expf(z[c] - zmax); if (c == label) zl = z[c]; }
      loss += (double)(zmax + logf(den) - zl);
      okc += arg == label ? 1.0 : 0.0;
    }
  }
  if (lane == 0) { s_loss[warp] = loss; s_ok[warp] = okc; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, b = 0.0;
    for (int w = 0; w < EV_THREADS / 32; ++w) { a += s_loss[w]; b += s_ok[w]; }
    out[((long long)m * EV_CHUNKS + chunk) * 2] = a;
    out[((long long)m * EV_CHUNKS + chunk) * 2 + 1] = b;
  }
}

// MLP: same contract as the training forward pass (operands of the two products rounded to bf16, fp32 sums).
// One warp per group of 4 rows; lane l owns hidden units l, l+32, ... (up to 8 per lane: H <= 256).
__global__ void __launch_bounds__(EV_THREADS) eval_mlp_kernel(const __grid_constant__ Params P, double* __restrict__ out) {
  __shared__ double s_loss[EV_THREADS / 32], s_ok[EV_THREADS / 32];
  constexpr int RW = 4, HL = 8;
  const int m = blockIdx.y, chunk = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int F = P.F, C = P.C, H = P.H;
  const long long n_m = P.n_samples[m];
  const __nv_bfloat16* __restrict__ X = static_cast<const __nv_bfloat16*>(P.X[m]);
  const float* __restrict__ W1 = P.theta;
  const float* __restrict__ b1 = W1 + (long long)F * H;
  const float* __restrict__ W2 = b1 + H;
  const float* __restrict__ b2 = W2 + (long long)H * C;
  double loss = 0.0, okc = 0.0;
  const long long n_groups = (n_m + RW - 1) / RW;
  for (long long gr = (long long)chunk * (EV_THREADS / 32) + warp; gr < n_groups; gr += (long long)EV_CHUNKS * (EV_THREADS / 32)) {
    float z1[RW][HL];
#pragma unroll
    for (int r = 0; r < RW; ++r)
#pragma unroll
      for (int e = 0; e < HL; ++e) z1[r][e] = 0.f;
    for (int f = 0; f < F; ++f) {
      float xv[RW];
#pragma unroll
      for (int r = 0; r < RW; ++r) { const long long row = gr * RW + r; xv[r] = row < n_m ? __bfloat162float(X[row * P.ldx + f]) : 0.f; }
      if (xv[0] == 0.f && xv[1] == 0.f && xv[2] == 0.f && xv[3] == 0.f) continue;
#pragma unroll
      for (int e = 0; e < HL; ++e) {
        const int h = lane + 32 * e;
        if (h < H) {
          const float w = __bfloat162float(__float2bfloat16_rn(W1[(long long)f * H + h]));
#pragma unroll
          for (int r = 0; r < RW; ++r) z1[r][e] = fmaf(xv[r], w, z1[r][e]);
        }
      }
    }
#pragma unroll
    for (int r = 0; r < RW; ++r) {
      const long long row = gr * RW + r;
      float z2[EV_CMAX];
#pragma unroll
      for (int c = 0; c < EV_CMAX; ++c) z2[c] = 0.f;
#pragma unroll
      for (int e = 0; e < HL; ++e) {
        const int h = lane + 32 * e;
        if (h < H) {
          const float a = z1[r][e] + b1[h];
          const float aq = a > 0.f ? __bfloat162float(__float2bfloat16_rn(a)) : 0.f;
#pragma unroll
          for (int c = 0; c < EV_CMAX; ++c)
            if (c < C) z2[c] = fmaf(aq, __bfloat162float(__float2bfloat16_rn(W2[(long long)h * C + c])), z2[c]);
        }
      }
      float zmax = -INFINITY;
      int arg = 0;
#pragma unroll
      for (int c = 0; c < EV_CMAX; ++c) {
        if (c < C) { z2[c] = warp_sum(z2[c]) + b2[c]; if (z2[c] > zmax) { zmax = z2[c]; arg = c; } }
      }
      if (row < n_m) {
        const int label = static_cast<const int*>(P.y[m])[row];
        float den = 0.f, zl = 0.f;
#pragma unroll
        for (int c = 0; c < EV_CMAX; ++c) if (c < C) { den += expf(z2[c] - zmax); if (c == label) zl = z2[c]; }
        loss += (double)(zmax + logf(den) - zl);
        okc += arg == label ? 1.0 : 0.0;
      }
    }
  }
  if (lane == 0) { s_loss[warp] = loss; s_ok[warp] = okc; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double a = 0.0, b = 0.0;
    for (int w = 0; w < EV_THREADS / 32; ++w) { a += s_loss[w]; b += s_ok[w]; }
    out[((long long)m * EV_CHUNKS + chunk) * 2] = a;
    out[((long long)m * EV_CHUNKS + chunk) * 2 + 1] = b;
  }
}

}  // namespace cada
