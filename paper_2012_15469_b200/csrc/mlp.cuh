// Two-point minibatch gradient of the 2-layer ReLU network (n_features - n_hidden - n_classes,
// softmax cross-entropy), plain-FMA version.
//
// Arithmetic contract (shared with the CPU oracle): the operands of every dense product -- the
// bf16 features, W1, W2, a1 = relu(z1), dz2 = (P - onehot)/B and dz1 -- are rounded to bfloat16
// (round to nearest even) immediately before the product; products are exact in fp32 and sums
// are accumulated in fp32; biases, the softmax and the bias gradients use unrounded fp32.
//
// Three kernels per iteration, each run for both iterates (blockIdx.z = 0: theta^k, 1: theta_hat_m):
//   mlp_f1_kernel   Z1 = X_B W1 + b1                      [B x H] per (worker, iterate)
//   mlp_f2_kernel   a1, Z2, softmax, dz2, dW2, db2, dA1, dz1, db1   (one CTA per (worker, iterate))
//   mlp_b1_kernel   dW1 = X_B^T dz1                        [F x H]
// Gradients land in the partial-slot buffer: slot (m, 0, 0) = grad at theta^k, (m, 0, 1) = grad at
// theta_hat_m; the trigger kernel forms their difference.
#pragma once
#include <cuda_bf16.h>
#include "common.cuh"

namespace cada {

__device__ __forceinline__ float bf16_round(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

struct MlpBufs {
  float* z1;     // [M][2][B][H]   hidden pre-activations
  float* dz1;    // [M][2][B][H]   their gradients, before the rounding to bf16
  float* dz2;    // [M][2][B][C]   output-layer gradients (P - onehot)/B, before the rounding to bf16
};

__device__ __forceinline__ const float* mlp_iterate(const Params& P, long long k, int m, int which) {
  return which == 0 ? P.theta : old_iterate(P, k, m);
}
__device__ __forceinline__ float* mlp_grad_out(const Params& P, int m, int which) {
  return P.part + ((long long)m * 2 + which) * P.ldp;
}

constexpr int MLP_THREADS = 256;
constexpr int MF1_TN = 64, MF1_TK = 16, MF1_ROWS = 128;

// Z1 tile: up to 128 minibatch rows x 64 hidden units.  grid (ceil(H/64), M * ceil(B/128), 2)
__global__ void __launch_bounds__(MLP_THREADS) mlp_f1_kernel(const __grid_constant__ Params P, MlpBufs mb) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  __shared__ float As[MF1_TK][MF1_ROWS + 4];
  __shared__ float Bs[MF1_TK][MF1_TN + 4];
  __shared__ long long s_row[MF1_ROWS];
  const int row_tiles = (P.B + MF1_ROWS - 1) / MF1_ROWS;
  const int m = blockIdx.y / row_tiles, rt = blockIdx.y - m * row_tiles, which = blockIdx.z;
  const int i0 = rt * MF1_ROWS, n0 = blockIdx.x * MF1_TN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int F = P.F, H = P.H;
  const long long k = P.st->k;
  const __nv_bfloat16* __restrict__ X = static_cast<const __nv_bfloat16*>(P.X[m]);
  const float* __restrict__ W1 = mlp_iterate(P, k, m, which);
  const float* __restrict__ b1 = W1 + (long long)F * H;
  if (tid < MF1_ROWS) s_row[tid] = (i0 + tid < P.B) ? minibatch_row(P, k, m, i0 + tid, P.n_samples[m]) : -1;
  __syncthreads();
  float acc[8][4];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  for (int k0 = 0; k0 < F; k0 += MF1_TK) {
    {  // A chunk: 128 rows x 16 features; thread -> (row, half of the 16)
      const int r = tid >> 1, kh = (tid & 1) * 8;
      const long long row = s_row[r];
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const int f = k0 + kh + e;
        As[kh + e][r] = (row >= 0 && f < F) ? __bfloat162float(X[row * P.ldx + f]) : 0.f;
      }
    }
    {  // B chunk: 16 x 64 weights, rounded
      const int kk = tid >> 4, nn = (tid & 15) * 4;
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int f = k0 + kk, h = n0 + nn + e;
        Bs[kk][nn + e] = (f < F && h < H) ? bf16_round(W1[(long long)f * H + h]) : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < MF1_TK; ++kk) {
      float a[8], b[4];
#pragma unroll
      for (int e = 0; e < 8; ++e) a[e] = As[kk][ty * 8 + e];
#pragma unroll
      for (int e = 0; e < 4; ++e) b[e] = Bs[kk][tx * 4 + e];
#pragma unroll
      for (int x = 0; x < 8; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
    }
    __syncthreads();
  }
  float* __restrict__ out = mb.z1 + (((long long)m * 2 + which) * P.B) * H;
#pragma unroll
  for (int x = 0; x < 8; ++x) {
    const int i = i0 + ty * 8 + x;
    if (i >= P.B) continue;
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int h = n0 + tx * 4 + y;
      if (h < H) out[(long long)i * H + h] = acc[x][y] + b1[h];
    }
  }
}

// Everything between the two large products.  One CTA per (worker, iterate); rows are processed in
// blocks of 64 so that shared memory does not grow with the batch.
constexpr int MF2_RB = 64;
__host__ __device__ inline size_t mlp_f2_smem(int H, int C) {
  const size_t hp = (size_t)H + 1;
  return sizeof(float) * (2 * MF2_RB * hp + (size_t)H * C + 3 * MF2_RB * (size_t)C + 2 * (size_t)C + (size_t)H) + 64;
}

__global__ void __launch_bounds__(MLP_THREADS) mlp_f2_kernel(const __grid_constant__ Params P, MlpBufs mb) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  extern __shared__ __align__(16) float sf[];
  const int m = blockIdx.x, which = blockIdx.y, tid = threadIdx.x;
  const int F = P.F, H = P.H, C = P.C, B = P.B, hp = H + 1;
  float* s_a1 = sf;                              // [RB][hp]  a1 rounded (0 where z1 <= 0)
  float* s_dz1 = s_a1 + (size_t)MF2_RB * hp;     // [RB][hp]  sign of z1, then dz1
  float* s_w2 = s_dz1 + (size_t)MF2_RB * hp;     // [H][C] rounded
  float* s_z2 = s_w2 + (size_t)H * C;            // [RB][C]
  float* s_dz2 = s_z2 + (size_t)MF2_RB * C;      // [RB][C] fp32
  float* s_dz2q = s_dz2 + (size_t)MF2_RB * C;    // [RB][C] rounded
  float* s_b2 = s_dz2q + (size_t)MF2_RB * C;     // [C]
  float* s_db2 = s_b2 + C;                       // [C]
  float* s_db1 = s_db2 + C;                      // [H]
  const long long k = P.st->k;
  const float* __restrict__ th = mlp_iterate(P, k, m, which);
  const float* __restrict__ W2 = th + (long long)F * H + H;
  const float* __restrict__ b2 = W2 + (long long)H * C;
  const int* __restrict__ ym = static_cast<const int*>(P.y[m]);
  const long long n_m = P.n_samples[m];
  const float* __restrict__ z1 = mb.z1 + (((long long)m * 2 + which) * B) * H;
  float* __restrict__ dz1o = mb.dz1 + (((long long)m * 2 + which) * B) * H;
  float* __restrict__ dz2o = mb.dz2 + (((long long)m * 2 + which) * B) * C;
  float* __restrict__ g = mlp_grad_out(P, m, which);
  float* __restrict__ g_b1 = g + (long long)F * H;
  float* __restrict__ g_w2 = g_b1 + H;
  float* __restrict__ g_b2 = g_w2 + (long long)H * C;
  const float invB = 1.0f / (float)B;

  for (int o = tid; o < H * C; o += MLP_THREADS) s_w2[o] = bf16_round(W2[o]);
  for (int c = tid; c < C; c += MLP_THREADS) { s_b2[c] = b2[c]; s_db2[c] = 0.f; }
  for (int h = tid; h < H; h += MLP_THREADS) s_db1[h] = 0.f;
  // dW2 accumulators: output o = h*C + c handled by thread o % 256, up to 8 outputs each pass
  constexpr int W2_PER = 8;
  float w2acc[W2_PER];
#pragma unroll
  for (int e = 0; e < W2_PER; ++e) w2acc[e] = 0.f;
  const int n_w2_pass = (H * C + MLP_THREADS * W2_PER - 1) / (MLP_THREADS * W2_PER);   // > 1 only for very wide layers
  __syncthreads();

  for (int pass = 0; pass < n_w2_pass; ++pass) {
#pragma unroll
    for (int e = 0; e < W2_PER; ++e) w2acc[e] = 0.f;
    for (int i0 = 0; i0 < B; i0 += MF2_RB) {
      const int nr = min(MF2_RB, B - i0);
      // a1 = relu(z1), rounded; remember the sign of z1 in s_dz1
      for (int o = tid; o < nr * H; o += MLP_THREADS) {
        const int i = o / H, h = o - i * H;
        const float z = z1[(long long)(i0 + i) * H + h];
        s_a1[i * hp + h] = z > 0.f ? bf16_round(z) : 0.f;
        s_dz1[i * hp + h] = z > 0.f ? 1.f : 0.f;
      }
      __syncthreads();
      // z2 = a1 W2 + b2
      for (int o = tid; o < nr * C; o += MLP_THREADS) {
        const int i = o / C, c = o - i * C;
        float acc = 0.f;
        for (int h = 0; h < H; ++h) acc = fmaf(s_a1[i * hp + h], s_w2[h * C + c], acc);
        s_z2[i * C + c] = acc + s_b2[c];
      }
      __syncthreads();
      // softmax and dz2 = (P - onehot)/B
      for (int i = tid; i < nr; i += MLP_THREADS) {
        const long long row = minibatch_row(P, k, m, i0 + i, n_m);
        const int label = ym[row];
        float mx = s_z2[i * C];
        for (int c = 1; c < C; ++c) mx = fmaxf(mx, s_z2[i * C + c]);
        float den = 0.f;
        for (int c = 0; c < C; ++c) den += expf(s_z2[i * C + c] - mx);
        const float inv = 1.f / den;
        for (int c = 0; c < C; ++c) {
          const float d = (expf(s_z2[i * C + c] - mx) * inv - (c == label ? 1.f : 0.f)) * invB;
          s_dz2[i * C + c] = d;
          s_dz2q[i * C + c] = bf16_round(d);
          if (pass == 0) dz2o[(long long)(i0 + i) * C + c] = d;
        }
      }
      __syncthreads();
      if (pass == 0) {
        // db2 (fp32, unrounded dz2)
        if (tid < C) { float a = s_db2[tid]; for (int i = 0; i < nr; ++i) a += s_dz2[i * C + tid]; s_db2[tid] = a; }
        // dA1 = dz2q W2q^T, dz1 = dA1 where z1 > 0
        for (int o = tid; o < nr * H; o += MLP_THREADS) {
          const int i = o / H, h = o - i * H;
          float acc = 0.f;
          for (int c = 0; c < C; ++c) acc = fmaf(s_dz2q[i * C + c], s_w2[h * C + c], acc);
          const float d = s_dz1[i * hp + h] > 0.f ? acc : 0.f;
          s_dz1[i * hp + h] = d;
          dz1o[(long long)(i0 + i) * H + h] = d;          // rounded to bf16 where the dW1 product loads it
        }
      }
      // dW2 += a1q^T dz2q
#pragma unroll
      for (int e = 0; e < W2_PER; ++e) {
        const int o = (pass * W2_PER + e) * MLP_THREADS + tid;
        if (o < H * C) {
          const int h = o / C, c = o - h * C;
          float acc = w2acc[e];
          for (int i = 0; i < nr; ++i) acc = fmaf(s_a1[i * hp + h], s_dz2q[i * C + c], acc);
          w2acc[e] = acc;
        }
      }
      __syncthreads();
      if (pass == 0) {   // db1 (fp32, unrounded dz1)
        for (int h = tid; h < H; h += MLP_THREADS) { float a = s_db1[h]; for (int i = 0; i < nr; ++i) a += s_dz1[i * hp + h]; s_db1[h] = a; }
      }
      __syncthreads();
    }
#pragma unroll
    for (int e = 0; e < W2_PER; ++e) {
      const int o = (pass * W2_PER + e) * MLP_THREADS + tid;
      if (o < H * C) g_w2[o] = w2acc[e];
    }
  }
  for (int c = tid; c < C; c += MLP_THREADS) g_b2[c] = s_db2[c];
  for (int h = tid; h < H; h += MLP_THREADS) g_b1[h] = s_db1[h];
}

// dW1 tile: 64 features x 64 hidden units, contraction over the minibatch.  grid (ceil(H/64), ceil(F/64), M*2)
constexpr int MB1_T = 64, MB1_TK = 16;
__global__ void __launch_bounds__(MLP_THREADS) mlp_b1_kernel(const __grid_constant__ Params P, MlpBufs mb) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  __shared__ float As[MB1_TK][MB1_T + 4];   // [row][feature]
  __shared__ float Bs[MB1_TK][MB1_T + 4];   // [row][hidden]
  __shared__ long long s_row[MB1_TK];
  const int m = blockIdx.z >> 1, which = blockIdx.z & 1;
  const int f0 = blockIdx.y * MB1_T, h0 = blockIdx.x * MB1_T;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int F = P.F, H = P.H, B = P.B;
  const long long k = P.st->k;
  const __nv_bfloat16* __restrict__ X = static_cast<const __nv_bfloat16*>(P.X[m]);
  const float* __restrict__ dz1 = mb.dz1 + (((long long)m * 2 + which) * B) * H;
  const long long n_m = P.n_samples[m];
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
  for (int i0 = 0; i0 < B; i0 += MB1_TK) {
    if (tid < MB1_TK) s_row[tid] = (i0 + tid < B) ? minibatch_row(P, k, m, i0 + tid, n_m) : -1;
    __syncthreads();
    {
      const int r = tid >> 4, c4 = (tid & 15) * 4;
      const long long row = s_row[r];
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int f = f0 + c4 + e, h = h0 + c4 + e;
        As[r][c4 + e] = (row >= 0 && f < F) ? __bfloat162float(X[row * P.ldx + f]) : 0.f;
        Bs[r][c4 + e] = (row >= 0 && h < H) ? bf16_round(dz1[(long long)(i0 + r) * H + h]) : 0.f;
      }
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < MB1_TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int e = 0; e < 4; ++e) { a[e] = As[kk][ty * 4 + e]; b[e] = Bs[kk][tx * 4 + e]; }
#pragma unroll
      for (int x = 0; x < 4; ++x)
#pragma unroll
        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
    }
    __syncthreads();
  }
  float* __restrict__ g = mlp_grad_out(P, m, which);
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const int f = f0 + ty * 4 + x;
    if (f >= F) continue;
#pragma unroll
    for (int y = 0; y < 4; ++y) {
      const int h = h0 + tx * 4 + y;
      if (h < H) g[(long long)f * H + h] = acc[x][y];
    }
  }
}

}  // namespace cada
