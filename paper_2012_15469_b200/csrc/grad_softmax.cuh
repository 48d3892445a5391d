// Two-point minibatch gradient for softmax regression with up to 16 classes.
//
// One CTA per (worker, block of 8 minibatch rows); warp i owns row i.
//   stage    the 8 rows are copied to shared memory once (read once from global memory)
//   forward  lane l of warp i walks features l, l+32, ...: for every NON-ZERO x it adds x * W[j][:]
//            and x * (W - W')[j][:] to its C logit accumulators (sparse inputs skip most features);
//            the 2C values are summed over the warp
//   softmax  lanes c < C of each warp form P, P - onehot and the accurate difference
//            P_c - P'_c = P_c (T - e_c) / (1 + T), e_c = expm1(-dz_c), T = sum_j P_j e_j
//   backward thread t owns features t, t+256, ...: for each it accumulates r[i][:] * x and dr[i][:] * x
//            over the 8 rows (again skipping zeros) and writes 2C partial sums
// Output: partial slot (worker, row block) of g_m and d_m = g_m - g'_m, without the regulariser.
#pragma once
#include "common.cuh"

namespace cada {

constexpr int GSM_THREADS = 256;
constexpr int GSM_ROWS = 8;          // rows per CTA = warps per CTA
constexpr int GSM_CMAX = 16;

// shared memory: the 8 rows, the residuals, an output staging tile, and (when `weights` is set) W and W - W'
constexpr int GSM_STAGE_FEATS = 128;          // features per coalesced store round
__host__ __device__ inline size_t grad_softmax_smem(int F, int C, int has_bias, bool weights) {
  size_t n = (size_t)GSM_ROWS * (F + 4) + 2 * GSM_ROWS * GSM_CMAX + 2 * (size_t)GSM_STAGE_FEATS * C;
  if (weights) n += 2 * ((size_t)(F + has_bias) * C + 4);
  return sizeof(float) * n + 64;
}
__host__ __device__ inline bool grad_softmax_weights_fit(int F, int C, int has_bias) {
  return grad_softmax_smem(F, C, has_bias, true) <= 100 * 1024;     // keeps two CTAs per SM
}

template <bool WSMEM>
__global__ void __launch_bounds__(GSM_THREADS) grad_softmax_kernel(const __grid_constant__ Params P) {
  extern __shared__ __align__(16) float ssm[];
  const int F = P.F, C = P.C, xp = F + 4;
  float* s_x = ssm;                                   // [8][F + 4]
  float* s_r = s_x + (size_t)GSM_ROWS * xp;           // [8][CMAX]  (P - onehot)/B
  float* s_dr = s_r + GSM_ROWS * GSM_CMAX;            // [8][CMAX]  (P - P')/B
  float* s_out = s_dr + GSM_ROWS * GSM_CMAX;          // [2][STAGE_FEATS * C] output staging
  float* s_w = s_out + 2 * (size_t)GSM_STAGE_FEATS * C;                       // [(F + bias) * C] W         (WSMEM)
  float* s_dw = s_w + ((size_t)(F + P.has_bias) * C + 3) / 4 * 4;             // [(F + bias) * C] W - W'    (WSMEM)
  const int m = blockIdx.y, chunk = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long k = P.st->k;
  const int i0 = chunk * GSM_ROWS;
  const int nrows = min(GSM_ROWS, P.B - i0);
  const float* __restrict__ X = static_cast<const float*>(P.X[m]);
  const long long n_m = P.n_samples[m];
  const float* __restrict__ th = P.theta;
  const float* __restrict__ tho = old_iterate(P, k, m);

  // stage: warp i copies row i
  long long row = -1;
  if (warp < nrows) {
    row = minibatch_row(P, k, m, i0 + warp, n_m);
    const float* __restrict__ x = X + row * P.ldx;
    for (int j = lane; j < F; j += 32) s_x[warp * xp + j] = x[j];
  }
  if (WSMEM) {            // the weights of both iterates, once per CTA, coalesced
    const int nw4 = ((F + P.has_bias) * C + 3) / 4;     // rows of the [M x p] buffers are padded, so the tail is readable
    for (int q = tid; q < nw4; q += GSM_THREADS) {
      const float4 a = reinterpret_cast<const float4*>(th)[q], b = reinterpret_cast<const float4*>(tho)[q];
      reinterpret_cast<float4*>(s_w)[q] = a;
      reinterpret_cast<float4*>(s_dw)[q] = make_float4(a.x - b.x, a.y - b.y, a.z - b.z, a.w - b.w);
    }
    __syncthreads();
  } else {
    __syncwarp();
  }

  // forward (each warp only reads the row it staged itself)
  float z[GSM_CMAX], dz[GSM_CMAX];
#pragma unroll
  for (int c = 0; c < GSM_CMAX; ++c) { z[c] = 0.f; dz[c] = 0.f; }
  if (warp < nrows) {
    for (int j = lane; j < F; j += 32) {
      const float xv = s_x[warp * xp + j];
      if (xv != 0.f) {
        if (WSMEM) {
#pragma unroll
          for (int c = 0; c < GSM_CMAX; ++c) {
            if (c < C) {
              z[c] = fmaf(xv, s_w[j * C + c], z[c]);
              dz[c] = fmaf(xv, s_dw[j * C + c], dz[c]);
            }
          }
        } else {
          const float* __restrict__ w = th + (long long)j * C;
          const float* __restrict__ wo = tho + (long long)j * C;
#pragma unroll
          for (int c = 0; c < GSM_CMAX; ++c) {
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
    for (int c = 0; c < GSM_CMAX; ++c) {
      if (c < C) { z[c] = warp_sum(z[c]); dz[c] = warp_sum(dz[c]); }
    }
    if (P.has_bias) {
#pragma unroll
      for (int c = 0; c < GSM_CMAX; ++c) {
        if (c < C) {
          const float b = th[(long long)F * C + c];
          z[c] += b;
          dz[c] += b - tho[(long long)F * C + c];
        }
      }
    }
    // softmax (every lane holds all logits; the arithmetic is replicated, lane c writes class c)
    const int label = static_cast<const int*>(P.y[m])[row];
    float zmax = z[0], dzmax = fabsf(dz[0]);
#pragma unroll
    for (int c = 1; c < GSM_CMAX; ++c) if (c < C) { zmax = fmaxf(zmax, z[c]); dzmax = fmaxf(dzmax, fabsf(dz[c])); }
    float pc[GSM_CMAX], den = 0.f;
#pragma unroll
    for (int c = 0; c < GSM_CMAX; ++c) { pc[c] = c < C ? expf(z[c] - zmax) : 0.f; den += pc[c]; }
    const float inv = 1.f / den, invB = 1.0f / (float)P.B;
    float rr = 0.f, dd = 0.f;                 // values of class `lane`
    if (dzmax <= 20.f) {
      float T = 0.f, ec[GSM_CMAX];
#pragma unroll
      for (int c = 0; c < GSM_CMAX; ++c) { ec[c] = c < C ? expm1f(-dz[c]) : 0.f; T = fmaf(pc[c] * inv, ec[c], T); }
      const float invS = 1.f / (1.f + T);
#pragma unroll
      for (int c = 0; c < GSM_CMAX; ++c) {
        if (c == lane) {
          const float Pc = pc[c] * inv;
          rr = (Pc - (c == label ? 1.f : 0.f)) * invB;
          dd = Pc * (T - ec[c]) * invS * invB;
        }
      }
    } else {
      float zomax = z[0] - dz[0];
#pragma unroll
      for (int c = 1; c < GSM_CMAX; ++c) if (c < C) zomax = fmaxf(zomax, z[c] - dz[c]);
      float deno = 0.f;
#pragma unroll
      for (int c = 0; c < GSM_CMAX; ++c) if (c < C) deno += expf(z[c] - dz[c] - zomax);
#pragma unroll
      for (int c = 0; c < GSM_CMAX; ++c) {
        if (c == lane) {
          const float Pc = pc[c] * inv, Po = expf(z[c] - dz[c] - zomax) / deno;
          rr = (Pc - (c == label ? 1.f : 0.f)) * invB;
          dd = (Pc - Po) * invB;
        }
      }
    }
    if (lane < C) { s_r[warp * GSM_CMAX + lane] = rr; s_dr[warp * GSM_CMAX + lane] = dd; }
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
      float acc[GSM_CMAX];
#pragma unroll
      for (int c = 0; c < GSM_CMAX; ++c) acc[c] = 0.f;
      for (int i = 0; i < nrows; ++i) {
        const float xv = j < F ? s_x[i * xp + j] : 1.f;
        if (xv != 0.f) {
#pragma unroll
          for (int c = 0; c < GSM_CMAX; ++c)
            if (c < C) acc[c] = fmaf(s_res[i * GSM_CMAX + c], xv, acc[c]);
        }
      }
#pragma unroll
      for (int c = 0; c < GSM_CMAX; ++c)
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
