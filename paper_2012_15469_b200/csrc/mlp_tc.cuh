// Tensor-core (tcgen05) version of the two large products of the MLP gradient:
//     Z1  = X_B W1 + b1          [B x H],  contraction over the F features        (mlp_f1_tc_kernel)
//     dW1 = X_B^T dz1            [F x H],  contraction over the B minibatch rows  (mlp_b1_tc_kernel)
// bf16 operands, fp32 accumulation in tensor memory, one CTA-wide MMA stream issued by one thread.
//
// Operand images.  All operands sit in shared memory in the un-swizzled canonical layout: 16-byte
// pieces (8 bf16) grouped into 128-byte core matrices of 8 pieces.  The natural memory order of
// every operand here has its 16-byte pieces running along the NON-contracted dimension or along the
// feature dimension, which gives:
//   X_B rows   piece (row i, feature chunk c) at ((i/8) * NC + c) * 128 + (i%8) * 16
//              - read as a K-major A operand by Z1 (rows = M, features = K), and
//              - read as an MN-major A operand by dW1 (features = M, rows = K): the SAME image
//   W1 (bf16)  piece (feature f, hidden chunk c) at ((f/8) * NHC + c) * 128 + (f%8) * 16   MN-major B (hidden = N)
//   dz1 (bf16) piece (row i, hidden chunk c)     at ((i/8) * NHC + c) * 128 + (i%8) * 16   MN-major B (hidden = N)
// W1 is rounded to bf16 and written in image order by mlp_prep_kernel, dz1 by mlp_f2_rows_kernel, so
// both arrive with one bulk copy; X_B rows are gathered with 16-byte async copies.
// Every wait is bounded and raises CADA_FLAG_TIMEOUT.
#pragma once
#include <cuda_bf16.h>
#include "common.cuh"
#include "grad_stream.cuh"   // mbarrier / bulk-copy helpers
#include "fused_small.cuh"   // cp.async helpers
#include "mlp.cuh"

namespace cada {

constexpr int TC_THREADS = 128;
constexpr int TC_KCHUNK = 112;            // features per pipeline stage of the Z1 product (7 MMA k-steps)
constexpr int TC_M = 128;                 // MMA M: minibatch rows (Z1) or features (dW1) per CTA

constexpr int MLP_F2_RB = 8;   // minibatch rows per CTA of mlp_f2_rows_kernel (a multiple of 8: whole row groups of the dz1 image)

struct MlpTcGeom {
  int nhc;              // hidden chunks of 8 after padding N to a multiple of 16
  int n;                // nhc * 8 = MMA N
  int n_kchunks;        // ceil(F / TC_KCHUNK)
  int bp;               // minibatch rows rounded up to a multiple of 16 (<= 128)
  int tmem_cols;        // power of two >= n
  unsigned w_chunk_bytes;   // bytes of one K-chunk of the W1 image: TC_KCHUNK * n * 2
  unsigned w_set_bytes;     // n_kchunks * w_chunk_bytes
  unsigned dz_bytes;        // dz1 image of one (worker, iterate): bp * n * 2
  int n_sets;           // W1 images: theta, then the old iterates (1 for CADA1, M for CADA2)
  int f2_blocks;        // ceil(B / MLP_F2_RB): CTAs of mlp_f2_rows_kernel per (worker, iterate)
  int small;            // H + H*C + C : floats of (b1, W2, b2) gradients
};

struct MlpTcBufs {
  unsigned char* w1_img;   // [n_sets][w_set_bytes]
  unsigned char* dz_img;   // [M][2][dz_bytes]
  float* small_part;       // [M][2][f2_blocks][small]
};

__host__ inline bool mlp_tc_plan(int F, int H, int C, int B, int M, int rule, long long ldx, MlpTcGeom& g) {
  if (F % 8 != 0 || ldx % 8 != 0 || H > 248 || B > 128 || C > 16 || H % 4 != 0) return false;
  g.nhc = (H + 15) / 16 * 2;
  g.n = g.nhc * 8;
  g.n_kchunks = (F + TC_KCHUNK - 1) / TC_KCHUNK;
  g.bp = (B + 15) / 16 * 16;
  g.tmem_cols = g.n <= 32 ? 32 : g.n <= 64 ? 64 : g.n <= 128 ? 128 : 256;
  g.w_chunk_bytes = (unsigned)TC_KCHUNK * g.n * 2;
  g.w_set_bytes = g.w_chunk_bytes * g.n_kchunks;
  g.dz_bytes = (unsigned)g.bp * g.n * 2;
  g.n_sets = 1 + (rule == 2 ? M : 1);
  g.f2_blocks = (B + MLP_F2_RB - 1) / MLP_F2_RB;
  g.small = H + H * C + C;
  return true;
}

namespace tc {
// Shared-memory matrix descriptor, no swizzle: start address, leading and stride byte offsets in 16-byte units.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// Instruction descriptor: fp32 accumulate, bf16 x bf16, majors, N >> 3 at bit 17, M >> 4 at bit 24.
__device__ __forceinline__ uint32_t instr_desc(int M, int N, bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn_major ? 1u << 15 : 0u) | (b_mn_major ? 1u << 16 : 0u) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}
__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, bool accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(da), "l"(db), "r"(idesc), "r"(accumulate ? 1u : 0u) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_free(uint32_t taddr, uint32_t cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// 16 consecutive fp32 columns of this thread's accumulator lane
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// Accumulator write-back through shared memory.  Each warp owns 32 accumulator lanes (= 32 output rows).  Columns are
// handled in panels of up to 112: the warp's lanes drop their 16-column pieces into a [32][116] staging tile (row pitch
// 116 floats = an odd number of 16-byte units, so the 128-bit writes of 8 lanes hit distinct banks), then the tile is
// written out row by row with consecutive lanes on consecutive 16-byte pieces.  `row_ok(r)` masks padding rows, `bias`
// (or nullptr) is added per column.  out_row0 points at row 0 of this warp; ld_out is the row pitch in floats (H).
constexpr int TC_PANEL = 112, TC_PANEL_PITCH = 116;
constexpr size_t TC_EPI_BYTES = (size_t)4 * 32 * TC_PANEL_PITCH * sizeof(float);     // 4 warps
template <class RowOk>
__device__ __forceinline__ void store_accumulators(uint32_t lane_base, float* stage /* this warp's tile */, int lane,
                                                   float* __restrict__ out_row0, int H, const float* __restrict__ bias,
                                                   RowOk row_ok) {
  for (int p0 = 0; p0 < H; p0 += TC_PANEL) {
    const int pw = min(TC_PANEL, H - p0), pw16 = (pw + 15) / 16 * 16;
    for (int n0 = 0; n0 < pw16; n0 += 16) {
      float v[16];
      tmem_ld16(lane_base + p0 + n0, v);
#pragma unroll
      for (int q = 0; q < 4; ++q)
        *reinterpret_cast<float4*>(stage + lane * TC_PANEL_PITCH + n0 + 4 * q) = make_float4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
    }
    __syncwarp();
    const int q4 = pw / 4;                          // whole 16-byte pieces per row (H is a multiple of 4 on this path or handled below)
    for (int idx = lane; idx < 32 * q4; idx += 32) {
      const int r = idx / q4, q = idx - r * q4;
      if (row_ok(r)) {
        float4 v = *reinterpret_cast<const float4*>(stage + r * TC_PANEL_PITCH + 4 * q);
        if (bias) { const float4 b = *reinterpret_cast<const float4*>(bias + p0 + 4 * q); v.x += b.x; v.y += b.y; v.z += b.z; v.w += b.w; }
        *reinterpret_cast<float4*>(out_row0 + (long long)r * H + p0 + 4 * q) = v;
      }
    }
    for (int idx = lane; idx < 32 * (pw - 4 * q4); idx += 32) {      // ragged tail columns (H % 4 != 0)
      const int r = idx / (pw - 4 * q4), c = 4 * q4 + idx - r * (pw - 4 * q4);
      if (row_ok(r)) out_row0[(long long)r * H + p0 + c] = stage[r * TC_PANEL_PITCH + c] + (bias ? bias[p0 + c] : 0.f);
    }
    __syncwarp();
  }
}
}  // namespace tc

// which W1 image belongs to (worker, iterate)
__device__ __forceinline__ int mlp_w_set(const Params& P, int m, int which) {
  return which == 0 ? 0 : (P.rule == 2 ? 1 + m : 1);
}

// Rounds W1 of every iterate in use to bf16 and writes it in image order.  grid (ceil(F/8), n_sets)
__global__ void __launch_bounds__(256) mlp_prep_kernel(const __grid_constant__ Params P, MlpTcGeom g, MlpTcBufs tb) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  const int fg = blockIdx.x, set = blockIdx.y;
  const long long k = P.st->k;
  const float* __restrict__ W1 = set == 0 ? P.theta : old_iterate(P, k, set - 1);     // CADA1: old_iterate ignores m
  const int F = P.F, H = P.H;
  // feature group fg (8 features) lives in K-chunk fg / 14 at local group fg % 14
  const int chunk = fg / (TC_KCHUNK / 8), lg = fg - chunk * (TC_KCHUNK / 8);
  unsigned char* img = tb.w1_img + (size_t)set * g.w_set_bytes + (size_t)chunk * g.w_chunk_bytes + (size_t)lg * g.nhc * 128;
  // one thread per (feature in group, hidden chunk): 16 bytes
  for (int o = threadIdx.x; o < 8 * g.nhc; o += blockDim.x) {
    const int hc = o >> 3, fr = o & 7, f = fg * 8 + fr;
    __align__(16) __nv_bfloat16 v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int h = hc * 8 + e;
      v[e] = __float2bfloat16_rn((f < F && h < H) ? W1[(long long)f * H + h] : 0.f);
    }
    *reinterpret_cast<uint4*>(img + (size_t)hc * 128 + fr * 16) = *reinterpret_cast<const uint4*>(v);
  }
}

// Z1 = X_B W1 + b1.  grid (M, 2).  Two-stage pipeline over K-chunks of 112 features.
__host__ __device__ inline size_t mlp_f1_tc_smem(const MlpTcGeom& g) {
  const size_t ops = 2 * ((size_t)TC_M * TC_KCHUNK * 2 + g.w_chunk_bytes);
  return (ops > tc::TC_EPI_BYTES ? ops : tc::TC_EPI_BYTES) + 256;
}

__global__ void __launch_bounds__(TC_THREADS, 1)
mlp_f1_tc_kernel(const __grid_constant__ Params P, const __grid_constant__ MlpTcGeom g, MlpBufs mb, MlpTcBufs tb) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  extern __shared__ __align__(128) unsigned char tcsm1[];
  constexpr unsigned A_BYTES = TC_M * TC_KCHUNK * 2;          // 28,672
  constexpr int NC = TC_KCHUNK / 8;                            // 14 feature chunks per stage
  const unsigned stage_bytes = A_BYTES + g.w_chunk_bytes;
  unsigned char* tail = tcsm1 + 2 * (size_t)stage_bytes;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(tail);   // [0..1] W landed, [2..3] MMAs of the stage done, [4] all done
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(tail + 64);
  __shared__ long long s_rowoff[TC_M];

  const int m = blockIdx.x, which = blockIdx.y, tid = threadIdx.x, warp = tid >> 5;
  const int F = P.F, H = P.H, B = P.B;
  const long long k = P.st->k;
  const __nv_bfloat16* __restrict__ X = static_cast<const __nv_bfloat16*>(P.X[m]);
  const unsigned char* __restrict__ wimg = tb.w1_img + (size_t)mlp_w_set(P, m, which) * g.w_set_bytes;
  const uint32_t bar0 = ptx::smem_u32(bars);

  s_rowoff[tid] = tid < B ? minibatch_row(P, k, m, tid, P.n_samples[m]) * P.ldx : -1;
  if (tid == 0) {
    for (int i = 0; i < 5; ++i) ptx::mbar_init(bar0 + 8 * i, 1);
    ptx::fence_barrier_init();
  }
  if (warp == 0) tc::tmem_alloc(ptx::smem_u32(s_tmem), (uint32_t)g.tmem_cols);
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = *s_tmem;

  auto load_stage = [&](int chunk, int buf) {
    unsigned char* a = tcsm1 + (size_t)buf * stage_bytes;
    unsigned char* b = a + A_BYTES;
    if (tid == 0) {
      ptx::mbar_expect_tx(bar0 + 8 * buf, g.w_chunk_bytes);
      ptx::bulk_g2s(ptx::smem_u32(b), wimg + (size_t)chunk * g.w_chunk_bytes, g.w_chunk_bytes, bar0 + 8 * buf);
      ptx::mbar_arrive(bar0 + 8 * buf);
    }
    // X pieces: thread = row, walks the 14 chunks of its row
    const long long off = s_rowoff[tid];
    unsigned char* dst = a + (size_t)(tid >> 3) * NC * 128 + (tid & 7) * 16;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
      const int f = chunk * TC_KCHUNK + c * 8;
      if (off >= 0 && f < F) cp_async16(dst + c * 128, X + off + f);
      else *reinterpret_cast<uint4*>(dst + c * 128) = make_uint4(0u, 0u, 0u, 0u);
    }
    cp_async_commit();
  };

  const uint32_t idesc = tc::instr_desc(TC_M, g.n, false, true);
  bool ok = true;
  load_stage(0, 0);
  for (int c = 0; c < g.n_kchunks && ok; ++c) {
    const int buf = c & 1;
    if (c + 1 < g.n_kchunks) {
      // the other stage is free once the MMAs that read it (chunk c-1) have completed
      if (c >= 1) ok = ptx::mbar_wait_bounded(bar0 + 8 * (2 + (buf ^ 1)), (uint32_t)(((c - 1) >> 1) & 1));
      if (ok) load_stage(c + 1, buf ^ 1);
      cp_async_wait<1>();
    } else {
      cp_async_wait<0>();
    }
    tc::fence_async_proxy();                      // my X pieces (generic proxy) -> visible to the tensor core
    if (ok) ok = ptx::mbar_wait_bounded(bar0 + 8 * buf, (uint32_t)((c >> 1) & 1));   // W chunk landed
    tc::fence_before_sync();
    __syncthreads();
    tc::fence_after_sync();
    if (tid == 0 && ok) {
      const uint32_t a0 = ptx::smem_u32(tcsm1 + (size_t)buf * stage_bytes), b0 = a0 + A_BYTES;
#pragma unroll
      for (int s = 0; s < TC_KCHUNK / 16; ++s) {
        const uint64_t da = tc::smem_desc(a0 + s * 256, 128, NC * 128);                       // K-major: LBO = next K chunk, SBO = next 8 rows
        const uint64_t db = tc::smem_desc(b0 + s * 2 * g.nhc * 128, g.nhc * 128, 128);        // MN-major: LBO = next 8 features, SBO = next 8 hidden
        tc::mma_bf16(tmem, da, db, idesc, c > 0 || s > 0);
      }
      tc::mma_commit(bar0 + 8 * (2 + buf));
      if (c + 1 == g.n_kchunks) tc::mma_commit(bar0 + 8 * 4);
    }
  }
  if (ok) ok = ptx::mbar_wait_bounded(bar0 + 8 * 4, 0);
  if (!ok && tid == 0) atomicOr(&P.st->status_flags, 4);
  __syncthreads();                 // nobody polls a barrier any more: shared memory may be reused for staging
  tc::fence_after_sync();
  // epilogue: accumulator lane = minibatch row; staged through the (now idle) operand buffers, written out coalesced
  if (ok) {
    const float* __restrict__ b1 = mlp_iterate(P, k, m, which) + (long long)F * H;
    float* __restrict__ out0 = mb.z1 + (((long long)m * 2 + which) * B + warp * 32) * H;
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
    float* stage = reinterpret_cast<float*>(tcsm1) + (size_t)warp * 32 * tc::TC_PANEL_PITCH;
    const int lane = tid & 31;
    const bool vec_ok = (H % 4 == 0);                    // rows of Z1 then start on 16-byte boundaries
    if (vec_ok) {
      tc::store_accumulators(lane_base, stage, lane, out0, H, b1, [&](int r) { return warp * 32 + r < B; });
    } else {
      for (int n0 = 0; n0 < H; n0 += 16) {
        float v[16];
        tc::tmem_ld16(lane_base + n0, v);
        if (tid < B) {
#pragma unroll
          for (int e = 0; e < 16; ++e) if (n0 + e < H) out0[(long long)lane * H + n0 + e] = v[e] + b1[n0 + e];
        }
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_free(tmem, (uint32_t)g.tmem_cols);
}

// Everything between the two large products for MLP_F2_RB minibatch rows of one (worker, iterate); writes dz1 in image order
// and the partial sums of the small gradients.  grid (f2_blocks, M, 2)
__host__ __device__ inline size_t mlp_f2_rows_smem(int H, int C) {
  return sizeof(float) * ((size_t)2 * MLP_F2_RB * (H + 1) + (size_t)H * C + 3 * MLP_F2_RB * (size_t)C + C) + 64;
}

__global__ void __launch_bounds__(MLP_THREADS)
mlp_f2_rows_kernel(const __grid_constant__ Params P, const __grid_constant__ MlpTcGeom g, MlpBufs mb, MlpTcBufs tb) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  extern __shared__ __align__(16) float sf[];
  constexpr int RB = MLP_F2_RB;
  const int rb = blockIdx.x, m = blockIdx.y, which = blockIdx.z, tid = threadIdx.x;
  const int F = P.F, H = P.H, C = P.C, B = P.B, hp = H + 1;
  float* s_a1 = sf;                              // [RB][hp]
  float* s_dz1 = s_a1 + (size_t)RB * hp;         // [RB][hp]
  float* s_w2 = s_dz1 + (size_t)RB * hp;         // [H][C] rounded
  float* s_z2 = s_w2 + (size_t)H * C;            // [RB][C]
  float* s_dz2 = s_z2 + RB * C;                  // [RB][C]
  float* s_dz2q = s_dz2 + RB * C;                // [RB][C]
  float* s_b2 = s_dz2q + RB * C;                 // [C]
  const long long k = P.st->k;
  const float* __restrict__ th = mlp_iterate(P, k, m, which);
  const float* __restrict__ W2 = th + (long long)F * H + H;
  const float* __restrict__ b2 = W2 + (long long)H * C;
  const int* __restrict__ ym = static_cast<const int*>(P.y[m]);
  const int i0 = rb * RB, nr = min(RB, B - i0);
  const float* __restrict__ z1 = mb.z1 + (((long long)m * 2 + which) * B + i0) * H;
  const float invB = 1.0f / (float)B;

  // W2 (rounded), b2 and this block's rows of z1 -> a1 (rounded) and the sign of z1; 128-bit loads, all independent
  for (int q = tid; q < (H * C + 3) / 4; q += MLP_THREADS) {
    const float4 v = reinterpret_cast<const float4*>(W2)[q];             // W2 starts at a multiple of 4 floats (H % 4 == 0)
    const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) if (4 * q + t < H * C) s_w2[4 * q + t] = bf16_round(e[t]);
  }
  for (int c = tid; c < C; c += MLP_THREADS) s_b2[c] = b2[c];
  const int hq = H / 4;
  for (int q = tid; q < RB * hq; q += MLP_THREADS) {
    const int i = q / hq, h = 4 * (q - i * hq);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < nr) v = *reinterpret_cast<const float4*>(z1 + (long long)i * H + h);
    const float e[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      s_a1[i * hp + h + t] = e[t] > 0.f ? bf16_round(e[t]) : 0.f;
      s_dz1[i * hp + h + t] = e[t] > 0.f ? 1.f : 0.f;
    }
  }
  __syncthreads();
  // z2 = a1 W2 + b2
  for (int o = tid; o < nr * C; o += MLP_THREADS) {
    const int i = o / C, c = o - i * C;
    float acc = 0.f;
#pragma unroll 8
    for (int h = 0; h < H; ++h) acc = fmaf(s_a1[i * hp + h], s_w2[h * C + c], acc);
    s_z2[i * C + c] = acc + s_b2[c];
  }
  __syncthreads();
  for (int i = tid; i < RB; i += MLP_THREADS) {
    if (i < nr) {
      const long long row = minibatch_row(P, k, m, i0 + i, P.n_samples[m]);
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
        mb.dz2[((((long long)m * 2 + which) * B) + i0 + i) * C + c] = d;
      }
    } else {
      for (int c = 0; c < C; ++c) { s_dz2[i * C + c] = 0.f; s_dz2q[i * C + c] = 0.f; }
    }
  }
  __syncthreads();
  // One thread per hidden unit h: dz1[:, h] = (dz2q W2q[h, :]^T) where z1 > 0, and in the same pass the partial sums
  // of db1[h] (unrounded dz1) and dW2[h, :] = a1q[:, h]^T dz2q over this block's rows, all in registers.
  float* __restrict__ sp = tb.small_part + (((size_t)m * 2 + which) * g.f2_blocks + rb) * g.small;   // [db1 (H) | dW2 (H*C) | db2 (C)]
  constexpr int CX = 16;
  for (int h = tid; h < H; h += MLP_THREADS) {
    float w2r[CX], dw2[CX];
#pragma unroll
    for (int c = 0; c < CX; ++c) { w2r[c] = c < C ? s_w2[h * C + c] : 0.f; dw2[c] = 0.f; }
    float db1 = 0.f;
#pragma unroll 4
    for (int i = 0; i < RB; ++i) {
      const float a = s_a1[i * hp + h];
      float da = 0.f;
#pragma unroll
      for (int c = 0; c < CX; ++c) {
        if (c < C) {
          const float dq = s_dz2q[i * C + c];
          da = fmaf(dq, w2r[c], da);
          dw2[c] = fmaf(a, dq, dw2[c]);
        }
      }
      const float d = s_dz1[i * hp + h] > 0.f ? da : 0.f;
      s_dz1[i * hp + h] = d;
      db1 += d;
    }
    sp[h] = db1;
#pragma unroll
    for (int c = 0; c < CX; ++c) if (c < C) sp[H + h * C + c] = dw2[c];
  }
  if (tid < C) {                                   // db2 (fp32, unrounded dz2)
    float a = 0.f;
    for (int i = 0; i < RB; ++i) a += s_dz2[i * C + tid];
    sp[H + H * C + tid] = a;
  }
  __syncthreads();
  // dz1 image: the block's rows are whole row groups of 8; piece (i, hidden chunk hc)
  unsigned char* img = tb.dz_img + ((size_t)m * 2 + which) * g.dz_bytes;
  float* __restrict__ dz1o = mb.dz1 + (((long long)m * 2 + which) * B) * H;        // the same values before rounding
  for (int o = tid; o < RB * g.nhc; o += MLP_THREADS) {
    const int i = o / g.nhc, hc = o - i * g.nhc, gi = i0 + i;
    __align__(16) __nv_bfloat16 v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int h = hc * 8 + e;
      const float d = h < H ? s_dz1[i * hp + h] : 0.f;
      v[e] = __float2bfloat16_rn(d);
      if (h < H && i < nr) dz1o[(long long)gi * H + h] = d;
    }
    *reinterpret_cast<uint4*>(img + ((size_t)(gi >> 3) * g.nhc + hc) * 128 + (gi & 7) * 16) = *reinterpret_cast<const uint4*>(v);
  }
}

// dW1 = X_B^T dz1 for one tile of 128 features.  grid (ceil(F/128), M, 2).  The feature-tile-0 CTA also folds the
// row-block partial sums of the small gradients (fixed order).
__host__ __device__ inline size_t mlp_b1_tc_smem(const MlpTcGeom& g) {
  const size_t ops = (size_t)(g.bp / 8) * 16 * 128 + g.dz_bytes;
  return (ops > tc::TC_EPI_BYTES ? ops : tc::TC_EPI_BYTES) + 256;
}

__global__ void __launch_bounds__(TC_THREADS)
mlp_b1_tc_kernel(const __grid_constant__ Params P, const __grid_constant__ MlpTcGeom g, MlpBufs mb, MlpTcBufs tb) {
  pdl_trigger();   // launched with programmatic serialisation: the next kernel may be scheduled,
  pdl_wait();      // and this one starts its work when the kernels before it have completed
  extern __shared__ __align__(128) unsigned char tcsm2[];
  const unsigned a_bytes = (unsigned)(g.bp / 8) * 16 * 128;
  unsigned char* s_a = tcsm2;                       // X sub-image: (row group, 16 feature chunks)
  unsigned char* s_b = tcsm2 + a_bytes;             // dz1 image
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(tcsm2 + a_bytes + g.dz_bytes);   // [0] dz landed, [1] MMAs done
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(bars + 4);
  const int ft = blockIdx.x, m = blockIdx.y, which = blockIdx.z, tid = threadIdx.x, warp = tid >> 5;
  const int F = P.F, H = P.H, B = P.B;
  const long long k = P.st->k;
  const __nv_bfloat16* __restrict__ X = static_cast<const __nv_bfloat16*>(P.X[m]);
  const uint32_t bar0 = ptx::smem_u32(bars);
  if (tid == 0) {
    ptx::mbar_init(bar0, 1);
    ptx::mbar_init(bar0 + 8, 1);
    ptx::fence_barrier_init();
  }
  if (warp == 0) tc::tmem_alloc(ptx::smem_u32(s_tmem), (uint32_t)g.tmem_cols);
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = *s_tmem;
  if (tid == 0) {
    ptx::mbar_expect_tx(bar0, g.dz_bytes);
    ptx::bulk_g2s(ptx::smem_u32(s_b), tb.dz_img + ((size_t)m * 2 + which) * g.dz_bytes, g.dz_bytes, bar0);
    ptx::mbar_arrive(bar0);
  }
  // X pieces: thread = minibatch row (rows >= B are zero), 16 feature chunks of this tile
  {
    const long long off = tid < B ? minibatch_row(P, k, m, tid, P.n_samples[m]) * P.ldx : -1;
    if (tid < g.bp) {
      unsigned char* dst = s_a + (size_t)(tid >> 3) * 16 * 128 + (tid & 7) * 16;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const int f = ft * TC_M + c * 8;
        if (off >= 0 && f < F) cp_async16(dst + c * 128, X + off + f);
        else *reinterpret_cast<uint4*>(dst + c * 128) = make_uint4(0u, 0u, 0u, 0u);
      }
    }
    cp_async_commit();
    cp_async_wait<0>();
    tc::fence_async_proxy();
  }
  bool ok = ptx::mbar_wait_bounded(bar0, 0);
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (tid == 0 && ok) {
    const uint32_t idesc = tc::instr_desc(TC_M, g.n, true, true);
    const uint32_t a0 = ptx::smem_u32(s_a), b0 = ptx::smem_u32(s_b);
    for (int s = 0; s < g.bp / 16; ++s) {
      const uint64_t da = tc::smem_desc(a0 + s * 2 * 16 * 128, 16 * 128, 128);          // MN-major: LBO = next 8 rows, SBO = next 8 features
      const uint64_t db = tc::smem_desc(b0 + s * 2 * g.nhc * 128, g.nhc * 128, 128);    // MN-major: LBO = next 8 rows, SBO = next 8 hidden
      tc::mma_bf16(tmem, da, db, idesc, s > 0);
    }
    tc::mma_commit(bar0 + 8);
  }
  // meanwhile: the small gradients (b1, W2, b2): every feature-tile CTA folds its share of the row-block partial sums,
  // row blocks in a fixed order
  float* __restrict__ gout = mlp_grad_out(P, m, which);
  {
    const float* __restrict__ sp = tb.small_part + (((size_t)m * 2 + which) * g.f2_blocks) * g.small;
    const int per = (g.small + gridDim.x - 1) / gridDim.x;
    const int o_end = min(g.small, (ft + 1) * per);
    for (int o = ft * per + tid; o < o_end; o += TC_THREADS) {
      float acc = 0.f;
#pragma unroll 8
      for (int r = 0; r < g.f2_blocks; ++r) acc += sp[(size_t)r * g.small + o];
      gout[(long long)F * H + o] = acc;            // layout of theta after W1: b1 (H) | W2 (H*C) | b2 (C)
    }
  }
  if (ok) ok = ptx::mbar_wait_bounded(bar0 + 8, 0);
  if (!ok && tid == 0) atomicOr(&P.st->status_flags, 4);
  __syncthreads();                 // nobody polls a barrier any more: shared memory may be reused for staging
  tc::fence_after_sync();
  if (ok) {
    // accumulator lane = feature of this tile; all MMAs are complete, so the operand images are free for staging
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);
    const int lane = tid & 31, f0 = ft * TC_M + warp * 32;
    float* __restrict__ out0 = gout + (long long)f0 * H;
    float* stage = reinterpret_cast<float*>(tcsm2) + (size_t)warp * 32 * tc::TC_PANEL_PITCH;
    if (H % 4 == 0) {
      tc::store_accumulators(lane_base, stage, lane, out0, H, nullptr, [&](int r) { return f0 + r < F; });
    } else {
      for (int n0 = 0; n0 < H; n0 += 16) {
        float v[16];
        tc::tmem_ld16(lane_base + n0, v);
        if (f0 + lane < F) {
#pragma unroll
          for (int e = 0; e < 16; ++e) if (n0 + e < H) out0[(long long)lane * H + n0 + e] = v[e];
        }
      }
    }
  }
  tc::fence_before_sync();
  __syncthreads();
  if (warp == 0) tc::tmem_free(tmem, (uint32_t)g.tmem_cols);
}

}  // namespace cada
