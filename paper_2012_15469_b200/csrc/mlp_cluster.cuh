// Two-point minibatch gradient of the 2-layer ReLU network AND the upload decision in ONE launch: a thread-block cluster
// per worker, CTA r of the cluster owning the features [112 r, 112 r + 112).
//
// Algorithm 1 asks every worker for two gradients on the SAME minibatch.  Here the sampled rows cross the memory system
// once per worker: CTA r gathers its 112-feature slice of the B rows into shared memory in the un-swizzled canonical
// layout (mlp_tc.cuh), and that one image is the A operand of both large products and of both iterates:
//
//   phase 1  partial Z1 = X_B[:, slice] W1[slice, :] for theta^k and for the old iterate, two tcgen05.mma streams with
//            the same A descriptor and different B images into 2 x 256 tensor-memory columns.  The bf16 images of W1 are
//            not re-rounded per iteration: the update kernel writes the image of theta^{k+1} into slot (k+1) mod (D+1) of
//            a ring, and the old iterate of a worker (theta^{k - tau_m}, CADA2) or the snapshot (CADA1) is found in the
//            slot of the iteration it was produced in.  The partial accumulators go to a scratch buffer [slice][column
//            group][row][4] (coalesced 16-byte stores straight from the accumulator lanes).
//   barrier  (cluster, release/acquire)
//   phase 2  CTA r takes ceil(B / n_slices) minibatch rows: adds the slices' partials in slice order, bias, ReLU, the
//            small output layer, softmax, dz2, dz1 and this CTA's share of the gradients of (b1, W2, b2); dz1 goes out
//            rounded to bf16 in operand-image order (and, unrounded, with z1 and dz2 into the buffers cada_read offers).
//   barrier
//   phase 3  dW1[slice, :] = X_B[:, slice]^T dz1 for both iterates from the SAME staged image (now read MN-major) and
//            the two dz1 images; the epilogue has g and g' of a coordinate side by side, so it writes g_m and
//            d_m = g_m - g'_m (regulariser included) to their final place and accumulates the left-hand side of Eq. 8 /
//            Eq. 6 / Eq. 4 in fp64 on the way: no partial slots, no trigger launch, no second pass over the gradients.
//   barrier  rank 0 adds the slices' left-hand-side parts in slice order and takes the decision (decide_upload).
// 512 threads: the phases between the products are chains of shared-memory and L2 latencies, so every loop below is laid
// out for many independent loads per thread (several items per trip, 128-bit shared-memory accesses) rather than for few
// instructions.
//
// The minibatch rows depend on the iteration number only, so the kernel takes k from the host and gathers them before it
// waits for the preceding update kernel (programmatic dependent launch).  Every mbarrier wait is bounded; a wait that
// runs out raises CADA_FLAG_TIMEOUT, and the CTA still walks through every cluster barrier (its work skipped) so that
// its peers are never left waiting, then frees its tensor memory.
#pragma once
#include "mlp_tc.cuh"
#include "fused_cluster.cuh"   // cluster barrier helpers

namespace cada {

constexpr int MC_THREADS = 512;
constexpr int MC_NCA = 16;                 // 16-byte feature chunks per 8-row group of the A image (14 used, 2 zero)
constexpr int MC_A_BYTES = 16 * MC_NCA * 128;      // 128 rows
constexpr int MC_RBLK = 20;                // most minibatch rows a CTA handles at a time in phase 2
constexpr int MC_MAX_SLICES = 8;

struct MlpClusterGeom {
  int ns;               // feature slices = CTAs per cluster
  int n_it;             // iterates evaluated: 2, or 1 for the stochastic-LAG rule
  int rp;               // minibatch rows per CTA in phase 2
  int rblk;             // ... taken this many at a time (<= MC_RBLK, as shared memory allows)
  int per_small;        // outputs of (b1, W2, b2) each CTA folds in phase 3
  int small4;           // pitch (floats) of one set of (db1 | dW2 | db2) sums: `small` rounded up to a multiple of 4
  int cp;               // classes rounded up to a multiple of 4 (pitch of the per-row class vectors in shared memory)
  int hk;               // bf16 pitch of a row of the a1 image in phase 2: H rounded up to 16, plus 8 (conflict-free 8 x 8 matrix loads)
  unsigned b_bytes;     // operand region: two W1 chunks (phase 1), phase-2 scratch, two dz1 images (phase 3)
  unsigned smem_bytes;
  size_t zpart_bytes;   // [M][n_it][ns][n/4][128][4] floats
  size_t small_bytes;   // [M][n_it][ns][small4] floats
};

struct MlpClusterBufs {
  float* zpart;
  float* small_part;
  double* lhs_part;     // [M][MC_MAX_SLICES]
};

__host__ inline size_t mlp_cluster_phase2_bytes(int H, int C, int n_it, int rblk) {
  const size_t pairs = (size_t)n_it * rblk, hp = (size_t)H + 4, cp = ((size_t)C + 3) / 4 * 4;
  const size_t small4 = ((size_t)H + (size_t)H * C + C + 3) / 4 * 4;
  const size_t h16 = ((size_t)H + 15) / 16 * 16, hk = h16 + 8;
  const size_t bf16_part = 2 * ((size_t)n_it * 32 * hk + (size_t)n_it * h16 * 24 + (size_t)n_it * 32 * 24);   // a1, W2, dz2 images
  return bf16_part + sizeof(float) * (pairs * hp + 2 * pairs * cp + (size_t)n_it * cp + (size_t)n_it * small4) + 64;
}
constexpr size_t MC_TILE_BYTES = (size_t)(MC_THREADS / 32) * 2 * 32 * 20 * sizeof(float);   // epilogue staging, aliases the operand region

__host__ inline bool mlp_cluster_plan(int F, int H, int C, int B, int M, int rule, const MlpTcGeom& tg, MlpClusterGeom& g) {
  g.ns = (F + TC_KCHUNK - 1) / TC_KCHUNK;
  if (g.ns < 1 || g.ns > MC_MAX_SLICES) return false;
  g.n_it = rule == 3 ? 1 : 2;
  g.rp = (B + g.ns - 1) / g.ns;
  g.per_small = (tg.small + g.ns - 1) / g.ns;
  size_t b = 0;
  for (g.rblk = g.rp < MC_RBLK ? g.rp : MC_RBLK; g.rblk >= 1; --g.rblk) {
    b = (size_t)2 * tg.w_chunk_bytes;
    if ((size_t)2 * tg.dz_bytes > b) b = (size_t)2 * tg.dz_bytes;
    const size_t p2 = mlp_cluster_phase2_bytes(H, C, g.n_it, g.rblk);
    if (p2 > b) b = p2;
    if (MC_TILE_BYTES > b) b = MC_TILE_BYTES;
    b = (b + 127) / 128 * 128;
    if (MC_A_BYTES + b + 512 <= 200 * 1024) break;
  }
  if (g.rblk < 1) return false;
  g.b_bytes = (unsigned)b;
  g.smem_bytes = (unsigned)(MC_A_BYTES + b + 512);
  g.small4 = (tg.small + 3) / 4 * 4;
  g.cp = (C + 3) / 4 * 4;
  g.hk = (H + 15) / 16 * 16 + 8;
  g.zpart_bytes = sizeof(float) * (size_t)M * g.n_it * g.ns * (size_t)(tg.n / 4) * 128 * 4;
  g.small_bytes = sizeof(float) * (size_t)M * g.n_it * g.ns * (size_t)((tg.small + 3) / 4 * 4);
  return g.smem_bytes <= 200 * 1024;
}

// x / d for 0 <= x < 2^22 and 1 <= d with inv = 1.0f / d: one multiply and a correction instead of an integer division
// (the loops between the tensor-core products are chains of latencies; a division by a run-time value is a long one).
__device__ __forceinline__ int div_small(int x, int d, float inv) {
  int q = (int)((float)x * inv);
  const int r = x - q * d;
  q += (r >= d) - (r < 0);
  return q;
}

// Ring slot that holds the bf16 image of the W1 block of (worker m, iterate `which`) at iteration k.
__device__ __forceinline__ int mlp_ring_slot(const Params& P, long long k, int m, int which) {
  long long j = k;
  if (which == 1) {
    if (P.rule == 2) { j = k - (long long)P.tau[m]; if (j < 0) j = 0; }     // theta^{k - tau_m}; before k = 0 every iterate is theta^0
    else if (P.rule == 1) j = k - k % P.D;                                    // the snapshot taken at the last multiple of D
  }
  return (int)(j % P.w1_slots);
}

// 4 consecutive hidden units of one W1 row, rounded to bf16, at their place in ring slot `slot` (H % 4 == 0).
__device__ __forceinline__ void mlp_ring_store4(const Params& P, int slot, long long q /* f * H + h, h % 4 == 0 */, float4 v) {
  const int H = P.H;
  const int f = (int)q / H, h = (int)q - f * H;                       // F * H < 2^31
  unsigned char* dst = P.w1_ring + (size_t)slot * P.w1_set_bytes;
  if (P.w1_hsplit) {                                                  // [hidden slice of 32][feature group of 8][4 hidden chunks][8 features x 16 B]
    const int hl = h & 31;
    dst += (size_t)(h >> 5) * P.w1_chunk_bytes + ((size_t)(f >> 3) * 4 + (hl >> 3)) * 128 + (f & 7) * 16 + (hl & 7) * 2;
  } else {                                                            // [112-feature chunk][feature group of 8][hidden chunk][8 features x 16 B]
    const int chunk = f / TC_KCHUNK, lf = f - chunk * TC_KCHUNK;
    dst += (size_t)chunk * P.w1_chunk_bytes + ((size_t)(lf >> 3) * P.w1_nhc + (h >> 3)) * 128 + (lf & 7) * 16 + (h & 7) * 2;
  }
  __align__(8) __nv_bfloat16 b[4] = {__float2bfloat16_rn(v.x), __float2bfloat16_rn(v.y), __float2bfloat16_rn(v.z), __float2bfloat16_rn(v.w)};
  *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(b);
}

// (Re)builds the ring slots the next iteration reads from the fp32 iterates: theta^k, and the old iterate of every
// worker (CADA2) or the snapshot (CADA1).  Runs at create and after state has been written from the host.
// grid (ceil(F*H/4 / 256), n_sets); set 0 = theta, set s >= 1 = worker s-1 / the snapshot.
__global__ void __launch_bounds__(256) mlp_ring_rebuild_kernel(const __grid_constant__ Params P, long long k) {
  const int set = blockIdx.y;
  const float* src = P.theta;
  int slot = (int)(k % P.w1_slots);
  if (set >= 1) {
    if (P.rule == 1 && k % P.D == 0) return;          // the snapshot is theta^k itself on these iterations
    src = old_iterate(P, k, set - 1);
    slot = mlp_ring_slot(P, k, set - 1, 1);
  }
  const long long q = ((long long)blockIdx.x * 256 + threadIdx.x) * 4;
  if (q < (long long)P.F * P.H) mlp_ring_store4(P, slot, q, *reinterpret_cast<const float4*>(src + q));
}

namespace mm {
// Warp-level tensor-core helpers for the small products of phase 2 (bf16 x bf16 -> fp32, m16n8k16).  Each lane passes
// the address of one 16-byte row of an 8 x 8 bf16 matrix: lanes 0-7 the rows of matrix 0, 8-15 of matrix 1, and so on.
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(ptx::smem_u32(p)) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(ptx::smem_u32(p)) : "memory");
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t (&r)[2], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(ptx::smem_u32(p)) : "memory");
}
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t (&r)[2], const void* p) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(ptx::smem_u32(p)) : "memory");
}
// d += a (16 x 16, row-major fragment) * b (16 x 8, column-major fragment)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}
}  // namespace mm

namespace tc {
// 16 accumulator columns without waiting for them: pair with tmem_ld_wait16 before the first use
__device__ __forceinline__ void tmem_ld16_issue(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr) : "memory");
}
// waits for every tcgen05.ld of this thread; the registers are operands so that no use of them is scheduled ahead of the wait
__device__ __forceinline__ void tmem_ld_wait16(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :: "memory");
}
}  // namespace tc

__global__ void __launch_bounds__(MC_THREADS, 1)
mlp_cluster_kernel(const __grid_constant__ Params P, const __grid_constant__ MlpTcGeom g, const __grid_constant__ MlpClusterGeom cg,
                   MlpBufs mb, MlpTcBufs tb, MlpClusterBufs cb, long long k /* iteration, as the host counts it */) {
  extern __shared__ __align__(128) unsigned char mcsm[];
  unsigned char* s_a = mcsm;                                   // A image: [16 row groups][16 chunks][8 rows x 16 B]
  unsigned char* s_b = mcsm + MC_A_BYTES;                      // operand region (see MlpClusterGeom::b_bytes)
  unsigned char* tail = s_b + cg.b_bytes;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(tail);      // [0] W landed, [1] Z1 MMAs done, [2] dz1 landed, [3] dW1 MMAs done
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(tail + 64);
  int* s_ok = reinterpret_cast<int*>(tail + 72);
  double* s_red = reinterpret_cast<double*>(tail + 128);       // [16]
  __shared__ long long s_rowoff[TC_M];
  __shared__ int s_label[TC_M];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qd = warp & 3, part = warp >> 2;                    // accumulator lane quarter this warp may read; its share of the columns
  const int m = blockIdx.y;
  unsigned rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int r = (int)rank, ns = cg.ns, n_it = cg.n_it;
  const int F = P.F, H = P.H, C = P.C, B = P.B, n = g.n, nhc = g.nhc;
  const long long FH = (long long)F * H;
  const __nv_bfloat16* __restrict__ X = static_cast<const __nv_bfloat16*>(P.X[m]);
  const uint32_t bar0 = ptx::smem_u32(bars);
  const uint32_t a0 = ptx::smem_u32(s_a), b0 = ptx::smem_u32(s_b);

  pdl_trigger();                                                // the update kernel may be scheduled behind this one
  if (P.idx_mode == IDX_EXPLICIT) pdl_wait();                   // explicit indices may have been produced on this stream just before
  if (tid < TC_M) s_rowoff[tid] = tid < B ? minibatch_row(P, k, m, tid, P.n_samples[m]) : -1;
  if (tid == 0) {
    for (int i = 0; i < 4; ++i) ptx::mbar_init(bar0 + 8 * i, 1);
    ptx::fence_barrier_init();
    *s_ok = 1;
  }
  if (warp == 0) tc::tmem_alloc(ptx::smem_u32(s_tmem), 512u);
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = *s_tmem;
  const uint32_t my_lanes = tmem + ((uint32_t)(qd * 32) << 16);

  // ---- gather: 16-byte pieces (row i, chunk c) of this slice; rows >= B, features >= F and chunks 14, 15 are zero ----
  for (int o = tid; o < TC_M * MC_NCA; o += MC_THREADS) {
    const int i = o >> 4, c = o & 15;
    unsigned char* dst = s_a + ((size_t)(i >> 3) * MC_NCA + c) * 128 + (i & 7) * 16;
    const long long off = s_rowoff[i];
    const int f = r * TC_KCHUNK + c * 8;
    if (off >= 0 && c < TC_KCHUNK / 8 && f < F) cp_async16(dst, X + off * P.ldx + f);
    else *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
  }
  cp_async_commit();
  if (tid < B) s_label[tid] = static_cast<const int*>(P.y[m])[s_rowoff[tid]];

  pdl_wait();                                                   // iterates, their images and the staleness belong to earlier kernels until now
  double* s_rhs = reinterpret_cast<double*>(tail + 256);       // this iteration's right-hand side (rank 0)
  if (r == 0 && warp == 1) {                                    // the newest window term, if the update kernel left it in parts; then the right-hand side
    const double rhs = window_refresh_rhs(P, k, lane);
    if (lane == 0) *s_rhs = rhs;
  }
  bool ok = true;
  const float* __restrict__ th = P.theta;
  const float* __restrict__ tho = old_iterate(P, k, m);

  // ---- phase 1: partial Z1 of this slice for every iterate ------------------------------------------------------
  if (tid == 0) {
    ptx::mbar_expect_tx(bar0, (uint32_t)n_it * g.w_chunk_bytes);
    for (int it = 0; it < n_it; ++it) {
      const unsigned char* src = P.w1_ring + (size_t)mlp_ring_slot(P, k, m, it) * P.w1_set_bytes + (size_t)r * g.w_chunk_bytes;
      ptx::bulk_g2s(b0 + it * g.w_chunk_bytes, src, g.w_chunk_bytes, bar0);
    }
    ptx::mbar_arrive(bar0);
  }
  cp_async_wait<0>();
  tc::fence_async_proxy();                                      // gathered pieces (generic proxy) -> visible to the tensor core
  ok = ptx::mbar_wait_bounded(bar0, 0);
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (tid == 0) {
    if (ok) {
      const uint32_t idesc = tc::instr_desc(TC_M, n, false, true);
      for (int it = 0; it < n_it; ++it) {
#pragma unroll
        for (int s = 0; s < TC_KCHUNK / 16; ++s) {
          const uint64_t da = tc::smem_desc(a0 + s * 256, 128, MC_NCA * 128);                                   // K-major: LBO = next 8 features, SBO = next 8 rows
          const uint64_t db = tc::smem_desc(b0 + it * g.w_chunk_bytes + s * 2 * nhc * 128, nhc * 128, 128);    // MN-major: LBO = next 8 features, SBO = next 8 hidden
          tc::mma_bf16(tmem + it * 256, da, db, idesc, s > 0);
        }
      }
    }
    tc::mma_commit(bar0 + 8);
  }
  if (!ptx::mbar_wait_bounded(bar0 + 8, 0)) ok = false;
  tc::fence_after_sync();
  // accumulator lane = minibatch row; the four warps of a lane quarter share the (iterate, 16-column block) list, two
  // blocks per trip so that two tensor-memory loads are in flight
  if (ok) {
    const int nb = n / 16, total = n_it * nb, row = qd * 32 + lane;
    for (int u = part; u < total; u += 8) {
      const int u2 = u + 4;
      const bool two = u2 < total;                              // warp-uniform
      const int it = u / nb, cbk = u - it * nb, it2 = two ? u2 / nb : 0, cbk2 = two ? u2 - it2 * nb : 0;
      uint32_t v[16], v2[16];
      tc::tmem_ld16_issue(my_lanes + it * 256 + cbk * 16, v);
      if (two) tc::tmem_ld16_issue(my_lanes + it2 * 256 + cbk2 * 16, v2);
      tc::tmem_ld_wait16(v);
      if (two) tc::tmem_ld_wait16(v2);
      float4* dst = reinterpret_cast<float4*>(cb.zpart) + ((((size_t)m * n_it + it) * ns + r) * (size_t)(n / 4) + cbk * 4) * 128 + row;
#pragma unroll
      for (int j = 0; j < 4; ++j)
        dst[(size_t)j * 128] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
      if (two) {
        float4* dst2 = reinterpret_cast<float4*>(cb.zpart) + ((((size_t)m * n_it + it2) * ns + r) * (size_t)(n / 4) + cbk2 * 4) * 128 + row;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          dst2[(size_t)j * 128] = make_float4(__uint_as_float(v2[4 * j]), __uint_as_float(v2[4 * j + 1]), __uint_as_float(v2[4 * j + 2]), __uint_as_float(v2[4 * j + 3]));
      }
    }
  }
  if (!ok) *s_ok = 0;
  tc::fence_before_sync();
  fc_cluster_arrive();
  fc_cluster_wait();                                            // every slice's partials are visible to the cluster
  tc::fence_after_sync();

  // ---- phase 2: this CTA's rows through the small layers --------------------------------------------------------
  // The three small products (z2 = a1 W2, dz1 = dz2 W2^T, dW2 = a1^T dz2) have bf16 operands by the rounding contract, so
  // they run as warp-level mma.sync (m16n8k16, fp32 accumulation) on operands kept in shared memory as bf16: with plain
  // FMAs the phase was bound by shared-memory bandwidth (every FMA fetched its operands again).
  {
    const int cp = cg.cp, small4 = cg.small4, RB = cg.rblk, hq = H / 4;
    const int hk = cg.hk, hp = H + 4;                            // bf16 row pitch of the a1 image; fp32 row pitch of dz1
    const int h16 = (H + 15) / 16 * 16;
    const float inv_hq = 1.0f / (float)hq, inv_nhc = 1.0f / (float)nhc;
    constexpr int RP = 32, NP = 24;                             // rows of an iterate's tile pair; bf16 pitch of class vectors
    unsigned char* pb = s_b;
    __nv_bfloat16* s_a1 = reinterpret_cast<__nv_bfloat16*>(pb);  pb += (size_t)n_it * RP * hk * 2;     // [n_it][32][hk]  a1 rounded (0 where z1 <= 0, beyond the rows and beyond H)
    __nv_bfloat16* s_w2 = reinterpret_cast<__nv_bfloat16*>(pb);  pb += (size_t)n_it * h16 * NP * 2;    // [n_it][h16][24] W2 rounded, zero padding
    __nv_bfloat16* s_dq = reinterpret_cast<__nv_bfloat16*>(pb);  pb += (size_t)n_it * RP * NP * 2;     // [n_it][32][24]  dz2 rounded, zero padding
    float* s_dz1 = reinterpret_cast<float*>(pb);                 pb += (size_t)n_it * RB * hp * 4;     // [n_it * RB][hp] dz1 (fp32)
    float* s_z2 = reinterpret_cast<float*>(pb);                  pb += (size_t)n_it * RB * cp * 4;     // [pairs][cp]
    float* s_dz2 = reinterpret_cast<float*>(pb);                 pb += (size_t)n_it * RB * cp * 4;     // [pairs][cp] unrounded
    float* s_b2 = reinterpret_cast<float*>(pb);                  pb += (size_t)n_it * cp * 4;          // [n_it][cp]
    float* s_small = reinterpret_cast<float*>(pb);                                                      // [n_it][small4] this CTA's sums of (db1 | dW2 | db2)
    const float invB = 1.0f / (float)B;
    for (int o = tid; o < n_it * h16 * NP; o += MC_THREADS) {
      const int it = o >= h16 * NP ? 1 : 0, e = o - it * h16 * NP, h = e / NP, c = e - h * NP;
      s_w2[o] = __float2bfloat16_rn((h < H && c < C) ? (it ? tho : th)[FH + H + (long long)h * C + c] : 0.f);
    }
    for (int o = tid; o < n_it * cp; o += MC_THREADS) {
      const int it = o >= cp ? 1 : 0, c = o - it * cp;
      s_b2[o] = c < C ? (it ? tho : th)[FH + H + (long long)H * C + c] : 0.f;
    }
    for (int o = tid; o < n_it * small4; o += MC_THREADS) s_small[o] = 0.f;
    const int i_begin = r * cg.rp, i_end = min(B, i_begin + cg.rp);
    const size_t slice_stride = (size_t)(n / 4) * 128;          // float4 elements between the partials of consecutive slices
    const int g8 = lane >> 2, t4 = lane & 3;                    // fragment coordinates of this lane
    for (int ib = i_begin; ib < i_end; ib += RB) {
      const int nr = min(RB, i_end - ib), pairs = n_it * nr;
      const int m_tiles = (nr + 15) / 16;                       // 16-row tiles per iterate (1 or 2)
      const float inv_nr = 1.0f / (float)nr;
      __syncthreads();
      // zero the a1 and dz2 images (rows beyond nr, columns beyond H / C must read as zero)
      for (int o = tid; o < n_it * RP * hk / 2; o += MC_THREADS) reinterpret_cast<uint32_t*>(s_a1)[o] = 0u;
      for (int o = tid; o < n_it * RP * NP / 2; o += MC_THREADS) reinterpret_cast<uint32_t*>(s_dq)[o] = 0u;
      __syncthreads();
      // z1 = b1 + sum over slices (slice order); a1 = relu(z1) rounded.  Consecutive threads take consecutive rows; two
      // items per trip keep 2 * n_slices loads in flight
      {
        const int n_items = n_it * hq * nr;
        for (int o = tid; o < n_items; o += 2 * MC_THREADS) {
          const int o2 = o + MC_THREADS;
          const bool two = o2 < n_items;
          int il[2], q4[2], it[2];
          float4 acc[2], pz[2][MC_MAX_SLICES];
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            const int oo = t == 0 ? o : (two ? o2 : o);
            const int tq = div_small(oo, nr, inv_nr);
            il[t] = oo - tq * nr;
            it[t] = tq >= hq ? 1 : 0;
            q4[t] = tq - it[t] * hq;
            acc[t] = *reinterpret_cast<const float4*>((it[t] ? tho : th) + FH + 4 * q4[t]);
            const float4* src = reinterpret_cast<const float4*>(cb.zpart) + ((((size_t)m * n_it + it[t]) * ns) * (size_t)(n / 4) + q4[t]) * 128 + ib + il[t];
#pragma unroll
            for (int sl = 0; sl < MC_MAX_SLICES; ++sl)
              if (sl < ns) pz[t][sl] = __ldcg(src + (size_t)sl * slice_stride);
          }
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            if (t == 1 && !two) break;
#pragma unroll
            for (int sl = 0; sl < MC_MAX_SLICES; ++sl)
              if (sl < ns) { acc[t].x += pz[t][sl].x; acc[t].y += pz[t][sl].y; acc[t].z += pz[t][sl].z; acc[t].w += pz[t][sl].w; }
            const float4 z = acc[t];
            *reinterpret_cast<float4*>(mb.z1 + (((long long)m * 2 + it[t]) * B + ib + il[t]) * H + 4 * q4[t]) = z;
            __align__(8) __nv_bfloat16 a4[4] = {__float2bfloat16_rn(fmaxf(z.x, 0.f)), __float2bfloat16_rn(fmaxf(z.y, 0.f)),
                                                __float2bfloat16_rn(fmaxf(z.z, 0.f)), __float2bfloat16_rn(fmaxf(z.w, 0.f))};
            *reinterpret_cast<uint2*>(s_a1 + ((size_t)it[t] * RP + il[t]) * hk + 4 * q4[t]) = *reinterpret_cast<const uint2*>(a4);
          }
        }
      }
      __syncthreads();
      // z2 = a1 W2 + b2: one warp per (iterate, 16-row tile, 8-class tile), the hidden units 16 at a time
      for (int u = warp; u < n_it * m_tiles * 2; u += MC_THREADS / 32) {
        const int nt = u & 1, mt = (u >> 1) % m_tiles, it = (u >> 1) / m_tiles;
        if (nt * 8 >= C) continue;
        float d[4] = {0.f, 0.f, 0.f, 0.f};
        const __nv_bfloat16* a_base = s_a1 + ((size_t)it * RP + mt * 16 + (lane & 15)) * hk + (lane >> 4) * 8;
        const __nv_bfloat16* b_base = s_w2 + ((size_t)it * h16 + (lane & 15)) * NP + nt * 8;
        for (int k0 = 0; k0 < h16; k0 += 16) {
          uint32_t a[4], bq[2];
          mm::ldmatrix_x4(a, a_base + k0);
          mm::ldmatrix_x2_trans(bq, b_base + (size_t)k0 * NP);
          mm::mma_bf16_16816(d, a, bq);
        }
        const int row0 = mt * 16 + g8, col = nt * 8 + 2 * t4;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int il = row0 + 8 * hh;
          if (il < nr) {
            if (col < C) s_z2[(it * RB + il) * cp + col] = d[2 * hh] + s_b2[it * cp + col];
            if (col + 1 < C) s_z2[(it * RB + il) * cp + col + 1] = d[2 * hh + 1] + s_b2[it * cp + col + 1];
          }
        }
      }
      __syncthreads();
      // softmax and dz2 = (P - onehot) / B: sixteen lanes per (row, iterate), one class each
      for (int base = 0; base < pairs * 16; base += MC_THREADS) {
        const int item = base + tid, c = item & 15, pr = item >> 4;
        const bool valid = pr < pairs && c < C;
        int it = 0, il = 0;
        if (pr < pairs) { it = pr >= nr ? 1 : 0; il = pr - it * nr; }
        const int rowi = (it * RB + il) * cp;
        const float z = valid ? s_z2[rowi + c] : -INFINITY;
        float mx = z;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float e = valid ? expf(z - mx) : 0.f;
        float den = e;
#pragma unroll
        for (int o = 8; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
        if (valid) {
          const float dv = (e * (1.f / den) - (c == s_label[ib + il] ? 1.f : 0.f)) * invB;
          s_dz2[rowi + c] = dv;
          s_dq[((size_t)it * RP + il) * NP + c] = __float2bfloat16_rn(dv);
          mb.dz2[(((long long)m * 2 + it) * B + ib + il) * C + c] = dv;
        }
      }
      __syncthreads();
      // dz1 = (dz2q W2q^T) where z1 > 0: one warp per (iterate, 16-row tile, 8 hidden units), the classes in one step
      {
        const int n_ht = (H + 7) / 8;
        for (int u = warp; u < n_it * m_tiles * n_ht; u += MC_THREADS / 32) {
          const int ht = u % n_ht, mt = (u / n_ht) % m_tiles, it = u / (n_ht * m_tiles);
          uint32_t a[4], bq[2];
          float d[4] = {0.f, 0.f, 0.f, 0.f};
          mm::ldmatrix_x4(a, s_dq + ((size_t)it * RP + mt * 16 + (lane & 15)) * NP + (lane >> 4) * 8);
          mm::ldmatrix_x2(bq, s_w2 + ((size_t)it * h16 + ht * 8 + (lane & 7)) * NP + ((lane >> 3) & 1) * 8);
          mm::mma_bf16_16816(d, a, bq);
          const int row0 = mt * 16 + g8, h = ht * 8 + 2 * t4;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const int il = row0 + 8 * hh;
            if (il < nr && h < H) {
              const __nv_bfloat162 a2 = *reinterpret_cast<const __nv_bfloat162*>(s_a1 + ((size_t)it * RP + il) * hk + h);
              const float2 av = __bfloat1622float2(a2);
              *reinterpret_cast<float2*>(s_dz1 + (size_t)(it * RB + il) * hp + h) =
                  make_float2(av.x > 0.f ? d[2 * hh] : 0.f, av.y > 0.f ? d[2 * hh + 1] : 0.f);
            }
          }
        }
      }
      // dW2 += a1q^T dz2q: one warp per (iterate, 16 hidden units, 8 classes), the rows 16 at a time
      {
        const int n_mt = h16 / 16;
        for (int u = warp; u < n_it * n_mt * 2; u += MC_THREADS / 32) {
          const int nt = u & 1, ht = (u >> 1) % n_mt, it = (u >> 1) / n_mt;
          if (nt * 8 >= C) continue;
          float d[4] = {0.f, 0.f, 0.f, 0.f};
          for (int k0 = 0; k0 < m_tiles * 16; k0 += 16) {
            uint32_t a[4], bq[2];
            // A = a1q^T (hidden x rows) read from the row-major image with transposing loads
            mm::ldmatrix_x4_trans(a, s_a1 + ((size_t)it * RP + k0 + (lane & 7) + ((lane >> 4) & 1) * 8) * hk + ht * 16 + ((lane >> 3) & 1) * 8);
            mm::ldmatrix_x2_trans(bq, s_dq + ((size_t)it * RP + k0 + (lane & 15)) * NP + nt * 8);
            mm::mma_bf16_16816(d, a, bq);
          }
          float* ss = s_small + (size_t)it * small4 + H;
          const int h0 = ht * 16 + g8, col = nt * 8 + 2 * t4;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            const int h = h0 + 8 * hh;
            if (h < H) {
              if (col < C) ss[h * C + col] += d[2 * hh];
              if (col + 1 < C) ss[h * C + col + 1] += d[2 * hh + 1];
            }
          }
        }
      }
      for (int o = tid; o < n_it * C; o += MC_THREADS) {        // db2 (fp32, unrounded dz2)
        const int it = o >= C ? 1 : 0, c = o - it * C;
        float a = 0.f;
        for (int il = 0; il < nr; ++il) a += s_dz2[(it * RB + il) * cp + c];
        s_small[(size_t)it * small4 + H + H * C + c] += a;
      }
      __syncthreads();
      // db1 (fp32, unrounded dz1), one thread per (iterate, hidden unit)
      for (int u = tid; u < n_it * H; u += MC_THREADS) {
        const int it = u >= H ? 1 : 0, h = u - it * H;
        float a = 0.f;
        for (int il = 0; il < nr; ++il) a += s_dz1[(size_t)(it * RB + il) * hp + h];
        s_small[(size_t)it * small4 + h] += a;
      }
      // dz1: operand image (bf16) and the unrounded values
      for (int o = tid; o < pairs * nhc; o += MC_THREADS) {
        const int pr = div_small(o, nhc, inv_nhc), hc = o - pr * nhc, it = pr >= nr ? 1 : 0, il = pr - it * nr, i = ib + il;
        const float* d1 = s_dz1 + (size_t)(it * RB + il) * hp + hc * 8;
        float e[8];
        if (hc * 8 + 8 <= H) {
          const float4 lo = *reinterpret_cast<const float4*>(d1), hi = *reinterpret_cast<const float4*>(d1 + 4);
          e[0] = lo.x; e[1] = lo.y; e[2] = lo.z; e[3] = lo.w; e[4] = hi.x; e[5] = hi.y; e[6] = hi.z; e[7] = hi.w;
        } else {
#pragma unroll
          for (int t = 0; t < 8; ++t) e[t] = hc * 8 + t < H ? d1[t] : 0.f;
        }
        __align__(16) __nv_bfloat16 v[8];
#pragma unroll
        for (int t = 0; t < 8; ++t) v[t] = __float2bfloat16_rn(e[t]);
        unsigned char* img = tb.dz_img + ((size_t)m * 2 + it) * g.dz_bytes;
        *reinterpret_cast<uint4*>(img + ((size_t)(i >> 3) * nhc + hc) * 128 + (i & 7) * 16) = *reinterpret_cast<const uint4*>(v);
      }
      for (int o = tid; o < pairs * hq; o += MC_THREADS) {
        const int pr = div_small(o, hq, inv_hq), q4 = o - pr * hq, it = pr >= nr ? 1 : 0, il = pr - it * nr, i = ib + il;
        *reinterpret_cast<float4*>(mb.dz1 + (((long long)m * 2 + it) * B + i) * H + 4 * q4) =
            *reinterpret_cast<const float4*>(s_dz1 + (size_t)(it * RB + il) * hp + 4 * q4);
      }
    }
    __syncthreads();
    for (int o = tid; o < n_it * (small4 / 4); o += MC_THREADS) {
      const int it = o >= small4 / 4 ? 1 : 0, e4 = o - it * (small4 / 4);
      reinterpret_cast<float4*>(cb.small_part + (((size_t)m * n_it + it) * ns + r) * small4)[e4] =
          reinterpret_cast<const float4*>(s_small + (size_t)it * small4)[e4];
    }
  }
  // generic-proxy writes (this CTA's scratch in the operand region, the dz1 images in global memory) are ordered before the
  // bulk copies that follow the barrier
  asm volatile("fence.proxy.async;" ::: "memory");
  fc_cluster_arrive();
  fc_cluster_wait();                                            // dz1 images and the small partial sums are complete

  // ---- phase 3: dW1 of this slice for every iterate, then g_m, d_m and the left-hand side --------------------------
  ok = *s_ok != 0;
  if (tid == 0) {
    ptx::mbar_expect_tx(bar0 + 16, (uint32_t)n_it * g.dz_bytes);
    for (int it = 0; it < n_it; ++it)
      ptx::bulk_g2s(b0 + it * g.dz_bytes, tb.dz_img + ((size_t)m * 2 + it) * g.dz_bytes, g.dz_bytes, bar0 + 16);
    ptx::mbar_arrive(bar0 + 16);
  }
  if (!ptx::mbar_wait_bounded(bar0 + 16, 0)) ok = false;
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  if (tid == 0) {
    if (ok && *s_ok) {
      const uint32_t idesc = tc::instr_desc(TC_M, n, true, true);
      for (int it = 0; it < n_it; ++it) {
        for (int s = 0; s < g.bp / 16; ++s) {
          const uint64_t da = tc::smem_desc(a0 + s * 2 * MC_NCA * 128, MC_NCA * 128, 128);                     // MN-major: LBO = next 8 rows, SBO = next 8 features
          const uint64_t db = tc::smem_desc(b0 + it * g.dz_bytes + s * 2 * nhc * 128, nhc * 128, 128);         // MN-major: LBO = next 8 rows, SBO = next 8 hidden
          tc::mma_bf16(tmem + it * 256, da, db, idesc, s > 0);
        }
      }
    }
    tc::mma_commit(bar0 + 24);
  }
  if (!ptx::mbar_wait_bounded(bar0 + 24, 0)) ok = false;
  if (!ok) *s_ok = 0;
  __syncthreads();                                              // the products are complete: the operand region is free for staging
  tc::fence_after_sync();
  ok = *s_ok != 0;

  double acc = 0.0;
  const bool cada1 = P.rule == 1, lag = P.rule == 3;
  const float lambda = P.lambda;
  const float* __restrict__ ref = cada1 ? P.delta_stored + (long long)m * P.ldp : lag ? P.G + (long long)m * P.ldp : nullptr;
  float* __restrict__ gf = P.g_fresh + (long long)m * P.ldp;
  float* __restrict__ df = P.d_fresh + (long long)m * P.ldp;
  if (ok) {
    // accumulator lane = feature of the slice; the four warps of a lane quarter share the 16-column blocks.  Each warp
    // stages a block of g and of g - g' ([32][20] floats each) and writes them out with four lanes per 64-byte row piece
    const int nb = (H + 15) / 16;
    float* tg_ = reinterpret_cast<float*>(s_b) + (size_t)warp * 2 * 32 * 20;
    float* td_ = tg_ + 32 * 20;
    const int f_base = r * TC_KCHUNK + qd * 32;                  // feature of lane 0 of this warp
    for (int cbk = part; cbk < nb; cbk += 4) {
      uint32_t v0[16], v1[16];
      tc::tmem_ld16_issue(my_lanes + cbk * 16, v0);
      if (n_it == 2) tc::tmem_ld16_issue(my_lanes + 256 + cbk * 16, v1);
      tc::tmem_ld_wait16(v0);
      if (n_it == 2) {
        tc::tmem_ld_wait16(v1);
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) v1[e] = v0[e];               // one gradient only: the difference is identically 0
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float g0 = __uint_as_float(v0[4 * j]), g1 = __uint_as_float(v0[4 * j + 1]), g2 = __uint_as_float(v0[4 * j + 2]),
                    g3 = __uint_as_float(v0[4 * j + 3]);
        *reinterpret_cast<float4*>(tg_ + lane * 20 + 4 * j) = make_float4(g0, g1, g2, g3);
        *reinterpret_cast<float4*>(td_ + lane * 20 + 4 * j) =
            make_float4(g0 - __uint_as_float(v1[4 * j]), g1 - __uint_as_float(v1[4 * j + 1]), g2 - __uint_as_float(v1[4 * j + 2]),
                        g3 - __uint_as_float(v1[4 * j + 3]));
      }
      __syncwarp();
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int idx = lane + 32 * j, rr = idx >> 2, q4 = idx & 3;
        const int lf = qd * 32 + rr, f = f_base + rr, h = cbk * 16 + 4 * q4;
        if (lf < TC_KCHUNK && f < F && h < H) {
          float4 g4 = *reinterpret_cast<const float4*>(tg_ + rr * 20 + 4 * q4);
          float4 d4 = *reinterpret_cast<const float4*>(td_ + rr * 20 + 4 * q4);
          const long long o = (long long)f * H + h;
          if (lambda != 0.f) {
            const float4 t4 = *reinterpret_cast<const float4*>(th + o), o4 = *reinterpret_cast<const float4*>(tho + o);
            g4.x = fmaf(lambda, t4.x, g4.x); g4.y = fmaf(lambda, t4.y, g4.y); g4.z = fmaf(lambda, t4.z, g4.z); g4.w = fmaf(lambda, t4.w, g4.w);
            d4.x = fmaf(lambda, t4.x - o4.x, d4.x); d4.y = fmaf(lambda, t4.y - o4.y, d4.y);
            d4.z = fmaf(lambda, t4.z - o4.z, d4.z); d4.w = fmaf(lambda, t4.w - o4.w, d4.w);
          }
          *reinterpret_cast<float4*>(gf + o) = g4;
          *reinterpret_cast<float4*>(df + o) = d4;
          float4 e4 = d4;                                        // Eq. 8
          if (ref) {
            const float4 r4 = *reinterpret_cast<const float4*>(ref + o);
            if (cada1) e4 = make_float4(d4.x - r4.x, d4.y - r4.y, d4.z - r4.z, d4.w - r4.w);       // Eq. 6
            else e4 = make_float4(g4.x - r4.x, g4.y - r4.y, g4.z - r4.z, g4.w - r4.w);             // Eq. 4
          }
          acc = fma((double)e4.x, (double)e4.x, acc); acc = fma((double)e4.y, (double)e4.y, acc);
          acc = fma((double)e4.z, (double)e4.z, acc); acc = fma((double)e4.w, (double)e4.w, acc);
        }
      }
      __syncwarp();
    }
    // this CTA's share of the gradients of (b1, W2, b2): the slices' sums in slice order
    const int small = g.small, small4 = cg.small4, o_end = min(small, (r + 1) * cg.per_small);
    for (int o = r * cg.per_small + tid; o < o_end; o += MC_THREADS) {
      float gs0 = 0.f, gs1 = 0.f;
      const float* sp0 = cb.small_part + (((size_t)m * n_it) * ns) * small4 + o;
      for (int sl = 0; sl < ns; ++sl) gs0 += __ldcg(sp0 + (size_t)sl * small4);
      if (n_it == 2) {
        const float* sp1 = sp0 + (size_t)ns * small4;
        for (int sl = 0; sl < ns; ++sl) gs1 += __ldcg(sp1 + (size_t)sl * small4);
      }
      const long long oo = FH + o;
      float gv = gs0, dv = n_it == 2 ? gs0 - gs1 : 0.f;
      if (lambda != 0.f) { gv = fmaf(lambda, th[oo], gv); dv = fmaf(lambda, th[oo] - tho[oo], dv); }
      gf[oo] = gv; df[oo] = dv;
      const float e = cada1 ? dv - ref[oo] : lag ? gv - ref[oo] : dv;
      acc = fma((double)e, (double)e, acc);
    }
  }
  // left-hand side: fixed order (shuffle tree, warps in order, slices in order)
  acc = warp_sum(acc);
  if (lane == 0) s_red[warp] = acc;
  __syncthreads();
  if (tid == 0) {
    double part_sum = 0.0;
#pragma unroll
    for (int w8 = 0; w8 < MC_THREADS / 32; ++w8) part_sum += s_red[w8];
    cb.lhs_part[(size_t)m * MC_MAX_SLICES + r] = part_sum;
    if (!ok) atomicOr(&P.st->status_flags, 4);
  }
  tc::fence_before_sync();
  fc_cluster_arrive();
  fc_cluster_wait();
  if (r == 0 && tid == 0) {
    double lhs = 0.0;
    for (int sl = 0; sl < ns; ++sl) lhs += __ldcg(&cb.lhs_part[(size_t)m * MC_MAX_SLICES + sl]);
    decide_upload(P, k, m, lhs, *s_rhs);
  }
  if (warp == 0) tc::tmem_free(tmem, 512u);
}

}  // namespace cada
