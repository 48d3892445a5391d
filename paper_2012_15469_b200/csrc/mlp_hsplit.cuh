// Two-point minibatch gradient of the 2-layer ReLU network AND the upload decision in ONE launch, the hidden layer split
// over a thread-block cluster per worker: CTA r of the cluster owns the hidden units [32 r, 32 r + 32).
//
// Algorithm 1 asks every worker for two gradients on the SAME minibatch.  With the hidden layer split, both large
// products are complete inside a CTA -- nothing of size B x H or F x H is exchanged:
//
//   gather   the B sampled rows (bf16) pass through a ring of stages of 112 features each, in the un-swizzled canonical
//            layout of mlp_tc.cuh.  The rows depend on k only, so the first stages are filled before the wait for the
//            preceding update kernel (programmatic dependent launch).
//   phase 1  Z1[:, slice] = X_B W1[:, slice] for theta^k and for the old iterate: a stage is the K-major A operand, the
//            matching 112-feature chunks of the 32-column slices of the two bf16 weight images arrive by bulk copy, one
//            thread issues tcgen05.mma (M = 128, N = 32) into 2 x 32 tensor-memory columns; four warps refill the stages
//            the products have released.  The weight images are never re-rounded: the update kernel writes the image of
//            theta^{k+1} into slot (k+1) mod (D+1) of a ring of images whose hidden slices are contiguous.
//   phase 2  a1 = relu(Z1 + b1) for this slice (bf16 image in shared memory); the CTA's contribution to the logits,
//            a1[:, slice] W2[slice, :], goes through distributed shared memory to the CTA that owns the row
//            (ceil(B / n_slices) rows each) -- cluster barrier -- the owner adds the contributions in slice order,
//            takes the softmax and sends dz2 (fp32, B x C) to every CTA -- cluster barrier -- every CTA forms
//            dz1[:, slice] = (dz2 W2[slice, :]^T) masked, its rows of dW2 and its part of db1 (warp-level mma.sync on
//            bf16 images; sums, biases, softmax and the bias gradients in fp32), and lays dz1 down as a bf16 operand image.
//   phase 3  dW1[:, slice] = X_B^T dz1[:, slice] for both iterates, one 112-feature block per stage: the SAME staged rows,
//            now read MN-major, against the two dz1 images; 2 x 32 tensor-memory columns per block.  The stages still
//            resident from phase 1 go first while the others are gathered again; the epilogue of a block starts when its
//            products are complete.  It has g and g' of a coordinate side by side: it writes g_m and d_m = g_m - g'_m
//            (regulariser included) to their final place and accumulates the left-hand side of Eq. 8 / Eq. 6 / Eq. 4 in
//            fp64 on the way.
//   barrier  rank 0 adds the slices' left-hand-side parts in slice order and takes the decision (decide_upload).
//
// Every sum has a fixed order (slice order, row order, fixed shuffle trees): results are bitwise reproducible.  Every
// mbarrier wait is bounded; a wait that runs out raises CADA_FLAG_TIMEOUT, and the CTA still walks through every cluster
// barrier (its work skipped) so that its peers are never left waiting, then frees its tensor memory.  All bulk copies
// have one CTA as destination and read this GPU's memory.
#pragma once
#include <algorithm>
#include "mlp_cluster.cuh"   // warp-level mma helpers, tensor-memory loads, ring slots

namespace cada {

constexpr int MH_THREADS = 512;
constexpr int MH_HS = 32;                  // hidden units per CTA = MMA N
constexpr int MH_KCH = 112;                // features per stage (7 MMA k-steps of phase 1, one M block of phase 3)
constexpr int MH_NPC = MH_KCH / 8;         // 16-byte pieces per row of a stage
constexpr unsigned MH_XS_BYTES = 16 * MH_NPC * 128;          // the rows of a stage: 128 rows x 112 features, bf16
constexpr unsigned MH_CHUNK_BYTES = MH_KCH * MH_HS * 2;      // the matching chunk of one weight-image slice
constexpr int MH_MAX_STAGES = 7;           // = most 112-feature chunks (tensor-memory columns: 64 + 7 x 2 x 32)
constexpr int MH_MAX_SLICES = 8;
constexpr int MH_A1P = 40;                 // bf16 pitch of a row of the a1 image (80 bytes: conflict-free 8 x 8 matrix loads)
constexpr int MH_NP = 24;                  // bf16 pitch of the class vectors (W2 rows, dz2 rows)
constexpr int MH_ZF = 16;                  // fp32 pitch of a dz2 row / a dW2 row
constexpr unsigned MH_TAIL_BYTES = 2176;   // barriers, flags, reduction scratch, row offsets, labels, the slices' left-hand-side parts
constexpr unsigned MH_SMEM_MAX = 232448;
constexpr unsigned MH_TILE_BYTES = (MH_THREADS / 32) * 32 * 20 * 4;       // epilogue staging: a [32][20] fp32 tile per warp

struct MlpHsplitGeom {
  int ns;               // hidden slices = CTAs per cluster
  int n_it;             // iterates evaluated: 2, or 1 for the stochastic-LAG rule
  int bp;               // minibatch rows rounded up to a multiple of 16
  int nck;              // 112-feature chunks
  int stages;           // stages of the ring (>= nck: every chunk stays resident)
  int rp;               // minibatch rows whose logits a CTA owns
  int cp;               // classes rounded up to a multiple of 4
  unsigned slice_bytes; // one hidden slice of a weight image: F * 64
  unsigned set_bytes;   // one weight image: ns * slice_bytes
  unsigned w_stage;     // weight chunks of a stage: n_it * MH_CHUNK_BYTES
  unsigned off_u;       // phase 1: weight chunks [stages][w_stage]; afterwards: a1 image, W2 image, dz2 / dz1 image, column sums, dW2, biases
  unsigned o_w2, o_dzf, o_cs, o_dw2, o_b;   // offsets inside that region (the a1 image sits at 0)
  unsigned off_zp;      // logits contributions [ns][n_it][rp][cp] fp32 (later: the bf16 image of dz2 [n_it][bp][24])
  unsigned off_tile;    // epilogue staging
  unsigned off_tail;
  unsigned smem_bytes;
};

__host__ inline bool mlp_hsplit_plan(int F, int H, int C, int B, int rule, long long ldx, MlpHsplitGeom& g) {
  if (F % 16 != 0 || F < 16 || F > MH_KCH * MH_MAX_STAGES || ldx % 8 != 0 || H % 4 != 0 || H < 4 || H > MH_HS * MH_MAX_SLICES ||
      C < 1 || C > 16 || B < 1 || B > 128)
    return false;
  g.ns = (H + MH_HS - 1) / MH_HS;
  g.n_it = rule == 3 ? 1 : 2;
  g.bp = (B + 15) / 16 * 16;
  g.nck = (F + MH_KCH - 1) / MH_KCH;
  g.rp = (B + g.ns - 1) / g.ns;
  g.cp = (C + 3) / 4 * 4;
  g.slice_bytes = (unsigned)F * 64;
  g.set_bytes = g.slice_bytes * g.ns;
  g.w_stage = (unsigned)g.n_it * MH_CHUNK_BYTES;
  auto up128 = [](size_t v) { return (unsigned)((v + 127) / 128 * 128); };
  const unsigned zp = up128(std::max((size_t)g.ns * g.n_it * g.rp * g.cp * 4, (size_t)g.n_it * g.bp * MH_NP * 2));
  unsigned o = up128((size_t)g.n_it * g.bp * MH_A1P * 2);
  g.o_w2 = o;  o += up128((size_t)g.n_it * MH_HS * MH_NP * 2);
  g.o_dzf = o; o += up128(std::max((size_t)g.n_it * g.bp * MH_ZF * 4, (size_t)g.n_it * g.bp * MH_HS * 2));
  g.o_cs = o;  o += up128((size_t)g.n_it * (g.bp / 16) * MH_HS * 4);
  g.o_dw2 = o; o += up128((size_t)g.n_it * MH_HS * MH_ZF * 4);
  g.o_b = o;   o += up128((size_t)g.n_it * 2 * 16 * 4);           // b2 | db2
  for (g.stages = g.nck; g.stages >= 2 || g.stages == g.nck; --g.stages) {
    // the last stage's M = 128 reads run 256 bytes past its rows: the weight region follows the stages
    g.off_u = (unsigned)g.stages * MH_XS_BYTES;
    const unsigned u = std::max(o, (unsigned)g.stages * g.w_stage);
    g.off_zp = g.off_u + up128(u);
    g.off_tile = g.off_zp + zp;
    g.off_tail = g.off_tile + MH_TILE_BYTES;
    g.smem_bytes = g.off_tail + MH_TAIL_BYTES;
    if (g.smem_bytes <= MH_SMEM_MAX) return true;
    if (g.stages <= 2) break;
  }
  return false;
}

__device__ __forceinline__ void mh_store_remote_f2(uint32_t ra, float a, float b) {
  asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(ra), "f"(a), "f"(b) : "memory");
}
__device__ __forceinline__ void mh_send_f2(uint32_t ra, float a, float b, uint32_t rbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.f32 [%0], {%1, %2}, [%3];"
               ::"r"(ra), "f"(a), "f"(b), "r"(rbar) : "memory");
}
__device__ __forceinline__ void mh_store_remote_f1(uint32_t ra, float a) {
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(ra), "f"(a) : "memory");
}
__device__ __forceinline__ uint32_t mh_map(uint32_t local_addr, unsigned rank) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  return ra;
}

// One row's 16-byte pieces of the 112-feature chunk `ck` into stage memory `xs` (rows >= B of the padded batch are zero).
__device__ __forceinline__ void mh_gather_piece(unsigned char* xs, const __nv_bfloat16* __restrict__ X, long long off, long long ldx,
                                                int ck, int i, int c) {
  unsigned char* dst = xs + ((size_t)(i >> 3) * MH_NPC + c) * 128 + (i & 7) * 16;
  if (off >= 0) cp_async16(dst, X + off * ldx + ck * MH_KCH + c * 8);
  else *reinterpret_cast<uint4*>(dst) = make_uint4(0u, 0u, 0u, 0u);
}

// The pieces of chunk `ck` dealt out to `nthr` threads (this one is number t): consecutive threads take consecutive pieces
// of a row, so that a warp's copies cover whole 32-byte sectors.
__device__ __forceinline__ void mh_gather_chunk(unsigned char* xs, const __nv_bfloat16* __restrict__ X, const long long* s_row, long long ldx,
                                                int ck, int np, int bp, int t, int nthr) {
  int i = t / np, c = t - i * np;
  const int di = nthr / np, dc = nthr - di * np;
  for (int o = t; o < bp * np; o += nthr) {
    mh_gather_piece(xs, X, s_row[i], ldx, ck, i, c);
    i += di;
    c += dc;
    if (c >= np) { c -= np; ++i; }
  }
}

__global__ void __launch_bounds__(MH_THREADS, 1)
mlp_hsplit_kernel(const __grid_constant__ Params P, const __grid_constant__ MlpHsplitGeom g, MlpBufs mb, double* lhs_part /* [M][8] */,
                  long long k /* iteration, as the host counts it */) {
  extern __shared__ __align__(128) unsigned char mhsm[];
  unsigned char* s_x = mhsm;                                   // [stages][MH_XS_BYTES]
  unsigned char* s_u = mhsm + g.off_u;
  unsigned char* s_zp_raw = mhsm + g.off_zp;
  unsigned char* tail = mhsm + g.off_tail;
  // tail: weights landed [7] | rows landed [7] (+64) | stage released [7] (+128) | block done [7] (+192) | z1 done (+256) |
  //       rows landed, phase 3 [7] (+264) |
  //       tensor-memory address (+320) | ok (+324) | reduction scratch (+336, 16 doubles) | row offsets (+512, 128 x 8) |
  //       labels (+1536, 128 x 4) | left-hand-side parts of the slices (+2048, 8 doubles; rank 0)
  //       exchange barriers (+472: logits, +480: dz2, +488: left-hand-side parts): the CTAs of the cluster send with
  //       asynchronous remote stores that credit the receiver's barrier with their bytes; each is used once per launch
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(tail + 320);
  int* s_ok = reinterpret_cast<int*>(tail + 324);
  double* s_red = reinterpret_cast<double*>(tail + 336);
  long long* s_row = reinterpret_cast<long long*>(tail + 512);
  int* s_label = reinterpret_cast<int*>(tail + 1536);
  double* s_lparts = reinterpret_cast<double*>(tail + 2048);
  bool dead = false;                                            // a bounded wait of this thread has run out

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int qd = warp & 3, part = warp >> 2;                    // accumulator lane quarter this warp may read; its share of the columns
  const int g8 = lane >> 2, t4 = lane & 3;                      // fragment coordinates of this lane (mma.sync)
  const int m = blockIdx.y;
  unsigned rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int r = (int)rank, ns = g.ns, n_it = g.n_it, bp = g.bp, nck = g.nck, S = g.stages;
  const int F = P.F, H = P.H, C = P.C, B = P.B;
  const long long FH = (long long)F * H;
  const int h0 = r * MH_HS;
  const __nv_bfloat16* __restrict__ X = static_cast<const __nv_bfloat16*>(P.X[m]);
  const uint32_t bar_w = ptx::smem_u32(tail), bar_x = bar_w + 64, bar_free = bar_w + 128, bar_done = bar_w + 192, bar_z1 = bar_w + 256,
                 bar_x3 = bar_w + 264, bar_lg = bar_w + 472, bar_dz = bar_w + 480, bar_lp = bar_w + 488;
  const uint32_t a0 = ptx::smem_u32(s_x), u0 = ptx::smem_u32(s_u);
  const bool gatherer = part == 3;                              // warps 12-15: their lanes 0 issue the products of phase 3

  pdl_trigger();                                                // the update kernel may be scheduled behind this one
  if (P.idx_mode == IDX_EXPLICIT) pdl_wait();                   // explicit indices may have been produced on this stream just before
  if (tid < 128) s_row[tid] = tid < B ? minibatch_row(P, k, m, tid, P.n_samples[m]) : -1;
  if (tid == 0) {
    for (int i = 0; i < MH_MAX_STAGES; ++i) {
      ptx::mbar_init(bar_w + 8 * i, 1);
      ptx::mbar_init(bar_x + 8 * i, 11 * 32);
      ptx::mbar_init(bar_x3 + 8 * i, MH_THREADS);
      ptx::mbar_init(bar_free + 8 * i, (uint32_t)(2 * n_it));
      ptx::mbar_init(bar_done + 8 * i, 1);
    }
    ptx::mbar_init(bar_z1, (uint32_t)(2 * n_it));
    ptx::mbar_init(bar_lg, 1); ptx::mbar_init(bar_dz, 1); ptx::mbar_init(bar_lp, 1);
    ptx::fence_barrier_init();
    // armed before this CTA arrives at the start barrier: whoever passes that barrier may send
    const int my_rows = max(0, min(g.rp, B - r * g.rp));
    fc_arrive_expect_tx(bar_lg, (uint32_t)(ns * n_it * my_rows * g.cp * 4));     // every slice's contribution to the logits of this CTA's rows
    fc_arrive_expect_tx(bar_dz, (uint32_t)(n_it * B * C * 4));                    // dz2 of every row
    fc_arrive_expect_tx(bar_lp, (uint32_t)(ns * 8));                              // (rank 0 waits for it)
    *s_ok = 1;
  }
  if (warp == 0) tc::tmem_alloc(ptx::smem_u32(s_tmem), 512u);
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  const uint32_t tmem = *s_tmem;
  const uint32_t my_lanes = tmem + ((uint32_t)(qd * 32) << 16);
  fc_cluster_arrive();                                          // "this CTA runs": waited for before the first store into a peer

  // ---- gather of the first stages: 16-byte pieces (row i, piece c) ---------------------------------------------------
  {
    const int n_first = min(S, nck);
    for (int ck = 0; ck < n_first; ++ck) {
      const int np = min(MH_KCH, F - ck * MH_KCH) / 8;
      const float inv_np = 1.0f / (float)np;
      unsigned char* xs = s_x + (size_t)ck * MH_XS_BYTES;
      for (int o = tid; o < bp * np; o += MH_THREADS) {
        const int i = div_small(o, np, inv_np), c = o - i * np;
        mh_gather_piece(xs, X, s_row[i], P.ldx, ck, i, c);
      }
    }
    cp_async_commit();
  }
  if (tid < B) s_label[tid] = static_cast<const int*>(P.y[m])[s_row[tid]];

  pdl_wait();                                                   // iterates, their images and the staleness belong to earlier kernels until now
  int tau_early = 0;
  if (r == 0 && tid == 0) tau_early = P.tau[m];                 // for the decision at the kernel's end
  const float* __restrict__ th = P.theta;
  const float* __restrict__ tho = old_iterate(P, k, m);

  cp_async_wait<0>();
  tc::fence_async_proxy();                                      // gathered pieces (generic proxy) -> visible to the tensor core
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  double* s_rhs = reinterpret_cast<double*>(tail + 464);       // this iteration's right-hand side (rank 0)
  if (r == 0 && warp == 5) {                                    // the newest window term, if the update kernel left it in parts; then the right-hand side
    const double rhs = window_refresh_rhs(P, k, lane);
    if (lane == 0) *s_rhs = rhs;
  }

  // operands that do not depend on the products: fetched into registers while they run (their place in shared memory
  // is under the chunk ring until the products are complete)
  __nv_bfloat16* s_a1 = reinterpret_cast<__nv_bfloat16*>(s_u);                   // [n_it][bp][40]  a1 rounded (0 where z1 <= 0, beyond B, beyond H)
  __nv_bfloat16* s_w2 = reinterpret_cast<__nv_bfloat16*>(s_u + g.o_w2);          // [n_it][32][24]  W2 rows of the slice rounded, zero padding
  float* s_dzf = reinterpret_cast<float*>(s_u + g.o_dzf);                        // [n_it][bp][16]  dz2 (fp32) as the owners send it
  unsigned char* s_img = s_u + g.o_dzf;                                          // ... later the dz1 operand image [bp/8][4 n_it hidden chunks][8 rows x 16 B]
  float* s_cs = reinterpret_cast<float*>(s_u + g.o_cs);                          // [n_it][bp/16][32] column sums of dz1 per row tile
  float* s_dw2 = reinterpret_cast<float*>(s_u + g.o_dw2);                        // [n_it][32][16]
  float* s_b2 = reinterpret_cast<float*>(s_u + g.o_b);                           // [n_it][16] b2, then [n_it][16] db2
  float* s_db2 = s_b2 + n_it * 16;
  float* s_zp = reinterpret_cast<float*>(s_zp_raw);
  __nv_bfloat16* s_dq = reinterpret_cast<__nv_bfloat16*>(s_zp_raw);              // [n_it][bp][24]  dz2 rounded, zero padding

  constexpr int W2_PER = (2 * MH_HS * MH_NP + MH_THREADS - 1) / MH_THREADS;      // 3
  float w2r[W2_PER];
#pragma unroll
  for (int t = 0; t < W2_PER; ++t) {
    const int o = tid + t * MH_THREADS;
    w2r[t] = 0.f;
    if (o < n_it * MH_HS * MH_NP) {
      const int it = o >= MH_HS * MH_NP ? 1 : 0, e = o - it * MH_HS * MH_NP, hl = e / MH_NP, c = e - hl * MH_NP;
      if (h0 + hl < H && c < C) w2r[t] = (it ? tho : th)[FH + H + (long long)(h0 + hl) * C + c];
    }
  }
  float b2r = 0.f;
  if (tid < n_it * 16) { const int it = tid >> 4, c = tid & 15; if (c < C) b2r = (it ? tho : th)[FH + H + (long long)H * C + c]; }
  // first-layer bias of the 16 columns this warp will read from tensor memory
  const int it_a = part >> 1, cb_a = part & 1;
  const bool reads_z1 = part < 2 * n_it;
  float b1r[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) b1r[e] = 0.f;
  if (reads_z1) {
    const float* bsrc = (it_a ? tho : th) + FH + h0 + cb_a * 16;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (h0 + cb_a * 16 + 4 * q < H) {
        const float4 b4 = *reinterpret_cast<const float4*>(bsrc + 4 * q);
        b1r[4 * q] = b4.x; b1r[4 * q + 1] = b4.y; b1r[4 * q + 2] = b4.z; b1r[4 * q + 3] = b4.w;
      }
  }

  // ---- phase 1: Z1 of this slice for every iterate, chunk by chunk --------------------------------------------------
  // Parities of the barriers a thread waits on are kept as bit masks (bit s = stage s): a barrier completes once per use.
  uint32_t par_x = 0;                                           // issuer's view of "rows landed" (refilled stages only)
  // A stream of N = 32 products is bound by the rate at which ONE lane can issue them (about 140 cycles each), not by the
  // tensor core, so up to four lanes issue, each into an accumulator of its own: lane 0 of warp w < 2 n_it takes iterate
  // w % n_it and the k-steps of parity w / n_it; the two parities of an iterate are added in phase 2 (fixed order).  The
  // lanes beside an issuing lane wait at a warp barrier.
  const int n_iss = 2 * n_it;
  if (warp == 4) {                                              // weight chunks
   if (lane == 0) {
    bool pok = true;
    uint32_t par_free = 0;
    for (int ck = 0; ck < nck && pok; ++ck) {
      const int s = ck % S;
      if (ck >= S) {
        if (!ptx::mbar_wait_bounded(bar_free + 8 * s, (par_free >> s) & 1u)) { pok = false; break; }
        par_free ^= 1u << s;
      }
      const uint32_t bytes = (uint32_t)min(MH_KCH, F - ck * MH_KCH) * 64u;
      ptx::mbar_expect_tx(bar_w + 8 * s, (uint32_t)n_it * bytes);
      for (int it = 0; it < n_it; ++it) {
        const unsigned char* src = P.w1_ring + (size_t)mlp_ring_slot(P, k, m, it) * P.w1_set_bytes + (size_t)r * g.slice_bytes +
                                   (size_t)ck * MH_CHUNK_BYTES;
        ptx::bulk_g2s(u0 + s * g.w_stage + it * MH_CHUNK_BYTES, src, bytes, bar_w + 8 * s);
      }
      ptx::mbar_arrive(bar_w + 8 * s);
    }
    if (!pok) *s_ok = 0;
   }
   __syncwarp();
  } else if (warp < n_iss) {                                    // issue the products
   if (lane == 0) {
    const int it = warp % n_it, kh = warp / n_it;
    bool iok = true;
    uint32_t par_w = 0;
    const uint32_t idesc = tc::instr_desc(128, MH_HS, false, true);
    const uint32_t d_acc = tmem + (uint32_t)(kh * n_it + it) * MH_HS;
    bool first = true;
    for (int ck = 0; ck < nck; ++ck) {
      const int s = ck % S;
      if (iok && !ptx::mbar_wait_bounded(bar_w + 8 * s, (par_w >> s) & 1u)) iok = false;
      par_w ^= 1u << s;
      if (iok && ck >= S) {
        if (!ptx::mbar_wait_bounded(bar_x + 8 * s, (par_x >> s) & 1u)) iok = false;
        par_x ^= 1u << s;
      }
      if (iok) {
        tc::fence_after_sync();
        const int ksteps = min(MH_KCH, F - ck * MH_KCH) / 16;
#pragma unroll
        for (int ks2 = 0; ks2 < (MH_KCH / 16 + 1) / 2; ++ks2) {
          const int ks = 2 * ks2 + kh;
          if (ks < ksteps) {
            const uint64_t da = tc::smem_desc(a0 + s * MH_XS_BYTES + ks * 256, 128, MH_NPC * 128);                        // K-major: LBO = next 8 features, SBO = next 8 rows
            const uint64_t db = tc::smem_desc(u0 + s * g.w_stage + it * MH_CHUNK_BYTES + ks * 1024, 512, 128);            // MN-major: LBO = next 8 features, SBO = next 8 hidden
            tc::mma_bf16(d_acc, da, db, idesc, !first);
            first = false;
          }
        }
      }
      tc::mma_commit(bar_free + 8 * s);
    }
    tc::mma_commit(bar_z1);
    if (!iok) *s_ok = 0;
   }
   __syncwarp();
  } else if (warp >= 5 && nck > S) {                            // rows of the chunks beyond the first stages: warps 5-15
    bool gok = true;
    uint32_t par_free = 0;
    for (int ck = S; ck < nck && gok; ++ck) {
      const int s = ck % S;
      if (!ptx::mbar_wait_bounded(bar_free + 8 * s, (par_free >> s) & 1u)) { gok = false; break; }
      par_free ^= 1u << s;
      mh_gather_chunk(s_x + (size_t)s * MH_XS_BYTES, X, s_row, P.ldx, ck, min(MH_KCH, F - ck * MH_KCH) / 8, bp, tid - 5 * 32, 11 * 32);
    }
    cp_async_commit();
    cp_async_wait<0>();
    tc::fence_async_proxy();
    if (gok) for (int ck = S; ck < nck; ++ck) ptx::mbar_arrive(bar_x + 8 * (ck % S));
    else *s_ok = 0;
  }

  bool ok = ptx::mbar_wait_bounded(bar_z1, 0);
  tc::fence_after_sync();
#pragma unroll
  for (int t = 0; t < W2_PER; ++t) {
    const int o = tid + t * MH_THREADS;
    if (o < n_it * MH_HS * MH_NP) s_w2[o] = __float2bfloat16_rn(w2r[t]);
  }
  if (tid < n_it * 16) s_b2[tid] = b2r;

  // ---- phase 2 -----------------------------------------------------------------------------------------------------
  // z1 = accumulator + b1; a1 = relu(z1) rounded.  Accumulator lane = minibatch row.
  if (reads_z1) {
    const int i = qd * 32 + lane;
    uint32_t v[16], v2[16];
    tc::tmem_ld16_issue(my_lanes + it_a * MH_HS + cb_a * 16, v);
    tc::tmem_ld16_issue(my_lanes + (n_it + it_a) * MH_HS + cb_a * 16, v2);
    tc::tmem_ld_wait16(v);
    tc::tmem_ld_wait16(v2);
    if (ok && i < bp) {
      __align__(16) __nv_bfloat16 a16[16];
      float z[16];
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        z[e] = (__uint_as_float(v[e]) + (F >= 32 ? __uint_as_float(v2[e]) : 0.f)) + b1r[e];   // one k-step only: the odd-parity accumulator was never written
        a16[e] = __float2bfloat16_rn((i < B && h0 + cb_a * 16 + e < H) ? fmaxf(z[e], 0.f) : 0.f);
      }
      uint4* dst = reinterpret_cast<uint4*>(s_a1 + ((size_t)it_a * bp + i) * MH_A1P + cb_a * 16);
      dst[0] = reinterpret_cast<const uint4*>(a16)[0];
      dst[1] = reinterpret_cast<const uint4*>(a16)[1];
      if (i < B) {
        float* zo = mb.z1 + (((long long)m * 2 + it_a) * B + i) * H + h0 + cb_a * 16;
#pragma unroll
        for (int q = 0; q < 4; ++q)
          if (h0 + cb_a * 16 + 4 * q < H) *reinterpret_cast<float4*>(zo + 4 * q) = make_float4(z[4 * q], z[4 * q + 1], z[4 * q + 2], z[4 * q + 3]);
      }
    }
  }
  if (!ok) *s_ok = 0;
  __syncthreads();

  // contributions of this slice to the logits: one warp per (iterate, 16-row tile, 8-class tile); each pair of values
  // goes to the CTA that owns the row
  const int mts = bp / 16, ntc = (C + 7) / 8, rp = g.rp, cp = g.cp;
  fc_cluster_wait();                                            // every CTA of the cluster has started
  {
    const float inv_rp = 1.0f / (float)rp;
    const uint32_t zp0 = ptx::smem_u32(s_zp);
    for (int u = warp; u < n_it * mts * ntc; u += MH_THREADS / 32) {
      const int nt = u % ntc, mt = (u / ntc) % mts, it = u / (ntc * mts);
      float d[4] = {0.f, 0.f, 0.f, 0.f};
      const __nv_bfloat16* a_base = s_a1 + ((size_t)it * bp + mt * 16 + (lane & 15)) * MH_A1P + (lane >> 4) * 8;
      const __nv_bfloat16* b_base = s_w2 + ((size_t)it * MH_HS + (lane & 15)) * MH_NP + nt * 8;
#pragma unroll
      for (int k0 = 0; k0 < MH_HS; k0 += 16) {
        uint32_t a[4], bq[2];
        mm::ldmatrix_x4(a, a_base + k0);
        mm::ldmatrix_x2_trans(bq, b_base + (size_t)k0 * MH_NP);
        mm::mma_bf16_16816(d, a, bq);
      }
      const int col = nt * 8 + 2 * t4;
#pragma unroll
      for (int hh = 0; hh < 2; ++hh) {
        const int i = mt * 16 + g8 + 8 * hh;
        if (i < B && col < cp) {
          const int owner = div_small(i, rp, inv_rp), il = i - owner * rp;
          const uint32_t la = zp0 + (uint32_t)((((r * n_it + it) * rp + il) * cp + col) * 4);
          mh_send_f2(mh_map(la, (unsigned)owner), d[2 * hh], d[2 * hh + 1], mh_map(bar_lg, (unsigned)owner));
        }
      }
    }
  }
  fc_wait(bar_lg, 0u, dead, &P.st->status_flags);               // every slice's contribution to this CTA's rows has arrived

  // the rows this CTA owns: logits in slice order, softmax, dz2 = (P - onehot) / B, sent to every CTA of the cluster
  {
    const int i_first = r * rp, nr = max(0, min(rp, B - i_first)), pairs = n_it * nr;
    const float invB = 1.0f / (float)B;
    const uint32_t dzf0 = ptx::smem_u32(s_dzf);
    for (int base = 0; base < pairs * 16; base += MH_THREADS) {
      const int item = base + tid, c = item & 15, pr = item >> 4;
      const bool valid = pr < pairs && c < C;
      int it = 0, il = 0;
      if (pr < pairs) { it = pr >= nr ? 1 : 0; il = pr - it * nr; }
      float z = -INFINITY;
      if (valid) {
        z = s_b2[it * 16 + c];
        for (int sl = 0; sl < ns; ++sl) z += s_zp[((sl * n_it + it) * rp + il) * cp + c];
      }
      float mx = z;
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float e = valid ? expf(z - mx) : 0.f;
      float den = e;
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
      if (valid) {
        const int i = i_first + il;
        const float dv = (e * (1.f / den) - (c == s_label[i] ? 1.f : 0.f)) * invB;
        mb.dz2[(((long long)m * 2 + it) * B + i) * C + c] = dv;
        const uint32_t la = dzf0 + (uint32_t)((((it * bp) + i) * MH_ZF + c) * 4);
        for (int t = 0; t < ns; ++t) fc_st_async_f32(mh_map(la, (unsigned)t), dv, mh_map(bar_dz, (unsigned)t));
      }
    }
  }
  fc_wait(bar_dz, 0u, dead, &P.st->status_flags);               // dz2 of every row is here

  // bf16 image of dz2 (zero beyond B and beyond C); rank 0 also sums db2 (fp32, unrounded, row order)
  for (int o = tid; o < n_it * bp * 3; o += MH_THREADS) {
    const int pr = o / 3, c8 = o - pr * 3, it = pr >= bp ? 1 : 0, i = pr - it * bp;
    __align__(16) __nv_bfloat16 v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int c = c8 * 8 + e;
      v[e] = __float2bfloat16_rn((i < B && c < C) ? s_dzf[((size_t)it * bp + i) * MH_ZF + c] : 0.f);
    }
    *reinterpret_cast<uint4*>(s_dq + ((size_t)it * bp + i) * MH_NP + c8 * 8) = *reinterpret_cast<const uint4*>(v);
  }
  if (r == 0 && tid < n_it * 16) {
    const int it = tid >> 4, c = tid & 15;
    float a = 0.f;
    if (c < C) for (int i = 0; i < B; ++i) a += s_dzf[((size_t)it * bp + i) * MH_ZF + c];
    s_db2[tid] = a;
  }
  __syncthreads();

  // dW2 rows of the slice (a1q^T dz2q) and dz1 of the slice ((dz2q W2q^T) where z1 > 0), one warp per tile
  {
    const int n_dw2 = n_it * 2 * ntc;
    for (int u = warp; u < n_dw2 + n_it * mts * 4; u += MH_THREADS / 32) {
      if (u < n_dw2) {
        const int nt = u % ntc, ht = (u / ntc) & 1, it = u / (ntc * 2);
        float d[4] = {0.f, 0.f, 0.f, 0.f};
        for (int k0 = 0; k0 < bp; k0 += 16) {
          uint32_t a[4], bq[2];
          // A = a1q^T (hidden x rows) read from the row-major image with transposing loads
          mm::ldmatrix_x4_trans(a, s_a1 + ((size_t)it * bp + k0 + (lane & 7) + ((lane >> 4) & 1) * 8) * MH_A1P + ht * 16 + ((lane >> 3) & 1) * 8);
          mm::ldmatrix_x2_trans(bq, s_dq + ((size_t)it * bp + k0 + (lane & 15)) * MH_NP + nt * 8);
          mm::mma_bf16_16816(d, a, bq);
        }
        const int col = nt * 8 + 2 * t4;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int hl = ht * 16 + g8 + 8 * hh;
          *reinterpret_cast<float2*>(s_dw2 + ((size_t)it * MH_HS + hl) * MH_ZF + col) = make_float2(d[2 * hh], d[2 * hh + 1]);
        }
      } else {
        const int v = u - n_dw2, ht = v & 3, mt = (v >> 2) % mts, it = (v >> 2) / mts;
        uint32_t a[4], bq[2];
        float d[4] = {0.f, 0.f, 0.f, 0.f};
        mm::ldmatrix_x4(a, s_dq + ((size_t)it * bp + mt * 16 + (lane & 15)) * MH_NP + (lane >> 4) * 8);
        mm::ldmatrix_x2(bq, s_w2 + ((size_t)it * MH_HS + ht * 8 + (lane & 7)) * MH_NP + ((lane >> 3) & 1) * 8);
        mm::mma_bf16_16816(d, a, bq);
        const int hl = ht * 8 + 2 * t4;
        float c0 = 0.f, c1 = 0.f;
#pragma unroll
        for (int hh = 0; hh < 2; ++hh) {
          const int i = mt * 16 + g8 + 8 * hh;
          const float2 av = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(s_a1 + ((size_t)it * bp + i) * MH_A1P + hl));
          const float e0 = av.x > 0.f ? d[2 * hh] : 0.f, e1 = av.y > 0.f ? d[2 * hh + 1] : 0.f;
          if (i < B && h0 + hl < H)
            *reinterpret_cast<float2*>(mb.dz1 + (((long long)m * 2 + it) * B + i) * H + h0 + hl) = make_float2(e0, e1);
          *reinterpret_cast<__nv_bfloat162*>(s_img + ((size_t)(i >> 3) * (4 * n_it) + it * 4 + (hl >> 3)) * 128 + (i & 7) * 16 + (hl & 7) * 2) =
              __floats2bfloat162_rn(e0, e1);
          c0 += e0; c1 += e1;
        }
        // column sums of the tile (db1, fp32, unrounded): rows g8 and g8 + 8 above, then over g8 by a fixed tree
#pragma unroll
        for (int o = 4; o < 32; o <<= 1) { c0 += __shfl_xor_sync(0xffffffffu, c0, o); c1 += __shfl_xor_sync(0xffffffffu, c1, o); }
        if (lane < 4) *reinterpret_cast<float2*>(s_cs + ((size_t)it * mts + mt) * MH_HS + hl) = make_float2(c0, c1);
      }
    }
  }
  tc::fence_async_proxy();                                      // the dz1 images (generic proxy) -> visible to the tensor core
  tc::fence_before_sync();
  __syncthreads();
  tc::fence_after_sync();
  ok = *s_ok != 0;

  // ---- phase 3: dW1 of this slice for every iterate, one 112-feature block per stage ------------------------------------
  // Block order: the chunks still resident from phase 1 first (the last `stages` of them), then chunks 0, 1, ..., each
  // gathered again into the stage of a block whose products are complete.  Lane 0 of each of warps 12-15 issues every
  // fourth block.
  const int n_res = min(S, nck), first_res = nck - n_res;
  // (a product costs the same for 32 as for 64 columns: the iterates' dz1 columns sit side by side in one image, N = 32 n_it)
  const uint32_t idesc3 = tc::instr_desc(128, MH_HS * n_it, true, true);
  const uint32_t img0 = ptx::smem_u32(s_img);
  auto issue_block = [&](int ck) {
    const int s = ck % S;
#pragma unroll
    for (int t = 0; t < 8; ++t)
      if (t < mts) {
        const uint64_t da = tc::smem_desc(a0 + s * MH_XS_BYTES + t * 2 * MH_NPC * 128, MH_NPC * 128, 128);     // MN-major: LBO = next 8 rows, SBO = next 8 features
        const uint64_t db = tc::smem_desc(img0 + t * 2 * (4 * n_it) * 128, (4 * n_it) * 128, 128);            // MN-major: LBO = next 8 rows, SBO = next 8 hidden
        tc::mma_bf16(tmem + 64 + ck * n_it * MH_HS, da, db, idesc3, t > 0);
      }
  };
  // resident blocks: those whose stage is gathered into again go first (chunk j's stage holds block j + S ...)
  auto resident_block = [&](int q) { return nck > S ? first_res + (q + (S - first_res % S)) % n_res : first_res + q; };
  if (gatherer) {                                               // lane 0 of each of warps 12-15 issues every fourth block
    if (lane == 0)
      for (int q = warp - 12; q < n_res; q += 4) {
        const int ck = resident_block(q);
        if (ok) issue_block(ck);
        tc::mma_commit(bar_done + 8 * ck);
      }
    __syncwarp();
  }
  // while the resident blocks run: the gradients of (b1, W2, b2) that belong to this slice, complete in this CTA
  double acc = 0.0;
  const bool cada1 = P.rule == 1, lag = P.rule == 3;
  const float lambda = P.lambda;
  const float* __restrict__ ref = cada1 ? P.delta_stored + (long long)m * P.ldp : lag ? P.G + (long long)m * P.ldp : nullptr;
  float* __restrict__ gf = P.g_fresh + (long long)m * P.ldp;
  float* __restrict__ df = P.d_fresh + (long long)m * P.ldp;
  if (ok) {
    const int n_small = MH_HS + MH_HS * C + (r == 0 ? C : 0);
    for (int o = tid; o < n_small; o += MH_THREADS) {
      float g0 = 0.f, g1 = 0.f;
      long long oo = -1;
      if (o < MH_HS) {
        const int hl = o;
        if (h0 + hl < H) {
          oo = FH + h0 + hl;
          for (int mt = 0; mt < mts; ++mt) g0 += s_cs[(size_t)mt * MH_HS + hl];
          if (n_it == 2) for (int mt = 0; mt < mts; ++mt) g1 += s_cs[((size_t)mts + mt) * MH_HS + hl];
        }
      } else if (o < MH_HS + MH_HS * C) {
        const int e = o - MH_HS, hl = e / C, c = e - hl * C;
        if (h0 + hl < H) {
          oo = FH + H + (long long)(h0 + hl) * C + c;
          g0 = s_dw2[(size_t)hl * MH_ZF + c];
          if (n_it == 2) g1 = s_dw2[((size_t)MH_HS + hl) * MH_ZF + c];
        }
      } else {
        const int c = o - MH_HS - MH_HS * C;
        oo = FH + H + (long long)H * C + c;
        g0 = s_db2[c];
        if (n_it == 2) g1 = s_db2[16 + c];
      }
      if (oo >= 0) {
        float gv = g0, dv = n_it == 2 ? g0 - g1 : 0.f;
        if (lambda != 0.f) { gv = fmaf(lambda, th[oo], gv); dv = fmaf(lambda, th[oo] - tho[oo], dv); }
        gf[oo] = gv; df[oo] = dv;
        const float e = cada1 ? dv - ref[oo] : lag ? gv - ref[oo] : dv;
        acc = fma((double)e, (double)e, acc);
      }
    }
  }

  // the blocks that are not resident: every thread takes part in gathering their rows (the epilogue is bound by its
  // stores -- starting it on the resident blocks meanwhile was measured: no gain), then the four issuing lanes send their
  // products
  if (nck > S) {
    bool gok = ok;
    for (int j = 0; j < nck - S && gok; ++j) {
      const int s = j % S;
      const int prev = j >= S ? j - S : j + S * ((nck - 1 - j) / S);          // the block whose rows the stage holds now
      if (!ptx::mbar_wait_bounded(bar_done + 8 * prev, 0)) { gok = false; break; }
      mh_gather_chunk(s_x + (size_t)s * MH_XS_BYTES, X, s_row, P.ldx, j, min(MH_KCH, F - j * MH_KCH) / 8, bp, tid, MH_THREADS);
    }
    cp_async_commit();
    cp_async_wait<0>();
    tc::fence_async_proxy();
    if (gok) for (int j = 0; j < nck - S; ++j) ptx::mbar_arrive(bar_x3 + 8 * (j % S));
    else { ok = false; *s_ok = 0; }
    if (gatherer) {
     if (lane == 0) {
      bool iok = gok;
      uint32_t px = 0;
      for (int j = 0; j < nck - S; ++j) {
        const int s = j % S;
        if (((n_res + j) & 3) == warp - 12) {
          if (iok && !ptx::mbar_wait_bounded(bar_x3 + 8 * s, (px >> s) & 1u)) iok = false;
          if (iok) { tc::fence_after_sync(); issue_block(j); }
          tc::mma_commit(bar_done + 8 * j);
        }
        px ^= 1u << s;
      }
      if (!iok) *s_ok = 0;
     }
     __syncwarp();
    }
  }

  if (ok) {
    // accumulator lane = feature of the block; the four warps of a lane quarter share the (block, 16-column half) list in
    // the order the blocks complete.  A warp stages g, then g - g', of a piece in its [32][20] tile and writes them with
    // four lanes per 64-byte row piece
    float* tile = reinterpret_cast<float*>(mhsm + g.off_tile) + (size_t)warp * 32 * 20;
    for (int u = part; u < nck * 2; u += 4) {
      const int q = u >> 1, cbk = u & 1;
      const int ck = q < n_res ? resident_block(q) : q - n_res;
      const int feats = min(MH_KCH, F - ck * MH_KCH);
      if (h0 + cbk * 16 >= H || qd * 32 >= feats) continue;     // warp-uniform
      if (!__all_sync(0xffffffffu, ptx::mbar_wait_bounded(bar_done + 8 * ck, 0))) { ok = false; break; }
      tc::fence_after_sync();
      uint32_t v0[16], v1[16];
      const uint32_t col = 64 + (uint32_t)(ck * n_it) * MH_HS + cbk * 16;
      tc::tmem_ld16_issue(my_lanes + col, v0);
      if (n_it == 2) tc::tmem_ld16_issue(my_lanes + col + MH_HS, v1);
      tc::tmem_ld_wait16(v0);
      if (n_it == 2) {
        tc::tmem_ld_wait16(v1);
      } else {
#pragma unroll
        for (int e = 0; e < 16; ++e) v1[e] = v0[e];               // one gradient only: the difference is identically 0
      }
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<float4*>(tile + lane * 20 + 4 * j) = make_float4(__uint_as_float(v0[4 * j]), __uint_as_float(v0[4 * j + 1]),
                                                                           __uint_as_float(v0[4 * j + 2]), __uint_as_float(v0[4 * j + 3]));
      __syncwarp();
      // left-hand side: the (at most 16) squares of a piece are added in fp32, the pieces in fp64 -- conversions to fp64
      // are slow enough that one per value bounded the whole epilogue
      float sq = 0.f;
      float4 gq[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int idx = lane + 32 * j;
        gq[j] = *reinterpret_cast<const float4*>(tile + (idx >> 2) * 20 + 4 * (idx & 3));
      }
      __syncwarp();
#pragma unroll
      for (int j = 0; j < 4; ++j)
        *reinterpret_cast<float4*>(tile + lane * 20 + 4 * j) =
            make_float4(__uint_as_float(v0[4 * j]) - __uint_as_float(v1[4 * j]), __uint_as_float(v0[4 * j + 1]) - __uint_as_float(v1[4 * j + 1]),
                        __uint_as_float(v0[4 * j + 2]) - __uint_as_float(v1[4 * j + 2]), __uint_as_float(v0[4 * j + 3]) - __uint_as_float(v1[4 * j + 3]));
      __syncwarp();
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int idx = lane + 32 * j, rr = idx >> 2, q4 = idx & 3;
        const int lf = qd * 32 + rr, f = ck * MH_KCH + lf, h = h0 + cbk * 16 + 4 * q4;
        if (lf < feats && h < H) {
          float4 g4 = gq[j];
          float4 d4 = *reinterpret_cast<const float4*>(tile + rr * 20 + 4 * q4);
          const long long o = (long long)f * H + h;
          if (lambda != 0.f) {
            const float4 t4v = *reinterpret_cast<const float4*>(th + o), o4 = *reinterpret_cast<const float4*>(tho + o);
            g4.x = fmaf(lambda, t4v.x, g4.x); g4.y = fmaf(lambda, t4v.y, g4.y); g4.z = fmaf(lambda, t4v.z, g4.z); g4.w = fmaf(lambda, t4v.w, g4.w);
            d4.x = fmaf(lambda, t4v.x - o4.x, d4.x); d4.y = fmaf(lambda, t4v.y - o4.y, d4.y);
            d4.z = fmaf(lambda, t4v.z - o4.z, d4.z); d4.w = fmaf(lambda, t4v.w - o4.w, d4.w);
          }
          *reinterpret_cast<float4*>(gf + o) = g4;
          *reinterpret_cast<float4*>(df + o) = d4;
          float4 e4 = d4;                                        // Eq. 8
          if (ref) {
            const float4 r4 = *reinterpret_cast<const float4*>(ref + o);
            if (cada1) e4 = make_float4(d4.x - r4.x, d4.y - r4.y, d4.z - r4.z, d4.w - r4.w);       // Eq. 6
            else e4 = make_float4(g4.x - r4.x, g4.y - r4.y, g4.z - r4.z, g4.w - r4.w);             // Eq. 4
          }
          sq = fmaf(e4.x, e4.x, sq); sq = fmaf(e4.y, e4.y, sq); sq = fmaf(e4.z, e4.z, sq); sq = fmaf(e4.w, e4.w, sq);
        }
      }
      acc += (double)sq;
      __syncwarp();
    }
  }
  if (!ok) *s_ok = 0;
  __syncthreads();
  ok = *s_ok != 0;
  // left-hand side: fixed order (shuffle tree, warps in order, slices in order)
  acc = warp_sum(acc);
  if (lane == 0) s_red[warp] = acc;
  tc::fence_before_sync();
  __syncthreads();
  if (tid == 0) {
    double part_sum = 0.0;
#pragma unroll
    for (int w8 = 0; w8 < MH_THREADS / 32; ++w8) part_sum += s_red[w8];
    fc_st_async_f64(mh_map(ptx::smem_u32(s_lparts + r), 0u), part_sum, mh_map(bar_lp, 0u));   // to rank 0
    if (!ok) atomicOr(&P.st->status_flags, 4);
  }
  if (r == 0 && tid == 0) {
    fc_wait(bar_lp, 0u, dead, &P.st->status_flags);
    double lhs = 0.0;
    for (int sl = 0; sl < ns; ++sl) lhs += s_lparts[sl];
    decide_upload_tau(P, k, m, lhs, *s_rhs, tau_early);
  }
  // every warp's reads of tensor memory precede the CTA-wide barrier above; everything sent to this CTA has been waited
  // for (rank 0: by the thread that decides), so the CTA may free its tensor memory and leave
  if (warp == 0) { tc::fence_after_sync(); tc::tmem_free(tmem, 512u); }
}

}  // namespace cada
