// Two-point minibatch gradient AND upload decision for softmax regression (up to 16 classes): one thread-block
// cluster per worker, each CTA of the cluster owning a slice of the features.
//
// With theta = [W (F x C) | b (C)] the gradient is two thin matrix products per worker,
//     Z = X_B [W | W - W']   (B x F by F x 2C)   and   [dW | dD] = X_B^T [R | dR]   (F x B by B x 2C),
// joined by a row-wise softmax.  CTA r of the cluster keeps the columns [f0, f0 + nloc) of the B sampled rows in
// shared memory (read once from global memory) together with the matching rows of W and W - W', so that
//   forward   it forms the partial logits of ALL rows over its features (register tiles of 4 rows x CG columns; a
//             thread's rows are n_rt apart so that the lanes of a warp read different bank groups),
//   exchange  sends each row's partial logits to the CTA that owns the row (st.shared::cluster); the owner adds the
//             partials in rank order, forms P, (P - onehot)/B and the accurate difference
//             P_c - P'_c = P_c (T - e_c) / (1 + T), e_c = expm1(-dz_c), T = sum_j P_j e_j, and sends both residual
//             rows to every CTA of the cluster,
//   backward  forms its slice of g_m and d_m = g_m - g'_m from the SAME staged columns (tiles of 4 features x CG
//             columns), adds the regulariser and writes the slice to its final place (no partial slots, no second pass),
//   decision  reduces its part of the left-hand side of Eq. 6 / Eq. 8 / Eq. 4 in fp64 and sends it to rank 0, which
//             adds the parts in rank order, compares with (c/d_max) * window sum, applies the tau >= D clause and
//             writes the decision, the new staleness and the counters (Algorithm 1, worker side).
// The constant-1 column of the bias is the feature with index F and belongs to the last slice.
// The minibatch rows depend on the iteration number only, so the kernel takes k as an argument and fetches them before
// it waits for the preceding update kernel (programmatic dependent launch): DRAM latency overlaps with that kernel.
// One cluster barrier: start (every CTA is running and has armed its mbarriers before anything is stored into it; arrive at
// the top, wait before the first remote store).  The three exchanges (logits, residuals, norms) are asynchronous remote
// stores that credit an mbarrier of the receiving CTA with their bytes; the receiver waits for the byte count it expects.
#pragma once
#include "common.cuh"
#include "fused_small.cuh"
#include "fused_cluster.cuh"
#include "grad_stream.cuh"

namespace cada {

constexpr int SC_THREADS = 320;   // measured on 784 features x 10 classes, batch 64, 20 workers x 8 CTAs: 512 threads 20.7 us per
                                  // iteration, 448 20.4, 416 20.1, 384 19.6, 352 19.9, 320 19.3, 288 21.9, 256 22.1 -- two CTAs of 512
                                  // threads x 64 registers fill an SM's register file, so the second CTA of an SM could not start
                                  // beside the update kernel it is launched behind, and its cluster waited for it
constexpr int SC_MAX_NC = 8;

struct SoftmaxClusterGeom {
  int nc;          // CTAs per cluster (= per worker)
  int fs;          // features per slice (multiple of 4), the constant-1 column counted as a feature
  int pitch;       // floats between staged rows: fs rounded up to 4 modulo 8 (consecutive rows start in different bank groups)
  int Bp;          // batch rounded up to a multiple of 4
  int cgp;         // columns of [Z | dZ] per column group (4 groups): ceil(2C / 4), rounded up to an instantiated width
  int gp;          // floats a column group occupies in shared memory (4 or 8)
  int ncol;        // 4 * cgp
  int n_rt;        // row tiles (Bp / 4)
  int kg;          // ways the forward pass splits the features of a slice
  int n_ft;        // feature tiles of the backward pass (fs / 4)
  int ig;          // ways the backward pass splits the rows
  int rows_per;    // rows whose softmax one CTA computes
  unsigned smem_bytes;
  unsigned off_x, off_w, off_part, off_zin, off_r, off_lhs, off_red, off_rows, off_bar;
};

// Columns per column group the kernel is instantiated for: ceil(2C / 4) rounded up to one of {2, 4, 5, 6, 8}.
__host__ inline int softmax_cluster_cgp(int C) { const int g = (2 * C + 3) / 4; return g <= 2 ? 2 : g <= 4 ? 4 : g <= 5 ? 5 : g <= 6 ? 6 : 8; }

__host__ inline bool softmax_cluster_plan(int F, int C, int has_bias, int B, int nc, SoftmaxClusterGeom& g) {
  if (C < 2 || C > 16 || nc < 1 || nc > SC_MAX_NC || B < 1 || B > 1024) return false;
  const int nfeat = F + (has_bias ? 1 : 0);
  g.nc = nc;
  g.fs = ((nfeat + nc - 1) / nc + 3) / 4 * 4;
  if ((long long)g.fs * (nc - 1) >= nfeat) return false;             // the last CTA would own nothing: use fewer CTAs
  g.pitch = g.fs;
  while (g.pitch % 8 != 4) g.pitch += 4;
  g.Bp = (B + 3) / 4 * 4;
  g.cgp = softmax_cluster_cgp(C);
  g.gp = g.cgp <= 4 ? 4 : 8;
  g.ncol = 4 * g.cgp;
  g.n_rt = g.Bp / 4;
  const int ntile = g.n_rt * 4;
  if (ntile > SC_THREADS) return false;
  g.kg = SC_THREADS / ntile;
  if (g.kg > g.fs / 4) g.kg = g.fs / 4;
  g.n_ft = g.fs / 4;
  if (g.n_ft * 4 > SC_THREADS) return false;
  g.ig = SC_THREADS / (g.n_ft * 4);
  if (g.ig > g.Bp) g.ig = g.Bp;
  g.rows_per = (B + nc - 1) / nc;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = (o + bytes + 15) / 16 * 16; return (unsigned)at; };
  g.off_x = take((size_t)4 * g.Bp * g.pitch);
  g.off_w = take((size_t)4 * g.fs * 4 * g.gp);
  const size_t fw_part = (size_t)4 * g.kg * g.Bp * g.ncol, bw_part = (size_t)4 * g.ig * g.fs * g.ncol;
  g.off_part = take(fw_part > bw_part ? fw_part : bw_part);
  g.off_zin = take((size_t)4 * nc * g.rows_per * g.ncol);
  g.off_r = take((size_t)4 * g.Bp * 4 * g.gp);
  g.off_lhs = take(sizeof(double) * SC_MAX_NC);
  g.off_red = take(sizeof(double) * 32);
  g.off_rows = take(sizeof(long long) * g.Bp);
  g.off_bar = take(32);                                                // mbarriers: rows landed | logits | residuals | left-hand-side parts
  g.smem_bytes = (unsigned)o;
  return o <= 110 * 1024;                                             // two CTAs per SM stay possible
}

// CGP = columns per column group (ceil(2C/4)), GP = its padded width in shared memory.
template <int CGP>
__global__ void __launch_bounds__(SC_THREADS) grad_softmax_cluster_kernel(const __grid_constant__ Params P,
                                                                          const __grid_constant__ SoftmaxClusterGeom sg,
                                                                          long long k /* iteration, as the host counts it */) {
  constexpr int GP = CGP <= 4 ? 4 : 8;
  constexpr int NCOL = 4 * CGP;
  extern __shared__ __align__(16) unsigned char sm[];
  float* s_x = reinterpret_cast<float*>(sm + sg.off_x);       // [Bp][pitch] staged columns of the sampled rows
  float* s_w = reinterpret_cast<float*>(sm + sg.off_w);       // [fs][4][GP] rows of [W | W - W'], by column group
  float* s_part = reinterpret_cast<float*>(sm + sg.off_part); // forward: [kg][Bp][NCOL]; backward: [ig][fs][NCOL]
  float* s_zin = reinterpret_cast<float*>(sm + sg.off_zin);   // [nc][rows_per][NCOL] partial logits of the rows this CTA owns
  float* s_r = reinterpret_cast<float*>(sm + sg.off_r);       // [Bp][4][GP] residual rows [R | dR], by column group
  double* s_lhs = reinterpret_cast<double*>(sm + sg.off_lhs); // [nc] parts of the left-hand side (rank 0)
  double* s_red = reinterpret_cast<double*>(sm + sg.off_red);
  long long* s_rows = reinterpret_cast<long long*>(sm + sg.off_rows);   // [Bp] sampled row of each minibatch element

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int m = blockIdx.y;
  unsigned rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int F = P.F, C = P.C, nc = sg.nc, fs = sg.fs, pitch = sg.pitch, Bp = sg.Bp;
  const int nfeat = F + (P.has_bias ? 1 : 0);
  const int f0 = (int)rank * fs;
  const int nloc = min(fs, nfeat - f0);                       // features (incl. the constant-1 column) of this slice
  const int nx = min(fs, max(0, F - f0));                     // ... of which are columns of X
  const int Bm = worker_batch(P, m);
  const float* __restrict__ X = static_cast<const float*>(P.X[m]);
  const long long n_m = P.n_samples[m];
  const unsigned long long mu_m = ~0ull / (unsigned long long)n_m;
  const float* __restrict__ th = P.theta;
  const float* __restrict__ tho = old_iterate(P, k, m);
  pdl_trigger();                                               // the update kernel may be scheduled behind this one
  // mbarriers: `bar` counts the bulk copies of the sampled rows; the other three count the bytes the CTAs of the cluster
  // send one another (asynchronous remote stores credit the receiver's barrier: nobody waits for an acknowledgement, and
  // there is no cluster-wide barrier behind the exchanges).  Each is used once per launch.  They are initialised and
  // armed BEFORE this CTA arrives at the start barrier, so that whoever passes that barrier may send.
  const uint32_t bar = ptx::smem_u32(sm + sg.off_bar);
  const uint32_t bar_z = bar + 8u, bar_r = bar + 16u, bar_l = bar + 24u;
  bool dead = false;                                           // a bounded wait of this thread has run out
  if (tid == 0) {
    ptx::mbar_init(bar, 1); ptx::mbar_init(bar_z, 1); ptx::mbar_init(bar_r, 1); ptx::mbar_init(bar_l, 1);
    ptx::fence_barrier_init();
    const int my_rows = max(0, min(sg.rows_per, Bp - (int)rank * sg.rows_per));   // rows whose softmax this CTA computes
    fc_arrive_expect_tx(bar_z, (uint32_t)(nc * my_rows * sg.ncol * 4));             // their partial logits from every CTA
    fc_arrive_expect_tx(bar_r, (uint32_t)(Bm * C * 8));                             // (R, dR) of every live row and class
    fc_arrive_expect_tx(bar_l, (uint32_t)(nc * 8));                                 // (rank 0 waits for it) a part per CTA
  }
  fc_cluster_arrive();                                         // start barrier, first half: this CTA is running
  auto col_slot = [&](int j) { const int grp = j / CGP; return grp * GP + (j - grp * CGP); };   // column j of [Z | dZ] in a padded row

  // ---- stage: columns [f0, f0 + nx) of the sampled rows; zero elsewhere -----------------------------------------
  // One bulk copy per row brings the 16-byte-aligned part of the slice (it reports to an mbarrier); the few columns
  // beyond it, the padding and the rows beyond the worker's batch are written by the threads.
  const bool vec = (reinterpret_cast<uintptr_t>(X) % 16 == 0) && (P.ldx % 4 == 0);
  const int nx4 = vec ? (nx / 4) * 4 : 0;                      // columns of each row that arrive by bulk copy
  // explicit row indices may have been produced on this stream just before the call: they are read only after the
  // kernels before this one have completed (X and y never change while the handle lives)
  double rhs_early = 0.0;
  int tau_early = 0;
  if (P.idx_mode == IDX_EXPLICIT) pdl_wait();
  for (int i = tid; i < Bm; i += SC_THREADS) s_rows[i] = minibatch_row(P, k, m, i, n_m, mu_m);
  for (int c = tid; c < fs * 4 * GP; c += SC_THREADS) s_w[c] = 0.f;
  for (int c = tid; c < Bp * 4 * GP; c += SC_THREADS) s_r[c] = 0.f;
  __syncthreads();
  if (nx4 > 0) {
    if (tid == 0)
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)(Bm * nx4 * 4)) : "memory");
    // the lanes of a warp issue their bulk copies one after the other: spread the rows over the warps first
    for (int i = lane * (SC_THREADS / 32) + warp; i < Bm; i += SC_THREADS)
      ptx::bulk_g2s(ptx::smem_u32(s_x + (size_t)i * pitch), X + s_rows[i] * P.ldx + f0, (uint32_t)(nx4 * 4), bar);
  }
  {
    const int rem = pitch - nx4;                               // columns per row written by hand
    for (int c = tid; c < Bm * rem; c += SC_THREADS) {
      const int i = c / rem, j = nx4 + (c - i * rem);
      s_x[(size_t)i * pitch + j] = j < nx ? X[s_rows[i] * P.ldx + f0 + j] : 0.f;
    }
    for (int c = Bm * pitch + tid; c < Bp * pitch; c += SC_THREADS) s_x[c] = 0.f;
    // Everything above reads only the caller's data (X) and the iteration number: when this kernel was launched
    // behind a still-running update kernel it has overlapped with it.  From here on the iterates are read.
    pdl_wait();
    if (rank == 0 && tid == 0) tau_early = P.tau[m];                         // for the decision at the kernel's end
    if (rank == 0 && tid < 32) rhs_early = window_refresh_rhs(P, k, tid);     // the newest window term, if the update kernel left it in parts; then this iteration's right-hand side (thread 0 of rank 0 decides)
    // rows of [W | W - W'] for this slice (the bias row is row F of the same matrix)
    for (int c = tid; c < nloc * C; c += SC_THREADS) {
      const int f = c / C, cc = c - f * C;
      const float a = th[(long long)f0 * C + c], b = tho[(long long)f0 * C + c];
      s_w[f * 4 * GP + col_slot(cc)] = a;
      s_w[f * 4 * GP + col_slot(C + cc)] = a - b;
    }
    __syncthreads();
    if (P.has_bias && f0 + nloc == nfeat)                      // the constant-1 column lives in the last slice
      for (int i = tid; i < Bm; i += SC_THREADS) s_x[(size_t)i * pitch + (nloc - 1)] = 1.f;
    // bounded wait for the rows; a timeout is recorded and the kernel goes on so that the barriers stay paired
    if (nx4 > 0 && !ptx::mbar_wait_bounded(bar, 0u)) atomicOr(&P.st->status_flags, 4);
  }
  __syncthreads();                                             // staging complete

  // ---- forward: partial logits of all rows over this slice ------------------------------------------------------
  {
    const int ntile = sg.n_rt * 4;
    const int kgi = tid / ntile, t = tid - kgi * ntile;
    if (kgi < sg.kg) {
      const int rt = t >> 2, ct = t & 3;
      float acc[4][CGP];
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int j = 0; j < CGP; ++j) acc[r][j] = 0.f;
      const int nks = (nloc + 3) / 4;
      for (int ks = kgi; ks < nks; ks += sg.kg) {
        float4 xr[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) xr[r] = *reinterpret_cast<const float4*>(s_x + (size_t)(rt + sg.n_rt * r) * pitch + 4 * ks);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float* wp = s_w + (size_t)(4 * ks + e) * 4 * GP + ct * GP;
          const float4 w0 = *reinterpret_cast<const float4*>(wp);
          float4 w1 = make_float4(0.f, 0.f, 0.f, 0.f);
          if (GP == 8) w1 = *reinterpret_cast<const float4*>(wp + 4);
          const float w[8] = {w0.x, w0.y, w0.z, w0.w, w1.x, w1.y, w1.z, w1.w};
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const float xv = e == 0 ? xr[r].x : e == 1 ? xr[r].y : e == 2 ? xr[r].z : xr[r].w;
#pragma unroll
            for (int j = 0; j < CGP; ++j) acc[r][j] = fmaf(xv, w[j], acc[r][j]);
          }
        }
      }
#pragma unroll
      for (int r = 0; r < 4; ++r)
#pragma unroll
        for (int j = 0; j < CGP; ++j) s_part[((size_t)kgi * Bp + rt + sg.n_rt * r) * NCOL + ct * CGP + j] = acc[r][j];
    }
    __syncthreads();
    // start barrier, second half: every CTA of the cluster is running, so its shared memory may be stored into (the
    // wait was left until here so that the others' start-up hides behind the staging and the forward pass)
    fc_cluster_wait();
    // add the kg partial tiles and send each row's NCOL values to the CTA that owns the row
    for (int c = tid; c < Bp * CGP; c += SC_THREADS) {
      const int i = c / CGP, q = c - i * CGP;
      float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int g = 0; g < sg.kg; ++g) {
        const float4 a = *reinterpret_cast<const float4*>(s_part + ((size_t)g * Bp + i) * NCOL + 4 * q);
        v.x += a.x; v.y += a.y; v.z += a.z; v.w += a.w;
      }
      const int dest = min(i / sg.rows_per, nc - 1), il = i - dest * sg.rows_per;
      if (il < sg.rows_per)
        fc_st_async_f4(fc_map(s_zin + ((size_t)rank * sg.rows_per + il) * NCOL + 4 * q, (unsigned)dest), v,
                       fc_map_u32(bar_z, (unsigned)dest));
    }
  }
  fc_wait(bar_z, 0u, dead, &P.st->status_flags);               // the partial logits of this CTA's rows are here

  // ---- softmax of the rows this CTA owns; residual rows go to every CTA -------------------------------------------
  // SEG lanes (the class count rounded up to a power of two) share a row, lane c of a segment holding class c; the
  // row-wise maxima and sums are butterflies inside the segment.  All lanes run every round (the shuffles need them).
  {
    const int SEG = C <= 2 ? 2 : C <= 4 ? 4 : C <= 8 ? 8 : 16;
    const int rows_per_warp = 32 / SEG, rows_per_round = rows_per_warp * (SC_THREADS / 32);
    const int c = lane & (SEG - 1);
    const bool live_c = c < C;
    const float invB = 1.0f / (float)Bm;
    auto seg_max = [&](float v) { for (int o = SEG >> 1; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o)); return v; };
    auto seg_sum = [&](float v) { for (int o = SEG >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o); return v; };
    for (int il0 = 0; il0 < sg.rows_per; il0 += rows_per_round) {
      const int il = il0 + warp * rows_per_warp + lane / SEG;
      const int i = (int)rank * sg.rows_per + il;
      const bool live = il < sg.rows_per && i < Bm;
      float z = 0.f, dz = 0.f;
      if (live && live_c) {
        for (int src = 0; src < nc; ++src) {                     // partial logits in rank order
          z += s_zin[((size_t)src * sg.rows_per + il) * NCOL + c];
          dz += s_zin[((size_t)src * sg.rows_per + il) * NCOL + C + c];
        }
      }
      const int label = live ? static_cast<const int*>(P.y[m])[s_rows[i]] : 0;
      const float zmax = seg_max(live_c ? z : -INFINITY);
      const float dzmax = seg_max(live_c ? fabsf(dz) : 0.f);
      const float pc = live_c ? expf(z - zmax) : 0.f;
      const float inv = 1.f / seg_sum(pc);
      const float Pc = pc * inv;
      const float rr = (Pc - (c == label ? 1.f : 0.f)) * invB;
      // accurate difference P_c - P'_c = P_c (T - e_c) / (1 + T) while every |dz| of the row is moderate
      const float ec = live_c ? expm1f(-fminf(fmaxf(dz, -20.f), 20.f)) : 0.f;
      const float T = seg_sum(Pc * ec);
      float dd = Pc * (T - ec) / (1.f + T) * invB;
      if (__any_sync(0xffffffffu, dzmax > 20.f)) {               // rare: the two softmaxes are far apart, subtract them
        const float zo = z - dz;
        const float zomax = seg_max(live_c ? zo : -INFINITY);
        const float po = live_c ? expf(zo - zomax) : 0.f;
        const float deno = seg_sum(po);
        if (dzmax > 20.f) dd = (Pc - po / deno) * invB;
      }
      if (live && live_c) {
        float* pr = s_r + (size_t)i * 4 * GP + col_slot(c);
        float* pd = s_r + (size_t)i * 4 * GP + col_slot(C + c);
        for (int dest = 0; dest < nc; ++dest) {
          const uint32_t rb = fc_map_u32(bar_r, (unsigned)dest);
          fc_st_async_f32(fc_map(pr, (unsigned)dest), rr, rb);
          fc_st_async_f32(fc_map(pd, (unsigned)dest), dd, rb);
        }
      }
    }
  }
  fc_wait(bar_r, 0u, dead, &P.st->status_flags);               // the residual rows of the whole minibatch are here

  // ---- backward: this slice of g_m and d_m from the staged columns --------------------------------------------
  {
    const int ntile = sg.n_ft * 4;
    const int igi = tid / ntile, t = tid - igi * ntile;
    if (igi < sg.ig) {
      const int ft = t >> 2, ct = t & 3;
      float acc[4][CGP];
#pragma unroll
      for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int j = 0; j < CGP; ++j) acc[e][j] = 0.f;
#pragma unroll 2
      for (int i = igi; i < Bm; i += sg.ig) {
        const float4 x4 = *reinterpret_cast<const float4*>(s_x + (size_t)i * pitch + 4 * ft);
        const float* rp = s_r + (size_t)i * 4 * GP + ct * GP;
        const float4 r0 = *reinterpret_cast<const float4*>(rp);
        float4 r1 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (GP == 8) r1 = *reinterpret_cast<const float4*>(rp + 4);
        const float r[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
        const float xs[4] = {x4.x, x4.y, x4.z, x4.w};
#pragma unroll
        for (int e = 0; e < 4; ++e)
#pragma unroll
          for (int j = 0; j < CGP; ++j) acc[e][j] = fmaf(xs[e], r[j], acc[e][j]);
      }
#pragma unroll
      for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int j = 0; j < CGP; ++j) s_part[((size_t)igi * fs + 4 * ft + e) * NCOL + ct * CGP + j] = acc[e][j];
    }
    __syncthreads();
  }
  // add the row-split partials and the regulariser, write the slice, accumulate the left-hand side
  double acc = 0.0;
  {
    const bool cada1 = P.rule == 1, lag = P.rule == 3;
    float* __restrict__ gf = P.g_fresh + (long long)m * P.ldp + (long long)f0 * C;
    float* __restrict__ df = P.d_fresh + (long long)m * P.ldp + (long long)f0 * C;
    const float* __restrict__ ref = cada1 ? P.delta_stored + (long long)m * P.ldp + (long long)f0 * C
                                    : lag ? P.G + (long long)m * P.ldp + (long long)f0 * C : nullptr;
    for (int c = tid; c < nloc * C; c += SC_THREADS) {
      const int f = c / C, cc = c - f * C;
      float g = 0.f, d = 0.f;
      for (int h = 0; h < sg.ig; ++h) {
        g += s_part[((size_t)h * fs + f) * NCOL + cc];
        d += s_part[((size_t)h * fs + f) * NCOL + C + cc];
      }
      g = fmaf(P.lambda, s_w[f * 4 * GP + col_slot(cc)], g);
      d = fmaf(P.lambda, s_w[f * 4 * GP + col_slot(C + cc)], d);
      gf[c] = g;
      df[c] = d;
      const float e_ = cada1 ? d - ref[c] : lag ? g - ref[c] : d;
      acc = fma((double)e_, (double)e_, acc);
    }
  }
  acc = warp_sum(acc);
  if (lane == 0) s_red[warp] = acc;
  __syncthreads();
  if (tid == 0) {
    double part = 0.0;
#pragma unroll
    for (int w = 0; w < SC_THREADS / 32; ++w) part += s_red[w];
    fc_st_async_f64(fc_map(s_lhs + rank, 0u), part, fc_map_u32(bar_l, 0u));
  }
  if (rank != 0 || tid != 0) return;             // everything sent to this CTA has been waited for: it may leave
  fc_wait(bar_l, 0u, dead, &P.st->status_flags);

  // ---- rank 0: the decision (Algorithm 1, "if Eq. 6 / Eq. 8 is violated or tau >= D") --------------------------
  double lhs = 0.0;
  for (int r = 0; r < nc; ++r) lhs += s_lhs[r];
  const double rhs = rhs_early;                  // (c / d_max) * window sum, taken right after the wait for the update kernel
  const int tau = tau_early;
  const bool forced = tau >= P.D;
  const bool violated = !(lhs <= rhs);
  const bool up = violated || forced;
  const unsigned char bits = (unsigned char)((up ? 1 : 0) | (forced ? 2 : 0));
  P.mask[m] = bits;
  P.lhs[m] = lhs;
  P.tau[m] = up ? 1 : tau + 1;
  if (up) {
    atomicAdd((unsigned long long*)&P.st->uploads_total, 1ull);
    atomicAdd((unsigned long long*)(forced ? &P.st->uploads_forced : &P.st->uploads_rule), 1ull);
    atomicAdd((unsigned long long*)&P.up_per_worker[m], 1ull);
  }
  if (!isfinite(lhs) || isnan(rhs)) atomicOr(&P.st->status_flags, 1);
  if (!isinf(rhs)) {
    const double big = fmax(lhs, rhs);
    if (fabs(lhs - rhs) <= 1e-4 * big && big > 0.0) atomicAdd((unsigned long long*)&P.st->near_ties, 1ull);
  }
  if (m == 0) P.st->last_rhs = rhs;
  if (P.hist_cap > 0) {
    const long long slot = k % P.hist_cap;
    P.hist_lhs[slot * P.M + m] = lhs;
    P.hist_mask[slot * P.M + m] = bits;
    if (m == 0) P.hist_rhs[slot] = rhs;
  }
}

}  // namespace cada
