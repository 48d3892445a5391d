// Whole CADA iterations in one launch for small binary-logistic problems whose workers fit into ONE
// thread-block cluster (up to 16 CTAs x 4 workers): the exchange between "workers" and "server" that
// Algorithm 1 performs once per iteration goes through distributed shared memory -- asynchronous remote
// stores that credit an mbarrier of the receiving CTA -- instead of through L2 and a polled flag array.
//
// A CTA holds W workers.  Each worker is served by a group of 224 compute threads with its own named
// barrier plus one producer warp that does nothing but fetch minibatches.  Every CTA keeps, in shared
// memory, a full copy of the server state (theta, h, vhat, the window of squared step norms) and of the
// M gradient slots G_m in two buffers with one selector bit per worker.
//
// Per iteration k (Algorithm 1):
//   producer the worker's producer warp hashes iteration k+1's row indices and copies those rows and
//            labels (cp.async) into the other half of a double buffer; the copies report to that half's
//            mbarrier.  Rows do not depend on theta, so DRAM latency and the cost of issuing a few hundred
//            16-byte copies stay off the compute threads' path.  A second, CTA-local mbarrier per half tells
//            the producer that the half has been read (the group's first thread arrives after the backward pass)
//   worker   forward and backward in one of two forms (two passes over the staged rows, or register-tiled: see
//            ClusterGeom::nch; the group's last thread forms the right-hand side of Eqs. 6 / 8 meanwhile), g_m, d_m
//            (four lanes per coordinate), left-hand side in fp64; every thread then takes the decision, tau >= D clause
//            included, from the same numbers, so it need not be handed round
//   upload   EVERY worker sends its fresh gradient to EVERY CTA of the cluster, into the slot buffer that is not the
//            worker's current one, plus its (decision, selector) word into the flag array of this iteration's parity:
//            st.async remote stores whose bytes are credited to the receiver's mbarrier of this iteration's parity.
//            An upload flips the selector, which makes that buffer the current one; after a skip it is never read.
//            Sending always -- about three workers in four skip -- is what makes the byte count of an iteration a
//            constant, M * (16 * quads + 4), that each receiver can wait for
//   wait     every compute thread waits for that count on its own CTA's mbarrier: no release fence in the senders (the
//            fence before a hardware cluster barrier waited ~1,000 cycles for the remote stores to be acknowledged),
//            no cluster-wide barrier, nothing polled in global memory
//   server   every CTA sums the M current slots from its own shared memory (4 threads per coordinate, fixed
//            order) and applies Eqs. 2a-2c to its copy of the server state (redundantly: nothing is broadcast);
//            the same thread writes theta - theta' for the next iteration of each of the CTA's workers and
//            refreshes the CADA1 snapshot.  One CTA-wide barrier ends the iteration; none opens the next
// Why this is enough: a CTA that runs ahead into iteration k+1 stores only into slot buffers that laggards (still in
// the server phase of k) do not read, into the flag array of the other parity, and credits the mbarrier of the other
// parity; it cannot get two iterations ahead, because completing k+1 takes every CTA's messages of k+1, which a laggard
// sends only after its server phase of k.  Every CTA has received everything sent to it when its loop ends; a cluster
// barrier before the exit (arrive after the loop, wait after the write-back) keeps all CTAs alive until then.
// Every wait is bounded in clock cycles; after the first one that runs out a thread stops waiting altogether, so a
// launch in which something went wrong ends quickly with the timeout flag raised.
// Global state is read at kernel start and written back at the end, in the layout every other path uses.
// STREAM = true is the form for minibatches that arrive from the caller's page-locked host memory (cada_step_host_n): the
// producer warps read step i's rows from the caller's buffers over the bus, three buffers deep and two iterations ahead
// (a fetch over the bus takes about two iterations), and each iteration stores its theta and upload mask into the caller's
// output buffers.  The arithmetic and its order are those of the resident form.
#pragma once
#include "common.cuh"
#include "fused_small.cuh"
#include "grad_stream.cuh"

namespace cada {

constexpr int FC_GROUP = 224;      // compute threads that serve one worker
constexpr int FC_GWARPS = FC_GROUP / 32;
constexpr int FC_MAX_W = 4;        // workers per CTA
constexpr int FC_MAX_CTAS = 16;    // CTAs of the cluster (above 8 needs the non-portable opt-in)
constexpr int FC_SRV = 4;          // threads that share one coordinate's slot sum in the server phase
constexpr int FC_MASK_STEPS = 16;  // streamed form: steps whose upload masks go to the caller's buffer in one piece

// Minibatches streamed from the caller's page-locked host memory (cada_step_host_n): step i of the launch takes rows
// 0..B-1 of block (i * M + m) of `x` / `y`, fetched over the bus by the producer warps one iteration ahead, and hands
// theta^{k+1} and the upload mask of the step to `out_theta` / `out_mask` (posted stores).  All four are addresses the
// device can use for that host memory; x == nullptr: the handle's resident data and its index stream are used.
struct HostStream {
  const float* x;            // [n][M][B][ldx]
  const float* y;            // [n][M][B]
  float* out_theta;          // [n][p] or nullptr
  unsigned char* out_mask;   // [n][M] or nullptr
};

struct ClusterGeom {
  int ncta, W;
  int pp;          // p rounded up to a multiple of 4
  int pitch;       // floats between staged rows (multiple of 4)
  int f4;          // 16-byte chunks per row
  int nqb;         // quads of theta
  int nrg;         // row groups of the backward pass (nqb * nrg <= FC_GROUP)
  int T;           // threads per row in the forward pass (1, 2, 4 or 8)
  int Mp;          // M rounded up to a multiple of 4
  int nch;         // 0: forward and backward as separate passes over the staged rows (T threads per row, then a thread per
                   // (quad, row group)).  1: the register-tiled form -- a thread keeps 4 rows x nch quads of the minibatch in
                   // registers for both passes; `tl` lanes (8, 16 or 32) share a group of 4 rows, nrg = ceil(B / 4) such groups
  int tl;
  int nbuf;        // minibatch buffers per worker: 2 (resident data, prefetch one iteration ahead) or 3 (streamed from host
                   // memory, two iterations ahead: a fetch over the bus outlasts an iteration)
  unsigned smem_bytes;
  // CTA-wide regions (byte offsets into dynamic shared memory)
  unsigned off_ring, off_stepred, off_theta, off_h, off_vhat, off_G, off_flags, off_maskout, off_rxbar, off_grp, grp_bytes;
  // offsets inside one group's region
  unsigned g_red, g_old, g_dth, g_dst, g_g, g_d, g_part, g_res, g_rows, g_y, g_x, g_misc, g_bar, g_cons, g_rhs;
};

// `ncta` may exceed ceil(M / W): the CTAs beyond the last worker idle through the worker phase and take
// part in the barrier and the (redundant) server phase only.
__host__ inline bool cluster_plan(int F, int has_bias, int B, int d_max, int rule, int M, int W, int ncta, ClusterGeom& g,
                                  int nbuf = 2, long long stream_ldx = 0, bool tiled = true) {
  const int p = F + has_bias;
  if (F > 508 || B > 1024 || W < 1 || W > FC_MAX_W || M < 1) return false;
  if (ncta > FC_MAX_CTAS || (long long)ncta * W < M) return false;
  g.W = W;
  g.ncta = ncta;
  g.nbuf = nbuf;
  g.pp = (p + 3) / 4 * 4;
  g.f4 = (F + 3) / 4;
  g.T = 1;
  while (g.T < 8 && 2 * g.T * B <= FC_GROUP && 2 * g.T <= g.f4) g.T *= 2;
  // chunk pitch congruent to T modulo 8 (odd for T = 1): the 8 threads of a quarter warp -- 8/T rows x T
  // parts -- then read 8 different 16-byte bank groups in the forward pass
  int p4 = g.f4;
  if (g.T == 1) p4 |= 1;
  else if (g.T < 8) while (p4 % 8 != g.T) ++p4;
  g.pitch = p4 * 4;
  // streamed minibatches whose rows are (nearly) as wide as the staged pitch keep the caller's row pitch instead: a worker's
  // block is then one contiguous piece and arrives with ONE bulk copy (the fetch over the bus, not the forward pass's
  // bank conflicts, bounds a streamed iteration)
  if (nbuf > 2 && stream_ldx >= 4 * g.f4 && stream_ldx % 4 == 0 && stream_ldx <= g.pitch) g.pitch = (int)stream_ldx;
  g.nqb = g.pp / 4;
  g.nrg = FC_GROUP / g.nqb;
  if (g.nrg < 1) g.nrg = 1;
  if (g.nrg > 32) g.nrg = 32;
  if (g.nrg > B) g.nrg = B;
  // register-tiled worker phase where 4-row groups x lanes fit the worker's threads (and the register budget: W <= 2).
  // Measured: one quad per lane (22 features, batch 32, 10 workers) 2.53 -> 2.35 us per iteration; two quads per lane
  // (54 features, batch 100, 20 workers; 128 registers) 4.27 -> 4.33 us, so only the former is offered
  g.nch = 0; g.tl = 0;
  if (tiled && W <= 2) {
    for (int nch = 1; nch <= 1 && g.nch == 0; ++nch) {
      int tl = 8;
      while (tl * nch < g.nqb) tl *= 2;
      const int groups = (B + 3) / 4;
      if (tl <= 32 && groups * tl <= FC_GROUP) { g.nch = nch; g.tl = tl; g.nrg = groups; }
    }
    // a quarter warp reads 128 consecutive bytes of one row whatever the pitch: rows are staged back to back
    if (g.nch) {
      g.pitch = g.f4 * 4;
      if (nbuf > 2 && stream_ldx % 4 == 0 && stream_ldx >= g.pitch && stream_ldx <= g.pitch + 16) g.pitch = (int)stream_ldx;
    }
  }
  g.Mp = (M + 3) / 4 * 4;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = (o + bytes + 15) / 16 * 16; return (unsigned)at; };
  g.off_ring = take(sizeof(double) * (d_max + 2));                 // window | RHS | last step norm
  g.off_stepred = take(sizeof(double) * 32);
  g.off_theta = take(4 * g.pp); g.off_h = take(4 * g.pp); g.off_vhat = take(4 * g.pp);
  g.off_G = take((size_t)4 * 2 * M * g.pp);
  g.off_flags = take((size_t)4 * 2 * g.Mp);
  g.off_maskout = take(nbuf > 2 ? (size_t)FC_MASK_STEPS * g.Mp : 0);  // streamed: upload masks of the last steps, flushed together
  g.off_rxbar = take(16);                                         // two mbarriers: "iteration's slots and decision words have arrived"
  g.off_grp = take(0);
  const size_t base = o;
  o = 0;
  g.g_red = take(sizeof(double) * 8);
  g.g_old = take(4 * g.pp); g.g_dth = take(4 * g.pp);
  g.g_dst = take(rule == 1 ? 4 * g.pp : 0);
  g.g_g = take(4 * g.pp); g.g_d = take(4 * g.pp);
  g.g_part = take((size_t)4 * g.nrg * 2 * g.pp);
  g.g_res = take((size_t)4 * 2 * B);
  g.g_rows = take((size_t)8 * B);
  g.g_y = take((size_t)4 * nbuf * B);
  g.g_x = take((size_t)4 * nbuf * B * g.pitch);
  g.g_misc = take(16);
  g.g_bar = take(32);                                              // one mbarrier per minibatch buffer
  g.g_cons = take(32);                                             // one mbarrier per minibatch buffer: "has been read"
  g.g_rhs = take(16);                                              // right-hand side of this iteration, per group
  g.grp_bytes = (unsigned)o;
  const size_t total = base + (size_t)W * o;
  g.smem_bytes = (unsigned)total;
  return total <= (nbuf > 2 ? 224 : 200) * 1024;
}

__device__ __forceinline__ void fc_group_sync(int gi) {
  asm volatile("bar.sync %0, %1;" ::"r"(gi + 1), "n"(FC_GROUP) : "memory");
}
template <int W>
__device__ __forceinline__ void fc_compute_sync() {                // all compute threads of the CTA (not the producers)
  asm volatile("bar.sync 8, %0;" ::"n"(FC_GROUP * W) : "memory");
}
// Address of this CTA's shared-memory object `p` in the CTA of rank `rank` of the cluster.
__device__ __forceinline__ uint32_t fc_map(const void* p, unsigned rank) {
  const uint32_t la = (uint32_t)__cvta_generic_to_shared(p);
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(la), "r"(rank));
  return ra;
}
__device__ __forceinline__ uint32_t fc_map_u32(uint32_t la, unsigned rank) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(la), "r"(rank));
  return ra;
}
__device__ __forceinline__ void fc_store_f4(uint32_t ra, float4 v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(ra), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void fc_store_u32(uint32_t ra, unsigned v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(ra), "r"(v) : "memory");
}
// Asynchronous remote stores: the value lands in the destination CTA's shared memory and its byte count is credited to the
// mbarrier `rbar` of that CTA (both addresses are shared::cluster addresses of the SAME CTA).  The sender does not wait.
__device__ __forceinline__ void fc_st_async_f4(uint32_t ra, float4 v, uint32_t rbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];"
               ::"r"(ra), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w), "r"(rbar) : "memory");
}
__device__ __forceinline__ void fc_st_async_u32(uint32_t ra, unsigned v, uint32_t rbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.u32 [%0], %1, [%2];" ::"r"(ra), "r"(v), "r"(rbar) : "memory");
}
__device__ __forceinline__ void fc_st_async_f32(uint32_t ra, float v, uint32_t rbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f32 [%0], %1, [%2];" ::"r"(ra), "f"(v), "r"(rbar) : "memory");
}
__device__ __forceinline__ void fc_st_async_f64(uint32_t ra, double v, uint32_t rbar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.f64 [%0], %1, [%2];" ::"r"(ra), "d"(v), "r"(rbar) : "memory");
}
__device__ __forceinline__ void fc_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for a phase of an mbarrier.  The bound is in clock cycles (about 70 ms); once a wait of this thread has run
// out, `dead` makes its later waits return at once, so that a launch in which something went wrong still ends quickly (with
// the timeout flag raised) instead of running every remaining iteration into the bound.
constexpr long long FC_WAIT_CYCLES = 1ll << 27;
__device__ __forceinline__ void fc_wait(uint32_t bar, uint32_t parity, bool& dead, int* status_flags) {
  if (dead) return;
  if (ptx::mbar_try_wait(bar, parity)) return;
  const long long t0 = clock64();
  while (!ptx::mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > FC_WAIT_CYCLES) { dead = true; atomicOr(status_flags, 4); return; }
  }
}
__device__ __forceinline__ void fc_cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void fc_cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// The mbarrier at `bar` receives one arrival once every cp.async this thread has issued so far has landed.
__device__ __forceinline__ void fc_copies_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

template <int W, bool STREAM = false, int NCH = 0>
__global__ void __launch_bounds__((FC_GROUP + 32) * W, 1)
fused_cluster_kernel(const __grid_constant__ Params P, const __grid_constant__ ClusterGeom cg, int n_iters,
                     long long k0 /* first iteration of this launch, as the host counts it */,
                     const __grid_constant__ HostStream hs) {
  // Launched with programmatic serialisation: consecutive calls overlap -- while the previous launch writes its state
  // back, this one sets up, and its producer warps hash and fetch the first minibatch (which depends on k0 and on the
  // caller's data only); the state is read after the wait for the previous launch.
  pdl_trigger();
  extern __shared__ __align__(16) unsigned char sm[];
  constexpr int NTHR = FC_GROUP * W, NWARP = NTHR / 32;             // compute threads / warps of the CTA
  constexpr int NB = STREAM ? 3 : 2;                                // minibatch buffers per worker (= cg.nbuf)
  const int tid = threadIdx.x;
  const bool producer = tid >= NTHR;
  const int gi = producer ? (tid - NTHR) >> 5 : tid / FC_GROUP;      // worker group this thread serves
  const int tg = producer ? (tid & 31) : tid - gi * FC_GROUP;        // index inside the group (producer: lane)
  unsigned rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int M = P.M, B = P.B, F = P.F, p = (int)P.p;
  const int m = (int)rank * W + gi;
  const bool active = m < M;                          // a group beyond the last worker only helps the server phase
  const bool cada1 = P.rule == 1;

  double* s_ring = reinterpret_cast<double*>(sm + cg.off_ring);       // [d_max] window, [d_max] = RHS of this iteration
  double* s_stepred = reinterpret_cast<double*>(sm + cg.off_stepred); // per-warp partials of the squared step norm
  float* s_theta = reinterpret_cast<float*>(sm + cg.off_theta);
  float* s_h = reinterpret_cast<float*>(sm + cg.off_h);
  float* s_vhat = reinterpret_cast<float*>(sm + cg.off_vhat);
  float* s_G = reinterpret_cast<float*>(sm + cg.off_G);               // [2][M][pp]
  unsigned* s_flags = reinterpret_cast<unsigned*>(sm + cg.off_flags); // [2][Mp]: bit0 upload, bit1 forced, bit2 selector
  unsigned char* s_maskout = sm + cg.off_maskout;                     // (streamed) [FC_MASK_STEPS][M]
  unsigned char* gs = sm + cg.off_grp + (size_t)gi * cg.grp_bytes;
  double* s_red = reinterpret_cast<double*>(gs + cg.g_red);
  float* s_old = reinterpret_cast<float*>(gs + cg.g_old);             // theta': theta_hat_m (CADA2) or the snapshot (CADA1)
  float* s_dth = reinterpret_cast<float*>(gs + cg.g_dth);             // theta - theta'
  float* s_dst = reinterpret_cast<float*>(gs + cg.g_dst);             // CADA1: innovation stored at the last upload
  float* s_g = reinterpret_cast<float*>(gs + cg.g_g);
  float* s_d = reinterpret_cast<float*>(gs + cg.g_d);
  float* s_part = reinterpret_cast<float*>(gs + cg.g_part);           // [nrg][2][pp]
  float* s_res = reinterpret_cast<float*>(gs + cg.g_res);             // [2][B]: r | dr
  long long* s_rows = reinterpret_cast<long long*>(gs + cg.g_rows);   // [B] producer's scratch: element offsets of the rows
  float* s_y = reinterpret_cast<float*>(gs + cg.g_y);                 // [NB][B]
  float* s_x = reinterpret_cast<float*>(gs + cg.g_x);                 // [NB][B][pitch]
  const uint32_t bar_x = ptx::smem_u32(gs + cg.g_bar);                // "minibatch has landed", + 8 * buffer
  double* s_rhs = reinterpret_cast<double*>(gs + cg.g_rhs);           // right-hand side of Eqs. 6 / 8 for this iteration
  const uint32_t bar_cons = ptx::smem_u32(gs + cg.g_cons);            // "minibatch buffer has been read", + 8 * buffer
  const uint32_t bar_rx = ptx::smem_u32(sm + cg.off_rxbar);           // "all slots and decision words of the iteration are here", + 8 * (it & 1)
  bool dead = false;                                                  // a bounded wait of this thread has run out

  const int mm = active ? m : 0;
  const float* __restrict__ Xm = static_cast<const float*>(P.X[mm]);
  const float* __restrict__ ym = static_cast<const float*>(P.y[mm]);
  const long long n_m = P.n_samples[mm];
  const unsigned long long mu_m = ~0ull / (unsigned long long)n_m;
  const int Bm = worker_batch(P, mm);
  const size_t slot_buf = (size_t)M * cg.pp;          // floats per slot buffer

  if (tid == 0) {
    for (int g = 0; g < W; ++g) {
      const uint32_t b = ptx::smem_u32(sm + cg.off_grp + (size_t)g * cg.grp_bytes + cg.g_bar);
      for (int i = 0; i < NB; ++i) ptx::mbar_init(b + 8u * i, 32);   // one arrival per producer lane
      const uint32_t c = ptx::smem_u32(sm + cg.off_grp + (size_t)g * cg.grp_bytes + cg.g_cons);
      for (int i = 0; i < NB; ++i) ptx::mbar_init(c + 8u * i, 1);    // the group's first thread, after the backward pass
    }
    ptx::mbar_init(bar_rx, 1);                        // this thread, with the byte count of an iteration's messages
    ptx::mbar_init(bar_rx + 8u, 1);
    ptx::fence_barrier_init();
  }
  __syncthreads();                                    // mbarriers initialised (reached before anyone waits for the previous launch)
  // Start barrier, first half: this CTA runs and its mbarriers exist.  Waited for before the first iteration, so that the
  // barrier completes while the launch still waits for its predecessor.  What the first iteration's messages touch in a
  // peer -- the second slot buffer, the flag array, the mbarrier of parity 0 -- is not written by the state load below
  fc_cluster_arrive();

  // ================================ producer warps ================================================
  if (producer) {
    // Minibatch of iteration k into half `buf`: row offsets and labels first (one row per lane and pass), then the
    // rows in 16-byte pieces, consecutive lanes on consecutive pieces.
    auto fetch = [&](long long k, int buf) {
      float* xb = s_x + (size_t)buf * B * cg.pitch;
      if constexpr (STREAM) {
        // streamed: rows 0..B-1 of this step's block of the caller's page-locked host memory, one bulk copy per row (and
        // one for the labels where their block is a whole number of 16-byte pieces).  Bulk copies read host memory over
        // the bus at the full rate (51 GB/s measured here); 16-byte cp.async pieces whose completion a later instruction
        // of the same warp tracks reached 24-37 GB/s.
        const long long blk = ((k - k0) * M + m) * (long long)B;
        const float* __restrict__ Xk = hs.x + blk * P.ldx;
        const float* __restrict__ yk = hs.y + blk;
        const uint32_t bar = bar_x + 8u * buf;
        const uint32_t row_bytes = (uint32_t)cg.f4 * 16u;
        const bool ybulk = (B & 3) == 0 && (reinterpret_cast<uintptr_t>(hs.y) & 15) == 0;
        const uint32_t ybytes = (uint32_t)((Bm + 3) / 4) * 16u;
        const bool whole = (long long)cg.pitch == P.ldx;     // staged pitch == caller's pitch: the block is one piece
        const uint32_t xbytes = whole ? (uint32_t)Bm * (uint32_t)cg.pitch * 4u : (uint32_t)Bm * row_bytes;
        if (tg == 0) ptx::mbar_expect_tx(bar, xbytes + (ybulk ? ybytes : 0u));
        __syncwarp();
        if (ybulk) {
          if (tg == 0) ptx::bulk_g2s(ptx::smem_u32(&s_y[buf * B]), yk, ybytes, bar);
        } else {
          for (int j = tg; j < Bm; j += 32) cp_async4(&s_y[buf * B + j], yk + j);
        }
        if (whole) {
          if (tg == 1) ptx::bulk_g2s(ptx::smem_u32(xb), Xk, xbytes, bar);
        } else {
          for (int j = tg; j < Bm; j += 32)
            ptx::bulk_g2s(ptx::smem_u32(xb + (size_t)j * cg.pitch), Xk + (long long)j * P.ldx, row_bytes, bar);
        }
        if (ybulk) ptx::mbar_arrive(bar);
        else fc_copies_arrive(bar);                   // this lane's arrival, once its 4-byte label copies have landed
      } else {
        for (int j = tg; j < Bm; j += 32) {
          const long long row = minibatch_row(P, k, m, j, n_m, mu_m);
          s_rows[j] = row * P.ldx;
          cp_async4(&s_y[buf * B + j], ym + row);
        }
        __syncwarp();
        int j = tg / cg.f4, q = tg - j * cg.f4;
        const int dj = 32 / cg.f4, dq = 32 - dj * cg.f4;
        while (j < Bm) {
          cp_async16(xb + (size_t)j * cg.pitch + 4 * q, Xm + s_rows[j] + 4 * q);
          j += dj; q += dq;
          if (q >= cg.f4) { q -= cg.f4; ++j; }
        }
        fc_copies_arrive(bar_x + 8u * buf);
      }
      __syncwarp();                                   // s_rows is rewritten by the next fetch
    };
    // the first minibatch depends on k0 and the caller's data only: it is fetched while the compute threads still wait
    // for the previous launch and load the state
    if (!STREAM && P.idx_mode == IDX_EXPLICIT) pdl_wait();   // explicit indices may have been produced on this stream just before
    if (active && n_iters > 0) fetch(k0, 0);
    if (STREAM && active && n_iters > 1) fetch(k0 + 1, 1);
    fc_cluster_wait();
    int nxt = STREAM ? 2 : 1;                         // buffer of the next fetch
    int cb = 0;                                       // buffer iteration it - 1 used, and the parity of its "has been read"
    uint32_t cpar = 0;
    for (int it = 0; it < n_iters; ++it) {
      // the buffer filled now was last read in iteration it - 1: the group's first thread says so after the backward
      // pass.  With two buffers it receives iteration it + 1, with three (streamed) iteration it + 2
      const bool more = STREAM ? it + 2 < n_iters : it + 1 < n_iters;
      if (active && more) {
        if (it >= 1) fc_wait(bar_cons + 8u * cb, cpar, dead, &P.st->status_flags);
        fetch(k0 + it + (STREAM ? 2 : 1), nxt);
      }
      if (it >= 1 && ++cb == NB) { cb = 0; cpar ^= 1u; }
      if (++nxt == NB) nxt = 0;
    }
    cp_async_wait<0>();
    fc_cluster_arrive();                              // no CTA leaves while messages to or from it may be in flight
    fc_cluster_wait();
    return;
  }

  // ================================ compute threads ===============================================
  // ---- load state ------------------------------------------------------------------------------
  pdl_wait();                                         // the previous launch has written its state back
  for (int j = tid; j < cg.pp; j += NTHR) {
    const bool in = j < p;
    s_theta[j] = in ? P.theta[j] : 0.f;
    s_h[j] = in ? P.h[j] : 0.f;
    s_vhat[j] = in ? P.vhat[j] : 0.f;
  }
  for (int c = tid; c < M * cg.pp; c += NTHR) {       // buffer 0 holds every worker's current slot at start
    const int w = c / cg.pp, j = c - w * cg.pp;
    s_G[c] = j < p ? P.G[(long long)w * P.ldp + j] : 0.f;   // (the second buffer is read only after a message has filled it)
  }
  for (int j = tid; j < P.d_max; j += NTHR) s_ring[j] = P.ring[j];
  if (active) {
    for (int j = tg; j < cg.pp; j += FC_GROUP) {
      const bool in = j < p;
      s_old[j] = in ? (cada1 ? P.theta_tilde[j] : P.theta_hat[(long long)m * P.ldp + j]) : 0.f;
      if (cada1) s_dst[j] = in ? P.delta_stored[(long long)m * P.ldp + j] : 0.f;
      s_g[j] = 0.f; s_d[j] = 0.f;
    }
  }
  int tau = active ? P.tau[m] : 0;
  unsigned sel = 0;                                   // which slot buffer holds worker m's current gradient
  long long n_up = 0, n_forced = 0, n_ties = 0;       // (thread 0 of the group reports them)
  double last_lhs = 0.0, last_rhs = 0.0;
  unsigned char last_bits = 0;

  // per-thread constants of the forward pass: part `fw_t` of row `fw_j0 + pass * rows_per_pass`
  const int T = cg.T, fw_t = tg & (T - 1), fw_j0 = tg / T, fw_rows = FC_GROUP / T;
  // ... and of the backward pass: quad q of theta, row group rg
  const int bw_rg = tg / cg.nqb, bw_q = tg - bw_rg * cg.nqb;
  const bool bw_active = bw_rg < cg.nrg;
  int bw_kind[4];                                     // 0: feature column, 1: the constant-1 column, 2: padding
#pragma unroll
  for (int e = 0; e < 4; ++e) { const int c = 4 * bw_q + e; bw_kind[e] = c < F ? 0 : (c == F && P.has_bias) ? 1 : 2; }
  // ... and of the register-tiled form (NCH > 0): lane `tl_t` of the `tl` lanes that share row group `tl_rg` owns quads
  // tl_t, tl_t + tl, ...; tl_fix has two bits per column of each owned quad (0: feature, 1: the constant-1 column, 2: padding)
  const int TL = NCH > 0 ? cg.tl : 1;
  const int tl_t = tg & (TL - 1), tl_rg = NCH > 0 ? tg / TL : 0;
  unsigned tl_fix = 0;
  if constexpr (NCH > 0) {
#pragma unroll
    for (int i = 0; i < NCH; ++i)
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int c = 4 * (tl_t + i * TL) + e;
        tl_fix |= (unsigned)(c < F ? 0 : (c == F && P.has_bias) ? 1 : 2) << (8 * i + 2 * e);
      }
  }
  // ... and of the server phase: FC_SRV consecutive lanes share coordinate sv_j and take workers sv_w, sv_w + FC_SRV, ...
  const int sv_w = tid & (FC_SRV - 1), sv_j0 = tid / FC_SRV;

  const double c_over_d = (double)P.c / (double)P.d_max;
  int ring_pos = (int)(k0 % P.d_max);                 // slot of the window that iteration k's step norm goes to
  int snap_ctr = (int)(k0 % P.D);                     // k mod D, kept without divisions
  int hist_pos = P.hist_cap > 0 ? (int)(k0 % P.hist_cap) : 0;

  fc_compute_sync<W>();                               // state loaded (compute threads only: the producers are fetching)
  if (active) {
    // theta - theta' for the first iteration, with Algorithm 1's snapshot step (CADA1): theta~ <- theta^k before the
    // gradients when k mod D == 0.  Later iterations get both from the server phase of the iteration before.
    const bool snap = cada1 && snap_ctr == 0;
    for (int j = tg; j < cg.pp; j += FC_GROUP) {
      if (snap) s_old[j] = s_theta[j];
      s_dth[j] = s_theta[j] - s_old[j];
    }
  }
  // start barrier, second half: every CTA of the cluster is running and has initialised its mbarriers
  fc_cluster_wait();

  int sbuf = 0, spar = 0;                             // (streamed) running buffer index and parity
  for (int it = 0; it < n_iters; ++it) {
    const long long k = k0 + it;
    int buf, par;                                     // minibatch buffer of this iteration and the parity of its mbarrier
    if constexpr (STREAM) { buf = sbuf; par = spar; if (++sbuf == NB) { sbuf = 0; spar ^= 1; } }
    else { buf = it & 1; par = (it >> 1) & 1; }
    // this iteration's minibatch has landed (bounded wait; a timeout is recorded and the iteration goes on so
    // that the barriers stay paired).  theta, theta - theta' and the step-norm partials were written before the
    // barrier that ended the iteration before: no barrier is needed here.
    if (active && !ptx::mbar_wait_bounded(bar_x + 8u * buf, (uint32_t)par)) atomicOr(&P.st->status_flags, 4);
    // this iteration's messages: every worker sends its slot (nqb quads) and its decision word to every CTA
    if (tid == 0) fc_arrive_expect_tx(bar_rx + 8u * (it & 1), (uint32_t)M * (uint32_t)(cg.nqb * 16 + 4));

    if (active) {
      if (tg == FC_GROUP - 1) {
        // right-hand side of Eqs. 6 / 8: the window in slot order, its newest entry (the squared step norm of the
        // iteration before, per-warp partials added in a fixed order) taken from the partials; every group forms the
        // same value and stores the same entry
        const int newest = ring_pos == 0 ? P.d_max - 1 : ring_pos - 1;
        double snew = 0.0;
        if (it > 0) {
#pragma unroll
          for (int w = 0; w < NWARP; ++w) snew += s_stepred[w];
        }
        double rhs;
        if (isinf(P.c)) rhs = (double)INFINITY;
        else {
          double w = 0.0;
          for (int i = 0; i < P.d_max; ++i) w += (it > 0 && i == newest) ? snew : s_ring[i];
          rhs = c_over_d * w;
        }
        if (it > 0) s_ring[newest] = snew;
        s_rhs[0] = rhs;
      }
      // ---- worker: forward, T threads per minibatch row ---------------------------------------
      const float* xb = s_x + (size_t)buf * B * cg.pitch;
      const float invB = 1.0f / (float)Bm;
      const int qfull = F >> 2;                          // chunks whose four columns are all features
      if constexpr (NCH == 0) {
        for (int j0 = 0; j0 < Bm; j0 += fw_rows) {         // uniform trip count: the shuffles below need whole warps
          const int j = j0 + fw_j0;
          float z = 0.f, dz = 0.f;
          if (j < Bm) {
            const float4* xr = reinterpret_cast<const float4*>(xb + (size_t)j * cg.pitch);
  #pragma unroll 4
            for (int q = fw_t; q < qfull; q += T) {
              const float4 x = xr[q];
              const float4 t = reinterpret_cast<const float4*>(s_theta)[q];
              const float4 e = reinterpret_cast<const float4*>(s_dth)[q];
              z = fmaf(x.x, t.x, z); dz = fmaf(x.x, e.x, dz);
              z = fmaf(x.y, t.y, z); dz = fmaf(x.y, e.y, dz);
              z = fmaf(x.z, t.z, z); dz = fmaf(x.z, e.z, dz);
              z = fmaf(x.w, t.w, z); dz = fmaf(x.w, e.w, dz);
            }
            if (qfull < cg.f4 && (qfull & (T - 1)) == fw_t) { // last chunk: columns beyond F are the caller's row padding
              const float4 x = xr[qfull];
              const int f = 4 * qfull;
              z = fmaf(x.x, s_theta[f], z); dz = fmaf(x.x, s_dth[f], dz);
              if (f + 1 < F) { z = fmaf(x.y, s_theta[f + 1], z); dz = fmaf(x.y, s_dth[f + 1], dz); }
              if (f + 2 < F) { z = fmaf(x.z, s_theta[f + 2], z); dz = fmaf(x.z, s_dth[f + 2], dz); }
            }
            if (P.has_bias && fw_t == 0) { z += s_theta[F]; dz += s_dth[F]; }
          }
          for (int o = T >> 1; o > 0; o >>= 1) {
            z += __shfl_xor_sync(0xffffffffu, z, o);
            dz += __shfl_xor_sync(0xffffffffu, dz, o);
          }
          if (j < Bm && fw_t == 0) {
            float sig, dsig;
            sigmoid_pair_fast(z, dz, sig, dsig);
            s_res[j] = (sig - 0.5f * (s_y[buf * B + j] + 1.0f)) * invB;
            s_res[B + j] = dsig * invB;
          }
        }
        fc_group_sync(gi);
        // ---- worker: backward, thread = (quad of columns, row group) ---------------------------
        if (bw_active) {
          float ag[4] = {0.f, 0.f, 0.f, 0.f}, ad[4] = {0.f, 0.f, 0.f, 0.f};
          const bool has_x = bw_q < cg.f4;
  #pragma unroll 1
          for (int i = bw_rg; i < Bm; i += cg.nrg) {
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (has_x) x = *reinterpret_cast<const float4*>(xb + (size_t)i * cg.pitch + 4 * bw_q);
            const float xs[4] = {x.x, x.y, x.z, x.w};
            const float r = s_res[i], dr = s_res[B + i];
  #pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float xv = bw_kind[e] == 0 ? xs[e] : bw_kind[e] == 1 ? 1.f : 0.f;
              ag[e] = fmaf(r, xv, ag[e]);
              ad[e] = fmaf(dr, xv, ad[e]);
            }
          }
          *reinterpret_cast<float4*>(s_part + (bw_rg * 2 + 0) * cg.pp + 4 * bw_q) = make_float4(ag[0], ag[1], ag[2], ag[3]);
          *reinterpret_cast<float4*>(s_part + (bw_rg * 2 + 1) * cg.pp + 4 * bw_q) = make_float4(ad[0], ad[1], ad[2], ad[3]);
        }
      } else {
        // ---- worker, register-tiled: a thread holds 4 rows x NCH quads of the minibatch for both passes -------------
        // Columns beyond F are set to 1 (the constant feature) or 0 (padding) as they are loaded, so that both passes
        // are plain products.  Rows beyond the worker's batch count as zero rows.
        float4 x[4][NCH];
        float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};    // (z, dz) of the thread's 4 rows, this thread's quads
        const int j_first = tl_rg * 4;
#pragma unroll
        for (int i = 0; i < NCH; ++i) {
          const int c = tl_t + i * TL;
          const bool own = c < cg.nqb && tl_rg < cg.nrg;
          float4 t4 = make_float4(0.f, 0.f, 0.f, 0.f), e4 = t4;
          if (own) { t4 = reinterpret_cast<const float4*>(s_theta)[c]; e4 = reinterpret_cast<const float4*>(s_dth)[c]; }
          const unsigned fix = (tl_fix >> (8 * i)) & 0xffu;
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            float4 xv = make_float4(0.f, 0.f, 0.f, 0.f);
            if (own && j_first + r < Bm) {
              if (c < cg.f4) xv = *reinterpret_cast<const float4*>(xb + (size_t)(j_first + r) * cg.pitch + 4 * c);
              if (fix) {
                xv.x = (fix & 3u) == 0 ? xv.x : (fix & 3u) == 1 ? 1.f : 0.f;
                xv.y = ((fix >> 2) & 3u) == 0 ? xv.y : ((fix >> 2) & 3u) == 1 ? 1.f : 0.f;
                xv.z = ((fix >> 4) & 3u) == 0 ? xv.z : ((fix >> 4) & 3u) == 1 ? 1.f : 0.f;
                xv.w = ((fix >> 6) & 3u) == 0 ? xv.w : ((fix >> 6) & 3u) == 1 ? 1.f : 0.f;
              }
            }
            x[r][i] = xv;
            v[2 * r] = fmaf(xv.x, t4.x, v[2 * r]); v[2 * r + 1] = fmaf(xv.x, e4.x, v[2 * r + 1]);
            v[2 * r] = fmaf(xv.y, t4.y, v[2 * r]); v[2 * r + 1] = fmaf(xv.y, e4.y, v[2 * r + 1]);
            v[2 * r] = fmaf(xv.z, t4.z, v[2 * r]); v[2 * r + 1] = fmaf(xv.z, e4.z, v[2 * r + 1]);
            v[2 * r] = fmaf(xv.w, t4.w, v[2 * r]); v[2 * r + 1] = fmaf(xv.w, e4.w, v[2 * r + 1]);
          }
        }
        // the 8 sums over the TL lanes of the row group, transposed: each stage halves what a lane keeps, so that
        // 4 + 2 + 1 shuffles (plus one per remaining lane bit) do the work of 8 per stage
        const bool up1 = tl_t & (TL >> 1), up2 = tl_t & (TL >> 2), up3 = tl_t & (TL >> 3);
        float w4[4], w2[2], w1;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float send = up1 ? v[q] : v[4 + q], keep = up1 ? v[4 + q] : v[q];
          w4[q] = keep + __shfl_xor_sync(0xffffffffu, send, TL >> 1);
        }
#pragma unroll
        for (int q = 0; q < 2; ++q) {
          const float send = up2 ? w4[q] : w4[2 + q], keep = up2 ? w4[2 + q] : w4[q];
          w2[q] = keep + __shfl_xor_sync(0xffffffffu, send, TL >> 2);
        }
        {
          const float send = up3 ? w2[0] : w2[1], keep = up3 ? w2[1] : w2[0];
          w1 = keep + __shfl_xor_sync(0xffffffffu, send, TL >> 3);
        }
        for (int o = TL >> 4; o > 0; o >>= 1) w1 += __shfl_xor_sync(0xffffffffu, w1, o);
        // the lane now holds z (up3 clear) or dz (up3 set) of row 2 * up1 + up2 of its group; its partner holds the other
        const float other = __shfl_xor_sync(0xffffffffu, w1, TL >> 3);
        const int my_row = j_first + (up1 ? 2 : 0) + (up2 ? 1 : 0);
        float rv = 0.f, drv = 0.f;
        if (tl_rg < cg.nrg && my_row < Bm) {
          float sig, dsig;
          sigmoid_pair_fast(up3 ? other : w1, up3 ? w1 : other, sig, dsig);
          rv = (sig - 0.5f * (s_y[buf * B + my_row] + 1.0f)) * invB;
          drv = dsig * invB;
        }
        // backward: rank-4 update of both accumulators from the rows held in registers
        float4 ag[NCH], ad[NCH];
#pragma unroll
        for (int i = 0; i < NCH; ++i) { ag[i] = make_float4(0.f, 0.f, 0.f, 0.f); ad[i] = ag[i]; }
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const int src = ((r >> 1) ? (TL >> 1) : 0) + ((r & 1) ? (TL >> 2) : 0);   // a lane of the group that holds row r
          const float res = __shfl_sync(0xffffffffu, rv, src, TL), dres = __shfl_sync(0xffffffffu, drv, src, TL);
#pragma unroll
          for (int i = 0; i < NCH; ++i) {
            ag[i].x = fmaf(res, x[r][i].x, ag[i].x); ag[i].y = fmaf(res, x[r][i].y, ag[i].y);
            ag[i].z = fmaf(res, x[r][i].z, ag[i].z); ag[i].w = fmaf(res, x[r][i].w, ag[i].w);
            ad[i].x = fmaf(dres, x[r][i].x, ad[i].x); ad[i].y = fmaf(dres, x[r][i].y, ad[i].y);
            ad[i].z = fmaf(dres, x[r][i].z, ad[i].z); ad[i].w = fmaf(dres, x[r][i].w, ad[i].w);
          }
        }
        if (tl_rg < cg.nrg) {
#pragma unroll
          for (int i = 0; i < NCH; ++i) {
            const int c = tl_t + i * TL;
            if (c < cg.nqb) {
              *reinterpret_cast<float4*>(s_part + (tl_rg * 2 + 0) * cg.pp + 4 * c) = ag[i];
              *reinterpret_cast<float4*>(s_part + (tl_rg * 2 + 1) * cg.pp + 4 * c) = ad[i];
            }
          }
        }
      }
      fc_group_sync(gi);
      if (tg == 0) ptx::mbar_arrive(bar_cons + 8u * buf);  // the minibatch buffer has been read: the producer may refill it
      // four lanes per coordinate: lane s adds the row groups s, s + 4, ... and a butterfly joins the four sums
      double acc = 0.0;
      for (int j0 = 0; j0 < p; j0 += FC_GROUP / 4) {      // uniform trip count (shuffles)
        const int j = j0 + (tg >> 2);
        float g = 0.f, d = 0.f;
        if (j < p) {
#pragma unroll 4
          for (int r = tg & 3; r < cg.nrg; r += 4) { g += s_part[(r * 2 + 0) * cg.pp + j]; d += s_part[(r * 2 + 1) * cg.pp + j]; }
        }
        g += __shfl_xor_sync(0xffffffffu, g, 1); d += __shfl_xor_sync(0xffffffffu, d, 1);
        g += __shfl_xor_sync(0xffffffffu, g, 2); d += __shfl_xor_sync(0xffffffffu, d, 2);
        if (j < p && (tg & 3) == 0) {
          g = fmaf(P.lambda, s_theta[j], g);
          d = fmaf(P.lambda, s_dth[j], d);
          s_g[j] = g; s_d[j] = d;
          const float e = cada1 ? d - s_dst[j] : d;
          acc = fma((double)e, (double)e, acc);
        }
      }
      acc += __shfl_xor_sync(0xffffffffu, acc, 4);         // the parts sit in every fourth lane
      acc += __shfl_xor_sync(0xffffffffu, acc, 8);
      acc += __shfl_xor_sync(0xffffffffu, acc, 16);
      if ((tg & 31) == 0) s_red[tg >> 5] = acc;
      fc_group_sync(gi);
      // every thread of the group takes the decision itself (same inputs, same arithmetic, own copies of the
      // staleness and of the selector): no second barrier to hand it round
      double lhs = 0.0;                                 // left-hand side of Eq. 6 / Eq. 8, fixed order
#pragma unroll
      for (int w = 0; w < FC_GWARPS; ++w) lhs += s_red[w];
      const double rhs = s_rhs[0];
      const bool forced = tau >= P.D, violated = !(lhs <= rhs), up = violated || forced;
      last_bits = (unsigned char)((up ? 1 : 0) | (forced ? 2 : 0));
      last_lhs = lhs; last_rhs = rhs;
      tau = up ? 1 : tau + 1;
      if (up) { ++n_up; if (forced) ++n_forced; sel ^= 1u; }
      const unsigned word = (unsigned)last_bits | (sel << 2);
      {
        // The fresh gradient goes to every CTA's copy of slot m, into the buffer that is NOT the current one before this
        // decision -- an upload makes it the current one, a skip leaves it unread -- together with the decision word.
        // Every worker sends every iteration, so that each CTA knows how many bytes an iteration brings: the stores are
        // asynchronous and credit the receiver's mbarrier, nobody waits for an acknowledgement
        const unsigned dst_buf = (word & 1u) ? ((word >> 2) & 1u) : (((word >> 2) & 1u) ^ 1u);
        float* slot = s_G + dst_buf * slot_buf + (size_t)m * cg.pp;
        const uint32_t rx = bar_rx + 8u * (it & 1);
        int dest = bw_rg, q = bw_q;                       // tg = dest * nqb + q
        for (int c = tg; c < cg.ncta * cg.nqb; c += FC_GROUP) {
          fc_st_async_f4(fc_map_u32(ptx::smem_u32(slot + 4 * q), (unsigned)dest), reinterpret_cast<const float4*>(s_g)[q],
                         fc_map_u32(rx, (unsigned)dest));
          q += FC_GROUP % cg.nqb; dest += FC_GROUP / cg.nqb;
          if (q >= cg.nqb) { q -= cg.nqb; ++dest; }
        }
        if (tg >= 32 && tg < 32 + cg.ncta)
          fc_st_async_u32(fc_map_u32(ptx::smem_u32(s_flags + (it & 1) * cg.Mp + m), (unsigned)(tg - 32)), word,
                          fc_map_u32(rx, (unsigned)(tg - 32)));
      }
      if (word & 1u) {                                  // upload: the worker's own records
        for (int j = tg; j < cg.pp; j += FC_GROUP) {
          if (cada1) s_dst[j] = s_d[j]; else s_old[j] = s_theta[j];
        }
      }
    }
    if (active && tg == 0) {                            // bookkeeping that nobody waits for
      if (!isfinite(last_lhs) || isnan(last_rhs)) atomicOr(&P.st->status_flags, 1);
      if (!isinf(last_rhs)) {
        const double big = fmax(last_lhs, last_rhs);
        if (fabs(last_lhs - last_rhs) <= 1e-4 * big && big > 0.0) ++n_ties;
      }
      if (P.hist_cap > 0) {
        P.hist_lhs[(long long)hist_pos * M + m] = last_lhs; P.hist_mask[(long long)hist_pos * M + m] = last_bits;
        if (m == 0) P.hist_rhs[hist_pos] = last_rhs;
      }
    }
    fc_wait(bar_rx + 8u * (it & 1), (uint32_t)(it >> 1) & 1u, dead, &P.st->status_flags);

    // ---- server: aggregate the current slots, Eqs. 2a-2c ------------------------------------------
    // FC_SRV lanes per coordinate: lane w sums workers w, w + FC_SRV, ... in that order, then a butterfly adds the
    // FC_SRV partial sums (a fixed order, the same in every CTA)
    const unsigned* fl = s_flags + (it & 1) * cg.Mp;
    const float invM = 1.0f / (float)M, alpha_k = step_size(P, k);
    const bool snap_now = cada1 && snap_ctr == 0, next_snap = cada1 && (snap_ctr + 1 == P.D ? 0 : snap_ctr + 1) == 0;
    double dsq = 0.0;
    for (int j0 = 0; j0 < p; j0 += NTHR / FC_SRV) {       // uniform trip count (shuffles)
      const int j = j0 + sv_j0;
      float sum = 0.f;
      if (j < p)
#pragma unroll 4
        for (int w = sv_w; w < M; w += FC_SRV) sum += s_G[((fl[w] >> 2) & 1u) * slot_buf + (size_t)w * cg.pp + j];
#pragma unroll
      for (int o = FC_SRV >> 1; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (j < p && sv_w == 0) {
        const float nab = sum * invM;
        const float hn = P.beta1 * s_h[j] + (1.0f - P.beta1) * nab;
        const float v = P.beta2 * s_vhat[j] + (1.0f - P.beta2) * nab * nab;
        const float vn = fmaxf(v, s_vhat[j]);
        const float t = s_theta[j];
        const float tn = t - alpha_k * hn / sqrtf(P.eps + vn);
        const double dl = (double)tn - (double)t;
        dsq = fma(dl, dl, dsq);
        s_h[j] = hn; s_vhat[j] = vn; s_theta[j] = tn;
        // theta - theta' of the next iteration for this CTA's workers.  Algorithm 1's snapshot step (CADA1): an
        // iteration with k mod D == 0 uses theta~ = theta^k, i.e. a zero difference (written by the iteration before,
        // or by the prologue); the snapshot record itself is refreshed here, from theta^k, so that it never runs ahead
#pragma unroll
        for (int g = 0; g < W; ++g) {
          if ((int)rank * W + g < M) {
            unsigned char* gg = sm + cg.off_grp + (size_t)g * cg.grp_bytes;
            float* optr = reinterpret_cast<float*>(gg + cg.g_old) + j;
            float o = *optr;
            if (snap_now) { o = t; *optr = t; }
            reinterpret_cast<float*>(gg + cg.g_dth)[j] = next_snap ? 0.f : tn - o;
          }
        }
      }
    }
    // only the first lane of each group of FC_SRV holds a part: the butterfly starts at that distance
#pragma unroll
    for (int o = FC_SRV; o < 32; o <<= 1) dsq += __shfl_xor_sync(0xffffffffu, dsq, o);
    if ((tid & 31) == 0) s_stepred[tid >> 5] = dsq;
    if (++ring_pos == P.d_max) ring_pos = 0;
    if (++snap_ctr == P.D) snap_ctr = 0;
    if (P.hist_cap > 0 && ++hist_pos == P.hist_cap) hist_pos = 0;
    if constexpr (STREAM) {                             // the step's upload mask: every CTA has all decision words
      if (rank == 0 && hs.out_mask && tid < M) s_maskout[(it & (FC_MASK_STEPS - 1)) * M + tid] = (unsigned char)(fl[tid] & 3u);
    }
    fc_compute_sync<W>();
    if constexpr (STREAM) {
      // the step's iterate, by one warp in consecutive 4-byte pieces (few, full writes on the bus); theta is not touched
      // again before the next server phase, which this warp takes part in.  The masks of FC_MASK_STEPS steps leave
      // together, as 4-byte pieces where the caller's buffer allows it: single bytes written over the bus one step at a
      // time cost several microseconds each
      if (rank == 0 && tid < 32) {
        if (hs.out_theta)
          for (int j = tid; j < p; j += 32) hs.out_theta[(long long)it * p + j] = s_theta[j];
        if (hs.out_mask && (((it + 1) & (FC_MASK_STEPS - 1)) == 0 || it + 1 == n_iters)) {
          const int it0 = it & ~(FC_MASK_STEPS - 1), nbytes = (it + 1 - it0) * M;
          unsigned char* dst = hs.out_mask + (long long)it0 * M;
          const int nw = (reinterpret_cast<uintptr_t>(dst) & 3) == 0 ? nbytes >> 2 : 0;
          for (int j = tid; j < nw; j += 32) reinterpret_cast<unsigned*>(dst)[j] = reinterpret_cast<const unsigned*>(s_maskout)[j];
          for (int j = 4 * nw + tid; j < nbytes; j += 32) dst[j] = s_maskout[j];
        }
      }
    }
  }

  // ---- write the state back ----------------------------------------------------------------
  fc_cluster_arrive();                                // (waited for at the very end) no CTA leaves while messages may be in flight
  const long long k_end = k0 + n_iters;
  if (tid == NTHR - 1 && n_iters > 0) {
    double s = 0.0;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) s += s_stepred[w];
    s_ring[ring_pos == 0 ? P.d_max - 1 : ring_pos - 1] = s;
    s_ring[P.d_max + 1] = s;
  }
  fc_compute_sync<W>();
  if (rank == 0) {
    for (int j = tid; j < p; j += NTHR) { P.theta[j] = s_theta[j]; P.h[j] = s_h[j]; P.vhat[j] = s_vhat[j]; }
    for (int j = tid; j < P.d_max; j += NTHR) P.ring[j] = s_ring[j];
  }
  if (active) {
    const unsigned cur = sel;                         // every thread of the group kept the selector
    for (int j = tg; j < p; j += FC_GROUP) {
      if (cada1) { P.delta_stored[(long long)m * P.ldp + j] = s_dst[j]; if (m == 0) P.theta_tilde[j] = s_old[j]; }
      else P.theta_hat[(long long)m * P.ldp + j] = s_old[j];
      if (n_iters > 0) {
        P.g_fresh[(long long)m * P.ldp + j] = s_g[j];
        P.d_fresh[(long long)m * P.ldp + j] = s_d[j];
        P.G[(long long)m * P.ldp + j] = s_G[cur * slot_buf + (size_t)m * cg.pp + j];
      }
    }
    if (tg == 0 && n_iters > 0) {
      P.tau[m] = tau; P.mask[m] = last_bits; P.lhs[m] = last_lhs; P.up_per_worker[m] += n_up;
      atomicAdd((unsigned long long*)&P.st->uploads_total, (unsigned long long)n_up);
      atomicAdd((unsigned long long*)&P.st->uploads_forced, (unsigned long long)n_forced);
      atomicAdd((unsigned long long*)&P.st->uploads_rule, (unsigned long long)(n_up - n_forced));
      atomicAdd((unsigned long long*)&P.st->near_ties, (unsigned long long)n_ties);
      if (m == 0) { P.st->last_rhs = last_rhs; P.st->last_step_sqnorm = s_ring[P.d_max + 1]; P.st->k = k_end; }
    }
  }
  fc_cluster_wait();
}

}  // namespace cada
