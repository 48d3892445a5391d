// cada_server_update_noalloc: the server update of Eqs. 2a-2c on caller-supplied vectors, for
// callers that must not allocate device memory.
//
// Who needs it: code that runs where cudaMalloc is off limits -- a plug-in inside a host
// application whose memory pool owns the whole GPU, a real-time loop that may not take the
// allocator's lock, a sandboxed extension that is handed buffers and nothing else.  Such a
// caller cannot give cada_create a workspace sized by cada_workspace_bytes, yet the update
// kernel needs a little scratch besides its inputs and outputs: one partial sum of the squared
// step norm per thread block and a "last block done" counter.  Here that scratch is a fixed
// array in the library's own device image.  Every GPU that loads the library carries it until
// the process exits; it bounds the vector length to CADA_NOALLOC_MAX_P.
//
// The array's name means something only to device code.  In host code it is a stand-in symbol,
// not a device address, so the host asks the runtime for the address once per device
// (cudaGetSymbolAddress, with that device current) and hands the kernel that pointer.
#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

#include <mutex>

#include "../../include/cada.h"

namespace {

constexpr int NA_THREADS = 256;                                   // 4 coordinates per thread
constexpr int NA_MAX_BLOCKS = (int)(CADA_NOALLOC_MAX_P / (4 * NA_THREADS));
constexpr int NA_MAX_DEVICES = 64;

// [0, 256): the block counter (first 4 bytes).  [256, ...): one double per block.
static __device__ __align__(256) unsigned char g_noalloc_scratch[256 + sizeof(double) * NA_MAX_BLOCKS];

__global__ void __launch_bounds__(NA_THREADS)
server_update_noalloc_kernel(float* __restrict__ theta, float* __restrict__ h, float* __restrict__ vhat,
                             const float* __restrict__ nabla, long long p, float alpha, float beta1, float beta2,
                             float eps, double* __restrict__ step_sqnorm_out, unsigned char* scratch) {
  __shared__ double s_warp[NA_THREADS / 32];
  __shared__ unsigned int s_ticket;
  unsigned int* ticket = reinterpret_cast<unsigned int*>(scratch);
  double* block_sums = reinterpret_cast<double*>(scratch + 256);
  const long long q = ((long long)blockIdx.x * NA_THREADS + threadIdx.x) * 4;
  double dsq = 0.0;
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    const long long i = q + e;
    if (i < p) {
      const float g = nabla[i];
      const float hn = beta1 * h[i] + (1.0f - beta1) * g;                       // Eq. 2a
      const float v = beta2 * vhat[i] + (1.0f - beta2) * g * g;                 // Eq. 2b
      const float vn = fmaxf(v, vhat[i]);
      const float t = theta[i];
      const float tn = t - alpha * hn / sqrtf(eps + vn);                        // Eq. 2c
      const double d = (double)tn - (double)t;
      dsq = fma(d, d, dsq);
      h[i] = hn; vhat[i] = vn; theta[i] = tn;
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) dsq += __shfl_xor_sync(0xffffffffu, dsq, o);
  if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = dsq;
  __syncthreads();
  if (threadIdx.x == 0) {
    double total = 0.0;
    for (int w = 0; w < NA_THREADS / 32; ++w) total += s_warp[w];
    block_sums[blockIdx.x] = total;
    __threadfence();
    s_ticket = atomicAdd(ticket, 1u);
    if (s_ticket == gridDim.x - 1) {          // last block: fixed-order sum of all block partials
      __threadfence();
      double s = 0.0;
      for (unsigned b = 0; b < gridDim.x; ++b) s += __ldcg(&block_sums[b]);
      *step_sqnorm_out = s;
      *ticket = 0;
    }
  }
}

std::mutex g_mu;
unsigned char* g_scratch_ptr[NA_MAX_DEVICES] = {};

}  // namespace

extern "C" __attribute__((visibility("default")))
int cada_server_update_noalloc(float* theta, float* h, float* vhat, const float* nabla, int64_t p, float alpha,
                               float beta1, float beta2, float eps, double* step_sqnorm_out, void* stream) {
  if (!theta || !h || !vhat || !nabla || !step_sqnorm_out) return CADA_ERR_INVALID_ARG;
  if (p < 1) return CADA_ERR_INVALID_ARG;
  if (p > (int64_t)CADA_NOALLOC_MAX_P) return CADA_ERR_UNSUPPORTED;     // beyond the built-in scratch
  if (!(alpha > 0.f) || !isfinite(alpha) || !(beta1 >= 0.f && beta1 < 1.f) || !(beta2 >= 0.f && beta2 < 1.f) ||
      !(eps >= 0.f) || !isfinite(eps))
    return CADA_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= NA_MAX_DEVICES) return CADA_ERR_CUDA;
  unsigned char* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {                // first call on this device: resolve the symbol's device address
      void* ptr = nullptr;
      if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || !ptr) return CADA_ERR_CUDA;
      g_scratch_ptr[dev] = static_cast<unsigned char*>(ptr);
    }
    scratch = g_scratch_ptr[dev];
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // the array keeps whatever the previous call (or an interrupted one) left: the counter must start at zero
  if (cudaMemsetAsync(scratch, 0, 256, s) != cudaSuccess) return CADA_ERR_CUDA;
  const int blocks = (int)((p + 4 * NA_THREADS - 1) / (4 * NA_THREADS));
  server_update_noalloc_kernel<<<blocks, NA_THREADS, 0, s>>>(theta, h, vhat, nabla, (long long)p, alpha, beta1, beta2,
                                                           eps, step_sqnorm_out, scratch);
  return cudaGetLastError() == cudaSuccess ? CADA_OK : CADA_ERR_CUDA;
}
