// asgd_eval_noalloc: the quantisation error E(w) with every byte of device scratch taken from a
// fixed array inside the library, for callers that are not allowed to allocate device memory.
// The contract is in include/asgd.h.

#include "../../include/asgd.h"

#include <cuda_runtime.h>

#include <mutex>

namespace {

constexpr int kRowsPerBlock = ASGD_EVAL_NOALLOC_ROWS_PER_BLOCK;
constexpr int kMaxBlocks = ASGD_EVAL_NOALLOC_MAX_BLOCKS;
constexpr int kThreads = 256;
constexpr int kMaxDevices = 64;

// Per-block partial sums.  One copy per GPU that loads the library, held until the process exits.
// In host code this name is only a handle for cudaGetSymbolAddress; kernels get the device address.
static __device__ __align__(256) double g_eval_partials[kMaxBlocks];

// Block c sums 1/2 min_k ||x_r - w_k||^2 over rows [c * kRowsPerBlock, (c+1) * kRowsPerBlock) and N.
__global__ void __launch_bounds__(kThreads)
eval_rows_kernel(const float* __restrict__ X, long long N, int d, int k, const float* __restrict__ wg,
                 double* partial) {
  extern __shared__ __align__(16) unsigned char noalloc_smem[];
  double* red = reinterpret_cast<double*>(noalloc_smem);
  float* w = reinterpret_cast<float*>(noalloc_smem + 32 * sizeof(double));
  for (int e = threadIdx.x; e < k * d; e += kThreads) w[e] = wg[e];
  __syncthreads();
  const long long lo = (long long)blockIdx.x * kRowsPerBlock;
  const long long hi = (lo + kRowsPerBlock < N) ? lo + kRowsPerBlock : N;
  double acc = 0.0;
  for (long long r = lo + threadIdx.x; r < hi; r += kThreads) {
    const float* x = X + (size_t)r * d;
    float bd = __int_as_float(0x7f800000);
    for (int a = 0; a < k; ++a) {
      const float* wa = w + (size_t)a * d;
      float s = 0.f;
      for (int j = 0; j < d; ++j) {
        const float df = __ldg(x + j) - wa[j];
        s = fmaf(df, df, s);
      }
      bd = fminf(bd, s);
    }
    acc += 0.5 * (double)bd;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int q = 0; q < kThreads / 32; ++q) s += red[q];
    partial[blockIdx.x] = s;            // every entry a call reads is overwritten by that call first
  }
}

// Adds the first `blocks` partials in ascending order (the result does not depend on the GPU's size).
__global__ void eval_total_kernel(const double* partial, int blocks, double* out) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    double s = 0.0;
    for (int q = 0; q < blocks; ++q) s += partial[q];
    *out = s;
  }
}

std::mutex g_mutex;
double* g_partials_dev[kMaxDevices];   // device address of g_eval_partials, per device; nullptr = not set up

// Once per device, with that device current: resolve the scratch array's device address and raise
// the kernel's shared-memory limit.  Neither call allocates.
int setup_device(int dev, double** out) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_partials_dev[dev]) {
    double* ptr = nullptr;
    if (cudaGetSymbolAddress((void**)&ptr, g_eval_partials) != cudaSuccess || !ptr) return ASGD_ECUDA;
    if (cudaFuncSetAttribute(eval_rows_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)(ASGD_EVAL_NOALLOC_MAX_KD * sizeof(float) + 32 * sizeof(double))) != cudaSuccess)
      return ASGD_ECUDA;
    g_partials_dev[dev] = ptr;
  }
  *out = g_partials_dev[dev];
  return ASGD_OK;
}

}  // namespace

extern "C" int asgd_eval_noalloc(const float* X_dev, int64_t N, int32_t d, int32_t k, const float* w_dev,
                                 double* E_dev, void* cuda_stream) {
  if (!X_dev || !w_dev || !E_dev || N <= 0 || d <= 0 || k <= 0) return ASGD_EINVAL;
  if ((long long)k * d > ASGD_EVAL_NOALLOC_MAX_KD) return ASGD_EUNSUPPORTED;       // centres must fit on chip
  const long long blocks = (N + kRowsPerBlock - 1) / kRowsPerBlock;
  if (blocks > kMaxBlocks) return ASGD_EUNSUPPORTED;                               // more rows than the fixed scratch covers
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ASGD_ECUDA;
  if (dev < 0 || dev >= kMaxDevices) return ASGD_EUNSUPPORTED;
  double* partials = nullptr;
  const int rc = setup_device(dev, &partials);
  if (rc != ASGD_OK) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t smem = (size_t)k * d * sizeof(float) + 32 * sizeof(double);
  eval_rows_kernel<<<(unsigned)blocks, kThreads, smem, st>>>(X_dev, N, d, k, w_dev, partials);
  eval_total_kernel<<<1, 32, 0, st>>>(partials, (int)blocks, E_dev);
  return cudaGetLastError() == cudaSuccess ? ASGD_OK : ASGD_ECUDA;
}
