// Issue-rate probes for sm_100a: how many cycles a scheduler (one of the four of an SM) spends per warp
// instruction for the instruction kinds the worker kernels are made of, alone and mixed.  They give the
// denominators that the notes on the kernels quote (what a packed FMA, a min/max, a legacy tensor-core
// product cost in issue slots), measured with clock64 on one block per SM, 16 warps each.
//
// Built into its own small library (libasgd_probe.so); nothing in the worker library depends on it.
#include <cuda_runtime.h>

#include "asgd_tc.cuh"   // descriptors and wrappers of tcgen05.mma, mbarrier helpers

namespace {

enum Mode { M_FFMA = 0, M_FFMA_ACC, M_FFMA2_ACC, M_FADD2, M_LOP3, M_FMNMX, M_FSET, M_IMAD, M_HMMA, M_LOP3_FFMA, M_LOP3_FFMA2,
            M_HMMA_6FFMA, M_HMMA_4LOP3, M_COUNT };

template <int MODE>
__global__ void __launch_bounds__(512) probe_kernel(float* out, int iters) {
  float f[16];
  unsigned u[8];
  unsigned long long d[8];
  float c[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
  for (int q = 0; q < 16; ++q) f[q] = threadIdx.x * 0.001f + q;
  for (int q = 0; q < 8; ++q) {
    u[q] = threadIdx.x * 77u + q;
    d[q] = ((unsigned long long)__float_as_uint(f[q]) << 32) | __float_as_uint(f[q] + 1.f);
  }
  const unsigned a0 = __float_as_uint(f[0]) & 0x3fffe000u, b0 = 0x3f800000u;
  const long long t0 = clock64();
  for (int it = 0; it < iters; ++it) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      if (MODE == M_FFMA) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[q]) : "f"(1.0001f), "f"(0.5f));
      if (MODE == M_FFMA_ACC) asm volatile("fma.rn.f32 %0, %1, %2, %0;" : "+f"(f[q]) : "f"(f[8 + (q & 3)]), "f"(f[12 + (q >> 1)]));
      if (MODE == M_FFMA2_ACC) asm volatile("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d[q & 3]) : "l"(d[4 + (q & 1)]), "l"(d[6 + ((q >> 1) & 1)]));
      if (MODE == M_FADD2) asm volatile("add.rn.f32x2 %0, %0, %1;" : "+l"(d[q & 3]) : "l"(d[7]));
      if (MODE == M_LOP3 || MODE == M_LOP3_FFMA || MODE == M_LOP3_FFMA2)
        asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(u[q]) : "r"(u[(q + 1) & 7]), "r"(0x1234567u));
      if (MODE == M_LOP3_FFMA) asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[q]) : "f"(1.0001f), "f"(0.5f));
      if (MODE == M_LOP3_FFMA2) asm volatile("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(d[q & 3]) : "l"(d[4 + (q & 1)]), "l"(d[6 + ((q >> 1) & 1)]));
      if (MODE == M_FMNMX) asm volatile("min.f32 %0, %0, %1;" : "+f"(f[q]) : "f"(f[(q + 1) & 7]));
      if (MODE == M_FSET) asm volatile("set.eq.f32.f32 %0, %0, %1;" : "+f"(f[q]) : "f"(f[(q + 1) & 7]));
      if (MODE == M_IMAD) asm volatile("mad.lo.s32 %0, %0, %1, %2;" : "+r"(u[q]) : "r"(u[(q + 1) & 7]), "r"(u[(q + 2) & 7]));
      if (MODE == M_HMMA || MODE == M_HMMA_6FFMA || MODE == M_HMMA_4LOP3) {
        if ((q & 3) == 0)
          asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%4,%4,%4}, {%5,%5}, {%0,%1,%2,%3};"
                       : "+f"(c[q >> 2][0]), "+f"(c[q >> 2][1]), "+f"(c[q >> 2][2]), "+f"(c[q >> 2][3]) : "r"(a0), "r"(b0));
      }
      if (MODE == M_HMMA_6FFMA && q != 0 && q != 4) {
        asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[q]) : "f"(1.0001f), "f"(0.5f));
        asm volatile("fma.rn.f32 %0, %0, %1, %2;" : "+f"(f[q + 8]) : "f"(1.0001f), "f"(0.5f));
      }
      if (MODE == M_HMMA_4LOP3) asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(u[q]) : "r"(u[(q + 1) & 7]), "r"(0x1234567u));
    }
  }
  const long long t1 = clock64();
  float s = 0.f;
  for (int q = 0; q < 16; ++q) s += f[q];
  for (int q = 0; q < 8; ++q) s += (float)d[q] + (float)u[q];
  for (int h = 0; h < 2; ++h) for (int q = 0; q < 4; ++q) s += c[h][q];
  out[1 + blockIdx.x * blockDim.x + threadIdx.x] = s;
  if (threadIdx.x == 0 && blockIdx.x == 0) out[0] = (float)(t1 - t0);
}

// warp instructions one pass of the inner loop issues
int instructions_per_pass(int mode) {
  switch (mode) {
    case M_HMMA: return 2;
    case M_LOP3_FFMA: case M_LOP3_FFMA2: return 16;
    case M_HMMA_6FFMA: return 2 + 12;
    case M_HMMA_4LOP3: return 2 + 8;
    default: return 8;
  }
}

template <int MODE>
int run_one(float* buf, int sms, float* cycles_per_instruction) {
  const int warps = 16, iters = 2048;
  probe_kernel<MODE><<<sms, warps * 32>>>(buf, iters);
  probe_kernel<MODE><<<sms, warps * 32>>>(buf, iters);
  if (cudaDeviceSynchronize() != cudaSuccess) return -3;
  float cyc = 0.f;
  if (cudaMemcpy(&cyc, buf, sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess) return -3;
  *cycles_per_instruction = cyc / ((float)iters * instructions_per_pass(MODE) * (warps / 4));
  return 0;
}

}  // namespace

// out_host[13]: cycles per warp instruction and scheduler for, in order: FFMA with two immediates; FFMA acc = x * w + acc
// (three register operands); the packed two-wide FMA in that form; the packed add; LOP3; FMNMX; FSET; IMAD; the legacy
// tensor-core product mma.sync m16n8k8 TF32; LOP3 and FFMA alternating; LOP3 and the packed FMA alternating; one
// tensor-core product with six FFMA; one with four LOP3.  scratch_dev: DEVICE, >= 4 * (1 + SMs * 512) bytes.
// Returns 0, or -1 for a bad argument, -3 when a CUDA call failed.
extern "C" int asgd_probe_issue_rates(float* out_host, int n_out, float* scratch_dev, int sms) {
  if (!out_host || !scratch_dev || n_out < (int)M_COUNT || sms < 1) return -1;
  int rc = 0;
#define RUN(M) if (rc == 0) rc = run_one<M>(scratch_dev, sms, out_host + M);
  RUN(M_FFMA) RUN(M_FFMA_ACC) RUN(M_FFMA2_ACC) RUN(M_FADD2) RUN(M_LOP3) RUN(M_FMNMX) RUN(M_FSET) RUN(M_IMAD) RUN(M_HMMA)
  RUN(M_LOP3_FFMA) RUN(M_LOP3_FFMA2) RUN(M_HMMA_6FFMA) RUN(M_HMMA_4LOP3)
#undef RUN
  return rc;
}

namespace {

// One block: thread 0 issues n_mma tcgen05.mma (kind::f16, FP16 operands of zeros in shared memory, M = 128, the given N,
// K = 16) back to back into two accumulator ranges, a commit after every `commit_every` of them (0: only at the end),
// and waits (bounded) for the last commit.  out[blockIdx.x] = cycles per product, or -1 when the wait ran out.
__global__ void __launch_bounds__(128) mma_probe_kernel(float* out, int n_mma, int n_cols, int commit_every, int spread, int variant) {
  extern __shared__ __align__(1024) unsigned char smem_dyn[];
  unsigned char* smem = smem_dyn + ((1024u - (asgd::smem_u32(smem_dyn) & 1023u)) & 1023u);
  unsigned char* sA = smem;                               // 4 chunks of 128 rows x 64 numbers (16 KB each)
  unsigned char* sB = smem + 4 * 16384;                   // 4 chunks of up to 256 rows x 64 numbers (32 KB each)
  __shared__ unsigned long long bars[2 + 8 + 2];
  __shared__ unsigned tmem_base;
  for (int e = threadIdx.x; e < (4 * 16384 + 4 * 32768) / 16; e += blockDim.x) reinterpret_cast<uint4*>(smem)[e] = make_uint4(0u, 0u, 0u, 0u);
  if (threadIdx.x == 0) {
    asgd::mbar_init(bars + 0, 1);
    asgd::mbar_init(bars + 1, commit_every > 0 ? (unsigned)(n_mma / commit_every) : 1u);
    for (int q = 0; q < 10; ++q) asgd::mbar_init(bars + 2 + q, 1);      // variants 1, 3: commits go round these, one arrival completes a phase; the last two end variant 3
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < 32) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(asgd::smem_u32(&tmem_base)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.proxy.async;" ::: "memory");
  asgd::tc_fence_before();
  __syncthreads();
  asgd::tc_fence_after();
  const unsigned tmem = tmem_base;
  if (variant == 3) {
    // two issuing threads (first lanes of warps 0 and 1), each with its own accumulator range, half of the products
    // and its own commits; thread 0 times both
    __shared__ long long t_start;
    if (threadIdx.x == 0) t_start = clock64();
    __syncthreads();
    if ((threadIdx.x & 31) == 0 && threadIdx.x < 64) {
      const int who = threadIdx.x >> 5;
      const unsigned idesc = (1u << 4) | ((unsigned)(n_cols >> 3) << 17) | ((unsigned)(128 >> 4) << 24);
      const unsigned long long dA0 = asgd::tc_smem_desc(sA, 0), dB0 = asgd::tc_smem_desc(sB, 0);
      for (int it = 0; it < n_mma / 2; ++it) {
        const int chunk = (it >> 2) & 3, k4 = it & 3;
        const unsigned long long da = dA0 + (unsigned long long)(chunk * (16384 >> 4) + 2 * k4);
        const unsigned long long db = dB0 + (unsigned long long)(chunk * (32768 >> 4) + 2 * k4);
        asgd::tc_mma_bf16(tmem + (unsigned)(who * n_cols), da, db, idesc, (it & 15) != 0);
        if (commit_every > 0 && (it + 1) % commit_every == 0) asgd::tc_commit(bars + 2 + who * 4 + ((it / commit_every) & 3));
      }
      asgd::tc_commit(bars + 10 + who);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      bool ok = asgd::mbar_wait_bounded(bars + 10, 0, 1u << 24);
      ok = asgd::mbar_wait_bounded(bars + 11, 0, 1u << 24) && ok;
      const long long t1 = clock64();
      out[blockIdx.x] = ok ? (float)(t1 - t_start) / (float)n_mma : -1.f;
    }
  } else if (threadIdx.x == 0) {
    const unsigned idesc = (1u << 4) | ((unsigned)(n_cols >> 3) << 17) | ((unsigned)(128 >> 4) << 24);
    const unsigned long long dA0 = asgd::tc_smem_desc(sA, 0), dB0 = asgd::tc_smem_desc(sB, 0);
    const long long t0 = clock64();
    for (int it = 0; it < n_mma; ++it) {
      // spread: walk over the four chunks of either operand as the worker kernel does; else the same chunk every time
      const int chunk = spread ? (it >> 2) & 3 : 0, k4 = it & 3;
      const unsigned long long da = dA0 + (unsigned long long)(chunk * (16384 >> 4) + 2 * k4);
      const unsigned long long db = dB0 + (unsigned long long)(chunk * (32768 >> 4) + 2 * k4);
      // variant 2: a fresh accumulator range after every commit (no product adds to columns a commit has just covered)
      const unsigned acc = (variant == 2 && commit_every > 0) ? (unsigned)(((it / commit_every) & 1) * n_cols) : (unsigned)(((it >> 4) & 1) * n_cols);
      const bool first = (variant == 2 && commit_every > 0) ? (it % commit_every) == 0 : (it & 15) == 0;
      asgd::tc_mma_bf16(tmem + acc, da, db, idesc, !first);
      if (commit_every > 0 && (it + 1) % commit_every == 0) asgd::tc_commit(variant == 1 ? bars + 2 + ((it / commit_every) & 7) : bars + 1);
    }
    asgd::tc_commit(bars + 0);
    const bool ok = asgd::mbar_wait_bounded(bars + 0, 0, 1u << 24);
    const long long t1 = clock64();
    out[blockIdx.x] = ok ? (float)(t1 - t0) / (float)n_mma : -1.f;
  }
  asgd::tc_fence_before();
  __syncthreads();
  if (threadIdx.x < 32) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

}  // namespace

// out_host[12] (the first six with 6 <= n_out < 12): cycles per tcgen05.mma (kind::f16, M = 128, K = 16, operands in
// shared memory, one block per SM) for: N = 256 on one pair of chunks; N = 256 walking over four chunks of each operand;
// the same with a commit after every four products; the same three with N = 128; N = 256 with a commit after every
// four, the commits going round eight barriers; with a fresh accumulator range after every commit; with a commit after
// every 16; the same on eight barriers; two issuing threads, four products and a commit in turn each; two issuing
// threads without commits.  scratch_dev: DEVICE, >= 4 * sms bytes.  Returns 0, -1 for a bad argument, -3 when a CUDA
// call failed, -4 when a wait on the products ran out.
extern "C" int asgd_probe_mma_rates(float* out_host, int n_out, float* scratch_dev, int sms) {
  if (!out_host || !scratch_dev || n_out < 6 || sms < 1) return -1;
  const int smem = 4 * 16384 + 4 * 32768 + 1024;
  if (cudaFuncSetAttribute(mma_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return -3;
  const int cfg[12][4] = {{256, 0, 0, 0}, {256, 0, 1, 0}, {256, 4, 1, 0}, {128, 0, 0, 0}, {128, 0, 1, 0}, {128, 4, 1, 0},
                          {256, 4, 1, 1}, {256, 4, 1, 2}, {256, 16, 1, 0}, {256, 16, 1, 1}, {256, 4, 1, 3}, {256, 0, 1, 3}};
  for (int c = 0; c < (n_out >= 12 ? 12 : 6); ++c) {
    const int n_mma = 4096;
    for (int rep = 0; rep < 2; ++rep) mma_probe_kernel<<<sms, 128, smem>>>(scratch_dev, n_mma, cfg[c][0], cfg[c][1], cfg[c][2], cfg[c][3]);
    if (cudaDeviceSynchronize() != cudaSuccess) return -3;
    float v = 0.f;
    if (cudaMemcpy(&v, scratch_dev, sizeof(float), cudaMemcpyDeviceToHost) != cudaSuccess) return -3;
    if (v < 0.f) return -4;
    out_host[c] = v;
  }
  return 0;
}
