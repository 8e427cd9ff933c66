// Issue-rate probes for sm_100a: how many cycles a scheduler (one of the four of an SM) spends per warp
// instruction for the instruction kinds the worker kernels are made of, alone and mixed.  They give the
// denominators that the notes on the kernels quote (what a packed FMA, a min/max, a legacy tensor-core
// product cost in issue slots), measured with clock64 on one block per SM, 16 warps each.
//
// Built into its own small library (libasgd_probe.so); nothing in the worker library depends on it.
#include <cuda_runtime.h>

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
