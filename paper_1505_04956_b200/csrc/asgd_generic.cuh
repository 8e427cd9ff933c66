// General fp32 path: any k, d, b.  One thread block per worker.  Distances in the direct
// difference form (Eq. 8), one thread per sample; sums through a stable grouping of the batch by
// centre, so a step's result does not depend on thread timing.  This is the path of last resort
// (and the on-device cross-check for the specialised paths); it is correct everywhere, fast nowhere.
#pragma once

#include "asgd_step_tail.cuh"

namespace asgd {

constexpr int GENERIC_THREADS = 256;

// Shared-memory bytes of the generic kernel.
inline size_t generic_smem_bytes(int k, int b, int kd_pad, bool state_on_chip) {
  size_t bytes = sizeof(TailScratch);
  bytes += (size_t)(k + (k + 1) + 2 * b + 8) * sizeof(int);
  if (state_on_chip) bytes += (size_t)2 * kd_pad * sizeof(float);
  return (bytes + 15) & ~(size_t)15;
}

// Exclusive prefix of cnt[0..k) into start[0..k], by warp 0.
__device__ inline void warp0_exclusive_scan(const int* cnt, int k, int* start) {
  if ((threadIdx.x >> 5) != 0) return;
  const int lane = threadIdx.x & 31;
  int carry = 0;
  for (int a0 = 0; a0 < k; a0 += 32) {
    const int a = a0 + lane;
    const int v = (a < k) ? cnt[a] : 0;
    int x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (a < k) start[a] = carry + x - v;
    carry += __shfl_sync(0xffffffffu, x, 31);
  }
  if (lane == 0) start[k] = carry;
}

template <bool kDet>
__global__ void __launch_bounds__(GENERIC_THREADS)
asgd_generic_kernel(const Params p, const long long steps, const int state_on_chip) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  TailScratch* ts = reinterpret_cast<TailScratch*>(smem_raw);
  unsigned char* cur = smem_raw + sizeof(TailScratch);
  float* w;
  float* SD;
  const int i = blockIdx.x;
  float* wglob = p.state + (size_t)i * p.kd_pad;
  if (state_on_chip) {
    w = reinterpret_cast<float*>(cur); cur += (size_t)p.kd_pad * sizeof(float);
    SD = reinterpret_cast<float*>(cur); cur += (size_t)p.kd_pad * sizeof(float);
  } else {
    w = wglob;
    SD = p.gsum + (size_t)i * p.kd_pad;
  }
  int* cnt = reinterpret_cast<int*>(cur);
  int* start = cnt + p.k;
  int* assign = start + p.k + 1;
  int* order = assign + p.b;

  const int tid = threadIdx.x, nt = blockDim.x;
  const int lane = tid & 31, wid = tid >> 5, nw = nt >> 5;
  const int k = p.k, d = p.d, b = p.b;

  if (state_on_chip) {
    for (int e = tid; e < p.kd; e += nt) w[e] = wglob[e];
  }
  unsigned long long t = p.stats[(size_t)i * ST_STRIDE + ST_STEPS];
  __syncthreads();

  for (long long step = 0; step < steps; ++step, ++t) {
    // draw the mini-batch: b consecutive rows of this worker's shard, in its seeded batch order
    const long long batch = p.perm[(size_t)i * p.B + (size_t)(t % (unsigned long long)p.B)];
    const float* M = p.X + ((size_t)i * p.H + (size_t)batch * b) * d;

    for (int a = tid; a < k; a += nt) cnt[a] = 0;
    __syncthreads();

    // Eq. 8: nearest prototype, ties to the lowest index
    for (int s = tid; s < b; s += nt) {
      const float* x = M + (size_t)s * d;
      int best = 0;
      float bd = __int_as_float(0x7f800000);
      for (int a = 0; a < k; ++a) {
        const float* wa = w + (size_t)a * d;
        float acc = 0.f;
        for (int j = 0; j < d; ++j) {
          const float df = __ldg(x + j) - wa[j];
          acc = fmaf(df, df, acc);
        }
        if (acc < bd) { bd = acc; best = a; }
      }
      assign[s] = best;
      atomicAdd(cnt + best, 1);
      if (p.assign_rec) p.assign_rec[(size_t)i * b + s] = best;
    }
    __syncthreads();
    warp0_exclusive_scan(cnt, k, start);
    __syncthreads();
    block_group_by_centre(assign, b, k, start, order);
    __syncthreads();

    // Eq. 9: per-centre sums, each centre summed by one warp in ascending sample order
    for (int a = wid; a < k; a += nw) {
      const int p0 = start[a], p1 = start[a + 1];
      for (int j0 = 0; j0 < d; j0 += 32) {
        const int j = j0 + lane;
        float acc = 0.f;
        if (j < d)
          for (int q = p0; q < p1; ++q) acc += __ldg(M + (size_t)order[q] * d + j);
        if (j < d) SD[(size_t)a * d + j] = acc;
      }
    }
    __syncthreads();

    step_tail<kDet>(p, i, t, w, d, SD, cnt, state_on_chip ? wglob : nullptr, ts);
    __syncthreads();
  }
}

}  // namespace asgd
