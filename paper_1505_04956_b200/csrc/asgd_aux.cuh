// Small kernels around the worker loop: initial broadcast of w0, delivery of a synchronous round's
// puts, external put, mean of the worker states, and the evaluation of E(w) (Eq. 8).
#pragma once

#include "asgd_common.cuh"

namespace asgd {

// Initialisation step of Section 4: the control thread's w0 goes to every worker.
__global__ void broadcast_state_kernel(float* state, const float* w0, int W, int kd, int kd_pad) {
  const size_t total = (size_t)W * kd_pad;
  for (size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x; g < total; g += (size_t)gridDim.x * blockDim.x) {
    const int e = (int)(g % kd_pad);
    state[g] = (e < kd) ? w0[e] : 0.f;
  }
}

// Delivery of one synchronous round (deterministic mode).  One block per receive buffer; the
// buffer takes the whole state of the last announcing sender (ascending sender, then recipient
// index), and its sequence number advances by the number of messages that were aimed at it.
__global__ void deliver_kernel(const Params p) {
  const size_t ri = blockIdx.x;           // receiver * S + slot
  const unsigned win = p.arb_win[ri];
  if (win == 0) return;
  const int sender = (int)((win - 1u) / (unsigned)p.f);
  if (p.rows_m > 0) {
    // per-centre message: the rows the sender drew for this message of the step it has just finished
    const int j = (int)((win - 1u) % (unsigned)p.f);
    const unsigned long long t = p.stats[(size_t)sender * ST_STRIDE + ST_STEPS] - 1ull;
    const int r0 = sched_first_row(p, sender, t, j);
    const float* src = p.state + (size_t)sender * p.kd_pad;
    float* dst = p.mail + ri * (size_t)p.kd_pad;
    for (int q = threadIdx.x; q < p.rows_m * p.d; q += blockDim.x) {
      int a = r0 + q / p.d;
      if (a >= p.k) a -= p.k;
      const int e = a * p.d + q % p.d;
      dst[e] = src[e];
    }
    if (threadIdx.x == 0) p.mail_rows[ri] = make_int2(r0, p.rows_m);
  } else {
    const float4* src = reinterpret_cast<const float4*>(p.state + (size_t)sender * p.kd_pad);
    float4* dst = reinterpret_cast<float4*>(p.mail + ri * (size_t)p.kd_pad);
    for (int e = threadIdx.x; e < p.kd_pad / 4; e += blockDim.x) dst[e] = src[e];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    p.seq[ri] += p.arb_cnt[ri];
    p.arb_win[ri] = 0;
    p.arb_cnt[ri] = 0;
  }
}

// A put from the host side of the library: whole message, then the sequence number.
__global__ void external_put_kernel(float* dst, const float* src, unsigned* seq, int kd) {
  for (int e = threadIdx.x; e < kd; e += blockDim.x) dst[e] = src[e];
  __syncthreads();
  if (threadIdx.x == 0) red_release_gpu_inc(seq);
}
// The same for a per-centre message: rows [r0, r0 + m) cyclically, their description, then the sequence number.
__global__ void external_put_rows_kernel(float* dst, const float* src, unsigned* seq, int2* rows, int k, int d, int r0, int m) {
  for (int q = threadIdx.x; q < m * d; q += blockDim.x) {
    int a = r0 + q / d;
    if (a >= k) a -= k;
    dst[a * d + q % d] = src[a * d + q % d];
  }
  __syncthreads();
  if (threadIdx.x == 0) { *rows = make_int2(r0, m); red_release_gpu_inc(seq); }
}

// Aggregation variant of Section 4.3: out = (1/W) sum_i w^i, summed in ascending worker order.
__global__ void mean_state_kernel(const float* state, int W, int kd, int kd_pad, float* out) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= kd) return;
  double acc = 0.0;
  for (int i = 0; i < W; ++i) acc += (double)state[(size_t)i * kd_pad + e];
  out[e] = (float)(acc / (double)W);
}

// Eq. 8: E(w) = sum_i 1/2 min_k ||x_i - w_k||^2.  Direct difference form in fp32 per sample,
// fp64 from the per-thread sum on.  One partial per block; the host adds them in block order.
constexpr int EVAL_THREADS = 256;
__global__ void __launch_bounds__(EVAL_THREADS)
eval_kernel(const float* __restrict__ X, long long N, int d, int k, const float* __restrict__ wg,
            int w_on_chip, double* partial) {
  extern __shared__ __align__(128) unsigned char smem_raw[];
  double* red = reinterpret_cast<double*>(smem_raw);
  float* ws = reinterpret_cast<float*>(smem_raw + 32 * sizeof(double));
  const float* w = wg;
  if (w_on_chip) {
    for (int e = threadIdx.x; e < k * d; e += blockDim.x) ws[e] = wg[e];
    w = ws;
  }
  __syncthreads();
  double acc = 0.0;
  for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < N; r += (long long)gridDim.x * blockDim.x) {
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
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w_ = 0; w_ < (int)(blockDim.x >> 5); ++w_) s += red[w_];
    partial[blockIdx.x] = s;
  }
}

// Eq. 8 for small states (even d <= 16, k <= 16): a thread keeps its row in registers (64-bit loads) and takes
// the k direct-difference distances with packed two-wide adds and FMAs (even and odd dimensions in the two halves);
// -w lies in shared memory as dimension pairs.  Same partials as eval_kernel: one fp64 sum per block.
template <int D, int K>
__global__ void __launch_bounds__(EVAL_THREADS)
eval_small_kernel(const float* __restrict__ X, long long N, const float* __restrict__ wg, double* partial) {
  static_assert(D % 2 == 0 && D <= 16 && K <= 16, "small states only");
  constexpr int D2 = D / 2;
  __shared__ float2 wneg[K * D2];
  __shared__ double red[EVAL_THREADS / 32];
  for (int e = threadIdx.x; e < K * D2; e += blockDim.x) wneg[e] = make_float2(-wg[2 * e], -wg[2 * e + 1]);
  __syncthreads();
  double acc = 0.0;
  for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < N; r += (long long)gridDim.x * blockDim.x) {
    const float2* x = reinterpret_cast<const float2*>(X + (size_t)r * D);     // rows are 8-byte aligned: D is even
    float2 xv[D2];
#pragma unroll
    for (int jp = 0; jp < D2; ++jp) xv[jp] = __ldg(x + jp);
    float bd = __int_as_float(0x7f800000);
#pragma unroll
    for (int a = 0; a < K; ++a) {
      float2 s = make_float2(0.f, 0.f);
#pragma unroll
      for (int jp = 0; jp < D2; ++jp) {
        const float2 df = __fadd2_rn(xv[jp], wneg[a * D2 + jp]);
        s = __ffma2_rn(df, df, s);
      }
      bd = fminf(bd, s.x + s.y);
    }
    acc += 0.5 * (double)bd;
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int w_ = 0; w_ < (int)(blockDim.x >> 5); ++w_) s += red[w_];
    partial[blockIdx.x] = s;
  }
}

// max_i ||x_i||^2 over the rows the workers can touch (one pass at initialisation).
__global__ void xmax2_kernel(const float* __restrict__ X, long long N, int d, unsigned* out_bits) {
  float m = 0.f;
  for (long long r = (long long)blockIdx.x * blockDim.x + threadIdx.x; r < N; r += (long long)gridDim.x * blockDim.x) {
    const float* x = X + (size_t)r * d;
    float s = 0.f;
    for (int j = 0; j < d; ++j) { const float v = __ldg(x + j); s = fmaf(v, v, s); }
    m = fmaxf(m, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if ((threadIdx.x & 31) == 0) atomicMax(out_bits, __float_as_uint(m));   // non-negative floats order as uints
}

}  // namespace asgd
