// Second half of a worker's step, shared by every distance path: local gradient (Eq. 9), receive
// buffers with lambda (Eq. 3) and the Parzen test (Eq. 4), merged update (Eq. 6 / Eq. 7 and the
// update line of Algorithm 5), and the send line of Algorithm 5.
#pragma once

#include "asgd_common.cuh"

namespace asgd {

constexpr int MAX_FANOUT = 16;
constexpr int MAX_SLOTS = 16;

// Scratch every path reserves in shared memory for this tail.
struct TailScratch {
  double red[96];
  int accept[MAX_SLOTS];
  int fresh[MAX_SLOTS];
  int peers[MAX_FANOUT];
  int pslots[MAX_FANOUT];
  int flag;
  int m;
};

// w     [k rows of d, row stride wstride]  this worker's state (shared or global memory), updated in place
// SD    [kd]  in: per-centre sums S_k of the mini-batch; out: the local gradient D
// cnt   [k]   per-centre counts n_k
// wglob       the worker's row of Params::state when w lives in shared memory, else nullptr
// sd_l2   the sums in SD were produced by reductions in L2: read them past L1
template <bool kDet>
__device__ inline void step_tail(const Params& p, int i, unsigned long long t, float* w, int wstride, float* SD,
                                 const int* cnt, float* wglob, TailScratch* ts, bool sd_l2 = false) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int kd = p.kd, d = p.d;
  const bool dense_rows = (wstride == d);
  auto widx = [&](int e) { return dense_rows ? e : (e / d) * wstride + (e % d); };
  const float inv_b = 1.0f / (float)p.b;
  const float eps = p.eps;

  // Eq. 9 (true-gradient sign, mean over the mini-batch size): D_k = (n_k w_k - S_k) / b
  for (int e = tid; e < kd; e += nt) {
    const int a = e / d;
    const float sums = sd_l2 ? __ldcg(SD + e) : SD[e];
    SD[e] = ((float)cnt[a] * w[widx(e)] - sums) * inv_b;
  }
  __syncthreads();

  // receive buffers: thread s looks at buffer s (all buffers at once, one L2 round trip)
  int m = 0;
  if (tid < p.S) {
    const size_t si = (size_t)i * p.S + tid;
    const unsigned sq = ld_acquire_gpu(p.seq + si);
    const unsigned sn = p.seen[si];
    ts->fresh[tid] = (sq != sn);
    if (sq != sn) {
      p.seen[si] = sq;
      unsigned long long* st = p.stats + (size_t)i * ST_STRIDE;
      atomicAdd(st + ST_RECV, 1ull);
      if (sq - sn > 1u) atomicAdd(st + ST_OVERWRITTEN, (unsigned long long)(sq - sn - 1u));
    }
  }
  __syncthreads();
  for (int s = 0; s < p.S; ++s) {
    const size_t si = (size_t)i * p.S + s;
    const bool fresh = ts->fresh[s] != 0;
    int acc = -1;
    if (fresh) {
      const float* v = p.mail + si * (size_t)p.kd_pad;
      double dot = 0.0, dd = 0.0, nv = 0.0;
      for (int e = tid; e < kd; e += nt) {
        const float vv = __ldcg(v + e);
        const float D = SD[e];
        const float df = w[widx(e)] - vv;
        dot += (double)D * (double)df;
        dd += (double)D * (double)D;
        nv += (double)vv * (double)vv;
      }
      block_sum3(dot, dd, nv, ts->red);
      // Eq. 4 expanded: ||(w - eps D) - v||^2 < ||w - v||^2  <=>  2 <D, w - v> > eps ||D||^2
      const bool delta = p.parzen ? (2.0 * dot > (double)eps * dd) : true;
      acc = (nv > 0.0 && delta) ? 1 : 0;   // lambda * delta
      m += acc;
    }
    if (tid == 0) { ts->accept[s] = acc; p.accept_rec[si] = acc; }
    __syncthreads();
  }

  // Eq. 6: Dbar = w - (w + sum_s a_s v_s) / (1 + sum_s a_s) + D ;  w <- w - eps * Dbar
  const float inv_m1 = 1.0f / (float)(1 + m);
  for (int e = tid; e < kd; e += nt) {
    float sumv = 0.f;
    for (int s = 0; s < p.S; ++s)
      if (ts->accept[s] == 1) sumv += __ldcg(p.mail + ((size_t)i * p.S + s) * (size_t)p.kd_pad + e);
    const int we = widx(e);
    const float ww = w[we];
    const float Dbar = (ww - (ww + sumv) * inv_m1) + SD[e];
    const float nw = ww - eps * Dbar;
    w[we] = nw;
    if (wglob) wglob[e] = nw;
  }
  __syncthreads();

  // send w_{t+1} to f random workers != i
  unsigned long long n_sent = 0;
  if (p.c > 0 && p.f > 0 && p.W > 1 && (t + 1) % (unsigned long long)p.c == 0) {
    if (tid == 0) {
      for (int j = 0; j < p.f; ++j) {
        ts->peers[j] = sched_peer(p, i, t, j, ts->peers);
        ts->pslots[j] = sched_slot(p, i, t, j);
      }
    }
    __syncthreads();
    if (kDet) {
      // synchronous rounds: only announce the put; the delivery kernel copies the payload of the
      // highest announcing (sender, j) once every worker has finished the round
      if (tid < p.f) {
        const size_t ri = (size_t)ts->peers[tid] * p.S + ts->pslots[tid];
        atomicMax(p.arb_win + ri, (unsigned)(i * p.f + tid + 1));
        atomicAdd(p.arb_cnt + ri, 1u);
      }
    } else {
      for (int j = 0; j < p.f; ++j) {
        const size_t ri = (size_t)ts->peers[j] * p.S + ts->pslots[j];
        float* dst = p.mail + ri * (size_t)p.kd_pad;
        for (int e = tid; e < kd; e += nt) dst[e] = w[widx(e)];
        __syncthreads();
        if (tid == 0) red_release_gpu_inc(p.seq + ri);
      }
    }
    n_sent = (unsigned long long)p.f;
  }

  if (tid == 0) {
    unsigned long long* st = p.stats + (size_t)i * ST_STRIDE;
    st[ST_STEPS] = t + 1;
    if (n_sent) atomicAdd(st + ST_SENT, n_sent);
    if (m) atomicAdd(st + ST_ACCEPT, (unsigned long long)m);
  }
}

}  // namespace asgd
