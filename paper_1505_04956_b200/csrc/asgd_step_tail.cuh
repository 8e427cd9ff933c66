// Second half of a worker's step, shared by every distance path: local gradient (Eq. 9), receive
// buffers with lambda (Eq. 3) and the Parzen test (Eq. 4), merged update (Eq. 6 / Eq. 7 and the
// update line of Algorithm 5), and the send line of Algorithm 5.  With per-centre messages
// (Section 4.4, Params::rows_m > 0) lambda, delta and the merge are taken centre row by centre row.
#pragma once

#include "asgd_common.cuh"

namespace asgd {

constexpr int MAX_FANOUT = 16;
constexpr int MAX_SLOTS = 16;

// Scratch every path reserves in shared memory for this tail.
struct alignas(16) TailScratch {
  double red[96];
  int accept[MAX_SLOTS];
  int fresh[MAX_SLOTS];
  int peers[MAX_FANOUT];
  int pslots[MAX_FANOUT];
  int flag;
  int m;
};
static_assert(sizeof(TailScratch) % 16 == 0, "arrays placed behind the scratch keep their 16-byte alignment");

// V floats at a time (V = 4: 128-bit accesses).
template <int V> struct TailVec { float v[V]; };
template <int V> __device__ inline TailVec<V> tail_ld(const float* q) {
  TailVec<V> r;
  if (V == 4) { const float4 t = *reinterpret_cast<const float4*>(q); r.v[0] = t.x; r.v[V > 1 ? 1 : 0] = t.y; r.v[V > 2 ? 2 : 0] = t.z; r.v[V > 3 ? 3 : 0] = t.w; }
  else r.v[0] = *q;
  return r;
}
template <int V> __device__ inline TailVec<V> tail_ldcg(const float* q) {
  TailVec<V> r;
  if (V == 4) { const float4 t = __ldcg(reinterpret_cast<const float4*>(q)); r.v[0] = t.x; r.v[V > 1 ? 1 : 0] = t.y; r.v[V > 2 ? 2 : 0] = t.z; r.v[V > 3 ? 3 : 0] = t.w; }
  else r.v[0] = __ldcg(q);
  return r;
}
template <int V> __device__ inline void tail_st(float* q, const TailVec<V>& r) {
  if (V == 4) *reinterpret_cast<float4*>(q) = make_float4(r.v[0], r.v[V > 1 ? 1 : 0], r.v[V > 2 ? 2 : 0], r.v[V > 3 ? 3 : 0]);
  else *q = r.v[0];
}

// The send line of Algorithm 5: after step t, when (t + 1) is a multiple of the interval, w_{t+1} goes to f random
// workers != i.  Called by all threads of the block with w complete and visible (a barrier before); returns the
// number of messages sent.  Free-running: every thread stores part of the payload, a barrier, then one release
// increment of the buffer's sequence number.  Synchronous rounds: the put is only announced; the delivery kernel
// copies the payload of the highest announcing (sender, j) once every worker has finished the round.
template <bool kDet, int V>
__device__ inline unsigned long long step_send(const Params& p, int i, unsigned long long t, const float* __restrict__ w,
                                               int wstride, TailScratch* ts) {
  if (!(p.c > 0 && p.f > 0 && p.W > 1 && (t + 1) % (unsigned long long)p.c == 0)) return 0;
  const int tid = threadIdx.x, nt = blockDim.x;
  const int d = p.d, nvec = p.kd / V;
  const bool dense_rows = (wstride == d);
  auto widx = [&](int e) { return dense_rows ? e : (e / d) * wstride + (e % d); };
  if (tid == 0) {
    for (int j = 0; j < p.f; ++j) {
      ts->peers[j] = sched_peer(p, i, t, j, ts->peers);
      ts->pslots[j] = sched_slot(p, i, t, j);
    }
  }
  __syncthreads();
  if (kDet) {
    if (tid < p.f) {
      const size_t ri = (size_t)ts->peers[tid] * p.S + ts->pslots[tid];
      atomicMax(p.arb_win + ri, (unsigned)(i * p.f + tid + 1));
      atomicAdd(p.arb_cnt + ri, 1u);
    }
  } else if (p.rows_m > 0) {
    // per-centre message: rows_m consecutive (cyclic) rows, then their description, then the release
    for (int j = 0; j < p.f; ++j) {
      const size_t ri = (size_t)ts->peers[j] * p.S + ts->pslots[j];
      float* dst = p.mail + ri * (size_t)p.kd_pad;
      const int r0 = sched_first_row(p, i, t, j);
      const int per_row = d / V;
      for (int q = tid; q < p.rows_m * per_row; q += nt) {
        int a = r0 + q / per_row;
        if (a >= p.k) a -= p.k;
        const int e = a * d + (q % per_row) * V;
        tail_st<V>(dst + e, tail_ld<V>(w + widx(e)));
      }
      __syncthreads();
      if (tid == 0) {
        p.mail_rows[ri] = make_int2(r0, p.rows_m);
        red_release_gpu_inc(p.seq + ri);
      }
    }
  } else {
    for (int j = 0; j < p.f; ++j) {
      const size_t ri = (size_t)ts->peers[j] * p.S + ts->pslots[j];
      float* dst = p.mail + ri * (size_t)p.kd_pad;
#pragma unroll 8
      for (int q = tid; q < nvec; q += nt) tail_st<V>(dst + q * V, tail_ld<V>(w + widx(q * V)));
      __syncthreads();
      if (tid == 0) red_release_gpu_inc(p.seq + ri);
    }
  }
  return (unsigned long long)p.f;
}

// w     [k rows of d, row stride wstride]  this worker's state (shared or global memory), updated in place
// SD    [kd]  per-centre sums S_k of the mini-batch (read only)
// cnt   [k]   per-centre counts n_k
// wglob       the worker's row of Params::state when w lives in shared memory, else nullptr
// sd_l2       the sums in SD were produced by reductions in L2: read them past L1
// V           elements per access; V = 4 needs d % 4 == 0 and 16-byte aligned w, SD, wglob rows
template <bool kDet, int V>
__device__ inline void step_tail_impl(const Params& p, int i, unsigned long long t, float* __restrict__ w, int wstride,
                                      float* __restrict__ SD, const int* __restrict__ cnt, float* __restrict__ wglob,
                                      TailScratch* ts, bool sd_l2) {
  const int tid = threadIdx.x, nt = blockDim.x;
  const int kd = p.kd, d = p.d;
  const int nvec = kd / V;                                  // V divides d, so an access never straddles two centres
  const bool dense_rows = (wstride == d);
  auto widx = [&](int e) { return dense_rows ? e : (e / d) * wstride + (e % d); };
  const float inv_b = 1.0f / (float)p.b;
  const float eps = p.eps;

  // Eq. 9 (true-gradient sign, mean over the mini-batch size): D_k = (n_k w_k - S_k) / b, formed from the sums where
  // it is needed (in the acceptance test and in the update) instead of in a pass of its own over the state
  auto gradient = [&](int e, const TailVec<V>& ww) {
    const float n = (float)cnt[e / d];
    const TailVec<V> sums = sd_l2 ? tail_ldcg<V>(SD + e) : tail_ld<V>(SD + e);
    TailVec<V> D;
#pragma unroll
    for (int u = 0; u < V; ++u) D.v[u] = (n * ww.v[u] - sums.v[u]) * inv_b;
    return D;
  };

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
  const bool by_rows = p.rows_m > 0;
  unsigned whole_bits = 0;                                   // whole-state messages: buffers accepted in this step
  unsigned* rowacc = by_rows ? p.rowacc + (size_t)i * p.k : nullptr;
  if (!by_rows) {
    for (int s = 0; s < p.S; ++s) {
      const size_t si = (size_t)i * p.S + s;
      const bool fresh = ts->fresh[s] != 0;
      int acc = -1;
      if (fresh) {
        const float* __restrict__ v = p.mail + si * (size_t)p.kd_pad;
        double dot = 0.0, dd = 0.0, nv = 0.0;
#pragma unroll 8
        for (int q = tid; q < nvec; q += nt) {
          const int e = q * V;
          const TailVec<V> vv = tail_ldcg<V>(v + e);
          const TailVec<V> ww = tail_ld<V>(w + widx(e));
          const TailVec<V> D = gradient(e, ww);
#pragma unroll
          for (int u = 0; u < V; ++u) {
            const float df = ww.v[u] - vv.v[u];
            dot += (double)D.v[u] * (double)df;
            dd += (double)D.v[u] * (double)D.v[u];
            nv += (double)vv.v[u] * (double)vv.v[u];
          }
        }
        block_sum3(dot, dd, nv, ts->red);
        // Eq. 4 expanded: ||(w - eps D) - v||^2 < ||w - v||^2  <=>  2 <D, w - v> > eps ||D||^2
        const bool delta = p.parzen ? (2.0 * dot > (double)eps * dd) : true;
        acc = (nv > 0.0 && delta) ? 1 : 0;   // lambda * delta
        m += acc;
        if (acc) whole_bits |= 1u << s;
      }
      if (tid == 0) { ts->accept[s] = acc; p.accept_rec[si] = acc; }
      __syncthreads();
    }
  } else {
    // Section 4.4: a warp per centre row; for every buffer with a new message that carries the row, the
    // row's own lambda and delta (fp64 sums over its d entries, fixed lane order)
    if (tid < p.S) ts->accept[tid] = ts->fresh[tid] ? 0 : -1;          // becomes the number of accepted rows
    __syncthreads();
    unsigned* rowin = p.rowin + (size_t)i * p.k;
    const int lane = tid & 31, wrp = tid >> 5, nw = nt >> 5;
    for (int a = wrp; a < p.k; a += nw) {
      unsigned bits = 0, inbits = 0;
      for (int s = 0; s < p.S; ++s) {
        if (!ts->fresh[s]) continue;
        const size_t si = (size_t)i * p.S + s;
        const int2 run = __ldcg(p.mail_rows + si);
        if (!row_in_run(a, run.x, run.y, p.k)) continue;
        inbits |= 1u << s;
        const float* __restrict__ v = p.mail + si * (size_t)p.kd_pad + (size_t)a * d;
        double dot = 0.0, dd = 0.0, nv = 0.0;
        for (int j = lane; j < d; j += 32) {
          const float vv = __ldcg(v + j), ww = w[widx(a * d + j)];
          const float D = ((float)cnt[a] * ww - (sd_l2 ? __ldcg(SD + a * d + j) : SD[a * d + j])) * inv_b;
          const float df = ww - vv;
          dot += (double)D * (double)df;
          dd += (double)D * (double)D;
          nv += (double)vv * (double)vv;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          dot += __shfl_xor_sync(0xffffffffu, dot, o);
          dd += __shfl_xor_sync(0xffffffffu, dd, o);
          nv += __shfl_xor_sync(0xffffffffu, nv, o);
        }
        const bool delta = p.parzen ? (2.0 * dot > (double)eps * dd) : true;
        if (nv > 0.0 && delta) {
          bits |= 1u << s;
          if (lane == 0) atomicAdd(&ts->accept[s], 1);
        }
      }
      if (lane == 0) { rowacc[a] = bits; rowin[a] = inbits; }
    }
    __syncthreads();
    for (int s = 0; s < p.S; ++s) m += (ts->accept[s] > 0);           // messages with at least one accepted row
    if (tid < p.S) p.accept_rec[(size_t)i * p.S + tid] = ts->accept[tid];
  }

  // Eq. 6: Dbar = w - (w + sum_s a_s v_s) / (1 + sum_s a_s) + D ;  w <- w - eps * Dbar   (a_s per row in per-centre mode)
  const float inv_m1_whole = 1.0f / (float)(1 + m);
#pragma unroll 8
  for (int q = tid; q < nvec; q += nt) {
    const int e = q * V;
    const unsigned bits = by_rows ? rowacc[e / d] : whole_bits;
    const float inv_m1 = by_rows ? 1.0f / (float)(1 + __popc(bits)) : inv_m1_whole;
    TailVec<V> sumv;
#pragma unroll
    for (int u = 0; u < V; ++u) sumv.v[u] = 0.f;
    for (int s = 0; s < p.S; ++s)
      if (bits & (1u << s)) {
        const TailVec<V> vv = tail_ldcg<V>(p.mail + ((size_t)i * p.S + s) * (size_t)p.kd_pad + e);
#pragma unroll
        for (int u = 0; u < V; ++u) sumv.v[u] += vv.v[u];
      }
    const int we = widx(e);
    const TailVec<V> ww = tail_ld<V>(w + we);
    const TailVec<V> D = gradient(e, ww);
    TailVec<V> nw;
#pragma unroll
    for (int u = 0; u < V; ++u) {
      const float Dbar = (ww.v[u] - (ww.v[u] + sumv.v[u]) * inv_m1) + D.v[u];
      nw.v[u] = ww.v[u] - eps * Dbar;
    }
    tail_st<V>(w + we, nw);
    if (wglob) tail_st<V>(wglob + e, nw);
  }
  __syncthreads();

  // send w_{t+1} to f random workers != i
  const unsigned long long n_sent = step_send<kDet, V>(p, i, t, w, wstride, ts);

  if (tid == 0) {
    unsigned long long* st = p.stats + (size_t)i * ST_STRIDE;
    st[ST_STEPS] = t + 1;
    if (n_sent) atomicAdd(st + ST_SENT, n_sent);
    if (m) atomicAdd(st + ST_ACCEPT, (unsigned long long)m);
  }
}

// Picks 128-bit accesses when the layout allows it.
template <bool kDet>
__device__ inline void step_tail(const Params& p, int i, unsigned long long t, float* w, int wstride, float* SD,
                                 const int* cnt, float* wglob, TailScratch* ts, bool sd_l2 = false) {
  const bool vec = (p.d % 4 == 0) && (wstride % 4 == 0) && ((((size_t)w) | ((size_t)SD) | ((size_t)wglob)) & 15) == 0;
  if (vec) step_tail_impl<kDet, 4>(p, i, t, w, wstride, SD, cnt, wglob, ts, sd_l2);
  else step_tail_impl<kDet, 1>(p, i, t, w, wstride, SD, cnt, wglob, ts, sd_l2);
}

// The send alone, for paths that fuse the plain local update into their own passes.
template <bool kDet>
__device__ inline unsigned long long step_send_any(const Params& p, int i, unsigned long long t, const float* w, int wstride,
                                                   TailScratch* ts) {
  const bool vec = (p.d % 4 == 0) && (wstride % 4 == 0) && (((size_t)w) & 15) == 0;
  return vec ? step_send<kDet, 4>(p, i, t, w, wstride, ts) : step_send<kDet, 1>(p, i, t, w, wstride, ts);
}

}  // namespace asgd
