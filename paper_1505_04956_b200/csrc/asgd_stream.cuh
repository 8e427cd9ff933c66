// Streaming fp32 path for small states (k <= 16, even d <= 16, b <= 512): the HBM-bound shape.
//
// One worker = one 128-thread block, 4 blocks per SM.  The worker's mini-batches are pulled into a
// two-slot shared-memory ring with bulk asynchronous copies (one elected thread issues them, an
// mbarrier per slot counts the bytes), so the next batch streams in while the current one is used.
//
// Assignment (Eq. 8): a warp owns 128 consecutive rows of the batch, a thread 4 of them (row =
// 32*q + lane of the warp's block).  Scores use the expanded form  ||w_a||^2 - 2 x.w_a  with packed
// two-wide FMAs (even and odd dimensions accumulate in the two halves).  The centre index rides in
// the low mantissa bits so that min/max instructions carry the argmin and the runner-up; a sample
// whose two best scores are closer than the rounding bound of this form is decided again in the
// direct difference form.
//
// Per-centre sums (Eq. 9): each warp orders its 128 rows by the centre they chose (rank inside a
// 32-row block from a match, so a centre's rows stay in row order; entries are byte offsets into the
// tile).  A centre's run starts at a multiple of eight entries and its unused tail points at a row of
// zeros kept behind the tile, so the order falls into groups of eight rows of one centre.  Lane g of
// the same warp adds the eight rows of group g over all dimensions; the update adds a centre's group
// sums in order.  The work per lane does not depend on how unevenly the centres are chosen, every sum
// has a fixed order (a step is reproducible), and the plain local step needs two block-wide barriers.
#pragma once

#include "asgd_step_tail.cuh"

namespace asgd {

constexpr int STREAM_THREADS = 128;
constexpr int STREAM_WARPS = STREAM_THREADS / 32;
constexpr int STREAM_STAGES = 2;
constexpr int STREAM_SPT = 4;                          // samples per thread = 32-row blocks per warp
constexpr int STREAM_MAX_B = STREAM_THREADS * STREAM_SPT;
constexpr int STREAM_WARP_SAMPLES = 32 * STREAM_SPT;
constexpr int STREAM_GROUP = 8;                        // rows of one centre added by one lane
constexpr unsigned STREAM_WAIT_LIMIT = 1u << 22;       // bounded mbarrier wait (iterations of try_wait)

__device__ inline unsigned smem_u32(const void* p) { return (unsigned)__cvta_generic_to_shared(p); }
__device__ inline void mbar_init(unsigned long long* bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ inline void mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ inline bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Returns false when the wait ran out (the caller reports it and leaves).
__device__ inline bool mbar_wait_bounded(unsigned long long* bar, unsigned parity) {
  for (unsigned it = 0; it < STREAM_WAIT_LIMIT; ++it)
    if (mbar_try_wait(bar, parity)) return true;
  return false;
}
__device__ inline void bulk_g2s(void* dst, const void* src, unsigned bytes, unsigned long long* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// three-input minimum (one instruction on sm_100)
__device__ inline float fmin3(float a, float b, float c) {
  float r;
  asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
  return r;
}
__device__ inline void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ inline unsigned ld_relaxed_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

template <int D, int K>
struct StreamLayout {
  static_assert(D % 2 == 0 && D <= 16 && K <= 16, "streaming path: even d <= 16, k <= 16");
  static constexpr int DP = (D + 3) / 4 * 4;        // padded row of -2w for 128-bit loads
  static constexpr int D2 = D / 2;                  // dimension pairs
  static constexpr int INDEX_BITS = (K <= 2) ? 1 : (K <= 4) ? 2 : (K <= 8) ? 3 : 4;
  static constexpr unsigned INDEX_MASK = (1u << INDEX_BITS) - 1u;
  static constexpr int CPW = 32 / D;                // centres a warp updates at a time
  static constexpr int ROWB = D * 4;                // bytes per sample
  static constexpr int ZR_EXTRA = (16 + ROWB - 1) / ROWB;   // rows between the batch's last row and the row of zeros (a copy may overrun by < 16 bytes)
  static constexpr int CWS = (K + 1 + 3) / 4 * 4;   // a warp's counts per centre, one spare counter for rows past the batch
  // a warp's rows ordered by centre, every centre's run padded to whole groups
  static constexpr int CAP = (STREAM_WARP_SAMPLES + (STREAM_GROUP - 1) * K + STREAM_GROUP - 1) / STREAM_GROUP * STREAM_GROUP;
  static constexpr int NGRP = CAP / STREAM_GROUP;   // groups a warp can have
  static_assert(NGRP <= 32, "one lane per group");
};

// Shared-memory map of the streaming kernel (byte offsets, every region 16-byte aligned).
template <int D, int K>
struct StreamSmem {
  using L = StreamLayout<D, K>;
  size_t ring, bars, flags, tail, wneg2, cnorm, w, sd, cw, cq, first, cnt, seen, order, gsum, total;
  // a ring slot: the batch (source rounded out to 16-byte bounds), then a row of zeros wherever the batch starts in the slot
  __host__ __device__ static size_t slot_bytes(int b) {
    return ((size_t)(b + L::ZR_EXTRA) * L::ROWB + 16 + L::ROWB + 127) / 128 * 128;
  }
  __host__ __device__ explicit StreamSmem(int b) {
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 15) / 16 * 16; return o; };
    ring = take(STREAM_STAGES * slot_bytes(b));
    bars = take(64);
    flags = take(64);
    tail = take(sizeof(TailScratch));
    wneg2 = take((size_t)K * L::DP * 4);
    cnorm = take((size_t)K * 8);                                // (||w_a||^2, 0) pairs
    w = take((size_t)K * D * 4);
    sd = take((size_t)K * D * 4);
    cw = take((size_t)STREAM_WARPS * L::CWS * 4);               // rows per (warp, centre)
    cq = take((size_t)STREAM_WARPS * STREAM_SPT * L::CWS * 4);  // rows per (warp, 32-row block, centre)
    first = take((size_t)STREAM_WARPS * L::CWS * 4);            // first group of (warp, centre); entry K = groups of the warp
    cnt = take((size_t)K * 4);
    seen = take((size_t)MAX_SLOTS * 4);
    order = take((size_t)STREAM_WARPS * L::CAP * 2);            // u16 byte offsets of rows in the tile, by centre
    gsum = take((size_t)STREAM_WARPS * L::NGRP * D * 4);        // sums of the groups
    total = (off + 127) / 128 * 128;
  }
};
template <int D, int K>
inline size_t stream_smem_bytes(int b) { return StreamSmem<D, K>(b).total; }

template <int D, int K, bool kDet>
__global__ void __launch_bounds__(STREAM_THREADS, 4)
asgd_stream_kernel(const Params p, const long long steps) {
  using L = StreamLayout<D, K>;
  constexpr int DP = L::DP, D2 = L::D2, KD = K * D, ROWB = L::ROWB, CWS = L::CWS, CAP = L::CAP, NGRP = L::NGRP;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int b = p.b;
  const unsigned slot_bytes = (unsigned)StreamSmem<D, K>::slot_bytes(b);
  const unsigned zr_off = (unsigned)(b + L::ZR_EXTRA) * ROWB;              // from a batch's first row to the row of zeros
  const StreamSmem<D, K> map(b);
  unsigned char* ring = smem_raw + map.ring;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + map.bars);   // [STAGES]
  int* flags = reinterpret_cast<int*>(smem_raw + map.flags);                               // [0] a buffer has news
  TailScratch* ts = reinterpret_cast<TailScratch*>(smem_raw + map.tail);
  float* wneg2 = reinterpret_cast<float*>(smem_raw + map.wneg2);
  float2* cnorm = reinterpret_cast<float2*>(smem_raw + map.cnorm);
  float* w = reinterpret_cast<float*>(smem_raw + map.w);
  float* SD = reinterpret_cast<float*>(smem_raw + map.sd);
  int* Cw = reinterpret_cast<int*>(smem_raw + map.cw);
  int* Cq = reinterpret_cast<int*>(smem_raw + map.cq);
  int* First = reinterpret_cast<int*>(smem_raw + map.first);
  float* Gsum = reinterpret_cast<float*>(smem_raw + map.gsum);
  int* cnt = reinterpret_cast<int*>(smem_raw + map.cnt);
  unsigned* seen_s = reinterpret_cast<unsigned*>(smem_raw + map.seen);
  unsigned short* order = reinterpret_cast<unsigned short*>(smem_raw + map.order);

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int i = blockIdx.x;
  float* wglob = p.state + (size_t)i * p.kd_pad;
  const unsigned char* Xend = reinterpret_cast<const unsigned char*>(p.X + (size_t)p.N * D);
  const unsigned char* shard = reinterpret_cast<const unsigned char*>(p.X + (size_t)i * p.H * D);
  const unsigned batch_bytes = (unsigned)b * D * 4;
  const float inv_b = 1.0f / (float)b;
  const float eps = p.eps;

  // state on chip: w, -2w (padded rows), (||w_a||^2, 0)
  for (int e = tid; e < K * DP; e += STREAM_THREADS) wneg2[e] = 0.f;
  for (int e = tid; e < STREAM_STAGES * (4 + D); e += STREAM_THREADS)       // the zeros behind each slot's batch, never overwritten
    reinterpret_cast<float*>(ring + (size_t)(e / (4 + D)) * slot_bytes + zr_off)[e % (4 + D)] = 0.f;
  __syncthreads();
  for (int e = tid; e < KD; e += STREAM_THREADS) {
    const float v = wglob[e];
    w[e] = v;
    wneg2[(e / D) * DP + (e % D)] = -2.f * v;
  }
  if (tid < K) cnt[tid] = 0;
  if (tid < p.S) seen_s[tid] = p.seen[(size_t)i * p.S + tid];
  if (tid == 0) {
    for (int q = 0; q < STREAM_STAGES; ++q) mbar_init(bars + q, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    flags[0] = 0;
  }
  __syncthreads();
  if (tid < K) {
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < D; ++j) s = fmaf(w[tid * D + j], w[tid * D + j], s);
    cnorm[tid] = make_float2(s, 0.f);
  }

  unsigned long long t = p.stats[(size_t)i * ST_STRIDE + ST_STEPS];
  // 32-bit running positions: place in the batch order, steps left until the next put
  const int* myperm = p.perm + (size_t)i * p.B;
  const int nB = (int)p.B;
  const int pos = (int)(t % (unsigned long long)p.B);
  const bool puts_on = p.c > 0 && p.f > 0 && p.W > 1;
  int to_put = puts_on ? p.c - (int)(t % (unsigned long long)p.c) : 0x7fffffff;   // a put is due at 1
  auto next_pos = [&](int q) { return q + 1 == nB ? 0 : q + 1; };

  // a batch's copy: source rounded down to 16 bytes, size rounded up; `head` = bytes to skip
  auto tile_src = [&](int batch, unsigned& head, unsigned& bytes) -> const unsigned char* {
    const unsigned char* src = shard + (size_t)batch * batch_bytes;
    head = (unsigned)((uintptr_t)src & 15);
    bytes = (head + batch_bytes + 15u) & ~15u;
    return src - head;
  };
  auto issue = [&](int batch, int slot) {
    unsigned head, bytes;
    const unsigned char* src = tile_src(batch, head, bytes);
    if (src + bytes <= Xend) {
      mbar_expect_tx(bars + slot, bytes);
      bulk_g2s(ring + (size_t)slot * slot_bytes, src, bytes, bars + slot);
    } else {
      mbar_expect_tx(bars + slot, 0);       // phase completes at once; consumers load the tile themselves
    }
  };

  // batch indices are read one step ahead so that no step waits on that load
  int pos1 = next_pos(pos);
  int batch_cur = myperm[pos];
  int batch_nxt = myperm[pos1];
  if (tid == 0 && steps > 0) issue(batch_cur, 0);
  __syncthreads();

  const float tau_scale = (float)(4 * D + 72) * 5.9604645e-8f;
  const float xmax2 = p.xmax2;                                              // max ||x||^2 over the samples
  int* myCw = Cw + wid * CWS;
  int* myCq = Cq + wid * (STREAM_SPT * CWS);
  int* myFirst = First + wid * CWS;
  unsigned short* myOrder = order + (size_t)wid * CAP;
  float* myGsum = Gsum + (size_t)wid * (NGRP * D);
  // total of centre a, dimension j over the warps' groups, in a fixed order
  auto centre_sum = [&](int a, int j) {
    constexpr int AHEAD = 4;                         // groups of a (warp, centre) whose loads are issued at once
    int g0[STREAM_WARPS], g1[STREAM_WARPS];
#pragma unroll
    for (int q = 0; q < STREAM_WARPS; ++q) { g0[q] = First[q * CWS + a]; g1[q] = First[q * CWS + a + 1]; }
    float v[STREAM_WARPS][AHEAD];
#pragma unroll
    for (int q = 0; q < STREAM_WARPS; ++q)
#pragma unroll
      for (int u = 0; u < AHEAD; ++u) v[q][u] = (g0[q] + u < g1[q]) ? Gsum[(size_t)(q * NGRP + g0[q] + u) * D + j] : 0.f;
    float ssum = 0.f;
#pragma unroll
    for (int q = 0; q < STREAM_WARPS; ++q) {
#pragma unroll
      for (int u = 0; u < AHEAD; ++u) ssum += v[q][u];
      for (int g = g0[q] + AHEAD; g < g1[q]; ++g) ssum += Gsum[(size_t)(q * NGRP + g) * D + j];
    }
    return ssum;
  };
  int abort = 0;
  for (long long step = 0; step < steps; ++step, ++t) {
    const int slot = (int)(step & 1);
    const unsigned parity = (unsigned)((step >> 1) & 1);

    // start the next batch's copy; peek at the receive buffers' sequence numbers (used after the sums)
    if (tid == 0 && step + 1 < steps) {
      fence_proxy_async_smem();
      issue(batch_nxt, slot ^ 1);
    }
    unsigned my_seq = 0;
    if (tid < p.S) my_seq = ld_relaxed_gpu(p.seq + (size_t)i * p.S + tid);
    const int pos2 = next_pos(pos1);
    const int batch_nn = myperm[pos2];
    {
      // this warp's order: every entry points at the row of zeros, counts zero
      const unsigned zz = zr_off | (zr_off << 16);
      if (lane < NGRP) reinterpret_cast<uint4*>(myOrder)[lane] = make_uint4(zz, zz, zz, zz);
      if (lane < STREAM_SPT * CWS / 4) reinterpret_cast<uint4*>(myCq)[lane] = make_uint4(0u, 0u, 0u, 0u);
    }

    unsigned head, bytes;
    const unsigned char* src = tile_src(batch_cur, head, bytes);
    unsigned char* tile = ring + (size_t)slot * slot_bytes;
    if (!mbar_wait_bounded(bars + slot, parity)) abort = 1;
    if (src + bytes > Xend) {
      // last rows of X: a rounded bulk copy would run past the array, use plain loads
      const float* g = reinterpret_cast<const float*>(src + head);
      float* sdst = reinterpret_cast<float*>(tile + head);
      for (int e = tid; e < b * D; e += STREAM_THREADS) sdst[e] = __ldg(g + e);
      __syncthreads();
    }
    const float* xs = reinterpret_cast<const float*>(tile + head);

    // ---- Eq. 8: scores of this thread's samples against every centre ----
    float2 xv[STREAM_SPT][D2];
#pragma unroll
    for (int q = 0; q < STREAM_SPT; ++q) {
      const int r = min(wid * STREAM_WARP_SAMPLES + q * 32 + lane, b - 1);   // rows past the batch re-read its last row
      const float2* xrow = reinterpret_cast<const float2*>(xs + (size_t)r * D);
#pragma unroll
      for (int jp = 0; jp < D2; ++jp) xv[q][jp] = xrow[jp];
    }
    float s1[STREAM_SPT], s2[STREAM_SPT];
#pragma unroll
    for (int q = 0; q < STREAM_SPT; ++q) { s1[q] = __int_as_float(0x7f800000); s2[q] = __int_as_float(0x7f800000); }
    float wmax2 = 0.f;
    // packed score of centre a for each of the thread's samples
    auto scores_of = [&](int a, float (&sp)[STREAM_SPT]) {
      float2 wr[DP / 2];
#pragma unroll
      for (int j4 = 0; j4 < DP / 4; ++j4) {
        const float4 v = *reinterpret_cast<const float4*>(wneg2 + a * DP + 4 * j4);
        wr[2 * j4] = make_float2(v.x, v.y);
        wr[2 * j4 + 1] = make_float2(v.z, v.w);
      }
      const float2 cn = cnorm[a];                       // (||w_a||^2, 0)
      wmax2 = fmaxf(wmax2, cn.x);
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) {
        float2 acc = cn;
#pragma unroll
        for (int jp = 0; jp < D2; ++jp) acc = __ffma2_rn(xv[q][jp], wr[jp], acc);
        const float sc = acc.x + acc.y;
        sp[q] = __uint_as_float((__float_as_uint(sc) & ~L::INDEX_MASK) | (unsigned)a);
      }
    };
    // two centres at a time: with lo <= hi the new pair is  s1' = min(s1, lo),  s2' = min(max(s1, lo), s2, hi)
#pragma unroll 1
    for (int a = 0; a + 1 < K; a += 2) {
      float pa[STREAM_SPT], pb[STREAM_SPT];
      scores_of(a, pa);
      scores_of(a + 1, pb);
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) {
        const float lo = fminf(pa[q], pb[q]), hi = fmaxf(pa[q], pb[q]);
        s2[q] = fmin3(fmaxf(s1[q], lo), s2[q], hi);
        s1[q] = fminf(s1[q], lo);
      }
    }
    if (K & 1) {
      float pa[STREAM_SPT];
      scores_of(K - 1, pa);
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) {
        s2[q] = fmaxf(s1[q], fminf(s2[q], pa[q]));
        s1[q] = fminf(s1[q], pa[q]);
      }
    }

    // ---- decide: index from the packed minimum; direct differences when the runner-up is too close ----
    int best[STREAM_SPT];
#pragma unroll
    for (int q = 0; q < STREAM_SPT; ++q) {
      best[q] = (int)(__float_as_uint(s1[q]) & L::INDEX_MASK);
      if (K > 1 && (s2[q] - s1[q]) <= tau_scale * (wmax2 + xmax2)) {       // cheap test with the global bound on ||x||^2 first
        float2 n2 = __fmul2_rn(xv[q][0], xv[q][0]);
#pragma unroll
        for (int jp = 1; jp < D2; ++jp) n2 = __ffma2_rn(xv[q][jp], xv[q][jp], n2);
        if ((s2[q] - s1[q]) <= tau_scale * (wmax2 + (n2.x + n2.y))) {
          float bd = __int_as_float(0x7f800000);
          int bb = 0;
          for (int a = 0; a < K; ++a) {
            float acc = 0.f;
#pragma unroll
            for (int jp = 0; jp < D2; ++jp) {
              const float d0 = xv[q][jp].x + 0.5f * wneg2[a * DP + 2 * jp];        // -0.5 * (-2w) = w, exact
              const float d1 = xv[q][jp].y + 0.5f * wneg2[a * DP + 2 * jp + 1];
              acc = fmaf(d0, d0, acc);
              acc = fmaf(d1, d1, acc);
            }
            if (acc < bd) { bd = acc; bb = a; }          // strict "<": the lowest index keeps a tie
          }
          best[q] = bb;
        }
      }
      if (wid * STREAM_WARP_SAMPLES + q * 32 + lane >= b) best[q] = K;   // rows past the batch form their own group
    }
    if (p.assign_rec) {
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) {
        const int r = wid * STREAM_WARP_SAMPLES + q * 32 + lane;
        if (r < b) p.assign_rec[(size_t)i * b + r] = best[q];
      }
    }
    // ---- order: this warp's rows by the centre they chose, in row order inside a centre ----
    __syncwarp();
    int rank[STREAM_SPT];
    int ngroups;
#pragma unroll
    for (int q = 0; q < STREAM_SPT; ++q) {
      const unsigned grp = __match_any_sync(0xffffffffu, best[q]);
      const unsigned below = grp & ((1u << lane) - 1u);
      rank[q] = __popc(below);
      if (below == 0) myCq[q * CWS + best[q]] = __popc(grp);               // rows past the batch count into the spare counter
    }
    if (tid < p.S && my_seq != seen_s[tid]) flags[0] = 1;
    __syncwarp();
    {
      // a row's place inside its centre: the centre's rows in the earlier 32-row blocks, then its rank in its own
#pragma unroll
      for (int q = 1; q < STREAM_SPT; ++q) {
        int before = 0;
#pragma unroll
        for (int r = 0; r < q; ++r) before += myCq[r * CWS + best[q]];
        rank[q] += before;
      }
      // lane = centre: its rows, its groups, and the first group by a running sum (lane K gets the total)
      int n = 0;
      if (lane < K) {
#pragma unroll
        for (int q = 0; q < STREAM_SPT; ++q) n += myCq[q * CWS + lane];
        myCw[lane] = n;
      }
      const int ng = (n + STREAM_GROUP - 1) / STREAM_GROUP;
      int inc = ng;
#pragma unroll
      for (int o = 1; o <= K; o <<= 1) {
        const int up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
      }
      const int first = inc - ng;
      if (lane <= K) myFirst[lane] = first;
      ngroups = __shfl_sync(0xffffffffu, inc, K);
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) {
        const int f = __shfl_sync(0xffffffffu, first, best[q]);            // best[q] <= K
        if (best[q] < K)
          myOrder[f * STREAM_GROUP + rank[q]] = (unsigned short)((wid * STREAM_WARP_SAMPLES + q * 32 + lane) * ROWB);
      }
    }
    __syncwarp();

    // ---- Eq. 9: lanes (group, dimension pair) add the eight rows of a group (all of one centre) from the tile ----
    {
      constexpr int GPR = 32 / D2;                                         // groups a warp adds at a time
      const int gl = lane / D2, jp = lane - gl * D2;
      const unsigned char* xb = reinterpret_cast<const unsigned char*>(xs) + jp * 8;
      auto row = [&](unsigned off) { return *reinterpret_cast<const float2*>(xb + off); };
      for (int g = gl; g < ngroups; g += GPR) {
        if (gl < GPR) {
          const uint4 pk = reinterpret_cast<const uint4*>(myOrder)[g];
          float2 acc0 = row(pk.x & 0xffffu), acc1 = row(pk.x >> 16);
          acc0 = __fadd2_rn(acc0, row(pk.y & 0xffffu)); acc1 = __fadd2_rn(acc1, row(pk.y >> 16));
          acc0 = __fadd2_rn(acc0, row(pk.z & 0xffffu)); acc1 = __fadd2_rn(acc1, row(pk.z >> 16));
          acc0 = __fadd2_rn(acc0, row(pk.w & 0xffffu)); acc1 = __fadd2_rn(acc1, row(pk.w >> 16));
          *reinterpret_cast<float2*>(myGsum + (size_t)g * D + 2 * jp) = __fadd2_rn(acc0, acc1);
        }
      }
    }

    // ---- barrier B: group sums and counts complete, the ring slot is free again ----
    if (__syncthreads_or(abort)) { abort = 1; break; }

    const bool put_now = (to_put == 1);
    if (flags[0] != 0) {
      // a message is waiting: totals into SD, then the general tail (which also sends when a put is due)
      for (int e = tid; e < KD; e += STREAM_THREADS) SD[e] = centre_sum(e / D, e % D);
      if (tid < K) {
        int n = 0;
#pragma unroll
        for (int q = 0; q < STREAM_WARPS; ++q) n += Cw[q * CWS + tid];
        cnt[tid] = n;
      }
      __syncthreads();
      step_tail<kDet>(p, i, t, w, D, SD, cnt, wglob, ts);
      if (tid < p.S) seen_s[tid] = p.seen[(size_t)i * p.S + tid];
      if (tid == 0) flags[0] = 0;
      if (tid < K) cnt[tid] = 0;
      for (int e = tid; e < KD; e += STREAM_THREADS) wneg2[(e / D) * DP + (e % D)] = -2.f * w[e];
      if (tid < K) {
        float s = 0.f;
#pragma unroll
        for (int j = 0; j < D; ++j) s = fmaf(w[tid * D + j], w[tid * D + j], s);
        cnorm[tid] = make_float2(s, 0.f);
      }
    } else {
      // common case: plain local step  w <- w - eps * D,  D = (n_a w - S) / b.  A warp updates CPW
      // centres at a time, lane = (centre, dimension), and reduces ||w_a||^2 over the centre's lanes.
      for (int a0 = wid * L::CPW; a0 < K; a0 += STREAM_WARPS * L::CPW) {
        const int a = a0 + lane / D, j = lane % D;
        const bool on = (lane < L::CPW * D) && (a < K);
        float sq = 0.f;
        if (on) {
          int n = 0;
#pragma unroll
          for (int q = 0; q < STREAM_WARPS; ++q) n += Cw[q * CWS + a];
          const float ssum = centre_sum(a, j);
          const float ww = w[a * D + j];
          const float Dg = ((float)n * ww - ssum) * inv_b;
          const float nw = ww - eps * Dg;
          w[a * D + j] = nw;
          wneg2[a * DP + j] = -2.f * nw;
          wglob[a * D + j] = nw;
          sq = nw * nw;
        }
#pragma unroll
        for (int o = 1; o < D; o <<= 1) {
          const float up = __shfl_down_sync(0xffffffffu, sq, o);
          if (j + o < D) sq += up;
        }
        __syncwarp();
        if (on && j == 0) cnorm[a] = make_float2(sq, 0.f);
      }
      unsigned long long n_sent = 0;
      if (put_now) {
        __syncthreads();                                 // the new w is complete
        n_sent = step_send_any<kDet>(p, i, t, w, D, ts);
      }
      if (kDet && p.rows_m > 0)                            // per-row record of a step that looked at no message
        for (int a = tid; a < p.k; a += STREAM_THREADS) p.rowin[(size_t)i * p.k + a] = 0;
      if (tid == 0) {
        if (kDet)
          for (int s = 0; s < p.S; ++s) p.accept_rec[(size_t)i * p.S + s] = -1;
        unsigned long long* st = p.stats + (size_t)i * ST_STRIDE;
        st[ST_STEPS] = t + 1;
        if (n_sent) atomicAdd(st + ST_SENT, n_sent);
      }
    }
    batch_cur = batch_nxt;
    batch_nxt = batch_nn;
    pos1 = pos2;
    if (puts_on) to_put = (to_put == 1) ? p.c : to_put - 1;
    __syncthreads();                                   // barrier E: w, -2w, ||w||^2 ready for the next step
  }

  if (abort) {
    if (tid == 0) atomicExch(p.status, DEV_TIMEOUT);
    // a copy may still be in flight into this block's shared memory: give it a bounded chance to land
    for (int q = 0; q < STREAM_STAGES; ++q) {
      mbar_wait_bounded(bars + q, 0);
      mbar_wait_bounded(bars + q, 1);
    }
  }
}

}  // namespace asgd
