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
constexpr unsigned DEFAULT_WAIT_LIMIT = 1u << 22;      // bounded mbarrier wait (iterations of try_wait), Params::wait_limit

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
__device__ inline bool mbar_wait_bounded(unsigned long long* bar, unsigned parity, unsigned limit) {
  for (unsigned it = 0; it < limit; ++it)
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

// Shared-memory accesses of the order and sum phases: 32-bit shared addresses with constant offsets, so that an
// access costs one instruction and no 64-bit address arithmetic.
template <int OFF> __device__ __forceinline__ unsigned lds_u32(unsigned a) {
  unsigned v;
  asm volatile("ld.shared.u32 %0, [%1+%2];" : "=r"(v) : "r"(a), "n"(OFF) : "memory");
  return v;
}
template <int OFF> __device__ __forceinline__ uint4 lds_v4(unsigned a) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4+%5];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a), "n"(OFF) : "memory");
  return v;
}
template <int OFF> __device__ __forceinline__ float2 lds_f2(unsigned a) {
  float2 v;
  asm volatile("ld.shared.v2.f32 {%0,%1}, [%2+%3];" : "=f"(v.x), "=f"(v.y) : "r"(a), "n"(OFF) : "memory");
  return v;
}
template <int OFF> __device__ __forceinline__ void sts_u32(unsigned a, unsigned v) {
  asm volatile("st.shared.u32 [%0+%2], %1;" ::"r"(a), "r"(v), "n"(OFF) : "memory");
}
template <int OFF> __device__ __forceinline__ void sts_u32_if(unsigned a, unsigned v, unsigned on) {
  asm volatile("{\n .reg .pred p;\n setp.ne.u32 p, %3, 0;\n @p st.shared.u32 [%0+%2], %1;\n}" ::"r"(a), "r"(v), "n"(OFF), "r"(on) : "memory");
}
template <int OFF> __device__ __forceinline__ void sts_v4(unsigned a, unsigned v) {
  asm volatile("st.shared.v4.u32 [%0+%2], {%1,%1,%1,%1};" ::"r"(a), "r"(v), "n"(OFF) : "memory");
}
template <int OFF> __device__ __forceinline__ void sts_f2(unsigned a, float2 v) {
  asm volatile("st.shared.v2.f32 [%0+%3], {%1,%2};" ::"r"(a), "f"(v.x), "f"(v.y), "n"(OFF) : "memory");
}
// running sum step: v += (value of the lane `o` below), lanes below `o` keep v
__device__ __forceinline__ int scan_step(int v, int o) {
  int r;
  asm volatile("{\n .reg .pred p;\n .reg .b32 t;\n shfl.sync.up.b32 t|p, %1, %2, 0, 0xffffffff;\n @p add.s32 t, t, %1;\n @!p mov.b32 t, %1;\n mov.b32 %0, t;\n}" : "=r"(r) : "r"(v), "r"(o));
  return r;
}

constexpr size_t stream_up16(size_t x) { return (x + 15) / 16 * 16; }

// Sizes and the shared-memory map of the streaming kernel.  Everything but the ring has a place that depends on
// (d, k) only, so those byte offsets are constants in the code; the ring (whose slots depend on b) comes last.
template <int D, int K>
struct StreamLayout {
  static_assert(D % 2 == 0 && D <= 16 && K <= 16, "streaming path: even d <= 16, k <= 16");
  static constexpr int DP = (D + 3) / 4 * 4;        // padded row of -2w for 128-bit loads
  static constexpr int D2 = D / 2;                  // dimension pairs
  static constexpr int INDEX_BITS = (K <= 2) ? 1 : (K <= 4) ? 2 : (K <= 8) ? 3 : 4;
  static constexpr unsigned INDEX_MASK = (1u << INDEX_BITS) - 1u;
  static constexpr int ROWB = D * 4;                // bytes per sample
  static constexpr int CWS = (K + 1 + 3) / 4 * 4;   // a warp's counts per centre, one spare counter for rows past the batch
  static constexpr int GPR = 32 / D2;               // groups a warp adds at a time: lanes (group, dimension pair)
  static constexpr int CPW = GPR;                   // centres a warp updates: lanes (centre, dimension pair)
  static constexpr int UPD_WARPS = (K + CPW - 1) / CPW;
  static_assert(UPD_WARPS <= STREAM_WARPS, "update: every centre has a warp");
  // a warp's rows ordered by centre, every centre's run padded to whole groups of eight
  static constexpr int NGRP = (STREAM_WARP_SAMPLES + (STREAM_GROUP - 1) * K + STREAM_GROUP - 1) / STREAM_GROUP;
  static constexpr int GCAP = (NGRP + 2 * GPR - 1) / (2 * GPR) * (2 * GPR);   // groups the adders may touch (whole double rounds)
  static_assert(NGRP <= 32, "a running sum over one warp covers the groups");

  // fixed part of the map (byte offsets)
  static constexpr size_t BARS = 0;
  static constexpr size_t FLAGS = 64;
  static constexpr size_t ZROW = 128;                                    // a row of zeros for the unused tail of a group
  static constexpr size_t TAIL = ZROW + stream_up16(ROWB + 16);
  static constexpr size_t WNEG2 = TAIL + stream_up16(sizeof(TailScratch));
  static constexpr size_t CNORM = WNEG2 + stream_up16((size_t)K * DP * 4);   // (||w_a||^2, 0) pairs
  static constexpr size_t W = CNORM + stream_up16((size_t)K * 8);
  static constexpr size_t SD = W + stream_up16((size_t)K * D * 4);
  static constexpr size_t CNT = SD + stream_up16((size_t)K * D * 4);
  static constexpr size_t SEEN = CNT + stream_up16((size_t)K * 4);
  static constexpr size_t WARP0 = SEEN + stream_up16((size_t)MAX_SLOTS * 4);
  // per warp: rows per (32-row block, centre); rows per centre; first group per centre; the order; the group sums
  static constexpr size_t W_CQ = 0;
  static constexpr size_t W_CW = W_CQ + (size_t)STREAM_SPT * CWS * 4;
  static constexpr size_t W_FIRST = W_CW + (size_t)CWS * 4;
  static constexpr size_t W_ORDER = W_FIRST + (size_t)CWS * 4;           // u32 shared addresses of rows
  static constexpr size_t W_GSUM = W_ORDER + (size_t)GCAP * STREAM_GROUP * 4;
  static constexpr size_t WARP_STRIDE = stream_up16(W_GSUM + (size_t)GCAP * D * 4);
  static constexpr size_t RING = (WARP0 + STREAM_WARPS * WARP_STRIDE + 127) / 128 * 128;
  // a ring slot: the batch with its source rounded out to 16-byte bounds
  __host__ __device__ static size_t slot_bytes(int b) { return ((size_t)b * ROWB + 32 + 127) / 128 * 128; }
  __host__ __device__ static size_t total(int b) { return RING + STREAM_STAGES * slot_bytes(b); }
};
template <int D, int K>
inline size_t stream_smem_bytes(int b) { return StreamLayout<D, K>::total(b); }

template <int D, int K, bool kDet>
__global__ void __launch_bounds__(STREAM_THREADS, 4)
asgd_stream_kernel(const Params p, const long long steps) {
  using L = StreamLayout<D, K>;
  constexpr int DP = L::DP, D2 = L::D2, KD = K * D, ROWB = L::ROWB, CWS = L::CWS, GCAP = L::GCAP, GPR = L::GPR;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int b = p.b;
  const unsigned slot_bytes = (unsigned)L::slot_bytes(b);
  unsigned char* ring = smem_raw + L::RING;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + L::BARS);   // [STAGES]
  int* flags = reinterpret_cast<int*>(smem_raw + L::FLAGS);                               // [0] a buffer has news
  TailScratch* ts = reinterpret_cast<TailScratch*>(smem_raw + L::TAIL);
  float* wneg2 = reinterpret_cast<float*>(smem_raw + L::WNEG2);
  float2* cnorm = reinterpret_cast<float2*>(smem_raw + L::CNORM);
  float* w = reinterpret_cast<float*>(smem_raw + L::W);
  float* SD = reinterpret_cast<float*>(smem_raw + L::SD);
  int* cnt = reinterpret_cast<int*>(smem_raw + L::CNT);
  unsigned* seen_s = reinterpret_cast<unsigned*>(smem_raw + L::SEEN);

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int i = blockIdx.x;
  float* wglob = p.state + (size_t)i * p.kd_pad;
  const unsigned char* Xend = reinterpret_cast<const unsigned char*>(p.X + (size_t)p.N * D);
  const unsigned char* shard = reinterpret_cast<const unsigned char*>(p.X + (size_t)i * p.H * D);
  const unsigned batch_bytes = (unsigned)b * D * 4;
  const float inv_b = 1.0f / (float)b;
  const float eps = p.eps;
  // shared addresses (32 bit): the block's base, this warp's arrays, the row of zeros
  const unsigned sbase = smem_u32(smem_raw);
  const unsigned wb = sbase + (unsigned)L::WARP0 + (unsigned)wid * (unsigned)L::WARP_STRIDE;
  const unsigned zrow = sbase + (unsigned)L::ZROW;
  auto warp_ptr = [&](int q, size_t off) { return smem_raw + L::WARP0 + (size_t)q * L::WARP_STRIDE + off; };

  // state on chip: w, -2w (padded rows), (||w_a||^2, 0)
  for (int e = tid; e < K * DP; e += STREAM_THREADS) wneg2[e] = 0.f;
  for (int e = tid; e < (ROWB + 16) / 4; e += STREAM_THREADS) reinterpret_cast<float*>(smem_raw + L::ZROW)[e] = 0.f;
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
  auto issue = [&](int batch, int slot, long long s) {   // s: the step of this launch that uses the batch
    unsigned head, bytes;
    const unsigned char* src = tile_src(batch, head, bytes);
    if (src + bytes <= Xend) {
      mbar_expect_tx(bars + slot, bytes);
      if (s != p.withhold_step) bulk_g2s(ring + (size_t)slot * slot_bytes, src, bytes, bars + slot);
    } else {
      mbar_expect_tx(bars + slot, 0);       // phase completes at once; consumers load the tile themselves
    }
  };

  // batch indices are read one step ahead so that no step waits on that load
  int pos1 = next_pos(pos);
  int batch_cur = myperm[pos];
  int batch_nxt = myperm[pos1];
  if (tid == 0 && steps > 0) {
    issue(batch_cur, 0, 0);
    if (steps > 1) issue(batch_nxt, 1, 1);
  }
  __syncthreads();

  const float tau_scale = (float)(4 * D + 72) * 5.9604645e-8f;
  const float xmax2 = p.xmax2;                                              // max ||x||^2 over the samples
  const unsigned lane_lt = (1u << lane) - 1u;
  const int lane_c = min(lane, K);                                         // lanes past the centres share the spare column
  const unsigned row0 = (unsigned)((wid * STREAM_WARP_SAMPLES + lane) * ROWB);   // this thread's first row in a tile

  // total of centre a, dimension pair jp over the warps' groups, in a fixed order
  auto centre_sum = [&](int a, int jp) {
    constexpr int AHEAD = 4;                         // groups of a (warp, centre) whose loads are issued at once
    float2 part[STREAM_WARPS];
#pragma unroll
    for (int q = 0; q < STREAM_WARPS; ++q) {
      const int* first = reinterpret_cast<const int*>(warp_ptr(q, L::W_FIRST));
      const float2* gs = reinterpret_cast<const float2*>(warp_ptr(q, L::W_GSUM));
      const int g0 = first[a], ng = first[a + 1] - g0;
      const float2* src = gs + (size_t)g0 * D2 + jp;
      float2 v[AHEAD];
#pragma unroll
      for (int u = 0; u < AHEAD; ++u) v[u] = (u < ng) ? src[u * D2] : make_float2(0.f, 0.f);
      part[q] = __fadd2_rn(__fadd2_rn(v[0], v[1]), __fadd2_rn(v[2], v[3]));
      for (int u = AHEAD; u < ng; ++u) part[q] = __fadd2_rn(part[q], src[u * D2]);
    }
    return __fadd2_rn(__fadd2_rn(part[0], part[1]), __fadd2_rn(part[2], part[3]));
  };
  auto centre_rows = [&](int a) {
    int n = 0;
#pragma unroll
    for (int q = 0; q < STREAM_WARPS; ++q) n += reinterpret_cast<const int*>(warp_ptr(q, L::W_CW))[a];
    return n;
  };

  int abort = 0;
  // A step's samples: the thread's rows of the batch in registers, the tile's shared address for the sums.
  float2 xv[STREAM_SPT][D2];
  unsigned xsa = 0;
  // Gets batch `batch` (the one of step `s`) ready: resets this warp's order and counts, waits for the copy
  // and loads the thread's rows.  Runs between the two barriers of the step before, beside the update.
  auto stage_in = [&](long long s, int batch) {
    {
      // this warp's order: every entry points at the row of zeros; counts zero
#pragma unroll
      for (int e = 0; e < (GCAP * STREAM_GROUP / 4 + 31) / 32; ++e)
        if (e * 32 + lane < GCAP * STREAM_GROUP / 4) {
          asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(wb + (unsigned)L::W_ORDER + (unsigned)(e * 32 + lane) * 16u), "r"(zrow) : "memory");
        }
      if (lane < STREAM_SPT * CWS / 4)
        asm volatile("st.shared.v4.u32 [%0], {%1,%1,%1,%1};" ::"r"(wb + (unsigned)L::W_CQ + (unsigned)lane * 16u), "r"(0u) : "memory");
    }
    unsigned head, bytes;
    const unsigned char* src = tile_src(batch, head, bytes);
    unsigned char* tile = ring + (size_t)(s & 1) * slot_bytes;
    if (!mbar_wait_bounded(bars + (s & 1), (unsigned)((s >> 1) & 1), p.wait_limit)) abort = 1;
    if (src + bytes > Xend) {
      // last rows of X: a rounded bulk copy would run past the array, use plain loads
      const float* g = reinterpret_cast<const float*>(src + head);
      float* sdst = reinterpret_cast<float*>(tile + head);
      for (int e = tid; e < b * D; e += STREAM_THREADS) sdst[e] = __ldg(g + e);
      __syncthreads();
    }
    const float* xs = reinterpret_cast<const float*>(tile + head);
    xsa = smem_u32(xs);
#pragma unroll
    for (int q = 0; q < STREAM_SPT; ++q) {
      const int r = min(wid * STREAM_WARP_SAMPLES + q * 32 + lane, b - 1);   // rows past the batch re-read its last row
      const float2* xrow = reinterpret_cast<const float2*>(xs + (size_t)r * D);
#pragma unroll
      for (int jp = 0; jp < D2; ++jp) xv[q][jp] = xrow[jp];
    }
  };
  if (steps > 0) stage_in(0, batch_cur);
  for (long long step = 0; step < steps; ++step, ++t) {
    const int slot = (int)(step & 1);

    // peek at the receive buffers' sequence numbers (used after the sums); next batch index but one
    unsigned my_seq = 0;
    if (tid < p.S) my_seq = ld_relaxed_gpu(p.seq + (size_t)i * p.S + tid);
    const int pos2 = next_pos(pos1);
    const int batch_nn = myperm[pos2];

    // ---- Eq. 8: scores of this thread's samples against every centre ----
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
    unsigned cqa[STREAM_SPT];                                              // address of this row's centre in the block counts
#pragma unroll
    for (int q = 0; q < STREAM_SPT; ++q) {
      const unsigned grp = __match_any_sync(0xffffffffu, best[q]);
      const unsigned below = grp & lane_lt;
      rank[q] = __popc(below);
      cqa[q] = wb + (unsigned)L::W_CQ + ((unsigned)best[q] << 2);          // rows past the batch count into the spare column
      if (q == 0) sts_u32_if<0 * CWS * 4>(cqa[q], (unsigned)__popc(grp), below == 0);
      if (q == 1) sts_u32_if<1 * CWS * 4>(cqa[q], (unsigned)__popc(grp), below == 0);
      if (q == 2) sts_u32_if<2 * CWS * 4>(cqa[q], (unsigned)__popc(grp), below == 0);
      if (q == 3) sts_u32_if<3 * CWS * 4>(cqa[q], (unsigned)__popc(grp), below == 0);
    }
    if (tid < p.S && my_seq != seen_s[tid]) flags[0] = 1;
    __syncwarp();
    int ngroups;
    {
      // a row's place inside its centre: the centre's rows in the earlier 32-row blocks, then its rank in its own
      static_assert(STREAM_SPT == 4, "four 32-row blocks per warp");
      rank[1] += (int)lds_u32<0>(cqa[1]);
      rank[2] += (int)(lds_u32<0>(cqa[2]) + lds_u32<CWS * 4>(cqa[2]));
      rank[3] += (int)(lds_u32<0>(cqa[3]) + lds_u32<CWS * 4>(cqa[3]) + lds_u32<2 * CWS * 4>(cqa[3]));
      // lane = centre: its rows, its groups, and the first group by a running sum (entry K holds the total)
      const unsigned ca = wb + (unsigned)L::W_CQ + ((unsigned)lane_c << 2);
      int n = (int)(lds_u32<0>(ca) + lds_u32<CWS * 4>(ca) + lds_u32<2 * CWS * 4>(ca) + lds_u32<3 * CWS * 4>(ca));
      n = (lane < K) ? n : 0;
      sts_u32<(int)(L::W_CW - L::W_CQ)>(ca, (unsigned)n);
      const int ng = (n + STREAM_GROUP - 1) / STREAM_GROUP;
      int inc = ng;
#pragma unroll
      for (int o = 1; o < K; o <<= 1) inc = scan_step(inc, o);
      const int first = inc - ng;
      ngroups = __shfl_sync(0xffffffffu, inc, K - 1);                      // the running sum reaches K - 1 lanes down
      sts_u32<(int)(L::W_FIRST - L::W_CQ)>(ca, (unsigned)((lane < K) ? first : ngroups));
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) {
        const int f = __shfl_sync(0xffffffffu, first, best[q]);            // best[q] <= K
        const unsigned at = wb + (unsigned)L::W_ORDER + (((unsigned)f * STREAM_GROUP + (unsigned)rank[q]) << 2);
        sts_u32_if<0>(at, xsa + row0 + (unsigned)(q * 32 * ROWB), best[q] < K);
      }
    }
    __syncwarp();

    // ---- Eq. 9: lanes (group, dimension pair) add the eight rows of a group (all of one centre) from the tile ----
    {
      const int gl = lane / D2, jp = lane - gl * D2;
      const unsigned jo = (unsigned)jp * 8u;
      auto group_sum = [&](const uint4& lo, const uint4& hi) {
        float2 acc0 = lds_f2<0>(lo.x + jo), acc1 = lds_f2<0>(lo.y + jo);
        acc0 = __fadd2_rn(acc0, lds_f2<0>(lo.z + jo)); acc1 = __fadd2_rn(acc1, lds_f2<0>(lo.w + jo));
        acc0 = __fadd2_rn(acc0, lds_f2<0>(hi.x + jo)); acc1 = __fadd2_rn(acc1, lds_f2<0>(hi.y + jo));
        acc0 = __fadd2_rn(acc0, lds_f2<0>(hi.z + jo)); acc1 = __fadd2_rn(acc1, lds_f2<0>(hi.w + jo));
        return __fadd2_rn(acc0, acc1);
      };
      // two groups per lane in flight; groups past the last one hold the row of zeros
      if (gl < GPR) {
        for (int g = gl; g < ngroups; g += 2 * GPR) {
          const unsigned oa = wb + (unsigned)L::W_ORDER + (unsigned)g * (STREAM_GROUP * 4);
          const uint4 a0 = lds_v4<0>(oa), a1 = lds_v4<16>(oa);
          const uint4 b0 = lds_v4<GPR * STREAM_GROUP * 4>(oa), b1 = lds_v4<GPR * STREAM_GROUP * 4 + 16>(oa);
          const float2 sa = group_sum(a0, a1), sb = group_sum(b0, b1);
          const unsigned ga = wb + (unsigned)L::W_GSUM + (unsigned)g * (D * 4) + jo;
          sts_f2<0>(ga, sa);
          sts_f2<GPR * D * 4>(ga, sb);
        }
      }
    }

    // ---- barrier B: group sums and counts complete, the ring slot is free again ----
    if (__syncthreads_or(abort)) { abort = 1; break; }

    // the slot's rows have been added: start the copy of the batch after the next into it
    if (tid == 0 && step + 2 < steps) {
      fence_proxy_async_smem();
      issue(batch_nn, slot, step + 2);
    }
    const bool put_now = (to_put == 1);
    if (flags[0] != 0) {
      // a message is waiting: totals into SD, then the general tail (which also sends when a put is due)
      for (int e = tid; e < K * D2; e += STREAM_THREADS)
        reinterpret_cast<float2*>(SD)[e] = centre_sum(e / D2, e % D2);
      if (tid < K) cnt[tid] = centre_rows(tid);
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
      // common case: plain local step  w <- w - eps * D,  D = (n_a w - S) / b.  The first warps update CPW
      // centres each, lane = (centre, dimension pair), and reduce ||w_a||^2 over the centre's lanes.
      if (wid < L::UPD_WARPS) {
        const int al = lane / D2, jp = lane - al * D2;
        const int a = wid * L::CPW + al;
        const bool on = (al < L::CPW) && (a < K);
        float sq = 0.f;
        if (on) {
          const int n = centre_rows(a);
          const float2 ssum = centre_sum(a, jp);
          const float2 ww = *reinterpret_cast<const float2*>(w + a * D + 2 * jp);
          float2 nw;
          nw.x = ww.x - eps * (((float)n * ww.x - ssum.x) * inv_b);
          nw.y = ww.y - eps * (((float)n * ww.y - ssum.y) * inv_b);
          *reinterpret_cast<float2*>(w + a * D + 2 * jp) = nw;
          *reinterpret_cast<float2*>(wneg2 + a * DP + 2 * jp) = make_float2(-2.f * nw.x, -2.f * nw.y);
          *reinterpret_cast<float2*>(wglob + a * D + 2 * jp) = nw;
          sq = fmaf(nw.y, nw.y, nw.x * nw.x);
        }
#pragma unroll
        for (int o = 1; o < D2; o <<= 1) {
          const float up = __shfl_down_sync(0xffffffffu, sq, o);
          if (jp + o < D2) sq += up;
        }
        if (on && jp == 0) cnorm[a] = make_float2(sq, 0.f);
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
    if (step + 1 < steps) stage_in(step + 1, batch_cur);
    __syncthreads();                                   // barrier E: w, -2w, ||w||^2 ready for the next step
  }

  if (abort) {
    if (tid == 0) atomicExch(p.status, DEV_TIMEOUT);
    // a copy may still be in flight into this block's shared memory: give it a bounded chance to land
    for (int q = 0; q < STREAM_STAGES; ++q) {
      mbar_wait_bounded(bars + q, 0, p.wait_limit);
      mbar_wait_bounded(bars + q, 1, p.wait_limit);
    }
  }
}

}  // namespace asgd
