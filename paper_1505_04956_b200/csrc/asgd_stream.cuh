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
// Per-centre sums and counts (Eq. 9): S = X^T . onehot(s) is formed by the warp on the tensor cores
// (mma.sync m16n8k8, TF32 operands, fp32 accumulators kept in registers over the warp's 128 rows).
// The one-hot operand is exact; every sample value goes in as two terms, hi = x with the 13 low
// mantissa bits cleared and lo = x - hi (exact in fp32; the tensor core keeps its leading bits), so a
// value enters a sum with a relative error below 2^-21.  The sample fragments come straight from the
// tile (a thread reads the dimension pair 2g, 2g+1 of rows 4 apart: 160 bytes for d = 10, which
// spreads the four rows of an access over all banks).  The counts n_k come out of the same products:
// the threads whose dimension pair lies past d read (1, 0) pairs instead of samples, which makes result
// row d/2 the number of rows per centre (for d = 16, where no result row is spare, a third product with a
// row of ones).  No row is gathered, nothing is sorted, and every sum has a fixed order (a step is
// reproducible bit for bit).
#pragma once

#include "asgd_step_tail.cuh"

namespace asgd {

constexpr int STREAM_SPT = 4;                          // samples per thread = 32-row blocks per warp
constexpr int STREAM_MAX_B = 512;
constexpr int STREAM_WARP_SAMPLES = 32 * STREAM_SPT;
constexpr int STREAM_WARPS = (STREAM_MAX_B + STREAM_WARP_SAMPLES - 1) / STREAM_WARP_SAMPLES;
constexpr int STREAM_THREADS = 32 * STREAM_WARPS;
constexpr int STREAM_ROWS = STREAM_WARPS * STREAM_WARP_SAMPLES;   // rows the warps cover (>= the largest batch)
constexpr int STREAM_STAGES = 2;
constexpr int STREAM_KSTEPS = STREAM_WARP_SAMPLES / 8; // tensor-core products of 8 rows per warp and step
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
// 1.0f where a == b, else 0.0f (one instruction)
__device__ __forceinline__ unsigned onehot_bits(float a, float b) {
  float r;
  asm("set.eq.f32.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
  return __float_as_uint(r);
}
// C[16x8] += A[16x8] . B[8x8] on the tensor cores, TF32 operands, fp32 accumulate.  Thread (g = lane / 4, t = lane % 4)
// holds A[g][t], A[g+8][t], A[g][t+4], A[g+8][t+4];  B[t][g], B[t+4][g];  C[g][2t], C[g][2t+1], C[g+8][2t], C[g+8][2t+1].
__device__ __forceinline__ void mma_tf32_16x8x8(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0,
                                                unsigned b1) {
  asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// The same product started from C = 0.
__device__ __forceinline__ void mma_tf32_16x8x8_first(float (&c)[4], unsigned a0, unsigned a1, unsigned a2, unsigned a3, unsigned b0,
                                                      unsigned b1) {
  asm("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3]) : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

constexpr size_t stream_up16(size_t x) { return (x + 15) / 16 * 16; }

// Sizes and the shared-memory map of the streaming kernel.  Everything but the ring has a place that depends on
// (d, k) only, so those byte offsets are constants in the code; the ring comes last.
template <int D, int K>
struct StreamLayout {
  static_assert(D % 2 == 0 && D <= 16 && K <= 16, "streaming path: even d <= 16, k <= 16");
  static constexpr int DP = (D + 2 + 3) / 4 * 4;    // row of -2w, then (||w_a||^2, 0), padded for 128-bit loads
  static constexpr int D2 = D / 2;                  // dimension pairs
  static constexpr int INDEX_BITS = (K <= 2) ? 1 : (K <= 4) ? 2 : (K <= 8) ? 3 : 4;
  static constexpr unsigned INDEX_MASK = (1u << INDEX_BITS) - 1u;
  static constexpr int ROWB = D * 4;                // bytes per sample
  static constexpr int NT = (K + 1 + 7) / 8;        // blocks of 8 one-hot columns: centres 0..K-1 and the spare index K of rows past the batch
  static constexpr int CPW = 32 / D2;               // centres a warp updates: lanes (centre, dimension pair)
  static constexpr int UPD_WARPS = (K + CPW - 1) / CPW;
  static_assert(UPD_WARPS <= STREAM_WARPS, "update: every centre has a warp");
  static constexpr int BEST_RUN = 160;              // bytes between the four runs of the best-centre table (128 used; 160 spreads them over the banks)

  // fixed part of the map (byte offsets)
  static constexpr size_t BARS = 0;
  static constexpr size_t FLAGS = 64;
  static constexpr size_t WMAX = 96;                                    // max_a ||w_a||^2 as found by each updating warp
  static constexpr size_t TAIL = 128;
  static constexpr size_t WNEG2 = TAIL + stream_up16(sizeof(TailScratch));
  static constexpr size_t W = WNEG2 + stream_up16((size_t)K * DP * 4);
  static constexpr size_t SD = W + stream_up16((size_t)K * D * 4);
  static constexpr size_t CNT = SD + stream_up16((size_t)K * D * 4);
  static constexpr size_t SEEN = CNT + stream_up16((size_t)K * 4);
  static constexpr size_t WARP0 = SEEN + stream_up16((size_t)MAX_SLOTS * 4);
  // per warp: the best centre of its rows in the order the one-hot operand reads them; its sums [K][D]; its counts [K]
  static constexpr size_t W_BEST = 0;
  static constexpr size_t W_SUM = W_BEST + 4 * BEST_RUN;
  static constexpr size_t W_CNT = W_SUM + stream_up16((size_t)K * D * 4);
  static constexpr size_t WARP_STRIDE = stream_up16(W_CNT + (size_t)K * 4);
  static constexpr size_t ONES = (WARP0 + STREAM_WARPS * WARP_STRIDE + 15) / 16 * 16;   // (1, 0) pairs: the rows of ones of the counts
  static constexpr size_t ONES_BYTES = (size_t)STREAM_WARP_SAMPLES * ROWB + 16;
  static constexpr size_t RING = (ONES + ONES_BYTES + 127) / 128 * 128;
  // a ring slot: up to 15 bytes in front of the batch (its source is rounded out to 16-byte bounds), room for the
  // rows of a full block (the tensor-core sums read all of them; rows past the batch hold old or zero data and
  // count for no centre) and for the dimension pairs past d that the last rows' fragments touch
  static constexpr size_t SLOT = ((size_t)16 + (size_t)STREAM_ROWS * ROWB + 64 + 127) / 128 * 128;
  static constexpr size_t TOTAL = RING + STREAM_STAGES * SLOT;
};
template <int D, int K>
inline size_t stream_smem_bytes(int /*b*/) { return StreamLayout<D, K>::TOTAL; }

template <int D, int K, bool kDet>
__global__ void __launch_bounds__(STREAM_THREADS, 4)
asgd_stream_kernel(const Params p, const long long steps) {
  using L = StreamLayout<D, K>;
  constexpr int DP = L::DP, D2 = L::D2, KD = K * D, ROWB = L::ROWB, NT = L::NT;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int b = p.b;
  unsigned char* ring = smem_raw + L::RING;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + L::BARS);   // [STAGES]
  int* flags = reinterpret_cast<int*>(smem_raw + L::FLAGS);                               // [0] a buffer has news
  float* wmaxs = reinterpret_cast<float*>(smem_raw + L::WMAX);                            // [UPD_WARPS]
  TailScratch* ts = reinterpret_cast<TailScratch*>(smem_raw + L::TAIL);
  float* wneg2 = reinterpret_cast<float*>(smem_raw + L::WNEG2);
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
  auto warp_ptr = [&](int q, size_t off) { return smem_raw + L::WARP0 + (size_t)q * L::WARP_STRIDE + off; };
  const bool warp_on = wid * STREAM_WARP_SAMPLES < b;                   // warps whose rows all lie past the batch sit a step out

  // state on chip: w, -2w (padded rows), (||w_a||^2, 0); ring and per-warp sums start at zero (rows past the batch
  // and idle warps must read finite numbers)
  for (int e = tid; e < K * DP; e += STREAM_THREADS) wneg2[e] = 0.f;
  for (size_t e = tid; e < STREAM_STAGES * L::SLOT / 16; e += STREAM_THREADS)
    reinterpret_cast<float4*>(ring)[e] = make_float4(0.f, 0.f, 0.f, 0.f);
  for (size_t e = tid; e < STREAM_WARPS * L::WARP_STRIDE / 4; e += STREAM_THREADS)
    reinterpret_cast<float*>(smem_raw + L::WARP0)[e] = 0.f;
  for (size_t e = tid; e < L::ONES_BYTES / 8; e += STREAM_THREADS)
    reinterpret_cast<float2*>(smem_raw + L::ONES)[e] = make_float2(1.f, 0.f);
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
    wneg2[tid * DP + D] = s;
  }
  __syncthreads();
  if (tid < L::UPD_WARPS) {
    float m = 0.f;
    for (int a = 0; a < K; ++a) m = fmaxf(m, wneg2[a * DP + D]);
    wmaxs[tid] = m;
  }
  fence_proxy_async_smem();                                              // the zeroed ring is written by bulk copies next

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
      if (s != p.withhold_step) bulk_g2s(ring + (size_t)slot * L::SLOT, src, bytes, bars + slot);
    } else {
      mbar_expect_tx(bars + slot, 0);       // phase completes at once; consumers load the tile themselves
    }
  };

  // batch indices are read one step ahead so that no step waits on that load
  int pos1 = next_pos(pos);
  int batch_cur = myperm[pos];
  int batch_nxt = myperm[pos1];
  __syncthreads();
  if (tid == 0 && steps > 0) {
    issue(batch_cur, 0, 0);
    if (steps > 1) issue(batch_nxt, 1, 1);
  }

  const float tau_scale = (float)(4 * D + 72) * 5.9604645e-8f;
  const float xmax2 = p.xmax2;                                              // max ||x||^2 over the samples

  // tensor-core fragments: thread (g, t4) reads the dimension pair (2g, 2g+1) of rows 4*t4 + 16*block + r of the
  // warp's rows; for g >= d/2 it reads past the row (finite numbers of the next rows) into result rows nobody uses
  const int g = lane >> 2, t4 = lane & 3;
  const unsigned frag_off = (unsigned)((wid * STREAM_WARP_SAMPLES + 4 * t4) * ROWB + 8 * g);
  // the best centre of row 32*q + lane goes to run (lane % 16) / 4, entry 8*q + 4*(lane / 16) + lane % 4, so that
  // thread (g, t4) finds the rows of its products, two rows per product, in order in run t4
  float* best_w = reinterpret_cast<float*>(warp_ptr(wid, L::W_BEST) + ((lane & 15) >> 2) * L::BEST_RUN) + 4 * (lane >> 4) + (lane & 3);
  const float4* best_r = reinterpret_cast<const float4*>(warp_ptr(wid, L::W_BEST) + t4 * L::BEST_RUN);
  const float2 neg1 = make_float2(-1.f, -1.f);
  float cg[NT];                                                            // this thread's one-hot columns (centres g, 8 + g)
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) cg[nt] = (float)(8 * nt + g);

  // total of centre a, dimension pair jp over the warps, in a fixed order
  auto centre_sum = [&](int a, int jp) {
    float2 part[STREAM_WARPS];
#pragma unroll
    for (int q = 0; q < STREAM_WARPS; ++q) part[q] = reinterpret_cast<const float2*>(warp_ptr(q, L::W_SUM))[a * D2 + jp];
    float2 tot = part[0];
#pragma unroll
    for (int q = 1; q < STREAM_WARPS; ++q) tot = __fadd2_rn(tot, part[q]);
    return tot;
  };
  auto centre_rows = [&](int a) {
    float n = 0.f;
#pragma unroll
    for (int q = 0; q < STREAM_WARPS; ++q) n += reinterpret_cast<const float*>(warp_ptr(q, L::W_CNT))[a];
    return n;                                                              // whole numbers up to 512: exact
  };

  int abort = 0;
  // A step's samples: the thread's rows of the batch in registers, the tile's place for the sums.
  float2 xv[STREAM_SPT][D2];
  const unsigned char* xtile = ring;
  // Gets batch `batch` (the one of step `s`) ready: waits for the copy and loads the thread's rows.  Runs between
  // the two barriers of the step before, beside the update.
  auto stage_in = [&](long long s, int batch) {
    unsigned head, bytes;
    const unsigned char* src = tile_src(batch, head, bytes);
    unsigned char* tile = ring + (size_t)(s & 1) * L::SLOT;
    if (!mbar_wait_bounded(bars + (s & 1), (unsigned)((s >> 1) & 1), p.wait_limit)) abort = 1;
    if (src + bytes > Xend) {
      // last rows of X: a rounded bulk copy would run past the array, use plain loads
      const float* gx = reinterpret_cast<const float*>(src + head);
      float* sdst = reinterpret_cast<float*>(tile + head);
      for (int e = tid; e < b * D; e += STREAM_THREADS) sdst[e] = __ldg(gx + e);
      __syncthreads();
    }
    xtile = tile + head;
    if (warp_on) {
      const float2* xrow = reinterpret_cast<const float2*>(xtile + (size_t)(wid * STREAM_WARP_SAMPLES + lane) * ROWB);
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q)
#pragma unroll
        for (int jp = 0; jp < D2; ++jp) xv[q][jp] = xrow[q * 32 * D2 + jp];
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
    float wmax2 = wmaxs[0];
#pragma unroll
    for (int q = 1; q < L::UPD_WARPS; ++q) wmax2 = fmaxf(wmax2, wmaxs[q]);

    if (warp_on) {
      // ---- Eq. 8: scores of this thread's samples against every centre ----
      float s1[STREAM_SPT], s2[STREAM_SPT];
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) { s1[q] = __int_as_float(0x7f800000); s2[q] = __int_as_float(0x7f800000); }
      // packed score of centre a for each of the thread's samples
      auto scores_of = [&](int a, float (&sp)[STREAM_SPT]) {
        float2 wr[DP / 2];
#pragma unroll
        for (int j4 = 0; j4 < DP / 4; ++j4) {
          const float4 v = *reinterpret_cast<const float4*>(wneg2 + a * DP + 4 * j4);
          wr[2 * j4] = make_float2(v.x, v.y);
          wr[2 * j4 + 1] = make_float2(v.z, v.w);
        }
        const float2 cn = wr[D2];                         // (||w_a||^2, 0)
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
#pragma unroll
      for (int a = 0; a + 1 < K; a += 2) {
        asm volatile("" ::: "memory");                     // keep the loads of this pair of centre rows behind the pair before
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
      bool close = false;
      const float thr0 = tau_scale * (wmax2 + xmax2);                        // cheap test with the global bound on ||x||^2 first
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) {
        best[q] = (int)(__float_as_uint(s1[q]) & L::INDEX_MASK);
        close |= (s2[q] - s1[q]) <= thr0;
      }
      if (K > 1 && close) {
#pragma unroll
        for (int q = 0; q < STREAM_SPT; ++q) {
          if ((s2[q] - s1[q]) <= thr0) {
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
        }
      }
      if ((wid + 1) * STREAM_WARP_SAMPLES > b) {            // the warp that holds the end of the batch: rows past it count for no centre
#pragma unroll
        for (int q = 0; q < STREAM_SPT; ++q)
          if (wid * STREAM_WARP_SAMPLES + q * 32 + lane >= b) best[q] = K;
      }
      if (p.assign_rec) {
#pragma unroll
        for (int q = 0; q < STREAM_SPT; ++q) {
          const int r = wid * STREAM_WARP_SAMPLES + q * 32 + lane;
          if (r < b) p.assign_rec[(size_t)i * b + r] = best[q];
        }
      }
      // ---- Eq. 9 on the tensor cores: S^T[dim][centre] += X^T[dim][row] . onehot[row][centre] over the warp's rows ----
      __syncwarp();                                        // the table's readers of the step before are done
#pragma unroll
      for (int q = 0; q < STREAM_SPT; ++q) best_w[8 * q] = (float)best[q];
      __syncwarp();
      float ch[NT][4], cl[NT][4];                          // sums of the hi terms (row d/2: counts), of the lo terms
      float cc[NT][4];                                     // counts when no result row is spare (d = 16)
      constexpr bool kSpareRow = D2 < 8;
      // threads past the dimension pairs read (1, 0) instead of samples: result row d/2 counts the rows of a centre
      const unsigned char* fa = (g < D2) ? xtile + frag_off : smem_raw + L::ONES;
      const unsigned ones_a = (g == 0) ? 0x3f800000u : 0u; // d = 16: first operand of the counts, row 0 all ones
#pragma unroll
      for (int j2 = 0; j2 < STREAM_KSTEPS / 2; ++j2) {
        const float4 bq = best_r[j2];                      // best centres of rows (t4, t4 + 4) of two products
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          // product 2*j2 + h takes rows 16*j2 + 2h + {0, 4, 8, 12} (columns t4 = 0..3) and the same rows + 1 (columns 4..7)
          const float2 xa = *reinterpret_cast<const float2*>(fa + (size_t)(16 * j2 + 2 * h) * ROWB);
          const float2 xb = *reinterpret_cast<const float2*>(fa + (size_t)(16 * j2 + 2 * h + 1) * ROWB);
          const unsigned h0 = __float_as_uint(xa.x) & 0xffffe000u, h1 = __float_as_uint(xa.y) & 0xffffe000u;
          const unsigned h2 = __float_as_uint(xb.x) & 0xffffe000u, h3 = __float_as_uint(xb.y) & 0xffffe000u;
          const float2 la = __ffma2_rn(make_float2(__uint_as_float(h0), __uint_as_float(h1)), neg1, xa);
          const float2 lb = __ffma2_rn(make_float2(__uint_as_float(h2), __uint_as_float(h3)), neg1, xb);
          const float ba = h ? bq.z : bq.x, bb = h ? bq.w : bq.y;
#pragma unroll
          for (int nt = 0; nt < NT; ++nt) {
            const unsigned b0 = onehot_bits(ba, cg[nt]), b1 = onehot_bits(bb, cg[nt]);
            if (j2 == 0 && h == 0) {
              mma_tf32_16x8x8_first(ch[nt], h0, h1, h2, h3, b0, b1);
              mma_tf32_16x8x8_first(cl[nt], __float_as_uint(la.x), __float_as_uint(la.y), __float_as_uint(lb.x), __float_as_uint(lb.y), b0, b1);
              if (!kSpareRow) mma_tf32_16x8x8_first(cc[nt], ones_a, 0u, ones_a, 0u, b0, b1);
            } else {
              mma_tf32_16x8x8(ch[nt], h0, h1, h2, h3, b0, b1);
              mma_tf32_16x8x8(cl[nt], __float_as_uint(la.x), __float_as_uint(la.y), __float_as_uint(lb.x), __float_as_uint(lb.y), b0, b1);
              if (!kSpareRow) mma_tf32_16x8x8(cc[nt], ones_a, 0u, ones_a, 0u, b0, b1);
            }
          }
        }
      }
      // the warp's sums and counts: thread (g, t4) holds centres 8*nt + 2*t4 (+1), dimensions 2g, 2g+1; the counts sit in
      // result row d/2 (threads g = d/2), for d = 16 in row 0 of their own product
      {
        float2* wsum = reinterpret_cast<float2*>(warp_ptr(wid, L::W_SUM));
        float* wcnt = reinterpret_cast<float*>(warp_ptr(wid, L::W_CNT));
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          const int c0 = 8 * nt + 2 * t4;
          if (g < D2) {
            if (c0 < K) wsum[c0 * D2 + g] = make_float2(ch[nt][0] + cl[nt][0], ch[nt][2] + cl[nt][2]);
            if (c0 + 1 < K) wsum[(c0 + 1) * D2 + g] = make_float2(ch[nt][1] + cl[nt][1], ch[nt][3] + cl[nt][3]);
          }
          if (kSpareRow ? (g == D2) : (g == 0)) {
            if (c0 < K) wcnt[c0] = kSpareRow ? ch[nt][0] : cc[nt][0];
            if (c0 + 1 < K) wcnt[c0 + 1] = kSpareRow ? ch[nt][1] : cc[nt][1];
          }
        }
      }
    }
    if (tid < p.S && my_seq != seen_s[tid]) flags[0] = 1;

    // ---- barrier B: the warps' sums and counts are complete, the ring slot is free again ----
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
      if (tid < K) cnt[tid] = (int)centre_rows(tid);
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
        wneg2[tid * DP + D] = s;
      }
      __syncthreads();
      if (tid < L::UPD_WARPS) {
        float m = 0.f;
        for (int a = 0; a < K; ++a) m = fmaxf(m, wneg2[a * DP + D]);
        wmaxs[tid] = m;
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
          const float n = centre_rows(a);
          const float2 ssum = centre_sum(a, jp);
          const float2 ww = *reinterpret_cast<const float2*>(w + a * D + 2 * jp);
          float2 nw;
          nw.x = ww.x - eps * ((n * ww.x - ssum.x) * inv_b);
          nw.y = ww.y - eps * ((n * ww.y - ssum.y) * inv_b);
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
        if (on && jp == 0) wneg2[a * DP + D] = sq;
        // max ||w_a||^2 over this warp's centres: non-negative floats order like their bit patterns
        const unsigned mbits = __reduce_max_sync(0xffffffffu, (on && jp == 0) ? __float_as_uint(sq) : 0u);
        if (lane == 0) wmaxs[wid] = __uint_as_float(mbits);
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
