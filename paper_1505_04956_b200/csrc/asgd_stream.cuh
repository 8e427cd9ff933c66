// Streaming fp32 path for small states (k, d <= 16): the HBM-bound shape of the method.
//
// One worker = one 128-thread block, 4 blocks per SM.  The worker's mini-batches are pulled into a
// two-slot shared-memory ring with bulk asynchronous copies (one elected thread issues them, an
// mbarrier per slot counts the bytes), so the next batch streams in while the current one is used.
// Assignment: one thread per sample, expanded form  score_a = ||w_a||^2 - 2 x.w_a  (exactly k*d
// FMAs), with the centre index packed into the low mantissa bits so that min/max instructions carry
// the argmin; a sample whose two best scores are closer than the rounding bound of that form is
// decided again in the direct difference form.  Per-centre sums: lanes of a warp that share a centre
// add their rows with a pointer-jumping shuffle reduction, the group's first lane adds the result
// to the warp's private accumulators in shared memory.  The order of every sum is fixed by sample
// position, so a step is reproducible.
#pragma once

#include "asgd_step_tail.cuh"

namespace asgd {

constexpr int STREAM_THREADS = 128;
constexpr int STREAM_WARPS = STREAM_THREADS / 32;
constexpr int STREAM_STAGES = 2;
constexpr unsigned STREAM_WAIT_LIMIT = 1u << 22;   // bounded mbarrier wait (iterations of try_wait)

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
__device__ inline void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

template <int D, int K>
struct StreamLayout {
  static constexpr int DP = (D + 3) / 4 * 4;        // padded row of -2w for 128-bit loads
  static constexpr int SP = D + 1;                  // row stride of the per-warp accumulators
  static constexpr int INDEX_BITS = (K <= 2) ? 1 : (K <= 4) ? 2 : (K <= 8) ? 3 : 4;
  static constexpr unsigned INDEX_MASK = (1u << INDEX_BITS) - 1u;
};

inline size_t stream_slot_bytes(int b, int d) { return ((size_t)b * d * 4 + 32 + 127) / 128 * 128; }

// Shared-memory map of the streaming kernel (byte offsets, every region 16-byte aligned).
template <int D, int K>
struct StreamSmem {
  using L = StreamLayout<D, K>;
  size_t ring, bars, flags, tail, wneg2, cnorm, w, sd, sw, cw, cnt, total;
  __host__ __device__ explicit StreamSmem(int b) {
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 15) / 16 * 16; return o; };
    ring = take(STREAM_STAGES * (((size_t)b * D * 4 + 32 + 127) / 128 * 128));
    bars = take(64);
    flags = take(64);
    tail = take(sizeof(TailScratch));
    wneg2 = take((size_t)K * L::DP * 4);
    cnorm = take((size_t)K * 4);
    w = take((size_t)K * D * 4);
    sd = take((size_t)K * D * 4);
    sw = take((size_t)STREAM_WARPS * K * L::SP * 4);
    cw = take((size_t)STREAM_WARPS * K * 4);
    cnt = take((size_t)K * 4);
    total = (off + 127) / 128 * 128;
  }
};
template <int D, int K>
inline size_t stream_smem_bytes(int b) { return StreamSmem<D, K>(b).total; }

// Squared distances of one sample in the direct difference form; strict "<" keeps the lowest index.
template <int D, int K>
__device__ inline int direct_argmin(const float (&x)[D], const float* wneg2, int DP) {
  int best = 0;
  float bd = __int_as_float(0x7f800000);
#pragma unroll
  for (int a = 0; a < K; ++a) {
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < D; ++j) {
      const float df = x[j] + 0.5f * wneg2[a * DP + j];     // -0.5 * (-2w) = w, exact
      s = fmaf(df, df, s);
    }
    if (s < bd) { bd = s; best = a; }
  }
  return best;
}

template <int D, int K, bool kDet>
__global__ void __launch_bounds__(STREAM_THREADS, 4)
asgd_stream_kernel(const Params p, const long long steps) {
  using L = StreamLayout<D, K>;
  constexpr int DP = L::DP, SP = L::SP, KD = K * D;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int b = p.b;
  const size_t slot_bytes = ((size_t)b * D * 4 + 32 + 127) / 128 * 128;
  const StreamSmem<D, K> map(b);
  unsigned char* ring = smem_raw + map.ring;
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + map.bars);   // [STAGES]
  int* flags = reinterpret_cast<int*>(smem_raw + map.flags);                               // [0] any fresh buffer
  TailScratch* ts = reinterpret_cast<TailScratch*>(smem_raw + map.tail);
  float* wneg2 = reinterpret_cast<float*>(smem_raw + map.wneg2);
  float* cnorm = reinterpret_cast<float*>(smem_raw + map.cnorm);
  float* w = reinterpret_cast<float*>(smem_raw + map.w);
  float* SD = reinterpret_cast<float*>(smem_raw + map.sd);
  float* Sw = reinterpret_cast<float*>(smem_raw + map.sw);
  int* Cw = reinterpret_cast<int*>(smem_raw + map.cw);
  int* cnt = reinterpret_cast<int*>(smem_raw + map.cnt);

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int i = blockIdx.x;
  float* wglob = p.state + (size_t)i * p.kd_pad;
  const float* Xend = p.X + (size_t)p.N * D;

  // state on chip: w, -2w (padded rows), ||w_a||^2
  for (int e = tid; e < K * DP; e += STREAM_THREADS) wneg2[e] = 0.f;
  __syncthreads();
  for (int e = tid; e < KD; e += STREAM_THREADS) {
    const float v = wglob[e];
    w[e] = v;
    wneg2[(e / D) * DP + (e % D)] = -2.f * v;
  }
  for (int e = tid; e < STREAM_WARPS * K * SP; e += STREAM_THREADS) Sw[e] = 0.f;
  for (int e = tid; e < STREAM_WARPS * K; e += STREAM_THREADS) Cw[e] = 0;
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
    cnorm[tid] = s;
  }

  unsigned long long t = p.stats[(size_t)i * ST_STRIDE + ST_STEPS];

  // a batch's copy: source rounded down to 16 bytes, size rounded up; `head` = bytes to skip
  const int* myperm = p.perm + (size_t)i * p.B;
  auto tile_src = [&](long long batch, unsigned& head, unsigned& bytes) -> const unsigned char* {
    const unsigned char* src = reinterpret_cast<const unsigned char*>(p.X + ((size_t)i * p.H + (size_t)batch * b) * D);
    head = (unsigned)((uintptr_t)src & 15);
    bytes = (head + (unsigned)b * D * 4 + 15u) & ~15u;
    return src - head;
  };
  // true when the rounded copy stays inside X (else the tile is fetched with plain loads)
  auto tile_bulk_ok = [&](const unsigned char* src, unsigned bytes) {
    return src + bytes <= reinterpret_cast<const unsigned char*>(Xend);
  };
  auto issue = [&](long long batch, int slot) {
    unsigned head, bytes;
    const unsigned char* src = tile_src(batch, head, bytes);
    if (tile_bulk_ok(src, bytes)) {
      mbar_expect_tx(bars + slot, bytes);
      bulk_g2s(ring + (size_t)slot * slot_bytes, src, bytes, bars + slot);
    } else {
      mbar_expect_tx(bars + slot, 0);       // phase completes at once; consumers load the tile themselves
    }
  };

  // batch indices are read one step ahead so that no step waits on that load
  long long batch_cur = myperm[t % (unsigned long long)p.B];
  long long batch_nxt = myperm[(t + 1) % (unsigned long long)p.B];
  if (tid == 0 && steps > 0) issue(batch_cur, 0);
  __syncthreads();

  int abort = 0;
  for (long long step = 0; step < steps; ++step, ++t) {
    const int slot = (int)(step & 1);
    const unsigned parity = (unsigned)((step >> 1) & 1);

    // thread 0: look at the receive buffers' sequence numbers early, start the next batch's copy
    if (tid == 0) {
      int any = 0;
      for (int s = 0; s < p.S; ++s) any |= (ld_acquire_gpu(p.seq + (size_t)i * p.S + s) != p.seen[(size_t)i * p.S + s]);
      flags[0] = any;
      if (step + 1 < steps) {
        fence_proxy_async_smem();
        issue(batch_nxt, slot ^ 1);
      }
    }
    const long long batch_nn = myperm[(t + 2) % (unsigned long long)p.B];

    unsigned head, bytes;
    const unsigned char* src = tile_src(batch_cur, head, bytes);
    unsigned char* tile = ring + (size_t)slot * slot_bytes;
    if (!mbar_wait_bounded(bars + slot, parity)) abort = 1;
    if (!tile_bulk_ok(src, bytes)) {
      // last rows of X: a rounded bulk copy would run past the array, use plain loads
      const float* g = reinterpret_cast<const float*>(src + head);
      float* sdst = reinterpret_cast<float*>(tile + head);
      for (int e = tid; e < b * D; e += STREAM_THREADS) sdst[e] = __ldg(g + e);
      __syncthreads();
    }
    const float* xs = reinterpret_cast<const float*>(tile + head);

    float cn[K];
    float wmax2 = 0.f;
#pragma unroll
    for (int a = 0; a < K; ++a) { cn[a] = cnorm[a]; wmax2 = fmaxf(wmax2, cn[a]); }
    const float tau_scale = (float)(4 * D + 72) * 5.9604645e-8f;

    for (int base = 0; base < b; base += STREAM_THREADS) {
      const int s = base + tid;
      const bool valid = s < b;
      float x[D];
      if (valid) {
        if (D % 2 == 0) {
#pragma unroll
          for (int j = 0; j < D; j += 2) {
            const float2 v = *reinterpret_cast<const float2*>(xs + (size_t)s * D + j);
            x[j] = v.x; x[j + 1] = v.y;
          }
        } else {
#pragma unroll
          for (int j = 0; j < D; ++j) x[j] = xs[(size_t)s * D + j];
        }
      } else {
#pragma unroll
        for (int j = 0; j < D; ++j) x[j] = 0.f;
      }
      float x2 = 0.f;
#pragma unroll
      for (int j = 0; j < D; ++j) x2 = fmaf(x[j], x[j], x2);

      // Eq. 8 in expanded form; index in the low mantissa bits
      float s1 = __int_as_float(0x7f800000), s2 = __int_as_float(0x7f800000);
#pragma unroll
      for (int a = 0; a < K; ++a) {
        float acc = cn[a];
        const float4* wr = reinterpret_cast<const float4*>(wneg2 + a * DP);
#pragma unroll
        for (int j4 = 0; j4 < DP / 4; ++j4) {
          const float4 wv = wr[j4];
          if (4 * j4 + 0 < D) acc = fmaf(x[4 * j4 + 0 < D ? 4 * j4 + 0 : 0], wv.x, acc);
          if (4 * j4 + 1 < D) acc = fmaf(x[4 * j4 + 1 < D ? 4 * j4 + 1 : 0], wv.y, acc);
          if (4 * j4 + 2 < D) acc = fmaf(x[4 * j4 + 2 < D ? 4 * j4 + 2 : 0], wv.z, acc);
          if (4 * j4 + 3 < D) acc = fmaf(x[4 * j4 + 3 < D ? 4 * j4 + 3 : 0], wv.w, acc);
        }
        const float sp = __uint_as_float((__float_as_uint(acc) & ~L::INDEX_MASK) | (unsigned)a);
        s2 = fmaxf(s1, fminf(s2, sp));
        s1 = fminf(s1, sp);
      }
      int best = (int)(__float_as_uint(s1) & L::INDEX_MASK);
      if (K > 1 && (s2 - s1) <= tau_scale * (wmax2 + x2)) best = direct_argmin<D, K>(x, wneg2, DP);
      if (!valid) best = K;                              // padding lanes form their own group
      if (valid && p.assign_rec) p.assign_rec[(size_t)i * b + s] = best;

      // Eq. 9: sum the rows of the lanes that chose the same centre (pointer jumping over the
      // group's lanes in ascending order), then the group's first lane adds to the warp's row
      const unsigned grp = __match_any_sync(0xffffffffu, best);
      const unsigned above = grp & ~((2u << lane) - 1u);
      int nxt = above ? (__ffs(above) - 1) : lane;
      const bool leader = (grp & ((1u << lane) - 1u)) == 0;
      const int gsize = __popc(grp);
      int rounds = 32 - __clz(__reduce_max_sync(0xffffffffu, (unsigned)gsize) - 1);   // ceil(log2(max size))
      for (int r = 0; r < rounds; ++r) {
        const bool have = nxt != lane;
#pragma unroll
        for (int j = 0; j < D; ++j) {
          const float o = __shfl_sync(0xffffffffu, x[j], nxt);
          if (have) x[j] += o;
        }
        const int nn = __shfl_sync(0xffffffffu, nxt, nxt);
        nxt = (!have || nn == nxt) ? lane : nn;
      }
      if (leader && best < K) {
        float* row = Sw + (wid * K + best) * SP;
#pragma unroll
        for (int j = 0; j < D; ++j) row[j] += x[j];
        Cw[wid * K + best] += gsize;
      }
      __syncwarp();
    }

    // ---- barrier A: every warp's sums are in shared memory, the slot is free again ----
    if (__syncthreads_or(abort)) { abort = 1; break; }

    // per-centre totals and the local gradient (Eq. 9), in place of the generic tail's first loop
    for (int e = tid; e < KD; e += STREAM_THREADS) {
      float ssum = 0.f;
#pragma unroll
      for (int q = 0; q < STREAM_WARPS; ++q) ssum += Sw[(q * K + e / D) * SP + (e % D)];
      SD[e] = ssum;
    }
    if (tid < K) {
      int c = 0;
#pragma unroll
      for (int q = 0; q < STREAM_WARPS; ++q) c += Cw[q * K + tid];
      cnt[tid] = c;
    }
    __syncthreads();
    for (int e = tid; e < STREAM_WARPS * K * SP; e += STREAM_THREADS) Sw[e] = 0.f;
    for (int e = tid; e < STREAM_WARPS * K; e += STREAM_THREADS) Cw[e] = 0;

    const bool put_now = p.c > 0 && p.f > 0 && p.W > 1 && (t + 1) % (unsigned long long)p.c == 0;
    if (flags[0] || put_now) {
      // a message is waiting or a put is due: the general tail handles both
      step_tail<kDet>(p, i, t, w, SD, cnt, wglob, ts);
    } else {
      // common case: plain local step  w <- w - eps * D
      for (int e = tid; e < KD; e += STREAM_THREADS) {
        const float ww = w[e];
        const float Dg = ((float)cnt[e / D] * ww - SD[e]) * (1.0f / (float)b);
        const float nw = ww - p.eps * Dg;
        w[e] = nw;
        wglob[e] = nw;
      }
      if (tid == 0) {
        for (int s = 0; s < p.S; ++s) p.accept_rec[(size_t)i * p.S + s] = -1;
        p.stats[(size_t)i * ST_STRIDE + ST_STEPS] = t + 1;
      }
      __syncthreads();
    }
    for (int e = tid; e < KD; e += STREAM_THREADS) wneg2[(e / D) * DP + (e % D)] = -2.f * w[e];
    if (tid < K) {
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < D; ++j) s = fmaf(w[tid * D + j], w[tid * D + j], s);
      cnorm[tid] = s;
    }
    batch_cur = batch_nxt;
    batch_nxt = batch_nn;
    __syncthreads();
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
