// Register-tiled fp32 path for mid-size states (k <= KP, d = D, -2w resident in shared memory):
// the shapes that are bound by the fp32 pipe, not by HBM.
//
// A thread block serves one or more workers in turn (worker = blockIdx.x + v * gridDim.x): a step
// loads the worker's state from HBM/L2, streams the mini-batch through a two-slot ring of sample
// tiles (four bulk copies per tile, one per quarter of its rows, each quarter shifted by one bank
// group; the -2w rows are padded by 4 floats: the rows a warp reads at once fall in different banks), and writes the state back through the shared step tail.
//
// Assignment (Eq. 8): the tile's scores  ||w_a||^2 - 2 x.w_a  are a small GEMM.  A warp covers
// 16 samples x 32 centres, a lane 4 x 4 of them (rows m of quarter sg, centres cg + 8*i):
// per four dimensions it reads four 128-bit pieces of x rows and four of -2w rows and issues 64
// FMAs.  The centre index rides in the low mantissa bits; minimum and runner-up are reduced over
// the lanes and warps that share a sample; a sample whose two best scores are closer than the
// rounding bound of this form is decided again by a warp with direct differences in fp64.
//
// Per-centre sums (Eq. 9): every warp owns the centres a = warp (mod warps); it finds the tile's
// rows of a centre with ballots and adds them, lane = dimension, into the centre's row of S in
// shared memory.  The order of every sum is fixed by row position.
#pragma once

#include <type_traits>

#include "asgd_step_tail.cuh"
#include "asgd_stream.cuh"   // bulk-copy and mbarrier helpers

namespace asgd {

constexpr int TILED_MAX_V = 32;     // workers one block can serve

template <int D, int KP, int WS, int WK>
struct TiledShape {
  static_assert(D % 32 == 0 && KP == 32 * WK && WK <= 4, "tiled path: d a multiple of 32, KP = 32 * WK, WK <= 4");
  static constexpr int THREADS = 32 * WS * WK;
  static constexpr int WARPS = WS * WK;
  static constexpr int TS0 = 16 * WS;             // samples the warps score at a time (a sub-tile)
  static constexpr int RB = (D == 32) ? 128 / TS0 : 1;   // sub-tiles per tile: short rows (d = 32) come 128 at a time, so that
                                                  // the merge, second-look and sum phases and their barriers run once per 128 rows
  static constexpr int TS = TS0 * RB;             // samples per tile
  static_assert(TS <= THREADS && TS <= 128, "a thread per tile row in the merge phase; the sums take up to 128 rows");
  static constexpr int XS = D;                    // row stride inside a quarter of a sample tile (floats)
  static constexpr int QR = 4 * WS;               // rows per quarter; a lane's sample group sg reads quarter sg
  static constexpr int QS = QR * D + 4;           // quarter stride: each quarter starts 4 floats (one bank group) later,
                                                  // so the four rows a warp reads at once fall in different banks
  static constexpr int WST = D + 4;               // padded row stride of -2w: the 8 rows a quarter-warp reads fall in different banks
  static constexpr int INDEX_BITS = 5;            // index inside the warp's block of 32 centres
  static constexpr unsigned INDEX_MASK = 31u;
  static constexpr int DR = D / 32;               // dimensions per lane in the sums
};

template <int D, int KP, int WS, int WK>
struct TiledSmem {
  using T = TiledShape<D, KP, WS, WK>;
  size_t wR, cn, S, cnt, xt, best, red, flagged, tbase, bars, misc, tail, total;
  __host__ __device__ explicit TiledSmem(int k) {
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off += (bytes + 15) / 16 * 16; return o; };
    wR = take((size_t)KP * T::WST * 4);
    cn = take((size_t)KP * 4);
    S = take((size_t)k * D * 4);
    cnt = take((size_t)KP * 4);
    xt = take((size_t)2 * T::RB * 4 * T::QS * 4);
    best = take((size_t)T::TS * 4);
    red = take((size_t)WK * T::TS * 8);
    flagged = take((size_t)(T::TS + 4) * 4);
    tbase = take((size_t)TILED_MAX_V * 8);
    bars = take(64);
    misc = take(64);
    tail = take(sizeof(TailScratch));
    total = (off + 127) / 128 * 128;
  }
};
template <int D, int KP, int WS, int WK>
inline size_t tiled_smem_bytes(int k) { return TiledSmem<D, KP, WS, WK>(k).total; }

template <int D, int KP, int WS, int WK, int MINB, bool kDet>
__global__ void __launch_bounds__(32 * WS * WK, MINB)
asgd_tiled_kernel(const Params p, const long long steps) {
  using T = TiledShape<D, KP, WS, WK>;
  constexpr int TS = T::TS, TS0 = T::TS0, RB = T::RB, XS = T::XS, QR = T::QR, QS = T::QS, WST = T::WST, THREADS = T::THREADS, WARPS = T::WARPS, DR = T::DR;
  extern __shared__ __align__(128) unsigned char smem_raw[];
  const int k = p.k, b = p.b;
  const TiledSmem<D, KP, WS, WK> map(k);
  float* wR = reinterpret_cast<float*>(smem_raw + map.wR);          // [KP][WST]  -2 w
  float* cn = reinterpret_cast<float*>(smem_raw + map.cn);          // [KP]      ||w_a||^2 (+inf for padding)
  float* S = reinterpret_cast<float*>(smem_raw + map.S);            // [k][D]
  int* cnt = reinterpret_cast<int*>(smem_raw + map.cnt);            // [KP]
  float* xt = reinterpret_cast<float*>(smem_raw + map.xt);          // [2][RB sub-tiles][4 quarters][QR][XS] (+4 floats per quarter)
  int* best = reinterpret_cast<int*>(smem_raw + map.best);          // [TS]
  float2* red = reinterpret_cast<float2*>(smem_raw + map.red);      // [WK][TS] (minimum, runner-up)
  int* flagged = reinterpret_cast<int*>(smem_raw + map.flagged);    // [0] count, [1..] tile rows to decide again
  unsigned long long* tbase = reinterpret_cast<unsigned long long*>(smem_raw + map.tbase);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem_raw + map.bars);
  float* misc = reinterpret_cast<float*>(smem_raw + map.misc);      // [0] max_a ||w_a||^2
  TailScratch* ts = reinterpret_cast<TailScratch*>(smem_raw + map.tail);

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int wk = wid % WK, wsi = wid / WK;        // the warp's centre block and sample block
  const int cg = lane & 7, sg = lane >> 3;        // the lane's centres cg + 8*i and rows sg + 4*m of the warp tile
  const int tiles = (b + TS - 1) / TS;
  const float tau_scale = (float)(4 * D + 8 + 4 * (1 << T::INDEX_BITS)) * 5.9604645e-8f;
  const float INF = __int_as_float(0x7f800000);

  const int G = (int)gridDim.x;
  const int nv = (p.W - (int)blockIdx.x + G - 1) / G;              // workers of this block
  if (tid < nv) tbase[tid] = p.stats[(size_t)((int)blockIdx.x + tid * G) * ST_STRIDE + ST_STEPS];
  if (tid == 0) {
    mbar_init(bars + 0, 1);
    mbar_init(bars + 1, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  // The launch consumes tiles in the order (step, worker slot, tile of the batch); tile g uses ring slot g & 1.
  const long long total_tiles = steps * nv * tiles;
  // (tile, worker slot, step) of the next tile to fetch, advanced by the issuing warp only
  int nx_tl = 0, nx_v = 0;
  long long nx_st = 0, nx_g = 0;
  auto issue_next = [&]() {                       // called by all lanes of the issuing warp
    const int tl = nx_tl, v = nx_v;
    const int i = (int)blockIdx.x + v * G;
    const unsigned long long t = tbase[v] + (unsigned long long)nx_st;
    const long long batch = p.perm[(size_t)i * p.B + (size_t)(t % (unsigned long long)p.B)];
    const int rows = min(TS, b - tl * TS);
    const int slot = (int)(nx_g & 1);
    float* dst = xt + (size_t)slot * RB * 4 * QS;
    const float* src = p.X + ((size_t)i * p.H + (size_t)batch * b + (size_t)tl * TS) * D;
    if (lane == 0) mbar_expect_tx(bars + slot, (unsigned)rows * D * 4);
    __syncwarp();
    const bool withheld = (tl == 0 && v == 0 && nx_st == p.withhold_step);      // failure drill: announced, never copied
    if (lane < 4 * RB && !withheld) {                 // one copy per quarter of every sub-tile
      const int first = (lane / 4) * TS0 + (lane % 4) * QR;          // the quarter's first row in the tile
      const int qrows = min(QR, rows - first);
      if (qrows > 0) bulk_g2s(dst + (size_t)lane * QS, src + (size_t)first * D, (unsigned)qrows * D * 4, bars + slot);
    }
    ++nx_g;
    if (++nx_tl == tiles) { nx_tl = 0; if (++nx_v == nv) { nx_v = 0; ++nx_st; } }
  };
  constexpr int ISSUER = WARPS - 1;               // the last warp has no row work in the merge phase
  if (wid == ISSUER && total_tiles > 0) issue_next();

  int abort = 0;
  long long g = 0;
  bool have_state = false;                        // shared memory holds the -2w rows and norms of the worker about to step
  for (long long st = 0; st < steps && !abort; ++st) {
    for (int v = 0; v < nv && !abort; ++v) {
      const int i = (int)blockIdx.x + v * G;
      const unsigned long long t = tbase[v] + (unsigned long long)st;
      float* wglob = p.state + (size_t)i * p.kd_pad;

      // ---- the worker's state: -2w rows, ||w_a||^2 (kept from the last step when this block serves one worker
      //      and that step took the fused update), empty sums ----
      if (!have_state) {
        for (int e = tid; e < KP * (D / 4); e += THREADS) {
          const int a = e / (D / 4), j4 = e % (D / 4);
          float4 v4 = make_float4(0.f, 0.f, 0.f, 0.f);
          if (a < k) {
            v4 = *reinterpret_cast<const float4*>(wglob + (size_t)a * D + 4 * j4);
            v4.x *= -2.f; v4.y *= -2.f; v4.z *= -2.f; v4.w *= -2.f;
          }
          *reinterpret_cast<float4*>(wR + (size_t)a * WST + 4 * j4) = v4;
        }
      }
      for (int e = tid; e < k * D; e += THREADS) S[e] = 0.f;
      for (int e = tid; e < KP; e += THREADS) cnt[e] = 0;
      __syncthreads();
      if (!have_state) {
        for (int a = wid; a < KP; a += WARPS) {
          float s = 0.f;
#pragma unroll
          for (int q = 0; q < DR; ++q) { const float u = wR[(size_t)a * WST + lane + 32 * q]; s = fmaf(u, u, s); }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
          if (lane == 0) cn[a] = (a < k) ? 0.25f * s : INF;
        }
        __syncthreads();
      }
      if (wid == 0) {
        float m = 0.f;
        for (int a = lane; a < k; a += 32) m = fmaxf(m, cn[a]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        if (lane == 0) misc[0] = m;
      }
      // a look at the receive buffers' sequence numbers (used after the last tile)
      int news = 0;
      if (tid < p.S) news = ld_relaxed_gpu(p.seq + (size_t)i * p.S + tid) != p.seen[(size_t)i * p.S + tid];

      for (int tl = 0; tl < tiles; ++tl, ++g) {
        const int slot = (int)(g & 1);
        const unsigned parity = (unsigned)((g >> 1) & 1);
        const int rows = min(TS, b - tl * TS);
        const float* xb = xt + (size_t)slot * RB * 4 * QS;
        auto xrowp = [&](int r) { return xb + (size_t)(r / QR) * QS + (size_t)(r % QR) * XS; };   // tile row r (quarters of all sub-tiles are QS apart)
        if (tid == 0) flagged[0] = 0;
        if (!mbar_wait_bounded(bars + slot, parity, p.wait_limit)) abort = 1;

        for (int rb = 0; rb < RB && rb * TS0 < rows; ++rb) {   // the tile's sub-tiles in turn (the same trip count for every thread)
          // ---- scores of the warp's 16 x 32 block: acc[m][i] = sum_j x[row m][j] * (-2 w[centre i][j]) ----
          float acc[4][4];
  #pragma unroll
          for (int m = 0; m < 4; ++m)
  #pragma unroll
            for (int c = 0; c < 4; ++c) acc[m][c] = 0.f;
          const float* xrow = xb + (size_t)(rb * 4 + sg) * QS + (size_t)(wsi * 4) * XS;    // rows rb*TS0 + sg*QR + wsi*4 + m
          const float* wrow = wR + (size_t)(wk * 32 + cg) * WST;
          // the warp's 32 centres come in four groups of eight (centres 8c + cg); a group that lies wholly past k is
          // padding and is left out (k = 100 in 128 columns: three of the last warp's four groups)
          auto score_groups = [&](auto ng_tag) {
            constexpr int NG = decltype(ng_tag)::value;
  #pragma unroll 2
            for (int j = 0; j < D; j += 4) {
              float4 xv[4], wv[NG];
  #pragma unroll
              for (int m = 0; m < 4; ++m) xv[m] = *reinterpret_cast<const float4*>(xrow + (size_t)m * XS + j);
  #pragma unroll
              for (int c = 0; c < NG; ++c) wv[c] = *reinterpret_cast<const float4*>(wrow + (size_t)(8 * c) * WST + j);
  #pragma unroll
              for (int m = 0; m < 4; ++m)
  #pragma unroll
                for (int c = 0; c < NG; ++c) {
                  acc[m][c] = fmaf(xv[m].x, wv[c].x, acc[m][c]);
                  acc[m][c] = fmaf(xv[m].y, wv[c].y, acc[m][c]);
                  acc[m][c] = fmaf(xv[m].z, wv[c].z, acc[m][c]);
                  acc[m][c] = fmaf(xv[m].w, wv[c].w, acc[m][c]);
                }
            }
          };
          const int ngroups = min(4, max(0, (k - wk * 32 + 7) / 8));          // the same for every lane of the warp
          if (ngroups == 4) score_groups(std::integral_constant<int, 4>());
          else if (ngroups == 3) score_groups(std::integral_constant<int, 3>());
          else if (ngroups == 2) score_groups(std::integral_constant<int, 2>());
          else if (ngroups == 1) score_groups(std::integral_constant<int, 1>());
          // minimum and runner-up over the lane's 4 centres, then over the 8 lanes that share the rows
          float cnv[4];
  #pragma unroll
          for (int c = 0; c < 4; ++c) cnv[c] = cn[wk * 32 + 8 * c + cg];
  #pragma unroll
          for (int m = 0; m < 4; ++m) {
            float s1 = INF, s2 = INF;
  #pragma unroll
            for (int c = 0; c < 4; ++c) {
              const float sc = acc[m][c] + cnv[c];
              const float sp = __uint_as_float((__float_as_uint(sc) & ~T::INDEX_MASK) | (unsigned)(8 * c + cg));
              s2 = fmaxf(s1, fminf(s2, sp));
              s1 = fminf(s1, sp);
            }
  #pragma unroll
            for (int o = 1; o < 8; o <<= 1) {
              const float o1 = __shfl_xor_sync(0xffffffffu, s1, o);
              const float o2 = __shfl_xor_sync(0xffffffffu, s2, o);
              s2 = fminf(fmaxf(s1, o1), fminf(s2, o2));
              s1 = fminf(s1, o1);
            }
            if (cg == 0) red[(size_t)wk * TS + rb * TS0 + sg * QR + wsi * 4 + m] = make_float2(s1, s2);
          }
        }
        // the ring slot of the previous tile is free since that tile's last barrier: fetch the next tile now
        if (wid == ISSUER && g + 1 < total_tiles) {
          fence_proxy_async_smem();
          issue_next();
        }
        __syncthreads();                                         // (1) red complete

        // ---- one thread per tile row: merge over the centre blocks, decide or flag ----
        if (tid < TS) {
          int bst = -1;
          if (tid < rows) {
            float s1 = INF, s2 = INF;
            int qwin = 0;
#pragma unroll
            for (int q = 0; q < WK; ++q) {
              const float2 r = red[(size_t)q * TS + tid];
              s2 = fminf(fmaxf(s1, r.x), fminf(s2, r.y));
              if (r.x < s1) { s1 = r.x; qwin = q; }             // equal packed scores of two blocks: second look below
            }
            bst = qwin * 32 + (int)(__float_as_uint(s1) & T::INDEX_MASK);
            if (k > 1 && (s2 - s1) <= tau_scale * (misc[0] + p.xmax2)) {       // cheap test with the bound on ||x||^2 over X first
              const float* xr = xrowp(tid);
              float xx = 0.f;
              for (int j = 0; j < D; j += 4) {
                const float4 u = *reinterpret_cast<const float4*>(xr + j);
                xx = fmaf(u.x, u.x, xx); xx = fmaf(u.y, u.y, xx); xx = fmaf(u.z, u.z, xx); xx = fmaf(u.w, u.w, xx);
              }
              if ((s2 - s1) <= tau_scale * (misc[0] + xx)) flagged[1 + atomicAdd(flagged, 1)] = tid;
            }
          }
          best[tid] = bst;
        }
        __syncthreads();                                         // (2) best, flagged complete

        // ---- rows too close for the expanded form: a warp per row, lanes over centres, direct
        //      differences in fp32; if that is still within rounding of a tie, in fp64 ----
        const int nflag = flagged[0];
        if (nflag > 0) {
          for (int f = wid; f < nflag; f += WARPS) {
            const int r = flagged[1 + f];
            const float* xr = xrowp(r);
            float fd1 = INF, fd2 = INF;
            int fi = 0x7fffffff;
            for (int a = lane; a < k; a += 32) {
              const float* wa = wR + (size_t)a * WST;
              float s = 0.f;
#pragma unroll 4
              for (int j = 0; j < D; ++j) {
                const float df = xr[j] + 0.5f * wa[j];                     // -0.5 * (-2w) = w, exact
                s = fmaf(df, df, s);
              }
              if (s < fd1) { fd2 = fd1; fd1 = s; fi = a; } else if (s < fd2) { fd2 = s; }
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
              const float o1 = __shfl_xor_sync(0xffffffffu, fd1, o);
              const float o2 = __shfl_xor_sync(0xffffffffu, fd2, o);
              const int oi = __shfl_xor_sync(0xffffffffu, fi, o);
              const bool take = (o1 < fd1) || (o1 == fd1 && oi < fi);
              fd2 = fminf(take ? fd1 : o1, fminf(fd2, o2));
              if (take) { fd1 = o1; fi = oi; }
            }
            int bi = fi;
            if (fd2 - fd1 <= (float)(4 * D + 16) * 5.9604645e-8f * fd2) {
              double bd = 1e300;
              bi = 0x7fffffff;
              for (int a = lane; a < k; a += 32) {
                const float* wa = wR + (size_t)a * WST;
                double s = 0.0;
                for (int j = 0; j < D; ++j) {
                  const double df = (double)xr[j] + 0.5 * (double)wa[j];
                  s = fma(df, df, s);
                }
                if (s < bd) { bd = s; bi = a; }                  // ascending a: the lowest index keeps a tie
              }
#pragma unroll
              for (int o = 16; o > 0; o >>= 1) {
                const double od = __shfl_xor_sync(0xffffffffu, bd, o);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
                if (od < bd || (od == bd && oi < bi)) { bd = od; bi = oi; }
              }
            }
            if (lane == 0) best[r] = bi;
          }
          __syncthreads();                                       // (2b) uniform: nflag is the same for all threads
        }
        if (p.assign_rec && tid < rows) p.assign_rec[(size_t)i * b + (size_t)tl * TS + tid] = best[tid];

        // ---- Eq. 9: the warp adds the tile's rows of the centres it owns, lane = dimension ----
        {
          const int b0 = (lane < TS) ? best[lane] : -1;
          const int b1 = (TS > 32 && 32 + lane < TS) ? best[32 + lane] : -1;
          const int b2 = (TS > 64 && 64 + lane < TS) ? best[64 + lane] : -1;
          const int b3 = (TS > 96 && 96 + lane < TS) ? best[96 + lane] : -1;
          for (int a = wid; a < k; a += WARPS) {
            unsigned msk[4];
            msk[0] = __ballot_sync(0xffffffffu, b0 == a);
            msk[1] = (TS > 32) ? __ballot_sync(0xffffffffu, b1 == a) : 0u;
            msk[2] = (TS > 64) ? __ballot_sync(0xffffffffu, b2 == a) : 0u;
            msk[3] = (TS > 96) ? __ballot_sync(0xffffffffu, b3 == a) : 0u;
            const int n = __popc(msk[0]) + __popc(msk[1]) + __popc(msk[2]) + __popc(msk[3]);
            if (n == 0) continue;
            float sum[DR];
#pragma unroll
            for (int q = 0; q < DR; ++q) sum[q] = 0.f;
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              unsigned m = msk[h];
              while (m) {
                const int r = 32 * h + __ffs(m) - 1;
                m &= m - 1;
                const float* xr = xrowp(r);
                float u[DR];
#pragma unroll
                for (int q = 0; q < DR; ++q) u[q] = xr[lane + 32 * q];
                if (m) {                                           // a second row in flight with the first
                  const int r2 = 32 * h + __ffs(m) - 1;
                  m &= m - 1;
                  const float* xr2 = xrowp(r2);
                  float u2[DR];
#pragma unroll
                  for (int q = 0; q < DR; ++q) u2[q] = xr2[lane + 32 * q];
#pragma unroll
                  for (int q = 0; q < DR; ++q) sum[q] = (sum[q] + u[q]) + u2[q];
                } else {
#pragma unroll
                  for (int q = 0; q < DR; ++q) sum[q] += u[q];
                }
              }
            }
#pragma unroll
            for (int q = 0; q < DR; ++q) S[(size_t)a * D + lane + 32 * q] += sum[q];
            if (lane == 0) cnt[a] += n;
          }
        }
        if (__syncthreads_or(abort)) { abort = 1; break; }      // (3) tile consumed
      }
      if (abort) break;

      if (__syncthreads_or(news)) {
        // a message is waiting: the general tail works on the state in shared memory; turn the -2w rows back into w (exact)
        for (int e = tid; e < k * (D / 4); e += THREADS) {
          float4* q4 = reinterpret_cast<float4*>(wR + (size_t)(e / (D / 4)) * WST + 4 * (e % (D / 4)));
          float4 u = *q4;
          u.x *= -0.5f; u.y *= -0.5f; u.z *= -0.5f; u.w *= -0.5f;
          *q4 = u;
        }
        __syncthreads();
        step_tail<kDet>(p, i, t, wR, WST, S, cnt, wglob, ts);
        have_state = false;
      } else {
        // common case: plain local step  w <- w - eps (n_a w - S) / b  on the -2w rows, new state to HBM, new ||w_a||^2
        constexpr int RV = D / 4;                            // 128-bit pieces per centre row (8 or 32: a power of two <= 32)
        const float inv_b = 1.0f / (float)b;
        const int pieces = k * RV;
        for (int e0 = 0; e0 < pieces; e0 += THREADS) {       // the same trip count for every thread (shuffles inside)
          const int e = e0 + tid;
          const bool on = e < pieces;
          const int a = on ? e / RV : 0, j4 = e % RV;
          float sq = 0.f;
          if (on) {
            float4* q4 = reinterpret_cast<float4*>(wR + (size_t)a * WST + 4 * j4);
            const float4 m2 = *q4;
            const float4 sm = *reinterpret_cast<const float4*>(S + (size_t)a * D + 4 * j4);
            const float fn = (float)cnt[a];
            float4 w4 = make_float4(-0.5f * m2.x, -0.5f * m2.y, -0.5f * m2.z, -0.5f * m2.w);
            w4.x -= p.eps * ((fn * w4.x - sm.x) * inv_b); w4.y -= p.eps * ((fn * w4.y - sm.y) * inv_b);
            w4.z -= p.eps * ((fn * w4.z - sm.z) * inv_b); w4.w -= p.eps * ((fn * w4.w - sm.w) * inv_b);
            *reinterpret_cast<float4*>(wglob + (size_t)a * D + 4 * j4) = w4;
            *q4 = make_float4(-2.f * w4.x, -2.f * w4.y, -2.f * w4.z, -2.f * w4.w);
            sq = fmaf(w4.x, w4.x, fmaf(w4.y, w4.y, fmaf(w4.z, w4.z, w4.w * w4.w)));
          }
#pragma unroll
          for (int o = 1; o < RV; o <<= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
          if (on && j4 == 0) cn[a] = sq;
        }
        unsigned long long n_sent = 0;
        if (p.c > 0 && p.f > 0 && p.W > 1 && (t + 1) % (unsigned long long)p.c == 0) {
          __syncthreads();                                   // the new state is complete in HBM for this block's threads
          n_sent = step_send_any<kDet>(p, i, t, wglob, D, ts);
        }
        if (kDet && p.rows_m > 0)
          for (int a = tid; a < p.k; a += THREADS) p.rowin[(size_t)i * p.k + a] = 0;
        if (tid == 0) {
          if (kDet)
            for (int s = 0; s < p.S; ++s) p.accept_rec[(size_t)i * p.S + s] = -1;
          unsigned long long* st_ = p.stats + (size_t)i * ST_STRIDE;
          st_[ST_STEPS] = t + 1;
          if (n_sent) atomicAdd(st_ + ST_SENT, n_sent);
        }
        have_state = (nv == 1);                              // the -2w rows and norms in shared memory are this worker's next state
      }
      __syncthreads();
    }
  }

  if (abort) {
    if (tid == 0) atomicExch(p.status, DEV_TIMEOUT);
    mbar_wait_bounded(bars + 0, 0, p.wait_limit); mbar_wait_bounded(bars + 0, 1, p.wait_limit);
    mbar_wait_bounded(bars + 1, 0, p.wait_limit); mbar_wait_bounded(bars + 1, 1, p.wait_limit);
  }
}

}  // namespace asgd
