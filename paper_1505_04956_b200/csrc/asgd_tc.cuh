// Tensor-core path (tcgen05, 16-bit operands, FP32 accumulate in tensor memory) for states of up to 1024 centres with
// d a multiple of 64 up to 256 and batches of at least 128 rows: the shapes where the scores of Eq. 8 are a dense
// contraction  -2 X W^T, e.g. of a 4096 x 256 mini-batch against a 1024 x 256 centre matrix.
//
// Two operand formats (template parameter kTerms):
//   1  FP16, one term per operand: x and -2w rounded to FP16 (11 significant bits), one product.  A score is good to
//      2^-10 ||x|| ||w||; the rows whose candidates lie closer than that (a few per cent) are decided exactly afterwards.
//      Needs |x|, |2w| inside FP16's range.
//   3  BF16, two terms per operand: x = x_hi + x_lo and -2w = w_hi + w_lo (x_lo, w_lo hold the rounding residues),
//      three products  x_hi.w_hi + x_lo.w_hi + x_hi.w_lo  into the same accumulator.  What is left out (x_lo.w_lo and
//      the residues of the residues) is below 6 * 2^-18 ||x|| ||w||: about 16 bits, any fp32 range, three times the
//      tensor work and twice the operand bytes.
// Either way Eq. 8 is decided exactly: a row is settled among ALL centres that the format's error bound cannot rule out.
//
// A block serves its workers in turn (one worker when there are as many blocks as workers).  Warp roles while the
// scores are computed:
//   warp 0   one lane issues the TMA loads: a 128-row sample tile in 128-byte-swizzled K-chunks of 64, resident while
//            all centre blocks pass, and the centre blocks (256 centres with one term, 128 with two, or the whole
//            state rounded up to 32 when it is smaller) through a ring of K-chunks (they come from L2);
//   warp 1   allocates tensor memory; one lane issues tcgen05.mma (128 x N x 16 per instruction) into one of two
//            accumulator stages and commits to mbarriers; with two or more centre blocks one lane of warp 2 does the
//            same for every other block (a commit holds its thread for a while; the other thread keeps the pipe fed);
//   warps 4 and up  read the accumulators (tcgen05.ld, one TMEM lane = one sample per thread; one, two or three warps
//            per quarter of the tile, taking the 32-column groups in turn), add ||w_a||^2 and ||x||^2 and keep, per
//            sample, the three smallest squared distances with the centre index packed into the low mantissa bits,
//            and a floor under the fourth, carried in registers over the centre blocks.
// Then all warps: a sample whose runner-up is inside the error bound is decided between its two candidates with
// fp32 inputs (fp64 sums when still close), likewise among three when the third is inside and the floor is not; one
// whose fourth candidate may be inside as well is measured against all centres the same way.  Rows are grouped by
// centre and each centre's sum of fp32 master samples, update, new 16-bit copy and ||w_a||^2 come from one pass.
// Every wait is bounded.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>

#include <type_traits>

#include "asgd_step_tail.cuh"
#include "asgd_stream.cuh"   // mbarrier helpers

namespace asgd {

// threads of a block: two blocks per SM; one block per SM with rows of up to 256 numbers (168 registers a thread); one
// block per SM with rows of at most 128 numbers (128 registers a thread)
constexpr int TC_THREADS = 256, TC_THREADS_MID = 384, TC_THREADS_WIDE = 512;
constexpr int TC_GROUP_WARPS = 8;                         // row blocks of the grouping phase (whatever the block's size)
constexpr int TC_M = 128, TC_KC = 64;                    // rows of an MMA's output tile; K chunk = 64 16-bit numbers = one swizzled 128-byte row
// most centres per block (the MMA's N): 256 with one term per operand, 128 with two (the sample tile then takes twice the room)
__host__ __device__ constexpr int tc_block_n(int terms) { return terms == 1 ? 256 : 128; }
// centres per block for a state of k centres: a state that fits one block takes whole groups of 32 columns (the
// accumulators are read 32 columns at a time, and every column read has been written by the MMA)
__host__ __device__ constexpr int tc_block_rows(int k, int terms) { return k >= tc_block_n(terms) ? tc_block_n(terms) : (k + 31) / 32 * 32; }
// tensor-memory columns of the two accumulator stages: a power of two, at least 32
__host__ __device__ constexpr int tc_tmem_cols(int bn) { int c = 32; while (c < 2 * bn) c *= 2; return c; }
constexpr int TC_A_STAGES = 4;                            // K chunks of the resident sample tile (d <= 256), each with a hi and a lo part
constexpr int TC_B_STAGES = 4;                            // ring slots for the centre blocks (one K chunk of w_hi or of w_lo each)
constexpr int TC_A_STAGE_BYTES = TC_M * TC_KC * 2;       // 16 KB per part
constexpr int TC_MAX_K = 1024, TC_MAX_D = 256, TC_MAX_B = 4096;
constexpr unsigned TC_INDEX_MASK = 1023u;
constexpr int TC_SCAN_ROWS = 16;                          // rows the full scan measures at a time
constexpr float TC_FAR = 1e30f;                          // stands for ||w_a||^2 of the padding centres

struct TcSmem {
  size_t B, A, cn, cnt, best, flagged, bars, misc, tail, total;
  int cn_stride;               // floats of ||w_a||^2 per worker of the block
  // (the workers' ||w_a||^2 stay on chip side by side)
  size_t stage;                // epilogue warps that share a row hand their parts to the first of them here
  // nv: workers the block serves in turn; threads: the block's size
  __host__ __device__ TcSmem(int k, int d, int b, int terms, int nv, int threads) {
    const int nb = tc_block_rows(k, terms);
    size_t off = 0;
    auto take = [&](size_t bytes, size_t align) { off = (off + align - 1) / align * align; size_t o = off; off += bytes; return o; };
    // [K chunk][hi, lo] of the resident sample tile; also the scratch of the grouping phase ([warps][k] counts, [b] ranks)
    const size_t tile = (size_t)(d / TC_KC) * (terms == 3 ? 2 : 1) * TC_A_STAGE_BYTES;
    const size_t scratch = (size_t)TC_GROUP_WARPS * k * 4 + (size_t)b * 2;
    A = take(tile > scratch ? tile : scratch, 1024);
    B = take((size_t)TC_B_STAGES * nb * TC_KC * 2, 1024);                // also [k] group starts and the scans' results (nb >= 32: 16 KB)
    cn_stride = (k + nb - 1) / nb * nb;
    cn = take((size_t)nv * cn_stride * 4, 16);
    cnt = take((size_t)k * 4, 16);
    // best[b] and flagged[b + 8] (pairs to settle from the front, rows for the full scan from the back) are dead while
    // the scores are computed: the epilogue's hand-over area [tile parity][part][row] of (s1, s2, s3, floor) shares their room
    const int per_row = (threads / 32 - 4) / 4;                       // epilogue warps per quarter of a sample tile
    const size_t best_bytes = ((size_t)b * 2 + 15) / 16 * 16, flag_bytes = ((size_t)b * 2 + 16 + 15) / 16 * 16;
    const size_t stage_bytes = per_row > 1 ? (size_t)2 * per_row * TC_M * 16 : 0;
    best = take(best_bytes + flag_bytes > stage_bytes ? best_bytes + flag_bytes : stage_bytes, 16);
    flagged = best + best_bytes;
    stage = best;
    bars = take(32 * 8, 16);
    misc = take(64, 16);
    tail = take(sizeof(TailScratch), 16);
    total = off + 1024;          // room to align the base to 1024 bytes
  }
};
inline size_t tc_smem_bytes(int k, int d, int b, int terms, int nv, int threads) { return TcSmem(k, d, b, terms, nv, threads).total; }

// L2 policies: the samples stream through once per pass (first out), a worker's 16-bit state is read again for
// every sample tile (last out)
__device__ inline unsigned long long l2_policy_evict_first() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ inline unsigned long long l2_policy_evict_last() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ inline void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, unsigned long long* bar, unsigned long long policy) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
               ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy) : "memory");
}
// a float4 of the fp32 samples, read once: first out of L2, not kept in L1
__device__ inline float4 ldg_stream4(const float4* p, unsigned long long policy) {
  float4 v;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p), "l"(policy));
  return v;
}
// Shared-memory operand descriptor: K-major rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ inline unsigned long long tc_smem_desc(const void* smem, unsigned byte_off) {
  const unsigned addr = smem_u32(smem) + byte_off;
  unsigned long long d = 0;
  d |= (unsigned long long)((addr & 0x3FFFFu) >> 4);
  d |= (unsigned long long)1 << 16;
  d |= (unsigned long long)(1024 >> 4) << 32;
  d |= (unsigned long long)1 << 46;
  d |= (unsigned long long)2 << 61;
  return d;
}
__device__ inline void tc_mma_bf16(unsigned d_tmem, unsigned long long a, unsigned long long b, unsigned idesc, bool acc) {
  asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
               ::"r"(d_tmem), "l"(a), "l"(b), "r"(idesc), "r"((unsigned)acc) : "memory");
}
__device__ inline void tc_commit(unsigned long long* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ inline void mbar_arrive(unsigned long long* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ inline void red_add_v4(float* addr, float4 v) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}

// samples -> BF16 hi and lo terms (initialisation).  hi_in: the caller's BF16 copy, or nullptr (then hi = round(x));
// lo = round(x - hi) either way, so that hi + lo is x to 16 bits whatever copy the caller brought.
__global__ void tc_split_x_kernel(const float* __restrict__ X, const __nv_bfloat16* __restrict__ hi_in, __nv_bfloat16* __restrict__ hi_out,
                                  __nv_bfloat16* __restrict__ lo_out, size_t n) {
  for (size_t e = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 2; e + 1 < n; e += (size_t)gridDim.x * blockDim.x * 2) {
    const float2 v = *reinterpret_cast<const float2*>(X + e);
    __nv_bfloat162 h = hi_in ? *reinterpret_cast<const __nv_bfloat162*>(hi_in + e) : __floats2bfloat162_rn(v.x, v.y);
    if (hi_out) *reinterpret_cast<__nv_bfloat162*>(hi_out + e) = h;
    const float2 hf = __bfloat1622float2(h);
    *reinterpret_cast<__nv_bfloat162*>(lo_out + e) = __floats2bfloat162_rn(v.x - hf.x, v.y - hf.y);
  }
}
// samples -> FP16 (initialisation, one-term format)
__global__ void tc_half_x_kernel(const float* __restrict__ X, __half* __restrict__ out, size_t n) {
  for (size_t e = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 2; e + 1 < n; e += (size_t)gridDim.x * blockDim.x * 2) {
    const float2 v = *reinterpret_cast<const float2*>(X + e);
    *reinterpret_cast<__half2*>(out + e) = __floats2half2_rn(v.x, v.y);
  }
}
// ||x_i||^2 of every row (fp32): added to the scores so that the numbers compared are squared distances, whose
// low mantissa bits (where the centre index rides) are worth far less than those of the raw scores.
__global__ void tc_row_norms_kernel(const float* __restrict__ X, long long N, int d, float* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  for (long long r = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < N; r += ((long long)gridDim.x * blockDim.x) >> 5) {
    const float* x = X + (size_t)r * d;
    float s = 0.f;
    for (int j = lane * 2; j < d; j += 64) { const float2 v = *reinterpret_cast<const float2*>(x + j); s = fmaf(v.x, v.x, s); s = fmaf(v.y, v.y, s); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) out[r] = s;
  }
}

// barrier slots
enum { TCB_BFULL = 0 /* [issuing thread][slot] */, TCB_BEMPTY = 2 * TC_B_STAGES, TCB_AFULL = 3 * TC_B_STAGES, TCB_AEMPTY = 3 * TC_B_STAGES + TC_A_STAGES,
       TCB_ACCFULL = 3 * TC_B_STAGES + 2 * TC_A_STAGES, TCB_ACCEMPTY = TCB_ACCFULL + 2, TCB_COUNT = TCB_ACCFULL + 4 };
static_assert(TCB_COUNT <= 32, "barrier slots");

// smallest three of (m1 <= m2 <= m3) and a new value, kept sorted (five min/max)
__device__ __forceinline__ void tc_top3_insert(float& m1, float& m2, float& m3, float v) {
  const float hi1 = fmaxf(m1, v);
  m1 = fminf(m1, v);
  const float hi2 = fmaxf(m2, hi1);
  m2 = fminf(m2, hi1);
  m3 = fminf(m3, hi2);
}

// the same for two new values at once (eight min/max, three of them three-input): with lo <= hi the new triple is
//   min(m1, lo),  min(max(m1, lo), m2, hi),  min(m3, max(m2, lo), max(m1, hi))
__device__ __forceinline__ void tc_top3_insert2(float& m1, float& m2, float& m3, float v, float u) {
  const float lo = fminf(v, u), hi = fmaxf(v, u);
  const float a = fmaxf(m1, lo), b2 = fmaxf(m2, lo), c = fmaxf(m1, hi);
  m3 = fmin3(m3, b2, c);
  m2 = fmin3(a, m2, hi);
  m1 = fminf(m1, lo);
}

// kMaxD: the largest d the instance holds in registers.  256: one block per SM.  128: half the registers, so that two
// blocks share an SM when their shared memory allows it; one block's scores then overlap the other's sums and update.
// kThreads: 256 where two blocks share an SM; a block that has an SM to itself takes 384 threads (two epilogue warps per
// quarter of a sample tile), or 512 with rows of at most 128 numbers (three), and as many more warps in every later phase.
template <bool kDet, int kTerms, int kMaxD, int kThreads>
__global__ void __launch_bounds__(kThreads, (kMaxD <= 128 && kThreads == TC_THREADS) ? 2 : 1)
asgd_tc_kernel(const Params p, const long long steps, const __grid_constant__ CUtensorMap mapXh,
               const __grid_constant__ CUtensorMap mapXl, const __grid_constant__ CUtensorMap mapW) {
  extern __shared__ __align__(1024) unsigned char smem_dyn[];
  unsigned char* smem = smem_dyn + ((1024u - (smem_u32(smem_dyn) & 1023u)) & 1023u);
  const int k = p.k, d = p.d, b = p.b;
  const int G = (int)gridDim.x;
  const int nv = (p.W - (int)blockIdx.x + G - 1) / G;                   // workers of this block: blockIdx.x + v * G
  constexpr int NT = kThreads, NW = kThreads / 32;                      // threads and warps of the block
  constexpr int GW = TC_GROUP_WARPS;
  static_assert(kThreads <= TC_THREADS_MID || kMaxD <= 128, "512 threads only with 128 registers a thread");
  const TcSmem map(k, d, b, kTerms, (p.W + G - 1) / G, NT);
  unsigned char* sB = smem + map.B;
  unsigned char* sA = smem + map.A;
  float* cn = reinterpret_cast<float*>(smem + map.cn);                 // ||w_a||^2 of the worker in turn; beyond k a large finite number (with
                                                                       // index bits packed in, an infinity would read as a NaN and upset the min/max chain)
  int* cnt = reinterpret_cast<int*>(smem + map.cnt);
  unsigned short* best = reinterpret_cast<unsigned short*>(smem + map.best);
  unsigned short* flagged = reinterpret_cast<unsigned short*>(smem + map.flagged);
  unsigned long long* bars = reinterpret_cast<unsigned long long*>(smem + map.bars);
  int* misc = reinterpret_cast<int*>(smem + map.misc);                 // [0] tmem base, [1] pairs to settle, [2] abort, [4] news, [5] rows for the full scan, [6] rows with three candidates, [7] next centre of the sum phase
  TailScratch* ts = reinterpret_cast<TailScratch*>(smem + map.tail);

  static_assert(kTerms == 1 || kTerms == 3, "one FP16 term or two BF16 terms per operand");
  constexpr int PPK = (kTerms == 3) ? 2 : 1;                            // parts (hi, lo) per K chunk of an operand
  constexpr int QN = kMaxD / 32;                                        // float4 pieces of a row per lane of an eight-lane group
  constexpr bool kWide = kMaxD > 128;                                   // rows of more than 128 numbers: a second float4 per lane in the scans
  const int TC_N = tc_block_rows(k, kTerms);                            // centres per block
  const int TC_B_CHUNK_BYTES = TC_N * TC_KC * 2;                        // a ring slot: one K chunk of a centre block
  const int TC_TMEM_COLS = tc_tmem_cols(TC_N);                          // two accumulator stages
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const int nkc = d / TC_KC;                                           // K chunks per tile
  const int n_tiles = (k + TC_N - 1) / TC_N, m_tiles = (b + TC_M - 1) / TC_M;
  // the worker in turn
  int i = blockIdx.x;
  float* wglob = nullptr;
  float* gsum = nullptr;
  unsigned short* wbf = nullptr;                                        // 16-bit -2w (w_hi) of the worker
  unsigned short* wbl = nullptr;                                        // w_lo: second half of the array (two-term format)
  float4* top3 = nullptr;                                               // per row: three smallest packed squared distances and the floor under the fourth
  auto take_worker = [&](int v) {
    i = (int)blockIdx.x + v * G;
    wglob = p.state + (size_t)i * p.kd_pad;
    gsum = p.gsum + (size_t)i * p.kd_pad;
    wbf = reinterpret_cast<unsigned short*>(p.wbf) + (size_t)i * k * d;
    wbl = wbf + (size_t)p.W * k * d;
    top3 = reinterpret_cast<float4*>(p.top2) + (size_t)i * b;
    cn = reinterpret_cast<float*>(smem + map.cn) + (size_t)v * map.cn_stride;
  };
  const float INF = __int_as_float(0x7f800000);
  const float inv_b = 1.0f / (float)b;

  if (tid == 0) {
    for (int q = 0; q < TC_B_STAGES; ++q) { mbar_init(bars + TCB_BFULL + q, 1); mbar_init(bars + TCB_BFULL + TC_B_STAGES + q, 1); mbar_init(bars + TCB_BEMPTY + q, 1); }
    // a sample chunk is free when every issuing thread has seen its last products on it complete
    for (int q = 0; q < TC_A_STAGES; ++q) { mbar_init(bars + TCB_AFULL + q, 1); mbar_init(bars + TCB_AEMPTY + q, (k + TC_N - 1) / TC_N >= 2 ? 2 : 1); }
    for (int q = 0; q < 2; ++q) { mbar_init(bars + TCB_ACCFULL + q, 1); mbar_init(bars + TCB_ACCEMPTY + q, NW - 4); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    misc[2] = 0;
  }
  if (wid == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(misc)), "r"((unsigned)TC_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // -2w as two BF16 terms and ||w_a||^2 of one centre held by eight lanes (lane l8: dimensions 4*l8 + 32*q)
  const int sub = lane >> 3, l8 = lane & 7;
  const int nq = d / 32;
  // 16-bit terms of -2w for four numbers of the state at element offset o (a multiple of 4): one 8-byte store per
  // term; returns the four numbers' sum of squares
  auto put16 = [&](size_t o, const float4& w) {
    const float v[4] = {-2.f * w.x, -2.f * w.y, -2.f * w.z, -2.f * w.w};     // exact
    if (kTerms == 1) {
      const __half2 h01 = __floats2half2_rn(v[0], v[1]), h23 = __floats2half2_rn(v[2], v[3]);
      *reinterpret_cast<uint2*>(wbf + o) = make_uint2(*reinterpret_cast<const unsigned*>(&h01), *reinterpret_cast<const unsigned*>(&h23));
    } else {
      const __nv_bfloat162 h01 = __floats2bfloat162_rn(v[0], v[1]), h23 = __floats2bfloat162_rn(v[2], v[3]);
      const float2 f01 = __bfloat1622float2(h01), f23 = __bfloat1622float2(h23);
      const __nv_bfloat162 l01 = __floats2bfloat162_rn(v[0] - f01.x, v[1] - f01.y), l23 = __floats2bfloat162_rn(v[2] - f23.x, v[3] - f23.y);
      *reinterpret_cast<uint2*>(wbf + o) = make_uint2(*reinterpret_cast<const unsigned*>(&h01), *reinterpret_cast<const unsigned*>(&h23));
      *reinterpret_cast<uint2*>(wbl + o) = make_uint2(*reinterpret_cast<const unsigned*>(&l01), *reinterpret_cast<const unsigned*>(&l23));
    }
    float sq = w.x * w.x;
    sq = fmaf(w.y, w.y, sq); sq = fmaf(w.z, w.z, sq); sq = fmaf(w.w, w.w, sq);
    return sq;
  };
  auto refresh = [&](int a, const float4 (&w4)[QN]) {
    float sq = 0.f;
#pragma unroll
    for (int q = 0; q < QN; ++q)
      if (q < nq) sq += put16((size_t)a * d + 4 * l8 + 32 * q, w4[q]);
    return sq;
  };
  auto refresh_all = [&]() {                                            // every centre from the fp32 state in HBM
    for (int a0 = wid * 4; a0 < n_tiles * TC_N; a0 += NW * 4) {
      const int a = a0 + sub;
      float sq = 0.f;
      if (a < k) {
        float4 w4[QN];
#pragma unroll
        for (int q = 0; q < QN; ++q)
          if (q < nq) w4[q] = *reinterpret_cast<const float4*>(wglob + (size_t)a * d + 4 * l8 + 32 * q);
        sq = refresh(a, w4);
      }
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if (l8 == 0) cn[a] = (a < k) ? sq : TC_FAR;
    }
  };
  for (int v = 0; v < nv; ++v) { take_worker(v); refresh_all(); }
  asm volatile("fence.proxy.async;" ::: "memory");                      // the 16-bit terms written above are read by TMA
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem = (unsigned)misc[0];
  // instruction descriptor: fp32 accumulate, operand format (0 = FP16, 1 = BF16) for both operands, N / 8, M / 16
  const unsigned fmt = (kTerms == 3) ? 1u : 0u;
  const unsigned idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((unsigned)(TC_N >> 3) << 17) | ((unsigned)(TC_M >> 4) << 24);

  // running phase counters of the pipelines (each role keeps its own copies in step)
  unsigned it_m = 0, it_bc = 0, it_acc = 0;
  unsigned bfull_par = 0;                                 // an issuing thread's next phase of each of its ring barriers (a bit per slot)
  const bool two_issuers = n_tiles >= 2;

  bool gave_up = false;
  for (long long step = 0; step < steps && !gave_up; ++step)
  for (int v = 0; v < nv; ++v) {                          // the block's workers take the step one after the other
    take_worker(v);
    const unsigned long long t = *reinterpret_cast<volatile unsigned long long*>(p.stats + (size_t)i * ST_STRIDE + ST_STEPS);   // written by this block at the end of the worker's last step
    const long long batch = p.perm[(size_t)i * p.B + (size_t)(t % (unsigned long long)p.B)];
    const long long row0 = (long long)i * p.H + batch * b;

    // ================= scores: three BF16 products per K chunk, three best per sample =================
    // A sample tile (128 rows, nkc K-chunks of x_hi and x_lo) stays in shared memory while the centre blocks stream
    // past it through the ring, w_hi then w_lo of every K chunk; the samples are read from HBM once.
    if (wid == 0) {
      if (lane == 0) {
        unsigned um = it_m, ibc = it_bc;
        bool ok = true;
        const unsigned long long pol_x = l2_policy_evict_first(), pol_w = l2_policy_evict_last();
        for (int m = 0; m < m_tiles && ok; ++m, ++um) {
          for (int kc = 0; kc < nkc && ok; ++kc) {
            if (um > 0) ok = mbar_wait_bounded(bars + TCB_AEMPTY + kc, (um - 1) & 1, p.wait_limit);     // last use of the chunk by the previous tile
            if (!ok) break;
            mbar_expect_tx(bars + TCB_AFULL + kc, (unsigned)(PPK * TC_A_STAGE_BYTES));
            const bool withheld = (m == 0 && kc == 0 && step == p.withhold_step);   // failure drill: announced, never copied
            if (!withheld) {
              tma_load_2d(sA + (size_t)(kc * PPK + 0) * TC_A_STAGE_BYTES, &mapXh, kc * TC_KC, (int)(row0 + (long long)m * TC_M), bars + TCB_AFULL + kc, pol_x);
              if (kTerms == 3)
                tma_load_2d(sA + (size_t)(kc * PPK + 1) * TC_A_STAGE_BYTES, &mapXl, kc * TC_KC, (int)(row0 + (long long)m * TC_M), bars + TCB_AFULL + kc, pol_x);
            }
          }
          for (int n = 0; n < n_tiles && ok; ++n) {
            // the full barrier of the thread that will issue this centre block's products
            const int q_full = two_issuers ? (int)((it_acc + (unsigned)(m * n_tiles + n)) & 1u) * TC_B_STAGES : 0;
            for (int g = 0; g < PPK * nkc; ++g, ++ibc) {               // g = PPK * K chunk + (0: w_hi, 1: w_lo)
              const int st = ibc % TC_B_STAGES;
              if (ibc >= TC_B_STAGES) ok = mbar_wait_bounded(bars + TCB_BEMPTY + st, ((ibc / TC_B_STAGES) - 1) & 1, p.wait_limit);
              if (!ok) break;
              mbar_expect_tx(bars + TCB_BFULL + q_full + st, (unsigned)TC_B_CHUNK_BYTES);
              tma_load_2d(sB + (size_t)st * TC_B_CHUNK_BYTES, &mapW, (g / PPK) * TC_KC, (g % PPK) * p.W * k + i * k + n * TC_N, bars + TCB_BFULL + q_full + st, pol_w);
            }
          }
        }
        if (!ok) atomicExch(&misc[2], 1);
      }
    } else if (wid == 1 || (wid == 2 && two_issuers)) {
      // Two issuing threads, one per accumulator stage (centre blocks in turn), when a sample tile meets at least two
      // centre blocks.  A tcgen05.commit holds the thread that issues it for several hundred cycles (measured: one
      // thread issuing four products and a commit in turn reaches 275 cycles per product, two threads doing so side
      // by side 133, the rate without commits 128), so the other thread's products keep the tensor pipe fed
      // meanwhile.  The pipe runs the products in the order they were issued, each block's products come from one
      // thread, a ring slot or a sample chunk is handed back by the thread that used it last, and each thread has its
      // own full barriers for the ring, so that it sees every phase of every barrier it waits on (a parity wait cannot
      // tell the last completed phase from the one before).  Both threads meet every sample tile.
      if (lane == 0) {
        const unsigned me = (unsigned)(wid - 1);
        unsigned um = it_m, ibc = it_bc, iacc = it_acc;
        bool ok = true;
        const unsigned long long dA0 = tc_smem_desc(sA, 0), dB0 = tc_smem_desc(sB, 0);
        for (int m = 0; m < m_tiles && ok; ++m, ++um) {
          bool first_here = true;                          // this thread's first centre block of the sample tile
          for (int n = 0; n < n_tiles && ok; ++n, ++iacc) {
            const int buf = iacc & 1;
            if (two_issuers && (unsigned)buf != me) { ibc += (unsigned)(PPK * nkc); continue; }      // the other thread's block
            if (iacc >= 2) ok = mbar_wait_bounded(bars + TCB_ACCEMPTY + buf, ((iacc >> 1) - 1) & 1, p.wait_limit);
            if (!ok) break;
            tc_fence_after();
            const unsigned acc_col = tmem + (unsigned)(buf * TC_N);
            for (int g = 0; g < PPK * nkc && ok; ++g, ++ibc) {
              const int st = ibc % TC_B_STAGES;
              const int kc = g / PPK, lo_w = g % PPK;
              if (first_here && lo_w == 0) ok = mbar_wait_bounded(bars + TCB_AFULL + kc, um & 1, p.wait_limit);
              // this thread's uses of the slot so far decide the phase
              if (ok) ok = mbar_wait_bounded(bars + TCB_BFULL + (two_issuers ? (int)me * TC_B_STAGES : 0) + st, (bfull_par >> st) & 1u, p.wait_limit);
              if (!ok) break;
              bfull_par ^= 1u << st;
              tc_fence_after();
              // operand descriptors: the base descriptor plus the chunk's offset in 16-byte units (the address field
              // holds address >> 4 and shared memory is below 256 KB, so the sum stays inside the field)
              const unsigned long long db = dB0 + (unsigned long long)(st * (TC_B_CHUNK_BYTES >> 4));
              const unsigned long long dah = dA0 + (unsigned long long)((kc * PPK + 0) * (TC_A_STAGE_BYTES >> 4));
              const unsigned long long dal = dA0 + (unsigned long long)((kc * PPK + 1) * (TC_A_STAGE_BYTES >> 4));
#pragma unroll
              for (int k4 = 0; k4 < TC_KC / 16; ++k4)                   // x_hi . w_hi  or  x_hi . w_lo
                tc_mma_bf16(acc_col, dah + (unsigned long long)(2 * k4), db + (unsigned long long)(2 * k4), idesc, (g | k4) != 0);
              if (kTerms == 3 && lo_w == 0) {
#pragma unroll
                for (int k4 = 0; k4 < TC_KC / 16; ++k4)                 // x_lo . w_hi
                  tc_mma_bf16(acc_col, dal + (unsigned long long)(2 * k4), db + (unsigned long long)(2 * k4), idesc, true);
              }
              tc_commit(bars + TCB_BEMPTY + st);                        // the ring slot is free when these MMAs have read it
              // and so is the sample chunk after this thread's last centre block of the tile
              if ((two_issuers ? n + 2 >= n_tiles : n == n_tiles - 1) && lo_w == PPK - 1) tc_commit(bars + TCB_AEMPTY + kc);
            }
            tc_commit(bars + TCB_ACCFULL + buf);                        // the accumulator stage is complete
            first_here = false;
          }
        }
        if (!ok) atomicExch(&misc[2], 1);
      }
    } else if (wid >= 4) {
      // the other warps read the accumulators: a warp can reach the TMEM lanes 32q .. 32q+31 with q = warp mod 4, i.e.
      // one row per thread; the EPW warps of a quarter take the 32-column groups of a centre block in turn
      constexpr int EPW = (NW - 4) / 4;
      const int quarter = wid & 3, part = (wid - 4) >> 2;
      float4* stage = reinterpret_cast<float4*>(smem + map.stage);    // [tile parity][part][row of the tile]
      unsigned iacc = it_acc;
      bool ok = true;
      for (int m = 0; m < m_tiles; ++m) {
        const int r = m * TC_M + quarter * 32 + lane;              // the thread's row of the batch
        const float xn = (r < b) ? __ldg(p.xnorm + row0 + r) : 0.f;
        float m1[4], m2[4], m3[4];                                  // four independent sorted triples, kept over the centre blocks
#pragma unroll
        for (int q = 0; q < 4; ++q) m1[q] = m2[q] = m3[q] = INF;
        for (int n = 0; n < n_tiles; ++n, ++iacc) {
          const int buf = iacc & 1;
          if (ok) ok = __all_sync(0xffffffffu, mbar_wait_bounded(bars + TCB_ACCFULL + buf, (iacc >> 1) & 1, p.wait_limit));
          if (!ok) continue;
          tc_fence_after();
          if (32 * part >= TC_N) {                        // fewer column groups than warps: nothing to read here
            tc_fence_before();
            if (lane == 0) mbar_arrive(bars + TCB_ACCEMPTY + buf);
          }
#pragma unroll 1
          for (int c0 = 32 * part; c0 < TC_N; c0 += 32 * EPW) {
            unsigned v[32];
            const unsigned taddr = tmem + ((unsigned)(quarter * 32) << 16) + (unsigned)(buf * TC_N + c0);
            asm volatile(
                "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                  "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
                  "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
                  "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
                : "r"(taddr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (c0 + 32 * EPW >= TC_N) {                  // this warp's last read of the accumulator stage: hand it back
              tc_fence_before();
              if (lane == 0) mbar_arrive(bars + TCB_ACCEMPTY + buf);
            }
            const int abase = n * TC_N + c0;
            const unsigned hi_or_base = ~TC_INDEX_MASK | (unsigned)abase;   // abase is a multiple of 32: its bits and a column's do not meet
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
              const float4 cn4 = *reinterpret_cast<const float4*>(cn + abase + c);
              const float cv[4] = {cn4.x, cn4.y, cn4.z, cn4.w};
              float sp[4];
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                // squared distance ||x||^2 - 2 x.w_a + ||w_a||^2 (fp32 adds), then one logic op: the value's high
                // bits, the block's and the column's index bits below them
                const float d2 = (__uint_as_float(v[c + u]) + cv[u]) + xn;
                unsigned spb;
                asm("lop3.b32 %0, %1, %2, %3, 0xE6;" : "=r"(spb) : "r"(__float_as_uint(d2)), "r"(hi_or_base), "r"(~TC_INDEX_MASK | (unsigned)(c + u)));
                sp[u] = __uint_as_float(spb);
              }
              const int sq = (c >> 1) & 2;                        // columns 0-3 of every eight feed triples 0 and 1, columns 4-7 triples 2 and 3
              tc_top3_insert2(m1[sq], m2[sq], m3[sq], sp[0], sp[1]);
              tc_top3_insert2(m1[sq + 1], m2[sq + 1], m3[sq + 1], sp[2], sp[3]);
            }
          }
        }
        {
          // the four smallest of the twelve kept values.  Every value that was not kept is at least the largest of its
          // triple, so the fourth smallest of ALL values is at least min(fourth smallest kept, smallest of the four
          // triples' largest): a floor under the fourth candidate that costs nothing in the loop above
          float a1 = INF, a2 = INF, a3 = INF, a4 = INF;
          auto put4 = [&](float v) {
            const float h1 = fmaxf(a1, v); a1 = fminf(a1, v);
            const float h2 = fmaxf(a2, h1); a2 = fminf(a2, h1);
            const float h3 = fmaxf(a3, h2); a3 = fminf(a3, h2);
            a4 = fminf(a4, h3);
          };
#pragma unroll
          for (int q = 0; q < 4; ++q) { put4(m1[q]); put4(m2[q]); put4(m3[q]); }
          float floor4 = fminf(a4, fminf(fminf(m3[0], m3[1]), fminf(m3[2], m3[3])));
          if (EPW > 1) {
            // the parts of a row meet in shared memory (every warp of the quarter comes to the barrier, whatever its
            // waits did): the three smallest of all parts are among the parts' three smallest, and the fourth smallest
            // of all is one of those or at least some part's floor
            float4* mine = stage + ((size_t)(m & 1) * EPW + part) * TC_M + quarter * 32 + lane;
            if (part > 0) *mine = make_float4(a1, a2, a3, floor4);
            asm volatile("bar.sync %0, %1;" ::"r"(1 + quarter), "r"(32 * EPW) : "memory");
            if (part == 0) {
              a4 = __int_as_float(0x7f800000);
#pragma unroll
              for (int q = 1; q < EPW; ++q) {
                const float4 o = mine[(size_t)q * TC_M];
                put4(o.x); put4(o.y); put4(o.z);
                floor4 = fminf(floor4, o.w);
              }
              floor4 = fminf(floor4, a4);
            }
          }
          if (ok && r < b && part == 0) __stcg(top3 + r, make_float4(a1, a2, a3, floor4));
        }
      }
      if (!ok && lane == 0) atomicExch(&misc[2], 1);
    }
    it_m += (unsigned)m_tiles;
    it_bc += (unsigned)(m_tiles * n_tiles * PPK * nkc);
    it_acc += (unsigned)(n_tiles * m_tiles);
    if (tid == 0) { misc[1] = 0; misc[5] = 0; misc[6] = 0; misc[7] = NW * 4; }
    for (int a = tid; a < k; a += NT) cnt[a] = 0;
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (misc[2]) { gave_up = true; break; }               // a wait ran out: report and leave (uniform)

    // ================= decide =================
    float wmax2 = 0.f;
    for (int a = lane; a < k; a += 32) wmax2 = fmaxf(wmax2, cn[a]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wmax2 = fmaxf(wmax2, __shfl_xor_sync(0xffffffffu, wmax2, o));
    // Error of a computed squared distance (see the file header and the tolerance note of the library):
    //   terms left out of the split product          6 * 2^-18 ||x|| ||w||
    //   fp32 accumulation of 3 d / 16 partial sums    (3 d / 16 + 1) * 2^-22 ||x|| ||w||     (each step at most one ulp of a sum <= 2 ||x|| ||w||)
    //   the two fp32 adds of the norms                3 * 2^-24 (||x||^2 + ||w||^2 + 2 ||x|| ||w||)
    // with a quarter on top; the index bits cost 2^10 ulp <= 2^-13 of the value itself, applied relative to the values compared.
    // One FP16 term per operand: both factors of a product are off by 2^-12 relative, the sum of |x_j| |2 w_j| is at
    // most 2 ||x|| ||w||: 2^-10 ||x|| ||w||; d / 16 partial sums; inputs below FP16's normal range (6.1e-5) lose at
    // most 2^-25 each in absolute terms: 2^-24 sqrt(d) (||x|| + 2 ||w||) in all.
    // The bound is taken per row, with the row's own ||x||^2 (and the largest ||w_a||^2).
    auto row_err = [&](float xn) {
      const float xw = sqrtf(xn * wmax2);
      return (kTerms == 3)
          ? 1.25f * ((2.289e-5f + (float)(3 * d / 16 + 1) * 2.384e-7f) * xw + 1.79e-7f * (xn + wmax2 + 2.f * xw))
          : 1.25f * ((9.766e-4f + (float)(d / 16 + 1) * 2.384e-7f) * xw + 1.79e-7f * (xn + wmax2 + 2.f * xw) +
                     5.96e-8f * sqrtf((float)d) * (sqrtf(xn) + 2.f * sqrtf(wmax2)));
    };
    auto inside = [&](float lo, float hi_, float err) { return (hi_ - lo) <= 2.f * err + 2.4415e-4f * fmaxf(fabsf(lo), fabsf(hi_)); };
    // Scratch for the rest of the step lives in the sample ring, which is idle until the next step's loads.
    int* wcnt = reinterpret_cast<int*>(sA);                                   // [GW][k] rows of a centre in a row block
    unsigned short* lrank = reinterpret_cast<unsigned short*>(sA + (size_t)GW * k * 4);   // [b] rank of a row among its block's rows of the centre
    unsigned short* order = flagged;                                          // [b] rows grouped by centre, ascending inside a group
    unsigned short* triples = lrank;                                          // until the grouping: rows with exactly three candidates

    // ---- decide: the minimum, unless the runner-up lies inside the bound (settle the pair) or the third does too (scan all) ----
    for (int e = tid; e < GW * k; e += NT) wcnt[e] = 0;
    for (int r = tid; r < b; r += NT) {
      const float4 s = __ldcg(top3 + r);
      best[r] = (unsigned short)(__float_as_uint(s.x) & TC_INDEX_MASK);
      const float err = row_err(__ldg(p.xnorm + row0 + r));
      if (k > 1 && inside(s.x, s.y, err)) {
        if (k > 2 && inside(s.x, s.z, err)) {
          if (k > 3 && inside(s.x, s.w, err)) order[b - 1 - atomicAdd(&misc[5], 1)] = (unsigned short)r;   // a fourth may be inside: all centres
          else triples[atomicAdd(&misc[6], 1)] = (unsigned short)r;                                         // exactly three candidates
        } else {
          order[atomicAdd(&misc[1], 1)] = (unsigned short)r;
        }
      }
    }
    __syncthreads();
    // ---- listed rows are settled among their two or three candidates with fp32 inputs (direct differences; fp64 sums
    //      when the two smallest fp32 distances are within rounding of each other): eight lanes per row (lane l8 holds
    //      dimensions 4*l8 + 32*q), a warp settles four rows at a time ----
    {
      const int npair = misc[1], ntrip = misc[6];
      const int groups = NW * 4;
      for (int fb = wid * 4; fb < npair + ntrip; fb += groups) {   // the same trip count for all lanes of a warp (shuffles inside)
        const int f = fb + sub;
        const bool have = f < npair + ntrip;
        const bool three = f >= npair;
        const int r = have ? (int)(three ? triples[f - npair] : order[f]) : -1;
        const float4 s = (r >= 0) ? __ldcg(top3 + r) : make_float4(0.f, 0.f, 0.f, 0.f);
        const int i1 = (int)(__float_as_uint(s.x) & TC_INDEX_MASK), i2 = (int)(__float_as_uint(s.y) & TC_INDEX_MASK);
        const int i3 = (have && three) ? (int)(__float_as_uint(s.z) & TC_INDEX_MASK) : i2;
        const float* x = p.X + (size_t)(row0 + max(r, 0)) * d + 4 * l8;
        const float* w1 = wglob + (size_t)i1 * d + 4 * l8;
        const float* w2 = wglob + (size_t)i2 * d + 4 * l8;
        const float* w3 = wglob + (size_t)i3 * d + 4 * l8;
        float4 xv[QN], c1[QN], c2[QN], c3[QN];
#pragma unroll
        for (int q = 0; q < QN; ++q) {
          if (q < nq && r >= 0) {
            xv[q] = __ldg(reinterpret_cast<const float4*>(x + 32 * q));
            c1[q] = *reinterpret_cast<const float4*>(w1 + 32 * q);
            c2[q] = *reinterpret_cast<const float4*>(w2 + 32 * q);
            c3[q] = *reinterpret_cast<const float4*>(w3 + 32 * q);
          } else {
            xv[q] = c1[q] = c2[q] = c3[q] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
        }
        // direct differences in fp32 first: each squared distance is off by at most (d + 2) u relative, so a gap
        // above (4 d + 16) u of the larger one decides; only rows closer than that are summed again in fp64
        float f1 = 0.f, f2 = 0.f, f3 = 0.f;
#pragma unroll
        for (int q = 0; q < QN; ++q) {
          float u;
          u = xv[q].x - c1[q].x; f1 = fmaf(u, u, f1); u = xv[q].y - c1[q].y; f1 = fmaf(u, u, f1);
          u = xv[q].z - c1[q].z; f1 = fmaf(u, u, f1); u = xv[q].w - c1[q].w; f1 = fmaf(u, u, f1);
          u = xv[q].x - c2[q].x; f2 = fmaf(u, u, f2); u = xv[q].y - c2[q].y; f2 = fmaf(u, u, f2);
          u = xv[q].z - c2[q].z; f2 = fmaf(u, u, f2); u = xv[q].w - c2[q].w; f2 = fmaf(u, u, f2);
          u = xv[q].x - c3[q].x; f3 = fmaf(u, u, f3); u = xv[q].y - c3[q].y; f3 = fmaf(u, u, f3);
          u = xv[q].z - c3[q].z; f3 = fmaf(u, u, f3); u = xv[q].w - c3[q].w; f3 = fmaf(u, u, f3);
        }
#pragma unroll
        for (int o = 1; o < 8; o <<= 1) {
          f1 += __shfl_xor_sync(0xffffffffu, f1, o); f2 += __shfl_xor_sync(0xffffffffu, f2, o); f3 += __shfl_xor_sync(0xffffffffu, f3, o);
        }
        if (!three) f3 = INF;                                                    // a pair has no third candidate
        const float lo = fminf(f1, fminf(f2, f3));
        const float mid = fmaxf(fminf(f1, f2), fminf(fmaxf(f1, f2), f3));       // the second smallest
        int pick = (f1 == lo) ? i1 : (f2 == lo) ? i2 : i3;
        const bool close = (mid - lo) <= (float)(4 * TC_MAX_D + 16) * 5.9604645e-8f * mid;
        if (__any_sync(0xffffffffu, close && r >= 0)) {       // warp-uniform: the shuffles below need every lane
          double d1 = 0.0, d2 = 0.0, d3 = 0.0;
#pragma unroll
          for (int q = 0; q < QN; ++q) {
            double u;
            u = (double)xv[q].x - (double)c1[q].x; d1 = fma(u, u, d1); u = (double)xv[q].y - (double)c1[q].y; d1 = fma(u, u, d1);
            u = (double)xv[q].z - (double)c1[q].z; d1 = fma(u, u, d1); u = (double)xv[q].w - (double)c1[q].w; d1 = fma(u, u, d1);
            u = (double)xv[q].x - (double)c2[q].x; d2 = fma(u, u, d2); u = (double)xv[q].y - (double)c2[q].y; d2 = fma(u, u, d2);
            u = (double)xv[q].z - (double)c2[q].z; d2 = fma(u, u, d2); u = (double)xv[q].w - (double)c2[q].w; d2 = fma(u, u, d2);
            u = (double)xv[q].x - (double)c3[q].x; d3 = fma(u, u, d3); u = (double)xv[q].y - (double)c3[q].y; d3 = fma(u, u, d3);
            u = (double)xv[q].z - (double)c3[q].z; d3 = fma(u, u, d3); u = (double)xv[q].w - (double)c3[q].w; d3 = fma(u, u, d3);
          }
#pragma unroll
          for (int o = 1; o < 8; o <<= 1) {
            d1 += __shfl_xor_sync(0xffffffffu, d1, o); d2 += __shfl_xor_sync(0xffffffffu, d2, o); d3 += __shfl_xor_sync(0xffffffffu, d3, o);
          }
          if (!three) d3 = 1e300;
          if (close) {                                        // the smallest, the lowest index among equals
            pick = i1;
            double bd = d1;
            if (d2 < bd || (d2 == bd && i2 < pick)) { bd = d2; pick = i2; }
            if (d3 < bd || (d3 == bd && i3 < pick)) { bd = d3; pick = i3; }
          }
        }
        if (r >= 0 && l8 == 0) best[r] = (unsigned short)pick;
      }
    }
    // ---- rows with three or more candidates are decided over all centres, TC_SCAN_ROWS rows at a time: every lane
    //      holds its dimensions of all the rows in registers, every warp walks its share of the centres (a centre row is
    //      one coalesced read, lanes over the dimensions, the next centre's row already on its way) and measures it
    //      against every row with direct differences in fp32; the lanes' partial sums of all rows are added up by a
    //      halving exchange (a run of lanes ends with row j's distance), and the first lane of the run keeps row j's three smallest.  A row
    //      whose two smallest are still within rounding of each other is measured once more in fp64. ----
    {
      __syncthreads();                                         // the pairs' readers of `order` and `top3` are done; the ring is idle
      const int nwide = misc[5];
      const int d4 = d / 4;
      const bool on0 = lane < d4, on1 = kWide && 32 + lane < d4;
      const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
      // one batch of R <= RB rows against CB centres per warp at a time: RB x CB = 16 (row, centre) pairs either way
      // (16 rows x 1 centre, or for the usual handful 4 rows x 4 centres, whose four rows of the state are on their way together)
      auto scan_batch = [&](auto rb_tag, auto cb_tag, const int base, const int R) {
        constexpr int RB = decltype(rb_tag)::value, CB = decltype(cb_tag)::value;
        constexpr int VR = RB * CB;                            // (centre slot c, row j) pairs, pair c * RB + j
        constexpr int LPR = 32 / VR;                           // lanes that end up with the same pair: LPR * v .. LPR * v + LPR - 1
        float* res = reinterpret_cast<float*>(sB);             // [NW][VR][5] per warp and pair: the three smallest, indices of the first two
        int* need64 = reinterpret_cast<int*>(res + NW * VR * 5);    // [RB][3]: 0 decided, 1 compare two in fp64, 2 scan all in fp64; the two indices
        float4 xr0[RB], xr1[RB];                               // this lane's dimensions of the rows (zeros past the last row)
#pragma unroll
        for (int j = 0; j < RB; ++j) {
          const float4* xrow = reinterpret_cast<const float4*>(p.X + (size_t)(row0 + (int)order[b - 1 - (base + min(j, R - 1))]) * d);
          xr0[j] = (j < R && on0) ? __ldg(xrow + lane) : z4;
          xr1[j] = (j < R && on1) ? __ldg(xrow + 32 + lane) : z4;
        }
        float bd1 = INF, bd2 = INF, bd3 = INF;                 // first lane of a pair's run: row j over the centres of slot c of this warp
        int bi1 = 0x7fffffff, bi2 = 0x7fffffff;
        const int c_mine = (lane / LPR) / RB;                  // the centre slot of the pair this lane ends up with
        // the warp's centres are wid, wid + 8, ...; an iteration takes CB of them, slot c the centre a + 8 c
        float4 w0v[CB], w1v[CB];
#pragma unroll
        for (int c = 0; c < CB; ++c) {
          const float4* wa = reinterpret_cast<const float4*>(wglob + (size_t)min(wid + NW * c, k - 1) * d);
          w0v[c] = on0 ? wa[lane] : z4;
          w1v[c] = on1 ? wa[32 + lane] : z4;
        }
        for (int a = wid; a < k; a += NW * CB) {         // ascending inside a slot: a strict "<" keeps the lowest index of a tie
          float4 n0[CB], n1[CB];                               // the next iteration's rows of the state
#pragma unroll
          for (int c = 0; c < CB; ++c) {
            const float4* wn = reinterpret_cast<const float4*>(wglob + (size_t)min(a + NW * (CB + c), k - 1) * d);
            n0[c] = on0 ? wn[lane] : z4;
            n1[c] = on1 ? wn[32 + lane] : z4;
          }
          float part[VR];
#pragma unroll
          for (int c = 0; c < CB; ++c)
#pragma unroll
            for (int j = 0; j < RB; ++j) {
              const float4 x0 = xr0[j], x1 = xr1[j];
              float s0 = 0.f, s1 = 0.f, e;
              e = x0.x - w0v[c].x; s0 = fmaf(e, e, s0); e = x0.y - w0v[c].y; s1 = fmaf(e, e, s1);
              e = x0.z - w0v[c].z; s0 = fmaf(e, e, s0); e = x0.w - w0v[c].w; s1 = fmaf(e, e, s1);
              if (kWide) {
                e = x1.x - w1v[c].x; s0 = fmaf(e, e, s0); e = x1.y - w1v[c].y; s1 = fmaf(e, e, s1);
                e = x1.z - w1v[c].z; s0 = fmaf(e, e, s0); e = x1.w - w1v[c].w; s1 = fmaf(e, e, s1);
              }
              part[c * RB + j] = s0 + s1;
            }
          // halving exchange: at offset o the lanes with that bit clear keep the lower half of the pairs still held
#pragma unroll
          for (int o = 16, n = VR / 2; n >= 1; o >>= 1, n >>= 1) {
            const bool up = (lane & o) != 0;
#pragma unroll
            for (int j = 0; j < n; ++j) {
              const float send = up ? part[j] : part[j + n];
              const float keep = up ? part[j + n] : part[j];
              part[j] = keep + __shfl_xor_sync(0xffffffffu, send, o);
            }
          }
          float tot = part[0];                                  // lanes LPR * v .. : pair v, each with a share of it
#pragma unroll
          for (int o = LPR / 2; o >= 1; o >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, o);
          const int a_mine = a + NW * c_mine;
          if ((lane & (LPR - 1)) == 0 && a_mine < k) {
            if (tot < bd1) { bd3 = bd2; bd2 = bd1; bi2 = bi1; bd1 = tot; bi1 = a_mine; }
            else if (tot < bd2) { bd3 = bd2; bd2 = tot; bi2 = a_mine; }
            else if (tot < bd3) { bd3 = tot; }
          }
#pragma unroll
          for (int c = 0; c < CB; ++c) { w0v[c] = n0[c]; w1v[c] = n1[c]; }
        }
        if ((lane & (LPR - 1)) == 0) {
          const int v = lane / LPR;
          float* o = res + (wid * VR + v) * 5;
          o[0] = bd1; o[1] = bd2; o[2] = bd3; o[3] = __int_as_float(bi1); o[4] = __int_as_float(bi2);
        }
        __syncthreads();
        if (tid < RB) {
          // the warps' shares merged: three smallest distances, the first two with their centres (equal distances: lowest index first)
          float fd1 = INF, fd2 = INF, fd3 = INF;
          int fi1 = 0x7fffffff, fi2 = 0x7fffffff;
          auto put = [&](float v, int idx) {
            if (v < fd1 || (v == fd1 && idx < fi1)) { fd3 = fd2; fd2 = fd1; fi2 = fi1; fd1 = v; fi1 = idx; }
            else if (v < fd2 || (v == fd2 && idx < fi2)) { fd3 = fd2; fd2 = v; fi2 = idx; }
            else if (v < fd3) { fd3 = v; }
          };
          for (int q = 0; q < NW * CB; ++q) {                   // every warp's every centre slot
            const float* o = res + (q * RB + tid) * 5;
            put(o[0], __float_as_int(o[3]));
            put(o[1], __float_as_int(o[4]));
            put(o[2], 0x7fffffff);
          }
          // fp32 distances are off by at most (d + 2) u relative: a gap above (4 d + 16) u of the larger one decides
          const float tol = (float)(4 * TC_MAX_D + 16) * 5.9604645e-8f;
          int how = 0;
          if (tid < R && fd2 - fd1 <= tol * fd2) how = (fd3 - fd1 <= tol * fd3) ? 2 : 1;
          need64[tid * 3 + 0] = how;
          need64[tid * 3 + 1] = fi1;
          need64[tid * 3 + 2] = fi2;
          if (tid < R && how == 0) best[order[b - 1 - (base + tid)]] = (unsigned short)fi1;
        }
        __syncthreads();
        for (int j = wid; j < R; j += NW) {                    // warp-uniform: need64[j] is the same for every lane
          const int how = need64[j * 3 + 0];
          if (how == 0) continue;
          const float4* xrow = reinterpret_cast<const float4*>(p.X + (size_t)(row0 + (int)order[b - 1 - (base + j)]) * d);
          const float4 x0 = on0 ? __ldg(xrow + lane) : z4;
          const float4 x1 = on1 ? __ldg(xrow + 32 + lane) : z4;
          auto dist64 = [&](int a) {                           // fp64 squared distance to centre a (the same value in every lane)
            const float4* wr = reinterpret_cast<const float4*>(wglob + (size_t)a * d);
            const float4 u0 = on0 ? wr[lane] : z4;
            const float4 u1 = on1 ? wr[32 + lane] : z4;
            double sacc = 0.0, e;
            e = (double)x0.x - (double)u0.x; sacc = fma(e, e, sacc); e = (double)x0.y - (double)u0.y; sacc = fma(e, e, sacc);
            e = (double)x0.z - (double)u0.z; sacc = fma(e, e, sacc); e = (double)x0.w - (double)u0.w; sacc = fma(e, e, sacc);
            if (kWide) {
              e = (double)x1.x - (double)u1.x; sacc = fma(e, e, sacc); e = (double)x1.y - (double)u1.y; sacc = fma(e, e, sacc);
              e = (double)x1.z - (double)u1.z; sacc = fma(e, e, sacc); e = (double)x1.w - (double)u1.w; sacc = fma(e, e, sacc);
            }
#pragma unroll
            for (int sh = 16; sh > 0; sh >>= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, sh);
            return sacc;
          };
          int bi;
          if (how == 1) {                                      // two candidates: the closer one, the lower index on a tie
            const int i1 = need64[j * 3 + 1], i2 = need64[j * 3 + 2];
            const double e1 = dist64(i1), e2 = dist64(i2);
            bi = (e2 < e1 || (e2 == e1 && i2 < i1)) ? i2 : i1;
          } else {                                             // three or more within rounding: every centre once more
            double bd = 1e300;
            bi = 0;
            for (int a = 0; a < k; ++a) {
              const double e1 = dist64(a);
              if (e1 < bd) { bd = e1; bi = a; }                  // ascending a: the lowest index keeps a tie
            }
          }
          if (lane == 0) best[order[b - 1 - (base + j)]] = (unsigned short)bi;
        }
        __syncthreads();                                       // before the next batch overwrites the results
      };
      int base = 0;                                            // block-uniform trip counts
      for (; nwide - base > 4; base += TC_SCAN_ROWS)
        scan_batch(std::integral_constant<int, TC_SCAN_ROWS>(), std::integral_constant<int, 1>(), base, min(TC_SCAN_ROWS, nwide - base));
      if (base < nwide) scan_batch(std::integral_constant<int, 4>(), std::integral_constant<int, 4>(), base, nwide - base);
    }
    __syncthreads();
    if (p.assign_rec)
      for (int r = tid; r < b; r += NT) p.assign_rec[(size_t)i * b + r] = best[r];

    // ---- rows grouped by centre, in row order (stable): ranks inside each warp's block of rows, then offsets ----
    {
      const int R = ((b + GW - 1) / GW + 31) / 32 * 32;                       // rows per block of rows, whole chunks of 32
      int* mine = wcnt + min(wid, GW - 1) * k;
      for (int r0 = wid * R; wid < GW && r0 < min(b, (wid + 1) * R); r0 += 32) {
        const int r = r0 + lane;
        const int a = (r < b) ? (int)best[r] : -1;
        const unsigned grp = __match_any_sync(0xffffffffu, a);
        const unsigned below = grp & ((1u << lane) - 1u);
        const int lead = __ffs(grp) - 1;
        int base = 0;
        if (a >= 0 && below == 0) { base = mine[a]; mine[a] = base + __popc(grp); }
        base = __shfl_sync(0xffffffffu, base, lead);
        if (a >= 0) lrank[r] = (unsigned short)(base + __popc(below));
        __syncwarp();
      }
    }
    __syncthreads();
    // per centre: total count, then start = exclusive prefix over centres (block scan of k <= 1024 values)
    {
      int tot[4], run = 0;
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int a = tid * 4 + u;
        int c = 0;
        if (a < k)
          for (int w8 = 0; w8 < GW; ++w8) { const int v = wcnt[w8 * k + a]; wcnt[w8 * k + a] = c; c += v; }   // per-block offsets
        tot[u] = c;
        run += c;
      }
      int incl = run;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) { const int y = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += y; }
      int* wsum = reinterpret_cast<int*>(ts->red);
      if (lane == 31) wsum[wid] = incl;
      __syncthreads();
      int before = incl - run;
      for (int w8 = 0; w8 < wid; ++w8) before += wsum[w8];
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int a = tid * 4 + u;
        if (a < k) { cnt[a] = tot[u]; reinterpret_cast<int*>(sB)[a] = before; }      // start[a] (the centre block is idle too)
        before += tot[u];
      }
    }
    __syncthreads();
    {
      const int* start = reinterpret_cast<const int*>(sB);
      const int R = ((b + GW - 1) / GW + 31) / 32 * 32;
      for (int r = tid; r < b; r += NT) {
        const int a = best[r];
        order[start[a] + wcnt[(r / R) * k + a] + lrank[r]] = (unsigned short)r;
      }
    }
    if (tid == 0) {                                       // one thread looks, so that the whole block takes the same branch
      int any = 0;
      for (int s = 0; s < p.S; ++s) any |= (ld_relaxed_gpu(p.seq + (size_t)i * p.S + s) != p.seen[(size_t)i * p.S + s]);
      misc[4] = any;
    }
    __syncthreads();
    const bool put_now = p.c > 0 && p.f > 0 && p.W > 1 && (t + 1) % (unsigned long long)p.c == 0;
    const bool plain = (misc[4] == 0);                    // no message waiting: the fused update below, then the send if one is due

    // ---- Eq. 9 and the update: eight lanes per centre add its rows (fp32 master, ascending row order);
    //      plain step: w <- w - eps (n w - S) / b at once; otherwise S goes to the sum buffer for the general tail.
    //      The 32 eight-lane groups of the block work through the centres independently: a group takes a few rows of
    //      its centre per turn, and when the centre is done it finishes it and draws the next centre from a counter, so
    //      that a group with a large centre does not hold up the three it shares a warp with (all lanes run the same
    //      instructions; what a group does not need is predicated off) ----
    {
      const int* start = reinterpret_cast<const int*>(sB);
      const float4 z4 = make_float4(0.f, 0.f, 0.f, 0.f);
      const unsigned long long pol_x = l2_policy_evict_first();
      auto sum_and_update = [&](auto rows_tag, auto qmax_tag) {
        constexpr int ROWS = decltype(rows_tag)::value, QMAX = decltype(qmax_tag)::value;   // rows per turn, float4 pieces per lane (nq <= QMAX)
        int a = wid * 4 + sub;                                 // the group's centre; the next ones come from the counter
        int n = (a < k) ? cnt[a] : 0, p0 = (a < k) ? start[a] : 0, e = 0;
        float4 S4[QMAX];
#pragma unroll
        for (int q = 0; q < QMAX; ++q) S4[q] = z4;
        while (__any_sync(0xffffffffu, a < k)) {
          const bool live = a < k;
          // a centre that ends with this turn's rows: its row of the state is asked for together with them
          const bool moves = plain && live && n > 0 && e + ROWS >= n;                 // (an empty centre stays where it is)
          float4 w4[QMAX];
#pragma unroll
          for (int q = 0; q < QMAX; ++q)
            w4[q] = (q < nq && moves) ? *reinterpret_cast<const float4*>(wglob + (size_t)a * d + 4 * l8 + 32 * q) : z4;
          {
            float4 v[ROWS][QMAX];
#pragma unroll
            for (int u = 0; u < ROWS; ++u) {
              const bool have = live && e + u < n;
              const float* x = p.X + (size_t)(row0 + (have ? (int)order[p0 + e + u] : 0)) * d + 4 * l8;
#pragma unroll
              for (int q = 0; q < QMAX; ++q) v[u][q] = (q < nq && have) ? ldg_stream4(reinterpret_cast<const float4*>(x + 32 * q), pol_x) : z4;
            }
#pragma unroll
            for (int u = 0; u < ROWS; ++u)
#pragma unroll
              for (int q = 0; q < QMAX; ++q) { S4[q].x += v[u][q].x; S4[q].y += v[u][q].y; S4[q].z += v[u][q].z; S4[q].w += v[u][q].w; }
          }
          e += ROWS;
          const bool done = live && e >= n;
          if (__any_sync(0xffffffffu, done)) {
            float sq = 0.f;
            if (plain) {
              const float fn = (float)n;
#pragma unroll
              for (int q = 0; q < QMAX; ++q) {
                if (q < nq && moves) {
                  float4 u = w4[q];
                  u.x -= p.eps * ((fn * u.x - S4[q].x) * inv_b); u.y -= p.eps * ((fn * u.y - S4[q].y) * inv_b);
                  u.z -= p.eps * ((fn * u.z - S4[q].z) * inv_b); u.w -= p.eps * ((fn * u.w - S4[q].w) * inv_b);
                  const size_t o = (size_t)a * d + 4 * l8 + 32 * q;
                  *reinterpret_cast<float4*>(wglob + o) = u;
                  sq += put16(o, u);
                }
              }
#pragma unroll
              for (int o = 1; o < 8; o <<= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
              if (moves && l8 == 0) cn[a] = sq;
            } else if (done) {
#pragma unroll
              for (int q = 0; q < QMAX; ++q)
                if (q < nq) *reinterpret_cast<float4*>(gsum + (size_t)a * d + 4 * l8 + 32 * q) = S4[q];
            }
            int nxt = 0;
            if (done && l8 == 0) nxt = atomicAdd(&misc[7], 1);
            nxt = __shfl_sync(0xffffffffu, nxt, lane & ~7);
            if (done) {
              a = nxt;
              e = 0;
              n = (a < k) ? cnt[a] : 0;
              p0 = (a < k) ? start[a] : 0;
#pragma unroll
              for (int q = 0; q < QMAX; ++q) S4[q] = z4;
            }
          }
        }
      };
      if (nq <= QN / 2) sum_and_update(std::integral_constant<int, 8>(), std::integral_constant<int, QN / 2>());
      else sum_and_update(std::integral_constant<int, 4>(), std::integral_constant<int, QN>());
    }
    if (!plain) {
      __syncthreads();
      step_tail<kDet>(p, i, t, wglob, d, gsum, cnt, nullptr, ts, false);
      __syncthreads();
      refresh_all();
    } else {
      unsigned long long n_sent = 0;
      if (put_now) {
        __syncthreads();                                  // every centre's new w is in place
        n_sent = step_send_any<kDet>(p, i, t, wglob, d, ts);
      }
      if (kDet && p.rows_m > 0)                            // per-row record of a step that looked at no message
        for (int a = tid; a < p.k; a += NT) p.rowin[(size_t)i * p.k + a] = 0;
      if (tid == 0) {
        if (kDet)
          for (int s = 0; s < p.S; ++s) p.accept_rec[(size_t)i * p.S + s] = -1;
        unsigned long long* st = p.stats + (size_t)i * ST_STRIDE;
        st[ST_STEPS] = t + 1;
        if (n_sent) atomicAdd(st + ST_SENT, n_sent);
      }
    }
    asm volatile("fence.proxy.async;" ::: "memory");      // the refreshed w_hi, w_lo are read by the next step's TMA
    __syncthreads();
  }

  if (misc[2] && tid == 0) {
    atomicExch(p.status, DEV_TIMEOUT);
    // copies may still be on their way into this block's shared memory: give each a bounded chance to land
    for (int q = 0; q < 2 * TC_B_STAGES; ++q) { mbar_wait_bounded(bars + TCB_BFULL + q, 0, p.wait_limit); mbar_wait_bounded(bars + TCB_BFULL + q, 1, p.wait_limit); }
    for (int q = 0; q < TC_A_STAGES; ++q) { mbar_wait_bounded(bars + TCB_AFULL + q, 0, p.wait_limit); mbar_wait_bounded(bars + TCB_AFULL + q, 1, p.wait_limit); }
  }
  tc_fence_before();
  __syncthreads();
  if (wid == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"((unsigned)TC_TMEM_COLS) : "memory");
}

}  // namespace asgd
