// Shared device-side definitions of the K-Means ASGD library: launch parameters, the schedule
// hash, memory-ordering helpers and block-level primitives.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

namespace asgd {

// Per-worker counters, one row of 8 x u64 per worker.
enum { ST_STEPS = 0, ST_SENT = 1, ST_RECV = 2, ST_ACCEPT = 3, ST_OVERWRITTEN = 4, ST_STRIDE = 8 };

// Device status word values (index 0 of Params::status); 0 = fine.
enum { DEV_OK = 0, DEV_TIMEOUT = 1 };

struct Params {
  const float* X;          // [N][d] samples (borrowed)
  long long N;
  int d, k, W, b;
  float eps;
  int c, f, S, parzen;
  unsigned long long seed;
  long long H, B;          // shard rows, batches per pass
  int kd, kd_pad;          // k*d and k*d rounded up to a multiple of 4 floats
  float* state;            // [W][kd_pad]     worker states (Algorithm 5: w^i)
  float* mail;             // [W][S][kd_pad]  receive buffers (Eq. 3: the N external buffers)
  unsigned* seq;           // [W][S]  messages ever written into the buffer (written by senders)
  unsigned* seen;          // [W][S]  value of seq at the owner's last look (owner only)
  unsigned* arb_win;       // [W][S]  deterministic delivery: 1 + (sender*f + j) of the last sender
  unsigned* arb_cnt;       // [W][S]  deterministic delivery: messages aimed at the buffer this round
  unsigned long long* stats;  // [W][ST_STRIDE]
  const int* perm;         // [W][B] batch order
  int* status;             // [4] device status word
  int* assign_rec;         // [W][b] or nullptr
  int* accept_rec;         // [W][S] acceptance of the last step
  float* gsum;             // [W][kd_pad] per-worker sums when the state does not fit on chip
  float xmax2;             // max_i ||x_i||^2 over X (error bound of the tensor-core path)
  void* wbf;               // [2][W][k][d] BF16 terms of -2w: w_hi, then w_lo (tensor-core path)
  float* top2;             // [W][b][4] the three smallest packed squared distances of every row (tensor-core path)
  const float* xnorm;      // [N] ||x_i||^2 (tensor-core path)
  int rows_m;              // per-centre messages (Section 4.4): centre rows per message, 0 = whole-state messages
  int2* mail_rows;         // [W][S] (first row, number of rows) of the buffer's last message (per-centre mode)
  unsigned* rowacc;        // [W][k] bit s: row accepted from buffer s in the worker's last step (per-centre mode)
  unsigned* rowin;         // [W][k] bit s: buffer s held a new message carrying the row
  unsigned wait_limit;     // iterations of try_wait after which a wait on one of the block's own copies is given up
  long long withhold_step; // failure drill: the first sample copy of this step of a launch is announced but not issued (-1 = never)
};

// ---------------------------------------------------------------------------------------------
// Schedule random numbers: SplitMix64 output function chained over (seed^tag, a, b, c).
// ---------------------------------------------------------------------------------------------
__host__ __device__ inline unsigned long long splitmix_first(unsigned long long x) {
  unsigned long long z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
enum : unsigned long long { TAG_PERM = 1, TAG_PEER = 2, TAG_SLOT = 3, TAG_ROWS = 4 };
__host__ __device__ inline unsigned long long sched_draw(unsigned long long seed, unsigned long long tag,
                                                         unsigned long long a, unsigned long long b,
                                                         unsigned long long c) {
  unsigned long long h = splitmix_first(seed ^ tag);
  h = splitmix_first(h + a);
  h = splitmix_first(h + b);
  return splitmix_first(h + c);
}

// j-th recipient of worker i's put after step t, given the earlier recipients prev[0..j).
__device__ inline int sched_peer(const Params& p, int i, unsigned long long t, int j, const int* prev) {
  int q = (int)(sched_draw(p.seed, TAG_PEER, (unsigned long long)i, t, (unsigned long long)j) %
                (unsigned long long)(p.W - 1));
  if (q >= i) q += 1;
  for (int guard = 0; guard <= p.W; ++guard) {
    bool dup = (q == i);
    for (int r = 0; r < j && !dup; ++r) dup = (prev[r] == q);
    if (!dup) break;
    q = (q + 1 == p.W) ? 0 : q + 1;
  }
  return q;
}
__device__ inline int sched_slot(const Params& p, int i, unsigned long long t, int j) {
  return (int)(sched_draw(p.seed, TAG_SLOT, (unsigned long long)i, t, (unsigned long long)j) %
               (unsigned long long)p.S);
}
// Per-centre messages: first of the rows_m consecutive (cyclic) centre rows of the j-th message.
__device__ inline int sched_first_row(const Params& p, int i, unsigned long long t, int j) {
  return (int)(sched_draw(p.seed, TAG_ROWS, (unsigned long long)i, t, (unsigned long long)j) %
               (unsigned long long)p.k);
}
// Is row a among the m rows that start (cyclically) at r0?
__device__ inline bool row_in_run(int a, int r0, int m, int k) {
  int off = a - r0;
  if (off < 0) off += k;
  return off < m;
}

// ---------------------------------------------------------------------------------------------
// Memory ordering for the single-sided put: payload stores, then a release-increment of the
// buffer's sequence number; the owner reads it with acquire and the payload past L1.
// ---------------------------------------------------------------------------------------------
__device__ inline unsigned ld_acquire_gpu(const unsigned* p) {
  unsigned v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ inline void red_release_gpu_inc(unsigned* p) {
  asm volatile("red.release.gpu.global.add.u32 [%0], 1;" ::"l"(p) : "memory");
}

// ---------------------------------------------------------------------------------------------
// Block reductions with a fixed order (so results do not depend on scheduling).
// ---------------------------------------------------------------------------------------------
__device__ inline double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
// Sums three doubles over the block; every thread gets the result.  scratch: >= 3*32 doubles.
__device__ inline void block_sum3(double& a, double& b, double& c, double* scratch) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  a = warp_sum(a); b = warp_sum(b); c = warp_sum(c);
  __syncthreads();
  if (lane == 0) { scratch[wid] = a; scratch[32 + wid] = b; scratch[64 + wid] = c; }
  __syncthreads();
  double x = 0, y = 0, z = 0;
  for (int w = 0; w < nw; ++w) { x += scratch[w]; y += scratch[32 + w]; z += scratch[64 + w]; }
  a = x; b = y; c = z;
}

// Stable counting sort of the mini-batch by assigned centre.  assign[b] -> order[b] (sample
// indices grouped by centre, ascending inside a group) and start[k+1] (group boundaries).
// Warps take centres round-robin and sweep the batch with ballots, so the result is exact and
// independent of timing.  Needs a preceding prefix of the counts in start[] (see caller).
__device__ inline void block_group_by_centre(const int* assign, int b, int k, const int* start, int* order) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
  for (int a = wid; a < k; a += nw) {
    int base = start[a];
    if (start[a + 1] == base) continue;
    for (int s0 = 0; s0 < b; s0 += 32) {
      const int s = s0 + lane;
      const bool mine = (s < b) && (assign[s] == a);
      const unsigned m = __ballot_sync(0xffffffffu, mine);
      if (mine) order[base + __popc(m & ((1u << lane) - 1u))] = s;
      base += __popc(m);
    }
  }
}

}  // namespace asgd
