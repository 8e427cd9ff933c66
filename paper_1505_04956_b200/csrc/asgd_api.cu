// C ABI of the K-Means ASGD library: context, argument checks, workspace layout, launches.
// Declarations and argument contracts are in include/asgd.h.

#include "../../include/asgd.h"

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "asgd_aux.cuh"
#include "asgd_generic.cuh"
#include "asgd_stream.cuh"
#include "asgd_tiled.cuh"
#include "asgd_tc.cuh"

#include <cudaTypedefs.h>

using namespace asgd;

namespace {

enum PathId { P_GENERIC = 0, P_STREAM = 1, P_TILED = 2, P_TC_BF16 = 3, P_TC_FP16 = 4 };

// (d, k) shapes the streaming path is compiled for
#define ASGD_STREAM_SHAPES(X) X(10, 10) X(16, 16) X(4, 5) X(2, 3)

// (d, padded k, warps along samples, warps along centres, blocks per SM) the tiled path is compiled for.
// Among the shapes with the same d and enough centres the one that keeps the most threads busy for the given
// number of workers is taken (small blocks when there are enough workers to fill the GPU with them: a block that
// serves one worker keeps its state on chip between steps); ties go to the later entry.
#define ASGD_TILED_SHAPES(X) X(32, 64, 8, 2, 1) X(32, 64, 4, 2, 2) X(32, 64, 2, 2, 4) X(128, 128, 4, 4, 1)

struct Layout {
  size_t state, mail, seq, seen, arb_win, arb_cnt, mail_rows, rowacc, rowin, stats, perm, status, assign_rec, accept_rec, gsum,
      eval_partial, tmp_state, xmax, wbf, top2, xbf, xbl, xnorm, total;
};

constexpr size_t kAlign = 256;
constexpr int kEvalBlocks = 148 * 8;
constexpr size_t kMaxDynSmem = 227 * 1024;
constexpr size_t kTwoBlockSmem = 113 * 1024;      // two blocks, each with its reserved kilobyte, in an SM's 228 KB

inline size_t up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

bool config_ok(const asgd_config* c) {
  if (!c) return false;
  if (c->N <= 0 || c->d <= 0 || c->k <= 0 || c->W <= 0 || c->b <= 0) return false;
  if (!(c->eps > 0.f)) return false;
  if (c->comm_interval < 0 || c->fanout < 0 || c->fanout > c->W - 1 || c->fanout > MAX_FANOUT) return false;
  if (c->slots < 1 || c->slots > MAX_SLOTS) return false;
  if (c->partial_rows < 0 || c->partial_rows > c->k) return false;
  if (c->dist_path < ASGD_PATH_AUTO || c->dist_path > ASGD_PATH_FP32_GENERAL) return false;
  if ((long long)c->k * c->d > (1ll << 28)) return false;
  const long long H = c->N / c->W;
  if (H < c->b) return false;
  if ((long long)c->W * c->fanout + 1 > 0x7fffffffll) return false;
  return true;
}

// shapes the tensor-core path can take: d a multiple of 64 up to 256, a batch of at least one 128-row tile
bool tc_supported(const asgd_config* c) {
  return c->d % TC_KC == 0 && c->d <= TC_MAX_D && c->k >= 1 && c->k <= TC_MAX_K && c->b >= TC_M && c->b <= TC_MAX_B &&
         tc_smem_bytes(c->k, c->d, c->b, 1, 1, TC_THREADS_MID) <= kMaxDynSmem && tc_smem_bytes(c->k, c->d, c->b, 3, 1, TC_THREADS_MID) <= kMaxDynSmem;
}
// ... and these are the library's own choice for them
bool tc_eligible(const asgd_config* c) { return tc_supported(c); }
// the path a configuration asks for is a tensor-core one
bool tc_wanted(const asgd_config* c) {
  if (c->dist_path == ASGD_PATH_TC_BF16 || c->dist_path == ASGD_PATH_TC_FP16) return tc_supported(c);
  return c->dist_path == ASGD_PATH_AUTO && tc_eligible(c);
}

Layout make_layout(const asgd_config* c) {
  Layout L{};
  const size_t W = c->W, S = c->slots;
  const size_t kd = (size_t)c->k * c->d, kd_pad = (kd + 3) / 4 * 4;
  const size_t H = c->N / c->W, B = H / c->b;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off += up(bytes); return o; };
  L.state = take(W * kd_pad * 4);
  L.mail = take(W * S * kd_pad * 4);
  L.seq = take(W * S * 4);
  L.seen = take(W * S * 4);
  L.arb_win = take(W * S * 4);
  L.arb_cnt = take(W * S * 4);
  L.mail_rows = take(W * S * 8);
  L.rowacc = take(c->partial_rows > 0 ? W * (size_t)c->k * 4 : 4);
  L.rowin = take(c->partial_rows > 0 ? W * (size_t)c->k * 4 : 4);
  L.stats = take(W * ST_STRIDE * 8);
  L.perm = take(W * B * 4);
  L.status = take(64);
  L.assign_rec = take(c->record_assign ? W * (size_t)c->b * 4 : 4);
  L.accept_rec = take(W * S * 4);
  L.gsum = take(W * kd_pad * 4);
  L.eval_partial = take((size_t)kEvalBlocks * 8);
  L.tmp_state = take(kd_pad * 4);
  L.xmax = take(64);
  // tensor-core path: 16-bit copies of -2w and of the samples (one FP16 term, or the two BF16 terms), the three
  // best per row, the row norms
  const bool tc = tc_wanted(c);
  const bool two_terms = tc && c->dist_path == ASGD_PATH_TC_BF16;
  L.wbf = take(tc ? (two_terms ? 2 : 1) * W * kd * 2 : 4);
  L.top2 = take(tc ? W * (size_t)c->b * 16 : 4);
  L.xbf = take(tc ? (size_t)c->N * c->d * 2 : 4);
  L.xbl = take(two_terms ? (size_t)c->N * c->d * 2 : 4);
  L.xnorm = take(tc ? (size_t)c->N * 4 : 4);
  L.total = off;
  return L;
}

}  // namespace

struct asgd_ctx {
  asgd_config cfg;
  Params p;
  Layout L;
  unsigned char* ws;
  cudaStream_t stream;
  int path;
  int state_on_chip;
  int grid;               // blocks of the worker kernel (tiled path: a block may serve several workers)
  int tiled_shape;        // index into ASGD_TILED_SHAPES of the shape in use
  int tc_inst;            // tensor-core path: 0 = 384 threads, one block per SM; 1 = 256 threads, two blocks share an SM; 2 = 512 threads
  size_t smem_bytes;
  long long t_host;       // steps every worker has done (uniform across workers)
  long long launches;
  int last_cuda;
  int sm_count;
  const void* xbf_user;   // caller's bf16 copy of X, or nullptr
  int no_tc;              // AUTO: the samples do not fit FP16, take an fp32 path
  CUtensorMap mapXh, mapXl, mapW; // tensor-core path: BF16 terms of the samples [N][d] each, of -2w [2*W*k][d]
};

namespace {

int cuda_fail(asgd_ctx* c, cudaError_t e) {
  if (c) c->last_cuda = (int)e;
  return ASGD_ECUDA;
}
#define CU(ctx, call)                                   \
  do {                                                  \
    cudaError_t e_ = (call);                            \
    if (e_ != cudaSuccess) return cuda_fail((ctx), e_); \
  } while (0)

// Batch order of one worker: Fisher-Yates from the top, driven by the schedule hash.
void fill_perm(const asgd_config& c, long long B, int worker, int* perm) {
  for (long long q = 0; q < B; ++q) perm[q] = (int)q;
  if (!c.shuffle) return;
  for (long long q = B - 1; q >= 1; --q) {
    const unsigned long long r =
        sched_draw(c.seed, TAG_PERM, (unsigned long long)worker, (unsigned long long)q, 0ull) % (unsigned long long)(q + 1);
    std::swap(perm[q], perm[r]);
  }
}

template <int D, int K>
int stream_prepare(asgd_ctx* c) {
  c->smem_bytes = stream_smem_bytes<D, K>(c->cfg.b);
  CU(c, cudaFuncSetAttribute(asgd_stream_kernel<D, K, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->smem_bytes));
  CU(c, cudaFuncSetAttribute(asgd_stream_kernel<D, K, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->smem_bytes));
  return ASGD_OK;
}
template <int D, int K>
void stream_launch(asgd_ctx* c, bool det, long long steps) {
  if (det)
    asgd_stream_kernel<D, K, true><<<c->p.W, STREAM_THREADS, c->smem_bytes, c->stream>>>(c->p, steps);
  else
    asgd_stream_kernel<D, K, false><<<c->p.W, STREAM_THREADS, c->smem_bytes, c->stream>>>(c->p, steps);
}

template <int D, int KP, int WS, int WK, int MINB>
int tiled_prepare(asgd_ctx* c, long long* busy_threads) {
  c->smem_bytes = tiled_smem_bytes<D, KP, WS, WK>(c->cfg.k);
  CU(c, cudaFuncSetAttribute(asgd_tiled_kernel<D, KP, WS, WK, MINB, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->smem_bytes));
  CU(c, cudaFuncSetAttribute(asgd_tiled_kernel<D, KP, WS, WK, MINB, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->smem_bytes));
  int per_sm = 0;
  CU(c, cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, asgd_tiled_kernel<D, KP, WS, WK, MINB, false>, 32 * WS * WK, c->smem_bytes));
  if (per_sm < 1) return ASGD_EUNSUPPORTED;
  const int resident = per_sm * c->sm_count;
  const int V = (c->cfg.W + resident - 1) / resident;          // workers per block, served in turn
  if (V > TILED_MAX_V) return ASGD_EUNSUPPORTED;
  c->grid = (c->cfg.W + V - 1) / V;
  *busy_threads = (long long)(c->grid < resident ? c->grid : resident) * (32 * WS * WK);
  return ASGD_OK;
}
template <int D, int KP, int WS, int WK, int MINB>
void tiled_launch(asgd_ctx* c, bool det, long long steps) {
  if (det)
    asgd_tiled_kernel<D, KP, WS, WK, MINB, true><<<c->grid, 32 * WS * WK, c->smem_bytes, c->stream>>>(c->p, steps);
  else
    asgd_tiled_kernel<D, KP, WS, WK, MINB, false><<<c->grid, 32 * WS * WK, c->smem_bytes, c->stream>>>(c->p, steps);
}

bool encode_16bit_map(CUtensorMap* map, bool fp16, const void* base, unsigned long long rows, unsigned long long cols, unsigned box_rows) {
  static PFN_cuTensorMapEncodeTiled encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || !fn) return false;
    encode = (PFN_cuTensorMapEncodeTiled)fn;
  }
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)TC_KC, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return encode(map, fp16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor-core path set-up: bf16 copy of X (unless the caller brought one), max ||x||^2, tensor maps.
// max_i ||x_i||^2 into Params::xmax2 (one pass over the samples at initialisation): the rounding bounds of the
// streaming, tiled and tensor-core paths use it.
int compute_xmax2(asgd_ctx* c) {
  Params& p = c->p;
  unsigned* xm = (unsigned*)(c->ws + c->L.xmax);
  CU(c, cudaMemsetAsync(xm, 0, 4, c->stream));
  xmax2_kernel<<<c->sm_count * 8, 256, 0, c->stream>>>(p.X, p.N, p.d, xm);
  c->launches += 1;
  CU(c, cudaGetLastError());
  float xmax2 = 0.f;
  CU(c, cudaMemcpyAsync(&xmax2, xm, 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  p.xmax2 = xmax2;
  return ASGD_OK;
}

// Tensor-core path set-up: 16-bit copies of X, row norms, max ||x||^2, tensor maps.  Returns ASGD_EUNSUPPORTED when
// the one-term FP16 format was asked for and the samples do not fit FP16's range.
int tc_prepare(asgd_ctx* c) {
  const asgd_config& cfg = c->cfg;
  Params& p = c->p;
  const bool fp16 = (c->path == P_TC_FP16);
  const int terms = fp16 ? 1 : 3;
  const int bn = tc_block_rows(cfg.k, terms);
  // Three instances.  Two blocks of 256 threads per SM when there are more workers than SMs, rows of at most 128
  // numbers, accumulators of at most 256 tensor-memory columns a block, and room for two blocks' shared memory.  Else,
  // for rows of at most 128 numbers, one block of 512 threads per SM if its shared memory fits.  Else one block of 384
  // threads.  The request is padded so that no more blocks than meant share an SM (tensor memory has 512
  // columns).
  {
    const int grid2 = std::min(cfg.W, 2 * c->sm_count);
    const size_t smem2 = tc_smem_bytes(cfg.k, cfg.d, cfg.b, terms, (cfg.W + grid2 - 1) / grid2, TC_THREADS);
    c->grid = std::min(cfg.W, c->sm_count);
    const int nv1 = (cfg.W + c->grid - 1) / c->grid;
    const size_t smem_wide = tc_smem_bytes(cfg.k, cfg.d, cfg.b, terms, nv1, TC_THREADS_WIDE);
    c->tc_inst = 0;
    if (cfg.W > c->sm_count && cfg.d <= 128 && tc_tmem_cols(bn) <= 256 && smem2 <= kTwoBlockSmem) {
      c->tc_inst = 1;
      c->grid = grid2;
      c->smem_bytes = std::max(smem2, (size_t)(kMaxDynSmem / 3 + 1024));
    } else if (cfg.d <= 128 && smem_wide <= kMaxDynSmem) {
      c->tc_inst = 2;
      c->smem_bytes = std::max(smem_wide, (size_t)(kMaxDynSmem / 2 + 1024));
    } else {
      c->smem_bytes = std::max(tc_smem_bytes(cfg.k, cfg.d, cfg.b, terms, nv1, TC_THREADS_MID), (size_t)(kMaxDynSmem / 2 + 1024));
      if (c->smem_bytes > kMaxDynSmem) return ASGD_EUNSUPPORTED;
    }
  }
#define TC_SET(DET_, T_, D_, NT_) CU(c, cudaFuncSetAttribute(asgd_tc_kernel<DET_, T_, D_, NT_>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->smem_bytes))
#define TC_SET_BOTH(T_, D_, NT_) { TC_SET(true, T_, D_, NT_); TC_SET(false, T_, D_, NT_); }
  if (fp16) {
    if (c->tc_inst == 1) TC_SET_BOTH(1, 128, TC_THREADS) else if (c->tc_inst == 2) TC_SET_BOTH(1, 128, TC_THREADS_WIDE) else TC_SET_BOTH(1, 256, TC_THREADS_MID)
  } else {
    if (c->tc_inst == 1) TC_SET_BOTH(3, 128, TC_THREADS) else if (c->tc_inst == 2) TC_SET_BOTH(3, 128, TC_THREADS_WIDE) else TC_SET_BOTH(3, 256, TC_THREADS_MID)
  }
#undef TC_SET_BOTH
#undef TC_SET
  p.wbf = c->ws + c->L.wbf;
  p.top2 = (float*)(c->ws + c->L.top2);
  { const int rc = compute_xmax2(c); if (rc != ASGD_OK) return rc; }
  // |x_j| <= ||x||, and a centre stays inside the hull of the samples and the initial state: keep a factor 4 of room
  if (fp16 && !(8.f * sqrtf(p.xmax2) < 65504.f)) return ASGD_EUNSUPPORTED;
  const void* xh = nullptr;
  const void* xl = nullptr;
  if (fp16) {
    tc_half_x_kernel<<<c->sm_count * 8, 256, 0, c->stream>>>(p.X, (__half*)(c->ws + c->L.xbf), (size_t)cfg.N * cfg.d);
    xh = xl = c->ws + c->L.xbf;
  } else {
    // x = x_hi + x_lo in BF16: x_hi is the caller's copy when one was given, x_lo the rounded residue either way
    xh = c->xbf_user ? c->xbf_user : (const void*)(c->ws + c->L.xbf);
    xl = c->ws + c->L.xbl;
    tc_split_x_kernel<<<c->sm_count * 8, 256, 0, c->stream>>>(p.X, (const __nv_bfloat16*)c->xbf_user,
                                                               c->xbf_user ? nullptr : (__nv_bfloat16*)(c->ws + c->L.xbf),
                                                               (__nv_bfloat16*)(c->ws + c->L.xbl), (size_t)cfg.N * cfg.d);
  }
  tc_row_norms_kernel<<<c->sm_count * 8, 256, 0, c->stream>>>(p.X, cfg.N, cfg.d, (float*)(c->ws + c->L.xnorm));
  c->launches += 2;
  CU(c, cudaGetLastError());
  p.xnorm = (const float*)(c->ws + c->L.xnorm);
  if (!encode_16bit_map(&c->mapXh, fp16, xh, (unsigned long long)cfg.N, (unsigned long long)cfg.d, TC_M)) return ASGD_ECUDA;
  if (!encode_16bit_map(&c->mapXl, fp16, xl, (unsigned long long)cfg.N, (unsigned long long)cfg.d, TC_M)) return ASGD_ECUDA;
  if (!encode_16bit_map(&c->mapW, fp16, p.wbf, (fp16 ? 1ull : 2ull) * cfg.W * cfg.k, (unsigned long long)cfg.d, (unsigned)bn)) return ASGD_ECUDA;
  return ASGD_OK;
}

int launch_workers(asgd_ctx* c, bool det, long long steps) {
  const Params& p = c->p;
  switch (c->path) {
#define TC_GO(DET_, T_, D_, NT_) asgd_tc_kernel<DET_, T_, D_, NT_><<<c->grid, NT_, c->smem_bytes, c->stream>>>(p, steps, c->mapXh, c->mapXl, c->mapW)
#define TC_GO_BOTH(T_, D_, NT_) { if (det) TC_GO(true, T_, D_, NT_); else TC_GO(false, T_, D_, NT_); }
    case P_TC_BF16:
      if (c->tc_inst == 1) TC_GO_BOTH(3, 128, TC_THREADS) else if (c->tc_inst == 2) TC_GO_BOTH(3, 128, TC_THREADS_WIDE) else TC_GO_BOTH(3, 256, TC_THREADS_MID)
      break;
    case P_TC_FP16:
      if (c->tc_inst == 1) TC_GO_BOTH(1, 128, TC_THREADS) else if (c->tc_inst == 2) TC_GO_BOTH(1, 128, TC_THREADS_WIDE) else TC_GO_BOTH(1, 256, TC_THREADS_MID)
      break;
#undef TC_GO_BOTH
#undef TC_GO
    case P_TILED: {
      int idx = 0;
#define X(D_, KP_, WS_, WK_, MB_) if (idx++ == c->tiled_shape) tiled_launch<D_, KP_, WS_, WK_, MB_>(c, det, steps);
      ASGD_TILED_SHAPES(X)
#undef X
      break;
    }
    case P_STREAM:
#define X(D_, K_) if (p.d == D_ && p.k == K_) stream_launch<D_, K_>(c, det, steps);
      ASGD_STREAM_SHAPES(X)
#undef X
      break;
    case P_GENERIC:
    default:
      if (det)
        asgd_generic_kernel<true><<<p.W, GENERIC_THREADS, c->smem_bytes, c->stream>>>(p, steps, c->state_on_chip);
      else
        asgd_generic_kernel<false><<<p.W, GENERIC_THREADS, c->smem_bytes, c->stream>>>(p, steps, c->state_on_chip);
      break;
  }
  c->launches += 1;
  CU(c, cudaGetLastError());
  return ASGD_OK;
}

int resolve_path(asgd_ctx* c) {
  const asgd_config& cfg = c->cfg;
  if (cfg.dist_path == ASGD_PATH_TC_BF16 || cfg.dist_path == ASGD_PATH_TC_FP16 ||
      (cfg.dist_path == ASGD_PATH_AUTO && tc_eligible(&cfg) && !c->no_tc)) {
    if (!tc_supported(&cfg)) return ASGD_EUNSUPPORTED;
    c->path = (cfg.dist_path == ASGD_PATH_TC_BF16) ? P_TC_BF16 : P_TC_FP16;
    c->state_on_chip = 0;
    return ASGD_OK;                       // device-side set-up (tc_prepare) runs once the workspace is cleared
  }
  // streaming path: small state, a mini-batch of at most 4 samples per thread
  if (cfg.dist_path == ASGD_PATH_AUTO || cfg.dist_path == ASGD_PATH_FP32) {
#define X(D_, K_)                                                                     \
  if (cfg.d == D_ && cfg.k == K_ && cfg.b <= STREAM_MAX_B &&                         \
      stream_smem_bytes<D_, K_>(cfg.b) <= 100 * 1024) {                             \
    c->path = P_STREAM;                                                               \
    c->state_on_chip = 1;                                                             \
    return stream_prepare<D_, K_>(c);                                                 \
  }
    ASGD_STREAM_SHAPES(X)
#undef X
  }
  if (cfg.dist_path == ASGD_PATH_AUTO || cfg.dist_path == ASGD_PATH_FP32) {
    int idx = 0, best = -1;
    long long best_busy = -1;
#define X(D_, KP_, WS_, WK_, MB_)                                                                  \
  if (cfg.d == D_ && cfg.k <= KP_ && tiled_smem_bytes<D_, KP_, WS_, WK_>(cfg.k) <= kMaxDynSmem) { \
    long long busy = 0;                                                                            \
    if (tiled_prepare<D_, KP_, WS_, WK_, MB_>(c, &busy) == ASGD_OK && busy >= best_busy) { best = idx; best_busy = busy; } \
  }                                                                                                \
  ++idx;
    ASGD_TILED_SHAPES(X)
#undef X
    if (best >= 0) {
      idx = 0;
      long long busy = 0;
      int rc = ASGD_EUNSUPPORTED;
#define X(D_, KP_, WS_, WK_, MB_) if (idx++ == best) rc = tiled_prepare<D_, KP_, WS_, WK_, MB_>(c, &busy);
      ASGD_TILED_SHAPES(X)
#undef X
      c->path = P_TILED;
      c->state_on_chip = 0;
      c->tiled_shape = best;
      return rc;
    }
  }
  c->path = P_GENERIC;
  const int kd_pad = c->p.kd_pad;
  size_t on = generic_smem_bytes(cfg.k, cfg.b, kd_pad, true);
  size_t off = generic_smem_bytes(cfg.k, cfg.b, kd_pad, false);
  if (on <= 200 * 1024) {
    c->state_on_chip = 1;
    c->smem_bytes = on;
  } else if (off <= kMaxDynSmem) {
    c->state_on_chip = 0;
    c->smem_bytes = off;
  } else {
    return ASGD_EUNSUPPORTED;
  }
  CU(c, cudaFuncSetAttribute(asgd_generic_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->smem_bytes));
  CU(c, cudaFuncSetAttribute(asgd_generic_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)c->smem_bytes));
  return ASGD_OK;
}

}  // namespace

extern "C" {

int asgd_workspace_bytes(const asgd_config* cfg, size_t* bytes) {
  if (!bytes || !config_ok(cfg)) return ASGD_EINVAL;
  *bytes = make_layout(cfg).total;
  return ASGD_OK;
}

int asgd_init(asgd_ctx** out, const asgd_config* cfg, const float* X_dev, const void* X_bf16_dev,
              const float* w0_dev, void* workspace_dev, size_t workspace_bytes, void* cuda_stream) {
  if (!out) return ASGD_EINVAL;
  *out = nullptr;
  if (!config_ok(cfg) || !X_dev || !w0_dev || !workspace_dev) return ASGD_EINVAL;
  if (((uintptr_t)X_dev & 15) || ((uintptr_t)workspace_dev & (kAlign - 1))) return ASGD_EINVAL;
  Layout L = make_layout(cfg);
  if (workspace_bytes < L.total) return ASGD_ENOMEM;

  int dev = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return ASGD_EUNSUPPORTED;
  if (prop.major != 10) return ASGD_EUNSUPPORTED;

  asgd_ctx* c = new (std::nothrow) asgd_ctx();
  if (!c) return ASGD_ENOMEM;
  c->cfg = *cfg;
  c->L = L;
  c->ws = (unsigned char*)workspace_dev;
  c->stream = (cudaStream_t)cuda_stream;
  c->t_host = 0;
  c->launches = 0;
  c->last_cuda = 0;
  c->sm_count = prop.multiProcessorCount;
  c->xbf_user = X_bf16_dev;
  c->no_tc = 0;

  Params& p = c->p;
  p.X = X_dev; p.N = cfg->N; p.d = cfg->d; p.k = cfg->k; p.W = cfg->W; p.b = cfg->b; p.eps = cfg->eps;
  p.c = cfg->comm_interval; p.f = cfg->fanout; p.S = cfg->slots; p.parzen = cfg->parzen ? 1 : 0;
  p.seed = cfg->seed;
  p.H = cfg->N / cfg->W; p.B = p.H / cfg->b;
  p.kd = cfg->k * cfg->d; p.kd_pad = (p.kd + 3) / 4 * 4;
  p.state = (float*)(c->ws + L.state);
  p.mail = (float*)(c->ws + L.mail);
  p.seq = (unsigned*)(c->ws + L.seq);
  p.seen = (unsigned*)(c->ws + L.seen);
  p.arb_win = (unsigned*)(c->ws + L.arb_win);
  p.arb_cnt = (unsigned*)(c->ws + L.arb_cnt);
  p.stats = (unsigned long long*)(c->ws + L.stats);
  p.perm = (const int*)(c->ws + L.perm);
  p.status = (int*)(c->ws + L.status);
  p.assign_rec = cfg->record_assign ? (int*)(c->ws + L.assign_rec) : nullptr;
  p.accept_rec = (int*)(c->ws + L.accept_rec);
  p.rows_m = cfg->partial_rows;
  p.mail_rows = (int2*)(c->ws + L.mail_rows);
  p.rowacc = (unsigned*)(c->ws + L.rowacc);
  p.rowin = (unsigned*)(c->ws + L.rowin);
  p.gsum = (float*)(c->ws + L.gsum);
  p.xmax2 = 0.f;
  p.wait_limit = DEFAULT_WAIT_LIMIT;
  p.withhold_step = -1;
  p.wbf = nullptr;
  p.top2 = nullptr;
  p.xnorm = nullptr;

  int rc = resolve_path(c);
  if (rc != ASGD_OK) { delete c; return rc; }

  // empty buffers, zero counters (everything between mail and perm, plus status/records)
  cudaError_t e = cudaMemsetAsync(c->ws + L.mail, 0, L.perm - L.mail, c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->ws + L.status, 0, L.total - L.status, c->stream);
  if (e != cudaSuccess) { delete c; return ASGD_ECUDA; }
  broadcast_state_kernel<<<256, 256, 0, c->stream>>>(p.state, w0_dev, p.W, p.kd, p.kd_pad);
  c->launches += 1;
  if (c->path == P_TC_BF16 || c->path == P_TC_FP16) {
    rc = tc_prepare(c);
    if (rc == ASGD_EUNSUPPORTED && cfg->dist_path == ASGD_PATH_AUTO) {      // samples outside FP16's range: an fp32 path instead
      c->no_tc = 1;
      rc = resolve_path(c);
      if (rc == ASGD_OK && (c->path == P_STREAM || c->path == P_TILED)) rc = compute_xmax2(c);
    }
    if (rc != ASGD_OK) { delete c; return rc; }
  } else if (c->path == P_STREAM || c->path == P_TILED) {
    rc = compute_xmax2(c);
    if (rc != ASGD_OK) { delete c; return rc; }
  }

  // batch orders
  {
    std::vector<int> perm;
    try { perm.resize((size_t)p.W * p.B); } catch (...) { delete c; return ASGD_ENOMEM; }
    for (int i = 0; i < p.W; ++i) fill_perm(*cfg, p.B, i, perm.data() + (size_t)i * p.B);
    e = cudaMemcpyAsync(c->ws + L.perm, perm.data(), perm.size() * sizeof(int), cudaMemcpyHostToDevice, c->stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // perm is a local: finish the copy
    if (e != cudaSuccess) { delete c; return ASGD_ECUDA; }
  }
  *out = c;
  return ASGD_OK;
}

int asgd_step(asgd_ctx* c, int64_t rounds) {
  if (!c || rounds < 0) return ASGD_EINVAL;
  const Params& p = c->p;
  for (int64_t r = 0; r < rounds; ++r) {
    int rc = launch_workers(c, true, 1);
    if (rc != ASGD_OK) return rc;
    if (p.c > 0 && p.f > 0 && p.W > 1 && (c->t_host + 1) % p.c == 0) {
      deliver_kernel<<<p.W * p.S, 128, 0, c->stream>>>(p);
      c->launches += 1;
      CU(c, cudaGetLastError());
    }
    c->t_host += 1;
  }
  return ASGD_OK;
}

int asgd_run(asgd_ctx* c, int64_t steps_per_worker) {
  if (!c || steps_per_worker < 0) return ASGD_EINVAL;
  if (steps_per_worker == 0) return ASGD_OK;
  int rc = launch_workers(c, false, steps_per_worker);
  if (rc != ASGD_OK) return rc;
  c->t_host += steps_per_worker;
  return ASGD_OK;
}

int asgd_get_state(asgd_ctx* c, int32_t worker, float* out_dev) {
  if (!c || !out_dev || worker < -1 || worker >= c->p.W) return ASGD_EINVAL;
  const Params& p = c->p;
  if (worker >= 0) {
    CU(c, cudaMemcpyAsync(out_dev, p.state + (size_t)worker * p.kd_pad, (size_t)p.kd * 4, cudaMemcpyDeviceToDevice, c->stream));
  } else {
    mean_state_kernel<<<(p.kd + 255) / 256, 256, 0, c->stream>>>(p.state, p.W, p.kd, p.kd_pad, out_dev);
    c->launches += 1;
    CU(c, cudaGetLastError());
  }
  return ASGD_OK;
}

int asgd_set_state(asgd_ctx* c, int32_t worker, const float* w_dev) {
  if (!c || !w_dev || worker < 0 || worker >= c->p.W) return ASGD_EINVAL;
  const Params& p = c->p;
  CU(c, cudaMemcpyAsync(p.state + (size_t)worker * p.kd_pad, w_dev, (size_t)p.kd * 4, cudaMemcpyDeviceToDevice, c->stream));
  return ASGD_OK;
}

int asgd_put(asgd_ctx* c, int32_t worker, int32_t slot, const float* payload_dev) {
  if (!c || !payload_dev || worker < 0 || worker >= c->p.W || slot < 0 || slot >= c->p.S) return ASGD_EINVAL;
  const Params& p = c->p;
  const size_t ri = (size_t)worker * p.S + slot;
  if (p.rows_m > 0) return asgd_put_rows(c, worker, slot, payload_dev, 0, p.k);      // a whole message carries every row
  external_put_kernel<<<1, 256, 0, c->stream>>>(p.mail + ri * (size_t)p.kd_pad, payload_dev, p.seq + ri, p.kd);
  c->launches += 1;
  CU(c, cudaGetLastError());
  return ASGD_OK;
}

int asgd_put_rows(asgd_ctx* c, int32_t worker, int32_t slot, const float* payload_dev, int32_t first_row, int32_t n_rows) {
  if (!c || !payload_dev || worker < 0 || worker >= c->p.W || slot < 0 || slot >= c->p.S) return ASGD_EINVAL;
  const Params& p = c->p;
  if (p.rows_m <= 0 || first_row < 0 || first_row >= p.k || n_rows < 1 || n_rows > p.k) return ASGD_EINVAL;
  const size_t ri = (size_t)worker * p.S + slot;
  external_put_rows_kernel<<<1, 256, 0, c->stream>>>(p.mail + ri * (size_t)p.kd_pad, payload_dev, p.seq + ri, p.mail_rows + ri,
                                                     p.k, p.d, first_row, n_rows);
  c->launches += 1;
  CU(c, cudaGetLastError());
  return ASGD_OK;
}

int asgd_eval(asgd_ctx* c, int32_t worker, double* E_host) {
  if (!c || !E_host || worker < -1 || worker >= c->p.W) return ASGD_EINVAL;
  const Params& p = c->p;
  const float* w = nullptr;
  if (worker >= 0) {
    w = p.state + (size_t)worker * p.kd_pad;
  } else {
    float* tmp = (float*)(c->ws + c->L.tmp_state);
    int rc = asgd_get_state(c, -1, tmp);
    if (rc != ASGD_OK) return rc;
    w = tmp;
  }
  const size_t wbytes = (size_t)p.kd * 4;
  const int on_chip = wbytes <= 160 * 1024;
  const size_t smem = 32 * sizeof(double) + (on_chip ? wbytes : 0);
  CU(c, cudaFuncSetAttribute(eval_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  double* partial = (double*)(c->ws + c->L.eval_partial);
  bool small = false;
#define X(D_, K_)                                                                                     \
  if (!small && p.d == D_ && p.k == K_) {                                                             \
    eval_small_kernel<D_, K_><<<kEvalBlocks, EVAL_THREADS, 0, c->stream>>>(p.X, p.N, w, partial);     \
    small = true;                                                                                     \
  }
  ASGD_STREAM_SHAPES(X)
#undef X
  if (!small) eval_kernel<<<kEvalBlocks, EVAL_THREADS, smem, c->stream>>>(p.X, p.N, p.d, p.k, w, on_chip, partial);
  c->launches += 1;
  CU(c, cudaGetLastError());
  std::vector<double> host;
  try { host.resize(kEvalBlocks); } catch (...) { return ASGD_ENOMEM; }
  CU(c, cudaMemcpyAsync(host.data(), partial, sizeof(double) * kEvalBlocks, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  double E = 0.0;
  for (int q = 0; q < kEvalBlocks; ++q) E += host[q];
  *E_host = E;
  return ASGD_OK;
}

int asgd_get_stats(asgd_ctx* c, int32_t worker, uint64_t* out_host) {
  if (!c || !out_host || worker < 0 || worker >= c->p.W) return ASGD_EINVAL;
  unsigned long long row[ST_STRIDE];
  CU(c, cudaMemcpyAsync(row, c->p.stats + (size_t)worker * ST_STRIDE, sizeof(row), cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  for (int q = 0; q < 5; ++q) out_host[q] = row[q];
  return ASGD_OK;
}

int asgd_get_assign(asgd_ctx* c, int32_t* out_dev) {
  if (!c || !out_dev || !c->p.assign_rec) return ASGD_EINVAL;
  CU(c, cudaMemcpyAsync(out_dev, c->p.assign_rec, (size_t)c->p.W * c->p.b * 4, cudaMemcpyDeviceToDevice, c->stream));
  return ASGD_OK;
}

int asgd_get_accept(asgd_ctx* c, int32_t worker, int32_t* out_host) {
  if (!c || !out_host || worker < 0 || worker >= c->p.W) return ASGD_EINVAL;
  CU(c, cudaMemcpyAsync(out_host, c->p.accept_rec + (size_t)worker * c->p.S, (size_t)c->p.S * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  return ASGD_OK;
}

int asgd_get_accept_rows(asgd_ctx* c, int32_t worker, int32_t* out_host) {
  if (!c || !out_host || worker < 0 || worker >= c->p.W) return ASGD_EINVAL;
  const Params& p = c->p;
  if (p.rows_m <= 0) return ASGD_EINVAL;
  std::vector<unsigned> acc, in;
  try { acc.resize(p.k); in.resize(p.k); } catch (...) { return ASGD_ENOMEM; }
  CU(c, cudaMemcpyAsync(acc.data(), p.rowacc + (size_t)worker * p.k, (size_t)p.k * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaMemcpyAsync(in.data(), p.rowin + (size_t)worker * p.k, (size_t)p.k * 4, cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  for (int s = 0; s < p.S; ++s)
    for (int a = 0; a < p.k; ++a)
      out_host[(size_t)s * p.k + a] = ((in[a] >> s) & 1u) ? (int32_t)((acc[a] >> s) & 1u) : -1;
  return ASGD_OK;
}

int asgd_sync(asgd_ctx* c) {
  if (!c) return ASGD_EINVAL;
  int st[4] = {0, 0, 0, 0};
  CU(c, cudaMemcpyAsync(st, c->p.status, sizeof(st), cudaMemcpyDeviceToHost, c->stream));
  CU(c, cudaStreamSynchronize(c->stream));
  if (st[0] == DEV_TIMEOUT) return ASGD_ETIMEOUT;
  return ASGD_OK;
}

int asgd_set_wait_drill(asgd_ctx* c, uint32_t wait_limit, int64_t withhold_step) {
  if (!c || wait_limit == 0) return ASGD_EINVAL;
  c->p.wait_limit = wait_limit;
  c->p.withhold_step = withhold_step < 0 ? -1 : withhold_step;
  return ASGD_OK;
}

int64_t asgd_launch_count(const asgd_ctx* c) { return c ? c->launches : 0; }

const char* asgd_path_name(const asgd_ctx* c) {
  if (!c) return "none";
  switch (c->path) {
    case P_GENERIC: return c->state_on_chip ? "fp32-generic" : "fp32-generic-offchip";
    case P_STREAM: return "fp32-stream";
    case P_TILED: return "fp32-tiled";
    case P_TC_BF16: return "tcgen05-bf16x3";
    case P_TC_FP16: return "tcgen05-fp16";
    default: return "unknown";
  }
}

int asgd_last_cuda_error(const asgd_ctx* c) { return c ? c->last_cuda : 0; }

const char* asgd_strerror(int s) {
  switch (s) {
    case ASGD_OK: return "ok";
    case ASGD_EINVAL: return "invalid argument";
    case ASGD_ENOMEM: return "workspace too small or host allocation failed";
    case ASGD_ECUDA: return "CUDA call failed";
    case ASGD_EUNSUPPORTED: return "unsupported device or problem size";
    case ASGD_ETIMEOUT: return "a bounded device-side wait expired";
    default: return "unknown status";
  }
}

void asgd_destroy(asgd_ctx* c) { delete c; }

int asgd_fit_host_bytes(const asgd_config* cfg, size_t* bytes) {
  if (!bytes || !config_ok(cfg)) return ASGD_EINVAL;
  const size_t kd = (size_t)cfg->k * cfg->d;
  *bytes = up((size_t)cfg->N * cfg->d * 4) + up(kd * 4) + up(kd * 4) + make_layout(cfg).total;
  return ASGD_OK;
}

int asgd_fit_host(const asgd_config* cfg, const float* X_host, const float* w0_host, int64_t steps_per_worker,
                  int32_t mode_async, float* w_out_host, void* scratch_dev, size_t scratch_bytes, void* cuda_stream) {
  size_t need = 0;
  if (asgd_fit_host_bytes(cfg, &need) != ASGD_OK || !X_host || !w0_host || !w_out_host || !scratch_dev ||
      steps_per_worker < 0)
    return ASGD_EINVAL;
  if (scratch_bytes < need) return ASGD_ENOMEM;
  if ((uintptr_t)scratch_dev & (kAlign - 1)) return ASGD_EINVAL;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  const size_t kd = (size_t)cfg->k * cfg->d, xb = (size_t)cfg->N * cfg->d * 4;
  unsigned char* base = (unsigned char*)scratch_dev;
  float* Xd = (float*)base;
  float* w0d = (float*)(base + up(xb));
  float* wod = (float*)(base + up(xb) + up(kd * 4));
  void* ws = base + up(xb) + 2 * up(kd * 4);
  if (cudaMemcpyAsync(Xd, X_host, xb, cudaMemcpyHostToDevice, st) != cudaSuccess) return ASGD_ECUDA;
  if (cudaMemcpyAsync(w0d, w0_host, kd * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) return ASGD_ECUDA;
  asgd_ctx* c = nullptr;
  int rc = asgd_init(&c, cfg, Xd, nullptr, w0d, ws, scratch_bytes - (size_t)((unsigned char*)ws - base), st);
  if (rc != ASGD_OK) return rc;
  rc = mode_async ? asgd_run(c, steps_per_worker) : asgd_step(c, steps_per_worker);
  if (rc == ASGD_OK) rc = asgd_get_state(c, 0, wod);
  if (rc == ASGD_OK && cudaMemcpyAsync(w_out_host, wod, kd * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) rc = ASGD_ECUDA;
  if (rc == ASGD_OK) rc = asgd_sync(c);
  asgd_destroy(c);
  return rc;
}

}  // extern "C"
