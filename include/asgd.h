/*
 * libasgd -- K-Means ASGD worker loop on one NVIDIA B200 (sm_100a), C ABI.
 *
 * The operations follow Keuper & Pfreundt, "Asynchronous Parallel Stochastic Gradient Descent"
 * (arXiv 1505.04956):
 *   - Algorithm 5 (ASGD): W workers, each owning a disjoint shard of the samples, repeat
 *       draw mini-batch -> externally modified update -> send the new state to random peers.
 *   - Eq. 8: assignment s_i(w) = index of the closest prototype; quantisation error E(w).
 *   - Eq. 9: K-Means mini-batch gradient (per-centre sums and counts of the assigned samples).
 *   - Eq. 3 / Eq. 4 / Eq. 6 / Eq. 7: N receive buffers per worker, the "buffer non-empty" indicator
 *     lambda, the Parzen-window acceptance test delta, and the merged step.
 *   - Section 1.2 / Section 3: single-sided communication; the sender never waits, the receiver
 *     uses whatever has arrived.
 *
 * On the GPU a worker is a thread block, a receive buffer is a region of device memory, and a put
 * is a sequence of global stores followed by a release-increment of the buffer's sequence number.
 *
 * General rules
 *   - Every pointer argument says whether it is HOST or DEVICE memory.  Device pointers must
 *     belong to the device that was current when asgd_init() ran.
 *   - Every function returns 0 (ASGD_OK) or a negative asgd_status.  Nothing throws or aborts.
 *   - The library allocates no device memory: the caller passes one workspace of
 *     asgd_workspace_bytes() bytes and keeps it alive until asgd_destroy().
 *   - All device work is enqueued on the stream given to asgd_init(); calls return after enqueue
 *     unless stated otherwise.  A context is not thread-safe.
 *   - There is no CPU fallback.  Without a CUDA device of compute capability 10.x asgd_init()
 *     returns ASGD_EUNSUPPORTED.
 */
#ifndef ASGD_H_
#define ASGD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum asgd_status {
  ASGD_OK = 0,
  ASGD_EINVAL = -1,       /* NULL / out-of-range / misaligned argument                      */
  ASGD_ENOMEM = -2,       /* workspace too small, or a host allocation failed               */
  ASGD_ECUDA = -3,        /* a CUDA call failed; code via asgd_last_cuda_error()            */
  ASGD_EUNSUPPORTED = -4, /* wrong device, or sizes outside what the chosen path supports   */
  ASGD_ETIMEOUT = -5      /* a bounded device-side wait expired (reported by asgd_sync)     */
} asgd_status;

/* Distance paths of the assignment (Eq. 8).  AUTO takes, in this order: the streaming kernel for the small shapes
 * it is compiled for (k, d <= 16, b <= 512); the tensor-core path with FP16 operands where d is a multiple of 64 up
 * to 256, k <= 1024 and 128 <= b <= 4096 (and the samples fit FP16, see below); the register-tiled kernel (d = 32
 * with k <= 64, d = 128 with k <= 128); else the shape-independent kernel.  Every path decides Eq. 8 exactly. */
enum {
  ASGD_PATH_AUTO = 0,
  ASGD_PATH_FP32 = 1,       /* CUDA cores, fp32 (the specialised kernel for the shape, if any) */
  ASGD_PATH_TC_FP16 = 2,    /* tcgen05, FP16 operands, fp32 accumulate; rows the rounding bound cannot   */
                            /* decide are decided exactly afterwards.  Needs 8 max ||x|| < 65504       */
                            /* (ASGD_EUNSUPPORTED otherwise; AUTO then takes an fp32 path)              */
  ASGD_PATH_TC_BF16 = 3,    /* tcgen05, BF16 operands in two terms each (x_hi + x_lo, w_hi + w_lo;     */
                            /* three products per score), fp32 accumulate: any fp32 range, same exact  */
                            /* decisions, three times the tensor work                                  */
  ASGD_PATH_FP32_GENERAL = 4 /* CUDA cores, fp32, the shape-independent kernel                */
};

/* Problem statement ASGD(X, T, eps, w0, b) of Algorithm 5 plus the communication parameters. */
typedef struct asgd_config {
  int64_t N;             /* rows of X                                                         */
  int32_t d;             /* dimensions per sample                                             */
  int32_t k;             /* centres (prototypes) per state                                    */
  int32_t W;             /* workers; worker i owns rows [i*H, (i+1)*H), H = N / W (floor)     */
  int32_t b;             /* mini-batch size, 1 <= b <= H.  A pass is B = H / b (floor) steps;  */
                         /* rows beyond W*H and the last H - B*b rows of a shard are unused    */
  float eps;             /* step size > 0                                                     */
  int32_t comm_interval; /* c: put after step t iff c > 0 and (t+1) % c == 0; 0 = silent      */
  int32_t fanout;        /* f: recipients per put, 0 <= f <= W-1                              */
  int32_t slots;         /* S: receive buffers per worker, >= 1                               */
  int32_t parzen;        /* 1 = Eq. 6 (acceptance test of Eq. 4), 0 = Eq. 3 (accept all)      */
  int32_t dist_path;     /* ASGD_PATH_*                                                       */
  int32_t shuffle;       /* 1 = seeded permutation of each worker's batch order, 0 = in order */
  int32_t record_assign; /* 1 = keep the last step's assignments for asgd_get_assign()        */
  int32_t partial_rows;  /* 0 = a put carries the whole state; m in 1..k = m centre rows      */
  uint64_t seed;         /* batch order, recipients, buffer choice                            */
} asgd_config;

typedef struct asgd_ctx asgd_ctx; /* opaque; owned by the library, freed by asgd_destroy() */

/* Bytes of device workspace asgd_init() needs for this configuration (256-byte aligned base). */
int asgd_workspace_bytes(const asgd_config *cfg, size_t *bytes /* HOST out */);

/*
 * Initialisation step of Section 4: shards are fixed, w0 is copied into all W worker states,
 * receive buffers are emptied, counters zeroed, batch orders drawn.
 *   X_dev        DEVICE [N*d] fp32 row-major, 16-byte aligned.  BORROWED: never written, must stay
 *                alive and unchanged until asgd_destroy().
 *   X_bf16_dev   DEVICE [N*d] bf16 copy of X for ASGD_PATH_TC_BF16 (taken as the leading term x_hi; the
 *                library forms the residue x_lo itself), or NULL.  BORROWED like X_dev.
 *   w0_dev       DEVICE [k*d] fp32.  COPIED.
 *   workspace    DEVICE, >= asgd_workspace_bytes(), 256-byte aligned.  BORROWED until destroy.
 *   cuda_stream  a cudaStream_t (NULL = default stream).
 */
int asgd_init(asgd_ctx **out, const asgd_config *cfg, const float *X_dev, const void *X_bf16_dev,
              const float *w0_dev, void *workspace_dev, size_t workspace_bytes, void *cuda_stream);

/*
 * Deterministic mode.  `rounds` synchronous rounds: in a round every worker performs one step of
 * Algorithm 5 (mini-batch, Eq. 8 assignment, Eq. 9 gradient, Eq. 4 tests, Eq. 6 update) from the
 * states and receive buffers it had when the round began; then the round's puts are delivered as
 * whole messages, senders in ascending order (the last sender into a buffer wins).
 */
int asgd_step(asgd_ctx *ctx, int64_t rounds);

/*
 * Free-running mode (Section 1.2): one persistent launch in which every worker performs
 * `steps_per_worker` steps at its own pace; puts are plain stores into the recipient's buffer
 * published by a release-increment of its sequence number, never acknowledged, never waited for.
 * Messages may be lost or torn (Section 4.4).  Returns after enqueue.
 */
int asgd_run(asgd_ctx *ctx, int64_t steps_per_worker);

/* State of one worker (worker 0 is the w^1 that Algorithm 5 returns); worker = -1 gives the mean
 * over all workers (the aggregation variant of Section 4.3).  out_dev: DEVICE [k*d], caller's. */
int asgd_get_state(asgd_ctx *ctx, int32_t worker, float *out_dev);
/* Overwrite one worker's state (resume from an earlier run, Section 4 "Initialization"). */
int asgd_set_state(asgd_ctx *ctx, int32_t worker, const float *w_dev /* DEVICE [k*d] */);
/* A put from outside: write a whole message into receive buffer `slot` of `worker`. */
int asgd_put(asgd_ctx *ctx, int32_t worker, int32_t slot, const float *payload_dev /* DEVICE [k*d] */);

/* Per-centre messages (Section 4.4: K-Means updates are split per centre row of the state),
 * cfg.partial_rows = m >= 1.  The paper states no formulas for them; the library applies Eq. 3, Eq. 4
 * and Eq. 6 to each centre row on its own: a put after step t carries the m consecutive rows (cyclic)
 * that start at row h(seed, 4, i, t, j) mod k of the sender's new state; for every new message that
 * carries row a, lambda is "the row is not all zero", delta compares ||(w_a - eps D_a) - v_a|| with
 * ||w_a - v_a||, and row a is merged with its own count of accepted rows.  A message counts as accepted
 * when at least one of its rows was.  asgd_put then writes a message that carries every row.
 *
 * asgd_put_rows: a put from outside carrying rows [first_row, first_row + n_rows) (cyclic) of
 * payload_dev (DEVICE [k*d]; other rows are not read).  ASGD_EINVAL unless cfg.partial_rows >= 1. */
int asgd_put_rows(asgd_ctx *ctx, int32_t worker, int32_t slot, const float *payload_dev, int32_t first_row,
                  int32_t n_rows);
/* Per-row acceptance of the last step of `worker` in per-centre mode: out_host[S*k], entry [s*k + a] is
 * -1 when buffer s held no new message carrying row a, else 0 (rejected) or 1 (accepted).  Synchronises.
 * asgd_get_accept then gives the number of accepted rows per buffer (-1 nothing new). */
int asgd_get_accept_rows(asgd_ctx *ctx, int32_t worker, int32_t *out_host /* HOST [S*k] */);

/* Eq. 8: E(w) of the given worker's state (-1 = mean state) over all N rows.  Synchronises. */
int asgd_eval(asgd_ctx *ctx, int32_t worker, double *E_host /* HOST out */);

/* The per-worker message counters of Fig. 12 (messages sent, received, and "good" ones, i.e. those the
 * Parzen window of Eq. 4 let through), plus the steps done and the messages overwritten before their
 * owner looked:  out_host[5] = steps, sent, received, accepted (delta = 1), overwritten unread.
 * Synchronises. */
int asgd_get_stats(asgd_ctx *ctx, int32_t worker, uint64_t *out_host /* HOST [5] */);

/* Assignments s_i(w) of the last deterministic round, [W*b] int32 in worker-major order.
 * Needs cfg.record_assign = 1.  out_dev: DEVICE, caller's. */
int asgd_get_assign(asgd_ctx *ctx, int32_t *out_dev);
/* Outcome of the acceptance test of Eq. 4 (times lambda of Eq. 3) per receive buffer in the last step of
 * `worker`: out_host[S], -1 nothing new, 0 rejected, 1 accepted.  Synchronises. */
int asgd_get_accept(asgd_ctx *ctx, int32_t worker, int32_t *out_host /* HOST [S] */);

/* Wait for the stream and return the device status word (ASGD_OK, or ASGD_ETIMEOUT when a worker kernel
 * gave up a bounded wait on one of its own copies).  Housekeeping of this library: the paper has no
 * counterpart (its workers never wait, Section 1.2; neither do these, on one another). */
int asgd_sync(asgd_ctx *ctx);
/*
 * Failure drill for the bounded waits (no counterpart in the paper).  A worker kernel waits only for its
 * own asynchronous copies of samples, and gives each wait up after `wait_limit` polls (default 2^22):
 * the block then raises the device status word, gives the copies it still has in flight the same bounded
 * chance to land, releases what it holds and returns, so the context stays usable and asgd_sync() reports
 * ASGD_ETIMEOUT.  With withhold_step = s >= 0 the first sample copy of step s of every following launch
 * (counted from the launch's first step) is announced to its barrier but never issued, which makes that
 * wait run out without any fault; -1 switches the drill off.  The generic kernel has no such waits.
 * Affects launches made after the call.  ASGD_EINVAL for a NULL context or wait_limit = 0.
 */
int asgd_set_wait_drill(asgd_ctx *ctx, uint32_t wait_limit, int64_t withhold_step);
/* Number of kernels this context has launched so far. */
int64_t asgd_launch_count(const asgd_ctx *ctx);
/* Name of the distance path the context resolved to ("fp32-generic", "fp32-stream", ...). */
const char *asgd_path_name(const asgd_ctx *ctx);
/* cudaError_t of the last failed CUDA call in this context (0 if none). */
int asgd_last_cuda_error(const asgd_ctx *ctx);
const char *asgd_strerror(int status);
void asgd_destroy(asgd_ctx *ctx);

/*
 * Whole job from HOST buffers (Algorithm 5 end to end): copies X and w0 to the device, runs
 * `steps_per_worker` steps per worker (free-running if cfg is used with mode_async != 0, else
 * deterministic rounds), copies worker 0's state back.  Synchronises before returning.
 *   X_host       HOST [N*d] fp32 (pinned memory gives the best copy rate)
 *   w0_host      HOST [k*d]
 *   w_out_host   HOST [k*d] out
 *   scratch_dev  DEVICE, >= asgd_fit_host_bytes(cfg) bytes, 256-byte aligned
 */
int asgd_fit_host_bytes(const asgd_config *cfg, size_t *bytes /* HOST out */);
int asgd_fit_host(const asgd_config *cfg, const float *X_host, const float *w0_host,
                  int64_t steps_per_worker, int32_t mode_async, float *w_out_host,
                  void *scratch_dev, size_t scratch_bytes, void *cuda_stream);

/*
 * E(w) of Eq. 8 for callers that must not allocate device memory.  (The paper has no counterpart
 * to this entry point; it exists for the sake of the caller, not of the method.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside a latency-critical serving
 * loop whose memory was carved up at start-up, under a framework's caching allocator whose pool the
 * caller may not grow, or in a process whose device memory is fully budgeted to someone else.  Such
 * a caller can own X, w and one double for the result, but cannot hand the library a workspace, so
 * asgd_eval() (which keeps its per-block partial sums in the context's workspace) is closed to it.
 * Here the partial sums live in a fixed array compiled into the library:
 * ASGD_EVAL_NOALLOC_MAX_BLOCKS doubles (32 KB) on every GPU that loads the library, until exit.
 *
 *   X_dev   DEVICE [N*d] fp32 row-major (input)       w_dev  DEVICE [k*d] fp32 (input)
 *   E_dev   DEVICE, one double (output): sum over rows of 1/2 min_k ||x - w_k||^2
 *
 * Limits: N <= ASGD_EVAL_NOALLOC_MAX_BLOCKS * ASGD_EVAL_NOALLOC_ROWS_PER_BLOCK (2^28 rows) and
 * k*d <= ASGD_EVAL_NOALLOC_MAX_KD (the centres are kept in shared memory); anything larger returns
 * ASGD_EUNSUPPORTED and launches nothing.  Rows are summed in blocks of a fixed size and the blocks
 * in ascending order, so the value does not depend on the GPU's size.
 *
 * The call enqueues two kernels on `cuda_stream` and returns; it calls no cudaMalloc, no cudaFree
 * and no allocating routine of any library.  The first call on each device also looks up the
 * array's device address (cudaGetSymbolAddress) and raises the kernel's shared-memory limit, with
 * that device current; make that first call before starting any stream capture.
 *
 * All calls on a device share the one array.  Nothing in it has to start at zero (a call writes
 * every entry it later reads), but two calls that overlap on the GPU -- different streams, or
 * different host threads -- race on it: keep calls on one device in stream order.
 */
#define ASGD_EVAL_NOALLOC_ROWS_PER_BLOCK 65536
#define ASGD_EVAL_NOALLOC_MAX_BLOCKS 4096
#define ASGD_EVAL_NOALLOC_MAX_KD 40960
int asgd_eval_noalloc(const float *X_dev, int64_t N, int32_t d, int32_t k, const float *w_dev,
                      double *E_dev, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ASGD_H_ */
