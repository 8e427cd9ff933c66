// TEST INFRASTRUCTURE -- not part of the product.
//
// Plain, slow, single-threaded CPU restatement of the K-Means ASGD worker loop of
// Keuper & Pfreundt, "Asynchronous Parallel Stochastic Gradient Descent" (arXiv 1505.04956).
// It exists only so that the CUDA library can be checked against something written directly
// from the paper.  It shares no code with the CUDA path and must never be called by it.
//
// Arithmetic: inputs and stored states are fp32 (the paper never states a precision); every
// intermediate quantity is fp64.  A state is rounded to fp32 once, when the step that produced
// it ends, because that is the value a peer would receive.
//
// What each function follows:
//   assignment  s_i(w)          -- Eq. 8 text: index of the closest prototype (ties -> lowest index)
//   quantisation error E(w)     -- Eq. 8
//   mini-batch gradient         -- Eq. 9, read as the true gradient dE/dw_k averaged over the
//                                  mini-batch size b:  D_k = (n_k w_k - S_k) / b
//   Parzen acceptance delta     -- Eq. 4 (literal two-norm form, strict "<")
//   lambda (buffer non-empty)   -- Eq. 3
//   merged step                 -- Eq. 6 / Eq. 7, then  w <- w - eps * Dbar  (Algorithm 5)
//   send                        -- Algorithm 5, send line: the new state goes to random workers other than i
//   partial (per-centre) puts   -- Section 4.4: a message carries some of the centre rows, lambda and
//                                  delta are then taken row by row (the reading is stated at worker_step_rows)
//
// Parity status: every function here is pinned by the CPU tests (brute force, closed forms,
// special cases, invariants); the optional parallel loop over the workers of a round is pinned
// bit for bit against the single-threaded loop.  The free-running asynchronous mode of the CUDA library has no
// step-wise counterpart here ("parity unpinned" for that mode only): races are part of the
// method, so it is compared statistically through E(w).
//
// Build:  g++ -O2 -std=c++17 -shared -fPIC [-fopenmp] asgd_oracle.cpp -o libasgd_oracle.so

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------------------------
// Counter-based random numbers.  SplitMix64 (Steele, Lea, Flood 2014): the generator's state
// advances by the golden-ratio increment and the output is a 3-stage xor-shift-multiply finaliser.
// sm64(x) below is "the first output of a SplitMix64 generator whose state was seeded with x".
// ---------------------------------------------------------------------------------------------
inline uint64_t sm64(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ull;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

// Stream tags: one independent stream per kind of draw.
constexpr uint64_t TAG_PERM = 1, TAG_PEER = 2, TAG_SLOT = 3, TAG_ROWS = 4;

// h(seed, tag, a, b, c): chain of four SplitMix64 outputs, each keyed by the next coordinate.
inline uint64_t draw(uint64_t seed, uint64_t tag, uint64_t a, uint64_t b, uint64_t c) {
  uint64_t h = sm64(seed ^ tag);
  h = sm64(h + a);
  h = sm64(h + b);
  h = sm64(h + c);
  return h;
}

struct Config {
  int64_t N;
  int32_t d, k, W, b;
  float eps;
  int32_t comm_interval, fanout, slots, parzen, shuffle;
  uint64_t seed;
  int32_t partial_rows = 0;   // 0: a put carries the whole state; m >= 1: m centre rows (Section 4.4)
};

struct Slot {
  std::vector<float> v;   // last payload written into this receive buffer
  std::vector<uint8_t> has;  // per centre row: 1 if the last message carried it (all 1 for whole-state messages)
  uint64_t seq = 0;       // number of messages ever written into it
  uint64_t seen = 0;      // value of seq when the owner last looked
};

struct Worker {
  std::vector<float> w;        // current state, k*d
  std::vector<float> w_next;   // state produced by the step in flight
  std::vector<Slot> mail;      // S receive buffers
  std::vector<int32_t> perm;   // batch order
  uint64_t t = 0;              // steps done
  uint64_t sent = 0, received = 0, accepted = 0, overwritten = 0;
  // trace of the last step (for single-step comparisons)
  std::vector<int32_t> assign;     // b
  std::vector<double> d1, d2;      // b: smallest and second smallest squared distance
  std::vector<int64_t> counts;     // k
  std::vector<int32_t> acc;        // S: acceptance a_s of the last step (-1 = slot had nothing new)
  std::vector<double> lhs, rhs;    // S: both sides of Eq. 4 (whole-state messages)
  std::vector<int32_t> row_acc;    // S*k: per-row acceptance of the last step in per-centre mode (-1 = row not in a new message)
  std::vector<double> row_lhs, row_rhs;   // S*k: both sides of Eq. 4 per row
};

struct Oracle {
  Config c;
  const float* X;
  int64_t H, B;
  std::vector<Worker> wk;
  int threads = 1;
};

// Algorithm 5, shuffle line (each worker shuffles its own samples), at mini-batch granularity: Fisher-Yates from the top.
void make_perm(const Config& c, int64_t B, int32_t worker, std::vector<int32_t>& perm) {
  perm.resize(B);
  for (int64_t p = 0; p < B; ++p) perm[p] = (int32_t)p;
  if (!c.shuffle) return;
  for (int64_t p = B - 1; p >= 1; --p) {
    uint64_t r = draw(c.seed, TAG_PERM, (uint64_t)worker, (uint64_t)p, 0) % (uint64_t)(p + 1);
    int32_t tmp = perm[p]; perm[p] = perm[r]; perm[r] = tmp;
  }
}

// Algorithm 5, send line (a random worker other than i): the j-th recipient of the put that follows step t.
// Uniform over the W-1 other workers; a repeat of an earlier recipient moves on to the next
// worker (cyclically, skipping the sender) until it is new.
void recipients(const Config& c, int32_t i, uint64_t t, int32_t* peers, int32_t* slots) {
  for (int32_t j = 0; j < c.fanout; ++j) {
    uint64_t r = draw(c.seed, TAG_PEER, (uint64_t)i, t, (uint64_t)j) % (uint64_t)(c.W - 1);
    int32_t p = (int32_t)r;
    if (p >= i) p += 1;
    for (;;) {
      bool dup = (p == i);
      for (int32_t q = 0; q < j && !dup; ++q) dup = (peers[q] == p);
      if (!dup) break;
      p = (p + 1) % c.W;
    }
    peers[j] = p;
    slots[j] = (int32_t)(draw(c.seed, TAG_SLOT, (uint64_t)i, t, (uint64_t)j) % (uint64_t)c.slots);
  }
}

// Eq. 8: squared distance of x to every prototype, direct difference form.
inline void nearest(const float* x, const float* w, int k, int d, int32_t& best, double& d1, double& d2) {
  best = -1; d1 = INFINITY; d2 = INFINITY;
  for (int kk = 0; kk < k; ++kk) {
    double s = 0.0;
    for (int j = 0; j < d; ++j) {
      double df = (double)x[j] - (double)w[(size_t)kk * d + j];
      s += df * df;
    }
    if (s < d1) { d2 = d1; d1 = s; best = kk; }   // strict: first (lowest) index keeps a tie
    else if (s < d2) { d2 = s; }
  }
}

void worker_step_rows(const Oracle& o, Worker& me, const std::vector<double>& D);

// One externally-modified mini-batch step of one worker (Algorithm 5, the "update" line).
void worker_step(const Oracle& o, Worker& me, int32_t i) {
  const Config& c = o.c;
  const int k = c.k, d = c.d, b = c.b;
  const size_t kd = (size_t)k * d;
  const double eps = (double)c.eps;

  // draw the mini-batch: the next b consecutive rows in this worker's (shuffled) batch order
  const int64_t batch = me.perm[me.t % (uint64_t)o.B];
  const float* M = o.X + ((size_t)i * o.H + (size_t)batch * b) * d;

  // assignment (Eq. 8) and per-centre sums / counts (Eq. 9)
  std::vector<double> S(kd, 0.0);
  me.counts.assign(k, 0);
  me.assign.resize(b); me.d1.resize(b); me.d2.resize(b);
  for (int s = 0; s < b; ++s) {
    const float* x = M + (size_t)s * d;
    int32_t a; double e1, e2;
    nearest(x, me.w.data(), k, d, a, e1, e2);
    me.assign[s] = a; me.d1[s] = e1; me.d2[s] = e2;
    me.counts[a] += 1;
    for (int j = 0; j < d; ++j) S[(size_t)a * d + j] += (double)x[j];
  }

  // local gradient (Eq. 9 as the true gradient of Eq. 8, mean over the mini-batch size)
  std::vector<double> D(kd);
  for (int kk = 0; kk < k; ++kk)
    for (int j = 0; j < d; ++j) {
      size_t e = (size_t)kk * d + j;
      D[e] = ((double)me.counts[kk] * (double)me.w[e] - S[e]) / (double)b;
    }

  if (c.partial_rows > 0) { worker_step_rows(o, me, D); return; }

  // receive buffers: lambda (Eq. 3) and delta (Eq. 4)
  const int Sn = c.slots;
  me.acc.assign(Sn, -1); me.lhs.assign(Sn, 0.0); me.rhs.assign(Sn, 0.0);
  std::vector<double> sumv(kd, 0.0);
  int m = 0;
  for (int s = 0; s < Sn; ++s) {
    Slot& sl = me.mail[s];
    if (sl.seq == sl.seen) continue;              // nothing new since the last look
    me.received += 1;
    me.overwritten += (sl.seq - sl.seen - 1);     // messages replaced before they were read
    sl.seen = sl.seq;
    double nv = 0.0, lhs = 0.0, rhs = 0.0;
    for (size_t e = 0; e < kd; ++e) {
      double v = (double)sl.v[e], w = (double)me.w[e];
      nv += v * v;
      double a = (w - eps * D[e]) - v, r = w - v;
      lhs += a * a; rhs += r * r;
    }
    me.lhs[s] = lhs; me.rhs[s] = rhs;
    int lambda = (nv > 0.0) ? 1 : 0;
    int delta = c.parzen ? ((lhs < rhs) ? 1 : 0) : 1;
    int a_s = lambda * delta;
    me.acc[s] = a_s;
    if (a_s) {
      m += 1;
      for (size_t e = 0; e < kd; ++e) sumv[e] += (double)sl.v[e];
    }
  }
  me.accepted += (uint64_t)m;

  // Eq. 6 / Eq. 7 and the update of Algorithm 5
  me.w_next.resize(kd);
  for (size_t e = 0; e < kd; ++e) {
    double w = (double)me.w[e];
    double Dbar = w - (w + sumv[e]) / (double)(1 + m) + D[e];
    me.w_next[e] = (float)(w - eps * Dbar);
  }
}

// The same step when messages carry single centre rows (Section 4.4: K-Means updates are split per
// centre row of the state).  The paper gives no formulas for this case; the reading
// taken here applies Eq. 3, Eq. 4 and Eq. 6 to each centre row k on its own:
//   lambda_{s,k} = 1 if buffer s holds a new message that carries row k and that row is not all zero,
//   delta_{s,k}  = [ ||(w_k - eps D_k) - v_{s,k}||^2 < ||w_k - v_{s,k}||^2 ],
//   Dbar_k = w_k - (w_k + sum_s a_{s,k} v_{s,k}) / (1 + sum_s a_{s,k}) + D_k,   a = lambda * delta.
// A message counts as accepted ("good") when at least one of its rows was.
void worker_step_rows(const Oracle& o, Worker& me, const std::vector<double>& D) {
  const Config& c = o.c;
  const int k = c.k, d = c.d, Sn = c.slots;
  const size_t kd = (size_t)k * d;
  const double eps = (double)c.eps;
  me.acc.assign(Sn, -1); me.lhs.assign(Sn, 0.0); me.rhs.assign(Sn, 0.0);
  me.row_acc.assign((size_t)Sn * k, -1); me.row_lhs.assign((size_t)Sn * k, 0.0); me.row_rhs.assign((size_t)Sn * k, 0.0);
  std::vector<double> sumv(kd, 0.0);
  std::vector<int> mrow(k, 0);
  for (int s = 0; s < Sn; ++s) {
    Slot& sl = me.mail[s];
    if (sl.seq == sl.seen) continue;
    me.received += 1;
    me.overwritten += (sl.seq - sl.seen - 1);
    sl.seen = sl.seq;
    int good_rows = 0;
    for (int kk = 0; kk < k; ++kk) {
      if (!sl.has[kk]) continue;
      double nv = 0.0, lhs = 0.0, rhs = 0.0;
      for (int j = 0; j < d; ++j) {
        size_t e = (size_t)kk * d + j;
        double v = (double)sl.v[e], w = (double)me.w[e];
        nv += v * v;
        double a = (w - eps * D[e]) - v, r = w - v;
        lhs += a * a; rhs += r * r;
      }
      int lambda = (nv > 0.0) ? 1 : 0;
      int delta = c.parzen ? ((lhs < rhs) ? 1 : 0) : 1;
      int a_sk = lambda * delta;
      me.row_acc[(size_t)s * k + kk] = a_sk;
      me.row_lhs[(size_t)s * k + kk] = lhs; me.row_rhs[(size_t)s * k + kk] = rhs;
      if (a_sk) {
        mrow[kk] += 1; good_rows += 1;
        for (int j = 0; j < d; ++j) sumv[(size_t)kk * d + j] += (double)sl.v[(size_t)kk * d + j];
      }
    }
    me.acc[s] = good_rows;
    if (good_rows > 0) me.accepted += 1;
  }
  me.w_next.resize(kd);
  for (int kk = 0; kk < k; ++kk)
    for (int j = 0; j < d; ++j) {
      size_t e = (size_t)kk * d + j;
      double w = (double)me.w[e];
      double Dbar = w - (w + sumv[e]) / (double)(1 + mrow[kk]) + D[e];
      me.w_next[e] = (float)(w - eps * Dbar);
    }
}

// Rows of the j-th message of worker i's put after step t in per-centre mode: m consecutive rows
// (cyclically) from a drawn first row.
void put_rows(const Config& c, int32_t i, uint64_t t, int32_t j, std::vector<uint8_t>& has) {
  has.assign(c.k, 0);
  const int32_t r0 = (int32_t)(draw(c.seed, TAG_ROWS, (uint64_t)i, t, (uint64_t)j) % (uint64_t)c.k);
  for (int32_t q = 0; q < c.partial_rows; ++q) has[(r0 + q) % c.k] = 1;
}

// One synchronous round: every worker steps once from the states and buffers it had at the start
// of the round; afterwards the round's puts are delivered, senders in ascending order, whole
// messages at a time (so a later sender into the same buffer wins).
void round_once(Oracle& o) {
  const Config& c = o.c;
  const int W = c.W;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) num_threads(o.threads)
#endif
  for (int i = 0; i < W; ++i) worker_step(o, o.wk[i], i);

  std::vector<int32_t> peers(c.fanout > 0 ? c.fanout : 1), slots(c.fanout > 0 ? c.fanout : 1);
  for (int i = 0; i < W; ++i) {
    Worker& me = o.wk[i];
    const uint64_t t = me.t;                      // index of the step just done
    if (c.comm_interval > 0 && c.fanout > 0 && W > 1 && (t + 1) % (uint64_t)c.comm_interval == 0) {
      recipients(c, i, t, peers.data(), slots.data());
      for (int j = 0; j < c.fanout; ++j) {
        Slot& sl = o.wk[peers[j]].mail[slots[j]];
        if (c.partial_rows > 0) {
          put_rows(c, i, t, j, sl.has);
          for (int kk = 0; kk < c.k; ++kk)
            if (sl.has[kk]) std::memcpy(sl.v.data() + (size_t)kk * c.d, me.w_next.data() + (size_t)kk * c.d, sizeof(float) * c.d);
        } else {
          sl.v = me.w_next;
          sl.has.assign(c.k, 1);
        }
        sl.seq += 1;
        me.sent += 1;
      }
    }
  }
  for (int i = 0; i < W; ++i) { o.wk[i].w.swap(o.wk[i].w_next); o.wk[i].t += 1; }
}

}  // namespace

extern "C" {

uint64_t oracle_sm64(uint64_t x) { return sm64(x); }
uint64_t oracle_draw(uint64_t seed, uint64_t tag, uint64_t a, uint64_t b, uint64_t c) { return draw(seed, tag, a, b, c); }

// Batch order of one worker without building a whole oracle (same draws as make_perm).
void oracle_batch_order(uint64_t seed, int32_t shuffle, int32_t worker, int64_t B, int32_t* out) {
  Config c{};
  c.seed = seed;
  c.shuffle = shuffle;
  std::vector<int32_t> perm;
  make_perm(c, B, worker, perm);
  std::memcpy(out, perm.data(), sizeof(int32_t) * (size_t)B);
}

void* oracle_create(int64_t N, int32_t d, int32_t k, int32_t W, int32_t b, float eps,
                    int32_t comm_interval, int32_t fanout, int32_t slots, int32_t parzen,
                    int32_t shuffle, uint64_t seed, const float* X, const float* w0) {
  if (N <= 0 || d <= 0 || k <= 0 || W <= 0 || b <= 0 || slots <= 0 || fanout < 0 || fanout > W - 1) return nullptr;
  Oracle* o = new Oracle();
  o->c = Config{N, d, k, W, b, eps, comm_interval, fanout, slots, parzen, shuffle, seed};
  o->X = X;
  o->H = N / W;
  o->B = o->H / b;
  if (o->B < 1) { delete o; return nullptr; }
  o->wk.resize(W);
  const size_t kd = (size_t)k * d;
  for (int i = 0; i < W; ++i) {
    Worker& w = o->wk[i];
    w.w.assign(w0, w0 + kd);
    w.w_next.assign(kd, 0.f);
    w.mail.resize(slots);
    for (auto& s : w.mail) { s.v.assign(kd, 0.f); s.has.assign(k, 0); }
    make_perm(o->c, o->B, i, w.perm);
  }
  return o;
}

void oracle_destroy(void* h) { delete (Oracle*)h; }

int oracle_set_threads(void* h, int n) {
  Oracle* o = (Oracle*)h;
#ifdef _OPENMP
  o->threads = n < 1 ? 1 : n;
#else
  o->threads = 1;
#endif
  return o->threads;
}

void oracle_rounds(void* h, int64_t rounds) {
  Oracle* o = (Oracle*)h;
  for (int64_t r = 0; r < rounds; ++r) round_once(*o);
}

void oracle_get_state(void* h, int32_t worker, float* out) {
  Oracle* o = (Oracle*)h;
  std::memcpy(out, o->wk[worker].w.data(), sizeof(float) * (size_t)o->c.k * o->c.d);
}
void oracle_set_state(void* h, int32_t worker, const float* in) {
  Oracle* o = (Oracle*)h;
  std::memcpy(o->wk[worker].w.data(), in, sizeof(float) * (size_t)o->c.k * o->c.d);
}
// A put from outside the worker set: write a whole message into one receive buffer.
void oracle_put(void* h, int32_t worker, int32_t slot, const float* payload) {
  Oracle* o = (Oracle*)h;
  Slot& s = o->wk[worker].mail[slot];
  s.v.assign(payload, payload + (size_t)o->c.k * o->c.d);
  s.has.assign(o->c.k, 1);
  s.seq += 1;
}
// Per-centre mode: m >= 1 rows per message (0 = whole-state messages).  Set before the first round.
int oracle_set_partial_rows(void* h, int32_t m) {
  Oracle* o = (Oracle*)h;
  if (m < 0 || m > o->c.k) return -1;
  o->c.partial_rows = m;
  return 0;
}
// A put from outside that carries only the rows flagged in has[k].
void oracle_put_rows(void* h, int32_t worker, int32_t slot, const float* payload, const uint8_t* has) {
  Oracle* o = (Oracle*)h;
  Slot& s = o->wk[worker].mail[slot];
  s.v.assign(payload, payload + (size_t)o->c.k * o->c.d);
  s.has.assign(has, has + o->c.k);
  s.seq += 1;
}
// Rows of the j-th message of worker i's put after step t (flags, k of them).
void oracle_put_row_flags(void* h, int32_t i, uint64_t t, int32_t j, uint8_t* out) {
  Oracle* o = (Oracle*)h;
  std::vector<uint8_t> has;
  put_rows(o->c, i, t, j, has);
  std::memcpy(out, has.data(), (size_t)o->c.k);
}
// Per-row trace of the last step in per-centre mode: acc[S*k] (-1 = row not in a new message), lhs, rhs.
void oracle_last_step_rows(void* h, int32_t worker, int32_t* acc, double* lhs, double* rhs) {
  Worker& w = ((Oracle*)h)->wk[worker];
  if (w.row_acc.empty()) return;
  if (acc) std::memcpy(acc, w.row_acc.data(), sizeof(int32_t) * w.row_acc.size());
  if (lhs) std::memcpy(lhs, w.row_lhs.data(), sizeof(double) * w.row_lhs.size());
  if (rhs) std::memcpy(rhs, w.row_rhs.data(), sizeof(double) * w.row_rhs.size());
}
// has[k] flags of a receive buffer's last message.
void oracle_get_mail_rows(void* h, int32_t worker, int32_t slot, uint8_t* out) {
  Oracle* o = (Oracle*)h;
  std::memcpy(out, o->wk[worker].mail[slot].has.data(), (size_t)o->c.k);
}
// Content and counters of a receive buffer: out[k*d], seq_seen[2] = {seq, seen}.
void oracle_get_mail(void* h, int32_t worker, int32_t slot, float* out, uint64_t* seq_seen) {
  Oracle* o = (Oracle*)h;
  Slot& s = o->wk[worker].mail[slot];
  std::memcpy(out, s.v.data(), sizeof(float) * (size_t)o->c.k * o->c.d);
  seq_seen[0] = s.seq; seq_seen[1] = s.seen;
}
// out[5] = steps, sent, received, accepted ("good"), overwritten
void oracle_get_stats(void* h, int32_t worker, uint64_t* out) {
  Worker& w = ((Oracle*)h)->wk[worker];
  out[0] = w.t; out[1] = w.sent; out[2] = w.received; out[3] = w.accepted; out[4] = w.overwritten;
}
void oracle_get_perm(void* h, int32_t worker, int32_t* out) {
  Oracle* o = (Oracle*)h;
  std::memcpy(out, o->wk[worker].perm.data(), sizeof(int32_t) * (size_t)o->B);
}
int64_t oracle_batches_per_pass(void* h) { return ((Oracle*)h)->B; }
int64_t oracle_shard_rows(void* h) { return ((Oracle*)h)->H; }
// Recipients and buffers of the put that worker i makes after its step t.
void oracle_recipients(void* h, int32_t i, uint64_t t, int32_t* peers, int32_t* slots) {
  recipients(((Oracle*)h)->c, i, t, peers, slots);
}
// Trace of the worker's last step.
void oracle_last_step(void* h, int32_t worker, int32_t* assign, double* d1, double* d2,
                      int64_t* counts, int32_t* acc, double* lhs, double* rhs) {
  Oracle* o = (Oracle*)h;
  Worker& w = o->wk[worker];
  if (w.assign.empty()) return;
  if (assign) std::memcpy(assign, w.assign.data(), sizeof(int32_t) * w.assign.size());
  if (d1) std::memcpy(d1, w.d1.data(), sizeof(double) * w.d1.size());
  if (d2) std::memcpy(d2, w.d2.data(), sizeof(double) * w.d2.size());
  if (counts) std::memcpy(counts, w.counts.data(), sizeof(int64_t) * w.counts.size());
  if (acc) std::memcpy(acc, w.acc.data(), sizeof(int32_t) * w.acc.size());
  if (lhs) std::memcpy(lhs, w.lhs.data(), sizeof(double) * w.lhs.size());
  if (rhs) std::memcpy(rhs, w.rhs.data(), sizeof(double) * w.rhs.size());
}

// Eq. 8 text: nearest prototype of each of n rows (plus the two smallest squared distances).
void oracle_assign(const float* X, int64_t n, int32_t d, const float* w, int32_t k,
                   int32_t* assign, double* d1, double* d2) {
  for (int64_t r = 0; r < n; ++r) {
    int32_t a; double e1, e2;
    nearest(X + (size_t)r * d, w, k, d, a, e1, e2);
    assign[r] = a;
    if (d1) d1[r] = e1;
    if (d2) d2[r] = e2;
  }
}

// Eq. 8: E(w) = sum_i 1/2 ||x_i - w_{s_i(w)}||^2 over n rows.
double oracle_eval(const float* X, int64_t n, int32_t d, const float* w, int32_t k, int threads) {
  double E = 0.0;
#ifdef _OPENMP
#pragma omp parallel for schedule(static) reduction(+ : E) num_threads(threads < 1 ? 1 : threads)
#endif
  for (int64_t r = 0; r < n; ++r) {
    int32_t a; double e1, e2;
    nearest(X + (size_t)r * d, w, k, d, a, e1, e2);
    E += 0.5 * e1;
  }
  return E;
}

int oracle_max_threads() {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"
