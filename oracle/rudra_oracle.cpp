// Rudra parameter-server oracle: TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// A plain, slow, single-threaded CPU statement of what the parameter server of
// arXiv 1509.04210 computes: the n-softsync protocol (Section 3.1, Eq. 5), the
// scalar timestamp / staleness / vector clock bookkeeping (Section 3.1, Eq. 2),
// the staleness-modulated learning rate (Section 5.1, Eq. 6), the weight update
// (Eq. 1c / 3 / 4 / 5) and pullWeights (Section 2, Section 3.2).  Floating
// point is carried in double and stored as fp32 (the paper's precision,
// Section 4.2).  Nothing is blocked, fused, vectorised or threaded.
//
// This file shares no code with the CUDA library and is never linked into it.
// Only tests, the smoke check and the benchmark's CPU-baseline leg use it.
//
// Parity status of the parts the paper does not write out:
//   * momentum / weight-decay form         : parity unpinned by the paper
//     (the paper names "momentum 0.9" and a "weight regularization penalty"
//     in Section 4.2 but prints no formula); the reading stated at
//     OraclePS::step below is pinned by closed forms and, at a constant rate,
//     by the trajectory of a library optimizer (torch.optim.SGD in float64).
//   * sigma = 0 floor in the per-gradient and group-mean rate policies
//     (alpha0/sigma is undefined at sigma = 0)  : parity unpinned by the paper.
//   * AdaGrad form (Section 5.5 names the method, prints no formula)
//                                           : parity unpinned by the paper; the
//     reading at OraclePS::step is pinned by the direction of the first step
//     (the sign of gradient plus penalty), by a decay-only scalar recurrence
//     and by brute force in decimal arithmetic with unequal per-gradient rates,
//     and at a constant rate by torch.optim.Adagrad's trajectory in float64.
//   * Rudra-adv's server tree (Section 3.3 says that a leaf averages its
//     learners' gradients and relays the average to its parent, and that the
//     root applies the update; it does not say when a leaf relays, which
//     timestamp a relayed average carries or which rate it gets)
//                                           : parity unpinned by the paper; the
//     reading at OraclePS::push_relay is pinned by its reduction to the flat
//     server (fan-in 1 bit for bit; equal rates to rounding, Eq. 7's argument)
//     and by hand-computed step sizes.
// Everything else is pinned by Eq. 2-6 and the staleness sets printed in
// Section 5.1 (see tests/).
//
// A second evaluation mode ("strict") carries the same rule in fp32 with one
// fused multiply-add per term, gradients in arrival order.  It is a debugging
// aid that lets an fp32 implementation be compared bit for bit; the parity
// criterion is the double-precision mode.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <deque>
#include <vector>

namespace {

// ---------------------------------------------------------------------------
// Counter-based generator: SplitMix64 (Steele, Lea, Flood 2014), from its
// published definition.  Each use draws from its own stream.
// ---------------------------------------------------------------------------
struct SplitMix64 {
  uint64_t s;
  explicit SplitMix64(uint64_t seed) : s(seed) {}
  uint64_t next() {
    s += 0x9E3779B97F4A7C15ull;
    uint64_t z = s;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
  }
};

// Stream state for (seed, purpose, id): purposes are 1 = push-order
// permutations, 2 = a learner's compute times.
uint64_t stream_state(uint64_t seed, uint64_t purpose, uint64_t id) {
  return seed ^ (purpose << 48) ^ id;
}

enum EventKind : int32_t {
  EV_PUSH = 1,       // learner's gradient arrives; pulled_ts = timestamp of the weights it used
  EV_STEP = 2,       // weights advance; ts = the new timestamp
  EV_PULL = 3,       // learner receives the weights; ts = their timestamp
  EV_PULL_SKIP = 4,  // timestamp inquiry found the learner's copy current (Section 3.2)
  EV_BROADCAST = 5,  // every learner receives the weights with timestamp ts
  EV_RELAY = 6,      // tree (Section 3.3): leaf `learner` sends the average of its last k gradients to the root
};

enum SchedMode : int32_t {
  MODE_HARDSYNC = 0,
  MODE_SOFTSYNC_ROUNDS = 1,
  MODE_SOFTSYNC_TIMED = 2,
};

struct Event {
  int32_t kind;
  uint32_t learner;
  uint64_t pulled_ts;
  uint64_t ts;
  uint64_t seq;   // PUSH: index of this learner's mini-batch (0-based); else 0
  uint64_t tick;  // simulated time of the event (timed mode), else the global push count
};

// ---------------------------------------------------------------------------
// Learner event model (Section 2 learner loop; Section 3.2: a learner pulls
// before each mini-batch, inquiring the timestamp first; the server handles
// messages strictly one at a time).
// ---------------------------------------------------------------------------
struct OracleSched {
  uint32_t lambda, n, c;
  int32_t mode;
  bool downcast;          // weights broadcast to every learner after each update (Section 3.3)
  double ln_sigma;
  uint64_t ts = 0;        // server timestamp, starts at 0 (Section 3.1)
  uint64_t pushes = 0;    // gradients that have reached the (root) server so far
  // Server tree of Section 3.3, two levels: learner l sends to leaf l / fanin; a leaf that holds
  // fanin gradients relays their average to the root at once.  fanin = 0: no tree, learners
  // send to the server directly.
  uint32_t fanin = 0;
  std::vector<uint32_t> leaf_fill;   // gradients waiting at each leaf
  std::vector<uint64_t> leaf_relays; // averages each leaf has relayed
  std::vector<uint64_t> local_ts;   // timestamp of the weights last delivered to each learner
  std::vector<uint64_t> grad_ts;    // timestamp of the weights its current mini-batch started from
  std::vector<uint64_t> nbatch;     // mini-batches each learner has pushed
  uint64_t handled = 0;             // push messages handled so far (rounds mode: the event tick)
  std::deque<Event> out;
  // rounds
  SplitMix64 perm_rng;
  // timed
  std::vector<SplitMix64> time_rng;
  std::vector<uint64_t> next_push;

  OracleSched(uint32_t lambda_, uint32_t n_, int32_t mode_, uint64_t seed, double ln_sigma_, bool downcast_,
              uint32_t fanin_ = 0)
      : lambda(lambda_), n(n_), c(lambda_ / n_), mode(mode_), downcast(downcast_), ln_sigma(ln_sigma_),
        fanin(fanin_), leaf_fill(fanin_ ? lambda_ / fanin_ : 0, 0), leaf_relays(fanin_ ? lambda_ / fanin_ : 0, 0),
        local_ts(lambda_, 0), grad_ts(lambda_, 0), nbatch(lambda_, 0), perm_rng(stream_state(seed, 1, 0)) {
    if (mode == MODE_SOFTSYNC_TIMED) {
      for (uint32_t l = 0; l < lambda; ++l) time_rng.emplace_back(stream_state(seed, 2, l));
      next_push.resize(lambda);
      for (uint32_t l = 0; l < lambda; ++l) next_push[l] = draw_ticks(l);  // all start at time 0
    }
  }

  // One compute time: lognormal(0, ln_sigma) in units of 2^-20, Box-Muller cosine branch.
  uint64_t draw_ticks(uint32_t l) {
    uint64_t a = time_rng[l].next() >> 11;
    uint64_t b = time_rng[l].next() >> 11;
    double u1 = (double)(a + 1) * 0x1.0p-53;   // (0, 1]
    double u2 = (double)b * 0x1.0p-53;         // [0, 1)
    double z = std::sqrt(-2.0 * std::log(u1)) * std::cos(6.283185307179586476925286766559 * u2);
    long long t = std::llround(std::exp(ln_sigma * z) * 1048576.0);
    return t < 1 ? 1ull : (uint64_t)t;
  }

  void emit(int32_t kind, uint32_t l, uint64_t pulled, uint64_t ts_, uint64_t seq, uint64_t tick) {
    out.push_back(Event{kind, l, pulled, ts_, seq, tick});
  }

  // The server handles learner l's push completely -- including the update it
  // may trigger -- before that learner's pull.
  void handle_push(uint32_t l, uint64_t tick) {
    emit(EV_PUSH, l, grad_ts[l], ts, nbatch[l], tick);
    nbatch[l] += 1;
    bool arrived = true;            // did gradients reach the root with this message?
    if (fanin == 0) {
      pushes += 1;
    } else {
      const uint32_t leaf = l / fanin;
      if (++leaf_fill[leaf] == fanin) {   // the leaf averages what it holds and relays it (Section 3.3)
        leaf_fill[leaf] = 0;
        emit(EV_RELAY, leaf, 0, ts, leaf_relays[leaf]++, tick);
        pushes += fanin;            // the average stands for fanin gradients
      } else {
        arrived = false;
      }
    }
    bool stepped = false;
    if (arrived && pushes % c == 0) {   // exactly c gradients per update (Eq. 5)
      ts += 1;                      // one increment per weight update (Section 3.1)
      stepped = true;
      emit(EV_STEP, l, 0, ts, 0, tick);
    }
    if (mode == MODE_HARDSYNC) {
      if (stepped) {                // new weights go to all learners (Section 3.1, hardsync)
        emit(EV_BROADCAST, 0, 0, ts, 0, tick);
        for (uint32_t k = 0; k < lambda; ++k) local_ts[k] = grad_ts[k] = ts;   // all wait at the barrier
      }
      return;
    }
    if (stepped && downcast) {
      // Weights reach every learner's receive buffer in the background; a learner in the middle
      // of a mini-batch keeps computing on the weights it started from (Section 3.3).
      emit(EV_BROADCAST, 0, 0, ts, 0, tick);
      for (uint32_t k = 0; k < lambda; ++k) local_ts[k] = ts;
    }
    if (local_ts[l] == ts) {
      emit(EV_PULL_SKIP, l, 0, ts, 0, tick);
    } else {
      local_ts[l] = ts;
      emit(EV_PULL, l, 0, ts, 0, tick);
    }
    grad_ts[l] = local_ts[l];       // the learner starts its next mini-batch from these weights
  }

  void refill() {
    if (mode == MODE_SOFTSYNC_TIMED) {
      uint32_t best = 0;            // earliest push; ties go to the smaller learner id
      for (uint32_t l = 1; l < lambda; ++l)
        if (next_push[l] < next_push[best]) best = l;
      uint64_t t = next_push[best];
      handle_push(best, t);
      next_push[best] = t + draw_ticks(best);
      return;
    }
    // One round: every learner pushes exactly once, in a fresh seeded order.
    std::vector<uint32_t> perm(lambda);
    for (uint32_t i = 0; i < lambda; ++i) perm[i] = i;
    for (uint32_t i = lambda - 1; i >= 1; --i) {
      uint32_t j = (uint32_t)(perm_rng.next() % (uint64_t)(i + 1));
      std::swap(perm[i], perm[j]);
    }
    for (uint32_t i = 0; i < lambda; ++i) handle_push(perm[i], ++handled);
  }

  Event next() {
    while (out.empty()) refill();
    Event e = out.front();
    out.pop_front();
    return e;
  }
};

// ---------------------------------------------------------------------------
// Parameter server state and the update rule.
// ---------------------------------------------------------------------------
enum LrPolicy : int32_t { LR_PAPER_N = 0, LR_PER_GRADIENT = 1, LR_GROUP_MEAN = 2 };
enum GradDtype : int32_t { GRAD_F32 = 0, GRAD_BF16 = 1 };
enum Optimizer : int32_t { OPT_MOMENTUM_SGD = 0, OPT_ADAGRAD = 1 };

// One message in the server's queue: a learner's gradient (fan-in 1), or the average that a
// leaf of the server tree relays for `fanin` of its learners' gradients (Section 3.3).  Either
// way it carries the timestamp of every gradient it stands for.
struct Message {
  const void* grad = nullptr;        // fan-in 1: the learner's buffer (borrowed)
  std::vector<float> avg;            // relay: the leaf's average, a 32-bit float vector like every message
  uint32_t fanin = 1;
  std::vector<uint64_t> pulled_ts;   // fanin entries
};

struct OraclePS {
  uint64_t N;
  uint32_t lambda, n, c;
  float alpha0, momentum, wd;
  int32_t policy = LR_PAPER_N;
  int32_t dtype = GRAD_F32;
  int32_t optimizer = OPT_MOMENTUM_SGD;
  float adagrad_eps = 1e-8f;
  bool strict = false;             // fp32 evaluation, one fmaf per term (debugging aid)
  std::vector<float> theta, vel;   // vel: velocity (momentum SGD) or squared-gradient sum (AdaGrad)
  uint64_t ts = 0;
  std::deque<Message> fifo;
  uint64_t queued = 0;             // gradients the queued messages stand for
  // record of the most recent update
  std::vector<uint64_t> clock;     // vector clock <p_1..p_c> (Section 3.1)
  std::vector<uint32_t> sigma;
  std::vector<float> scale;        // per gradient: its message's step size over the message's fan-in
  std::vector<float> msg_step;     // per message: the step size its vector is multiplied by
  std::vector<uint32_t> msg_fanin;
  float abar = 0.f;
  double avg_sigma = 0.0;

  OraclePS(uint64_t N_, uint32_t lambda_, uint32_t n_, float a0, float m, float wd_)
      : N(N_), lambda(lambda_), n(n_), c(lambda_ / n_), alpha0(a0), momentum(m), wd(wd_),
        theta(N_, 0.f), vel(N_, 0.f) {}

  double grad_at(const void* g, uint64_t k) const {
    if (dtype == GRAD_F32) return (double)((const float*)g)[k];
    uint32_t bits = (uint32_t)((const uint16_t*)g)[k] << 16;   // bf16 is the top half of an fp32
    float f;
    std::memcpy(&f, &bits, 4);
    return (double)f;
  }

  double value_at(const Message& m, uint64_t k) const {
    return m.fanin == 1 && m.avg.empty() ? grad_at(m.grad, k) : (double)m.avg[k];
  }

  int64_t push(const void* g, uint64_t pulled_ts) {
    if (pulled_ts > ts) return -2;          // weights with that timestamp do not exist yet (Section 3.1)
    Message m;
    m.grad = g;
    m.pulled_ts.assign(1, pulled_ts);
    fifo.push_back(std::move(m));
    queued += 1;
    return (int64_t)queued;
  }

  // A leaf of the server tree (Section 3.3): averages the k gradients its learners sent, in
  // arrival order, and relays the average to the root, which is this server.  Reading: the relay
  // happens as soon as the leaf holds k gradients; the message carries all k timestamps, so the
  // root's vector clock and Eq. 2 are those of a server that received the k gradients itself; a
  // relayed average stands for k of the c gradients of an update and never straddles two updates.
  int64_t push_relay(const void* const* g, const uint64_t* pulled, uint32_t k) {
    if (k == 0 || k > c) return -1;
    for (uint32_t l = 0; l < k; ++l)
      if (pulled[l] > ts) return -2;
    if (queued % c + k > c) return -5;
    Message m;
    m.fanin = k;
    m.pulled_ts.assign(pulled, pulled + k);
    m.avg.resize(N);
    if (strict) {
      const float inv_k = (float)(1.0 / (double)k);
      for (uint64_t i = 0; i < N; ++i) {
        float acc = 0.f;
        for (uint32_t l = 0; l < k; ++l) acc = std::fmaf(inv_k, (float)grad_at(g[l], i), acc);
        m.avg[i] = acc;
      }
    } else {
      for (uint64_t i = 0; i < N; ++i) {
        double sum = 0.0;
        for (uint32_t l = 0; l < k; ++l) sum += grad_at(g[l], i);
        m.avg[i] = (float)(sum / (double)k);   // the relayed message is a 32-bit float vector (Section 4.2)
      }
    }
    fifo.push_back(std::move(m));
    queued += k;
    return (int64_t)queued;
  }

  int step() {
    if (queued < c) return 0;
    // the leading messages that together stand for exactly c gradients
    std::vector<Message> grp;
    for (uint32_t have = 0; have < c;) {
      have += fifo.front().fanin;
      grp.push_back(std::move(fifo.front()));
      fifo.pop_front();
    }
    queued -= c;
    const uint32_t nmsg = (uint32_t)grp.size();
    // staleness of each gradient: server timestamp j minus gradient timestamp i (Section 3.1)
    clock.assign(c, 0);
    sigma.assign(c, 0);
    std::vector<uint64_t> msg_sigma(nmsg, 0);   // sum of the staleness of the gradients a message stands for
    uint64_t sum_sigma = 0, sum_p = 0;
    uint32_t l = 0;
    for (uint32_t j = 0; j < nmsg; ++j) {
      for (uint64_t p : grp[j].pulled_ts) {
        clock[l] = p;
        sigma[l] = (uint32_t)(ts - p);
        msg_sigma[j] += sigma[l];
        sum_sigma += sigma[l];
        sum_p += p;
        ++l;
      }
    }
    // Eq. 2: <sigma> = (i-1) - mean(i_1..i_c), (i-1) being the timestamp before this update.
    avg_sigma = (double)ts - (double)sum_p / (double)c;
    // Step size of each message: learning rate (Eq. 6, or a variant of it) times the share k/c of
    // Eq. 5's average that the message stands for (k = 1 for a learner's own gradient: 1/c).
    msg_step.assign(nmsg, 0.f);
    msg_fanin.assign(nmsg, 0);
    scale.assign(c, 0.f);
    double sum_s = 0.0;
    l = 0;
    for (uint32_t j = 0; j < nmsg; ++j) {
      const double k = (double)grp[j].fanin;
      double num = (double)alpha0 * k, div;
      if (policy == LR_PAPER_N) {
        div = (double)n * (double)c;                                   // alpha0 / n, Eq. 6
      } else if (policy == LR_PER_GRADIENT) {
        // alpha0 / sigma of the message (Section 5.1 footnote): the mean staleness of the gradients
        // it stands for, floored at 1; alpha0 / max(sum/k, 1) = alpha0 k / max(sum, k)
        num *= k;
        div = (double)std::max<uint64_t>(msg_sigma[j], (uint64_t)grp[j].fanin) * (double)c;
      } else {
        div = (double)std::max<uint64_t>(sum_sigma, (uint64_t)c);      // alpha0 / <sigma> of Eq. 2, then k / c
      }
      msg_step[j] = (float)(num / div);
      msg_fanin[j] = grp[j].fanin;
      sum_s += (double)msg_step[j];
      for (uint32_t i = 0; i < grp[j].fanin; ++i) scale[l++] = (float)((double)msg_step[j] / k);
    }
    abar = (float)sum_s;   // the group's learning rate: sum of the step sizes

    if (strict) {
      step_strict(grp);
      ts += 1;
      return 1;
    }
    for (uint64_t k = 0; k < N; ++k) {
      if (optimizer == OPT_MOMENTUM_SGD) {
        // sumGradients: staleness-scaled average of the c gradients (Eq. 5 with Eq. 6 folded in)
        double acc = 0.0;
        for (uint32_t j = 0; j < nmsg; ++j) acc += (double)msg_step[j] * value_at(grp[j], k);
        // applyUpdate, reading: L2 penalty joins the gradient at the group's rate; heavy-ball
        // velocity carries the learning rate; with momentum = wd = 0 this is Eq. 5 exactly.
        double u = acc + (double)abar * (double)wd * (double)theta[k];
        double v = (double)momentum * (double)vel[k] + u;
        double th = (double)theta[k] - v;
        vel[k] = (float)v;
        theta[k] = (float)th;
      } else {
        // AdaGrad at the server (Section 5.5), reading: the averaged gradient of Eq. 5 plus the
        // L2 penalty feeds a running sum of squares; the step is rate * g / (sqrt(sum) + eps).
        // (with a zero rate every step size is 0: the weights are then Eq. 5's plain k/c)
        double gbar = 0.0;
        for (uint32_t j = 0; j < nmsg; ++j)
          gbar += (abar > 0.f ? (double)msg_step[j] / (double)abar : (double)grp[j].fanin / (double)c) * value_at(grp[j], k);
        gbar += (double)wd * (double)theta[k];
        double h = (double)vel[k] + gbar * gbar;
        double th = (double)theta[k] - (double)abar * gbar / (std::sqrt(h) + (double)adagrad_eps);
        vel[k] = (float)h;
        theta[k] = (float)th;
      }
    }
    ts += 1;   // each weight update increments the timestamp by one (Section 3.1)
    return 1;
  }

  // The same rule in fp32: acc = fma(s_j, g_j, acc) over the messages from acc = 0, then one fma per
  // remaining term.  Same reading of momentum / decay / AdaGrad as above.
  void step_strict(const std::vector<Message>& grp) {
    const float awd = (float)((double)abar * (double)wd);
    const uint32_t nmsg = (uint32_t)grp.size();
    for (uint64_t k = 0; k < N; ++k) {
      float acc = 0.f;
      if (optimizer == OPT_MOMENTUM_SGD) {
        for (uint32_t j = 0; j < nmsg; ++j) acc = std::fmaf(msg_step[j], (float)value_at(grp[j], k), acc);
        const float u = std::fmaf(awd, theta[k], acc);
        const float v = momentum != 0.f ? std::fmaf(momentum, vel[k], u) : u;
        theta[k] = theta[k] - v;
        vel[k] = v;
      } else {
        for (uint32_t j = 0; j < nmsg; ++j) {
          const float wj = abar > 0.f ? (float)((double)msg_step[j] / (double)abar) : (float)((double)grp[j].fanin / (double)c);
          acc = std::fmaf(wj, (float)value_at(grp[j], k), acc);
        }
        const float g = std::fmaf(wd, theta[k], acc);
        const float h = std::fmaf(g, g, vel[k]);
        const float num = abar * g;
        const float den = std::sqrt(h) + adagrad_eps;
        theta[k] = theta[k] - num / den;
        vel[k] = h;
      }
    }
  }

  int64_t pull(float* dst) const {   // pullWeights: the weights and their timestamp (Section 3.2)
    for (uint64_t k = 0; k < N; ++k) dst[k] = theta[k];
    return (int64_t)ts;
  }
};

}  // namespace

extern "C" {

void ora_splitmix64(uint64_t seed, uint64_t count, uint64_t* out) {
  SplitMix64 g(seed);
  for (uint64_t i = 0; i < count; ++i) out[i] = g.next();
}

void* ora_sched_create_tree(uint32_t lambda, uint32_t n, int32_t mode, uint64_t seed, double ln_sigma, int32_t downcast,
                            uint32_t fanin) {
  if (lambda == 0 || n == 0 || n > lambda) return nullptr;
  if (mode < 0 || mode > 2) return nullptr;
  if (mode == MODE_HARDSYNC && n != 1) return nullptr;
  // a leaf's average stands for fanin of the c gradients of one update, and every learner has a leaf
  if (fanin != 0 && (lambda % fanin != 0 || (lambda / n) % fanin != 0)) return nullptr;
  return new OracleSched(lambda, n, mode, seed, ln_sigma, downcast != 0, fanin);
}
void* ora_sched_create(uint32_t lambda, uint32_t n, int32_t mode, uint64_t seed, double ln_sigma, int32_t downcast) {
  return ora_sched_create_tree(lambda, n, mode, seed, ln_sigma, downcast, 0);
}
void ora_sched_destroy(void* s) { delete (OracleSched*)s; }
// A learner reports the timestamp of the weights it really computes on (a late or lost pull).
int32_t ora_sched_on_pull(void* s, uint32_t learner, uint64_t ts) {
  OracleSched* S = (OracleSched*)s;
  if (learner >= S->lambda) return -1;
  if (ts > S->ts) return -2;
  S->local_ts[learner] = S->grad_ts[learner] = ts;
  return 0;
}
// Writes count events into out (6 x 8-byte fields each: kind|learner packed as two 32-bit words,
// pulled_ts, ts, seq, tick).
void ora_sched_run(void* s, uint64_t count, Event* out) {
  OracleSched* S = (OracleSched*)s;
  for (uint64_t i = 0; i < count; ++i) out[i] = S->next();
}

void* ora_ps_create(uint64_t N, uint32_t lambda, uint32_t n, float alpha0, float momentum, float wd) {
  if (N == 0 || lambda == 0 || n == 0 || n > lambda) return nullptr;
  return new OraclePS(N, lambda, n, alpha0, momentum, wd);
}
void ora_ps_destroy(void* p) { delete (OraclePS*)p; }
void ora_ps_set_policy(void* p, int32_t policy) { ((OraclePS*)p)->policy = policy; }
void ora_ps_set_grad_dtype(void* p, int32_t dtype) { ((OraclePS*)p)->dtype = dtype; }
void ora_ps_set_optimizer(void* p, int32_t opt, float eps) {
  ((OraclePS*)p)->optimizer = opt;
  ((OraclePS*)p)->adagrad_eps = eps;
}
void ora_ps_set_strict(void* p, int32_t on) { ((OraclePS*)p)->strict = on != 0; }
void ora_ps_set_alpha0(void* p, float a0) { ((OraclePS*)p)->alpha0 = a0; }
void ora_ps_set_weights(void* p, const float* src) {
  OraclePS* P = (OraclePS*)p;
  for (uint64_t k = 0; k < P->N; ++k) { P->theta[k] = src[k]; P->vel[k] = 0.f; }
  P->ts = 0;
  P->fifo.clear();
  P->queued = 0;
}
int64_t ora_ps_push(void* p, const void* grad, uint64_t pulled_ts) { return ((OraclePS*)p)->push(grad, pulled_ts); }
int64_t ora_ps_push_relay(void* p, const void* const* grads, const uint64_t* pulled_ts, uint32_t k) {
  return ((OraclePS*)p)->push_relay(grads, pulled_ts, k);
}
// Step sizes of the most recent update's messages and the number of gradients each stands for.
int32_t ora_ps_last_messages(void* p, float* step, uint32_t* fanin) {
  OraclePS* P = (OraclePS*)p;
  for (size_t j = 0; j < P->msg_step.size(); ++j) {
    if (step) step[j] = P->msg_step[j];
    if (fanin) fanin[j] = P->msg_fanin[j];
  }
  return (int32_t)P->msg_step.size();
}
int32_t ora_ps_step(void* p) { return ((OraclePS*)p)->step(); }
int64_t ora_ps_pull(void* p, float* dst) { return ((OraclePS*)p)->pull(dst); }
int64_t ora_ps_timestamp(void* p) { return (int64_t)((OraclePS*)p)->ts; }
void ora_ps_state(void* p, float* vel_out) {
  OraclePS* P = (OraclePS*)p;
  for (uint64_t k = 0; k < P->N; ++k) vel_out[k] = P->vel[k];
}
int32_t ora_ps_last_clock(void* p, uint64_t* pulled, uint32_t* sigma, float* scale, double* avg_sigma, float* abar) {
  OraclePS* P = (OraclePS*)p;
  uint32_t c = (uint32_t)P->clock.size();
  for (uint32_t l = 0; l < c; ++l) {
    if (pulled) pulled[l] = P->clock[l];
    if (sigma) sigma[l] = P->sigma[l];
    if (scale) scale[l] = P->scale[l];
  }
  if (avg_sigma) *avg_sigma = P->avg_sigma;
  if (abar) *abar = P->abar;
  return (int32_t)c;
}

}  // extern "C"
