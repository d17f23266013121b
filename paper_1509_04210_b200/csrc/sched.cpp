// Host-side learner event scheduler (no CUDA): the arrival order of pushGradient / pullWeights
// messages for lambda simulated learners.  The server of Section 3.2 handles messages one at a
// time, so this total order is the whole protocol state besides the weights: server timestamp
// (Section 3.1), each learner's delivered and in-use weight timestamps, group boundaries every
// c = floor(lambda / n) pushes (Eq. 5).
#include <cmath>
#include <cstdint>
#include <new>
#include <queue>
#include <utility>
#include <vector>

#include "../../include/rudra_ps.h"

namespace {

// SplitMix64 (Steele, Lea, Flood 2014): additive Weyl sequence + 64-bit finalizer.
class Rng {
 public:
  explicit Rng(uint64_t state) : state_(state) {}
  uint64_t operator()() {
    uint64_t z = (state_ += UINT64_C(0x9E3779B97F4A7C15));
    z ^= z >> 30; z *= UINT64_C(0xBF58476D1CE4E5B9);
    z ^= z >> 27; z *= UINT64_C(0x94D049BB133111EB);
    z ^= z >> 31;
    return z;
  }
 private:
  uint64_t state_;
};

constexpr uint64_t kPurposeOrder = 1;   // push-order permutations
constexpr uint64_t kPurposeTime = 2;    // per-learner compute times

inline uint64_t substream(uint64_t seed, uint64_t purpose, uint64_t id) {
  return seed ^ (purpose << 48) ^ id;
}

}  // namespace

struct rudra_sched {
  uint32_t lambda, n, c;
  int mode;
  bool downcast;
  double spread;

  uint32_t fanin;                       // learners per leaf of the server tree (Section 3.3); 0 = no tree
  std::vector<uint32_t> at_leaf;        // gradients each leaf holds
  std::vector<uint64_t> relayed;        // averages each leaf has sent up
  uint64_t at_root = 0;                 // gradients that have reached the root (directly or averaged)

  uint64_t server_ts = 0;
  uint64_t handled = 0;                 // pushes handled so far
  std::vector<uint64_t> delivered_ts;   // timestamp of the weights in each learner's receive buffer
  std::vector<uint64_t> in_use_ts;      // timestamp of the weights its running mini-batch uses
  std::vector<uint64_t> batches;        // mini-batches pushed per learner

  Rng order_rng;
  std::vector<Rng> time_rng;
  using Arrival = std::pair<uint64_t, uint32_t>;   // (tick, learner): lexicographic = time, then id
  std::priority_queue<Arrival, std::vector<Arrival>, std::greater<Arrival>> arrivals;

  std::vector<uint32_t> round;          // current round's push order
  uint32_t round_pos = 0;

  std::vector<rudra_event> pending;     // events produced by the push being handled
  size_t pending_pos = 0;

  rudra_sched(uint32_t lam, uint32_t n_, int mode_, uint64_t seed, double spread_, bool downcast_, uint32_t fanin_)
      : lambda(lam), n(n_), c(lam / n_), mode(mode_), downcast(downcast_), spread(spread_), fanin(fanin_),
        at_leaf(fanin_ ? lam / fanin_ : 0, 0), relayed(fanin_ ? lam / fanin_ : 0, 0),
        delivered_ts(lam, 0), in_use_ts(lam, 0), batches(lam, 0), order_rng(substream(seed, kPurposeOrder, 0)) {
    if (mode == RUDRA_SCHED_SOFTSYNC_TIMED) {
      time_rng.reserve(lam);
      for (uint32_t l = 0; l < lam; ++l) {
        time_rng.emplace_back(substream(seed, kPurposeTime, l));
        arrivals.emplace(compute_ticks(l), l);   // everyone pulls timestamp 0 at time 0
      }
    } else {
      round_pos = lam;   // forces a fresh order on first use
    }
  }

  // lognormal(0, spread) compute time in 2^-20 units; standard normal by Box-Muller (cosine branch)
  // from two 53-bit uniforms, the first shifted into (0, 1].
  uint64_t compute_ticks(uint32_t l) {
    const uint64_t a = time_rng[l]() >> 11, b = time_rng[l]() >> 11;
    const double u1 = std::ldexp((double)(a + 1), -53);
    const double u2 = std::ldexp((double)b, -53);
    const double z = std::sqrt(-2.0 * std::log(u1)) * std::cos(6.283185307179586476925286766559 * u2);
    const long long t = std::llround(std::exp(spread * z) * 1048576.0);
    return t < 1 ? UINT64_C(1) : (uint64_t)t;
  }

  void shuffle_round() {
    round.resize(lambda);
    for (uint32_t i = 0; i < lambda; ++i) round[i] = i;
    for (uint32_t i = lambda; i-- > 1;) {                 // Fisher-Yates, i = lambda-1 .. 1
      const uint32_t j = (uint32_t)(order_rng() % (uint64_t)(i + 1));
      std::swap(round[i], round[j]);
    }
    round_pos = 0;
  }

  void add(int32_t kind, uint32_t learner, uint64_t pulled, uint64_t ts, uint64_t seq, uint64_t tick) {
    pending.push_back(rudra_event{kind, learner, pulled, ts, seq, tick});
  }

  // One pushGradient message, handled to completion (update included) before the same learner's
  // pullWeights is served.
  void on_push(uint32_t l, uint64_t tick) {
    add(RUDRA_EV_PUSH, l, in_use_ts[l], server_ts, batches[l]++, tick);
    ++handled;
    bool closes_group = false;
    if (fanin == 0) {
      closes_group = ++at_root % c == 0;
    } else if (++at_leaf[l / fanin] == fanin) {   // the leaf is full: its average goes up now
      const uint32_t leaf = l / fanin;
      at_leaf[leaf] = 0;
      add(RUDRA_EV_RELAY, leaf, 0, server_ts, relayed[leaf]++, tick);
      at_root += fanin;
      closes_group = at_root % c == 0;
    }
    finish_push(l, tick, closes_group);
  }

  void finish_push(uint32_t l, uint64_t tick, bool closes_group) {
    if (closes_group) add(RUDRA_EV_STEP, l, 0, ++server_ts, 0, tick);

    if (mode == RUDRA_SCHED_HARDSYNC) {
      if (closes_group) {   // barrier: everyone receives and starts from the new weights
        add(RUDRA_EV_BROADCAST, 0, 0, server_ts, 0, tick);
        for (uint32_t k = 0; k < lambda; ++k) delivered_ts[k] = in_use_ts[k] = server_ts;
      }
      return;
    }
    if (closes_group && downcast) {
      add(RUDRA_EV_BROADCAST, 0, 0, server_ts, 0, tick);
      for (uint32_t k = 0; k < lambda; ++k) delivered_ts[k] = server_ts;   // receive buffers only
    }
    const bool current = delivered_ts[l] == server_ts;      // timestamp inquiry
    add(current ? RUDRA_EV_PULL_SKIP : RUDRA_EV_PULL, l, 0, server_ts, 0, tick);
    delivered_ts[l] = server_ts;
    in_use_ts[l] = server_ts;                                // next mini-batch starts now
  }

  void produce() {
    pending.clear();
    pending_pos = 0;
    if (mode == RUDRA_SCHED_SOFTSYNC_TIMED) {
      const Arrival a = arrivals.top();
      arrivals.pop();
      on_push(a.second, a.first);
      arrivals.emplace(a.first + compute_ticks(a.second), a.second);
    } else {
      if (round_pos == lambda) shuffle_round();
      on_push(round[round_pos++], handled + 1);
    }
  }

  rudra_event next() {
    if (pending_pos == pending.size()) produce();
    return pending[pending_pos++];
  }
};

extern "C" {

rudra_sched* rudra_sched_create_tree(uint32_t lambda, uint32_t n, int mode, uint64_t seed,
                                     double lognormal_sigma, int downcast, uint32_t fanin) {
  if (lambda == 0 || n == 0 || n > lambda) return nullptr;
  if (mode != RUDRA_SCHED_HARDSYNC && mode != RUDRA_SCHED_SOFTSYNC_ROUNDS && mode != RUDRA_SCHED_SOFTSYNC_TIMED)
    return nullptr;
  if (mode == RUDRA_SCHED_HARDSYNC && n != 1) return nullptr;
  if (!(lognormal_sigma >= 0.0) || !std::isfinite(lognormal_sigma)) return nullptr;
  if (fanin != 0 && (lambda % fanin != 0 || (lambda / n) % fanin != 0)) return nullptr;
  try {
    return new rudra_sched(lambda, n, mode, seed, lognormal_sigma, downcast != 0, fanin);
  } catch (...) {
    return nullptr;
  }
}

rudra_sched* rudra_sched_create(uint32_t lambda, uint32_t n, int mode, uint64_t seed,
                                double lognormal_sigma, int downcast) {
  return rudra_sched_create_tree(lambda, n, mode, seed, lognormal_sigma, downcast, 0);
}

int rudra_sched_on_pull(rudra_sched* s, uint32_t learner, uint64_t ts) {
  if (!s || learner >= s->lambda) return RUDRA_E_INVAL;
  if (ts > s->server_ts) return RUDRA_E_BAD_TS;
  s->delivered_ts[learner] = s->in_use_ts[learner] = ts;
  return 0;
}

void rudra_sched_destroy(rudra_sched* s) { delete s; }

int64_t rudra_sched_next(rudra_sched* s, rudra_event* out, uint64_t count) {
  if (!s || (!out && count)) return RUDRA_E_INVAL;
  try {
    for (uint64_t i = 0; i < count; ++i) out[i] = s->next();
  } catch (...) {
    return RUDRA_E_NOMEM;
  }
  return (int64_t)count;
}

}  // extern "C"
