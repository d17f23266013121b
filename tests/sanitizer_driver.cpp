// Test driver, built with -fsanitize=address,undefined: runs the library's host-only scheduler and
// the CPU oracle (two separate code bases) side by side and checks that their event traces are
// byte-identical, then exercises the oracle's update loop on small vectors.  Any out-of-bounds
// access, use after free, signed overflow or misaligned access aborts the program.
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <vector>

#include "rudra_ps.h"

struct OraEvent { int32_t kind; uint32_t learner; uint64_t pulled_ts, ts, seq, tick; };
extern "C" {
void* ora_sched_create(uint32_t, uint32_t, int32_t, uint64_t, double, int32_t);
void* ora_sched_create_tree(uint32_t, uint32_t, int32_t, uint64_t, double, int32_t, uint32_t);
int32_t ora_sched_on_pull(void*, uint32_t, uint64_t);
int64_t ora_ps_push_relay(void*, const void* const*, const uint64_t*, uint32_t);
void ora_sched_destroy(void*);
void ora_sched_run(void*, uint64_t, OraEvent*);
void* ora_ps_create(uint64_t, uint32_t, uint32_t, float, float, float);
void ora_ps_destroy(void*);
void ora_ps_set_policy(void*, int32_t);
void ora_ps_set_grad_dtype(void*, int32_t);
void ora_ps_set_optimizer(void*, int32_t, float);
void ora_ps_set_strict(void*, int32_t);
void ora_ps_set_weights(void*, const float*);
int64_t ora_ps_push(void*, const void*, uint64_t);
int32_t ora_ps_step(void*);
int64_t ora_ps_pull(void*, float*);
}

int main() {
  static_assert(sizeof(OraEvent) == sizeof(rudra_event), "event records differ");
  const struct { uint32_t lam, n; int mode; double spread; int downcast; } cases[] = {
      {4, 1, 0, 0.3, 0}, {1, 1, 1, 0.3, 0}, {30, 30, 1, 0.3, 0}, {30, 4, 1, 0.3, 1}, {54, 18, 1, 0.3, 0},
      {60, 4, 2, 0.3, 0}, {128, 4, 2, 1.0, 1}, {7, 3, 2, 0.0, 0}};
  for (const auto& cs : cases) {
    for (uint64_t seed : {1ull, 20150914ull, ~0ull}) {
      const uint64_t count = 20000;
      std::vector<rudra_event> a(count);
      std::vector<OraEvent> b(count);
      rudra_sched* s = rudra_sched_create(cs.lam, cs.n, cs.mode, seed, cs.spread, cs.downcast);
      void* o = ora_sched_create(cs.lam, cs.n, cs.mode, seed, cs.spread, cs.downcast);
      if (!s || !o) return 1;
      for (uint64_t done = 0; done < count; done += 777) {
        const uint64_t take = count - done < 777 ? count - done : 777;
        if (rudra_sched_next(s, a.data() + done, take) != (int64_t)take) return 2;
      }
      ora_sched_run(o, count, b.data());
      if (std::memcmp(a.data(), b.data(), count * sizeof(rudra_event)) != 0) return 3;
      rudra_sched_destroy(s);
      ora_sched_destroy(o);
    }
  }
  if (rudra_sched_create(4, 5, 1, 0, 0.3, 0) != nullptr) return 4;
  // learners -> leaves -> root, with one learner reporting the weights it really holds now and then
  const struct { uint32_t lam, n; int mode; uint32_t fanin; } trees[] = {{12, 2, 1, 3}, {54, 18, 1, 3}, {8, 1, 0, 4}, {60, 4, 2, 5}, {6, 2, 2, 1}};
  for (const auto& t : trees) {
    rudra_sched* s = rudra_sched_create_tree(t.lam, t.n, t.mode, 7, 0.3, 0, t.fanin);
    void* o = ora_sched_create_tree(t.lam, t.n, t.mode, 7, 0.3, 0, t.fanin);
    if (!s || !o) return 11;
    uint64_t held = 0;
    for (int i = 0; i < 20000; ++i) {
      rudra_event a;
      OraEvent b;
      if (rudra_sched_next(s, &a, 1) != 1) return 12;
      ora_sched_run(o, 1, &b);
      if (std::memcmp(&a, &b, sizeof(a)) != 0) return 13;
      if (a.learner == 0 && (a.kind == RUDRA_EV_PULL || a.kind == RUDRA_EV_PULL_SKIP) && t.mode != 0) {
        if (i % 3 == 0) held = a.ts;
        else if (rudra_sched_on_pull(s, 0, held) != 0 || ora_sched_on_pull(o, 0, held) != 0) return 14;
      }
    }
    rudra_sched_destroy(s);
    ora_sched_destroy(o);
  }
  // the oracle's update loop: every optimizer, policy, precision mode and gradient type, ragged sizes
  for (uint64_t N : {1ull, 7ull, 1000ull}) {
    for (int opt = 0; opt < 2; ++opt) for (int pol = 0; pol < 3; ++pol) for (int dt = 0; dt < 2; ++dt) for (int strict = 0; strict < 2; ++strict) {
      void* ps = ora_ps_create(N, 6, 2, 0.01f, opt ? 0.f : 0.9f, 5e-4f);
      if (!ps) return 5;
      ora_ps_set_optimizer(ps, opt, 1e-8f);
      ora_ps_set_policy(ps, pol);
      ora_ps_set_grad_dtype(ps, dt);
      ora_ps_set_strict(ps, strict);
      std::vector<float> th(N, 0.01f), out(N);
      std::vector<float> g32(N, 1e-3f);
      std::vector<uint16_t> g16(N, 0x3A83);   // bf16 pattern of about 1e-3
      ora_ps_set_weights(ps, th.data());
      for (int step = 0; step < 5; ++step) {
        for (int l = 0; l < 3; ++l) {
          const uint64_t pulled = (uint64_t)(step > l ? step - l : 0);
          if (ora_ps_push(ps, dt ? (const void*)g16.data() : (const void*)g32.data(), pulled) != l + 1) return 6;
        }
        if (ora_ps_step(ps) != 1) return 7;
      }
      // one more update through the server tree: a leaf's average of two, and a third gradient directly
      {
        const void* two[2] = {dt ? (const void*)g16.data() : (const void*)g32.data(), dt ? (const void*)g16.data() : (const void*)g32.data()};
        const uint64_t stamps[2] = {5, 3};
        if (ora_ps_push_relay(ps, two, stamps, 2) != 2) return 15;
        if (ora_ps_push_relay(ps, two, stamps, 2) >= 0) return 16;   // would straddle two updates
        if (ora_ps_push(ps, two[0], 4) != 3 || ora_ps_step(ps) != 1) return 17;
        for (int l = 0; l < 3; ++l) ora_ps_push(ps, two[0], 6);
        ora_ps_step(ps);
      }
      if (ora_ps_push(ps, g32.data(), 99) >= 0) return 8;   // a gradient from the future
      if (ora_ps_pull(ps, out.data()) != 7) return 9;
      if (!(out[N - 1] < 0.01f)) return 10;
      ora_ps_destroy(ps);
    }
  }
  std::puts("sanitizer driver ok");
  return 0;
}
