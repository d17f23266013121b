// Host side of the parameter server: the message queue, the integer bookkeeping of Section 3.1
// (scalar timestamp, staleness, vector clock, Eq. 2), the step-size table of Eq. 5 / Eq. 6 and
// the launches.  All floating-point work on the model happens in the kernels of update.cu and
// snapshot.cu; nothing here touches a weight.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <deque>
#include <new>
#include <vector>

#include <cuda_runtime.h>

#include "../../include/rudra_ps.h"
#include "kernels.cuh"

namespace {

thread_local char g_error[512] = "";

int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_error, sizeof(g_error), fmt, ap);
  va_end(ap);
  return code;
}

int cuda_fail(cudaError_t e, const char* what) {
  return fail(RUDRA_E_CUDA, "%s: %s (%s)", what, cudaGetErrorName(e), cudaGetErrorString(e));
}

// Runs the body of an exported function; a C++ exception (in practice std::bad_alloc from a host
// container) becomes an error code instead of crossing the C boundary.
template <typename F>
auto guarded(F&& body) -> decltype(body()) {
  using R = decltype(body());
  try {
    return body();
  } catch (const std::bad_alloc&) {
    return (R)fail(RUDRA_E_NOMEM, "out of host memory");
  } catch (...) {
    return (R)fail(RUDRA_E_NOMEM, "unexpected C++ exception");
  }
}

constexpr uint32_t kMagic = 0x52554452u;   // "RUDR"
constexpr uintptr_t kAlignMask = 31;       // 256-bit vector accesses

bool aligned(const void* p) { return p != nullptr && (reinterpret_cast<uintptr_t>(p) & kAlignMask) == 0; }

// One gradient the queue stands for.  A learner's own gradient is a message of one entry.  The
// average a leaf of the server tree relays for k gradients (Section 3.3) is a message of k entries,
// one per timestamp it carries: the first holds the vector (the leaf's average), the others none.
// A leaf that shares the server's GPU hands over its k raw vectors instead, one per entry, and the
// update kernel does the averaging.
struct Pending {
  const void* grad;     // vector to read, or nullptr (an entry of an averaged message after the first)
  uint64_t pulled_ts;
  int slot;             // staging slot that holds the data, or -1 for a borrowed caller buffer
  uint32_t fanin;       // first entry of a message: gradients it stands for; later entries: 0
  bool uploaded;        // the slot is filled by the upload stream: its reader waits for slot_ready
};

// Makes the handle's device current for the duration of a call.
class DeviceScope {
 public:
  explicit DeviceScope(int device) : prev_(-1), ok_(true) {
    if (cudaGetDevice(&prev_) != cudaSuccess) { ok_ = false; return; }
    if (prev_ != device) { ok_ = cudaSetDevice(device) == cudaSuccess; switched_ = ok_; }
  }
  ~DeviceScope() { if (switched_) cudaSetDevice(prev_); }
  bool ok() const { return ok_; }
 private:
  int prev_;
  bool ok_;
  bool switched_ = false;
};

}  // namespace

struct rudra_ps {
  uint32_t magic = kMagic;
  uint64_t N = 0;
  uint32_t lambda = 0, n = 0, c = 0;
  float alpha0 = 0.f, momentum = 0.f, wd = 0.f, eps = 1e-8f;
  int gtype = RUDRA_GRAD_F32, policy = RUDRA_LR_PAPER_N, optim = RUDRA_OPTIM_MOMENTUM_SGD;
  int push_mode = RUDRA_PUSH_BORROW;
  uint32_t fanin = 0;              // learners per leaf when rudra_ps_run_events plays a server tree; 0 = none
  std::vector<std::vector<Pending>> leaf_pending;   // per leaf: gradients received, not yet relayed
  int device = 0;
  int sm_count = 0;
  uint32_t sweep = 0;              // launches so far: successive launches sweep in opposite directions
  cudaStream_t stream = nullptr;
  float* theta = nullptr;
  float* state = nullptr;
  uint64_t ts = 0;
  std::deque<Pending> queue;
  // Host-buffer path: gradients arrive over PCIe on an upload stream into staging slots, pulled
  // weights leave on a download stream from snapshot buffers, so both directions of the link
  // and the update kernels overlap.  Events order slot re-use against the kernels that read them.
  cudaStream_t up_stream = nullptr, down_stream = nullptr;
  std::vector<void*> slots;        // staging buffers for gradients pushed from host memory
  std::vector<cudaEvent_t> slot_ready;   // upload into the slot has finished
  std::vector<cudaEvent_t> slot_spent;   // the update that read the slot has finished
  std::vector<uint8_t> slot_upload_unread;   // an upload filled the slot and no launch has waited for it yet
  std::vector<int> free_slots;
  struct DownBuf { float* buf = nullptr; cudaEvent_t filled = nullptr, drained = nullptr; };
  std::vector<DownBuf> down;       // snapshots on their way to host memory
  uint32_t down_next = 0;
  bool has_clock = false;
  std::vector<uint64_t> clock;
  std::vector<uint32_t> sigma;
  std::vector<float> scale;
  std::vector<float> msg_step;     // last update: step size of each message
  std::vector<uint32_t> msg_fanin; // last update: gradients each message stood for
  double avg_sigma = 0.0;
  // Record of past updates (Section 3.2: the server records the vector clock of each weight
  // update to keep track of the average staleness): a ring of the last kClockLog updates, c
  // gradient timestamps each, and a histogram of every staleness value seen since create.
  static constexpr uint32_t kClockLog = 4096;
  static constexpr uint32_t kHistBins = RUDRA_HIST_BINS;
  std::vector<uint64_t> log_pulled;     // kClockLog * c
  std::vector<uint64_t> log_ts;         // timestamp before the update in that ring position, or ~0
  std::vector<uint64_t> sigma_hist;     // count per staleness value, grown on demand
  uint64_t counters[8] = {0, 0, 0, 0, 0, 0, 0, 0};

  // Zero-copy pulls (rudra_ps_enable_views): a pool of immutable weight versions.  A pull hands
  // the learner a pointer to the version with the current timestamp; learners that pull the same
  // timestamp share one buffer, so a version is written once however many learners read it.
  struct Version { float* buf = nullptr; uint64_t ts = 0; uint32_t refs = 0; bool valid = false; };
  std::vector<Version> versions;
  std::vector<int> view_of;        // per learner: index into versions, or -1
  bool views_enabled() const { return !versions.empty(); }

  size_t grad_bytes() const { return (size_t)N * (gtype == RUDRA_GRAD_BF16 ? 2u : 4u); }
};

namespace {

bool valid(const rudra_ps* ps) { return ps != nullptr && ps->magic == kMagic; }

void release_queue(rudra_ps* ps) {
  for (const Pending& e : ps->queue)
    if (e.slot >= 0) ps->free_slots.push_back(e.slot);
  ps->queue.clear();
  for (auto& leaf : ps->leaf_pending) {
    for (const Pending& e : leaf)
      if (e.slot >= 0) ps->free_slots.push_back(e.slot);
    leaf.clear();
  }
}

cudaError_t sync_all(rudra_ps* ps) {
  cudaError_t e = cudaStreamSynchronize(ps->stream);
  if (e == cudaSuccess && ps->up_stream) e = cudaStreamSynchronize(ps->up_stream);
  if (e == cudaSuccess && ps->down_stream) e = cudaStreamSynchronize(ps->down_stream);
  return e;
}

cudaError_t ensure_copy_streams(rudra_ps* ps) {
  cudaError_t e = cudaSuccess;
  if (!ps->up_stream) e = cudaStreamCreateWithFlags(&ps->up_stream, cudaStreamNonBlocking);
  if (e == cudaSuccess && !ps->down_stream) e = cudaStreamCreateWithFlags(&ps->down_stream, cudaStreamNonBlocking);
  return e;
}

int free_staging(rudra_ps* ps) {
  cudaError_t e = sync_all(ps);
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  for (void* s : ps->slots) cudaFree(s);
  for (cudaEvent_t ev : ps->slot_ready) cudaEventDestroy(ev);
  for (cudaEvent_t ev : ps->slot_spent) cudaEventDestroy(ev);
  ps->slots.clear();
  ps->slot_ready.clear();
  ps->slot_spent.clear();
  ps->slot_upload_unread.clear();
  ps->free_slots.clear();
  return 0;
}

void free_host_path(rudra_ps* ps) {
  free_staging(ps);
  for (auto& d : ps->down) {
    cudaFree(d.buf);
    if (d.filled) cudaEventDestroy(d.filled);
    if (d.drained) cudaEventDestroy(d.drained);
  }
  ps->down.clear();
  if (ps->up_stream) cudaStreamDestroy(ps->up_stream);
  if (ps->down_stream) cudaStreamDestroy(ps->down_stream);
  ps->up_stream = ps->down_stream = nullptr;
}

int64_t enqueue(rudra_ps* ps, const void* grad, uint64_t pulled_ts, int slot, bool uploaded = false) {
  ps->queue.push_back(Pending{grad, pulled_ts, slot, 1u, uploaded});
  ps->counters[0] += 1;
  return (int64_t)ps->queue.size();
}

// A staging slot of grad_bytes() bytes: a free one, else a new allocation.  *fresh tells whether it
// was just allocated (no earlier reader to wait for).
cudaError_t acquire_slot(rudra_ps* ps, int* slot, bool* fresh) {
  if (!ps->free_slots.empty()) {
    *slot = ps->free_slots.back();
    ps->free_slots.pop_back();
    *fresh = false;
    return cudaSuccess;
  }
  void* buf = nullptr;
  cudaEvent_t ready = nullptr, spent = nullptr;
  cudaError_t e = cudaMalloc(&buf, ps->grad_bytes());
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ready, cudaEventDisableTiming);
  if (e == cudaSuccess) e = cudaEventCreateWithFlags(&spent, cudaEventDisableTiming);
  if (e != cudaSuccess) {
    cudaFree(buf);
    if (ready) cudaEventDestroy(ready);
    return e;
  }
  ps->slots.push_back(buf);
  ps->slot_ready.push_back(ready);
  ps->slot_spent.push_back(spent);
  ps->slot_upload_unread.push_back(0);
  *slot = (int)ps->slots.size() - 1;
  *fresh = true;
  return cudaSuccess;
}

// COPY push mode (Section 3.2: the push message carries the gradient itself): the vector is copied
// into a staging slot on the handle's stream at push time, so the caller's buffer is free again
// for anything ordered after this call on that stream.  The slot's last reader ran on the same
// stream, so the copy needs no event -- unless the slot was filled by an upload that was dropped
// unread (rudra_ps_set_weights / import_state with gradients still queued): that upload may still
// be in flight on the upload stream.
int stage_device_copy(rudra_ps* ps, const void* src, int* slot) {
  bool fresh = false;
  cudaError_t e = acquire_slot(ps, slot, &fresh);
  if (e != cudaSuccess) return cuda_fail(e, "staging buffer allocation");
  if (ps->slot_upload_unread[*slot]) {
    e = cudaStreamWaitEvent(ps->stream, ps->slot_ready[*slot], 0);
    if (e != cudaSuccess) {
      ps->free_slots.push_back(*slot);
      return cuda_fail(e, "cudaStreamWaitEvent");
    }
    ps->slot_upload_unread[*slot] = 0;
  }
  e = cudaMemcpyAsync(ps->slots[*slot], src, ps->grad_bytes(), cudaMemcpyDeviceToDevice, ps->stream);
  if (e != cudaSuccess) {
    ps->free_slots.push_back(*slot);
    return cuda_fail(e, "gradient device-to-device copy");
  }
  return 0;
}

int check_push(rudra_ps* ps, uint64_t pulled_ts) {
  // a learner cannot have pulled weights that do not exist yet: staleness is never negative
  if (pulled_ts > ps->ts)
    return fail(RUDRA_E_BAD_TS, "pulled_ts %llu is ahead of the server timestamp %llu",
                (unsigned long long)pulled_ts, (unsigned long long)ps->ts);
  if (ps->queue.size() >= RUDRA_QUEUE_CAP) return fail(RUDRA_E_QUEUE_FULL, "%d gradients already queued", RUDRA_QUEUE_CAP);
  return 0;
}

// A launch under construction: a window of consecutive updates and the pulls between them.
struct Window {
  rudra::UpdateParams p;
  cudaError_t wait_error = cudaSuccess;   // first failure while ordering the launch after its uploads
  uint32_t nupd = 0, ndst = 0;
  uint32_t npulls = 0;           // learner pulls served (a shared version serves several with one copy)
  uint32_t nversions = 0;        // versions written by this launch
  std::vector<int> used_slots;   // staging slots the window's gradients occupy
};

// Bookkeeping of the version pool, separate from the device buffers so that a batch can be
// replayed on a copy before anything is launched.
struct ViewBook {
  std::vector<uint64_t> ts;
  std::vector<uint32_t> refs;
  std::vector<uint8_t> valid;
  std::vector<int> view_of;

  explicit ViewBook(const rudra_ps* ps) : view_of(ps->view_of) {
    for (const auto& v : ps->versions) { ts.push_back(v.ts); refs.push_back(v.refs); valid.push_back(v.valid); }
  }
  // Learner l takes the version with timestamp now.  Returns its index, sets *fresh when the
  // version has to be written first; -1 when every buffer is still held by some learner.
  int adopt(uint32_t l, uint64_t now, bool* fresh) {
    *fresh = false;
    int idx = -1;
    for (size_t i = 0; i < ts.size(); ++i)
      if (valid[i] && ts[i] == now) { idx = (int)i; break; }
    if (idx < 0) {
      const int own = view_of[l];   // the learner's own old version becomes free with this pull
      for (size_t i = 0; i < ts.size(); ++i)
        if (refs[i] == 0 || ((int)i == own && refs[i] == 1)) { idx = (int)i; break; }
      if (idx < 0) return -1;
      *fresh = true;
    }
    if (view_of[l] >= 0) refs[view_of[l]] -= 1;
    if (*fresh) { ts[idx] = now; valid[idx] = 1; }
    refs[idx] += 1;
    view_of[l] = idx;
    return idx;
  }
  void store(rudra_ps* ps) const {
    for (size_t i = 0; i < ts.size(); ++i) { ps->versions[i].ts = ts[i]; ps->versions[i].refs = refs[i]; ps->versions[i].valid = valid[i] != 0; }
    ps->view_of = view_of;
  }
};

// Vectors the next update will read: one per learner's own gradient, one per relayed average, k per
// group of raw vectors handed over by a leaf on this GPU.
uint32_t next_update_vectors(const rudra_ps* ps) {
  uint32_t nvec = 0;
  for (uint32_t l = 0; l < ps->c; ++l) nvec += ps->queue[l].grad != nullptr;
  return nvec;
}

// Group close (Section 3.1, Eq. 2) and the step-size table (Eq. 5's share of the average times the
// rate of Eq. 6 or one of its two variants) for the messages that stand for the c oldest queued
// gradients, appended to the window as its next update.  Integers first, then one rounding to
// fp32 per table entry.  Raises the timestamp.
void append_update(rudra_ps* ps, Window& w) {
  const uint32_t c = ps->c;
  rudra::UpdateParams& p = w.p;
  if (w.nupd == 0) p.grad_end[0] = 0;
  uint32_t vec = p.grad_end[w.nupd];
  ps->clock.resize(c);
  ps->sigma.resize(c);
  ps->scale.resize(c);
  ps->msg_step.clear();
  ps->msg_fanin.clear();
  uint64_t sum_sigma = 0, sum_pulled = 0;
  for (uint32_t l = 0; l < c; ++l) {
    const Pending& e = ps->queue[l];
    ps->clock[l] = e.pulled_ts;
    ps->sigma[l] = (uint32_t)(ps->ts - e.pulled_ts);
    sum_sigma += ps->sigma[l];
    sum_pulled += e.pulled_ts;
    if (e.slot >= 0) {
      if (e.uploaded) {   // the kernel starts after its uploads
        const cudaError_t we = cudaStreamWaitEvent(ps->stream, ps->slot_ready[e.slot], 0);
        if (we != cudaSuccess && w.wait_error == cudaSuccess) w.wait_error = we;
        ps->slot_upload_unread[e.slot] = 0;
      }
      w.used_slots.push_back(e.slot);
    }
  }
  ps->avg_sigma = (double)ps->ts - (double)sum_pulled / (double)c;
  {
    if (ps->log_ts.empty()) {
      ps->log_ts.assign(rudra_ps::kClockLog, ~0ull);
      ps->log_pulled.assign((size_t)rudra_ps::kClockLog * c, 0);
    }
    const size_t pos = (size_t)(ps->ts % rudra_ps::kClockLog);
    ps->log_ts[pos] = ps->ts;
    for (uint32_t l = 0; l < c; ++l) {
      ps->log_pulled[pos * c + l] = ps->clock[l];
      // the last bin counts every staleness of kHistBins - 1 and more, so one very late gradient
      // cannot ask for a histogram as long as the timestamp
      const uint32_t bin = ps->sigma[l] < rudra_ps::kHistBins - 1 ? ps->sigma[l] : rudra_ps::kHistBins - 1;
      if (bin >= ps->sigma_hist.size()) ps->sigma_hist.resize((size_t)bin + 1, 0);
      ps->sigma_hist[bin] += 1;
    }
  }
  // Step size of each message: rate times the share k / c of Eq. 5's average it stands for.
  double sum_step = 0.0;
  for (uint32_t l = 0; l < c;) {
    const uint32_t k = ps->queue[l].fanin;
    uint64_t msg_sigma = 0;
    for (uint32_t i = 0; i < k; ++i) msg_sigma += ps->sigma[l + i];
    double num = (double)ps->alpha0 * (double)k, divisor;
    switch (ps->policy) {
      case RUDRA_LR_PER_GRADIENT:   // alpha0 / max(mean staleness of the message, 1) = alpha0 k / max(sum, k)
        num *= (double)k;
        divisor = (double)(msg_sigma > k ? msg_sigma : (uint64_t)k) * (double)c;
        break;
      case RUDRA_LR_GROUP_MEAN:     // alpha0 / max(<sigma>, 1) with Eq. 2's <sigma> = sum / c
        divisor = (double)(sum_sigma > c ? sum_sigma : (uint64_t)c);
        break;
      default:                      // alpha0 / n
        divisor = (double)ps->n * (double)c;
        break;
    }
    const float step = (float)(num / divisor);
    ps->msg_step.push_back(step);
    ps->msg_fanin.push_back(k);
    sum_step += (double)step;
    for (uint32_t i = 0; i < k; ++i) ps->scale[l + i] = (float)((double)step / (double)k);
    l += k;
  }
  const float abar = (float)sum_step;
  // The kernel's table: one entry per vector.  An averaged message is one vector with the
  // message's step size; raw vectors get their message's step size over its fan-in each.
  // AdaGrad combines the vectors with weights (step / sum of steps); with a zero rate every step
  // is 0 and the weights fall back to Eq. 5's plain shares (the weights do not move, the sum of
  // squares does).
  uint32_t m = 0;
  for (uint32_t l = 0; l < c; ++m) {
    const uint32_t k = ps->queue[l].fanin;
    uint32_t nvec = 0;
    for (uint32_t i = 0; i < k; ++i) nvec += ps->queue[l + i].grad != nullptr;
    const double step = (double)ps->msg_step[m];
    const double weight = abar > 0.f ? step / (double)abar : (double)k / (double)c;
    for (uint32_t i = 0; i < k; ++i) {
      const Pending& e = ps->queue[l + i];
      if (!e.grad) continue;
      p.grad[vec] = e.grad;
      p.scale[vec] = (float)((ps->optim == RUDRA_OPTIM_ADAGRAD ? weight : step) / (double)nvec);
      vec += 1;
    }
    l += k;
  }
  p.awd[w.nupd] = (float)((double)abar * (double)ps->wd);
  p.abar[w.nupd] = abar;
  p.dst_end[w.nupd] = (uint8_t)w.ndst;   // pulls so far belong to the state before this update
  w.nupd += 1;
  p.grad_end[w.nupd] = (uint8_t)vec;
  ps->has_clock = true;
  for (uint32_t l = 0; l < c; ++l) ps->queue.pop_front();
  ps->ts += 1;   // exactly one increment per weight update
}

bool window_has_room_for_update(const rudra_ps* ps, const Window& w, uint32_t max_updates) {
  const uint32_t used = w.nupd ? w.p.grad_end[w.nupd] : 0;
  return w.nupd < max_updates && used + next_update_vectors(ps) <= (uint32_t)rudra::kMaxGroup;
}

// Enqueues the window: the fused kernel if it holds updates, a plain snapshot if it holds only pulls.
int flush_window(rudra_ps* ps, Window& w) {
  if (w.nupd == 0 && w.ndst == 0) {   // nothing to launch; pulls may still have been served by sharing
    ps->counters[2] += w.npulls;
    w.npulls = 0;
    return 0;
  }
  cudaError_t e = w.wait_error;
  w.wait_error = cudaSuccess;
  uint32_t launches = 0;
  auto copy_weights = [&](uint32_t d0, uint32_t d1) {   // 1 -> (d1 - d0) copy of the current weights
    if (d1 == d0 || e != cudaSuccess) return;
    rudra::SnapshotParams sp;
    for (uint32_t d = d0; d < d1; ++d) sp.dst[d - d0] = w.p.dst[d];
    sp.src = ps->theta;
    sp.n = ps->N;
    sp.ndst = d1 - d0;
    sp.reverse = ps->sweep++ & 1u;
    e = rudra::launch_snapshot(sp, ps->stream);
    launches += 1;
  };
  if (w.nupd == 0) {
    copy_weights(0, w.ndst);
  } else {
    rudra::UpdateParams& p = w.p;
    p.dst_end[w.nupd] = (uint8_t)w.ndst;
    // A single update with a broadcast to dozens of learners around it is faster as separate
    // launches (measured at 61 M weights, bf16, c = 32, 128 copies: 5.25 ms against 5.65 ms fused):
    // the copies then run in the copy kernel's shape, at the price of one more read of the weights.
    const bool split = w.nupd == 1 && w.ndst >= 64 && ps->N >= (1u << 22);
    const uint32_t pre = p.dst_end[0], post = w.ndst;
    if (split) {
      copy_weights(0, pre);
      p.dst_end[0] = p.dst_end[1] = 0;
    }
    p.theta = ps->theta;
    p.state = ps->state;
    p.n = ps->N;
    p.nupd = w.nupd;
    p.grad_end[w.nupd + 1] = p.grad_end[w.nupd];
    p.momentum = ps->momentum;
    p.wd = ps->wd;
    p.eps = ps->eps;
    p.reverse = ps->sweep++ & 1u;
    if (e == cudaSuccess) {
      e = rudra::launch_update(p, ps->gtype == RUDRA_GRAD_BF16 ? rudra::kBF16 : rudra::kF32,
                               ps->optim == RUDRA_OPTIM_ADAGRAD ? rudra::kAdagrad : rudra::kMomentumSgd, ps->sm_count,
                               ps->stream);
      launches += 1;
    }
    if (split) copy_weights(pre, post);
  }
  for (int slot : w.used_slots) {   // the next upload into the slot waits for this launch
    const cudaError_t re = cudaEventRecord(ps->slot_spent[slot], ps->stream);
    if (re != cudaSuccess && e == cudaSuccess) e = re;
    ps->free_slots.push_back(slot);
  }
  ps->counters[1] += w.nupd;
  ps->counters[2] += w.npulls;
  ps->counters[3] += launches;
  ps->counters[6] += w.ndst;
  ps->counters[7] += w.nversions;
  w.used_slots.clear();
  w.nupd = w.ndst = w.npulls = w.nversions = 0;
  if (e != cudaSuccess) return cuda_fail(e, "kernel launch");
  return 0;
}

int do_step(rudra_ps* ps, float* const* dsts, uint32_t k) {
  if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
  if (k > RUDRA_MAX_DSTS) return fail(RUDRA_E_INVAL, "k = %u exceeds RUDRA_MAX_DSTS", k);
  if (k && !dsts) return fail(RUDRA_E_INVAL, "null destination list");
  for (uint32_t d = 0; d < k; ++d)
    if (!aligned(dsts[d])) return fail(RUDRA_E_INVAL, "destination %u is null or not 32-byte aligned", d);
  if (ps->queue.size() < ps->c) return 0;   // group still open: nothing changes
  DeviceScope dev(ps->device);
  if (!dev.ok()) return fail(RUDRA_E_CUDA, "cannot select device %d", ps->device);
  Window w;
  append_update(ps, w);
  for (uint32_t d = 0; d < k; ++d) w.p.dst[w.ndst++] = dsts[d];
  w.npulls = k;
  if (int r = flush_window(ps, w)) return r;
  return 1;
}

}  // namespace

extern "C" {

const char* rudra_last_error(void) { return g_error; }

rudra_ps* rudra_ps_create(uint64_t nparams, uint32_t lambda, uint32_t n, float alpha0, float momentum,
                          float weight_decay) {
  if (nparams == 0 || lambda == 0 || n == 0 || n > lambda) {
    fail(RUDRA_E_INVAL, "need nparams > 0 and 1 <= n <= lambda (got nparams=%llu lambda=%u n=%u)",
         (unsigned long long)nparams, lambda, n);
    return nullptr;
  }
  if (lambda / n > RUDRA_MAX_GROUP) {
    fail(RUDRA_E_INVAL, "c = floor(lambda/n) = %u exceeds RUDRA_MAX_GROUP = %d", lambda / n, RUDRA_MAX_GROUP);
    return nullptr;
  }
  if (!std::isfinite(alpha0) || !std::isfinite(momentum) || !std::isfinite(weight_decay) || alpha0 < 0.f ||
      momentum < 0.f || momentum >= 1.f || weight_decay < 0.f) {
    fail(RUDRA_E_INVAL, "alpha0, momentum, weight_decay must be finite, non-negative, momentum < 1");
    return nullptr;
  }
  rudra_ps* ps = new (std::nothrow) rudra_ps;
  if (!ps) { fail(RUDRA_E_NOMEM, "out of host memory"); return nullptr; }
  ps->N = nparams; ps->lambda = lambda; ps->n = n; ps->c = lambda / n;
  ps->alpha0 = alpha0; ps->momentum = momentum; ps->wd = weight_decay;
  cudaError_t e = cudaGetDevice(&ps->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ps->sm_count, cudaDevAttrMultiProcessorCount, ps->device);
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ps->theta), nparams * sizeof(float));
  if (e == cudaSuccess) e = cudaMalloc(reinterpret_cast<void**>(&ps->state), nparams * sizeof(float));
  if (e == cudaSuccess) e = cudaMemset(ps->theta, 0, nparams * sizeof(float));
  if (e == cudaSuccess) e = cudaMemset(ps->state, 0, nparams * sizeof(float));
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) {
    cuda_fail(e, "rudra_ps_create");
    cudaFree(ps->theta);
    cudaFree(ps->state);
    ps->magic = 0;
    delete ps;
    return nullptr;
  }
  return ps;
}

void rudra_ps_destroy(rudra_ps* ps) {
  if (!valid(ps)) return;
  DeviceScope dev(ps->device);
  free_host_path(ps);
  for (auto& v : ps->versions) cudaFree(v.buf);
  cudaFree(ps->theta);
  cudaFree(ps->state);
  ps->magic = 0;
  delete ps;
}

int rudra_ps_set_stream(rudra_ps* ps, void* cuda_stream) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    ps->stream = static_cast<cudaStream_t>(cuda_stream);
    return 0;
  });
}

int rudra_ps_set_option(rudra_ps* ps, int key, int64_t value) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!ps->queue.empty()) return fail(RUDRA_E_STATE, "options can only change while no gradient is queued");
    for (const auto& leaf : ps->leaf_pending)
      if (!leaf.empty()) return fail(RUDRA_E_STATE, "options can only change while no leaf holds a gradient");
    DeviceScope dev(ps->device);
    switch (key) {
      case RUDRA_OPT_GRAD_DTYPE:
        if (value != RUDRA_GRAD_F32 && value != RUDRA_GRAD_BF16) return fail(RUDRA_E_INVAL, "unknown gradient type %lld", (long long)value);
        if ((int)value != ps->gtype) {
          int r = free_staging(ps);   // staging buffers are sized for the gradient type
          if (r < 0) return r;
          ps->gtype = (int)value;
        }
        return 0;
      case RUDRA_OPT_LR_POLICY:
        if (value < RUDRA_LR_PAPER_N || value > RUDRA_LR_GROUP_MEAN) return fail(RUDRA_E_INVAL, "unknown learning-rate policy %lld", (long long)value);
        ps->policy = (int)value;
        return 0;
      case RUDRA_OPT_OPTIMIZER:
        if (value != RUDRA_OPTIM_MOMENTUM_SGD && value != RUDRA_OPTIM_ADAGRAD) return fail(RUDRA_E_INVAL, "unknown optimizer %lld", (long long)value);
        if ((int)value != ps->optim) {
          cudaError_t e = cudaMemsetAsync(ps->state, 0, ps->N * sizeof(float), ps->stream);
          if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
          ps->optim = (int)value;
        }
        return 0;
      case RUDRA_OPT_PUSH_MODE:
        if (value != RUDRA_PUSH_BORROW && value != RUDRA_PUSH_COPY) return fail(RUDRA_E_INVAL, "unknown push mode %lld", (long long)value);
        ps->push_mode = (int)value;
        return 0;
      case RUDRA_OPT_TREE_FANIN:
        if (value < 0 || (value > 0 && (ps->lambda % value != 0 || ps->c % value != 0)))
          return fail(RUDRA_E_INVAL, "fan-in %lld must divide lambda = %u and c = %u", (long long)value, ps->lambda, ps->c);
        ps->fanin = (uint32_t)value;
        ps->leaf_pending.assign(value ? ps->lambda / (uint32_t)value : 0, {});
        return 0;
      default:
        return fail(RUDRA_E_INVAL, "unknown option key %d", key);
    }
  });
}

int rudra_ps_set_alpha0(rudra_ps* ps, float alpha0) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!std::isfinite(alpha0) || alpha0 < 0.f) return fail(RUDRA_E_INVAL, "alpha0 must be finite and non-negative");
    ps->alpha0 = alpha0;
    return 0;
  });
}

static int set_weights_common(rudra_ps* ps, const float* src, cudaMemcpyKind kind) {
  if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
  if (!src) return fail(RUDRA_E_INVAL, "null source");
  DeviceScope dev(ps->device);
  cudaError_t e = cudaMemcpyAsync(ps->theta, src, ps->N * sizeof(float), kind, ps->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(ps->state, 0, ps->N * sizeof(float), ps->stream);
  if (e != cudaSuccess) return cuda_fail(e, "rudra_ps_set_weights");
  if (kind == cudaMemcpyHostToDevice) ps->counters[4] += ps->N * sizeof(float);
  release_queue(ps);
  ps->ts = 0;
  ps->has_clock = false;
  for (auto& v : ps->versions) v.valid = false;   // held views keep their contents; none matches the new weights
  std::fill(ps->log_ts.begin(), ps->log_ts.end(), ~0ull);   // timestamps start over: the log would be ambiguous
  return 0;
}

int rudra_ps_set_weights(rudra_ps* ps, const float* src_dev) {
  return guarded([&]() -> int { return set_weights_common(ps, src_dev, cudaMemcpyDeviceToDevice); });
}

int rudra_ps_set_weights_host(rudra_ps* ps, const float* src_host) {
  return guarded([&]() -> int { return set_weights_common(ps, src_host, cudaMemcpyHostToDevice); });
}

int64_t rudra_ps_push(rudra_ps* ps, const void* grad_dev, uint64_t pulled_ts) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!aligned(grad_dev)) return fail(RUDRA_E_INVAL, "gradient pointer is null or not 32-byte aligned");
    if (int r = check_push(ps, pulled_ts)) return r;
    if (ps->push_mode == RUDRA_PUSH_BORROW) return enqueue(ps, grad_dev, pulled_ts, -1);
    DeviceScope dev(ps->device);
    int slot = -1;
    if (int r = stage_device_copy(ps, grad_dev, &slot)) return r;
    return enqueue(ps, ps->slots[slot], pulled_ts, slot);
  });
}

int64_t rudra_ps_push_host(rudra_ps* ps, const void* grad_host, uint64_t pulled_ts) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!grad_host) return fail(RUDRA_E_INVAL, "null gradient pointer");
    if (int r = check_push(ps, pulled_ts)) return r;
    DeviceScope dev(ps->device);
    cudaError_t e = ensure_copy_streams(ps);
    if (e != cudaSuccess) return cuda_fail(e, "copy stream creation");
    int slot = -1;
    bool fresh = false;
    e = acquire_slot(ps, &slot, &fresh);
    if (e != cudaSuccess) return cuda_fail(e, "staging buffer allocation");
    if (!fresh) {
      // the slot's last reader must be done; a slot last filled by a COPY-mode push was read on the
      // main stream too, and its slot_spent was recorded after that launch
      e = cudaStreamWaitEvent(ps->up_stream, ps->slot_spent[slot], 0);
      if (e != cudaSuccess) {
        ps->free_slots.push_back(slot);
        return cuda_fail(e, "cudaStreamWaitEvent");
      }
    }
    e = cudaMemcpyAsync(ps->slots[slot], grad_host, ps->grad_bytes(), cudaMemcpyHostToDevice, ps->up_stream);
    if (e == cudaSuccess) e = cudaEventRecord(ps->slot_ready[slot], ps->up_stream);
    if (e != cudaSuccess) {
      ps->free_slots.push_back(slot);
      return cuda_fail(e, "gradient host-to-device copy");
    }
    ps->counters[4] += ps->grad_bytes();
    ps->slot_upload_unread[slot] = 1;
    return enqueue(ps, ps->slots[slot], pulled_ts, slot, true);
  });
}

// Appends one message that stands for k gradients: vecs[0..nvec-1] with nvec == 1 (an average) or
// nvec == k (raw vectors).  Arguments are already validated.
static int64_t enqueue_group(rudra_ps* ps, const Pending* vecs, uint32_t nvec, const uint64_t* pulled_ts, uint32_t k) {
  for (uint32_t i = 0; i < k; ++i) {
    Pending e = i < nvec ? vecs[i] : Pending{nullptr, 0, -1, 0u, false};
    e.pulled_ts = pulled_ts[i];
    e.fanin = i == 0 ? k : 0u;
    ps->queue.push_back(e);
  }
  ps->counters[0] += k;
  return (int64_t)ps->queue.size();
}

int64_t rudra_ps_push_group(rudra_ps* ps, const void* const* vecs_dev, uint32_t nvec, const uint64_t* pulled_ts,
                            uint32_t k) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (k == 0 || k > ps->c || !vecs_dev || !pulled_ts) return fail(RUDRA_E_INVAL, "need 1 <= k <= c and non-null tables");
    if (nvec != 1 && nvec != k) return fail(RUDRA_E_INVAL, "nvec must be 1 (an average) or k (raw gradients)");
    if (nvec == 1 && k > 1 && ps->gtype != RUDRA_GRAD_F32)
      return fail(RUDRA_E_STATE, "a relayed average is a float vector: the handle's gradient type must be RUDRA_GRAD_F32");
    for (uint32_t i = 0; i < nvec; ++i)
      if (!aligned(vecs_dev[i])) return fail(RUDRA_E_INVAL, "vector %u is null or not 32-byte aligned", i);
    for (uint32_t i = 0; i < k; ++i)
      if (pulled_ts[i] > ps->ts)
        return fail(RUDRA_E_BAD_TS, "pulled_ts[%u] = %llu is ahead of the server timestamp %llu", i,
                    (unsigned long long)pulled_ts[i], (unsigned long long)ps->ts);
    if (ps->queue.size() % ps->c + k > ps->c)
      return fail(RUDRA_E_STATE, "a message for %u gradients does not fit the open group (%zu of %u queued)", k,
                  ps->queue.size() % ps->c, ps->c);
    if (ps->queue.size() + k > RUDRA_QUEUE_CAP) return fail(RUDRA_E_QUEUE_FULL, "%d gradients already queued", RUDRA_QUEUE_CAP);
    Pending vecs[RUDRA_MAX_GROUP];
    DeviceScope dev(ps->device);
    for (uint32_t i = 0; i < nvec; ++i) {
      vecs[i] = Pending{vecs_dev[i], 0, -1, 0u, false};
      if (ps->push_mode == RUDRA_PUSH_COPY) {
        int slot = -1;
        if (int r = stage_device_copy(ps, vecs_dev[i], &slot)) {
          for (uint32_t u = 0; u < i; ++u) ps->free_slots.push_back(vecs[u].slot);
          return r;
        }
        vecs[i].grad = ps->slots[slot];
        vecs[i].slot = slot;
      }
    }
    return enqueue_group(ps, vecs, nvec, pulled_ts, k);
  });
}

int rudra_ps_last_messages(const rudra_ps* ps, uint32_t* fanin_out, float* step_out) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!ps->has_clock) return 0;
    for (size_t j = 0; j < ps->msg_step.size(); ++j) {
      if (fanin_out) fanin_out[j] = ps->msg_fanin[j];
      if (step_out) step_out[j] = ps->msg_step[j];
    }
    return (int)ps->msg_step.size();
  });
}

int rudra_leaf_average(const void* const* grads_dev, uint32_t k, int grad_dtype, uint64_t nparams, float* avg_dev,
                       void* cuda_stream) {
  return guarded([&]() -> int {
    if (k == 0 || k > RUDRA_MAX_GROUP || !grads_dev || nparams == 0) return fail(RUDRA_E_INVAL, "need 1 <= k <= RUDRA_MAX_GROUP, nparams > 0 and a gradient table");
    if (grad_dtype != RUDRA_GRAD_F32 && grad_dtype != RUDRA_GRAD_BF16) return fail(RUDRA_E_INVAL, "unknown gradient type %d", grad_dtype);
    if (!aligned(avg_dev)) return fail(RUDRA_E_INVAL, "output is null or not 32-byte aligned");
    rudra::LeafParams p;
    for (uint32_t l = 0; l < k; ++l) {
      if (!aligned(grads_dev[l])) return fail(RUDRA_E_INVAL, "gradient %u is null or not 32-byte aligned", l);
      p.grad[l] = grads_dev[l];
    }
    p.out = avg_dev;
    p.n = nparams;
    p.k = k;
    p.inv_k = (float)(1.0 / (double)k);
    const cudaError_t e = rudra::launch_leaf_average(p, grad_dtype == RUDRA_GRAD_BF16 ? rudra::kBF16 : rudra::kF32,
                                                     static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return cuda_fail(e, "leaf average kernel launch");
    return 0;
  });
}

int rudra_ps_step(rudra_ps* ps) {
  return guarded([&]() -> int { return do_step(ps, nullptr, 0); });
}

int rudra_ps_step_pull_many(rudra_ps* ps, float* const* dsts_dev, uint32_t k) {
  return guarded([&]() -> int { return do_step(ps, dsts_dev, k); });
}

int64_t rudra_ps_run_events(rudra_ps* ps, const rudra_event* events, uint64_t count,
                            const void* const* grads_dev, float* const* slots_dev, uint32_t max_window) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (count && !events) return fail(RUDRA_E_INVAL, "null event list");
    const uint32_t cap = max_window == 0 || max_window > (uint32_t)rudra::kMaxWindow ? (uint32_t)rudra::kMaxWindow : max_window;
    // Pass 1: replay the integers only.  Nothing is queued or launched unless the whole batch is legal.
    const bool views = ps->views_enabled();
    {
      uint64_t ts = ps->ts;
      uint64_t queued = ps->queue.size();
      ViewBook sim(ps);
      bool fresh;
      const uint32_t fanin = ps->fanin;
      std::vector<uint32_t> leaf_fill(ps->leaf_pending.size());
      for (size_t j = 0; j < leaf_fill.size(); ++j) leaf_fill[j] = (uint32_t)ps->leaf_pending[j].size();
      for (uint64_t i = 0; i < count; ++i) {
        const rudra_event& ev = events[i];
        const bool needs_learner = ev.kind == RUDRA_EV_PUSH || ev.kind == RUDRA_EV_PULL;
        if (needs_learner && ev.learner >= ps->lambda) return fail(RUDRA_E_INVAL, "event %llu: learner %u out of range", (unsigned long long)i, ev.learner);
        switch (ev.kind) {
          case RUDRA_EV_PUSH:
            if (!grads_dev || !aligned(grads_dev[ev.learner])) return fail(RUDRA_E_INVAL, "event %llu: gradient buffer of learner %u is null or not 32-byte aligned", (unsigned long long)i, ev.learner);
            if (ev.pulled_ts > ts) return fail(RUDRA_E_BAD_TS, "event %llu: pulled_ts %llu is ahead of the server timestamp %llu", (unsigned long long)i, (unsigned long long)ev.pulled_ts, (unsigned long long)ts);
            if (ev.ts != ts) return fail(RUDRA_E_STATE, "event %llu: push expects server timestamp %llu, server has %llu", (unsigned long long)i, (unsigned long long)ev.ts, (unsigned long long)ts);
            if (fanin) {   // the gradient goes to the learner's leaf, not to the root's queue
              if (++leaf_fill[ev.learner / fanin] > fanin) return fail(RUDRA_E_STATE, "event %llu: leaf %u holds more than %u gradients without a relay", (unsigned long long)i, ev.learner / fanin, fanin);
              break;
            }
            if (++queued > RUDRA_QUEUE_CAP) return fail(RUDRA_E_QUEUE_FULL, "event %llu: queue full", (unsigned long long)i);
            break;
          case RUDRA_EV_RELAY:
            if (!fanin) return fail(RUDRA_E_STATE, "event %llu: relay, but RUDRA_OPT_TREE_FANIN is not set", (unsigned long long)i);
            if (ev.learner >= leaf_fill.size()) return fail(RUDRA_E_INVAL, "event %llu: leaf %u out of range", (unsigned long long)i, ev.learner);
            if (leaf_fill[ev.learner] != fanin) return fail(RUDRA_E_STATE, "event %llu: leaf %u relays with %u of %u gradients", (unsigned long long)i, ev.learner, leaf_fill[ev.learner], fanin);
            if (ev.ts != ts) return fail(RUDRA_E_STATE, "event %llu: relay expects server timestamp %llu, server has %llu", (unsigned long long)i, (unsigned long long)ev.ts, (unsigned long long)ts);
            if (queued % ps->c + fanin > ps->c) return fail(RUDRA_E_STATE, "event %llu: the relayed average does not fit the open group", (unsigned long long)i);
            leaf_fill[ev.learner] = 0;
            if ((queued += fanin) > RUDRA_QUEUE_CAP) return fail(RUDRA_E_QUEUE_FULL, "event %llu: queue full", (unsigned long long)i);
            break;
          case RUDRA_EV_STEP:
            if (queued < ps->c) return fail(RUDRA_E_STATE, "event %llu: update with %llu of %u gradients queued", (unsigned long long)i, (unsigned long long)queued, ps->c);
            queued -= ps->c;
            ts += 1;
            if (ev.ts != ts) return fail(RUDRA_E_STATE, "event %llu: update expects new timestamp %llu, server reaches %llu", (unsigned long long)i, (unsigned long long)ev.ts, (unsigned long long)ts);
            break;
          case RUDRA_EV_PULL:
            if (ev.ts != ts) return fail(RUDRA_E_STATE, "event %llu: pull expects timestamp %llu, server has %llu", (unsigned long long)i, (unsigned long long)ev.ts, (unsigned long long)ts);
            if (views) {
              if (sim.adopt(ev.learner, ts, &fresh) < 0) return fail(RUDRA_E_STATE, "event %llu: all %zu weight versions are still held by learners", (unsigned long long)i, sim.ts.size());
            } else if (!slots_dev || !aligned(slots_dev[ev.learner])) {
              return fail(RUDRA_E_INVAL, "event %llu: slot of learner %u is null or not 32-byte aligned", (unsigned long long)i, ev.learner);
            }
            break;
          case RUDRA_EV_PULL_SKIP:
            break;
          case RUDRA_EV_BROADCAST:
            if (views) {
              for (uint32_t l = 0; l < ps->lambda; ++l)
                if (sim.adopt(l, ts, &fresh) < 0) return fail(RUDRA_E_STATE, "event %llu: all %zu weight versions are still held by learners", (unsigned long long)i, sim.ts.size());
              break;
            }
            if (!slots_dev) return fail(RUDRA_E_INVAL, "event %llu: broadcast without slots", (unsigned long long)i);
            for (uint32_t l = 0; l < ps->lambda; ++l)
              if (!aligned(slots_dev[l])) return fail(RUDRA_E_INVAL, "event %llu: slot of learner %u is null or not 32-byte aligned", (unsigned long long)i, l);
            break;
          default:
            return fail(RUDRA_E_INVAL, "event %llu: unknown kind %d", (unsigned long long)i, ev.kind);
        }
      }
    }
    // Pass 2: handle the messages in order, packing consecutive updates and the pulls between them
    // into one launch for as long as the launch tables have room.
    DeviceScope dev(ps->device);
    if (!dev.ok()) return fail(RUDRA_E_CUDA, "cannot select device %d", ps->device);
    Window w;
    int64_t updates = 0;
    ViewBook book(ps);
    auto add_copy = [&](float* dst) -> int {
      if (w.ndst == (uint32_t)rudra::kMaxDsts)
        if (int r = flush_window(ps, w)) return r;
      w.p.dst[w.ndst++] = dst;
      return 0;
    };
    // One learner's pull: a copy into its slot, or (zero-copy mode) a reference to the version with
    // the current timestamp, which is written at most once however many learners take it.
    auto add_pull = [&](uint32_t learner) -> int {
      w.npulls += 1;
      if (!views) return add_copy(slots_dev[learner]);
      bool fresh = false;
      const int idx = book.adopt(learner, ps->ts, &fresh);
      if (fresh) {
        if (int r = add_copy(ps->versions[idx].buf)) return r;
        w.nversions += 1;
      }
      return 0;
    };
    for (uint64_t i = 0; i < count; ++i) {
      const rudra_event& ev = events[i];
      switch (ev.kind) {
        case RUDRA_EV_PUSH: {
          Pending e{grads_dev[ev.learner], ev.pulled_ts, -1, 1u, false};
          if (ps->push_mode == RUDRA_PUSH_COPY) {
            if (int r = stage_device_copy(ps, e.grad, &e.slot)) return r;
            e.grad = ps->slots[e.slot];
          }
          if (ps->fanin) {
            ps->leaf_pending[ev.learner / ps->fanin].push_back(e);
          } else {
            ps->queue.push_back(e);
            ps->counters[0] += 1;
          }
          break;
        }
        case RUDRA_EV_RELAY: {
          // The leaf shares this GPU with the root: it hands over its learners' raw vectors and the
          // update kernel averages them on the way (no intermediate vector is written).
          std::vector<Pending>& leaf = ps->leaf_pending[ev.learner];
          uint64_t stamps[RUDRA_MAX_GROUP];
          for (uint32_t l = 0; l < ps->fanin; ++l) stamps[l] = leaf[l].pulled_ts;
          enqueue_group(ps, leaf.data(), ps->fanin, stamps, ps->fanin);
          leaf.clear();
          break;
        }
        case RUDRA_EV_STEP:
          if (!window_has_room_for_update(ps, w, cap))
            if (int r = flush_window(ps, w)) return r;
          append_update(ps, w);
          updates += 1;
          break;
        case RUDRA_EV_PULL:
          if (int r = add_pull(ev.learner)) return r;
          break;
        case RUDRA_EV_BROADCAST:
          for (uint32_t l = 0; l < ps->lambda; ++l)
            if (int r = add_pull(l)) return r;
          break;
        default:
          break;
      }
    }
    if (views) book.store(ps);
    if (int r = flush_window(ps, w)) return r;
    return updates;
  });
}

int rudra_ps_enable_views(rudra_ps* ps, uint32_t nversions) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (nversions < 2 || nversions > 4096) return fail(RUDRA_E_INVAL, "need 2 <= nversions <= 4096");
    for (int v : ps->view_of)
      if (v >= 0) return fail(RUDRA_E_STATE, "learners still hold views");
    DeviceScope dev(ps->device);
    cudaError_t e = cudaStreamSynchronize(ps->stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    for (auto& v : ps->versions) cudaFree(v.buf);
    ps->versions.clear();
    ps->view_of.assign(ps->lambda, -1);
    for (uint32_t i = 0; i < nversions; ++i) {
      rudra_ps::Version v;
      e = cudaMalloc(reinterpret_cast<void**>(&v.buf), ps->N * sizeof(float));
      if (e != cudaSuccess) {
        for (auto& u : ps->versions) cudaFree(u.buf);
        ps->versions.clear();
        return cuda_fail(e, "weight version allocation");
      }
      ps->versions.push_back(v);
    }
    return 0;
  });
}

int64_t rudra_ps_pull_view(rudra_ps* ps, uint32_t learner, const float** view_out) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!ps->views_enabled()) return fail(RUDRA_E_STATE, "call rudra_ps_enable_views first");
    if (learner >= ps->lambda || !view_out) return fail(RUDRA_E_INVAL, "learner out of range or null output");
    ViewBook book(ps);
    bool fresh = false;
    const int idx = book.adopt(learner, ps->ts, &fresh);
    if (idx < 0) return fail(RUDRA_E_STATE, "all %zu weight versions are still held by learners", ps->versions.size());
    DeviceScope dev(ps->device);
    Window w;
    w.npulls = 1;
    if (fresh) {
      w.p.dst[w.ndst++] = ps->versions[idx].buf;
      w.nversions = 1;
    }
    book.store(ps);
    if (int r = flush_window(ps, w)) return r;   // a snapshot launch if the version is new
    *view_out = ps->versions[idx].buf;
    return (int64_t)ps->ts;
  });
}

int64_t rudra_ps_view_of(const rudra_ps* ps, uint32_t learner, const float** view_out) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!ps->views_enabled() || learner >= ps->lambda || !view_out) return fail(RUDRA_E_INVAL, "views not enabled, learner out of range or null output");
    const int idx = ps->view_of[learner];
    if (idx < 0) return fail(RUDRA_E_STATE, "learner %u holds no view", learner);
    *view_out = ps->versions[idx].buf;
    return (int64_t)ps->versions[idx].ts;
  });
}

int64_t rudra_ps_pull_many(rudra_ps* ps, float* const* dsts_dev, uint32_t k) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (k == 0) return (int64_t)ps->ts;
    if (k > RUDRA_MAX_DSTS) return fail(RUDRA_E_INVAL, "k = %u exceeds RUDRA_MAX_DSTS", k);
    if (!dsts_dev) return fail(RUDRA_E_INVAL, "null destination list");
    rudra::SnapshotParams p;
    for (uint32_t d = 0; d < k; ++d) {
      if (!aligned(dsts_dev[d])) return fail(RUDRA_E_INVAL, "destination %u is null or not 32-byte aligned", d);
      p.dst[d] = dsts_dev[d];
    }
    p.src = ps->theta;
    p.n = ps->N;
    p.ndst = k;
    p.reverse = ps->sweep++ & 1u;
    DeviceScope dev(ps->device);
    cudaError_t e = rudra::launch_snapshot(p, ps->stream);
    if (e != cudaSuccess) return cuda_fail(e, "snapshot kernel launch");
    ps->counters[2] += k;
    ps->counters[3] += 1;
    ps->counters[6] += k;
    return (int64_t)ps->ts;
  });
}

int64_t rudra_ps_pull(rudra_ps* ps, float* dst_dev) { return rudra_ps_pull_many(ps, &dst_dev, 1); }

int64_t rudra_ps_pull_host(rudra_ps* ps, float* dst_host) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!dst_host) return fail(RUDRA_E_INVAL, "null destination");
    DeviceScope dev(ps->device);
    cudaError_t e = ensure_copy_streams(ps);
    if (e != cudaSuccess) return cuda_fail(e, "copy stream creation");
    constexpr uint32_t kDownBufs = 4;   // snapshots that may be on their way to the host at once
    if (ps->down.size() < kDownBufs) {
      rudra_ps::DownBuf d;
      e = cudaMalloc(reinterpret_cast<void**>(&d.buf), ps->N * sizeof(float));
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&d.filled, cudaEventDisableTiming);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&d.drained, cudaEventDisableTiming);
      if (e != cudaSuccess) {
        cudaFree(d.buf);
        if (d.filled) cudaEventDestroy(d.filled);
        return cuda_fail(e, "snapshot buffer allocation");
      }
      ps->down.push_back(d);
    }
    rudra_ps::DownBuf& d = ps->down[ps->down_next++ % ps->down.size()];
    // snapshot on the main stream (after every update issued so far), then the copy to the host
    // on the download stream, so later updates need not wait for PCIe
    e = cudaStreamWaitEvent(ps->stream, d.drained, 0);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamWaitEvent");
    rudra::SnapshotParams sp;
    sp.dst[0] = d.buf;
    sp.src = ps->theta;
    sp.n = ps->N;
    sp.ndst = 1;
    sp.reverse = ps->sweep++ & 1u;
    e = rudra::launch_snapshot(sp, ps->stream);
    if (e == cudaSuccess) e = cudaEventRecord(d.filled, ps->stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ps->down_stream, d.filled, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(dst_host, d.buf, ps->N * sizeof(float), cudaMemcpyDeviceToHost, ps->down_stream);
    if (e == cudaSuccess) e = cudaEventRecord(d.drained, ps->down_stream);
    if (e != cudaSuccess) return cuda_fail(e, "weights device-to-host copy");
    ps->counters[2] += 1;
    ps->counters[3] += 1;
    ps->counters[5] += ps->N * sizeof(float);
    ps->counters[6] += 1;
    return (int64_t)ps->ts;
  });
}

int64_t rudra_ps_timestamp(const rudra_ps* ps) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    return (int64_t)ps->ts;
  });
}

int rudra_ps_last_clock(const rudra_ps* ps, uint64_t* pulled_ts_out, uint32_t* sigma_out, float* scale_out,
                        double* avg_sigma_out) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    if (!ps->has_clock) return 0;
    for (uint32_t l = 0; l < ps->c; ++l) {
      if (pulled_ts_out) pulled_ts_out[l] = ps->clock[l];
      if (sigma_out) sigma_out[l] = ps->sigma[l];
      if (scale_out) scale_out[l] = ps->scale[l];
    }
    if (avg_sigma_out) *avg_sigma_out = ps->avg_sigma;
    return (int)ps->c;
  });
}

int64_t rudra_ps_clock_log(const rudra_ps* ps, uint64_t first_ts, uint64_t count, uint64_t* pulled_ts_out,
                           double* avg_sigma_out) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    uint64_t got = 0;
    for (; got < count; ++got) {
      const uint64_t t = first_ts + got;
      if (t >= ps->ts || ps->log_ts.empty()) break;
      const size_t pos = (size_t)(t % rudra_ps::kClockLog);
      if (ps->log_ts[pos] != t) {
        if (got == 0) return fail(RUDRA_E_STATE, "update %llu is no longer in the log (the last %u are kept)", (unsigned long long)t, rudra_ps::kClockLog);
        break;
      }
      uint64_t sum = 0;
      for (uint32_t l = 0; l < ps->c; ++l) {
        const uint64_t p = ps->log_pulled[pos * ps->c + l];
        if (pulled_ts_out) pulled_ts_out[got * ps->c + l] = p;
        sum += p;
      }
      if (avg_sigma_out) avg_sigma_out[got] = (double)t - (double)sum / (double)ps->c;
    }
    return (int64_t)got;
  });
}

int64_t rudra_ps_staleness_histogram(const rudra_ps* ps, uint64_t* counts_out, uint32_t nbins) {
  return guarded([&]() -> int64_t {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    for (uint32_t b = 0; b < nbins && counts_out; ++b) counts_out[b] = b < ps->sigma_hist.size() ? ps->sigma_hist[b] : 0;
    return (int64_t)ps->sigma_hist.size();
  });
}

int rudra_ps_export_state(rudra_ps* ps, float* theta_dst_dev, float* state_dst_dev) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    DeviceScope dev(ps->device);
    cudaError_t e = cudaSuccess;
    if (theta_dst_dev) e = cudaMemcpyAsync(theta_dst_dev, ps->theta, ps->N * sizeof(float), cudaMemcpyDeviceToDevice, ps->stream);
    if (e == cudaSuccess && state_dst_dev)
      e = cudaMemcpyAsync(state_dst_dev, ps->state, ps->N * sizeof(float), cudaMemcpyDeviceToDevice, ps->stream);
    if (e != cudaSuccess) return cuda_fail(e, "rudra_ps_export_state");
    return 0;
  });
}

int rudra_ps_import_state(rudra_ps* ps, const float* theta_src_dev, const float* state_src_dev, uint64_t ts) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    DeviceScope dev(ps->device);
    cudaError_t e = cudaSuccess;
    if (theta_src_dev) e = cudaMemcpyAsync(ps->theta, theta_src_dev, ps->N * sizeof(float), cudaMemcpyDeviceToDevice, ps->stream);
    if (e == cudaSuccess && state_src_dev)
      e = cudaMemcpyAsync(ps->state, state_src_dev, ps->N * sizeof(float), cudaMemcpyDeviceToDevice, ps->stream);
    if (e != cudaSuccess) return cuda_fail(e, "rudra_ps_import_state");
    release_queue(ps);
    ps->ts = ts;
    ps->has_clock = false;
    for (auto& v : ps->versions) v.valid = false;
    std::fill(ps->log_ts.begin(), ps->log_ts.end(), ~0ull);
    return 0;
  });
}

int rudra_ps_sync(rudra_ps* ps) {
  return guarded([&]() -> int {
    if (!valid(ps)) return fail(RUDRA_E_INVAL, "bad handle");
    DeviceScope dev(ps->device);
    cudaError_t e = sync_all(ps);
    if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
    return 0;
  });
}

int rudra_ps_counters(const rudra_ps* ps, uint64_t out[8]) {
  return guarded([&]() -> int {
    if (!valid(ps) || !out) return fail(RUDRA_E_INVAL, "bad handle or null output");
    std::memcpy(out, ps->counters, sizeof(ps->counters));
    return 0;
  });
}

}  // extern "C"
