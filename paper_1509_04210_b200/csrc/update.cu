// Fused sumGradients + applyUpdate kernel (Section 2; Eq. 5 with the rate of Eq. 6 folded into
// per-gradient step sizes), sm_100a.
//
// The path is element-wise: weight k's new value depends on its own old value, its own state and
// the c gradient values at index k.  So there is no reduction across threads, no shared memory
// and no atomics; the kernel's only job is to keep enough bytes in flight to saturate HBM3e and
// to touch every byte exactly once: c gradient reads, one read and one write of the weights and
// of the state vector, and (optionally) writes of the new weights into learner buffers.  A launch
// can carry a window of several consecutive updates: weights and state then stay in registers
// from one update to the next, and the pulls between them become plain stores.
//
// A thread works on units of 8 consecutive weights.  fp32 vectors move with 256-bit global loads
// and stores (ld/st.global.v8.f32, new with sm_100), bf16 gradients with 128-bit loads, so a
// warp instruction covers 1 KB (fp32) or 512 B (bf16) of contiguous memory.  Gradients are read
// once and never again: they are loaded with an evict-first L2 policy and bypass L1, which leaves
// L2 to the weights and state.  Weights and state are loaded and stored evict-last.
//
// Launch shape: one tile of THREADS * U units per block and as many blocks as tiles, handed out
// by the hardware in index order, so the grid sweeps memory as one moving front (measured ~6 %
// faster on B200 than a persistent grid-stride loop).  Successive launches sweep in alternating
// directions: a launch starts on the tail the previous one just wrote, which is still in the
// 126 MB L2, so those lines are neither re-read from HBM nor written back twice.
#include "kernels.cuh"
#include "vec.cuh"

namespace rudra {
namespace {

constexpr uint64_t kSmallModel = 262144;   // below this many weights the one-weight-per-thread kernel runs

// Tile shape for vectors between kSmallModel and ~4.8 M weights (build-time knobs; the defaults
// are the fastest of a sweep over 32..256 threads and 4..16 loads in flight at 1 M weights).
#ifndef RUDRA_MID_THREADS
#define RUDRA_MID_THREADS 32
#endif
#ifndef RUDRA_MID_DEPTH
#define RUDRA_MID_DEPTH 16
#endif
// Block size and loads in flight of the one-weight-per-thread kernel.
#ifndef RUDRA_SMALL_THREADS
#define RUDRA_SMALL_THREADS 128
#endif
#ifndef RUDRA_SMALL_DEPTH
#define RUDRA_SMALL_DEPTH 8
#endif

// The per-weight rule.  Momentum SGD: u = acc + (sum s) wd theta; v' = m v + u; theta' = theta - v'.
// AdaGrad: g = acc + wd theta (acc already the weighted mean gradient); h' = h + g^2;
// theta' = theta - (sum s) g / (sqrt(h') + eps).
template <int OPT, bool STATE>
__device__ __forceinline__ void apply(const UpdateParams& p, float awd, float abar, float acc, float& theta,
                                      float& state) {
  if (OPT == kMomentumSgd) {
    const float u = fmaf(awd, theta, acc);
    const float v = STATE ? fmaf(p.momentum, state, u) : u;
    theta = theta - v;
    state = v;
  } else {
    const float g = fmaf(p.wd, theta, acc);
    const float h = fmaf(g, g, state);
    theta = theta - __fdiv_rn(abar * g, __fsqrt_rn(h) + p.eps);
    state = h;
  }
}

// A thread's units through the whole window: weights and state are loaded once, carried in
// registers across the nupd updates and stored once; each update streams its own c gradients and
// the pulls that follow it are stores of the registers.  Weights never interact, so this is the
// same arithmetic, in the same order, as nupd separate launches.
//
// The window's nupd * c gradient vectors are walked as one flat list, DEPTH loads in flight at a
// time regardless of where one update ends and the next begins: the loads do not depend on the
// running weights, only the short fma chain does, so a small model (few blocks, latency-bound)
// does not pay one memory round trip per update.
template <typename G, int OPT, bool STATE, int DEPTH, int U, int THREADS, bool GUARD>
__device__ __forceinline__ void process_tile(const UpdateParams& p, uint64_t unit0, uint64_t nunits) {
  F8 th[U], st[U];
  float acc[U][kUnit];
#pragma unroll
  for (int j = 0; j < U; ++j) {
    const uint64_t u = unit0 + (uint64_t)j * THREADS;
    if (!GUARD || u < nunits) {
      th[j] = ld8(p.theta + u * kUnit);
      if (STATE) st[j] = ld8(p.state + u * kUnit);
    }
#pragma unroll
    for (int e = 0; e < kUnit; ++e) acc[j][e] = 0.f;
  }
  uint32_t d = 0;
  for (const uint32_t d1 = p.dst_end[0]; d < d1; ++d) {   // pulls that arrived before the first update
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const uint64_t u = unit0 + (uint64_t)j * THREADS;
      if (!GUARD || u < nunits) st8_stream(p.dst[d] + u * kUnit, th[j]);
    }
  }
  const uint32_t total = p.grad_end[p.nupd];
  uint32_t w = 0;                    // update being accumulated
  uint32_t last = p.grad_end[1];     // one past its last gradient vector
  for (uint32_t l0 = 0; l0 < total; l0 += DEPTH) {
    GradUnit<G> g[DEPTH][U];
#pragma unroll
    for (int i = 0; i < DEPTH; ++i) {
      if (l0 + i < total) {   // uniform across the grid
        const void* base = p.grad[l0 + i];
#pragma unroll
        for (int j = 0; j < U; ++j) {
          const uint64_t u = unit0 + (uint64_t)j * THREADS;
          if (!GUARD || u < nunits) g[i][j].load(base, u); else g[i][j].zero();
        }
      }
    }
#pragma unroll
    for (int i = 0; i < DEPTH; ++i) {
      if (l0 + i < total) {
        const float s = p.scale[l0 + i];
#pragma unroll
        for (int j = 0; j < U; ++j)
#pragma unroll
          for (int e = 0; e < kUnit; ++e) acc[j][e] = fmaf(s, g[i][j].get(e), acc[j][e]);
        if (l0 + i + 1 == last) {   // last gradient of update w: applyUpdate, then the pulls that follow it
          const float awd = p.awd[w], abar = p.abar[w];
#pragma unroll
          for (int j = 0; j < U; ++j)
#pragma unroll
            for (int e = 0; e < kUnit; ++e) {
              float sv = STATE ? st[j].v[e] : 0.f;
              apply<OPT, STATE>(p, awd, abar, acc[j][e], th[j].v[e], sv);
              if (STATE) st[j].v[e] = sv;
              acc[j][e] = 0.f;
            }
          ++w;
          last = p.grad_end[w + 1];   // (the entry after the last update is never compared: the loop ends first)
          for (const uint32_t d1 = p.dst_end[w]; d < d1; ++d) {
#pragma unroll
            for (int j = 0; j < U; ++j) {
              const uint64_t u = unit0 + (uint64_t)j * THREADS;
              if (!GUARD || u < nunits) st8_stream(p.dst[d] + u * kUnit, th[j]);
            }
          }
        }
      }
    }
  }
#pragma unroll
  for (int j = 0; j < U; ++j) {
    const uint64_t u = unit0 + (uint64_t)j * THREADS;
    if (!GUARD || u < nunits) {
      st8(p.theta + u * kUnit, th[j]);
      if (STATE) st8(p.state + u * kUnit, st[j]);
    }
  }
}

// One tile of THREADS * U units per block; the last, ragged tile takes the guarded path and the
// n % 8 trailing weights are done one by one by the block that owns tile 0.
template <typename G, int OPT, bool STATE, int DEPTH, int U, int THREADS>
__global__ void __launch_bounds__(THREADS) update_kernel(const __grid_constant__ UpdateParams p) {
  const uint64_t nunits = p.n / kUnit;
  constexpr uint64_t kTile = (uint64_t)THREADS * U;
  const uint64_t tile = p.reverse ? (uint64_t)gridDim.x - 1 - blockIdx.x : (uint64_t)blockIdx.x;
  if ((tile + 1) * kTile <= nunits)
    process_tile<G, OPT, STATE, DEPTH, U, THREADS, false>(p, tile * kTile + threadIdx.x, nunits);
  else
    process_tile<G, OPT, STATE, DEPTH, U, THREADS, true>(p, tile * kTile + threadIdx.x, nunits);
  const uint64_t k = nunits * kUnit + threadIdx.x;
  if (tile == 0 && k < p.n) {
    float th = p.theta[k];
    float s = STATE ? p.state[k] : 0.f;
    uint32_t d = 0, l = 0;
    for (const uint32_t d1 = p.dst_end[0]; d < d1; ++d) p.dst[d][k] = th;
    for (uint32_t w = 0; w < p.nupd; ++w) {
      float acc = 0.f;
      for (const uint32_t l1 = p.grad_end[w + 1]; l < l1; ++l) acc = fmaf(p.scale[l], GradUnit<G>::scalar(p.grad[l], k), acc);
      apply<OPT, STATE>(p, p.awd[w], p.abar[w], acc, th, s);
      for (const uint32_t d1 = p.dst_end[w + 1]; d < d1; ++d) p.dst[d][k] = th;
    }
    p.theta[k] = th;
    if (STATE) p.state[k] = s;
  }
}

// Small models (a few hundred thousand weights and fewer: the paper's CIFAR10 network has ~90 K)
// are not bandwidth-bound but latency-bound: with 8 weights per thread there are only a handful of
// warps per SM and every instruction's latency shows.  This variant gives every weight its own
// thread (coalesced 4-byte accesses) and keeps DEPTH gradient loads in flight; the arithmetic and
// its order are those of the kernel above.
template <typename G, int OPT, bool STATE, int DEPTH, int THREADS>
__global__ void __launch_bounds__(THREADS) update_kernel_small(const __grid_constant__ UpdateParams p) {
  const uint32_t k = blockIdx.x * THREADS + threadIdx.x;   // fewer than 2^18 weights: 32-bit indexing
  if (k >= (uint32_t)p.n) return;
  float th = p.theta[k];
  float st = STATE ? p.state[k] : 0.f;
  uint32_t d = 0;
  for (const uint32_t d1 = p.dst_end[0]; d < d1; ++d) p.dst[d][k] = th;
  // The vector table is padded to a whole number of chunks (launch_small), so neither the loads nor
  // the fma chain need bounds checks; what a padding entry adds to acc after the last update is
  // never used.
  const uint32_t padded = (p.grad_end[p.nupd] + DEPTH - 1) / DEPTH * DEPTH;
  uint32_t w = 0;
  float acc = 0.f;
  for (uint32_t l0 = 0; l0 < padded; l0 += DEPTH) {
    // the chunk's table entries are fetched together with its gradients, ahead of the dependent chain
    float g[DEPTH], s[DEPTH];
    uint32_t after[DEPTH];
#pragma unroll
    for (int i = 0; i < DEPTH; ++i) {
      g[i] = GradUnit<G>::scalar(p.grad[l0 + i], k);
      s[i] = p.scale[l0 + i];
      after[i] = p.after[l0 + i];
    }
#pragma unroll
    for (int i = 0; i < DEPTH; ++i) {
      acc = fmaf(s[i], g[i], acc);
      const uint32_t pulls = after[i];
      if (pulls != kNotLast) {   // last vector of update w: applyUpdate, then the pulls that follow it
        apply<OPT, STATE>(p, p.awd[w], p.abar[w], acc, th, st);
        acc = 0.f;
        ++w;
        for (const uint32_t d1 = d + pulls; d < d1; ++d) p.dst[d][k] = th;
      }
    }
  }
  p.theta[k] = th;
  if (STATE) p.state[k] = st;
}

template <typename G, int OPT, bool STATE>
cudaError_t launch_small(const UpdateParams& window, cudaStream_t stream) {
  constexpr int THREADS = RUDRA_SMALL_THREADS, DEPTH = RUDRA_SMALL_DEPTH;
  static_assert(kMaxGroup % DEPTH == 0, "the padded vector table must fit");
  UpdateParams p = window;
  const uint32_t total = p.grad_end[p.nupd];
  for (uint32_t l = 0; l < (uint32_t)kMaxGroup; ++l) p.after[l] = kNotLast;
  for (uint32_t u = 0; u < p.nupd; ++u) p.after[p.grad_end[u + 1] - 1] = (uint8_t)(p.dst_end[u + 1] - p.dst_end[u]);
  for (uint32_t l = total; l % DEPTH != 0; ++l) {   // padding: a readable vector, no effect
    p.grad[l] = p.grad[0];
    p.scale[l] = 0.f;
  }
  const uint64_t blocks = (p.n + THREADS - 1) / THREADS;
  update_kernel_small<G, OPT, STATE, DEPTH, THREADS><<<(unsigned)blocks, THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

template <typename G>
cudaError_t launch_small_typed(const UpdateParams& p, Optim optim, cudaStream_t stream) {
  if (optim == kAdagrad) return launch_small<G, kAdagrad, true>(p, stream);
  if (p.momentum != 0.f) return launch_small<G, kMomentumSgd, true>(p, stream);
  return launch_small<G, kMomentumSgd, false>(p, stream);
}

template <typename G, int OPT, bool STATE, int DEPTH, int U, int THREADS>
cudaError_t launch_one(const UpdateParams& p, cudaStream_t stream) {
  const uint64_t nunits = p.n / kUnit;
  uint64_t tiles = (nunits + (uint64_t)THREADS * U - 1) / ((uint64_t)THREADS * U);
  if (tiles == 0) tiles = 1;                                      // n < 8: only the scalar tail
  if (tiles > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
  update_kernel<G, OPT, STATE, DEPTH, U, THREADS><<<(unsigned)tiles, THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

template <typename G, int DEPTH, int THREADS>
cudaError_t launch_typed(const UpdateParams& p, Optim optim, cudaStream_t stream) {
  if (optim == kAdagrad) return launch_one<G, kAdagrad, true, DEPTH, 1, THREADS>(p, stream);
  if (p.momentum != 0.f) return launch_one<G, kMomentumSgd, true, DEPTH, 1, THREADS>(p, stream);
  return launch_one<G, kMomentumSgd, false, DEPTH, 1, THREADS>(p, stream);   // no velocity kept
}

}  // namespace

cudaError_t launch_update(const UpdateParams& p, GradType gtype, Optim optim, int sm_count, cudaStream_t stream) {
  if (p.n < kSmallModel)   // latency-bound: one weight per thread
    return gtype == kBF16 ? launch_small_typed<__nv_bfloat16>(p, optim, stream) : launch_small_typed<float>(p, optim, stream);
  // Large vectors: 256-thread tiles (measured: any tile shape saturates HBM).  Vectors that give
  // fewer than ~16 such tiles per SM are latency-bound or leave the last wave ragged: 64-thread
  // tiles spread them over four times as many blocks.
  const uint64_t sms = sm_count > 0 ? (uint64_t)sm_count : 148;
  const bool small = p.n / kUnit < sms * 16 * 256;
  if (gtype == kBF16)
    return small ? launch_typed<__nv_bfloat16, 8, 64>(p, optim, stream) : launch_typed<__nv_bfloat16, 8, 256>(p, optim, stream);
  return small ? launch_typed<float, RUDRA_MID_DEPTH, RUDRA_MID_THREADS>(p, optim, stream) : launch_typed<float, 4, 256>(p, optim, stream);
}

}  // namespace rudra
