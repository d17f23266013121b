// pullWeights as the server sees it (Section 2, Section 3.2): a copy of the weight vector into
// one or more learner buffers.  One read of the weights serves all ndst destinations, so a
// broadcast to k learners moves 4 + 4k bytes per weight instead of 8k.  256-bit loads and stores,
// no shared memory, no synchronisation.
#include "kernels.cuh"

namespace rudra {
namespace {

constexpr int kUnit = 8;

struct alignas(32) F8 { float v[kUnit]; };

__device__ __forceinline__ F8 ld8(const float* p) {
  F8 r;
  asm volatile("ld.global.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
               : "l"(p));
  return r;
}

__device__ __forceinline__ void st8(float* p, const F8& r) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               :: "l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
               : "memory");
}

template <int U, int THREADS>
__global__ void __launch_bounds__(THREADS) snapshot_kernel(const __grid_constant__ SnapshotParams p) {
  const uint64_t nunits = p.n / kUnit;
  constexpr uint64_t kTile = (uint64_t)THREADS * U;
  const uint64_t tile = p.reverse ? (uint64_t)gridDim.x - 1 - blockIdx.x : (uint64_t)blockIdx.x;
  const uint64_t unit0 = tile * kTile + threadIdx.x;
  F8 w[U];
#pragma unroll
  for (int j = 0; j < U; ++j) {
    const uint64_t u = unit0 + (uint64_t)j * THREADS;
    if (u < nunits) w[j] = ld8(p.src + u * kUnit);
  }
  for (uint32_t d = 0; d < p.ndst; ++d) {
    float* out = p.dst[d];
#pragma unroll
    for (int j = 0; j < U; ++j) {
      const uint64_t u = unit0 + (uint64_t)j * THREADS;
      if (u < nunits) st8(out + u * kUnit, w[j]);
    }
  }
  const uint64_t k = nunits * kUnit + threadIdx.x;   // the n % 8 trailing weights
  if (tile == 0 && k < p.n) {
    const float w1 = p.src[k];
    for (uint32_t d = 0; d < p.ndst; ++d) p.dst[d][k] = w1;
  }
}

}  // namespace

// One tile per block, blocks handed out in index order; direction alternates with the update
// launches so the copy starts on the part of the weights that is still in L2.
cudaError_t launch_snapshot(const SnapshotParams& p, cudaStream_t stream) {
  constexpr int U = 2, THREADS = 256;
  const uint64_t nunits = p.n / kUnit;
  uint64_t tiles = (nunits + (uint64_t)THREADS * U - 1) / ((uint64_t)THREADS * U);
  if (tiles == 0) tiles = 1;
  if (tiles > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
  snapshot_kernel<U, THREADS><<<(unsigned)tiles, THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace rudra
