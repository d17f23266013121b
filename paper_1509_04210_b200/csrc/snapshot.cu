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
  const uint64_t tiles = (nunits + kTile - 1) / kTile;
  for (uint64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
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
  }
  const uint64_t k = nunits * kUnit + threadIdx.x;   // the n % 8 trailing weights
  if (blockIdx.x == 0 && k < p.n) {
    const float w = p.src[k];
    for (uint32_t d = 0; d < p.ndst; ++d) p.dst[d][k] = w;
  }
}

}  // namespace

cudaError_t launch_snapshot(const SnapshotParams& p, const LaunchShape& shape, cudaStream_t stream) {
  constexpr int U = 4, THREADS = 256;
  auto kern = snapshot_kernel<U, THREADS>;
  static int cached_blocks_per_sm = 0;
  int per_sm = shape.blocks_per_sm;
  if (per_sm <= 0) {
    if (cached_blocks_per_sm == 0) {
      int b = 0;
      cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, kern, THREADS, 0);
      if (e != cudaSuccess) return e;
      cached_blocks_per_sm = b > 0 ? b : 1;
    }
    per_sm = cached_blocks_per_sm;
  }
  const uint64_t nunits = p.n / kUnit;
  const uint64_t tiles = (nunits + (uint64_t)THREADS * U - 1) / ((uint64_t)THREADS * U);
  uint64_t grid = (uint64_t)shape.sm_count * (uint64_t)per_sm;
  if (tiles < grid) grid = tiles;
  if (grid == 0) grid = 1;
  kern<<<(unsigned)grid, THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace rudra
