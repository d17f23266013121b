// rudra_stream_probe: a measurement utility (no counterpart in the paper).  It streams nreads
// source vectors and writes nwrites destination vectors with the access shape of the update
// kernel (one 256-thread tile per block, 256-bit accesses, evict-first loads) and no other work,
// so that a benchmark can measure, on the same GPU and in the same run, what HBM delivers for a
// given mix of reads and writes.  On B200 pure reads and pure writes each reach about 7.4 TB/s,
// while any mix of the two lands near 6.7 - 6.9 TB/s: that mixed figure, not the copy bandwidth,
// is the ceiling the update kernel should be judged against.
#include <cstdint>

#include <cuda_runtime.h>

// Built into its own shared object (librudra_probe.so) for the benchmark; it is not part of the
// parameter-server library and not declared in its header.
//
//   int rudra_stream_probe(const float* const* srcs_dev, uint32_t nreads, float* const* dsts_dev,
//                          uint32_t nwrites, uint64_t nfloats, void* cuda_stream);
//
// Enqueues one kernel that reads nreads vectors (host array srcs_dev of device pointers) and
// writes nwrites vectors (dsts_dev; their contents become meaningless), nfloats floats each,
// 32-byte aligned, at most 64 of each.  Returns 0, -1 for bad arguments, -4 if the launch failed.
namespace {

constexpr int kBadArgument = -1, kLaunchFailed = -4;

constexpr int kMaxStreams = 64;

struct ProbeParams {
  const float* src[kMaxStreams];
  float* dst[kMaxStreams];
  uint64_t nunits;
  uint32_t nreads, nwrites;
};

struct alignas(32) F8 { float v[8]; };

__device__ __forceinline__ F8 ld8(const float* p) {
  F8 r;
  asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
               : "l"(p));
  return r;
}

__device__ __forceinline__ void st8(float* p, const F8& r) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               :: "l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
               : "memory");
}

__global__ void __launch_bounds__(256) probe_kernel(const __grid_constant__ ProbeParams p) {
  const uint64_t u = (uint64_t)blockIdx.x * 256 + threadIdx.x;
  if (u >= p.nunits) return;
  F8 acc;
#pragma unroll
  for (int e = 0; e < 8; ++e) acc.v[e] = 1.f;
  for (uint32_t l0 = 0; l0 < p.nreads; l0 += 4) {
    F8 g[4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (l0 + i < p.nreads) g[i] = ld8(p.src[l0 + i] + u * 8);
#pragma unroll
    for (int i = 0; i < 4; ++i)
      if (l0 + i < p.nreads)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc.v[e] = fmaf(0.5f, g[i].v[e], acc.v[e]);
  }
  for (uint32_t d = 0; d < p.nwrites; ++d) st8(p.dst[d] + u * 8, acc);
}

}  // namespace

extern "C" int rudra_stream_probe(const float* const* srcs_dev, uint32_t nreads, float* const* dsts_dev,
                                  uint32_t nwrites, uint64_t nfloats, void* cuda_stream) {
  if (nreads > kMaxStreams || nwrites > kMaxStreams || nreads + nwrites == 0 || nfloats < 8) return kBadArgument;
  if ((nreads && !srcs_dev) || (nwrites && !dsts_dev)) return kBadArgument;
  ProbeParams p;
  for (uint32_t i = 0; i < nreads; ++i) {
    if (!srcs_dev[i] || (reinterpret_cast<uintptr_t>(srcs_dev[i]) & 31)) return kBadArgument;
    p.src[i] = srcs_dev[i];
  }
  for (uint32_t i = 0; i < nwrites; ++i) {
    if (!dsts_dev[i] || (reinterpret_cast<uintptr_t>(dsts_dev[i]) & 31)) return kBadArgument;
    p.dst[i] = dsts_dev[i];
  }
  p.nunits = nfloats / 8;
  p.nreads = nreads;
  p.nwrites = nwrites;
  const uint64_t blocks = (p.nunits + 255) / 256;
  if (blocks > 0x7FFFFFFFull) return kBadArgument;
  probe_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(p);
  return cudaGetLastError() == cudaSuccess ? 0 : kLaunchFailed;
}
