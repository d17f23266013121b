// Gradient averaging at a leaf of the server tree (Section 3.3, Rudra-adv): a leaf node sits with
// the learners it is responsible for, averages the gradients they send and relays one vector to
// its parent, so that the root receives 1/k of the traffic.  Element-wise like the update itself:
// k reads (fp32 or bf16) and one fp32 write per weight, 256-bit accesses, no shared memory, no
// synchronisation.  out may live on another GPU (the root's): it is written with plain stores.
//
// out[i] = fma(1/k, g_k[i], ... fma(1/k, g_1[i], 0)) in arrival order, 1/k rounded once to fp32.
#include "kernels.cuh"
#include "vec.cuh"

namespace rudra {
namespace {

template <typename G, int DEPTH, int THREADS>
__global__ void __launch_bounds__(THREADS) leaf_average_kernel(const __grid_constant__ LeafParams p) {
  const uint64_t nunits = p.n / kUnit;
  const uint64_t u = (uint64_t)blockIdx.x * THREADS + threadIdx.x;
  if (u < nunits) {
    F8 acc;
#pragma unroll
    for (int e = 0; e < kUnit; ++e) acc.v[e] = 0.f;
    for (uint32_t l0 = 0; l0 < p.k; l0 += DEPTH) {
      GradUnit<G> g[DEPTH];
#pragma unroll
      for (int i = 0; i < DEPTH; ++i)
        if (l0 + i < p.k) g[i].load(p.grad[l0 + i], u);
#pragma unroll
      for (int i = 0; i < DEPTH; ++i)
        if (l0 + i < p.k)
#pragma unroll
          for (int e = 0; e < kUnit; ++e) acc.v[e] = fmaf(p.inv_k, g[i].get(e), acc.v[e]);
    }
    st8_stream(p.out + u * kUnit, acc);
  }
  const uint64_t i = nunits * kUnit + threadIdx.x;   // the n % 8 trailing weights
  if (blockIdx.x == 0 && i < p.n) {
    float acc = 0.f;
    for (uint32_t l = 0; l < p.k; ++l) acc = fmaf(p.inv_k, GradUnit<G>::scalar(p.grad[l], i), acc);
    p.out[i] = acc;
  }
}

template <typename G, int DEPTH>
cudaError_t launch(const LeafParams& p, cudaStream_t stream) {
  constexpr int THREADS = 256;
  uint64_t blocks = (p.n / kUnit + THREADS - 1) / THREADS;
  if (blocks == 0) blocks = 1;
  if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
  leaf_average_kernel<G, DEPTH, THREADS><<<(unsigned)blocks, THREADS, 0, stream>>>(p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_leaf_average(const LeafParams& p, GradType gtype, cudaStream_t stream) {
  return gtype == kBF16 ? launch<__nv_bfloat16, 8>(p, stream) : launch<float, 4>(p, stream);
}

}  // namespace rudra
