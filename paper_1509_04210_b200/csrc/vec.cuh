// 256-bit global memory accesses and gradient element types shared by the sm_100a kernels.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>

namespace rudra {
namespace {

constexpr int kUnit = 8;   // weights per thread per unit

struct alignas(32) F8 { float v[kUnit]; };

__device__ __forceinline__ F8 ld8(const float* p) {
  F8 r;
  asm volatile("ld.global.L2::evict_last.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=f"(r.v[0]), "=f"(r.v[1]), "=f"(r.v[2]), "=f"(r.v[3]), "=f"(r.v[4]), "=f"(r.v[5]), "=f"(r.v[6]), "=f"(r.v[7])
               : "l"(p));
  return r;
}

__device__ __forceinline__ void st8(float* p, const F8& r) {
  asm volatile("st.global.L2::evict_last.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               :: "l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
               : "memory");
}

// Pull destinations: plain write-back stores (measured 1 % faster on B200 than evict-first or
// evict-last hints when half the traffic of a window is pull writes).
__device__ __forceinline__ void st8_stream(float* p, const F8& r) {
  asm volatile("st.global.v8.f32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
               :: "l"(p), "f"(r.v[0]), "f"(r.v[1]), "f"(r.v[2]), "f"(r.v[3]), "f"(r.v[4]), "f"(r.v[5]), "f"(r.v[6]), "f"(r.v[7])
               : "memory");
}

// One unit of one gradient stream, as loaded (fp32: 8 floats; bf16: 8 halves in 4 words).
template <typename G> struct GradUnit;
template <> struct GradUnit<float> {
  F8 raw;
  __device__ __forceinline__ void load(const void* base, uint64_t unit) {
    const float* p = static_cast<const float*>(base) + unit * kUnit;
    asm volatile("ld.global.L1::no_allocate.L2::evict_first.v8.f32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(raw.v[0]), "=f"(raw.v[1]), "=f"(raw.v[2]), "=f"(raw.v[3]), "=f"(raw.v[4]), "=f"(raw.v[5]), "=f"(raw.v[6]), "=f"(raw.v[7])
                 : "l"(p));
  }
  __device__ __forceinline__ void zero() {
#pragma unroll
    for (int e = 0; e < kUnit; ++e) raw.v[e] = 0.f;
  }
  __device__ __forceinline__ float get(int e) const { return raw.v[e]; }
  static __device__ __forceinline__ float scalar(const void* base, uint64_t k) { return static_cast<const float*>(base)[k]; }
};
template <> struct GradUnit<__nv_bfloat16> {
  uint4 raw;
  __device__ __forceinline__ void load(const void* base, uint64_t unit) {
    raw = __ldcs(static_cast<const uint4*>(base) + unit);
  }
  __device__ __forceinline__ void zero() { raw = make_uint4(0u, 0u, 0u, 0u); }
  // bf16 is the upper half of an fp32: widening is a shift, exact.
  __device__ __forceinline__ float get(int e) const {
    const uint32_t w = e < 2 ? raw.x : e < 4 ? raw.y : e < 6 ? raw.z : raw.w;
    return __uint_as_float((e & 1) ? (w & 0xFFFF0000u) : (w << 16));
  }
  static __device__ __forceinline__ float scalar(const void* base, uint64_t k) {
    return __uint_as_float((uint32_t)static_cast<const uint16_t*>(base)[k] << 16);
  }
};

}  // namespace
}  // namespace rudra
