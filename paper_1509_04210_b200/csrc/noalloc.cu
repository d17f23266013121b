// rudra_ps_update_host_noalloc: the fused update for callers that must not allocate.
//
// Some programs cannot call cudaMalloc once they are running: a serving or training process that
// has handed the whole device to its own memory pool at start-up (a later driver allocation fails
// or fragments the pool), or a control loop that cannot afford the device-wide synchronisation an
// allocation implies.  The regular host-buffer path (rudra_ps_push_host) stages gradients in
// device buffers it allocates on demand.  This entry point does the same work -- copy c host
// gradients to the device, run the fused sumGradients + applyUpdate kernel over them -- but
// stages them in a fixed array that is part of the library image, so it allocates nothing: no
// cudaMalloc, no cudaFree, no allocating library routine.
//
// The price: the array is RUDRA_NOALLOC_MAX_FLOATS floats (16 MiB) on every GPU that loads the
// library, for the life of the process; requests that do not fit are refused; and all calls on a
// device share the one array, so two calls whose device work overlaps (different streams, or
// different host threads) race on it.  Calls ordered on one stream are safe.  The array keeps the
// previous call's gradients; nothing in it has to start at zero, because each call overwrites
// every element it later reads.
#include <cstdint>
#include <cstdio>
#include <mutex>

#include <cuda_runtime.h>

#include "../../include/rudra_ps.h"
#include "kernels.cuh"

// File-scope staging array.  In host code this name is only a stand-in for the device symbol,
// not a device address: the address comes from cudaGetSymbolAddress below.
static __device__ __align__(256) float g_noalloc_scratch[RUDRA_NOALLOC_MAX_FLOATS];

namespace {

constexpr int kMaxDevices = 64;
constexpr uint64_t kSlotAlign = 64;   // floats: every gradient slot starts on a 256-byte boundary

std::mutex g_setup_mutex;
float* g_scratch_addr[kMaxDevices] = {};   // per device, filled on that device's first call

thread_local char g_noalloc_error[256] = "";

// Device address of the staging array on the current device (set-up once per device).
cudaError_t scratch_for_current_device(float** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    float* ptr = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    if (ptr == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" {

const char* rudra_noalloc_last_error(void) { return g_noalloc_error; }

int rudra_ps_update_host_noalloc(float* theta_dev, float* state_dev, uint64_t nparams,
                                 const float* const* grads_host, const float* scales, uint32_t c,
                                 float momentum, float weight_decay, void* cuda_stream) {
  auto fail = [](int code, const char* msg) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error), "%s", msg);
    return code;
  };
  if (!theta_dev || (reinterpret_cast<uintptr_t>(theta_dev) & 31)) return fail(RUDRA_E_INVAL, "theta_dev is null or not 32-byte aligned");
  if (momentum != 0.f && (!state_dev || (reinterpret_cast<uintptr_t>(state_dev) & 31)))
    return fail(RUDRA_E_INVAL, "state_dev is null or not 32-byte aligned");
  if (nparams == 0 || c == 0 || c > RUDRA_MAX_GROUP || !grads_host || !scales) return fail(RUDRA_E_INVAL, "bad nparams, c or null tables");
  if (!(momentum >= 0.f && momentum < 1.f) || !(weight_decay >= 0.f)) return fail(RUDRA_E_INVAL, "bad momentum or weight_decay");
  const uint64_t stride = (nparams + kSlotAlign - 1) / kSlotAlign * kSlotAlign;
  if (stride > RUDRA_NOALLOC_MAX_FLOATS / c) {
    snprintf(g_noalloc_error, sizeof(g_noalloc_error),
             "c * nparams = %u * %llu does not fit the fixed staging array of %llu floats", c,
             (unsigned long long)nparams, (unsigned long long)RUDRA_NOALLOC_MAX_FLOATS);
    return RUDRA_E_INVAL;
  }
  for (uint32_t l = 0; l < c; ++l)
    if (!grads_host[l]) return fail(RUDRA_E_INVAL, "null gradient pointer");

  float* scratch = nullptr;
  cudaError_t e = scratch_for_current_device(&scratch);
  if (e != cudaSuccess) return fail(RUDRA_E_CUDA, cudaGetErrorString(e));
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

  rudra::UpdateParams p;
  double sum_scale = 0.0;
  for (uint32_t l = 0; l < c; ++l) {
    float* slot = scratch + (uint64_t)l * stride;
    e = cudaMemcpyAsync(slot, grads_host[l], nparams * sizeof(float), cudaMemcpyHostToDevice, stream);
    if (e != cudaSuccess) return fail(RUDRA_E_CUDA, cudaGetErrorString(e));
    p.grad[l] = slot;
    p.scale[l] = scales[l];
    sum_scale += (double)scales[l];
  }
  const float abar = (float)sum_scale;
  p.theta = theta_dev;
  p.state = state_dev;
  p.n = nparams;
  p.nupd = 1;
  p.grad_end[0] = 0;
  p.grad_end[1] = p.grad_end[2] = (uint8_t)c;
  p.dst_end[0] = p.dst_end[1] = 0;
  p.momentum = momentum;
  p.awd[0] = (float)((double)abar * (double)weight_decay);
  p.abar[0] = abar;
  p.wd = weight_decay;
  p.eps = 0.f;
  p.reverse = 0;
  e = rudra::launch_update(p, rudra::kF32, rudra::kMomentumSgd, 0, stream);
  if (e != cudaSuccess) return fail(RUDRA_E_CUDA, cudaGetErrorString(e));
  return 0;
}

}  // extern "C"
