// Launch interface between the host side of the parameter server and its sm_100a kernels.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace rudra {

constexpr int kMaxGroup = 128;   // RUDRA_MAX_GROUP
constexpr int kMaxDsts = 128;    // RUDRA_MAX_DSTS

enum GradType : int { kF32 = 0, kBF16 = 1 };
enum Optim : int { kMomentumSgd = 0, kAdagrad = 1 };

constexpr int kMaxWindow = 32;   // most updates one launch can carry
constexpr uint8_t kNotLast = 0xFF;

// Everything one launch of the fused kernel needs: a window of nupd consecutive updates (each
// sumGradients + applyUpdate over c gradients) with the pulls that fall between them.  Passed by
// value as a __grid_constant__ kernel parameter: the gradient pointers, step sizes and pull
// destinations form a small table in the constant bank, read with uniform addresses, so a window
// costs one launch and no other stream operation.  Update u uses the vectors
// grad[grad_end[u] .. grad_end[u+1]-1] (c of them when every learner's gradient arrives by itself,
// fewer when leaves of a server tree relay averages); pull destinations
// dst[dst_end[u] .. dst_end[u+1]-1] receive the weights after update u, and dst[0 .. dst_end[0]-1]
// the weights as they were before the window.
struct UpdateParams {
  const void* grad[kMaxGroup];   // the window's gradient vectors, arrival order
  float* dst[kMaxDsts];          // learner buffers, in the order the pulls arrived
  float scale[kMaxGroup];        // step size (momentum SGD) or weight in the mean (AdaGrad), aligned with grad[]
  float awd[kMaxWindow];         // per update, momentum SGD: sum(s) * weight_decay
  float abar[kMaxWindow];        // per update, AdaGrad: sum(s), the group's learning rate
  uint8_t dst_end[kMaxWindow + 1];
  uint8_t grad_end[kMaxWindow + 2];   // grad_end[0] = 0; one spare entry, read but never used, after the last update
  // Filled by launch_update for the one-weight-per-thread kernel: per vector, kNotLast if it is not
  // the last vector of its update, else the number of pull destinations served after that update.
  uint8_t after[kMaxGroup];
  float* theta;
  float* state;                  // velocity (momentum SGD) or sum of squared gradients (AdaGrad)
  uint64_t n;                    // number of weights
  uint32_t nupd;                 // updates in this window (>= 1)
  float momentum;
  float wd;                      // AdaGrad: weight decay
  float eps;                     // AdaGrad: denominator floor
  uint32_t reverse;              // sweep the vector from the end (alternates launch to launch)
};
static_assert(sizeof(UpdateParams) <= 4096, "kernel parameters are limited to 4 KB");
static_assert(kMaxDsts <= 255 && kMaxGroup <= 255, "table indices are stored in bytes");

struct SnapshotParams {
  float* dst[kMaxDsts];
  const float* src;
  uint64_t n;
  uint32_t ndst;
  uint32_t reverse;
};

// Enqueue one window of fused updates (and their pulls) on stream.  Returns the CUDA status of the launch.
// sm_count: multiprocessors of the device the stream belongs to (0 = unknown).
cudaError_t launch_update(const UpdateParams& p, GradType gtype, Optim optim, int sm_count, cudaStream_t stream);

// Enqueue one 1 -> ndst copy of the weights.
cudaError_t launch_snapshot(const SnapshotParams& p, cudaStream_t stream);

// What a leaf of the server tree does (Section 3.3): out[i] = mean of k gradient vectors at i.
struct LeafParams {
  const void* grad[kMaxGroup];
  float* out;
  uint64_t n;
  uint32_t k;
  float inv_k;
};
cudaError_t launch_leaf_average(const LeafParams& p, GradType gtype, cudaStream_t stream);

}  // namespace rudra
